"""Host-side checks of the seeded input generators (no layer arithmetic involved)."""
import numpy as np
import torch

from paper_2503_22673_b200 import inputs


def test_bf16_rounding_matches_torch_rne():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.standard_normal(20000).astype(np.float32) * 3.0,
                        np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895e38, 1e-40, np.inf, -np.inf],
                                 dtype=np.float32)])
    ours = inputs.f32_to_bf16_bits(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(ours, ref)
    back = inputs.bf16_bits_to_f32(ours)
    assert np.array_equal(back, torch.from_numpy(ref.view(np.int16)).view(torch.bfloat16).float().numpy())
    assert inputs.bf16_to_f64(ours).dtype == np.float64


def test_workloads_have_the_stated_shapes_and_statistics():
    (p, t), = list(inputs.draw_workload(0, seed=0))
    assert (p.T, p.d_in, p.d_out, p.r, p.scale) == (256, 512, 512, 8, 2.0)
    assert t["X"].shape == (256, 512) and t["W"].shape == (512, 512)
    assert t["A"].shape == (8, 512) and t["B"].shape == (512, 8) and t["dY"].shape == (256, 512)
    assert all(v.dtype == np.uint16 for v in t.values())
    X, W, B = (inputs.bf16_to_f64(t[k]) for k in ("X", "W", "B"))
    assert abs(X.std() - 1.0) < 0.02
    assert abs(W.std() - 512 ** -0.5) < 0.02 * 512 ** -0.5
    assert abs(B.std() - 0.02 ** 0.5) < 0.05 * 0.02 ** 0.5 and np.count_nonzero(B) > 0
    # same seed -> same bytes; other seed -> other bytes
    (_, t2), = list(inputs.draw_workload(0, seed=0))
    (_, t3), = list(inputs.draw_workload(0, seed=1))
    assert all(np.array_equal(t[k], t2[k]) for k in t)
    assert not np.array_equal(t["X"], t3["X"])


def test_reduced_workloads_keep_their_recipes():
    (p2, t2), = list(inputs.draw_workload(2, T=64))
    x = inputs.bf16_to_f64(t2["X"])
    assert p2.d_out == 14336 and p2.r == 16
    np.testing.assert_allclose(np.sqrt((x ** 2).mean(axis=1)), 1.0, atol=5e-3)      # unit-RMS rows
    assert abs(inputs.bf16_to_f64(t2["dY"]).std() - 0.1) < 0.005
    (p3, t3), = list(inputs.draw_workload(3, T=32))
    x3 = inputs.bf16_to_f64(t3["X"])
    assert p3.d_in == 14336 and p3.r == 64 and p3.scale == 0.5
    assert abs(x3.mean()) < 0.01 and 0.4 < x3.std() < 0.8                            # SiLU(g)*u: centred, O(1)
    projs = list(inputs.draw_workload(4, T=128))
    assert [p.name for p, _ in projs] == ["q_proj", "k_proj", "v_proj", "o_proj", "gate_proj", "up_proj", "down_proj"]
    assert projs[0][1]["X"] is projs[1][1]["X"] is projs[2][1]["X"]                   # q, k, v share X
    assert projs[4][1]["X"] is projs[5][1]["X"] and projs[3][1]["X"] is not projs[0][1]["X"]
    assert not np.array_equal(projs[1][1]["W"], projs[2][1]["W"])


def test_packed_lengths_cover_the_batch():
    lens = inputs.packed_lengths(32768, seed=0)
    assert lens.sum() == 32768 and lens[:-1].min() >= 256 and lens.max() <= 4096
    cu = inputs.cu_seqlens(4, 32768)
    assert cu[0] == 0 and cu[-1] == 32768 and np.all(np.diff(cu) > 0)
    assert list(inputs.cu_seqlens(1, 8192)) == [0, 2048, 4096, 6144, 8192]


def test_flop_count_formula():
    p = inputs.workload(1)[0]
    assert p.flops == 4 * 8192 * 4096 * 4096 + 6 * 8192 * 16 * 8192


def test_paper_setting_workload():
    ps = inputs.workload(5)
    assert [p.name for p in ps] == ["q_proj", "k_proj", "v_proj", "o_proj"]
    assert all(p.T == 49152 and p.r == 32 and p.scale == 2.0 and p.d_in == 4096 for p in ps)
    assert [p.d_out for p in ps] == [4096, 1024, 1024, 4096]
    assert ps[0].x_group == ps[1].x_group == ps[2].x_group != ps[3].x_group
    cs = inputs.cu_seqlens(5, 49152)
    assert cs[0] == 0 and cs[-1] == 49152 and len(cs) == 7 and np.all(np.diff(cs) == 8192)
    small = list(inputs.draw_workload(5, seed=0, T=64))
    assert len(small) == 4 and small[1][1]["X"] is small[0][1]["X"] or np.array_equal(small[1][1]["X"], small[0][1]["X"])
