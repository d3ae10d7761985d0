"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle on the same seeded inputs.

Tolerances (stated for the layer's outputs): max|gpu - ref| / max|ref| <= 2e-2 for the bf16 outputs Y and dX,
<= 5e-3 for the fp32 adapter gradients dA and dB.
"""
import numpy as np
import pytest
import torch

from oracle import lora_oracle as oracle
from paper_2503_22673_b200 import binding, inputs

pytestmark = pytest.mark.gpu

TOL_BF16 = 2e-2
TOL_F32 = 5e-3


def dev(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).cuda()


def host64(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


def guarded(shape, dtype, guard_elems=2048):
    """An output tensor carved out of a larger NaN-poisoned buffer, to catch stray writes."""
    n = int(np.prod(shape))
    buf = torch.full((n + 2 * guard_elems,), float("nan"), dtype=dtype, device="cuda")
    return buf, buf[guard_elems:guard_elems + n].view(*shape)


def guards_intact(buf, n, guard_elems=2048):
    return bool(torch.isnan(buf[:guard_elems]).all() and torch.isnan(buf[guard_elems + n:]).all())


def run_layer(p, t):
    d = {k: dev(v) for k, v in t.items()}
    plan = binding.LoraLinearPlan(p.T, p.d_in, p.d_out, p.r)
    bufs = {}
    out = {}
    for name, shape, dt in (("Y", (p.T, p.d_out), torch.bfloat16), ("dX", (p.T, p.d_in), torch.bfloat16),
                            ("dA", (p.r, p.d_in), torch.float32), ("dB", (p.d_out, p.r), torch.float32)):
        bufs[name], out[name] = guarded(shape, dt)
    plan.fwd(d["X"], d["W"], d["A"], d["B"], p.scale, out["Y"])
    plan.bwd(d["dY"], d["X"], d["W"], d["A"], d["B"], p.scale, out["dX"], out["dA"], out["dB"])
    code, msg = plan.device_status()
    assert code == 0, msg
    for name in out:
        assert guards_intact(bufs[name], out[name].numel()), f"{name}: write outside the tensor"
        assert not torch.isnan(out[name].float()).any(), f"{name}: element left unwritten"
    plan.close()
    return out


def check_full(p, t):
    out = run_layer(p, t)
    f = {k: inputs.bf16_to_f64(v) for k, v in t.items()}
    Y = oracle.forward(f["X"], f["W"], f["A"], f["B"], p.scale)
    dX, dA, dB = oracle.backward(f["dY"], f["X"], f["W"], f["A"], f["B"], p.scale)
    errs = {"Y": oracle.rel_err(host64(out["Y"]), Y), "dX": oracle.rel_err(host64(out["dX"]), dX),
            "dA": oracle.rel_err(host64(out["dA"]), dA), "dB": oracle.rel_err(host64(out["dB"]), dB)}
    assert errs["Y"] <= TOL_BF16 and errs["dX"] <= TOL_BF16, errs
    assert errs["dA"] <= TOL_F32 and errs["dB"] <= TOL_F32, errs
    return out, errs


# ---------------------------------------------------------------------------------------------
# small and ragged shapes, element by element
# ---------------------------------------------------------------------------------------------
SMALL = [
    # T, d_in, d_out, r, scale      (tile rows 128/256; tile columns up to 240; k-blocks of 64; token slabs of 128)
    (1, 8, 8, 8, 2.0),
    (7, 72, 200, 8, 1.7),
    (127, 520, 72, 16, 2.0),
    (129, 200, 520, 24, 0.5),
    (255, 1032, 264, 32, 1.7),
    (257, 264, 1032, 48, 2.0),
    (300, 520, 200, 64, 0.5),
    (640, 768, 1160, 16, 2.0),        # several tiles per row and column, ragged last column tile
    (1000, 2048, 512, 64, 0.5),       # r = 64 with a long contraction
    (2100, 512, 3080, 32, 2.0),       # more tiles than CTAs on a 148-SM part: persistent loop + ragged tail
    (4500, 1024, 4096, 16, 2.0),      # many tiles per persistent CTA
]


@pytest.mark.parametrize("T,d_in,d_out,r,scale", SMALL)
def test_small_shapes_elementwise(T, d_in, d_out, r, scale):
    p, t = inputs.draw_custom(T, d_in, d_out, r, scale, seed=3)
    check_full(p, t)


def test_tiny_workload_config0():
    (p, t), = list(inputs.draw_workload(0, seed=0))
    check_full(p, t)


def test_paper_benchmark_adapter_setting_r32_alpha64():
    # Section 4.5: q/k/v/o adapted with lora_r = 32, alpha = 64 (scale 2); reduced token count
    for d_out in (4096, 1024):
        p, t = inputs.draw_custom(512, 4096, d_out, 32, 2.0, seed=5)
        check_full(p, t)


# ---------------------------------------------------------------------------------------------
# exact cases
# ---------------------------------------------------------------------------------------------
def _pad_example():
    """The hand-derived rank-1 example (tests/golden/rank1_example.txt) zero-padded to the smallest
    shape the kernels take (multiples of 8).  Every value is a small integer: results must be exact."""
    from tests.test_oracle import GOLDEN, _read_golden
    g = _read_golden(GOLDEN)
    T, d_in, d_out, r = 2, 8, 8, 8

    def pad(a, shape):
        out = np.zeros(shape)
        out[:a.shape[0], :a.shape[1]] = a
        return out
    t = {"X": pad(g["X"], (T, d_in)), "W": pad(g["W"], (d_out, d_in)), "A": pad(g["A"], (r, d_in)),
         "B": pad(g["B"], (d_out, r)), "dY": pad(g["dY"], (T, d_out))}
    want = {"Y": pad(g["Y"], (T, d_out)), "dX": pad(g["dX"], (T, d_in)), "dA": pad(g["dA"], (r, d_in)),
            "dB": pad(g["dB"], (d_out, r))}
    return float(g["s"][0, 0]), t, want


def test_hand_derived_example_is_exact_on_gpu():
    s, t, want = _pad_example()
    p = inputs.Projection("rank1", 2, 8, 8, 8, s)
    bits = {k: inputs.f32_to_bf16_bits(v.astype(np.float32)) for k, v in t.items()}
    out = run_layer(p, bits)
    for k in want:
        assert np.array_equal(host64(out[k]), want[k]), k


def test_closed_forms_zero_factors():
    p, t = inputs.draw_custom(300, 264, 200, 16, 2.0, seed=7)
    f = {k: inputs.bf16_to_f64(v) for k, v in t.items()}
    # B = 0: Y = X W^T, dX = dY W, dA = 0 exactly
    tb = dict(t, B=np.zeros_like(t["B"]))
    out = run_layer(p, tb)
    assert torch.count_nonzero(out["dA"]) == 0
    assert oracle.rel_err(host64(out["Y"]), f["X"] @ f["W"].T) <= TOL_BF16
    assert oracle.rel_err(host64(out["dX"]), f["dY"] @ f["W"]) <= TOL_BF16
    _, _, dB = oracle.backward(f["dY"], f["X"], f["W"], f["A"], 0 * f["B"], p.scale)
    assert oracle.rel_err(host64(out["dB"]), dB) <= TOL_F32
    # the adapter path adds exactly +0: Y is bitwise what it is with A = 0 as well
    ta = dict(t, A=np.zeros_like(t["A"]))
    out_a = run_layer(p, ta)
    assert torch.equal(out["Y"].view(torch.int16), out_a["Y"].view(torch.int16))
    assert torch.count_nonzero(out_a["dB"]) == 0
    # W = 0: only the rank-r path is left, at full scale
    tw = dict(t, W=np.zeros_like(t["W"]))
    out_w = run_layer(p, tw)
    assert oracle.rel_err(host64(out_w["Y"]), p.scale * (f["X"] @ f["A"].T) @ f["B"].T) <= TOL_BF16
    assert oracle.rel_err(host64(out_w["dX"]), p.scale * (f["dY"] @ f["B"]) @ f["A"]) <= TOL_BF16


def test_linearity_in_scale():
    p, t = inputs.draw_custom(256, 264, 136, 16, 1.0, seed=9)
    outs = {}
    for s in (0.0, 1.0, 1.7):
        outs[s] = {k: host64(v) for k, v in run_layer(inputs.Projection("lin", 256, 264, 136, 16, s), t).items()}
    assert np.count_nonzero(outs[0.0]["dA"]) == 0 and np.count_nonzero(outs[0.0]["dB"]) == 0
    for k in ("dA", "dB"):
        assert oracle.rel_err(outs[1.7][k], 1.7 * outs[1.0][k]) <= TOL_F32
    for k in ("Y", "dX"):
        lhs = outs[1.7][k] - outs[0.0][k]
        rhs = 1.7 * (outs[1.0][k] - outs[0.0][k])
        assert np.max(np.abs(lhs - rhs)) <= 2 * TOL_BF16 * np.max(np.abs(outs[1.7][k]))


def test_bitwise_reproducible():
    p, t = inputs.draw_custom(1500, 1032, 776, 16, 2.0, seed=11)
    a = run_layer(p, t)
    b = run_layer(p, t)
    for k in a:
        it = torch.int32 if a[k].dtype == torch.float32 else torch.int16
        assert torch.equal(a[k].view(it), b[k].view(it)), k


@pytest.mark.parametrize("merged", ["1", "0"])
def test_stage_entry_points_match_the_single_call(merged, monkeypatch):
    """lora_linear_bwd against the same launches issued one by one through the stage calls (both forms of the backward
    pass: dY B + X A^T | GEMM | dA + dB, and dY B | GEMM | dA | dB): bit-identical."""
    monkeypatch.setenv("LORA_FORCE_BWD_MERGED", merged)
    for T in (700, 100):                                            # CTA pairs; single-CTA GEMM that computes dY B itself
        p, t = inputs.draw_custom(T, 520, 392, 16, 2.0, seed=13)
        d = {k: dev(v) for k, v in t.items()}
        plan = binding.LoraLinearPlan(p.T, p.d_in, p.d_out, p.r)
        assert plan.config()["bwd_merged"] == int(merged)
        assert len(plan.bwd_stage_names()) == (3 if merged == "1" else 4)
        dX1, dA1, dB1 = plan.bwd(d["dY"], d["X"], d["W"], d["A"], d["B"], p.scale)
        dX2, dA2, dB2 = torch.empty_like(dX1), torch.empty_like(dA1), torch.empty_like(dB1)
        plan.bwd_stages(d["dY"], d["X"], d["W"], d["A"], d["B"], p.scale, dX2, dA2, dB2)
        torch.cuda.synchronize()
        assert torch.equal(dX1.view(torch.int16), dX2.view(torch.int16))
        assert torch.equal(dA1, dA2) and torch.equal(dB1, dB2)
        f = {k: inputs.bf16_to_f64(v) for k, v in t.items()}
        dXr, dAr, dBr = oracle.backward(f["dY"], f["X"], f["W"], f["A"], f["B"], p.scale)
        assert oracle.rel_err(host64(dX2), dXr) <= TOL_BF16
        assert oracle.rel_err(host64(dA2), dAr) <= TOL_F32 and oracle.rel_err(host64(dB2), dBr) <= TOL_F32
        plan.close()


# ---------------------------------------------------------------------------------------------
# argument handling on a device
# ---------------------------------------------------------------------------------------------
def test_empty_batch_and_argument_errors():
    plan = binding.LoraLinearPlan(0, 64, 72, 16)
    bf = torch.bfloat16
    X = torch.empty(0, 64, dtype=bf, device="cuda")
    W = torch.zeros(72, 64, dtype=bf, device="cuda")
    A = torch.zeros(16, 64, dtype=bf, device="cuda")
    B = torch.zeros(72, 16, dtype=bf, device="cuda")
    dY = torch.empty(0, 72, dtype=bf, device="cuda")
    assert plan.fwd(X, W, A, B, 2.0).shape == (0, 72)
    dX, dA, dB = plan.bwd(dY, X, W, A, B, 2.0,
                          dA=torch.full((16, 64), 3.0, device="cuda"), dB=torch.full((72, 16), 3.0, device="cuda"))
    torch.cuda.synchronize()
    assert torch.count_nonzero(dA) == 0 and torch.count_nonzero(dB) == 0
    plan.close()

    plan = binding.LoraLinearPlan(128, 64, 72, 16)
    X = torch.zeros(128, 64, dtype=bf, device="cuda")
    dY = torch.zeros(128, 72, dtype=bf, device="cuda")
    lib = binding.load()
    Y = torch.zeros(128 * 72 + 8, dtype=bf, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    # misaligned output pointer
    rc = lib.lora_linear_fwd(plan._h, X.data_ptr(), W.data_ptr(), A.data_ptr(), B.data_ptr(), 2.0, Y.data_ptr() + 2, stream)
    assert rc == binding.LORA_ERR_MISALIGNED
    rc = lib.lora_linear_fwd(plan._h, X.data_ptr(), None, A.data_ptr(), B.data_ptr(), 2.0, Y.data_ptr(), stream)
    assert rc == binding.LORA_ERR_INVALID_ARG
    # backward without a workspace
    dXb = torch.zeros(128, 64, dtype=bf, device="cuda")
    dAb = torch.zeros(16, 64, device="cuda")
    dBb = torch.zeros(72, 16, device="cuda")
    rc = lib.lora_linear_bwd(plan._h, dY.data_ptr(), X.data_ptr(), W.data_ptr(), A.data_ptr(), B.data_ptr(), 2.0,
                             dXb.data_ptr(), dAb.data_ptr(), dBb.data_ptr(), stream)
    assert rc == binding.LORA_ERR_WORKSPACE
    small = torch.zeros(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.LoraError) as ei:
        plan.set_workspace(small)
    assert ei.value.code == binding.LORA_ERR_WORKSPACE
    assert "T=128" in plan.describe()
    assert plan.device_status()[0] == 0
    plan.close()


def test_host_buffer_step_matches_device_calls():
    p, t = inputs.draw_custom(384, 264, 200, 16, 2.0, seed=17)
    d = {k: dev(v) for k, v in t.items()}
    plan = binding.LoraLinearPlan(p.T, p.d_in, p.d_out, p.r)
    Y = plan.fwd(d["X"], d["W"], d["A"], d["B"], p.scale)
    dX, dA, dB = plan.bwd(d["dY"], d["X"], d["W"], d["A"], d["B"], p.scale)
    h = {k: d[k].cpu().pin_memory() for k in ("X", "A", "B", "dY")}
    hY, hdX = torch.empty_like(Y, device="cpu").pin_memory(), torch.empty_like(dX, device="cpu").pin_memory()
    hdA, hdB = torch.empty_like(dA, device="cpu").pin_memory(), torch.empty_like(dB, device="cpu").pin_memory()
    staging = torch.empty(plan.step_host_staging_bytes(), dtype=torch.uint8, device="cuda")
    plan.step_host(h["X"], d["W"], h["A"], h["B"], h["dY"], p.scale, hY, hdX, hdA, hdB, staging)
    torch.cuda.synchronize()
    assert torch.equal(hY.view(torch.int16), Y.cpu().view(torch.int16))
    assert torch.equal(hdX.view(torch.int16), dX.cpu().view(torch.int16))
    assert torch.equal(hdA, dA.cpu()) and torch.equal(hdB, dB.cpu())
    plan.close()


def test_backward_with_saved_forward_product_matches_oracle():
    """lora_linear_bwd_saved_p reuses X A^T of the preceding forward; it must meet the same tolerances."""
    for (T, d_in, d_out, r, scale) in [(700, 520, 392, 16, 2.0), (1300, 1032, 2056, 64, 0.5), (129, 264, 136, 8, 1.7)]:
        p, t = inputs.draw_custom(T, d_in, d_out, r, scale, seed=19)
        d = {k: dev(v) for k, v in t.items()}
        f = {k: inputs.bf16_to_f64(v) for k, v in t.items()}
        plan = binding.LoraLinearPlan(T, d_in, d_out, r)
        lib = binding.load()
        dX, dA, dB = (torch.full((T, d_in), float("nan"), dtype=torch.bfloat16, device="cuda"),
                      torch.full((r, d_in), float("nan"), device="cuda"), torch.full((d_out, r), float("nan"), device="cuda"))
        # without a forward on a registered workspace there is nothing to reuse
        plan.ensure_workspace()
        with pytest.raises(binding.LoraError):
            plan.bwd(d["dY"], d["X"], d["W"], d["A"], d["B"], scale, dX, dA, dB, saved_p=True)
        Y = plan.fwd(d["X"], d["W"], d["A"], d["B"], scale)
        with pytest.raises(binding.LoraError):                      # other scale than the forward's
            plan.bwd(d["dY"], d["X"], d["W"], d["A"], d["B"], scale + 1.0, dX, dA, dB, saved_p=True)
        plan.bwd(d["dY"], d["X"], d["W"], d["A"], d["B"], scale, dX, dA, dB, saved_p=True)
        assert plan.device_status()[0] == 0
        dXr, dAr, dBr = oracle.backward(f["dY"], f["X"], f["W"], f["A"], f["B"], scale)
        assert oracle.rel_err(host64(Y), oracle.forward(f["X"], f["W"], f["A"], f["B"], scale)) <= TOL_BF16
        assert oracle.rel_err(host64(dX), dXr) <= TOL_BF16
        assert oracle.rel_err(host64(dA), dAr) <= TOL_F32 and oracle.rel_err(host64(dB), dBr) <= TOL_F32
        plan.close()


@pytest.mark.parametrize("T,d_in,d_outs,r,scale", [
    (900, 520, [768, 256, 256], 16, 2.0),          # q/k/v style, r = 16: one 48-row side job, one dA job
    (1300, 1032, [512, 256, 256], 32, 2.0),        # the paper's adapter rank (Section 4.5): 96 adapter rows -> two X jobs
    (700, 264, [768, 768], 64, 0.5),               # gate/up style at the largest rank
    (2100, 512, [256, 512, 256, 256], 16, 1.7),    # four groups, more tiles than CTA pairs per group
])
def test_grouped_projections_sharing_x_match_separate_oracles(T, d_in, d_outs, r, scale):
    """lora_linear_fwd_grouped / lora_linear_bwd_grouped: every projection of the group must match ITS OWN oracle, and dX
    the sum of the groups' oracles' dX."""
    from paper_2503_22673_b200.grouped import GroupedLoraPlan
    projs = [inputs.draw_custom(T, d_in, d, r, scale, seed=30 + g, tag=70 + g) for g, d in enumerate(d_outs)]
    X_bits = projs[0][1]["X"]
    f64 = lambda b: inputs.bf16_to_f64(b)
    gp = GroupedLoraPlan(T, d_in, d_outs, r)
    W, A, B = gp.pack([dev(t["W"]) for _, t in projs], [dev(t["A"]) for _, t in projs], [dev(t["B"]) for _, t in projs])
    X = dev(X_bits)
    dY = torch.cat([dev(t["dY"]) for _, t in projs], dim=1).contiguous()
    bufs = {}
    out = {}
    D = sum(d_outs)
    for name, shape, dt in (("Y", (T, D), torch.bfloat16), ("dX", (T, d_in), torch.bfloat16),
                            ("dA", (len(d_outs) * r, d_in), torch.float32), ("dB", (D, r), torch.float32)):
        bufs[name], out[name] = guarded(shape, dt)
    for rep in range(2):                                   # twice: the arrival counters must be back at zero
        Y = gp.fwd(X, W, A, B, scale, out["Y"])
        dX, dAs, dBs = gp.bwd(dY, X, W, A, B, scale, out["dX"], out["dA"], out["dB"])
        code, msg = gp.device_status()
        assert code == 0, msg
        for name in out:
            assert guards_intact(bufs[name], out[name].numel()), f"{name}: write outside the tensor"
            assert not torch.isnan(out[name].float()).any(), f"{name}: element left unwritten"
        dX_ref = 0.0
        for g, (p, t) in enumerate(projs):
            Wg, Ag, Bg, dYg = f64(t["W"]), f64(t["A"]), f64(t["B"]), f64(t["dY"])
            Yr = oracle.forward(f64(X_bits), Wg, Ag, Bg, scale)
            dXr, dAr, dBr = oracle.backward(dYg, f64(X_bits), Wg, Ag, Bg, scale)
            dX_ref = dX_ref + dXr
            assert oracle.rel_err(host64(gp.split_outputs(Y)[g]), Yr) <= TOL_BF16, (g, rep)
            assert oracle.rel_err(host64(dAs[g]), dAr) <= TOL_F32, (g, rep)
            assert oracle.rel_err(host64(dBs[g]), dBr) <= TOL_F32, (g, rep)
        assert oracle.rel_err(host64(dX), dX_ref) <= TOL_BF16
    gp.close()


def test_grouped_plan_rejects_what_it_does_not_cover():
    from paper_2503_22673_b200.grouped import GroupedLoraPlan
    for args in ((900, 520, [768, 200], 16), (900, 520, [768, 256], 24), (100, 520, [768, 256], 16), (900, 520, [256] * 4, 64)):
        with pytest.raises(binding.LoraError) as e:
            GroupedLoraPlan(*args)
        assert e.value.code == binding.LORA_ERR_UNSUPPORTED_SHAPE, args
    gp = GroupedLoraPlan(900, 520, [768, 256], 16)
    plain = binding.LoraLinearPlan(900, 520, 1024, 16)
    X = torch.zeros((900, 520), dtype=torch.bfloat16, device="cuda")
    W = torch.zeros((1024, 520), dtype=torch.bfloat16, device="cuda")
    A = torch.zeros((16, 520), dtype=torch.bfloat16, device="cuda")
    B = torch.zeros((1024, 16), dtype=torch.bfloat16, device="cuda")
    Y = torch.zeros((900, 1024), dtype=torch.bfloat16, device="cuda")
    lib = binding.load()
    sp = torch.cuda.current_stream().cuda_stream
    assert lib.lora_linear_fwd(gp._h, X.data_ptr(), W.data_ptr(), A.data_ptr(), B.data_ptr(), 1.0, Y.data_ptr(), sp) == binding.LORA_ERR_INVALID_ARG
    assert lib.lora_linear_fwd_grouped(plain._h, X.data_ptr(), W.data_ptr(), A.data_ptr(), B.data_ptr(), 1.0, Y.data_ptr(), sp) == binding.LORA_ERR_INVALID_ARG
    gp.close()
    plain.close()


def test_split_k_paths_match_oracle(monkeypatch):
    """Grids that cannot fill the GPU are split along K (fp32 partial tiles + fixed-order reduce).  One shape takes the
    split by the selector's own rule; the others force it (3 splits) on ragged shapes, forward and dX."""
    p, t = inputs.draw_custom(257, 14336, 264, 64, 0.5, seed=23)
    cfg = binding.select_config(p.T, p.d_in, p.d_out, p.r)
    assert cfg["split_k"] > 1 and cfg["fwd_ext"] == 1
    check_full(p, t)
    monkeypatch.setenv("LORA_FORCE_SPLIT_K", "3")
    for shape in [(700, 520, 392, 16, 2.0), (300, 2048, 1032, 24, 1.7)]:
        p, t = inputs.draw_custom(*shape, seed=24)
        a, _ = check_full(p, t)
        b, _ = check_full(p, t)
        for k in a:                                   # still bitwise reproducible
            it = torch.int32 if a[k].dtype == torch.float32 else torch.int16
            assert torch.equal(a[k].view(it), b[k].view(it)), k


@pytest.mark.parametrize("force", ["0", "1"])
def test_both_forms_of_the_x_a_product_in_backward(force, monkeypatch):
    """Backward recomputes X A^T either inside the dA launch (default up to rank 32) or in its own skinny pass over X
    (default for larger ranks); both forms, forced here at r = 16 and r = 64, against the oracle."""
    monkeypatch.setenv("LORA_FORCE_DA_WITH_P", force)
    monkeypatch.setenv("LORA_FORCE_BWD_MERGED", "0")              # the split form: dY B | GEMM | dA | dB
    for T, d_in, d_out, r, s in ((4096, 2048, 2304, 16, 2.0), (1500, 1032, 520, 64, 0.5)):
        p, t = inputs.draw_custom(T, d_in, d_out, r, s, seed=12)
        plan_cfg = binding.select_config(T, d_in, d_out, r, 148)
        assert plan_cfg["da_with_p"] == int(force)
        check_full(p, t)


def test_staged_pre_pass_is_used_once_and_discarded_by_other_calls():
    """lora_linear_bwd_q stages s (dY B)^T for the NEXT lora_linear_bwd_dx only: with the matching dY the staged GEMM gives
    the same bits as the unstaged call, and a full backward in between (other dY) makes a later bwd_dx run its own pre-pass."""
    p, t = inputs.draw_custom(520, 264, 776, 16, 2.0, seed=21)
    _, t2 = inputs.draw_custom(520, 264, 776, 16, 2.0, seed=22)
    d = {k: dev(v) for k, v in t.items()}
    dY2 = dev(t2["dY"])
    plan = binding.LoraLinearPlan(p.T, p.d_in, p.d_out, p.r)
    ref = plan.bwd_dx(d["dY"], d["W"], d["A"], d["B"], p.scale, torch.empty_like(d["X"])).clone()
    plan.bwd_q(d["dY"], d["B"], p.scale)
    staged = plan.bwd_dx(d["dY"], d["W"], d["A"], d["B"], p.scale, torch.empty_like(d["X"]))
    assert torch.equal(staged, ref)
    plan.bwd_q(dY2, d["B"], p.scale)                                   # staged for dY2 ...
    plan.bwd(dY2, d["X"], d["W"], d["A"], d["B"], p.scale)             # ... but a full backward comes first
    again = plan.bwd_dx(d["dY"], d["W"], d["A"], d["B"], p.scale, torch.empty_like(d["X"]))
    assert torch.equal(again, ref)
    code, msg = plan.device_status()
    assert code == 0, msg
    plan.close()


@pytest.mark.parametrize("T1,T2,d_in,d_out,r", [(300, 212, 264, 520, 16),        # tiny: the streaming kernels write dA / dB themselves
                                                 (4096, 2100, 1024, 1160, 32)])   # partial sums + finalize kernel
def test_gradient_accumulation_over_micro_batches(T1, T2, d_in, d_out, r):
    """With lora_plan_set_grad_accumulation the backward calls add into dA / dB: two micro-batches give the gradients of the
    concatenated batch (the sums over token rows are additive), dX stays per micro-batch."""
    scale = 2.0
    p, t = inputs.draw_custom(T1 + T2, d_in, d_out, r, scale, seed=31)
    d = {k: dev(v) for k, v in t.items()}
    dA = torch.zeros((r, d_in), dtype=torch.float32, device="cuda")
    dB = torch.zeros((d_out, r), dtype=torch.float32, device="cuda")
    dX = torch.empty((T1 + T2, d_in), dtype=torch.bfloat16, device="cuda")
    for lo, hi in ((0, T1), (T1, T1 + T2)):
        plan = binding.LoraLinearPlan(hi - lo, d_in, d_out, r)
        plan.set_grad_accumulation(True)
        plan.bwd(d["dY"][lo:hi], d["X"][lo:hi], d["W"], d["A"], d["B"], scale, dX[lo:hi], dA, dB)
        code, msg = plan.device_status()
        assert code == 0, msg
        plan.close()
    f = {k: inputs.bf16_to_f64(v) for k, v in t.items()}
    dXr, dAr, dBr = oracle.backward(f["dY"], f["X"], f["W"], f["A"], f["B"], scale)
    assert oracle.rel_err(host64(dX), dXr) <= TOL_BF16
    assert oracle.rel_err(host64(dA), dAr) <= TOL_F32 and oracle.rel_err(host64(dB), dBr) <= TOL_F32
    # switched off again, the same call overwrites
    plan = binding.LoraLinearPlan(T2, d_in, d_out, r)
    plan.bwd(d["dY"][T1:], d["X"][T1:], d["W"], d["A"], d["B"], scale, dX[T1:], dA, dB)
    _, dA2, dB2 = oracle.backward(f["dY"][T1:], f["X"][T1:], f["W"], f["A"], f["B"], scale)
    assert oracle.rel_err(host64(dA), dA2) <= TOL_F32 and oracle.rel_err(host64(dB), dB2) <= TOL_F32
    plan.close()
