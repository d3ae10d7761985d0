"""GPU parity of the dense weight gradient dW = dY^T X (full fine-tuning, Section 4.5 "Full-model tuning")
against the CPU oracle, through the C ABI (lora_dense_dw).

dW is a bf16 output: max|gpu - ref| / max|ref| <= 2e-2, the layer's tolerance for bf16 outputs.
"""
import numpy as np
import pytest
import torch

from oracle import lora_oracle as oracle
from paper_2503_22673_b200 import binding, inputs
from tests.test_parity_gpu import dev, guarded, guards_intact, host64

pytestmark = pytest.mark.gpu

TOL_BF16 = 2e-2


def run_dw(p, t, force_split=None):
    d = {k: dev(t[k]) for k in ("X", "dY")}
    plan = binding.LoraLinearPlan(p.T, p.d_in, p.d_out, p.r)
    buf, dW = guarded((p.d_out, p.d_in), torch.bfloat16)
    plan.dense_dw(d["dY"], d["X"], dW)
    code, msg = plan.device_status()
    assert code == 0, msg
    assert guards_intact(buf, dW.numel()), "dW: write outside the tensor"
    assert not torch.isnan(dW.float()).any(), "dW: element left unwritten"
    cfg = plan.config()
    plan.close()
    return dW, cfg


SHAPES = [
    # T, d_in, d_out          (tiles: 256 rows of d_out x up to 256 columns of d_in; k-blocks of 64 tokens)
    (1, 8, 8),
    (63, 72, 200),
    (64, 264, 520),
    (129, 1032, 264),
    (1000, 520, 1160),         # ragged in all three dimensions
    (4100, 2048, 512),         # long contraction, ragged last k-block
    (640, 3080, 2056),         # more tiles than CTA pairs: persistent loop
    (20000, 256, 264),         # few tiles, many tokens: the contraction is split
]


@pytest.mark.parametrize("T,d_in,d_out", SHAPES)
def test_dense_dw_elementwise(T, d_in, d_out):
    p, t = inputs.draw_custom(T, d_in, d_out, 8, 1.0, seed=11)
    dW, cfg = run_dw(p, t)
    ref = oracle.dense_weight_grad(inputs.bf16_to_f64(t["dY"]), inputs.bf16_to_f64(t["X"]))
    err = oracle.rel_err(host64(dW), ref)
    assert err <= TOL_BF16, (err, cfg)


def test_dense_dw_split_is_selected_for_few_tiles():
    assert binding.select_config(20000, 256, 264, 8)["dw_split_k"] > 1
    assert binding.select_config(8192, 4096, 4096, 16)["dw_split_k"] == 1


def test_dense_dw_hand_example_is_exact():
    """The worked example of tests/golden/dense_dw_example.txt, zero-padded to multiples of 8: small integers, exact."""
    import os
    from tests.test_oracle import _read_golden
    g = _read_golden(os.path.join(os.path.dirname(__file__), "golden", "dense_dw_example.txt"))
    X = np.zeros((3, 8))
    dY = np.zeros((3, 8))
    X[:, :2], dY[:, :3] = g["X"], g["dY"]
    plan = binding.LoraLinearPlan(3, 8, 8, 8)
    dW = plan.dense_dw(torch.tensor(dY, dtype=torch.bfloat16).cuda(), torch.tensor(X, dtype=torch.bfloat16).cuda())
    got = host64(dW)
    plan.close()
    assert np.array_equal(got[:3, :2], g["dW"])
    assert np.all(got[3:] == 0) and np.all(got[:, 2:] == 0)


def test_dense_dw_empty_batch_and_reproducible():
    plan = binding.LoraLinearPlan(0, 64, 72, 8)
    dW = torch.full((72, 64), float("nan"), dtype=torch.bfloat16, device="cuda")
    plan.dense_dw(torch.empty((0, 72), dtype=torch.bfloat16, device="cuda"),
                  torch.empty((0, 64), dtype=torch.bfloat16, device="cuda"), dW)
    torch.cuda.synchronize()
    assert torch.all(dW == 0)
    plan.close()
    p, t = inputs.draw_custom(3000, 520, 776, 8, 1.0, seed=2)
    a, _ = run_dw(p, t)
    b, _ = run_dw(p, t)
    assert torch.equal(a, b)


def test_dense_dw_projects_onto_adapter_gradients():
    """dA = s B^T dW and dB = s dW A^T: the layer's own fp32 adapter gradients agree with projections of the GPU's dW
    (fp64 on the host) within the bf16 tolerance of dW."""
    p, t = inputs.draw_custom(2048, 1024, 768, 16, 2.0, seed=9)
    dW, _ = run_dw(p, t)
    f = {k: inputs.bf16_to_f64(v) for k, v in t.items()}
    dA, dB = oracle.backward_adapter_grads(f["dY"], f["X"], f["A"], f["B"], p.scale)
    W64 = host64(dW)
    assert oracle.rel_err(p.scale * f["B"].T @ W64, dA) <= TOL_BF16
    assert oracle.rel_err(p.scale * W64 @ f["A"].T, dB) <= TOL_BF16
