"""GPU parity on seeded random shapes: every entry point of the layer (forward, backward, saved-P backward, dense dW, and
the NF4 forms where d_in allows) against the CPU oracle, element by element, on shapes drawn around the tile, slab and
k-block borders (token counts next to multiples of 128 and 256, feature counts any multiple of 8, every rank from 8 to 64).

Tolerances as everywhere: max|gpu - ref| / max|ref| <= 2e-2 for bf16 outputs, <= 5e-3 for the fp32 dA / dB."""
import random

import numpy as np
import pytest
import torch

from oracle import lora_oracle as oracle
from oracle import nf4_oracle as nf4
from paper_2503_22673_b200 import binding, inputs
from tests.test_parity_gpu import dev, host64

pytestmark = pytest.mark.gpu

TOL_BF16 = 2e-2
TOL_F32 = 5e-3


def _shapes(seed, n):
    rng = random.Random(seed)
    out = []
    for _ in range(n):
        T = rng.choice([1, 5, 64, 127, 128, 129, 200, 255, 256, 257, 300, 511, 513, 700, 1000, 1500, 2049, 3000])
        d_in, d_out = 8 * rng.randint(1, 300), 8 * rng.randint(1, 300)
        if rng.random() < 0.35:
            d_in = 64 * rng.randint(1, 40)                    # NF4 needs whole 64-element blocks
        out.append((T, d_in, d_out, rng.choice([8, 16, 24, 32, 40, 48, 56, 64]), rng.choice([0.5, 1.0, 1.7, 2.0])))
    return out


@pytest.mark.parametrize("T,d_in,d_out,r,scale", _shapes(2503, 24))
def test_random_shape_all_entry_points(T, d_in, d_out, r, scale):
    p, t = inputs.draw_custom(T, d_in, d_out, r, scale, seed=T + d_in + d_out + r)
    d = {k: dev(v) for k, v in t.items()}
    f = {k: inputs.bf16_to_f64(v) for k, v in t.items()}
    plan = binding.LoraLinearPlan(T, d_in, d_out, r)
    plan.ensure_workspace()
    got = {"Y": plan.fwd(d["X"], d["W"], d["A"], d["B"], scale)}
    got["dX"], got["dA"], got["dB"] = plan.bwd(d["dY"], d["X"], d["W"], d["A"], d["B"], scale)
    plan.fwd(d["X"], d["W"], d["A"], d["B"], scale)
    got["dX_saved"], got["dA_saved"], got["dB_saved"] = plan.bwd(d["dY"], d["X"], d["W"], d["A"], d["B"], scale, saved_p=True)
    got["dW"] = plan.dense_dw(d["dY"], d["X"])
    ref = {"Y": oracle.forward(f["X"], f["W"], f["A"], f["B"], scale), "dW": oracle.dense_weight_grad(f["dY"], f["X"])}
    ref["dX"], ref["dA"], ref["dB"] = oracle.backward(f["dY"], f["X"], f["W"], f["A"], f["B"], scale)
    ref["dX_saved"], ref["dA_saved"], ref["dB_saved"] = ref["dX"], ref["dA"], ref["dB"]
    if d_in % 64 == 0 and d_out % 4 == 0:
        codes, absmax = nf4.quantize(f["W"].astype(np.float32))
        cd, ad = torch.from_numpy(codes).cuda(), torch.from_numpy(absmax).cuda()
        ref["Y_nf4"] = nf4.forward(f["X"], codes, absmax, f["A"], f["B"], scale)
        ref["dX_nf4"] = nf4.backward(f["dY"], f["X"], codes, absmax, f["A"], f["B"], scale)[0]
        scratch = torch.empty((d_out, d_in), dtype=torch.bfloat16, device="cuda")
        got["Y_nf4"] = plan.fwd_nf4(d["X"], cd, ad, d["A"], d["B"], scale, w_scratch=scratch)
        got["dX_nf4"] = plan.bwd_nf4(d["dY"], d["X"], cd, ad, d["A"], d["B"], scale, w_scratch=scratch)[0]
        if T > 128:                                              # in-kernel form
            ref["Y_nf4_in_kernel"], ref["dX_nf4_in_kernel"] = ref["Y_nf4"], ref["dX_nf4"]
            got["Y_nf4_in_kernel"] = plan.fwd_nf4(d["X"], cd, ad, d["A"], d["B"], scale)
            got["dX_nf4_in_kernel"] = plan.bwd_nf4(d["dY"], d["X"], cd, ad, d["A"], d["B"], scale)[0]
    code, msg = plan.device_status()
    plan.close()
    assert code == 0, msg
    errs = {k: oracle.rel_err(host64(got[k]), ref[k]) for k in ref}
    for k, e in errs.items():
        tol = TOL_F32 if k.startswith(("dA", "dB")) else TOL_BF16
        assert e <= tol, (k, errs)
