"""GPU parity of the quantised-LoRA path (Section 4.5, Q+LoRA): NF4 quantiser bit-exact against the oracle's, and the
layer with the NF4 weight against the oracle on the same codes and scales, through the C ABI.

Tolerances as for the bf16 layer: max|gpu - ref| / max|ref| <= 2e-2 (Y, dX), <= 5e-3 (dA, dB).  Codes and scales are
integer / exact float32 decisions and must match bit for bit."""
import os

import numpy as np
import pytest
import torch

from oracle import nf4_oracle as nf4
from oracle import lora_oracle as oracle
from paper_2503_22673_b200 import binding, inputs
from tests.test_parity_gpu import dev, guarded, guards_intact, host64

pytestmark = pytest.mark.gpu

TOL_BF16 = 2e-2
TOL_F32 = 5e-3


def _bf16_weight(d_out, d_in, seed):
    p, t = inputs.draw_custom(8, d_in, d_out, 8, 1.0, seed=seed)
    return t["W"]                                              # bf16 bit patterns, W ~ N(0, 1/d_in)


@pytest.mark.parametrize("d_out,d_in", [(4, 64), (72, 192), (1000, 1024), (4096, 4096)])
def test_quantiser_is_bit_exact(d_out, d_in):
    bits = _bf16_weight(d_out, d_in, seed=d_out)
    W = inputs.bf16_to_f64(bits).astype(np.float32)
    W[0, :64] = 0.0                                            # an all-zero block
    if d_in >= 128:
        mids = nf4.midpoints()
        W[1 % d_out, 64] = 1.0                                 # absmax 1 in that block (bf16-exact), then values on / next to midpoints
        W[1 % d_out, 65:80] = 0.0
    Wt = torch.tensor(W).to(torch.bfloat16)                    # exact: every value is already bf16 (or 0 / 1)
    W = Wt.float().numpy()
    codes, absmax = binding.nf4_quantize(Wt.cuda().contiguous())
    torch.cuda.synchronize()
    ref_codes, ref_absmax = nf4.quantize(W)
    assert np.array_equal(absmax.cpu().numpy(), ref_absmax)
    assert np.array_equal(codes.cpu().numpy(), ref_codes)


def test_quantiser_hand_worked_block():
    from tests.test_oracle import _read_golden
    g = _read_golden(os.path.join(os.path.dirname(__file__), "golden", "nf4_block_example.txt"))
    W = torch.zeros((4, 64), dtype=torch.bfloat16)
    W[0, :8] = torch.tensor(g["w8"][0], dtype=torch.bfloat16)
    codes, absmax = binding.nf4_quantize(W.cuda())
    torch.cuda.synchronize()
    assert absmax[0, 0].item() == 4.0 and torch.all(absmax[0, 1:] == 0)
    assert codes[0, :5].cpu().tolist() == [int(v) for v in g["bytes5"][0]]
    assert torch.all(codes[1:] == 119)


def test_dequantiser_is_bit_exact():
    bits = _bf16_weight(520, 1024, seed=3)
    W = inputs.bf16_to_f64(bits).astype(np.float32)
    W[5, 128:192] = 0.0
    codes, absmax = nf4.quantize(W)
    got = binding.nf4_dequantize(torch.from_numpy(codes).cuda(), torch.from_numpy(absmax).cuda())
    torch.cuda.synchronize()
    assert np.array_equal(host64(got), nf4.dequantize(codes, absmax))


def run_nf4_layer(p, t, codes, absmax, use_scratch=False, band_tiles=0):
    """band_tiles > 0: the scratch buffer holds that many n-tiles of the smallest band the plan accepts (banded form)."""
    d = {k: dev(t[k]) for k in ("X", "A", "B", "dY")}
    cd, ad = torch.from_numpy(codes).cuda(), torch.from_numpy(absmax).cuda()
    plan = binding.LoraLinearPlan(p.T, p.d_in, p.d_out, p.r)
    bufs, out = {}, {}
    for name, shape, dt in (("Y", (p.T, p.d_out), torch.bfloat16), ("dX", (p.T, p.d_in), torch.bfloat16),
                            ("dA", (p.r, p.d_in), torch.float32), ("dB", (p.d_out, p.r), torch.float32)):
        bufs[name], out[name] = guarded(shape, dt)
    if band_tiles:
        lo, full = plan.nf4_scratch_bytes()
        assert full == 2 * p.d_out * p.d_in and 0 < lo <= max(full, lo)
        sbuf, scratch = guarded((band_tiles * lo // 2,), torch.bfloat16)
    else:
        sbuf, scratch = guarded((p.d_out, p.d_in), torch.bfloat16) if use_scratch else (None, None)
    plan.fwd_nf4(d["X"], cd, ad, d["A"], d["B"], p.scale, out["Y"], w_scratch=scratch)
    if scratch is not None:
        scratch.fill_(float("nan"))                     # backward must rebuild the weight itself
    plan.bwd_nf4(d["dY"], d["X"], cd, ad, d["A"], d["B"], p.scale, out["dX"], out["dA"], out["dB"], w_scratch=scratch)
    if scratch is not None:
        assert guards_intact(sbuf, scratch.numel()), "w_scratch: write outside the buffer"
    code, msg = plan.device_status()
    assert code == 0, msg
    for name in out:
        assert guards_intact(bufs[name], out[name].numel()), f"{name}: write outside the tensor"
        assert not torch.isnan(out[name].float()).any(), f"{name}: element left unwritten"
    plan.close()
    return out


NF4_SHAPES = [
    # T, d_in, d_out, r, scale           (d_in a multiple of 64; T > 128: CTA-pair kernels)
    (129, 64, 8, 8, 2.0),
    (300, 192, 200, 16, 1.7),
    (640, 768, 1160, 16, 2.0),
    (1000, 2048, 520, 64, 0.5),
    (2100, 512, 3080, 32, 2.0),           # more tiles than CTA pairs
    (4500, 1024, 4096, 16, 2.0),
]


@pytest.mark.parametrize("use_scratch", [False, True], ids=["in_kernel", "scratch"])
@pytest.mark.parametrize("T,d_in,d_out,r,scale", NF4_SHAPES)
def test_nf4_layer_elementwise(T, d_in, d_out, r, scale, use_scratch):
    p, t = inputs.draw_custom(T, d_in, d_out, r, scale, seed=4)
    W32 = inputs.bf16_to_f64(t["W"]).astype(np.float32)
    codes, absmax = nf4.quantize(W32)                          # the ORACLE's codes go to both sides
    out = run_nf4_layer(p, t, codes, absmax, use_scratch)
    f = {k: inputs.bf16_to_f64(t[k]) for k in ("X", "A", "B", "dY")}
    Y = nf4.forward(f["X"], codes, absmax, f["A"], f["B"], p.scale)
    dX, dA, dB = nf4.backward(f["dY"], f["X"], codes, absmax, f["A"], f["B"], p.scale)
    errs = {"Y": oracle.rel_err(host64(out["Y"]), Y), "dX": oracle.rel_err(host64(out["dX"]), dX),
            "dA": oracle.rel_err(host64(out["dA"]), dA), "dB": oracle.rel_err(host64(out["dB"]), dB)}
    assert errs["Y"] <= TOL_BF16 and errs["dX"] <= TOL_BF16, errs
    assert errs["dA"] <= TOL_F32 and errs["dB"] <= TOL_F32, errs


BANDED_SHAPES = [
    # T, d_in, d_out, r, scale, n-tiles of scratch      (bands of output rows forward, of input columns backward)
    (640, 768, 1160, 16, 2.0, 1),          # one n-tile per band: five forward bands with a ragged last one, three backward
    (1000, 2048, 520, 64, 0.5, 1),
    (2100, 512, 3080, 32, 2.0, 3),         # forward bands of several tiles, a short last band
    (4500, 1024, 4096, 16, 2.0, 2),
    (300, 1344, 1344, 16, 1.0, 2),         # 1344 is no multiple of the tile width: narrow last bands in both directions
]


@pytest.mark.parametrize("T,d_in,d_out,r,scale,tiles", BANDED_SHAPES)
def test_nf4_banded_scratch_matches_whole_weight_form_bitwise(T, d_in, d_out, r, scale, tiles):
    """A scratch buffer smaller than the weight: the weight is expanded and multiplied band by band.  Same tiles and order of
    summation as with the whole weight in scratch, so the outputs must agree bit for bit; and both with the oracle."""
    p, t = inputs.draw_custom(T, d_in, d_out, r, scale, seed=14)
    codes, absmax = nf4.quantize(inputs.bf16_to_f64(t["W"]).astype(np.float32))
    whole = run_nf4_layer(p, t, codes, absmax, use_scratch=True)
    banded = run_nf4_layer(p, t, codes, absmax, band_tiles=tiles)
    for name in ("Y", "dX", "dA", "dB"):
        assert torch.equal(whole[name], banded[name]), name
    f = {k: inputs.bf16_to_f64(t[k]) for k in ("X", "A", "B", "dY")}
    Y = nf4.forward(f["X"], codes, absmax, f["A"], f["B"], p.scale)
    dX, dA, dB = nf4.backward(f["dY"], f["X"], codes, absmax, f["A"], f["B"], p.scale)
    assert oracle.rel_err(host64(banded["Y"]), Y) <= TOL_BF16 and oracle.rel_err(host64(banded["dX"]), dX) <= TOL_BF16
    assert oracle.rel_err(host64(banded["dA"]), dA) <= TOL_F32 and oracle.rel_err(host64(banded["dB"]), dB) <= TOL_F32


def test_nf4_banded_weight_only_is_tight():
    """One-hot X / dY rows through the banded form: every band lands in its own columns of Y and dX."""
    T, d_in, d_out, r = 512, 768, 1024, 8
    p, t = inputs.draw_custom(T, d_in, d_out, r, 1.0, seed=16)
    codes, absmax = nf4.quantize(inputs.bf16_to_f64(t["W"]).astype(np.float32))
    what = nf4.dequantize(codes, absmax)
    bits = lambda x: x.contiguous().view(torch.int16).numpy().view(np.uint16)
    t2 = dict(t)
    # forward reads weight columns through one-hot X rows (T = 512 < d_in: the first 512 input features); backward weight
    # rows through one-hot dY rows (the first 512 output features)
    t2["X"] = bits(torch.eye(T, d_in, dtype=torch.bfloat16))
    t2["dY"] = bits(torch.eye(T, d_out, dtype=torch.bfloat16))
    t2["A"], t2["B"] = np.zeros_like(t["A"]), np.zeros_like(t["B"])
    out = run_nf4_layer(p, t2, codes, absmax, band_tiles=1)
    assert np.array_equal(host64(out["Y"]), what[:, :T].T)     # Y[t, :] = w_hat[:, t]
    assert np.array_equal(host64(out["dX"]), what[:T, :])      # dX[t, :] = w_hat[t, :]


def test_nf4_banded_rejects_what_it_cannot_serve():
    plan = binding.LoraLinearPlan(1000, 512, 1024, 16)
    lib = binding.load()
    lo, full = plan.nf4_scratch_bytes()
    cfg = plan.config()                                          # one n-tile of weight rows (forward) or columns (backward)
    assert lo == 2 * max(cfg["fwd_block_n"] * 512, cfg["dx_block_n"] * 1024) and full == 2 * 1024 * 512
    assert lib.lora_plan_set_nf4_scratch_bytes(plan._h, lo - 16) == binding.LORA_ERR_WORKSPACE
    assert lib.lora_plan_set_nf4_scratch_bytes(plan._h, lo) == binding.LORA_OK
    assert lib.lora_plan_set_nf4_scratch_bytes(plan._h, 0) == binding.LORA_OK
    plan.close()
    small = binding.LoraLinearPlan(64, 128, 512, 8)              # T <= 128: single-CTA plan, whole-weight scratch only
    assert lib.lora_plan_set_nf4_scratch_bytes(small._h, 2 * 256 * 128) == binding.LORA_ERR_UNSUPPORTED_SHAPE
    assert lib.lora_plan_set_nf4_scratch_bytes(small._h, 2 * 512 * 128) == binding.LORA_OK
    small.close()


def test_nf4_scratch_form_covers_small_batches():
    """With a scratch weight the bf16 kernels run, so batches of at most 128 tokens work too."""
    p, t = inputs.draw_custom(100, 128, 72, 8, 2.0, seed=8)
    W32 = inputs.bf16_to_f64(t["W"]).astype(np.float32)
    codes, absmax = nf4.quantize(W32)
    out = run_nf4_layer(p, t, codes, absmax, use_scratch=True)
    f = {k: inputs.bf16_to_f64(t[k]) for k in ("X", "A", "B", "dY")}
    Y = nf4.forward(f["X"], codes, absmax, f["A"], f["B"], p.scale)
    dX, dA, dB = nf4.backward(f["dY"], f["X"], codes, absmax, f["A"], f["B"], p.scale)
    assert oracle.rel_err(host64(out["Y"]), Y) <= TOL_BF16 and oracle.rel_err(host64(out["dX"]), dX) <= TOL_BF16
    assert oracle.rel_err(host64(out["dA"]), dA) <= TOL_F32 and oracle.rel_err(host64(out["dB"]), dB) <= TOL_F32


@pytest.mark.parametrize("use_scratch", [False, True], ids=["in_kernel", "scratch"])
def test_nf4_weight_only_is_tight(use_scratch):
    """A = 0, B = 0 and one-hot X / dY rows read single rows and columns of the dequantised weight: Y and dX must then be
    the oracle's bf16(level * absmax) values exactly (one product, one rounding, no accumulation)."""
    T, d_in, d_out, r = 256, 256, 256, 8
    p, t = inputs.draw_custom(T, d_in, d_out, r, 1.0, seed=6)
    W32 = inputs.bf16_to_f64(t["W"]).astype(np.float32)
    codes, absmax = nf4.quantize(W32)
    what = nf4.dequantize(codes, absmax)
    eye = torch.eye(256, dtype=torch.bfloat16)
    t2 = dict(t)
    bits = lambda x: x.contiguous().view(torch.int16).numpy().view(np.uint16)
    t2["X"], t2["dY"] = bits(eye), bits(eye)
    t2["A"] = np.zeros_like(t["A"])
    t2["B"] = np.zeros_like(t["B"])
    out = run_nf4_layer(p, t2, codes, absmax, use_scratch)
    assert np.array_equal(host64(out["Y"]), what.T)            # Y = I w_hat^T
    assert np.array_equal(host64(out["dX"]), what)             # dX = I w_hat


def test_nf4_rejects_unsupported():
    plan = binding.LoraLinearPlan(64, 128, 128, 8)             # T <= 128: single-CTA plan
    x = torch.zeros((64, 128), dtype=torch.bfloat16, device="cuda")
    c = torch.zeros((128, 64), dtype=torch.uint8, device="cuda")
    a = torch.zeros((2, 128), dtype=torch.float32, device="cuda")
    A = torch.zeros((8, 128), dtype=torch.bfloat16, device="cuda")
    B = torch.zeros((128, 8), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.LoraError) as e:
        plan.fwd_nf4(x, c, a, A, B, 1.0)
    assert e.value.code == binding.LORA_ERR_UNSUPPORTED_SHAPE
    plan.close()
