"""GPU parity at the full benchmark sizes, in the launch configuration bench.py times (default plan).

Single-projection workloads (q_proj, gate/up_proj, down_proj): the WHOLE of Y and dX is compared element by element
with the oracle, which is evaluated in blocks of 2048 token rows so that the float64 arrays stay small (token rows are
independent); the error measure max|gpu - ref| / max|ref| is taken over the complete matrix.  The same holds for all
seven projections of the whole-layer workload (T = 32768).  The paper's own r = 32 setting (T = 49152), the dense
weight gradient and the NF4 weight are compared on a dense row sample:
two rows of every 128-row slab (so every tile row, every persistent-loop position and both TMEM accumulator buffers are
hit), the rows on both sides of the tile borders, the first and the last row; all columns of each sampled row.
dA and dB are always compared in full.  Two adjoint identities that hold at any size are checked on the GPU outputs as
a whole:  <dY, Y> = <dX, X>  and  <dA, A> = <dB, B>.

Tolerances: max|gpu - ref| / max|ref| <= 2e-2 (Y, dX, bf16), <= 5e-3 (dA, dB, fp32).
"""
import gc

import numpy as np
import pytest
import torch

from oracle import lora_oracle as oracle
from paper_2503_22673_b200 import binding, inputs

pytestmark = pytest.mark.gpu

TOL_BF16 = 2e-2
TOL_F32 = 5e-3


def dev(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).cuda()


def host64(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def sample_rows(T, n_random=40, seed=0):
    fixed = [0, 1, 127, 128, 129, 255, 256, 257, 511, 512, T // 2 - 1, T // 2, T - 257, T - 256, T - 129, T - 128, T - 2, T - 1]
    rng = np.random.default_rng(seed)
    rows = sorted({r for r in fixed if 0 <= r < T} | set(rng.integers(0, T, n_random).tolist()))
    return np.asarray(rows, dtype=np.int64)


def slab_rows(T, seed=0, slab=128):
    """Two rows of every `slab`-row slab (one at a position that walks through the slab, one random) plus the border rows."""
    rng = np.random.default_rng(seed)
    n = -(-T // slab)
    walk = np.arange(n) * slab + (np.arange(n) * 37) % slab
    rnd = np.arange(n) * slab + rng.integers(0, slab, n)
    rows = np.concatenate([walk, rnd, sample_rows(T, 0)])
    return np.unique(rows[rows < T]).astype(np.int64)


BLOCK_ROWS = 2048


def full_rel_err(gpu, act_bits, ref_rows_fn):
    """max|gpu - ref| / max|ref| over the complete [T, n] matrix, the oracle evaluated BLOCK_ROWS token rows at a time."""
    num = den = 0.0
    for lo in range(0, act_bits.shape[0], BLOCK_ROWS):
        hi = min(lo + BLOCK_ROWS, act_bits.shape[0])
        ref = ref_rows_fn(inputs.bf16_to_f64(act_bits[lo:hi]))
        got = host64(gpu[lo:hi])
        num = max(num, float(np.max(np.abs(got - ref))))
        den = max(den, float(np.max(np.abs(ref))))
    return num / den if den > 0 else (0.0 if num == 0 else float("inf"))


def dot64(a, b):
    return float((a.double() * b.double()).sum().item())


def check_projection(p, t, x_dev=None, whole=False):
    d = {k: dev(v) for k, v in t.items() if k != "X"}
    d["X"] = x_dev if x_dev is not None else dev(t["X"])
    plan = binding.LoraLinearPlan(p.T, p.d_in, p.d_out, p.r)
    Y = plan.fwd(d["X"], d["W"], d["A"], d["B"], p.scale)
    dX, dA, dB = plan.bwd(d["dY"], d["X"], d["W"], d["A"], d["B"], p.scale)
    code, msg = plan.device_status()
    assert code == 0, msg
    W, A, B = (inputs.bf16_to_f64(t[k]) for k in ("W", "A", "B"))
    if whole:
        # ---- every element of Y and dX ----
        eY = full_rel_err(Y, t["X"], lambda xb: oracle.forward(xb, W, A, B, p.scale))
        eX = full_rel_err(dX, t["dY"], lambda gb: oracle.backward_dx_rows(np.arange(gb.shape[0]), gb, W, A, B, p.scale))
    else:
        # ---- two rows of every 128-row slab + border rows of Y and dX ----
        rows = slab_rows(p.T)
        rows_t = torch.from_numpy(rows).cuda()
        Yr = oracle.forward_rows(np.arange(len(rows)), inputs.bf16_to_f64(t["X"][rows]), W, A, B, p.scale)
        dXr = oracle.backward_dx_rows(np.arange(len(rows)), inputs.bf16_to_f64(t["dY"][rows]), W, A, B, p.scale)
        eY = oracle.rel_err(host64(Y[rows_t]), Yr)
        eX = oracle.rel_err(host64(dX[rows_t]), dXr)
    del W
    # ---- adapter gradients in full ----
    Xf = inputs.bf16_to_f64(t["X"])
    dYf = inputs.bf16_to_f64(t["dY"])
    dAr, dBr = oracle.backward_adapter_grads(dYf, Xf, A, B, p.scale)
    del Xf, dYf
    eA = oracle.rel_err(host64(dA), dAr)
    eB = oracle.rel_err(host64(dB), dBr)
    # ---- identities on the complete GPU outputs ----
    lhs, rhs = dot64(d["dY"], Y), dot64(dX, d["X"])
    a, b = dot64(dA, d["A"]), dot64(dB, d["B"])
    scale_yx = (d["dY"].double().norm() * Y.double().norm()).item()
    scale_ab = (dA.double().norm() * d["A"].double().norm() + dB.double().norm() * d["B"].double().norm()).item()
    plan.close()
    errs = {"Y": eY, "dX": eX, "dA": eA, "dB": eB, "adjoint_yx": abs(lhs - rhs) / scale_yx,
            "adjoint_ab": abs(a - b) / scale_ab}
    assert eY <= TOL_BF16 and eX <= TOL_BF16, (p.name, errs)
    assert eA <= TOL_F32 and eB <= TOL_F32, (p.name, errs)
    assert errs["adjoint_yx"] <= 1e-3, (p.name, errs)      # bf16 rounding of Y and dX averages out over T x d entries
    # both sides carry the bf16 rounding of s*P and s*Q; the inner products cancel heavily, so the difference is
    # measured against the norms (Cauchy-Schwarz scale), not against the value itself
    assert errs["adjoint_ab"] <= 5e-3, (p.name, errs)
    del d, Y, dX, dA, dB
    gc.collect()
    torch.cuda.empty_cache()
    return errs


@pytest.mark.parametrize("idx", [1, 2, 3])
def test_single_projection_workloads_full_size(idx):
    (p, t), = list(inputs.draw_workload(idx, seed=0))
    check_projection(p, t, whole=True)


def test_seven_projection_layer_full_size():
    x_dev = {}
    for p, t in inputs.draw_workload(4, seed=0):
        if p.x_group not in x_dev:
            x_dev.clear()
            x_dev[p.x_group] = dev(t["X"])
        check_projection(p, t, x_dev[p.x_group], whole=True)


# ---------------------------------------------------------------------------------------------
# the two further rows at full size: dense weight gradient (full fine-tuning) and the NF4 weight (Q+LoRA)
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("idx", [1, 3])
def test_dense_dw_full_size_sampled(idx):
    """dW = dY^T X at the benchmark sizes: two rows of every 128-row slab of dW (each row o is dY[:, o]^T X, one fp64
    matrix-vector product) against the oracle's definition, rows on both sides of the tile borders included; plus the
    identity  <dW, M> = <dY, X M^T>  for a random bf16 M on the complete output (fp64 on the device)."""
    (p, t), = list(inputs.draw_workload(idx, seed=0))
    X, dY = dev(t["X"]), dev(t["dY"])
    plan = binding.LoraLinearPlan(p.T, p.d_in, p.d_out, p.r)
    dW = plan.dense_dw(dY, X)
    code, msg = plan.device_status()
    assert code == 0, msg
    rows = slab_rows(p.d_out, seed=1)
    Xf = inputs.bf16_to_f64(t["X"])
    ref = oracle.dense_weight_grad(inputs.bf16_to_f64(t["dY"][:, rows]), Xf)
    del Xf
    err = oracle.rel_err(host64(dW[torch.from_numpy(rows).cuda()]), ref)
    assert err <= TOL_BF16, (p.name, err)
    M = torch.randn((p.d_out, p.d_in), device="cuda", dtype=torch.float32).to(torch.bfloat16)
    lhs = dot64(dW, M)
    rhs = dot64(dY, (X.float() @ M.float().T))        # library matmul only inside the CHECK, fp32 accumulate
    scale = (dW.double().norm() * M.double().norm()).item()
    assert abs(lhs - rhs) / scale <= 1e-3, (p.name, lhs, rhs, scale)
    plan.close()
    del X, dY, dW, M
    gc.collect()
    torch.cuda.empty_cache()


@pytest.mark.parametrize("use_scratch", [True, "band", False], ids=["scratch", "banded_8MiB", "in_kernel"])
def test_nf4_full_size_config1(use_scratch):
    """Q+LoRA at the q_proj size (T = 8192, 4096 -> 4096, r = 16): the GPU quantiser's codes and scales must equal the
    oracle's bit for bit; Y and dX on two rows of every 128-row slab and dA, dB in full against the oracle on the dequantised weight."""
    from oracle import nf4_oracle as nf4
    (p, t), = list(inputs.draw_workload(1, seed=0))
    d = {k: dev(v) for k, v in t.items()}
    codes, absmax = binding.nf4_quantize(d["W"])
    ref_codes, ref_absmax = nf4.quantize(inputs.bf16_to_f64(t["W"]).astype(np.float32))
    assert np.array_equal(codes.cpu().numpy(), ref_codes) and np.array_equal(absmax.cpu().numpy(), ref_absmax)
    plan = binding.LoraLinearPlan(p.T, p.d_in, p.d_out, p.r)
    scratch = torch.empty((p.d_out, p.d_in), dtype=torch.bfloat16, device="cuda") if use_scratch else None
    if use_scratch == "band":                          # a quarter of the 32 MiB weight: four bands each way
        scratch = torch.empty((4 << 20,), dtype=torch.bfloat16, device="cuda")
    Y = plan.fwd_nf4(d["X"], codes, absmax, d["A"], d["B"], p.scale, w_scratch=scratch)
    dX, dA, dB = plan.bwd_nf4(d["dY"], d["X"], codes, absmax, d["A"], d["B"], p.scale, w_scratch=scratch)
    code, msg = plan.device_status()
    assert code == 0, msg
    rows = slab_rows(p.T)
    rows_t = torch.from_numpy(rows).cuda()
    What, A, B = nf4.dequantize(ref_codes, ref_absmax), inputs.bf16_to_f64(t["A"]), inputs.bf16_to_f64(t["B"])
    Yr = oracle.forward_rows(np.arange(len(rows)), inputs.bf16_to_f64(t["X"][rows]), What, A, B, p.scale)
    dXr = oracle.backward_dx_rows(np.arange(len(rows)), inputs.bf16_to_f64(t["dY"][rows]), What, A, B, p.scale)
    dAr, dBr = oracle.backward_adapter_grads(inputs.bf16_to_f64(t["dY"]), inputs.bf16_to_f64(t["X"]), A, B, p.scale)
    errs = {"Y": oracle.rel_err(host64(Y[rows_t]), Yr), "dX": oracle.rel_err(host64(dX[rows_t]), dXr),
            "dA": oracle.rel_err(host64(dA), dAr), "dB": oracle.rel_err(host64(dB), dBr)}
    plan.close()
    assert errs["Y"] <= TOL_BF16 and errs["dX"] <= TOL_BF16, errs
    assert errs["dA"] <= TOL_F32 and errs["dB"] <= TOL_F32, errs
    del d, Y, dX, dA, dB
    gc.collect()
    torch.cuda.empty_cache()


def test_paper_adapter_setting_full_size():
    """The paper's own setting (Section 4.5: q/k/v/o adapters, lora_r = 32, alpha = 64) at its batch shape, 6 x 8k = 49152
    packed tokens: the 4096-wide q projection and the 1024-wide k projection (v and o repeat their shapes)."""
    x_dev = None
    for p, t in inputs.draw_workload(5, seed=0):
        if p.name not in ("q_proj", "k_proj"):
            break
        if x_dev is None:
            x_dev = dev(t["X"])
        check_projection(p, t, x_dev)


@pytest.mark.parametrize("wl,ids", [(4, (0, 1, 2)), (4, (4, 5)), (5, (0, 1, 2))], ids=["qkv_r16", "gate_up_r16", "qkv_r32"])
def test_grouped_projections_full_size(wl, ids):
    """The grouped calls at the benchmark sizes (q/k/v and gate/up of the whole-layer workload, q/k/v of the paper's own
    r = 32 setting at 49152 tokens): every projection against ITS OWN oracle - two rows of every 128-row slab of Y_g, dA_g
    and dB_g in full - and dX against the sum of the groups' oracles on the same row sample."""
    from paper_2503_22673_b200.grouped import GroupedLoraPlan
    projs = [(p, t) for j, (p, t) in enumerate(inputs.draw_workload(wl, seed=0)) if j in ids]
    p0 = projs[0][0]
    gp = GroupedLoraPlan(p0.T, p0.d_in, [p.d_out for p, _ in projs], p0.r)
    W, A, B = gp.pack([dev(t["W"]) for _, t in projs], [dev(t["A"]) for _, t in projs], [dev(t["B"]) for _, t in projs])
    X = dev(projs[0][1]["X"])
    dY = torch.cat([dev(t["dY"]) for _, t in projs], dim=1).contiguous()
    Y = gp.fwd(X, W, A, B, p0.scale)
    dX, dAs, dBs = gp.bwd(dY, X, W, A, B, p0.scale)
    code, msg = gp.device_status()
    assert code == 0, msg
    rows = slab_rows(p0.T)
    rows_t = torch.from_numpy(rows).cuda()
    Xr = inputs.bf16_to_f64(projs[0][1]["X"][rows])
    Xf = inputs.bf16_to_f64(projs[0][1]["X"])
    dX_ref = 0.0
    errs = {}
    for g, (p, t) in enumerate(projs):
        Wg, Ag, Bg = (inputs.bf16_to_f64(t[k]) for k in ("W", "A", "B"))
        Yr = oracle.forward(Xr, Wg, Ag, Bg, p.scale)
        dX_ref = dX_ref + oracle.backward_dx_rows(np.arange(len(rows)), inputs.bf16_to_f64(t["dY"][rows]), Wg, Ag, Bg, p.scale)
        dAr, dBr = oracle.backward_adapter_grads(inputs.bf16_to_f64(t["dY"]), Xf, Ag, Bg, p.scale)
        errs[p.name] = (oracle.rel_err(host64(gp.split_outputs(Y)[g][rows_t]), Yr), oracle.rel_err(host64(dAs[g]), dAr),
                        oracle.rel_err(host64(dBs[g]), dBr))
        del Wg
    eX = oracle.rel_err(host64(dX[rows_t]), dX_ref)
    gp.close()
    for name, (eY, eA, eB) in errs.items():
        assert eY <= TOL_BF16 and eA <= TOL_F32 and eB <= TOL_F32, (name, errs)
    assert eX <= TOL_BF16, eX
    del X, dY, Y, dX, W
    gc.collect()
    torch.cuda.empty_cache()


def test_more_than_2_31_elements_per_tensor():
    """Index arithmetic beyond 32 bits: X and dX hold 540000 x 4096 = 2.2e9 elements (4.4 GB each).  The oracle cannot hold
    such a matrix in float64, so: sampled rows of Y and dX (first, last, around the 2^31-element boundary, random) against
    the oracle row by row; dA and dB against the sum of the layer's own results on the two halves of the token range
    (additivity over token rows, each half below 2^31 elements) and the adjoint identity <dA, A> = <dB, B>."""
    T, d_in, d_out, r, scale = 540000, 4096, 520, 16, 2.0
    g = torch.Generator(device="cuda").manual_seed(7)
    X = torch.randn((T, d_in), device="cuda", generator=g, dtype=torch.float32).to(torch.bfloat16)
    dY = torch.randn((T, d_out), device="cuda", generator=g, dtype=torch.float32).to(torch.bfloat16)
    W = (torch.randn((d_out, d_in), device="cuda", generator=g) / 64).to(torch.bfloat16)
    A = (torch.randn((r, d_in), device="cuda", generator=g) / 64).to(torch.bfloat16)
    B = (torch.randn((d_out, r), device="cuda", generator=g) * 0.14).to(torch.bfloat16)
    plan = binding.LoraLinearPlan(T, d_in, d_out, r)
    Y = plan.fwd(X, W, A, B, scale)
    dX, dA, dB = plan.bwd(dY, X, W, A, B, scale)
    code, msg = plan.device_status()
    assert code == 0, msg
    plan.close()
    edge = (1 << 31) // d_in                                            # first row past 2^31 elements of X
    rows = np.unique(np.concatenate([sample_rows(T, 24, seed=3), [edge - 129, edge - 1, edge, edge + 1, edge + 127, edge + 128]]))
    rt = torch.from_numpy(rows).cuda()
    Wf, Af, Bf = host64(W), host64(A), host64(B)
    Yr = oracle.forward(host64(X[rt]), Wf, Af, Bf, scale)
    dXr = oracle.backward_dx_rows(np.arange(len(rows)), host64(dY[rt]), Wf, Af, Bf, scale)
    assert oracle.rel_err(host64(Y[rt]), Yr) <= TOL_BF16
    assert oracle.rel_err(host64(dX[rt]), dXr) <= TOL_BF16
    half = 270080                                                       # a multiple of 128: both halves below 2^31 elements
    dA_sum = torch.zeros_like(dA, dtype=torch.float64)
    dB_sum = torch.zeros_like(dB, dtype=torch.float64)
    for lo, hi in ((0, half), (half, T)):
        ph = binding.LoraLinearPlan(hi - lo, d_in, d_out, r)
        _, dA_h, dB_h = ph.bwd(dY[lo:hi], X[lo:hi], W, A, B, scale)
        dA_sum += dA_h.double()
        dB_sum += dB_h.double()
        ph.close()
    # not bit-equal: the second factors s (dY B) and s (X A^T) are rounded to bf16 from fp32 sums whose order depends on the
    # plan's grid, so a few of the 540000 tokens' values flip by one bf16 step between the full and the half-size plans
    assert oracle.rel_err(host64(dA), dA_sum.cpu().numpy()) <= 5e-4
    assert oracle.rel_err(host64(dB), dB_sum.cpu().numpy()) <= 5e-4
    # the halves themselves against the oracle on a slab it can hold: the first 8192 tokens
    ps = binding.LoraLinearPlan(8192, d_in, d_out, r)
    _, dA_s, dB_s = ps.bwd(dY[:8192], X[:8192], W, A, B, scale)
    dAr, dBr = oracle.backward_adapter_grads(host64(dY[:8192]), host64(X[:8192]), Af, Bf, scale)
    assert oracle.rel_err(host64(dA_s), dAr) <= TOL_F32 and oracle.rel_err(host64(dB_s), dBr) <= TOL_F32
    ps.close()
    a, b = dot64(dA, A), dot64(dB, B)
    scale_ab = (dA.double().norm() * A.double().norm() + dB.double().norm() * B.double().norm()).item()
    assert abs(a - b) / scale_ab <= 5e-3
    del X, dY, Y, dX
    gc.collect()
    torch.cuda.empty_cache()
