"""The allocation-free contraction entry point, against the plain definition and the planned backward pass.

Some users of the library cannot allocate device memory at call time (a fixed pool that forbids cudaMalloc after
start-up, a latency-critical loop).  For them `lora_grad_contract_noalloc` keeps its scratch in a static device
array.  This test calls it through the C ABI twice in a row - the array is shared and keeps old contents, so the
second call would expose anything left uncleared - and compares the result
  * with the definition  out[c, j] = sum_t S[t, c] Rt[j, t]  evaluated in float64 on the very bf16 values passed in, and
  * with dB from `lora_linear_bwd` (the existing entry point that runs the same contraction with planned scratch),
both within the fp32 adapter-gradient tolerance used everywhere else (5e-3 of the largest entry).
"""
import gc

import numpy as np
import pytest
import torch

from paper_2503_22673_b200 import binding, inputs

pytestmark = pytest.mark.gpu
TOL_F32 = 5e-3


def _dev(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).cuda()


def _rel(a, b):
    return float((a - b).abs().max() / b.abs().max())


def _second_factor(t, s, ld):
    """bf16 bit patterns of scale * (X A^T)^T, [r, ld] with zero padding past T, and the same values in float64."""
    Xf, Af = inputs.bf16_to_f64(t["X"]), inputs.bf16_to_f64(t["A"])
    P = (s * (Xf @ Af.T)).T.astype(np.float32)                       # [r, T]
    bits = np.zeros((P.shape[0], ld), dtype=np.uint16)
    bits[:, :P.shape[1]] = inputs.f32_to_bf16_bits(P)
    return bits, inputs.bf16_to_f64(bits[:, :P.shape[1]])


CASES = [
    # T, d_in, d_out, r, scale, seed, ld - T
    (1500, 520, 1032, 16, 2.0, 21, 4),      # several feature chunks, a cluster of token chunks each
    (900, 264, 392, 32, 0.5, 22, 4),
    (700, 136, 200, 8, 2.0, 23, 36),        # r = 8: rows 8..15 of the second-factor box lie outside Rt (zero fill); ld > T
    (100, 72, 136, 24, 1.0, 24, 4),         # one slab: a single token chunk, no cluster
]


def test_noalloc_contraction_matches_definition_and_planned_backward_twice():
    lib = binding.load()
    assert lib.lora_grad_contract_noalloc_max_scratch() == 4096
    for T, d_in, d_out, r, s, seed, extra in CASES:
        p, t = inputs.draw_custom(T, d_in, d_out, r, s, seed=seed)
        d = {k: _dev(v) for k, v in t.items()}
        plan = binding.LoraLinearPlan(T, d_in, d_out, r)
        _, _, dB_planned = plan.bwd(d["dY"], d["X"], d["W"], d["A"], d["B"], s)
        torch.cuda.synchronize()
        ld = (T + extra + 7) // 8 * 8
        pt_bits, pt64 = _second_factor(t, s, ld)
        Pt = _dev(pt_bits)
        expected = torch.from_numpy(inputs.bf16_to_f64(t["dY"]).T @ pt64.T).cuda()      # [d_out, r], float64
        for call in range(2):
            out = torch.full((d_out, r), float("nan"), dtype=torch.float32, device="cuda")
            gc.collect()                                           # tensors of earlier tests go now, not during the call
            torch.cuda.synchronize()
            before, free_before = torch.cuda.memory_allocated(), torch.cuda.mem_get_info()[0]
            binding.grad_contract_noalloc(d["dY"], Pt, out)
            torch.cuda.synchronize()
            assert torch.cuda.memory_allocated() <= before        # nothing was taken from torch's allocator ...
            if call == 1:                                          # ... nor from the driver (the first call on a device may
                assert torch.cuda.mem_get_info()[0] >= free_before  # load the kernel; the second one must not move it)
            assert binding.grad_contract_noalloc_status() == binding.LORA_OK
            assert not torch.isnan(out).any(), (T, call)
            assert _rel(out.double(), expected) <= TOL_F32, (T, d_out, r, call, _rel(out.double(), expected))
            assert _rel(out, dB_planned) <= TOL_F32, (T, d_out, r, call, _rel(out, dB_planned))
            del out
        plan.close()


def test_noalloc_contraction_at_a_benchmark_size():
    """16384 x 4096 with r = 64 (the down-projection's dB shape): clusters of 16 token chunks, four accumulator blocks per
    CTA.  Checked against the float64 definition, twice."""
    T, C, r = 16384, 4096, 64
    g = np.random.Generator(np.random.Philox(key=77))
    s_bits = inputs.f32_to_bf16_bits(g.standard_normal((T, C), dtype=np.float32))
    r_bits = inputs.f32_to_bf16_bits(g.standard_normal((r, T), dtype=np.float32))
    S, Rt = _dev(s_bits), _dev(r_bits)
    expected = torch.from_numpy(inputs.bf16_to_f64(s_bits).T @ inputs.bf16_to_f64(r_bits).T).cuda()
    for call in range(2):
        out = torch.full((C, r), float("nan"), dtype=torch.float32, device="cuda")
        binding.grad_contract_noalloc(S, Rt, out)
        assert binding.grad_contract_noalloc_status() == binding.LORA_OK
        assert _rel(out.double(), expected) <= TOL_F32, (call, _rel(out.double(), expected))


def test_noalloc_contraction_rejects_sizes_beyond_its_limits():
    lib = binding.load()
    stream = torch.cuda.current_stream().cuda_stream
    # real, fully sized tensors: nothing can be touched out of bounds whatever the call decides
    T, C, r = 8, (1 << 24) + 8, 8
    S = torch.zeros((T, C), dtype=torch.bfloat16, device="cuda")
    Rt = torch.zeros((r, T), dtype=torch.bfloat16, device="cuda")
    o = torch.zeros((C, r), dtype=torch.float32, device="cuda")
    # more than 2^24 features: beyond what the entry point serves
    rc = lib.lora_grad_contract_noalloc(S.data_ptr(), Rt.data_ptr(), T, C, r, T, o.data_ptr(), stream)
    assert rc == binding.LORA_ERR_UNSUPPORTED_SHAPE
    rc = lib.lora_grad_contract_noalloc(S.data_ptr(), Rt.data_ptr(), 128, 60, 16, 128, o.data_ptr(), stream)
    assert rc == binding.LORA_ERR_UNSUPPORTED_SHAPE
    rc = lib.lora_grad_contract_noalloc(None, Rt.data_ptr(), 128, 64, 16, 128, o.data_ptr(), stream)
    assert rc == binding.LORA_ERR_INVALID_ARG
    torch.cuda.synchronize()
