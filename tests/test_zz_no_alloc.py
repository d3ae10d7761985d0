"""The allocation-free contraction entry point against the planned backward pass.

Some users of the library cannot allocate device memory at call time (a fixed pool, a latency-critical
loop).  For them `lora_grad_contract_noalloc` keeps its scratch in a static device array.  This test calls
it through the C ABI twice in a row - the array is shared and keeps old contents, so the second call would
expose anything left uncleared - and compares with dB from `lora_linear_bwd`, within the fp32 adapter
gradient tolerance used everywhere else (5e-3 of the largest entry).
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


def test_noalloc_contraction_matches_planned_backward_twice():
    lib = binding.load()
    assert lib.lora_grad_contract_noalloc_max_scratch() == 8 << 20
    cases = [(1500, 520, 1032, 16, 2.0, 21), (900, 264, 392, 32, 0.5, 22)]
    for T, d_in, d_out, r, s, seed in cases:
        p, t = inputs.draw_custom(T, d_in, d_out, r, s, seed=seed)
        d = {k: _dev(v) for k, v in t.items()}
        plan = binding.LoraLinearPlan(T, d_in, d_out, r)
        _, _, dB_ref = plan.bwd(d["dY"], d["X"], d["W"], d["A"], d["B"], s)
        torch.cuda.synchronize()
        # the second factor the planned path builds internally: scale * (X A^T)^T rounded to bf16, [r, ld]
        ld = (T + 7) // 8 * 8
        Pt = torch.zeros((r, ld), dtype=torch.bfloat16, device="cuda")
        Pt[:, :T] = ((d["X"].float() @ d["A"].float().t()) * s).t().to(torch.bfloat16)
        for call in range(2):
            out = torch.full((d_out, r), float("nan"), dtype=torch.float32, device="cuda")
            gc.collect()                                           # tensors of earlier tests go now, not during the call
            torch.cuda.synchronize()
            before = torch.cuda.memory_allocated()
            binding.grad_contract_noalloc(d["dY"], Pt, out)
            torch.cuda.synchronize()
            assert torch.cuda.memory_allocated() <= before        # nothing was taken from torch's allocator
            assert not torch.isnan(out).any(), (T, call)
            assert _rel(out, dB_ref) <= TOL_F32, (T, d_out, r, call, _rel(out, dB_ref))
            del out
        plan.close()


def test_noalloc_contraction_rejects_what_does_not_fit():
    lib = binding.load()
    stream = torch.cuda.current_stream().cuda_stream
    # real, fully sized tensors: nothing can be touched out of bounds whatever the call decides
    T, C, r = 16384, 4096, 64
    S = torch.zeros((T, C), dtype=torch.bfloat16, device="cuda")
    Rt = torch.zeros((r, T), dtype=torch.bfloat16, device="cuda")
    o = torch.zeros((C, r), dtype=torch.float32, device="cuda")
    # 16 feature chunks x 9 token chunks x 64 x 4096 fp32 partial sums = 9.4 MiB > the 8 MiB static array
    rc = lib.lora_grad_contract_noalloc(S.data_ptr(), Rt.data_ptr(), T, C, r, T, o.data_ptr(), stream)
    assert rc == binding.LORA_ERR_WORKSPACE
    rc = lib.lora_grad_contract_noalloc(S.data_ptr(), Rt.data_ptr(), 128, 60, 16, 128, o.data_ptr(), stream)
    assert rc == binding.LORA_ERR_UNSUPPORTED_SHAPE
    rc = lib.lora_grad_contract_noalloc(None, Rt.data_ptr(), 128, 64, 16, 128, o.data_ptr(), stream)
    assert rc == binding.LORA_ERR_INVALID_ARG
    torch.cuda.synchronize()
