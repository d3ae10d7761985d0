"""Failure detection on the device: a bounded wait that runs out is reported, and the plan stays usable.

The wait is made to run out in the allowed form: one CTA of the adapter-gradient kernel is launched through
`lora_debug_starved_wait` with its second-factor loader switched off, and the plan's wait limit is set to about a
millisecond.  The MMA warp's wait for the second factor gives up, records (reason, CTA) in the plan's status block,
the other warps see the abort flag and leave, the tensor memory is freed and the kernel returns.  Nothing faults,
traps or spins without a limit.
"""
import numpy as np
import pytest
import torch

from oracle import lora_oracle as oracle
from paper_2503_22673_b200 import binding, inputs

pytestmark = pytest.mark.gpu


def dev(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).cuda()


def test_wait_that_runs_out_is_reported_and_the_plan_recovers():
    T, d_in, d_out, r, s = 384, 256, 264, 16, 2.0
    p, t = inputs.draw_custom(T, d_in, d_out, r, s, seed=31)
    d = {k: dev(v) for k, v in t.items()}
    plan = binding.LoraLinearPlan(T, d_in, d_out, r)
    code, msg = plan.device_status()
    assert code == binding.LORA_OK, msg
    plan.set_wait_limit(2_000_000)                               # ~1 ms of SM clock ticks
    out = torch.full((d_in, r), float("nan"), dtype=torch.float32, device="cuda")
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    plan.debug_starved_wait(d["X"], out)
    t1.record()
    code, msg = plan.device_status()                             # synchronises the stream
    assert code == binding.LORA_ERR_DEVICE_TIMEOUT, (code, msg)
    # three roles wait at once (the MMA warp for its second factor, a producer for a free stage, the epilogue for the
    # accumulator); whichever gives up first writes the record, the others leave through the abort flag
    assert msg.startswith("device wait ran out:") and msg.endswith("(CTA 0)"), msg
    assert t0.elapsed_time(t1) < 200.0                           # ended by the limit (ms), nowhere near the 2 s default
    assert torch.isnan(out).all()                                # the starved launch wrote nothing
    code, msg = plan.device_status()                             # the record was cleared by the first query
    assert code == binding.LORA_OK, msg
    # the next ordinary calls on the same plan are correct
    plan.set_wait_limit(0)
    Y = plan.fwd(d["X"], d["W"], d["A"], d["B"], s)
    dX, dA, dB = plan.bwd(d["dY"], d["X"], d["W"], d["A"], d["B"], s)
    code, msg = plan.device_status()
    assert code == binding.LORA_OK, msg
    f = {k: inputs.bf16_to_f64(v) for k, v in t.items()}
    Yr = oracle.forward(f["X"], f["W"], f["A"], f["B"], s)
    dXr, dAr, dBr = oracle.backward(f["dY"], f["X"], f["W"], f["A"], f["B"], s)
    h = lambda x: x.float().cpu().numpy().astype(np.float64)
    assert oracle.rel_err(h(Y), Yr) <= 2e-2 and oracle.rel_err(h(dX), dXr) <= 2e-2
    assert oracle.rel_err(h(dA), dAr) <= 5e-3 and oracle.rel_err(h(dB), dBr) <= 5e-3
    plan.close()


def test_starved_wait_hook_rejects_large_shapes():
    plan = binding.LoraLinearPlan(256, 512, 512, 16)
    S = torch.zeros((2048, 512), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros((512, 16), dtype=torch.float32, device="cuda")
    with pytest.raises(binding.LoraError) as e:
        plan.debug_starved_wait(S, out)
    assert e.value.code == binding.LORA_ERR_UNSUPPORTED_SHAPE
    plan.close()
