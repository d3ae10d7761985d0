"""The forward and backward calls only enqueue work on the caller's stream (no allocation, no synchronisation, no host
read-back), so a step can be captured into a CUDA graph and replayed.  Checked here: a captured fwd + bwd, replayed on new
input VALUES in the same buffers, reproduces the eager calls bit for bit (the path is bitwise reproducible), for a
launch-bound tiny shape (single-CTA kernels) and a shape on the CTA-pair kernels with clustered gradient launches."""
import pytest
import torch

from paper_2503_22673_b200 import binding, inputs
from tests.test_parity_gpu import dev

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("T,d_in,d_out,r", [(256, 512, 512, 8), (1000, 1024, 1536, 16)])
def test_captured_step_replays_bitwise(T, d_in, d_out, r):
    s = 2.0
    draws = [inputs.draw_custom(T, d_in, d_out, r, s, seed=sd)[1] for sd in (31, 32)]
    cur = {k: dev(v).clone() for k, v in draws[0].items()}          # static buffers the graph reads
    plan = binding.LoraLinearPlan(T, d_in, d_out, r)
    plan.ensure_workspace()
    out = {"Y": torch.empty((T, d_out), dtype=torch.bfloat16, device="cuda"),
           "dX": torch.empty((T, d_in), dtype=torch.bfloat16, device="cuda"),
           "dA": torch.empty((r, d_in), dtype=torch.float32, device="cuda"),
           "dB": torch.empty((d_out, r), dtype=torch.float32, device="cuda")}

    def step():
        plan.fwd(cur["X"], cur["W"], cur["A"], cur["B"], s, out["Y"])
        plan.bwd(cur["dY"], cur["X"], cur["W"], cur["A"], cur["B"], s, out["dX"], out["dA"], out["dB"])

    eager = []
    for t in draws:                                                  # eager results for both input sets
        for k, v in t.items():
            cur[k].copy_(dev(v))
        step()
        torch.cuda.synchronize()
        eager.append({k: v.clone() for k, v in out.items()})
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):                                    # the binding launches on the current (capturing) stream
        step()
    for rep in range(2):
        for i, t in enumerate(draws):
            for k, v in t.items():
                cur[k].copy_(dev(v))
            for v in out.values():
                v.fill_(float("nan"))
            graph.replay()
            torch.cuda.synchronize()
            for k in out:
                got, want = out[k], eager[i][k]
                if got.dtype == torch.bfloat16:
                    got, want = got.view(torch.int16), want.view(torch.int16)
                same = torch.equal(got, want)
                assert same, (k, i, rep)
    code, msg = plan.device_status()
    assert code == 0, msg
    del graph
    plan.close()
