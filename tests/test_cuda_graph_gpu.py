"""The forward and backward calls allocate nothing and only enqueue kernels, so they can be captured in a CUDA graph
and replayed (the way a launch-bound loop of ring steps would be run).  Replays must reproduce the eager bits."""
import pytest

from paper_2604_26294_b200 import binding as b
from paper_2604_26294_b200 import build
from tests.helpers import DeviceProblem

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build_library()


@pytest.mark.parametrize("S,H,F,D", [(512, 256, 1024, 2), (256, 256, 768, 2)])   # CTA-pair kernels / single-CTA kernels
def test_forward_and_backward_replay_from_a_cuda_graph(S, H, F, D):
    import torch

    prob = DeviceProblem(S, H, F, D, seed=51, with_dy=True)
    plan = b.tsp_mlp_plan(H, F, D)
    try:
        ws = torch.empty(b.tsp_mlp_workspace_bytes(plan, S, b.TSP_WS_BACKWARD), dtype=torch.uint8, device="cuda")
        b.tsp_mlp_set_workspace(plan, ws)
        Y = torch.empty(S, H, dtype=torch.bfloat16, device="cuda")
        dX = torch.empty_like(Y)
        dWg = torch.empty(D, H, F // D, dtype=torch.float32, device="cuda")
        dWu = torch.empty_like(dWg)
        dWd = torch.empty(D, F // D, H, dtype=torch.float32, device="cuda")

        def step(stream=None):
            b.tsp_mlp_forward(plan, prob.X, prob.Wg, prob.Wu, prob.Wd, Y, S, D, stream)
            b.tsp_mlp_backward(plan, prob.X, prob.Wg, prob.Wu, prob.Wd, prob.dY, dX, dWg, dWu, dWd, S, D, stream)

        step()                                   # eager: also sets the kernels' shared-memory attributes
        torch.cuda.synchronize()
        eager = [t.clone() for t in (Y, dX, dWg, dWu, dWd)]

        graph = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            with torch.cuda.graph(graph, stream=side):
                step(side)
        for _ in range(2):
            for t in (Y, dX, dWg, dWu, dWd):
                t.fill_(float("nan"))
            graph.replay()
            torch.cuda.synchronize()
            assert b.tsp_mlp_status(plan) == b.TSP_OK
            for got, ref in zip((Y, dX, dWg, dWu, dWd), eager):
                assert torch.equal(got.view(torch.int32 if got.dtype == torch.float32 else torch.int16),
                                   ref.view(torch.int32 if ref.dtype == torch.float32 else torch.int16))
    finally:
        b.tsp_mlp_plan_destroy(plan)
