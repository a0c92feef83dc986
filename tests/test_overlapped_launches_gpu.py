"""Programmatic stream serialisation of the CTA-pair kernels (plan option overlap_launches).

A kernel's CTAs may start while the previous kernel of the stream is finishing; they set up barriers and tensor memory
and then wait, on the device, for the previous grid to complete before their first access to global memory.  Nothing
about the results may change: not within one call (the down projection reads the A the gate|up kernel wrote), and not
across calls that reuse the same workspace (the next call's gate|up kernel overwrites the A the previous call's down
projection is still reading, unless it waits).
"""
import pytest

from paper_2604_26294_b200 import binding as b
from paper_2604_26294_b200 import build
from tests.helpers import DeviceProblem

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build_library()


def _bits(t):
    import torch

    return t.view(torch.int32) if t.dtype == torch.float32 else t.view(torch.int16)


def _train_steps(probs, overlap, reps):
    """Forward + backward of several problems back to back through ONE plan and workspace, no host synchronisation
    in between; returns every step's outputs."""
    import torch

    S, H, F, D = probs[0].S, probs[0].H, probs[0].F, probs[0].D
    plan = b.tsp_mlp_plan_ex(H, F, D, overlap_launches=overlap)
    try:
        ws = torch.empty(b.tsp_mlp_workspace_bytes(plan, S, b.TSP_WS_BACKWARD), dtype=torch.uint8, device="cuda")
        b.tsp_mlp_set_workspace(plan, ws)
        outs = []
        for rep in range(reps):
            for prob in probs:
                Y = torch.empty((S, H), dtype=torch.bfloat16, device="cuda")
                dX = torch.empty((S, H), dtype=torch.bfloat16, device="cuda")
                dWg = torch.empty((D, H, F // D), dtype=torch.float32, device="cuda")
                dWu = torch.empty((D, H, F // D), dtype=torch.float32, device="cuda")
                dWd = torch.empty((D, F // D, H), dtype=torch.float32, device="cuda")
                b.tsp_mlp_forward(plan, prob.X, prob.Wg, prob.Wu, prob.Wd, Y, S, D)
                b.tsp_mlp_backward(plan, prob.X, prob.Wg, prob.Wu, prob.Wd, prob.dY, dX, dWg, dWu, dWd, S, D)
                outs.append((Y, dX, dWg, dWu, dWd))
        torch.cuda.synchronize()
        assert b.tsp_mlp_status(plan) == b.TSP_OK
    finally:
        b.tsp_mlp_plan_destroy(plan)
    return outs


# the second shape has several rounds of tiles per kernel
@pytest.mark.parametrize("S,H,F,D", [(512, 256, 1024, 2), (4096, 1024, 3584, 4)])
def test_back_to_back_steps_on_one_workspace_keep_every_bit(S, H, F, D):
    import torch

    probs = [DeviceProblem(S, H, F, D, seed=71 + i, with_dy=True) for i in range(2)]
    plain = _train_steps(probs, overlap=0, reps=1)
    overlapped = _train_steps(probs, overlap=1, reps=3)
    assert len(overlapped) == 6
    for i, outs in enumerate(overlapped):
        for got, want in zip(outs, plain[i % 2]):
            assert torch.equal(_bits(got), _bits(want))
    # the two problems really differ, so a step that read the other step's A would have been noticed
    assert not torch.equal(_bits(plain[0][0]), _bits(plain[1][0]))


def test_ring_steps_of_one_rank_keep_every_bit():
    """Per-rank ring steps: 2 D short launches per pass, each reading what its predecessor wrote (A, the carried sums)."""
    import torch

    S, H, F, D = 2048, 512, 2048, 4
    prob = DeviceProblem(S, H, F, D, seed=73)
    S_loc = S // D
    results = []
    for overlap in (0, 1):
        plan = b.tsp_mlp_plan_ex(H, F, D, overlap_launches=overlap)
        try:
            ws = torch.empty(b.tsp_mlp_workspace_bytes_ring(plan, S_loc, 0), dtype=torch.uint8, device="cuda")
            b.tsp_mlp_set_workspace(plan, ws)
            Ys = []
            for rep in range(3):
                for r in range(D):
                    Y = torch.full((S_loc, H), float("nan"), dtype=torch.bfloat16, device="cuda")
                    X_r = prob.X[r * S_loc:(r + 1) * S_loc]
                    for t in range(D):
                        k = (r - t) % D
                        b.tsp_mlp_ring_step(plan, X_r, prob.Wg[k], prob.Wu[k], prob.Wd[k], Y, S_loc, t, D)
                    Ys.append(Y)
            torch.cuda.synchronize()
            assert b.tsp_mlp_status(plan) == b.TSP_OK
        finally:
            b.tsp_mlp_plan_destroy(plan)
        results.append(torch.cat(Ys))
    assert torch.equal(_bits(results[0]), _bits(results[1]))
