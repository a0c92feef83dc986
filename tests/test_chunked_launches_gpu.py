"""Long problems are cut into several launches per kernel.  Here the cut is forced on small shapes (tiny chunks through
the tunables, which a plan reads when it is created): every output must keep its bits, with ragged token counts and
chunk counts that do not divide the work."""
import pytest

from paper_2604_26294_b200 import binding as b
from paper_2604_26294_b200 import build
from tests.helpers import DeviceProblem

pytestmark = pytest.mark.gpu

TINY_CHUNKS = {"TSP_MLP_BAND": "1", "TSP_MLP_CHUNK_BANDS": "1", "TSP_MLP_CHUNK_TILES": "2", "TSP_MLP_DW_CHUNK_ROUNDS": "1"}
ONE_LAUNCH = {"TSP_MLP_CHUNK_BANDS": "0", "TSP_MLP_CHUNK_TILES": "0", "TSP_MLP_DW_CHUNK_ROUNDS": "-1"}


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build_library()


def _run(prob, env, monkeypatch):
    import torch

    for k in set(TINY_CHUNKS) | set(ONE_LAUNCH):
        monkeypatch.delenv(k, raising=False)
    for k, v in env.items():
        monkeypatch.setenv(k, v)
    S, H, F, D = prob.S, prob.H, prob.F, prob.D
    plan = b.tsp_mlp_plan(H, F, D)          # the tunables are read here
    try:
        ws = torch.empty(b.tsp_mlp_workspace_bytes(plan, S, b.TSP_WS_BACKWARD), dtype=torch.uint8, device="cuda")
        b.tsp_mlp_set_workspace(plan, ws)
        Y = torch.full((S, H), float("nan"), dtype=torch.bfloat16, device="cuda")
        dX = torch.full((S, H), float("nan"), dtype=torch.bfloat16, device="cuda")
        dWg = torch.full((D, H, F // D), float("nan"), dtype=torch.float32, device="cuda")
        dWu = torch.full((D, H, F // D), float("nan"), dtype=torch.float32, device="cuda")
        dWd = torch.full((D, F // D, H), float("nan"), dtype=torch.float32, device="cuda")
        b.tsp_mlp_forward(plan, prob.X, prob.Wg, prob.Wu, prob.Wd, Y, S, D)
        b.tsp_mlp_backward(plan, prob.X, prob.Wg, prob.Wu, prob.Wd, prob.dY, dX, dWg, dWu, dWd, S, D)
        torch.cuda.synchronize()
        assert b.tsp_mlp_status(plan) == b.TSP_OK
        launches = (b.tsp_mlp_kernels_per_call(plan, b.TSP_WS_FORWARD), b.tsp_mlp_kernels_per_call(plan, b.TSP_WS_BACKWARD))
    finally:
        b.tsp_mlp_plan_destroy(plan)
    return (Y, dX, dWg, dWu, dWd), launches


@pytest.mark.parametrize("S,H,F,D", [(2048, 256, 512, 2),     # 8 token tiles: 8 / 4 chunks
                                     (3000, 256, 1536, 3),    # 1000 tokens per rank: ragged last tile of every rank
                                     (1280, 512, 512, 1),     # 5 token tiles: the remainder joins the last chunk
                                     (3584, 256, 1792, 7)])    # 14 token tiles, 7 ranks
def test_chunked_launches_keep_every_bit(S, H, F, D, monkeypatch):
    import torch

    prob = DeviceProblem(S, H, F, D, seed=61, with_dy=True)
    ref, n_ref = _run(prob, ONE_LAUNCH, monkeypatch)
    got, n_got = _run(prob, TINY_CHUNKS, monkeypatch)
    assert n_ref == (2, 4)
    assert n_got[0] > 2 and n_got[1] > 4            # the cut really happened
    for a, r in zip(got, ref):
        assert bool(torch.isfinite(a.float()).all())
        view = torch.int32 if a.dtype == torch.float32 else torch.int16
        assert torch.equal(a.view(view), r.view(view))
