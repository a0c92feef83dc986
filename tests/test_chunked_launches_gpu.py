"""Long problems are cut into several launches per kernel.  Here the cut is forced on small shapes (tiny chunks through
the plan options): every output must keep its bits, with ragged token counts and chunk counts that do not divide
the work."""
import pytest

from paper_2604_26294_b200 import binding as b
from paper_2604_26294_b200 import build
from tests.helpers import DeviceProblem

pytestmark = pytest.mark.gpu

TINY_CHUNKS = {"gate_band": 1, "chunk_bands": 1, "chunk_tiles": 2, "dw_chunk_rounds": 1}
ONE_LAUNCH = {"chunk_bands": 0, "chunk_tiles": 0, "dw_chunk_rounds": 0}


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build_library()


def _run(prob, options):
    import torch

    S, H, F, D = prob.S, prob.H, prob.F, prob.D
    plan = b.tsp_mlp_plan_ex(H, F, D, **options)
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
def test_chunked_launches_keep_every_bit(S, H, F, D):
    import torch

    prob = DeviceProblem(S, H, F, D, seed=61, with_dy=True)
    ref, n_ref = _run(prob, ONE_LAUNCH)
    got, n_got = _run(prob, TINY_CHUNKS)
    assert n_ref == (2, 4)
    assert n_got[0] > 2 and n_got[1] > 4            # the cut really happened
    for a, r in zip(got, ref):
        assert bool(torch.isfinite(a.float()).all())
        view = torch.int32 if a.dtype == torch.float32 else torch.int16
        assert torch.equal(a.view(view), r.view(view))


def test_weight_gradient_list_of_wide_and_narrow_tiles_cut_into_launches():
    # S = 16384 at the 7B widths: the weight-gradient tile list is 1332 tiles of 256 x 512 followed by 24 of 256 x 256
    # (the narrow ones fill the last round of the 74 CTA pairs).  Cut into launches of one round each, the last launch
    # starts at list index 1258 and holds both kinds: the MMA lane has to take a tile's width from the position in the
    # whole list, not from the position inside the launch, or it would wait for a column half nobody loaded.
    import numpy as np
    import torch

    from oracle import tsp_mlp_oracle as orc
    from paper_2604_26294_b200 import inputs as inp
    from tests.helpers import rel_fro, tensor_to_f64

    S, H, F, D = 16384, 4096, 14336, 8
    prob = DeviceProblem(S, H, F, D, seed=62, with_dy=True)
    plan = b.tsp_mlp_plan_ex(H, F, D, dw_chunk_rounds=1, timeout_ms=500)
    try:
        ws = torch.empty(b.tsp_mlp_workspace_bytes(plan, S, b.TSP_WS_BACKWARD), dtype=torch.uint8, device="cuda")
        b.tsp_mlp_set_workspace(plan, ws)
        dX = torch.empty(S, H, dtype=torch.bfloat16, device="cuda")
        dWg = torch.full((D, H, F // D), float("nan"), dtype=torch.float32, device="cuda")
        dWu = torch.full((D, H, F // D), float("nan"), dtype=torch.float32, device="cuda")
        dWd = torch.full((D, F // D, H), float("nan"), dtype=torch.float32, device="cuda")
        b.tsp_mlp_backward(plan, prob.X, prob.Wg, prob.Wu, prob.Wd, prob.dY, dX, dWg, dWu, dWd, S, D)
        torch.cuda.synchronize()
        assert b.tsp_mlp_status(plan) == b.TSP_OK
        assert b.tsp_mlp_kernels_per_call(plan, b.TSP_WS_BACKWARD) >= 3 + 18     # the list really was cut
    finally:
        b.tsp_mlp_plan_destroy(plan)
    cols = inp.sample_columns(F, D, 32, seed=5)
    X, Wg, Wu, Wd, dY = prob.f64()
    rWg, rWu, rWd = orc.backward_columns(X, Wg, Wu, Wd, dY, cols)
    gWg = inp.unshard_columns(tensor_to_f64(dWg))[:, cols]
    gWu = inp.unshard_columns(tensor_to_f64(dWu))[:, cols]
    gWd = inp.unshard_rows(tensor_to_f64(dWd))[cols, :]
    for n, g, r in (("dWg", gWg, rWg), ("dWu", gWu, rWu), ("dWd", gWd, rWd)):
        assert np.all(np.isfinite(g)), n
        assert rel_fro(g, r) <= 1e-2, (n, rel_fro(g, r))
    assert bool(torch.isfinite(dWg).all()) and bool(torch.isfinite(dWu).all()) and bool(torch.isfinite(dWd).all())
