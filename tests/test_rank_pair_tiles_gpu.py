"""Two-rank tiles: one tile holds the same 256 token rows of ranks 2q+1 and 2q and loads every weight panel once.

Rank 2q meets the shards in the order of rank 2q+1 shifted by one ring step (Algorithm 2: shard (r - t) mod D at step
t), so the kernel runs D + 1 slots and feeds each loaded panel to both ranks' accumulators, each in its own step.  The
per-rank accumulation order is unchanged, so every output must keep every bit of the one-rank kernels' result.
"""
import pytest

from oracle import tsp_mlp_oracle as orc
from paper_2604_26294_b200 import binding as b
from paper_2604_26294_b200 import build
from tests.helpers import DeviceProblem, rel_fro, tensor_to_f64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build_library()


def _run(prob, reps=2, **options):
    import torch

    S, H, F, D = prob.S, prob.H, prob.F, prob.D
    plan = b.tsp_mlp_plan_ex(H, F, D, **options)
    try:
        ws = torch.empty(b.tsp_mlp_workspace_bytes(plan, S, b.TSP_WS_BACKWARD), dtype=torch.uint8, device="cuda")
        b.tsp_mlp_set_workspace(plan, ws)
        outs = []
        for rep in range(reps):   # more than once: the scheduler words must be back at zero after every launch
            Y = torch.full((S, H), float("nan"), dtype=torch.bfloat16, device="cuda")
            dX = torch.full((S, H), float("nan"), dtype=torch.bfloat16, device="cuda")
            dWg = torch.empty((D, H, F // D), dtype=torch.float32, device="cuda")
            dWu = torch.empty((D, H, F // D), dtype=torch.float32, device="cuda")
            dWd = torch.empty((D, F // D, H), dtype=torch.float32, device="cuda")
            b.tsp_mlp_forward(plan, prob.X, prob.Wg, prob.Wu, prob.Wd, Y, S, D)
            b.tsp_mlp_backward(plan, prob.X, prob.Wg, prob.Wu, prob.Wd, prob.dY, dX, dWg, dWu, dWd, S, D)
            torch.cuda.synchronize()
            assert b.tsp_mlp_status(plan) == b.TSP_OK
            outs.append((Y, dX))
    finally:
        b.tsp_mlp_plan_destroy(plan)
    return outs


def _same_bits(a, c):
    import torch

    return torch.equal(a.view(torch.int16), c.view(torch.int16))


# every position a two-rank tile (option bit 2); D = 2 is the shortest ring (three slots), the third shape has two
# token tiles per rank, the fourth an 8-rank ring, the last a ragged last token tile per rank (1000 tokens = 3 tiles + 232 rows)
@pytest.mark.parametrize("S,H,F,D", [(512, 512, 1024, 2), (1024, 256, 1536, 4), (2048, 256, 1536, 4), (2048, 512, 2048, 8),
                                     (4000, 256, 1536, 4)])
def test_two_rank_tiles_keep_every_bit_and_match_the_oracle(S, H, F, D):
    prob = DeviceProblem(S, H, F, D, seed=61, with_dy=True)
    one_rank = _run(prob, reps=1, rank_pair_tiles=0)[0]
    for Y, dX in _run(prob, rank_pair_tiles=7):
        assert _same_bits(Y, one_rank[0])
        assert _same_bits(dX, one_rank[1])
    X, Wg, Wu, Wd, dY = prob.f64()
    assert rel_fro(tensor_to_f64(one_rank[0]), orc.gated_mlp_forward(X, Wg, Wu, Wd)) <= 1e-2
    assert rel_fro(tensor_to_f64(one_rank[1]), orc.gated_mlp_backward(X, Wg, Wu, Wd, dY)[0]) <= 1e-2


# 96 positions on 74 CTA pairs: one round of two-rank tiles, then 44 one-rank tiles on alternating accumulators
def test_mixed_list_of_two_rank_and_one_rank_tiles():
    prob = DeviceProblem(3072, 4096, 768, 6, seed=62, with_dy=True)
    one_rank = _run(prob, reps=1, rank_pair_tiles=0)[0]
    for Y, dX in _run(prob, rank_pair_tiles=3):
        assert _same_bits(Y, one_rank[0])
        assert _same_bits(dX, one_rank[1])
    X, Wg, Wu, Wd, dY = prob.f64()
    assert rel_fro(tensor_to_f64(one_rank[0]), orc.gated_mlp_forward(X, Wg, Wu, Wd)) <= 1e-2


# the 7B-shaped training configuration: 222 two-rank tiles + 68 one-rank tiles per kernel
def test_7b_shape_same_bits_as_one_rank_tiles():
    prob = DeviceProblem(8192, 4096, 14336, 8, seed=63, with_dy=True)
    one_rank = _run(prob, reps=1, rank_pair_tiles=0)[0]
    for Y, dX in _run(prob, rank_pair_tiles=3):
        assert _same_bits(Y, one_rank[0])
        assert _same_bits(dX, one_rank[1])


# odd D, many token tiles per rank, or a static hand-out: the option is ignored and the one-rank kernels run
@pytest.mark.parametrize("S,H,F,D,extra", [(768, 256, 768, 3, {}), (9216, 256, 512, 2, {}), (1024, 256, 1024, 4, {"dynamic_tiles": 0})])
def test_option_is_ignored_where_ranks_do_not_pair_up(S, H, F, D, extra):
    prob = DeviceProblem(S, H, F, D, seed=64, with_dy=True)
    one_rank = _run(prob, reps=1, rank_pair_tiles=0, **extra)[0]
    Y, dX = _run(prob, reps=1, rank_pair_tiles=7, **extra)[0]
    assert _same_bits(Y, one_rank[0])
    assert _same_bits(dX, one_rank[1])
