"""Dynamic tile hand-out: CTA pairs draw list indices from a device counter instead of taking them round-robin.

Which pair runs a tile does not change what the tile computes (its K loop, hence its ring accumulation order, is a
function of the list index alone), so every output must keep every bit of the static kernels' result.
"""
import numpy as np
import pytest

from oracle import tsp_mlp_oracle as orc
from paper_2604_26294_b200 import binding as b
from paper_2604_26294_b200 import build
from paper_2604_26294_b200 import inputs as inp
from tests.helpers import DeviceProblem, rel_fro, tensor_to_f64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build_library()


def _run(prob, **options):
    import torch

    S, H, F, D = prob.S, prob.H, prob.F, prob.D
    plan = b.tsp_mlp_plan_ex(H, F, D, **options)
    try:
        ws = torch.empty(b.tsp_mlp_workspace_bytes(plan, S, b.TSP_WS_BACKWARD), dtype=torch.uint8, device="cuda")
        b.tsp_mlp_set_workspace(plan, ws)
        outs = []
        for rep in range(2):   # twice: the scheduler words must be back at zero after every launch
            Y = torch.full((S, H), float("nan"), dtype=torch.bfloat16, device="cuda")
            dX = torch.full((S, H), float("nan"), dtype=torch.bfloat16, device="cuda")
            dWg = torch.full((D, H, F // D), float("nan"), dtype=torch.float32, device="cuda")
            dWu = torch.full((D, H, F // D), float("nan"), dtype=torch.float32, device="cuda")
            dWd = torch.full((D, F // D, H), float("nan"), dtype=torch.float32, device="cuda")
            b.tsp_mlp_forward(plan, prob.X, prob.Wg, prob.Wu, prob.Wd, Y, S, D)
            b.tsp_mlp_backward(plan, prob.X, prob.Wg, prob.Wu, prob.Wd, prob.dY, dX, dWg, dWu, dWd, S, D)
            torch.cuda.synchronize()
            assert b.tsp_mlp_status(plan) == b.TSP_OK
            outs.append((Y, dX, dWg, dWu, dWd))
    finally:
        b.tsp_mlp_plan_destroy(plan)
    return outs


# the second shape gives every kernel several rounds of tiles (e.g. 8 token tiles x 28 column blocks for gate|up)
@pytest.mark.parametrize("S,H,F,D", [(512, 256, 1024, 2), (2048, 1024, 3584, 2), (1200, 512, 1536, 3)])
@pytest.mark.parametrize("wide", [0, 7])
def test_dynamic_hand_out_keeps_every_bit(S, H, F, D, wide):
    import torch

    def bits(t):
        return t.view(torch.int32) if t.dtype == torch.float32 else t.view(torch.int16)

    prob = DeviceProblem(S, H, F, D, seed=51, with_dy=True)
    static = _run(prob, dynamic_tiles=0, wide_mask=wide)[0]
    for outs in _run(prob, dynamic_tiles=15, wide_mask=wide):      # all four kernel kinds draw dynamically
        for got, want in zip(outs, static):
            assert torch.equal(bits(got), bits(want))
    X, Wg, Wu, Wd, dY = prob.f64()
    assert rel_fro(tensor_to_f64(static[0]), orc.gated_mlp_forward(X, Wg, Wu, Wd)) <= 1e-2
    rdX = orc.gated_mlp_backward(X, Wg, Wu, Wd, dY)[0]
    assert rel_fro(tensor_to_f64(static[1]), rdX) <= 1e-2
