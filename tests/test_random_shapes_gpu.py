"""Seeded sweep over legal shapes: every path the shape allows (forward, recomputing backward, stored-activation
backward, staged forward) against the fp64 oracle.  The shapes are drawn once from a fixed seed so the test is
deterministic; they mix odd shard counts, tile counts that do not divide the band / group sizes, one and several
k-blocks per shard, ragged token counts per rank, and both kernel families (single CTA vs CTA pairs)."""
import numpy as np
import pytest

from oracle import tsp_mlp_oracle as orc
from paper_2604_26294_b200 import binding as b
from paper_2604_26294_b200 import build
from paper_2604_26294_b200 import inputs as inp
from tests.helpers import TOL_ROW, DeviceProblem, rel_fro, tensor_to_f64, worst_row_error

pytestmark = pytest.mark.gpu

TOL = 1e-2


def _shapes():
    rng = np.random.default_rng(20260426)
    out = []
    while len(out) < 18:
        D = int(rng.choice([1, 2, 3, 4, 5, 6, 8]))
        s_loc = int(rng.choice([72, 128, 200, 256, 384, 500, 512, 768, 1000]))
        H = int(rng.choice([256, 512, 768, 1024]))
        f_d = int(rng.choice([128, 256, 384, 512, 640]))
        S, F = D * s_loc, D * f_d
        if S * F > 3_000_000 or S * H * F > 2.5e9:
            continue
        out.append((S, H, F, D))
    return out


SHAPES = _shapes()


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build_library()


@pytest.mark.parametrize("S,H,F,D", SHAPES)
def test_every_available_path_matches_the_oracle(S, H, F, D):
    import torch

    prob = DeviceProblem(S, H, F, D, seed=S + H + F + D, with_dy=True)
    X, Wg, Wu, Wd, dY = prob.f64()
    Yref = orc.gated_mlp_forward(X, Wg, Wu, Wd)
    gref = orc.gated_mlp_backward(X, Wg, Wu, Wd, dY)

    def check(name, got, ref):
        assert np.all(np.isfinite(got)), name
        assert rel_fro(got, ref) <= TOL, (name, rel_fro(got, ref))
        assert worst_row_error(got, ref) <= TOL_ROW, name

    check("Y", tensor_to_f64(prob.forward()), Yref)
    dX, dWg, dWu, dWd = prob.backward()
    for n, g, r in zip(("dX", "dWg", "dWu", "dWd"),
                       (tensor_to_f64(dX), inp.unshard_columns(tensor_to_f64(dWg)), inp.unshard_columns(tensor_to_f64(dWu)),
                        inp.unshard_rows(tensor_to_f64(dWd))), gref):
        check(n, g, r)

    s_loc = S // D
    pair_tokens = ((s_loc + 255) // 256 * 256) * 100 <= ((s_loc + 127) // 128 * 128) * 106   # the library's own rule
    plan = b.tsp_mlp_plan(H, F, D)
    try:
        if pair_tokens:
            # staged forward
            ws = torch.empty(max(b.tsp_mlp_workspace_bytes_staged(plan, S), b.tsp_mlp_workspace_bytes(plan, S, 1)),
                             dtype=torch.uint8, device="cuda")
            b.tsp_mlp_set_workspace(plan, ws)
            Ys = torch.full((S, H), float("nan"), dtype=torch.bfloat16, device="cuda")
            cs, xs = torch.cuda.Stream(), torch.cuda.Stream()
            cs.wait_stream(torch.cuda.current_stream())
            b.tsp_mlp_forward_staged(plan, prob.X, prob.Wg, prob.Wu, prob.Wd, Ys, S, D, cs, xs)
            cs.synchronize()
            xs.synchronize()
            assert b.tsp_mlp_status(plan) == b.TSP_OK
            check("Y staged", tensor_to_f64(Ys), Yref)
        if pair_tokens and F % 256 == 0:
            # stored-activation training step
            saved = torch.empty(b.tsp_mlp_saved_bytes(plan, S), dtype=torch.uint8, device="cuda")
            ws = torch.empty(b.tsp_mlp_workspace_bytes(plan, S, 1), dtype=torch.uint8, device="cuda")
            b.tsp_mlp_set_workspace(plan, ws)
            Y2 = torch.full((S, H), float("nan"), dtype=torch.bfloat16, device="cuda")
            dX2 = torch.full((S, H), float("nan"), dtype=torch.bfloat16, device="cuda")
            g2 = [torch.full_like(t, float("nan")) for t in (dWg, dWu, dWd)]
            b.tsp_mlp_forward_save(plan, prob.X, prob.Wg, prob.Wu, prob.Wd, Y2, saved, S, D)
            b.tsp_mlp_backward_saved(plan, prob.X, prob.Wg, prob.Wu, prob.Wd, prob.dY, saved, dX2, *g2, S, D)
            torch.cuda.synchronize()
            assert b.tsp_mlp_status(plan) == b.TSP_OK
            check("Y stored", tensor_to_f64(Y2), Yref)
            for n, g, r in zip(("dX", "dWg", "dWu", "dWd"),
                               (tensor_to_f64(dX2), inp.unshard_columns(tensor_to_f64(g2[0])),
                                inp.unshard_columns(tensor_to_f64(g2[1])), inp.unshard_rows(tensor_to_f64(g2[2]))), gref):
                check(n + " stored", g, r)
    finally:
        b.tsp_mlp_plan_destroy(plan)
