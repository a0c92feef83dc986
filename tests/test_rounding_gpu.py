"""The precision reading: G and U are never rounded (they live in tensor memory in fp32), the intermediate A (and dG, dU
in the backward pass) is rounded ONCE, to nearest-even, to bf16.  If G or U were rounded to bf16 before the product,
about half of the bf16 values of A would differ from the correctly rounded ones; with a single rounding only values
that sit next to a rounding boundary can differ, and then by one ulp."""
import numpy as np
import pytest

from oracle import tsp_mlp_oracle as orc
from paper_2604_26294_b200 import binding as b
from paper_2604_26294_b200 import build
from paper_2604_26294_b200 import inputs as inp
from tests.helpers import DeviceProblem

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build_library()


def _ulp_distance(bits_a: np.ndarray, bits_b: np.ndarray) -> np.ndarray:
    """Distance in bf16 steps between two bf16 bit patterns (sign-magnitude -> ordered integers)."""
    def ordered(u):
        u = u.astype(np.int32)
        return np.where(u & 0x8000, -(u & 0x7FFF), u & 0x7FFF)
    return np.abs(ordered(bits_a) - ordered(bits_b))


@pytest.mark.parametrize("S,H,F,D", [(256, 256, 768, 2), (1024, 512, 1536, 2)])   # single-CTA path, CTA-pair path
def test_intermediates_are_rounded_exactly_once(S, H, F, D):
    import torch

    prob = DeviceProblem(S, H, F, D, seed=51, with_dy=True)
    X, Wg, Wu, Wd, dY = prob.f64()
    G, U = X @ Wg, X @ Wu
    sG = orc.silu(G)
    dA = dY @ Wd.T
    want = {"A": sG * U, "dG": dA * U * orc.silu_prime(G), "dU": dA * sG}

    plan = b.tsp_mlp_plan(H, F, D)
    try:
        nbytes = b.tsp_mlp_workspace_bytes(plan, S, b.TSP_WS_BACKWARD)
        ws = torch.zeros(nbytes, dtype=torch.uint8, device="cuda")
        b.tsp_mlp_set_workspace(plan, ws)
        dX = torch.empty(S, H, dtype=torch.bfloat16, device="cuda")
        dWg = torch.empty(D, H, F // D, dtype=torch.float32, device="cuda")
        dWu = torch.empty_like(dWg)
        dWd = torch.empty(D, F // D, H, dtype=torch.float32, device="cuda")
        b.tsp_mlp_backward(plan, prob.X, prob.Wg, prob.Wu, prob.Wd, prob.dY, dX, dWg, dWu, dWd, S, D)
        torch.cuda.synchronize()
        assert b.tsp_mlp_status(plan) == b.TSP_OK
    finally:
        b.tsp_mlp_plan_destroy(plan)
    one = nbytes // 5      # workspace = A | dG | dU (bf16) | dA (fp32, two units)
    for i, name in enumerate(("A", "dG", "dU")):
        got = ws[i * one:i * one + S * F * 2].view(torch.int16).view(S, F).cpu().numpy().view(np.uint16)
        # shard-major columns of the workspace are the unsharded columns: shard k holds columns k*F/D..(k+1)*F/D
        ref_bits = inp.f32_to_bf16_bits(want[name].astype(np.float32))
        dist = _ulp_distance(got, ref_bits)
        exact = float(np.mean(dist == 0))
        assert exact >= 0.99, (name, exact)
        big = np.abs(want[name]) > 1e-3 * np.abs(want[name]).max()
        assert dist[big].max() <= 1, (name, int(dist[big].max()))
