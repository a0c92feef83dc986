"""STAGED mode: Algorithm 2 step by step, the shard transfer emulated by copies on a second stream."""
import numpy as np
import pytest

from oracle import tsp_mlp_oracle as orc
from paper_2604_26294_b200 import binding as b
from paper_2604_26294_b200 import build
from paper_2604_26294_b200 import inputs as inp
from tests.helpers import TOL_ROW, DeviceProblem, rel_fro, tensor_to_f64, worst_row_error

pytestmark = pytest.mark.gpu

TOL_ORACLE = 1e-2
TOL_MODES = 5e-3   # staged vs direct differ only in fp32 summation order


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build_library()


def _staged(prob):
    import torch

    S, H, F, D = prob.S, prob.H, prob.F, prob.D
    plan = b.tsp_mlp_plan(H, F, D)
    try:
        nbytes = b.tsp_mlp_workspace_bytes_staged(plan, S)
        ws = torch.zeros(nbytes, dtype=torch.uint8, device="cuda")
        b.tsp_mlp_set_workspace(plan, ws)
        Y = torch.full((S, H), float("nan"), dtype=torch.bfloat16, device="cuda")
        compute, copy = torch.cuda.Stream(), torch.cuda.Stream()
        compute.wait_stream(torch.cuda.current_stream())
        for _ in range(2):   # twice: events and receive buffers are reused across calls
            b.tsp_mlp_forward_staged(plan, prob.X, prob.Wg, prob.Wu, prob.Wd, Y, S, D, compute, copy)
        compute.synchronize()
        copy.synchronize()
        assert b.tsp_mlp_status(plan) == b.TSP_OK
    finally:
        b.tsp_mlp_plan_destroy(plan)
    return Y, ws


@pytest.mark.parametrize("S,H,F,D", [(256, 256, 256, 1), (512, 256, 512, 2), (1024, 512, 1536, 4), (2048, 256, 1024, 8),
                                     (2000, 256, 512, 2)])   # the last one: 1000 tokens per rank (ragged last tile)
def test_staged_forward_matches_oracle_and_direct(S, H, F, D):
    prob = DeviceProblem(S, H, F, D, seed=21)
    Y, ws = _staged(prob)
    got = tensor_to_f64(Y)
    ref = orc.gated_mlp_forward(*prob.f64())
    assert np.all(np.isfinite(got))
    assert rel_fro(got, ref) <= TOL_ORACLE, rel_fro(got, ref)
    assert worst_row_error(got, ref) <= TOL_ROW
    direct = tensor_to_f64(prob.forward())
    assert rel_fro(got, direct) <= TOL_MODES, rel_fro(got, direct)


def test_receive_buffers_hold_the_ring_rotated_shards():
    # after the last transfer (step D-2 -> D-1), rank r's current buffer holds shard (r - (D-1)) mod D = (r+1) mod D
    import torch

    S, H, F, D = 1024, 256, 512, 4
    prob = DeviceProblem(S, H, F, D, seed=22)
    _, ws = _staged(prob)
    F_d = F // D
    a_step = (S * F_d * 2 + 255) // 256 * 256
    y_acc = (S * H * 4 + 255) // 256 * 256
    w = (H * F * 2 + 255) // 256 * 256
    parity = (D - 1) & 1
    mats = (prob.Wg, prob.Wu, prob.Wd)
    for m in range(3):
        off = a_step + y_acc + (parity * 3 + m) * w
        buf = ws[off:off + H * F * 2].view(torch.bfloat16).view(D, -1)
        own = mats[m].reshape(D, -1)
        for r in range(D):
            assert bool((buf[r].view(torch.int16) == own[(r + 1) % D].view(torch.int16)).all()), (m, r)


def test_staged_refuses_one_stream_and_odd_shapes():
    import torch

    prob = DeviceProblem(256, 256, 768, 2, seed=0)    # 128 tokens per rank: the single-CTA kernels' territory
    plan = b.tsp_mlp_plan(256, 768, 2)
    try:
        ws = torch.empty(b.tsp_mlp_workspace_bytes_staged(plan, 256), dtype=torch.uint8, device="cuda")
        b.tsp_mlp_set_workspace(plan, ws)
        s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
        with pytest.raises(b.TspError) as err:
            b.tsp_mlp_forward_staged(plan, prob.X, prob.Wg, prob.Wu, prob.Wd, prob.Y, 256, 2, s1, s2)
        assert err.value.code == b.TSP_ERR_UNSUPPORTED_SHAPE
        with pytest.raises(b.TspError) as err:
            b.tsp_mlp_forward_staged(plan, prob.X, prob.Wg, prob.Wu, prob.Wd, prob.Y, 512, 2, s1, s1)
        assert err.value.code == b.TSP_ERR_INVALID_ARG
    finally:
        b.tsp_mlp_plan_destroy(plan)
