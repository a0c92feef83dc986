"""C-ABI behaviour on the GPU: argument checks, workspace rules, status word, ring table, profiling."""
import ctypes

import pytest

from paper_2604_26294_b200 import binding as b
from paper_2604_26294_b200 import build
from tests.helpers import DeviceProblem

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build_library()


@pytest.fixture()
def plan():
    p = b.tsp_mlp_plan(256, 768, 2)
    yield p
    b.tsp_mlp_plan_destroy(p)


def test_workspace_sizes(plan):
    S = 256
    fwd = b.tsp_mlp_workspace_bytes(plan, S, b.TSP_WS_FORWARD)
    bwd = b.tsp_mlp_workspace_bytes(plan, S, b.TSP_WS_BACKWARD)
    assert fwd >= S * 768 * 2 and fwd % 256 == 0
    assert bwd >= 3 * S * 768 * 2 + S * 768 * 4      # A, dG, dU in bf16 and dA in fp32
    assert b.tsp_mlp_workspace_bytes(plan, 0, 0) == 0 and b.tsp_mlp_workspace_bytes(plan, S, 7) == 0
    assert b.tsp_mlp_workspace_bytes_host(plan, S) > fwd


def test_forward_refuses_bad_calls_without_launching(plan):
    import torch

    prob = DeviceProblem(256, 256, 768, 2, seed=0)
    lib = b.load_library()
    args = [prob.X.data_ptr(), prob.Wg.data_ptr(), prob.Wu.data_ptr(), prob.Wd.data_ptr(), prob.Y.data_ptr()]
    stream = torch.cuda.current_stream().cuda_stream
    # no workspace yet
    assert lib.tsp_mlp_forward(plan, *args, 256, 2, stream) == b.TSP_ERR_WORKSPACE
    ws = torch.empty(b.tsp_mlp_workspace_bytes(plan, 256, 0), dtype=torch.uint8, device="cuda")
    # too small a workspace
    b.tsp_mlp_set_workspace(plan, ws, ws.numel() - 256)
    assert lib.tsp_mlp_forward(plan, *args, 256, 2, stream) == b.TSP_ERR_WORKSPACE
    # misaligned workspace pointer
    assert lib.tsp_mlp_set_workspace(plan, ws.data_ptr() + 16, 1024) == b.TSP_ERR_INVALID_ARG
    b.tsp_mlp_set_workspace(plan, ws)
    # D differs from the plan's; S not divisible into D equal token shards; null and misaligned pointers
    assert lib.tsp_mlp_forward(plan, *args, 256, 4, stream) == b.TSP_ERR_INVALID_ARG
    assert lib.tsp_mlp_forward(plan, *args, 255, 2, stream) == b.TSP_ERR_UNSUPPORTED_SHAPE
    assert lib.tsp_mlp_forward(plan, *args, 0, 2, stream) == b.TSP_ERR_INVALID_ARG
    assert lib.tsp_mlp_forward(plan, None, *args[1:], 256, 2, stream) == b.TSP_ERR_INVALID_ARG
    assert lib.tsp_mlp_forward(plan, args[0] + 2, *args[1:], 256, 2, stream) == b.TSP_ERR_INVALID_ARG
    # backward needs the larger workspace
    assert lib.tsp_mlp_backward(plan, *args[:4], args[0], args[4], args[0], args[0], args[0], 256, 2,
                                stream) == b.TSP_ERR_WORKSPACE
    torch.cuda.synchronize()
    assert b.tsp_mlp_status(plan) == b.TSP_OK
    # and a good call still works afterwards
    assert lib.tsp_mlp_forward(plan, *args, 256, 2, stream) == b.TSP_OK
    torch.cuda.synchronize()
    assert b.tsp_mlp_status(plan) == b.TSP_OK


def test_ring_order_table_matches_algorithm_2():
    for D in (1, 2, 4, 8):
        p = b.tsp_mlp_plan(256, 128 * D, D)
        try:
            table = b.tsp_mlp_ring_order(p, D)
        finally:
            b.tsp_mlp_plan_destroy(p)
        for r in range(D):
            assert table[r][0] == r
            assert sorted(table[r]) == list(range(D))
            for t in range(1, D):
                assert table[r][t] == table[(r - 1) % D][t - 1]   # what rank r holds came from rank r-1


def test_expired_device_wait_is_reported_and_plan_stays_usable(plan):
    import torch

    assert b.tsp_mlp_status(plan) == b.TSP_OK
    b.tsp_mlp_selftest_wait_expiry(plan, 20)
    torch.cuda.synchronize()
    assert b.tsp_mlp_status(plan) == b.TSP_ERR_DEVICE_TIMEOUT
    assert b.tsp_mlp_last_cuda_error(plan) == 6          # the self-test's wait code
    assert b.tsp_mlp_status(plan) == b.TSP_OK            # reading clears the word
    prob = DeviceProblem(256, 256, 768, 2, seed=0)
    ws = torch.empty(b.tsp_mlp_workspace_bytes(plan, 256, 0), dtype=torch.uint8, device="cuda")
    b.tsp_mlp_set_workspace(plan, ws)
    b.tsp_mlp_forward(plan, prob.X, prob.Wg, prob.Wu, prob.Wd, prob.Y, 256, 2)
    torch.cuda.synchronize()
    assert b.tsp_mlp_status(plan) == b.TSP_OK
    assert bool(torch.isfinite(prob.Y.float()).all())


def test_profile_events_cover_every_kernel(plan):
    import torch

    prob = DeviceProblem(256, 256, 768, 2, seed=0, with_dy=True)
    ws = torch.empty(b.tsp_mlp_workspace_bytes(plan, 256, 1), dtype=torch.uint8, device="cuda")
    b.tsp_mlp_set_workspace(plan, ws)
    dX = torch.empty(256, 256, dtype=torch.bfloat16, device="cuda")
    dWg = torch.empty(2, 256, 384, dtype=torch.float32, device="cuda")
    dWu = torch.empty_like(dWg)
    dWd = torch.empty(2, 384, 256, dtype=torch.float32, device="cuda")
    b.tsp_mlp_profile_begin(plan, 2)
    b.tsp_mlp_forward(plan, prob.X, prob.Wg, prob.Wu, prob.Wd, prob.Y, 256, 2)
    b.tsp_mlp_backward(plan, prob.X, prob.Wg, prob.Wu, prob.Wd, prob.dY, dX, dWg, dWu, dWd, 256, 2)
    b.tsp_mlp_forward(plan, prob.X, prob.Wg, prob.Wu, prob.Wd, prob.Y, 256, 2)   # beyond max_calls: not recorded
    torch.cuda.synchronize()
    fwd = b.tsp_mlp_profile_read(plan, 0)
    bwd = b.tsp_mlp_profile_read(plan, 1)
    assert len(fwd) == b.tsp_mlp_kernels_per_call(plan, b.TSP_WS_FORWARD) == 2
    assert len(bwd) == b.tsp_mlp_kernels_per_call(plan, b.TSP_WS_BACKWARD) == 3
    assert all(ms > 0 for ms in fwd + bwd)
    with pytest.raises(b.TspError):
        b.tsp_mlp_profile_read(plan, 2)
    b.tsp_mlp_profile_end(plan)


def test_host_buffer_forward_matches_device_forward():
    import numpy as np
    import torch

    from paper_2604_26294_b200 import inputs as inp

    S, H, F, D = 512, 256, 512, 2
    prob = DeviceProblem(S, H, F, D, seed=9)
    want = prob.forward().clone()
    p = b.tsp_mlp_plan(H, F, D)
    try:
        ws = torch.empty(b.tsp_mlp_workspace_bytes_host(p, S), dtype=torch.uint8, device="cuda")
        b.tsp_mlp_set_workspace(p, ws)
        h = prob.host
        hY = np.empty((S, H), dtype=np.uint16)
        b.tsp_mlp_forward_host(p, h.X, inp.shard_columns(h.Wg, D), inp.shard_columns(h.Wu, D),
                               inp.shard_rows(h.Wd, D), hY, S, D)
        torch.cuda.synchronize()
        assert b.tsp_mlp_status(p) == b.TSP_OK
    finally:
        b.tsp_mlp_plan_destroy(p)
    assert np.array_equal(hY, want.view(torch.int16).cpu().numpy().view(np.uint16))
