"""tsp_mlp_forward_static: the forward for callers that cannot allocate device memory.

Some users of the library run where a device allocation is impossible or unwelcome: inside a host
framework that has already taken the whole GPU for its own pool (cudaMalloc fails), on a
latency-critical path that cannot accept the device-wide synchronisation an allocation implies, or
under a rule that forbids allocating after start-up.  For them the library offers one entry point
whose scratch (the bf16 intermediate and the status word) is a fixed array inside the library.

This file is collected last on purpose, so that a run stopping at the first failure has already run
every other test.  It checks the new entry point against tsp_mlp_forward through the C ABI on two
calls in a row (the shared array keeps the first call's contents), and that an oversized problem is
refused with a clear error.
"""
import ctypes

import numpy as np
import pytest

from oracle import tsp_mlp_oracle as orc
from paper_2604_26294_b200 import binding as b
from paper_2604_26294_b200 import build
from tests.helpers import DeviceProblem, rel_fro, tensor_to_f64

pytestmark = pytest.mark.gpu

TOL = 1e-2  # relative Frobenius tolerance used by the other forward parity tests


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build_library()


def _static_forward(prob):
    import torch

    Y = torch.full((prob.S, prob.H), float("nan"), dtype=torch.bfloat16, device="cuda")
    flag = ctypes.c_int(-1)
    b.tsp_mlp_forward_static(prob.H, prob.F, prob.D, prob.X, prob.Wg, prob.Wu, prob.Wd, Y, prob.S, flag)
    torch.cuda.synchronize()
    assert flag.value == 0, "a device-side wait expired"
    return Y


def test_static_forward_matches_plan_forward_on_two_calls_in_a_row():
    import torch

    # first call: 512 x 1536 intermediate; second call: a different, smaller problem, so stale scratch would show
    probs = [DeviceProblem(512, 512, 1536, 4, seed=11), DeviceProblem(256, 256, 768, 2, seed=12)]
    for i, prob in enumerate(probs):
        free_before = torch.cuda.mem_get_info()[0]
        got = _static_forward(prob)
        if i == 1:
            # by the second call every kernel is loaded: the call itself must not have taken device memory
            assert torch.cuda.mem_get_info()[0] == free_before
        want = prob.forward()
        g, w = tensor_to_f64(got), tensor_to_f64(want)
        assert np.all(np.isfinite(g))
        assert rel_fro(g, w) <= TOL, rel_fro(g, w)
        assert bool((got.view(torch.int16) == want.view(torch.int16)).all())  # same kernels, same order: same bits
        assert rel_fro(g, orc.gated_mlp_forward(*prob.f64())) <= TOL


def test_static_forward_refuses_what_does_not_fit():
    import torch

    # S * F * 2 bytes = 16 MiB > 8 MiB of fixed scratch: refused before any launch, with its own error code
    S, H, F, D = 2048, 256, 4096, 2
    assert S * F * 2 > b.TSP_MLP_STATIC_SCRATCH_BYTES
    x = torch.zeros(16, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(b.TspError) as err:
        b.tsp_mlp_forward_static(H, F, D, x, x, x, x, x, S)
    assert err.value.code == b.TSP_ERR_STATIC_LIMIT
    assert "fixed scratch" in str(err.value)
    # shape rules still come first (101 tokens cannot be split into 2 equal shards)
    with pytest.raises(b.TspError) as err:
        b.tsp_mlp_forward_static(H, F, D, x, x, x, x, x, 101)
    assert err.value.code == b.TSP_ERR_UNSUPPORTED_SHAPE


def test_static_forward_without_flag_and_on_a_side_stream():
    import torch

    # a caller on a latency-critical path passes no flag (nothing makes the host wait) or a flag in pinned memory,
    # and usually launches on a stream of its own
    prob = DeviceProblem(256, 256, 768, 2, seed=13)
    want = prob.forward()
    side = torch.cuda.Stream()
    pinned = torch.full((1,), -1, dtype=torch.int32).pin_memory()
    for flag in (None, ctypes.cast(pinned.data_ptr(), ctypes.POINTER(ctypes.c_int)).contents):
        Y = torch.full((prob.S, prob.H), float("nan"), dtype=torch.bfloat16, device="cuda")
        torch.cuda.synchronize()
        with torch.cuda.stream(side):
            b.tsp_mlp_forward_static(prob.H, prob.F, prob.D, prob.X, prob.Wg, prob.Wu, prob.Wd, Y, prob.S, flag, side)
        side.synchronize()
        assert bool((Y.view(torch.int16) == want.view(torch.int16)).all())
    assert int(pinned[0]) == 0
    assert b.tsp_mlp_last_cuda_error(None) == 0
