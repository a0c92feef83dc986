"""Per-rank ring-step entry points: the D ranks of Algorithm 2 emulated one after the other on one GPU.

Every (rank, step) is its own call on one stream, so no kernel waits for another; the shards "travel" by index.
"""
import numpy as np
import pytest

from oracle import tsp_mlp_oracle as orc
from paper_2604_26294_b200 import binding as b
from paper_2604_26294_b200 import build
from paper_2604_26294_b200 import inputs as inp
from paper_2604_26294_b200 import ring
from tests.helpers import TOL_ROW, DeviceProblem, rel_fro, tensor_to_f64, worst_row_error

pytestmark = pytest.mark.gpu

TOL_ORACLE = 1e-2
TOL_MODES = 5e-3


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build_library()


def _rank_rows(t, r, S_loc):
    return t[r * S_loc:(r + 1) * S_loc]


def _ring_forward_emulated(prob, act=None):
    import torch

    S, H, F, D = prob.S, prob.H, prob.F, prob.D
    S_loc = S // D
    plan = b.tsp_mlp_plan(H, F, D)
    try:
        if act is not None:
            b.tsp_mlp_set_activation(plan, act)
        nbytes = b.tsp_mlp_workspace_bytes_ring(plan, S_loc, b.TSP_WS_FORWARD)
        ws = [torch.empty(nbytes, dtype=torch.uint8, device="cuda") for _ in range(D)]
        Y = torch.full((S, H), float("nan"), dtype=torch.bfloat16, device="cuda")
        for t in range(D):
            for r in range(D):
                k = ring.shard_at_step(r, t, D)
                b.tsp_mlp_set_workspace(plan, ws[r])
                b.tsp_mlp_ring_step(plan, _rank_rows(prob.X, r, S_loc), prob.Wg[k], prob.Wu[k], prob.Wd[k],
                                    _rank_rows(Y, r, S_loc), S_loc, t, D)
        torch.cuda.synchronize()
        assert b.tsp_mlp_status(plan) == b.TSP_OK
    finally:
        b.tsp_mlp_plan_destroy(plan)
    return Y


def _staged(prob):
    import torch

    S, H, F, D = prob.S, prob.H, prob.F, prob.D
    plan = b.tsp_mlp_plan(H, F, D)
    try:
        ws = torch.zeros(b.tsp_mlp_workspace_bytes_staged(plan, S), dtype=torch.uint8, device="cuda")
        b.tsp_mlp_set_workspace(plan, ws)
        Y = torch.full((S, H), float("nan"), dtype=torch.bfloat16, device="cuda")
        compute, copy = torch.cuda.Stream(), torch.cuda.Stream()
        compute.wait_stream(torch.cuda.current_stream())
        b.tsp_mlp_forward_staged(plan, prob.X, prob.Wg, prob.Wu, prob.Wd, Y, S, D, compute, copy)
        compute.synchronize()
        copy.synchronize()
        assert b.tsp_mlp_status(plan) == b.TSP_OK
    finally:
        b.tsp_mlp_plan_destroy(plan)
    return Y


@pytest.mark.parametrize("S,H,F,D", [(256, 256, 256, 1), (512, 256, 512, 2), (768, 512, 1152, 3), (2048, 256, 1024, 8),
                                     (2000, 256, 512, 2), (21, 256, 384, 3)])
def test_ring_steps_forward_match_oracle_and_staged(S, H, F, D):
    import torch

    prob = DeviceProblem(S, H, F, D, seed=31)
    Y = _ring_forward_emulated(prob)
    got = tensor_to_f64(Y)
    ref = orc.gated_mlp_forward(*prob.f64())
    assert np.all(np.isfinite(got))
    assert rel_fro(got, ref) <= TOL_ORACLE, rel_fro(got, ref)
    assert worst_row_error(got, ref) <= TOL_ROW
    if S // D >= 200:   # the staged entry point wants token counts the pair kernels take without much padding
        assert torch.equal(Y.view(torch.int16), _staged(prob).view(torch.int16))   # same kernels, same summation order
    direct = tensor_to_f64(prob.forward())
    assert rel_fro(got, direct) <= TOL_MODES


def test_ring_steps_forward_gelu():
    prob = DeviceProblem(512, 256, 768, 2, seed=32)
    got = tensor_to_f64(_ring_forward_emulated(prob, act=b.TSP_ACT_GELU))
    ref = orc.gated_mlp_forward(*prob.f64(), act="gelu")
    assert rel_fro(got, ref) <= TOL_ORACLE


def _ring_backward_emulated(prob, act=None):
    """Ranks in turn; the accumulator of shard k is one buffer that every rank holding k adds to (it 'travels')."""
    import torch

    S, H, F, D = prob.S, prob.H, prob.F, prob.D
    S_loc, F_d = S // D, F // D
    plan = b.tsp_mlp_plan(H, F, D)
    try:
        if act is not None:
            b.tsp_mlp_set_activation(plan, act)
        nbytes = b.tsp_mlp_workspace_bytes_ring(plan, S_loc, b.TSP_WS_BACKWARD)
        ws = [torch.empty(nbytes, dtype=torch.uint8, device="cuda") for _ in range(D)]
        dX = torch.full((S, H), float("nan"), dtype=torch.bfloat16, device="cuda")
        dWg = torch.full((D, H, F_d), float("nan"), dtype=torch.float32, device="cuda")
        dWu = torch.full((D, H, F_d), float("nan"), dtype=torch.float32, device="cuda")
        dWd = torch.full((D, F_d, H), float("nan"), dtype=torch.float32, device="cuda")
        for t in range(D):
            for r in range(D):
                k = ring.shard_at_step(r, t, D)
                b.tsp_mlp_set_workspace(plan, ws[r])
                Xr, dYr = _rank_rows(prob.X, r, S_loc), _rank_rows(prob.dY, r, S_loc)
                b.tsp_mlp_ring_step_backward_dx(plan, Xr, prob.Wg[k], prob.Wu[k], prob.Wd[k], dYr,
                                                _rank_rows(dX, r, S_loc), S_loc, t, D)
                b.tsp_mlp_ring_step_backward_dw(plan, Xr, dYr, dWg[k], dWu[k], dWd[k], S_loc, int(t > 0), D)
        torch.cuda.synchronize()
        assert b.tsp_mlp_status(plan) == b.TSP_OK
    finally:
        b.tsp_mlp_plan_destroy(plan)
    return dX, dWg, dWu, dWd


@pytest.mark.parametrize("S,H,F,D", [(256, 256, 256, 1), (512, 256, 512, 2), (768, 512, 2304, 3), (2048, 256, 2048, 8),
                                     (600, 256, 512, 2), (63, 256, 768, 3)])
def test_ring_steps_backward_match_oracle_and_single_call(S, H, F, D):
    prob = DeviceProblem(S, H, F, D, seed=33, with_dy=True)
    dX, dWg, dWu, dWd = _ring_backward_emulated(prob)
    rdX, rdWg, rdWu, rdWd = orc.gated_mlp_backward(*prob.f64())
    sX, sWg, sWu, sWd = prob.backward()
    got_x = tensor_to_f64(dX)
    assert np.all(np.isfinite(got_x))
    assert rel_fro(got_x, rdX) <= TOL_ORACLE
    assert worst_row_error(got_x, rdX) <= TOL_ROW
    assert rel_fro(got_x, tensor_to_f64(sX)) <= TOL_MODES
    for got, ref_full, single, unshard in ((dWg, rdWg, sWg, inp.unshard_columns), (dWu, rdWu, sWu, inp.unshard_columns),
                                           (dWd, rdWd, sWd, inp.unshard_rows)):
        g = unshard(tensor_to_f64(got))
        assert np.all(np.isfinite(g))
        assert rel_fro(g, ref_full) <= TOL_ORACLE
        assert rel_fro(g, unshard(tensor_to_f64(single))) <= TOL_MODES


def test_ring_steps_backward_gelu():
    prob = DeviceProblem(512, 256, 512, 2, seed=35, with_dy=True)
    dX, dWg, dWu, dWd = _ring_backward_emulated(prob, act=b.TSP_ACT_GELU)
    rdX, rdWg, rdWu, rdWd = orc.gated_mlp_backward(*prob.f64(), act="gelu")
    assert rel_fro(tensor_to_f64(dX), rdX) <= TOL_ORACLE
    assert rel_fro(inp.unshard_columns(tensor_to_f64(dWg)), rdWg) <= TOL_ORACLE
    assert rel_fro(inp.unshard_columns(tensor_to_f64(dWu)), rdWu) <= TOL_ORACLE
    assert rel_fro(inp.unshard_rows(tensor_to_f64(dWd)), rdWd) <= TOL_ORACLE


def test_ring_mlp_object_single_rank():
    # D = 1 needs no transport: the class drives the step kernels directly
    import torch

    S, H, F = 384, 256, 512
    prob = DeviceProblem(S, H, F, 1, seed=34, with_dy=True)
    m = ring.TspRingMlp(H, F, 1, 0, S, training=True)
    try:
        shard = ring.pack_shard(prob.Wg[0], prob.Wu[0], prob.Wd[0])
        Y = m.forward(prob.X, shard)
        dX, (dWg, dWu, dWd) = m.backward(prob.X, shard, prob.dY)
        torch.cuda.synchronize()
        assert b.tsp_mlp_status(m.plan) == b.TSP_OK
    finally:
        m.close()
    X, Wg, Wu, Wd, dY = prob.f64()
    assert rel_fro(tensor_to_f64(Y), orc.gated_mlp_forward(X, Wg, Wu, Wd)) <= TOL_ORACLE
    rdX, rdWg, rdWu, rdWd = orc.gated_mlp_backward(X, Wg, Wu, Wd, dY)
    assert rel_fro(tensor_to_f64(dX), rdX) <= TOL_ORACLE
    assert rel_fro(tensor_to_f64(dWg), rdWg) <= TOL_ORACLE
    assert rel_fro(tensor_to_f64(dWu), rdWu) <= TOL_ORACLE
    assert rel_fro(tensor_to_f64(dWd), rdWd) <= TOL_ORACLE


def test_ring_step_argument_errors():
    import torch

    H, F, D, S_loc = 256, 768, 2, 128   # F/D = 384: fine for the forward step, not for the backward steps
    plan = b.tsp_mlp_plan(H, F, D)
    try:
        x = torch.zeros(S_loc, H, dtype=torch.bfloat16, device="cuda")
        wg = torch.zeros(H, F // D, dtype=torch.bfloat16, device="cuda")
        wd = torch.zeros(F // D, H, dtype=torch.bfloat16, device="cuda")
        y = torch.empty_like(x)
        with pytest.raises(b.TspError) as e:
            b.tsp_mlp_ring_step(plan, x, wg, wg, wd, y, S_loc, 0, D)
        assert e.value.code == b.TSP_ERR_WORKSPACE
        ws = torch.empty(b.tsp_mlp_workspace_bytes_ring(plan, S_loc, b.TSP_WS_BACKWARD), dtype=torch.uint8, device="cuda")
        b.tsp_mlp_set_workspace(plan, ws)
        for bad_t in (-1, D):
            with pytest.raises(b.TspError) as e:
                b.tsp_mlp_ring_step(plan, x, wg, wg, wd, y, S_loc, bad_t, D)
            assert e.value.code == b.TSP_ERR_INVALID_ARG
        with pytest.raises(b.TspError) as e:
            b.tsp_mlp_ring_step(plan, x, wg, wg, wd, y, S_loc, 0, D + 1)
        assert e.value.code == b.TSP_ERR_INVALID_ARG
        with pytest.raises(b.TspError) as e:
            b.tsp_mlp_ring_step_backward_dx(plan, x, wg, wg, wd, x, y, S_loc, 0, D)
        assert e.value.code == b.TSP_ERR_UNSUPPORTED_SHAPE
        dw = torch.empty(H, F // D, dtype=torch.float32, device="cuda")
        dwd = torch.empty(F // D, H, dtype=torch.float32, device="cuda")
        with pytest.raises(b.TspError) as e:
            b.tsp_mlp_ring_step_backward_dw(plan, x, x, dw, dw, dwd, S_loc, 0, D)
        assert e.value.code == b.TSP_ERR_UNSUPPORTED_SHAPE
        assert b.tsp_mlp_workspace_bytes_ring(plan, 0, b.TSP_WS_FORWARD) == 0
    finally:
        b.tsp_mlp_plan_destroy(plan)


def test_gate_and_down_halves_on_two_streams_keep_the_bits():
    # one rank, all shards local: the down projection of step t on a second stream overlaps the gate|up GEMM of
    # step t + 1 (ordering by events, as the header prescribes); the result must equal the one-stream sequence
    import torch

    S_loc, H, F, D = 512, 256, 2048, 8
    prob = DeviceProblem(S_loc, H, F, D, seed=36)       # X of one rank; D shards
    plan = b.tsp_mlp_plan(H, F, D)
    try:
        ws = torch.empty(b.tsp_mlp_workspace_bytes_ring(plan, S_loc, b.TSP_WS_FORWARD), dtype=torch.uint8, device="cuda")
        b.tsp_mlp_set_workspace(plan, ws)
        Y1 = torch.full((S_loc, H), float("nan"), dtype=torch.bfloat16, device="cuda")
        for t in range(D):
            k = ring.shard_at_step(0, t, D)
            b.tsp_mlp_ring_step(plan, prob.X, prob.Wg[k], prob.Wu[k], prob.Wd[k], Y1, S_loc, t, D)
        torch.cuda.synchronize()
        Y2 = torch.full((S_loc, H), float("nan"), dtype=torch.bfloat16, device="cuda")
        s_gate, s_down = torch.cuda.Stream(), torch.cuda.Stream()
        gate_done = [torch.cuda.Event() for _ in range(D)]
        down_done = [torch.cuda.Event() for _ in range(D)]
        for rep in range(2):                              # twice: the scratch buffers are reused across passes
            s_gate.wait_stream(s_down)
            for t in range(D):
                k = ring.shard_at_step(0, t, D)
                if t >= 2:
                    s_gate.wait_event(down_done[t - 2])
                b.tsp_mlp_ring_step_gate(plan, prob.X, prob.Wg[k], prob.Wu[k], S_loc, t, D, s_gate)
                gate_done[t].record(s_gate)
                s_down.wait_event(gate_done[t])
                b.tsp_mlp_ring_step_down(plan, prob.Wd[k], Y2, S_loc, t, D, s_down)
                down_done[t].record(s_down)
            s_down.synchronize()
            s_gate.synchronize()
            assert b.tsp_mlp_status(plan) == b.TSP_OK
            assert torch.equal(Y1.view(torch.int16), Y2.view(torch.int16))
            Y2.fill_(float("nan")) if rep == 0 else None
        with pytest.raises(b.TspError) as e:
            b.tsp_mlp_ring_step_down(plan, prob.Wd[0], 0, S_loc, 0, D)
        assert e.value.code == b.TSP_ERR_INVALID_ARG
    finally:
        b.tsp_mlp_plan_destroy(plan)
    # and against the definition: rank 0 of a problem whose other ranks' tokens do not matter for these rows
    X, Wg, Wu, Wd = prob.f64()
    ref = orc.gated_mlp_forward(X, Wg, Wu, Wd)
    assert rel_fro(tensor_to_f64(Y1), ref) <= TOL_ORACLE


@pytest.mark.parametrize("S_loc,H,F,D,n", [(512, 256, 2048, 8, 4), (1000, 256, 1024, 4, 2), (300, 512, 768, 6, 3),
                                           (256, 256, 1280, 5, 2), (64, 256, 512, 4, 4)])
def test_grouped_ring_steps_match_oracle_and_single_steps(S_loc, H, F, D, n):
    # one rank, its D shards in packed buffers a constant distance apart, n ring steps per call
    import torch

    prob = DeviceProblem(S_loc, H, F, D, seed=37)
    F_d = F // D
    order = [ring.shard_at_step(0, t, D) for t in range(D)]                 # the order rank 0 meets the shards
    slot = 3 * H * F_d + 64                                                  # some slack between the packed buffers
    packed = torch.zeros(D, slot, dtype=torch.bfloat16, device="cuda")
    for t, k in enumerate(order):
        packed[t, :3 * H * F_d] = ring.pack_shard(prob.Wg[k], prob.Wu[k], prob.Wd[k])
    plan = b.tsp_mlp_plan(H, F, D)
    try:
        nbytes = max(b.tsp_mlp_workspace_bytes_ring_group(plan, S_loc, n), b.tsp_mlp_workspace_bytes_ring(plan, S_loc, 0))
        ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        b.tsp_mlp_set_workspace(plan, ws)
        Yg = torch.full((S_loc, H), float("nan"), dtype=torch.bfloat16, device="cuda")
        for t0 in range(0, D, n):
            m = min(n, D - t0)                                               # the last group may be shorter
            Wg, Wu, Wd = ring.unpack_shard(packed[t0], H, F_d)
            b.tsp_mlp_ring_steps(plan, prob.X, Wg, Wu, Wd, slot, m, Yg, S_loc, t0, D)
        Ys = torch.full((S_loc, H), float("nan"), dtype=torch.bfloat16, device="cuda")
        for t, k in enumerate(order):
            b.tsp_mlp_ring_step(plan, prob.X, prob.Wg[k], prob.Wu[k], prob.Wd[k], Ys, S_loc, t, D)
        torch.cuda.synchronize()
        assert b.tsp_mlp_status(plan) == b.TSP_OK
        with pytest.raises(b.TspError) as e:
            b.tsp_mlp_ring_steps(plan, prob.X, prob.Wg[0], prob.Wu[0], prob.Wd[0], slot, 2, Yg, S_loc, D - 1, D)
        assert e.value.code == b.TSP_ERR_INVALID_ARG                         # t_first + n > D
        with pytest.raises(b.TspError) as e:
            b.tsp_mlp_ring_steps(plan, prob.X, prob.Wg[0], prob.Wu[0], prob.Wd[0], 12, 2, Yg, S_loc, 0, D)
        assert e.value.code == b.TSP_ERR_INVALID_ARG                         # stride shorter than a matrix
    finally:
        b.tsp_mlp_plan_destroy(plan)
    X, Wg64, Wu64, Wd64 = prob.f64()
    ref = orc.gated_mlp_forward(X, Wg64, Wu64, Wd64)
    got = tensor_to_f64(Yg)
    assert np.all(np.isfinite(got))
    assert rel_fro(got, ref) <= TOL_ORACLE, rel_fro(got, ref)
    assert worst_row_error(got, ref) <= TOL_ROW
    assert rel_fro(got, tensor_to_f64(Ys)) <= TOL_MODES


@pytest.mark.parametrize("S_loc,H,F,D,n", [(1024, 1024, 7168, 4, 1), (1024, 512, 3584, 2, 2), (300, 512, 768, 6, 3),
                                           (2304, 256, 1024, 4, 4), (40, 256, 512, 4, 1)])
def test_fused_ring_steps_keep_the_bits_of_the_two_launch_path(S_loc, H, F, D, n):
    # One launch per call (gate|up tiles, then down-projection tiles that wait for their token rows of A) against
    # the two-launch path selected by a plan option: same tiles, same K order, same epilogues, so the same bits.
    # Three passes with the fused plan: the ready counters alternate between two sets and must come back clean.
    import torch

    prob = DeviceProblem(S_loc, H, F, D, seed=38)
    F_d = F // D
    order = [ring.shard_at_step(0, t, D) for t in range(D)]
    packed = torch.stack([ring.pack_shard(prob.Wg[k], prob.Wu[k], prob.Wd[k]) for k in order])
    results = {}
    for fused in (1, 0):
        plan = b.tsp_mlp_plan_ex(H, F, D, fuse_ring_steps=fused)
        try:
            nbytes = max(b.tsp_mlp_workspace_bytes_ring_group(plan, S_loc, n),
                         b.tsp_mlp_workspace_bytes_ring(plan, S_loc, b.TSP_WS_FORWARD))
            ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
            b.tsp_mlp_set_workspace(plan, ws)
            outs = []
            for rep in range(3 if fused else 1):
                Y = torch.full((S_loc, H), float("nan"), dtype=torch.bfloat16, device="cuda")
                ws.fill_(0xFF)                                   # stale scratch must not matter
                if n == 1:
                    for t, k in enumerate(order):
                        b.tsp_mlp_ring_step(plan, prob.X, prob.Wg[k], prob.Wu[k], prob.Wd[k], Y, S_loc, t, D)
                else:
                    for t0 in range(0, D, n):
                        Wg, Wu, Wd = ring.unpack_shard(packed[t0], H, F_d)
                        b.tsp_mlp_ring_steps(plan, prob.X, Wg, Wu, Wd, packed.shape[1], min(n, D - t0), Y, S_loc, t0, D)
                torch.cuda.synchronize()
                assert b.tsp_mlp_status(plan) == b.TSP_OK
                outs.append(Y)
            calls = D if n == 1 else (D + n - 1) // n
            assert b.tsp_mlp_kernels_per_call(plan, b.TSP_WS_FORWARD) == (1 if fused else 2), calls
            results[fused] = outs
        finally:
            b.tsp_mlp_plan_destroy(plan)
    for Y in results[1]:
        assert torch.equal(Y.view(torch.int16), results[0][0].view(torch.int16))
    X, Wg64, Wu64, Wd64 = prob.f64()
    ref = orc.gated_mlp_forward(X, Wg64, Wu64, Wd64)
    got = tensor_to_f64(results[1][0])
    assert rel_fro(got, ref) <= TOL_ORACLE, rel_fro(got, ref)
    assert worst_row_error(got, ref) <= TOL_ROW


def _backward_grouped_emulated(prob, g):
    """All D ranks through the grouped backward calls: per group every rank runs its _dx call, then the accumulators
    take their hops step by step (shard k at step t is at rank (k + t) mod D, which adds its share)."""
    import torch

    S, H, F, D = prob.S, prob.H, prob.F, prob.D
    S_loc, F_d = S // D, F // D
    plan = b.tsp_mlp_plan(H, F, D)
    try:
        nbytes = b.tsp_mlp_workspace_bytes_ring_group_backward(plan, S_loc, g)
        ws = [torch.empty(nbytes, dtype=torch.uint8, device="cuda") for _ in range(D)]
        dX = torch.full((S, H), float("nan"), dtype=torch.bfloat16, device="cuda")
        dW = torch.full((D, 3 * H * F_d), float("nan"), dtype=torch.float32, device="cuda")
        slot = 3 * H * F_d
        for t0 in range(0, D, g):
            n = min(g, D - t0)
            for r in range(D):
                order = [ring.shard_at_step(r, t0 + i, D) for i in range(n)]
                packed = torch.stack([ring.pack_shard(prob.Wg[k], prob.Wu[k], prob.Wd[k]) for k in order])
                Wg, Wu, Wd = ring.unpack_shard(packed[0], H, F_d)
                b.tsp_mlp_set_workspace(plan, ws[r])
                b.tsp_mlp_ring_steps_backward_dx(plan, _rank_rows(prob.X, r, S_loc), Wg, Wu, Wd, slot, n,
                                                 _rank_rows(prob.dY, r, S_loc), _rank_rows(dX, r, S_loc), S_loc, t0, D)
                torch.cuda.synchronize()           # `packed` is a temporary
            for i in range(n):
                for r in range(D):
                    k = ring.shard_at_step(r, t0 + i, D)
                    gWg, gWu, gWd = ring.unpack_shard(dW[k], H, F_d)
                    b.tsp_mlp_set_workspace(plan, ws[r])
                    b.tsp_mlp_ring_steps_backward_dw(plan, _rank_rows(prob.X, r, S_loc), _rank_rows(prob.dY, r, S_loc),
                                                     gWg, gWu, gWd, S_loc, i, n, int(t0 + i > 0), D)
        torch.cuda.synchronize()
        assert b.tsp_mlp_status(plan) == b.TSP_OK
    finally:
        b.tsp_mlp_plan_destroy(plan)
    parts = [ring.unpack_shard(dW[k], H, F_d) for k in range(D)]
    return (dX, torch.stack([p[0] for p in parts]), torch.stack([p[1] for p in parts]), torch.stack([p[2] for p in parts]))


@pytest.mark.parametrize("S,H,F,D,g", [(2048, 256, 2048, 8, 4), (768, 512, 2304, 3, 2), (600, 256, 512, 2, 2),
                                       (1280, 256, 1280, 5, 2), (1024, 512, 2048, 4, 1), (4096, 1024, 7168, 4, 4)])
def test_grouped_backward_ring_steps_match_oracle_and_single_steps(S, H, F, D, g):
    import torch

    prob = DeviceProblem(S, H, F, D, seed=39, with_dy=True)
    dX, dWg, dWu, dWd = _backward_grouped_emulated(prob, g)
    sX, sWg, sWu, sWd = _ring_backward_emulated(prob)           # one step per call
    # the weight gradients are computed and accumulated by the same kernel in the same order: every bit agrees
    for got, want in ((dWg, sWg), (dWu, sWu), (dWd, sWd)):
        assert torch.equal(got.view(torch.int32), want.view(torch.int32))
    # dX sums the shards of a group in tensor memory before the fp32 carry is added: same order, other grouping
    if g == 1:
        assert torch.equal(dX.view(torch.int16), sX.view(torch.int16))
    assert rel_fro(tensor_to_f64(dX), tensor_to_f64(sX)) <= TOL_MODES
    rdX, rdWg, rdWu, rdWd = orc.gated_mlp_backward(*prob.f64())
    got_x = tensor_to_f64(dX)
    assert np.all(np.isfinite(got_x))
    assert rel_fro(got_x, rdX) <= TOL_ORACLE
    assert worst_row_error(got_x, rdX) <= TOL_ROW
    for got, ref_full, unshard in ((dWg, rdWg, inp.unshard_columns), (dWu, rdWu, inp.unshard_columns),
                                   (dWd, rdWd, inp.unshard_rows)):
        gg = unshard(tensor_to_f64(got))
        assert np.all(np.isfinite(gg))
        assert rel_fro(gg, ref_full) <= TOL_ORACLE


def test_grouped_backward_argument_errors():
    import torch

    H, F, D, S_loc = 256, 1024, 4, 128
    plan = b.tsp_mlp_plan(H, F, D)
    try:
        x = torch.zeros(S_loc, H, dtype=torch.bfloat16, device="cuda")
        w = torch.zeros(3 * H * F // D, dtype=torch.bfloat16, device="cuda")
        Wg, Wu, Wd = ring.unpack_shard(w, H, F // D)
        dw = torch.zeros(3 * H * F // D, dtype=torch.float32, device="cuda")
        gWg, gWu, gWd = ring.unpack_shard(dw, H, F // D)
        with pytest.raises(b.TspError) as e:
            b.tsp_mlp_ring_steps_backward_dx(plan, x, Wg, Wu, Wd, w.numel(), 2, x, x.clone(), S_loc, 0, D)
        assert e.value.code == b.TSP_ERR_WORKSPACE
        ws = torch.empty(b.tsp_mlp_workspace_bytes_ring_group_backward(plan, S_loc, 2), dtype=torch.uint8, device="cuda")
        b.tsp_mlp_set_workspace(plan, ws)
        with pytest.raises(b.TspError) as e:
            b.tsp_mlp_ring_steps_backward_dx(plan, x, Wg, Wu, Wd, w.numel(), 2, x, x.clone(), S_loc, D - 1, D)
        assert e.value.code == b.TSP_ERR_INVALID_ARG            # t_first + n > D
        with pytest.raises(b.TspError) as e:
            b.tsp_mlp_ring_steps_backward_dw(plan, x, x, gWg, gWu, gWd, S_loc, 2, 2, 0, D)
        assert e.value.code == b.TSP_ERR_INVALID_ARG            # shard 2 of a group of 2
        assert b.tsp_mlp_workspace_bytes_ring_group_backward(plan, S_loc, D + 1) == 0
    finally:
        b.tsp_mlp_plan_destroy(plan)


@pytest.mark.parametrize("S_loc,H,F,D", [(1024, 512, 2048, 4), (300, 256, 768, 3), (40, 256, 1024, 4), (2304, 256, 512, 2)])
def test_carried_sums_through_the_tma_unit_keep_the_bits(S_loc, H, F, D):
    # The per-step calls carry fp32 partial sums (Yacc, dXacc) from launch to launch.  By default they are stored, added
    # (by the memory system) and read back through the TMA unit; the plan option selects element-wise accesses from
    # registers instead.  Either way every step adds once in fp32 round-to-nearest, so the results agree bit for bit,
    # ragged token counts (rows clipped by the TMA unit) included.
    import torch

    prob = DeviceProblem(S_loc, H, F, D, seed=40, with_dy=True)
    outs = {}
    for tma in (1, 0):
        plan = b.tsp_mlp_plan_ex(H, F, D, tma_carry=tma)
        try:
            nbytes = max(b.tsp_mlp_workspace_bytes_ring(plan, S_loc, b.TSP_WS_BACKWARD),
                         b.tsp_mlp_workspace_bytes_ring(plan, S_loc, b.TSP_WS_FORWARD))
            ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
            b.tsp_mlp_set_workspace(plan, ws)
            Y = torch.full((S_loc, H), float("nan"), dtype=torch.bfloat16, device="cuda")
            dX = torch.full((S_loc, H), float("nan"), dtype=torch.bfloat16, device="cuda")
            dW = torch.empty(3 * H * (F // D), dtype=torch.float32, device="cuda")
            gWg, gWu, gWd = ring.unpack_shard(dW, H, F // D)
            for rep in range(2):                       # twice: staging buffers and barriers are reused across calls
                for t in range(D):
                    b.tsp_mlp_ring_step(plan, prob.X, prob.Wg[t], prob.Wu[t], prob.Wd[t], Y, S_loc, t, D)
                if (F // D) % 256 == 0:
                    for t in range(D):          # one accumulator for all shards: written at t = 0, added to afterwards
                        b.tsp_mlp_ring_step_backward_dx(plan, prob.X, prob.Wg[t], prob.Wu[t], prob.Wd[t], prob.dY, dX, S_loc, t, D)
                        b.tsp_mlp_ring_step_backward_dw(plan, prob.X, prob.dY, gWg, gWu, gWd, S_loc, int(t > 0), D)
            torch.cuda.synchronize()
            assert b.tsp_mlp_status(plan) == b.TSP_OK
            outs[tma] = (Y, dX, dW)
        finally:
            b.tsp_mlp_plan_destroy(plan)
    assert torch.equal(outs[1][0].view(torch.int16), outs[0][0].view(torch.int16))
    if (F // D) % 256 == 0:
        assert torch.equal(outs[1][1].view(torch.int16), outs[0][1].view(torch.int16))
        assert bool(torch.isfinite(outs[1][2]).all())
        assert torch.equal(outs[1][2].view(torch.int32), outs[0][2].view(torch.int32))    # weight gradients (sum over shards)
    # shards were applied in index order 0 .. D-1 here: any order gives the same Y up to rounding
    ref = orc.gated_mlp_forward(*prob.f64()[:4])
    assert rel_fro(tensor_to_f64(outs[1][0]), ref) <= TOL_ORACLE
