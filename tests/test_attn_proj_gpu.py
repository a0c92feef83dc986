"""Projection GEMMs of TSP attention (Algorithm 1) on the GPU against the fp64 oracle, through the C ABI."""
import numpy as np
import pytest

from oracle import tsp_attn_proj_oracle as orc
from paper_2604_26294_b200 import binding as b
from paper_2604_26294_b200 import build
from paper_2604_26294_b200 import inputs as inp
from tests.helpers import bf16_tensor, rel_fro, tensor_to_f64, worst_row_error

pytestmark = pytest.mark.gpu

# bf16 inputs, fp32 accumulation, one bf16 rounding of the output: RMS relative error about 1.6e-3 (half an ulp of
# 2^-7 spread uniformly, mantissas in [1, 2))
TOL = 5e-3


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build_library()


def _run(S, H, Hq, Hkv, D, seed=0, host=None):
    import torch

    host = host if host is not None else inp.make_attn_inputs(S, H, Hq, Hkv, seed=seed)
    X, Wq, Wk, Wv, A = (bf16_tensor(a) for a in (host.X, host.Wq, host.Wk, host.Wv, host.A))
    Wo = bf16_tensor(inp.shard_out_columns(host.Wo, D))
    Q = torch.full((S, Hq), float("nan"), dtype=torch.bfloat16, device="cuda")
    K = torch.full((S, Hkv), float("nan"), dtype=torch.bfloat16, device="cuda")
    V = torch.full((S, Hkv), float("nan"), dtype=torch.bfloat16, device="cuda")
    Y = torch.full((S, H), float("nan"), dtype=torch.bfloat16, device="cuda")
    plan = b.tsp_attn_plan(H, Hq, Hkv, D)
    try:
        b.tsp_attn_qkv_forward(plan, X, Wq, Wk, Wv, Q, K, V, S, D)
        b.tsp_attn_out_forward(plan, A, Wo, Y, S, D)
        torch.cuda.synchronize()
        assert b.tsp_attn_status(plan) == b.TSP_OK
    finally:
        b.tsp_attn_plan_destroy(plan)
    return host, Q, K, V, Y


def _f64(host):
    return {n: inp.bf16_bits_to_f64(getattr(host, n)) for n in ("X", "Wq", "Wk", "Wv", "A", "Wo")}


@pytest.mark.parametrize("S,H,Hq,Hkv,D", [
    (256, 256, 512, 256, 2),       # the tiny workload
    (512, 256, 256, 256, 1),
    (768, 512, 1024, 256, 4),      # GQA, g = 4
    (1024, 256, 1536, 768, 3),     # shard width 512 / 256, three shards
    (1000, 256, 512, 512, 8),      # ragged last token tile (232 rows), shard width 64
    (77, 512, 256, 256, 2),        # fewer tokens than half a tile: the second CTA's rows are all padding
    (2304, 256, 256, 256, 4),      # more token tiles than one group / band
])
def test_projections_match_oracle(S, H, Hq, Hkv, D):
    host, Q, K, V, Y = _run(S, H, Hq, Hkv, D, seed=41)
    f = _f64(host)
    rQ, rK, rV = orc.qkv_projection(f["X"], f["Wq"], f["Wk"], f["Wv"])
    rY = orc.output_projection(f["A"], f["Wo"])
    for got, ref in ((Q, rQ), (K, rK), (V, rV), (Y, rY)):
        g = tensor_to_f64(got)
        assert np.all(np.isfinite(g))
        assert rel_fro(g, ref) <= TOL, rel_fro(g, ref)
        assert worst_row_error(g, ref) <= 0.05


def test_output_projection_agrees_across_shard_counts_and_is_deterministic():
    import torch

    S, H, Hq, Hkv = 512, 256, 1024, 1024
    host = inp.make_attn_inputs(S, H, Hq, Hkv, seed=42)
    outs = {}
    for D in (1, 2, 4, 8, 16):
        _, Q, _, _, Y = _run(S, H, Hq, Hkv, D, host=host)
        outs[D] = (Q, Y)
    for D in (2, 4, 8, 16):
        # the shard count only regroups an ascending contraction and the rows of Wq: nothing may change
        assert torch.equal(outs[D][0].view(torch.int16), outs[1][0].view(torch.int16))
        assert torch.equal(outs[D][1].view(torch.int16), outs[1][1].view(torch.int16))
    _, Q2, _, _, Y2 = _run(S, H, Hq, Hkv, 4, host=host)
    assert torch.equal(Y2.view(torch.int16), outs[4][1].view(torch.int16))
    assert torch.equal(Q2.view(torch.int16), outs[4][0].view(torch.int16))


def test_selector_weights_copy_columns_exactly():
    # 0/1 weights: every output is one input value, so the result must be bit-exact; a transposed or shifted
    # weight tile, or a wrong head-to-column mapping, shows as a wrong column
    import torch

    S, H, Hq, Hkv, D = 256, 256, 512, 256, 2
    host = inp.make_attn_inputs(S, H, Hq, Hkv, seed=43)
    rng = np.random.default_rng(7)
    one = inp.f32_to_bf16_bits(np.ones(1, dtype=np.float32))[0]
    pq, pk, pv, po = rng.integers(0, H, Hq), rng.integers(0, H, Hkv), rng.integers(0, H, Hkv), rng.integers(0, Hq, H)
    for W, perm in ((host.Wq, pq), (host.Wk, pk), (host.Wv, pv), (host.Wo, po)):
        W[...] = 0
        W[np.arange(len(perm)), perm] = one
    _, Q, K, V, Y = _run(S, H, Hq, Hkv, D, host=host)
    X = torch.from_numpy(host.X.view(np.int16)).cuda()
    A = torch.from_numpy(host.A.view(np.int16)).cuda()
    assert torch.equal(Q.view(torch.int16), X[:, torch.from_numpy(pq).cuda()])
    assert torch.equal(K.view(torch.int16), X[:, torch.from_numpy(pk).cuda()])
    assert torch.equal(V.view(torch.int16), X[:, torch.from_numpy(pv).cuda()])
    assert torch.equal(Y.view(torch.int16), A[:, torch.from_numpy(po).cuda()])


def test_plan_and_call_errors():
    import torch

    for bad in ((256, 512, 256, 0), (256, 512, 256, 65), (0, 512, 256, 2)):
        with pytest.raises(b.TspError) as e:
            b.tsp_attn_plan(*bad)
        assert e.value.code == b.TSP_ERR_INVALID_ARG
    for bad in ((128, 512, 256, 2), (256, 384, 256, 2), (256, 512, 128, 2), (256, 512, 256, 3), (256, 256, 256, 8)):
        with pytest.raises(b.TspError) as e:
            b.tsp_attn_plan(*bad)
        assert e.value.code == b.TSP_ERR_UNSUPPORTED_SHAPE
    plan = b.tsp_attn_plan(256, 256, 256, 2)
    try:
        x = torch.zeros(256, 256, dtype=torch.bfloat16, device="cuda")
        with pytest.raises(b.TspError) as e:
            b.tsp_attn_qkv_forward(plan, x, x, x, x, x, x, x, 256, 4)      # D differs from the plan's
        assert e.value.code == b.TSP_ERR_INVALID_ARG
        with pytest.raises(b.TspError) as e:
            b.tsp_attn_out_forward(plan, x, x, 0, 256, 2)                  # null output
        assert e.value.code == b.TSP_ERR_INVALID_ARG
        with pytest.raises(b.TspError) as e:
            b.tsp_attn_out_forward(plan, x, x, x, 0, 2)
        assert e.value.code == b.TSP_ERR_INVALID_ARG
        with pytest.raises(b.TspError) as e:
            b.tsp_attn_qkv_forward(plan, x.view(-1)[1:], x, x, x, x, x, x, 255, 2)   # misaligned X
        assert e.value.code == b.TSP_ERR_INVALID_ARG
    finally:
        b.tsp_attn_plan_destroy(plan)


@pytest.mark.parametrize("name", ["attn_7b_mha", "attn_7b_gqa4"])
def test_full_size_sampled_rows(name):
    wl = inp.ATTN_WORKLOADS[name]
    host, Q, K, V, Y = _run(wl.S, wl.H, wl.Hq, wl.Hkv, wl.D, seed=0)
    rows = inp.sample_rows(wl.S, wl.D, block=128, per_block=1, seed=3)
    f = _f64(host)
    rQ, rK, rV = orc.qkv_rows(f["X"], f["Wq"], f["Wk"], f["Wv"], rows)
    rY = orc.output_rows(f["A"], f["Wo"], rows)
    idx = __import__("torch").from_numpy(rows).cuda()
    for got, ref in ((Q, rQ), (K, rK), (V, rV), (Y, rY)):
        g = tensor_to_f64(got[idx])
        assert rel_fro(g, ref) <= TOL
        assert worst_row_error(g, ref) <= 0.05
        assert bool(__import__("torch").isfinite(got.float()).all())


# ------------------------------------------------------------------------------------------------------ backward
def _run_backward(S, H, Hq, Hkv, D, seed=0):
    import torch

    host = inp.make_attn_inputs(S, H, Hq, Hkv, seed=seed, with_grads=True)
    X, Wq, Wk, Wv, A = (bf16_tensor(a) for a in (host.X, host.Wq, host.Wk, host.Wv, host.A))
    dQ, dK, dV, dY = (bf16_tensor(a) for a in (host.dQ, host.dK, host.dV, host.dY))
    Wo = bf16_tensor(inp.shard_out_columns(host.Wo, D))
    nan = float("nan")
    dX = torch.full((S, H), nan, dtype=torch.bfloat16, device="cuda")
    dA = torch.full((S, Hq), nan, dtype=torch.bfloat16, device="cuda")
    dWq = torch.full((Hq, H), nan, dtype=torch.float32, device="cuda")
    dWk = torch.full((Hkv, H), nan, dtype=torch.float32, device="cuda")
    dWv = torch.full((Hkv, H), nan, dtype=torch.float32, device="cuda")
    dWo = torch.full((D, H, Hq // D), nan, dtype=torch.float32, device="cuda")
    plan = b.tsp_attn_plan(H, Hq, Hkv, D)
    try:
        b.tsp_attn_out_backward(plan, A, Wo, dY, dA, dWo, S, D)
        b.tsp_attn_qkv_backward(plan, X, Wq, Wk, Wv, dQ, dK, dV, dX, dWq, dWk, dWv, S, D)
        torch.cuda.synchronize()
        assert b.tsp_attn_status(plan) == b.TSP_OK
    finally:
        b.tsp_attn_plan_destroy(plan)
    return host, dX, dWq, dWk, dWv, dA, dWo


@pytest.mark.parametrize("S,H,Hq,Hkv,D", [
    (256, 256, 512, 256, 2),
    (512, 256, 256, 256, 1),
    (768, 512, 1024, 256, 4),
    (1024, 256, 1536, 768, 3),
    (1000, 256, 512, 512, 8),      # ragged token tail (also inside the last 64-token k-block), shard width 64
    (77, 512, 256, 256, 2),
    (4160, 256, 256, 256, 4),      # more token tiles than one group
])
def test_backward_matches_oracle(S, H, Hq, Hkv, D):
    host, dX, dWq, dWk, dWv, dA, dWo = _run_backward(S, H, Hq, Hkv, D, seed=44)
    f = _f64(host)
    g = {n: inp.bf16_bits_to_f64(getattr(host, n)) for n in ("dQ", "dK", "dV", "dY")}
    rdX, rdWq, rdWk, rdWv = orc.qkv_projection_backward(f["X"], f["Wq"], f["Wk"], f["Wv"], g["dQ"], g["dK"], g["dV"])
    rdA, rdWo = orc.output_projection_backward(f["A"], f["Wo"], g["dY"])
    got_dWo = inp.unshard_columns(tensor_to_f64(dWo))
    for name, got, ref in (("dX", tensor_to_f64(dX), rdX), ("dA", tensor_to_f64(dA), rdA),
                           ("dWq", tensor_to_f64(dWq), rdWq), ("dWk", tensor_to_f64(dWk), rdWk),
                           ("dWv", tensor_to_f64(dWv), rdWv), ("dWo", got_dWo, rdWo)):
        assert np.all(np.isfinite(got)), name
        # bf16 outputs carry one rounding (1.7e-3); the fp32 weight gradients only fp32 accumulation error
        tol = TOL if name in ("dX", "dA") else 1e-4
        assert rel_fro(got, ref) <= tol, (name, rel_fro(got, ref))
        assert worst_row_error(got, ref) <= 0.05, name


def test_backward_is_deterministic_and_independent_of_shard_count():
    import torch

    S, H, Hq, Hkv = 512, 256, 1024, 512
    ref = None
    for D in (1, 4, 16, 4):
        _, dX, dWq, dWk, dWv, dA, dWo = _run_backward(S, H, Hq, Hkv, D, seed=45)
        cur = (dX.view(torch.int16), dWq, dWk, dWv, dA.view(torch.int16),
               dWo.permute(1, 0, 2).reshape(H, Hq).contiguous())
        if ref is None:
            ref = cur
        else:
            for a, c in zip(ref, cur):
                assert torch.equal(a, c)   # the shard count only changes where dWo's columns are stored


def test_backward_argument_errors():
    import torch

    plan = b.tsp_attn_plan(256, 256, 256, 2)
    try:
        x = torch.zeros(256, 256, dtype=torch.bfloat16, device="cuda")
        w = torch.zeros(256, 256, dtype=torch.float32, device="cuda")
        with pytest.raises(b.TspError) as e:
            b.tsp_attn_qkv_backward(plan, x, x, x, x, x, x, x, x, w, w, 0, 256, 2)
        assert e.value.code == b.TSP_ERR_INVALID_ARG
        with pytest.raises(b.TspError) as e:
            b.tsp_attn_out_backward(plan, x, x, x, x, w.view(-1)[1:], 256, 2)     # fp32 output not 32-byte aligned
        assert e.value.code == b.TSP_ERR_INVALID_ARG
        with pytest.raises(b.TspError) as e:
            b.tsp_attn_out_backward(plan, x, x, x, x, w, 256, 3)
        assert e.value.code == b.TSP_ERR_INVALID_ARG
    finally:
        b.tsp_attn_plan_destroy(plan)


def test_random_shapes_and_tile_orders(monkeypatch):
    """Seeded sweep over shapes, ragged token counts and tile-order tunables (read when a plan is created); the
    reference here is the oracle's formulas evaluated per case on the CPU."""
    import random

    rnd = random.Random(7)
    tun = ("TSP_MLP_BAND", "TSP_MLP_CHUNK_BANDS", "TSP_MLP_CHUNK_TILES", "TSP_MLP_GROUP", "TSP_MLP_DX_GROUP", "TSP_MLP_DW_GROUP")
    done = 0
    while done < 16:
        D = rnd.choice([1, 2, 4, 8])
        H, Hq = rnd.choice([256, 512]), rnd.choice([512, 1024])
        Hkv = rnd.choice([h for h in (256, 512, 1024) if h <= Hq])
        S = rnd.choice([1, 63, 200, 257, 511, 777, 1300])
        for k in tun:
            monkeypatch.delenv(k, raising=False)
        if done % 4:      # every fourth case runs with the defaults
            monkeypatch.setenv("TSP_MLP_BAND", rnd.choice(["1", "2"]))
            monkeypatch.setenv("TSP_MLP_CHUNK_BANDS", rnd.choice(["0", "1", "2"]))
            monkeypatch.setenv("TSP_MLP_CHUNK_TILES", rnd.choice(["0", "1", "3"]))
            monkeypatch.setenv("TSP_MLP_GROUP", rnd.choice(["1", "3"]))
            monkeypatch.setenv("TSP_MLP_DX_GROUP", rnd.choice(["0", "2"]))
            monkeypatch.setenv("TSP_MLP_DW_GROUP", rnd.choice(["0", "1", "3"]))
        host, dX, dWq, dWk, dWv, dA, dWo = _run_backward(S, H, Hq, Hkv, D, seed=100 + done)
        _, Q, K, V, Y = _run(S, H, Hq, Hkv, D, host=host)
        f = _f64(host)
        g = {n: inp.bf16_bits_to_f64(getattr(host, n)) for n in ("dQ", "dK", "dV", "dY")}
        rQ, rK, rV = orc.qkv_projection(f["X"], f["Wq"], f["Wk"], f["Wv"])
        rY = orc.output_projection(f["A"], f["Wo"])
        rdX, rdWq, rdWk, rdWv = orc.qkv_projection_backward(f["X"], f["Wq"], f["Wk"], f["Wv"], g["dQ"], g["dK"], g["dV"])
        rdA, rdWo = orc.output_projection_backward(f["A"], f["Wo"], g["dY"])
        pairs = [(Q, rQ), (K, rK), (V, rV), (Y, rY), (dX, rdX), (dA, rdA), (dWq, rdWq), (dWk, rdWk), (dWv, rdWv),
                 (inp.unshard_columns(tensor_to_f64(dWo)), rdWo)]
        for got, ref in pairs:
            got = got if isinstance(got, np.ndarray) else tensor_to_f64(got)
            assert np.all(np.isfinite(got)), (S, H, Hq, Hkv, D)
            assert rel_fro(got, ref) <= TOL, (S, H, Hq, Hkv, D, rel_fro(got, ref))
        done += 1
