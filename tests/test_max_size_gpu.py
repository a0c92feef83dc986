"""The largest token counts the library accepts: S = 2^24 tokens (forward) and element counts beyond 2^31 (backward).

At these sizes S*H and S*F reach 2^32 elements, so any 32-bit element or byte offset in a kernel or in the host code
would wrap.  Inputs are drawn on the GPU (seeded torch generator, the distributions of the input recipe); the fp64 CPU
oracle checks sampled token rows, chosen around the offsets where 32-bit arithmetic would wrap and at both ends.
The weight gradients are compared with the same formulas evaluated in fp64 by torch on the GPU, token chunk by token
chunk (that helper shares no code with the kernels and is itself checked against the CPU oracle at a small size first).
"""
import numpy as np
import pytest

from oracle import tsp_mlp_oracle as orc
from paper_2604_26294_b200 import binding as b
from paper_2604_26294_b200 import build
from tests.helpers import TOL_ROW, rel_fro, tensor_to_f64, worst_row_error

pytestmark = pytest.mark.gpu

TOL_ORACLE = 1e-2


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build_library()


def _draw(shape, std, gen, chunk_rows=1 << 20):
    import torch

    out = torch.empty(shape, dtype=torch.bfloat16, device="cuda")
    for r0 in range(0, shape[0], chunk_rows):
        r1 = min(shape[0], r0 + chunk_rows)
        out[r0:r1] = (torch.randn((r1 - r0,) + tuple(shape[1:]), device="cuda", generator=gen) * std).bfloat16()
    return out


def _rows_to_check(S, n_random, seed):
    rng = np.random.default_rng(seed)
    special = [0, 1, 255, 256, S // 2 - 1, S // 2, S // 2 + 1, S - 257, S - 256, S - 2, S - 1]
    rows = np.unique(np.concatenate([np.array(special), rng.integers(0, S, n_random)]))
    return rows[(rows >= 0) & (rows < S)]


def _all_finite(t, chunk_rows=1 << 20):
    import torch

    return all(bool(torch.isfinite(t[r0:r0 + chunk_rows].float()).all()) for r0 in range(0, t.shape[0], chunk_rows))


def test_forward_at_the_largest_token_count():
    import torch

    S, H, F, D = 1 << 24, 256, 256, 2          # X, Y, A: 2^32 elements each
    gen = torch.Generator(device="cuda")
    gen.manual_seed(11)
    X = _draw((S, H), 1.0, gen)
    Wg, Wu = _draw((D, H, F // D), H ** -0.5, gen), _draw((D, H, F // D), H ** -0.5, gen)
    Wd = _draw((D, F // D, H), F ** -0.5, gen)
    Y = torch.empty(S, H, dtype=torch.bfloat16, device="cuda")
    plan = b.tsp_mlp_plan(H, F, D)
    try:
        ws = torch.empty(b.tsp_mlp_workspace_bytes(plan, S, b.TSP_WS_FORWARD), dtype=torch.uint8, device="cuda")
        b.tsp_mlp_set_workspace(plan, ws)
        b.tsp_mlp_forward(plan, X, Wg, Wu, Wd, Y, S, D)
        torch.cuda.synchronize()
        assert b.tsp_mlp_status(plan) == b.TSP_OK
        with pytest.raises(b.TspError) as e:       # one rank's worth of tokens more is refused
            b.tsp_mlp_forward(plan, X, Wg, Wu, Wd, Y, S + D, D)
        assert e.value.code == b.TSP_ERR_UNSUPPORTED_SHAPE
    finally:
        b.tsp_mlp_plan_destroy(plan)
    assert _all_finite(Y)
    rows = _rows_to_check(S, 300, seed=1)
    idx = torch.from_numpy(rows).cuda()
    Wg64 = np.concatenate(list(tensor_to_f64(Wg)), axis=1)     # [D][H][F/D] -> [H, F]
    Wu64 = np.concatenate(list(tensor_to_f64(Wu)), axis=1)
    Wd64 = tensor_to_f64(Wd).reshape(F, H)
    ref = orc.gated_mlp_forward(tensor_to_f64(X[idx]), Wg64, Wu64, Wd64)
    got = tensor_to_f64(Y[idx])
    assert rel_fro(got, ref) <= TOL_ORACLE, rel_fro(got, ref)
    assert worst_row_error(got, ref) <= TOL_ROW


def _backward_fp64_on_gpu(X, Wg, Wu, Wd, dY, chunk=1 << 17):
    """dWg, dWu [H, F], dWd [F, H] of the plain definition in fp64 (torch, token chunks); SiLU gate."""
    import torch

    D, H, F_d = Wg.shape
    F = D * F_d
    Wg64 = Wg.double().permute(1, 0, 2).reshape(H, F)
    Wu64 = Wu.double().permute(1, 0, 2).reshape(H, F)
    Wd64 = Wd.double().reshape(F, H)
    dWg = torch.zeros(H, F, dtype=torch.float64, device="cuda")
    dWu = torch.zeros_like(dWg)
    dWd = torch.zeros(F, H, dtype=torch.float64, device="cuda")
    for r0 in range(0, X.shape[0], chunk):
        x, dy = X[r0:r0 + chunk].double(), dY[r0:r0 + chunk].double()
        G, U = x @ Wg64, x @ Wu64
        sig = torch.sigmoid(G)
        dA = dy @ Wd64.T
        dWd += (G * sig * U).T @ dy
        dWg += x.T @ (dA * U * sig * (1 + G * (1 - sig)))
        dWu += x.T @ (dA * G * sig)
    return dWg.cpu().numpy(), dWu.cpu().numpy(), dWd.cpu().numpy()


def _backward(S, H, F, D, seed):
    import torch

    gen = torch.Generator(device="cuda")
    gen.manual_seed(seed)
    X, dY = _draw((S, H), 1.0, gen), _draw((S, H), 1.0, gen)
    Wg, Wu = _draw((D, H, F // D), H ** -0.5, gen), _draw((D, H, F // D), H ** -0.5, gen)
    Wd = _draw((D, F // D, H), F ** -0.5, gen)
    dX = torch.empty(S, H, dtype=torch.bfloat16, device="cuda")
    dWg = torch.empty(D, H, F // D, dtype=torch.float32, device="cuda")
    dWu = torch.empty_like(dWg)
    dWd = torch.empty(D, F // D, H, dtype=torch.float32, device="cuda")
    plan = b.tsp_mlp_plan(H, F, D)
    try:
        ws = torch.empty(b.tsp_mlp_workspace_bytes(plan, S, b.TSP_WS_BACKWARD), dtype=torch.uint8, device="cuda")
        b.tsp_mlp_set_workspace(plan, ws)
        b.tsp_mlp_backward(plan, X, Wg, Wu, Wd, dY, dX, dWg, dWu, dWd, S, D)
        torch.cuda.synchronize()
        assert b.tsp_mlp_status(plan) == b.TSP_OK
    finally:
        b.tsp_mlp_plan_destroy(plan)
    del ws
    return X, Wg, Wu, Wd, dY, dX, dWg, dWu, dWd


def _unshard(Wg, Wu, Wd):
    D, H, F_d = Wg.shape
    return (np.concatenate(list(tensor_to_f64(Wg)), axis=1), np.concatenate(list(tensor_to_f64(Wu)), axis=1),
            tensor_to_f64(Wd).reshape(D * F_d, H))


def test_fp64_gpu_helper_agrees_with_the_cpu_oracle():
    X, Wg, Wu, Wd, dY, dX, dWg, dWu, dWd = _backward(1024, 256, 512, 2, seed=12)
    h = _backward_fp64_on_gpu(X, Wg, Wu, Wd, dY, chunk=300)
    Wg64, Wu64, Wd64 = _unshard(Wg, Wu, Wd)
    _, rWg, rWu, rWd = orc.gated_mlp_backward(tensor_to_f64(X), Wg64, Wu64, Wd64, tensor_to_f64(dY))
    for got, ref in zip(h, (rWg, rWu, rWd)):
        assert rel_fro(got, ref) <= 1e-12


def test_backward_beyond_2_31_elements():
    import torch

    S, H, F, D = 1 << 22, 256, 512, 2          # S*F = 2^31 elements: dA (fp32) spans 8 GiB, A / dG / dU 4 GiB each
    X, Wg, Wu, Wd, dY, dX, dWg, dWu, dWd = _backward(S, H, F, D, seed=13)
    assert _all_finite(dX)
    Wg64, Wu64, Wd64 = _unshard(Wg, Wu, Wd)
    rows = _rows_to_check(S, 200, seed=2)
    idx = torch.from_numpy(rows).cuda()
    rdX = orc.backward_rows(tensor_to_f64(X[idx]), Wg64, Wu64, Wd64, tensor_to_f64(dY[idx]), np.arange(len(rows)))
    got = tensor_to_f64(dX[idx])
    assert rel_fro(got, rdX) <= TOL_ORACLE, rel_fro(got, rdX)
    assert worst_row_error(got, rdX) <= TOL_ROW
    rWg, rWu, rWd = _backward_fp64_on_gpu(X, Wg, Wu, Wd, dY)
    gWg, gWu, gWd = _unshard(dWg, dWu, dWd)
    for g, r in ((gWg, rWg), (gWu, rWu), (gWd, rWd)):
        assert np.all(np.isfinite(g))
        # 1.7e-3 is the bf16 rounding of A, dG, dU; an unchunked contraction over 2^22 tokens would add a 4e-3 drift
        # towards zero (truncating tensor-core accumulation)
        assert rel_fro(g, r) <= 3e-3, rel_fro(g, r)
        assert worst_row_error(g, r) <= TOL_ROW


@pytest.mark.parametrize("S,D", [((1 << 18) + 320, 2), (3 * (1 << 18) - 64 * 3, 3)])
def test_weight_gradients_across_a_token_chunk_boundary(S, D):
    # just above the chunk length of the weight-gradient contraction: two / three launches, the later ones accumulating
    H, F = 256, 256 * D
    X, Wg, Wu, Wd, dY, dX, dWg, dWu, dWd = _backward(S, H, F, D, seed=15)
    rWg, rWu, rWd = _backward_fp64_on_gpu(X, Wg, Wu, Wd, dY)
    gWg, gWu, gWd = _unshard(dWg, dWu, dWd)
    for g, r in ((gWg, rWg), (gWu, rWu), (gWd, rWd)):
        assert np.all(np.isfinite(g))
        assert rel_fro(g, r) <= 3e-3, rel_fro(g, r)
        assert worst_row_error(g, r) <= TOL_ROW


def test_attention_projections_at_the_largest_token_count():
    import torch

    from oracle import tsp_attn_proj_oracle as aorc

    S, H, Hq, Hkv, D = 1 << 24, 256, 256, 256, 2
    gen = torch.Generator(device="cuda")
    gen.manual_seed(14)
    X, A, dY = _draw((S, H), 1.0, gen), _draw((S, Hq), 1.0, gen), _draw((S, H), 1.0, gen)
    Wq, Wk, Wv = (_draw((n, H), H ** -0.5, gen) for n in (Hq, Hkv, Hkv))
    Wo = _draw((D, H, Hq // D), Hq ** -0.5, gen)
    Q = torch.empty(S, Hq, dtype=torch.bfloat16, device="cuda")
    K, V = torch.empty(S, Hkv, dtype=torch.bfloat16, device="cuda"), torch.empty(S, Hkv, dtype=torch.bfloat16, device="cuda")
    Y, dA = torch.empty(S, H, dtype=torch.bfloat16, device="cuda"), torch.empty(S, Hq, dtype=torch.bfloat16, device="cuda")
    dWo = torch.empty(D, H, Hq // D, dtype=torch.float32, device="cuda")
    plan = b.tsp_attn_plan(H, Hq, Hkv, D)
    try:
        b.tsp_attn_qkv_forward(plan, X, Wq, Wk, Wv, Q, K, V, S, D)
        b.tsp_attn_out_forward(plan, A, Wo, Y, S, D)
        b.tsp_attn_out_backward(plan, A, Wo, dY, dA, dWo, S, D)
        torch.cuda.synchronize()
        assert b.tsp_attn_status(plan) == b.TSP_OK
        with pytest.raises(b.TspError) as e:
            b.tsp_attn_out_forward(plan, A, Wo, Y, S + 1, D)
        assert e.value.code == b.TSP_ERR_UNSUPPORTED_SHAPE
    finally:
        b.tsp_attn_plan_destroy(plan)
    rows = _rows_to_check(S, 300, seed=3)
    idx = torch.from_numpy(rows).cuda()
    Wo64 = np.concatenate(list(tensor_to_f64(Wo)), axis=1)     # [D][H][Hq/D] -> [H, Hq]
    rQ, rK, rV = aorc.qkv_projection(tensor_to_f64(X[idx]), tensor_to_f64(Wq), tensor_to_f64(Wk), tensor_to_f64(Wv))
    rY = aorc.output_projection(tensor_to_f64(A[idx]), Wo64)
    rdA, _ = aorc.output_projection_backward(tensor_to_f64(A[idx]), Wo64, tensor_to_f64(dY[idx]))
    for got, ref in ((Q, rQ), (K, rK), (V, rV), (Y, rY), (dA, rdA)):
        g = tensor_to_f64(got[idx])
        assert rel_fro(g, ref) <= 5e-3, rel_fro(g, ref)
        assert worst_row_error(g, ref) <= 0.05
        assert _all_finite(got)
    # dWo = dY^T A over all 2^24 tokens, against fp64 on the GPU in token chunks
    ref = torch.zeros(H, Hq, dtype=torch.float64, device="cuda")
    for r0 in range(0, S, 1 << 20):
        ref += dY[r0:r0 + (1 << 20)].double().T @ A[r0:r0 + (1 << 20)].double()
    got = np.concatenate(list(tensor_to_f64(dWo)), axis=1)
    assert rel_fro(got, ref.cpu().numpy()) <= 1e-3
