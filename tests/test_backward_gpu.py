"""Parity of tsp_mlp_backward (CUDA, through the C ABI) with the CPU fp64 oracle."""
import numpy as np
import pytest

from oracle import tsp_mlp_oracle as orc
from paper_2604_26294_b200 import build
from paper_2604_26294_b200 import inputs as inp
from tests.helpers import TOL_ROW, DeviceProblem, rel_fro, tensor_to_f64, worst_row_error

pytestmark = pytest.mark.gpu

TOL_ORACLE = 1e-2    # relative Frobenius error vs the fp64 oracle, every output
TOL_ACROSS_D = 5e-3  # relative Frobenius difference between runs with different D


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build_library()


def _grads(prob):
    dX, dWg, dWu, dWd = prob.backward()
    return (tensor_to_f64(dX), inp.unshard_columns(tensor_to_f64(dWg)), inp.unshard_columns(tensor_to_f64(dWu)),
            inp.unshard_rows(tensor_to_f64(dWd)))


def _check_full(S, H, F, D, seed=0):
    prob = DeviceProblem(S, H, F, D, seed=seed, with_dy=True)
    got = _grads(prob)
    ref = orc.gated_mlp_backward(*prob.f64())
    for name, g, r in zip(("dX", "dWg", "dWu", "dWd"), got, ref):
        assert g.shape == r.shape, name
        assert np.all(np.isfinite(g)), name
        assert rel_fro(g, r) <= TOL_ORACLE, (name, rel_fro(g, r))
        assert worst_row_error(g, r) <= TOL_ROW, (name, worst_row_error(g, r))
    return got


def test_tiny_config_full_compare():
    _check_full(256, 256, 768, 2, seed=0)


@pytest.mark.parametrize("S,H,F,D", [
    (128, 256, 128, 1),
    (512, 512, 1536, 4),
    (1536, 768, 1280, 2),
    (2048, 256, 2048, 16),
    (2304, 256, 1536, 3),    # D = 3, pair path incl. the split backward (F % 256 == 0) and pair dW (512 per shard)
    (2304, 256, 1152, 3),    # D = 3, pair tokens but 384-wide shards: single-CTA dW, fused single-CTA gate kernel
    (3840, 512, 1280, 5),    # D = 5
])
def test_multi_tile_shapes_full_compare(S, H, F, D):
    _check_full(S, H, F, D, seed=1)


@pytest.mark.parametrize("S,H,F,D", [
    (80, 256, 256, 2),       # 40 tokens per rank
    (600, 256, 768, 2),      # 300 tokens per rank: single-CTA path; dW contracts the tokens in ascending order
    (2000, 256, 1024, 2),    # 1000 tokens per rank: CTA pairs, split backward, pair dW with a zero-filled tail k-block
    (1536, 256, 768, 3),     # 512 per rank (control: multiple of every tile size)
    (1304, 256, 512, 4),     # 326 tokens per rank
])
def test_ragged_token_counts_full_compare(S, H, F, D):
    _check_full(S, H, F, D, seed=7)


def test_wide_tiles_forced():
    # 256 x 512 tiles for the down projection, dX and dW (normally chosen from the tile counts; forced by a plan option)
    S, H, F, D = 1024, 1024, 1024, 2
    prob = DeviceProblem(S, H, F, D, seed=8, with_dy=True, options={"wide_mask": 7})
    Y = tensor_to_f64(prob.forward())
    X, Wg, Wu, Wd, dY = prob.f64()
    assert rel_fro(Y, orc.gated_mlp_forward(X, Wg, Wu, Wd)) <= TOL_ORACLE
    got = _grads(prob)
    ref = orc.gated_mlp_backward(X, Wg, Wu, Wd, dY)
    for name, g, r in zip(("dX", "dWg", "dWu", "dWd"), got, ref):
        assert rel_fro(g, r) <= TOL_ORACLE, (name, rel_fro(g, r))
        assert worst_row_error(g, r) <= TOL_ROW, name
    narrow = _grads(DeviceProblem(S, H, F, D, host=prob.host, with_dy=True, options={"wide_mask": 0}))
    for g, n in zip(got, narrow):
        assert rel_fro(g, n) <= 1e-6     # same accumulation order, same bits expected


def test_more_tiles_than_sms():
    _check_full(20480, 256, 512, 4, seed=2)


def test_gradients_agree_across_D():
    S, H, F = 2048, 512, 2048
    host = inp.make_inputs(S, H, F, seed=3, with_dy=True)
    outs = {D: _grads(DeviceProblem(S, H, F, D, host=host, with_dy=True)) for D in (1, 2, 4, 8, 16)}
    for D, got in outs.items():
        for name, g, g1 in zip(("dX", "dWg", "dWu", "dWd"), got, outs[1]):
            assert rel_fro(g, g1) <= TOL_ACROSS_D, (D, name, rel_fro(g, g1))


def test_euler_identities_hold_on_gpu_output():
    # <dWu, Wu> = <dWd, Wd> = <dY, Y>: ties the backward outputs to the forward output
    prob = DeviceProblem(512, 512, 1536, 4, seed=6, with_dy=True)
    _, dWg, dWu, dWd = _grads(prob)
    X, Wg, Wu, Wd, dY = prob.f64()
    Y = tensor_to_f64(prob.forward())
    L = float(np.sum(dY * Y))
    scale = np.linalg.norm(dY) * np.linalg.norm(Y)
    assert abs(np.sum(dWu * Wu) - L) <= 1e-2 * scale
    assert abs(np.sum(dWd * Wd) - L) <= 1e-2 * scale


def test_zero_upstream_gradient_gives_zero_gradients():
    prob = DeviceProblem(256, 256, 768, 2, seed=5, with_dy=True)
    prob.dY.zero_()
    for g in prob.backward():
        assert float(g.float().abs().max()) == 0.0
