"""Parity of tsp_mlp_forward (CUDA, through the C ABI) with the CPU fp64 oracle."""
import numpy as np
import pytest

from oracle import tsp_mlp_oracle as orc
from paper_2604_26294_b200 import build
from paper_2604_26294_b200 import inputs as inp
from tests.helpers import TOL_ROW, DeviceProblem, rel_fro, tensor_to_f64, worst_row_error

pytestmark = pytest.mark.gpu

TOL_ORACLE = 1e-2   # relative Frobenius error vs the fp64 oracle (bf16 inputs, fp32 accumulation)
TOL_ACROSS_D = 5e-3  # relative Frobenius difference between runs with different D


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build_library()


def _check_full(S, H, F, D, seed=0):
    prob = DeviceProblem(S, H, F, D, seed=seed)
    Y = tensor_to_f64(prob.forward())
    ref = orc.gated_mlp_forward(*prob.f64())
    assert np.all(np.isfinite(Y))
    assert rel_fro(Y, ref) <= TOL_ORACLE, rel_fro(Y, ref)
    assert worst_row_error(Y, ref) <= TOL_ROW, worst_row_error(Y, ref)
    return Y


def test_tiny_config_full_compare():
    # D=2, S=256 (128 tokens per shard), H=256, F=768 (2 shards of 384), seed 0
    _check_full(256, 256, 768, 2, seed=0)


@pytest.mark.parametrize("S,H,F,D", [
    (128, 256, 128, 1),      # one tile of each kernel
    (512, 512, 1536, 4),     # several tiles, 3 column blocks per shard
    (1536, 768, 1280, 2),    # H = 3 x 256, 5 column blocks per shard, 12 token blocks
    (2048, 256, 2048, 16),   # D = 16 with the narrowest shard (128)
    (2304, 256, 1152, 3),    # D = 3: 768 tokens and 384 columns per rank, 9 pair tiles (odd), 3 column blocks
    (3840, 512, 1280, 5),    # D = 5: 15 pair tiles, band / group sizes do not divide the tile counts
    (384, 256, 384, 3),      # D = 3 on the single-CTA path (128 tokens per rank)
])
def test_multi_tile_shapes_full_compare(S, H, F, D):
    _check_full(S, H, F, D, seed=1)


@pytest.mark.parametrize("S,H,F,D", [
    (80, 256, 256, 2),       # 40 tokens per rank: one partial 128-row tile per rank
    (200, 256, 256, 1),      # 128 + 72 rows
    (600, 256, 768, 2),      # 300 tokens per rank: single-CTA tiling, 44-row tail
    (2000, 256, 1024, 2),    # 1000 tokens per rank: CTA pairs, 232-row tail tile
    (3000, 512, 768, 3),     # three ranks of 1000 tokens
    (1304, 256, 512, 4),     # 326 tokens per rank (not a multiple of 64 either)
])
def test_ragged_token_counts_full_compare(S, H, F, D):
    # any number of tokens per rank: the last tile of a rank is loaded whole but only its valid rows are stored
    _check_full(S, H, F, D, seed=7)


def test_more_tiles_than_sms():
    # 20480 rows -> 160 token blocks > 148 SMs: persistent CTAs take a second tile (both TMEM buffers, phase flip)
    _check_full(20480, 256, 512, 4, seed=2)


def test_results_agree_across_D():
    S, H, F = 2048, 512, 2048
    host = inp.make_inputs(S, H, F, seed=3)
    outs = {}
    for D in (1, 2, 4, 8, 16):
        outs[D] = tensor_to_f64(DeviceProblem(S, H, F, D, host=host).forward())
    ref = orc.gated_mlp_forward(*[inp.bf16_bits_to_f64(a) for a in (host.X, host.Wg, host.Wu, host.Wd)])
    for D, Y in outs.items():
        assert rel_fro(Y, ref) <= TOL_ORACLE
        assert rel_fro(Y, outs[1]) <= TOL_ACROSS_D, (D, rel_fro(Y, outs[1]))


def test_forward_is_deterministic():
    prob = DeviceProblem(512, 512, 1536, 4, seed=4)
    a = prob.forward().clone()
    b_ = prob.forward()
    assert bool((a.view(dtype=__import__("torch").int16) == b_.view(dtype=__import__("torch").int16)).all())


def test_zero_input_gives_zero_output():
    import torch

    prob = DeviceProblem(256, 256, 768, 2, seed=5)
    prob.X.zero_()
    assert float(prob.forward().float().abs().max()) == 0.0
    prob = DeviceProblem(256, 256, 768, 2, seed=5)
    prob.Wg.zero_()
    assert float(prob.forward().float().abs().max()) == 0.0
    assert torch.isfinite(prob.Y.float()).all()
