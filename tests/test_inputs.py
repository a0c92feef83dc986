"""The seeded input generator: bf16 rounding, layouts, determinism."""
import numpy as np
import torch

from paper_2604_26294_b200 import inputs as inp


def test_bf16_rounding_matches_torch_rne():
    rng = np.random.default_rng(0)
    a = rng.standard_normal(100000).astype(np.float32)
    # add exact ties: values halfway between two bf16 neighbours
    ties = (np.arange(1, 2001, dtype=np.uint32) << np.uint32(16) | np.uint32(0x8000)) + np.uint32(0x3F000000)
    a = np.concatenate([a, ties.view(np.float32)])
    ours = inp.f32_to_bf16_bits(a)
    theirs = torch.from_numpy(a).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(ours, theirs)
    back = inp.bf16_bits_to_f32(ours)
    assert np.array_equal(inp.f32_to_bf16_bits(back), ours)


def test_generator_is_seeded_and_independent_of_D():
    a = inp.make_inputs(64, 32, 48, seed=0, with_dy=True)
    b = inp.make_inputs(64, 32, 48, seed=0, with_dy=True)
    c = inp.make_inputs(64, 32, 48, seed=1)
    for f in ("X", "Wg", "Wu", "Wd", "dY"):
        assert np.array_equal(getattr(a, f), getattr(b, f))
    assert not np.array_equal(a.X, c.X)
    assert c.dY is None
    # draw order X, Wg, Wu, Wd, dY: a forward-only draw shares the first four tensors
    d = inp.make_inputs(64, 32, 48, seed=0)
    assert np.array_equal(a.Wd, d.Wd)


def test_distribution_scales():
    H, F = 256, 768
    x = inp.make_inputs(512, H, F, seed=3)
    assert abs(inp.bf16_bits_to_f64(x.X).std() - 1.0) < 0.02
    assert abs(inp.bf16_bits_to_f64(x.Wg).std() * H ** 0.5 - 1.0) < 0.02
    assert abs(inp.bf16_bits_to_f64(x.Wu).std() * H ** 0.5 - 1.0) < 0.02
    assert abs(inp.bf16_bits_to_f64(x.Wd).std() * F ** 0.5 - 1.0) < 0.02


def test_shard_layouts_round_trip():
    H, F, D = 8, 24, 4
    W = np.arange(H * F, dtype=np.uint16).reshape(H, F)
    Wk = inp.shard_columns(W, D)
    assert Wk.shape == (D, H, F // D)
    for k in range(D):
        assert np.array_equal(Wk[k], W[:, k * F // D:(k + 1) * F // D])
    assert np.array_equal(inp.unshard_columns(Wk), W)
    Wd = np.arange(F * H, dtype=np.uint16).reshape(F, H)
    Wdk = inp.shard_rows(Wd, D)
    for k in range(D):
        assert np.array_equal(Wdk[k], Wd[k * F // D:(k + 1) * F // D])
    assert np.array_equal(inp.unshard_rows(Wdk), Wd)


def test_samplers_cover_every_block_and_shard():
    rows = inp.sample_rows(1024, 8)
    assert len(rows) == 8 and all(i * 128 <= r < (i + 1) * 128 for i, r in enumerate(rows))
    cols = inp.sample_columns(768, 4, 16)
    assert set(c // 192 for c in cols) == {0, 1, 2, 3}
