"""The seeded generator: determinism, shapes and the stated distributions."""

import numpy as np

from paper_2609_33645_b200 import workloads as wl


def test_same_seed_same_bits_and_shapes():
    cfg = wl.reduced(wl.CONFIGS["c2"], V=4096, name="c2-small")
    a = wl.make_batch(cfg)
    b = wl.make_batch(cfg)
    for k in ("hidden", "W", "targets", "input_lengths", "target_lengths"):
        np.testing.assert_array_equal(getattr(a, k), getattr(b, k))
    assert a.hidden.shape == (cfg.N, int(a.input_lengths.max()), cfg.D)
    assert a.W.shape == (cfg.V, cfg.D)
    assert cfg.T_lo <= a.input_lengths.min() and a.input_lengths.max() <= cfg.T_hi
    assert cfg.U_lo <= a.target_lengths.min() and a.target_lengths.max() <= cfg.U_hi
    for n in range(cfg.N):
        row = a.targets[n, : a.target_lengths[n]]
        assert row.min() >= 1 and row.max() < cfg.V
        assert np.all(a.hidden[n, a.input_lengths[n]:] == 0)
    # values are exactly representable in bf16
    np.testing.assert_array_equal(wl.round_to_bf16(a.hidden), a.hidden)
    np.testing.assert_array_equal(wl.round_to_bf16(a.W), a.W)


def test_bf16_rounding_is_nearest_even():
    torch = __import__("torch")
    x = np.random.default_rng(0).standard_normal(10000).astype(np.float32) * 100
    ref = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    np.testing.assert_array_equal(wl.round_to_bf16(x), ref)
    bits = wl.bf16_bits(ref)
    np.testing.assert_array_equal((bits.astype(np.uint32) << 16).view(np.float32), ref)


def test_variants():
    cfg = wl.reduced(wl.CONFIGS["c3"], V=2048, D=64, T_div=8, name="c3-small", blank=5)
    b = wl.make_batch(cfg, with_bias=True, permute_ids=True, poison_padding=True)
    assert b.bias is not None and b.blank == 5
    for n in range(cfg.N):
        row = b.targets[n, : b.target_lengths[n]]
        assert np.all(row != 5) and row.min() >= 0 and row.max() < cfg.V
        if b.input_lengths[n] < b.T:
            assert np.all(np.abs(b.hidden[n, b.input_lengths[n]:]) > 1e4)
    # RMS-normalised frames
    h = b.hidden[0, : b.input_lengths[0]].astype(np.float64)
    np.testing.assert_allclose(np.sqrt((h ** 2).mean(1)), 1.0, atol=5e-3)
    # Zipf ids: adjacent repeats occur at full size
    full = wl.make_batch(wl.reduced(wl.CONFIGS["c2"], D=8, name="c2-thin"))
    reps = sum(int(np.sum(full.targets[n, 1:full.target_lengths[n]] == full.targets[n, :full.target_lengths[n] - 1]))
               for n in range(full.cfg.N))
    assert reps > 0
