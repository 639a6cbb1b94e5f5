"""The seeded generators: reproducible, of the stated distributions, and free of
the method's arithmetic (they only draw numbers and pack notification bits)."""
import numpy as np

from paper_2203_17063_b200 import inputs


def test_reproducible_and_distinct_streams():
    a = inputs.normal_f32(1002, 3, 1000)
    b = inputs.normal_f32(1002, 3, 1000)
    c = inputs.normal_f32(1002, 4, 1000)
    assert np.array_equal(a, b) and not np.array_equal(a, c)
    bufs = inputs.rank_buffers("normal_f32", 1002, 6, 1000)
    assert np.array_equal(bufs[3], a)


def test_distributions():
    u = inputs.uniform_f32(1, 0, 200000)
    assert u.dtype == np.float32 and u.min() >= -1 and u.max() < 1 and abs(u.mean()) < 0.01
    g = inputs.normal_f32(1, 0, 200000)
    assert abs(g.mean()) < 0.01 and abs(g.std() - 1) < 0.01
    b = inputs.normal_bf16_bits(1, 0, 200000, 1e-3)
    w = inputs.bf16_bits_to_f32(b)
    assert b.dtype == np.uint16 and abs(w.std() / 1e-3 - 1) < 0.02
    i = inputs.int64_below(1, 0, 100000)
    assert i.min() >= 0 and i.max() < (1 << 20)
    f = inputs.int64_full_range(1, 0, 100000)
    assert f.min() < -(2 ** 62) and f.max() > 2 ** 62


def test_bf16_rounding_is_nearest_even():
    x = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 2 ** -7, 1.0 + 3 * 2 ** -8, -2.5, 3.0e38], dtype=np.float32)
    w = inputs.bf16_bits_to_f32(inputs.f32_to_bf16_bits(x))
    # 1 + 2^-8 is a tie between 1 and 1 + 2^-7 -> even (1); 1 + 3*2^-8 is a tie -> even (1 + 2^-6)
    assert w.tolist()[:5] == [1.0, 1.0, 1.0 + 2 ** -7, 1.0 + 2 ** -6, -2.5]


def test_schedule_and_masks():
    P, S = 70, 500
    rounds = inputs.arrival_rounds(2002, P, S, 0.7)
    assert rounds.min() == 1 and rounds.max() == 3
    assert abs((rounds == 1).mean() - 0.7) < 0.02
    assert abs((rounds == 2).mean() - 0.15) < 0.02
    masks = inputs.cumulative_masks(rounds)
    assert len(masks) == 3 and masks[0].shape == (S, 2)
    for t, m in enumerate(masks, 1):
        for r in (0, 63, 64, 69):
            bits = (m[:, r // 64] >> np.uint64(r % 64)) & np.uint64(1)
            assert np.array_equal(bits.astype(bool), rounds[r] <= t)
        assert (m[:, 1] >> np.uint64(6) == 0).all()          # no bits at or above P
    assert (masks[2][:, 0] == np.uint64(2 ** 64 - 1)).all()  # slack 2: everything has landed by round 3


def test_gather_and_kmeans_inputs():
    counts = inputs.gather_counts(1004, 256)
    assert counts.min() >= 1024 and counts.max() <= 65536 and counts.dtype == np.int64
    bufs = inputs.gather_buffers(1004, counts[:4])
    assert [len(b) for b in bufs] == counts[:4].tolist()
    pts, comp, centres = inputs.kmeans_mixture(1005, 5000, 32, 64)
    assert pts.shape == (5000, 32) and pts.dtype == np.float32 and np.abs(centres).max() <= 10
    assert abs((pts - centres[comp]).std() - 1) < 0.02
    init = inputs.kmeans_first_of_component(pts, comp, 64)
    assert init.shape == (64, 32)
    for k in (0, 17, 63):
        assert np.array_equal(init[k], pts[np.nonzero(comp == k)[0][0]])
    masks = inputs.kmeans_masks(2005, 3, 64, 64, 0.75)
    assert len(masks) == 3 and masks[0].shape == (64, 1)
