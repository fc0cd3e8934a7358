"""CPU pins for the oracle's top-K selection, compaction and retention schedules
(Section 3.1 "Token Selection", Section 3.2, appendix "Reduction Schedule Configurations")."""
import itertools
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "step_schedules.txt")


def test_topk_brute_force_on_tiny_inputs():
    r = np.random.default_rng(0)
    for n in range(1, 7):
        s = r.uniform(size=n)
        for k in range(n + 1):
            kept = oracle.topk_select(s, k)
            best = max(itertools.combinations(range(n), k), key=lambda c: sum(s[list(c)]))
            assert list(kept) == sorted(best)


def test_topk_properties():
    r = np.random.default_rng(1)
    s = r.uniform(size=500).astype(np.float32)
    for k in (0, 1, 125, 499, 500):
        kept = oracle.topk_select(s, k)
        assert kept.dtype == np.int32 and len(kept) == k
        assert np.all(np.diff(kept) > 0)                       # temporal order, no repeats
        dropped = np.setdiff1d(np.arange(500), kept)
        if k and len(dropped):
            assert s[kept].min() >= s[dropped].max()
        assert set(kept) == set(np.argsort(-s, kind="stable")[:k])
    assert list(oracle.topk_select(s, 500)) == list(range(500))  # 100% budget is the identity


def test_topk_ties_prefer_earlier_tokens():
    s = np.array([0.5, 1.0, 0.5, 0.5, 1.0, 0.5])
    assert list(oracle.topk_select(s, 3)) == [0, 1, 4]
    assert list(oracle.topk_select(s, 4)) == [0, 1, 2, 4]
    assert list(oracle.topk_select(np.zeros(5), 2)) == [0, 1]


def test_compact_gathers_rows_and_composes_index_map():
    r = np.random.default_rng(2)
    T, M, D = 20, 3, 4
    h = r.normal(size=(T, D)).astype(np.float32)
    pos = np.arange(T, dtype=np.int32)
    idx = np.arange(T, dtype=np.int32)
    kept1 = np.array([0, 2, 3, 7, 8, 11, 15, 16], dtype=np.int32)
    h1, p1, i1 = oracle.compact(h, pos, idx, kept1, M)
    assert h1.shape == (8 + M, D) and h1.dtype == h.dtype
    assert np.array_equal(h1[:8], h[kept1]) and np.array_equal(h1[8:], h[T - M:])
    assert list(p1) == list(kept1) + [17, 18, 19] and np.array_equal(p1, i1)
    kept2 = np.array([1, 4, 6], dtype=np.int32)
    h2, p2, i2 = oracle.compact(h1, p1, i1, kept2, M)
    assert list(i2) == [2, 8, 15, 17, 18, 19]                  # original token ids
    assert np.array_equal(h2, h[i2]) and np.all(np.diff(p2) > 0)
    h3, p3, i3 = oracle.compact(h, pos, idx, np.arange(T - M, dtype=np.int32), M)
    assert np.array_equal(h3, h) and np.array_equal(i3, idx)   # 100% budget is the identity


def _golden():
    rows = []
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        name, comp, segs = [f.strip() for f in line.split("|")]
        parsed = []
        for seg in segs.split():
            rng_, a = seg.split("=")
            lo, hi = rng_.split(":")
            parsed.append((int(lo), int(hi), round(float(a) * 10000)))
        rows.append((name, float(comp), parsed))
    return rows


@pytest.mark.parametrize("name,comp,segments", _golden())
def test_step_schedule_reproduces_printed_compression(name, comp, segments):
    alpha = oracle.step_schedule(62, segments)
    assert abs(oracle.mean_retention(alpha) - comp) < 0.05 + 1e-9     # printed to one decimal
    # the same mean comes out of the keep counts, so alpha is a fraction of the ORIGINAL count
    n0 = 36864                                                        # 256 frames x 144 tokens
    K = oracle.schedule_keep_counts(alpha, n0, 144)
    assert abs(100.0 * sum(K) / (62 * n0) - comp) < 0.06


def test_keep_counts_follow_the_progressive_schedule():
    alpha = [10000] * 4 + [5000] * 4 + [2500] * 4
    assert oracle.schedule_keep_counts(alpha, 32768, 256) == [32768] * 4 + [16384] * 4 + [8192] * 4
    assert oracle.schedule_keep_counts([10000, 1000, 1000], 16384, 256) == [16384, 1638, 1638]
    assert oracle.schedule_keep_counts([5000, 100, 9000], 1000, 144) == [500, 144, 144]   # floor, never grows
    assert oracle.schedule_keep_counts([10000, 2500], 100, 144) == [100, 100]            # single image kept whole
    assert oracle.schedule_keep_counts([10000] * 3, 777, 0) == [777] * 3                 # 100% keeps everything


def test_sigmoid_schedule_shape():
    a = oracle.sigmoid_schedule(62, 20.0, 0.24, 1.0, 0.125)
    assert np.all(np.diff(a) < 0) and a[0] > 0.99 and abs(a[-1] - 0.125) < 1e-4
    mid = oracle.sigmoid_schedule(100, 20.0, 0.5, 1.0, 0.125)[50]
    np.testing.assert_allclose(mid, 0.125 + 0.875 * 0.5, rtol=1e-12)


def test_score_density_closed_forms_and_brute_force():
    """The sparsity statistic (Section 2: tokens needed for a given share of the importance mass)."""
    # uniform vector: ceil(frac n) tokens (values a power of two so that every partial sum is exact)
    for n, frac, want in ((10, 0.8, 8), (10, 0.5, 5), (1000, 0.801, 801), (7, 1.0, 7)):
        assert oracle.score_density(np.full(n, 0.25), frac) == want
    # all mass on one token; nothing at all
    onehot = np.zeros(50); onehot[17] = 3.0
    assert oracle.score_density(onehot, 0.8) == 1 and oracle.score_density(onehot, 1.0) == 1
    assert oracle.score_density(np.zeros(9), 0.8) == 0
    # two levels: h heavy tokens of weight 8 and l light tokens of weight 1 -> mass 8h + l
    h, l = 4, 32                                           # total 64; 80% = 51.2 -> 4 heavy (32) + 20 light
    v = np.concatenate([np.ones(l), np.full(h, 8.0)])
    assert oracle.score_density(v, 0.8) == 24 and oracle.score_density(v, 0.5) == 4 and oracle.score_density(v, 0.51) == 5
    # order of the input does not matter; brute force over prefixes of the sorted vector
    r = np.random.default_rng(12)
    for _ in range(20):
        s = r.exponential(size=r.integers(1, 40))
        frac = r.uniform(0.05, 1.0)
        srt = sorted(s, reverse=True)
        want = next(k for k in range(1, len(s) + 1) if sum(srt[:k]) >= frac * sum(srt) - 1e-15)
        assert oracle.score_density(r.permutation(s), frac) == want
    # a heavy-tailed vector is denser than a flat one (the paper's 10.9% against 30.6% contrast, in kind)
    flat = r.uniform(0.5, 1.0, size=4096)
    peaky = flat * 1e-2
    peaky[r.choice(4096, size=400, replace=False)] += r.exponential(1.0, size=400)
    assert oracle.score_density(peaky, 0.8) < 0.2 * 4096 < oracle.score_density(flat, 0.8)


def test_ffn_layers_never_reduce_in_the_schedule():
    """With layer kinds given, a cut that the schedule places on an FFN layer moves to the next Mamba / attention layer."""
    alpha = [10000, 5000, 5000, 2500, 2500, 1000]
    plain = oracle.schedule_keep_counts(alpha, 1000, 0)
    assert plain == [1000, 500, 500, 250, 250, 100]
    assert oracle.schedule_keep_counts(alpha, 1000, 0, "MAMAMA") == plain              # no FFN layer: unchanged
    got = oracle.schedule_keep_counts(alpha, 1000, 0, "MFAFMF")
    assert got == [1000, 1000, 500, 500, 250, 250]
    # an FFN layer's count equals its incoming count; every other layer takes the schedule's own value
    n_cur = 1000
    for kind, k, p in zip("MFAFMF", got, plain):
        assert k == (n_cur if kind == "F" else min(n_cur, p))
        n_cur = k
    # the library's helper is the same rule
    from paper_2603_00198_b200 import binding
    for pattern in ("MFAFMF", "FFMAMA", "MAMAMA", "AFAFAF"):
        assert binding.str_schedule_keep_counts_layers(alpha, pattern, 1000, 16) == oracle.schedule_keep_counts(alpha, 1000, 16, pattern)
