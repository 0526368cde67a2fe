"""Pins for the oracle's appended-rows functions (CPU only): the row interval [n0, n1] of
App. C ("The interval itself"), whose endpoints are the whole prefill and the decode step, and
which is what a chunk of a chunked prefill computes (Sec. 7.3)."""
import json
import os

import numpy as np

from oracle import atf_oracle as orc

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "paper_values.json")))


def _rand(shape, seed):
    rng = np.random.default_rng(seed)
    return orc.round_to_bf16(rng.standard_normal(shape))


def test_interval_counts_endpoints_and_additivity():
    for base, d, N in ((1e6, 64, 8192), (5e5, 128, 4096), (1e7, 128, 50000)):
        W, _ = orc.window_table(base, d, 2.0, N)
        assert orc.kept_terms_interval(W, 0, N) == orc.kept_terms_prefill(W, N)
        assert orc.kept_terms_interval(W, N - 1, N) == orc.kept_terms_decode(W, N)
        cuts = [0, 1, 255, 256, 1000, N // 2, N - 1, N]
        assert sum(orc.kept_terms_interval(W, a, b) for a, b in zip(cuts, cuts[1:])) == orc.kept_terms_prefill(W, N)
        assert orc.kept_terms_interval(W, 77, 77) == 0


def test_interval_counts_brute_force():
    rng = np.random.default_rng(11)
    for _ in range(20):
        h = int(rng.integers(1, 9))
        N = int(rng.integers(2, 60))
        n0 = int(rng.integers(0, N))
        W = np.sort(rng.integers(0, 80, size=h)).astype(np.int64)
        brute = sum(1 for n in range(n0, N) for m in range(n + 1) for r in range(h) if n - m <= W[r])
        assert orc.kept_terms_interval(W, n0, N) == brute


def test_second_half_is_1p7_points_above_the_whole_prefill():
    # discrete counts, unscaled base 1e6 (the paper's B for this statement), k = 2
    want = GOLD["second_half_constant"]["points_above_prefill"]
    gap = GOLD["decode_prefill_gap_points"]["value"]
    for N in (8192, 32768):
        W, _ = orc.window_table(1e6, 64, 2.0, N)
        whole = orc.pruned_share_prefill(W, 64, N)
        half = orc.pruned_share_interval(W, 64, N // 2, N)
        last = orc.pruned_share_row(W, 64, N - 1)
        assert round(100 * (half - whole), 1) == want
        # "half of the 3.6-point gap to decode"
        assert abs(100 * (half - whole) - gap / 2) < 0.2
        assert whole < half < last


def test_appended_rows_equal_single_shot_rows_and_decode():
    N, d = 300, 16
    W = np.array([3, 9, 20, 41, 90, 150, 300, 300], dtype=np.int64)
    theta = orc.effective_theta(1e4, d)
    Q = orc.rope_half_split(_rand((N, d), 1), theta)
    K = orc.rope_half_split(_rand((N, d), 2), theta)
    V = _rand((N, d), 3)
    O_all, L_all = orc.attention_rows(Q, K, V, W, range(N))
    # one chunk from an arbitrary start
    for n0 in (0, 1, 127, 128, 200, 299):
        O, L = orc.attention_appended_rows(Q[n0:], K, V, W, n0)
        assert np.array_equal(O, O_all[n0:]) and np.array_equal(L, L_all[n0:])
    # a chunked prefill: every chunk sees only the keys that exist so far
    cuts = [0, 100, 228, 300]
    parts = [orc.attention_appended_rows(Q[a:b], K[:b], V[:b], W, a) for a, b in zip(cuts, cuts[1:])]
    assert np.array_equal(np.concatenate([p[0] for p in parts]), O_all)
    assert np.array_equal(np.concatenate([p[1] for p in parts]), L_all)
    # one appended row is the decode step (a separately written oracle function)
    o_dec = orc.decode(Q[None, None, N - 1], K[None, None], V[None, None], W)
    o_dec = o_dec[0] if isinstance(o_dec, tuple) else o_dec
    O1, _ = orc.attention_appended_rows(Q[N - 1:], K, V, W, N - 1)
    assert np.allclose(np.asarray(o_dec).reshape(-1), O1.reshape(-1), rtol=0, atol=1e-12)


def test_appended_rows_brute_force():
    N, d, n0 = 40, 8, 25
    W = np.array([2, 5, 11, 40], dtype=np.int64)
    Q, K, V = _rand((N, d), 4), _rand((N, d), 5), _rand((N, d), 6)
    O_bf, L_bf = orc.brute_force_attention(Q, K, V, W)
    O, L = orc.attention_appended_rows(Q[n0:], K, V, W, n0)
    assert np.allclose(O, O_bf[n0:], rtol=0, atol=1e-12)
    assert np.allclose(L, L_bf[n0:], rtol=0, atol=1e-12)
