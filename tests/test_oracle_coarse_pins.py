"""Pins that tie the coarse-mode attention functions of the oracle (the ones the GPU coarse outputs
are compared with) to things fixed outside them (CPU only).

coarse_kept_terms_prefill is pinned by Table 4's printed ceilings (test_oracle_table_counts.py).  It is
a separate implementation from coarse_first_pair, which coarse_attention_rows uses, so here
  - the per-tile pair set of coarse_first_pair, summed over every (query tile, key tile) of the three
    Table 4 prompts, must give exactly that pinned count (and a rounding to the nearest group, or a
    max-distance rule, must not);
  - with one-token tiles the tile rule is the per-cell rule, so the coarse function must equal the
    exact per-term definition on a raised table: rounding outward to whole groups of G pairs is the
    same as giving every pair of a group the widest window of the group.  Inward rounding would
    correspond to the narrowest window instead, and the test tells the two apart;
  - the same for coarse_decode, whose groups are counted from pair 0 upward.
"""
import json
import math
import os

import numpy as np

from oracle import atf_oracle as orc

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "paper_values.json")))


def _rand(shape, seed):
    rng = np.random.default_rng(seed)
    return orc.round_to_bf16(rng.standard_normal(shape))


def _tile_sum(W, N, T, G, first_pair):
    """Terms kept when every off-diagonal (query tile, key tile) pair uses the pairs from first_pair(z_min)
    up and the diagonal tiles use every pair on their causal cells.  N must be a multiple of T."""
    h = len(W)
    nt = N // T
    total = nt * h * (T * (T + 1) // 2)
    for dt in range(1, nt):
        z_min = dt * T - (T - 1)  # first row of the query tile against the last key of the key tile
        total += (nt - dt) * T * T * (h - first_pair(z_min))
    return total


def test_per_tile_pair_set_sums_to_the_table4_pinned_count():
    g = GOLD["table4_ceilings"]
    h = g["d"] // 2
    for N in (int(n) for n in g["rows"]):
        W, _ = orc.window_table(g["base"], g["d"], 2.0, N)
        want = orc.coarse_kept_terms_prefill(W, N, 128, 128, 8)
        got = _tile_sum(W, N, 128, 8, lambda z: orc.coarse_first_pair(W, z, 8))
        assert got == want, N
        # the printed ceiling follows from this sum as well
        s = got / orc.full_terms_prefill(g["d"], N)
        assert abs(2.0 / (1.0 + s) - g["rows"][str(N)]) <= 0.006
        # other readings of the rule give other sums: nearest group instead of outward ...
        def nearest(z):
            r_any = int(np.searchsorted(W, z, side="left"))
            return min(h, h - 8 * int(math.floor((h - r_any) / 8 + 0.5)))
        assert _tile_sum(W, N, 128, 8, nearest) != want
        # ... and the tile's farthest cell instead of its nearest one
        assert _tile_sum(W, N, 128, 8, lambda z: orc.coarse_first_pair(W, z + 254, 8)) != want


def _raised_table(W, G, from_low_frequency_end=True):
    """Every pair gets the widest window of its group of G pairs (groups counted from the low-frequency end
    for prefill, from pair 0 for decode).  W is non-decreasing, so that is the group's highest pair."""
    h = len(W)
    up = np.empty_like(W)
    for r in range(h):
        top = h - 1 - ((h - 1 - r) // G) * G if from_low_frequency_end else min(h - 1, (r // G) * G + G - 1)
        up[r] = W[top]
    return up


def test_one_token_tiles_make_the_coarse_rule_the_exact_rule_on_a_raised_table():
    d, h, N = 32, 16, 90
    Q, K, V = _rand((N, d), 60), _rand((N, d), 61), _rand((N, d), 62)
    W = np.array([0, 1, 2, 4, 6, 9, 13, 18, 25, 33, 41, 50, 58, 66, 75, 200], dtype=np.int64)
    rows = range(N)
    # groups of one pair: nothing is rounded, the coarse function is the per-term definition
    Oc, Lc = orc.coarse_attention_rows(Q, K, V, W, rows, 1, 1, 1)
    Oe, Le = orc.attention_rows(Q, K, V, W, rows)
    assert np.allclose(Oc, Oe, atol=1e-12) and np.allclose(Lc, Le, atol=1e-12)
    for G in (2, 4, 8):
        Oc, Lc = orc.coarse_attention_rows(Q, K, V, W, rows, 1, 1, G)
        Wup = _raised_table(W, G)
        Oe, Le = orc.attention_rows(Q, K, V, Wup, rows)
        assert np.allclose(Oc, Oe, atol=1e-12) and np.allclose(Lc, Le, atol=1e-12), G
        # inward rounding would be the narrowest window of each group: a different result
        Wdown = np.array([W[(h - 1 - ((h - 1 - r) // G) * G) - (G - 1)] for r in range(h)], dtype=np.int64)
        Od, _ = orc.attention_rows(Q, K, V, Wdown, rows)
        assert not np.allclose(Oc, Od, atol=1e-6), G
    # a table that is constant on every group of 8 is its own raised table: coarse = exact
    W8 = np.repeat(np.array([7, 300], dtype=np.int64), 8)
    Oc, Lc = orc.coarse_attention_rows(Q, K, V, W8, rows, 1, 1, 8)
    Oe, Le = orc.attention_rows(Q, K, V, W8, rows)
    assert np.allclose(Oc, Oe, atol=1e-12) and np.allclose(Lc, Le, atol=1e-12)


def test_coarse_decode_is_exact_decode_on_a_raised_table():
    B, Hq, Hkv, L, d = 1, 4, 2, 120, 32
    h = d // 2
    q = _rand((B, Hq, d), 70)
    Kc, Vc = _rand((B, Hkv, L, d), 71), _rand((B, Hkv, L, d), 72)
    W = np.array([0, 2, 3, 5, 8, 12, 17, 23, 30, 38, 47, 57, 68, 80, 93, 500], dtype=np.int64)
    for G in (2, 4, 8):
        Oc, Lc = orc.coarse_decode(q, Kc, Vc, W, G)
        # rounding the first live pair DOWN to a multiple of G keeps the whole group of the first live pair
        Wup = _raised_table(W, G, from_low_frequency_end=False)
        Oe, Le = orc.decode(q, Kc, Vc, Wup)
        assert np.allclose(Oc, Oe, atol=1e-12) and np.allclose(Lc, Le, atol=1e-12), G
        assert orc.coarse_kept_terms_decode(W, L, G) == orc.kept_terms_decode(Wup, L)
        # rounding up instead would keep only whole groups that are live: the narrowest window of each group
        Wdown = np.array([W[(r // G) * G] for r in range(h)], dtype=np.int64)
        Od, _ = orc.decode(q, Kc, Vc, Wdown)
        assert not np.allclose(Oc, Od, atol=1e-6), G


def test_coarse_tile_rule_against_the_count_of_its_own_cells():
    # For tiles of T tokens, the terms coarse_attention_rows uses in a row are: every pair on the keys of the
    # tiles that touch the diagonal, and h - coarse_first_pair(z_min) pairs on each earlier tile.  Summed over
    # the rows this is the Table-4-pinned count function (small sizes, ragged N).
    rng = np.random.default_rng(80)
    for _ in range(8):
        h = 8
        N = int(rng.integers(9, 80))
        T = int(rng.choice([4, 8, 16]))
        G = int(rng.choice([2, 4, 8]))
        W = np.sort(rng.integers(0, 90, size=h)).astype(np.int64)
        total = 0
        for n in range(N):
            q0 = (n // T) * T
            for k0 in range(0, n + 1, T):
                k1 = min(k0 + T, N) - 1
                cells = min(k1, n) - k0 + 1
                total += cells * (h if k1 > q0 else h - orc.coarse_first_pair(W, q0 - k1, G))
        assert total == orc.coarse_kept_terms_prefill(W, N, T, T, G)
