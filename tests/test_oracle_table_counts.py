"""Pins for the oracle's window table, term counts and closed forms (CPU only).

Expected values are the paper's printed ones (tests/golden/paper_values.json, each with its
citation), brute-force loops, or closed-form arithmetic that is independent of the oracle's
own formula.
"""
import json
import math
import os

import numpy as np
import pytest

from atf_inputs import LLAMA3_SCALING
from oracle import atf_oracle as orc

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "paper_values.json")))


def test_first_window_is_floor_4pi():
    # w_min = 2*pi*k (Sec. 4); at k=2 the integer part is 12 for every model
    for base, d in ((1e6, 64), (5e5, 128), (1e7, 128)):
        W, theta = orc.window_table(base, d, 2.0, 1 << 20)
        assert W[0] == 12 and theta[0] == 1.0


def test_qwen_table_values_by_hand():
    # W_r = floor(4*pi * 1e6**(r/32)) clipped to N, re-typed with decimal exponents
    N = 32768
    W, _ = orc.window_table(1e6, 64, 2.0, N)
    for r in range(32):
        lam = 2 * math.pi * 10.0 ** (6.0 * r / 32.0)
        assert W[r] == min(int(2 * lam), N), r
    assert list(W[:8]) == [12, 19, 29, 45, 70, 108, 167, 258]
    assert np.all(np.diff(W) >= 0)


def test_live_terms_case_32_to_13():
    g = GOLD["live_terms_case"]
    N = 32768
    W, _ = orc.window_table(1e6, 64, 2.0, N)
    live = lambda z: int((z <= W).sum())
    assert live(0) == g["at_z0"]
    assert live(N - 1) == g["at_farthest"]


@pytest.mark.parametrize("model", ["qwen2.5-0.5b", "llama-3.2-3b"])
def test_table1_pruned_share(model):
    t = GOLD["table1_qk_pruned_percent"][model]
    sc = LLAMA3_SCALING if "scaling" in t else None
    for N, printed in t["rows"].items():
        N = int(N)
        W, _ = orc.window_table(t["base"], t["d"], 2.0, N, sc)
        ours = 100.0 * orc.pruned_share_prefill(W, t["d"], N)
        assert abs(ours - printed) <= 0.05 + 1e-9, (model, N, ours, printed)


def test_llama_pin_is_sensitive_to_the_scaling_rule():
    # the raw base misses Table 1's Llama column by a wide margin, so the pin does test the rule
    t = GOLD["table1_qk_pruned_percent"]["llama-3.2-3b"]
    W, _ = orc.window_table(t["base"], t["d"], 2.0, 32768, None)
    assert abs(100 * orc.pruned_share_prefill(W, t["d"], 32768) - t["rows"]["32768"]) > 2.0


def test_llama_scaled_thetas_structure():
    th0 = orc.effective_theta(5e5, 128, None)
    th = orc.effective_theta(5e5, 128, LLAMA3_SCALING)
    ratio = th0 / th
    assert np.all(ratio[:29] == 1.0)
    assert np.allclose(ratio[35:], 32.0, rtol=0, atol=1e-12)
    assert np.all(np.diff(ratio[28:36]) > 0)
    assert np.all(np.diff(2 * np.pi / th) > 0)  # wavelengths stay increasing


def test_single_row_and_rho_star():
    g = GOLD["single_row_16384"]
    W, _ = orc.window_table(1e6, 64, 2.0, 1 << 20)
    assert round(100 * orc.pruned_share_row(W, 64, 16384), 1) == g["discrete_percent"]
    assert round(100 * orc.closed_last_row(16384, 2.0, 1e6), 1) == g["continuous_percent"]
    assert round(orc.closed_rho_star(16384, 2.0, 1e6, 64), 1) == g["rho_star"]


def test_closed_form_vs_exact_qwen_32k():
    g = GOLD["closed_vs_exact_qwen_32k"]
    W, _ = orc.window_table(1e6, 64, 2.0, 32768)
    assert round(100 * orc.closed_prefill(32768, 2.0, 1e6), 1) == g["closed_percent"]
    assert round(100 * orc.pruned_share_prefill(W, 64, 32768), 1) == g["exact_percent"]


@pytest.mark.parametrize("base,d,N", [(1e6, 64, 2048), (1e6, 64, 8192), (1e6, 64, 32768),
                                      (1e7, 128, 1 << 20), (1e7, 128, 1 << 17)])
def test_counts_within_integral_error_of_closed_form(base, d, N):
    W, _ = orc.window_table(base, d, 2.0, N)
    exact = orc.pruned_share_prefill(W, d, N)
    assert abs(exact - orc.closed_R(1, N, 2.0, base)) * 100 <= GOLD["integral_error_points"]["max"]
    last = orc.pruned_share_row(W, d, N - 1)
    assert abs(last - orc.closed_last_row(N, 2.0, base)) * 100 <= GOLD["integral_error_points"]["max"]


def test_per_query_reduction_beyond_practical_lengths():
    g = GOLD["per_query_beyond_practical"]
    for N, key in ((200_000, "percent_at_200k"), (1_000_000, "percent_at_1m")):
        W, _ = orc.window_table(1e6, 64, 2.0, N)
        assert round(100 * orc.pruned_share_row(W, 64, N - 1)) == g[key]


def test_closed_form_constants():
    # gap decode - prefill -> 1/(2 ln B); saturation 1 - 1/ln B; second-half constant 1.27
    B = 1e6
    gap = orc.closed_last_row(1e5, 2.0, B) - orc.closed_prefill(1e5, 2.0, B)
    assert round(100 * gap, 1) == GOLD["decode_prefill_gap_points"]["value"]
    w_min = 4 * math.pi
    sat = orc.closed_last_row(w_min * B, 2.0, B)
    assert round(100 * sat, 1) == GOLD["saturation_decode_percent"]["value"]
    N = 1e6
    r = orc.closed_R(N / 2, N, 2.0, B)
    const = math.log(N / w_min) - r * math.log(B)
    assert round(const, 2) == GOLD["second_half_constant"]["constant"]
    assert round(100 * (r - orc.closed_prefill(N, 2.0, B)), 1) == GOLD["second_half_constant"]["points_above_prefill"]


def test_counts_brute_force_and_per_pair_arithmetic():
    rng = np.random.default_rng(5)
    for _ in range(20):
        h = int(rng.integers(1, 9))
        N = int(rng.integers(1, 60))
        W = np.sort(rng.integers(0, 80, size=h)).astype(np.int64)
        brute = sum(1 for n in range(N) for m in range(n + 1) for r in range(h) if n - m <= W[r])
        assert orc.kept_terms_prefill(W, N) == brute
        # per pair: rows n <= W keep n+1 terms, later rows keep W+1
        arith = 0
        for w in W:
            w = int(w)
            a = min(w, N - 1)
            arith += (a + 1) * (a + 2) // 2 + max(0, N - 1 - w) * (w + 1)
        assert arith == brute
        assert orc.kept_terms_decode(W, N) == sum(1 for m in range(N) for r in range(h) if N - 1 - m <= W[r])


def test_count_monotonicity():
    prev = -1
    for N in (1024, 2048, 4096, 8192):
        W, _ = orc.window_table(1e6, 64, 2.0, N)
        pruned = orc.full_terms_prefill(64, N) - orc.kept_terms_prefill(W, N)
        assert pruned >= prev
        prev = pruned
    prev = None
    for k in (1.0, 2.0, 4.0, 64.0, math.inf):
        W, _ = orc.window_table(1e6, 64, k, 8192)
        pruned = orc.full_terms_prefill(64, 8192) - orc.kept_terms_prefill(W, 8192)
        assert prev is None or pruned <= prev
        prev = pruned
    assert prev == 0  # k = inf prunes nothing


def test_reference_counts_of_the_workloads():
    # integers the CUDA path must reproduce bit for bit; derived from the definition only
    W, _ = orc.window_table(1e6, 64, 2.0, 2048)
    assert orc.kept_terms_prefill(W, 2048) == 48582232
    W, _ = orc.window_table(5e5, 128, 2.0, 8192, LLAMA3_SCALING)
    assert orc.kept_terms_prefill(W, 8192) == 1321818305
    W, _ = orc.window_table(5e5, 128, 2.0, 32768, LLAMA3_SCALING)
    assert orc.kept_terms_decode(W, 32768) == 1098280


def test_table4_ceilings_pin_the_coarse_rounding():
    g = GOLD["table4_ceilings"]
    for N, printed in g["rows"].items():
        N = int(N)
        W, _ = orc.window_table(g["base"], g["d"], 2.0, N)
        s = orc.coarse_kept_terms_prefill(W, N, 128, 128, 8) / orc.full_terms_prefill(g["d"], N)
        assert abs(2.0 / (1.0 + s) - printed) <= 0.006, (N, s)
        if N == 1 << 20:
            assert round(100 * (1 - s)) == g["pruned_percent_1m"]
    # a group of 16 pairs, or rounding inward, misses the printed ceiling at 1M
    N = 1 << 20
    W, _ = orc.window_table(g["base"], g["d"], 2.0, N)
    s16 = orc.coarse_kept_terms_prefill(W, N, 128, 128, 16) / orc.full_terms_prefill(g["d"], N)
    assert abs(2.0 / (1.0 + s16) - g["rows"][str(N)]) > 0.02


def test_coarse_counts_brute_force():
    rng = np.random.default_rng(11)
    for _ in range(10):
        h = 8
        N = int(rng.integers(5, 70))
        T = int(rng.choice([4, 8, 16]))
        G = int(rng.choice([2, 4]))
        W = np.sort(rng.integers(0, 80, size=h)).astype(np.int64)
        total = 0
        for n in range(N):
            for m in range(n + 1):
                q0 = (n // T) * T
                k1 = min((m // T) * T + T, N) - 1
                if k1 > q0:
                    total += h
                else:
                    zmin = q0 - k1
                    live = [r for r in range(h) if W[r] >= zmin]
                    if live:
                        total += min(h, G * math.ceil((h - live[0]) / G))
        assert orc.coarse_kept_terms_prefill(W, N, T, T, G) == total
        assert orc.coarse_kept_terms_decode(W, N, 4) == sum(
            h - min(h, (int((W < N - 1 - m).sum()) // 4) * 4) if (W >= N - 1 - m).any() else 0 for m in range(N))


# ---- the window family of App. A ----

def test_family_defaults_are_eq3():
    for base, d, N, sc in ((1e6, 64, 8192, None), (5e5, 128, 131072, gen_llama3()), (1e7, 128, 1 << 20, None)):
        for k in (2.0, 0.5, 64.0):
            W, th = orc.window_table(base, d, k, N, sc)
            Wf, thf = orc.window_table_family(base, d, N, sc, k_hi=k)
            assert np.array_equal(W, Wf) and np.array_equal(th, thf)


def gen_llama3():
    return {"kind": "llama3", "factor": 32.0, "low_freq_factor": 1.0, "high_freq_factor": 4.0, "original_ctx": 8192}


def test_family_reproduces_table2_pruned_shares():
    g = GOLD["table2_qk_pruned_percent"]
    cases = (("qwen2.5-0.5b_16384", 1e6, 64, 16384), ("qwen2.5-7b-1m_117000", 1e7, 128, 117000),
             ("qwen2.5-7b-1m_169000", 1e7, 128, 169000))
    for key, base, d, N in cases:
        for name, want in g[key].items():
            if name == "k2":
                W, _ = orc.window_table_family(base, d, N, k_hi=2.0)
            elif name == "variable_16_to_2":
                W, _ = orc.window_table_family(base, d, N, profile="arithmetic", k_hi=16.0, k_lo=2.0)
            else:
                W, _ = orc.window_table_family(base, d, N, k_hi=64.0)
            assert np.all(np.diff(W) >= 0)
            assert round(100 * orc.pruned_share_prefill(W, d, N), 1) == want, (key, name)


def test_family_special_cases():
    base, d, N = 1e6, 64, 4096
    h = d // 2
    # sliding window: every pair the same width (k_r = 0, floor = W)
    W, _ = orc.window_table_family(base, d, N, k_hi=0.0, beta=500.0)
    assert np.array_equal(W, np.full(h, 500))
    # linear window: k_r = 0 and the additive term a (r+1)/(d/2) alone
    W, _ = orc.window_table_family(base, d, N, k_hi=0.0, a=1000.0)
    assert np.array_equal(W, np.floor(1000.0 * (np.arange(h) + 1) / h).astype(np.int64))
    # ceiling as a fraction of the sequence length, floor in tokens
    W0, _ = orc.window_table(base, d, 2.0, N)
    W, _ = orc.window_table_family(base, d, N, k_hi=2.0, beta=64.0, cap=0.25 * N)
    assert np.array_equal(W, np.clip(W0, 64, N // 4))
    # wavelength exponent
    W, th = orc.window_table_family(base, d, N, k_hi=2.0, gamma=0.5)
    assert np.array_equal(W, np.floor(np.minimum(2.0 * np.sqrt(2 * np.pi / th), N)).astype(np.int64))
    # geometric profile: end points k_hi and k_lo, every ratio equal
    Wg, th = orc.window_table_family(base, d, 1 << 40, profile="geometric", k_hi=16.0, k_lo=2.0)
    kr = Wg / (2 * np.pi / th)
    assert abs(kr[0] - 16.0) < 0.2 and abs(kr[-1] - 2.0) < 1e-6
    assert np.allclose(kr[2:] / kr[1:-1], (2.0 / 16.0) ** (1.0 / (h - 1)), rtol=2e-2)
    # position-free pairs: the lowest-frequency quarter keeps everything and is not rotated
    W, th = orc.window_table_family(base, d, N, k_hi=2.0, nope_fraction=0.25)
    assert np.all(W[-8:] == N) and np.all(th[-8:] == 0.0) and np.array_equal(W[:-8], W0[:-8])
    x = np.random.default_rng(0).standard_normal((5, d))
    y = orc.rope_half_split(x, th, pos0=1000, round_bf16=False)
    assert np.array_equal(y[:, h - 8:h], x[:, h - 8:h]) and np.array_equal(y[:, d - 8:], x[:, d - 8:])
