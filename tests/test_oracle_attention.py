"""Pins for the oracle's RoPE and attention functions (CPU only): identities the paper
states (Eq. 1), reductions to textbook routines, special cases, and brute force."""
import math

import numpy as np
import torch

from oracle import atf_oracle as orc


def _rand(shape, seed):
    rng = np.random.default_rng(seed)
    return orc.round_to_bf16(rng.standard_normal(shape))


def test_round_to_bf16_matches_torch():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.standard_normal(20000) * 10.0 ** rng.integers(-6, 6, 20000),
                        np.array([0.0, 1.0, -1.0, 1.00390625, 1.01171875, 3.0e38])])
    ours = orc.round_to_bf16(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(ours, ref)
    # ties go to even: 1 + 2^-8 is halfway between 1 and 1 + 2^-7
    assert orc.round_to_bf16(np.array([1.0 + 2.0 ** -8]))[0] == 1.0
    assert orc.round_to_bf16(np.array([1.0 + 3 * 2.0 ** -8]))[0] == 1.0 + 2.0 ** -6


def test_pair_decomposition_from_unrotated_vectors():
    # Eq. 1: per-pair product of the rotated vectors = a_r cos(z th_r) + b_r sin(z th_r)
    d, h = 64, 32
    theta = orc.effective_theta(1e6, d)
    rng = np.random.default_rng(1)
    q, k = rng.standard_normal(d), rng.standard_normal(d)
    for n, m in ((5, 5), (100, 3), (100000, 99000), (7, 0)):
        qr = orc.rope_half_split(q[None, :], theta, pos0=n, round_bf16=False)[0]
        kr = orc.rope_half_split(k[None, :], theta, pos0=m, round_bf16=False)[0]
        z = n - m
        a = q[:h] * k[:h] + q[h:] * k[h:]
        b = q[:h] * k[h:] - q[h:] * k[:h]
        dx = a * np.cos(z * theta) + b * np.sin(z * theta)
        per_pair = qr[:h] * kr[:h] + qr[h:] * kr[h:]
        assert np.allclose(per_pair, dx, rtol=0, atol=1e-9)
        assert abs(per_pair.sum() - qr @ kr) < 1e-12


def test_rope_preserves_pair_norms_and_identity_at_zero():
    d, h = 128, 64
    theta = orc.effective_theta(5e5, d)
    x = _rand((3, 50, d), 2)
    y = orc.rope_half_split(x, theta, pos0=1000, round_bf16=False)
    assert np.allclose(x[..., :h] ** 2 + x[..., h:] ** 2, y[..., :h] ** 2 + y[..., h:] ** 2, atol=1e-12)
    y0 = orc.rope_half_split(x[:, :1], theta, pos0=0)
    assert np.array_equal(y0, x[:, :1])


def _textbook_causal(Q, K, V, window=None):
    N, d = Q.shape
    S = (Q @ K.T) / math.sqrt(d)
    n, m = np.arange(N)[:, None], np.arange(N)[None, :]
    mask = m <= n
    if window is not None:
        mask &= (n - m) <= window
    S = np.where(mask, S, -np.inf)
    mu = S.max(axis=1, keepdims=True)
    P = np.exp(S - mu)
    ell = P.sum(axis=1, keepdims=True)
    return (P @ V) / ell, (mu + np.log(ell))[:, 0]


def test_full_attention_when_every_window_covers_the_sequence():
    N, d = 96, 64
    Q, K, V = _rand((N, d), 3), _rand((N, d), 4), _rand((N, d), 5)
    # k = inf, and the smallest finite k with k*lambda_min >= N
    for k in (math.inf, N / (2 * math.pi) + 1e-9):
        W, _ = orc.window_table(1e6, d, k, N)
        assert np.all(W >= N - 1)
        O, LSE = orc.attention_rows(Q, K, V, W, range(N))
        Or, Lr = _textbook_causal(Q, K, V)
        assert np.allclose(O, Or, atol=1e-12) and np.allclose(LSE, Lr, atol=1e-12)
    # the library routine
    tq, tk, tv = (torch.from_numpy(a)[None, None] for a in (Q, K, V))
    Ot = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)[0, 0].numpy()
    assert np.allclose(O, Ot, atol=1e-10)


def test_uniform_table_is_the_sliding_window():
    N, d = 80, 32
    Q, K, V = _rand((N, d), 6), _rand((N, d), 7), _rand((N, d), 8)
    for w in (0, 1, 7, 33):
        W = np.full(d // 2, w, dtype=np.int64)
        O, LSE = orc.attention_rows(Q, K, V, W, range(N))
        Or, Lr = _textbook_causal(Q, K, V, window=w)
        assert np.allclose(O, Or, atol=1e-12) and np.allclose(LSE, Lr, atol=1e-12)


def test_brute_force_on_tiny_inputs():
    d, h = 16, 8
    for seed, N, W in ((9, 40, [0, 1, 2, 3, 5, 8, 13, 21]),      # keys beyond 21 are dropped
                       (10, 33, [3, 3, 3, 40, 40, 40, 40, 40]),   # clipped entries
                       (11, 25, [2, 30, 4, 30, 1, 0, 30, 7])):    # non-monotone is fine for the definition
        Q, K, V = _rand((N, d), seed), _rand((N, d), seed + 100), _rand((N, d), seed + 200)
        W = np.array(W, dtype=np.int64)
        O, LSE = orc.attention_rows(Q, K, V, W, range(N))
        Ob, Lb = orc.brute_force_attention(Q, K, V, W)
        assert np.allclose(O, Ob, atol=1e-12) and np.allclose(LSE, Lb, atol=1e-12)


def test_single_term_swap_changes_the_answer():
    # a dropped term must show: the window boundary is inclusive (z <= W_r keeps the term)
    d, h = 8, 4
    N = 6
    Q, K, V = _rand((N, d), 20), _rand((N, d), 21), _rand((N, d), 22)
    W = np.array([2, 5, 5, 5], dtype=np.int64)
    s = orc.windowed_scores_row(Q[5], K, W, 5)
    m = 3  # z = 2 == W_0: pair 0 still counted
    full = (Q[5] @ K[m]) / math.sqrt(d)
    assert abs(s[m] - full) < 1e-14
    m = 2  # z = 3 > W_0: pair 0 gone
    wo = (Q[5] @ K[m] - Q[5, 0] * K[m, 0] - Q[5, h] * K[m, h]) / math.sqrt(d)
    assert abs(s[m] - wo) < 1e-14


def test_gqa_decode_and_convexity():
    B, Hq, Hkv, L, d = 2, 6, 2, 70, 32
    q = _rand((B, Hq, d), 30)
    Kc, Vc = _rand((B, Hkv, L, d), 31), _rand((B, Hkv, L, d), 32)
    W, _ = orc.window_table(1e4, d, 2.0, L)
    O, LSE = orc.decode(q, Kc, Vc, W)
    # decode = last row of prefill with that query in place
    for b in range(B):
        for hq in range(Hq):
            Qfull = np.zeros((L, d)); Qfull[L - 1] = q[b, hq]
            O1, L1 = orc.attention_rows(Qfull, Kc[b, hq // 3], Vc[b, hq // 3], W, [L - 1])
            assert np.allclose(O[b, hq], O1[0], atol=1e-13) and abs(LSE[b, hq] - L1[0]) < 1e-13
            assert np.all(O[b, hq] <= Vc[b, hq // 3].max(axis=0) + 1e-12)
            assert np.all(O[b, hq] >= Vc[b, hq // 3].min(axis=0) - 1e-12)
    # heads of one group with the same query give the same row
    q2 = q.copy(); q2[:, 1] = q2[:, 0]
    O2, _ = orc.decode(q2, Kc, Vc, W)
    assert np.array_equal(O2[:, 0], O2[:, 1])
    # attention_gqa maps heads the same way
    Q4 = _rand((B, Hq, 20, d), 33)
    Og, Lg = orc.attention_gqa(Q4, Kc[:, :, :20], Vc[:, :, :20], W, rows=[19])
    Od, Ld = orc.decode(Q4[:, :, 19], Kc[:, :, :20], Vc[:, :, :20], W)
    assert np.allclose(Og[:, :, 0], Od) and np.allclose(Lg[:, :, 0], Ld)


def _coarse_brute(Q, K, V, W, T, G):
    N, d = Q.shape
    h = d // 2
    O = np.zeros((N, d)); LSE = np.zeros(N)
    for n in range(N):
        sc = []
        for m in range(n + 1):
            q0 = (n // T) * T
            k1 = min((m // T) * T + T, N) - 1
            if k1 > q0:
                r0 = 0
            else:
                live = [r for r in range(h) if W[r] >= q0 - k1]
                r0 = h if not live else h - min(h, G * math.ceil((h - live[0]) / G))
            if r0 >= h:
                sc.append(-math.inf)
            else:
                sc.append(sum(Q[n, r] * K[m, r] + Q[n, r + h] * K[m, r + h] for r in range(r0, h)) / math.sqrt(d))
        sc = np.array(sc); mu = sc.max(); p = np.exp(sc - mu)
        O[n] = (p[:, None] * V[: n + 1]).sum(0) / p.sum(); LSE[n] = mu + math.log(p.sum())
    return O, LSE


def test_coarse_mode_definition_and_special_cases():
    d, h, N, T, G = 16, 8, 50, 8, 2
    Q, K, V = _rand((N, d), 40), _rand((N, d), 41), _rand((N, d), 42)
    W = np.array([1, 3, 6, 10, 15, 22, 30, 50], dtype=np.int64)
    O, LSE = orc.coarse_attention_rows(Q, K, V, W, range(N), T, T, G)
    Ob, Lb = _coarse_brute(Q, K, V, W, T, G)
    assert np.allclose(O, Ob, atol=1e-12) and np.allclose(LSE, Lb, atol=1e-12)
    # every window covering the sequence: coarse = exact = full
    Wf = np.full(h, N, dtype=np.int64)
    Oc, Lc = orc.coarse_attention_rows(Q, K, V, Wf, range(N), T, T, G)
    Oe, Le = orc.attention_rows(Q, K, V, Wf, range(N))
    assert np.allclose(Oc, Oe, atol=1e-13) and np.allclose(Lc, Le, atol=1e-13)
    # coarse never keeps fewer terms than exact
    assert orc.coarse_kept_terms_prefill(W, N, T, T, G) >= orc.kept_terms_prefill(W, N)


def test_coarse_decode_definition():
    B, Hq, Hkv, L, d = 1, 2, 1, 90, 32
    h = d // 2
    q = _rand((B, Hq, d), 50)
    Kc, Vc = _rand((B, Hkv, L, d), 51), _rand((B, Hkv, L, d), 52)
    W = np.sort(np.random.default_rng(53).integers(0, 120, h)).astype(np.int64)
    W[-1] = 200
    O, LSE = orc.coarse_decode(q, Kc, Vc, W, 8)
    for hq in range(Hq):
        sc = []
        for m in range(L):
            z = L - 1 - m
            live = [r for r in range(h) if z <= W[r]]
            r0 = (live[0] // 8) * 8
            sc.append(sum(q[0, hq, r] * Kc[0, 0, m, r] + q[0, hq, r + h] * Kc[0, 0, m, r + h]
                          for r in range(r0, h)) / math.sqrt(d))
        sc = np.array(sc); mu = sc.max(); p = np.exp(sc - mu)
        assert np.allclose(O[0, hq], (p[:, None] * Vc[0, 0]).sum(0) / p.sum(), atol=1e-12)
        assert abs(LSE[0, hq] - (mu + math.log(p.sum()))) < 1e-12
    # thresholds on chunk boundaries: coarse decode = exact decode
    W8 = np.repeat(np.array([5, 40], dtype=np.int64), 8)
    W8[8:] = 200
    Oc, Lc = orc.coarse_decode(q, Kc, Vc, W8, 8)
    Oe, Le = orc.decode(q, Kc, Vc, W8)
    assert np.allclose(Oc, Oe, atol=1e-13) and np.allclose(Lc, Le, atol=1e-13)
