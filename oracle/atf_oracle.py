"""Slow, plain fp64 CPU oracle for attention with per-RoPE-wavelength distance windows.

TEST INFRASTRUCTURE ONLY.  This module is the independent definition the CUDA library is
checked against.  Nothing on the product path may import it; it imports nothing from the
CUDA package and shares no code, table or constant with it.  Everything here is NumPy in
float64 (bf16 inputs are widened exactly), written as the definitions read, with no
blocking, fusion or reordering.

Pinned functions (pins live in tests/test_oracle_*.py, all CPU-only):
  effective_theta / window_table  - printed window widths and pruned shares (Table 1, Sec. 3.2)
  rope_half_split                 - Eq. 1 identity from unrotated vectors, norm preservation
  attention_rows / decode         - pair-sum identity (Eq. 1), textbook causal softmax at
                                    k = inf, sliding-window special case (Sec. 3.2),
                                    pure-Python brute force
  kept_terms_*                    - printed shares (Table 1, Fig. 7), closed forms (Eq. 5,
                                    App. C), brute force
  coarse_* (second named mode)    - the speed ceilings of Table 4 pin the rounding rule of the
                                    count; coarse_first_pair / coarse_attention_rows /
                                    coarse_decode are tied to that count and to the per-term
                                    definition on a raised table (tests/test_oracle_coarse_pins.py).
                                    What stays a reading: nearest versus farthest cell of a tile
                                    at Table 4's printed precision, and the tile size.
  split-precision scores          - no function of their own: the reference is attention_rows on fp32 values
                                    widened exactly; tests/test_oracle_split_precision.py derives the
                                    tolerance from it (hi + lo representation, dropped lo x lo terms)
  window_table_family             - Table 2's pruned shares (arithmetic and constant profiles);
                                    the geometric profile: PARITY UNPINNED (App. A names it and
                                    prints no value).
"""
from __future__ import annotations

import math

import numpy as np

# ----------------------------------------------------------------------------------------
# bf16 rounding (type conversion, round-to-nearest-even), done directly from float64 so no
# double rounding through float32 can occur.
# ----------------------------------------------------------------------------------------


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float64 values to the nearest bfloat16 (8 significant bits, ties to even).

    Returns float64 holding exactly representable bf16 values.  Normal range only (the
    workloads never produce bf16 subnormals other than exact zero).
    """
    x = np.asarray(x, dtype=np.float64)
    m, e = np.frexp(x)  # x = m * 2**e, 0.5 <= |m| < 1
    m = np.rint(m * 256.0) / 256.0  # 8 significant bits; np.rint rounds ties to even
    return np.ldexp(m, e)


# ----------------------------------------------------------------------------------------
# Window table (Sec. 3.1 theta_r, Eq. 2 wavelength, Eq. 3 window, Sec. 3.2 effective theta)
# ----------------------------------------------------------------------------------------


def effective_theta(base: float, d: int, scaling: dict | None = None) -> np.ndarray:
    """Angular velocity of each pair r in [0, d/2): theta_r = base**(-2r/d)  (Sec. 3.1).

    `scaling` = None, or {"kind": "llama3", "factor", "low_freq_factor", "high_freq_factor",
    "original_ctx"}.  The paper only names llama3-style scaling (Sec. 3.2); the rule taken
    here is the one whose pruned shares reproduce Table 1's Llama-3.2-3B column: a pair whose
    wavelength is shorter than original_ctx/high_freq_factor keeps theta, one longer than
    original_ctx/low_freq_factor gets theta/factor, and in between the two are blended
    linearly in t = (original_ctx/lambda - low_freq_factor)/(high_freq_factor - low_freq_factor).
    """
    h = d // 2
    theta = np.array([math.pow(base, -2.0 * r / d) for r in range(h)], dtype=np.float64)
    if scaling is None or scaling.get("kind", "none") == "none":
        return theta
    if scaling["kind"] != "llama3":
        raise ValueError("unknown scaling kind")
    f = float(scaling["factor"])
    lf = float(scaling["low_freq_factor"])
    hf = float(scaling["high_freq_factor"])
    c = float(scaling["original_ctx"])
    if not (f > 0.0 and 0.0 < lf < hf and c > 0.0 and math.isfinite(f) and math.isfinite(hf)):
        raise ValueError("llama3 scaling needs factor > 0, 0 < low_freq_factor < high_freq_factor, original_ctx > 0")
    out = np.empty_like(theta)
    for r in range(h):
        lam = 2.0 * math.pi / theta[r]
        if lam < c / hf:
            out[r] = theta[r]
        elif lam > c / lf:
            out[r] = theta[r] / f
        else:
            t = (c / lam - lf) / (hf - lf)
            out[r] = (1.0 - t) * theta[r] / f + t * theta[r]
    return out


def window_table(base: float, d: int, k: float, N: int, scaling: dict | None = None):
    """Integer window widths W_r = floor(min(k * lambda'_r, N)), lambda'_r = 2 pi / theta'_r.

    Eq. 2 and Eq. 3.  The predicate is "distance z <= w_r" with integer z, so the integer
    part of w_r decides.  k = inf gives W_r = N for every pair (full attention).
    Returns (W int64[d/2], theta' float64[d/2]).
    """
    theta = effective_theta(base, d, scaling)
    W = np.empty(d // 2, dtype=np.int64)
    for r in range(d // 2):
        lam = 2.0 * math.pi / theta[r]
        w = k * lam
        W[r] = N if not (w < N) else int(math.floor(w))
    return W, theta


def window_table_family(base: float, d: int, N: int, scaling: dict | None = None, *, profile: str = "constant",
                        k_hi: float = 2.0, k_lo: float | None = None, gamma: float = 1.0, beta: float = 0.0,
                        cap: float | None = None, a: float = 0.0, nope_fraction: float = 0.0):
    """The window family of App. A:  w_r = min(max(k_r * lambda'_r**gamma + a*(r+1)/(d/2), beta), cap),
    then W_r = floor(min(w_r, N)) as in Eq. 3.

    k_r is the retention profile over the pair index r = 0 (highest frequency) .. d/2-1:
    "constant" k_hi; "arithmetic" falls from k_hi to k_lo by a constant amount per pair
    (k_r = k_hi - (k_hi - k_lo)/(d/2 - 1) * r; 16 -> 2 is the paper's variable-k profile);
    "geometric" falls by a constant ratio per pair (k_r = k_hi * (k_lo/k_hi)**(r/(d/2 - 1))).
    cap = None means no ceiling other than N.  nope_fraction: that share of the pairs, taken
    from the low-frequency end and rounded to the nearest whole pair, is position-free: its
    rotation is removed (theta'_r = 0) and it is kept at every distance (W_r = N).
    The default arguments are Eq. 3 with k = 2.  Returns (W int64[d/2], theta' float64[d/2]).
    """
    if profile not in ("constant", "arithmetic", "geometric"):
        raise ValueError("unknown profile")
    theta = effective_theta(base, d, scaling).copy()
    h = d // 2
    k_lo = k_hi if k_lo is None else k_lo
    n_free = int(math.floor(nope_fraction * h + 0.5))
    W = np.empty(h, dtype=np.int64)
    for r in range(h):
        if r >= h - n_free:
            theta[r] = 0.0
            W[r] = N
            continue
        lam = 2.0 * math.pi / theta[r]
        if profile == "constant" or h == 1:
            k_r = k_hi
        elif profile == "arithmetic":
            k_r = k_hi - (k_hi - k_lo) / (h - 1) * r
        else:
            k_r = k_hi * math.pow(k_lo / k_hi, r / (h - 1))
        lam_g = lam if gamma == 1.0 else math.pow(lam, gamma)
        w = k_r * lam_g + a * (r + 1) / h
        w = max(w, beta)
        if cap is not None:
            w = min(w, cap)
        W[r] = N if not (w < N) else int(math.floor(w))
    return W, theta


# ----------------------------------------------------------------------------------------
# RoPE, half-split layout: pair r is dims (r, r + d/2)  (Sec. 3.1)
# ----------------------------------------------------------------------------------------


def rope_half_split(x: np.ndarray, theta: np.ndarray, pos0: int = 0, round_bf16: bool = True) -> np.ndarray:
    """Rotate x[..., N, d] pair by pair by the angle pos * theta_r, pos = pos0 + row index.

    x'_r = x_r cos - x_{r+h} sin ;  x'_{r+h} = x_{r+h} cos + x_r sin.  fp64, then one
    rounding to bf16 (round_bf16=False returns the unrounded fp64 rotation).
    """
    x = np.asarray(x, dtype=np.float64)
    N, d = x.shape[-2], x.shape[-1]
    h = d // 2
    pos = (pos0 + np.arange(N, dtype=np.float64))[:, None]
    ang = pos * theta[None, :]
    c, s = np.cos(ang), np.sin(ang)
    lo, hi = x[..., :h], x[..., h:]
    out = np.concatenate([lo * c - hi * s, hi * c + lo * s], axis=-1)
    return round_to_bf16(out) if round_bf16 else out


# ----------------------------------------------------------------------------------------
# Attention, per-term definition (Eq. 1 + the predicate under Eq. 3), one head
# ----------------------------------------------------------------------------------------


def _softmax_row(s: np.ndarray, V: np.ndarray):
    """Plain softmax over the finite entries of s; returns (o, lse)."""
    mu = np.max(s)
    p = np.exp(s - mu)  # exp(-inf) = 0 for dropped keys
    ell = np.sum(p)
    o = (p[:, None] * V).sum(axis=0) / ell
    return o, mu + math.log(ell)


def windowed_scores_row(q: np.ndarray, K: np.ndarray, W: np.ndarray, n: int) -> np.ndarray:
    """Scaled scores of query row n (rotated q[d]) against rotated keys K[0..n] (K[n+1, d]).

    s_m = (1/sqrt d) * sum over pairs r with (n - m) <= W_r of (q_r K_{m,r} + q_{r+h} K_{m,r+h}).
    A key for which no pair is live is dropped (score -inf): beyond the widest window a key
    is unreachable, which is what makes a uniform table the ordinary sliding window.
    """
    d = q.shape[0]
    h = d // 2
    Kn = K[: n + 1]
    per_pair = q[None, :h] * Kn[:, :h] + q[None, h:] * Kn[:, h:]  # [n+1, h]
    z = (n - np.arange(n + 1, dtype=np.int64))[:, None]
    live = z <= W[None, :]
    s = np.where(live, per_pair, 0.0).sum(axis=1) / math.sqrt(d)
    s[~live.any(axis=1)] = -np.inf
    return s


def attention_rows(Q, K, V, W, rows):
    """Windowed causal attention of one head for the listed query rows.

    Q[N,d], K[N,d] rotated, V[N,d]; returns (O[len(rows), d], LSE[len(rows)]), natural log.
    """
    rows = list(rows)
    d = Q.shape[1]
    O = np.empty((len(rows), d), dtype=np.float64)
    LSE = np.empty(len(rows), dtype=np.float64)
    for i, n in enumerate(rows):
        s = windowed_scores_row(Q[n], K, W, n)
        O[i], LSE[i] = _softmax_row(s, V[: n + 1])
    return O, LSE


def attention_appended_rows(Qc, K, V, W, n0, rows=None):
    """Appended rows (App. C, "The interval itself"; Sec. 7.3 runs prefill in such chunks): the
    context already holds keys 0..n0-1; the Nq new rows sit at positions n0..n0+Nq-1 and see keys
    0..n0+Nq-1.  Qc[Nq,d] rotated at those positions, K[Nk,d] rotated, V[Nk,d], Nk = n0 + Nq.
    Each row is the row of the single-shot definition at its position.  `rows` indexes Qc.
    Returns (O[len(rows), d], LSE[len(rows)]).
    """
    Nq, d = Qc.shape
    assert K.shape[0] == n0 + Nq and V.shape[0] == n0 + Nq
    rows = range(Nq) if rows is None else list(rows)
    O = np.empty((len(rows), d), dtype=np.float64)
    LSE = np.empty(len(rows), dtype=np.float64)
    for j, i in enumerate(rows):
        n = n0 + i
        s = windowed_scores_row(Qc[i], K, W, n)
        O[j], LSE[j] = _softmax_row(s, V[: n + 1])
    return O, LSE


def attention_gqa(Q, K, V, W, rows=None):
    """All heads: Q[B,Hq,N,d], K/V[B,Hkv,N,d]; query head hq reads KV head hq // (Hq/Hkv)."""
    B, Hq, N, d = Q.shape
    Hkv = K.shape[1]
    g = Hq // Hkv
    rows = range(N) if rows is None else list(rows)
    nr = len(rows)
    O = np.empty((B, Hq, nr, d))
    LSE = np.empty((B, Hq, nr))
    for b in range(B):
        for hq in range(Hq):
            O[b, hq], LSE[b, hq] = attention_rows(Q[b, hq], K[b, hq // g], V[b, hq // g], W, rows)
    return O, LSE


def decode(q, Kc, Vc, W):
    """One new token per sequence: q[B,Hq,d] sits at position L-1 of caches Kc/Vc[B,Hkv,L,d]
    (the cache already holds the new token's own key and value).  Returns (O[B,Hq,d], LSE[B,Hq]).
    """
    B, Hq, d = q.shape
    Hkv, L = Kc.shape[1], Kc.shape[2]
    g = Hq // Hkv
    O = np.empty((B, Hq, d))
    LSE = np.empty((B, Hq))
    for b in range(B):
        for hq in range(Hq):
            s = windowed_scores_row(q[b, hq], Kc[b, hq // g], W, L - 1)
            O[b, hq], LSE[b, hq] = _softmax_row(s, Vc[b, hq // g])
    return O, LSE


def brute_force_attention(Q, K, V, W):
    """Triple loop over (n, m, r) in pure Python; tiny N only.  One head."""
    N, d = Q.shape
    h = d // 2
    O = [[0.0] * d for _ in range(N)]
    LSE = [0.0] * N
    for n in range(N):
        sc = []
        for m in range(n + 1):
            z = n - m
            acc, cnt = 0.0, 0
            for r in range(h):
                if z <= int(W[r]):
                    acc += float(Q[n, r]) * float(K[m, r]) + float(Q[n, r + h]) * float(K[m, r + h])
                    cnt += 1
            sc.append(acc / math.sqrt(d) if cnt else -math.inf)
        mu = max(sc)
        p = [math.exp(v - mu) if v != -math.inf else 0.0 for v in sc]
        ell = math.fsum(p)
        for c in range(d):
            O[n][c] = math.fsum(p[m] * float(V[m, c]) for m in range(n + 1)) / ell
        LSE[n] = mu + math.log(ell)
    return np.array(O), np.array(LSE)


# ----------------------------------------------------------------------------------------
# Term counts (Sec. 4: cost = number of query-key inner-product terms)
# ----------------------------------------------------------------------------------------


def kept_terms_row(W: np.ndarray, n: int) -> int:
    """Terms kept in query row n (positions from 0; the row has n+1 causal cells z = 0..n)."""
    return int(sum(min(int(w), n) + 1 for w in W))


def kept_terms_prefill(W: np.ndarray, N: int) -> int:
    """Terms kept over all rows 0..N-1 of one head."""
    n = np.arange(N, dtype=np.int64)[:, None]
    return int((np.minimum(np.asarray(W, dtype=np.int64)[None, :], n) + 1).sum(dtype=np.int64))


def kept_terms_interval(W: np.ndarray, n0: int, n1: int) -> int:
    """Terms kept over the rows n0..n1-1 (positions from 0) of one head: the appended-rows step
    of App. C; [0, N) is the whole prefill, [L-1, L) the decode step."""
    n = np.arange(n0, n1, dtype=np.int64)[:, None]
    return int((np.minimum(np.asarray(W, dtype=np.int64)[None, :], n) + 1).sum(dtype=np.int64))


def pruned_share_interval(W, d, n0, n1) -> float:
    full = (d // 2) * (n1 * (n1 + 1) // 2 - n0 * (n0 + 1) // 2)
    return 1.0 - kept_terms_interval(W, n0, n1) / full


def kept_terms_decode(W: np.ndarray, L: int) -> int:
    return kept_terms_row(W, L - 1)


def full_terms_prefill(d: int, N: int) -> int:
    return (d // 2) * (N * (N + 1) // 2)


def pruned_share_prefill(W, d, N) -> float:
    return 1.0 - kept_terms_prefill(W, N) / full_terms_prefill(d, N)


def pruned_share_row(W, d, n) -> float:
    return 1.0 - kept_terms_row(W, n) / ((d // 2) * (n + 1))


# ----------------------------------------------------------------------------------------
# Closed forms (Eq. 5; App. C Steps 1-3), default window only
# ----------------------------------------------------------------------------------------


def closed_F(n: float, w_min: float) -> float:
    """Primitive F(n) = n^2 (ln(n/w_min) - 3/2) + 2 w_min n  (App. C, Step 1)."""
    return n * n * (math.log(n / w_min) - 1.5) + 2.0 * w_min * n


def closed_R(n0: float, n1: float, k: float, base: float) -> float:
    """Reduction over the row interval [n0, n1]: [F]_{n0}^{n1} / ((n1^2 - n0^2) ln B)."""
    w_min = 2.0 * math.pi * k
    return (closed_F(n1, w_min) - closed_F(n0, w_min)) / ((n1 * n1 - n0 * n0) * math.log(base))


def closed_prefill(N: float, k: float, base: float) -> float:
    """Eq. 5: (ln(N/w_min) - 3/2) / ln B."""
    return (math.log(N / (2.0 * math.pi * k)) - 1.5) / math.log(base)


def closed_last_row(N: float, k: float, base: float) -> float:
    """Last row evaluated directly (App. C, Step 2): [ln(N/w_min) - 1 + w_min/N] / ln B."""
    w_min = 2.0 * math.pi * k
    return (math.log(N / w_min) - 1.0 + w_min / N) / math.log(base)


def closed_rho_star(n: float, k: float, base: float, d: int) -> float:
    """Saturation boundary rho*(n) = (d/2) ln(n/w_min) / ln B."""
    return 0.5 * d * math.log(n / (2.0 * math.pi * k)) / math.log(base)


# ----------------------------------------------------------------------------------------
# Second named mode: "coarse" (the granularity the paper's ports run at, Sec. 3.3 / Sec. 5 /
# App. E).  Prefill: the live set is decided per (query tile, key tile) and its boundary is
# rounded outward to whole groups of G pairs counted from the low-frequency end; tiles that
# touch the diagonal use every pair with the causal mask.  Decode: per key, the first live
# pair is rounded down to a multiple of 8 pairs (one 16-byte load of bf16 per half).
# ----------------------------------------------------------------------------------------


def coarse_first_pair(W: np.ndarray, z_min: int, G: int) -> int:
    """First pair index kept for a tile whose nearest cell is at distance z_min."""
    h = len(W)
    live = [r for r in range(h) if int(W[r]) >= z_min]
    if not live:
        return h
    r_any = live[0]
    return h - G * (-(-(h - r_any) // G))


def coarse_attention_rows(Q, K, V, W, rows, Tq=128, Tk=128, G=8):
    """Coarse-mode prefill for one head, listed rows.  Tiles are aligned at position 0."""
    rows = list(rows)
    N, d = Q.shape
    h = d // 2
    O = np.empty((len(rows), d))
    LSE = np.empty(len(rows))
    for i, n in enumerate(rows):
        q0 = (n // Tq) * Tq  # first row of the query tile
        q1 = min(q0 + Tq, N) - 1
        s = np.empty(n + 1)
        for k0 in range(0, n + 1, Tk):
            k1 = min(k0 + Tk, N) - 1  # last key of the tile
            if k1 > q0:  # some cell of the tile is above the diagonal: masked band, full depth
                r0 = 0
            else:
                r0 = coarse_first_pair(W, q0 - k1, G)
            m = np.arange(k0, min(k1, n) + 1)
            if r0 >= h:
                s[m] = -np.inf
                continue
            per_pair = Q[n, None, r0:h] * K[m, r0:h] + Q[n, None, h + r0 :] * K[m, h + r0 :]
            s[m] = per_pair.sum(axis=1) / math.sqrt(d)
        del q1
        O[i], LSE[i] = _softmax_row(s, V[: n + 1])
    return O, LSE


def coarse_kept_terms_prefill(W, N, Tq=128, Tk=128, G=8) -> int:
    """Terms the coarse mode keeps (causal cells x pairs used), one head.  Needs a
    non-decreasing table (the live set is then a contiguous low-frequency slice)."""
    W = np.asarray(W, dtype=np.int64)
    assert np.all(np.diff(W) >= 0)
    h = len(W)
    total = 0
    for q0 in range(0, N, Tq):
        q1 = min(q0 + Tq, N) - 1
        k0 = np.arange(0, q1 + 1, Tk, dtype=np.int64)
        k1 = np.minimum(k0 + Tk, N) - 1
        diag = k1 > q0
        # off-diagonal tiles: every cell is causal; pairs from the rounded boundary up
        r_any = np.searchsorted(W, q0 - k1[~diag], side="left")  # first r with W_r >= z_min
        used = np.minimum(G * (-(-(h - r_any) // G)), h)
        total += int(((q1 - q0 + 1) * (k1[~diag] - k0[~diag] + 1) * used).sum())
        # tiles touching the diagonal: all pairs, causal cells only
        for a, b in zip(k0[diag], k1[diag]):
            n = np.arange(max(q0, int(a)), q1 + 1)
            total += int((np.minimum(b, n) - a + 1).sum()) * h
    return total


def coarse_decode_first_pair(W: np.ndarray, z, chunk_pairs: int = 8):
    """First pair kept at distance z (scalar or array): the first live pair rounded down to a
    multiple of chunk_pairs.  Needs a non-decreasing table."""
    W = np.asarray(W, dtype=np.int64)
    assert np.all(np.diff(W) >= 0)
    first_live = np.searchsorted(W, z, side="left")  # number of pairs with W_r < z
    return np.where(first_live >= len(W), len(W), (first_live // chunk_pairs) * chunk_pairs)


def coarse_decode(q, Kc, Vc, W, chunk_pairs=8):
    B, Hq, d = q.shape
    h = d // 2
    Hkv, L = Kc.shape[1], Kc.shape[2]
    g = Hq // Hkv
    O = np.empty((B, Hq, d))
    LSE = np.empty((B, Hq))
    r0 = coarse_decode_first_pair(W, L - 1 - np.arange(L, dtype=np.int64), chunk_pairs)
    keep = np.arange(h)[None, :] >= r0[:, None]  # [L, h]
    for b in range(B):
        for hq in range(Hq):
            Kh = Kc[b, hq // g]
            per_pair = q[b, hq, None, :h] * Kh[:, :h] + q[b, hq, None, h:] * Kh[:, h:]
            s = np.where(keep, per_pair, 0.0).sum(axis=1) / math.sqrt(d)
            s[~keep.any(axis=1)] = -np.inf
            O[b, hq], LSE[b, hq] = _softmax_row(s, Vc[b, hq // g])
    return O, LSE


def coarse_kept_terms_decode(W, L, chunk_pairs=8) -> int:
    r0 = coarse_decode_first_pair(W, L - 1 - np.arange(L, dtype=np.int64), chunk_pairs)
    return int((len(W) - r0).sum())
