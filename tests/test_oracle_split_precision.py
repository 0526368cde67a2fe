"""What the oracle says about score precision (CPU only): the ground for the tolerance of the
split-precision prefill (App. D, "Precision as the other side of the compute-accuracy trade": the paper
splits a low-precision product to recover accuracy; Sec. 6.2 scores five tasks with fp32 attention scores).

The reference of that mode is the per-term definition (attention_rows) on Q and K given in fp32, widened
exactly.  A bf16 x bf16 tensor-core product can represent such an input as hi + lo with hi = bf16(x) and
lo = bf16(x - hi); the score then is q_hi k_hi + q_hi k_lo + q_lo k_hi (the lo * lo term is left out).
These tests fix, with the oracle and plain arithmetic only,
  - that hi + lo reproduces an fp32 value to 2^-17 of its magnitude (so a product term to ~2^-16),
  - that the LSE of the definition moves by less than SPLIT_LSE_TOL = 1.5e-5 x max(1, largest |logit| of the
    rows) when the inputs are replaced by hi + lo and the lo * lo terms are dropped: a logit is a sum of
    product terms each good to ~2^-16 of its size, so the bound scales with the logits (the outlier variant
    of the inputs, four pairs scaled by 8, has logits up to ~160 and is held to the same rule),
  - and that rounding the inputs to bf16 (what the ordinary path is given) moves it by over 100 times more
    (2^8 in theory): the tolerance separates the two modes.
"""
import numpy as np

from oracle import atf_oracle as orc


def split_lse_tol(max_abs_logit):
    """Tolerance of the split-precision mode on the LSE (natural log), see the module text."""
    return 1.5e-5 * max(1.0, max_abs_logit)


def _inputs(N, d, seed, outlier):
    rng = np.random.default_rng(seed)
    Q = rng.standard_normal((N, d)).astype(np.float32)
    K = rng.standard_normal((N, d)).astype(np.float32)
    V = orc.round_to_bf16(rng.standard_normal((N, d)))
    if outlier:
        h = d // 2
        for t in (Q, K):
            t[:, h - 4:h] *= 8
            t[:, d - 4:d] *= 8
    theta = orc.effective_theta(1e4, d)
    # rotation in fp64, kept in fp32: the inputs of the split mode are rotated values that were never rounded to bf16
    Q = orc.rope_half_split(Q.astype(np.float64), theta, 0, round_bf16=False).astype(np.float32)
    K = orc.rope_half_split(K.astype(np.float64), theta, 0, round_bf16=False).astype(np.float32)
    return Q, K, V


def _split(x32):
    hi = orc.round_to_bf16(x32.astype(np.float64))
    lo = orc.round_to_bf16(x32.astype(np.float64) - hi)
    return hi, lo


def test_hi_plus_lo_holds_an_fp32_value_to_2_pow_minus_17():
    rng = np.random.default_rng(5)
    x = (rng.standard_normal(200000) * np.exp(rng.uniform(-20, 20, 200000))).astype(np.float32)
    hi, lo = _split(x)
    rel = np.abs(x.astype(np.float64) - hi - lo) / np.abs(x.astype(np.float64))
    assert rel.max() <= 2.0 ** -17
    # and hi alone, the ordinary path's input, only to 2^-9
    assert (np.abs(x.astype(np.float64) - hi) / np.abs(x.astype(np.float64))).max() > 2.0 ** -10


def _lse_with_dropped_lo_lo(Qh, Ql, Kh, Kl, V, W, rows):
    """The definition with every product term q k replaced by q_hi k_hi + q_hi k_lo + q_lo k_hi.  The rule is
    linear in the products, so this is definition(hi + lo inputs) minus the part that comes from lo * lo alone:
    scores(q_hi + q_lo, k_hi + k_lo) - scores(q_lo, k_lo), both with the same window."""
    out = np.empty(len(rows))
    for i, n in enumerate(rows):
        s = orc.windowed_scores_row(Qh[n] + Ql[n], Kh + Kl, W, n)
        s_ll = orc.windowed_scores_row(Ql[n], Kl, W, n)
        live = np.isfinite(s)
        s = np.where(live, s - np.where(live, s_ll, 0.0), s)
        out[i] = orc._softmax_row(s, V[: n + 1])[1]
    return out


def test_split_inputs_keep_the_lse_and_bf16_inputs_do_not():
    N, d = 700, 64
    W, _ = orc.window_table(1e4, d, 2.0, N)
    rows = list(range(0, N, 7)) + [N - 1]
    for outlier in (False, True):
        Q, K, V = _inputs(N, d, 11 + outlier, outlier)
        Q64, K64 = Q.astype(np.float64), K.astype(np.float64)
        _, ref = orc.attention_rows(Q64, K64, V, W, rows)
        Qh, Ql = _split(Q)
        Kh, Kl = _split(K)
        e_split = np.abs(_lse_with_dropped_lo_lo(Qh, Ql, Kh, Kl, V, W, rows) - ref).max()
        _, l16 = orc.attention_rows(Qh, Kh, V, W, rows)
        e_bf16 = np.abs(l16 - ref).max()
        smax = max(np.abs(orc.windowed_scores_row(Q64[n], K64, W, n)[: n + 1]).max() for n in rows)
        assert (smax > 100) == outlier          # the outlier variant really has large logits
        assert e_split <= split_lse_tol(smax) / 1.5, (outlier, e_split, smax)
        assert e_bf16 >= 20 * split_lse_tol(smax), (outlier, e_bf16)   # far outside the split mode's tolerance
        assert e_bf16 >= 100 * e_split
