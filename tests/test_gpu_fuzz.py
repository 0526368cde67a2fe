"""Randomised small shapes against the fp64 oracle: ragged lengths, batch and GQA ratios, both
head sizes, random non-decreasing tables (with dropped keys), both modes, appended rows, and
decode at the same cache.  Seeds are fixed; every case is checked element by element."""
import numpy as np
import pytest
import torch

import atf_inputs as gen
from oracle import atf_oracle as orc

pytestmark = pytest.mark.gpu

O_MAX, O_MEAN, LSE_TOL = 2e-2, 2e-3, 1e-3


@pytest.fixture(scope="module")
def atf():
    import paper_2608_02947_b200 as m
    m.lib()
    return m


def _random_table(rng, h, N):
    kind = rng.integers(0, 4)
    if kind == 0:   # geometric, like Eq. 3
        W = np.minimum(np.floor(4 * np.pi * (N ** (np.arange(h) / (h - 1)))), N)
    elif kind == 1:  # arbitrary non-decreasing, may drop far keys
        W = np.sort(rng.integers(0, max(2, N // 2), size=h))
    elif kind == 2:  # few distinct values, long plateaus, some at N
        W = np.sort(rng.choice([0, 1, 31, 32, 127, 128, 129, 255, 256, N // 2, N], size=h))
    else:           # everything live
        W = np.full(h, N)
    return W.astype(np.int64)


@pytest.mark.parametrize("seed", range(12))
def test_random_small_case(atf, seed):
    rng = np.random.default_rng(1000 + seed)
    d = int(rng.choice([64, 128]))
    h = d // 2
    Hkv = int(rng.integers(1, 3))
    g = int(rng.choice([1, 2, 3, 4, 7, 8]))
    Hq = Hkv * g
    B = int(rng.integers(1, 3))
    N = int(rng.choice([1, 2, 63, 127, 128, 129, 255, 257, 300, 383, 511, 640]))
    mode = int(rng.integers(0, 2))
    W = _random_table(rng, h, N)
    theta = orc.effective_theta(1e4, d)
    Q = gen.normal_bf16((B, Hq, N, d), 5000 + seed)
    K = gen.normal_bf16((B, Hkv, N, d), 6000 + seed)
    V = gen.normal_bf16((B, Hkv, N, d), 7000 + seed)
    Qg, Kg, Vg = Q.cuda(), K.cuda(), V.cuda()
    th = torch.from_numpy(theta)
    atf.atf_rope(Qg, th)
    atf.atf_rope(Kg, th)
    tab = torch.from_numpy(W)
    kept = torch.zeros(B * Hq, dtype=torch.int64, device="cuda")
    O, L = atf.atf_prefill(Qg, Kg, Vg, table=tab, mode=mode, kept_terms=kept)
    n0 = int(rng.integers(0, N))
    Oc, Lc = atf.atf_prefill(Qg[:, :, n0:].contiguous(), Kg, Vg, table=tab, mode=mode)
    Od = atf.atf_decode(Qg[:, :, -1].contiguous(), Kg, Vg, table=tab, mode=mode) if g <= 8 else None
    torch.cuda.synchronize()
    atf.binding.check_status()
    tag = dict(seed=seed, d=d, B=B, Hq=Hq, Hkv=Hkv, N=N, mode=mode, n0=n0)
    assert torch.equal(Oc.view(torch.int16), O[:, :, n0:].contiguous().view(torch.int16)), tag
    assert torch.equal(Lc, L[:, :, n0:]), tag
    Qr = orc.rope_half_split(gen.to_f64(Q), theta)
    Kr = orc.rope_half_split(gen.to_f64(K), theta)
    Vr = gen.to_f64(V)
    if mode == 0:
        O_ref, L_ref = orc.attention_gqa(Qr, Kr, Vr, W)
        assert kept.cpu().tolist() == [orc.kept_terms_prefill(W, N)] * (B * Hq), tag
        O_dec = orc.decode(Qr[:, :, -1], Kr, Vr, W)
    else:
        O_ref = np.empty((B, Hq, N, d))
        L_ref = np.empty((B, Hq, N))
        for b in range(B):
            for hq in range(Hq):
                O_ref[b, hq], L_ref[b, hq] = orc.coarse_attention_rows(Qr[b, hq], Kr[b, hq // g], Vr[b, hq // g], W,
                                                                       range(N))
        assert kept.cpu().tolist() == [orc.coarse_kept_terms_prefill(W, N)] * (B * Hq), tag
        O_dec = orc.coarse_decode(Qr[:, :, -1], Kr, Vr, W)
    O_dec = O_dec[0] if isinstance(O_dec, tuple) else O_dec
    err = np.abs(gen.to_f64(O) - O_ref)
    assert np.isfinite(gen.to_f64(O)).all(), tag
    assert err.max() <= O_MAX and err.mean() <= O_MEAN, (tag, err.max(), err.mean())
    assert np.abs(L.double().cpu().numpy() - L_ref).max() <= LSE_TOL, tag
    if Od is not None:
        errd = np.abs(gen.to_f64(Od) - O_dec)
        assert errd.max() <= O_MAX and errd.mean() <= O_MEAN, (tag, errd.max())
