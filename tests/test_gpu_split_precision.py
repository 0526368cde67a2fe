"""GPU parity of the split-precision prefill (App. D: a low-precision product split to recover accuracy;
Sec. 6.2: tasks scored with fp32 attention scores) against the per-term definition on the fp32 inputs.

Both sides rotate the same unrotated fp32 draws themselves (the oracle in fp64, rounded once to fp32; the
library with atf_rope_f32), so no oracle input comes from the GPU.  Tolerances: the LSE within
1.5e-5 x max(1, largest |logit| of the checked rows) (derived and pinned on the CPU in
test_oracle_split_precision.py), O as for every prefill (P and V are bf16 there too); term counts bit-exact.
The ordinary bf16 path, given the same values rounded to bf16, must be at least 20 times further from the
fp32 definition: that is what the mode is for."""
import numpy as np
import pytest
import torch

import atf_inputs as gen
from oracle import atf_oracle as orc

pytestmark = pytest.mark.gpu

O_MAX, O_MEAN = 2e-2, 2e-3


def split_lse_tol(max_abs_logit):
    return 1.5e-5 * max(1.0, max_abs_logit)


@pytest.fixture(scope="module")
def atf():
    import paper_2608_02947_b200 as m
    m.lib()
    return m


def _rotated(atf, w, theta):
    """(GPU fp32 rotated Q, K, V) and the oracle's own rotation of the same draws, as fp32 values in fp64."""
    Q, K, V = gen.prefill_inputs_f32(w)
    Qg, Kg = Q.cuda(), K.cuda()
    atf.atf_rope_f32(Qg, theta)
    atf.atf_rope_f32(Kg, theta)
    Qo = orc.rope_half_split(Q.numpy().astype(np.float64), theta, 0, round_bf16=False).astype(np.float32)
    Ko = orc.rope_half_split(K.numpy().astype(np.float64), theta, 0, round_bf16=False).astype(np.float32)
    # the two rotations agree to an fp32 unit in the last place (sincos of two libraries)
    for a, b in ((Qg, Qo), (Kg, Ko)):
        diff = np.abs(a.cpu().numpy().astype(np.float64) - b.astype(np.float64))
        assert (diff <= 2.0 ** -22 * np.maximum(np.abs(b), 2.0 ** -10)).all()
    return Qg, Kg, V.cuda(), Qo.astype(np.float64), Ko.astype(np.float64), gen.to_f64(V)


def _case(atf, w, mode, table=None, rows=None, compare_bf16=True):
    Wo, theta = orc.window_table(w.base, w.d, w.k, w.N, w.scaling)
    if table is not None:
        Wo = np.asarray(table, dtype=np.int64)
    Qg, Kg, Vg, Qo, Ko, Vo = _rotated(atf, w, theta)
    kept = torch.zeros(w.B * w.Hq, dtype=torch.int64, device="cuda")
    O, LSE = atf.atf_prefill_split(Qg, Kg, Vg, table=torch.from_numpy(Wo), mode=mode, kept_terms=kept)
    torch.cuda.synchronize()
    atf.binding.check_status()
    want = orc.kept_terms_prefill(Wo, w.N) if mode == atf.ATF_MODE_EXACT else orc.coarse_kept_terms_prefill(Wo, w.N)
    assert kept.cpu().tolist() == [want] * (w.B * w.Hq)
    rows = list(range(w.N)) if rows is None else rows
    g = w.Hq // w.Hkv
    if compare_bf16:
        O16, L16 = atf.atf_prefill(Qg.to(torch.bfloat16), Kg.to(torch.bfloat16), Vg, table=torch.from_numpy(Wo), mode=mode)
    e_split, e_bf16, smax_all = [], [], 0.0
    for b in range(w.B):
        for hq in range(w.Hq):
            hk = hq // g
            if mode == atf.ATF_MODE_EXACT:
                Or, Lr = orc.attention_rows(Qo[b, hq], Ko[b, hk], Vo[b, hk], Wo, rows)
                smax = max(np.abs(s[np.isfinite(s)]).max() for s in
                           (orc.windowed_scores_row(Qo[b, hq, n], Ko[b, hk], Wo, n) for n in rows[:: max(1, len(rows) // 64)]))
            else:
                Or, Lr = orc.coarse_attention_rows(Qo[b, hq], Ko[b, hk], Vo[b, hk], Wo, rows)
                smax = np.abs(Lr).max() + 8.0  # a logit is at most the LSE; the largest sits within a few units of it
            smax_all = max(smax_all, smax)
            Og = gen.to_f64(O[b, hq])[rows]
            err = np.abs(Og - Or)
            assert np.isfinite(Og).all()
            assert err.max() <= O_MAX and err.mean() <= O_MEAN, (b, hq, err.max(), err.mean())
            le = np.abs(LSE[b, hq].double().cpu().numpy()[rows] - Lr)
            assert le.max() <= split_lse_tol(smax), (b, hq, le.max(), smax)
            e_split.append(le)
            if compare_bf16:
                e_bf16.append(np.abs(L16[b, hq].double().cpu().numpy()[rows] - Lr))
    if compare_bf16 and w.N >= 256:
        es, eb = np.concatenate(e_split), np.concatenate(e_bf16)
        assert eb.mean() >= 20 * es.mean(), (eb.mean(), es.mean())
    return float(np.concatenate(e_split).max()), smax_all


@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("B,Hq,Hkv,d,N", [(1, 2, 1, 64, 1), (1, 2, 1, 64, 129), (2, 4, 2, 128, 300), (1, 3, 1, 64, 700),
                                          (1, 2, 2, 128, 1000)])
def test_split_small(atf, mode, B, Hq, Hkv, d, N):
    w = gen.Workload("split", B, Hq, Hkv, d, N, 1e4, 2.0, None, gen.SEED0 + 200 + N)
    _case(atf, w, mode)


@pytest.mark.parametrize("d", [64, 128])
def test_split_outlier_channels(atf, d):
    """Four pairs scaled by 8: logits in the hundreds, where bf16 inputs are off by tenths."""
    w = gen.Workload("split-outlier", 1, 2, 1, d, 900, 1e4, 2.0, None, gen.SEED0 + 210 + d, True)
    e, smax = _case(atf, w, 0)
    assert smax > 50
    _case(atf, w, 1)


def test_split_dropped_keys_and_uniform_table(atf):
    w = gen.Workload("split", 1, 2, 1, 64, 900, 1e4, 2.0, None, gen.SEED0 + 220)
    tab = np.minimum(np.array([3 * (r + 1) ** 2 for r in range(32)], dtype=np.int64), 400)
    _case(atf, w, 0, table=tab)
    _case(atf, w, 1, table=tab)
    _case(atf, w, 0, table=np.full(32, 900, dtype=np.int64))   # k = inf: every term


def test_split_llama_8k_sampled_rows(atf):
    """Llama-3.2-3B head shape (d = 128, llama3-scaled windows) at 8K, sampled rows (first / last tile, rows
    next to every window boundary, random rows), one batch and two KV groups."""
    w = gen.Workload("llama-split", 1, 6, 2, 128, 8192, 5e5, 2.0, gen.LLAMA3_SCALING, gen.SEED0 + 230)
    Wo, _ = orc.window_table(w.base, w.d, w.k, w.N, w.scaling)
    rows = gen.sample_rows(w.N, Wo, 64, 77)
    _case(atf, w, 0, rows=rows)
    _case(atf, w, 1, rows=rows)


def test_split_refusals(atf):
    Q = torch.zeros((1, 2, 128, 64), dtype=torch.float32, device="cuda")
    V = torch.zeros((1, 1, 128, 64), dtype=torch.bfloat16, device="cuda")
    K = torch.zeros((1, 1, 128, 64), dtype=torch.float32, device="cuda")
    with pytest.raises(atf.AtfError):
        atf.atf_prefill_split(Q.to(torch.bfloat16), K, V)          # Q must be fp32
    with pytest.raises(atf.AtfError):
        atf.atf_prefill_split(Q, K, V, causal=False)
    with pytest.raises(atf.AtfError):
        atf.atf_prefill_split(Q, K[:, :, :64].contiguous(), V)


def test_split_appended_rows_bit_identical_to_single_shot(atf):
    """Rows cut off at an aligned and at an unaligned position, computed as appended rows, have the bits of the
    single shot (both modes)."""
    w = gen.Workload("split", 2, 4, 2, 128, 1100, 1e4, 2.0, None, gen.SEED0 + 240)
    Wo, theta = orc.window_table(w.base, w.d, w.k, w.N, w.scaling)
    Qg, Kg, Vg, *_ = _rotated(atf, w, theta)
    Wt = torch.from_numpy(Wo)
    for mode in (0, 1):
        O, L = atf.atf_prefill_split(Qg, Kg, Vg, table=Wt, mode=mode)
        for n0 in (512, 333, 1099):
            kept = torch.zeros(w.B * w.Hq, dtype=torch.int64, device="cuda")
            Oc, Lc = atf.atf_prefill_split(Qg[:, :, n0:].contiguous(), Kg, Vg, table=Wt, mode=mode, kept_terms=kept)
            assert torch.equal(Oc, O[:, :, n0:]) and torch.equal(Lc, L[:, :, n0:]), (mode, n0)
            if mode == 0:
                assert kept.cpu().tolist() == [orc.kept_terms_interval(Wo, n0, w.N)] * (w.B * w.Hq)
    atf.binding.check_status()
