"""GPU parity of the appended-rows entry point (atf_prefill_chunk, through the binding): the
rows of a chunk against the fp64 oracle, bit-identity with the single-shot prefill (Sec. 7.3:
chunked prefill is bit-identical to single shot), and term counts of the row interval."""
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


def _rotated(atf, w):
    Q, K, V = gen.prefill_inputs(w)
    Wt, theta = atf.atf_window_table(w.base, w.d, w.k, w.N, w.scaling)
    Qg, Kg, Vg = Q.cuda(), K.cuda(), V.cuda()
    atf.atf_rope(Qg, theta)
    atf.atf_rope(Kg, theta)
    return Qg, Kg, Vg, Wt


@pytest.mark.parametrize("d,Hq,Hkv,mode", [(128, 4, 2, 0), (64, 2, 1, 0), (128, 2, 1, 1)])
def test_chunk_rows_bit_identical_to_single_shot(atf, d, Hq, Hkv, mode):
    w = gen.Workload("chunk-small", 1, Hq, Hkv, d, 700, 5e5 if d == 128 else 1e6, 2.0, None, gen.SEED0 + 40 + d)
    Qg, Kg, Vg, Wt = _rotated(atf, w)
    W = Wt.numpy().copy()
    W[:8] = np.array([3, 9, 17, 40, 77, 130, 200, 311])  # several pairs end inside 700 tokens
    W = np.sort(W)
    tab = torch.from_numpy(W)
    kept_all = torch.zeros(Hq, dtype=torch.int64, device="cuda")
    O_all, L_all = atf.atf_prefill(Qg, Kg, Vg, table=tab, mode=mode, kept_terms=kept_all)
    for n0 in (1, 100, 128, 255, 256, 300, 450, 699):
        kept = torch.zeros(Hq, dtype=torch.int64, device="cuda")
        O, L = atf.atf_prefill(Qg[:, :, n0:].contiguous(), Kg, Vg, table=tab, mode=mode, kept_terms=kept)
        torch.cuda.synchronize()
        atf.binding.check_status()
        assert torch.equal(O.view(torch.int16), O_all[:, :, n0:].contiguous().view(torch.int16)), n0
        assert torch.equal(L, L_all[:, :, n0:]), n0
        if mode == 0:
            assert kept.cpu().tolist() == [orc.kept_terms_interval(W, n0, w.N)] * Hq, n0
    if mode == 0:
        assert kept_all.cpu().tolist() == [orc.kept_terms_prefill(W, w.N)] * Hq


def test_chunked_prefill_matches_oracle_and_single_shot(atf):
    # three chunks, each seeing only the keys that exist so far (the table is clipped at each
    # chunk's own key count, which never changes a score)
    w = gen.Workload("chunked", 2, 4, 2, 128, 1000, 5e5, 2.0, gen.LLAMA3_SCALING, gen.SEED0 + 41)
    Qg, Kg, Vg, Wt = _rotated(atf, w)
    O_all, L_all = atf.atf_prefill(Qg, Kg, Vg, table=Wt)
    cuts = [0, 300, 812, 1000]
    outs = []
    for a, b in zip(cuts, cuts[1:]):
        Wb, _ = atf.atf_window_table(w.base, w.d, w.k, b, w.scaling)
        outs.append(atf.atf_prefill(Qg[:, :, a:b].contiguous(), Kg[:, :, :b].contiguous(), Vg[:, :, :b].contiguous(),
                                    table=Wb))
    torch.cuda.synchronize()
    atf.binding.check_status()
    O = torch.cat([o for o, _ in outs], dim=2)
    L = torch.cat([l for _, l in outs], dim=2)
    assert torch.equal(O.view(torch.int16), O_all.view(torch.int16))
    assert torch.equal(L, L_all)
    # the last chunk against the oracle's appended rows
    Wo, theta_o = orc.window_table(w.base, w.d, w.k, w.N, w.scaling)
    Q, K, V = gen.prefill_inputs(w)
    Qr = orc.rope_half_split(gen.to_f64(Q), theta_o)
    Kr = orc.rope_half_split(gen.to_f64(K), theta_o)
    Vr = gen.to_f64(V)
    n0 = cuts[-2]
    Og, Lg = outs[-1]
    for b in range(w.B):
        for hq in range(w.Hq):
            hk = hq // (w.Hq // w.Hkv)
            O_ref, L_ref = orc.attention_appended_rows(Qr[b, hq, n0:], Kr[b, hk], Vr[b, hk], Wo, n0)
            err = np.abs(gen.to_f64(Og[b, hq]) - O_ref)
            assert err.max() <= O_MAX and err.mean() <= O_MEAN, (b, hq, err.max(), err.mean())
            assert np.abs(Lg[b, hq].double().cpu().numpy() - L_ref).max() <= LSE_TOL


def test_one_appended_row_equals_decode(atf):
    w = gen.Workload("chunk-decode", 1, 8, 2, 128, 2000, 5e5, 2.0, gen.LLAMA3_SCALING, gen.SEED0 + 42)
    Qg, Kg, Vg, Wt = _rotated(atf, w)
    O1, _ = atf.atf_prefill(Qg[:, :, -1:].contiguous(), Kg, Vg, table=Wt)
    Od = atf.atf_decode(Qg[:, :, -1].contiguous(), Kg, Vg, table=Wt)
    Od = Od[0] if isinstance(Od, tuple) else Od
    torch.cuda.synchronize()
    # two different kernels (tcgen05 prefill, split-K decode): equal within the output tolerance
    err = (O1[:, :, 0].float() - Od.float()).abs()
    assert err.max().item() <= O_MAX and err.mean().item() <= O_MEAN


def test_chunk_rejects_bad_lengths(atf):
    Q = torch.zeros((1, 2, 64, 128), dtype=torch.bfloat16, device="cuda")
    K = torch.zeros((1, 2, 32, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(atf.AtfError):
        atf.atf_prefill(Q, K, K.clone())


def test_last_quarter_of_a_32k_prompt(atf):
    # Llama-3.2-3B shape, N = 32768, the last 8192 rows appended to a 24576-token context
    w = gen.llama32_3b(32768)
    Qg, Kg, Vg, Wt = _rotated(atf, w)
    n0 = 24576
    kept = torch.zeros(w.Hq, dtype=torch.int64, device="cuda")
    O, L = atf.atf_prefill(Qg[:, :, n0:].contiguous(), Kg, Vg, table=Wt, kept_terms=kept)
    torch.cuda.synchronize()
    atf.binding.check_status()
    Wo, theta_o = orc.window_table(w.base, w.d, w.k, w.N, w.scaling)
    assert kept.cpu().tolist() == [orc.kept_terms_interval(Wo, n0, w.N)] * w.Hq
    Q, K, V = gen.prefill_inputs(w)
    rows = [0, 1, 127, 128, 4095, 8191] + list(np.random.default_rng(5).integers(0, 8192, 10))
    for hq in (0, 13, 23):
        hk = hq // (w.Hq // w.Hkv)
        Kr = orc.rope_half_split(gen.to_f64(K[0, hk]), theta_o)
        Qr = orc.rope_half_split(gen.to_f64(Q[0, hq, n0:]), theta_o, pos0=n0)
        O_ref, L_ref = orc.attention_appended_rows(Qr, Kr, gen.to_f64(V[0, hk]), Wo, n0, rows=rows)
        err = np.abs(gen.to_f64(O[0, hq, rows]) - O_ref)
        assert err.max() <= O_MAX and err.mean() <= O_MEAN, (hq, err.max(), err.mean())
        assert np.abs(L[0, hq, rows].double().cpu().numpy() - L_ref).max() <= LSE_TOL


def test_128k_prompt_in_two_64k_chunks_is_the_single_shot(atf):
    """The benchmark's shape run the way Sec. 7.3 runs long prompts: 64K chunks, each seeing the
    keys that exist so far; bit-identical to the single-shot prefill, interval counts exact."""
    w = gen.llama32_3b(131072, seed_off=6)
    Q, K, V = gen.prefill_inputs(w, device="cuda")
    Wt, theta = atf.atf_window_table(w.base, w.d, w.k, w.N, w.scaling)
    Wo, _ = orc.window_table(w.base, w.d, w.k, w.N, w.scaling)
    atf.atf_rope(Q, theta)
    atf.atf_rope(K, theta)
    O_all, L_all = atf.atf_prefill(Q, K, V, table=Wt)
    half = w.N // 2
    # first chunk: 64K rows over 64K keys, its own table (clipped at 64K keys)
    W1, _ = atf.atf_window_table(w.base, w.d, w.k, half, w.scaling)
    kept1 = torch.zeros(w.Hq, dtype=torch.int64, device="cuda")
    O1, L1 = atf.atf_prefill(Q[:, :, :half].contiguous(), K[:, :, :half].contiguous(), V[:, :, :half].contiguous(),
                             table=W1, kept_terms=kept1)
    # second chunk: the last 64K rows over all 128K keys
    kept2 = torch.zeros(w.Hq, dtype=torch.int64, device="cuda")
    O2, L2 = atf.atf_prefill(Q[:, :, half:].contiguous(), K, V, table=Wt, kept_terms=kept2)
    torch.cuda.synchronize()
    atf.binding.check_status()
    assert torch.equal(O1.view(torch.int16), O_all[:, :, :half].contiguous().view(torch.int16))
    assert torch.equal(O2.view(torch.int16), O_all[:, :, half:].contiguous().view(torch.int16))
    assert torch.equal(L1, L_all[:, :, :half]) and torch.equal(L2, L_all[:, :, half:])
    assert kept1.cpu().tolist() == [orc.kept_terms_interval(Wo, 0, half)] * w.Hq
    assert kept2.cpu().tolist() == [orc.kept_terms_interval(Wo, half, w.N)] * w.Hq
    assert kept1[0].item() + kept2[0].item() == orc.kept_terms_prefill(Wo, w.N)
