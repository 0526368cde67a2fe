"""GPU parity at the full sizes of the benchmark workloads, in the launch configuration bench.py
times: inputs are generated on the device from the seeded generators, the CUDA path runs the whole
problem, and the oracle recomputes sampled outputs one by one (first and last tile, rows next to
every window boundary, seeded random rows) on a few heads; term counts are compared for every head."""
import numpy as np
import pytest
import torch

import atf_inputs as gen
from oracle import atf_oracle as orc

pytestmark = pytest.mark.gpu
O_MAX, O_MEAN, LSE_TOL = 2e-2, 2e-3, 1e-3
# With i.i.d. inputs a late row's output is small (an average over many keys), so the absolute
# tolerances alone say little there: each sampled row must also agree with the oracle to a few percent
# of that row's own magnitude (bf16 rounding of P and of O gives a few tenths of a percent).
ROW_REL = 0.05


def _check_rows(O_gpu_rows, O_ref, tag):
    err = np.abs(O_gpu_rows - O_ref)
    assert np.isfinite(O_gpu_rows).all(), tag
    assert err.max() <= O_MAX and err.mean() <= O_MEAN, (tag, err.max(), err.mean())
    rel = np.sqrt((err ** 2).sum(axis=-1)) / np.maximum(np.sqrt((O_ref ** 2).sum(axis=-1)), 1e-30)
    assert rel.max() <= ROW_REL, (tag, float(rel.max()), int(rel.argmax()))


@pytest.fixture(scope="module")
def atf():
    import paper_2608_02947_b200 as m
    m.lib()
    return m


def _oracle_rows(Qh, Kh, Vh, theta_o, Wo, rows, mode, atf):
    """Qh/Kh/Vh: un-rotated bf16 tensors of one head on the device; oracle RoPE, then the sampled rows."""
    Kr = orc.rope_half_split(gen.to_f64(Kh), theta_o)
    Vr = gen.to_f64(Vh)
    N, d = Kr.shape
    Qr = np.zeros((N, d))
    qsel = gen.to_f64(Qh[rows])
    for i, n in enumerate(rows):
        Qr[n] = orc.rope_half_split(qsel[i:i + 1], theta_o, pos0=n)[0]
    fn = orc.attention_rows if mode == 0 else orc.coarse_attention_rows
    return fn(Qr, Kr, Vr, Wo, rows)


def _prefill_fullsize(atf, w, heads, n_random, mode=0, tile_rows=True):
    Q, K, V = gen.prefill_inputs(w, device="cuda")
    W, theta = atf.atf_window_table(w.base, w.d, w.k, w.N, w.scaling)
    Wo, theta_o = orc.window_table(w.base, w.d, w.k, w.N, w.scaling)
    assert np.array_equal(W.numpy(), Wo)
    Qg, Kg = Q.clone(), K.clone()
    atf.atf_rope(Qg, theta)
    atf.atf_rope(Kg, theta)
    kept = torch.zeros(w.B * w.Hq, dtype=torch.int64, device="cuda")
    O, LSE = atf.atf_prefill(Qg, Kg, V, table=W, mode=mode, kept_terms=kept)
    torch.cuda.synchronize()
    atf.binding.check_status()
    want = orc.kept_terms_prefill(Wo, w.N) if mode == 0 else orc.coarse_kept_terms_prefill(Wo, w.N)
    assert kept.cpu().tolist() == [want] * (w.B * w.Hq)
    rows = gen.sample_rows(w.N, Wo, n_random, w.seed, tile=128 if tile_rows else 4)
    g = w.Hq // w.Hkv
    for hq in heads:
        Or, Lr = _oracle_rows(Q[0, hq], K[0, hq // g], V[0, hq // g], theta_o, Wo, rows, mode, atf)
        _check_rows(gen.to_f64(O[0, hq][rows]), Or, hq)
        assert np.abs(LSE[0, hq][rows].double().cpu().numpy() - Lr).max() <= LSE_TOL


@pytest.mark.parametrize("outlier", [False, True])
def test_qwen05b_8192(atf, outlier):
    _prefill_fullsize(atf, gen.qwen05b(8192, outlier=outlier), heads=[0, 13], n_random=128)


def test_qwen05b_32768_coarse_and_exact(atf):
    _prefill_fullsize(atf, gen.qwen05b(32768), heads=[6], n_random=32, tile_rows=False)
    _prefill_fullsize(atf, gen.qwen05b(32768), heads=[7], n_random=32, mode=1, tile_rows=False)


def test_llama_8192(atf):
    _prefill_fullsize(atf, gen.llama32_3b(8192, seed_off=4), heads=[0, 11, 23], n_random=128)


def test_llama_32768(atf):
    _prefill_fullsize(atf, gen.llama32_3b(32768, seed_off=5), heads=[5], n_random=48, tile_rows=False)


def test_llama_32768_outlier_channels(atf):
    """Peaked scores (|s| up to ~100, outputs of order 1): a mishandled cell shows at full size, and rows whose
    later scores overshoot the reference maximum of their first tile by far exercise the redo path."""
    _prefill_fullsize(atf, gen.llama32_3b(32768, seed_off=13, outlier=True), heads=[2, 20], n_random=48, tile_rows=False)


def test_llama_131072(atf):
    """The benchmark's own configuration."""
    _prefill_fullsize(atf, gen.llama32_3b(131072, seed_off=6), heads=[17], n_random=24, tile_rows=False)


@pytest.mark.parametrize("B,L", [(8, 32768), (1, 131072), (8, 131072)])
def test_llama_decode_fullsize(atf, B, L):
    w = gen.llama32_3b(L, B=B, seed_off=7 + (B > 1) + 2 * (L > 32768))
    q, Kc, Vc = gen.decode_inputs(w, device="cuda")
    W, _ = atf.atf_window_table(w.base, w.d, w.k, w.N, w.scaling)
    Wo = orc.window_table(w.base, w.d, w.k, w.N, w.scaling)[0]
    kept = torch.zeros(w.B * w.Hq, dtype=torch.int64, device="cuda")
    O, lse = atf.atf_decode(q, Kc, Vc, table=W, kept_terms=kept, return_lse=True)
    Kg = atf.atf_kcache_pack(Kc)
    Og, lseg = atf.atf_decode(q, Kg, Vc, table=W, return_lse=True)
    torch.cuda.synchronize()
    assert kept.cpu().tolist() == [orc.kept_terms_decode(Wo, L)] * (w.B * w.Hq)
    g = w.Hq // w.Hkv
    for b, hq in ((0, 0), (B - 1, 23), (B // 2, 10)):
        Or, Lr = orc.decode(gen.to_f64(q[b:b + 1, hq:hq + 1]), gen.to_f64(Kc[b:b + 1, hq // g:hq // g + 1]),
                            gen.to_f64(Vc[b:b + 1, hq // g:hq // g + 1]), Wo)
        for Ox, lx in ((O, lse), (Og, lseg)):
            err = np.abs(gen.to_f64(Ox[b, hq]) - Or[0, 0])
            assert err.max() <= O_MAX and err.mean() <= O_MEAN
            assert abs(float(lx[b, hq]) - Lr[0, 0]) <= LSE_TOL


def test_qwen7b_1m_decode(atf):
    w = gen.qwen7b_1m(1 << 20)
    q, Kc, Vc = gen.decode_inputs(w, device="cuda")
    W, _ = atf.atf_window_table(w.base, w.d, w.k, w.N, w.scaling)
    Wo = orc.window_table(w.base, w.d, w.k, w.N, w.scaling)[0]
    kept = torch.zeros(w.Hq, dtype=torch.int64, device="cuda")
    O, lse = atf.atf_decode(q, Kc, Vc, table=W, kept_terms=kept, return_lse=True)
    torch.cuda.synchronize()
    assert kept.cpu().tolist() == [orc.kept_terms_decode(Wo, w.N)] * w.Hq == [23588285] * w.Hq
    for hq in (0, 27):
        Or, Lr = orc.decode(gen.to_f64(q[:, hq:hq + 1]), gen.to_f64(Kc[:, hq // 7:hq // 7 + 1]),
                            gen.to_f64(Vc[:, hq // 7:hq // 7 + 1]), Wo)
        err = np.abs(gen.to_f64(O[0, hq]) - Or[0, 0])
        assert err.max() <= O_MAX and err.mean() <= O_MEAN
        assert abs(float(lse[0, hq]) - Lr[0, 0]) <= LSE_TOL


def test_qwen7b_1m_prefill_counts_and_rows(atf):
    """Single-layer causal prefill at N = 2^20: every head's term count, and a handful of rows of one head."""
    w = gen.qwen7b_1m(1 << 20)
    Q, K, V = gen.prefill_inputs(w, device="cuda")
    W, theta = atf.atf_window_table(w.base, w.d, w.k, w.N, w.scaling)
    Wo, theta_o = orc.window_table(w.base, w.d, w.k, w.N, w.scaling)
    hq = 9
    rows = [0, 127, 128, 65535, 65536, 524287, 816037, 816038, (1 << 20) - 129, (1 << 20) - 1]
    q_keep = Q[0, hq][rows].clone()      # un-rotated copies for the oracle, before the in-place RoPE
    k_keep = K[0, hq // 7].clone()
    atf.atf_rope(Q, theta)
    atf.atf_rope(K, theta)
    kept = torch.zeros(w.Hq, dtype=torch.int64, device="cuda")
    O, LSE = atf.atf_prefill(Q, K, V, table=W, kept_terms=kept)
    torch.cuda.synchronize()
    atf.binding.check_status()
    assert kept.cpu().tolist() == [13447325211374] * w.Hq
    Kr = orc.rope_half_split(gen.to_f64(k_keep), theta_o)
    Vr = gen.to_f64(V[0, hq // 7])
    qsel = gen.to_f64(q_keep)
    for i, n in enumerate(rows):
        qn = orc.rope_half_split(qsel[i:i + 1], theta_o, pos0=n)[0]
        s = orc.windowed_scores_row(qn, Kr, Wo, n)
        o, l = orc._softmax_row(s, Vr[: n + 1])
        _check_rows(gen.to_f64(O[0, hq, n])[None, :], o[None, :], n)
        assert abs(float(LSE[0, hq, n]) - l) <= LSE_TOL


@pytest.mark.parametrize("B,L", [(1, 131072), (8, 32768)])
def test_llama_decode_unrotated_cache_fullsize(atf, B, L):
    """The benchmark's decode shapes on an unrotated group-major cache (rotation at read, App. B): the oracle
    rotates the stored keys itself and decodes; three (batch, head) samples and every head's term count."""
    w = gen.llama32_3b(L, B=B, seed_off=27 + (B > 1))
    q, Ku, Vc = gen.decode_inputs(w, device="cuda")     # Ku: keys before RoPE
    W, theta = atf.atf_window_table(w.base, w.d, w.k, w.N, w.scaling)
    Wo, theta_o = orc.window_table(w.base, w.d, w.k, w.N, w.scaling)
    Kg = atf.atf_kcache_pack(Ku)
    tabs = atf.atf_rope_tables(theta, w.d, L)
    kept = torch.zeros(w.B * w.Hq, dtype=torch.int64, device="cuda")
    O, lse = atf.atf_decode(q, Kg, Vc, table=W, kept_terms=kept, return_lse=True, rope_tables=tabs)
    torch.cuda.synchronize()
    atf.binding.check_status()
    assert kept.cpu().tolist() == [orc.kept_terms_decode(Wo, L)] * (w.B * w.Hq)
    g = w.Hq // w.Hkv
    for b, hq in ((0, 0), (B - 1, 23), (B // 2, 10)):
        Kr = orc.rope_half_split(gen.to_f64(Ku[b:b + 1, hq // g:hq // g + 1]), theta_o)
        Or, Lr = orc.decode(gen.to_f64(q[b:b + 1, hq:hq + 1]), Kr, gen.to_f64(Vc[b:b + 1, hq // g:hq // g + 1]), Wo)
        err = np.abs(gen.to_f64(O[b, hq]) - Or[0, 0])
        assert err.max() <= O_MAX and err.mean() <= O_MEAN
        assert abs(float(lse[b, hq]) - Lr[0, 0]) <= LSE_TOL


def test_llama_32768_split_precision(atf):
    """Split-precision prefill at the 32K Llama shape (whole problem on the GPU), sampled rows of two heads
    against the definition on the fp32 values, every head's term count."""
    w = gen.llama32_3b(32768, seed_off=31)
    Q, K, V = gen.prefill_inputs_f32(w, device="cuda")
    W, theta = atf.atf_window_table(w.base, w.d, w.k, w.N, w.scaling)
    Wo, theta_o = orc.window_table(w.base, w.d, w.k, w.N, w.scaling)
    Qg, Kg = Q.clone(), K.clone()
    atf.atf_rope_f32(Qg, theta)
    atf.atf_rope_f32(Kg, theta)
    kept = torch.zeros(w.B * w.Hq, dtype=torch.int64, device="cuda")
    O, LSE = atf.atf_prefill_split(Qg, Kg, V, table=W, kept_terms=kept)
    torch.cuda.synchronize()
    atf.binding.check_status()
    assert kept.cpu().tolist() == [orc.kept_terms_prefill(Wo, w.N)] * (w.B * w.Hq)
    rows = gen.sample_rows(w.N, Wo, 24, 91, tile=32)
    g = w.Hq // w.Hkv
    for hq in (5, 22):
        Kr = orc.rope_half_split(K[0, hq // g].cpu().numpy().astype(np.float64), theta_o, 0, round_bf16=False)
        Kr = Kr.astype(np.float32).astype(np.float64)
        Qr = np.zeros_like(Kr)
        qsel = Q[0, hq][rows].cpu().numpy().astype(np.float64)
        for i, n in enumerate(rows):
            Qr[n] = orc.rope_half_split(qsel[i:i + 1], theta_o, pos0=n, round_bf16=False)[0].astype(np.float32)
        Or, Lr = orc.attention_rows(Qr, Kr, gen.to_f64(V[0, hq // g]), Wo, rows)
        _check_rows(gen.to_f64(O[0, hq])[rows], Or, f"split head {hq}")
        le = np.abs(LSE[0, hq].double().cpu().numpy()[rows] - Lr)
        smax = max(np.abs(s[np.isfinite(s)]).max() for s in (orc.windowed_scores_row(Qr[n], Kr, Wo, n) for n in rows[::16]))
        assert le.max() <= 1.5e-5 * max(1.0, smax), (hq, le.max(), smax)
