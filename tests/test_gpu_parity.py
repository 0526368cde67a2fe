"""GPU parity: the CUDA library (through its C ABI binding) against the fp64 CPU oracle, element
by element on the same seeded inputs.  Tolerances are the ones the task fixes for bf16 inputs
with fp32 accumulation: O max-abs 2e-2 and mean-abs 2e-3, LSE 1e-3; tables and term counts
are bit-exact."""
import math

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


def _bf16_ulp_diff(a: torch.Tensor, b_f64: np.ndarray):
    ai = a.cpu().view(torch.int16).numpy().astype(np.int32)
    bi = torch.from_numpy(b_f64).to(torch.bfloat16).view(torch.int16).numpy().astype(np.int32)
    # sign-magnitude -> monotone integer
    ai = np.where(ai < 0, -(ai & 0x7FFF), ai)
    bi = np.where(bi < 0, -(bi & 0x7FFF), bi)
    return np.abs(ai - bi)


def _check_out(O_gpu, LSE_gpu, O_ref, LSE_ref, tag=""):
    Og = gen.to_f64(O_gpu)
    err = np.abs(Og - O_ref)
    assert np.isfinite(Og).all(), tag
    assert err.max() <= O_MAX, (tag, err.max())
    assert err.mean() <= O_MEAN, (tag, err.mean())
    if LSE_gpu is not None:
        le = np.abs(LSE_gpu.double().cpu().numpy() - LSE_ref)
        assert le.max() <= LSE_TOL, (tag, le.max())


@pytest.mark.parametrize("d,base,N,pos0,scaling", [(64, 1e6, 300, 0, None), (128, 5e5, 257, 1_000_000, gen.LLAMA3_SCALING),
                                                    (128, 1e7, 130, (1 << 20) - 130, None)])
def test_rope_matches_oracle(atf, d, base, N, pos0, scaling):
    _, theta = atf.atf_window_table(base, d, 2.0, 4096, scaling)
    _, theta_o = orc.window_table(base, d, 2.0, 4096, scaling)
    x = gen.normal_bf16((2, 3, N, d), 77)
    y = atf.atf_rope(x.cuda().clone(), theta, pos0)
    ref = orc.rope_half_split(gen.to_f64(x), theta_o, pos0)
    ulp = _bf16_ulp_diff(y, ref)
    assert ulp.max() <= 1
    assert (ulp > 0).mean() < 1e-3  # fp64 evaluation: essentially every element is the correctly rounded one
    yf = gen.to_f64(y)
    h = d // 2
    xf = gen.to_f64(x)
    assert np.allclose(yf[..., :h] ** 2 + yf[..., h:] ** 2, xf[..., :h] ** 2 + xf[..., h:] ** 2, rtol=2e-2, atol=1e-3)


def _prefill_case(atf, w: gen.Workload, table, mode, rows=None, count=True):
    Q, K, V = gen.prefill_inputs(w)
    Wt, theta = atf.atf_window_table(w.base, w.d, w.k, w.N, w.scaling)
    Wo, theta_o = orc.window_table(w.base, w.d, w.k, w.N, w.scaling)
    assert np.array_equal(Wt.numpy(), Wo)
    if table is not None:
        Wo = np.asarray(table, dtype=np.int64)
    Qg, Kg, Vg = Q.cuda(), K.cuda(), V.cuda()
    atf.atf_rope(Qg, theta)
    atf.atf_rope(Kg, theta)
    kept = torch.zeros(w.B * w.Hq, dtype=torch.int64, device="cuda") if count else None
    O, LSE = atf.atf_prefill(Qg, Kg, Vg, table=torch.from_numpy(Wo), mode=mode, kept_terms=kept)
    torch.cuda.synchronize()
    atf.binding.check_status()
    Qr = orc.rope_half_split(gen.to_f64(Q), theta_o)
    Kr = orc.rope_half_split(gen.to_f64(K), theta_o)
    Vr = gen.to_f64(V)
    rows = list(range(w.N)) if rows is None else rows
    g = w.Hq // w.Hkv
    for b in range(w.B):
        for hq in range(w.Hq):
            if mode == atf.ATF_MODE_EXACT:
                Or, Lr = orc.attention_rows(Qr[b, hq], Kr[b, hq // g], Vr[b, hq // g], Wo, rows)
            else:
                Or, Lr = orc.coarse_attention_rows(Qr[b, hq], Kr[b, hq // g], Vr[b, hq // g], Wo, rows)
            _check_out(O[b, hq][rows], LSE[b, hq][rows], Or, Lr, tag=f"b{b} h{hq}")
    if count:
        want = orc.kept_terms_prefill(Wo, w.N) if mode == atf.ATF_MODE_EXACT else orc.coarse_kept_terms_prefill(Wo, w.N)
        assert kept.cpu().tolist() == [want] * (w.B * w.Hq)
    return O, LSE


@pytest.mark.parametrize("N", [1, 100, 128, 129, 600])
@pytest.mark.parametrize("d", [64, 128])
def test_prefill_small_exact(atf, N, d):
    w = gen.Workload("small", 1, 2, 1, d, N, 1e4 if d == 64 else 5e5, 2.0, None, gen.SEED0 + 20 + N)
    _prefill_case(atf, w, None, atf.ATF_MODE_EXACT)


@pytest.mark.parametrize("d", [64, 128])
def test_prefill_small_coarse(atf, d):
    w = gen.Workload("small", 2, 4, 2, d, 700, 1e4, 2.0, None, gen.SEED0 + 31)
    _prefill_case(atf, w, None, atf.ATF_MODE_COARSE)


def test_prefill_dropped_keys_and_uniform_table(atf):
    # hand-made tables: keys beyond the widest window are dropped; uniform table = sliding window
    w = gen.Workload("small", 1, 2, 2, 64, 520, 1e4, 2.0, None, gen.SEED0 + 40)
    tab = np.minimum(np.array([3 * (r + 1) ** 2 for r in range(32)], dtype=np.int64), 300)
    _prefill_case(atf, w, tab, atf.ATF_MODE_EXACT)
    _prefill_case(atf, w, np.full(32, 100, dtype=np.int64), atf.ATF_MODE_EXACT)
    _prefill_case(atf, w, tab, atf.ATF_MODE_COARSE)


def test_prefill_tiny_config(atf):
    """The tiny prefill workload: B=1, Hq=2, Hkv=1, d=64, base 1e6, N=2048, k=2, and k=inf = full attention."""
    w = gen.tiny()
    O2, L2 = _prefill_case(atf, w, None, atf.ATF_MODE_EXACT)
    winf = gen.tiny(k=math.inf)
    Oi, Li = _prefill_case(atf, winf, None, atf.ATF_MODE_EXACT, rows=list(range(0, 2048, 7)))
    # table = NULL is bit-identical to k = inf
    Q, K, V = gen.prefill_inputs(winf)
    _, theta = atf.atf_window_table(winf.base, winf.d, winf.k, winf.N)
    Qg, Kg, Vg = Q.cuda(), K.cuda(), V.cuda()
    atf.atf_rope(Qg, theta); atf.atf_rope(Kg, theta)
    On, Ln = atf.atf_prefill(Qg, Kg, Vg, table=None)
    assert torch.equal(On, Oi) and torch.equal(Ln, Li)
    # and it is textbook causal attention (library routine, fp32)
    ref = torch.nn.functional.scaled_dot_product_attention(Qg.float(), Kg.float().repeat_interleave(2, 1),
                                                           Vg.float().repeat_interleave(2, 1), is_causal=True)
    assert (On.float() - ref).abs().max() <= O_MAX


@pytest.mark.parametrize("d", [64, 128])
def test_prefill_outlier_logits_take_the_safe_pass(atf, d):
    """Four pairs scaled by 8 give logits in the hundreds.  The fast path takes every exponential against the
    row's reference maximum from the diagonal tile; here later keys exceed it by far more than 2^64 for most rows,
    so a tile's fast pass ends with infinite partial sums and the CTA must run the tile again with the exchanged,
    running maximum.  Results and term counts must be the definition's all the same (a fast path that went
    unnoticed would return NaN or infinity)."""
    w = gen.Workload("outlier", 1, 2, 1, d, 900, 1e4, 2.0, None, gen.SEED0 + 300 + d, True)
    O, LSE = _prefill_case(atf, w, None, atf.ATF_MODE_EXACT)
    assert torch.isfinite(LSE).all() and float(LSE.abs().max()) > 60      # the logits really are that large
    _prefill_case(atf, w, None, atf.ATF_MODE_COARSE)


def _decode_case(atf, w: gen.Workload, mode, table=None):
    q, Kc, Vc = gen.decode_inputs(w)
    Wt, _ = atf.atf_window_table(w.base, w.d, w.k, w.N, w.scaling)
    Wo = np.asarray(table, dtype=np.int64) if table is not None else orc.window_table(w.base, w.d, w.k, w.N, w.scaling)[0]
    if table is None:
        assert np.array_equal(Wt.numpy(), Wo)
    kept = torch.zeros(w.B * w.Hq, dtype=torch.int64, device="cuda")
    O, lse = atf.atf_decode(q.cuda(), Kc.cuda(), Vc.cuda(), table=torch.from_numpy(Wo), mode=mode, kept_terms=kept,
                            return_lse=True)
    torch.cuda.synchronize()
    fn = orc.decode if mode == atf.ATF_MODE_EXACT else orc.coarse_decode
    Or, Lr = fn(gen.to_f64(q), gen.to_f64(Kc), gen.to_f64(Vc), Wo)
    _check_out(O, lse, Or, Lr)
    want = orc.kept_terms_decode(Wo, w.N) if mode == atf.ATF_MODE_EXACT else orc.coarse_kept_terms_decode(Wo, w.N)
    assert kept.cpu().tolist() == [want] * (w.B * w.Hq)
    # second call on the same workspace (split counters must have been reset)
    O2 = atf.atf_decode(q.cuda(), Kc.cuda(), Vc.cuda(), table=torch.from_numpy(Wo), mode=mode)
    assert torch.equal(O2, O)
    # the same step from a group-major K cache: same terms, so the same counts and the same answer
    Kg = atf.atf_kcache_pack(Kc.cuda())
    kept.zero_()
    O3, lse3 = atf.atf_decode(q.cuda(), Kg, Vc.cuda(), table=torch.from_numpy(Wo), mode=mode, kept_terms=kept,
                              return_lse=True)
    torch.cuda.synchronize()
    _check_out(O3, lse3, Or, Lr, tag="group-major")
    assert kept.cpu().tolist() == [want] * (w.B * w.Hq)


def test_kcache_pack_layout(atf):
    """Tile T, group j of the packed cache hold pairs r = h-1-8j-i (i = 0..7) of keys T*KT.. as (dim r, dim r+h);
    keys whose index in the tile has bit 2 set store the two 16-byte halves of that entry swapped."""
    B, Hkv, n, d = 2, 3, 150, 128
    h, kt = d // 2, 64
    K = gen.normal_bf16((B, Hkv, n, d), 123).cuda()
    Kg = torch.zeros((B, Hkv, 3, d // 16, kt, 16), dtype=torch.bfloat16, device="cuda")
    atf.atf_kcache_pack(K, Kg, pos0=5)
    ref = torch.zeros_like(Kg)
    for m in range(n):
        pos = 5 + m
        for j in range(d // 16):
            for i in range(8):
                r = h - 1 - (8 * j + i)
                e = 2 * i if not ((pos % kt) >> 2) & 1 else (2 * i + 8) % 16
                ref[:, :, pos // kt, j, pos % kt, e] = K[:, :, m, r]
                ref[:, :, pos // kt, j, pos % kt, e + 1] = K[:, :, m, r + h]
    assert torch.equal(Kg, ref)


@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("B,Hq,Hkv,d,L", [(1, 2, 1, 64, 1), (2, 6, 2, 128, 37), (1, 24, 8, 128, 3000),
                                          (2, 14, 2, 64, 5000), (1, 28, 4, 128, 9001), (8, 24, 8, 128, 2048)])
def test_decode_small(atf, mode, B, Hq, Hkv, d, L):
    base = 1e4
    w = gen.Workload("dec", B, Hq, Hkv, d, L, base, 2.0, None, gen.SEED0 + 50 + L)
    _decode_case(atf, w, mode)


def test_decode_dropped_keys(atf):
    w = gen.Workload("dec", 1, 4, 2, 64, 900, 1e4, 2.0, None, gen.SEED0 + 60)
    tab = np.minimum(np.array([3 * (r + 1) ** 2 for r in range(32)], dtype=np.int64), 400)
    _decode_case(atf, w, 0, tab)
    _decode_case(atf, w, 1, tab)


def test_decode_llama_32k(atf):
    """The Llama-3.2-3B decode workload at B=1, L=32768 (llama3-scaled table)."""
    w = gen.llama32_3b(32768, B=1, seed_off=7)
    _decode_case(atf, w, 0)
    _decode_case(atf, w, 1)
