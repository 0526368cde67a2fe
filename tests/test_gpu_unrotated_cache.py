"""GPU parity of the decode on an UNROTATED group-major K cache (App. B: a position-independent cache
stores keys before RoPE and the rotation is applied when the cache is read).

The oracle side is the definition: rotate the stored keys at positions pos0 + m (fp64, one rounding to
bf16), then the per-term decode.  The GPU side packs the unrotated keys, builds the (cos, sin) tables once
and lets the decode kernel rotate the pairs it fetches.  Term counts are bit-exact; outputs meet the same
tolerances as every other decode test."""
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


def _case(atf, w: gen.Workload, mode, pos0=0, capacity=None, table=None):
    q, Ku, Vc = gen.decode_inputs(w)       # Ku: keys BEFORE RoPE; q is taken as already rotated
    L = w.N
    Wo, theta = orc.window_table(w.base, w.d, w.k, L, w.scaling)
    if table is not None:
        Wo = np.asarray(table, dtype=np.int64)
    cap = capacity or L
    Kg = atf.new_kcache_groups(w.B, w.Hkv, cap, w.d, "cuda")
    atf.atf_kcache_pack(Ku.cuda(), Kg)
    tabs = atf.atf_rope_tables(theta, w.d, cap, pos0=pos0)
    kept = torch.zeros(w.B * w.Hq, dtype=torch.int64, device="cuda")
    O, lse = atf.atf_decode(q.cuda(), Kg, Vc.cuda(), table=torch.from_numpy(Wo), mode=mode, kept_terms=kept,
                            return_lse=True, rope_tables=tabs)
    torch.cuda.synchronize()
    atf.binding.check_status()
    Kr = orc.rope_half_split(gen.to_f64(Ku), theta, pos0)
    fn = orc.decode if mode == atf.ATF_MODE_EXACT else orc.coarse_decode
    Or, Lr = fn(gen.to_f64(q), Kr, gen.to_f64(Vc), Wo)
    Og = gen.to_f64(O)
    err = np.abs(Og - Or)
    assert np.isfinite(Og).all()
    assert err.max() <= O_MAX and err.mean() <= O_MEAN, (err.max(), err.mean())
    assert np.abs(lse.double().cpu().numpy() - Lr).max() <= LSE_TOL
    want = orc.kept_terms_decode(Wo, L) if mode == atf.ATF_MODE_EXACT else orc.coarse_kept_terms_decode(Wo, L)
    assert kept.cpu().tolist() == [want] * (w.B * w.Hq)
    # against the GPU's own rotated-cache path: the same keys rotated by atf_rope and packed
    Kc = Ku.cuda().clone()
    atf.atf_rope(Kc, theta, pos0=pos0)
    Kg2 = atf.new_kcache_groups(w.B, w.Hkv, cap, w.d, "cuda")
    atf.atf_kcache_pack(Kc, Kg2)
    O2, lse2 = atf.atf_decode(q.cuda(), Kg2, Vc.cuda(), table=torch.from_numpy(Wo), mode=mode, return_lse=True)
    # the fp32 rotation at read may move a key element by one bf16 unit; the outputs stay far inside the tolerance
    assert (O.float() - O2.float()).abs().max().item() <= O_MAX / 4
    assert (lse - lse2).abs().max().item() <= LSE_TOL / 4
    return O


@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("B,Hq,Hkv,d,L,pos0", [(1, 2, 1, 64, 1, 0), (2, 6, 2, 128, 37, 11), (1, 24, 8, 128, 3000, 0),
                                               (2, 14, 2, 64, 5000, 70000), (1, 28, 4, 128, 9001, 1_000_003)])
def test_decode_unrotated_small(atf, mode, B, Hq, Hkv, d, L, pos0):
    w = gen.Workload("dec-unrot", B, Hq, Hkv, d, L, 1e4, 2.0, None, gen.SEED0 + 150 + L)
    _case(atf, w, mode, pos0=pos0)


def test_decode_unrotated_cache_with_room(atf):
    """A cache and tables laid out for more keys than the step uses (the tokens to come)."""
    w = gen.Workload("dec-unrot", 1, 8, 2, 128, 1500, 1e4, 2.0, None, gen.SEED0 + 160)
    _case(atf, w, 0, pos0=5, capacity=4096)


def test_decode_unrotated_dropped_keys(atf):
    w = gen.Workload("dec-unrot", 1, 4, 2, 64, 900, 1e4, 2.0, None, gen.SEED0 + 161)
    tab = np.minimum(np.array([3 * (r + 1) ** 2 for r in range(32)], dtype=np.int64), 400)
    _case(atf, w, 0, table=tab)
    _case(atf, w, 1, table=tab)


def test_decode_unrotated_llama_32k(atf):
    """Llama-3.2-3B decode shape at L = 32768 with the llama3-scaled frequencies."""
    w = gen.llama32_3b(32768, B=1, seed_off=17)
    _case(atf, w, 0)
    _case(atf, w, 1)


def test_rope_tables_refusals(atf):
    theta = orc.window_table(1e4, 128, 2.0, 1024)[1]
    with pytest.raises(atf.AtfError):
        atf.atf_rope_tables(theta, 96, 1024)
    with pytest.raises(atf.AtfError):
        atf.atf_rope_tables(theta[:10], 128, 1024)
    bad = np.array(theta)
    bad[3] = 0.0
    with pytest.raises(atf.AtfError):
        atf.atf_rope_tables(bad, 128, 1024)
    tabs = atf.atf_rope_tables(theta, 128, 1024)
    q = gen.normal_bf16((1, 8, 128), 1).cuda()
    K = gen.normal_bf16((1, 2, 2048, 128), 2).cuda()
    V = gen.normal_bf16((1, 2, 2048, 128), 3).cuda()
    # tables built for fewer keys than L
    with pytest.raises(atf.AtfError):
        atf.atf_decode(q, atf.atf_kcache_pack(K), V, rope_tables=tabs)
    # the row-layout cache has no rotate-at-read path
    with pytest.raises(atf.AtfError):
        atf.atf_decode(q, K, V, rope_tables=atf.atf_rope_tables(theta, 128, 2048))
