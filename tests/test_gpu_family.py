"""GPU parity with tables from the window family of App. A (atf_window_table_family): the
variable-k profile, a floor and a ceiling, and position-free pairs, prefill and decode against
the fp64 oracle; term counts bit-exact."""
import numpy as np
import pytest
import torch

import atf_inputs as gen
from oracle import atf_oracle as orc

pytestmark = pytest.mark.gpu

O_MAX, O_MEAN, LSE_TOL = 2e-2, 2e-3, 1e-3

CASES = [
    dict(profile="arithmetic", k_hi=16.0, k_lo=2.0),
    dict(profile="geometric", k_hi=16.0, k_lo=2.0),
    dict(k_hi=2.0, beta=64.0, cap=400.0),
    dict(k_hi=1.0, gamma=1.1, nope_fraction=0.25),
    dict(k_hi=0.0, beta=150.0),  # sliding window: keys farther than 150 are dropped
]


@pytest.fixture(scope="module")
def atf():
    import paper_2608_02947_b200 as m
    m.lib()
    return m


@pytest.mark.parametrize("d,base,Hq,Hkv", [(128, 5e5, 4, 2), (64, 1e6, 2, 1)])
def test_family_tables_prefill_and_decode(atf, d, base, Hq, Hkv):
    w = gen.Workload("family", 1, Hq, Hkv, d, 900, base, 2.0, None, gen.SEED0 + 50 + d)
    Q, K, V = gen.prefill_inputs(w)
    for kw in CASES:
        Wt, theta = atf.atf_window_table_family(w.base, w.d, w.N, None, **kw)
        Wo, theta_o = orc.window_table_family(w.base, w.d, w.N, None, **kw)
        assert np.array_equal(Wt.numpy(), Wo) and np.array_equal(theta.numpy(), theta_o)
        Qg, Kg, Vg = Q.cuda(), K.cuda(), V.cuda()
        atf.atf_rope(Qg, theta)
        atf.atf_rope(Kg, theta)
        kept = torch.zeros(Hq, dtype=torch.int64, device="cuda")
        O, L = atf.atf_prefill(Qg, Kg, Vg, table=Wt, kept_terms=kept)
        kept_d = torch.zeros(Hq, dtype=torch.int64, device="cuda")
        Od = atf.atf_decode(Qg[:, :, -1].contiguous(), Kg, Vg, table=Wt, kept_terms=kept_d)
        torch.cuda.synchronize()
        atf.binding.check_status()
        assert kept.cpu().tolist() == [orc.kept_terms_prefill(Wo, w.N)] * Hq, kw
        assert kept_d.cpu().tolist() == [orc.kept_terms_decode(Wo, w.N)] * Hq, kw
        Qr = orc.rope_half_split(gen.to_f64(Q), theta_o)
        Kr = orc.rope_half_split(gen.to_f64(K), theta_o)
        Vr = gen.to_f64(V)
        O_ref, L_ref = orc.attention_gqa(Qr, Kr, Vr, Wo)
        err = np.abs(gen.to_f64(O) - O_ref)
        assert err.max() <= O_MAX and err.mean() <= O_MEAN, (kw, err.max(), err.mean())
        assert np.abs(L.double().cpu().numpy() - L_ref).max() <= LSE_TOL, kw
        errd = np.abs(gen.to_f64(Od) - O_ref[:, :, -1])
        assert errd.max() <= O_MAX and errd.mean() <= O_MEAN, (kw, errd.max())
