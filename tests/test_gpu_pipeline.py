"""Prefill -> decode with no conversion in between (Sec. 7.2: the cache the prefill wrote is the cache the decode
reads): a prefill given atf_opts.kcache_groups writes the tiled group-major K cache itself, single shot, in
chunks and through the host-tensor path, and decode on that cache agrees with the oracle's decode."""
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


@pytest.mark.parametrize("d,B,Hq,Hkv,N,scaling", [(128, 2, 6, 2, 1000, gen.LLAMA3_SCALING), (64, 1, 14, 2, 777, None),
                                                   (128, 1, 24, 8, 4099, gen.LLAMA3_SCALING)])
def test_decode_reads_the_cache_the_prefill_wrote(atf, d, B, Hq, Hkv, N, scaling):
    base = 5e5 if d == 128 else 1e6
    w = gen.Workload("pipe", B, Hq, Hkv, d, N, base, 2.0, scaling, gen.SEED0 + 70 + d)
    Q, K, V = gen.prefill_inputs(w)
    W, theta = atf.atf_window_table(w.base, w.d, w.k, w.N, w.scaling)
    Wo, theta_o = orc.window_table(w.base, w.d, w.k, w.N, w.scaling)
    Qg, Kg, Vg = Q.cuda(), K.cuda(), V.cuda()
    atf.atf_rope(Qg, theta)
    atf.atf_rope(Kg, theta)
    cap = N + 300  # a cache with room for later tokens
    cache = atf.new_kcache_groups(B, Hkv, cap, d, "cuda")
    O, LSE = atf.atf_prefill(Qg, Kg, Vg, table=W, kcache_groups=cache)
    torch.cuda.synchronize()
    # the cache is what the separate pack pass would have written
    ref = atf.atf_kcache_pack(Kg, atf.new_kcache_groups(B, Hkv, cap, d, "cuda"))
    assert torch.equal(cache.view(torch.int16), ref.view(torch.int16))
    # chunked prefill (appended rows, growing K/V) fills the same cache piece by piece
    cache2 = atf.new_kcache_groups(B, Hkv, cap, d, "cuda")
    cuts = [0, N // 3 + 5, 2 * N // 3 + 1, N]
    for a, b_ in zip(cuts[:-1], cuts[1:]):
        atf.atf_prefill(Qg[:, :, a:b_].contiguous(), Kg[:, :, :b_].contiguous(), Vg[:, :, :b_].contiguous(), table=W,
                        kcache_groups=cache2)
    torch.cuda.synchronize()
    assert torch.equal(cache2.view(torch.int16), ref.view(torch.int16))
    # so does the host-tensor path
    cache3 = atf.new_kcache_groups(B, Hkv, cap, d, "cuda")
    atf.atf_prefill_host(Qg.cpu(), Kg.cpu(), Vg.cpu(), table=W, chunk_rows=256, kcache_groups=cache3)
    torch.cuda.synchronize()
    assert torch.equal(cache3.view(torch.int16), ref.view(torch.int16))
    # decode of the last token straight from that cache (same layout object, N keys): no pack call
    qd = Qg[:, :, -1].contiguous()
    Od, lse = atf.atf_decode(qd, cache, Vg, table=W, return_lse=True)
    torch.cuda.synchronize()
    atf.binding.check_status()
    Qr = orc.rope_half_split(gen.to_f64(Q[:, :, -1:]), theta_o, pos0=N - 1)[:, :, 0]
    Kr = orc.rope_half_split(gen.to_f64(K), theta_o)
    Or, Lr = orc.decode(Qr, Kr, gen.to_f64(V), Wo)
    err = np.abs(gen.to_f64(Od) - Or)
    assert err.max() <= O_MAX and err.mean() <= O_MEAN
    assert np.abs(lse.double().cpu().numpy() - Lr).max() <= LSE_TOL
    # and it is the prefill's own last row, within the output tolerance
    assert (Od.float() - O[:, :, -1].float()).abs().max() <= O_MAX
