"""GPU results against closed forms that need no oracle: with Q = 0 every score is 0, so a row's
output is the plain mean of the V rows it may see and its LSE is the log of their number."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def atf():
    import paper_2608_02947_b200 as m
    m.lib()
    return m


@pytest.mark.parametrize("d,N,Wunif", [(128, 700, None), (64, 515, None), (128, 700, 200), (64, 515, 37)])
def test_zero_queries_give_prefix_means(atf, d, N, Wunif):
    g = torch.Generator().manual_seed(5)
    B, Hq, Hkv = 1, 2, 1
    Q = torch.zeros((B, Hq, N, d), dtype=torch.bfloat16, device="cuda")
    K = torch.randn((B, Hkv, N, d), generator=g).to(torch.bfloat16).cuda()
    V = torch.randn((B, Hkv, N, d), generator=g).to(torch.bfloat16).cuda()
    table = None if Wunif is None else torch.full((d // 2,), Wunif, dtype=torch.int64)
    for mode in (0, 1):
        if mode == 1 and Wunif is not None:
            continue  # the coarse mode keeps whole tiles: its key set is not the sliding window
        O, L = atf.atf_prefill(Q, K, V, table=table, mode=mode)
        Od = atf.atf_decode(Q[:, :, -1].contiguous(), K, V, table=table, mode=mode)
        torch.cuda.synchronize()
        atf.binding.check_status()
        Vf = V[0, 0].double().cpu().numpy()
        cs = np.concatenate([np.zeros((1, d)), np.cumsum(Vf, axis=0)])
        n = np.arange(N)
        lo = np.zeros(N, dtype=np.int64) if Wunif is None else np.maximum(0, n - Wunif)
        cnt = (n + 1 - lo)[:, None]
        want = (cs[n + 1] - cs[lo]) / cnt
        for hq in range(Hq):
            got = O[0, hq].double().cpu().numpy()
            # P = 1 exactly, fp32 accumulation, one bf16 rounding of O
            assert np.abs(got - want).max() <= 2.0 ** -8 * np.abs(want).max() + 1e-3, (d, N, Wunif, mode)
            assert np.abs(L[0, hq].double().cpu().numpy() - np.log(cnt[:, 0])).max() <= 1e-4
        gd = Od[0].double().cpu().numpy()
        assert np.abs(gd - want[-1][None, :]).max() <= 2.0 ** -8 * np.abs(want).max() + 1e-3
