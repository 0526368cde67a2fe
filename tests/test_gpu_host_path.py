"""atf_prefill_host (host tensors in, host tensors out, chunked and overlapped inside the C call)
against atf_prefill on device tensors: bit-identical for every chunk size, counts included."""
import numpy as np
import pytest
import torch

import atf_inputs as gen
from oracle import atf_oracle as orc

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def atf():
    import paper_2608_02947_b200 as m
    m.lib()
    return m


@pytest.mark.parametrize("d,B,Hq,Hkv,N", [(128, 2, 4, 2, 3000), (64, 1, 2, 1, 1111)])
def test_host_path_is_the_device_path(atf, d, B, Hq, Hkv, N):
    w = gen.Workload("host", B, Hq, Hkv, d, N, 5e5 if d == 128 else 1e6, 2.0, None, gen.SEED0 + 60 + d)
    Q, K, V = gen.prefill_inputs(w)
    Wt, theta = atf.atf_window_table(w.base, w.d, w.k, w.N, w.scaling)
    Qg, Kg, Vg = Q.cuda(), K.cuda(), V.cuda()
    atf.atf_rope(Qg, theta)
    atf.atf_rope(Kg, theta)
    kept_dev = torch.zeros(B * Hq, dtype=torch.int64, device="cuda")
    O_dev, L_dev = atf.atf_prefill(Qg, Kg, Vg, table=Wt, kept_terms=kept_dev)
    torch.cuda.synchronize()
    Qh, Kh, Vh = Qg.cpu().pin_memory(), Kg.cpu().pin_memory(), Vg.cpu().pin_memory()
    for chunk in (0, 256, 700, 1024, 5000):
        for pinned in (True, False):
            kept = torch.zeros(B * Hq, dtype=torch.int64, device="cuda")
            src = (Qh, Kh, Vh) if pinned else (Qg.cpu(), Kg.cpu(), Vg.cpu())
            O, L = atf.atf_prefill_host(*src, table=Wt, kept_terms=kept, chunk_rows=chunk)
            atf.binding.check_status()
            assert not O.is_cuda and not L.is_cuda
            assert torch.equal(O.view(torch.int16), O_dev.cpu().view(torch.int16)), (chunk, pinned)
            assert torch.equal(L, L_dev.cpu()), (chunk, pinned)
            assert torch.equal(kept, kept_dev), (chunk, pinned)
    Wo, _ = orc.window_table(w.base, w.d, w.k, w.N, w.scaling)
    assert kept_dev.cpu().tolist() == [orc.kept_terms_prefill(Wo, N)] * (B * Hq)
    # the generic entry point takes the same route for host tensors, results into caller-owned buffers
    Oh = torch.empty(Q.shape, dtype=torch.bfloat16, pin_memory=True)
    O2, L2 = atf.atf_prefill(Qh, Kh, Vh, table=Wt, O=Oh, return_lse=False)
    assert O2 is Oh and L2 is None
    assert torch.equal(O2.view(torch.int16), O_dev.cpu().view(torch.int16))


def test_host_path_rejects_device_tensors_and_small_scratch(atf):
    x = torch.zeros((1, 2, 64, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(atf.AtfError):
        atf.atf_prefill_host(x, x, x)
    import ctypes as C
    lib = atf.lib()
    fake = C.c_void_p(4096)
    assert lib.atf_prefill_host_scratch_bytes(1, 2, 2, 1024, 128, 0) > 0
    assert lib.atf_prefill_host(fake, fake, fake, fake, None, 1, 2, 2, 1024, 128, None, 1, None, fake, 1024, 0, None) == 4
    assert lib.atf_prefill_host(fake, fake, fake, fake, None, 1, 2, 2, 1024, 128, None, 1, None, None, 0, 0, None) == 4


def test_host_path_32k_llama_shape(atf):
    """The benchmark's end-to-end route at a full-size shape: default chunking, pinned tensors."""
    w = gen.llama32_3b(32768, seed_off=5)
    Q, K, V = gen.prefill_inputs(w, device="cuda")
    Wt, theta = atf.atf_window_table(w.base, w.d, w.k, w.N, w.scaling)
    atf.atf_rope(Q, theta)
    atf.atf_rope(K, theta)
    O_dev, L_dev = atf.atf_prefill(Q, K, V, table=Wt)
    torch.cuda.synchronize()
    Qh, Kh, Vh = (t.cpu().pin_memory() for t in (Q, K, V))
    Oh = torch.empty(Q.shape, dtype=torch.bfloat16, pin_memory=True)
    Lh = torch.empty(Q.shape[:3], dtype=torch.float32, pin_memory=True)
    for _ in range(2):  # the second call reuses scratch, streams and result buffers
        Oh.zero_()
        O, L = atf.atf_prefill(Qh, Kh, Vh, table=Wt, O=Oh, LSE=Lh)
        atf.binding.check_status()
        assert O is Oh and L is Lh
        assert torch.equal(O.view(torch.int16), O_dev.cpu().view(torch.int16))
        assert torch.equal(L, L_dev.cpu())
