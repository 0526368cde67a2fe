"""atf_decode_static: the decode entry point for callers that cannot allocate device memory.

Such callers (a plug-in running inside another runtime's callback, a host whose device
allocator is locked after start-up) get the split-K scratch from an array built into the
library.  This test calls that entry point through the C ABI, twice in a row on the same
inputs and once more on different ones (the array keeps the previous call's contents, so a
second call checks that the entry point clears what it must), and compares every result with
the ordinary atf_decode, which takes its scratch from a bound workspace.  The file is named so
that pytest collects it last."""
import ctypes as C

import pytest
import torch

import atf_inputs as gen

pytestmark = pytest.mark.gpu


def _call_static(lib, q, Kc, Vc, table):
    B, Hq, d = q.shape
    Hkv, L = Kc.shape[1], Kc.shape[2]
    O = torch.empty_like(q)
    arr = (C.c_int64 * (d // 2))(*table.tolist())
    rc = lib.atf_decode_static(C.c_void_p(q.data_ptr()), C.c_void_p(Kc.data_ptr()), C.c_void_p(Vc.data_ptr()),
                               C.c_void_p(O.data_ptr()), B, Hq, Hkv, L, d, arr,
                               C.c_void_p(torch.cuda.current_stream().cuda_stream))
    return rc, O


def test_decode_static_matches_decode_twice_in_a_row():
    import paper_2608_02947_b200 as atf
    lib = atf.lib()
    assert lib.atf_decode_static_capacity() >= 2 * 1024 * 1024
    for B, L, seed in ((1, 5000, 71), (2, 3001, 72)):
        w = gen.Workload("static", B, 24, 8, 128, L, 5e5, 2.0, gen.LLAMA3_SCALING, gen.SEED0 + seed)
        q, Kc, Vc = (t.cuda() for t in gen.decode_inputs(w))
        W, _ = atf.atf_window_table(w.base, w.d, w.k, w.N, w.scaling)
        ref = atf.atf_decode(q, Kc, Vc, table=W)
        torch.cuda.synchronize()
        for _ in range(2):  # two calls in a row share the built-in array
            rc, O = _call_static(lib, q, Kc, Vc, W)
            torch.cuda.synchronize()
            assert rc == 0, lib.atf_last_error().decode()
            err = (O.float() - ref.float()).abs()
            assert err.max().item() <= 2e-2 and err.mean().item() <= 2e-3
            assert torch.equal(O, ref)  # same kernel, same split: in fact identical


def test_decode_static_refuses_what_does_not_fit():
    import paper_2608_02947_b200 as atf
    lib = atf.lib()
    B, Hq, Hkv, d, L = 64, 32, 8, 128, 4096
    q = torch.zeros((B, Hq, d), dtype=torch.bfloat16, device="cuda")
    Kc = torch.zeros((B, Hkv, L, d), dtype=torch.bfloat16, device="cuda")
    need = atf.atf_workspace_bytes(1, B, Hq, Hkv, L, d)
    assert need > lib.atf_decode_static_capacity()
    rc, _ = _call_static(lib, q, Kc, Kc, torch.full((d // 2,), L, dtype=torch.int64))
    assert rc == 4  # ATF_ERR_WORKSPACE
    assert b"built-in array" in lib.atf_last_error()
