"""CPU-only checks of the C-ABI library: it loads without a GPU, exports every function the
header declares, its host-only entry point reproduces the oracle's tables bit for bit, and
argument validation answers with error codes before anything touches a device."""
import ctypes as C
import math
import os
import re

import numpy as np
import pytest

from atf_inputs import LLAMA3_SCALING
from oracle import atf_oracle as orc

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def atf():
    import paper_2608_02947_b200 as m
    from paper_2608_02947_b200 import build
    build.build()
    m.lib()
    return m


def test_every_declared_symbol_is_exported(atf):
    header = open(os.path.join(ROOT, "include", "atflash.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    names = set(re.findall(r"\b(atf_[a-z0-9_]+)\s*\(", header))
    assert {"atf_window_table", "atf_rope", "atf_prefill", "atf_decode", "atf_decode_static"} <= names
    lib = C.CDLL(atf.lib_path())
    for n in sorted(names):
        assert hasattr(lib, n), f"{n} is declared in atflash.h but not exported"


@pytest.mark.parametrize("base,d,k,N,sc", [(1e6, 64, 2.0, 2048, None), (1e6, 64, 2.0, 32768, None),
                                           (5e5, 128, 2.0, 8192, LLAMA3_SCALING), (5e5, 128, 2.0, 131072, LLAMA3_SCALING),
                                           (1e7, 128, 2.0, 1 << 20, None), (1e6, 64, math.inf, 2048, None),
                                           (1e4, 128, 3.5, 777, None), (5e5, 128, 64.0, 65536, LLAMA3_SCALING)])
def test_host_table_equals_oracle_table(atf, base, d, k, N, sc):
    W, th = atf.atf_window_table(base, d, k, N, sc)
    Wo, tho = orc.window_table(base, d, k, N, sc)
    assert np.array_equal(W.numpy(), Wo)
    assert np.array_equal(th.numpy(), tho)


def test_validation_returns_codes_without_a_device(atf):
    lib = atf.lib()
    w = (C.c_int64 * 32)()
    assert lib.atf_window_table(1e6, 63, 2.0, 100, None, w, None) == 1       # odd d
    assert lib.atf_window_table(1e6, 64, 2.0, 0, None, w, None) == 1        # N < 1
    assert lib.atf_window_table(1e6, 64, -1.0, 10, None, w, None) == 1      # negative k
    assert lib.atf_window_table(1e6, 64, 2.0, 10, None, None, None) == 1    # null output
    assert b"w_out" in lib.atf_last_error()
    # null tensors / unsupported shapes are refused on the host
    assert lib.atf_prefill(None, None, None, None, None, 1, 2, 1, 128, 64, None, 1, None) == 1
    fake = C.c_void_p(4096)
    assert lib.atf_prefill(fake, fake, fake, fake, None, 1, 2, 1, 128, 96, None, 1, None) == 2    # d
    assert lib.atf_prefill(fake, fake, fake, fake, None, 1, 3, 2, 128, 64, None, 1, None) == 1    # Hq % Hkv
    assert lib.atf_prefill(fake, fake, fake, fake, None, 1, 2, 1, 128, 64, None, 0, None) == 2    # non-causal
    bad = (C.c_int64 * 32)(*([5] * 16 + [4] * 16))
    assert lib.atf_prefill(fake, fake, fake, fake, None, 1, 2, 1, 128, 64, bad, 1, None) == 2     # decreasing table
    neg = (C.c_int64 * 32)(*([-1] * 32))
    assert lib.atf_decode(fake, fake, fake, fake, 1, 2, 1, 128, 64, neg, None) == 1               # negative width
    assert lib.atf_decode(fake, fake, fake, fake, 1, 18, 2, 128, 64, None, None) == 2             # Hq/Hkv > 8
    assert lib.atf_bind_workspace(C.c_void_p(4097), 1 << 20) == 1                                  # alignment
    assert lib.atf_bind_workspace(None, 0) == 0
    assert lib.atf_decode(fake, fake, fake, fake, 1, 2, 1, 128, 64, None, None) == 4              # no workspace
    assert lib.atf_workspace_bytes(0, 1, 2, 1, 128, 96) == 0
    assert lib.atf_workspace_bytes(0, 1, 24, 8, 131072, 128) > 1 << 30
    assert lib.atf_kcache_tile_keys(128) == 64 and lib.atf_kcache_tile_keys(64) == 128
