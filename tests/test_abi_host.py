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


def test_degenerate_scaling_is_refused_by_both_sides(atf):
    """A llama3 scaling whose blend is undefined (equal factors, non-positive factor or context) would give an
    infinite or NaN frequency: the C side answers ATF_ERR_INVALID_ARG, the oracle raises."""
    for bad in (dict(high_freq_factor=1.0), dict(factor=0.0), dict(factor=-2.0), dict(original_ctx=0),
                dict(low_freq_factor=0.0), dict(low_freq_factor=5.0), dict(factor=math.inf)):
        sc = dict(LLAMA3_SCALING, **bad)
        with pytest.raises(atf.AtfError) as e:
            atf.atf_window_table(5e5, 128, 2.0, 8192, sc)
        assert e.value.code == 1
        with pytest.raises(ValueError):
            orc.window_table(5e5, 128, 2.0, 8192, sc)
        with pytest.raises(atf.AtfError):
            atf.atf_window_table_family(5e5, 128, 8192, sc)


def test_static_decode_and_status_refusals_without_a_device(atf):
    lib = atf.lib()
    fake = C.c_void_p(4096)
    # shapes are checked before anything touches a device
    assert lib.atf_decode_static(fake, fake, fake, fake, 0, 24, 8, 1024, 128, None, None) == 1
    assert lib.atf_decode_static(fake, fake, fake, fake, 1, 24, 7, 1024, 128, None, None) == 1
    assert lib.atf_decode_static(fake, fake, fake, fake, 1, 24, 8, 1024, 96, None, None) == 1
    # a problem beyond the built-in array is refused with both sizes in the text
    assert lib.atf_decode_static(fake, fake, fake, fake, 64, 24, 8, 131072, 128, None, None) == 4
    msg = lib.atf_last_error().decode()
    assert str(lib.atf_decode_static_capacity()) in msg and "atf_decode" in msg
    assert lib.atf_check_status_at(None, None) == 1
    assert lib.atf_selftest_bounded_wait(0, None) in (1, 4)   # no workspace bound, or a limit out of range
    # the binding refuses tensors that are not CUDA bf16, and a cache that does not match q, before the C call
    import torch
    q = torch.zeros((1, 24, 128), dtype=torch.bfloat16)
    kc = torch.zeros((1, 8, 64, 128), dtype=torch.bfloat16)
    with pytest.raises(atf.AtfError):
        atf.atf_decode_static(q, kc, kc)


FAMILY_CASES = [
    dict(),  # Eq. 3 with k = 2
    dict(k_hi=64.0),
    dict(profile="arithmetic", k_hi=16.0, k_lo=2.0),
    dict(profile="geometric", k_hi=16.0, k_lo=2.0),
    dict(k_hi=2.0, gamma=0.5),
    dict(k_hi=2.0, gamma=1.25, cap=3000.0),
    dict(k_hi=2.0, beta=64.0, cap=0.25 * 8192),
    dict(k_hi=0.0, beta=500.0),                # sliding window
    dict(k_hi=0.0, a=1000.0),                  # linear window
    dict(k_hi=1.0, a=300.0, nope_fraction=0.25),
    dict(profile="arithmetic", k_hi=3.0, k_lo=8.0, a=-20.0, beta=5.0),
]


@pytest.mark.parametrize("base,d,N,sc", [(1e6, 64, 8192, None), (5e5, 128, 131072, LLAMA3_SCALING), (1e7, 128, 169000, None)])
def test_host_family_table_equals_oracle(atf, base, d, N, sc):
    for kw in FAMILY_CASES:
        W, th = atf.atf_window_table_family(base, d, N, sc, **kw)
        Wo, tho = orc.window_table_family(base, d, N, sc, **kw)
        assert np.array_equal(W.numpy(), Wo), kw
        assert np.array_equal(th.numpy(), tho), kw
    W, th = atf.atf_window_table_family(base, d, N, sc, k_hi=2.0)
    W2, th2 = atf.atf_window_table(base, d, 2.0, N, sc)
    assert np.array_equal(W.numpy(), W2.numpy()) and np.array_equal(th.numpy(), th2.numpy())


def test_family_validation_and_non_monotone_tables(atf):
    lib = atf.lib()
    for bad in (dict(profile="nope"), dict(k_hi=-1.0), dict(profile="geometric", k_hi=2.0, k_lo=0.0),
                dict(beta=-1.0), dict(nope_fraction=1.5), dict(gamma=float("nan"))):
        with pytest.raises(atf.AtfError):
            atf.atf_window_table_family(1e6, 64, 4096, None, **bad)
    assert lib.atf_window_table_family(1e6, 64, 4096, None, None, (C.c_int64 * 32)(), None) == 1
    # a profile that rises faster than the wavelengths fall gives a table that is not monotone:
    # the generator returns it, the attention entry points refuse it
    W, _ = atf.atf_window_table_family(1e6, 64, 1 << 20, None, profile="geometric", k_hi=1e6, k_lo=1e-3)
    assert np.any(np.diff(W.numpy()) < 0)
    fake = C.c_void_p(4096)
    tab = (C.c_int64 * 32)(*W.tolist())
    assert lib.atf_prefill(fake, fake, fake, fake, None, 1, 2, 1, 1 << 20, 64, tab, 1, None) == 2


def test_rope_tables_validation_without_a_device(atf):
    lib = atf.lib()
    th = (C.c_double * 64)(*([0.5] * 64))
    fake = C.c_void_p(4096)
    assert lib.atf_rope_tables_bytes(128, 131072) == (64 + 2048) * 64 * 8    # one row per key of a tile + one per tile
    assert lib.atf_rope_tables_bytes(64, 1) == (128 + 1) * 32 * 8
    assert lib.atf_rope_tables_bytes(96, 1024) == 0
    assert lib.atf_rope_tables(None, 128, 0, 1024, fake, 1 << 20, None) == 1          # null theta
    assert lib.atf_rope_tables(th, 96, 0, 1024, fake, 1 << 20, None) == 2             # d
    assert lib.atf_rope_tables(th, 128, -1, 1024, fake, 1 << 20, None) == 1           # negative position
    assert lib.atf_rope_tables(th, 128, 0, 1024, C.c_void_p(4100), 1 << 20, None) == 1  # misaligned
    assert lib.atf_rope_tables(th, 128, 0, 1024, fake, 1024, None) == 4               # buffer too small
    assert b"needs" in lib.atf_last_error()
    th[7] = 0.0
    assert lib.atf_rope_tables(th, 128, 0, 1024, fake, 1 << 20, None) == 1            # theta must be positive
