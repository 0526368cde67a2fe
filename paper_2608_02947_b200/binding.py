"""ctypes binding of libatflash.so.  Argument marshalling only; every step runs in the library."""
from __future__ import annotations

import ctypes as C
import math
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
ATF_MODE_EXACT, ATF_MODE_COARSE = 0, 1
ATF_OP_PREFILL, ATF_OP_DECODE, ATF_OP_PREFILL_SPLIT = 0, 1, 2
ATF_KLAYOUT_ROWS, ATF_KLAYOUT_GROUPS = 0, 1


class AtfError(RuntimeError):
    def __init__(self, code, text):
        super().__init__(f"atflash error {code}: {text}")
        self.code = code


class _Scaling(C.Structure):
    _fields_ = [("kind", C.c_int), ("factor", C.c_double), ("low_freq_factor", C.c_double),
                ("high_freq_factor", C.c_double), ("original_ctx", C.c_int64)]


class _Opts(C.Structure):
    _fields_ = [("mode", C.c_int), ("kept_terms", C.c_void_p), ("lse", C.c_void_p),
                ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t), ("k_layout", C.c_int),
                ("kcache_groups", C.c_void_p), ("kcache_capacity", C.c_int64),
                ("rope_tables", C.c_void_p), ("rope_tables_capacity", C.c_int64)]


def lib_path():
    """Path of the shared library (ATFLASH_LIB overrides the in-tree build, e.g. to compare builds)."""
    return os.environ.get("ATFLASH_LIB") or os.path.join(_HERE, "libatflash.so")


_lib = None


def lib():
    """Loads libatflash.so (built by `python -m paper_2608_02947_b200.build`). Raises if absent."""
    global _lib
    if _lib is not None:
        return _lib
    p = lib_path()
    if not os.path.exists(p):
        raise AtfError(-1, f"{p} is missing: build it with `python -m paper_2608_02947_b200.build` "
                           "(there is no fallback implementation)")
    L = C.CDLL(p)
    vp, i, i64, dbl = C.c_void_p, C.c_int, C.c_int64, C.c_double
    L.atf_window_table.argtypes = [dbl, i, dbl, i64, C.POINTER(_Scaling), C.POINTER(C.c_int64), C.POINTER(C.c_double)]
    L.atf_window_table_family.argtypes = [dbl, i, i64, C.POINTER(_Scaling), C.POINTER(_Family), C.POINTER(C.c_int64),
                                          C.POINTER(C.c_double)]
    L.atf_rope.argtypes = [vp, i, i, i64, i, C.POINTER(C.c_double), i64, vp]
    L.atf_prefill.argtypes = [vp, vp, vp, vp, vp, i, i, i, i64, i, C.POINTER(C.c_int64), i, vp]
    L.atf_prefill_split.argtypes = [vp, vp, vp, vp, vp, i, i, i, i64, i, C.POINTER(C.c_int64), i, C.POINTER(_Opts), vp]
    L.atf_rope_f32.argtypes = [vp, i, i, i64, i, C.POINTER(C.c_double), i64, vp]
    L.atf_prefill_split_chunk.argtypes = [vp, vp, vp, vp, vp, i, i, i, i64, i64, i, C.POINTER(C.c_int64), i, C.POINTER(_Opts), vp]
    L.atf_prefill_ex.argtypes = [vp, vp, vp, vp, vp, i, i, i, i64, i, C.POINTER(C.c_int64), i, C.POINTER(_Opts), vp]
    L.atf_prefill_chunk.argtypes = [vp, vp, vp, vp, vp, i, i, i, i64, i64, i, C.POINTER(C.c_int64), i, vp]
    L.atf_prefill_chunk_ex.argtypes = [vp, vp, vp, vp, vp, i, i, i, i64, i64, i, C.POINTER(C.c_int64), i,
                                       C.POINTER(_Opts), vp]
    L.atf_prefill_host.argtypes = [vp, vp, vp, vp, vp, i, i, i, i64, i, C.POINTER(C.c_int64), i, C.POINTER(_Opts), vp,
                                   C.c_size_t, i64, vp]
    L.atf_prefill_host_scratch_bytes.argtypes = [i, i, i, i64, i, i64]
    L.atf_prefill_host_scratch_bytes.restype = C.c_size_t
    L.atf_decode.argtypes = [vp, vp, vp, vp, i, i, i, i64, i, C.POINTER(C.c_int64), vp]
    L.atf_decode_ex.argtypes = [vp, vp, vp, vp, i, i, i, i64, i, C.POINTER(C.c_int64), C.POINTER(_Opts), vp]
    L.atf_kcache_pack.argtypes = [vp, vp, i, i, i64, i64, i64, i, vp]
    L.atf_rope_tables_bytes.argtypes = [i, i64]
    L.atf_rope_tables_bytes.restype = C.c_size_t
    L.atf_rope_tables.argtypes = [C.POINTER(C.c_double), i, i64, i64, vp, C.c_size_t, vp]
    L.atf_kcache_tile_keys.argtypes = [i]
    L.atf_kcache_tile_keys.restype = C.c_int64
    L.atf_decode_static.argtypes = [vp, vp, vp, vp, i, i, i, i64, i, C.POINTER(C.c_int64), vp]
    L.atf_decode_static.restype = C.c_int
    L.atf_decode_static_capacity.restype = C.c_size_t
    L.atf_workspace_bytes.argtypes = [i, i, i, i, i64, i]
    L.atf_workspace_bytes.restype = C.c_size_t
    L.atf_bind_workspace.argtypes = [vp, C.c_size_t]
    L.atf_check_status.argtypes = [vp]
    L.atf_check_status_at.argtypes = [vp, vp]
    L.atf_selftest_bounded_wait.argtypes = [C.c_uint, vp]
    L.atf_probe_masked_read.argtypes = [vp, C.c_size_t, C.c_uint, vp]
    L.atf_last_error.restype = C.c_char_p
    for name in ("atf_window_table", "atf_window_table_family", "atf_rope", "atf_prefill", "atf_prefill_ex", "atf_prefill_chunk",
                 "atf_prefill_chunk_ex", "atf_prefill_host", "atf_decode", "atf_decode_ex",
                 "atf_kcache_pack", "atf_rope_tables", "atf_prefill_split", "atf_prefill_split_chunk", "atf_rope_f32",
                 "atf_bind_workspace", "atf_check_status", "atf_check_status_at", "atf_selftest_bounded_wait", "atf_probe_masked_read"):
        getattr(L, name).restype = C.c_int
    _lib = L
    return L


def _check(code):
    if code != 0:
        raise AtfError(code, lib().atf_last_error().decode())


def llama3_scaling(factor=32.0, low_freq_factor=1.0, high_freq_factor=4.0, original_ctx=8192):
    return {"kind": "llama3", "factor": factor, "low_freq_factor": low_freq_factor,
            "high_freq_factor": high_freq_factor, "original_ctx": original_ctx}


def _scaling_ref(scaling):
    if scaling is None or scaling.get("kind", "none") == "none":
        return None
    kind = {"llama3": 1}.get(scaling["kind"], 99)
    return C.byref(_Scaling(kind, float(scaling["factor"]), float(scaling["low_freq_factor"]),
                            float(scaling["high_freq_factor"]), int(scaling["original_ctx"])))


def atf_window_table(base, d, k, N, scaling=None):
    """Returns (W int64[d/2] tensor on the host, theta float64[d/2] tensor on the host)."""
    h = max(d // 2, 1)
    w = (C.c_int64 * h)()
    th = (C.c_double * h)()
    _check(lib().atf_window_table(float(base), int(d), float(k), int(N), _scaling_ref(scaling), w, th))
    return torch.tensor(list(w), dtype=torch.int64), torch.tensor(list(th), dtype=torch.float64)


class _Family(C.Structure):
    _fields_ = [("profile", C.c_int), ("k_hi", C.c_double), ("k_lo", C.c_double), ("gamma", C.c_double),
                ("beta", C.c_double), ("cap", C.c_double), ("a", C.c_double), ("nope_fraction", C.c_double)]


_PROFILES = {"constant": 0, "arithmetic": 1, "geometric": 2}


def atf_window_table_family(base, d, N, scaling=None, profile="constant", k_hi=2.0, k_lo=None, gamma=1.0, beta=0.0,
                            cap=None, a=0.0, nope_fraction=0.0):
    """The window family of App. A; same return as atf_window_table."""
    h = max(d // 2, 1)
    w = (C.c_int64 * h)()
    th = (C.c_double * h)()
    fam = _Family(_PROFILES.get(profile, 99), float(k_hi), float(k_hi if k_lo is None else k_lo), float(gamma),
                  float(beta), 0.0 if cap is None else float(cap), float(a), float(nope_fraction))
    _check(lib().atf_window_table_family(float(base), int(d), int(N), _scaling_ref(scaling), C.byref(fam), w, th))
    return torch.tensor(list(w), dtype=torch.int64), torch.tensor(list(th), dtype=torch.float64)


def _stream(t):
    return C.c_void_p(torch.cuda.current_stream(t.device).cuda_stream)


def _one_device(*tensors):
    """All device tensors of a call must live on one GPU: the C side launches on the current device, and the
    binding makes that the tensors' device for the duration of the call."""
    devs = {t.device for t in tensors if t is not None}
    if len(devs) != 1:
        raise AtfError(1, f"all tensors of a call must be on the same CUDA device (got {sorted(map(str, devs))})")
    return torch.cuda.device(devs.pop())


def _dev_bf16(t, name):
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous()):
        raise AtfError(1, f"{name} must be a contiguous CUDA bf16 tensor")
    return C.c_void_p(t.data_ptr())


class WindowTable:
    """A window table marshalled once (host int64 array) so that repeated calls pay nothing for it."""

    def __init__(self, table):
        t = torch.as_tensor(table, dtype=torch.int64).cpu().contiguous()
        self.n = t.numel()
        self.arr = (C.c_int64 * self.n)(*t.tolist())


def _table_ptr(table, d):
    if table is None:
        return None, None
    wt = table if isinstance(table, WindowTable) else WindowTable(table)
    if wt.n != d // 2:
        raise AtfError(1, f"table must have d/2 = {d // 2} entries")
    return wt.arr, wt


_ws = None


def atf_workspace_bytes(op, B, Hq, Hkv, N, d):
    return int(lib().atf_workspace_bytes(op, B, Hq, Hkv, N, d))


def ensure_workspace(nbytes, device):
    """Keeps one zero-initialised device buffer bound as the library's workspace (grown on demand)."""
    global _ws
    if _ws is None or _ws.numel() < nbytes or _ws.device != torch.device(device):
        _ws = None
        _ws = torch.zeros(max(nbytes, 256), dtype=torch.uint8, device=device)
        _check(lib().atf_bind_workspace(C.c_void_p(_ws.data_ptr()), _ws.numel()))
    return _ws


def atf_rope(X, theta, pos0=0):
    """In-place half-split RoPE of X [B,H,N,d] (CUDA bf16) at positions pos0..pos0+N-1."""
    _dev_bf16(X, "X")
    B, H, N, d = X.shape
    th = torch.as_tensor(theta, dtype=torch.float64).cpu()
    arr = (C.c_double * th.numel())(*th.tolist())
    with torch.cuda.device(X.device):
        _check(lib().atf_rope(C.c_void_p(X.data_ptr()), B, H, N, d, arr, int(pos0), _stream(X)))
    return X


def _opts(mode, kept_terms, lse, k_layout=ATF_KLAYOUT_ROWS, kcache_groups=None):
    if mode == ATF_MODE_EXACT and kept_terms is None and lse is None and k_layout == ATF_KLAYOUT_ROWS and kcache_groups is None:
        return None
    o = _Opts()
    if kcache_groups is not None:
        o.kcache_groups = kcache_groups.data_ptr()
        o.kcache_capacity = kcache_groups.shape[2] * kcache_groups.shape[4]
    o.mode = int(mode)
    o.k_layout = int(k_layout)
    o.kept_terms = kept_terms.data_ptr() if kept_terms is not None else None
    o.lse = lse.data_ptr() if lse is not None else None
    o.workspace = None
    o.workspace_bytes = 0
    return o


def _to_pinned_host(t, dst=None):
    """Device -> host copy into `dst` (a host tensor of the same shape and dtype, ideally pinned and
    reused by the caller: pinning a fresh buffer costs more than the copy) or into a new pinned
    tensor (a pageable destination would halve the PCIe rate)."""
    if dst is None:
        dst = torch.empty(t.shape, dtype=t.dtype, pin_memory=True)
    elif dst.shape != t.shape or dst.dtype != t.dtype or dst.is_cuda:
        raise AtfError(1, "host output tensor has the wrong shape, dtype or device")
    dst.copy_(t, non_blocking=True)
    torch.cuda.current_stream(t.device).synchronize()
    return dst


def _host_roundtrip(tensors):
    """For host inputs: pinned staging + device copies (the end-to-end path of the binding)."""
    return [t.pin_memory().to("cuda", non_blocking=True) if not t.is_cuda else t for t in tensors]


def new_kcache_groups(B, Hkv, capacity, d, device):
    """A zeroed tiled group-major K cache for `capacity` keys per (batch, KV head): [B,Hkv,tiles,d/16,KT,16]."""
    kt = int(lib().atf_kcache_tile_keys(d))
    return torch.zeros((B, Hkv, (capacity + kt - 1) // kt, d // 16, kt, 16), dtype=torch.bfloat16, device=device)


def _check_kcache_groups(Kg, B, Hkv, N, d):
    kt = int(lib().atf_kcache_tile_keys(d))
    _dev_bf16(Kg, "kcache_groups")
    if Kg.dim() != 6 or Kg.shape[:2] != (B, Hkv) or Kg.shape[3:] != (d // 16, kt, 16) or Kg.shape[2] * kt < N:
        raise AtfError(1, f"kcache_groups must be [B,Hkv,tiles,d/16,{kt},16] with room for N keys")


def atf_prefill(Q, K, V, table=None, causal=True, mode=ATF_MODE_EXACT, kept_terms=None, return_lse=True,
                O=None, LSE=None, kcache_groups=None):
    """Windowed causal attention.  Q [B,Hq,Nq,d], K/V [B,Hkv,N,d] bf16, already rotated.

    Nq == N is the whole prefill (atf_prefill_ex); Nq < N are appended rows: Q holds the last Nq
    positions of the N-key context (atf_prefill_chunk_ex).
    Device tensors are used in place; host tensors are copied to the current CUDA device and
    the results copied back (host in -> host out; O / LSE, if given, are then host tensors that
    receive the results).  Returns (O, LSE) (LSE None if not asked).
    """
    on_host = not Q.is_cuda
    O_host = LSE_host = None
    if on_host and Q.shape[2] == K.shape[2]:
        return atf_prefill_host(Q, K, V, table=table, causal=causal, mode=mode, kept_terms=kept_terms,
                                return_lse=return_lse, O=O, LSE=LSE, kcache_groups=kcache_groups)
    if on_host:
        Q, K, V = _host_roundtrip([Q, K, V])
        O_host, LSE_host, O, LSE = O, LSE, None, None
    for t, nm in ((Q, "Q"), (K, "K"), (V, "V")):
        _dev_bf16(t, nm)
    B, Hq, Nq, d = Q.shape
    Hkv, N = K.shape[1], K.shape[2]
    if K.shape != (B, Hkv, N, d) or V.shape != K.shape:
        raise AtfError(1, "K and V must be [B,Hkv,N,d] matching Q")
    if O is None:
        O = torch.empty_like(Q)
    if LSE is None and return_lse:
        LSE = torch.empty((B, Hq, Nq), dtype=torch.float32, device=Q.device)
    if kcache_groups is not None:
        _check_kcache_groups(kcache_groups, B, Hkv, N, d)
    dev = _one_device(Q, K, V, O, LSE, kept_terms, kcache_groups)
    ensure_workspace(atf_workspace_bytes(ATF_OP_PREFILL, B, Hq, Hkv, N, d), Q.device)
    tab, _keep = _table_ptr(table, d)
    o = _opts(mode, kept_terms, None, kcache_groups=kcache_groups)
    lse_ptr = C.c_void_p(LSE.data_ptr()) if LSE is not None else None
    with dev:
        if Nq == N:
            _check(lib().atf_prefill_ex(C.c_void_p(Q.data_ptr()), C.c_void_p(K.data_ptr()), C.c_void_p(V.data_ptr()),
                                        C.c_void_p(O.data_ptr()), lse_ptr, B, Hq, Hkv, N, d, tab, 1 if causal else 0,
                                        C.byref(o) if o is not None else None, _stream(Q)))
        else:
            _check(lib().atf_prefill_chunk_ex(C.c_void_p(Q.data_ptr()), C.c_void_p(K.data_ptr()),
                                              C.c_void_p(V.data_ptr()), C.c_void_p(O.data_ptr()), lse_ptr, B, Hq, Hkv,
                                              Nq, N, d, tab, 1 if causal else 0,
                                              C.byref(o) if o is not None else None, _stream(Q)))
    if on_host:
        return _to_pinned_host(O, O_host), (_to_pinned_host(LSE, LSE_host) if LSE is not None else None)
    return O, LSE


def _dev_f32(t, name):
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == torch.float32 and t.is_contiguous()):
        raise AtfError(1, f"{name} must be a contiguous CUDA fp32 tensor")


def atf_rope_f32(X, theta, pos0=0):
    """In-place half-split RoPE of X [B,H,N,d] (CUDA fp32) at positions pos0..pos0+N-1, kept in fp32."""
    _dev_f32(X, "X")
    B, H, N, d = X.shape
    th = torch.as_tensor(theta, dtype=torch.float64).cpu()
    arr = (C.c_double * th.numel())(*th.tolist())
    with torch.cuda.device(X.device):
        _check(lib().atf_rope_f32(C.c_void_p(X.data_ptr()), B, H, N, d, arr, int(pos0), _stream(X)))
    return X


def atf_prefill_split(Q, K, V, table=None, causal=True, mode=ATF_MODE_EXACT, kept_terms=None, return_lse=True,
                      O=None, LSE=None):
    """atf_prefill with split-precision scores: Q [B,Hq,N,d] and K [B,Hkv,N,d] are CUDA fp32 (rotated, never
    rounded to bf16), V is bf16; each score is three bf16 tensor-core products (hi*hi + hi*lo + lo*hi).
    Q may hold only the last Nq rows of the N-key context (appended rows).  Returns (O bf16, LSE fp32 or None)."""
    _dev_f32(Q, "Q")
    _dev_f32(K, "K")
    _dev_bf16(V, "V")
    B, Hq, Nq, d = Q.shape
    Hkv, N = K.shape[1], K.shape[2]
    if K.shape != (B, Hkv, N, d) or V.shape != K.shape:
        raise AtfError(1, "K and V must be [B,Hkv,N,d] matching Q")
    if O is None:
        O = torch.empty(Q.shape, dtype=torch.bfloat16, device=Q.device)
    _dev_bf16(O, "O")
    if LSE is None and return_lse:
        LSE = torch.empty((B, Hq, Nq), dtype=torch.float32, device=Q.device)
    dev = _one_device(Q, K, V, O, LSE, kept_terms)
    ensure_workspace(atf_workspace_bytes(ATF_OP_PREFILL_SPLIT, B, Hq, Hkv, N, d), Q.device)
    tab, _keep = _table_ptr(table, d)
    o = _opts(mode, kept_terms, None)
    with dev:
        _check(lib().atf_prefill_split_chunk(C.c_void_p(Q.data_ptr()), C.c_void_p(K.data_ptr()), C.c_void_p(V.data_ptr()),
                                             C.c_void_p(O.data_ptr()), C.c_void_p(LSE.data_ptr()) if LSE is not None else None,
                                             B, Hq, Hkv, Nq, N, d, tab, 1 if causal else 0,
                                       C.byref(o) if o is not None else None, _stream(Q)))
    return O, LSE


def atf_prefill_host(Q, K, V, table=None, causal=True, mode=ATF_MODE_EXACT, kept_terms=None, return_lse=True,
                     O=None, LSE=None, chunk_rows=0, device=None, kcache_groups=None):
    """atf_prefill for HOST tensors (Q [B,Hq,N,d], K/V [B,Hkv,N,d] bf16, rotated): the C call copies,
    computes and copies back chunk by chunk on three streams.  Pinned tensors overlap; O / LSE, if
    given, are host tensors that receive the results (reuse pinned ones across calls).
    Returns (O, LSE) on the host, complete."""
    for t, nm in ((Q, "Q"), (K, "K"), (V, "V")):
        if t.is_cuda or t.dtype != torch.bfloat16 or not t.is_contiguous():
            raise AtfError(1, f"{nm} must be a contiguous host bf16 tensor")
    B, Hq, N, d = Q.shape
    Hkv = K.shape[1]
    if K.shape != (B, Hkv, N, d) or V.shape != K.shape:
        raise AtfError(1, "K and V must be [B,Hkv,N,d] matching Q")
    device = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
    if O is None:
        O = torch.empty(Q.shape, dtype=torch.bfloat16, pin_memory=True)
    if LSE is None and return_lse:
        LSE = torch.empty((B, Hq, N), dtype=torch.float32, pin_memory=True)
    for t, shp, dt in ((O, Q.shape, torch.bfloat16), (LSE, (B, Hq, N), torch.float32)):
        if t is not None and (t.is_cuda or tuple(t.shape) != tuple(shp) or t.dtype != dt or not t.is_contiguous()):
            raise AtfError(1, "host output tensor has the wrong shape, dtype or device")
    need = int(lib().atf_prefill_host_scratch_bytes(B, Hq, Hkv, N, d, int(chunk_rows)))
    if need == 0:
        raise AtfError(1, "unsupported shape")
    ws = ensure_workspace(need, device)  # the scratch starts with the workspace header the status check reads
    tab, _keep = _table_ptr(table, d)
    if kcache_groups is not None:
        _check_kcache_groups(kcache_groups, B, Hkv, N, d)
    o = _opts(mode, kept_terms, None, kcache_groups=kcache_groups)
    with torch.cuda.device(device):
        stream = torch.cuda.current_stream(device)
        _check(lib().atf_prefill_host(C.c_void_p(Q.data_ptr()), C.c_void_p(K.data_ptr()), C.c_void_p(V.data_ptr()),
                                      C.c_void_p(O.data_ptr()), C.c_void_p(LSE.data_ptr()) if LSE is not None else None,
                                      B, Hq, Hkv, N, d, tab, 1 if causal else 0,
                                      C.byref(o) if o is not None else None, C.c_void_p(ws.data_ptr()), ws.numel(),
                                      int(chunk_rows), C.c_void_p(stream.cuda_stream)))
        stream.synchronize()
    return O, LSE


def atf_kcache_pack(K, Kg=None, pos0=0):
    """Copies rotated key rows K [B,Hkv,n,d] into a tiled group-major cache
    Kg [B,Hkv,tiles,d/16,KT,16] at positions pos0.. (allocates a zeroed cache for exactly pos0+n keys
    if Kg is None). Returns Kg."""
    _dev_bf16(K, "K")
    B, Hkv, n, d = K.shape
    kt = int(lib().atf_kcache_tile_keys(d))
    if Kg is None:
        Kg = torch.zeros((B, Hkv, (pos0 + n + kt - 1) // kt, d // 16, kt, 16), dtype=torch.bfloat16, device=K.device)
    _dev_bf16(Kg, "Kg")
    if Kg.dim() != 6 or Kg.shape[:2] != (B, Hkv) or Kg.shape[3:] != (d // 16, kt, 16):
        raise AtfError(1, f"Kg must be [B,Hkv,tiles,d/16,{kt},16]")
    with _one_device(K, Kg):
        _check(lib().atf_kcache_pack(C.c_void_p(K.data_ptr()), C.c_void_p(Kg.data_ptr()), B, Hkv, n, Kg.shape[2] * kt,
                                     int(pos0), d, _stream(K)))
    return Kg


class RopeTables:
    """The device tables of atf_rope_tables with the shape they were built for."""

    def __init__(self, buf, d, pos0, capacity):
        self.buf, self.d, self.pos0, self.capacity = buf, d, pos0, capacity


def atf_rope_tables(theta, d, capacity, pos0=0, device="cuda"):
    """Rotation tables for decode on an unrotated group-major K cache of up to `capacity` keys whose
    key 0 sits at position pos0 (pass the result to atf_decode as rope_tables)."""
    device = torch.device(device)
    nbytes = lib().atf_rope_tables_bytes(int(d), int(capacity))
    if nbytes == 0:
        raise AtfError(1, f"atf_rope_tables: unsupported shape d={d}, capacity={capacity}")
    th = torch.as_tensor(theta, dtype=torch.float64).cpu()
    if th.numel() != d // 2:
        raise AtfError(1, "theta must have d/2 entries")
    arr = (C.c_double * th.numel())(*th.tolist())
    with torch.cuda.device(device):
        buf = torch.empty(nbytes, dtype=torch.uint8, device=device)
        _check(lib().atf_rope_tables(arr, int(d), int(pos0), int(capacity), C.c_void_p(buf.data_ptr()), nbytes,
                                     C.c_void_p(torch.cuda.current_stream(device).cuda_stream)))
    return RopeTables(buf, int(d), int(pos0), int(capacity))


def atf_decode(q, Kcache, Vcache, table=None, mode=ATF_MODE_EXACT, kept_terms=None, return_lse=False, O=None,
               rope_tables=None):
    """One decode step: q [B,Hq,d] at position L-1 against Kcache/Vcache [B,Hkv,L,d] (bf16).
    Kcache may also be a tiled group-major cache [B,Hkv,tiles,d/16,KT,16] from atf_kcache_pack; with
    rope_tables (atf_rope_tables) that cache holds unrotated keys and the kernel rotates what it fetches."""
    on_host = not q.is_cuda
    if on_host:
        q, Kcache, Vcache = _host_roundtrip([q, Kcache, Vcache])
    for t, nm in ((q, "q"), (Kcache, "Kcache"), (Vcache, "Vcache")):
        _dev_bf16(t, nm)
    B, Hq, d = q.shape
    Hkv, L = Vcache.shape[1], Vcache.shape[2]
    k_layout = ATF_KLAYOUT_GROUPS if Kcache.dim() == 6 else ATF_KLAYOUT_ROWS
    if k_layout == ATF_KLAYOUT_GROUPS:
        _check_kcache_groups(Kcache, B, Hkv, L, d)  # may be laid out for more keys than it holds yet
    elif tuple(Kcache.shape) != (B, Hkv, L, d):
        raise AtfError(1, "Kcache must be [B,Hkv,L,d] or a group-major cache [B,Hkv,tiles,d/16,KT,16], matching q")
    if Vcache.shape != (B, Hkv, L, d):
        raise AtfError(1, "Vcache must be [B,Hkv,L,d], matching q")
    if O is None:
        O = torch.empty_like(q)
    lse = torch.empty((B, Hq), dtype=torch.float32, device=q.device) if return_lse else None
    dev = _one_device(q, Kcache, Vcache, O, kept_terms, rope_tables.buf if rope_tables is not None else None)
    ensure_workspace(atf_workspace_bytes(ATF_OP_DECODE, B, Hq, Hkv, L, d), q.device)
    tab, _keep = _table_ptr(table, d)
    o = _opts(mode, kept_terms, lse, k_layout, kcache_groups=Kcache if k_layout == ATF_KLAYOUT_GROUPS else None)
    if rope_tables is not None:
        if on_host:
            raise AtfError(1, "rope_tables need device tensors")
        if k_layout != ATF_KLAYOUT_GROUPS:
            raise AtfError(2, "rope_tables need a group-major K cache")
        if rope_tables.d != d:
            raise AtfError(1, "rope_tables were built for another head dimension")
        o.rope_tables = rope_tables.buf.data_ptr()
        o.rope_tables_capacity = rope_tables.capacity
    with dev:
        _check(lib().atf_decode_ex(C.c_void_p(q.data_ptr()), C.c_void_p(Kcache.data_ptr()), C.c_void_p(Vcache.data_ptr()),
                                   C.c_void_p(O.data_ptr()), B, Hq, Hkv, L, d, tab,
                                   C.byref(o) if o is not None else None, _stream(q)))
    if on_host:
        return (_to_pinned_host(O), _to_pinned_host(lse)) if return_lse else _to_pinned_host(O)
    return (O, lse) if return_lse else O


def atf_decode_static(q, Kcache, Vcache, table=None, O=None):
    """atf_decode for callers that may not allocate: the library's built-in scratch array is used
    instead of a workspace (exact mode, row-layout cache; problems beyond its capacity raise).
    Only argument marshalling happens here; pass O to avoid the one output allocation."""
    for t, nm in ((q, "q"), (Kcache, "Kcache"), (Vcache, "Vcache")):
        _dev_bf16(t, nm)
    if q.dim() != 3 or Kcache.dim() != 4:
        raise AtfError(1, "q must be [B,Hq,d] and Kcache [B,Hkv,L,d]")
    B, Hq, d = q.shape
    Hkv, L = Kcache.shape[1], Kcache.shape[2]
    if tuple(Kcache.shape) != (B, Hkv, L, d) or Vcache.shape != Kcache.shape:
        raise AtfError(1, "Kcache and Vcache must both be [B,Hkv,L,d], matching q [B,Hq,d]")
    if O is None:
        O = torch.empty_like(q)
    if O.shape != q.shape:
        raise AtfError(1, "O must have the shape of q")
    _dev_bf16(O, "O")
    tab, _keep = _table_ptr(table, d)
    with _one_device(q, Kcache, Vcache, O):
        _check(lib().atf_decode_static(C.c_void_p(q.data_ptr()), C.c_void_p(Kcache.data_ptr()),
                                       C.c_void_p(Vcache.data_ptr()), C.c_void_p(O.data_ptr()), B, Hq, Hkv, L, d, tab,
                                       _stream(q)))
    return O


def check_status(workspace=None):
    """Raises AtfError(ATF_ERR_TIMEOUT) if a kernel gave up a bounded wait since the last check: in the bound
    workspace (and the built-in array of atf_decode_static), or in the given workspace tensor."""
    if workspace is None:
        _check(lib().atf_check_status(C.c_void_p(torch.cuda.current_stream().cuda_stream)))
    else:
        with torch.cuda.device(workspace.device):
            _check(lib().atf_check_status_at(C.c_void_p(workspace.data_ptr()),
                                             C.c_void_p(torch.cuda.current_stream(workspace.device).cuda_stream)))


def selftest_bounded_wait(limit_us=1000):
    """Launches the library's wait-that-runs-out self-test on the current device (needs a bound workspace)."""
    _check(lib().atf_selftest_bounded_wait(int(limit_us), C.c_void_p(torch.cuda.current_stream().cuda_stream)))


def probe_masked_read(buf, chunkmask):
    """Launches the row-read diagnostic on a CUDA byte buffer (see atf_probe_masked_read in the header)."""
    with torch.cuda.device(buf.device):
        _check(lib().atf_probe_masked_read(C.c_void_p(buf.data_ptr()), buf.numel() * buf.element_size(), int(chunkmask),
                                           C.c_void_p(torch.cuda.current_stream(buf.device).cuda_stream)))
