"""B200 (sm_100a) library for causal GQA attention with per-RoPE-wavelength distance windows.

The compute lives in libatflash.so (hand-written CUDA behind a C ABI, see include/atflash.h);
this package is the thin Python binding: it marshals torch tensors (device memory and
streams only) into the C calls of the same names.  There is no CPU fallback: without the
built library, or without a CUDA device for the device entry points, calls raise.
"""
from .binding import (  # noqa: F401
    ATF_MODE_COARSE,
    ATF_MODE_EXACT,
    AtfError,
    WindowTable,
    atf_decode,
    atf_decode_static,
    atf_kcache_pack,
    atf_prefill,
    atf_prefill_host,
    atf_rope,
    atf_window_table,
    atf_window_table_family,
    atf_workspace_bytes,
    ensure_workspace,
    lib,
    lib_path,
    llama3_scaling,
    new_kcache_groups,
    atf_prefill_split,
    atf_rope_f32,
    ATF_OP_PREFILL_SPLIT,
    atf_rope_tables,
    RopeTables,
)
