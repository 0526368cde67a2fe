// atf_prefill_split: the windowed causal prefill with scores of more than bf16 input precision
// (App. D, "Precision as the other side of the compute-accuracy trade": a low-precision product is
// split to recover accuracy, paid for with part of what the window saves; Sec. 6.2 had to score
// five tasks with fp32 attention scores because bf16 rounding flipped low-margin retrievals).
//
// Q and K arrive as fp32, already rotated and never rounded to bf16.  A pre-pass writes each as
// two bf16 tensors, hi = bf16(x) and lo = bf16(x - hi) (hi + lo holds x to 2^-17 of its size), in
// the pair-interleaved lowest-frequency-first column order of atf_prefill, so the live pairs of
// a tile are again a column prefix.  The scores are
//     S = Q_hi K_hi^T + Q_hi K_lo^T + Q_lo K_hi^T
// accumulated in fp32 in tensor memory: three tcgen05.mma per 16-column step of the LIVE depth
// only (the lo x lo product, 2^-16 of the result, is left out).  The kernel is the prefill kernel
// of atf_prefill_pipe.cu in its SPLIT form: both Q parts resident, a K stage = a hi tile and a lo
// tile, the per-cell finish of the exact mode with the same three products, every exponential
// MUFU ex2 (no polynomial), the row sums from the unrounded fp32 values.  V, P and O are bf16
// operands with fp32 accumulation as in atf_prefill; term counts are those of atf_prefill.
#include <cuda.h>

#include "atf_common.cuh"
#include "atf_prefill_pipe.cuh"

namespace {

constexpr int T = 128;

// hi = bf16(x), lo = bf16(x - hi), written in the pair-interleaved column order: column 2p holds
// dim (h-1-p), column 2p+1 holds dim (d-1-p).  One thread writes 8 consecutive output columns.
__global__ void __launch_bounds__(256)
atf_split_repack_kernel(const float* __restrict__ X, __nv_bfloat16* __restrict__ Yhi, __nv_bfloat16* __restrict__ Ylo,
                        int64_t rows, int D) {
  const int H = D / 2;
  const int per_row = D / 8;
  const int64_t gid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (gid >= rows * per_row) return;
  const int64_t row = gid / per_row;
  const int t = (int)(gid % per_row);
  const float* src = X + row * D;
  __align__(16) __nv_bfloat16 hi[8], lo[8];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int p = 4 * t + i;
    const float a = src[H - 1 - p], b = src[D - 1 - p];
    hi[2 * i] = __float2bfloat16_rn(a);
    hi[2 * i + 1] = __float2bfloat16_rn(b);
    lo[2 * i] = __float2bfloat16_rn(a - __bfloat162float(hi[2 * i]));
    lo[2 * i + 1] = __float2bfloat16_rn(b - __bfloat162float(hi[2 * i + 1]));
  }
  *reinterpret_cast<uint4*>(Yhi + row * D + 8 * t) = *reinterpret_cast<const uint4*>(hi);
  *reinterpret_cast<uint4*>(Ylo + row * D + 8 * t) = *reinterpret_cast<const uint4*>(lo);
}

size_t part_bytes(int B, int H, int64_t N, int d) {
  size_t b = (size_t)B * H * N * d * 2;
  return (b + 255) & ~(size_t)255;
}

}  // namespace

atf_status atf_validate_table(const char* who, const int64_t* table, int d, int64_t N, AtfTable* out);

// band schedule of the kernel: eight words per tile distance
static size_t split_sched_bytes(int64_t N) { return ((size_t)((N + T - 1) / T + 1) * 32 + 255) & ~(size_t)255; }

size_t atf_prefill_split_workspace_bytes(int B, int Hq, int Hkv, int64_t N, int d) {
  return ATF_WS_HEADER + split_sched_bytes(N) + 2 * part_bytes(B, Hq, N, d) + 2 * part_bytes(B, Hkv, N, d);
}

extern "C" atf_status atf_prefill_split_chunk(const float* Q, const float* K, const void* V, void* O, float* LSE, int B,
                                              int Hq, int Hkv, int64_t Nq, int64_t N, int d, const int64_t* table,
                                              int causal, const atf_opts* opts, void* stream) {
  if (!Q || !K || !V || !O) return atf_fail(ATF_ERR_INVALID_ARG, "atf_prefill_split: null pointer");
  if (d != 64 && d != 128) return atf_fail(ATF_ERR_UNSUPPORTED, "atf_prefill_split: d must be 64 or 128 (got %d)", d);
  if (B < 1 || Hq < 1 || Hkv < 1 || N < 1) return atf_fail(ATF_ERR_INVALID_ARG, "atf_prefill_split: bad shape");
  if (Nq < 1 || Nq > N) return atf_fail(ATF_ERR_INVALID_ARG, "atf_prefill_split: need 1 <= Nq <= N (got Nq = %lld, N = %lld)", (long long)Nq, (long long)N);
  if (Hq % Hkv) return atf_fail(ATF_ERR_INVALID_ARG, "atf_prefill_split: Hq must be a multiple of Hkv");
  if (!causal) return atf_fail(ATF_ERR_UNSUPPORTED, "atf_prefill_split: only causal attention is defined (distance z = n - m >= 0)");
  if (N >= (1ll << 31) - 4 * T) return atf_fail(ATF_ERR_UNSUPPORTED, "atf_prefill_split: N too large");
  if (Hq > 65535 || B > 65535) return atf_fail(ATF_ERR_UNSUPPORTED, "atf_prefill_split: B and Hq must be <= 65535");
  if (((uintptr_t)Q | (uintptr_t)K | (uintptr_t)V | (uintptr_t)O) & 15)
    return atf_fail(ATF_ERR_INVALID_ARG, "atf_prefill_split: pointers must be 16-byte aligned");
  const int mode = opts ? opts->mode : ATF_MODE_EXACT;
  if (mode != ATF_MODE_EXACT && mode != ATF_MODE_COARSE) return atf_fail(ATF_ERR_INVALID_ARG, "atf_prefill_split: unknown mode %d", mode);
  if (opts && (opts->kcache_groups || opts->rope_tables))
    return atf_fail(ATF_ERR_UNSUPPORTED, "atf_prefill_split: kcache_groups and rope_tables are not taken by this call");
  AtfTable t;
  atf_status st = atf_validate_table("atf_prefill_split", table, d, N, &t);
  if (st != ATF_OK) return st;

  AtfWorkspace ws = atf_bound_workspace();
  if (opts && opts->workspace) ws = AtfWorkspace{opts->workspace, opts->workspace_bytes};
  const size_t need = atf_prefill_split_workspace_bytes(B, Hq, Hkv, N, d);
  if (!ws.ptr) return atf_fail(ATF_ERR_WORKSPACE, "atf_prefill_split: no workspace bound");
  if (ws.bytes < need) return atf_fail(ATF_ERR_WORKSPACE, "atf_prefill_split: workspace has %zu bytes, needs %zu", ws.bytes, need);
  if ((uintptr_t)ws.ptr & 255) return atf_fail(ATF_ERR_INVALID_ARG, "atf_prefill_split: workspace must be 256-byte aligned");

  char* base = (char*)ws.ptr;
  const size_t qb = part_bytes(B, Hq, Nq, d), kb = part_bytes(B, Hkv, N, d);
  char* parts = base + ATF_WS_HEADER + split_sched_bytes(N);
  __nv_bfloat16* Qhi = (__nv_bfloat16*)parts;
  __nv_bfloat16* Qlo = (__nv_bfloat16*)(parts + qb);
  __nv_bfloat16* Khi = (__nv_bfloat16*)(parts + 2 * qb);
  __nv_bfloat16* Klo = (__nv_bfloat16*)(parts + 2 * qb + kb);
  cudaStream_t s = (cudaStream_t)stream;
  {
    const int64_t rows_q = (int64_t)B * Hq * Nq, rows_k = (int64_t)B * Hkv * N;
    const int64_t bq = (rows_q * (d / 8) + 255) / 256, bk = (rows_k * (d / 8) + 255) / 256;
    if (bq > 0x7FFFFFFF) return atf_fail(ATF_ERR_UNSUPPORTED, "atf_prefill_split: problem too large for the repack grid");
    atf_split_repack_kernel<<<(unsigned)bq, 256, 0, s>>>(Q, Qhi, Qlo, rows_q, d);
    atf_split_repack_kernel<<<(unsigned)bk, 256, 0, s>>>(K, Khi, Klo, rows_k, d);
    ATF_CUDA_CHECK(cudaGetLastError());
  }
  CUtensorMap tqh, tql, tkh, tkl, tv;
  if ((st = atf_make_tile_map(&tqh, Qhi, (int64_t)B * Hq, Nq, d, Nq, T)) != ATF_OK) return st;
  if ((st = atf_make_tile_map(&tql, Qlo, (int64_t)B * Hq, Nq, d, Nq, T)) != ATF_OK) return st;
  if ((st = atf_make_tile_map(&tkh, Khi, (int64_t)B * Hkv, N, d, N, T)) != ATF_OK) return st;
  if ((st = atf_make_tile_map(&tkl, Klo, (int64_t)B * Hkv, N, d, N, T)) != ATF_OK) return st;
  if ((st = atf_make_tile_map(&tv, V, (int64_t)B * Hkv, N, d, N, T)) != ATF_OK) return st;

  AtfPipeParams P;
  P.sched = (uint32_t*)(base + ATF_WS_HEADER);
  P.Qp = Qhi;
  P.Qp_lo = Qlo;
  P.O = (__nv_bfloat16*)O;
  P.LSE = LSE;
  P.kept = opts ? (unsigned long long*)opts->kept_terms : nullptr;
  P.status = (unsigned int*)base;
  P.Hq = Hq;
  P.Hkv = Hkv;
  P.N = (int)N;
  P.Nq = (int)Nq;
  return atf_launch_prefill_pipe_split(tqh, tql, tkh, tkl, tv, P, t, B, d, mode, P.kept != nullptr, s);
}

extern "C" atf_status atf_prefill_split(const float* Q, const float* K, const void* V, void* O, float* LSE, int B, int Hq,
                                        int Hkv, int64_t N, int d, const int64_t* table, int causal,
                                        const atf_opts* opts, void* stream) {
  return atf_prefill_split_chunk(Q, K, V, O, LSE, B, Hq, Hkv, N, N, d, table, causal, opts, stream);
}
