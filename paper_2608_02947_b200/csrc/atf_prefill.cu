// atf_prefill: windowed causal attention for all query rows (Sec. 3.3, Fig. 3) on the sm_100a
// tensor cores.  This file holds the host side (validation, workspace, tensor maps, entry points)
// and the layout pre-pass; the kernel is in atf_prefill_pipe.cu.
//
// Data layout.  A pre-pass copies Q and K into a pair-interleaved column order, lowest
// frequency first: column 2p holds dim (h-1-p), column 2p+1 holds dim (d-1-p), h = d/2.  A
// query-key dot product does not change under a common column permutation, and in this order
// the pairs that are live at a distance (a contiguous low-frequency slice, Sec. 3.3) are a
// PREFIX of the columns, so "advance the start of the pair loop" becomes "contract over the
// first few 16-column MMA steps", and the K columns beyond the prefix are not loaded.  The K
// pass can also write the tiled group-major K cache that decode reads (Sec. 7.2: the cache the
// prefill wrote is the cache the decode reads).
#include <cuda.h>

#include "atf_common.cuh"
#include "atf_prefill_pipe.cuh"

namespace {

constexpr int T = 128;  // query rows per tile and key columns per tile

__global__ void __launch_bounds__(256)
atf_repack_kernel(const __nv_bfloat16* __restrict__ X, __nv_bfloat16* __restrict__ Y, int64_t rows, int D,
                  int64_t n_per_head, int64_t src_head_rows, __nv_bfloat16* __restrict__ Kg, int64_t kg_tiles,
                  int64_t kg_first_row) {
  // one thread writes 8 consecutive output columns (4 pairs) of one row; the source holds
  // src_head_rows rows per head of which the first n_per_head are copied, the result is dense.
  // With Kg the same 16 bytes also go into the tiled group-major K cache (kg_tiles tiles per head), for
  // the rows from kg_first_row on: a group of that cache is two such 16-byte pieces of a key.
  const int H = D / 2;
  const int per_row = D / 8;
  const int64_t gid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (gid >= rows * per_row) return;
  const int64_t row = gid / per_row;
  const int t = (int)(gid % per_row);
  const int64_t head = row / n_per_head;
  const int64_t m = row - head * n_per_head;  // position of the row in its head
  const __nv_bfloat16* src = X + (head * src_head_rows + m) * D;
  __align__(16) __nv_bfloat16 out[8];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int p = 4 * t + i;
    out[2 * i] = src[H - 1 - p];
    out[2 * i + 1] = src[D - 1 - p];
  }
  *reinterpret_cast<uint4*>(Y + row * D + 8 * t) = *reinterpret_cast<const uint4*>(out);
  if (Kg && m >= kg_first_row) {
    const int64_t KT = 8192 / D;  // keys per 16 KiB tile
    const int64_t tile = m / KT, kin = m % KT;
    const int j = t >> 1, half = (t & 1) ^ (int)((kin >> 2) & 1);
    *reinterpret_cast<uint4*>(Kg + (((head * kg_tiles + tile) * (D / 16) + j) * KT + kin) * 16 + half * 8) =
        *reinterpret_cast<const uint4*>(out);
  }
}

size_t repack_bytes(int B, int H, int64_t N, int d) {
  size_t b = (size_t)B * H * N * d * 2;
  return (b + 255) & ~(size_t)255;
}

}  // namespace

atf_status atf_validate_table(const char* who, const int64_t* table, int d, int64_t N, AtfTable* out);

// band schedule: one 32-byte record (eight words) per tile distance a launch over N keys can meet
static int sched_entries(int64_t N) { return (int)((N + T - 1) / T) + 1; }
static size_t sched_bytes(int64_t N) { return ((size_t)sched_entries(N) * 32 + 255) & ~(size_t)255; }

size_t atf_prefill_workspace_bytes(int B, int Hq, int Hkv, int64_t N, int d) {
  return ATF_WS_HEADER + sched_bytes(N) + repack_bytes(B, Hq, N, d) + repack_bytes(B, Hkv, N, d);
}
static size_t prefill_chunk_workspace_bytes(int B, int Hq, int Hkv, int64_t Nq, int64_t N, int d) {
  return ATF_WS_HEADER + sched_bytes(N) + repack_bytes(B, Hq, Nq, d) + repack_bytes(B, Hkv, N, d);
}

// kv_head_rows: rows between two heads of K and of V in memory (>= N; N for dense tensors).  A caller that
// fills a full-length cache chunk by chunk passes the cache's length here and the rows present as N.
atf_status atf_prefill_impl(const void* Q, const void* K, const void* V, void* O, float* LSE, int B, int Hq, int Hkv,
                            int64_t Nq, int64_t N, int d, const int64_t* table, int causal, const atf_opts* opts,
                            void* stream, int64_t kv_head_rows) {
  if (!Q || !K || !V || !O) return atf_fail(ATF_ERR_INVALID_ARG, "atf_prefill: null pointer");
  if (kv_head_rows < N) return atf_fail(ATF_ERR_INVALID_ARG, "atf_prefill: K/V head stride smaller than N");
  if (Nq < 1 || Nq > N) return atf_fail(ATF_ERR_INVALID_ARG, "atf_prefill: need 1 <= Nq <= N (got Nq = %lld, N = %lld)", (long long)Nq, (long long)N);
  if (d != 64 && d != 128) return atf_fail(ATF_ERR_UNSUPPORTED, "atf_prefill: d must be 64 or 128 (got %d)", d);
  if (B < 1 || Hq < 1 || Hkv < 1 || N < 1) return atf_fail(ATF_ERR_INVALID_ARG, "atf_prefill: bad shape");
  if (Hq % Hkv) return atf_fail(ATF_ERR_INVALID_ARG, "atf_prefill: Hq must be a multiple of Hkv");
  if (!causal) return atf_fail(ATF_ERR_UNSUPPORTED, "atf_prefill: only causal attention is defined (distance z = n - m >= 0)");
  if (N >= (1ll << 31) - 4 * T) return atf_fail(ATF_ERR_UNSUPPORTED, "atf_prefill: N too large");
  if (Hq > 65535 || B > 65535) return atf_fail(ATF_ERR_UNSUPPORTED, "atf_prefill: B and Hq must be <= 65535");
  if (((uintptr_t)Q | (uintptr_t)K | (uintptr_t)V | (uintptr_t)O) & 15)
    return atf_fail(ATF_ERR_INVALID_ARG, "atf_prefill: pointers must be 16-byte aligned");
  const int mode = opts ? opts->mode : ATF_MODE_EXACT;
  if (mode != ATF_MODE_EXACT && mode != ATF_MODE_COARSE) return atf_fail(ATF_ERR_INVALID_ARG, "atf_prefill: unknown mode %d", mode);
  if (opts && opts->kcache_groups) {
    if (opts->kcache_capacity < N) return atf_fail(ATF_ERR_INVALID_ARG, "atf_prefill: kcache_capacity (%lld) is smaller than N", (long long)opts->kcache_capacity);
    if ((uintptr_t)opts->kcache_groups & 15) return atf_fail(ATF_ERR_INVALID_ARG, "atf_prefill: kcache_groups must be 16-byte aligned");
  }
  AtfTable t;
  atf_status st = atf_validate_table("atf_prefill", table, d, N, &t);
  if (st != ATF_OK) return st;

  AtfWorkspace ws = atf_bound_workspace();
  if (opts && opts->workspace) ws = AtfWorkspace{opts->workspace, opts->workspace_bytes};
  const size_t need = prefill_chunk_workspace_bytes(B, Hq, Hkv, Nq, N, d);
  if (!ws.ptr) return atf_fail(ATF_ERR_WORKSPACE, "atf_prefill: no workspace bound");
  if (ws.bytes < need) return atf_fail(ATF_ERR_WORKSPACE, "atf_prefill: workspace has %zu bytes, needs %zu", ws.bytes, need);
  if ((uintptr_t)ws.ptr & 255) return atf_fail(ATF_ERR_INVALID_ARG, "atf_prefill: workspace must be 256-byte aligned");

  char* base = (char*)ws.ptr;
  uint32_t* sched = (uint32_t*)(base + ATF_WS_HEADER);
  __nv_bfloat16* Qp = (__nv_bfloat16*)(base + ATF_WS_HEADER + sched_bytes(N));
  __nv_bfloat16* Kp = (__nv_bfloat16*)(base + ATF_WS_HEADER + sched_bytes(N) + repack_bytes(B, Hq, Nq, d));
  cudaStream_t s = (cudaStream_t)stream;

  {
    const int64_t rows_q = (int64_t)B * Hq * Nq, rows_k = (int64_t)B * Hkv * N;
    const int64_t bq = (rows_q * (d / 8) + 255) / 256, bk = (rows_k * (d / 8) + 255) / 256;
    if (bq > 0x7FFFFFFF) return atf_fail(ATF_ERR_UNSUPPORTED, "atf_prefill: problem too large for the repack grid");
    __nv_bfloat16* Kg = opts ? (__nv_bfloat16*)opts->kcache_groups : nullptr;
    const int64_t kt = 8192 / d;
    const int64_t kg_tiles = Kg ? (opts->kcache_capacity + kt - 1) / kt : 0;
    atf_repack_kernel<<<(unsigned)bq, 256, 0, s>>>((const __nv_bfloat16*)Q, Qp, rows_q, d, Nq, Nq, nullptr, 0, 0);
    atf_repack_kernel<<<(unsigned)bk, 256, 0, s>>>((const __nv_bfloat16*)K, Kp, rows_k, d, N, kv_head_rows, Kg, kg_tiles,
                                                   N - Nq);
    ATF_CUDA_CHECK(cudaGetLastError());
  }

  CUtensorMap tq, tk, tv;
  if ((st = atf_make_tile_map(&tq, Qp, (int64_t)B * Hq, Nq, d, Nq, T)) != ATF_OK) return st;
  if ((st = atf_make_tile_map(&tk, Kp, (int64_t)B * Hkv, N, d, N, T)) != ATF_OK) return st;
  if ((st = atf_make_tile_map(&tv, V, (int64_t)B * Hkv, N, d, kv_head_rows, T)) != ATF_OK) return st;

  AtfPipeParams P;
  P.sched = sched;
  P.Qp = Qp;
  P.Qp_lo = nullptr;
  P.O = (__nv_bfloat16*)O;
  P.LSE = LSE;
  P.kept = opts ? (unsigned long long*)opts->kept_terms : nullptr;
  P.status = (unsigned int*)base;
  P.Hq = Hq;
  P.Hkv = Hkv;
  P.N = (int)N;
  P.Nq = (int)Nq;
  return atf_launch_prefill_pipe(tq, tk, tv, P, t, B, d, mode, P.kept != nullptr, s);
}

extern "C" atf_status atf_prefill_chunk_ex(const void* Q, const void* K, const void* V, void* O, float* LSE, int B,
                                           int Hq, int Hkv, int64_t Nq, int64_t N, int d, const int64_t* table,
                                           int causal, const atf_opts* opts, void* stream) {
  return atf_prefill_impl(Q, K, V, O, LSE, B, Hq, Hkv, Nq, N, d, table, causal, opts, stream, N);
}

extern "C" atf_status atf_prefill_ex(const void* Q, const void* K, const void* V, void* O, float* LSE, int B, int Hq,
                                     int Hkv, int64_t N, int d, const int64_t* table, int causal,
                                     const atf_opts* opts, void* stream) {
  return atf_prefill_chunk_ex(Q, K, V, O, LSE, B, Hq, Hkv, N, N, d, table, causal, opts, stream);
}

extern "C" atf_status atf_prefill_chunk(const void* Q, const void* K, const void* V, void* O, float* LSE, int B, int Hq,
                                        int Hkv, int64_t Nq, int64_t N, int d, const int64_t* table, int causal,
                                        void* stream) {
  return atf_prefill_chunk_ex(Q, K, V, O, LSE, B, Hq, Hkv, Nq, N, d, table, causal, nullptr, stream);
}

extern "C" atf_status atf_prefill(const void* Q, const void* K, const void* V, void* O, float* LSE, int B, int Hq,
                                  int Hkv, int64_t N, int d, const int64_t* table, int causal, void* stream) {
  return atf_prefill_ex(Q, K, V, O, LSE, B, Hq, Hkv, N, d, table, causal, nullptr, stream);
}
