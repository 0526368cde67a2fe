// atf_prefill: windowed causal attention for all query rows (Sec. 3.3, Fig. 3) on the
// sm_100a tensor cores.
//
// Data layout.  A pre-pass copies Q and K into a pair-interleaved column order, lowest
// frequency first: column 2p holds dim (h-1-p), column 2p+1 holds dim (d-1-p), h = d/2.  A
// query-key dot product does not change under a common column permutation, and in this order
// the pairs that are live at a distance (a contiguous low-frequency slice, Sec. 3.3) are a
// PREFIX of the columns, so "advance the start of the pair loop" becomes "contract over the
// first few 16-column MMA steps", and the K columns beyond the prefix are not loaded.
//
// Kernel.  One CTA owns a 128-row query tile of one head and walks the key tiles from the
// diagonal outwards.  Per key tile: TMA brings K (the live 64-column blocks) and V into
// 128-byte-swizzled shared memory; tcgen05.mma accumulates S = Q K^T over the live depth into
// tensor memory; the four warps read S (one row per thread), finish the window rule, apply
// the causal mask and the online softmax, rescale O in tensor memory, write P as bf16 to
// shared memory; tcgen05.mma accumulates O += P V.
//
// Exact mode (the per-term definition).  For a tile at tile distance D the cells span
// distances [z_min, z_max].  Pairs with w >= z_max are live in every cell: they are the MMA
// depth.  Pairs with w < z_min are dead in every cell.  Pairs in between ("straddling") are
// added per cell on the CUDA cores, only where z <= w.  Because an MMA step covers 8 pairs, the
// pairs of the last step that are not live in every cell are zeroed in the CTA's own copy of
// the Q tile; pairs only die as the distance grows, so the zeroing is monotone.
// Coarse mode: depth = pairs live in any cell of the tile, rounded up to 8; diagonal tile full.
#include <cuda.h>

#include "atf_common.cuh"

namespace {

constexpr int T = 128;           // query rows and key columns per tile
constexpr int BLK_BYTES = T * 128;  // one [128 x 64] bf16 block, 128-byte rows

struct PrefillParams {
  const __nv_bfloat16* Qp;  // pair-interleaved copy of Q, [B*Hq, N, D]
  __nv_bfloat16* O;
  float* LSE;
  unsigned long long* kept;
  unsigned int* status;
  int Hq, Hkv, N;
};

template <int D>
struct PrefillSmem {
  static constexpr int NB = D / 64;  // 64-column blocks per tile row
  static constexpr int Q_OFF = 0;
  static constexpr int K_OFF = Q_OFF + NB * BLK_BYTES;
  static constexpr int V_OFF = K_OFF + NB * BLK_BYTES;
  static constexpr int P_OFF = V_OFF + NB * BLK_BYTES;
  static constexpr int BAR_OFF = P_OFF + 2 * BLK_BYTES;
  static constexpr int TOTAL = BAR_OFF + 64;
  static constexpr int DYN_BYTES = TOTAL + 1024;  // slack for 1024-byte alignment
};

__global__ void __launch_bounds__(256)
atf_repack_kernel(const __nv_bfloat16* __restrict__ X, __nv_bfloat16* __restrict__ Y, int64_t rows, int D) {
  // one thread writes 8 consecutive output columns (4 pairs) of one row
  const int H = D / 2;
  const int per_row = D / 8;
  const int64_t gid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (gid >= rows * per_row) return;
  const int64_t row = gid / per_row;
  const int t = (int)(gid % per_row);
  const __nv_bfloat16* src = X + row * D;
  __align__(16) __nv_bfloat16 out[8];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int p = 4 * t + i;
    out[2 * i] = src[H - 1 - p];
    out[2 * i + 1] = src[D - 1 - p];
  }
  *reinterpret_cast<uint4*>(Y + row * D + 8 * t) = *reinterpret_cast<const uint4*>(out);
}

__device__ __forceinline__ int count_ge(const int* w, int H, int z) {
  // number of pairs whose window reaches distance z (w is non-decreasing)
  int n = 0;
  for (int r = 0; r < H; ++r) n += (w[r] >= z) ? 1 : 0;
  return n;
}

template <int D, int MODE, bool COUNT>
__global__ void __launch_bounds__(128, 1)
atf_prefill_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                   const __grid_constant__ CUtensorMap tmV, const __grid_constant__ PrefillParams P,
                   const __grid_constant__ AtfTable table) {
  using SM = PrefillSmem<D>;
  constexpr int H = D / 2;
  constexpr int NB = D / 64;
  constexpr uint32_t TMEM_COLS = 256;
  constexpr uint32_t IDESC_QK = make_idesc_bf16(128, T, 0, 0);
  constexpr uint32_t IDESC_PV = make_idesc_bf16(128, D, 0, 1);
  const float kScaleLog2 = 1.4426950408889634f / sqrtf((float)D);

  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t sQ = smem_base + SM::Q_OFF, sK = smem_base + SM::K_OFF, sV = smem_base + SM::V_OFF,
                 sP = smem_base + SM::P_OFF;
  const uint32_t bar_q = smem_base + SM::BAR_OFF, bar_kv = bar_q + 8, bar_mma = bar_q + 16;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_gen + SM::BAR_OFF + 32);
  __shared__ int sW[ATF_MAX_PAIRS];

  const int tid = threadIdx.x, warp = tid >> 5;
  const int nqt = (P.N + T - 1) / T;
  const int it = nqt - 1 - (int)blockIdx.x;  // longest rows first
  const int hq = blockIdx.y, b = blockIdx.z;
  const int bhq = b * P.Hq + hq;
  const int bhk = b * P.Hkv + hq / (P.Hq / P.Hkv);
  const int row = tid;
  const int n = it * T + row;

  if (tid < H) sW[tid] = table.w[tid];
  if (tid == 0) {
    mbar_init(bar_q, 1);
    mbar_init(bar_kv, 1);
    mbar_init(bar_mma, 1);
    mbar_fence_init();
    fence_proxy_async_smem();
    tma_prefetch_desc(&tmQ);
    tma_prefetch_desc(&tmK);
    tma_prefetch_desc(&tmV);
  }
  if (warp == 0) {
    tmem_alloc(smem_u32((const void*)tmem_slot), TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t tS = tmem_base, tO = tmem_base + T;
  const uint32_t lane_off = (uint32_t)(warp * 32) << 16;
  const int Wmax = sW[H - 1];

  if (tid == 0) {
    mbar_expect_tx(bar_q, NB * BLK_BYTES);
    for (int kb = 0; kb < NB; ++kb) tma_load_3d(sQ + kb * BLK_BYTES, &tmQ, bar_q, kb * 64, it * T, bhq);
  }
  bool ok = __syncthreads_and(mbar_wait(bar_q, 0) ? 1 : 0);
  unsigned int fail_site = ok ? 0u : 1u;

  float m_run = -INFINITY, l_run = 0.f;
  int zeroed_from = H;  // pairs p >= zeroed_from are zero in the shared copy of Q
  uint32_t ph_kv = 0, ph_mma = 0;
  bool first = true;
  unsigned long long cnt = 0;

  for (int jt = it; jt >= 0 && ok; --jt) {
    const int dt = it - jt;
    const int zmin = dt == 0 ? 0 : (dt - 1) * T + 1;
    const int zmax = (dt + 1) * T - 1;
    const int p_any = count_ge(sW, H, zmin);
    const int p_all = count_ge(sW, H, zmax);
    if (p_any == 0) break;  // no pair reaches this tile, nor any farther one
    int depth;
    if (MODE == ATF_MODE_EXACT)
      depth = p_all;
    else
      depth = dt == 0 ? H : min(H, (p_any + 7) / 8 * 8);
    const int natoms = (depth + 7) / 8;
    const int ncols_k = MODE == ATF_MODE_EXACT ? 2 * p_any : 2 * depth;
    const int nkb = (ncols_k + 63) / 64;

    if (MODE == ATF_MODE_EXACT && p_all < zeroed_from) {
      for (int p = p_all; p < zeroed_from; ++p) {
        const int col = 2 * p;
        uint8_t* qa = smem_gen + SM::Q_OFF + (col >> 6) * BLK_BYTES + sw128_offset(row, (col & 63) >> 3) + (col & 7) * 2;
        *reinterpret_cast<uint32_t*>(qa) = 0u;
      }
      zeroed_from = p_all;
      fence_proxy_async_smem();
    }
    if (tid == 0) {
      mbar_expect_tx(bar_kv, (nkb + NB) * BLK_BYTES);
      for (int kb = 0; kb < nkb; ++kb) tma_load_3d(sK + kb * BLK_BYTES, &tmK, bar_kv, kb * 64, jt * T, bhk);
      for (int kb = 0; kb < NB; ++kb) tma_load_3d(sV + kb * BLK_BYTES, &tmV, bar_kv, kb * 64, jt * T, bhk);
    }
    __syncthreads();
    ok = __syncthreads_and(mbar_wait(bar_kv, ph_kv) ? 1 : 0);
    ph_kv ^= 1;
    if (!ok) { fail_site = 2; break; }

    // ---- S = Q K^T over the live depth ----
    if (natoms > 0) {
      if (tid == 0) {
        tc_fence_after();
        for (int a = 0; a < natoms; ++a) {
          const uint32_t off = (a >> 2) * BLK_BYTES + (a & 3) * 32;
          tc_mma_ss(tS, make_smem_desc_sw128(sQ + off, 16, 1024), make_smem_desc_sw128(sK + off, 16, 1024), IDESC_QK,
                    a > 0 ? 1u : 0u);
        }
        tc_commit(bar_mma);
      }
      ok = __syncthreads_and(mbar_wait(bar_mma, ph_mma) ? 1 : 0);
      ph_mma ^= 1;
      if (!ok) { fail_site = 3; break; }
      tc_fence_after();
    }

    float s[T];
    if (natoms > 0) {
#pragma unroll
      for (int q4 = 0; q4 < 4; ++q4) tc_ld32(tS + lane_off + q4 * 32, reinterpret_cast<uint32_t*>(s) + q4 * 32);
      tc_wait_ld();
    } else {
#pragma unroll
      for (int c = 0; c < T; ++c) s[c] = 0.f;
    }

    const int m0 = jt * T;
    // ---- straddling pairs: add the term only where the distance is inside the pair's window ----
    if (MODE == ATF_MODE_EXACT) {
      for (int p = p_all; p < p_any; ++p) {
        const int wp = sW[H - 1 - p];
        float q0 = 0.f, q1 = 0.f;
        if (n < P.N) {
          const uint32_t qq = *reinterpret_cast<const uint32_t*>(P.Qp + ((int64_t)bhq * P.N + n) * D + 2 * p);
          q0 = bf16lo_to_f32(qq);
          q1 = bf16hi_to_f32(qq);
        }
        const int col = 2 * p;
        const uint8_t* kbase = smem_gen + SM::K_OFF + (col >> 6) * BLK_BYTES + (col & 7) * 2;
        const int chunk = (col & 63) >> 3;
        const int zrow = n - m0;  // distance to column 0 of the tile
#pragma unroll
        for (int c = 0; c < T; ++c) {
          const uint32_t kk = *reinterpret_cast<const uint32_t*>(kbase + c * 128 + ((chunk ^ (c & 7)) << 4));
          const float add = fmaf(q0, bf16lo_to_f32(kk), q1 * bf16hi_to_f32(kk));
          s[c] += (zrow - c <= wp) ? add : 0.f;
        }
        if (COUNT && n < P.N) {
          const int lo = max(0, zrow - wp), hi = min(T - 1, zrow);
          cnt += (unsigned long long)max(0, hi - lo + 1);
        }
      }
    }
    if (COUNT && n < P.N) {
      const int ncols = dt == 0 ? row + 1 : T;
      cnt += (unsigned long long)depth * (unsigned long long)ncols;
    }

    // ---- scale, causal mask, drop keys no pair reaches (exact mode: per cell; coarse mode
    //      decides per tile, which the loop exit above already did), online softmax ----
    const int zdrop = MODE == ATF_MODE_EXACT ? Wmax : 0x7FFFFFFF;
    const bool need_mask = (dt == 0) || (zmax > zdrop);
    float mx = -INFINITY;
    if (need_mask) {
      const int zrow = n - m0;
#pragma unroll
      for (int c = 0; c < T; ++c) {
        const int z = zrow - c;
        s[c] = (z >= 0 && z <= zdrop) ? s[c] * kScaleLog2 : -INFINITY;
        mx = fmaxf(mx, s[c]);
      }
    } else {
#pragma unroll
      for (int c = 0; c < T; ++c) {
        s[c] *= kScaleLog2;
        mx = fmaxf(mx, s[c]);
      }
    }
    const float m_new = fmaxf(m_run, mx);
    const float m_safe = (m_new == -INFINITY) ? 0.f : m_new;
    const float alpha = exp2f(m_run - m_safe);
    m_run = m_new;
    float psum = 0.f;
#pragma unroll
    for (int c = 0; c < T; ++c) {
      s[c] = exp2f(s[c] - m_safe);
      psum += s[c];
    }
    l_run = l_run * alpha + psum;

    // ---- P (bf16) into tensor memory, over the first 64 columns of S: column c of a lane
    //      holds keys 2c (low half) and 2c+1 (high half) of that query row ----
    {
      uint32_t pk[64];
#pragma unroll
      for (int c = 0; c < 64; ++c) pk[c] = pack_bf16x2(s[2 * c], s[2 * c + 1]);
      tc_st32(tS + lane_off, pk);
      tc_st32(tS + lane_off + 32, pk + 32);
    }
    // ---- rescale O ----
    if (!first) {
#pragma unroll
      for (int q4 = 0; q4 < D / 32; ++q4) {
        uint32_t o[32];
        tc_ld32(tO + lane_off + q4 * 32, o);
        tc_wait_ld();
#pragma unroll
        for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
        tc_st32(tO + lane_off + q4 * 32, o);
      }
    }
    tc_wait_st();
    tc_fence_before();
    __syncthreads();

    // ---- O += P V ----
    if (tid == 0) {
      tc_fence_after();
#pragma unroll
      for (int ks = 0; ks < T / 16; ++ks) {
        const uint64_t db = make_smem_desc_sw128(sV + ks * 2048, BLK_BYTES, 1024);
        tc_mma_ts(tO, tS + ks * 8, db, IDESC_PV, (first && ks == 0) ? 0u : 1u);
      }
      tc_commit(bar_mma);
    }
    ok = __syncthreads_and(mbar_wait(bar_mma, ph_mma) ? 1 : 0);
    ph_mma ^= 1;
    if (!ok) { fail_site = 4; break; }
    tc_fence_after();
    first = false;
  }

  if (ok) {
    // ---- epilogue: O / l, LSE ----
    const float inv = 1.f / l_run;
    __nv_bfloat16* orow = P.O + ((int64_t)bhq * P.N + n) * D;
#pragma unroll
    for (int q4 = 0; q4 < D / 32; ++q4) {
      uint32_t o[32];
      tc_ld32(tO + lane_off + q4 * 32, o);
      tc_wait_ld();
      if (n < P.N) {
#pragma unroll
        for (int e = 0; e < 32; e += 8) {
          uint4 v;
          v.x = pack_bf16x2(__uint_as_float(o[e]) * inv, __uint_as_float(o[e + 1]) * inv);
          v.y = pack_bf16x2(__uint_as_float(o[e + 2]) * inv, __uint_as_float(o[e + 3]) * inv);
          v.z = pack_bf16x2(__uint_as_float(o[e + 4]) * inv, __uint_as_float(o[e + 5]) * inv);
          v.w = pack_bf16x2(__uint_as_float(o[e + 6]) * inv, __uint_as_float(o[e + 7]) * inv);
          *reinterpret_cast<uint4*>(orow + q4 * 32 + e) = v;
        }
      }
    }
    if (P.LSE && n < P.N) P.LSE[(int64_t)bhq * P.N + n] = (m_run + log2f(l_run)) * 0.6931471805599453f;
    if (COUNT) {
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, off);
      if ((tid & 31) == 0 && cnt) atomicAdd(P.kept + bhq, cnt);
    }
  } else if (tid == 0) {
    atomicExch(P.status, 1u);
    atomicExch(P.status + 1, fail_site);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, TMEM_COLS);
}

// ---- host ----
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn) return fn;
  void* p = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess) return nullptr;
  if (qres != cudaDriverEntryPointSuccess) return nullptr;
  fn = (EncodeTiledFn)p;
  return fn;
}

// [BH, N, D] bf16 tensor, box = 64 columns x 128 rows x 1, 128-byte swizzle, zero fill outside.
atf_status make_tile_map(CUtensorMap* m, const void* base, int64_t BH, int64_t N, int D) {
  EncodeTiledFn enc = get_encode_fn();
  if (!enc) return atf_fail(ATF_ERR_CUDA, "cuTensorMapEncodeTiled is not available from this driver");
  cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)N, (cuuint64_t)BH};
  cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)N * D * 2};
  cuuint32_t box[3] = {64, (cuuint32_t)T, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return atf_fail(ATF_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);
  return ATF_OK;
}

template <int D>
atf_status launch_prefill(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const PrefillParams& P,
                          const AtfTable& t, int B, int mode, bool count, cudaStream_t s) {
  const int nqt = (P.N + T - 1) / T;
  dim3 grid(nqt, P.Hq, B);
  const int smem = PrefillSmem<D>::DYN_BYTES;
#define ATF_PF_LAUNCH(MODE_, COUNT_)                                                                        \
  do {                                                                                                      \
    auto kern = atf_prefill_kernel<D, MODE_, COUNT_>;                                                       \
    ATF_CUDA_CHECK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));          \
    kern<<<grid, 128, smem, s>>>(tq, tk, tv, P, t);                                                         \
  } while (0)
  if (mode == ATF_MODE_EXACT) {
    if (count) ATF_PF_LAUNCH(ATF_MODE_EXACT, true); else ATF_PF_LAUNCH(ATF_MODE_EXACT, false);
  } else {
    if (count) ATF_PF_LAUNCH(ATF_MODE_COARSE, true); else ATF_PF_LAUNCH(ATF_MODE_COARSE, false);
  }
#undef ATF_PF_LAUNCH
  ATF_CUDA_CHECK(cudaGetLastError());
  return ATF_OK;
}

size_t repack_bytes(int B, int H, int64_t N, int d) {
  size_t b = (size_t)B * H * N * d * 2;
  return (b + 255) & ~(size_t)255;
}

}  // namespace

atf_status atf_validate_table(const char* who, const int64_t* table, int d, int64_t N, AtfTable* out);

size_t atf_prefill_workspace_bytes(int B, int Hq, int Hkv, int64_t N, int d) {
  return ATF_WS_HEADER + repack_bytes(B, Hq, N, d) + repack_bytes(B, Hkv, N, d);
}

extern "C" atf_status atf_prefill_ex(const void* Q, const void* K, const void* V, void* O, float* LSE, int B, int Hq,
                                     int Hkv, int64_t N, int d, const int64_t* table, int causal,
                                     const atf_opts* opts, void* stream) {
  if (!Q || !K || !V || !O) return atf_fail(ATF_ERR_INVALID_ARG, "atf_prefill: null pointer");
  if (d != 64 && d != 128) return atf_fail(ATF_ERR_UNSUPPORTED, "atf_prefill: d must be 64 or 128 (got %d)", d);
  if (B < 1 || Hq < 1 || Hkv < 1 || N < 1) return atf_fail(ATF_ERR_INVALID_ARG, "atf_prefill: bad shape");
  if (Hq % Hkv) return atf_fail(ATF_ERR_INVALID_ARG, "atf_prefill: Hq must be a multiple of Hkv");
  if (!causal) return atf_fail(ATF_ERR_UNSUPPORTED, "atf_prefill: only causal attention is defined (distance z = n - m >= 0)");
  if (N >= (1ll << 31) - 2 * T) return atf_fail(ATF_ERR_UNSUPPORTED, "atf_prefill: N too large");
  if (Hq > 65535 || B > 65535) return atf_fail(ATF_ERR_UNSUPPORTED, "atf_prefill: B and Hq must be <= 65535");
  if (((uintptr_t)Q | (uintptr_t)K | (uintptr_t)V | (uintptr_t)O) & 15)
    return atf_fail(ATF_ERR_INVALID_ARG, "atf_prefill: pointers must be 16-byte aligned");
  const int mode = opts ? opts->mode : ATF_MODE_EXACT;
  if (mode != ATF_MODE_EXACT && mode != ATF_MODE_COARSE) return atf_fail(ATF_ERR_INVALID_ARG, "atf_prefill: unknown mode %d", mode);
  AtfTable t;
  atf_status st = atf_validate_table("atf_prefill", table, d, N, &t);
  if (st != ATF_OK) return st;

  AtfWorkspace ws = atf_bound_workspace();
  if (opts && opts->workspace) ws = AtfWorkspace{opts->workspace, opts->workspace_bytes};
  const size_t need = atf_prefill_workspace_bytes(B, Hq, Hkv, N, d);
  if (!ws.ptr) return atf_fail(ATF_ERR_WORKSPACE, "atf_prefill: no workspace bound");
  if (ws.bytes < need) return atf_fail(ATF_ERR_WORKSPACE, "atf_prefill: workspace has %zu bytes, needs %zu", ws.bytes, need);
  if ((uintptr_t)ws.ptr & 255) return atf_fail(ATF_ERR_INVALID_ARG, "atf_prefill: workspace must be 256-byte aligned");

  char* base = (char*)ws.ptr;
  __nv_bfloat16* Qp = (__nv_bfloat16*)(base + ATF_WS_HEADER);
  __nv_bfloat16* Kp = (__nv_bfloat16*)(base + ATF_WS_HEADER + repack_bytes(B, Hq, N, d));
  cudaStream_t s = (cudaStream_t)stream;

  {
    const int64_t rows_q = (int64_t)B * Hq * N, rows_k = (int64_t)B * Hkv * N;
    const int64_t bq = (rows_q * (d / 8) + 255) / 256, bk = (rows_k * (d / 8) + 255) / 256;
    if (bq > 0x7FFFFFFF) return atf_fail(ATF_ERR_UNSUPPORTED, "atf_prefill: problem too large for the repack grid");
    atf_repack_kernel<<<(unsigned)bq, 256, 0, s>>>((const __nv_bfloat16*)Q, Qp, rows_q, d);
    atf_repack_kernel<<<(unsigned)bk, 256, 0, s>>>((const __nv_bfloat16*)K, Kp, rows_k, d);
    ATF_CUDA_CHECK(cudaGetLastError());
  }

  CUtensorMap tq, tk, tv;
  if ((st = make_tile_map(&tq, Qp, (int64_t)B * Hq, N, d)) != ATF_OK) return st;
  if ((st = make_tile_map(&tk, Kp, (int64_t)B * Hkv, N, d)) != ATF_OK) return st;
  if ((st = make_tile_map(&tv, V, (int64_t)B * Hkv, N, d)) != ATF_OK) return st;

  PrefillParams P;
  P.Qp = Qp;
  P.O = (__nv_bfloat16*)O;
  P.LSE = LSE;
  P.kept = opts ? (unsigned long long*)opts->kept_terms : nullptr;
  P.status = (unsigned int*)base;
  P.Hq = Hq;
  P.Hkv = Hkv;
  P.N = (int)N;
  const bool count = P.kept != nullptr;
  return d == 64 ? launch_prefill<64>(tq, tk, tv, P, t, B, mode, count, s)
                 : launch_prefill<128>(tq, tk, tv, P, t, B, mode, count, s);
}

extern "C" atf_status atf_prefill(const void* Q, const void* K, const void* V, void* O, float* LSE, int B, int Hq,
                                  int Hkv, int64_t N, int d, const int64_t* table, int causal, void* stream) {
  return atf_prefill_ex(Q, K, V, O, LSE, B, Hq, Hkv, N, d, table, causal, nullptr, stream);
}
