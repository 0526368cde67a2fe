// atf_decode: split-K windowed attention of one query row per (batch, head) against a
// contiguous KV cache (Sec. 5; the last row of Fig. 3).  Bandwidth-bound: every load is a
// 16-byte vector load, a row of the cache is covered by consecutive lanes, and a lane whose
// 16-byte chunk of a key row lies wholly outside the key's live pair range issues no load
// (Sec. 3.3: out-of-window components are not brought on chip).  V rows are read in full.
//
// Work split: grid = (splits, Hkv, B).  A block owns a contiguous key range; each of its 8
// warps walks that range in blocks of keys with its own online-softmax state for the G = Hq/Hkv
// query heads that share the KV head, the warps are merged through shared memory, the block
// writes one partial (m, l, o) per head, and the last block to finish for a (batch, KV head)
// merges the partials of all splits by their log-sum-exp and writes O (and LSE).
#include <cfloat>

#include "atf_common.cuh"

namespace {

constexpr int DEC_THREADS = 256;
constexpr int DEC_WARPS = DEC_THREADS / 32;
constexpr int DEC_NLD = 8;  // loads in flight per lane for K, and again for V

__device__ __forceinline__ uint4 ld_nc_v4(const void* p) {
  uint4 r;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
               : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
               : "l"(p));
  return r;
}
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t sel) {
  uint32_t d;
  asm("prmt.b32 %0, %1, 0, %2;" : "=r"(d) : "r"(a), "r"(sel));
  return d;
}

struct DecodeParams {
  const __nv_bfloat16* q;
  const __nv_bfloat16* K;
  const __nv_bfloat16* V;
  __nv_bfloat16* O;
  float* lse;            // may be null
  float* partials;       // [B*Hkv][nsplit][G][D + 2]
  unsigned int* counters;  // [B*Hkv], zero between launches
  unsigned long long* kept;  // may be null
  int Hq, Hkv, L, nsplit, keys_per_split;
};

template <int D, int G, int MODE, bool COUNT>
__global__ void __launch_bounds__(DEC_THREADS)
atf_decode_kernel(const __grid_constant__ DecodeParams P, const __grid_constant__ AtfTable table) {
  constexpr int H = D / 2;
  constexpr int LPR = D / 8;         // lanes per key row (16-byte chunks per row)
  constexpr int KPL = 32 / LPR;      // keys covered by one warp-wide load
  constexpr int KB = DEC_NLD * KPL;  // keys per warp iteration
  constexpr int PSTRIDE = D + 2;     // floats per (split, head) partial: m, l, o[D]
  const float kScaleLog2 = 1.4426950408889634f / sqrtf((float)D);

  const int split = blockIdx.x, hkv = blockIdx.y, b = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int sub = lane / LPR;  // which key of a warp-wide load
  const int c = lane % LPR;    // 16-byte chunk of the row
  const int p0 = (c % (LPR / 2)) * 8;  // first pair of the chunk (same in both halves)
  const int L = P.L;
  const int m0 = split * P.keys_per_split;
  const int m1 = min(L, m0 + P.keys_per_split);
  const int64_t slab = ((int64_t)b * P.Hkv + hkv) * (int64_t)L * D;
  const __nv_bfloat16* Kb = P.K + slab;
  const __nv_bfloat16* Vb = P.V + slab;

  int Wl[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) Wl[i] = table.w[p0 + i];
  const int Wmax = table.w[H - 1];

  // query chunk of each head of the group, pre-multiplied by scale*log2(e)
  float qf[G][8];
#pragma unroll
  for (int g = 0; g < G; ++g) {
    const __nv_bfloat16* qp = P.q + ((int64_t)b * P.Hq + hkv * G + g) * D + c * 8;
    uint4 v = *reinterpret_cast<const uint4*>(qp);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      qf[g][2 * j] = bf16lo_to_f32(w[j]) * kScaleLog2;
      qf[g][2 * j + 1] = bf16hi_to_f32(w[j]) * kScaleLog2;
    }
  }

  float mrun[G], lrun[G], o[G][8];
#pragma unroll
  for (int g = 0; g < G; ++g) {
    mrun[g] = -INFINITY;
    lrun[g] = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) o[g][i] = 0.f;
  }
  unsigned long long cnt = 0;

  for (int kb0 = m0 + warp * KB; kb0 < m1; kb0 += DEC_WARPS * KB) {
    // ---- issue every load of this block of keys ----
    uint4 kreg[DEC_NLD], vreg[DEC_NLD];
#pragma unroll
    for (int i = 0; i < DEC_NLD; ++i) {
      const int key = kb0 + i * KPL + sub;
      const int z = L - 1 - key;
      const bool valid = key < m1;
      kreg[i] = make_uint4(0, 0, 0, 0);
      if (valid && z <= Wl[7]) kreg[i] = ld_nc_v4(Kb + (int64_t)key * D + c * 8);
    }
#pragma unroll
    for (int i = 0; i < DEC_NLD; ++i) {
      const int key = kb0 + i * KPL + sub;
      vreg[i] = make_uint4(0, 0, 0, 0);
      if (key < m1) vreg[i] = ld_nc_v4(Vb + (int64_t)key * D + c * 8);
    }

    // ---- per-element selectors (exact mode): is the window predicate constant over the block? ----
    uint32_t sel_lo[4], sel_hi[4];
    bool uniform = true;
    if (MODE == ATF_MODE_EXACT) {
      const int z_near = L - 1 - min(kb0 + KB - 1, m1 - 1);
      const int z_far = L - 1 - kb0;
      bool same = true;
#pragma unroll
      for (int i = 0; i < 8; ++i) same = same && ((z_near <= Wl[i]) == (z_far <= Wl[i]));
      uniform = __all_sync(0xffffffffu, same);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        sel_lo[j] = (z_far <= Wl[2 * j]) ? 0x1044u : 0x4444u;
        sel_hi[j] = (z_far <= Wl[2 * j + 1]) ? 0x3244u : 0x4444u;
      }
    }

    // ---- scores ----
    float s[DEC_NLD][G];
#pragma unroll
    for (int i = 0; i < DEC_NLD; ++i) {
      const int key = kb0 + i * KPL + sub;
      const int z = L - 1 - key;
      const uint32_t w[4] = {kreg[i].x, kreg[i].y, kreg[i].z, kreg[i].w};
      float kf[8];
      if (MODE == ATF_MODE_EXACT) {
        if (!uniform) {
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            sel_lo[j] = (z <= Wl[2 * j]) ? 0x1044u : 0x4444u;
            sel_hi[j] = (z <= Wl[2 * j + 1]) ? 0x3244u : 0x4444u;
          }
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          kf[2 * j] = __uint_as_float(prmt(w[j], sel_lo[j]));
          kf[2 * j + 1] = __uint_as_float(prmt(w[j], sel_hi[j]));
        }
      } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          kf[2 * j] = bf16lo_to_f32(w[j]);
          kf[2 * j + 1] = bf16hi_to_f32(w[j]);
        }
      }
      if (COUNT) {
        if (key < m1 && c < LPR / 2) {
          if (MODE == ATF_MODE_EXACT) {
#pragma unroll
            for (int e = 0; e < 8; ++e) cnt += (z <= Wl[e]) ? 1 : 0;
          } else {
            cnt += (z <= Wl[7]) ? 8 : 0;
          }
        }
      }
#pragma unroll
      for (int g = 0; g < G; ++g) {
        float a = 0.f;
#pragma unroll
        for (int e = 0; e < 8; ++e) a = fmaf(qf[g][e], kf[e], a);
#pragma unroll
        for (int off = 1; off < LPR; off <<= 1) a += __shfl_xor_sync(0xffffffffu, a, off);
        s[i][g] = (key < m1 && z <= Wmax) ? a : -INFINITY;
      }
    }

    // ---- online softmax (log2 domain) and P*V ----
#pragma unroll
    for (int g = 0; g < G; ++g) {
      float bm = s[0][g];
#pragma unroll
      for (int i = 1; i < DEC_NLD; ++i) bm = fmaxf(bm, s[i][g]);
#pragma unroll
      for (int off = LPR; off < 32; off <<= 1) bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, off));
      const float mnew = fmaxf(mrun[g], bm);
      const float msafe = (mnew == -INFINITY) ? 0.f : mnew;
      const float alpha = exp2f(mrun[g] - msafe);
      mrun[g] = mnew;
      float psum = 0.f;
#pragma unroll
      for (int e = 0; e < 8; ++e) o[g][e] *= alpha;
#pragma unroll
      for (int i = 0; i < DEC_NLD; ++i) {
        const float p = exp2f(s[i][g] - msafe);
        psum += p;
        const uint32_t w[4] = {vreg[i].x, vreg[i].y, vreg[i].z, vreg[i].w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          o[g][2 * j] = fmaf(p, bf16lo_to_f32(w[j]), o[g][2 * j]);
          o[g][2 * j + 1] = fmaf(p, bf16hi_to_f32(w[j]), o[g][2 * j + 1]);
        }
      }
      lrun[g] = lrun[g] * alpha + psum;
    }
  }

  // ---- merge the key sub-groups of the warp (they share mrun) ----
#pragma unroll
  for (int g = 0; g < G; ++g) {
#pragma unroll
    for (int off = LPR; off < 32; off <<= 1) {
      lrun[g] += __shfl_xor_sync(0xffffffffu, lrun[g], off);
#pragma unroll
      for (int e = 0; e < 8; ++e) o[g][e] += __shfl_xor_sync(0xffffffffu, o[g][e], off);
    }
  }

  // ---- merge the warps of the block ----
  extern __shared__ float sm[];  // [DEC_WARPS][G][PSTRIDE]
  if (sub == 0) {
#pragma unroll
    for (int g = 0; g < G; ++g) {
      float* dst = sm + ((warp * G + g) * PSTRIDE);
      if (c == 0) {
        dst[0] = mrun[g];
        dst[1] = lrun[g];
      }
#pragma unroll
      for (int e = 0; e < 8; ++e) dst[2 + c * 8 + e] = o[g][e];
    }
  }
  __syncthreads();
  const int64_t grp = (int64_t)b * P.Hkv + hkv;
  float* part = P.partials + (grp * P.nsplit + split) * (int64_t)(G * PSTRIDE);
  for (int idx = threadIdx.x; idx < G * D; idx += DEC_THREADS) {
    const int g = idx / D, col = idx % D;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < DEC_WARPS; ++w) M = fmaxf(M, sm[(w * G + g) * PSTRIDE]);
    const float Ms = (M == -INFINITY) ? 0.f : M;
    float acc = 0.f, lacc = 0.f;
#pragma unroll
    for (int w = 0; w < DEC_WARPS; ++w) {
      const float* src = sm + (w * G + g) * PSTRIDE;
      const float f = exp2f(src[0] - Ms);
      acc += f * src[2 + col];
      lacc += f * src[1];
    }
    part[g * PSTRIDE + 2 + col] = acc;
    if (col == 0) {
      part[g * PSTRIDE] = M;
      part[g * PSTRIDE + 1] = lacc;
    }
  }
  if (COUNT) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, off);
    if (lane == 0 && cnt) {
      for (int g = 0; g < G; ++g) atomicAdd(P.kept + (int64_t)b * P.Hq + hkv * G + g, cnt);
    }
  }

  // ---- last block of this (batch, KV head) merges all splits ----
  __shared__ unsigned int s_last;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const unsigned int done = atomicAdd(P.counters + grp, 1u);
    s_last = (done == (unsigned)P.nsplit - 1) ? 1u : 0u;
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  const float* allp = P.partials + grp * P.nsplit * (int64_t)(G * PSTRIDE);
  // one warp per head: lanes stride over the splits for the LSE merge, then over columns
  for (int g = warp; g < G; g += DEC_WARPS) {
    float M = -INFINITY;
    for (int sp = lane; sp < P.nsplit; sp += 32) M = fmaxf(M, __ldcg(allp + ((int64_t)sp * G + g) * PSTRIDE));
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, off));
    const float Ms = (M == -INFINITY) ? 0.f : M;
    float Lsum = 0.f;
    for (int sp = lane; sp < P.nsplit; sp += 32) {
      const float* src = allp + ((int64_t)sp * G + g) * PSTRIDE;
      Lsum += exp2f(__ldcg(src) - Ms) * __ldcg(src + 1);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) Lsum += __shfl_xor_sync(0xffffffffu, Lsum, off);
    const float inv = 1.f / Lsum;
    float acc[D / 32];
#pragma unroll
    for (int t = 0; t < D / 32; ++t) acc[t] = 0.f;
    for (int sp = 0; sp < P.nsplit; ++sp) {
      const float* src = allp + ((int64_t)sp * G + g) * PSTRIDE;
      const float f = exp2f(__ldcg(src) - Ms);
#pragma unroll
      for (int t = 0; t < D / 32; ++t) acc[t] = fmaf(f, __ldcg(src + 2 + t * 32 + lane), acc[t]);
    }
    const int64_t hq = (int64_t)b * P.Hq + hkv * G + g;
#pragma unroll
    for (int t = 0; t < D / 32; ++t) P.O[hq * D + t * 32 + lane] = __float2bfloat16_rn(acc[t] * inv);
    if (P.lse && lane == 0) P.lse[hq] = (Ms + log2f(Lsum)) * 0.6931471805599453f;
  }
  if (threadIdx.x == 0) P.counters[grp] = 0;  // ready for the next launch
}

template <int D, int G>
atf_status launch_decode(const DecodeParams& P, const AtfTable& t, int B, int mode, bool count, cudaStream_t s) {
  dim3 grid(P.nsplit, P.Hkv, B);
  const size_t smem = (size_t)DEC_WARPS * G * (D + 2) * sizeof(float);
#define ATF_DEC_LAUNCH(MODE_, COUNT_)                                                                   \
  do {                                                                                                  \
    auto kern = atf_decode_kernel<D, G, MODE_, COUNT_>;                                                 \
    if (smem > 48 * 1024) ATF_CUDA_CHECK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)); \
    kern<<<grid, DEC_THREADS, smem, s>>>(P, t);                                                         \
  } while (0)
  if (mode == ATF_MODE_EXACT) {
    if (count) ATF_DEC_LAUNCH(ATF_MODE_EXACT, true); else ATF_DEC_LAUNCH(ATF_MODE_EXACT, false);
  } else {
    if (count) ATF_DEC_LAUNCH(ATF_MODE_COARSE, true); else ATF_DEC_LAUNCH(ATF_MODE_COARSE, false);
  }
#undef ATF_DEC_LAUNCH
  ATF_CUDA_CHECK(cudaGetLastError());
  return ATF_OK;
}

template <int D>
atf_status dispatch_group(int G, const DecodeParams& P, const AtfTable& t, int B, int mode, bool count, cudaStream_t s) {
  switch (G) {
    case 1: return launch_decode<D, 1>(P, t, B, mode, count, s);
    case 2: return launch_decode<D, 2>(P, t, B, mode, count, s);
    case 3: return launch_decode<D, 3>(P, t, B, mode, count, s);
    case 4: return launch_decode<D, 4>(P, t, B, mode, count, s);
    case 5: return launch_decode<D, 5>(P, t, B, mode, count, s);
    case 6: return launch_decode<D, 6>(P, t, B, mode, count, s);
    case 7: return launch_decode<D, 7>(P, t, B, mode, count, s);
    case 8: return launch_decode<D, 8>(P, t, B, mode, count, s);
    default: return atf_fail(ATF_ERR_UNSUPPORTED, "atf_decode: Hq/Hkv must be in 1..8 (got %d)", G);
  }
}

}  // namespace

atf_status atf_validate_table(const char* who, const int64_t* table, int d, int64_t N, AtfTable* out);

static size_t decode_ws_bytes(int B, int Hq, int Hkv, int64_t L, int d) {
  const int ns = atf_decode_num_splits(B, Hkv, L);
  size_t partials = (size_t)B * Hq * ns * (d + 2) * sizeof(float);
  partials = (partials + 255) & ~(size_t)255;
  return ATF_WS_HEADER + partials;
}
size_t atf_decode_workspace_bytes(int B, int Hq, int Hkv, int64_t L, int d) { return decode_ws_bytes(B, Hq, Hkv, L, d); }

extern "C" atf_status atf_decode_ex(const void* q, const void* Kcache, const void* Vcache, void* O, int B, int Hq,
                                    int Hkv, int64_t L, int d, const int64_t* table, const atf_opts* opts,
                                    void* stream) {
  if (!q || !Kcache || !Vcache || !O) return atf_fail(ATF_ERR_INVALID_ARG, "atf_decode: null pointer");
  if (d != 64 && d != 128) return atf_fail(ATF_ERR_UNSUPPORTED, "atf_decode: d must be 64 or 128 (got %d)", d);
  if (B < 1 || Hq < 1 || Hkv < 1 || L < 1) return atf_fail(ATF_ERR_INVALID_ARG, "atf_decode: bad shape");
  if (Hq % Hkv) return atf_fail(ATF_ERR_INVALID_ARG, "atf_decode: Hq must be a multiple of Hkv");
  if (L * (int64_t)d >= (1ll << 31)) return atf_fail(ATF_ERR_UNSUPPORTED, "atf_decode: L*d must be below 2^31");
  if (B > 65535 || Hkv > 65535 || (int64_t)B * Hkv > ATF_WS_COUNTER_SLOTS)
    return atf_fail(ATF_ERR_UNSUPPORTED, "atf_decode: B*Hkv must be <= %d", ATF_WS_COUNTER_SLOTS);
  if (((uintptr_t)q | (uintptr_t)Kcache | (uintptr_t)Vcache | (uintptr_t)O) & 15)
    return atf_fail(ATF_ERR_INVALID_ARG, "atf_decode: pointers must be 16-byte aligned");
  const int mode = opts ? opts->mode : ATF_MODE_EXACT;
  if (mode != ATF_MODE_EXACT && mode != ATF_MODE_COARSE) return atf_fail(ATF_ERR_INVALID_ARG, "atf_decode: unknown mode %d", mode);
  AtfTable t;
  atf_status st = atf_validate_table("atf_decode", table, d, L, &t);
  if (st != ATF_OK) return st;

  AtfWorkspace ws = atf_bound_workspace();
  if (opts && opts->workspace) ws = AtfWorkspace{opts->workspace, opts->workspace_bytes};
  const size_t need = decode_ws_bytes(B, Hq, Hkv, L, d);
  if (!ws.ptr) return atf_fail(ATF_ERR_WORKSPACE, "atf_decode: no workspace bound");
  if (ws.bytes < need) return atf_fail(ATF_ERR_WORKSPACE, "atf_decode: workspace has %zu bytes, needs %zu", ws.bytes, need);
  if ((uintptr_t)ws.ptr & 255) return atf_fail(ATF_ERR_INVALID_ARG, "atf_decode: workspace must be 256-byte aligned");

  DecodeParams P;
  P.q = (const __nv_bfloat16*)q;
  P.K = (const __nv_bfloat16*)Kcache;
  P.V = (const __nv_bfloat16*)Vcache;
  P.O = (__nv_bfloat16*)O;
  P.lse = opts ? opts->lse : nullptr;
  P.kept = opts ? (unsigned long long*)opts->kept_terms : nullptr;
  P.Hq = Hq;
  P.Hkv = Hkv;
  P.L = (int)L;
  P.nsplit = atf_decode_num_splits(B, Hkv, L);
  const int kb = 8 * (32 / (d / 8));  // keys per warp iteration
  int64_t kps = (L + P.nsplit - 1) / P.nsplit;
  kps = (kps + kb - 1) / kb * kb;
  P.keys_per_split = (int)kps;
  P.nsplit = (int)((L + kps - 1) / kps);  // drop splits the rounding emptied
  char* base = (char*)ws.ptr;
  P.counters = (unsigned int*)(base + ATF_WS_STATUS_BYTES);
  P.partials = (float*)(base + ATF_WS_HEADER);
  cudaStream_t s = (cudaStream_t)stream;
  const bool count = P.kept != nullptr;
  return d == 64 ? dispatch_group<64>(Hq / Hkv, P, t, B, mode, count, s)
                 : dispatch_group<128>(Hq / Hkv, P, t, B, mode, count, s);
}

extern "C" atf_status atf_decode(const void* q, const void* Kcache, const void* Vcache, void* O, int B, int Hq,
                                 int Hkv, int64_t L, int d, const int64_t* table, void* stream) {
  return atf_decode_ex(q, Kcache, Vcache, O, B, Hq, Hkv, L, d, table, nullptr, stream);
}
