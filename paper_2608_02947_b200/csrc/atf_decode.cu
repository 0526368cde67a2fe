// atf_decode: split-K windowed attention of one query row per (batch, head) against a
// contiguous KV cache (Sec. 5; the last row of Fig. 3).  Bandwidth-bound: what matters is which
// bytes leave DRAM.
//
// K cache layouts.  In the row layout [L, d] (the layout atf_prefill takes) every 128-byte half
// of a key row ends in live low-frequency pairs, and DRAM moves whole 128-byte lines, so the
// window cannot save traffic there: rows are copied whole and the dead pairs are masked in
// registers (a key no pair reaches is not copied at all).  In the tiled group-major layout
// (written by atf_kcache_pack or by atf_prefill itself) the pairs a far key keeps are a contiguous
// prefix of each tile, and only that prefix is fetched (Sec. 3.3: components outside the window
// never come on chip).  V rows are read in full in both.
//
// Work split: grid = (splits, Hkv, B).  Tiles of 64 (d = 128) or 128 (d = 64) keys are dealt
// round-robin to the splits; each of a block's 4 warps takes a quarter of a tile through its own
// two-stage cp.async ring.  Per block of keys a warp computes, for the (up to 8) query heads that
// share the KV head at once:
//   S = q K^T   with mma.sync (m16n8k16, bf16 in, fp32 accumulate; the heads are the M rows),
//   the online softmax in registers (log2 domain, lazy rescaling),
//   O += P V    with mma.sync, V fragments transposed by ldmatrix.
// The arithmetic is a few instructions per key, so the loads in flight set the speed.  The
// warps are merged through shared memory, the block writes one partial (m, l, o) per head, and
// the last block to finish for a (batch, KV head) merges the partials of all splits by their
// log-sum-exp and writes O (and LSE).
#include <algorithm>
#include <cfloat>
#include <cmath>
#include <cstring>

#include "atf_common.cuh"

namespace {

constexpr int DEC_WARPS = 4;
constexpr int DEC_THREADS = DEC_WARPS * 32;
#ifndef ATF_DEC_STAGES
#define ATF_DEC_STAGES 2
#endif
constexpr int DEC_STAGES = ATF_DEC_STAGES;
constexpr int DEC_TILE_BYTES = 4096;                               // one K or V block of a warp in the cache
// In shared memory a block's rows are padded by 16 bytes (row layouts: per cache row; group-major
// K: per 4 keys of a group) so that ldmatrix is free of bank conflicts with plain, unswizzled,
// compile-time offsets.
constexpr int DEC_TILE_SMEM = 4608;
constexpr int DEC_STAGE_SMEM = 2 * DEC_TILE_SMEM;                  // K block + V block
constexpr int DEC_WARP_SMEM = DEC_STAGES * DEC_STAGE_SMEM;         // K and V rings of one warp
constexpr int DEC_SMEM = DEC_WARPS * DEC_WARP_SMEM;
constexpr int DEC_SMEM_ROWS = 110 * 1024;  // row layout: ask for enough to keep it at 2 blocks per SM
constexpr float DEC_RESCALE_THRESHOLD = 8.f;

struct DecodeParams {
  const __nv_bfloat16* q;
  const __nv_bfloat16* K;
  const __nv_bfloat16* V;
  __nv_bfloat16* O;
  float* lse;                // may be null
  float* partials;           // [B*Hkv][nsplit][G][D + 2]
  unsigned int* status;      // two status words of the workspace (give-up report)
  unsigned int* counters;    // [B*Hkv], zero between launches
  unsigned long long* kept;  // may be null
  int Hq, Hkv, G, L, nsplit;
  int ktiles;                // group-major K cache: tiles per (batch, KV head), >= ceil(L / tile keys)
  const float2* rot_key;     // unrotated cache only: (cos, sin) of key-in-tile * theta, [pair][key in tile]
  const float2* rot_tile;    // unrotated cache only: (cos, sin) of (pos0 + tile * tile keys) * theta, [tile][pair]
};

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
// D (16x8, fp32) += A (16x16, bf16, rows 8..15 zero) * B (16x8, bf16)
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

template <int D, int MODE, bool COUNT>
__global__ void __launch_bounds__(DEC_THREADS, 2)
atf_decode_kernel(const __grid_constant__ DecodeParams P, const __grid_constant__ AtfTable table) {
  constexpr int H = D / 2;
  constexpr int CPR = D / 8;            // 16-byte chunks per cache row
  constexpr int ROWB = D * 2;           // bytes per cache row
  constexpr int KB = DEC_TILE_BYTES / ROWB;  // keys per block (16 for d=128, 32 for d=64)
  constexpr int NKG = KB / 8;           // groups of 8 keys (MMA N tiles of S)
  constexpr int NKS = D / 16;           // MMA K steps of q K^T
  constexpr int NNT = D / 8;            // MMA N tiles of O
  constexpr int PSTRIDE = D + 2;        // floats per (split, head) partial: m, l, o[D]
  constexpr int CP_PER_LANE = KB * CPR / 32;
  const float kScaleLog2 = 1.4426950408889634f / sqrtf((float)D);

  extern __shared__ __align__(128) uint8_t dsm[];
  __shared__ int sW[ATF_MAX_PAIRS];
  __shared__ unsigned int s_last;

  const int split = blockIdx.x, hkv = blockIdx.y, b = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;  // MMA fragment row (query head) and column pair
  const int G = P.G, L = P.L;
  // Tiles of DEC_WARPS * KB keys are dealt round-robin to the splits of a (batch, KV head), so
  // that at any moment the splits read neighbouring tiles: DRAM sees a few moving sequential
  // streams instead of one stream per block (measured faster than contiguous ranges per split).
  const int m0 = split * (DEC_WARPS * KB);
  const int m1 = L;
  const int64_t slab = ((int64_t)b * P.Hkv + hkv) * (int64_t)L * D;
  const __nv_bfloat16* Kb = P.K + slab;
  if (threadIdx.x < H) sW[threadIdx.x] = table.w[threadIdx.x];
  __syncthreads();
  const int Wmax = sW[H - 1];

  // A fragments of q for every K step: rows = heads of the group (rows >= G stay zero); K step j
  // contracts dims 16j..16j+15.
  uint32_t qa[NKS][2];
#pragma unroll
  for (int j = 0; j < NKS; ++j) {
    qa[j][0] = 0u;
    qa[j][1] = 0u;
    if (g < G) {
      const __nv_bfloat16* qrow = P.q + ((int64_t)b * P.Hq + hkv * G + g) * D;
      qa[j][0] = *reinterpret_cast<const uint32_t*>(qrow + 16 * j + 2 * t);
      qa[j][1] = *reinterpret_cast<const uint32_t*>(qrow + 16 * j + 8 + 2 * t);
    }
  }

  // ---- copy and fragment addressing, fixed per lane ----
  constexpr int PITCH = ROWB + 16;          // shared-memory row pitch of a row-layout block
  constexpr int RSTEP = 32 / CPR;           // rows covered by one warp-wide copy
  static_assert(KB * PITCH <= DEC_TILE_SMEM, "block does not fit its shared-memory tile");
  const int cp_chunk = lane % CPR;          // this lane's 16-byte chunk of a cache row
  const int cp_row0 = lane / CPR;           // first row this lane copies; then every RSTEP rows
  const uint32_t cp_dst0 = cp_row0 * PITCH + cp_chunk * 16;
  const uint32_t warp_smem = smem_u32(dsm) + warp * DEC_WARP_SMEM;
  const int lm_i = lane >> 3, lm_r = lane & 7;  // ldmatrix: matrix fed by this lane and row in it
  const uint32_t k_lane_off = ((lm_i >> 1) * 8 + lm_r) * PITCH + (lm_i & 1) * 16;
  const uint32_t v_lane_off = ((lm_i & 1) * 8 + lm_r) * PITCH + (lm_i >> 1) * 16;

  const __nv_bfloat16* Vb = P.V + slab;
  auto issue_block = [&](int kb0, int stage) {
    const uint32_t ks = warp_smem + stage * DEC_STAGE_SMEM, vs = ks + DEC_TILE_SMEM;
    // every key of the block exists and is reached by some pair: no predicates
    const bool fast = (kb0 + KB <= m1) && (L - 1 - kb0 <= Wmax);
    // V rows, and K rows in the row layout, are copied whole: a 128-byte half row always ends in
    // live low-frequency pairs and DRAM moves whole 128-byte lines, so leaving out dead 16-byte
    // chunks of a row would save no traffic.  A key no pair reaches is not copied at all.
    if (fast) {
      const int64_t goff = (int64_t)(kb0 + cp_row0) * D + cp_chunk * 8;
#pragma unroll
      for (int i = 0; i < CP_PER_LANE; ++i) {
        cp_async16(ks + cp_dst0 + i * RSTEP * PITCH, Kb + goff + i * RSTEP * D, 16);
        cp_async16(vs + cp_dst0 + i * RSTEP * PITCH, Vb + goff + i * RSTEP * D, 16);
      }
    } else {
#pragma unroll
      for (int i = 0; i < CP_PER_LANE; ++i) {
        const int key = kb0 + cp_row0 + i * RSTEP;
        const bool valid = key < m1 && (L - 1 - key) <= Wmax;
        const int keyc = key < m1 ? key : m1 - 1;
        const int64_t goff = (int64_t)keyc * D + cp_chunk * 8;
        cp_async16(ks + cp_dst0 + i * RSTEP * PITCH, Kb + goff, valid ? 16 : 0);
        cp_async16(vs + cp_dst0 + i * RSTEP * PITCH, Vb + goff, valid ? 16 : 0);
      }
    }
  };

  float oacc[NNT][4];
#pragma unroll
  for (int nt = 0; nt < NNT; ++nt)
#pragma unroll
    for (int e = 0; e < 4; ++e) oacc[nt][e] = 0.f;
  float m_used = -INFINITY, l_part = 0.f;  // row g of this lane; l_part over this lane's key columns
  unsigned long long cnt = 0;
  int r_far = 0;  // first live pair at the far end of the current block (cursor: only moves down as keys advance)
  {
    const int z0 = L - 1 - (m0 + warp * KB);
    while (r_far < H && sW[r_far] < z0) ++r_far;
  }

  // ---- prologue: fill the ring ----
  const int kb_first = m0 + warp * KB;
  const int kb_step = P.nsplit * DEC_WARPS * KB;
#pragma unroll
  for (int s = 0; s < DEC_STAGES - 1; ++s) {
    const int kb0 = kb_first + s * kb_step;
    if (kb0 < m1) issue_block(kb0, s);
    cp_async_commit();
  }

  int it = 0;
  for (int kb0 = kb_first; kb0 < m1; kb0 += kb_step, ++it) {
    cp_async_wait<DEC_STAGES - 2>();
    __syncwarp();
    {
      const int kbn = kb0 + (DEC_STAGES - 1) * kb_step;
      if (kbn < m1) issue_block(kbn, (it + DEC_STAGES - 1) % DEC_STAGES);
      cp_async_commit();
    }
    const uint32_t ks = warp_smem + (it % DEC_STAGES) * DEC_STAGE_SMEM, vs = ks + DEC_TILE_SMEM;
    const bool blk_fast = (kb0 + KB <= m1) && (L - 1 - kb0 <= Wmax);

    // ---- live pair range over the block (coarse mode: first live pair rounded down to 8) ----
    const int z_far = L - 1 - kb0;                      // the block's first key is the farthest
    const int z_near = max(L - 1 - (kb0 + KB - 1), 0);
    while (r_far > 0 && sW[r_far - 1] >= z_far) --r_far;
    int r_near = r_far;
    while (r_near > 0 && sW[r_near - 1] >= z_near) --r_near;
    const int rq_far = MODE == ATF_MODE_COARSE ? (r_far >= H ? H : (r_far & ~7)) : r_far;
    const int rq_near = MODE == ATF_MODE_COARSE ? (r_near & ~7) : r_near;
    const bool uniform = rq_near == rq_far;
    // general blocks (the block straddles a window boundary): first live pair of this lane's key in each group
    int r_lane[NKG];
#pragma unroll
    for (int kg = 0; kg < NKG; ++kg) r_lane[kg] = rq_far;
    if (!uniform) {
#pragma unroll
      for (int kg = 0; kg < NKG; ++kg) {
        const int z = L - 1 - (kb0 + kg * 8 + g);
        int r = r_near;
        while (r < r_far && sW[r] < z) ++r;
        r_lane[kg] = MODE == ATF_MODE_COARSE ? (r >= H ? H : (r & ~7)) : r;
      }
    }
    float sc[NKG][4];
#pragma unroll
    for (int kg = 0; kg < NKG; ++kg)
#pragma unroll
      for (int e = 0; e < 4; ++e) sc[kg][e] = 0.f;

    {
      // ---- S = q K^T ----
      // K steps (16 pairs of one half) below the nearest key's first live pair are dead for every key
      const int jl = rq_near >> 4;
      // element masks of the K step that holds a first live pair r: lane t holds pairs 2t, 2t+1 of the
      // step's first chunk and 8+2t, 9+2t of its second chunk
      auto step_masks = [&](int r, uint32_t& mk0, uint32_t& mk1) {
        const int e = r & 15;
        mk0 = ((2 * t >= e) ? 0x0000FFFFu : 0u) | ((2 * t + 1 >= e) ? 0xFFFF0000u : 0u);
        mk1 = ((8 + 2 * t >= e) ? 0x0000FFFFu : 0u) | ((9 + 2 * t >= e) ? 0xFFFF0000u : 0u);
      };
      uint32_t mku0 = 0xFFFFFFFFu, mku1 = 0xFFFFFFFFu;
      if (uniform) step_masks(rq_far, mku0, mku1);
#pragma unroll
      for (int j = 0; j < NKS; ++j) {
        const int jh = j % (NKS / 2);  // K step within its half
        if (jh < jl) continue;         // warp-uniform
#pragma unroll
        for (int kp = 0; kp < NKG / 2; ++kp) {
          // matrices: (group 2kp, chunk 2j), (group 2kp, chunk 2j+1), (group 2kp+1, chunk 2j), (group 2kp+1, chunk 2j+1)
          uint32_t bf[4];
          ldsm_x4(ks + k_lane_off + kp * 16 * PITCH + j * 32, bf);
          if (uniform) {
            if (jh == (rq_far >> 4)) {
              bf[0] &= mku0;
              bf[1] &= mku1;
              bf[2] &= mku0;
              bf[3] &= mku1;
            }
          } else {
#pragma unroll
            for (int h2 = 0; h2 < 2; ++h2) {
              const int r = r_lane[2 * kp + h2];
              uint32_t mk0 = 0xFFFFFFFFu, mk1 = 0xFFFFFFFFu;
              if (jh < (r >> 4)) {
                mk0 = 0u;
                mk1 = 0u;
              } else if (jh == (r >> 4)) {
                step_masks(r, mk0, mk1);
              }
              bf[2 * h2] &= mk0;
              bf[2 * h2 + 1] &= mk1;
            }
          }
          mma_bf16_16816(sc[2 * kp], qa[j][0], qa[j][1], bf[0], bf[1]);
          mma_bf16_16816(sc[2 * kp + 1], qa[j][0], qa[j][1], bf[2], bf[3]);
        }
      }
    }
    if (COUNT) {
      // one lane per key: lanes t == 0 own key (group, g)
      if (t == 0) {
#pragma unroll
        for (int kg = 0; kg < NKG; ++kg) {
          const int key = kb0 + kg * 8 + g;
          if (key < m1) cnt += (unsigned long long)(H - r_lane[kg]);
        }
      }
    }

    // ---- online softmax (log2 domain); this lane holds keys 2t, 2t+1 of every group for head g ----
    float mx = -INFINITY;
    if (blk_fast) {
#pragma unroll
      for (int kg = 0; kg < NKG; ++kg) {
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          sc[kg][e] *= kScaleLog2;
          mx = fmaxf(mx, sc[kg][e]);
        }
      }
    } else {
#pragma unroll
      for (int kg = 0; kg < NKG; ++kg) {
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int key = kb0 + kg * 8 + 2 * t + e;
          const int z = L - 1 - key;
          sc[kg][e] = (key < m1 && z <= Wmax) ? sc[kg][e] * kScaleLog2 : -INFINITY;
          mx = fmaxf(mx, sc[kg][e]);
        }
      }
    }
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
    float scale_o = 1.f;
    bool moved = false;
    if (mx > m_used + (m_used == -INFINITY ? 0.f : DEC_RESCALE_THRESHOLD)) {
      scale_o = (m_used == -INFINITY) ? 0.f : ex2f(m_used - mx);
      m_used = mx;
      moved = true;
    }
    if (__any_sync(0xffffffffu, moved)) {
      l_part *= scale_o;
#pragma unroll
      for (int nt = 0; nt < NNT; ++nt) {
        oacc[nt][0] *= scale_o;
        oacc[nt][1] *= scale_o;
      }
    }
    const float mref = (m_used == -INFINITY) ? 0.f : m_used;
    uint32_t pa[NKG];
#pragma unroll
    for (int kg = 0; kg < NKG; ++kg) {
      const float p0 = ex2f(sc[kg][0] - mref), p1 = ex2f(sc[kg][1] - mref);
      l_part += p0 + p1;
      pa[kg] = pack_bf16x2(p0, p1);
    }

    // ---- O += P V ----
#pragma unroll
    for (int pk = 0; pk < NKG / 2; ++pk) {
#pragma unroll
      for (int np = 0; np < NNT / 2; ++np) {
        // matrices: (keys 0-7, chunk 2np), (keys 8-15, chunk 2np), (keys 0-7, chunk 2np+1), (keys 8-15, chunk 2np+1)
        uint32_t bf[4];
        ldsm_x4_trans(vs + v_lane_off + pk * 16 * PITCH + np * 32, bf);
        mma_bf16_16816(oacc[2 * np], pa[2 * pk], pa[2 * pk + 1], bf[0], bf[1]);
        mma_bf16_16816(oacc[2 * np + 1], pa[2 * pk], pa[2 * pk + 1], bf[2], bf[3]);
      }
    }
  }
  cp_async_wait<0>();

  // ---- merge the warps of the block (the rings are free now) ----
  l_part += __shfl_xor_sync(0xffffffffu, l_part, 1);
  l_part += __shfl_xor_sync(0xffffffffu, l_part, 2);
  __syncthreads();
  float* sm = reinterpret_cast<float*>(dsm);  // [DEC_WARPS][G][PSTRIDE]
  if (g < G) {
    float* dst = sm + (warp * G + g) * PSTRIDE;
    if (t == 0) {
      dst[0] = m_used;
      dst[1] = l_part;
    }
#pragma unroll
    for (int nt = 0; nt < NNT; ++nt) {
      dst[2 + nt * 8 + 2 * t] = oacc[nt][0];
      dst[2 + nt * 8 + 2 * t + 1] = oacc[nt][1];
    }
  }
  __syncthreads();
  const int64_t grp = (int64_t)b * P.Hkv + hkv;
  float* part = P.partials + (grp * P.nsplit + split) * (int64_t)(G * PSTRIDE);
  for (int idx = threadIdx.x; idx < G * D; idx += DEC_THREADS) {
    const int gg = idx / D, col = idx % D;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < DEC_WARPS; ++w) M = fmaxf(M, sm[(w * G + gg) * PSTRIDE]);
    const float Ms = (M == -INFINITY) ? 0.f : M;
    float acc = 0.f, lacc = 0.f;
#pragma unroll
    for (int w = 0; w < DEC_WARPS; ++w) {
      const float* src = sm + (w * G + gg) * PSTRIDE;
      const float f = ex2f(src[0] - Ms);
      acc += f * src[2 + col];
      lacc += f * src[1];
    }
    part[gg * PSTRIDE + 2 + col] = acc;
    if (col == 0) {
      part[gg * PSTRIDE] = M;
      part[gg * PSTRIDE + 1] = lacc;
    }
  }
  if (COUNT) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, off);
    if (lane == 0 && cnt) {
      for (int gg = 0; gg < G; ++gg) atomicAdd(P.kept + (int64_t)b * P.Hq + hkv * G + gg, cnt);
    }
  }

  // ---- last block of this (batch, KV head) merges all splits ----
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
  for (int gg = warp; gg < G; gg += DEC_WARPS) {
    float M = -INFINITY;
    for (int sp = lane; sp < P.nsplit; sp += 32) M = fmaxf(M, __ldcg(allp + ((int64_t)sp * G + gg) * PSTRIDE));
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, off));
    const float Ms = (M == -INFINITY) ? 0.f : M;
    float Lsum = 0.f;
    for (int sp = lane; sp < P.nsplit; sp += 32) {
      const float* src = allp + ((int64_t)sp * G + gg) * PSTRIDE;
      Lsum += ex2f(__ldcg(src) - Ms) * __ldcg(src + 1);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) Lsum += __shfl_xor_sync(0xffffffffu, Lsum, off);
    const float inv = 1.f / Lsum;
    float acc[D / 32];
#pragma unroll
    for (int c = 0; c < D / 32; ++c) acc[c] = 0.f;
#pragma unroll 8
    for (int sp = 0; sp < P.nsplit; ++sp) {
      const float* src = allp + ((int64_t)sp * G + gg) * PSTRIDE;
      const float f = ex2f(__ldcg(src) - Ms);
#pragma unroll
      for (int c = 0; c < D / 32; ++c) acc[c] = fmaf(f, __ldcg(src + 2 + c * 32 + lane), acc[c]);
    }
    const int64_t hq = (int64_t)b * P.Hq + hkv * G + gg;
#pragma unroll
    for (int c = 0; c < D / 32; ++c) P.O[hq * D + c * 32 + lane] = __float2bfloat16_rn(acc[c] * inv);
    if (P.lse && lane == 0) P.lse[hq] = (Ms + log2f(Lsum)) * 0.6931471805599453f;
  }
  if (threadIdx.x == 0) P.counters[grp] = 0;  // ready for the next launch
}

// ------------------------------------------------------------------------------------------
// Decode on the tiled group-major K cache: bulk copies instead of per-lane 16-byte copies.
//
// A tile is KT keys (16 KiB of K, 16 KiB of V).  In the cache a K tile is [group of 8 pairs, lowest
// frequency first][key][16 elements], so the pairs the tile's nearest key keeps are a contiguous
// prefix of the tile: ONE untiled bulk copy fetches exactly the live bytes.  The two 16-byte
// halves of a key's group entry are stored swapped for keys with bit 2 set, which makes the
// ldmatrix reads of the copied image free of bank conflicts without padding.  The V tile (rows of
// the ordinary cache) comes by TMA with the 128-byte swizzle for the same reason.
// Block = 4 consumer warps (a quarter of the tile each, the arithmetic of the row-layout kernel)
// + 1 producer warp (one thread issues the copies of the next tiles into a 3-stage ring; full and
// empty mbarriers per stage, every wait bounded).
// ------------------------------------------------------------------------------------------
#ifndef ATF_TL_STAGES
#define ATF_TL_STAGES 3
#endif
constexpr int TL_STAGES = ATF_TL_STAGES;
constexpr int TL_THREADS = (DEC_WARPS + 1) * 32;
constexpr int TL_TILE_BYTES = 16384;
constexpr int TL_STAGE_BYTES = 2 * TL_TILE_BYTES;
#ifndef ATF_ROT_BATCH
#define ATF_ROT_BATCH 2
#endif
constexpr int TL_ROT_BYTES = 1024;  // room for one row of the tile-level rotation table (keeps the stages 1 KiB aligned)
constexpr int TL_SMEM = TL_STAGES * TL_STAGE_BYTES + 1024 /* alignment slack */ + 64 /* barriers */;
__device__ __forceinline__ float2 lds_f2(uint32_t addr) {
  float2 v;
  asm volatile("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(addr));
  return v;
}

// One (dim r, dim r + h) pair of an unrotated key, turned by the angle a + b given as (cos, sin) of a and of b
// (App. B: the rotation applied when the cache is read).  fp32, one rounding to bf16.
__device__ __forceinline__ uint32_t rotate_pair(uint32_t v, float2 a, float2 b) {
  const float c = fmaf(a.x, b.x, -a.y * b.y), s = fmaf(a.y, b.x, a.x * b.y);
  const float x = __uint_as_float(v << 16), y = __uint_as_float(v & 0xffff0000u);
  return pack_bf16x2(fmaf(x, c, -y * s), fmaf(y, c, x * s));
}

template <int D, int MODE, bool COUNT, bool ROT>
__global__ void __launch_bounds__(TL_THREADS, ATF_DECODE_SLOTS_GROUPS / 148)
atf_decode_tiles_kernel(const __grid_constant__ CUtensorMap tmV, const __grid_constant__ DecodeParams P,
                        const __grid_constant__ AtfTable table) {
  constexpr int H = D / 2;
  constexpr int KT = TL_TILE_BYTES / (D * 2);  // keys per tile (64 for d = 128, 128 for d = 64)
  constexpr int KB = KT / DEC_WARPS;            // keys per consumer warp and tile
  constexpr int NKG = KB / 8;
  constexpr int NKS = D / 16;                   // groups of 8 pairs = MMA K steps of q K^T
  constexpr int NNT = D / 8;
  constexpr int NVB = D / 64;                   // 64-column boxes of a V tile
  constexpr int PSTRIDE = D + 2;
  constexpr int GBYTES = KT * 32;               // one group of a K tile
  // rotate-at-read: the tile's row of the tile-level (cos, sin) table rides along in the stage
  constexpr int STAGE = TL_STAGE_BYTES + (ROT ? TL_ROT_BYTES : 0);
  const float kScaleLog2 = 1.4426950408889634f / sqrtf((float)D);

  extern __shared__ uint8_t dsm_raw[];
  __shared__ int sW[ATF_MAX_PAIRS];
  __shared__ unsigned int s_last;
  __shared__ int s_abort;
  const uint32_t sbase = (smem_u32(dsm_raw) + 1023u) & ~1023u;
  uint8_t* sgen = dsm_raw + (sbase - smem_u32(dsm_raw));
  const uint32_t bars = sbase + TL_STAGES * STAGE;
  auto full_bar = [&](int st) { return bars + 8u * (uint32_t)st; };
  auto empty_bar = [&](int st) { return bars + 8u * (uint32_t)(TL_STAGES + st); };

  const int split = blockIdx.x, hkv = blockIdx.y, b = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t4 = lane & 3;
  const int G = P.G, L = P.L;
  const int64_t grp = (int64_t)b * P.Hkv + hkv;
  const int ntiles = (L + KT - 1) / KT;
  if (threadIdx.x < H) sW[threadIdx.x] = table.w[threadIdx.x];
  if (threadIdx.x == 0) {
    s_abort = 0;
    for (int st = 0; st < TL_STAGES; ++st) {
      mbar_init(full_bar(st), 1);
      mbar_init(empty_bar(st), DEC_WARPS);
    }
    mbar_fence_init();
    fence_proxy_async_smem();
    tma_prefetch_desc(&tmV);
  }
  __syncthreads();
  const int Wmax = sW[H - 1];
  // the first tile that holds a key some pair reaches; tiles are dealt round-robin to the splits
  const int t_lo = max(0, L - 1 - Wmax) / KT;
  const int t_first = t_lo + split;
  const __nv_bfloat16* Kb = P.K + grp * (int64_t)P.ktiles * KT * D;
  unsigned int fail_site = 0;
  volatile int* abortp = &s_abort;
  auto bounded_wait = [&](uint32_t bar, uint32_t parity) {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_timer_ns();
    for (;;) {
#pragma unroll 1
      for (int i = 0; i < 128; ++i)
        if (mbar_try_wait(bar, parity)) return true;
      if (*abortp) return false;
      if (global_timer_ns() - t0 > ATF_WAIT_LIMIT_NS) {
        *abortp = 1;
        return false;
      }
    }
  };

  float oacc[NNT][4];
#pragma unroll
  for (int nt = 0; nt < NNT; ++nt)
#pragma unroll
    for (int e = 0; e < 4; ++e) oacc[nt][e] = 0.f;
  float m_used = -INFINITY, l_part = 0.f;
  unsigned long long cnt = 0;

  if (warp == DEC_WARPS) {
    // =============================== producer ===============================
    if (lane == 0) {
      int r_near = 0;  // first live pair of the tile's nearest key: only moves down as the tiles advance
      {
        const int z0 = max(L - 1 - (t_first * KT + KT - 1), 0);
        while (r_near < H && sW[r_near] < z0) ++r_near;
      }
      int it = 0;
      for (int t = t_first; t < ntiles; t += P.nsplit, ++it) {
        const int st = it % TL_STAGES;
        if (it >= TL_STAGES && !bounded_wait(empty_bar(st), ((it / TL_STAGES) - 1) & 1)) { fail_site = 40; break; }
        const int z_near = max(L - 1 - (t * KT + KT - 1), 0);
        while (r_near > 0 && sW[r_near - 1] >= z_near) --r_near;
        const int rq = MODE == ATF_MODE_COARSE ? (r_near & ~7) : r_near;
        const int ngl = (H - rq + 7) >> 3;  // live groups of the nearest key: the prefix to fetch
        const uint32_t kdst = sbase + st * STAGE, vdst = kdst + TL_TILE_BYTES;
        mbar_expect_tx(full_bar(st), (uint32_t)(ngl * GBYTES + TL_TILE_BYTES + (ROT ? ngl * 64 : 0)));
        bulk_load_1d(kdst, Kb + (int64_t)t * KT * D, (uint32_t)(ngl * GBYTES), full_bar(st));
        if (ROT) bulk_load_1d(kdst + TL_STAGE_BYTES, P.rot_tile + (int64_t)t * H, (uint32_t)(ngl * 64), full_bar(st));
#pragma unroll
        for (int vb = 0; vb < NVB; ++vb)
          tma_load_3d(vdst + vb * (KT * 128), &tmV, full_bar(st), vb * 64, t * KT, (int)grp);
      }
    }
  } else {
    // =============================== consumers ===============================
    // A fragments of q: K step j contracts the 8 pairs of group j, each pair as (dim r, dim r + h)
    uint32_t qa[NKS][2];
#pragma unroll
    for (int j = 0; j < NKS; ++j) {
      qa[j][0] = 0u;
      qa[j][1] = 0u;
      if (g < G) {
        const uint16_t* q16 = reinterpret_cast<const uint16_t*>(P.q + ((int64_t)b * P.Hq + hkv * G + g) * D);
        const int ra = H - 1 - (8 * j + t4), rb = H - 1 - (8 * j + 4 + t4);
        qa[j][0] = (uint32_t)q16[ra] | ((uint32_t)q16[ra + H] << 16);
        qa[j][1] = (uint32_t)q16[rb] | ((uint32_t)q16[rb + H] << 16);
      }
    }
    const int lm_i = lane >> 3, lm_r = lane & 7;
    // K: matrices (keys 0-7 first half), (keys 0-7 second half), (keys 8-15 first half), (keys 8-15 second half)
    const int kkey = warp * KB + (lm_i >> 1) * 8 + lm_r;  // + 16 * kp
    const uint32_t k_lane_off = (uint32_t)kkey * 32u + (uint32_t)(((lm_i & 1) ^ ((kkey >> 2) & 1)) << 4);
    // V: matrices (keys 0-7, chunk 2np), (keys 8-15, chunk 2np), (keys 0-7, chunk 2np+1), (keys 8-15, chunk 2np+1)
    const int vrow = warp * KB + (lm_i & 1) * 8 + lm_r;  // + 16 * pk
    const uint32_t v_row_off = (uint32_t)vrow * 128u;
    int r_far = 0;
    {
      const int z0 = L - 1 - (t_first * KT + warp * KB);
      while (r_far < H && sW[r_far] < z0) ++r_far;
    }
    int it = 0;
    for (int t = t_first; t < ntiles; t += P.nsplit, ++it) {
      const int st = it % TL_STAGES;
      if (!bounded_wait(full_bar(st), (it / TL_STAGES) & 1)) { fail_site = 41; break; }
      const uint32_t ks = sbase + st * STAGE, vs = ks + TL_TILE_BYTES;
      const int kb0 = t * KT + warp * KB;
      const bool blk_fast = (kb0 + KB <= L) && (L - 1 - kb0 <= Wmax);

      // ---- live pair range over the warp's keys (coarse mode: first live pair rounded down to 8) ----
      const int z_far = L - 1 - kb0;
      const int z_near = max(L - 1 - (kb0 + KB - 1), 0);
      while (r_far > 0 && sW[r_far - 1] >= z_far) --r_far;
      int r_near = r_far;
      while (r_near > 0 && sW[r_near - 1] >= z_near) --r_near;
      const int rq_far = MODE == ATF_MODE_COARSE ? (r_far >= H ? H : (r_far & ~7)) : r_far;
      const int rq_near = MODE == ATF_MODE_COARSE ? (r_near & ~7) : r_near;
      int r_lane[NKG];
#pragma unroll
      for (int kg = 0; kg < NKG; ++kg) r_lane[kg] = rq_far;
      if (rq_near != rq_far) {
#pragma unroll
        for (int kg = 0; kg < NKG; ++kg) {
          const int z = L - 1 - (kb0 + kg * 8 + g);
          int r = r_near;
          while (r < r_far && sW[r] < z) ++r;
          r_lane[kg] = MODE == ATF_MODE_COARSE ? (r >= H ? H : (r & ~7)) : r;
        }
      }
      float sc[NKG][4];
#pragma unroll
      for (int kg = 0; kg < NKG; ++kg)
#pragma unroll
        for (int e = 0; e < 4; ++e) sc[kg][e] = 0.f;

      // ---- S = q K^T: K step j = the 8 pairs of group j; a key with first live pair r keeps its first H - r pairs ----
      const int ngl = (H - rq_near + 7) >> 3;
      // Rotate-at-read works on JB groups per branch, so that the table reads and the rotations of several
      // groups overlap; a group beyond the fetched prefix holds stale bytes, which the masks below zero.
      constexpr int JB = ROT ? ATF_ROT_BATCH : 1;
#pragma unroll
      for (int jb = 0; jb < NKS; jb += JB) {
        if (jb >= ngl) continue;  // warp-uniform
        float2 ak[ROT ? JB : 1][ROT ? NKG / 2 : 1][2][2], at[ROT ? JB : 1][2];
        if (ROT) {
#pragma unroll
          for (int jj = 0; jj < JB; ++jj)
#pragma unroll
            for (int c = 0; c < 2; ++c) {
              const int p = 8 * (jb + jj) + 4 * c + t4;
              at[jj][c] = lds_f2(ks + TL_STAGE_BYTES + p * 8);
#pragma unroll
              for (int kp = 0; kp < NKG / 2; ++kp)
#pragma unroll
                for (int h2 = 0; h2 < 2; ++h2) ak[jj][kp][c][h2] = __ldg(P.rot_key + p * KT + warp * KB + (2 * kp + h2) * 8 + g);
            }
        }
#pragma unroll
        for (int jj = 0; jj < JB; ++jj) {
          const int j = jb + jj;
#pragma unroll
          for (int kp = 0; kp < NKG / 2; ++kp) {
            uint32_t bf[4];
            ldsm_x4(ks + j * GBYTES + kp * 512 + k_lane_off, bf);
            if (ROT) {
              // bf[2 * h2 + c] is pair 8j + 4c + t4 of key (2kp + h2) * 8 + g of the warp's part of the tile
#pragma unroll
              for (int c = 0; c < 2; ++c)
#pragma unroll
                for (int h2 = 0; h2 < 2; ++h2) bf[2 * h2 + c] = rotate_pair(bf[2 * h2 + c], at[jj][c], ak[jj][kp][c][h2]);
            }
#pragma unroll
            for (int h2 = 0; h2 < 2; ++h2) {
              const int live = H - r_lane[2 * kp + h2];
              if (8 * j + t4 >= live) bf[2 * h2] = 0u;
              if (8 * j + 4 + t4 >= live) bf[2 * h2 + 1] = 0u;
            }
            mma_bf16_16816(sc[2 * kp], qa[j][0], qa[j][1], bf[0], bf[1]);
            mma_bf16_16816(sc[2 * kp + 1], qa[j][0], qa[j][1], bf[2], bf[3]);
          }
        }
      }
      if (COUNT && t4 == 0) {
#pragma unroll
        for (int kg = 0; kg < NKG; ++kg)
          if (kb0 + kg * 8 + g < L) cnt += (unsigned long long)(H - r_lane[kg]);
      }

      // ---- online softmax (log2 domain); this lane holds keys 2t, 2t+1 of every group of 8 keys for head g ----
      float mx = -INFINITY;
      if (blk_fast) {
#pragma unroll
        for (int kg = 0; kg < NKG; ++kg)
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            sc[kg][e] *= kScaleLog2;
            mx = fmaxf(mx, sc[kg][e]);
          }
      } else {
#pragma unroll
        for (int kg = 0; kg < NKG; ++kg)
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const int key = kb0 + kg * 8 + 2 * t4 + e;
            sc[kg][e] = (key < L && L - 1 - key <= Wmax) ? sc[kg][e] * kScaleLog2 : -INFINITY;
            mx = fmaxf(mx, sc[kg][e]);
          }
      }
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
      float scale_o = 1.f;
      bool moved = false;
      if (mx > m_used + (m_used == -INFINITY ? 0.f : DEC_RESCALE_THRESHOLD)) {
        scale_o = (m_used == -INFINITY) ? 0.f : ex2f(m_used - mx);
        m_used = mx;
        moved = true;
      }
      if (__any_sync(0xffffffffu, moved)) {
        l_part *= scale_o;
#pragma unroll
        for (int nt = 0; nt < NNT; ++nt) {
          oacc[nt][0] *= scale_o;
          oacc[nt][1] *= scale_o;
        }
      }
      const float mref = (m_used == -INFINITY) ? 0.f : m_used;
      uint32_t pa[NKG];
#pragma unroll
      for (int kg = 0; kg < NKG; ++kg) {
        const float p0 = ex2f(sc[kg][0] - mref), p1 = ex2f(sc[kg][1] - mref);
        l_part += p0 + p1;
        pa[kg] = pack_bf16x2(p0, p1);
      }

      // ---- O += P V (V tile in 128-byte-swizzled 64-column boxes) ----
#pragma unroll
      for (int pk = 0; pk < NKG / 2; ++pk) {
#pragma unroll
        for (int np = 0; np < NNT / 2; ++np) {
          const int chunk = 2 * np + (lm_i >> 1);  // 16-byte column chunk of the row, 0 .. D/8 - 1
          uint32_t bf[4];
          ldsm_x4_trans(vs + (chunk >> 3) * (KT * 128) + pk * 2048 + v_row_off + (((chunk & 7) ^ lm_r) << 4), bf);
          mma_bf16_16816(oacc[2 * np], pa[2 * pk], pa[2 * pk + 1], bf[0], bf[1]);
          mma_bf16_16816(oacc[2 * np + 1], pa[2 * pk], pa[2 * pk + 1], bf[2], bf[3]);
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(empty_bar(st));
    }
  }

  // ---- merge the warps of the block (the ring is free once everybody is here) ----
  l_part += __shfl_xor_sync(0xffffffffu, l_part, 1);
  l_part += __shfl_xor_sync(0xffffffffu, l_part, 2);
  if (fail_site) {
    atomicExch(P.status, 1u);
    atomicExch(P.status + 1, fail_site);
  }
  __syncthreads();
  float* sm = reinterpret_cast<float*>(sgen);  // [DEC_WARPS][G][PSTRIDE]
  if (warp < DEC_WARPS && g < G) {
    float* dst = sm + (warp * G + g) * PSTRIDE;
    if (t4 == 0) {
      dst[0] = m_used;
      dst[1] = l_part;
    }
#pragma unroll
    for (int nt = 0; nt < NNT; ++nt) {
      dst[2 + nt * 8 + 2 * t4] = oacc[nt][0];
      dst[2 + nt * 8 + 2 * t4 + 1] = oacc[nt][1];
    }
  }
  __syncthreads();
  float* part = P.partials + (grp * P.nsplit + split) * (int64_t)(G * PSTRIDE);
  for (int idx = threadIdx.x; idx < G * D; idx += TL_THREADS) {
    const int gg = idx / D, col = idx % D;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < DEC_WARPS; ++w) M = fmaxf(M, sm[(w * G + gg) * PSTRIDE]);
    const float Ms = (M == -INFINITY) ? 0.f : M;
    float acc = 0.f, lacc = 0.f;
#pragma unroll
    for (int w = 0; w < DEC_WARPS; ++w) {
      const float* src = sm + (w * G + gg) * PSTRIDE;
      const float f = ex2f(src[0] - Ms);
      acc += f * src[2 + col];
      lacc += f * src[1];
    }
    part[gg * PSTRIDE + 2 + col] = acc;
    if (col == 0) {
      part[gg * PSTRIDE] = M;
      part[gg * PSTRIDE + 1] = lacc;
    }
  }
  if (COUNT && warp < DEC_WARPS) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, off);
    if (lane == 0 && cnt) {
      for (int gg = 0; gg < G; ++gg) atomicAdd(P.kept + (int64_t)b * P.Hq + hkv * G + gg, cnt);
    }
  }

  // ---- last block of this (batch, KV head) merges all splits ----
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
  for (int gg = warp; gg < G; gg += DEC_WARPS + 1) {
    float M = -INFINITY;
    for (int sp = lane; sp < P.nsplit; sp += 32) M = fmaxf(M, __ldcg(allp + ((int64_t)sp * G + gg) * PSTRIDE));
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, off));
    const float Ms = (M == -INFINITY) ? 0.f : M;
    float Lsum = 0.f;
    for (int sp = lane; sp < P.nsplit; sp += 32) {
      const float* src = allp + ((int64_t)sp * G + gg) * PSTRIDE;
      Lsum += ex2f(__ldcg(src) - Ms) * __ldcg(src + 1);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) Lsum += __shfl_xor_sync(0xffffffffu, Lsum, off);
    const float inv = 1.f / Lsum;
    float acc[D / 32];
#pragma unroll
    for (int c = 0; c < D / 32; ++c) acc[c] = 0.f;
#pragma unroll 8
    for (int sp = 0; sp < P.nsplit; ++sp) {
      const float* src = allp + ((int64_t)sp * G + gg) * PSTRIDE;
      const float f = ex2f(__ldcg(src) - Ms);
#pragma unroll
      for (int c = 0; c < D / 32; ++c) acc[c] = fmaf(f, __ldcg(src + 2 + c * 32 + lane), acc[c]);
    }
    const int64_t hq = (int64_t)b * P.Hq + hkv * G + gg;
#pragma unroll
    for (int c = 0; c < D / 32; ++c) P.O[hq * D + c * 32 + lane] = __float2bfloat16_rn(acc[c] * inv);
    if (P.lse && lane == 0) P.lse[hq] = (Ms + log2f(Lsum)) * 0.6931471805599453f;
  }
  if (threadIdx.x == 0) P.counters[grp] = 0;  // ready for the next launch
}

// K cache rows -> tiled group-major order [slab][tile][group][key in tile][16].  One thread per
// (key, group of 8 pairs): gathers the 16 elements of the group (pair p = 8*group + i is dims
// h-1-p and d-1-p) and writes 32 bytes (the two 16-byte halves swapped for keys with bit 2 set).
__global__ void __launch_bounds__(256)
atf_kcache_pack_kernel(const __nv_bfloat16* __restrict__ K, __nv_bfloat16* __restrict__ Kg, int64_t slabs, int64_t n,
                       int64_t ntiles, int64_t pos0, int D) {
  const int H = D / 2, NG = D / 16;
  const int64_t KT = (int64_t)DEC_WARPS * (DEC_TILE_BYTES / (D * 2));
  const int64_t gid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (gid >= slabs * n * NG) return;
  const int gi = (int)(gid % NG);
  const int64_t m = (gid / NG) % n, sl = gid / (NG * n);
  const __nv_bfloat16* src = K + (sl * n + m) * D;
  __align__(16) __nv_bfloat16 out[16];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int r = H - 1 - (8 * gi + i);
    out[2 * i] = src[r];
    out[2 * i + 1] = src[r + H];
  }
  const int64_t pos = pos0 + m, tile = pos / KT, kin = pos % KT;
  uint4* dst = reinterpret_cast<uint4*>(Kg + (((sl * ntiles + tile) * NG + gi) * KT + kin) * 16);
  const int swap = (int)((kin >> 2) & 1);  // keys with bit 2 set store their two 16-byte halves swapped
  dst[swap] = reinterpret_cast<const uint4*>(out)[0];
  dst[swap ^ 1] = reinterpret_cast<const uint4*>(out)[1];
}

template <int D>
atf_status launch_decode(const DecodeParams& P, const AtfTable& t, int B, int mode, bool count, cudaStream_t s) {
  dim3 grid(P.nsplit, P.Hkv, B);
#define ATF_DEC_LAUNCH(MODE_, COUNT_)                                                                   \
  do {                                                                                                  \
    auto kern = atf_decode_kernel<D, MODE_, COUNT_>;                                                    \
    const int smem = DEC_SMEM_ROWS;                                                                     \
    ATF_CUDA_CHECK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));      \
    ATF_CUDA_CHECK(cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout,           \
                                        cudaSharedmemCarveoutMaxShared));                                \
    kern<<<grid, DEC_THREADS, smem, s>>>(P, t);                                                     \
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
atf_status launch_decode_tiles(const CUtensorMap& tmV, const DecodeParams& P, const AtfTable& t, int B, int mode, bool count,
                               cudaStream_t s) {
  dim3 grid(P.nsplit, P.Hkv, B);
#define ATF_TL_LAUNCH(MODE_, COUNT_)                                                                        \
  do {                                                                                                      \
    auto kern = P.rot_tile ? atf_decode_tiles_kernel<D, MODE_, COUNT_, true>                                \
                           : atf_decode_tiles_kernel<D, MODE_, COUNT_, false>;                              \
    const int smem = TL_SMEM + (P.rot_tile ? TL_STAGES * TL_ROT_BYTES : 0);                                 \
    ATF_CUDA_CHECK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));          \
    ATF_CUDA_CHECK(cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout,               \
                                        cudaSharedmemCarveoutMaxShared));                                    \
    kern<<<grid, TL_THREADS, smem, s>>>(tmV, P, t);                                                           \
  } while (0)
  if (mode == ATF_MODE_EXACT) {
    if (count) ATF_TL_LAUNCH(ATF_MODE_EXACT, true); else ATF_TL_LAUNCH(ATF_MODE_EXACT, false);
  } else {
    if (count) ATF_TL_LAUNCH(ATF_MODE_COARSE, true); else ATF_TL_LAUNCH(ATF_MODE_COARSE, false);
  }
#undef ATF_TL_LAUNCH
  ATF_CUDA_CHECK(cudaGetLastError());
  return ATF_OK;
}

}  // namespace

atf_status atf_validate_table(const char* who, const int64_t* table, int d, int64_t N, AtfTable* out);

static size_t decode_ws_bytes(int B, int Hq, int Hkv, int64_t L, int d) {
  const int ns = std::max(atf_decode_num_splits(B, Hkv, L, ATF_DECODE_SLOTS_ROWS),
                          atf_decode_num_splits(B, Hkv, L, ATF_DECODE_SLOTS_GROUPS));
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
  if (Hq / Hkv > 8) return atf_fail(ATF_ERR_UNSUPPORTED, "atf_decode: Hq/Hkv must be at most 8 (got %d)", Hq / Hkv);
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
  P.G = Hq / Hkv;
  P.L = (int)L;
  const int kl_ = opts ? opts->k_layout : ATF_KLAYOUT_ROWS;
  P.nsplit = atf_decode_num_splits(B, Hkv, L, kl_ == ATF_KLAYOUT_GROUPS ? ATF_DECODE_SLOTS_GROUPS : ATF_DECODE_SLOTS_ROWS);
  const int64_t kt = DEC_WARPS * (DEC_TILE_BYTES / (d * 2));  // keys per tile; tiles go round-robin to the splits
  const int64_t ntiles = (L + kt - 1) / kt;
  if (P.nsplit > ntiles) P.nsplit = (int)ntiles;
  // a group-major cache laid out for more keys than it holds yet (room for the tokens to come)
  const int64_t cap = (opts && opts->kcache_capacity > 0) ? opts->kcache_capacity : L;
  if (cap < L) return atf_fail(ATF_ERR_INVALID_ARG, "atf_decode: kcache_capacity (%lld) is smaller than L", (long long)cap);
  P.ktiles = (int)((cap + kt - 1) / kt);
  P.rot_tile = nullptr;
  P.rot_key = nullptr;
  if (opts && opts->rope_tables) {
    // App. B: the cache holds position-independent (unrotated) keys and the rotation happens at read
    if (kl_ != ATF_KLAYOUT_GROUPS)
      return atf_fail(ATF_ERR_UNSUPPORTED, "atf_decode: rope_tables needs the group-major K cache");
    if ((uintptr_t)opts->rope_tables & 255)
      return atf_fail(ATF_ERR_INVALID_ARG, "atf_decode: rope_tables must be 256-byte aligned");
    const int64_t tcap = opts->rope_tables_capacity;
    if (tcap < L) return atf_fail(ATF_ERR_INVALID_ARG, "atf_decode: rope_tables cover %lld keys, L is %lld", (long long)tcap, (long long)L);
    P.rot_key = (const float2*)opts->rope_tables;
    P.rot_tile = P.rot_key + kt * (d / 2);
  }
  char* base = (char*)ws.ptr;
  P.status = (unsigned int*)base;
  P.counters = (unsigned int*)(base + ATF_WS_STATUS_BYTES);
  P.partials = (float*)(base + ATF_WS_HEADER);
  cudaStream_t s = (cudaStream_t)stream;
  const bool count = P.kept != nullptr;
  const int kl = opts ? opts->k_layout : ATF_KLAYOUT_ROWS;
  if (kl != ATF_KLAYOUT_ROWS && kl != ATF_KLAYOUT_GROUPS) return atf_fail(ATF_ERR_INVALID_ARG, "atf_decode: unknown k_layout %d", kl);
  if (kl == ATF_KLAYOUT_ROWS)
    return d == 64 ? launch_decode<64>(P, t, B, mode, count, s) : launch_decode<128>(P, t, B, mode, count, s);
  // tiled group-major K cache: bulk copies of the live prefix of each K tile, V tiles by TMA
  CUtensorMap tmV;
  if ((st = atf_make_tile_map(&tmV, Vcache, (int64_t)B * Hkv, L, d, L, (int)kt)) != ATF_OK) return st;
  return d == 64 ? launch_decode_tiles<64>(tmV, P, t, B, mode, count, s) : launch_decode_tiles<128>(tmV, P, t, B, mode, count, s);
}

extern "C" int64_t atf_kcache_tile_keys(int d) { return (d == 64 || d == 128) ? DEC_WARPS * (DEC_TILE_BYTES / (d * 2)) : 0; }

extern "C" atf_status atf_kcache_pack(const void* K, void* Kg, int B, int Hkv, int64_t n, int64_t Lcap, int64_t pos0,
                                      int d, void* stream) {
  if (!K || !Kg) return atf_fail(ATF_ERR_INVALID_ARG, "atf_kcache_pack: null pointer");
  if (d != 64 && d != 128) return atf_fail(ATF_ERR_UNSUPPORTED, "atf_kcache_pack: d must be 64 or 128 (got %d)", d);
  if (B < 1 || Hkv < 1 || n < 1 || pos0 < 0 || pos0 + n > Lcap) return atf_fail(ATF_ERR_INVALID_ARG, "atf_kcache_pack: bad shape");
  if (((uintptr_t)K | (uintptr_t)Kg) & 15) return atf_fail(ATF_ERR_INVALID_ARG, "atf_kcache_pack: pointers must be 16-byte aligned");
  const int64_t total = (int64_t)B * Hkv * n * (d / 16);
  const int64_t blocks = (total + 255) / 256;
  if (blocks > 0x7FFFFFFF) return atf_fail(ATF_ERR_UNSUPPORTED, "atf_kcache_pack: too large");
  const int64_t kt = atf_kcache_tile_keys(d);
  atf_kcache_pack_kernel<<<(unsigned)blocks, 256, 0, (cudaStream_t)stream>>>(
      (const __nv_bfloat16*)K, (__nv_bfloat16*)Kg, (int64_t)B * Hkv, n, (Lcap + kt - 1) / kt, pos0, d);
  ATF_CUDA_CHECK(cudaGetLastError());
  return ATF_OK;
}

// ------------------------------------------------------------------------------------------
// Rotation tables for the decode on an unrotated K cache (App. B).  The angle of key m in pair r is
// (pos0 + m) * theta_r = (pos0 + tile * KT) * theta_r + (m mod KT) * theta_r, so two small tables of
// (cos, sin) - one row per tile, one row per key of a tile - give every angle by one angle addition.
// Entries are computed in fp64 and stored in fp32; pairs are counted from the lowest frequency, like
// the groups of the cache.  Layout: [pair][key in tile] then [tile][pair].
// ------------------------------------------------------------------------------------------
struct RotTheta {
  double t[ATF_MAX_PAIRS];
};
__global__ void atf_rope_tables_kernel(const __grid_constant__ RotTheta th, long long pos0, int KT, int H, int64_t ntiles,
                                       float2* __restrict__ out) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t nkey = (int64_t)KT * H;
  if (i >= nkey + ntiles * H) return;
  int p;
  double pos;
  if (i < nkey) {
    p = (int)(i / KT);
    pos = (double)(i % KT);
  } else {
    const int64_t k = i - nkey;
    p = (int)(k % H);
    pos = (double)(pos0 + (k / H) * KT);
  }
  double sn, cs;
  sincos(pos * th.t[H - 1 - p], &sn, &cs);
  out[i] = make_float2((float)cs, (float)sn);
}

extern "C" size_t atf_rope_tables_bytes(int d, int64_t capacity) {
  if ((d != 64 && d != 128) || capacity < 1) return 0;
  const int64_t kt = atf_kcache_tile_keys(d);
  return (size_t)(kt + (capacity + kt - 1) / kt) * (d / 2) * sizeof(float2);
}

extern "C" atf_status atf_rope_tables(const double* theta, int d, int64_t pos0, int64_t capacity, void* tables,
                                      size_t bytes, void* stream) {
  if (!theta || !tables) return atf_fail(ATF_ERR_INVALID_ARG, "atf_rope_tables: null pointer");
  if (d != 64 && d != 128) return atf_fail(ATF_ERR_UNSUPPORTED, "atf_rope_tables: d must be 64 or 128 (got %d)", d);
  if (capacity < 1 || pos0 < 0 || pos0 + capacity >= (1ll << 40)) return atf_fail(ATF_ERR_INVALID_ARG, "atf_rope_tables: bad range");
  if ((uintptr_t)tables & 255) return atf_fail(ATF_ERR_INVALID_ARG, "atf_rope_tables: tables must be 256-byte aligned");
  const size_t need = atf_rope_tables_bytes(d, capacity);
  if (bytes < need) return atf_fail(ATF_ERR_WORKSPACE, "atf_rope_tables: buffer has %zu bytes, needs %zu", bytes, need);
  RotTheta th;
  for (int r = 0; r < d / 2; ++r) {
    if (!(theta[r] > 0.0) || !std::isfinite(theta[r])) return atf_fail(ATF_ERR_INVALID_ARG, "atf_rope_tables: theta[%d] must be positive and finite", r);
    th.t[r] = theta[r];
  }
  const int64_t kt = atf_kcache_tile_keys(d);
  const int64_t ntiles = (capacity + kt - 1) / kt;
  const int64_t total = (kt + ntiles) * (d / 2);
  atf_rope_tables_kernel<<<(unsigned)((total + 255) / 256), 256, 0, (cudaStream_t)stream>>>(th, (long long)pos0, (int)kt, d / 2,
                                                                                              ntiles, (float2*)tables);
  ATF_CUDA_CHECK(cudaGetLastError());
  return ATF_OK;
}

extern "C" atf_status atf_decode(const void* q, const void* Kcache, const void* Vcache, void* O, int B, int Hq,
                                 int Hkv, int64_t L, int d, const int64_t* table, void* stream) {
  return atf_decode_ex(q, Kcache, Vcache, O, B, Hq, Hkv, L, d, table, nullptr, stream);
}

// ------------------------------------------------------------------------------------------
// atf_decode_static: the same decode step for callers that may not allocate device memory.
//
// Some hosts cannot hand this library a workspace: a plug-in that runs inside another
// runtime's callback (an inference server's custom op, a host that has locked its device
// allocator after start-up, a process pinned to a fixed memory budget) may neither call
// cudaMalloc - it synchronises the device and can fail or deadlock under the host's memory
// manager - nor own a buffer of its own.  For them the split-K scratch of the decode kernel
// (the per-split partial results and the per-(batch, KV head) split counters) lives in the
// array below, which is part of the library image: every GPU that loads the library holds
// these ATF_STATIC_SCRATCH_BYTES bytes until the process exits.
//
// In host code the array's name is only a host-side stand-in for the device object, not a
// device address.  The address is obtained once per device, with that device current, from
// cudaGetSymbolAddress, and that pointer is what the kernel gets.
// ------------------------------------------------------------------------------------------
constexpr size_t ATF_STATIC_SCRATCH_BYTES = ATF_WS_HEADER + (size_t)2 * 1024 * 1024;
static __device__ __align__(256) unsigned char g_atf_static_scratch[ATF_STATIC_SCRATCH_BYTES];

constexpr int ATF_MAX_DEVICES = 64;
static void* g_static_scratch_ptr[ATF_MAX_DEVICES] = {nullptr};

extern "C" size_t atf_decode_static_capacity(void) { return ATF_STATIC_SCRATCH_BYTES; }

extern "C" atf_status atf_decode_static(const void* q, const void* Kcache, const void* Vcache, void* O, int B, int Hq,
                                        int Hkv, int64_t L, int d, const int64_t* table, void* stream) {
  if (B < 1 || Hq < 1 || Hkv < 1 || L < 1 || (d != 64 && d != 128) || Hq % Hkv)
    return atf_fail(ATF_ERR_INVALID_ARG, "atf_decode_static: bad shape");
  if ((int64_t)B * Hkv > ATF_WS_COUNTER_SLOTS) return atf_fail(ATF_ERR_UNSUPPORTED, "atf_decode_static: B*Hkv must be <= %d", ATF_WS_COUNTER_SLOTS);
  const size_t need = decode_ws_bytes(B, Hq, Hkv, L, d);
  if (need > ATF_STATIC_SCRATCH_BYTES)
    return atf_fail(ATF_ERR_WORKSPACE,
                    "atf_decode_static: this problem needs %zu bytes of scratch, the built-in array holds %zu; "
                    "use atf_decode with a bound workspace", need, ATF_STATIC_SCRATCH_BYTES);
  int dev = -1;
  ATF_CUDA_CHECK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= ATF_MAX_DEVICES) return atf_fail(ATF_ERR_UNSUPPORTED, "atf_decode_static: device index %d out of range", dev);
  if (!g_static_scratch_ptr[dev]) {
    // set-up, once per device, with that device current
    void* p = nullptr;
    ATF_CUDA_CHECK(cudaGetSymbolAddress(&p, g_atf_static_scratch));
    if (!p) return atf_fail(ATF_ERR_CUDA, "atf_decode_static: cudaGetSymbolAddress returned a null address");
    g_static_scratch_ptr[dev] = p;
    atf_register_status_words(dev, p);
  }
  void* scratch = g_static_scratch_ptr[dev];
  // The array keeps whatever the last call left.  The split counters must start at zero (the kernel
  // leaves them so, but a launch that gave up may not have): a memset on the stream, not an
  // allocation.  The partials are overwritten; the status words are left alone, so that a give-up of
  // an earlier launch is still there for atf_check_status.
  ATF_CUDA_CHECK(cudaMemsetAsync((char*)scratch + ATF_WS_STATUS_BYTES, 0, (size_t)B * Hkv * sizeof(unsigned int),
                                 (cudaStream_t)stream));
  atf_opts o;
  memset(&o, 0, sizeof(o));
  o.mode = ATF_MODE_EXACT;
  o.workspace = scratch;
  o.workspace_bytes = ATF_STATIC_SCRATCH_BYTES;
  o.k_layout = ATF_KLAYOUT_ROWS;
  return atf_decode_ex(q, Kcache, Vcache, O, B, Hq, Hkv, L, d, table, &o, stream);
}
