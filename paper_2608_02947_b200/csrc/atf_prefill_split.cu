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
// only (the lo x lo product, 2^-16 of the result, is left out).  V, P and O are as in atf_prefill
// (bf16 operands, fp32 accumulation); every exponential is MUFU ex2 (no polynomial), the row sum
// is taken from the unrounded fp32 values.
//
// The four Q/K operands of two query tiles do not fit shared memory, so one CTA owns ONE 128-row
// query tile of one head (d = 128: Q_hi, Q_lo 64 KiB; two K stages of hi + lo 128 KiB; one V
// stage 32 KiB).  Tensor memory then has room for two S buffers and two P buffers beside O, and
// the pipeline needs no alternation of tiles: the issuer writes S(t + 1) while the softmax warps
// work on S(t), and O += P(t) V follows when P(t) is stored.
//   warp 0      TMA producer (Q once; K hi/lo, live 64-column blocks only; V)
//   warp 1      MMA issuer (one thread)
//   warps 4-7   softmax, one query row per thread: read S, finish the window rule per cell,
//               mask, online softmax with lazy rescaling of O, write P (bf16) to tensor memory
// Exact mode, per quarter of the query rows (one softmax warp) as in atf_prefill: pairs live in every
// cell of the quarter's 32 x 128 cells need nothing; a pair live in most of them stays in the MMA
// and its three products are taken back out of the cells beyond its window on the CUDA cores; a
// pair live in a minority is zeroed in the quarter's rows of the CTA's copies of Q_hi and Q_lo and
// added where it is live (pairs only die as the distance grows and the tiles are walked outwards
// from the diagonal, so the zeroing is monotone).  The MMA depth of a tile is what the nearest
// quarter keeps, rounded up to a 16-column step.  Coarse mode: depth = pairs live anywhere in the
// tile rounded up to 8, every pair on the diagonal tile, no per-cell work.  Term counts are those
// of atf_prefill, bit for bit.
// Every wait is bounded and reports through the workspace status words.
#include <cuda.h>

#include <algorithm>

#include "atf_common.cuh"

namespace {

constexpr int T = 128;              // query rows per tile and keys per tile
constexpr int BLK_BYTES = T * 128;  // one [128 x 64] bf16 block, 128-byte rows
constexpr int SP_THREADS = 256;
constexpr float RESCALE_THRESHOLD = 8.f;  // log2 units the reference maximum may lag behind

struct SplitParams {
  const __nv_bfloat16* Qhi;  // pair-interleaved hi / lo parts of Q, [B*Hq, N, D]
  const __nv_bfloat16* Qlo;
  __nv_bfloat16* O;
  float* LSE;
  unsigned long long* kept;
  unsigned int* status;
  int Hq, Hkv, N;
};

template <int D>
struct SplitSmem {
  static constexpr int NB = D / 64;
  static constexpr int TILE = NB * BLK_BYTES;
  static constexpr int QHI_OFF = 0;
  static constexpr int QLO_OFF = TILE;
  static constexpr int K_OFF = 2 * TILE;  // stage s: hi at K_OFF + 2 s TILE, lo one TILE further
  static constexpr int V_OFF = K_OFF + 4 * TILE;
  static constexpr int BAR_OFF = V_OFF + TILE;
  static constexpr int TOTAL = BAR_OFF + 256;
  static constexpr int DYN_BYTES = TOTAL + 1024;  // slack for 1024-byte alignment
};
// barrier slots (8 bytes each); [2] = one per S / P buffer or K stage
enum { S_QFULL = 0, S_KFULL = 1, S_KEMPTY = 3, S_VFULL = 5, S_VEMPTY = 6, S_SFULL = 7, S_SREAD = 9, S_PFULL = 11,
       S_PVDONE = 13, S_OFULL = 15, S_QZ = 16, S_COUNT = 17 };

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

__device__ __forceinline__ float ex2_mufu(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Bounded wait that also gives up as soon as another role of the CTA has given up.
__device__ __forceinline__ bool wait_or_abort(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_timer_ns();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 128; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (global_timer_ns() - t0 > ATF_WAIT_LIMIT_NS) {
      *abort_flag = 1;
      return false;
    }
  }
}

template <int D, int MODE, bool COUNT>
__global__ void __launch_bounds__(SP_THREADS, 1)
atf_prefill_split_kernel(const __grid_constant__ CUtensorMap tmQhi, const __grid_constant__ CUtensorMap tmQlo,
                         const __grid_constant__ CUtensorMap tmKhi, const __grid_constant__ CUtensorMap tmKlo,
                         const __grid_constant__ CUtensorMap tmV, const __grid_constant__ SplitParams P,
                         const __grid_constant__ AtfTable table) {
  using SM = SplitSmem<D>;
  constexpr int H = D / 2;
  constexpr int NB = D / 64;
  constexpr uint32_t TMEM_COLS = 512;  // S0, S1 (128 each) | O (D) at 256 | P0, P1 (64 each) at 384
  constexpr uint32_t IDESC_QK = make_idesc_bf16(128, T, 0, 0);
  constexpr uint32_t IDESC_PV = make_idesc_bf16(128, D, 0, 1);
  const float kScaleLog2 = 1.4426950408889634f / sqrtf((float)D);

  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t sQhi = smem_base + SM::QHI_OFF, sQlo = smem_base + SM::QLO_OFF, sK = smem_base + SM::K_OFF,
                 sV = smem_base + SM::V_OFF;
  const uint32_t bars = smem_base + SM::BAR_OFF;
  auto bar = [&](int slot) { return bars + 8u * (uint32_t)slot; };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_gen + SM::BAR_OFF + 8 * S_COUNT);
  __shared__ int sW[ATF_MAX_PAIRS];
  __shared__ int s_abort;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int ntq = (P.N + T - 1) / T;
  const int it = ntq - 1 - (int)blockIdx.x;  // longest rows first
  const int hq = blockIdx.y, b = blockIdx.z;
  const int bhq = b * P.Hq + hq;
  const int bhk = b * P.Hkv + hq / (P.Hq / P.Hkv);

  if (tid < H) sW[tid] = table.w[tid];
  if (tid == 0) {
    s_abort = 0;
    mbar_init(bar(S_QFULL), 1);
    mbar_init(bar(S_VFULL), 1);
    mbar_init(bar(S_VEMPTY), 1);
    mbar_init(bar(S_OFULL), 1);
    mbar_init(bar(S_QZ), 4);
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar(S_KFULL + i), 1);
      mbar_init(bar(S_KEMPTY + i), 4);  // one arrival per softmax warp, at the end of its step on the tile
      mbar_init(bar(S_SFULL + i), 1);
      mbar_init(bar(S_SREAD + i), 4);
      mbar_init(bar(S_PFULL + i), 4);
      mbar_init(bar(S_PVDONE + i), 1);
    }
    mbar_fence_init();
    fence_proxy_async_smem();
    tma_prefetch_desc(&tmQhi);
    tma_prefetch_desc(&tmQlo);
    tma_prefetch_desc(&tmKhi);
    tma_prefetch_desc(&tmKlo);
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
  const int Wmax = sW[H - 1];
  const int dlim = (Wmax + T - 1) / T + 1;  // first tile distance no pair reaches
  const int nt = min(it + 1, dlim);         // key tiles it, it - 1, ... walked outwards from the diagonal
  volatile int* abortp = &s_abort;
  unsigned int fail_site = 0;

  // Pairs (counted from the low-frequency end) whose window reaches distance z.  Every role asks for
  // non-decreasing distances, so each question keeps its own cursor r into the non-decreasing table.
  auto pairs_reaching = [&](int& r, int z) {
    while (r < H && sW[r] < z) ++r;
    return H - r;
  };
  // For the 32 rows of quarter wq against the 128 keys of the tile at tile distance dt: the smallest distance,
  // the distance from the quarter's middle row to the tile's middle column, the largest distance
  auto z_any = [](int dt, int wq) { return dt == 0 ? 0 : dt * T + 32 * wq - (T - 1); };
  auto z_mid = [](int dt, int wq) { return dt == 0 ? 16 * wq + 15 : dt * T + 32 * wq - 48; };
  auto z_all = [](int dt, int wq) { return dt * T + 32 * wq + 31; };
  // 16-column MMA steps of the S product of a tile: what the nearest quarter keeps in the MMA (exact: pairs live
  // in most of its cells), the pairs live anywhere in the tile rounded up to 8 and everything on the diagonal (coarse)
  auto natoms_of = [&](int& r, int dt) {
    if (MODE == ATF_MODE_EXACT) return (pairs_reaching(r, z_mid(dt, 0)) + 7) / 8;
    return dt == 0 ? H / 8 : (pairs_reaching(r, z_any(dt, 0)) + 7) / 8;
  };
  if (warp == 0) {
    // =============================== TMA producer ===============================
    if (lane == 0) {
      mbar_expect_tx(bar(S_QFULL), 2 * SM::TILE);
      for (int kb = 0; kb < NB; ++kb) {
        tma_load_3d(sQhi + kb * BLK_BYTES, &tmQhi, bar(S_QFULL), kb * 64, it * T, bhq);
        tma_load_3d(sQlo + kb * BLK_BYTES, &tmQlo, bar(S_QFULL), kb * 64, it * T, bhq);
      }
      int r_k = 0;
      auto load_k = [&](int t) {
        const int ks = t & 1;
        if (!wait_or_abort(bar(S_KEMPTY + ks), ((t >> 1) & 1) ^ 1, abortp)) return false;
        // 64-column K blocks to load: exact mode also reads the pairs it adds per cell
        const int cols = MODE == ATF_MODE_EXACT ? 2 * pairs_reaching(r_k, z_any(t, 0)) : 16 * natoms_of(r_k, t);
        const int nkb = max(1, (cols + 63) / 64);
        mbar_expect_tx(bar(S_KFULL + ks), 2 * nkb * BLK_BYTES);
        for (int kb = 0; kb < nkb; ++kb) {
          tma_load_3d(sK + (2 * ks) * SM::TILE + kb * BLK_BYTES, &tmKhi, bar(S_KFULL + ks), kb * 64, (it - t) * T, bhk);
          tma_load_3d(sK + (2 * ks + 1) * SM::TILE + kb * BLK_BYTES, &tmKlo, bar(S_KFULL + ks), kb * 64, (it - t) * T, bhk);
        }
        return true;
      };
      bool ok = load_k(0);
      if (!ok) fail_site = 50;
      for (int t = 0; t < nt && ok; ++t) {
        if (t + 1 < nt && !load_k(t + 1)) { fail_site = 50; break; }
        if (!wait_or_abort(bar(S_VEMPTY), (t & 1) ^ 1, abortp)) { fail_site = 51; break; }
        mbar_expect_tx(bar(S_VFULL), SM::TILE);
        for (int kb = 0; kb < NB; ++kb)
          tma_load_3d(sV + kb * BLK_BYTES, &tmV, bar(S_VFULL), kb * 64, (it - t) * T, bhk);
      }
    }
  } else if (warp == 1) {
    // =============================== MMA issuer ===============================
    if (lane == 0) {
      // K-major operands advance 32 bytes per 16-column step inside a 64-column block and one block
      // per four steps (descriptor start-address units of 16 bytes); V advances 16 key rows.
      const uint64_t dQhi = make_smem_desc_sw128(sQhi, 16, 1024), dQlo = make_smem_desc_sw128(sQlo, 16, 1024);
      const uint64_t dV = make_smem_desc_sw128(sV, BLK_BYTES, 1024);
      auto pv = [&](int u) {
        if (!wait_or_abort(bar(S_PFULL + (u & 1)), (u >> 1) & 1, abortp)) return false;
        if (!wait_or_abort(bar(S_VFULL), u & 1, abortp)) return false;
        tc_fence_after();
        const uint32_t tO = tmem_base + 2 * T, tP = tmem_base + 3 * T + (u & 1) * 64;
#pragma unroll
        for (int i = 0; i < T / 16; ++i)
          tc_mma_ts(tO, tP + 8 * i, dV + (uint64_t)(128 * i), IDESC_PV, (u > 0 || i > 0) ? 1u : 0u);
        tc_commit(bar(S_VEMPTY));
        tc_commit(bar(S_PVDONE + (u & 1)));
        return true;
      };
      bool ok = wait_or_abort(bar(S_QFULL), 0, abortp);
      if (!ok) fail_site = 60;
      int r_n = 0;
      for (int t = 0; t < nt && ok; ++t) {
        const int sb = t & 1;
        const int natoms = natoms_of(r_n, t);
        ok = wait_or_abort(bar(S_KFULL + sb), (t >> 1) & 1, abortp);
        // the softmax warps hold S(t - 2) in registers: its buffer may be written again
        if (ok && t >= 2) ok = wait_or_abort(bar(S_SREAD + sb), ((t >> 1) - 1) & 1, abortp);
        // exact mode: the pairs that are live nowhere in this tile have been zeroed in Q
        if (ok && MODE == ATF_MODE_EXACT) ok = wait_or_abort(bar(S_QZ), t & 1, abortp);
        if (!ok) { fail_site = 61; break; }
        tc_fence_after();
        const uint64_t dKhi = make_smem_desc_sw128(sK + (2 * sb) * SM::TILE, 16, 1024),
                       dKlo = make_smem_desc_sw128(sK + (2 * sb + 1) * SM::TILE, 16, 1024);
        const uint32_t tS = tmem_base + sb * T;
        for (int a = 0; a < natoms; ++a) {
          const uint64_t off = (uint64_t)((a & 3) * 2 + (a >> 2) * (BLK_BYTES / 16));
          tc_mma_ss(tS, dQhi + off, dKhi + off, IDESC_QK, a > 0 ? 1u : 0u);
          tc_mma_ss(tS, dQhi + off, dKlo + off, IDESC_QK, 1u);
          tc_mma_ss(tS, dQlo + off, dKhi + off, IDESC_QK, 1u);
        }
        tc_commit(bar(S_SFULL + sb));
        if (t >= 1 && !pv(t - 1)) { ok = false; fail_site = 62; break; }
      }
      if (ok && nt > 0) {
        if (!pv(nt - 1)) {
          fail_site = 63;
        } else {
          tc_commit(bar(S_OFULL));
        }
      }
    }
  } else if (warp >= 4) {
    // =============================== softmax ===============================
    const int row = tid - 128;
    const int n = it * T + row;
    const bool row_ok = n < P.N;
    const int64_t qrow = (int64_t)bhq * P.N + (row_ok ? n : P.N - 1);  // row of Q, O and LSE
    const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t tO = tmem_base + 2 * T + lane_off;
    const __nv_bfloat16* qhi_src = P.Qhi + qrow * D;
    const __nv_bfloat16* qlo_src = P.Qlo + qrow * D;

    const int wq = warp & 3;
    bool ok = true;
    int zeroed_from = H;  // pairs p >= zeroed_from are zero in this row of the shared copies of Q
    auto zero_q_down_to = [&](int p_keep) {
      for (int p = p_keep; p < zeroed_from; ++p) {
        const int col = 2 * p;
        const uint32_t off = (col >> 6) * BLK_BYTES + sw128_offset(row, (col & 63) >> 3) + (col & 7) * 2;
        *reinterpret_cast<uint32_t*>(smem_gen + SM::QHI_OFF + off) = 0u;
        *reinterpret_cast<uint32_t*>(smem_gen + SM::QLO_OFF + off) = 0u;
      }
      zeroed_from = min(zeroed_from, p_keep);
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(S_QZ));
    };
    int r_any = 0, r_mid = 0, r_all = 0, r_n = 0;
    int p_mid = pairs_reaching(r_mid, z_mid(0, wq));  // of the step at hand; the next one's is taken a step ahead
    if (MODE == ATF_MODE_EXACT) {
      ok = wait_or_abort(bar(S_QFULL), 0, abortp);
      if (!ok) fail_site = 70;
      if (ok) zero_q_down_to(p_mid);
    }
    float m_used = -INFINITY, l_run = 0.f;  // m_used in raw score units
    unsigned long long cnt = 0;

    for (int t = 0; t < nt && ok; ++t) {
      const int sb = t & 1;
      const int dt = t;
      const int p_any = pairs_reaching(r_any, z_any(dt, wq)), p_all = pairs_reaching(r_all, z_all(dt, wq));
      const int natoms = natoms_of(r_n, dt);
      const int p_mid_next = t + 1 < nt ? pairs_reaching(r_mid, z_mid(dt + 1, wq)) : 0;
      const int zrow = dt * T + row;  // distance from this row to column 0 of the key tile
      const uint32_t tS = tmem_base + sb * T + lane_off;
      const uint32_t tP = tmem_base + 3 * T + sb * 64 + lane_off;
      if (!wait_or_abort(bar(S_SFULL + sb), (t >> 1) & 1, abortp)) { ok = false; fail_site = 71; break; }
      tc_fence_after();
      // S(t) is complete, so Q is not being read: zero what the quarter does not keep in the MMA of the next tile
      if (MODE == ATF_MODE_EXACT && t + 1 < nt) zero_q_down_to(p_mid_next);
      float s[T];
      if (natoms > 0) {
#pragma unroll
        for (int q4 = 0; q4 < T / 32; ++q4) tc_ld32(tS + q4 * 32, reinterpret_cast<uint32_t*>(s) + q4 * 32);
        tc_wait_ld();
      } else {  // no pair is kept in the MMA of this tile: nothing was written, every live term is added below
#pragma unroll
        for (int c = 0; c < T; ++c) s[c] = 0.f;
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(S_SREAD + sb));

      // ---- straddling pairs.  Pairs [p_all, p_mid) went through the MMA: take their three products back
      //      out of the cells beyond the pair's window.  Pairs [p_mid, p_any) did not (zero in Q): add them in
      //      the cells inside the window.  32 columns at a time, skipping what no row of the warp needs. ----
      if (MODE == ATF_MODE_EXACT && p_all < p_any) {
        if (!wait_or_abort(bar(S_KFULL + sb), (t >> 1) & 1, abortp)) { ok = false; fail_site = 72; break; }
        const int zw_lo = dt * T + wq * 32, zw_hi = zw_lo + 31;  // zrow over the warp's rows
        for (int p = p_all; p < p_any; ++p) {
          const int wp = sW[H - 1 - p];
          const bool subtract = p < p_mid;
          // distances of the warp's cells in the chunk of columns 32 q4 .. 32 q4 + 31: [zw_lo - 32 q4 - 31, zw_hi - 32 q4]
          bool touched[T / 32];
          bool any = false;
#pragma unroll
          for (int q4 = 0; q4 < T / 32; ++q4) {
            const int hi = zw_hi - 32 * q4, lo = zw_lo - 32 * q4 - 31;
            touched[q4] = subtract ? (hi > wp) : (lo <= wp && hi >= 0);
            any |= touched[q4];
          }
          if (!any) continue;
          const uint32_t qh = *reinterpret_cast<const uint32_t*>(qhi_src + 2 * p);
          const uint32_t ql = *reinterpret_cast<const uint32_t*>(qlo_src + 2 * p);
          float qh0 = bf16lo_to_f32(qh), qh1 = bf16hi_to_f32(qh);
          float qs0 = qh0 + bf16lo_to_f32(ql), qs1 = qh1 + bf16hi_to_f32(ql);  // exact: 16 significant bits
          if (subtract) {
            qh0 = -qh0; qh1 = -qh1; qs0 = -qs0; qs1 = -qs1;
          }
          const int col = 2 * p;
          const uint32_t khi = sK + (2 * sb) * SM::TILE + (col >> 6) * BLK_BYTES + (col & 7) * 2;
          const int chunk = (col & 63) >> 3;
          // cells with column >= jb = zrow - w are inside the window: adding uses sat(c - jb + 1), taking back sat(jb - c)
          const float jbf = (float)(zrow - wp);
          const float ca = subtract ? -1.f : 1.f, cb = subtract ? jbf : 1.f - jbf;
#pragma unroll
          for (int q4 = 0; q4 < T / 32; ++q4) {
            if (touched[q4]) {  // warp-uniform
              uint32_t kh[32], kl[32];
#pragma unroll
              for (int cc = 0; cc < 32; ++cc) {
                const int c = 32 * q4 + cc;
                const uint32_t a = khi + ((chunk ^ (c & 7)) << 4) + c * 128;
                asm volatile("ld.shared.b32 %0, [%1];" : "=r"(kh[cc]) : "r"(a));
                asm volatile("ld.shared.b32 %0, [%1];" : "=r"(kl[cc]) : "r"(a + SM::TILE));
              }
#pragma unroll
              for (int cc = 0; cc < 32; ++cc) {
                const int c = 32 * q4 + cc;
                float term = qs0 * bf16lo_to_f32(kh[cc]);
                term = fmaf(qs1, bf16hi_to_f32(kh[cc]), term);
                term = fmaf(qh0, bf16lo_to_f32(kl[cc]), term);
                term = fmaf(qh1, bf16hi_to_f32(kl[cc]), term);
                const float coef = __saturatef(fmaf(ca, (float)c, cb));
                s[c] = fmaf(term, coef, s[c]);
              }
            }
          }
        }
      }
      // ---- causal mask on the diagonal tile, dropped keys (exact mode: no pair reaches the cell) ----
      if (dt == 0 || (MODE == ATF_MODE_EXACT && dt * T + T - 1 > Wmax)) {
        const int zdrop = MODE == ATF_MODE_EXACT ? Wmax : 0x7FFFFFFF;
#pragma unroll
        for (int c = 0; c < T; ++c) {
          const int z = zrow - c;
          s[c] = (z >= 0 && z <= zdrop) ? s[c] : -INFINITY;
        }
      }
      if (COUNT && row_ok) {
        const int ncols = dt == 0 ? row + 1 : T;
        if (MODE == ATF_MODE_EXACT) {
          cnt += (unsigned long long)p_all * (unsigned long long)ncols;
          for (int p = p_all; p < p_any; ++p) {
            const int wp = sW[H - 1 - p];
            const int lo = max(0, zrow - wp), hi = min(T - 1, zrow);
            cnt += (unsigned long long)max(0, hi - lo + 1);
          }
        } else {
          cnt += (unsigned long long)min(H, 8 * natoms) * (unsigned long long)ncols;
        }
      }
      // ---- online softmax, lazy rescaling ----
      float mx = -INFINITY;
#pragma unroll
      for (int c = 0; c < T; ++c) mx = fmaxf(mx, s[c]);
      float scale_o = 1.f;
      bool moved = false;
      if (mx > m_used && (m_used == -INFINITY || (mx - m_used) * kScaleLog2 > RESCALE_THRESHOLD)) {
        scale_o = m_used == -INFINITY ? 0.f : ex2_mufu((m_used - mx) * kScaleLog2);
        m_used = mx;
        moved = t > 0;  // nothing has been accumulated before the first tile
      }
      if (__any_sync(0xffffffffu, moved)) {
        // every product into O issued so far must be complete: O += P(t - 1) V is the last of them
        if (!wait_or_abort(bar(S_PVDONE + ((t - 1) & 1)), ((t - 1) >> 1) & 1, abortp)) { ok = false; fail_site = 73; break; }
        tc_fence_after();
#pragma unroll
        for (int q4 = 0; q4 < D / 32; ++q4) {
          uint32_t o[32];
          tc_ld32(tO + q4 * 32, o);
          tc_wait_ld();
#pragma unroll
          for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * scale_o);
          tc_st32(tO + q4 * 32, o);
        }
        tc_wait_st();
      }
      // the product that read the previous contents of this P buffer must be complete
      if (t >= 2 && !wait_or_abort(bar(S_PVDONE + sb), ((t - 2) >> 1) & 1, abortp)) { ok = false; fail_site = 74; break; }
      const float neg_m = m_used == -INFINITY ? 0.f : -m_used * kScaleLog2;
      float lsum = 0.f;
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
        uint32_t pk[32];
        float a0 = 0.f, a1 = 0.f;
#pragma unroll
        for (int c = 0; c < 64; c += 2) {
          const float e0 = ex2_mufu(fmaf(s[64 * hf + c], kScaleLog2, neg_m));
          const float e1 = ex2_mufu(fmaf(s[64 * hf + c + 1], kScaleLog2, neg_m));
          a0 += e0;
          a1 += e1;
          pk[c >> 1] = pack_bf16x2(e0, e1);
        }
        lsum += a0 + a1;
        tc_st32(tP + hf * 32, pk);
      }
      l_run = l_run * scale_o + lsum;
      tc_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(bar(S_PFULL + sb));
        mbar_arrive(bar(S_KEMPTY + sb));
      }
      p_mid = p_mid_next;
    }
    if (ok && nt > 0) {
      if (!wait_or_abort(bar(S_OFULL), 0, abortp)) {
        ok = false;
        fail_site = 75;
      }
    }
    if (ok && nt > 0) {
      tc_fence_after();
      const float inv = 1.f / l_run;
      __nv_bfloat16* orow = P.O + qrow * D;
#pragma unroll
      for (int q4 = 0; q4 < D / 32; ++q4) {
        uint32_t o[32];
        tc_ld32(tO + q4 * 32, o);
        tc_wait_ld();
        if (row_ok) {
#pragma unroll
          for (int e = 0; e < 32; e += 8) {
            uint4 v4;
            v4.x = pack_bf16x2(__uint_as_float(o[e]) * inv, __uint_as_float(o[e + 1]) * inv);
            v4.y = pack_bf16x2(__uint_as_float(o[e + 2]) * inv, __uint_as_float(o[e + 3]) * inv);
            v4.z = pack_bf16x2(__uint_as_float(o[e + 4]) * inv, __uint_as_float(o[e + 5]) * inv);
            v4.w = pack_bf16x2(__uint_as_float(o[e + 6]) * inv, __uint_as_float(o[e + 7]) * inv);
            *reinterpret_cast<uint4*>(orow + q4 * 32 + e) = v4;
          }
        }
      }
      if (P.LSE && row_ok) P.LSE[qrow] = (m_used * kScaleLog2 + log2f(l_run)) * 0.6931471805599453f;
      if (COUNT) {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, off);
        if (lane == 0 && cnt) atomicAdd(P.kept + bhq, cnt);
      }
    }
  }

  if (fail_site) {
    atomicExch(P.status, 1u);
    atomicExch(P.status + 1, fail_site);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, TMEM_COLS);
}

template <int D>
atf_status launch_split(const CUtensorMap& tqh, const CUtensorMap& tql, const CUtensorMap& tkh, const CUtensorMap& tkl,
                        const CUtensorMap& tv, const SplitParams& P, const AtfTable& t, int B, int mode, bool count,
                        cudaStream_t s) {
  dim3 grid((P.N + T - 1) / T, P.Hq, B);
  const int smem = SplitSmem<D>::DYN_BYTES;
#define ATF_SP_LAUNCH(MODE_, COUNT_)                                                                   \
  do {                                                                                                 \
    auto kern = atf_prefill_split_kernel<D, MODE_, COUNT_>;                                            \
    ATF_CUDA_CHECK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));     \
    kern<<<grid, SP_THREADS, smem, s>>>(tqh, tql, tkh, tkl, tv, P, t);                                 \
  } while (0)
  if (mode == ATF_MODE_EXACT) {
    if (count) ATF_SP_LAUNCH(ATF_MODE_EXACT, true); else ATF_SP_LAUNCH(ATF_MODE_EXACT, false);
  } else {
    if (count) ATF_SP_LAUNCH(ATF_MODE_COARSE, true); else ATF_SP_LAUNCH(ATF_MODE_COARSE, false);
  }
#undef ATF_SP_LAUNCH
  ATF_CUDA_CHECK(cudaGetLastError());
  return ATF_OK;
}

size_t part_bytes(int B, int H, int64_t N, int d) {
  size_t b = (size_t)B * H * N * d * 2;
  return (b + 255) & ~(size_t)255;
}

}  // namespace

atf_status atf_validate_table(const char* who, const int64_t* table, int d, int64_t N, AtfTable* out);

size_t atf_prefill_split_workspace_bytes(int B, int Hq, int Hkv, int64_t N, int d) {
  return ATF_WS_HEADER + 2 * part_bytes(B, Hq, N, d) + 2 * part_bytes(B, Hkv, N, d);
}

extern "C" atf_status atf_prefill_split(const float* Q, const float* K, const void* V, void* O, float* LSE, int B, int Hq,
                                        int Hkv, int64_t N, int d, const int64_t* table, int causal,
                                        const atf_opts* opts, void* stream) {
  if (!Q || !K || !V || !O) return atf_fail(ATF_ERR_INVALID_ARG, "atf_prefill_split: null pointer");
  if (d != 64 && d != 128) return atf_fail(ATF_ERR_UNSUPPORTED, "atf_prefill_split: d must be 64 or 128 (got %d)", d);
  if (B < 1 || Hq < 1 || Hkv < 1 || N < 1) return atf_fail(ATF_ERR_INVALID_ARG, "atf_prefill_split: bad shape");
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
  const size_t qb = part_bytes(B, Hq, N, d), kb = part_bytes(B, Hkv, N, d);
  __nv_bfloat16* Qhi = (__nv_bfloat16*)(base + ATF_WS_HEADER);
  __nv_bfloat16* Qlo = (__nv_bfloat16*)(base + ATF_WS_HEADER + qb);
  __nv_bfloat16* Khi = (__nv_bfloat16*)(base + ATF_WS_HEADER + 2 * qb);
  __nv_bfloat16* Klo = (__nv_bfloat16*)(base + ATF_WS_HEADER + 2 * qb + kb);
  cudaStream_t s = (cudaStream_t)stream;
  {
    const int64_t rows_q = (int64_t)B * Hq * N, rows_k = (int64_t)B * Hkv * N;
    const int64_t bq = (rows_q * (d / 8) + 255) / 256, bk = (rows_k * (d / 8) + 255) / 256;
    if (bq > 0x7FFFFFFF) return atf_fail(ATF_ERR_UNSUPPORTED, "atf_prefill_split: problem too large for the repack grid");
    atf_split_repack_kernel<<<(unsigned)bq, 256, 0, s>>>(Q, Qhi, Qlo, rows_q, d);
    atf_split_repack_kernel<<<(unsigned)bk, 256, 0, s>>>(K, Khi, Klo, rows_k, d);
    ATF_CUDA_CHECK(cudaGetLastError());
  }
  CUtensorMap tqh, tql, tkh, tkl, tv;
  if ((st = atf_make_tile_map(&tqh, Qhi, (int64_t)B * Hq, N, d, N, T)) != ATF_OK) return st;
  if ((st = atf_make_tile_map(&tql, Qlo, (int64_t)B * Hq, N, d, N, T)) != ATF_OK) return st;
  if ((st = atf_make_tile_map(&tkh, Khi, (int64_t)B * Hkv, N, d, N, T)) != ATF_OK) return st;
  if ((st = atf_make_tile_map(&tkl, Klo, (int64_t)B * Hkv, N, d, N, T)) != ATF_OK) return st;
  if ((st = atf_make_tile_map(&tv, V, (int64_t)B * Hkv, N, d, N, T)) != ATF_OK) return st;

  SplitParams P;
  P.Qhi = Qhi;
  P.Qlo = Qlo;
  P.O = (__nv_bfloat16*)O;
  P.LSE = LSE;
  P.kept = opts ? (unsigned long long*)opts->kept_terms : nullptr;
  P.status = (unsigned int*)base;
  P.Hq = Hq;
  P.Hkv = Hkv;
  P.N = (int)N;
  const bool count = P.kept != nullptr;
  return d == 64 ? launch_split<64>(tqh, tql, tkh, tkl, tv, P, t, B, mode, count, s)
                 : launch_split<128>(tqh, tql, tkh, tkl, tv, P, t, B, mode, count, s);
}
