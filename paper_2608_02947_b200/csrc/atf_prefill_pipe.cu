// atf_prefill kernel: windowed causal attention for all query rows (Sec. 3.3, Fig. 3) on the sm_100a
// tensor cores, ONE 128-row query tile of one head per CTA.  (Layout of the operands: atf_prefill.cu.)
//
// With a single query tile the 512 tensor-memory columns hold two S buffers, two P buffers and O, so
// the chain "softmax -> O += P V -> next S -> softmax" is cut: S(t + 1) = Q K(t + 1)^T is computed
// while the softmax groups work on S(t), and O += P(t) V runs whenever P(t) is stored.  Warp roles:
//   warp 0      TMA producer: Q (again per pass, see below), K (live 64-column blocks) and V
//               tiles into three-stage rings of 128-byte-swizzled shared memory;
//   warp 1      issuer of S(t) = Q K(t)^T over the live depth (one thread, tcgen05.mma SS form);
//   warp 2      issuer of O += P(t) V(t), half a tile at a time (one thread, TS form: P is read from
//               tensor memory, V through the MN-major descriptor);
//   warps 4-7   softmax group 0: keys 0..63 of every tile, one query row per thread;
//   warps 8-11  softmax group 1: keys 64..127 of the same rows.
// The two threads of a row never meet in the common step: exponentials are taken against the
// row's reference maximum from the diagonal tile (any reference gives the same softmax as long
// as nothing overflows: P is bf16, O and the row sums are fp32), each thread keeps its own
// partial row sum, and the halves are added at the end.  A thread whose sum of a step is not
// below 2^64 raises a flag; the CTA then runs its tile a second time in the safe form (the two
// groups exchange their row maxima through shared memory every step and rescale O at once).
//
// Steps far from the diagonal and from every window boundary ("plain") need neither the mask nor the
// per-cell finish and run in a loop of their own, kept small so that it stays in the instruction
// cache; everything else takes the general step, one step at a time.
//
// Exact mode (the per-term definition).  Whether a pair stays in the MMA is decided per quarter of
// the rows over the whole 128 keys (the pair is live at the distance from the quarter's middle row
// to the tile's middle column); the pairs a quarter does not keep are zeroed in its rows of the
// CTA's copy of Q (pairs only die as the distance grows and the tiles are walked outwards from
// the diagonal, so the zeroing is monotone).  A warp then finishes its 32 x 64 cells on the CUDA
// cores: pairs in the MMA are taken back out of the cells beyond their window, pairs zeroed in Q
// are added where live.  Coarse mode: depth = pairs live anywhere in the tile rounded up to 8,
// everything on the diagonal tile, no per-cell work.
//
// Appended rows (App. C, "The interval itself"; Sec. 7.3): the tiles stay aligned at position 0 of the
// context, the grid covers only the tiles that hold query rows, Q is addressed at tile * 128 - n0.
// Every wait is bounded and reports through the workspace status words.
#include <cuda.h>

#include <algorithm>

#include "atf_common.cuh"
#include "atf_prefill_pipe.cuh"

namespace {

constexpr int T = 128;
constexpr int BLK_BYTES = T * 128;
constexpr int PP_THREADS = 384;
constexpr float RESCALE_THRESHOLD = 8.f;      // safe form: log2 units the reference may lag behind
constexpr float REF_HEADROOM = 60.f;            // fast pass: log2 units the row's reference sits above the diagonal tile's maximum
constexpr float STALE_REF_GUARD = 1.8446744e19f;  // 2^64: a step's partial row sum must stay below it
static_assert(128 * 56 + 256 * 224 <= PP_THREADS * 168, "setmaxnreg budget exceeds the launch allocation");

// SPLIT (the split-precision mode, atf_prefill_split.cu): Q and K come as bf16 hi and lo parts; the CTA holds both
// Q parts, a K stage is a hi tile followed by a lo tile, and the rings shrink to two K stages and one V stage.
template <int D, bool SPLIT>
struct PipeSmem {
  static constexpr int NB = D / 64;
  static constexpr int TILE = NB * BLK_BYTES;
  static constexpr int QN = SPLIT ? 2 : 1;       // operand parts: hi, lo
  static constexpr int KS = SPLIT ? 2 : 3;       // ring depths
  static constexpr int VS = SPLIT ? 1 : 3;
  static constexpr int KSTAGE = QN * TILE;
  static constexpr int Q_OFF = 0;                // hi part, then lo part
  static constexpr int K_OFF = QN * TILE;
  static constexpr int V_OFF = K_OFF + KS * KSTAGE;
  static constexpr int BAR_OFF = V_OFF + VS * TILE;
  static constexpr int X_OFF = BAR_OFF + 256;  // exchange area of the two softmax groups: [2][128] floats
  static constexpr int TOTAL = X_OFF + 1024;
  static constexpr int DYN_BYTES = TOTAL + 1024;  // slack for 1024-byte alignment
};
enum { B_QFULL = 0, B_KFULL = 1, B_KEMPTY = 4, B_VFULL = 7, B_VEMPTY = 10, B_SFULL = 13, B_SREAD = 15, B_PFULL = 17,
       B_PVDONE = 21, B_OFULL = 23, B_XCH = 24, B_QZ = 25, B_COUNT = 26 };

__device__ __forceinline__ float2 exp2_poly2(float2 x) {
  x.x = fmaxf(x.x, -126.f);
  x.y = fmaxf(x.y, -126.f);
  const float2 magic = make_float2(12582912.f, 12582912.f);
  const float2 t = __fadd2_rn(x, magic);
  const float2 nf = __fadd2_rn(t, make_float2(-12582912.f, -12582912.f));
  const float2 f = __fadd2_rn(x, make_float2(-nf.x, -nf.y));
  float2 p = __ffma2_rn(make_float2(0.05520550534f, 0.05520550534f), f, make_float2(0.24261397123f, 0.24261397123f));
  p = __ffma2_rn(p, f, make_float2(0.69325476885f, 0.69325476885f));
  p = __ffma2_rn(p, f, make_float2(0.99992769957f, 0.99992769957f));
  float2 r;
  r.x = __int_as_float(__float_as_int(p.x) + (__float_as_int(t.x) << 23));
  r.y = __int_as_float(__float_as_int(p.y) + (__float_as_int(t.y) << 23));
  return r;
}
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
#ifndef ATF_PIPE_POLY_OF_4
#define ATF_PIPE_POLY_OF_4 1
#endif
// P = 2^(s * scale + neg_m) for 64 columns, packed to bf16 pairs, and their fp32 sum; one packed pair in
// four takes a cubic polynomial on the FMA pipe (relative error < 8e-5, below the bf16 rounding of P), the rest
// MUFU; POLY = 0 (the split-precision mode, whose row sums must be good to 1e-6) is MUFU only.
template <int POLY>
__device__ __forceinline__ float exp_half(float (&s)[64], float scale, float neg_m, uint32_t (&pk)[32]) {
  const float2 sc2 = make_float2(scale, scale), nm2 = make_float2(neg_m, neg_m);
  float2 acc[4] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
#pragma unroll
  for (int c = 0; c < 64; c += 2) {
    float2 x = __ffma2_rn(make_float2(s[c], s[c + 1]), sc2, nm2);
    if (((c >> 1) & 3) < POLY) {
      x = exp2_poly2(x);
    } else {
      x.x = ex2_approx(x.x);
      x.y = ex2_approx(x.y);
    }
    acc[(c >> 1) & 3] = __fadd2_rn(acc[(c >> 1) & 3], x);
    pk[c >> 1] = pack_bf16x2(x.x, x.y);
  }
  const float2 a01 = __fadd2_rn(acc[0], acc[1]), a23 = __fadd2_rn(acc[2], acc[3]);
  return (a01.x + a01.y) + (a23.x + a23.y);
}

// Band schedule (Sec. 3.3: the active pairs of a tile are known statically).  What a step needs depends only on
// the tile distance dt and on which 32 rows x 64 keys of the tile a softmax warp owns (quarter wq of the rows,
// half h of the keys); it is the same for every CTA of a launch.  A pre-kernel writes one word per (dt, wq, h):
//   p_all  [0:7)   pairs live in every cell of the warp's block,      p_any [7:14)  pairs live in some cell of it,
//   p_mid  [14:21) pairs quarter wq keeps in the MMA (live at the distance from its middle row to the tile's
//                  middle column); the others are zero in its rows of Q,
//   natoms [21:25) 16-column MMA steps of S,   nkb [25:27) 64-column K blocks to load minus one,
//   plain  [27]    the block needs neither mask nor per-cell finish and S is not empty.
// Roles read their word a step ahead, so no schedule arithmetic sits in front of a step.
struct PipeWord {
  int p_all, p_any, p_mid, natoms, nkb;
  bool plain;
  __device__ __forceinline__ explicit PipeWord(uint32_t e)
      : p_all(e & 127), p_any((e >> 7) & 127), p_mid((e >> 14) & 127), natoms((e >> 21) & 15), nkb(((e >> 25) & 3) + 1),
        plain((e >> 27) & 1) {}
};

template <int MODE>
__global__ void __launch_bounds__(128)
atf_pipe_sched_kernel(const __grid_constant__ AtfTable table, int H, int ndt, uint32_t* __restrict__ out) {
  // one thread per word: 16 tile distances x 8 (quarter, half) blocks per CTA, the table in shared memory
  __shared__ int w[ATF_MAX_PAIRS];
  if (threadIdx.x < H) w[threadIdx.x] = table.w[threadIdx.x];
  __syncthreads();
  const int dt = blockIdx.x * 16 + (threadIdx.x >> 3);
  if (dt >= ndt) return;
  const int wq = (threadIdx.x >> 1) & 3, h = threadIdx.x & 1;
  const int Wmax = w[H - 1];
  auto reaching = [&](int z) {  // pairs (from the low-frequency end) whose window reaches distance z
    int lo = 0, hi = H;         // first r with w[r] >= z, w non-decreasing
    while (lo < hi) {
      const int mid = (lo + hi) >> 1;
      if (w[mid] < z) lo = mid + 1; else hi = mid;
    }
    return H - lo;
  };
  const int tile_any = reaching(dt == 0 ? 0 : dt * T - (T - 1));  // live somewhere in the tile
  const int mid0 = reaching(dt == 0 ? 15 : dt * T - 48);           // what the nearest quarter keeps in the MMA
  const int natoms = MODE == ATF_MODE_EXACT ? (mid0 + 7) / 8 : (dt == 0 ? H / 8 : (tile_any + 7) / 8);
  const int cols = MODE == ATF_MODE_EXACT ? 2 * tile_any : 16 * natoms;  // exact mode also reads the pairs it adds per cell
  const int nkb = max(1, (cols + 63) / 64);
  const int zmax = dt * T + 32 * wq + 31 - 64 * h, zmin = dt * T + 32 * wq - 64 * h - 63;
  const int p_all = reaching(max(0, zmax)), p_any = reaching(max(0, zmin));
  const int p_mid = reaching(dt == 0 ? 16 * wq + 15 : dt * T + 32 * wq - 48);
  bool plain = dt > 0 && natoms > 0;
  if (MODE == ATF_MODE_EXACT) plain = plain && zmax <= Wmax && min(p_all, p_mid) >= max(p_any, p_mid);
  out[8 * dt + 2 * wq + h] = (uint32_t)p_all | ((uint32_t)p_any << 7) | ((uint32_t)p_mid << 14) | ((uint32_t)natoms << 21) |
                             ((uint32_t)(nkb - 1) << 25) | ((uint32_t)plain << 27);
}

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

template <int D, int MODE, bool COUNT, bool SPLIT>
__global__ void __launch_bounds__(PP_THREADS, 1)
atf_prefill_pipe_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmQlo,
                        const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmKlo,
                        const __grid_constant__ CUtensorMap tmV, const __grid_constant__ AtfPipeParams P,
                        const __grid_constant__ AtfTable table) {
  using SM = PipeSmem<D, SPLIT>;
  constexpr int KS = SM::KS, VS = SM::VS;
  constexpr int POLY = SPLIT ? 0 : ATF_PIPE_POLY_OF_4;
  constexpr int H = D / 2;
  constexpr int NB = D / 64;
  constexpr uint32_t TMEM_COLS = 512;  // S0, S1 (128 each) | O (D) at 256 | P0, P1 (64 each) at 384
  constexpr uint32_t IDESC_QK = make_idesc_bf16(128, T, 0, 0);
  constexpr uint32_t IDESC_PV = make_idesc_bf16(128, D, 0, 1);
  const float kScaleLog2 = 1.4426950408889634f / sqrtf((float)D);

  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t sQ = smem_base + SM::Q_OFF, sK = smem_base + SM::K_OFF, sV = smem_base + SM::V_OFF;
  const uint32_t bars = smem_base + SM::BAR_OFF;
  auto bar = [&](int slot) { return bars + 8u * (uint32_t)slot; };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_gen + SM::BAR_OFF + 8 * B_COUNT);
  volatile float* xch = reinterpret_cast<volatile float*>(smem_gen + SM::X_OFF);  // [2][128]
  __shared__ int sW[ATF_MAX_PAIRS];
  __shared__ int s_abort;
  __shared__ int s_redo;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int ntq = (P.N + T - 1) / T;
  const int it = ntq - 1 - (int)blockIdx.x;  // longest rows first; the grid stops at the tile holding row n0
  const int n0 = P.N - P.Nq;
  const int hq = blockIdx.y, b = blockIdx.z;
  const int bhq = b * P.Hq + hq;
  const int bhk = b * P.Hkv + hq / (P.Hq / P.Hkv);

  if (tid < H) sW[tid] = table.w[tid];
  if (tid == 0) {
    s_abort = 0;
    s_redo = 0;
    mbar_init(bar(B_QFULL), 1);
    mbar_init(bar(B_OFULL), 1);
    mbar_init(bar(B_XCH), 8);
    mbar_init(bar(B_QZ), 4);
    for (int i = 0; i < 3; ++i) {
      mbar_init(bar(B_KFULL + i), 1);
      // exact mode: the softmax warps read K for the per-cell finish and release the stage; coarse: the issuer's commit
      mbar_init(bar(B_KEMPTY + i), MODE == ATF_MODE_EXACT ? 8 : 1);
      mbar_init(bar(B_VFULL + i), 1);
      mbar_init(bar(B_VEMPTY + i), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar(B_SFULL + i), 1);
      mbar_init(bar(B_SREAD + i), 8);
      mbar_init(bar(B_PFULL + 2 * i), 4);
      mbar_init(bar(B_PFULL + 2 * i + 1), 4);
      mbar_init(bar(B_PVDONE + i), 1);
    }
    mbar_fence_init();
    fence_proxy_async_smem();
    tma_prefetch_desc(&tmQ);
    tma_prefetch_desc(&tmK);
    if (SPLIT) {
      tma_prefetch_desc(&tmQlo);
      tma_prefetch_desc(&tmKlo);
    }
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

  // Every role runs the tile once and, if a softmax thread raised s_redo, once more in the safe form.  The
  // passes end at a CTA-wide barrier (the same barrier from every role's branch); barrier phases of the
  // pipeline run on across the passes (g = steps since the start of the kernel).
  auto another_pass = [&](int pass) {
    asm volatile("bar.sync 0;" ::: "memory");
    return pass == 0 && *reinterpret_cast<volatile int*>(&s_redo) != 0;
  };

  if (warp == 0) {
    // =============================== TMA producer ===============================
    asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
    for (int pass = 0; pass < 2; ++pass) {
      const int g0 = pass * nt;
      if (lane == 0) {
        mbar_expect_tx(bar(B_QFULL), SM::QN * SM::TILE);
        for (int kb = 0; kb < NB; ++kb) {
          // rows before n0 do not exist in Q: the (possibly negative) coordinate reads zero fill there
          tma_load_3d(sQ + kb * BLK_BYTES, &tmQ, bar(B_QFULL), kb * 64, it * T - n0, bhq);
          if (SPLIT) tma_load_3d(sQ + SM::TILE + kb * BLK_BYTES, &tmQlo, bar(B_QFULL), kb * 64, it * T - n0, bhq);
        }
        auto load_k = [&](int t) {
          const int g = g0 + t, ks = g % KS;
          if (!wait_or_abort(bar(B_KEMPTY + ks), ((g / KS) & 1) ^ 1, abortp)) return false;
          const int nkb = PipeWord(__ldg(P.sched + 8 * t)).nkb;
          mbar_expect_tx(bar(B_KFULL + ks), SM::QN * nkb * BLK_BYTES);
          for (int kb = 0; kb < nkb; ++kb) {
            tma_load_3d(sK + ks * SM::KSTAGE + kb * BLK_BYTES, &tmK, bar(B_KFULL + ks), kb * 64, (it - t) * T, bhk);
            if (SPLIT)
              tma_load_3d(sK + ks * SM::KSTAGE + SM::TILE + kb * BLK_BYTES, &tmKlo, bar(B_KFULL + ks), kb * 64, (it - t) * T, bhk);
          }
          return true;
        };
        auto load_v = [&](int t) {
          const int g = g0 + t, vs = g % VS;
          if (!wait_or_abort(bar(B_VEMPTY + vs), ((g / VS) & 1) ^ 1, abortp)) return false;
          mbar_expect_tx(bar(B_VFULL + vs), SM::TILE);
          for (int kb = 0; kb < NB; ++kb)
            tma_load_3d(sV + vs * SM::TILE + kb * BLK_BYTES, &tmV, bar(B_VFULL + vs), kb * 64, (it - t) * T, bhk);
          return true;
        };
        if (SPLIT) {
          // one V stage: V(t) has to wait for O += P(t - 1) V, so K(t + 1) goes first
          bool pok = nt == 0 || load_k(0);
          for (int t = 0; t < nt && pok; ++t) pok = (t + 1 >= nt || load_k(t + 1)) && load_v(t);
          if (!pok) fail_site = 10;
        } else {
          for (int t = 0; t < nt; ++t)
            if (!load_k(t) || !load_v(t)) { fail_site = 10; break; }
        }
      }
      if (!another_pass(pass)) break;
    }
  } else if (warp == 1) {
    // =============================== issuer of S = Q K^T ===============================
    asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
    for (int pass = 0; pass < 2; ++pass) {
      const int g0 = pass * nt;
      if (lane == 0) {
        const uint64_t dQ = make_smem_desc_sw128(sQ, 16, 1024);
        bool iok = wait_or_abort(bar(B_QFULL), pass & 1, abortp);
        if (!iok) fail_site = 20;
        for (int t = 0; t < nt && iok; ++t) {
          const int g = g0 + t, sb = g & 1, ks = g % KS;
          const int natoms = PipeWord(__ldg(P.sched + 8 * t)).natoms;
          iok = wait_or_abort(bar(B_KFULL + ks), (g / KS) & 1, abortp);
          // both softmax groups hold S(g - 2) in registers: its buffer may be written again
          if (iok && g >= 2) iok = wait_or_abort(bar(B_SREAD + sb), ((g >> 1) - 1) & 1, abortp);
          // exact mode: the pairs a quarter does not keep in the MMA of this tile are zero in its rows of Q
          if (iok && MODE == ATF_MODE_EXACT) iok = wait_or_abort(bar(B_QZ), g & 1, abortp);
          if (!iok) { fail_site = 21; break; }
          tc_fence_after();
          const uint64_t dK = make_smem_desc_sw128(sK + ks * SM::KSTAGE, 16, 1024);
          const uint32_t tS = tmem_base + sb * T;
          for (int a = 0; a < natoms; ++a) {
            // K-major operands advance 32 bytes per 16-column step inside a 64-column block, one block per four steps
            const uint64_t off = (uint64_t)((a & 3) * 2 + (a >> 2) * (BLK_BYTES / 16));
            tc_mma_ss(tS, dQ + off, dK + off, IDESC_QK, a > 0 ? 1u : 0u);
            if (SPLIT) {  // + Q_hi K_lo^T + Q_lo K_hi^T (the lo parts sit one tile after the hi parts)
              tc_mma_ss(tS, dQ + off, dK + off + (uint64_t)(SM::TILE / 16), IDESC_QK, 1u);
              tc_mma_ss(tS, dQ + off + (uint64_t)(SM::TILE / 16), dK + off, IDESC_QK, 1u);
            }
          }
          tc_commit(bar(B_SFULL + sb));
          if (MODE != ATF_MODE_EXACT) tc_commit(bar(B_KEMPTY + ks));
        }
      }
      if (!another_pass(pass)) break;
    }
  } else if (warp == 2) {
    // =============================== issuer of O += P V ===============================
    asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
    for (int pass = 0; pass < 2; ++pass) {
      const int g0 = pass * nt;
      if (lane == 0) {
        bool iok = true;
        for (int t = 0; t < nt && iok; ++t) {
          const int g = g0 + t, sb = g & 1, vs = g % VS;
          const uint64_t dV = make_smem_desc_sw128(sV + vs * SM::TILE, BLK_BYTES, 1024);
          const uint32_t tO = tmem_base + 2 * T, tP = tmem_base + 3 * T + sb * 64;
          iok = wait_or_abort(bar(B_VFULL + vs), (g / VS) & 1, abortp);
          for (int h = 0; h < 2 && iok; ++h) {
            iok = wait_or_abort(bar(B_PFULL + 2 * sb + h), (g >> 1) & 1, abortp);
            if (!iok) break;
            tc_fence_after();
#pragma unroll
            for (int i = 0; i < 4; ++i)  // V advances 16 key rows (2048 bytes) per step, P 8 columns
              tc_mma_ts(tO, tP + 32 * h + 8 * i, dV + (uint64_t)(512 * h + 128 * i), IDESC_PV,
                        (t > 0 || h > 0 || i > 0) ? 1u : 0u);
          }
          if (!iok) { fail_site = 22; break; }
          tc_commit(bar(B_VEMPTY + vs));
          tc_commit(bar(B_PVDONE + sb));
        }
        if (iok) tc_commit(bar(B_OFULL));
      }
      if (!another_pass(pass)) break;
    }
  } else if (warp == 3) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
    for (int pass = 0; pass < 2; ++pass)
      if (!another_pass(pass)) break;
  } else {
    // =============================== softmax groups ===============================
    asm volatile("setmaxnreg.inc.sync.aligned.u32 224;");
    const int h = warp >= 8 ? 1 : 0;  // keys 64h .. 64h + 63 of every tile
    const int wq = warp & 3;
    const int row = (tid - 128) & 127;
    const int n = it * T + row;
    const bool row_ok = n >= n0 && n < P.N;
    const int64_t qrow = (int64_t)bhq * P.Nq + (row_ok ? n - n0 : 0);
    const uint32_t lane_off = (uint32_t)(wq * 32) << 16;
    const uint32_t tO = tmem_base + 2 * T + lane_off;
    const __nv_bfloat16* qsrc = P.Qp + qrow * D;
    const __nv_bfloat16* qsrc_lo = SPLIT ? P.Qp_lo + qrow * D : nullptr;
    float m_used = -INFINITY, l_run = 0.f;
    unsigned long long cnt = 0;
    uint32_t xphase = 0;
    bool ok = true;
    // all eight softmax warps meet (bounded): what each wrote to the exchange area before is visible after
    auto softmax_sync = [&]() {
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(B_XCH));
      const bool r = wait_or_abort(bar(B_XCH), xphase & 1, abortp);
      ++xphase;
      return r;
    };
    for (int pass = 0; pass < 2; ++pass) {
      const int g0 = pass * nt;
      const bool safe = pass == 1;
      m_used = -INFINITY;
      l_run = 0.f;
      cnt = 0;
      bool overflow = false;
      int zeroed_from = H;  // pairs p >= zeroed_from are zero in this row of the shared copy of Q
      // group 0 owns the rows of Q: zero what the quarter does not keep in the MMA, then tell the issuer
      auto zero_q_down_to = [&](int p_keep) {
        if (h == 0) {
          for (int p = p_keep; p < zeroed_from; ++p) {
            const int col = 2 * p;
            const uint32_t off = (col >> 6) * BLK_BYTES + sw128_offset(row, (col & 63) >> 3) + (col & 7) * 2;
            *reinterpret_cast<uint32_t*>(smem_gen + SM::Q_OFF + off) = 0u;
            if (SPLIT) *reinterpret_cast<uint32_t*>(smem_gen + SM::Q_OFF + SM::TILE + off) = 0u;
          }
          zeroed_from = min(zeroed_from, p_keep);
          fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar(B_QZ));
        }
      };
      const uint32_t* sched = P.sched + 2 * wq + h;
      uint32_t e_cur = __ldg(sched);  // schedule word of the step at hand; the next one is fetched a step ahead
      int p_mid = PipeWord(e_cur).p_mid;
      if (MODE == ATF_MODE_EXACT) {
        if (ok && !wait_or_abort(bar(B_QFULL), pass & 1, abortp)) { ok = false; fail_site = 30; }
        if (ok) zero_q_down_to(p_mid);
      }
      int t = 0;
      while (t < nt && ok) {
        // ---- plain steps: no mask, no per-cell finish, reference from the diagonal tile.  A loop of its own,
        //      kept small so that it stays in the instruction cache; everything else takes the general step. ----
        for (; t < nt && !safe && t > 0; ++t) {
          const int g = g0 + t, sb = g & 1, ks = g % KS;
          const PipeWord E(e_cur);
          if (!E.plain) break;
          const uint32_t e_next = t + 1 < nt ? __ldg(sched + 8 * (t + 1)) : 0u;
          const int p_all = E.p_all, natoms = E.natoms;
          const int p_mid_next = PipeWord(e_next).p_mid;
          if (!wait_or_abort(bar(B_SFULL + sb), (g >> 1) & 1, abortp)) { ok = false; fail_site = 31; break; }
          tc_fence_after();
          if (MODE == ATF_MODE_EXACT && t + 1 < nt) zero_q_down_to(p_mid_next);
          float s[64];
          tc_ld32(tmem_base + sb * T + 64 * h + lane_off, reinterpret_cast<uint32_t*>(s));
          tc_ld32(tmem_base + sb * T + 64 * h + lane_off + 32, reinterpret_cast<uint32_t*>(s) + 32);
          tc_wait_ld();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) {
            mbar_arrive(bar(B_SREAD + sb));
            if (MODE == ATF_MODE_EXACT) mbar_arrive(bar(B_KEMPTY + ks));
          }
          if (COUNT && row_ok)
            cnt += (unsigned long long)(MODE == ATF_MODE_EXACT ? p_all : min(H, 8 * natoms)) * 64ull;
          uint32_t pk[32];
          const float lsum = exp_half<POLY>(s, kScaleLog2, -m_used * kScaleLog2, pk);
          overflow |= !(lsum < STALE_REF_GUARD);
          if (g >= 2 && !wait_or_abort(bar(B_PVDONE + sb), ((g - 2) >> 1) & 1, abortp)) { ok = false; fail_site = 35; break; }
          tc_st32(tmem_base + 3 * T + sb * 64 + 32 * h + lane_off, pk);
          l_run += lsum;
          tc_wait_st();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar(B_PFULL + 2 * sb + h));
          p_mid = p_mid_next;
          e_cur = e_next;
        }
        if (t >= nt || !ok) break;
        // ---- one general step ----
        const int g = g0 + t, sb = g & 1, ks = g % KS;
        const int dt = t;
        const int zrow = dt * T + row;             // distance from this row to column 0 of the key tile
        const int zmax_w = dt * T + 32 * wq + 31 - 64 * h;  // over the warp's 32 x 64 cells
        const int zmin_w = dt * T + 32 * wq - 64 * h - 63;
        const PipeWord E(e_cur);
        const uint32_t e_next = t + 1 < nt ? __ldg(sched + 8 * (t + 1)) : 0u;
        const int p_all = E.p_all, p_any = E.p_any, natoms = E.natoms;
        const int p_mid_next = PipeWord(e_next).p_mid;
        const uint32_t tS = tmem_base + sb * T + 64 * h + lane_off;
        const uint32_t tP = tmem_base + 3 * T + sb * 64 + 32 * h + lane_off;
        if (!wait_or_abort(bar(B_SFULL + sb), (g >> 1) & 1, abortp)) { ok = false; fail_site = 31; break; }
        tc_fence_after();
        // S(t) is complete, so Q is not being read: zero what the quarter does not keep in the next tile's MMA
        if (MODE == ATF_MODE_EXACT && t + 1 < nt) zero_q_down_to(p_mid_next);
        float s[64];
        if (natoms > 0) {
          tc_ld32(tS, reinterpret_cast<uint32_t*>(s));
          tc_ld32(tS + 32, reinterpret_cast<uint32_t*>(s) + 32);
          tc_wait_ld();
        } else {  // no pair is kept in the MMA of this tile: every live term is added below
#pragma unroll
          for (int c = 0; c < 64; ++c) s[c] = 0.f;
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(B_SREAD + sb));

        if (MODE == ATF_MODE_EXACT) {
          // ---- per-cell finish.  Pairs [p_all, p_mid) went through the MMA and are not live in every cell of
          //      the warp's block: take their term back out of the cells beyond the window.  Pairs [p_mid, p_any)
          //      are zero in Q and live somewhere in the block: add their term inside the window.  32 columns at
          //      a time, skipping what no row of the warp needs. ----
          const int p_lo = min(p_all, p_mid), p_hi = max(p_any, p_mid);
          if (p_lo < p_hi && zmax_w >= 0) {
            if (!wait_or_abort(bar(B_KFULL + ks), (g / KS) & 1, abortp)) { ok = false; fail_site = 32; break; }
            const int zw_lo = dt * T + wq * 32, zw_hi = zw_lo + 31;  // zrow over the warp's rows
            for (int p = p_lo; p < p_hi; ++p) {
              const bool subtract = p < p_mid;
              if (subtract ? p < p_all : p >= p_any) continue;  // live everywhere and in the MMA / dead everywhere and zeroed
              const int wp = sW[H - 1 - p];
              // distances of the warp's cells in columns 64h + 32q .. + 31: [zw_lo - c1, zw_hi - c0]
              bool touched[2];
#pragma unroll
              for (int q = 0; q < 2; ++q) {
                const int c0 = 64 * h + 32 * q;
                const int hi = zw_hi - c0, lo = zw_lo - c0 - 31;
                touched[q] = subtract ? (hi > wp) : (lo <= wp && hi >= 0);
              }
              if (!touched[0] && !touched[1]) continue;
              // q0, q1: the pair's two elements of this row (hi parts in the split mode); qs0, qs1: hi + lo there
              // (exact in fp32: 16 significant bits), so that the term below is the three products of the MMA
              const uint32_t qq = *reinterpret_cast<const uint32_t*>(qsrc + 2 * p);
              float q0 = bf16lo_to_f32(qq), q1 = bf16hi_to_f32(qq);
              float qs0 = q0, qs1 = q1;
              if (SPLIT) {
                const uint32_t ql = *reinterpret_cast<const uint32_t*>(qsrc_lo + 2 * p);
                qs0 += bf16lo_to_f32(ql);
                qs1 += bf16hi_to_f32(ql);
              }
              if (subtract) {
                q0 = -q0;
                q1 = -q1;
                qs0 = -qs0;
                qs1 = -qs1;
              }
              const int col = 2 * p;
              const uint32_t kb32 = sK + ks * SM::KSTAGE + (col >> 6) * BLK_BYTES + (col & 7) * 2;
              const int chunk = (col & 63) >> 3;
              // cells with column >= jb = zrow - w are inside the window: adding uses sat(c - jb + 1), taking back
              // sat(jb - c), formed on the FMA pipe
              const float jbf = (float)(zrow - wp - 64 * h);
              const float ca = subtract ? -1.f : 1.f, cb = subtract ? jbf : 1.f - jbf;
#pragma unroll
              for (int q = 0; q < 2; ++q) {
                if (touched[q]) {  // warp-uniform
                  uint32_t kk[32], kl[SPLIT ? 32 : 1];
#pragma unroll
                  for (int cc = 0; cc < 32; ++cc) {
                    const int c = 64 * h + 32 * q + cc;  // key of the tile; (c & 7) does not depend on h
                    asm volatile("ld.shared.b32 %0, [%1];" : "=r"(kk[cc]) : "r"(kb32 + ((chunk ^ (c & 7)) << 4) + c * 128));
                    if (SPLIT)
                      asm volatile("ld.shared.b32 %0, [%1];" : "=r"(kl[cc]) : "r"(kb32 + SM::TILE + ((chunk ^ (c & 7)) << 4) + c * 128));
                  }
#pragma unroll
                  for (int cc = 0; cc < 32; ++cc) {
                    const int cl = 32 * q + cc;  // column of this thread's half
                    float term = fmaf(qs0, bf16lo_to_f32(kk[cc]), qs1 * bf16hi_to_f32(kk[cc]));
                    if (SPLIT) term = fmaf(q0, bf16lo_to_f32(kl[cc]), fmaf(q1, bf16hi_to_f32(kl[cc]), term));
                    const float coef = __saturatef(fmaf(ca, (float)cl, cb));
                    s[cl] = fmaf(term, coef, s[cl]);
                  }
                }
              }
            }
          }
        }
        // ---- causal mask on the diagonal tile, dropped keys (exact mode: no pair reaches the cell) ----
        if (dt == 0 || (MODE == ATF_MODE_EXACT && zmax_w > Wmax)) {
          const int zdrop = MODE == ATF_MODE_EXACT ? Wmax : 0x7FFFFFFF;
#pragma unroll
          for (int c = 0; c < 64; ++c) {
            const int z = zrow - 64 * h - c;
            s[c] = (z >= 0 && z <= zdrop) ? s[c] : -INFINITY;
          }
        }
        if (COUNT && row_ok) {
          const int c_lo = 64 * h, c_hi = min(64 * h + 63, zrow);  // causal cells of this thread's half
          if (c_hi >= c_lo) {
            if (MODE == ATF_MODE_EXACT) {
              cnt += (unsigned long long)p_all * (unsigned long long)(c_hi - c_lo + 1);
              for (int p = p_all; p < p_any; ++p) {
                const int lo = max(c_lo, zrow - sW[H - 1 - p]);
                cnt += (unsigned long long)max(0, c_hi - lo + 1);
              }
            } else {
              cnt += (unsigned long long)min(H, 8 * natoms) * (unsigned long long)(c_hi - c_lo + 1);
            }
          }
        }
        if (MODE == ATF_MODE_EXACT) {  // done with K of this tile
          __syncwarp();
          if (lane == 0) mbar_arrive(bar(B_KEMPTY + ks));
        }

        // ---- reference maximum ----
        float scale_o = 1.f;
        if (t == 0 || safe) {
          float mx = -INFINITY;
#pragma unroll
          for (int c = 0; c < 64; ++c) mx = fmaxf(mx, s[c]);
          xch[h * 128 + row] = mx;
          if (!softmax_sync()) { ok = false; fail_site = 33; break; }
          mx = fmaxf(mx, xch[(h ^ 1) * 128 + row]);
          if (!softmax_sync()) { ok = false; fail_site = 33; break; }  // both have read: the area may be written again
          bool moved = false;
          if (mx > m_used && (m_used == -INFINITY || (mx - m_used) * kScaleLog2 > RESCALE_THRESHOLD)) {
            scale_o = m_used == -INFINITY ? 0.f : ex2_approx((m_used - mx) * kScaleLog2);
            m_used = mx;
            // Fast pass: the reference stays for the whole row, so it is put REF_HEADROOM above the diagonal tile's
            // maximum: sums overflow only ~120 log2 units above that maximum instead of ~60, and what the shift can
            // flush to zero lies 2^-66 below the diagonal's own largest term.
            if (!safe) m_used += REF_HEADROOM / kScaleLog2;
            moved = t > 0;  // nothing has been accumulated before the first tile
          }
          if (__any_sync(0xffffffffu, moved)) {
            // every product into O issued so far must be complete; the two threads of a row take half of O each
            if (!wait_or_abort(bar(B_PVDONE + ((g - 1) & 1)), ((g - 1) >> 1) & 1, abortp)) { ok = false; fail_site = 34; break; }
            tc_fence_after();
#pragma unroll
            for (int q4 = 0; q4 < D / 64; ++q4) {
              uint32_t o[32];
              tc_ld32(tO + (D / 2) * h + q4 * 32, o);
              tc_wait_ld();
#pragma unroll
              for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * scale_o);
              tc_st32(tO + (D / 2) * h + q4 * 32, o);
            }
            tc_wait_st();
          }
        }
        uint32_t pk[32];
        const float lsum = exp_half<POLY>(s, kScaleLog2, m_used == -INFINITY ? 0.f : -m_used * kScaleLog2, pk);
        overflow |= !(lsum < STALE_REF_GUARD);
        // the product that read the previous contents of this P buffer must be complete
        if (g >= 2 && !wait_or_abort(bar(B_PVDONE + sb), ((g - 2) >> 1) & 1, abortp)) { ok = false; fail_site = 35; break; }
        tc_st32(tP, pk);
        l_run = l_run * scale_o + lsum;
        tc_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(B_PFULL + 2 * sb + h));
        p_mid = p_mid_next;
        e_cur = e_next;
        ++t;
      }
      if (ok && nt > 0 && !wait_or_abort(bar(B_OFULL), pass & 1, abortp)) { ok = false; fail_site = 36; }
      if (!safe && overflow && row_ok) s_redo = 1;
      if (!another_pass(pass)) break;
    }
    // ---- both halves of the row sum, then the output ----
    xch[h * 128 + row] = l_run;
    if (ok && !softmax_sync()) { ok = false; fail_site = 37; }
    const float l_tot = l_run + xch[(h ^ 1) * 128 + row];
    if (ok && nt > 0) {
      tc_fence_after();
      const float inv = 1.f / l_tot;
      __nv_bfloat16* orow = P.O + qrow * D;
#pragma unroll
      for (int q4 = 0; q4 < D / 64; ++q4) {
        const int cbase = (D / 2) * h + q4 * 32;  // group h writes its half of the row
        uint32_t o[32];
        tc_ld32(tO + cbase, o);
        tc_wait_ld();
        if (row_ok) {
#pragma unroll
          for (int e = 0; e < 32; e += 8) {
            uint4 v4;
            v4.x = pack_bf16x2(__uint_as_float(o[e]) * inv, __uint_as_float(o[e + 1]) * inv);
            v4.y = pack_bf16x2(__uint_as_float(o[e + 2]) * inv, __uint_as_float(o[e + 3]) * inv);
            v4.z = pack_bf16x2(__uint_as_float(o[e + 4]) * inv, __uint_as_float(o[e + 5]) * inv);
            v4.w = pack_bf16x2(__uint_as_float(o[e + 6]) * inv, __uint_as_float(o[e + 7]) * inv);
            *reinterpret_cast<uint4*>(orow + cbase + e) = v4;
          }
        }
      }
      if (P.LSE && row_ok && h == 0) P.LSE[qrow] = (m_used * kScaleLog2 + log2f(l_tot)) * 0.6931471805599453f;
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

template <int D, bool SPLIT>
atf_status launch_pipe(const CUtensorMap& tq, const CUtensorMap& tql, const CUtensorMap& tk, const CUtensorMap& tkl,
                       const CUtensorMap& tv, const AtfPipeParams& P, const AtfTable& t, int B, int mode, bool count,
                       cudaStream_t s) {
  const int ntq = (P.N + T - 1) / T;
  const int it0 = (P.N - P.Nq) / T;  // first tile with a query row
  dim3 grid(ntq - it0, P.Hq, B);
  if (mode == ATF_MODE_EXACT)
    atf_pipe_sched_kernel<ATF_MODE_EXACT><<<(ntq + 15) / 16, 128, 0, s>>>(t, D / 2, ntq, P.sched);
  else
    atf_pipe_sched_kernel<ATF_MODE_COARSE><<<(ntq + 15) / 16, 128, 0, s>>>(t, D / 2, ntq, P.sched);
  const int smem = PipeSmem<D, SPLIT>::DYN_BYTES;
#define ATF_PP_LAUNCH(MODE_, COUNT_)                                                                   \
  do {                                                                                                 \
    auto kern = atf_prefill_pipe_kernel<D, MODE_, COUNT_, SPLIT>;                                      \
    ATF_CUDA_CHECK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));     \
    kern<<<grid, PP_THREADS, smem, s>>>(tq, tql, tk, tkl, tv, P, t);                                   \
  } while (0)
  if (mode == ATF_MODE_EXACT) {
    if (count) ATF_PP_LAUNCH(ATF_MODE_EXACT, true); else ATF_PP_LAUNCH(ATF_MODE_EXACT, false);
  } else {
    if (count) ATF_PP_LAUNCH(ATF_MODE_COARSE, true); else ATF_PP_LAUNCH(ATF_MODE_COARSE, false);
  }
#undef ATF_PP_LAUNCH
  ATF_CUDA_CHECK(cudaGetLastError());
  return ATF_OK;
}

}  // namespace

atf_status atf_launch_prefill_pipe(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
                                   const AtfPipeParams& P, const AtfTable& t, int B, int d, int mode, bool count,
                                   cudaStream_t s) {
  return d == 64 ? launch_pipe<64, false>(tq, tq, tk, tk, tv, P, t, B, mode, count, s)
                 : launch_pipe<128, false>(tq, tq, tk, tk, tv, P, t, B, mode, count, s);
}

atf_status atf_launch_prefill_pipe_split(const CUtensorMap& tqh, const CUtensorMap& tql, const CUtensorMap& tkh,
                                         const CUtensorMap& tkl, const CUtensorMap& tv, const AtfPipeParams& P,
                                         const AtfTable& t, int B, int d, int mode, bool count, cudaStream_t s) {
  return d == 64 ? launch_pipe<64, true>(tqh, tql, tkh, tkl, tv, P, t, B, mode, count, s)
                 : launch_pipe<128, true>(tqh, tql, tkh, tkl, tv, P, t, B, mode, count, s);
}
