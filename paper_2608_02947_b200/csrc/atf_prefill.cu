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
// Kernel.  One CTA owns 256 query rows of one head as two 128-row tiles, A (rows 256i..) and
// B (the next 128), and walks the key tiles from B's diagonal outwards.  Warp roles:
//   warp 0      TMA producer: Q once, then K (live 64-column blocks only) and V tiles into
//               two-stage rings of 128-byte-swizzled shared memory;
//   warps 1, 2  MMA issuers (one thread each) of tile B and tile A: S_X = Q_X K^T over the live
//               depth into tensor memory, O_X += P_X V with P read from tensor memory;
//   warps 4-7   softmax of tile A, warps 8-11 softmax of tile B: one query row per thread:
//               read S, finish the window rule, mask, online softmax with lazy rescaling of
//               O, write P (bf16) over S in tensor memory.
// S_X of a (query tile, key tile) pair is one 128 x 128 x depth product (a 64-key product costs the
// tensor pipe as much as a 128-key one).  The softmax group turns it into P in two halves of 64
// keys and signals each half, so O_X += P(half 0) V runs while the group works on half 1; after
// O_X += P(half 1) V the issuer writes the next S_X over the same columns.  While a query tile
// waits for that, the warps of the other query tile have the schedulers and the MUFU unit to
// themselves; the two issuers hand each other a token so that their closing batches (the second
// O product and the next S) reach the tensor pipe one after the other, which keeps the two
// query tiles in alternation instead of working and waiting at the same time.
//
// Exact mode (the per-term definition).  For a tile at tile distance D the cells span
// distances [z_min, z_max].  Pairs with w >= z_max are live in every cell: they are the MMA
// depth.  Pairs with w < z_min are dead in every cell.  Pairs in between ("straddling") are
// added per cell on the CUDA cores, only where z <= w.  Because an MMA step covers 8 pairs, the
// pairs of the last step that are not live in every cell are zeroed in the CTA's own copy of
// the Q tile; pairs only die as the distance grows, so the zeroing is monotone.
// Coarse mode: depth = pairs live in any cell of the tile, rounded up to 8; diagonal tile full.
//
// Band schedule (Sec. 3.3: the active pairs of a tile are known statically; Sec. 5: distance
// bands).  What a tile needs depends only on its tile distance and, in exact mode, on which
// quarter of the query rows a warp owns, and it is the same for every CTA of a launch.  A small
// pre-kernel therefore writes one 32-bit word per (tile distance, row quarter) once per launch;
// every role of the main kernel reads its word one step ahead and does no schedule arithmetic.
#include <cuda.h>

#include <cstdlib>

#include "atf_common.cuh"
#include "atf_prefill_pipe.cuh"

namespace {

constexpr int T = 128;              // query rows per tile and key columns per tile
constexpr int BLK_BYTES = T * 128;  // one [128 x 64] bf16 block, 128-byte rows
constexpr int KS = 2, VS = 2;       // ring depths
constexpr int PF_THREADS = 384;
#ifndef ATF_PRODUCER_WARP
#define ATF_PRODUCER_WARP 0
#endif
#ifndef ATF_ORDER_BATCHES
#define ATF_ORDER_BATCHES 1
#endif
// Register budget.  The kernel is compiled for 168 registers per thread (65536 / 384, rounded
// down to a multiple of 8), i.e. 64512 in use at launch.  The producer/MMA warpgroup then
// shrinks to 56 and the two softmax warpgroups grow to 224: 128*56 + 256*224 = 64512 (measured: 72/216
// is 0.5-2 % slower, 40/232 no better, 24/240 slower: the issuer thread starts to spill).  The
// total after the change must not exceed the total at launch, or the growing warps wait for
// registers that never come.
static_assert(128 * 56 + 256 * 224 <= PF_THREADS * 168, "setmaxnreg budget exceeds the launch allocation");
constexpr float RESCALE_THRESHOLD = 8.f;  // log2 units the running max may lag behind

struct PrefillParams {
  const uint32_t* sched;  // band schedule, [tile distance][row quarter], see SchedEntry
  const __nv_bfloat16* Qp;  // pair-interleaved copy of Q, [B*Hq, Nq, D]
  __nv_bfloat16* O;
  float* LSE;
  unsigned long long* kept;
  unsigned int* status;
  int Hq, Hkv;
  int N;   // number of keys; positions 0..N-1
  int Nq;  // number of query rows: the last Nq positions, n0 = N - Nq .. N-1 (Nq = N: whole prefill)
};

template <int D>
struct PrefillSmem {
  static constexpr int NB = D / 64;  // 64-column blocks per tile row
  static constexpr int TILE = NB * BLK_BYTES;
  static constexpr int Q_OFF = 0;  // tile A, then tile B
  static constexpr int K_OFF = Q_OFF + 2 * TILE;
  static constexpr int V_OFF = K_OFF + KS * TILE;
  static constexpr int BAR_OFF = V_OFF + VS * TILE;
  static constexpr int TOTAL = BAR_OFF + 256;
  static constexpr int DYN_BYTES = TOTAL + 1024;  // slack for 1024-byte alignment
};
// barrier slots (8 bytes each) inside the BAR area
// B_SFULL / B_PV0 / B_OFULL / B_QZ: slot + X for query tile X (0 = A, 1 = B); B_PFULL: slot + 2 * X + h
// for key half h of the tile.  B_PV0: the product O_X += P(half 0) V of the step is complete.
// B_ORDER + X: issuer X has issued the closing batch of its step on the current key tile.
// d = 64 only (P has tensor-memory columns of its own there): B_SREAD + X: every softmax warp of tile X holds
// its part of S in registers, the next S may be written; B_PV1 + X: O_X += P(half 1) V of the step is complete.
enum { B_QFULL = 0, B_KFULL = 1, B_KEMPTY = 3, B_VFULL = 5, B_VEMPTY = 7, B_SFULL = 9, B_PV0 = 11, B_PFULL = 13,
       B_OFULL = 17, B_QZ = 19, B_ORDER = 21, B_SREAD = 23, B_PV1 = 25, B_COUNT = 27 };
constexpr int HK = T / 2;  // keys per half tile: S and P are produced and consumed in halves

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

// Band schedule word of (tile distance dt, row quarter wq), tiles of 128 aligned at 0.  The 32
// query rows of quarter wq and the 128 keys of a tile at distance dt span the cell distances
// [zlo, zhi].  w[] is non-decreasing, so the pairs reaching a distance z are r >= r0(z); counted
// from the low-frequency end (p = h - r) the word holds
//   p_all  pairs live in every one of those cells (w >= zhi),
//   p_mid  pairs kept in the MMA for those rows: live at the distance from the quarter's middle
//          row to the tile's middle column, i.e. in most cells (the few cells where such a pair
//          is dead are taken back out; pairs live in only a minority of cells are left out and
//          added where live),
//   p_any  pairs live in some cell (w >= zlo),
// and, the same in all four words of a tile distance (the view of quarter 0, whose rows are
// nearest to the keys: a pair it keeps is in the MMA depth of the whole tile, the rows of the
// other quarters that do not keep it hold a zero in that column of Q),
//   natoms 16-column MMA steps of the S product, nkb 64-column K blocks to load,
//   mask   the tile needs the per-cell causal / dropped-key test,
//   plain  (per quarter) none of mask, per-cell finish, empty S or diagonal tile applies.
// Coarse mode: every quarter gets quarter 0's word; depth = pairs live anywhere in the tile
// rounded up to a group of 8, everything on the diagonal tile.
struct SchedEntry {
  int p_all, p_mid, p_any, natoms, nkb;
  bool mask;
  __device__ __forceinline__ explicit SchedEntry(uint32_t e)
      : p_all(e & 127), p_mid((e >> 7) & 127), p_any((e >> 14) & 127), natoms((e >> 21) & 15), nkb((e >> 25) & 3),
        mask((e >> 27) & 1) {}
  // plain: the quarter's cells need neither the mask nor the per-cell finish, S is not empty and
  // it is not the diagonal tile (so every row already has a reference maximum)
  static __device__ __forceinline__ bool plain(uint32_t e) { return (e >> 28) & 1; }
};

template <int MODE>
__global__ void __launch_bounds__(128)
atf_sched_kernel(const __grid_constant__ AtfTable table, int H, int ndt, uint32_t* __restrict__ out) {
  const int dt = blockIdx.x * blockDim.x + threadIdx.x;
  if (dt >= ndt) return;
  const int Wmax = table.w[H - 1];
  auto first_reaching = [&](int z) {  // first pair r with w[r] >= z
    int r = 0;
    while (r < H && table.w[r] < z) ++r;
    return r;
  };
  uint32_t word[4];
  int natoms = 0, nkb = 1;
  for (int wq = 0; wq < 4; ++wq) {
    const int zlo = dt == 0 ? 0 : dt * T + 32 * wq - (T - 1);
    const int zhi = dt * T + 32 * wq + 31;
    const int zmid = dt == 0 ? 16 * wq + 15 : dt * T + 32 * wq - 48;
    const int p_any = H - first_reaching(zlo), p_mid = H - first_reaching(zmid), p_all = H - first_reaching(zhi);
    if (wq == 0) {
      const int depth = MODE == ATF_MODE_EXACT ? p_mid : (dt == 0 ? H : min(H, (p_any + 7) / 8 * 8));
      natoms = (depth + 7) / 8;
      const int ncols = MODE == ATF_MODE_EXACT ? 2 * p_any : 2 * depth;
      nkb = max(1, (ncols + 63) / 64);
    }
    const bool mask = dt == 0 || (MODE == ATF_MODE_EXACT && (dt + 1) * T - 1 > Wmax);
    const bool plain = !mask && natoms > 0 && dt > 0 && (MODE != ATF_MODE_EXACT || p_all == p_any);
    word[wq] = (uint32_t)p_all | ((uint32_t)p_mid << 7) | ((uint32_t)p_any << 14) | ((uint32_t)natoms << 21) |
               ((uint32_t)nkb << 25) | ((uint32_t)mask << 27) | ((uint32_t)plain << 28);
    if (MODE != ATF_MODE_EXACT) word[wq] = word[0];
  }
  *reinterpret_cast<uint4*>(out + 4 * dt) = make_uint4(word[0], word[1], word[2], word[3]);
}
// 2^x for a pair of values on the FMA pipe (x <= ~8; anything below -126, -inf included, gives
// ~1e-38): round x to the nearest integer n with the 1.5*2^23 trick, evaluate a cubic minimax
// of 2^f on f = x - n in [-0.5, 0.5] (relative error < 8e-5, below the bf16 rounding of P),
// and add n to the exponent field.
#ifndef ATF_POLY_OF_4
#define ATF_POLY_OF_4 1
#endif
constexpr int POLY_OF_4 = ATF_POLY_OF_4;  // of every 4 packed pairs, this many take the polynomial, the rest MUFU
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

// P = 2^(s * scale + neg_m) for the 64 columns of one half of S, packed to bf16 pairs, and their
// fp32 sum.  POLY of every 4 packed pairs take the polynomial (FMA pipe), the rest MUFU.
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
// A half whose exponentials were taken against the row's existing reference maximum is redone
// with its own maximum if their sum is not below this (it also catches infinities and NaNs).
// Far below the fp32 range: O accumulates up to 2^20 such terms times |V|.
constexpr float STALE_REF_GUARD = 1.8446744e19f;  // 2^64

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
__global__ void __launch_bounds__(PF_THREADS, 1)
atf_prefill_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                   const __grid_constant__ CUtensorMap tmV, const __grid_constant__ PrefillParams P,
                   const __grid_constant__ AtfTable table) {
  using SM = PrefillSmem<D>;
  constexpr int H = D / 2;
  constexpr int NB = D / 64;
  constexpr uint32_t TMEM_COLS = 512;
  // Tensor memory: S_A, S_B (128 columns each), O_A, O_B (D columns each).  At d = 128 that is all 512 columns
  // and P (bf16) is written over the S columns it came from, so the next S has to wait for O += P V.  At
  // d = 64 there are 128 columns left: P gets them (64 per query tile), and the next S is issued as soon as
  // the softmax group holds the current one in registers, a whole product earlier.
  constexpr bool FREE_P = D == 64;
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
  __shared__ int sW[ATF_MAX_PAIRS];
  __shared__ int s_abort;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int npt = (P.N + 2 * T - 1) / (2 * T);
  const int ip = npt - 1 - (int)blockIdx.x;  // longest rows first; the grid stops at the pair holding row n0
  const int n0 = P.N - P.Nq;
  const int hq = blockIdx.y, b = blockIdx.z;
  const int bhq = b * P.Hq + hq;
  const int bhk = b * P.Hkv + hq / (P.Hq / P.Hkv);
  const int itA = 2 * ip, itB = 2 * ip + 1;

  if (tid < H) sW[tid] = table.w[tid];
  if (tid == 0) {
    s_abort = 0;
    mbar_init(bar(B_QFULL), 1);
    for (int i = 0; i < KS; ++i) {
      mbar_init(bar(B_KFULL + i), 1);
      mbar_init(bar(B_KEMPTY + i), 8);  // every softmax warp, once it has seen both halves of S of its tile
    }
    for (int i = 0; i < VS; ++i) {
      mbar_init(bar(B_VFULL + i), 1);
      mbar_init(bar(B_VEMPTY + i), 2);  // one arrival per MMA issuer
    }
    for (int x = 0; x < 2; ++x) {
      mbar_init(bar(B_SFULL + x), 1);
      mbar_init(bar(B_PV0 + x), 1);
      mbar_init(bar(B_ORDER + x), 1);
      mbar_init(bar(B_SREAD + x), 4);
      mbar_init(bar(B_PV1 + x), 1);
      for (int h = 0; h < 2; ++h) mbar_init(bar(B_PFULL + 2 * x + h), 4);  // one arrival per softmax warp of the tile
      mbar_init(bar(B_OFULL + x), 1);
      mbar_init(bar(B_QZ + x), 128);
    }
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
  const int Wmax = sW[H - 1];
  // steps of each query tile and number of key tiles walked (identical in every role)
  const int dlim = (Wmax + T - 1) / T + 1;  // first tile distance no pair reaches
  const int nA = min(itA + 1, dlim);
  const int nB = (itB * T < P.N) ? min(itB + 1, dlim) : 0;
  const int Tt = max(nB, nA + 1);
  volatile int* abortp = &s_abort;
  unsigned int fail_site = 0;

  if (warp == ATF_PRODUCER_WARP) {
    // =============================== TMA producer ===============================
    asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
    if (lane == 0) {
      mbar_expect_tx(bar(B_QFULL), 2 * SM::TILE);
      for (int x = 0; x < 2; ++x)
        for (int kb = 0; kb < NB; ++kb)
          // rows before n0 do not exist in Q: the (possibly negative) coordinate reads zero fill there
          tma_load_3d(sQ + x * SM::TILE + kb * BLK_BYTES, &tmQ, bar(B_QFULL), kb * 64, (itA + x) * T - n0, bhq);
      uint32_t e_next = __ldg(P.sched);
      for (int t = 0; t < Tt; ++t) {
        const int j = itB - t;
        // the K columns to load are those of the closer user of this key tile (distance max(t - 1, 0))
        const int nkb = SchedEntry(e_next).nkb;
        if (t >= 1 && t + 1 < Tt) e_next = __ldg(P.sched + 4 * t);
        const int ks = t % KS, vs = t % VS;
        if (!wait_or_abort(bar(B_KEMPTY + ks), ((t / KS) & 1) ^ 1, abortp)) { fail_site = 10; break; }
        mbar_expect_tx(bar(B_KFULL + ks), nkb * BLK_BYTES);
        for (int kb = 0; kb < nkb; ++kb)
          tma_load_3d(sK + ks * SM::TILE + kb * BLK_BYTES, &tmK, bar(B_KFULL + ks), kb * 64, j * T, bhk);
        if (!wait_or_abort(bar(B_VEMPTY + vs), ((t / VS) & 1) ^ 1, abortp)) { fail_site = 11; break; }
        mbar_expect_tx(bar(B_VFULL + vs), SM::TILE);
        for (int kb = 0; kb < NB; ++kb)
          tma_load_3d(sV + vs * SM::TILE + kb * BLK_BYTES, &tmV, bar(B_VFULL + vs), kb * 64, j * T, bhk);
      }
    }
  } else if (warp == 1 || warp == 2) {
    // =============================== MMA issuers ===============================
    // warp 1 serves query tile B, warp 2 query tile A (one thread each).  A tcgen05.mma issue
    // blocks while the tensor pipe's queue is full and a lone thread runs its bookkeeping slowly,
    // so two issuers keep the pipe fed where one could not.
    asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
    if (lane == 0) {
      static_assert(KS == 2 && VS == 2, "stage selection below assumes two-stage rings");
      const int X = warp == 1 ? 1 : 0;
      const int nX = X ? nB : nA;
      const int toff = X ? 0 : 1;  // step v of this query tile works on key tile v + toff
      // Descriptors are built once; an MMA step only adds a constant to the start-address field
      // (16-byte units): K-major operands advance 32 bytes per 16-column step inside a
      // 64-column block and one block per four steps; V advances 16 key rows (2048 bytes).
      const uint64_t dQ = make_smem_desc_sw128(sQ + X * SM::TILE, 16, 1024);
      const uint64_t dK0 = make_smem_desc_sw128(sK, 16, 1024), dK1 = make_smem_desc_sw128(sK + SM::TILE, 16, 1024);
      const uint64_t dV0 = make_smem_desc_sw128(sV, BLK_BYTES, 1024),
                     dV1 = make_smem_desc_sw128(sV + SM::TILE, BLK_BYTES, 1024);
      // S_X = Q_X K(tile)^T over natoms 16-column steps, into the tile's 128 S columns.
      auto issue_qk = [&](int tile, int natoms) {
        const uint64_t k0 = (tile & 1) ? dK1 : dK0;
        const uint32_t tSx = tmem_base + X * T;
        asm volatile(
            "{\n\t"
            ".reg .pred pf, p0, p1, p2, p3, p4, p5, p6, p7;\n\t"
            ".reg .b64 qd, kd;\n\t"
            "setp.eq.u32 pf, %4, 0xffffffff;\n\t"  // false: the first step overwrites S
            "setp.gt.u32 p0, %4, 0;\n\t"
            "setp.gt.u32 p1, %4, 1;\n\t"
            "setp.gt.u32 p2, %4, 2;\n\t"
            "setp.gt.u32 p3, %4, 3;\n\t"
            "setp.gt.u32 p4, %4, 4;\n\t"
            "setp.gt.u32 p5, %4, 5;\n\t"
            "setp.gt.u32 p6, %4, 6;\n\t"
            "setp.gt.u32 p7, %4, 7;\n\t"
            "@p0 tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, pf;\n\t"
            "add.u64 qd, %1, 2;\n\t add.u64 kd, %2, 2;\n\t"
            "@p1 tcgen05.mma.cta_group::1.kind::f16 [%0], qd, kd, %3, p0;\n\t"
            "add.u64 qd, %1, 4;\n\t add.u64 kd, %2, 4;\n\t"
            "@p2 tcgen05.mma.cta_group::1.kind::f16 [%0], qd, kd, %3, p0;\n\t"
            "add.u64 qd, %1, 6;\n\t add.u64 kd, %2, 6;\n\t"
            "@p3 tcgen05.mma.cta_group::1.kind::f16 [%0], qd, kd, %3, p0;\n\t"
            "add.u64 qd, %1, 1024;\n\t add.u64 kd, %2, 1024;\n\t"
            "@p4 tcgen05.mma.cta_group::1.kind::f16 [%0], qd, kd, %3, p0;\n\t"
            "add.u64 qd, %1, 1026;\n\t add.u64 kd, %2, 1026;\n\t"
            "@p5 tcgen05.mma.cta_group::1.kind::f16 [%0], qd, kd, %3, p0;\n\t"
            "add.u64 qd, %1, 1028;\n\t add.u64 kd, %2, 1028;\n\t"
            "@p6 tcgen05.mma.cta_group::1.kind::f16 [%0], qd, kd, %3, p0;\n\t"
            "add.u64 qd, %1, 1030;\n\t add.u64 kd, %2, 1030;\n\t"
            "@p7 tcgen05.mma.cta_group::1.kind::f16 [%0], qd, kd, %3, p0;\n\t"
            "}"
            ::"r"(tSx), "l"(dQ), "l"(k0), "r"(IDESC_QK), "r"((uint32_t)natoms)
            : "memory");
      };
      // O_X (+)= P_X(half h) V(tile, keys 64h..64h+63) over four 16-key steps.  P is read from
      // tensor memory (8 columns per step, at the start of the half's S columns), V through the
      // MN-major descriptor.  `first` marks the very first product of the query tile.
      auto issue_pv = [&](int tile, int h, bool first) {
        const uint64_t v0 = ((tile & 1) ? dV1 : dV0) + (uint64_t)(h * 512);
        const uint32_t tOx = tmem_base + 2 * T + X * D;
        const uint32_t tPx = FREE_P ? tmem_base + 2 * T + 2 * D + X * 64 + h * 32 : tmem_base + X * T + h * HK;
        asm volatile(
            "{\n\t"
            ".reg .pred pf, pt;\n\t"
            ".reg .b64 vd;\n\t"
            ".reg .b32 pa;\n\t"
            "setp.eq.b32 pf, %4, 0;\n\t"  // only the very first step of the tile overwrites O
            "setp.eq.u32 pt, %4, %4;\n\t"
            "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, pf;\n\t"
            "add.u32 pa, %1, 8;\n\t add.u64 vd, %2, 128;\n\t"
            "tcgen05.mma.cta_group::1.kind::f16 [%0], [pa], vd, %3, pt;\n\t"
            "add.u32 pa, %1, 16;\n\t add.u64 vd, %2, 256;\n\t"
            "tcgen05.mma.cta_group::1.kind::f16 [%0], [pa], vd, %3, pt;\n\t"
            "add.u32 pa, %1, 24;\n\t add.u64 vd, %2, 384;\n\t"
            "tcgen05.mma.cta_group::1.kind::f16 [%0], [pa], vd, %3, pt;\n\t"
            "}"
            ::"r"(tOx), "r"(tPx), "l"(v0), "r"(IDESC_PV), "r"((uint32_t)(first ? 1 : 0))
            : "memory");
      };
      // Per step: O += P(half 0) V as soon as the softmax group has signalled that half (it is then
      // working on half 1), O += P(half 1) V, and the next S over the same columns (the tensor pipe
      // executes one thread's products in issue order).
      // A V stage is released by one arrival per issuer; an issuer that has no use for a key
      // tile still accounts for it, once the tile has been loaded (so that the arrival falls
      // into the right phase of the barrier).
      auto skip_v = [&](int t) {
        if (!wait_or_abort(bar(B_VFULL + t % VS), (t / VS) & 1, abortp)) return false;
        mbar_arrive(bar(B_VEMPTY + t % VS));
        return true;
      };
      bool ok = wait_or_abort(bar(B_QFULL), 0, abortp) && wait_or_abort(bar(B_QZ + X), 0, abortp);
      if (!ok) fail_site = 20;
      for (int t = 0; t < toff && ok; ++t) ok = skip_v(t);
      int natoms = 0;
      uint32_t e_next = 0;  // schedule word of the next step, fetched a step ahead
      if (ok && nX > 0) {
        natoms = SchedEntry(__ldg(P.sched)).natoms;
        if (nX > 1) e_next = __ldg(P.sched + 4);
        ok = wait_or_abort(bar(B_KFULL + toff % KS), (toff / KS) & 1, abortp);
        if (ok) {
          tc_fence_after();
          issue_qk(toff, natoms);
          tc_commit(bar(B_SFULL + X));
        } else {
          fail_site = 21;
        }
      }
      for (int v = 0; v < nX && ok; ++v) {
        const int t = v + toff;
        const bool more = v + 1 < nX;
        if (more) {
          natoms = SchedEntry(e_next).natoms;
          if (v + 2 < nX) e_next = __ldg(P.sched + 4 * (v + 2));
        }
        ok = wait_or_abort(bar(B_VFULL + t % VS), (t / VS) & 1, abortp);
        if (more) ok = ok && wait_or_abort(bar(B_KFULL + (t + 1) % KS), ((t + 1) / KS) & 1, abortp);
        if (!ok) { fail_site = 22; break; }
        if (!wait_or_abort(bar(B_PFULL + 2 * X), v & 1, abortp)) { ok = false; fail_site = 23; break; }
        tc_fence_after();
        issue_pv(t, 0, v == 0);
        tc_commit(bar(B_PV0 + X));
        if (FREE_P && more) {
          // the softmax group has S(v) in registers: S(v + 1) can go over it while the group is still at work
          if (!wait_or_abort(bar(B_SREAD + X), v & 1, abortp)) { ok = false; fail_site = 27; break; }
          tc_fence_after();
          issue_qk(t + 1, natoms);
          tc_commit(bar(B_SFULL + X));
        }
        if (!wait_or_abort(bar(B_PFULL + 2 * X + 1), v & 1, abortp)) { ok = false; fail_site = 23; break; }
        // The closing batches of the two query tiles go to the tensor pipe in a fixed order, tile B's
        // for key tile t, tile A's for key tile t, tile B's for t + 1, ...  Issued at the same time
        // they would interleave and both finish late, and the two softmax groups would then work and
        // wait in step with each other; one after the other, each group works while the other waits.
        // A batch is announced only where the other issuer waits for it.
        if (ATF_ORDER_BATCHES && !FREE_P) {
          const bool other_before = X == 0 ? t < nB : (t >= 2 && t - 1 <= nA);  // tile B's batch of t / tile A's of t - 1
          const int tp = X == 0 ? t : t - 1;                                  // its key tile: announcements start at 1
          if (other_before && !wait_or_abort(bar(B_ORDER + (X ^ 1)), (tp - 1) & 1, abortp)) { ok = false; fail_site = 26; break; }
        }
        tc_fence_after();
        issue_pv(t, 1, false);
        if (FREE_P) {
          tc_commit(bar(B_PV1 + X));
          if (!more) tc_commit(bar(B_OFULL + X));
        } else if (more) {
          issue_qk(t + 1, natoms);
          tc_commit(bar(B_SFULL + X));  // S(v + 1) is there, and every product before it is complete
        } else {
          tc_commit(bar(B_OFULL + X));
        }
        if (ATF_ORDER_BATCHES && !FREE_P) {
          const bool other_waits = X == 0 ? t + 1 < nB : (t >= 1 && t <= nA);
          if (other_waits) mbar_arrive(bar(B_ORDER + X));
        }
        tc_commit(bar(B_VEMPTY + t % VS));
      }
      for (int t = toff + nX; t < Tt && ok; ++t) ok = skip_v(t);
      if (!ok && !fail_site) fail_site = 25;
    }
  } else if (warp >= 4) {
    // =============================== softmax groups ===============================
    asm volatile("setmaxnreg.inc.sync.aligned.u32 224;");
    const int X = warp >= 8 ? 1 : 0;
    const int row = tid - (X ? 256 : 128);
    const int itX = X ? itB : itA;
    const int nX = X ? nB : nA;
    const int n = itX * T + row;
    const bool row_ok = n >= n0 && n < P.N;
    const int64_t qrow = (int64_t)bhq * P.Nq + (row_ok ? n - n0 : 0);  // row of Q, O and LSE
    const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t tS = tmem_base + X * T + lane_off;
    const uint32_t tO = tmem_base + 2 * T + X * D + lane_off;
    // where P(half h) goes: columns of its own at d = 64, the first 32 columns of the half's S otherwise
    const uint32_t tP0 = FREE_P ? tmem_base + 2 * T + 2 * D + X * 64 + lane_off : tS;
    constexpr int P_HALF_COLS = FREE_P ? 32 : HK;
    uint8_t* qrow_base = smem_gen + SM::Q_OFF + X * SM::TILE;

    bool ok = wait_or_abort(bar(B_QFULL), 0, abortp);
    if (!ok) fail_site = 30;
    // exact mode keeps/zeroes pairs per quarter of the rows; coarse mode decides per tile (every
    // quarter's schedule word is quarter 0's there)
    const uint32_t* sched = P.sched + (warp & 3);
    int zeroed_from = H;  // pairs p >= zeroed_from are zero in the shared copy of Q_X
    auto zero_q_down_to = [&](int p_keep) {
      if (MODE == ATF_MODE_EXACT && p_keep < zeroed_from) {
        for (int p = p_keep; p < zeroed_from; ++p) {
          const int col = 2 * p;
          *reinterpret_cast<uint32_t*>(qrow_base + (col >> 6) * BLK_BYTES + sw128_offset(row, (col & 63) >> 3) +
                                       (col & 7) * 2) = 0u;
        }
        zeroed_from = p_keep;
        fence_proxy_async_smem();
      }
    };
    uint32_t e_cur = 0;  // schedule word of the step at hand; the next one is fetched a step ahead
    if (ok) {
      e_cur = __ldg(sched);
      zero_q_down_to(SchedEntry(e_cur).p_mid);
      mbar_arrive(bar(B_QZ + X));
    }

    float m_used = -INFINITY, l_run = 0.f;  // m_used in raw score units; -inf until a live cell is seen
    unsigned long long cnt = 0;
    const int zdrop = MODE == ATF_MODE_EXACT ? Wmax : 0x7FFFFFFF;
    const __nv_bfloat16* qsrc = P.Qp + qrow * D;

    // The steps come in two kinds.  Far from the diagonal and from every window boundary a tile
    // needs neither the mask nor the per-cell finish, and the row already has a reference maximum:
    // the exponentials are taken against it directly (any reference gives the same softmax as
    // long as nothing overflows), which saves the row maximum and its dependency in front of the
    // exponentials.  Those "plain" steps are most of a long prompt and run in a loop of their own,
    // kept small so that it stays in the instruction cache; everything else takes the general step
    // below, one step at a time.
    int t = 0;
    int h_enter = 0;  // half at which the general step starts (1: the plain loop handed over its second half)
    bool s_released = false;  // d = 64: the half handed over is no longer in tensor memory
    bool s_seen = false;      // the plain loop has waited for S of the step it hands over
    while (ok) {
      // ---------------- plain steps ----------------
      for (; t < Tt; ++t) {
        const int v = X ? t : t - 1;
        if (v < 1 || v >= nX || !SchedEntry::plain(e_cur)) break;
        const uint32_t e_next = v + 1 < nX ? __ldg(sched + 4 * (v + 1)) : 0u;
        const int ks = t % KS;
        bool handed_over = false;
        if (!wait_or_abort(bar(B_SFULL + X), v & 1, abortp)) { ok = false; fail_site = 36; break; }
        tc_fence_after();
#pragma unroll 1
        for (int h = 0; h < 2; ++h) {
          const int c0 = h * HK;
          float s[HK];
          tc_ld32(tS + c0, reinterpret_cast<uint32_t*>(s));
          tc_ld32(tS + c0 + 32, reinterpret_cast<uint32_t*>(s) + 32);
          tc_wait_ld();
          if (FREE_P && h == 1) {  // all of S(v) is in registers now
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(B_SREAD + X));
          }
          uint32_t pk[HK / 2];
          const float lsum = exp_half<POLY_OF_4>(s, kScaleLog2, -m_used * kScaleLog2, pk);
          if (__any_sync(0xffffffffu, !(lsum < STALE_REF_GUARD))) {
            // The general step redoes this half.  S is still in tensor memory (P has not been stored) unless
            // its columns have just been released (d = 64, second half): then the half is recomputed from Q and K.
            h_enter = h;
            handed_over = true;
            s_seen = true;
            s_released = FREE_P && h == 1;
            break;
          }
          if (h == 1) {  // done with this K tile: both halves of S have been computed
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(B_KEMPTY + ks));
          }
          if (FREE_P && h == 1) {  // the product that read the previous P(half 1) must be complete
            if (!wait_or_abort(bar(B_PV1 + X), (v - 1) & 1, abortp)) { ok = false; fail_site = 38; break; }
          }
          tc_st32(tP0 + h * P_HALF_COLS, pk);
          l_run += lsum;
          if (h == 0) {
            if (COUNT && row_ok) {  // every cell of the tile holds the same pairs (coarse: whole groups of 8, i.e. 8 per MMA step)
              const SchedEntry E(e_cur);
              cnt += (unsigned long long)(MODE == ATF_MODE_EXACT ? E.p_all : min(H, 8 * E.natoms)) * (unsigned long long)T;
            }
            if (MODE == ATF_MODE_EXACT && v + 1 < nX) {
              const int p_keep = SchedEntry(e_next).p_mid;
              zero_q_down_to(p_keep);  // S(v) is complete, and S(v + 1) is not issued before both halves of P are signalled
            }
          }
          tc_wait_st();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar(B_PFULL + 2 * X + h));
        }
        if (handed_over || !ok) break;
        e_cur = e_next;
      }
      if (!ok) break;
      // ---------------- one general step ----------------
      if (t >= Tt) break;
      do {
      const int v = X ? t : t - 1;  // step of this query tile = its tile distance to key tile t
      const bool active = v >= 0 && v < nX;
      const int ks = t % KS;
      if (!active) {
        // The arrival must fall into this use of the stage: the tile is loaded only after the
        // previous use has been released by everyone.
        if (!wait_or_abort(bar(B_KFULL + ks), (t / KS) & 1, abortp)) { ok = false; fail_site = 31; break; }
        if (lane == 0) mbar_arrive(bar(B_KEMPTY + ks));
        break;
      }
      const int dt = v;
      const SchedEntry E(e_cur);
      const uint32_t e_next = v + 1 < nX ? __ldg(sched + 4 * (v + 1)) : 0u;
      const int p_any = E.p_any, p_mid = E.p_mid, p_all = E.p_all, natoms = E.natoms;
      const int zrow = dt * T + row;  // distance from this row to column 0 of the key tile
      const bool straddle = MODE == ATF_MODE_EXACT && p_all < p_any;
      if (straddle) {
        // the finish below reads K from shared memory
        if (!wait_or_abort(bar(B_KFULL + ks), (t / KS) & 1, abortp)) { ok = false; fail_site = 31; break; }
      }

      // (not again for a step the plain loop hands over: at d = 64 the barrier may be a phase further by now)
      if (!s_seen && !wait_or_abort(bar(B_SFULL + X), v & 1, abortp)) { ok = false; fail_site = 32; break; }
      s_seen = false;
      tc_fence_after();
#pragma unroll 1
      for (int h = h_enter; h < 2; ++h) {
        const int c0 = h * HK;  // first key column of this half
        float s[HK];
        if (FREE_P && s_released) {
          // S(v) has been given up already: this half again from Q and K, pair by pair.  A plain step: every
          // cell holds the same pairs (coarse mode: the tile's whole groups of 8), none of them zeroed in Q.
          if (!wait_or_abort(bar(B_KFULL + ks), (t / KS) & 1, abortp)) { ok = false; fail_site = 31; break; }
          const int np = MODE == ATF_MODE_EXACT ? p_all : min(H, 8 * natoms);
#pragma unroll
          for (int c = 0; c < HK; ++c) s[c] = 0.f;
          for (int p = 0; p < np; ++p) {
            const uint32_t qq = *reinterpret_cast<const uint32_t*>(qsrc + 2 * p);
            const float q0 = bf16lo_to_f32(qq), q1 = bf16hi_to_f32(qq);
            const int col = 2 * p;
            const uint32_t kb32 = sK + ks * SM::TILE + (col >> 6) * BLK_BYTES + (col & 7) * 2;
            const int chunk = (col & 63) >> 3;
#pragma unroll
            for (int c = 0; c < HK; ++c) {
              uint32_t kk;
              asm volatile("ld.shared.b32 %0, [%1];" : "=r"(kk) : "r"(kb32 + ((chunk ^ (c & 7)) << 4) + (c0 + c) * 128));
              s[c] = fmaf(q0, bf16lo_to_f32(kk), fmaf(q1, bf16hi_to_f32(kk), s[c]));
            }
          }
          s_released = false;
        } else {
          if (natoms > 0) {
            tc_ld32(tS + c0, reinterpret_cast<uint32_t*>(s));
            tc_ld32(tS + c0 + 32, reinterpret_cast<uint32_t*>(s) + 32);
            tc_wait_ld();
          } else {
#pragma unroll
            for (int c = 0; c < HK; ++c) s[c] = 0.f;
          }
          if (FREE_P && h == 1) {  // all of S(v) is in registers now
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(B_SREAD + X));
          }
        }

        uint32_t pk[HK / 2];  // P (bf16) goes over the first 32 columns of this half of S (column c holds keys 2c, 2c+1)
        float lsum = 0.f, scale_o = 1.f;
        {
          // ---- straddling pairs.  Pairs [p_all, p_mid) went through the MMA: take their term back
          //      out of the cells beyond the pair's window.  Pairs [p_mid, p_any) did not: add their
          //      term in the cells inside the window.  Work in 32-column chunks and skip a chunk when
          //      no row of this warp has such a cell in it. ----
          if (straddle) {
            const int zw_lo = dt * T + (warp & 3) * 32, zw_hi = zw_lo + 31;  // zrow over the warp's rows
            for (int p = p_all; p < p_any; ++p) {
              const int wp = sW[H - 1 - p];
              const bool subtract = p < p_mid;
              // distances of the warp's cells in chunk q (columns c0 + 32q ..) span
              // [zw_lo - c0 - 32q - 31, zw_hi - c0 - 32q]
              bool touched[2];
  #pragma unroll
              for (int q = 0; q < 2; ++q) {
                const int hi = zw_hi - c0 - 32 * q, lo = zw_lo - c0 - 32 * q - 31;
                touched[q] = subtract ? (hi > wp) : (lo <= wp && hi >= 0);
              }
              if (!touched[0] && !touched[1]) continue;
              const uint32_t qq = *reinterpret_cast<const uint32_t*>(qsrc + 2 * p);
              float q0 = bf16lo_to_f32(qq), q1 = bf16hi_to_f32(qq);
              if (subtract) {
                q0 = -q0;
                q1 = -q1;
              }
              const int col = 2 * p;
              // shared-space address of this pair in key row 0 of the tile, one per swizzle phase of the row
              const uint32_t kb32 = sK + ks * SM::TILE + (col >> 6) * BLK_BYTES + (col & 7) * 2;
              const int chunk = (col & 63) >> 3;
              uint32_t base8[8];
  #pragma unroll
              for (int k8 = 0; k8 < 8; ++k8) base8[k8] = kb32 + ((chunk ^ k8) << 4);
              // Cells with column >= jb = zrow - wp are inside the pair's window.  The 0/1 factor of a cell
              // is formed on the FMA pipe as a saturated affine function of its column (the integer and
              // select pipes run at half rate): adding uses sat(c - jb + 1), taking back uses sat(jb - c).
              const float jbf = (float)(zrow - wp - c0);
              const float ca = subtract ? -1.f : 1.f, cb = subtract ? jbf : 1.f - jbf;
  #pragma unroll
              for (int q = 0; q < 2; ++q) {
                if (touched[q]) {
                  // all 32 loads first (same address across the warp: a broadcast), then the arithmetic
                  uint32_t kk[32];
  #pragma unroll
                  for (int cc = 0; cc < 32; ++cc) {
                    const int c = q * 32 + cc;
                    asm volatile("ld.shared.b32 %0, [%1];" : "=r"(kk[cc]) : "r"(base8[c & 7] + (c0 + c) * 128));
                  }
  #pragma unroll
                  for (int cc = 0; cc < 32; ++cc) {
                    const int c = q * 32 + cc;
                    const float term = fmaf(q0, bf16lo_to_f32(kk[cc]), q1 * bf16hi_to_f32(kk[cc]));
                    const float coef = __saturatef(fmaf(ca, (float)c, cb));
                    s[c] = fmaf(term, coef, s[c]);
                  }
                }
              }
            }
          }
          // ---- causal mask, dropped keys (exact mode: per cell) ----
          if (E.mask) {
  #pragma unroll
            for (int c = 0; c < HK; ++c) {
              const int z = zrow - c0 - c;
              s[c] = (z >= 0 && z <= zdrop) ? s[c] : -INFINITY;
            }
          }
          float mx;
          {
            float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
  #pragma unroll
            for (int c = 0; c < HK; c += 8) {
  #pragma unroll
              for (int i = 0; i < 4; ++i) m4[i] = fmaxf(m4[i], fmaxf(s[c + 2 * i], s[c + 2 * i + 1]));
            }
            mx = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
          }
          // lazy rescaling: the reference maximum only moves when it lags by more than the threshold
          // (or when the row sees its first live cell)
          bool moved = false;
          if (mx > m_used && (m_used == -INFINITY || (mx - m_used) * kScaleLog2 > RESCALE_THRESHOLD)) {
            scale_o = m_used == -INFINITY ? 0.f : ex2_approx((m_used - mx) * kScaleLog2);
            m_used = mx;
            moved = !(v == 0 && h == 0);  // nothing has been accumulated before the first half
          }
          if (__any_sync(0xffffffffu, moved)) {  // rare after the first tiles
            // Every product into O issued so far must be complete.  Those of the earlier steps are:
            // S(v) was issued after them.  In the second half, O += P(v, 0) V is on its way too.
            if (h == 1) {
              if (!wait_or_abort(bar(B_PV0 + X), v & 1, abortp)) { ok = false; fail_site = 34; break; }
              tc_fence_after();
            } else if (FREE_P && v > 0) {  // d = 64: S(v) was issued before O += P(v - 1, 1) V
              if (!wait_or_abort(bar(B_PV1 + X), (v - 1) & 1, abortp)) { ok = false; fail_site = 34; break; }
              tc_fence_after();
            }
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
          lsum = exp_half<POLY_OF_4>(s, kScaleLog2, m_used == -INFINITY ? 0.f : -m_used * kScaleLog2, pk);
        }
        if (h == 1) {  // done with this K tile: both halves of S have been computed
          __syncwarp();
          if (lane == 0) mbar_arrive(bar(B_KEMPTY + ks));
        }

        if (FREE_P && h == 1 && v > 0) {  // the product that read the previous P(half 1) must be complete
          if (!wait_or_abort(bar(B_PV1 + X), (v - 1) & 1, abortp)) { ok = false; fail_site = 38; break; }
        }
        tc_st32(tP0 + h * P_HALF_COLS, pk);
        l_run = l_run * scale_o + lsum;

        if (h == 0) {
          if (COUNT && row_ok) {
            const int ncols = dt == 0 ? row + 1 : T;
            // coarse mode: the tile's depth is whole groups of 8 pairs, i.e. 8 per MMA step
            cnt += (unsigned long long)(MODE == ATF_MODE_EXACT ? p_all : min(H, 8 * natoms)) * (unsigned long long)ncols;
            if (MODE == ATF_MODE_EXACT) {
              for (int p = p_all; p < p_any; ++p) {
                const int wp = sW[H - 1 - p];
                const int lo = max(0, zrow - wp), hi = min(T - 1, zrow);
                cnt += (unsigned long long)max(0, hi - lo + 1);
              }
            }
          }
          // Zero the Q columns that stop being live in most cells at the next step: S(v) is complete,
          // and S(v + 1) is not issued before both halves of P are signalled.
          if (MODE == ATF_MODE_EXACT && v + 1 < nX) zero_q_down_to(SchedEntry(e_next).p_mid);
        }
        tc_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(B_PFULL + 2 * X + h));
      }
      e_cur = e_next;
      } while (false);
      ++t;
      h_enter = 0;
    }
    if (ok && nX > 0) {
      if (!wait_or_abort(bar(B_OFULL + X), 0, abortp)) {
        ok = false;
        fail_site = 33;
      }
    }
    if (ok && nX > 0) {
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
  } else {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
  }

  if (fail_site) {
    atomicExch(P.status, 1u);
    atomicExch(P.status + 1, fail_site);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, TMEM_COLS);
}

// ---- host ----
template <int D>
atf_status launch_prefill(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const PrefillParams& P,
                          const AtfTable& t, int B, int mode, bool count, cudaStream_t s) {
  const int npt = (P.N + 2 * T - 1) / (2 * T);
  const int ip0 = (P.N - P.Nq) / (2 * T);  // first tile pair with a query row
  dim3 grid(npt - ip0, P.Hq, B);
  const int smem = PrefillSmem<D>::DYN_BYTES;
#define ATF_PF_LAUNCH(MODE_, COUNT_)                                                                        \
  do {                                                                                                      \
    auto kern = atf_prefill_kernel<D, MODE_, COUNT_>;                                                       \
    ATF_CUDA_CHECK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));          \
    kern<<<grid, PF_THREADS, smem, s>>>(tq, tk, tv, P, t);                                                         \
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

// band schedule: one 16-byte record per tile distance a launch over N keys can meet
static int sched_entries(int64_t N) { return 2 * (int)((N + 2 * T - 1) / (2 * T)) + 1; }
static size_t sched_bytes(int64_t N) { return ((size_t)sched_entries(N) * 32 + 255) & ~(size_t)255; }  // room for either pipeline's records

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
    const int ndt = sched_entries(N);
    if (mode == ATF_MODE_EXACT)
      atf_sched_kernel<ATF_MODE_EXACT><<<(ndt + 127) / 128, 128, 0, s>>>(t, d / 2, ndt, sched);
    else
      atf_sched_kernel<ATF_MODE_COARSE><<<(ndt + 127) / 128, 128, 0, s>>>(t, d / 2, ndt, sched);
  }

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

  {
    static const int pipe = [] { const char* e = getenv("ATF_PREFILL_PIPE"); return e ? atoi(e) : 1; }();
    if (pipe) {
      AtfPipeParams PP;
      PP.sched = sched;
      PP.Qp = Qp;
      PP.O = (__nv_bfloat16*)O;
      PP.LSE = LSE;
      PP.kept = opts ? (unsigned long long*)opts->kept_terms : nullptr;
      PP.status = (unsigned int*)base;
      PP.Hq = Hq;
      PP.Hkv = Hkv;
      PP.N = (int)N;
      PP.Nq = (int)Nq;
      return atf_launch_prefill_pipe(tq, tk, tv, PP, t, B, d, mode, PP.kept != nullptr, s);
    }
  }
  PrefillParams P;
  P.sched = sched;
  P.Qp = Qp;
  P.O = (__nv_bfloat16*)O;
  P.LSE = LSE;
  P.kept = opts ? (unsigned long long*)opts->kept_terms : nullptr;
  P.status = (unsigned int*)base;
  P.Hq = Hq;
  P.Hkv = Hkv;
  P.N = (int)N;
  P.Nq = (int)Nq;
  const bool count = P.kept != nullptr;
  return d == 64 ? launch_prefill<64>(tq, tk, tv, P, t, B, mode, count, s)
                 : launch_prefill<128>(tq, tk, tv, P, t, B, mode, count, s);
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
