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
// A key tile is processed as two halves of 64 keys.  Each half of a query tile's 128 S columns
// is a buffer of its own: when the softmax group has turned S(v, h) into P(v, h) the issuer
// runs O += P(v, h) V(half h) and then S(v + 1, h) into the same columns, while the group is
// already working on the other half.  The softmax groups, which are the busiest unit of the
// kernel (one MUFU exponential per cell), so never wait for a product that is not yet issued.
//
// Exact mode (the per-term definition).  For a tile at tile distance D the cells span
// distances [z_min, z_max].  Pairs with w >= z_max are live in every cell: they are the MMA
// depth.  Pairs with w < z_min are dead in every cell.  Pairs in between ("straddling") are
// added per cell on the CUDA cores, only where z <= w.  Because an MMA step covers 8 pairs, the
// pairs of the last step that are not live in every cell are zeroed in the CTA's own copy of
// the Q tile; pairs only die as the distance grows, so the zeroing is monotone.
// Coarse mode: depth = pairs live in any cell of the tile, rounded up to 8; diagonal tile full.
#include <cuda.h>

#include <cstdlib>

#include "atf_common.cuh"

namespace {

constexpr int T = 128;              // query rows per tile and key columns per tile
constexpr int BLK_BYTES = T * 128;  // one [128 x 64] bf16 block, 128-byte rows
constexpr int KS = 2, VS = 2;       // ring depths
constexpr int PF_THREADS = 384;
#ifndef ATF_PRODUCER_WARP
#define ATF_PRODUCER_WARP 0
#endif
// Register budget.  The kernel is compiled for 168 registers per thread (65536 / 384, rounded
// down to a multiple of 8), i.e. 64512 in use at launch.  The producer/MMA warpgroup then
// shrinks to 56 and the two softmax warpgroups grow to 224: 128*56 + 256*224 = 64512 (measured: 72/216
// is 0.5-2 % slower, 40/232 no better, 24/240 slower: the issuer thread starts to spill).  The
// total after the change must not exceed the total at launch, or the growing warps wait for
// registers that never come.
static_assert(128 * 56 + 256 * 224 <= PF_THREADS * 168, "setmaxnreg budget exceeds the launch allocation");
constexpr float RESCALE_THRESHOLD = 8.f;  // log2 units the running max may lag behind

// Optional timeline tracing (compile with -DATF_TRACE): one CTA stamps %clock64 at a few events
// per half step into a caller-provided device buffer of 16 x 64 words: slots 6 / 7 = one softmax
// warp of tile B before / after its wait for S, slots 10 / 13 = tile B's issuer when it sees P
// and after it has committed the next S.  A stamp costs on the order of 100 clocks, so few are
// kept.  Off in normal builds.
#ifdef ATF_TRACE
#define ATF_STAMP(slot, step) do { if (blockIdx.x == ATF_TRACE_BLOCK && blockIdx.y == 0 && blockIdx.z == 0 && (step) < 64) \
    P.trace[(slot) * 64 + (step)] = clock64(); } while (0)
#else
#define ATF_STAMP(slot, step) do { } while (0)
#endif
#ifndef ATF_TRACE_BLOCK
#define ATF_TRACE_BLOCK 0
#endif
struct PrefillParams {
  long long* trace;
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
// B_SFULL / B_PFULL: slot + 2 * X + h for query tile X (0 = A, 1 = B) and key half h of the tile
enum { B_QFULL = 0, B_KFULL = 1, B_KEMPTY = 3, B_VFULL = 5, B_VEMPTY = 7, B_SFULL = 9, B_PFULL = 13, B_OFULL = 17,
       B_QZ = 19, B_COUNT = 21 };
constexpr int HK = T / 2;  // keys per half tile: S and P are produced and consumed in halves

__global__ void __launch_bounds__(256)
atf_repack_kernel(const __nv_bfloat16* __restrict__ X, __nv_bfloat16* __restrict__ Y, int64_t rows, int D,
                  int64_t n_per_head, int64_t src_head_rows) {
  // one thread writes 8 consecutive output columns (4 pairs) of one row; the source holds
  // src_head_rows rows per head of which the first n_per_head are copied, the result is dense
  const int H = D / 2;
  const int per_row = D / 8;
  const int64_t gid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (gid >= rows * per_row) return;
  const int64_t row = gid / per_row;
  const int t = (int)(gid % per_row);
  const int64_t head = row / n_per_head;
  const __nv_bfloat16* src = X + (head * src_head_rows + (row - head * n_per_head)) * D;
  __align__(16) __nv_bfloat16 out[8];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int p = 4 * t + i;
    out[2 * i] = src[H - 1 - p];
    out[2 * i + 1] = src[D - 1 - p];
  }
  *reinterpret_cast<uint4*>(Y + row * D + 8 * t) = *reinterpret_cast<const uint4*>(out);
}

// Live-pair bookkeeping for a tile at tile distance dt (tiles of 128, aligned at 0): cells
// span distances [zmin, zmax].  w[] is non-decreasing, so the pairs reaching a distance z are
// r >= r0(z), and r0 only grows with dt: the cursors are advanced, never rewound.
struct TileSched {
  // For the 32 query rows of softmax warp wq (0..3) of a tile at tile distance dt, the cells span
  // distances [zlo, zhi].  r_any / r_all: first pair live in some / in every one of those cells.
  // r_mid: first pair kept in the MMA for those rows, i.e. live at the distance from the warp's
  // middle row to the tile's middle column (live in most of the warp's cells).  A pair kept by
  // warp 0 (the rows nearest to the keys) is in the MMA depth of the whole tile; the rows of the
  // other warps that do not keep it hold a zero in that column of Q.
  int r_any = 0, r_mid = 0, r_all = 0;
  __device__ __forceinline__ void advance(const int* w, int H, int dt, int wq) {
    const int zlo = dt == 0 ? 0 : dt * T + 32 * wq - (T - 1);
    const int zhi = dt * T + 32 * wq + 31;
    const int zmid = dt == 0 ? 16 * wq + 15 : dt * T + 32 * wq - 48;
    while (r_any < H && w[r_any] < zlo) ++r_any;
    while (r_mid < H && w[r_mid] < zmid) ++r_mid;
    while (r_all < H && w[r_all] < zhi) ++r_all;
  }
};
// Pairs contracted by the MMA for a tile.  Exact mode: the pairs live in most cells (the few
// cells where a pair of those is dead are subtracted afterwards; pairs live in only a minority
// of the cells are left out and added where live).  Coarse mode: pairs live anywhere in the
// tile, rounded up to a group of 8; everything on the diagonal tile.
template <int MODE>
__device__ __forceinline__ int tile_depth(int H, int p_any, int p_mid, int dt) {
  if (MODE == ATF_MODE_EXACT) return p_mid;
  return dt == 0 ? H : min(H, (p_any + 7) / 8 * 8);
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
  constexpr uint32_t IDESC_QK = make_idesc_bf16(128, HK, 0, 0);
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
  __shared__ int s_nat[2][2];  // MMA depth of query tile X at its next step (by step parity), from its softmax group

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
      mbar_init(bar(B_KEMPTY + i), 256);  // every softmax thread, once it has seen both halves of S of its tile
    }
    for (int i = 0; i < VS; ++i) {
      mbar_init(bar(B_VFULL + i), 1);
      mbar_init(bar(B_VEMPTY + i), 2);  // one arrival per MMA issuer
    }
    for (int x = 0; x < 2; ++x) {
      for (int h = 0; h < 2; ++h) {
        mbar_init(bar(B_SFULL + 2 * x + h), 1);
        mbar_init(bar(B_PFULL + 2 * x + h), 128);
      }
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
      TileSched sc;
      for (int t = 0; t < Tt; ++t) {
        const int j = itB - t;
        const int dnear = max(t - 1, 0);  // the closer user of this key tile
        sc.advance(sW, H, dnear, 0);
        const int depth = tile_depth<MODE>(H, H - sc.r_any, H - sc.r_mid, dnear);
        const int ncols = MODE == ATF_MODE_EXACT ? 2 * (H - sc.r_any) : 2 * depth;
        const int nkb = max(1, (ncols + 63) / 64);
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
      // S_X(half h) = Q_X K(tile, keys 64h..64h+63)^T over natoms 16-column steps, into columns
      // [64h, 64h+64) of the tile's S region; then signal the softmax group.
      auto issue_qk = [&](int tile, int h, int natoms) {
        const uint64_t k0 = ((tile & 1) ? dK1 : dK0) + (uint64_t)(h * 512);
        const uint32_t tSx = tmem_base + X * T + h * HK;
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
        const uint32_t tOx = tmem_base + 2 * T + X * D, tPx = tmem_base + X * T + h * HK;
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
      // Each half of a query tile's S region is its own buffer: as soon as the softmax group has
      // turned S(v, h) into P(v, h), the issuer runs O += P(v, h) V and then S(v + 1, h) into the
      // same columns (the tensor pipe executes one thread's products in issue order), while the
      // group is already working on the other half.  The softmax groups therefore never wait
      // for the tensor pipe as long as it keeps up.
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
      if (ok && nX > 0) {
        TileSched sc0;
        sc0.advance(sW, H, 0, 0);
        natoms = (tile_depth<MODE>(H, H - sc0.r_any, H - sc0.r_mid, 0) + 7) / 8;
        ok = wait_or_abort(bar(B_KFULL + toff % KS), (toff / KS) & 1, abortp);
        if (ok) {
          tc_fence_after();
          issue_qk(toff, 0, natoms);
          tc_commit(bar(B_SFULL + 2 * X));
          issue_qk(toff, 1, natoms);
          tc_commit(bar(B_SFULL + 2 * X + 1));
        } else {
          fail_site = 21;
        }
      }
      for (int v = 0; v < nX && ok; ++v) {
        const int t = v + toff;
        const bool more = v + 1 < nX;
        ok = wait_or_abort(bar(B_VFULL + t % VS), (t / VS) & 1, abortp);
        if (more) ok = ok && wait_or_abort(bar(B_KFULL + (t + 1) % KS), ((t + 1) / KS) & 1, abortp);
        if (!ok) { fail_site = 22; break; }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          if (!wait_or_abort(bar(B_PFULL + 2 * X + h), v & 1, abortp)) { ok = false; fail_site = 23; break; }
          tc_fence_after();
          if (h == 0 && more) natoms = *reinterpret_cast<volatile int*>(&s_nat[X][(v + 1) & 1]);
          if (X == 1) ATF_STAMP(10, 2 * v + h);
          issue_pv(t, h, v == 0 && h == 0);
          if (more) issue_qk(t + 1, h, natoms);
          tc_commit(bar(B_SFULL + 2 * X + h));  // S(v + 1, h) is there, and every product before it is complete
          if (X == 1) ATF_STAMP(13, 2 * v + h);
        }
        if (!ok) break;
        if (!more) tc_commit(bar(B_OFULL + X));
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
    uint8_t* qrow_base = smem_gen + SM::Q_OFF + X * SM::TILE;

    bool ok = wait_or_abort(bar(B_QFULL), 0, abortp);
    if (!ok) fail_site = 30;
    // exact mode keeps/zeroes pairs per warp of rows; coarse mode decides per tile (warp 0's view)
    const int wq = MODE == ATF_MODE_EXACT ? (warp & 3) : 0;
    TileSched sc;
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
    if (ok) {
      sc.advance(sW, H, 0, wq);
      zero_q_down_to(H - sc.r_mid);
      mbar_arrive(bar(B_QZ + X));
    }

    float m_used = -INFINITY, l_run = 0.f;  // m_used in raw score units; -inf until a live cell is seen
    unsigned long long cnt = 0;
    const int zdrop = MODE == ATF_MODE_EXACT ? Wmax : 0x7FFFFFFF;
    const __nv_bfloat16* qsrc = P.Qp + qrow * D;

    for (int t = 0; t < Tt && ok; ++t) {
      const int v = X ? t : t - 1;  // step of this query tile = its tile distance to key tile t
      const bool active = v >= 0 && v < nX;
      const int ks = t % KS;
      if (!wait_or_abort(bar(B_KFULL + ks), (t / KS) & 1, abortp)) { ok = false; fail_site = 31; break; }
      if (!active) {
        mbar_arrive(bar(B_KEMPTY + ks));
        continue;
      }
      const int dt = v;
      const int zmax = (dt + 1) * T - 1;
      const int p_any = H - sc.r_any, p_mid = H - sc.r_mid, p_all = H - sc.r_all;  // cursors already at dt
      const int depth = tile_depth<MODE>(H, p_any, p_mid, dt);
      const int natoms = (depth + 7) / 8;
      const int zrow = dt * T + row;  // distance from this row to column 0 of the key tile
      const int zw_lo = dt * T + (warp & 3) * 32, zw_hi = zw_lo + 31;  // the same over the warp's rows

#pragma unroll 1
      for (int h = 0; h < 2; ++h) {
        const int c0 = h * HK;  // first key column of this half
        if (X == 1 && lane == 0 && (warp & 3) == 2) ATF_STAMP(6, 2 * v + h);
        if (!wait_or_abort(bar(B_SFULL + 2 * X + h), v & 1, abortp)) { ok = false; fail_site = 32; break; }
        tc_fence_after();
        if (X == 1 && lane == 0 && (warp & 3) == 2) ATF_STAMP(7, 2 * v + h);
        float s[HK];
        if (natoms > 0) {
          tc_ld32(tS + c0, reinterpret_cast<uint32_t*>(s));
          tc_ld32(tS + c0 + 32, reinterpret_cast<uint32_t*>(s) + 32);
          tc_wait_ld();
        } else {
#pragma unroll
          for (int c = 0; c < HK; ++c) s[c] = 0.f;
        }
        
        // ---- straddling pairs.  Pairs [p_all, p_mid) went through the MMA: take their term back
        //      out of the cells beyond the pair's window.  Pairs [p_mid, p_any) did not: add their
        //      term in the cells inside the window.  Work in 32-column chunks and skip a chunk when
        //      no row of this warp has such a cell in it. ----
        if (MODE == ATF_MODE_EXACT) {
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
        if (h == 1) mbar_arrive(bar(B_KEMPTY + ks));  // done with this K tile

        // ---- causal mask, dropped keys (exact mode: per cell) ----
        if (dt == 0 || zmax > zdrop) {
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
        float scale_o = 1.f;
        bool moved = false;
        if (mx > m_used && (m_used == -INFINITY || (mx - m_used) * kScaleLog2 > RESCALE_THRESHOLD)) {
          scale_o = m_used == -INFINITY ? 0.f : ex2_approx((m_used - mx) * kScaleLog2);
          m_used = mx;
          moved = !(v == 0 && h == 0);  // nothing has been accumulated before the first half
        }
        if (__any_sync(0xffffffffu, moved)) {  // rare after the first tiles
          // every product issued so far must be complete: the issuer signals the other half's S
          // barrier after each product (S(v, 1) follows P(v-1, 1) V; S(v+1, 0) follows P(v, 0) V)
          const int vo = h == 0 ? v : v + 1;
          if (!wait_or_abort(bar(B_SFULL + 2 * X + (h ^ 1)), vo & 1, abortp)) { ok = false; fail_site = 34; break; }
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
        const float neg_m = m_used == -INFINITY ? 0.f : -m_used * kScaleLog2;
        const float2 sc2 = make_float2(kScaleLog2, kScaleLog2), nm2 = make_float2(neg_m, neg_m);
        float2 acc[4] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
        // ---- P (bf16) over the first 32 columns of this half of S (column c holds keys 2c and 2c+1) ----
        uint32_t pk[HK / 2];
#pragma unroll
        for (int c = 0; c < HK; c += 2) {
          float2 x = __ffma2_rn(make_float2(s[c], s[c + 1]), sc2, nm2);
          if (((c >> 1) & 3) < POLY_OF_4) {
            x = exp2_poly2(x);
          } else {
            x.x = ex2_approx(x.x);
            x.y = ex2_approx(x.y);
          }
          acc[(c >> 1) & 3] = __fadd2_rn(acc[(c >> 1) & 3], x);
          pk[c >> 1] = pack_bf16x2(x.x, x.y);
        }
        tc_st32(tS + c0, pk);
        {
          const float2 a01 = __fadd2_rn(acc[0], acc[1]), a23 = __fadd2_rn(acc[2], acc[3]);
          l_run = l_run * scale_o + ((a01.x + a01.y) + (a23.x + a23.y));
        }
        
        if (h == 0) {
          if (COUNT && row_ok) {
            const int ncols = dt == 0 ? row + 1 : T;
            cnt += (unsigned long long)(MODE == ATF_MODE_EXACT ? p_all : depth) * (unsigned long long)ncols;
            if (MODE == ATF_MODE_EXACT) {
              for (int p = p_all; p < p_any; ++p) {
                const int wp = sW[H - 1 - p];
                const int lo = max(0, zrow - wp), hi = min(T - 1, zrow);
                cnt += (unsigned long long)max(0, hi - lo + 1);
              }
            }
          }
          // Zero the Q columns that stop being live in most cells at the next step.  S(v + 1, 0) is
          // issued once this half of P is signalled, so the zeroing has to happen here; S(v, 1) still
          // needs the columns, so wait until it has been computed (it was issued long ago).
          if (v + 1 < nX) {
            sc.advance(sW, H, dt + 1, wq);
            if ((warp & 3) == 0 && lane == 0)  // this warp's view (wq = 0) is the depth of the whole tile
              s_nat[X][(v + 1) & 1] = (tile_depth<MODE>(H, H - sc.r_any, H - sc.r_mid, dt + 1) + 7) / 8;
            if (MODE == ATF_MODE_EXACT && H - sc.r_mid < zeroed_from) {
              if (!wait_or_abort(bar(B_SFULL + 2 * X + 1), v & 1, abortp)) { ok = false; fail_site = 35; break; }
              zero_q_down_to(H - sc.r_mid);
            }
          }
        }
        tc_wait_st();
        tc_fence_before();
        mbar_arrive(bar(B_PFULL + 2 * X + h));
      }
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
atf_status make_tile_map(CUtensorMap* m, const void* base, int64_t BH, int64_t N, int D, int64_t head_rows = 0) {
  if (head_rows == 0) head_rows = N;  // rows between two heads in memory (>= N)
  EncodeTiledFn enc = get_encode_fn();
  if (!enc) return atf_fail(ATF_ERR_CUDA, "cuTensorMapEncodeTiled is not available from this driver");
  cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)N, (cuuint64_t)BH};
  cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)head_rows * D * 2};
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

// With -DATF_TRACE the caller passes a device buffer address for the timeline in ATF_TRACE_PTR.
static void* getenv_trace_ptr() {
#ifdef ATF_TRACE
  const char* e = getenv("ATF_TRACE_PTR");
  return e ? (void*)strtoull(e, nullptr, 0) : nullptr;
#else
  return nullptr;
#endif
}

size_t atf_prefill_workspace_bytes(int B, int Hq, int Hkv, int64_t N, int d) {
  return ATF_WS_HEADER + repack_bytes(B, Hq, N, d) + repack_bytes(B, Hkv, N, d);
}
static size_t prefill_chunk_workspace_bytes(int B, int Hq, int Hkv, int64_t Nq, int64_t N, int d) {
  return ATF_WS_HEADER + repack_bytes(B, Hq, Nq, d) + repack_bytes(B, Hkv, N, d);
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
  __nv_bfloat16* Qp = (__nv_bfloat16*)(base + ATF_WS_HEADER);
  __nv_bfloat16* Kp = (__nv_bfloat16*)(base + ATF_WS_HEADER + repack_bytes(B, Hq, Nq, d));
  cudaStream_t s = (cudaStream_t)stream;

  {
    const int64_t rows_q = (int64_t)B * Hq * Nq, rows_k = (int64_t)B * Hkv * N;
    const int64_t bq = (rows_q * (d / 8) + 255) / 256, bk = (rows_k * (d / 8) + 255) / 256;
    if (bq > 0x7FFFFFFF) return atf_fail(ATF_ERR_UNSUPPORTED, "atf_prefill: problem too large for the repack grid");
    atf_repack_kernel<<<(unsigned)bq, 256, 0, s>>>((const __nv_bfloat16*)Q, Qp, rows_q, d, Nq, Nq);
    atf_repack_kernel<<<(unsigned)bk, 256, 0, s>>>((const __nv_bfloat16*)K, Kp, rows_k, d, N, kv_head_rows);
    ATF_CUDA_CHECK(cudaGetLastError());
  }

  CUtensorMap tq, tk, tv;
  if ((st = make_tile_map(&tq, Qp, (int64_t)B * Hq, Nq, d)) != ATF_OK) return st;
  if ((st = make_tile_map(&tk, Kp, (int64_t)B * Hkv, N, d)) != ATF_OK) return st;
  if ((st = make_tile_map(&tv, V, (int64_t)B * Hkv, N, d, kv_head_rows)) != ATF_OK) return st;

  PrefillParams P;
  P.trace = (long long*)getenv_trace_ptr();
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
