// Host-side parts of the atflash library: window table (Eq. 2, Eq. 3, Sec. 3.2), error
// text, workspace binding and the device status word.
#include <cuda.h>

#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <initializer_list>

#include "atf_common.cuh"

static thread_local char g_err[512] = "";
static AtfWorkspace g_ws = {nullptr, 0};
// further places a kernel may have left a status in: the built-in scratch of atf_decode_static, per device
static void* g_extra_status[64] = {nullptr};

void atf_register_status_words(int device, void* dev_ptr) {
  if (device >= 0 && device < 64) g_extra_status[device] = dev_ptr;
}

atf_status atf_fail(atf_status code, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
  return code;
}

AtfWorkspace atf_bound_workspace() { return g_ws; }

// ---- tiled tensor maps for TMA ----
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn) return fn;
  void* p = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess) return nullptr;
  if (qres != cudaDriverEntryPointSuccess) return nullptr;
  fn = (EncodeTiledFn)p;
  return fn;
}

// [BH, N, D] bf16 tensor whose heads are head_rows (>= N) rows apart in memory; box = 64 columns x
// box_rows rows x 1, 128-byte swizzle, zero fill outside.
atf_status atf_make_tile_map(CUtensorMap* m, const void* base, int64_t BH, int64_t N, int D, int64_t head_rows,
                             int box_rows) {
  EncodeTiledFn enc = get_encode_fn();
  if (!enc) return atf_fail(ATF_ERR_CUDA, "cuTensorMapEncodeTiled is not available from this driver");
  cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)N, (cuuint64_t)BH};
  cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)head_rows * D * 2};
  cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return atf_fail(ATF_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);
  return ATF_OK;
}

// Splits of the key range per (batch, KV head) for decode: the smallest split count that fills
// whole waves of the `slots` resident CTAs best, with at least ATF_DECODE_MIN_SPLIT keys per split.
int atf_decode_num_splits(int B, int Hkv, int64_t L, int slots_) {
  const int64_t groups = (int64_t)B * Hkv;
  const int64_t slots = slots_;
  int64_t most = L / ATF_DECODE_MIN_SPLIT;
  if (most < 1) most = 1;
  if (most > 4 * slots) most = 4 * slots;
  double best = -1.0;
  int best_ns = 1;
  for (int64_t ns = 1; ns <= most; ++ns) {
    const int64_t total = groups * ns;
    const int64_t waves = (total + slots - 1) / slots;
    const double eff = (double)total / (double)(waves * slots);
    if (eff > best + 0.02) {
      best = eff;
      best_ns = (int)ns;
    }
  }
  return best_ns;
}

// Checks a caller's table (host, d/2 entries; NULL = full attention) and converts it to the
// int32 form the kernels take.  The live pair set at a distance must be a contiguous
// low-frequency slice (Sec. 3.3), which needs widths that do not decrease with r.
atf_status atf_validate_table(const char* who, const int64_t* table, int d, int64_t N, AtfTable* out) {
  const int h = d / 2;
  for (int r = 0; r < ATF_MAX_PAIRS; ++r) out->w[r] = 0x7FFFFFFF;
  for (int r = 0; r < h; ++r) {
    int64_t w = table ? table[r] : N;
    if (w < 0) return atf_fail(ATF_ERR_INVALID_ARG, "%s: table[%d] is negative", who, r);
    if (table && r > 0 && table[r] < table[r - 1])
      return atf_fail(ATF_ERR_UNSUPPORTED, "%s: table must be non-decreasing in r (entry %d)", who, r);
    if (w > N) w = N;  // distances never exceed N-1, so clipping changes nothing
    out->w[r] = (int32_t)w;
  }
  return ATF_OK;
}

// Waits on a barrier nobody arrives on, with the kernels' own bounded wait but a short limit, and
// reports the give-up the way they do (status word 0 = 1, word 1 = the site).
__global__ void atf_bounded_wait_selftest_kernel(unsigned int* status, unsigned long long limit_ns) {
  __shared__ alignas(8) unsigned long long barmem;
  const uint32_t bar = smem_u32(&barmem);
  if (threadIdx.x == 0) {
    mbar_init(bar, 1);
    mbar_fence_init();
    bool done = mbar_try_wait(bar, 0);
    const unsigned long long t0 = global_timer_ns();
    while (!done && global_timer_ns() - t0 <= limit_ns) {
#pragma unroll 1
      for (int i = 0; i < 64 && !done; ++i) done = mbar_try_wait(bar, 0);
    }
    if (!done) {
      atomicExch(status, 1u);
      atomicExch(status + 1, 99u);
    }
  }
}

// Reads a buffer as 256-byte rows (a K row at d = 128), two rows per warp instruction, lane % 16 = the 16-byte
// chunk of the row; chunks whose bit in `chunkmask` is clear are not read.  Only the time and the DRAM
// counters matter: it shows what leaving out parts of a row saves at DRAM's 128-byte line granularity.
__global__ void __launch_bounds__(256) atf_probe_masked_read_kernel(const uint4* __restrict__ buf, size_t nrows,
                                                                     unsigned chunkmask, unsigned* sink) {
  const int lane = threadIdx.x & 31, c = lane & 15, sub = lane >> 4;
  const bool live = (chunkmask >> c) & 1;
  const size_t warp = (blockIdx.x * (size_t)blockDim.x + threadIdx.x) >> 5;
  const size_t nwarps = ((size_t)gridDim.x * blockDim.x) >> 5;
  const size_t per_warp = (nrows + nwarps - 1) / nwarps;
  const size_t r0 = warp * per_warp, r1 = r0 + per_warp < nrows ? r0 + per_warp : nrows;
  unsigned acc = 0;
  for (size_t r = r0; r + 16 <= r1; r += 16) {
    uint4 v[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      v[i] = make_uint4(0, 0, 0, 0);
      if (live)
        asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                     : "=r"(v[i].x), "=r"(v[i].y), "=r"(v[i].z), "=r"(v[i].w)
                     : "l"(buf + (r + 2 * i + sub) * 16 + c));
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) acc ^= v[i].x ^ v[i].y ^ v[i].z ^ v[i].w;
  }
  if (acc == 0x12345678u) sink[0] = acc;  // keeps the loads alive
}

size_t atf_decode_workspace_bytes(int B, int Hq, int Hkv, int64_t L, int d);
size_t atf_prefill_workspace_bytes(int B, int Hq, int Hkv, int64_t N, int d);
size_t atf_prefill_split_workspace_bytes(int B, int Hq, int Hkv, int64_t N, int d);

extern "C" {

size_t atf_workspace_bytes(int op, int B, int Hq, int Hkv, int64_t N, int d) {
  if (B < 1 || Hq < 1 || Hkv < 1 || N < 1 || (d != 64 && d != 128)) return 0;
  if (op == ATF_OP_PREFILL) return atf_prefill_workspace_bytes(B, Hq, Hkv, N, d);
  if (op == ATF_OP_DECODE) return atf_decode_workspace_bytes(B, Hq, Hkv, N, d);
  if (op == ATF_OP_PREFILL_SPLIT) return atf_prefill_split_workspace_bytes(B, Hq, Hkv, N, d);
  return 0;
}

const char* atf_last_error(void) { return g_err; }

atf_status atf_window_table(double base, int d, double k, int64_t N, const atf_scaling* s,
                            int64_t* w_out, double* theta_out) {
  if (d <= 0 || (d & 1)) return atf_fail(ATF_ERR_INVALID_ARG, "atf_window_table: d must be even and positive (got %d)", d);
  if (N < 1) return atf_fail(ATF_ERR_INVALID_ARG, "atf_window_table: N must be >= 1");
  if (!(k >= 0.0)) return atf_fail(ATF_ERR_INVALID_ARG, "atf_window_table: k must be >= 0 (INFINITY = full attention)");
  if (!(base > 1.0)) return atf_fail(ATF_ERR_INVALID_ARG, "atf_window_table: base must be > 1");
  if (!w_out) return atf_fail(ATF_ERR_INVALID_ARG, "atf_window_table: w_out is NULL");
  if (s && s->kind != 0 && s->kind != 1) return atf_fail(ATF_ERR_UNSUPPORTED, "atf_window_table: unknown scaling kind %d", s->kind);
  if (s && s->kind == 1 &&
      !(s->factor > 0.0 && s->low_freq_factor > 0.0 && s->high_freq_factor > s->low_freq_factor && s->original_ctx > 0 &&
        s->factor < INFINITY && s->high_freq_factor < INFINITY))
    return atf_fail(ATF_ERR_INVALID_ARG,
                    "atf_window_table: llama3 scaling needs factor > 0, 0 < low_freq_factor < high_freq_factor and original_ctx > 0");
  const double two_pi = 2.0 * M_PI;
  const int h = d / 2;
  for (int r = 0; r < h; ++r) {
    double theta = std::pow(base, -2.0 * (double)r / (double)d);
    if (s && s->kind == 1) {
      const double lam = two_pi / theta;
      const double c = (double)s->original_ctx;
      if (lam < c / s->high_freq_factor) {
        // short wavelength: unchanged
      } else if (lam > c / s->low_freq_factor) {
        theta = theta / s->factor;
      } else {
        const double t = (c / lam - s->low_freq_factor) / (s->high_freq_factor - s->low_freq_factor);
        theta = (1.0 - t) * theta / s->factor + t * theta;
      }
    }
    if (theta_out) theta_out[r] = theta;
    const double w = k * (two_pi / theta);
    w_out[r] = (w < (double)N) ? (int64_t)std::floor(w) : N;
  }
  return ATF_OK;
}

atf_status atf_window_table_family(double base, int d, int64_t N, const atf_scaling* s, const atf_window_family* f,
                                   int64_t* w_out, double* theta_out) {
  if (!f) return atf_fail(ATF_ERR_INVALID_ARG, "atf_window_table_family: f is NULL");
  if (f->profile < ATF_PROFILE_CONSTANT || f->profile > ATF_PROFILE_GEOMETRIC)
    return atf_fail(ATF_ERR_INVALID_ARG, "atf_window_table_family: unknown profile %d", f->profile);
  if (!(f->k_hi >= 0.0)) return atf_fail(ATF_ERR_INVALID_ARG, "atf_window_table_family: k_hi must be >= 0");
  if (f->profile != ATF_PROFILE_CONSTANT && !(f->k_lo >= 0.0))
    return atf_fail(ATF_ERR_INVALID_ARG, "atf_window_table_family: k_lo must be >= 0");
  if (f->profile == ATF_PROFILE_GEOMETRIC && !(f->k_lo > 0.0 && f->k_hi > 0.0))
    return atf_fail(ATF_ERR_INVALID_ARG, "atf_window_table_family: the geometric profile needs k_hi, k_lo > 0");
  if (!(f->beta >= 0.0)) return atf_fail(ATF_ERR_INVALID_ARG, "atf_window_table_family: beta must be >= 0");
  if (!(f->nope_fraction >= 0.0 && f->nope_fraction <= 1.0))
    return atf_fail(ATF_ERR_INVALID_ARG, "atf_window_table_family: nope_fraction must be in [0, 1]");
  if (f->gamma != f->gamma || f->a != f->a || f->cap != f->cap)
    return atf_fail(ATF_ERR_INVALID_ARG, "atf_window_table_family: NaN parameter");
  // effective frequencies (and every argument check they share) from the Eq. 3 generator
  double theta_local[ATF_MAX_PAIRS * 4];
  if (d > 0 && d / 2 > ATF_MAX_PAIRS * 4)
    return atf_fail(ATF_ERR_UNSUPPORTED, "atf_window_table_family: d/2 must be <= %d", ATF_MAX_PAIRS * 4);
  atf_status st = atf_window_table(base, d, 1.0, N, s, w_out, theta_local);
  if (st != ATF_OK) return st;
  const double two_pi = 2.0 * M_PI;
  const int h = d / 2;
  const int n_free = (int)std::floor(f->nope_fraction * (double)h + 0.5);
  const bool has_cap = f->cap > 0.0 && f->cap < INFINITY;
  for (int r = 0; r < h; ++r) {
    if (r >= h - n_free) {
      if (theta_out) theta_out[r] = 0.0;
      w_out[r] = N;
      continue;
    }
    const double theta = theta_local[r];
    if (theta_out) theta_out[r] = theta;
    const double lam = two_pi / theta;
    double k_r = f->k_hi;
    if (h > 1 && f->profile == ATF_PROFILE_ARITHMETIC) k_r = f->k_hi - (f->k_hi - f->k_lo) / (double)(h - 1) * (double)r;
    if (h > 1 && f->profile == ATF_PROFILE_GEOMETRIC) k_r = f->k_hi * std::pow(f->k_lo / f->k_hi, (double)r / (double)(h - 1));
    const double lam_g = f->gamma == 1.0 ? lam : std::pow(lam, f->gamma);
    double w = k_r * lam_g + f->a * (double)(r + 1) / (double)h;
    w = w > f->beta ? w : f->beta;  // max(w, beta)
    if (has_cap && f->cap < w) w = f->cap;
    w_out[r] = (w < (double)N) ? (int64_t)std::floor(w) : N;
  }
  return ATF_OK;
}

atf_status atf_bind_workspace(void* dev_ptr, size_t bytes) {
  if (dev_ptr && ((uintptr_t)dev_ptr & 255)) return atf_fail(ATF_ERR_INVALID_ARG, "atf_bind_workspace: pointer must be 256-byte aligned");
  if (dev_ptr && bytes < ATF_WS_HEADER) return atf_fail(ATF_ERR_WORKSPACE, "atf_bind_workspace: workspace smaller than its header");
  g_ws.ptr = dev_ptr;
  g_ws.bytes = dev_ptr ? bytes : 0;
  return ATF_OK;
}

// Reads and clears two status words at `words` (device); *hit receives whether a kernel had given up.
static atf_status read_status_words(void* words, cudaStream_t s, unsigned int* st) {
  st[0] = st[1] = 0;
  ATF_CUDA_CHECK(cudaMemcpyAsync(st, words, 2 * sizeof(unsigned int), cudaMemcpyDeviceToHost, s));
  ATF_CUDA_CHECK(cudaStreamSynchronize(s));
  if (st[0] != 0) {
    ATF_CUDA_CHECK(cudaMemsetAsync(words, 0, 2 * sizeof(unsigned int), s));
    ATF_CUDA_CHECK(cudaStreamSynchronize(s));
  }
  return ATF_OK;
}

atf_status atf_check_status_at(void* workspace, void* stream) {
  if (!workspace) return atf_fail(ATF_ERR_INVALID_ARG, "atf_check_status_at: workspace is NULL");
  unsigned int st[2];
  atf_status rc = read_status_words(workspace, (cudaStream_t)stream, st);
  if (rc != ATF_OK) return rc;
  if (st[0] != 0) return atf_fail(ATF_ERR_TIMEOUT, "a kernel gave up a bounded wait (code %u at site %u)", st[0], st[1]);
  return ATF_OK;
}

atf_status atf_probe_masked_read(const void* buf, size_t bytes, unsigned int chunkmask, void* stream) {
  if (!buf || bytes < (1u << 20) || ((uintptr_t)buf & 255)) return atf_fail(ATF_ERR_INVALID_ARG, "atf_probe_masked_read: need a 256-byte aligned buffer of at least 1 MiB");
  if (!g_ws.ptr) return atf_fail(ATF_ERR_WORKSPACE, "atf_probe_masked_read: no workspace bound");
  atf_probe_masked_read_kernel<<<148 * 8, 256, 0, (cudaStream_t)stream>>>((const uint4*)buf, bytes / 256, chunkmask & 0xFFFFu,
                                                                          (unsigned*)g_ws.ptr + 16);
  ATF_CUDA_CHECK(cudaGetLastError());
  return ATF_OK;
}

atf_status atf_selftest_bounded_wait(unsigned int limit_us, void* stream) {
  if (!g_ws.ptr) return atf_fail(ATF_ERR_WORKSPACE, "atf_selftest_bounded_wait: no workspace bound");
  if (limit_us < 1 || limit_us > 100000) return atf_fail(ATF_ERR_INVALID_ARG, "atf_selftest_bounded_wait: limit must be 1..100000 us");
  atf_bounded_wait_selftest_kernel<<<1, 32, 0, (cudaStream_t)stream>>>((unsigned int*)g_ws.ptr, 1000ull * limit_us);
  ATF_CUDA_CHECK(cudaGetLastError());
  return ATF_OK;
}

atf_status atf_check_status(void* stream) {
  int dev = -1;
  void* extra = (cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < 64) ? g_extra_status[dev] : nullptr;
  if (!g_ws.ptr && !extra) return atf_fail(ATF_ERR_WORKSPACE, "atf_check_status: no workspace bound");
  unsigned int st[2] = {0, 0}, hit[2] = {0, 0};
  for (void* words : {g_ws.ptr, extra}) {
    if (!words) continue;
    atf_status rc = read_status_words(words, (cudaStream_t)stream, st);
    if (rc != ATF_OK) return rc;
    if (st[0] != 0 && hit[0] == 0) {
      hit[0] = st[0];
      hit[1] = st[1];
    }
  }
  if (hit[0] != 0) return atf_fail(ATF_ERR_TIMEOUT, "a kernel gave up a bounded wait (code %u at site %u)", hit[0], hit[1]);
  return ATF_OK;
}

}  // extern "C"
