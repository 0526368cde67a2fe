// atf_rope: half-split rotary embedding in place (Sec. 3.1).  Memory-bound elementwise pass;
// the angle pos*theta_r, its sine/cosine and the rotation are evaluated in fp64 so that the
// result is the correctly rounded bf16 of the exact rotation even at positions ~2^20.
#include "atf_common.cuh"

struct RopeTheta {
  double t[ATF_MAX_PAIRS];
};

// One thread owns 8 consecutive pairs of one row (two 16-byte segments, one per half) and
// walks over the heads assigned to its blockIdx.y, so sincos is evaluated once per (row, pair).
template <int D>
__global__ void __launch_bounds__(256) atf_rope_kernel(__nv_bfloat16* __restrict__ X, int BH, int64_t N, int64_t pos0,
                                                        const __grid_constant__ RopeTheta theta) {
  constexpr int H = D / 2;
  constexpr int CHUNKS = H / 8;  // 16-byte chunks per half row
  const int64_t gid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t n = gid / CHUNKS;
  const int c = (int)(gid % CHUNKS);
  if (n >= N) return;
  double cs[8], sn[8];
  const double pos = (double)(pos0 + n);
#pragma unroll
  for (int i = 0; i < 8; ++i) sincos(pos * theta.t[c * 8 + i], &sn[i], &cs[i]);
  for (int bh = blockIdx.y; bh < BH; bh += gridDim.y) {
    __nv_bfloat16* row = X + ((int64_t)bh * N + n) * D;
    uint4 lo = *reinterpret_cast<const uint4*>(row + c * 8);
    uint4 hi = *reinterpret_cast<const uint4*>(row + H + c * 8);
    const __nv_bfloat16* lp = reinterpret_cast<const __nv_bfloat16*>(&lo);
    const __nv_bfloat16* hp = reinterpret_cast<const __nv_bfloat16*>(&hi);
    uint4 olo, ohi;
    __nv_bfloat16* ol = reinterpret_cast<__nv_bfloat16*>(&olo);
    __nv_bfloat16* oh = reinterpret_cast<__nv_bfloat16*>(&ohi);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const double a = (double)__bfloat162float(lp[i]);
      const double b = (double)__bfloat162float(hp[i]);
      ol[i] = __double2bfloat16(a * cs[i] - b * sn[i]);
      oh[i] = __double2bfloat16(b * cs[i] + a * sn[i]);
    }
    *reinterpret_cast<uint4*>(row + c * 8) = olo;
    *reinterpret_cast<uint4*>(row + H + c * 8) = ohi;
  }
}

// The same rotation on fp32 rows, result kept in fp32 (one rounding from the fp64 rotation): the input of the
// split-precision prefill, whose point is that the rotated values are never rounded to bf16.
template <int D>
__global__ void __launch_bounds__(256) atf_rope_f32_kernel(float* __restrict__ X, int BH, int64_t N, int64_t pos0,
                                                            const __grid_constant__ RopeTheta theta) {
  constexpr int H = D / 2;
  constexpr int CHUNKS = H / 8;
  const int64_t gid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t n = gid / CHUNKS;
  const int c = (int)(gid % CHUNKS);
  if (n >= N) return;
  double cs[8], sn[8];
  const double pos = (double)(pos0 + n);
#pragma unroll
  for (int i = 0; i < 8; ++i) sincos(pos * theta.t[c * 8 + i], &sn[i], &cs[i]);
  for (int bh = blockIdx.y; bh < BH; bh += gridDim.y) {
    float* row = X + ((int64_t)bh * N + n) * D;
    float lo[8], hi[8];
    *reinterpret_cast<float4*>(lo) = *reinterpret_cast<const float4*>(row + c * 8);
    *reinterpret_cast<float4*>(lo + 4) = *reinterpret_cast<const float4*>(row + c * 8 + 4);
    *reinterpret_cast<float4*>(hi) = *reinterpret_cast<const float4*>(row + H + c * 8);
    *reinterpret_cast<float4*>(hi + 4) = *reinterpret_cast<const float4*>(row + H + c * 8 + 4);
    float olo[8], ohi[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const double a = (double)lo[i], b = (double)hi[i];
      olo[i] = (float)(a * cs[i] - b * sn[i]);
      ohi[i] = (float)(b * cs[i] + a * sn[i]);
    }
    *reinterpret_cast<float4*>(row + c * 8) = *reinterpret_cast<const float4*>(olo);
    *reinterpret_cast<float4*>(row + c * 8 + 4) = *reinterpret_cast<const float4*>(olo + 4);
    *reinterpret_cast<float4*>(row + H + c * 8) = *reinterpret_cast<const float4*>(ohi);
    *reinterpret_cast<float4*>(row + H + c * 8 + 4) = *reinterpret_cast<const float4*>(ohi + 4);
  }
}

static atf_status rope_check(const char* who, const void* X, const double* theta, int B, int H, int64_t N, int d,
                             int64_t pos0) {
  if (!X || !theta) return atf_fail(ATF_ERR_INVALID_ARG, "%s: null pointer", who);
  if (d != 64 && d != 128) return atf_fail(ATF_ERR_UNSUPPORTED, "%s: d must be 64 or 128 (got %d)", who, d);
  if (B < 1 || H < 1 || N < 1 || pos0 < 0) return atf_fail(ATF_ERR_INVALID_ARG, "%s: bad shape", who);
  if ((uintptr_t)X & 15) return atf_fail(ATF_ERR_INVALID_ARG, "%s: X must be 16-byte aligned", who);
  return ATF_OK;
}

extern "C" atf_status atf_rope_f32(float* X, int B, int H, int64_t N, int d, const double* theta, int64_t pos0,
                                   void* stream) {
  atf_status st = rope_check("atf_rope_f32", X, theta, B, H, N, d, pos0);
  if (st != ATF_OK) return st;
  RopeTheta th;
  for (int r = 0; r < d / 2; ++r) th.t[r] = theta[r];
  for (int r = d / 2; r < ATF_MAX_PAIRS; ++r) th.t[r] = 0.0;
  const int64_t threads = N * (d / 16);
  const int64_t blocks = (threads + 255) / 256;
  if (blocks > 0x7FFFFFFF) return atf_fail(ATF_ERR_UNSUPPORTED, "atf_rope_f32: N too large");
  const int BH = B * H;
  int gy = 1;
  while (gy < BH && blocks * gy < 148 * 8) gy *= 2;
  if (gy > BH) gy = BH;
  dim3 grid((unsigned)blocks, (unsigned)gy);
  cudaStream_t s = (cudaStream_t)stream;
  if (d == 64)
    atf_rope_f32_kernel<64><<<grid, 256, 0, s>>>(X, BH, N, pos0, th);
  else
    atf_rope_f32_kernel<128><<<grid, 256, 0, s>>>(X, BH, N, pos0, th);
  ATF_CUDA_CHECK(cudaGetLastError());
  return ATF_OK;
}

extern "C" atf_status atf_rope(void* X, int B, int H, int64_t N, int d, const double* theta, int64_t pos0,
                               void* stream) {
  if (!X || !theta) return atf_fail(ATF_ERR_INVALID_ARG, "atf_rope: null pointer");
  if (d != 64 && d != 128) return atf_fail(ATF_ERR_UNSUPPORTED, "atf_rope: d must be 64 or 128 (got %d)", d);
  if (B < 1 || H < 1 || N < 1 || pos0 < 0) return atf_fail(ATF_ERR_INVALID_ARG, "atf_rope: bad shape");
  if ((uintptr_t)X & 15) return atf_fail(ATF_ERR_INVALID_ARG, "atf_rope: X must be 16-byte aligned");
  RopeTheta th;
  for (int r = 0; r < d / 2; ++r) th.t[r] = theta[r];
  for (int r = d / 2; r < ATF_MAX_PAIRS; ++r) th.t[r] = 0.0;
  const int64_t threads = N * (d / 16);
  const int64_t blocks = (threads + 255) / 256;
  if (blocks > 0x7FFFFFFF) return atf_fail(ATF_ERR_UNSUPPORTED, "atf_rope: N too large");
  const int BH = B * H;
  // enough blocks along y to fill the GPU when N is short, few enough to amortise sincos
  int gy = 1;
  while (gy < BH && blocks * gy < 148 * 8) gy *= 2;
  if (gy > BH) gy = BH;
  dim3 grid((unsigned)blocks, (unsigned)gy);
  cudaStream_t s = (cudaStream_t)stream;
  if (d == 64)
    atf_rope_kernel<64><<<grid, 256, 0, s>>>((__nv_bfloat16*)X, BH, N, pos0, th);
  else
    atf_rope_kernel<128><<<grid, 256, 0, s>>>((__nv_bfloat16*)X, BH, N, pos0, th);
  ATF_CUDA_CHECK(cudaGetLastError());
  return ATF_OK;
}
