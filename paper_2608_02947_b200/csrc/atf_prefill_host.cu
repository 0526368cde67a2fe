// atf_prefill_host: the prefill for callers whose tensors live in HOST memory.
//
// The prompt is cut into chunks of query rows.  Chunk c needs its own Q rows and the K/V rows
// up to its end; the K/V rows of earlier chunks are already on the device.  So the host->device
// copy of chunk c+1, the kernels of chunk c and the device->host copy of chunk c-1 run at the
// same time on three streams, and the whole call costs little more than its kernels: a chunk
// is the appended-rows step of atf_prefill_chunk (App. C, "The interval itself"; Sec. 7.3 runs
// long prompts in such chunks), and a prefill cut into chunks is bit-identical to the single shot.
#include <cuda_runtime.h>

#include <algorithm>
#include <vector>

#include "atf_common.cuh"

atf_status atf_prefill_impl(const void* Q, const void* K, const void* V, void* O, float* LSE, int B, int Hq, int Hkv,
                            int64_t Nq, int64_t N, int d, const int64_t* table, int causal, const atf_opts* opts,
                            void* stream, int64_t kv_head_rows);
size_t atf_prefill_workspace_bytes(int B, int Hq, int Hkv, int64_t N, int d);

namespace {

constexpr int64_t DEFAULT_CHUNK = 16384;

size_t align256(size_t b) { return (b + 255) & ~(size_t)255; }

struct HostPlan {
  int64_t chunk;
  size_t ws, kv, qbuf, lbuf, total;
};

HostPlan make_plan(int B, int Hq, int Hkv, int64_t N, int d, int64_t chunk_rows) {
  HostPlan p;
  // chunks start at multiples of the kernel's 128-row tile: a cut inside a tile could change which pass a tile
  // takes (see atf_prefill_chunk) and with it the last bit of a result
  const int64_t want = chunk_rows > 0 ? (chunk_rows + 127) / 128 * 128 : DEFAULT_CHUNK;
  p.chunk = std::min<int64_t>(want, N);
  // workspace of one chunk call: header + repacked Q chunk + repacked K of up to N rows
  p.ws = align256(atf_prefill_workspace_bytes(B, Hq, Hkv, N, d));
  p.kv = align256((size_t)B * Hkv * N * d * 2);
  p.qbuf = align256((size_t)B * Hq * p.chunk * d * 2);
  p.lbuf = align256((size_t)B * Hq * p.chunk * 4);
  p.total = p.ws + 2 * p.kv + 4 * p.qbuf + 2 * p.lbuf;  // K, V; Q x2, O x2; LSE x2
  return p;
}

struct Streams {
  cudaStream_t h2d = nullptr, d2h = nullptr;
};
// One pair of copy streams per device, created at the first call on that device and kept.
atf_status get_streams(Streams** out) {
  static Streams per_dev[64];
  int dev = 0;
  ATF_CUDA_CHECK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return atf_fail(ATF_ERR_UNSUPPORTED, "atf_prefill_host: device index %d", dev);
  Streams& s = per_dev[dev];
  if (!s.h2d) {
    ATF_CUDA_CHECK(cudaStreamCreateWithFlags(&s.h2d, cudaStreamNonBlocking));
    ATF_CUDA_CHECK(cudaStreamCreateWithFlags(&s.d2h, cudaStreamNonBlocking));
  }
  *out = &s;
  return ATF_OK;
}

}  // namespace

extern "C" size_t atf_prefill_host_scratch_bytes(int B, int Hq, int Hkv, int64_t N, int d, int64_t chunk_rows) {
  if ((d != 64 && d != 128) || B < 1 || Hq < 1 || Hkv < 1 || N < 1 || chunk_rows < 0) return 0;
  return make_plan(B, Hq, Hkv, N, d, chunk_rows).total;
}

extern "C" atf_status atf_prefill_host(const void* Qh, const void* Kh, const void* Vh, void* Oh, float* LSEh, int B,
                                       int Hq, int Hkv, int64_t N, int d, const int64_t* table, int causal,
                                       const atf_opts* opts, void* dev_scratch, size_t scratch_bytes,
                                       int64_t chunk_rows, void* stream) {
  if (!Qh || !Kh || !Vh || !Oh) return atf_fail(ATF_ERR_INVALID_ARG, "atf_prefill_host: null host pointer");
  if (d != 64 && d != 128) return atf_fail(ATF_ERR_UNSUPPORTED, "atf_prefill_host: d must be 64 or 128 (got %d)", d);
  if (B < 1 || Hq < 1 || Hkv < 1 || N < 1 || chunk_rows < 0) return atf_fail(ATF_ERR_INVALID_ARG, "atf_prefill_host: bad shape");
  if (Hq % Hkv) return atf_fail(ATF_ERR_INVALID_ARG, "atf_prefill_host: Hq must be a multiple of Hkv");
  if (opts && opts->workspace) return atf_fail(ATF_ERR_INVALID_ARG, "atf_prefill_host: opts->workspace is taken from dev_scratch");
  const HostPlan p = make_plan(B, Hq, Hkv, N, d, chunk_rows);
  if (!dev_scratch) return atf_fail(ATF_ERR_WORKSPACE, "atf_prefill_host: dev_scratch is NULL");
  if ((uintptr_t)dev_scratch & 255) return atf_fail(ATF_ERR_INVALID_ARG, "atf_prefill_host: dev_scratch must be 256-byte aligned");
  if (scratch_bytes < p.total)
    return atf_fail(ATF_ERR_WORKSPACE, "atf_prefill_host: scratch has %zu bytes, needs %zu", scratch_bytes, p.total);
  Streams* st = nullptr;
  atf_status rc = get_streams(&st);
  if (rc != ATF_OK) return rc;
  cudaStream_t comp = (cudaStream_t)stream;

  char* base = (char*)dev_scratch;
  char* ws = base;
  char* Kd = ws + p.ws;
  char* Vd = Kd + p.kv;
  char* Qd[2] = {Vd + p.kv, Vd + p.kv + p.qbuf};
  char* Od[2] = {Qd[1] + p.qbuf, Qd[1] + 2 * p.qbuf};
  char* Ld[2] = {Od[1] + p.qbuf, Od[1] + p.qbuf + p.lbuf};

  atf_opts o = {};
  if (opts) o = *opts;
  o.workspace = ws;
  o.workspace_bytes = p.ws;

  const int64_t nchunks = (N + p.chunk - 1) / p.chunk;
  std::vector<cudaEvent_t> in_ready(nchunks), computed(nchunks), out_done(nchunks);
  cudaEvent_t start_ev;
  auto destroy_all = [&]() {
    for (auto v : {&in_ready, &computed, &out_done})
      for (cudaEvent_t e : *v)
        if (e) cudaEventDestroy(e);
    if (start_ev) cudaEventDestroy(start_ev);
  };
  for (auto v : {&in_ready, &computed, &out_done})
    for (auto& e : *v) e = nullptr;
  start_ev = nullptr;
#define HOST_CHECK(expr)                  \
  do {                                    \
    cudaError_t e_ = (expr);              \
    if (e_ != cudaSuccess) {              \
      destroy_all();                      \
      ATF_CUDA_CHECK(e_);                 \
    }                                     \
  } while (0)
  HOST_CHECK(cudaEventCreateWithFlags(&start_ev, cudaEventDisableTiming));
  for (int64_t c = 0; c < nchunks; ++c) {
    HOST_CHECK(cudaEventCreateWithFlags(&in_ready[c], cudaEventDisableTiming));
    HOST_CHECK(cudaEventCreateWithFlags(&computed[c], cudaEventDisableTiming));
    HOST_CHECK(cudaEventCreateWithFlags(&out_done[c], cudaEventDisableTiming));
  }
  // everything follows the work already queued on the caller's stream
  // the split counters start at zero; the status words are left as they are (the caller zero-fills the
  // header once), so a give-up of an earlier call is still there for atf_check_status
  HOST_CHECK(cudaMemsetAsync(ws + ATF_WS_STATUS_BYTES, 0, ATF_WS_HEADER - ATF_WS_STATUS_BYTES, comp));
  HOST_CHECK(cudaEventRecord(start_ev, comp));
  HOST_CHECK(cudaStreamWaitEvent(st->h2d, start_ev, 0));
  HOST_CHECK(cudaStreamWaitEvent(st->d2h, start_ev, 0));

  const size_t row_bytes = (size_t)d * 2;
  const size_t host_pitch = (size_t)N * row_bytes;  // bytes between two heads in the host tensors and in Kd / Vd
  for (int64_t c = 0; c < nchunks; ++c) {
    const int64_t n0 = c * p.chunk, n1 = std::min<int64_t>(N, n0 + p.chunk), rows = n1 - n0;
    const int b = (int)(c & 1);
    const size_t chunk_bytes = (size_t)rows * row_bytes;
    // ---- host -> device: Q rows of the chunk (dense [B*Hq, rows, d]), K and V rows into the caches ----
    if (c >= 2) HOST_CHECK(cudaStreamWaitEvent(st->h2d, computed[c - 2], 0));  // the Q buffer is free again
    HOST_CHECK(cudaMemcpy2DAsync(Qd[b], chunk_bytes, (const char*)Qh + (size_t)n0 * row_bytes, host_pitch, chunk_bytes,
                                 (size_t)B * Hq, cudaMemcpyHostToDevice, st->h2d));
    HOST_CHECK(cudaMemcpy2DAsync(Kd + (size_t)n0 * row_bytes, host_pitch, (const char*)Kh + (size_t)n0 * row_bytes,
                                 host_pitch, chunk_bytes, (size_t)B * Hkv, cudaMemcpyHostToDevice, st->h2d));
    HOST_CHECK(cudaMemcpy2DAsync(Vd + (size_t)n0 * row_bytes, host_pitch, (const char*)Vh + (size_t)n0 * row_bytes,
                                 host_pitch, chunk_bytes, (size_t)B * Hkv, cudaMemcpyHostToDevice, st->h2d));
    HOST_CHECK(cudaEventRecord(in_ready[c], st->h2d));
    // ---- kernels: the chunk's rows against the n1 keys present ----
    HOST_CHECK(cudaStreamWaitEvent(comp, in_ready[c], 0));
    if (c >= 2) HOST_CHECK(cudaStreamWaitEvent(comp, out_done[c - 2], 0));  // the O / LSE buffers are free again
    rc = atf_prefill_impl(Qd[b], Kd, Vd, Od[b], LSEh ? (float*)Ld[b] : nullptr, B, Hq, Hkv, rows, n1, d, table, causal,
                          &o, comp, N);
    if (rc != ATF_OK) {
      destroy_all();
      return rc;
    }
    HOST_CHECK(cudaEventRecord(computed[c], comp));
    // ---- device -> host: O (and LSE) rows of the chunk ----
    HOST_CHECK(cudaStreamWaitEvent(st->d2h, computed[c], 0));
    HOST_CHECK(cudaMemcpy2DAsync((char*)Oh + (size_t)n0 * row_bytes, host_pitch, Od[b], chunk_bytes, chunk_bytes,
                                 (size_t)B * Hq, cudaMemcpyDeviceToHost, st->d2h));
    if (LSEh)
      HOST_CHECK(cudaMemcpy2DAsync((char*)LSEh + (size_t)n0 * 4, (size_t)N * 4, Ld[b], (size_t)rows * 4, (size_t)rows * 4,
                                   (size_t)B * Hq, cudaMemcpyDeviceToHost, st->d2h));
    HOST_CHECK(cudaEventRecord(out_done[c], st->d2h));
  }
  // the caller's stream is done when the last results are on the host
  HOST_CHECK(cudaStreamWaitEvent(comp, out_done[nchunks - 1], 0));
  if (nchunks >= 2) HOST_CHECK(cudaStreamWaitEvent(comp, out_done[nchunks - 2], 0));
#undef HOST_CHECK
  destroy_all();  // events still in use are released by the driver once they have completed
  return ATF_OK;
}
