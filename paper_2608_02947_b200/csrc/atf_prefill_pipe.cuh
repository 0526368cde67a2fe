// Launch interface of the one-tile-per-CTA prefill pipeline (atf_prefill_pipe.cu); the host code of
// atf_prefill.cu (validation, repacking, tensor maps) serves both pipelines.
#pragma once

#include "atf_common.cuh"

struct AtfPipeParams {
  uint32_t* sched;            // band schedule, 8 words per tile distance, ceil(N / 128) distances; written per launch
  const __nv_bfloat16* Qp;     // pair-interleaved copy of Q, [B*Hq, Nq, D] (its bf16 hi part in the split-precision mode)
  const __nv_bfloat16* Qp_lo;  // split-precision mode: the lo part, else unused
  __nv_bfloat16* O;
  float* LSE;
  unsigned long long* kept;
  unsigned int* status;
  int Hq, Hkv;
  int N;   // number of keys; positions 0..N-1
  int Nq;  // number of query rows: the last Nq positions
};

atf_status atf_launch_prefill_pipe(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
                                   const AtfPipeParams& P, const AtfTable& t, int B, int d, int mode, bool count,
                                   cudaStream_t s);
// Split-precision mode: Q and K as hi and lo parts, S = Q_hi K_hi^T + Q_hi K_lo^T + Q_lo K_hi^T.
atf_status atf_launch_prefill_pipe_split(const CUtensorMap& tqh, const CUtensorMap& tql, const CUtensorMap& tkh,
                                         const CUtensorMap& tkl, const CUtensorMap& tv, const AtfPipeParams& P,
                                         const AtfTable& t, int B, int d, int mode, bool count, cudaStream_t s);
