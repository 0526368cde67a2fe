/*
 * atflash.h - C ABI of the B200 (sm_100a) library for causal GQA attention with
 * per-RoPE-wavelength distance windows.
 *
 * The score of query position n against key position m (distance z = n - m >= 0) is the sum
 * over RoPE frequency pairs r of the pair's contribution (paper Eq. 1); pair r is kept only
 * while z <= w_r, w_r = min(k * lambda_r, N), lambda_r = 2*pi / theta_r (Eq. 2, Eq. 3).
 * Softmax, the P*V product and the online-softmax recurrence are the usual ones (Sec. 3.3).
 *
 * Conventions shared by every entry point
 *   - All tensors are contiguous, row-major, with the shapes given below; bf16 unless stated.
 *   - "dev" pointers are CUDA device pointers, "host" pointers are ordinary host memory.
 *   - The caller owns every buffer.  The library allocates no device memory; scratch comes
 *     from the workspace the caller binds with atf_bind_workspace().
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls are
 *     asynchronous with respect to the host unless stated.
 *   - Every function returns an atf_status; nothing throws or aborts.  Arguments are checked
 *     on the host before any launch.  atf_last_error() gives a text for the last failure of
 *     the calling thread.
 *   - Head dimension d is 64 or 128; Hq must be a multiple of Hkv; query head hq reads KV head
 *     hq / (Hq/Hkv).  The softmax scale is 1/sqrt(d) (Eq. 1).  Pair r is dims (r, r + d/2)
 *     ("half-split" RoPE layout).
 */
#ifndef ATFLASH_H
#define ATFLASH_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int atf_status;
enum {
  ATF_OK = 0,
  ATF_ERR_INVALID_ARG = 1, /* null pointer, bad shape, malformed table                      */
  ATF_ERR_UNSUPPORTED = 2, /* valid request the library does not implement                   */
  ATF_ERR_CUDA = 3,        /* a CUDA runtime/driver call failed (text in atf_last_error)      */
  ATF_ERR_WORKSPACE = 4,   /* no workspace bound, or it is too small for this call            */
  ATF_ERR_TIMEOUT = 5      /* a bounded device-side wait ran out during an earlier launch; only
                              atf_check_status / atf_check_status_at report it, and the results
                              of that launch are not valid                                     */
};

/* Modes (second argument of the *_ex calls).
 * ATF_MODE_EXACT : the per-term definition (the predicate under Eq. 3 applied to every term).
 * ATF_MODE_COARSE: the granularity the paper's ports run at (Sec. 3.3, Sec. 5, App. E).
 *   Prefill: the live pair set is chosen per (128-query, 128-key) tile from the tile's nearest
 *   cell and rounded outward to whole groups of 8 pairs counted from the low-frequency end;
 *   the tile on the diagonal uses every pair.  Decode: per key, the first live pair is rounded
 *   down to a multiple of 8 pairs (one 16-byte load per half row).                           */
enum { ATF_MODE_EXACT = 0, ATF_MODE_COARSE = 1 };

/* RoPE frequency scaling (Sec. 3.2: the table is built from the effective frequencies).
 * kind 0: none.  kind 1: llama3-style - with lambda = 2*pi/theta and c = original_ctx, a pair
 * with lambda < c/high_freq_factor keeps theta, one with lambda > c/low_freq_factor gets
 * theta/factor, and in between theta' = (1-t)*theta/factor + t*theta with
 * t = (c/lambda - low_freq_factor) / (high_freq_factor - low_freq_factor).                   */
typedef struct {
  int kind;
  double factor, low_freq_factor, high_freq_factor;
  int64_t original_ctx;
} atf_scaling;

/* Layout of the K cache handed to atf_decode_ex.
 * ATF_KLAYOUT_ROWS  : [B, Hkv, L, d], the layout of K in atf_prefill (default).
 * ATF_KLAYOUT_GROUPS: [B, Hkv, T, d/16, KT, 16] as written by atf_kcache_pack or by a prefill with
 *   atf_opts.kcache_groups: the keys are cut into T = ceil(L/KT) tiles of KT =
 *   atf_kcache_tile_keys(d) keys (16 KiB per tile); inside a tile, group j holds, for each of its
 *   keys, the 8 pairs r = d/2-1-8j ... d/2-8-8j (lowest frequency first), each pair as (dim r,
 *   dim r + d/2) side by side; for keys whose index in the tile has bit 2 set the two 16-byte
 *   halves of that 32-byte entry are swapped (the copied image is then free of shared-memory
 *   bank conflicts).  The pairs a far key keeps (a low-frequency slice, Sec. 3.3) are the
 *   leading groups, i.e. a contiguous prefix of the tile, so decode fetches only live bytes, with
 *   one bulk copy per tile; in the row layout DRAM's 128-byte lines make it fetch every row
 *   whole.  This layout is an extension: the paper's ports keep the row layout.             */
enum { ATF_KLAYOUT_ROWS = 0, ATF_KLAYOUT_GROUPS = 1 };

/* Optional arguments of the *_ex calls.  Zero-initialise, then set what is needed. */
typedef struct {
  int mode;              /* ATF_MODE_EXACT or ATF_MODE_COARSE                                  */
  uint64_t* kept_terms;  /* dev, [B*Hq] or NULL.  If set, the kernel ADDS to entry b*Hq+hq the
                            number of (cell, pair) inner-product terms it executed for that head
                            (Sec. 4 cost measure); the caller zeroes it beforehand.             */
  float* lse;            /* decode only: dev, [B*Hq] fp32 natural-log LSE, or NULL              */
  void* workspace;       /* dev scratch for this call, or NULL to use the bound workspace       */
  size_t workspace_bytes;
  int k_layout;          /* decode only: ATF_KLAYOUT_ROWS (default) or ATF_KLAYOUT_GROUPS        */
  void* kcache_groups;   /* prefill only: dev, a group-major K cache (ATF_KLAYOUT_GROUPS) of
                            kcache_capacity keys per (batch, KV head), or NULL.  If set, the prefill
                            also writes the K rows of this call's new positions (N-Nq .. N-1; all
                            of them for atf_prefill) into it, so that decode can read the cache
                            the prefill wrote with no conversion pass (Sec. 7.2).               */
  int64_t kcache_capacity; /* keys the group-major cache is laid out for, >= N (its tile count fixes the
                              layout).  Decode with ATF_KLAYOUT_GROUPS reads it too: 0 = exactly L.    */
  const void* rope_tables; /* decode with ATF_KLAYOUT_GROUPS only: dev, the tables atf_rope_tables wrote, or
                              NULL.  If set, Kcache holds UNROTATED keys (position-independent, App. B)
                              and the kernel rotates the pairs it fetches while it reads them.      */
  int64_t rope_tables_capacity; /* the capacity the tables were built for, >= L                       */
} atf_opts;

/* Window table (Eq. 2, Eq. 3; effective frequencies per Sec. 3.2).  Host only, no GPU needed.
 *   theta_r = base^(-2r/d) in IEEE double, scaled per `s` (NULL = none);
 *   w_out[r] = floor(min(k * 2*pi/theta'_r, N)) for r in [0, d/2): the predicate "z <= w_r" on
 *   integer distances only sees the integer part.  k = INFINITY gives w_out[r] = N.
 *   theta_out (host, d/2 doubles) receives theta'_r if not NULL (the input atf_rope wants).
 * Errors: ATF_ERR_INVALID_ARG for d odd or <= 0, N < 1, k < 0 or NaN, null w_out, or llama3
 *   scaling without factor > 0, 0 < low_freq_factor < high_freq_factor and original_ctx > 0.  */
atf_status atf_window_table(double base, int d, double k, int64_t N, const atf_scaling* s,
                            int64_t* w_out, double* theta_out);

/* The window family of App. A (its Eq. for w_r):
 *   w_r = min(max(k_r * lambda'_r^gamma + a * (r+1)/(d/2), beta), cap),  W_r = floor(min(w_r, N)).
 * k_r is the retention profile over the pair index r = 0 (highest frequency) .. d/2-1:
 *   ATF_PROFILE_CONSTANT    k_r = k_hi;
 *   ATF_PROFILE_ARITHMETIC  k_r = k_hi - (k_hi - k_lo)/(d/2-1) * r   (16 -> 2: the variable-k profile);
 *   ATF_PROFILE_GEOMETRIC   k_r = k_hi * (k_lo/k_hi)^(r/(d/2-1)).
 * cap <= 0 or INFINITY: no ceiling other than N.  nope_fraction: that share of the pairs, from the
 * low-frequency end, rounded to the nearest whole pair, is position-free: theta_out[r] = 0 (atf_rope
 * then leaves the pair unrotated) and w_out[r] = N.  {CONSTANT, k_hi = k, gamma = 1, beta = 0,
 * cap = 0, a = 0, nope_fraction = 0} is atf_window_table, bit for bit.
 * The table may come out non-monotone in r (e.g. a steep profile or a negative a); the attention
 * entry points accept only non-decreasing tables and return ATF_ERR_UNSUPPORTED otherwise.
 * Errors: as atf_window_table, plus ATF_ERR_INVALID_ARG for f NULL, an unknown profile, k_hi < 0,
 * k_lo < 0 (k_lo <= 0 with the geometric profile), beta < 0, nope_fraction outside [0, 1], NaNs.  */
enum { ATF_PROFILE_CONSTANT = 0, ATF_PROFILE_ARITHMETIC = 1, ATF_PROFILE_GEOMETRIC = 2 };
typedef struct {
  int profile;
  double k_hi, k_lo;     /* k_lo is ignored by the constant profile */
  double gamma;          /* wavelength exponent */
  double beta;           /* floor, tokens */
  double cap;            /* ceiling, tokens; <= 0 or INFINITY = none */
  double a;              /* coefficient of the term linear in the pair index */
  double nope_fraction;  /* share of position-free pairs at the low-frequency end */
} atf_window_family;
atf_status atf_window_table_family(double base, int d, int64_t N, const atf_scaling* s,
                                   const atf_window_family* f, int64_t* w_out, double* theta_out);

/* Half-split rotary embedding, in place (Sec. 3.1).
 *   X: dev bf16 [B, H, N, d]; row n is rotated by the angle (pos0 + n) * theta[r] in pair r:
 *   x'_r = x_r cos - x_{r+d/2} sin,  x'_{r+d/2} = x_{r+d/2} cos + x_r sin.
 *   theta: host, d/2 doubles.  Angles and the rotation are evaluated in fp64 and rounded once
 *   to bf16, so positions up to 2^20 and beyond keep full accuracy.                           */
atf_status atf_rope(void* X, int B, int H, int64_t N, int d, const double* theta, int64_t pos0,
                    void* stream);

/* Prefill: windowed causal attention for all N query rows (Sec. 3.3, Fig. 3).
 *   Q, O: dev bf16 [B, Hq, N, d];  K, V: dev bf16 [B, Hkv, N, d];  Q and K already rotated.
 *   LSE: dev fp32 [B, Hq, N], natural log of the sum of exp(scaled score); may be NULL.
 *   table: host int64 [d/2] from atf_window_table, non-decreasing in r and >= 0;
 *          NULL = full attention (identical, bit for bit, to a table whose entries are all N).
 *   A key with no live pair at all (z greater than every w_r) is dropped from the softmax.
 *   causal must be 1: the paper defines the distance only for causal attention; 0 returns
 *   ATF_ERR_UNSUPPORTED.  Needs a workspace of atf_workspace_bytes(ATF_OP_PREFILL, ...).
 *   atf_prefill == atf_prefill_ex with opts = NULL (exact mode, no counters).                 */
atf_status atf_prefill(const void* Q, const void* K, const void* V, void* O, float* LSE, int B,
                       int Hq, int Hkv, int64_t N, int d, const int64_t* table, int causal,
                       void* stream);
atf_status atf_prefill_ex(const void* Q, const void* K, const void* V, void* O, float* LSE, int B,
                          int Hq, int Hkv, int64_t N, int d, const int64_t* table, int causal,
                          const atf_opts* opts, void* stream);

/* Appended rows: the context already holds keys 0..N-Nq-1; the Nq new query rows sit at the
 * positions N-Nq..N-1 and attend to all N keys.  This is the row interval [n0, n1] of App. C
 * ("The interval itself"), whose two end points are the whole prefill and the decode step, and
 * the chunked prefill of Sec. 7.3.  Every row gets exactly what atf_prefill gives it at that
 * position of a length-N prompt, so a prefill cut into chunks has the bits of the single shot.
 * (One exception, rounding-sized: a 128-row tile whose logits rise more than ~120 log2 units above
 * its diagonal maximum is recomputed with a running maximum; if a cut falls INSIDE such a tile and the
 * rows that trigger it lie before the cut, the rows after it differ from the single shot in the last
 * bit of P.  Cuts at multiples of 128, as atf_prefill_host makes, never do.)
 *   Q, O: dev bf16 [B, Hq, Nq, d];  LSE: dev fp32 [B, Hq, Nq] or NULL;
 *   K, V: dev bf16 [B, Hkv, N, d], rotated at positions 0..N-1;  1 <= Nq <= N (else
 *   ATF_ERR_INVALID_ARG).  table, causal, opts, workspace, errors: as atf_prefill; the table's
 *   entries are clipped at N, the number of keys.  opts->kept_terms counts the Nq rows only.
 *   Workspace: atf_workspace_bytes(ATF_OP_PREFILL, ..., N, d) is enough for any Nq <= N.       */
atf_status atf_prefill_chunk(const void* Q, const void* K, const void* V, void* O, float* LSE,
                             int B, int Hq, int Hkv, int64_t Nq, int64_t N, int d,
                             const int64_t* table, int causal, void* stream);
atf_status atf_prefill_chunk_ex(const void* Q, const void* K, const void* V, void* O, float* LSE,
                                int B, int Hq, int Hkv, int64_t Nq, int64_t N, int d,
                                const int64_t* table, int causal, const atf_opts* opts,
                                void* stream);

/* Prefill from and to HOST memory.  Same arguments and results as atf_prefill_ex, but Qh, Kh, Vh,
 * Oh (bf16) and LSEh (fp32 or NULL) are HOST pointers, [B,H,N,d] / [B,Hq,N] dense.  The prompt is
 * processed in chunks of chunk_rows query rows (rounded up to a multiple of 128; 0 = 16384) as successive appended-rows steps
 * (see atf_prefill_chunk; bit-identical to the single shot for every chunk size), so that the
 * host->device copy of the next chunk, the kernels of this one and the device->host copy of the
 * previous one overlap on three streams.  Page-locked host buffers are needed for that overlap;
 * pageable ones work but serialise.
 *   dev_scratch: device memory, 256-byte aligned, at least atf_prefill_host_scratch_bytes(...)
 *   bytes (the K/V caches, two Q / O / LSE chunk buffers and the prefill workspace; its first
 *   bytes are a workspace header, which the caller zero-fills once: atf_check_status_at, or
 *   atf_check_status after binding it with atf_bind_workspace, reads the kernels' status
 *   there).  opts->workspace must be NULL.  The library allocates no
 *   device memory; it creates two copy streams per device at the first call and keeps them.
 *   The call returns once everything is queued; `stream` (and the host results) are complete when
 *   the caller has synchronised `stream`.  Work already queued on `stream` is waited for.
 * Errors: as atf_prefill_ex; ATF_ERR_WORKSPACE if the scratch is missing or too small.           */
size_t atf_prefill_host_scratch_bytes(int B, int Hq, int Hkv, int64_t N, int d, int64_t chunk_rows);
atf_status atf_prefill_host(const void* Qh, const void* Kh, const void* Vh, void* Oh, float* LSEh,
                            int B, int Hq, int Hkv, int64_t N, int d, const int64_t* table,
                            int causal, const atf_opts* opts, void* dev_scratch,
                            size_t scratch_bytes, int64_t chunk_rows, void* stream);

/* Decode: one new query token per sequence against a contiguous KV cache (Sec. 5; the last
 * row of Fig. 3).  The cache already contains the new token; the query sits at position L-1,
 * so key m is at distance z = L-1-m.
 *   q, O: dev bf16 [B, Hq, d];  Kcache, Vcache: dev bf16 [B, Hkv, L, d] (the layout of K and V
 *   in atf_prefill, so a prefill cache is read with no conversion).
 *   What is read: V rows in full.  K in this row layout: every row in full (a key no pair reaches
 *   is skipped) with the dead pairs masked on chip - each 128-byte half of a row ends in live
 *   low-frequency pairs and DRAM moves 128-byte lines, so leaving out the dead part of a row
 *   saves no traffic.  The memory side of the window (Sec. 3.3) needs the tiled group-major K
 *   cache (ATF_KLAYOUT_GROUPS through atf_decode_ex), in which only the live prefix of each tile
 *   is fetched.
 *   Needs a workspace of atf_workspace_bytes(ATF_OP_DECODE, ...).                             */
atf_status atf_decode(const void* q, const void* Kcache, const void* Vcache, void* O, int B,
                      int Hq, int Hkv, int64_t L, int d, const int64_t* table, void* stream);
atf_status atf_decode_ex(const void* q, const void* Kcache, const void* Vcache, void* O, int B,
                         int Hq, int Hkv, int64_t L, int d, const int64_t* table,
                         const atf_opts* opts, void* stream);

/* Prefill with scores of more than bf16 input precision (App. D, "Precision as the other side of the
 * compute-accuracy trade": a low-precision product split in two to recover accuracy, paid for with part
 * of what the window saves; Sec. 6.2 scored five tasks with fp32 attention scores because bf16 rounding
 * flipped low-margin retrievals under the window).
 *   Q : dev fp32 [B, Hq, N, d], K: dev fp32 [B, Hkv, N, d], already rotated (atf_rope_f32) and never
 *       rounded to bf16; V: dev bf16 [B, Hkv, N, d]; O: dev bf16 [B, Hq, N, d]; LSE: dev fp32
 *       [B, Hq, N] or NULL.  All 16-byte aligned, row-major, caller-owned.
 *   The library writes each of Q and K as hi = bf16(x) and lo = bf16(x - hi) (hi + lo holds x to 2^-17 of
 *   its size) and accumulates S = Q_hi K_hi^T + Q_hi K_lo^T + Q_lo K_hi^T in fp32 over the live pairs of
 *   each tile: three tensor-core products instead of one.  The window rule, both modes, the term counts
 *   (opts->kept_terms) and the treatment of V, P and O are those of atf_prefill; every exponential is the
 *   hardware ex2.  Against the per-term definition on the fp32 inputs the LSE is good to about
 *   1.5e-5 x max(1, largest |logit|): a logit is a sum of products each held to ~2^-16 of its size.
 *   opts: mode, kept_terms, workspace are read; kcache_groups and rope_tables return ATF_ERR_UNSUPPORTED.
 *   Needs a workspace of atf_workspace_bytes(ATF_OP_PREFILL_SPLIT, ...) (the four bf16 parts).
 *   Errors: as atf_prefill.  d = 64 or 128; causal must be 1.
 * atf_rope_f32: atf_rope on fp32 rows, the result kept in fp32 (the fp64 rotation rounded once).      */
atf_status atf_prefill_split(const float* Q, const float* K, const void* V, void* O, float* LSE, int B,
                             int Hq, int Hkv, int64_t N, int d, const int64_t* table, int causal,
                             const atf_opts* opts, void* stream);
/* The same for Nq rows appended to a context of N keys (Q, O: [B, Hq, Nq, d]; LSE: [B, Hq, Nq]; the rows sit
 * at positions N-Nq..N-1), as atf_prefill_chunk is to atf_prefill; atf_prefill_split is the Nq = N case. */
atf_status atf_prefill_split_chunk(const float* Q, const float* K, const void* V, void* O, float* LSE,
                                   int B, int Hq, int Hkv, int64_t Nq, int64_t N, int d,
                                   const int64_t* table, int causal, const atf_opts* opts, void* stream);
atf_status atf_rope_f32(float* X, int B, int H, int64_t N, int d, const double* theta, int64_t pos0,
                        void* stream);

/* Copies n rotated key rows into a group-major K cache (see ATF_KLAYOUT_GROUPS: the layout in
 * which the memory side of the window, Sec. 3.3, holds at DRAM line granularity).
 *   K : dev bf16 [B, Hkv, n, d], rows for positions pos0 .. pos0+n-1;
 *   Kg: dev bf16 [B, Hkv, ceil(Lcap/KT), d/16, KT, 16], the cache, Lcap >= pos0 + n its length
 *       in keys, KT = atf_kcache_tile_keys(d) (64 for d = 128, 128 for d = 64).
 * atf_decode_ex with k_layout = ATF_KLAYOUT_GROUPS takes the cache with atf_opts.kcache_capacity = Lcap
 * (0 means a cache of exactly ceil(L/KT) tiles).                                                */
int64_t atf_kcache_tile_keys(int d);
atf_status atf_kcache_pack(const void* K, void* Kg, int B, int Hkv, int64_t n, int64_t Lcap,
                           int64_t pos0, int d, void* stream);

/* Rotation tables for decode on an unrotated, position-independent K cache (App. B: a cache that is
 * reused at another position stores keys before RoPE, and the rotation is applied at read; only the
 * pairs the window keeps are fetched, so only those are rotated).
 *   theta   : host, d/2 doubles, the effective frequencies (atf_window_table's theta_out);
 *   pos0    : position of key 0 of the cache; capacity: keys the tables cover (>= every L used);
 *   tables  : dev, 256-byte aligned, atf_rope_tables_bytes(d, capacity) bytes, owned by the caller.
 * The tables hold (cos, sin) in fp32, computed in fp64: one row per key of a tile and one row per
 * tile; the kernel adds the two angles.  They depend on (theta, pos0) only, so one build serves
 * every decode step of a sequence.  Pass them as atf_opts.rope_tables with k_layout =
 * ATF_KLAYOUT_GROUPS; the cache is written by atf_kcache_pack from UNROTATED key rows, q is rotated
 * by the caller (atf_rope at position pos0 + L - 1).  The result equals decode on the rotated
 * cache up to the fp32 rotation (a key element may differ by one bf16 unit in the last place).
 * Errors: ATF_ERR_INVALID_ARG (null, misaligned, theta not positive and finite, bad range),
 * ATF_ERR_UNSUPPORTED (d), ATF_ERR_WORKSPACE (buffer too small); atf_rope_tables_bytes returns 0 for
 * a shape it does not support.                                                                  */
size_t atf_rope_tables_bytes(int d, int64_t capacity);
atf_status atf_rope_tables(const double* theta, int d, int64_t pos0, int64_t capacity, void* tables,
                           size_t bytes, void* stream);

/* Decode without any device allocation.  (The paper has no counterpart: this entry point exists
 * for the callers described here, not for a passage of the method.)
 * Some callers can neither allocate device memory nor pass a workspace: code that runs inside
 * another runtime's callback - a custom op of an inference server, a host that has locked its
 * device allocator after start-up, a process held to a fixed memory budget - must not call
 * cudaMalloc, which synchronises the device and may fail or deadlock under the host's memory
 * manager.  atf_decode_static is atf_decode (exact mode, row-layout K cache, same arguments,
 * same result) whose split-K scratch is a fixed array inside the library image instead of the
 * bound workspace.  It calls no cudaMalloc, cudaFree or allocating library routine.
 *   - Capacity: atf_decode_static_capacity() bytes (2 MiB + the 64.25 KiB header).  Every GPU
 *     that loads the library holds that much memory until the process exits.  A problem that
 *     needs more (roughly B*Hq*splits*(d+2)*4 bytes; e.g. B = 8, Hq = 24, d = 128 fits, B = 32
 *     does not) is refused with ATF_ERR_WORKSPACE and a message naming both sizes.
 *   - The first call on each device looks the array's device address up (cudaGetSymbolAddress,
 *     with that device current); make that first call before any stream capture begins.
 *   - All calls on a device share the one array, which keeps the previous call's contents; each
 *     call clears the words that must start at zero itself.  Two calls that overlap on the GPU
 *     (different streams, no ordering between them) race on it: keep calls on one device ordered. */
size_t atf_decode_static_capacity(void);
atf_status atf_decode_static(const void* q, const void* Kcache, const void* Vcache, void* O, int B,
                             int Hq, int Hkv, int64_t L, int d, const int64_t* table, void* stream);

/* Workspace.  The library keeps no allocation of its own: the caller allocates
 * atf_workspace_bytes() bytes of device memory (256-byte aligned), zero-fills it once, and
 * binds it.  The binding is ONE pointer per process (it is only stored), not one per device: a
 * process that drives several GPUs passes each call its own workspace in atf_opts.workspace.
 * A workspace sized for the largest call
 * serves prefill and decode in turn: its first 64.25 KiB (status words and decode's split
 * counters, which the kernels leave zeroed) are never used as scratch.  One call at a time may use a given
 * workspace; calls that overlap on the GPU need separate workspaces (atf_opts.workspace).     */
enum { ATF_OP_PREFILL = 0, ATF_OP_DECODE = 1, ATF_OP_PREFILL_SPLIT = 2 };
size_t atf_workspace_bytes(int op, int B, int Hq, int Hkv, int64_t N, int d);
atf_status atf_bind_workspace(void* dev_ptr, size_t bytes);

/* Reads (and clears) the device status words of the bound workspace and, if atf_decode_static
 * has run on the current device, of its built-in array; synchronises `stream`.  Returns
 * ATF_ERR_TIMEOUT if a kernel gave up on a bounded wait since the last check (every device-side
 * wait gives up after 2 s of wall time and the kernel then ends; its results are not valid).
 * atf_check_status_at does the same for a workspace that was passed in atf_opts.workspace or as
 * dev_scratch of atf_prefill_host (which leaves the status words of earlier calls in place).   */
atf_status atf_check_status(void* stream);
atf_status atf_check_status_at(void* workspace, void* stream);

/* Self-test of that report path: launches one small kernel that waits, with the kernels' bounded
 * wait and a limit of limit_us microseconds (1..100000), for a barrier nobody signals, gives up
 * and records it in the bound workspace.  The next atf_check_status returns ATF_ERR_TIMEOUT once. */
atf_status atf_selftest_bounded_wait(unsigned int limit_us, void* stream);

/* Diagnostic behind the choice of K-cache layouts: reads `bytes` of device memory as 256-byte rows (a K row
 * at d = 128), leaving out the 16-byte chunks of every row whose bit in chunkmask (16 bits, bit c = chunk c)
 * is clear.  Timed by the caller; with the DRAM counters of a profiler it shows that a chunk skipped inside
 * a 128-byte line saves no traffic (a mask like 0xF0F0 costs what 0xFFFF costs), while whole lines do
 * (0xFF00).  Needs a bound workspace (one word of it is the kernel's sink).                              */
atf_status atf_probe_masked_read(const void* buf, size_t bytes, unsigned int chunkmask, void* stream);

/* Text of the calling thread's last error ("" if none). Never NULL. */
const char* atf_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* ATFLASH_H */
