/*
 * cowa.h -- C ABI of the CoWindow Attention (CoWA) library for NVIDIA B200 (sm_100a).
 *
 * The operator: causal grouped-query attention in which KV head h sees, for the
 * query at bottom-right-aligned causal distance delta = i_q + (N_k - N_q) - i_k
 * (Eq. fwa_distance), the union (Eq. fwa_support) of
 *   near  { 0 <= delta < near }
 *   sink  { i_k < sink, delta >= 0 }
 *   long  { near + gap <= delta < near + gap + len }
 * with one 4-tuple (sink, near, gap, len) per KV head (Sec. 2.1, after Eq. fwa_support).
 * QO head h uses KV head floor(h * Hkv / Hq) and its tuple (GQA, Sec. 2.1).
 *
 * General conventions
 *   - Every tensor pointer is a DEVICE pointer unless a comment says "host".
 *   - q, k, v, o, d_o, dq, dk, dv are bf16; lse and workspaces are fp32/bytes.
 *   - Default layout is contiguous head-major [B, H, T, D] with D innermost
 *     (Algorithm 1/2 REQUIRE lines, plus a batch axis).  Base pointers must be
 *     16-byte aligned.  Other layouts of the batched calls are described by element
 *     strides in cowa_params_t (D always contiguous): e.g. a [B, T, H, D] projection
 *     output or a [B, Tmax, Hkv, D] cache is passed without a copy.
 *   - lse is the natural-log logsumexp of softmax_scale * q.k over the visible keys
 *     (Algorithm 1 line 17), fp32 [B, Hq, T].
 *   - The caller owns every buffer, workspaces included.  The library allocates no
 *     device memory and keeps no state between calls except cached kernel
 *     attributes and the per-thread error code behind cowa_last_cuda_error().
 *     All work is enqueued on `stream`; no call synchronises.
 *   - Return value: COWA_OK (0) or a negative cowa_status_t.  Arguments are validated
 *     before anything is launched.  There is no CPU fallback.
 *   - Preconditions not checked on the device: near >= 1 for every head (so each
 *     query sees at least its own position), lens[b] in [1, Tmax].
 */
#ifndef COWA_H_
#define COWA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  COWA_OK = 0,
  COWA_ERR_INVALID_ARG = -1,        /* null pointer, non-positive size, Hq % Hkv != 0, bad window */
  COWA_ERR_UNSUPPORTED = -2,        /* D not in {64,128}; strides given to a call that takes none */
  COWA_ERR_MISALIGNED = -3,         /* a base pointer is not 16-byte aligned, or a stride is not a multiple of
                                       8 elements (16 bytes) */
  COWA_ERR_WORKSPACE_TOO_SMALL = -4,
  COWA_ERR_CUDA = -5,               /* a CUDA call failed; see cowa_last_cuda_error() */
  COWA_ERR_DEVICE_TIMEOUT = -6,     /* reported by cowa_check_device_status(): a bounded device wait ran out */
  COWA_ERR_STATIC_SCRATCH_EXCEEDED = -7, /* cowa_decode_static: the call needs more scratch than the built-in array holds */
  COWA_ERR_DEVICE_BAD_SEQLENS = -8, /* reported by cowa_check_device_status(): cowa_prefill_varlen met a sequence
                                       with N_q > N_k in its device-side offset arrays and skipped it */
  COWA_ERR_DEVICE_DQ_RANGE = -9     /* reported by cowa_check_device_status(): a backward call with
                                       deterministic = 1 met a dQ partial sum outside the fixed-point range
                                       (|x| >= 8192), or a final |dQ| >= 4096; its dq is not to be trusted */
} cowa_status_t;

/* One KV head's windows: the paper's 4-tuple (sink width, near width, gap after the
 * near window, long-range width), Sec. 2.1.  len == 0 means no long-range window. */
typedef struct {
  int32_t sink, near, gap, len;
} cowa_window_t;

typedef struct {
  int32_t sink;        /* w_sink of the default rule (Eq. fwa_long_range_span) */
  int32_t local;       /* w_near of the default rule; must be >= 1 */
  int32_t block_q;     /* tile sizes used by cowa_schedule_dump (the kernels tile 128x128) */
  int32_t block_k;
  int32_t hkv_global;  /* global number of KV heads (Eq. fwa_global_head); 0 => Hkv */
  int32_t hkv_offset;  /* global index of this call's KV head 0; 0 on one GPU */
  const cowa_window_t* windows; /* HOST pointer to Hkv explicit tuples, or NULL for the default rule.
                                   Read during the call; not retained.  Ignored by cowa_decode. */
  int32_t full_attn;   /* 1 => every head sees the whole causal prefix (dense FullAttn path) */
  float softmax_scale; /* scores are softmax_scale * q.k (the paper pre-scales Q by 1/sqrt(d_h)) */
  int32_t deterministic; /* cowa_bwd only.  0: dQ partial sums are added in fp32 in whatever order the
                            blocks arrive (Algorithm 2 line 15's AtomicAdd; results vary in the last bits
                            from run to run).  1: the partial sums are added as 32-bit fixed point with
                            18 fractional bits, which is exact and order-independent, so dQ is bitwise
                            reproducible; requires |dQ| < 8192 and rounds each partial to 2^-19.  A partial
                            sum of one tile that leaves that range, or a final |dQ| >= 4096 (half of it: a
                            wrapped total lands there in most cases), sets a device flag that
                            cowa_check_device_status() returns as COWA_ERR_DEVICE_DQ_RANGE. */
  /* Element strides (batch, head, token) of q, k, v, o; the D axis is contiguous.  All three zero (the
   * default) means contiguous head-major [B, H, T, D].  Otherwise every stride must be a non-negative multiple
   * of 8 elements and the token stride at least D.  Used by cowa_fwd, cowa_prefill, cowa_bwd, cowa_bwd_prefill
   * (there d_o is laid out like o, dq like q, dk like k, dv like v) and by cowa_decode / cowa_decode_static
   * (k_strides, v_strides describe the cache; q and o stay [B, Hq, D]).  The packed (varlen), multi-token and
   * paged calls take contiguous tensors only and return COWA_ERR_UNSUPPORTED when a stride is set.  lse is
   * always contiguous. */
  int64_t q_strides[3], k_strides[3], v_strides[3], o_strides[3];
  /* cowa_bwd / cowa_bwd_prefill / cowa_bwd_varlen only: optional CUDA events (cudaEvent_t handles owned by the
   * caller, or NULL) recorded on the call's stream just before and just after the main backward kernel
   * (Algorithm 2's loops), so that a profiler can time that kernel apart from the preprocess, memset and
   * conversion launches of the same call. */
  void* bwd_main_start_event;
  void* bwd_main_stop_event;
} cowa_params_t;

/* Training / prefill forward, Algorithm 1.  N_q = N_k = T.
 *   q [B,Hq,T,D], k,v [B,Hkv,T,D] in; o [B,Hq,T,D] bf16 and lse [B,Hq,T] fp32 out.
 * D in {64,128}; Hq a multiple of Hkv.  No workspace. */
int cowa_fwd(const void* q, const void* k, const void* v, void* o, float* lse,
             int B, int T, int Hq, int Hkv, int D, const cowa_params_t* p, void* stream);

/* Inference prefill, also chunked prefill into an existing cache: the same forward operator with
 * N_q <= N_k (Sec. 2.3 "Forward execution"; Sec. 2.1: query i_q sits at key position i_q + (N_k - N_q),
 * Eq. fwa_distance, and the windows are built from N_k).
 *   q [B,Hq,Nq,D]; k,v [B,Hkv,Nk,D] in; o [B,Hq,Nq,D] bf16 and lse [B,Hq,Nq] fp32 out.
 * Every sequence of the batch has the same Nq and Nk.  cowa_fwd is this call with Nq = Nk = T. */
int cowa_prefill(const void* q, const void* k, const void* v, void* o, float* lse,
                 int B, int Nq, int Nk, int Hq, int Hkv, int D, const cowa_params_t* p, void* stream);

/* Prefill over a packed batch of B sequences of different lengths (Sec. 2.1: each sequence b has its own
 * N_q[b] <= N_k[b]; its queries sit at key positions i_q + (N_k[b] - N_q[b]), Eq. fwa_distance, and its
 * long-range breakpoints follow from its own N_k[b], Eq. fwa_long_range_span; Sec. 2.3 "Forward execution").
 *   q [Hq,total_q,D]; k,v [Hkv,total_k,D] in; o [Hq,total_q,D] bf16 and lse [Hq,total_q] fp32 out: the
 *   sequences are concatenated along the token axis, head-major, contiguous.
 *   cu_seqlens_q, cu_seqlens_k: DEVICE int32[B+1], non-decreasing row offsets with cu[0] = 0,
 *   cu_q[B] = total_q, cu_k[B] = total_k; sequence b owns rows [cu[b], cu[b+1]).  N_q[b] = 0 is allowed
 *   (the sequence is skipped).
 * Explicit tuples in p->windows apply to every sequence unchanged; the default rule and full_attn are
 * evaluated per sequence on the device.  The offsets are read on the device only: a sequence with
 * N_q > N_k, or whose rows leave the tensors, is skipped (N_q < 0 counts as empty) and
 * cowa_check_device_status() then returns COWA_ERR_DEVICE_BAD_SEQLENS.  No workspace; nothing is
 * retained.  Blocks are issued sequence after sequence: passing long sequences first shortens the tail. */
int cowa_prefill_varlen(const void* q, const void* k, const void* v, void* o, float* lse,
                        const int32_t* cu_seqlens_q, const int32_t* cu_seqlens_k, int B, int total_q,
                        int total_k, int Hq, int Hkv, int D, const cowa_params_t* p, void* stream);

/* Training backward, Algorithm 2: exact gradient of cowa_fwd.
 *   in: q,k,v,o,lse as produced by cowa_fwd, d_o [B,Hq,T,D];
 *   out: dq [B,Hq,T,D], dk,dv [B,Hkv,T,D] bf16 (fully overwritten).
 * dk,dv are summed over the QO heads of each group inside one thread block, or, when there are too few
 * (batch, KV head, KV tile) triples to fill the GPU or the sink tiles would dominate, by a few blocks whose
 * fp32 partial sums a last kernel adds in a fixed order: no atomics (Algorithm 2 line 17 has them), always
 * bitwise reproducible; for dq see cowa_params_t.deterministic.
 * `workspace` (device, >= cowa_bwd_workspace_bytes for the same B, T, Hq, Hkv, D and params, 16-byte
 * aligned) holds the fp32 dq accumulator, the row vector rowsum(o*d_o) (Algorithm 2 line 13) and those
 * partial sums; it needs no initialisation. */
int cowa_bwd(const void* q, const void* k, const void* v, const void* o, const float* lse,
             const void* d_o, void* dq, void* dk, void* dv,
             int B, int T, int Hq, int Hkv, int D, const cowa_params_t* p,
             void* workspace, size_t workspace_bytes, void* stream);

/* Backward of cowa_prefill: the same Algorithm 2 with N_q <= N_k (queries bottom-right aligned, Eq.
 * fwa_distance; windows from N_k).  q, o, d_o, dq [B,Hq,Nq,D]; k, v, dk, dv [B,Hkv,Nk,D]; lse [B,Hq,Nq].
 * Keys no query sees get zero gradients.  cowa_bwd is this call with Nq = Nk = T; workspace size from
 * cowa_bwd_prefill_workspace_bytes. */
int cowa_bwd_prefill(const void* q, const void* k, const void* v, const void* o, const float* lse,
                     const void* d_o, void* dq, void* dk, void* dv,
                     int B, int Nq, int Nk, int Hq, int Hkv, int D, const cowa_params_t* p,
                     void* workspace, size_t workspace_bytes, void* stream);
size_t cowa_bwd_prefill_workspace_bytes(int B, int Nq, int Nk, int Hq, int Hkv, int D, const cowa_params_t* p);

/* Training backward over a packed batch of B sequences of different lengths (self-attention: N_q = N_k =
 * the sequence's length; Algorithm 2 applied per sequence, each with windows from its own length, Sec. 2.1).
 *   q, o, d_o, dq [Hq,total,D]; k, v, dk, dv [Hkv,total,D] bf16; lse [Hq,total] fp32 as written by
 *   cowa_prefill_varlen for the same offsets with cu_seqlens_q = cu_seqlens_k = cu_seqlens;
 *   cu_seqlens: DEVICE int32[B+1], cu[0] = 0, cu[B] = total, non-decreasing.
 * dq, dk, dv are fully overwritten for every row of every sequence.  Malformed offsets are reported as for
 * cowa_prefill_varlen.  `workspace`: device, >= cowa_bwd_varlen_workspace_bytes(B, total, ...), 16-byte
 * aligned, no initialisation needed.  cowa_params_t.deterministic applies as in cowa_bwd. */
int cowa_bwd_varlen(const void* q, const void* k, const void* v, const void* o, const float* lse,
                    const void* d_o, void* dq, void* dk, void* dv, const int32_t* cu_seqlens,
                    int B, int total, int Hq, int Hkv, int D, const cowa_params_t* p,
                    void* workspace, size_t workspace_bytes, void* stream);
size_t cowa_bwd_varlen_workspace_bytes(int B, int total, int Hq, int Hkv, int D, const cowa_params_t* p);

/* Single-token decode over a KV cache (Sec. 2.3 "Decoding"): the forward with N_q = 1.
 *   q [B,Hq,D]; kcache,vcache [B,Hkv,Tmax,D]; lens int32 [B] on the DEVICE, lens[b] = N_k
 *   = cached tokens + 1, the current token's K/V already stored at index lens[b]-1.
 *   Breakpoints are recomputed from lens[b] for every sequence (default rule only).
 *   out: o [B,Hq,D] bf16; lse [B,Hq] fp32 (may be NULL).
 * Only the visible rows of each head are read.  Split-KV partial states go to `workspace`
 * (device, >= cowa_decode_workspace_bytes, 16-byte aligned, no initialisation needed) and
 * are merged by a second kernel on the same stream. */
int cowa_decode(const void* q, const void* kcache, const void* vcache, const int32_t* lens,
                void* o, float* lse, int B, int Tmax, int Hq, int Hkv, int D,
                const cowa_params_t* p, void* workspace, size_t workspace_bytes, void* stream);

/* Decode for callers that cannot allocate device memory.  (No counterpart in the paper: this
 * is a packaging variant of cowa_decode, same arguments minus the workspace, same results.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a serving loop that
 * forbids allocation after start-up, in a plugin whose host owns all device memory, or in a
 * region where an allocation's implicit synchronisation would stall other streams.  Such a
 * caller cannot size and hand over the split-KV workspace that cowa_decode wants, so here the
 * partial states go to a fixed array compiled into the library's device image instead
 * (cowa_decode_static_capacity() bytes, 8 MiB; each GPU that loads the library holds that much
 * until the process ends).  The call itself performs no cudaMalloc/cudaFree and calls nothing
 * that allocates.
 *
 * Limits and rules:
 *   - The call is rejected with COWA_ERR_STATIC_SCRATCH_EXCEEDED, before any launch, when
 *     cowa_decode_workspace_bytes(...) for the same arguments exceeds the capacity
 *     (for orientation: batch 8 x 32 QO heads x D 128 over a 128K cache needs 4.9 MiB).
 *   - The first call on each device looks up the array's device address (one
 *     cudaGetSymbolAddress with that device current).  Make that first call during set-up,
 *     before any stream capture.
 *   - All calls on a device share the one array.  It keeps the previous call's contents; that
 *     is harmless because every value the merge kernel reads is rewritten by the same call's
 *     split kernel first.  Two calls that overlap on the GPU (different streams, no ordering
 *     between them) race on the array and give wrong results: serialise them. */
int cowa_decode_static(const void* q, const void* kcache, const void* vcache, const int32_t* lens,
                       void* o, float* lse, int B, int Tmax, int Hq, int Hkv, int D,
                       const cowa_params_t* p, void* stream);
size_t cowa_decode_static_capacity(void);

/* Decode of the Nq newest tokens of every sequence in one call (speculative / multi-token decoding).
 * The paper's decode step is the forward with N_q = 1 (Sec. 2.3 "Decoding"); this is the same forward with
 * N_q = Nq: token t of sequence b sits at key position lens[b] - Nq + t, sees keys by Eq. fwa_support at its
 * own distance (Eq. fwa_distance with N_k = lens[b]), and the windows are built from lens[b] for all Nq
 * tokens alike.  The paper describes no such variant; the distance rule is unchanged.
 *   q [B,Nq,Hq,D] in; o [B,Nq,Hq,D] bf16 and lse [B,Nq,Hq] fp32 (may be NULL) out;
 *   kcache, vcache [B,Hkv,Tmax,D] already hold the Nq new tokens; lens: DEVICE int32[B], Nq <= lens[b] <= Tmax.
 * 1 <= Nq <= 64; Hq/Hkv in {1,2,4,8}.  Tokens are packed into the 8 columns of the score MMA together with
 * the group's heads: 8/(Hq/Hkv) tokens share one pass over the visible rows, more tokens take more blocks
 * (their re-reads mostly hit in L2; beyond about three such passes cowa_prefill / cowa_prefill_varlen, whose
 * cost does not grow with Nq up to 128, is the faster call).  `workspace`: device, >= cowa_decode_multi_workspace_bytes, 16-byte
 * aligned, no initialisation needed.  cowa_params_t.windows is ignored, as in cowa_decode. */
int cowa_decode_multi(const void* q, const void* kcache, const void* vcache, const int32_t* lens,
                      void* o, float* lse, int B, int Nq, int Tmax, int Hq, int Hkv, int D,
                      const cowa_params_t* p, void* workspace, size_t workspace_bytes, void* stream);

/* The same over a paged KV cache (not in the paper: a serving-side memory layout).
 *   kpages, vpages [num_pages, Hkv, page_size, D] bf16; block_table: DEVICE int32 [B, max_pages], entry
 *   [b, i] = page holding tokens [i*page_size, (i+1)*page_size) of sequence b (entries past the sequence's
 *   last page are not read); page_size a multiple of 16; lens[b] <= max_pages * page_size.
 * Other arguments, Nq included (Nq = 1 is plain paged decode), as for cowa_decode_multi; workspace size from
 * cowa_decode_multi_workspace_bytes with Tmax = max_pages * page_size.  Page indices are not range-checked. */
int cowa_decode_paged(const void* q, const void* kpages, const void* vpages, const int32_t* block_table,
                      const int32_t* lens, void* o, float* lse, int B, int Nq, int max_pages, int page_size,
                      int Hq, int Hkv, int D, const cowa_params_t* p, void* workspace, size_t workspace_bytes,
                      void* stream);
size_t cowa_decode_multi_workspace_bytes(int B, int Nq, int Tmax, int Hq, int Hkv, int D, const cowa_params_t* p);

size_t cowa_bwd_workspace_bytes(int B, int T, int Hq, int Hkv, int D, const cowa_params_t* p);
size_t cowa_decode_workspace_bytes(int B, int Tmax, int Hq, int Hkv, int D, const cowa_params_t* p);

/* Host-only.  Default 4-tuples (sink, local, b_h, b_{h+1}-b_h), b_h = floor(h*L/Hkv_global),
 * L = max(Nk - sink - local, 0), for global heads hkv_offset .. hkv_offset+Hkv_local-1
 * (Eq. fwa_long_range_span, Eq. fwa_global_head).  out: HOST array of Hkv_local tuples. */
int cowa_default_windows(int Nk, int Hkv_global, int hkv_offset, int Hkv_local,
                         int sink, int local, cowa_window_t* out);

/* Host-only.  Equal-area breakpoints for training / prefill: tuples of the same form
 * (sink, local, b_h, b_{h+1}-b_h) whose bands still tile [0, L), so collective coverage
 * (Eq. fwa_collective_coverage) holds, but with the breakpoints moved so that every head's band holds
 * about the same number of legal (query, key) pairs.  Sec. 2.1 allows other breakpoint schedules under
 * the same support rule and leaves equal-area allocation out of its scope: the rule below is this
 * library's.  Band offset x (distance local + x) weighs c(x) = number of queries i_q in [0, Nq) with
 * i_q + (Nk - Nq) - (local + x) >= sink; W(b) = sum_{x<b} c(x); b_h = the smallest b with
 * Hkv_global * W(b) >= h * W(L).  Pass the result as cowa_params_t.windows.  out: HOST array of Hkv_local
 * tuples for global heads hkv_offset .. hkv_offset+Hkv_local-1.  Cost O(L). */
int cowa_equal_area_windows(int Nq, int Nk, int Hkv_global, int hkv_offset, int Hkv_local,
                            int sink, int local, cowa_window_t* out);

/* Host-only.  Writes the analytic tile schedule (Sec. 2.3: block sets J_h(i), I_h(j)) that the
 * kernels' scheduler computes, as an int32 stream into the HOST buffer `out`:
 *   COWA_SCHED_FWD    for each head h, QO tile i:  h, i, n, then n pairs (j, full) with j descending
 *   COWA_SCHED_BWD    for each head h, KV tile j:  h, j, n, then n pairs (i, full) with i ascending
 *   COWA_SCHED_DECODE for each head h: h, r, then r pairs (start, end) of visible key ranges [start,end)
 *                     ascending, then m, then m visited block_k-block indices; Nq = 1 is the decode step,
 *                     Nq > 1 the union over the Nq newest tokens (what cowa_decode_multi streams)
 * full = 1 when every pair of the nominal block_q x block_k tile is legal, else 0 (boundary tile).
 * *out_len receives the number of int32 needed; COWA_ERR_WORKSPACE_TOO_SMALL if out_cap is less
 * (nothing beyond out_cap is written). */
enum { COWA_SCHED_FWD = 0, COWA_SCHED_BWD = 1, COWA_SCHED_DECODE = 2 };
int cowa_schedule_dump(int which, int Nq, int Nk, int Hkv, const cowa_params_t* p,
                       int32_t* out, size_t out_cap, size_t* out_len);

/* Visited-tile counts of the 128x128 kernel tiling summed over the Hkv heads (host-only):
 * out[0] = visited, out[1] = full, out[2] = causal tiles.  Used for FLOP accounting. */
int cowa_tile_counts(int Nq, int Nk, int Hkv, const cowa_params_t* p, int64_t out[3]);

/* The kernels bound every device-side wait; a wait that runs out sets a flag in a device word
 * instead of hanging.  This call synchronises `stream`, reads and clears the flags, and returns
 * COWA_OK, COWA_ERR_DEVICE_TIMEOUT, COWA_ERR_DEVICE_BAD_SEQLENS or COWA_ERR_DEVICE_DQ_RANGE, in that
 * order of precedence when several are set (COWA_ERR_CUDA if the stream itself reports an error). */
int cowa_check_device_status(void* stream);

/* Self-test of the bounded waits (no counterpart in the paper).  Enqueues a one-block kernel that waits,
 * with the same wait routine the training kernels use but a limit of `limit_clocks` SM clocks (clamped to
 * [2^10, 2^24]), on a barrier that nothing ever arrives at.  The wait must give up, set the timeout flag
 * and let the kernel end normally: the next cowa_check_device_status() then returns
 * COWA_ERR_DEVICE_TIMEOUT once.  Nothing else is touched. */
int cowa_selftest_bounded_wait(long long limit_clocks, void* stream);

const char* cowa_status_string(int status);
/* cudaError_t value of the most recent failing CUDA call made by this library on this thread. */
int cowa_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* COWA_H_ */
