/*
 * albireo_sample.h -- C ABI of the B200 (sm_100a) batched token sampler.
 *
 * The library implements the sampling task T4 of "Albireo" (arxiv 2606.01927, section
 * 2.1): after every decode step, for each row of the (s x v) logits matrix, choose the
 * next token.  The paper leaves the per-row sampling arithmetic as it is in the serving
 * framework (section 6.1, step 3) and enables every feature in its evaluation (section 8.1, Workload): top-p,
 * top-k, min-p, temperature, and repetition / presence / frequency penalties driven by
 * per-sequence metadata (section 3.1, Optimization 3).  Rows are independent (section
 * 6.1), the result per row is one token id plus its probability (section 6.2, result
 * gather; Appendix A, "update sequence"), and the draw must not depend on how rows are
 * partitioned over workers (section 6.2, deterministic random number generation).
 *
 * Per row b (global row id R = row_base + b) the library computes, in this order:
 *   x      = logits widened to fp32
 *   c_t    = occurrences of token t in the row's history (ids outside [0,V) ignored)
 *   a_t    = x_t                              if c_t == 0
 *          = ((x_t > 0 ? x_t / r : x_t * r) - f * c_t) - p   otherwise (fp32, one rounding per op;
 *            with ext->history_output_start see there)
 *   z_t    = a_t * (1 / T)   (fp32; T <= 0 means greedy: top_k = 1 on a_t, other cuts ignored)
 *   order  = ids sorted by (z descending, id ascending); -0.0 sorts below +0.0
 *   top-k  : keep the first min(k, #finite z)          (k <= 0 or k >= V: off)
 *   min-p  : keep z - z_max >= ln(min_p), at least one (min_p <= 0: off)
 *   top-p  : smallest prefix whose mass reaches top_p * (mass of the survivors) (top_p >= 1: off)
 *   logprob: log of the softmax over the final kept set
 *   draw   : w_t = word (t & 3) of Philox4x32-10(counter = (t >> 2, R, step lo, step hi),
 *            key = (seed lo, seed hi)); v = (w + 1/2) / 2^32; E = -log1p(-v);
 *            token = argmax_t (z_t - z_max) - ln E_t   (ties: lowest id)
 *
 * All data pointers are DEVICE pointers unless a parameter says "host".  The caller
 * owns every buffer, including the workspace; the library owns only the opaque handle
 * (host memory) and never allocates or frees device memory.
 */
#ifndef ALBIREO_SAMPLE_H
#define ALBIREO_SAMPLE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct albireo_sampler albireo_sampler_t; /* opaque; created by init, freed by destroy */

enum { ALBIREO_F32 = 0, ALBIREO_BF16 = 1, ALBIREO_F16 = 2 /* IEEE binary16: the paper's models are FP16, section 8.1 */ };

enum {
    ALBIREO_OK = 0,
    ALBIREO_EINVAL = -1,       /* bad argument; nothing was launched                     */
    ALBIREO_ENOMEM = -2,       /* host allocation of the handle failed                   */
    ALBIREO_ECUDA = -3,        /* a CUDA runtime call failed; see albireo_last_error     */
    ALBIREO_EUNSUPPORTED = -4  /* shape outside what the kernels support (see limits)    */
};

/* limits */
#define ALBIREO_MAX_VOCAB 524288   /* V above this is rejected                            */
#define ALBIREO_MAX_NUM_TOP 128    /* largest num_top (top-N logprob list)                */
#define ALBIREO_MAX_SEGMENTS 64    /* largest num_segments                                */
#define ALBIREO_MAX_PEER_SEGMENTS 16 /* largest num_segments with segment_ptrs            */

/* bits of out_row_status[b] */
#define ALBIREO_ROW_GENERAL_PATH 1u  /* informational: row took the multi-pass general path */
#define ALBIREO_ROW_BAD_PARAM 2u     /* T < 0 or NaN, r <= 0, ...: row treated per the clamps */
#define ALBIREO_ROW_HISTORY_OVERFLOW 4u /* history did not fit the workspace: penalties skipped */
#define ALBIREO_ROW_TIMEOUT 8u       /* a bounded on-chip wait expired: no result for this row;
                                        out_tokens[b] = -1 and out_logprobs[b] = NaN mark it for
                                        callers that pass no status array                        */

/* flags of albireo_sample_ext_t.flags */
#define ALBIREO_FLAG_FORCE_GENERAL 1u /* testing: send every row down the general path     */
#define ALBIREO_FLAG_TOPK_KEEP_TIES 2u /* top-k keeps every score not below the k-th largest
                                         (what masking "logits < k-th value" gives) instead of
                                         exactly k ids; equal means equal in the order, so -0.0
                                         stays below +0.0; greedy rows are not affected          */
#define ALBIREO_FLAG_LOGPROB_FULL_VOCAB 4u /* out_logprobs and out_top_logprobs are relative to the
                                         softmax over every finite score of the row (after penalties
                                         and temperature; greedy rows: over the unscaled scores)
                                         instead of the final kept set; the token drawn does not
                                         change.  Costs one more pass over the row, from L2.  A
                                         top-N list (num_top > 0) then holds the first entries of the
                                         whole row's order, not of the kept set; rows with such a
                                         list take the general path                               */
#define ALBIREO_FLAG_PROGRAMMATIC_LAUNCH 8u /* launch with programmatic stream serialisation: the
                                         kernel's CTAs may be scheduled while the kernel ahead of it
                                         in the stream is still running (its launch latency and CTA
                                         scheduling then overlap that kernel's tail); each CTA waits
                                         for that kernel to complete before it reads or writes
                                         anything, so the results are unchanged                      */

/*
 * Optional arguments of albireo_sample (pass NULL for all defaults).  Zero-initialise,
 * set struct_size = sizeof(albireo_sample_ext_t), then fill what is needed.
 */
typedef struct albireo_sample_ext {
    uint32_t struct_size;
    uint32_t flags;
    int64_t row_stride_elems;  /* elements between rows of logits; 0 means V               */
    uint32_t row_base;         /* global id of row 0 (keeps draws invariant under row
                                  sharding, section 6.2)                                   */
    int32_t num_top;           /* > 0: also return the first min(num_top, kept) entries of
                                  the kept set in order                                     */
    int32_t *out_top_ids;      /* [B, num_top] device, padded with -1                       */
    float *out_top_logprobs;   /* [B, num_top] device, padded with -inf                     */
    int32_t *out_num_kept;     /* [B] device: size of the final kept set (diagnostic)       */
    int32_t *out_num_topk;     /* [B] device: size of the set kept by the top-k stage       */
    int32_t dbg_cap;           /* capacity per row of dbg_topk_ids                          */
    int32_t *dbg_topk_ids;     /* [B, dbg_cap] device: ids kept by the top-k stage, in no
                                  particular order, -1 padded; written only for rows with an
                                  active top-k (1 <= k < V, or greedy) whose top-k stage
                                  keeps <= dbg_cap ids                                      */
    uint32_t *out_row_status;  /* [B] device: ALBIREO_ROW_* bits                            */

    /* Pre-generated random numbers (section 6.2: the random numbers of a batch are drawn
       ahead of the sampling step so that every worker sees the same ones).  When exp1 is
       not NULL the draw reads E_t = exp1[b * stride + t], an Exp(1) variate per (row,
       token), instead of running the counter-based generator; seeds and step are then
       unused.  Only entries of kept tokens are read.  Each E must be a positive finite
       fp32 (otherwise the row's token is unspecified but in range).                       */
    const float *exp1;         /* [B, exp1_stride_elems] device, 4-byte aligned, or NULL    */
    int64_t exp1_stride_elems; /* elements between rows of exp1; 0 means V                  */

    /* Early feedback (section 5.2: the sampler hands each new token straight to the next
       iteration's input and to the output processor instead of waiting for the host).
       backfill_ids: the next iteration's input-id tensor; row b's token is stored at
       backfill_ids[backfill_index[b]] (backfill_index NULL: at [b]); a negative index
       skips the row, an index >= backfill_len is skipped and sets ALBIREO_ROW_BAD_PARAM.
       feedback_ring: records (global row id << 32 | token) written with one 8-byte store
       each at slot (feedback_head + b) mod feedback_cap; the memory may be mapped pinned
       host memory that the output processor polls (it resets a slot after reading it).
       Rows whose status has ALBIREO_ROW_TIMEOUT write neither.                             */
    int32_t *backfill_ids;         /* [backfill_len] device, or NULL                         */
    const int32_t *backfill_index; /* [B] device, or NULL                                    */
    int64_t backfill_len;
    uint64_t *feedback_ring;       /* [feedback_cap] device-visible, 8-byte aligned, or NULL */
    int64_t feedback_cap;
    int64_t feedback_head;

    /* Rows in pieces (sequence-parallel sampling, section 6.1 steps 2-3): after the all-to-all
       that turns vocabulary shards into row shards, a worker holds each of its rows as
       num_segments pieces of V / num_segments logits, one per sending worker.  With
       num_segments >= 2 the sampler reads them where they landed: element i of row b is
       logits[(i / Vs) * segment_stride_elems + b * row_stride + (i % Vs)], Vs = V / num_segments
       (row_stride_elems 0 then means Vs).  For the receive buffer [t, B, V/t] of an all-to-all
       that is segment_stride_elems = B * V / t.  num_segments must divide V and be <= 64; the
       base pointer and, in bytes, Vs, the row stride and the segment stride must be multiples
       of 16 (ALBIREO_EUNSUPPORTED otherwise).  0 or 1: rows are contiguous.                */
    int32_t num_segments;
    int64_t segment_stride_elems;

    /* Prompt / output split of the histories (the per-sequence sampling metadata of section 3.1
       keeps prompt and generated tokens apart).  history_output_start[b] = number of leading ids
       of row b's history that are the prompt; the rest is generated output.  The repetition
       penalty then applies to a token seen in either part, the frequency penalty uses the
       occurrences in the output alone and the presence penalty applies only if there is one:
       a = rep(x); a -= f * c_out; if (c_out > 0) a -= p.  Values are clamped to [0, length].
       NULL: every id counts as output (the three penalties share one history).             */
    const int32_t *history_output_start; /* [B] device, or NULL                              */

    /* Rows in pieces without an exchange step: with segment_ptrs (a HOST array of num_segments
       device pointers, <= ALBIREO_MAX_PEER_SEGMENTS) piece j of row b is read from
       segment_ptrs[j] + (segment_row_offset + b) * row_stride + (i % Vs), i.e. from the
       vocabulary shard [s, V/t] as it lies in worker j's own memory (peer-mapped: symmetric memory,
       IPC or cudaMemcpyPeer-capable mappings all do).  The logits then cross NVLink once, straight
       into the sampler's shared memory, and the all-to-all of section 6.1 step 2 disappears; the
       caller makes sure every worker's shard is complete before the launch and not overwritten
       before the call has finished.  `logits` is ignored (pass segment_ptrs[0]);
       segment_stride_elems is unused; every pointer must be 16-byte aligned.  NULL: one buffer. */
    const void *const *segment_ptrs;     /* host array of device pointers, or NULL              */
    int64_t segment_row_offset;          /* rows before this call's row 0 in every piece buffer  */
} albireo_sample_ext_t;

/*
 * Device bytes the caller must provide as `workspace` to albireo_sample_init.
 * The workspace holds per-row history occurrence counts for rows whose history has more
 * distinct ids than fit on chip (sized by max_history_total, the largest
 * history_offsets[B] of any call).  Pure function of its arguments; returns 0 on
 * nonsensical input (negative sizes).
 */
size_t albireo_sample_workspace_bytes(int32_t max_rows, int32_t max_vocab, int64_t max_history_total);

/*
 * Extra device bytes albireo_sample_host needs after the first
 * albireo_sample_workspace_bytes(...) bytes of the same workspace (staging copies of
 * every input and output; logits staged at 4 bytes per element).
 */
size_t albireo_sample_host_staging_bytes(int32_t max_rows, int32_t max_vocab, int64_t max_history_total);

/*
 * Creates a sampler bound to CUDA device `device`.
 *   workspace / workspace_bytes: caller-owned device memory on that device, 256-byte
 *     aligned, at least albireo_sample_workspace_bytes(...) long (plus the staging
 *     bytes if albireo_sample_host will be used); must outlive the handle.
 * Does not allocate device memory and does not synchronise.  Sets per-device kernel
 * attributes, so call it before capturing a stream that will use the handle.
 * Returns ALBIREO_OK and stores the handle in *out, or an error code (then *out = NULL).
 */
int albireo_sample_init(albireo_sampler_t **out, int32_t device,
                        int32_t max_rows, int32_t max_vocab, int64_t max_history_total,
                        void *workspace, size_t workspace_bytes);

/*
 * Samples one token per row (section 6.1 step 3: Y = Sample(Pr)).  Enqueues work on
 * `stream` and returns without synchronising; outputs are valid once the stream
 * reaches that point.  `device` of the handle must be current.
 *
 *   logits        [B, V] row-major (row stride = ext->row_stride_elems or V), dtype
 *                 ALBIREO_F32 (float), ALBIREO_BF16 (bfloat16) or ALBIREO_F16 (half).  Each value finite or
 *                 -inf, at least one finite per row (NaN / +inf: result unspecified but
 *                 in range).  Never written.  16-byte aligned rows take the vector path;
 *                 any element-aligned pointer/stride is accepted.
 *   temperature, top_p, min_p, repetition_penalty, presence_penalty, frequency_penalty
 *                 float[B], top_k int32[B]; a NULL array switches the feature off for
 *                 every row (T = 1, k = 0, top_p = 1, min_p = 0, r = 1, p = 0, f = 0).
 *   history_ids   int32[history_offsets[B]], history_offsets int32[B + 1] (CSR, first
 *                 entry 0); both NULL for "no history".  One history drives all three
 *                 penalties.
 *   seeds         uint64[B] (NULL: all 0); `step` is the decode iteration.
 *   out_tokens    int32[B]; out_logprobs float[B] (log-probability of the token under the
 *                 final kept-set distribution).
 *   stream        a cudaStream_t passed as void* (NULL: the legacy default stream).
 *
 * B = 0 returns ALBIREO_OK without launching.  Errors detectable on the host (NULL
 * required pointer, B < 0 or > max_rows, V < 1 or > max_vocab, unknown dtype, wrong
 * current device, bad ext) return ALBIREO_EINVAL / ALBIREO_EUNSUPPORTED with nothing
 * launched; per-row parameter values live on the device and are clamped as stated above.
 * One call at a time per handle (the workspace is shared by the rows of one call).
 */
int albireo_sample(albireo_sampler_t *h,
                   const void *logits, int32_t B, int32_t V, int32_t dtype,
                   const float *temperature, const int32_t *top_k,
                   const float *top_p, const float *min_p,
                   const float *repetition_penalty, const float *presence_penalty,
                   const float *frequency_penalty,
                   const int32_t *history_ids, const int32_t *history_offsets,
                   const uint64_t *seeds, uint64_t step,
                   int32_t *out_tokens, float *out_logprobs,
                   void *stream, const albireo_sample_ext_t *ext);

/*
 * The same call with every array in HOST memory (pinned memory makes the copies
 * asynchronous): copies the inputs to staging space in the workspace, samples, copies
 * out_tokens / out_logprobs (and the optional ext outputs) back and waits for `stream`.
 * `history_total` is history_offsets[B] (0 without history).  The pointers inside `ext`
 * are host pointers too.  Needs the staging bytes in the workspace given to init.
 */
int albireo_sample_host(albireo_sampler_t *h,
                        const void *logits, int32_t B, int32_t V, int32_t dtype,
                        const float *temperature, const int32_t *top_k,
                        const float *top_p, const float *min_p,
                        const float *repetition_penalty, const float *presence_penalty,
                        const float *frequency_penalty,
                        const int32_t *history_ids, const int32_t *history_offsets,
                        int64_t history_total,
                        const uint64_t *seeds, uint64_t step,
                        int32_t *out_tokens, float *out_logprobs,
                        void *stream, const albireo_sample_ext_t *ext);

/* Frees the handle (host memory only). NULL is accepted. */
int albireo_sample_destroy(albireo_sampler_t *h);

/* Text of the last error recorded on this handle ("" if none); valid until the next call. */
const char *albireo_last_error(const albireo_sampler_t *h);

/* Number of kernel launches albireo_sample has enqueued through this handle so far. */
uint64_t albireo_sample_launch_count(const albireo_sampler_t *h);

/*
 * Measurement aid (the paper has no counterpart): streams the rows of a dense [B, V] logits matrix
 * through the sampler's own shared-memory ring, in the sampler's launch shape, testing every tile
 * against a threshold nothing reaches -- and does nothing else.  Its duration is what the stream
 * alone costs on this GPU at this size; benchmarks report it beside the sampler's.
 *   sink  uint32[B] device: one word per row is written (so that the loads are kept): the number of
 *         (warp, tile) pairs that held a value reaching the threshold -- only +inf does, so 0 for ordinary
 *         rows --, with bit 31 set if a bounded on-chip wait expired.  Only the 16-byte-aligned middle of a
 *         row is streamed (what the sampler's ring carries); a ragged head or tail is not looked at.
 *   drop_tile  -1 for a measurement.  >= 0: the copy of that tile of every row is announced to its
 *         barrier but never issued, so the bounded wait on it must expire: the rows then report bit 31,
 *         the copies still in flight are waited for, and the kernel returns normally.  This is how the
 *         tests exercise the expiry of the ring's bounded waits (the sampler's wait routine, with a bound
 *         of 2^14 polls instead of 2^20 so that the launch stays short) without anything that hangs or faults.
 * Asynchronous on `stream`; errors as albireo_sample.
 */
int albireo_stream_only(albireo_sampler_t *h, const void *logits, int32_t B, int32_t V, int32_t dtype,
                        uint32_t *sink, int32_t drop_tile, void *stream);

/* largest history_total albireo_sample_fixed_scratch accepts (entries of its fixed scratch array) */
#define ALBIREO_FIXED_MAX_HISTORY (1 << 20)

/*
 * albireo_sample for callers that cannot allocate device memory (the paper has no
 * counterpart: this entry point exists for integration, not for the method).
 *
 * Who needs it: code that gets control when every byte of device memory has already been
 * handed to someone else's pool, code that must not call cudaMalloc because that would
 * stall the GPU work around it, and code under a "no allocation after start-up" rule.
 * Such a caller has nowhere to take the workspace of albireo_sample_init from.  Here the
 * one piece of scratch the sampler needs -- the per-row history occurrence counts of rows
 * whose history has more distinct ids than fit on chip -- is a fixed array of
 * ALBIREO_FIXED_MAX_HISTORY 32-bit counters (4 MiB) inside the library's device image;
 * every GPU that loads the library holds that array until the process exits.  There is
 * no handle and no workspace; the entry point calls no allocation routine of any kind.
 *
 * Arguments are those of albireo_sample (device pointers, same meaning and layout),
 * plus history_total = history_offsets[B] as the host knows it (0 without history).
 * Limits: history_total <= ALBIREO_FIXED_MAX_HISTORY, V <= ALBIREO_MAX_VOCAB; anything
 * larger returns ALBIREO_EUNSUPPORTED and launches nothing.  Other host-detectable
 * mistakes return ALBIREO_EINVAL.  The text of the last error on the calling thread is
 * returned by albireo_sample_fixed_scratch_error().
 *
 * First call on each device: looks up the device address of the scratch array and sets
 * the kernels' shared-memory attributes, with that device current.  Make that first call
 * before any stream capture on the device; later calls only enqueue a kernel.
 *
 * The array is shared by every call in the process and keeps whatever the previous call
 * left in it.  Nothing has to be cleared by the caller: each row zeroes the counters it is
 * about to use before counting.  Two calls whose kernels can overlap on the same GPU
 * (different streams, or threads launching at once) race on the array -- serialise them.
 */
int albireo_sample_fixed_scratch(const void *logits, int32_t B, int32_t V, int32_t dtype,
                                 const float *temperature, const int32_t *top_k,
                                 const float *top_p, const float *min_p,
                                 const float *repetition_penalty, const float *presence_penalty,
                                 const float *frequency_penalty,
                                 const int32_t *history_ids, const int32_t *history_offsets,
                                 int64_t history_total,
                                 const uint64_t *seeds, uint64_t step,
                                 int32_t *out_tokens, float *out_logprobs,
                                 void *stream, const albireo_sample_ext_t *ext);

/* Text of the last error albireo_sample_fixed_scratch recorded on the calling thread ("" if none). */
const char *albireo_sample_fixed_scratch_error(void);

#ifdef __cplusplus
}
#endif
#endif /* ALBIREO_SAMPLE_H */
