/*
 * st3.h -- C ABI of the ST^3 decode-attention + visual-token-trimming library (sm_100a).
 *
 * The library keeps, per decoder layer and per sequence, a key/value cache whose rows are
 * [system | kept visual | instruction text | generated] tokens (Eq. 1 of the ST^3 paper:
 * X = [S, V, I, O]).  One decode step, for every requested layer and sequence,
 *   1. appends the new token's key/value row,
 *   2. computes the current query's softmax attention over every cached row (Eq. 2, last row),
 *   3. accumulates each visual token's attention probability over heads (the score alpha
 *      of Sec. 3.2),
 *   4. if the retention schedule asks for fewer visual rows than are held, keeps the
 *      top-scoring ones (Eq. 3, ties toward the lower original visual index), and
 *   5. compacts the kept K/V rows in place.
 * The retention schedule is PVTP per layer (Sec. 3.2, Algorithm 1, Eq. 9) times VTA per step
 * (Sec. 3.3, Eq. 7 and Eq. 8).
 *
 * Conventions for every entry point
 *   - "dev" pointers are CUDA device pointers, "host" pointers are ordinary host memory.
 *   - All device pointers must be 16-byte aligned; tensors are dense, row-major, in the
 *     element type named by st3_config.dtype.
 *   - The caller owns every buffer, including the workspace; the library allocates no device
 *     memory and frees only its own host-side context.
 *   - Work is enqueued on the given CUDA stream (a cudaStream_t passed as void*) and the call
 *     returns without waiting for it unless stated otherwise.  Calls on one context must be
 *     issued in program order; buffers must stay valid until the enqueued work has finished.
 *   - Inputs are read in plain stream order: whatever the stream ran before the call has finished, and its
 *     writes are visible, before a kernel of the call reads them (see st3_set_overlap for the one exception).
 *   - A call that fails with ST3_ERR_CUDA after it has begun to enqueue work leaves the context unusable:
 *     every later prefill or decode call on it returns ST3_ERR_BAD_STATE.  Destroy it and create a new one.
 *   - Errors are reported through the return code.  Problems detected on the device (a count
 *     that disagrees with the schedule, a non-finite score, a copy that never arrived) are
 *     OR-ed into a device status word read with st3_get_status.  The library never aborts,
 *     throws or traps.
 */
#ifndef ST3_H_
#define ST3_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct st3_ctx st3_ctx;

typedef enum {
  ST3_OK = 0,
  ST3_ERR_INVALID_ARG = 1,         /* null / misaligned pointer, out-of-range value            */
  ST3_ERR_WORKSPACE_TOO_SMALL = 2, /* workspace smaller than st3_workspace_size reports        */
  ST3_ERR_BAD_STATE = 3,           /* call order violated (decode before prefill, step gap)    */
  ST3_ERR_CAPACITY = 4,            /* text length or step beyond the configured maximum        */
  ST3_ERR_CUDA = 5,                /* a CUDA runtime call failed                               */
  ST3_ERR_DEVICE_CHECK = 6,        /* st3_get_status found a non-zero device status word       */
  ST3_ERR_UNSUPPORTED = 7          /* shape outside what the kernels are built for             */
} st3_status;

typedef enum { ST3_F32 = 0, ST3_BF16 = 1 } st3_dtype;

/* Attenuation function beta(t) of VTA: Eq. 8 (cosine) and the two alternatives of Sec. 4.4. */
typedef enum { ST3_ANNEAL_COSINE = 0, ST3_ANNEAL_NONE = 1, ST3_ANNEAL_LINEAR = 2, ST3_ANNEAL_EXP = 3 } st3_anneal;

/* Bits of the device status word. */
enum {
  ST3_DEV_COUNT_MISMATCH = 1,  /* a layer's device-side visual count differs from the schedule */
  ST3_DEV_NONFINITE = 2,       /* a visual score was NaN/Inf/negative                          */
  ST3_DEV_COPY_TIMEOUT = 4,    /* an asynchronous shared-memory copy did not complete in time  */
  ST3_DEV_RANGE = 8            /* an index left its buffer (the access was skipped)            */
};

typedef struct {
  int32_t num_layers;        /* L: decoder layers (<= 64)                                       */
  int32_t num_heads;         /* H: multi-head attention, kv heads == query heads (<= 128)       */
  int32_t head_dim;          /* D: 64 or 128                                                    */
  int32_t dtype;             /* st3_dtype of q/k/v/out and of the cache                          */
  int32_t batch;             /* B: independent sequences                                        */
  int32_t sys_len;           /* |S|: system-prompt tokens in front of the visual span           */
  int32_t num_visual;        /* |V| at the input of layer 0                                     */
  int32_t max_text_len;      /* capacity for |I| per sequence                                   */
  int32_t max_decode_steps;  /* capacity for |O|                                                */
  int32_t first_prune_layer; /* 3: layers 0-2 are never pruned (Sec. 3.2)                       */
  int32_t stride;            /* S: prune at layers first, first+S, ... (Algorithm 1)            */
  int32_t first_ratio_bp;    /* P in basis points of |V|; the paper sets 50% = 5000 (Eq. 9)     */
  int32_t step_ratio_bp;     /* R in basis points of |V| removed at each later pruning layer    */
  int32_t anneal;            /* st3_anneal                                                      */
  int32_t disable_trim;      /* 1: same kernels, nothing is ever evicted (full-KV comparison)   */
  int32_t rows_per_chunk;    /* cache rows of one work item of the attention kernel; 0 = choose  */
  int32_t static_rank;       /* 1: Algorithm 3 as printed, see below; 0: re-rank at every step   */
  int32_t stage_shared;      /* 1: the layers between two pruning layers keep the pruning layer's */
                             /*    choice (Sec. 3.2, strided pruning); 0: every layer chooses     */
  int32_t host_prefill;      /* 1: the workspace holds two per-layer staging areas for the prompt's */
                             /*    K/V, which st3_prefill_select_host needs; 0: no such areas      */
  uint64_t lazy_mask;        /* bit l set: layer l is lazy (QK heredity, Eq. 6, Algorithm 2)      */
  double tau;                /* Eq. 8: beta = cos(t*pi/(2 tau)) for t < tau, else 0             */
  double sigma;              /* only ST3_ANNEAL_EXP: beta = exp(-t/sigma)                       */
} st3_config;

/* static_rank = 1 selects the decode half of Algorithm 3 literally: prefill stores the kept visual
 * rows in the order of the saved top-index list T[l] (best score first, ties toward the lower
 * original index), and decode step t first cuts the visual rows to the first n(l, t) of that order
 * (T' = T[l][:n], C = C[T']: no scoring, no selection, no row moves) and then attends.  With
 * static_rank = 0 (default) every step attends first and then re-ranks the held rows by the current
 * query's scores. */

/* stage_shared = 1: pruning layers are first, first+S, ...; a layer between two of them evicts
 * exactly the tokens its pruning layer evicts (decided by the pruning layer's scores), so all layers
 * of a stage hold the same visual tokens in the same order.  Within one step the pruning layer must be
 * processed before (or in the same call as) the layers that follow it, else ST3_ERR_BAD_STATE. */

/* lazy_mask: a lazy layer inherits Softmax(Q K^T / sqrt(d)) of the nearest lower layer that is not
 * lazy and applies it to its own values (Eq. 6; Algorithm 2's A = U[-1]): its q and k_new inputs are
 * ignored and its key rows are never read.  Source and lazy layer must hold the same tokens in the
 * same order: both below first_prune_layer, or both in one pruning stage with stage_shared = 1 (else
 * st3_create returns ST3_ERR_INVALID_ARG), and they must be processed in the same call (else
 * ST3_ERR_UNSUPPORTED).  In this version a lazy layer re-reads its source's keys (same bytes as a
 * normal layer); what it saves is the key cache and the key/query projections of the caller. */

/* Scheduled visual-row count n(l, t) of layer `layer` after decode step `step` (0 = after
 * prefill).  Pure host function.  PVTP: layers below first_prune_layer keep everything; layer l
 * in stage k = (l - first)/S keeps floor(|V| * (1 - P - k R)) (Eq. 9 read additively, the
 * reading that reproduces the paper's printed (S, R, C) tables).  VTA: n(l,t) =
 * floor(n(l,0) * beta(t)) (Eq. 7, Eq. 8).  Returns -1 on an invalid argument. */
int32_t st3_schedule_count(const st3_config* cfg, int32_t layer, int32_t step);

/* Bytes of device workspace st3_create needs for `cfg` (host call, no CUDA work). */
st3_status st3_workspace_size(const st3_config* cfg, size_t* bytes);

/* Builds a context over a caller-owned device workspace (256-byte aligned, `bytes` long, on the
 * current device).  Host-side set-up (it also creates two CUDA streams and a few events for the
 * host-buffer calls; no device memory) plus one cudaMemsetAsync of the bookkeeping area on the
 * default stream, which is synchronised before returning.  *out is NULL on failure. */
st3_status st3_create(const st3_config* cfg, void* dev_workspace, size_t bytes, st3_ctx** out);

/* Prefill half of Algorithm 3 for layers [layer_begin, layer_begin+layer_count): ingests the
 * prompt's K/V rows into the cache, attends with the last prompt token's query over the whole
 * prompt, scores the visual tokens and keeps the n(l,0) best (Eq. 3).
 *   q_last   dev  [layer_count][B][H][D]
 *   k, v     dev  [layer_count][B][H][t0_max][D], t0_max = sys_len + num_visual + max_text_len,
 *                 rows in the order [S | V | I]; rows past a sequence's text length are ignored
 *   text_len host [B], each in [1, max_text_len]; read before the call returns; must be the
 *                 same values for every layer range of one generation
 *   out      dev  [layer_count][B][H][D] attention output of the last prompt token
 * Resets the step counter of those layers to 0.  A call with layer_begin == 0 (or with other text lengths
 * than the last one) opens a new generation: every other layer must be prefilled again before it decodes,
 * so prefill layer 0 first when the layers are prefilled one call at a time. */
st3_status st3_prefill_select(st3_ctx* ctx, int32_t layer_begin, int32_t layer_count,
                              const void* q_last, const void* k, const void* v,
                              const int32_t* text_len, void* out, void* cuda_stream);

/* Prefill as Algorithm 1 and Eq. 3 word it: the visual tokens of each layer are pruned BEFORE the
 * layer runs, by scores that come from outside (the previous layer's alpha), and the layer then
 * attends over [S | kept V | I] only.  Same arguments as st3_prefill_select plus
 *   scores   dev  [layer_count][B][num_visual] fp32, any finite values, indexed by original visual
 *                 index; the n(l,0) largest are kept (ties toward the lower index)
 * st3_get_kept's mass then returns these scores. */
st3_status st3_prefill_select_scored(st3_ctx* ctx, int32_t layer_begin, int32_t layer_count,
                                     const void* q_last, const void* k, const void* v,
                                     const int32_t* text_len, const float* scores, void* out,
                                     void* cuda_stream);

/* One decode step (Algorithm 3's decode half with Eq. 7) for the given layers: append, attend,
 * score, select, compact.  `step` counts from 1 and must be the previous step of each of these
 * layers plus one (else ST3_ERR_BAD_STATE); step > max_decode_steps gives ST3_ERR_CAPACITY.
 *   q, k_new, v_new  dev [layer_count][B][H][D]   query and new key/value row of this step
 *   out              dev [layer_count][B][H][D]   attention output
 * After the call the cache of layer l holds n(l, step) visual rows. */
st3_status st3_decode_step(st3_ctx* ctx, int32_t step, int32_t layer_begin, int32_t layer_count,
                           const void* q, const void* k_new, const void* v_new, void* out,
                           void* cuda_stream);

/* Lets a decode step's attention kernel start while the launch ahead of it in the stream is still running
 * (programmatic dependent launch; on = 1).  Back-to-back decode steps then overlap: the next step's attention
 * over rows that the previous step's selection does not touch runs under that selection, and per-(layer,
 * sequence) flags order the rest.  The price is a promise by the caller: q, k_new and v_new of a step are
 * complete in device memory BEFORE the launch ahead of st3_decode_step in the stream begins; in particular
 * the kernel that produces them must not signal programmatic completion (griddepcontrol.launch_dependents,
 * cudaTriggerProgrammaticLaunchCompletion) before its last write to them.  Off by default: every kernel of
 * a call then starts only after all earlier work of the stream has finished. */
st3_status st3_set_overlap(st3_ctx* ctx, int32_t on);

/* Same step with HOST buffers (pinned memory, else the copies do not overlap anything): the library copies
 * q/k_new/v_new to one of two staging areas inside its workspace, runs the step on `cuda_stream` and copies
 * `out` back.  The copies travel on two streams of the library's own, so that the inputs of step t+1 and the
 * output of step t-1 move while the kernels of step t run.  Consequences for the caller:
 *   - the input buffers must hold their final contents when the call is made (they are read without waiting
 *     for earlier work of `cuda_stream`) and must stay untouched until the step's kernels have run;
 *   - out_host is complete once `cuda_stream` has passed a later st3_host_sync (or after st3_get_status, which
 *     waits for everything).
 * When the three inputs lie back to back in host memory (k_new_host = q_host + size, v_new_host = k_new_host
 * + size), they travel as one copy. */
st3_status st3_decode_step_host(st3_ctx* ctx, int32_t step, int32_t layer_begin, int32_t layer_count,
                                const void* q_host, const void* k_new_host, const void* v_new_host,
                                void* out_host, void* cuda_stream);

/* st3_prefill_select with HOST buffers (pinned), same shapes: the prompt's K/V rows travel layer by layer
 * through two staging areas (st3_config.host_prefill = 1, else ST3_ERR_BAD_STATE), so that layer l is ingested,
 * attended and trimmed while layer l+1 is on the bus.  Same rules for the buffers as st3_decode_step_host.
 * Not available with lazy layers (a lazy layer and its source must share a call): ST3_ERR_UNSUPPORTED. */
st3_status st3_prefill_select_host(st3_ctx* ctx, int32_t layer_begin, int32_t layer_count, const void* q_last_host,
                                   const void* k_host, const void* v_host, const int32_t* text_len,
                                   void* out_host, void* cuda_stream);

/* Makes `cuda_stream` wait for every copy back to host memory that the two calls above have started. */
st3_status st3_host_sync(st3_ctx* ctx, void* cuda_stream);

/* Observability: copies layer `layer`'s kept original visual indices (ids dev [B][num_visual],
 * first count[b] entries valid, cache order), counts (count dev [B]) and, if mass != NULL, the
 * score computed at each token's most recent selection indexed by ORIGINAL visual index
 * (mass dev [B][num_visual]; entries of tokens never scored are 0). */
st3_status st3_get_kept(st3_ctx* ctx, int32_t layer, int32_t* ids, int32_t* count, float* mass,
                        void* cuda_stream);

/* Copies cache rows of (layer, sequence b, head h) to dev buffers of the cache dtype, for tests:
 * k_vis/v_vis [num_visual][D] (first count rows valid), k_txt/v_txt [cap][D] with
 * cap = sys_len + max_text_len + max_decode_steps, rows [S | I | O].  Any pointer may be NULL. */
st3_status st3_get_rows(st3_ctx* ctx, int32_t layer, int32_t b, int32_t h, void* k_vis, void* v_vis,
                        void* k_txt, void* v_txt, void* cuda_stream);

/* Synchronises the stream last used by this context (and the library's copy streams) and returns the device status word through
 * *word (host).  Returns ST3_ERR_DEVICE_CHECK if it is non-zero; the word is sticky and the results of
 * a context that has reported one are undefined from then on: destroy it and create a new one. */
st3_status st3_get_status(st3_ctx* ctx, int32_t* word);

/* Visual + non-visual K/V rows currently held, summed over layers and sequences (host
 * bookkeeping, exact by the schedule); multiply by 2*H*D*sizeof(element) for bytes. */
st3_status st3_rows_held(st3_ctx* ctx, int64_t* visual_rows, int64_t* other_rows);

/* Kernel timing for roofline reports.  While enabled, every prefill/decode call records CUDA
 * events around its attention kernel and around its select/compact kernel on the call's stream.
 * st3_profile_read synchronises, returns the accumulated milliseconds and launch counts since
 * enabling (any pointer may be NULL) and clears them. */
st3_status st3_profile_enable(st3_ctx* ctx, int32_t on);
st3_status st3_profile_read(st3_ctx* ctx, double* attn_ms, double* finish_ms, int64_t* attn_launches,
                            int64_t* finish_launches);

/* Total kernels this context has launched so far (host counter). */
int64_t st3_launch_count(const st3_ctx* ctx);

/* Causal self-attention of a whole prompt (Eq. 2: A = Softmax((Q K^T + M)/sqrt(d)), out = A V, row i sees
 * keys 0..i), the step that produces what st3_prefill_select consumes.  Runs on the tcgen05 tensor cores;
 * bf16 and head_dim 128 only (else ST3_ERR_UNSUPPORTED).  A "head instance" is one (sequence, head) pair.
 *   q, k, v     dev [num_inst][seq_len][128] bf16, instance = sequence * num_heads + head
 *   out         dev [num_inst][seq_len][128] bf16
 *   head_probs  dev [num_inst][num_visual] fp32 scratch (the last row's probabilities per head)
 *   scores      dev [num_inst / num_heads][num_visual] fp32: the last query row's attention on the visual
 *               positions [sys_len, sys_len + num_visual), summed over heads -- the alpha of Sec. 3.2 that
 *               Eq. 3 uses to prune the NEXT layer (feed it to st3_prefill_select_scored).
 *               head_probs and scores may be NULL when num_visual is 0.
 *   dev_status  dev int, may be NULL: ST3_DEV_COPY_TIMEOUT is OR-ed in if a copy or an MMA never completes,
 *               ST3_DEV_RANGE if a block finds its shared-memory window misaligned (it then does nothing)
 * Needs no context and no workspace beyond head_probs. */
st3_status st3_prefill_attend(const void* q, const void* k, const void* v, void* out, float* head_probs,
                              float* scores, int* dev_status, int32_t num_inst, int32_t num_heads,
                              int32_t seq_len, int32_t head_dim, int32_t dtype, int32_t sys_len,
                              int32_t num_visual, void* cuda_stream);

/* The same for a layer that runs on the visual tokens an earlier layer kept (Algorithm 1: the sequence that
 * enters layer l is [S | kept V | I]; Eq. 3 prunes layer l+1 by layer l's alpha).  num_visual is the number of
 * kept tokens in the prompt given here, and
 *   ids               dev [num_inst / num_heads][num_visual] int32: original index (< num_visual_total) of the
 *                     token at each visual position, e.g. what st3_get_kept returned for this layer
 *   scores            dev [num_inst / num_heads][num_visual_total] fp32, indexed by ORIGINAL visual index: the
 *                     head-summed probability of the tokens held, -1 for every token not held (below any
 *                     probability, so st3_prefill_select_scored of the next layer never keeps one of them while
 *                     its count does not exceed num_visual)
 * An id outside [0, num_visual_total) sets ST3_DEV_RANGE in *dev_status and is skipped.  With num_visual = 0
 * the scores are all -1. */
st3_status st3_prefill_attend_kept(const void* q, const void* k, const void* v, void* out, float* head_probs,
                                   float* scores, int* dev_status, int32_t num_inst, int32_t num_heads,
                                   int32_t seq_len, int32_t head_dim, int32_t dtype, int32_t sys_len,
                                   int32_t num_visual, const int32_t* ids, int32_t num_visual_total,
                                   void* cuda_stream);

/* Attention of one query per head over dense K/V with NO workspace and no allocation of any kind
 * (the paper has no counterpart; this exists for callers that may not allocate device memory:
 * a plugin handed only its input and output tensors, code running inside a region whose memory
 * another allocator owns, a process whose device memory is already fully committed).
 *   q   dev [H][D]            k, v  dev [H][num_rows][D]            out  dev [H][D]
 * computes out[h] = softmax(q[h] . k[h]^T / sqrt(D)) v[h], i.e. Eq. 2's last row, like
 * st3_prefill_select does for a prompt of num_rows tokens.  The split partials go to a fixed
 * array inside the library image (4 259 840 bytes, resident on every GPU that has loaded the
 * library until the process exits), which limits a call to
 *     num_heads * ceil(num_rows / 128) <= 8192        (else ST3_ERR_CAPACITY, nothing is launched).
 * No cudaMalloc/cudaFree and no allocating library routine is called.  The first call on each
 * device looks up the array's device address (cudaGetSymbolAddress, with that device current);
 * make that first call before starting any stream capture.  All calls on a device share the one
 * array and it keeps the previous call's contents: nothing in it needs to start at zero (every
 * slot a call reads it has written first), but two calls whose kernels overlap on the GPU
 * (different streams, no dependency between them) race on it and must be ordered by the caller. */
st3_status st3_attend_noalloc(const void* q, const void* k, const void* v, void* out, int32_t num_heads,
                              int32_t num_rows, int32_t head_dim, int32_t dtype, void* cuda_stream);

const char* st3_status_string(st3_status s);

/* Frees the host-side context.  Does not synchronise and does not touch the workspace. */
st3_status st3_destroy(st3_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* ST3_H_ */
