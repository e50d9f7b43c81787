/*
 * baklava.h - C ABI of the B200 (sm_100a) library for budgeted-KV decode attention.
 *
 * The method: BaKlaVa (arXiv 2502.13176).  Every KV cache (one per layer and KV
 * head) gets its own capacity from a one-time importance profile (Algorithm 1)
 * and a threshold / reduction reallocation rule (Algorithm 2); at inference a
 * cache that is full evicts a token (Eq. 5-6) and attention runs over what is
 * left plus the current token (Eq. 7).
 *
 * Conventions
 *  - Every function returns BAKLAVA_OK (0) or a negative BAKLAVA_ERR_* code and
 *    never throws, aborts or traps.  baklava_strerror() names a code.
 *  - "host" / "device" on a pointer says where the memory lives.  The caller owns
 *    every buffer; the library allocates nothing on the device and keeps no
 *    pointer after a call returns.  Scratch comes from a caller-supplied
 *    workspace whose size the *_workspace_size() functions return.  (One
 *    exception, stated at its declaration: baklava_evict_static keeps its
 *    scratch in an array inside the library image and remembers that array's
 *    device address between calls.)
 *  - Device work is enqueued on `stream` (a cudaStream_t passed as void*) and the
 *    call returns without synchronising.  Argument errors are found on the host
 *    before anything is enqueued.  State errors found on the device (append into
 *    a full cache, inconsistent length) set bits in the cache's device `status`
 *    word, skip the offending head's update and leave the rest of the step
 *    intact; the caller reads the word after synchronising.
 *  - No kernel waits without a limit.  A wait on a tile or on another block that
 *    does not end within the limit (baklava_set_wait_limit; about 50 ms by default)
 *    gives up: BAKLAVA_STATUS_TIMEOUT is set, the kernel first lets every copy it
 *    has requested land, and the head it was working on keeps the state it had
 *    before the step (no output, no score update, no append bookkeeping).  All
 *    counters in the workspace return to zero, so the next step may run on the
 *    same workspace.  The calls that take no cache (baklava_profile_heads,
 *    baklava_prefill_scores) report the same event in the first 32-bit word of
 *    their workspace: the call clears it, bit 0 set after synchronising means a
 *    wait gave up and the results are not to be used.
 *  - slab_off entries, capacities and seq_stride_tokens are multiples of 16 rows
 *    (baklava_allocate produces such layouts); seq_stride_tokens is checked on the
 *    host, a head whose offset or capacity is not is skipped with BAD_STATE.
 *  - bf16 tensors are row-major with the last index fastest; all device pointers
 *    must be 16-byte aligned.
 *  - Supported shapes: D in {64, 128}; Hq a multiple of Hkv with g = Hq / Hkv <= 8;
 *    page a positive multiple of 16; capacities multiples of page.
 */
#ifndef BAKLAVA_H
#define BAKLAVA_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define BAKLAVA_OK                 0
#define BAKLAVA_ERR_INVALID_ARG   (-1)  /* NULL / misaligned pointer, bad range, bad flag            */
#define BAKLAVA_ERR_SHAPE         (-2)  /* unsupported D, g, page ...                                 */
#define BAKLAVA_ERR_CAPACITY      (-3)  /* budget cannot be met inside [min, max]                     */
#define BAKLAVA_ERR_WORKSPACE     (-4)  /* workspace / output buffer too small                        */
#define BAKLAVA_ERR_CUDA          (-5)  /* a CUDA runtime call failed (launch error, no device)       */
#define BAKLAVA_ERR_TIMEOUT       (-6)  /* reserved for bounded device waits                          */
#define BAKLAVA_ERR_UNSUPPORTED   (-7)  /* valid request that this build does not implement           */

/* bits of the device status word */
#define BAKLAVA_STATUS_OVERFLOW    1u   /* a token was offered to a cache with no free slot: not appended */
#define BAKLAVA_STATUS_BAD_STATE   2u   /* len / free_slot outside [0, cap]: head skipped                  */
#define BAKLAVA_STATUS_TIMEOUT     4u   /* a bounded wait inside a kernel gave up: that head's step is lost  */

/* flags of baklava_decode_attn */
#define BAKLAVA_FLAG_NO_APPEND     1u   /* attend over the cache as it is; k_new / v_new ignored      */
#define BAKLAVA_FLAG_NO_SCORE      2u   /* do not accumulate attention into `score`.  Implies NO_EVICT,  */
                                        /*   except under the pure sinks + window policy (recent_num ==   */
                                        /*   recent_den), where the oldest row outside both is evicted:  */
                                        /*   the paper's evaluated policy, with no score traffic at all  */
#define BAKLAVA_FLAG_NO_EVICT      4u   /* never evict; a cache that fills up stays full              */
#define BAKLAVA_FLAG_OVERLAP_PREV   8u   /* this call may start while the work in front of it on the   */
                                        /*   stream is still finishing (see baklava_decode_attn)      */
#define BAKLAVA_FLAG_TEST_STALL  256u   /* test aid, never set it in production: the first chunk of   */
                                        /*   every head is fed its first 64 rows only, so               */
                                        /*   that the bounded wait for the next ones runs out and the   */
                                        /*   time-out path runs (use with a short baklava_set_wait_limit) */

#define BAKLAVA_SCOPE_LAYER        0    /* Algorithm 2 inside each layer                              */
#define BAKLAVA_SCOPE_MODEL        1    /* Algorithm 2 over all L * Hkv caches at once                */

#define BAKLAVA_MAX_GROUP          8

#define BAKLAVA_KV_BF16            0
#define BAKLAVA_KV_FP8_E4M3        1

/* Model attention shape and retention policy. */
typedef struct baklava_shape {
    int32_t L;           /* layers                                                            */
    int32_t Hq;          /* query heads per layer                                             */
    int32_t Hkv;         /* KV heads (= KV caches) per layer; g = Hq / Hkv query heads share one */
    int32_t D;           /* head dimension                                                    */
    int32_t page;        /* capacity granularity in tokens                                    */
    int32_t n_sink;      /* tokens at positions < n_sink are never evicted                    */
    int32_t recent_num;  /* the last W positions are never evicted,                           */
    int32_t recent_den;  /*   W = floor((cap - 1 - n_sink) * recent_num / recent_den)        */
} baklava_shape;

/*
 * The budgeted cache: B sequences, each holding one fixed-capacity slab per
 * (layer, KV head).  All pointers are device memory owned by the caller.
 *
 * Row `slot` of head (l, h) of sequence b is token row
 *     b * seq_stride_tokens + slab_off[l * Hkv + h] + slot          (0 <= slot < cap[l * Hkv + h])
 * of k_slab / v_slab (D bf16 each, or D bytes with BAKLAVA_KV_FP8_E4M3) and the same index of pos / score.
 * len[(b * L + l) * Hkv + h] rows are valid.  They are the slots 0 .. len without
 * free_slot (just 0 .. len-1 while free_slot == len, i.e. until the cache first
 * fills).  The next appended token is written at free_slot.  A cache reset
 * (the RESET_CACHE of Algorithm 3) is len = free_slot = 0.
 *
 * Quantised slabs (the paper names quantisation as a complement to budget allocation and fixes no
 * scheme): with kv_dtype = BAKLAVA_KV_FP8_E4M3 a row element x of head (l, h) is stored as the FP8
 * E4M3 code of fl32(x) * (1 / scale), rounded to nearest even and saturated to +-448, and stands for
 * code * scale from then on, with one caller-chosen fp32 scale for K and one for V per (l, h); the
 * reciprocals are passed alongside so that every implementation multiplies by the same number.
 * baklava_decode_attn(_varlen) and baklava_evict(_varlen) quantise the rows they write (k_new / v_new,
 * the dense prompt) and read the slabs accordingly; queries stay bf16 (they must be finite in fp16:
 * |q| < 65504).  Only D = 128.  Everything else (positions, scores, policy) is unchanged.
 */
typedef struct baklava_cache {
    void*          k_slab;             /* bf16 [B * seq_stride_tokens, D]        */
    void*          v_slab;             /* bf16 [B * seq_stride_tokens, D]        */
    int32_t*       pos;                /* token position of each row             */
    float*         score;              /* accumulated attention of each row      */
    int32_t*       len;                /* [B, L, Hkv]                            */
    int32_t*       free_slot;          /* [B, L, Hkv]                            */
    const int32_t* cap;                /* [L, Hkv] capacity in tokens            */
    const int64_t* slab_off;           /* [L, Hkv] first row of the head's slab  */
    int64_t        seq_stride_tokens;  /* rows per sequence                      */
    int32_t        B;
    uint32_t*      status;             /* one word, OR of BAKLAVA_STATUS_* bits  */
    int32_t        kv_dtype;           /* BAKLAVA_KV_BF16 or BAKLAVA_KV_FP8_E4M3 */
    const float*   kv_scale;           /* FP8 only: [L, Hkv, 4] = K scale, 1 / K scale, V scale, 1 / V scale */
} baklava_cache;

/* Parameters of Algorithm 2 (threshold t, reduction r) and the bounds the paper leaves open. */
typedef struct baklava_alloc_params {
    double        t;                 /* caches with importance < t are reduced                       */
    int32_t       r_num, r_den;      /* each by floor(size * r_num / r_den) pages                    */
    int32_t       scope;             /* BAKLAVA_SCOPE_*                                              */
    int32_t       min_tokens;        /* no cache below this (rounded up to pages)                    */
    int32_t       max_tokens;        /* no cache above this (rounded up to pages)                    */
    const double* layer_importance;  /* host [L] or NULL: with SCOPE_LAYER, Algorithm 2 is first     */
    double        t_layer;           /*   applied to the layers' totals with these parameters;       */
    int32_t       rl_num, rl_den;    /*   NULL splits the total evenly over layers                   */
} baklava_alloc_params;

/* What baklava_decode_plan decided; passed back to baklava_decode_attn unchanged. */
typedef struct baklava_plan_info {
    int32_t n_items;        /* attention work items (one chunk of one head of one sequence each)    */
    int32_t n_score_items;  /* short launches only (all chunks resident at once): pieces of the heads  */
                            /*   for a score / eviction pass of its own, listed after the items; else 0 */
    int32_t n_units;        /* (layer, sequence, KV head) triples in the layer range                */
    int32_t chunk_tokens;   /* target chunk length the plan used                                    */
    int32_t layer_begin, layer_end, B;
    int64_t ws_bytes;       /* workspace baklava_decode_attn needs with this plan                   */
} baklava_plan_info;

const char* baklava_strerror(int code);

/* ------------------------------------------------------------------ Algorithm 1
 * Step 1 on the device: for every prompt p and query head h of ONE layer,
 *   O = softmax(Q K^T / sqrt(D) + causal mask) V,  c_t = cos(V_t, O_t),  s[p, h] = mean_{t < len_p} c_t
 * with V the value rows of KV head h / g (the head's "input") and O its output.
 * The scale and the mask are the model's own (Eq. 1); a zero-norm row gives c_t = 0.
 *   q            device bf16 [P, Hq, T, D]
 *   k, v         device bf16 [P, Hkv, T, D]
 *   prompt_len   device int32 [P] (1 <= len <= T) or NULL for len = T
 *   head_cos     device fp32 [P, Hq], overwritten
 *   token_cos    device fp32 [P, Hq, T] or NULL; rows t >= len_p are left untouched
 *   ws           device workspace, >= baklava_profile_workspace_size() bytes
 */
int baklava_profile_heads(const baklava_shape* shape, const void* q, const void* k, const void* v,
                          const int32_t* prompt_len, int32_t P, int32_t T,
                          float* head_cos, float* token_cos, void* ws, size_t ws_bytes, void* stream);
size_t baklava_profile_workspace_size(const baklava_shape* shape, int32_t P, int32_t T);

/* Step 2 on the host: head similarities -> KV-cache importance.
 *   head_cos       host fp32 [P, L, Hq]  (step 1's output gathered over layers)
 *   kv_importance  host fp64 [L, Hkv]:  1 - mean_{h in group} (mean_p s[p, l, h] + 1) / 2
 * The cosine range [-1, 1] is mapped affinely to [0, 1] before the complement, as
 * the head-importance paragraph describes. */
int baklava_importance(const baklava_shape* shape, const float* head_cos, int32_t P, double* kv_importance);

/* ------------------------------------------------------------------ Algorithm 2
 * Host code, integer page arithmetic.  Start from a uniform split of total_tokens;
 * every cache with importance < t gives up floor(size * r) pages (never going below
 * min); the freed pages are shared by the k = min(n, m - n) most important caches at
 * or above t (ties: lower index), leftovers one page each from the most important
 * down; nothing moves when no cache or every cache is below t.  A cache never exceeds
 * max: what it cannot take goes, one page at a time by descending importance, to the
 * other caches at or above t and then back to the reduced ones.
 *   kv_importance  host fp64 [L, Hkv]
 *   total_tokens   whole-model budget per sequence; must be a multiple of page
 *   cap_out        host int32 [L, Hkv]   capacities in tokens (multiples of page)
 *   slab_off_out   host int64 [L, Hkv]   exclusive prefix sum of cap_out in (l, h) order
 *   seq_stride_out host int64            sum of cap_out
 * BAKLAVA_ERR_CAPACITY if the uniform share is outside [min, max] or the total does not fit. */
int baklava_allocate(const baklava_shape* shape, const double* kv_importance,
                     const baklava_alloc_params* params, int64_t total_tokens,
                     int32_t* cap_out, int64_t* slab_off_out, int64_t* seq_stride_out);

/* ------------------------------------------------------------------ decode step (Eq. 4 - 7)
 * baklava_decode_plan (host): cut the heads of layers [layer_begin, layer_end) of B
 * sequences into work items for one launch.  Largest heads come first; a head of
 * capacity C is cut into chunks of equal length (a multiple of 64 tokens).
 *   cap           host int32 [L, Hkv]
 *   chunk_tokens  target chunk length, 0 = choose from the total work and n_sm
 *   n_sm          streaming multiprocessors of the device (used when chunk_tokens = 0)
 *   kv_dtype      BAKLAVA_KV_* of the cache the plan is for: with one-byte rows a chunk of the same
 *                 length is half the bytes, so the automatic choice makes chunks twice as long
 *   items_out     host int32 [4 * items_capacity] or NULL to only fill `info`
 * The caller copies items_out ((info->n_items + info->n_score_items) * 16 bytes) to the device and hands it
 * to baklava_decode_attn together with `info`. */
int baklava_decode_plan(const baklava_shape* shape, const int32_t* cap, int32_t B,
                        int32_t layer_begin, int32_t layer_end, int32_t chunk_tokens, int32_t n_sm,
                        int32_t kv_dtype, int64_t seq_stride_tokens, int32_t* items_out,
                        int64_t items_capacity, baklava_plan_info* info);

/* One decode step for layers [layer_begin, layer_end) of every sequence, in this order
 * per (sequence, layer, KV head):
 *   1. append k_new / v_new at free_slot with pos = t_pos, score = 0            (Eq. 4)
 *   2. o_q = sum_j softmax_j(q_q . k_j / sqrt(D)) v_j over every valid row, for the g query
 *      heads of the group in one pass over K and V                               (Eq. 7)
 *   3. score_j += sum_q softmax_j(...)_q                        (accumulated attention)
 *   4. if the cache now holds cap rows: evict one.  Never evicted: pos < n_sink and the
 *      last W positions (pos > t_pos - W).  Of the rest the lowest score goes; among equal
 *      scores the latest token goes.  Its slot becomes free_slot.               (Eq. 5-6)
 * t_pos must be larger than every position already in the cache.
 *   q        device bf16 [layers, B, Hq, D]      layers = layer_end - layer_begin
 *   k_new    device bf16 [layers, B, Hkv, D]     (ignored with NO_APPEND)
 *   v_new    device bf16 [layers, B, Hkv, D]
 *   out      device bf16 [layers, B, Hq, D]
 *   lse      device fp32 [layers, B, Hq] natural-log normaliser, or NULL
 *   items    device int32, the plan's items (complete before the call is enqueued, or written by
 *            earlier work on the same stream);  info: the plan's info
 *   ws       device workspace >= info->ws_bytes; must be zero-filled before its first use
 *            and not shared by steps that overlap in time; the library restores the
 *            parts that must be zero before it returns the stream to the caller, also
 *            after a step that set BAKLAVA_STATUS_TIMEOUT.
 * A head with no valid row gives out = 0 and lse = -inf.
 *
 * Ordering on the stream.  A call is one kernel (two for an unflagged short launch: the score update of
 * its few long heads is then spread over a second one), launched with programmatic stream serialisation: its
 * blocks may become resident while the work in front of it drains, and they wait for that work to
 * complete before they read anything.  A model calls attention one layer at a time (Eq. 7 per layer),
 * and a call for one layer is too short to fill the GPU: most of its time is the start-up and the tail
 * (merge of the partial results, score update, eviction) of its few heads.  BAKLAVA_FLAG_OVERLAP_PREV
 * lets a call start streaming its K / V rows at once, beside the tails of the calls in front of it.
 * A run of calls is an unflagged call followed by flagged ones.  By setting the flag the caller vouches
 * that nothing this call reads or writes (the cache state of its layer range, q, k_new, v_new, t_pos,
 * items, out, lse, ws) is written, or has what this call writes read, by any earlier call of the same run
 * or by anything else enqueued on the stream since the run's first call was enqueued: within a run the
 * kernels may all be in flight at once.  The calls for the layers of one decode step qualify when each
 * layer has its own workspace and all their inputs were written before the first of them was enqueued
 * (the first one unflagged, the rest flagged); a call whose q comes out of the kernel just in front of
 * it, or the next step of the same layers, does not.  An unflagged call, and any other work enqueued
 * after a run, starts only when every call of the run has completed (no kernel of the library completes
 * before the kernel in front of it). */
int baklava_decode_attn(const baklava_shape* shape, const baklava_cache* cache,
                        const void* q, const void* k_new, const void* v_new, int32_t t_pos,
                        void* out, float* lse, uint32_t flags,
                        const int32_t* items, const baklava_plan_info* info,
                        void* ws, size_t ws_bytes, void* stream);

/* The same step for a batch whose sequences are at different positions (requests that joined at
 * different times, prompts of different lengths).  Eq. 4-7 are per sequence, so nothing in them
 * changes: sequence b runs the step above with t_pos[b].  A negative t_pos[b] marks a sequence that
 * sits this step out: none of its cache, out or lse entries is read or written.
 *   t_pos    device int32 [B]; every other argument as for baklava_decode_attn */
int baklava_decode_attn_varlen(const baklava_shape* shape, const baklava_cache* cache,
                               const void* q, const void* k_new, const void* v_new, const int32_t* t_pos,
                               void* out, float* lse, uint32_t flags,
                               const int32_t* items, const baklava_plan_info* info,
                               void* ws, size_t ws_bytes, void* stream);

/* Upper bound, in SM clock cycles, of every wait inside the decode kernels from the next call on
 * (process-wide; default 100 000 000, about 50 ms).  A wait that runs out sets BAKLAVA_STATUS_TIMEOUT
 * as the conventions above describe.  sm_cycles > 0. */
int baklava_set_wait_limit(int64_t sm_cycles);

/* ------------------------------------------------------------------ bulk eviction (Eq. 5-6)
 * Cut dense prefilled heads of T tokens down to their capacities and compact them into
 * the slabs (the MAKE_CACHE of Algorithm 3).  Row t of head (layer, b, h) is token row
 *     (layer - layer_begin) * stride_layer + b * stride_seq + h * stride_head + t
 * of k_dense / v_dense (D bf16 each) and of score_dense (fp32, NULL = all zero); its
 * position is t.  With R = cap - reserve: all rows are kept if T <= R; otherwise the
 * rows with pos < n_sink, the last W = floor((R - n_sink) * recent_num / recent_den)
 * positions, and the R - n_sink - W rows of the rest that rank first by (score
 * descending, position ascending).  Kept rows land in slots 0 .. n'-1 in ascending
 * position with their scores; len = free_slot = n'.   reserve >= 1.
 *   ws   device workspace >= baklava_evict_workspace_size() bytes
 *
 * In place (k_dense = v_dense = NULL; score_dense must be NULL too, the strides are ignored): the
 * same rule applied to the len rows every slab already holds, with their own positions and scores
 * (the latest position present takes the place of T - 1): a budget that shrank, a cache that filled
 * up under NO_EVICT, a freed slot to close.  Eq. 5-6 remove rows and keep the order of the others:
 * the kept rows move down to slots 0 .. n'-1 in the order they have in the slab (ascending position
 * for a slab that baklava_evict filled); len = free_slot = n'.  Here T only sizes the workspace and
 * must be at least the largest capacity in the layer range (a larger head is skipped with
 * BAD_STATE, as is one whose len / free_slot are inconsistent). */
int baklava_evict(const baklava_shape* shape, const baklava_cache* cache,
                  int32_t layer_begin, int32_t layer_end,
                  const void* k_dense, const void* v_dense, const float* score_dense, int32_t T,
                  int64_t stride_layer, int64_t stride_seq, int64_t stride_head, int32_t reserve,
                  void* ws, size_t ws_bytes, void* stream);
size_t baklava_evict_workspace_size(const baklava_shape* shape, int32_t B, int32_t layers, int32_t T);

/* The same for prompts of different lengths: sequence b has prompt_len[b] tokens (clamped to
 * 0 .. T; rows at or past it are not tokens and are never read), and the rule above is applied
 * with that length in place of T.  A sequence of length 0 ends with len = free_slot = 0.
 *   prompt_len  device int32 [B], or NULL for T everywhere (then identical to baklava_evict)
 * The workspace is sized for T as in baklava_evict. */
int baklava_evict_varlen(const baklava_shape* shape, const baklava_cache* cache,
                         int32_t layer_begin, int32_t layer_end,
                         const void* k_dense, const void* v_dense, const float* score_dense, int32_t T,
                         const int32_t* prompt_len,
                         int64_t stride_layer, int64_t stride_seq, int64_t stride_head, int32_t reserve,
                         void* ws, size_t ws_bytes, void* stream);

/* ------------------------------------------------------------------ prompt scores (seed of step 3)
 * The accumulated attention a prompt leaves on its own tokens, for ONE layer: with the causal
 * attention matrix A_h = softmax(Q_h K^T / sqrt(D)) of Eq. 1,
 *     score[b, c, j] = sum over the g query heads h of KV head c, sum over rows i >= j of A_h[i, j],
 * exactly what decoding the prompt one token at a time through baklava_decode_attn would have
 * accumulated.  It is the score_dense input of baklava_evict (stride_seq = Hkv * T, stride_head = T).
 *   q           device bf16 [B, Hq, T, D]
 *   k           device bf16 [B, Hkv, T, D]
 *   prompt_len  device int32 [B] (rows and keys at or past len count for nothing) or NULL for len = T
 *   lse         device fp32 [B, Hq, T] or NULL: the natural-log normaliser of every causal row i,
 *               log sum_{j <= i} exp(q_i . k_j / sqrt(D)), as the attention kernel that processed the
 *               prompt leaves it (rows at or past prompt_len are not read).  With it the call makes one
 *               pass over Q K^T instead of two; the result is the same up to the rounding of lse.
 *   score       device fp32 [B, Hkv, T], overwritten
 *   ws          device workspace >= baklava_prefill_workspace_size() bytes */
int baklava_prefill_scores(const baklava_shape* shape, const void* q, const void* k,
                           const int32_t* prompt_len, const float* lse, int32_t B, int32_t T,
                           float* score, void* ws, size_t ws_bytes, void* stream);
size_t baklava_prefill_workspace_size(const baklava_shape* shape, int32_t B, int32_t T);

/* ------------------------------------------------------------------ Algorithm 3 (parameter search)
 * The search evaluates every candidate (t, r): make the cache (baklava_allocate + baklava_evict),
 * run the evaluation chunks through it, average the chunk losses, keep the best.  The paper's
 * loss is a model's perplexity; this library has no model, so it offers the loss that can be
 * computed from the attention path alone: how far the budgeted cache moves the attention outputs
 * away from those of the dense cache,
 *     loss = mean over rows i of ||out_i - ref_i||^2 / max(||ref_i||^2, 1e-30),
 * rows being the output vectors of every (layer, sequence, query head) of one or more steps.
 *   out, ref   device bf16 [rows, D], D even
 *   loss       device fp64 [1], overwritten (0 for rows = 0)
 *   ws         device workspace >= baklava_output_error_workspace_size(rows) bytes
 * Row sums are taken in fp32, the mean over rows in fp64, both in a fixed order. */
int baklava_output_error(const void* out, const void* ref, int64_t rows, int32_t D, double* loss,
                         void* ws, size_t ws_bytes, void* stream);
size_t baklava_output_error_workspace_size(int64_t rows);

/* The search's selection rule, on the host: *best = index of the first strictly smallest average
 * loss (a later equal loss does not replace it, a NaN never wins), -1 if no entry is below +inf.
 *   avg_loss   host fp64 [n] */
int baklava_search_pick(const double* avg_loss, int32_t n, int32_t* best);

/* ------------------------------------------------------------------ bulk eviction, no workspace
 * (No counterpart in the paper: this is a packaging variant of baklava_evict.)
 * Same operation, arguments, results and return codes as baklava_evict, for callers that cannot provide a
 * workspace because they cannot allocate device memory where the call is made: code running
 * inside a host framework whose memory pool is exhausted or frozen, plug-ins that are handed
 * only their input and output buffers, and start-up code that runs before an allocator exists.
 * The list of kept rows is kept in a fixed array that is part of the library image: 4 MiB
 * (BAKLAVA_EVICT_STATIC_MAX_ENTRIES = 2^20 int32 entries) on every GPU that loads the
 * library, held until the process exits.  The call itself allocates and frees nothing.
 *  - Limit: (layer_end - layer_begin) * B * Hkv * T <= BAKLAVA_EVICT_STATIC_MAX_ENTRIES;
 *    larger requests return BAKLAVA_ERR_WORKSPACE before anything is enqueued.
 *  - The first call on each device looks up the array's device address (the device must be
 *    current) and the library remembers it.  Make that first call outside any stream capture.
 *    The address dies with the device's context: a process that calls cudaDeviceReset must not
 *    call this entry point afterwards.
 *  - All calls on a device share the one array and it keeps the previous call's contents.
 *    Every entry that is read is written earlier in the same call, so nothing has to be
 *    cleared; but two calls whose kernels overlap on the GPU (different streams) race on it.
 *    Serialise them on one stream, or use baklava_evict with separate workspaces. */
#define BAKLAVA_EVICT_STATIC_MAX_ENTRIES (1u << 20)
int baklava_evict_static(const baklava_shape* shape, const baklava_cache* cache,
                         int32_t layer_begin, int32_t layer_end,
                         const void* k_dense, const void* v_dense, const float* score_dense, int32_t T,
                         int64_t stride_layer, int64_t stride_seq, int64_t stride_head, int32_t reserve,
                         void* stream);

#ifdef __cplusplus
}
#endif
#endif /* BAKLAVA_H */
