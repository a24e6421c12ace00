/*
 * lethe.h — C ABI of the B200 (sm_100a) Lethe hot path.
 *
 * Lethe (arXiv 2511.06029) keeps the KV cache of a decoding LLM small by pruning it
 * repeatedly during generation: per layer, guided by measured attention sparsity
 * (Sec. 4.2), and per token, guided by a decayed record of the attention each cached
 * token has received (RASR, Sec. 4.3, Eq. 5).  This library is the data-parallel part
 * of that loop:
 *
 *   lethe_decode_attend      one decode step: append the new token's k/v, softmax
 *                            attention of the new query over the retained tokens, and
 *                            the Eq. 5 relevance update, in one pass over K and V
 *   lethe_estimate_sparsity  Eq. 1 (Hoyer) on the relevance vectors -> one value per
 *                            (layer, sequence)
 *   lethe_alloc_budgets      per-layer token budgets from those sparsities (Sec. 4.2)
 *   lethe_rasr_prune         protected top-k retention + in-place stable compaction
 *                            (Sec. 4.3; sink / recent sets of Algorithm 1)
 *   lethe_prefill_seed       the same relevance for the prompt, from the prefill attention
 *                            (Eq. 2 with Q > 1)
 *   lethe_segment_prune      Algorithm 1 itself: segmented breakpoint search, retention
 *                            set and eviction-threshold update (Sec. 4.2)
 *   lethe_collapsed_prune    retention by the head- and batch-collapsed score of Eq. 2
 *
 * General conventions
 *   - Unless marked HOST, every pointer is a DEVICE pointer to memory owned by the
 *     caller; the library owns only the scratch inside lethe_ctx.
 *   - All arrays are dense row-major in the index order written beside them.
 *   - Every call that takes a `stream` enqueues its work there (a cudaStream_t passed as
 *     void*, NULL = the legacy default stream) and returns without synchronising.
 *   - Errors detectable on the host return a status and enqueue nothing.  Conditions
 *     only the device can see (a full cache on append, a budget below the protected
 *     count, a page id outside the pool) never trap: the kernel skips or clamps the
 *     item as documented, and records the first such event in a status word that
 *     lethe_poll_status reads.
 *   - Same inputs and same tuning give bitwise-identical results.  budgets, keep_idx,
 *     len and the moved rows have exactly one correct value; out, rel and sparsity are
 *     floating-point results.
 *
 * Notation: L layers, B sequences, Hq / Hkv query / KV heads, G = Hq / Hkv query heads
 * per KV head (head h reads KV head h / G — the contiguous grouping that Eq. 3's
 * `repeat` would produce), D head dimension.  An "item" is one (layer, sequence, KV
 * head); n = len[item] is its number of retained tokens; slot j < n of an item is its
 * j-th retained token in original order.
 */
#ifndef LETHE_H
#define LETHE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct lethe_ctx lethe_ctx; /* opaque: device id, scratch, status word, tuning */

typedef enum {
    LETHE_OK = 0,
    LETHE_ERR_INVALID_ARG = 1, /* null pointer, bad shape / dtype / range */
    LETHE_ERR_CAPACITY = 2,    /* device-side: append on an item with len == capacity */
    LETHE_ERR_BUDGET = 3,      /* budget below the protected (sink + recent) count, or total < L * k_min */
    LETHE_ERR_CUDA = 4,        /* a CUDA runtime call failed; see lethe_last_error */
    LETHE_ERR_TIMEOUT = 5,     /* device-side: a bounded wait inside a kernel ran out (see lethe_set_wait_limit) */
    LETHE_ERR_UNSUPPORTED = 6, /* valid request outside what the kernels cover */
    LETHE_ERR_PAGE = 7,        /* device-side: page id outside [0, n_pages) */
    LETHE_ERR_TOO_LARGE = 8    /* lethe_rasr_prune_static: the cache exceeds LETHE_STATIC_PRUNE_MAX_ENTRIES */
} lethe_status;

enum { LETHE_F32 = 0, LETHE_BF16 = 1, LETHE_FP8_E4M3 = 2, LETHE_FP8_E5M2 = 3 };
enum { LETHE_CONTIG = 0, LETHE_PAGED = 1 };

/* Cache state of all layers (Sec. 4.1: per-layer K, V; Sec. 4.3: the score vector s_t). */
typedef struct {
    int32_t n_layers, batch, n_q_heads, n_kv_heads;
    int32_t head_dim;    /* 64 or 128 */
    int32_t dtype;       /* LETHE_F32 or LETHE_BF16: type of k, v, q, k_new, v_new, out.  LETHE_FP8_E4M3 / LETHE_FP8_E5M2:
                            k and v are bytes of that format (see k_scale), q, k_new, v_new, out are bf16 */
    int32_t layout;      /* LETHE_CONTIG or LETHE_PAGED */
    int32_t capacity;    /* CONTIG: token slots per item.  PAGED: page-table entries per item */
    int32_t page_tokens; /* PAGED: tokens per page (16); CONTIG: ignored */
    void *k, *v;         /* CONTIG: [L][B][Hkv][capacity][D].  PAGED: pools [n_pages][page_tokens][D] */
    float *rel;          /* [L][B][Hkv][cap_tokens]  Eq. 5 state s_t, indexed by logical slot           */
    int32_t *pos;        /* [L][B][Hkv][cap_tokens]  original position of the token in each slot        */
    int32_t *len;        /* [L][B][Hkv]              retained tokens per item                           */
    int32_t *page_table; /* PAGED: [L][B][Hkv][capacity] page ids (never written by the library)       */
    int64_t n_pages;     /* PAGED: pages in each pool                                                    */
    const float *k_scale; /* byte formats only: HOST float[L] or NULL (= 1): a stored key byte x means k_scale[l] * x */
    const float *v_scale; /* the same for values                                                                      */
} lethe_cache;
/* cap_tokens = capacity (CONTIG) or capacity * page_tokens (PAGED).  k, v and rel must be 16-byte aligned.
 *
 * Quantised caches.  The paper's related work notes that quantised caches compose with eviction and fixes no
 * format; this library offers two byte formats, each with one positive scale per layer for keys and one for values:
 * LETHE_FP8_E4M3 (1-4-3, bias 7, no infinities, largest value 448) and LETHE_FP8_E5M2 (1-5-2, bias 15, the upper
 * byte of an IEEE half, largest finite value 57344; coarser, but free to expand).  lethe_decode_attend appends
 * k_new / k_scale[l] and v_new / v_scale[l] (fp32 division, round to nearest even, saturating at the largest finite
 * value: no infinity or NaN is ever produced from finite input) and reads a byte x as exactly
 * scale * x; the prune calls move rows as bytes and never look at the storage type.  Supported: head_dim 64 or
 * 128, up to 8 query heads per KV head, contiguous or 16-token pages; lethe_prefill_seed is not (prompt keys are
 * scored before they are quantised). */

/* Create a context on CUDA device `device`.  scratch_bytes_hint (0 = default) sizes the
 * device scratch the calls may use; it grows on demand.  Growth synchronises the device, frees the
 * old buffer and allocates a larger one: a CUDA graph captured from earlier calls may still name the
 * old buffer and must be captured again, and a call that would have to grow scratch while its stream
 * is being captured is refused with LETHE_ERR_UNSUPPORTED (size the scratch with scratch_bytes_hint,
 * or make the same call once before capturing).
 * Returns LETHE_ERR_CUDA if no usable sm_100 device / runtime is present. */
lethe_status lethe_create(lethe_ctx **ctx, int device, size_t scratch_bytes_hint);
void lethe_destroy(lethe_ctx *ctx);

/* HOST string describing the last host-side error of this context (never NULL). */
const char *lethe_last_error(const lethe_ctx *ctx);

/* Synchronise `stream`, then return and clear the device status word: LETHE_OK or the first
 * device-side error since the last poll.  info (HOST, optional, int32[2]) receives
 * {status, flat item index l*B*Hkv + b*Hkv + h of the first offender}. */
lethe_status lethe_poll_status(lethe_ctx *ctx, void *stream, int32_t *info);

/* Tuning knobs (HOST values).
 * variant: 0 = automatic; 1 = CUDA-core kernel; 2..7 = clustered tensor-core (mma) kernel with (warps per
 * CTA, pipeline stages per warp) = (4,3) (8,3) (4,2) (8,2) (4,4) (2,4); 8..15 = persistent tensor-core
 * kernel (one CTA per SM, dynamic item queue, cross-item prefetch) with (8,2) (6,3) (10,2) (8,3) (7,3) (5,4)
 * (6,2) (5,3); 16..21 = the persistent kernel with an asynchronous epilogue (extra warps, four with (8,2) and two otherwise, merge and write
 * item i while the streaming warps already read item i+1) with (8,2) (7,2) (6,3) (5,3) (6,2) (4,4); 24..29 = the same six shapes with
 * the K / V tiles staged by TMA (cp.async.bulk.tensor, 128-byte swizzle) instead of 16-byte cp.async;
 * 32..37 = the clustered kernel's six shapes with the CTAs of an item merged through global scratch (the last
 * CTA to finish completes the item) instead of a thread-block cluster; splits may then be any value 0..16.
 * Tensor-core variants need a bf16 cache (and 16-token pages when paged).
 * A quantised cache runs its own tensor-core kernels: variants 2..7 force the clustered one with
 * shape (4,4) (8,4) (4,2) (4,3) (2,4) (8,2) (splits as above), variants 8..13 the persistent one with shape (8,4)
 * (12,3) (10,4) (8,5) (16,2) (12,2) (e4m3 only); variant 14 the tensor-memory kernel (tcgen05 kind::f8f6f4 MMAs on the
 * cache's bytes with the query and the probabilities split into three e4m3 terms, K / V tiles by TMA, one CTA per SM;
 * head_dim 128, splits 0 or 1, and a capacity whose logits fit on chip: 2 * (heads per KV head) * capacity * 4 bytes
 * beside a 64 KB tile ring; with more than five heads per KV head at least 0.4 of that, the rest overflows to
 * scratch; else LETHE_ERR_UNSUPPORTED).  Automatic (variant 0): for launches of at least two items per
 * SM the tensor-memory kernel where the cache fits it, else (e4m3, head_dim 128) the persistent kernel with shape (8,4);
 * otherwise (launches of few items, e.g. one layer at a time) the layer kernel described below for variants 44..49 in
 * its byte-cache form (4 warps x 4 stages, head_dim 128; variant 44 forces it); for any other value, and for head_dim 64,
 * the clustered kernel with shape (4,4).
 * 44..49 = the clustered kernel's six shapes for launches of one layer at a time (few items per launch): the CTAs of
 * an item merge by one-sided pushes through distributed shared memory (no cluster barriers), and — when variant 51
 * is also set — a launch fetches cached K / V tiles while the previous launch is still finishing.
 * variant 50 / 51 switch that layer pipelining off / on and leave everything else as it is.  It applies to a decode
 * call that follows, through the same context and on the same stream, a decode call on the same cache over other
 * layers (what a model's layer loop issues); such a call reads len, the page table and K / V rows of its own layers
 * before the kernel enqueued just before it on the stream has completed, so between the two calls nothing else
 * may be enqueued on that stream that writes those (any other call of this library in between switches the early
 * fetch off for the next decode call by itself).
 * variant 40..42 select the engine of lethe_prefill_seed and leave everything else as it is: 40 = tcgen05
 * kernels (accumulators in tensor memory, operand tiles by TMA; the default), 41 = mma.sync kernels,
 * 42 = tcgen05 kernels with cp.async tiles; splits is ignored.
 * splits: 0 = automatic, else CTAs per item (1, 2, 4, 8 or 16; they form one thread-block cluster); the
 * persistent variants take 0 or 1.
 * Returns LETHE_ERR_INVALID_ARG for other values.
 * A context serialises its calls: issue them to one stream at a time (the status word and the persistent
 * kernel's work queue are per context). */
lethe_status lethe_set_tuning(lethe_ctx *ctx, int variant, int splits);

/*
 * Failure detection inside the kernels (the paper has no counterpart).  The warp-specialised kernels — the
 * persistent decode kernel with the asynchronous epilogue and the tensor-memory kernels of lethe_prefill_seed —
 * hand work between their warps through mbarriers.  Every such wait is bounded: after `polls` looks at the
 * barrier the waiting thread gives up, the CTA's other roles leave their loops, copies and MMAs still in flight
 * are waited for (with the built-in limit), tensor memory is freed, the work queue is left ready for the next
 * launch, and LETHE_ERR_TIMEOUT is recorded with the CTA (decode) or item (prefill) that gave up.  The launch
 * always returns; the cache contents it was working on are then unspecified.  polls = 0 restores the defaults
 * (hundreds of thousands of polls: seconds, far beyond any legitimate wait); a small value makes the waits run
 * out on purpose, which is how the give-up path is tested without hanging anything (the first poll never
 * blocks, so polls = 1 gives up unless the barrier has already completed).
 */
lethe_status lethe_set_wait_limit(lethe_ctx *ctx, int32_t polls);

/*
 * One decode step for layers [layer_begin, layer_end)  (Sec. 4.1; Eq. 3; Eq. 5).
 * With li = layer - layer_begin and nl = layer_end - layer_begin:
 *   q      [nl][B][Hq][D]   query of the token being generated
 *   k_new  [nl][B][Hkv][D]  its key and value; both NULL = attend without appending
 *   v_new  [nl][B][Hkv][D]
 *   token_pos [B] int32     original position of that token (written to pos[]); may be NULL
 *                           when k_new is NULL
 *   scale  HOST float[L]    softmax scale per layer, indexed by absolute layer (1/sqrt(D),
 *                           or 1/(sqrt(D) T_l) for a layer temperature T_l)
 *   gamma                   decay of Eq. 5, 0 < gamma <= 1
 *   out    [nl][B][Hq][D]   attention output, cache dtype (bf16: round to nearest even)
 *   lse    [nl][B][Hq] fp32 optional (NULL to skip): log-sum-exp of the scaled logits
 * Per item: the new k/v row is written to slot n = len, rel[n] = 0, pos[n] = token_pos[b],
 * len = n + 1; every query head h of the group attends over slots 0..n (the new token
 * included): p_h = softmax_j(scale * q_h . K_j), out_h = sum_j p_hj V_j; then
 * rel[j] = gamma * rel[j] + sum_{h in group} p_hj for every slot j.
 * An item with len == cap_tokens cannot append: it is left untouched, its out rows are
 * zero-filled, and LETHE_ERR_CAPACITY is recorded in the status word.
 * An empty item (no append, len == 0) gives out = 0 and lse = -inf.
 * Calls on the same items must be ordered (same stream or events): the call reads and
 * writes k, v (the appended row), rel, pos and len.
 */
lethe_status lethe_decode_attend(lethe_ctx *ctx, const lethe_cache *cache, int layer_begin, int layer_end,
                                 const void *q, const void *k_new, const void *v_new, const int32_t *token_pos,
                                 const float *scale, float gamma, void *out, float *lse, void *stream);

/*
 * The same step with HOST-resident per-step tensors: q, k_new, v_new, token_pos and
 * out (and lse if not NULL) are HOST pointers.  The results are valid in host memory once
 * `stream` has been synchronised; the input buffers must stay unchanged until then.  The
 * cache stays on the device.  Two paths, chosen per call from the kind of memory:
 *  - page-locked buffers (cudaHostAlloc / cudaHostRegister): the kernel writes out (and
 *    lse) straight into the caller's buffers and, when the inputs are page-locked too,
 *    reads q, k_new, v_new, token_pos from them, so that no copy precedes or follows the
 *    launch (page-locked results with pageable inputs: the inputs are uploaded to
 *    context-owned device staging first);
 *  - pageable buffers: inputs are uploaded to the staging, lethe_decode_attend runs, and
 *    out (and lse) are copied back.  A call that covers many layers is cut into two
 *    chunks of layers whose uploads and downloads run on two context-owned streams under
 *    the kernel of the other chunk (the kernels stay on `stream`, which also waits for the
 *    last download); smaller calls do everything on `stream`.
 */
lethe_status lethe_decode_attend_host(lethe_ctx *ctx, const lethe_cache *cache, int layer_begin, int layer_end,
                                      const void *q_host, const void *k_new_host, const void *v_new_host,
                                      const int32_t *token_pos_host, const float *scale, float gamma, void *out_host,
                                      float *lse_host, void *stream);

/*
 * Layer sparsity estimate (Eq. 1, Sec. 3.1; used per layer in Sec. 4.2).
 * For every item, a = rel[0..n): S_item = (sqrt(n) - |a|_1 / |a|_2) / (sqrt(n) - 1), taken
 * as 0 when n <= 1 or |a|_2 == 0 and clamped to [0, 1];
 * sparsity[l][b] = mean over the Hkv items of (l, b).     sparsity: [L][B] fp32.
 */
lethe_status lethe_estimate_sparsity(lethe_ctx *ctx, const lethe_cache *cache, float *sparsity, void *stream);

/*
 * Per-layer budgets from sparsity (Sec. 4.2: sparse layers are given fewer tokens, dense
 * layers more).  Integer arithmetic after one fp32 subtraction, so results are exact:
 *   w_l = max(1, rint((1 - clamp(S_l, 0, 1)) * 2^20))   (NaN reads as S = 0)
 *   F   = total_budget[b] - L * k_min
 *   k_l = k_min + floor(w_l F / W) + [l among the F - sum floor(..) largest remainders
 *                                      (w_l F) mod W, ties to the lower layer],  W = sum_l w_l
 * so sum_l k_l == total_budget[b] and k_l >= k_min.
 *   sparsity [L][B] fp32; total_budget [B] int64; budgets [L][B] int32 (output); L <= 1024.
 * A sequence with total_budget[b] < L * k_min gets k_l = k_min for all l and records
 * LETHE_ERR_BUDGET in the status word.
 */
lethe_status lethe_alloc_budgets(lethe_ctx *ctx, int n_layers, int batch, const float *sparsity,
                                 const int64_t *total_budget, int32_t k_min, int32_t *budgets, void *stream);

/*
 * RASR retention for every item (Sec. 4.3; Algorithm 1's sink and recent sets), in place.
 * With n = len[item], k = budgets[l][b]:
 *   k >= n: the item is not touched.
 *   else  : keep slots j < min(sink, n), slots j >= n - min(recent, n), and of the
 *           remaining slots those with the largest rel (equal values: lower slot first)
 *           until k slots are kept; if the protected slots alone outnumber k, exactly
 *           they are kept and LETHE_ERR_BUDGET is recorded.  Survivors' rows of k, v, rel
 *           and pos move to slots 0..k-1 in their old order (PAGED: logical slot i lives
 *           in page page_table[i / page_tokens], offset i % page_tokens; pages from index
 *           ceil(len / page_tokens) on are free for the caller to reuse); len = k.
 *   budgets  [L][B] int32
 *   keep_idx optional (NULL to skip) [L][B][Hkv][max_k] int32: the old slot of each
 *            survivor in ascending order, -1 padded; an untouched item lists 0..n-1
 *            (the first max_k of them).
 */
lethe_status lethe_rasr_prune(lethe_ctx *ctx, const lethe_cache *cache, const int32_t *budgets, int32_t recent,
                              int32_t sink, int32_t *keep_idx, int32_t max_k, void *stream);

/*
 * Algorithm 1 (segmented attention-based token shrinking) with the size trigger of Sec. 4.1, for every item,
 * in place — the paper's budget-free retention rule, an alternative to lethe_alloc_budgets + lethe_rasr_prune.
 * With n = len[item] and Le = l_evict[item]:
 *   n <= Le: not triggered, the item is not touched.
 *   else   : order the scores rel[0..n) descending (equal scores: lower slot first); cut points
 *            c_d = floor(n d / n_segments), d = 1 .. n_segments-1; the breakpoint is the first c_d with
 *            top[0] >= tau * top[c_d] (one fp32 multiply; Eq. 4 as printed, v_head / v_cut <= tau with tau > 1,
 *            could only hold at the first cut or never, so it is read the other way round);
 *            found    : slots j < min(sink, n), slots j >= n - recent and the `breakpoint` highest-scoring slots
 *                       survive and are compacted exactly as by lethe_rasr_prune; Le <- max(Le, breakpoint + recent);
 *            not found: nothing is pruned ("conservatively delay pruning"); Le <- min(2 Le, 2^30).
 *   n_segments >= 2; tau >= 1 (the paper's sparse_ratio, 400 by default); l_evict [L][B][Hkv] int32, read and
 *   updated; keep_idx / max_k as in lethe_rasr_prune.
 */
lethe_status lethe_segment_prune(lethe_ctx *ctx, const lethe_cache *cache, int32_t n_segments, float tau,
                                 int32_t recent, int32_t sink, int32_t *l_evict, int32_t *keep_idx, int32_t max_k,
                                 void *stream);

/*
 * Retention with the collapsed score of Eq. 2 as the paper prints it: the attention a token received is summed
 * over ALL heads of the layer (LETHE_COLLAPSE_HEADS) and also over the batch (LETHE_COLLAPSE_HEADS_BATCH), giving
 * one score per token and ONE retention set shared by every item summed over, instead of one per KV head.
 *   group   : the Hkv items of one (layer, sequence), or the B * Hkv items of one layer;
 *   budgets : one int32 per group — [L][B], or [L];
 *   score[j] = sum of rel[item][j] over the group's items in ascending (sequence, KV head) order, in fp32 with
 *              one rounded add per item (the sum decides who is kept, so its precision and order are fixed);
 *   then exactly as lethe_rasr_prune: k >= n keeps everything; otherwise the first `sink` and last `recent`
 *   slots plus the highest scores among the rest (ties to the lower slot) survive, and every item of the group is
 *   compacted in place by that one slot list (each keeps its own K, V, rel, pos rows); len becomes the count.
 * Slot j must be the same token in every item of a group, so all of them must have the same len — true for a
 * cache that was only ever appended to and pruned with this call.  A group that breaks this is left untouched
 * and LETHE_ERR_INVALID_ARG is recorded (with its first item); a budget below the protected count keeps exactly
 * the protected slots and records LETHE_ERR_BUDGET.
 * keep_idx (optional) [groups][max_k] int32: old slots of the survivors, ascending, padded with -1 (all -1 for
 * a refused group).
 */
typedef enum { LETHE_COLLAPSE_HEADS = 0, LETHE_COLLAPSE_HEADS_BATCH = 1 } lethe_collapse;

lethe_status lethe_collapsed_prune(lethe_ctx *ctx, const lethe_cache *cache, const int32_t *budgets, int32_t recent,
                                   int32_t sink, int32_t scope, int32_t *keep_idx, int32_t max_k, void *stream);

/*
 * Relevance of the prompt tokens from the prefill attention (Eq. 2 with Q > 1, folded through Eq. 5), so that
 * decoding does not start from rel = 0.  q_prompt [L][B][P][Hq][D] (bf16) holds the queries of the P = prompt_len
 * prompt tokens; their keys must already be slots 0..P-1 of every item (len >= P, else the item is skipped and
 * LETHE_ERR_CAPACITY recorded).  With causal rows A_h(i, :) = softmax over j <= i of scale_l * q_{i,h} . K_j,
 *   rel[j] = sum_{i=j}^{P-1} gamma^(P-1-i) * sum_{h in group} A_h(i, j)        for j < P
 * which is what P single-token decode steps would have left.  rel[0..P) is overwritten; nothing else changes.
 * scale: HOST float[L].  bf16 caches only; contiguous or paged.
 */
lethe_status lethe_prefill_seed(lethe_ctx *ctx, const lethe_cache *cache, const void *q_prompt, int32_t prompt_len,
                                const float *scale, float gamma, void *stream);

/*
 * lethe_rasr_prune without a context and without any allocation.  (The paper has no counterpart: this entry
 * point exists for the way the library is deployed, not for the method.)
 *
 * Who needs it: callers that must not allocate device memory when a prune round is due — an inference server
 * that handed all device memory to its own pool at start-up (a driver allocation could fail or fragment that
 * pool), or a latency-critical decode loop in which a driver allocation, which may stall the whole device, is
 * not acceptable.  Such callers cannot even create a lethe_ctx, whose creation allocates.
 *
 * Same semantics, arguments and results as lethe_rasr_prune, with these differences:
 *   - it runs on the CURRENT CUDA device, which must be the one that holds the cache;
 *   - its scratch (each item's list of survivors, LETHE_STATIC_PRUNE_MAX_ENTRIES int32 = 16 MiB, plus a
 *     256-byte status block) is a fixed array inside the library image: every GPU that loads the library
 *     carries it until the process exits.  A cache with n_layers * batch * n_kv_heads * cap_tokens above
 *     LETHE_STATIC_PRUNE_MAX_ENTRIES is refused with LETHE_ERR_TOO_LARGE and nothing is enqueued;
 *   - it calls no cudaMalloc / cudaFree and no allocating library routine; it enqueues one 8-byte memset, one
 *     kernel and (with status_out) one 8-byte copy on `stream`;
 *   - the first call on a device looks up the scratch's device address (cudaGetSymbolAddress).  With CUDA's lazy
 *     module loading that first use is also when the runtime places this library's device image, the 16 MiB
 *     array included, on the device: a one-time load that takes device memory from the driver and can fail
 *     (LETHE_ERR_CUDA) if none is left.  So make the first call at start-up — on a small dummy cache if need be —
 *     before the caller's own pool claims the rest of the device, and before any stream capture begins; from the
 *     second call on, a call leaves the device's free memory exactly as it found it;
 *   - all calls share the one array, which still holds whatever the previous call left in it (the status
 *     block is cleared at the start of each call; the lists are always written before they are read).  Two
 *     calls whose kernels could overlap on the GPU — different streams without an ordering event, or several
 *     host threads — race on it: order them;
 *   - status_out: optional DEVICE pointer to int32[2], caller-owned; after the call's work on `stream` it
 *     holds {0, 0} or {LETHE_ERR_BUDGET or LETHE_ERR_PAGE, flat item index} of the first device-side event.
 * Host-detectable errors return LETHE_ERR_INVALID_ARG / LETHE_ERR_UNSUPPORTED / LETHE_ERR_TOO_LARGE /
 * LETHE_ERR_CUDA and enqueue nothing.
 */
#define LETHE_STATIC_PRUNE_MAX_ENTRIES (4 * 1024 * 1024)
lethe_status lethe_rasr_prune_static(const lethe_cache *cache, const int32_t *budgets, int32_t recent, int32_t sink,
                                     int32_t *keep_idx, int32_t max_k, int32_t *status_out, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* LETHE_H */
