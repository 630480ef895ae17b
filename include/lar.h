/*
 * lar.h — C ABI of the LineAR hot path on one B200 (sm_100a).
 *
 * The library manages, per transformer layer, a per-head KV cache that is bounded to a few raster
 * lines (paper Sec. 3.3) and computes the per-token decode attention over it (Sec. 3.1, Eq. 2).
 * Every (layer, sequence, KV head) is an independent unit: its live cache is
 *     [ C conditional tokens | N_init anchor tokens | retained mid tokens | r most recent lines ]
 * and never holds more than C + B entries, B = budget_lines * line_width.
 *
 * General conventions
 *   - All entry points return a lar_status_t; nothing throws or aborts.
 *   - "device" pointers are CUDA device addresses on the device that was current at
 *     lar_cache_create; "host" pointers are ordinary (preferably pinned) host addresses.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Hot-path
 *     calls only enqueue work on it: no host synchronisation, no allocation.
 *   - The caller owns every buffer it passes, including the slab; the library owns only host-side
 *     bookkeeping.  Buffers must stay valid until the enqueued work has run.
 *   - Sequences decode in lock-step (one visual token per call for the whole batch), as in the
 *     paper's batched runs; lengths are nevertheless stored per unit in device memory.
 *   - Tensor layouts are dense, row-major, innermost dimension head_dim:
 *       q, out : [batch, n_q_heads, head_dim]            k, v : [batch, n_kv_heads, n_tokens, head_dim]
 *     Query head hq uses KV head hq / (n_q_heads / n_kv_heads).
 *   - Element type is bf16 or fp32 (config); logits, softmax and accumulation are fp32.
 */
#ifndef LAR_H_
#define LAR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct lar_cache lar_cache_t; /* opaque host object; device state lives in the caller's slab */

typedef enum {
    LAR_OK = 0,
    LAR_ERR_INVALID_ARG = 1,  /* null pointer, bad size, unsupported shape */
    LAR_ERR_BAD_STATE = 2,    /* call order violates the decode protocol (see each call) */
    LAR_ERR_CAPACITY = 3,     /* append beyond the n-token line buffer / beyond N tokens */
    LAR_ERR_CUDA = 4,         /* a CUDA runtime call failed; lar_last_cuda_error() has its code */
    LAR_ERR_NOMEM = 5,        /* slab too small / host allocation failed */
    LAR_ERR_DEVICE_CHECK = 6  /* a kernel recorded a failed bounds / wait-limit check */
} lar_status_t;

typedef enum { LAR_BF16 = 0, LAR_FP32 = 1 } lar_dtype_t;

/* config.flags */
#define LAR_FLAG_NO_HOST_CHECKS 0x1u /* skip the host-side call-order checks.  Needed when calls are captured
                                        into CUDA graphs: the host-side counters advance at capture, not at
                                        replay.  The live length of a step is a closed form of the step index
                                        and is passed to the decode kernel by the host, so a graph holds the
                                        lengths of the steps it was captured at: capture the calls of a
                                        generation in order and replay the graphs in that same order (the
                                        kernels check the length against device memory and record bit 16
                                        otherwise).  Device-side checks stay active. */
#define LAR_FLAG_PDL 0x2u            /* launch decode kernels with programmatic dependent launch: a decode kernel lets
                                        its successors be scheduled at once, and a successor may fetch cached K/V of
                                        its own layer before the preceding kernels on the stream have finished.  The
                                        library guards this itself: launches on a cache are numbered, a device word
                                        records up to which number they have completed, and a kernel fetches ahead
                                        only if the launch that last wrote its layer's cache is covered.  Contract
                                        for the caller: a kernel of its own that uses programmatic dependent launch
                                        on the same stream waits on its dependency before it completes, and nothing
                                        but this library writes the slab. */
#define LAR_FLAG_SHUFFLE_PAGES 0x4u  /* test hook: assign physical pages in a pseudo-random order */
#define LAR_FLAG_TILE_RANGES 0x8u    /* bf16 decode: always deal 32-row tiles (not whole units) to the CTAs, even
                                        where whole units would balance well enough */
#define LAR_FLAG_SCORE_CACHE_NORM 0x10u /* variant of Eq. 9 (Sec. 3.3): the softmax of every guide query runs over
                                        all entries that were live when its token was decoded (conditional,
                                        anchor, mid, recent and the line's own tokens up to itself) instead of
                                        over the mid keys only; the score of a mid token is then the attention
                                        probability Eq. 2-3 gave it, averaged over the n steps of the line and
                                        the G heads.  The line-end kernel stages C + B keys in shared memory:
                                        configurations where they do not fit are rejected at creation. */

#define LAR_FLAG_SCORE_ACCUM 0x40u   /* scoring of the paper's ablation "w. AttAcc" (Sec. 4.4, Table 6; the accumulated-attention
                                        rule of the H2O-style baselines of Sec. 4.2): a cached token's score is the attention
                                        probability Eq. 2-3 gave it, summed over every decode step since it was appended and
                                        over the G heads, divided by n G.  Every line end (also below budget) adds the line's
                                        sums -- the cache-normalised form of Eq. 9 over all live entries -- to one float per
                                        slot in the slab; a compressing line end ranks the mid entries by that sum, and an
                                        entry keeps its sum when the compaction moves it.  Needs the C + B live keys in shared
                                        memory, as LAR_FLAG_SCORE_CACHE_NORM does (which it implies). */

#define LAR_FLAG_SLOT_REUSE 0x80u    /* the line end does not compact (Eq. 5-7 define the kept SET; Eq. 2 does not depend on
                                        the order of the cache): the n evicted slots take the n rows of the newest line, so
                                        n rows of K and V move instead of every row behind the first hole, and the cache
                                        stays dense for the decode kernel.  Slots then no longer follow original positions
                                        (the index map is not monotone); the line end finds the mid region of Sec. 3.3
                                        through the index map.  Kept sets, outputs and scores are unchanged. */

#define LAR_FLAG_TEST_STALL 0x100u    /* test hook for the bounded waits of the bf16 decode kernel: its producer warps request no
                                        K/V tile, so every consumer warp's wait for its first tile runs into the limit
                                        (~1 s of SM clocks); the CTA's roles then give up, the launch ends by itself after
                                        1-3 s, outputs are undefined and status bit 4 (wait limit) is recorded.  The
                                        device and the slab stay usable.  No counterpart in the paper. */

#define LAR_FLAG_HOST_DEFER_OUT 0x20u /* lar_decode_step_host does not make `stream` wait for its copy-out: the
                                        copy-out of a call then overlaps the kernels of the next calls as well.
                                        `out_host` of a call is complete only after lar_cache_host_join (or four
                                        further lar_decode_step_host calls) on the same stream.  Call
                                        lar_cache_host_join before a stream capture ends and before switching
                                        between captured and uncaptured calls (else LAR_ERR_BAD_STATE). */

typedef struct lar_config {
    uint32_t struct_size;  /* = sizeof(lar_config_t) */
    int32_t n_layers;      /* L */
    int32_t batch;         /* S: sequences, after classifier-free-guidance doubling */
    int32_t n_q_heads;     /* Hq */
    int32_t n_kv_heads;    /* Hkv, divides Hq; Hq/Hkv in {1,2,4,8} */
    int32_t head_dim;      /* d: 64 or 128 */
    int32_t dtype;         /* lar_dtype_t */
    int32_t cond_len;      /* C: conditional prefix (Sec. 3.1 prefill); always kept, not counted in B */
    int32_t line_width;    /* n: tokens per raster line, including a line-end token if the model has one */
    int32_t n_lines;       /* h: N = h * n visual tokens per image (Sec. 3.3, 2D view) */
    int32_t anchor_len;    /* N_init: the first N_init visual tokens are never evicted (Sec. 3.3) */
    int32_t recent_lines;  /* r >= 1: the last r lines are never evicted (Sec. 3.3) */
    int32_t budget_lines;  /* B / n (Sec. 3.3 "Cache Budget"); >= n_lines selects the full-cache path */
    float softmax_scale;   /* 0 selects 1/sqrt(head_dim) (Eq. 2) */
    int32_t page_tokens;   /* tokens per physical page: fp32 16, 32 or 64 (0 selects 16); bf16 32 or 64 (0 selects 32) */
    uint32_t flags;        /* LAR_FLAG_* */
    int32_t kv_splits;     /* fp32 only: CTAs (one thread-block cluster) per unit in decode: 0 auto, else 1,2,4,8 */
    int32_t warps_per_cta; /* decode warps: bf16 consumer warps per CTA, 0 auto, else 1..6;
                              fp32 warps per CTA, 0 auto, else 1..8 */
    int32_t stages;        /* K/V stages: bf16 depth of the CTA's ring of 32-row tiles, 0 auto, else 2..32 (rounded
                              down to a common multiple of the consumer warps and the two producer warps);
                              fp32 16-row stages in flight per warp, 0 auto, else 1..4 */
    uint32_t page_seed;    /* seed of LAR_FLAG_SHUFFLE_PAGES */
    int32_t decode_ctas;   /* bf16 only: CTAs of the persistent decode grid: 0 lets the library choose (one to three per
                              SM of a B200, or a multiple of the unit count when there are fewer units than SMs), else 1..1024 */
} lar_config_t;

/* What lar_cache_create derived from a config (introspection; also usable without a GPU). */
typedef struct lar_plan {
    int32_t capacity;       /* slots per unit: C + min(B, N) */
    int32_t pages_per_unit;
    int32_t page_tokens;
    int32_t mid_len;        /* M = B - N_init - r n at a compressing line end; 0 on the full-cache path */
    int32_t kv_splits, warps_per_cta, stages;
    int32_t decode_smem_bytes;
    int32_t line_end_smem_bytes;
    int32_t compressing;    /* 1 if budget_lines < n_lines */
    uint64_t slab_bytes;
    int32_t decode_ctas;    /* CTAs per decode launch */
    int32_t max_segments;   /* bf16: most CTAs one unit's rows are spread over (scratch partials per unit) */
    uint64_t scratch_bytes; /* part of the slab used as decode scratch (partials, tickets) */
} lar_plan_t;

/* Validate a config and report the derived plan.  No CUDA call is made.
 * Rejects (LAR_ERR_INVALID_ARG): Hq % Hkv != 0, group not in {1,2,4,8}, d not in {64,128}, r < 1,
 * negative sizes, and compressing budgets with fewer than n mid candidates
 * (B < N_init + (r+1) n) — the paper does not define the method there. */
lar_status_t lar_plan_query(const lar_config_t* cfg, lar_plan_t* plan_out);

/* Bytes of device memory the caller must provide for a cache of this config (0 if invalid).
 * The slab holds the paged K/V pools of all layers, page tables, per-unit lengths, the slot ->
 * original-position index maps, the guide queues (Eq. 8), the last score vectors (Eq. 9) and the
 * decode scratch (partial results of units whose rows are spread over several CTAs).
 * The scratch is shared by all layers: calls on one cache must be ordered on one stream. */
size_t lar_cache_slab_bytes(const lar_config_t* cfg);

/* Create a cache over a caller-allocated device slab (256-byte aligned, >= lar_cache_slab_bytes).
 * Writes page tables and zeroes the state on the legacy default stream and synchronises once.
 * *out is owned by the caller until lar_cache_destroy. */
lar_status_t lar_cache_create(const lar_config_t* cfg, void* dev_slab, size_t slab_bytes, lar_cache_t** out);

/* Forget all cached tokens of every layer (start of a new image).  Asynchronous on `stream`. */
lar_status_t lar_cache_reset(lar_cache_t* c, void* stream);

/* Cache append (Eq. 4).  k, v: device, [batch, n_kv_heads, n_tokens, head_dim].
 * The first call on a layer after create/reset is the prefill (Sec. 3.1): n_tokens must equal C
 * (skip it if C = 0).  Every later call appends one visual token (n_tokens = 1) and must be
 * followed by lar_decode_attn of that layer before the next append.
 * LAR_ERR_CAPACITY: the line's n-token buffer is full (a line-end call is due) or N tokens exist. */
lar_status_t lar_append_kv(lar_cache_t* c, int layer, const void* k, const void* v, int n_tokens, void* stream);

/* Decode attention (Eq. 2-3) of the token appended last: out = softmax(q K^T scale) V over every live
 * entry of the unit (prefix + retained visual tokens + the new token), per query head.
 * q, out: device, [batch, n_q_heads, head_dim], 16-byte aligned.  Also stores q in the layer's guide
 * queue (Eq. 8).
 * LAR_ERR_BAD_STATE unless a visual token was appended to this layer since its last decode. */
lar_status_t lar_decode_attn(lar_cache_t* c, int layer, const void* q, void* out, void* stream);

/* lar_append_kv(n_tokens = 1) + lar_decode_attn fused into one kernel launch (Eq. 4 then Eq. 2).
 * k, v: device, [batch, n_kv_heads, head_dim], 16-byte aligned. */
lar_status_t lar_decode_step(lar_cache_t* c, int layer, const void* q, const void* k, const void* v,
                             void* out, void* stream);

/* lar_decode_step on views of larger tensors (bf16 storage only): consecutive sequences of q, k, v, out lie
 * *_seq_stride ELEMENTS apart, the heads of one sequence back to back -- e.g. q, k and v as column ranges of the
 * [batch, (n_q_heads + 2 n_kv_heads) * head_dim] output of a fused QKV projection (the three strides are then that row
 * length), and out as a view of the buffer the output projection reads.  The cache therefore takes the keys exactly as
 * the caller hands them over: a model with rotary position embedding passes post-rotation k and q, so that the guide
 * queries of Eq. 8 and the cached keys of Eq. 9 live in the same space (Sec. 3.3).
 * Every stride is a multiple of 8 elements (16 bytes) and at least the dense row of its tensor, every pointer 16-byte
 * aligned; otherwise LAR_ERR_INVALID_ARG (also for fp32 caches).  Call order and errors as lar_decode_step. */
lar_status_t lar_decode_step_strided(lar_cache_t* c, int layer, const void* q, const void* k, const void* v, void* out,
                                     int64_t q_seq_stride, int64_t k_seq_stride, int64_t v_seq_stride,
                                     int64_t out_seq_stride, void* stream);

/* lar_decode_step_strided with the rotary position embedding of q and k fused in (bf16 storage only): the kernel rotates
 * the G query rows of every unit and the new key row before anything else uses them, so the cache receives rotated keys
 * and the guide queue rotated queries -- the space in which Eq. 8-9 compare them (Sec. 3.3) -- without a separate pass
 * over q and k.  cos_sin: device, fp32, [batch, head_dim]: for each sequence the cosines of the head_dim / 2 rotation
 * angles of this step's position, then the sines.  interleaved = 0 rotates the pairs (i, i + head_dim / 2), interleaved
 * != 0 the pairs (2 i, 2 i + 1):
 *     x' = x cos_i - y sin_i,  y' = y cos_i + x sin_i     (fp32, every product and sum rounded, result rounded to bf16)
 * v is not rotated.  Strides, alignment, call order and errors as lar_decode_step_strided (pass the dense row lengths
 * for dense tensors). */
lar_status_t lar_decode_step_rope(lar_cache_t* c, int layer, const void* q, const void* k, const void* v, void* out,
                                  int64_t q_seq_stride, int64_t k_seq_stride, int64_t v_seq_stride, int64_t out_seq_stride,
                                  const float* cos_sin, int interleaved, void* stream);

/* lar_decode_step with HOST buffers (pinned memory): copies q, k, v to a staging area of the slab, runs the
 * fused kernel and copies `out` back, asynchronously.  Seen from `stream` the call is one stream-ordered
 * operation: `out_host` is complete once work enqueued on `stream` after the call runs (or `stream` is
 * synchronised).  Inside, the copies run on two streams the cache owns and four staging slots take turns, so the
 * copy-in of a call overlaps the kernel and copy-out of the call before it; the host buffers must stay
 * untouched until then.  The call may be captured into a CUDA graph (the side streams join the capture and
 * have re-joined `stream` when the call returns).
 * k_host and v_host may both be NULL: q_host then holds q, k and v back to back in ONE host allocation (the
 * layout a fused QKV projection leaves) and they cross the bus in one copy.  Adjacent but separately
 * allocated buffers must be passed as three pointers. */
lar_status_t lar_decode_step_host(lar_cache_t* c, int layer, const void* q_host, const void* k_host,
                                  const void* v_host, void* out_host, void* stream);

/* Makes `stream` wait for every copy-out that lar_decode_step_host deferred (LAR_FLAG_HOST_DEFER_OUT); a no-op
 * otherwise.  No counterpart in the paper (host plumbing). */
lar_status_t lar_cache_host_join(lar_cache_t* c, void* stream);

/* Line-boundary step (Sec. 3.3, Eq. 5-10).  Legal only when the layer has just completed a line
 * (visual count multiple of n, every token decoded), else LAR_ERR_BAD_STATE.
 * While fewer than B visual tokens are cached (or on the full-cache path) it only restarts the guide
 * queue.  Otherwise, per unit: scores the M mid tokens with the line's n*G guide queries
 * (softmax over the mid keys, mean over queries and heads), evicts the n lowest (ties: the higher
 * position goes first), and compacts K, V and the index map in place to
 * [prefix | anchor | kept mid | recent], leaving an n-token buffer for the next line. */
lar_status_t lar_line_end_score_evict(lar_cache_t* c, int layer, void* stream);

/* lar_line_end_score_evict for every layer of the cache in ONE kernel launch (the line end is a synchronisation
 * point of the whole model, Sec. 3.3; layers are independent, so their units share a grid).  Legal only when every
 * layer has just completed the line, else LAR_ERR_BAD_STATE and nothing is launched. */
lar_status_t lar_line_end_score_evict_all(lar_cache_t* c, void* stream);

/* Destroy the host object.  The slab is the caller's and is not touched. */
lar_status_t lar_cache_destroy(lar_cache_t* c);

/* Introspection for tests: synchronises `stream`, then copies to HOST buffers (each may be NULL)
 *   lens       [batch * n_kv_heads]              live entries per unit
 *   index_map  [batch * n_kv_heads, capacity]    original position of each slot (prefix j -> j,
 *                                                visual token i (1-based) -> C + i - 1); -1 beyond len
 *   scores     [batch * n_kv_heads, mid_len]     Eq. 9 scores of the last compressing line end */
lar_status_t lar_cache_get_state(lar_cache_t* c, int layer, int32_t* lens, int32_t* index_map, float* scores,
                                 void* stream);

/* Synchronises `stream` and returns LAR_ERR_DEVICE_CHECK if any kernel recorded a failed check since
 * the last poll (bits in *bits_out, may be NULL: 1 capacity, 2 line-end off boundary, 4 wait limit,
 * 8 decode on an empty cache, 16 the length the host passed to a decode kernel differs from
 * the device's, e.g. a captured graph replayed out of order, 32 a line end met a score that is not finite -- a NaN
 * or Inf in a key or query; such entries rank lowest, exactly n are still evicted); clears the word. */
lar_status_t lar_cache_poll_device_status(lar_cache_t* c, uint32_t* bits_out, void* stream);

/* Enable (1) / disable (0) the host-side call-order checks at run time (see LAR_FLAG_NO_HOST_CHECKS). */
lar_status_t lar_cache_set_host_checks(lar_cache_t* c, int enabled);

/* Number of kernels this cache has launched so far (bookkeeping for benchmarks). */
uint64_t lar_cache_launch_count(const lar_cache_t* c);

/* The plan a cache was created with. */
lar_status_t lar_cache_get_plan(const lar_cache_t* c, lar_plan_t* plan_out);

/* Decode attention over dense K/V without any scratch buffer from the caller (the paper has no counterpart of this
 * call; it exists for callers that cannot allocate).  The other entry points keep their split-KV partials in the
 * caller's slab.  A caller that only owns its q / K / V / out tensors and may not call cudaMalloc at this point --
 * code running inside a framework's memory-pool "no allocation" region, a serving loop that has already handed all
 * free memory to its KV-cache manager, a plug-in that was given pointers and nothing else -- has no slab to offer.
 * For them the partials live in a file-scope device array of the library: 8 MiB on every GPU that loads the
 * library, held until the process exits.
 *
 *   out[u][g] = softmax(q[u][g] K[u]^T scale) V[u]      (Eq. 2 per unit u and query head g of its group)
 *   q, out : device, bf16, [n_units, group, head_dim]      k, v : device, bf16, [n_units, len, head_dim], dense
 *   group 1..8, head_dim 64 or 128, len >= 1, softmax_scale 0 selects 1/sqrt(head_dim).
 *
 * Limits: n_units <= 16384 (one ticket per unit), otherwise LAR_ERR_CAPACITY and nothing is launched.  A unit's keys
 * are cut into at most 8 ranges (one CTA each) while n_units * ranges <= 296; the partials of such a launch take at
 * most 1.3 MB of the array.  With more than 148 units every unit is one range and only the tickets are touched.
 * The call enqueues one memset (the tickets of the units it uses must start at zero; the array keeps whatever the
 * previous call left) and one kernel on `stream`, and calls no allocating routine.  The first call on a device looks
 * the array's device address up (cudaGetSymbolAddress, with that device current): make that first call outside any
 * stream capture.  All calls on a device share the one array: two calls whose kernels may overlap on the GPU
 * (different streams, no dependency) race on it -- order them. */
lar_status_t lar_attend_dense_noalloc(const void* q, const void* k, const void* v, void* out, int n_units, int group,
                                      int head_dim, int len, float softmax_scale, void* stream);

const char* lar_status_str(lar_status_t s);
int lar_last_cuda_error(void); /* cudaError_t of the last failed runtime call in this thread, 0 if none */

#ifdef __cplusplus
}
#endif
#endif /* LAR_H_ */
