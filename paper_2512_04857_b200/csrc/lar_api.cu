// Host side of the C ABI declared in include/lar.h: config validation, slab layout, the call-order
// state machine and the kernel launches.  No torch types, no allocation on the hot path.
#include "../../include/lar.h"

#include <cuda_runtime.h>
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <new>
#include <vector>

#include "common.cuh"
#include "decode_attn.cuh"
#include "decode_stream.cuh"
#include "line_end.cuh"
#include "attend_noalloc.cuh"

namespace {

thread_local int g_last_cuda_error = 0;

#define LAR_CUDA(call)                                   \
    do {                                                 \
        cudaError_t e__ = (call);                        \
        if (e__ != cudaSuccess) {                        \
            g_last_cuda_error = (int)e__;                \
            (void)cudaGetLastError();                    \
            if (getenv("LAR_DEBUG"))                     \
                fprintf(stderr, "lar: line %d: %s -> %s\n", __LINE__, #call, cudaGetErrorString(e__)); \
            return LAR_ERR_CUDA;                         \
        }                                                \
    } while (0)

constexpr int kHostSlots = 4;  // staging slots of the host-buffer entry point (calls in flight)

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct Layout {
    // per-cache
    size_t off_status, off_staging;
    // per-layer strides and the offset of layer 0
    size_t off_state, stride_state;
    size_t off_ptab, stride_ptab;
    size_t off_imap, stride_imap;
    size_t off_guide, stride_guide;
    size_t off_scores, stride_scores;
    size_t off_acc, stride_acc;  // accumulated attention per slot (LAR_FLAG_SCORE_ACCUM only, else empty)
    size_t off_kpool, off_vpool, stride_pool;
    size_t off_partials, off_tickets, tickets_bytes;  // decode scratch (shared by the layers)
    size_t staging_q, staging_k, staging_v, staging_o;  // offsets inside one staging slot
    size_t staging_stride;                               // bytes between consecutive staging slots
    size_t total;
};

struct Derived {
    int units, group, elt, row_bytes, cap, ppu, P, cap_pad, M, mid_pad, compressing, B, N;
    int ctas, max_seg;  // bf16 decode: CTAs of the persistent grid, most segments one unit is cut into
    int unit_ranges;    // bf16 decode: 1 if the CTAs' ranges end on unit boundaries
    int q_slots, p_bufs;  // bf16 decode: depth of a CTA's query ring, number of its partial buffers
    int le_threads;     // threads per CTA of the line-end kernel
    int le_guide_global;  // line-end kernel: the guide rows are read from global memory instead of being staged
};

constexpr int kDefaultDecodeCtas = 148;  // one per SM of a B200

bool derive(const lar_config_t* c, Derived& d) {
    if (!c || c->struct_size != sizeof(lar_config_t)) return false;
    if (c->n_layers < 1 || c->batch < 1 || c->n_q_heads < 1 || c->n_kv_heads < 1) return false;
    if (c->n_q_heads % c->n_kv_heads) return false;
    d.group = c->n_q_heads / c->n_kv_heads;
    if (!(d.group == 1 || d.group == 2 || d.group == 4 || d.group == 8)) return false;
    if (!(c->head_dim == 64 || c->head_dim == 128)) return false;
    if (!(c->dtype == LAR_BF16 || c->dtype == LAR_FP32)) return false;
    if (c->cond_len < 0 || c->line_width < 1 || c->n_lines < 1 || c->anchor_len < 0) return false;
    if (c->recent_lines < 1 || c->budget_lines < 1) return false;
    if (c->page_tokens != 0 && c->page_tokens != 16 && c->page_tokens != 32 && c->page_tokens != 64) return false;
    if (c->dtype == LAR_BF16 && c->page_tokens == 16) return false;  // a 32-row tile of the bf16 decode kernel lies in one page
    if (c->kv_splits != 0 && c->kv_splits != 1 && c->kv_splits != 2 && c->kv_splits != 4 && c->kv_splits != 8) return false;
    if (c->dtype == LAR_BF16) {
        if (c->warps_per_cta < 0 || c->warps_per_cta > 6 || c->stages < 0 || c->stages == 1 || c->stages > 32) return false;
    } else {
        if (c->warps_per_cta < 0 || c->warps_per_cta > 8 || c->stages < 0 || c->stages > 4) return false;
    }
    if (c->decode_ctas < 0 || c->decode_ctas > 1024) return false;
    if (!(c->softmax_scale >= 0.f) || !isfinite(c->softmax_scale)) return false;
    const long long N = (long long)c->line_width * c->n_lines;
    if (N > (1 << 24) || (long long)c->batch * c->n_kv_heads > (1 << 24)) return false;
    d.N = (int)N;
    d.compressing = c->budget_lines < c->n_lines ? 1 : 0;
    d.B = d.compressing ? c->budget_lines * c->line_width : d.N;
    if (c->anchor_len > d.N) return false;
    d.M = 0;
    if (d.compressing) {
        d.M = d.B - c->anchor_len - c->recent_lines * c->line_width;
        if (d.M < c->line_width) return false;  // fewer than n mid candidates: not defined by the method
    }
    d.units = c->batch * c->n_kv_heads;
    d.elt = c->dtype == LAR_BF16 ? 2 : 4;
    d.row_bytes = c->head_dim * d.elt;
    d.cap = c->cond_len + d.B;
    d.P = c->page_tokens ? c->page_tokens : (c->dtype == LAR_BF16 ? 32 : 16);
    d.ppu = (d.cap + d.P - 1) / d.P;
    d.cap_pad = d.ppu * d.P;
    d.mid_pad = (int)align_up((size_t)(d.M > 0 ? d.M : 1), 4);
    // Grid of the persistent bf16 decode kernel.  With fewer units than SMs every unit gets the same whole
    // number of CTAs (none is idle, merges stay k-way).  Whole units per CTA wherever that keeps the busiest
    // CTA within 25 % of the average (nothing to merge across CTAs); equal tile ranges otherwise.
    d.ctas = c->decode_ctas ? c->decode_ctas : kDefaultDecodeCtas;
    // 128-byte rows in many short units: the per-unit work of a CTA (queries in, partials merged, row out) weighs
    // more than its streaming; three small CTAs per SM share it
    if (!c->decode_ctas && c->head_dim == 64 && d.units >= 3 * kDefaultDecodeCtas) d.ctas = 3 * kDefaultDecodeCtas;
    // 256-byte rows: with three or more short units (up to 8 tiles) per SM, two CTAs per SM (two pairs of producers, two
    // epilogue warps) stream faster; long units are better served by one CTA with more consumers
    if (!c->decode_ctas && c->head_dim == 128 && d.units >= 3 * kDefaultDecodeCtas &&
        (d.cap + lar::kStreamTile - 1) / lar::kStreamTile <= 8)
        d.ctas = 2 * kDefaultDecodeCtas;
    if (!c->decode_ctas && d.units < d.ctas) {
        // Merging a unit's partials across CTAs costs a few microseconds of latency per launch, more than a 40 MB stream
        // gains from the extra SMs (measured: 16 units run in 7.8 µs on 16 CTAs, 10.0 µs on 32, 11.8 µs on 48): one CTA
        // per unit, unless there are only a handful of long units; then every unit gets the same number of CTAs of at
        // least 8 tiles each.
        const int t_cap = (d.cap + lar::kStreamTile - 1) / lar::kStreamTile;
        int k = 1;
        if (d.units < 8) {
            k = d.ctas / d.units;
            if (k > t_cap / 8) k = t_cap / 8;
            if (k < 1) k = 1;
        }
        d.ctas = d.units * k;
    }
    {
        const long long per = ((long long)d.units + d.ctas - 1) / d.ctas;
        d.unit_ranges = (d.units >= d.ctas && (long long)d.units * 10 >= per * d.ctas * 8) ? 1 : 0;
        if (c->flags & LAR_FLAG_TILE_RANGES) d.unit_ranges = 0;
    }
    {
        // segments a CTA works on per launch at most: whole units, or (tile ranges) not known in closed form
        const int pe = d.units < d.ctas ? d.units : d.ctas;
        const int segs = d.unit_ranges ? (d.units + pe - 1) / pe : 8;
        d.q_slots = lar::stream_q_slots(d.group, segs);
        d.p_bufs = lar::stream_partial_bufs(segs);
    }
    // A unit of T tiles is cut into at most ceil(T / floor(U T / P)) + 1 segments (never more than T or P).
    // line end: one CTA per unit, 8 warps; few units with a large mid region get one warp per 16 guide rows (16..32 warps)
    d.le_threads = 256;
    // A short line against a small mid region (at most two 16-row blocks of guide rows, 64 mid keys) is a chain of
    // short block-wide phases: smaller CTAs, and so more of them per SM, hide its latencies better (measured per
    // generation: 14.9 -> 11.5 ms on the Janus-Pro-7B shape with 4 warps, 17.2 -> 9.6 ms on the LlamaGen-XL shape with 2)
    // (the written form of Eq. 9 only: the variants that stage the whole live cache have enough work for 8 warps)
    if (c->dtype == LAR_BF16 && c->line_width * d.group <= 32 && d.M <= 64 &&
        !(c->flags & (LAR_FLAG_SCORE_CACHE_NORM | LAR_FLAG_SCORE_ACCUM)))
        d.le_threads = d.row_bytes <= 128 ? 64 : 128;
    d.le_guide_global = 0;
    // (with a column sum per warp over every live row -- accumulated attention, or the cache-normalised form without
    // compaction -- the plan takes warps away again until the CTA fits into shared memory)
    if (d.units <= 2 * kDefaultDecodeCtas && d.M >= 128) {
        const int blocks = (c->line_width * d.group + 15) / 16;
        d.le_threads = 32 * (blocks < 16 ? 16 : blocks > 32 ? 32 : blocks);
    }
    d.max_seg = 1;
    const int t_max = (d.cap + lar::kStreamTile - 1) / lar::kStreamTile;
    if (c->dtype == LAR_BF16 && (long long)d.units * t_max >= (1ll << 30)) return false;  // the kernel's tile indices are 32-bit
    for (int T = 1; T <= t_max; ++T) {
        const long long chunk = (long long)d.units * T / d.ctas;
        long long b = chunk >= 1 ? (T + chunk - 1) / chunk + 1 : T;
        if (b > T) b = T;
        if (b > d.ctas) b = d.ctas;
        if (b > d.max_seg) d.max_seg = (int)b;
    }
    return true;
}

void make_layout(const lar_config_t* c, const Derived& d, Layout& L) {
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    const size_t Lyr = (size_t)c->n_layers, U = (size_t)d.units;
    L.off_status = take(256);
    const size_t qb = (size_t)c->batch * c->n_q_heads * d.row_bytes, kb = (size_t)c->batch * c->n_kv_heads * d.row_bytes;
    L.staging_q = 0;
    L.staging_k = align_up(qb, 256);
    L.staging_v = L.staging_k + align_up(kb, 256);
    L.staging_o = L.staging_v + align_up(kb, 256);
    L.staging_stride = align_up(L.staging_o + qb, 256);
    L.off_staging = take(kHostSlots * L.staging_stride);
    L.stride_state = align_up(U * sizeof(lar::UnitState), 256);
    L.off_state = take(L.stride_state * Lyr);
    L.stride_ptab = align_up(U * d.ppu * 4, 256);
    L.off_ptab = take(L.stride_ptab * Lyr);
    L.stride_imap = align_up(U * d.cap_pad * 4, 256);
    L.off_imap = take(L.stride_imap * Lyr);
    L.stride_guide = align_up(U * c->line_width * d.group * d.row_bytes, 256);
    L.off_guide = take(L.stride_guide * Lyr);
    L.stride_scores = align_up(U * d.mid_pad * 4, 256);
    L.off_scores = take(L.stride_scores * Lyr);
    L.stride_acc = (c->flags & LAR_FLAG_SCORE_ACCUM) ? align_up(U * d.cap_pad * 4, 256) : 0;
    L.off_acc = take(L.stride_acc * Lyr);
    L.stride_pool = align_up(U * d.ppu * d.P * d.row_bytes, 256);
    L.off_kpool = take(L.stride_pool * Lyr);
    L.off_vpool = take(L.stride_pool * Lyr);
    L.off_partials = take(c->dtype == LAR_BF16 ? U * d.max_seg * d.group * (c->head_dim + lar::kPartialPad) * sizeof(float) : 0);
    L.tickets_bytes = U * sizeof(int);  // one ticket per unit
    L.off_tickets = take(L.tickets_bytes);
    L.total = off;
}


// Launch shape of the decode kernel.
// bf16: persistent streaming kernel; per CTA two producer warps, W consumer warps, an epilogue warp and a ring of NS
// 32-row K/V stages.  Measured on B200: two stages per consumer stream as fast as anything deeper; the consumer count
// follows the grid (derive(): one to three CTAs per SM).
// fp32: one cluster of X CTAs per unit, W warps per CTA, NS stages per warp.
void choose_plan(const lar_config_t* c, const Derived& d, lar_plan_t& p) {
    if (c->dtype == LAR_BF16) {
        // (grids of two or three CTAs per SM get three or two consumers each)
        const int per_sm = c->decode_ctas ? 1 : (d.ctas + kDefaultDecodeCtas - 1) / kDefaultDecodeCtas;  // CTAs per SM of the default grids
        // ... and a CTA that holds (part of) one long unit gets a fifth
        const int W = c->warps_per_cta ? c->warps_per_cta : (per_sm >= 3 ? 2 : per_sm == 2 ? 3 : (d.units <= d.ctas && !c->decode_ctas) ? 5 : 4);
        int NS = c->stages ? c->stages : 2 * W;
        // a stage must always be read by the same consumer warp and filled by the same producer warp:
        // ring depth = a multiple of W and of the number of producers
        const int step = W % lar::kProducers == 0 ? W : W * lar::kProducers;
        NS = NS / step * step;
        if (NS < step) NS = step;
        p.kv_splits = 1;
        p.warps_per_cta = W;
        p.stages = NS;
        p.decode_ctas = d.ctas;
        p.max_segments = d.max_seg;
        p.decode_smem_bytes = lar::stream_smem_bytes(c->head_dim, d.group, W, NS, d.q_slots, d.p_bufs);
        return;
    }
    const int tiles = (d.cap + lar::kGranule - 1) / lar::kGranule;  // tiles at the longest live length
    int X = c->kv_splits;
    if (X == 0) {
        X = 1;
        while (X < 8 && d.units * X < 740 && tiles / (X * 2) >= 2) X *= 2;
    }
    int W = c->warps_per_cta;
    if (W == 0) W = 2;
    int NS = c->stages;
    if (NS == 0) {
        const int per_warp = (tiles + X * W - 1) / (X * W);
        NS = per_warp < 2 ? 1 : 2;
    }
    p.kv_splits = X;
    p.warps_per_cta = W;
    p.stages = NS;
    p.decode_ctas = d.units * X;
    p.max_segments = 1;
    p.decode_smem_bytes = lar::decode_smem_bytes(2 * lar::kGranule * d.row_bytes, W, NS, X, d.group, c->head_dim);
}

lar_status_t plan_query_impl(const lar_config_t* cfg, lar_plan_t* out, Derived* dout, Layout* lout) {
    Derived d;
    if (!cfg || !derive(cfg, d)) return LAR_ERR_INVALID_ARG;
    Layout L;
    make_layout(cfg, d, L);
    lar_plan_t p;
    memset(&p, 0, sizeof(p));
    p.capacity = d.cap;
    p.pages_per_unit = d.ppu;
    p.page_tokens = d.P;
    p.mid_len = d.M;
    p.compressing = d.compressing;
    choose_plan(cfg, d, p);
    auto le_bytes = [&]() {
        return lar::line_end_smem_bytes(d.row_bytes, cfg->head_dim, d.M, d.M - cfg->line_width + cfg->recent_lines * cfg->line_width, d.le_threads / 32,
                                        cfg->line_width * d.group, cfg->dtype == LAR_BF16 ? 1 : 0, cfg->cond_len + d.B,
                                        (cfg->flags & (LAR_FLAG_SCORE_CACHE_NORM | LAR_FLAG_SCORE_ACCUM)) ? 1 : 0,
                                        (cfg->flags & LAR_FLAG_SCORE_ACCUM) ? 1 : 0, (cfg->flags & LAR_FLAG_SLOT_REUSE) ? 1 : 0, d.N,
                                        d.le_guide_global);
    };
    p.line_end_smem_bytes = d.compressing ? le_bytes() : 0;
    const bool all_cols = (cfg->flags & LAR_FLAG_SCORE_ACCUM) ||
                          ((cfg->flags & LAR_FLAG_SLOT_REUSE) && (cfg->flags & LAR_FLAG_SCORE_CACHE_NORM));
    while (all_cols && p.line_end_smem_bytes > 227 * 1024 && d.le_threads > 256) {
        d.le_threads -= 32;  // one row of column sums (every live row) less
        p.line_end_smem_bytes = le_bytes();
    }
    if (p.line_end_smem_bytes > 227 * 1024 && cfg->dtype == LAR_BF16 &&
        !(cfg->flags & (LAR_FLAG_SCORE_CACHE_NORM | LAR_FLAG_SCORE_ACCUM))) {
        // a mid region too large to stage next to the guide rows: 8 warps, guide rows read from global memory
        d.le_threads = 256;
        d.le_guide_global = 1;
        p.line_end_smem_bytes = le_bytes();
    }
    p.slab_bytes = L.total;
    p.scratch_bytes = (L.off_tickets + L.tickets_bytes) - L.off_partials;
    if (p.decode_smem_bytes > 227 * 1024 || p.line_end_smem_bytes > 227 * 1024) return LAR_ERR_INVALID_ARG;
    if (out) *out = p;
    if (dout) *dout = d;
    if (lout) *lout = L;
    return LAR_OK;
}

struct LayerShadow {
    bool prefilled = false;
    bool pending_decode = false;
    int v = 0;          // live visual entries
    int n_tok = 0;      // visual tokens appended
    int line_fill = 0;  // tokens of the current line decoded so far
};

}  // namespace

struct lar_cache {
    lar_config_t cfg;
    lar_plan_t plan;
    Derived d;
    Layout L;
    char* slab;
    int device;
    int sm_count;  // SMs of that device
    bool host_checks;
    float scale;
    uint64_t launches;
    int last_layer;  // layer whose cache the most recent library kernel may have written (-1 none)
    int seq;         // launches on this cache since the last reset (the kernels that write a cache are numbered)
    std::vector<int> last_writer;  // per layer: number of the launch that last wrote the layer's cache (0: none)
    lar::TensorMaps tmaps;  // bf16 only
    int rows_per_layer;     // pool rows between consecutive layers
    std::vector<LayerShadow> sh;
    // host-buffer entry point: copies run on streams of the library's own so that the inputs of the next call
    // cross the bus while the kernel of this one runs
    cudaStream_t s_in = nullptr, s_out = nullptr;
    cudaEvent_t e_fork = nullptr, e_in[kHostSlots] = {}, e_k[kHostSlots] = {}, e_out[kHostSlots] = {};
    bool out_pending[kHostSlots] = {};        // copy-out recorded in e_out[slot], not yet waited for by the caller's stream
    uint64_t host_calls = 0;
    bool slot_used[kHostSlots] = {};
    unsigned long long slot_capture[kHostSlots] = {};  // capture the slot's kernel was recorded in (0: none, run eagerly)
    unsigned long long last_host_capture = 0;
    ~lar_cache() {
        if (s_in) cudaStreamDestroy(s_in);
        if (s_out) cudaStreamDestroy(s_out);
        if (e_fork) cudaEventDestroy(e_fork);
        for (int i = 0; i < kHostSlots; ++i) {
            if (e_out[i]) cudaEventDestroy(e_out[i]);
            if (e_in[i]) cudaEventDestroy(e_in[i]);
            if (e_k[i]) cudaEventDestroy(e_k[i]);
        }
    }
};

namespace {

lar::LayerView view_of(const lar_cache* c, int layer) {
    lar::LayerView v;
    const Layout& L = c->L;
    const Derived& d = c->d;
    v.k_pool = c->slab + L.off_kpool + L.stride_pool * layer;
    v.v_pool = c->slab + L.off_vpool + L.stride_pool * layer;
    v.page_table = reinterpret_cast<const int*>(c->slab + L.off_ptab + L.stride_ptab * layer);
    v.index_map = reinterpret_cast<int*>(c->slab + L.off_imap + L.stride_imap * layer);
    v.state = reinterpret_cast<lar::UnitState*>(c->slab + L.off_state + L.stride_state * layer);
    v.guide = c->slab + L.off_guide + L.stride_guide * layer;
    v.scores = reinterpret_cast<float*>(c->slab + L.off_scores + L.stride_scores * layer);
    v.acc = L.stride_acc ? reinterpret_cast<float*>(c->slab + L.off_acc + L.stride_acc * layer) : nullptr;
    v.status = reinterpret_cast<unsigned*>(c->slab + L.off_status);
    v.pages_per_unit = d.ppu;
    v.page_tokens = d.P;
    v.cap = d.cap;
    v.cap_pad = d.cap_pad;
    v.mid_pad = d.mid_pad;
    v.cond_len = c->cfg.cond_len;
    v.line_width = c->cfg.line_width;
    v.budget_tokens = d.B;
    v.anchor_len = c->cfg.anchor_len;
    v.recent_lines = c->cfg.recent_lines;
    v.compressing = d.compressing;
    v.n_kv_heads = c->cfg.n_kv_heads;
    v.group = d.group;
    v.identity_pages = (c->cfg.flags & LAR_FLAG_SHUFFLE_PAGES) ? 0 : 1;
    return v;
}

// ---- tensor maps (bf16 decode path) -----------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

lar_status_t make_tensor_maps(lar_cache* c) {
    void* fp = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t ce = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fp, cudaEnableDefault, &qres);
    if (ce != cudaSuccess || !fp || qres != cudaDriverEntryPointSuccess) {
        g_last_cuda_error = (int)(ce != cudaSuccess ? ce : cudaErrorUnknown);
        (void)cudaGetLastError();
        return LAR_ERR_CUDA;
    }
    EncodeTiledFn encode = reinterpret_cast<EncodeTiledFn>(fp);
    c->rows_per_layer = (int)(c->L.stride_pool / (size_t)c->d.row_bytes);
    // {head_dim, pool rows of all layers, {K pool, V pool}}
    const cuuint64_t gdim[3] = {(cuuint64_t)c->cfg.head_dim, (cuuint64_t)c->rows_per_layer * (cuuint64_t)c->cfg.n_layers, 2};
    const cuuint64_t gstride[2] = {(cuuint64_t)c->d.row_bytes, (cuuint64_t)(c->L.off_vpool - c->L.off_kpool)};
    const cuuint32_t estr[3] = {1, 1, 1};
    for (int h = 0; h < 8; ++h) {
        const cuuint32_t box[3] = {64, (cuuint32_t)(4 * (h + 1)), 2};
        CUresult r = encode(&c->tmaps.kv[h], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, c->slab + c->L.off_kpool, gdim, gstride, box,
                            estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) {
            g_last_cuda_error = (int)cudaErrorInvalidValue;
            return LAR_ERR_CUDA;
        }
    }
    return LAR_OK;
}

// ---- kernel tables ------------------------------------------------------------------------------
using DecodeStreamFn = void (*)(const lar::StreamArgs, const lar::TensorMaps);
template <int D, bool VIEWS>
DecodeStreamFn decode_stream_for_group(int G) {
    switch (G) {
        case 1: return lar::decode_stream_kernel<D, 1, VIEWS>;
        case 2: return lar::decode_stream_kernel<D, 2, VIEWS>;
        case 4: return lar::decode_stream_kernel<D, 4, VIEWS>;
        case 8: return lar::decode_stream_kernel<D, 8, VIEWS>;
    }
    return nullptr;
}
// views: q / k / v / out with sequence strides and / or the rotary embedding fused in
DecodeStreamFn decode_stream_fn(const lar_config_t& c, int G, bool views = false) {
    if (views) return c.head_dim == 64 ? decode_stream_for_group<64, true>(G) : decode_stream_for_group<128, true>(G);
    return c.head_dim == 64 ? decode_stream_for_group<64, false>(G) : decode_stream_for_group<128, false>(G);
}
using DecodeFn = void (*)(const lar::DecodeArgs);
using LineEndFn = void (*)(const lar::LayerView, const lar::LayerStrides, float, int);

template <typename T, int D>
DecodeFn decode_for_group(int G) {
    switch (G) {
        case 1: return lar::decode_kernel<T, D, 1>;
        case 2: return lar::decode_kernel<T, D, 2>;
        case 4: return lar::decode_kernel<T, D, 4>;
        case 8: return lar::decode_kernel<T, D, 8>;
    }
    return nullptr;
}
DecodeFn decode_fn(const lar_config_t& c, int G) {
    return c.head_dim == 64 ? decode_for_group<float, 64>(G) : decode_for_group<float, 128>(G);
}
template <typename T, int D>
LineEndFn line_end_for_group(int G) {
    switch (G) {
        case 1: return lar::line_end_kernel<T, D, 1>;
        case 2: return lar::line_end_kernel<T, D, 2>;
        case 4: return lar::line_end_kernel<T, D, 4>;
        case 8: return lar::line_end_kernel<T, D, 8>;
    }
    return nullptr;
}
LineEndFn line_end_fn(const lar_config_t& c, int G) {
    if (c.dtype == LAR_BF16) return c.head_dim == 64 ? line_end_for_group<__nv_bfloat16, 64>(G) : line_end_for_group<__nv_bfloat16, 128>(G);
    return c.head_dim == 64 ? line_end_for_group<float, 64>(G) : line_end_for_group<float, 128>(G);
}

lar_status_t launch_append(lar_cache* c, int layer, const void* k, const void* v, int n_tokens, int is_prefix,
                           cudaStream_t s) {
    const lar::LayerView lv = view_of(c, layer);
    const int U = c->d.units;
    if (c->cfg.dtype == LAR_BF16) {
        if (c->cfg.head_dim == 64)
            lar::append_kernel<__nv_bfloat16, 64><<<U, 128, 0, s>>>(lv, (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, n_tokens, is_prefix);
        else
            lar::append_kernel<__nv_bfloat16, 128><<<U, 128, 0, s>>>(lv, (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, n_tokens, is_prefix);
    } else {
        if (c->cfg.head_dim == 64)
            lar::append_kernel<float, 64><<<U, 128, 0, s>>>(lv, (const float*)k, (const float*)v, n_tokens, is_prefix);
        else
            lar::append_kernel<float, 128><<<U, 128, 0, s>>>(lv, (const float*)k, (const float*)v, n_tokens, is_prefix);
    }
    LAR_CUDA(cudaGetLastError());
    c->launches++;
    c->last_layer = layer;
    c->last_writer[layer] = ++c->seq;
    return LAR_OK;
}

// Elements between consecutive sequences of q, k, v and out (0 = dense).
struct SeqStrides {
    long long q = 0, k = 0, v = 0, out = 0;
    const float* rope = nullptr;  // rotary embedding applied to q and k by the kernel (nullptr: none)
    int rope_mode = 0;
};

lar_status_t launch_decode(lar_cache* c, int layer, const void* q, const void* k, const void* v, void* out, int fused,
                           cudaStream_t s, const SeqStrides& ss = SeqStrides()) {
    const bool pdl = (c->cfg.flags & LAR_FLAG_PDL) != 0;
    // With programmatic dependent launch a CTA moves in as soon as an SM is free, a few microseconds before the
    // preceding kernel is done.  It requests its first ring of cached K/V tiles then, so that arithmetic starts when
    // the dependency resolves.
    int prefetch = 0;
    if (c->cfg.dtype == LAR_BF16)
        prefetch = pdl ? 1 : 0;
    else if (pdl && c->last_layer != layer && c->last_layer >= 0)
        prefetch = 1;
    const float scale_log2 = c->scale * 1.4426950408889634f;

    cudaLaunchConfig_t lc;
    memset(&lc, 0, sizeof(lc));
    lc.dynamicSmemBytes = (size_t)c->plan.decode_smem_bytes;
    lc.stream = s;
    cudaLaunchAttribute attrs[2];
    unsigned na = 0;
    if (pdl) {
        attrs[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attrs[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
    }
    if (c->cfg.dtype == LAR_BF16) {
        // bulk copies of q / k / v rows need 16-byte aligned sources
        if ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(out) | reinterpret_cast<uintptr_t>(k) |
             reinterpret_cast<uintptr_t>(v)) & 15u)
            return LAR_ERR_INVALID_ARG;
        lar::StreamArgs a;
        a.lv = view_of(c, layer);
        a.q = q;
        a.k_new = k;
        a.v_new = v;
        a.out = out;
        a.partials = reinterpret_cast<float*>(c->slab + c->L.off_partials);
        a.tickets = reinterpret_cast<int*>(c->slab + c->L.off_tickets);
        {
            // live rows before this step's append, from the host-side counters (they follow the device's by
            // construction: every call that changes the length updates both)
            const LayerShadow& sh = c->sh[layer];
            const int live = (sh.prefilled ? c->cfg.cond_len : 0) + sh.v;
            a.len = live < c->d.cap ? live : c->d.cap;
            a.n_tok = sh.n_tok;
        }
        a.unit_ranges = c->d.unit_ranges;
        {
            // the launch's tile list: T tiles per unit; the CTAs' ranges are whole units or tiles
            const int T = a.len > 0 ? (a.len + lar::kStreamTile - 1) / lar::kStreamTile : 1;
            const long long items = c->d.unit_ranges ? (long long)c->d.units : (long long)c->d.units * T;
            const int pe = (int)(items < c->d.ctas ? items : c->d.ctas);
            a.tiles_per_unit = T;
            a.tiles_magic = (unsigned)((1ull << 32) / (unsigned)T + 1ull);
            a.range_ctas = pe;
            a.range_q = (int)(items / pe);
            a.range_r = (int)(items % pe);
            int sh = 0;
            while ((1 << sh) < c->d.P) ++sh;
            a.page_shift = sh;
        }
        a.scale_log2 = scale_log2;
        a.fused = fused;
        a.prefetch = prefetch;
        a.n_units = c->d.units;
        a.n_stages = c->plan.stages;
        a.max_seg = c->d.max_seg;
        a.seq = ++c->seq;
        a.need_seq = c->last_writer[layer];
        if (prefetch) {
            // How far back can a launch of this cache still be in flight?  A decode kernel lets its successor start at once
            // and leaves only after its predecessor has completed, so every launch in flight but the oldest holds all its
            // CTAs: with `slots` CTAs of this size resident on the GPU at most, the oldest is (slots - 1) / ctas + 1 back.
            const long long per_sm = 233472 / ((long long)c->plan.decode_smem_bytes + 1024);
            const long long slots = (long long)c->sm_count * (per_sm < 1 ? 1 : per_sm > 32 ? 32 : per_sm);
            const long long depth = (slots - 1) / c->d.ctas + 1;
            if ((long long)a.seq - a.need_seq > depth + 1) a.prefetch = 2;  // (one launch of margin)
        }
        c->last_writer[layer] = a.seq;
        a.done_seq = reinterpret_cast<int*>(c->slab + c->L.off_status + 128);
        a.q_slots = c->d.q_slots;
        a.stall_test = (c->cfg.flags & LAR_FLAG_TEST_STALL) ? 1 : 0;
        a.p_bufs = c->d.p_bufs;
        a.pool_row_base = layer * c->rows_per_layer;
        a.q_seq_stride = ss.q;
        a.k_seq_stride = ss.k;
        a.v_seq_stride = ss.v;
        a.out_seq_stride = ss.out;
        a.rope = ss.rope;
        a.rope_mode = ss.rope_mode;
        lc.gridDim = dim3((unsigned)c->d.ctas, 1, 1);
        lc.blockDim = dim3((unsigned)(32 * (c->plan.warps_per_cta + lar::kProducers + 1)), 1, 1);
        lc.attrs = attrs;
        lc.numAttrs = na;
        DecodeStreamFn fn = decode_stream_fn(c->cfg, c->d.group, ss.rope_mode != 0 || ss.q || ss.k || ss.v || ss.out);
        LAR_CUDA(cudaLaunchKernelEx(&lc, fn, a, c->tmaps));
    } else {
        if (ss.q || ss.k || ss.v || ss.out || ss.rope) return LAR_ERR_INVALID_ARG;  // fp32 storage: dense tensors only
        lar::DecodeArgs a;
        a.lv = view_of(c, layer);
        a.q = q;
        a.k_new = k;
        a.v_new = v;
        a.out = out;
        a.scale_log2 = scale_log2;
        a.fused = fused;
        a.prefetch = prefetch;
        a.splits = c->plan.kv_splits;
        a.stages = c->plan.stages;
        lc.gridDim = dim3((unsigned)(c->d.units * c->plan.kv_splits), 1, 1);
        lc.blockDim = dim3((unsigned)(32 * c->plan.warps_per_cta), 1, 1);
        if (c->plan.kv_splits > 1) {
            attrs[na].id = cudaLaunchAttributeClusterDimension;
            attrs[na].val.clusterDim.x = (unsigned)c->plan.kv_splits;
            attrs[na].val.clusterDim.y = 1;
            attrs[na].val.clusterDim.z = 1;
            ++na;
        }
        lc.attrs = attrs;
        lc.numAttrs = na;
        DecodeFn fn = decode_fn(c->cfg, c->d.group);
        LAR_CUDA(cudaLaunchKernelEx(&lc, fn, a));
    }
    c->launches++;
    c->last_layer = layer;
    return LAR_OK;
}

bool bad_layer(const lar_cache* c, int layer) { return !c || layer < 0 || layer >= c->cfg.n_layers; }

// host-side protocol: visual append
lar_status_t check_visual_append(lar_cache* c, LayerShadow& sh) {
    if (!c->host_checks) return LAR_OK;
    if (!sh.prefilled && c->cfg.cond_len > 0) return LAR_ERR_BAD_STATE;
    if (sh.pending_decode) return LAR_ERR_BAD_STATE;
    if (sh.n_tok >= c->d.N) return LAR_ERR_CAPACITY;
    if (sh.line_fill >= c->cfg.line_width) return LAR_ERR_CAPACITY;  // line complete: the line-end call is due
    if (sh.v >= c->d.B) return LAR_ERR_CAPACITY;
    return LAR_OK;
}

}  // namespace

extern "C" {

const char* lar_status_str(lar_status_t s) {
    switch (s) {
        case LAR_OK: return "ok";
        case LAR_ERR_INVALID_ARG: return "invalid argument";
        case LAR_ERR_BAD_STATE: return "call order violates the decode protocol";
        case LAR_ERR_CAPACITY: return "capacity exceeded";
        case LAR_ERR_CUDA: return "CUDA runtime error";
        case LAR_ERR_NOMEM: return "out of memory / slab too small";
        case LAR_ERR_DEVICE_CHECK: return "device-side check failed";
    }
    return "unknown status";
}

int lar_last_cuda_error(void) { return g_last_cuda_error; }

lar_status_t lar_plan_query(const lar_config_t* cfg, lar_plan_t* plan_out) {
    return plan_query_impl(cfg, plan_out, nullptr, nullptr);
}

size_t lar_cache_slab_bytes(const lar_config_t* cfg) {
    lar_plan_t p;
    if (plan_query_impl(cfg, &p, nullptr, nullptr) != LAR_OK) return 0;
    return (size_t)p.slab_bytes;
}

lar_status_t lar_cache_create(const lar_config_t* cfg, void* dev_slab, size_t slab_bytes, lar_cache_t** out) {
    if (!out) return LAR_ERR_INVALID_ARG;
    *out = nullptr;
    lar_plan_t plan;
    Derived d;
    Layout L;
    lar_status_t st = plan_query_impl(cfg, &plan, &d, &L);
    if (st != LAR_OK) return st;
    if (!dev_slab || (reinterpret_cast<uintptr_t>(dev_slab) & 255u)) return LAR_ERR_INVALID_ARG;
    if (slab_bytes < L.total) return LAR_ERR_NOMEM;

    lar_cache* c = new (std::nothrow) lar_cache();
    if (!c) return LAR_ERR_NOMEM;
    c->cfg = *cfg;
    c->plan = plan;
    c->d = d;
    c->L = L;
    c->slab = static_cast<char*>(dev_slab);
    c->host_checks = (cfg->flags & LAR_FLAG_NO_HOST_CHECKS) == 0;
    c->scale = cfg->softmax_scale > 0.f ? cfg->softmax_scale : 1.0f / sqrtf((float)cfg->head_dim);
    c->launches = 0;
    c->last_layer = -1;
    c->sh.assign((size_t)cfg->n_layers, LayerShadow());
    c->seq = 0;
    c->last_writer.assign((size_t)cfg->n_layers, 0);

    auto fail = [&](lar_status_t e) { delete c; return e; };
    cudaError_t ce = cudaGetDevice(&c->device);
    if (ce == cudaSuccess) ce = cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, c->device);
    if (ce != cudaSuccess) { g_last_cuda_error = (int)ce; return fail(LAR_ERR_CUDA); }

    // page tables: unit u owns pages_per_unit pages of its layer's pool (identity, or shuffled)
    const size_t per_layer = (size_t)d.units * d.ppu;
    std::vector<int> tab(per_layer);
    for (int layer = 0; layer < cfg->n_layers; ++layer) {
        for (size_t i = 0; i < per_layer; ++i) tab[i] = (int)i;
        if (cfg->flags & LAR_FLAG_SHUFFLE_PAGES) {
            uint64_t x = 0x9E3779B97F4A7C15ull * (cfg->page_seed + 1u) + (uint64_t)layer * 0xD1B54A32D192ED03ull;
            for (size_t i = per_layer; i > 1; --i) {
                x ^= x >> 12; x ^= x << 25; x ^= x >> 27;
                const size_t j = (size_t)((x * 0x2545F4914F6CDD1Dull) >> 33) % i;
                const int t = tab[i - 1]; tab[i - 1] = tab[j]; tab[j] = t;
            }
        }
        ce = cudaMemcpy(c->slab + L.off_ptab + L.stride_ptab * layer, tab.data(), per_layer * sizeof(int), cudaMemcpyHostToDevice);
        if (ce != cudaSuccess) { g_last_cuda_error = (int)ce; (void)cudaGetLastError(); return fail(LAR_ERR_CUDA); }
    }
    ce = cudaMemset(c->slab + L.off_status, 0, 256);
    if (ce == cudaSuccess) ce = cudaMemset(c->slab + L.off_state, 0, L.stride_state * cfg->n_layers);
    if (ce == cudaSuccess) ce = cudaMemset(c->slab + L.off_imap, 0xff, L.stride_imap * cfg->n_layers);
    if (ce == cudaSuccess) ce = cudaMemset(c->slab + L.off_scores, 0, L.stride_scores * cfg->n_layers);
    if (ce == cudaSuccess && L.stride_acc) ce = cudaMemset(c->slab + L.off_acc, 0, L.stride_acc * cfg->n_layers);
    if (ce == cudaSuccess) ce = cudaMemset(c->slab + L.off_guide, 0, L.stride_guide * cfg->n_layers);
    // rows of a page beyond the live length are read by short tiles with weight 0: they must be finite
    if (ce == cudaSuccess) ce = cudaMemset(c->slab + L.off_kpool, 0, L.stride_pool * cfg->n_layers);
    if (ce == cudaSuccess) ce = cudaMemset(c->slab + L.off_vpool, 0, L.stride_pool * cfg->n_layers);
    if (ce == cudaSuccess) ce = cudaMemset(c->slab + L.off_tickets, 0, L.tickets_bytes);
    if (ce == cudaSuccess)
        ce = cudaFuncSetAttribute(cfg->dtype == LAR_BF16 ? (const void*)decode_stream_fn(*cfg, d.group) : (const void*)decode_fn(*cfg, d.group),
                                  cudaFuncAttributeMaxDynamicSharedMemorySize, plan.decode_smem_bytes);
    if (ce == cudaSuccess && cfg->dtype == LAR_BF16)  // (the variant for views of larger tensors / the rotary embedding)
        ce = cudaFuncSetAttribute((const void*)decode_stream_fn(*cfg, d.group, true), cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  plan.decode_smem_bytes);
    if (ce == cudaSuccess && d.compressing)
        ce = cudaFuncSetAttribute((const void*)line_end_fn(*cfg, d.group), cudaFuncAttributeMaxDynamicSharedMemorySize, plan.line_end_smem_bytes);
    if (ce == cudaSuccess) ce = cudaStreamCreateWithFlags(&c->s_in, cudaStreamNonBlocking);
    if (ce == cudaSuccess) ce = cudaStreamCreateWithFlags(&c->s_out, cudaStreamNonBlocking);
    if (ce == cudaSuccess) ce = cudaEventCreateWithFlags(&c->e_fork, cudaEventDisableTiming);
    for (int i = 0; i < kHostSlots && ce == cudaSuccess; ++i) {
        ce = cudaEventCreateWithFlags(&c->e_out[i], cudaEventDisableTiming);
        if (ce != cudaSuccess) break;
        ce = cudaEventCreateWithFlags(&c->e_in[i], cudaEventDisableTiming);
        if (ce == cudaSuccess) ce = cudaEventCreateWithFlags(&c->e_k[i], cudaEventDisableTiming);
    }
    if (ce == cudaSuccess) ce = cudaDeviceSynchronize();
    if (ce != cudaSuccess) { g_last_cuda_error = (int)ce; (void)cudaGetLastError(); return fail(LAR_ERR_CUDA); }
    if (cfg->dtype == LAR_BF16) {
        lar_status_t ts = make_tensor_maps(c);
        if (ts != LAR_OK) return fail(ts);
    }
    *out = c;
    return LAR_OK;
}

lar_status_t lar_cache_destroy(lar_cache_t* c) {
    if (!c) return LAR_ERR_INVALID_ARG;
    delete c;
    return LAR_OK;
}

lar_status_t lar_cache_reset(lar_cache_t* c, void* stream) {
    if (!c) return LAR_ERR_INVALID_ARG;
    LAR_CUDA(cudaMemsetAsync(c->slab + c->L.off_state, 0, c->L.stride_state * c->cfg.n_layers, (cudaStream_t)stream));
    LAR_CUDA(cudaMemsetAsync(c->slab + c->L.off_tickets, 0, c->L.tickets_bytes, (cudaStream_t)stream));
    if (c->L.stride_acc)  // accumulated attention restarts with the image
        LAR_CUDA(cudaMemsetAsync(c->slab + c->L.off_acc, 0, c->L.stride_acc * c->cfg.n_layers, (cudaStream_t)stream));
    LAR_CUDA(cudaMemsetAsync(c->slab + c->L.off_status + 128, 0, sizeof(int), (cudaStream_t)stream));
    for (auto& s : c->sh) s = LayerShadow();
    c->last_layer = -1;
    c->seq = 0;
    c->last_writer.assign(c->last_writer.size(), 0);
    // host-buffer entry point: whatever was in flight is ordered before the reset on `stream` by the caller; forget it
    for (int i = 0; i < kHostSlots; ++i) {
        c->out_pending[i] = false;
        c->slot_used[i] = false;
        c->slot_capture[i] = 0;
    }
    c->last_host_capture = 0;
    return LAR_OK;
}

lar_status_t lar_cache_set_host_checks(lar_cache_t* c, int enabled) {
    if (!c) return LAR_ERR_INVALID_ARG;
    c->host_checks = enabled != 0;
    return LAR_OK;
}

uint64_t lar_cache_launch_count(const lar_cache_t* c) { return c ? c->launches : 0; }

lar_status_t lar_cache_get_plan(const lar_cache_t* c, lar_plan_t* plan_out) {
    if (!c || !plan_out) return LAR_ERR_INVALID_ARG;
    *plan_out = c->plan;
    return LAR_OK;
}

lar_status_t lar_append_kv(lar_cache_t* c, int layer, const void* k, const void* v, int n_tokens, void* stream) {
    if (bad_layer(c, layer) || !k || !v || n_tokens < 1) return LAR_ERR_INVALID_ARG;
    LayerShadow& sh = c->sh[layer];
    const bool is_prefix = !sh.prefilled && c->cfg.cond_len > 0;
    if (is_prefix) {
        if (c->host_checks && n_tokens != c->cfg.cond_len) return LAR_ERR_INVALID_ARG;
    } else {
        if (n_tokens != 1) return LAR_ERR_INVALID_ARG;
        lar_status_t st = check_visual_append(c, sh);
        if (st != LAR_OK) return st;
    }
    lar_status_t st = launch_append(c, layer, k, v, n_tokens, is_prefix ? 1 : 0, (cudaStream_t)stream);
    if (st != LAR_OK) return st;
    if (is_prefix) {
        sh.prefilled = true;
    } else {
        sh.pending_decode = true;
        sh.v += 1;
        sh.n_tok += 1;
    }
    return LAR_OK;
}

lar_status_t lar_decode_attn(lar_cache_t* c, int layer, const void* q, void* out, void* stream) {
    if (bad_layer(c, layer) || !q || !out) return LAR_ERR_INVALID_ARG;
    LayerShadow& sh = c->sh[layer];
    if (c->host_checks && !sh.pending_decode) return LAR_ERR_BAD_STATE;
    lar_status_t st = launch_decode(c, layer, q, nullptr, nullptr, out, 0, (cudaStream_t)stream);
    if (st != LAR_OK) return st;
    sh.pending_decode = false;
    sh.line_fill += 1;
    return LAR_OK;
}

lar_status_t lar_decode_step(lar_cache_t* c, int layer, const void* q, const void* k, const void* v, void* out,
                             void* stream) {
    if (bad_layer(c, layer) || !q || !k || !v || !out) return LAR_ERR_INVALID_ARG;
    LayerShadow& sh = c->sh[layer];
    lar_status_t st = check_visual_append(c, sh);
    if (st != LAR_OK) return st;
    st = launch_decode(c, layer, q, k, v, out, 1, (cudaStream_t)stream);
    if (st != LAR_OK) return st;
    sh.v += 1;
    sh.n_tok += 1;
    sh.line_fill += 1;
    return LAR_OK;
}

static lar_status_t decode_step_views(lar_cache_t* c, int layer, const void* q, const void* k, const void* v, void* out,
                                      int64_t q_seq_stride, int64_t k_seq_stride, int64_t v_seq_stride, int64_t out_seq_stride,
                                      const float* rope, int rope_mode, void* stream);

lar_status_t lar_decode_step_strided(lar_cache_t* c, int layer, const void* q, const void* k, const void* v, void* out,
                                     int64_t q_seq_stride, int64_t k_seq_stride, int64_t v_seq_stride, int64_t out_seq_stride,
                                     void* stream) {
    return decode_step_views(c, layer, q, k, v, out, q_seq_stride, k_seq_stride, v_seq_stride, out_seq_stride, nullptr, 0, stream);
}

lar_status_t lar_decode_step_rope(lar_cache_t* c, int layer, const void* q, const void* k, const void* v, void* out,
                                  int64_t q_seq_stride, int64_t k_seq_stride, int64_t v_seq_stride, int64_t out_seq_stride,
                                  const float* cos_sin, int interleaved, void* stream) {
    if (!cos_sin || (reinterpret_cast<uintptr_t>(cos_sin) & 3u)) return LAR_ERR_INVALID_ARG;
    return decode_step_views(c, layer, q, k, v, out, q_seq_stride, k_seq_stride, v_seq_stride, out_seq_stride, cos_sin,
                             interleaved ? 2 : 1, stream);
}

static lar_status_t decode_step_views(lar_cache_t* c, int layer, const void* q, const void* k, const void* v, void* out,
                                      int64_t q_seq_stride, int64_t k_seq_stride, int64_t v_seq_stride, int64_t out_seq_stride,
                                      const float* rope, int rope_mode, void* stream) {
    if (bad_layer(c, layer) || !q || !k || !v || !out) return LAR_ERR_INVALID_ARG;
    if (c->cfg.dtype != LAR_BF16) return LAR_ERR_INVALID_ARG;
    const int64_t d = c->cfg.head_dim, hq = c->cfg.n_q_heads, hkv = c->cfg.n_kv_heads;
    // a sequence's heads must fit between two sequences; bulk copies need 16-byte (8-element) aligned rows
    if (q_seq_stride < hq * d || out_seq_stride < hq * d || k_seq_stride < hkv * d || v_seq_stride < hkv * d) return LAR_ERR_INVALID_ARG;
    if ((q_seq_stride | k_seq_stride | v_seq_stride | out_seq_stride) & 7) return LAR_ERR_INVALID_ARG;
    LayerShadow& sh = c->sh[layer];
    lar_status_t st = check_visual_append(c, sh);
    if (st != LAR_OK) return st;
    SeqStrides ss;
    // (a stride that equals the dense one is passed as 0: the kernel then needs no division per unit)
    ss.q = q_seq_stride == hq * d ? 0 : q_seq_stride;
    ss.k = k_seq_stride == hkv * d ? 0 : k_seq_stride;
    ss.v = v_seq_stride == hkv * d ? 0 : v_seq_stride;
    ss.out = out_seq_stride == hq * d ? 0 : out_seq_stride;
    ss.rope = rope;
    ss.rope_mode = rope_mode;
    st = launch_decode(c, layer, q, k, v, out, 1, (cudaStream_t)stream, ss);
    if (st != LAR_OK) return st;
    sh.v += 1;
    sh.n_tok += 1;
    sh.line_fill += 1;
    return LAR_OK;
}

// Host buffers in, host buffer out.  Three streams: the caller's (kernel), s_in (host -> device), s_out (device ->
// host).  kHostSlots staging slots take turns, so the copy-in of call t + 1 overlaps the kernel and the copy-out of call t; the
// caller's stream waits for the copy-out before the call returns its place in the stream, which keeps every effect of
// the call ordered in that stream.  Works the same under stream capture: the side streams join the capture through
// events and have re-joined the caller's stream when the call returns, so a capture may end after any call.
lar_status_t lar_decode_step_host(lar_cache_t* c, int layer, const void* q_host, const void* k_host, const void* v_host,
                                  void* out_host, void* stream) {
    if (bad_layer(c, layer) || !q_host || !out_host || (!k_host) != (!v_host)) return LAR_ERR_INVALID_ARG;
    {
        const lar_status_t pre = check_visual_append(c, c->sh[layer]);  // before anything is enqueued
        if (pre != LAR_OK) return pre;
    }
    cudaStream_t s = (cudaStream_t)stream;
    const size_t qb = (size_t)c->cfg.batch * c->cfg.n_q_heads * c->d.row_bytes;
    const size_t kb = (size_t)c->cfg.batch * c->cfg.n_kv_heads * c->d.row_bytes;
    const bool packed = !k_host;  // q | k | v back to back at q_host (one host allocation: one copy can span them)
    if (packed) {
        k_host = static_cast<const char*>(q_host) + qb;
        v_host = static_cast<const char*>(q_host) + qb + kb;
    }
    const int slot = (int)(c->host_calls % kHostSlots);
    char* stg = c->slab + c->L.off_staging + c->L.staging_stride * slot;

    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone, cap_in = cudaStreamCaptureStatusNone;
    unsigned long long cap_id = 0, cap_in_id = 0;
    LAR_CUDA(cudaStreamGetCaptureInfo(s, &cap, &cap_id));
    LAR_CUDA(cudaStreamGetCaptureInfo(c->s_in, &cap_in, &cap_in_id));
    const bool capturing = cap == cudaStreamCaptureStatusActive;
    if (!capturing) cap_id = 0;
    for (int i = 0; i < kHostSlots; ++i)  // deferred copy-outs never cross a capture boundary: lar_cache_host_join comes first
        if (c->out_pending[i] && c->slot_capture[i] != cap_id) return LAR_ERR_BAD_STATE;
    // When must s_in be ordered behind everything already in the caller's stream?  Under capture, if it is not part of
    // the capture yet; eagerly, if the previous call was captured (its graph runs in the caller's stream).  Otherwise
    // s_in only waits for the kernel that last read this staging slot.
    const bool join = capturing ? cap_in != cudaStreamCaptureStatusActive : c->last_host_capture != 0;
    if (join) {
        LAR_CUDA(cudaEventRecord(c->e_fork, s));
        LAR_CUDA(cudaStreamWaitEvent(c->s_in, c->e_fork, 0));
    } else if (c->slot_used[slot] && c->slot_capture[slot] == cap_id) {
        LAR_CUDA(cudaStreamWaitEvent(c->s_in, c->e_k[slot], 0));
    }
    // (a slot last used in an earlier capture or eagerly, seen from a new capture: that work precedes the graph in the
    // caller's stream whenever the graph runs, and join is true for the capture's first call anyway)

    if (packed && c->L.staging_k == qb && c->L.staging_v == qb + kb) {
        LAR_CUDA(cudaMemcpyAsync(stg + c->L.staging_q, q_host, qb + 2 * kb, cudaMemcpyHostToDevice, c->s_in));  // q | k | v in one piece
    } else {
        LAR_CUDA(cudaMemcpyAsync(stg + c->L.staging_q, q_host, qb, cudaMemcpyHostToDevice, c->s_in));
        LAR_CUDA(cudaMemcpyAsync(stg + c->L.staging_k, k_host, kb, cudaMemcpyHostToDevice, c->s_in));
        LAR_CUDA(cudaMemcpyAsync(stg + c->L.staging_v, v_host, kb, cudaMemcpyHostToDevice, c->s_in));
    }
    LAR_CUDA(cudaEventRecord(c->e_in[slot], c->s_in));
    LAR_CUDA(cudaStreamWaitEvent(s, c->e_in[slot], 0));
    if (c->out_pending[slot]) {  // deferred copy-out of kHostSlots calls ago: it reads the output slot this kernel writes
        LAR_CUDA(cudaStreamWaitEvent(s, c->e_out[slot], 0));
        c->out_pending[slot] = false;
    }

    const int saved = c->last_layer;
    c->last_layer = layer;  // a copy precedes the kernel: never prefetch ahead of it
    lar_status_t st = lar_decode_step(c, layer, stg + c->L.staging_q, stg + c->L.staging_k, stg + c->L.staging_v,
                                      stg + c->L.staging_o, stream);
    if (st != LAR_OK) { c->last_layer = saved; return st; }   // s_in has re-joined the caller's stream above
    LAR_CUDA(cudaEventRecord(c->e_k[slot], s));
    c->slot_used[slot] = true;
    c->slot_capture[slot] = cap_id;
    c->last_host_capture = cap_id;
    c->host_calls++;

    LAR_CUDA(cudaStreamWaitEvent(c->s_out, c->e_k[slot], 0));
    LAR_CUDA(cudaMemcpyAsync(out_host, stg + c->L.staging_o, qb, cudaMemcpyDeviceToHost, c->s_out));
    LAR_CUDA(cudaEventRecord(c->e_out[slot], c->s_out));
    if (c->cfg.flags & LAR_FLAG_HOST_DEFER_OUT)
        c->out_pending[slot] = true;
    else
        LAR_CUDA(cudaStreamWaitEvent(s, c->e_out[slot], 0));
    return LAR_OK;
}

lar_status_t lar_cache_host_join(lar_cache_t* c, void* stream) {
    if (!c) return LAR_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    unsigned long long cap_id = 0;
    LAR_CUDA(cudaStreamGetCaptureInfo(s, &cap, &cap_id));
    if (cap != cudaStreamCaptureStatusActive) cap_id = 0;
    for (int slot = 0; slot < kHostSlots; ++slot) {
        if (!c->out_pending[slot]) continue;
        if (c->slot_capture[slot] != cap_id) return LAR_ERR_BAD_STATE;  // recorded in another capture (or eagerly)
        LAR_CUDA(cudaStreamWaitEvent(s, c->e_out[slot], 0));
        c->out_pending[slot] = false;
    }
    return LAR_OK;
}

// scoring mode of the line-end kernel: bit 0 softmax over the whole live cache, bit 1 accumulated attention
static int line_end_mode(const lar_cache* c) {
    return ((c->cfg.flags & LAR_FLAG_SCORE_CACHE_NORM) ? 1 : 0) | ((c->cfg.flags & LAR_FLAG_SCORE_ACCUM) ? 2 : 0) |
           ((c->cfg.flags & LAR_FLAG_SLOT_REUSE) ? 4 : 0) | (c->d.le_guide_global ? 8 : 0);
}

static lar::LayerStrides layer_strides(const lar_cache* c) {
    lar::LayerStrides ls;
    ls.pool = c->L.stride_pool;
    ls.page_table = c->L.stride_ptab;
    ls.index_map = c->L.stride_imap;
    ls.state = c->L.stride_state;
    ls.guide = c->L.stride_guide;
    ls.scores = c->L.stride_scores;
    ls.acc = c->L.stride_acc;
    return ls;
}

lar_status_t lar_line_end_score_evict(lar_cache_t* c, int layer, void* stream) {
    if (bad_layer(c, layer)) return LAR_ERR_INVALID_ARG;
    LayerShadow& sh = c->sh[layer];
    if (c->host_checks) {
        if (sh.pending_decode || sh.line_fill != c->cfg.line_width) return LAR_ERR_BAD_STATE;
    }
    if (c->d.compressing) {
        const lar::LayerView lv = view_of(c, layer);
        LineEndFn fn = line_end_fn(c->cfg, c->d.group);
        fn<<<dim3((unsigned)c->d.units, 1, 1), c->d.le_threads, c->plan.line_end_smem_bytes, (cudaStream_t)stream>>>(
            lv, layer_strides(c), c->scale * 1.4426950408889634f, line_end_mode(c));
        LAR_CUDA(cudaGetLastError());
        c->launches++;
        c->last_layer = -2;  // rows of the cache were just moved: the next decode launch must not fetch ahead
        c->last_writer[layer] = ++c->seq;
        if (sh.v >= c->d.B) sh.v -= c->cfg.line_width;
    }
    sh.line_fill = 0;
    return LAR_OK;
}

lar_status_t lar_line_end_score_evict_all(lar_cache_t* c, void* stream) {
    if (!c) return LAR_ERR_INVALID_ARG;
    if (c->host_checks)
        for (const LayerShadow& sh : c->sh)
            if (sh.pending_decode || sh.line_fill != c->cfg.line_width) return LAR_ERR_BAD_STATE;
    if (c->d.compressing) {
        const lar::LayerView lv = view_of(c, 0);
        LineEndFn fn = line_end_fn(c->cfg, c->d.group);
        fn<<<dim3((unsigned)c->d.units, (unsigned)c->cfg.n_layers, 1), c->d.le_threads, c->plan.line_end_smem_bytes,
             (cudaStream_t)stream>>>(lv, layer_strides(c), c->scale * 1.4426950408889634f,
                                     line_end_mode(c));
        LAR_CUDA(cudaGetLastError());
        c->launches++;
        c->last_layer = -2;  // every layer's cache was just written: the next decode launch must not fetch ahead
        c->last_writer.assign(c->last_writer.size(), ++c->seq);
        for (LayerShadow& sh : c->sh)
            if (sh.v >= c->d.B) sh.v -= c->cfg.line_width;
    }
    for (LayerShadow& sh : c->sh) sh.line_fill = 0;
    return LAR_OK;
}

lar_status_t lar_cache_get_state(lar_cache_t* c, int layer, int32_t* lens, int32_t* index_map, float* scores,
                                 void* stream) {
    if (bad_layer(c, layer)) return LAR_ERR_INVALID_ARG;
    LAR_CUDA(cudaStreamSynchronize((cudaStream_t)stream));
    const int U = c->d.units;
    std::vector<lar::UnitState> st((size_t)U);
    LAR_CUDA(cudaMemcpy(st.data(), c->slab + c->L.off_state + c->L.stride_state * layer, (size_t)U * sizeof(lar::UnitState),
                        cudaMemcpyDeviceToHost));
    if (lens)
        for (int u = 0; u < U; ++u) lens[u] = st[u].len;
    if (index_map) {
        std::vector<int> raw((size_t)U * c->d.cap_pad);
        LAR_CUDA(cudaMemcpy(raw.data(), c->slab + c->L.off_imap + c->L.stride_imap * layer, raw.size() * sizeof(int),
                            cudaMemcpyDeviceToHost));
        for (int u = 0; u < U; ++u)
            for (int s = 0; s < c->d.cap; ++s)
                index_map[(size_t)u * c->d.cap + s] = s < st[u].len ? raw[(size_t)u * c->d.cap_pad + s] : -1;
    }
    if (scores && c->d.M > 0) {
        std::vector<float> raw((size_t)U * c->d.mid_pad);
        LAR_CUDA(cudaMemcpy(raw.data(), c->slab + c->L.off_scores + c->L.stride_scores * layer, raw.size() * sizeof(float),
                            cudaMemcpyDeviceToHost));
        for (int u = 0; u < U; ++u)
            memcpy(scores + (size_t)u * c->d.M, raw.data() + (size_t)u * c->d.mid_pad, (size_t)c->d.M * sizeof(float));
    }
    return LAR_OK;
}

lar_status_t lar_cache_poll_device_status(lar_cache_t* c, uint32_t* bits_out, void* stream) {
    if (!c) return LAR_ERR_INVALID_ARG;
    LAR_CUDA(cudaStreamSynchronize((cudaStream_t)stream));
    unsigned bits = 0;
    LAR_CUDA(cudaMemcpy(&bits, c->slab + c->L.off_status, sizeof(bits), cudaMemcpyDeviceToHost));
    if (bits) LAR_CUDA(cudaMemset(c->slab + c->L.off_status, 0, sizeof(bits)));
    if (bits_out) *bits_out = bits;
    return bits ? LAR_ERR_DEVICE_CHECK : LAR_OK;
}

lar_status_t lar_attend_dense_noalloc(const void* q, const void* k, const void* v, void* out, int n_units, int group,
                                      int head_dim, int len, float softmax_scale, void* stream) {
    if (!q || !k || !v || !out || n_units < 1 || len < 1) return LAR_ERR_INVALID_ARG;
    if (group < 1 || group > 8 || !(head_dim == 64 || head_dim == 128)) return LAR_ERR_INVALID_ARG;
    if (!(softmax_scale >= 0.f) || !isfinite(softmax_scale)) return LAR_ERR_INVALID_ARG;
    if (n_units > lar::kStaticMaxUnits) return LAR_ERR_CAPACITY;  // one ticket per unit in the static array
    unsigned char* scratch = nullptr;
    LAR_CUDA(lar::static_scratch_address(&scratch));
    const int splits = lar::static_scratch_splits(n_units, len);
    const float scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)head_dim);
    cudaStream_t s = (cudaStream_t)stream;
    // the array keeps what the last call left: the tickets of this call must start at zero
    LAR_CUDA(cudaMemsetAsync(scratch, 0, (size_t)n_units * sizeof(int), s));
    const dim3 grid((unsigned)(n_units * splits));
    if (head_dim == 64)
        lar::attend_dense_kernel<64><<<grid, 128, 0, s>>>((const __nv_bfloat16*)q, (const __nv_bfloat16*)k, (const __nv_bfloat16*)v,
                                                          (__nv_bfloat16*)out, scratch, group, len, splits, scale * 1.4426950408889634f);
    else
        lar::attend_dense_kernel<128><<<grid, 128, 0, s>>>((const __nv_bfloat16*)q, (const __nv_bfloat16*)k, (const __nv_bfloat16*)v,
                                                           (__nv_bfloat16*)out, scratch, group, len, splits, scale * 1.4426950408889634f);
    LAR_CUDA(cudaGetLastError());
    return LAR_OK;
}

}  // extern "C"
