// bf16 decode attention (Eq. 2-3) as one persistent, warp-specialised streaming kernel per layer-step,
// fused with the append of the step's token (Eq. 4) and the guide-queue push (Eq. 8).
//
// Work decomposition.  The live rows of every unit = (sequence, KV head) are cut into 32-row tiles;
// all tiles of the layer form one list (unit-major) that is dealt out in contiguous ranges to the CTAs
// of the grid (one to three CTAs per SM).  Where whole units can be dealt out evenly enough the ranges end on unit
// boundaries; otherwise they are equal in tiles, so that every SM streams the same number of bytes
// whatever the number of units.  The part of a unit that falls into one CTA is a *segment*.  A unit
// that lies inside one CTA is finished there; a unit cut by a range boundary leaves one partial
// (m, l, o) per segment in a global scratch area and the CTA that delivers the last partial (an atomic
// ticket, no waiting) merges them.
// The live length is the same for every unit (sequences decode in lock-step) and is a closed form of
// the step index; the host passes it, so that all CTAs agree on the tile list, and the CTA that closes a
// unit checks it against the unit's length in device memory before advancing that.
//
// Inside a CTA three roles run concurrently, coupled only by mbarriers (every wait is bounded):
//   warps 0, 1       producers: walk the CTA's tile range (every other tile each) and keep a ring of NS
//                    stages filled with K and V tiles (cp.async.bulk.tensor, 3-D tiled, 128-byte swizzle).
//   next W warps     consumers: tile j of the range goes to consumer j % W:
//                        S^T = K q^T   mma.sync m16n8k16 (bf16 in, fp32 out): the 32 keys of the tile are the M rows,
//                                      the G heads the 8 columns, so no MMA row is padding
//                        online softmax in fp32 (base-2 ex2.approx, scale folded into the logits)
//                        O^T += V^T P^T  same instruction with the d rows as M: P^T (B operand) is the 8 x 8
//                                      transposes (movmatrix) of the packed probabilities, V^T fragments come from
//                                      ldmatrix.trans
//                    and at the end of a segment each consumer leaves its partial in shared memory.
//   last warp        epilogue: fetches the queries (and the step's new k, v row) of each segment into a
//                    small ring; merges the W partials of a segment with the step's own token,
//                    writes the output row (or the scratch partial + ticket), stores the new K/V
//                    row, the index-map entry and the guide-queue row.
// The producer never waits for arithmetic, so the HBM stream is continuous across unit boundaries.
// Launched with programmatic dependent launch, a CTA lets its dependents be scheduled at once; the CTAs of the next
// layers' kernels move in as SMs free up and, before their own griddepcontrol.wait, fill their rings with tiles of
// their layer's cache -- if the cache's completion word shows that the launch that last wrote that layer has
// completed (every decode kernel publishes, after its own wait, the sequence number of its predecessor).
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace lar {

struct TensorMaps {
    // 3-D maps over {head_dim, pool rows of all layers, {K pool, V pool}}: one copy brings the K rows and
    // the V rows of a tile; box = 64 elements x 4 (i + 1) rows x 2
    CUtensorMap kv[8];
};

constexpr int kStreamTile = 32;  // rows of K (and of V) per tile of the streaming kernel; a tile lies inside one page

struct StreamArgs {
    LayerView lv;
    const void* q;      // [units * G][d]
    const void* k_new;  // [units][d]   (fused only)
    const void* v_new;
    void* out;          // [units * G][d]
    float* partials;    // scratch [units][max_seg][G][d + 2]
    int* tickets;       // scratch [units], zero between launches
    float scale_log2;   // softmax scale * log2(e)
    int len, n_tok;     // live rows per unit / visual tokens appended so far, before this step's append
    int unit_ranges;    // 1: CTA ranges end on unit boundaries
    const float* rope;  // rotary embedding: [sequence][d] floats, cos of the d/2 pairs then sin, for this step's position
    int rope_mode;      // 0: none; 1: pairs (i, i + d/2); 2: pairs (2 i, 2 i + 1)
    int fused;          // 1: the step's token comes from k_new / v_new and is appended by this kernel
    int prefetch;       // the CTA may fill its ring before waiting for the preceding kernel: 1 if the completion word covers
                        // need_seq; 2 unconditionally (the host knows that launch need_seq cannot be in flight any more)
    int n_units, n_stages, max_seg;
    // what the host knows about the launch's tile list, so that a CTA divides nothing on its way to its first copy:
    int tiles_per_unit;        // T = ceil(len / 32), 1 for an empty cache
    unsigned tiles_magic;      // floor(2^32 / T) + 1: x / T = umulhi(x, magic) up to a correction of one
    int range_ctas, range_q, range_r;  // CTAs that get work, items per CTA, CTAs that get one item more (items: units or tiles)
    int page_shift;            // log2(page_tokens)
    int seq, need_seq;  // sequence number of this launch on its cache / of the launch that last wrote this layer's cache
    int* done_seq;      // device word: every launch up to this number has completed
    int q_slots, p_bufs;  // depth of the CTA's query ring / number of partial buffers
    int stall_test;     // test hook: the producers issue no copy, so that the consumers' bounded waits run out
    int pool_row_base;  // first pool row of this layer in the tensor maps
    // elements between consecutive sequences of q / k_new / v_new / out (0: dense, heads of a sequence back to back and
    // sequences back to back); within a sequence the heads are always back to back
    long long q_seq_stride, k_seq_stride, v_seq_stride, out_seq_stride;
};

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar, uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3, %4}], [%5], %6;" ::"r"(dst),
        "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(z), "r"(bar), "l"(policy)
        : "memory");
}
// hint: bring [p, p + bytes) into L2 (p 16-byte aligned, bytes a multiple of 16); no data reaches the SM
__device__ __forceinline__ void l2_prefetch_bulk(const void* p, uint32_t bytes) {
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(p), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
// D (16x8, fp32) += A (16x16, bf16, row) * B (16x8, bf16, col)
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&t);
}
// 2^x, x <= 0 or -inf (relative error 2^-22; -inf gives 0)
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// transpose of an 8 x 8 matrix of 16-bit elements held one 32-bit pair per thread (row lane / 4, columns 2 (lane % 4), + 1)
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t x) {
    uint32_t y;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(y) : "r"(x));
    return y;
}
__device__ __forceinline__ float bf16_bits_to_float(uint16_t b) { return __uint_as_float((uint32_t)b << 16); }

template <int D>
struct MmaTraits {
    static constexpr int ROW_BYTES = D * 2;
    static constexpr int HALVES = D / 64;                  // 128-byte column blocks per row
    static constexpr int HALF_BYTES = 2 * kStreamTile * 128;  // one swizzled block: [K rows | V rows][64 elements]
    static constexpr int STAGE_BYTES = HALVES * HALF_BYTES;
    static constexpr int KSTEPS = D / 16;
    static constexpr int NTILES = D / 8;
};

// A stage holds HALVES blocks of 128-byte lines; a block is what one copy of box height b delivers: lines
// 0 .. b-1 are the K rows, lines b .. 2b-1 the V rows (128-byte swizzle on the line index).
// Byte offset of 16-byte chunk `c` of line `r` of a stage:
template <int D>
__device__ __forceinline__ uint32_t tile_off(int r, int c) {
    return (uint32_t)((c >> 3) * MmaTraits<D>::HALF_BYTES + r * 128 + (((c & 7) ^ (r & 7)) << 4));
}

// ---- shared-memory plan of decode_stream_kernel (host and device agree through these) -------------
constexpr int kMaxConsumers = 6;  // consumer warps per CTA at most
constexpr int kPartialPad = 4;    // floats behind the D values of a partial: m, l and padding that keeps rows 16-byte aligned
constexpr int kProducers = 2;     // producer warps per CTA: tile j is fetched by producer j % kProducers
constexpr int kMaxQSlots = 8;     // depth of the query ring at most
// query ring / partial buffers of a CTA that works on at most `segs` segments per launch
// (a power of two, so that ring positions are masks and shifts: every warp takes them once per segment)
__host__ __device__ constexpr int stream_q_slots(int G, int segs) {
    const int q = G <= 2 ? 8 : 4;
    int r = 1;
    while (2 * r <= segs && 2 * r <= q) r *= 2;
    return r;
}
__host__ __device__ constexpr int stream_partial_bufs(int segs) { return segs < 2 ? 1 : 2; }
__host__ __device__ constexpr int stream_q_entry_bytes(int D, int G) { return ((G + 2) * D * 2 + 127) / 128 * 128; }
__host__ __device__ constexpr int stream_fixed_smem_bytes(int D, int G, int W, int NQ, int NPB) {
    return 1024                                  // slack: the ring starts on a 1024-byte boundary
           + NQ * stream_q_entry_bytes(D, G)     // query ring
           + NPB * (W + 1) * G * (D + kPartialPad) * 4  // partial buffers
           + (3 * kMaxQSlots + 4) * 8 + 16;      // query / partial barriers, abort flag
}
__host__ __device__ constexpr int stream_smem_bytes(int D, int G, int W, int NS, int NQ, int NPB) {
    return stream_fixed_smem_bytes(D, G, W, NQ, NPB) + NS * (2 * (D / 64) * kStreamTile * 128 + 16);  // stage + its 2 barriers
}

// Wait on an mbarrier phase; gives up (and raises the CTA-wide abort flag) after ~1 s of SM clocks or as
// soon as another role has given up, so that no role can hang.
__device__ __forceinline__ bool wait_or_abort(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    unsigned spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 15u) == 0u) {
            if (*abort_flag) return false;
            if (clock64() - t0 > 2000000000LL) {
                *abort_flag = 1;
                return false;
            }
        }
    }
    return true;
}
// barrier initialisations become visible to the copy engine's arrivals (shared memory only: nothing in flight to
// global memory is waited for)
__device__ __forceinline__ void mbar_fence_init_smem() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
// named CTA barriers: `threads` threads take part; arrive does not wait
__device__ __forceinline__ void named_bar_sync(int id, int threads) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory"); }
__device__ __forceinline__ void named_bar_arrive(int id, int threads) { asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(threads) : "memory"); }
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void fence_proxy_async_global() { asm volatile("fence.proxy.async.global;" ::: "memory"); }
__device__ __forceinline__ int ld_acquire_gpu(const int* p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_gpu(int* p, int v) {
    asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ float exp2_or_zero(float m_part, float m_all) {
    return m_part == -INFINITY ? 0.f : ex2_approx(m_part - m_all);
}

// A list of n items is dealt to P <= n CTAs in contiguous ranges, the first n % P of them one item longer.
// (32-bit arithmetic throughout: the host rejects configurations with 2^30 tiles or more per layer.)
__device__ __forceinline__ int range_begin(int n, int P, int p) {
    const int q = n / P, r = n - q * P;
    return p * q + (p < r ? p : r);
}
// CTA that owns item t
__device__ __forceinline__ int range_owner(int t, int n, int P) {
    const int q = n / P, r = n - q * P;
    const int head = r * (q + 1);
    return t < head ? t / (q + 1) : r + (t - head) / q;
}

// VIEWS: q / k / v / out may be views of larger tensors (the *_seq_stride arguments) and the rotary embedding of q and
// the new k may be fused in (a.rope, a.rope_mode); a kernel of its own, so that launches on dense tensors carry none of
// that per-segment work (with many short units per CTA the epilogue warp's work per unit sets the pace)
template <int D, int G, bool VIEWS>
__global__ void __launch_bounds__(288, 1) decode_stream_kernel(const StreamArgs a, const __grid_constant__ TensorMaps tm) {
    using TR = MmaTraits<D>;
    using T16 = __nv_bfloat16;
    const int NQ = a.q_slots, NPB = a.p_bufs;  // powers of two
    const int qsh = __ffs(NQ) - 1, psh = NPB - 1;
    constexpr int QENT = stream_q_entry_bytes(D, G);
    constexpr int PS = D + kPartialPad;  // floats per (warp, head) partial: o[D], m, l (+ padding: 16-byte aligned rows)
    constexpr int PER = D / 32;
    extern __shared__ unsigned char smem_raw[];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int W = (int)(blockDim.x >> 5) - kProducers - 1;  // consumer warps
    const int NS = a.n_stages;
    const int p = (int)blockIdx.x;
    const LayerView& lv = a.lv;

    const uint32_t ring = (smem_u32(smem_raw) + 1023u) & ~1023u;
    unsigned char* smem = smem_raw + (ring - smem_u32(smem_raw));
    unsigned char* qring_ptr = smem + (size_t)NS * TR::STAGE_BYTES;
    const uint32_t qring = smem_u32(qring_ptr);
    float* pbuf = reinterpret_cast<float*>(qring_ptr + NQ * QENT);
    const int pbuf_floats = (W + 1) * G * PS;
    unsigned char* bars_ptr = reinterpret_cast<unsigned char*>(pbuf + NPB * pbuf_floats);
    const uint32_t bars = smem_u32(bars_ptr);
    const uint32_t bar_full = bars, bar_empty = bars + NS * 8;
    const uint32_t bar_qfull = bars + 2 * NS * 8, bar_qempty = bar_qfull + kMaxQSlots * 8;
    const uint32_t bar_pfull = bar_qempty + kMaxQSlots * 8, bar_pempty = bar_pfull + 2 * 8;
    const uint32_t bar_qrot = bar_pempty + 2 * 8;  // (rotary embedding) the slot's q and k rows have been rotated
    // what the consumers wait for before they take a segment's queries
    const uint32_t bar_qready = (VIEWS && a.rope_mode) ? bar_qrot : bar_qfull;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bars_ptr + (2 * NS + 3 * kMaxQSlots + 4) * 8);

    // Dependents may be scheduled from now on: they only hint the L2 before their own griddepcontrol.wait, and a
    // dependent's wait covers this whole grid (which itself waits for its predecessor below).
    grid_dep_launch();

    // The set-up of a launch is on the path between two launches: the two producer warps initialise every barrier (each
    // thread one or two), agree among themselves, tell the other warps without waiting for them (bar.arrive) and go on
    // to their first copies; the other warps wait for that signal only.
    if (warp < kProducers) {
        const int n_bars = 2 * NS + 3 * NQ + 4;
        for (int t = (int)threadIdx.x; t < n_bars; t += kProducers * 32) {
            if (t < 2 * NS) {
                mbar_init(bar_full + t * 8, 1);  // full / empty of the K/V ring (adjacent in memory)
            } else if (t < 2 * NS + NQ) {
                mbar_init(bar_qfull + (t - 2 * NS) * 8, 1);
            } else if (t < 2 * NS + 2 * NQ) {
                mbar_init(bar_qempty + (t - 2 * NS - NQ) * 8, (uint32_t)(W + 1));
            } else if (t < 2 * NS + 2 * NQ + 2) {
                mbar_init(bar_pfull + (t - 2 * NS - 2 * NQ) * 8, (uint32_t)W);
            } else if (t < 2 * NS + 2 * NQ + 4) {
                mbar_init(bar_pempty + (t - 2 * NS - 2 * NQ - 2) * 8, 1);
            } else {
                mbar_init(bar_qrot + (t - 2 * NS - 2 * NQ - 4) * 8, 1);
            }
        }
        if (threadIdx.x == 0) *abort_flag = 0;
        mbar_fence_init_smem();
        named_bar_sync(2, kProducers * 32);
        named_bar_arrive(1, (int)blockDim.x);
    } else {
        named_bar_sync(1, (int)blockDim.x);
    }


    // ---- the layer's tile list and this CTA's range of it
    const int len = a.len, n_tok = a.n_tok;
    const int T = a.tiles_per_unit;  // ceil(len / 32); an empty cache is one tile of 0 rows
    const int total = a.n_units * T;
    // x / T for 0 <= x < 2^30 without a division (the host's multiplier, corrected by at most one)
    auto div_T = [&](int x) {
        if (T == 1) return x;  // (the multiplier of 1 does not fit 32 bits)
        int q = (int)__umulhi((unsigned)x, a.tiles_magic);
        if (q * T > x) --q;
        else if ((q + 1) * T <= x) ++q;
        return q;
    };
    int t_begin = 0, t_end = 0;
    const int Pe = a.range_ctas;  // CTAs that get work: every range is non-empty
    if (p < Pe) {
        // the first range_r CTAs get range_q + 1 items, the others range_q (items: whole units, or tiles)
        const int b0 = p * a.range_q + (p < a.range_r ? p : a.range_r), b1 = b0 + a.range_q + (p < a.range_r ? 1 : 0);
        t_begin = a.unit_ranges ? b0 * T : b0;
        t_end = a.unit_ranges ? b1 * T : b1;
    }
    const int n_tiles = t_end - t_begin;
    const int u0 = div_T(t_begin);
    const int n_segs = n_tiles > 0 ? div_T(t_end - 1) - u0 + 1 : 0;

    // One lane requests the inputs of segment `seg`: its queries and, where the segment closes its unit in a fused
    // step, the new k and v rows.  Issued by the epilogue warp, which is idle when a launch starts, so that the
    // producer's first K/V copies are not queued behind them.
    // element offset of unit `u`'s rows in a [sequence][head][d] tensor with `per_head` elements per KV head
    auto unit_offset = [&](int u, long long seq_stride, int per_head) -> size_t {
        if (!VIEWS || seq_stride == 0) return (size_t)u * per_head;
        const int sq = u / lv.n_kv_heads;
        return (size_t)sq * (size_t)seq_stride + (size_t)(u - sq * lv.n_kv_heads) * per_head;
    };
    auto issue_inputs = [&](int seg) -> bool {
        const int slot = seg & (NQ - 1);
        if (seg >= NQ && !wait_or_abort(bar_qempty + slot * 8, (uint32_t)(((seg >> qsh) - 1) & 1), abort_flag)) return false;
        const int unit = u0 + seg;
        const bool closes = (unit + 1) * T <= t_end;  // the segment holds the unit's last tile
        const bool with_kv = a.fused && closes;
        const uint32_t bar = bar_qfull + slot * 8, dst = qring + slot * QENT;
        mbar_expect_tx(bar, (uint32_t)((G + (with_kv ? 2 : 0)) * D * 2));
        bulk_g2s(dst, reinterpret_cast<const T16*>(a.q) + unit_offset(unit, a.q_seq_stride, G * D), G * D * 2, bar);
        if (with_kv) {
            bulk_g2s(dst + G * D * 2, reinterpret_cast<const T16*>(a.k_new) + unit_offset(unit, a.k_seq_stride, D), D * 2, bar);
            bulk_g2s(dst + (G + 1) * D * 2, reinterpret_cast<const T16*>(a.v_new) + unit_offset(unit, a.v_seq_stride, D), D * 2, bar);
        }
        return true;
    };

    if (warp < kProducers) {
        // =========================================================================== producers
        // Producer pw fetches the tiles pw, pw + kProducers, ... of the CTA's range (a single thread sustains only one
        // tiled copy per ~140 cycles, two keep the ring ahead of the consumers).  NS is a multiple of kProducers, so
        // a stage is always filled by the same producer.
        const int pw = warp;
        bool ok = true;
        // ---- before the dependency: may the ring be filled already?  Every launch on a cache carries a sequence
        // number; a decode kernel whose own dependency has resolved publishes the number of its predecessor (all
        // launches up to that one have completed and their writes are visible to it).  The rows of this layer are
        // final once the launch that last wrote them (need_seq, from the host) is covered by that word -- or, without
        // looking, if that launch lies further back than launches can be in flight at all (the host's bound: every
        // launch but the oldest in flight is wholly resident, waiting for its predecessor).
        int fill_end = 0;
        if (a.prefetch == 2 || (a.prefetch == 1 && ld_acquire_gpu(a.done_seq) >= a.need_seq)) {
            fence_proxy_async_global();  // the copies below read what the acquire made visible
            fill_end = n_tiles < NS ? n_tiles : NS;
        }
        bool dep_waited = false;
        // (test hook stall_test: the producers have nothing to request; the consumers' waits for their first tiles run
        // into the limit and the launch ends with the wait-limit status bit)
        const int n_local = (n_tiles > pw && !a.stall_test) ? (n_tiles - pw + kProducers - 1) / kProducers : 0;

        auto describe = [&](int jj, int& y, int& rows, int& tile) {
            const int t = t_begin + jj;
            const int unit = div_T(t);
            tile = t - unit * T;
            const int row0 = tile * kStreamTile;
            rows = len - row0 < kStreamTile ? len - row0 : kStreamTile;
            if (rows > 0) {
                const int pidx = unit * lv.pages_per_unit + (row0 >> a.page_shift);
                const int page = lv.identity_pages ? pidx : __ldg(&lv.page_table[pidx]);
                y = a.pool_row_base + (page << a.page_shift) + (row0 & (lv.page_tokens - 1));
            } else {
                y = 0;
            }
        };
        // Lane 0 issues; all lanes look the page ids of a batch of 32 tiles up together, one batch ahead.
        // Stage and phase advance incrementally (no division in the per-tile path).
        int y_n = 0, rt_n = 0;  // rt = rows | tile << 8
        {
            int r = 0, t = 0;
            if (lane < n_local) describe(kProducers * lane + pw, y_n, r, t);
            rt_n = r | (t << 8);
        }
        // every cached row is read once per step: let it leave L2 first
        const uint64_t pol_stream = l2_policy_evict_first();
        int stage = pw;
        uint32_t empty_parity = 1;
        for (int i0 = 0; i0 < n_local; i0 += 32) {
            const int y = y_n, rt = rt_n;
            if (i0 + 32 + lane < n_local) {  // next batch: hides the table reads
                int r = 0, t = 0;
                describe(kProducers * (i0 + 32 + lane) + pw, y_n, r, t);
                rt_n = r | (t << 8);
            }
            const int cnt = n_local - i0 < 32 ? n_local - i0 : 32;
            for (int i = 0; i < cnt; ++i) {
                if (!dep_waited && kProducers * (i0 + i) + pw >= fill_end) {
                    grid_dep_wait();  // every tile from here on may still be written by the preceding kernels
                    dep_waited = true;
                }
                const int yi = __shfl_sync(0xffffffffu, y, i), rti = __shfl_sync(0xffffffffu, rt, i);
                if (lane == 0 && ok) {
                    const int ri = rti & 0xff;
                    // (the first trip round the ring finds every stage free: no wait on the way to the first copies)
                    if (i0 + i >= NS / kProducers) ok = wait_or_abort(bar_empty + stage * 8, empty_parity, abort_flag);
                    if (ok) {
                        const uint32_t bar = bar_full + stage * 8, dst = ring + (uint32_t)stage * TR::STAGE_BYTES;
                        if (ri > 0) {
                            const int hsel = (ri + 3) / 4 - 1;  // box of 4 * (hsel + 1) rows
                            mbar_expect_tx(bar, (uint32_t)(2 * 4 * (hsel + 1) * TR::ROW_BYTES));
#pragma unroll
                            for (int h = 0; h < TR::HALVES; ++h) tma_load_3d(dst + h * TR::HALF_BYTES, &tm.kv[hsel], h * 64, yi, 0, bar, pol_stream);
                        } else {
                            mbar_arrive(bar);  // nothing to fetch: release the consumer
                        }
                    }
                    stage += kProducers;
                    if (stage >= NS) {
                        stage -= NS;
                        empty_parity ^= 1u;
                    }
                }
            }
        }
        if (!dep_waited) grid_dep_wait();
        if (!ok && lane == 0) atomicOr(lv.status, kStWaitLimit);
    } else if (warp < kProducers + W) {
        // =========================================================================== consumers
        grid_dep_wait();
        const int cw = warp - kProducers;
        const int quad = lane & 3, qrow = lane >> 2;  // fragment coordinates
        bool ok = true;
        // This consumer takes tiles cw, cw + W, ... of the CTA's range.  NS is a multiple of W, so a stage is
        // always read by the same consumer, which has seen every earlier phase of its barrier.
        int j = cw, stage = cw;
        uint32_t full_parity = 0;
        for (int seg = 0; seg < n_segs && ok; ++seg) {
            const int unit = u0 + seg;
            const int ub = unit * T;
            const int je = (ub + T < t_end ? ub + T : t_end) - t_begin;

            // ---- Q fragments (B operand): column qrow = head, 16 dims per k-step; heads >= G are zero columns
            const int qs = seg & (NQ - 1);
            // The queries of the CTA's first unit are what the whole launch waits for once its dependency has resolved:
            // the consumers read them straight from global memory (L2: hinted there before the wait), which is quicker
            // than waiting for the epilogue warp's copy into shared memory and its barrier.  (Not with the fused rotary
            // embedding: the rotated rows exist in shared memory only.)
            const bool q_direct = seg == 0 && !(VIEWS && a.rope_mode);
            uint32_t qa0[TR::KSTEPS], qa2[TR::KSTEPS];
            if (q_direct) {
                const uint32_t* Qg = reinterpret_cast<const uint32_t*>(reinterpret_cast<const T16*>(a.q) + unit_offset(unit, a.q_seq_stride, G * D));
#pragma unroll
                for (int s = 0; s < TR::KSTEPS; ++s) {
                    qa0[s] = 0u;
                    qa2[s] = 0u;
                    if (qrow < G) {
                        qa0[s] = __ldcg(Qg + (qrow * D + 16 * s + 2 * quad) / 2);
                        qa2[s] = __ldcg(Qg + (qrow * D + 16 * s + 8 + 2 * quad) / 2);
                    }
                }
            } else {
                ok = wait_or_abort(bar_qready + qs * 8, (uint32_t)(((seg >> qsh)) & 1), abort_flag);
                if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
                const unsigned char* Qs = qring_ptr + qs * QENT;
#pragma unroll
                for (int s = 0; s < TR::KSTEPS; ++s) {
                    qa0[s] = 0u;
                    qa2[s] = 0u;
                    if (qrow < G) {
                        qa0[s] = *reinterpret_cast<const uint32_t*>(Qs + (qrow * D + 16 * s + 2 * quad) * 2);
                        qa2[s] = *reinterpret_cast<const uint32_t*>(Qs + (qrow * D + 16 * s + 8 + 2 * quad) * 2);
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_qempty + qs * 8);
            }

            // running maximum and this thread's share of the row sum of heads 2 quad and 2 quad + 1
            float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
            // O^T: o[t][0], o[t][1] = heads 2 quad, 2 quad + 1 at d = 16 t + qrow; o[t][2], o[t][3] at d + 8
            float o[TR::KSTEPS][4];
#pragma unroll
            for (int t = 0; t < TR::KSTEPS; ++t) o[t][0] = o[t][1] = o[t][2] = o[t][3] = 0.f;

            for (; j < je; j += W) {
                const int s = stage;
                ok = wait_or_abort(bar_full + s * 8, full_parity, abort_flag);
                if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
                stage += W;
                if (stage >= NS) {
                    stage -= NS;
                    full_parity ^= 1u;
                }
                const int tile = t_begin + j - ub;
                const int rows = len - tile * kStreamTile < kStreamTile ? len - tile * kStreamTile : kStreamTile;
                const uint32_t St = ring + (uint32_t)s * TR::STAGE_BYTES;
                if (rows > 0) {
                    const int box_rows = (rows + 3) & ~3;  // K rows are lines 0.., V rows lines box_rows.. of a block
                    // S^T[key][head] = K q^T for the 32 keys of the tile: the keys are the M rows (two 16-key tiles), the
                    // heads the 8 columns, so no MMA row is padding; even and odd k-steps go to accumulators of their own
                    float c[2][2][4];
#pragma unroll
                    for (int mt = 0; mt < 2; ++mt) {
#pragma unroll
                        for (int e = 0; e < 2; ++e) c[mt][e][0] = c[mt][e][1] = c[mt][e][2] = c[mt][e][3] = 0.f;
#pragma unroll
                        for (int ks = 0; ks < TR::KSTEPS; ++ks) {
                            uint32_t af[4];  // keys 16 mt + (lane & 15), 16 dims from 16 ks
                            ldmatrix_x4(St + tile_off<D>(16 * mt + (lane & 15), 2 * ks + (lane >> 4)), af);
                            mma_bf16(c[mt][ks & 1], af[0], af[1], af[2], af[3], qa0[ks], qa2[ks]);
                        }
                    }
                    // this thread: keys qrow + {0, 8, 16, 24}, heads 2 quad and 2 quad + 1
                    float sv[4][2];
#pragma unroll
                    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                        for (int hf = 0; hf < 2; ++hf) {
                            const bool live = 16 * mt + 8 * hf + qrow < rows;
                            sv[2 * mt + hf][0] = live ? (c[mt][0][2 * hf] + c[mt][1][2 * hf]) * a.scale_log2 : -INFINITY;
                            sv[2 * mt + hf][1] = live ? (c[mt][0][2 * hf + 1] + c[mt][1][2 * hf + 1]) * a.scale_log2 : -INFINITY;
                        }
                    float mx0 = fmaxf(fmaxf(sv[0][0], sv[1][0]), fmaxf(sv[2][0], sv[3][0]));
                    float mx1 = fmaxf(fmaxf(sv[0][1], sv[1][1]), fmaxf(sv[2][1], sv[3][1]));
#pragma unroll
                    for (int off = 4; off <= 16; off <<= 1) {
                        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, off));
                        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, off));
                    }
                    // rows >= 1: the tile has a live key, so the new maxima are finite
                    const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);
                    const float ca = ex2_approx(m0 - mn0), cb = ex2_approx(m1 - mn1);
                    float pr[4][2];
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        pr[k][0] = ex2_approx(sv[k][0] - mn0);
                        pr[k][1] = ex2_approx(sv[k][1] - mn1);
                    }
                    l0 = l0 * ca + ((pr[0][0] + pr[1][0]) + (pr[2][0] + pr[3][0]));
                    l1 = l1 * cb + ((pr[0][1] + pr[1][1]) + (pr[2][1] + pr[3][1]));
                    m0 = mn0;
                    m1 = mn1;
                    // the accumulator columns of this thread belong to the same two heads
#pragma unroll
                    for (int t = 0; t < TR::KSTEPS; ++t) { o[t][0] *= ca; o[t][1] *= cb; o[t][2] *= ca; o[t][3] *= cb; }
                    // P^T as B operand (keys 2 quad, 2 quad + 1 of an 8-key block; head qrow): transpose the 8 x 8 blocks
                    const uint32_t pb00 = movmatrix_trans(pack_bf16(pr[0][0], pr[0][1])), pb01 = movmatrix_trans(pack_bf16(pr[1][0], pr[1][1]));
                    const uint32_t pb10 = movmatrix_trans(pack_bf16(pr[2][0], pr[2][1])), pb11 = movmatrix_trans(pack_bf16(pr[3][0], pr[3][1]));
                    // a short box leaves the lines behind its V rows unwritten: their weight is 0, but
                    // 0 * (stale NaN) is not
                    if (box_rows < kStreamTile) {
                        const int n16 = (kStreamTile - box_rows) * 8;  // 16-byte chunks per block
                        for (int i = lane; i < n16 * TR::HALVES; i += 32) {
                            const int h = i / n16, c = i - h * n16;
                            asm volatile("st.shared.v4.u32 [%0], {%1, %1, %1, %1};" ::"r"(St + h * TR::HALF_BYTES + 2 * box_rows * 128 + c * 16), "r"(0u) : "memory");
                        }
                        __syncwarp();
                    }
                    // O^T[d][head] += V^T[d][key] P^T[key][head]
#pragma unroll
                    for (int t = 0; t < TR::KSTEPS; ++t) {
                        uint32_t af[4];
                        ldmatrix_x4_trans(St + tile_off<D>(box_rows + (lane & 7) + 8 * (lane >> 4), 2 * t + ((lane >> 3) & 1)), af);
                        mma_bf16(o[t], af[0], af[1], af[2], af[3], pb00, pb01);
                        ldmatrix_x4_trans(St + tile_off<D>(box_rows + 16 + (lane & 7) + 8 * (lane >> 4), 2 * t + ((lane >> 3) & 1)), af);
                        mma_bf16(o[t], af[0], af[1], af[2], af[3], pb10, pb11);
                    }
                    if (box_rows < kStreamTile) fence_proxy_async_smem();  // zero-fill before the next TMA write
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_empty + s * 8);
            }
            if (!ok) break;
            if (q_direct) {
                // the slot of the first segment is released here, after its copy has landed (long ago: a waiter must
                // have seen every phase of a barrier it will wait on again)
                ok = wait_or_abort(bar_qready + qs * 8, 0u, abort_flag);
                if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
                if (lane == 0) mbar_arrive(bar_qempty + qs * 8);
            }

            // ---- this warp's partial of the segment -> shared memory
            const int buf = seg & (NPB - 1);
            if (seg >= NPB) {
                ok = wait_or_abort(bar_pempty + buf * 8, (uint32_t)(((seg >> psh) - 1) & 1), abort_flag);
                if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
            }
#pragma unroll
            for (int off = 4; off <= 16; off <<= 1) {
                l0 += __shfl_xor_sync(0xffffffffu, l0, off);
                l1 += __shfl_xor_sync(0xffffffffu, l1, off);
            }
            {
                float* wp = pbuf + buf * pbuf_floats + cw * G * PS;
                if (2 * quad < G) {
#pragma unroll
                    for (int t = 0; t < TR::KSTEPS; ++t) {
                        wp[2 * quad * PS + 16 * t + qrow] = o[t][0];
                        wp[2 * quad * PS + 16 * t + 8 + qrow] = o[t][2];
                    }
                    if (qrow == 0) {
                        wp[2 * quad * PS + D] = m0;
                        wp[2 * quad * PS + D + 1] = l0;
                    }
                }
                if (2 * quad + 1 < G) {
#pragma unroll
                    for (int t = 0; t < TR::KSTEPS; ++t) {
                        wp[(2 * quad + 1) * PS + 16 * t + qrow] = o[t][1];
                        wp[(2 * quad + 1) * PS + 16 * t + 8 + qrow] = o[t][3];
                    }
                    if (qrow == 0) {
                        wp[(2 * quad + 1) * PS + D] = m1;
                        wp[(2 * quad + 1) * PS + D + 1] = l1;
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_pfull + buf * 8);
        }
        if (!ok && lane == 0) atomicOr(lv.status, kStWaitLimit);
    } else {
        // =========================================================================== epilogue
        if (a.prefetch) {
            // a hint only (L2 is the point of coherence): the inputs of the first segments -- the ones the launch waits for
            // -- start their way from HBM before the dependency resolves, if the kernel that produced them has not left
            // them in L2 anyway
            for (int sg = lane; sg < n_segs && sg < NQ; sg += 32) {
                const int un = u0 + sg;
                l2_prefetch_bulk(reinterpret_cast<const T16*>(a.q) + unit_offset(un, a.q_seq_stride, G * D), G * D * 2);
                if (a.fused && (un + 1) * T <= t_end) {
                    l2_prefetch_bulk(reinterpret_cast<const T16*>(a.k_new) + unit_offset(un, a.k_seq_stride, D), D * 2);
                    l2_prefetch_bulk(reinterpret_cast<const T16*>(a.v_new) + unit_offset(un, a.v_seq_stride, D), D * 2);
                }
            }
        }
        grid_dep_wait();
        if (p == 0 && lane == 0) st_release_gpu(a.done_seq, a.seq - 1);  // everything before this launch has completed
        bool ok = true;
        if (lane == 0)
            for (int sg = 0; sg < NQ && sg < n_segs && ok; ++sg) ok = issue_inputs(sg);  // the input ring's first round
        ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
        T16* outp = reinterpret_cast<T16*>(a.out);
        // What closing a unit needs from global memory (the page that takes the new row, the unit's length
        // in device memory) is requested one segment ahead, so that its latency never stalls this warp.
        const int new_page_idx = len / lv.page_tokens, new_row_in_page = len - new_page_idx * lv.page_tokens;
        const int step_tok = a.fused ? n_tok : n_tok - 1;  // 0-based visual index of this step's token
        const int guide_slot = step_tok >= 0 ? step_tok % lv.line_width : 0;
        auto closing_loads = [&](int sg, int& page, int& dev_len) {
            const int un = u0 + sg;
            page = 0;
            dev_len = len;
            if (sg < n_segs && (un + 1) * T <= t_end) {
                if (a.fused && len < lv.cap) {
                    const int pidx = un * lv.pages_per_unit + new_page_idx;
                    page = lv.identity_pages ? pidx : __ldg(&lv.page_table[pidx]);
                }
                dev_len = __ldcg(&lv.state[un].len);
            }
        };
        int page_cur, dev_len_cur, page_nxt = 0, dev_len_nxt = 0;
        closing_loads(0, page_cur, dev_len_cur);
        for (int seg = 0; seg < n_segs && ok; ++seg, page_cur = page_nxt, dev_len_cur = dev_len_nxt) {
            const int unit = u0 + seg;
            const int ub = unit * T;
            const bool opens = ub >= t_begin, closes = ub + T <= t_end;
            const size_t out_base = unit_offset(unit, a.out_seq_stride, G * D);
            const int qs = seg & (NQ - 1), buf = seg & (NPB - 1);
            closing_loads(seg + 1, page_nxt, dev_len_nxt);
            // rotary embedding: cos and sin of this sequence's position for the pairs this lane rotates (on their way
            // while the inputs arrive)
            float rc[D / 64], rs[D / 64];
            if (VIEWS && a.rope_mode) {
                const float* cs = a.rope + (size_t)(unit / lv.n_kv_heads) * D;
#pragma unroll
                for (int k = 0; k < D / 64; ++k) {
                    rc[k] = __ldg(cs + lane + 32 * k);
                    rs[k] = __ldg(cs + D / 2 + lane + 32 * k);
                }
            }
            ok = wait_or_abort(bar_qfull + qs * 8, (uint32_t)(((seg >> qsh)) & 1), abort_flag);
            if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
            const unsigned char* Qs = qring_ptr + qs * QENT;
            const uint16_t* Q16 = reinterpret_cast<const uint16_t*>(Qs);
            if (VIEWS && a.rope_mode) {
                // q (all G heads) and the new k row are rotated in place, pair by pair, in fp32 with every product and
                // sum rounded separately, then rounded to bf16: the cache, the guide queue and the logits see rotated rows
                T16* rows = reinterpret_cast<T16*>(qring_ptr + qs * QENT);
                const int n_rows = G + ((a.fused && closes) ? 1 : 0);
                for (int r = 0; r < n_rows; ++r) {
#pragma unroll
                    for (int k = 0; k < D / 64; ++k) {
                        const int i = lane + 32 * k;  // pair: (i, i + d/2), or (2 i, 2 i + 1) in the interleaved convention
                        const int ia = a.rope_mode == 1 ? i : 2 * i, ib = a.rope_mode == 1 ? i + D / 2 : 2 * i + 1;
                        const float x = __bfloat162float(rows[r * D + ia]), y = __bfloat162float(rows[r * D + ib]);
                        rows[r * D + ia] = __float2bfloat16_rn(__fsub_rn(__fmul_rn(x, rc[k]), __fmul_rn(y, rs[k])));
                        rows[r * D + ib] = __float2bfloat16_rn(__fadd_rn(__fmul_rn(y, rc[k]), __fmul_rn(x, rs[k])));
                    }
                }
                fence_proxy_async_smem();  // these writes come before the copy that refills the slot
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_qrot + qs * 8);
            }

            // ---- the token of this step (Eq. 4, 8): logit per head, value row, stores
            // Merge layout: the warp's lanes are split over the G heads, LPH lanes per head; lane (hg, sub) owns the EPH
            // consecutive elements from e0 = sub * EPH of head hg (vector loads from the partials, one vector store of the
            // output) -- one set of exponentials per lane, not G.
            constexpr int LPH = 32 / G, EPH = D / LPH;
            constexpr int VEC = EPH % 4 == 0 ? 4 : 2;  // floats per shared-memory load
            const int hg = lane / LPH, sub = lane % LPH, e0 = sub * EPH;
            float s_new[G], v_new[EPH];
            const bool with_new = a.fused && closes;
#pragma unroll
            for (int g = 0; g < G; ++g) s_new[g] = -INFINITY;
#pragma unroll
            for (int i = 0; i < EPH; ++i) v_new[i] = 0.f;
            if (closes) {
                if (with_new) {
                    const uint16_t* K16 = Q16 + G * D;
                    const uint16_t* V16 = K16 + D;
                    float kf[PER];
#pragma unroll
                    for (int i = 0; i < PER; ++i) kf[i] = bf16_bits_to_float(K16[lane + 32 * i]);
#pragma unroll
                    for (int i = 0; i < EPH; ++i) v_new[i] = bf16_bits_to_float(V16[e0 + i]);
#pragma unroll
                    for (int g = 0; g < G; ++g) {
                        float sv = 0.f;
#pragma unroll
                        for (int i = 0; i < PER; ++i) sv = fmaf(bf16_bits_to_float(Q16[g * D + lane + 32 * i]), kf[i], sv);
#pragma unroll
                        for (int off = 16; off >= 1; off >>= 1) sv += __shfl_xor_sync(0xffffffffu, sv, off);
                        s_new[g] = sv * a.scale_log2;
                    }
                    if (len < lv.cap) {
                        const size_t off = ((size_t)page_cur * lv.page_tokens + new_row_in_page) * TR::ROW_BYTES;
                        const uint32_t* K32 = reinterpret_cast<const uint32_t*>(K16);
                        const uint32_t* V32 = reinterpret_cast<const uint32_t*>(V16);
                        for (int i = lane; i < D / 2; i += 32) {
                            reinterpret_cast<uint32_t*>(lv.k_pool + off)[i] = K32[i];
                            reinterpret_cast<uint32_t*>(lv.v_pool + off)[i] = V32[i];
                        }
                        if (lane == 0) lv.index_map[(size_t)unit * lv.cap_pad + len] = lv.cond_len + n_tok;
                    } else if (lane == 0) {
                        atomicOr(lv.status, kStCapacity);
                    }
                } else if (!a.fused && len == 0 && lane == 0) {
                    atomicOr(lv.status, kStEmpty);
                }
                if (lane == 0) {
                    if (dev_len_cur != len) atomicOr(lv.status, kStLength);
                    if (a.fused) {
                        UnitState ns;
                        ns.len = len < lv.cap ? len + 1 : len;
                        ns.n_tok = n_tok + 1;
                        lv.state[unit] = ns;
                    }
                }
                // Eq. 8: the queries join the guide queue of the line being generated
                if (step_tok >= 0) {
                    uint32_t* gq = reinterpret_cast<uint32_t*>(reinterpret_cast<T16*>(lv.guide) +
                                                               (((size_t)unit * lv.line_width + guide_slot) * G) * D);
                    const uint32_t* Q32 = reinterpret_cast<const uint32_t*>(Qs);
                    for (int i = lane; i < G * D / 2; i += 32) gq[i] = Q32[i];
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_qempty + qs * 8);

            // ---- merge the consumers' partials (+ the step's token)
            ok = wait_or_abort(bar_pfull + buf * 8, (uint32_t)(((seg >> psh)) & 1), abort_flag);
            if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
            const float* pb = pbuf + buf * pbuf_floats;
            // branch-free and unrolled over the (at most kMaxConsumers) consumer warps, so that the shared-memory
            // loads are in flight together
            float s_mine = s_new[0];
#pragma unroll
            for (int g = 1; g < G; ++g) s_mine = hg == g ? s_new[g] : s_mine;
            float Mh, Lh, Oh[EPH];
            {
                float mw[kMaxConsumers];
                float M = s_mine;
#pragma unroll
                for (int w = 0; w < kMaxConsumers; ++w) {
                    mw[w] = w < W ? pb[(w * G + hg) * PS + D] : -INFINITY;
                    M = fmaxf(M, mw[w]);
                }
                const float f_new = exp2_or_zero(s_mine, M);
                float L = f_new;
#pragma unroll
                for (int i = 0; i < EPH; ++i) Oh[i] = v_new[i] * f_new;
#pragma unroll
                for (int w = 0; w < kMaxConsumers; ++w) {
                    const float* pw = pb + ((w < W ? w : 0) * G + hg) * PS;
                    const float f = exp2_or_zero(mw[w], M);
                    L = fmaf(pw[D + 1], f, L);
#pragma unroll
                    for (int i = 0; i < EPH; i += VEC) {
                        float t[4];
                        if constexpr (VEC == 4) {
                            const float4 x = *reinterpret_cast<const float4*>(pw + e0 + i);
                            t[0] = x.x; t[1] = x.y; t[2] = x.z; t[3] = x.w;
                        } else {
                            const float2 x = *reinterpret_cast<const float2*>(pw + e0 + i);
                            t[0] = x.x; t[1] = x.y;
                        }
#pragma unroll
                        for (int k = 0; k < VEC; ++k) Oh[i + k] = fmaf(t[k], f, Oh[i + k]);
                    }
                }
                Mh = M;
                Lh = L;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_pempty + buf * 8);
            // this segment's slot of the input ring is free once every consumer has taken its fragments: refill it
            if (lane == 0 && seg + NQ < n_segs) ok = issue_inputs(seg + NQ);
            if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }

            if (opens && closes) {
                // the whole unit lies in this CTA
                const float inv = Lh > 0.f ? 1.f / Lh : 0.f;
                uint32_t packed[EPH / 2];
#pragma unroll
                for (int i = 0; i < EPH / 2; ++i) packed[i] = pack_bf16(Oh[2 * i] * inv, Oh[2 * i + 1] * inv);
                T16* dst = outp + out_base + (size_t)hg * D + e0;  // EPH * 2 bytes, aligned to their size (up to 16)
                if constexpr (EPH % 8 == 0) {
#pragma unroll
                    for (int i = 0; i < EPH / 8; ++i)
                        reinterpret_cast<uint4*>(dst)[i] = make_uint4(packed[4 * i], packed[4 * i + 1], packed[4 * i + 2], packed[4 * i + 3]);
                } else if constexpr (EPH == 4) {
                    *reinterpret_cast<uint2*>(dst) = make_uint2(packed[0], packed[1]);
                } else {
                    *reinterpret_cast<uint32_t*>(dst) = packed[0];
                }
            } else {
                // the unit is shared with neighbouring CTAs: leave a partial, the last one to arrive merges
                const int p_first = range_owner(ub, total, Pe);
                const int n_parts = range_owner(ub + T - 1, total, Pe) - p_first + 1;
                if (n_parts > a.max_seg) {  // cannot happen with the host's sizing of the scratch area
                    if (lane == 0) atomicOr(lv.status, kStCapacity);
                    continue;
                }
                float* mine = a.partials + ((size_t)unit * a.max_seg + (p - p_first)) * G * PS;
#pragma unroll
                for (int i = 0; i < EPH; ++i) mine[hg * PS + e0 + i] = Oh[i];
                if (sub == 0) {
                    mine[hg * PS + D] = Mh;
                    mine[hg * PS + D + 1] = Lh;
                }
                __threadfence();
                __syncwarp();
                int ticket = 0;
                if (lane == 0) ticket = atomicAdd(a.tickets + unit, 1);
                ticket = __shfl_sync(0xffffffffu, ticket, 0);
                if (ticket == n_parts - 1) {
                    __threadfence();
                    // Heads in groups of GC, parts in pairs: the loads of a pair (m, l and the o row of every head
                    // of the group) are independent of one another and of any exponential, so a pair costs one
                    // trip to L2; the pairs are folded in online-softmax fashion.
                    const float* all = a.partials + (size_t)unit * a.max_seg * G * PS;
                    constexpr int GC = G < 4 ? G : 4;
#pragma unroll
                    for (int g0 = 0; g0 < G; g0 += GC) {
                        float M[GC], L[GC], O[GC][PER];
#pragma unroll
                        for (int c = 0; c < GC; ++c) {
                            M[c] = -INFINITY;
                            L[c] = 0.f;
#pragma unroll
                            for (int i = 0; i < PER; ++i) O[c][i] = 0.f;
                        }
                        for (int s0 = 0; s0 < n_parts; s0 += 2) {
                            float mv[2][GC], lv2[2][GC], ov[2][GC][PER];
#pragma unroll
                            for (int u = 0; u < 2; ++u) {
                                const bool have = s0 + u < n_parts;
                                const float* ps = all + ((have ? s0 + u : s0) * G + g0) * PS;
#pragma unroll
                                for (int c = 0; c < GC; ++c) {
                                    mv[u][c] = __ldcg(ps + c * PS + D);
                                    lv2[u][c] = __ldcg(ps + c * PS + D + 1);
#pragma unroll
                                    for (int i = 0; i < PER; ++i) ov[u][c][i] = __ldcg(ps + c * PS + lane + 32 * i);
                                    if (!have) mv[u][c] = -INFINITY;
                                }
                            }
#pragma unroll
                            for (int c = 0; c < GC; ++c) {
                                const float Mn = fmaxf(M[c], fmaxf(mv[0][c], mv[1][c]));
                                const float f_old = exp2_or_zero(M[c], Mn), f0 = exp2_or_zero(mv[0][c], Mn), f1 = exp2_or_zero(mv[1][c], Mn);
                                L[c] = L[c] * f_old + lv2[0][c] * f0 + lv2[1][c] * f1;
#pragma unroll
                                for (int i = 0; i < PER; ++i) O[c][i] = O[c][i] * f_old + ov[0][c][i] * f0 + ov[1][c][i] * f1;
                                M[c] = Mn;
                            }
                        }
#pragma unroll
                        for (int c = 0; c < GC; ++c) {
                            const float inv = L[c] > 0.f ? 1.f / L[c] : 0.f;
#pragma unroll
                            for (int i = 0; i < PER; ++i)
                                outp[out_base + (size_t)(g0 + c) * D + lane + 32 * i] = __float2bfloat16_rn(O[c][i] * inv);
                        }
                    }
                    if (lane == 0) a.tickets[unit] = 0;
                }
            }
        }
        if (!ok && lane == 0) atomicOr(lv.status, kStWaitLimit);
    }

    // ---- a role gave up: let the copies still in flight land before the shared memory is released
    __syncthreads();
    if (*abort_flag && threadIdx.x == 0) {
        for (int s = 0; s < NS && s < n_tiles; ++s) {
            const int j_last = s + (n_tiles - 1 - s) / NS * NS;  // last tile that may have been sent to stage s
            const long long t0 = clock64();
            while (!mbar_try_wait(bar_full + s * 8, (uint32_t)((j_last / NS) & 1)) && clock64() - t0 < 200000000LL) {}
        }
    }
}

}  // namespace lar
