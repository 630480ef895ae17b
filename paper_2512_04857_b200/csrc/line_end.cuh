// Cache append (Eq. 4, prefill of Sec. 3.1) and the line-boundary step (Sec. 3.3, Eq. 5-10):
// score the mid region with the finished line's queries, drop the n least salient entries per unit,
// compact K, V and the index map in place.
#pragma once
#include "common.cuh"
#include "decode_attn.cuh"    // warp_max / warp_sum
#include "decode_stream.cuh"  // ldmatrix / mma wrappers

namespace lar {

// ------------------------------------------------------------------------------------- append
// One CTA per unit copies n_tokens rows of k and v ([units][n_tokens][d]) behind the live entries.
template <typename T, int D>
__global__ void __launch_bounds__(128) append_kernel(const LayerView lv, const T* __restrict__ k,
                                                     const T* __restrict__ v, int n_tokens, int is_prefix) {
    constexpr int ROW_BYTES = D * (int)sizeof(T);
    constexpr int CHUNKS = ROW_BYTES / 16;
    // No early release of dependents: a decode kernel launched behind this one may read the cache as soon as it is
    // scheduled, so it must not be scheduled before this grid has completed.
    grid_dep_wait();
    const int unit = blockIdx.x;
    const UnitState st = lv.state[unit];
    const int room = lv.cap - st.len;
    const int take = n_tokens < room ? n_tokens : room;
    const char* ksrc = reinterpret_cast<const char*>(k) + (size_t)unit * n_tokens * ROW_BYTES;
    const char* vsrc = reinterpret_cast<const char*>(v) + (size_t)unit * n_tokens * ROW_BYTES;
    for (int idx = threadIdx.x; idx < take * CHUNKS; idx += blockDim.x) {
        const int t = idx / CHUNKS, c = idx - t * CHUNKS;
        const size_t off = row_offset(lv, unit, st.len + t, ROW_BYTES) + c * 16;
        *reinterpret_cast<uint4*>(lv.k_pool + off) = *reinterpret_cast<const uint4*>(ksrc + (size_t)t * ROW_BYTES + c * 16);
        *reinterpret_cast<uint4*>(lv.v_pool + off) = *reinterpret_cast<const uint4*>(vsrc + (size_t)t * ROW_BYTES + c * 16);
    }
    for (int t = threadIdx.x; t < take; t += blockDim.x)
        lv.index_map[(size_t)unit * lv.cap_pad + st.len + t] = is_prefix ? st.len + t : lv.cond_len + st.n_tok + t;
    __syncthreads();
    if (threadIdx.x == 0) {
        UnitState ns;
        ns.len = st.len + take;
        ns.n_tok = st.n_tok + (is_prefix ? 0 : n_tokens);
        lv.state[unit] = ns;
        if (take < n_tokens) atomicOr(lv.status, kStCapacity);
    }
}

// ------------------------------------------------------------------------------------- line end
// Shared memory of line_end_kernel (bytes): M mid keys, nq = n * G guide rows, W warps.
// bf16 (tensor-core scoring): the guide rows are staged next to the keys; fp32: per-warp row buffers.
// cache_norm (the softmax of Eq. 9 taken over the whole live cache): all live_rows = C + B keys are staged, plus one
// cleared 8-key tile behind them; the bf16 path then reads the guide rows straight from global memory.
__host__ __device__ inline int line_end_staged_rows(int M, int live_rows, int cache_norm) {
    return cache_norm ? (live_rows + 7) / 8 * 8 + 8 : (M + 7) / 8 * 8;
}
// accum (attention accumulated over all history; implies cache_norm): the column sums cover every live row, not only
// the mid ones.
// reuse (the evicted slots are refilled, nothing is compacted): the mid entries are found through the index map; their
// slots and a bitmap of the mid positions (n_visual bits, with word-wise prefix counts) are kept in shared memory as well.
__host__ __device__ inline int line_end_smem_bytes(int row_bytes, int D, int M, int total_rows, int warps, int nq, int is_bf16,
                                                   int live_rows, int cache_norm, int accum, int reuse, int n_visual,
                                                   int guide_global = 0) {
    const int cols = (accum || (reuse && cache_norm)) ? live_rows : M;  // columns whose probabilities are summed
    int b = line_end_staged_rows(M, live_rows, cache_norm) * (row_bytes + 16);  // keys, rows padded by one chunk against bank conflicts
    if (is_bf16)
        b += ((cache_norm || guide_global) ? 0 : ((nq + 15) / 16 * 16) * (row_bytes + 16)) + warps * cols * 4;  // guide rows (whole 16-row tiles), column sums per warp
    else
        b += warps * (D + (cache_norm ? live_rows : M) + cols) * 4;  // per warp: query row (fp32), logits row, score accumulator
    b += M * 4;                            // final scores
    b += ((M + 3) / 4) * 4;                // keep flags
    b += total_rows * 4;                   // source slot of every surviving row
    if (reuse) b += (M + 2 * ((n_visual + 31) / 32)) * 4;  // slots of the mid entries, bitmap of mid positions + prefix counts
    return (b + 15) / 16 * 16 + 16;
}

// Eq. 9 on tensor cores (bf16).  keys: staged key rows of KROW bytes, colsum: [W][M] zeroed, one row per warp (summed
// in a fixed order afterwards: the scores, and with them the kept sets, are reproducible from run to run).  Every warp
// takes 16-row blocks of guide rows; a block's logits are formed twice with mma.sync m16n8k16 -- once for the row
// maxima and sums, once more to add the normalised probabilities into the column sums -- which is cheaper than
// keeping a [16][M] tile of logits anywhere.
//   CACHE = false: the rows are normalised over the M mid keys (keys = those M rows; guide rows staged at qg).
//   CACHE = true:  keys holds all n_keys live rows, the mid ones from row mid_off; guide row (t, g) is normalised over
//                  the keys that were live when token t of the line was decoded (rows < n_keys - n + t + 1) and read
//                  from global memory (gq32: rows of D / 2 words).
template <int D, bool CACHE, bool GQ_GLOBAL = CACHE>
__device__ __forceinline__ void score_mma(const unsigned char* keys, const unsigned char* qg, const uint32_t* gq32, float* colsum,
                                          int n_keys, int mid_off, int M, int nq, int G, int n, float scale_log2, int warp,
                                          int lane, int W) {
    constexpr int KROW = D * 2 + 16;
    constexpr int KSTEPS = D / 16;
    const int quad = lane & 3, grow = lane >> 2;
    const uint32_t kbase = smem_u32(keys), qbase = smem_u32(qg);
    for (int rb = warp; rb * 16 < nq; rb += W) {
        const int r0 = rb * 16 + grow, r1 = r0 + 8;
        uint32_t a[KSTEPS][4];
#pragma unroll
        for (int ks = 0; ks < KSTEPS; ++ks) {
            if constexpr (GQ_GLOBAL) {
                a[ks][0] = r0 < nq ? __ldg(gq32 + (size_t)r0 * (D / 2) + ks * 8 + quad) : 0u;
                a[ks][1] = r1 < nq ? __ldg(gq32 + (size_t)r1 * (D / 2) + ks * 8 + quad) : 0u;
                a[ks][2] = r0 < nq ? __ldg(gq32 + (size_t)r0 * (D / 2) + ks * 8 + 4 + quad) : 0u;
                a[ks][3] = r1 < nq ? __ldg(gq32 + (size_t)r1 * (D / 2) + ks * 8 + 4 + quad) : 0u;
            } else {
                ldmatrix_x4(qbase + (uint32_t)((rb * 16 + (lane & 15)) * KROW + (2 * ks + (lane >> 4)) * 16), a[ks]);
            }
        }
        // logits of the block against the 8 keys from staged row `row0`, scaled; this thread: keys 2 quad, 2 quad + 1
        auto logits = [&](int row0, float (&c)[4]) {
            c[0] = c[1] = c[2] = c[3] = 0.f;
#pragma unroll
            for (int i = 0; i < KSTEPS / 2; ++i) {
                uint32_t b[4];
                ldmatrix_x4(kbase + (uint32_t)((row0 + (lane & 7)) * KROW + (4 * i + (lane >> 3)) * 16), b);
                mma_bf16(c, a[2 * i][0], a[2 * i][1], a[2 * i][2], a[2 * i][3], b[0], b[1]);
                mma_bf16(c, a[2 * i + 1][0], a[2 * i + 1][1], a[2 * i + 1][2], a[2 * i + 1][3], b[2], b[3]);
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) c[i] *= scale_log2;
        };
        // keys every row of this thread is normalised over
        int lim0 = n_keys, lim1 = n_keys;
        if constexpr (CACHE) {
            lim0 = min(n_keys, n_keys - n + r0 / G + 1);
            lim1 = min(n_keys, n_keys - n + r1 / G + 1);
        }
        // pass 1: maximum and sum of every row (rows grow and grow + 8 of the block; this thread's columns first);
        // a thread that has seen no key of a row yet keeps (-inf, 0) -- the reference point 0 avoids inf - inf
        float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
        for (int k0 = 0; k0 < n_keys; k0 += 8) {
            float c[4];
            logits(k0, c);
            const int key = k0 + 2 * quad;
            c[0] = key < lim0 ? c[0] : -INFINITY;
            c[1] = key + 1 < lim0 ? c[1] : -INFINITY;
            c[2] = key < lim1 ? c[2] : -INFINITY;
            c[3] = key + 1 < lim1 ? c[3] : -INFINITY;
            const float n0 = fmaxf(m0, fmaxf(c[0], c[1])), n1 = fmaxf(m1, fmaxf(c[2], c[3]));
            const float f0 = n0 == -INFINITY ? 0.f : n0, f1 = n1 == -INFINITY ? 0.f : n1;
            l0 = l0 * exp2f(m0 - f0) + exp2f(c[0] - f0) + exp2f(c[1] - f0);
            l1 = l1 * exp2f(m1 - f1) + exp2f(c[2] - f1) + exp2f(c[3] - f1);
            m0 = n0;
            m1 = n1;
        }
#pragma unroll
        for (int off = 1; off <= 2; off <<= 1) {
            const float om0 = __shfl_xor_sync(0xffffffffu, m0, off), ol0 = __shfl_xor_sync(0xffffffffu, l0, off);
            const float om1 = __shfl_xor_sync(0xffffffffu, m1, off), ol1 = __shfl_xor_sync(0xffffffffu, l1, off);
            const float n0 = fmaxf(m0, om0), n1 = fmaxf(m1, om1);
            const float f0 = n0 == -INFINITY ? 0.f : n0, f1 = n1 == -INFINITY ? 0.f : n1;
            l0 = l0 * exp2f(m0 - f0) + ol0 * exp2f(om0 - f0);
            l1 = l1 * exp2f(m1 - f1) + ol1 * exp2f(om1 - f1);
            m0 = n0;
            m1 = n1;
        }
        // rows beyond the queue (the last block may be ragged) carry no weight
        const float w0 = r0 < nq ? 1.f / l0 : 0.f, w1 = r1 < nq ? 1.f / l1 : 0.f;
        // pass 2: probabilities of the mid keys, summed over the block's rows, into the column sums
        for (int k0 = 0; k0 < M; k0 += 8) {
            float c[4];
            logits(mid_off + k0, c);
            // (a column may be a token of the line itself: a row gives it mass only if it was live for that row)
            const int key = mid_off + k0 + 2 * quad;
            float v0 = (w0 != 0.f && key < lim0 ? exp2f(c[0] - m0) * w0 : 0.f) + (w1 != 0.f && key < lim1 ? exp2f(c[2] - m1) * w1 : 0.f);
            float v1 = (w0 != 0.f && key + 1 < lim0 ? exp2f(c[1] - m0) * w0 : 0.f) + (w1 != 0.f && key + 1 < lim1 ? exp2f(c[3] - m1) * w1 : 0.f);
#pragma unroll
            for (int off = 4; off <= 16; off <<= 1) {
                v0 += __shfl_xor_sync(0xffffffffu, v0, off);
                v1 += __shfl_xor_sync(0xffffffffu, v1, off);
            }
            if (grow == 0) {  // lanes 0..3 own two keys each of this tile in the warp's row of column sums
                const int col = k0 + 2 * quad;
                float* mine = colsum + warp * M;
                if (col < M) mine[col] += v0;
                if (col + 1 < M) mine[col + 1] += v1;
            }
        }
    }
}

// One CTA per unit; blockIdx.y counts layers from the one `lv0` describes (a grid may span all layers of a cache:
// they are independent).  cache_norm != 0 selects the variant of Eq. 9 whose softmax runs over the whole live cache
// (every guide query over the entries that were live when it was decoded).  Scoring: bf16 on tensor cores (score_mma); fp32 on CUDA cores, where every lane owns the keys
// m = lane, lane + 32, ... and computes whole dot products against a query row broadcast from shared memory.
template <typename T, int D, int G>
__global__ void __launch_bounds__(1024) line_end_kernel(const LayerView lv0, const LayerStrides ls, float scale_log2, int mode) {
    constexpr int EPL = Elt<T>::kPerChunk;
    constexpr int ROW_BYTES = D * (int)sizeof(T);
    constexpr int CHUNKS = ROW_BYTES / 16;
    constexpr int KROW = ROW_BYTES + 16;
    extern __shared__ __align__(128) unsigned char smem[];
    // (no early release of dependents, as in append_kernel: rows move until the very end)
    grid_dep_wait();

    const LayerView lv = layer_view_at(lv0, ls, (int)blockIdx.y);
    const int unit = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, W = blockDim.x >> 5;
    const UnitState st = lv.state[unit];
    const int C = lv.cond_len, n = lv.line_width, B = lv.budget_tokens;
    const int v = st.len - C;
    if (st.n_tok == 0 || st.n_tok % n != 0 || v > B) {
        if (tid == 0) atomicOr(lv.status, kStBoundary);
        return;
    }
    // mode bit 0: softmax of Eq. 9 over the whole live cache; bit 1: rank by the attention accumulated over all decode
    // steps (the per-line sums of the cache-normalised form, added up line by line in lv.acc)
    // bit 2: no compaction -- the n evicted slots take the n rows of the newest line (n rows move instead of every row
    // behind the first hole); slots then no longer follow positions, and the mid region is found through the index map
    // bit 3: the guide rows are not staged in shared memory (a mid region too large to stage both): read from global
    const bool accum = (mode & 2) != 0, reuse = (mode & 4) != 0, guide_global = (mode & 8) != 0;
    const int cache_norm = (mode & 1) | (accum ? 1 : 0);
    const bool compress = v == B;
    if (!compress && !accum) return;  // cache below budget: nothing to evict (the queue restarts by itself)

    const int mid0 = C + lv.anchor_len;                       // first mid slot
    const int M = B - lv.anchor_len - lv.recent_lines * n;    // mid entries
    const int n_rec = lv.recent_lines * n;
    const int n_keep = M - n;
    const int total_rows = n_keep + n_rec;                    // rows behind the anchor after compaction
    const int nq = n * G;

    constexpr bool kMma = sizeof(T) == 2;  // bf16: tensor-core scoring; fp32: CUDA cores
    const int nq16 = (nq + 15) / 16 * 16;
    const int stage0 = cache_norm ? 0 : mid0;          // first staged slot
    const int n_stage = cache_norm ? st.len : M;       // staged keys
    const int mid_off = mid0 - stage0;                 // staged row of the first mid key
    const int rows_pad = line_end_staged_rows(M, st.len, cache_norm);
    unsigned char* kst = smem;
    unsigned char* after_k = smem + (size_t)rows_pad * KROW;
    unsigned char* qg = after_k;                                                // [nq16][KROW]   (bf16, mid-only scoring)
    // columns whose probabilities are summed: the M mid keys, or (accum) every staged row
    const bool all_cols = accum || (reuse && cache_norm);
    const int cols = all_cols ? n_stage : M, col_off = all_cols ? 0 : mid_off;
    float* colsum = reinterpret_cast<float*>(after_k + ((cache_norm || guide_global) ? (size_t)0 : (size_t)nq16 * KROW));  // [W][cols] (bf16)
    const int wstride = D + n_stage + cols;
    float* wbuf = reinterpret_cast<float*>(after_k);                            // [W][D + n_stage + cols]   (fp32)
    float* S = kMma ? colsum + W * cols : wbuf + W * wstride;
    unsigned char* keep = reinterpret_cast<unsigned char*>(S + M);
    int* srcmap = reinterpret_cast<int*>(keep + ((M + 3) / 4) * 4);
    int* mid_slot = srcmap + total_rows;  // [M]   (reuse) slot of the mid entries, in ascending original position
    unsigned* pos_bits = reinterpret_cast<unsigned*>(mid_slot + M);  // (reuse) bit p - lo_pos: a live entry has mid position p
    int* imap = lv.index_map + (size_t)unit * lv.cap_pad;

    if (reuse && compress) {
        // ---- the mid region by position (Sec. 3.3): visual index in (N_init, (l - r) n].  The live mid positions are
        // marked in a bitmap; an entry's place in ascending position is the number of marked bits below its own.
        const int lo_pos = C + lv.anchor_len, hi_pos = C + (st.n_tok / n - lv.recent_lines) * n;  // mid: lo_pos <= pos < hi_pos
        const int n_words = (hi_pos - lo_pos + 31) / 32;
        int* below = reinterpret_cast<int*>(pos_bits + n_words);   // marked bits in the words before this one
        for (int i = tid; i < n_words; i += blockDim.x) pos_bits[i] = 0u;
        __syncthreads();
        for (int sl = C + tid; sl < st.len; sl += blockDim.x) {
            const int p = imap[sl];
            if (p >= lo_pos && p < hi_pos) atomicOr(&pos_bits[(p - lo_pos) >> 5], 1u << ((p - lo_pos) & 31));
        }
        __syncthreads();
        if (warp == 0) {
            int run = 0;
            for (int i0 = 0; i0 < n_words; i0 += 32) {
                const int cnt = i0 + lane < n_words ? __popc(pos_bits[i0 + lane]) : 0;
                int inc = cnt;
#pragma unroll
                for (int off = 1; off < 32; off <<= 1) {
                    const int t = __shfl_up_sync(0xffffffffu, inc, off);
                    if (lane >= off) inc += t;
                }
                if (i0 + lane < n_words) below[i0 + lane] = run + inc - cnt;
                run += __shfl_sync(0xffffffffu, inc, 31);
            }
            if (lane == 0 && run != M) atomicOr(lv.status, kStBoundary);  // not exactly M mid entries: the index map is damaged
        }
        __syncthreads();
        for (int sl = C + tid; sl < st.len; sl += blockDim.x) {
            const int p = imap[sl];
            if (p >= lo_pos && p < hi_pos) {
                const int w = (p - lo_pos) >> 5, bit = (p - lo_pos) & 31;
                const int rank = below[w] + __popc(pos_bits[w] & ((1u << bit) - 1u));
                if (rank < M) mid_slot[rank] = sl;
            }
        }
        __syncthreads();
    }

    // ---- stage the keys (rows behind the last one are cleared)
    for (int idx = tid; idx < rows_pad * CHUNKS; idx += blockDim.x) {
        const int r = idx / CHUNKS, c = idx - r * CHUNKS;
        uint4 val = make_uint4(0u, 0u, 0u, 0u);
        if (r < n_stage) {
            const int sl = (reuse && !cache_norm) ? mid_slot[r] : stage0 + r;
            val = *reinterpret_cast<const uint4*>(lv.k_pool + row_offset(lv, unit, sl, ROW_BYTES) + c * 16);
        }
        *reinterpret_cast<uint4*>(kst + r * KROW + c * 16) = val;
    }
    const T* gq = reinterpret_cast<const T*>(lv.guide) + (size_t)unit * nq * D;
    if constexpr (kMma) {
        // ---- Eq. 9 on tensor cores: stage the guide rows (mid-only scoring), clear the column sums
        if (!cache_norm && !guide_global) {
            for (int idx = tid; idx < nq16 * CHUNKS; idx += blockDim.x) {
                const int r = idx / CHUNKS, c = idx - r * CHUNKS;
                uint4 val = make_uint4(0u, 0u, 0u, 0u);
                if (r < nq) val = *reinterpret_cast<const uint4*>(reinterpret_cast<const unsigned char*>(gq) + (size_t)r * ROW_BYTES + c * 16);
                *reinterpret_cast<uint4*>(qg + r * KROW + c * 16) = val;
            }
        }
        for (int mm = tid; mm < W * cols; mm += blockDim.x) colsum[mm] = 0.f;
        __syncthreads();
        if (cache_norm)
            score_mma<D, true>(kst, qg, reinterpret_cast<const uint32_t*>(gq), colsum, n_stage, col_off, cols, nq, G, n, scale_log2, warp, lane, W);
        else if (guide_global)
            score_mma<D, false, true>(kst, qg, reinterpret_cast<const uint32_t*>(gq), colsum, n_stage, col_off, cols, nq, G, n, scale_log2, warp, lane, W);
        else
            score_mma<D, false>(kst, qg, nullptr, colsum, n_stage, col_off, cols, nq, G, n, scale_log2, warp, lane, W);
        __syncthreads();
    } else {
        // ---- Eq. 9 on CUDA cores: every guide row is soft-maxed over its keys (the M mid keys, or the entries that
        // were live when its token was decoded); the mid columns of the rows are summed per key
        float* qrow = wbuf + warp * wstride;
        float* logit = qrow + D;
        float* sacc = logit + n_stage;
        for (int mm = lane; mm < cols; mm += 32) sacc[mm] = 0.f;
        __syncthreads();
        for (int j = warp; j < nq; j += W) {
            for (int c = lane; c < CHUNKS; c += 32) {
                const uint4 raw = *reinterpret_cast<const uint4*>(gq + (size_t)j * D + c * EPL);
                float f[EPL];
                Elt<T>::unpack(raw, f);
#pragma unroll
                for (int e = 0; e < EPL; ++e) qrow[c * EPL + e] = f[e] * scale_log2;
            }
            __syncwarp();
            const int lim = cache_norm ? n_stage - n + j / G + 1 : n_stage;
            float mx = -INFINITY;
            for (int kk = lane; kk < lim; kk += 32) {
                const unsigned char* kr = kst + kk * KROW;
                float acc = 0.f;
#pragma unroll 4
                for (int c = 0; c < CHUNKS; ++c) {
                    float kf[EPL];
                    Elt<T>::unpack(*reinterpret_cast<const uint4*>(kr + c * 16), kf);
#pragma unroll
                    for (int e = 0; e < EPL; ++e) acc = fmaf(qrow[c * EPL + e], kf[e], acc);
                }
                logit[kk] = acc;
                mx = fmaxf(mx, acc);
            }
            mx = warp_max(mx);
            float sum = 0.f;
            for (int kk = lane; kk < lim; kk += 32) {
                const float p = exp2f(logit[kk] - mx);
                logit[kk] = p;
                sum += p;
            }
            sum = warp_sum(sum);
            const float inv = 1.f / sum;
            __syncwarp();
            for (int mm = lane; mm < cols && col_off + mm < lim; mm += 32) sacc[mm] = fmaf(logit[col_off + mm], inv, sacc[mm]);
            __syncwarp();
        }
        __syncthreads();
    }
    // ---- the line's score of every column: the warps' sums added in a fixed order (reproducible kept sets)
    {
        const float* wsum = kMma ? colsum : wbuf + D + n_stage;
        const int wsum_stride = kMma ? cols : wstride;
        const float inv_nq = 1.f / (float)nq;
        if (!accum) {
            for (int mm = tid; mm < M; mm += blockDim.x) {
                const int col = all_cols ? mid_slot[mm] : mm;  // (all columns summed: pick the mid entry's slot)
                float sc = 0.f;
                for (int w = 0; w < W; ++w) sc += wsum[w * wsum_stride + col];
                sc *= inv_nq;
                S[mm] = sc;
                lv.scores[(size_t)unit * lv.mid_pad + mm] = sc;
            }
        } else {
            // every live slot adds the line's mass to what it had; the line's own tokens (the last n slots) start here
            float* acc = lv.acc + (size_t)unit * lv.cap_pad;
            for (int sl = tid; sl < n_stage; sl += blockDim.x) {
                float sc = 0.f;
                for (int w = 0; w < W; ++w) sc += wsum[w * wsum_stride + sl];
                sc *= inv_nq;
                acc[sl] = (sl >= n_stage - n ? 0.f : acc[sl]) + sc;
            }
            __syncthreads();
            if (compress) {
                for (int mm = tid; mm < M; mm += blockDim.x) {
                    const float total = acc[reuse ? mid_slot[mm] : mid0 + mm];
                    S[mm] = total;
                    lv.scores[(size_t)unit * lv.mid_pad + mm] = total;
                }
            }
        }
        __syncthreads();
    }
    if (!compress) return;  // (accumulated-attention scoring below budget: the sums are updated, nothing is evicted)

    // ---- Eq. 10: keep the M - n most salient; equal scores keep the lower slot (older token).
    // A score that is not finite (a NaN or Inf in a key or query) has no rank: it is treated as the lowest possible
    // score, which keeps the ranking a total order and the kept count at M - n, and the status word records it.
    for (int mm = tid; mm < M; mm += blockDim.x) {
        if (!isfinite(S[mm])) {
            S[mm] = -INFINITY;
            atomicOr(lv.status, kStNonFinite);
        }
    }
    __syncthreads();
    for (int mm = tid; mm < M; mm += blockDim.x) {
        const float s = S[mm];
        int rank = 0;
        for (int j = 0; j < M; ++j) {
            const float sj = S[j];
            rank += (sj > s || (sj == s && j < mm)) ? 1 : 0;
        }
        keep[mm] = rank < n_keep ? 1 : 0;
    }
    __syncthreads();

    if (reuse) {
        // ---- Eq. 5-7 without compaction: the n evicted slots take the n rows of the newest line (the last n slots; none
        // of them is a hole, since the last r >= 1 lines are never evicted), so the cache stays dense
        if (warp == 0) {
            int base = 0;
            for (int m0 = 0; m0 < M; m0 += 32) {
                const int mm = m0 + lane;
                const bool ev = mm < M && !keep[mm];
                const unsigned bal = __ballot_sync(0xffffffffu, ev);
                if (ev && base + __popc(bal & ((1u << lane) - 1u)) < n) srcmap[base + __popc(bal & ((1u << lane) - 1u))] = mid_slot[mm];
                base += __popc(bal);
            }
        }
        __syncthreads();
        const int tail0 = st.len - n;
        for (int idx = tid; idx < n * CHUNKS; idx += blockDim.x) {
            const int j = idx / CHUNKS, c = idx - j * CHUNKS;
            const size_t src = row_offset(lv, unit, tail0 + j, ROW_BYTES) + c * 16, dst = row_offset(lv, unit, srcmap[j], ROW_BYTES) + c * 16;
            *reinterpret_cast<uint4*>(lv.k_pool + dst) = *reinterpret_cast<const uint4*>(lv.k_pool + src);
            *reinterpret_cast<uint4*>(lv.v_pool + dst) = *reinterpret_cast<const uint4*>(lv.v_pool + src);
        }
        for (int j = tid; j < n; j += blockDim.x) {
            imap[srcmap[j]] = imap[tail0 + j];
            if (accum) lv.acc[(size_t)unit * lv.cap_pad + srcmap[j]] = lv.acc[(size_t)unit * lv.cap_pad + tail0 + j];
        }
        if (tid == 0) {
            UnitState ns;
            ns.len = st.len - n;
            ns.n_tok = st.n_tok;
            lv.state[unit] = ns;
        }
        return;
    }

    // ---- Eq. 5-6: source slot (relative to mid0) of every row behind the anchor after compaction
    if (warp == 0) {
        int base = 0;
        for (int m0 = 0; m0 < M; m0 += 32) {
            const int mm = m0 + lane;
            const bool kp = mm < M && keep[mm];
            const unsigned bal = __ballot_sync(0xffffffffu, kp);
            if (kp && base + __popc(bal & ((1u << lane) - 1u)) < n_keep) srcmap[base + __popc(bal & ((1u << lane) - 1u))] = mm;
            base += __popc(bal);
        }
    }
    for (int j = tid; j < n_rec; j += blockDim.x) srcmap[n_keep + j] = M + j;
    __syncthreads();

    // rows move towards lower slots only (src >= dst); tiles ascending, load - barrier - store;
    // every thread carries 4 chunks of K and 4 of V per tile (64 .. 256 rows per tile)
    constexpr int PER_THREAD = 4;
    const int nthr = (int)blockDim.x;
    const int tile_rows = nthr * PER_THREAD / CHUNKS;  // <= nthr
    for (int t0 = 0; t0 < total_rows; t0 += tile_rows) {
        const int rows = min(tile_rows, total_rows - t0);
        uint4 kbuf[PER_THREAD], vbuf[PER_THREAD];
        int ibuf = 0;
        float abuf = 0.f;
#pragma unroll
        for (int i = 0; i < PER_THREAD; ++i) {
            const int idx = tid + i * nthr;
            const int r = idx / CHUNKS, c = idx - r * CHUNKS;
            if (idx < rows * CHUNKS) {
                const int src = srcmap[t0 + r];
                if (src != t0 + r) {
                    const size_t off = row_offset(lv, unit, mid0 + src, ROW_BYTES) + c * 16;
                    kbuf[i] = *reinterpret_cast<const uint4*>(lv.k_pool + off);
                    vbuf[i] = *reinterpret_cast<const uint4*>(lv.v_pool + off);
                }
            }
        }
        if (tid < rows) {
            ibuf = imap[mid0 + srcmap[t0 + tid]];
            if (accum) abuf = lv.acc[(size_t)unit * lv.cap_pad + mid0 + srcmap[t0 + tid]];
        }
        __syncthreads();
#pragma unroll
        for (int i = 0; i < PER_THREAD; ++i) {
            const int idx = tid + i * nthr;
            const int r = idx / CHUNKS, c = idx - r * CHUNKS;
            if (idx < rows * CHUNKS) {
                if (srcmap[t0 + r] != t0 + r) {
                    const size_t off = row_offset(lv, unit, mid0 + t0 + r, ROW_BYTES) + c * 16;
                    *reinterpret_cast<uint4*>(lv.k_pool + off) = kbuf[i];
                    *reinterpret_cast<uint4*>(lv.v_pool + off) = vbuf[i];
                }
            }
        }
        if (tid < rows) {
            imap[mid0 + t0 + tid] = ibuf;
            if (accum) lv.acc[(size_t)unit * lv.cap_pad + mid0 + t0 + tid] = abuf;
        }
        __syncthreads();
    }
    if (tid == 0) {
        UnitState ns;
        ns.len = st.len - n;
        ns.n_tok = st.n_tok;
        lv.state[unit] = ns;
    }
}

}  // namespace lar
