// Cache append (Eq. 4, prefill of Sec. 3.1) and the line-boundary step (Sec. 3.3, Eq. 5-10):
// score the mid region with the finished line's queries, drop the n least salient entries per unit,
// compact K, V and the index map in place.
#pragma once
#include "common.cuh"
#include "decode_attn.cuh"  // warp_max / warp_sum

namespace lar {

// ------------------------------------------------------------------------------------- append
// One CTA per unit copies n_tokens rows of k and v ([units][n_tokens][d]) behind the live entries.
template <typename T, int D>
__global__ void __launch_bounds__(128) append_kernel(const LayerView lv, const T* __restrict__ k,
                                                     const T* __restrict__ v, int n_tokens, int is_prefix) {
    constexpr int ROW_BYTES = D * (int)sizeof(T);
    constexpr int CHUNKS = ROW_BYTES / 16;
    grid_dep_wait();
    grid_dep_launch();
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
// Shared memory of line_end_kernel (bytes), M mid keys, W warps.
__host__ __device__ inline int line_end_smem_bytes(int row_bytes, int D, int M, int total_rows, int warps) {
    int b = M * (row_bytes + 16);          // mid keys, rows padded by one chunk against bank conflicts
    b += warps * (D + 2 * M) * 4;          // per warp: query row (fp32), logits row, score accumulator
    b += M * 4;                            // final scores
    b += ((M + 3) / 4) * 4;                // keep flags
    b += total_rows * 4;                   // source slot of every surviving row
    return (b + 15) / 16 * 16 + 16;
}

// One CTA per unit.  CUDA-core version: every lane owns the keys m = lane, lane + 32, ... and computes
// whole dot products against a query row broadcast from shared memory.
template <typename T, int D, int G>
__global__ void __launch_bounds__(256) line_end_kernel(const LayerView lv, float scale_log2) {
    constexpr int EPL = Elt<T>::kPerChunk;
    constexpr int ROW_BYTES = D * (int)sizeof(T);
    constexpr int CHUNKS = ROW_BYTES / 16;
    constexpr int KROW = ROW_BYTES + 16;
    extern __shared__ __align__(128) unsigned char smem[];
    grid_dep_wait();
    grid_dep_launch();

    const int unit = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, W = blockDim.x >> 5;
    const UnitState st = lv.state[unit];
    const int C = lv.cond_len, n = lv.line_width, B = lv.budget_tokens;
    const int v = st.len - C;
    if (st.n_tok == 0 || st.n_tok % n != 0 || v > B) {
        if (tid == 0) atomicOr(lv.status, kStBoundary);
        return;
    }
    if (v < B) return;  // cache below budget: nothing to evict (the queue restarts by itself)

    const int mid0 = C + lv.anchor_len;                       // first mid slot
    const int M = B - lv.anchor_len - lv.recent_lines * n;    // mid entries
    const int n_rec = lv.recent_lines * n;
    const int n_keep = M - n;
    const int total_rows = n_keep + n_rec;                    // rows behind the anchor after compaction
    const int nq = n * G;

    unsigned char* kmid = smem;
    float* wbuf = reinterpret_cast<float*>(smem + (size_t)M * KROW);
    float* qrow = wbuf + warp * (D + 2 * M);
    float* logit = qrow + D;
    float* sacc = logit + M;
    float* S = wbuf + W * (D + 2 * M);
    unsigned char* keep = reinterpret_cast<unsigned char*>(S + M);
    int* srcmap = reinterpret_cast<int*>(keep + ((M + 3) / 4) * 4);

    // ---- stage the mid keys
    for (int idx = tid; idx < M * CHUNKS; idx += blockDim.x) {
        const int r = idx / CHUNKS, c = idx - r * CHUNKS;
        const size_t off = row_offset(lv, unit, mid0 + r, ROW_BYTES) + c * 16;
        *reinterpret_cast<uint4*>(kmid + r * KROW + c * 16) = *reinterpret_cast<const uint4*>(lv.k_pool + off);
    }
    for (int mm = lane; mm < M; mm += 32) sacc[mm] = 0.f;
    __syncthreads();

    // ---- Eq. 9: every guide row is soft-maxed over the M mid keys; rows are summed per key
    const T* gq = reinterpret_cast<const T*>(lv.guide) + (size_t)unit * nq * D;
    for (int j = warp; j < nq; j += W) {
        for (int c = lane; c < CHUNKS; c += 32) {
            const uint4 raw = *reinterpret_cast<const uint4*>(gq + (size_t)j * D + c * EPL);
            float f[EPL];
            Elt<T>::unpack(raw, f);
#pragma unroll
            for (int e = 0; e < EPL; ++e) qrow[c * EPL + e] = f[e] * scale_log2;
        }
        __syncwarp();
        float mx = -INFINITY;
        for (int mm = lane; mm < M; mm += 32) {
            const unsigned char* kr = kmid + mm * KROW;
            float acc = 0.f;
#pragma unroll 4
            for (int c = 0; c < CHUNKS; ++c) {
                float kf[EPL];
                Elt<T>::unpack(*reinterpret_cast<const uint4*>(kr + c * 16), kf);
#pragma unroll
                for (int e = 0; e < EPL; ++e) acc = fmaf(qrow[c * EPL + e], kf[e], acc);
            }
            logit[mm] = acc;
            mx = fmaxf(mx, acc);
        }
        mx = warp_max(mx);
        float sum = 0.f;
        for (int mm = lane; mm < M; mm += 32) {
            const float p = exp2f(logit[mm] - mx);
            logit[mm] = p;
            sum += p;
        }
        sum = warp_sum(sum);
        const float inv = 1.f / sum;
        for (int mm = lane; mm < M; mm += 32) sacc[mm] = fmaf(logit[mm], inv, sacc[mm]);
        __syncwarp();
    }
    __syncthreads();
    const float inv_nq = 1.f / (float)nq;
    for (int mm = tid; mm < M; mm += blockDim.x) {
        float s = 0.f;
        for (int w = 0; w < W; ++w) s += wbuf[w * (D + 2 * M) + D + M + mm];
        s *= inv_nq;
        S[mm] = s;
        lv.scores[(size_t)unit * lv.mid_pad + mm] = s;
    }
    __syncthreads();

    // ---- Eq. 10: keep the M - n most salient; equal scores keep the lower slot (older token)
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

    // ---- Eq. 5-6: source slot (relative to mid0) of every row behind the anchor after compaction
    if (warp == 0) {
        int base = 0;
        for (int m0 = 0; m0 < M; m0 += 32) {
            const int mm = m0 + lane;
            const bool kp = mm < M && keep[mm];
            const unsigned bal = __ballot_sync(0xffffffffu, kp);
            if (kp) srcmap[base + __popc(bal & ((1u << lane) - 1u))] = mm;
            base += __popc(bal);
        }
    }
    for (int j = tid; j < n_rec; j += blockDim.x) srcmap[n_keep + j] = M + j;
    __syncthreads();

    // rows move towards lower slots only (src >= dst); tiles ascending, load - barrier - store
    constexpr int TILE_ROWS = 32;
    int* imap = lv.index_map + (size_t)unit * lv.cap_pad;
    for (int t0 = 0; t0 < total_rows; t0 += TILE_ROWS) {
        const int rows = min(TILE_ROWS, total_rows - t0);
        uint4 kbuf[(TILE_ROWS * CHUNKS + 255) / 256], vbuf[(TILE_ROWS * CHUNKS + 255) / 256];
        int ibuf = 0;
#pragma unroll
        for (int i = 0; i < (TILE_ROWS * CHUNKS + 255) / 256; ++i) {
            const int idx = tid + i * 256;
            const int r = idx / CHUNKS, c = idx - r * CHUNKS;
            if (idx < rows * CHUNKS && (int)blockDim.x == 256) {
                const int src = srcmap[t0 + r];
                if (src != t0 + r) {
                    const size_t off = row_offset(lv, unit, mid0 + src, ROW_BYTES) + c * 16;
                    kbuf[i] = *reinterpret_cast<const uint4*>(lv.k_pool + off);
                    vbuf[i] = *reinterpret_cast<const uint4*>(lv.v_pool + off);
                }
            }
        }
        if (tid < rows) ibuf = imap[mid0 + srcmap[t0 + tid]];
        __syncthreads();
#pragma unroll
        for (int i = 0; i < (TILE_ROWS * CHUNKS + 255) / 256; ++i) {
            const int idx = tid + i * 256;
            const int r = idx / CHUNKS, c = idx - r * CHUNKS;
            if (idx < rows * CHUNKS && (int)blockDim.x == 256) {
                if (srcmap[t0 + r] != t0 + r) {
                    const size_t off = row_offset(lv, unit, mid0 + t0 + r, ROW_BYTES) + c * 16;
                    *reinterpret_cast<uint4*>(lv.k_pool + off) = kbuf[i];
                    *reinterpret_cast<uint4*>(lv.v_pool + off) = vbuf[i];
                }
            }
        }
        if (tid < rows) imap[mid0 + t0 + tid] = ibuf;
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
