// Decode attention over the paged, line-compressed cache (Eq. 2-3), optionally fused with the
// append of the new token (Eq. 4) and the guide-queue push (Eq. 8).
//
// One thread-block cluster of `splits` CTAs serves one unit = (sequence, KV head) and all G query
// heads that share it.  The live rows are cut into 16-row tiles; tile t belongs to CTA (t % splits),
// warp ((t / splits) % warps).  Every warp runs its own pipeline: lane 0 issues 1-D bulk async copies
// (TMA unit) of a K tile and a V tile into the warp's shared-memory stages and the warp waits on the
// stage's mbarrier, so no block-wide barrier sits in the main loop and each SM keeps
// warps * stages * 2 tiles in flight.  A row is spread over LPR = row_bytes / 16 lanes (one 16-byte
// chunk each); partial dot products are combined with a reduce-scatter of shuffles so that every
// lane ends up with one logit.  Softmax is online in fp32 (base-2 exponent, scale folded into q).
// Warp partials (m, l, o) are merged in shared memory; CTA partials of a cluster are pushed into
// CTA 0's shared memory (distributed shared memory) and merged there: no global scratch.
#pragma once
#include "common.cuh"

namespace lar {

struct DecodeArgs {
    LayerView lv;
    const void* q;      // [units * G][d]
    const void* k_new;  // [units][d]   (fused only)
    const void* v_new;
    void* out;          // [units * G][d]
    float scale_log2;   // softmax scale * log2(e)
    int fused;          // 1: rows [0, len) come from the cache and the new token from k_new / v_new
    int prefetch;       // 1: issue the first cache loads before waiting on the preceding kernel
    int splits;         // CTAs per unit (cluster size)
    int stages;         // tiles in flight per warp
};

template <typename T, int D>
struct DecodeTraits {
    static constexpr int EPL = Elt<T>::kPerChunk;      // elements per lane chunk
    static constexpr int LPR = D / EPL;                // lanes per row
    static constexpr int RPI = 32 / LPR;               // rows per warp iteration
    static constexpr int IT = kGranule / RPI;          // iterations per tile (= LPR / 2)
    static constexpr int ROW_BYTES = D * (int)sizeof(T);
    static constexpr int GRAN_BYTES = kGranule * ROW_BYTES;
    static constexpr int STAGE_BYTES = 2 * GRAN_BYTES;  // K tile + V tile
    static_assert(LPR == 8 || LPR == 16 || LPR == 32, "unsupported row size");
};

__host__ __device__ inline int decode_smem_bytes(int stage_bytes, int warps, int stages, int splits, int G, int D) {
    int b = warps * stages * stage_bytes;
    b += ((warps * stages * 8 + 15) / 16) * 16;
    b += warps * G * (D + 2) * 4;
    if (splits > 1) b += splits * G * (D + 2) * 4;
    return b;
}

// Sum `a[i]` over the LPR lanes of a row group; on return lane `sub` holds the total of entry
// (sub >> 1) (lanes 2t and 2t+1 both hold entry t).  LPR/2 + ... shuffles instead of IT * log2(LPR).
template <int LPR>
__device__ __forceinline__ float reduce_scatter(float (&a)[LPR / 2], int lane) {
#pragma unroll
    for (int off = LPR / 2; off >= 2; off >>= 1) {
        const int half = off / 2;
        const bool upper = (lane & off) != 0;
#pragma unroll
        for (int k = 0; k < half; ++k) {
            const float send = upper ? a[k] : a[k + half];
            const float keep = upper ? a[k + half] : a[k];
            a[k] = keep + __shfl_xor_sync(0xffffffffu, send, off);
        }
    }
    a[0] += __shfl_xor_sync(0xffffffffu, a[0], 1);
    return a[0];
}

__device__ __forceinline__ float warp_max(float x) {
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
    return x;
}
__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}
__device__ __forceinline__ float exp2_safe(float m_part, float m_all) {
    return m_part == -INFINITY ? 0.f : exp2f(m_part - m_all);
}

template <typename T, int D, int G>
__global__ void __launch_bounds__(256) decode_kernel(const DecodeArgs a) {
    using TR = DecodeTraits<T, D>;
    constexpr int EPL = TR::EPL, LPR = TR::LPR, RPI = TR::RPI, IT = TR::IT;
    extern __shared__ __align__(128) unsigned char smem[];

    const int W = blockDim.x >> 5, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int X = a.splits, NS = a.stages;
    const int rank = X > 1 ? (int)cluster_rank() : 0;
    const int unit = blockIdx.x / X;
    const LayerView& lv = a.lv;

    unsigned char* my_stages = smem + (size_t)warp * NS * TR::STAGE_BYTES;
    unsigned char* after = smem + (size_t)W * NS * TR::STAGE_BYTES;
    const uint32_t my_bars = smem_u32(after) + warp * NS * 8;
    after += ((W * NS * 8 + 15) / 16) * 16;
    float* part_o = reinterpret_cast<float*>(after);  // [W][G][D]
    float* part_ml = part_o + W * G * D;              // [W][G][2]
    float* cl_o = part_ml + W * G * 2;                // [X][G][D]   (clusters only)
    float* cl_ml = cl_o + X * G * D;                  // [X][G][2]

    // every CTA of the cluster must have started before its shared memory is written remotely:
    // arrive now, wait just before the first remote store
    if (X > 1) cluster_arrive();
    if (!a.prefetch) grid_dep_wait();

    if (lane == 0) {
        for (int s = 0; s < NS; ++s) mbar_init(my_bars + s * 8, 1);
        mbar_fence_init();
    }
    __syncwarp();

    const UnitState st = lv.state[unit];
    const int len_tma = st.len;  // rows read from the cache
    const int NG = (len_tma + kGranule - 1) / kGranule;
    const int first = rank + X * warp, stride = X * W;
    const int my_n = first < NG ? (NG - first + stride - 1) / stride : 0;

    auto issue = [&](int k) {
        const int g = first + k * stride, s = k % NS;
        const int row0 = g * kGranule;
        const int rows = min(kGranule, len_tma - row0);
        const uint32_t bytes = (uint32_t)rows * TR::ROW_BYTES;
        const size_t off = row_offset(lv, unit, row0, TR::ROW_BYTES);
        const uint32_t bar = my_bars + s * 8;
        const uint32_t dst = smem_u32(my_stages + (size_t)s * TR::STAGE_BYTES);
        mbar_expect_tx(bar, 2 * bytes);
        bulk_g2s(dst, lv.k_pool + off, bytes, bar);
        bulk_g2s(dst + TR::GRAN_BYTES, lv.v_pool + off, bytes, bar);
    };
    if (lane == 0) {
        const int pro = my_n < NS ? my_n : NS;
        for (int k = 0; k < pro; ++k) issue(k);
    }
    if (a.prefetch) grid_dep_wait();
    grid_dep_launch();

    // ---- queries of the G heads of this unit: this lane's 16-byte chunk, scale folded in
    const int sub = lane % LPR, grp = lane / LPR;
    const T* qbase = reinterpret_cast<const T*>(a.q) + (size_t)unit * G * D;
    uint4 qraw[G];
    float qf[G][EPL];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        qraw[g] = __ldg(reinterpret_cast<const uint4*>(qbase + g * D + sub * EPL));
        Elt<T>::unpack(qraw[g], qf[g]);
#pragma unroll
        for (int e = 0; e < EPL; ++e) qf[g][e] *= a.scale_log2;
    }

    float m[G], l[G], o[G][EPL];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        m[g] = -INFINITY;
        l[g] = 0.f;
#pragma unroll
        for (int e = 0; e < EPL; ++e) o[g][e] = 0.f;
    }

    bool ok = true;
    for (int k = 0; k < my_n; ++k) {
        const int s = k % NS;
        const bool arrived = mbar_wait_bounded(my_bars + s * 8, (uint32_t)((k / NS) & 1));
        if (!__all_sync(0xffffffffu, arrived)) { ok = false; break; }
        const int rows = min(kGranule, len_tma - (first + k * stride) * kGranule);
        const unsigned char* Ks = my_stages + (size_t)s * TR::STAGE_BYTES;
        const unsigned char* Vs = Ks + TR::GRAN_BYTES;

        // logits: partial dot products of this lane's chunk for the IT rows it touches
        float part[G][IT];
#pragma unroll
        for (int it = 0; it < IT; ++it) {
            const int row = it * RPI + grp;
            const uint4 c = *reinterpret_cast<const uint4*>(Ks + row * TR::ROW_BYTES + sub * 16);
            float kf[EPL];
            Elt<T>::unpack(c, kf);
#pragma unroll
            for (int g = 0; g < G; ++g) {
                float acc = 0.f;
#pragma unroll
                for (int e = 0; e < EPL; ++e) acc = fmaf(qf[g][e], kf[e], acc);
                part[g][it] = acc;
            }
        }
        const int my_row = (sub >> 1) * RPI + grp;  // row whose logit this lane holds after the reduce-scatter
        const bool my_valid = my_row < rows;
        float p[G];
#pragma unroll
        for (int g = 0; g < G; ++g) {
            float sv = reduce_scatter<LPR>(part[g], lane);
            sv = my_valid ? sv : -INFINITY;
            const float m_new = fmaxf(m[g], warp_max(sv));
            const float corr = exp2f(m[g] - m_new);
            p[g] = exp2f(sv - m_new);
            m[g] = m_new;
            l[g] = l[g] * corr + ((lane & 1) ? 0.f : p[g]);
#pragma unroll
            for (int e = 0; e < EPL; ++e) o[g][e] *= corr;
        }
        // o += p V
#pragma unroll
        for (int it = 0; it < IT; ++it) {
            const int row = it * RPI + grp;
            float pr[G];
#pragma unroll
            for (int g = 0; g < G; ++g) pr[g] = __shfl_sync(0xffffffffu, p[g], grp * LPR + 2 * it);
            if (row < rows) {
                const uint4 c = *reinterpret_cast<const uint4*>(Vs + row * TR::ROW_BYTES + sub * 16);
                float vf[EPL];
                Elt<T>::unpack(c, vf);
#pragma unroll
                for (int g = 0; g < G; ++g)
#pragma unroll
                    for (int e = 0; e < EPL; ++e) o[g][e] = fmaf(pr[g], vf[e], o[g][e]);
            }
        }
        __syncwarp();
        if (lane == 0 && k + NS < my_n) issue(k + NS);
    }
    if (!ok && lane == 0) atomicOr(lv.status, kStWaitLimit);

    // ---- the token of this step: attend to it from registers, store it, push q to the guide queue
    const int owner_rank = NG % X, owner_warp = (NG / X) % W;
    if (rank == owner_rank && warp == owner_warp) {
        if (a.fused) {
            const T* kn = reinterpret_cast<const T*>(a.k_new) + (size_t)unit * D + sub * EPL;
            const T* vn = reinterpret_cast<const T*>(a.v_new) + (size_t)unit * D + sub * EPL;
            const uint4 kc = __ldg(reinterpret_cast<const uint4*>(kn));
            const uint4 vc = __ldg(reinterpret_cast<const uint4*>(vn));
            float kf[EPL], vf[EPL];
            Elt<T>::unpack(kc, kf);
            Elt<T>::unpack(vc, vf);
#pragma unroll
            for (int g = 0; g < G; ++g) {
                float sv = 0.f;
#pragma unroll
                for (int e = 0; e < EPL; ++e) sv = fmaf(qf[g][e], kf[e], sv);
#pragma unroll
                for (int off = LPR / 2; off >= 1; off >>= 1) sv += __shfl_xor_sync(0xffffffffu, sv, off);
                const float m_new = fmaxf(m[g], sv);
                const float corr = exp2f(m[g] - m_new);
                const float pn = exp2f(sv - m_new);
                m[g] = m_new;
                l[g] = l[g] * corr + (lane == 0 ? pn : 0.f);
                const float pv = grp == 0 ? pn : 0.f;
#pragma unroll
                for (int e = 0; e < EPL; ++e) o[g][e] = fmaf(pv, vf[e], o[g][e] * corr);
            }
            if (st.len < lv.cap) {
                if (grp == 0) {
                    const size_t off = row_offset(lv, unit, st.len, TR::ROW_BYTES) + sub * 16;
                    *reinterpret_cast<uint4*>(lv.k_pool + off) = kc;
                    *reinterpret_cast<uint4*>(lv.v_pool + off) = vc;
                }
                if (lane == 0) lv.index_map[(size_t)unit * lv.cap_pad + st.len] = lv.cond_len + st.n_tok;
            } else if (lane == 0) {
                atomicOr(lv.status, kStCapacity);
            }
        } else if (len_tma == 0 && lane == 0) {
            atomicOr(lv.status, kStEmpty);
        }
        // Eq. 8: the query joins the guide queue of the line being generated
        const int tok = a.fused ? st.n_tok : st.n_tok - 1;  // 0-based visual index of this step's token
        if (tok >= 0 && grp == 0) {
            const int slot = tok % lv.line_width;
            T* gq = reinterpret_cast<T*>(lv.guide) + (((size_t)unit * lv.line_width + slot) * G) * D + sub * EPL;
#pragma unroll
            for (int g = 0; g < G; ++g) *reinterpret_cast<uint4*>(gq + g * D) = qraw[g];
        }
    }

    // ---- merge: lane groups -> warp, warps -> CTA, CTAs -> cluster
#pragma unroll
    for (int g = 0; g < G; ++g) {
#pragma unroll
        for (int off = LPR; off < 32; off <<= 1)
#pragma unroll
            for (int e = 0; e < EPL; ++e) o[g][e] += __shfl_xor_sync(0xffffffffu, o[g][e], off);
        l[g] = warp_sum(l[g]);
        if (grp == 0) {
#pragma unroll
            for (int e = 0; e < EPL; ++e) part_o[(warp * G + g) * D + sub * EPL + e] = o[g][e];
        }
        if (lane == 0) {
            part_ml[(warp * G + g) * 2 + 0] = m[g];
            part_ml[(warp * G + g) * 2 + 1] = l[g];
        }
    }
    __syncthreads();

    T* outp = reinterpret_cast<T*>(a.out) + (size_t)unit * G * D;
    if (X > 1) cluster_wait();
    for (int idx = threadIdx.x; idx < G * D; idx += blockDim.x) {
        const int g = idx / D, e = idx - g * D;
        float M = -INFINITY;
        for (int w = 0; w < W; ++w) M = fmaxf(M, part_ml[(w * G + g) * 2]);
        float L = 0.f, O = 0.f;
        for (int w = 0; w < W; ++w) {
            const float sc = exp2_safe(part_ml[(w * G + g) * 2], M);
            L = fmaf(part_ml[(w * G + g) * 2 + 1], sc, L);
            O = fmaf(part_o[(w * G + g) * D + e], sc, O);
        }
        if (X == 1) {
            outp[idx] = Elt<T>::from_float(O / L);
        } else {
            st_cluster_f32(map_to_rank(smem_u32(cl_o + (rank * G + g) * D + e), 0), O);
            if (e == 0) {
                st_cluster_f32(map_to_rank(smem_u32(cl_ml + (rank * G + g) * 2), 0), M);
                st_cluster_f32(map_to_rank(smem_u32(cl_ml + (rank * G + g) * 2 + 1), 0), L);
            }
        }
    }
    if (X > 1) {
        cluster_sync_all();
        if (rank == 0) {
            for (int idx = threadIdx.x; idx < G * D; idx += blockDim.x) {
                const int g = idx / D, e = idx - g * D;
                float M = -INFINITY;
                for (int x = 0; x < X; ++x) M = fmaxf(M, cl_ml[(x * G + g) * 2]);
                float L = 0.f, O = 0.f;
                for (int x = 0; x < X; ++x) {
                    const float sc = exp2_safe(cl_ml[(x * G + g) * 2], M);
                    L = fmaf(cl_ml[(x * G + g) * 2 + 1], sc, L);
                    O = fmaf(cl_o[(x * G + g) * D + e], sc, O);
                }
                outp[idx] = Elt<T>::from_float(O / L);
            }
        }
    }
    if (a.fused && rank == 0 && threadIdx.x == 0) {
        UnitState ns;
        ns.len = st.len < lv.cap ? st.len + 1 : st.len;
        ns.n_tok = st.n_tok + 1;
        lv.state[unit] = ns;
    }
}

}  // namespace lar
