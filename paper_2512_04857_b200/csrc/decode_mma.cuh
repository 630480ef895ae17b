// bf16 decode attention (Eq. 2-3) with tensor-map TMA staging and warp-level MMA.
//
// Same decomposition as decode_attn.cuh (cluster of `splits` CTAs per unit, 16-key tiles dealt
// round-robin to CTAs and warps, one mbarrier pipeline per warp, partials merged in shared memory
// and across the cluster through distributed shared memory), but the arithmetic per tile is
//     S = Q K^T      mma.sync m16n8k16 (bf16 in, fp32 out): rows = the G query heads of the unit
//     O += P V       same instruction, P rounded to bf16, V fragments via ldmatrix.trans
// which removes the per-element unpack / FMA / shuffle work of the CUDA-core version: the kernel is
// bound by HBM, not by instruction issue.  K and V tiles are fetched with cp.async.bulk.tensor
// (2-D tiled, 128-byte swizzle) so that ldmatrix reads them without bank conflicts.  A tile that
// holds fewer than 16 live rows is fetched with a shorter box (4, 8 or 12 rows).
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "decode_attn.cuh"

namespace lar {

struct TensorMaps {
    CUtensorMap k[4];  // box heights 4, 8, 12, 16 rows over the K pools of all layers
    CUtensorMap v[4];
};

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
        "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar)
        : "memory");
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

template <int D>
struct MmaTraits {
    static constexpr int ROW_BYTES = D * 2;
    static constexpr int HALVES = D / 64;             // 128-byte column blocks per row
    static constexpr int SUB_BYTES = kGranule * 128;  // one [16][64] swizzled block
    static constexpr int TILE_BYTES = HALVES * SUB_BYTES;
    static constexpr int STAGE_BYTES = 2 * TILE_BYTES;  // K tile + V tile
    static constexpr int KSTEPS = D / 16;
    static constexpr int NTILES = D / 8;
};

__host__ __device__ inline int decode_mma_smem_bytes(int D, int warps, int stages, int splits, int G) {
    int b = 1024;  // alignment slack: stages start on a 1024-byte boundary (swizzle period)
    b += warps * stages * (2 * (D / 64) * kGranule * 128);
    b += ((warps * stages * 8 + 15) / 16) * 16;
    b += (warps + 1) * G * (D + 2) * 4;
    if (splits > 1) b += splits * G * (D + 2) * 4;
    return b;
}

// byte offset of 16-byte chunk `c` of row `r` inside a tile stored as HALVES swizzled [16][128 B] blocks
template <int D>
__device__ __forceinline__ uint32_t tile_off(int r, int c) {
    return (uint32_t)((c >> 3) * MmaTraits<D>::SUB_BYTES + r * 128 + (((c & 7) ^ (r & 7)) << 4));
}

template <int D, int G>
__global__ void __launch_bounds__(256) decode_mma_kernel(const DecodeArgs a, const __grid_constant__ TensorMaps tm,
                                                         const int pool_row_base) {
    using TR = MmaTraits<D>;
    using T = __nv_bfloat16;
    extern __shared__ unsigned char smem_raw[];

    const int W = blockDim.x >> 5, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int X = a.splits, NS = a.stages;
    const int rank = X > 1 ? (int)cluster_rank() : 0;
    const int unit = blockIdx.x / X;
    const LayerView& lv = a.lv;
    const int quad = lane & 3, qrow = lane >> 2;  // fragment coordinates

    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    unsigned char* smem = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t my_stages = base + (uint32_t)(warp * NS) * TR::STAGE_BYTES;
    unsigned char* after = smem + (size_t)W * NS * TR::STAGE_BYTES;
    const uint32_t my_bars = smem_u32(after) + warp * NS * 8;
    after += ((W * NS * 8 + 15) / 16) * 16;
    float* part_o = reinterpret_cast<float*>(after);  // [W + 1][G][D]   (slot W: the token of this step)
    float* part_ml = part_o + (W + 1) * G * D;        // [W + 1][G][2]
    float* cl_o = part_ml + (W + 1) * G * 2;          // [X][G][D]       (clusters only)
    float* cl_ml = cl_o + X * G * D;                  // [X][G][2]

    if (X > 1) cluster_arrive();  // matched by cluster_wait() before the first remote store
    if (!a.prefetch) grid_dep_wait();

    if (lane == 0) {
        for (int s = 0; s < NS; ++s) mbar_init(my_bars + s * 8, 1);
        mbar_fence_init();
    }
    __syncwarp();

    const UnitState st = lv.state[unit];
    const int len_tma = st.len;
    const int NG = (len_tma + kGranule - 1) / kGranule;
    const int first = rank + X * warp, stride = X * W;
    const int my_n = first < NG ? (NG - first + stride - 1) / stride : 0;

    auto issue = [&](int k) {
        const int g = first + k * stride, s = k % NS;
        const int row0 = g * kGranule;
        const int rows = min(kGranule, len_tma - row0);
        const int hsel = (rows + 3) / 4 - 1;  // box of 4 * (hsel + 1) rows
        const int page = lv.page_table[unit * lv.pages_per_unit + row0 / lv.page_tokens];
        const int y = pool_row_base + page * lv.page_tokens + row0 % lv.page_tokens;
        const uint32_t bar = my_bars + s * 8;
        const uint32_t dst = my_stages + (uint32_t)s * TR::STAGE_BYTES;
        mbar_expect_tx(bar, (uint32_t)(2 * 4 * (hsel + 1) * TR::ROW_BYTES));
#pragma unroll
        for (int h = 0; h < TR::HALVES; ++h) {
            tma_load_2d(dst + h * TR::SUB_BYTES, &tm.k[hsel], h * 64, y, bar);
            tma_load_2d(dst + TR::TILE_BYTES + h * TR::SUB_BYTES, &tm.v[hsel], h * 64, y, bar);
        }
    };
    // lanes 0 .. NS-1 each start one stage, so their page-table reads overlap
    if (lane < NS && lane < my_n) issue(lane);

    if (a.prefetch) grid_dep_wait();
    grid_dep_launch();

    // ---- Q fragments (A operand): row qrow = head, 16 columns per k-step; heads >= G are zero rows
    const T* qbase = reinterpret_cast<const T*>(a.q) + (size_t)unit * G * D;
    uint32_t qa0[TR::KSTEPS], qa2[TR::KSTEPS];
#pragma unroll
    for (int s = 0; s < TR::KSTEPS; ++s) {
        qa0[s] = 0u;
        qa2[s] = 0u;
        if (qrow < G) {
            qa0[s] = __ldg(reinterpret_cast<const uint32_t*>(qbase + qrow * D + 16 * s + 2 * quad));
            qa2[s] = __ldg(reinterpret_cast<const uint32_t*>(qbase + qrow * D + 16 * s + 8 + 2 * quad));
        }
    }

    float m = -INFINITY, l = 0.f;  // head qrow; l is this thread's share of the row sum
    float o[TR::NTILES][4];
#pragma unroll
    for (int t = 0; t < TR::NTILES; ++t) o[t][0] = o[t][1] = o[t][2] = o[t][3] = 0.f;

    bool ok = true;
    for (int k = 0; k < my_n; ++k) {
        const int s = k % NS;
        const bool arrived = mbar_wait_bounded(my_bars + s * 8, (uint32_t)((k / NS) & 1));
        if (!__all_sync(0xffffffffu, arrived)) { ok = false; break; }
        const int rows = min(kGranule, len_tma - (first + k * stride) * kGranule);
        const uint32_t Ks = my_stages + (uint32_t)s * TR::STAGE_BYTES;
        const uint32_t Vs = Ks + TR::TILE_BYTES;

        // S[head][key] for the 16 keys of the tile: two n-tiles of 8 keys
        float sc[2][4];
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            sc[j][0] = sc[j][1] = sc[j][2] = sc[j][3] = 0.f;
#pragma unroll
            for (int i = 0; i < TR::KSTEPS / 2; ++i) {
                uint32_t b[4];
                ldmatrix_x4(Ks + tile_off<D>(8 * j + (lane & 7), 4 * i + (lane >> 3)), b);
                mma_bf16(sc[j], qa0[2 * i], 0u, qa2[2 * i], 0u, b[0], b[1]);
                mma_bf16(sc[j], qa0[2 * i + 1], 0u, qa2[2 * i + 1], 0u, b[2], b[3]);
            }
        }
        // online softmax over the keys this thread holds: 2*quad, 2*quad+1 (+8)
        float sv[4];
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            sv[2 * j + 0] = (8 * j + 2 * quad + 0 < rows) ? sc[j][0] * a.scale_log2 : -INFINITY;
            sv[2 * j + 1] = (8 * j + 2 * quad + 1 < rows) ? sc[j][1] * a.scale_log2 : -INFINITY;
        }
        float mx = fmaxf(fmaxf(sv[0], sv[1]), fmaxf(sv[2], sv[3]));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        const float m_new = fmaxf(m, mx);
        const float corr = exp2f(m - m_new);
        float p[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) p[i] = exp2f(sv[i] - m_new);
        l = l * corr + (p[0] + p[1]) + (p[2] + p[3]);
        m = m_new;
        if (__any_sync(0xffffffffu, corr != 1.f)) {
#pragma unroll
            for (int t = 0; t < TR::NTILES; ++t) { o[t][0] *= corr; o[t][1] *= corr; }
        }
        const uint32_t pa0 = pack_bf16(p[0], p[1]), pa2 = pack_bf16(p[2], p[3]);
        // a short box leaves rows of the V tile unwritten: their weight is 0, but 0 * (stale NaN) is not
        const int box_rows = (rows + 3) & ~3;
        if (box_rows < kGranule) {
            const int n16 = (kGranule - box_rows) * 8;  // 16-byte chunks per 128-byte-wide block
            for (int i = lane; i < n16 * TR::HALVES; i += 32) {
                const int h = i / n16, c = i - h * n16;
                asm volatile("st.shared.v4.u32 [%0], {%1, %1, %1, %1};" ::"r"(Vs + h * TR::SUB_BYTES + box_rows * 128 + c * 16), "r"(0u) : "memory");
            }
            __syncwarp();
        }
        // O[head][d] += P V
#pragma unroll
        for (int t = 0; t < TR::NTILES / 2; ++t) {
            uint32_t b[4];
            ldmatrix_x4_trans(Vs + tile_off<D>((lane & 7) + 8 * ((lane >> 3) & 1), 2 * t + (lane >> 4)), b);
            mma_bf16(o[2 * t], pa0, 0u, pa2, 0u, b[0], b[1]);
            mma_bf16(o[2 * t + 1], pa0, 0u, pa2, 0u, b[2], b[3]);
        }
        __syncwarp();
        if (lane == 0 && k + NS < my_n) issue(k + NS);
    }
    if (!ok && lane == 0) atomicOr(lv.status, kStWaitLimit);

    // ---- warp partial -> shared memory
    l += __shfl_xor_sync(0xffffffffu, l, 1);
    l += __shfl_xor_sync(0xffffffffu, l, 2);
    if (qrow < G) {
#pragma unroll
        for (int t = 0; t < TR::NTILES; ++t)
            *reinterpret_cast<float2*>(part_o + (warp * G + qrow) * D + 8 * t + 2 * quad) = make_float2(o[t][0], o[t][1]);
        if (quad == 0) {
            part_ml[(warp * G + qrow) * 2 + 0] = m;
            part_ml[(warp * G + qrow) * 2 + 1] = l;
        }
    }

    // ---- the token of this step (slot W of the partials), its store, the guide queue (Eq. 4, 8)
    const int owner_rank = NG % X, owner_warp = (NG / X) % W;
    const bool owner = rank == owner_rank && warp == owner_warp;
    if (warp == owner_warp) {
        constexpr int PER = D / 32;  // elements per lane
        float kf[PER], vf[PER];
        if (owner && a.fused) {
            const T* kn = reinterpret_cast<const T*>(a.k_new) + (size_t)unit * D + lane * PER;
            const T* vn = reinterpret_cast<const T*>(a.v_new) + (size_t)unit * D + lane * PER;
#pragma unroll
            for (int e = 0; e < PER; ++e) { kf[e] = __bfloat162float(kn[e]); vf[e] = __bfloat162float(vn[e]); }
#pragma unroll
            for (int g = 0; g < G; ++g) {
                float sv = 0.f;
#pragma unroll
                for (int e = 0; e < PER; ++e) sv = fmaf(__bfloat162float(qbase[g * D + lane * PER + e]), kf[e], sv);
                sv = warp_sum(sv) * a.scale_log2;
#pragma unroll
                for (int e = 0; e < PER; ++e) part_o[(W * G + g) * D + lane * PER + e] = vf[e];
                if (lane == 0) {
                    part_ml[(W * G + g) * 2 + 0] = sv;
                    part_ml[(W * G + g) * 2 + 1] = 1.f;
                }
            }
            if (st.len < lv.cap) {
                const size_t off = row_offset(lv, unit, st.len, TR::ROW_BYTES) + lane * PER * 2;
#pragma unroll
                for (int e = 0; e < PER; e += 2) {
                    *reinterpret_cast<uint32_t*>(lv.k_pool + off + e * 2) = *reinterpret_cast<const uint32_t*>(kn + e);
                    *reinterpret_cast<uint32_t*>(lv.v_pool + off + e * 2) = *reinterpret_cast<const uint32_t*>(vn + e);
                }
                if (lane == 0) lv.index_map[(size_t)unit * lv.cap_pad + st.len] = lv.cond_len + st.n_tok;
            } else if (lane == 0) {
                atomicOr(lv.status, kStCapacity);
            }
        } else {
            // no token from registers in this CTA: an empty partial
            for (int g = lane; g < G; g += 32) {
                part_ml[(W * G + g) * 2 + 0] = -INFINITY;
                part_ml[(W * G + g) * 2 + 1] = 0.f;
            }
            if (owner && len_tma == 0 && lane == 0) atomicOr(lv.status, kStEmpty);
        }
        if (owner) {
            const int tok = a.fused ? st.n_tok : st.n_tok - 1;  // 0-based visual index of this step's token
            if (tok >= 0) {
                const int slot = tok % lv.line_width;
                T* gq = reinterpret_cast<T*>(lv.guide) + (((size_t)unit * lv.line_width + slot) * G) * D;
                for (int i = lane; i < G * D / 2; i += 32)
                    reinterpret_cast<uint32_t*>(gq)[i] = __ldg(reinterpret_cast<const uint32_t*>(qbase) + i);
            }
        }
    }
    __syncthreads();

    // ---- merge warps (+ the step's token) -> CTA, CTAs -> cluster
    T* outp = reinterpret_cast<T*>(a.out) + (size_t)unit * G * D;
    if (X > 1) cluster_wait();
    for (int idx = threadIdx.x; idx < G * D; idx += blockDim.x) {
        const int g = idx / D, e = idx - g * D;
        float M = -INFINITY;
        for (int w = 0; w <= W; ++w) M = fmaxf(M, part_ml[(w * G + g) * 2]);
        float L = 0.f, O = 0.f;
        for (int w = 0; w <= W; ++w) {
            const float f = exp2_safe(part_ml[(w * G + g) * 2], M);
            if (f != 0.f) {
                L = fmaf(part_ml[(w * G + g) * 2 + 1], f, L);
                O = fmaf(part_o[(w * G + g) * D + e], f, O);
            }
        }
        if (X == 1) {
            outp[idx] = __float2bfloat16_rn(O / L);
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
                    const float f = exp2_safe(cl_ml[(x * G + g) * 2], M);
                    if (f != 0.f) {
                        L = fmaf(cl_ml[(x * G + g) * 2 + 1], f, L);
                        O = fmaf(cl_o[(x * G + g) * D + e], f, O);
                    }
                }
                outp[idx] = __float2bfloat16_rn(O / L);
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
