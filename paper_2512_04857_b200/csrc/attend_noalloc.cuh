// Decode attention over dense caller-owned K/V with library-owned static scratch: the split-KV scheme of the
// decode kernels (partial (m, l, o) per key range, ticket per unit, the last CTA to arrive merges) for callers
// that cannot provide a scratch buffer.  The paper has no counterpart of this entry point.
//
// The scratch is a file-scope device array: every GPU that loads the library holds it (kStaticScratchBytes)
// until the process exits.  Its name is a device symbol: host code must not pass the name itself to a kernel
// (on the host it is only a stand-in); the address comes from cudaGetSymbolAddress, once per device.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

namespace lar {

constexpr size_t kStaticScratchBytes = 8u << 20;              // 8 MiB per GPU
constexpr int kStaticMaxUnits = 16384;                        // one ticket per unit at the front of the array
constexpr size_t kStaticTicketBytes = kStaticMaxUnits * sizeof(int);
constexpr int kStaticMaxSplits = 8;

static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// q, out: [units][G][D]; k, v: [units][len][D] (bf16, dense).  Grid = units * splits CTAs of 128 threads.
template <int D>
__global__ void __launch_bounds__(128) attend_dense_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                                                           const __nv_bfloat16* __restrict__ v, __nv_bfloat16* __restrict__ out,
                                                           unsigned char* scratch, int G, int len, int splits, float scale_log2) {
    constexpr int PER = D / 32;  // elements per lane: lane holds d = lane * PER .. + PER - 1
    constexpr int PS = D + 2;    // floats per partial: o[D], m, l
    constexpr int GMAX = 8;
    __shared__ float part[4][GMAX][PS];
    __shared__ int s_ticket;
    const int unit = blockIdx.x / splits, split = blockIdx.x - unit * splits;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int r0 = (int)((long long)split * len / splits), r1 = (int)((long long)(split + 1) * len / splits);

    float qf[GMAX][PER], o[GMAX][PER], m[GMAX], l[GMAX];
#pragma unroll
    for (int g = 0; g < GMAX; ++g) {
        m[g] = -INFINITY;
        l[g] = 0.f;
#pragma unroll
        for (int i = 0; i < PER; ++i) {
            o[g][i] = 0.f;
            qf[g][i] = g < G ? __bfloat162float(q[((size_t)unit * G + g) * D + lane * PER + i]) * scale_log2 : 0.f;
        }
    }
    const __nv_bfloat16* kb = k + (size_t)unit * len * D;
    const __nv_bfloat16* vb = v + (size_t)unit * len * D;
    for (int r = r0 + warp; r < r1; r += 4) {
        float kf[PER], vf[PER];
#pragma unroll
        for (int i = 0; i < PER; ++i) {
            kf[i] = __bfloat162float(kb[(size_t)r * D + lane * PER + i]);
            vf[i] = __bfloat162float(vb[(size_t)r * D + lane * PER + i]);
        }
#pragma unroll
        for (int g = 0; g < GMAX; ++g) {
            if (g < G) {
                float s = 0.f;
#pragma unroll
                for (int i = 0; i < PER; ++i) s = fmaf(qf[g][i], kf[i], s);
#pragma unroll
                for (int off = 16; off >= 1; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
                const float m_new = fmaxf(m[g], s);
                const float corr = exp2f(m[g] - m_new), p = exp2f(s - m_new);
                m[g] = m_new;
                l[g] = l[g] * corr + p;
#pragma unroll
                for (int i = 0; i < PER; ++i) o[g][i] = fmaf(p, vf[i], o[g][i] * corr);
            }
        }
    }
#pragma unroll
    for (int g = 0; g < GMAX; ++g) {
        if (g < G) {
#pragma unroll
            for (int i = 0; i < PER; ++i) part[warp][g][lane * PER + i] = o[g][i];
            if (lane == 0) {
                part[warp][g][D] = m[g];
                part[warp][g][D + 1] = l[g];
            }
        }
    }
    __syncthreads();

    int* tickets = reinterpret_cast<int*>(scratch);
    float* partials = reinterpret_cast<float*>(scratch + kStaticTicketBytes);
    float* mine = partials + ((size_t)unit * splits + split) * G * PS;
    // merge the four warps: thread -> (head, element)
    for (int idx = threadIdx.x; idx < G * D; idx += blockDim.x) {
        const int g = idx / D, e = idx - g * D;
        float M = -INFINITY;
        for (int w = 0; w < 4; ++w) M = fmaxf(M, part[w][g][D]);
        float L = 0.f, O = 0.f;
        for (int w = 0; w < 4; ++w) {
            const float f = part[w][g][D] == -INFINITY ? 0.f : exp2f(part[w][g][D] - M);
            L = fmaf(part[w][g][D + 1], f, L);
            O = fmaf(part[w][g][e], f, O);
        }
        if (splits == 1) {
            out[((size_t)unit * G + g) * D + e] = __float2bfloat16_rn(L > 0.f ? O / L : 0.f);
        } else {
            mine[g * PS + e] = O;
            if (e == 0) {
                mine[g * PS + D] = M;
                mine[g * PS + D + 1] = L;
            }
        }
    }
    if (splits == 1) return;

    // the CTA that delivers the last partial of a unit merges them (nobody waits)
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_ticket = atomicAdd(tickets + unit, 1);
    __syncthreads();
    if (s_ticket != splits - 1) return;
    __threadfence();
    const float* all = partials + (size_t)unit * splits * G * PS;
    for (int idx = threadIdx.x; idx < G * D; idx += blockDim.x) {
        const int g = idx / D, e = idx - g * D;
        float M = -INFINITY;
        for (int s = 0; s < splits; ++s) M = fmaxf(M, __ldcg(all + (s * G + g) * PS + D));
        float L = 0.f, O = 0.f;
        for (int s = 0; s < splits; ++s) {
            const float ms = __ldcg(all + (s * G + g) * PS + D);
            const float f = ms == -INFINITY ? 0.f : exp2f(ms - M);
            L = fmaf(__ldcg(all + (s * G + g) * PS + D + 1), f, L);
            O = fmaf(__ldcg(all + (s * G + g) * PS + e), f, O);
        }
        out[((size_t)unit * G + g) * D + e] = __float2bfloat16_rn(L > 0.f ? O / L : 0.f);
    }
    if (threadIdx.x == 0) tickets[unit] = 0;  // the array outlives the call: leave the ticket as it was found
}

// Device address of the static scratch on the current device (looked up once per device).
inline cudaError_t static_scratch_address(unsigned char** out) {
    static std::mutex mu;
    static unsigned char* addr[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(mu);
    if (!addr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);  // the symbol's address on the device that is current
        if (e != cudaSuccess) return e;
        addr[dev] = static_cast<unsigned char*>(p);
    }
    *out = addr[dev];
    return cudaSuccess;
}

// Key ranges per unit: enough CTAs for two per SM of a B200 and at least 16 rows each; with more than 148 units every
// unit is one range and no partial is written.  n_units * ranges never exceeds kStaticMaxCtas, so the partials take at
// most kStaticMaxCtas * 8 heads * (128 + 2) floats: they always fit behind the tickets.
constexpr int kStaticMaxCtas = 296;
static_assert((size_t)kStaticMaxCtas * 8 * (128 + 2) * sizeof(float) <= kStaticScratchBytes - kStaticTicketBytes,
              "the partials of the largest split launch must fit into the static array");
inline int static_scratch_splits(int n_units, int len) {
    int splits = kStaticMaxCtas / n_units;
    if (splits > kStaticMaxSplits) splits = kStaticMaxSplits;
    if (splits > len / 16) splits = len / 16;
    if (splits < 1) splits = 1;
    return splits;
}

}  // namespace lar
