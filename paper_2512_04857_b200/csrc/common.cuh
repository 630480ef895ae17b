// Shared device helpers: PTX wrappers (mbarrier, bulk async copy, cluster, dependent launch),
// element unpacking, and the device-side view of one layer of the cache.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace lar {

constexpr int kGranule = 16;  // rows of K (and V) moved by one bulk copy and processed as one tile

// device status bits (lar_cache_poll_device_status)
constexpr unsigned kStCapacity = 1u, kStBoundary = 2u, kStWaitLimit = 4u, kStEmpty = 8u, kStLength = 16u, kStNonFinite = 32u;

struct UnitState {
    int len;    // live entries (prefix + visual)
    int n_tok;  // visual tokens appended so far
};

// Everything a kernel needs to address one layer of the cache.
struct LayerView {
    char* k_pool;           // [pages][page_tokens][d] elements
    char* v_pool;
    const int* page_table;  // [units][pages_per_unit] -> page id inside the pools
    int* index_map;         // [units][cap_pad]
    UnitState* state;       // [units]
    char* guide;            // [units][n][G][d] elements
    float* scores;          // [units][mid_pad]
    float* acc;             // [units][cap_pad] attention mass accumulated per slot (accumulated-attention scoring only)
    unsigned* status;       // one word per cache
    int pages_per_unit, page_tokens, cap, cap_pad, mid_pad;
    int cond_len, line_width, budget_tokens, anchor_len, recent_lines, compressing;
    int n_kv_heads, group;
    int identity_pages;     // 1: unit u owns pages u * pages_per_unit ... in order (the table need not be read)
};

// Byte distance between the same array of consecutive layers (a kernel whose grid spans several layers).
struct LayerStrides {
    size_t pool, page_table, index_map, state, guide, scores, acc;
};
__host__ __device__ inline LayerView layer_view_at(LayerView lv, const LayerStrides& ls, int layers_ahead) {
    const size_t y = (size_t)layers_ahead;
    lv.k_pool += y * ls.pool;
    lv.v_pool += y * ls.pool;
    lv.page_table = reinterpret_cast<const int*>(reinterpret_cast<const char*>(lv.page_table) + y * ls.page_table);
    lv.index_map = reinterpret_cast<int*>(reinterpret_cast<char*>(lv.index_map) + y * ls.index_map);
    lv.state = reinterpret_cast<UnitState*>(reinterpret_cast<char*>(lv.state) + y * ls.state);
    lv.guide += y * ls.guide;
    lv.scores = reinterpret_cast<float*>(reinterpret_cast<char*>(lv.scores) + y * ls.scores);
    if (lv.acc) lv.acc = reinterpret_cast<float*>(reinterpret_cast<char*>(lv.acc) + y * ls.acc);
    return lv;
}

// ---------------------------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: gives up after ~1 s of SM clocks and reports failure instead of hanging.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (clock64() - t0 > 2000000000LL) return false;
    }
    return true;
}
// 1-D bulk copy global -> shared through the TMA unit; completion is signalled on `bar` (bytes).
// dst, src 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_arrive() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
}
__device__ __forceinline__ void cluster_wait() {
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// address of `local_smem_addr` in the shared memory of CTA `rank` of this cluster
__device__ __forceinline__ uint32_t map_to_rank(uint32_t local_smem_addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_smem_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void st_cluster_f32(uint32_t addr, float v) {
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}

// ---------------------------------------------------------------------------------- elements
template <typename T>
struct Elt;
template <>
struct Elt<__nv_bfloat16> {
    static constexpr int kPerChunk = 8;  // elements in one 16-byte chunk
    static __device__ __forceinline__ void unpack(const uint4& c, float (&f)[8]) {
        f[0] = __uint_as_float(c.x << 16); f[1] = __uint_as_float(c.x & 0xffff0000u);
        f[2] = __uint_as_float(c.y << 16); f[3] = __uint_as_float(c.y & 0xffff0000u);
        f[4] = __uint_as_float(c.z << 16); f[5] = __uint_as_float(c.z & 0xffff0000u);
        f[6] = __uint_as_float(c.w << 16); f[7] = __uint_as_float(c.w & 0xffff0000u);
    }
    static __device__ __forceinline__ __nv_bfloat16 from_float(float x) { return __float2bfloat16_rn(x); }
};
template <>
struct Elt<float> {
    static constexpr int kPerChunk = 4;
    static __device__ __forceinline__ void unpack(const uint4& c, float (&f)[4]) {
        f[0] = __uint_as_float(c.x); f[1] = __uint_as_float(c.y);
        f[2] = __uint_as_float(c.z); f[3] = __uint_as_float(c.w);
    }
    static __device__ __forceinline__ float from_float(float x) { return x; }
};

// byte address of row `slot` of a unit inside a pool
__device__ __forceinline__ size_t row_offset(const LayerView& lv, int unit, int slot, int row_bytes) {
    const int pidx = unit * lv.pages_per_unit + slot / lv.page_tokens;
    const int page = lv.identity_pages ? pidx : lv.page_table[pidx];
    return (static_cast<size_t>(page) * lv.page_tokens + (slot % lv.page_tokens)) * row_bytes;
}

}  // namespace lar
