// Stable LSD radix sort of (key, value) pairs of uint32 on the low `bits` bits of the key, 8 bits per
// pass.  One warp owns a chunk of RADIX_CHUNK consecutive items: it histograms the chunk, a global
// exclusive scan of the [digit][chunk] table gives every (digit, chunk) its output offset, and the
// warp scatters its items in input order (ranks inside a round of 32 from a match on the digit), so
// equal keys keep their order.  The item count may live on the device (n_dev) or be fixed (n_fixed);
// when *err_dev is non-zero the sort does nothing.  No block waits on another.
#pragma once

#include "common.cuh"

namespace gart {

constexpr int RADIX_CHUNK = 2048;
constexpr int RADIX_WARPS = 4;

__device__ __forceinline__ uint32_t radix_count(const uint32_t* n_dev, uint32_t n_fixed, const uint32_t* err_dev) {
    if (err_dev && *err_dev) return 0u;
    return n_dev ? *n_dev : n_fixed;
}

static __global__ void __launch_bounds__(RADIX_WARPS * 32) radix_hist_kernel(const uint32_t* __restrict__ keys, const uint32_t* n_dev,
                                                                             uint32_t n_fixed, const uint32_t* err_dev, int shift,
                                                                             int nchunks, uint32_t* __restrict__ table) {
    __shared__ uint32_t hist[RADIX_WARPS][256];
    const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int chunk = blockIdx.x * RADIX_WARPS + w;
    for (int d = lane; d < 256; d += 32) hist[w][d] = 0;
    __syncwarp();
    const uint32_t n = radix_count(n_dev, n_fixed, err_dev);
    if (chunk < nchunks) {
        const int64_t base = (int64_t)chunk * RADIX_CHUNK;
        for (int r = 0; r < RADIX_CHUNK / 32; ++r) {
            const int64_t i = base + r * 32 + lane;
            if (i < n) atomicAdd(&hist[w][(keys[i] >> shift) & 255u], 1u);
        }
        __syncwarp();
        for (int d = lane; d < 256; d += 32) table[(size_t)d * nchunks + chunk] = hist[w][d];
    }
}

struct RadixTableF {
    const uint32_t* t;
    __device__ __forceinline__ uint32_t operator()(int64_t i) const { return t[i]; }
};

static __global__ void __launch_bounds__(RADIX_WARPS * 32) radix_scatter_kernel(const uint32_t* __restrict__ keys_in, const uint32_t* __restrict__ vals_in,
                                                                                const uint32_t* n_dev, uint32_t n_fixed, const uint32_t* err_dev,
                                                                                int shift, int nchunks, const uint32_t* __restrict__ table_scanned,
                                                                                uint32_t* __restrict__ keys_out, uint32_t* __restrict__ vals_out) {
    __shared__ uint32_t cursor[RADIX_WARPS][256];
    const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int chunk = blockIdx.x * RADIX_WARPS + w;
    if (chunk >= nchunks) return;
    const uint32_t n = radix_count(n_dev, n_fixed, err_dev);
    const int64_t base = (int64_t)chunk * RADIX_CHUNK;
    if (base >= n) return;
    for (int d = lane; d < 256; d += 32) cursor[w][d] = table_scanned[(size_t)d * nchunks + chunk];
    __syncwarp();
    for (int r = 0; r < RADIX_CHUNK / 32; ++r) {
        const int64_t i = base + r * 32 + lane;
        const bool act = i < n;
        const unsigned amask = __ballot_sync(0xffffffffu, act);
        if (act) {
            const uint32_t k = keys_in[i];
            const uint32_t v = vals_in[i];
            const uint32_t d = (k >> shift) & 255u;
            const unsigned peers = __match_any_sync(amask, d);
            const uint32_t rank = __popc(peers & ((1u << lane) - 1u));
            const uint32_t pos = cursor[w][d] + rank;
            __syncwarp(amask);
            if (rank == 0) cursor[w][d] += __popc(peers);
            __syncwarp(amask);
            keys_out[pos] = k;
            vals_out[pos] = v;
        }
        if (amask != 0xffffffffu) break;
    }
}

static inline int radix_passes(int bits) { return (bits + 7) / 8; }
static inline int64_t radix_chunks(int64_t cap) { return ceil_div(cap > 0 ? cap : 1, RADIX_CHUNK); }
static inline size_t radix_table_bytes(int64_t cap) { return align256((size_t)(256 * radix_chunks(cap) + 1) * 4); }
static inline size_t radix_scan_bytes(int64_t cap) { return scan_workspace_bytes(256 * radix_chunks(cap)); }

// Sorts the pairs held in (k[cur], v[cur]); buffers alternate, the result ends in index (cur + passes) & 1.
static inline gart_status radix_sort_pairs(uint32_t* const k[2], uint32_t* const v[2], int cur, int bits, int64_t cap,
                                           const uint32_t* n_dev, uint32_t n_fixed, const uint32_t* err_dev,
                                           uint32_t* table, void* scan_ws, uint64_t* total64, cudaStream_t st) {
    const int nchunks = (int)radix_chunks(cap);
    const int blocks = (int)ceil_div(nchunks, RADIX_WARPS);
    for (int pass = 0; pass < radix_passes(bits); ++pass) {
        const int shift = 8 * pass;
        radix_hist_kernel<<<blocks, RADIX_WARPS * 32, 0, st>>>(k[cur], n_dev, n_fixed, err_dev, shift, nchunks, table);
        GART_LAUNCH_CHECK();
        RadixTableF tf{table};
        // in place: every block of the apply pass reads its items before it writes them, and the
        // reduce pass (a separate launch) has finished before any write
        const gart_status s = exclusive_scan(tf, (int64_t)256 * nchunks, table, total64, scan_ws, st);
        if (s != GART_OK) return s;
        radix_scatter_kernel<<<blocks, RADIX_WARPS * 32, 0, st>>>(k[cur], v[cur], n_dev, n_fixed, err_dev, shift, nchunks, table,
                                                                  k[cur ^ 1], v[cur ^ 1]);
        GART_LAUNCH_CHECK();
        cur ^= 1;
    }
    return GART_OK;
}

}  // namespace gart
