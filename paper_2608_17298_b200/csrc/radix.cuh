// Stable LSD radix sort of (key, value) pairs of uint32 on the low `bits` bits of the key, 8 bits per
// pass.  One block owns a chunk of RADIX_CHUNK consecutive items.  A pass is: histogram of every chunk, a global
// exclusive scan of the [digit][chunk] table (every (digit, chunk) gets its output offset), and the scatter.
// The scatter block loads its items at once, ranks them (a warp ranks its 512 consecutive items round by round
// with a match on the digit; warps and digits are then prefixed), sorts the chunk in shared memory, and writes it
// out in sorted order: consecutive threads write consecutive addresses of a digit's run, so the stores are
// full sectors instead of 4 scattered bytes.  Equal keys keep their order.  The item count may live on the device
// (n_dev) or be fixed (n_fixed); when *err_dev is non-zero the sort does nothing.  No block waits on another.
#pragma once

#include "common.cuh"

namespace gart {

constexpr int RADIX_THREADS = 256;
constexpr int RADIX_WARPS = RADIX_THREADS / 32;
constexpr int RADIX_ITEMS = 16;                               // per thread
constexpr int RADIX_CHUNK = RADIX_THREADS * RADIX_ITEMS;      // 4096 items per block
constexpr int RADIX_WARP_ITEMS = 32 * RADIX_ITEMS;            // a warp's consecutive share of the chunk

__device__ __forceinline__ uint32_t radix_count(const uint32_t* n_dev, uint32_t n_fixed, const uint32_t* err_dev) {
    if (err_dev && *err_dev) return 0u;
    return n_dev ? *n_dev : n_fixed;
}

static __global__ void __launch_bounds__(RADIX_THREADS) radix_hist_kernel(const uint32_t* __restrict__ keys, const uint32_t* n_dev,
                                                                          uint32_t n_fixed, const uint32_t* err_dev, int shift,
                                                                          int nchunks, uint32_t* __restrict__ table) {
    __shared__ uint32_t hist[256];
    const int chunk = blockIdx.x;
    hist[threadIdx.x] = 0;
    __syncthreads();
    const uint32_t n = radix_count(n_dev, n_fixed, err_dev);
    const int64_t base = (int64_t)chunk * RADIX_CHUNK;
#pragma unroll 4
    for (int r = 0; r < RADIX_ITEMS; ++r) {
        const int64_t i = base + r * RADIX_THREADS + threadIdx.x;
        if (i < n) atomicAdd(&hist[(keys[i] >> shift) & 255u], 1u);
    }
    __syncthreads();
    table[(size_t)threadIdx.x * nchunks + chunk] = hist[threadIdx.x];
}

struct RadixTableF {
    const uint32_t* t;
    __device__ __forceinline__ uint32_t operator()(int64_t i) const { return t[i]; }
};

static __global__ void __launch_bounds__(RADIX_THREADS) radix_scatter_kernel(const uint32_t* __restrict__ keys_in, const uint32_t* __restrict__ vals_in,
                                                                             const uint32_t* n_dev, uint32_t n_fixed, const uint32_t* err_dev,
                                                                             int shift, int nchunks, const uint32_t* __restrict__ table_scanned,
                                                                             uint32_t* __restrict__ keys_out, uint32_t* __restrict__ vals_out) {
    __shared__ uint32_t whist[RADIX_WARPS][256];   // per warp and digit: running count, then the prefix over the warps before it
    __shared__ uint32_t dbase[256];                // start of every digit's run inside the sorted chunk
    __shared__ uint32_t gbase[256];                // start of this chunk's run of every digit in the output
    __shared__ uint32_t wtot[RADIX_WARPS];
    __shared__ uint2 stage[RADIX_CHUNK];
    const int t = threadIdx.x, w = t >> 5, lane = t & 31;
    const int chunk = blockIdx.x;
    const uint32_t n = radix_count(n_dev, n_fixed, err_dev);
    const int64_t base = (int64_t)chunk * RADIX_CHUNK;
    if (base >= n) return;
    const int64_t left = (int64_t)n - base;
    const int cnt = left < RADIX_CHUNK ? (int)left : RADIX_CHUNK;
    // the warp's items, all loads in flight together (item r of lane l: position w * 512 + r * 32 + l of the chunk)
    uint32_t k[RADIX_ITEMS], v[RADIX_ITEMS];
#pragma unroll
    for (int r = 0; r < RADIX_ITEMS; ++r) {
        const int li = w * RADIX_WARP_ITEMS + r * 32 + lane;
        const bool act = li < cnt;
        k[r] = act ? keys_in[base + li] : 0u;
        v[r] = act ? vals_in[base + li] : 0u;
    }
#pragma unroll
    for (int q = 0; q < RADIX_WARPS; ++q) whist[q][t] = 0u;
    gbase[t] = table_scanned[(size_t)t * nchunks + chunk];
    __syncthreads();
    // rank inside (warp, digit), in the order of the items
    uint16_t lpos[RADIX_ITEMS];
#pragma unroll
    for (int r = 0; r < RADIX_ITEMS; ++r) {
        const bool act = w * RADIX_WARP_ITEMS + r * 32 + lane < cnt;
        const unsigned amask = __ballot_sync(0xffffffffu, act);
        lpos[r] = 0;
        if (act) {
            const uint32_t d = (k[r] >> shift) & 255u;
            const unsigned peers = __match_any_sync(amask, d);
            const uint32_t rank = __popc(peers & ((1u << lane) - 1u));
            const uint32_t old = whist[w][d];
            __syncwarp(amask);
            if (rank == 0) whist[w][d] = old + __popc(peers);
            __syncwarp(amask);
            lpos[r] = (uint16_t)(old + rank);
        }
    }
    __syncthreads();
    // digit t: prefix over the warps, total; then the exclusive scan of the totals over the digits
    uint32_t tot = 0;
#pragma unroll
    for (int q = 0; q < RADIX_WARPS; ++q) {
        const uint32_t c = whist[q][t];
        whist[q][t] = tot;
        tot += c;
    }
    uint32_t inc = tot;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t up = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += up;
    }
    if (lane == 31) wtot[w] = inc;
    __syncthreads();
    uint32_t before = 0;
#pragma unroll
    for (int q = 0; q < RADIX_WARPS; ++q) before += q < w ? wtot[q] : 0u;
    dbase[t] = before + inc - tot;
    __syncthreads();
    // sort the chunk in shared memory
#pragma unroll
    for (int r = 0; r < RADIX_ITEMS; ++r) {
        if (w * RADIX_WARP_ITEMS + r * 32 + lane < cnt) {
            const uint32_t d = (k[r] >> shift) & 255u;
            stage[dbase[d] + whist[w][d] + lpos[r]] = make_uint2(k[r], v[r]);
        }
    }
    __syncthreads();
    // write out in sorted order: a digit's run is contiguous in the output
    for (int i = t; i < cnt; i += RADIX_THREADS) {
        const uint2 kv = stage[i];
        const uint32_t d = (kv.x >> shift) & 255u;
        const uint32_t pos = gbase[d] + ((uint32_t)i - dbase[d]);
        keys_out[pos] = kv.x;
        vals_out[pos] = kv.y;
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
    for (int pass = 0; pass < radix_passes(bits); ++pass) {
        const int shift = 8 * pass;
        radix_hist_kernel<<<nchunks, RADIX_THREADS, 0, st>>>(k[cur], n_dev, n_fixed, err_dev, shift, nchunks, table);
        GART_LAUNCH_CHECK();
        RadixTableF tf{table};
        // in place: every block of the apply pass reads its items before it writes them, and the
        // reduce pass (a separate launch) has finished before any write
        const gart_status s = exclusive_scan(tf, (int64_t)256 * nchunks, table, total64, scan_ws, st);
        if (s != GART_OK) return s;
        radix_scatter_kernel<<<nchunks, RADIX_THREADS, 0, st>>>(k[cur], v[cur], n_dev, n_fixed, err_dev, shift, nchunks, table,
                                                               k[cur ^ 1], v[cur ^ 1]);
        GART_LAUNCH_CHECK();
        cur ^= 1;
    }
    return GART_OK;
}

}  // namespace gart
