// gart_tile_map: reverse tile mapping (Sec. 4.3).  Every Gaussian emits one (tile, id) pair per
// tile overlapped by its rectangle; a stable LSD radix sort on the tile id groups the pairs by
// tile (ids stay ascending inside a tile because emission is id-major); the tile offset table
// marks the group boundaries.  The pair count lives on the device: kernels are sized by the
// caller's capacity and read the actual count.
#include "common.cuh"

namespace gart {

struct TileCountF {
    const int4* rect;
    int64_t n;
    int ts;
    __device__ __forceinline__ uint32_t operator()(int64_t i) const {
        if (i >= n) return 0u;
        const int4 r = rect[i];
        if (r.z < r.x || r.w < r.y) return 0u;
        return (uint32_t)((r.z / ts - r.x / ts + 1) * (r.w / ts - r.y / ts + 1));
    }
};

// Sum of rectangle areas (capacity bound of the intermediate buffer, Eq. 15) into counts[SLOTS].
__global__ void __launch_bounds__(256) area_sum_kernel(const int4* __restrict__ rect, int64_t n, uint32_t* counts) {
    unsigned long long s = 0;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
        const int4 r = rect[i];
        if (r.z >= r.x && r.w >= r.y) s += (unsigned long long)(r.z - r.x + 1) * (unsigned long long)(r.w - r.y + 1);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_down_sync(0xffffffffu, s, o);
    if ((threadIdx.x & 31) == 0 && s) atomicAdd(reinterpret_cast<unsigned long long*>(counts + GART_CNT_SLOTS_LO), s);
}

// total64[0] = P.  Records it, flags an overflow, clears tile_off on overflow.
__global__ void pairs_total_kernel(const uint64_t* total64, int64_t cap_pairs, uint32_t* counts) {
    const uint64_t P = total64[0];
    if (P > (uint64_t)cap_pairs) {
        counts[GART_CNT_PAIRS] = P > 0xffffffffull ? 0xffffffffu : (uint32_t)P;
        atomicOr(&counts[GART_CNT_ERROR], GART_ERRBIT_PAIRS);
    } else {
        counts[GART_CNT_PAIRS] = (uint32_t)P;
    }
}

// One thread per pair slot: find the owning Gaussian by bisection of the emission offsets.
__global__ void __launch_bounds__(256) emit_pairs_kernel(const int4* __restrict__ rect, const uint32_t* __restrict__ emit_off,
                                                         int64_t n, int ts, int tiles_x, const uint32_t* __restrict__ counts,
                                                         uint32_t* __restrict__ keys, uint32_t* __restrict__ vals) {
    if (counts[GART_CNT_ERROR]) return;
    const uint32_t P = counts[GART_CNT_PAIRS];
    const int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (p >= P) return;
    int64_t lo = 0, hi = n;  // emit_off[lo] <= p < emit_off[hi]
    while (hi - lo > 1) {
        const int64_t mid = (lo + hi) >> 1;
        if (emit_off[mid] <= (uint32_t)p) lo = mid; else hi = mid;
    }
    const int4 r = rect[lo];
    const int tx0 = r.x / ts, ntx = r.z / ts - tx0 + 1, ty0 = r.y / ts;
    const int local = (int)((uint32_t)p - emit_off[lo]);
    keys[p] = (uint32_t)((ty0 + local / ntx) * tiles_x + tx0 + local % ntx);
    vals[p] = (uint32_t)lo;
}

// ---- stable LSD radix sort, 8-bit digits, one warp per chunk of RADIX_CHUNK consecutive items
constexpr int RADIX_CHUNK = 2048;
constexpr int RADIX_WARPS = 4;

__global__ void __launch_bounds__(RADIX_WARPS * 32) radix_hist_kernel(const uint32_t* __restrict__ keys, const uint32_t* __restrict__ counts,
                                                                      int shift, int nchunks, uint32_t* __restrict__ table) {
    __shared__ uint32_t hist[RADIX_WARPS][256];
    const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int chunk = blockIdx.x * RADIX_WARPS + w;
    for (int d = lane; d < 256; d += 32) hist[w][d] = 0;
    __syncwarp();
    const uint32_t P = counts[GART_CNT_ERROR] ? 0u : counts[GART_CNT_PAIRS];
    if (chunk < nchunks) {
        const int64_t base = (int64_t)chunk * RADIX_CHUNK;
        for (int r = 0; r < RADIX_CHUNK / 32; ++r) {
            const int64_t i = base + r * 32 + lane;
            if (i < P) atomicAdd(&hist[w][(keys[i] >> shift) & 255u], 1u);
        }
        __syncwarp();
        for (int d = lane; d < 256; d += 32) table[(size_t)d * nchunks + chunk] = hist[w][d];
    }
}

struct TableF {
    const uint32_t* t;
    __device__ __forceinline__ uint32_t operator()(int64_t i) const { return t[i]; }
};

__global__ void __launch_bounds__(RADIX_WARPS * 32) radix_scatter_kernel(const uint32_t* __restrict__ keys_in, const uint32_t* __restrict__ vals_in,
                                                                         const uint32_t* __restrict__ counts, int shift, int nchunks,
                                                                         const uint32_t* __restrict__ table_scanned,
                                                                         uint32_t* __restrict__ keys_out, uint32_t* __restrict__ vals_out) {
    __shared__ uint32_t cursor[RADIX_WARPS][256];
    const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int chunk = blockIdx.x * RADIX_WARPS + w;
    if (chunk >= nchunks) return;
    const uint32_t P = counts[GART_CNT_ERROR] ? 0u : counts[GART_CNT_PAIRS];
    const int64_t base = (int64_t)chunk * RADIX_CHUNK;
    if (base >= P) return;
    for (int d = lane; d < 256; d += 32) cursor[w][d] = table_scanned[(size_t)d * nchunks + chunk];
    __syncwarp();
    for (int r = 0; r < RADIX_CHUNK / 32; ++r) {
        const int64_t i = base + r * 32 + lane;
        const bool act = i < P;
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

// tile_off[t] = first sorted position whose tile id is >= t; tile_off[T] = P.
__global__ void __launch_bounds__(256) tile_offsets_kernel(const uint32_t* __restrict__ keys_sorted, const uint32_t* __restrict__ counts,
                                                           int T, uint32_t* __restrict__ tile_off) {
    if (counts[GART_CNT_ERROR]) return;
    const uint32_t P = counts[GART_CNT_PAIRS];
    const int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (p >= P) return;
    const int k = (int)keys_sorted[p];
    const int prev = p > 0 ? (int)keys_sorted[p - 1] : -1;
    for (int t = prev + 1; t <= k; ++t) tile_off[t] = (uint32_t)p;
    if (p == (int64_t)P - 1)
        for (int t = k + 1; t <= T; ++t) tile_off[t] = P;
}

struct TileMapWs {
    uint32_t *emit_off, *keys0, *keys1, *vals1, *table;
    uint64_t* total64;
    void* scan_ws;
    size_t bytes;
};

static TileMapWs tile_map_layout(void* base, int64_t n, int64_t cap_pairs) {
    TileMapWs w;
    char* p = (char*)base;
    size_t off = 0;
    auto take = [&](size_t b) { void* r = p ? (void*)(p + off) : nullptr; off += align256(b); return r; };
    const int64_t cp = cap_pairs > 0 ? cap_pairs : 1;
    const int64_t nchunks = ceil_div(cp, RADIX_CHUNK);
    w.total64 = (uint64_t*)take(256);
    w.emit_off = (uint32_t*)take((size_t)(n + 1) * 4);
    w.keys0 = (uint32_t*)take((size_t)cp * 4);
    w.keys1 = (uint32_t*)take((size_t)cp * 4);
    w.vals1 = (uint32_t*)take((size_t)cp * 4);
    w.table = (uint32_t*)take((size_t)(256 * nchunks + 1) * 4);
    const int64_t scan_n = (n > 256 * nchunks ? n : 256 * nchunks);
    w.scan_ws = take(scan_workspace_bytes(scan_n));
    w.bytes = off;
    return w;
}

}  // namespace gart

extern "C" size_t gart_tile_map_workspace_bytes(int64_t n, int32_t width, int32_t height, int32_t tile_size, int64_t cap_pairs) {
    (void)width; (void)height; (void)tile_size;
    return gart::tile_map_layout(nullptr, n > 0 ? n : 1, cap_pairs).bytes;
}

extern "C" gart_status gart_tile_map(const gart_config* cfg, const int32_t* rect, int64_t n, int32_t width, int32_t height,
                                     uint32_t* tile_off, uint32_t* pair_gid, int64_t cap_pairs, uint32_t* counts,
                                     void* workspace, size_t workspace_bytes, void* stream) {
    using namespace gart;
    if (!cfg || !tile_off || !counts || n < 0 || width <= 0 || height <= 0 || cap_pairs < 0) return GART_ERR_INVALID_ARG;
    if (cfg->tile_size != 8 && cfg->tile_size != 16) return GART_ERR_INVALID_ARG;
    if (n > 0 && !rect) return GART_ERR_INVALID_ARG;
    if (cap_pairs > 0 && !pair_gid) return GART_ERR_INVALID_ARG;
    if (cap_pairs > 0xfffffff0ll) return GART_ERR_INVALID_ARG;
    const int ts = cfg->tile_size;
    const int tiles_x = (width + ts - 1) / ts, tiles_y = (height + ts - 1) / ts;
    const int T = tiles_x * tiles_y;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemsetAsync(tile_off, 0, (size_t)(T + 1) * 4, st) != cudaSuccess) return GART_ERR_CUDA;
    if (n == 0) return GART_OK;
    if (!workspace || ((uintptr_t)workspace & 255)) return GART_ERR_INVALID_ARG;
    TileMapWs w = tile_map_layout(workspace, n, cap_pairs);
    if (w.bytes > workspace_bytes) return GART_ERR_WORKSPACE_TOO_SMALL;
    const int4* rect4 = reinterpret_cast<const int4*>(rect);

    area_sum_kernel<<<(unsigned)(ceil_div(n, 256) < 1184 ? ceil_div(n, 256) : 1184), 256, 0, st>>>(rect4, n, counts);
    GART_LAUNCH_CHECK();
    TileCountF cf{rect4, n, ts};
    gart_status s = exclusive_scan(cf, n, w.emit_off, w.total64, w.scan_ws, st);
    if (s != GART_OK) return s;
    pairs_total_kernel<<<1, 1, 0, st>>>(w.total64, cap_pairs, counts);
    GART_LAUNCH_CHECK();
    if (cap_pairs == 0) return GART_OK;

    int bits = 1;
    while ((1 << bits) < T) ++bits;
    const int passes = (bits + 7) / 8;
    // value buffers alternate between pair_gid and ws.vals1 so that the last pass lands in pair_gid
    uint32_t* vbuf[2] = {pair_gid, w.vals1};
    uint32_t* kbuf[2] = {w.keys0, w.keys1};
    int cur = passes & 1;  // emission target: after `passes` flips we are at index 0 = pair_gid
    const int64_t pair_blocks = ceil_div(cap_pairs, 256);
    emit_pairs_kernel<<<(unsigned)pair_blocks, 256, 0, st>>>(rect4, w.emit_off, n, ts, tiles_x, counts, kbuf[cur], vbuf[cur]);
    GART_LAUNCH_CHECK();
    const int nchunks = (int)ceil_div(cap_pairs, RADIX_CHUNK);
    const int rblocks = (int)ceil_div(nchunks, RADIX_WARPS);
    for (int pass = 0; pass < passes; ++pass) {
        const int shift = 8 * pass;
        radix_hist_kernel<<<rblocks, RADIX_WARPS * 32, 0, st>>>(kbuf[cur], counts, shift, nchunks, w.table);
        GART_LAUNCH_CHECK();
        TableF tf{w.table};
        // in-place scan is safe: every block reads its items before any block's apply phase runs
        // (separate launches), and apply re-reads through the functor before writing the same index
        s = exclusive_scan(tf, (int64_t)256 * nchunks, w.table, w.total64, w.scan_ws, st);
        if (s != GART_OK) return s;
        radix_scatter_kernel<<<rblocks, RADIX_WARPS * 32, 0, st>>>(kbuf[cur], vbuf[cur], counts, shift, nchunks, w.table,
                                                                   kbuf[cur ^ 1], vbuf[cur ^ 1]);
        GART_LAUNCH_CHECK();
        cur ^= 1;
    }
    tile_offsets_kernel<<<(unsigned)pair_blocks, 256, 0, st>>>(kbuf[cur], counts, T, tile_off);
    GART_LAUNCH_CHECK();
    return GART_OK;
}
