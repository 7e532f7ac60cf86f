// gart_tile_map: reverse tile mapping (Sec. 4.3).  Every Gaussian emits one (tile, id) pair per
// tile overlapped by its rectangle; a stable LSD radix sort on the tile id groups the pairs by
// tile (ids stay ascending inside a tile because emission is id-major); the tile offset table
// marks the group boundaries.  The pair count lives on the device: kernels are sized by the
// caller's capacity and read the actual count.
#include "radix.cuh"

#include <atomic>

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

// One thread per Gaussian writes its pairs (row-major over the tiles of its rectangle) from its emission offset.
// Rectangles of more than EMIT_SERIAL tiles (large or near Gaussians; a straddler covers every tile) are written
// by the whole warp, one such lane at a time.
constexpr int EMIT_SERIAL = 16;
__global__ void __launch_bounds__(256) emit_pairs_kernel(const int4* __restrict__ rect, const uint32_t* __restrict__ emit_off,
                                                         int64_t n, int ts, int tiles_x, const uint32_t* __restrict__ counts,
                                                         uint32_t* __restrict__ keys, uint32_t* __restrict__ vals) {
    if (counts[GART_CNT_ERROR]) return;
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int lane = threadIdx.x & 31;
    int tx0 = 0, ty0 = 0, ntx = 0, cnt = 0;
    uint32_t off = 0;
    if (i < n) {
        const int4 r = rect[i];
        if (r.z >= r.x && r.w >= r.y) {
            tx0 = r.x / ts; ty0 = r.y / ts;
            ntx = r.z / ts - tx0 + 1;
            cnt = ntx * (r.w / ts - ty0 + 1);
            off = emit_off[i];
        }
    }
    if (cnt <= EMIT_SERIAL) {
        for (int l = 0; l < cnt; ++l) {
            keys[off + l] = (uint32_t)((ty0 + l / ntx) * tiles_x + tx0 + l % ntx);
            vals[off + l] = (uint32_t)i;
        }
    }
    unsigned big = __ballot_sync(0xffffffffu, cnt > EMIT_SERIAL);
    while (big) {
        const int src = __ffs((int)big) - 1;
        big &= big - 1u;
        const int c = __shfl_sync(0xffffffffu, cnt, src), w = __shfl_sync(0xffffffffu, ntx, src);
        const int bx = __shfl_sync(0xffffffffu, tx0, src), by = __shfl_sync(0xffffffffu, ty0, src);
        const uint32_t o = __shfl_sync(0xffffffffu, off, src);
        const uint32_t id = (uint32_t)(i - lane + src);
        for (int l = lane; l < c; l += 32) {
            keys[o + l] = (uint32_t)((by + l / w) * tiles_x + bx + l % w);
            vals[o + l] = id;
        }
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
    w.total64 = (uint64_t*)take(256);
    w.emit_off = (uint32_t*)take((size_t)(n + 1) * 4);
    w.keys0 = (uint32_t*)take((size_t)cp * 4);
    w.keys1 = (uint32_t*)take((size_t)cp * 4);
    w.vals1 = (uint32_t*)take((size_t)cp * 4);
    w.table = (uint32_t*)take(radix_table_bytes(cp));
    const size_t s1 = scan_workspace_bytes(n), s2 = radix_scan_bytes(cp);
    w.scan_ws = take(s1 > s2 ? s1 : s2);
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
    // value buffers alternate between pair_gid and a scratch array so that the last pass lands in pair_gid
    uint32_t* const vbuf[2] = {pair_gid, w.vals1};
    uint32_t* const kbuf[2] = {w.keys0, w.keys1};
    const int cur = radix_passes(bits) & 1;   // emission target: after the passes the result is at index 0
    const int64_t pair_blocks = ceil_div(cap_pairs, 256);
    emit_pairs_kernel<<<(unsigned)ceil_div(n > 0 ? n : 1, 256), 256, 0, st>>>(rect4, w.emit_off, n, ts, tiles_x, counts, kbuf[cur], vbuf[cur]);
    GART_LAUNCH_CHECK();
    s = radix_sort_pairs(kbuf, vbuf, cur, bits, cap_pairs, counts + GART_CNT_PAIRS, 0u, counts + GART_CNT_ERROR, w.table, w.scan_ws,
                         w.total64, st);
    if (s != GART_OK) return s;
    tile_offsets_kernel<<<(unsigned)pair_blocks, 256, 0, st>>>(kbuf[0], counts, T, tile_off);
    GART_LAUNCH_CHECK();
    return GART_OK;
}

// ------------------------------------------------------------------------------------------------
// gart_tile_map_static: the tile map for callers that cannot provide scratch memory.
//
// Some hosts cannot allocate device memory at the point where they call this library: an engine that
// hands its whole device budget to its own arena at start-up and forbids later driver allocations,
// a plug-in running under a memory quota, a real-time loop in which an allocation (which may
// synchronise the device or fail on a fragmented heap) is not acceptable.  For them the scratch of
// gart_tile_map lives in a fixed array inside the library image: every GPU that loads libgart.so
// holds GART_TILE_MAP_STATIC_BYTES of device memory for it until the process exits.
//
// The array is shared by every call on a device and keeps the previous call's contents.  Nothing in
// the tile map relies on zero-initialised scratch (every word is written before it is read), so
// nothing needs clearing; but two calls that overlap on the GPU (different streams, no ordering
// between them) would race on it.
static __device__ __align__(256) unsigned char g_tile_map_scratch[GART_TILE_MAP_STATIC_BYTES];

// In host code the array's name is only a stand-in for the symbol, not a device address: the
// address a kernel can use comes from cudaGetSymbolAddress, asked once per device with that device
// current.
// Threads that make a device's first call together may all run the query; they store the same value, atomically.
static std::atomic<void*> g_tile_map_scratch_ptr[64];

extern "C" gart_status gart_tile_map_static(const gart_config* cfg, const int32_t* rect, int64_t n, int32_t width, int32_t height,
                                            uint32_t* tile_off, uint32_t* pair_gid, int64_t cap_pairs, uint32_t* counts,
                                            void* stream) {
    // the argument checks of gart_tile_map that the size test below relies on, then the size test: a problem beyond the
    // fixed array is refused before anything is launched
    if (!cfg || (cfg->tile_size != 8 && cfg->tile_size != 16)) return GART_ERR_INVALID_ARG;
    if (n < 0 || cap_pairs < 0 || width <= 0 || height <= 0) return GART_ERR_INVALID_ARG;
    if (gart_tile_map_workspace_bytes(n, width, height, cfg->tile_size, cap_pairs) > (size_t)GART_TILE_MAP_STATIC_BYTES)
        return GART_ERR_WORKSPACE_TOO_SMALL;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return GART_ERR_CUDA;
    void* p = g_tile_map_scratch_ptr[dev].load(std::memory_order_acquire);
    if (!p) {
        if (cudaGetSymbolAddress(&p, g_tile_map_scratch) != cudaSuccess || !p) return GART_ERR_CUDA;
        g_tile_map_scratch_ptr[dev].store(p, std::memory_order_release);
    }
    return gart_tile_map(cfg, rect, n, width, height, tile_off, pair_gid, cap_pairs, counts, p, (size_t)GART_TILE_MAP_STATIC_BYTES, stream);
}
