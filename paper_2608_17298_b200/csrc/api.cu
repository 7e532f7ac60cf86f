// Host-side conveniences of the C ABI: reading the counts block and the end-to-end call for
// callers that hold host arrays.
#include "common.cuh"

namespace gart {

struct HostArena {
    float *mean, *scale, *quat, *opacity, *sh, *pre, *color, *t_final, *lt, *dL_dC, *grad;
    int32_t* rect;
    uint8_t* cls;
    uint32_t *counts, *tile_off, *pair_gid, *slot_of_gid, *gid_of_slot, *hit_count, *ray_off;
    void *view, *ws;
    size_t view_bytes, ws_bytes;
    size_t bytes;
};

static HostArena arena_layout(void* base, int64_t n, int K, int width, int height, int ts, int64_t cap_pairs, int64_t cap_hits) {
    HostArena a;
    char* p = (char*)base;
    size_t off = 0;
    auto take = [&](size_t b) { void* r = p ? (void*)(p + off) : nullptr; off += align256(b > 0 ? b : 1); return r; };
    const int64_t nn = n > 0 ? n : 1, cp = cap_pairs > 0 ? cap_pairs : 1, ch = cap_hits > 0 ? cap_hits : 1;
    const int64_t hw = (int64_t)width * height;
    const int T = ((width + ts - 1) / ts) * ((height + ts - 1) / ts);
    a.mean = (float*)take(nn * 12); a.scale = (float*)take(nn * 12); a.quat = (float*)take(nn * 16);
    a.opacity = (float*)take(nn * 4); a.sh = (float*)take(nn * 12 * K);
    a.rect = (int32_t*)take(nn * 16); a.cls = (uint8_t*)take(nn); a.pre = (float*)take(nn * 4 * (size_t)(((20 + 3 * K + 3) & ~3) + 8 + 4));
    a.slot_of_gid = (uint32_t*)take(nn * 4); a.gid_of_slot = (uint32_t*)take(nn * 4);
    a.counts = (uint32_t*)take(GART_COUNTS_WORDS * 4);
    a.tile_off = (uint32_t*)take((size_t)(T + 1) * 4); a.pair_gid = (uint32_t*)take(cp * 4);
    a.view_bytes = gart_view_bytes(nn, width, height, ts, cap_pairs);
    a.view = take(a.view_bytes);
    a.color = (float*)take(hw * 12); a.t_final = (float*)take(hw * 4); a.hit_count = (uint32_t*)take(hw * 4);
    a.lt = (float*)take(ch * 16); a.ray_off = (uint32_t*)take((hw + 1) * 4);
    a.dL_dC = (float*)take(hw * 12); a.grad = (float*)take(nn * GART_GRAD_WORDS * 4);
    a.ws_bytes = gart_workspace_bytes(nn, width, height, ts, cap_pairs, cap_hits);
    a.ws = take(a.ws_bytes);
    a.bytes = off;
    return a;
}

}  // namespace gart

extern "C" gart_status gart_read_counts(const uint32_t* counts, uint32_t* counts_host, void* stream) {
    if (!counts || !counts_host) return GART_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemcpyAsync(counts_host, counts, GART_COUNTS_WORDS * sizeof(uint32_t), cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return GART_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return GART_ERR_CUDA;
    return GART_OK;
}

extern "C" gart_status gart_sync_status(const uint32_t* counts, uint32_t* counts_host, void* stream) {
    uint32_t local[GART_COUNTS_WORDS];
    uint32_t* h = counts_host ? counts_host : local;
    const gart_status s = gart_read_counts(counts, h, stream);
    if (s != GART_OK) return s;
    if (h[GART_CNT_ERROR] & GART_ERRBIT_TIMEOUT) return GART_ERR_TIMEOUT;
    if (h[GART_CNT_ERROR]) return GART_ERR_CAPACITY_EXCEEDED;
    return GART_OK;
}

extern "C" size_t gart_workspace_bytes(int64_t n, int32_t width, int32_t height, int32_t tile_size, int64_t cap_pairs, int64_t cap_hits) {
    const int64_t nn = n > 0 ? n : 1;
    size_t b = gart_bounds_workspace_bytes(nn);
    const size_t w1 = gart_tile_map_workspace_bytes(nn, width, height, tile_size, cap_pairs);
    const size_t w2 = gart_forward_workspace_bytes(width, height, tile_size, cap_pairs, cap_hits);
    const size_t w3 = gart_backward_hybrid_workspace_bytes(nn, 3);   // (the largest backward need: the hybrid pass at SH degree 3)
    if (w1 > b) b = w1;
    if (w2 > b) b = w2;
    if (w3 > b) b = w3;
    return b;
}

extern "C" size_t gart_view_host_arena_bytes(int64_t n, int32_t sh_degree, int32_t width, int32_t height, int32_t tile_size,
                                             int64_t cap_pairs, int64_t cap_hits) {
    if (sh_degree < 0 || sh_degree > 3 || (tile_size != 8 && tile_size != 16) || width <= 0 || height <= 0) return 0;
    const int K = (sh_degree + 1) * (sh_degree + 1);
    return gart::arena_layout(nullptr, n, K, width, height, tile_size, cap_pairs, cap_hits).bytes;
}

extern "C" gart_status gart_view_host_async(const gart_config* cfg, const gart_gaussians* gh, const gart_camera* cam,
                                            const float* dL_dcolor_host, float* color_host, float* grad_host,
                                            int64_t cap_pairs, int64_t cap_hits, uint32_t* counts_host,
                                            void* arena, size_t arena_bytes, void* stream) {
    using namespace gart;
    if (!cfg || !gh || !cam || !dL_dcolor_host || !color_host || !counts_host || !arena) return GART_ERR_INVALID_ARG;
    if (gh->n < 0 || gh->sh_degree < 0 || gh->sh_degree > 3) return GART_ERR_INVALID_ARG;
    if (cfg->tile_size != 8 && cfg->tile_size != 16) return GART_ERR_INVALID_ARG;
    if (cam->width <= 0 || cam->height <= 0) return GART_ERR_INVALID_ARG;
    if (gh->n > 0 && (!gh->mean || !gh->scale || !gh->quat || !gh->opacity || !gh->sh || !grad_host)) return GART_ERR_INVALID_ARG;
    if ((uintptr_t)arena & 255) return GART_ERR_INVALID_ARG;
    const int K = (gh->sh_degree + 1) * (gh->sh_degree + 1);
    const int64_t n = gh->n, hw = (int64_t)cam->width * cam->height;
    HostArena a = arena_layout(arena, n, K, cam->width, cam->height, cfg->tile_size, cap_pairs, cap_hits);
    if (a.bytes > arena_bytes) return GART_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t st = (cudaStream_t)stream;
#define GART_H2D(dst, src, bytes) \
    if ((bytes) > 0 && cudaMemcpyAsync(dst, src, bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return GART_ERR_CUDA
    GART_H2D(a.mean, gh->mean, (size_t)n * 12);
    GART_H2D(a.scale, gh->scale, (size_t)n * 12);
    GART_H2D(a.quat, gh->quat, (size_t)n * 16);
    GART_H2D(a.opacity, gh->opacity, (size_t)n * 4);
    GART_H2D(a.sh, gh->sh, (size_t)n * 12 * K);
    GART_H2D(a.dL_dC, dL_dcolor_host, (size_t)hw * 12);
#undef GART_H2D
    gart_gaussians gd = *gh;
    gd.mean = a.mean; gd.scale = a.scale; gd.quat = a.quat; gd.opacity = a.opacity; gd.sh = a.sh;
    gart_status s = gart_bounds(cfg, &gd, cam, a.rect, a.cls, a.pre, a.slot_of_gid, a.gid_of_slot, a.counts, a.ws, a.ws_bytes, stream);
    if (s != GART_OK) return s;
    s = gart_tile_map(cfg, a.rect, n, cam->width, cam->height, a.tile_off, a.pair_gid, cap_pairs, a.counts, a.ws, a.ws_bytes, stream);
    if (s != GART_OK) return s;
    s = gart_forward(cfg, &gd, cam, a.pre, a.slot_of_gid, a.gid_of_slot, a.tile_off, a.pair_gid, cap_pairs, a.color, a.t_final, a.hit_count,
                     a.lt, cap_hits, a.ray_off, nullptr, nullptr, a.view, a.view_bytes, a.counts, a.ws, a.ws_bytes, stream);
    if (s != GART_OK) return s;
    if (cfg->lt_layout == GART_LT_TILE_MAJOR)
        s = gart_backward_tile(cfg, &gd, cam, a.pre, a.slot_of_gid, a.gid_of_slot, a.tile_off, a.view, a.view_bytes, cap_pairs, a.lt, a.dL_dC,
                               a.grad, a.counts, a.ws, a.ws_bytes, stream);
    else
        s = gart_backward(cfg, &gd, cam, a.pre, a.slot_of_gid, a.gid_of_slot, a.tile_off, a.view, a.view_bytes, cap_pairs, a.lt, a.dL_dC,
                          a.grad, a.counts, a.ws, a.ws_bytes, stream);
    if (s != GART_OK) return s;
    if (cudaMemcpyAsync(color_host, a.color, (size_t)hw * 12, cudaMemcpyDeviceToHost, st) != cudaSuccess) return GART_ERR_CUDA;
    if (n > 0 && cudaMemcpyAsync(grad_host, a.grad, (size_t)n * GART_GRAD_WORDS * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return GART_ERR_CUDA;
    if (cudaMemcpyAsync(counts_host, a.counts, GART_COUNTS_WORDS * sizeof(uint32_t), cudaMemcpyDeviceToHost, st) != cudaSuccess) return GART_ERR_CUDA;
    return GART_OK;
}

extern "C" gart_status gart_counts_status(const uint32_t* counts_host) {
    if (!counts_host) return GART_ERR_INVALID_ARG;
    if (counts_host[GART_CNT_ERROR] & GART_ERRBIT_TIMEOUT) return GART_ERR_TIMEOUT;
    if (counts_host[GART_CNT_ERROR]) return GART_ERR_CAPACITY_EXCEEDED;
    return GART_OK;
}

extern "C" gart_status gart_view_host(const gart_config* cfg, const gart_gaussians* gh, const gart_camera* cam,
                                      const float* dL_dcolor_host, float* color_host, float* grad_host,
                                      int64_t cap_pairs, int64_t cap_hits, uint32_t* counts_host,
                                      void* arena, size_t arena_bytes, void* stream) {
    const gart_status s = gart_view_host_async(cfg, gh, cam, dL_dcolor_host, color_host, grad_host, cap_pairs, cap_hits, counts_host, arena,
                                               arena_bytes, stream);
    if (s != GART_OK) return s;
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return GART_ERR_CUDA;
    return gart_counts_status(counts_host);
}
