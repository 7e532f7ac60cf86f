// gart_forward: ray evaluation (Sec. 3.2-3.3) over the tile lists and the compact intermediate
// buffer (Sec. 4.2-4.3).
//
// The paper finds the hits of a ray with hardware ray tracing over a BVH of bounded proxies;
// here candidates come from the tile lists (same hit set: a hit is alpha >= alpha_min, i.e.
// the ray meets the clamped ellipsoid whose projection the rectangle bounds).  Four phases:
//   1. fwd_mask   block per tile, thread per pixel: every pixel of the tile evaluates every
//                 Gaussian of the tile list (records broadcast from shared memory); a warp
//                 ballot yields the pair's hit mask; pixels count their hits.
//   2. scans      hits per pair -> pair_lt_off (slot base of every pair in LT: pair-major,
//                 then pixel -- each hit owns one slot, so forward writes never collide and
//                 the backward thread of a pair reads one contiguous run); hits per ray ->
//                 ray_off.
//   3. fwd_keys   block per tile, thread per pixel: for every set mask bit compute t*, alpha
//                 and the SH colour (SH coefficients staged per tile in shared memory) and
//                 append (t*, index) keys plus payload to the ray's segment.
//   4. fwd_sort_sweep  warp per ray: sort the segment by (t*, id), scan the transmittance
//                 front to back, then sum colour back to front so that each hit gets the
//                 colour composited behind it without cancellation; write LT, C, T_final.
#include "common.cuh"

namespace gart {

// ------------------------------------------------------------------------------------------ phase 1
template <int TS>
__global__ void __launch_bounds__(TS * TS) fwd_mask_kernel(const float4* __restrict__ pre4, const uint32_t* __restrict__ tile_off,
                                                           const uint32_t* __restrict__ pair_gid, CamF cam, float alpha_min,
                                                           uint32_t* __restrict__ pair_mask, uint32_t* __restrict__ hit_count,
                                                           uint32_t* __restrict__ counts) {
    constexpr int NT = TS * TS, MW = NT / 32, CH = 64;
    __shared__ float4 sp[CH * 5];
    __shared__ uint32_t smax[NT / 32];
    if (counts[GART_CNT_ERROR]) return;
    const int tile = blockIdx.x;
    const int tx = tile % cam.tiles_x, ty = tile / cam.tiles_x;
    const int p = threadIdx.x, lane = p & 31, warp = p >> 5;
    const int x = tx * TS + p % TS, y = ty * TS + p / TS;
    const bool inside = x < cam.width && y < cam.height;
    const uint32_t begin = tile_off[tile], end = tile_off[tile + 1];
    uint32_t cnt = 0;
    for (uint32_t base = begin; base < end; base += CH) {
        const int nb = min((uint32_t)CH, end - base);
        for (int i = p; i < nb * 5; i += NT) {
            const int pair = i / 5, q = i - pair * 5;
            sp[i] = __ldg(pre4 + (size_t)__ldg(pair_gid + base + pair) * 5 + q);
        }
        __syncthreads();
        for (int j = 0; j < nb; ++j) {
            const PreRec P = unpack_pre(sp[j * 5], sp[j * 5 + 1], sp[j * 5 + 2], sp[j * 5 + 3], sp[j * 5 + 4]);
            const RayEval r = ray_eval(P, (float)(x - P.ix) - P.rx, (float)(y - P.iy) - P.ry);
            const bool hit = inside && (r.alpha >= alpha_min) && (r.tnum > 0.0f);
            const unsigned b = __ballot_sync(0xffffffffu, hit);
            if (lane == 0) pair_mask[(size_t)(base + j) * MW + warp] = b;
            cnt += hit ? 1u : 0u;
        }
        __syncthreads();
    }
    if (inside) hit_count[(size_t)y * cam.width + x] = cnt;
    uint32_t m = cnt;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_down_sync(0xffffffffu, m, o));
    if (lane == 0) smax[warp] = m;
    __syncthreads();
    if (p == 0) {
        for (int w = 1; w < NT / 32; ++w) m = max(m, smax[w]);
        if (m) atomicMax(&counts[GART_CNT_MAX_RAY_HITS], m);
    }
}

// ------------------------------------------------------------------------------------------ phase 2
struct PairHitsF {
    const uint32_t* mask;
    const uint32_t* counts;
    int mw;
    __device__ __forceinline__ uint32_t operator()(int64_t i) const {
        if (counts[GART_CNT_ERROR] || i >= counts[GART_CNT_PAIRS]) return 0u;
        uint32_t s = 0;
        for (int q = 0; q < mw; ++q) s += __popc(mask[(size_t)i * mw + q]);
        return s;
    }
};

struct RayHitsF {
    const uint32_t* hit_count;
    const uint32_t* counts;
    __device__ __forceinline__ uint32_t operator()(int64_t i) const {
        return counts[GART_CNT_ERROR] ? 0u : hit_count[i];
    }
};

__global__ void hits_total_kernel(const uint64_t* total64, int64_t cap_hits, uint32_t* counts) {
    const uint64_t H = total64[0];
    counts[GART_CNT_HITS] = H > 0xffffffffull ? 0xffffffffu : (uint32_t)H;
    if (H > (uint64_t)cap_hits) atomicOr(&counts[GART_CNT_ERROR], GART_ERRBIT_HITS);
}

// ------------------------------------------------------------------------------------------ phase 3
template <int TS, int DEG>
__global__ void __launch_bounds__(TS * TS) fwd_keys_kernel(const float4* __restrict__ pre4, const float* __restrict__ sh,
                                                           const uint32_t* __restrict__ tile_off, const uint32_t* __restrict__ pair_gid,
                                                           const uint32_t* __restrict__ pair_mask, const uint32_t* __restrict__ pair_lt_off,
                                                           const uint32_t* __restrict__ ray_off, CamF cam,
                                                           uint64_t* __restrict__ keys, float4* __restrict__ payload,
                                                           uint32_t* __restrict__ hit_gid, uint32_t* __restrict__ hit_slot,
                                                           const uint32_t* __restrict__ counts) {
    constexpr int NT = TS * TS, MW = NT / 32, CH = 32, K = (DEG + 1) * (DEG + 1), SW = 3 * K;
    __shared__ float4 sp[CH * 5];
    __shared__ float ssh[CH * SW];
    __shared__ uint32_t smask[CH * MW];
    __shared__ uint32_t sbase[CH];
    __shared__ uint32_t sgid[CH];
    if (counts[GART_CNT_ERROR]) return;
    const int tile = blockIdx.x;
    const int tx = tile % cam.tiles_x, ty = tile / cam.tiles_x;
    const int p = threadIdx.x, lane = p & 31, warp = p >> 5;
    const int x = tx * TS + p % TS, y = ty * TS + p / TS;
    const bool inside = x < cam.width && y < cam.height;
    const uint32_t begin = tile_off[tile], end = tile_off[tile + 1];
    if (begin == end) return;
    float Y[K];
    sh_basis<K>(pixel_dir(cam, min(x, cam.width - 1), min(y, cam.height - 1)), Y);
    size_t w = inside ? (size_t)ray_off[(size_t)y * cam.width + x] : 0;
    uint32_t local = 0;
    for (uint32_t base = begin; base < end; base += CH) {
        const int nb = min((uint32_t)CH, end - base);
        for (int i = p; i < nb; i += NT) {
            sgid[i] = __ldg(pair_gid + base + i);
            sbase[i] = __ldg(pair_lt_off + base + i);
        }
        for (int i = p; i < nb * MW; i += NT) smask[i] = __ldg(pair_mask + (size_t)base * MW + i);
        __syncthreads();
        for (int i = p; i < nb * 5; i += NT) {
            const int pair = i / 5, q = i - pair * 5;
            sp[i] = __ldg(pre4 + (size_t)sgid[pair] * 5 + q);
        }
        for (int i = p; i < nb * SW; i += NT) {
            const int pair = i / SW, q = i - pair * SW;
            ssh[i] = __ldg(sh + (size_t)sgid[pair] * SW + q);
        }
        __syncthreads();
        for (int j = 0; j < nb; ++j) {
            const uint32_t word = smask[j * MW + warp];
            if ((word >> lane) & 1u) {
                const PreRec P = unpack_pre(sp[j * 5], sp[j * 5 + 1], sp[j * 5 + 2], sp[j * 5 + 3], sp[j * 5 + 4]);
                const RayEval r = ray_eval(P, (float)(x - P.ix) - P.rx, (float)(y - P.iy) - P.ry);
                const float t = fmaxf(r.tnum * r.inv_a, 0.0f);
                float c0 = 0.5f, c1 = 0.5f, c2 = 0.5f;
                const float* s = ssh + j * SW;
#pragma unroll
                for (int k = 0; k < K; ++k) {
                    c0 = fmaf(Y[k], s[3 * k], c0);
                    c1 = fmaf(Y[k], s[3 * k + 1], c1);
                    c2 = fmaf(Y[k], s[3 * k + 2], c2);
                }
                uint32_t slot = sbase[j] + __popc(word & ((1u << lane) - 1u));
                for (int q = 0; q < warp; ++q) slot += __popc(smask[j * MW + q]);
                keys[w] = ((uint64_t)__float_as_uint(t) << 32) | (uint64_t)local;
                payload[w] = make_float4(r.alpha, fmaxf(c0, 0.0f), fmaxf(c1, 0.0f), fmaxf(c2, 0.0f));
                hit_gid[w] = sgid[j];
                hit_slot[w] = slot;
                ++w;
                ++local;
            }
        }
        __syncthreads();
    }
}

// ------------------------------------------------------------------------------------------ phase 4
constexpr int SORT_CAP = 1024;   // keys per warp held in shared memory; longer rays sort in global memory
constexpr int SWEEP_WARPS = 4;

__device__ __forceinline__ void cmp_swap(uint64_t* a, int i, int l) {
    const uint64_t x = a[i], y = a[l];
    if (x > y) { a[i] = y; a[l] = x; }
}

// Ascending sort of a[0..n) by one warp.  Sorting network whose compare-exchanges all put the
// smaller key at the lower index, so positions >= n act as +infinity without being stored.
__device__ __forceinline__ void warp_sort(uint64_t* a, int n, int lane) {
    int np2 = 1;
    while (np2 < n) np2 <<= 1;
    const int half = np2 >> 1;
    for (int k = 2; k <= np2; k <<= 1) {
        const int hk = k >> 1;
        for (int t = lane; t < half; t += 32) {
            const int blk = t / hk, off = t - blk * hk;
            const int i = blk * k + off, l = blk * k + k - 1 - off;
            if (l < n) cmp_swap(a, i, l);
        }
        __syncwarp();
        for (int j = k >> 2; j >= 1; j >>= 1) {
            for (int t = lane; t < half; t += 32) {
                const int i = 2 * j * (t / j) + (t % j), l = i + j;
                if (l < n) cmp_swap(a, i, l);
            }
            __syncwarp();
        }
    }
}

__global__ void __launch_bounds__(SWEEP_WARPS * 32) fwd_sort_sweep_kernel(const uint32_t* __restrict__ ray_off, uint64_t* __restrict__ keys,
                                                                          const float4* __restrict__ payload, const uint32_t* __restrict__ hit_gid,
                                                                          const uint32_t* __restrict__ hit_slot, int64_t n_rays,
                                                                          float bg0, float bg1, float bg2,
                                                                          float* __restrict__ color, float* __restrict__ t_final,
                                                                          float4* __restrict__ lt, uint32_t* __restrict__ ray_gid,
                                                                          uint32_t* __restrict__ ray_slot, const uint32_t* __restrict__ counts) {
    __shared__ uint64_t skeys[SWEEP_WARPS][SORT_CAP];
    if (counts[GART_CNT_ERROR]) return;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t r = (int64_t)blockIdx.x * SWEEP_WARPS + warp;
    if (r >= n_rays) return;
    const size_t b = ray_off[r];
    const int n = (int)(ray_off[r + 1] - ray_off[r]);
    if (n == 0) {
        if (lane == 0) {
            color[3 * r] = bg0; color[3 * r + 1] = bg1; color[3 * r + 2] = bg2;
            t_final[r] = 1.0f;
        }
        return;
    }
    uint64_t* kp;
    if (n <= SORT_CAP) {
        kp = skeys[warp];
        for (int i = lane; i < n; i += 32) kp[i] = keys[b + i];
    } else {
        kp = keys + b;
    }
    __syncwarp();
    warp_sort(kp, n, lane);

    // front to back: transmittance in front of every hit (Eq. 7); stored in the key's high word
    float carryT = 1.0f;
    for (int base = 0; base < n; base += 32) {
        const int i = base + lane;
        const bool valid = i < n;
        const uint32_t c = valid ? (uint32_t)kp[i] : 0u;
        const float alpha = valid ? payload[b + c].x : 0.0f;
        float prod = 1.0f - alpha;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const float t = __shfl_up_sync(0xffffffffu, prod, o);
            if (lane >= o) prod *= t;
        }
        float excl = __shfl_up_sync(0xffffffffu, prod, 1);
        if (lane == 0) excl = 1.0f;
        const float T = carryT * excl;
        if (valid) kp[i] = ((uint64_t)__float_as_uint(T) << 32) | (uint64_t)c;
        carryT *= __shfl_sync(0xffffffffu, prod, 31);
    }
    __syncwarp();
    const float Tfin = carryT;

    // back to front: colour composited behind every hit (background term first)
    float k0 = Tfin * bg0, k1 = Tfin * bg1, k2 = Tfin * bg2;
    for (int base = 0; base < n; base += 32) {
        const int i = n - 1 - (base + lane);
        const bool valid = i >= 0;
        float T = 0.0f, v0 = 0.0f, v1 = 0.0f, v2 = 0.0f;
        uint32_t c = 0;
        if (valid) {
            const uint64_t key = kp[i];
            c = (uint32_t)key;
            T = __uint_as_float((uint32_t)(key >> 32));
            const float4 pl = payload[b + c];
            const float wgt = T * pl.x;
            v0 = wgt * pl.y; v1 = wgt * pl.z; v2 = wgt * pl.w;
        }
        float s0 = v0, s1 = v1, s2 = v2;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const float a0 = __shfl_up_sync(0xffffffffu, s0, o);
            const float a1 = __shfl_up_sync(0xffffffffu, s1, o);
            const float a2 = __shfl_up_sync(0xffffffffu, s2, o);
            if (lane >= o) { s0 += a0; s1 += a1; s2 += a2; }
        }
        float e0 = __shfl_up_sync(0xffffffffu, s0, 1), e1 = __shfl_up_sync(0xffffffffu, s1, 1), e2 = __shfl_up_sync(0xffffffffu, s2, 1);
        if (lane == 0) { e0 = 0.0f; e1 = 0.0f; e2 = 0.0f; }
        if (valid) {
            const uint32_t slot = hit_slot[b + c];
            lt[slot] = make_float4(k0 + e0, k1 + e1, k2 + e2, T);
            ray_gid[b + i] = hit_gid[b + c];
            ray_slot[b + i] = slot;
        }
        k0 += __shfl_sync(0xffffffffu, s0, 31);
        k1 += __shfl_sync(0xffffffffu, s1, 31);
        k2 += __shfl_sync(0xffffffffu, s2, 31);
    }
    if (lane == 0) {
        color[3 * r] = k0; color[3 * r + 1] = k1; color[3 * r + 2] = k2;
        t_final[r] = Tfin;
    }
}

// ------------------------------------------------------------------------------------------ host
struct ForwardWs {
    uint64_t* total64;
    void* scan_ws;
    uint64_t* keys;
    float4* payload;
    uint32_t *hit_gid, *hit_slot;
    size_t bytes;
};

static ForwardWs forward_layout(void* base, int64_t n_rays, int64_t cap_pairs, int64_t cap_hits) {
    ForwardWs w;
    char* p = (char*)base;
    size_t off = 0;
    auto take = [&](size_t b) { void* r = p ? (void*)(p + off) : nullptr; off += align256(b); return r; };
    const int64_t ch = cap_hits > 0 ? cap_hits : 1;
    w.total64 = (uint64_t*)take(256);
    w.scan_ws = take(scan_workspace_bytes(cap_pairs > n_rays ? cap_pairs : n_rays));
    w.keys = (uint64_t*)take((size_t)ch * 8);
    w.payload = (float4*)take((size_t)ch * 16);
    w.hit_gid = (uint32_t*)take((size_t)ch * 4);
    w.hit_slot = (uint32_t*)take((size_t)ch * 4);
    w.bytes = off;
    return w;
}

template <int TS>
static gart_status launch_keys(int deg, int T, cudaStream_t st, const float4* pre4, const float* sh, const uint32_t* tile_off,
                               const uint32_t* pair_gid, const uint32_t* pair_mask, const uint32_t* pair_lt_off,
                               const uint32_t* ray_off, const CamF& cam, const ForwardWs& w, const uint32_t* counts) {
#define GART_KEYS(D)                                                                                                   \
    fwd_keys_kernel<TS, D><<<T, TS * TS, 0, st>>>(pre4, sh, tile_off, pair_gid, pair_mask, pair_lt_off, ray_off, cam, \
                                                  w.keys, w.payload, w.hit_gid, w.hit_slot, counts)
    switch (deg) {
        case 0: GART_KEYS(0); break;
        case 1: GART_KEYS(1); break;
        case 2: GART_KEYS(2); break;
        default: GART_KEYS(3); break;
    }
#undef GART_KEYS
    GART_LAUNCH_CHECK();
    return GART_OK;
}

}  // namespace gart

extern "C" size_t gart_forward_workspace_bytes(int32_t width, int32_t height, int32_t tile_size, int64_t cap_pairs, int64_t cap_hits) {
    (void)tile_size;
    return gart::forward_layout(nullptr, (int64_t)width * height, cap_pairs > 0 ? cap_pairs : 1, cap_hits).bytes;
}

extern "C" gart_status gart_forward(const gart_config* cfg, const gart_gaussians* g, const gart_camera* cam, const float* pre,
                                    const uint32_t* tile_off, const uint32_t* pair_gid, int64_t cap_pairs,
                                    float* color, float* t_final, uint32_t* hit_count,
                                    uint32_t* pair_mask, uint32_t* pair_lt_off, float* lt, int64_t cap_hits,
                                    uint32_t* ray_off, uint32_t* ray_gid, uint32_t* ray_slot, uint32_t* counts,
                                    void* workspace, size_t workspace_bytes, void* stream) {
    using namespace gart;
    if (!cfg || !g || !cam || !tile_off || !color || !t_final || !hit_count || !pair_lt_off || !ray_off || !counts)
        return GART_ERR_INVALID_ARG;
    if (cfg->tile_size != 8 && cfg->tile_size != 16) return GART_ERR_INVALID_ARG;
    if (g->sh_degree < 0 || g->sh_degree > 3 || cap_pairs < 0 || cap_hits < 0) return GART_ERR_INVALID_ARG;
    if (cap_hits > 0xfffffff0ll || cap_pairs > 0xfffffff0ll) return GART_ERR_INVALID_ARG;
    if (cap_pairs > 0 && (!pair_gid || !pair_mask || !pre || !g->sh)) return GART_ERR_INVALID_ARG;
    if (cap_hits > 0 && (!lt || !ray_gid || !ray_slot)) return GART_ERR_INVALID_ARG;
    if (!workspace || ((uintptr_t)workspace & 255)) return GART_ERR_INVALID_ARG;
    const int ts = cfg->tile_size;
    const CamF cf = make_camf(cam, ts);
    const int T = cf.tiles_x * cf.tiles_y;
    const int64_t n_rays = (int64_t)cam->width * cam->height;
    const int64_t cp = cap_pairs > 0 ? cap_pairs : 1;
    ForwardWs w = forward_layout(workspace, n_rays, cp, cap_hits);
    if (w.bytes > workspace_bytes) return GART_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t st = (cudaStream_t)stream;
    const float4* pre4 = reinterpret_cast<const float4*>(pre);

    if (ts == 8) fwd_mask_kernel<8><<<T, 64, 0, st>>>(pre4, tile_off, pair_gid, cf, cfg->alpha_min, pair_mask, hit_count, counts);
    else fwd_mask_kernel<16><<<T, 256, 0, st>>>(pre4, tile_off, pair_gid, cf, cfg->alpha_min, pair_mask, hit_count, counts);
    GART_LAUNCH_CHECK();

    PairHitsF pf{pair_mask, counts, ts * ts / 32};
    gart_status s = exclusive_scan(pf, cp, pair_lt_off, w.total64, w.scan_ws, st);
    if (s != GART_OK) return s;
    RayHitsF rf{hit_count, counts};
    s = exclusive_scan(rf, n_rays, ray_off, w.total64, w.scan_ws, st);
    if (s != GART_OK) return s;
    hits_total_kernel<<<1, 1, 0, st>>>(w.total64, cap_hits, counts);
    GART_LAUNCH_CHECK();

    if (ts == 8) s = launch_keys<8>(g->sh_degree, T, st, pre4, g->sh, tile_off, pair_gid, pair_mask, pair_lt_off, ray_off, cf, w, counts);
    else s = launch_keys<16>(g->sh_degree, T, st, pre4, g->sh, tile_off, pair_gid, pair_mask, pair_lt_off, ray_off, cf, w, counts);
    if (s != GART_OK) return s;

    const int64_t blocks = ceil_div(n_rays, SWEEP_WARPS);
    fwd_sort_sweep_kernel<<<(unsigned)blocks, SWEEP_WARPS * 32, 0, st>>>(ray_off, w.keys, w.payload, w.hit_gid, w.hit_slot, n_rays,
                                                                         cfg->background[0], cfg->background[1], cfg->background[2],
                                                                         color, t_final, reinterpret_cast<float4*>(lt), ray_gid,
                                                                         ray_slot, counts);
    GART_LAUNCH_CHECK();
    return GART_OK;
}
