// gart_backward_hybrid: the hybrid backward (Sec. 4.4 "Hybrid approach", "Hybrid" of Sec. 5.1).
//
// Colour gradients (dL/dsh, 3K of the 11 + 3K words, where most of the atomic traffic of a pixel-centric pass
// goes) are accumulated primitive-centric, one thread per (tile, Gaussian) pair, from an intermediate buffer
// that holds ONE word per hit: the blending weight w = T alpha with the clamp flags (word 3 of the 16-byte
// entry).  The remaining terms (mean, scale, quaternion, opacity) are accumulated pixel-centric: one thread per
// ray walks the ray's hits in compositing order and issues scalar atomics per hit.  Memory per hit: 4 bytes of
// LT + 4 bytes of the ray's ordered id list (the paper re-traces the ray instead of keeping that list).
//
// The pixel-centric pass needs, per hit, T in front of it and the colour composited behind it.  It walks the
// ray twice: front to back for log T_final = sum log(1 - alpha), then back to front with
//     log T_i = log T_{i+1} - log(1 - alpha_i)          (no underflow, no division by a vanishing T)
//     Cb_{i-1} = alpha_i c_i + (1 - alpha_i) Cb_i       (colour behind, not premultiplied; Cb_last = background)
// so that alpha dL/dalpha = w_i <dL/dC, c_i - Cb_i>  (Eq. 6-8); nothing is a difference of nearly equal sums.
#include "backward_common.cuh"
#include "view_layout.cuh"

namespace gart {

constexpr int HYB_WARPS = 4;
constexpr int HYB_THREADS = HYB_WARPS * 32;
constexpr int HYB_CHUNK = 16;                       // weight words per lane and per pipeline stage
constexpr int HYB_STAGES = 2;
constexpr int HYB_STAGE_WORDS = HYB_CHUNK * 32;     // 2 KB per stage

// ------------------------------------------------------------------------------- colour part, primitive-centric
template <int TS, int DEG>
__global__ void __launch_bounds__(HYB_THREADS) bwd_sh_kernel(const uint32_t* __restrict__ tile_off, const uint32_t* __restrict__ rank_sid,
                                                             const uint32_t* __restrict__ rank_mask, const uint32_t* __restrict__ rank_gstart,
                                                             const uint32_t* __restrict__ tile_lt_base, const float* __restrict__ lt_w,
                                                             const float* __restrict__ dL_dC, CamF cam, Gacc gacc,
                                                             uint32_t* __restrict__ counts, const uint32_t wait_limit) {
    constexpr int NT = TS * TS, MW = NT / 32, K = (DEG + 1) * (DEG + 1), SW = 3 * K, PIXF4 = PixLayout<TS>::F4;
    constexpr int AW = (11 + SW + 3) & ~3;
    __shared__ __align__(128) float stage[HYB_WARPS][HYB_STAGES][HYB_STAGE_WORDS];
    __shared__ __align__(16) float4 spix[PIXF4];
    __shared__ __align__(8) uint64_t bars[HYB_WARPS][HYB_STAGES];
    if (counts[GART_CNT_ERROR]) return;
    const int tile = blockIdx.x;
    const uint32_t begin = tile_off[tile], n = tile_off[tile + 1] - begin;
    if (n == 0) return;
    const int x0 = (tile % cam.tiles_x) * TS, y0 = (tile / cam.tiles_x) * TS;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) {
#pragma unroll
        for (int q = 0; q < HYB_STAGES; ++q) mbar_init(smem_u32(&bars[warp][q]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int t = threadIdx.x; t < 2 * NT; t += HYB_THREADS) {
        const int p = t >> 1, h = t & 1;
        const int x = x0 + p % TS, y = y0 + p / TS;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (x < cam.width && y < cam.height) {
            if (h) {
                const float* gp = dL_dC + ((size_t)y * cam.width + x) * 3;
                v.x = gp[0]; v.y = gp[1]; v.z = gp[2];
            } else {
                const float3 d = pixel_dir(cam, x, y);
                v.x = d.x; v.y = d.y; v.z = d.z;
            }
        }
#pragma unroll
        for (int c = 0; c < PixLayout<TS>::COPIES; ++c) spix[PixLayout<TS>::index(p, h, c)] = v;
    }
    __syncthreads();

    const float* lt_tile = lt_w + tile_lt_base[tile];
    const float4* spix_lane = spix + (lane & (PixLayout<TS>::COPIES - 1));
    const uint32_t stage_addr = smem_u32(&stage[warp][0][0]);
    const uint32_t bar_addr = smem_u32(&bars[warp][0]);
    const uint64_t pol_stream = l2_policy_evict_first(), pol_keep = l2_policy_evict_last();
    // the same pipeline as the full pair kernel: unit u uses stage u % HYB_STAGES with parity (u / HYB_STAGES) & 1
    uint32_t unit = 0, produced = 0;
    int pw = 0, pk = 0;
    auto produce = [&](const GroupDesc<MW>& a, const GroupDesc<MW>& b, const GroupDesc<MW>& c, const int maxw) {
        while (produced - unit < (uint32_t)HYB_STAGES && pw <= maxw) {
            int cm;
            uint32_t gs;
            if (pw == 0) { cm = a.cmax; gs = a.gstart; }
            else if (pw == 1) { cm = b.cmax; gs = b.gstart; }
            else { cm = c.cmax; gs = c.gstart; }
            if (cm == 0) break;
            if (pk * HYB_CHUNK >= cm) { ++pw; pk = 0; continue; }
            if (lane == 0) {
                const int ne = min(HYB_CHUNK, cm - pk * HYB_CHUNK);
                const uint32_t bytes = (uint32_t)ne * 128u, s = produced % HYB_STAGES;
                mbar_expect_tx(bar_addr + 8u * s, bytes);
                bulk_g2s_hint(stage_addr + s * (HYB_STAGE_WORDS * 4u), lt_tile + gs + (size_t)pk * HYB_STAGE_WORDS, bytes, bar_addr + 8u * s, pol_stream);
            }
            ++produced;
            ++pk;
        }
    };
    auto fail = [&]() {
        if (lane == 0) atomicOr(&counts[GART_CNT_ERROR], GART_ERRBIT_TIMEOUT);
        for (uint32_t u = unit; u != produced; ++u) mbar_wait_bounded(bar_addr + 8u * (u % HYB_STAGES), (u / HYB_STAGES) & 1u);
    };

    uint32_t r0 = warp * 32;
    GroupDesc<MW> cur = load_group<MW>(rank_sid, rank_mask, rank_gstart, begin, n, r0, lane);
    if (cur.cmax == 0) return;
    GroupDesc<MW> nxt = load_group<MW>(rank_sid, rank_mask, rank_gstart, begin, n, r0 + HYB_THREADS, lane);
    while (true) {
        const GroupDesc<MW> nxt2 = load_group<MW>(rank_sid, rank_mask, rank_gstart, begin, n, r0 + 2 * HYB_THREADS, lane);
        produce(cur, nxt, nxt2, 1);
        ShRegs<K> R;
        R.clear();
        const int nchunks = (cur.cmax + HYB_CHUNK - 1) / HYB_CHUNK;
        for (int k = 0; k < nchunks; ++k) {
            const uint32_t s = unit % HYB_STAGES;
            if (!__all_sync(0xffffffffu, mbar_wait_bounded(bar_addr + 8u * s, (unit / HYB_STAGES) & 1u, wait_limit))) { fail(); return; }
            const float* sl = &stage[warp][s][lane];
            const int e_end = min(cur.c, (k + 1) * HYB_CHUNK);
            auto hit = [&](const int p, const float wv) {
                const float4 pa = spix_lane[PixLayout<TS>::index(p, 0, 0)], pb = spix_lane[PixLayout<TS>::index(p, 1, 0)];
                float Y[K], w[3];
                sh_poly<K>(make_float3(pa.x, pa.y, pa.z), Y);
                lt_weights(make_float4(0.f, 0.f, 0.f, wv), make_float3(pb.x, pb.y, pb.z), w);
                R.accumulate(Y, w);
            };
            int e = k * HYB_CHUNK;
            for (; e + 1 < e_end; e += 2, sl += 64) {   // two hits per iteration: independent chains to interleave
                const int p0 = cur.pm.next();
                const int p1 = cur.pm.next();
                const float w0 = sl[0], w1 = sl[32];
                hit(p0, w0);
                hit(p1, w1);
            }
            if (e < e_end) hit(cur.pm.next(), sl[0]);
            fence_proxy_async();
            __syncwarp();
            ++unit;
            produce(cur, nxt, nxt2, 2);
        }
        if (cur.c != 0) {
            // words 11 .. 10 + 3K of the slot's accumulation record (the float4 holding word 11 starts at word 8)
#pragma unroll
            for (int q = 2; q < AW / 4; ++q) {
                float v[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int wd = 4 * q + i;
                    v[i] = (wd >= 11 && wd < 11 + SW) ? R.word(wd - 11) : 0.0f;
                }
                red_add_f4_hint(gacc_piece(gacc, cur.sid, q), v[0], v[1], v[2], v[3], pol_keep);
            }
        }
        if (nxt.cmax == 0) break;
        cur = nxt;
        nxt = nxt2;
        r0 += HYB_THREADS;
        --pw;
    }
}

// ------------------------------------------------------------------------------- remaining terms, pixel-centric
// One thread per ray; per hit three 16-byte vector reductions on the moments of the Gaussian's accumulation record
// (v, Q, sum alpha dL/dalpha: the same record that the primitive-centric pass fills, converted afterwards).
template <int DEG>
__global__ void __launch_bounds__(128) bwd_pixel_geo_kernel(const float4* __restrict__ rec, const float4* __restrict__ sh_slot, const uint32_t* __restrict__ slot_of_gid,
                                                            const uint32_t* __restrict__ ray_off, const uint32_t* __restrict__ ray_gid,
                                                            const float* __restrict__ dL_dC, CamF cam, float bg0, float bg1, float bg2,
                                                            Gacc gacc, const uint32_t* __restrict__ counts) {
    constexpr int K = (DEG + 1) * (DEG + 1), SW = 3 * K, RS4 = REC_F4;
    if (counts[GART_CNT_ERROR]) return;
    const int64_t ray = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (ray >= (int64_t)cam.width * cam.height) return;
    const uint32_t b = ray_off[ray], e = ray_off[ray + 1];
    if (b == e) return;
    const int x = (int)(ray % cam.width), y = (int)(ray / cam.width);
    float B[K];
    sh_basis<K>(pixel_dir(cam, x, y), B);   // (with the basis constants: the coefficients come straight from the caller's array)
    const float3 g = make_float3(dL_dC[3 * ray], dL_dC[3 * ray + 1], dL_dC[3 * ray + 2]);
    const uint64_t pol_keep = l2_policy_evict_last();
    // front to back: log of the final transmittance
    float logT = 0.0f;
    for (uint32_t h = b; h < e; ++h) {
        const PreRec P = load_pre(rec + (size_t)__ldg(slot_of_gid + ray_gid[h]) * RS4);
        const RayEval r = ray_eval(P, (float)(x - P.ix) - P.rx, (float)(y - P.iy) - P.ry);
        logT += log1pf(-r.alpha);
    }
    // back to front
    float cb0 = bg0, cb1 = bg1, cb2 = bg2;
    for (uint32_t h = e; h-- > b;) {
        const uint32_t gid = ray_gid[h];
        const uint32_t sid = __ldg(slot_of_gid + gid);
        const float4* rp = rec + (size_t)sid * RS4;
        const PreRec P = load_pre(rp);
        const RayEval r = ray_eval(P, (float)(x - P.ix) - P.rx, (float)(y - P.iy) - P.ry);
        float c0 = 0.5f, c1 = 0.5f, c2 = 0.5f;
        const float4* sp = sh_slot + (size_t)sid * ((SW + 3) / 4);   // the slot's coefficient row (a copy in slot order: rays of a warp meet the same few rows)
#pragma unroll
        for (int q = 0; q < (SW + 3) / 4; ++q) {
            const float4 t = __ldg(sp + q);
            const float sv[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int wd = 4 * q + i;
                if (wd < SW) {
                    const float term = B[wd / 3] * sv[i];
                    if (wd % 3 == 0) c0 += term;
                    else if (wd % 3 == 1) c1 += term;
                    else c2 += term;
                }
            }
        }
        c0 = fmaxf(c0, 0.0f); c1 = fmaxf(c1, 0.0f); c2 = fmaxf(c2, 0.0f);
        logT -= log1pf(-r.alpha);                       // log of the transmittance in front of this hit
        const float wgt = __expf(logT) * r.alpha;
        const float ad = wgt * fmaf(g.x, c0 - cb0, fmaf(g.y, c1 - cb1, g.z * (c2 - cb2)));   // alpha dL/dalpha
        const float G = -0.5f * ad;
        const float3 xg = ray_xg(r);
        const float gx = G * xg.x, gy = G * xg.y, gz = G * xg.z;
        // words 0..9 of the slot's accumulation record as three 16-byte vector reductions (word 10 is unused and word
        // 11, the first SH word, gets + 0)
        red_add_f4_hint(gacc_piece(gacc, sid, 0), gx, gy, gz, gx * xg.x, pol_keep);
        red_add_f4_hint(gacc_piece(gacc, sid, 1), gy * xg.y, gz * xg.z, gx * xg.y, gx * xg.z, pol_keep);
        red_add_f4_hint(gacc_piece(gacc, sid, 2), gy * xg.z, ad, 0.0f, 0.0f, pol_keep);
        const float om = 1.0f - r.alpha;
        cb0 = fmaf(r.alpha, c0, om * cb0); cb1 = fmaf(r.alpha, c1, om * cb1); cb2 = fmaf(r.alpha, c2, om * cb2);
    }
}

// The coefficient rows of the view's slots, copied once per call in slot order (rows padded to whole 16-byte pieces): the
// pixel pass reads a hit's row once per hit, and read by Gaussian id those reads scatter over the whole scene.
static __global__ void __launch_bounds__(256) hyb_gather_sh_kernel(const float* __restrict__ sh, const uint32_t* __restrict__ gid_of_slot, int sw,
                                                                   float* __restrict__ sh_slot, const uint32_t* __restrict__ counts) {
    const int swp = (sw + 3) & ~3;
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t slot = t / swp;
    const int e = (int)(t - slot * swp);
    if (slot >= (int64_t)counts[GART_CNT_VISIBLE]) return;
    sh_slot[t] = e < sw ? __ldg(sh + (size_t)gid_of_slot[slot] * sw + e) : 0.0f;
}

static inline size_t hybrid_sh_bytes(int64_t n, int sh_degree) {
    const int sw = 3 * (sh_degree + 1) * (sh_degree + 1);
    return align256((size_t)n * ((sw + 3) & ~3) * 4);
}

template <int TS>
static gart_status launch_sh(int deg, int T, cudaStream_t st, const uint32_t* tile_off, const uint32_t* rank_sid, const uint32_t* rank_mask,
                             const uint32_t* rank_gstart, const uint32_t* tile_lt_base, const float* lt_w, const float* dL_dC,
                             const CamF& cam, const Gacc& gacc, uint32_t* counts, uint32_t wait_limit) {
#define GART_SH(D) bwd_sh_kernel<TS, D><<<T, HYB_THREADS, 0, st>>>(tile_off, rank_sid, rank_mask, rank_gstart, tile_lt_base, lt_w, dL_dC, cam, gacc, counts, wait_limit)
    switch (deg) {
        case 0: GART_SH(0); break;
        case 1: GART_SH(1); break;
        case 2: GART_SH(2); break;
        default: GART_SH(3); break;
    }
#undef GART_SH
    GART_LAUNCH_CHECK();
    return GART_OK;
}

}  // namespace gart

extern "C" size_t gart_backward_hybrid_workspace_bytes(int64_t n, int32_t sh_degree) {
    const int64_t nn = n > 0 ? n : 1;
    return gart_backward_workspace_bytes(nn) + gart::hybrid_sh_bytes(nn, sh_degree < 0 ? 0 : (sh_degree > 3 ? 3 : sh_degree));
}

extern "C" gart_status gart_backward_hybrid(const gart_config* cfg, const gart_gaussians* g, const gart_camera* cam, const float* pre,
                                            const uint32_t* slot_of_gid, const uint32_t* gid_of_slot, const uint32_t* tile_off,
                                            const void* view, size_t view_bytes, int64_t cap_pairs,
                                            const float* lt_w, const uint32_t* ray_off, const uint32_t* ray_gid,
                                            const float* dL_dcolor, float* grad, uint32_t* counts, void* workspace, size_t workspace_bytes,
                                            void* stream) {
    using namespace gart;
    if (!cfg || !g || !cam || !counts || !tile_off || !dL_dcolor || !ray_off) return GART_ERR_INVALID_ARG;
    if (cfg->tile_size != 8 && cfg->tile_size != 16) return GART_ERR_INVALID_ARG;
    if (cfg->lt_format != 1 || cfg->lt_layout != GART_LT_TILE_MAJOR) return GART_ERR_INVALID_ARG;   // this pass reads the 4-byte LT format, tile-major
    if (cfg->max_hits != 0 || cfg->t_min > 0.0f || cfg->alpha_max < 1.0f) return GART_ERR_INVALID_ARG;   // its pixel-centric part re-derives every hit's alpha: no cap, no early end, no clamp
    if (cfg->kernel_degree != 0 && cfg->kernel_degree != 2) return GART_ERR_INVALID_ARG;                   // ... with the Gaussian response
    if (g->n < 0 || g->sh_degree < 0 || g->sh_degree > 3 || cap_pairs < 0 || (g->n > 0 && !g->sh)) return GART_ERR_INVALID_ARG;
    if (cam->width <= 0 || cam->height <= 0) return GART_ERR_INVALID_ARG;
    if (g->n == 0) return GART_OK;
    if (!grad || !pre || !slot_of_gid || !gid_of_slot || !lt_w || !ray_gid || !view || ((uintptr_t)view & 255)) return GART_ERR_INVALID_ARG;
    if (!workspace || ((uintptr_t)workspace & 255)) return GART_ERR_INVALID_ARG;
    if (gart_backward_hybrid_workspace_bytes(g->n, g->sh_degree) > workspace_bytes) return GART_ERR_WORKSPACE_TOO_SMALL;
    const ViewLayout v = view_layout(const_cast<void*>(view), g->n, cam->width, cam->height, cfg->tile_size, cap_pairs);
    if (v.bytes > view_bytes) return GART_ERR_WORKSPACE_TOO_SMALL;
    const uint32_t *rank_sid = v.rank_sid, *rank_mask = v.rank_mask, *rank_gstart = v.rank_gstart, *tile_lt_base = v.tile_lt_base;
    cudaStream_t st = (cudaStream_t)stream;
    const Gacc gacc = make_gacc(workspace, g->n);
    gart_status s = launch_zero_accumulators(gacc, g->n, counts, st);
    if (s != GART_OK) return s;
    const CamF cf = make_camf(cam, cfg->tile_size);
    const int T = cf.tiles_x * cf.tiles_y;
    const float4* rec = reinterpret_cast<const float4*>(pre);
    if (cfg->tile_size == 8) s = launch_sh<8>(g->sh_degree, T, st, tile_off, rank_sid, rank_mask, rank_gstart, tile_lt_base, lt_w, dL_dcolor, cf, gacc, counts, wait_limit_of(cfg->wait_polls));
    else s = launch_sh<16>(g->sh_degree, T, st, tile_off, rank_sid, rank_mask, rank_gstart, tile_lt_base, lt_w, dL_dcolor, cf, gacc, counts, wait_limit_of(cfg->wait_polls));
    if (s != GART_OK) return s;
    const int64_t n_rays = (int64_t)cam->width * cam->height;
    const unsigned blocks = (unsigned)ceil_div(n_rays, 128);
    const float* bg = cfg->background;
    float* sh_slot = reinterpret_cast<float*>(reinterpret_cast<char*>(workspace) + gart_backward_workspace_bytes(g->n));
    {
        const int sw = 3 * (g->sh_degree + 1) * (g->sh_degree + 1), swp = (sw + 3) & ~3;
        hyb_gather_sh_kernel<<<(unsigned)ceil_div(g->n * (int64_t)swp, 256), 256, 0, st>>>(g->sh, gid_of_slot, sw, sh_slot, counts);
        GART_LAUNCH_CHECK();
    }
#define GART_GEO(D) bwd_pixel_geo_kernel<D><<<blocks, 128, 0, st>>>(rec, reinterpret_cast<const float4*>(sh_slot), slot_of_gid, ray_off, ray_gid, dL_dcolor, cf, bg[0], bg[1], bg[2], gacc, counts)
    switch (g->sh_degree) {
        case 0: GART_GEO(0); break;
        case 1: GART_GEO(1); break;
        case 2: GART_GEO(2); break;
        default: GART_GEO(3); break;
    }
#undef GART_GEO
    GART_LAUNCH_CHECK();
    const float4* qs = rec + (size_t)g->n * REC_F4;
    return launch_finalize(g->n, qs, slot_of_gid, gid_of_slot, gacc, grad, counts, st);
}
