// gart_forward: ray evaluation (Sec. 3.2-3.3) over the tile lists and the compact intermediate
// buffer (Sec. 4.2-4.3).
//
// The paper finds the hits of a ray with hardware ray tracing over a BVH of bounded proxies;
// here candidates come from the tile lists (same hit set: a hit is alpha >= alpha_min, i.e.
// the ray meets the clamped ellipsoid whose projection the rectangle bounds).  Phases:
//   1. fwd_mask    block per tile, thread per (tile, Gaussian) pair: per image row the interval of
//                  columns where the response reaches alpha_min (roots of a quadratic, settled on
//                  the test itself) -> the pair's hit mask; hits per pixel counted in shared memory.
//   2. tile_sort   warp per tile: stable counting sort of the tile's pairs by descending hit
//                  count -> pair_order, with copies of slot id and mask in rank order (rank_sid,
//                  rank_mask: read coalesced later); groups of 32 consecutive ranks share an LT
//                  block in which entry e of lane l sits at 32 e + l -> rank_gstart; per-tile LT size.
//      scans       LT size per tile -> tile_lt_base; hits per ray -> ray_off.
//   3. fwd_eval    block per tile, one thread per (tile, Gaussian) pair, warps walk rank groups:
//                  for every hit pixel of the pair compute t*, alpha and the SH colour with the
//                  Gaussian in registers, and append a 32-byte record to the ray's segment
//                  (position from a shared-memory cursor per pixel).
//   4. fwd_sort_sweep  warp per ray: sort the segment by (t*, id), scan the transmittance
//                  front to back, then sum colour back to front so that each hit gets the
//                  colour composited behind it without cancellation; write LT, C, T_final.
#include "gm_build.cuh"

namespace gart {

// ------------------------------------------------------------------------------------------ phase 1
// Hit test without the exponential: alpha >= alpha_min  <=>  D^2 <= tau := 2 ln(sigma / alpha_min), and with
// D^2 = |o_g x d_g|^2 / |d_g|^2 and both vectors affine in the pixel position (u, v) inside the tile,
//     Q(u, v) = |o_g x d_g|^2 - tau |d_g|^2 = Quu u^2 + 2 Quv u v + Qvv v^2 + 2 Qu u + 2 Qv v + Q0 <= 0,
// and t* > 0 is t1 u + t2 v + tA > 0.  On row v the hit columns are those with q(u) = qA u^2 + 2 qBh u + qC <= 0.
// The projected ellipsoid is convex, so (qA > 0) they form one interval, whose ends are the roots of q (and the
// zero of t).  qA <= 0 (the camera inside or beside the clamped ellipsoid) tests every column.
constexpr int MASK_WARPS = 4;

// The quadratic is expanded about the pixel (uc, vc) of the tile nearest to the Gaussian's reference position: Q is a
// difference of two squares that nearly cancel at the boundary of a small Gaussian, and about the tile's corner its
// coefficients would be up to (tile size / footprint)^2 times larger than the values that decide.  A row works in
// u - uc and shifts its roots back by us = uc.
struct RowQuad {
    float qA, qB2, qC, t1, t0, us;   // qB2 = 2 qBh
    __device__ __forceinline__ bool hit(float u) const {   // u: column inside the tile
        const float w = u - us;
        return fmaf(fmaf(qA, w, qB2), w, qC) <= 0.0f && fmaf(t1, w, t0) > 0.0f;
    }
};

__device__ __forceinline__ float fast_sqrt(float x) {
    float y;
    asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// floor / ceil of |x| < 2^22 without the conversion unit: adding and subtracting 1.5 * 2^23 rounds to nearest.
__device__ __forceinline__ float fast_floor(float x) {
    const float r = (x + 12582912.0f) - 12582912.0f;
    return r > x ? r - 1.0f : r;
}
__device__ __forceinline__ float fast_ceil(float x) {
    const float r = (x + 12582912.0f) - 12582912.0f;
    return r < x ? r + 1.0f : r;
}
__device__ __forceinline__ int small_float_to_int(float x) {   // x integral, 0 <= x < 2^22
    return __float_as_int(x + 12582912.0f) - 0x4B400000;
}

// Bits 0..ncol-1: the columns of one row that the Gaussian's response reaches.  `regular`: qA > 0 and t1 != 0,
// with inv_qA = 1 / qA and inv_t1 = 1 / t1.  The roots come from the cancellation-free form
// (z = -(qBh + sign(qBh) sqrt(disc)); roots z / qA and qC / z), so inside the tile they are good to a few ulp: a pixel
// whose decision that rounding could flip lies within 1e-5 pixel of the boundary, i.e. its response is within
// 1e-5 of alpha_min.
// TPOS: t* > 0 on every pixel of the tile for every pair of the warp (the usual case): the side of the zero of t is not
// looked at, which takes a third of the row's instructions away.
template <int TS, bool TPOS>
__device__ __forceinline__ uint32_t row_hits(const RowQuad& q, bool regular, float inv_qA, float inv_t1, int ncol) {
    uint32_t bits = 0u;
    if (regular) {
        const float qBh = 0.5f * q.qB2;
        const float disc = fmaf(qBh, qBh, -q.qA * q.qC);
        // no branch on the sign of disc: the lanes of a warp stay together, the result is masked at the end
        const float z = -(qBh + copysignf(fast_sqrt(fmaxf(disc, 0.0f)), qBh));
        const float r1 = z * inv_qA;
        const float r2 = z != 0.0f ? q.qC * fast_rcp(z) : r1;
        const float ulo = fminf(r1, r2) + q.us, uhi = fmaxf(r1, r2) + q.us;
        float flo = fast_ceil(fminf(fmaxf(ulo, -1.0f), 4194303.0f)), fhi = fast_floor(fminf(fmaxf(uhi, -2.0f), 4194303.0f));
        if (!TPOS) {
            const float ut = fminf(fmaxf(fmaf(-q.t0, inv_t1, q.us), -2.0f), 4194303.0f);   // t* > 0 on one side of it, strictly
            const bool up = q.t1 > 0.0f;
            flo = up ? fmaxf(flo, fast_floor(ut) + 1.0f) : flo;     // smallest integer > ut
            fhi = up ? fhi : fminf(fhi, fast_ceil(ut) - 1.0f);      // largest integer < ut
        }
        flo = fmaxf(flo, 0.0f);
        fhi = fminf(fhi, (float)(ncol - 1));
        const bool any = disc >= 0.0f && flo <= fhi;             // (NaN compares false)
        const uint32_t span = (2u << (small_float_to_int(fhi) & 31)) - (1u << (small_float_to_int(flo) & 31));
        bits = any ? span : 0u;
    } else {
#pragma unroll
        for (int c = 0; c < TS; ++c)
            if (c < ncol && q.hit((float)c)) bits |= 1u << c;
    }
    return bits;
}

// Transpose of the 32 x 32 bit matrix whose row l is lane l's word x: the result's bit i is bit `lane` of lane i's x.
// Five exchanges of half-blocks with the lane 16, 8, 4, 2, 1 away.
__device__ __forceinline__ uint32_t warp_transpose_bits(uint32_t x, int lane) {
#pragma unroll
    for (int s = 16; s >= 1; s >>= 1) {
        const uint32_t m = s == 16 ? 0x0000FFFFu : s == 8 ? 0x00FF00FFu : s == 4 ? 0x0F0F0F0Fu : s == 2 ? 0x33333333u : 0x55555555u;
        const uint32_t y = __shfl_xor_sync(0xffffffffu, x, s);
        x = (lane & s) ? (((y >> s) & m) | (x & ~m)) : ((x & m) | ((y & m) << s));
    }
    return x;
}

// Block per tile, thread per (tile, Gaussian) pair: row by row the interval of hit columns -> the pair's mask.
// Hits per pixel: a shared-memory counter per pixel.
template <int TS>
__global__ void __launch_bounds__(MASK_WARPS * 32) fwd_mask_kernel(const float4* __restrict__ rec, int rs4, const uint32_t* __restrict__ slot_of_gid,
                                                                   const uint32_t* __restrict__ tile_off,
                                                                   const uint32_t* __restrict__ pair_gid, CamF cam, float alpha_min, bool narrow,
                                                                   uint32_t* __restrict__ pair_mask, uint32_t* __restrict__ pair_sid,
                                                                   const int4* __restrict__ srect, const uint32_t* __restrict__ gpair_off,
                                                                   uint32_t* __restrict__ gm_mask, uint32_t* __restrict__ pair_gpos,
                                                                   uint32_t* __restrict__ hit_count, uint32_t* __restrict__ counts) {
    constexpr int NT = TS * TS, MW = NT / 32, RPW = 32 / TS;   // rows per mask word
    __shared__ uint32_t scnt[NT];
    if (counts[GART_CNT_ERROR]) return;
    const int tile = blockIdx.x;
    const int tx = tile % cam.tiles_x, ty = tile / cam.tiles_x;
    const int x0 = tx * TS, y0 = ty * TS;
    const int lane = threadIdx.x & 31;
    const int ncol = min(TS, cam.width - x0), nrow = min(TS, cam.height - y0);
    const uint32_t begin = tile_off[tile], end = tile_off[tile + 1];
    for (int p = threadIdx.x; p < NT; p += MASK_WARPS * 32) scnt[p] = 0u;
    __syncthreads();
    uint32_t pcnt[MW];   // hits of pixel 32 q + lane among the pairs this warp has seen
#pragma unroll
    for (int q = 0; q < MW; ++q) pcnt[q] = 0u;
    const float inv_amin = 1.0f / alpha_min;
    // the chain pair -> Gaussian -> slot -> record is three dependent loads: slot ids run two iterations ahead,
    // records one
    constexpr uint32_t STEP = MASK_WARPS * 32;
    auto load_sid = [&](uint32_t jj) {   // (each pair once: the slot id is also left for the tile sort, in pair order)
        if (jj >= end) return 0u;
        const uint32_t sid = __ldg(slot_of_gid + __ldg(pair_gid + jj));
        pair_sid[jj] = sid;
        return sid;
    };
    const uint32_t jfirst = begin + threadIdx.x;
    uint32_t sid_nx = load_sid(jfirst + STEP);
    float4 ra[5];
    // the pair's place in the primitive-major order: first pair of its Gaussian + its tile's index in the rectangle's tiles
    auto gpos_of = [&](uint32_t sid, bool act) {
        if (!act || !gm_mask) return 0u;   // (gm_mask is NULL in the tile-major layout)
        const int4 r = __ldg(srect + sid);
        const int gx0 = r.x / TS, gy0 = r.y / TS;
        return __ldg(gpair_off + sid) + (uint32_t)((ty - gy0) * (r.z / TS - gx0 + 1) + (tx - gx0));
    };
    uint32_t gpa;
    {
        const uint32_t sid0 = load_sid(jfirst);
#pragma unroll
        for (int q = 0; q < 5; ++q) ra[q] = jfirst < end ? __ldg(rec + (size_t)sid0 * rs4 + q) : make_float4(0.f, 0.f, 0.f, 0.f);
        gpa = gpos_of(sid0, jfirst < end);
    }
    for (uint32_t j0 = begin + (threadIdx.x & ~31u); j0 < end; j0 += STEP) {
        const uint32_t j = j0 + lane;
        const uint32_t sid_nx2 = load_sid(j + 2 * STEP);
        float4 rb[5];
#pragma unroll
        for (int q = 0; q < 5; ++q) rb[q] = j + STEP < end ? __ldg(rec + (size_t)sid_nx * rs4 + q) : make_float4(0.f, 0.f, 0.f, 0.f);
        const uint32_t gpb = gpos_of(sid_nx, j + STEP < end);
        sid_nx = sid_nx2;
        uint32_t w[MW];
#pragma unroll
        for (int q = 0; q < MW; ++q) w[q] = 0u;
        bool tpos = true, sreg = false;
        float sQuv = 0.f, sQu = 0.f, sQvv = 0.f, sQv = 0.f, sQ0 = 0.f, st2 = 0.f, stA = 0.f, svc = 0.f, sia = 0.f, sit = 0.f;
        RowQuad rq;
        rq.qA = 0.f; rq.qB2 = 0.f; rq.qC = 0.f; rq.t1 = 0.f; rq.t0 = 0.f; rq.us = 0.f;
        if (j < end) {
            const PreRec P = unpack_pre(ra[0], ra[1], ra[2], ra[3], ra[4]);
            // 2 ln(sigma / alpha_min); the degree-4 kernel reaches alpha_min where D^4 = that, i.e. D^2 = its square root
            const float tau2 = 1.3862943611198906f * __log2f(P.sigma * inv_amin);
            const float tau = narrow ? fast_sqrt(fmaxf(tau2, 0.0f)) : tau2;
            const float3 a1 = make_float3(P.c0.y * P.m.z - P.c0.z * P.m.y, P.c0.z * P.m.x - P.c0.x * P.m.z, P.c0.x * P.m.y - P.c0.y * P.m.x);
            const float3 b1 = make_float3(P.c1.y * P.m.z - P.c1.z * P.m.y, P.c1.z * P.m.x - P.c1.x * P.m.z, P.c1.x * P.m.y - P.c1.y * P.m.x);
            // o_g x d_g and d_g at the pixel of the tile nearest to the reference position
            const int xc = min(max(P.ix, x0), x0 + TS - 1), yc = min(max(P.iy, y0), y0 + TS - 1);
            const float dx0 = (float)(xc - P.ix) - P.rx, dy0 = (float)(yc - P.iy) - P.ry;
            const float vc = (float)(yc - y0);
            const float3 dgA = make_float3(fmaf(P.c0.x, dx0, fmaf(P.c1.x, dy0, P.dgr.x)), fmaf(P.c0.y, dx0, fmaf(P.c1.y, dy0, P.dgr.y)),
                                           fmaf(P.c0.z, dx0, fmaf(P.c1.z, dy0, P.dgr.z)));
            const float3 crA = make_float3(fmaf(a1.x, dx0, fmaf(b1.x, dy0, P.k.x)), fmaf(a1.y, dx0, fmaf(b1.y, dy0, P.k.y)),
                                           fmaf(a1.z, dx0, fmaf(b1.z, dy0, P.k.z)));
            auto dot = [](const float3 a, const float3 b) { return fmaf(a.x, b.x, fmaf(a.y, b.y, a.z * b.z)); };
            const float Quu = dot(a1, a1) - tau * dot(P.c0, P.c0), Qvv = dot(b1, b1) - tau * dot(P.c1, P.c1);
            const float Quv = dot(a1, b1) - tau * dot(P.c0, P.c1);
            const float Qu = dot(crA, a1) - tau * dot(dgA, P.c0), Qv = dot(crA, b1) - tau * dot(dgA, P.c1);
            const float Q0 = dot(crA, crA) - tau * dot(dgA, dgA);
            const float tA = dot(P.m, dgA), t2 = dot(P.m, P.c1);
            rq.qA = Quu;
            rq.t1 = dot(P.m, P.c0);
            rq.us = (float)(xc - x0);
            const bool regular = rq.qA > 0.0f && rq.t1 != 0.0f;
            const float inv_qA = fast_rcp(rq.qA), inv_t1 = fast_rcp(rq.t1);
            // smallest t (up to its positive denominator) over the tile's pixels: t is affine in the pixel position
            const float tlo = tA + fminf(rq.t1 * (0.0f - rq.us), rq.t1 * ((float)(TS - 1) - rq.us)) + fminf(t2 * (0.0f - vc), t2 * ((float)(TS - 1) - vc));
            tpos = regular && tlo > 1e-4f * (fabsf(tA) + (float)TS * (fabsf(rq.t1) + fabsf(t2)));   // (well clear of zero: a near case takes the path that looks)
            sQuv = Quv; sQu = Qu; sQvv = Qvv; sQv = Qv; sQ0 = Q0; st2 = t2; stA = tA; svc = vc; sreg = regular; sia = inv_qA; sit = inv_t1;
        }
        // (every lane of the warp takes the same path: the pairs beyond the tile's list count as "positive")
        if (__all_sync(0xffffffffu, tpos)) {
            if (j < end) {
#pragma unroll
                for (int r = 0; r < TS; ++r) {
                    if (r < nrow) {
                        const float v = (float)r - svc;
                        rq.qB2 = 2.0f * fmaf(sQuv, v, sQu);
                        rq.qC = fmaf(fmaf(sQvv, v, 2.0f * sQv), v, sQ0);
                        rq.t0 = fmaf(st2, v, stA);
                        w[r / RPW] |= row_hits<TS, true>(rq, sreg, sia, sit, ncol) << ((r % RPW) * TS);
                    }
                }
            }
        } else if (j < end) {
#pragma unroll
            for (int r = 0; r < TS; ++r) {
                if (r < nrow) {
                    const float v = (float)r - svc;
                    rq.qB2 = 2.0f * fmaf(sQuv, v, sQu);
                    rq.qC = fmaf(fmaf(sQvv, v, 2.0f * sQv), v, sQ0);
                    rq.t0 = fmaf(st2, v, stA);
                    w[r / RPW] |= row_hits<TS, false>(rq, sreg, sia, sit, ncol) << ((r % RPW) * TS);
                }
            }
        }
        if (j < end) {
#pragma unroll
            for (int q = 0; q < MW; ++q) pair_mask[(size_t)j * MW + q] = w[q];
            if (gm_mask) {
#pragma unroll
                for (int q = 0; q < MW; ++q) gm_mask[(size_t)gpa * MW + q] = w[q];
                pair_gpos[j] = gpa;
            }
        }
        // hits per pixel: the warp's 32 masks are a 32 x 32 bit matrix per mask word (row = pair); transposed, lane b holds
        // the column of pixel 32 q + b, whose population count is the number of this iteration's pairs that hit the pixel
        // (a loop of one shared-memory increment per hit ran as long as the warp's largest pair and took half the kernel)
#pragma unroll
        for (int q = 0; q < MW; ++q) pcnt[q] += __popc(warp_transpose_bits(w[q], lane));
#pragma unroll
        for (int q = 0; q < 5; ++q) ra[q] = rb[q];
        gpa = gpb;
    }
#pragma unroll
    for (int q = 0; q < MW; ++q)
        if (pcnt[q]) atomicAdd(&scnt[q * 32 + lane], pcnt[q]);
    __syncthreads();
    uint32_t m = 0;
    for (int p = threadIdx.x; p < NT; p += MASK_WARPS * 32) {
        const int x = x0 + p % TS, y = y0 + p / TS;
        if (x < cam.width && y < cam.height) {
            hit_count[(size_t)y * cam.width + x] = scnt[p];
            m = max(m, scnt[p]);
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_down_sync(0xffffffffu, m, o));
    if (lane == 0 && m) atomicMax(&counts[GART_CNT_MAX_RAY_HITS], m);
}

// ------------------------------------------------------------------------------------------ phase 2
constexpr int SORT_WARPS = 4;

template <int MW>
__device__ __forceinline__ uint32_t mask_popc(const uint32_t* __restrict__ pair_mask, uint32_t j) {
    uint32_t c = 0;
#pragma unroll
    for (int q = 0; q < MW; ++q) c += __popc(__ldg(pair_mask + (size_t)j * MW + q));
    return c;
}

template <int TS>
__global__ void __launch_bounds__(SORT_WARPS * 32) tile_sort_kernel(const uint32_t* __restrict__ tile_off, const uint32_t* __restrict__ pair_sid,
                                                                    const uint32_t* __restrict__ pair_mask, const uint32_t* __restrict__ pair_gpos,
                                                                    int T, uint32_t* pair_order,
                                                                    uint32_t* __restrict__ rank_sid, uint32_t* __restrict__ rank_mask,
                                                                    uint32_t* __restrict__ rank_gstart, uint32_t* __restrict__ rank_gpos,
                                                                    uint32_t* __restrict__ tile_slots, const uint32_t* __restrict__ counts) {
    constexpr int NT = TS * TS, MW = NT / 32, NB = NT + 1;
    __shared__ uint32_t hist[SORT_WARPS][NB];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int tile = blockIdx.x * SORT_WARPS + w;
    if (tile >= T) return;
    if (counts[GART_CNT_ERROR]) { if (lane == 0) tile_slots[tile] = 0; return; }
    const uint32_t begin = tile_off[tile], n = tile_off[tile + 1] - begin;
    if (n == 0) { if (lane == 0) tile_slots[tile] = 0; return; }
    for (int d = lane; d < NB; d += 32) hist[w][d] = 0;
    __syncwarp();
    // every pass walks the tile's pairs 32 at a time; TSU chunks are loaded together so that their (dependent)
    // loads overlap
    constexpr int TSU = 4;
    for (uint32_t r0 = 0; r0 < n; r0 += 32 * TSU) {
        uint32_t c[TSU];
#pragma unroll
        for (int u = 0; u < TSU; ++u) c[u] = r0 + 32 * u + lane < n ? mask_popc<MW>(pair_mask, begin + r0 + 32 * u + lane) : 0xffffffffu;
#pragma unroll
        for (int u = 0; u < TSU; ++u)
            if (c[u] != 0xffffffffu) atomicAdd(&hist[w][c[u]], 1u);
    }
    __syncwarp();
    if (lane == 0) {   // first rank of every hit count, largest count first
        uint32_t run = 0;
        for (int c = NT; c >= 0; --c) { const uint32_t t = hist[w][c]; hist[w][c] = run; run += t; }
    }
    __syncwarp();
    for (uint32_t r0 = 0; r0 < n; r0 += 32 * TSU) {
        uint32_t c[TSU];
#pragma unroll
        for (int u = 0; u < TSU; ++u) c[u] = r0 + 32 * u + lane < n ? mask_popc<MW>(pair_mask, begin + r0 + 32 * u + lane) : 0xffffffffu;
#pragma unroll
        for (int u = 0; u < TSU; ++u) {   // in order: equal counts keep the order of the pair list
            const bool act = c[u] != 0xffffffffu;
            const unsigned amask = __ballot_sync(0xffffffffu, act);
            if (act) {
                const unsigned peers = __match_any_sync(amask, c[u]);
                const uint32_t rk = __popc(peers & ((1u << lane) - 1u));
                const uint32_t pos = hist[w][c[u]] + rk;
                __syncwarp(amask);
                if (rk == 0) hist[w][c[u]] += __popc(peers);
                __syncwarp(amask);
                pair_order[begin + pos] = begin + r0 + 32 * u + lane;
            }
        }
    }
    __threadfence_block();
    __syncwarp();
    uint32_t run = 0;
    for (uint32_t r0 = 0; r0 < n; r0 += 32 * TSU) {
        uint32_t j[TSU], sid[TSU], gp[TSU], wv[TSU][MW];
#pragma unroll
        for (int u = 0; u < TSU; ++u) j[u] = r0 + 32 * u + lane < n ? __ldcg(pair_order + begin + r0 + 32 * u + lane) : 0xffffffffu;
#pragma unroll
        for (int u = 0; u < TSU; ++u) {
            const bool act = j[u] != 0xffffffffu;
#pragma unroll
            for (int m = 0; m < MW; ++m) wv[u][m] = act ? __ldg(pair_mask + (size_t)j[u] * MW + m) : 0u;
            sid[u] = act ? __ldg(pair_sid + j[u]) : 0u;
            gp[u] = (act && rank_gpos) ? __ldg(pair_gpos + j[u]) : 0u;   // (rank_gpos is NULL in the tile-major layout)
        }
#pragma unroll
        for (int u = 0; u < TSU; ++u) {
            uint32_t c = 0;
#pragma unroll
            for (int m = 0; m < MW; ++m) c += __popc(wv[u][m]);
            if (j[u] != 0xffffffffu) {
                const size_t q = (size_t)begin + r0 + 32 * u + lane;
#pragma unroll
                for (int m = 0; m < MW; ++m) rank_mask[q * MW + m] = wv[u][m];
                rank_sid[q] = sid[u];
                if (rank_gpos) rank_gpos[q] = gp[u];
                rank_gstart[q] = run;
            }
            const uint32_t cmax = __shfl_sync(0xffffffffu, c, 0);
            run += 32u * cmax;
        }
    }
    if (lane == 0) tile_slots[tile] = run;
}

struct TileSlotsF {
    const uint32_t* tile_slots;
    __device__ __forceinline__ uint32_t operator()(int64_t i) const { return tile_slots[i]; }
};

struct RayHitsF {
    const uint32_t* hit_count;
    const uint32_t* counts;
    __device__ __forceinline__ uint32_t operator()(int64_t i) const {
        return counts[GART_CNT_ERROR] ? 0u : hit_count[i];
    }
};

__global__ void hits_total_kernel(const uint64_t* total_slots, const uint64_t* total_hits, int64_t cap_hits, uint32_t* counts) {
    const uint64_t L = total_slots[0], H = total_hits[0];
    counts[GART_CNT_HITS] = H > 0xffffffffull ? 0xffffffffu : (uint32_t)H;
    counts[GART_CNT_LT_SLOTS] = L > 0xffffffffull ? 0xffffffffu : (uint32_t)L;
    if (L > (uint64_t)cap_hits || H > (uint64_t)cap_hits) atomicOr(&counts[GART_CNT_ERROR], GART_ERRBIT_HITS);
}

// ------------------------------------------------------------------------------------------ phase 3
constexpr int EVAL_WARPS = 4;
constexpr int EVAL_THREADS = EVAL_WARPS * 32;

// What a lane needs to know about its pair of a rank group (read coalesced from the rank-ordered copies).
template <int MW>
struct EvalDesc {
    PairMask<MW> pm;
    uint32_t sid, gstart;
    uint32_t gid;     // id of the pair's Gaussian (its SH coefficients are read from the caller's array)
    uint32_t pbase;   // primitive-major layout: window index of the pair's tile origin
    int c;      // hits of this lane's pair
    int cmax;   // hits of the group's first pair (the largest)
};

// GMAJ: rank_gstart holds the LT slot of the pair's first hit in the primitive-major layout (resolved per rank position
// by gm_rank_ltb_kernel) instead of the start of the tile's rank group.
template <int MW, bool GMAJ>
__device__ __forceinline__ EvalDesc<MW> load_eval_desc(const uint32_t* __restrict__ rank_sid, const uint32_t* __restrict__ rank_mask,
                                                       const uint32_t* __restrict__ rank_gstart, const uint32_t* __restrict__ rank_pbase,
                                                       const uint32_t* __restrict__ gid_of_slot,
                                                       uint32_t begin, uint32_t n, uint32_t r0, int lane) {
    EvalDesc<MW> d;
    const bool act = r0 < n && r0 + lane < n;
    const uint32_t q = begin + r0 + lane;
    d.pm.load(rank_mask, act ? q : 0u, act);
    d.c = d.pm.count();
    d.sid = act ? __ldg(rank_sid + q) : 0u;
    d.gstart = act ? __ldg(rank_gstart + q) : 0u;
    d.pbase = (GMAJ && act) ? __ldg(rank_pbase + q) : 0u;
    d.cmax = __shfl_sync(0xffffffffu, d.c, 0);
    d.gid = (act && d.c != 0) ? __ldg(gid_of_slot + d.sid) : 0u;   // (two groups ahead of its use: the chain slot -> id -> coefficients is hidden)
    return d;
}

// Per-pixel data of the tile in shared memory, one float4 per pixel: the unit ray direction.
// Lanes read DIFFERENT pixels at the same time; with 8 copies, copy j confined to the 16-byte bank group j and
// lane l reading copy l mod 8, the 8 lanes served together by a 16-byte shared load never collide.
template <int TS>
struct EvalPix {
    static constexpr int COPIES = TS == 8 ? 8 : 1;
    static constexpr int F4 = TS * TS * COPIES;
    __device__ static __forceinline__ int index(int p, int copy) { return p * COPIES + copy; }
};

// A small non-negative integer as a float without a conversion instruction (exact below 2^23).
__device__ __forceinline__ float small_int_float(int v) { return __uint_as_float(0x4b000000u | (uint32_t)v) - 8388608.0f; }

// Block per tile, one thread per (tile, Gaussian) pair; warps walk the rank groups.  The records of the
// next group's Gaussians are copied into shared memory (16-byte asynchronous copies of each lane) while the
// current group is evaluated.  The colour is 0.5 + sum_k B_k(d) sh'_k with the bare SH polynomials B_k and
// the record's coefficients sh'_k, which carry the normalisation constants.
template <int TS, int DEG, bool GMAJ>
__global__ void __launch_bounds__(EVAL_THREADS) fwd_eval_kernel(const float4* __restrict__ rec, const float* __restrict__ sh, const uint32_t* __restrict__ gid_of_slot,
                                                                const uint32_t* __restrict__ tile_off, const uint32_t* __restrict__ rank_sid,
                                                                const uint32_t* __restrict__ rank_mask, const uint32_t* __restrict__ rank_gstart,
                                                                const uint32_t* __restrict__ tile_lt_base, const uint32_t* __restrict__ rank_pbase,
                                                                const uint32_t* __restrict__ ray_off, CamF cam, float alpha_max, bool narrow,
                                                                float4* __restrict__ recs, uint32_t* __restrict__ counts) {
    constexpr int NT = TS * TS, MW = NT / 32, K = (DEG + 1) * (DEG + 1), SW = 3 * K, PF4 = (20 + SW + 3) / 4;
    constexpr int PSTR = PF4 | 1;   // odd lane stride: the lanes' 16-byte reads fall into distinct banks
    __shared__ __align__(16) float4 spix[EvalPix<TS>::F4];
    extern __shared__ __align__(128) float4 spar[];   // [EVAL_THREADS][PSTR] staged records
    __shared__ uint32_t scur[NT];
    if (counts[GART_CNT_ERROR]) return;
    const int tile = blockIdx.x;
    const uint32_t begin = tile_off[tile], n = tile_off[tile + 1] - begin;
    if (n == 0) return;
    const int tx = tile % cam.tiles_x, ty = tile / cam.tiles_x;
    const int x0 = tx * TS, y0 = ty * TS;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int p = threadIdx.x; p < NT; p += EVAL_THREADS) {
        const int x = x0 + p % TS, y = y0 + p / TS;
        const float3 d = pixel_dir(cam, min(x, cam.width - 1), min(y, cam.height - 1));
        const uint32_t ro = (x < cam.width && y < cam.height) ? ray_off[(size_t)y * cam.width + x] : 0u;
        const float4 a = make_float4(d.x, d.y, d.z, 0.0f);
#pragma unroll
        for (int c = 0; c < EvalPix<TS>::COPIES; ++c) spix[EvalPix<TS>::index(p, c)] = a;
        scur[p] = ro;   // the next free place of the ray's segment of hit records
    }
    __syncthreads();
    const uint32_t lt_base = tile_lt_base[tile];
    const float4* spix_lane = spix + (lane & (EvalPix<TS>::COPIES - 1));
    float4* my_par = spar + (size_t)(warp * 32 + lane) * PSTR;
    const uint32_t par_addr = smem_u32(my_par);
    // Copy what the lanes need of a group's 32 Gaussians into the warp's buffers: per lane the 5 float4 of the evaluation
    // record (by slot) followed by the 3K SH coefficients (from the caller's array, by Gaussian id).  Where a row of
    // coefficients is a whole number of 16-byte pieces (degrees 1 and 3), LP lanes take the first LP pieces of one lane's
    // buffer (contiguous sources: whole sectors per request instead of one request per piece), 32 / LP buffers per
    // instruction, and a lane copies the pieces beyond LP of its own buffer; otherwise (degrees 0 and 2: rows of 12 and 108
    // bytes) a lane copies its own row word by word.  A lane therefore writes other lanes' buffers: warp barriers around the use.
    constexpr bool SH16 = SW % 4 == 0;
    constexpr int LP = PF4 <= 8 ? 8 : 16, PPI = 32 / LP;
    const uint32_t warp_par_addr = smem_u32(spar + (size_t)warp * 32 * PSTR);
    auto issue_params = [&](const EvalDesc<MW>& d) {
        const uint32_t tag = d.c != 0 ? d.sid : 0xffffffffu;
        const int piece = lane % LP;
#pragma unroll
        for (int i = 0; i < 32 / PPI; ++i) {
            const int pair = i * PPI + lane / LP;
            const uint32_t sd = __shfl_sync(0xffffffffu, tag, pair);
            const uint32_t gd = __shfl_sync(0xffffffffu, d.gid, pair);
            if (sd != 0xffffffffu && piece < (SH16 ? PF4 : REC_F4)) {
                const void* src = piece < REC_F4 ? reinterpret_cast<const void*>(rec + (size_t)sd * REC_F4 + piece)
                                                 : reinterpret_cast<const void*>(sh + (size_t)gd * SW + 4 * (piece - REC_F4));
                cp_async16(warp_par_addr + 16u * (uint32_t)(pair * PSTR + piece), src);
            }
        }
        if (d.c != 0) {
            if constexpr (SH16) {
#pragma unroll
                for (int q = LP; q < PF4; ++q) cp_async16(par_addr + 16u * q, sh + (size_t)d.gid * SW + 4 * (q - REC_F4));
            } else {
                const float* src = sh + (size_t)d.gid * SW;
#pragma unroll
                for (int e = 0; e < SW; ++e) cp_async4(par_addr + 4u * (uint32_t)(4 * REC_F4 + e), src + e);
            }
        }
    };

    uint32_t r0 = warp * 32;
    EvalDesc<MW> cur = load_eval_desc<MW, GMAJ>(rank_sid, rank_mask, rank_gstart, rank_pbase, gid_of_slot, begin, n, r0, lane);
    if (cur.cmax == 0) return;   // ranks descend in hit count: nothing for this warp
    issue_params(cur);
    EvalDesc<MW> nxt = load_eval_desc<MW, GMAJ>(rank_sid, rank_mask, rank_gstart, rank_pbase, gid_of_slot, begin, n, r0 + EVAL_THREADS, lane);
    while (true) {
        const EvalDesc<MW> nxt2 = load_eval_desc<MW, GMAJ>(rank_sid, rank_mask, rank_gstart, rank_pbase, gid_of_slot, begin, n, r0 + 2 * EVAL_THREADS, lane);
        const uint32_t gid = cur.gid;
        cp_async_wait_all();   // the copies this lane issued have landed
        __syncwarp();          // ... and so have those of the other lanes, which hold pieces of this lane's record
        const PreRec P = unpack_pre(my_par[0], my_par[1], my_par[2], my_par[3], my_par[4]);   // (stale for lanes without hits: unused)
        float shc[SW + 3];
#pragma unroll
        for (int q = 0; q < (SW + 3) / 4; ++q) {
            const float4 t = my_par[5 + q];   // (times the basis constants: the hits evaluate the bare polynomials)
            shc[4 * q] = t.x * sh_norm_word(4 * q); shc[4 * q + 1] = t.y * sh_norm_word(4 * q + 1);
            shc[4 * q + 2] = t.z * sh_norm_word(4 * q + 2); shc[4 * q + 3] = t.w * sh_norm_word(4 * q + 3);
        }
        __syncwarp();                           // every lane has read its record: the buffers may be overwritten
        if (nxt.cmax != 0) issue_params(nxt);
        uint32_t slot = GMAJ ? cur.gstart : lt_base + cur.gstart + lane;
        const float fbx = (float)(x0 - P.ix), fby = (float)(y0 - P.iy);
        const uint32_t wdx = (cur.pbase / GM_SUP) & 1u, wdy = cur.pbase / (GM_WIN * GM_SUP);   // the tile's super-tile inside the owner's window
        // one hit: evaluate, take the next free place of the ray's segment, write the 32-byte record
        auto hit = [&](const int p, const uint32_t slot_e) {
            const float4 pa = spix_lane[EvalPix<TS>::index(p, 0)];
            const uint32_t pos = atomicAdd(&scur[p], 1u);
            const RayEval r = ray_eval(P, (fbx + small_int_float(p % TS)) - P.rx, (fby + small_int_float(p / TS)) - P.ry, narrow);   // small integers: the sums are exact
            const float t = fmaxf(r.tnum * r.inv_a, 0.0f);
            float B[K];
            sh_poly<K>(make_float3(pa.x, pa.y, pa.z), B);
            float c0 = 0.5f, c1 = 0.5f, c2 = 0.5f;
#pragma unroll
            for (int k = 0; k < K; ++k) {
                c0 = fmaf(B[k], shc[3 * k], c0);
                c1 = fmaf(B[k], shc[3 * k + 1], c1);
                c2 = fmaf(B[k], shc[3 * k + 2], c2);
            }
            float4* out = recs + (size_t)pos * 2;
            // The lowest mantissa bit of the first two colour words tells the sweep in which of the 2 x 2 super-tiles of the
            // owner's window this pixel lies (the primitive-major LT entry names its pixel inside that window).  The sweep
            // composites the words without that bit, so both layouts composite the very same numbers.
            c0 = __uint_as_float((__float_as_uint(fmaxf(c0, 0.0f)) & ~1u) | wdx);
            c1 = __uint_as_float((__float_as_uint(fmaxf(c1, 0.0f)) & ~1u) | wdy);
            st_global_32B(out, make_float4(t, __uint_as_float(gid), __uint_as_float(slot_e), fminf(r.alpha, alpha_max)),
                          make_float4(c0, c1, fmaxf(c2, 0.0f), 0.0f));
        };
        // two hits per iteration: two independent dependency chains for the scheduler to interleave.  The next hit's slot:
        // 32 entries on in the tile-major layout; in the primitive-major layout entries go two by two (gm_slot):
        // the odd one follows its even one, the next even one lies 63 further.
        auto after = [](uint32_t sl) { return GMAJ ? ((sl & 1u) ? sl + 63u : sl + 1u) : sl + 32u; };
        int e = 0;
        for (; e + 1 < cur.c; e += 2) {
            const int p0 = cur.pm.next();
            const int p1 = cur.pm.next();
            const uint32_t slot1 = after(slot);
            hit(p0, slot);
            hit(p1, slot1);
            slot = after(slot1);
        }
        if (e < cur.c) hit(cur.pm.next(), slot);
        if (nxt.cmax == 0) break;
        cur = nxt;
        nxt = nxt2;
        r0 += EVAL_THREADS;
    }
}

// ------------------------------------------------------------------------------------------ phase 4
constexpr int SORT_CAP = 512;    // hits per ray sorted in registers; longer rays sort in global memory
constexpr int SWEEP_WARPS = 1;   // rays per block: with several, a block's shared memory and registers stay allocated until its longest ray is done

// ---- rays of up to SORT_CAP hits: one warp, keys in registers (R per lane, lane l holds positions l R .. l R + R - 1)
// A key is one 32-bit word: t* in 23 bits of fixed point over the ray's own depth range, above KEY_IDX_BITS bits of
// record index.  Sorting these orders the hits by t* up to 2^-23 of that range; neighbours whose quantised t* coincide
// are then put in exact (t*, id) order by a few odd-even exchanges on the full values (rare).  Padding keys are all
// ones and sort last (the largest quantised t* is 2^23 - 2).
constexpr int KEY_IDX_BITS = 9;
static_assert((1 << KEY_IDX_BITS) >= SORT_CAP, "record index must fit the key");
constexpr uint32_t KEY_IDX_MASK = (1u << KEY_IDX_BITS) - 1u;

// Ascending bitonic sort of the 32 R keys of a warp (lane l holds positions l R .. l R + R - 1), in the form whose
// compare-exchanges all put the smaller key at the lower position: a merge of size kk first pairs position i with
// i ^ (kk - 1), then with i ^ j for j = kk/4 ... 1.  No direction flags; partners inside a lane are compile-time
// register pairs, partners in another lane cost one shuffle and one min-or-max chosen per lane.
template <int R>
__device__ __forceinline__ void sort_regs(uint32_t (&k)[R], int lane) {
    auto cmpswap = [](uint32_t& a, uint32_t& b) {
        const uint32_t lo = min(a, b), hi = max(a, b);
        a = lo; b = hi;
    };
    // merges inside a lane
#pragma unroll
    for (int kk = 2; kk <= R; kk <<= 1) {
#pragma unroll
        for (int r = 0; r < R; ++r)
            if ((r ^ (kk - 1)) > r) cmpswap(k[r], k[r ^ (kk - 1)]);
#pragma unroll
        for (int j = kk >> 2; j >= 1; j >>= 1)
#pragma unroll
            for (int r = 0; r < R; ++r)
                if ((r ^ j) > r) cmpswap(k[r], k[r ^ j]);
    }
    // merges across m lanes (run-time loops: small code, the instruction cache matters more than loop overhead)
#pragma unroll 1
    for (int m = 2; m <= 32; m <<= 1) {
        {
            const bool lower = (lane & (m >> 1)) == 0;
            if (R == 1) {
                const uint32_t o = __shfl_xor_sync(0xffffffffu, k[0], m - 1);
                k[0] = lower ? min(k[0], o) : max(k[0], o);
            }
#pragma unroll
            for (int r = 0; r < R / 2; ++r) {   // registers r and R - 1 - r meet each other's mirror image
                const uint32_t oa = __shfl_xor_sync(0xffffffffu, k[R - 1 - r], m - 1);
                const uint32_t ob = __shfl_xor_sync(0xffffffffu, k[r], m - 1);
                k[r] = lower ? min(k[r], oa) : max(k[r], oa);
                k[R - 1 - r] = lower ? min(k[R - 1 - r], ob) : max(k[R - 1 - r], ob);
            }
        }
#pragma unroll 1
        for (int lj = m >> 2; lj >= 1; lj >>= 1) {
            const bool lower = (lane & lj) == 0;
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const uint32_t o = __shfl_xor_sync(0xffffffffu, k[r], lj);
                k[r] = lower ? min(k[r], o) : max(k[r], o);
            }
        }
#pragma unroll
        for (int j = R >> 1; j >= 1; j >>= 1)
#pragma unroll
            for (int r = 0; r < R; ++r)
                if ((r ^ j) > r) cmpswap(k[r], k[r ^ j]);
    }
}

// A hit's colour words as they are composited: without the lowest mantissa bit of the first two (see pix_of).
__device__ __forceinline__ float strip_low_bit(float c) { return __uint_as_float(__float_as_uint(c) & ~1u); }

// Index of the ray's pixel inside the 32 x 32-pixel window of a hit's owner: pixlow = (y mod 16) * 32 + x mod 16 from the
// ray, plus the super-tile offsets that the evaluation left in the lowest bit of the hit's first two colour words;
// -1 (nothing to embed) where pixlow < 0, i.e. in the tile-major layout.  A hit that is not composited (behind a hit cap)
// gets index 0: its entry is all zero bits and adds exactly nothing, whatever pixel it names.
__device__ __forceinline__ int pix_of(int pixlow, float c0, float c1, bool composited) {
    if (pixlow < 0) return -1;
    return composited ? pixlow + (int)((__float_as_uint(c0) & 1u) * GM_SUP + (__float_as_uint(c1) & 1u) * (GM_SUP * GM_WIN)) : 0;
}

// Store a hit's LT entry in the format the caller asked for: all 16 bytes (with the pixel's window index in the low
// mantissa bits where the layout is primitive-major: pix >= 0), only the weight word (4 bytes), or the four words as
// halves (8 bytes).
__device__ __forceinline__ void lt_store(float4* __restrict__ lt, int lt_fmt, uint32_t slot, const float4 e, int pix) {
    if (lt_fmt == 0) lt[slot] = pix >= 0 ? lt_embed_pix(e, (uint32_t)pix) : e;
    else if (lt_fmt == 1) reinterpret_cast<float*>(lt)[slot] = e.w;
    else reinterpret_cast<uint2*>(lt)[slot] = lt_pack_half(e);
}

// true if record a must come after record b: larger t*, or equal t* and larger Gaussian id  (read from the ray's records
// in global memory: with keys as fine as they are this is asked for a few rays in a hundred)
__device__ __forceinline__ bool rec_after(const float4* __restrict__ rec, uint32_t ka, uint32_t kb) {
    const float4 a = __ldg(&rec[2 * (ka & KEY_IDX_MASK)]), b = __ldg(&rec[2 * (kb & KEY_IDX_MASK)]);
    const uint32_t ta = __float_as_uint(a.x), tb = __float_as_uint(b.x);   // t* >= 0: its bit pattern orders like its value
    return ta > tb || (ta == tb && __float_as_uint(a.y) > __float_as_uint(b.y));
}

// The warp first stages the ray's records in shared memory (one coalesced 32-byte read per hit): colour and LT
// slot as one float4, alpha apart; after the sort the three passes gather from there by sorted index.
template <int R, bool GM, bool OPT>   // GM: entries carry their pixel's window index; OPT: early termination or alpha clamp may be on
__device__ __forceinline__ void sweep_ray_regs(const float4* __restrict__ rec, int n, int n_comp, int lane, size_t b, int64_t r_idx, int pixlow,
                                               float t_min, float alpha_max, float bg0, float bg1, float bg2, float* __restrict__ color, float* __restrict__ t_final,
                                               float4* __restrict__ lt, int lt_fmt, uint32_t* __restrict__ ray_gid, uint32_t* __restrict__ ray_slot,
                                               float4* __restrict__ s_cs, float* __restrict__ s_al) {
    uint32_t k[R];
    float tlo = 3.0e38f, thi = 0.0f;
#pragma unroll
    for (int r = 0; r < R; ++r) {
        // load striped (coalesced), the network does not care about the initial arrangement
        const int i = r * 32 + lane;
        k[r] = 0xffffffffu;
        if (i < n) {
            float4 ra, rb;
            ld_global_nc_32B(&rec[2 * i], ra, rb);
            k[r] = __float_as_uint(ra.x);
            tlo = fminf(tlo, ra.x); thi = fmaxf(thi, ra.x);
            s_cs[i] = make_float4(rb.x, rb.y, rb.z, ra.z);
            s_al[i] = ra.w;
        }
    }
    // The key's upper bits: t* on a scale of 2^23 - 2 steps between the ray's nearest and farthest hit (monotone in t*:
    // a difference and a product with a positive number round monotonically), finer than the leading bits of the
    // float itself by the ratio of t* to the ray's depth range, so that far fewer neighbours tie.
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        tlo = fminf(tlo, __shfl_xor_sync(0xffffffffu, tlo, o));
        thi = fmaxf(thi, __shfl_xor_sync(0xffffffffu, thi, o));
    }
    const float kscale = thi > tlo ? 8388606.0f / (thi - tlo) : 0.0f;
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const int i = r * 32 + lane;
        if (i < n) k[r] = (min(__float2uint_rd((__uint_as_float(k[r]) - tlo) * kscale), 8388606u) << KEY_IDX_BITS) | (uint32_t)i;
    }
    __syncwarp();
    sort_regs<R>(k, lane);
    {
        // neighbours with the same truncated t* (a padding key never ties: t* is finite): bit r of tm says that positions
        // r and r + 1 of this lane tie (r + 1 = R: the next lane's first)
        uint32_t tm = 0u;
#pragma unroll
        for (int r = 0; r + 1 < R; ++r) tm |= (uint32_t)(((k[r] ^ k[r + 1]) >> KEY_IDX_BITS) == 0u && k[r + 1] != 0xffffffffu) << r;
        const uint32_t nb = __shfl_down_sync(0xffffffffu, k[0], 1);
        tm |= (uint32_t)(lane < 31 && ((k[R - 1] ^ nb) >> KEY_IDX_BITS) == 0u && nb != 0xffffffffu) << (R - 1);
        if (__any_sync(0xffffffffu, tm != 0u)) {
            // a tie directly after a tie means a run of three or more equal keys
            const uint32_t tm_next = __shfl_down_sync(0xffffffffu, tm, 1);
            const bool chain = (tm & (tm << 1)) != 0u || (lane < 31 && ((tm >> (R - 1)) & 1u) && (tm_next & 1u));
            if (!__any_sync(0xffffffffu, chain)) {
                // isolated pairs (the usual case): one exact comparison each
#pragma unroll
                for (int r = 0; r + 1 < R; ++r) {
                    if (((tm >> r) & 1u) && rec_after(rec, k[r], k[r + 1])) { const uint32_t t = k[r]; k[r] = k[r + 1]; k[r + 1] = t; }
                }
                const bool mine = (tm >> (R - 1)) & 1u;
                if (__any_sync(0xffffffffu, mine)) {   // pairs across a lane boundary
                    const bool swap = mine && rec_after(rec, k[R - 1], nb);
                    const uint32_t from_prev = __shfl_up_sync(0xffffffffu, k[R - 1], 1);
                    const bool prev_swapped = __shfl_up_sync(0xffffffffu, (int)swap, 1) != 0 && lane > 0;
                    if (swap) k[R - 1] = nb;
                    if (prev_swapped) k[0] = from_prev;
                }
            } else {
                // general case: odd-even exchanges on the exact values until nothing moves, n rounds at most
                for (int round = 0; round < n; ++round) {
                    bool moved = false;
#pragma unroll
                    for (int r = 0; r + 1 < R; ++r) {
                        if (lane * R + r + 1 < n && (k[r] >> KEY_IDX_BITS) == (k[r + 1] >> KEY_IDX_BITS) && rec_after(rec, k[r], k[r + 1])) {
                            const uint32_t t = k[r]; k[r] = k[r + 1]; k[r + 1] = t; moved = true;
                        }
                    }
                    // across the lane boundary: even lanes lead on even rounds, odd lanes on odd rounds
                    const uint32_t up = __shfl_down_sync(0xffffffffu, k[0], 1), dn = __shfl_up_sync(0xffffffffu, k[R - 1], 1);
                    const bool lead = ((lane ^ round) & 1) == 0;
                    if (lead) {
                        if (lane < 31 && (lane + 1) * R < n && (k[R - 1] >> KEY_IDX_BITS) == (up >> KEY_IDX_BITS) && rec_after(rec, k[R - 1], up)) { k[R - 1] = up; moved = true; }
                    } else {
                        if (lane > 0 && lane * R < n && (dn >> KEY_IDX_BITS) == (k[0] >> KEY_IDX_BITS) && rec_after(rec, dn, k[0])) { k[0] = dn; moved = true; }
                    }
                    if (!__any_sync(0xffffffffu, moved) && (round & 1)) break;
                }
            }
        }
    }
    // front to back: transmittance in front of every hit (Eq. 7); padding positions get alpha = 0, and so do the hits
    // behind a cap on the composited hits (n_comp < n): they keep their place and their LT slot but weigh nothing
    float al[R];
    float lp = 1.0f;
#pragma unroll
    for (int r = 0; r < R; ++r) {
        al[r] = lane * R + r < n_comp ? s_al[k[r] & KEY_IDX_MASK] : 0.0f;
        lp *= 1.0f - al[r];
    }
    float inc = lp;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const float t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc *= t;
    }
    float T0 = __shfl_up_sync(0xffffffffu, inc, 1);
    if (lane == 0) T0 = 1.0f;
    float Tfin = __shfl_sync(0xffffffffu, inc, 31);
    if (OPT && t_min > 0.0f) {
        // early termination: the ray ends before the first hit whose transmittance in front is below t_min.  That hit and
        // the later ones get alpha = 0 (they keep their place and their LT slot), T_final is the transmittance reached.
        int first = 0x7fffffff;
        float Tat = 0.0f, T = T0;
#pragma unroll
        for (int r = 0; r < R; ++r) {
            if (T < t_min && lane * R + r < n_comp && first == 0x7fffffff) { first = lane * R + r; Tat = T; }
            T *= 1.0f - al[r];
        }
        int pstar = first;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) pstar = min(pstar, __shfl_xor_sync(0xffffffffu, pstar, o));
        if (pstar < n_comp) {
            const unsigned owner = __ballot_sync(0xffffffffu, first == pstar);
            Tfin = __shfl_sync(0xffffffffu, Tat, __ffs((int)owner) - 1);
            n_comp = pstar;
#pragma unroll
            for (int r = 0; r < R; ++r)
                if (lane * R + r >= pstar) al[r] = 0.0f;
        }
    }
    // back to front: colour composited behind every hit; first the lane totals ...
    float s0 = 0.0f, s1 = 0.0f, s2 = 0.0f;
    {
        float T = T0;
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const float w0 = T * al[r];   // zero on padding positions
            const float4 c = s_cs[lane * R + r < n ? (k[r] & KEY_IDX_MASK) : 0u];
            s0 = fmaf(w0, strip_low_bit(c.x), s0); s1 = fmaf(w0, strip_low_bit(c.y), s1); s2 = fmaf(w0, c.z, s2);
            T *= 1.0f - al[r];
        }
    }
    float u0 = s0, u1 = s1, u2 = s2;   // inclusive suffix over lanes
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const float a0 = __shfl_down_sync(0xffffffffu, u0, o), a1 = __shfl_down_sync(0xffffffffu, u1, o), a2 = __shfl_down_sync(0xffffffffu, u2, o);
        if (lane + o < 32) { u0 += a0; u1 += a1; u2 += a2; }
    }
    float e0 = __shfl_down_sync(0xffffffffu, u0, 1), e1 = __shfl_down_sync(0xffffffffu, u1, 1), e2 = __shfl_down_sync(0xffffffffu, u2, 1);
    if (lane == 31) { e0 = 0.0f; e1 = 0.0f; e2 = 0.0f; }
    // ... then every hit: background term + lanes behind + hits behind inside the lane
    float k0 = fmaf(Tfin, bg0, e0), k1 = fmaf(Tfin, bg1, e1), k2 = fmaf(Tfin, bg2, e2);
    {
        float Ts[R];
        float T = T0;
#pragma unroll
        for (int r = 0; r < R; ++r) { Ts[r] = T; T *= 1.0f - al[r]; }
#pragma unroll
        for (int r = R - 1; r >= 0; --r) {
            const int i = lane * R + r;
            if (i < n) {
                const uint32_t c = k[r] & KEY_IDX_MASK;
                const float4 cs = s_cs[c];
                const uint32_t slot = __float_as_uint(cs.w);
                const float wgt = Ts[r] * al[r];
                const float cx = strip_low_bit(cs.x), cy = strip_low_bit(cs.y);
                float4 en = lt_entry(wgt, al[r], cx, cy, cs.z, k0, k1, k2);
                if (OPT && al[r] >= alpha_max) { en.x = 0.0f; en.y = 0.0f; en.z = 0.0f; }   // a clamped alpha is a constant: no gradient through it
                lt_store(lt, lt_fmt, slot, en, GM ? pix_of(pixlow, cs.x, cs.y, i < n_comp) : -1);
                if (ray_gid) { ray_gid[b + i] = __float_as_uint(__ldg(&rec[2 * c].y)); ray_slot[b + i] = slot; }
                k0 = fmaf(wgt, cx, k0); k1 = fmaf(wgt, cy, k1); k2 = fmaf(wgt, cs.z, k2);
            }
        }
    }
    if (lane == 0) {   // lane 0's running sum has reached the front of the ray
        color[3 * r_idx] = k0; color[3 * r_idx + 1] = k1; color[3 * r_idx + 2] = k2;
        t_final[r_idx] = Tfin;
    }
}

// ---- longer rays: keys in global memory, sorting network over memory
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

template <bool GM, bool OPT>
__device__ __noinline__ void sweep_ray_long(const float4* __restrict__ rec, uint64_t* __restrict__ kp, int n, int n_comp, int lane, size_t b, int64_t r, int pixlow,
                                            float t_min, float alpha_max, float bg0, float bg1, float bg2, float* __restrict__ color, float* __restrict__ t_final,
                                            float4* __restrict__ lt, int lt_fmt, uint32_t* __restrict__ ray_gid, uint32_t* __restrict__ ray_slot) {
    for (int i = lane; i < n; i += 32) kp[i] = ((uint64_t)__float_as_uint(__ldg(&rec[2 * i].x)) << 32) | (uint64_t)i;
    __syncwarp();
    warp_sort(kp, n, lane);
    bool tie = false;
    for (int i = lane; i + 1 < n; i += 32) tie = tie || ((uint32_t)(kp[i] >> 32) == (uint32_t)(kp[i + 1] >> 32));
    if (__any_sync(0xffffffffu, tie)) {
        if (lane == 0) {   // insertion sort of the runs of equal t* by Gaussian id
            for (int i = 1; i < n; ++i) {
                const uint64_t x = kp[i];
                const uint32_t tx = (uint32_t)(x >> 32), gx = __float_as_uint(rec[2 * (uint32_t)x].y);
                int m = i;
                while (m > 0 && (uint32_t)(kp[m - 1] >> 32) == tx && __float_as_uint(rec[2 * (uint32_t)kp[m - 1]].y) > gx) {
                    kp[m] = kp[m - 1];
                    --m;
                }
                kp[m] = x;
            }
        }
        __syncwarp();
    }
    float carryT = 1.0f;
    int pstar = 0x7fffffff;   // early termination: first position with less than t_min transmittance in front
    float Tstar = 0.0f;
    for (int base = 0; base < n; base += 32) {
        const int i = base + lane;
        const bool valid = i < n;
        const uint32_t c = valid ? (uint32_t)kp[i] : 0u;
        const float alpha = i < n_comp ? __ldg(&rec[2 * c].w) : 0.0f;   // (n_comp <= n)
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
        if (OPT && t_min > 0.0f && pstar == 0x7fffffff) {
            const unsigned below = __ballot_sync(0xffffffffu, i < n_comp && T < t_min);
            if (below) {
                const int l0 = __ffs((int)below) - 1;
                pstar = base + l0;
                Tstar = __shfl_sync(0xffffffffu, T, l0);
            }
        }
    }
    __syncwarp();
    if (pstar < n_comp) { n_comp = pstar; carryT = Tstar; }   // the hits from there on are not composited (their stored T is never used: alpha = 0)
    const float Tfin = carryT;
    float k0 = Tfin * bg0, k1 = Tfin * bg1, k2 = Tfin * bg2;
    for (int base = 0; base < n; base += 32) {
        const int i = n - 1 - (base + lane);
        const bool valid = i >= 0;
        float wgt = 0.0f, v0 = 0.0f, v1 = 0.0f, v2 = 0.0f;
        float4 ra = make_float4(0.f, 0.f, 0.f, 0.f), rb = ra;
        if (valid) {
            const uint64_t key = kp[i];
            const uint32_t c = (uint32_t)key;
            ra = __ldg(&rec[2 * c]);
            rb = __ldg(&rec[2 * c + 1]);
            if (i >= n_comp) ra.w = 0.0f;   // behind the cap: not composited
            wgt = __uint_as_float((uint32_t)(key >> 32)) * ra.w;
            v0 = wgt * strip_low_bit(rb.x); v1 = wgt * strip_low_bit(rb.y); v2 = wgt * rb.z;
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
            const uint32_t slot = __float_as_uint(ra.z);
            float4 en = lt_entry(wgt, ra.w, strip_low_bit(rb.x), strip_low_bit(rb.y), rb.z, k0 + e0, k1 + e1, k2 + e2);
            if (OPT && ra.w >= alpha_max) { en.x = 0.0f; en.y = 0.0f; en.z = 0.0f; }
            lt_store(lt, lt_fmt, slot, en, GM ? pix_of(pixlow, rb.x, rb.y, i < n_comp) : -1);
            if (ray_gid) { ray_gid[b + i] = __float_as_uint(ra.y); ray_slot[b + i] = slot; }
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

// One launch per class of ray length, so that each gets the registers and the shared memory it needs and no more
// (the shorter rays then run at a higher occupancy than the longest): class 1 up to 256 hits, class 2 beyond.
// Every launch walks all rays and a warp returns at once if its ray belongs to the other class; class 1 also
// writes the background colour of rays without hits.
template <int CLS>
struct SweepClass {
    static_assert(CLS == 1 || CLS == 2, "two classes");
    static constexpr int LO = CLS == 1 ? 0 : 256;                    // exclusive lower bound of n
    static constexpr int CAP = CLS == 1 ? 256 : SORT_CAP;            // entries staged per warp
    static constexpr int MIN_BLOCKS = CLS == 1 ? 24 : 16;
    static constexpr int SMEM = SWEEP_WARPS * CAP * 20;
};
// Shared-memory share of the multiprocessor's 256 KB asked for, in per cent of the 228 KB maximum: 164 KB, which holds 14
// long rays (or all the short ones the registers allow) and leaves 92 KB of L1.  The sweep is that sensitive to the
// L1: with 196 KB of shared memory (17 long rays resident, 60 KB of L1) the forward pass of the 6M-Gaussian
// configuration takes 0.37 ms longer, with all 228 KB 0.45 ms, and with 132 KB (11 rays) 0.12 ms.
constexpr int SWEEP_CARVEOUT = 65;

// FMT: the LT format; GM: primitive-major layout with 16-byte entries (they carry their pixel's window index); OPT: early
// termination or the alpha clamp may be on.  Compile-time constants keep the usual case free of their tests and registers.
template <int CLS, int FMT, bool GM, bool OPT>
__global__ void __launch_bounds__(SWEEP_WARPS * 32, SweepClass<CLS>::MIN_BLOCKS)
fwd_sort_sweep_kernel(const uint32_t* __restrict__ ray_off, const float4* __restrict__ recs, uint64_t* __restrict__ long_keys, int64_t n_rays,
                      int width, int tile_size, int tiles_x,
                      float bg0, float bg1, float bg2, float* __restrict__ color, float* __restrict__ t_final,
                      float4* __restrict__ lt, uint32_t* __restrict__ ray_gid, uint32_t* __restrict__ ray_slot,
                      int max_comp, float t_min, float alpha_max, const uint32_t* __restrict__ counts) {
    constexpr int CAP = SweepClass<CLS>::CAP;
    constexpr int lt_fmt = FMT;
    if (counts[GART_CNT_ERROR]) return;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // rays in tile-major order: the 64 (256) rays of a tile are taken by neighbouring blocks, so the two halves of an
    // LT sector (entries of two pairs of the same tile) are written close in time and merge in L2
    const int64_t lin = (int64_t)blockIdx.x * SWEEP_WARPS + warp;
    int64_t r = lin;
    if (CLS == 2) {   // (the short rays' launches mostly find blocks with nothing to do: plain order is cheaper there)
        const int nt = tile_size * tile_size;
        const int64_t tile = lin / nt;
        const int pix = (int)(lin - tile * nt);
        const int x = (int)(tile % tiles_x) * tile_size + pix % tile_size, y = (int)(tile / tiles_x) * tile_size + pix / tile_size;
        if (x >= width) return;
        r = (int64_t)y * width + x;
    }
    if (r >= n_rays) return;
    const size_t b = ray_off[r];
    const int n = (int)(ray_off[r + 1] - ray_off[r]);
    if (n == 0) {
        if (CLS == 1 && lane == 0) {
            color[3 * r] = bg0; color[3 * r + 1] = bg1; color[3 * r + 2] = bg2;
            t_final[r] = 1.0f;
        }
        return;
    }
    if (n <= SweepClass<CLS>::LO || (CLS < 2 && n > CAP)) return;
    const int n_comp = min(n, max_comp);   // hits that are composited (all of them unless the caller set a cap)
    const int pixlow = GM ? (int)((r / width) % GM_SUP) * GM_WIN + (int)((r % width) % GM_SUP) : -1;
    const float4* rec = recs + b * 2;
    extern __shared__ __align__(16) float4 sweep_smem[];   // CAP entries per warp: float4 (colour, slot), then float (alpha)
    float4* s_cs = sweep_smem + (size_t)warp * CAP;
    float* s_al = reinterpret_cast<float*>(sweep_smem + (size_t)SWEEP_WARPS * CAP) + (size_t)warp * CAP;
#define GART_SWEEP(R) sweep_ray_regs<R, GM, OPT>(rec, n, n_comp, lane, b, r, pixlow, t_min, alpha_max, bg0, bg1, bg2, color, t_final, lt, lt_fmt, ray_gid, ray_slot, s_cs, s_al)
    if (CLS == 1) {
        if (n <= 32) GART_SWEEP(1);
        else if (n <= 64) GART_SWEEP(2);
        else if (n <= 128) GART_SWEEP(4);
        else GART_SWEEP(8);
    } else {
        if (n <= SORT_CAP) GART_SWEEP(16);
        else sweep_ray_long<GM, OPT>(rec, long_keys + b, n, n_comp, lane, b, r, pixlow, t_min, alpha_max, bg0, bg1, bg2, color, t_final, lt, lt_fmt, ray_gid, ray_slot);
    }
#undef GART_SWEEP
}

// ------------------------------------------------------------------------------------------ host
struct ForwardWs {
    uint64_t *total_slots, *total_hits, *total_gm;
    void* scan_ws;
    uint32_t* tile_slots;
    uint32_t* pair_sid;     // slot of every pair's Gaussian, in pair order (written by fwd_mask, read by tile_sort)
    uint32_t *ikeys0, *ikeys1, *ivals0, *ivals1, *itable;   // sort of the primitive-major items by super-tile
    float4* recs;
    uint64_t* long_keys;
    size_t bytes;
};

static ForwardWs forward_layout(void* base, int64_t n_rays, int T, int64_t cap_pairs, int64_t cap_hits) {
    ForwardWs w;
    char* p = (char*)base;
    size_t off = 0;
    auto take = [&](size_t b) { void* r = p ? (void*)(p + off) : nullptr; off += align256(b); return r; };
    const int64_t ch = cap_hits > 0 ? cap_hits : 1, cp = cap_pairs > 0 ? cap_pairs : 1;
    w.total_slots = (uint64_t*)take(256);
    w.total_hits = (uint64_t*)take(256);
    w.total_gm = (uint64_t*)take(256);
    // scans over rays, tiles, super-tiles (fewer than tiles), the slots that have pairs (no more than the pair
    // capacity) and the radix tables of the item sort
    const int64_t scan_n = n_rays > T ? n_rays : T;
    size_t sb = scan_workspace_bytes(scan_n > cp ? scan_n : cp);
    if (radix_scan_bytes(cp) > sb) sb = radix_scan_bytes(cp);
    w.scan_ws = take(sb);
    w.tile_slots = (uint32_t*)take((size_t)(T + 1) * 4);
    w.pair_sid = (uint32_t*)take((size_t)cp * 4);
    w.ikeys0 = (uint32_t*)take((size_t)cp * 4); w.ikeys1 = (uint32_t*)take((size_t)cp * 4);
    w.ivals0 = (uint32_t*)take((size_t)cp * 4); w.ivals1 = (uint32_t*)take((size_t)cp * 4);
    w.itable = (uint32_t*)take(radix_table_bytes(cp));
    w.recs = (float4*)take((size_t)ch * 32);
    w.long_keys = (uint64_t*)take((size_t)ch * 8);
    w.bytes = off;
    return w;
}

template <int TS, bool GMAJ>
static gart_status launch_eval(int deg, int T, cudaStream_t st, const float4* rec, const float* sh, const uint32_t* gid_of_slot, const uint32_t* tile_off,
                               const uint32_t* rank_sid, const uint32_t* rank_mask, const uint32_t* rank_gstart,
                               const uint32_t* tile_lt_base, const uint32_t* rank_pbase, const uint32_t* ray_off,
                               const CamF& cam, float alpha_max, bool narrow, const ForwardWs& w, uint32_t* counts) {
#define GART_EVAL(D)                                                                                                        \
    {                                                                                                                      \
        auto kern = fwd_eval_kernel<TS, D, GMAJ>;                                                                          \
        constexpr int smem = EVAL_THREADS * (((20 + 3 * (D + 1) * (D + 1) + 3) / 4) | 1) * 16;                             \
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return GART_ERR_CUDA; \
        kern<<<T, EVAL_THREADS, smem, st>>>(rec, sh, gid_of_slot, tile_off, rank_sid, rank_mask, rank_gstart, tile_lt_base, rank_pbase, ray_off, cam, \
                                            alpha_max, narrow, w.recs, counts);                                                               \
    }
    switch (deg) {
        case 0: GART_EVAL(0); break;
        case 1: GART_EVAL(1); break;
        case 2: GART_EVAL(2); break;
        default: GART_EVAL(3); break;
    }
#undef GART_EVAL
    GART_LAUNCH_CHECK();
    return GART_OK;
}

}  // namespace gart

extern "C" size_t gart_view_bytes(int64_t n, int32_t width, int32_t height, int32_t tile_size, int64_t cap_pairs) {
    if ((tile_size != 8 && tile_size != 16) || width <= 0 || height <= 0 || n < 0 || cap_pairs < 0) return 0;
    return gart::view_layout(nullptr, n, width, height, tile_size, cap_pairs).bytes;
}

extern "C" gart_status gart_view_array(int64_t n, int32_t width, int32_t height, int32_t tile_size, int64_t cap_pairs, int32_t which,
                                       size_t* offset, size_t* bytes) {
    using namespace gart;
    if ((tile_size != 8 && tile_size != 16) || width <= 0 || height <= 0 || n < 0 || cap_pairs < 0 || !offset || !bytes) return GART_ERR_INVALID_ARG;
    char* const base = reinterpret_cast<char*>((uintptr_t)256);   // (a non-null base: only differences are used)
    const ViewLayout v = view_layout(base, n, width, height, tile_size, cap_pairs);
    const int64_t cp = cap_pairs > 0 ? cap_pairs : 1, nn = n > 0 ? n : 1;
    const int T = ((width + tile_size - 1) / tile_size) * ((height + tile_size - 1) / tile_size), mw = tile_size * tile_size / 32;
    const void* ptr = nullptr;
    size_t b = 0;
    switch (which) {
        case GART_VIEW_PAIR_MASK: ptr = v.pair_mask; b = (size_t)cp * 4 * mw; break;
        case GART_VIEW_PAIR_ORDER: ptr = v.pair_order; b = (size_t)cp * 4; break;
        case GART_VIEW_RANK_SID: ptr = v.rank_sid; b = (size_t)cp * 4; break;
        case GART_VIEW_RANK_MASK: ptr = v.rank_mask; b = (size_t)cp * 4 * mw; break;
        case GART_VIEW_RANK_GSTART: ptr = v.rank_gstart; b = (size_t)cp * 4; break;
        case GART_VIEW_TILE_LT_BASE: ptr = v.tile_lt_base; b = (size_t)(T + 1) * 4; break;
        case GART_VIEW_PAIR_GPOS: ptr = v.pair_gpos; b = (size_t)cp * 4; break;
        case GART_VIEW_GPAIR_OFF: ptr = v.gpair_off; b = (size_t)(nn + 1) * 4; break;
        case GART_VIEW_GM_MASK: ptr = v.gm_mask; b = (size_t)cp * 4 * mw; break;
        case GART_VIEW_GM_LTB: ptr = v.gm_ltb; b = (size_t)cp * 4; break;
        case GART_VIEW_ITEM_DESC: ptr = v.rk_desc; b = (size_t)cp * 16; break;
        case GART_VIEW_ITEM_GSTART: ptr = v.rk_gstart; b = (size_t)cp * 4; break;
        case GART_VIEW_ST_OFF: ptr = v.st_off; b = (size_t)(v.ns + 1) * 4; break;
        case GART_VIEW_ST_LT_BASE: ptr = v.st_lt_base; b = (size_t)(v.ns + 1) * 4; break;
        case GART_VIEW_INFO: ptr = v.info; b = GM_INFO_WORDS * 4; break;
        default: return GART_ERR_INVALID_ARG;
    }
    *offset = (size_t)(reinterpret_cast<const char*>(ptr) - base);
    *bytes = b;
    return GART_OK;
}

extern "C" size_t gart_forward_workspace_bytes(int32_t width, int32_t height, int32_t tile_size, int64_t cap_pairs, int64_t cap_hits) {
    if (tile_size != 8 && tile_size != 16) return 0;
    const int T = ((width + tile_size - 1) / tile_size) * ((height + tile_size - 1) / tile_size);
    return gart::forward_layout(nullptr, (int64_t)width * height, T, cap_pairs, cap_hits).bytes;
}

extern "C" gart_status gart_forward(const gart_config* cfg, const gart_gaussians* g, const gart_camera* cam, const float* pre,
                                    const uint32_t* slot_of_gid, const uint32_t* gid_of_slot, const uint32_t* tile_off, const uint32_t* pair_gid, int64_t cap_pairs,
                                    float* color, float* t_final, uint32_t* hit_count,
                                    float* lt, int64_t cap_hits,
                                    uint32_t* ray_off, uint32_t* ray_gid, uint32_t* ray_slot,
                                    void* view, size_t view_bytes, uint32_t* counts,
                                    void* workspace, size_t workspace_bytes, void* stream) {
    using namespace gart;
    if (!cfg || !g || !cam || !tile_off || !color || !t_final || !hit_count || !ray_off || !counts)
        return GART_ERR_INVALID_ARG;
    if (cfg->tile_size != 8 && cfg->tile_size != 16) return GART_ERR_INVALID_ARG;
    if (cfg->lt_format < 0 || cfg->lt_format > 2 || cfg->max_hits < 0 || !kernel_degree_ok(cfg->kernel_degree)) return GART_ERR_INVALID_ARG;
    if (!(cfg->t_min >= 0.0f) || !(cfg->t_min < 1.0f) || !(cfg->alpha_max > 0.0f)) return GART_ERR_INVALID_ARG;
    if (cfg->lt_layout != GART_LT_PRIMITIVE_MAJOR && cfg->lt_layout != GART_LT_TILE_MAJOR) return GART_ERR_INVALID_ARG;
    if (cfg->lt_format != 0 && cfg->lt_layout != GART_LT_TILE_MAJOR) return GART_ERR_INVALID_ARG;   // the 4- and 8-byte formats serve the tile-major passes
    if (g->n < 0 || g->sh_degree < 0 || g->sh_degree > 3 || cap_pairs < 0 || cap_hits < 0) return GART_ERR_INVALID_ARG;
    if (cap_hits > 0xfffffff0ll || cap_pairs > 0xfffffff0ll) return GART_ERR_INVALID_ARG;
    if (cam->width <= 0 || cam->height <= 0 || cam->width > 65535 * 8 || cam->height > 65535 * 8) return GART_ERR_INVALID_ARG;
    if (cap_pairs > 0 && (!pair_gid || !pre || !slot_of_gid || !gid_of_slot || (g->n > 0 && !g->sh))) return GART_ERR_INVALID_ARG;
    if (((uintptr_t)g->sh & 15) != 0) return GART_ERR_INVALID_ARG;   // the evaluation copies rows of coefficients in 16-byte pieces
    if (cap_hits > 0 && (!lt || (ray_gid == nullptr) != (ray_slot == nullptr))) return GART_ERR_INVALID_ARG;
    if (!workspace || ((uintptr_t)workspace & 255) || !view || ((uintptr_t)view & 255)) return GART_ERR_INVALID_ARG;
    const int ts = cfg->tile_size;
    const CamF cf = make_camf(cam, ts);
    const int T = cf.tiles_x * cf.tiles_y;
    const int64_t n_rays = (int64_t)cam->width * cam->height;
    ForwardWs w = forward_layout(workspace, n_rays, T, cap_pairs, cap_hits);
    if (w.bytes > workspace_bytes) return GART_ERR_WORKSPACE_TOO_SMALL;
    const ViewLayout v = view_layout(view, g->n, cam->width, cam->height, ts, cap_pairs);
    if (v.bytes > view_bytes) return GART_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t st = (cudaStream_t)stream;
    const float4* rec = reinterpret_cast<const float4*>(pre);
    const int rs4 = REC_F4;
    const int4* srect = reinterpret_cast<const int4*>(rec + (size_t)g->n * (rs4 + 2));   // the rectangles in slot order, behind the records
    const bool gmaj = cfg->lt_layout == GART_LT_PRIMITIVE_MAJOR;
    const int sup_x = (cam->width + GM_SUP - 1) / GM_SUP;
    gart_status s;
    const float amax = cfg->alpha_max < 1.0f ? cfg->alpha_max : 2.0f;   // (2: no alpha reaches it, the clamp is off)
    const bool narrow = kernel_degree_is4(cfg->kernel_degree);

    // first primitive-major pair position of every slot (the mask kernel files every pair's mask there)
    if (cudaMemsetAsync(v.info, 0, GM_INFO_WORDS * 4, st) != cudaSuccess) return GART_ERR_CUDA;
    if (cudaMemsetAsync(v.st_off, 0, (size_t)(v.ns + 1) * 4, st) != cudaSuccess) return GART_ERR_CUDA;
    // (a visible Gaussian has at least one pair: without a capacity error the slots in use number at most cap_pairs)
    const int64_t nscan = g->n < cap_pairs ? g->n : cap_pairs;
    if (gmaj && nscan > 0) {
        SlotTilesF tf{srect, counts, ts};
        s = exclusive_scan(tf, nscan, v.gpair_off, w.total_gm, w.scan_ws, st);
        if (s != GART_OK) return s;
    }

    uint32_t* const gm_mask = gmaj ? v.gm_mask : nullptr;
    if (ts == 8) fwd_mask_kernel<8><<<T, MASK_WARPS * 32, 0, st>>>(rec, rs4, slot_of_gid, tile_off, pair_gid, cf, cfg->alpha_min, narrow, v.pair_mask, w.pair_sid, srect, v.gpair_off, gm_mask, v.pair_gpos, hit_count, counts);
    else fwd_mask_kernel<16><<<T, MASK_WARPS * 32, 0, st>>>(rec, rs4, slot_of_gid, tile_off, pair_gid, cf, cfg->alpha_min, narrow, v.pair_mask, w.pair_sid, srect, v.gpair_off, gm_mask, v.pair_gpos, hit_count, counts);
    GART_LAUNCH_CHECK();

    const int sblocks = (int)ceil_div(T, SORT_WARPS);
    // (in the primitive-major layout the evaluation looks the LT slot up by the pair's primitive-major position: the
    // rank-ordered copy of those positions takes the place of the tile layout's group starts)
    if (ts == 8) tile_sort_kernel<8><<<sblocks, SORT_WARPS * 32, 0, st>>>(tile_off, w.pair_sid, v.pair_mask, v.pair_gpos, T, v.pair_order, v.rank_sid, v.rank_mask, v.rank_gstart, gmaj ? v.rank_gpos : nullptr, w.tile_slots, counts);
    else tile_sort_kernel<16><<<sblocks, SORT_WARPS * 32, 0, st>>>(tile_off, w.pair_sid, v.pair_mask, v.pair_gpos, T, v.pair_order, v.rank_sid, v.rank_mask, v.rank_gstart, gmaj ? v.rank_gpos : nullptr, w.tile_slots, counts);
    GART_LAUNCH_CHECK();

    TileSlotsF tsf{w.tile_slots};
    s = exclusive_scan(tsf, (int64_t)T, v.tile_lt_base, w.total_slots, w.scan_ws, st);
    if (s != GART_OK) return s;

    if (gmaj && nscan > 0) {
        // items: one per Gaussian that fits a window, one per touched super-tile otherwise; grouped by owner
        SlotItemsF itf{srect, counts};
        s = exclusive_scan(itf, nscan, v.item_off, w.total_gm, w.scan_ws, st);
        if (s != GART_OK) return s;
        gm_items_total_kernel<<<1, 1, 0, st>>>(w.total_gm, cap_pairs, v.info, counts);
        GART_LAUNCH_CHECK();
        int bits = 1;
        while ((1 << bits) < v.ns) ++bits;
        uint32_t* const kbuf[2] = {w.ikeys0, w.ikeys1};
        uint32_t* const vbuf[2] = {w.ivals0, w.ivals1};
        const int cur = radix_passes(bits) & 1;   // after the passes the sorted arrays are at index 0
        gm_emit_items_kernel<<<(unsigned)ceil_div(nscan, 256), 256, 0, st>>>(srect, v.item_off, sup_x, counts, kbuf[cur], vbuf[cur], v.em_slot);
        GART_LAUNCH_CHECK();
        s = radix_sort_pairs(kbuf, vbuf, cur, bits, cap_pairs, v.info + GM_INFO_ITEMS, 0u, counts + GART_CNT_ERROR, w.itable, w.scan_ws, w.total_gm, st);
        if (s != GART_OK) return s;
        const unsigned iblocks = (unsigned)ceil_div(cap_pairs, 256);
        gm_segment_offsets_kernel<<<iblocks, 256, 0, st>>>(kbuf[0], v.info + GM_INFO_ITEMS, counts, v.ns, v.st_off);
        GART_LAUNCH_CHECK();
        if (ts == 8) gm_item_desc_kernel<8><<<iblocks, 256, 0, st>>>(kbuf[0], vbuf[0], v.em_slot, v.item_off, srect, v.gpair_off, v.gm_mask, sup_x, v.info, counts, v.it_desc);
        else gm_item_desc_kernel<16><<<iblocks, 256, 0, st>>>(kbuf[0], vbuf[0], v.em_slot, v.item_off, srect, v.gpair_off, v.gm_mask, sup_x, v.info, counts, v.it_desc);
        GART_LAUNCH_CHECK();
        gm_rank_kernel<<<(unsigned)ceil_div(v.ns, GM_RANK_WARPS), GM_RANK_WARPS * 32, 0, st>>>(v.st_off, v.it_desc, v.ns, v.rk_desc, v.rk_gstart, v.st_len, v.st_parts, counts);
        GART_LAUNCH_CHECK();
        ArrayF lf{v.st_len};
        s = exclusive_scan(lf, (int64_t)v.ns, v.st_lt_base, w.total_slots, w.scan_ws, st);   // the LT size of this layout replaces the tile layout's
        if (s != GART_OK) return s;
        ArrayF pf{v.st_parts};
        s = exclusive_scan(pf, (int64_t)v.ns, v.blk_off, w.total_gm, w.scan_ws, st);
        if (s != GART_OK) return s;
        gm_blocks_kernel<<<(unsigned)ceil_div(v.ns, 256), 256, 0, st>>>(v.blk_off, v.st_parts, v.ns, v.blocks_cap, v.blk_desc, v.info, counts);
        GART_LAUNCH_CHECK();
        if (ts == 8) gm_ltb_kernel<8><<<(unsigned)v.ns, 128, 0, st>>>(v.st_off, v.st_lt_base, v.ns, v.rk_desc, v.rk_gstart, v.gm_mask, v.gm_ltb, v.gm_pbase, counts);
        else gm_ltb_kernel<16><<<(unsigned)v.ns, 128, 0, st>>>(v.st_off, v.st_lt_base, v.ns, v.rk_desc, v.rk_gstart, v.gm_mask, v.gm_ltb, v.gm_pbase, counts);
        GART_LAUNCH_CHECK();
        gm_rank_ltb_kernel<<<(unsigned)ceil_div(cap_pairs, 256), 256, 0, st>>>(v.rank_gpos, v.gm_ltb, v.gm_pbase, v.rank_pbase, counts);
        GART_LAUNCH_CHECK();
    }

    RayHitsF rf{hit_count, counts};
    s = exclusive_scan(rf, n_rays, ray_off, w.total_hits, w.scan_ws, st);
    if (s != GART_OK) return s;
    hits_total_kernel<<<1, 1, 0, st>>>(w.total_slots, w.total_hits, cap_hits, counts);
    GART_LAUNCH_CHECK();

    if (gmaj) {
        if (ts == 8) s = launch_eval<8, true>(g->sh_degree, T, st, rec, g->sh, gid_of_slot, tile_off, v.rank_sid, v.rank_mask, v.rank_gpos, v.tile_lt_base, v.rank_pbase, ray_off, cf, amax, narrow, w, counts);
        else s = launch_eval<16, true>(g->sh_degree, T, st, rec, g->sh, gid_of_slot, tile_off, v.rank_sid, v.rank_mask, v.rank_gpos, v.tile_lt_base, v.rank_pbase, ray_off, cf, amax, narrow, w, counts);
    } else {
        if (ts == 8) s = launch_eval<8, false>(g->sh_degree, T, st, rec, g->sh, gid_of_slot, tile_off, v.rank_sid, v.rank_mask, v.rank_gstart, v.tile_lt_base, v.rank_pbase, ray_off, cf, amax, narrow, w, counts);
        else s = launch_eval<16, false>(g->sh_degree, T, st, rec, g->sh, gid_of_slot, tile_off, v.rank_sid, v.rank_mask, v.rank_gstart, v.tile_lt_base, v.rank_pbase, ray_off, cf, amax, narrow, w, counts);
    }
    if (s != GART_OK) return s;

    const int64_t blocks = ceil_div((int64_t)T * ts * ts, SWEEP_WARPS);
    float4* lt4 = reinterpret_cast<float4*>(lt);
    const int lt_fmt = cfg->lt_format;
    const int max_comp = cfg->max_hits > 0 ? cfg->max_hits : 0x7fffffff;
    const float* bg = cfg->background;
#define GART_SWEEP_LAUNCH(C, F, GM, OPT)                                                                                                                 \
    {                                                                                                                                                    \
        if (cudaFuncSetAttribute(fwd_sort_sweep_kernel<C, F, GM, OPT>, cudaFuncAttributeMaxDynamicSharedMemorySize, SweepClass<C>::SMEM) != cudaSuccess) \
            return GART_ERR_CUDA;                                                                                                                        \
        if (cudaFuncSetAttribute(fwd_sort_sweep_kernel<C, F, GM, OPT>, cudaFuncAttributePreferredSharedMemoryCarveout, SWEEP_CARVEOUT) != cudaSuccess)   \
            return GART_ERR_CUDA;                                                                                                                        \
        fwd_sort_sweep_kernel<C, F, GM, OPT><<<(unsigned)blocks, SWEEP_WARPS * 32, SweepClass<C>::SMEM, st>>>(ray_off, w.recs, w.long_keys, n_rays, cam->width, ts, cf.tiles_x, bg[0],   \
                                                                                                             bg[1], bg[2], color, t_final, lt4, ray_gid, ray_slot, max_comp, cfg->t_min, amax, counts); \
        GART_LAUNCH_CHECK();                                                                                                                             \
    }
#define GART_SWEEP_BOTH(F, GM, OPT) GART_SWEEP_LAUNCH(2, F, GM, OPT) GART_SWEEP_LAUNCH(1, F, GM, OPT)   // the longest rays first
    const bool opt = cfg->t_min > 0.0f || cfg->alpha_max < 1.0f;
    if (lt_fmt == 0) {
        if (gmaj) { if (opt) { GART_SWEEP_BOTH(0, true, true) } else { GART_SWEEP_BOTH(0, true, false) } }
        else { if (opt) { GART_SWEEP_BOTH(0, false, true) } else { GART_SWEEP_BOTH(0, false, false) } }
    } else if (lt_fmt == 1) {
        GART_SWEEP_BOTH(1, false, false)     // (the hybrid pass takes neither option)
    } else {
        if (opt) { GART_SWEEP_BOTH(2, false, true) } else { GART_SWEEP_BOTH(2, false, false) }
    }
#undef GART_SWEEP_BOTH
#undef GART_SWEEP_LAUNCH
    GART_LAUNCH_CHECK();
    return GART_OK;
}
