// gart_backward: primitive-centric backward (Sec. 4.4).
//
// One thread block per tile, one thread per (tile, Gaussian) pair.  Lane l of a warp owns the pair
// of rank 32 g + l in the tile's hit-count order, so the lanes of a warp run (nearly) the same
// number of iterations; the LT entries of such a group of 32 pairs are interleaved entry by entry
// (lt[base + 32 e + l]), i.e. the whole group's LT block is one contiguous range.  Each warp streams
// these blocks into shared memory with bulk asynchronous copies (cp.async.bulk, completion on an
// mbarrier), double buffered, so that tens of KB of LT data per SM are in flight while the warp
// computes; lanes then read their entry with conflict-free 16-byte shared loads.  The records of the
// next group's Gaussians (evaluation record + SH coefficients, one contiguous piece per slot of the
// view's order) arrive the same way.  A thread accumulates (v, Q, sum alpha dL/dalpha, dL/dsh) of its
// pair in registers and adds them to the accumulation record of the Gaussian's slot with one vector
// atomic per 16 bytes -- no per-pixel atomics; slots are ordered by tile, so neighbouring tiles update
// neighbouring memory.  A per-Gaussian pass then converts the moments into d mean, d scale, d quat,
// d opacity and writes the caller's gradient records.
#include "backward_common.cuh"

namespace gart {

constexpr int BWD_WARPS = 4;
constexpr int BWD_THREADS = BWD_WARPS * 32;
constexpr int BWD_CHUNK = 16;                          // LT entries per lane and per pipeline stage
constexpr int BWD_STAGE_F4 = BWD_CHUNK * 32;           // float4 per stage (8 KB)
constexpr int BWD_LT_SMEM = BWD_WARPS * 2 * BWD_STAGE_F4 * 16;
constexpr int bwd_dyn_smem(int sw) { return BWD_LT_SMEM + BWD_THREADS * (((20 + sw + 3) / 4) | 1) * 16; }

template <int K>
struct PixLayout {
    static constexpr int W = (K + 3 + 3) & ~3;   // floats per pixel record: Y[K], g[3], zero padding
};

// Descriptor of one rank group as seen by a lane (read from the rank-ordered copies: coalesced).
template <int MW>
struct GroupDesc {
    PairMask<MW> pm;
    uint32_t sid;      // slot of the pair's Gaussian in the view's order
    int c;             // hits of this lane's pair
    int cmax;          // hits of the group's first pair = the largest of the group
    uint32_t gstart;   // first LT entry of the group, relative to the tile's base
};

template <int MW>
__device__ __forceinline__ GroupDesc<MW> load_group(const uint32_t* __restrict__ rank_sid, const uint32_t* __restrict__ rank_mask,
                                                    const uint32_t* __restrict__ rank_gstart, uint32_t begin, uint32_t n,
                                                    uint32_t r0, int lane) {
    GroupDesc<MW> d;
    const bool act = r0 < n && r0 + lane < n;
    const uint32_t q = begin + r0 + lane;
    d.pm.load(rank_mask, act ? q : 0u, act);
    d.c = d.pm.count();
    d.sid = act ? __ldg(rank_sid + q) : 0u;
    const uint32_t s0 = act ? __ldg(rank_gstart + q) : 0u;
    d.cmax = __shfl_sync(0xffffffffu, d.c, 0);
    d.gstart = __shfl_sync(0xffffffffu, s0, 0);
    return d;
}

// Gradient terms of one hit (pixel p of the tile, LT entry L) added to the pair's accumulators:
// geo[0..2] = v, geo[3..8] = Q (xx, yy, zz, xy, xz, yz), geo[9] = sum alpha dL/dalpha, R.acc = dL/dsh.
template <int TS, int K, int PW>
__device__ __forceinline__ void bwd_hit(const PreRec& P, ShRegs<K>& R, float* geo, const float* spix, int bx, int by, int p,
                                        const float4 L) {
    const RayEval r = ray_eval(P, (float)(bx + p % TS) - P.rx, (float)(by + p / TS) - P.ry);
    const float* rec = spix + p * PW;
    float Y[K];
    if (K % 4 == 0) {
#pragma unroll
        for (int k4 = 0; k4 < K / 4; ++k4) {
            const float4 t = reinterpret_cast<const float4*>(rec)[k4];
            Y[4 * k4] = t.x; Y[4 * k4 + 1] = t.y; Y[4 * k4 + 2] = t.z; Y[4 * k4 + 3] = t.w;
        }
    } else {
#pragma unroll
        for (int kk = 0; kk < K; ++kk) Y[kk] = rec[kk];
    }
    const float3 g = make_float3(rec[K], rec[K + 1], rec[K + 2]);
    float c[3], w[3];
    R.colour(Y, c);
    const float T = L.w, Ta = T * r.alpha;
    const float inv = fast_rcp(1.0f - r.alpha);
    w[0] = c[0] > 0.0f ? Ta * g.x : 0.0f;
    w[1] = c[1] > 0.0f ? Ta * g.y : 0.0f;
    w[2] = c[2] > 0.0f ? Ta * g.z : 0.0f;
    const float t0 = fmaf(T, fmaxf(c[0], 0.0f), -L.x * inv);
    const float t1 = fmaf(T, fmaxf(c[1], 0.0f), -L.y * inv);
    const float t2 = fmaf(T, fmaxf(c[2], 0.0f), -L.z * inv);
    const float dalpha = fmaf(g.x, t0, fmaf(g.y, t1, g.z * t2));
    R.accumulate(Y, w);
    const float ad = r.alpha * dalpha;
    geo[9] += ad;
    const float G = -0.5f * ad;
    const float3 xg = ray_xg(r);
    const float gx = G * xg.x, gy = G * xg.y, gz = G * xg.z;
    geo[0] += gx; geo[1] += gy; geo[2] += gz;
    geo[3] = fmaf(gx, xg.x, geo[3]); geo[4] = fmaf(gy, xg.y, geo[4]); geo[5] = fmaf(gz, xg.z, geo[5]);
    geo[6] = fmaf(gx, xg.y, geo[6]); geo[7] = fmaf(gx, xg.z, geo[7]); geo[8] = fmaf(gy, xg.z, geo[8]);
}

template <int TS, int DEG>
__global__ void __launch_bounds__(BWD_THREADS) bwd_pairs_kernel(const float4* __restrict__ rec,
                                                                const uint32_t* __restrict__ tile_off, const uint32_t* __restrict__ rank_sid,
                                                                const uint32_t* __restrict__ rank_mask, const uint32_t* __restrict__ rank_gstart,
                                                                const uint32_t* __restrict__ tile_lt_base,
                                                                const float4* __restrict__ lt, const float* __restrict__ dL_dC, CamF cam,
                                                                float* __restrict__ gacc, uint32_t* __restrict__ counts) {
    constexpr int NT = TS * TS, MW = NT / 32, K = (DEG + 1) * (DEG + 1), SW = 3 * K, PW = PixLayout<K>::W;
    constexpr int AW = (11 + SW + 3) & ~3;   // accumulator words, multiple of 4
    // record (evaluation record + SH coefficients) of a lane's Gaussian, staged through shared memory one
    // group ahead; PF4 float4 per lane
    constexpr int PF4 = (20 + SW + 3) / 4;
    constexpr int PSTR = PF4 | 1;   // lane stride in the buffer, odd: the lanes' 16-byte reads fall into distinct banks
    extern __shared__ __align__(128) float4 dyn[];   // [warp][2][BWD_STAGE_F4] LT stages, then [warp][32][PF4] parameters
    __shared__ __align__(16) float spix[NT * PW];
    __shared__ __align__(8) uint64_t bars[BWD_WARPS][3];
    if (counts[GART_CNT_ERROR]) return;
    const int tile = blockIdx.x;
    const uint32_t begin = tile_off[tile], n = tile_off[tile + 1] - begin;
    if (n == 0) return;
    const int tx = tile % cam.tiles_x, ty = tile / cam.tiles_x;
    const int x0 = tx * TS, y0 = ty * TS;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) {
        mbar_init(smem_u32(&bars[warp][0]), 1);
        mbar_init(smem_u32(&bars[warp][1]), 1);
        mbar_init(smem_u32(&bars[warp][2]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // per-pixel data of the tile: SH basis of the ray direction and the upstream gradient
    for (int p = threadIdx.x; p < NT; p += BWD_THREADS) {
        const int x = x0 + p % TS, y = y0 + p / TS;
        float* rec = spix + p * PW;
        if (x < cam.width && y < cam.height) {
            float Y[K];
            sh_basis<K>(pixel_dir(cam, x, y), Y);
#pragma unroll
            for (int k = 0; k < K; ++k) rec[k] = Y[k];
            const float* gp = dL_dC + ((size_t)y * cam.width + x) * 3;
            rec[K] = gp[0]; rec[K + 1] = gp[1]; rec[K + 2] = gp[2];
        } else {
#pragma unroll
            for (int k = 0; k < K + 3; ++k) rec[k] = 0.0f;
        }
    }
    __syncthreads();

    const float4* lt_tile = lt + tile_lt_base[tile];
    float4* my_stage = dyn + (size_t)warp * 2 * BWD_STAGE_F4;
    float4* my_par = dyn + (size_t)BWD_WARPS * 2 * BWD_STAGE_F4 + (size_t)(warp * 32 + lane) * PSTR;
    const uint32_t stage_addr = smem_u32(my_stage);
    const uint32_t par_addr = smem_u32(my_par);
    const uint32_t bar_addr = smem_u32(&bars[warp][0]);
    const uint32_t pbar_addr = bar_addr + 16u;
    uint32_t unit = 0;     // LT pipeline units (chunks) consumed so far by this warp: stage = unit & 1, parity = (unit >> 1) & 1
    uint32_t pphase = 0;   // parity of the parameter barrier

    // copy chunk `k` of a group's LT block into the stage that unit number `u` will use
    auto issue = [&](const GroupDesc<MW>& d, int k, uint32_t u) {
        if (lane == 0) {
            const int ne = min(BWD_CHUNK, d.cmax - k * BWD_CHUNK);
            const uint32_t bytes = (uint32_t)ne * 512u, s = u & 1u;
            mbar_expect_tx(bar_addr + 8u * s, bytes);
            bulk_g2s(stage_addr + s * (BWD_STAGE_F4 * 16u), lt_tile + d.gstart + (size_t)k * BWD_STAGE_F4, bytes, bar_addr + 8u * s);
        }
    };
    // copy the Gaussian records and SH coefficients of a group's pairs into the parameter buffer
    auto issue_params = [&](const GroupDesc<MW>& d) {
        const unsigned m = __ballot_sync(0xffffffffu, d.c != 0);
        if (lane == 0) mbar_expect_tx(pbar_addr, (uint32_t)__popc(m) * (uint32_t)(PF4 * 16));
        if (d.c != 0) bulk_g2s(par_addr, rec + (size_t)d.sid * PF4, (uint32_t)(PF4 * 16), pbar_addr);
    };
    auto fail = [&]() {
        // a copy never completed: report, give copies that may still be in flight a second bounded
        // chance to land before this warp's shared memory may be released, and stop
        if (lane == 0) atomicOr(&counts[GART_CNT_ERROR], GART_ERRBIT_TIMEOUT);
        mbar_wait_bounded(bar_addr, (unit >> 1) & 1u);
        mbar_wait_bounded(bar_addr + 8u, (unit >> 1) & 1u);
        mbar_wait_bounded(pbar_addr, pphase);
    };

    uint32_t r0 = warp * 32;
    GroupDesc<MW> cur = load_group<MW>(rank_sid, rank_mask, rank_gstart, begin, n, r0, lane);
    if (cur.cmax == 0) return;   // ranks descend in hit count: nothing for this warp
    issue(cur, 0, unit);
    issue_params(cur);
    GroupDesc<MW> nxt = load_group<MW>(rank_sid, rank_mask, rank_gstart, begin, n, r0 + BWD_THREADS, lane);
    while (true) {
        // descriptor two groups ahead: needed only at the start of the next iteration
        const GroupDesc<MW> nxt2 = load_group<MW>(rank_sid, rank_mask, rank_gstart, begin, n, r0 + 2 * BWD_THREADS, lane);
        PreRec P;
        ShRegs<K> R;
        float geo[11];
#pragma unroll
        for (int q = 0; q < 11; ++q) geo[q] = 0.0f;
        if (!__all_sync(0xffffffffu, mbar_wait_bounded(pbar_addr, pphase))) { fail(); return; }
        pphase ^= 1u;
        P = unpack_pre(my_par[0], my_par[1], my_par[2], my_par[3], my_par[4]);   // (stale data for lanes without hits: never used)
#pragma unroll
        for (int q = 0; q < (SW + 3) / 4; ++q) {
            const float4 t = my_par[5 + q];
            R.set(4 * q, t.x);
            if (4 * q + 1 < SW) R.set(4 * q + 1, t.y);
            if (4 * q + 2 < SW) R.set(4 * q + 2, t.z);
            if (4 * q + 3 < SW) R.set(4 * q + 3, t.w);
        }
        fence_proxy_async();
        __syncwarp();   // every lane has read its record: the buffer may be overwritten
        if (nxt.cmax != 0) issue_params(nxt);
        const int bx = x0 - P.ix, by = y0 - P.iy;
        const int nchunks = (cur.cmax + BWD_CHUNK - 1) / BWD_CHUNK;
        for (int k = 0; k < nchunks; ++k) {
            // keep the next unit's copy in flight while this one is consumed
            if (k + 1 < nchunks) issue(cur, k + 1, unit + 1);
            else if (nxt.cmax != 0) issue(nxt, 0, unit + 1);
            const uint32_t s = unit & 1u;
            if (!__all_sync(0xffffffffu, mbar_wait_bounded(bar_addr + 8u * s, (unit >> 1) & 1u))) { fail(); return; }
            const float4* sl = my_stage + s * BWD_STAGE_F4 + lane;
            const int e_end = min(cur.c, (k + 1) * BWD_CHUNK);
            // two hits per iteration: two independent dependency chains for the scheduler to interleave
            int e = k * BWD_CHUNK;
            const float4* se = sl;
            for (; e + 1 < e_end; e += 2, se += 64) {
                const int p0 = cur.pm.next();
                const int p1 = cur.pm.next();
                const float4 L0 = se[0], L1 = se[32];
                bwd_hit<TS, K, PW>(P, R, geo, spix, bx, by, p0, L0);
                bwd_hit<TS, K, PW>(P, R, geo, spix, bx, by, p1, L1);
            }
            if (e < e_end) bwd_hit<TS, K, PW>(P, R, geo, spix, bx, by, cur.pm.next(), se[0]);
            fence_proxy_async();
            __syncwarp();   // every lane is done with this stage before a later copy may overwrite it
            ++unit;
        }
        if (cur.c != 0) {
            // one vector atomic per 16 bytes of the Gaussian's record
            float4* gp = reinterpret_cast<float4*>(gacc + (size_t)cur.sid * GART_GRAD_WORDS);
#pragma unroll
            for (int q = 0; q < AW / 4; ++q) {
                float v[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int wd = 4 * q + i;
                    v[i] = wd < 11 ? geo[wd] : (wd < 11 + SW ? R.word(wd - 11) : 0.0f);
                }
                atomicAdd(gp + q, make_float4(v[0], v[1], v[2], v[3]));
            }
        }
        if (nxt.cmax == 0) break;
        cur = nxt;
        nxt = nxt2;
        r0 += BWD_THREADS;
    }
}

// Zero the accumulation records of the view's slots (their number lives on the device).
__global__ void __launch_bounds__(256) bwd_zero_kernel(float4* __restrict__ gacc4, const uint32_t* __restrict__ counts) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < (size_t)counts[GART_CNT_VISIBLE] * (GART_GRAD_WORDS / 4)) gacc4[i] = make_float4(0.f, 0.f, 0.f, 0.f);
}

// Three roles by block range; every write covers whole 32-byte sectors of a gradient record.
//   [0, conv_blocks)            one thread per slot: convert the accumulated moments (words 0..9) into
//                               d mean, d scale, d quat, d opacity and write words 0..15 of the record
//                               (all 32 lanes busy with the ~300-instruction conversion);
//   [conv_blocks, +copy_blocks) 16 lanes per slot, 12 of them copy words 16..63 (SH gradient);
//   the rest                    16 lanes per Gaussian: zero the record if the Gaussian has no slot.
// Reads run in slot order (sequential), the writes scatter by Gaussian id.
__global__ void __launch_bounds__(256) bwd_finalize_kernel(int64_t n, int64_t conv_blocks, int64_t copy_blocks, const float4* __restrict__ qs,
                                                           const uint32_t* __restrict__ slot_of_gid, const uint32_t* __restrict__ gid_of_slot,
                                                           const float4* __restrict__ gacc4, float4* __restrict__ grad4,
                                                           const uint32_t* __restrict__ counts) {
    if (counts[GART_CNT_ERROR]) return;
    constexpr int F4 = GART_GRAD_WORDS / 4;
    const int64_t V = counts[GART_CNT_VISIBLE];
    if ((int64_t)blockIdx.x < conv_blocks) {
        const int64_t sid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
        if (sid >= V) return;
        const float4* gp = gacc4 + (size_t)sid * F4;
        const float4 a = gp[0], b = gp[1], c = gp[2], d = gp[3];
        const float4 q4 = qs[2 * sid], s4 = qs[2 * sid + 1];   // quaternion; scale and opacity
        float4* out = grad4 + (size_t)gid_of_slot[sid] * F4;
        const float v[3] = {a.x, a.y, a.z};
        const float Q[6] = {a.w, b.x, b.y, b.z, b.w, c.x};
        const float q[4] = {q4.x, q4.y, q4.z, q4.w};
        const float sc[3] = {s4.x, s4.y, s4.z};
        const GeoGrad o = moments_to_grads(v, Q, q, sc);
        out[0] = make_float4(o.dmu[0], o.dmu[1], o.dmu[2], o.ds[0]);
        out[1] = make_float4(o.ds[1], o.ds[2], o.dq[0], o.dq[1]);
        out[2] = make_float4(o.dq[2], o.dq[3], c.y / s4.w, c.w);
        out[3] = d;
    } else if ((int64_t)blockIdx.x < conv_blocks + copy_blocks) {
        const int64_t t = ((int64_t)blockIdx.x - conv_blocks) * blockDim.x + threadIdx.x;
        const int64_t sid = t >> 4;
        const int l = (int)(t & 15);
        if (sid >= V || l < 4) return;
        grad4[(size_t)gid_of_slot[sid] * F4 + l] = gacc4[(size_t)sid * F4 + l];
    } else {
        const int64_t t = ((int64_t)blockIdx.x - conv_blocks - copy_blocks) * blockDim.x + threadIdx.x;
        const int64_t i = t >> 4;
        if (i >= n) return;
        if (slot_of_gid[i] == 0xffffffffu) grad4[(size_t)i * F4 + (t & 15)] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
}

template <int TS, int DEG>
static gart_status launch_pairs_deg(int T, cudaStream_t st, const float4* rec, const uint32_t* tile_off,
                                    const uint32_t* rank_sid, const uint32_t* rank_mask, const uint32_t* rank_gstart,
                                    const uint32_t* tile_lt_base, const float4* lt,
                                    const float* dL_dC, const CamF& cam, float* gacc, uint32_t* counts) {
    auto kern = bwd_pairs_kernel<TS, DEG>;
    constexpr int smem = bwd_dyn_smem(3 * (DEG + 1) * (DEG + 1));
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return GART_ERR_CUDA;
    kern<<<T, BWD_THREADS, smem, st>>>(rec, tile_off, rank_sid, rank_mask, rank_gstart, tile_lt_base, lt, dL_dC, cam, gacc, counts);
    GART_LAUNCH_CHECK();
    return GART_OK;
}

template <int TS>
static gart_status launch_pairs(int deg, int T, cudaStream_t st, const float4* rec, const uint32_t* tile_off,
                                const uint32_t* rank_sid, const uint32_t* rank_mask, const uint32_t* rank_gstart,
                                const uint32_t* tile_lt_base, const float4* lt,
                                const float* dL_dC, const CamF& cam, float* gacc, uint32_t* counts) {
#define GART_PAIRS(D) \
    return launch_pairs_deg<TS, D>(T, st, rec, tile_off, rank_sid, rank_mask, rank_gstart, tile_lt_base, lt, dL_dC, cam, gacc, counts)
    switch (deg) {
        case 0: GART_PAIRS(0);
        case 1: GART_PAIRS(1);
        case 2: GART_PAIRS(2);
        default: GART_PAIRS(3);
    }
#undef GART_PAIRS
}

}  // namespace gart

extern "C" size_t gart_backward_workspace_bytes(int64_t n) {
    return gart::align256((size_t)(n > 0 ? n : 1) * GART_GRAD_WORDS * sizeof(float));
}

extern "C" gart_status gart_backward(const gart_config* cfg, const gart_gaussians* g, const gart_camera* cam, const float* pre,
                                     const uint32_t* slot_of_gid, const uint32_t* gid_of_slot, const uint32_t* tile_off,
                                     const uint32_t* rank_sid, const uint32_t* rank_mask, const uint32_t* rank_gstart, const uint32_t* tile_lt_base,
                                     const float* lt, const float* dL_dcolor,
                                     float* grad, uint32_t* counts, void* workspace, size_t workspace_bytes, void* stream) {
    using namespace gart;
    if (!cfg || !g || !cam || !counts || !tile_off || !tile_lt_base || !dL_dcolor) return GART_ERR_INVALID_ARG;
    if (cfg->tile_size != 8 && cfg->tile_size != 16) return GART_ERR_INVALID_ARG;
    if (g->n < 0 || g->sh_degree < 0 || g->sh_degree > 3) return GART_ERR_INVALID_ARG;
    if (g->n == 0) return GART_OK;
    if (!grad || !pre || !slot_of_gid || !gid_of_slot) return GART_ERR_INVALID_ARG;
    if (!workspace || ((uintptr_t)workspace & 255)) return GART_ERR_INVALID_ARG;
    if (gart_backward_workspace_bytes(g->n) > workspace_bytes) return GART_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t st = (cudaStream_t)stream;
    float* gacc = reinterpret_cast<float*>(workspace);
    const int64_t f4 = g->n * (GART_GRAD_WORDS / 4);
    bwd_zero_kernel<<<(unsigned)ceil_div(f4, 256), 256, 0, st>>>(reinterpret_cast<float4*>(gacc), counts);
    GART_LAUNCH_CHECK();
    const CamF cf = make_camf(cam, cfg->tile_size);
    const int T = cf.tiles_x * cf.tiles_y;
    const float4* rec = reinterpret_cast<const float4*>(pre);
    const float4* lt4 = reinterpret_cast<const float4*>(lt);
    gart_status s;
    if (cfg->tile_size == 8) s = launch_pairs<8>(g->sh_degree, T, st, rec, tile_off, rank_sid, rank_mask, rank_gstart, tile_lt_base, lt4, dL_dcolor, cf, gacc, counts);
    else s = launch_pairs<16>(g->sh_degree, T, st, rec, tile_off, rank_sid, rank_mask, rank_gstart, tile_lt_base, lt4, dL_dcolor, cf, gacc, counts);
    if (s != GART_OK) return s;
    const int64_t conv_blocks = ceil_div(g->n, 256), copy_blocks = ceil_div(g->n * 16, 256);
    const float4* qs = rec + (size_t)g->n * rec_f4(g->sh_degree);   // per slot: quaternion, scale, opacity (behind the records)
    bwd_finalize_kernel<<<(unsigned)(conv_blocks + 2 * copy_blocks), 256, 0, st>>>(g->n, conv_blocks, copy_blocks, qs, slot_of_gid, gid_of_slot,
                                                                                  reinterpret_cast<const float4*>(gacc),
                                                                                  reinterpret_cast<float4*>(grad), counts);
    GART_LAUNCH_CHECK();
    return GART_OK;
}
