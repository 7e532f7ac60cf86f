// gart_backward_tile: primitive-centric backward in the paper's own decomposition (Sec. 4.4): block per tile.
//
// One thread block per tile, one thread per (tile, Gaussian) pair.  Lane l of a warp owns the pair
// of rank 32 g + l in the tile's hit-count order, so the lanes of a warp run (nearly) the same
// number of iterations; the LT entries of such a group of 32 pairs are interleaved entry by entry
// (lt[base + 32 e + l]), i.e. the whole group's LT block is one contiguous range.  Each warp streams
// these blocks into shared memory with bulk asynchronous copies (cp.async.bulk, completion on an
// mbarrier), double buffered, so that tens of KB of LT data per SM are in flight while the warp
// computes; lanes then read their entry with conflict-free 16-byte shared loads.  The records of the
// next group's Gaussians (80 bytes each, the head of the slot's record) arrive the same way.  The LT
// entry carries alpha dC/dalpha and the blending weight, so a hit costs the geometry of the maximum-
// response point, one dot product and the SH outer product: no exponential, no colour evaluation.
// A thread accumulates (v, Q, sum alpha dL/dalpha, dL/dsh) of its pair in registers and adds them to the accumulation record of the Gaussian's slot with one vector
// atomic per 16 bytes -- no per-pixel atomics; slots are ordered by tile, so neighbouring tiles update
// neighbouring memory.  A per-Gaussian pass then converts the moments into d mean, d scale, d quat,
// d opacity and writes the caller's gradient records.
#include "backward_common.cuh"
#include "view_layout.cuh"

namespace gart {

constexpr int BWD_WARPS = 4;
constexpr int BWD_THREADS = BWD_WARPS * 32;
constexpr int BWD_CHUNK = 7;                           // LT entries per lane and per pipeline stage
constexpr int BWD_STAGE_F4 = BWD_CHUNK * 32;           // float4 per stage (8 KB)
constexpr int BWD_STAGES = 2;                          // LT pipeline depth per warp
constexpr int BWD_LT_SMEM = BWD_WARPS * BWD_STAGES * BWD_STAGE_F4 * 16;
constexpr int BWD_PF4 = 5;                             // float4 per lane of the staged evaluation record
constexpr int BWD_DYN_SMEM = BWD_LT_SMEM + BWD_THREADS * BWD_PF4 * 16;

// A pair's geometry, affine in the pixel position: with (uc, vc) the pixel of the tile nearest to the Gaussian's
// reference position, d_g = dgC + (u - uc) c0 + (v - vc) c1 and o_g x d_g = crC + (u - uc) a1 + (v - vc) b1
// (a1 = c0 x m, b1 = c1 x m; dgC, crC the values at that pixel).  o_g x d_g vanishes at the Gaussian's centre: expanded
// about the tile's corner instead, a small Gaussian's hits would be differences of numbers up to tile size / offset
// times larger, and lose that many digits.
struct PairGeo {
    float3 c0, c1, dgC, a1, b1, crC;
    float uc, vc;
};

template <int TS>
__device__ __forceinline__ PairGeo pair_geo(const PreRec& P, int x0, int y0) {
    PairGeo g;
    g.c0 = P.c0; g.c1 = P.c1;
    g.a1 = make_float3(P.c0.y * P.m.z - P.c0.z * P.m.y, P.c0.z * P.m.x - P.c0.x * P.m.z, P.c0.x * P.m.y - P.c0.y * P.m.x);
    g.b1 = make_float3(P.c1.y * P.m.z - P.c1.z * P.m.y, P.c1.z * P.m.x - P.c1.x * P.m.z, P.c1.x * P.m.y - P.c1.y * P.m.x);
    const int xc = min(max(P.ix, x0), x0 + TS - 1), yc = min(max(P.iy, y0), y0 + TS - 1);
    g.uc = (float)(xc - x0); g.vc = (float)(yc - y0);
    const float dxc = (float)(xc - P.ix) - P.rx, dyc = (float)(yc - P.iy) - P.ry;
    g.dgC = make_float3(fmaf(P.c0.x, dxc, fmaf(P.c1.x, dyc, P.dgr.x)), fmaf(P.c0.y, dxc, fmaf(P.c1.y, dyc, P.dgr.y)),
                        fmaf(P.c0.z, dxc, fmaf(P.c1.z, dyc, P.dgr.z)));
    g.crC = make_float3(fmaf(g.a1.x, dxc, fmaf(g.b1.x, dyc, P.k.x)), fmaf(g.a1.y, dxc, fmaf(g.b1.y, dyc, P.k.y)),
                        fmaf(g.a1.z, dxc, fmaf(g.b1.z, dyc, P.k.z)));
    return g;
}

// d_g and o_g x d_g of pixel (u, v) of the tile
__device__ __forceinline__ void pair_geo_at(const PairGeo& P, float u, float v, float3& dg, float3& cr) {
    const float du = u - P.uc, dv = v - P.vc;   // small integers: exact
    dg = make_float3(fmaf(P.c0.x, du, fmaf(P.c1.x, dv, P.dgC.x)), fmaf(P.c0.y, du, fmaf(P.c1.y, dv, P.dgC.y)),
                     fmaf(P.c0.z, du, fmaf(P.c1.z, dv, P.dgC.z)));
    cr = make_float3(fmaf(P.a1.x, du, fmaf(P.b1.x, dv, P.crC.x)), fmaf(P.a1.y, du, fmaf(P.b1.y, dv, P.crC.y)),
                     fmaf(P.a1.z, du, fmaf(P.b1.z, dv, P.crC.z)));
}

// Gradient terms of one hit (pixel p of the tile, LT entry L) added to the pair's accumulators:
// geo[0..2] = v, geo[3..8] = Q (xx, yy, zz, xy, xz, yz), geo[9] = sum alpha dL/dalpha, R.acc = dL/dsh.
// With y = d_g x (o_g x d_g) and a = |d_g|^2 the maximum-response point is x_g = y / a, so
// G x_g = (G / a) y and G x_g x_g^T = (G / a^2) y y^T.  G = dL/d(D^2) = -(alpha dL/dalpha) (KD / 4) (D^2)^(KD/2 - 1) for the
// response exp(-D^KD / 2): -1/2 of alpha dL/dalpha for the Gaussian (KD = 2), -D^2 times it for the degree-4 kernel, with
// D^2 = |o_g x d_g|^2 / a.
template <int TS, int K, int KD = 2>
__device__ __forceinline__ void bwd_hit(const PairGeo& P, ShRegs<K>& R, float* geo, const float4* spix, int p, const float4 L) {
    const float4 pa = spix[PixLayout<TS>::index(p, 0, 0)], pb = spix[PixLayout<TS>::index(p, 1, 0)];   // spix points at the lane's copy
    float3 dg, cr;
    pair_geo_at(P, pa.w, pb.w, dg, cr);
    const float inv_a = fast_rcp(fmaf(dg.x, dg.x, fmaf(dg.y, dg.y, dg.z * dg.z)));
    float Y[K];
    sh_poly<K>(make_float3(pa.x, pa.y, pa.z), Y);
    const float3 g = make_float3(pb.x, pb.y, pb.z);
    float w[3];
    lt_weights(L, g, w);
    R.accumulate(Y, w);
    const float ad = fmaf(g.x, L.x, fmaf(g.y, L.y, g.z * L.z));   // alpha dL/dalpha
    geo[9] += ad;
    const float yx = dg.y * cr.z - dg.z * cr.y, yy = dg.z * cr.x - dg.x * cr.z, yz = dg.x * cr.y - dg.y * cr.x;
    float s1 = -0.5f * ad * inv_a;
    if constexpr (KD == 4) s1 *= 2.0f * inv_a * fmaf(cr.x, cr.x, fmaf(cr.y, cr.y, cr.z * cr.z));
    const float s2 = s1 * inv_a;
    geo[0] = fmaf(s1, yx, geo[0]); geo[1] = fmaf(s1, yy, geo[1]); geo[2] = fmaf(s1, yz, geo[2]);
    const float tx = s2 * yx, ty = s2 * yy, tz = s2 * yz;
    geo[3] = fmaf(tx, yx, geo[3]); geo[4] = fmaf(ty, yy, geo[4]); geo[5] = fmaf(tz, yz, geo[5]);
    geo[6] = fmaf(tx, yy, geo[6]); geo[7] = fmaf(tx, yz, geo[7]); geo[8] = fmaf(ty, yz, geo[8]);
}

// FMT: 0 = 16-byte LT entries, 2 = 8-byte entries (four halves, twice as many per pipeline stage).
template <int TS, int DEG, int FMT, int KD>
__global__ void __launch_bounds__(BWD_THREADS, 4) bwd_pairs_kernel(const float4* __restrict__ rec,
                                                                const uint32_t* __restrict__ tile_off, const uint32_t* __restrict__ rank_sid,
                                                                const uint32_t* __restrict__ rank_mask, const uint32_t* __restrict__ rank_gstart,
                                                                const uint32_t* __restrict__ tile_lt_base,
                                                                const float4* __restrict__ lt, const float* __restrict__ dL_dC, CamF cam,
                                                                Gacc gacc, uint32_t* __restrict__ counts, const uint32_t wait_limit) {
    constexpr int NT = TS * TS, MW = NT / 32, K = (DEG + 1) * (DEG + 1), SW = 3 * K, PIXF4 = PixLayout<TS>::F4;
    constexpr int AW = (11 + SW + 3) & ~3;   // accumulator words, multiple of 4
    constexpr int EB = FMT == 2 ? 8 : 16;                  // bytes per LT entry
    constexpr int CH = BWD_STAGE_F4 * 16 / (32 * EB);      // entries per lane and per stage
    // evaluation record of a lane's Gaussian (the first 5 float4 of the slot's record), staged through shared
    // memory one group ahead
    constexpr int PF4 = BWD_PF4, RS4 = REC_F4;
    constexpr int PSTR = PF4;       // lane stride in the buffer, odd: the lanes' 16-byte reads fall into distinct banks
    extern __shared__ __align__(128) float4 dyn[];   // [warp][2][BWD_STAGE_F4] LT stages, then [warp][32][5] evaluation records
    __shared__ __align__(16) float4 spix[PIXF4];
    __shared__ __align__(8) uint64_t bars[BWD_WARPS][BWD_STAGES];   // one per LT stage
    if (counts[GART_CNT_ERROR]) return;
    const int tile = blockIdx.x;
    const uint32_t begin = tile_off[tile], n = tile_off[tile + 1] - begin;
    if (n == 0) return;
    const int tx = tile % cam.tiles_x, ty = tile / cam.tiles_x;
    const int x0 = tx * TS, y0 = ty * TS;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) {
#pragma unroll
        for (int q = 0; q < BWD_STAGES; ++q) mbar_init(smem_u32(&bars[warp][q]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // per-pixel data of the tile: ray direction, upstream gradient, position in the tile
    for (int t = threadIdx.x; t < 2 * NT; t += BWD_THREADS) {
        const int p = t >> 1, h = t & 1;
        const int x = x0 + p % TS, y = y0 + p / TS;
        float4 v = make_float4(0.f, 0.f, 0.f, h ? (float)(p / TS) : (float)(p % TS));
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

    const char* lt_tile = reinterpret_cast<const char*>(lt) + (size_t)tile_lt_base[tile] * EB;
    const float4* spix_lane = spix + (lane & (PixLayout<TS>::COPIES - 1));
    float4* my_stage = dyn + (size_t)warp * BWD_STAGES * BWD_STAGE_F4;
    float4* my_par = dyn + (size_t)BWD_WARPS * BWD_STAGES * BWD_STAGE_F4 + (size_t)(warp * 32 + lane) * PSTR;
    const uint32_t stage_addr = smem_u32(my_stage);
    const uint32_t par_addr = smem_u32(my_par);
    const uint32_t bar_addr = smem_u32(&bars[warp][0]);
    // LT pipeline: unit u (a chunk of BWD_CHUNK entries per lane) uses stage u % BWD_STAGES, and the wait for
    // it uses parity (u / BWD_STAGES) & 1.  `unit` counts the units consumed, `produced` the units whose copy
    // has been issued; the producer cursor (pw, pk) = (group relative to the current one, chunk) runs up to
    // BWD_STAGES units and two groups ahead of the consumer.
    uint32_t unit = 0, produced = 0;
    int pw = 0, pk = 0;

    // issue copies while fewer than BWD_STAGES units are in flight; looks at most `maxw` groups ahead of the current one
    auto produce = [&](const GroupDesc<MW>& a, const GroupDesc<MW>& b, const GroupDesc<MW>& c, const int maxw) {
        while (produced - unit < (uint32_t)BWD_STAGES && pw <= maxw) {
            int cm;
            uint32_t gs;
            if (pw == 0) { cm = a.cmax; gs = a.gstart; }
            else if (pw == 1) { cm = b.cmax; gs = b.gstart; }
            else { cm = c.cmax; gs = c.gstart; }
            if (cm == 0) break;                                   // ranks descend in hit count: no later group has hits
            if (pk * CH >= cm) { ++pw; pk = 0; continue; }
            if (lane == 0) {
                const int ne = min(CH, cm - pk * CH);
                const uint32_t bytes = (uint32_t)ne * (32u * EB), s = produced % BWD_STAGES;
                mbar_expect_tx(bar_addr + 8u * s, bytes);
                bulk_g2s_hint(stage_addr + s * (BWD_STAGE_F4 * 16u), lt_tile + ((size_t)gs + (size_t)pk * (CH * 32)) * EB, bytes, bar_addr + 8u * s, l2_policy_evict_first());
            }
            ++produced;
            ++pk;
        }
    };
    // copy the evaluation records of a group's Gaussians into the parameter buffer
    auto issue_params = [&](const GroupDesc<MW>& d) {
        if (d.c != 0) {
            const float4* src = rec + (size_t)d.sid * RS4;
#pragma unroll
            for (int q = 0; q < PF4; ++q) cp_async16(par_addr + 16u * q, src + q);
        }
    };
    auto fail = [&]() {
        // a copy never completed: report, give copies that may still be in flight a second bounded
        // chance to land before this warp's shared memory may be released, and stop
        if (lane == 0) atomicOr(&counts[GART_CNT_ERROR], GART_ERRBIT_TIMEOUT);
        for (uint32_t u = unit; u != produced; ++u) mbar_wait_bounded(bar_addr + 8u * (u % BWD_STAGES), (u / BWD_STAGES) & 1u);
        cp_async_wait_all();
    };

    // The warp's j-th group is group j * BWD_WARPS + (j even ? warp : BWD_WARPS - 1 - warp) of the tile: groups descend
    // in hit count, and this serpentine deal gives every warp of the block nearly the same number of iterations.
    auto first_rank = [&](uint32_t j) { return 32u * (j * BWD_WARPS + ((j & 1u) ? (uint32_t)(BWD_WARPS - 1 - warp) : (uint32_t)warp)); };
    uint32_t gj = 0;
    GroupDesc<MW> cur = load_group<MW>(rank_sid, rank_mask, rank_gstart, begin, n, first_rank(0), lane);
    if (cur.cmax == 0) return;   // ranks descend in hit count: nothing for this warp
    issue_params(cur);
    GroupDesc<MW> nxt = load_group<MW>(rank_sid, rank_mask, rank_gstart, begin, n, first_rank(1), lane);
    while (true) {
        // descriptor two groups ahead: the producer may reach it later in this group (not yet: its loads are in flight)
        const GroupDesc<MW> nxt2 = load_group<MW>(rank_sid, rank_mask, rank_gstart, begin, n, first_rank(gj + 2), lane);
        produce(cur, nxt, nxt2, 1);
        ShRegs<K> R;
        float geo[11];
#pragma unroll
        for (int q = 0; q < 11; ++q) geo[q] = 0.0f;
        cp_async_wait_all();   // this lane's record has landed (a lane reads only what it copied itself)
        const PairGeo P = pair_geo<TS>(unpack_pre(my_par[0], my_par[1], my_par[2], my_par[3], my_par[4]), x0, y0);   // (stale data for lanes without hits: never used)
        R.clear();
        if (nxt.cmax != 0) issue_params(nxt);   // the lane has read its record: its buffer may be overwritten
        const int nchunks = (cur.cmax + CH - 1) / CH;
        for (int k = 0; k < nchunks; ++k) {
            const uint32_t s = unit % BWD_STAGES;
            if (!__all_sync(0xffffffffu, mbar_wait_bounded(bar_addr + 8u * s, (unit / BWD_STAGES) & 1u, wait_limit))) { fail(); return; }
            const char* sl = reinterpret_cast<const char*>(my_stage + s * BWD_STAGE_F4) + lane * EB;   // entry j of the stage: sl + j * 32 * EB
            auto entry = [&](const char* q) {
                if constexpr (FMT == 2) return lt_unpack_half(*reinterpret_cast<const uint2*>(q));
                else return *reinterpret_cast<const float4*>(q);
            };
            const int e_end = min(cur.c, (k + 1) * CH);
            // two hits per iteration: two independent dependency chains for the scheduler to interleave
            int e = k * CH;
            const char* se = sl;
            for (; e + 1 < e_end; e += 2, se += 64 * EB) {
                const int p0 = cur.pm.next();
                const int p1 = cur.pm.next();
                const float4 L0 = entry(se), L1 = entry(se + 32 * EB);
                bwd_hit<TS, K, KD>(P, R, geo, spix_lane, p0, L0);
                bwd_hit<TS, K, KD>(P, R, geo, spix_lane, p1, L1);
            }
            if (e < e_end) bwd_hit<TS, K, KD>(P, R, geo, spix_lane, cur.pm.next(), entry(se));
            fence_proxy_async();
            __syncwarp();   // every lane is done with this stage before a later copy may overwrite it
            ++unit;
            if (k + 1 < nchunks) produce(cur, nxt, nxt2, 2);   // refill the stage just released (after the last chunk it first serves the flush)
        }
        {
            // Flush through the stage just released, so that neighbouring lanes add neighbouring 16-byte pieces of one
            // record: the atomics of a record then reach L2 as whole 32-byte sectors (about 9 sector updates per pair
            // instead of 15).  Two rounds of FLUSH_Q pieces per lane, then the last piece directly.
            constexpr int NQ = AW / 4, FLUSH_Q = BWD_CHUNK;
            static_assert(NQ <= 2 * FLUSH_Q + 1 && NQ >= 1 && FLUSH_Q <= 8, "flush rounds");
            float4* tb = my_stage + ((unit - 1u) % BWD_STAGES) * BWD_STAGE_F4;
            const uint32_t tag = cur.c != 0 ? cur.sid : 0xffffffffu;
            const uint64_t pol_keep = l2_policy_evict_last();   // (made where they are used: the policies hold no register across the hit loop)
            auto piece = [&](int q) {
                float v[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int wd = 4 * q + i;
                    v[i] = wd < 11 ? geo[wd] : (wd < 11 + SW ? R.word(wd - 11) : 0.0f);   // (bare polynomials: the basis constants are applied when the records are converted)
                }
                return make_float4(v[0], v[1], v[2], v[3]);
            };
            // Reading the staged pieces back, eight lanes serve one record: lanes 8 g .. 8 g + nq - 1 take the round's nq
            // pieces of record 4 j + g.  A lane's piece, and with it the array, the row stride and the offset in the row, is
            // then the same for all eight reads of a round, and the address of a reduction is one multiply-add (with the
            // pieces dealt lane by lane across records it took an integer division per read).
            const int hl = lane >> 3, pc = lane & 7;
#pragma unroll
            for (int q0 = 0; q0 + 1 < NQ; q0 += FLUSH_Q) {
                const int nq = NQ - 1 - q0 < FLUSH_Q ? NQ - 1 - q0 : FLUSH_Q;   // compile-time after unrolling
#pragma unroll
                for (int j = 0; j < FLUSH_Q; ++j)
                    if (j < nq) tb[lane * nq + j] = piece(q0 + j);
                __syncwarp();
                const int q = q0 + pc;
                const bool in_a = q < GACC_A_WORDS / 4;
                char* const row0 = in_a ? reinterpret_cast<char*>(gacc.a) + 16 * q : reinterpret_cast<char*>(gacc.b) + 16 * (q - GACC_A_WORDS / 4);
                const uint32_t row_bytes = in_a ? GACC_A_WORDS * 4u : GACC_B_WORDS * 4u;
                const float4* tl = tb + hl * nq + pc;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const uint32_t sd = __shfl_sync(0xffffffffu, tag, 4 * j + hl);
                    if (pc < nq && sd != 0xffffffffu) {
                        const float4 v = tl[4 * j * nq];
                        red_add_f4_hint(reinterpret_cast<float4*>(row0 + (size_t)sd * row_bytes), v.x, v.y, v.z, v.w, pol_keep);
                    }
                }
                __syncwarp();
            }
            if (tag != 0xffffffffu) {
                const float4 v = piece(NQ - 1);
                red_add_f4_hint(gacc_piece(gacc, tag, NQ - 1), v.x, v.y, v.z, v.w, pol_keep);
            }
            fence_proxy_async();
            __syncwarp();
            produce(cur, nxt, nxt2, 2);   // now refill the stage
        }
        if (nxt.cmax == 0) break;
        cur = nxt;
        nxt = nxt2;
        ++gj;
        --pw;   // the producer is never behind the consumer: pw >= 1 here
    }
}

template <int TS, int DEG, int FMT, int KD>
static gart_status launch_pairs_deg(int T, cudaStream_t st, const float4* rec, const uint32_t* tile_off,
                                    const uint32_t* rank_sid, const uint32_t* rank_mask, const uint32_t* rank_gstart,
                                    const uint32_t* tile_lt_base, const float4* lt,
                                    const float* dL_dC, const CamF& cam, const Gacc& gacc, uint32_t* counts, uint32_t wait_limit) {
    auto kern = bwd_pairs_kernel<TS, DEG, FMT, KD>;
    constexpr int smem = BWD_DYN_SMEM;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return GART_ERR_CUDA;
    kern<<<T, BWD_THREADS, smem, st>>>(rec, tile_off, rank_sid, rank_mask, rank_gstart, tile_lt_base, lt, dL_dC, cam, gacc, counts, wait_limit);
    GART_LAUNCH_CHECK();
    return GART_OK;
}

template <int TS, int FMT>
static gart_status launch_pairs(int deg, bool narrow, int T, cudaStream_t st, const float4* rec, const uint32_t* tile_off,
                                const uint32_t* rank_sid, const uint32_t* rank_mask, const uint32_t* rank_gstart,
                                const uint32_t* tile_lt_base, const float4* lt,
                                const float* dL_dC, const CamF& cam, const Gacc& gacc, uint32_t* counts, uint32_t wait_limit) {
#define GART_PAIRS(D)                                                                                                                                       \
    return narrow ? launch_pairs_deg<TS, D, FMT, 4>(T, st, rec, tile_off, rank_sid, rank_mask, rank_gstart, tile_lt_base, lt, dL_dC, cam, gacc, counts, wait_limit) \
                  : launch_pairs_deg<TS, D, FMT, 2>(T, st, rec, tile_off, rank_sid, rank_mask, rank_gstart, tile_lt_base, lt, dL_dC, cam, gacc, counts, wait_limit)
    switch (deg) {
        case 0: GART_PAIRS(0);
        case 1: GART_PAIRS(1);
        case 2: GART_PAIRS(2);
        default: GART_PAIRS(3);
    }
#undef GART_PAIRS
}

}  // namespace gart

extern "C" size_t gart_backward_workspace_bytes(int64_t n) { return gart::gacc_bytes(n > 0 ? n : 1); }

// Argument checks shared by the tile-major passes; on success `v` holds the arrays of the view block.
static gart_status tile_pass_args(const gart_config* cfg, const gart_gaussians* g, const gart_camera* cam, const float* pre,
                                  const uint32_t* slot_of_gid, const uint32_t* gid_of_slot, const uint32_t* tile_off,
                                  const void* view, size_t view_bytes, int64_t cap_pairs, const float* lt, const float* dL_dcolor,
                                  const float* grad, const uint32_t* counts, const void* workspace, size_t workspace_bytes,
                                  gart::ViewLayout* v) {
    if (!cfg || !g || !cam || !counts || !tile_off || !dL_dcolor) return GART_ERR_INVALID_ARG;
    if (cfg->tile_size != 8 && cfg->tile_size != 16) return GART_ERR_INVALID_ARG;
    if (cfg->lt_layout != GART_LT_TILE_MAJOR) return GART_ERR_INVALID_ARG;   // these passes read LT in the tile-major layout
    if (!gart::kernel_degree_ok(cfg->kernel_degree)) return GART_ERR_INVALID_ARG;
    if (g->n < 0 || g->sh_degree < 0 || g->sh_degree > 3 || cap_pairs < 0) return GART_ERR_INVALID_ARG;
    if (cam->width <= 0 || cam->height <= 0) return GART_ERR_INVALID_ARG;
    if (g->n == 0) return GART_OK;
    if (!grad || !pre || !slot_of_gid || !gid_of_slot || !lt || !view || ((uintptr_t)view & 255)) return GART_ERR_INVALID_ARG;
    if (!workspace || ((uintptr_t)workspace & 255)) return GART_ERR_INVALID_ARG;
    if (gart_backward_workspace_bytes(g->n) > workspace_bytes) return GART_ERR_WORKSPACE_TOO_SMALL;
    *v = gart::view_layout(const_cast<void*>(view), g->n, cam->width, cam->height, cfg->tile_size, cap_pairs);
    if (v->bytes > view_bytes) return GART_ERR_WORKSPACE_TOO_SMALL;
    return GART_OK;
}

extern "C" gart_status gart_backward_tile(const gart_config* cfg, const gart_gaussians* g, const gart_camera* cam, const float* pre,
                                          const uint32_t* slot_of_gid, const uint32_t* gid_of_slot, const uint32_t* tile_off,
                                          const void* view, size_t view_bytes, int64_t cap_pairs,
                                          const float* lt, const float* dL_dcolor,
                                          float* grad, uint32_t* counts, void* workspace, size_t workspace_bytes, void* stream) {
    using namespace gart;
    ViewLayout v;
    gart_status s = tile_pass_args(cfg, g, cam, pre, slot_of_gid, gid_of_slot, tile_off, view, view_bytes, cap_pairs, lt, dL_dcolor, grad, counts,
                                   workspace, workspace_bytes, &v);
    if (s != GART_OK || g->n == 0) return s;
    if (cfg->lt_format != 0 && cfg->lt_format != 2) return GART_ERR_INVALID_ARG;   // this pass reads 16-byte or 8-byte LT entries
    const uint32_t *rank_sid = v.rank_sid, *rank_mask = v.rank_mask, *rank_gstart = v.rank_gstart, *tile_lt_base = v.tile_lt_base;
    cudaStream_t st = (cudaStream_t)stream;
    const Gacc gacc = make_gacc(workspace, g->n);
    s = launch_zero_accumulators(gacc, g->n, counts, st);
    if (s != GART_OK) return s;
    const CamF cf = make_camf(cam, cfg->tile_size);
    const int T = cf.tiles_x * cf.tiles_y;
    const float4* rec = reinterpret_cast<const float4*>(pre);
    const float4* lt4 = reinterpret_cast<const float4*>(lt);
#define GART_PAIRS_TS(TSV, F) launch_pairs<TSV, F>(g->sh_degree, kernel_degree_is4(cfg->kernel_degree), T, st, rec, tile_off, rank_sid, rank_mask, rank_gstart, tile_lt_base, lt4, dL_dcolor, cf, gacc, counts, wait_limit_of(cfg->wait_polls))
    if (cfg->lt_format == 0) s = cfg->tile_size == 8 ? GART_PAIRS_TS(8, 0) : GART_PAIRS_TS(16, 0);
    else s = cfg->tile_size == 8 ? GART_PAIRS_TS(8, 2) : GART_PAIRS_TS(16, 2);
#undef GART_PAIRS_TS
    if (s != GART_OK) return s;
    const float4* qs = rec + (size_t)g->n * REC_F4;   // per slot: quaternion, scale, opacity (behind the records)
    return launch_finalize(g->n, qs, slot_of_gid, gid_of_slot, gacc, grad, counts, st);
}

// ------------------------------------------------------------------------------------------------------------
// Ownership ablation (Sec. 4.4 reports warp-per-pair ownership as possible but slower): the same
// gradient with one WARP per (tile, Gaussian) pair.  Lane e takes the pair's e-th (and e+32nd ...) hit, the 11 + 3K
// terms are summed over the warp with shuffles, and lanes 0..14 flush one 16-byte piece each.  Reads the LT
// buffer in the layout made for thread ownership (a pair's entries lie 512 bytes apart).
namespace gart {

template <int MW>
__device__ __forceinline__ int nth_set_bit(const uint32_t* m, int e) {   // position of the e-th (0-based) set bit of an MW-word mask
    int base = 0;
#pragma unroll
    for (int q = 0; q < MW; ++q) {
        const int c = __popc(m[q]);
        if (e < c) return base + (int)__fns(m[q], 0, e + 1);
        e -= c;
        base += 32;
    }
    return 0;
}

template <int TS, int DEG>
__global__ void __launch_bounds__(BWD_THREADS) bwd_pairs_warp_kernel(const float4* __restrict__ rec, const uint32_t* __restrict__ tile_off,
                                                                     const uint32_t* __restrict__ rank_sid, const uint32_t* __restrict__ rank_mask,
                                                                     const uint32_t* __restrict__ rank_gstart, const uint32_t* __restrict__ tile_lt_base,
                                                                     const float4* __restrict__ lt, const float* __restrict__ dL_dC, CamF cam,
                                                                     Gacc gacc, const uint32_t* __restrict__ counts, const bool narrow) {
    constexpr int NT = TS * TS, MW = NT / 32, K = (DEG + 1) * (DEG + 1), SW = 3 * K, RS4 = REC_F4;
    constexpr int AW = (11 + SW + 3) & ~3;
    __shared__ __align__(16) float4 spix[NT * 2];   // (d, u), (g, v) per pixel, one copy: the lanes of a warp read different pixels
    if (counts[GART_CNT_ERROR]) return;
    const int tile = blockIdx.x;
    const uint32_t begin = tile_off[tile], n = tile_off[tile + 1] - begin;
    if (n == 0) return;
    const int x0 = (tile % cam.tiles_x) * TS, y0 = (tile / cam.tiles_x) * TS;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int t = threadIdx.x; t < 2 * NT; t += BWD_THREADS) {
        const int p = t >> 1, h = t & 1;
        const int x = x0 + p % TS, y = y0 + p / TS;
        float4 v = make_float4(0.f, 0.f, 0.f, h ? (float)(p / TS) : (float)(p % TS));
        if (x < cam.width && y < cam.height) {
            if (h) {
                const float* gp = dL_dC + ((size_t)y * cam.width + x) * 3;
                v.x = gp[0]; v.y = gp[1]; v.z = gp[2];
            } else {
                const float3 d = pixel_dir(cam, x, y);
                v.x = d.x; v.y = d.y; v.z = d.z;
            }
        }
        spix[2 * p + h] = v;
    }
    __syncthreads();
    const float4* lt_tile = lt + tile_lt_base[tile];
    for (uint32_t r = warp; r < n; r += BWD_WARPS) {
        const uint32_t q = begin + r;
        uint32_t m[MW];
        int c = 0;
#pragma unroll
        for (int i = 0; i < MW; ++i) { m[i] = __ldg(rank_mask + (size_t)q * MW + i); c += __popc(m[i]); }
        if (c == 0) break;   // ranks descend in hit count
        const uint32_t sid = __ldg(rank_sid + q);
        const float4* rp = rec + (size_t)sid * RS4;
        const PairGeo P = pair_geo<TS>(unpack_pre(__ldg(rp), __ldg(rp + 1), __ldg(rp + 2), __ldg(rp + 3), __ldg(rp + 4)), x0, y0);
        const float4* lp = lt_tile + __ldg(rank_gstart + q) + (r & 31u);
        float acc[AW];
#pragma unroll
        for (int i = 0; i < AW; ++i) acc[i] = 0.0f;
        for (int e = lane; e < c; e += 32) {
            const int p = nth_set_bit<MW>(m, e);
            const float4 L = __ldg(lp + (size_t)32 * e);
            const float4 pa = spix[2 * p], pb = spix[2 * p + 1];
            float3 dg, cr;
            pair_geo_at(P, pa.w, pb.w, dg, cr);
            const float inv_a = fast_rcp(fmaf(dg.x, dg.x, fmaf(dg.y, dg.y, dg.z * dg.z)));
            float Y[K], w[3];
            sh_poly<K>(make_float3(pa.x, pa.y, pa.z), Y);
            const float3 g = make_float3(pb.x, pb.y, pb.z);
            lt_weights(L, g, w);
            const float ad = fmaf(g.x, L.x, fmaf(g.y, L.y, g.z * L.z));
            const float yx = dg.y * cr.z - dg.z * cr.y, yy = dg.z * cr.x - dg.x * cr.z, yz = dg.x * cr.y - dg.y * cr.x;
            float s1 = -0.5f * ad * inv_a;
            if (narrow) s1 *= 2.0f * inv_a * fmaf(cr.x, cr.x, fmaf(cr.y, cr.y, cr.z * cr.z));   // degree-4 kernel: dL/d(D^2) = -D^2 alpha dL/dalpha
            const float s2 = s1 * inv_a;
            acc[0] = fmaf(s1, yx, acc[0]); acc[1] = fmaf(s1, yy, acc[1]); acc[2] = fmaf(s1, yz, acc[2]);
            acc[3] = fmaf(s2 * yx, yx, acc[3]); acc[4] = fmaf(s2 * yy, yy, acc[4]); acc[5] = fmaf(s2 * yz, yz, acc[5]);
            acc[6] = fmaf(s2 * yx, yy, acc[6]); acc[7] = fmaf(s2 * yx, yz, acc[7]); acc[8] = fmaf(s2 * yy, yz, acc[8]);
            acc[9] += ad;
#pragma unroll
            for (int k = 0; k < K; ++k) {
                acc[11 + 3 * k] = fmaf(Y[k], w[0], acc[11 + 3 * k]);
                acc[11 + 3 * k + 1] = fmaf(Y[k], w[1], acc[11 + 3 * k + 1]);
                acc[11 + 3 * k + 2] = fmaf(Y[k], w[2], acc[11 + 3 * k + 2]);
            }
        }
        // sum over the warp; lane i ends up with piece i (words 4 i .. 4 i + 3)
        float4 mine = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int i = 0; i < AW; ++i) {
            float v = acc[i];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
            if (lane == i / 4) {
                if (i % 4 == 0) mine.x = v;
                else if (i % 4 == 1) mine.y = v;
                else if (i % 4 == 2) mine.z = v;
                else mine.w = v;
            }
        }
        if (lane < AW / 4) atomicAdd(gacc_piece(gacc, sid, lane), mine);
    }
}

}  // namespace gart

extern "C" gart_status gart_backward_warp(const gart_config* cfg, const gart_gaussians* g, const gart_camera* cam, const float* pre,
                                          const uint32_t* slot_of_gid, const uint32_t* gid_of_slot, const uint32_t* tile_off,
                                          const void* view, size_t view_bytes, int64_t cap_pairs,
                                          const float* lt, const float* dL_dcolor,
                                          float* grad, uint32_t* counts, void* workspace, size_t workspace_bytes, void* stream) {
    using namespace gart;
    ViewLayout v;
    gart_status s = tile_pass_args(cfg, g, cam, pre, slot_of_gid, gid_of_slot, tile_off, view, view_bytes, cap_pairs, lt, dL_dcolor, grad, counts,
                                   workspace, workspace_bytes, &v);
    if (s != GART_OK || g->n == 0) return s;
    if (cfg->lt_format != 0) return GART_ERR_INVALID_ARG;
    const uint32_t *rank_sid = v.rank_sid, *rank_mask = v.rank_mask, *rank_gstart = v.rank_gstart, *tile_lt_base = v.tile_lt_base;
    cudaStream_t st = (cudaStream_t)stream;
    const Gacc gacc = make_gacc(workspace, g->n);
    s = launch_zero_accumulators(gacc, g->n, counts, st);
    if (s != GART_OK) return s;
    const CamF cf = make_camf(cam, cfg->tile_size);
    const int T = cf.tiles_x * cf.tiles_y;
    const float4* rec = reinterpret_cast<const float4*>(pre);
    const float4* lt4 = reinterpret_cast<const float4*>(lt);
#define GART_WARP(TS, D) bwd_pairs_warp_kernel<TS, D><<<T, BWD_THREADS, 0, st>>>(rec, tile_off, rank_sid, rank_mask, rank_gstart, tile_lt_base, lt4, dL_dcolor, cf, gacc, counts, kernel_degree_is4(cfg->kernel_degree))
    if (cfg->tile_size == 8) {
        switch (g->sh_degree) { case 0: GART_WARP(8, 0); break; case 1: GART_WARP(8, 1); break; case 2: GART_WARP(8, 2); break; default: GART_WARP(8, 3); break; }
    } else {
        switch (g->sh_degree) { case 0: GART_WARP(16, 0); break; case 1: GART_WARP(16, 1); break; case 2: GART_WARP(16, 2); break; default: GART_WARP(16, 3); break; }
    }
#undef GART_WARP
    GART_LAUNCH_CHECK();
    const float4* qs = rec + (size_t)g->n * REC_F4;
    return launch_finalize(g->n, qs, slot_of_gid, gid_of_slot, gacc, grad, counts, st);
}
