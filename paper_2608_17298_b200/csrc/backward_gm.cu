// gart_backward: primitive-centric backward (Sec. 4.4) over the primitive-major work lists.
//
// The paper gives a thread one (tile, Gaussian) pair and lets it add its sums to the Gaussian's gradient with one
// atomic update per pair.  On this GPU the arithmetic of a hit and the bytes of its LT entry are in balance, and what
// then costs most is exactly those updates: a Gaussian covers 3.6 tiles on average, so its 240-byte record is
// read, modified and written back several times, by blocks that run tens of microseconds apart (more than the
// L2 holds), and must be zeroed before and converted after.  Here a thread still gathers (tile, Gaussian) pairs, but
// it walks ALL pairs of one work item -- a whole Gaussian whenever its rectangle fits a 32 x 32-pixel window, else the
// part of a large Gaussian inside one 16 x 16 super-tile -- one after the other with the sums in registers.  A whole
// Gaussian (96 % of them at the benchmark's scale) then needs no atomic and no accumulation record: its thread converts
// the moments and writes the final 256-byte gradient record once.  Only the pieces of large Gaussians use vector
// atomics on an accumulation record (one per piece), converted by a small per-slot pass.
//
// A block serves up to GM_GROUPS_PER_BLOCK rank groups of one super-tile: it stages dL/dC of the super-tile's window in
// shared memory (one copy: 16 KB), its warps take the groups in serpentine order, lanes own items of (nearly) equal hit
// count, and the group's interleaved LT block streams in through bulk asynchronous copies (cp.async.bulk + mbarrier,
// double buffered, every wait bounded).  A 16-byte LT entry carries the index of its pixel inside the window in its low
// mantissa bits, so the hit loop touches no mask: walking per-lane masks costs more than the arithmetic of the hits
// (every lane changes pair at its own time, and each change stalls the whole warp on that lane's load).  The ray direction is affine in the pixel position before normalisation, so a
// hit recomputes it (12 instructions) instead of loading it: with lanes reading different pixels of a 1024-pixel window,
// shared-memory loads conflict, and the direction would double them.
#include "backward_common.cuh"
#include "view_layout.cuh"

namespace gart {

constexpr int GMB_WARPS = 4;
constexpr int GMB_THREADS = GMB_WARPS * 32;
constexpr int GMB_CHUNK = 6;                           // LT entries per lane and per pipeline stage (16-byte entries); even
constexpr int GMB_STAGE_F4 = GMB_CHUNK * 32;           // float4 per stage
constexpr int GMB_STAGES = 2;
constexpr int GMB_MIN_BLOCKS = 4;                      // resident blocks per SM that the register budget is set for
constexpr int GMB_LT_SMEM = GMB_WARPS * GMB_STAGES * GMB_STAGE_F4 * 16;
constexpr int GMB_PIX = GM_WIN * GM_WIN;
constexpr int GMB_PF4 = 7;                             // float4 per lane of the staged per-Gaussian data: evaluation record 5, quaternion, scale + opacity
constexpr int GMB_DYN_SMEM = GMB_LT_SMEM + GMB_PIX * 16 + GMB_THREADS * GMB_PF4 * 16;
static_assert(GMB_CHUNK % 2 == 0, "entries are interleaved two by two");
static_assert(GM_GROUPS_PER_BLOCK % GMB_WARPS == 0, "groups are dealt to the warps in rounds");

__device__ __forceinline__ float fast_rsqrt(float x) {
    float y;
    asm("rsqrt.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// float of a small non-negative integer without the conversion unit
__device__ __forceinline__ float small_int_to_float(uint32_t v) { return __uint_as_float(0x4B000000u | v) - 8388608.0f; }

// What a lane knows of its item of a rank group.
struct GmItem {
    uint4 d;           // descriptor (view_layout.cuh)
    uint32_t gstart;   // LT index of the group's block
    int c;             // hits of this lane's item (0 for a lane without item)
    int cmax;          // hits of the group's first item = the largest of the group
    bool valid;        // the lane has an item
};

__device__ __forceinline__ GmItem gm_load_item(const uint4* __restrict__ rk_desc, const uint32_t* __restrict__ rk_gstart,
                                               uint32_t begin, uint32_t n, uint32_t r0, bool in_part, int lane) {
    GmItem g;
    g.valid = in_part && r0 + lane < n;
    g.d = g.valid ? __ldg(rk_desc + begin + r0 + lane) : make_uint4(0u, 0u, 0u, 0u);
    const uint32_t gs = g.valid ? __ldg(rk_gstart + begin + r0 + lane) : 0u;
    g.c = (int)(g.d.w & 0xffffu);
    g.cmax = __shfl_sync(0xffffffffu, g.c, 0);
    g.gstart = __shfl_sync(0xffffffffu, gs, 0);
    return g;
}

// The item's geometry, affine in the window position (xf, yf): d_g = dgC + (xf - uc) c0 + (yf - vc) c1 and
// o_g x d_g = crC + (xf - uc) a1 + (yf - vc) b1, expanded about the pixel of the item's extent nearest to the Gaussian's
// reference position (o_g x d_g vanishes at the centre: about a far corner a small Gaussian's hits would be
// differences of much larger numbers).
struct ItemGeo {
    float3 c0, c1, dgC, a1, b1, crC;
    float uc, vc;
};

template <int TS>
__device__ __forceinline__ ItemGeo item_geo(const PreRec& P, const uint4 d, int wx0, int wy0) {
    ItemGeo g;
    const int ntx = (d.z >> 16) & 15, nty = (d.z >> 20) & 15, otx = (d.z >> 24) & 15, oty = (d.z >> 28) & 15;
    const int xlo = wx0 + otx * TS, ylo = wy0 + oty * TS;
    g.c0 = P.c0; g.c1 = P.c1;
    g.a1 = make_float3(P.c0.y * P.m.z - P.c0.z * P.m.y, P.c0.z * P.m.x - P.c0.x * P.m.z, P.c0.x * P.m.y - P.c0.y * P.m.x);
    g.b1 = make_float3(P.c1.y * P.m.z - P.c1.z * P.m.y, P.c1.z * P.m.x - P.c1.x * P.m.z, P.c1.x * P.m.y - P.c1.y * P.m.x);
    const int xc = min(max(P.ix, xlo), xlo + ntx * TS - 1), yc = min(max(P.iy, ylo), ylo + nty * TS - 1);
    g.uc = (float)(xc - wx0); g.vc = (float)(yc - wy0);
    const float dxc = (float)(xc - P.ix) - P.rx, dyc = (float)(yc - P.iy) - P.ry;
    g.dgC = make_float3(fmaf(P.c0.x, dxc, fmaf(P.c1.x, dyc, P.dgr.x)), fmaf(P.c0.y, dxc, fmaf(P.c1.y, dyc, P.dgr.y)),
                        fmaf(P.c0.z, dxc, fmaf(P.c1.z, dyc, P.dgr.z)));
    g.crC = make_float3(fmaf(g.a1.x, dxc, fmaf(g.b1.x, dyc, P.k.x)), fmaf(g.a1.y, dxc, fmaf(g.b1.y, dyc, P.k.y)),
                        fmaf(g.a1.z, dxc, fmaf(g.b1.z, dyc, P.k.z)));
    return g;
}

// Coefficients of the un-normalised ray direction D = A x + B y + C through pixel (x, y) of the image: the same for the
// whole launch, passed by value (operands from the constant bank: no registers).
struct DirAffine {
    float3 A, B, C;
};
static inline DirAffine make_dir_affine(const CamF& cam) {
    DirAffine d;
    const float ifx = 1.0f / cam.fx, ify = 1.0f / cam.fy;
    const float u0 = (0.5f - cam.cx) * ifx, v0 = (0.5f - cam.cy) * ify;
    d.A = make_float3(cam.r[0] * ifx, cam.r[1] * ifx, cam.r[2] * ifx);
    d.B = make_float3(cam.r[3] * ify, cam.r[4] * ify, cam.r[5] * ify);
    d.C = make_float3(cam.r[0] * u0 + cam.r[3] * v0 + cam.r[6], cam.r[1] * u0 + cam.r[4] * v0 + cam.r[7],
                      cam.r[2] * u0 + cam.r[5] * v0 + cam.r[8]);
    return d;
}

// Gradient terms of one hit added to the item's accumulators: geo[0..2] = v, geo[3..8] = Q (xx, yy, zz, xy, xz, yz),
// geo[9] = sum alpha dL/dalpha, R.acc = dL/dsh against the bare SH polynomials.
template <int K, int KD>
__device__ __forceinline__ void gm_hit(const ItemGeo& P, const DirAffine& dir, float wxf, float wyf, ShRegs<K>& R, float* geo, const float4* __restrict__ spix, int pix, const float4 L) {
    const float4 gq = spix[pix];
    const float xf = small_int_to_float((uint32_t)pix & (GM_WIN - 1)), yf = small_int_to_float((uint32_t)pix / GM_WIN);
    const float xa = xf + wxf, ya = yf + wyf;   // pixel in the image (integers below 2^22: exact)
    const float Dx = fmaf(dir.A.x, xa, fmaf(dir.B.x, ya, dir.C.x)), Dy = fmaf(dir.A.y, xa, fmaf(dir.B.y, ya, dir.C.y)),
                Dz = fmaf(dir.A.z, xa, fmaf(dir.B.z, ya, dir.C.z));
    const float inv = fast_rsqrt(fmaf(Dx, Dx, fmaf(Dy, Dy, Dz * Dz)));
    float Y[K];
    sh_poly<K>(make_float3(Dx * inv, Dy * inv, Dz * inv), Y);
    const float3 g = make_float3(gq.x, gq.y, gq.z);
    float w[3];
    lt_weights(L, g, w);
    R.accumulate(Y, w);
    const float ad = fmaf(g.x, L.x, fmaf(g.y, L.y, g.z * L.z));   // alpha dL/dalpha
    geo[9] += ad;
    const float du = xf - P.uc, dv = yf - P.vc;   // small integers: exact
    const float3 dg = make_float3(fmaf(P.c0.x, du, fmaf(P.c1.x, dv, P.dgC.x)), fmaf(P.c0.y, du, fmaf(P.c1.y, dv, P.dgC.y)),
                                  fmaf(P.c0.z, du, fmaf(P.c1.z, dv, P.dgC.z)));
    const float3 cr = make_float3(fmaf(P.a1.x, du, fmaf(P.b1.x, dv, P.crC.x)), fmaf(P.a1.y, du, fmaf(P.b1.y, dv, P.crC.y)),
                                  fmaf(P.a1.z, du, fmaf(P.b1.z, dv, P.crC.z)));
    const float inv_a = fast_rcp(fmaf(dg.x, dg.x, fmaf(dg.y, dg.y, dg.z * dg.z)));
    // y = d_g x (o_g x d_g); x_g = y / |d_g|^2
    const float yx = dg.y * cr.z - dg.z * cr.y, yy = dg.z * cr.x - dg.x * cr.z, yz = dg.x * cr.y - dg.y * cr.x;
    float s1 = -0.5f * ad * inv_a;
    if constexpr (KD == 4) s1 *= 2.0f * inv_a * fmaf(cr.x, cr.x, fmaf(cr.y, cr.y, cr.z * cr.z));   // degree-4 kernel: dL/d(D^2) = -D^2 alpha dL/dalpha
    const float s2 = s1 * inv_a;
    geo[0] = fmaf(s1, yx, geo[0]); geo[1] = fmaf(s1, yy, geo[1]); geo[2] = fmaf(s1, yz, geo[2]);
    const float tx = s2 * yx, ty = s2 * yy, tz = s2 * yz;
    geo[3] = fmaf(tx, yx, geo[3]); geo[4] = fmaf(ty, yy, geo[4]); geo[5] = fmaf(tz, yz, geo[5]);
    geo[6] = fmaf(tx, yy, geo[6]); geo[7] = fmaf(tx, yz, geo[7]); geo[8] = fmaf(ty, yz, geo[8]);
}

template <int TS, int DEG, int KD>
__global__ void __launch_bounds__(GMB_THREADS, GMB_MIN_BLOCKS) bwd_gm_kernel(const float4* __restrict__ rec, const float4* __restrict__ qs,
                                                             const uint32_t* __restrict__ gid_of_slot, const uint2* __restrict__ blk_desc,
                                                             const uint32_t* __restrict__ info, const uint32_t* __restrict__ st_off,
                                                             const uint4* __restrict__ rk_desc, const uint32_t* __restrict__ rk_gstart,
                                                             const float4* __restrict__ lt,
                                                             const float* __restrict__ dL_dC, int width, int height, const DirAffine dir,
                                                             int sup_x, Gacc gacc,
                                                             float4* __restrict__ grad4, uint32_t* __restrict__ counts,
                                                             const uint32_t wait_limit) {
    constexpr int K = (DEG + 1) * (DEG + 1), SW = 3 * K, RS4 = REC_F4;
    constexpr int AW = (11 + SW + 3) & ~3;                 // accumulator words, multiple of 4
    constexpr int EB = 16;                                 // bytes per LT entry
    constexpr int CH = GMB_STAGE_F4 * 16 / (32 * EB);      // entries per lane and per stage (even)
    constexpr int PSTR = GMB_PF4;                          // staged per-Gaussian data; odd lane stride: the lanes' 16-byte reads fall into distinct banks
    extern __shared__ __align__(128) float4 dyn[];   // [warp][2][GMB_STAGE_F4] LT stages, dL/dC of the window, [thread][PF4] per-Gaussian data
    __shared__ __align__(8) uint64_t bars[GMB_WARPS][GMB_STAGES];
    __shared__ uint32_t sgid[GMB_THREADS];   // staged id of the lane's Gaussian
    if (counts[GART_CNT_ERROR]) return;
    if (blockIdx.x >= info[GM_INFO_BLOCKS]) return;
    const uint2 bd = blk_desc[blockIdx.x];
    const int S = (int)bd.x;
    const uint32_t begin = st_off[S], n = st_off[S + 1] - begin;
    const int wx0 = (S % sup_x) * GM_SUP, wy0 = (S / sup_x) * GM_SUP;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) {
#pragma unroll
        for (int q = 0; q < GMB_STAGES; ++q) mbar_init(smem_u32(&bars[warp][q]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    float4* spix = dyn + GMB_WARPS * GMB_STAGES * GMB_STAGE_F4;
    for (int t = threadIdx.x; t < GMB_PIX; t += GMB_THREADS) {
        const int x = wx0 + (t & (GM_WIN - 1)), y = wy0 + t / GM_WIN;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (x < width && y < height) {
            const float* gp = dL_dC + ((size_t)y * width + x) * 3;
            v.x = gp[0]; v.y = gp[1]; v.z = gp[2];
        }
        spix[t] = v;
    }
    __syncthreads();
    const float wxf = (float)wx0, wyf = (float)wy0;

    float4* my_stage = dyn + (size_t)warp * GMB_STAGES * GMB_STAGE_F4;
    float4* my_par = spix + GMB_PIX + (size_t)(warp * 32 + lane) * PSTR;
    const uint32_t stage_addr = smem_u32(my_stage);
    const uint32_t par_addr = smem_u32(my_par);
    const uint32_t bar_addr = smem_u32(&bars[warp][0]);
    const char* lt_bytes = reinterpret_cast<const char*>(lt);
    // LT pipeline: unit u (a chunk of CH entries per lane, i.e. CH / 2 rows of 32 two-entry sectors) uses stage
    // u % GMB_STAGES, and the wait for it uses parity (u / GMB_STAGES) & 1.  `unit` counts the units consumed, `produced`
    // those whose copy has been issued; the producer cursor (pw, pk) = (group relative to the current one, chunk) runs up to
    // GMB_STAGES units and two groups ahead.  A group holds 32 x (its largest count rounded up to even) entries.
    uint32_t unit = 0, produced = 0;
    int pw = 0, pk = 0;
    auto produce = [&](const GmItem& a, const GmItem& b, const int c_cmax, const uint32_t c_gstart, const int maxw) {
        while (produced - unit < (uint32_t)GMB_STAGES && pw <= maxw) {
            int cm;
            uint32_t gs;
            if (pw == 0) { cm = a.cmax; gs = a.gstart; }
            else if (pw == 1) { cm = b.cmax; gs = b.gstart; }
            else { cm = c_cmax; gs = c_gstart; }
            if (cm == 0) break;                                   // ranks descend in hit count: no later group has hits
            cm += cm & 1;
            if (pk * CH >= cm) { ++pw; pk = 0; continue; }
            if (lane == 0) {
                const int ne = min(CH, cm - pk * CH);
                const uint32_t bytes = (uint32_t)ne * (32u * EB), s = produced % GMB_STAGES;
                mbar_expect_tx(bar_addr + 8u * s, bytes);
                bulk_g2s_hint(stage_addr + s * (GMB_STAGE_F4 * 16u), lt_bytes + ((size_t)gs + (size_t)pk * (CH * 32)) * EB, bytes, bar_addr + 8u * s, l2_policy_evict_first());
            }
            ++produced;
            ++pk;
        }
    };
    // copy the per-Gaussian data of a group's items into the lane's buffer, one group ahead: the evaluation record (read
    // before the hit loop) and what the final conversion needs (quaternion, scale + opacity, id: read after the loop, so
    // that they occupy no register across it)
    const uint32_t gid_addr = smem_u32(&sgid[threadIdx.x]);
    // Every issue closes one copy group, and the two kinds alternate (record of group j + 1 at the start of group j, tail
    // of group j + 1 at its end), so "all groups but the newest have landed" is exactly what each reader needs: the record
    // at the start of a group (the tail just issued may still fly), the tail at its end (the next record may still fly).
    auto issue_rec = [&](const GmItem& d) {
        if (d.valid) {
            const float4* src = rec + (size_t)d.d.x * RS4;
#pragma unroll
            for (int q = 0; q < 5; ++q) cp_async16(par_addr + 16u * q, src + q);
        }
        cp_async_commit();
    };
    auto issue_tail = [&](const GmItem& d) {
        if (d.valid && (d.d.w & GM_DESC_WHOLE)) {
            const float4* sq = qs + 2 * (size_t)d.d.x;
            cp_async16(par_addr + 16u * 5, sq);
            cp_async16(par_addr + 16u * 6, sq + 1);
            asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(gid_addr), "l"(gid_of_slot + d.d.x) : "memory");
        }
        cp_async_commit();
    };
    auto fail = [&]() {
        // a copy never completed: report, give copies that may still be in flight a second bounded chance to land
        // before this warp's shared memory may be released, and stop
        if (lane == 0) atomicOr(&counts[GART_CNT_ERROR], GART_ERRBIT_TIMEOUT);
        for (uint32_t u = unit; u != produced; ++u) mbar_wait_bounded(bar_addr + 8u * (u % GMB_STAGES), (u / GMB_STAGES) & 1u);
        cp_async_wait_all();
    };

    // The block's groups are [g0, g0 + GM_GROUPS_PER_BLOCK) of the super-tile; the warp's j-th group is
    // g0 + j * GMB_WARPS + (j even ? warp : GMB_WARPS - 1 - warp): groups descend in hit count, and this serpentine deal
    // gives every warp nearly the same number of iterations.
    const uint32_t g0 = bd.y * GM_GROUPS_PER_BLOCK;
    constexpr uint32_t ROUNDS = GM_GROUPS_PER_BLOCK / GMB_WARPS;
    auto first_rank = [&](uint32_t j) { return 32u * (g0 + j * GMB_WARPS + ((j & 1u) ? (uint32_t)(GMB_WARPS - 1 - warp) : (uint32_t)warp)); };
    auto load = [&](uint32_t j) { return gm_load_item(rk_desc, rk_gstart, begin, n, first_rank(j), j < ROUNDS, lane); };

    uint32_t gj = 0;
    GmItem cur = load(0);
    issue_rec(cur);
    issue_tail(cur);
    GmItem nxt = load(1);
    bool first = true;
    while (__any_sync(0xffffffffu, cur.valid)) {
        const GmItem nxt2 = load(gj + 2);   // (two groups ahead: its loads are in flight during this group)
        const int c2_cmax = nxt2.cmax;
        const uint32_t c2_gstart = nxt2.gstart;
        produce(cur, nxt, c2_cmax, c2_gstart, 1);
        const uint32_t sid = cur.d.x;
        const bool whole = (cur.d.w & GM_DESC_WHOLE) != 0u;
        if (first) cp_async_wait_all(); else cp_async_wait_but_one();   // this lane's record has landed (a lane reads only what it copied itself)
        first = false;
        const PreRec P = unpack_pre(my_par[0], my_par[1], my_par[2], my_par[3], my_par[4]);   // (stale data for lanes without item: never used)
        issue_rec(nxt);        // the lane has read its record: that part of its buffer may be overwritten
        const ItemGeo IG = item_geo<TS>(P, cur.d, wx0, wy0);
        ShRegs<K> R;
        R.clear();
        float geo[11];
#pragma unroll
        for (int q = 0; q < 11; ++q) geo[q] = 0.0f;
        const int cme = cur.cmax + (cur.cmax & 1);
        const int nchunks = (cme + CH - 1) / CH;
        // lanes 4..7 of every eight read the second entry of their sector first: the eight lanes that a 16-byte shared load
        // serves together then touch eight different bank groups (their sectors lie 32 bytes apart)
        const bool flip = (lane & 4) != 0;
        for (int k = 0; k < nchunks; ++k) {
            const uint32_t s = unit % GMB_STAGES;
            if (!__all_sync(0xffffffffu, mbar_wait_bounded(bar_addr + 8u * s, (unit / GMB_STAGES) & 1u, wait_limit))) { fail(); return; }
            // entries 2m and 2m + 1 of the lane: the 2 EB bytes at row m (32 lanes x 2 EB bytes) + lane x 2 EB
            const char* se = reinterpret_cast<const char*>(my_stage + s * GMB_STAGE_F4) + lane * (2 * EB);
            const int e_end = min(cur.c, (k + 1) * CH);
            for (int e = k * CH; e < e_end; e += 2, se += 64 * EB) {
                const float4 a = *reinterpret_cast<const float4*>(se + (flip ? 16 : 0));
                const float4 b = *reinterpret_cast<const float4*>(se + (flip ? 0 : 16));
                const float4 L0 = flip ? b : a, L1 = flip ? a : b;
                // two hits per iteration: two independent dependency chains for the scheduler to interleave; the entry
                // names its pixel
                if (e + 1 < e_end) {
                    gm_hit<K, KD>(IG, dir, wxf, wyf, R, geo, spix, (int)lt_pix(L0), L0);
                    gm_hit<K, KD>(IG, dir, wxf, wyf, R, geo, spix, (int)lt_pix(L1), L1);
                } else {
                    gm_hit<K, KD>(IG, dir, wxf, wyf, R, geo, spix, (int)lt_pix(L0), L0);
                }
            }
            fence_proxy_async();
            __syncwarp();   // every lane is done with this stage before a later copy may overwrite it
            ++unit;
            produce(cur, nxt, c2_cmax, c2_gstart, 2);
        }
        // ---- the item's sums leave the registers
        if (cur.valid) {
            if (whole) {
                // the thread holds every hit of its Gaussian: convert the moments and write the gradient record once
                cp_async_wait_but_one();   // (the tail data of this group; the next group's record may still be in flight)
                const float4 q4 = my_par[5], s4 = my_par[6];
                const uint32_t gid = sgid[threadIdx.x];
                const float qv[4] = {q4.x, q4.y, q4.z, q4.w};
                const float sc[3] = {s4.x, s4.y, s4.z};
                const GeoGrad o = moments_to_grads(geo, geo + 3, qv, sc);
                const float gw[11] = {o.dmu[0], o.dmu[1], o.dmu[2], o.ds[0], o.ds[1], o.ds[2], o.dq[0], o.dq[1], o.dq[2], o.dq[3], geo[9] / s4.w};
                float4* out = grad4 + (size_t)gid * (GART_GRAD_WORDS / 4);
#pragma unroll
                for (int q = 0; q < GART_GRAD_WORDS / 4; ++q) {
                    float v[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int wd = 4 * q + i;
                        v[i] = wd < 11 ? gw[wd] : (wd < 11 + SW ? sh_norm((wd - 11) / 3) * R.word(wd - 11) : 0.0f);
                    }
                    __stcs(out + q, make_float4(v[0], v[1], v[2], v[3]));
                }
            } else if (cur.c != 0) {
                // a piece of a large Gaussian: one vector atomic per 16 bytes of the slot's accumulation record
                const uint64_t pol_keep = l2_policy_evict_last();
#pragma unroll
                for (int q = 0; q < AW / 4; ++q) {
                    float v[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int wd = 4 * q + i;
                        v[i] = wd < 10 ? geo[wd] : (wd >= 11 && wd < 11 + SW ? R.word(wd - 11) : 0.0f);
                    }
                    red_add_f4_hint(gacc_piece(gacc, sid, q), v[0], v[1], v[2], v[3], pol_keep);
                }
            }
        }
        issue_tail(nxt);   // (its conversion data: the lane has read the current item's)
        cur = nxt;
        nxt = nxt2;
        ++gj;
        --pw;
        if (pw < 0) { pw = 0; pk = 0; }   // (a group without hits leaves the producer behind: it restarts at the new current group)
    }
    cp_async_wait_all();
}

// ---- the large Gaussians (cut into pieces): zero their accumulation records before, convert them after.  One thread
// per slot looks at the rectangle; the few large ones (a few per cent) do the work.
static __global__ void __launch_bounds__(256) gm_zero_big_kernel(const int4* __restrict__ srect, Gacc gacc, const uint32_t* __restrict__ counts) {
    if (counts[GART_CNT_ERROR]) return;
    const int64_t sid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (sid >= (int64_t)counts[GART_CNT_VISIBLE]) return;
    if (gm_is_whole(__ldg(srect + sid))) return;
#pragma unroll
    for (int q = 0; q < (GACC_A_WORDS + GACC_B_WORDS) / 4; ++q) *gacc_piece(gacc, (uint32_t)sid, q) = make_float4(0.f, 0.f, 0.f, 0.f);
}

static __global__ void __launch_bounds__(256) gm_convert_big_kernel(const int4* __restrict__ srect, const float4* __restrict__ qs,
                                                                    const uint32_t* __restrict__ gid_of_slot, Gacc gacc,
                                                                    float4* __restrict__ grad4, const uint32_t* __restrict__ counts) {
    if (counts[GART_CNT_ERROR]) return;
    constexpr int F4 = GART_GRAD_WORDS / 4;
    const int64_t sid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (sid >= (int64_t)counts[GART_CNT_VISIBLE]) return;
    if (gm_is_whole(__ldg(srect + sid))) return;
    float4* out = grad4 + (size_t)gid_of_slot[sid] * F4;
    const float4* gp = reinterpret_cast<const float4*>(gacc.a) + (size_t)sid * (GACC_A_WORDS / 4);
    const float4 a = gp[0], b = gp[1], c = gp[2], d = gp[3];
    const float4 q4 = qs[2 * sid], s4 = qs[2 * sid + 1];
    const float v[3] = {a.x, a.y, a.z};
    const float Q[6] = {a.w, b.x, b.y, b.z, b.w, c.x};
    const float q[4] = {q4.x, q4.y, q4.z, q4.w};
    const float sc[3] = {s4.x, s4.y, s4.z};
    const GeoGrad o = moments_to_grads(v, Q, q, sc);
    out[0] = make_float4(o.dmu[0], o.dmu[1], o.dmu[2], o.ds[0]);
    out[1] = make_float4(o.ds[1], o.ds[2], o.dq[0], o.dq[1]);
    out[2] = make_float4(o.dq[2], o.dq[3], c.y / s4.w, sh_word_norm(11) * c.w);
    out[3] = make_float4(sh_word_norm(12) * d.x, sh_word_norm(13) * d.y, sh_word_norm(14) * d.z, sh_word_norm(15) * d.w);
    const float4* bp = reinterpret_cast<const float4*>(gacc.b) + (size_t)sid * (GACC_B_WORDS / 4);
#pragma unroll
    for (int l = 4; l < 15; ++l) {
        const float4 t = bp[l - 4];
        out[l] = make_float4(sh_word_norm(4 * l) * t.x, sh_word_norm(4 * l + 1) * t.y, sh_word_norm(4 * l + 2) * t.z,
                             4 * l + 3 < 59 ? sh_word_norm(4 * l + 3) * t.w : 0.0f);
    }
    out[15] = make_float4(0.f, 0.f, 0.f, 0.f);
}

// A zero record for every Gaussian without a slot: a thread looks at one Gaussian, the warp then writes the flagged
// records two at a time (16 lanes per 256-byte record).
static __global__ void __launch_bounds__(256) gm_fill_kernel(int64_t n, const uint32_t* __restrict__ slot_of_gid, float4* __restrict__ grad4,
                                                             const uint32_t* __restrict__ counts) {
    if (counts[GART_CNT_ERROR]) return;
    const int64_t gid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int lane = threadIdx.x & 31;
    const bool none = gid < n && __ldg(slot_of_gid + gid) == 0xffffffffu;
    unsigned m = __ballot_sync(0xffffffffu, none);
    const int64_t g0 = gid - lane;
    while (m) {
        const int a = __ffs((int)m) - 1;
        m &= m - 1u;
        int b = -1;
        if (m) { b = __ffs((int)m) - 1; m &= m - 1u; }
        const int mine = lane < 16 ? a : b;
        if (mine >= 0) __stcs(grad4 + (size_t)(g0 + mine) * (GART_GRAD_WORDS / 4) + (lane & 15), make_float4(0.f, 0.f, 0.f, 0.f));
    }
}

template <int TS>
static gart_status launch_gm(int deg, bool narrow, unsigned grid, cudaStream_t st, const float4* rec, const float4* qs, const uint32_t* gid_of_slot,
                             const ViewLayout& v, const float4* lt, const float* dL_dC, const CamF& cam, int sup_x, const Gacc& gacc,
                             float4* grad4, uint32_t* counts, uint32_t wait_limit) {
#define GART_GM(D)                                                                                                                \
    {                                                                                                                            \
        auto kern = narrow ? bwd_gm_kernel<TS, D, 4> : bwd_gm_kernel<TS, D, 2>;                                                   \
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, GMB_DYN_SMEM) != cudaSuccess) return GART_ERR_CUDA; \
        kern<<<grid, GMB_THREADS, GMB_DYN_SMEM, st>>>(rec, qs, gid_of_slot, v.blk_desc, v.info, v.st_off, v.rk_desc, v.rk_gstart, lt, \
                                                      dL_dC, cam.width, cam.height, make_dir_affine(cam), sup_x, gacc, grad4, counts, wait_limit); \
    }
    switch (deg) {
        case 0: GART_GM(0); break;
        case 1: GART_GM(1); break;
        case 2: GART_GM(2); break;
        default: GART_GM(3); break;
    }
#undef GART_GM
    GART_LAUNCH_CHECK();
    return GART_OK;
}

}  // namespace gart

extern "C" gart_status gart_backward(const gart_config* cfg, const gart_gaussians* g, const gart_camera* cam, const float* pre,
                                     const uint32_t* slot_of_gid, const uint32_t* gid_of_slot, const uint32_t* tile_off,
                                     const void* view, size_t view_bytes, int64_t cap_pairs,
                                     const float* lt, const float* dL_dcolor,
                                     float* grad, uint32_t* counts, void* workspace, size_t workspace_bytes, void* stream) {
    using namespace gart;
    (void)tile_off;
    if (!cfg || !g || !cam || !counts || !dL_dcolor) return GART_ERR_INVALID_ARG;
    if (cfg->tile_size != 8 && cfg->tile_size != 16) return GART_ERR_INVALID_ARG;
    if (cfg->lt_layout == GART_LT_TILE_MAJOR)    // the other layout: the block-per-tile pass reads it
        return gart_backward_tile(cfg, g, cam, pre, slot_of_gid, gid_of_slot, tile_off, view, view_bytes, cap_pairs, lt, dL_dcolor, grad, counts,
                                  workspace, workspace_bytes, stream);
    if (cfg->lt_layout != GART_LT_PRIMITIVE_MAJOR) return GART_ERR_INVALID_ARG;
    if (cfg->lt_format != 0) return GART_ERR_INVALID_ARG;                          // the item pass reads 16-byte LT entries (they name their pixel)
    if (!kernel_degree_ok(cfg->kernel_degree)) return GART_ERR_INVALID_ARG;
    if (g->n < 0 || g->sh_degree < 0 || g->sh_degree > 3 || cap_pairs < 0) return GART_ERR_INVALID_ARG;
    if (cam->width <= 0 || cam->height <= 0) return GART_ERR_INVALID_ARG;
    if (g->n == 0) return GART_OK;
    if (!grad || !pre || !slot_of_gid || !gid_of_slot || !lt || !view || ((uintptr_t)view & 255)) return GART_ERR_INVALID_ARG;
    if (!workspace || ((uintptr_t)workspace & 255)) return GART_ERR_INVALID_ARG;
    if (gart_backward_workspace_bytes(g->n) > workspace_bytes) return GART_ERR_WORKSPACE_TOO_SMALL;
    const ViewLayout v = view_layout(const_cast<void*>(view), g->n, cam->width, cam->height, cfg->tile_size, cap_pairs);
    if (v.bytes > view_bytes) return GART_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t st = (cudaStream_t)stream;
    const Gacc gacc = make_gacc(workspace, g->n);
    const CamF cf = make_camf(cam, cfg->tile_size);
    const int sup_x = (cam->width + GM_SUP - 1) / GM_SUP;
    const float4* rec = reinterpret_cast<const float4*>(pre);
    const int rs4 = REC_F4;
    const float4* qs = rec + (size_t)g->n * rs4;                                         // per slot: quaternion, scale, opacity
    const int4* srect = reinterpret_cast<const int4*>(rec + (size_t)g->n * (rs4 + 2));   // per slot: rectangle
    const float4* lt4 = reinterpret_cast<const float4*>(lt);
    float4* grad4 = reinterpret_cast<float4*>(grad);
    const unsigned slot_blocks = (unsigned)ceil_div(g->n, 256);
    gm_zero_big_kernel<<<slot_blocks, 256, 0, st>>>(srect, gacc, counts);
    GART_LAUNCH_CHECK();
    gm_fill_kernel<<<slot_blocks, 256, 0, st>>>(g->n, slot_of_gid, grad4, counts);
    GART_LAUNCH_CHECK();
    const unsigned grid = (unsigned)v.blocks_cap;
    gart_status s;
    if (cfg->tile_size == 8) s = launch_gm<8>(g->sh_degree, kernel_degree_is4(cfg->kernel_degree), grid, st, rec, qs, gid_of_slot, v, lt4, dL_dcolor, cf, sup_x, gacc, grad4, counts, wait_limit_of(cfg->wait_polls));
    else s = launch_gm<16>(g->sh_degree, kernel_degree_is4(cfg->kernel_degree), grid, st, rec, qs, gid_of_slot, v, lt4, dL_dcolor, cf, sup_x, gacc, grad4, counts, wait_limit_of(cfg->wait_polls));
    if (s != GART_OK) return s;
    gm_convert_big_kernel<<<slot_blocks, 256, 0, st>>>(srect, qs, gid_of_slot, gacc, grad4, counts);
    GART_LAUNCH_CHECK();
    return GART_OK;
}
