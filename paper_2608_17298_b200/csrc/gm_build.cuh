// Kernels that build the primitive-major work lists and the LT layout made from them (see view_layout.cuh).
// All counts live on the device; every kernel is sized by a capacity and reads the count.  No block waits on
// another: scans are three launches, the per-super-tile ranking is a warp's own counting sort.
#pragma once

#include "radix.cuh"
#include "view_layout.cuh"

namespace gart {

// tiles per slot (its pairs) and items per slot, for the two scans over the slots
struct SlotTilesF {
    const int4* srect;
    const uint32_t* counts;
    int ts;
    __device__ __forceinline__ uint32_t operator()(int64_t i) const {
        if (counts[GART_CNT_ERROR] || i >= (int64_t)counts[GART_CNT_VISIBLE]) return 0u;
        const int4 r = srect[i];
        return (uint32_t)((r.z / ts - r.x / ts + 1) * (r.w / ts - r.y / ts + 1));
    }
};
struct SlotItemsF {
    const int4* srect;
    const uint32_t* counts;
    __device__ __forceinline__ uint32_t operator()(int64_t i) const {
        if (counts[GART_CNT_ERROR] || i >= (int64_t)counts[GART_CNT_VISIBLE]) return 0u;
        const int4 r = srect[i];
        if (gm_is_whole(r)) return 1u;
        return (uint32_t)((r.z / GM_SUP - r.x / GM_SUP + 1) * (r.w / GM_SUP - r.y / GM_SUP + 1));
    }
};

static __global__ void gm_items_total_kernel(const uint64_t* total64, int64_t cap_items, uint32_t* info, uint32_t* counts) {
    const uint64_t I = total64[0];
    if (I > (uint64_t)cap_items) {   // cannot happen while the pair count fits (items <= pairs); kept as a guard
        info[GM_INFO_ITEMS] = 0u;
        atomicOr(&counts[GART_CNT_ERROR], GART_ERRBIT_PAIRS);
    } else {
        info[GM_INFO_ITEMS] = (uint32_t)I;
    }
}

// One thread per slot writes its items: key = owning super-tile, value = index in emission order.  A Gaussian cut
// into many pieces (a near one; a straddler touches every super-tile) is written by the whole warp.
constexpr int GM_EMIT_SERIAL = 16;
static __global__ void __launch_bounds__(256) gm_emit_items_kernel(const int4* __restrict__ srect, const uint32_t* __restrict__ item_off,
                                                                   int sup_x, const uint32_t* __restrict__ counts,
                                                                   uint32_t* __restrict__ keys, uint32_t* __restrict__ vals,
                                                                   uint32_t* __restrict__ em_slot) {
    if (counts[GART_CNT_ERROR]) return;
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int lane = threadIdx.x & 31;
    int sx0 = 0, sy0 = 0, nsx = 0, cnt = 0;
    uint32_t off = 0;
    if (i < (int64_t)counts[GART_CNT_VISIBLE]) {
        const int4 r = srect[i];
        sx0 = r.x / GM_SUP; sy0 = r.y / GM_SUP;
        off = item_off[i];
        if (gm_is_whole(r)) { nsx = 1; cnt = 1; }
        else { nsx = r.z / GM_SUP - sx0 + 1; cnt = nsx * (r.w / GM_SUP - sy0 + 1); }
    }
    if (cnt <= GM_EMIT_SERIAL) {
        for (int l = 0; l < cnt; ++l) {
            keys[off + l] = (uint32_t)((sy0 + l / nsx) * sup_x + sx0 + l % nsx);
            vals[off + l] = off + l;
            em_slot[off + l] = (uint32_t)i;
        }
    }
    unsigned big = __ballot_sync(0xffffffffu, cnt > GM_EMIT_SERIAL);
    while (big) {
        const int src = __ffs((int)big) - 1;
        big &= big - 1u;
        const int c = __shfl_sync(0xffffffffu, cnt, src), w = __shfl_sync(0xffffffffu, nsx, src);
        const int bx = __shfl_sync(0xffffffffu, sx0, src), by = __shfl_sync(0xffffffffu, sy0, src);
        const uint32_t o = __shfl_sync(0xffffffffu, off, src);
        const uint32_t id = (uint32_t)(i - lane + src);
        for (int l = lane; l < c; l += 32) {
            keys[o + l] = (uint32_t)((by + l / w) * sup_x + bx + l % w);
            vals[o + l] = o + l;
            em_slot[o + l] = id;
        }
    }
}

// seg_off[s] = first sorted position whose key is >= s; seg_off[nseg] = count.  (seg_off is zeroed beforehand: it stays
// zero when there is no item.)
static __global__ void __launch_bounds__(256) gm_segment_offsets_kernel(const uint32_t* __restrict__ keys_sorted, const uint32_t* __restrict__ n_dev,
                                                                        const uint32_t* __restrict__ counts, int nseg, uint32_t* __restrict__ seg_off) {
    if (counts[GART_CNT_ERROR]) return;
    const uint32_t n = *n_dev;
    const int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (p >= n) return;
    const int k = (int)keys_sorted[p];
    const int prev = p > 0 ? (int)keys_sorted[p - 1] : -1;
    for (int t = prev + 1; t <= k; ++t) seg_off[t] = (uint32_t)p;
    if (p == (int64_t)n - 1)
        for (int t = k + 1; t <= nseg; ++t) seg_off[t] = n;
}

// One thread per item in super-tile order: its descriptor (which pairs of which Gaussian) and its hit count.
template <int TS>
__global__ void __launch_bounds__(256) gm_item_desc_kernel(const uint32_t* __restrict__ keys_sorted, const uint32_t* __restrict__ vals_sorted,
                                                           const uint32_t* __restrict__ em_slot, const uint32_t* __restrict__ item_off,
                                                           const int4* __restrict__ srect, const uint32_t* __restrict__ gpair_off,
                                                           const uint32_t* __restrict__ gm_mask, int sup_x,
                                                           const uint32_t* __restrict__ info, const uint32_t* __restrict__ counts,
                                                           uint4* __restrict__ it_desc) {
    constexpr int MW = TS * TS / 32, TPS = GM_SUP / TS;   // tiles per super-tile edge
    if (counts[GART_CNT_ERROR]) return;
    const int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= (int64_t)info[GM_INFO_ITEMS]) return;
    const uint32_t i = vals_sorted[r], S = keys_sorted[r];
    const uint32_t slot = em_slot[i];
    const int4 rc = srect[slot];
    const int tx0 = rc.x / TS, ty0 = rc.y / TS, tx1 = rc.z / TS, ty1 = rc.w / TS;
    const int ntx = tx1 - tx0 + 1;
    const int sx = (int)(S % (uint32_t)sup_x), sy = (int)(S / (uint32_t)sup_x);
    int fx, fy, lx, ly;   // first and last tile of the item
    uint32_t flag;
    if (gm_is_whole(rc)) { fx = tx0; fy = ty0; lx = tx1; ly = ty1; flag = GM_DESC_WHOLE; }
    else {
        fx = max(tx0, sx * TPS); lx = min(tx1, sx * TPS + TPS - 1);
        fy = max(ty0, sy * TPS); ly = min(ty1, sy * TPS + TPS - 1);
        flag = 0u;
    }
    const uint32_t gpos0 = gpair_off[slot] + (uint32_t)((fy - ty0) * ntx + (fx - tx0));
    uint32_t c = 0;
    for (int y = fy; y <= ly; ++y)
        for (int x = fx; x <= lx; ++x) {
            const uint32_t* m = gm_mask + (size_t)(gpos0 + (uint32_t)((y - fy) * ntx + (x - fx))) * MW;
#pragma unroll
            for (int q = 0; q < MW; ++q) c += __popc(__ldg(m + q));
        }
    it_desc[r] = make_uint4(slot, gpos0, gm_pack_dims((uint32_t)ntx, (uint32_t)(lx - fx + 1), (uint32_t)(ly - fy + 1),
                                                      (uint32_t)(fx - sx * TPS), (uint32_t)(fy - sy * TPS)),
                            c | flag);
}

// Warp per super-tile: stable counting sort of its items by descending hit count -> rk_desc; 32 consecutive ranks
// form a group occupying 32 x (its largest count, rounded up to even) LT entries -> rk_gstart (relative to the
// super-tile), st_len; blocks of the backward for this super-tile -> st_parts.
constexpr int GM_RANK_WARPS = 4;
constexpr int GM_RANK_BINS = GM_WIN * GM_WIN + 1;
static __global__ void __launch_bounds__(GM_RANK_WARPS * 32) gm_rank_kernel(const uint32_t* __restrict__ st_off, const uint4* __restrict__ it_desc, int ns,
                                                                            uint4* __restrict__ rk_desc, uint32_t* __restrict__ rk_gstart,
                                                                            uint32_t* __restrict__ st_len, uint32_t* __restrict__ st_parts,
                                                                            const uint32_t* __restrict__ counts) {
    __shared__ uint32_t hist[GM_RANK_WARPS][GM_RANK_BINS];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int S = blockIdx.x * GM_RANK_WARPS + w;
    if (S >= ns) return;
    if (counts[GART_CNT_ERROR]) { if (lane == 0) { st_len[S] = 0; st_parts[S] = 0; } return; }
    const uint32_t begin = st_off[S], n = st_off[S + 1] - begin;
    if (n == 0) { if (lane == 0) { st_len[S] = 0; st_parts[S] = 0; } return; }
    for (int d = lane; d < GM_RANK_BINS; d += 32) hist[w][d] = 0;
    __syncwarp();
    constexpr int U = 4;
    auto cnt_of = [&](uint32_t r) { return min(__ldg(&it_desc[begin + r].w) & 0xffffu, (uint32_t)(GM_RANK_BINS - 1)); };
    for (uint32_t r0 = 0; r0 < n; r0 += 32 * U) {
        uint32_t c[U];
#pragma unroll
        for (int u = 0; u < U; ++u) c[u] = r0 + 32 * u + lane < n ? cnt_of(r0 + 32 * u + lane) : 0xffffffffu;
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (c[u] != 0xffffffffu) atomicAdd(&hist[w][c[u]], 1u);
    }
    __syncwarp();
    {   // first rank of every hit count, largest count first: a warp-wide exclusive scan over the bins in descending order
        uint32_t carry = 0;
        for (int hi = GM_RANK_BINS - 1; hi >= 0; hi -= 32) {
            const int b = hi - lane;
            const uint32_t v = b >= 0 ? hist[w][b] : 0u;
            const uint32_t inc = warp_incl_scan(v);
            if (b >= 0) hist[w][b] = carry + inc - v;
            carry += __shfl_sync(0xffffffffu, inc, 31);
        }
    }
    __syncwarp();
    for (uint32_t r0 = 0; r0 < n; r0 += 32 * U) {
        uint4 d[U];
        bool actv[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            actv[u] = r0 + 32 * u + lane < n;
            d[u] = actv[u] ? __ldg(&it_desc[begin + r0 + 32 * u + lane]) : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {   // in order: equal counts keep the order of the item list
            const unsigned amask = __ballot_sync(0xffffffffu, actv[u]);
            if (actv[u]) {
                const uint32_t c = min(d[u].w & 0xffffu, (uint32_t)(GM_RANK_BINS - 1));
                const unsigned peers = __match_any_sync(amask, c);
                const uint32_t rk = __popc(peers & ((1u << lane) - 1u));
                const uint32_t pos = hist[w][c] + rk;
                __syncwarp(amask);
                if (rk == 0) hist[w][c] += __popc(peers);
                __syncwarp(amask);
                rk_desc[begin + pos] = d[u];
            }
        }
    }
    __threadfence_block();
    __syncwarp();
    uint32_t run = 0;
    for (uint32_t r0 = 0; r0 < n; r0 += 32) {
        const bool act = r0 + lane < n;
        const uint32_t c = act ? (__ldcg(&rk_desc[begin + r0 + lane].w) & 0xffffu) : 0u;
        if (act) rk_gstart[begin + r0 + lane] = run;
        const uint32_t cm = __shfl_sync(0xffffffffu, c, 0);
        run += 32u * (cm + (cm & 1u));
    }
    if (lane == 0) {
        st_len[S] = run;
        const uint32_t groups = (n + 31u) / 32u;
        st_parts[S] = (groups + GM_GROUPS_PER_BLOCK - 1) / GM_GROUPS_PER_BLOCK;
    }
}

struct ArrayF {
    const uint32_t* a;
    __device__ __forceinline__ uint32_t operator()(int64_t i) const { return a[i]; }
};

// LT index of a work item's e-th hit (e counts through the item's pairs in turn) for the item of lane `lane` of a group
// that starts at entry gs: entries are interleaved two by two, entries 2m and 2m + 1 of a lane share one 32-byte sector
// (they are neighbouring pixels of one Gaussian, written by the forward close in time: whole-sector writes), the 32
// lanes' sectors of the same m are consecutive (the backward reads them as one 1 KB row).
__host__ __device__ __forceinline__ uint32_t gm_slot(uint32_t gs, uint32_t lane, uint32_t e) {
    return gs + (e >> 1) * 64u + 2u * lane + (e & 1u);
}

// Block per super-tile, thread per item: LT index of the first hit of every pair of every item (a pair's hits follow
// those of the item's earlier pairs), and the group starts made absolute.
template <int TS>
__global__ void __launch_bounds__(128) gm_ltb_kernel(const uint32_t* __restrict__ st_off, const uint32_t* __restrict__ st_lt_base, int ns,
                                                     const uint4* __restrict__ rk_desc, uint32_t* __restrict__ rk_gstart,
                                                     const uint32_t* __restrict__ gm_mask, uint32_t* __restrict__ gm_ltb,
                                                     uint32_t* __restrict__ gm_pbase, const uint32_t* __restrict__ counts) {
    constexpr int MW = TS * TS / 32;
    if (counts[GART_CNT_ERROR]) return;
    const int S = blockIdx.x;
    const uint32_t begin = st_off[S], n = st_off[S + 1] - begin;
    const uint32_t base = st_lt_base[S];
    for (uint32_t r = threadIdx.x; r < n; r += blockDim.x) {
        const uint4 d = rk_desc[begin + r];
        const uint32_t gs = rk_gstart[begin + r] + base;
        rk_gstart[begin + r] = gs;
        const uint32_t stride = d.z & 0xffffu, ntx = (d.z >> 16) & 15u, nty = (d.z >> 20) & 15u;
        const uint32_t otx = (d.z >> 24) & 15u, oty = (d.z >> 28) & 15u;
        uint32_t before = 0;
        for (uint32_t y = 0; y < nty; ++y)
            for (uint32_t x = 0; x < ntx; ++x) {
                const uint32_t gp = d.y + y * stride + x;
                gm_ltb[gp] = gm_slot(gs, r & 31u, before);
                gm_pbase[gp] = (oty + y) * TS * GM_WIN + (otx + x) * TS;
                const uint32_t* m = gm_mask + (size_t)gp * MW;
#pragma unroll
                for (int q = 0; q < MW; ++q) before += __popc(__ldg(m + q));
            }
    }
}

// The LT index of every pair's first hit and the window index of its tile origin in the tile's rank order (what the
// evaluation kernel walks); the former replaces, in place, the rank-ordered primitive-major positions.
static __global__ void __launch_bounds__(256) gm_rank_ltb_kernel(uint32_t* __restrict__ rank_gpos, const uint32_t* __restrict__ gm_ltb,
                                                                 const uint32_t* __restrict__ gm_pbase, uint32_t* __restrict__ rank_pbase,
                                                                 const uint32_t* __restrict__ counts) {
    if (counts[GART_CNT_ERROR]) return;
    const int64_t q = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= (int64_t)counts[GART_CNT_PAIRS]) return;
    const uint32_t gp = rank_gpos[q];
    rank_gpos[q] = __ldg(gm_ltb + gp);
    rank_pbase[q] = __ldg(gm_pbase + gp);
}

// (super-tile, part) of every block of the backward; the block count.
static __global__ void __launch_bounds__(256) gm_blocks_kernel(const uint32_t* __restrict__ blk_off, const uint32_t* __restrict__ st_parts, int ns,
                                                               int64_t blocks_cap, uint2* __restrict__ blk_desc, uint32_t* __restrict__ info,
                                                               const uint32_t* __restrict__ counts) {
    const int S = blockIdx.x * blockDim.x + threadIdx.x;
    if (S == 0) info[GM_INFO_BLOCKS] = counts[GART_CNT_ERROR] ? 0u : (blk_off[ns] <= (uint64_t)blocks_cap ? blk_off[ns] : 0u);
    if (S >= ns || counts[GART_CNT_ERROR]) return;
    const uint32_t b0 = blk_off[S], np = st_parts[S];
    for (uint32_t p = 0; p < np; ++p)
        if ((int64_t)(b0 + p) < blocks_cap) blk_desc[b0 + p] = make_uint2((uint32_t)S, p);
}

}  // namespace gart
