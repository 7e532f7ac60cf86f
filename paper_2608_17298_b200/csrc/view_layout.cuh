// The per-view layout block: every private array that gart_forward builds for the backward passes, carved
// from one caller-owned buffer (size: gart_view_bytes).  Two families of arrays live here.
//
// Tile-major (Sec. 4.3, 4.4: block per tile): per (tile, Gaussian) pair the hit mask, the rank of the pair
// in its tile's descending hit-count order, and copies of slot id and mask in rank order; the LT layout made
// from them groups 32 consecutive ranks of a tile.
//
// Primitive-major: the same pairs seen from the Gaussian.  The image is cut into "super-tiles" of
// GM_SUP x GM_SUP pixels; a Gaussian whose rectangle spans at most two super-tiles per axis is ONE work item
// owned by the super-tile of its rectangle's corner (its pixels then lie in the 2 x 2 super-tile window of the
// owner); larger Gaussians are cut at the super-tile grid into one item per super-tile they touch.  The items
// of a super-tile are ranked by descending hit count, 32 consecutive ranks form a group whose LT entries are
// interleaved (entry e of lane l at 32 e + l), and a thread of the backward pass walks all (tile, Gaussian)
// pairs of its item with the accumulators in registers: a Gaussian that is one item needs no atomic update and
// no accumulation record at all.
#pragma once

#include "common.cuh"

namespace gart {

constexpr int GM_SUP = 16;              // super-tile edge in pixels (a multiple of both tile sizes)
constexpr int GM_WIN = 2 * GM_SUP;      // window edge: an item's pixels lie within GM_WIN x GM_WIN of its owner's origin
constexpr int GM_GROUPS_PER_BLOCK = 16; // rank groups of one super-tile handled by one block of the backward

// words of the info block (device): counts that only the device knows
enum { GM_INFO_ITEMS = 0, GM_INFO_BLOCKS = 1, GM_INFO_WORDS = 64 };

struct ViewLayout {
    // tile-major
    uint32_t *pair_mask, *pair_order, *rank_sid, *rank_mask, *rank_gstart, *tile_lt_base;
    uint32_t *pair_gpos, *rank_gpos;   // primitive-major position of every pair, in pair order and in rank order
    uint32_t *gm_pbase, *rank_pbase;   // index (y * GM_WIN + x) of the pair's tile origin in its owner's window, by primitive-major position and in rank order
    // primitive-major
    uint32_t* gpair_off;    // [n+1]  first primitive-major pair position of every slot
    uint32_t* gm_mask;      // [cap_pairs, MW] hit masks in primitive-major order (a Gaussian's tiles row by row)
    uint32_t* gm_ltb;       // [cap_pairs] LT index of the first hit of every pair, by primitive-major position
    uint32_t* item_off;     // [n+1]  first item (in emission order) of every slot
    uint32_t* em_slot;      // [cap_pairs] slot of every item in emission order
    uint4* it_desc;         // [cap_pairs] item descriptors in super-tile order (before ranking)
    uint4* rk_desc;         // [cap_pairs] item descriptors, per super-tile in rank order
    uint32_t* rk_gstart;    // [cap_pairs] LT index of the item's group
    uint32_t* st_off;       // [NS+1] first item of every super-tile
    uint32_t* st_len;       // [NS+1] LT entries of every super-tile
    uint32_t* st_lt_base;   // [NS+1]
    uint32_t* st_parts;     // [NS+1] blocks of every super-tile
    uint32_t* blk_off;      // [NS+1]
    uint2* blk_desc;        // [blocks_cap] (super-tile, part) of every block of the backward
    uint32_t* info;         // [GM_INFO_WORDS]
    int64_t blocks_cap;
    int ns;
    size_t bytes;
};

static inline int gm_super_tiles(int width, int height) {
    return ((width + GM_SUP - 1) / GM_SUP) * ((height + GM_SUP - 1) / GM_SUP);
}

static inline int64_t gm_blocks_cap(int ns, int64_t cap_pairs) {
    // a super-tile with G groups takes ceil(G / GM_GROUPS_PER_BLOCK) blocks; groups in all <= items / 32 + NS
    return (int64_t)ns + (cap_pairs / 32 + ns) / GM_GROUPS_PER_BLOCK + 1;
}

static inline ViewLayout view_layout(void* base, int64_t n, int width, int height, int ts, int64_t cap_pairs) {
    ViewLayout v;
    char* p = (char*)base;
    size_t off = 0;
    auto take = [&](size_t b) { void* r = p ? (void*)(p + off) : nullptr; off += align256(b > 0 ? b : 1); return r; };
    const int64_t nn = n > 0 ? n : 1, cp = cap_pairs > 0 ? cap_pairs : 1;
    const int T = ((width + ts - 1) / ts) * ((height + ts - 1) / ts);
    const int mw = ts * ts / 32;
    v.ns = gm_super_tiles(width, height);
    v.blocks_cap = gm_blocks_cap(v.ns, cp);
    v.pair_mask = (uint32_t*)take((size_t)cp * 4 * mw);
    v.pair_order = (uint32_t*)take((size_t)cp * 4);
    v.rank_sid = (uint32_t*)take((size_t)cp * 4);
    v.rank_mask = (uint32_t*)take((size_t)cp * 4 * mw);
    v.rank_gstart = (uint32_t*)take((size_t)cp * 4);
    v.tile_lt_base = (uint32_t*)take((size_t)(T + 1) * 4);
    v.pair_gpos = (uint32_t*)take((size_t)cp * 4);
    v.rank_gpos = (uint32_t*)take((size_t)cp * 4);
    v.gm_pbase = (uint32_t*)take((size_t)cp * 4);
    v.rank_pbase = (uint32_t*)take((size_t)cp * 4);
    v.gpair_off = (uint32_t*)take((size_t)(nn + 1) * 4);
    v.gm_mask = (uint32_t*)take((size_t)cp * 4 * mw);
    v.gm_ltb = (uint32_t*)take((size_t)cp * 4);
    v.item_off = (uint32_t*)take((size_t)(nn + 1) * 4);
    v.em_slot = (uint32_t*)take((size_t)cp * 4);
    v.it_desc = (uint4*)take((size_t)cp * 16);
    v.rk_desc = (uint4*)take((size_t)cp * 16);
    v.rk_gstart = (uint32_t*)take((size_t)cp * 4);
    v.st_off = (uint32_t*)take((size_t)(v.ns + 1) * 4);
    v.st_len = (uint32_t*)take((size_t)(v.ns + 1) * 4);
    v.st_lt_base = (uint32_t*)take((size_t)(v.ns + 1) * 4);
    v.st_parts = (uint32_t*)take((size_t)(v.ns + 1) * 4);
    v.blk_off = (uint32_t*)take((size_t)(v.ns + 1) * 4);
    v.blk_desc = (uint2*)take((size_t)v.blocks_cap * 8);
    v.info = (uint32_t*)take(GM_INFO_WORDS * 4);
    v.bytes = off;
    return v;
}

// ---- item descriptor (uint4)
//   x: slot of the Gaussian
//   y: primitive-major position of the item's first pair
//   z: row stride between the item's tile rows in primitive-major positions (the Gaussian's tiles per row) in the low
//      16 bits, then 4 bits each: tiles per row of the item, tile rows of the item, x and y of its first tile
//      relative to the owner's window origin (in tiles)
//   w: hits of the item in the low 16 bits (at most GM_WIN^2), bit 16: the item is the whole Gaussian
constexpr uint32_t GM_DESC_WHOLE = 1u << 16;
__host__ __device__ __forceinline__ uint32_t gm_pack_dims(uint32_t stride, uint32_t ntx, uint32_t nty, uint32_t otx, uint32_t oty) {
    return (stride & 0xffffu) | (ntx << 16) | (nty << 20) | (otx << 24) | (oty << 28);
}

// Is the Gaussian with pixel rectangle r one item (its rectangle spans at most two super-tiles per axis)?
__host__ __device__ __forceinline__ bool gm_is_whole(const int4 r) {
    return (r.z / GM_SUP - r.x / GM_SUP) <= 1 && (r.w / GM_SUP - r.y / GM_SUP) <= 1;
}

}  // namespace gart
