/*
 * gart.h -- C ABI of the B200 (sm_100a) library for the hot path of primitive-centric
 * ray-traced Gaussian rendering (3DGART).
 *
 * One view is processed by four calls, in this order:
 *
 *   gart_bounds    per-Gaussian conservative screen rectangle and ray-evaluation record
 *   gart_tile_map  (tile, Gaussian) pair list, radix-sorted by tile, and the tile offset table
 *   gart_forward   ray evaluation: hits ordered by maximum-response distance, compositing,
 *                  and the compact per-hit buffer LT (16 bytes per hit: alpha dC/dalpha and the
 *                  blending weight T alpha, see gart_forward)
 *   gart_backward  primitive-centric backward, in the decomposition that matches the layout of LT
 *                  (cfg->lt_layout): tile-major -- the paper's: block per tile, thread per (tile, Gaussian)
 *                  pair, one vector atomic update per pair (the faster whole step on B200); primitive-major
 *                  -- a thread gathers the gradients of one Gaussian over the hit pixels of all its pairs
 *                  and writes its record once (half the DRAM traffic of the pass, a dearer forward)
 *   gart_backward_tile     the tile-major pass by name (what gart_backward runs for that layout)
 *   gart_backward_atomic   the pixel-centric baseline: one thread per ray, atomicAdd per hit
 *   gart_backward_warp     gart_backward_tile with a warp per pair (ownership ablation)
 *   gart_backward_hybrid   colour gradients primitive-centric from 4 bytes per hit, the rest pixel-centric
 *
 * Conventions
 *   - Every array pointer is a DEVICE pointer owned by the caller unless the comment says
 *     "host".  Arrays are dense, row-major, fp32 unless the type says otherwise.
 *   - The library allocates no device memory.  Scratch comes from a caller-supplied
 *     workspace whose size is returned by the matching *_workspace_bytes query (or by
 *     gart_workspace_bytes, the largest of them); the workspace must be 256-byte aligned
 *     and may be reused by the next call on the same stream.  What gart_forward builds for
 *     the backward passes beside LT (hit masks, work lists, the LT layout) lives in one
 *     opaque, caller-owned "view block" of gart_view_bytes bytes, 256-byte aligned, which
 *     must stay untouched between gart_forward and the backward pass of the same view.
 *   - There is no context object: the configuration travels with every call as a host
 *     struct, the per-view state is the caller's buffers, and what the device alone can
 *     see comes back through the counts block (gart_sync_status reads it and turns its
 *     error bits into a status).
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  All calls
 *     are asynchronous; none synchronises with the host.
 *   - Return value: GART_OK or an error code from argument checking / kernel launch.
 *     Conditions only the device can see (a capacity that turns out too small) are
 *     recorded in the counts block (GART_CNT_ERROR) and skip the affected work; read
 *     the block back with gart_read_counts after synchronising.
 *   - Camera: pinhole, x right, y down, z forward; pixel (x,y) has its centre at
 *     (x+0.5, y+0.5); world-to-camera matrix [R|t] row-major; unit ray direction
 *     d = normalize(R^T ((x+0.5-cx)/fx, (y+0.5-cy)/fy, 1)), origin o = -R^T t.
 *   - Quaternions are (w,x,y,z) and used as given (no normalisation).
 *   - Tiles are tile_size x tile_size pixels (8 or 16); tile id = ty * tiles_x + tx with
 *     tiles_x = ceil(width / tile_size).
 */
#ifndef GART_H
#define GART_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    GART_OK = 0,
    GART_ERR_INVALID_ARG = 1,
    GART_ERR_WORKSPACE_TOO_SMALL = 2,
    GART_ERR_CAPACITY_EXCEEDED = 3,
    GART_ERR_CUDA = 4,
    GART_ERR_TIMEOUT = 5          /* a bounded wait on an asynchronous copy inside a kernel ran out (gart_sync_status) */
} gart_status;

/* Layouts of the intermediate buffer LT (gart_config.lt_layout). */
enum {
    GART_LT_PRIMITIVE_MAJOR = 0,  /* hits grouped by Gaussian (work items of a 16 x 16-pixel super-tile): gart_backward's item pass */
    GART_LT_TILE_MAJOR = 1        /* hits grouped by (tile, Gaussian) pair inside each tile: gart_backward's block-per-tile pass
                                     (= gart_backward_tile), gart_backward_warp, gart_backward_hybrid.  The faster whole step:
                                     callers that do not care should set this one (the Python binding's default). */
};

/* Host struct. */
typedef struct {
    float alpha_min;      /* minimum response of a hit; the paper uses 1/255 (Sec. 3.4) */
    float near_z;         /* depth of the near plane used only to classify Gaussians */
    float background[3];  /* colour multiplied by the final transmittance */
    int32_t tile_size;    /* 8 (the paper's choice, Sec. 4.4) or 16 */
    int32_t lt_format;    /* what gart_forward stores per hit: 0 = the 16-byte entry that gart_backward reads,
                             1 = only its fourth word, 4 bytes per hit (for gart_backward_hybrid, Sec. 4.4
                             "Hybrid approach"); lt then holds cap_hits floats;
                             2 = the entry as four halves, 8 bytes per hit (the half-precision buffer that the
                             paper's limitations section, "VRAM Consumption", names as a way to save
                             memory), for gart_backward_tile; formats 1 and 2 need lt_layout = GART_LT_TILE_MAJOR */
    int32_t max_hits;     /* 0: every hit of a ray is composited (the paper's benchmark sets no hit cap, Sec. 5).
                             m > 0: gart_forward composites only the first m hits of a ray in (t*, id)
                             order, the cap that the paper lists among the compromises of 3DGRT.  The hits behind
                             the cap keep their place in every list and their LT slot, with a zero entry: they
                             add nothing to the colour, to T_final or to a gradient (the backward passes that
                             read lt need no change; gart_backward_hybrid rejects a cap) */
    int32_t lt_layout;    /* GART_LT_PRIMITIVE_MAJOR (0) or GART_LT_TILE_MAJOR (1): where gart_forward puts a hit's entry in lt,
                             and with it which pass gart_backward runs.  The entries' contents are the same (the
                             primitive-major entries also carry their pixel's index in low mantissa bits).  gart_bounds
                             reads it too (the order of the slots follows the layout): use one value for a whole view. */
    float t_min;          /* 0: off (the paper's setting).  > 0: early termination, as in the tracers the paper compares with
                             (Sec. 5.5): a ray ends before the first hit whose transmittance in front is below t_min; that
                             hit and the later ones keep their place in every list and get a zero LT entry, like the hits
                             behind max_hits; T_final is the transmittance reached */
    float alpha_max;      /* >= 1: off (the paper's setting).  < 1: a hit's alpha is min(sigma rho, alpha_max).  Where the
                             clamp is active alpha is a constant: the hit's LT entry has zero words 0..2 (no gradient to
                             opacity, mean, scale, rotation) and w = T alpha_max (its colour still gets its gradient).
                             gart_backward_hybrid takes neither option (it re-derives every alpha) */
    int32_t atomic_mode;  /* gart_backward_atomic only.  GART_ATOMIC_SCALAR (0): one atomicAdd per gradient word per hit, the
                             form Sec. 3.5 describes; GART_ATOMIC_VECTOR (1): the same sums as 16-byte vector reductions,
                             ceil((11 + 3K) / 4) per hit (15 at degree 3), the strongest plain form of the scatter on
                             this hardware */
    int32_t wait_polls;   /* 0: the library's limit (2^22 polls) on every wait of a kernel for one of its own asynchronous
                             copies; > 0: that many polls; < 0: no poll at all, so every such wait gives up at once (a test
                             hook for the path below).  A wait that gives up sets GART_ERRBIT_TIMEOUT in
                             counts[GART_CNT_ERROR]; the warp then waits, with the library's limit, for its copies in flight
                             and returns.  The call's outputs are then undefined, the context stays usable, and
                             gart_sync_status returns GART_ERR_TIMEOUT.  Read by gart_backward, gart_backward_tile and
                             gart_backward_hybrid (the kernels that stream the intermediate buffer through shared memory). */
    int32_t kernel_degree; /* k of the response rho = exp(-D^k / 2), D the Mahalanobis distance of the ray's closest point (Eq. 5).
                             0 or 2: the Gaussian of Eq. 4, the paper's setting (Sec. 5.2).  4: a narrow kernel, the last of the
                             compromises that Sec. 5.5 lists for 3DGRT (flatter top, faster fall-off); the paper prints no
                             formula for it, this is the reading taken.  The clamping radius of Eq. 9-10 becomes
                             (2 ln(sigma / alpha_min))^(1/k), the maximum-response point and t* do not change, and
                             d alpha / d(D^2) = -alpha (k/4) (D^2)^(k/2 - 1).  Read by gart_bounds, gart_forward and every
                             backward pass (use one value for a whole view); other values are GART_ERR_INVALID_ARG, and so is
                             4 in gart_backward_hybrid */
} gart_config;

/* Host struct. */
typedef struct {
    int32_t width, height;
    double fx, fy, cx, cy;
    double w2c[12];       /* row-major [R | t] */
} gart_camera;

/* Host struct holding device pointers (Sec. 3.1: mean, Sigma = R S S^T R^T, opacity, SH radiance). */
typedef struct {
    int64_t n;
    int32_t sh_degree;     /* 0..3; K = (sh_degree+1)^2 coefficients per channel */
    const float *mean;     /* [n,3] */
    const float *scale;    /* [n,3] */
    const float *quat;     /* [n,4] (w,x,y,z) */
    const float *opacity;  /* [n]   */
    const float *sh;       /* [n,K,3] */
} gart_gaussians;

/* Words of the counts block (device memory, GART_COUNTS_WORDS x uint32, zeroed by gart_bounds). */
enum {
    GART_CNT_VISIBLE = 0,   /* Gaussians with a non-empty rectangle */
    GART_CNT_PAIRS = 1,     /* P: (tile, Gaussian) pairs */
    GART_CNT_SLOTS_LO = 2,  /* S = sum of rectangle areas, low/high words: the capacity bound */
    GART_CNT_SLOTS_HI = 3,  /*     of the intermediate buffer (Eq. 15 with lambda_s = 1)      */
    GART_CNT_HITS = 4,      /* H: ray-Gaussian hits of the view = entries used in LT */
    GART_CNT_ERROR = 5,     /* bit 0: pair capacity exceeded; bit 1: hit capacity exceeded (L > cap_hits); bit 2: timeout */
    GART_CNT_MAX_RAY_HITS = 6,
    GART_CNT_STRADDLE = 7,  /* Gaussians whose support crosses the near plane */
    GART_CNT_LT_SLOTS = 8,  /* L >= H: entries of LT in use, including the padding of its interleaved layout */
    GART_COUNTS_WORDS = 12
};
#define GART_ATOMIC_SCALAR 0
#define GART_ATOMIC_VECTOR 1

#define GART_ERRBIT_PAIRS 1u
#define GART_ERRBIT_HITS 2u
#define GART_ERRBIT_TIMEOUT 4u   /* a bounded wait on an asynchronous copy gave up (never expected) */

#define GART_GRAD_WORDS 64  /* stride of a gradient record: mean 3, scale 3, quat 4, opacity 1,
                               sh 3K (coefficient-major, channel-minor, as the input), zero padding */

const char *gart_status_string(gart_status s);

/* Words (uint32) of hit mask per pair: tile_size^2 / 32. */
int32_t gart_mask_words(int32_t tile_size);

/*
 * Step 1 -- conservative perspective-correct bounds (Sec. 4.2, Eq. 11-14) with the opacity
 * dependent clamping radius alpha_c = sqrt(2 ln(sigma/alpha_min)) (Eq. 10), evaluated in
 * double precision, and the pre-computations of the ray evaluation (W = S^-1 R^T and o_g of
 * Eq. 5, expressed relative to a per-Gaussian reference pixel so that fp32 evaluation stays
 * well conditioned).  Gaussians with a non-empty rectangle are renumbered for the view: a stable
 * sort on the 16 x 16-pixel super-tile of the rectangle's corner ((y0 / 16) * ceil(width / 16) + x0 / 16) gives
 * each a slot 0..V-1 (V = counts[VISIBLE]); later steps read per-Gaussian data by slot, so that what
 * neighbouring tiles touch is neighbouring memory (the scene's own order carries no such locality), and the
 * Gaussians that a super-tile owns in the backward pass are one run of slots.
 *   rect   [n,4] int32 out: inclusive pixel range x0,y0,x1,y1 of pixel centres inside the
 *                bound, clipped to the image; (0,0,-1,-1) if empty.
 *   cls    [n]   uint8 out: 0 culled (sigma <= alpha_min, or support entirely at depth <= near_z),
 *                1 in front of the near plane, 2 straddling it (rectangle = whole image unless
 *                the bounding sphere is outside a side plane of the frustum).
 *   pre    [n * gart_pre_words(sh_degree)] fp32 out: per slot, the 80-byte evaluation record, and behind all
 *                records quaternion, scale, opacity and the rectangle in slot order; contents are private to the
 *                library.  (The SH coefficients are not copied: gart_forward and gart_backward_hybrid read them
 *                from g->sh by Gaussian id, so g->sh must stay valid, unchanged and 16-byte aligned for the view.)
 *   slot_of_gid [n] uint32 out: slot of every Gaussian, 0xffffffff if it has none.
 *   gid_of_slot [n] uint32 out: the inverse (first V entries; 0xffffffff beyond).
 *   counts [GART_COUNTS_WORDS] uint32 out: zeroed, then VISIBLE and STRADDLE are set.
 * Errors: INVALID_ARG for null pointers, n < 0, sh_degree outside 0..3, tile size not 8/16,
 * non-positive image size, unaligned workspace; WORKSPACE_TOO_SMALL.
 */
int32_t gart_pre_words(int32_t sh_degree);
size_t gart_bounds_workspace_bytes(int64_t n);
gart_status gart_bounds(const gart_config *cfg, const gart_gaussians *g, const gart_camera *cam,
                        int32_t *rect, uint8_t *cls, float *pre, uint32_t *slot_of_gid, uint32_t *gid_of_slot,
                        uint32_t *counts, void *workspace, size_t workspace_bytes, void *stream);

/*
 * Step 2 -- reverse tile mapping (Sec. 4.3): every Gaussian emits one (tile, id) pair per tile
 * its rectangle overlaps; the pairs are radix-sorted by tile (stable, so ids ascend inside a
 * tile) and the tile offset table is the prefix sum of pairs per tile.  Also sums the
 * rectangle areas (the footprint prefix sum of "Primitive offset", kept as the total S).
 *   tile_off [T+1] uint32 out, T = tiles_x * tiles_y; tile t owns pair_gid[tile_off[t] .. tile_off[t+1]).
 *   pair_gid [cap_pairs] uint32 out.
 *   counts: PAIRS, SLOTS set.  If P > cap_pairs the error bit GART_ERRBIT_PAIRS is set,
 *   tile_off is all zero and later calls do nothing.
 */
size_t gart_tile_map_workspace_bytes(int64_t n, int32_t width, int32_t height, int32_t tile_size, int64_t cap_pairs);
gart_status gart_tile_map(const gart_config *cfg, const int32_t *rect, int64_t n, int32_t width, int32_t height,
                          uint32_t *tile_off, uint32_t *pair_gid, int64_t cap_pairs, uint32_t *counts,
                          void *workspace, size_t workspace_bytes, void *stream);

/*
 * The same tile map for callers that cannot hand over scratch memory (the paper has no counterpart:
 * this entry point exists for hosts in which device allocations are not possible at call time -- an
 * engine that gave its whole device budget to its own arena, a plug-in under a memory quota, a loop
 * that must not touch the allocator).  Arguments, results and errors are those of gart_tile_map; the
 * scratch is a fixed array of GART_TILE_MAP_STATIC_BYTES inside the library, which every GPU that
 * loads the library keeps allocated until the process exits.  The call allocates nothing.
 *   - Limit: gart_tile_map_workspace_bytes(n, width, height, tile_size, cap_pairs) must not exceed
 *     GART_TILE_MAP_STATIC_BYTES (about n + 3 cap_pairs words: e.g. n = 200k with cap_pairs = 500k);
 *     larger problems are refused with GART_ERR_WORKSPACE_TOO_SMALL before any work is queued.
 *   - The first call on a device looks up the array's device address (a host-side query, done with
 *     that device current) and keeps it for the life of the process; make that first call before any
 *     stream capture begins.  Host threads may make it together.  `stream` must belong to the device
 *     that is current in the calling thread (the array used is the current device's).  cudaDeviceReset
 *     invalidates the kept address: do not call this entry point after a reset of its device.
 *   - All calls on a device share the array: calls that may overlap on the GPU (different streams
 *     without ordering) race on it.  The array keeps the previous call's contents; the tile map
 *     writes every scratch word before reading it, so nothing has to be cleared.
 */
#define GART_TILE_MAP_STATIC_BYTES (8u << 20)
gart_status gart_tile_map_static(const gart_config *cfg, const int32_t *rect, int64_t n, int32_t width, int32_t height,
                                 uint32_t *tile_off, uint32_t *pair_gid, int64_t cap_pairs, uint32_t *counts,
                                 void *stream);

/*
 * The view block: private arrays that gart_forward builds and the backward passes read (per pair the hit mask and
 * its rank in the tile; per Gaussian the work items of the primitive-major order; the LT layout of both orders).
 * Opaque to the caller, who owns the memory: `view` is a device buffer of at least gart_view_bytes bytes, 256-byte
 * aligned.  n, image size, tile size and cap_pairs must be the same in the query, in gart_forward and in the backward
 * pass.  gart_view_array returns offset and size of one named array inside the block (for tests and diagnostics;
 * the names are not a stable interface).
 */
size_t gart_view_bytes(int64_t n, int32_t width, int32_t height, int32_t tile_size, int64_t cap_pairs);
enum {
    GART_VIEW_PAIR_MASK = 0,    /* [cap_pairs, gart_mask_words] bit p of pair j: pixel p = ly * tile_size + lx of its tile is hit */
    GART_VIEW_PAIR_ORDER = 1,   /* [cap_pairs] per tile, the pairs by descending hit count (stable) */
    GART_VIEW_RANK_SID = 2,     /* [cap_pairs] slot of the Gaussian, in rank order */
    GART_VIEW_RANK_MASK = 3,    /* [cap_pairs, gart_mask_words] hit mask, in rank order */
    GART_VIEW_RANK_GSTART = 4,  /* [cap_pairs] tile-major LT layout: start of the pair's 32-rank group inside its tile */
    GART_VIEW_TILE_LT_BASE = 5, /* [T+1] tile-major LT layout: first entry of every tile */
    GART_VIEW_PAIR_GPOS = 6,    /* [cap_pairs] position of the pair in the primitive-major order */
    GART_VIEW_GPAIR_OFF = 7,    /* [n+1] first primitive-major position of every slot (the slot's tiles follow row by row) */
    GART_VIEW_GM_MASK = 8,      /* [cap_pairs, gart_mask_words] hit masks in primitive-major order */
    GART_VIEW_GM_LTB = 9,       /* [cap_pairs] primitive-major LT layout: entry of the first hit of every pair, by primitive-major position */
    GART_VIEW_ITEM_DESC = 10,   /* [cap_pairs, 4] work items per super-tile in rank order: slot, first pair, dimensions, hits | whole-flag << 16 */
    GART_VIEW_ITEM_GSTART = 11, /* [cap_pairs] LT entry where the item's 32-rank group starts */
    GART_VIEW_ST_OFF = 12,      /* [NS+1] first item of every super-tile, NS = ceil(width / 16) * ceil(height / 16) */
    GART_VIEW_ST_LT_BASE = 13,  /* [NS+1] first LT entry of every super-tile */
    GART_VIEW_INFO = 14         /* [64] word 0: items, word 1: blocks of the backward pass */
};
gart_status gart_view_array(int64_t n, int32_t width, int32_t height, int32_t tile_size, int64_t cap_pairs, int32_t which,
                            size_t *offset, size_t *bytes);

/*
 * Step 3 -- forward ray evaluation (Sec. 3.2-3.3, Eq. 3-8; intermediate buffer of Sec. 4.2-4.3).
 * For every pixel ray and every Gaussian of its tile list: t* = -(o_g.d_g)/(d_g.d_g),
 * alpha = sigma exp(-|o_g + t* d_g|^2 / 2); a hit iff alpha >= alpha_min and t* > 0.  Hits of a
 * ray are ordered by (t*, id) and composited front to back, C = sum T_i alpha_i c_i + T_final bg,
 * c_i = max(0, 0.5 + sum_k Y_k(d) sh_ik).  The coefficients sh_ik are read from g->sh (device memory, by Gaussian id,
 * 16-byte aligned: INVALID_ARG otherwise); everything else of a Gaussian comes from `pre`.
 *   color      [H,W,3] out;  t_final [H,W] out;  hit_count [H,W] uint32 out.
 *   lt         [cap_hits,4] out: per hit, with w = T alpha its blending weight (T the transmittance
 *              in front of it), c its clamped colour and B the colour composited BEHIND it
 *              (background term included): words 0..2 = w c - alpha / (1 - alpha) B, which is
 *              alpha dC/dalpha by Eq. 6-8; word 3 = w, whose three low mantissa bits are replaced by
 *              flags "channel r, g, b of c is not clamped".  This is all the backward pass needs of
 *              the ray's state, and nothing in it is a difference of nearly equal sums.
 *              With cfg->lt_format = 2 the entry of slot i is the 8 bytes at lt + 8 i: four IEEE halves
 *              h0..h3, h_ch = 4096 x word ch (clamped to +-60000) rounded to nine mantissa bits (nearest,
 *              ties to even) with the half's lowest bit replaced by the flag of channel ch, h3 = the half
 *              nearest to 4096 w.  A decoded colour word is within 2^-10 (relative) of the fp32 value, the
 *              weight within 2^-11; magnitudes below 2^-26 lose relative precision, below 2^-37 vanish.
 *              Where a hit's entry lives: every hit owns one slot (forward writes never collide).  Both layouts
 *              rank work units by descending hit count and interleave the entries of 32 consecutive ranks, so that a
 *              warp of the backward reads its lanes' entries as contiguous rows and a group's block is one contiguous
 *              range; a group occupies 32 x (its largest hit count) entries, L >= H counts that padding.
 *              GART_LT_TILE_MAJOR: the unit is a (tile, Gaussian) pair, groups are formed inside each tile; entry e
 *              of rank r sits at group start + 32 e + r mod 32.
 *              GART_LT_PRIMITIVE_MAJOR: the unit is a work item -- a Gaussian whose rectangle spans at most two
 *              16 x 16-pixel super-tiles per axis, else the part of a Gaussian inside one super-tile; its entries are
 *              those of its (tile, Gaussian) pairs in turn (tiles row by row, pixels in mask order); groups are
 *              formed among the items owned by one super-tile.  Entries go two by two: entry e of rank r sits at
 *              group start + 64 (e / 2) + 2 (r mod 32) + e mod 2 (the group's largest count is rounded up to even), so
 *              that a 32-byte sector holds two neighbouring hits of one Gaussian, which the forward writes close in time.
 *              In this layout the entry also names its pixel: the 10-bit index y * 32 + x of the hit's pixel inside
 *              the 32 x 32-pixel window whose corner is the owner super-tile's replaces the three low mantissa bits of
 *              each of the words 0..2 (index bits 0..2, 3..5, 6..8) and bit 3 of word 3 (index bit 9) -- a relative
 *              change below 2^-20 of numbers that are needed to 1e-3 -- so that the backward pass walks no hit mask.
 *   ray_off    [H*W+1] uint32 out; ray_gid, ray_slot [cap_hits] uint32 out: per ray, in
 *              compositing order, the Gaussian id and LT slot of each hit.  Only the pixel-centric
 *              baseline and parity checks read the two lists: pass NULL for both to skip them.
 *   view       the view block (above), out.
 *   counts: HITS, LT_SLOTS, MAX_RAY_HITS.  If L > cap_hits, GART_ERRBIT_HITS is set and color,
 *   t_final, lt, ray_gid, ray_slot are not written.  Because ranks descend in hit count, a tile (super-tile) pads
 *   by less than 32 x its largest count, and H <= S (the slot bound of gart_tile_map), so
 *   cap_hits = S + 32 tile_size^2 T (tile-major) or S + 32 * 1024 * NS (primitive-major) always suffices; the
 *   exact need is L.
 * Errors: INVALID_ARG also for an image wider or higher than 524280 pixels, and for lt_format 1 or 2 with the
 * primitive-major layout (the 4- and 8-byte formats serve the tile-major passes).
 */
size_t gart_forward_workspace_bytes(int32_t width, int32_t height, int32_t tile_size, int64_t cap_pairs, int64_t cap_hits);
gart_status gart_forward(const gart_config *cfg, const gart_gaussians *g, const gart_camera *cam, const float *pre,
                         const uint32_t *slot_of_gid, const uint32_t *gid_of_slot, const uint32_t *tile_off, const uint32_t *pair_gid, int64_t cap_pairs,
                         float *color, float *t_final, uint32_t *hit_count,
                         float *lt, int64_t cap_hits,
                         uint32_t *ray_off, uint32_t *ray_gid, uint32_t *ray_slot,
                         void *view, size_t view_bytes, uint32_t *counts,
                         void *workspace, size_t workspace_bytes, void *stream);

/*
 * Step 4 -- primitive-centric backward (Sec. 4.4).  With cfg->lt_layout = GART_LT_TILE_MAJOR this call IS
 * gart_backward_tile (below).  With GART_LT_PRIMITIVE_MAJOR a thread gathers the gradient sums of ONE work item of the
 * primitive-major order: it walks the item's (tile, Gaussian) pairs one after the other and, per pair, the pair's hit
 * pixels, reads their LT entries (coalesced across the warp thanks to the interleaved layout) and accumulates in
 * registers.  No per-pixel atomics.  An item that is a whole Gaussian (its rectangle fits a 32 x 32-pixel window: nearly
 * all of them) ends with the conversion of the moments and ONE write of the 256-byte gradient record -- no atomic, no
 * accumulation record; the pieces of larger Gaussians add to an accumulation record with one vector atomic per 16 bytes
 * and piece, converted by a small per-slot pass.  gart_bounds and gart_forward must have run with the same lt_layout.
 *   dL_dcolor [H,W,3] in.
 *   grad [n,GART_GRAD_WORDS] out, fully overwritten: d mean, d scale, d quat, d opacity, d sh
 *        of L = sum <dL_dcolor, color>; zero for Gaussians without hits.
 *   view, cap_pairs: the view block that gart_forward filled and the capacity it was laid out for.
 *   counts: read (a set error bit skips the work); GART_ERRBIT_TIMEOUT is set if a wait on an
 *        asynchronous copy ran out, in which case grad is incomplete.
 * In the primitive-major layout cfg->lt_format must be 0 (INVALID_ARG otherwise): the pass finds a hit's pixel in its
 * 16-byte entry.
 * The main kernel uses 54 KB of dynamic shared memory per block: LT blocks are streamed in with bulk
 * asynchronous copies, one rank group ahead, beside dL/dC of the block's 32 x 32-pixel window and the
 * Gaussians' records.
 */
size_t gart_backward_workspace_bytes(int64_t n);
gart_status gart_backward(const gart_config *cfg, const gart_gaussians *g, const gart_camera *cam, const float *pre,
                          const uint32_t *slot_of_gid, const uint32_t *gid_of_slot, const uint32_t *tile_off,
                          const void *view, size_t view_bytes, int64_t cap_pairs,
                          const float *lt, const float *dL_dcolor,
                          float *grad, uint32_t *counts, void *workspace, size_t workspace_bytes, void *stream);

/*
 * The same pass in the decomposition that Sec. 4.4 describes: one thread block per tile, one thread per
 * (tile, Gaussian) pair; the thread walks the pair's hit pixels, accumulates in registers and performs one vector
 * atomic update per pair of the accumulation record of the Gaussian's slot; a per-Gaussian pass then converts the
 * accumulated moments and writes the gradient records.  Needs lt_layout = GART_LT_TILE_MAJOR.  Arguments, result
 * (up to summation order) and errors as gart_backward, but cfg->lt_format may be 0 or 2: with 8-byte
 * entries every gradient word, being linear in the four words of its hits' entries, moves by at most 2^-10
 * of the sum of the absolute per-hit, per-channel terms of that word.  38 KB of dynamic shared memory per block.
 */
gart_status gart_backward_tile(const gart_config *cfg, const gart_gaussians *g, const gart_camera *cam, const float *pre,
                               const uint32_t *slot_of_gid, const uint32_t *gid_of_slot, const uint32_t *tile_off,
                               const void *view, size_t view_bytes, int64_t cap_pairs,
                               const float *lt, const float *dL_dcolor,
                               float *grad, uint32_t *counts, void *workspace, size_t workspace_bytes, void *stream);

/*
 * Pixel-centric baseline (Sec. 3.5): one thread per ray walks the ray's hits and issues one
 * atomicAdd per gradient word per hit (11 + 3K; 59 at degree 3), or, with cfg->atomic_mode = GART_ATOMIC_VECTOR,
 * one 16-byte vector reduction per four words.  Same result as gart_backward up to summation order.  Reads 16-byte LT entries through ray_slot, so either layout serves; needs the
 * per-ray lists of gart_forward (INVALID_ARG if they are NULL).
 */
gart_status gart_backward_atomic(const gart_config *cfg, const gart_gaussians *g, const gart_camera *cam,
                                 const float *pre, const uint32_t *slot_of_gid, const uint32_t *ray_off, const uint32_t *ray_gid,
                                 const uint32_t *ray_slot, const float *lt, const float *dL_dcolor,
                                 float *grad, const uint32_t *counts, void *stream);

/*
 * Ownership ablation (Sec. 4.4): gart_backward_tile with one warp, not one thread, per (tile, Gaussian) pair.  Same
 * arguments, same result up to summation order; Sec. 4.4 reports it as slower, and so it is here.  16-byte entries only.
 */
gart_status gart_backward_warp(const gart_config *cfg, const gart_gaussians *g, const gart_camera *cam, const float *pre,
                               const uint32_t *slot_of_gid, const uint32_t *gid_of_slot, const uint32_t *tile_off,
                               const void *view, size_t view_bytes, int64_t cap_pairs,
                               const float *lt, const float *dL_dcolor,
                               float *grad, uint32_t *counts, void *workspace, size_t workspace_bytes, void *stream);

/*
 * Hybrid backward (Sec. 4.4 "Hybrid approach"; "Hybrid" of Sec. 5.1): the colour gradients dL/dsh are accumulated
 * primitive-centric (block per tile) from an intermediate buffer of ONE word per hit, the remaining terms (mean, scale,
 * quaternion, opacity) pixel-centric with three vector atomics per hit.  Needs gart_forward run with
 * cfg->lt_format = 1, lt_layout = GART_LT_TILE_MAJOR (lt_w [cap_hits] fp32: word 3 of the full entry) and with the per-ray id
 * list (ray_off, ray_gid); the 4 + 4 bytes per hit replace the 16 of the full entry (the paper, which re-traces
 * the ray in its pixel-centric part, keeps 4).  Same result as gart_backward up to rounding and summation order;
 * same workspace as gart_backward.  Errors as gart_backward; INVALID_ARG if cfg->lt_format != 1.
 */
size_t gart_backward_hybrid_workspace_bytes(int64_t n, int32_t sh_degree);   /* gart_backward_workspace_bytes(n) + a copy of the coefficient rows in slot order */
gart_status gart_backward_hybrid(const gart_config *cfg, const gart_gaussians *g, const gart_camera *cam, const float *pre,
                                 const uint32_t *slot_of_gid, const uint32_t *gid_of_slot, const uint32_t *tile_off,
                                 const void *view, size_t view_bytes, int64_t cap_pairs,
                                 const float *lt_w, const uint32_t *ray_off, const uint32_t *ray_gid,
                                 const float *dL_dcolor, float *grad, uint32_t *counts, void *workspace, size_t workspace_bytes,
                                 void *stream);

/* The largest of the four per-step workspace needs (bounds, tile map, forward, backward): one buffer serves a whole view. */
size_t gart_workspace_bytes(int64_t n, int32_t width, int32_t height, int32_t tile_size, int64_t cap_pairs, int64_t cap_hits);

/* Copy the counts block to host memory (synchronises the stream). counts_host: host, GART_COUNTS_WORDS words. */
gart_status gart_read_counts(const uint32_t *counts, uint32_t *counts_host, void *stream);

/* gart_read_counts, then the block's error word as a status: GART_ERR_CAPACITY_EXCEEDED (pair or hit capacity),
 * GART_ERR_TIMEOUT (a bounded wait inside a kernel ran out), else GART_OK.  counts_host may be NULL. */
gart_status gart_sync_status(const uint32_t *counts, uint32_t *counts_host, void *stream);

/*
 * End-to-end convenience for callers holding HOST arrays: uploads the scene and dL_dcolor,
 * runs the four steps for one view, downloads color [H,W,3] and grad [n,GART_GRAD_WORDS].
 * All five array arguments and the members of `g_host` are HOST pointers.  `arena` is a device
 * buffer of `arena_bytes` bytes from which every device array is carved; query the size with
 * gart_view_host_arena_bytes (cap_pairs / cap_hits are capacities chosen by the caller).
 * counts_host (host, GART_COUNTS_WORDS words) receives the counts block.  Synchronous.
 * Returns GART_ERR_CAPACITY_EXCEEDED if a capacity was too small.
 */
size_t gart_view_host_arena_bytes(int64_t n, int32_t sh_degree, int32_t width, int32_t height, int32_t tile_size,
                                  int64_t cap_pairs, int64_t cap_hits);
gart_status gart_view_host(const gart_config *cfg, const gart_gaussians *g_host, const gart_camera *cam,
                           const float *dL_dcolor_host, float *color_host, float *grad_host,
                           int64_t cap_pairs, int64_t cap_hits, uint32_t *counts_host,
                           void *arena, size_t arena_bytes, void *stream);

/*
 * The same, without waiting: every copy and kernel of the view is queued on `stream` and the call returns.  The host
 * arrays (pinned, for the copies to be asynchronous) and counts_host are valid once the stream has been synchronised;
 * gart_counts_status(counts_host) then gives the status gart_view_host would have returned.  Two views in flight on two
 * streams, each with an arena and output arrays of its own, overlap one view's uploads with the other's downloads
 * (the two directions of the host link) and with its kernels.
 */
gart_status gart_view_host_async(const gart_config *cfg, const gart_gaussians *g_host, const gart_camera *cam,
                           const float *dL_dcolor_host, float *color_host, float *grad_host,
                           int64_t cap_pairs, int64_t cap_hits, uint32_t *counts_host,
                           void *arena, size_t arena_bytes, void *stream);

/* The status that a counts block copied to the host encodes: GART_ERR_TIMEOUT, GART_ERR_CAPACITY_EXCEEDED or GART_OK. */
gart_status gart_counts_status(const uint32_t *counts_host);

#ifdef __cplusplus
}
#endif
#endif /* GART_H */
