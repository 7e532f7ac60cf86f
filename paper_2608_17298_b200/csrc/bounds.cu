// gart_bounds: conservative perspective-correct screen rectangles (Sec. 4.2, Eq. 11-14), the
// opacity-dependent clamping radius (Eq. 10) and the ray-evaluation record (Eq. 5), one thread
// per Gaussian, in double precision: the rectangle edges are integer decisions (ceil / floor of
// p -/+ h) and the pass is O(n), so fp64 costs nothing that matters and keeps the edges exact.
//
// The Gaussians that reach the image are then renumbered for this view: a stable radix sort on the
// 16 x 16-pixel super-tile of the rectangle's first corner gives every visible Gaussian a "slot", and its
// evaluation record and SH coefficients are gathered into one contiguous record per slot.  Tiles are
// processed in tile order and the backward walks the slots in order, so per-pair reads of these records
// touch memory that neighbouring work also touches, instead of random 200-byte pieces of gigabyte-sized
// arrays; the Gaussians that one super-tile owns are one contiguous run of slots.
#include "radix.cuh"
#include "view_layout.cuh"

namespace gart {

constexpr int PRE_TMP_F4 = 8;   // float4 per Gaussian in the id-ordered temporary: 5 of the record, quaternion, scale + opacity, rectangle
                                // (128 bytes: the gather reads one whole line per Gaussian and nothing else)
constexpr int PRE_TMP_PAD = PRE_TMP_F4 + 1;   // lane stride of the staging rows in shared memory (odd: no bank conflicts)

struct CamD {
    int width, height;
    double fx, fy, cx, cy;
    double ifx, ify;   // 1 / fx, 1 / fy: the record's quotients are products (fp64 divisions are what this kernel's time goes to)
    double w2c[12];
};

__device__ __forceinline__ void quat_to_rot(const double w, const double x, const double y, const double z, double* R) {
    R[0] = 1.0 - 2.0 * (y * y + z * z); R[1] = 2.0 * (x * y - w * z); R[2] = 2.0 * (x * z + w * y);
    R[3] = 2.0 * (x * y + w * z); R[4] = 1.0 - 2.0 * (x * x + z * z); R[5] = 2.0 * (y * z - w * x);
    R[6] = 2.0 * (x * z - w * y); R[7] = 2.0 * (y * z + w * x); R[8] = 1.0 - 2.0 * (x * x + y * y);
}

__global__ void __launch_bounds__(128, 6) bounds_kernel(int64_t n, const float* __restrict__ mean, const float* __restrict__ scale,
                                                     const float* __restrict__ quat, const float* __restrict__ opacity,
                                                     CamD cam, double alpha_min, int narrow, double near_z,
                                                     int sup_x, uint32_t key_none,
                                                     int32_t* __restrict__ rect, uint8_t* __restrict__ cls,
                                                     float4* __restrict__ pre4, uint32_t* __restrict__ keys,
                                                     uint32_t* __restrict__ vals, uint32_t* __restrict__ counts) {
    __shared__ float4 s_out[128 * PRE_TMP_PAD];   // the block's 128 temporaries, staged so that the stores are whole rows
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    int vis = 0, straddle = 0;
    float4 q0 = make_float4(0, 0, 0, 0), q1 = q0, q2 = q0, q3 = q0, q4 = q0, q5 = q0, q6 = q0, q7 = q0;
    if (i < n) {
        int x0 = 0, y0 = 0, x1 = -1, y1 = -1, c = 0;
        const double sigma = (double)opacity[i];
        if (sigma > alpha_min) {
            const double tau_c = 2.0 * log(sigma / alpha_min);
            const double alpha_c = narrow ? sqrt(sqrt(tau_c)) : sqrt(tau_c);  // Eq. 10 (fourth root for the degree-4 kernel)
            double R[9];
            quat_to_rot((double)quat[4 * i], (double)quat[4 * i + 1], (double)quat[4 * i + 2], (double)quat[4 * i + 3], R);
            const double s[3] = {(double)scale[3 * i], (double)scale[3 * i + 1], (double)scale[3 * i + 2]};
            const double mu[3] = {(double)mean[3 * i], (double)mean[3 * i + 1], (double)mean[3 * i + 2]};
            const double* M = cam.w2c;
            // camera-space support axes  Ac = Rc * (R S alpha_c)  and centre
            double Ac[9], muc[3];
#pragma unroll
            for (int r = 0; r < 3; ++r) {
#pragma unroll
                for (int k = 0; k < 3; ++k)
                    Ac[3 * r + k] = (M[4 * r] * R[k] + M[4 * r + 1] * R[3 + k] + M[4 * r + 2] * R[6 + k]) * s[k] * alpha_c;
                muc[r] = M[4 * r] * mu[0] + M[4 * r + 1] * mu[1] + M[4 * r + 2] * mu[2] + M[4 * r + 3];
            }
            const double ez = sqrt(Ac[6] * Ac[6] + Ac[7] * Ac[7] + Ac[8] * Ac[8]);
            if (muc[2] + ez > near_z) {
                c = (muc[2] - ez >= near_z) ? 1 : 2;
                if (c == 1) {
                    // rows x, y, w of T' in pixel units; v = (1,1,1,-1)
                    double sden = -muc[2] * muc[2], pxn = 0.0, pyn = 0.0, qxn = 0.0, qyn = 0.0;
                    const double tx3 = cam.fx * muc[0] + cam.cx * muc[2], ty3 = cam.fy * muc[1] + cam.cy * muc[2];
#pragma unroll
                    for (int k = 0; k < 3; ++k) {
                        const double tw = Ac[6 + k];
                        const double tx = cam.fx * Ac[k] + cam.cx * tw, ty = cam.fy * Ac[3 + k] + cam.cy * tw;
                        sden += tw * tw;
                        pxn += tx * tw; pyn += ty * tw;
                        qxn += tx * tx; qyn += ty * ty;
                    }
                    pxn -= tx3 * muc[2]; pyn -= ty3 * muc[2];
                    qxn -= tx3 * tx3;   qyn -= ty3 * ty3;
                    const double px = pxn / sden, py = pyn / sden;
                    const double hx = sqrt(fmax(0.0, px * px - qxn / sden)), hy = sqrt(fmax(0.0, py * py - qyn / sden));
                    const double fx0 = fmax(0.0, ceil(px - hx - 0.5)), fx1 = fmin((double)(cam.width - 1), floor(px + hx - 0.5));
                    const double fy0 = fmax(0.0, ceil(py - hy - 0.5)), fy1 = fmin((double)(cam.height - 1), floor(py + hy - 0.5));
                    if (fx1 >= fx0 && fy1 >= fy0) { x0 = (int)fx0; y0 = (int)fy0; x1 = (int)fx1; y1 = (int)fy1; }
                } else {
                    const double rad = alpha_c * fmax(s[0], fmax(s[1], s[2]));
                    const double pl[4][3] = {{cam.fx, 0.0, cam.cx}, {-cam.fx, 0.0, cam.width - cam.cx},
                                             {0.0, cam.fy, cam.cy}, {0.0, -cam.fy, cam.height - cam.cy}};
                    bool outside = false;
#pragma unroll
                    for (int p = 0; p < 4; ++p) {
                        const double len = sqrt(pl[p][0] * pl[p][0] + pl[p][1] * pl[p][1] + pl[p][2] * pl[p][2]);
                        const double dist = (pl[p][0] * muc[0] + pl[p][1] * muc[1] + pl[p][2] * muc[2]) / len;
                        outside = outside || (dist < -rad);
                    }
                    if (!outside) { x0 = 0; y0 = 0; x1 = cam.width - 1; y1 = cam.height - 1; }
                    straddle = 1;
                }
                if (x1 >= x0) {
                    vis = 1;
                    // ---- ray-evaluation record
                    // W = S^-1 R^T ; Wc = W Rc^T ; m = W (mu - o), o = -Rc^T t
                    double Wc[9], m[3];
                    const double o[3] = {-(M[0] * M[3] + M[4] * M[7] + M[8] * M[11]),
                                         -(M[1] * M[3] + M[5] * M[7] + M[9] * M[11]),
                                         -(M[2] * M[3] + M[6] * M[7] + M[10] * M[11])};
#pragma unroll
                    for (int k = 0; k < 3; ++k) {
                        const double is = 1.0 / s[k];
                        const double w0 = R[k] * is, w1 = R[3 + k] * is, w2 = R[6 + k] * is;  // row k of W
#pragma unroll
                        for (int j = 0; j < 3; ++j) Wc[3 * k + j] = w0 * M[4 * j] + w1 * M[4 * j + 1] + w2 * M[4 * j + 2];
                        m[k] = w0 * (mu[0] - o[0]) + w1 * (mu[1] - o[1]) + w2 * (mu[2] - o[2]);
                    }
                    // reference position: projected centre when that is a sane pixel coordinate
                    double rpx = cam.cx, rpy = cam.cy;
                    if (c == 1) {
                        const double iz = 1.0 / muc[2];
                        const double ppx = cam.fx * muc[0] * iz + cam.cx, ppy = cam.fy * muc[1] * iz + cam.cy;
                        if (fabs(ppx) < 1.0e6 && fabs(ppy) < 1.0e6) { rpx = ppx; rpy = ppy; }
                    }
                    const double fix = floor(rpx), fiy = floor(rpy);
                    const float rx = (float)(rpx - 0.5 - fix), ry = (float)(rpy - 0.5 - fiy);
                    const double ex_px = fix + 0.5 + (double)rx, ex_py = fiy + 0.5 + (double)ry;  // exactly what the kernels use
                    const double du = (ex_px - cam.cx) * cam.ifx, dv = (ex_py - cam.cy) * cam.ify;
                    double dgr[3], kk[3];
#pragma unroll
                    for (int k = 0; k < 3; ++k) dgr[k] = Wc[3 * k] * du + Wc[3 * k + 1] * dv + Wc[3 * k + 2];
                    // k = o_g x dgr = dgr x m
                    kk[0] = dgr[1] * m[2] - dgr[2] * m[1];
                    kk[1] = dgr[2] * m[0] - dgr[0] * m[2];
                    kk[2] = dgr[0] * m[1] - dgr[1] * m[0];
                    q0 = make_float4((float)(Wc[0] * cam.ifx), (float)(Wc[3] * cam.ifx), (float)(Wc[6] * cam.ifx), (float)(Wc[1] * cam.ify));
                    q1 = make_float4((float)(Wc[4] * cam.ify), (float)(Wc[7] * cam.ify), (float)dgr[0], (float)dgr[1]);
                    q2 = make_float4((float)dgr[2], (float)m[0], (float)m[1], (float)m[2]);
                    q3 = make_float4((float)kk[0], (float)kk[1], (float)kk[2], (float)sigma);
                    q4 = make_float4(rx, ry, __int_as_float((int)fix), __int_as_float((int)fiy));
                }
            }
        }
        reinterpret_cast<int4*>(rect)[i] = make_int4(x0, y0, x1, y1);
        cls[i] = (uint8_t)c;
        if (vis) {   // quaternion, scale, opacity ride along so that the gather reads one contiguous piece
            q5 = make_float4(quat[4 * i], quat[4 * i + 1], quat[4 * i + 2], quat[4 * i + 3]);
            q6 = make_float4(scale[3 * i], scale[3 * i + 1], scale[3 * i + 2], opacity[i]);
            q7 = make_float4(__int_as_float(x0), __int_as_float(y0), __int_as_float(x1), __int_as_float(y1));
        }
        // super-tile of the rectangle's corner (its row alone where the caller sorts by rows: sup_x = 1)
        keys[i] = vis ? (uint32_t)((y0 / GM_SUP) * sup_x + (sup_x > 1 ? x0 / GM_SUP : 0)) : key_none;
        vals[i] = (uint32_t)i;
    }
    {
        // a warp's 32 temporaries are contiguous in memory: through shared memory (lane stride 9 float4, odd: no bank
        // conflicts) and out as 8 coalesced 512-byte rows
        const int lane = threadIdx.x & 31, wbase = (threadIdx.x & ~31) * PRE_TMP_PAD;
        float4* mine = s_out + wbase + lane * PRE_TMP_PAD;
        mine[0] = q0; mine[1] = q1; mine[2] = q2; mine[3] = q3; mine[4] = q4; mine[5] = q5; mine[6] = q6; mine[7] = q7;
        __syncwarp();
        const int64_t i_w = i - lane;                      // first Gaussian of the warp
        const int64_t left = (n - i_w) * PRE_TMP_F4;       // float4 of this warp that exist
        float4* dst = pre4 + (size_t)i_w * PRE_TMP_F4;
#pragma unroll
        for (int j = 0; j < PRE_TMP_F4; ++j) {
            const int idx = j * 32 + lane;
            if (idx < left) dst[idx] = s_out[wbase + (idx / PRE_TMP_F4) * PRE_TMP_PAD + idx % PRE_TMP_F4];
        }
    }
    const unsigned bv = __ballot_sync(0xffffffffu, vis), bs = __ballot_sync(0xffffffffu, straddle);
    if ((threadIdx.x & 31) == 0) {
        if (bv) atomicAdd(&counts[GART_CNT_VISIBLE], __popc(bv));
        if (bs) atomicAdd(&counts[GART_CNT_STRADDLE], __popc(bs));
    }
}

// One thread per 16 bytes of a slot's 128-byte temporary: eight threads read the whole line of their Gaussian and write
// the evaluation record (5 float4), the quaternion and scale + opacity (2) and the rectangle (1) into their
// slot-ordered arrays.  Also fills the two maps between ids and slots.
constexpr int GATHER_UNROLL = 2;

__global__ void __launch_bounds__(256) gather_records_kernel(uint32_t n, uint32_t key_none,
                                                             const uint32_t* __restrict__ keys_sorted, const uint32_t* __restrict__ vals_sorted,
                                                             const float4* __restrict__ pre_tmp,
                                                             float4* __restrict__ rec, float4* __restrict__ qs, int4* __restrict__ srect,
                                                             uint32_t* __restrict__ slot_of_gid, uint32_t* __restrict__ gid_of_slot) {
    constexpr uint32_t RS4 = REC_F4;
    // GATHER_UNROLL pieces per thread, their loads issued together (the chain id -> record otherwise leaves too few bytes in flight)
    uint32_t slot[GATHER_UNROLL], q[GATHER_UNROLL], gid[GATHER_UNROLL];
    bool vis[GATHER_UNROLL];
#pragma unroll
    for (int u = 0; u < GATHER_UNROLL; ++u) {
        const uint32_t t = (blockIdx.x * GATHER_UNROLL + u) * blockDim.x + threadIdx.x;
        slot[u] = t / PRE_TMP_F4;
        q[u] = t % PRE_TMP_F4;
        const bool in = slot[u] < n;
        gid[u] = in ? vals_sorted[slot[u]] : 0u;
        vis[u] = in && keys_sorted[slot[u]] != key_none;
        if (in && q[u] == 0) {
            slot_of_gid[gid[u]] = vis[u] ? slot[u] : 0xffffffffu;
            gid_of_slot[slot[u]] = vis[u] ? gid[u] : 0xffffffffu;
        }
    }
    float4 v[GATHER_UNROLL];
#pragma unroll
    for (int u = 0; u < GATHER_UNROLL; ++u) {
        v[u] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (vis[u]) v[u] = pre_tmp[(size_t)gid[u] * PRE_TMP_F4 + q[u]];
    }
#pragma unroll
    for (int u = 0; u < GATHER_UNROLL; ++u) {
        if (!vis[u]) continue;
        if (q[u] < RS4) rec[(size_t)slot[u] * RS4 + q[u]] = v[u];
        else if (q[u] < RS4 + 2) qs[2 * (size_t)slot[u] + (q[u] - RS4)] = v[u];   // quaternion; scale and opacity (the backward's per-Gaussian pass)
        else srect[slot[u]] = make_int4(__float_as_int(v[u].x), __float_as_int(v[u].y), __float_as_int(v[u].z), __float_as_int(v[u].w));
    }
}

struct BoundsWs {
    float4* pre_tmp;
    uint32_t *keys0, *keys1, *vals0, *vals1, *table;
    uint64_t* total64;
    void* scan_ws;
    size_t bytes;
};

static BoundsWs bounds_layout(void* base, int64_t n) {
    BoundsWs w;
    char* p = (char*)base;
    size_t off = 0;
    auto take = [&](size_t b) { void* r = p ? (void*)(p + off) : nullptr; off += align256(b); return r; };
    const int64_t nn = n > 0 ? n : 1;
    w.total64 = (uint64_t*)take(256);
    w.pre_tmp = (float4*)take((size_t)nn * PRE_TMP_F4 * 16);
    w.keys0 = (uint32_t*)take((size_t)nn * 4); w.keys1 = (uint32_t*)take((size_t)nn * 4);
    w.vals0 = (uint32_t*)take((size_t)nn * 4); w.vals1 = (uint32_t*)take((size_t)nn * 4);
    w.table = (uint32_t*)take(radix_table_bytes(nn));
    w.scan_ws = take(radix_scan_bytes(nn));
    w.bytes = off;
    return w;
}

}  // namespace gart

extern "C" const char* gart_status_string(gart_status s) {
    switch (s) {
        case GART_OK: return "ok";
        case GART_ERR_INVALID_ARG: return "invalid argument";
        case GART_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case GART_ERR_CAPACITY_EXCEEDED: return "capacity exceeded";
        case GART_ERR_CUDA: return "CUDA error";
        case GART_ERR_TIMEOUT: return "a bounded wait inside a kernel ran out";
    }
    return "unknown status";
}

extern "C" int32_t gart_mask_words(int32_t tile_size) { return tile_size * tile_size / 32; }

// Per Gaussian: the slot's evaluation record (20 words); in a second block behind all records, 8 words (quaternion, scale,
// opacity) in slot order; in a third, the rectangle.  (The same for every SH degree: the coefficients are read in place.)
extern "C" int32_t gart_pre_words(int32_t sh_degree) { (void)sh_degree; return 4 * gart::REC_F4 + 8 + 4; }

extern "C" size_t gart_bounds_workspace_bytes(int64_t n) { return gart::bounds_layout(nullptr, n).bytes; }

extern "C" gart_status gart_bounds(const gart_config* cfg, const gart_gaussians* g, const gart_camera* cam,
                                   int32_t* rect, uint8_t* cls, float* pre, uint32_t* slot_of_gid, uint32_t* gid_of_slot,
                                   uint32_t* counts, void* workspace, size_t workspace_bytes, void* stream) {
    using namespace gart;
    if (!cfg || !g || !cam || !counts) return GART_ERR_INVALID_ARG;
    if (g->n < 0 || g->n > 0xfffffff0ll || g->sh_degree < 0 || g->sh_degree > 3) return GART_ERR_INVALID_ARG;
    if (cfg->tile_size != 8 && cfg->tile_size != 16) return GART_ERR_INVALID_ARG;
    if (!kernel_degree_ok(cfg->kernel_degree)) return GART_ERR_INVALID_ARG;
    if (cam->width <= 0 || cam->height <= 0 || !(cam->fx > 0.0) || !(cam->fy > 0.0)) return GART_ERR_INVALID_ARG;
    if (g->n > 0 && (!g->mean || !g->scale || !g->quat || !g->opacity || !g->sh || !rect || !cls || !pre || !slot_of_gid || !gid_of_slot))
        return GART_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemsetAsync(counts, 0, GART_COUNTS_WORDS * sizeof(uint32_t), st) != cudaSuccess) return GART_ERR_CUDA;
    if (g->n == 0) return GART_OK;
    if (!workspace || ((uintptr_t)workspace & 255)) return GART_ERR_INVALID_ARG;
    BoundsWs w = bounds_layout(workspace, g->n);
    if (w.bytes > workspace_bytes) return GART_ERR_WORKSPACE_TOO_SMALL;
    gart::CamD c;
    c.width = cam->width; c.height = cam->height;
    c.fx = cam->fx; c.fy = cam->fy; c.cx = cam->cx; c.cy = cam->cy;
    c.ifx = 1.0 / c.fx; c.ify = 1.0 / c.fy;
    for (int i = 0; i < 12; ++i) c.w2c[i] = cam->w2c[i];
    // Slots are numbered in the order of the super-tile (16 x 16 pixels) of the rectangle's corner: neighbours in the image
    // are neighbours in every per-slot array.  The primitive-major layout wants the full order (its work items of a
    // super-tile are then consecutive slots); for the tile-major layout the row alone gives the locality and needs one
    // radix pass less.
    const int sup_x = cfg->lt_layout == GART_LT_PRIMITIVE_MAJOR ? (cam->width + GM_SUP - 1) / GM_SUP : 1;
    const uint32_t key_none = (uint32_t)(sup_x * ((cam->height + GM_SUP - 1) / GM_SUP));   // sorts after every visible Gaussian
    int bits = 1;
    while ((1u << bits) <= key_none) ++bits;
    uint32_t* const kbuf[2] = {w.keys0, w.keys1};
    uint32_t* const vbuf[2] = {w.vals0, w.vals1};
    const int cur = radix_passes(bits) & 1;   // after the passes the sorted arrays are at index 0
    const int threads = 128;
    const int64_t blocks = ceil_div(g->n, threads);
    bounds_kernel<<<(unsigned)blocks, threads, 0, st>>>(g->n, g->mean, g->scale, g->quat, g->opacity, c,
                                                       (double)cfg->alpha_min, kernel_degree_is4(cfg->kernel_degree) ? 1 : 0, (double)cfg->near_z, sup_x, key_none, rect, cls,
                                                       w.pre_tmp, kbuf[cur], vbuf[cur], counts);
    GART_LAUNCH_CHECK();
    gart_status s = radix_sort_pairs(kbuf, vbuf, cur, bits, g->n, nullptr, (uint32_t)g->n, nullptr, w.table, w.scan_ws, w.total64, st);
    if (s != GART_OK) return s;
    const int rs4 = REC_F4;
    const int64_t gthreads = g->n * PRE_TMP_F4;
    if (gthreads >= (int64_t)1 << 32) return GART_ERR_INVALID_ARG;   // (32-bit thread indices)
    float4* rec_out = reinterpret_cast<float4*>(pre);
    gather_records_kernel<<<(unsigned)ceil_div(gthreads, 256 * GATHER_UNROLL), 256, 0, st>>>((uint32_t)g->n, key_none, kbuf[0], vbuf[0], w.pre_tmp,
                                                                                rec_out, rec_out + (size_t)g->n * rs4,
                                                                                reinterpret_cast<int4*>(rec_out + (size_t)g->n * (rs4 + 2)), slot_of_gid, gid_of_slot);
    GART_LAUNCH_CHECK();
    return GART_OK;
}
