// Shared device/host helpers of the gart CUDA library (sm_100a).
//
// Contents: launch-error macro, the fp32 camera block passed to kernels by value, the
// per-Gaussian ray-evaluation record and the single ray/Gaussian evaluation routine that
// every kernel uses (Eq. 4, 5, 8 of the 3DGART paper in a cancellation-free form), the real
// spherical-harmonics basis, and a three-kernel exclusive scan without device-side waiting.
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "gart.h"

#define GART_LAUNCH_CHECK()                                   \
    do {                                                      \
        if (cudaGetLastError() != cudaSuccess) return GART_ERR_CUDA; \
    } while (0)

namespace gart {

static inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }
static inline size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

// ---------------------------------------------------------------------------------------------
// Camera, fp32, by value.
struct CamF {
    int width, height;
    int tiles_x, tiles_y;
    float fx, fy, cx, cy;
    float r[9];  // world-to-camera rotation, row-major; world direction of d_c is r^T d_c
};

static inline CamF make_camf(const gart_camera* cam, int ts) {
    CamF c;
    c.width = cam->width;
    c.height = cam->height;
    c.tiles_x = (cam->width + ts - 1) / ts;
    c.tiles_y = (cam->height + ts - 1) / ts;
    c.fx = (float)cam->fx; c.fy = (float)cam->fy; c.cx = (float)cam->cx; c.cy = (float)cam->cy;
    for (int i = 0; i < 3; ++i)
        for (int j = 0; j < 3; ++j) c.r[3 * i + j] = (float)cam->w2c[4 * i + j];
    return c;
}

// Unit world-space direction of the ray through the centre of pixel (x, y).
__device__ __forceinline__ float3 pixel_dir(const CamF& c, int x, int y) {
    const float u = ((float)x + 0.5f - c.cx) / c.fx;
    const float v = ((float)y + 0.5f - c.cy) / c.fy;
    float wx = fmaf(c.r[0], u, fmaf(c.r[3], v, c.r[6]));
    float wy = fmaf(c.r[1], u, fmaf(c.r[4], v, c.r[7]));
    float wz = fmaf(c.r[2], u, fmaf(c.r[5], v, c.r[8]));
    const float inv = rsqrtf(fmaf(wx, wx, fmaf(wy, wy, wz * wz)));
    return make_float3(wx * inv, wy * inv, wz * inv);
}

// ---------------------------------------------------------------------------------------------
// Per-Gaussian ray-evaluation record: 20 floats = 5 float4 (the head of a slot's record).
//
// With W = S^-1 R^T (Eq. 5), the camera rotation Rc and origin o, and the un-normalised ray
// direction d_c = ((x+.5-cx)/fx, (y+.5-cy)/fy, 1) in camera space:
//   c0, c1 : columns 0 and 1 of W Rc^T divided by fx, fy -> d_g changes by c0*dx + c1*dy when
//            the pixel moves by (dx, dy) pixels away from the reference pixel position
//   dgr    : d_g at the reference position (the projected centre for Gaussians in front)
//   m      : -o_g = W (mu - o)
//   k      : o_g x dgr (zero up to rounding when the reference is the projected centre)
//   sigma  : opacity
//   rx, ry : fractional part of the reference position, ix, iy its integer part:
//            dx = float(x - ix) - rx is exact to one rounding however far the pixel is from 0.
// Then o_g x d_g = k + e x m with e = c0*dx + c1*dy, and
//   D^2 = |o_g x d_g|^2 / |d_g|^2,  x_g = d_g x (o_g x d_g) / |d_g|^2,  t* = (m . d_g) / |d_g|^2,
// none of which subtracts large nearly equal numbers (the textbook |o_g|^2 - (o_g.d_g)^2/|d_g|^2
// loses all digits in fp32 when the Gaussian is small and far).
struct PreRec {
    float3 c0, c1, dgr, m, k;
    float sigma, rx, ry;
    int ix, iy;
};

__device__ __forceinline__ PreRec unpack_pre(const float4& a, const float4& b, const float4& c,
                                             const float4& d, const float4& e) {
    PreRec p;
    p.c0 = make_float3(a.x, a.y, a.z);
    p.c1 = make_float3(a.w, b.x, b.y);
    p.dgr = make_float3(b.z, b.w, c.x);
    p.m = make_float3(c.y, c.z, c.w);
    p.k = make_float3(d.x, d.y, d.z);
    p.sigma = d.w;
    p.rx = e.x;
    p.ry = e.y;
    p.ix = __float_as_int(e.z);
    p.iy = __float_as_int(e.w);
    return p;
}

// A slot's record: the 5 float4 of PreRec.  (The SH coefficients are not copied per view: the evaluation reads them from
// the caller's array by Gaussian id.)
constexpr int REC_F4 = 5;

__device__ __forceinline__ PreRec load_pre(const float4* __restrict__ rec) {
    return unpack_pre(__ldg(rec), __ldg(rec + 1), __ldg(rec + 2), __ldg(rec + 3), __ldg(rec + 4));
}

// One-instruction reciprocal and 2^x of the special-function unit (about 1 and 2 ulp).
__device__ __forceinline__ float fast_rcp(float x) {
    float y;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

struct RayEval {
    float alpha;   // sigma * exp(-D^2 / 2)
    float tnum;    // m . d_g : same sign as t*
    float inv_a;   // 1 / |d_g|^2
    float3 dg;     // d_g
    float3 cr;     // o_g x d_g
};

// The configuration's kernel degree: 2 (also for 0) or 4; anything else is refused.
static inline bool kernel_degree_ok(int32_t k) { return k == 0 || k == 2 || k == 4; }
static inline bool kernel_degree_is4(int32_t k) { return k == 4; }

// Response of the Gaussian along the ray through the pixel at offset (dx, dy) pixels from the
// record's reference position.  narrow: the degree-4 kernel exp(-D^4 / 2) instead of exp(-D^2 / 2).
__device__ __forceinline__ RayEval ray_eval(const PreRec& p, float dx, float dy, bool narrow = false) {
    RayEval r;
    const float ex = fmaf(p.c0.x, dx, p.c1.x * dy);
    const float ey = fmaf(p.c0.y, dx, p.c1.y * dy);
    const float ez = fmaf(p.c0.z, dx, p.c1.z * dy);
    r.dg = make_float3(p.dgr.x + ex, p.dgr.y + ey, p.dgr.z + ez);
    r.cr.x = fmaf(ey, p.m.z, fmaf(-ez, p.m.y, p.k.x));
    r.cr.y = fmaf(ez, p.m.x, fmaf(-ex, p.m.z, p.k.y));
    r.cr.z = fmaf(ex, p.m.y, fmaf(-ey, p.m.x, p.k.z));
    const float a = fmaf(r.dg.x, r.dg.x, fmaf(r.dg.y, r.dg.y, r.dg.z * r.dg.z));
    const float cc = fmaf(r.cr.x, r.cr.x, fmaf(r.cr.y, r.cr.y, r.cr.z * r.cr.z));
    r.inv_a = fast_rcp(a);
    const float D2 = cc * r.inv_a;
    r.alpha = p.sigma * fast_exp2(-0.72134752044448170f * (narrow ? D2 * D2 : D2));
    r.tnum = fmaf(p.m.x, r.dg.x, fmaf(p.m.y, r.dg.y, p.m.z * r.dg.z));
    return r;
}

// Maximum-response point in the Gaussian's normalised space.
template <class RayT>
__device__ __forceinline__ float3 ray_xg(const RayT& r) {
    return make_float3((r.dg.y * r.cr.z - r.dg.z * r.cr.y) * r.inv_a,
                       (r.dg.z * r.cr.x - r.dg.x * r.cr.z) * r.inv_a,
                       (r.dg.x * r.cr.y - r.dg.y * r.cr.x) * r.inv_a);
}


// ---------------------------------------------------------------------------------------------
// LT entry of a hit: what the backward pass needs of the ray's compositing state (Sec. 4.2), 16 bytes.
// With w = T alpha the hit's blending weight, c its clamped colour and B the colour composited behind
// it (background included), the pixel colour C satisfies
//     alpha dC/dalpha = w c - alpha / (1 - alpha) B        (from Eq. 6-8)
// so the entry holds that vector and w.  The backward pass then needs neither alpha nor the hit's
// colour again: alpha dL/dalpha = <dL/dC, xyz>, and dL/dc = w dL/dC on the channels that are not
// clamped, flagged in the three low mantissa bits of w (a relative change of w below 2^-20).
__device__ __forceinline__ float4 lt_entry(float w, float alpha, float c0, float c1, float c2, float b0, float b1, float b2) {
    const float r = __fdividef(alpha, 1.0f - alpha);
    const uint32_t flags = (c0 > 0.0f ? 1u : 0u) | (c1 > 0.0f ? 2u : 0u) | (c2 > 0.0f ? 4u : 0u);
    return make_float4(fmaf(w, c0, -r * b0), fmaf(w, c1, -r * b1), fmaf(w, c2, -r * b2),
                       __uint_as_float((__float_as_uint(w) & ~7u) | flags));
}

// In the primitive-major layout the entry also names the pixel it belongs to: the 10-bit index y * 32 + x of the hit's
// pixel inside the 32 x 32-pixel window of the work item's owner replaces the three low mantissa bits of each of the
// words 0..2 (bits 0..2, 3..5, 6..8 of the index) and bit 3 of word 3 (bit 9): a relative change below 2^-20 of
// numbers needed to 1e-3.  The backward pass then finds a hit's pixel without walking any hit mask.
__device__ __forceinline__ float4 lt_embed_pix(const float4 e, const uint32_t pix) {
    return make_float4(__uint_as_float((__float_as_uint(e.x) & ~7u) | (pix & 7u)),
                       __uint_as_float((__float_as_uint(e.y) & ~7u) | ((pix >> 3) & 7u)),
                       __uint_as_float((__float_as_uint(e.z) & ~7u) | ((pix >> 6) & 7u)),
                       __uint_as_float((__float_as_uint(e.w) & ~8u) | ((pix >> 6) & 8u)));
}
__device__ __forceinline__ uint32_t lt_pix(const float4 e) {
    return (__float_as_uint(e.x) & 7u) | ((__float_as_uint(e.y) & 7u) << 3) | ((__float_as_uint(e.z) & 7u) << 6) |
           ((__float_as_uint(e.w) & 8u) << 6);
}

// The per-channel weights dL/dc = w g of an LT entry (zero on clamped channels).
__device__ __forceinline__ void lt_weights(const float4 L, const float3 g, float* wch) {
    const uint32_t b = __float_as_uint(L.w);
    const float w = __uint_as_float(b & ~15u);
    wch[0] = (b & 1u) ? w * g.x : 0.0f;
    wch[1] = (b & 2u) ? w * g.y : 0.0f;
    wch[2] = (b & 4u) ? w * g.z : 0.0f;
}

// The 8-byte form of an LT entry (lt_format 2): four halves, each the value times 4096 (weights reach down to
// alpha_min times a small transmittance: the scale keeps them in the half's normal range; +-60000 saturates).  The
// three colour words are first rounded to nine mantissa bits (nearest, ties to even), so the half's lowest bit is
// free for the channel's "not clamped" flag: a decoded word is within 2^-10 of its value, the weight within 2^-11.
constexpr float LT_HALF_SCALE = 4096.0f;
__device__ __forceinline__ uint32_t lt_half_word9(float x, uint32_t flag) {
    const float y = fminf(fmaxf(x * LT_HALF_SCALE, -60000.0f), 60000.0f);
    uint32_t u = __float_as_uint(y);
    u += 0x1FFFu + ((u >> 14) & 1u);
    u &= ~0x3FFFu;
    return ((uint32_t)__half_as_ushort(__float2half_rn(__uint_as_float(u))) & 0xFFFEu) | flag;
}
__device__ __forceinline__ uint2 lt_pack_half(const float4 e) {
    const uint32_t b = __float_as_uint(e.w);
    const float w = __uint_as_float(b & ~15u);
    const uint32_t h3 = __half_as_ushort(__float2half_rn(w * LT_HALF_SCALE));
    return make_uint2(lt_half_word9(e.x, b & 1u) | (lt_half_word9(e.y, (b >> 1) & 1u) << 16),
                      lt_half_word9(e.z, (b >> 2) & 1u) | (h3 << 16));
}
// Back to the layout of the 16-byte entry (flags in the low mantissa bits of w, which a widened half leaves zero).
__device__ __forceinline__ float4 lt_unpack_half(const uint2 p) {
    const uint32_t flags = (p.x & 1u) | ((p.x >> 15) & 2u) | ((p.y & 1u) << 2);
    const uint32_t lo = p.x & 0xFFFEFFFEu, hi = p.y & 0xFFFFFFFEu;
    const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&lo));
    const float2 c = __half22float2(*reinterpret_cast<const __half2*>(&hi));
    constexpr float inv = 1.0f / LT_HALF_SCALE;
    return make_float4(a.x * inv, a.y * inv, c.x * inv, __uint_as_float(__float_as_uint(c.y * inv) | flags));
}

// ---------------------------------------------------------------------------------------------
// Hit mask of a (tile, Gaussian) pair held as 64-bit words, walked bit by bit in pixel order.
// One loop over all words, so that the trip count of a lane is its hit count (lanes of a warp
// own pairs of nearly equal hit count) whatever the distribution of the bits over the words.
template <int MW>
struct PairMask {
    static constexpr int N64 = MW / 2;
    unsigned long long w[N64];
    unsigned long long cur;
    int qi;
    __device__ __forceinline__ void load(const uint32_t* __restrict__ pair_mask, uint32_t j, bool act) {
#pragma unroll
        for (int q = 0; q < N64; ++q) {
            const uint2 t = act ? __ldg(reinterpret_cast<const uint2*>(pair_mask + (size_t)j * MW) + q) : make_uint2(0u, 0u);
            w[q] = ((unsigned long long)t.y << 32) | t.x;
        }
        cur = w[0];
        qi = 0;
    }
    __device__ __forceinline__ int count() const {
        int c = 0;
#pragma unroll
        for (int q = 0; q < N64; ++q) c += __popcll(w[q]);
        return c;
    }
    // index (pixel of the tile) of the next set bit; call at most count() times
    __device__ __forceinline__ int next() {
        while (cur == 0ull) {
            ++qi;
            cur = qi == 1 ? w[1 % N64] : (qi == 2 ? w[2 % N64] : w[3 % N64]);
        }
        const int b = __ffsll((long long)cur) - 1;
        cur &= cur - 1ull;
        return qi * 64 + b;
    }
};

// 64-pixel tiles: two 32-bit words walked with 32-bit operations.
template <>
struct PairMask<2> {
    uint32_t lo, hi;
    int base;
    __device__ __forceinline__ void load(const uint32_t* __restrict__ pair_mask, uint32_t j, bool act) {
        const uint2 t = act ? __ldg(reinterpret_cast<const uint2*>(pair_mask + (size_t)j * 2)) : make_uint2(0u, 0u);
        lo = t.x; hi = t.y; base = 0;
    }
    __device__ __forceinline__ int count() const { return __popc(lo) + __popc(hi); }
    __device__ __forceinline__ int next() {
        if (lo == 0u) { lo = hi; hi = 0u; base = 32; }
        const int b = __ffs((int)lo) - 1;
        lo &= lo - 1u;
        return base + b;
    }
};

// ---------------------------------------------------------------------------------------------
// Real spherical harmonics (index k = l(l+1)+m) of a unit vector, first K values.
template <int K>
__device__ __forceinline__ void sh_basis(const float3 d, float* Y) {
    Y[0] = 0.28209479177387814f;
    if (K > 1) {
        Y[1] = -0.4886025119029199f * d.y;
        Y[2] = 0.4886025119029199f * d.z;
        Y[3] = -0.4886025119029199f * d.x;
    }
    if (K > 4) {
        const float xx = d.x * d.x, yy = d.y * d.y, zz = d.z * d.z;
        const float xy = d.x * d.y, yz = d.y * d.z, xz = d.x * d.z;
        Y[4] = 1.0925484305920792f * xy;
        Y[5] = -1.0925484305920792f * yz;
        Y[6] = 0.31539156525252005f * (2.0f * zz - xx - yy);
        Y[7] = -1.0925484305920792f * xz;
        Y[8] = 0.5462742152960396f * (xx - yy);
        if (K > 9) {
            Y[9] = -0.5900435899266435f * d.y * (3.0f * xx - yy);
            Y[10] = 2.890611442640554f * xy * d.z;
            Y[11] = -0.4570457994644658f * d.y * (4.0f * zz - xx - yy);
            Y[12] = 0.3731763325901154f * d.z * (2.0f * zz - 3.0f * xx - 3.0f * yy);
            Y[13] = -0.4570457994644658f * d.x * (4.0f * zz - xx - yy);
            Y[14] = 1.445305721320277f * d.z * (xx - yy);
            Y[15] = -0.5900435899266435f * d.x * (xx - 3.0f * yy);
        }
    }
}

// The same basis without its normalisation constants: Y[k] = sh_norm(k) * B[k].  A sum of B[k] * (weights) over
// many directions can take the constant once at the end; the first four B cost nothing (1, y, z, x).
template <int K>
__device__ __forceinline__ void sh_poly(const float3 d, float* B) {
    B[0] = 1.0f;
    if (K > 1) { B[1] = d.y; B[2] = d.z; B[3] = d.x; }
    if (K > 4) {
        const float xx = d.x * d.x, yy = d.y * d.y, zz = d.z * d.z;
        const float xy = d.x * d.y;
        const float e = xx - yy;
        B[4] = xy;
        B[5] = d.y * d.z;
        B[6] = fmaf(2.0f, zz, -xx) - yy;
        B[7] = d.x * d.z;
        B[8] = e;
        if (K > 9) {
            const float t = fmaf(4.0f, zz, -xx) - yy;
            B[9] = d.y * fmaf(3.0f, xx, -yy);
            B[10] = xy * d.z;
            B[11] = d.y * t;
            B[12] = d.z * fmaf(-3.0f, xx + yy, 2.0f * zz);
            B[13] = d.x * t;
            B[14] = d.z * e;
            B[15] = d.x * fmaf(-3.0f, yy, xx);
        }
    }
}
__device__ __forceinline__ constexpr float sh_norm(int k);
// normalisation constant of SH word e = 3 k + channel (1 beyond the 16 basis functions: padding words)
__device__ __forceinline__ constexpr float sh_norm_word(int e) { return e < 48 ? sh_norm(e / 3) : 0.0f; }
__device__ __forceinline__ constexpr float sh_norm(int k) {
    return k == 0 ? 0.28209479177387814f
         : k == 1 ? -0.4886025119029199f : k == 2 ? 0.4886025119029199f : k == 3 ? -0.4886025119029199f
         : k == 4 ? 1.0925484305920792f : k == 5 ? -1.0925484305920792f : k == 6 ? 0.31539156525252005f
         : k == 7 ? -1.0925484305920792f : k == 8 ? 0.5462742152960396f
         : k == 9 ? -0.5900435899266435f : k == 10 ? 2.890611442640554f : k == 11 ? -0.4570457994644658f
         : k == 12 ? 0.3731763325901154f : k == 13 ? -0.4570457994644658f : k == 14 ? 1.445305721320277f
         : -0.5900435899266435f;
}

// ---------------------------------------------------------------------------------------------
// Asynchronous bulk copies global -> shared with completion on an mbarrier.  Every wait is bounded.
constexpr uint32_t ASYNC_WAIT_LIMIT = 1u << 22;   // polls before a wait gives up (then the caller sets an error bit)

// ---- mbarrier / bulk copy (shared::cta addresses as 32-bit)
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0u;
}
// the limit a configuration asks for (gart_config::wait_polls)
static inline uint32_t wait_limit_of(int32_t wait_polls) {
    return wait_polls == 0 ? ASYNC_WAIT_LIMIT : (wait_polls < 0 ? 0u : (uint32_t)wait_polls);
}
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, uint32_t limit = ASYNC_WAIT_LIMIT) {
    for (uint32_t i = 0; i < limit; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
// Orders this thread's earlier shared-memory accesses (generic proxy) before later accesses of the
// asynchronous proxy: issued before a bulk copy overwrites a buffer that was just read.
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
// Per-thread asynchronous 16-byte copies global -> shared (one warp instruction serves all lanes, unlike a bulk
// copy, which every lane would have to issue by itself); completion by cp.async.wait_all of the issuing thread.
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async4(uint32_t dst, const void* src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }
// groups of per-thread copies: commit closes the group of the copies issued so far; wait_but_one returns when all groups
// but the most recently committed one have landed
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_but_one() { asm volatile("cp.async.wait_group 1;" ::: "memory"); }

// 32-byte (one sector) global store / read-only load; the address must be 32-byte aligned
__device__ __forceinline__ void st_global_32B(void* dst, const float4 a, const float4 b) {
    asm volatile("st.global.v8.f32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                 ::"l"(dst), "f"(a.x), "f"(a.y), "f"(a.z), "f"(a.w), "f"(b.x), "f"(b.y), "f"(b.z), "f"(b.w)
                 : "memory");
}
__device__ __forceinline__ void ld_global_nc_32B(const void* src, float4& a, float4& b) {
    asm volatile("ld.global.nc.v8.f32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=f"(a.x), "=f"(a.y), "=f"(a.z), "=f"(a.w), "=f"(b.x), "=f"(b.y), "=f"(b.z), "=f"(b.w)
                 : "l"(src));
}

// L2 eviction policies for data read once (streamed) and for data that is re-used soon.
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    return p;
}
// global -> shared bulk copy of `bytes` (multiple of 16, both addresses 16-byte aligned) with an L2 eviction policy
__device__ __forceinline__ void bulk_g2s_hint(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar, uint64_t policy) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(policy)
                 : "memory");
}
// 16-byte vector reduction into global memory with an L2 eviction policy
__device__ __forceinline__ void red_add_f4_hint(float4* dst, float a, float b, float c, float d, uint64_t policy) {
    asm volatile("red.global.add.L2::cache_hint.v4.f32 [%0], {%1, %2, %3, %4}, %5;"
                 ::"l"(dst), "f"(a), "f"(b), "f"(c), "f"(d), "l"(policy)
                 : "memory");
}


// ---------------------------------------------------------------------------------------------
// SH coefficients of a pair's Gaussian and the pair's dL/dsh accumulators, in registers.  For an even
// number of coefficients both are kept as (k, k+1) pairs per channel, so that colour evaluation and
// gradient accumulation issue packed two-wide FMAs (fma.rn.f32x2: half the issue slots).
template <int K, bool PACKED = (K % 2 == 0)>
struct ShRegs;

template <int K>
struct ShRegs<K, false> {
    float sh[3 * K], acc[3 * K];
    __device__ __forceinline__ void set(int e, float v) { sh[e] = v; acc[e] = 0.0f; }   // e = 3 k + channel
    __device__ __forceinline__ void clear() {
#pragma unroll
        for (int e = 0; e < 3 * K; ++e) acc[e] = 0.0f;
    }
    __device__ __forceinline__ float word(int e) const { return acc[e]; }
    __device__ __forceinline__ void colour(const float* Y, float* c) const {
        c[0] = 0.5f; c[1] = 0.5f; c[2] = 0.5f;
#pragma unroll
        for (int k = 0; k < K; ++k) {
            c[0] = fmaf(Y[k], sh[3 * k], c[0]);
            c[1] = fmaf(Y[k], sh[3 * k + 1], c[1]);
            c[2] = fmaf(Y[k], sh[3 * k + 2], c[2]);
        }
    }
    __device__ __forceinline__ void accumulate(const float* Y, const float* w) {
#pragma unroll
        for (int k = 0; k < K; ++k) {
            acc[3 * k] = fmaf(Y[k], w[0], acc[3 * k]);
            acc[3 * k + 1] = fmaf(Y[k], w[1], acc[3 * k + 1]);
            acc[3 * k + 2] = fmaf(Y[k], w[2], acc[3 * k + 2]);
        }
    }
};

template <int K>
struct ShRegs<K, true> {
    float2 sh[3][K / 2], acc[3][K / 2];
    __device__ __forceinline__ void set(int e, float v) {
        const int k = e / 3, c = e % 3;
        if (k & 1) { sh[c][k >> 1].y = v; acc[c][k >> 1].y = 0.0f; }
        else { sh[c][k >> 1].x = v; acc[c][k >> 1].x = 0.0f; }
    }
    __device__ __forceinline__ void clear() {
#pragma unroll
        for (int c = 0; c < 3; ++c)
#pragma unroll
            for (int i = 0; i < K / 2; ++i) acc[c][i] = make_float2(0.0f, 0.0f);
    }
    __device__ __forceinline__ float word(int e) const {
        const int k = e / 3, c = e % 3;
        return (k & 1) ? acc[c][k >> 1].y : acc[c][k >> 1].x;
    }
    __device__ __forceinline__ void colour(const float* Y, float* c) const {
        float2 a0 = make_float2(0.5f, 0.0f), a1 = a0, a2 = a0;
#pragma unroll
        for (int i = 0; i < K / 2; ++i) {
            const float2 y = make_float2(Y[2 * i], Y[2 * i + 1]);
            a0 = __ffma2_rn(y, sh[0][i], a0);
            a1 = __ffma2_rn(y, sh[1][i], a1);
            a2 = __ffma2_rn(y, sh[2][i], a2);
        }
        c[0] = a0.x + a0.y; c[1] = a1.x + a1.y; c[2] = a2.x + a2.y;
    }
    __device__ __forceinline__ void accumulate(const float* Y, const float* w) {
        const float2 w0 = make_float2(w[0], w[0]), w1 = make_float2(w[1], w[1]), w2 = make_float2(w[2], w[2]);
#pragma unroll
        for (int i = 0; i < K / 2; ++i) {
            const float2 y = make_float2(Y[2 * i], Y[2 * i + 1]);
            acc[0][i] = __ffma2_rn(y, w0, acc[0][i]);
            acc[1][i] = __ffma2_rn(y, w1, acc[1][i]);
            acc[2][i] = __ffma2_rn(y, w2, acc[2][i]);
        }
    }
};


// ---------------------------------------------------------------------------------------------
// Exclusive scan of f(0..n_cap-1) into out[0..n_cap] (uint32; out[n_cap] = total) with three
// launches and no waiting between blocks: per-block sums, one block scans the sums, per-block
// rescan.  Sums are carried in 64 bits so that an overflowing total is seen (total64_out).
// f(i) is a device functor returning uint32.
constexpr int SCAN_THREADS = 256;
constexpr int SCAN_ITEMS = 16;
constexpr int SCAN_TILE = SCAN_THREADS * SCAN_ITEMS;

__device__ __forceinline__ uint32_t warp_incl_scan(uint32_t v) {
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += t;
    }
    return v;
}

// Block-wide exclusive scan of one value per thread (SCAN_THREADS threads); returns the
// exclusive prefix and the block total.
__device__ __forceinline__ uint32_t block_excl_scan(uint32_t v, uint32_t* total) {
    __shared__ uint32_t wsum[SCAN_THREADS / 32];
    __shared__ uint32_t wtot;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const uint32_t inc = warp_incl_scan(v);
    __syncthreads();
    if (lane == 31) wsum[w] = inc;
    __syncthreads();
    if (w == 0) {
        const uint32_t s = lane < SCAN_THREADS / 32 ? wsum[lane] : 0u;
        const uint32_t si = warp_incl_scan(s);
        if (lane < SCAN_THREADS / 32) wsum[lane] = si - s;
        if (lane == SCAN_THREADS / 32 - 1) wtot = si;
    }
    __syncthreads();
    *total = wtot;
    return inc - v + wsum[w];
}

template <class F>
__global__ void __launch_bounds__(SCAN_THREADS) scan_reduce_kernel(F f, int64_t n_cap, uint64_t* block_sums) {
    const int64_t base = (int64_t)blockIdx.x * SCAN_TILE + (int64_t)threadIdx.x * SCAN_ITEMS;
    uint32_t s = 0;
#pragma unroll 4
    for (int i = 0; i < SCAN_ITEMS; ++i) {
        const int64_t idx = base + i;
        if (idx < n_cap) s += f(idx);
    }
    uint32_t tot;
    block_excl_scan(s, &tot);
    if (threadIdx.x == 0) block_sums[blockIdx.x] = tot;
}

// One block: exclusive scan of block_sums in place (uint64), total to total64_out[0].
static __global__ void __launch_bounds__(1024) scan_blocks_kernel(uint64_t* block_sums, int nb, uint64_t* total64_out) {
    __shared__ uint64_t wsum[32];
    __shared__ uint64_t carry_s;
    if (threadIdx.x == 0) carry_s = 0;
    __syncthreads();
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    for (int base = 0; base < nb; base += 1024) {
        const int i = base + threadIdx.x;
        const uint64_t v = i < nb ? block_sums[i] : 0ull;
        uint64_t inc = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint64_t t = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += t;
        }
        if (lane == 31) wsum[w] = inc;
        __syncthreads();
        if (w == 0) {
            const uint64_t s = wsum[lane];
            uint64_t si = s;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint64_t t = __shfl_up_sync(0xffffffffu, si, o);
                if (lane >= o) si += t;
            }
            wsum[lane] = si - s;
        }
        __syncthreads();
        const uint64_t carry = carry_s;
        const uint64_t excl = carry + wsum[w] + inc - v;
        if (i < nb) block_sums[i] = excl;
        __syncthreads();
        if (threadIdx.x == 1023) carry_s = excl + v;
        __syncthreads();
    }
    if (threadIdx.x == 0) total64_out[0] = carry_s;
}

template <class F>
__global__ void __launch_bounds__(SCAN_THREADS) scan_apply_kernel(F f, int64_t n_cap, const uint64_t* block_offs, uint32_t* out) {
    const int64_t base = (int64_t)blockIdx.x * SCAN_TILE + (int64_t)threadIdx.x * SCAN_ITEMS;
    uint32_t v[SCAN_ITEMS];
    uint32_t s = 0;
#pragma unroll
    for (int i = 0; i < SCAN_ITEMS; ++i) {
        const int64_t idx = base + i;
        v[i] = idx < n_cap ? f(idx) : 0u;
        s += v[i];
    }
    uint32_t tot;
    uint32_t run = block_excl_scan(s, &tot) + (uint32_t)block_offs[blockIdx.x];
#pragma unroll
    for (int i = 0; i < SCAN_ITEMS; ++i) {
        const int64_t idx = base + i;
        if (idx < n_cap) out[idx] = run;
        run += v[i];
        if (idx == n_cap - 1) out[n_cap] = run;
    }
}

static inline size_t scan_workspace_bytes(int64_t n_cap) {
    return align256((size_t)(ceil_div(n_cap > 0 ? n_cap : 1, SCAN_TILE) + 1) * sizeof(uint64_t)) + 256;
}

// out[0..n_cap] = exclusive scan of f; total64 (device, 8-byte aligned) receives the 64-bit total.
// ws must hold scan_workspace_bytes(n_cap) bytes.  n_cap >= 1.
template <class F>
static inline gart_status exclusive_scan(F f, int64_t n_cap, uint32_t* out, uint64_t* total64, void* ws, cudaStream_t st) {
    const int nb = (int)ceil_div(n_cap, SCAN_TILE);
    uint64_t* block_sums = (uint64_t*)ws;
    scan_reduce_kernel<F><<<nb, SCAN_THREADS, 0, st>>>(f, n_cap, block_sums);
    GART_LAUNCH_CHECK();
    scan_blocks_kernel<<<1, 1024, 0, st>>>(block_sums, nb, total64);
    GART_LAUNCH_CHECK();
    scan_apply_kernel<F><<<nb, SCAN_THREADS, 0, st>>>(f, n_cap, block_sums, out);
    GART_LAUNCH_CHECK();
    return GART_OK;
}

}  // namespace gart
