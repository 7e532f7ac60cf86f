// gart_backward: primitive-centric backward (Sec. 4.4) and gart_backward_atomic, the
// pixel-centric baseline (Sec. 3.5).
//
// Per hit (ray r, Gaussian i), with g = dL/dC_r, T = transmittance in front of the hit, Rb =
// colour composited behind it (both from the LT buffer), alpha, x_g recomputed from the record:
//   dL/dsh_k   += Y_k(d_r) * T alpha g            (channels whose raw colour is positive)
//   dL/dalpha   = g . (T c - Rb / (1 - alpha))
//   dL/dsigma  += dL/dalpha * alpha / sigma
//   G           = dL/d(D^2) = -alpha dL/dalpha / 2       (the maximum-response point is
//                 stationary in t, so t* carries no gradient)
//   v += G x_g,  Q += G x_g x_g^T
// and, once per Gaussian (all sums are linear in v and Q, with W = S^-1 R^T):
//   dL/dmu = -2 W^T v,  dL/ds_k = -2 Q_kk / s_k,  dL/dR = 2 R^-T S Q S^-1,  dL/dq by the chain
//   rule through the polynomial rotation formula.
// gart_backward accumulates (v, Q, sum alpha dL/dalpha, dL/dsh) per (tile, Gaussian) pair in
// registers, adds them to the Gaussian's record with one vector atomic per 16 bytes, and a
// per-Gaussian pass converts the record in place.  The baseline converts per hit and issues one
// scalar atomicAdd per gradient word per hit.
#include "common.cuh"

namespace gart {

// -------------------------------------------------------------------------------- per-Gaussian conversion
struct GeoGrad {
    float dmu[3], ds[3], dq[4];
};

// v[3], Q = (xx, yy, zz, xy, xz, yz) -> gradients of mean, scale, quaternion.
__device__ __forceinline__ GeoGrad moments_to_grads(const float* v, const float* Q, const float* q, const float* s) {
    const float w = q[0], x = q[1], y = q[2], z = q[3];
    float R[9];
    R[0] = 1.0f - 2.0f * (y * y + z * z); R[1] = 2.0f * (x * y - w * z); R[2] = 2.0f * (x * z + w * y);
    R[3] = 2.0f * (x * y + w * z); R[4] = 1.0f - 2.0f * (x * x + z * z); R[5] = 2.0f * (y * z - w * x);
    R[6] = 2.0f * (x * z - w * y); R[7] = 2.0f * (y * z + w * x); R[8] = 1.0f - 2.0f * (x * x + y * y);
    const float is[3] = {1.0f / s[0], 1.0f / s[1], 1.0f / s[2]};
    GeoGrad o;
    const float vs[3] = {v[0] * is[0], v[1] * is[1], v[2] * is[2]};
#pragma unroll
    for (int j = 0; j < 3; ++j) o.dmu[j] = -2.0f * (R[3 * j] * vs[0] + R[3 * j + 1] * vs[1] + R[3 * j + 2] * vs[2]);
    o.ds[0] = -2.0f * Q[0] * is[0];
    o.ds[1] = -2.0f * Q[1] * is[1];
    o.ds[2] = -2.0f * Q[2] * is[2];
    // R^-T = cof(R) / det(R)
    float C[9];
    C[0] = R[4] * R[8] - R[5] * R[7]; C[1] = R[5] * R[6] - R[3] * R[8]; C[2] = R[3] * R[7] - R[4] * R[6];
    C[3] = R[2] * R[7] - R[1] * R[8]; C[4] = R[0] * R[8] - R[2] * R[6]; C[5] = R[1] * R[6] - R[0] * R[7];
    C[6] = R[1] * R[5] - R[2] * R[4]; C[7] = R[2] * R[3] - R[0] * R[5]; C[8] = R[0] * R[4] - R[1] * R[3];
    const float idet = 1.0f / (R[0] * C[0] + R[1] * C[1] + R[2] * C[2]);
    // B = S Q S^-1
    const float Qm[9] = {Q[0], Q[3], Q[4], Q[3], Q[1], Q[5], Q[4], Q[5], Q[2]};
    float B[9];
#pragma unroll
    for (int l = 0; l < 3; ++l)
#pragma unroll
        for (int k = 0; k < 3; ++k) B[3 * l + k] = s[l] * Qm[3 * l + k] * is[k];
    float dR[9];
#pragma unroll
    for (int j = 0; j < 3; ++j)
#pragma unroll
        for (int k = 0; k < 3; ++k)
            dR[3 * j + k] = 2.0f * idet * (C[3 * j] * B[k] + C[3 * j + 1] * B[3 + k] + C[3 * j + 2] * B[6 + k]);
    o.dq[0] = 2.0f * (-z * dR[1] + y * dR[2] + z * dR[3] - x * dR[5] - y * dR[6] + x * dR[7]);
    o.dq[1] = 2.0f * (y * dR[1] + z * dR[2] + y * dR[3] - 2.0f * x * dR[4] - w * dR[5] + z * dR[6] + w * dR[7] - 2.0f * x * dR[8]);
    o.dq[2] = 2.0f * (-2.0f * y * dR[0] + x * dR[1] + w * dR[2] + x * dR[3] + z * dR[5] - w * dR[6] + z * dR[7] - 2.0f * y * dR[8]);
    o.dq[3] = 2.0f * (-2.0f * z * dR[0] - w * dR[1] + x * dR[2] + w * dR[3] - 2.0f * z * dR[4] + y * dR[5] + x * dR[6] + y * dR[7]);
    return o;
}

// Per-hit gradient terms shared by both backward variants.
template <int K>
struct HitGrad {
    float wch[3];   // T alpha g per channel, zero where the colour is clamped
    float dalpha;   // dL/dalpha
};

template <int K>
__device__ __forceinline__ HitGrad<K> hit_grad(const float* Y, const float* shc, const float3 g, const float4 L, const float alpha) {
    float c0 = 0.5f, c1 = 0.5f, c2 = 0.5f;
#pragma unroll
    for (int k = 0; k < K; ++k) {
        c0 = fmaf(Y[k], shc[3 * k], c0);
        c1 = fmaf(Y[k], shc[3 * k + 1], c1);
        c2 = fmaf(Y[k], shc[3 * k + 2], c2);
    }
    const float T = L.w;
    const float Ta = T * alpha;
    const float inv = __frcp_rn(1.0f - alpha);
    HitGrad<K> h;
    h.wch[0] = c0 > 0.0f ? Ta * g.x : 0.0f;
    h.wch[1] = c1 > 0.0f ? Ta * g.y : 0.0f;
    h.wch[2] = c2 > 0.0f ? Ta * g.z : 0.0f;
    const float t0 = fmaf(T, fmaxf(c0, 0.0f), -L.x * inv);
    const float t1 = fmaf(T, fmaxf(c1, 0.0f), -L.y * inv);
    const float t2 = fmaf(T, fmaxf(c2, 0.0f), -L.z * inv);
    h.dalpha = fmaf(g.x, t0, fmaf(g.y, t1, g.z * t2));
    return h;
}

// -------------------------------------------------------------------------------- primitive-centric
constexpr int BWD_THREADS = 128;

template <int K>
struct PixLayout {
    static constexpr int W = (K + 3 + 3) & ~3;   // floats per pixel record: Y[K], g[3], zero padding
};

template <int TS, int DEG>
__global__ void __launch_bounds__(BWD_THREADS) bwd_pairs_kernel(const float4* __restrict__ pre4, const float* __restrict__ sh,
                                                                const uint32_t* __restrict__ tile_off, const uint32_t* __restrict__ pair_gid,
                                                                const uint32_t* __restrict__ pair_mask, const uint32_t* __restrict__ pair_lt_off,
                                                                const float4* __restrict__ lt, const float* __restrict__ dL_dC, CamF cam,
                                                                float* __restrict__ grad, const uint32_t* __restrict__ counts) {
    constexpr int NT = TS * TS, MW = NT / 32, K = (DEG + 1) * (DEG + 1), SW = 3 * K, PW = PixLayout<K>::W;
    constexpr int AW = (11 + SW + 3) & ~3;   // accumulator words, multiple of 4
    __shared__ __align__(16) float spix[NT * PW];
    if (counts[GART_CNT_ERROR]) return;
    const int tile = blockIdx.x;
    const uint32_t begin = tile_off[tile], end = tile_off[tile + 1];
    if (begin == end) return;
    const int tx = tile % cam.tiles_x, ty = tile / cam.tiles_x;
    const int x0 = tx * TS, y0 = ty * TS;
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

    for (uint32_t j = begin + threadIdx.x; j < end; j += BWD_THREADS) {
        uint32_t mk[MW];
        uint32_t any = 0;
#pragma unroll
        for (int q = 0; q < MW; ++q) { mk[q] = __ldg(pair_mask + (size_t)j * MW + q); any |= mk[q]; }
        if (!any) continue;
        const uint32_t gid = __ldg(pair_gid + j);
        const PreRec P = load_pre(pre4, gid);
        float shc[SW];
        {
            const float* sp = sh + (size_t)gid * SW;
            if (SW % 4 == 0) {
#pragma unroll
                for (int q = 0; q < SW / 4; ++q) {
                    const float4 t = __ldg(reinterpret_cast<const float4*>(sp) + q);
                    shc[4 * q] = t.x; shc[4 * q + 1] = t.y; shc[4 * q + 2] = t.z; shc[4 * q + 3] = t.w;
                }
            } else {
#pragma unroll
                for (int q = 0; q < SW; ++q) shc[q] = __ldg(sp + q);
            }
        }
        float acc[AW];
#pragma unroll
        for (int q = 0; q < AW; ++q) acc[q] = 0.0f;
        const float4* lp = lt + __ldg(pair_lt_off + j);
        const int bx = x0 - P.ix, by = y0 - P.iy;
#pragma unroll
        for (int q = 0; q < MW; ++q) {
            uint32_t word = mk[q];
            while (word) {
                const int b = __ffs(word) - 1;
                word &= word - 1;
                const int p = q * 32 + b;
                const float4 L = __ldg(lp++);
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
                    for (int k = 0; k < K; ++k) Y[k] = rec[k];
                }
                const float3 g = make_float3(rec[K], rec[K + 1], rec[K + 2]);
                const HitGrad<K> h = hit_grad<K>(Y, shc, g, L, r.alpha);
#pragma unroll
                for (int k = 0; k < K; ++k) {
                    acc[11 + 3 * k] = fmaf(Y[k], h.wch[0], acc[11 + 3 * k]);
                    acc[11 + 3 * k + 1] = fmaf(Y[k], h.wch[1], acc[11 + 3 * k + 1]);
                    acc[11 + 3 * k + 2] = fmaf(Y[k], h.wch[2], acc[11 + 3 * k + 2]);
                }
                const float ad = r.alpha * h.dalpha;
                acc[9] += ad;
                const float G = -0.5f * ad;
                const float3 xg = ray_xg(r);
                const float gx = G * xg.x, gy = G * xg.y, gz = G * xg.z;
                acc[0] += gx; acc[1] += gy; acc[2] += gz;
                acc[3] = fmaf(gx, xg.x, acc[3]); acc[4] = fmaf(gy, xg.y, acc[4]); acc[5] = fmaf(gz, xg.z, acc[5]);
                acc[6] = fmaf(gx, xg.y, acc[6]); acc[7] = fmaf(gx, xg.z, acc[7]); acc[8] = fmaf(gy, xg.z, acc[8]);
            }
        }
        // one vector atomic per 16 bytes of the Gaussian's record
        float4* gp = reinterpret_cast<float4*>(grad + (size_t)gid * GART_GRAD_WORDS);
#pragma unroll
        for (int q = 0; q < AW / 4; ++q) atomicAdd(gp + q, make_float4(acc[4 * q], acc[4 * q + 1], acc[4 * q + 2], acc[4 * q + 3]));
    }
}

// In-place conversion of the accumulated moments (words 0..9) into d mean, d scale, d quat, d opacity.
__global__ void __launch_bounds__(256) bwd_finalize_kernel(int64_t n, const float* __restrict__ scale, const float* __restrict__ quat,
                                                           const float* __restrict__ opacity, float* __restrict__ grad,
                                                           const uint32_t* __restrict__ counts) {
    if (counts[GART_CNT_ERROR]) return;
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    float4* gp = reinterpret_cast<float4*>(grad + (size_t)i * GART_GRAD_WORDS);
    const float4 a = gp[0], b = gp[1], c = gp[2];
    const float v[3] = {a.x, a.y, a.z};
    const float Q[6] = {a.w, b.x, b.y, b.z, b.w, c.x};
    bool nz = c.y != 0.0f;
#pragma unroll
    for (int k = 0; k < 3; ++k) nz = nz || v[k] != 0.0f;
#pragma unroll
    for (int k = 0; k < 6; ++k) nz = nz || Q[k] != 0.0f;
    if (!nz) return;
    const float q[4] = {quat[4 * i], quat[4 * i + 1], quat[4 * i + 2], quat[4 * i + 3]};
    const float s[3] = {scale[3 * i], scale[3 * i + 1], scale[3 * i + 2]};
    const GeoGrad o = moments_to_grads(v, Q, q, s);
    gp[0] = make_float4(o.dmu[0], o.dmu[1], o.dmu[2], o.ds[0]);
    gp[1] = make_float4(o.ds[1], o.ds[2], o.dq[0], o.dq[1]);
    gp[2] = make_float4(o.dq[2], o.dq[3], c.y / opacity[i], c.w);
}

// -------------------------------------------------------------------------------- pixel-centric baseline
template <int DEG>
__global__ void __launch_bounds__(128) bwd_atomic_kernel(const float4* __restrict__ pre4, const float* __restrict__ sh,
                                                         const float* __restrict__ scale, const float* __restrict__ quat,
                                                         const float* __restrict__ opacity, const uint32_t* __restrict__ ray_off,
                                                         const uint32_t* __restrict__ ray_gid, const uint32_t* __restrict__ ray_slot,
                                                         const float4* __restrict__ lt, const float* __restrict__ dL_dC, CamF cam,
                                                         float* __restrict__ grad, const uint32_t* __restrict__ counts) {
    constexpr int K = (DEG + 1) * (DEG + 1), SW = 3 * K;
    if (counts[GART_CNT_ERROR]) return;
    const int64_t ray = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (ray >= (int64_t)cam.width * cam.height) return;
    const uint32_t b = ray_off[ray], e = ray_off[ray + 1];
    if (b == e) return;
    const int x = (int)(ray % cam.width), y = (int)(ray / cam.width);
    float Y[K];
    sh_basis<K>(pixel_dir(cam, x, y), Y);
    const float3 g = make_float3(dL_dC[3 * ray], dL_dC[3 * ray + 1], dL_dC[3 * ray + 2]);
    for (uint32_t h = b; h < e; ++h) {
        const uint32_t gid = ray_gid[h];
        const float4 L = lt[ray_slot[h]];
        const PreRec P = load_pre(pre4, gid);
        const RayEval r = ray_eval(P, (float)(x - P.ix) - P.rx, (float)(y - P.iy) - P.ry);
        float shc[SW];
#pragma unroll
        for (int q = 0; q < SW; ++q) shc[q] = __ldg(sh + (size_t)gid * SW + q);
        const HitGrad<K> hg = hit_grad<K>(Y, shc, g, L, r.alpha);
        const float ad = r.alpha * hg.dalpha;
        const float G = -0.5f * ad;
        const float3 xg = ray_xg(r);
        const float v[3] = {G * xg.x, G * xg.y, G * xg.z};
        const float Q[6] = {v[0] * xg.x, v[1] * xg.y, v[2] * xg.z, v[0] * xg.y, v[0] * xg.z, v[1] * xg.z};
        const float q[4] = {quat[4 * gid], quat[4 * gid + 1], quat[4 * gid + 2], quat[4 * gid + 3]};
        const float s[3] = {scale[3 * gid], scale[3 * gid + 1], scale[3 * gid + 2]};
        const GeoGrad o = moments_to_grads(v, Q, q, s);
        float* gp = grad + (size_t)gid * GART_GRAD_WORDS;
        atomicAdd(gp + 0, o.dmu[0]); atomicAdd(gp + 1, o.dmu[1]); atomicAdd(gp + 2, o.dmu[2]);
        atomicAdd(gp + 3, o.ds[0]); atomicAdd(gp + 4, o.ds[1]); atomicAdd(gp + 5, o.ds[2]);
        atomicAdd(gp + 6, o.dq[0]); atomicAdd(gp + 7, o.dq[1]); atomicAdd(gp + 8, o.dq[2]); atomicAdd(gp + 9, o.dq[3]);
        atomicAdd(gp + 10, ad / opacity[gid]);
#pragma unroll
        for (int k = 0; k < K; ++k) {
            atomicAdd(gp + 11 + 3 * k, Y[k] * hg.wch[0]);
            atomicAdd(gp + 11 + 3 * k + 1, Y[k] * hg.wch[1]);
            atomicAdd(gp + 11 + 3 * k + 2, Y[k] * hg.wch[2]);
        }
    }
}

template <int TS>
static gart_status launch_pairs(int deg, int T, cudaStream_t st, const float4* pre4, const float* sh, const uint32_t* tile_off,
                                const uint32_t* pair_gid, const uint32_t* pair_mask, const uint32_t* pair_lt_off, const float4* lt,
                                const float* dL_dC, const CamF& cam, float* grad, const uint32_t* counts) {
#define GART_PAIRS(D) \
    bwd_pairs_kernel<TS, D><<<T, BWD_THREADS, 0, st>>>(pre4, sh, tile_off, pair_gid, pair_mask, pair_lt_off, lt, dL_dC, cam, grad, counts)
    switch (deg) {
        case 0: GART_PAIRS(0); break;
        case 1: GART_PAIRS(1); break;
        case 2: GART_PAIRS(2); break;
        default: GART_PAIRS(3); break;
    }
#undef GART_PAIRS
    GART_LAUNCH_CHECK();
    return GART_OK;
}

}  // namespace gart

extern "C" gart_status gart_backward(const gart_config* cfg, const gart_gaussians* g, const gart_camera* cam, const float* pre,
                                     const uint32_t* tile_off, const uint32_t* pair_gid, const uint32_t* pair_mask,
                                     const uint32_t* pair_lt_off, const float* lt, const float* dL_dcolor,
                                     float* grad, const uint32_t* counts, void* stream) {
    using namespace gart;
    if (!cfg || !g || !cam || !counts || !tile_off || !pair_lt_off || !dL_dcolor) return GART_ERR_INVALID_ARG;
    if (cfg->tile_size != 8 && cfg->tile_size != 16) return GART_ERR_INVALID_ARG;
    if (g->n < 0 || g->sh_degree < 0 || g->sh_degree > 3) return GART_ERR_INVALID_ARG;
    if (g->n == 0) return GART_OK;
    if (!grad || !pre || !g->scale || !g->quat || !g->opacity || !g->sh) return GART_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemsetAsync(grad, 0, (size_t)g->n * GART_GRAD_WORDS * sizeof(float), st) != cudaSuccess) return GART_ERR_CUDA;
    const CamF cf = make_camf(cam, cfg->tile_size);
    const int T = cf.tiles_x * cf.tiles_y;
    const float4* pre4 = reinterpret_cast<const float4*>(pre);
    const float4* lt4 = reinterpret_cast<const float4*>(lt);
    gart_status s;
    if (cfg->tile_size == 8) s = launch_pairs<8>(g->sh_degree, T, st, pre4, g->sh, tile_off, pair_gid, pair_mask, pair_lt_off, lt4, dL_dcolor, cf, grad, counts);
    else s = launch_pairs<16>(g->sh_degree, T, st, pre4, g->sh, tile_off, pair_gid, pair_mask, pair_lt_off, lt4, dL_dcolor, cf, grad, counts);
    if (s != GART_OK) return s;
    bwd_finalize_kernel<<<(unsigned)ceil_div(g->n, 256), 256, 0, st>>>(g->n, g->scale, g->quat, g->opacity, grad, counts);
    GART_LAUNCH_CHECK();
    return GART_OK;
}

extern "C" gart_status gart_backward_atomic(const gart_config* cfg, const gart_gaussians* g, const gart_camera* cam,
                                            const float* pre, const uint32_t* ray_off, const uint32_t* ray_gid,
                                            const uint32_t* ray_slot, const float* lt, const float* dL_dcolor,
                                            float* grad, const uint32_t* counts, void* stream) {
    using namespace gart;
    if (!cfg || !g || !cam || !counts || !ray_off || !dL_dcolor) return GART_ERR_INVALID_ARG;
    if (cfg->tile_size != 8 && cfg->tile_size != 16) return GART_ERR_INVALID_ARG;
    if (g->n < 0 || g->sh_degree < 0 || g->sh_degree > 3) return GART_ERR_INVALID_ARG;
    if (g->n == 0) return GART_OK;
    if (!grad || !pre || !g->scale || !g->quat || !g->opacity || !g->sh) return GART_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemsetAsync(grad, 0, (size_t)g->n * GART_GRAD_WORDS * sizeof(float), st) != cudaSuccess) return GART_ERR_CUDA;
    const CamF cf = make_camf(cam, cfg->tile_size);
    const int64_t n_rays = (int64_t)cam->width * cam->height;
    const float4* pre4 = reinterpret_cast<const float4*>(pre);
    const float4* lt4 = reinterpret_cast<const float4*>(lt);
    const unsigned blocks = (unsigned)ceil_div(n_rays, 128);
#define GART_ATOMIC(D) \
    bwd_atomic_kernel<D><<<blocks, 128, 0, st>>>(pre4, g->sh, g->scale, g->quat, g->opacity, ray_off, ray_gid, ray_slot, lt4, dL_dcolor, cf, grad, counts)
    switch (g->sh_degree) {
        case 0: GART_ATOMIC(0); break;
        case 1: GART_ATOMIC(1); break;
        case 2: GART_ATOMIC(2); break;
        default: GART_ATOMIC(3); break;
    }
#undef GART_ATOMIC
    GART_LAUNCH_CHECK();
    return GART_OK;
}
