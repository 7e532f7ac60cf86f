// gart_backward_atomic: the pixel-centric baseline (Sec. 3.5).  One thread per ray walks the ray's
// hits in compositing order, converts every hit's terms to gradients of the Gaussian's parameters
// and issues one scalar atomicAdd per gradient word per hit (11 + 3K; 59 at SH degree 3): the
// contention-heavy scatter that the primitive-centric pass replaces.  A second mode issues the same sums as
// 16-byte vector reductions (four words each), which is as strong as the plain scatter gets on this hardware.
#include "backward_common.cuh"

namespace gart {

// -------------------------------------------------------------------------------- pixel-centric baseline
template <int DEG, bool VEC>
__global__ void __launch_bounds__(128) bwd_atomic_kernel(const float4* __restrict__ rec, const uint32_t* __restrict__ slot_of_gid,
                                                         const float* __restrict__ scale, const float* __restrict__ quat,
                                                         const float* __restrict__ opacity, const uint32_t* __restrict__ ray_off,
                                                         const uint32_t* __restrict__ ray_gid, const uint32_t* __restrict__ ray_slot,
                                                         const float4* __restrict__ lt, const float* __restrict__ dL_dC, CamF cam,
                                                         float* __restrict__ grad, const uint32_t* __restrict__ counts, const bool narrow) {
    constexpr int K = (DEG + 1) * (DEG + 1), RS4 = REC_F4;
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
        const float4* rp = rec + (size_t)__ldg(slot_of_gid + gid) * RS4;
        const PreRec P = load_pre(rp);
        const RayEval r = ray_eval(P, (float)(x - P.ix) - P.rx, (float)(y - P.iy) - P.ry);
        float wch[3];
        lt_weights(L, g, wch);
        const float ad = fmaf(g.x, L.x, fmaf(g.y, L.y, g.z * L.z));   // alpha dL/dalpha
        const float3 xg = ray_xg(r);
        // dL/d(D^2): -1/2 alpha dL/dalpha for the Gaussian, -D^2 alpha dL/dalpha for the degree-4 kernel (D^2 = |x_g|^2)
        const float G = narrow ? -ad * fmaf(xg.x, xg.x, fmaf(xg.y, xg.y, xg.z * xg.z)) : -0.5f * ad;
        const float v[3] = {G * xg.x, G * xg.y, G * xg.z};
        const float Q[6] = {v[0] * xg.x, v[1] * xg.y, v[2] * xg.z, v[0] * xg.y, v[0] * xg.z, v[1] * xg.z};
        const float q[4] = {quat[4 * gid], quat[4 * gid + 1], quat[4 * gid + 2], quat[4 * gid + 3]};
        const float s[3] = {scale[3 * gid], scale[3 * gid + 1], scale[3 * gid + 2]};
        const GeoGrad o = moments_to_grads(v, Q, q, s);
        float* gp = grad + (size_t)gid * GART_GRAD_WORDS;
        if (VEC) {
            constexpr int NV = (11 + 3 * K + 3) / 4;
            float out[4 * NV];
            out[0] = o.dmu[0]; out[1] = o.dmu[1]; out[2] = o.dmu[2];
            out[3] = o.ds[0]; out[4] = o.ds[1]; out[5] = o.ds[2];
            out[6] = o.dq[0]; out[7] = o.dq[1]; out[8] = o.dq[2]; out[9] = o.dq[3];
            out[10] = ad / opacity[gid];
#pragma unroll
            for (int k = 0; k < K; ++k) {
                out[11 + 3 * k] = Y[k] * wch[0];
                out[11 + 3 * k + 1] = Y[k] * wch[1];
                out[11 + 3 * k + 2] = Y[k] * wch[2];
            }
#pragma unroll
            for (int q = 11 + 3 * K; q < 4 * NV; ++q) out[q] = 0.0f;
#pragma unroll
            for (int q = 0; q < NV; ++q)
                asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(gp + 4 * q), "f"(out[4 * q]), "f"(out[4 * q + 1]),
                             "f"(out[4 * q + 2]), "f"(out[4 * q + 3])
                             : "memory");
            continue;
        }
        atomicAdd(gp + 0, o.dmu[0]); atomicAdd(gp + 1, o.dmu[1]); atomicAdd(gp + 2, o.dmu[2]);
        atomicAdd(gp + 3, o.ds[0]); atomicAdd(gp + 4, o.ds[1]); atomicAdd(gp + 5, o.ds[2]);
        atomicAdd(gp + 6, o.dq[0]); atomicAdd(gp + 7, o.dq[1]); atomicAdd(gp + 8, o.dq[2]); atomicAdd(gp + 9, o.dq[3]);
        atomicAdd(gp + 10, ad / opacity[gid]);
#pragma unroll
        for (int k = 0; k < K; ++k) {
            atomicAdd(gp + 11 + 3 * k, Y[k] * wch[0]);
            atomicAdd(gp + 11 + 3 * k + 1, Y[k] * wch[1]);
            atomicAdd(gp + 11 + 3 * k + 2, Y[k] * wch[2]);
        }
    }
}

}  // namespace gart

extern "C" gart_status gart_backward_atomic(const gart_config* cfg, const gart_gaussians* g, const gart_camera* cam,
                                            const float* pre, const uint32_t* slot_of_gid, const uint32_t* ray_off, const uint32_t* ray_gid,
                                            const uint32_t* ray_slot, const float* lt, const float* dL_dcolor,
                                            float* grad, const uint32_t* counts, void* stream) {
    using namespace gart;
    if (!cfg || !g || !cam || !counts || !ray_off || !dL_dcolor) return GART_ERR_INVALID_ARG;
    if (cfg->tile_size != 8 && cfg->tile_size != 16) return GART_ERR_INVALID_ARG;
    if (g->n < 0 || g->sh_degree < 0 || g->sh_degree > 3) return GART_ERR_INVALID_ARG;
    if (g->n == 0) return GART_OK;
    if (!grad || !pre || !slot_of_gid || !g->scale || !g->quat || !g->opacity || !ray_gid || !ray_slot || !lt) return GART_ERR_INVALID_ARG;
    if (cfg->atomic_mode != GART_ATOMIC_SCALAR && cfg->atomic_mode != GART_ATOMIC_VECTOR) return GART_ERR_INVALID_ARG;
    if (cfg->lt_format != 0) return GART_ERR_INVALID_ARG;   // reads 16-byte LT entries (either layout: the slot of every hit comes from ray_slot)
    if (!kernel_degree_ok(cfg->kernel_degree)) return GART_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemsetAsync(grad, 0, (size_t)g->n * GART_GRAD_WORDS * sizeof(float), st) != cudaSuccess) return GART_ERR_CUDA;
    const CamF cf = make_camf(cam, cfg->tile_size);
    const int64_t n_rays = (int64_t)cam->width * cam->height;
    const float4* rec = reinterpret_cast<const float4*>(pre);
    const float4* lt4 = reinterpret_cast<const float4*>(lt);
    const unsigned blocks = (unsigned)ceil_div(n_rays, 128);
#define GART_ATOMIC_ARGS <<<blocks, 128, 0, st>>>(rec, slot_of_gid, g->scale, g->quat, g->opacity, ray_off, ray_gid, ray_slot, lt4, dL_dcolor, cf, grad, counts, kernel_degree_is4(cfg->kernel_degree))
#define GART_ATOMIC(D)                                                             \
    if (cfg->atomic_mode == GART_ATOMIC_VECTOR) bwd_atomic_kernel<D, true> GART_ATOMIC_ARGS; \
    else bwd_atomic_kernel<D, false> GART_ATOMIC_ARGS
    switch (g->sh_degree) {
        case 0: GART_ATOMIC(0); break;
        case 1: GART_ATOMIC(1); break;
        case 2: GART_ATOMIC(2); break;
        default: GART_ATOMIC(3); break;
    }
#undef GART_ATOMIC
#undef GART_ATOMIC_ARGS
    GART_LAUNCH_CHECK();
    return GART_OK;
}
