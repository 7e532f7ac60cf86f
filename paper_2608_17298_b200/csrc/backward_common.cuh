// Arithmetic shared by the two backward variants: the per-hit gradient terms and the per-Gaussian
// conversion of the accumulated moments into gradients of mean, scale and quaternion.
//
// Per hit (ray r, Gaussian i), with g = dL/dC_r, T = transmittance in front of the hit, Rb =
// colour composited behind it (both from the LT buffer), alpha, x_g recomputed from the record:
//   dL/dsh_k   += Y_k(d_r) * T alpha g            (channels whose raw colour is positive)
//   dL/dalpha   = g . (T c - Rb / (1 - alpha))
//   dL/dsigma  += dL/dalpha * alpha / sigma
//   G           = dL/d(D^2) = -alpha dL/dalpha / 2       (the maximum-response point is
//                 stationary in t, so t* carries no gradient)
//   v += G x_g,  Q += G x_g x_g^T
// and, per Gaussian (all sums are linear in v and Q, with W = S^-1 R^T):
//   dL/dmu = -2 W^T v,  dL/ds_k = -2 Q_kk / s_k,  dL/dR = 2 R^-T S Q S^-1,  dL/dq by the chain
//   rule through the polynomial rotation formula.
#pragma once

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

// Per-pixel data of the tile in shared memory: two float4 per pixel, (d.x, d.y, d.z, x) and (g.r, g.g, g.b, y)
// with d the unit ray direction, g = dL/dC and (x, y) the pixel's position in the tile.  Lanes of a warp read
// DIFFERENT pixels at the same time, so a single copy suffers bank conflicts at random; with C copies, copy j
// laid out in the 16-byte bank groups j, j + C, ... only and lane l reading copy l mod C, the 8 lanes that a
// 16-byte shared load serves together collide 8 / C at a time at most.  Four copies (8 KB): measured 0.02 ms faster
// per view than eight, which never collide but take twice as long to fill for every tile; two copies are 0.03 ms slower.
// (Tiles of 256 pixels keep one copy, 3 float4 apart.)
template <int TS>
struct PixLayout {
    static constexpr int COPIES = TS == 8 ? 4 : 1;
    static constexpr int STRIDE = COPIES == 1 ? 3 : 2;                 // float4 per pixel within a copy
    static constexpr int F4 = TS * TS * STRIDE * COPIES;               // float4 in all
    __device__ static __forceinline__ int index(int p, int h, int copy) { return (p * STRIDE + h) * COPIES + copy; }
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

// The accumulation record of a slot, as the gradient record's words 0..59 in two pieces: words 0..15 (moments v, Q,
// sum alpha dL/dalpha, one unused word, the first five dL/dsh words) in one array of 64-byte rows, words 16..59 (the
// rest of dL/dsh) in another of 176-byte rows.  The conversion then reads compact, coalesced rows, and nothing is
// moved or zeroed for the record's four padding words.
constexpr int GACC_A_WORDS = 16, GACC_B_WORDS = 44;
struct Gacc {
    float* a;   // [n][GACC_A_WORDS]
    float* b;   // [n][GACC_B_WORDS]
};
static inline size_t gacc_bytes(int64_t n) { return align256((size_t)n * GACC_A_WORDS * 4) + align256((size_t)n * GACC_B_WORDS * 4); }
static inline Gacc make_gacc(void* workspace, int64_t n) {
    Gacc g;
    g.a = reinterpret_cast<float*>(workspace);
    g.b = reinterpret_cast<float*>(reinterpret_cast<char*>(workspace) + align256((size_t)n * GACC_A_WORDS * 4));
    return g;
}
// float4 number q (0..14) of slot sid's record
__device__ __forceinline__ float4* gacc_piece(const Gacc& g, uint32_t sid, int q) {
    return q < 4 ? reinterpret_cast<float4*>(g.a + (size_t)sid * GACC_A_WORDS) + q
                 : reinterpret_cast<float4*>(g.b + (size_t)sid * GACC_B_WORDS) + (q - 4);
}

// Zero the accumulation records of the view's slots (their number lives on the device): grid-stride.
static __global__ void __launch_bounds__(256) bwd_zero_kernel(Gacc gacc, const uint32_t* __restrict__ counts) {
    const size_t V = counts[GART_CNT_VISIBLE];
    const size_t na = V * (GACC_A_WORDS / 4), total = na + V * (GACC_B_WORDS / 4);
    float4* a4 = reinterpret_cast<float4*>(gacc.a);
    float4* b4 = reinterpret_cast<float4*>(gacc.b);
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        if (i < na) a4[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        else b4[i - na] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
}

// The accumulation records hold dL/dsh against the bare SH polynomials (the kernels that fill them leave the basis
// constants out, as the forward does): word 11 + 3 k + c is multiplied by the constant of basis function k when the
// record is converted into the caller's gradient record.
__device__ __forceinline__ float sh_word_norm(int word) {   // factor of gradient word `word` (11 <= word < 59)
    return sh_norm((word - 11) / 3);
}

// One thread per slot: convert the accumulated moments (words 0..9) into d mean, d scale, d quat, d opacity and
// write words 0..15 of the Gaussian's gradient record (all 32 lanes busy with the ~300-instruction conversion).
static __global__ void __launch_bounds__(256) bwd_convert_kernel(const float4* __restrict__ qs, const uint32_t* __restrict__ gid_of_slot,
                                                          Gacc gacc, float4* __restrict__ grad4,
                                                          const uint32_t* __restrict__ counts) {
    if (counts[GART_CNT_ERROR]) return;
    constexpr int F4 = GART_GRAD_WORDS / 4;
    const int64_t sid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (sid >= (int64_t)counts[GART_CNT_VISIBLE]) return;
    const float4* gp = reinterpret_cast<const float4*>(gacc.a) + (size_t)sid * (GACC_A_WORDS / 4);
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
    out[2] = make_float4(o.dq[2], o.dq[3], c.y / s4.w, sh_word_norm(11) * c.w);
    out[3] = make_float4(sh_word_norm(12) * d.x, sh_word_norm(13) * d.y, sh_word_norm(14) * d.z, sh_word_norm(15) * d.w);
}

// In the order of the gradient records (sequential writes): 16 lanes per Gaussian; a Gaussian without a slot gets
// a zero record, the others words 16..63 (dL/dsh) of their slot's accumulation record.  A half-warp handles
// FIN_ROWS Gaussians with all their loads in flight at once.
constexpr int FIN_ROWS = 4;
static __global__ void __launch_bounds__(256) bwd_scatter_kernel(int64_t n, const uint32_t* __restrict__ slot_of_gid,
                                                          Gacc gacc, float4* __restrict__ grad4,
                                                          const uint32_t* __restrict__ counts) {
    if (counts[GART_CNT_ERROR]) return;
    constexpr int F4 = GART_GRAD_WORDS / 4;
    const float4* b4 = reinterpret_cast<const float4*>(gacc.b);
    const int64_t hw = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 4;   // half-warp
    const int l = threadIdx.x & 15;
    const int64_t i0 = hw * FIN_ROWS;
    uint32_t s[FIN_ROWS];
#pragma unroll
    for (int r = 0; r < FIN_ROWS; ++r) s[r] = i0 + r < n ? __ldg(slot_of_gid + i0 + r) : 0xffffffffu;
    float4 v[FIN_ROWS];
#pragma unroll
    for (int r = 0; r < FIN_ROWS; ++r)
        v[r] = (s[r] != 0xffffffffu && l >= 4 && l < 15) ? __ldcs(b4 + (size_t)s[r] * (GACC_B_WORDS / 4) + (l - 4)) : make_float4(0.f, 0.f, 0.f, 0.f);
    // basis constants of this lane's four words (lanes 4..14 carry words 16..59; word 59 is padding); chosen while the loads are in flight
    float4 nf = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int q = 4; q < 15; ++q)
        if (l == q) nf = make_float4(sh_word_norm(4 * q), sh_word_norm(4 * q + 1), sh_word_norm(4 * q + 2), 4 * q + 3 < 59 ? sh_word_norm(4 * q + 3) : 0.0f);
#pragma unroll
    for (int r = 0; r < FIN_ROWS; ++r)
        if (i0 + r < n && (l >= 4 || s[r] == 0xffffffffu))
            __stcs(grad4 + (size_t)(i0 + r) * F4 + l, make_float4(nf.x * v[r].x, nf.y * v[r].y, nf.z * v[r].z, nf.w * v[r].w));
}


// Launches shared by the backward variants: zero the accumulation records of the view's slots; after the
// accumulation, convert the moments per slot and write the caller's gradient records.
static inline gart_status launch_zero_accumulators(const Gacc& gacc, int64_t n, const uint32_t* counts, cudaStream_t st) {
    const int64_t zero_blocks = ceil_div(n * ((GACC_A_WORDS + GACC_B_WORDS) / 4), 256);
    bwd_zero_kernel<<<(unsigned)(zero_blocks < 148 * 32 ? zero_blocks : 148 * 32), 256, 0, st>>>(gacc, counts);
    GART_LAUNCH_CHECK();
    return GART_OK;
}
static inline gart_status launch_finalize(int64_t n, const float4* qs, const uint32_t* slot_of_gid, const uint32_t* gid_of_slot,
                                          const Gacc& gacc, float* grad, const uint32_t* counts, cudaStream_t st) {
    bwd_convert_kernel<<<(unsigned)ceil_div(n, 256), 256, 0, st>>>(qs, gid_of_slot, gacc,
                                                                   reinterpret_cast<float4*>(grad), counts);
    GART_LAUNCH_CHECK();
    bwd_scatter_kernel<<<(unsigned)ceil_div(ceil_div(n, FIN_ROWS) * 16, 256), 256, 0, st>>>(n, slot_of_gid, gacc,
                                                                                            reinterpret_cast<float4*>(grad), counts);
    GART_LAUNCH_CHECK();
    return GART_OK;
}

}  // namespace gart
