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

}  // namespace gart
