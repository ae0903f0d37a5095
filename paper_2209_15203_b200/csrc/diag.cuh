// Per-iteration estimate of the gap constants of the convergence analysis (the quantities
// of the paper's Table 1): with a^q the vector worker q compresses, D_a = sum_q p_q a^q,
// D_g = sum_q p_q g^q and S = sum_q p_q Top_K(a^q),
//   unidirectional  rho_hat = || Top_K(D_a) - S ||                         / || scale D_g ||
//   bidirectional   rho     = || Top_K(delta + D_a) - Top_K(delta + S) ||  / || scale D_g ||
// The dense sums are what the method itself never forms — this is a diagnostic that reads
// the gradients a second time and runs one more dense selection; it is off unless asked for.
#pragma once

#include "common.cuh"

namespace tk {

// Da[j] = (delta[j] +) sum_q p_q a_q[j],  a_q = eps_q + alpha g_q (or g_q without memories);
// sums[0] += sum_j (scale * sum_q p_q g_q[j])^2.  fp32, worker order, one rounding per operation.
__global__ void __launch_bounds__(256)
dense_sums_kernel(const float* __restrict__ G, const float* __restrict__ eps, const float* __restrict__ delta,
                  const float* __restrict__ p, int N, size_t d, float alpha, float scale, float* Da, double* sums) {
    double den = 0.0;
    for (size_t j = (size_t)blockIdx.x * blockDim.x + threadIdx.x; j < d; j += (size_t)gridDim.x * blockDim.x) {
        float sa = 0.0f, sg = 0.0f;
        for (int q = 0; q < N; ++q) {
            float g = __ldg(G + (size_t)q * d + j);
            float a = eps ? __fadd_rn(__ldg(eps + (size_t)q * d + j), __fmul_rn(alpha, g)) : g;
            sa = __fadd_rn(sa, __fmul_rn(p[q], a));
            sg = __fadd_rn(sg, __fmul_rn(p[q], g));
        }
        if (delta) sa = __fadd_rn(delta[j], sa);
        Da[j] = sa;
        double v = (double)scale * (double)sg;
        den += v * v;
    }
    warp_add_double(&sums[0], den);
}

// Z[idx] += sign * value for the first min(*count, cap) entries of a list (count may be NULL:
// then all `cap` entries).  Indices within one list are distinct.
__global__ void __launch_bounds__(256)
diff_scatter_kernel(const uint2* __restrict__ list, const u32* count, u32 cap, float sign, float* Z, u32 d) {
    u32 n = count ? min(*count, cap) : cap;
    u32 i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    uint2 e = list[i];
    if (e.x < d) Z[e.x] = __fadd_rn(Z[e.x], __fmul_rn(sign, __uint_as_float(e.y)));
}

// sums[1] += sum over the list's entries of Z[idx]^2, and Z[idx] <- 0 (so that an index
// present in two lists is counted once and Z is all zero again afterwards).
__global__ void __launch_bounds__(256)
diff_norm_kernel(const uint2* __restrict__ list, const u32* count, u32 cap, float* Z, u32 d, double* sums) {
    u32 n = count ? min(*count, cap) : cap;
    u32 i = blockIdx.x * blockDim.x + threadIdx.x;
    double v = 0.0;
    if (i < n) {
        u32 j = list[i].x;
        if (j < d) {
            double z = (double)Z[j];
            v = z * z;
            Z[j] = 0.0f;
        }
    }
    warp_add_double(&sums[1], v);
}

}  // namespace tk
