// Compression front-end on the device (Section 4.1 with S = I: Eq. 3 is then the plain SVD; Eq. 6-8 fold the
// singular values into the factors): rank-r factors U[out, r], V[r, in] of a dense weight W[out, in].
//
// One-sided (Hestenes) Jacobi in fp32 with fp64 dot products.  The vectors that are made orthogonal are the
// rows of a work matrix B[n, m], n <= m: B = W^T (rows = columns of W) when in <= out, B = W otherwise, so a
// vector is always contiguous.  A sweep is n - 1 steps of n / 2 disjoint pairs (round-robin pairing), one CTA
// per pair, one kernel launch per step; the same rotations are applied to the rows of R[n, n] (identity at the
// start).  At convergence row j of B is sigma_j times a singular vector of the long side and row j of R the
// matching singular vector of the short side.  This is an offline step (seconds for a 4096 x 11008 matrix):
// bandwidth per step is what a pass over B costs, nothing here is tuned beyond coalescing.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace compress {

constexpr int kThreads = 256;

// B[j, i] = W[i, j] (transpose = 1: B is n = in rows of length m = out) or a copy of W; R = identity.
__global__ void __launch_bounds__(kThreads)
init_kernel(const float* __restrict__ W, int out, int in, int transpose, int n, int m, float* __restrict__ B, float* __restrict__ R) {
    const long total = (long)n * m;
    for (long idx = (long)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (long)gridDim.x * blockDim.x) {
        const int j = (int)(idx / m), i = (int)(idx - (long)j * m);
        B[idx] = transpose ? W[(long)i * in + j] : W[idx];
    }
    for (long idx = (long)blockIdx.x * blockDim.x + threadIdx.x; idx < (long)n * n; idx += (long)gridDim.x * blockDim.x)
        R[idx] = (idx / n == idx % n) ? 1.f : 0.f;
}

__device__ __forceinline__ double block_sum(double v, double* sh) {
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
    __syncthreads();
    if (l == 0) sh[w] = v;
    __syncthreads();
    double t = 0.0;
    for (int i = 0; i < kThreads / 32; ++i) t += sh[i];
    return t;
}

// Step k of a sweep: CTA c rotates the pair (p, q) of the round-robin schedule so that rows p and q of B become
// orthogonal.  n_even = n rounded up to even; an index >= n is the bye.  *rotated counts the pairs that were not
// yet orthogonal to within tol.
__global__ void __launch_bounds__(kThreads)
step_kernel(float* __restrict__ B, float* __restrict__ R, int n, int m, int n_even, int k, double tol, int* __restrict__ rotated) {
    __shared__ double sh[kThreads / 32];
    const int c = blockIdx.x, ring = n_even - 1;
    int p, q;
    if (c == 0) { p = ring; q = k % ring; }
    else { p = (k + c) % ring; q = (k - c + ring) % ring; }
    if (p >= n || q >= n) return;
    if (p > q) { const int t = p; p = q; q = t; }
    float* bp = B + (long)p * m;
    float* bq = B + (long)q * m;
    double a = 0.0, b = 0.0, g = 0.0;
    for (int i = threadIdx.x; i < m; i += kThreads) {
        const double x = bp[i], y = bq[i];
        a += x * x; b += y * y; g += x * y;
    }
    a = block_sum(a, sh); b = block_sum(b, sh); g = block_sum(g, sh);
    if (fabs(g) <= tol * sqrt(a * b) || g == 0.0) return;   // uniform across the CTA
    if (threadIdx.x == 0) atomicAdd(rotated, 1);
    const double zeta = (b - a) / (2.0 * g);
    const double t = (zeta >= 0.0 ? 1.0 : -1.0) / (fabs(zeta) + sqrt(1.0 + zeta * zeta));
    const double cs = 1.0 / sqrt(1.0 + t * t), sn = cs * t;
    const float cf = (float)cs, sf = (float)sn;
    for (int i = threadIdx.x; i < m; i += kThreads) {
        const float x = bp[i], y = bq[i];
        bp[i] = cf * x - sf * y;
        bq[i] = sf * x + cf * y;
    }
    float* rp = R + (long)p * n;
    float* rq = R + (long)q * n;
    for (int i = threadIdx.x; i < n; i += kThreads) {
        const float x = rp[i], y = rq[i];
        rp[i] = cf * x - sf * y;
        rq[i] = sf * x + cf * y;
    }
}

// sigma[j] = |row j of B|
__global__ void __launch_bounds__(kThreads)
norms_kernel(const float* __restrict__ B, int n, int m, float* __restrict__ sigma) {
    __shared__ double sh[kThreads / 32];
    const float* b = B + (long)blockIdx.x * m;
    double a = 0.0;
    for (int i = threadIdx.x; i < m; i += kThreads) { const double x = b[i]; a += x * x; }
    a = block_sum(a, sh);
    if (threadIdx.x == 0) sigma[blockIdx.x] = (float)sqrt(a);
}

// Factors of the r largest singular values; order[k] = row of B / R holding the k-th largest.
//   transpose (in <= out): row j of B = sigma_j u_j (length out), row j of R = v_j (length in)
//   otherwise:             row j of B = sigma_j v_j (length in),  row j of R = u_j (length out)
// split = 0: U diag(sigma) and V (the storage of benchmark configuration 1); split = 1: sqrt(sigma) in both (Eq. 6-7).
__global__ void __launch_bounds__(kThreads)
emit_kernel(const float* __restrict__ B, const float* __restrict__ R, const float* __restrict__ sigma, const int* __restrict__ order,
            int out, int in, int r, int transpose, int n, int m, int split, __nv_bfloat16* __restrict__ U, __nv_bfloat16* __restrict__ V) {
    const long nu = (long)out * r, nv = (long)r * in;
    for (long idx = (long)blockIdx.x * blockDim.x + threadIdx.x; idx < nu + nv; idx += (long)gridDim.x * blockDim.x) {
        if (idx < nu) {   // U[i, k]
            const int i = (int)(idx / r), k = (int)(idx - (long)i * r), j = order[k];
            const float s = sigma[j];
            const float su = split ? sqrtf(s) : s;             // weight of u_k
            float v;
            if (transpose) v = s > 0.f ? B[(long)j * m + i] * (su / s) : 0.f;
            else v = R[(long)j * n + i] * su;
            U[idx] = __float2bfloat16_rn(v);
        } else {          // V[k, c]
            const long e = idx - nu;
            const int k = (int)(e / in), c = (int)(e - (long)k * in), j = order[k];
            const float s = sigma[j];
            const float sv = split ? sqrtf(s) : 1.f;           // weight of v_k
            float v;
            if (transpose) v = R[(long)j * n + c] * sv;
            else v = s > 0.f ? B[(long)j * m + c] * (sv / s) : 0.f;
            V[e] = __float2bfloat16_rn(v);
        }
    }
}

}  // namespace compress
