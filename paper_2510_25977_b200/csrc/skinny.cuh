// Weight-streaming kernels for small token counts (decode): the factored MLP is bound by the
// HBM read of the six factor tensors, each element used once per token.  Weights go to the M
// side of warp-level m16n8k16 bf16 MMAs ("swap-AB": 16 weight rows x 8 tokens per instruction)
// straight from 128-bit global loads, tokens sit on the N side, fp32 accumulators stay in
// registers.  fp32 intermediates (Z, H, Zd) are fed back into the next MMA as an exact
// hi + lo pair of bf16 values, so no intermediate is rounded to 16 bits.
//
// Fragment trick: a lane's 16-byte load holds 8 consecutive k of one weight row.  The dot
// product over k does not care about order, so those 8 values are used as the lane's k-pairs of
// two MMAs (elements 0-1 | 2-3 for the first, 4-5 | 6-7 for the second) and the activation
// fragment is read with the same permutation: both operands come from contiguous 16-byte loads
// and no shared-memory transpose of the weights is needed.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace skinny {

constexpr int kPad = 32;  // bf16 elements added to each shared-memory row (64 B): conflict-free 16 B reads

__device__ __forceinline__ uint4 ldg_stream(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

__device__ __forceinline__ void mma16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ float silu_f32(float g) { return g / (1.0f + __expf(-g)); }

// Shared-memory activation tile: ROWS token rows x (kc + kPad) bf16, hi part and (if SPLIT) lo part.
// Source rows t0 .. t0+ROWS-1 (rows >= T read as zero), columns k0 .. k0+kc-1 (columns >= K zero).
template <int ROWS>
__device__ __forceinline__ void stage_act_bf16(__nv_bfloat16* s_hi, int pitch, const __nv_bfloat16* __restrict__ src,
                                               long ld, int T, int t0, int K, int k0, int kc) {
    const int vec_per_row = kc / 8;
    for (int i = threadIdx.x; i < ROWS * vec_per_row; i += blockDim.x) {
        int tr = i / vec_per_row, kv = (i - tr * vec_per_row) * 8;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (t0 + tr < T && k0 + kv < K) v = *reinterpret_cast<const uint4*>(src + (long)(t0 + tr) * ld + k0 + kv);
        *reinterpret_cast<uint4*>(s_hi + tr * pitch + kv) = v;
    }
}

__device__ __forceinline__ void split_bf16(float v, __nv_bfloat16& hi, __nv_bfloat16& lo) {
    hi = __float2bfloat16_rn(v);
    lo = __float2bfloat16_rn(v - __bfloat162float(hi));
}

template <int ROWS>
__device__ __forceinline__ void stage_act_f32(__nv_bfloat16* s_hi, __nv_bfloat16* s_lo, int pitch,
                                              const float* __restrict__ src, long ld, int T, int t0, int K, int k0,
                                              int kc) {
    const int vec_per_row = kc / 4;
    for (int i = threadIdx.x; i < ROWS * vec_per_row; i += blockDim.x) {
        int tr = i / vec_per_row, kv = (i - tr * vec_per_row) * 4;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (t0 + tr < T && k0 + kv < K) v = *reinterpret_cast<const float4*>(src + (long)(t0 + tr) * ld + k0 + kv);
        __nv_bfloat16 h[4], l[4];
        split_bf16(v.x, h[0], l[0]); split_bf16(v.y, h[1], l[1]);
        split_bf16(v.z, h[2], l[2]); split_bf16(v.w, h[3], l[3]);
        *reinterpret_cast<uint2*>(s_hi + tr * pitch + kv) = *reinterpret_cast<uint2*>(h);
        *reinterpret_cast<uint2*>(s_lo + tr * pitch + kv) = *reinterpret_cast<uint2*>(l);
    }
}

// acc[nt][*] += W[16 rows, kbeg..kend) * act[8*nt tokens, same k]^T for one warp.
// rowA / rowB point at the weight rows of lane group g and g+8 (nullptr = row out of range).
// s_hi/s_lo hold the activations for k starting at ks0 (a multiple of 32 at or below kbeg).
template <int NT, bool SPLIT, int UNROLL>
__device__ __forceinline__ void stream_tile(const __nv_bfloat16* __restrict__ rowA,
                                            const __nv_bfloat16* __restrict__ rowB, int kbeg, int kend, int ks0,
                                            const __nv_bfloat16* s_hi, const __nv_bfloat16* s_lo, int pitch,
                                            float (&acc)[NT][4]) {
    const int lane = threadIdx.x & 31, g = lane >> 2, tig = lane & 3;
    for (int kb = kbeg; kb < kend; kb += 32 * UNROLL) {
        uint4 wa[UNROLL], wb[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            int k = kb + 32 * u + 8 * tig;
            wa[u] = (rowA != nullptr && k < kend) ? ldg_stream(rowA + k) : make_uint4(0, 0, 0, 0);
            wb[u] = (rowB != nullptr && k < kend) ? ldg_stream(rowB + k) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            int k = kb + 32 * u + 8 * tig;
            if (kb + 32 * u < kend) {
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    const int so = (nt * 8 + g) * pitch + (k - ks0);
                    uint4 xh = *reinterpret_cast<const uint4*>(s_hi + so);
                    mma16816(acc[nt], wa[u].x, wb[u].x, wa[u].y, wb[u].y, xh.x, xh.y);
                    mma16816(acc[nt], wa[u].z, wb[u].z, wa[u].w, wb[u].w, xh.z, xh.w);
                    if (SPLIT) {
                        uint4 xl = *reinterpret_cast<const uint4*>(s_lo + so);
                        mma16816(acc[nt], wa[u].x, wb[u].x, wa[u].y, wb[u].y, xl.x, xl.y);
                        mma16816(acc[nt], wa[u].z, wb[u].z, wa[u].w, wb[u].w, xl.z, xl.w);
                    }
                }
            }
        }
    }
}

__device__ __forceinline__ void zero_region(float* p, long n) {
    if (p == nullptr) return;
    long nblk = (long)gridDim.x * gridDim.y * gridDim.z;
    long bid = ((long)blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x;
    for (long i = (bid * blockDim.x + threadIdx.x) * 4; i < n; i += nblk * blockDim.x * 4) {
        if (i + 4 <= n) *reinterpret_cast<float4*>(p + i) = make_float4(0.f, 0.f, 0.f, 0.f);
        else for (long j = i; j < n; ++j) p[j] = 0.f;
    }
}

// ---- stage 1:  Z[T, ra+rb] += X[T, K] * [Va; Vb]^T   (phase 1 of Algorithm 3 for both branches) ----
// grid (row groups of 4 tiles, K splits of kc, token chunks of 8*NT); 128 threads.
// Z is accumulated with fp32 reductions across K splits and must be zero on entry.
// Also clears `zero_ptr[0 .. zero_n)` (the accumulator of a later stage).
template <int NT>
__global__ void __launch_bounds__(128)
stage1_kernel(const __nv_bfloat16* __restrict__ X, long ldx, int T, int K, const __nv_bfloat16* __restrict__ Va, int ra,
              const __nv_bfloat16* __restrict__ Vb, int rb, float* __restrict__ Z, int kc, float* zero_ptr,
              long zero_n) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __nv_bfloat16* s_x = reinterpret_cast<__nv_bfloat16*>(smem_raw);
    const int pitch = kc + kPad;
    const int t0 = blockIdx.z * NT * 8, k0 = blockIdx.y * kc;
    zero_region(zero_ptr, zero_n);
    stage_act_bf16<NT * 8>(s_x, pitch, X, ldx, T, t0, K, k0, kc);
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, tig = lane & 3;
    const int R = ra + rb;
    const int row0 = (blockIdx.x * 4 + warp) * 16;
    if (row0 >= R) return;
    auto rowptr = [&](int r) -> const __nv_bfloat16* {
        if (r >= R) return nullptr;
        return r < ra ? Va + (long)r * K : Vb + (long)(r - ra) * K;
    };
    float acc[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
    const int kend = min(K, k0 + kc);
    stream_tile<NT, false, 8>(rowptr(row0 + g), rowptr(row0 + g + 8), k0, kend, k0, s_x, nullptr, pitch, acc);
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            int r = row0 + g + (c >> 1) * 8, t = t0 + nt * 8 + 2 * tig + (c & 1);
            if (r < R && t < T) atomicAdd(Z + (long)t * R + r, acc[nt][c]);
        }
    }
}

// ---- stages 2-4 fused:  H[:, j0..j0+64) = SiLU(Zg Ug^T) .* (Zu Uu^T);  Zd += H Vd[:, j0..j0+64)^T ----
// (phase 2 of Algorithm 3 with its SiLU epilogue, then phase 1 of the down-projection XUV chain,
//  split over ffn so that H never leaves the SM).  grid (ceil(ffn/64), 1, token chunks); 256 threads.
// Z is [T, rg+ru] fp32 (gate columns first).  Zd[T, rd] fp32 is reduced across blocks: zero on entry.
template <int NT>
__global__ void __launch_bounds__(256)
gateup_down1_kernel(const float* __restrict__ Z, int T, int rg, int ru, const __nv_bfloat16* __restrict__ Ug,
                    const __nv_bfloat16* __restrict__ Uu, int ffn, const __nv_bfloat16* __restrict__ Vd, int rd,
                    float* __restrict__ Zd) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    constexpr int ROWS = NT * 8, JS = 64;
    const int pg = rg + kPad, pu = ru + kPad, ph = JS + kPad;
    __nv_bfloat16* zg_hi = reinterpret_cast<__nv_bfloat16*>(smem_raw);
    __nv_bfloat16* zg_lo = zg_hi + ROWS * pg;
    __nv_bfloat16* zu_hi = zg_lo + ROWS * pg;
    __nv_bfloat16* zu_lo = zu_hi + ROWS * pu;
    __nv_bfloat16* h_hi = zu_lo + ROWS * pu;
    __nv_bfloat16* h_lo = h_hi + ROWS * ph;
    float* gs = reinterpret_cast<float*>(h_lo + ROWS * ph);  // [ROWS][JS + 1]
    const int t0 = blockIdx.z * ROWS, j0 = blockIdx.x * JS;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, tig = lane & 3;
    const int rg32 = (rg + 31) & ~31, ru32 = (ru + 31) & ~31;

    stage_act_f32<ROWS>(zg_hi, zg_lo, pg, Z, rg + ru, T, t0, rg, 0, rg32);
    stage_act_f32<ROWS>(zu_hi, zu_lo, pu, Z + rg, rg + ru, T, t0, ru, 0, ru32);
    __syncthreads();

    float acc[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
    {
        const bool is_up = warp >= 4;
        const int jr = j0 + (warp & 3) * 16;
        const __nv_bfloat16* Wm = is_up ? Uu : Ug;
        const int r = is_up ? ru : rg;
        const __nv_bfloat16* rowA = (jr + g < ffn) ? Wm + (long)(jr + g) * r : nullptr;
        const __nv_bfloat16* rowB = (jr + g + 8 < ffn) ? Wm + (long)(jr + g + 8) * r : nullptr;
        if (is_up) stream_tile<NT, true, 8>(rowA, rowB, 0, r, 0, zu_hi, zu_lo, pu, acc);
        else       stream_tile<NT, true, 8>(rowA, rowB, 0, r, 0, zg_hi, zg_lo, pg, acc);
    }
    const int jl = (warp & 3) * 16 + g;  // local j of c0/c1 (c2/c3: +8)
    if (warp < 4) {
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int c = 0; c < 4; ++c)
                gs[(nt * 8 + 2 * tig + (c & 1)) * (JS + 1) + jl + (c >> 1) * 8] = acc[nt][c];
    }
    __syncthreads();
    if (warp >= 4) {
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                int tr = nt * 8 + 2 * tig + (c & 1), jj = jl + (c >> 1) * 8;
                float hval = silu_f32(gs[tr * (JS + 1) + jj]) * acc[nt][c];
                __nv_bfloat16 hi, lo;
                split_bf16(hval, hi, lo);
                h_hi[tr * ph + jj] = hi;
                h_lo[tr * ph + jj] = lo;
            }
    }
    __syncthreads();
    const int jend = min(ffn, j0 + JS);
    for (int tile = warp; tile * 16 < rd; tile += 8) {
        const int i0 = tile * 16;
        const __nv_bfloat16* rowA = (i0 + g < rd) ? Vd + (long)(i0 + g) * ffn : nullptr;
        const __nv_bfloat16* rowB = (i0 + g + 8 < rd) ? Vd + (long)(i0 + g + 8) * ffn : nullptr;
        float a2[NT][4];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) a2[nt][0] = a2[nt][1] = a2[nt][2] = a2[nt][3] = 0.f;
        stream_tile<NT, true, 2>(rowA, rowB, j0, jend, j0, h_hi, h_lo, ph, a2);
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                int i = i0 + g + (c >> 1) * 8, t = t0 + nt * 8 + 2 * tig + (c & 1);
                if (i < rd && t < T) atomicAdd(Zd + (long)t * rd + i, a2[nt][c]);
            }
    }
}

// ---- last stage:  Y[T, N] = A[T, r] * U[N, r]^T  (+ residual) with fp32 A (phase 2 of the XUV chain) ----
// grid (ceil(N/64), 1, token chunks); 128 threads, one 16-row tile of U per warp.
// Output: bf16 or fp32; if `resid` != nullptr the fp32 output is resid + product.
// Also clears zero_ptr[0..zero_n) (the stage-1 accumulator for the next call).
template <int NT>
__global__ void __launch_bounds__(128)
expand_kernel(const float* __restrict__ A, int T, int r, const __nv_bfloat16* __restrict__ U, int N, void* Yout,
              int y_fp32, const float* __restrict__ resid, float* zero_ptr, long zero_n) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    constexpr int ROWS = NT * 8;
    const int pitch = r + kPad, r32 = (r + 31) & ~31;
    __nv_bfloat16* a_hi = reinterpret_cast<__nv_bfloat16*>(smem_raw);
    __nv_bfloat16* a_lo = a_hi + ROWS * pitch;
    const int t0 = blockIdx.z * ROWS;
    stage_act_f32<ROWS>(a_hi, a_lo, pitch, A, r, T, t0, r, 0, r32);
    __syncthreads();
    zero_region(zero_ptr, zero_n);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, tig = lane & 3;
    const int c0 = (blockIdx.x * 4 + warp) * 16;
    if (c0 >= N) return;
    const __nv_bfloat16* rowA = (c0 + g < N) ? U + (long)(c0 + g) * r : nullptr;
    const __nv_bfloat16* rowB = (c0 + g + 8 < N) ? U + (long)(c0 + g + 8) * r : nullptr;
    float acc[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
    stream_tile<NT, true, 8>(rowA, rowB, 0, r, 0, a_hi, a_lo, pitch, acc);
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            int col = c0 + g + (c >> 1) * 8, t = t0 + nt * 8 + 2 * tig + (c & 1);
            if (col < N && t < T) {
                float v = acc[nt][c];
                long o = (long)t * N + col;
                if (resid != nullptr) v += resid[o];
                if (y_fp32) reinterpret_cast<float*>(Yout)[o] = v;
                else reinterpret_cast<__nv_bfloat16*>(Yout)[o] = __float2bfloat16_rn(v);
            }
        }
}

// RMSNorm with unit weight, fp32 in, bf16 out: one block per token row.  Rows of up to 8192 elements are held in
// registers (all loads issued before the first use, one pass over memory); longer rows are read twice.
// Launched with programmatic stream serialization: the row is only read after the preceding kernel has finished.
__global__ void __launch_bounds__(256)
rmsnorm_kernel(const float* __restrict__ h, int d, float eps, __nv_bfloat16* __restrict__ out) {
    __shared__ float red[8];
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const float* row = h + (long)blockIdx.x * d;
    __nv_bfloat16* o = out + (long)blockIdx.x * d;
    const bool in_regs = d <= 8 * 256 * 4;
    float4 v[8];
    float ss = 0.f;
    if (in_regs) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int i = (j * 256 + threadIdx.x) * 4;
            v[j] = (i < d) ? *reinterpret_cast<const float4*>(row + i) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) ss += v[j].x * v[j].x + v[j].y * v[j].y + v[j].z * v[j].z + v[j].w * v[j].w;
    } else {
        for (int i = threadIdx.x * 4; i < d; i += blockDim.x * 4) {
            const float4 w = *reinterpret_cast<const float4*>(row + i);
            ss += w.x * w.x + w.y * w.y + w.z * w.z + w.w * w.w;
        }
    }
    for (int off = 16; off > 0; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
    for (int w = 0; w < 8; ++w) tot += red[w];
    const float inv = rsqrtf(tot / (float)d + eps);
    auto emit = [&](int i, const float4& w) {
        __nv_bfloat162 a = __floats2bfloat162_rn(w.x * inv, w.y * inv), b = __floats2bfloat162_rn(w.z * inv, w.w * inv);
        uint2 pk;
        pk.x = *reinterpret_cast<uint32_t*>(&a);
        pk.y = *reinterpret_cast<uint32_t*>(&b);
        *reinterpret_cast<uint2*>(o + i) = pk;
    };
    if (in_regs) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int i = (j * 256 + threadIdx.x) * 4;
            if (i < d) emit(i, v[j]);
        }
    } else {
        for (int i = threadIdx.x * 4; i < d; i += blockDim.x * 4) emit(i, *reinterpret_cast<const float4*>(row + i));
    }
}

}  // namespace skinny
