// Persistent, warp-specialised tcgen05 GEMM for the large-T path:
//     C[M, N] = A[M, K] * B[N, K]^T      (both operands K-major 16-bit, fp32 accumulate in TMEM)
// with the variants the factored MLP needs:
//   NB = 2      two B operands (gate and up factors) with their own A (Zg, Zu) accumulate into two
//               TMEM tiles and the epilogue writes SiLU(G) .* Up  (Algorithm 3, phase 2 + epilogue)
//   ARES        the A row strip [128, K] stays resident in shared memory while the CTA walks the
//               N tiles of that strip (the narrow-intermediate strip cache of Section 4.2.1:
//               the second GEMM of a chain has K = r, so the whole strip fits on chip)
//   batch       independent problems in one launch (gate and up halves of the first projection)
//   ksplit      split-K with fp32 partial outputs (long-K, narrow-N first GEMM of the down chain)
// Roles: warp 0 = TMA producer (one lane), warp 1 = MMA issuer (one lane) + TMEM owner,
// warps 2-9 = epilogue (TMEM -> registers -> swizzled shared memory -> TMA store for 16-bit outputs,
// direct global stores for fp32 outputs).  Accumulators are double-buffered in TMEM
// whenever 2 * NB * BN <= 512 columns so the epilogue of tile i overlaps the MMAs of tile i+1.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "umma.cuh"

namespace tensorpath {

constexpr int BM = 128, BK = 64;
constexpr int kABytes = BM * BK * 2;  // one [128 x 64] 16-bit operand chunk
constexpr int kMaxStages = 12;
constexpr int kThreads = 320;  // TMA warp, MMA warp, 8 epilogue warps (two per TMEM lane quadrant)
constexpr int kPairThreads = 384;  // the CTA-pair kernel adds warp 10 (second MMA issuer when it runs two branches) and warp 11 (second TMA producer)
constexpr int kPairProducer2 = 11;
constexpr int kEpiWarps = 8;
constexpr int kErrTimeout = -7;

enum OutMode { OUT_F16 = 0, OUT_BF16 = 1, OUT_F32 = 2 };

struct GemmParams {
    CUtensorMap tmA[2];  // NB == 2: per branch; NB == 1: per batch entry
    CUtensorMap tmB[2];
    CUtensorMap tmC;     // output map for the TMA-store epilogue (box [32 rows, 64 columns], 16-bit)
    int c_tma;           // 1: 16-bit output goes through shared memory and TMA stores
    int M, N, K;
    int tiles_m, tiles_n, batch, ksplit;
    int chunks_total, chunks_per_split;  // K chunks of 64
    void* C;
    long ldc;            // elements
    long split_stride;   // elements between split-K partial outputs
    long batch_col_off;  // output column offset per batch entry
    int out_mode;
    int stages;
    int cps;             // K chunks per ring slot of the streaming CTA-pair kernel (0 or 1: one)
    int a_fmt, b_fmt;    // umma::kFmtF16 / kFmtBF16
    const float* resid;  // optional fp32 [M, ldc] added to an OUT_F32 result (residual connection)
    int* status;         // device status word (written on timeout)
    // Layout flags of the XUV operator (Algorithm 2's is_XT / req_OT); streaming one-branch kernels only.
    int a_mn;            // 1: A is given transposed, A^T[K, M]: tmA has boxes [64 k][64 m], the tile is an MN-major operand
    int c_t;             // 1: the 16-bit TMA-store epilogue writes C^T[N, M]: tmC has boxes [64 n][32 m], no swizzle
    // Split-K inside a cluster (streaming one-branch CTA-pair kernel only): the cluster is cks CTA pairs, pair s takes
    // K split s of the cluster's one tile, and the partial accumulators are summed through distributed shared memory
    // (no partial buffer, no reduction launch).  0 or 1: off.
    int cks;
};

__device__ __forceinline__ float fast_silu(float g) {
    // SiLU(g) = g * sigmoid(g) = 0.5 g (1 + tanh(g / 2)): one MUFU op per element
    float t;
    asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(0.5f * g));
    return 0.5f * g * (1.0f + t);
}

// Two SiLU(g) * u products rounded to fp16: 0.5 g (1 + tanh(g / 2)) u = w + w t with w = 0.5 g u. The tanh runs
// on the packed half-precision unit (one MUFU op per two elements, the same 2^-11 accuracy class as the fp32
// approximation), w is formed in fp32 and rounded once, and one packed FMA finishes both elements.
__device__ __forceinline__ uint32_t silu_mul_pack_f16(float g0, float g1, float u0, float u1) {
    const float h0 = 0.5f * g0, h1 = 0.5f * g1;
    const __half2 a = __floats2half2_rn(h0, h1);
    uint32_t t;
    asm("tanh.approx.f16x2 %0, %1;" : "=r"(t) : "r"(*reinterpret_cast<const uint32_t*>(&a)));
    const __half2 w = __floats2half2_rn(h0 * u0, h1 * u1);
    const __half2 r = __hfma2(w, *reinterpret_cast<const __half2*>(&t), w);
    return *reinterpret_cast<const uint32_t*>(&r);
}

__device__ __forceinline__ uint32_t pack_f16(float a, float b) {
    __half2 h = __floats2half2_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
    __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&h);
}

// Store 32 consecutive fp32 values of one output row (predicated on the column bound).
__device__ __forceinline__ void store_row32(const GemmParams& p, char* rowbase, long col, int ncols_valid,
                                            const float (&v)[32]) {
    if (p.out_mode == OUT_F32) {
        float* o = reinterpret_cast<float*>(rowbase) + col;
#pragma unroll
        for (int j = 0; j < 32; j += 4)
            if (j + 4 <= ncols_valid) *reinterpret_cast<float4*>(o + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
    } else {
        uint16_t* o = reinterpret_cast<uint16_t*>(rowbase) + col;
#pragma unroll
        for (int j = 0; j < 32; j += 8) {
            if (j + 8 <= ncols_valid) {
                uint4 w;
                if (p.out_mode == OUT_F16) {
                    w.x = pack_f16(v[j], v[j + 1]); w.y = pack_f16(v[j + 2], v[j + 3]);
                    w.z = pack_f16(v[j + 4], v[j + 5]); w.w = pack_f16(v[j + 6], v[j + 7]);
                } else {
                    w.x = pack_bf16(v[j], v[j + 1]); w.y = pack_bf16(v[j + 2], v[j + 3]);
                    w.z = pack_bf16(v[j + 4], v[j + 5]); w.w = pack_bf16(v[j + 6], v[j + 7]);
                }
                *reinterpret_cast<uint4*>(o + j) = w;
            }
        }
    }
}

struct TileCoord { int m, n, z, ks; };

template <bool ARES>
__device__ __forceinline__ TileCoord decode_tile(const GemmParams& p, int t) {
    TileCoord c;
    if (ARES) { c.m = t / p.tiles_n; c.n = t - c.m * p.tiles_n; c.z = 0; c.ks = 0; }
    else {
        c.n = t % p.tiles_n; t /= p.tiles_n;
        c.m = t % p.tiles_m; t /= p.tiles_m;
        c.ks = t % p.ksplit; c.z = t / p.ksplit;
    }
    return c;
}

template <int NB, int BN, bool ARES>
__global__ void __launch_bounds__(kThreads, 1) gemm_kernel(const __grid_constant__ GemmParams p) {
    constexpr int B_BYTES = BN * BK * 2;
    constexpr int ACC_COLS = NB * BN;
    constexpr int NUM_ACC = (2 * ACC_COLS <= 512) ? 2 : 1;
    constexpr int TMEM_COLS = (NUM_ACC * ACC_COLS <= 32) ? 32 : (NUM_ACC * ACC_COLS <= 64) ? 64 :
                              (NUM_ACC * ACC_COLS <= 128) ? 128 : (NUM_ACC * ACC_COLS <= 256) ? 256 : 512;
    static_assert(ACC_COLS <= 512, "accumulators exceed TMEM");
    // Ring slot: with a resident A strip one slot holds one branch's B chunk (gate and up chunks
    // alternate, so many small slots are in flight); otherwise a slot holds all operands of a chunk.
    constexpr int SLOT_BYTES = ARES ? B_BYTES : NB * (kABytes + B_BYTES);
    constexpr int SLOTS_PER_CHUNK = ARES ? NB : 1;

    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = smem_raw + ((1024u - (umma::smem_u32(smem_raw) & 1023u)) & 1023u);  // 1024-byte aligned in the shared window
    const int a_chunks = p.chunks_total;
    unsigned char* a_res = smem;
    unsigned char* ring = smem + (ARES ? NB * a_chunks * kABytes : 0);
    unsigned char* stage_out = ring + p.stages * SLOT_BYTES;  // one 4 KiB staging tile per epilogue warp (TMA-store path)
    uint64_t* bars = reinterpret_cast<uint64_t*>(stage_out + (p.c_tma ? kEpiWarps * 4096 : 0));
    uint64_t* full = bars;
    uint64_t* empty = bars + kMaxStages;
    uint64_t* tfull = bars + 2 * kMaxStages;
    uint64_t* tempty = tfull + 2;
    uint64_t* afull = tempty + 2;
    uint64_t* aempty = afull + 1;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(aempty + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int total_tiles = p.tiles_m * p.tiles_n * p.batch * p.ksplit;
    const int per_cta = (total_tiles + gridDim.x - 1) / gridDim.x;
    const int tile_begin = blockIdx.x * per_cta;
    const int tile_end = min(total_tiles, tile_begin + per_cta);

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) { umma::mbar_init(&full[s], 1); umma::mbar_init(&empty[s], 1); }
        for (int a = 0; a < 2; ++a) { umma::mbar_init(&tfull[a], 1); umma::mbar_init(&tempty[a], kEpiWarps); }
        umma::mbar_init(afull, 1);
        umma::mbar_init(aempty, 1);
        *abort_flag = 0;
        umma::fence_mbar_init();
        umma::prefetch_tmap(&p.tmA[0]); umma::prefetch_tmap(&p.tmB[0]);
        if (NB == 2 || p.batch == 2) { umma::prefetch_tmap(&p.tmA[1]); umma::prefetch_tmap(&p.tmB[1]); }
        if (p.c_tma) umma::prefetch_tmap(&p.tmC);
    }
    if (warp == 1) { umma::tmem_alloc(tmem_slot, TMEM_COLS); umma::tmem_relinquish(); }
    umma::tc_fence_before_sync();
    __syncthreads();
    umma::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    // Programmatic dependent launch: everything above overlapped the previous kernel's tail; its
    // results (our A operand, and buffers we overwrite) may only be touched after this wait.
    umma::pdl_launch_dependents();
    // The B operands are weights, which no earlier kernel writes: the first tile's chunks are requested into L2
    // before this grid waits for its predecessor, so their first (HBM) touch overlaps the predecessor's tail.
    if (warp == 0 && lane == 0 && tile_begin < tile_end) {
        const TileCoord tc = decode_tile<ARES>(p, tile_begin);
        const int c_begin = tc.ks * p.chunks_per_split, c_end = min(p.chunks_total, c_begin + min(p.chunks_per_split, 16));
        for (int b = 0; b < NB; ++b)
            for (int c = c_begin; c < c_end; ++c)
                umma::tma_prefetch_2d(&p.tmB[NB == 2 ? b : tc.z], c * BK, tc.n * BN);
    }
    umma::pdl_wait();

    if (warp == 0) {
        {  // ---------------- TMA producer: the warp walks the tiles together, one elected lane issues ----------------
            int stage = 0, cur_m = -1;
            uint32_t phase = 0, a_phase = 0;
            bool ok = true;
            for (int t = tile_begin; t < tile_end && ok; ++t) {
                const TileCoord tc = decode_tile<ARES>(p, t);
                if (ARES && tc.m != cur_m) {
                    if (cur_m >= 0) { ok = umma::mbar_wait_warp(aempty, a_phase, abort_flag); a_phase ^= 1; if (!ok) break; }
                    if (umma::elect_one()) {
                        umma::mbar_expect_tx(afull, NB * a_chunks * kABytes);
                        for (int b = 0; b < NB; ++b)
                            for (int c = 0; c < a_chunks; ++c)
                                umma::tma_load_2d(a_res + (b * a_chunks + c) * kABytes, &p.tmA[b], afull, c * BK, tc.m * BM);
                    }
                    __syncwarp();
                    cur_m = tc.m;
                }
                const int c_begin = tc.ks * p.chunks_per_split;
                const int c_end = min(p.chunks_total, c_begin + p.chunks_per_split);
                for (int c = c_begin; c < c_end && ok; ++c) {
                    for (int sl = 0; sl < SLOTS_PER_CHUNK; ++sl) {
                        ok = umma::mbar_wait_warp(&empty[stage], phase ^ 1, abort_flag);
                        if (!ok) break;
                        if (umma::elect_one()) {
                            umma::mbar_expect_tx(&full[stage], SLOT_BYTES);
                            unsigned char* st = ring + stage * SLOT_BYTES;
                            if (ARES) {
                                umma::tma_load_2d(st, &p.tmB[NB == 2 ? sl : tc.z], &full[stage], c * BK, tc.n * BN);
                            } else {
                                for (int b = 0; b < NB; ++b) {
                                    if (p.a_mn) {  // two boxes [64 k][64 m] of A^T
                                        umma::tma_load_2d(st + b * kABytes, &p.tmA[NB == 2 ? b : tc.z], &full[stage], tc.m * BM, c * BK);
                                        umma::tma_load_2d(st + b * kABytes + kABytes / 2, &p.tmA[NB == 2 ? b : tc.z], &full[stage], tc.m * BM + 64, c * BK);
                                    } else {
                                        umma::tma_load_2d(st + b * kABytes, &p.tmA[NB == 2 ? b : tc.z], &full[stage], c * BK, tc.m * BM);
                                    }
                                }
                                for (int b = 0; b < NB; ++b)
                                    umma::tma_load_2d(st + NB * kABytes + b * B_BYTES, &p.tmB[NB == 2 ? b : tc.z],
                                                      &full[stage], c * BK, tc.n * BN);
                            }
                        }
                        __syncwarp();
                        if (++stage == p.stages) { stage = 0; phase ^= 1; }
                    }
                }
            }
        }
    } else if (warp == 1) {
        {  // ---------------- MMA issuer: warp-uniform waits, one elected lane issues ----------------
            const uint32_t idesc = umma::make_idesc(p.a_fmt, p.b_fmt, BM, BN) | (p.a_mn ? umma::kIdescAMnMajor : 0u);
            const uint64_t a_step = p.a_mn ? 128 : 2;  // descriptor units of 16 B per K = 16: two 8-k groups, or 32 B inside the swizzle atom
            int stage = 0, cur_m = -1, acc = 0;
            uint32_t phase = 0, a_phase = 0, acc_phase0 = 0, acc_phase1 = 0;
            bool ok = true;
            for (int t = tile_begin; t < tile_end && ok; ++t) {
                const TileCoord tc = decode_tile<ARES>(p, t);
                ok = umma::mbar_wait_warp(&tempty[acc], (acc ? acc_phase1 : acc_phase0) ^ 1, abort_flag);
                if (!ok) break;
                if (ARES && tc.m != cur_m) {
                    ok = umma::mbar_wait_warp(afull, a_phase, abort_flag);
                    a_phase ^= 1; cur_m = tc.m;
                    if (!ok) break;
                }
                umma::tc_fence_after_sync();
                const int c_begin = tc.ks * p.chunks_per_split;
                const int c_end = min(p.chunks_total, c_begin + p.chunks_per_split);
                for (int c = c_begin; c < c_end && ok; ++c) {
                    for (int sl = 0; sl < SLOTS_PER_CHUNK; ++sl) {
                        ok = umma::mbar_wait_warp(&full[stage], phase, abort_flag);
                        if (!ok) break;
                        umma::tc_fence_after_sync();
                        unsigned char* st = ring + stage * SLOT_BYTES;
                        if (umma::elect_one()) {
                            // Descriptors step by 32 bytes (2 in units of 16) along K inside the swizzle atom;
                            // shared memory is below 256 KiB, so the 14-bit address field never carries.
                            const uint32_t dcol = tmem_base + acc * ACC_COLS;
                            if (ARES) {
                                const uint64_t ad = umma::smem_desc_sw128(umma::smem_u32(a_res + (sl * a_chunks + c) * kABytes));
                                const uint64_t bd = umma::smem_desc_sw128(umma::smem_u32(st));
#pragma unroll
                                for (int kk = 0; kk < BK / 16; ++kk)
                                    umma::mma_f16_ss(dcol + sl * BN, ad + 2 * kk, bd + 2 * kk, idesc, (c > c_begin) || (kk > 0));
                            } else {
                                uint64_t ad[NB], bd[NB];
#pragma unroll
                                for (int b = 0; b < NB; ++b) {
                                    ad[b] = p.a_mn ? umma::smem_desc_sw128_mn(umma::smem_u32(st + b * kABytes), kABytes / 2)
                                                   : umma::smem_desc_sw128(umma::smem_u32(st + b * kABytes));
                                    bd[b] = umma::smem_desc_sw128(umma::smem_u32(st + NB * kABytes + b * B_BYTES));
                                }
#pragma unroll
                                for (int kk = 0; kk < BK / 16; ++kk)
#pragma unroll
                                    for (int b = 0; b < NB; ++b)
                                        umma::mma_f16_ss(dcol + b * BN, ad[b] + a_step * kk, bd[b] + 2 * kk, idesc,
                                                         (c > c_begin) || (kk > 0));
                            }
                            umma::mma_commit(&empty[stage]);
                        }
                        __syncwarp();
                        if (++stage == p.stages) { stage = 0; phase ^= 1; }
                    }
                }
                if (!ok) break;
                const bool last_of_m = ARES && ((t + 1 == tile_end) || (decode_tile<ARES>(p, t + 1).m != tc.m));
                if (umma::elect_one()) {
                    umma::mma_commit(&tfull[acc]);
                    if (last_of_m) umma::mma_commit(aempty);
                }
                __syncwarp();
                if (acc) acc_phase1 ^= 1; else acc_phase0 ^= 1;
                acc = (acc + 1) % NUM_ACC;
            }
        }
    } else {  // ---------------- epilogue warps 2..9: quadrant = warp % 4, column half = (warp - 2) / 4 ----------------
        const int q = warp & 3, half = (warp - 2) >> 2;
        int acc = 0;
        uint32_t acc_phase0 = 0, acc_phase1 = 0;
        bool ok = true;
        const int esz = (p.out_mode == OUT_F32) ? 4 : 2;
        const bool f16_out = p.out_mode == OUT_F16;
        unsigned char* my_stage = stage_out + (warp - 2) * 4096;
        // residual rows are requested into L2 one tile ahead of the epilogue that adds them
        auto prefetch_resid = [&](int tt) {
            if (p.resid == nullptr) return;
            const TileCoord pc = decode_tile<ARES>(p, tt);
            const int prow = pc.m * BM + q * 32 + lane;
            if (prow < p.M)
                for (int c0 = half * (BN / 2); c0 < (half + 1) * (BN / 2); c0 += 32)
                    if (pc.n * BN + c0 < p.N) umma::prefetch_l2(p.resid + (long)prow * p.ldc + pc.n * BN + c0);
        };
        if (tile_begin < tile_end) prefetch_resid(tile_begin);
        for (int t = tile_begin; t < tile_end && ok; ++t) {
            const TileCoord tc = decode_tile<ARES>(p, t);
            if (t + 1 < tile_end) prefetch_resid(t + 1);
            ok = umma::mbar_wait_warp(&tfull[acc], acc ? acc_phase1 : acc_phase0, abort_flag);
            if (!ok) break;
            umma::tc_fence_after_sync();
            const int row = tc.m * BM + q * 32 + lane;
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + acc * ACC_COLS;
            // The accumulator goes back to the issuer as soon as this warp's last TMEM load has landed in
            // registers: the arithmetic and the stores below no longer hold up the tile after next.
            auto release_acc = [&]() {
                umma::tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) umma::mbar_arrive(&tempty[acc]);
            };
            const int c_last32 = (half + 1) * (BN / 2) - 32, c_last64 = (half + 1) * (BN / 2) - 64;
            if (p.c_tma && p.out_mode == OUT_F32) {
                // fp32 output (optionally + residual) through shared memory: 32 columns = one 128-byte row
                // of the swizzled staging tile per thread, stored as [32 x 32] fp32 tiles by TMA.
#pragma unroll 1
                for (int c0 = half * (BN / 2); c0 < (half + 1) * (BN / 2); c0 += 32) {
                    const int col = tc.n * BN + c0;
                    // Residual: the warp reads the [32 x 32] tile cooperatively (lane = 16-byte chunk (lane & 7) of
                    // rows 4 i + lane / 8: every load instruction covers four whole 128-byte lines) and adds it to
                    // the staged tile in shared memory. The loads are issued before the TMEM wait; one row per lane
                    // (32 lines per instruction) took about 2000 cycles per group.
                    float4 rs[8];
                    const int rrow0 = tc.m * BM + q * 32 + (lane >> 3), rcol = col + 4 * (lane & 7);
                    const bool radd = p.resid != nullptr && rcol + 4 <= p.N;
                    if (radd) {
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            rs[i] = (rrow0 + 4 * i < p.M) ? *reinterpret_cast<const float4*>(p.resid + (long)(rrow0 + 4 * i) * p.ldc + rcol)
                                                          : make_float4(0.f, 0.f, 0.f, 0.f);
                    }
                    uint32_t ra[32];
                    float v[32];
                    umma::tmem_ld32(taddr + c0, ra);
                    if (NB == 2) {
                        uint32_t rb[32];
                        umma::tmem_ld32(taddr + BN + c0, rb);
                        umma::tmem_ld_wait();
                        if (c0 == c_last32) release_acc();
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] = fast_silu(__uint_as_float(ra[j])) * __uint_as_float(rb[j]);
                    } else {
                        umma::tmem_ld_wait();
                        if (c0 == c_last32) release_acc();
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(ra[j]);
                    }
                    umma::bulk_wait_read0();
                    __syncwarp();
#pragma unroll
                    for (int ch = 0; ch < 8; ++ch)
                        *reinterpret_cast<float4*>(my_stage + lane * 128 + ((ch ^ (lane & 7)) << 4)) =
                            make_float4(v[4 * ch], v[4 * ch + 1], v[4 * ch + 2], v[4 * ch + 3]);
                    if (p.resid != nullptr) __syncwarp();  // warp-uniform: every lane's row is staged before any chunk is updated
                    if (radd) {
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            const int rr = 4 * i + (lane >> 3);
                            float4* cell = reinterpret_cast<float4*>(my_stage + rr * 128 + (((lane & 7) ^ (rr & 7)) << 4));
                            float4 o = *cell;
                            o.x += rs[i].x; o.y += rs[i].y; o.z += rs[i].z; o.w += rs[i].w;
                            *cell = o;
                        }
                    }
                    umma::fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0 && col < p.N && tc.m * BM + q * 32 < p.M) {
                        umma::tma_store_2d(&p.tmC, my_stage, col + (int)(tc.z * p.batch_col_off), tc.m * BM + q * 32);
                        umma::bulk_commit();
                    }
                }
            } else if (p.c_tma) {
                // 16-bit output through shared memory: this warp owns BN/2 columns of its 32 rows; all TMEM
                // loads of a 64-column group are issued before the single wait, each thread packs its row
                // into the 128-byte-swizzled staging tile and one lane hands the [32 x 64] tile to a TMA store.
#pragma unroll 1
                for (int c0 = half * (BN / 2); c0 < (half + 1) * (BN / 2); c0 += 64) {
                    uint32_t ra[2][32], rb[2][32], packed[32];
                    umma::tmem_ld32(taddr + c0, ra[0]);
                    if (NB == 2) umma::tmem_ld32(taddr + BN + c0, rb[0]);
                    umma::tmem_ld32(taddr + c0 + 32, ra[1]);
                    if (NB == 2) umma::tmem_ld32(taddr + BN + c0 + 32, rb[1]);
                    umma::tmem_ld_wait();
                    if (c0 == c_last64) release_acc();
                    if (NB == 2 && f16_out) {
#pragma unroll
                        for (int hh = 0; hh < 2; ++hh)
#pragma unroll
                            for (int j = 0; j < 16; ++j)
                                packed[hh * 16 + j] = silu_mul_pack_f16(__uint_as_float(ra[hh][2 * j]), __uint_as_float(ra[hh][2 * j + 1]),
                                                                        __uint_as_float(rb[hh][2 * j]), __uint_as_float(rb[hh][2 * j + 1]));
                    } else {
#pragma unroll
                        for (int hh = 0; hh < 2; ++hh)
#pragma unroll
                            for (int j = 0; j < 16; ++j) {
                                float v0 = __uint_as_float(ra[hh][2 * j]), v1 = __uint_as_float(ra[hh][2 * j + 1]);
                                if (NB == 2) {
                                    v0 = fast_silu(v0) * __uint_as_float(rb[hh][2 * j]);
                                    v1 = fast_silu(v1) * __uint_as_float(rb[hh][2 * j + 1]);
                                }
                                packed[hh * 16 + j] = f16_out ? pack_f16(v0, v1) : pack_bf16(v0, v1);
                            }
                    }
                    umma::bulk_wait_read0();  // the previous store has finished reading the staging tile
                    __syncwarp();
                    if (p.c_t) {   // transposed tile [64 columns][32 rows]: a column's 32 rows are one 64-byte line
                        uint16_t* st16 = reinterpret_cast<uint16_t*>(my_stage);
#pragma unroll
                        for (int i = 0; i < 32; ++i) {
                            st16[(2 * i) * 32 + lane] = (uint16_t)(packed[i] & 0xffffu);
                            st16[(2 * i + 1) * 32 + lane] = (uint16_t)(packed[i] >> 16);
                        }
                    } else {
#pragma unroll
                    for (int ch = 0; ch < 8; ++ch)
                        *reinterpret_cast<uint4*>(my_stage + lane * 128 + ((ch ^ (lane & 7)) << 4)) =
                            make_uint4(packed[4 * ch], packed[4 * ch + 1], packed[4 * ch + 2], packed[4 * ch + 3]);
                    }
                    umma::fence_proxy_async_smem();
                    __syncwarp();
                    const int col = tc.n * BN + c0;
                    if (lane == 0 && col < p.N && tc.m * BM + q * 32 < p.M) {
                        if (p.c_t) umma::tma_store_2d(&p.tmC, my_stage, tc.m * BM + q * 32, col + (int)(tc.z * p.batch_col_off));
                        else umma::tma_store_2d(&p.tmC, my_stage, col + (int)(tc.z * p.batch_col_off), tc.m * BM + q * 32);
                        umma::bulk_commit();
                    }
                }
            } else {
                char* rowbase = reinterpret_cast<char*>(p.C) +
                                ((long)tc.ks * p.split_stride + (long)row * p.ldc + (long)tc.z * p.batch_col_off) * esz;
#pragma unroll 1
                for (int c0 = half * (BN / 2); c0 < (half + 1) * (BN / 2); c0 += 32) {
                    uint32_t ra[32];
                    float v[32];
                    umma::tmem_ld32(taddr + c0, ra);
                    if (NB == 2) {
                        uint32_t rb[32];
                        umma::tmem_ld32(taddr + BN + c0, rb);
                        umma::tmem_ld_wait();
                        if (c0 == c_last32) release_acc();
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] = fast_silu(__uint_as_float(ra[j])) * __uint_as_float(rb[j]);
                    } else {
                        umma::tmem_ld_wait();
                        if (c0 == c_last32) release_acc();
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(ra[j]);
                    }
                    const int col = tc.n * BN + c0;
                    if (row < p.M && col < p.N) {
                        if (p.resid != nullptr) {
                            const float* rr = p.resid + (long)row * p.ldc + col;
#pragma unroll
                            for (int j = 0; j < 32; j += 4)
                                if (j + 4 <= p.N - col) {
                                    float4 x = *reinterpret_cast<const float4*>(rr + j);
                                    v[j] += x.x; v[j + 1] += x.y; v[j + 2] += x.z; v[j + 3] += x.w;
                                }
                        }
                        store_row32(p, rowbase, col, p.N - col, v);
                    }
                }
            }
            if (acc) acc_phase1 ^= 1; else acc_phase0 ^= 1;
            acc = (acc + 1) % NUM_ACC;
        }
        if (p.c_tma) umma::bulk_wait_all();  // stores issued by this lane have been written
    }

    umma::tc_fence_before_sync();
    __syncthreads();
    if (*abort_flag) {
        if (threadIdx.x == 0 && p.status != nullptr) atomicExch(p.status, kErrTimeout);
        // give copies that may still be in flight time to land before the CTA's memory is released
        const uint64_t t0 = umma::globaltimer_ns();
        while (umma::globaltimer_ns() - t0 < 1000000ull) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 1) { umma::tc_fence_after_sync(); umma::tmem_dealloc(tmem_base, TMEM_COLS); }
}

// ---------------------------------------------------------------------------------------------
// CTA-pair variant (tcgen05 cta_group::2).  ARES: resident-A-strip GEMM for the short-K second GEMM
// of a chain (K = r); otherwise both operands stream through the ring (long-K first GEMM).  In both the MMA spans two CTAs of a cluster, each holding the A strip of its own 128
// token rows and loading only half of every B chunk, so a factor chunk fetched from L2 serves 256
// token rows instead of 128.  That halves both the L2 traffic and the shared-memory bytes that
// must be in flight per SM, which is what bounds the single-CTA kernel when K is short.
// Barriers: loads of both CTAs complete on the leader's (rank 0) "full"/"afull" barriers; the
// leader's MMA commits are multicast to the "empty"/"tfull"/"aempty" barriers of both CTAs; the
// epilogue warps of both CTAs arrive on the leader's "tempty".
template <int NB, int BN, bool ARES>
__global__ void __launch_bounds__(kPairThreads, 1) gemm_pair_kernel(const __grid_constant__ GemmParams p) {
    constexpr int HB_BYTES = (BN / 2) * BK * 2;  // this CTA's half of one B chunk
    // one ring slot (one barrier wait by the MMA issuer) per K chunk: every branch's half B chunk, and when A is
    // streamed every branch's A chunk too - a wait costs the issuer about as long as four N = 128 MMAs run
    constexpr int SLOT_BYTES = ARES ? NB * HB_BYTES : NB * (kABytes + HB_BYTES);
    constexpr int SLOTS_PER_CHUNK = 1;
    // streaming kernel: a slot may hold several consecutive K chunks, so that one issuer wait covers more MMAs
    const int cps = (ARES || p.cps < 1) ? 1 : p.cps;
    const int slot_bytes = cps * SLOT_BYTES;
    constexpr int ACC_COLS = NB * BN;
    // Two branches: each has its own issuer warp (1: gate, 10: up). A tcgen05.mma costs its issuing thread
    // about 50 cycles, close to the 64 tensor-pipe cycles of a 256 x 128 x 16 MMA, so one thread cannot keep
    // the pipe fed on 128-wide tiles; the two instruction streams touch different accumulators and every
    // barrier they signal (slot empty, accumulator full, strip empty) simply expects both.
    constexpr int NISS = (NB == 2) ? 2 : 1;
    constexpr int NUM_ACC = (2 * ACC_COLS <= 512) ? 2 : 1;
    constexpr int TMEM_COLS = (NUM_ACC * ACC_COLS <= 32) ? 32 : (NUM_ACC * ACC_COLS <= 64) ? 64 :
                              (NUM_ACC * ACC_COLS <= 128) ? 128 : (NUM_ACC * ACC_COLS <= 256) ? 256 : 512;

    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = smem_raw + ((1024u - (umma::smem_u32(smem_raw) & 1023u)) & 1023u);
    const int a_chunks = p.chunks_total;
    unsigned char* a_res = smem;
    unsigned char* ring = smem + (ARES ? NB * a_chunks * kABytes : 0);
    unsigned char* stage_out = ring + p.stages * slot_bytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(stage_out + (p.c_tma ? kEpiWarps * 4096 : 0));
    uint64_t* full = bars;
    uint64_t* empty = bars + kMaxStages;
    uint64_t* tfull = bars + 2 * kMaxStages;
    uint64_t* tempty = tfull + 2;
    uint64_t* afull = tempty + 2;
    uint64_t* aempty = afull + 1;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(aempty + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // Cluster = one CTA pair, or (split-K inside the cluster) cks pairs that share a tile: crank = 2 split + rank.
    const uint32_t crank = umma::cluster_ctarank();
    const int cks = (!ARES && NB == 1 && p.cks > 1) ? p.cks : 1;
    const uint32_t rank = crank & 1u;        // rank within the pair
    const uint32_t lead = crank & ~1u;       // cluster rank of the pair's leader
    const int split = (int)(crank >> 1);
    const uint16_t pair_mask = (uint16_t)(3u << lead);
    const bool leader = rank == 0;
    const int cluster_id = blockIdx.x / (2 * cks), nclusters = gridDim.x / (2 * cks);
    const int pairs_m = (p.tiles_m + 1) / 2;
    const int total_tiles = pairs_m * p.tiles_n * p.batch * p.ksplit;   // ksplit = 1 with split-K inside the cluster
    const int per_cluster = (total_tiles + nclusters - 1) / nclusters;  // 1 with split-K inside the cluster
    const int tile_begin = cluster_id * per_cluster;
    const int tile_end = min(total_tiles, tile_begin + per_cluster);
    // tile index -> (row-strip pair, column tile, split-K part, batch entry)
    auto decode = [&](int t, int& mp, int& n, int& ks, int& z) {
        if (ARES) { mp = t / p.tiles_n; n = t - mp * p.tiles_n; ks = 0; z = 0; }
        else { n = t % p.tiles_n; t /= p.tiles_n; mp = t % pairs_m; t /= pairs_m; ks = t % p.ksplit; z = t / p.ksplit; }
        if (cks > 1) ks = split;   // chunks_per_split is the cluster's split size
    };

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) { umma::mbar_init(&full[s], 1); umma::mbar_init(&empty[s], NISS); }
        for (int a = 0; a < 2; ++a) { umma::mbar_init(&tfull[a], NISS); umma::mbar_init(&tempty[a], 2 * kEpiWarps); }
        umma::mbar_init(afull, 1);
        umma::mbar_init(aempty, NISS);
        *abort_flag = 0;
        umma::fence_mbar_init();
        umma::prefetch_tmap(&p.tmA[0]); umma::prefetch_tmap(&p.tmB[0]);
        if (NB == 2) { umma::prefetch_tmap(&p.tmA[1]); umma::prefetch_tmap(&p.tmB[1]); }
        if (p.c_tma) umma::prefetch_tmap(&p.tmC);
    }
    if (warp == 1) { umma::tmem_alloc_pair(tmem_slot, TMEM_COLS); umma::tmem_relinquish_pair(); }
    umma::tc_fence_before_sync();
    __syncthreads();
    umma::cluster_sync();  // the partner's barriers are initialised before anything is signalled on them
    umma::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    umma::pdl_launch_dependents();
    // The B operands are weights, which no earlier kernel writes: the first tile's chunks are requested into L2
    // before this grid waits for its predecessor, so their first (HBM) touch overlaps the predecessor's tail.
    if (warp == 0 && lane == 0 && tile_begin < tile_end) {
        int mp, n, ks, z;
        decode(tile_begin, mp, n, ks, z);
        const int c_begin = ks * p.chunks_per_split, c_end = min(p.chunks_total, c_begin + min(p.chunks_per_split, 16));
        for (int b = 0; b < NB; ++b)
            for (int c = c_begin; c < c_end; ++c)
                umma::tma_prefetch_2d(&p.tmB[NB == 2 ? b : z], c * BK, n * BN + (int)rank * (BN / 2));
    }
    umma::pdl_wait();
    bool cl_ready = false;   // split-K inside the cluster: this epilogue warp's accumulator is complete

    if (warp == 0 || warp == kPairProducer2) {
        // ---------------- TMA producers (both CTAs): own A strip, own half of every B chunk ----------------
        // Waiting for a free slot, arming its barrier and issuing its copies cost one thread about 550 cycles
        // per slot, as long as the tensor pipe needs for the slot's MMAs; two warps take alternate slots so
        // that the ring is refilled at twice that rate. The first one also loads the resident A strips.
        const int pw = (warp == 0) ? 0 : 1;
        int stage = 0, cur_mp = -1, slot_no = 0;
        uint32_t phase = 0, a_phase = 0;
        bool ok = true;
        for (int t = tile_begin; t < tile_end && ok; ++t) {
            int mp, n, ks, z;
            decode(t, mp, n, ks, z);
            const int m = 2 * mp + (int)rank;
            if (ARES && pw == 0 && mp != cur_mp) {
                if (cur_mp >= 0) { ok = umma::mbar_wait_warp(aempty, a_phase, abort_flag); a_phase ^= 1; if (!ok) break; }
                if (umma::elect_one()) {
                    if (leader) umma::mbar_expect_tx(afull, 2 * NB * a_chunks * kABytes);
                    const uint32_t bar = umma::map_to_rank(afull, lead);
                    for (int b = 0; b < NB; ++b)
                        for (int c = 0; c < a_chunks; ++c)
                            umma::tma_load_2d_pair(a_res + (b * a_chunks + c) * kABytes, &p.tmA[b], bar, c * BK, m * BM);
                }
                __syncwarp();
                cur_mp = mp;
            }
            const int c_begin = ks * p.chunks_per_split, c_end = min(p.chunks_total, c_begin + p.chunks_per_split);
            for (int c = c_begin; c < c_end && ok; c += cps) {
                for (int sl = 0; sl < SLOTS_PER_CHUNK; ++sl) {
                    if (((slot_no++) & 1) != pw) {  // the other producer's slot
                        if (++stage == p.stages) { stage = 0; phase ^= 1; }
                        continue;
                    }
                    ok = umma::mbar_wait_warp(&empty[stage], phase ^ 1, abort_flag);
                    if (!ok) break;
                    if (umma::elect_one()) {
                        if (leader) umma::mbar_expect_tx(&full[stage], 2 * slot_bytes);
                        const uint32_t bar = umma::map_to_rank(&full[stage], lead);
                        unsigned char* st = ring + stage * slot_bytes;
                        if (ARES) {
#pragma unroll
                            for (int b = 0; b < NB; ++b)
                                umma::tma_load_2d_pair(st + b * HB_BYTES, &p.tmB[b], bar, c * BK, n * BN + (int)rank * (BN / 2));
                        } else {  // per chunk of the slot: every branch's A chunk and B half (chunks past the end read as zero or are ignored)
                            for (int j = 0; j < cps; ++j)
#pragma unroll
                                for (int b = 0; b < NB; ++b) {
                                    unsigned char* sb = st + j * SLOT_BYTES + b * (kABytes + HB_BYTES);
                                    if (p.a_mn) {  // two boxes [64 k][64 m] of A^T
                                        umma::tma_load_2d_pair(sb, &p.tmA[NB == 2 ? b : z], bar, m * BM, (c + j) * BK);
                                        umma::tma_load_2d_pair(sb + kABytes / 2, &p.tmA[NB == 2 ? b : z], bar, m * BM + 64, (c + j) * BK);
                                    } else {
                                        umma::tma_load_2d_pair(sb, &p.tmA[NB == 2 ? b : z], bar, (c + j) * BK, m * BM);
                                    }
                                    umma::tma_load_2d_pair(sb + kABytes, &p.tmB[NB == 2 ? b : z], bar, (c + j) * BK,
                                                           n * BN + (int)rank * (BN / 2));
                                }
                        }
                    }
                    __syncwarp();
                    if (++stage == p.stages) { stage = 0; phase ^= 1; }
                }
            }
        }
    } else if (warp == 1 || (NISS == 2 && warp == 10)) {
        if (leader) {  // ---------------- MMA issuer(s) (leader CTA only) ----------------
            const int bsel = (warp == 1) ? 0 : 1;  // with two issuers: the branch this one feeds
            const uint32_t idesc = umma::make_idesc(p.a_fmt, p.b_fmt, 2 * BM, BN) | (p.a_mn ? umma::kIdescAMnMajor : 0u);
            const uint64_t a_step = p.a_mn ? 128 : 2;
            int stage = 0, cur_mp = -1, acc = 0;
            uint32_t phase = 0, a_phase = 0, acc_phase0 = 0, acc_phase1 = 0;
            bool ok = true;
            // The tile coordinates advance incrementally: an integer division per tile sat on the issuer's
            // critical path at every tile boundary.
            int mp = 0, n = 0, ks = 0, z = 0;
            if (tile_begin < tile_end) decode(tile_begin, mp, n, ks, z);
            bool ready = false;  // the next slot's barrier, sampled while the previous slot's MMAs were being issued
            for (int t = tile_begin; t < tile_end && ok; ++t) {
                ok = umma::mbar_wait_warp(&tempty[acc], (acc ? acc_phase1 : acc_phase0) ^ 1, abort_flag);
                if (!ok) break;
                if (ARES && mp != cur_mp) {
                    ok = umma::mbar_wait_warp(afull, a_phase, abort_flag);
                    a_phase ^= 1; cur_mp = mp;
                    if (!ok) break;
                }
                umma::tc_fence_after_sync();
                const int c_begin = ks * p.chunks_per_split, c_end = min(p.chunks_total, c_begin + p.chunks_per_split);
                for (int c = c_begin; c < c_end && ok; c += cps) {
                    for (int sl = 0; sl < SLOTS_PER_CHUNK; ++sl) {
                        if (!ready) {
                            ok = umma::mbar_wait_warp(&full[stage], phase, abort_flag);
                            if (!ok) break;
                        }
                        {   // non-blocking look at the next slot: its latency hides behind this slot's MMAs
                            const int nstage = (stage + 1 == p.stages) ? 0 : stage + 1;
                            ready = __all_sync(0xffffffffu, umma::mbar_test_wait(&full[nstage], nstage ? phase : phase ^ 1));
                        }
                        if (umma::elect_one()) {
                            const unsigned char* st = ring + stage * slot_bytes;
                            for (int j = 0; j < cps && c + j < c_end; ++j)
#pragma unroll
                                for (int b = 0; b < NB; ++b) {
                                    if (NISS == 2 && b != bsel) continue;
                                    const int br = b;  // branch whose accumulator this group feeds
                                    const unsigned char* a_ptr = ARES ? a_res + (b * a_chunks + c) * kABytes : st + j * SLOT_BYTES + b * (kABytes + HB_BYTES);
                                    const unsigned char* b_ptr = ARES ? st + b * HB_BYTES : a_ptr + kABytes;
                                    // Descriptors step by 32 bytes (2 in address units of 16) along K inside the
                                    // swizzle atom; shared memory is below 256 KiB, so the 14-bit field never carries.
                                    const uint64_t ad = (!ARES && p.a_mn) ? umma::smem_desc_sw128_mn(umma::smem_u32(a_ptr), kABytes / 2)
                                                                          : umma::smem_desc_sw128(umma::smem_u32(a_ptr));
                                    const uint64_t bd = umma::smem_desc_sw128(umma::smem_u32(b_ptr));
                                    const uint32_t dcol = tmem_base + acc * ACC_COLS + br * BN;
#pragma unroll
                                    for (int kk = 0; kk < BK / 16; ++kk)
                                        umma::mma_f16_ss_pair(dcol, ad + a_step * kk, bd + 2 * kk, idesc,
                                                              (c + j > c_begin) || (kk > 0));
                                }
                            umma::mma_commit_pair(&empty[stage], pair_mask);
                        }
                        __syncwarp();
                        if (++stage == p.stages) { stage = 0; phase ^= 1; }
                    }
                }
                if (!ok) break;
                const bool last_of_m = ARES && ((t + 1 == tile_end) || (n + 1 == p.tiles_n));
                if (umma::elect_one()) {
                    umma::mma_commit_pair(&tfull[acc], pair_mask);
                    if (last_of_m) umma::mma_commit_pair(aempty, pair_mask);
                }
                __syncwarp();
                if (acc) acc_phase1 ^= 1; else acc_phase0 ^= 1;
                acc = (acc + 1) % NUM_ACC;
                if (++n == p.tiles_n) {
                    n = 0;
                    if (ARES) ++mp;
                    else if (++mp == pairs_m) { mp = 0; if (++ks == p.ksplit) { ks = 0; ++z; } }
                }
            }
        }
    } else if (warp < 2 + kEpiWarps) {  // ---------------- epilogue warps 2..9 (both CTAs, own 128 rows) ----------------
        const int q = warp & 3, half = (warp - 2) >> 2;
        int acc = 0;
        uint32_t acc_phase0 = 0, acc_phase1 = 0;
        bool ok = true;
        const int esz = (p.out_mode == OUT_F32) ? 4 : 2;
        const bool f16_out = p.out_mode == OUT_F16;
        unsigned char* my_stage = stage_out + (warp - 2) * 4096;
        const uint32_t tempty_leader[2] = {umma::map_to_rank(&tempty[0], lead), umma::map_to_rank(&tempty[1], lead)};
        // The residual rows this warp will add are requested into L2 one tile ahead (the first tile's at kernel
        // start): read on demand, each 32-column group waited a full HBM round trip inside the epilogue.
        auto prefetch_resid = [&](int tt) {
            if (p.resid == nullptr) return;
            int pmp, pn, pks, pz;
            decode(tt, pmp, pn, pks, pz);
            const int prow = (2 * pmp + (int)rank) * BM + q * 32 + lane;
            if (prow < p.M)
                for (int c0 = half * (BN / 2); c0 < (half + 1) * (BN / 2); c0 += 32)
                    if (pn * BN + c0 < p.N) umma::prefetch_l2(p.resid + (long)prow * p.ldc + pn * BN + c0);
        };
        if (tile_begin < tile_end) prefetch_resid(tile_begin);
        for (int t = tile_begin; t < tile_end && ok; ++t) {
            int mp, n, ks, z;
            decode(t, mp, n, ks, z);
            const int m = 2 * mp + (int)rank;
            if (t + 1 < tile_end) prefetch_resid(t + 1);
            // fp32 + residual epilogue: the residual of a 32-column group is loaded one group ahead (the first
            // group's before the accumulator is even complete), so its latency hides behind the mainloop and
            // behind the previous group's staging and store instead of standing in front of every group.
            float4 rs[8];
            auto load_rs = [&](int c0n) {
                const int rrow0 = m * BM + q * 32 + (lane >> 3), rcol = n * BN + c0n + 4 * (lane & 7);
                if (p.resid != nullptr && rcol + 4 <= p.N) {
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        rs[i] = (rrow0 + 4 * i < p.M) ? *reinterpret_cast<const float4*>(p.resid + (long)(rrow0 + 4 * i) * p.ldc + rcol)
                                                      : make_float4(0.f, 0.f, 0.f, 0.f);
                }
            };
            if (p.c_tma && p.out_mode == OUT_F32) load_rs(half * (BN / 2));
            ok = umma::mbar_wait_warp(&tfull[acc], acc ? acc_phase1 : acc_phase0, abort_flag);
            if (!ok) break;
            umma::tc_fence_after_sync();
            if (cks > 1) { cl_ready = true; break; }   // the sum over the cluster's splits follows below, for all roles together
            const int row = m * BM + q * 32 + lane;
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + acc * ACC_COLS;
            // The accumulator goes back to the issuer as soon as this warp's last TMEM load has landed in
            // registers: the arithmetic and the stores below no longer hold up the tile after next.
            auto release_acc = [&]() {
                umma::tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) umma::mbar_arrive_cluster(tempty_leader[acc]);
            };
            const int c_last32 = (half + 1) * (BN / 2) - 32, c_last64 = (half + 1) * (BN / 2) - 64;
            if (p.c_tma && p.out_mode == OUT_F32) {
                // fp32 output (optionally + residual) through shared memory: 32 columns = one 128-byte row
                // of the swizzled staging tile per thread, stored as [32 x 32] fp32 tiles by TMA.
#pragma unroll 1
                for (int c0 = half * (BN / 2); c0 < (half + 1) * (BN / 2); c0 += 32) {
                    const int col = n * BN + c0;
                    // Residual: the warp reads the [32 x 32] tile cooperatively (lane = 16-byte chunk (lane & 7) of
                    // rows 4 i + lane / 8: every load instruction covers four whole 128-byte lines) and adds it to
                    // the staged tile in shared memory (one row per lane, 32 lines per instruction, took about 2000
                    // cycles per group).  rs holds this group's values, loaded one group ago.
                    const int rcol = col + 4 * (lane & 7);
                    const bool radd = p.resid != nullptr && rcol + 4 <= p.N;
                    uint32_t ra[32];
                    float v[32];
                    umma::tmem_ld32(taddr + c0, ra);
                    if (NB == 2) {
                        uint32_t rb[32];
                        umma::tmem_ld32(taddr + BN + c0, rb);
                        umma::tmem_ld_wait();
                        if (c0 == c_last32) release_acc();
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] = fast_silu(__uint_as_float(ra[j])) * __uint_as_float(rb[j]);
                    } else {
                        umma::tmem_ld_wait();
                        if (c0 == c_last32) release_acc();
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(ra[j]);
                    }
                    umma::bulk_wait_read0();
                    __syncwarp();
#pragma unroll
                    for (int ch = 0; ch < 8; ++ch)
                        *reinterpret_cast<float4*>(my_stage + lane * 128 + ((ch ^ (lane & 7)) << 4)) =
                            make_float4(v[4 * ch], v[4 * ch + 1], v[4 * ch + 2], v[4 * ch + 3]);
                    if (p.resid != nullptr) __syncwarp();  // warp-uniform: every lane's row is staged before any chunk is updated
                    if (radd) {
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            const int rr = 4 * i + (lane >> 3);
                            float4* cell = reinterpret_cast<float4*>(my_stage + rr * 128 + (((lane & 7) ^ (rr & 7)) << 4));
                            float4 o = *cell;
                            o.x += rs[i].x; o.y += rs[i].y; o.z += rs[i].z; o.w += rs[i].w;
                            *cell = o;
                        }
                    }
                    if (c0 + 32 < (half + 1) * (BN / 2)) load_rs(c0 + 32);   // the next group's residual, in flight from here on
                    umma::fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0 && col < p.N && m * BM + q * 32 < p.M) {
                        umma::tma_store_2d(&p.tmC, my_stage, col + (int)(z * p.batch_col_off), m * BM + q * 32);
                        umma::bulk_commit();
                    }
                }
            } else if (p.c_tma) {
                // 16-bit output through shared memory: this warp owns BN/2 columns of its 32 rows; all TMEM
                // loads of a 64-column group are issued before the single wait, each thread packs its row
                // into the 128-byte-swizzled staging tile and one lane hands the [32 x 64] tile to a TMA store.
#pragma unroll 1
                for (int c0 = half * (BN / 2); c0 < (half + 1) * (BN / 2); c0 += 64) {
                    uint32_t ra[2][32], rb[2][32], packed[32];
                    umma::tmem_ld32(taddr + c0, ra[0]);
                    if (NB == 2) umma::tmem_ld32(taddr + BN + c0, rb[0]);
                    umma::tmem_ld32(taddr + c0 + 32, ra[1]);
                    if (NB == 2) umma::tmem_ld32(taddr + BN + c0 + 32, rb[1]);
                    umma::tmem_ld_wait();
                    if (c0 == c_last64) release_acc();
                    if (NB == 2 && f16_out) {
#pragma unroll
                        for (int hh = 0; hh < 2; ++hh)
#pragma unroll
                            for (int j = 0; j < 16; ++j)
                                packed[hh * 16 + j] = silu_mul_pack_f16(__uint_as_float(ra[hh][2 * j]), __uint_as_float(ra[hh][2 * j + 1]),
                                                                        __uint_as_float(rb[hh][2 * j]), __uint_as_float(rb[hh][2 * j + 1]));
                    } else {
#pragma unroll
                        for (int hh = 0; hh < 2; ++hh)
#pragma unroll
                            for (int j = 0; j < 16; ++j) {
                                float v0 = __uint_as_float(ra[hh][2 * j]), v1 = __uint_as_float(ra[hh][2 * j + 1]);
                                if (NB == 2) {
                                    v0 = fast_silu(v0) * __uint_as_float(rb[hh][2 * j]);
                                    v1 = fast_silu(v1) * __uint_as_float(rb[hh][2 * j + 1]);
                                }
                                packed[hh * 16 + j] = f16_out ? pack_f16(v0, v1) : pack_bf16(v0, v1);
                            }
                    }
                    umma::bulk_wait_read0();  // the previous store has finished reading the staging tile
                    __syncwarp();
                    if (p.c_t) {   // transposed tile [64 columns][32 rows]: a column's 32 rows are one 64-byte line
                        uint16_t* st16 = reinterpret_cast<uint16_t*>(my_stage);
#pragma unroll
                        for (int i = 0; i < 32; ++i) {
                            st16[(2 * i) * 32 + lane] = (uint16_t)(packed[i] & 0xffffu);
                            st16[(2 * i + 1) * 32 + lane] = (uint16_t)(packed[i] >> 16);
                        }
                    } else {
#pragma unroll
                    for (int ch = 0; ch < 8; ++ch)
                        *reinterpret_cast<uint4*>(my_stage + lane * 128 + ((ch ^ (lane & 7)) << 4)) =
                            make_uint4(packed[4 * ch], packed[4 * ch + 1], packed[4 * ch + 2], packed[4 * ch + 3]);
                    }
                    umma::fence_proxy_async_smem();
                    __syncwarp();
                    const int col = n * BN + c0;
                    if (lane == 0 && col < p.N && m * BM + q * 32 < p.M) {
                        if (p.c_t) umma::tma_store_2d(&p.tmC, my_stage, m * BM + q * 32, col + (int)(z * p.batch_col_off));
                        else umma::tma_store_2d(&p.tmC, my_stage, col + (int)(z * p.batch_col_off), m * BM + q * 32);
                        umma::bulk_commit();
                    }
                }
            } else {
                char* rowbase = reinterpret_cast<char*>(p.C) +
                                ((long)ks * p.split_stride + (long)row * p.ldc + (long)z * p.batch_col_off) * esz;
#pragma unroll 1
                for (int c0 = half * (BN / 2); c0 < (half + 1) * (BN / 2); c0 += 32) {
                    uint32_t ra[32];
                    float v[32];
                    umma::tmem_ld32(taddr + c0, ra);
                    if (NB == 2) {
                        uint32_t rb[32];
                        umma::tmem_ld32(taddr + BN + c0, rb);
                        umma::tmem_ld_wait();
                        if (c0 == c_last32) release_acc();
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] = fast_silu(__uint_as_float(ra[j])) * __uint_as_float(rb[j]);
                    } else {
                        umma::tmem_ld_wait();
                        if (c0 == c_last32) release_acc();
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(ra[j]);
                    }
                    const int col = n * BN + c0;
                    if (row < p.M && col < p.N) {
                        if (p.resid != nullptr) {
                            const float* rr = p.resid + (long)row * p.ldc + col;
#pragma unroll
                            for (int j = 0; j < 32; j += 4)
                                if (j + 4 <= p.N - col) {
                                    float4 x = *reinterpret_cast<const float4*>(rr + j);
                                    v[j] += x.x; v[j + 1] += x.y; v[j + 2] += x.z; v[j + 3] += x.w;
                                }
                        }
                        store_row32(p, rowbase, col, p.N - col, v);
                    }
                }
            }
            if (acc) acc_phase1 ^= 1; else acc_phase0 ^= 1;
            acc = (acc + 1) % NUM_ACC;
        }
        if (p.c_tma) umma::bulk_wait_all();
    }

    if (cks > 1) {
        // ---- split-K inside the cluster: reduce-scatter of the cks partial accumulators through distributed shared memory.
        // Pair s owns the columns [s W, (s + 1) W) of the tile, W = BN / cks.  Every epilogue thread pushes its row's 32-column
        // groups into the owner's receive buffer (the ring, idle by now): [source split][128 rows][W floats + 4 of padding];
        // then every CTA sums its W columns over the sources in split order (a fixed order: the result does not depend on
        // timing) and stores them.  Both cluster barriers are reached by every thread of every CTA, whatever happened before.
        // Receive layout: [source split][32-row block][16-byte piece of the W columns][row in block][4 floats], so that a
        // warp instruction (lane = row) writes, and later reads, 512 contiguous bytes.
        const int W = BN / cks, blk = W * 128;        // bytes of one 32-row block: W / 4 pieces x 512 B
        umma::cluster_sync();   // every CTA's MMAs have finished reading its ring
        const bool epi = warp >= 2 && warp < 2 + kEpiWarps;
        if (epi && cl_ready) {
            const int q = warp & 3, half = (warp - 2) >> 2;
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
#pragma unroll 1
            for (int c0 = half * (BN / 2); c0 < (half + 1) * (BN / 2); c0 += 32) {
                uint32_t ra[32];
                umma::tmem_ld32(taddr + c0, ra);
                umma::tmem_ld_wait();
                const int owner = c0 / W, cw = c0 - owner * W;   // a 32-column group never straddles two owners (W >= 32)
                const uint32_t dst = umma::map_to_rank(ring + (size_t)(split * 4 + q) * blk + (cw / 4) * 512 + lane * 16, 2u * owner + rank);
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    umma::st_cluster_f32x4(dst + 512 * j, __uint_as_float(ra[4 * j]), __uint_as_float(ra[4 * j + 1]),
                                           __uint_as_float(ra[4 * j + 2]), __uint_as_float(ra[4 * j + 3]));
            }
        }
        umma::cluster_sync();   // all pushes have landed (release / acquire at cluster scope)
        if (epi && tile_begin < tile_end) {
            int mp, n, ks, z;
            decode(tile_begin, mp, n, ks, z);
            const int te = threadIdx.x - 64, r = te & (BM - 1), part = te >> 7;   // 256 threads: row, column half of the slice
            const int row = (2 * mp + (int)rank) * BM + r, hw = W / 2;
            const int col0 = n * BN + split * W + part * hw;
            if (row < p.M) {
                char* out = reinterpret_cast<char*>(p.C) + ((long)row * p.ldc + (long)z * p.batch_col_off + col0) * 2;
                for (int c = 0; c < hw; c += 8) {
                    float acc8[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
                    for (int src = 0; src < cks; ++src) {
                        const unsigned char* cell = ring + (size_t)(src * 4 + (r >> 5)) * blk + ((part * hw + c) / 4) * 512 + (r & 31) * 16;
                        const float4 a = *reinterpret_cast<const float4*>(cell), b = *reinterpret_cast<const float4*>(cell + 512);
                        acc8[0] += a.x; acc8[1] += a.y; acc8[2] += a.z; acc8[3] += a.w;
                        acc8[4] += b.x; acc8[5] += b.y; acc8[6] += b.z; acc8[7] += b.w;
                    }
                    if (col0 + c + 8 <= p.N) {
                        uint4 w;
                        if (p.out_mode == OUT_F16) {
                            w.x = pack_f16(acc8[0], acc8[1]); w.y = pack_f16(acc8[2], acc8[3]);
                            w.z = pack_f16(acc8[4], acc8[5]); w.w = pack_f16(acc8[6], acc8[7]);
                        } else {
                            w.x = pack_bf16(acc8[0], acc8[1]); w.y = pack_bf16(acc8[2], acc8[3]);
                            w.z = pack_bf16(acc8[4], acc8[5]); w.w = pack_bf16(acc8[6], acc8[7]);
                        }
                        *reinterpret_cast<uint4*>(out + c * 2) = w;
                    }
                }
            }
        }
    }
    umma::tc_fence_before_sync();
    __syncthreads();
    if (*abort_flag) {
        if (threadIdx.x == 0 && p.status != nullptr) atomicExch(p.status, kErrTimeout);
        const uint64_t t0 = umma::globaltimer_ns();
        while (umma::globaltimer_ns() - t0 < 1000000ull) __nanosleep(1000);
        __syncthreads();
    }
    umma::cluster_sync();  // neither CTA's shared memory or TMEM goes away while the partner may still use it
    if (warp == 1) { umma::tc_fence_after_sync(); umma::tmem_dealloc_pair(tmem_base, TMEM_COLS); }
}

// out[c, r] = in[r, c] for a 16-bit matrix in[rows, cols] (32 x 32 tiles through shared memory).  Used only for
// the transposed layouts of the XUV operator at T <= 32, where the weight-streaming kernels run.
__global__ void __launch_bounds__(256)
transpose16_kernel(const uint16_t* __restrict__ in, int rows, int cols, uint16_t* __restrict__ out) {
    __shared__ uint16_t tile[32][33];
    const int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32, tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    for (int i = ty; i < 32; i += 8)
        if (r0 + i < rows && c0 + tx < cols) tile[i][tx] = in[(long)(r0 + i) * cols + c0 + tx];
    __syncthreads();
    for (int i = ty; i < 32; i += 8)
        if (c0 + i < cols && r0 + tx < rows) out[(long)(c0 + i) * rows + r0 + tx] = tile[tx][i];
}

// Exact re-encoding of bf16 weights as fp16 (tcgen05 kind::f16 wants A and B in the same 16-bit
// format, and the intermediates it multiplies them with are kept in fp16 for precision).
// bf16's 8-bit significand always fits; only the range differs: *flag is set to 1 if a value is
// beyond fp16's largest finite number, values below 2^-14 lose low bits (absolute error <= 2^-25).
__global__ void __launch_bounds__(256)
bf16_to_f16_kernel(const __nv_bfloat16* __restrict__ in, __half* __restrict__ out, long n, int* flag) {
    bool bad = false;
    for (long i = ((long)blockIdx.x * blockDim.x + threadIdx.x) * 8; i < n; i += (long)gridDim.x * blockDim.x * 8) {
        uint4 v = *reinterpret_cast<const uint4*>(in + i);
        const __nv_bfloat162* b = reinterpret_cast<const __nv_bfloat162*>(&v);
        uint4 w;
        uint32_t* o = reinterpret_cast<uint32_t*>(&w);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            float2 f = __bfloat1622float2(b[j]);
            bad |= !(fabsf(f.x) <= 65504.f) || !(fabsf(f.y) <= 65504.f);
            o[j] = pack_f16(f.x, f.y);
        }
        *reinterpret_cast<uint4*>(out + i) = w;
    }
    if (bad) atomicExch(flag, 1);
}

// Sum split-K fp32 partials [ksplit][M, N] and write fp16 [M, N] (and, on request, the fp32 sums as well).
__global__ void __launch_bounds__(256)
reduce_partials_kernel(const float* __restrict__ part, int ksplit, long split_stride, long n, __half* __restrict__ out,
                       float* __restrict__ out32) {
    umma::pdl_launch_dependents();
    umma::pdl_wait();  // launched with programmatic stream serialization: the partials come from the previous grid
    for (long i = ((long)blockIdx.x * blockDim.x + threadIdx.x) * 4; i < n; i += (long)gridDim.x * blockDim.x * 4) {
        float4 s = *reinterpret_cast<const float4*>(part + i);
        for (int k = 1; k < ksplit; ++k) {
            float4 v = *reinterpret_cast<const float4*>(part + k * split_stride + i);
            s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
        }
        uint2 w;
        w.x = pack_f16(s.x, s.y);
        w.y = pack_f16(s.z, s.w);
        *reinterpret_cast<uint2*>(out + i) = w;
        if (out32 != nullptr) *reinterpret_cast<float4*>(out32 + i) = s;   // the unrounded sum, for a caller that adds shards
    }
}

// The same sum for many splits (more than 16).
// Block = 32 output quads x 8 slices of the splits: with many splits (the fused kernel cuts a short batch into up
// to 80) a thread that walks all of them alone is bound by L2 latency, so eight threads share an output quad.
__global__ void __launch_bounds__(256)
reduce_partials_wide_kernel(const float* __restrict__ part, int ksplit, long split_stride, long n, __half* __restrict__ out,
                       float* __restrict__ out32) {
    __shared__ float4 sh[8][32];
    umma::pdl_launch_dependents();
    umma::pdl_wait();  // launched with programmatic stream serialization: the partials come from the previous grid
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    for (long i0 = (long)blockIdx.x * 128; i0 < n; i0 += (long)gridDim.x * 128) {
        const long i = i0 + tx * 4;
        float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
        if (i < n) {
            for (int k0 = ty; k0 < ksplit; k0 += 32) {   // four loads in flight per thread
                float4 v[4];
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    v[j] = (k0 + 8 * j < ksplit) ? *reinterpret_cast<const float4*>(part + (long)(k0 + 8 * j) * split_stride + i)
                                                 : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int j = 0; j < 4; ++j) { s.x += v[j].x; s.y += v[j].y; s.z += v[j].z; s.w += v[j].w; }
            }
        }
        sh[ty][tx] = s;
        __syncthreads();
        if (ty == 0 && i < n) {
#pragma unroll
            for (int j = 1; j < 8; ++j) { const float4 v = sh[j][tx]; s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w; }
            uint2 w;
            w.x = pack_f16(s.x, s.y);
            w.y = pack_f16(s.z, s.w);
            *reinterpret_cast<uint2*>(out + i) = w;
            if (out32 != nullptr) *reinterpret_cast<float4*>(out32 + i) = s;   // the unrounded sum, for a caller that adds shards
        }
        __syncthreads();
    }
}

// fp32 [n] -> fp16 [n] (n a multiple of 4): a sum of partial Zd shards becomes the operand of the last product.
__global__ void __launch_bounds__(256)
f32_to_f16_kernel(const float* __restrict__ in, __half* __restrict__ out, long n) {
    umma::pdl_launch_dependents();
    umma::pdl_wait();
    for (long i = ((long)blockIdx.x * blockDim.x + threadIdx.x) * 4; i < n; i += (long)gridDim.x * blockDim.x * 4) {
        const float4 s = *reinterpret_cast<const float4*>(in + i);
        uint2 w;
        w.x = pack_f16(s.x, s.y);
        w.y = pack_f16(s.z, s.w);
        *reinterpret_cast<uint2*>(out + i) = w;
    }
}

}  // namespace tensorpath
