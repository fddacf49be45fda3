// Gate+up expansion with the Z strip in tensor memory (phase 2 of Algorithm 3 with its SiLU(G).*Up
// epilogue) for equal gate/up ranks up to 256:  H[T, ffn] = SiLU(Zg Ug^T) .* (Zu Uu^T), fp16 in, fp16 out.
//
// Why a kernel of its own: with both operands in shared memory a 128-column tile of this product moves about
// 384 KB through shared memory per CTA (256 KB of operand reads, 64 KB of TMA fills, 64 KB of staged output),
// 3000 cycles at 128 B/clk against 2048 tensor-pipe cycles, and the resident [128, 2r] strip of Z (the paper's
// on-chip strip cache, Section 4.2.1 "Caching") leaves only 64 KB for the factor ring.  Here the strip is
// copied once per row strip from shared memory into TMEM (tcgen05.cp) and every MMA takes its A operand from
// there (tcgen05.mma with a TMEM A operand): an MMA reads only its factor chunk from shared memory, and the
// 128 KB the strip occupied becomes ring slots.
//
// TMEM columns (512): [0, 128) gate strip, [128, 256) up strip (fp16 pairs: 32-bit column c = k 2c, 2c + 1),
// [256, 384) G accumulator, [384, 512) Up accumulator.  The accumulators cannot be double-buffered, so the two
// branches are handed over separately and their MMA streams run half a tile apart: while the tensor pipe works
// on Up of a tile the epilogue warps pull G into registers, hand its columns back and compute SiLU(G) (packed
// fp16), and while it works on G of the next tile they pull Up, multiply and store, so neither side waits for
// the other in steady state.
//
// CTA pair (cta_group::2): each CTA owns 128 token rows; of every 128-wide factor tile each CTA loads 64 rows.
// A ring slot holds two K chunks of one branch (16 KB per CTA; the last slot of an odd chunk count holds one);
// the strip's own [128 x 64] chunks travel through the same ring on their way to TMEM.
// Warps: 0 and 11 TMA producers (alternate slots), 1 and 10 tcgen05 issuers
// (leader CTA; G and Up; warp 1 also copies the strips and owns TMEM), 2-9 epilogue (lane quadrant x column
// half; staged [32 x 64] fp16 tiles leave by TMA store).  Every wait is bounded; on a timeout the status word is set and the kernel tears down
// normally (TMEM freed, cluster sync before exit).
#pragma once
#include "tensor_gemm.cuh"

namespace tensorpath {

constexpr int kTsMaxSlots = 12;              // ring slots (16 KiB): two [64 x 64] factor chunks or one [128 x 64] strip chunk
static_assert(kTsMaxSlots % 4 == 0, "a ring slot must always serve the same branch within a row strip");
constexpr int kTsChunkBytes = 64 * BK * 2;   // one CTA's half of a [128 x 64] factor chunk
constexpr int kTsSlotBytes = 2 * kTsChunkBytes;
static_assert(kTsSlotBytes == kABytes, "a ring slot also carries one strip chunk on its way to TMEM");
constexpr int kTsBarrierBytes = (2 * kTsMaxSlots + 6) * 8 + 16;
constexpr int kTsSmemBytes = 1024 + kTsMaxSlots * kTsSlotBytes + kEpiWarps * 4096 + kTsBarrierBytes;

// 128 lanes x 256 bits per lane from a K-major swizzled shared-memory tile into TMEM, in both CTAs of the pair
__device__ __forceinline__ void tmem_cp_128x256b_pair(uint32_t taddr, uint64_t sdesc) {
    asm volatile("tcgen05.cp.cta_group::2.128x256b [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]^T across the CTA pair; A: lane = row, 32-bit column c = (k = 2c, 2c + 1).
__device__ __forceinline__ void mma_f16_ts_pair(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, bool accumulate) {
    const uint32_t zero = 0;
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], [%1], %2, %3, {%5, %6, %7, %8, %9, %10, %11, %12}, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"((uint32_t)accumulate),
          "r"(zero), "r"(zero), "r"(zero), "r"(zero), "r"(zero), "r"(zero), "r"(zero), "r"(zero) : "memory");
}

// p: tmA[0/1] = Zg / Zu ([T, r] fp16, box [128, 64]); tmB[0/1] = Ug / Uu ([ffn, r] fp16, box [64, 64]);
// tmC = H ([T, ffn] fp16, box [32, 64]); M = T, N = ffn, K = r <= 256; tiles_m = ceil(T / 128),
// tiles_n = ceil(ffn / 128), chunks_total = ceil(r / 64); stages = ring slots (2 .. kTsMaxSlots).
__global__ void __launch_bounds__(kPairThreads, 1) gateup_ts_pair_kernel(const __grid_constant__ GemmParams p) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = smem_raw + ((1024u - (umma::smem_u32(smem_raw) & 1023u)) & 1023u);
    unsigned char* ring = smem;
    unsigned char* stage_out = ring + kTsMaxSlots * kTsSlotBytes;
    uint64_t* full = reinterpret_cast<uint64_t*>(stage_out + kEpiWarps * 4096);
    uint64_t* empty = full + kTsMaxSlots;
    uint64_t* tfull = empty + kTsMaxSlots;   // [branch]
    uint64_t* tempty = tfull + 2;   // [branch]
    uint64_t* adone = tempty + 2;
    uint64_t* aready = adone + 1;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(aready + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = umma::cluster_ctarank();
    const bool leader = rank == 0;
    const int cluster_id = blockIdx.x >> 1, nclusters = gridDim.x >> 1;
    const int pairs_m = (p.tiles_m + 1) / 2;
    const int total_tiles = pairs_m * p.tiles_n;
    const int per_cluster = (total_tiles + nclusters - 1) / nclusters;
    const int tile_begin = cluster_id * per_cluster;
    const int tile_end = min(total_tiles, tile_begin + per_cluster);
    const int chunks = p.chunks_total, nslot = p.stages;

    if (threadIdx.x == 0) {
        for (int s = 0; s < nslot; ++s) { umma::mbar_init(&full[s], 1); umma::mbar_init(&empty[s], 1); }
        for (int a = 0; a < 2; ++a) { umma::mbar_init(&tfull[a], 1); umma::mbar_init(&tempty[a], 2 * kEpiWarps); }
        umma::mbar_init(adone, 2);
        umma::mbar_init(aready, 1);
        *abort_flag = 0;
        umma::fence_mbar_init();
        umma::prefetch_tmap(&p.tmA[0]); umma::prefetch_tmap(&p.tmA[1]);
        umma::prefetch_tmap(&p.tmB[0]); umma::prefetch_tmap(&p.tmB[1]);
        umma::prefetch_tmap(&p.tmC);
    }
    if (warp == 1) { umma::tmem_alloc_pair(tmem_slot, 512); umma::tmem_relinquish_pair(); }
    umma::tc_fence_before_sync();
    __syncthreads();
    umma::cluster_sync();  // the partner's barriers are initialised before anything is signalled on them
    umma::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    umma::pdl_launch_dependents();
    // The factors are weights, which no earlier kernel writes: the first tile's chunks are requested into L2
    // before this grid waits for its predecessor.
    if (warp == 0 && lane == 0 && tile_begin < tile_end) {
        const int n0 = tile_begin % p.tiles_n;
        for (int b = 0; b < 2; ++b)
            for (int c = 0; c < chunks; ++c) umma::tma_prefetch_2d(&p.tmB[b], c * BK, n0 * 128 + (int)rank * 64);
    }
    umma::pdl_wait();

    if (warp == 0 || warp == kPairProducer2) {
        // ---------------- TMA producers (both CTAs): own rows of the Z strip, own 64 rows of every factor chunk ----------------
        // Slot sequence of a tile: for the first tile of a row strip the strip's chunks (gate 0.., up 0..), then the
        // tile's G slots, then its Up slots.  The strip of the next row strip is thus fetched as far ahead as the
        // ring allows, while the last tiles of the current one are still being computed.
        const int pw = (warp == 0) ? 0 : 1;
        int stage = 0, cur_mp = -1, slot_no = 0;
        uint32_t phase = 0;
        bool ok = true;
        auto next_slot = [&]() { if (++stage == nslot) { stage = 0; phase ^= 1; } };
        for (int t = tile_begin; t < tile_end && ok; ++t) {
            const int mp = t / p.tiles_n, n = t - mp * p.tiles_n;
            const int m = 2 * mp + (int)rank;
            if (mp != cur_mp) {
                for (int b = 0; b < 2 && ok; ++b)
                    for (int c = 0; c < chunks; ++c) {
                        if (((slot_no++) & 1) != pw) { next_slot(); continue; }
                        ok = umma::mbar_wait_warp(&empty[stage], phase ^ 1, abort_flag);
                        if (!ok) break;
                        if (umma::elect_one()) {
                            if (leader) umma::mbar_expect_tx(&full[stage], 2 * kABytes);
                            umma::tma_load_2d_pair(ring + stage * kTsSlotBytes, &p.tmA[b], umma::map_to_rank(&full[stage], 0), c * BK, m * BM);
                        }
                        __syncwarp();
                        next_slot();
                    }
                cur_mp = mp;
            }
            for (int b = 0; b < 2 && ok; ++b)
                for (int c = 0; c < chunks; c += 2) {
                    if (((slot_no++) & 1) != pw) { next_slot(); continue; }  // the other producer's slot
                    ok = umma::mbar_wait_warp(&empty[stage], phase ^ 1, abort_flag);
                    if (!ok) break;
                    if (umma::elect_one()) {
                        const int nc = min(2, chunks - c);
                        if (leader) umma::mbar_expect_tx(&full[stage], 2 * nc * kTsChunkBytes);
                        const uint32_t bar = umma::map_to_rank(&full[stage], 0);
                        for (int j = 0; j < nc; ++j)
                            umma::tma_load_2d_pair(ring + stage * kTsSlotBytes + j * kTsChunkBytes, &p.tmB[b], bar, (c + j) * BK,
                                                   n * 128 + (int)rank * 64);
                    }
                    __syncwarp();
                    next_slot();
                }
        }
    } else if (warp == 1 || warp == 10) {
        if (leader) {  // ---------------- tcgen05 issuers (leader CTA only): warp 1 feeds G, warp 10 feeds Up ----------------
            // A thread issues one tcgen05.mma per ~55 cycles and an N = 128 MMA occupies the pipe for 64, so one
            // thread that also waits on barriers cannot keep the pipe fed.  Each branch has its own issuer and its
            // own accumulator hand-over; the two instruction streams share the pipe and drift apart, so that one
            // branch's MMAs run while the other's accumulator is being read out.
            // Two consumers on one ring with one-bit phase parities: a wait for fill f of a slot also passes while the
            // slot is still in fill f - 1, so no issuer may reach a slot whose previous fill belongs to the other
            // issuer and may be unfinished.  Within a row strip a slot always serves the same branch (12 slots are a
            // multiple of the 2 or 4 slots of a tile); across a strip change, where the strip's chunks shift the
            // pattern, `adone` and `aready` order every earlier fill before the first wait that follows.
            const int b = (warp == 1) ? 0 : 1;
            const int spb = (chunks + 1) / 2;  // ring slots per branch and tile
            const uint32_t idesc = umma::make_idesc(p.a_fmt, p.b_fmt, 2 * BM, 128);
            int stage = 0, cur_mp = -1, n = 0, mp = 0;
            uint32_t phase = 0, ph = 0, strip_phase = 0;
            bool ok = true;
            auto skip_slots = [&](int k) { stage += k; while (stage >= nslot) { stage -= nslot; phase ^= 1; } };
            if (tile_begin < tile_end) { mp = tile_begin / p.tiles_n; n = tile_begin - mp * p.tiles_n; }
            for (int t = tile_begin; t < tile_end && ok; ++t) {
                if (mp != cur_mp) {
                    if (b == 0) {
                        if (cur_mp >= 0) {  // both branches' MMAs of the previous strip have finished reading it
                            ok = umma::mbar_wait_warp(adone, strip_phase ^ 1, abort_flag);
                            if (!ok) break;
                        }
                        for (int bb = 0; bb < 2 && ok; ++bb)
                            for (int c = 0; c < chunks; ++c) {
                                ok = umma::mbar_wait_warp(&full[stage], phase, abort_flag);
                                if (!ok) break;
                                umma::tc_fence_after_sync();
                                if (umma::elect_one()) {
                                    const uint64_t sd = umma::smem_desc_sw128(umma::smem_u32(ring + stage * kTsSlotBytes));
#pragma unroll
                                    for (int kk = 0; kk < BK / 16; ++kk)
                                        tmem_cp_128x256b_pair(tmem_base + bb * 128 + c * 32 + kk * 8, sd + 2 * kk);
                                    umma::mma_commit_pair(&empty[stage]);
                                }
                                __syncwarp();
                                if (++stage == nslot) { stage = 0; phase ^= 1; }
                            }
                        if (!ok) break;
                        if (umma::elect_one()) umma::mma_commit_pair(aready);  // the strips are in TMEM
                        __syncwarp();
                    } else {
                        skip_slots(2 * chunks);
                        ok = umma::mbar_wait_warp(aready, strip_phase, abort_flag);
                        if (!ok) break;
                        umma::tc_fence_after_sync();
                    }
                    strip_phase ^= 1;
                    cur_mp = mp;
                }
                if (b == 1) skip_slots(spb);  // G's slots of this tile
                // this branch's accumulator columns have been read out by every epilogue warp of both CTAs
                ok = umma::mbar_wait_warp(&tempty[b], ph ^ 1, abort_flag);
                if (!ok) break;
                umma::tc_fence_after_sync();
                for (int c = 0; c < chunks; c += 2) {
                    ok = umma::mbar_wait_warp(&full[stage], phase, abort_flag);
                    if (!ok) break;
                    if (umma::elect_one()) {
                        const uint64_t bd0 = umma::smem_desc_sw128(umma::smem_u32(ring + stage * kTsSlotBytes));
                        const uint32_t dcol = tmem_base + 256 + b * 128, acol = tmem_base + b * 128 + c * 32;
                        const int nc = min(2, chunks - c);
                        for (int j = 0; j < nc; ++j)
#pragma unroll
                            for (int kk = 0; kk < BK / 16; ++kk)
                                mma_f16_ts_pair(dcol, acol + j * 32 + kk * 8, bd0 + j * (kTsChunkBytes >> 4) + 2 * kk, idesc,
                                                (c + j > 0) || (kk > 0));
                        umma::mma_commit_pair(&empty[stage]);
                    }
                    __syncwarp();
                    if (++stage == nslot) { stage = 0; phase ^= 1; }
                }
                if (!ok) break;
                const bool last_of_strip = (t + 1 == tile_end) || (n + 1 == p.tiles_n);
                if (umma::elect_one()) {
                    umma::mma_commit_pair(&tfull[b]);
                    if (last_of_strip) umma::mma_commit_pair(adone);
                }
                __syncwarp();
                ph ^= 1;
                if (b == 0) skip_slots(spb);  // Up's slots of this tile
                if (++n == p.tiles_n) { n = 0; ++mp; }
            }
        }
    } else if (warp < 2 + kEpiWarps) {  // ---------------- epilogue warps 2..9 (both CTAs, own 128 rows) ----------------
        const int q = warp & 3, half = (warp - 2) >> 2;
        uint32_t ph = 0;
        bool ok = true;
        const uint32_t tempty_g = umma::map_to_rank(&tempty[0], 0), tempty_u = umma::map_to_rank(&tempty[1], 0);
        unsigned char* my_stage = stage_out + (warp - 2) * 4096;
        const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + 256 + half * 64;
        int mp = tile_begin / p.tiles_n, n = tile_begin - mp * p.tiles_n;
        for (int t = tile_begin; t < tile_end && ok; ++t, (++n == p.tiles_n ? (n = 0, ++mp) : 0)) {
            const int m = 2 * mp + (int)rank;
            uint32_t rr[2][32], sg[32];
            // G: this warp's 32 rows x 64 columns into registers, then its columns go back to the issuer
            ok = umma::mbar_wait_warp(&tfull[0], ph, abort_flag);
            if (!ok) break;
            umma::tc_fence_after_sync();
            umma::tmem_ld32(taddr, rr[0]);
            umma::tmem_ld32(taddr + 32, rr[1]);
            umma::tmem_ld_wait();
            umma::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) umma::mbar_arrive_cluster(tempty_g);
            // SiLU(G) = h + h tanh(h), h = G / 2, as packed fp16 while the tensor pipe is still busy with Up: the
            // MUFU-bound part of the epilogue (1024 cycles per tile and scheduler) hides behind Up's MMAs.
#pragma unroll
            for (int hh = 0; hh < 2; ++hh)
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const __half2 h2 = __floats2half2_rn(0.5f * __uint_as_float(rr[hh][2 * j]), 0.5f * __uint_as_float(rr[hh][2 * j + 1]));
                    uint32_t t2;
                    asm("tanh.approx.f16x2 %0, %1;" : "=r"(t2) : "r"(*reinterpret_cast<const uint32_t*>(&h2)));
                    const __half2 s2 = __hfma2(h2, *reinterpret_cast<const __half2*>(&t2), h2);
                    sg[hh * 16 + j] = *reinterpret_cast<const uint32_t*>(&s2);
                }
            // Up likewise, multiplied in as it arrives
            ok = umma::mbar_wait_warp(&tfull[1], ph, abort_flag);
            if (!ok) break;
            umma::tc_fence_after_sync();
            umma::tmem_ld32(taddr + 128, rr[0]);
            umma::tmem_ld32(taddr + 160, rr[1]);
            umma::tmem_ld_wait();
            umma::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) umma::mbar_arrive_cluster(tempty_u);
            ph ^= 1;
#pragma unroll
            for (int hh = 0; hh < 2; ++hh)
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const __half2 u2 = __floats2half2_rn(__uint_as_float(rr[hh][2 * j]), __uint_as_float(rr[hh][2 * j + 1]));
                    const __half2 r2 = __hmul2(*reinterpret_cast<const __half2*>(&sg[hh * 16 + j]), u2);
                    sg[hh * 16 + j] = *reinterpret_cast<const uint32_t*>(&r2);
                }
            umma::bulk_wait_read0();  // the previous store has finished reading the staging tile
            __syncwarp();
#pragma unroll
            for (int ch = 0; ch < 8; ++ch)
                *reinterpret_cast<uint4*>(my_stage + lane * 128 + ((ch ^ (lane & 7)) << 4)) =
                    make_uint4(sg[4 * ch], sg[4 * ch + 1], sg[4 * ch + 2], sg[4 * ch + 3]);
            umma::fence_proxy_async_smem();
            __syncwarp();
            const int col = n * 128 + half * 64;
            if (lane == 0 && col < p.N && m * BM + q * 32 < p.M) {
                umma::tma_store_2d(&p.tmC, my_stage, col, m * BM + q * 32);
                umma::bulk_commit();
            }
        }
        umma::bulk_wait_all();
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
    if (warp == 1) { umma::tc_fence_after_sync(); umma::tmem_dealloc_pair(tmem_base, 512); }
}

}  // namespace tensorpath
