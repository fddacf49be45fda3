// Gate+up expansion, SiLU(G).*Up and the first half of the down chain in ONE kernel, for ranks up to 128:
//     Zd_part[T, r_down] = (SiLU(Zg Ug^T) .* (Zu Uu^T))[:, F] Vd[:, F]^T        (F: a segment of the ffn columns)
// H never exists in global memory: the epilogue warps write each [128 x 128] fp16 tile of H into shared memory in
// the swizzled K-major layout a tcgen05 A operand has, and the tile is multiplied by the matching [r_down x 128]
// tile of Vd into a Zd accumulator that stays in tensor memory while the CTA pair walks its ffn tiles.  This is the
// paper's "execute entirely within on-chip memory" (Section 4.2) carried into the second half of the MLP; at
// r = 128 the two-kernel form moves 4 ffn bytes per token through HBM for H (write + read), more than the
// tensor work takes.
//
// TMEM columns (512): [0, 64) gate strip, [64, 128) up strip (fp16 pairs: 32-bit column c = k 2c, 2c + 1; r <= 128),
// [128, 256) Zd accumulator (r_down <= 128), [256, 384) G accumulator, [384, 512) Up accumulator.
//
// Work units: (row-strip pair of 256 tokens) x (one of S segments of the ffn tiles).  A unit loads its Z strip into
// TMEM, walks its ffn tiles and leaves one fp32 partial of Zd (split-K over ffn with S splits, summed by the
// reduction kernel that follows).  Units are dealt round-robin to the CTA pairs.
//
// CTA pair (cta_group::2) as in gateup_ts.cuh: each CTA owns 128 token rows and loads 64 rows of every factor tile.
// Ring slots (16 KiB): a [128 x 64] strip chunk, or two [64 x 64] chunks of Ug / Uu / Vd; a tile takes three slots
// (G, Up, Vd) and the ring has a multiple of three, so inside a unit a slot always serves the same consumer.
// Warps: 0 and 11 TMA producers (alternate slots); 1 issues G and copies the strips, 10 issues Up, 12 issues the Zd
// MMAs (one thread issues a tcgen05.mma about every 55 cycles: two issuers for the 24 MMAs of a tile were the
// kernel's bound); 2-9 epilogue (lane quadrant x column half).  Ring slots change hands between the issuers only
// at unit boundaries, where `adone` / `aready` order every earlier fill before the first wait that follows
// (one-bit phase parities cannot tell a fill that has not landed from the one two fills later).  Every wait is bounded.
#pragma once
#include "gateup_ts.cuh"

namespace tensorpath {

constexpr int kFuSlots = 12;
constexpr int kFuHBufs = 1;                                 // H tiles in shared memory (one: its Zd MMAs end long before the epilogue has the next tile)
constexpr int kFuThreads = 13 * 32;                          // the pair kernels' twelve warps + warp 12, the Zd issuer
constexpr int kFuZdWarp = 12;
constexpr int kFuHBytes = kEpiWarps * 4096;                 // one [128 x 128] fp16 tile of H per CTA
constexpr int kFuBarrierBytes = (2 * kFuSlots + 16) * 8 + 16;
constexpr int kFuSmemBytes = 1024 + kFuSlots * kTsSlotBytes + kFuHBufs * kFuHBytes + kFuBarrierBytes;
static_assert(kFuSlots % 3 == 0, "inside a unit a ring slot must always serve the same issuer");
static_assert(kFuSmemBytes <= 232448, "shared memory of one SM");

// p: tmA[0/1] = Zg / Zu ([T, r] fp16, box [128, 64]); tmB[0/1] = Ug / Uu ([ffn, r] fp16, box [64, 64]);
// tmC = Vd ([r_down, ffn] fp16, box [64, 64]); C = fp32 partials [ksplit][T, ldc], ldc = r_down,
// split_stride = T r_down; M = T, N = ffn, K = r <= 128; tiles_m = ceil(T / 128), tiles_n = ceil(ffn / 128),
// chunks_total = ceil(r / 64); ksplit = S segments per row-strip pair (S <= tiles_n); stages = kFuSlots.
__global__ void __launch_bounds__(kFuThreads, 1) gateup_down1_ts_pair_kernel(const __grid_constant__ GemmParams p) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = smem_raw + ((1024u - (umma::smem_u32(smem_raw) & 1023u)) & 1023u);
    unsigned char* ring = smem;
    unsigned char* hbuf = ring + kFuSlots * kTsSlotBytes;    // the H tile(s), 1024-byte aligned
    uint64_t* full = reinterpret_cast<uint64_t*>(hbuf + kFuHBufs * kFuHBytes);
    uint64_t* empty = full + kFuSlots;
    uint64_t* tfull = empty + kFuSlots;   // [branch]
    uint64_t* tempty = tfull + 2;         // [branch]
    uint64_t* adone = tempty + 2;
    uint64_t* aready = adone + 1;
    uint64_t* hready = aready + 1;        // [H buffer] written by the epilogue warps of both CTAs (leader's copy counts)
    uint64_t* hfree = hready + 2;         // [H buffer] its Zd MMAs have completed
    uint64_t* zfull = hfree + 2;          // the unit's Zd accumulator is complete
    uint64_t* zempty = zfull + 1;         // ... and has been read out by every epilogue warp of both CTAs
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(zempty + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = umma::cluster_ctarank();
    const bool leader = rank == 0;
    const int cluster_id = blockIdx.x >> 1, nclusters = gridDim.x >> 1;
    const int pairs_m = (p.tiles_m + 1) / 2;
    const int S = p.ksplit, units = pairs_m * S;
    const int chunks = p.chunks_total, nslot = kFuSlots;
    const int spb = (chunks + 1) / 2;     // ring slots of one branch's factor tile (1 for r <= 128)
    auto unit_tiles = [&](int u, int& mp, int& seg, int& n0, int& n1) {
        mp = u / S; seg = u - mp * S;
        n0 = (int)((long)seg * p.tiles_n / S); n1 = (int)((long)(seg + 1) * p.tiles_n / S);
    };

    if (threadIdx.x == 0) {
        for (int s = 0; s < nslot; ++s) { umma::mbar_init(&full[s], 1); umma::mbar_init(&empty[s], 1); }
        for (int a = 0; a < 2; ++a) {
            umma::mbar_init(&tfull[a], 1); umma::mbar_init(&tempty[a], 2 * kEpiWarps);
            umma::mbar_init(&hready[a], 2 * kEpiWarps); umma::mbar_init(&hfree[a], 1);
        }
        umma::mbar_init(adone, 3);   // one commit per issuer warp at the end of a unit
        umma::mbar_init(aready, 1);
        umma::mbar_init(zfull, 1);
        umma::mbar_init(zempty, 2 * kEpiWarps);
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
    umma::pdl_wait();

    if (warp == 0 || warp == kPairProducer2) {
        // ---------------- TMA producers (both CTAs): own rows of the Z strip, own 64 rows of every factor tile ----------------
        // Slot sequence of a unit: the strip's chunks (gate 0.., up 0..), then per tile its G, Up and Vd slots.
        const int pw = (warp == 0) ? 0 : 1;
        int stage = 0, slot_no = 0;
        uint32_t phase = 0;
        bool ok = true;
        auto next_slot = [&]() { if (++stage == nslot) { stage = 0; phase ^= 1; } };
        auto mine = [&]() -> bool {   // false: the other producer's slot (skipped); true: slot is free and ours
            if (((slot_no++) & 1) != pw) { next_slot(); return false; }
            ok = umma::mbar_wait_warp(&empty[stage], phase ^ 1, abort_flag);
            return ok;
        };
        for (int u = cluster_id; u < units && ok; u += nclusters) {
            int mp, seg, n0, n1;
            unit_tiles(u, mp, seg, n0, n1);
            const int m = 2 * mp + (int)rank;
            for (int b = 0; b < 2 && ok; ++b)
                for (int c = 0; c < chunks && ok; ++c) {
                    if (!mine()) continue;
                    if (umma::elect_one()) {
                        if (leader) umma::mbar_expect_tx(&full[stage], 2 * kABytes);
                        umma::tma_load_2d_pair(ring + stage * kTsSlotBytes, &p.tmA[b], umma::map_to_rank(&full[stage], 0), c * BK, m * BM);
                    }
                    __syncwarp();
                    next_slot();
                }
            for (int n = n0; n < n1 && ok; ++n) {
                for (int b = 0; b < 2 && ok; ++b)
                    for (int c = 0; c < chunks && ok; c += 2) {
                        if (!mine()) continue;
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
                if (!ok || !mine()) continue;
                if (umma::elect_one()) {   // Vd[this CTA's 64 rows of r_down, the tile's 128 ffn columns] as two K chunks
                    if (leader) umma::mbar_expect_tx(&full[stage], 2 * 2 * kTsChunkBytes);
                    const uint32_t bar = umma::map_to_rank(&full[stage], 0);
                    for (int j = 0; j < 2; ++j)
                        umma::tma_load_2d_pair(ring + stage * kTsSlotBytes + j * kTsChunkBytes, &p.tmC, bar, n * 128 + j * BK, (int)rank * 64);
                }
                __syncwarp();
                next_slot();
            }
        }
    } else if (warp == 1) {
        if (leader) {  // ---------------- tcgen05 issuer of G; copies the strips into TMEM ----------------
            const uint32_t idesc = umma::make_idesc(p.a_fmt, p.b_fmt, 2 * BM, 128);
            int stage = 0;
            uint32_t phase = 0, ph = 0, strip_phase = 0;
            bool ok = true, first = true;
            auto skip_slots = [&](int k) { stage += k; while (stage >= nslot) { stage -= nslot; phase ^= 1; } };
            for (int u = cluster_id; u < units && ok; u += nclusters) {
                int mp, seg, n0, n1;
                unit_tiles(u, mp, seg, n0, n1);
                if (!first) {  // both branches' MMAs of the previous unit have finished reading its strips
                    ok = umma::mbar_wait_warp(adone, strip_phase ^ 1, abort_flag);
                    if (!ok) break;
                }
                first = false;
                for (int bb = 0; bb < 2 && ok; ++bb)
                    for (int c = 0; c < chunks; ++c) {
                        ok = umma::mbar_wait_warp(&full[stage], phase, abort_flag);
                        if (!ok) break;
                        umma::tc_fence_after_sync();
                        if (umma::elect_one()) {
                            const uint64_t sd = umma::smem_desc_sw128(umma::smem_u32(ring + stage * kTsSlotBytes));
#pragma unroll
                            for (int kk = 0; kk < BK / 16; ++kk)
                                tmem_cp_128x256b_pair(tmem_base + bb * 64 + c * 32 + kk * 8, sd + 2 * kk);
                            umma::mma_commit_pair(&empty[stage]);
                        }
                        __syncwarp();
                        if (++stage == nslot) { stage = 0; phase ^= 1; }
                    }
                if (!ok) break;
                if (umma::elect_one()) umma::mma_commit_pair(aready);  // the strips are in TMEM
                __syncwarp();
                strip_phase ^= 1;
                for (int n = n0; n < n1 && ok; ++n) {
                    // G's accumulator columns have been read out by every epilogue warp of both CTAs
                    ok = umma::mbar_wait_warp(&tempty[0], ph ^ 1, abort_flag);
                    if (!ok) break;
                    umma::tc_fence_after_sync();
                    for (int c = 0; c < chunks; c += 2) {
                        ok = umma::mbar_wait_warp(&full[stage], phase, abort_flag);
                        if (!ok) break;
                        if (umma::elect_one()) {
                            const uint64_t bd0 = umma::smem_desc_sw128(umma::smem_u32(ring + stage * kTsSlotBytes));
                            const uint32_t dcol = tmem_base + 256, acol = tmem_base + c * 32;
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
                    if (umma::elect_one()) {
                        umma::mma_commit_pair(&tfull[0]);
                        if (n + 1 == n1) umma::mma_commit_pair(adone);
                    }
                    __syncwarp();
                    ph ^= 1;
                    skip_slots(spb + 1);  // Up's and Vd's slots of this tile
                }
            }
        }
    } else if (warp == 10) {
        if (leader) {  // ---------------- tcgen05 issuer of Up ----------------
            const uint32_t idesc = umma::make_idesc(p.a_fmt, p.b_fmt, 2 * BM, 128);
            int stage = 0;
            uint32_t phase = 0, ph = 0, strip_phase = 0;
            bool ok = true;
            auto skip_slots = [&](int k) { stage += k; while (stage >= nslot) { stage -= nslot; phase ^= 1; } };
            for (int u = cluster_id; u < units && ok; u += nclusters) {
                int mp, seg, n0, n1;
                unit_tiles(u, mp, seg, n0, n1);
                skip_slots(2 * chunks);
                ok = umma::mbar_wait_warp(aready, strip_phase, abort_flag);
                if (!ok) break;
                umma::tc_fence_after_sync();
                strip_phase ^= 1;
                for (int n = n0; n < n1 && ok; ++n) {
                    skip_slots(spb);  // G's slots of this tile
                    ok = umma::mbar_wait_warp(&tempty[1], ph ^ 1, abort_flag);
                    if (!ok) break;
                    umma::tc_fence_after_sync();
                    for (int c = 0; c < chunks; c += 2) {
                        ok = umma::mbar_wait_warp(&full[stage], phase, abort_flag);
                        if (!ok) break;
                        if (umma::elect_one()) {
                            const uint64_t bd0 = umma::smem_desc_sw128(umma::smem_u32(ring + stage * kTsSlotBytes));
                            const uint32_t dcol = tmem_base + 384, acol = tmem_base + 64 + c * 32;
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
                    if (umma::elect_one()) {
                        umma::mma_commit_pair(&tfull[1]);
                        if (n + 1 == n1) umma::mma_commit_pair(adone);
                    }
                    __syncwarp();
                    ph ^= 1;
                    skip_slots(1);  // Vd's slot of this tile
                }
            }
        }
    } else if (warp == kFuZdWarp) {
        if (leader) {  // ---------------- tcgen05 issuer of Zd += H Vd^T (a tile behind the other two by construction) ----------------
            const uint32_t idesc = umma::make_idesc(p.a_fmt, p.b_fmt, 2 * BM, 128);
            int stage = 0;
            uint32_t phase = 0, strip_phase = 0;
            int g = 0;            // tiles handled so far by this CTA pair: H buffer g % kFuHBufs, its phase (g / kFuHBufs) & 1
            int ui = 0;           // units handled so far
            bool ok = true;
            auto skip_slots = [&](int k) { stage += k; while (stage >= nslot) { stage -= nslot; phase ^= 1; } };
            for (int u = cluster_id; u < units && ok; u += nclusters, ++ui) {
                int mp, seg, n0, n1;
                unit_tiles(u, mp, seg, n0, n1);
                skip_slots(2 * chunks);
                // every issuer has finished the previous unit (its ring slots are consumed): see `adone`
                ok = umma::mbar_wait_warp(aready, strip_phase, abort_flag);
                if (!ok) break;
                strip_phase ^= 1;
                for (int n = n0; n < n1 && ok; ++n, ++g) {
                    skip_slots(2 * spb);  // G's and Up's slots of this tile
                    const int hb = g % kFuHBufs;
                    ok = umma::mbar_wait_warp(&hready[hb], (uint32_t)(g / kFuHBufs) & 1u, abort_flag) &&
                         umma::mbar_wait_warp(&full[stage], phase, abort_flag);
                    // the accumulator of the previous unit has been read out before the first MMA overwrites it
                    if (ok && n == n0) ok = umma::mbar_wait_warp(zempty, (uint32_t)(ui & 1) ^ 1u, abort_flag);
                    if (!ok) break;
                    umma::tc_fence_after_sync();
                    if (umma::elect_one()) {
                        const uint32_t ha = umma::smem_u32(hbuf + hb * kFuHBytes), va = umma::smem_u32(ring + stage * kTsSlotBytes);
#pragma unroll
                        for (int j = 0; j < 2; ++j) {
                            const uint64_t ad = umma::smem_desc_sw128(ha + j * (kFuHBytes / 2)), bd = umma::smem_desc_sw128(va + j * kTsChunkBytes);
#pragma unroll
                            for (int kk = 0; kk < BK / 16; ++kk)
                                umma::mma_f16_ss_pair(tmem_base + 128, ad + 2 * kk, bd + 2 * kk, idesc, n > n0 || j > 0 || kk > 0);
                        }
                        umma::mma_commit_pair(&empty[stage]);
                        umma::mma_commit_pair(&hfree[hb]);
                        if (n + 1 == n1) { umma::mma_commit_pair(zfull); umma::mma_commit_pair(adone); }
                    }
                    __syncwarp();
                    if (++stage == nslot) { stage = 0; phase ^= 1; }
                }
            }
        }
    } else if (warp < 2 + kEpiWarps) {  // ---------------- epilogue warps 2..9 (both CTAs, own 128 rows) ----------------
        const int q = warp & 3, half = (warp - 2) >> 2;
        uint32_t ph = 0;
        bool ok = true;
        const uint32_t tempty_g = umma::map_to_rank(&tempty[0], 0), tempty_u = umma::map_to_rank(&tempty[1], 0);
        const uint32_t hready_l[2] = {umma::map_to_rank(&hready[0], 0), umma::map_to_rank(&hready[1], 0)};
        const uint32_t zempty_l = umma::map_to_rank(zempty, 0);
        // this warp's [32 rows x 64 columns] of an H tile: rows 32 q .. of the K chunk `half` ([128 rows x 128 B], swizzled)
        const int my_off = half * (kFuHBytes / 2) + q * 4096;
        const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + 256 + half * 64;
        const uint32_t taddr_zd = tmem_base + ((uint32_t)(q * 32) << 16) + 128 + half * 64;
        int g = 0, ui = 0;
        for (int u = cluster_id; u < units && ok; u += nclusters, ++ui) {
            int mp, seg, n0, n1;
            unit_tiles(u, mp, seg, n0, n1);
            const int m = 2 * mp + (int)rank;
            for (int n = n0; n < n1 && ok; ++n, ++g) {
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
                // SiLU(G) = h + h tanh(h), h = G / 2, as packed fp16 while the tensor pipe is busy with Up
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
                // H tile into shared memory as the A operand of Zd += H Vd^T; the buffer's previous tile has been multiplied
                const int hb = g % kFuHBufs;
                ok = umma::mbar_wait_warp(&hfree[hb], ((uint32_t)(g / kFuHBufs) & 1u) ^ 1u, abort_flag);
                if (!ok) break;
                unsigned char* dst = hbuf + hb * kFuHBytes + my_off;
#pragma unroll
                for (int ch = 0; ch < 8; ++ch)
                    *reinterpret_cast<uint4*>(dst + lane * 128 + ((ch ^ (lane & 7)) << 4)) =
                        make_uint4(sg[4 * ch], sg[4 * ch + 1], sg[4 * ch + 2], sg[4 * ch + 3]);
                umma::fence_proxy_async_smem();   // generic-proxy writes become visible to the tensor core's reads
                __syncwarp();
                if (lane == 0) umma::mbar_arrive_cluster(hready_l[hb]);
            }
            if (!ok) break;
            // the unit's Zd accumulator: this warp's 32 rows x 64 columns as an fp32 partial of the split over ffn
            ok = umma::mbar_wait_warp(zfull, (uint32_t)(ui & 1), abort_flag);
            if (!ok) break;
            umma::tc_fence_after_sync();
            uint32_t zz[2][32];
            umma::tmem_ld32(taddr_zd, zz[0]);
            umma::tmem_ld32(taddr_zd + 32, zz[1]);
            umma::tmem_ld_wait();
            umma::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) umma::mbar_arrive_cluster(zempty_l);
            const int row = m * BM + q * 32 + lane;
            if (row < p.M) {
                float* out = reinterpret_cast<float*>(p.C) + (long)seg * p.split_stride + (long)row * p.ldc;
#pragma unroll
                for (int hh = 0; hh < 2; ++hh)
#pragma unroll
                    for (int j = 0; j < 32; j += 4) {
                        const int col = half * 64 + hh * 32 + j;
                        if (col + 4 <= (int)p.ldc)
                            *reinterpret_cast<float4*>(out + col) = make_float4(__uint_as_float(zz[hh][j]), __uint_as_float(zz[hh][j + 1]),
                                                                                __uint_as_float(zz[hh][j + 2]), __uint_as_float(zz[hh][j + 3]));
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
    if (warp == 1) { umma::tc_fence_after_sync(); umma::tmem_dealloc_pair(tmem_base, 512); }
}

}  // namespace tensorpath
