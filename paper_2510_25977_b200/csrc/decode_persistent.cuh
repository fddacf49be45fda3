// Decode (T <= 32) path: the whole factored MLP as ONE persistent kernel, one CTA per SM (a
// programmatic dependent launch; a cooperative launch on request).  At small T the MLP is a stream
// of 6 r (d + ffn) weight bytes through a chain of three dependent products, so the design goal is
// that HBM never waits for the chain:
//
//  * Create-time packing gives every CTA one contiguous block per phase, already in the order and
//    layout its warps consume, so the producer warp moves it with a few large 1-D bulk copies into a
//    ring of 32 KiB shared-memory slots and only ever blocks on ring capacity.  The blocks of all
//    three phases are requested back to back: factors of later phases stream in while earlier
//    phases compute and while the grid-wide barriers between the phases are crossed.
//  * Work is split so that no phase needs a cross-CTA reduction except the one the algebra forces:
//      phase A  Z  = X [Vg; Vu]^T     CTA b owns ~2r/G rows of [Vg; Vu] over the full K = d
//                                     (X is small and is streamed by every CTA); plain stores of Z.
//      phase B  Zd += (SiLU(Zg Ug^T) .* (Zu Uu^T))[:, cols_b] Vd[:, cols_b]^T
//                                     CTA b owns ~ffn/(16 G) tiles of 16 ffn columns; split-K over
//                                     ffn is inherent, reduced with vector fp32 reductions into a
//                                     few copies of Zd that phase D adds up.
//      phase D  Y  = Zd Ud^T (+ resid) CTA b owns ~d/(16 G) tiles of 16 output columns.
//    Units are dealt out evenly (counts differ by at most one), not in fixed 64-wide slices.
//  * Products run on mma.sync m16n8k16 with fp32 accumulation.  All factor data is stored as
//    "panels" of [16 rows x 16 k] (512 B): a thread's fragment is one 8-byte load and a half-warp
//    reads 128 contiguous bytes, so shared-memory reads are conflict-free without swizzling.
//    The k positions inside a 16-step are permuted identically for both operands (thread tig takes
//    k = 4 tig .. 4 tig + 3), which leaves the sum unchanged.
//  * Phase A multiplies bf16 X by the bf16 V factors exactly.  Z, H and Zd are rounded to fp16
//    (|rel| <= 2^-12) and the second-stage factors Ug, Uu, Vd, Ud are re-encoded bf16 -> fp16 at
//    create time (exact inside the fp16 normal range; a value outside it disables this path).
//  * Grid barrier: arrivals are fire-and-forget release-reductions on a counter that only grows;
//    the launch number is read from memory at kernel start (the last CTA action of a launch bumps
//    it), so a replayed CUDA graph needs no per-launch parameter.  Every wait is bounded.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "umma.cuh"

namespace dpersist {

constexpr int kNW = 12;                  // consumer warps
constexpr int kConsumers = kNW * 32;
constexpr int kThreads = kConsumers + 32;  // + one producer warp
constexpr int kSlotBytes = 32768;
constexpr int kMaxSlots = 8;
constexpr int kCopiesZd = 2;             // replicated reduction targets of phase B
constexpr int kPanel = 512;              // bytes of a [16 x 16] 16-bit panel
constexpr int kZdPitch = 32;              // floats per Zd row (token index fastest; T <= 32)
constexpr int kBarStride = 16;           // u64 words between the barrier words (128 B apart)

// Even deal of `units` work units over G CTAs: CTA b gets count units starting at start.
struct Part { int start, count; };
__host__ __device__ inline Part part(int units, int G, int b) {
    const int base = units / G, rem = units % G;
    Part p;
    p.count = base + (b < rem ? 1 : 0);
    p.start = b * base + (b < rem ? b : rem);
    return p;
}
__host__ __device__ inline int ceil_div(int a, int b) { return (a + b - 1) / b; }
// Row pitch in bytes for fragment reads of 8 bytes per thread: a multiple of 32 that is an odd
// multiple of 32, so four consecutive rows start in four different 32-byte bank groups.
__host__ __device__ inline int odd32(int bytes) {
    int q = (bytes + 31) / 32;
    if ((q & 1) == 0) ++q;
    return q * 32;
}

// Shapes and derived constants shared by host planning, the packing kernels and the main kernel.
struct Shape {
    int T, d, ffn, r, rd, G;
    __host__ __device__ int ksd() const { return ceil_div(d, 16); }     // k16 steps of phase A
    __host__ __device__ int ksr() const { return ceil_div(r, 16); }     // k16 steps of the gate/up expansion
    __host__ __device__ int zt() const { return ceil_div(rd, 16); }     // 16-row tiles of Zd = k16 steps of phase D
    __host__ __device__ int units_a() const { return 2 * r; }           // rows of [Vg; Vu]
    __host__ __device__ int units_b() const { return ceil_div(ffn, 16); }
    __host__ __device__ int units_d() const { return ceil_div(d, 16); }
    __host__ __device__ int max_a() const { return ceil_div(units_a(), G); }
    __host__ __device__ int max_b() const { return ceil_div(units_b(), G); }
    __host__ __device__ int max_d() const { return ceil_div(units_d(), G); }
    // k16 steps per ring group of the gate/up expansion for a CTA with `tiles` tiles (2 tasks per tile)
    __host__ __device__ int kg_b(int tiles) const { int k = kSlotBytes / kPanel / (2 * tiles); return k < ksr() ? k : ksr(); }
    // Zd row tiles per ring group of the first half of the down chain
    __host__ __device__ int gz_b(int tiles) const { int g = kSlotBytes / kPanel / tiles; return g < zt() ? g : zt(); }
    // k16 steps per ring group of phase D for a CTA with `tiles` output tiles
    __host__ __device__ int kg_d(int tiles) const { int k = kSlotBytes / kPanel / tiles; return k < zt() ? k : zt(); }
};

// Shared-memory layout behind the ring (byte offsets from the end of the ring's barriers).
struct Layout {
    int rows;       // token rows held (8 NT)
    int ga;         // k16 steps per phase-A group
    int a_v_off;    // offset of the V block inside a phase-A slot (the X part sits at 0)
    int xres_bytes; // size of the resident X buffer in front of the ring (0: X travels with the groups)
    int pitch_x;    // bytes between token rows of X inside a slot
    int pitch_z, pitch_d, pitch_h, gp;  // activation pitches (bytes) and the fp32 G pitch (floats)
    int zs, hs, gs, red, xn, total;  // xn: normalised X rows of one phase-A group (fused RMSNorm only)
};
__host__ __device__ inline Layout make_layout(const Shape& s, int NT, int NTA, bool fused_norm, bool x_res) {
    Layout L;
    L.rows = 8 * NT;
    // phase-A slot: the group's columns of X first, then [ga steps][rows of the CTA][32 B] of V.
    // X comes either as one 3-D TMA box [ga/4 column blocks][T rows][64 columns] with the 128-byte swizzle
    // (x_tma; ga*32 bytes per token), or as T row pieces of ga*32 bytes at a pitch of ga*32 + 32 bytes.
    // With x_res the whole of X (T d 2 bytes, one TMA box, same swizzled layout) sits in its own buffer in front
    // of the ring for the life of phase A, and the slots carry V only.
    const int ma = s.max_a() > 0 ? s.max_a() : 1;
    int ga_max = (x_res ? kSlotBytes / (32 * ma) : (kSlotBytes - 32 * s.T) / (32 * (ma + s.T))) & ~3;
    if (ga_max > 1024) ga_max = 1024;  // TMA box: at most 256 column blocks
    if (ga_max < 4) ga_max = 4;  // the host rejects layouts whose slot does not fit
    const int ngroups = ceil_div(s.ksd(), ga_max);
    L.ga = (ceil_div(s.ksd(), ngroups) + 3) & ~3;
    L.pitch_x = L.ga * 32 + 32;
    L.a_v_off = x_res ? 0 : (s.T * L.pitch_x + 127) & ~127;
    L.xres_bytes = x_res ? (s.T * s.d * 2 + 1023) & ~1023 : 0;
    const int r16 = s.ksr() * 16, rd16 = s.zt() * 16, tm = s.max_b() > 0 ? s.max_b() : 1;
    L.pitch_z = odd32(2 * r16 * 2);
    L.pitch_d = odd32(rd16 * 2);
    L.pitch_h = odd32(tm * 16 * 2);
    L.gp = tm * 16 + 1;
    const int zbytes = L.rows * (L.pitch_z > L.pitch_d ? L.pitch_z : L.pitch_d);
    const int MT = (NT + 1) / 2;
    const int red_a = kNW * 16 * MT * 8 * NTA * 4, red_d = kNW * 16 * (L.rows + 1) * 4;
    L.zs = 0;
    L.hs = L.zs + ((zbytes + 127) & ~127);
    L.gs = L.hs + ((L.rows * L.pitch_h + 127) & ~127);
    L.red = L.gs + ((L.rows * L.gp * 4 + 127) & ~127);
    L.xn = L.red + (((red_a > red_d ? red_a : red_d) + 127) & ~127);
    L.total = L.xn + (fused_norm ? ((s.T * L.pitch_x + 127) & ~127) : 0);
    return L;
}
constexpr int kRingOverhead = 1024 + (2 * kMaxSlots + 4) * 8;  // alignment slack + barriers + abort word

// bf16 -> fp16 of 8 packed values; exact inside the fp16 normal range.  Values whose magnitude
// exceeds the fp16 maximum raise *flag (the caller then keeps to the bf16 kernels).
__device__ __forceinline__ uint4 bf16x8_to_f16x8(uint4 v, int* flag) {
    const __nv_bfloat16* b = reinterpret_cast<const __nv_bfloat16*>(&v);
    uint4 o;
    __half* h = reinterpret_cast<__half*>(&o);
    bool over = false;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const float f = __bfloat162float(b[i]);
        over = over || !(fabsf(f) <= 65504.f);
        h[i] = __float2half_rn(f);
    }
    if (over) atomicOr(flag, 1);
    return o;
}

// ---- create-time packing: one CTA of the packing grid per CTA of the decode grid --------------
// Phase A block of CTA b: rows [start, start+count) of [Vg; Vu] as [k16 step][row][16 k] bf16.
__global__ void __launch_bounds__(256)
pack_a_kernel(const __nv_bfloat16* __restrict__ Vg, const __nv_bfloat16* __restrict__ Vu, Shape s,
              unsigned char* __restrict__ out) {
    const Part pa = part(s.units_a(), s.G, blockIdx.x);
    const int ksd = s.ksd();
    unsigned char* dst = out + (size_t)pa.start * ksd * 32;
    const int total = pa.count * ksd * 2;
    for (int idx = threadIdx.x; idx < total; idx += blockDim.x) {
        const int st = idx / (pa.count * 2), rem = idx - st * pa.count * 2, row = rem >> 1, half = rem & 1;
        const int gr = pa.start + row, k = st * 16 + half * 8;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (k < s.d) v = *reinterpret_cast<const uint4*>((gr < s.r ? Vg + (size_t)gr * s.d : Vu + (size_t)(gr - s.r) * s.d) + k);
        *reinterpret_cast<uint4*>(dst + (size_t)idx * 16) = v;
    }
}

// Gate/up block of CTA b: [k group][task = 2 tile + (0 gate | 1 up)][k16 step in group][16 rows][16 k] fp16.
__global__ void __launch_bounds__(256)
pack_b_kernel(const __nv_bfloat16* __restrict__ Ug, const __nv_bfloat16* __restrict__ Uu, Shape s,
              unsigned char* __restrict__ out, int* flag) {
    const Part pb = part(s.units_b(), s.G, blockIdx.x);
    if (pb.count == 0) return;
    const int ksr = s.ksr(), ntask = 2 * pb.count, kg = s.kg_b(pb.count);
    unsigned char* dst = out + (size_t)pb.start * 2 * ksr * kPanel;
    const int total = ntask * ksr * 32;
    for (int idx = threadIdx.x; idx < total; idx += blockDim.x) {
        const int p = idx >> 5, c = idx & 31, row = c >> 1, half = c & 1;
        const int q = p / (ntask * kg), ns = min(kg, ksr - q * kg), pp = p - q * ntask * kg;
        const int task = pp / ns, st = pp - task * ns;
        const int j = (pb.start + (task >> 1)) * 16 + row, k = (q * kg + st) * 16 + half * 8;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (j < s.ffn && k < s.r)
            v = bf16x8_to_f16x8(*reinterpret_cast<const uint4*>(((task & 1) ? Uu : Ug) + (size_t)j * s.r + k), flag);
        *reinterpret_cast<uint4*>(dst + (size_t)idx * 16) = v;
    }
}

// Down-1 block of CTA b: [Zd row tile][ffn tile of the CTA][16 rows of Vd][16 ffn columns] fp16.
__global__ void __launch_bounds__(256)
pack_vd_kernel(const __nv_bfloat16* __restrict__ Vd, Shape s, unsigned char* __restrict__ out, int* flag) {
    const Part pb = part(s.units_b(), s.G, blockIdx.x);
    if (pb.count == 0) return;
    const int zt = s.zt();
    unsigned char* dst = out + (size_t)pb.start * zt * kPanel;
    const int total = zt * pb.count * 32;
    for (int idx = threadIdx.x; idx < total; idx += blockDim.x) {
        const int p = idx >> 5, c = idx & 31, row = c >> 1, half = c & 1;
        const int z = p / pb.count, j = p - z * pb.count;
        const int i = z * 16 + row, k = (pb.start + j) * 16 + half * 8;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (i < s.rd && k < s.ffn) v = bf16x8_to_f16x8(*reinterpret_cast<const uint4*>(Vd + (size_t)i * s.ffn + k), flag);
        *reinterpret_cast<uint4*>(dst + (size_t)idx * 16) = v;
    }
}

// Phase D block of CTA b: [k group][output tile of the CTA][k16 step in group][16 rows of Ud][16 k] fp16.
__global__ void __launch_bounds__(256)
pack_ud_kernel(const __nv_bfloat16* __restrict__ Ud, Shape s, unsigned char* __restrict__ out, int* flag) {
    const Part pd = part(s.units_d(), s.G, blockIdx.x);
    if (pd.count == 0) return;
    const int ks = s.zt(), kg = s.kg_d(pd.count);
    unsigned char* dst = out + (size_t)pd.start * ks * kPanel;
    const int total = pd.count * ks * 32;
    for (int idx = threadIdx.x; idx < total; idx += blockDim.x) {
        const int p = idx >> 5, c = idx & 31, row = c >> 1, half = c & 1;
        const int q = p / (pd.count * kg), ns = min(kg, ks - q * kg), pp = p - q * pd.count * kg;
        const int tile = pp / ns, st = pp - tile * ns;
        const int col = (pd.start + tile) * 16 + row, k = (q * kg + st) * 16 + half * 8;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (col < s.d && k < s.rd) v = bf16x8_to_f16x8(*reinterpret_cast<const uint4*>(Ud + (size_t)col * s.rd + k), flag);
        *reinterpret_cast<uint4*>(dst + (size_t)idx * 16) = v;
    }
}

// ---- ring of shared-memory slots filled by bulk copies ----------------------------------------
struct Cursor {
    int slot;
    uint32_t phase;
    __device__ __forceinline__ Cursor() : slot(0), phase(0) {}
    __device__ __forceinline__ void advance(int nslot) {
        if (++slot == nslot) { slot = 0; phase ^= 1u; }
    }
};

struct Ring {
    unsigned char* slots;
    uint64_t* full;    // one arrival (the producer's expect_tx) + the copies' bytes
    uint64_t* empty;   // kNW arrivals: every consumer warp hands the slot back itself
    int nslot;
    volatile int* abort;
    __device__ __forceinline__ unsigned char* slot(const Cursor& c) const { return slots + c.slot * kSlotBytes; }
};

__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(umma::smem_u32(dst)), "l"(src), "r"(bytes), "r"(umma::smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void consumer_bar() { asm volatile("bar.sync 1, %0;" ::"n"(kConsumers) : "memory"); }

__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_f16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint2 lds64(const unsigned char* p) { return *reinterpret_cast<const uint2*>(p); }
__device__ __forceinline__ float silu(float g) { return g / (1.0f + __expf(-g)); }
// Z (fp16) elements double as ready flags between phases A and B: an element that has not been stored yet holds
// kZUnset (a NaN pattern that arithmetic never produces; a result that happens to equal it is stored as the
// canonical NaN instead).
constexpr uint32_t kZUnset = 0xFFFFu;
__device__ __forceinline__ void st_z(__half* addr, float v) {
    unsigned short bits = __half_as_ushort(__float2half_rn(v));
    if (bits == kZUnset) bits = 0x7FFFu;
    asm volatile("st.relaxed.gpu.global.u16 [%0], %1;" ::"l"(addr), "h"(bits) : "memory");
}
__device__ __forceinline__ uint4 ld_z8(const __half* addr) {
    uint4 v;
    asm volatile("ld.relaxed.gpu.global.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(addr) : "memory");
    return v;
}
__device__ __forceinline__ bool z_pair_set(uint32_t w) { return (w & 0xFFFFu) != kZUnset && (w >> 16) != kZUnset; }
__device__ __forceinline__ void red_add_v4(float* addr, float a, float b, float c, float d) {
    asm volatile("red.relaxed.gpu.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(addr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}
__device__ __forceinline__ void red_add_v2(float* addr, float a, float b) {
    asm volatile("red.relaxed.gpu.global.add.v2.f32 [%0], {%1, %2};" ::"l"(addr), "f"(a), "f"(b) : "memory");
}

struct Params {
    Shape s;
    CUtensorMap mX;                               // x_tma: X as [64 columns][T rows][d/64 column blocks], box [64][T][ga/4]
    int x_tma, x_res;                             // x_res: one box holds all of X, loaded once into its own buffer
    const __nv_bfloat16* X;                       // [T, d]  (unused with fused RMSNorm)
    const float* hin; float eps;                  // fused RMSNorm: X = bf16(hin / sqrt(mean(hin^2) + eps)), hin fp32 [T, d], T <= 8
    const unsigned char *pA, *pB, *pVd, *pUd;     // packed factors (pack_*_kernel)
    __half* Z;                                    // [T, 2 r] fp16, written in phase A; all kZUnset between launches
    float* Zd;                                    // [2 (launch parity)][kCopiesZd][16 zt][kZdPitch] fp32 (token index fastest)
    void* Y; int y_fp32;
    const float* resid;
    unsigned long long* bar;                      // [0] arrivals at the B -> D barrier, [kBarStride] launch number, [2 kBarStride] A -> B arrivals
    int nslot, window;                            // ring slots; groups in flight (< nslot)
    int* status;
};

// Grid-wide barrier for the consumer threads of all CTAs.  `ctr` only grows: launch number e (read
// at kernel start) means all G CTAs have arrived once the counter reaches (e + 1) G.
template <bool FENCED>
__device__ __forceinline__ bool grid_arrive_wait(unsigned long long* ctr, unsigned long long target, volatile int* abort) {
    if (FENCED) __threadfence();  // every thread: its stores and reductions are performed before the CTA's arrival
    consumer_bar();
    if (threadIdx.x == 0) {
        if (FENCED) asm volatile("red.release.gpu.global.add.u64 [%0], 1;" ::"l"(ctr) : "memory");
        else asm volatile("red.relaxed.gpu.global.add.u64 [%0], 1;" ::"l"(ctr) : "memory");
        unsigned long long cur;
        const uint64_t t0 = umma::globaltimer_ns();
        for (uint32_t i = 1;; ++i) {
            asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(cur) : "l"(ctr) : "memory");
            if (cur >= target) break;
            if ((i & 63u) == 0u && (*abort || umma::globaltimer_ns() - t0 > umma::kWaitLimitNs)) { if (!*abort) *abort = FENCED ? 0x500 : 0x600; break; }
        }
    }
    consumer_bar();
    return *abort == 0;
}

template <int NT, int NTA, bool FUSED>
__global__ void __launch_bounds__(kThreads, 1)
mlp_kernel(const __grid_constant__ Params p) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ unsigned long long s_epoch;
    __shared__ float s_scale[8];  // fused RMSNorm: 1 / sqrt(mean(h^2) + eps) per token
    constexpr int ROWS = 8 * NT, MT = (NT + 1) / 2;
    const Shape& s = p.s;
    constexpr bool fused_norm = FUSED;  // RMSNorm of p.hin computed here instead of reading p.X
    const Layout L = make_layout(s, NT, NTA, fused_norm, p.x_res != 0);
    unsigned char* base = smem_raw + ((1024u - (umma::smem_u32(smem_raw) & 1023u)) & 1023u);
    Ring ring;
    unsigned char* xres = base;  // resident X (x_res), 1024-byte aligned for the swizzle
    ring.slots = base + L.xres_bytes;
    ring.nslot = p.nslot;
    uint64_t* bars = reinterpret_cast<uint64_t*>(ring.slots + p.nslot * kSlotBytes);
    ring.full = bars;
    ring.empty = bars + kMaxSlots;
    ring.abort = reinterpret_cast<volatile int*>(bars + 2 * kMaxSlots);
    uint64_t* xbar = bars + 2 * kMaxSlots + 2;  // resident X has landed
    unsigned char* rest = reinterpret_cast<unsigned char*>(bars + 2 * kMaxSlots + 4);
    if (threadIdx.x == 0) {
        for (int i = 0; i < p.nslot; ++i) { umma::mbar_init(&ring.full[i], 1); umma::mbar_init(&ring.empty[i], kNW); }
        umma::mbar_init(xbar, 1);
        *ring.abort = 0;
        umma::fence_mbar_init();
    }
    __syncthreads();
    // Programmatic dependent launch: the next kernel in the stream may take this SM as soon as this CTA leaves
    // it, and this CTA was allowed to start (and set up its barriers) while the tail of the preceding kernel was
    // still running.  Everything below touches memory that kernel may still use, so wait for it first.
    umma::pdl_launch_dependents();
    umma::pdl_wait();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, tig = lane & 3;
    const int b = blockIdx.x, nslot = p.nslot;
    const int ksd = s.ksd(), ksr = s.ksr(), zt = s.zt();
    const Part pa = part(s.units_a(), s.G, b), pb = part(s.units_b(), s.G, b), pd = part(s.units_d(), s.G, b);

    if (warp == kNW) {
        // ---- producer: the warp walks the CTA's group list in order.  Lane 0 does the waiting and arms the slot;
        // ---- the copies of a group are then issued by lane 0 (factor block) and lanes 0..T-1 (rows of X).
        // At most p.window groups are in flight (issued, not yet landed): enough bytes to keep HBM busy, few
        // enough that the latency-critical traffic of the phase hand-overs does not queue behind megabytes.
        // The warp stays converged from group to group (the shuffle below), so when group i is handled no later
        // group has been armed and the parity waits cannot alias.
        Cursor cur, landed;   // landed trails cur by p.window groups
        int issued = 0;
        bool ok = true;
        auto arm = [&](uint32_t bytes) -> bool {
            bool good = ok;
            if (lane == 0 && ok) {
                if (issued >= p.window) good = umma::mbar_wait_patient(&ring.full[landed.slot], landed.phase, ring.abort, 0x200 + issued);
                if (good) good = umma::mbar_wait_patient(&ring.empty[cur.slot], cur.phase ^ 1u, ring.abort, 0x300 + issued);
                if (good) umma::mbar_expect_tx(&ring.full[cur.slot], bytes);
            }
            ok = __shfl_sync(0xffffffffu, good ? 1 : 0, 0) != 0;
            if (issued >= p.window) landed.advance(nslot);
            ++issued;
            return ok;
        };
        auto copy0 = [&](const unsigned char* src, uint32_t bytes) {  // one block into the current slot
            if (arm(bytes) && lane == 0) bulk_g2s(ring.slot(cur), src, bytes, &ring.full[cur.slot]);
            cur.advance(nslot);
        };
        if (pa.count > 0 && p.x_res && lane == 0) {
            umma::mbar_expect_tx(xbar, (uint32_t)(s.d / 64) * s.T * 128u);
            asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
                         ::"r"(umma::smem_u32(xres)), "l"(reinterpret_cast<uint64_t>(&p.mX)), "r"(umma::smem_u32(xbar)), "r"(0), "r"(0), "r"(0) : "memory");
        }
        if (pa.count > 0) {
            const unsigned char* src = p.pA + (size_t)pa.start * ksd * 32;
            const int nga = ceil_div(ksd, L.ga);
            for (int q = 0; q < nga; ++q) {
                const int s0 = q * L.ga;
                const int ns = min(L.ga, ksd - s0);
                const uint32_t vbytes = (uint32_t)ns * pa.count * 32;
                const uint32_t xrow = (uint32_t)min(ns * 32, (s.d - s0 * 16) * 2);
                const uint32_t xbytes = (fused_norm || p.x_res) ? 0u : p.x_tma ? (uint32_t)L.ga * 32u * s.T : xrow * s.T;  // the TMA box is always whole
                if (arm(vbytes + xbytes)) {
                    if (lane == 0) {
                        bulk_g2s(ring.slot(cur) + L.a_v_off, src + (size_t)s0 * pa.count * 32, vbytes, &ring.full[cur.slot]);
                        if (p.x_tma && !fused_norm && !p.x_res)
                            asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
                                         ::"r"(umma::smem_u32(ring.slot(cur))), "l"(reinterpret_cast<uint64_t>(&p.mX)),
                                           "r"(umma::smem_u32(&ring.full[cur.slot])), "r"(0), "r"(0), "r"(s0 >> 2) : "memory");
                    }
                    if (lane < s.T && !fused_norm && !p.x_tma)   // T <= 32
                        bulk_g2s(ring.slot(cur) + lane * L.pitch_x, p.X + (size_t)lane * s.d + s0 * 16, xrow, &ring.full[cur.slot]);
                }
                cur.advance(nslot);
            }
        }
        if (pb.count > 0) {
            const int ntask = 2 * pb.count, kg = s.kg_b(pb.count), gz = s.gz_b(pb.count);
            const unsigned char* src = p.pB + (size_t)pb.start * 2 * ksr * kPanel;
            for (int k0 = 0; k0 < ksr; k0 += kg) {
                const uint32_t bytes = (uint32_t)ntask * min(kg, ksr - k0) * kPanel;
                copy0(src, bytes);
                src += bytes;
            }
            src = p.pVd + (size_t)pb.start * zt * kPanel;
            for (int z0 = 0; z0 < zt; z0 += gz) {
                const uint32_t bytes = (uint32_t)min(gz, zt - z0) * pb.count * kPanel;
                copy0(src, bytes);
                src += bytes;
            }
        }
        if (pd.count > 0) {
            const int kg = s.kg_d(pd.count);
            const unsigned char* src = p.pUd + (size_t)pd.start * zt * kPanel;
            for (int k0 = 0; k0 < zt; k0 += kg) {
                const uint32_t bytes = (uint32_t)pd.count * min(kg, zt - k0) * kPanel;
                copy0(src, bytes);
                src += bytes;
            }
        }
        if (*ring.abort && p.status != nullptr && lane == 0) atomicExch(p.status, -7);
        return;
    }

    // ---------------- consumers ----------------
    Cursor cur;
    bool dead = false;  // a wait gave up: keep walking (every named barrier is still reached) without waiting
    int nwaited = 0;  // diagnostics: index of the group a consumer wait gave up on
    auto wait = [&]() { if (!dead && !umma::mbar_wait_warp(&ring.full[cur.slot], cur.phase, ring.abort, 0x400 + nwaited)) dead = true; ++nwaited; };
    auto release = [&]() {
        __syncwarp();
        if (lane == 0) umma::mbar_arrive(&ring.empty[cur.slot]);
        cur.advance(nslot);
    };
    const int tid = threadIdx.x;
    if (tid == 0) {  // launch number: needed from phase A on by every consumer thread (parity of the Zd buffer)
        unsigned long long e;
        asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(e) : "l"(p.bar + kBarStride) : "memory");
        s_epoch = e;
    }
    consumer_bar();
    const unsigned long long epoch = s_epoch;
    const unsigned long long target = (epoch + 1ull) * (unsigned long long)gridDim.x;
    // Zd buffers: two halves (launch parity) of kCopiesZd x [16 zt][kZdPitch] floats; a launch uses the front of
    // its half with rows of ROWS floats, and clears the whole other half so that the next launch may use any T.
    const int zd_elems = zt * 16 * ROWS, zd_half = kCopiesZd * zt * 16 * kZdPitch;
    // Zd is double-buffered by launch parity: this launch reduces into one half and clears the other half
    // for the next launch, so the clearing needs no ordering against this launch's reductions.
    float* zd_cur = p.Zd + (size_t)(epoch & 1ull) * zd_half;
    float* zd_next = p.Zd + (size_t)((epoch + 1ull) & 1ull) * zd_half;

    {   // ---- phase A: Z[:, rows of this CTA] = X V^T over the full K; warps split the k16 steps of each group
        for (long i = ((long)b * kConsumers + tid) * 4; i < zd_half; i += (long)gridDim.x * kConsumers * 4)
            *reinterpret_cast<float4*>(zd_next + i) = make_float4(0.f, 0.f, 0.f, 0.f);
        if (fused_norm) {
            // per-token sum of squares over the full row (every CTA needs every scale; T <= 8 rows, read through L2)
            float ss[8];
#pragma unroll
            for (int t = 0; t < 8; ++t) {
                ss[t] = 0.f;
                if (t < s.T)
                    for (int k = tid * 4; k < s.d; k += kConsumers * 4) {
                        const float4 v = __ldg(reinterpret_cast<const float4*>(p.hin + (size_t)t * s.d + k));
                        ss[t] += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
                    }
            }
            float* red = reinterpret_cast<float*>(rest + L.red);
#pragma unroll
            for (int t = 0; t < 8; ++t) {
                for (int o = 16; o > 0; o >>= 1) ss[t] += __shfl_xor_sync(0xffffffffu, ss[t], o);
                if (lane == 0) red[warp * 8 + t] = ss[t];
            }
            consumer_bar();
            if (tid < s.T) {
                float tot = 0.f;
                for (int w = 0; w < kNW; ++w) tot += red[w * 8 + tid];
                s_scale[tid] = rsqrtf(tot / (float)s.d + p.eps);
            }
            consumer_bar();
        }
        if (pa.count > 0) {
            float acc[2][MT][NTA][4];
#pragma unroll
            for (int e = 0; e < 2; ++e)
#pragma unroll
                for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                    for (int j = 0; j < NTA; ++j) acc[e][mt][j][0] = acc[e][mt][j][1] = acc[e][mt][j][2] = acc[e][mt][j][3] = 0.f;
            const int nga = ceil_div(ksd, L.ga);
            unsigned char* xn = rest + L.xn;
            if (p.x_res && !dead && !umma::mbar_wait_warp(xbar, 0, ring.abort, 0x800)) dead = true;
            for (int q = 0; q < nga; ++q) {
                const int s0 = q * L.ga;
                const int ns = min(L.ga, ksd - s0);
                if (fused_norm) {
                    // this group's columns of X = bf16(h * scale), written by the consumers themselves while the
                    // V block is still on its way (the previous group's reads of xn ended at the barrier below)
                    for (int t = 0; t < s.T; ++t)
                        for (int c = tid; c < ns * 4; c += kConsumers) {
                            const int k = s0 * 16 + c * 4;
                            if (k < s.d) {
                                const float4 v = __ldg(reinterpret_cast<const float4*>(p.hin + (size_t)t * s.d + k));
                                const float sc = s_scale[t];
                                __nv_bfloat162 lo = __floats2bfloat162_rn(v.x * sc, v.y * sc), hi = __floats2bfloat162_rn(v.z * sc, v.w * sc);
                                uint2 o;
                                o.x = *reinterpret_cast<uint32_t*>(&lo);
                                o.y = *reinterpret_cast<uint32_t*>(&hi);
                                *reinterpret_cast<uint2*>(xn + t * L.pitch_x + c * 8) = o;
                            }
                        }
                    consumer_bar();
                }
                wait();
                const unsigned char* vs = ring.slot(cur) + L.a_v_off;
                const unsigned char* xs = fused_norm ? xn : p.x_res ? xres : ring.slot(cur);
                const bool swz = p.x_tma && !fused_norm;
                const int kb0 = p.x_res ? (s0 >> 2) : 0;  // resident X: column blocks are numbered from the start of the row
                // Warps take whole column blocks (4 k16 steps = one 128-byte row piece of X) in turn, so that the
                // addresses inside the unrolled body differ by constants; rows that do not exist read row 0 and are
                // zeroed by a select (no branches), even/odd steps use separate accumulators.
                const int nkb = (ns + 3) >> 2;
                const unsigned vstride = (unsigned)pa.count * 32u;
                if (swz) {
                    // TMA-fed X: d is a multiple of 64, so every column block is whole, and no operand needs
                    // masking: token rows beyond T and factor rows beyond this CTA's count re-read row 0, which
                    // only fills accumulator entries that are never stored.  This keeps the loop at a handful of
                    // address operations per MMA (the masked form below is bound by instruction issue).
                    const unsigned char* vrow[NTA];
#pragma unroll
                    for (int j = 0; j < NTA; ++j) vrow[j] = vs + (8 * j + g < pa.count ? 8 * j + g : 0) * 32 + tig * 8;
                    const int tsel = ((tig >> 1) << 4) | ((tig & 1) << 3);
                    for (int kb = warp; kb < nkb; kb += kNW) {
                        uint2 a[4][MT][2], bv[4][NTA];
#pragma unroll
                        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                            for (int hh = 0; hh < 2; ++hh) {
                                if (mt * 16 + hh * 8 < ROWS) {
                                    const int row = mt * 16 + hh * 8 + g;
                                    const int rr = (kb0 + kb) * s.T + (row < s.T ? row : 0), sw = (rr & 7) << 4;
                                    const unsigned char* xb = xs + (rr << 7);
#pragma unroll
                                    for (int e = 0; e < 4; ++e) a[e][mt][hh] = lds64(xb + ((2 * e * 16 + tsel) ^ sw));
                                } else {
#pragma unroll
                                    for (int e = 0; e < 4; ++e) a[e][mt][hh] = make_uint2(0, 0);
                                }
                            }
#pragma unroll
                        for (int j = 0; j < NTA; ++j)
#pragma unroll
                            for (int e = 0; e < 4; ++e) bv[e][j] = lds64(vrow[j] + (unsigned)(kb * 4 + e) * vstride);
#pragma unroll
                        for (int e = 0; e < 4; ++e)
#pragma unroll
                            for (int j = 0; j < NTA; ++j)
#pragma unroll
                                for (int mt = 0; mt < MT; ++mt)
                                    mma_bf16(acc[e & 1][mt][j], a[e][mt][0].x, a[e][mt][1].x, a[e][mt][0].y, a[e][mt][1].y, bv[e][j].x, bv[e][j].y);
                    }
                } else
                for (int kb = warp; kb < nkb; kb += kNW) {
                    const int stb = kb * 4;  // first step of the block within the group
                    uint2 a[4][MT][2], bv[4][NTA];
#pragma unroll
                    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                        for (int hh = 0; hh < 2; ++hh) {
                            if (mt * 16 + hh * 8 < ROWS) {  // compile time: the upper half of the last m tile may not exist
                                const int row = mt * 16 + hh * 8 + g, rowc = row < s.T ? row : 0;
                                if (swz) {  // [column block][token][128 B], 16-byte pieces XOR-swizzled by the 128-byte row index
                                    const int rr = (kb0 + kb) * s.T + rowc, sw = rr & 7;
                                    const unsigned char* xb = xs + (rr << 7) + ((((tig >> 1) ^ (sw & 1)) << 4) | ((tig & 1) << 3));
                                    const int swhi = (sw & 6) << 4;
#pragma unroll
                                    for (int e = 0; e < 4; ++e) a[e][mt][hh] = lds64(xb + ((2 * e * 16) ^ swhi));
                                } else {
                                    const unsigned char* xb = xs + rowc * L.pitch_x + stb * 32 + tig * 8;
#pragma unroll
                                    for (int e = 0; e < 4; ++e) a[e][mt][hh] = lds64(xb + e * 32);
                                }
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    const bool keep = row < s.T && stb + e < ns && (swz || (s0 + stb + e) * 16 + 4 * tig + 4 <= s.d);
                                    a[e][mt][hh] = make_uint2(keep ? a[e][mt][hh].x : 0u, keep ? a[e][mt][hh].y : 0u);
                                }
                            } else {
#pragma unroll
                                for (int e = 0; e < 4; ++e) a[e][mt][hh] = make_uint2(0, 0);
                            }
                        }
#pragma unroll
                    for (int j = 0; j < NTA; ++j) {
                        const int row = 8 * j + g;
                        const unsigned char* vb = vs + (unsigned)stb * vstride + (row < pa.count ? row : 0) * 32 + tig * 8;
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            bv[e][j] = lds64(vb + (stb + e < ns ? e : 0) * vstride);
                            if (row >= pa.count) bv[e][j] = make_uint2(0, 0);
                        }
                    }
#pragma unroll
                    for (int e = 0; e < 4; ++e)
#pragma unroll
                        for (int j = 0; j < NTA; ++j)
#pragma unroll
                            for (int mt = 0; mt < MT; ++mt)
                                mma_bf16(acc[e & 1][mt][j], a[e][mt][0].x, a[e][mt][1].x, a[e][mt][0].y, a[e][mt][1].y, bv[e][j].x, bv[e][j].y);
                }
                release();
                if (fused_norm && q + 1 < nga) consumer_bar();  // xn is rewritten for the next group
            }
            float* red = reinterpret_cast<float*>(rest + L.red);  // [warp][16 MT tokens][8 NTA rows]
#pragma unroll
            for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                for (int j = 0; j < NTA; ++j)
#pragma unroll
                    for (int c = 0; c < 4; ++c)
                        red[(warp * 16 * MT + mt * 16 + g + 8 * (c >> 1)) * (8 * NTA) + j * 8 + 2 * tig + (c & 1)] = acc[0][mt][j][c] + acc[1][mt][j][c];
        }
        consumer_bar();
        if (pa.count > 0 && !dead) {
            const float* red = reinterpret_cast<const float*>(rest + L.red);
            for (int idx = tid; idx < s.T * pa.count; idx += kConsumers) {
                const int t = idx / pa.count, c = idx - t * pa.count;
                float sum = 0.f;
#pragma unroll
                for (int w = 0; w < kNW; ++w) sum += red[(w * 16 * MT + t) * (8 * NTA) + c];
                st_z(p.Z + (size_t)t * 2 * s.r + pa.start + c, sum);
            }
        }
    }
    // A -> B hand-over.  The arrival count is only a hint that Z is probably complete (no fence orders the Z
    // stores before it); what makes the hand-over safe is that Z carries its own validity: an element that
    // has not been stored yet still holds kZUnset (phase D resets it), and the staging loop below re-reads
    // until none is left.  This saves the fence's round trip through a loaded memory system.
    if (!grid_arrive_wait<false>(p.bar + 2 * kBarStride, target, ring.abort)) dead = true;

    unsigned char* zs = rest + L.zs;
    if (pb.count > 0) {
        // ---- phase B: stage Z as fp16 [token][gate k | up k]
        const int r = s.r, r16 = ksr * 16, q8 = 2 * r / 8;
        // Z is the signal itself: every element holds kZUnset until its owner has stored it (and is reset to
        // that pattern in phase D), so a load that still sees the pattern is simply repeated.
        // Thread map without divisions: 32, 64 or 128 threads (enough for the 16-byte pieces of a row) walk a token
        // row, 12, 6 or 3 rows at a time; up to ZR x ZC loads are in flight per thread before the first one is
        // looked at, so that a whole Z of up to 36 (18, 9) tokens costs one round trip.
        constexpr int ZR = 3, ZC = 2;
        const int lw = q8 <= 32 ? 5 : q8 <= 64 ? 6 : 7, tpr = 1 << lw, nrg = kConsumers >> lw;
        const int zc0 = tid & (tpr - 1), zt0 = tid >> lw;
        const uint64_t t0 = umma::globaltimer_ns();
        for (int tb = zt0; tb < s.T; tb += nrg * ZR)
            for (int cb = zc0; cb < q8; cb += tpr * ZC) {
                uint4 v[ZR][ZC];
                bool have[ZR][ZC];
#pragma unroll
                for (int a = 0; a < ZR; ++a)
#pragma unroll
                    for (int c = 0; c < ZC; ++c) have[a][c] = !(tb + nrg * a < s.T && cb + tpr * c < q8);  // nothing to fetch
                for (uint32_t spin = 1;; ++spin) {
#pragma unroll
                    for (int a = 0; a < ZR; ++a)
#pragma unroll
                        for (int c = 0; c < ZC; ++c)
                            if (!have[a][c]) v[a][c] = ld_z8(p.Z + (size_t)(tb + nrg * a) * 2 * r + (cb + tpr * c) * 8);
                    bool all = true;
#pragma unroll
                    for (int a = 0; a < ZR; ++a)
#pragma unroll
                        for (int c = 0; c < ZC; ++c)
                            if (!have[a][c]) {
                                have[a][c] = z_pair_set(v[a][c].x) && z_pair_set(v[a][c].y) && z_pair_set(v[a][c].z) && z_pair_set(v[a][c].w);
                                all = all && have[a][c];
                            }
                    if (all || dead) break;
                    if ((spin & 15u) == 0u && (*ring.abort || umma::globaltimer_ns() - t0 > umma::kWaitLimitNs)) { if (!*ring.abort) *ring.abort = 0x700; dead = true; }
                }
#pragma unroll
                for (int a = 0; a < ZR; ++a)
#pragma unroll
                    for (int c = 0; c < ZC; ++c)
                        if (tb + nrg * a < s.T && cb + tpr * c < q8) {
                            const int c8 = (cb + tpr * c) * 8, pos = c8 < r ? c8 : r16 + (c8 - r);
                            *reinterpret_cast<uint4*>(zs + (tb + nrg * a) * L.pitch_z + pos * 2) = v[a][c];
                        }
            }
        if (r16 != r)
            for (int idx = tid; idx < s.T * 2 * (r16 - r); idx += kConsumers) {
                const int t = idx / (2 * (r16 - r)), rem = idx - t * 2 * (r16 - r), hf = rem / (r16 - r), k = r + rem - hf * (r16 - r);
                *reinterpret_cast<__half*>(zs + t * L.pitch_z + (hf * r16 + k) * 2) = __float2half_rn(0.f);
            }
        consumer_bar();

        // gate/up expansion: warp task = (tile, gate | up) over the full K = r
        const int ntask = 2 * pb.count, kg = s.kg_b(pb.count);
        float acc[2][NT][4];
#pragma unroll
        for (int it = 0; it < 2; ++it)
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) acc[it][nt][0] = acc[it][nt][1] = acc[it][nt][2] = acc[it][nt][3] = 0.f;
        for (int k0 = 0; k0 < ksr; k0 += kg) {
            const int ns = min(kg, ksr - k0);
            wait();
            const unsigned char* slot = ring.slot(cur);
#pragma unroll
            for (int it = 0; it < 2; ++it) {
                const int ti = warp + it * kNW;
                if (ti < ntask) {
                    const unsigned char* w = slot + (size_t)ti * ns * kPanel + g * 32 + tig * 8;
                    const unsigned char* x = zs + g * L.pitch_z + ((ti & 1) ? r16 * 2 : 0) + k0 * 32 + tig * 8;
#pragma unroll 4
                    for (int st = 0; st < ns; ++st) {
                        const uint2 wa = lds64(w + st * kPanel), wb = lds64(w + st * kPanel + 256);
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt) {
                            const uint2 xv = lds64(x + nt * 8 * L.pitch_z + st * 32);
                            mma_f16(acc[it][nt], wa.x, wb.x, wa.y, wb.y, xv.x, xv.y);
                        }
                    }
                }
            }
            release();
        }
        // SiLU(gate) .* up through shared memory: gate tasks publish G, up tasks build H (fp16)
        float* gs = reinterpret_cast<float*>(rest + L.gs);
        unsigned char* hs = rest + L.hs;
#pragma unroll
        for (int it = 0; it < 2; ++it) {
            const int ti = warp + it * kNW;
            if (ti < ntask && !(ti & 1)) {
#pragma unroll
                for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                    for (int c = 0; c < 4; ++c)
                        gs[(nt * 8 + 2 * tig + (c & 1)) * L.gp + (ti >> 1) * 16 + g + 8 * (c >> 1)] = acc[it][nt][c];
            }
        }
        consumer_bar();
#pragma unroll
        for (int it = 0; it < 2; ++it) {
            const int ti = warp + it * kNW;
            if (ti < ntask && (ti & 1)) {
#pragma unroll
                for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        const int tok = nt * 8 + 2 * tig + (c & 1), col = (ti >> 1) * 16 + g + 8 * (c >> 1);
                        *reinterpret_cast<__half*>(hs + tok * L.pitch_h + col * 2) = __float2half_rn(silu(gs[tok * L.gp + col]) * acc[it][nt][c]);
                    }
            }
        }
        consumer_bar();

        // first half of the down chain: Zd[:, 16-row tile] += H[:, cols of this CTA] Vd[tile, cols]^T
        const int gz = s.gz_b(pb.count);
        float* zdc = zd_cur + (size_t)(b % kCopiesZd) * zd_elems;
        for (int z0 = 0; z0 < zt; z0 += gz) {
            const int nz = min(gz, zt - z0);
            wait();
            const unsigned char* slot = ring.slot(cur);
            for (int z = warp; z < nz; z += kNW) {
                float a2[NT][4];
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) a2[nt][0] = a2[nt][1] = a2[nt][2] = a2[nt][3] = 0.f;
                const unsigned char* w = slot + (size_t)z * pb.count * kPanel + g * 32 + tig * 8;
                const unsigned char* x = hs + g * L.pitch_h + tig * 8;
#pragma unroll 4
                for (int j = 0; j < pb.count; ++j) {
                    const uint2 wa = lds64(w + j * kPanel), wb = lds64(w + j * kPanel + 256);
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        const uint2 xv = lds64(x + nt * 8 * L.pitch_h + j * 32);
                        mma_f16(a2[nt], wa.x, wb.x, wa.y, wb.y, xv.x, xv.y);
                    }
                }
                if (!dead) {
                    // lane pairs (tig, tig ^ 1) swap halves so that each lane owns four consecutive tokens of one
                    // row: even tig keeps row g, odd tig row g + 8; one 16-byte reduction per lane and token tile
                    const bool odd = tig & 1;
                    const int i = (z0 + z) * 16 + g + (odd ? 8 : 0);
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        const float r0 = __shfl_xor_sync(0xffffffffu, odd ? a2[nt][0] : a2[nt][2], 1);
                        const float r1 = __shfl_xor_sync(0xffffffffu, odd ? a2[nt][1] : a2[nt][3], 1);
                        const int t0 = nt * 8 + 4 * (tig >> 1);
                        if (i < s.rd && t0 < s.T) {
                            if (odd) red_add_v4(zdc + (size_t)i * ROWS + t0, r0, r1, a2[nt][2], a2[nt][3]);
                            else red_add_v4(zdc + (size_t)i * ROWS + t0, a2[nt][0], a2[nt][1], r0, r1);
                        }
                    }
                }
            }
            release();
        }
    }
    if (!grid_arrive_wait<true>(p.bar, target, ring.abort)) dead = true;
    // every CTA staged Z before it arrived at the barrier: mark this CTA's entries unset for the next launch
    for (int idx = tid; idx < s.T * pa.count; idx += kConsumers) {
        const int t = idx / pa.count, c = idx - t * pa.count;
        reinterpret_cast<unsigned short*>(p.Z)[(size_t)t * 2 * s.r + pa.start + c] = (unsigned short)kZUnset;
    }

    if (pd.count > 0) {
        // ---- phase D: stage Zd (sum of the copies) as fp16 [token][k], then Y tiles = Ud tiles x Zd^T
        const int rd = s.rd, rd16 = zt * 16, tq = (s.T + 3) / 4;
        // thread map without divisions: TQ (a power of two >= tq) threads per Zd row, kConsumers / TQ rows at a
        // time; DI rows x kCopiesZd copies are loaded before any is used
        constexpr int DI = 2;
        const int lq = tq <= 1 ? 0 : tq <= 2 ? 1 : tq <= 4 ? 2 : 3, TQ = 1 << lq, q = tid & (TQ - 1), istep = kConsumers >> lq;
        if (q < tq)
            for (int ib = tid >> lq; ib < rd; ib += DI * istep) {
                float4 v[DI][kCopiesZd];
#pragma unroll
                for (int a = 0; a < DI; ++a)
#pragma unroll
                    for (int c = 0; c < kCopiesZd; ++c)
                        if (ib + a * istep < rd) v[a][c] = __ldcg(reinterpret_cast<const float4*>(zd_cur + (size_t)c * zd_elems + (size_t)(ib + a * istep) * ROWS + 4 * q));
#pragma unroll
                for (int a = 0; a < DI; ++a) {
                    const int i = ib + a * istep;
                    if (i < rd) {
                        float sum[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                        for (int c = 0; c < kCopiesZd; ++c) { sum[0] += v[a][c].x; sum[1] += v[a][c].y; sum[2] += v[a][c].z; sum[3] += v[a][c].w; }
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            if (4 * q + e < s.T) *reinterpret_cast<__half*>(zs + (4 * q + e) * L.pitch_d + i * 2) = __float2half_rn(sum[e]);
                    }
                }
            }
        if (rd16 != rd)
            for (int idx = tid; idx < s.T * (rd16 - rd); idx += kConsumers) {
                const int t = idx / (rd16 - rd), k = rd + idx - t * (rd16 - rd);
                *reinterpret_cast<__half*>(zs + t * L.pitch_d + k * 2) = __float2half_rn(0.f);
            }
        consumer_bar();
        const int cnt = pd.count, kparts = kNW / cnt, kpart = warp / cnt, tile = warp - kpart * cnt;
        const bool active = kpart < kparts;
        const int kg = s.kg_d(cnt);
        float accd[NT][4];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) accd[nt][0] = accd[nt][1] = accd[nt][2] = accd[nt][3] = 0.f;
        for (int k0 = 0; k0 < zt; k0 += kg) {
            const int ns = min(kg, zt - k0);
            wait();
            if (active) {
                const unsigned char* w = ring.slot(cur) + (size_t)tile * ns * kPanel + g * 32 + tig * 8;
                const unsigned char* x = zs + g * L.pitch_d + k0 * 32 + tig * 8;
#pragma unroll 2
                for (int st = kpart; st < ns; st += kparts) {
                    const uint2 wa = lds64(w + st * kPanel), wb = lds64(w + st * kPanel + 256);
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        const uint2 xv = lds64(x + nt * 8 * L.pitch_d + st * 32);
                        mma_f16(accd[nt], wa.x, wb.x, wa.y, wb.y, xv.x, xv.y);
                    }
                }
            }
            release();
        }
        float* red = reinterpret_cast<float*>(rest + L.red);  // [k part][tile][16 rows][ROWS + 1 tokens]
        if (active) {
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    red[((kpart * cnt + tile) * 16 + g + 8 * (c >> 1)) * (ROWS + 1) + nt * 8 + 2 * tig + (c & 1)] = accd[nt][c];
        }
        consumer_bar();
        if (!dead) {
            for (int idx = tid; idx < cnt * 16 * s.T; idx += kConsumers) {
                const int t = idx / (cnt * 16), row16 = idx - t * cnt * 16, col = pd.start * 16 + row16;
                if (col < s.d) {
                    float v = 0.f;
                    for (int kp = 0; kp < kparts; ++kp) v += red[(kp * cnt * 16 + row16) * (ROWS + 1) + t];
                    const size_t o = (size_t)t * s.d + col;
                    if (p.resid != nullptr) v += p.resid[o];
                    if (p.y_fp32) reinterpret_cast<float*>(p.Y)[o] = v;
                    else reinterpret_cast<__nv_bfloat16*>(p.Y)[o] = __float2bfloat16_rn(v);
                }
            }
        }
    }
    // every CTA has read the launch number before it arrived at the second barrier: bump it for the next launch
    if (b == 0 && tid == 0) p.bar[kBarStride] = epoch + 1ull;
    if (*ring.abort && p.status != nullptr && lane == 0) atomicExch(p.status, -7);
}

}  // namespace dpersist
