// libsvdmlp: C-ABI entry points and host-side launch logic (see include/svdmlp.h).
// Every step of the forward pass runs in the CUDA kernels of skinny.cuh (small T, weight
// streaming) and tensor_gemm.cuh (large T, tcgen05); this file only validates arguments,
// owns the workspace, encodes TMA tensor maps and enqueues launches.
#include "../../include/svdmlp.h"
#include "../../include/svdmlp_bench.h"

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <numeric>
#include <vector>
#include <new>

#include "decode_persistent.cuh"
#include "skinny.cuh"
#include "tensor_gemm.cuh"
#include "gateup_ts.cuh"
#include "mlp_fused_ts.cuh"
#include "tp_exchange.cuh"
#include "gateup_wide.cuh"
#include "compress.cuh"

namespace {

constexpr int kMaxKSplit = 32;             // most K splits of a split-K GEMM (short batches: one tile per SM needs them)
constexpr int kSkinnyMaxT = 32;            // T <= this uses the weight-streaming kernels
constexpr int kSmemBudget = 232448 - 1024; // opt-in shared memory per CTA minus alignment slack
constexpr int kBarrierBytes = 512;

#define CUDA_TRY(expr)                          \
    do {                                        \
        cudaError_t e__ = (expr);               \
        if (e__ != cudaSuccess) {               \
            cudaGetLastError();                 \
            return SVDMLP_ERR_CUDA;             \
        }                                       \
    } while (0)

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_arch() {
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return SVDMLP_ERR_CUDA; }
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) {
        cudaGetLastError();
        return SVDMLP_ERR_CUDA;
    }
    return major == 10 ? SVDMLP_OK : SVDMLP_ERR_ARCH;
}

// ---- TMA tensor maps ------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (fn == nullptr) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
        else
            cudaGetLastError();
    }
    return fn;
}

// Row-major 16-bit matrix [rows, cols] with leading dimension ld (elements); box = [box_rows, 64],
// 128-byte swizzle, out-of-range elements read as zero.
int make_map(CUtensorMap* m, const void* base, long rows, long cols, long ld, int box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) return SVDMLP_ERR_CUDA;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
    cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? SVDMLP_OK : SVDMLP_ERR_CUDA;
}

// X[T, d] bf16 seen as [64 columns][T rows][d/64 column blocks] (d a multiple of 64): one box of
// [64][T][blocks] is a group of column blocks for every token, each 128-byte row piece swizzled.
int make_map_x3(CUtensorMap* m, const void* base, int T, int d, int blocks) {
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) return SVDMLP_ERR_CUDA;
    cuuint64_t dims[3] = {64, (cuuint64_t)T, (cuuint64_t)(d / 64)};
    cuuint64_t strides[2] = {(cuuint64_t)d * 2, 128};
    cuuint32_t box[3] = {64, (cuuint32_t)T, (cuuint32_t)blocks};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? SVDMLP_OK : SVDMLP_ERR_CUDA;
}

// Row-major fp32 matrix [rows, cols]: box = [32 rows, 32 columns] (128-byte rows), 128-byte swizzle.
int make_map_f32(CUtensorMap* m, const void* base, long rows, long cols, long ld) {
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) return SVDMLP_ERR_CUDA;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld * 4};
    cuuint32_t box[2] = {32, 32};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? SVDMLP_OK : SVDMLP_ERR_CUDA;
}

// Row-major 16-bit matrix [rows, cols] written in boxes of [64 rows, 32 columns] without swizzle: the transposed
// output C^T[N, M] of a GEMM whose epilogue stages [64 n][32 m] tiles.
int make_map_t(CUtensorMap* m, const void* base, long rows, long cols, long ld) {
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) return SVDMLP_ERR_CUDA;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
    cuuint32_t box[2] = {32, 64};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? SVDMLP_OK : SVDMLP_ERR_CUDA;
}

// ---- tensor-path launch helper ----------------------------------------------------------------
struct GemmPlan {
    int nb, bn;
    bool ares;
    bool pair;  // CTA-pair (cta_group::2) kernel: resident A strip, each CTA loads half of every B chunk
    tensorpath::GemmParams p;
    int grid;
    size_t smem;
};

template <int NB, int BN, bool ARES>
int launch_gemm_t(const GemmPlan& g, cudaStream_t s) {
    static bool attr_set = false;  // per process; a second device would need its own call
    static int attr_dev = -1;
    int dev = 0;
    cudaGetDevice(&dev);
    if (!attr_set || attr_dev != dev) {
        CUDA_TRY(cudaFuncSetAttribute(tensorpath::gemm_kernel<NB, BN, ARES>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      kSmemBudget + 1024));
        attr_set = true;
        attr_dev = dev;
    }
    // Programmatic dependent launch: the kernel's set-up may overlap the tail of its predecessor;
    // it executes griddepcontrol.wait before touching anything the predecessor wrote.
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(g.grid); cfg.blockDim = dim3(tensorpath::kThreads); cfg.dynamicSmemBytes = g.smem; cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    CUDA_TRY(cudaLaunchKernelEx(&cfg, tensorpath::gemm_kernel<NB, BN, ARES>, g.p));
    return SVDMLP_OK;
}

template <int NB, int BN, bool ARES>
int launch_gemm_pair_t(const GemmPlan& g, cudaStream_t s) {
    // Two producer warps take alternate ring slots; with a single slot they would wait on the same barrier for
    // different fills, which its one-bit phase parity cannot tell apart.
    if (g.p.stages < 2) return SVDMLP_ERR_UNSUPPORTED;
    static bool attr_set = false;
    static int attr_dev = -1;
    int dev = 0;
    cudaGetDevice(&dev);
    if (!attr_set || attr_dev != dev) {
        CUDA_TRY(cudaFuncSetAttribute(tensorpath::gemm_pair_kernel<NB, BN, ARES>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      kSmemBudget + 1024));
        attr_set = true;
        attr_dev = dev;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(g.grid); cfg.blockDim = dim3(tensorpath::kPairThreads); cfg.dynamicSmemBytes = g.smem; cfg.stream = s;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2 * std::max(1, g.p.cks);   // one CTA pair, or the pairs that split K among themselves
    attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 2;
    CUDA_TRY(cudaLaunchKernelEx(&cfg, tensorpath::gemm_pair_kernel<NB, BN, ARES>, g.p));
    return SVDMLP_OK;
}

int launch_gemm(const GemmPlan& g, cudaStream_t s) {
    if (g.pair && g.ares && g.nb == 1 && g.bn == 128) return launch_gemm_pair_t<1, 128, true>(g, s);
    if (g.pair && g.ares && g.nb == 1 && g.bn == 256) return launch_gemm_pair_t<1, 256, true>(g, s);
    if (g.pair && g.ares && g.nb == 2 && g.bn == 128) return launch_gemm_pair_t<2, 128, true>(g, s);
    if (g.pair && !g.ares && g.nb == 1 && g.bn == 256) return launch_gemm_pair_t<1, 256, false>(g, s);
    if (g.pair && !g.ares && g.nb == 1 && g.bn == 128) return launch_gemm_pair_t<1, 128, false>(g, s);
    if (g.pair && !g.ares && g.nb == 2 && g.bn == 128) return launch_gemm_pair_t<2, 128, false>(g, s);
    if (g.pair) return SVDMLP_ERR_UNSUPPORTED;
    if (g.nb == 1 && g.bn == 128 && !g.ares) return launch_gemm_t<1, 128, false>(g, s);
    if (g.nb == 1 && g.bn == 256 && !g.ares) return launch_gemm_t<1, 256, false>(g, s);
    if (g.nb == 1 && g.bn == 128 && g.ares) return launch_gemm_t<1, 128, true>(g, s);
    if (g.nb == 2 && g.bn == 128 && g.ares) return launch_gemm_t<2, 128, true>(g, s);
    if (g.nb == 2 && g.bn == 128 && !g.ares) return launch_gemm_t<2, 128, false>(g, s);
    return SVDMLP_ERR_UNSUPPORTED;
}

int num_sms() {
    static int n = 0;
    if (n == 0) {
        int dev = 0;
        cudaGetDevice(&dev);
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    }
    return n;
}

// Gate+up on 256 x 256 pair tiles with both operands streamed (gateup_wide.cuh): ranks above 256.
int launch_gateup_wide(const GemmPlan& g, cudaStream_t s) {
    static bool attr_set = false;
    static int attr_dev = -1;
    int dev = 0;
    cudaGetDevice(&dev);
    if (!attr_set || attr_dev != dev) {
        CUDA_TRY(cudaFuncSetAttribute(tensorpath::gateup_wide_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      tensorpath::kWideSmemBytes));
        attr_set = true;
        attr_dev = dev;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(g.grid); cfg.blockDim = dim3(tensorpath::kPairThreads); cfg.dynamicSmemBytes = tensorpath::kWideSmemBytes; cfg.stream = s;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 2;
    CUDA_TRY(cudaLaunchKernelEx(&cfg, tensorpath::gateup_wide_pair_kernel, g.p));
    return SVDMLP_OK;
}

// Gate+up with the Z strip in tensor memory (gateup_ts.cuh): CTA pairs, 128-column tiles, ranks up to 256.
int launch_gateup_ts(const GemmPlan& g, cudaStream_t s) {
    static bool attr_set = false;
    static int attr_dev = -1;
    int dev = 0;
    cudaGetDevice(&dev);
    if (!attr_set || attr_dev != dev) {
        CUDA_TRY(cudaFuncSetAttribute(tensorpath::gateup_ts_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      tensorpath::kTsSmemBytes));
        attr_set = true;
        attr_dev = dev;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(g.grid); cfg.blockDim = dim3(tensorpath::kPairThreads); cfg.dynamicSmemBytes = tensorpath::kTsSmemBytes; cfg.stream = s;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 2;
    CUDA_TRY(cudaLaunchKernelEx(&cfg, tensorpath::gateup_ts_pair_kernel, g.p));
    return SVDMLP_OK;
}


// Gate+up, SiLU and the first down product in one kernel with H kept on chip (mlp_fused_ts.cuh): ranks up to 128.
int launch_gateup_down1_fused(const GemmPlan& g, cudaStream_t s) {
    static bool attr_set = false;
    static int attr_dev = -1;
    int dev = 0;
    cudaGetDevice(&dev);
    if (!attr_set || attr_dev != dev) {
        CUDA_TRY(cudaFuncSetAttribute(tensorpath::gateup_down1_ts_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      tensorpath::kFuSmemBytes));
        attr_set = true;
        attr_dev = dev;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(g.grid); cfg.blockDim = dim3(tensorpath::kFuThreads); cfg.dynamicSmemBytes = tensorpath::kFuSmemBytes; cfg.stream = s;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 2;
    CUDA_TRY(cudaLaunchKernelEx(&cfg, tensorpath::gateup_down1_ts_pair_kernel, g.p));
    return SVDMLP_OK;
}

// Segments per row-strip pair for the fused kernel: units = pairs x S should fill whole rounds of the CTA pairs.
// Returns 0 if no admissible S keeps at least three quarters of the pairs busy.  With few tokens (one or two
// row-strip pairs) a strip is cut into up to 80 segments of one or two ffn tiles: the partial buffer is sized for
// that at create time (80 splits of at most 1024 rows).
constexpr int kMaxFusedSegments = 80;
int fused_segments(int T, int ffn, int rd, size_t part_elems) {
    const int nc = std::max(1, num_sms() / 2), pairs_m = (T + 255) / 256, tiles_n = (ffn + 127) / 128;
    auto eff_of = [&](int S) {
        const int units = pairs_m * S, rounds = (units + nc - 1) / nc;
        return (double)units / ((double)rounds * nc);
    };
    int s_max = std::min(kMaxFusedSegments, tiles_n);
    while (s_max > 0 && (size_t)s_max * T * rd > part_elems) --s_max;
    double best = 0.0;
    for (int S = 1; S <= s_max; ++S) best = std::max(best, eff_of(S));
    int best_s = 0;
    for (int S = 1; S <= s_max; ++S)
        if (eff_of(S) >= best - 0.03) { best_s = S; break; }   // a finer split must buy 3 % to be worth shorter units
    return best >= 0.75 ? best_s : 0;
}

// Tile width of Zd = H Vd^T (N = r_down): 256 unless the padding of N to whole tiles wastes much more than with
// 128-wide tiles (r = 320: 512 against 384 columns).
int down1_tile_width(int rd) {
    const int pad256 = (rd + 255) / 256 * 256, pad128 = (rd + 127) / 128 * 128;
    return (rd <= 128 || pad256 * 4 > pad128 * 5) ? 128 : 256;
}

// Gate/up at ranks above 256: do 256-wide pair tiles quantise onto the clusters about as well as 128-wide ones?
bool gateup_wide_pays(int tiles_m, int ffn) {
    const long nc = num_sms() / 2, pm = (tiles_m + 1) / 2;
    const long t256 = pm * ((ffn + 255) / 256), t128 = pm * ((ffn + 127) / 128);
    const long rounds256 = (t256 + nc - 1) / nc, rounds128 = (t128 + nc - 1) / nc;
    return 2 * rounds256 * 100 <= rounds128 * 108;
}

// Elements of the split-K partial buffer for a handle made for max_T tokens.
// A split GEMM has at most one tile (128 x 256, or 256 x 256 for a CTA pair) per SM (or SM pair) over all its
// splits, which bounds the partial elements whatever T is; a GEMM that is not split still leaves its one fp32
// copy here; the fused gate/up + down-1 kernel cuts short batches into many ffn segments.
size_t part_elems_for(int max_T, int R, int r_gate, int r_down) {
    const size_t one = (size_t)max_T * std::max(R, r_down);
    size_t n = std::max(one, std::min((size_t)kMaxKSplit * one, (size_t)num_sms() * 128 * 256));
    if (r_gate <= 128 && r_down <= 128)
        n = std::max({n, (size_t)kMaxFusedSegments * std::min(max_T, 1024) * r_down, (size_t)32 * max_T * r_down});
    return n;
}

// How many clusters of four CTAs (two CTA pairs) of the streaming pair kernel can be resident at once: fewer than
// SMs / 4, because a cluster must fit inside one GPC (B200: 33 of 37; clusters of eight: 15 of 18).
int max_active_clusters4() {
    static int n = -1;
    if (n < 0) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(4 * 64); cfg.blockDim = dim3(tensorpath::kPairThreads); cfg.dynamicSmemBytes = kSmemBudget + 1024;
        cudaLaunchAttribute a[1];
        a[0].id = cudaLaunchAttributeClusterDimension;
        a[0].val.clusterDim.x = 4; a[0].val.clusterDim.y = 1; a[0].val.clusterDim.z = 1;
        cfg.attrs = a; cfg.numAttrs = 1;
        int v = 0;
        cudaFuncSetAttribute(tensorpath::gemm_pair_kernel<1, 256, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget + 1024);
        if (cudaOccupancyMaxActiveClusters(&v, tensorpath::gemm_pair_kernel<1, 256, false>, &cfg) != cudaSuccess) { cudaGetLastError(); v = 0; }
        n = v;
    }
    return n;
}

// Fill the shape-dependent part of a plan (tensor maps are set by the caller).
// want_res: keep the A strip resident if it fits.  allow_split: use split-K to fill the machine.
void plan_gemm(GemmPlan& g, int nb, int bn, bool want_res, bool allow_split, int M, int N, int K, int batch,
               bool c_tma = false, bool want_pair = false, int force_ksplit = 0, bool allow_cluster = false) {
    using namespace tensorpath;
    g.nb = nb; g.bn = bn; g.pair = false;
    GemmParams& p = g.p;
    p.M = M; p.N = N; p.K = K; p.batch = batch;
    p.c_tma = c_tma ? 1 : 0;
    p.tiles_m = (M + BM - 1) / BM;
    p.tiles_n = (N + bn - 1) / bn;
    p.chunks_total = (K + BK - 1) / BK;
    const size_t b_bytes = (size_t)bn * BK * 2;
    const size_t a_res_bytes = (size_t)nb * p.chunks_total * kABytes;
    const size_t staging = c_tma ? (size_t)kEpiWarps * 4096 : 0;
    // resident A strip: one ring slot per branch chunk, and at least 4 of them in flight
    g.ares = want_res && (a_res_bytes + staging + 4 * b_bytes + kBarrierBytes <= (size_t)kSmemBudget);
    const size_t slot_bytes = g.ares ? b_bytes : (size_t)nb * (kABytes + b_bytes);
    const size_t fixed = (g.ares ? a_res_bytes : 0) + staging + kBarrierBytes;
    int stages = (int)((kSmemBudget - fixed) / slot_bytes);
    stages = std::max(1, std::min(stages, kMaxStages));
    p.stages = stages;
    g.smem = fixed + (size_t)stages * slot_bytes + 1024;
    const bool stream_pair = want_pair && !g.ares && (nb == 1 || (nb == 2 && bn == 128 && batch == 1)) && p.tiles_m >= 2;
    const int m_units = stream_pair ? (p.tiles_m + 1) / 2 : p.tiles_m;  // tiles (or tile pairs) along M
    const int units = stream_pair ? num_sms() / 2 : num_sms();          // CTAs (or clusters) available
    p.ksplit = 1;
    if (allow_split && !g.ares) {
        const int base_tiles = m_units * p.tiles_n * batch;
        int ks = std::max(1, units / std::max(1, base_tiles));
        ks = std::min(ks, std::max(1, p.chunks_total / 8));  // keep at least 8 chunks per split
        ks = std::min(ks, kMaxKSplit);
        p.ksplit = force_ksplit > 0 ? force_ksplit : ks;   // forced: token slabs of one forward share one partial layout
    }
    p.chunks_per_split = (p.chunks_total + p.ksplit - 1) / p.ksplit;
    p.ksplit = (p.chunks_total + p.chunks_per_split - 1) / p.chunks_per_split;  // no empty split
    const int total = m_units * p.tiles_n * batch * p.ksplit;
    g.grid = std::min(total, num_sms());
    if (stream_pair) {
        p.cps = (nb == 1 && bn == 128) ? 2 : 1;  // narrow tiles: two K chunks per slot, i.e. per wait of the MMA issuer
        const size_t slot = (size_t)p.cps * nb * (kABytes + b_bytes / 2);
        p.stages = std::max(1, std::min((int)((kSmemBudget - fixed) / slot), kMaxStages));
        g.smem = fixed + (size_t)p.stages * slot + 1024;
        g.grid = 2 * std::min(total, num_sms() / 2);
        g.pair = true;
    }
    if (want_pair && g.ares && (bn == 128 || (bn == 256 && nb == 1)) && batch == 1 && p.tiles_m >= 2) {
        // CTA pairs: ring slots hold half a B chunk, so twice as many chunks are in flight
        const size_t half = (size_t)nb * (b_bytes / 2);  // one slot per chunk: every branch's half B chunk
        int st2 = (int)((kSmemBudget - fixed) / half);
        p.stages = std::max(1, std::min(st2, kMaxStages));
        g.smem = fixed + (size_t)p.stages * half + 1024;
        const int pair_tiles = ((p.tiles_m + 1) / 2) * p.tiles_n;
        g.grid = 2 * std::min(pair_tiles, num_sms() / 2);
        g.pair = true;
    }
    p.split_stride = 0; p.batch_col_off = 0; p.resid = nullptr;
    p.a_mn = 0; p.c_t = 0; p.cks = 0;
    // Two splits on CTA pairs: the two pairs that split a tile's K range form one cluster of four CTAs and sum their
    // accumulators through distributed shared memory; the fp32 partial buffer and the reduction launch disappear
    // (config 3: first projection at T = 2048 16.6 -> 14.7 us, first down product at T = 8192 53.9 -> 46.2 us).
    // One tile per cluster (the receive buffers are the ring), 16-bit output only.  Four pairs per cluster (the
    // kernel supports it) measured twice as slow as four partials and a reduction launch (T = 4096: 47.6 against
    // 33.1 us): at most 15 clusters of eight CTAs are resident at once (a cluster must fit inside a GPC) and every
    // shape here has 16 tiles; clusters of four: 33.
    if (allow_cluster && g.pair && !g.ares && nb == 1 && force_ksplit == 0 && p.ksplit == 2) {
        const int cks = 2;
        const int tiles = ((p.tiles_m + 1) / 2) * p.tiles_n * batch;
        const size_t ring_bytes = (size_t)p.stages * (size_t)std::max(1, p.cps) * (kABytes + (size_t)bn / 2 * BK * 2);
        const size_t recv_bytes = (size_t)BM * bn * 4;   // [split][128 rows][bn / cks floats]
        const int cps_k = (p.chunks_total + cks - 1) / cks;
        if (tiles <= max_active_clusters4() && recv_bytes <= ring_bytes && (cks - 1) * cps_k < p.chunks_total) {
            p.cks = cks; p.ksplit = 1; p.chunks_per_split = cps_k;
            g.grid = 2 * cks * tiles;
        }
    }
    if (!(g.pair && !g.ares)) p.cps = 1;
}

}  // namespace

// Token slabs: gate/up and the first half of the down chain run slab by slab so that a slab's H is read back while
// it is still in L2.  Each slab has its own tensor maps (the same buffers, offset by the slab's first row).
struct SlabMaps { CUtensorMap zg, zu, hc, h; };
constexpr int kMaxSlabs = 32;
struct SlabPlan {
    int T, rows, n;   // T the plan was made for (0: none), rows per slab (a multiple of 256), number of slabs
    SlabMaps maps[kMaxSlabs];
};

struct svdmlp {
    int d, ffn, rg, ru, rd, max_T;
    unsigned flags;
    const __nv_bfloat16 *Ug, *Vg, *Uu, *Vu, *Ud, *Vd;
    // skinny-path workspace (fp32 accumulators, zero between calls)
    int t_skinny;  // rows available in Zs/Zds
    float *Zs, *Zds;
    // tensor-path workspace
    bool tensor_ok;
    __half *Z16, *H16, *Zd16;
    __half *Ug16, *Uu16, *Vd16, *Ud16;  // fp16 re-encodings of the second-stage factors (owned)
    float* part;  // split-K partials (shared by stage 1 and the down chain)
    size_t part_elems;
    // pre-norm path / host path staging
    __nv_bfloat16* Xn;
    void *Xdev, *Ydev;
    // svdmlp_forward_host: the copy-in, the forward and the copy-out of the last (X_host, Y_host, T) as one graph
    cudaGraphExec_t host_exec;
    const void* host_x; void* host_y; int host_T;
    unsigned long long host_launches;  // kernels in that graph (added to the launch count on every replay)
    int* status_dev;
    unsigned long long launches;
    // tensor maps that do not depend on the call
    CUtensorMap mVg, mVu, mUg, mUu, mVd, mUd, mZg, mZu, mH, mZd;
    // cached X map and output maps of the TMA-store epilogues (box [32 rows, 64 columns])
    const void* x_ptr; int x_T; CUtensorMap mX;
    CUtensorMap mHc, mYc; const void* y_ptr; int y_T, y_f32;
    float* zd_out32;                  // svdmlp_forward_partial: where the fp32 Zd of this call goes (else NULL)
    unsigned int* tp_counter;         // block counter of the tensor-parallel push kernel (zero between launches)
    unsigned long long tp_limit_ns;   // how long the tensor-parallel gather waits for its peers
    SlabPlan slabs;                   // token slabs of the gate/up -> down-1 pair for the last T seen (maps cached)
    CUtensorMap mUg64, mUu64, mUd64;  // half-tile boxes [64 rows, 64 columns] for the CTA-pair kernels
    CUtensorMap mVg64, mVu64, mVg128, mVu128, mVdHalf;  // half-tile boxes of the first-GEMM factors
    // persistent decode kernel: cached tensor map of X, packed factors (owned), intermediates and barrier words
    CUtensorMap sX; const void* sx_ptr; int sx_T, sx_blocks; bool sx_ok;
    unsigned char *pA, *pB, *pVdp, *pUdp;
    __half* Zp;
    float* Zdp;
    bool persist_ok;
    int persist_grid;               // grid the factors were packed for (the SM count at create time)
    unsigned long long* gridbar;    // 3 words, 128 bytes apart: two arrival counters and the launch number
    unsigned stage_mask;  // measurement aid: which kernels of the path later forwards launch (default all)
    // optional per-kernel event timing
    bool prof;
    int prof_n;
    cudaEvent_t prof_ev[2 * 16];
    const char* prof_name[16];
};

namespace {

// Brackets one kernel launch with events when profiling is on.
struct ProfScope {
    svdmlp* h; cudaStream_t s; int idx;
    ProfScope(svdmlp* h_, const char* name, cudaStream_t s_) : h(h_), s(s_), idx(-1) {
        if (h->prof && h->prof_n < 16) {
            idx = h->prof_n++;
            h->prof_name[idx] = name;
            cudaEventRecord(h->prof_ev[2 * idx], s);
        }
    }
    ~ProfScope() { if (idx >= 0) cudaEventRecord(h->prof_ev[2 * idx + 1], s); }
};

template <int NT>
int skinny_forward_nt(svdmlp* h, const __nv_bfloat16* X, int T, void* Y, int y_fp32, const float* resid,
                      cudaStream_t s) {
    using namespace skinny;
    const int R = h->rg + h->ru;
    const int chunks = (T + NT * 8 - 1) / (NT * 8);
    if (h->stage_mask & 1u) {   // stage 1
        const int kc = 256;
        dim3 grid((R / 16 + 3 + (R % 16 ? 1 : 0)) / 4, (h->d + kc - 1) / kc, chunks);
        size_t smem = (size_t)NT * 8 * (kc + kPad) * 2;
        ProfScope ps(h, "stage1", s);
        stage1_kernel<NT><<<grid, 128, smem, s>>>(X, h->d, T, h->d, h->Vg, h->rg, h->Vu, h->ru, h->Zs, kc, h->Zds,
                                                  (long)T * h->rd);
    }
    if (h->stage_mask & 2u) {   // gate/up expansion + SiLU + first half of the down chain
        dim3 grid((h->ffn + 63) / 64, 1, chunks);
        size_t smem = (size_t)NT * 8 * (2 * (h->rg + kPad) + 2 * (h->ru + kPad) + 2 * (64 + kPad)) * 2 +
                      (size_t)NT * 8 * 65 * 4;
        static size_t smem_set = 0;
        if (smem > 48 * 1024 && smem > smem_set) {
            CUDA_TRY(cudaFuncSetAttribute(gateup_down1_kernel<NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
            smem_set = 227 * 1024;
        }
        ProfScope ps(h, "gateup_down1", s);
        gateup_down1_kernel<NT><<<grid, 256, smem, s>>>(h->Zs, T, h->rg, h->ru, h->Ug, h->Uu, h->ffn, h->Vd, h->rd, h->Zds);
    }
    if (h->stage_mask & 8u) {   // second half of the down chain
        dim3 grid((h->d + 63) / 64, 1, chunks);
        size_t smem = (size_t)NT * 8 * 2 * (h->rd + kPad) * 2;
        static size_t smem_set = 0;
        if (smem > 48 * 1024 && smem > smem_set) {
            CUDA_TRY(cudaFuncSetAttribute(expand_kernel<NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
            smem_set = 227 * 1024;
        }
        ProfScope ps(h, "down2", s);
        expand_kernel<NT><<<grid, 128, smem, s>>>(h->Zds, T, h->rd, h->Ud, h->d, Y, y_fp32, resid, h->Zs, (long)T * R);
    }
    CUDA_TRY(cudaGetLastError());
    h->launches += 3;
    return SVDMLP_OK;
}

template <typename Kern>
int ensure_smem(Kern kern, size_t smem) {
    if (smem > 48 * 1024) CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
    return SVDMLP_OK;
}

constexpr size_t kGridbarBytes = 3 * dpersist::kBarStride * sizeof(unsigned long long);
constexpr size_t kPersistSmemBudget = 227 * 1024 - 64;  // dynamic shared memory next to the kernel's few static bytes

size_t persist_z_bytes(const svdmlp* h) { return (size_t)kSkinnyMaxT * (h->rg + h->ru) * 2; }
size_t persist_zd_bytes(const svdmlp* h) { return (size_t)2 * dpersist::kCopiesZd * ((h->rd + 15) / 16 * 16) * kSkinnyMaxT * 4; }

// State the persistent decode kernel expects between launches: barrier words zero, every Z element
// "unset" (all ones), both Zd buffers zero.
int persist_reset(svdmlp* h, cudaStream_t s) {
    CUDA_TRY(cudaMemsetAsync(h->gridbar, 0, kGridbarBytes, s));
    if (h->Zp) CUDA_TRY(cudaMemsetAsync(h->Zp, 0xFF, persist_z_bytes(h), s));
    if (h->Zdp) CUDA_TRY(cudaMemsetAsync(h->Zdp, 0, persist_zd_bytes(h), s));
    return SVDMLP_OK;
}

dpersist::Shape persist_shape(const svdmlp* h, int T) {
    dpersist::Shape sh;
    sh.T = T; sh.d = h->d; sh.ffn = h->ffn; sh.r = h->rg; sh.rd = h->rd; sh.G = h->persist_grid;
    return sh;
}

// Number of ring slots the persistent decode kernel gets for T tokens (0: the shape does not fit it).
int persist_fit(const svdmlp* h, int T, int nt, int nta, bool fused_norm = false, bool x_res = false);
int persist_slots(const svdmlp* h, int T, int nt, int nta, bool fused_norm = false, bool x_res = false) {
    return h->persist_ok ? persist_fit(h, T, nt, nta, fused_norm, x_res) : 0;
}
// The same for a handle whose packed blocks may not exist yet (create-time planning).
int persist_fit(const svdmlp* h, int T, int nt, int nta, bool fused_norm, bool x_res) {
    if (h->persist_grid <= 0 || h->rg != h->ru || T > 8 * nt || (fused_norm && T > 8)) return 0;
    const dpersist::Shape sh = persist_shape(h, T);
    if (sh.max_a() > 8 * nta || sh.max_b() > dpersist::kNW || sh.max_d() > dpersist::kNW) return 0;
    const dpersist::Layout L = dpersist::make_layout(sh, nt, nta, fused_norm, x_res);
    if ((size_t)L.a_v_off + (size_t)L.ga * sh.max_a() * 32 > (size_t)dpersist::kSlotBytes) return 0;
    const size_t other = (size_t)L.total + dpersist::kRingOverhead + (size_t)L.xres_bytes;
    if (other + 3 * (size_t)dpersist::kSlotBytes > kPersistSmemBudget) return 0;
    return (int)std::min<size_t>(dpersist::kMaxSlots, (kPersistSmemBudget - other) / dpersist::kSlotBytes);
}

// Whole-MLP persistent kernel (decode_persistent.cuh): one cooperative launch per forward.
template <int NT, int NTA, bool FUSED = false>
int persist_forward(svdmlp* h, const __nv_bfloat16* X, int T, void* Y, int y_fp32, const float* resid, cudaStream_t s,
                    const float* hin = nullptr, float eps = 0.f) {
    dpersist::Params p;
    p.hin = hin; p.eps = eps;
    p.s = persist_shape(h, T);
    p.X = X; p.pA = h->pA; p.pB = h->pB; p.pVd = h->pVdp; p.pUd = h->pUdp;
    p.Z = h->Zp; p.Zd = h->Zdp; p.Y = Y; p.y_fp32 = y_fp32; p.resid = resid;
    p.bar = h->gridbar; p.status = h->status_dev;
    // X: resident (one TMA box for the whole of X, if it is small enough to sit next to the ring), or one TMA box
    // per group, or - when d is not a multiple of 64 or the map cannot be made - one bulk copy per token row.
    // Maps are cached per X pointer, T and box size.
    p.x_tma = 0; p.x_res = 0;
    auto x_map = [&](int blocks) {
        if (h->sx_ptr != X || h->sx_T != T || h->sx_blocks != blocks) {
            h->sx_ok = make_map_x3(&h->sX, X, T, h->d, blocks) == SVDMLP_OK;
            h->sx_ptr = X; h->sx_T = T; h->sx_blocks = blocks;
        }
        if (h->sx_ok) p.mX = h->sX;
        return h->sx_ok;
    };
    const bool can_tma = hin == nullptr && h->d % 64 == 0;
    if (can_tma && h->d / 64 <= 256 && (size_t)T * h->d * 2 <= 65536 && persist_slots(h, T, NT, NTA, false, true) >= 4 &&
        x_map(h->d / 64)) {
        p.x_tma = 1; p.x_res = 1;
    }
    p.nslot = persist_slots(h, T, NT, NTA, hin != nullptr, p.x_res != 0);
    const dpersist::Layout L = dpersist::make_layout(p.s, NT, NTA, hin != nullptr, p.x_res != 0);
    if (can_tma && !p.x_res && x_map(L.ga / 4)) p.x_tma = 1;
    const size_t smem = (size_t)L.total + dpersist::kRingOverhead + (size_t)L.xres_bytes + (size_t)p.nslot * dpersist::kSlotBytes;
    p.window = std::min(p.nslot - 1, 2);
    static bool smem_set = false;  // per instantiation
    if (!smem_set) {
        CUDA_TRY(cudaFuncSetAttribute(dpersist::mlp_kernel<NT, NTA, FUSED>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kPersistSmemBudget));
        smem_set = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(h->persist_grid); cfg.blockDim = dim3(dpersist::kThreads); cfg.dynamicSmemBytes = smem; cfg.stream = s;
    // The CTAs wait on one another, so all of them must become resident: one CTA per SM and a grid of at most
    // the SM count.  Default: programmatic dependent launch (a CTA starts on an SM as soon as the preceding
    // kernel's CTA has left it and orders itself behind that kernel with griddepcontrol.wait; 0.6 us per step
    // less than a cooperative launch, which drains the GPU first).  SVDMLP_FLAG_DECODE_COOPERATIVE asks for the
    // cooperative launch, whose residency the driver guarantees even when other work shares the GPU.
    cudaLaunchAttribute attr[1];
    if (h->flags & SVDMLP_FLAG_DECODE_COOPERATIVE) {
        attr[0].id = cudaLaunchAttributeCooperative;
        attr[0].val.cooperative = 1;
    } else {
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
    }
    cfg.attrs = attr; cfg.numAttrs = 1;
    {
        ProfScope ps(h, "mlp_decode", s);
        CUDA_TRY(cudaLaunchKernelEx(&cfg, dpersist::mlp_kernel<NT, NTA, FUSED>, p));
    }
    h->launches += 1;
    return SVDMLP_OK;
}

size_t skinny_smem_need(const svdmlp* h, int nt) {
    size_t a = (size_t)nt * 8 * (2 * (h->rg + skinny::kPad) + 2 * (h->ru + skinny::kPad) + 2 * (64 + skinny::kPad)) * 2 +
               (size_t)nt * 8 * 65 * 4;
    size_t b = (size_t)nt * 8 * 2 * (h->rd + skinny::kPad) * 2;
    return std::max(a, b);
}

// hin != nullptr: X = RMSNorm(hin) is wanted and has NOT been computed; returns SVDMLP_ERR_UNSUPPORTED if the
// persistent kernel (the only one with the normalisation built in) cannot take the shape.
int skinny_forward(svdmlp* h, const __nv_bfloat16* X, int T, void* Y, int y_fp32, const float* resid, cudaStream_t s,
                   const float* hin = nullptr, float eps = 0.f) {
    if (T > h->t_skinny) return SVDMLP_ERR_INVALID_ARG;
    int nt = T <= 8 ? 1 : T <= 16 ? 2 : 4;
    if (h->stage_mask == ~0u && h->persist_ok) {
        const int nta = persist_shape(h, T).max_a() <= 8 ? 1 : 2;
        if (persist_slots(h, T, nt, nta, hin != nullptr) > 0) {
            if (nta == 1) {
                if (nt == 1) return hin ? persist_forward<1, 1, true>(h, X, T, Y, y_fp32, resid, s, hin, eps) : persist_forward<1, 1>(h, X, T, Y, y_fp32, resid, s);
                if (nt == 2) return persist_forward<2, 1>(h, X, T, Y, y_fp32, resid, s);
                return persist_forward<4, 1>(h, X, T, Y, y_fp32, resid, s);
            }
            if (nt == 1) return hin ? persist_forward<1, 2, true>(h, X, T, Y, y_fp32, resid, s, hin, eps) : persist_forward<1, 2>(h, X, T, Y, y_fp32, resid, s);
            if (nt == 2) return persist_forward<2, 2>(h, X, T, Y, y_fp32, resid, s);
            return persist_forward<4, 2>(h, X, T, Y, y_fp32, resid, s);
        }
    }
    if (hin != nullptr) return SVDMLP_ERR_UNSUPPORTED;
    while (nt > 1 && skinny_smem_need(h, nt) > 227 * 1024) nt >>= 1;
    if (skinny_smem_need(h, nt) > 227 * 1024) return SVDMLP_ERR_UNSUPPORTED;
    if (nt == 1) return skinny_forward_nt<1>(h, X, T, Y, y_fp32, resid, s);
    if (nt == 2) return skinny_forward_nt<2>(h, X, T, Y, y_fp32, resid, s);
    return skinny_forward_nt<4>(h, X, T, Y, y_fp32, resid, s);
}

// Failure-detection self-test: one warp waits, through the same bounded-wait routine as the production
// kernels, on a barrier that nothing ever signals; when the limit passes it records the timeout status and
// returns normally.  Nothing faults, traps or spins without bound.
__global__ void __launch_bounds__(32) wait_selftest_kernel(int* status, unsigned long long limit_ns) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) { umma::mbar_init(&bar, 1); abort_flag = 0; umma::fence_mbar_init(); }
    __syncwarp();
    const bool ok = umma::mbar_wait_for(&bar, 0, &abort_flag, limit_ns, 1);
    if (!ok && threadIdx.x == 0 && status != nullptr) atomicExch(status, SVDMLP_ERR_TIMEOUT);
}

// One line per change of kernel path when SVDMLP_LOG=1 is set in the environment (stderr).
void log_path(const svdmlp* h, int T, const char* path) {
    static const bool on = [] { const char* e = getenv("SVDMLP_LOG"); return e != nullptr && e[0] == '1'; }();
    static const svdmlp* last_h = nullptr;
    static int last_T = -1;
    if (!on || (last_h == h && last_T == T)) return;
    last_h = h; last_T = T;
    fprintf(stderr, "[svdmlp] handle %p T=%d d=%d ffn=%d r=(%d,%d,%d): %s\n", (const void*)h, T, h->d, h->ffn, h->rg, h->ru, h->rd, path);
}

int launch_convert(const void* in, __half* out, long n, int* flag, cudaStream_t s) {
    int blocks = (int)std::min<long>((n / 8 + 255) / 256, 8 * num_sms());
    tensorpath::bf16_to_f16_kernel<<<std::max(blocks, 1), 256, 0, s>>>((const __nv_bfloat16*)in, out, n, flag);
    CUDA_TRY(cudaGetLastError());
    return SVDMLP_OK;
}

int launch_reduce(const float* part, int ksplit, long split_stride, long n, __half* out, cudaStream_t s, float* out32 = nullptr) {
    const bool wide = ksplit > 16;   // many splits: eight threads share an output quad (a block covers 128 outputs)
    int blocks = wide ? (int)std::min<long>((n + 127) / 128, 8 * num_sms()) : (int)std::min<long>((n / 4 + 255) / 256, 4 * num_sms());
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(std::max(blocks, 1)); cfg.blockDim = dim3(256); cfg.dynamicSmemBytes = 0; cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    if (wide) CUDA_TRY(cudaLaunchKernelEx(&cfg, tensorpath::reduce_partials_wide_kernel, part, ksplit, split_stride, n, out, out32));
    else CUDA_TRY(cudaLaunchKernelEx(&cfg, tensorpath::reduce_partials_kernel, part, ksplit, split_stride, n, out, out32));
    return SVDMLP_OK;
}

// H bytes one slab may hold with SVDMLP_FLAG_TOKEN_SLABS: inside the 126 MB L2 next to the factors, Z and the
// split-K partials.  Without the flag the two kernels run over all T rows at once: measured on B200, every slab
// boundary (two more launches, fewer tiles per wave, deeper split-K) costs more than the HBM traffic of H it
// saves (config 4, r = 128, T = 8192: 159 us unslabbed, 192 / 202 / 232 us with 64 / 48 / 32 MB slabs).
constexpr size_t kSlabBytes = (size_t)64 << 20;

const SlabPlan* slab_plan(svdmlp* h, int T) {
    SlabPlan& sp = h->slabs;
    if (sp.T == T) return &sp;
    const size_t row_bytes = (size_t)h->ffn * 2;
    int n = 1;
    if ((h->flags & SVDMLP_FLAG_TOKEN_SLABS) && (size_t)T * row_bytes > kSlabBytes + kSlabBytes / 2)
        n = (int)(((size_t)T * row_bytes + kSlabBytes - 1) / kSlabBytes);
    n = std::min(n, kMaxSlabs);
    int rows = ((T + n - 1) / n + 255) / 256 * 256;   // whole CTA-pair row strips
    n = (T + rows - 1) / rows;
    const int R = h->rg + h->ru;
    for (int i = 0; i < n; ++i) {
        const int row0 = i * rows, Ts = std::min(rows, T - row0);
        SlabMaps& m = sp.maps[i];
        if (make_map(&m.zg, h->Z16 + (size_t)row0 * R, Ts, h->rg, R, 128) != SVDMLP_OK ||
            make_map(&m.zu, h->Z16 + (size_t)row0 * R + h->rg, Ts, h->ru, R, 128) != SVDMLP_OK ||
            make_map(&m.hc, h->H16 + (size_t)row0 * h->ffn, Ts, h->ffn, h->ffn, 32) != SVDMLP_OK ||
            make_map(&m.h, h->H16 + (size_t)row0 * h->ffn, Ts, h->ffn, h->ffn, 128) != SVDMLP_OK) {
            sp.T = 0;
            return nullptr;
        }
    }
    sp.T = T; sp.rows = rows; sp.n = n;
    return &sp;
}

// Segments of the fused gate/up + down-1 kernel for this handle and T, 0 if the two-kernel form runs instead.
int fused_plan(const svdmlp* h, int T) {
    if (!h->tensor_ok || (h->flags & (SVDMLP_FLAG_NO_CTA_PAIRS | SVDMLP_FLAG_NO_TMEM_STRIP | SVDMLP_FLAG_NO_FUSED_DOWN1 | SVDMLP_FLAG_TOKEN_SLABS)))
        return 0;
    if (h->rg != h->ru || h->rg > 128 || h->rd > 128) return 0;
    return fused_segments(T, h->ffn, h->rd, h->part_elems);
}

int tensor_forward(svdmlp* h, const __nv_bfloat16* X, int T, void* Y, int y_fp32, const float* resid, cudaStream_t s) {
    using namespace tensorpath;
    if (!h->tensor_ok) return SVDMLP_ERR_UNSUPPORTED;
    const int R = h->rg + h->ru;
    int rc;
    if ((h->stage_mask & 1u) && (h->x_ptr != X || h->x_T != T)) {
        if ((rc = make_map(&h->mX, X, T, h->d, h->d, BM)) != SVDMLP_OK) return rc;
        h->x_ptr = X; h->x_T = T;
    }
    GemmPlan g;
    const unsigned mask = h->stage_mask;
    const bool pairs_ok = !(h->flags & SVDMLP_FLAG_NO_CTA_PAIRS);
    // 1. Z = X [Vg; Vu]^T   (phase 1 of Algorithm 3), fp16 out
    if (mask & 1u) {
    // ranks that are whole 256-column tiles, with enough tiles to fill the machine without splitting K: 256 x 256 pair
    // tiles halve the re-reads of X (r = 256, T = 8192: 34.5 -> 29.5 us; with fewer tiles the split and its sum cost more)
    const int bn1 = (pairs_ok && h->rg >= 256 && h->rg % 256 == 0 && (long)((T + 255) / 256) * (h->rg / 256) * 2 >= 48) ? 256 : 128;
    plan_gemm(g, 1, bn1, false, true, T, h->rg, h->d, 2, false, pairs_ok, 0, !(h->flags & SVDMLP_FLAG_NO_CLUSTER_SPLITK));
    g.p.tmA[0] = h->mX; g.p.tmA[1] = h->mX;
    g.p.tmB[0] = g.pair ? (bn1 == 256 ? h->mVg128 : h->mVg64) : h->mVg; g.p.tmB[1] = g.pair ? (bn1 == 256 ? h->mVu128 : h->mVu64) : h->mVu;
    g.p.a_fmt = umma::kFmtBF16; g.p.b_fmt = umma::kFmtBF16; g.p.status = h->status_dev;
    g.p.batch_col_off = h->rg;
    if (g.p.ksplit > 1) {
        if ((size_t)g.p.ksplit * T * R > h->part_elems) return SVDMLP_ERR_NOMEM;
        g.p.C = h->part; g.p.ldc = R; g.p.split_stride = (long)T * R; g.p.out_mode = OUT_F32;
        { ProfScope ps(h, "stage1", s); rc = launch_gemm(g, s); }
        if (rc != SVDMLP_OK) return rc;
        { ProfScope ps(h, "stage1_reduce", s); rc = launch_reduce(h->part, g.p.ksplit, (long)T * R, (long)T * R, h->Z16, s); }
        if (rc != SVDMLP_OK) return rc;
        h->launches += 2;
    } else {
        g.p.C = h->Z16; g.p.ldc = R; g.p.out_mode = OUT_F16;
        { ProfScope ps(h, "stage1", s); rc = launch_gemm(g, s); }
        if (rc != SVDMLP_OK) return rc;
        h->launches += 1;
    }
    }
    // 2. H = SiLU(Zg Ug^T) .* (Zu Uu^T)   (phase 2 of Algorithm 3 with its epilogue), fp16 out
    // 3. Zd = H Vd^T   (phase 1 of the down-projection XUV chain), split-K fp32 partials -> fp16
    // On request (SVDMLP_FLAG_TOKEN_SLABS) the two run slab by slab over the token rows when H as a whole would
    // not stay in L2 between its one write and its one read (the analogue of the paper's row-strip loop,
    // Section 4.2.1): a slab's H is produced and consumed while it is still cache-resident.
    const SlabPlan* sp = slab_plan(h, T);
    if (sp == nullptr) return SVDMLP_ERR_CUDA;
    int down1_ksplit = 0;
    bool down1_in_cluster = false;
    // Ranks up to 128: both products in one kernel, H stays in shared memory (mlp_fused_ts.cuh)
    const int fused_S = ((mask & 6u) == 6u && sp->n == 1) ? fused_plan(h, T) : 0;
    if (fused_S > 0) {
        plan_gemm(g, 2, 128, true, false, T, h->ffn, h->rg, 1, true, true);
        g.p.tmA[0] = h->mZg; g.p.tmA[1] = h->mZu;
        g.p.tmB[0] = h->mUg64; g.p.tmB[1] = h->mUu64;
        g.p.tmC = h->mVdHalf;
        g.p.a_fmt = umma::kFmtF16; g.p.b_fmt = umma::kFmtF16; g.p.status = h->status_dev;
        g.p.C = h->part; g.p.ldc = h->rd; g.p.split_stride = (long)T * h->rd; g.p.out_mode = OUT_F32;
        g.p.ksplit = fused_S; g.p.stages = tensorpath::kFuSlots;
        g.grid = 2 * std::min(((g.p.tiles_m + 1) / 2) * fused_S, num_sms() / 2);
        { ProfScope ps(h, "gateup_down1", s); rc = launch_gateup_down1_fused(g, s); }
        if (rc != SVDMLP_OK) return rc;
        { ProfScope ps(h, "down1_reduce", s); rc = launch_reduce(h->part, fused_S, (long)T * h->rd, (long)T * h->rd, h->Zd16, s, h->zd_out32); }
        if (rc != SVDMLP_OK) return rc;
        h->launches += 2;
    } else {
    for (int si = 0; si < sp->n; ++si) {
    const int row0 = si * sp->rows, Ts = std::min(sp->rows, T - row0);
    const SlabMaps& sm = sp->maps[si];
    if (mask & 2u) {
    plan_gemm(g, 2, 128, true, false, Ts, h->ffn, h->rg, 1, true, !(h->flags & SVDMLP_FLAG_NO_CTA_PAIRS));
    g.p.tmC = sm.hc;
    g.p.tmA[0] = sm.zg; g.p.tmA[1] = sm.zu;
    g.p.tmB[0] = g.pair ? h->mUg64 : h->mUg; g.p.tmB[1] = g.pair ? h->mUu64 : h->mUu;
    g.p.a_fmt = umma::kFmtF16; g.p.b_fmt = umma::kFmtF16; g.p.status = h->status_dev;
    g.p.C = h->H16 + (size_t)row0 * h->ffn; g.p.ldc = h->ffn; g.p.out_mode = OUT_F16;
    // ranks up to 256 on CTA pairs: the Z strip lives in tensor memory and the branches run one after the other
    const bool ts = g.pair && g.ares && h->rg == h->ru && h->rg <= 256 && !(h->flags & SVDMLP_FLAG_NO_TMEM_STRIP);
    if (ts) {
        g.p.stages = tensorpath::kTsMaxSlots;
        g.grid = 2 * std::min(((g.p.tiles_m + 1) / 2) * g.p.tiles_n, num_sms() / 2);
    }
    // ranks above 256 on CTA pairs: 256-wide tiles (an N = 256 MMA outlasts the tensor core's issue interval), when
    // the tile count quantises onto the clusters about as well as 128-wide tiles do
    bool wide = false;
    if (!ts && g.pair && !g.ares && h->rg == h->ru && h->rg > 256 && !(h->flags & SVDMLP_FLAG_NO_WIDE_GATEUP)) {
        const long nc = num_sms() / 2, t256 = (long)((g.p.tiles_m + 1) / 2) * ((h->ffn + 255) / 256);
        wide = gateup_wide_pays(g.p.tiles_m, h->ffn);
        if (wide) {
            g.p.tiles_n = (h->ffn + 255) / 256;
            g.grid = 2 * (int)std::min<long>(t256, nc);
            g.p.tmB[0] = h->mUg; g.p.tmB[1] = h->mUu;
        }
    }
    { ProfScope ps(h, "gateup", s); rc = ts ? launch_gateup_ts(g, s) : wide ? launch_gateup_wide(g, s) : launch_gemm(g, s); }
    if (rc != SVDMLP_OK) return rc;
    h->launches += 1;
    }
    if (mask & 4u) {
    const int bn3 = down1_tile_width(h->rd);
    // (the sum inside a cluster writes fp16 Zd itself: not when the caller wants the fp32 sum, not with token slabs)
    const bool cl_ok = sp->n == 1 && h->zd_out32 == nullptr && !(h->flags & SVDMLP_FLAG_NO_CLUSTER_SPLITK);
    plan_gemm(g, 1, bn3, false, true, Ts, h->rd, h->ffn, 1, false, pairs_ok, down1_ksplit, cl_ok);
    if (si == 0) down1_ksplit = g.p.ksplit;
    if (g.p.ksplit != down1_ksplit) return SVDMLP_ERR_UNSUPPORTED;  // cannot happen: the split depends on K alone once forced
    g.p.tmA[0] = sm.h; g.p.tmA[1] = sm.h;
    g.p.tmB[0] = g.pair ? h->mVdHalf : h->mVd; g.p.tmB[1] = g.p.tmB[0];
    g.p.a_fmt = umma::kFmtF16; g.p.b_fmt = umma::kFmtF16; g.p.status = h->status_dev;
    down1_in_cluster = g.p.cks > 1;
    if (down1_in_cluster) {
        g.p.C = h->Zd16; g.p.ldc = h->rd; g.p.out_mode = OUT_F16;
    } else {
        if ((size_t)g.p.ksplit * T * h->rd > h->part_elems) return SVDMLP_ERR_NOMEM;
        g.p.C = h->part + (size_t)row0 * h->rd; g.p.ldc = h->rd; g.p.split_stride = (long)T * h->rd; g.p.out_mode = OUT_F32;
    }
    { ProfScope ps(h, "down1", s); rc = launch_gemm(g, s); }
    if (rc != SVDMLP_OK) return rc;
    h->launches += 1;
    }
    }
    if ((mask & 4u) && !down1_in_cluster) {
    { ProfScope ps(h, "down1_reduce", s); rc = launch_reduce(h->part, down1_ksplit, (long)T * h->rd, (long)T * h->rd, h->Zd16, s, h->zd_out32); }
    if (rc != SVDMLP_OK) return rc;
    h->launches += 1;
    }
    }   // not fused
    // 4. Y = Zd Ud^T   (phase 2 of the XUV chain)
    if (mask & 8u) {
    const bool y_tma = true;  // bf16 and fp32 (+ residual) outputs both leave through TMA stores
    if (h->y_ptr != Y || h->y_T != T || h->y_f32 != y_fp32) {
        rc = y_fp32 ? make_map_f32(&h->mYc, Y, T, h->d, h->d) : make_map(&h->mYc, Y, T, h->d, h->d, 32);
        if (rc != SVDMLP_OK) return rc;
        h->y_ptr = Y; h->y_T = T; h->y_f32 = y_fp32;
    }
    // an MMA with N = 128 reads 128 B/clk of operands from shared memory (its limit); N = 256 reads 96 B/clk
    // (wide tiles unless their coarser quantisation over the CTA pairs costs more than that gains)
    const int pairs = std::max(1, num_sms() / 2), pm = (T + 2 * BM - 1) / (2 * BM);
    const int waves256 = 2 * ((pm * ((h->d + 255) / 256) + pairs - 1) / pairs), waves128 = (pm * ((h->d + 127) / 128) + pairs - 1) / pairs;
    const bool wide2 = pairs_ok && T > BM && waves256 * 100 <= waves128 * 115;
    plan_gemm(g, 1, wide2 ? 256 : 128, true, false, T, h->d, h->rd, 1, y_tma, pairs_ok);
    if (!g.ares && pairs_ok && T > BM) plan_gemm(g, 1, 256, false, false, T, h->d, h->rd, 1, y_tma, true);  // Zd strip too wide to keep: stream 256 x 256 pair tiles
    if (y_tma) g.p.tmC = h->mYc;
    g.p.tmA[0] = h->mZd; g.p.tmA[1] = h->mZd;
    g.p.tmB[0] = g.pair ? (g.bn == 256 ? h->mUd : h->mUd64) : h->mUd; g.p.tmB[1] = g.p.tmB[0];
    g.p.a_fmt = umma::kFmtF16; g.p.b_fmt = umma::kFmtF16; g.p.status = h->status_dev;
    g.p.C = Y; g.p.ldc = h->d; g.p.out_mode = y_fp32 ? OUT_F32 : OUT_BF16; g.p.resid = resid;
    { ProfScope ps(h, "down2", s); rc = launch_gemm(g, s); }
    if (rc != SVDMLP_OK) return rc;
    h->launches += 1;
    }
    return SVDMLP_OK;
}

// Does the persistent decode kernel's shared-memory layout fit for T tokens (whether or not its blocks are packed)?
bool persist_takes(const svdmlp* h, int T) {
    if (h->persist_grid <= 0) return false;
    const int nt = T <= 8 ? 1 : T <= 16 ? 2 : 4;
    const int nta = persist_shape(h, T).max_a() <= 8 ? 1 : 2;
    return persist_fit(h, T, nt, nta) > 0;
}

bool use_skinny(const svdmlp* h, int T) {
    if (h->flags & SVDMLP_FLAG_PATH_SKINNY) return true;
    if (h->flags & SVDMLP_FLAG_PATH_TENSOR) return false;
    if (T > kSkinnyMaxT) return !h->tensor_ok;
    if (T <= 8 || !h->tensor_ok) return true;
    // 8 < T <= 32: the persistent kernel if it takes the shape; its three-kernel fallback is slower here than the
    // tcgen05 kernels (T = 32, ranks 1024: 147 us against 48 us)
    return h->persist_ok && persist_takes(h, T);
}

int forward_impl(svdmlp* h, const __nv_bfloat16* X, int T, void* Y, int y_fp32, const float* resid, cudaStream_t s,
                 bool keep_prof = false) {
    if (!keep_prof) h->prof_n = 0;
    log_path(h, T, use_skinny(h, T) ? "weight-streaming (small T) kernels" : "tcgen05 (large T) kernels");
    if (use_skinny(h, T)) return skinny_forward(h, X, T, Y, y_fp32, resid, s);
    return tensor_forward(h, X, T, Y, y_fp32, resid, s);
}

}  // namespace

extern "C" {

const char* svdmlp_strerror(int status) {
    switch (status) {
        case SVDMLP_OK: return "ok";
        case SVDMLP_ERR_INVALID_ARG: return "invalid argument";
        case SVDMLP_ERR_UNSUPPORTED: return "unsupported shape for the selected kernel path";
        case SVDMLP_ERR_ALIGNMENT: return "pointer not 16-byte aligned or dimension not a multiple of 8";
        case SVDMLP_ERR_CUDA: return "CUDA call failed";
        case SVDMLP_ERR_ARCH: return "device is not compute capability 10.x (sm_100)";
        case SVDMLP_ERR_NOMEM: return "out of device memory or workspace too small";
        case SVDMLP_ERR_TIMEOUT: return "a bounded device-side wait timed out";
        default: return "unknown status";
    }
}

int svdmlp_block_aligned_rank(int k, int n, double ratio, int block, double alpha) {
    if (k <= 0 || n <= 0 || block <= 0 || !(ratio >= 0.0) || !(ratio < 1.0) || !(alpha >= 0.0) || !(alpha <= 1.0))
        return SVDMLP_ERR_INVALID_ARG;
    const double x = (double)k * (double)n * (1.0 - ratio) / (((double)k + (double)n) * (double)block) + alpha;
    const long long q = (long long)floor(x);
    const long long r = q * (long long)block;
    return r > 0x7fffffffLL ? SVDMLP_ERR_INVALID_ARG : (int)r;
}

int svdmlp_model(int d, int ffn, int r, int T, double tensor_tflops, double hbm_gbs, double l2_bytes, svdmlp_model_t* out) {
    if (out == nullptr || d <= 0 || ffn <= 0 || r <= 0 || T <= 0) return SVDMLP_ERR_INVALID_ARG;
    if (!(tensor_tflops > 0.0)) tensor_tflops = 1648.0;
    if (!(hbm_gbs > 0.0)) hbm_gbs = 6547.0;
    if (!(l2_bytes > 0.0)) l2_bytes = 126e6;
    svdmlp_model_t m;
    memset(&m, 0, sizeof(m));
    m.d = d; m.ffn = ffn; m.r = r; m.T = T;
    // the routing of svdmlp_forward, on a handle that holds the shape only
    svdmlp* h = new (std::nothrow) svdmlp();
    if (h == nullptr) return SVDMLP_ERR_NOMEM;
    memset(h, 0, sizeof(*h));
    h->d = d; h->ffn = ffn; h->rg = h->ru = h->rd = r; h->max_T = T;
    h->persist_grid = num_sms(); h->persist_ok = true; h->tensor_ok = true; h->stage_mask = ~0u;
    h->part_elems = part_elems_for(T, 2 * r, r, r);
    const bool stream_weights = use_skinny(h, T);
    const int S = stream_weights ? 0 : fused_plan(h, T);
    delete h;
    const double s2 = 2.0;  // bytes per element of X, Y, the factors and the 16-bit intermediates
    m.flops = 2.0 * T * r * (3.0 * d + 3.0 * ffn);
    const double factors = s2 * 3.0 * r * ((double)d + ffn), h_bytes = s2 * T * (double)ffn;
    if (stream_weights) {
        m.path = 0;
        m.strip_rows = T <= 8 ? 8 : T <= 16 ? 16 : 32;
        // mma.sync path: no tensor memory; shared memory = the whole opt-in budget (ring slots take what the
        // activations leave)
        m.smem_bytes = (long)kPersistSmemBudget;
    } else {
        using namespace tensorpath;
        m.path = S > 0 ? 2 : 1;
        const int tiles_m = (T + BM - 1) / BM;
        m.strip_rows = tiles_m >= 2 ? 2 * BM : BM;
        GemmPlan g;
        plan_gemm(g, 2, 128, true, false, T, ffn, r, 1, true, true);
        const bool ts = g.pair && g.ares && r <= 256;
        const bool wide = !ts && g.pair && !g.ares && r > 256 && gateup_wide_pays(g.p.tiles_m, ffn);
        if (S > 0) {          // strips [0, 128), Zd [128, 256), G [256, 384), Up [384, 512)
            m.z_in_tmem = 1; m.tmem_cols_strip = 128; m.tmem_cols_zd = 128; m.tmem_cols_acc = 256;
            m.smem_bytes = kFuSmemBytes;
        } else if (ts) {      // gate strip [0, 128), up strip [128, 256), G [256, 384), Up [384, 512)
            m.z_in_tmem = 1; m.tmem_cols_strip = 256; m.tmem_cols_acc = 256;
            m.smem_bytes = kTsSmemBytes;
        } else if (wide) {    // two 256-column accumulators, both operands streamed
            m.tmem_cols_acc = 512;
            m.smem_bytes = kWideSmemBytes;
        } else {              // 128-wide tiles, G and Up double-buffered; the Z strip in shared memory if it fits
            m.tmem_cols_acc = 512;
            m.smem_bytes = (long)g.smem;
        }
    }
    m.tmem_cols_total = m.tmem_cols_strip + m.tmem_cols_acc + m.tmem_cols_zd;
    const bool h_fused = m.path != 1;   // decode and fused kernels keep H on the SM
    m.hbm_bytes = factors + 2.0 * s2 * T * (double)d + ((!h_fused && h_bytes > l2_bytes) ? 2.0 * h_bytes : 0.0);
    const double strips = (double)((T + m.strip_rows - 1) / m.strip_rows);
    // X and Y once; the factors once per row strip; Z (2r) and Zd (r) written and read once; H written and read once
    m.sm_bytes = 2.0 * s2 * T * (double)d + strips * factors + 2.0 * s2 * T * 3.0 * r + (h_fused ? 0.0 : 2.0 * h_bytes);
    m.intensity_hbm = m.flops / m.hbm_bytes;
    m.intensity_sm = m.flops / m.sm_bytes;
    m.ridge_hbm = tensor_tflops * 1e3 / hbm_gbs;
    m.t_tensor_us = m.flops / (tensor_tflops * 1e6);
    m.t_hbm_us = m.hbm_bytes / (hbm_gbs * 1e3);
    m.t_floor_us = std::max(m.t_tensor_us, m.t_hbm_us);
    *out = m;
    return SVDMLP_OK;
}

int svdmlp_create(svdmlp_t** out, int d, int ffn, int r_gate, int r_up, int r_down, const void* Ug, const void* Vg,
                  const void* Uu, const void* Vu, const void* Ud, const void* Vd, int max_T, unsigned flags,
                  void* stream) {
    if (out == nullptr) return SVDMLP_ERR_INVALID_ARG;
    *out = nullptr;
    if (d <= 0 || ffn <= 0 || r_gate <= 0 || r_up <= 0 || r_down <= 0 || max_T <= 0) return SVDMLP_ERR_INVALID_ARG;
    if (!Ug || !Vg || !Uu || !Vu || !Ud || !Vd) return SVDMLP_ERR_INVALID_ARG;
    if ((flags & SVDMLP_FLAG_PATH_SKINNY) && (flags & SVDMLP_FLAG_PATH_TENSOR)) return SVDMLP_ERR_INVALID_ARG;
    if ((d | ffn | r_gate | r_up | r_down) & 7) return SVDMLP_ERR_ALIGNMENT;
    if (!aligned16(Ug) || !aligned16(Vg) || !aligned16(Uu) || !aligned16(Vu) || !aligned16(Ud) || !aligned16(Vd))
        return SVDMLP_ERR_ALIGNMENT;
    int rc = check_arch();
    if (rc != SVDMLP_OK) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    svdmlp* h = new (std::nothrow) svdmlp();
    if (h == nullptr) return SVDMLP_ERR_NOMEM;
    memset(h, 0, sizeof(*h));
    h->stage_mask = ~0u;
    h->d = d; h->ffn = ffn; h->rg = r_gate; h->ru = r_up; h->rd = r_down; h->max_T = max_T; h->flags = flags;
    h->Ug = (const __nv_bfloat16*)Ug; h->Vg = (const __nv_bfloat16*)Vg; h->Uu = (const __nv_bfloat16*)Uu;
    h->Vu = (const __nv_bfloat16*)Vu; h->Ud = (const __nv_bfloat16*)Ud; h->Vd = (const __nv_bfloat16*)Vd;
    const int R = r_gate + r_up;
    h->tensor_ok = (r_gate == r_up) && !(flags & SVDMLP_FLAG_PATH_SKINNY);
    const bool need_skinny = !(flags & SVDMLP_FLAG_PATH_TENSOR);
    h->t_skinny = !need_skinny ? 0 : (h->tensor_ok ? std::min(max_T, kSkinnyMaxT) : max_T);
    bool ok = true;
    auto alloc = [&](void** p, size_t bytes) {
        if (!ok) return;
        if (cudaMalloc(p, std::max<size_t>(bytes, 256)) != cudaSuccess) { cudaGetLastError(); ok = false; *p = nullptr; }
    };
    alloc((void**)&h->status_dev, sizeof(int));
    alloc((void**)&h->gridbar, kGridbarBytes);
    alloc((void**)&h->tp_counter, 256);
    h->tp_limit_ns = 2000000000ull;
    if (h->t_skinny > 0) {
        alloc((void**)&h->Zs, (size_t)h->t_skinny * R * 4);
        alloc((void**)&h->Zds, (size_t)h->t_skinny * r_down * 4);
    }
    // The tcgen05 kernels (and their fp16 copies of the second-stage factors) are set up when some T needs them:
    // above 32 tokens, on request, or between 9 and 32 tokens when the persistent decode kernel cannot take the shape.
    h->persist_grid = (r_gate == r_up && !(flags & SVDMLP_FLAG_DECODE_REGISTERS)) ? num_sms() : 0;
    const bool mid_needs_tensor = max_T > 8 && !persist_takes(h, std::min(max_T, kSkinnyMaxT));
    if (h->tensor_ok && (max_T > kSkinnyMaxT || mid_needs_tensor || (flags & SVDMLP_FLAG_PATH_TENSOR))) {
        alloc((void**)&h->Z16, (size_t)max_T * R * 2);
        alloc((void**)&h->H16, (size_t)max_T * ffn * 2);
        alloc((void**)&h->Zd16, (size_t)max_T * r_down * 2);
        h->part_elems = part_elems_for(max_T, R, r_gate, r_down);
        alloc((void**)&h->part, h->part_elems * 4);
        alloc((void**)&h->Ug16, (size_t)ffn * r_gate * 2);
        alloc((void**)&h->Uu16, (size_t)ffn * r_up * 2);
        alloc((void**)&h->Vd16, (size_t)r_down * ffn * 2);
        alloc((void**)&h->Ud16, (size_t)d * r_down * 2);
    } else {
        h->tensor_ok = false;
    }
    if (!ok) { svdmlp_destroy(h); return SVDMLP_ERR_NOMEM; }
    bool cuda_ok = cudaMemsetAsync(h->status_dev, 0, sizeof(int), s) == cudaSuccess &&
                   cudaMemsetAsync(h->gridbar, 0, kGridbarBytes, s) == cudaSuccess &&
                   cudaMemsetAsync(h->tp_counter, 0, 256, s) == cudaSuccess;
    if (h->Zs) cuda_ok = cuda_ok && cudaMemsetAsync(h->Zs, 0, (size_t)h->t_skinny * R * 4, s) == cudaSuccess;
    if (h->Zds) cuda_ok = cuda_ok && cudaMemsetAsync(h->Zds, 0, (size_t)h->t_skinny * r_down * 4, s) == cudaSuccess;
    if (cuda_ok && h->tensor_ok) {
        cuda_ok = launch_convert(Ug, h->Ug16, (long)ffn * r_gate, h->status_dev, s) == SVDMLP_OK &&
                  launch_convert(Uu, h->Uu16, (long)ffn * r_up, h->status_dev, s) == SVDMLP_OK &&
                  launch_convert(Vd, h->Vd16, (long)r_down * ffn, h->status_dev, s) == SVDMLP_OK &&
                  launch_convert(Ud, h->Ud16, (long)d * r_down, h->status_dev, s) == SVDMLP_OK;
    }
    cuda_ok = cuda_ok && cudaStreamSynchronize(s) == cudaSuccess;
    if (!cuda_ok) { cudaGetLastError(); svdmlp_destroy(h); return SVDMLP_ERR_CUDA; }
    if (h->tensor_ok) {
        int over = 0;
        if (cudaMemcpy(&over, h->status_dev, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess ||
            cudaMemset(h->status_dev, 0, sizeof(int)) != cudaSuccess) {
            cudaGetLastError(); svdmlp_destroy(h); return SVDMLP_ERR_CUDA;
        }
        if (over != 0) {  // a factor value exceeds the fp16 range: only the bf16 weight-streaming path is usable
            if (flags & SVDMLP_FLAG_PATH_TENSOR) { svdmlp_destroy(h); return SVDMLP_ERR_UNSUPPORTED; }
            h->tensor_ok = false;
            if (h->t_skinny < max_T) { svdmlp_destroy(h); return SVDMLP_ERR_UNSUPPORTED; }
        }
    }
    if (h->t_skinny > 0 && r_gate == r_up && !(flags & SVDMLP_FLAG_DECODE_REGISTERS)) {
        // Persistent decode kernel: per-CTA blocks of the factors in streaming order (second-stage factors as
        // fp16), packed for a grid of one CTA per SM.  Any failure here just leaves the three-kernel path.
        h->persist_grid = num_sms();
        const dpersist::Shape sh = persist_shape(h, std::min(max_T, kSkinnyMaxT));
        bool pk = sh.G > 0 &&
                  cudaMalloc((void**)&h->pA, (size_t)sh.units_a() * sh.ksd() * 32 + 256) == cudaSuccess &&
                  cudaMalloc((void**)&h->pB, (size_t)sh.units_b() * 2 * sh.ksr() * dpersist::kPanel + 256) == cudaSuccess &&
                  cudaMalloc((void**)&h->pVdp, (size_t)sh.units_b() * sh.zt() * dpersist::kPanel + 256) == cudaSuccess &&
                  cudaMalloc((void**)&h->pUdp, (size_t)sh.units_d() * sh.zt() * dpersist::kPanel + 256) == cudaSuccess &&
                  cudaMalloc((void**)&h->Zp, persist_z_bytes(h)) == cudaSuccess &&
                  cudaMalloc((void**)&h->Zdp, persist_zd_bytes(h)) == cudaSuccess &&
                  persist_reset(h, s) == SVDMLP_OK;
        if (pk) {
            dpersist::pack_a_kernel<<<sh.G, 256, 0, s>>>(h->Vg, h->Vu, sh, h->pA);
            dpersist::pack_b_kernel<<<sh.G, 256, 0, s>>>(h->Ug, h->Uu, sh, h->pB, h->status_dev);
            dpersist::pack_vd_kernel<<<sh.G, 256, 0, s>>>(h->Vd, sh, h->pVdp, h->status_dev);
            dpersist::pack_ud_kernel<<<sh.G, 256, 0, s>>>(h->Ud, sh, h->pUdp, h->status_dev);
            int over = 0;
            pk = cudaGetLastError() == cudaSuccess && cudaStreamSynchronize(s) == cudaSuccess &&
                 cudaMemcpy(&over, h->status_dev, sizeof(int), cudaMemcpyDeviceToHost) == cudaSuccess &&
                 cudaMemset(h->status_dev, 0, sizeof(int)) == cudaSuccess && over == 0;
        }
        if (!pk) cudaGetLastError();
        h->persist_ok = pk;
    }
    if (h->tensor_ok) {
        int e = SVDMLP_OK;
        auto mk = [&](CUtensorMap* m, const void* base, long rows, long cols, long ld, int box_rows) {
            if (e == SVDMLP_OK) e = make_map(m, base, rows, cols, ld, box_rows);
        };
        mk(&h->mVg, Vg, r_gate, d, d, 128);
        mk(&h->mVu, Vu, r_up, d, d, 128);
        mk(&h->mUg, h->Ug16, ffn, r_gate, r_gate, 128);
        mk(&h->mUu, h->Uu16, ffn, r_up, r_up, 128);
        mk(&h->mVd, h->Vd16, r_down, ffn, ffn, down1_tile_width(r_down));
        mk(&h->mUd, h->Ud16, d, r_down, r_down, 128);
        mk(&h->mZg, h->Z16, max_T, r_gate, R, 128);
        mk(&h->mZu, h->Z16 + r_gate, max_T, r_up, R, 128);
        mk(&h->mH, h->H16, max_T, ffn, ffn, 128);
        mk(&h->mHc, h->H16, max_T, ffn, ffn, 32);
        mk(&h->mUg64, h->Ug16, ffn, r_gate, r_gate, 64);
        mk(&h->mUu64, h->Uu16, ffn, r_up, r_up, 64);
        mk(&h->mUd64, h->Ud16, d, r_down, r_down, 64);
        mk(&h->mVg64, Vg, r_gate, d, d, 64);
        mk(&h->mVu64, Vu, r_up, d, d, 64);
        mk(&h->mVg128, Vg, r_gate, d, d, 128);
        mk(&h->mVu128, Vu, r_up, d, d, 128);
        mk(&h->mVdHalf, h->Vd16, r_down, ffn, ffn, down1_tile_width(r_down) / 2);
        mk(&h->mZd, h->Zd16, max_T, r_down, r_down, 128);
        if (e != SVDMLP_OK) { svdmlp_destroy(h); return e; }
    }
    *out = h;
    return SVDMLP_OK;
}

int svdmlp_forward(svdmlp_t* h, const void* X, int T, void* Y, void* stream) {
    if (h == nullptr || X == nullptr || Y == nullptr || T <= 0 || T > h->max_T) return SVDMLP_ERR_INVALID_ARG;
    if (!aligned16(X) || !aligned16(Y)) return SVDMLP_ERR_ALIGNMENT;
    return forward_impl(h, (const __nv_bfloat16*)X, T, Y, (h->flags & SVDMLP_FLAG_Y_FP32) ? 1 : 0, nullptr,
                        static_cast<cudaStream_t>(stream));
}

int svdmlp_forward_host(svdmlp_t* h, const void* X_host, int T, void* Y_host, void* stream) {
    if (h == nullptr || X_host == nullptr || Y_host == nullptr || T <= 0 || T > h->max_T) return SVDMLP_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t ysz = (h->flags & SVDMLP_FLAG_Y_FP32) ? 4 : 2;
    if (h->Xdev == nullptr) {
        if (cudaMalloc(&h->Xdev, (size_t)h->max_T * h->d * 2) != cudaSuccess ||
            cudaMalloc(&h->Ydev, (size_t)h->max_T * h->d * ysz) != cudaSuccess) {
            cudaGetLastError();
            return SVDMLP_ERR_NOMEM;
        }
    }
    // Repeated calls with the same host buffers and T (a serving loop) replay one instantiated graph of the
    // operations: one launch call instead of three, and the dependencies are resolved on the device.
    if (h->host_exec != nullptr && h->host_x == X_host && h->host_y == Y_host && h->host_T == T) {
        h->launches += h->host_launches;
        CUDA_TRY(cudaGraphLaunch(h->host_exec, s));
        CUDA_TRY(cudaStreamSynchronize(s));
        return SVDMLP_OK;
    }
    if (h->host_exec != nullptr) { cudaGraphExecDestroy(h->host_exec); h->host_exec = nullptr; }
    // Small T: if Y_host is page-locked and mapped, the last kernel stores Y straight into it (a few tens of KB
    // of posted writes) and the copy-out, with its dependency latency, disappears.
    void* y_direct = nullptr;
    if (use_skinny(h, T)) {
        cudaPointerAttributes at;
        if (cudaPointerGetAttributes(&at, Y_host) == cudaSuccess && at.type == cudaMemoryTypeHost && at.devicePointer != nullptr &&
            aligned16(at.devicePointer))
            y_direct = at.devicePointer;
        else
            cudaGetLastError();
    }
    auto enqueue = [&]() -> int {
        if (cudaMemcpyAsync(h->Xdev, X_host, (size_t)T * h->d * 2, cudaMemcpyHostToDevice, s) != cudaSuccess) return SVDMLP_ERR_CUDA;
        const int rc = forward_impl(h, (const __nv_bfloat16*)h->Xdev, T, y_direct != nullptr ? y_direct : h->Ydev, ysz == 4, nullptr, s);
        if (rc != SVDMLP_OK) return rc;
        if (y_direct == nullptr &&
            cudaMemcpyAsync(Y_host, h->Ydev, (size_t)T * h->d * ysz, cudaMemcpyDeviceToHost, s) != cudaSuccess)
            return SVDMLP_ERR_CUDA;
        return SVDMLP_OK;
    };
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    const bool can_capture = s != nullptr && cudaStreamIsCapturing(s, &cap) == cudaSuccess && cap == cudaStreamCaptureStatusNone &&
                             !h->prof;
    if (can_capture && cudaStreamBeginCapture(s, cudaStreamCaptureModeThreadLocal) == cudaSuccess) {
        const unsigned long long before = h->launches;
        const int rc = enqueue();
        h->host_launches = h->launches - before;
        cudaGraph_t graph = nullptr;
        const cudaError_t e = cudaStreamEndCapture(s, &graph);
        if (rc == SVDMLP_OK && e == cudaSuccess && graph != nullptr &&
            cudaGraphInstantiate(&h->host_exec, graph, 0) == cudaSuccess) {
            cudaGraphDestroy(graph);
            h->host_x = X_host; h->host_y = Y_host; h->host_T = T;
            CUDA_TRY(cudaGraphLaunch(h->host_exec, s));
            CUDA_TRY(cudaStreamSynchronize(s));
            return SVDMLP_OK;
        }
        if (graph != nullptr) cudaGraphDestroy(graph);
        h->host_exec = nullptr;
        cudaGetLastError();
        if (rc != SVDMLP_OK) return rc;
    }
    const int rc = enqueue();
    if (rc != SVDMLP_OK) return rc;
    CUDA_TRY(cudaStreamSynchronize(s));
    return SVDMLP_OK;
}

int svdmlp_forward_prenorm_residual(svdmlp_t* h, const float* h_in, float* h_out, int T, float eps, void* stream) {
    if (h == nullptr || h_in == nullptr || h_out == nullptr || T <= 0 || T > h->max_T || !(eps >= 0.f))
        return SVDMLP_ERR_INVALID_ARG;
    if (!aligned16(h_in) || !aligned16(h_out)) return SVDMLP_ERR_ALIGNMENT;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    h->prof_n = 0;
    if (T <= 8 && use_skinny(h, T) && h->stage_mask == ~0u) {  // small T: RMSNorm inside the persistent decode kernel
        const int rc = skinny_forward(h, nullptr, T, h_out, 1, h_in, s, h_in, eps);
        if (rc != SVDMLP_ERR_UNSUPPORTED) return rc;
    }
    if (h->Xn == nullptr) {  // first call that needs the normalised rows in global memory
        if (cudaMalloc((void**)&h->Xn, (size_t)h->max_T * h->d * 2) != cudaSuccess) { cudaGetLastError(); return SVDMLP_ERR_NOMEM; }
    }
    if (h->stage_mask & 16u) {
        ProfScope ps(h, "rmsnorm", s);
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(T); cfg.blockDim = dim3(256); cfg.dynamicSmemBytes = 0; cfg.stream = s;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr; cfg.numAttrs = 1;
        CUDA_TRY(cudaLaunchKernelEx(&cfg, skinny::rmsnorm_kernel, h_in, h->d, eps, h->Xn));
    }
    CUDA_TRY(cudaGetLastError());
    h->launches += 1;
    return forward_impl(h, h->Xn, T, h_out, 1, h_in, s, true);
}

// ---- tensor-parallel halves of the forward pass ------------------------------------------------------------
int svdmlp_forward_partial(svdmlp_t* h, const void* X, int T, float* Zd_out, void* stream) {
    if (h == nullptr || X == nullptr || Zd_out == nullptr || T <= 0 || T > h->max_T) return SVDMLP_ERR_INVALID_ARG;
    if (!aligned16(X) || !aligned16(Zd_out)) return SVDMLP_ERR_ALIGNMENT;
    if (h->stage_mask != ~0u) return SVDMLP_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const __nv_bfloat16* Xb = (const __nv_bfloat16*)X;
    h->prof_n = 0;
    if (use_skinny(h, T)) {
        // register-streaming kernels: the first two of the three, which leave Zd in the handle's fp32 accumulator
        if (T > h->t_skinny || h->Zs == nullptr) return SVDMLP_ERR_UNSUPPORTED;
        int nt = T <= 8 ? 1 : T <= 16 ? 2 : 4;
        while (nt > 1 && skinny_smem_need(h, nt) > 227 * 1024) nt >>= 1;
        if (skinny_smem_need(h, nt) > 227 * 1024) return SVDMLP_ERR_UNSUPPORTED;
        h->stage_mask = 1u | 2u;
        const int rc = nt == 1 ? skinny_forward_nt<1>(h, Xb, T, nullptr, 0, nullptr, s)
                     : nt == 2 ? skinny_forward_nt<2>(h, Xb, T, nullptr, 0, nullptr, s)
                               : skinny_forward_nt<4>(h, Xb, T, nullptr, 0, nullptr, s);
        h->stage_mask = ~0u;
        if (rc != SVDMLP_OK) return rc;
        CUDA_TRY(cudaMemcpyAsync(Zd_out, h->Zds, (size_t)T * h->rd * 4, cudaMemcpyDeviceToDevice, s));
        // the third kernel, which is not run, would have cleared the first product's accumulator
        CUDA_TRY(cudaMemsetAsync(h->Zs, 0, (size_t)h->t_skinny * (h->rg + h->ru) * 4, s));
        return SVDMLP_OK;
    }
    h->stage_mask = 1u | 2u | 4u;
    h->zd_out32 = Zd_out;
    const int rc = tensor_forward(h, Xb, T, nullptr, 0, nullptr, s);
    h->zd_out32 = nullptr;
    h->stage_mask = ~0u;
    return rc;
}

int svdmlp_forward_finish(svdmlp_t* h, const float* Zd, int T, void* Y, void* stream) {
    if (h == nullptr || Zd == nullptr || Y == nullptr || T <= 0 || T > h->max_T) return SVDMLP_ERR_INVALID_ARG;
    if (!aligned16(Zd) || !aligned16(Y)) return SVDMLP_ERR_ALIGNMENT;
    if (h->stage_mask != ~0u) return SVDMLP_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int y_fp32 = (h->flags & SVDMLP_FLAG_Y_FP32) ? 1 : 0;
    h->prof_n = 0;
    if (use_skinny(h, T)) {
        using namespace skinny;
        int nt = T <= 8 ? 1 : T <= 16 ? 2 : 4;
        while (nt > 1 && (size_t)nt * 8 * 2 * (h->rd + kPad) * 2 > 227 * 1024) nt >>= 1;
        const size_t smem = (size_t)nt * 8 * 2 * (h->rd + kPad) * 2;
        if (smem > 227 * 1024) return SVDMLP_ERR_UNSUPPORTED;
        const int chunks = (T + nt * 8 - 1) / (nt * 8);
        dim3 grid((h->d + 63) / 64, 1, chunks);
#define SVDMLP_FINISH(NT)                                                                                              \
        {                                                                                                              \
            if (smem > 48 * 1024)                                                                                      \
                CUDA_TRY(cudaFuncSetAttribute(expand_kernel<NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024)); \
            expand_kernel<NT><<<grid, 128, smem, s>>>(Zd, T, h->rd, h->Ud, h->d, Y, y_fp32, nullptr, nullptr, 0);    \
        }
        if (nt == 1) SVDMLP_FINISH(1) else if (nt == 2) SVDMLP_FINISH(2) else SVDMLP_FINISH(4)
#undef SVDMLP_FINISH
        CUDA_TRY(cudaGetLastError());
        h->launches += 1;
        return SVDMLP_OK;
    }
    if (!h->tensor_ok) return SVDMLP_ERR_UNSUPPORTED;
    {
        const long n = (long)T * h->rd;
        const int blocks = (int)std::min<long>((n / 4 + 255) / 256, 4 * num_sms());
        tensorpath::f32_to_f16_kernel<<<std::max(blocks, 1), 256, 0, s>>>(Zd, h->Zd16, n);
        CUDA_TRY(cudaGetLastError());
        h->launches += 1;
    }
    h->stage_mask = 8u;
    const int rc = tensor_forward(h, nullptr, T, Y, y_fp32, nullptr, s);
    h->stage_mask = ~0u;
    return rc;
}

// ---- tensor-parallel forward with the exchange done by the library's own kernels (tp_exchange.cuh) -----------
size_t svdmlp_tp_recv_bytes(int G, int max_T, int r_down) {
    if (G <= 0 || G > tpx::kMaxRanks || max_T <= 0 || r_down <= 0) return 0;
    return (size_t)2 * G * max_T * r_down * sizeof(float);
}

int svdmlp_forward_partial_push(svdmlp_t* h, const void* X, int T, const svdmlp_tp_peers_t* peers, unsigned long long step,
                                void* stream) {
    if (h == nullptr || peers == nullptr || step == 0) return SVDMLP_ERR_INVALID_ARG;
    const int G = peers->world, rank = peers->rank;
    if (G <= 0 || G > tpx::kMaxRanks || rank < 0 || rank >= G) return SVDMLP_ERR_INVALID_ARG;
    tpx::Peers pp;
    for (int p = 0; p < G; ++p) {
        if (peers->recv[p] == nullptr || peers->flags[p] == nullptr) return SVDMLP_ERR_INVALID_ARG;
        if (!aligned16(peers->recv[p]) || (reinterpret_cast<uintptr_t>(peers->flags[p]) & 7)) return SVDMLP_ERR_ALIGNMENT;
        pp.recv[p] = peers->recv[p]; pp.flags[p] = peers->flags[p];
    }
    const long slot = (long)h->max_T * h->rd, slot_off = ((long)(step & 1ull) * G + rank) * slot;
    // this rank's partial goes straight into its own slot of its own receive buffer ...
    const int rc = svdmlp_forward_partial(h, X, T, peers->recv[rank] + slot_off, stream);
    if (rc != SVDMLP_OK) return rc;
    // ... and from there to the same slot of every peer; the flags follow the data
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const long n = (long)T * h->rd;
    const int blocks = (int)std::max<long>(1, std::min<long>((n / 4 + 255) / 256, 2L * num_sms()));
    tpx::push_kernel<<<blocks, 256, 0, s>>>(peers->recv[rank] + slot_off, n, pp, G, rank, slot_off, step, h->tp_counter);
    CUDA_TRY(cudaGetLastError());
    h->launches += 1;
    return SVDMLP_OK;
}

int svdmlp_forward_finish_gather(svdmlp_t* h, float* recv, const unsigned long long* flags, int G, unsigned long long step,
                                 int T, void* Y, void* stream) {
    if (h == nullptr || recv == nullptr || flags == nullptr || Y == nullptr || step == 0 || G <= 0 || G > tpx::kMaxRanks ||
        T <= 0 || T > h->max_T)
        return SVDMLP_ERR_INVALID_ARG;
    if (!aligned16(recv) || (reinterpret_cast<uintptr_t>(flags) & 7)) return SVDMLP_ERR_ALIGNMENT;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const long slot = (long)h->max_T * h->rd, n = (long)T * h->rd;
    float* base = recv + (long)(step & 1ull) * G * slot;
    const int blocks = (int)std::max<long>(1, std::min<long>((n / 4 + 255) / 256, 2L * num_sms()));
    // the sum replaces slot 0 of this step's buffer (each element is read, then written, by one thread)
    tpx::gather_sum_kernel<<<blocks, 256, 0, s>>>(base, flags, G, step, n, slot, base, h->status_dev, h->tp_limit_ns);
    CUDA_TRY(cudaGetLastError());
    h->launches += 1;
    return svdmlp_forward_finish(h, base, T, Y, stream);
}

int svdmlp_tp_wait_limit_ns(svdmlp_t* h, unsigned long long limit_ns) {
    if (h == nullptr || limit_ns == 0) return SVDMLP_ERR_INVALID_ARG;
    h->tp_limit_ns = limit_ns;
    return SVDMLP_OK;
}

int svdmlp_destroy(svdmlp_t* h) {
    if (h == nullptr) return SVDMLP_OK;
    cudaDeviceSynchronize();
    cudaGetLastError();
    void* bufs[] = {h->Zs, h->Zds, h->Z16, h->H16, h->Zd16, h->part, h->Ug16, h->Uu16, h->Vd16, h->Ud16,
                    h->Xn, h->Xdev, h->Ydev, h->status_dev, h->gridbar, h->tp_counter,
                    h->pA, h->pB, h->pVdp, h->pUdp, h->Zp, h->Zdp};
    for (void* b : bufs)
        if (b != nullptr) cudaFree(b);
    for (cudaEvent_t e : h->prof_ev)
        if (e != nullptr) cudaEventDestroy(e);
    if (h->host_exec != nullptr) cudaGraphExecDestroy(h->host_exec);
    delete h;
    return SVDMLP_OK;
}

int svdmlp_last_device_status(svdmlp_t* h) {
    if (h == nullptr) return SVDMLP_ERR_INVALID_ARG;
    int v = 0;
    if (cudaDeviceSynchronize() != cudaSuccess) { cudaGetLastError(); return SVDMLP_ERR_CUDA; }
    CUDA_TRY(cudaMemcpy(&v, h->status_dev, sizeof(int), cudaMemcpyDeviceToHost));
    if (v != 0) {  // a wait gave up: barrier words and accumulators may be inconsistent, start clean
        CUDA_TRY(cudaMemset(h->status_dev, 0, sizeof(int)));
        { int rr = persist_reset(h, nullptr); if (rr != SVDMLP_OK) return rr; }
        CUDA_TRY(cudaDeviceSynchronize());
        if (h->Zs) CUDA_TRY(cudaMemset(h->Zs, 0, (size_t)h->t_skinny * (h->rg + h->ru) * 4));
        if (h->Zds) CUDA_TRY(cudaMemset(h->Zds, 0, (size_t)h->t_skinny * h->rd * 4));
    }
    return v;
}

int svdmlp_selftest_timeout(svdmlp_t* h, unsigned limit_us, void* stream) {
    if (h == nullptr || limit_us == 0 || limit_us > 1000000u) return SVDMLP_ERR_INVALID_ARG;
    wait_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(h->status_dev, (unsigned long long)limit_us * 1000ull);
    CUDA_TRY(cudaGetLastError());
    return SVDMLP_OK;
}

int svdmlp_stage_mask(svdmlp_t* h, unsigned mask) {
    if (h == nullptr) return SVDMLP_ERR_INVALID_ARG;
    const bool restore = mask == ~0u && h->stage_mask != ~0u;
    h->stage_mask = mask;
    if (restore) {
        // a partial mask breaks the chain in which neighbouring kernels clear each other's accumulators:
        // put the workspace back into the state a full forward expects
        CUDA_TRY(cudaDeviceSynchronize());
        if (h->Zs) CUDA_TRY(cudaMemset(h->Zs, 0, (size_t)h->t_skinny * (h->rg + h->ru) * 4));
        if (h->Zds) CUDA_TRY(cudaMemset(h->Zds, 0, (size_t)h->t_skinny * h->rd * 4));
        const int rr = persist_reset(h, nullptr);
        if (rr != SVDMLP_OK) return rr;
        CUDA_TRY(cudaDeviceSynchronize());
    }
    return SVDMLP_OK;
}

int svdmlp_profile_enable(svdmlp_t* h, int enable) {
    if (h == nullptr) return SVDMLP_ERR_INVALID_ARG;
    if (enable && h->prof_ev[0] == nullptr)
        for (cudaEvent_t& e : h->prof_ev) CUDA_TRY(cudaEventCreate(&e));
    h->prof = enable != 0;
    h->prof_n = 0;
    return SVDMLP_OK;
}

int svdmlp_profile_read(svdmlp_t* h, float* ms, int capacity) {
    if (h == nullptr || ms == nullptr || capacity < 0) return SVDMLP_ERR_INVALID_ARG;
    for (int i = 0; i < h->prof_n; ++i) {
        CUDA_TRY(cudaEventSynchronize(h->prof_ev[2 * i + 1]));
        float t = 0.f;
        CUDA_TRY(cudaEventElapsedTime(&t, h->prof_ev[2 * i], h->prof_ev[2 * i + 1]));
        if (i < capacity) ms[i] = t;
    }
    return h->prof_n;
}

const char* svdmlp_profile_name(const svdmlp_t* h, int index) {
    if (h == nullptr || index < 0 || index >= h->prof_n) return nullptr;
    return h->prof_name[index];
}

unsigned long long svdmlp_launch_count(const svdmlp_t* h) { return h ? h->launches : 0ull; }

const char* svdmlp_path_name(const svdmlp_t* h, int T) {
    if (h == nullptr) return "none";
    if (use_skinny(h, T)) return "skinny";
    return fused_plan(h, T) > 0 ? "tensor-fused" : "tensor";
}

}  // extern "C"

// ---- XUV operator without allocation ---------------------------------------------------------------
// Scratch for svdlinear_forward_noalloc: the fp32 accumulator Z[T, r].  In host code this name is
// only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) float g_noalloc_scratch[SVDLINEAR_NOALLOC_MAX_ELEMS];

namespace {
constexpr int kMaxDevices = 64;
float* g_noalloc_ptr[kMaxDevices];  // device address of g_noalloc_scratch, per device (nullptr = not looked up yet)

// Device address of the scratch array on the current device; looked up once per device.
int noalloc_scratch(float** out) {
    int dev = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return SVDMLP_ERR_UNSUPPORTED;
    float* p = __atomic_load_n(&g_noalloc_ptr[dev], __ATOMIC_ACQUIRE);
    if (p == nullptr) {
        void* sym = nullptr;
        CUDA_TRY(cudaGetSymbolAddress(&sym, g_noalloc_scratch));
        if (sym == nullptr) return SVDMLP_ERR_CUDA;
        p = static_cast<float*>(sym);
        __atomic_store_n(&g_noalloc_ptr[dev], p, __ATOMIC_RELEASE);  // same value from any thread
    }
    *out = p;
    return SVDMLP_OK;
}
}  // namespace

extern "C" int svdlinear_forward_noalloc(const void* X, int T, int in, int out, int r, const void* U, const void* V,
                                         void* Y, void* stream) {
    if (!X || !U || !V || !Y || T <= 0 || in <= 0 || out <= 0 || r <= 0) return SVDMLP_ERR_INVALID_ARG;
    if ((in | out | r) & 7) return SVDMLP_ERR_ALIGNMENT;
    if (!aligned16(X) || !aligned16(U) || !aligned16(V) || !aligned16(Y)) return SVDMLP_ERR_ALIGNMENT;
    if (T > SVDLINEAR_NOALLOC_MAX_T || (long)T * r > SVDLINEAR_NOALLOC_MAX_ELEMS || r > SVDLINEAR_NOALLOC_MAX_R)
        return SVDMLP_ERR_UNSUPPORTED;
    using namespace skinny;
    // the second kernel keeps a [8 nt, r] strip of Z (as a hi + lo bf16 pair) in shared memory: settle the token
    // tile and check that it fits before anything is enqueued
    int nt = T <= 8 ? 1 : T <= 16 ? 2 : 4;
    while (nt > 1 && (size_t)nt * 8 * 2 * (r + kPad) * 2 > 227 * 1024) nt >>= 1;
    if ((size_t)nt * 8 * 2 * (r + kPad) * 2 > 227 * 1024) return SVDMLP_ERR_UNSUPPORTED;
    int rc = check_arch();
    if (rc != SVDMLP_OK) return rc;
    float* z = nullptr;
    if ((rc = noalloc_scratch(&z)) != SVDMLP_OK) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int kc = 256;
    const int chunks = (T + nt * 8 - 1) / (nt * 8);
    dim3 g1(((r + 15) / 16 + 3) / 4, (in + kc - 1) / kc, chunks), g2((out + 63) / 64, 1, chunks);
    const size_t sm1 = (size_t)nt * 8 * (kc + kPad) * 2, sm2 = (size_t)nt * 8 * 2 * (r + kPad) * 2;
    // the accumulator keeps whatever the previous call left: clear the part this call sums into
    CUDA_TRY(cudaMemsetAsync(z, 0, (size_t)T * r * sizeof(float), s));
    const __nv_bfloat16 *Xb = (const __nv_bfloat16*)X, *Ub = (const __nv_bfloat16*)U, *Vb = (const __nv_bfloat16*)V;
#define SVDLIN_NOALLOC(NT)                                                                                       \
    {                                                                                                            \
        if (sm2 > 48 * 1024)                                                                                     \
            CUDA_TRY(cudaFuncSetAttribute(expand_kernel<NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024)); \
        stage1_kernel<NT><<<g1, 128, sm1, s>>>(Xb, in, T, in, Vb, r, nullptr, 0, z, kc, nullptr, 0);             \
        expand_kernel<NT><<<g2, 128, sm2, s>>>(z, T, r, Ub, out, Y, 0, nullptr, nullptr, 0);                     \
    }
    if (nt == 1) SVDLIN_NOALLOC(1) else if (nt == 2) SVDLIN_NOALLOC(2) else SVDLIN_NOALLOC(4)
#undef SVDLIN_NOALLOC
    CUDA_TRY(cudaGetLastError());
    return SVDMLP_OK;
}

struct svdlinear {
    int in, out, r, max_T;
    const void *U, *V;
    void* ws; size_t ws_bytes;
    float* f32; __half *z16, *u16;
    bool u16_ok;
    CUtensorMap mV, mU, mZ, mZc;
    const void* x_ptr; int x_T; unsigned x_layout; CUtensorMap mX;
    const void* y_ptr; int y_T; unsigned y_layout; CUtensorMap mYc;
    uint16_t *xt, *yt;   // [32, in] and [32, out] scratch: transposed layouts at T <= 32
};

namespace {
// The two products of the XUV operator on the tcgen05 kernels.  Both stream their operands; with at least two
// token tiles they run on CTA pairs (cta_group::2, 256 x 256 tiles, each CTA loading half of the B tile) and
// leave through TMA stores.  Z[T, r] passes through global memory in fp16 (L2-resident at these sizes).
int lin_tensor_run(const CUtensorMap& mX, const CUtensorMap& mV, const CUtensorMap& mU, const CUtensorMap& mZ,
                   const CUtensorMap& mZc, const CUtensorMap& mYc, float* f32, __half* z16, void* Y, int T, int in,
                   int out, int r, cudaStream_t s, unsigned layout = 0) {
    using namespace tensorpath;
    int rc;
    const bool pr = T > BM;
    const int bn = pr ? 256 : 128;
    GemmPlan g;
    plan_gemm(g, 1, bn, false, true, T, r, in, 1, true, pr);
    g.p.tmA[0] = mX; g.p.tmA[1] = mX; g.p.tmB[0] = mV; g.p.tmB[1] = mV; g.p.tmC = mZc;
    g.p.a_fmt = umma::kFmtBF16; g.p.b_fmt = umma::kFmtBF16; g.p.status = nullptr;
    g.p.a_mn = (layout & SVDLINEAR_X_TRANSPOSED) ? 1 : 0;   // mX then maps X^T[in, T]: the tile is an MN-major operand
    if (g.p.ksplit > 1) {
        g.p.c_tma = 0;  // fp32 partials are stored directly
        g.p.C = f32; g.p.ldc = r; g.p.split_stride = (long)T * r; g.p.out_mode = OUT_F32;
        if ((rc = launch_gemm(g, s)) != SVDMLP_OK) return rc;
        if ((rc = launch_reduce(f32, g.p.ksplit, (long)T * r, (long)T * r, z16, s)) != SVDMLP_OK) return rc;
    } else {
        g.p.C = z16; g.p.ldc = r; g.p.out_mode = OUT_F16;
        if ((rc = launch_gemm(g, s)) != SVDMLP_OK) return rc;
    }
    plan_gemm(g, 1, bn, false, false, T, out, r, 1, true, pr);
    g.p.tmA[0] = mZ; g.p.tmA[1] = mZ; g.p.tmB[0] = mU; g.p.tmB[1] = mU; g.p.tmC = mYc;
    g.p.a_fmt = umma::kFmtF16; g.p.b_fmt = umma::kFmtF16; g.p.status = nullptr;
    g.p.C = Y; g.p.ldc = out; g.p.out_mode = OUT_BF16;
    g.p.c_t = (layout & SVDLINEAR_Y_TRANSPOSED) ? 1 : 0;    // mYc then maps Y^T[out, T]
    return launch_gemm(g, s);
}
}  // namespace

extern "C" {

// ---- XUV operator --------------------------------------------------------------------------------
// Workspace layout: [ fp32 region: max(T*r skinny accumulator, ksplit partials) | fp16 Z[T, r] ]
static size_t lin_f32_elems(int T, int r) { return (size_t)16 * T * r; }

size_t svdlinear_workspace_bytes(int T, int in, int out, int r) {
    if (T <= 0 || in <= 0 || out <= 0 || r <= 0) return 0;
    size_t f32 = (lin_f32_elems(T, r) * 4 + 255) & ~(size_t)255;
    size_t f16 = ((size_t)T * r * 2 + 255) & ~(size_t)255;
    size_t u16 = ((size_t)out * r * 2 + 255) & ~(size_t)255;  // fp16 re-encoding of U for the tcgen05 path
    return f32 + f16 + u16 + 256;
}

int svdlinear_forward(const void* X, int T, int in, int out, int r, const void* U, const void* V, void* Y,
                      void* workspace, size_t workspace_bytes, void* stream) {
    if (!X || !U || !V || !Y || !workspace || T <= 0 || in <= 0 || out <= 0 || r <= 0) return SVDMLP_ERR_INVALID_ARG;
    if ((in | out | r) & 7) return SVDMLP_ERR_ALIGNMENT;
    if (!aligned16(X) || !aligned16(U) || !aligned16(V) || !aligned16(Y) || (reinterpret_cast<uintptr_t>(workspace) & 255))
        return SVDMLP_ERR_ALIGNMENT;
    if (workspace_bytes < svdlinear_workspace_bytes(T, in, out, r)) return SVDMLP_ERR_NOMEM;
    int rc = check_arch();
    if (rc != SVDMLP_OK) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    float* f32 = reinterpret_cast<float*>(workspace);
    __half* z16 = reinterpret_cast<__half*>(reinterpret_cast<char*>(workspace) + ((lin_f32_elems(T, r) * 4 + 255) & ~(size_t)255));
    const __nv_bfloat16* Xb = (const __nv_bfloat16*)X;
    if (T <= kSkinnyMaxT) {
        using namespace skinny;
        const int nt_want = T <= 8 ? 1 : T <= 16 ? 2 : 4;
        int nt = nt_want;
        while (nt > 1 && (size_t)nt * 8 * 2 * (r + kPad) * 2 > 227 * 1024) nt >>= 1;
        if ((size_t)nt * 8 * 2 * (r + kPad) * 2 > 227 * 1024) return SVDMLP_ERR_UNSUPPORTED;
        CUDA_TRY(cudaMemsetAsync(f32, 0, (size_t)T * r * 4, s));
        const int kc = 256;
        const int chunks = (T + nt * 8 - 1) / (nt * 8);
        dim3 g1(((r + 15) / 16 + 3) / 4, (in + kc - 1) / kc, chunks), g2((out + 63) / 64, 1, chunks);
        size_t sm1 = (size_t)nt * 8 * (kc + kPad) * 2, sm2 = (size_t)nt * 8 * 2 * (r + kPad) * 2;
#define SVDLIN_SKINNY(NT)                                                                                      \
        {                                                                                                      \
            if (sm2 > 48 * 1024)                                                                               \
                CUDA_TRY(cudaFuncSetAttribute(expand_kernel<NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024)); \
            stage1_kernel<NT><<<g1, 128, sm1, s>>>(Xb, in, T, in, (const __nv_bfloat16*)V, r, nullptr, 0, f32, kc, nullptr, 0); \
            expand_kernel<NT><<<g2, 128, sm2, s>>>(f32, T, r, (const __nv_bfloat16*)U, out, Y, 0, nullptr, nullptr, 0); \
        }
        if (nt == 1) SVDLIN_SKINNY(1) else if (nt == 2) SVDLIN_SKINNY(2) else SVDLIN_SKINNY(4)
#undef SVDLIN_SKINNY
        CUDA_TRY(cudaGetLastError());
        return SVDMLP_OK;
    }
    using namespace tensorpath;
    CUtensorMap mX, mV, mU, mZ;
    if ((rc = make_map(&mX, X, T, in, in, BM)) != SVDMLP_OK) return rc;
    if ((rc = make_map(&mV, V, r, in, in, 128)) != SVDMLP_OK) return rc;
    __half* u16 = z16 + (((size_t)T * r * 2 + 255) & ~(size_t)255) / 2;
    int* flag = reinterpret_cast<int*>(u16 + (((size_t)out * r * 2 + 255) & ~(size_t)255) / 2);
    CUDA_TRY(cudaMemsetAsync(flag, 0, sizeof(int), s));
    if ((rc = launch_convert(U, u16, (long)out * r, flag, s)) != SVDMLP_OK) return rc;
    if ((rc = make_map(&mU, u16, out, r, r, 128)) != SVDMLP_OK) return rc;
    if ((rc = make_map(&mZ, z16, T, r, r, 128)) != SVDMLP_OK) return rc;
    CUtensorMap mZc, mYc;
    if ((rc = make_map(&mZc, z16, T, r, r, 32)) != SVDMLP_OK) return rc;
    if ((rc = make_map(&mYc, Y, T, out, out, 32)) != SVDMLP_OK) return rc;
    return lin_tensor_run(mX, mV, mU, mZ, mZc, mYc, f32, z16, Y, T, in, out, r, s);
}

// ---- XUV operator with a handle: everything that does not depend on the call is done once ---------------
int svdlinear_create(svdlinear_t** out_h, int in, int out, int r, const void* U, const void* V, int max_T, void* stream) {
    if (out_h == nullptr) return SVDMLP_ERR_INVALID_ARG;
    *out_h = nullptr;
    if (!U || !V || in <= 0 || out <= 0 || r <= 0 || max_T <= 0) return SVDMLP_ERR_INVALID_ARG;
    if ((in | out | r) & 7) return SVDMLP_ERR_ALIGNMENT;
    if (!aligned16(U) || !aligned16(V)) return SVDMLP_ERR_ALIGNMENT;
    int rc = check_arch();
    if (rc != SVDMLP_OK) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    svdlinear* h = new (std::nothrow) svdlinear();
    if (h == nullptr) return SVDMLP_ERR_NOMEM;
    memset(h, 0, sizeof(*h));
    h->in = in; h->out = out; h->r = r; h->max_T = max_T; h->U = U; h->V = V;
    h->ws_bytes = svdlinear_workspace_bytes(max_T, in, out, r);
    if (cudaMalloc(&h->ws, h->ws_bytes) != cudaSuccess) { cudaGetLastError(); delete h; return SVDMLP_ERR_NOMEM; }
    if (cudaMalloc((void**)&h->xt, (size_t)kSkinnyMaxT * (in + out) * 2) != cudaSuccess) { cudaGetLastError(); svdlinear_destroy(h); return SVDMLP_ERR_NOMEM; }
    h->yt = h->xt + (size_t)kSkinnyMaxT * in;
    h->f32 = reinterpret_cast<float*>(h->ws);
    h->z16 = reinterpret_cast<__half*>(reinterpret_cast<char*>(h->ws) + ((lin_f32_elems(max_T, r) * 4 + 255) & ~(size_t)255));
    h->u16 = h->z16 + (((size_t)max_T * r * 2 + 255) & ~(size_t)255) / 2;
    int* flag = reinterpret_cast<int*>(h->u16 + (((size_t)out * r * 2 + 255) & ~(size_t)255) / 2);
    int over = 0;
    bool ok = cudaMemsetAsync(flag, 0, sizeof(int), s) == cudaSuccess &&
              launch_convert(U, h->u16, (long)out * r, flag, s) == SVDMLP_OK &&
              cudaMemcpyAsync(&over, flag, sizeof(int), cudaMemcpyDeviceToHost, s) == cudaSuccess &&
              cudaStreamSynchronize(s) == cudaSuccess;
    if (!ok) { cudaGetLastError(); svdlinear_destroy(h); return SVDMLP_ERR_CUDA; }
    h->u16_ok = over == 0;   // a value of U beyond the fp16 range: only the small-T (bf16) kernels can be used
    if (h->u16_ok && max_T > kSkinnyMaxT) {
        rc = make_map(&h->mV, V, r, in, in, 128);
        if (rc == SVDMLP_OK) rc = make_map(&h->mU, h->u16, out, r, r, 128);
        if (rc == SVDMLP_OK) rc = make_map(&h->mZ, h->z16, max_T, r, r, 128);
        if (rc == SVDMLP_OK) rc = make_map(&h->mZc, h->z16, max_T, r, r, 32);
        if (rc != SVDMLP_OK) { svdlinear_destroy(h); return rc; }
    }
    *out_h = h;
    return SVDMLP_OK;
}

int svdlinear_apply(svdlinear_t* h, const void* X, int T, void* Y, void* stream) {
    return svdlinear_apply_layout(h, X, T, Y, 0u, stream);
}

int svdlinear_apply_layout(svdlinear_t* h, const void* X, int T, void* Y, unsigned layout, void* stream) {
    if (h == nullptr || X == nullptr || Y == nullptr || T <= 0 || T > h->max_T) return SVDMLP_ERR_INVALID_ARG;
    if (layout & ~(SVDLINEAR_X_TRANSPOSED | SVDLINEAR_Y_TRANSPOSED)) return SVDMLP_ERR_INVALID_ARG;
    if (!aligned16(X) || !aligned16(Y)) return SVDMLP_ERR_ALIGNMENT;
    if (layout != 0 && (T & 7)) return SVDMLP_ERR_ALIGNMENT;   // rows of X^T / Y^T are T elements: 16-byte pitch
    const bool xt = layout & SVDLINEAR_X_TRANSPOSED, yt = layout & SVDLINEAR_Y_TRANSPOSED;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (T <= kSkinnyMaxT) {
        // weight-streaming kernels read the bf16 factors as they are; they take row-major X and Y, so a
        // transposed operand (at most 32 rows) passes through a scratch copy
        const void* Xr = X;
        void* Yr = Y;
        if (xt) {
            tensorpath::transpose16_kernel<<<dim3((T + 31) / 32, (h->in + 31) / 32), 256, 0, s>>>((const uint16_t*)X, h->in, T, h->xt);
            Xr = h->xt;
        }
        if (yt) Yr = h->yt;
        int rc = svdlinear_forward(Xr, T, h->in, h->out, h->r, h->U, h->V, Yr, h->ws, h->ws_bytes, stream);
        if (rc != SVDMLP_OK) return rc;
        if (yt) tensorpath::transpose16_kernel<<<dim3((h->out + 31) / 32, (T + 31) / 32), 256, 0, s>>>(h->yt, T, h->out, (uint16_t*)Y);
        CUDA_TRY(cudaGetLastError());
        return SVDMLP_OK;
    }
    if (!h->u16_ok) return SVDMLP_ERR_UNSUPPORTED;
    int rc;
    if (h->x_ptr != X || h->x_T != T || h->x_layout != (layout & SVDLINEAR_X_TRANSPOSED)) {
        // X^T[in, T]: boxes of [64 k][64 tokens]; X[T, in]: boxes of [128 tokens][64 k]
        rc = xt ? make_map(&h->mX, X, h->in, T, T, 64) : make_map(&h->mX, X, T, h->in, h->in, tensorpath::BM);
        if (rc != SVDMLP_OK) return rc;
        h->x_ptr = X; h->x_T = T; h->x_layout = layout & SVDLINEAR_X_TRANSPOSED;
    }
    if (h->y_ptr != Y || h->y_T != T || h->y_layout != (layout & SVDLINEAR_Y_TRANSPOSED)) {
        rc = yt ? make_map_t(&h->mYc, Y, h->out, T, T) : make_map(&h->mYc, Y, T, h->out, h->out, 32);
        if (rc != SVDMLP_OK) return rc;
        h->y_ptr = Y; h->y_T = T; h->y_layout = layout & SVDLINEAR_Y_TRANSPOSED;
    }
    return lin_tensor_run(h->mX, h->mV, h->mU, h->mZ, h->mZc, h->mYc, h->f32, h->z16, Y, T, h->in, h->out, h->r, s, layout);
}

int svdlinear_destroy(svdlinear_t* h) {
    if (h == nullptr) return SVDMLP_OK;
    cudaDeviceSynchronize();
    cudaGetLastError();
    if (h->ws != nullptr) cudaFree(h->ws);
    if (h->xt != nullptr) cudaFree(h->xt);
    delete h;
    return SVDMLP_OK;
}

}  // extern "C"

// ---- compression front-end ---------------------------------------------------------------------------
extern "C" size_t svdmlp_compress_workspace_bytes(int out, int in) {
    if (out <= 0 || in <= 0) return 0;
    const size_t n = (size_t)std::min(out, in), m = (size_t)std::max(out, in);
    return ((n * m + n * n + n) * sizeof(float) + n * sizeof(int) + 256 + 255) & ~(size_t)255;
}

extern "C" int svdmlp_compress(const float* W, int out, int in, int r, void* U_out, void* V_out, float* sigma_out,
                               void* workspace, size_t workspace_bytes, unsigned flags, void* stream) {
    if (!W || !U_out || !V_out || !workspace || out <= 0 || in <= 0 || r <= 0 || r > std::min(out, in)) return SVDMLP_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(workspace) & 255) return SVDMLP_ERR_ALIGNMENT;
    if (workspace_bytes < svdmlp_compress_workspace_bytes(out, in)) return SVDMLP_ERR_NOMEM;
    int rc = check_arch();
    if (rc != SVDMLP_OK) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int transpose = in <= out ? 1 : 0;           // the vectors made orthogonal: columns of W, or its rows
    const int n = std::min(out, in), m = std::max(out, in), n_even = (n + 1) & ~1;
    float* B = reinterpret_cast<float*>(workspace);
    float* R = B + (size_t)n * m;
    float* sigma = R + (size_t)n * n;
    int* order = reinterpret_cast<int*>(sigma + n);
    int* rotated = order + n;
    const int blocks = std::min(8 * num_sms(), (int)std::min<size_t>(((size_t)n * m + 255) / 256, 1u << 20));
    compress::init_kernel<<<std::max(blocks, 1), compress::kThreads, 0, s>>>(W, out, in, transpose, n, m, B, R);
    CUDA_TRY(cudaGetLastError());
    const int max_sweeps = 40;
    const double tol = 1e-7;   // fp32 storage: pairs whose cosine is below this count as orthogonal
    if (n > 1) {
        for (int sweep = 0; sweep < max_sweeps; ++sweep) {
            CUDA_TRY(cudaMemsetAsync(rotated, 0, sizeof(int), s));
            for (int k = 0; k < n_even - 1; ++k)
                compress::step_kernel<<<n_even / 2, compress::kThreads, 0, s>>>(B, R, n, m, n_even, k, tol, rotated);
            CUDA_TRY(cudaGetLastError());
            int h_rot = 0;
            CUDA_TRY(cudaMemcpyAsync(&h_rot, rotated, sizeof(int), cudaMemcpyDeviceToHost, s));
            CUDA_TRY(cudaStreamSynchronize(s));
            if (h_rot == 0) break;
        }
    }
    compress::norms_kernel<<<n, compress::kThreads, 0, s>>>(B, n, m, sigma);
    CUDA_TRY(cudaGetLastError());
    std::vector<float> hs(n);
    CUDA_TRY(cudaMemcpyAsync(hs.data(), sigma, (size_t)n * sizeof(float), cudaMemcpyDeviceToHost, s));
    CUDA_TRY(cudaStreamSynchronize(s));
    std::vector<int> ho(n);
    std::iota(ho.begin(), ho.end(), 0);
    std::stable_sort(ho.begin(), ho.end(), [&](int a, int b) { return hs[a] > hs[b]; });
    CUDA_TRY(cudaMemcpyAsync(order, ho.data(), (size_t)n * sizeof(int), cudaMemcpyHostToDevice, s));
    if (sigma_out != nullptr)
        for (int k = 0; k < n; ++k) sigma_out[k] = hs[ho[k]];   // HOST array, descending
    const long total = (long)out * r + (long)r * in;
    const int eb = (int)std::min<long>((total + 255) / 256, 8L * num_sms());
    compress::emit_kernel<<<std::max(eb, 1), compress::kThreads, 0, s>>>(B, R, sigma, order, out, in, r, transpose, n, m,
                                                                        (flags & SVDMLP_COMPRESS_SPLIT_SQRT) ? 1 : 0,
                                                                        (__nv_bfloat16*)U_out, (__nv_bfloat16*)V_out);
    CUDA_TRY(cudaGetLastError());
    CUDA_TRY(cudaStreamSynchronize(s));   // `ho` is read by the copy above
    return SVDMLP_OK;
}
