// Exchange step of the tensor-parallel forward (Section 4.2.2, Figure 4: the one all-reduce of the partitioned MLP;
// with factored weights it falls on the narrow fp32 Zd[T, r_down]).  No collective library: every rank PUSHES its
// partial into its slot of every peer's receive buffer with plain peer stores and then raises a flag per peer;
// the consumer waits (bounded) for the G flags of the step and sums the G slots.  The only accesses to a
// peer's memory are ordinary st.global / ld.global on peer-mapped device memory.
//
// Receive buffer of a rank: float [2][G][slot] (slot = max_T * r_down), the first index = step parity.  Two
// buffers are enough: a peer pushes step e + 2 only after it has gathered step e + 1, which needed this rank's push
// of e + 1, which this rank enqueues after its own gather of step e.  Flags: one 64-bit word per source rank,
// holding the number of the last step whose data has landed (zero at start; steps count from 1).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace tpx {

constexpr int kMaxRanks = 8;
struct Peers {
    float* recv[kMaxRanks];
    unsigned long long* flags[kMaxRanks];
};

__device__ __forceinline__ unsigned long long ld_acquire_sys(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.acquire.sys.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_sys(unsigned long long* p, unsigned long long v) {
    asm volatile("st.release.sys.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ unsigned long long now_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

// src[n] (this rank's partial, already in its own slot) -> slot `rank` of every other peer; then the flags.
// n is a multiple of 4.  *counter is zero on entry and on exit.
__global__ void __launch_bounds__(256)
push_kernel(const float* __restrict__ src, long n, Peers peers, int G, int rank, long slot_off, unsigned long long step,
            unsigned int* counter) {
    for (long i = ((long)blockIdx.x * blockDim.x + threadIdx.x) * 4; i < n; i += (long)gridDim.x * blockDim.x * 4) {
        const float4 v = *reinterpret_cast<const float4*>(src + i);
        for (int p = 0; p < G; ++p)
            if (p != rank) *reinterpret_cast<float4*>(peers.recv[p] + slot_off + i) = v;
    }
    __threadfence_system();   // this thread's peer stores are visible system-wide before the count below
    __syncthreads();
    if (threadIdx.x == 0) {
        const unsigned int prev = atomicAdd(counter, 1u);
        if (prev == gridDim.x - 1) {   // every block has stored and fenced
            *counter = 0;
            __threadfence_system();
            for (int p = 0; p < G; ++p) st_release_sys(peers.flags[p] + rank, step);
        }
    }
}

// out[i] = sum over g of recv[g][i] once flags[g] >= step for every g.  A wait that outlasts limit_ns writes
// kErrTimeout (-7) to *status and the kernel returns without touching out.
__global__ void __launch_bounds__(256)
gather_sum_kernel(const float* recv, const unsigned long long* __restrict__ flags, int G, unsigned long long step,
                  long n, long slot, float* out, int* status, unsigned long long limit_ns) {
    __shared__ int bad;
    if (threadIdx.x == 0) bad = 0;
    __syncthreads();
    if (threadIdx.x < G) {
        const unsigned long long t0 = now_ns();
        while (ld_acquire_sys(flags + threadIdx.x) < step) {
            if (now_ns() - t0 > limit_ns) { atomicExch(&bad, 1); break; }
            __nanosleep(200);
        }
    }
    __syncthreads();
    if (bad) {
        if (threadIdx.x == 0 && status != nullptr) atomicExch(status, -7);
        return;
    }
    for (long i = ((long)blockIdx.x * blockDim.x + threadIdx.x) * 4; i < n; i += (long)gridDim.x * blockDim.x * 4) {
        float4 s = *reinterpret_cast<const float4*>(recv + i);
        for (int g = 1; g < G; ++g) {
            const float4 v = *reinterpret_cast<const float4*>(recv + g * slot + i);
            s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
        }
        *reinterpret_cast<float4*>(out + i) = s;
    }
}

}  // namespace tpx
