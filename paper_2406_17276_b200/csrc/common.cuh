// Shared device helpers: ordered bf16 keys, mbarrier / bulk-copy wrappers with bounded
// waits, deterministic block reductions.  sm_100a only.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace ot {

constexpr int kThreads = 256;               // threads per CTA in every kernel of the library
constexpr int kWarps = kThreads / 32;
constexpr int kMaxK = 32;
constexpr int kMaxN = 256;

// Device status codes mirror opt_tree_status.
constexpr int kErrTimeout = -4;
constexpr int kErrInternal = -5;

__device__ __forceinline__ void set_status(int* status, int code) {
    atomicCAS(status, 0, code);             // keep the first error
}

// ---------------------------------------------------------------------------------------------
// bf16 bit pattern -> 16-bit key whose unsigned order equals the numeric order of the values
// (-0 is folded into +0 so that equal values have equal keys).
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t ord16(uint32_t bits) {
    bits &= 0xFFFFu;
    if (bits == 0x8000u) bits = 0u;
    return (bits & 0x8000u) ? (~bits & 0xFFFFu) : (bits | 0x8000u);
}
__device__ __forceinline__ uint32_t ord16_inv(uint32_t key) {     // key -> bf16 bits
    return (key & 0x8000u) ? (key & 0x7FFFu) : (~key & 0xFFFFu);
}
__device__ __forceinline__ float bf16_bits_to_float(uint32_t bits) { return __uint_as_float(bits << 16); }

// Candidate key: larger key = better under (logit descending, token id ascending).
__device__ __forceinline__ unsigned long long cand_key(uint32_t bf16_bits, uint32_t token) {
    return ((unsigned long long)ord16(bf16_bits) << 32) | (unsigned long long)(0xFFFFFFFFu - token);
}
__device__ __forceinline__ uint32_t cand_token(unsigned long long key) { return 0xFFFFFFFFu - (uint32_t)key; }
__device__ __forceinline__ float cand_logit(unsigned long long key) {
    return bf16_bits_to_float(ord16_inv((uint32_t)(key >> 32)));
}

constexpr uint32_t kOrdNegInf = 0x007Fu;    // ord16(0xFF80)

// ---------------------------------------------------------------------------------------------
// Small PTX wrappers.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ uint32_t max_bf16x2(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
// d = a * b + c on two packed fp32 lanes.
__device__ __forceinline__ void fma2(float& d0, float& d1, float a0, float a1, float b, float c) {
    unsigned long long A, B, Cc, D;
    asm("mov.b64 %0, {%1, %2};" : "=l"(A) : "f"(a0), "f"(a1));
    asm("mov.b64 %0, {%1, %1};" : "=l"(B) : "f"(b));
    asm("mov.b64 %0, {%1, %1};" : "=l"(Cc) : "f"(c));
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(D) : "l"(A), "l"(B), "l"(Cc));
    asm("mov.b64 {%0, %1}, %2;" : "=f"(d0), "=f"(d1) : "l"(D));
}
__device__ __forceinline__ void add2(float& d0, float& d1, float a0, float a1, float b0, float b1) {
    unsigned long long A, B, D;
    asm("mov.b64 %0, {%1, %2};" : "=l"(A) : "f"(a0), "f"(a1));
    asm("mov.b64 %0, {%1, %2};" : "=l"(B) : "f"(b0), "f"(b1));
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(D) : "l"(A), "l"(B));
    asm("mov.b64 {%0, %1}, %2;" : "=f"(d0), "=f"(d1) : "l"(D));
}

// --- mbarrier + 1-D bulk async copy (global -> this CTA's shared memory, no multicast) ---
__device__ __forceinline__ void mbar_init(unsigned long long* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(unsigned long long* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gmem_src, uint32_t bytes, unsigned long long* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(smem_dst)), "l"(gmem_src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned long long* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\t"
                 "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                 "selp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: gives up after kWaitLimit polls (each poll itself blocks for a hardware-defined
// time slice), records a timeout in the status word and returns false.
constexpr uint32_t kWaitLimit = 1u << 22;
__device__ __forceinline__ bool mbar_wait(unsigned long long* bar, uint32_t parity, int* status) {
    for (uint32_t it = 0; it < kWaitLimit; ++it)
        if (mbar_try_wait(bar, parity)) return true;
    set_status(status, kErrTimeout);
    return false;
}

// ---------------------------------------------------------------------------------------------
// Deterministic block reductions (fixed tree: lanes by xor-shuffle, then warps in order).
// `scratch` needs kWarps entries; every thread gets the result.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}
__device__ __forceinline__ double block_sum(double v, double* scratch) {
    v = warp_sum(v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
    __syncthreads();
    double t = 0.0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) t += scratch[w];
    return t;
}
__device__ __forceinline__ unsigned long long block_max_u64(unsigned long long v, unsigned long long* scratch) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        unsigned long long u = __shfl_xor_sync(0xFFFFFFFFu, v, o);
        v = u > v ? u : v;
    }
    __syncthreads();
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
    __syncthreads();
    unsigned long long t = 0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) t = scratch[w] > t ? scratch[w] : t;
    return t;
}
// Exclusive block scan of one int per thread (thread order); also returns the block total.
__device__ __forceinline__ int block_excl_scan(int v, int* scratch /*kWarps*/, int& total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int u = __shfl_up_sync(0xFFFFFFFFu, inc, o);
        if (lane >= o) inc += u;
    }
    __syncthreads();
    if (lane == 31) scratch[warp] = inc;
    __syncthreads();
    int base = 0, tot = 0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {
        int s = scratch[w];
        if (w < warp) base += s;
        tot += s;
    }
    total = tot;
    return base + inc - v;
}

}  // namespace ot
