// Shared device helpers: ordered bf16 keys, mbarrier / bulk-copy wrappers with bounded
// waits, warp-level reductions.  sm_100a only.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace ot {

// CTA shape of the row pipeline (one CTA per SM): 16 consumer warps stream the logits, an issuer
// warp feeds the shared-memory ring, a fetcher warp obtains row descriptors ahead of time, several
// finisher warps (one row each, round robin) turn finished rows into probabilities and tree
// updates, and a layer team (the layer warp and its assistants) selects the next layer of the
// trees the CTA follows.
//
// Warp w of a CTA issues from scheduler w % 4 of its SM: the consumers are warps 0..15, the
// helpers follow, ordered so that the four warps of the layer team sit on four different
// schedulers.  (Helper warps advance at roughly half their speed while the consumers are busy,
// which is why the layer selection, the longest serial step between two layers, is spread over
// several of them.)
constexpr int kConsumerWarps = 16;
constexpr int kConsumers = kConsumerWarps * 32;     // 512 consumer threads
constexpr int kFinishers = 6;
constexpr int kTeamWarps = 4;                       // layer warp + assistants
constexpr int kTeam = kTeamWarps * 32;
constexpr int kHelperWarps = 2 + kTeamWarps + kFinishers;
constexpr int kWarps = kConsumerWarps + kHelperWarps;
constexpr int kThreads = kWarps * 32;               // 896 threads per CTA
enum { kHelperIssuer = 0, kHelperFetcher = 1, kHelperLayer = 2, kHelperFirstAssistant = 3, kHelperFirstFinisher = 2 + kTeamWarps };
constexpr int kMaxK = 32;
constexpr int kMaxN = 1024;

// Device status codes mirror opt_tree_status.
constexpr int kErrTimeout = -4;
constexpr int kErrInternal = -5;

__device__ __forceinline__ void set_status(int* status, int code) {
    atomicCAS(status, 0, code);             // keep the first error
}

// Every wait in the library is bounded by this many SM clock cycles (about two seconds); on
// expiry the waiter records kErrTimeout in the status word and gives up, so a protocol error
// ends as an error code, never as a hang.  The waits take the limit as an argument only so that
// the self-test (opt_tree_selftest_waits) can make each of them run out within microseconds.
constexpr long long kWaitCycles = 1ll << 32;
constexpr int kWaitPolls = 1 << 22;                 // limit of the waits that count polls instead of cycles

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
// Packed fp32 pairs (two lanes per instruction).
__device__ __forceinline__ unsigned long long pack2(float lo, float hi) {
    unsigned long long r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(unsigned long long v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ unsigned long long fma2(unsigned long long a, unsigned long long b, unsigned long long c) {
    unsigned long long d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ unsigned long long mul2(unsigned long long a, unsigned long long b) {
    unsigned long long d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ unsigned long long add2(unsigned long long a, unsigned long long b) {
    unsigned long long d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}

__device__ __forceinline__ void named_barrier_sync(int id, int nthreads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

// --- mbarrier + 1-D bulk async copy (global -> this CTA's shared memory, no multicast) ---
__device__ __forceinline__ void mbar_init(unsigned long long* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned long long* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
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
// Bounded wait, called by every lane of a converged warp (try_wait suspends the thread in hardware
// for a while, so the loop turns over slowly; the clock is read only once in 256 turns).  Returns
// false to the whole warp (status set) when kWaitCycles pass without completion.
__device__ __forceinline__ bool mbar_wait_warp(unsigned long long* bar, uint32_t parity, int* status, long long limit = kWaitCycles) {
    if (mbar_try_wait(bar, parity)) return true;
    long long t0 = 0;
    int turns = 0;
    bool ok = true;
    while (!mbar_try_wait(bar, parity)) {
        if ((++turns & 255) == 0) {
            const long long now = clock64();
            if (t0 == 0) t0 = now;
            else if (now - t0 > limit) { ok = false; break; }
        }
    }
    if (!ok) set_status(status, kErrTimeout);
    return __all_sync(0xFFFFFFFFu, ok);
}

// Non-blocking test of a phase (does not suspend the thread).
__device__ __forceinline__ bool mbar_test_wait(unsigned long long* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\t"
                 "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                 "selp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// The same wait for a single thread whose warp mates are busy elsewhere (no warp-wide vote).
__device__ __forceinline__ bool mbar_wait_thread(unsigned long long* bar, uint32_t parity, int* status, long long limit = kWaitCycles) {
    if (mbar_try_wait(bar, parity)) return true;
    long long t0 = 0;
    int turns = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++turns & 255) == 0) {
            const long long now = clock64();
            if (t0 == 0) t0 = now;
            else if (now - t0 > limit) { set_status(status, kErrTimeout); return false; }
        }
    }
    return true;
}

// --- programmatic dependent launch: a kernel launched "after" another in the same stream may be
//     set up while its predecessor drains; nothing of the predecessor's may be read or overwritten
//     before this returns (no effect in a kernel launched the ordinary way) ---
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// --- barrier of the layer team (named barrier 1; barrier 0 is the CTA's) ---
__device__ __forceinline__ void team_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kTeam) : "memory"); }

// --- asynchronous global -> shared copies (16 bytes, L2 only: the data was written by other SMs;
//     all copies of a sweep are in flight at once and need no registers) ---
__device__ __forceinline__ void cp_async_16(void* smem_dst, const void* gmem_src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(smem_dst)), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() {
    asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
}

// --- global-memory flags and mailbox words (gpu scope) ---
__device__ __forceinline__ unsigned long long ld_acquire_u64(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ unsigned long long ld_relaxed_u64(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void atom_add_relaxed_s32(int* p, int v) {
    asm volatile("red.relaxed.gpu.global.add.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ unsigned int ld_relaxed_u32(const unsigned int* p) {
    unsigned int v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_u64(unsigned long long* p, unsigned long long v) {
    asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ int ld_acquire_s32(const int* p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_relaxed_u64(unsigned long long* p, unsigned long long v) {
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ void st_release_s32(int* p, int v) {
    asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// ---------------------------------------------------------------------------------------------
// Warp-level reductions / scans (fixed shuffle trees: deterministic).
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}
__device__ __forceinline__ unsigned long long warp_sum_u64(unsigned long long v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max_f32(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
    return v;
}
__device__ __forceinline__ unsigned long long warp_max_u64(unsigned long long v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        unsigned long long u = __shfl_xor_sync(0xFFFFFFFFu, v, o);
        v = u > v ? u : v;
    }
    return v;
}
__device__ __forceinline__ int warp_sum_i32(int v) { return __reduce_add_sync(0xFFFFFFFFu, v); }
// Exclusive scan of one int per lane; total returned through `total`.
__device__ __forceinline__ int warp_excl_scan(int v, int& total) {
    const int lane = threadIdx.x & 31;
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int u = __shfl_up_sync(0xFFFFFFFFu, inc, o);
        if (lane >= o) inc += u;
    }
    total = __shfl_sync(0xFFFFFFFFu, inc, 31);
    return inc - v;
}

}  // namespace ot
