// K1: fused row softmax + top-k over the vocabulary (the row step of Algorithm 1: the
// children of a node are its k most probable next tokens; their probabilities feed Eq. 2).
//
// A row of V bf16 logits is read exactly once from HBM, as 32 KB chunks that the issuer warp
// streams into a shared-memory ring with 1-D bulk async copies.
//
// The 16 consumer warps make ONE branch-free pass over every chunk.  A consumer thread owns a
// fixed set of 16-byte vectors of the row (vector index = tid mod 512) and keeps, over the row,
//   * the maximum of its logits (packed bf16x2 max),
//   * the sum of 2^(x*log2e - E) over its logits, E an integer exponent >= its running maximum
//     (raising E rescales the sum by an exact power of two), in packed fp32x2 FMA + ex2.approx.
// Nothing in that pass depends on a threshold, so consecutive rows stream without a bubble.
//
// A finisher warp then turns the 512 per-thread (max, sum) pairs into the row's result:
//   * tau = a lower bound of the row's k-th largest logit, taken from the per-thread maxima, so
//     every winner lives in a thread whose maximum is >= tau ("flagged", a few more than k of 512);
//   * the flagged threads' vectors are read again (they are still in L2) to find the logits >= tau,
//     the candidates, with their tokens; their approximate terms are taken out of the sums again;
//   * candidates are ranked exactly on (bf16 bits, token id) and their exponentials taken in fp64;
//     the threads' sums are combined in fp64; probabilities of the k winners follow.
// Rows this cannot handle (fewer than k finite per-thread maxima, heavy ties, extreme magnitudes)
// are redone by the finisher warp with an exact radix-select path that re-reads the whole row.
#pragma once

#include <cstddef>

#include "common.cuh"

namespace ot {

constexpr int kVecPerThread = 4;                   // 16-byte vectors per consumer thread per chunk
constexpr int kChunkVecs = kConsumers * kVecPerThread;   // 2048
constexpr int kChunkElems = kChunkVecs * 8;        // 16384 bf16 elements per stage (32 KB)
constexpr int kStages = 4;                         // ring depth (128 KB)
constexpr int kSlots = kFinishers + 2;             // finished rows waiting for / held by finishers
constexpr int kCandCap = 128;                      // candidate list capacity per row
constexpr int kMaxFlag = 64;                       // flagged threads the fast finisher accepts
constexpr int kDesc = 4;                           // rows a CTA may hold between ticket and descriptor read
constexpr int kDescRing = 16;                      // descriptors kept: a row's lives until its finisher has copied it
constexpr int kLaneTauMaxK = 16;                   // largest k for which the finisher's threshold comes from the lane maxima
constexpr int kPerLane = kConsumers / 32;          // per-thread results one finisher lane handles (16)

constexpr float kLog2e = 1.44269504088896340736f;
constexpr double kLog2eD = 1.44269504088896340736;
constexpr double kFixScale = 4503599627370496.0;   // 2^52: fixed-point unit of the candidate terms
constexpr float kExpFloor = -16000.0f;             // exponent of a thread that has seen no finite logit
constexpr int kExpLimit = 15000;                   // |E| beyond this: magnitudes the fp32 pass cannot scale

// Fetcher -> issuer / consumers: which row the next chunks of the stream belong to.
struct RowDesc {
    const uint16_t* row;      // global address of the row's first logit
    double pphat;             // tree build: path value of the node being expanded
    int b, d, slot;           // caller's coordinates (sequence, layer, frontier slot / list index)
    int fsize;                // rows in this (sequence, layer)
    int stop;                 // 1: no more rows, shut the pipeline down
};

// Consumers -> finisher: what the fused pass leaves behind for one row.  Thread t's sum is
// relative to the exponent of its warp, warpE[t / 32].  The finisher reads tsum and tkey with
// 16-byte loads, so every slot of the array must start on a 16-byte boundary.
struct alignas(16) RowSlot {
    float tsum[kConsumers];
    uint16_t tkey[kConsumers];     // per-thread maximum as an ordered key
    int warpE[kConsumerWarps];
};

struct alignas(16) FinScratch {    // private to one finisher warp (hist is cleared and read with 16-byte accesses)
    unsigned long long cand[kCandCap];         // candidate keys of the row in hand, unordered
    int hist[256];
    int flist[kMaxFlag];                       // flagged thread ids
    int cand_count;
};

struct LayerJob {                  // what the layer warp hands its assistants (kind 0: leave)
    int kind, d, fsize, n, k, kk;
    double* cand_phat; int32_t* cand_tok; int32_t* T_tok; int32_t* T_par; double* T_phat;
    const int32_t* fmap;           // pruned draft: layer slot of the node behind each frontier row (null: the identity)
    // kind 2 (pruned draft, one selection over the running top-n and the candidates together):
    int nR_old, off;               // old top-n in keys[0..nR_old), candidates from keys[off] (off even, >= nR_old)
    int32_t* Rnew;                 // the new top-n's gids, ascending
};

constexpr int kStageCap = 1024;                    // candidates of a layer that the shared-memory staging holds
constexpr int kSmallN = 256;                       // node budgets up to this use the smaller of the two scratch layouts

// Private to the layer team of a CTA.  NCAP is the largest node budget the layout serves: the kernels
// exist once for NCAP = kSmallN and once for NCAP = kMaxN, so that the common small budgets keep the
// CTA's shared memory (and with it the SM's L1) where it is best for them.
template <int NCAP>
struct alignas(16) LayerScratchT {
    static constexpr int kKeys = (2 * NCAP > kStageCap ? 2 * NCAP : kStageCap) + 2;
    unsigned long long keys[kKeys];            // staged candidate keys, then the keys of R + layer
    unsigned long long lkeys[NCAP];            // keys of the new layer, slot order
    double vals[NCAP];                         // path values of the new running top-n
    int toks[kStageCap + 4];                   // staged candidate tokens
    int gids[2 * NCAP];
    int rsel[NCAP];                            // gids of the new running top-n, ascending
    int ltok[NCAP];                            // tokens of the new layer, slot order
    int hist[256];
    int thist[3][256];                         // the team's digit counts, rotating (all zero between selections)
    unsigned long long red_or[kTeamWarps], red_and[kTeamWarps];
    int scan_a[kTeamWarps], scan_b[kTeamWarps];
    LayerJob job;
    double last_esub;                          // E_sub and |R| of the last update of the running top-n
    int last_nR;
    int scan_c[kTeamWarps];
    int cache_b, cache_d;                      // rsel / vals hold the top-n of this sequence after this layer (-1: nothing)
};

static_assert(sizeof(RowSlot) % 16 == 0, "slots must keep 16-byte alignment in an array");
static_assert(sizeof(FinScratch) % 16 == 0 && offsetof(FinScratch, hist) % 16 == 0, "hist must be 16-byte aligned in every finisher's scratch");
// rows between "descriptor written" and "finisher has its copy": kDesc known + 1 streaming + kSlots handed on
static_assert(kDescRing >= kDesc + 1 + kSlots + 1, "descriptor ring too short");

// The row pipeline's part of a CTA's shared memory (the same for every node budget) ...
struct alignas(128) CtaCore {
    uint16_t stage[kStages][kChunkElems];
    RowSlot slot[kSlots];
    FinScratch fin[kFinishers];
    RowDesc desc[kDescRing];                   // row r in entry r % kDescRing
    unsigned long long full_bar[kStages];      // issuer -> consumers (bulk copy landed)
    unsigned long long empty_bar[kStages];     // consumers -> issuer (stage may be overwritten)
    unsigned long long ready_bar[kSlots];      // consumers -> finisher (slot filled)
    unsigned long long free_bar[kSlots];       // finisher -> consumers (slot may be refilled)
    unsigned long long desc_full[kDesc];       // fetcher -> issuer (descriptor written)
    unsigned long long desc_empty[kDesc];      // consumers -> fetcher (descriptor may be overwritten)
    volatile int stop_row;                     // first row index that is the stop marker
};
// ... and the whole of it, with the layer team's scratch.
template <int NCAP>
struct alignas(128) CtaSmemT {
    CtaCore core;
    LayerScratchT<NCAP> layer;
};
using CtaSmem = CtaSmemT<kSmallN>;
static_assert(sizeof(CtaSmemT<kMaxN>) <= 232448, "the larger layout must fit a CTA's shared memory");

__device__ __forceinline__ int chunk_elems(int V, int c) {
    int rem = V - c * kChunkElems;
    return rem < kChunkElems ? rem : kChunkElems;
}

// ------------------------------------------------------------------------------------------------
// Consumer side.
// ------------------------------------------------------------------------------------------------
struct ThreadAcc {                 // one consumer thread's running state over a row
    unsigned long long acc0, acc1; // packed fp32 pairs
    uint32_t pm;                   // packed bf16x2 running maximum
    float E;                       // integer-valued exponent the sums are relative to
    __device__ __forceinline__ void reset() { acc0 = 0ull; acc1 = 0ull; pm = 0xFF80FF80u; E = kExpFloor; }
};

__device__ __forceinline__ float pow2_float(int d) {            // 2^d for d <= 0; 0 below the normal range
    return __int_as_float(max(d + 127, 0) << 23);
}

// One chunk's share of a consumer thread, taken out of the ring into registers: kVecPerThread
// vectors of 8 logits, their packed maximum and the integer exponent that maximum asks for.
struct ChunkRegs {
    uint4 w[kVecPerThread];
    uint32_t m2;
    float Ec;
};

__device__ __forceinline__ void chunk_take(ChunkRegs& c, const uint4* vec, int nv, int tid) {
#pragma unroll
    for (int u = 0; u < kVecPerThread; ++u) {
        const int v = tid + u * kConsumers;
        c.w[u] = v < nv ? vec[v] : make_uint4(0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u);   // -inf padding
    }
}

// Maximum of the 32 logits and the exponent they want to be summed against (any integer >= max*log2e
// will do: the magic-number add rounds max*log2e + 1 to the nearest integer on the FMA pipe).
__device__ __forceinline__ void chunk_chain(ChunkRegs& c) {
    uint32_t m2 = 0xFF80FF80u;
#pragma unroll
    for (int u = 0; u < kVecPerThread; ++u)
        m2 = max_bf16x2(m2, max_bf16x2(max_bf16x2(c.w[u].x, c.w[u].y), max_bf16x2(c.w[u].z, c.w[u].w)));
    c.m2 = m2;
    const float f = fmaxf(__uint_as_float(m2 << 16), __uint_as_float(m2 & 0xFFFF0000u));
    const float t = fminf(fmaxf(fmaf(f, kLog2e, 1.0f), kExpFloor), -kExpFloor);
    c.Ec = (t + 12582912.0f) - 12582912.0f;
}

// Folds the chunk's maximum into the thread's state (raising E rescales the sums by an exact power
// of two) and returns the packed constant -E for the exponentials.
__device__ __forceinline__ unsigned long long chunk_apply(ThreadAcc& a, const ChunkRegs& c) {
    a.pm = max_bf16x2(a.pm, c.m2);
    const float En = fmaxf(a.E, c.Ec);
    const int d = __float_as_int((a.E - En) + 12582912.0f) - 0x4B400000;     // a.E - En as an integer (<= 0, exact)
    const float sc = pow2_float(d);
    const unsigned long long sc2 = pack2(sc, sc);
    a.acc0 = mul2(a.acc0, sc2);
    a.acc1 = mul2(a.acc1, sc2);
    a.E = En;
    return pack2(-En, -En);
}

// The 32 exponentials of a chunk: 2^(x*log2e - E) in packed fp32x2 FMA + ex2.approx.
__device__ __forceinline__ void chunk_exps(ThreadAcc& a, const ChunkRegs& c, unsigned long long C2) {
    const unsigned long long L2 = pack2(kLog2e, kLog2e);
#pragma unroll
    for (int u = 0; u < kVecPerThread; ++u) {
        const uint32_t ww[4] = {c.w[u].x, c.w[u].y, c.w[u].z, c.w[u].w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float lo = __uint_as_float(ww[i] << 16), hi = __uint_as_float(ww[i] & 0xFFFF0000u);
            float a0, a1;
            unpack2(fma2(pack2(lo, hi), L2, C2), a0, a1);            // x*log2e - E
            const unsigned long long e2 = pack2(ex2_approx(a0), ex2_approx(a1));
            if (i & 1) a.acc1 = add2(a.acc1, e2);
            else       a.acc0 = add2(a.acc0, e2);
        }
    }
}

// End of a row: every thread's sum is brought to its warp's largest exponent and stored.
__device__ __forceinline__ void store_thread_result(RowSlot& slot, const ThreadAcc& a, int tid) {
    float s0, s1;
    unpack2(add2(a.acc0, a.acc1), s0, s1);
    const int e = (int)a.E;
    const int ew = __reduce_max_sync(0xFFFFFFFFu, e);
    slot.tsum[tid] = (s0 + s1) * pow2_float(e - ew);
    slot.tkey[tid] = (uint16_t)max(ord16(a.pm & 0xFFFFu), ord16(a.pm >> 16));
    if ((tid & 31) == 0) slot.warpE[tid >> 5] = ew;
}

// ------------------------------------------------------------------------------------------------
// Finisher side (one warp per row).
// ------------------------------------------------------------------------------------------------
struct RowOut {        // lane j < kk holds the j-th most probable token and its probability
    int kk;
    int32_t tok;
    double p;
};

// 64 keys, two per lane (element i = lane + 32*q is x[q]), sorted descending by element index.
__device__ __forceinline__ void warp_sort64_desc(unsigned long long& x0, unsigned long long& x1) {
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int size = 2; size <= 64; size <<= 1) {
#pragma unroll
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            if (stride == 32) {
                // partner of element lane is element lane+32; in the last merge all pairs keep the maximum low
                const unsigned long long hi = x0 > x1 ? x0 : x1, lo = x0 > x1 ? x1 : x0;
                x0 = hi; x1 = lo;
            } else {
                const unsigned long long p0 = __shfl_xor_sync(0xFFFFFFFFu, x0, stride);
                const unsigned long long p1 = __shfl_xor_sync(0xFFFFFFFFu, x1, stride);
                const bool lower = (lane & stride) == 0;
                const bool desc0 = (lane & size) == 0;                   // block of element lane
                const bool desc1 = ((lane + 32) & size) == 0;            // block of element lane+32
                x0 = (lower == desc0) ? (x0 > p0 ? x0 : p0) : (x0 < p0 ? x0 : p0);
                x1 = (lower == desc1) ? (x1 > p1 ? x1 : p1) : (x1 < p1 ? x1 : p1);
            }
        }
    }
}

// 32 keys, one per lane, sorted descending across lanes.
__device__ __forceinline__ unsigned long long warp_sort32_desc(unsigned long long v) {
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int size = 2; size <= 32; size <<= 1) {
#pragma unroll
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            const unsigned long long p = __shfl_xor_sync(0xFFFFFFFFu, v, stride);
            const bool keep_max = ((lane & stride) == 0) == ((lane & size) == 0);
            v = keep_max ? (v > p ? v : p) : (v < p ? v : p);
        }
    }
    return v;
}

// The finisher's code is walked once per row, by several warps at different places at once, next to
// the consumers' loop: its size decides how often instructions have to be fetched again.  So its
// common path is kept short (packed 16-bit operations, loops instead of unrolled sequences), and
// everything rare sits in functions of its own that are not inlined.

// k-th largest of a slot's per-thread keys (lane l owns tkey[16 l .. 16 l + 16)): two 8-bit radix
// passes over a shared histogram.  1 <= k <= 512.  Rare: only when the maxima spread over more
// than 256 key values.
__device__ __noinline__ uint32_t warp_kth_largest16(const uint16_t* tkey, int k, int* hist) {
    const int lane = threadIdx.x & 31;
    uint32_t prefix = 0;
    int need = k;
    for (int pass = 1; pass >= 0; --pass) {
        for (int j = 0; j < 8; ++j) hist[lane * 8 + j] = 0;
        __syncwarp();
        for (int j = 0; j < kPerLane; ++j) {
            const uint32_t key = tkey[lane * kPerLane + j];
            if (pass == 1 || (key >> 8) == prefix) atomicAdd(&hist[(key >> (8 * pass)) & 255u], 1);
        }
        __syncwarp();
        int c[8], mine = 0;
        for (int j = 0; j < 8; ++j) { c[j] = hist[lane * 8 + j]; mine += c[j]; }
        int incl = mine;                                   // suffix sums over lanes from the top
        for (int o = 1; o < 32; o <<= 1) {
            const int u = __shfl_down_sync(0xFFFFFFFFu, incl, o);
            if (lane + o < 32) incl += u;
        }
        const int above = incl - mine;
        const bool here = above < need && need <= incl;
        int bin = 0, nd = 0;
        if (here) {
            int a = above, bb = 7;
            while (bb > 0 && a + c[bb] < need) { a += c[bb]; --bb; }
            bin = lane * 8 + bb; nd = need - a;
        }
        const int src = __ffs(__ballot_sync(0xFFFFFFFFu, here)) - 1;
        bin = __shfl_sync(0xFFFFFFFFu, bin, src);
        need = __shfl_sync(0xFFFFFFFFu, nd, src);
        prefix = pass == 1 ? (uint32_t)bin : ((prefix << 8) | (uint32_t)bin);
        __syncwarp();
    }
    return prefix;
}

// The kk-th largest of a slot's 512 per-thread maxima, exactly: a histogram with one bin per key
// value over the 256 values below the largest usually holds kk of them (the maxima of a row lie close
// together); otherwise two generic radix passes.  Used when kk is too large for the lanes' maxima to
// give a useful bound (see finish_row_warp).
__device__ __noinline__ uint32_t tau_from_histogram(FinScratch& f, const uint16_t* tkey, uint32_t mk, int kk) {
    const int lane = threadIdx.x & 31;
    const uint32_t base = mk > 255u ? mk - 255u : 0u;
    for (int j = 0; j < 8; ++j) f.hist[lane * 8 + j] = 0;
    __syncwarp();
    for (int q = 0; q < kPerLane; ++q) {
        const uint32_t key = tkey[lane * kPerLane + q];
        if (key >= base) atomicAdd(&f.hist[key - base], 1);
    }
    __syncwarp();
    int c[8], mine = 0;
    for (int j = 0; j < 8; ++j) { c[j] = f.hist[lane * 8 + j]; mine += c[j]; }
    int incl = mine;                                   // suffix sums over lanes from the top
    for (int o = 1; o < 32; o <<= 1) {
        const int u = __shfl_down_sync(0xFFFFFFFFu, incl, o);
        if (lane + o < 32) incl += u;
    }
    const int above = incl - mine;
    const bool here = above < kk && kk <= incl;
    int bin = 0;
    if (here) {
        int a = above, bb = 7;
        while (bb > 0 && a + c[bb] < kk) { a += c[bb]; --bb; }
        bin = lane * 8 + bb;
    }
    const unsigned hm = __ballot_sync(0xFFFFFFFFu, here);
    __syncwarp();
    if (hm) return base + (uint32_t)__shfl_sync(0xFFFFFFFFu, bin, __ffs(hm) - 1);
    return warp_kth_largest16(tkey, kk, f.hist);
}

// Exact path for one row by one warp: radix select on the 16-bit keys, ordered tie handling,
// fp64 sum.  Leaves exactly kk candidates in f.cand and returns the row maximum and sum.
__device__ __noinline__ void row_exact_warp(FinScratch& f, const uint16_t* row, int V, int kk, double& m_out, double& S_out) {
    const int lane = threadIdx.x & 31;
    uint32_t mk = 0;
    for (int v = lane; v < V; v += 32) mk = max(mk, ord16(__ldg(row + v)));
    mk = __reduce_max_sync(0xFFFFFFFFu, mk);
    const double m = (double)bf16_bits_to_float(ord16_inv(mk));
    uint32_t prefix = 0, pmask = 0;
    int need = kk;
    for (int pass = 1; pass >= 0; --pass) {
        for (int j = 0; j < 8; ++j) f.hist[lane * 8 + j] = 0;
        __syncwarp();
        for (int v = lane; v < V; v += 32) {
            const uint32_t key = ord16(__ldg(row + v));
            if ((key & pmask) == prefix) atomicAdd(&f.hist[(key >> (8 * pass)) & 255u], 1);
        }
        __syncwarp();
        int c[8], mine = 0;
        for (int j = 0; j < 8; ++j) { c[j] = f.hist[lane * 8 + j]; mine += c[j]; }
        int incl = mine;
        for (int o = 1; o < 32; o <<= 1) {
            int u = __shfl_down_sync(0xFFFFFFFFu, incl, o);
            if (lane + o < 32) incl += u;
        }
        const int above = incl - mine;
        const bool here = above < need && need <= incl;
        int bin = 0, nd = 0;
        if (here) {
            int a = above, b = 7;
            while (b > 0 && a + c[b] < need) { a += c[b]; --b; }
            bin = lane * 8 + b; nd = need - a;
        }
        const int src = __ffs(__ballot_sync(0xFFFFFFFFu, here)) - 1;
        bin = __shfl_sync(0xFFFFFFFFu, bin, src);
        need = __shfl_sync(0xFFFFFFFFu, nd, src);
        prefix |= (uint32_t)bin << (8 * pass);
        pmask |= 0xFFu << (8 * pass);
        __syncwarp();
    }
    const uint32_t thr = prefix;       // kk-th largest key; `need` of its copies belong, lowest tokens first
    int count = 0, eq_seen = 0;
    double acc = 0.0;
    uint32_t memo_bits = 0x10000u;     // one-entry memo of the last exponential (tie-heavy rows)
    double memo_e = 0.0;
    for (int v0 = 0; v0 < V; v0 += 32) {
        const int v = v0 + lane;
        uint32_t bits = 0xFF80u, key = 0;
        const bool valid = v < V;
        if (valid) { bits = __ldg(row + v); key = ord16(bits); }
        const unsigned eqm = __ballot_sync(0xFFFFFFFFu, valid && key == thr);
        const int eq_rank = eq_seen + __popc(eqm & ((1u << lane) - 1u));
        eq_seen += __popc(eqm);
        const bool take = valid && (key > thr || (key == thr && eq_rank < need));
        const unsigned tm = __ballot_sync(0xFFFFFFFFu, take);
        if (take) f.cand[count + __popc(tm & ((1u << lane) - 1u))] = cand_key(bits, (uint32_t)v);
        count += __popc(tm);
        if (valid && key > kOrdNegInf) {
            if (bits != memo_bits) { memo_bits = bits; memo_e = exp((double)bf16_bits_to_float(bits) - m); }
            acc += memo_e;
        }
    }
    __syncwarp();
    if (lane == 0) f.cand_count = count;
    __syncwarp();
    m_out = m;
    S_out = warp_sum(acc);
}

// One 16-byte vector of the row (8 logits starting at token 8*vi) as four packed words; logits at or
// beyond V read as -inf.  `aligned` rows take one vector load, others eight scalar loads.
__device__ __noinline__ uint4 load_row_vec_scalar(const uint16_t* row, int vi, int V) {
    uint32_t h[8];
    for (int e = 0; e < 8; ++e) h[e] = (vi * 8 + e < V) ? (uint32_t)__ldg(row + vi * 8 + e) : 0xFF80u;
    return make_uint4(h[0] | (h[1] << 16), h[2] | (h[3] << 16), h[4] | (h[5] << 16), h[6] | (h[7] << 16));
}
__device__ __forceinline__ uint4 load_row_vec(const uint16_t* row, int vi, int V, bool aligned) {
    if (aligned) {
        uint4 v;
        asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];"
                     : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(reinterpret_cast<const uint4*>(row) + vi));
        return v;
    }
    return load_row_vec_scalar(row, vi, V);
}

__device__ __noinline__ double exp_f64(double x) { return exp(x); }    // one copy of the routine for all its callers

// bf16x2 "a >= b" per half: 0xFFFF where true
__device__ __forceinline__ uint32_t ge_bf16x2(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("set.ge.u32.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}

// Ranks M <= 64 candidates (f.cand[0..M), distinct keys) and gives lane j < kk the j-th largest with
// its probability.  S is the row's sum without the candidates unless `exact`.  The common case, up
// to one candidate per lane, ranks by counting; more than 32 are sorted (rare).
__device__ __noinline__ void finish_many(FinScratch& f, int M, int kk, double m, double S, bool exact, RowOut& out) {
    const int lane = threadIdx.x & 31;
    unsigned long long x0 = f.cand[lane], x1 = lane + 32 < M ? f.cand[lane + 32] : 0ull;
    warp_sort64_desc(x0, x1);
    const double e0 = exp_f64((double)cand_logit(x0) - m);
    const double e1 = x1 ? exp_f64((double)cand_logit(x1) - m) : 0.0;
    if (!exact) S += (double)warp_sum_u64(__double2ull_rn(e0 * kFixScale) + __double2ull_rn(e1 * kFixScale)) / kFixScale;
    if (lane < kk) { out.tok = (int32_t)cand_token(x0); out.p = e0 / S; }
}

// Turns a finished slot into the row's k winners.  Whole finisher warp; f is its private scratch.
__device__ __forceinline__ void finish_row_warp(FinScratch& f, const RowSlot& slot, const uint16_t* row, int V, int k, bool aligned, RowOut& out) {
    const int lane = threadIdx.x & 31;
    const int kk = k < V ? k : V;
    const int nvec = (V + 7) >> 3;

    // this lane's 16 consecutive threads all belong to consumer warp lane / 2; two 16-bit keys per word
    uint32_t kw[kPerLane / 2];
    {
        const uint4* kp = reinterpret_cast<const uint4*>(&slot.tkey[lane * kPerLane]);
        const uint4 a = kp[0], b = kp[1];
        kw[0] = a.x; kw[1] = a.y; kw[2] = a.z; kw[3] = a.w; kw[4] = b.x; kw[5] = b.y; kw[6] = b.z; kw[7] = b.w;
    }
    const int myE = slot.warpE[lane >> 1];
    const int emax = __reduce_max_sync(0xFFFFFFFFu, myE);
    uint32_t lane_mk = kw[0];
#pragma unroll
    for (int q = 1; q < kPerLane / 2; ++q) lane_mk = __vmaxu2(lane_mk, kw[q]);
    const uint32_t mk = __reduce_max_sync(0xFFFFFFFFu, max(lane_mk & 0xFFFFu, lane_mk >> 16));

    // tau: the kk-th largest of the 32 lanes' maxima (each the largest of 16 per-thread maxima).  That
    // is at most the kk-th largest per-thread maximum, hence at most the row's kk-th largest logit, so
    // every winner still lives in a thread whose maximum is >= tau; a few more threads than kk get
    // flagged, and in exchange tau takes sixteen ballots instead of a histogram over 512 keys.
    // With fewer than kk finite lane maxima tau is -inf and the row goes the exact way.  The bound gets
    // loose as kk approaches the 32 lanes (about 32 ln(32 / (32 - kk)) threads are flagged), so beyond
    // kLaneTauMaxK the exact kk-th largest per-thread maximum is used instead.
    uint32_t tau_key = 0;
    if (kk > kLaneTauMaxK) {
        tau_key = tau_from_histogram(f, slot.tkey, mk, kk);
    } else {
        const uint32_t lane_max = max(lane_mk & 0xFFFFu, lane_mk >> 16);
        unsigned cand = 0xFFFFFFFFu;                       // lanes whose maximum matches tau's bits so far
        int need = kk;
#pragma unroll 1
        for (int bit = 15; bit >= 0; --bit) {
            const unsigned ones = __ballot_sync(0xFFFFFFFFu, (lane_max >> bit) & 1u) & cand;
            const int c = __popc(ones);
            if (c >= need) { tau_key |= 1u << bit; cand = ones; }
            else { need -= c; cand &= ~ones; }
        }
    }
    bool exact = tau_key <= kOrdNegInf || emax >= kExpLimit || emax <= -kExpLimit;

    // the sum of all threads' partial sums; flagged threads (maximum >= tau) listed in thread order
    uint32_t fmask = 0;
    float part32 = 0.0f;
    {
        const uint32_t tau2 = tau_key | (tau_key << 16);
#pragma unroll
        for (int q = 0; q < kPerLane / 2; ++q) {
            const uint32_t g = __vcmpgeu2(kw[q], tau2);    // 0xFFFF per key >= tau
            fmask |= ((g & 1u) | ((g >> 15) & 2u)) << (2 * q);
        }
        const float4* sp = reinterpret_cast<const float4*>(&slot.tsum[lane * kPerLane]);
#pragma unroll
        for (int q = 0; q < kPerLane / 4; ++q) {
            const float4 t4 = sp[q];
            part32 += (t4.x + t4.y) + (t4.z + t4.w);
        }
    }
    int nflag = 0;
    if (!exact) {
        const int base = warp_excl_scan(__popc(fmask), nflag);
        if (nflag <= kMaxFlag) {
            int pos = base;
            for (uint32_t mm = fmask; mm; mm &= mm - 1) f.flist[pos++] = lane * kPerLane + (__ffs(mm) - 1);
        } else {
            exact = true;
        }
    }
    if (lane == 0) f.cand_count = 0;
    __syncwarp();

    double m = (double)bf16_bits_to_float(ord16_inv(mk)), S = 0.0;
    int M = 0;
    if (!exact) {
        const double part = (double)(part32 * pow2_float(myE - emax));
        // Flagged threads: their vectors are read again only to find the candidates (logit >= tau) and
        // their tokens.  A candidate's term is already inside its thread's partial sum; the same
        // approximate term is taken out again here (the two differ by rounding of the exponent, a
        // few 1e-8 of the term), and the candidate comes back below with an exact exponential.
        // Work item i: flagged thread i mod P (P = nflag rounded up to a power of two), vector i / P.
        const uint32_t tau_bits = ord16_inv(tau_key);
        const float tau_f = bf16_bits_to_float(tau_bits);
        const uint32_t tau_b2 = tau_bits | (tau_bits << 16);
        const int nchunks = (V + kChunkElems - 1) / kChunkElems;
        const int vpt = nchunks * kVecPerThread;
        const int lg = nflag > 1 ? 32 - __clz(nflag - 1) : 0;
        const int total = vpt << lg;
        const float negE = -(float)emax;
        float sub = 0.0f;
        double corr = 1.0;                                  // e^gap, see below; computed while the first loads are in flight
#pragma unroll 1
        for (int i0 = 0; i0 < total; i0 += 32 * 4) {
            uint4 w[4];
            int vis[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int idx = i0 + u * 32 + lane;
                const int fi = idx & ((1 << lg) - 1), j = idx >> lg;
                vis[u] = -1;
                w[u] = make_uint4(0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u);
                if (idx < total && fi < nflag) {
                    const int vi = (j / kVecPerThread) * kChunkVecs + (j % kVecPerThread) * kConsumers + f.flist[fi];
                    if (vi < nvec) { vis[u] = vi; w[u] = load_row_vec(row, vi, V, aligned); }
                }
            }
            if (i0 == 0) {
                // Bulk terms are 2^(fl(x*L32) - E) with L32 the fp32 log2(e); wanted e^(x-m) = 2^((x-m)*L).
                // The exponent gap E - m*L + x*(L - L32) is evaluated at a typical bulk logit x = tau - 2.
                const double gap = (double)emax - m * kLog2eD + ((double)tau_f - 2.0) * (kLog2eD - (double)kLog2e);
                corr = exp_f64(gap * 0.693147180559945309417);
            }
            // bit 8u+e of m32: element e of vector u is a candidate (most vectors hold none)
            uint32_t m32 = 0;
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const uint32_t gx = ge_bf16x2(w[u].x, tau_b2), gy = ge_bf16x2(w[u].y, tau_b2);
                const uint32_t gz = ge_bf16x2(w[u].z, tau_b2), gw = ge_bf16x2(w[u].w, tau_b2);
                const uint32_t m8 = ((gx & 1u) | ((gx >> 15) & 2u)) | (((gy & 1u) | ((gy >> 15) & 2u)) << 2) |
                                    (((gz & 1u) | ((gz >> 15) & 2u)) << 4) | (((gw & 1u) | ((gw >> 15) & 2u)) << 6);
                m32 |= (vis[u] < 0 ? 0u : m8) << (8 * u);
            }
#pragma unroll 1
            while (m32) {
                const int e = __ffs(m32) - 1;
                m32 &= m32 - 1;
                const int u = e >> 3, h = e & 7;
                const uint4 wu = u < 2 ? (u == 0 ? w[0] : w[1]) : (u == 2 ? w[2] : w[3]);
                const int vi = u < 2 ? (u == 0 ? vis[0] : vis[1]) : (u == 2 ? vis[2] : vis[3]);
                const uint32_t word = h < 4 ? (h < 2 ? wu.x : wu.y) : (h < 6 ? wu.z : wu.w);
                const uint32_t bits = (h & 1) ? (word >> 16) : (word & 0xFFFFu);
                const int pos = atomicAdd(&f.cand_count, 1);
                if (pos < kCandCap) f.cand[pos] = cand_key(bits, (uint32_t)(vi * 8 + h));
                sub += ex2_approx(fmaf(bf16_bits_to_float(bits), kLog2e, negE));
            }
        }
        __syncwarp();
        M = f.cand_count;
        if (M > 64) exact = true;
        else {
            S = warp_sum(part - (double)sub) * corr;
        }
    }
    if (exact) {
        row_exact_warp(f, row, V, kk, m, S);
        M = f.cand_count;                                     // == kk <= 32
    }
    __syncwarp();

    out.kk = kk; out.tok = -1; out.p = 0.0;
    if (M <= 32) {
        // one candidate per lane: every lane's exponential once; its rank is the number of larger
        // candidates (keys are distinct), and rank j's token and term go to lane j through the scratch
        const unsigned long long mine = lane < M ? f.cand[lane] : 0ull;
        const double e = lane < M ? exp_f64((double)cand_logit(mine) - m) : 0.0;
        if (!exact) S += (double)warp_sum_u64(__double2ull_rn(e * kFixScale)) / kFixScale;   // integer sum: order free
        int rank = 0;
#pragma unroll 4
        for (int j = 0; j < M; ++j) rank += __shfl_sync(0xFFFFFFFFu, mine, j) > mine ? 1 : 0;
        __syncwarp();
        if (lane < M) { f.cand[rank] = mine; f.cand[32 + rank] = (unsigned long long)__double_as_longlong(e); }
        __syncwarp();
        if (lane < kk) {
            out.tok = (int32_t)cand_token(f.cand[lane]);
            out.p = __longlong_as_double((long long)f.cand[32 + lane]) / S;
        }
        __syncwarp();
    } else {
        finish_many(f, M, kk, m, S, exact, out);
    }
}

}  // namespace ot
