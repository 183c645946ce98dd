// K1: fused row softmax + top-k over the vocabulary (the row step of Algorithm 1: the
// children of a node are its k most probable next tokens; their probabilities feed Eq. 2).
//
// A row of V bf16 logits is read exactly once from global memory, as 16 KB chunks that a
// producer warp streams into a shared-memory ring with 1-D bulk async copies.  The eight
// consumer warps
//   * scan the first chunk(s) of the row for per-thread maxima; the k-th largest of those is a
//     lower bound tau of the row's k-th largest logit;
//   * then make ONE fused pass over every chunk: a logit >= tau goes to a small candidate list
//     (it may be a winner, and it certainly includes the row maximum), every other logit adds
//     2^((x - tau) * log2 e) to an fp32 partial sum (packed fp32x2 FMA + ex2.approx);
// and a finisher warp turns the candidate list and the partial sums into the row's result:
// exact ranking of the candidates on (bf16 bits, token id), fp64 exponentials for the candidates,
// fp64 combine of the bulk, probabilities of the k winners.
// Rows whose candidate list overflows (heavy ties, mostly -inf rows, tiny V) are redone by the
// finisher warp with an exact radix-select path that re-reads the row from global memory.
#pragma once

#include "common.cuh"

namespace ot {

constexpr int kChunkElems = 8192;                  // bf16 elements per stage (16 KB)
constexpr int kChunkVecs = kChunkElems / 8;        // 16-byte vectors per stage
constexpr int kVecPerThread = kChunkVecs / kConsumers;   // 4
constexpr int kStages = 3;                         // ring depth (48 KB)
constexpr int kCandCap = 512;                      // candidate list capacity per row
constexpr int kDesc = 8;                           // row descriptors in flight (> kStages)

constexpr float kLog2e = 1.44269504088896340736f;
constexpr double kLog2eD = 1.44269504088896340736;
constexpr double kFixScale = 4503599627370496.0;   // 2^52: fixed-point unit of the candidate terms

// Producer -> consumers: which row the next chunks of the stream belong to.
struct RowDesc {
    const uint16_t* row;      // global address of the row's first logit
    int b, d, slot;           // caller's coordinates (sequence, layer, frontier slot / list index)
    int fsize;                // rows in this (sequence, layer)
    int stop;                 // 1: no more rows, shut the pipeline down
};

// Consumers -> finisher: everything the fused pass leaves behind for one row.
struct RowSlot {
    unsigned long long cand[kCandCap];     // candidate keys, unordered
    double warp_part[kConsumerWarps];      // per-warp sums of 2^((x-tau)*log2e) over non-candidates
    RowDesc desc;
    int cand_count;                        // may exceed kCandCap: overflow -> exact path
    uint32_t tau_key;                      // ord16 of tau; <= kOrdNegInf -> exact path
};

struct alignas(128) CtaSmem {
    uint16_t stage[kStages][kChunkElems];
    RowSlot slot[2];
    RowDesc desc[kDesc];
    unsigned long long full_bar[kStages];      // producer -> consumers (bulk copy landed)
    unsigned long long empty_bar[kStages];     // consumers -> producer (stage may be overwritten)
    unsigned long long ready_bar[2];           // consumers -> finisher (slot filled)
    unsigned long long free_bar[2];            // finisher -> consumers (slot may be refilled)
    uint32_t tmax[kConsumerWarps][32];
    uint32_t tau_key;
    // finisher scratch
    unsigned long long keys[1024];
    double vals[kMaxN];
    int gids[2 * kMaxN];
    int hist[256];
};

// ---- k-th largest of one 16-bit key per consumer thread (k <= 32) ---------------------------
__device__ __forceinline__ uint32_t warp_sort_desc(uint32_t v) {
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int size = 2; size <= 32; size <<= 1) {
#pragma unroll
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            uint32_t p = __shfl_xor_sync(0xFFFFFFFFu, v, stride);
            bool keep_max = ((lane & stride) == 0) == ((lane & size) == 0);
            v = keep_max ? max(v, p) : min(v, p);
        }
    }
    return v;
}
// a, b sorted descending across lanes -> the 32 largest of both, sorted descending.
__device__ __forceinline__ uint32_t warp_merge_top32(uint32_t a, uint32_t b) {
    const int lane = threadIdx.x & 31;
    uint32_t v = max(a, __shfl_sync(0xFFFFFFFFu, b, 31 - lane));
#pragma unroll
    for (int stride = 16; stride > 0; stride >>= 1) {
        uint32_t p = __shfl_xor_sync(0xFFFFFFFFu, v, stride);
        v = ((lane & stride) == 0) ? max(v, p) : min(v, p);
    }
    return v;
}
// Called by all consumer threads (named barrier 1).
__device__ __forceinline__ uint32_t consumers_kth_largest(uint32_t key, int k, CtaSmem& s) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    s.tmax[warp][lane] = warp_sort_desc(key);
    named_barrier_sync(1, kConsumers);
    if (warp == 0) {
        uint32_t v[kConsumerWarps];
#pragma unroll
        for (int w = 0; w < kConsumerWarps; ++w) v[w] = s.tmax[w][lane];
#pragma unroll
        for (int step = 1; step < kConsumerWarps; step <<= 1)
#pragma unroll
            for (int w = 0; w + step < kConsumerWarps; w += 2 * step) v[w] = warp_merge_top32(v[w], v[w + step]);
        uint32_t kth = __shfl_sync(0xFFFFFFFFu, v[0], k - 1);
        if (lane == 0) s.tau_key = kth;
    }
    named_barrier_sync(1, kConsumers);
    return s.tau_key;
}

__device__ __forceinline__ int chunk_elems(int V, int c) {
    int rem = V - c * kChunkElems;
    return rem < kChunkElems ? rem : kChunkElems;
}

__device__ __forceinline__ void push_cand(RowSlot& slot, uint32_t bits, uint32_t token) {
    int pos = atomicAdd(&slot.cand_count, 1);
    if (pos < kCandCap) slot.cand[pos] = cand_key(bits, token);
}

// Rare path of the fused pass: this thread's vectors of the chunk hold at least one candidate.
__device__ __noinline__ float chunk_pass_slow(RowSlot& slot, uint4 w0, uint4 w1, uint4 w2, uint4 w3, uint32_t token_base,
                                               int tid, float tau, float c_tau) {
    static_assert(kVecPerThread == 4, "chunk_pass_slow takes four vectors");
    float sum = 0.0f;
#pragma unroll
    for (int u = 0; u < kVecPerThread; ++u) {
        const uint4 wu = u == 0 ? w0 : (u == 1 ? w1 : (u == 2 ? w2 : w3));
        const uint32_t ww[4] = {wu.x, wu.y, wu.z, wu.w};
        const uint32_t tok0 = token_base + (uint32_t)(tid + u * kConsumers) * 8u;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint32_t bits = (i & 1) ? (ww[i >> 1] >> 16) : (ww[i >> 1] & 0xFFFFu);
            const float x = bf16_bits_to_float(bits);
            if (x >= tau) push_cand(slot, bits, tok0 + i);
            else sum += ex2_approx(fmaf(x, kLog2e, c_tau));
        }
    }
    return sum;
}

// Fused pass over this thread's share of one chunk (kVecPerThread vectors of 8 logits).
__device__ __forceinline__ float chunk_pass(RowSlot& slot, const uint4* vec, int nv, uint32_t token_base, int tid,
                                            float tau, float c_tau) {
    uint4 w[kVecPerThread];
#pragma unroll
    for (int u = 0; u < kVecPerThread; ++u) {
        const int v = tid + u * kConsumers;
        w[u] = v < nv ? vec[v] : make_uint4(0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u);   // -inf padding
    }
    const unsigned long long L2 = pack2(kLog2e, kLog2e), C2 = pack2(c_tau, c_tau);
    unsigned long long acc0 = 0ull, acc1 = 0ull;       // packed (0.0f, 0.0f)
    float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
    for (int u = 0; u < kVecPerThread; ++u) {
        const uint32_t ww[4] = {w[u].x, w[u].y, w[u].z, w[u].w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float lo = __uint_as_float(ww[i] << 16), hi = __uint_as_float(ww[i] & 0xFFFF0000u);
            float a0, a1;
            unpack2(fma2(pack2(lo, hi), L2, C2), a0, a1);            // (x - tau) * log2(e)
            const unsigned long long e2 = pack2(ex2_approx(a0), ex2_approx(a1));
            if (i & 1) { acc1 = add2(acc1, e2); mx1 = max3(mx1, lo, hi); }
            else       { acc0 = add2(acc0, e2); mx0 = max3(mx0, lo, hi); }
        }
    }
    if (fmaxf(mx0, mx1) >= tau) return chunk_pass_slow(slot, w[0], w[1], w[2], w[3], token_base, tid, tau, c_tau);
    float s0, s1;
    unpack2(add2(acc0, acc1), s0, s1);
    return s0 + s1;
}

// Per-thread packed maximum over this thread's share of one chunk (the sampling pass).
__device__ __forceinline__ uint32_t chunk_max(const uint4* vec, int nv, int tid, uint32_t pm) {
#pragma unroll
    for (int u = 0; u < kVecPerThread; ++u) {
        const int v = tid + u * kConsumers;
        if (v < nv) {
            const uint4 w = vec[v];
            pm = max_bf16x2(max_bf16x2(pm, w.x), max_bf16x2(w.y, max_bf16x2(w.z, w.w)));
        }
    }
    return pm;
}

// ------------------------------------------------------------------------------------------------
// Finisher side (one warp).
// ------------------------------------------------------------------------------------------------
struct RowOut {        // lane j < kk holds the j-th most probable token and its probability
    int kk;
    int32_t tok;
    double p;
};

// Exact path for one row by one warp: radix select on the 16-bit keys, ordered tie handling,
// fp64 sum.  Leaves exactly kk candidates in slot.cand and returns the row maximum and sum.
__device__ __noinline__ void row_exact_warp(CtaSmem& s, RowSlot& slot, const uint16_t* row, int V, int kk,
                                            double& m_out, double& S_out) {
    const int lane = threadIdx.x & 31;
    uint32_t mk = 0;
    for (int v = lane; v < V; v += 32) mk = max(mk, ord16(__ldg(row + v)));
    mk = __reduce_max_sync(0xFFFFFFFFu, mk);
    const double m = (double)bf16_bits_to_float(ord16_inv(mk));
    uint32_t prefix = 0, pmask = 0;
    int need = kk;
    for (int pass = 1; pass >= 0; --pass) {
        for (int j = 0; j < 8; ++j) s.hist[lane * 8 + j] = 0;
        __syncwarp();
        for (int v = lane; v < V; v += 32) {
            const uint32_t key = ord16(__ldg(row + v));
            if ((key & pmask) == prefix) atomicAdd(&s.hist[(key >> (8 * pass)) & 255u], 1);
        }
        __syncwarp();
        int c[8], mine = 0;
        for (int j = 0; j < 8; ++j) { c[j] = s.hist[lane * 8 + j]; mine += c[j]; }
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
        if (take) slot.cand[count + __popc(tm & ((1u << lane) - 1u))] = cand_key(bits, (uint32_t)v);
        count += __popc(tm);
        if (valid && key > kOrdNegInf) {
            if (bits != memo_bits) { memo_bits = bits; memo_e = exp((double)bf16_bits_to_float(bits) - m); }
            acc += memo_e;
        }
    }
    __syncwarp();
    if (lane == 0) slot.cand_count = count;
    __syncwarp();
    m_out = m;
    S_out = warp_sum(acc);
}

// Turns a finished slot into the row's k winners.  Whole finisher warp.
__device__ __forceinline__ void finish_row_warp(CtaSmem& s, RowSlot& slot, int V, int k, RowOut& out) {
    const int lane = threadIdx.x & 31;
    const int kk = k < V ? k : V;
    int M = slot.cand_count;
    const uint32_t tau_key = slot.tau_key;
    double m, S;
    if (tau_key <= kOrdNegInf || M > kCandCap) {
        row_exact_warp(s, slot, slot.desc.row, V, kk, m, S);
        M = slot.cand_count;
    } else {
        unsigned long long best = 0ull;
        for (int c = lane; c < M; c += 32) best = max(best, slot.cand[c]);
        best = warp_max_u64(best);
        m = (double)cand_logit(best);
        unsigned long long fx = 0ull;
        for (int c = lane; c < M; c += 32) fx += __double2ull_rn(exp((double)cand_logit(slot.cand[c]) - m) * kFixScale);
        fx = warp_sum_u64(fx);                       // integer sum: independent of the push order
        double bulk = 0.0;
#pragma unroll
        for (int w = 0; w < kConsumerWarps; ++w) bulk += slot.warp_part[w];
        // Bulk terms are 2^(x*L32 + c_tau) with c_tau = fl(-tau*L32); wanted e^(x-m) = 2^((x-m)*L).
        // The exponent gap x*(L-L32) - m*L - c_tau is evaluated at a typical bulk logit x = tau - 2.
        const float tau = bf16_bits_to_float(ord16_inv(tau_key));
        const double c_tau = (double)(-tau * kLog2e);
        const double gap = ((double)tau - 2.0) * (kLog2eD - (double)kLog2e) - m * kLog2eD - c_tau;
        S = bulk * exp2(gap) + (double)fx / kFixScale;
    }
    // Selection by repeated warp argmax (all keys distinct).
    unsigned long long lbest = 0ull, mine = 0ull;
    int lidx = -1;
    for (int c = lane; c < M; c += 32) { const unsigned long long key = slot.cand[c]; if (key > lbest) { lbest = key; lidx = c; } }
    for (int j = 0; j < kk; ++j) {
        const unsigned long long wbest = warp_max_u64(lbest);
        if (lane == j) mine = wbest;
        if (lbest == wbest && lidx >= 0) {           // this lane owned the winner: retire it and rescan
            slot.cand[lidx] = 0ull;
            lbest = 0ull; lidx = -1;
            for (int c = lane; c < M; c += 32) { const unsigned long long key = slot.cand[c]; if (key > lbest) { lbest = key; lidx = c; } }
        }
    }
    out.kk = kk;
    out.tok = -1;
    out.p = 0.0;
    if (lane < kk) {
        out.tok = (int32_t)cand_token(mine);
        out.p = exp((double)cand_logit(mine) - m) / S;
    }
}

}  // namespace ot
