// K1: fused row softmax + top-k over the vocabulary (the row step of Algorithm 1: the
// children of a node are its k most probable next tokens; their probabilities feed Eq. 2).
//
// One CTA handles one bf16 row of V logits, read exactly once from global memory:
//   * the row is streamed in 16 KB chunks through a ring of shared-memory stages filled by
//     1-D bulk async copies (cp.async.bulk, completion on an mbarrier, no multicast);
//   * "sample" chunks (as many as the ring holds) are scanned twice from shared memory:
//     pass A takes per-thread maxima, whose k-th largest is a lower bound tau of the row's
//     k-th largest logit; pass B and all later chunks (single fused pass) push every logit
//     >= tau into a small candidate list and add exp of every other logit to a sum;
//   * the candidate list (>= k entries, all the large logits incl. the row maximum) is
//     ranked exactly on (bf16 bits, token id); the candidates' exponentials are evaluated in
//     fp64, the bulk in fp32 per thread with an fp64 combine.
// Rows whose candidate list overflows (heavy ties, tau = -inf, tiny V) take an exact but slow
// block-wide path that re-reads the row from global memory.
#pragma once

#include "common.cuh"

namespace ot {

constexpr int kChunkElems = 8192;                  // bf16 elements per stage (16 KB)
constexpr int kChunkVecs = kChunkElems / 8;        // 16-byte vectors per stage
constexpr int kStages = 4;                         // ring depth (64 KB)
constexpr int kCandCap = 1024;                     // candidate list capacity

constexpr float kLog2e = 1.44269504088896340736f;                 // rounds to 0x3FB8AA3B
constexpr double kLog2eD = 1.44269504088896340736;
constexpr double kFixScale = 4503599627370496.0;                  // 2^52: fixed-point scale of candidate terms

struct alignas(128) BlockSmem {
    uint16_t stage[kStages][kChunkElems];          // ring of row chunks
    unsigned long long cand[kCandCap];             // candidate keys (unordered)
    unsigned long long full_bar[kStages];          // one mbarrier per stage
    unsigned long long red_u64[kWarps];
    unsigned long long win[kMaxK];                 // winners by rank
    unsigned long long cand_sum_fixed;             // sum of candidate exponentials, 2^-52 units
    unsigned long long sel_thr;                    // radix select: running prefix / result
    double red_f64[kWarps];
    double bcast_f64[2];
    uint32_t tmax[kWarps][32];
    int hist[256];
    int red_i32[kWarps];
    int cand_count;
    int sel_need;
    int sel_bin;
    uint32_t tau_key;
    int flag;
};

// Result of one row, valid in every thread after row_softmax_topk returns.
struct RowResult {
    int kk;          // min(k, V) winners in smem.win[0..kk)
    double m;        // row maximum
    double S;        // sum_v exp(l_v - m)
};

// ---- k-th largest of one 16-bit key per thread (k <= 32) -------------------------------------
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
__device__ __forceinline__ uint32_t block_kth_largest(uint32_t key, int k, BlockSmem& s) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    s.tmax[warp][lane] = warp_sort_desc(key);
    __syncthreads();
    if (warp == 0) {
        uint32_t v[kWarps];
#pragma unroll
        for (int w = 0; w < kWarps; ++w) v[w] = s.tmax[w][lane];
#pragma unroll
        for (int step = 1; step < kWarps; step <<= 1)
#pragma unroll
            for (int w = 0; w + step < kWarps; w += 2 * step) v[w] = warp_merge_top32(v[w], v[w + step]);
        uint32_t kth = __shfl_sync(0xFFFFFFFFu, v[0], k - 1);
        if (lane == 0) s.tau_key = kth;
    }
    __syncthreads();
    return s.tau_key;
}

// ---- chunk geometry ---------------------------------------------------------------------------
__device__ __forceinline__ int chunk_elems(int V, int c) {
    int rem = V - c * kChunkElems;
    return rem < kChunkElems ? rem : kChunkElems;
}

// Fills stage `st` with chunk c of the row.  aligned: one thread issues a bulk async copy that
// completes on full_bar[st]; otherwise all threads copy element-wise, pad the last vector with
// -inf and synchronise.
__device__ __forceinline__ void load_chunk(BlockSmem& s, const uint16_t* row, int V, int c, int st, bool aligned) {
    const int ne = chunk_elems(V, c);
    if (aligned) {
        if (threadIdx.x == 0) {
            mbar_expect_tx(&s.full_bar[st], (uint32_t)ne * 2u);
            bulk_load(&s.stage[st][0], row + (size_t)c * kChunkElems, (uint32_t)ne * 2u, &s.full_bar[st]);
        }
    } else {
        const int padded = (ne + 7) & ~7;
        for (int e = threadIdx.x; e < padded; e += kThreads)
            s.stage[st][e] = e < ne ? __ldg(row + (size_t)c * kChunkElems + e) : (uint16_t)0xFF80u;
        __syncthreads();
    }
}

// ---- one 16-byte vector of pass B / the fused pass ---------------------------------------------
__device__ __forceinline__ void push_cand(BlockSmem& s, uint32_t bits, uint32_t token) {
    int pos = atomicAdd(&s.cand_count, 1);
    if (pos < kCandCap) s.cand[pos] = cand_key(bits, token);
}

__device__ __forceinline__ float accumulate_vec(BlockSmem& s, uint4 w, uint32_t token0, float tau, float c_tau) {
    const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
    float x[8], e[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        x[2 * i] = __uint_as_float(ww[i] << 16);
        x[2 * i + 1] = __uint_as_float(ww[i] & 0xFFFF0000u);
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float a0, a1;
        fma2(a0, a1, x[2 * i], x[2 * i + 1], kLog2e, c_tau);      // (x - tau) * log2(e), c_tau = -tau*log2(e)
        e[2 * i] = ex2_approx(a0);
        e[2 * i + 1] = ex2_approx(a1);
    }
    const float mx = max3(max3(x[0], x[1], x[2]), max3(x[3], x[4], x[5]), fmaxf(x[6], x[7]));
    if (mx >= tau) {                                               // rare: this vector holds a candidate
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            if (x[i] >= tau) {
                push_cand(s, (i & 1) ? (ww[i >> 1] >> 16) : (ww[i >> 1] & 0xFFFFu), token0 + i);
                e[i] = 0.0f;
            }
        }
    }
    float s0, s1, s2, s3;
    add2(s0, s1, e[0], e[1], e[2], e[3]);
    add2(s2, s3, e[4], e[5], e[6], e[7]);
    add2(s0, s1, s0, s1, s2, s3);
    return s0 + s1;
}

// ---- exact slow path: whole block, row re-read from global, any alignment ---------------------
__device__ void row_exact_slow(BlockSmem& s, const uint16_t* row, int V, int kk, RowResult& res) {
    const int tid = threadIdx.x;
    // row maximum
    uint32_t mk = 0;
    for (int v = tid; v < V; v += kThreads) mk = max(mk, ord16(__ldg(row + v)));
    mk = (uint32_t)block_max_u64(mk, s.red_u64);
    const double m = (double)bf16_bits_to_float(ord16_inv(mk));
    // kk-th largest 16-bit key: two 8-bit radix passes
    uint32_t prefix = 0, pmask = 0;
    int need = kk;
    for (int pass = 1; pass >= 0; --pass) {
        s.hist[tid] = 0;
        __syncthreads();
        for (int v = tid; v < V; v += kThreads) {
            uint32_t key = ord16(__ldg(row + v));
            if ((key & pmask) == prefix) atomicAdd(&s.hist[(key >> (8 * pass)) & 255u], 1);
        }
        __syncthreads();
        if (tid == 0) {
            int b = 255, above = 0;
            while (b > 0 && above + s.hist[b] < need) { above += s.hist[b]; --b; }
            s.sel_bin = b;
            s.sel_need = need - above;
        }
        __syncthreads();
        prefix |= (uint32_t)s.sel_bin << (8 * pass);
        pmask |= 0xFFu << (8 * pass);
        need = s.sel_need;
        __syncthreads();
    }
    const uint32_t thr = prefix;                  // kk-th largest key; take `need` of its copies, lowest tokens first
    if (tid == 0) s.cand_count = 0;
    __syncthreads();
    int eq_base = 0;
    double acc = 0.0;
    for (int v0 = 0; v0 < V; v0 += kThreads) {
        const int v = v0 + tid;
        uint32_t bits = 0xFF80u, key = 0;
        bool valid = v < V;
        if (valid) { bits = __ldg(row + v); key = ord16(bits); }
        const bool eq = valid && key == thr;
        int tot;
        const int eq_rank = eq_base + block_excl_scan(eq ? 1 : 0, s.red_i32, tot);
        eq_base += tot;
        if (valid && (key > thr || (eq && eq_rank < need))) push_cand(s, bits, (uint32_t)v);
        if (valid) acc += exp((double)bf16_bits_to_float(bits) - m);
    }
    res.kk = kk;
    res.m = m;
    res.S = block_sum(acc, s.red_f64);            // includes a trailing barrier pair
}

// ---- the row step ------------------------------------------------------------------------------
// All kThreads threads call.  `parity` holds one phase bit per stage and persists across rows
// handled by the same CTA.  Returns false if a bounded wait expired (status word set).
// On success smem.win[0..kk) hold the winners' keys in rank order.
__device__ bool row_softmax_topk(BlockSmem& s, const uint16_t* row, int V, int k, bool aligned,
                                 uint32_t& parity, int* status, RowResult& res) {
    const int tid = threadIdx.x;
    const int kk = k < V ? k : V;
    const int nchunks = (V + kChunkElems - 1) / kChunkElems;
    const int ns = nchunks < kStages ? nchunks : kStages;
    bool slow = false;

    if (tid == 0) { s.cand_count = 0; s.cand_sum_fixed = 0ull; }
    for (int c = 0; c < ns; ++c) load_chunk(s, row, V, c, c, aligned);

    // Pass A over the sample chunks: per-thread maximum (packed bf16 max).
    uint32_t pm = 0xFF80FF80u;
    for (int c = 0; c < ns; ++c) {
        if (aligned) {
            if (!mbar_wait(&s.full_bar[c], (parity >> c) & 1u, status)) return false;
            parity ^= 1u << c;
        }
        const int nv = (chunk_elems(V, c) + 7) >> 3;
        const uint4* vec = reinterpret_cast<const uint4*>(&s.stage[c][0]);
        for (int v = tid; v < nv; v += kThreads) {
            uint4 w = vec[v];
            pm = max_bf16x2(max_bf16x2(pm, w.x), max_bf16x2(w.y, max_bf16x2(w.z, w.w)));
        }
    }
    const uint32_t tkey = max(ord16(pm & 0xFFFFu), ord16(pm >> 16));
    const uint32_t tau_key = block_kth_largest(tkey, kk, s);
    if (tau_key <= kOrdNegInf) slow = true;        // fewer than kk threads saw a finite value

    double acc = 0.0;
    if (!slow) {
        const float tau = bf16_bits_to_float(ord16_inv(tau_key));
        const float c_tau = -tau * kLog2e;
        for (int c = 0; c < nchunks; ++c) {
            const int st = c % kStages;
            if (c >= ns) {
                if (aligned) {
                    if (!mbar_wait(&s.full_bar[st], (parity >> st) & 1u, status)) return false;
                    parity ^= 1u << st;
                }
            }
            const int nv = (chunk_elems(V, c) + 7) >> 3;
            const uint4* vec = reinterpret_cast<const uint4*>(&s.stage[st][0]);
            float part = 0.0f;
            for (int v = tid; v < nv; v += kThreads)
                part += accumulate_vec(s, vec[v], (uint32_t)(c * kChunkElems + v * 8), tau, c_tau);
            acc += (double)part;
            if (c + kStages < nchunks) {           // hand the stage back and prefetch
                __syncthreads();
                load_chunk(s, row, V, c + kStages, st, aligned);
            }
        }
        __syncthreads();
        if (s.cand_count > kCandCap) slow = true;
    }

    if (slow) {
        __syncthreads();
        row_exact_slow(s, row, V, kk, res);
    } else {
        const int M = s.cand_count;
        unsigned long long best = 0ull;
        for (int c = tid; c < M; c += kThreads) best = max(best, s.cand[c]);
        best = block_max_u64(best, s.red_u64);
        const float mf = cand_logit(best);
        const double m = (double)mf;
        for (int c = tid; c < M; c += kThreads) {
            double e = exp((double)cand_logit(s.cand[c]) - m);
            atomicAdd(&s.cand_sum_fixed, __double2ull_rn(e * kFixScale));
        }
        const double bulk = block_sum(acc, s.red_f64);              // barrier inside also publishes cand_sum_fixed
        if (tid == 0) {
            // bulk terms are 2^(x*L32 + c_tau); wanted e^(x-m) = 2^((x-m)*L).  The exponent gap is
            // x*(L-L32) - m*L - c_tau, evaluated at a typical bulk logit x = tau - 2.
            const float tau = bf16_bits_to_float(ord16_inv(tau_key));
            const double c_tau = (double)(-tau * kLog2e);
            const double gap = ((double)tau - 2.0) * (kLog2eD - (double)kLog2e) - m * kLog2eD - c_tau;
            s.bcast_f64[0] = bulk * exp2(gap) + (double)s.cand_sum_fixed / kFixScale;
        }
        __syncthreads();
        res.kk = kk;
        res.m = m;
        res.S = s.bcast_f64[0];
    }

    // Rank the candidates (all keys distinct): winners are those beaten by fewer than kk others.
    {
        const int M = s.cand_count < kCandCap ? s.cand_count : kCandCap;
        for (int c = tid; c < M; c += kThreads) {
            const unsigned long long key = s.cand[c];
            int r = 0;
            for (int j = 0; j < M; ++j) r += s.cand[j] > key;
            if (r < kk) s.win[r] = key;
        }
    }
    __syncthreads();
    return true;
}

}  // namespace ot
