// K2 / K3: layer selection (the n candidates of largest path value), running E_sub(T, n),
// the loop test of Algorithm 1, and the scan-based tree packer.  All block-wide (kThreads).
//
// Selection never sorts: an 8-pass radix select on the 64-bit keys finds the threshold of the
// "need" largest, then an ordered compaction (block scans) emits the kept elements in index
// order, which is exactly the storage order the method wants (candidate-index order for a layer,
// (depth, slot) order for the running top-n, which is also the packed order of the final tree).
#pragma once

#include "row_topk.cuh"

namespace ot {

// Positive doubles order like their bit patterns; +1 keeps every valid key above the "invalid" key 0.
__device__ __forceinline__ unsigned long long phat_key(double p) { return (unsigned long long)__double_as_longlong(p) + 1ull; }

// Threshold of the `need` largest keys among keyf(0..N).  On return thr is that key and need_eq
// how many of the elements equal to thr belong to the selection (lowest indices first).
// Requires 1 <= need <= number of non-zero keys.
template <class KeyFn>
__device__ void radix_select(KeyFn keyf, int N, int need, BlockSmem& s, unsigned long long& thr, int& need_eq) {
    const int tid = threadIdx.x;
    unsigned long long prefix = 0ull, pmask = 0ull;
    for (int pass = 7; pass >= 0; --pass) {
        s.hist[tid] = 0;
        __syncthreads();
        for (int i = tid; i < N; i += kThreads) {
            const unsigned long long key = keyf(i);
            if ((key & pmask) == prefix) atomicAdd(&s.hist[(int)((key >> (8 * pass)) & 255ull)], 1);
        }
        __syncthreads();
        if (tid < 32) {
            // lane L owns bins [8L, 8L+8); suffix sums over lanes from the top
            int c[8], mine = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) { c[j] = s.hist[8 * tid + j]; mine += c[j]; }
            int incl = mine;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                int u = __shfl_down_sync(0xFFFFFFFFu, incl, o);
                if (tid + o < 32) incl += u;
            }
            const int above = incl - mine;                 // elements in higher lanes' bins
            if (above < need && need <= incl) {
                int a = above, b = 7;
                while (b > 0 && a + c[b] < need) { a += c[b]; --b; }
                s.sel_bin = 8 * tid + b;
                s.sel_need = need - a;
            }
        }
        __syncthreads();
        prefix |= (unsigned long long)s.sel_bin << (8 * pass);
        pmask |= 0xFFull << (8 * pass);
        need = s.sel_need;
    }
    thr = prefix;
    need_eq = need;
}

// Emits, in index order, the elements with key > thr and the first need_eq with key == thr.
// emit(pos, i) is called once per kept element; returns the number kept.
template <class KeyFn, class EmitFn>
__device__ int compact_selected(KeyFn keyf, int N, unsigned long long thr, int need_eq, BlockSmem& s, EmitFn emit) {
    const int tid = threadIdx.x;
    int eq_base = 0, take_base = 0;
    for (int i0 = 0; i0 < N; i0 += kThreads) {
        const int i = i0 + tid;
        const unsigned long long key = i < N ? keyf(i) : 0ull;
        const bool eq = i < N && key == thr;
        int tot;
        const int eq_rank = eq_base + block_excl_scan(eq ? 1 : 0, s.red_i32, tot);
        eq_base += tot;
        const bool take = i < N && (key > thr || (eq && eq_rank < need_eq));
        const int pos = take_base + block_excl_scan(take ? 1 : 0, s.red_i32, tot);
        take_base += tot;
        if (take) emit(pos, i);
    }
    return take_base;
}

// Per-sequence state and arrays in the workspace (device pointers already offset to the sequence).
struct SeqWork {
    double* cand_phat;     // [n*k]    path values of this round's candidates (Eq. 2), slot-major
    int32_t* cand_tok;     // [n*k]
    int32_t* T_tok;        // [D*n]    drafted nodes, gid = (depth-1)*n + slot
    int32_t* T_par;        // [D*n]    slot of the parent in the previous layer
    double* T_phat;        // [D*n]
    int32_t* R;            // [2][n]   running top-n as gids in ascending order, double-buffered by layer parity
    double* E_prev;        // [1]      E of Algorithm 1
    int32_t* st;           // [8]      0: frontier size, 1: active, 2: rows done this round, 3: |R|, 4: layers drafted
};
enum { kStFsize = 0, kStActive = 1, kStDone = 2, kStNR = 3, kStDepth = 4 };

struct TreeOut {           // mirrors opt_tree_out, pointers offset to the sequence
    int32_t *token, *parent, *depth;
    double* phat;
    int32_t *n_sel, *depth_reached;
    double* expected_len;
    double* esub_trace;    // may be null
};

// After all rows of layer d (1-based) of one sequence are expanded: choose the layer, update the
// running top-n and E_sub, apply the loop test, and pack the tree if the sequence is finished.
// Returns true if the sequence continues with layer d+1.
__device__ bool finish_layer(BlockSmem& s, const SeqWork& w, const TreeOut& out, int d, int n, int k, int kk,
                             int Dcap, int max_depth, float delta) {
    const int tid = threadIdx.x;
    const int fsize = __ldcg(&w.st[kStFsize]);
    const int nR_old = __ldcg(&w.st[kStNR]);
    const int N = fsize * k;
    const int nvalid = fsize * kk;
    const int nl = nvalid < n ? nvalid : n;
    const int gid0 = (d - 1) * n;

    // --- next layer: the nl candidates of largest path value, stored in candidate-index order ---
    auto ckey = [&](int i) -> unsigned long long {
        return (i % k) < kk ? phat_key(__ldcg(&w.cand_phat[i])) : 0ull;
    };
    unsigned long long thr; int need_eq;
    radix_select(ckey, N, nl, s, thr, need_eq);
    compact_selected(ckey, N, thr, need_eq, s, [&](int pos, int i) {
        w.T_tok[gid0 + pos] = __ldcg(&w.cand_tok[i]);
        w.T_par[gid0 + pos] = i / k;
        w.T_phat[gid0 + pos] = __ldcg(&w.cand_phat[i]);
    });
    __syncthreads();

    // --- E_sub(T, n): the n largest path values among the previous top-n and the new layer ---
    const int32_t* Rold = w.R + ((d - 1) & 1) * n;
    int32_t* Rnew = w.R + (d & 1) * n;
    const int NR = nR_old + nl;
    const int nR = NR < n ? NR : n;
    auto gid_of = [&](int i) -> int { return i < nR_old ? __ldcg(&Rold[i]) : gid0 + (i - nR_old); };
    auto rkey = [&](int i) -> unsigned long long { return phat_key(__ldcg(&w.T_phat[gid_of(i)])); };
    radix_select(rkey, NR, nR, s, thr, need_eq);
    compact_selected(rkey, NR, thr, need_eq, s, [&](int pos, int i) { Rnew[pos] = gid_of(i); });
    __syncthreads();
    double part = 0.0;
    for (int i = tid; i < nR; i += kThreads) part += __ldcg(&w.T_phat[__ldcg(&Rnew[i])]);
    const double esub = block_sum(part, s.red_f64);
    const double eprev = __ldcg(w.E_prev);
    const bool more = d < Dcap && (esub - eprev > (double)delta);
    if (out.esub_trace && tid == 0) out.esub_trace[d - 1] = esub;

    if (tid == 0) {
        w.st[kStFsize] = nl;
        w.st[kStNR] = nR;
        w.st[kStDone] = 0;
        w.st[kStDepth] = d;
        w.st[kStActive] = more ? 1 : 0;
        *w.E_prev = esub;
    }
    if (!more) {
        // --- pack: T_opt = the running top-n, already in (depth, parent's index, sibling rank) order ---
        if (out.esub_trace) for (int i = d + tid; i < max_depth; i += kThreads) out.esub_trace[i] = 0.0;
        for (int i = tid; i < n; i += kThreads) {
            int32_t tok = -1, par = -1, dep = 0;
            double ph = 0.0;
            if (i < nR) {
                const int gid = __ldcg(&Rnew[i]);
                dep = gid / n + 1;
                tok = __ldcg(&w.T_tok[gid]);
                ph = __ldcg(&w.T_phat[gid]);
                if (dep > 1) {
                    const int pg = (dep - 2) * n + __ldcg(&w.T_par[gid]);
                    int lo = 0, hi = i;                          // the parent is packed before its child
                    while (lo < hi) {
                        const int mid = (lo + hi) >> 1;
                        if (__ldcg(&Rnew[mid]) < pg) lo = mid + 1; else hi = mid;
                    }
                    par = lo;
                }
            }
            out.token[i] = tok; out.parent[i] = par; out.depth[i] = dep; out.phat[i] = ph;
        }
        if (tid == 0) { *out.n_sel = nR; *out.depth_reached = d; *out.expected_len = esub; }
    }
    __syncthreads();
    return more;
}

}  // namespace ot
