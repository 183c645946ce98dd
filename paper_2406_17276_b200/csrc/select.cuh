// K2 / K3: layer selection (the n candidates of largest path value) by the layer team, running
// E_sub(T, n), the loop test of Algorithm 1 and the scan-based tree packer by the layer warp.
//
// Selection never sorts: an 8-pass radix select on the 64-bit keys finds the threshold of the
// "need" largest, then an ordered compaction (ballot scans) emits the kept elements in index
// order, which is exactly the storage order the method wants (candidate-index order for a layer;
// (depth, slot) order for the running top-n, which is also the packed order of the final tree).
#pragma once

#include "row_topk.cuh"

namespace ot {

// Positive doubles order like their bit patterns; +1 keeps every valid key above the "invalid" key 0.
__device__ __forceinline__ unsigned long long phat_key(double p) { return (unsigned long long)__double_as_longlong(p) + 1ull; }

__device__ __forceinline__ unsigned long long warp_or_u64(unsigned long long v) {
    const uint32_t lo = __reduce_or_sync(0xFFFFFFFFu, (uint32_t)v), hi = __reduce_or_sync(0xFFFFFFFFu, (uint32_t)(v >> 32));
    return ((unsigned long long)hi << 32) | lo;
}
__device__ __forceinline__ unsigned long long warp_and_u64(unsigned long long v) {
    const uint32_t lo = __reduce_and_sync(0xFFFFFFFFu, (uint32_t)v), hi = __reduce_and_sync(0xFFFFFFFFu, (uint32_t)(v >> 32));
    return ((unsigned long long)hi << 32) | lo;
}

// Threshold of the `need` largest keys among keyf(0..N); key 0 means "not an element".
// key_or / key_and are the bitwise OR / AND over all non-zero keys (the caller folds them into the
// sweep that stages the keys): the bits on which all keys agree need no pass, and a pass whose
// threshold bin holds exactly the elements still needed ends the search.  On return the selection
// is {key > thr} plus the first need_eq elements (lowest indices) with key == thr.
// Requires 1 <= need <= number of non-zero keys.  Whole warp; hist has 256 ints.
template <class KeyFn>
__device__ void warp_radix_select(KeyFn keyf, int N, int need, int* hist, unsigned long long key_or,
                                  unsigned long long key_and, unsigned long long& thr, int& need_eq) {
    const int lane = threadIdx.x & 31;
    const unsigned long long diff = key_or ^ key_and;
    if (diff == 0ull) { thr = key_or; need_eq = need; return; }          // all elements equal
    int top = 64 - __clzll((long long)diff);                             // the low `top` bits vary
    unsigned long long prefix = top == 64 ? 0ull : ((key_or >> top) << top);
    while (top > 0) {
        const int wbits = top < 8 ? top : 8, shift = top - wbits;
        const unsigned int dmask = (1u << wbits) - 1u;
#pragma unroll
        for (int j = 0; j < 8; ++j) hist[lane * 8 + j] = 0;
        __syncwarp();
        #pragma unroll 1
        for (int i = lane; i < N; i += 32) {
            const unsigned long long key = keyf(i);
            const bool match = key != 0ull && (top == 64 || (key >> top) == (prefix >> top));
            if (match) atomicAdd(&hist[(int)((unsigned int)(key >> shift) & dmask)], 1);
        }
        __syncwarp();
        int c[8], mine = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) { c[j] = hist[lane * 8 + j]; mine += c[j]; }
        int incl = mine;                                   // suffix sums over lanes from the top
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int u = __shfl_down_sync(0xFFFFFFFFu, incl, o);
            if (lane + o < 32) incl += u;
        }
        const int above = incl - mine;
        const bool here = above < need && need <= incl;
        int bin = 0, nd = 0, cb = 0;
        if (here) {
            int a = above;
            bin = lane * 8;
#pragma unroll
            for (int b = 7; b >= 0; --b) {                 // highest bin whose suffix count reaches need
                if (nd == 0) {
                    if (a + c[b] >= need) { bin = lane * 8 + b; nd = need - a; cb = c[b]; }
                    else a += c[b];
                }
            }
        }
        const int src = __ffs(__ballot_sync(0xFFFFFFFFu, here)) - 1;
        bin = __shfl_sync(0xFFFFFFFFu, bin, src);
        need = __shfl_sync(0xFFFFFFFFu, nd, src);
        cb = __shfl_sync(0xFFFFFFFFu, cb, src);
        prefix |= (unsigned long long)bin << shift;
        top = shift;
        __syncwarp();
        if (cb == need && prefix != 0ull) { thr = prefix - 1ull; need_eq = 0; return; }   // the whole bin belongs
    }
    thr = prefix;
    need_eq = need;
}

// Emits, in index order, the elements with key > thr and the first need_eq with key == thr.
// emit(pos, i) is called once per kept element; returns the number kept.  Whole warp.
template <class KeyFn, class EmitFn>
__device__ int warp_compact_selected(KeyFn keyf, int N, unsigned long long thr, int need_eq, EmitFn emit) {
    const int lane = threadIdx.x & 31;
    const unsigned below = (1u << lane) - 1u;
    int eq_seen = 0, taken = 0;
    #pragma unroll 1
    for (int i0 = 0; i0 < N; i0 += 32) {
        const int i = i0 + lane;
        const unsigned long long key = i < N ? keyf(i) : 0ull;
        const bool eq = i < N && key == thr;
        const unsigned eqm = __ballot_sync(0xFFFFFFFFu, eq);
        const bool take = i < N && (key > thr || (eq && eq_seen + __popc(eqm & below) < need_eq));
        const unsigned tm = __ballot_sync(0xFFFFFFFFu, take);
        if (take) emit(taken + __popc(tm & below), i);
        eq_seen += __popc(eqm);
        taken += __popc(tm);
    }
    return taken;
}

// Per-sequence state and arrays in the workspace (device pointers already offset to the sequence).
struct SeqWork {
    double* cand_phat;     // [n*k, padded to a multiple of 4, 16-byte aligned]  path values of this layer's candidates (Eq. 2), slot-major
    int32_t* cand_tok;     // [n*k]
    int32_t* T_tok;        // [D*n]    drafted nodes, gid = (depth-1)*n + slot
    int32_t* T_par;        // [D*n]    slot of the parent in the previous layer
    double* T_phat;        // [D*n]
    int32_t* R;            // [2][n]   running top-n as gids in ascending order, double-buffered by layer parity
    double* E_prev;        // [1]      E of Algorithm 1
    int32_t* st;           // [8]      1: rows finished since the build began, 2: |R|, 3: rows sent out in all
    int32_t* fmap;         // [n]      pruned draft: layer slot of the node behind each frontier row
};
enum { kStDone = 1, kStNR = 2, kStRows = 3, kStDepth = 4, kStFsize = 5, kStL1 = 6 };   // 4, 5: layer-by-layer build: layer awaited (0: finished), its rows
// 6: how the root's row was handled (top bit: decided; the rest: rows of layer 2 if its finisher grew layer 1 itself, else 0)

struct TreeOut {           // mirrors opt_tree_out, pointers offset to the sequence
    int32_t *token, *parent, *depth;
    double* phat;
    int32_t *n_sel, *depth_reached;
    double* expected_len;
    double* esub_trace;    // may be null
};

// Starts the asynchronous copies of a layer's candidates (path values and tokens) into the layer
// warp's scratch; the layer warp waits for them before it starts the team.  Separate so that other round trips (the
// mailbox reservations) can be in flight at the same time.
template <class LS>
__device__ __forceinline__ void stage_layer_candidates(LS& s, const SeqWork& w, int fsize, int k, int off = 0) {
    const int lane = threadIdx.x & 31;
    const int N = fsize * k;
    if (off + N > kStageCap) return;                       // (off is even: the copies keep their 16-byte alignment)
    const unsigned long long* gph = reinterpret_cast<const unsigned long long*>(w.cand_phat);
    const unsigned int* gtk = reinterpret_cast<const unsigned int*>(w.cand_tok);
    #pragma unroll 1
    for (int i = lane * 2; i < N; i += 64) cp_async_16(&s.keys[off + i], &gph[i]);
    #pragma unroll 1
    for (int i = lane * 4; i < N; i += 128) cp_async_16(&s.toks[i], &gtk[i]);
}

// A candidate word that was not there yet when it was looked at is read again until it is (bounded).
// Rare, so out of line.
__device__ __noinline__ unsigned long long poll_phat_word(const unsigned long long* p, int* status, int polls = kWaitPolls) {
    unsigned long long x = ld_relaxed_u64(p);
    for (int t = 0; !(x >> 63) && t < polls; ++t) x = ld_relaxed_u64(p);
    if (!(x >> 63)) { set_status(status, kErrTimeout); x = ~0ull; }
    return x;
}
__device__ __noinline__ unsigned int poll_tok_word(const unsigned int* p, int* status, int polls = kWaitPolls) {
    unsigned int x = ld_relaxed_u32(p);
    for (int t = 0; !(x >> 31) && t < polls; ++t) x = ld_relaxed_u32(p);
    if (!(x >> 31)) { set_status(status, kErrTimeout); x = ~0u; }
    return x;
}

// ------------------------------------------------------------------------------------------------
// The same layer selection by the layer team (kTeam threads: the layer warp and its assistants;
// thread tt of the team).  Every step that loops over the candidates is split over the team;
// the decisions in between are computed by each warp for itself from the same shared-memory
// counts, so all warps take the same path and meet at the same barriers.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ int team_excl_scan(int v, int* wtot, int tw, int& total) {
    int wt;
    const int base = warp_excl_scan(v, wt);
    if ((threadIdx.x & 31) == 0) wtot[tw] = wt;
    team_sync();
    int before = 0;
    total = 0;
#pragma unroll
    for (int q = 0; q < kTeamWarps; ++q) { const int x = wtot[q]; total += x; before += q < tw ? x : 0; }
    return base + before;
}

// Threshold of the `need` largest keys among s.keys[0..N) (0 = not an element); see
// warp_radix_select for the result and the shortcuts.  The digit counts rotate through three
// arrays that are all zero on entry: pass p counts into array p % 3 and clears the one pass p-1
// read, so one barrier per pass is enough.  Returns the array that is left non-zero (the caller
// clears it after its next barrier), or -1.
// kGlobal: the keys are not staged; they are read from the candidate words gw[0..N) in global memory
// (all written: the caller has looked at every one), eight loads in flight per thread.
__device__ __forceinline__ unsigned long long key_of_word(unsigned long long x) {
    return x == ~0ull ? 0ull : (x & 0x7FFFFFFFFFFFFFFFull) + 1ull;
}
template <bool kGlobal, class LS>
__device__ int team_radix_select(LS& s, const unsigned long long* gw, int N, int need, int tt, unsigned long long key_or,
                                 unsigned long long key_and, unsigned long long& thr, int& need_eq) {
    const int lane = threadIdx.x & 31;
    const unsigned long long diff = key_or ^ key_and;
    if (diff == 0ull) { thr = key_or; need_eq = need; return -1; }       // all elements equal
    int top = 64 - __clzll((long long)diff);                             // the low `top` bits vary
    unsigned long long prefix = top == 64 ? 0ull : ((key_or >> top) << top);
    int pass = 0;
    while (top > 0) {
        const int wbits = top < 8 ? top : 8, shift = top - wbits;
        const unsigned int dmask = (1u << wbits) - 1u;
        int* hist = s.thist[pass % 3];
        if (!kGlobal) {
            #pragma unroll 1
            for (int i = tt; i < N; i += kTeam) {
                const unsigned long long key = s.keys[i];
                const bool match = key != 0ull && (top == 64 || (key >> top) == (prefix >> top));
                if (match) atomicAdd(&hist[(int)((unsigned int)(key >> shift) & dmask)], 1);
            }
        } else {
            #pragma unroll 1
            for (int i0 = tt; i0 < N; i0 += 8 * kTeam) {
                unsigned long long x[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) x[u] = i0 + u * kTeam < N ? ld_relaxed_u64(&gw[i0 + u * kTeam]) : ~0ull;
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const unsigned long long key = key_of_word(x[u]);
                    const bool match = key != 0ull && (top == 64 || (key >> top) == (prefix >> top));
                    if (match) atomicAdd(&hist[(int)((unsigned int)(key >> shift) & dmask)], 1);
                }
            }
        }
        team_sync();
        int c[8], mine = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) { c[j] = hist[lane * 8 + j]; mine += c[j]; }
        {   // the array read one pass ago is free again
            int* z = s.thist[(pass + 2) % 3];
            z[tt] = 0; z[tt + kTeam] = 0;
        }
        int incl = mine;                                   // suffix sums over lanes from the top
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int u = __shfl_down_sync(0xFFFFFFFFu, incl, o);
            if (lane + o < 32) incl += u;
        }
        const int above = incl - mine;
        const bool here = above < need && need <= incl;
        int bin = 0, nd = 0, cb = 0;
        if (here) {
            int a = above;
            bin = lane * 8;
#pragma unroll
            for (int b = 7; b >= 0; --b) {                 // highest bin whose suffix count reaches need
                if (nd == 0) {
                    if (a + c[b] >= need) { bin = lane * 8 + b; nd = need - a; cb = c[b]; }
                    else a += c[b];
                }
            }
        }
        const int src = __ffs(__ballot_sync(0xFFFFFFFFu, here)) - 1;
        bin = __shfl_sync(0xFFFFFFFFu, bin, src);
        need = __shfl_sync(0xFFFFFFFFu, nd, src);
        cb = __shfl_sync(0xFFFFFFFFu, cb, src);
        prefix |= (unsigned long long)bin << shift;
        top = shift;
        ++pass;
        if (cb == need && prefix != 0ull) { thr = prefix - 1ull; need_eq = 0; return (pass - 1) % 3; }   // the whole bin belongs
    }
    thr = prefix;
    need_eq = need;
    return (pass - 1) % 3;
}

// The team's part of a layer selection (N = fsize * k <= 1024; the candidates were staged into s
// by the layer warp).  On return (after a last barrier) the new layer's nodes are in T and its
// tokens and keys in s.ltok / s.lkeys.  Returns nl.
template <bool kPrune, class LS>
__device__ __noinline__ int select_layer_team(LS& s, const LayerJob& j, int tt, int* status) {
    const int lane = threadIdx.x & 31, tw = tt >> 5;
    const int N = j.fsize * j.k;
    const int nvalid = j.fsize * j.kk;
    const int nl = nvalid < j.n ? nvalid : j.n;
    const int gid0 = (j.d - 1) * j.n;
    const unsigned long long* gph = reinterpret_cast<const unsigned long long*>(j.cand_phat);
    const unsigned int* gtk = reinterpret_cast<const unsigned int*>(j.cand_tok);
    unsigned long long ko = 0ull, ka = ~0ull;
    #pragma unroll 1
    for (int i = tt; i < N; i += kTeam) {
        // words that were not there yet when they were staged are read again until they are (bounded)
        unsigned long long x = s.keys[i];
        if (!(x >> 63)) x = poll_phat_word(&gph[i], status);
        const unsigned long long key = x == ~0ull ? 0ull : (x & 0x7FFFFFFFFFFFFFFFull) + 1ull;
        s.keys[i] = key;
        if (key) { ko |= key; ka &= key; }
        unsigned int t32 = (unsigned int)s.toks[i];
        if (!(t32 >> 31)) { t32 = poll_tok_word(&gtk[i], status); s.toks[i] = (int)t32; }
    }
    ko = warp_or_u64(ko); ka = warp_and_u64(ka);
    if (lane == 0) { s.red_or[tw] = ko; s.red_and[tw] = ka; }
    team_sync();
    ko = 0ull; ka = ~0ull;
#pragma unroll
    for (int q = 0; q < kTeamWarps; ++q) { ko |= s.red_or[q]; ka &= s.red_and[q]; }
    // every candidate has been read: the arrays are free for the next layer's rows once they are zero again
    #pragma unroll 1
    for (int i = tt * 2; i < N; i += 2 * kTeam) *reinterpret_cast<uint4*>(&j.cand_phat[i]) = make_uint4(0, 0, 0, 0);
    #pragma unroll 1
    for (int i = tt * 4; i < N; i += 4 * kTeam) *reinterpret_cast<uint4*>(&j.cand_tok[i]) = make_uint4(0, 0, 0, 0);
    unsigned long long thr = 0ull;                         // with no more candidates than wanted, all of them (key > 0) are taken
    int need_eq = 0, dirty = -1;
    if (nl < nvalid) dirty = team_radix_select<false>(s, nullptr, N, nl, tt, ko, ka, thr, need_eq);
    // ordered compaction: thread tt owns a contiguous stretch of candidates
    const int per = (N + kTeam - 1) / kTeam;
    const int lo = min(tt * per, N), hi = min(lo + per, N);
    int gt = 0, eq = 0;
    #pragma unroll 1
    for (int i = lo; i < hi; ++i) {
        const unsigned long long key = s.keys[i];
        gt += key > thr ? 1 : 0;
        eq += key == thr ? 1 : 0;
    }
    int total_eq, total;
    int eq_take = 0;
    if (need_eq > 0) {                                     // (the same for all warps) ties at the threshold: lowest indices first
        const int eq_before = team_excl_scan(eq, s.scan_a, tw, total_eq);
        eq_take = need_eq - eq_before;
        eq_take = eq_take < 0 ? 0 : (eq_take > eq ? eq : eq_take);
    }
    int pos = team_excl_scan(gt + eq_take, s.scan_b, tw, total);
    if (dirty >= 0) { s.thist[dirty][tt] = 0; s.thist[dirty][tt + kTeam] = 0; }     // everyone is past the last pass
    int frow = lo / j.k, frank = lo - frow * j.k;          // frontier row and sibling rank of candidate i, carried along
    #pragma unroll 1
    for (int i = lo; i < hi; ++i) {
        const unsigned long long key = s.keys[i];
        bool take = key > thr;
        if (key == thr && eq_take > 0) { take = true; --eq_take; }
        if (take) {
            const unsigned int t32 = (unsigned int)s.toks[i];
            const int tok = t32 == ~0u ? -1 : (int)(t32 & 0x7FFFFFFFu);
            j.T_tok[gid0 + pos] = tok;
            s.ltok[pos] = tok;
            j.T_par[gid0 + pos] = kPrune ? __ldcg(&j.fmap[frow]) : frow;
            j.T_phat[gid0 + pos] = __longlong_as_double((long long)(key - 1ull));
            s.lkeys[pos] = key;
            ++pos;
        }
        if (++frank == j.k) { frank = 0; ++frow; }
    }
    if (total != nl) set_status(status, kErrInternal);
    team_sync();
    return nl;
}

// Pruned draft, both halves of a layer job in one selection: the new running top-n is the n largest
// of the old one and the layer's candidates together (what a candidate outside them could add to T
// can never matter, see opt_tree_build_pruned).  s.keys[0..nR_old) / s.gids[0..nR_old) hold the old
// top-n (keys, gids ascending), s.keys[off..off+N) the staged candidate words (entries between are 0).
// Array order is tie order (shallower first, then candidate index).  On return s.rsel / s.vals hold
// the new top-n (gids ascending; also written to j.Rnew), its new members are T's nodes
// gid0 .. gid0+cnt in candidate order with tokens and keys in s.ltok / s.lkeys, and s.scan_c sums
// to the number of old members kept.  Returns |new top-n|.
template <class LS>
__device__ __noinline__ int select_running_team(LS& s, const LayerJob& j, int tt, int* status) {
    const int lane = threadIdx.x & 31, tw = tt >> 5;
    const int N = j.fsize * j.k, nRo = j.nR_old, off = j.off, M = off + N;
    const int nvalid = j.fsize * j.kk;
    const int need = nRo + nvalid < j.n ? nRo + nvalid : j.n;
    const int gid0 = (j.d - 1) * j.n;
    const unsigned long long* gph = reinterpret_cast<const unsigned long long*>(j.cand_phat);
    const unsigned int* gtk = reinterpret_cast<const unsigned int*>(j.cand_tok);
    unsigned long long ko = 0ull, ka = ~0ull;
    #pragma unroll 1
    for (int i = tt; i < M; i += kTeam) {
        unsigned long long key;
        if (i >= off) {
            unsigned long long x = s.keys[i];
            if (!(x >> 63)) x = poll_phat_word(&gph[i - off], status);
            key = key_of_word(x);
            s.keys[i] = key;
            unsigned int t32 = (unsigned int)s.toks[i - off];
            if (!(t32 >> 31)) { t32 = poll_tok_word(&gtk[i - off], status); s.toks[i - off] = (int)t32; }
        } else {
            key = i < nRo ? s.keys[i] : 0ull;
            if (i >= nRo) s.keys[i] = 0ull;
        }
        if (key) { ko |= key; ka &= key; }
    }
    ko = warp_or_u64(ko); ka = warp_and_u64(ka);
    if (lane == 0) { s.red_or[tw] = ko; s.red_and[tw] = ka; }
    team_sync();
    ko = 0ull; ka = ~0ull;
#pragma unroll
    for (int q = 0; q < kTeamWarps; ++q) { ko |= s.red_or[q]; ka &= s.red_and[q]; }
    #pragma unroll 1
    for (int i = tt * 2; i < N; i += 2 * kTeam) *reinterpret_cast<uint4*>(&j.cand_phat[i]) = make_uint4(0, 0, 0, 0);
    #pragma unroll 1
    for (int i = tt * 4; i < N; i += 4 * kTeam) *reinterpret_cast<uint4*>(&j.cand_tok[i]) = make_uint4(0, 0, 0, 0);
    unsigned long long thr = 0ull;
    int need_eq = 0, dirty = -1;
    if (need < nRo + nvalid) dirty = team_radix_select<false>(s, nullptr, M, need, tt, ko, ka, thr, need_eq);
    const int per = (M + kTeam - 1) / kTeam;
    const int lo = min(tt * per, M), hi = min(lo + per, M);
    int gt = 0, eq = 0;
    #pragma unroll 1
    for (int i = lo; i < hi; ++i) {
        const unsigned long long key = s.keys[i];
        gt += key > thr ? 1 : 0;
        eq += (key == thr && key != 0ull) ? 1 : 0;
    }
    int total_eq, total;
    int eq_take = 0;
    if (need_eq > 0) {
        const int eq_before = team_excl_scan(eq, s.scan_a, tw, total_eq);
        eq_take = need_eq - eq_before;
        eq_take = eq_take < 0 ? 0 : (eq_take > eq ? eq : eq_take);
    }
    // old members kept: counted per thread, summed over the team along with the scan below
    int kept_mine = 0;
    {
        int e = eq_take;
        #pragma unroll 1
        for (int i = lo; i < hi && i < nRo; ++i) {
            const unsigned long long key = s.keys[i];
            bool take = key > thr;
            if (key == thr && key != 0ull && e > 0) { take = true; --e; }
            kept_mine += take ? 1 : 0;
        }
    }
    kept_mine = __reduce_add_sync(0xFFFFFFFFu, kept_mine);
    if (lane == 0) s.scan_c[tw] = kept_mine;
    int pos = team_excl_scan(gt + eq_take, s.scan_b, tw, total);       // (its barrier also publishes scan_c)
    if (dirty >= 0) { s.thist[dirty][tt] = 0; s.thist[dirty][tt + kTeam] = 0; }
    int kept_old = 0;
#pragma unroll
    for (int q = 0; q < kTeamWarps; ++q) kept_old += s.scan_c[q];
    #pragma unroll 1
    for (int i = lo; i < hi; ++i) {
        const unsigned long long key = s.keys[i];
        bool take = key > thr;
        if (key == thr && key != 0ull && eq_take > 0) { take = true; --eq_take; }
        if (!take) continue;
        int gid;
        if (i < nRo) {
            gid = s.gids[i];
        } else {
            const int c = i - off, slot = pos - kept_old;
            const unsigned int t32 = (unsigned int)s.toks[c];
            const int tok = t32 == ~0u ? -1 : (int)(t32 & 0x7FFFFFFFu);
            gid = gid0 + slot;
            j.T_tok[gid] = tok;
            j.T_par[gid] = __ldcg(&j.fmap[c / j.k]);      // layer slot of the node behind the candidate's frontier row
            j.T_phat[gid] = __longlong_as_double((long long)(key - 1ull));
            s.ltok[slot] = tok;
            s.lkeys[slot] = key;
        }
        s.rsel[pos] = gid;
        s.vals[pos] = __longlong_as_double((long long)(key - 1ull));
        j.Rnew[pos] = gid;
        ++pos;
    }
    if (total != need) set_status(status, kErrInternal);
    team_sync();
    return need;
}

// The team's selection for layers with more candidates than the shared-memory staging holds
// (1024 < N <= n*k): the same steps, but every sweep reads the candidate words from global memory
// (they sit in L2), a thread's loads eight at a time.  The candidate arrays are cleared at the end.
template <bool kPrune, class LS>
__device__ __noinline__ int select_layer_team_big(LS& s, const LayerJob& j, int tt, int* status) {
    const int lane = threadIdx.x & 31, tw = tt >> 5;
    const int N = j.fsize * j.k;
    const int nvalid = j.fsize * j.kk;
    const int nl = nvalid < j.n ? nvalid : j.n;
    const int gid0 = (j.d - 1) * j.n;
    const unsigned long long* gph = reinterpret_cast<const unsigned long long*>(j.cand_phat);
    const unsigned int* gtk = reinterpret_cast<const unsigned int*>(j.cand_tok);
    unsigned long long ko = 0ull, ka = ~0ull;
    #pragma unroll 1
    for (int i0 = tt; i0 < N; i0 += 8 * kTeam) {
        unsigned long long x[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) x[u] = i0 + u * kTeam < N ? ld_relaxed_u64(&gph[i0 + u * kTeam]) : ~0ull;
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            if (!(x[u] >> 63)) x[u] = poll_phat_word(&gph[i0 + u * kTeam], status);      // not written yet: read again
            const unsigned long long key = key_of_word(x[u]);
            if (key) { ko |= key; ka &= key; }
        }
    }
    ko = warp_or_u64(ko); ka = warp_and_u64(ka);
    if (lane == 0) { s.red_or[tw] = ko; s.red_and[tw] = ka; }
    team_sync();
    ko = 0ull; ka = ~0ull;
#pragma unroll
    for (int q = 0; q < kTeamWarps; ++q) { ko |= s.red_or[q]; ka &= s.red_and[q]; }
    unsigned long long thr = 0ull;
    int need_eq = 0, dirty = -1;
    if (nl < nvalid) dirty = team_radix_select<true>(s, gph, N, nl, tt, ko, ka, thr, need_eq);
    // ordered compaction: thread tt owns a contiguous stretch of candidates (a multiple of 8 long)
    const int per = (((N + kTeam - 1) / kTeam) + 7) & ~7;
    const int lo = min(tt * per, N), hi = min(lo + per, N);
    int gt = 0, eq = 0;
    #pragma unroll 1
    for (int i0 = lo; i0 < hi; i0 += 8) {
        unsigned long long x[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) x[u] = i0 + u < hi ? ld_relaxed_u64(&gph[i0 + u]) : ~0ull;
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const unsigned long long key = key_of_word(x[u]);
            gt += key > thr ? 1 : 0;
            eq += (key == thr && key != 0ull) ? 1 : 0;
        }
    }
    int total_eq, total;
    int eq_take = 0;
    if (need_eq > 0) {
        const int eq_before = team_excl_scan(eq, s.scan_a, tw, total_eq);
        eq_take = need_eq - eq_before;
        eq_take = eq_take < 0 ? 0 : (eq_take > eq ? eq : eq_take);
    }
    int pos = team_excl_scan(gt + eq_take, s.scan_b, tw, total);
    if (dirty >= 0) { s.thist[dirty][tt] = 0; s.thist[dirty][tt + kTeam] = 0; }
    if (gt + eq_take > 0) {
        #pragma unroll 1
        for (int i = lo; i < hi; ++i) {
            const unsigned long long key = key_of_word(ld_relaxed_u64(&gph[i]));
            bool take = key > thr;
            if (key == thr && key != 0ull && eq_take > 0) { take = true; --eq_take; }
            if (take) {
                unsigned int t32 = ld_relaxed_u32(&gtk[i]);
                if (!(t32 >> 31)) t32 = poll_tok_word(&gtk[i], status);
                const int tok = t32 == ~0u ? -1 : (int)(t32 & 0x7FFFFFFFu);
                j.T_tok[gid0 + pos] = tok;
                s.ltok[pos] = tok;
                j.T_par[gid0 + pos] = kPrune ? __ldcg(&j.fmap[i / j.k]) : i / j.k;
                j.T_phat[gid0 + pos] = __longlong_as_double((long long)(key - 1ull));
                s.lkeys[pos] = key;
                ++pos;
            }
        }
    }
    if (total != nl) set_status(status, kErrInternal);
    team_sync();                                           // everyone has read what it needs: the arrays can be cleared
    #pragma unroll 1
    for (int i = tt * 2; i < N; i += 2 * kTeam) *reinterpret_cast<uint4*>(&j.cand_phat[i]) = make_uint4(0, 0, 0, 0);
    #pragma unroll 1
    for (int i = tt * 4; i < N; i += 4 * kTeam) *reinterpret_cast<uint4*>(&j.cand_tok[i]) = make_uint4(0, 0, 0, 0);
    team_sync();
    return nl;
}

// Once per sequence, when it is finished: T_opt = the running top-n (s.rsel / s.vals, already in
// (depth, parent's index, sibling rank) order), packed with parent indices.
template <class LS>
__device__ __noinline__ void pack_tree_warp(LS& s, const SeqWork& w, const TreeOut& out, int d, int nR, int n, int max_depth,
                                            double esub, int* status) {
    const int lane = threadIdx.x & 31;
    if (out.esub_trace) for (int i = d + lane; i < max_depth; i += 32) out.esub_trace[i] = 0.0;
    #pragma unroll 1
    for (int i = lane; i < n; i += 32) {
        int32_t tok = -1, par = -1, dep = 0;
        double ph = 0.0;
        if (i < nR) {
            const int gid = s.rsel[i];
            dep = gid / n + 1;
            tok = __ldcg(&w.T_tok[gid]);
            ph = s.vals[i];
            if (dep > 1) {
                const int pg = (dep - 2) * n + __ldcg(&w.T_par[gid]);
                int lo = 0, hi = i;                        // the parent is packed before its child
                while (lo < hi) {
                    const int mid = (lo + hi) >> 1;
                    if (s.rsel[mid] < pg) lo = mid + 1; else hi = mid;
                }
                if (lo >= i || s.rsel[lo] != pg) set_status(status, kErrInternal);   // closure violated
                par = lo;
            }
        }
        out.token[i] = tok; out.parent[i] = par; out.depth[i] = dep; out.phat[i] = ph;
    }
    if (lane == 0) { *out.n_sel = nR; *out.depth_reached = d; *out.expected_len = esub; }
}

// Layer job, second half: the running top-n and E_sub(T, n) with the new layer (left in s by
// the selection), the loop test of Algorithm 1, and the packed tree if the sequence is
// finished.  All layers of a sequence are handled by the same warp, in order.  Returns true if the
// sequence continues with layer d+1, false if it is finished (outputs written).
template <class LS>
__device__ __noinline__ bool update_running_warp(LS& s, const SeqWork& w, const TreeOut& out, int d, int nl, int n, int Dcap,
                                    int max_depth, float delta, int* status) {
    const int lane = threadIdx.x & 31;
    int* hist = s.hist;
    const int gid0 = (d - 1) * n;
    unsigned long long thr;
    int need_eq;
    const int nR_old = d == 1 ? 0 : __ldcg(&w.st[kStNR]);
    const double eprev = d == 1 ? 0.0 : __ldcg(w.E_prev);

    // --- E_sub(T, n): the n largest path values among the previous top-n and the new layer ---
    const int32_t* Rold = w.R + ((d - 1) & 1) * n;
    int32_t* Rnew = w.R + (d & 1) * n;
    const int NR = nR_old + nl;                           // <= 2n
    const int nR = NR < n ? NR : n;
    unsigned long long ko = 0ull, ka = ~0ull;
    #pragma unroll 1
    for (int i = lane; i < NR; i += 32) {
        int gid;
        unsigned long long key;
        if (i < nR_old) { gid = __ldcg(&Rold[i]); key = phat_key(__ldcg(&w.T_phat[gid])); }
        else { gid = gid0 + (i - nR_old); key = s.lkeys[i - nR_old]; }
        s.gids[i] = gid;
        s.keys[i] = key;
        ko |= key; ka &= key;
    }
    __syncwarp();
    auto rkey = [&](int i) -> unsigned long long { return s.keys[i]; };
    warp_radix_select(rkey, NR, nR, hist, warp_or_u64(ko), warp_and_u64(ka), thr, need_eq);
    warp_compact_selected(rkey, NR, thr, need_eq, [&](int pos, int i) {
        Rnew[pos] = s.gids[i];
        s.rsel[pos] = s.gids[i];
        s.vals[pos] = __longlong_as_double((long long)(s.keys[i] - 1ull));
    });
    __syncwarp();
    double part = 0.0;
    #pragma unroll 1
    for (int i = lane; i < nR; i += 32) part += s.vals[i];
    const double esub = warp_sum(part);                   // fixed order: lanes stride the packed order
    const bool more = d < Dcap && (esub - eprev > (double)delta);     // loop test of Algorithm 1
    if (out.esub_trace && lane == 0) out.esub_trace[d - 1] = esub;
    if (lane == 0) {
        w.st[kStNR] = nR;
        *w.E_prev = esub;
    }
    __syncwarp();
    if (lane == 0) { s.last_nR = nR; s.last_esub = esub; }
    __syncwarp();
    if (more) return true;
    pack_tree_warp(s, w, out, d, nR, n, max_depth, esub, status);
    return false;
}

}  // namespace ot
