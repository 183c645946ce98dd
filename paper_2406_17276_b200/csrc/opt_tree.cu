// OPT-Tree draft-tree construction, tree mask and greedy verification for B200 (sm_100a):
// kernels and the C ABI declared in include/opt_tree.h.
#include "../../include/opt_tree.h"

#include <cuda_runtime.h>
#include <math.h>
#include <new>
#include <stdio.h>
#include <string.h>

#include "pipeline.cuh"
#include "select.cuh"

namespace ot {

constexpr int kRowMul = 31;                 // row of (token t, depth d) = (t*31 + d) mod H
constexpr int kSmallThreads = 256;          // block size of the mask / init kernels
// Verify: one CTA per target row.  With 128 threads sixteen CTAs fit an SM, so the n + 1 rows of 32
// sequences (c4: 2080 CTAs) are all resident at once instead of in two uneven waves; a thread keeps
// eight 16-byte loads in flight.
constexpr int kVerifyThreads = 128;

__device__ __forceinline__ int row_of(int token, int depth, int H) {
    return (int)(((long long)token * kRowMul + depth) % H);
}

// ------------------------------------------------------------------------------------------------
// Workspace
// ------------------------------------------------------------------------------------------------
struct Workspace {
    // build
    double* cand_phat;     // [B][cand_stride]
    int32_t* cand_tok;     // [B][cand_stride]
    int32_t* T_tok;        // [B][D*n]
    int32_t* T_par;        // [B][D*n]
    double* T_phat;        // [B][D*n]
    int32_t* R;            // [B][2][n]
    double* E_prev;        // [B]
    int32_t* st;           // [B][8]
    int32_t* fmap;         // [B][n]   pruned draft: layer slot behind each frontier row
    // layer-by-layer build (logits handed in per layer)
    double* front_phat;    // [B][n]   path values of the nodes whose logits come next
    int32_t* rtok;         // [B*n][k] row results of the layer in hand
    double* rprob;         // [B*n][k]
    // row mailboxes of the build: one per CTA, filled by the layer warps, never wrapped within a build.
    // The rows of a build are numbered by one running count (q_ctl[kQCursor]): row g goes to CTA
    // g % grid, entry g / grid of its mailbox.
    unsigned long long* mb_items;  // [grid][mcap]  one item per (sequence, layer, frontier slot)
    unsigned long long* mb_phat;   // [grid][mcap]  bit 63 valid | bits of the node's path value (a double >= 0)
    int32_t* q_ctl;        // [8]  2: sequences finished, 3: all done, 4: rows numbered so far
    // verify
    int32_t* g;            // [B][n+1]  target argmax after the root (0) and after node i (i+1)
    int32_t* vdone;        // [B]
    int32_t* status;       // [1]
    // device copies of inputs / outputs for the host-buffer step
    int32_t *h_root, *h_base;                          // [B]
    int32_t *o_token, *o_parent, *o_depth; double* o_phat;
    int32_t *o_nsel, *o_dreach; double* o_elen;
    uint64_t* o_mask; int32_t* o_pos;
    int32_t *o_alen, *o_atok, *o_anode, *o_next;
};
enum { kQFinished = 2, kQDone = 3, kQCursor = 4 };

constexpr int kMaxGrid = 4096;              // CTAs of the persistent kernels (SMs x occupancy) this layout supports

// Consecutive rows go to consecutive CTAs, so a CTA receives its even share of all rows of a build
// (one root and at most Dcap layers of n rows per sequence); its mailbox holds them all.
static size_t mailbox_capacity(const opt_tree_config& c, int grid) {
    const size_t Dcap = c.max_depth < c.n ? c.max_depth : c.n;
    const size_t rows = (size_t)c.max_batch * (1 + Dcap * (size_t)c.n);
    // + 8: a fetcher takes a few tickets beyond the last row it will ever get; those must stay inside
    return (rows + grid - 1) / grid + 8;
}

// Entries per sequence in the candidate arrays: n*k rounded up to a multiple of four (16-byte vectors).
static size_t cand_stride(int n, int k) { return ((size_t)n * k + 3) & ~(size_t)3; }

struct Layout {
    size_t total = 0;
    template <class T> size_t take(size_t count) {
        size_t off = (total + 255) & ~(size_t)255;
        total = off + count * sizeof(T);
        return off;
    }
};

static size_t carve(const opt_tree_config& c, int grid, char* base, Workspace* w) {
    const size_t B = c.max_batch, n = c.n, D = c.max_depth, W = (c.n + 63) / 64;
    const size_t cs = cand_stride(c.n, c.k);
    Layout L;
    size_t o;
#define OT_TAKE(field, T, count) o = L.take<T>(count); if (w) w->field = reinterpret_cast<T*>(base + o);
    OT_TAKE(cand_phat, double, B * cs)
    OT_TAKE(cand_tok, int32_t, B * cs)
    OT_TAKE(T_tok, int32_t, B * D * n)
    OT_TAKE(T_par, int32_t, B * D * n)
    OT_TAKE(T_phat, double, B * D * n)
    OT_TAKE(R, int32_t, B * 2 * n)
    OT_TAKE(E_prev, double, B)
    OT_TAKE(st, int32_t, B * 8)
    OT_TAKE(fmap, int32_t, B * n)
    OT_TAKE(front_phat, double, B * n)
    OT_TAKE(rtok, int32_t, B * n * (size_t)c.k)
    OT_TAKE(rprob, double, B * n * (size_t)c.k)
    OT_TAKE(mb_items, unsigned long long, mailbox_capacity(c, grid) * grid)
    OT_TAKE(mb_phat, unsigned long long, mailbox_capacity(c, grid) * grid)
    OT_TAKE(q_ctl, int32_t, 8)
    OT_TAKE(g, int32_t, B * (n + 1))
    OT_TAKE(vdone, int32_t, B)
    OT_TAKE(status, int32_t, 1)
    OT_TAKE(h_root, int32_t, B)
    OT_TAKE(h_base, int32_t, B)
    OT_TAKE(o_token, int32_t, B * n)
    OT_TAKE(o_parent, int32_t, B * n)
    OT_TAKE(o_depth, int32_t, B * n)
    OT_TAKE(o_phat, double, B * n)
    OT_TAKE(o_nsel, int32_t, B)
    OT_TAKE(o_dreach, int32_t, B)
    OT_TAKE(o_elen, double, B)
    OT_TAKE(o_mask, uint64_t, B * n * W)
    OT_TAKE(o_pos, int32_t, B * n)
    OT_TAKE(o_alen, int32_t, B)
    OT_TAKE(o_atok, int32_t, B * (D + 1))
    OT_TAKE(o_anode, int32_t, B * D)
    OT_TAKE(o_next, int32_t, B)
#undef OT_TAKE
    return (L.total + 255) & ~(size_t)255;
}

struct Params {            // by-value kernel parameters
    int V, H, n, k, kk, Dcap, max_depth, B;
    float delta;
    int aligned;
    int mcap, grid, cstride;
    int prune;             // draft only from layer nodes that are still among the n largest
};

__device__ __forceinline__ SeqWork seq_work(const Workspace& w, const Params& p, int b) {
    SeqWork s;
    s.cand_phat = w.cand_phat + (size_t)b * p.cstride;
    s.cand_tok = w.cand_tok + (size_t)b * p.cstride;
    s.T_tok = w.T_tok + (size_t)b * p.max_depth * p.n;
    s.T_par = w.T_par + (size_t)b * p.max_depth * p.n;
    s.T_phat = w.T_phat + (size_t)b * p.max_depth * p.n;
    s.R = w.R + (size_t)b * 2 * p.n;
    s.E_prev = w.E_prev + b;
    s.st = w.st + (size_t)b * 8;
    s.fmap = w.fmap + (size_t)b * p.n;
    return s;
}
__device__ __forceinline__ TreeOut tree_out(const opt_tree_out& o, const Params& p, int b) {
    TreeOut t;
    t.token = o.token + (size_t)b * p.n;
    t.parent = o.parent + (size_t)b * p.n;
    t.depth = o.depth + (size_t)b * p.n;
    t.phat = o.phat + (size_t)b * p.n;
    t.n_sel = o.n_sel + b;
    t.depth_reached = o.depth_reached + b;
    t.expected_len = o.expected_len + b;
    t.esub_trace = o.esub_trace ? o.esub_trace + (size_t)b * p.max_depth : nullptr;
    return t;
}

// Mailbox item: bit 63 valid | b (15 bits) | layer d (9) | void flag (1) | frontier slot (10, from bit 22) | table row of the node to
// expand (22).  A second word at the same mailbox position carries the node's path value (bit 63
// valid; a path value is never negative).  Both words validate themselves, so a row can be expanded
// from them alone and the publisher needs no fence before writing them.
constexpr int kMaxTableRows = 1 << 22;
constexpr int kMaxLayers = 510;             // layers a build may draft: layer d+1 must fit the item's 9-bit field
__device__ __forceinline__ unsigned long long item_encode(int b, int d, int slot, int row) {
    return (1ull << 63) | ((unsigned long long)b << 48) | ((unsigned long long)d << 39) |
           ((unsigned long long)slot << 22) | (unsigned long long)row;
}

// An entry that was handed out but is not needed after all (the pruned draft reserves a layer's entries
// before it knows how many rows the layer will have): fetchers drop such a ticket.
constexpr unsigned long long kItemVoid = 1ull << 38;

__device__ __forceinline__ unsigned long long phat_word(double p) {
    return (1ull << 63) | (unsigned long long)__double_as_longlong(p);
}

// ------------------------------------------------------------------------------------------------
// Kernels
// ------------------------------------------------------------------------------------------------
// Clears the mailboxes, sends the root row of sequence b to CTA b % grid and resets the per-sequence state.
__global__ void init_build_kernel(Workspace w, Params p, const int32_t* __restrict__ root_token) {
    grid_dependency_wait();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < p.grid * p.mcap) {
        const int c = i / p.mcap, j = i - c * p.mcap;
        const long long b = (long long)c + (long long)j * p.grid;         // the j-th root sent to CTA c
        unsigned long long item = 0ull, ph = 0ull;
        if (b < p.B) {
            int token = root_token[b];
            if (token < 0 || token >= p.V) { set_status(w.status, kErrInternal); token = 0; }
            item = item_encode((int)b, 1, 0, row_of(token, 0, p.H));
            ph = phat_word(1.0);                                          // the root counts as factor 1
        }
        w.mb_items[i] = item;
        w.mb_phat[i] = ph;
    }
    for (long long j = i; j < (long long)p.B * p.cstride; j += (long long)gridDim.x * blockDim.x) {
        reinterpret_cast<unsigned long long*>(w.cand_phat)[j] = 0ull;
        w.cand_tok[j] = 0;
    }
    // frontier row f stands for layer slot f unless a pruned layer says otherwise
    for (long long j = i; j < (long long)p.B * p.n; j += (long long)gridDim.x * blockDim.x) w.fmap[j] = (int32_t)(j % p.n);
    if (i < p.B) {
        int32_t* st = w.st + (size_t)i * 8;
        st[kStDone] = 0; st[kStNR] = 0; st[kStRows] = 0; st[kStL1] = 0;
        w.E_prev[i] = 0.0;
    }
    if (i == 0) { w.q_ctl[kQFinished] = 0; w.q_ctl[kQDone] = 0; w.q_ctl[kQCursor] = p.B; }   // the roots are rows 0 .. B-1
}

// Source of the tree build: the rows other CTAs' layer warps have put into this CTA's mailbox.
template <bool kPrune>
struct BuildSource {
    static constexpr bool kHasEmpty = kPrune;              // only the pruned draft voids entries
    Workspace w; Params p;
    const uint16_t* draft;
    __device__ long long claim(int i) { return i < p.mcap ? (long long)blockIdx.x * p.mcap + i : -1; }
    // Both words of an entry validate themselves; the "all done" flag is looked at only when
    // check_done is set.
    __device__ int poll(long long idx, RowDesc& d, bool check_done) {
        const unsigned long long item = ld_relaxed_u64(&w.mb_items[idx]), ph = ld_relaxed_u64(&w.mb_phat[idx]);
        if (!((item & ph) >> 63)) return check_done && ld_acquire_s32(&w.q_ctl[kQDone]) ? -1 : 0;
        if (kPrune && (item & kItemVoid)) return 2;
        d.b = (int)((item >> 48) & 0x7FFFu); d.d = (int)((item >> 39) & 0x1FFu);
        d.slot = (int)((item >> 22) & 0x3FFu); d.fsize = 0;
        d.pphat = __longlong_as_double((long long)(ph & 0x7FFFFFFFFFFFFFFFull));
        int row = (int)(item & 0x3FFFFFu);
        if (row >= p.H) { set_status(w.status, kErrInternal); row = 0; }
        d.row = draft + (size_t)row * p.V;
        return 1;
    }
};

// Sink of the tree build.  Finisher warps: candidates' path values (Eq. 2) and the layer's row
// counter.  Layer warp: the layer warp of CTA c owns sequences c, c + gridDim.x, ...; it watches
// their row counters, and when a layer is complete does the layer selection, publishes the next
// layer's rows, brings the running top-n up to date and applies the loop test of Algorithm 1.
// kPrune: the pruned draft (opt_tree_build_pruned); a compile-time choice so that the ordinary build
// carries none of its code.
template <bool kPrune>
struct BuildSink {
    Workspace w; Params p; opt_tree_out out;
    // Layer 1 by the finisher of the root's row.  The root's children are the only candidates of layer 1; when
    // they all fit the node budget nothing has to be selected: the finisher stores them as layer 1, as the
    // running top-n with its E_sub, applies the loop test and, if the tree grows on, sends out the rows of
    // layer 2 itself, which takes the layer team's round trip out of the first layer.  Returns false (nothing
    // done) when layer 1 needs a selection or the tree ends with it; the layer team then does it the ordinary way.
    __device__ bool first_layer_direct(const RowDesc& d, const RowOut& r, const SeqWork& sw) {
        const int lane = threadIdx.x & 31;
        const double ph = lane < r.kk ? d.pphat * r.p : 0.0;              // Eq. 2
        const double esub = warp_sum(ph);                                  // (the order update_running_warp sums in)
        const bool more = 1 < p.Dcap && (esub > (double)p.delta);          // loop test of Algorithm 1 with E = 0
        if (r.kk > p.n || !more) return false;
        const TreeOut to = tree_out(out, p, d.b);
        unsigned g0 = 0;
        if (lane == 0) g0 = atomicAdd(reinterpret_cast<unsigned int*>(&w.q_ctl[kQCursor]), (unsigned)r.kk);
        g0 = __shfl_sync(0xFFFFFFFFu, g0, 0);
        if (lane < r.kk) {
            int token = r.tok;
            if (token < 0 || token >= p.V) { set_status(w.status, kErrInternal); token = 0; }
            sw.T_tok[lane] = token; sw.T_par[lane] = 0; sw.T_phat[lane] = ph;
            sw.R[p.n + lane] = lane;                                       // the running top-n after layer 1 (buffer of odd layers)
            if (kPrune) sw.fmap[lane] = lane;
            const unsigned g = g0 + (unsigned)lane, c = g % (unsigned)p.grid, e = g / (unsigned)p.grid;
            if (e < (unsigned)p.mcap) {
                const size_t pos = (size_t)c * p.mcap + e;
                st_relaxed_u64(&w.mb_phat[pos], phat_word(ph));
                st_relaxed_u64(&w.mb_items[pos], item_encode(d.b, 2, lane, row_of(token, 1, p.H)));
            } else {
                set_status(w.status, kErrInternal);
            }
        }
        if (lane == 0) {
            if (to.esub_trace) to.esub_trace[0] = esub;
            sw.st[kStNR] = r.kk;
            *sw.E_prev = esub;
        }
        return true;
    }
    __device__ void row_done(const RowDesc& d, const RowOut& r, FinScratch&) {
        const int lane = threadIdx.x & 31;
        const SeqWork sw = seq_work(w, p, d.b);
        if (d.d == 1) {                                                    // the root's row
            const bool direct = first_layer_direct(d, r, sw);
            __syncwarp();
            if (lane == 0) {
                *reinterpret_cast<volatile unsigned int*>(&sw.st[kStL1]) = 0x80000000u | (direct ? (unsigned)r.kk : 0u);
                if (direct) atom_add_relaxed_s32(&sw.st[kStDone], 1);
            }
            if (direct) return;
        }
        // Candidate words validate themselves (top bit; an absent child is all ones), so neither they nor
        // the row count need a fence: the layer warp re-reads whatever it finds not yet written.
        if (lane < p.k) {
            unsigned long long* ph = reinterpret_cast<unsigned long long*>(sw.cand_phat) + d.slot * p.k + lane;
            unsigned int* tk = reinterpret_cast<unsigned int*>(sw.cand_tok) + d.slot * p.k + lane;
            *ph = lane < r.kk ? phat_word(d.pphat * r.p) : ~0ull;
            *tk = lane < r.kk ? (0x80000000u | (unsigned int)r.tok) : ~0u;
        }
        __syncwarp();
        if (lane == 0) atom_add_relaxed_s32(&sw.st[kStDone], 1);     // the count runs on over the layers of a build
    }
    // The rows of a new layer take the next numbers of the build's running row count and with them
    // their CTAs (row g: CTA g % grid, mailbox entry g / grid).  Whatever the order in which the
    // sequences publish, every CTA is sent the same number of rows to within one, and a layer spreads
    // over as many SMs as it has rows.  reserve_layer only starts the atomic (lane 0 keeps the result
    // in a register; nothing waits for it until publish_layer writes the entries).
    __device__ unsigned reserve_layer(int nl) {
        unsigned g0 = 0;
        if ((threadIdx.x & 31) == 0) g0 = atomicAdd(reinterpret_cast<unsigned int*>(&w.q_ctl[kQCursor]), (unsigned)nl);
        return g0;
    }
    // pick != null (pruned draft): only the layer slots pick[0..nl) are sent out, as frontier rows 0..nl;
    // the map from frontier row to layer slot is left in fmap for the next selection.
    template <class LS>
    __device__ void publish_layer(LS& ls, int b, int d, int nl, unsigned g0, const int* pick = nullptr,
                                  int32_t* fmap = nullptr) {
        const int lane = threadIdx.x & 31;
        g0 = __shfl_sync(0xFFFFFFFFu, g0, 0);
        for (int i = lane; i < nl; i += 32) {
            const int slot = pick ? pick[i] : i;
            if (fmap) fmap[i] = slot;
            int token = ls.ltok[slot];
            if (token < 0 || token >= p.V) { set_status(w.status, kErrInternal); token = 0; }
            const unsigned g = g0 + (unsigned)i, c = g % (unsigned)p.grid, e = g / (unsigned)p.grid;
            if (e < (unsigned)p.mcap) {
                const size_t pos = (size_t)c * p.mcap + e;
                st_relaxed_u64(&w.mb_phat[pos], (1ull << 63) | (ls.lkeys[slot] - 1ull));
                st_relaxed_u64(&w.mb_items[pos], item_encode(b, d + 1, i, row_of(token, d, p.H)));
            } else {
                set_status(w.status, kErrInternal);
            }
        }
        __syncwarp();
    }
    // Entries g0+from .. g0+to of a reservation are not needed.
    __device__ void void_entries(unsigned g0, int from, int to) {
        const int lane = threadIdx.x & 31;
        g0 = __shfl_sync(0xFFFFFFFFu, g0, 0);
        for (int i = from + lane; i < to; i += 32) {
            const unsigned g = g0 + (unsigned)i, c = g % (unsigned)p.grid, e = g / (unsigned)p.grid;
            if (e < (unsigned)p.mcap) {
                const size_t pos = (size_t)c * p.mcap + e;
                st_relaxed_u64(&w.mb_phat[pos], 1ull << 63);
                st_relaxed_u64(&w.mb_items[pos], (1ull << 63) | kItemVoid);
            } else {
                set_status(w.status, kErrInternal);
            }
        }
        __syncwarp();
    }
    // Pruned draft, a whole layer job with one selection (see select_running_team).  Returns the number
    // of rows of the next layer, or -1 if the sequence is finished.
    template <class LS>
    __device__ int merged_layer_job(LS& ls, const SeqWork& sw, int b, int d, int fsize, int nR_old, int off) {
        const int lane = threadIdx.x & 31;
        const int nvalid = fsize * p.kk, reserve = nvalid < p.n ? nvalid : p.n;
        stage_layer_candidates(ls, sw, fsize, p.k, off);
        const unsigned g0 = d < p.Dcap ? reserve_layer(reserve) : 0u;      // entries for the next layer, before its size is known
        // the old top-n: still in the scratch if this warp's last job was this sequence's previous layer
        const int32_t* Rold = sw.R + ((d - 1) & 1) * p.n;
        const bool cached = ls.cache_b == b && ls.cache_d == d - 1;
        for (int i = lane; i < nR_old; i += 32) {
            int gid;
            unsigned long long key;
            if (cached) { gid = ls.rsel[i]; key = phat_key(ls.vals[i]); }
            else { gid = __ldcg(&Rold[i]); key = phat_key(__ldcg(&sw.T_phat[gid])); }
            ls.gids[i] = gid;
            ls.keys[i] = key;
        }
        if (lane == 0) {
            LayerJob& j = ls.job;
            j.kind = 2; j.d = d; j.fsize = fsize; j.n = p.n; j.k = p.k; j.kk = p.kk;
            j.cand_phat = sw.cand_phat; j.cand_tok = sw.cand_tok;
            j.T_tok = sw.T_tok; j.T_par = sw.T_par; j.T_phat = sw.T_phat;
            j.fmap = sw.fmap; j.nR_old = nR_old; j.off = off; j.Rnew = sw.R + (d & 1) * p.n;
        }
        cp_async_wait_all();
        __syncwarp();
        team_sync();
        const LayerJob j = ls.job;
        const int nR = select_running_team(ls, j, lane, w.status);
        int kept_old = 0;
#pragma unroll
        for (int q = 0; q < kTeamWarps; ++q) kept_old += ls.scan_c[q];
        const int cnt = nR - kept_old;                      // new members = the rows of the next layer
        double part = 0.0;
        for (int i = lane; i < nR; i += 32) part += ls.vals[i];
        const double esub = warp_sum(part);
        const double eprev = d == 1 ? 0.0 : __ldcg(sw.E_prev);
        bool more = d < p.Dcap && (esub - eprev > (double)p.delta);
        const TreeOut to = tree_out(out, p, b);
        if (lane == 0) {
            if (to.esub_trace) to.esub_trace[d - 1] = esub;
            sw.st[kStNR] = nR;
            *sw.E_prev = esub;
            ls.cache_b = b; ls.cache_d = d;
        }
        __syncwarp();
        if (more && cnt > 0) {
            for (int i = lane; i < cnt; i += 32) ls.gids[i] = i;       // members are sent out in slot order
            __syncwarp();
            publish_layer(ls, b, d, cnt, g0, ls.gids, sw.fmap);
            void_entries(g0, cnt, reserve);
            return cnt;
        }
        if (d < p.Dcap) void_entries(g0, 0, reserve);
        int d_end = d;
        if (more) {                                         // nothing left to draft from: the loop would go on testing a gain of zero
            d_end = p.delta < 0.0f ? p.Dcap : d + 1;
            if (to.esub_trace) for (int i = d + lane; i < d_end; i += 32) to.esub_trace[i] = esub;
            __syncwarp();
        }
        pack_tree_warp(ls, sw, to, d_end, nR, p.n, p.max_depth, esub, w.status);
        return -1;
    }
    // The layer warp follows its sequences (layer_follow); whenever a layer is complete it hands the
    // selection to the whole team: the job goes into shared memory, the team barrier starts it.  The
    // assistants wait at that barrier in between and leave when they find a job of kind 0.
    template <class LS>
    __device__ void layer_loop(LS& ls) {
        layer_follow(ls);
        if ((threadIdx.x & 31) == 0) ls.job.kind = 0;
        __syncwarp();
        team_sync();
    }
    template <class LS>
    __device__ void layer_assist(LS& ls, int tw) {
        const int tt = tw * 32 + (int)(threadIdx.x & 31);
        for (;;) {
            team_sync();
            const LayerJob j = ls.job;
            if (j.kind == 0) return;
            if (j.kind == 2) select_running_team(ls, j, tt, w.status);
            else if (j.fsize * j.k <= kStageCap) select_layer_team<kPrune>(ls, j, tt, w.status);
            else select_layer_team_big<kPrune>(ls, j, tt, w.status);
        }
    }
    template <class LS>
    __device__ void layer_follow(LS& ls) {
        const int lane = threadIdx.x & 31;
        constexpr int kOwn = 4;                            // sequences one layer warp follows at a time
        for (int b0 = blockIdx.x; b0 < p.B; b0 += kOwn * gridDim.x) {
            // layer in flight (0 = finished / none), its row count, rows expected in all layers so far
            int cur_d[kOwn], cur_f[kOwn], cur_tot[kOwn];
            int live = 0;
#pragma unroll
            for (int q = 0; q < kOwn; ++q) {
                const bool has = b0 + q * (int)gridDim.x < p.B;
                cur_d[q] = has ? 1 : 0; cur_f[q] = 1; cur_tot[q] = 1; live += has ? 1 : 0;
            }
            long long t0 = clock64();
            while (live > 0) {
                bool progressed = false;
#pragma unroll 1                                          // one copy of the body: it is long, and instruction fetch is what the helper warps wait for
                for (int q = 0; q < kOwn; ++q) {
                    if (cur_d[q] == 0) continue;
                    const int b = b0 + q * (int)gridDim.x;
                    const SeqWork sw = seq_work(w, p, b);
                    int done = 0;
                    if (lane == 0) done = ld_acquire_s32(&sw.st[kStDone]);
                    done = __shfl_sync(0xFFFFFFFFu, done, 0);
                    if (done < cur_tot[q]) continue;
                    progressed = true;
                    if (cur_d[q] == 1) {
                        // the finisher of the root's row says whether it grew layer 1 itself (then layer 2 is on its way)
                        unsigned int how = 0;
                        if (lane == 0) how = poll_tok_word(reinterpret_cast<const unsigned int*>(&sw.st[kStL1]), w.status);
                        how = __shfl_sync(0xFFFFFFFFu, how, 0) & 0x7FFFFFFFu;
                        if (how != 0x7FFFFFFFu && how > 0) {
                            cur_d[q] = 2; cur_f[q] = (int)how; cur_tot[q] += (int)how;
                            if (kPrune && lane == 0) sw.st[kStRows] = cur_tot[q];
                            continue;
                        }
                    }
                    const int d = cur_d[q], fsize = cur_f[q];
                    const int nvalid = fsize * p.kk, nl = nvalid < p.n ? nvalid : p.n;
                    // Without a threshold the loop test only looks at the depth: the next layer's rows
                    // can go out before the running top-n is brought up to date.
                    // The pruned draft always takes the one-selection layer job; the ordinary build takes it for
                    // the layer at the depth limit, after which nothing is drafted: the nodes of that layer that
                    // do not reach the running top-n need not be stored, and one selection does instead of two.
                    if (kPrune || d == p.Dcap) {
                        const int nR_old = d == 1 ? 0 : __ldcg(&sw.st[kStNR]);
                        const int off = (nR_old + 1) & ~1;
                        if (off + fsize * p.k <= kStageCap) {
                            const int sent = merged_layer_job(ls, sw, b, d, fsize, nR_old, off);
                            if (sent > 0) { cur_d[q] = d + 1; cur_f[q] = sent; cur_tot[q] += sent; }
                            if (kPrune && lane == 0) sw.st[kStRows] = cur_tot[q];
                            if (sent <= 0) {
                                cur_d[q] = 0; --live;
                                __threadfence();
                                if (lane == 0 && atomicAdd(&w.q_ctl[kQFinished], 1) == p.B - 1) st_release_s32(&w.q_ctl[kQDone], 1);
                            }
                            __syncwarp();
                            continue;
                        }
                    }
                    const bool early = !kPrune && d < p.Dcap && p.delta == -INFINITY;
                    stage_layer_candidates(ls, sw, fsize, p.k);
                    unsigned g0 = 0;
                    if (early) g0 = reserve_layer(nl);        // the rows' numbers, while the candidates load
                    {
                        const bool small = fsize * p.k <= kStageCap;    // the candidates fit the shared-memory staging
                        if (lane == 0) {
                            LayerJob& j = ls.job;
                            j.kind = 1; j.d = d; j.fsize = fsize; j.n = p.n; j.k = p.k; j.kk = p.kk;
                            j.cand_phat = sw.cand_phat; j.cand_tok = sw.cand_tok;
                            j.T_tok = sw.T_tok; j.T_par = sw.T_par; j.T_phat = sw.T_phat;
                            j.fmap = kPrune ? sw.fmap : nullptr;
                        }
                        if (small) cp_async_wait_all();       // the staged candidates are in shared memory
                        __syncwarp();
                        team_sync();                          // ... and, with the job, visible to the assistants
                        const LayerJob j = ls.job;
                        if (small) select_layer_team<kPrune>(ls, j, lane, w.status);
                        else select_layer_team_big<kPrune>(ls, j, lane, w.status);
                    }
                    if (early) publish_layer(ls, b, d, nl, g0);
                    bool more = update_running_warp(ls, sw, tree_out(out, p, b), d, nl, p.n, p.Dcap, p.max_depth, p.delta,
                                                    w.status);
                    if (lane == 0) { ls.cache_b = b; ls.cache_d = d; }                // rsel / vals now hold this top-n
                    int sent = nl;                             // rows of the next layer
                    if (kPrune && more) {
                        // The new layer's nodes among the n largest are the tail of the ascending list rsel
                        // (their gids are the largest); only they are drafted from.
                        const int gid0 = (d - 1) * p.n;
                        const int nR = ls.last_nR;
                        const double esub = ls.last_esub;
                        int mine = 0;
                        for (int i = lane; i < nR; i += 32) mine += ls.rsel[i] >= gid0 ? 1 : 0;
                        sent = __reduce_add_sync(0xFFFFFFFFu, mine);
                        for (int i = lane; i < sent; i += 32) ls.gids[i] = ls.rsel[nR - sent + i] - gid0;
                        __syncwarp();
                        if (sent > 0) {
                            publish_layer(ls, b, d, sent, reserve_layer(sent), ls.gids, sw.fmap);
                        } else {
                            // Nothing left to draft from: further layers change neither T_opt nor E_sub.  The loop
                            // of Algorithm 1 would go on testing a gain of zero: to the depth limit if the
                            // threshold is negative, else for one more layer.
                            const int d_end = p.delta < 0.0f ? p.Dcap : d + 1;
                            const TreeOut to = tree_out(out, p, b);
                            if (to.esub_trace) for (int i = d + lane; i < d_end; i += 32) to.esub_trace[i] = esub;
                            __syncwarp();
                            pack_tree_warp(ls, sw, to, d_end, nR, p.n, p.max_depth, esub, w.status);
                            more = false;
                        }
                    } else if (more && !early) {
                        publish_layer(ls, b, d, nl, reserve_layer(nl));
                    }
                    if (more) { cur_d[q] = d + 1; cur_f[q] = sent; cur_tot[q] += sent; }
                    if (kPrune && lane == 0) sw.st[kStRows] = cur_tot[q];
                    if (!more) {
                        cur_d[q] = 0; --live;
                        __threadfence();
                        if (lane == 0 && atomicAdd(&w.q_ctl[kQFinished], 1) == p.B - 1) st_release_s32(&w.q_ctl[kQDone], 1);
                    }
                    __syncwarp();
                }
                if (progressed) t0 = clock64();
                else {
                    if (clock64() - t0 > kWaitCycles) { set_status(w.status, kErrTimeout); return; }
                    __nanosleep(100);
                }
            }
        }
    }
};

// Algorithm 1 for a whole batch in one launch: persistent CTAs take rows from their mailboxes; layers
// of different sequences overlap freely because sequences never exchange data.
template <bool kPrune, int NCAP>
__global__ void __launch_bounds__(kThreads)
build_kernel(Workspace w, Params p, const uint16_t* __restrict__ draft, opt_tree_out out) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    CtaSmemT<NCAP>& s = *reinterpret_cast<CtaSmemT<NCAP>*>(smem_raw);
    BuildSource<kPrune> src{w, p, draft};
    BuildSink<kPrune> sink{w, p, out};
    run_pipeline(s, src, sink, p.V, p.k, p.aligned != 0, w.status);
}

// The row step alone over a list of rows (static round-robin over the CTAs).
struct ListSource {
    static constexpr bool kHasEmpty = false;
    const uint16_t* logits; const int32_t* rows; int nrows, V, H, first, stride; int* status;
    __device__ long long claim(int r) {
        const long long idx = (long long)first + (long long)r * stride;
        return idx < nrows ? idx : -1;
    }
    __device__ int poll(long long idx, RowDesc& d, bool) {
        int row = rows ? rows[idx] : (int)idx;             // no list: row idx of a dense buffer
        if (row < 0 || row >= H) { set_status(status, kErrInternal); row = 0; }
        d.row = logits + (size_t)row * V; d.slot = (int)idx; d.b = d.d = 0; d.fsize = 1;
        return 1;
    }
};
struct ListSink {
    int32_t* tok_out; double* prob_out; int k;
    template <class LS> __device__ void layer_loop(LS&) {}
    template <class LS> __device__ void layer_assist(LS&, int) {}
    __device__ void row_done(const RowDesc& d, const RowOut& r, FinScratch&) {
        const int lane = threadIdx.x & 31;
        if (lane < k) {
            tok_out[(size_t)d.slot * k + lane] = r.tok;
            prob_out[(size_t)d.slot * k + lane] = r.p;
        }
    }
};
__global__ void __launch_bounds__(kThreads)
row_topk_kernel(Params p, const uint16_t* __restrict__ logits, const int32_t* __restrict__ rows, int nrows,
                int32_t* tok_out, double* prob_out, int* status) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    CtaSmem& s = *reinterpret_cast<CtaSmem*>(smem_raw);
    ListSource src{logits, rows, nrows, p.V, p.H, (int)blockIdx.x, (int)gridDim.x, status};
    ListSink sink{tok_out, prob_out, p.k};
    run_pipeline(s, src, sink, p.V, p.k, p.aligned != 0, status);
}

// ------------------------------------------------------------------------------------------------
// Layer-by-layer build: the caller (a real draft model) hands in the logits of one layer's nodes at
// a time.  Per layer one launch of the row kernel over the dense buffer and one of layer_step_kernel:
// a CTA of kTeam threads per sequence forms the candidates (Eq. 2), selects the layer with the same
// team selection as the persistent build, updates the running top-n / E_sub, applies the loop test
// and hands back the next layer's tokens; a sequence that stops is packed on the spot.
// ------------------------------------------------------------------------------------------------
__global__ void layers_begin_kernel(Workspace w, Params p) {
    grid_dependency_wait();
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= p.B) return;
    int32_t* st = w.st + (size_t)b * 8;
    st[kStDone] = 0; st[kStNR] = 0; st[kStRows] = 0; st[kStDepth] = 1; st[kStFsize] = 1;
    w.E_prev[b] = 0.0;
    w.front_phat[(size_t)b * p.n] = 1.0;                       // the root counts as factor 1
    w.fmap[(size_t)b * p.n] = 0;
}

template <int NCAP>
__global__ void __launch_bounds__(kTeam)
layer_step_kernel(Workspace w, Params p, int fstride, opt_tree_out out, int32_t* next_tokens, int32_t* next_parent,
                  int32_t* next_count) {
    extern __shared__ __align__(16) unsigned char ls_raw[];
    LayerScratchT<NCAP>& ls = *reinterpret_cast<LayerScratchT<NCAP>*>(ls_raw);
    grid_dependency_wait();
    const int b = blockIdx.x, tt = threadIdx.x, lane = tt & 31;
    for (int i = tt; i < 3 * 256; i += kTeam) (&ls.thist[0][0])[i] = 0;
    const SeqWork sw = seq_work(w, p, b);
    const int d = sw.st[kStDepth], fsize = sw.st[kStFsize];
    if (d == 0) {                                            // this sequence stopped at an earlier layer
        if (tt == 0) next_count[b] = 0;
        return;
    }
    if (fsize < 1 || fsize > fstride || fsize > p.n) { if (tt == 0) { set_status(w.status, kErrInternal); next_count[b] = 0; } return; }
    // candidates of the layer (Eq. 2), left the way the finishers of the persistent build leave them
    const int N = fsize * p.k;
    const double* fph = w.front_phat + (size_t)b * p.n;
    for (int i = tt; i < N; i += kTeam) {
        const int f = i / p.k, r = i - f * p.k;
        const size_t src = ((size_t)b * fstride + f) * p.k + r;
        const int tok = w.rtok[src];
        const bool valid = r < p.kk && tok >= 0;
        reinterpret_cast<unsigned long long*>(sw.cand_phat)[i] = valid ? phat_word(fph[f] * w.rprob[src]) : ~0ull;
        reinterpret_cast<unsigned int*>(sw.cand_tok)[i] = valid ? (0x80000000u | (unsigned int)tok) : ~0u;
    }
    __syncthreads();
    const bool small = N <= kStageCap;
    if (tt < 32 && small) { stage_layer_candidates(ls, sw, fsize, p.k); cp_async_wait_all(); }
    if (tt == 0) {
        LayerJob& j = ls.job;
        j.kind = 1; j.d = d; j.fsize = fsize; j.n = p.n; j.k = p.k; j.kk = p.kk;
        j.cand_phat = sw.cand_phat; j.cand_tok = sw.cand_tok;
        j.T_tok = sw.T_tok; j.T_par = sw.T_par; j.T_phat = sw.T_phat;
        j.fmap = nullptr; j.nR_old = 0; j.off = 0; j.Rnew = nullptr;
    }
    __syncthreads();
    const LayerJob j = ls.job;
    const int nl = small ? select_layer_team<false>(ls, j, tt, w.status) : select_layer_team_big<false>(ls, j, tt, w.status);
    if (tt >= 32) return;                                    // the rest is one warp's work
    const bool more = update_running_warp(ls, sw, tree_out(out, p, b), d, nl, p.n, p.Dcap, p.max_depth, p.delta, w.status);
    if (more) {
        const int gid0 = (d - 1) * p.n;
        for (int i = lane; i < nl; i += 32) {
            next_tokens[(size_t)b * p.n + i] = ls.ltok[i];
            next_parent[(size_t)b * p.n + i] = __ldcg(&sw.T_par[gid0 + i]);
            w.front_phat[(size_t)b * p.n + i] = __longlong_as_double((long long)(ls.lkeys[i] - 1ull));
        }
        if (lane == 0) { sw.st[kStDepth] = d + 1; sw.st[kStFsize] = nl; next_count[b] = nl; }
    } else if (lane == 0) {
        sw.st[kStDepth] = 0; next_count[b] = 0;
    }
}

// Tree attention mask + position ids: one CTA per sequence, a thread per node (in rounds of the block
// size when n is larger): the node's ancestor chain is walked and its bits gathered in registers.
__global__ void __launch_bounds__(kSmallThreads)
mask_kernel(const int32_t* __restrict__ parent, const int32_t* __restrict__ depth, const int32_t* __restrict__ n_sel,
            const int32_t* __restrict__ base_pos, int n, uint64_t* mask, int32_t* position_ids, int* status) {
    grid_dependency_wait();
    const int b = blockIdx.x;
    const int W = (n + 63) >> 6;
    const int ns = n_sel[b];
    const int32_t* par = parent + (size_t)b * n;
    for (int i = threadIdx.x; i < n; i += kSmallThreads) {
        uint64_t bits[kMaxN / 64];
#pragma unroll
        for (int wd = 0; wd < kMaxN / 64; ++wd) bits[wd] = 0ull;
        int pos = 0;
        if (i < ns) {
            int a = i, steps = 0;
            while (a >= 0 && steps <= n) {                  // an ancestor chain is at most n long
                if (a >= n) { set_status(status, kErrInternal); break; }
#pragma unroll
                for (int wd = 0; wd < kMaxN / 64; ++wd)
                    if ((a >> 6) == wd) bits[wd] |= 1ull << (a & 63);
                a = par[a];
                ++steps;
            }
            pos = (base_pos ? base_pos[b] : 0) + depth[(size_t)b * n + i];
        }
#pragma unroll
        for (int wd = 0; wd < kMaxN / 64; ++wd)
            if (wd < W) mask[((size_t)b * n + i) * W + wd] = bits[wd];
        position_ids[(size_t)b * n + i] = pos;
    }
}

// After verification: the bitmask expanded to the dense (n+1) x (n+1) form, position 0 being the
// root, and the step positions whose keys and values stay in the caches (the root and the matched
// nodes, in path order).  One CTA per sequence.
__global__ void __launch_bounds__(kSmallThreads)
post_verify_kernel(const int32_t* __restrict__ n_sel, const uint64_t* __restrict__ mask, const int32_t* __restrict__ accept_len,
                   const int32_t* __restrict__ accept_nodes, int n, int max_depth, uint8_t* dense, int32_t* kv_gather,
                   int32_t* kv_keep, int* status) {
    grid_dependency_wait();
    const int b = blockIdx.x, tid = threadIdx.x;
    const int S = n + 1, W = (n + 63) >> 6;
    const int ns = n_sel[b];
    const uint64_t* mb = mask + (size_t)b * n * W;
    uint8_t* db = dense + (size_t)b * S * S;
    for (int idx = tid; idx < S * S; idx += kSmallThreads) {
        const int r = idx / S, c = idx - r * S;
        bool on = r == c;
        if (r >= 1 && r - 1 < ns) {
            if (c == 0) on = true;
            else on = (mb[(size_t)(r - 1) * W + ((c - 1) >> 6)] >> ((c - 1) & 63)) & 1ull;
        }
        db[idx] = on ? 1 : 0;
    }
    int A = accept_len[b];
    if (A < 1 || A > max_depth + 1) { set_status(status, kErrInternal); A = 1; }
    for (int j = tid; j <= max_depth; j += kSmallThreads) {
        int g = -1;
        if (j == 0) g = 0;
        else if (j < A) {
            const int node = accept_nodes[(size_t)b * max_depth + j - 1];
            if (node < 0 || node >= ns) set_status(status, kErrInternal);
            else g = 1 + node;
        }
        kv_gather[(size_t)b * (max_depth + 1) + j] = g;
    }
    if (tid == 0) kv_keep[b] = A;
}

__device__ __forceinline__ uint4 ld_nc_v4(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

struct VerifySmem {
    unsigned long long red_u64[kVerifyThreads / 32];
    int flag;
    int hit;
};

// The end of a verification CTA: position j's token y is recorded; the CTA that records a sequence's
// last token walks the tree: accept the child that carries the recorded token, until none does.
__device__ void verify_tail(VerifySmem& s, const Workspace& w, const Params& p, int b, int j, int ns, int y,
                            const int32_t* tok, const int32_t* par, int32_t* accept_len, int32_t* accept_tokens,
                            int32_t* accept_nodes, int32_t* next_root) {
    const int tid = threadIdx.x;
    int32_t* g = w.g + (size_t)b * (p.n + 1);
    if (tid == 0) {
        g[j] = y;
        __threadfence();
        s.flag = (atomicAdd(&w.vdone[b], 1) == ns);
    }
    __syncthreads();
    if (!s.flag) return;
    __threadfence();

    // acceptance walk (block-wide child search; children of one node carry distinct tokens)
    int32_t* at = accept_tokens + (size_t)b * (p.max_depth + 1);
    int32_t* an = accept_nodes + (size_t)b * p.max_depth;
    for (int i = tid; i <= p.max_depth; i += kVerifyThreads) at[i] = -1;
    for (int i = tid; i < p.max_depth; i += kVerifyThreads) an[i] = -1;
    __syncthreads();
    int cur = -1, A = 0;
    for (int step = 0; step <= p.max_depth; ++step) {
        const int yy = __ldcg(&g[cur + 1]);
        if (tid == 0) { at[A] = yy; s.hit = -1; }
        ++A;
        __syncthreads();
        if (A > p.max_depth) break;
        for (int i = tid; i < ns; i += kVerifyThreads)
            if (par[i] == cur && tok[i] == yy) s.hit = i;
        __syncthreads();
        const int hit = s.hit;
        __syncthreads();
        if (hit < 0) break;
        if (tid == 0) an[A - 1] = hit;
        cur = hit;
    }
    if (tid == 0) {
        accept_len[b] = A;
        next_root[b] = __ldcg(&g[cur + 1]);
        w.vdone[b] = 0;
    }
}

// Greedy verification.  CTA (j, b): j = 0 takes the target row after the root, j >= 1 the row after
// kept node j-1; each finds the row's argmax (lowest token on ties).  The last CTA of a sequence
// then walks the tree: accept the child that carries the target's token, until none does.
__global__ void __launch_bounds__(kVerifyThreads)
verify_kernel(Workspace w, Params p, const uint16_t* __restrict__ target, const int32_t* __restrict__ root_token,
              opt_tree_out tree, int32_t* accept_len, int32_t* accept_tokens, int32_t* accept_nodes, int32_t* next_root) {
    __shared__ VerifySmem s;
    grid_dependency_wait();
    const int b = blockIdx.y, j = blockIdx.x, tid = threadIdx.x;
    const int ns = tree.n_sel[b];
    if (j > ns) return;
    const int32_t* tok = tree.token + (size_t)b * p.n;
    const int32_t* par = tree.parent + (size_t)b * p.n;
    int token = j == 0 ? root_token[b] : tok[j - 1];
    const int depth = j == 0 ? 0 : tree.depth[(size_t)b * p.n + j - 1];
    if (token < 0 || token >= p.V) { set_status(w.status, kErrInternal); token = 0; }
    const uint16_t* row = target + (size_t)row_of(token, depth, p.H) * p.V;

    unsigned long long best_key = 0ull;
    if (p.aligned) {
        const uint4* vec = reinterpret_cast<const uint4*>(row);
        const int nv = p.V >> 3;
        float best = -INFINITY;
        int best_v = -1;
#pragma unroll 1
        for (int v0 = tid; v0 < nv; v0 += 8 * kVerifyThreads) {
            uint4 q[8];
#pragma unroll
            for (int u = 0; u < 8; ++u)
                q[u] = v0 + u * kVerifyThreads < nv ? ld_nc_v4(vec + v0 + u * kVerifyThreads)
                                                    : make_uint4(0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u);
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const uint32_t m2 = max_bf16x2(max_bf16x2(q[u].x, q[u].y), max_bf16x2(q[u].z, q[u].w));
                const float f = fmaxf(__uint_as_float(m2 << 16), __uint_as_float(m2 & 0xFFFF0000u));
                if (v0 + u * kVerifyThreads < nv && (f > best || best_v < 0)) { best = f; best_v = v0 + u * kVerifyThreads; }
            }
        }
        if (best_v >= 0) {
            const uint4 q = vec[best_v];
            const uint32_t ww[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
            for (int e = 7; e >= 0; --e) {
                const uint32_t bits = (e & 1) ? (ww[e >> 1] >> 16) : (ww[e >> 1] & 0xFFFFu);
                if (bf16_bits_to_float(bits) == best) best_key = cand_key(bits, (uint32_t)(best_v * 8 + e));
            }
        }
    } else {
        for (int v = tid; v < p.V; v += kVerifyThreads) {
            const unsigned long long key = cand_key(__ldg(row + v), (uint32_t)v);
            best_key = key > best_key ? key : best_key;
        }
    }
    best_key = warp_max_u64(best_key);
    if ((tid & 31) == 0) s.red_u64[tid >> 5] = best_key;
    __syncthreads();
    if (tid == 0)
        for (int q = 1; q < kVerifyThreads / 32; ++q) best_key = s.red_u64[q] > best_key ? s.red_u64[q] : best_key;
    verify_tail(s, w, p, b, j, ns, (int32_t)cand_token(best_key), tok, par, accept_len, accept_tokens, accept_nodes, next_root);
}

// ------------------------------------------------------------------------------------------------
// Verification with sampling (temperature tau > 0): at every position the next token is drawn from
// softmax(x / tau) of the target row by inverse CDF in token order, with one uniform per (sequence,
// position) from the counter-based generator Philox4x32-10 (Salmon et al. 2011; key = seed, counter =
// (position, sequence, step low, step high)); the walk is the greedy one on the drawn tokens.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0, uint32_t k1,
                                              uint32_t& o0, uint32_t& o1) {
#pragma unroll 1
    for (int round = 0; round < 10; ++round) {
        const uint32_t h0 = __umulhi(0xD2511F53u, c0), l0 = 0xD2511F53u * c0;
        const uint32_t h1 = __umulhi(0xCD9E8D57u, c2), l1 = 0xCD9E8D57u * c2;
        const uint32_t n0 = h1 ^ c1 ^ k0, n2 = h0 ^ c3 ^ k1;
        c0 = n0; c1 = l1; c2 = n2; c3 = l0;
        k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
    }
    o0 = c0; o1 = c1;
}
__device__ __forceinline__ double uniform53(unsigned long long seed, unsigned long long step, int sequence, int position) {
    uint32_t o0, o1;
    philox4x32_10((uint32_t)position, (uint32_t)sequence, (uint32_t)step, (uint32_t)(step >> 32), (uint32_t)seed,
                  (uint32_t)(seed >> 32), o0, o1);
    const unsigned long long bits = (((unsigned long long)o1 << 32) | o0) >> 11;
    return (double)bits * (1.0 / 9007199254740992.0);
}

// Sampling works on segments of 64 vectors (512 logits): one warp, two coalesced 16-byte loads per lane.
constexpr int kSegVecs = 64;
constexpr int kSegTokens = kSegVecs * 8;
constexpr int kMaxSeg = 640;                 // rows of up to 327 680 logits take the one-pass path
constexpr int kSampleExpLimit = 1 << 22;     // |exponent| beyond which the single-precision pass cannot scale
struct alignas(8) SegPart { float sum; int E; };       // a segment's sum of 2^(x*c - E), E an integer
struct SampleSmem {
    union { SegPart part[kMaxSeg]; double cum[kMaxSeg]; };   // per segment: its partial sum, then the running sum up to and including it
    double wsum[kVerifyThreads / 32];
    double S;
    float wmax[kVerifyThreads / 32];
    int wE[kVerifyThreads / 32];
    int chosen, last_live, seg, live_seg;
};

// The plain way, for rows the one-pass path does not take (unaligned rows, very long rows, extreme
// magnitudes): thread t owns the tokens [t*L, (t+1)*L); the row's maximum, then every thread's sum of
// double-precision exponentials in token order, a scan over the threads, and the thread in whose stretch
// u*S falls walks it once more.  Returns the drawn token to every thread.
__device__ __noinline__ int sample_row_plain(SampleSmem& q, const uint16_t* row, int V, bool vec, double tau, double u) {
    const int tid = threadIdx.x, lane = tid & 31, wp = tid >> 5;
    const int L = (((V + kVerifyThreads - 1) / kVerifyThreads) + 7) & ~7;       // tokens per thread, a multiple of 8
    const int lo = min(tid * L, V), hi = min(lo + L, V);
    auto logit = [&](int v) -> float { return bf16_bits_to_float(__ldg(row + v)); };
    const uint4* rv = reinterpret_cast<const uint4*>(row);
    float mx = -INFINITY;
    if (vec) {
        for (int v8 = lo >> 3; v8 < hi >> 3; ++v8) {
            const uint4 x = ld_nc_v4(rv + v8);
            const uint32_t m2 = max_bf16x2(max_bf16x2(x.x, x.y), max_bf16x2(x.z, x.w));
            mx = fmaxf(mx, fmaxf(__uint_as_float(m2 << 16), __uint_as_float(m2 & 0xFFFF0000u)));
        }
    } else {
        for (int v = lo; v < hi; ++v) mx = fmaxf(mx, logit(v));
    }
    mx = warp_max_f32(mx);
    __syncthreads();                                         // (the scratch may still be in use by the one-pass path)
    if (lane == 0) q.wmax[wp] = mx;
    if (tid == 0) { q.chosen = -1; q.last_live = -1; }
    __syncthreads();
    mx = q.wmax[0];
#pragma unroll
    for (int i = 1; i < kVerifyThreads / 32; ++i) mx = fmaxf(mx, q.wmax[i]);
    const double m = (double)mx;
    double mine = 0.0;
    int live = -1;                                           // last token of the stretch with a positive term
    for (int v = lo; v < hi; ++v) {
        const double e = exp(((double)logit(v) - m) / tau);
        mine += e;
        if (e > 0.0) live = v;
    }
    double incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const double up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += up;
    }
    if (lane == 31) q.wsum[wp] = incl;
    __syncthreads();
    double base = 0.0, S = 0.0;                              // running sums before this warp / of the row, added up in one fixed order
#pragma unroll
    for (int i = 0; i < kVerifyThreads / 32; ++i) { if (i == wp) base = S; S += q.wsum[i]; }
    // a thread's stretch begins exactly where the previous thread's ends: the same expression on both sides
    double prev = __shfl_up_sync(0xFFFFFFFFu, incl, 1);
    if (lane == 0) prev = 0.0;
    const double excl_t = base + prev, incl_t = base + incl;
    const double t = u * S;
    atomicMax(&q.last_live, live);
    if (incl_t > t && !(excl_t > t) && hi > lo) {            // the stretch in which the running sum passes t: one thread
        double run = excl_t;
        int y = live;
        for (int v = lo; v < hi; ++v) {
            run += exp(((double)logit(v) - m) / tau);
            if (run > t) { y = v; break; }
        }
        atomicMax(&q.chosen, y);
    }
    __syncthreads();
    int y = q.chosen;
    if (y < 0) y = q.last_live < 0 ? 0 : q.last_live;        // rounding left no stretch: the last token with a positive term
    return y;
}

// CTA (j, b) as in verify_kernel.  One pass over the row: warp w takes the segments w, w + 4, ...; a
// segment's terms 2^(x*c - E) (c = log2(e) / tau, E an integer just above the segment's largest exponent)
// are summed in single precision with ex2.approx and kept per segment, so the running sum is known in
// token order at segment granularity.  The exponent x*c is formed with c split into a 16-bit head and a
// tail: x is bf16, so x * head is exact, and the rounding of c does not grow with |x*c| (low temperatures).
// Then: a double-precision scan over the segments, the segment in which u*S falls, and inside that segment
// (512 logits, four per thread) double-precision exponentials and an exact scan.  What can differ from a
// double-precision inverse CDF over the whole row is the placement of u*S relative to a segment's start, by
// the rounding of the single-precision sums (a few 1e-7 of S).
__global__ void __launch_bounds__(kVerifyThreads)
verify_sampled_kernel(Workspace w, Params p, const uint16_t* __restrict__ target, const int32_t* __restrict__ root_token,
                      opt_tree_out tree, double tau, unsigned long long seed, unsigned long long step, int32_t* accept_len,
                      int32_t* accept_tokens, int32_t* accept_nodes, int32_t* next_root) {
    __shared__ VerifySmem s;
    __shared__ SampleSmem q;
    grid_dependency_wait();
    const int b = blockIdx.y, j = blockIdx.x, tid = threadIdx.x, lane = tid & 31, wp = tid >> 5;
    const int ns = tree.n_sel[b];
    if (j > ns) return;
    const int32_t* tok = tree.token + (size_t)b * p.n;
    const int32_t* par = tree.parent + (size_t)b * p.n;
    int token = j == 0 ? root_token[b] : tok[j - 1];
    const int depth = j == 0 ? 0 : tree.depth[(size_t)b * p.n + j - 1];
    if (token < 0 || token >= p.V) { set_status(w.status, kErrInternal); token = 0; }
    const uint16_t* row = target + (size_t)row_of(token, depth, p.H) * p.V;
    const double u = uniform53(seed, step, b, j);
    const int nv = p.V >> 3, nseg = (nv + kSegVecs - 1) / kSegVecs;
    const double c64 = kLog2eD / tau;
    bool fast = p.aligned != 0 && nseg <= kMaxSeg && c64 < 1e30;
    int y = 0;
    if (fast) {
        const float c32 = (float)c64;
        const float c_hi = __uint_as_float(__float_as_uint(c32) & 0xFFFFFF00u);      // 16 significant bits
        const float c_lo = (float)(c64 - (double)c_hi);
        const uint4* rv = reinterpret_cast<const uint4*>(row);
        if (tid == 0) { q.chosen = -1; q.last_live = -1; q.seg = 0x7FFFFFFF; q.live_seg = -1; }
        // two segments per turn: four 16-byte loads in flight per lane
        const unsigned long long chi2 = pack2(c_hi, c_hi), clo2 = pack2(c_lo, c_lo);
        constexpr int kStep = kVerifyThreads / 32;
#pragma unroll 1
        for (int sg0 = wp; sg0 < nseg; sg0 += 2 * kStep) {
            const uint4 pad = make_uint4(0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u);
            uint4 qq[2][2];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int v0 = (sg0 + h * kStep) * kSegVecs + lane, v1 = v0 + 32;
                qq[h][0] = v0 < nv ? ld_nc_v4(rv + v0) : pad;
                qq[h][1] = v1 < nv ? ld_nc_v4(rv + v1) : pad;
            }
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int sg = sg0 + h * kStep;
                if (sg >= nseg) break;                            // (warp-uniform)
                const uint32_t ww[8] = {qq[h][0].x, qq[h][0].y, qq[h][0].z, qq[h][0].w, qq[h][1].x, qq[h][1].y, qq[h][1].z, qq[h][1].w};
                uint32_t m2 = ww[0];
#pragma unroll
                for (int i = 1; i < 8; ++i) m2 = max_bf16x2(m2, ww[i]);
                const uint32_t wkey = __reduce_max_sync(0xFFFFFFFFu, max(ord16(m2 & 0xFFFFu), ord16(m2 >> 16)));
                float sum = 0.0f, Ef = 0.0f;
                if (wkey > kOrdNegInf) {                          // (warp-uniform) the segment holds a finite logit
                    const float fmx = bf16_bits_to_float(ord16_inv(wkey));
                    Ef = rintf(fminf(fmaxf(fmaf(fmx, c32, 1.0f), -1e9f), 1e9f));
                    const unsigned long long nE2 = pack2(-Ef, -Ef);
                    unsigned long long acc2 = 0ull;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const uint32_t cw = max_bf16x2(ww[i], 0xF149F149u);       // -inf -> -1e30: keeps the two-step product finite
                        const unsigned long long x2 = pack2(__uint_as_float(cw << 16), __uint_as_float(cw & 0xFFFF0000u));
                        float a0, a1;
                        unpack2(fma2(x2, clo2, fma2(x2, chi2, nE2)), a0, a1);
                        acc2 = add2(acc2, pack2(ex2_approx(a0), ex2_approx(a1)));
                    }
                    float s0, s1;
                    unpack2(acc2, s0, s1);
                    sum = s0 + s1;
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xFFFFFFFFu, sum, o);
                }
                if (lane == 0) { q.part[sg].sum = sum; q.part[sg].E = (int)Ef; }
            }
        }
        __syncthreads();
        int e = -0x7FFFFFFF;
        for (int sg = tid; sg < nseg; sg += kVerifyThreads) if (q.part[sg].sum > 0.0f) e = max(e, q.part[sg].E);
        e = __reduce_max_sync(0xFFFFFFFFu, e);
        if (lane == 0) q.wE[wp] = e;
        __syncthreads();
        int Eg = q.wE[0];
#pragma unroll
        for (int i = 1; i < kVerifyThreads / 32; ++i) Eg = max(Eg, q.wE[i]);
        fast = Eg > -kSampleExpLimit && Eg < kSampleExpLimit;                     // the same for every thread
        if (fast) {
            if (wp == 0) {                                    // running sums over the segments, in token order
                double carry = 0.0;
                for (int s0 = 0; s0 < nseg; s0 += 32) {
                    const int sg = s0 + lane;
                    double v = 0.0;
                    if (sg < nseg) { const SegPart pt = q.part[sg]; v = pt.sum > 0.0f ? ldexp((double)pt.sum, pt.E - Eg) : 0.0; }
                    double incl = v;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const double up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                        if (lane >= o) incl += up;
                    }
                    incl += carry;
                    __syncwarp();
                    if (sg < nseg) q.cum[sg] = incl;
                    carry = __shfl_sync(0xFFFFFFFFu, incl, 31);
                }
                if (lane == 0) q.S = carry;
            }
            __syncthreads();
            const double t = u * q.S;
            for (int sg = tid; sg < nseg; sg += kVerifyThreads) {
                const double c = q.cum[sg];
                if (c > t) atomicMin(&q.seg, sg);
                if (c > (sg > 0 ? q.cum[sg - 1] : 0.0)) atomicMax(&q.live_seg, sg);
            }
            __syncthreads();
            int sg = q.seg;
            if (sg == 0x7FFFFFFF) sg = q.live_seg < 0 ? 0 : q.live_seg;          // u*S rounded up to S: the last segment with a positive sum
            const double before = sg > 0 ? q.cum[sg - 1] : 0.0;
            // inside the segment: four logits per thread, double precision
            const int t0 = sg * kSegTokens + 4 * tid;
            double ev[4] = {0.0, 0.0, 0.0, 0.0};
            int live = -1;
            if (t0 < p.V) {                                   // V is a multiple of 8, so all four exist
                const uint2 x = *reinterpret_cast<const uint2*>(row + t0);
                const uint32_t h[4] = {x.x & 0xFFFFu, x.x >> 16, x.y & 0xFFFFu, x.y >> 16};
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float xf = bf16_bits_to_float(h[i]);
                    ev[i] = xf == -INFINITY ? 0.0 : exp2((double)xf * c64 - (double)Eg);
                    if (ev[i] > 0.0) live = t0 + i;
                }
            }
            const double mine = ((ev[0] + ev[1]) + ev[2]) + ev[3];
            double incl = mine;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const double up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                if (lane >= o) incl += up;
            }
            if (lane == 31) q.wsum[wp] = incl;
            __syncthreads();
            double base = before;                             // running sum where this warp's stretch begins (one fixed order)
            for (int i = 0; i < wp; ++i) base += q.wsum[i];
            double prev = __shfl_up_sync(0xFFFFFFFFu, incl, 1);
            if (lane == 0) prev = 0.0;
            const double excl_t = base + prev, incl_t = base + incl;
            atomicMax(&q.last_live, live);
            if (incl_t > t && !(excl_t > t)) {                // this thread's four logits: one thread
                double run = excl_t;
                int yy = live;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    run += ev[i];
                    if (run > t && ev[i] > 0.0) { yy = t0 + i; break; }
                }
                atomicMax(&q.chosen, yy);
            }
            __syncthreads();
            y = q.chosen;
            if (y < 0) y = q.last_live < 0 ? min(sg * kSegTokens, p.V - 1) : q.last_live;   // the exact sums end just below u*S: the segment's last live token
        }
    }
    if (!fast) y = sample_row_plain(q, row, p.V, p.aligned != 0, tau, u);
    verify_tail(s, w, p, b, j, ns, y, tok, par, accept_len, accept_tokens, accept_nodes, next_root);
}

// ------------------------------------------------------------------------------------------------
// Self-test of the bounded waits: one CTA whose warps each enter one kind of wait on something that
// nobody will ever complete or write (a fresh mbarrier, words that stay zero, a source that never has
// a row), with a limit of microseconds.  Every wait must give up, record kErrTimeout in its own
// status word and let the kernel end.  No bulk copy is in flight and nothing else runs in the CTA.
// ------------------------------------------------------------------------------------------------
struct NeverSource {
    static constexpr bool kHasEmpty = false;
    __device__ long long claim(int i) { return i; }
    __device__ int poll(long long, RowDesc&, bool) { return 0; }
};
__global__ void __launch_bounds__(kThreads)
wait_probe_kernel(int* result, const unsigned long long* zero_words, long long limit, int polls) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    CtaSmem& s = *reinterpret_cast<CtaSmem*>(smem_raw);
    pipeline_init(s.core, s.layer);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (warp == 0) {
        mbar_wait_warp(&s.core.full_bar[0], 0u, &result[0], limit);
    } else if (warp == 1) {
        if (lane == 0) mbar_wait_thread(&s.core.full_bar[1], 0u, &result[1], limit);
    } else if (warp == 2) {
        if (lane == 0) poll_phat_word(zero_words, &result[2], polls);
    } else if (warp == 3) {
        if (lane == 0) poll_tok_word(reinterpret_cast<const unsigned int*>(zero_words + 1), &result[3], polls);
    } else if (warp == 4) {
        NeverSource src;
        fetcher_role(s.core, src, &result[4], limit);
    }
}

}  // namespace ot

// ------------------------------------------------------------------------------------------------
// C ABI
// ------------------------------------------------------------------------------------------------
struct opt_tree_ctx {
    opt_tree_config cfg;
    ot::Workspace ws;
    void* base;
    size_t bytes;
    int device;
    int grid;              // resident CTAs of the persistent kernels (SMs x occupancy)
    size_t smem;           // dynamic shared memory of one such CTA (cta_smem_bytes(cfg.n))
    int mcap;
    int64_t launches;
    // pinned host staging of opt_tree_step_host: the step's inputs and outputs cross the bus in one
    // copy each and are spread to / gathered from the caller's arrays on the host
    char* hstage;
    size_t in_bytes, out_bytes;     // device ranges [h_root, end of h_base) and [o_token, end of o_next)
};

namespace {

bool valid_cfg(const opt_tree_config* c) {
    return c && c->V >= 1 && c->H >= 1 && c->n >= 1 && c->k >= 1 && c->max_depth >= 1 && c->max_batch >= 1;
}
int supported_cfg(const opt_tree_config* c) {
    if (c->n > OPT_TREE_MAX_N || c->k > OPT_TREE_MAX_K || c->k > c->V) return OPT_TREE_ERR_UNSUPPORTED;
    if ((long long)c->V * 31 + c->max_depth > 2147483647LL) return OPT_TREE_ERR_UNSUPPORTED;
    if (c->max_batch > 32767 || c->max_depth > 65535 || c->H > ot::kMaxTableRows) return OPT_TREE_ERR_UNSUPPORTED;
    if ((c->max_depth < c->n ? c->max_depth : c->n) > ot::kMaxLayers) return OPT_TREE_ERR_UNSUPPORTED;   // the mailbox item's layer field
    return OPT_TREE_OK;
}
ot::Params make_params(const opt_tree_ctx* ctx, const void* table, float delta) {
    const opt_tree_config& c = ctx->cfg;
    ot::Params p;
    p.V = c.V; p.H = c.H; p.n = c.n; p.k = c.k; p.kk = c.k < c.V ? c.k : c.V;
    p.Dcap = c.max_depth < c.n ? c.max_depth : c.n;
    p.max_depth = c.max_depth;
    p.B = 0;
    p.prune = 0;
    p.mcap = ctx->mcap;
    p.grid = ctx->grid;
    p.cstride = (int)ot::cand_stride(c.n, c.k);
    p.delta = delta;
    p.aligned = ((reinterpret_cast<uintptr_t>(table) & 15u) == 0 && (c.V % 8) == 0) ? 1 : 0;
    return p;
}
// Launches a kernel that may be set up while the kernel before it in the stream drains (every kernel of
// this library waits for its predecessor before it touches global memory, see grid_dependency_wait).
template <class... KArgs, class... Args>
void launch_after(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
bool bad_tree(const opt_tree_out* t) {
    return !t || !t->token || !t->parent || !t->depth || !t->phat || !t->n_sel || !t->depth_reached || !t->expected_len;
}
int check_launch() { return cudaGetLastError() == cudaSuccess ? OPT_TREE_OK : OPT_TREE_ERR_CUDA; }

}  // namespace

extern "C" {

// CTAs of the persistent kernels on the current device (one CTA of kThreads per SM as long as its
// shared memory fits); 0 if there is no usable device.
// Shared memory of a CTA of the persistent kernels for node budget n (one of two layouts).
static bool small_n(int n) { return n <= ot::kSmallN; }
static size_t cta_smem_bytes(int n) { return small_n(n) ? sizeof(ot::CtaSmemT<ot::kSmallN>) : sizeof(ot::CtaSmemT<ot::kMaxN>); }
static size_t layer_smem_bytes(int n) { return small_n(n) ? sizeof(ot::LayerScratchT<ot::kSmallN>) : sizeof(ot::LayerScratchT<ot::kMaxN>); }

static int persistent_grid(int n) {
    int dev = 0, per_sm = 0, sms = 0;
    constexpr int S = ot::kSmallN, L = ot::kMaxN;
    const auto dyn = cudaFuncAttributeMaxDynamicSharedMemorySize;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return 0; }
    if (cudaFuncSetAttribute(ot::build_kernel<false, S>, dyn, (int)sizeof(ot::CtaSmemT<S>)) != cudaSuccess ||
        cudaFuncSetAttribute(ot::build_kernel<true, S>, dyn, (int)sizeof(ot::CtaSmemT<S>)) != cudaSuccess ||
        cudaFuncSetAttribute(ot::build_kernel<false, L>, dyn, (int)sizeof(ot::CtaSmemT<L>)) != cudaSuccess ||
        cudaFuncSetAttribute(ot::build_kernel<true, L>, dyn, (int)sizeof(ot::CtaSmemT<L>)) != cudaSuccess ||
        cudaFuncSetAttribute(ot::row_topk_kernel, dyn, (int)sizeof(ot::CtaSmem)) != cudaSuccess ||
        cudaFuncSetAttribute(ot::layer_step_kernel<S>, dyn, (int)sizeof(ot::LayerScratchT<S>)) != cudaSuccess ||
        cudaFuncSetAttribute(ot::layer_step_kernel<L>, dyn, (int)sizeof(ot::LayerScratchT<L>)) != cudaSuccess ||
        (small_n(n) ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, ot::build_kernel<true, S>, ot::kThreads, sizeof(ot::CtaSmemT<S>))
                    : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, ot::build_kernel<true, L>, ot::kThreads, sizeof(ot::CtaSmemT<L>))) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    const int grid = per_sm * sms;
    return grid >= 1 && grid <= ot::kMaxGrid ? grid : 0;
}

size_t opt_tree_workspace_bytes(const opt_tree_config* cfg) {
    if (!valid_cfg(cfg) || supported_cfg(cfg) != OPT_TREE_OK) return 0;
    int grid = persistent_grid(cfg->n);
    if (grid == 0) grid = 148;                       // no device here: the size on a B200
    return ot::carve(*cfg, grid, nullptr, nullptr);
}

int opt_tree_create(opt_tree_ctx** out, const opt_tree_config* cfg) {
    if (!out) return OPT_TREE_ERR_INVALID_ARG;
    *out = nullptr;
    if (!valid_cfg(cfg)) return OPT_TREE_ERR_INVALID_ARG;
    int rc = supported_cfg(cfg);
    if (rc != OPT_TREE_OK) return rc;
    opt_tree_ctx* ctx = new (std::nothrow) opt_tree_ctx();
    if (!ctx) return OPT_TREE_ERR_CUDA;
    ctx->cfg = *cfg;
    ctx->launches = 0;
    ctx->grid = persistent_grid(cfg->n);
    ctx->smem = cta_smem_bytes(cfg->n);
    if (ctx->grid == 0) { delete ctx; return OPT_TREE_ERR_CUDA; }
    ctx->mcap = (int)ot::mailbox_capacity(*cfg, ctx->grid);
    ctx->bytes = ot::carve(*cfg, ctx->grid, nullptr, nullptr);
    if ((long long)ctx->mcap * ctx->grid > 0x7FFFFFFFLL) { delete ctx; return OPT_TREE_ERR_UNSUPPORTED; }
    if (cudaGetDevice(&ctx->device) != cudaSuccess || cudaMalloc(&ctx->base, ctx->bytes) != cudaSuccess) {
        cudaGetLastError();
        delete ctx;
        return OPT_TREE_ERR_CUDA;
    }
    ot::carve(*cfg, ctx->grid, static_cast<char*>(ctx->base), &ctx->ws);
    // (carve lays h_root, h_base out next to each other, and likewise o_token ... o_next)
    ctx->in_bytes = (size_t)(reinterpret_cast<char*>(ctx->ws.h_base + cfg->max_batch) - reinterpret_cast<char*>(ctx->ws.h_root));
    ctx->out_bytes = (size_t)(reinterpret_cast<char*>(ctx->ws.o_next + cfg->max_batch) - reinterpret_cast<char*>(ctx->ws.o_token));
    ctx->hstage = nullptr;
    if (cudaMemset(ctx->base, 0, ctx->bytes) != cudaSuccess ||
        cudaHostAlloc(reinterpret_cast<void**>(&ctx->hstage), ctx->in_bytes + ctx->out_bytes, cudaHostAllocDefault) != cudaSuccess) {
        cudaGetLastError();
        cudaFree(ctx->base);
        delete ctx;
        return OPT_TREE_ERR_CUDA;
    }
    *out = ctx;
    return OPT_TREE_OK;
}

int opt_tree_destroy(opt_tree_ctx* ctx) {
    if (!ctx) return OPT_TREE_ERR_INVALID_ARG;
    if (ctx->hstage) cudaFreeHost(ctx->hstage);
    cudaError_t e = cudaFree(ctx->base);
    delete ctx;
    return e == cudaSuccess ? OPT_TREE_OK : OPT_TREE_ERR_CUDA;
}

static int build_common(opt_tree_ctx* ctx, const void* draft, const int32_t* root_token, int32_t B, float delta,
                        const opt_tree_out* out, int prune, int32_t* rows_read, void* stream) {
    if (!ctx || !draft || !root_token || bad_tree(out) || B < 1 || delta != delta) return OPT_TREE_ERR_INVALID_ARG;
    if (B > ctx->cfg.max_batch) return OPT_TREE_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    ot::Params p = make_params(ctx, draft, delta);
    p.B = B;
    p.prune = prune;
    const long long init_threads = (long long)ctx->grid * ctx->mcap > B ? (long long)ctx->grid * ctx->mcap : B;
    launch_after(ot::init_build_kernel, dim3((unsigned)((init_threads + 255) / 256)), dim3(256), 0, st, ctx->ws, p, root_token);
    auto kernel = small_n(ctx->cfg.n) ? (prune ? ot::build_kernel<true, ot::kSmallN> : ot::build_kernel<false, ot::kSmallN>)
                                      : (prune ? ot::build_kernel<true, ot::kMaxN> : ot::build_kernel<false, ot::kMaxN>);
    launch_after(kernel, dim3(ctx->grid), dim3(ot::kThreads), ctx->smem, st, ctx->ws, p, static_cast<const uint16_t*>(draft), *out);
    ctx->launches += 2;
    int rc = check_launch();
    if (rc == OPT_TREE_OK && rows_read &&
        cudaMemcpy2DAsync(rows_read, sizeof(int32_t), ctx->ws.st + ot::kStRows, 8 * sizeof(int32_t), sizeof(int32_t), (size_t)B,
                          cudaMemcpyDeviceToDevice, st) != cudaSuccess)
        rc = OPT_TREE_ERR_CUDA;
    return rc;
}

int opt_tree_build(opt_tree_ctx* ctx, const void* draft, const int32_t* root_token, int32_t B, float delta,
                   const opt_tree_out* out, void* stream) {
    return build_common(ctx, draft, root_token, B, delta, out, 0, nullptr, stream);
}

int opt_tree_build_pruned(opt_tree_ctx* ctx, const void* draft, const int32_t* root_token, int32_t B, float delta,
                          const opt_tree_out* out, int32_t* rows_read, void* stream) {
    return build_common(ctx, draft, root_token, B, delta, out, 1, rows_read, stream);
}

int opt_tree_mask(opt_tree_ctx* ctx, const opt_tree_out* tree, int32_t B, const int32_t* base_pos, uint64_t* mask,
                  int32_t* position_ids, void* stream) {
    if (!ctx || bad_tree(tree) || !mask || !position_ids || B < 1 || B > ctx->cfg.max_batch) return OPT_TREE_ERR_INVALID_ARG;
    launch_after(ot::mask_kernel, dim3(B), dim3(ot::kSmallThreads), 0, static_cast<cudaStream_t>(stream),
                 tree->parent, tree->depth, tree->n_sel, base_pos, ctx->cfg.n, mask, position_ids, ctx->ws.status);
    ctx->launches++;
    return check_launch();
}

int opt_tree_verify(opt_tree_ctx* ctx, const opt_tree_out* tree, const void* target, const int32_t* root_token, int32_t B,
                    int32_t* accept_len, int32_t* accept_tokens, int32_t* accept_nodes, int32_t* next_root, void* stream) {
    if (!ctx || bad_tree(tree) || !target || !root_token || !accept_len || !accept_tokens || !accept_nodes || !next_root ||
        B < 1 || B > ctx->cfg.max_batch)
        return OPT_TREE_ERR_INVALID_ARG;
    const ot::Params p = make_params(ctx, target, 0.0f);
    launch_after(ot::verify_kernel, dim3(ctx->cfg.n + 1, B), dim3(ot::kVerifyThreads), 0, static_cast<cudaStream_t>(stream),
                 ctx->ws, p, static_cast<const uint16_t*>(target), root_token, *tree, accept_len, accept_tokens, accept_nodes, next_root);
    ctx->launches++;
    return check_launch();
}

int opt_tree_verify_sampled(opt_tree_ctx* ctx, const opt_tree_out* tree, const void* target, const int32_t* root_token, int32_t B,
                            double tau, uint64_t seed, uint64_t step, int32_t* accept_len, int32_t* accept_tokens,
                            int32_t* accept_nodes, int32_t* next_root, void* stream) {
    if (!ctx || bad_tree(tree) || !target || !root_token || !accept_len || !accept_tokens || !accept_nodes || !next_root ||
        B < 1 || B > ctx->cfg.max_batch || !(tau > 0.0))
        return OPT_TREE_ERR_INVALID_ARG;
    const ot::Params p = make_params(ctx, target, 0.0f);
    launch_after(ot::verify_sampled_kernel, dim3(ctx->cfg.n + 1, B), dim3(ot::kVerifyThreads), 0, static_cast<cudaStream_t>(stream),
                 ctx->ws, p, static_cast<const uint16_t*>(target), root_token, *tree, tau, (unsigned long long)seed,
                 (unsigned long long)step, accept_len, accept_tokens, accept_nodes, next_root);
    ctx->launches++;
    return check_launch();
}

int opt_tree_post_verify(opt_tree_ctx* ctx, const opt_tree_out* tree, const uint64_t* mask, const int32_t* accept_len,
                         const int32_t* accept_nodes, int32_t B, uint8_t* dense_mask, int32_t* kv_gather, int32_t* kv_keep,
                         void* stream) {
    if (!ctx || bad_tree(tree) || !mask || !accept_len || !accept_nodes || !dense_mask || !kv_gather || !kv_keep || B < 1 ||
        B > ctx->cfg.max_batch)
        return OPT_TREE_ERR_INVALID_ARG;
    launch_after(ot::post_verify_kernel, dim3(B), dim3(ot::kSmallThreads), 0, static_cast<cudaStream_t>(stream),
                 tree->n_sel, mask, accept_len, accept_nodes, ctx->cfg.n, ctx->cfg.max_depth, dense_mask, kv_gather, kv_keep,
                 ctx->ws.status);
    ctx->launches++;
    return check_launch();
}

int opt_tree_layers_begin(opt_tree_ctx* ctx, int32_t B, void* stream) {
    if (!ctx || B < 1 || B > ctx->cfg.max_batch) return OPT_TREE_ERR_INVALID_ARG;
    ot::Params p = make_params(ctx, nullptr, 0.0f);
    p.B = B;
    launch_after(ot::layers_begin_kernel, dim3((unsigned)((B + 127) / 128)), dim3(128), 0, static_cast<cudaStream_t>(stream), ctx->ws, p);
    ctx->launches++;
    return check_launch();
}

int opt_tree_layers_step(opt_tree_ctx* ctx, const void* frontier_logits, int32_t frontier_stride, int32_t B, float delta,
                         const opt_tree_out* out, int32_t* next_tokens, int32_t* next_parent, int32_t* next_count, void* stream) {
    if (!ctx || !frontier_logits || bad_tree(out) || !next_tokens || !next_parent || !next_count || B < 1 ||
        B > ctx->cfg.max_batch || frontier_stride < 1 || frontier_stride > ctx->cfg.n || delta != delta)
        return OPT_TREE_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    ot::Params p = make_params(ctx, frontier_logits, delta);
    p.B = B;
    const int nrows = B * frontier_stride;
    ot::Params pr = p;
    pr.H = nrows;                                            // the dense buffer is the "table" of the row step
    const int grid = nrows < ctx->grid ? nrows : ctx->grid;
    launch_after(ot::row_topk_kernel, dim3(grid), dim3(ot::kThreads), sizeof(ot::CtaSmem), st,
                 pr, static_cast<const uint16_t*>(frontier_logits), static_cast<const int32_t*>(nullptr), nrows, ctx->ws.rtok,
                 ctx->ws.rprob, ctx->ws.status);
    launch_after(small_n(ctx->cfg.n) ? ot::layer_step_kernel<ot::kSmallN> : ot::layer_step_kernel<ot::kMaxN>, dim3(B), dim3(ot::kTeam),
                 layer_smem_bytes(ctx->cfg.n), st, ctx->ws, p, frontier_stride, *out, next_tokens,
                 next_parent, next_count);
    ctx->launches += 2;
    return check_launch();
}

int opt_tree_row_softmax_topk(opt_tree_ctx* ctx, const void* logits, const int32_t* rows, int32_t nrows, int32_t* tok_out,
                              double* prob_out, void* stream) {
    if (!ctx || !logits || !rows || !tok_out || !prob_out || nrows < 0) return OPT_TREE_ERR_INVALID_ARG;
    if (nrows == 0) return OPT_TREE_OK;
    const ot::Params p = make_params(ctx, logits, 0.0f);
    const int grid = nrows < ctx->grid ? nrows : ctx->grid;
    ot::row_topk_kernel<<<grid, ot::kThreads, sizeof(ot::CtaSmem), static_cast<cudaStream_t>(stream)>>>(
        p, static_cast<const uint16_t*>(logits), rows, nrows, tok_out, prob_out, ctx->ws.status);
    ctx->launches++;
    return check_launch();
}

int opt_tree_step_host(opt_tree_ctx* ctx, const void* draft, const void* target, const int32_t* root_host,
                       const int32_t* base_host, int32_t B, float delta, const opt_tree_host_out* ho, void* stream) {
    if (!ctx || !draft || !target || !root_host || !ho || B < 1 || B > ctx->cfg.max_batch) return OPT_TREE_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const ot::Workspace& w = ctx->ws;
    const size_t n = ctx->cfg.n, D = ctx->cfg.max_depth, W = (ctx->cfg.n + 63) / 64, Bz = B;
    // inputs: one copy of the range that holds both device arrays
    char* hin = ctx->hstage;
    char* hout = ctx->hstage + ctx->in_bytes;
    const char* din = reinterpret_cast<const char*>(w.h_root);
    memcpy(hin, root_host, Bz * 4);
    if (base_host) memcpy(hin + (reinterpret_cast<const char*>(w.h_base) - din), base_host, Bz * 4);
    if (cudaMemcpyAsync(w.h_root, hin, ctx->in_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return OPT_TREE_ERR_CUDA;
    opt_tree_out t = {w.o_token, w.o_parent, w.o_depth, w.o_phat, w.o_nsel, w.o_dreach, w.o_elen, nullptr};
    int rc = opt_tree_build(ctx, draft, w.h_root, B, delta, &t, stream);
    if (rc == OPT_TREE_OK) rc = opt_tree_mask(ctx, &t, B, base_host ? w.h_base : nullptr, w.o_mask, w.o_pos, stream);
    if (rc == OPT_TREE_OK) rc = opt_tree_verify(ctx, &t, target, w.h_root, B, w.o_alen, w.o_atok, w.o_anode, w.o_next, stream);
    if (rc != OPT_TREE_OK) return rc;
    // outputs: one copy of the range that holds all result arrays, then each to the caller's array
    const char* dout = reinterpret_cast<const char*>(w.o_token);
    if (cudaMemcpyAsync(hout, dout, ctx->out_bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess)
        return OPT_TREE_ERR_CUDA;
#define OT_OUT(dst, src, bytes) if (dst) memcpy((dst), hout + (reinterpret_cast<const char*>(src) - dout), (bytes));
    OT_OUT(ho->token, w.o_token, Bz * n * 4) OT_OUT(ho->parent, w.o_parent, Bz * n * 4) OT_OUT(ho->depth, w.o_depth, Bz * n * 4)
    OT_OUT(ho->phat, w.o_phat, Bz * n * 8) OT_OUT(ho->n_sel, w.o_nsel, Bz * 4) OT_OUT(ho->depth_reached, w.o_dreach, Bz * 4)
    OT_OUT(ho->expected_len, w.o_elen, Bz * 8) OT_OUT(ho->mask, w.o_mask, Bz * n * W * 8) OT_OUT(ho->position_ids, w.o_pos, Bz * n * 4)
    OT_OUT(ho->accept_len, w.o_alen, Bz * 4) OT_OUT(ho->accept_tokens, w.o_atok, Bz * (D + 1) * 4)
    OT_OUT(ho->accept_nodes, w.o_anode, Bz * D * 4) OT_OUT(ho->next_root, w.o_next, Bz * 4)
#undef OT_OUT
    return OPT_TREE_OK;
}

int opt_tree_selftest_waits(opt_tree_ctx* ctx, int32_t* result, void* stream) {
    if (!ctx || !result) return OPT_TREE_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaFuncSetAttribute(ot::wait_probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(ot::CtaSmem)) != cudaSuccess ||
        cudaMemsetAsync(result, 0, OPT_TREE_SELFTEST_WAITS * sizeof(int32_t), st) != cudaSuccess ||
        cudaMemsetAsync(ctx->ws.rprob, 0, 2 * sizeof(unsigned long long), st) != cudaSuccess) {     // two words nobody writes
        cudaGetLastError();
        return OPT_TREE_ERR_CUDA;
    }
    ot::wait_probe_kernel<<<1, ot::kThreads, sizeof(ot::CtaSmem), st>>>(
        result, reinterpret_cast<const unsigned long long*>(ctx->ws.rprob), 1ll << 16, 1 << 10);
    ctx->launches++;
    return check_launch();
}

int opt_tree_last_device_status(opt_tree_ctx* ctx, int32_t* status_host) {
    if (!ctx || !status_host) return OPT_TREE_ERR_INVALID_ARG;
    if (cudaDeviceSynchronize() != cudaSuccess) return OPT_TREE_ERR_CUDA;
    if (cudaMemcpy(status_host, ctx->ws.status, 4, cudaMemcpyDeviceToHost) != cudaSuccess) return OPT_TREE_ERR_CUDA;
    if (cudaMemset(ctx->ws.status, 0, 4) != cudaSuccess) return OPT_TREE_ERR_CUDA;
    return OPT_TREE_OK;
}

int64_t opt_tree_launch_count(const opt_tree_ctx* ctx) { return ctx ? ctx->launches : 0; }

const char* opt_tree_strerror(int code) {
    switch (code) {
        case OPT_TREE_OK: return "ok";
        case OPT_TREE_ERR_INVALID_ARG: return "invalid argument";
        case OPT_TREE_ERR_UNSUPPORTED: return "unsupported configuration";
        case OPT_TREE_ERR_CUDA: return "CUDA runtime error";
        case OPT_TREE_ERR_TIMEOUT: return "device-side wait timed out";
        case OPT_TREE_ERR_INTERNAL: return "device-side bounds check failed";
        default: return "unknown error";
    }
}

}  // extern "C"

// ------------------------------------------------------------------------------------------------
// Verification without any allocation (opt_tree_verify_static).
// ------------------------------------------------------------------------------------------------
// The verify kernel needs three pieces of scratch: the target's best token per node, a per-sequence
// arrival counter and a status word.  A context keeps them in memory it got from cudaMalloc; this
// variant keeps them in the array below, which is part of the loaded library image on every GPU.
namespace {

constexpr size_t kStaticG = (size_t)OPT_TREE_STATIC_MAX_BATCH * (OPT_TREE_STATIC_MAX_N + 1);   // ints
constexpr size_t kStaticInts = kStaticG + OPT_TREE_STATIC_MAX_BATCH + 1;
constexpr size_t kStaticBytes = (kStaticInts * sizeof(int32_t) + 255) & ~(size_t)255;

static __device__ __align__(256) unsigned char g_verify_scratch[kStaticBytes];

constexpr int kMaxDevices = 64;
int32_t* g_scratch_addr[kMaxDevices];      // device address of g_verify_scratch on each device, once looked up

// The array's name means nothing to a kernel when used from host code; the device address comes from
// the runtime, once per device, with that device current.  No lock: two threads racing here both
// store the same value.
int static_scratch(int32_t** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return OPT_TREE_ERR_CUDA;
    if (!g_scratch_addr[dev]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_verify_scratch) != cudaSuccess || !ptr) {
            cudaGetLastError();
            return OPT_TREE_ERR_CUDA;
        }
        g_scratch_addr[dev] = static_cast<int32_t*>(ptr);
    }
    *out = g_scratch_addr[dev];
    return OPT_TREE_OK;
}

}  // namespace

extern "C" int opt_tree_verify_static(const opt_tree_config* cfg, const opt_tree_out* tree, const void* target,
                                      const int32_t* root_token, int32_t B, int32_t* accept_len, int32_t* accept_tokens,
                                      int32_t* accept_nodes, int32_t* next_root, int32_t* device_status, void* stream) {
    if (!cfg) return OPT_TREE_ERR_INVALID_ARG;
    opt_tree_config sized = *cfg;
    sized.max_batch = 1;                                     // this entry point does not look at max_batch
    if (!valid_cfg(&sized) || bad_tree(tree) || !target || !root_token || !accept_len || !accept_tokens || !accept_nodes ||
        !next_root || B < 1)
        return OPT_TREE_ERR_INVALID_ARG;
    if (supported_cfg(&sized) != OPT_TREE_OK) return OPT_TREE_ERR_UNSUPPORTED;
    if (B > OPT_TREE_STATIC_MAX_BATCH || cfg->n > OPT_TREE_STATIC_MAX_N) return OPT_TREE_ERR_UNSUPPORTED;
    int32_t* base = nullptr;
    const int rc = static_scratch(&base);
    if (rc != OPT_TREE_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    ot::Workspace ws;
    memset(&ws, 0, sizeof ws);
    ws.g = base;
    ws.vdone = base + kStaticG;
    ws.status = base + kStaticG + OPT_TREE_STATIC_MAX_BATCH;
    // counters and status start from zero whatever the previous call left behind
    if (cudaMemsetAsync(ws.vdone, 0, (OPT_TREE_STATIC_MAX_BATCH + 1) * sizeof(int32_t), st) != cudaSuccess) return OPT_TREE_ERR_CUDA;
    ot::Params p;
    memset(&p, 0, sizeof p);
    p.V = cfg->V; p.H = cfg->H; p.n = cfg->n; p.k = cfg->k; p.kk = cfg->k < cfg->V ? cfg->k : cfg->V;
    p.max_depth = cfg->max_depth; p.Dcap = cfg->max_depth < cfg->n ? cfg->max_depth : cfg->n;
    p.aligned = ((reinterpret_cast<uintptr_t>(target) & 15u) == 0 && (cfg->V % 8) == 0) ? 1 : 0;
    ot::verify_kernel<<<dim3(cfg->n + 1, B), ot::kVerifyThreads, 0, st>>>(
        ws, p, static_cast<const uint16_t*>(target), root_token, *tree, accept_len, accept_tokens, accept_nodes, next_root);
    if (cudaGetLastError() != cudaSuccess) return OPT_TREE_ERR_CUDA;
    if (device_status && cudaMemcpyAsync(device_status, ws.status, sizeof(int32_t), cudaMemcpyDeviceToDevice, st) != cudaSuccess)
        return OPT_TREE_ERR_CUDA;
    return OPT_TREE_OK;
}
