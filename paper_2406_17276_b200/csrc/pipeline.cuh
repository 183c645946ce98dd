// The persistent, warp-specialised row pipeline of one CTA.
//
//   producer warp   asks a Source for the next row, then streams that row's chunks into the ring
//                   (bulk async copies) as stages are handed back;
//   consumer warps  sample, threshold and make the fused pass over each row (row_topk.cuh), then
//                   hand the row's candidate list and partial sums to the finisher through one of
//                   two slots and go straight on to the next row;
//   finisher warp   computes the row's winners and gives them to a Sink (which may, for the tree
//                   build, select a layer and publish new rows).
//
// The chunks of consecutive rows form one stream: chunk g lives in stage g % kStages and is the
// (g / kStages)-th use of that stage, which fixes every mbarrier parity.  Every row has the same
// number of chunks (V is fixed).  All waits are bounded (common.cuh); a role that times out
// leaves its loop, and the others then time out on it in turn, so the CTA always ends.
#pragma once

#include "row_topk.cuh"

namespace ot {

__device__ __forceinline__ void pipeline_init(CtaSmem& s) {
    if (threadIdx.x == 0) {
        for (int i = 0; i < kStages; ++i) { mbar_init(&s.full_bar[i], 1); mbar_init(&s.empty_bar[i], kConsumerWarps); }
        for (int i = 0; i < 2; ++i) { mbar_init(&s.ready_bar[i], kConsumerWarps); mbar_init(&s.free_bar[i], 1); }
        s.slot[0].cand_count = 0;
        s.slot[1].cand_count = 0;
        mbar_fence_init();
    }
    __syncthreads();
}

// ---- producer warp -----------------------------------------------------------------------------
// Source::next(RowDesc&) is called by lane 0 only and returns false when there is no more work.
// With `aligned` false (table base or row pitch not 16-byte aligned) the whole warp copies the
// chunk with ordinary loads instead of a bulk copy.
template <class Source>
__device__ void producer_role(CtaSmem& s, Source& src, int V, bool aligned, int* status) {
    const int lane = threadIdx.x & 31;
    const int nchunks = (V + kChunkElems - 1) / kChunkElems;
    long long g = 0;
    for (int r = 0;; ++r) {
        RowDesc dsc;
        dsc.row = nullptr; dsc.b = dsc.d = dsc.slot = dsc.fsize = 0; dsc.stop = 0;
        int go = 0;
        if (lane == 0) go = src.next(dsc) ? 1 : 0;
        go = __shfl_sync(0xFFFFFFFFu, go, 0);
        const uint16_t* row = reinterpret_cast<const uint16_t*>(
            __shfl_sync(0xFFFFFFFFu, (unsigned long long)reinterpret_cast<uintptr_t>(dsc.row), 0));
        const int nc = go ? nchunks : 1;                       // the stop marker takes one (empty) chunk slot
        for (int c = 0; c < nc; ++c, ++g) {
            const int st = (int)(g % kStages);
            if (g >= kStages && !mbar_wait_warp(&s.empty_bar[st], (uint32_t)((g / kStages) - 1) & 1u, status)) return;
            if (c == 0 && lane == 0) {
                dsc.stop = go ? 0 : 1;
                s.desc[r % kDesc] = dsc;                       // published by the arrive below (release)
            }
            if (!go) {
                if (lane == 0) mbar_arrive(&s.full_bar[st]);
                return;
            }
            const int ne = chunk_elems(V, c);
            if (aligned) {
                if (lane == 0) {
                    mbar_expect_tx(&s.full_bar[st], (uint32_t)ne * 2u);
                    bulk_load(&s.stage[st][0], row + (size_t)c * kChunkElems, (uint32_t)ne * 2u, &s.full_bar[st]);
                }
            } else {
                const int padded = (ne + 7) & ~7;
                for (int e = lane; e < padded; e += 32)
                    s.stage[st][e] = e < ne ? __ldg(row + (size_t)c * kChunkElems + e) : (uint16_t)0xFF80u;
                __syncwarp();
                if (lane == 0) mbar_arrive(&s.full_bar[st]);
            }
        }
    }
}

// ---- consumer warps ----------------------------------------------------------------------------
__device__ void consumer_role(CtaSmem& s, int V, int k, int* status) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int kk = k < V ? k : V;
    const int nchunks = (V + kChunkElems - 1) / kChunkElems;
    int ns = (nchunks + 3) / 4;                               // sampled chunks: about a quarter of the row,
    ns = ns < 1 ? 1 : (ns > kStages - 1 ? kStages - 1 : ns);  // at least one, never the whole ring
    long long g = 0;
    for (int r = 0;; ++r) {
        const int sl = r & 1;
        RowSlot& slot = s.slot[sl];
        // first chunk of the row (or the stop marker)
        if (!mbar_wait_warp(&s.full_bar[g % kStages], (uint32_t)(g / kStages) & 1u, status)) return;
        const RowDesc dsc = s.desc[r % kDesc];
        if (r >= 2 && !mbar_wait_warp(&s.free_bar[sl], (uint32_t)((r >> 1) - 1) & 1u, status)) return;
        if (dsc.stop) {
            if (tid == 0) slot.desc = dsc;
            __syncwarp();
            if (lane == 0) mbar_arrive(&s.ready_bar[sl]);
            return;
        }
        // sampling pass: per-thread maxima over the first ns chunks
        uint32_t pm = 0xFF80FF80u;
        for (int c = 0; c < ns; ++c) {
            const int st = (int)((g + c) % kStages);
            if (c > 0 && !mbar_wait_warp(&s.full_bar[st], (uint32_t)((g + c) / kStages) & 1u, status)) return;
            pm = chunk_max(reinterpret_cast<const uint4*>(&s.stage[st][0]), (chunk_elems(V, c) + 7) >> 3, tid, pm);
        }
        const uint32_t tau_key = consumers_kth_largest(max(ord16(pm & 0xFFFFu), ord16(pm >> 16)), kk, s);
        const bool exact = tau_key <= kOrdNegInf;              // fewer than kk threads saw a finite logit
        const float tau = bf16_bits_to_float(ord16_inv(tau_key));
        const float c_tau = -tau * kLog2e;
        // fused pass
        double acc = 0.0;
        for (int c = 0; c < nchunks; ++c) {
            const int st = (int)((g + c) % kStages);
            if (c >= ns && !mbar_wait_warp(&s.full_bar[st], (uint32_t)((g + c) / kStages) & 1u, status)) return;
            if (!exact)
                acc += (double)chunk_pass(slot, reinterpret_cast<const uint4*>(&s.stage[st][0]), (chunk_elems(V, c) + 7) >> 3,
                                          (uint32_t)(c * kChunkElems), tid, tau, c_tau);
            __syncwarp();
            if (lane == 0) mbar_arrive(&s.empty_bar[st]);
        }
        g += nchunks;
        // hand the row to the finisher
        const double wsum = warp_sum(acc);
        if (lane == 0) slot.warp_part[warp] = wsum;
        if (tid == 0) { slot.desc = dsc; slot.tau_key = tau_key; }
        __syncwarp();
        if (lane == 0) mbar_arrive(&s.ready_bar[sl]);
    }
}

// ---- finisher warp -----------------------------------------------------------------------------
// Sink::row_done(const RowDesc&, const RowOut&) is called by the whole warp.
template <class Sink>
__device__ void finisher_role(CtaSmem& s, Sink& sink, int V, int k, int* status) {
    const int lane = threadIdx.x & 31;
    for (int r = 0;; ++r) {
        const int sl = r & 1;
        RowSlot& slot = s.slot[sl];
        if (!mbar_wait_warp(&s.ready_bar[sl], (uint32_t)(r >> 1) & 1u, status)) return;
        if (slot.desc.stop) return;
        RowOut out;
        finish_row_warp(s, slot, V, k, out);
        const RowDesc dsc = slot.desc;
        __syncwarp();
        if (lane == 0) { slot.cand_count = 0; mbar_arrive(&s.free_bar[sl]); }     // the slot can be refilled
        sink.row_done(dsc, out);
    }
}

template <class Source, class Sink>
__device__ __forceinline__ void run_pipeline(CtaSmem& s, Source& src, Sink& sink, int V, int k, bool aligned, int* status) {
    pipeline_init(s);
    const int warp = threadIdx.x >> 5;
    if (warp < kConsumerWarps) consumer_role(s, V, k, status);
    else if (warp == kProducerWarp) producer_role(s, src, V, aligned, status);
    else finisher_role(s, sink, V, k, status);
}

}  // namespace ot
