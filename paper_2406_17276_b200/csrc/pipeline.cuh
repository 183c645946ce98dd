// The persistent, warp-specialised row pipeline of one CTA.
//
//   fetcher warp    asks a Source for row descriptors, several at a time and ahead of the
//                   consumers, so that the latency of obtaining work (a mailbox entry, an index load)
//                   is hidden, and hands them on in the order in which they become known;
//   issuer warp     streams each described row's chunks into the ring (bulk async copies) as
//                   stages are handed back;
//   consumer warps  make the fused pass over each row (row_topk.cuh), then hand the row's
//                   per-thread maxima and partial sums to a finisher through a slot and go
//                   straight on to the next row;
//   finisher warps  row r goes to finisher r mod kFinishers: it computes the row's winners and
//                   gives them to a Sink (for the tree build: candidates' path values and the
//                   layer's row counter);
//   layer warp      runs Sink::layer_loop (for the tree build: watches the row counters of its
//                   sequences, selects each next layer and publishes its rows); its assistants
//                   run Sink::layer_assist and share the selection's work.
//
// The chunks of consecutive rows form one stream: chunk g lives in stage g % kStages and is the
// (g / kStages)-th use of that stage, which fixes every mbarrier parity; likewise row r uses
// descriptor r % kDesc and slot r % kSlots.  Every row has the same number of chunks (V is fixed).
// All waits are bounded (common.cuh); a role that times out leaves its loop, and the others then
// time out on it in turn, so the CTA always ends.  The one wait without a clock is the layer team's
// barrier: the assistants sit there between jobs, and the layer warp, whose own waits are all
// bounded, reaches it however it leaves its loop (it then posts a last job that sends them home).
#pragma once

#include "row_topk.cuh"

namespace ot {

template <class LS>
__device__ __forceinline__ void pipeline_init(CtaCore& s, LS& layer) {
    if (threadIdx.x == 0) {
        for (int i = 0; i < kStages; ++i) { mbar_init(&s.full_bar[i], 1); mbar_init(&s.empty_bar[i], kConsumerWarps); }
        for (int i = 0; i < kSlots; ++i) { mbar_init(&s.ready_bar[i], kConsumerWarps); mbar_init(&s.free_bar[i], 1); }
        for (int i = 0; i < kDesc; ++i) { mbar_init(&s.desc_full[i], 1); mbar_init(&s.desc_empty[i], kConsumerWarps); }
        s.stop_row = 0x7FFFFFFF;
        mbar_fence_init();
    }
    for (int i = threadIdx.x; i < 3 * 256; i += kThreads) (&layer.thist[0][0])[i] = 0;
    if (threadIdx.x == 0) { layer.cache_b = -1; layer.cache_d = -1; }
    __syncthreads();
}

// ---- fetcher warp ------------------------------------------------------------------------------
// Obtaining a row costs global-memory round trips (a mailbox entry, an index load) that
// take about as long as streaming the row, so kFetchLanes lanes hold one ticket each and poll
// concurrently; the warp stays converged in one polling loop so that the lanes' round trips
// overlap.  Rows are handed on in the order in which they become known (the a-th known row goes to
// descriptor a % kDesc), never in ticket order: a ticket whose item is published late must not hold
// up a row that is ready.  Tickets are only taken while fewer than kDesc rows are between "ticket
// taken" and "descriptor read by the consumers", which bounds what a CTA keeps from the others.
//   Source::claim(i)          ticket for this CTA's i-th claim, or a negative value: no more work
//   Source::poll(ticket, dsc) 1: descriptor filled, 0: not yet, 2: the ticket turned out empty, -1: no more work
// Once a Source has said "no more work" no ticket of this CTA can still turn into a row.
constexpr int kFetchLanes = 4;
template <class Source>
__device__ void fetcher_role(CtaCore& s, Source& src, int* status, long long limit = kWaitCycles) {
    const int lane = threadIdx.x & 31;
    const unsigned below = (1u << lane) - 1u;
    bool holding = false;                 // this lane has a ticket
    long long ticket = 0;
    int claimed = 0, known = 0, consumed = 0;      // warp-uniform counts of this CTA's rows
    int consumed_empty = 0;                        // tickets that turned out empty
    long long t0 = clock64();
    for (int turn = 0;; ++turn) {
        // rows whose descriptors the consumers have let go of
        while (consumed < known && mbar_test_wait(&s.desc_empty[consumed % kDesc], (uint32_t)(consumed / kDesc) & 1u)) ++consumed;
        // new tickets, as far as the bound allows
        const bool want = lane < kFetchLanes && !holding;
        const unsigned wm = __ballot_sync(0xFFFFFFFFu, want);
        const int my_claim = claimed + __popc(wm & below);
        const bool take = want && my_claim - consumed_empty - consumed < kDesc;
        if (take) { ticket = src.claim(my_claim); holding = true; }
        claimed += __popc(__ballot_sync(0xFFFFFFFFu, take));
        // one poll per held ticket
        RowDesc dsc;
        dsc.row = nullptr; dsc.pphat = 0.0; dsc.b = dsc.d = dsc.slot = dsc.fsize = 0; dsc.stop = 0;
        int got = 0;
        if (holding) got = ticket < 0 ? -1 : src.poll(ticket, dsc, (turn & 15) == 15);
        if (Source::kHasEmpty) {   // an entry that was handed out but not needed: the ticket is gone, and does not count as a row in hand
            const bool empty = got == 2;
            if (empty) { holding = false; got = 0; }
            consumed_empty += __popc(__ballot_sync(0xFFFFFFFFu, empty));
        }
        const unsigned rm = __ballot_sync(0xFFFFFFFFu, got > 0), em = __ballot_sync(0xFFFFFFFFu, got < 0);
        if (got > 0) {
            const int a = known + __popc(rm & below);
            s.desc[a % kDescRing] = dsc;
            mbar_arrive(&s.desc_full[a % kDesc]);              // release: publishes the descriptor
            holding = false;
        }
        known += __popc(rm);
        if (em) {                                              // no more work: one stop marker after the last row
            if (lane == __ffs(em) - 1) {
                dsc.stop = 1;
                s.desc[known % kDescRing] = dsc;
                mbar_arrive(&s.desc_full[known % kDesc]);
            }
            return;
        }
        if (rm) t0 = clock64();
        else {
            if ((turn & 63) == 63 && clock64() - t0 > limit) { set_status(status, kErrTimeout); return; }
            __nanosleep(100);
        }
    }
}

// ---- issuer warp -------------------------------------------------------------------------------
// A chunk of a row that bulk copies cannot take (see issuer_role), by the whole warp; rare, out of line.
__device__ __noinline__ void copy_chunk_plain(uint16_t* stage, const uint16_t* src, int ne) {
    const int lane = threadIdx.x & 31;
    const int padded = (ne + 7) & ~7;
    for (int i = lane; i < padded; i += 32) stage[i] = i < ne ? __ldg(src + i) : (uint16_t)0xFF80u;
    __syncwarp();
}

// With `aligned` false (table base or row pitch not 16-byte aligned) the whole warp copies the
// chunk with ordinary loads instead of a bulk copy.
__device__ void issuer_role(CtaCore& s, int V, bool aligned, int* status) {
    const int lane = threadIdx.x & 31;
    const int nchunks = (V + kChunkElems - 1) / kChunkElems;
    long long g = 0;
    for (int r = 0;; ++r) {
        const int e = r % kDesc;
        if (!mbar_wait_warp(&s.desc_full[e], (uint32_t)(r / kDesc) & 1u, status)) return;
        const uint16_t* row = s.desc[r % kDescRing].row;
        const int go = s.desc[r % kDescRing].stop ? 0 : 1;
        const int nc = go ? nchunks : 1;                       // the stop marker takes one (empty) chunk slot
        for (int c = 0; c < nc; ++c, ++g) {
            const int st = (int)(g % kStages);
            if (g >= kStages && !mbar_wait_warp(&s.empty_bar[st], (uint32_t)((g / kStages) - 1) & 1u, status)) return;
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
                copy_chunk_plain(&s.stage[st][0], row + (size_t)c * kChunkElems, ne);
                if (lane == 0) mbar_arrive(&s.full_bar[st]);
            }
        }
    }
}

// ---- consumer warps ----------------------------------------------------------------------------
// A warp takes its share of a chunk out of the ring into registers and hands the stage back at once
// (so the issuer can refill it while the exponentials run); a row's descriptor is only looked at for
// its stop flag.
__device__ void consumer_role(CtaCore& s, int cwarp, int V, int* status) {
    const int lane = threadIdx.x & 31, tid = cwarp * 32 + lane;     // index among the consumer threads
    const int nchunks = (V + kChunkElems - 1) / kChunkElems;
    ThreadAcc acc;
    acc.reset();
    ChunkRegs ch;
    long long g = 0;
    for (int r = 0;; ++r) {
        for (int c = 0; c < nchunks; ++c, ++g) {
            const int st = (int)(g % kStages);
            if (!mbar_wait_warp(&s.full_bar[st], (uint32_t)(g / kStages) & 1u, status)) return;
            if (c == 0) {
                if (s.desc[r % kDescRing].stop) {
                    if (tid == 0) s.stop_row = r;                  // the finishers poll this
                    return;
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&s.desc_empty[r % kDesc]);      // this warp has looked at the descriptor
            }
            chunk_take(ch, reinterpret_cast<const uint4*>(&s.stage[st][0]), (chunk_elems(V, c) + 7) >> 3, tid);
            __syncwarp();
            if (lane == 0) mbar_arrive(&s.empty_bar[st]);          // the data is in registers: the stage is free
            chunk_chain(ch);
            const unsigned long long C2 = chunk_apply(acc, ch);
            chunk_exps(acc, ch, C2);
        }
        // hand the row to its finisher
        const int sl = r % kSlots;
        if (r >= kSlots && !mbar_wait_warp(&s.free_bar[sl], (uint32_t)((r / kSlots) - 1) & 1u, status)) return;
        store_thread_result(s.slot[sl], acc, tid);
        __syncwarp();
        if (lane == 0) mbar_arrive(&s.ready_bar[sl]);
        acc.reset();
    }
}

// ---- finisher warps ----------------------------------------------------------------------------
// Sink::row_done(const RowDesc&, const RowOut&, FinScratch&) is called by the whole warp.
template <class Sink>
__device__ void finisher_role(CtaCore& s, Sink& sink, int fidx, int V, int k, bool aligned, int* status) {
    const int lane = threadIdx.x & 31;
    FinScratch& f = s.fin[fidx];
    for (int r = fidx;; r += kFinishers) {
        const int sl = r % kSlots;
        const uint32_t parity = (uint32_t)(r / kSlots) & 1u;
        // wait for the row, or learn that the stream ended before it (every lane polls)
        if (!mbar_try_wait(&s.ready_bar[sl], parity)) {
            long long t0 = 0;
            int turns = 0, ok = 1;
            while (!mbar_try_wait(&s.ready_bar[sl], parity)) {
                if (s.stop_row <= r) { ok = 0; break; }
                if ((++turns & 255) == 0) {
                    const long long now = clock64();
                    if (t0 == 0) t0 = now;
                    else if (now - t0 > kWaitCycles) { set_status(status, kErrTimeout); ok = 0; break; }
                }
            }
            if (!__all_sync(0xFFFFFFFFu, ok)) return;
        }
        const RowSlot& slot = s.slot[sl];
        const RowDesc dsc = s.desc[r % kDescRing];
        RowOut out;
        finish_row_warp(f, slot, dsc.row, V, k, aligned, out);
        __syncwarp();
        if (lane == 0) mbar_arrive(&s.free_bar[sl]);                              // the slot can be refilled
        sink.row_done(dsc, out, f);
    }
}

template <class Smem, class Source, class Sink>
__device__ __forceinline__ void run_pipeline(Smem& sm, Source& src, Sink& sink, int V, int k, bool aligned, int* status) {
    CtaCore& s = sm.core;
    pipeline_init(s, sm.layer);
    grid_dependency_wait();                                // shared memory is set up; global memory from here on
    const int warp = threadIdx.x >> 5;
    if (warp < kConsumerWarps) { consumer_role(s, warp, V, status); return; }
    const int helper = warp - kConsumerWarps;
    if (helper == kHelperIssuer) issuer_role(s, V, aligned, status);
    else if (helper == kHelperFetcher) fetcher_role(s, src, status);
    else if (helper == kHelperLayer) sink.layer_loop(sm.layer);
    else if (helper < kHelperFirstFinisher) sink.layer_assist(sm.layer, helper - kHelperLayer);
    else finisher_role(s, sink, helper - kHelperFirstFinisher, V, k, aligned, status);
}

}  // namespace ot
