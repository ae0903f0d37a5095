// Everything of a step that follows the streaming pass, as ONE cooperatively launched kernel
// (clusters of `cs` CTAs, 1 CTA per SM), so that what used to be launch boundaries between
// latency-bound kernels are grid-wide barriers:
//
//   V  verification + exact fallback     general_body: exits at once when every row verified
//   S  uplink selection                  one cluster per row (clusters take rows in turn),
//                                        the emission files every entry under its coordinate
//      -- grid barrier --
//   A  server sum over the union         agg_block, one entry per thread
//      -- grid barrier --
//   D  downlink selection + update       the whole grid selects from the union list
//
// (Algorithm 1/2: SEND(Top_K(a^q)); g = sum_q p_q Top_K(a^q); SEND(Top_K(g)); w <- w - message.)
// Any subset of the phases can be asked for; a plain batched selection is V+S.
#pragma once

#include "aggregate.cuh"
#include "select.cuh"

namespace tk {

constexpr int kTailThreads = 1024;
static_assert(kTailThreads == kSelectThreads && kTailThreads == kGeneralThreads, "one block shape for all phases");

enum : int { kPhaseVerify = 1, kPhaseSelect = 2, kPhaseAggregate = 4, kPhaseDownlink = 8 };

struct TailArgs {
    int phases;
    Ctrl* ctrl;
    // V + S: batched selection over `rows` rows of x
    const float* x;
    int rows;
    int64_t d;
    u32 K;
    u32 tpr;          // tiles of kGeneralTileVecs float4 per row
    u32 cap;
    RowState* rs;
    u32* hist;
    uint2* cand;
    uint2* out;       // [rows][K]
    ApplyArgs apply_up;
    LinkArgs link;
    int stats;
    // A: the server sum
    const uint2* up;  // [total] uplink entries
    u32 total, K_up;
    const float* p;
    u32* head;
    u32* next;
    u32* slots;
    u32 row_words;
    RowState* uni;
    uint2* U;
    u32 ucap;
    float* w;
    float alpha;
    int apply_uni;
    float* delta;
    u32 d32;
    // D: downlink selection over the union
    u32 K_down;
    uint2* sel;
    ApplyArgs apply_down;
    u32* ghist;
};

union TailShared {
    GeneralShared gen;
    SelectShared sel;
    AggShared agg;
};

__global__ void __launch_bounds__(kTailThreads, 1) tail_kernel(const __grid_constant__ TailArgs a) {
    extern __shared__ __align__(16) unsigned char tail_smem[];
    TailShared& sh = *reinterpret_cast<TailShared*>(tail_smem);
    cg::grid_group grid = cg::this_grid();
    cg::cluster_group cluster = cg::this_cluster();
    dependency_wait();   // lists, bounds and messages come from the kernels before
    allow_dependents();
    const bool stamper = threadIdx.x == 0;
    if (stamper) phase_stamp(a.ctrl, kStampTailStart);
    const DenseArgs no_dense = {nullptr, nullptr, 0};
    if (a.phases & kPhaseVerify) {
        general_body(sh.gen, a.x, a.rows, a.d, a.K, a.tpr, a.cap, a.rs, a.hist, a.cand, a.ctrl, a.stats);
        __syncthreads();  // the shared memory changes hands
        if (stamper) phase_stamp(a.ctrl, kStampVerified);
    }
    if (a.phases & kPhaseSelect) {
        const u32 cs = cluster.num_blocks();
        const u32 nclusters = gridDim.x / cs, cid = blockIdx.x / cs;
        for (u32 row = cid; row < (u32)a.rows; row += nclusters) {
            select_body<false, false>(sh.sel, row, a.cand, a.cap, a.cap, a.rs, a.K, a.out, (size_t)a.K, a.apply_up, a.link,
                                      a.ctrl, nullptr, no_dense, false);
            __syncthreads();
        }
        if (stamper) phase_stamp(a.ctrl, kStampSelected);
    }
    if (a.phases & kPhaseAggregate) {
        if (a.phases & (kPhaseVerify | kPhaseSelect)) grid.sync();  // every entry is filed
        if (stamper) phase_stamp(a.ctrl, kStampSelectedAll);
        agg_phase<kTailThreads>(sh.agg, a.up, a.total, a.K_up, a.p, a.head, a.next, a.slots, a.row_words, a.uni, a.U, a.ucap,
                                a.w, a.alpha, a.apply_uni, a.delta, a.ctrl, a.d32, a.stats,
                                (a.phases & kPhaseDownlink) ? a.ghist : nullptr);
        if (stamper) phase_stamp(a.ctrl, kStampAggregated);
    }
    if (a.phases & kPhaseDownlink) {
        if (a.phases & kPhaseAggregate) grid.sync();  // the union list is complete
        if (stamper) phase_stamp(a.ctrl, kStampAggregatedAll);
        LinkArgs nolink = {nullptr, nullptr, 0, 0, nullptr, 0, a.stats, nullptr, 0};
        select_body<true, false>(sh.sel, 0, a.U, a.ucap, a.ucap, a.uni, a.K_down, a.sel, (size_t)a.ucap, a.apply_down, nolink,
                                 a.ctrl, a.ghist, no_dense, (a.phases & kPhaseAggregate) != 0);
    }
    if (stamper) phase_stamp(a.ctrl, kStampDone);
}

}  // namespace tk
