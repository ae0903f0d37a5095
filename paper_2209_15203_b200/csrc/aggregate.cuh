// Server step of Algorithm 1/2:  g = sum_{q=1..N} p_q Top_K(a^q),  summed in
// worker order so that the fp32 result does not depend on scheduling.
//
// The dense server buffer (one 32-bit word per coordinate, all zero between
// steps) is the scatter target: the uplink selection, as it emits entry number
// e = q*K_up + slot with coordinate j, threads it onto j's chain
// (next[e] = exchange(head[j], e+1), see emit_entry); agg_reduce lets the entry at the
// head of each chain walk it in ascending worker order, accumulate
//        g_j = fl(g_j + fl(p_q * v_{q,j}))        starting from +0,
// append (j, g_j) to the union list U, put the word back to zero, and — in
// unidirectional mode, where the downlink carries g itself — apply
// w_j <- w_j - alpha g_j  right there (last worker step of Algorithm 1).
// With the server memory of Algorithm 2 it adds the sum into delta instead.
// The work is O(N K_up); no pass over the d coordinates is ever made.
#pragma once

#include "common.cuh"

namespace tk {

// Threads every entry of a gathered message buffer onto its coordinate's chain — what the
// uplink selection's emission does on the fly when the messages are produced on this GPU.
// Also resets the union's state for the step.
__global__ void __launch_bounds__(256)
agg_link_kernel(const uint2* __restrict__ up, u32 total, u32* head, u32* next, RowState* uni, Ctrl* ctrl, u32 d) {
    u32 e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e == 0) {
        uni->lo = 0; uni->cand_count = 0; uni->max_key = 0; uni->out_count = 0; uni->flags = 0;
        uni->sum_sq = 0.0; uni->sel_sq = 0.0; uni->nnz = 0;
    }
    if (e >= total) return;
    u32 j = up[e].x;
    if (j >= d) { raise_status(ctrl, -5); next[e] = 0; return; }
    next[e] = atomicExch(&head[j], e + 1);
}

__global__ void __launch_bounds__(256)
agg_reduce_kernel(const uint2* __restrict__ up, u32 total, u32 K_up, const float* __restrict__ p,
                  u32* head, const u32* __restrict__ next, RowState* uni /* the union's state */,
                  uint2* U, u32 ucap, float* w, float alpha, int apply, float* delta, Ctrl* ctrl, u32 d,
                  int stats) {
    dependency_wait();   // the chains are built by the kernel before
    u32 e = blockIdx.x * blockDim.x + threadIdx.x;
    bool owner = false;
    u32 j = 0;
    float acc = 0.0f;
    if (e < total) {
        j = up[e].x;
        owner = j < d && __ldcg(&head[j]) == e + 1;
    }
    if (owner) {
        // walk the chain once per term, each time taking the smallest worker not yet added
        int last_q = -1;
        for (u32 guard = 0; guard <= total; ++guard) {
            int best_q = 0x7fffffff;
            u32 best_e = 0;
            for (u32 c = e + 1, hops = 0; c != 0 && hops <= total; c = next[c - 1], ++hops) {
                int q = (int)((c - 1) / K_up);
                if (q > last_q && q < best_q) { best_q = q; best_e = c - 1; }
            }
            if (best_q == 0x7fffffff) break;
            float term = __fmul_rn(p[best_q], __uint_as_float(up[best_e].y));
            acc = __fadd_rn(acc, term);
            last_q = best_q;
        }
        head[j] = 0;
        if (apply) w[j] = __fsub_rn(w[j], __fmul_rn(alpha, acc));
        // server memory (Algorithm 2): g = sum + delta, kept in the memory until the downlink
        // selection takes its Top_K out of it
        if (delta) delta[j] = __fadd_rn(acc, delta[j]);
    }
    // append (j, g_j) to the union list: one counter update and one maximum per CTA (every entry
    // of every worker passes through here; per-warp atomics on the two words would serialise)
    __shared__ u32 sh_scratch[33];
    __shared__ u32 sh_base, sh_max;
    if (threadIdx.x == 0) sh_max = 0;
    u32 bits = __float_as_uint(acc);
    u32 owners;
    u32 incl = block_inclusive_scan(owner ? 1u : 0u, sh_scratch, &owners);
    u32 wm = __reduce_max_sync(0xffffffffu, owner ? key_of(bits) : 0u);
    if (lane_id() == 0 && wm) atomicMax(&sh_max, wm);
    __syncthreads();
    if (threadIdx.x == 0 && owners) {
        sh_base = atomicAdd(&uni->cand_count, owners);
        atomicMax(&uni->max_key, sh_max);  // the downlink selection wants the largest aggregated magnitude
    }
    __syncthreads();
    if (owner) {
        u32 slot = sh_base + incl - 1;
        if (slot < ucap) U[slot] = make_uint2(j, bits);
    }
    if (stats) {  // diagnostics: non-zeros of the aggregate (Section 4.2) and its squared norm
        u32 nz = __reduce_add_sync(0xffffffffu, (owner && key_of(bits) != 0) ? 1u : 0u);
        if (lane_id() == 0 && nz) atomicAdd(&uni->nnz, nz);
        warp_add_double(&uni->sum_sq, owner ? (double)acc * (double)acc : 0.0);
    }
}

// ---- helpers of the inspection calls (not on the per-step path) ----

// Entries of `sel` with a non-zero magnitude go to msg; flags[idx] = 1 marks the ones below `limit`.
__global__ void msg_collect_kernel(const uint2* sel, u32 n, uint2* msg, u32* msg_count,
                                   unsigned char* flags, u32 limit) {
    u32 i = blockIdx.x * blockDim.x + threadIdx.x;
    bool pred = false;
    uint2 e = make_uint2(0, 0);
    if (i < n) {
        e = sel[i];
        pred = key_of(e.y) != 0;
        if (pred && e.x < limit) flags[e.x] = 1;
    }
    warp_append(pred, e.x, e.y, msg_count, msg, 0xffffffffu);
}

// Append the first `pad` indices j in [0, limit) with flags[j] == 0 as (j, +0.0).  One CTA.
__global__ void __launch_bounds__(1024)
msg_pad_kernel(const unsigned char* flags, u32 limit, u32 pad, uint2* msg, u32 at) {
    __shared__ u32 scratch[33];
    u32 done = 0;
    for (u32 base = 0; base < limit && done < pad; base += blockDim.x) {
        u32 j = base + threadIdx.x;
        u32 free_ = (j < limit && flags[j] == 0) ? 1u : 0u;
        u32 total;
        u32 incl = block_inclusive_scan(free_, scratch, &total);
        u32 rank = done + incl - free_;
        if (free_ && rank < pad) msg[at + rank] = make_uint2(j, 0u);
        done += total;
        __syncthreads();
    }
}

}  // namespace tk
