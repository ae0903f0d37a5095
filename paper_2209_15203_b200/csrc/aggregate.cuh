// Server step of Algorithm 1/2:  g = sum_{q=1..N} p_q Top_K(a^q),  summed in
// worker order so that the fp32 result does not depend on scheduling.
//
// The dense server buffer (one 32-bit word per coordinate, all zero between
// steps) is the scatter target.  Entry number e = q*K_up + slot of the uplink
// messages carries (coordinate j, value v) of worker q; the uplink selection
// files it under j as it emits it (see emit_entry), in one of two ways:
//
//   slots   (at most kSlotWorkers workers and a slot table that fits the budget)
//           head[j] keeps the first entry e0 to arrive: it owns the coordinate and
//           says so in its own mark word (next[e0], one word per entry).  Every later
//           entry marks next[e0] as shared, sets its worker's bit in the 128-bit mask
//           at the start of row e0 of the table and writes its value to its worker's
//           column of that row.  agg_reduce reads the marks in entry order — the
//           coordinate words themselves, scattered over a buffer far larger than L2,
//           are only written (back to zero).  An owner whose coordinate is not shared
//           has the whole sum in its own entry; a shared one reads the mask and then
//           the columns it names — independent loads, eight at a time — and adds
//           them, its own value at its own worker's place, in worker order.
//   chains  (otherwise)  next[e] = exchange(head[j], e+1); the entry at the head
//           of a chain walks it — dependent loads, one per sender — and puts
//           the terms in worker order.
//
// Either way the owner accumulates
//        g_j = fl(g_j + fl(p_q * v_{q,j}))        starting from +0,
// appends (j, g_j) to the union list U, puts the words it used back to zero, and
// — in unidirectional mode, where the downlink carries g itself — applies
// w_j <- w_j - alpha g_j  right there (last worker step of Algorithm 1).
// With the server memory of Algorithm 2 it adds the sum into delta instead.
// The work is O(N K_up); no pass over the d coordinates is ever made.
#pragma once

#include "common.cuh"

namespace tk {

constexpr int kSlotWorkers = 128;  // the slot table is used up to this many workers (its mask has 128 bits)

// Files every entry of a gathered message buffer under its coordinate — what the uplink
// selection's emission does on the fly when the messages are produced on this GPU.
// Also resets the union's state for the step.
__global__ void __launch_bounds__(256)
agg_link_kernel(const uint2* __restrict__ up, u32 total, u32 K_up, const float* __restrict__ p, u32* head, u32* next,
                u32* slots, u32 row_words, RowState* uni, Ctrl* ctrl, u32 d) {
    u32 e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e == 0) {
        uni->lo = 0; uni->cand_count = 0; uni->max_key = 0; uni->out_count = 0; uni->flags = 0;
        uni->sum_sq = 0.0; uni->sel_sq = 0.0; uni->nnz = 0;
    }
    // the downlink selection's first level wants a key no single worker's term lies below (union_bin):
    // here, with no row thresholds at hand, the smallest p_q * |v| itself (bin_base was set to the
    // largest value when the messages were produced, see reset_state)
    {
        u32 k = 0xffffffffu;
        if (e < total) k = key_of(__float_as_uint(__fmul_rn(p[e / K_up], __uint_as_float(up[e].y))));
        k = __reduce_min_sync(0xffffffffu, k);
        if (lane_id() == 0 && k != 0xffffffffu) atomicMin(&uni->bin_base, k);
    }
    if (e >= total) return;
    u32 j = up[e].x;
    if (j >= d) { raise_status(ctrl, -5); next[e] = 0; return; }
    if (slots) {
        file_in_slot(next, slots, row_words, atomicCAS(&head[j], 0u, e + 1), e, e / K_up, up[e].y);
    } else {
        next[e] = atomicExch(&head[j], e + 1);
    }
}

constexpr int kWindow = 128;  // consecutive workers whose terms one walk of a chain gathers (two 64-bit masks)

#ifndef TK_AGG_THREADS
#define TK_AGG_THREADS 256
#endif
constexpr int kAggThreads = TK_AGG_THREADS;
// all 2048 threads of an SM stay resident — the kernel lives on memory parallelism
__global__ void __launch_bounds__(kAggThreads, 2048 / kAggThreads)
agg_reduce_kernel(const uint2* __restrict__ up, u32 total, u32 K_up, const float* __restrict__ p,
                  u32* head, u32* next, u32* slots, u32 row_words, RowState* uni /* the union's state */,
                  uint2* U, u32 ucap, float* w, float alpha, int apply, float* delta, Ctrl* ctrl, u32 d,
                  int stats, u32* level0) {
    // level0, when given (kHistBins words of global memory, zero on entry): the sums' keys are also
    // counted by union_bin — the first level of the downlink selection, complete when this grid ends
    __shared__ u32 sh_hist[kHistBins];
    if (level0)
        for (int b = threadIdx.x; b < kHistBins; b += blockDim.x) sh_hist[b] = 0;
    dependency_wait();   // the entries are filed by the kernel before
    if (threadIdx.x == 0) phase_stamp(ctrl, kStampAggStart);
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        // once per step: may the rows of the next step start from this step's thresholds?  Not for a
        // while after a step in which a warm-started bound failed (2, 4, ... 1024 steps; see predict_kernel)
        u32 wait = uni->reuse_wait & 0xffffu, backoff = uni->reuse_wait >> 16;
        if (uni->reuse_fails) {
            backoff = backoff < 2u ? 2u : (backoff < 1024u ? backoff * 2u : 1024u);
            // an eighth of the rows or more at once is no accident: these vectors' thresholds do not hold still
            if ((u64)uni->reuse_fails * 8u * K_up >= total && backoff < 64u) backoff = 64u;
            wait = backoff;
            uni->reuse_fails = 0;
        } else if (uni->reuse_ok) {
            backoff >>= 1;
        }
        const bool allow = wait == 0u;
        if (wait) --wait;
        uni->reuse_ok = allow ? 1u : 0u;
        uni->reuse_wait = (backoff << 16) | wait;
    }
    const u32 bin_base = level0 ? union_base(uni) : 0u;
    u32 e = blockIdx.x * blockDim.x + threadIdx.x;
    bool owner = false;
    u32 j = 0, own_bits = 0;
    float acc = 0.0f;
    bool shared = false;
    float own_p = 0.0f;
    if (e < total) {
        uint2 mine = up[e];
        own_p = p[e / K_up];  // asked for now, not after the coordinate's word has come back
        j = mine.x;
        own_bits = mine.y;
        if (slots) {
            // this entry's mark says whether it owns its coordinate and whether others sent it too: no
            // look at the coordinate's own word, which sits in a buffer far larger than L2
            const u32 m = __ldcg(&next[e]);
            if (m) next[e] = 0;
            owner = (m & kMarkOwner) != 0 && j < d;
            shared = (m & kMarkShared) != 0;
        } else {
            owner = j < d && __ldcg(&head[j]) == e + 1;
        }
    }
    if (owner && slots) {
        const u32 own_q = e / K_up;
        if (!shared) {
            acc = __fadd_rn(acc, __fmul_rn(own_p, __uint_as_float(own_bits)));
        } else {
            u32* row = slots + (size_t)e * row_words;
            const uint4 m = __ldcg(reinterpret_cast<const uint4*>(row));
            u64 m0 = (u64)m.x | ((u64)m.y << 32), m1 = (u64)m.z | ((u64)m.w << 32);
            if (own_q < 64u) m0 |= 1ull << own_q;
            else m1 |= 1ull << (own_q - 64u);
            while (m0 | m1) {
                u32 qs[8], vs[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) {  // the next eight senders, their values all requested at once
                    qs[i] = 0xffffffffu;
                    if (m0) { qs[i] = (u32)__ffsll((long long)m0) - 1u; m0 &= m0 - 1; }
                    else if (m1) { qs[i] = (u32)__ffsll((long long)m1) + 63u; m1 &= m1 - 1; }
                    vs[i] = 0;
                    if (qs[i] == own_q) vs[i] = own_bits;
                    else if (qs[i] != 0xffffffffu) vs[i] = __ldcg(row + kSlotMaskWords + qs[i]);
                }
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    if (qs[i] == 0xffffffffu) continue;
                    acc = __fadd_rn(acc, __fmul_rn(p[qs[i]], __uint_as_float(vs[i])));
                    if (qs[i] != own_q) row[kSlotMaskWords + qs[i]] = 0;
                }
            }
            *reinterpret_cast<uint4*>(row) = make_uint4(0, 0, 0, 0);
        }
    } else if (owner) {  // chains
        // Entry ids grow with the worker (e = q*K_up + slot) and a worker sends a coordinate at most
        // once.  A walk of the chain is a string of dependent loads, the expensive part; each hop
        // also fetches the entry's value, so the two latencies overlap.  The values of the workers
        // in a window of kWindow consecutive numbers go into a small table with a bit mask saying
        // which are present; the terms are then added in ascending worker order.  With at most
        // kWindow workers that is a single walk; with more, one walk finds the first sender and
        // one walk per window that has senders follows.
        u32 byv[kWindow];
        u32 qlo = 0;  // workers below qlo are done
        if (total > (u32)kWindow * K_up) {
            u32 min_id = e;
            for (u32 c = next[e], hops = 0; c != 0 && hops <= total; c = next[c - 1], ++hops) min_id = min(min_id, c - 1);
            qlo = min_id / K_up;
        }
        for (u32 guard = 0; guard <= total; ++guard) {
            u64 m0 = 0, m1 = 0;
            u32 qnext = 0xffffffffu;
            for (u32 c = e + 1, hops = 0; c != 0 && hops <= total; ++hops) {
                const u32 id = c - 1;
                const u32 nx = next[id];
                const u32 v = up[id].y;
                const u32 q = id / K_up;
                if (q >= qlo) {
                    const u32 o = q - qlo;
                    if (o < (u32)kWindow) {
                        byv[o] = v;
                        if (o < 64u) m0 |= 1ull << o;
                        else m1 |= 1ull << (o - 64u);
                    } else {
                        qnext = min(qnext, q);
                    }
                }
                c = nx;
            }
            while (m0) {
                const int b = __ffsll((long long)m0) - 1;
                m0 &= m0 - 1;
                acc = __fadd_rn(acc, __fmul_rn(p[qlo + (u32)b], __uint_as_float(byv[b])));
            }
            while (m1) {
                const int b = __ffsll((long long)m1) + 63;
                m1 &= m1 - 1;
                acc = __fadd_rn(acc, __fmul_rn(p[qlo + (u32)b], __uint_as_float(byv[b])));
            }
            if (qnext == 0xffffffffu) break;
            qlo = qnext;
        }
    }
    if (owner) {
        head[j] = 0;
        if (apply) w[j] = __fsub_rn(w[j], __fmul_rn(alpha, acc));
        // server memory (Algorithm 2): g = sum + delta, kept in the memory until the downlink
        // selection takes its Top_K out of it
        if (delta) delta[j] = __fadd_rn(acc, delta[j]);
    }
    // append (j, g_j) to the union list: one counter update per CTA (every entry of every worker
    // passes through here; per-warp atomics on the one word would serialise)
    __shared__ u32 sh_scratch[33];
    __shared__ u32 sh_base;
    u32 bits = __float_as_uint(acc);
    u32 owners;
    u32 incl = block_inclusive_scan(owner ? 1u : 0u, sh_scratch, &owners);
    if (level0) {
        // the sums crowd into a few bins: one shared-memory atomic per distinct bin and warp
        // (the scan above has passed a barrier since sh_hist was cleared)
        const u32 bin = union_bin(key_of(bits), bin_base);
        const u32 peers = __match_any_sync(0xffffffffu, owner ? bin : 0xffffffffu);
        if (owner && (int)lane_id() == __ffs(peers) - 1) atomicAdd(&sh_hist[bin], (u32)__popc(peers));
    } else if (ucap <= 4096u) {
        // a union this small is selected from by a single CTA, which wants the largest aggregated
        // magnitude as the upper end of its first range instead of the counts
        u32 wm = __reduce_max_sync(0xffffffffu, owner ? key_of(bits) : 0u);
        if (lane_id() == 0 && wm) atomicMax(&uni->max_key, wm);
    }
    if (threadIdx.x == 0 && owners) sh_base = atomicAdd(&uni->cand_count, owners);
    __syncthreads();
    if (owner) {
        u32 slot = sh_base + incl - 1;
        if (slot < ucap) U[slot] = make_uint2(j, bits);
    }
    if (level0)
        for (int b = threadIdx.x; b < kHistBins; b += blockDim.x)
            if (sh_hist[b]) atomicAdd(&level0[b], sh_hist[b]);
    if (stats) {  // diagnostics: non-zeros of the aggregate (Section 4.2) and its squared norm
        u32 nz = __reduce_add_sync(0xffffffffu, (owner && key_of(bits) != 0) ? 1u : 0u);
        if (lane_id() == 0 && nz) atomicAdd(&uni->nnz, nz);
        warp_add_double(&uni->sum_sq, owner ? (double)acc * (double)acc : 0.0);
    }
    if (TK_PHASE_CLOCK) {
        __syncthreads();
        if (threadIdx.x == 0) phase_stamp(ctrl, kStampAggEnd);
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
