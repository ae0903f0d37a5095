// Batched exact Top_K selection (Section 1's compressor; the uplink and downlink
// steps of Algorithm 1/2) as four kernels:
//
//   predict_kernel   reads a small strided sample of every row and sets a
//                    conservative lower bound `lo` on the K-th composite key — or
//                    keeps the bound that served the row's last selection well
//   filter_kernel    the one streaming pass over all rows*d values: appends every
//                    component with ck >= lo to the row's candidate list and
//                    counts them exactly (tiles dealt out in advance, the last few
//                    of each range claimed from a counter)
//   general_kernel   verification + exact fallback.  A row whose count is below
//                    K or above the list capacity (or every row, when no
//                    prediction was made) gets its bound from full-row radix
//                    histograms (11+11+9 key bits, then 11+11+10 index bits, as
//                    far as needed) and is filtered again.  Exits at once when
//                    every row verified.
//   select_kernel    one thread-block cluster per row (or, for one long list, the
//                    whole grid): range-adaptive radix select of the K largest
//                    composite keys among the candidates, then emission of
//                    exactly K entries.  Few short rows skip the three kernels
//                    above: the same kernel takes every component of the row
//                    as a candidate.
//
// The result is always the exact Top_K; the sample only decides how many
// passes over the data it takes.
#pragma once

#include "common.cuh"

namespace tk {

// ---------------------------------------------------------------------------
// predict: sample -> lower bound
// ---------------------------------------------------------------------------
// The sample of a row is `lines` runs of 32 consecutive values (one 128-byte
// line each: DRAM delivers whole lines, so narrower runs cost the same traffic)
// spread evenly over the row (run g starts at (g * stride_fp) >> 32, rounded
// down to a multiple of 32).  Eight neighbouring threads share a line, 4 values
// each; a thread issues all its `turns` loads at once (the kernel is a chain of
// DRAM latencies otherwise).  Every pair of threads keeps the largest key it
// saw: kSampleSlots maxima per row.  The last CTA of the row to finish takes a
// lower bound of the `rank`-th largest maximum — exact in its leading 22 bits,
// which costs two histogram passes instead of four — as the row's bound: at
// least `rank` sampled values are >= it.
//
// Bound reuse.  Consecutive steps of a training run have close thresholds.  Every selection of
// a row leaves the key of its K-th largest magnitude (prev_T_key) and a decaying maximum of how
// far that key moved between consecutive selections (drift); the next selection's bound is that
// key minus a margin of four times the drift — at least kReuseMinMargin keys, 1.5-3 % in value —
// and with `reuse` set the row's CTAs return at once: no sample is read, nothing is ranked.  A
// row whose threshold wanders gets a wider margin (more candidates); when four times the drift
// exceeds kReuseMaxMargin (25-50 %) the row is sampled as usual.  The result stays exact either
// way: the bound is verified by the exact count like a sampled one, and a row whose count falls
// below K or above the list's capacity is redone by the multi-pass path in the same step, after
// which it is sampled for the next 2, 4, ... 64 selections before a warm start is tried again.
// Within a step of a context the back-off is shared by all rows (`gate`, the union's state,
// updated once per step by the server sum): with many rows whose thresholds jump now and then
// — tie groups around the K-th value — a failed attempt then costs one step in up to 1024,
// not one row in every step.
constexpr u32 kReuseMinMargin = 1u << 18;   // keys; a key step is 2^-23 .. 2^-24 of the value
constexpr u32 kReuseMaxMargin = 1u << 22;
constexpr u32 kReuseFirstDrift = 1u << 17;  // assumed before two thresholds have been seen
__device__ __forceinline__ void reset_state(RowState* r, u64 lo, u32 flags) {
    r->lo = lo;
    r->cand_count = 0;
    r->max_key = 0;
    r->out_count = 0;
    r->flags = flags;
    r->ticket = 0;
    r->tile_ticket = 0;
    r->bin_base = 0xffffffffu;
    r->g_active = 0;
    r->sum_sq = 0.0;
    r->sel_sq = 0.0;
    r->nnz = 0;
}

// kLight: at most kPredictLightTurns loads per thread; needs half the registers, so two CTAs
// fit an SM (used when the rows are many and the sample per row is small).
template <bool kEF, bool kLight>
__global__ void __launch_bounds__(kPredictThreads, kLight ? 2 : 1)
predict_kernel(const float* __restrict__ x, int64_t d, int turns, u64 stride_fp, u32 rank, u32 K,
               RowState* rs, u32* smax, RowState* also_reset, EfArgs ef, Ctrl* ctrl, int reuse,
               const RowState* gate) {
    __shared__ u32 sh_hist[kHistBins];
    __shared__ u32 sh_scratch[33];
    __shared__ u32 sh_res[2];
    __shared__ u32 sh_ticket;
    allow_dependents();  // the filter kernel may take its place on the SMs; it waits for this grid to end
    if (threadIdx.x == 0) phase_stamp(ctrl, kStampPredictStart);
    const int row = blockIdx.y;
    const u32 t = blockIdx.x * kPredictThreads + threadIdx.x;   // 0 .. 2*kSampleSlots-1
    if (also_reset && row == 0 && t == 0) reset_state(also_reset, 0ull, 0u);
    // (the same answer in all CTAs of the row: nothing in this kernel writes either word)
    if (reuse && rs[row].reuse_ok && (!gate || gate->reuse_ok)) {
        if (t == 0) {
            reset_state(rs + row, (u64)rs[row].next_lo_key << 32, kRowReused);
            phase_stamp(ctrl, kStampPredictEnd);
        }
        return;
    }
    const float* xr = x + (size_t)row * (size_t)d;
    const float* er = kEF ? ef.eps + (size_t)row * (size_t)d : nullptr;
    // runs start at multiples of 32 elements
    const bool vec_ok = (((uintptr_t)xr) & 15u) == 0 && (!kEF || (((uintptr_t)er) & 15u) == 0);
    constexpr u32 kLinesPerTurn = 2 * kSampleSlots / 8;
    // two loads per turn with memories
    constexpr int kTurns = kLight ? (kEF ? kPredictLightTurns / 2 : kPredictLightTurns)
                                  : (kEF ? kPredictMaxTurns / 2 : kPredictMaxTurns);
    uint4 v[kTurns], m[kEF ? kTurns : 1];
#pragma unroll
    for (int k = 0; k < kTurns; ++k) {
        v[k] = make_uint4(0, 0, 0, 0);
        if (kEF) m[k] = make_uint4(0, 0, 0, 0);
        if (k < turns) {
            u64 g = (u64)(t >> 3) + (u64)k * kLinesPerTurn;
            u64 e = (((g * stride_fp) >> 32) & ~31ull) + 4u * (t & 7u);
            if (vec_ok) {
                v[k] = ld_stream(reinterpret_cast<const uint4*>(xr + e));
                if (kEF) m[k] = ld_stream(reinterpret_cast<const uint4*>(er + e));
            } else {
                v[k] = make_uint4(__float_as_uint(__ldg(xr + e)), __float_as_uint(__ldg(xr + e + 1)),
                                  __float_as_uint(__ldg(xr + e + 2)), __float_as_uint(__ldg(xr + e + 3)));
                if (kEF)
                    m[k] = make_uint4(__float_as_uint(__ldg(er + e)), __float_as_uint(__ldg(er + e + 1)),
                                      __float_as_uint(__ldg(er + e + 2)), __float_as_uint(__ldg(er + e + 3)));
            }
        }
    }
    if (kEF) {
#pragma unroll
        for (int k = 0; k < kTurns; ++k) {
            v[k].x = compensated(v[k].x, m[k].x, ef.alpha);
            v[k].y = compensated(v[k].y, m[k].y, ef.alpha);
            v[k].z = compensated(v[k].z, m[k].z, ef.alpha);
            v[k].w = compensated(v[k].w, m[k].w, ef.alpha);
        }
    }
    u32 mx = 0;
#pragma unroll
    for (int k = 0; k < kTurns; ++k)
        mx = max(mx, max(max(key_of(v[k].x), key_of(v[k].y)), max(key_of(v[k].z), key_of(v[k].w))));
    mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
    if ((t & 1u) == 0) smax[(size_t)row * kSampleSlots + (t >> 1)] = mx;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) sh_ticket = atomicAdd(&rs[row].ticket, 1u);
    __syncthreads();
    if (sh_ticket != kPredictCtas - 1) {
        if (threadIdx.x == 0) phase_stamp(ctrl, kStampPredictEnd);
        return;
    }
    __threadfence();

    // last CTA of the row: the rank-th largest of the kSampleSlots maxima, to 22 leading bits
    constexpr int PER = kSampleSlots / kPredictThreads;
    const volatile u32* vm = smax + (size_t)row * kSampleSlots;
    u32 mine[PER];
#pragma unroll
    for (int i = 0; i < PER; ++i) mine[i] = vm[threadIdx.x + i * kPredictThreads];
    u32 prefix = 0, need = rank;
    for (int pass = 0; pass < 2; ++pass) {
        const int shift = pass == 0 ? 20 : 9;           // key bits 30..20, then 19..9
        for (int b = threadIdx.x; b < kHistBins; b += kPredictThreads) sh_hist[b] = 0;
        if (threadIdx.x == 0) sh_res[0] = 0xffffffffu;
        __syncthreads();
#pragma unroll
        for (int i = 0; i < PER; ++i) {
            // the maxima crowd into a few bins: one shared-memory atomic per distinct bin and warp
            u32 val = mine[i];
            bool ok = pass == 0 || (val >> 20) == (prefix >> 20);
            u32 bin = (val >> shift) & (u32)(kHistBins - 1);
            u32 peers = __match_any_sync(0xffffffffu, ok ? bin : 0xffffffffu);
            if (ok && (int)lane_id() == __ffs(peers) - 1) atomicAdd(&sh_hist[bin], (u32)__popc(peers));
        }
        __syncthreads();
        u32 b, above;
        find_bucket<kHistBins / kPredictThreads>(sh_hist, kHistBins, need, sh_scratch, sh_res, &b, &above);
        if (b == 0xffffffffu) { b = 0; above = 0; }     // cannot happen (rank <= kSampleSlots)
        prefix |= b << shift;
        need -= above;
    }
    // A bound of key 0 means the row is nearly all zeros.  Taking every component would overflow the
    // list; (key 0, index K-1) is a valid bound as well: it admits every non-zero and the zeros among
    // the first K components, and if fewer than K components are non-zero, the first K components
    // hold enough zeros to make up the difference (zeros rank by ascending index).
    u64 lo = (u64)prefix << 32;
    if (prefix == 0) lo = composite(0u, K - 1u);
    if (threadIdx.x == 0) {
        reset_state(rs + row, lo, 0u);
        phase_stamp(ctrl, kStampPredictEnd);
    }
}

// eps <- eps + alpha * g over n values (the compensated vector, for the paths that do not
// fuse it into the filter pass).
__global__ void __launch_bounds__(256) compensate_kernel(float* eps, const float* __restrict__ g, float alpha, size_t n) {
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
        eps[i] = __fadd_rn(eps[i], __fmul_rn(alpha, __ldg(g + i)));
}

// No prediction: mark every row for the multi-pass path.
__global__ void reset_rows_kernel(RowState* rs, int rows, RowState* also_reset) {
    int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r < rows) reset_state(rs + r, ~0ull, kRowGeneral | kRowNoFilter);
    if (also_reset && r == 0) reset_state(also_reset, 0ull, 0u);
}

// ---------------------------------------------------------------------------
// filter: the streaming pass
// ---------------------------------------------------------------------------
// Geometry of one row: `head` scalar components up to the first 16-byte
// boundary, then nv float4, then `tail` scalars.
struct RowGeom {
    const float* base;
    const uint4* vec;
    u32 head, tail;
    u32 nv;
};

__device__ __forceinline__ RowGeom row_geom(const float* x, int row, int64_t d) {
    RowGeom g;
    g.base = x + (size_t)row * (size_t)d;
    u32 mis = (u32)(((uintptr_t)g.base >> 2) & 3u);
    u32 head = (4u - mis) & 3u;
    if ((int64_t)head > d) head = (u32)d;
    g.head = head;
    g.nv = (u32)((d - head) >> 2);
    g.tail = (u32)(d - head - 4 * (int64_t)g.nv);
    g.vec = reinterpret_cast<const uint4*>(g.base + head);
    return g;
}

// Candidates are first collected per warp in shared memory and appended to the
// row's list in batches: hits cluster in the layers with the largest scale, and
// one global atomic per hit on the row's single counter would serialise there.
#ifndef TK_COOP_PDL
#define TK_COOP_PDL 1
#endif
#ifndef TK_FILTER_DYN_MIN
#define TK_FILTER_DYN_MIN 32
#endif
#ifndef TK_STAGE_SLOTS
#define TK_STAGE_SLOTS 128
#endif
constexpr int kStageSlots = TK_STAGE_SLOTS;  // per warp; at least 32 (128 measured 0.3-0.7 % faster per step than 64)

struct WarpStage {
    uint2* buf;  // this warp's kStageSlots entries
    u32* n;      // this warp's fill count
};

__device__ __forceinline__ WarpStage warp_stage(uint2* sh_buf, u32* sh_n) {
    WarpStage st;
    u32 warp = threadIdx.x >> 5;
    st.buf = sh_buf + warp * kStageSlots;
    st.n = sh_n + warp;
    return st;
}

// Append the warp's staged entries to the row's candidate list.  All lanes call.
__device__ __forceinline__ void stage_flush(const WarpStage& st, RowState* rs, uint2* cand, u32 cap) {
    u32 n = *st.n;
    if (n == 0) return;
    u32 lane = lane_id(), base = 0, mx = 0;
    if (lane == 0) base = atomicAdd(&rs->cand_count, n);
    base = __shfl_sync(0xffffffffu, base, 0);
    for (u32 i = lane; i < n; i += 32) {
        uint2 e = st.buf[i];
        mx = max(mx, key_of(e.y));
        if (base + i < cap) cand[base + i] = e;
    }
    mx = __reduce_max_sync(0xffffffffu, mx);
    if (lane == 0) atomicMax(&rs->max_key, mx);
    __syncwarp();
    if (lane == 0) *st.n = 0;
    __syncwarp();
}

// One component in the rare path: stage it if ck >= lo.  All lanes call.
__device__ __forceinline__ void consider(bool live, u32 idx, u32 bits, u64 lo, const WarpStage& st,
                                         RowState* rs, uint2* cand, u32 cap) {
    bool pred = live && composite(key_of(bits), idx) >= lo;
    u32 m = __ballot_sync(0xffffffffu, pred);
    if (m == 0) return;
    u32 cnt = (u32)__popc(m);
    if (*st.n + cnt > kStageSlots) stage_flush(st, rs, cand, cap);
    u32 n = *st.n;
    u32 lane = lane_id();
    if (pred) st.buf[n + (u32)__popc(m & ((1u << lane) - 1u))] = make_uint2(idx, bits);
    __syncwarp();
    if (lane == 0) *st.n = n + cnt;
    __syncwarp();
}

// The four components of one float4 per lane, with at least one hit somewhere in the warp:
// stage all qualifying components with a single update of the warp's fill count.
__device__ __forceinline__ void consider4(uint4 v, u32 i0, u32 tk, u64 lo, const WarpStage& st,
                                          RowState* rs, uint2* cand, u32 cap) {
    bool p0 = key_of(v.x) >= tk, p1 = key_of(v.y) >= tk, p2 = key_of(v.z) >= tk, p3 = key_of(v.w) >= tk;
    if ((u32)lo != 0u) {  // the bound reaches into the index bits (multi-pass path only): exact test
        p0 = p0 && composite(key_of(v.x), i0 + 0) >= lo;
        p1 = p1 && composite(key_of(v.y), i0 + 1) >= lo;
        p2 = p2 && composite(key_of(v.z), i0 + 2) >= lo;
        p3 = p3 && composite(key_of(v.w), i0 + 3) >= lo;
    }
    const u32 m0 = __ballot_sync(0xffffffffu, p0), m1 = __ballot_sync(0xffffffffu, p1);
    const u32 m2 = __ballot_sync(0xffffffffu, p2), m3 = __ballot_sync(0xffffffffu, p3);
    const u32 c0 = (u32)__popc(m0), c1 = (u32)__popc(m1), c2 = (u32)__popc(m2), c3 = (u32)__popc(m3);
    const u32 cnt = c0 + c1 + c2 + c3;
    if (cnt == 0) return;
    if (cnt > kStageSlots) {  // more than the stage holds (needs > 16 hits per component on average)
        consider(p0, i0 + 0, v.x, 0ull, st, rs, cand, cap);
        consider(p1, i0 + 1, v.y, 0ull, st, rs, cand, cap);
        consider(p2, i0 + 2, v.z, 0ull, st, rs, cand, cap);
        consider(p3, i0 + 3, v.w, 0ull, st, rs, cand, cap);
        return;
    }
    if (*st.n + cnt > kStageSlots) stage_flush(st, rs, cand, cap);
    const u32 n = *st.n;
    const u32 lt = (1u << lane_id()) - 1u;
    if (p0) st.buf[n + (u32)__popc(m0 & lt)] = make_uint2(i0 + 0, v.x);
    if (p1) st.buf[n + c0 + (u32)__popc(m1 & lt)] = make_uint2(i0 + 1, v.y);
    if (p2) st.buf[n + c0 + c1 + (u32)__popc(m2 & lt)] = make_uint2(i0 + 2, v.z);
    if (p3) st.buf[n + c0 + c1 + c2 + (u32)__popc(m3 & lt)] = make_uint2(i0 + 3, v.w);
    __syncwarp();
    if (lane_id() == 0) *st.n = n + cnt;
    __syncwarp();
}

// Cheap per-float4 pre-test: could any of the four components have key >= tk?  Done in
// floating point (|x| >= thr with thr = the float whose bits are tk; "not less than", so
// that a NaN on either side passes) because the absolute value is free there.  It may
// pass too much, never too little; the staging code repeats the test exactly on the keys.
__device__ __forceinline__ bool may_hit(uint4 v, float thr) {
    // bitwise, not short-circuit: four compares and no branches
    return (!(fabsf(__uint_as_float(v.x)) < thr)) | (!(fabsf(__uint_as_float(v.y)) < thr)) |
           (!(fabsf(__uint_as_float(v.z)) < thr)) | (!(fabsf(__uint_as_float(v.w)) < thr));
}

// Process tile `tile` (THREADS * UNROLL float4) of a row.  All THREADS threads of the CTA call.
// With kEF the row's memory `erow` is read as well, the compensated vector a = eps + alpha*g
// is what gets filtered, and it is written back to the memory (the entries sent later are
// zeroed there by the selection's emission: eps <- a - Top_K(a)).
// With kStats the squares of all values of the tile are added to `sq` (per thread, fp32).
template <int THREADS, int UNROLL, bool kEF, bool kStats>
__device__ __forceinline__ void filter_tile(const RowGeom& g, u32 tile, u64 lo, const WarpStage& st,
                                            RowState* rs, uint2* cand, u32 cap, float* erow, float alpha,
                                            float& sq) {
    const u32 tk = (u32)(lo >> 32);
    const float thr = __uint_as_float(tk);
    const u32 j0 = tile * (THREADS * UNROLL) + threadIdx.x;
    const uint4* p = g.vec + j0;
    uint4* pe = kEF ? reinterpret_cast<uint4*>(erow + g.head) + j0 : nullptr;
    uint4 v[UNROLL];
    uint4 m[kEF ? UNROLL : 1];
    bool inb[UNROLL];
    const bool full = (tile + 1) * (u32)(THREADS * UNROLL) <= g.nv;
    if (full) {
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            v[u] = ld_stream(p + u * THREADS);
            if (kEF) m[u] = ld_once(pe + u * THREADS);
            inb[u] = true;
        }
    } else {
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            inb[u] = j0 + u * THREADS < g.nv;
            v[u] = inb[u] ? ld_stream(p + u * THREADS) : make_uint4(0, 0, 0, 0);
            if (kEF) m[u] = inb[u] ? ld_once(pe + u * THREADS) : make_uint4(0, 0, 0, 0);
        }
    }
    if (kEF) {
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            v[u].x = compensated(v[u].x, m[u].x, alpha);
            v[u].y = compensated(v[u].y, m[u].y, alpha);
            v[u].z = compensated(v[u].z, m[u].z, alpha);
            v[u].w = compensated(v[u].w, m[u].w, alpha);
            if (inb[u]) __stcs(pe + u * THREADS, v[u]);
            else v[u] = make_uint4(0, 0, 0, 0);
        }
    }
    if (kStats) {  // lanes outside the row hold zeros
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) sq = sq4(v[u], sq);
    }
    if (tk != 0) {
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            bool hit = inb[u] && may_hit(v[u], thr);
            // padding lanes hold zeros, whose key is below tk
            if (__any_sync(0xffffffffu, hit)) consider4(v[u], g.head + 4u * (j0 + u * THREADS), tk, lo, st, rs, cand, cap);
        }
    } else {
        // key 0 in the bound (a row of nearly all zeros, or one where everything qualifies): every
        // non-zero passes, and the zeros up to the bound's index; exact test per component
        const u32 last_zero = 0xffffffffu - (u32)lo;
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const u32 i0 = g.head + 4u * (j0 + u * THREADS);
            bool hit = inb[u] && ((((v[u].x | v[u].y | v[u].z | v[u].w) & 0x7fffffffu) != 0u) || i0 <= last_zero);
            if (__any_sync(0xffffffffu, hit)) {
                consider(hit, i0 + 0, v[u].x, lo, st, rs, cand, cap);
                consider(hit, i0 + 1, v[u].y, lo, st, rs, cand, cap);
                consider(hit, i0 + 2, v[u].z, lo, st, rs, cand, cap);
                consider(hit, i0 + 3, v[u].w, lo, st, rs, cand, cap);
            }
        }
    }
    if (tile == 0 && threadIdx.x < 32 && (g.head | g.tail)) {
        u32 lane = threadIdx.x;
        bool live = false;
        u32 idx = 0;
        if (lane < g.head) { live = true; idx = lane; }
        else if (lane >= 8 && lane - 8 < g.tail) { live = true; idx = g.head + 4u * g.nv + (lane - 8); }
        u32 bits = live ? __float_as_uint(__ldg(g.base + idx)) : 0u;
        if (kEF && live) {
            bits = compensated(bits, __float_as_uint(erow[idx]), alpha);
            erow[idx] = __uint_as_float(bits);
        }
        if (kStats && live) sq = fmaf(__uint_as_float(bits), __uint_as_float(bits), sq);
        consider(live, idx, bits, lo, st, rs, cand, cap);
    }
}

// The tile space (row-major: all tiles of row 0, then row 1, ...) is cut into `parts`
// equal contiguous ranges; `cpp` CTAs share a range and interleave its tiles.  With one
// range every CTA would visit every row, and each change of row costs a flush of the
// staged candidates (a global atomic round trip); with one range per CTA a CTA that
// lands in a layer full of candidates would finish late.
template <bool kEF, bool kStats>
__global__ void __launch_bounds__(kFilterThreads, kFilterCtasPerSm)
filter_kernel(const float* __restrict__ x, int rows, int64_t d, u32 tpr, u32 parts, u32 cpp,
              RowState* rs, uint2* cand, u32 cap, EfArgs ef, Ctrl* ctrl) {
    constexpr int kUnroll = kEF ? kFilterEfUnroll : kFilterUnroll;
    extern __shared__ u64 sh_lo[];  // every row's bound, fetched once
    __shared__ uint2 sh_buf[(kFilterThreads / 32) * kStageSlots];
    __shared__ u32 sh_n[kFilterThreads / 32];
    __shared__ u32 sh_claim[2];
    const u32 part = blockIdx.x / cpp;
#if TK_COOP_PDL
    allow_dependents();
#endif
    if (part >= parts) return;
    dependency_wait();  // the bounds and the zeroed tickets come from the sampling kernel
    if (threadIdx.x == 0) phase_stamp(ctrl, kStampFilterStart);
    for (int r = threadIdx.x; r < rows; r += kFilterThreads) sh_lo[r] = rs[r].lo;
    if (threadIdx.x < kFilterThreads / 32) sh_n[threadIdx.x] = 0;
    __syncthreads();
    const WarpStage st = warp_stage(sh_buf, sh_n);
    const u64 total = (u64)rows * tpr;
    const u64 t_begin = (u64)part * total / parts, t_end = (u64)(part + 1) * total / parts;
    // The last tiles of the range (about kFilterDynTiles per CTA, at most an eighth of the range) are
    // not dealt out in advance but claimed one at a time from a counter: the CTAs of a range finish
    // their fixed shares a few per cent apart (measured on the benchmark workload: 545 .. 572 us,
    // no pattern from launch to launch), and with the claimed end they all run dry within a few
    // tiles' time of each other.
    // (not for short ranges, under TK_FILTER_DYN_MIN = 32 tiles per CTA: there the barrier per claimed tile
    // costs more than the fixed shares differ)
    u64 n_dyn = (u64)cpp * kFilterDynTiles;
    if (n_dyn > (t_end - t_begin) / 8) n_dyn = (t_end - t_begin) / 8;
    if ((t_end - t_begin) < (u64)cpp * TK_FILTER_DYN_MIN) n_dyn = 0;
    const u64 t_dyn = t_end - n_dyn;
    u64 t = t_begin + (blockIdx.x - part * cpp);
    int cur = -1;
    RowGeom g;
    u64 lo = 0;
    int row = (int)(t / tpr);
    u32 tile = (u32)(t - (u64)row * tpr);
    float sq = 0.0f;
    for (; t < t_dyn; t += cpp) {
        if (row != cur) {
            if (cur >= 0) {
                stage_flush(st, rs + cur, cand + (size_t)cur * cap, cap);
                if (kStats) { warp_add_double(&rs[cur].sum_sq, (double)sq); sq = 0.0f; }
            }
            cur = row;
            g = row_geom(x, row, d);
            lo = sh_lo[row];
        }
        if (tile * (u32)(kFilterThreads * kUnroll) < g.nv || tile == 0)
            filter_tile<kFilterThreads, kUnroll, kEF, kStats>(g, tile, lo, st, rs + row, cand + (size_t)row * cap, cap,
                                                              kEF ? ef.eps + (size_t)row * (size_t)d : nullptr, ef.alpha,
                                                              sq);
        tile += cpp;
        while (tile >= tpr) { tile -= tpr; ++row; }
    }
    if (n_dyn > 0) {
        // sh_claim[i & 1] = the i-th claim of this CTA; the next one is asked for before the current tile
        // is read and parked after it, so its round trip is hidden
        u32* ticket = &rs[part].tile_ticket;  // zeroed by the sampling kernel (range numbers are row numbers too)
        if (threadIdx.x == 0) sh_claim[0] = atomicAdd(ticket, 1u);
        __syncthreads();
        for (u32 i = 0;; ++i) {
            const u32 c = sh_claim[i & 1];
            if ((u64)c >= n_dyn) break;
            u32 next_claim = 0;
            if (threadIdx.x == 0) next_claim = atomicAdd(ticket, 1u);
            t = t_dyn + c;
            row = (int)(t / tpr);
            tile = (u32)(t - (u64)row * tpr);
            if (row != cur) {
                if (cur >= 0) {
                    stage_flush(st, rs + cur, cand + (size_t)cur * cap, cap);
                    if (kStats) { warp_add_double(&rs[cur].sum_sq, (double)sq); sq = 0.0f; }
                }
                cur = row;
                g = row_geom(x, row, d);
                lo = sh_lo[row];
            }
            if (tile * (u32)(kFilterThreads * kUnroll) < g.nv || tile == 0)
                filter_tile<kFilterThreads, kUnroll, kEF, kStats>(g, tile, lo, st, rs + row, cand + (size_t)row * cap,
                                                                  cap, kEF ? ef.eps + (size_t)row * (size_t)d : nullptr,
                                                                  ef.alpha, sq);
            if (threadIdx.x == 0) sh_claim[(i + 1) & 1] = next_claim;
            __syncthreads();
        }
    }
    if (cur >= 0) {
        stage_flush(st, rs + cur, cand + (size_t)cur * cap, cap);
        if (kStats) warp_add_double(&rs[cur].sum_sq, (double)sq);
    }
    if (threadIdx.x == 0) phase_stamp(ctrl, kStampFilterEnd);
}

// ---------------------------------------------------------------------------
// general: verification and the exact multi-pass path (cooperative launch)
// ---------------------------------------------------------------------------
// Refinement levels over the 63-bit composite key: {shift, bits}.
__device__ __constant__ int kLevelShift[6] = {52, 41, 32, 21, 10, 0};
__device__ __constant__ int kLevelBits[6] = {11, 11, 9, 11, 11, 10};

__device__ __forceinline__ void hist_component(bool live, u32 idx, u32 bits, int level, int shift,
                                               int nbits, u64 lo, u32* sh_hist) {
    if (!live) return;
    u32 k = key_of(bits);
    if (level == 0) {
        atomicAdd(&sh_hist[k >> 20], 1u);
        return;
    }
    // cheap test on the key's known leading bits first
    int top = shift + nbits;  // bits above this level's digit are fixed by lo
    int kshift = top >= 32 ? top - 32 : 0;
    if (((k ^ (u32)(lo >> 32)) >> kshift) != 0 && kshift < 32) return;
    u64 ck = composite(k, idx);
    if ((ck >> top) != (lo >> top)) return;
    atomicAdd(&sh_hist[(u32)(ck >> shift) & ((1u << nbits) - 1u)], 1u);
}

// `sq`, when given, also receives the squares of all values of the tile (diagnostics).
__device__ __forceinline__ void hist_tile(const RowGeom& g, u32 tile, int level, u64 lo,
                                          u32* sh_hist, float* sq) {
    const int shift = kLevelShift[level], nbits = kLevelBits[level];
    const u32 j0 = tile * kGeneralTileVecs + threadIdx.x;
#pragma unroll
    for (int u = 0; u < kStreamUnroll; ++u) {
        u32 j = j0 + u * kGeneralThreads;
        if (j < g.nv) {
            uint4 v = ld_stream(g.vec + j);
            u32 i0 = g.head + 4u * j;
            if (sq) *sq = sq4(v, *sq);
            hist_component(true, i0 + 0, v.x, level, shift, nbits, lo, sh_hist);
            hist_component(true, i0 + 1, v.y, level, shift, nbits, lo, sh_hist);
            hist_component(true, i0 + 2, v.z, level, shift, nbits, lo, sh_hist);
            hist_component(true, i0 + 3, v.w, level, shift, nbits, lo, sh_hist);
        }
    }
    if (tile == 0 && threadIdx.x < 32 && (g.head | g.tail)) {
        u32 lane = threadIdx.x;
        bool live = false;
        u32 idx = 0;
        if (lane < g.head) { live = true; idx = lane; }
        else if (lane >= 8 && lane - 8 < g.tail) { live = true; idx = g.head + 4u * g.nv + (lane - 8); }
        u32 bits = live ? __float_as_uint(__ldg(g.base + idx)) : 0u;
        if (sq && live) *sq = fmaf(__uint_as_float(bits), __uint_as_float(bits), *sq);
        hist_component(live, idx, bits, level, shift, nbits, lo, sh_hist);
    }
}

// Ordered list (in shared memory) of the rows r < rows with pred(r); returns its length.
template <typename Pred>
__device__ __forceinline__ int build_row_list(int rows, unsigned short* sh_list, u32* scratch,
                                              Pred pred) {
    constexpr int PER = kMaxRowsPerLaunch / kGeneralThreads;
    u32 flags = 0, cnt = 0;
#pragma unroll
    for (int i = 0; i < PER; ++i) {
        int r = (int)threadIdx.x * PER + i;
        if (r < rows && pred(r)) { flags |= 1u << i; ++cnt; }
    }
    u32 total;
    u32 pos = block_inclusive_scan(cnt, scratch, &total) - cnt;
#pragma unroll
    for (int i = 0; i < PER; ++i)
        if (flags & (1u << i)) sh_list[pos++] = (unsigned short)((int)threadIdx.x * PER + i);
    __syncthreads();
    return (int)total;
}

__global__ void __launch_bounds__(kGeneralThreads)
general_kernel(const float* __restrict__ x, int rows, int64_t d, u32 K, u32 tpr, u32 cap,
               RowState* rs, u32* hist, uint2* cand, Ctrl* ctrl, int stats) {
    __shared__ u32 sh_hist[kHistBins];
    __shared__ unsigned short sh_list[kMaxRowsPerLaunch];
    __shared__ u32 sh_scratch[33];
    __shared__ u32 sh_res[2];
    __shared__ uint2 sh_buf[(kGeneralThreads / 32) * kStageSlots];
    __shared__ u32 sh_n[kGeneralThreads / 32];
    cg::grid_group grid = cg::this_grid();
    allow_dependents();  // the uplink select may queue up behind this grid
    dependency_wait();   // (returns at once unless launched as a programmatic dependent)
    if (threadIdx.x == 0) phase_stamp(ctrl, kStampVerifyStart);

    // Which rows failed verification?  Nothing below modifies a RowState before
    // the first grid-wide barrier, so every CTA sees the same answer.
    auto failed = [&](int r) {
        u32 c = rs[r].cand_count;
        return (rs[r].flags & kRowGeneral) != 0 || c < K || c > cap;
    };
    {
        int any = 0;
        for (int r = threadIdx.x; r < rows; r += blockDim.x) any |= failed(r) ? 1 : 0;
        if (!__syncthreads_or(any)) {
            if (blockIdx.x == 0 && threadIdx.x == 0) ctrl->rows_general = 0;
            if (threadIdx.x == 0) phase_stamp(ctrl, kStampVerifyEnd);
            return;
        }
    }
    int nF = build_row_list(rows, sh_list, sh_scratch, failed);
    if (blockIdx.x == 0 && threadIdx.x == 0) ctrl->rows_general = (u32)nF;

    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < nF; i += gridDim.x * blockDim.x) {
        RowState* r = rs + sh_list[i];
        r->flags |= kRowGeneral;
        r->g_active = 1;
        r->g_lo = 0;
        r->g_need = K;
        r->g_level = 0;
    }
    grid.sync();

    for (int iter = 0; iter < 6; ++iter) {
        int nA = build_row_list(rows, sh_list, sh_scratch, [&](int r) { return rs[r].g_active != 0; });
        if (nA == 0) break;
        // phase A: histograms of the active rows; each CTA takes a contiguous run of tiles
        {
            u64 total = (u64)nA * tpr;
            u64 chunk = (total + gridDim.x - 1) / gridDim.x;
            u64 t0 = (u64)blockIdx.x * chunk, t1 = min(total, t0 + chunk);
            int cur = -1, row = 0, level = 0;
            u64 lo = 0;
            RowGeom g;
            float sq = 0.0f;
            bool want_sq = false;  // the first full pass over a row no filter pass has read also sums its squares
            for (u64 t = t0; t < t1; ++t) {
                int li = (int)(t / tpr);
                u32 tile = (u32)(t - (u64)li * tpr);
                if (li != cur) {
                    if (cur >= 0) {
                        __syncthreads();
                        for (int b = threadIdx.x; b < kHistBins; b += blockDim.x)
                            if (sh_hist[b]) atomicAdd(&hist[(size_t)row * kHistBins + b], sh_hist[b]);
                        if (want_sq) warp_add_double(&rs[row].sum_sq, (double)sq);
                        sq = 0.0f;
                    }
                    __syncthreads();
                    cur = li;
                    row = sh_list[li];
                    g = row_geom(x, row, d);
                    lo = rs[row].g_lo;
                    level = (int)rs[row].g_level;
                    want_sq = stats && level == 0 && (rs[row].flags & kRowNoFilter) != 0;
                    for (int b = threadIdx.x; b < kHistBins; b += blockDim.x) sh_hist[b] = 0;
                    __syncthreads();
                }
                if ((u64)tile * kGeneralTileVecs >= (u64)g.nv && tile != 0) continue;
                hist_tile(g, tile, level, lo, sh_hist, want_sq ? &sq : nullptr);
            }
            if (cur >= 0) {
                __syncthreads();
                for (int b = threadIdx.x; b < kHistBins; b += blockDim.x)
                    if (sh_hist[b]) atomicAdd(&hist[(size_t)row * kHistBins + b], sh_hist[b]);
                if (want_sq) warp_add_double(&rs[row].sum_sq, (double)sq);
            }
        }
        grid.sync();
        // phase B: one CTA per active row picks the bucket of the K-th key
        for (int li = blockIdx.x; li < nA; li += gridDim.x) {
            int row = sh_list[li];
            RowState* r = rs + row;
            int level = (int)r->g_level;
            int nb = 1 << kLevelBits[level];
            __syncthreads();
            for (int b = threadIdx.x; b < kHistBins; b += blockDim.x) {
                u32* hp = &hist[(size_t)row * kHistBins + b];
                sh_hist[b] = __ldcg(hp);
                *hp = 0;
            }
            if (threadIdx.x == 0) sh_res[0] = 0xffffffffu;
            __syncthreads();
            u32 need = r->g_need, b, above;
            find_bucket<kHistBins / kGeneralThreads>(sh_hist, nb, need, sh_scratch, sh_res, &b, &above);
            if (threadIdx.x == 0) {
                if (b == 0xffffffffu) {           // the row holds fewer than `need` entries: cannot happen
                    raise_status(ctrl, -5);
                    b = 0; above = 0;
                    r->g_level = 5;               // ends the refinement below
                    level = 5;
                }
                u64 lo = r->g_lo | ((u64)b << kLevelShift[level]);
                u32 ge = (K - need) + above + sh_hist[b];  // components with ck >= lo
                if (ge <= cap || level == 5) {
                    r->g_active = 0;
                    r->lo = lo;
                    r->cand_count = 0;
                    r->max_key = 0;
                } else {
                    r->g_lo = lo;
                    r->g_need = need - above;
                    r->g_level = (u32)level + 1;
                }
            }
        }
        grid.sync();
    }

    // phase C: filter the failed rows again with their exact bound
    nF = build_row_list(rows, sh_list, sh_scratch, [&](int r) { return (rs[r].flags & kRowGeneral) != 0; });
    if (threadIdx.x < kGeneralThreads / 32) sh_n[threadIdx.x] = 0;
    __syncthreads();
    const WarpStage st = warp_stage(sh_buf, sh_n);
    u64 total = (u64)nF * tpr;
    int cur = -1, row = 0;
    u64 lo = 0;
    RowGeom g;
    for (u64 t = blockIdx.x; t < total; t += gridDim.x) {
        int li = (int)(t / tpr);
        u32 tile = (u32)(t - (u64)li * tpr);
        if (li != cur) {
            if (cur >= 0) stage_flush(st, rs + row, cand + (size_t)row * cap, cap);
            cur = li;
            row = sh_list[li];
            g = row_geom(x, row, d);
            lo = rs[row].lo;
        }
        if ((u64)tile * kGeneralTileVecs >= (u64)g.nv && tile != 0) continue;
        {
            float unused = 0.0f;
            filter_tile<kGeneralThreads, kStreamUnroll, false, false>(g, tile, lo, st, rs + row, cand + (size_t)row * cap,
                                                                      cap, nullptr, 0.0f, unused);
        }
    }
    if (cur >= 0) stage_flush(st, rs + row, cand + (size_t)row * cap, cap);
    if (threadIdx.x == 0) phase_stamp(ctrl, kStampVerifyEnd);
}

// ---------------------------------------------------------------------------
// select: exact K largest composite keys among a row's candidates (one cluster per row)
// ---------------------------------------------------------------------------
struct ApplyArgs {
    float* w;      // if non-NULL: w[idx] -= alpha * val for every emitted entry (last worker step)
    float alpha;
};

// If head is non-NULL every emitted entry (row, slot) is also threaded onto the chain of its
// coordinate in the dense server buffer (first half of the server step, see aggregate.cuh).
struct LinkArgs {
    u32* head;
    u32* next;
    u32 d;
    u32 row_base;  // entry ids count rows from here (rows are processed in batches)
    // Error memories: if zero_src is non-NULL the vector the entries were taken from,
    // zero_src[row][idx] with rows zero_stride apart, is set to +0 at every emitted entry
    // (eps <- a - Top_K(a), delta <- g - Top_K(g): second worker / server line of Algorithm 1/2).
    float* zero_src;
    size_t zero_stride;
    int stats;  // diagnostics: add the squares of the emitted values to RowState.sel_sq
    // Few workers: instead of chains, head[idx] keeps the first entry e0 to arrive at the coordinate and
    // next[] holds one mark word per entry (owner / shared); every later entry files its value in row e0
    // of the slot table (row_words words per row, all zero at rest); see aggregate.cuh.
    u32* slots;
    u32 row_words;
    // server step, for the downlink selection's first level (union_bin): the weights p_q and the
    // union's state, whose bin_base every row lowers to p_q * |its K-th value|
    const float* p;
    RowState* uni;
};

constexpr int kSelectRegs = 12;  // entries each thread keeps in registers across the levels

// Short rows with no sampled bound: the selection reads the row itself instead of a candidate
// list (entry i is component i), which replaces the multi-pass kernel and its launches.
struct DenseArgs {
    const float* x;          // [rows][list_stride] the rows themselves
    RowState* also_reset;    // union state to reset for the step (may be NULL)
    int stats;               // diagnostics: also sum the squares of every row into RowState.sum_sq
};

__device__ __forceinline__ void emit_entry(u32 row, u32 slot, u32 Keff, u32 idx, u32 bits, uint2* orow,
                                           size_t out_stride, const ApplyArgs& apply, const LinkArgs& link,
                                           Ctrl* ctrl) {
    if (slot >= Keff) { raise_status(ctrl, -5); return; }
    orow[slot] = make_uint2(idx, bits);
    if (apply.w) {
        float upd = __fmul_rn(apply.alpha, __uint_as_float(bits));
        apply.w[idx] = __fsub_rn(apply.w[idx], upd);
    }
    if (link.zero_src) link.zero_src[(size_t)row * link.zero_stride + idx] = 0.0f;
    if (link.head) {
        u32 e = (link.row_base + row) * (u32)out_stride + slot;
        if (idx >= link.d) {
            link.next[e] = 0;
            raise_status(ctrl, -5);
        } else if (link.slots) {
            file_in_slot(link.next, link.slots, link.row_words, atomicCAS(&link.head[idx], 0u, e + 1), e, link.row_base + row, bits);
        } else {
            link.next[e] = atomicExch(&link.head[idx], e + 1);
        }
    }
}

// lists[row] holds the row's candidates: exactly the entries with ck >= rs[row].lo, all with
// key <= rs[row].max_key, rs[row].cand_count of them.
//
// Two ways to spread one row over several CTAs:
//   kGrid == false  one thread-block cluster per row; the CTAs' histograms are combined
//                   through distributed shared memory, cluster barriers between levels
//   kGrid == true   a single row spread over the whole (cooperatively launched) grid, for
//                   lists too long for one cluster (the union of N uplink messages);
//                   histograms are combined in `ghist` (3 x kHistBins words of global
//                   memory, all zero when the kernel starts), grid barriers between levels.
//                   With `prebuilt` the first level's histogram — every entry's key by
//                   union_bin — is already complete in ghist[0 .. kHistBins) (the server sum
//                   counted it while it appended the entries), so the first pass over the list
//                   and its barrier are not needed.
//
// kDense (cluster variant only): the "list" of row r is the row dense.x[r][0..cap) itself, every
// component a candidate; the kernel then also does what the sampling / reset kernels do for
// the other paths (row state, union state).
template <bool kGrid, bool kDense = false>
__global__ void __launch_bounds__(kSelectThreads)
select_kernel(const uint2* __restrict__ lists, size_t list_stride, u32 cap, RowState* rs, u32 K,
              uint2* out, size_t out_stride, ApplyArgs apply, LinkArgs link, Ctrl* ctrl, u32* ghist,
              DenseArgs dense, int prebuilt) {
    __shared__ u32 sh_hist[2][kHistBins];  // double-buffered: peers may still read level L while L+1 fills
    __shared__ u32 sh_tot[kHistBins];
    __shared__ u32 sh_scratch[33];
    __shared__ u32 sh_res[2];
    __shared__ u64 sh_list[kRankMax];  // the bucket that gets ranked directly (cluster: gathered in CTA 0's copy)
    __shared__ u32 sh_list_n;
    __shared__ u64 sh_T;
    cg::cluster_group cluster = cg::this_cluster();
    cg::grid_group grid = cg::this_grid();
    if (threadIdx.x == 0) sh_list_n = 0;  // read by peers only after a cluster barrier
    dependency_wait();   // candidates and bounds come from the kernels before
    allow_dependents();
    constexpr int stamp0 = kGrid ? kStampDownStart : kStampUpStart;  // start, loaded, level, threshold, end
    if (TK_PHASE_CLOCK && !kDense && threadIdx.x == 0) phase_stamp(ctrl, stamp0);
    const u32 CS = kGrid ? gridDim.x : cluster.num_blocks();
    const u32 rank = kGrid ? blockIdx.x : cluster.block_rank();
    const u32 row = kGrid ? 0u : blockIdx.x / CS;
    RowState* r = rs + row;
    if (kDense) {
        if (rank == 0 && threadIdx.x == 0) {
            reset_state(r, 1ull, 0u);
            r->cand_count = cap;
        }
        if (blockIdx.x == 0 && threadIdx.x == 0) {
            if (dense.also_reset) reset_state(dense.also_reset, 0ull, 0u);
            ctrl->rows_general = 0;
        }
        cluster.sync();  // the row's counters are reset before any CTA of the row adds to them
    }
    const u32 C = kDense ? cap : min(r->cand_count, cap);
    const u32 Keff = min(K, C);
    const uint2* list = kDense ? nullptr : lists + (size_t)row * list_stride;
    const float* xrow = kDense ? dense.x + (size_t)row * list_stride : nullptr;
    auto read_entry = [&](u32 i) -> uint2 {
        return kDense ? make_uint2(i, __float_as_uint(__ldg(xrow + i))) : list[i];
    };
    const u32 first = rank * kSelectThreads + threadIdx.x;
    const u32 stride = CS * kSelectThreads;
    const u32 rest = first + kSelectRegs * stride;  // entries from here on are re-read every level

    // this thread's entries first + k*stride, k < kSelectRegs, stay in registers as composite
    // keys (0 = absent; a real entry's composite key is never 0) plus one sign bit each.
    // Only the first `nslots` register slots can hold anything (the same for all threads of
    // the row): the unrolled loops below skip the others.
    const u32 nslots = min((u32)kSelectRegs, (C + stride - 1) / stride);
    u64 eck[kSelectRegs];
    u32 esign = 0;
#pragma unroll
    for (int k = 0; k < kSelectRegs; ++k) {
        u32 i = first + (u32)k * stride;
        eck[k] = 0;
        if ((u32)k < nslots && i < C) {
            uint2 e = read_entry(i);
            eck[k] = composite(key_of(e.y), e.x);
            esign |= (e.y >> 31) << k;
        }
    }
    if (kDense && dense.stats) {  // diagnostics: the row's squared norm (no streaming pass reads these rows)
        float sq = 0.0f;
#pragma unroll
        for (int k = 0; k < kSelectRegs; ++k) {
            if ((u32)k >= nslots) break;
            float v = __uint_as_float((u32)(eck[k] >> 32));
            sq = fmaf(v, v, sq);
        }
        for (u32 i = rest; i < C; i += stride) {
            float v = __ldg(xrow + i);
            sq = fmaf(v, v, sq);
        }
        warp_add_double(&r->sum_sq, (double)sq);
    }

    if (TK_PHASE_CLOCK && !kDense && threadIdx.x == 0) phase_stamp(ctrl, stamp0 + 1);
    u64 T = 1;  // emit entries with ck >= T (absent ones are 0)
    const bool pre = kGrid && prebuilt != 0;
    const bool solo = kGrid && CS == 1 && !pre;  // one CTA and nothing to fetch from the global scratch
    if (pre && C <= Keff && rank == 0)  // nothing to select: the prebuilt counts are not needed
        for (int b = threadIdx.x; b < kHistBins; b += kSelectThreads) ghist[b] = 0;
    if (C > Keff) {
        u64 lo = max(r->lo, 1ull);
        u64 hi = kDense ? 0x7fffffffffffffffull : ((u64)r->max_key << 32) | 0xffffffffull;  // dense: no maximum is known
        if (pre) {  // the whole range; the first level's buckets are union_bin's, all kHistBins of them
            lo = 1ull;
            hi = 0x7fffffffffffffffull;
        }
        if (hi < lo) hi = lo;
        u32 need = Keff;
        bool found = false, ranked = false;
        for (int level = 0; level < 8 && !found; ++level) {
            u32* hist = sh_hist[level & 1];
            u64 width = hi - lo;
            int s = width ? max(0, 64 - __clzll((long long)width) - 11) : 0;
            int nb = (int)(width >> s) + 1;
            const bool ready = pre && level == 0;  // this level's counts are already in ghist
            if (threadIdx.x == 0) sh_res[0] = 0xffffffffu;
            if (!ready) {
                for (int b = threadIdx.x; b < nb; b += kSelectThreads) hist[b] = 0;
                __syncthreads();
#pragma unroll
                for (int k = 0; k < kSelectRegs; ++k) {
                    if ((u32)k >= nslots) break;
                    u64 off = eck[k] - lo;              // wraps to a huge value when eck < lo
                    if (off <= width) atomicAdd(&hist[(u32)(off >> s)], 1u);
                }
                for (u32 i = rest; i < C; i += stride) {
                    uint2 e = read_entry(i);
                    u64 off = composite(key_of(e.y), e.x) - lo;
                    if (off <= width) atomicAdd(&hist[(u32)(off >> s)], 1u);
                }
            }
            if (solo) {  // the whole list in one CTA: its own histogram is the total
                __syncthreads();
                for (int b = threadIdx.x; b < nb; b += kSelectThreads) sh_tot[b] = hist[b];
            } else if (kGrid) {
                u32* gh = ghist + (u32)(level % 3) * kHistBins;
                if (!ready) {
                    __syncthreads();
                    for (int b = threadIdx.x; b < nb; b += kSelectThreads)
                        if (hist[b]) atomicAdd(&gh[b], hist[b]);
                    grid.sync();  // every CTA has added its counts
                }
                for (int b = threadIdx.x; b < nb; b += kSelectThreads) sh_tot[b] = __ldcg(&gh[b]);
                // the buffer read at the previous level is idle now and is not written before the
                // next barrier: clear it for the level after next
                if (rank == 0) {
                    u32* idle = ghist + (u32)((level + 2) % 3) * kHistBins;
                    for (int b = threadIdx.x; b < kHistBins; b += kSelectThreads) idle[b] = 0;
                }
            } else {
                cluster.sync();  // all CTAs of the row have filled this level's histogram
                for (int b = threadIdx.x; b < nb; b += kSelectThreads) {
                    u32 sum = 0;
                    for (u32 c = 0; c < CS; ++c) sum += cluster.map_shared_rank(hist, c)[b];
                    sh_tot[b] = sum;
                }
            }
            __syncthreads();
            u32 b, above;
            find_bucket<kHistBins / kSelectThreads>(sh_tot, nb, need, sh_scratch, sh_res, &b, &above);
            if (b == 0xffffffffu) {
                if (threadIdx.x == 0 && rank == 0) raise_status(ctrl, -5);
                break;
            }
            if (TK_PHASE_CLOCK && !kDense && level == 0 && threadIdx.x == 0) phase_stamp(ctrl, stamp0 + 2);
            need -= above;
            u64 blo = lo + ((u64)b << s);
            u64 bhi = blo + ((1ull << s) - 1ull);
            if (bhi > hi) bhi = hi;
            if (ready) {  // bucket b of union_bin as a range of composite keys
                const u64 base = union_base(r);
                const u64 klo = b == 0u ? 0ull : base + ((u64)(b - 1u) << kUnionBinShift);
                u64 khi = b == 0u ? base - 1ull : klo + ((1ull << kUnionBinShift) - 1ull);  // (bucket 0 is empty when base is 0)
                if (b == (u32)(kHistBins - 1) || khi > 0x7fffffffull) khi = 0x7fffffffull;
                blo = max(klo << 32, 1ull);
                bhi = (khi << 32) | 0xffffffffull;
            }
            const u32 cnt = sh_tot[b];
            lo = blo;
            hi = bhi;
            __syncthreads();
            if (need == cnt) {
                T = blo;
                found = true;
            } else if (cnt <= (u32)kRankMax) {
                // Few entries left in the bucket: gather them in one place, let every CTA copy them and
                // find the need-th largest by counting, for each entry, the entries above it (composite
                // keys are all different, so exactly one entry has need-1 above it).  One barrier instead
                // of one or two more levels.
                u64* gather = kGrid ? (solo ? sh_list : reinterpret_cast<u64*>(ghist + 3 * kHistBins + 4))
                                  : cluster.map_shared_rank(sh_list, 0);
                u32* fill = kGrid ? (solo ? &sh_list_n : ghist + 3 * kHistBins)
                                  : cluster.map_shared_rank(&sh_list_n, 0);
                const u64 width2 = hi - lo;
#pragma unroll
                for (int k = 0; k < kSelectRegs; ++k) {
                    if ((u32)k >= nslots) break;
                    if (eck[k] - lo <= width2) gather[atomicAdd(fill, 1u)] = eck[k];
                }
                for (u32 i = rest; i < C; i += stride) {
                    uint2 e = read_entry(i);
                    u64 ck = composite(key_of(e.y), e.x);
                    if (ck - lo <= width2) gather[atomicAdd(fill, 1u)] = ck;
                }
                if (solo) {
                    __syncthreads();
                } else if (kGrid) {
                    grid.sync();  // the list is complete; nobody reads the histograms or the counter any more
                    if (rank == 0) {
                        for (int i = threadIdx.x; i < 3 * kHistBins + 4; i += kSelectThreads) ghist[i] = 0;
                    }
                    for (u32 i = threadIdx.x; i < cnt; i += kSelectThreads) sh_list[i] = __ldcg(gather + i);
                    __syncthreads();
                } else {
                    cluster.sync();
                    if (rank != 0)
                        for (u32 i = threadIdx.x; i < cnt; i += kSelectThreads) sh_list[i] = gather[i];
                    __syncthreads();
                }
                for (u32 i = threadIdx.x; i < cnt; i += kSelectThreads) {
                    const u64 me = sh_list[i];
                    u32 above = 0;
                    for (u32 o = 0; o < cnt; ++o) above += sh_list[o] > me ? 1u : 0u;
                    if (above == need - 1) sh_T = me;
                }
                __syncthreads();
                T = sh_T;
                found = true;
                ranked = true;
            }
        }
        if (!found) {
            T = lo;
            if (threadIdx.x == 0 && rank == 0) raise_status(ctrl, -5);
        }
        if (solo) {
            // nothing was exchanged
        } else if (kGrid) {
            // leave the scratch all zero for the next launch: once everybody has read the last level
            // (the ranking step has done both already)
            if (!ranked) {
                grid.sync();
                if (rank == 0)
                    for (int b = threadIdx.x; b < 3 * kHistBins; b += kSelectThreads) ghist[b] = 0;
            }
        } else {
            cluster.sync();  // no CTA leaves while a peer may still read its histograms
        }
    }

    if (TK_PHASE_CLOCK && !kDense && threadIdx.x == 0) phase_stamp(ctrl, stamp0 + 3);
    if (!kGrid && link.uni && rank == 0 && threadIdx.x == 0) {
        // no emitted magnitude of this row is below its K-th value (key T >> 32; 0 when the whole list goes out)
        const float least = __fmul_rn(link.p[link.row_base + row], __uint_as_float((u32)(T >> 32)));
        atomicMin(&link.uni->bin_base, key_of(__float_as_uint(least)));
    }
    // emission: every entry with ck >= T, exactly Keff of them; one counter update per warp
    uint2* orow = out + (size_t)row * out_stride;
    double sel_sq = 0.0;
    u32 mine = 0;
#pragma unroll
    for (int k = 0; k < kSelectRegs; ++k) {
        if ((u32)k >= nslots) break;
        mine += eck[k] >= T ? 1u : 0u;
    }
    {
        u32 lane = lane_id();
        u32 incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            u32 y = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= (u32)o) incl += y;
        }
        u32 wtotal = __shfl_sync(0xffffffffu, incl, 31);
        u32 base = 0;
        if (wtotal) {
            if (lane == 31) base = atomicAdd(&r->out_count, wtotal);
            base = __shfl_sync(0xffffffffu, base, 31);
        }
        const u32 slot0 = base + incl - mine;
        // The entries of one thread go to different coordinates, so their memory round trips (the
        // old value of w, the previous head of the chain) are independent: issue them all, then
        // finish them all, instead of one dependent load-store pair after the other.
        u32 fetched[kSelectRegs];
        u32 slot = slot0;
#pragma unroll
        for (int k = 0; k < kSelectRegs; ++k) {
            fetched[k] = 0;
            if ((u32)k >= nslots) break;
            if (eck[k] >= T) {
                u32 idx = 0xffffffffu - (u32)eck[k];
                if (slot < Keff && idx < 0x80000000u) {
                    if (apply.w) fetched[k] = __float_as_uint(apply.w[idx]);
                    if (link.head && idx < link.d) {
                        const u32 e1 = (link.row_base + row) * (u32)out_stride + slot + 1;
                        fetched[k] = link.slots ? atomicCAS(&link.head[idx], 0u, e1) : atomicExch(&link.head[idx], e1);
                    }
                }
                ++slot;
            }
        }
        slot = slot0;
#pragma unroll
        for (int k = 0; k < kSelectRegs; ++k) {
            if ((u32)k >= nslots) break;
            if (eck[k] >= T) {
                u32 idx = 0xffffffffu - (u32)eck[k];
                u32 bits = (u32)(eck[k] >> 32) | (((esign >> k) & 1u) << 31);
                if (slot >= Keff) {
                    raise_status(ctrl, -5);
                } else {
                    orow[slot] = make_uint2(idx, bits);
                    if (apply.w)
                        apply.w[idx] = __fsub_rn(__uint_as_float(fetched[k]), __fmul_rn(apply.alpha, __uint_as_float(bits)));
                    if (link.zero_src) link.zero_src[(size_t)row * link.zero_stride + idx] = 0.0f;
                    if (link.head) {
                        u32 e = (link.row_base + row) * (u32)out_stride + slot;
                        if (idx >= link.d) { link.next[e] = 0; raise_status(ctrl, -5); }
                        else if (link.slots) file_in_slot(link.next, link.slots, link.row_words, fetched[k], e, link.row_base + row, bits);
                        else link.next[e] = fetched[k];
                    }
                    if (link.stats) sel_sq += (double)__uint_as_float(bits) * (double)__uint_as_float(bits);
                }
                ++slot;
            }
        }
    }
    for (u32 i0 = rank * kSelectThreads + kSelectRegs * stride; i0 < C; i0 += stride) {
        u32 i = i0 + threadIdx.x;
        bool pred = false;
        uint2 e = make_uint2(0, 0);
        if (i < C) {
            e = read_entry(i);
            pred = composite(key_of(e.y), e.x) >= T;
        }
        u32 m = __ballot_sync(0xffffffffu, pred);
        if (m == 0) continue;
        u32 lane = lane_id(), base = 0;
        int leader = __ffs(m) - 1;
        if ((int)lane == leader) base = atomicAdd(&r->out_count, (u32)__popc(m));
        base = __shfl_sync(0xffffffffu, base, leader);
        if (pred) {
            emit_entry(row, base + (u32)__popc(m & ((1u << lane) - 1u)), Keff, e.x, e.y, orow, out_stride, apply, link,
                       ctrl);
            if (link.stats) sel_sq += (double)__uint_as_float(e.y) * (double)__uint_as_float(e.y);
        }
    }
    if (link.stats) warp_add_double(&r->sel_sq, sel_sq);
    // warm start of the row's next selection (cand_count and flags are not written by this kernel)
    if (!kGrid && !kDense && rank == 0 && threadIdx.x == 0) {
        const bool redone = (r->flags & kRowGeneral) != 0u, kept = (r->flags & kRowReused) != 0u;
        const u32 Tkey = C > Keff ? (u32)(T >> 32) : 0u;  // 0: the whole list went out, there is no threshold
        u32 drift = r->drift;
        const u32 before = r->prev_T_key;
        if (Tkey && before) drift = max(Tkey > before ? Tkey - before : before - Tkey, drift - drift / 16u);
        else if (Tkey) drift = kReuseFirstDrift;
        u32 wait = r->reuse_wait & 0xffffu, backoff = r->reuse_wait >> 16;
        if (kept && redone) {            // a warm-started bound failed: sample for a while, twice as long as last time
            backoff = backoff < 2u ? 2u : (backoff < 64u ? backoff * 2u : 64u);
            wait = backoff;
            if (link.uni) atomicAdd(&link.uni->reuse_fails, 1u);  // ... and so do the context's other rows
        } else if (kept) {               // a warm-started bound held
            backoff >>= 1;
        }
        const u64 margin = max((u64)kReuseMinMargin, 4ull * drift);
        bool ok = !redone && (u32)r->lo == 0u && Tkey != 0u && margin <= (u64)kReuseMaxMargin && (u64)Tkey > margin;
        if (wait > 0u) { ok = false; --wait; }
        r->prev_T_key = Tkey;
        r->drift = drift;
        r->next_lo_key = ok ? Tkey - (u32)margin : 0u;
        r->reuse_ok = ok ? 1u : 0u;
        r->reuse_wait = (backoff << 16) | wait;
    }
    // the next step's first level is centred on this step's threshold (every CTA is past its last look
    // at the buckets: a grid barrier lies behind whenever they were used)
    if (kGrid && prebuilt && rank == 0 && threadIdx.x == 0) r->bin_hint = C > Keff ? union_hint((u32)(T >> 32)) : 0u;
    if (TK_PHASE_CLOCK && !kDense) {
        __syncthreads();
        if (threadIdx.x == 0) phase_stamp(ctrl, stamp0 + 4);
    }
}

}  // namespace tk
