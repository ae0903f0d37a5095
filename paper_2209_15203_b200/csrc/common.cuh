// Shared device-side definitions of libtopk: per-row selection state, the
// composite ordering key, warp/block primitives.
//
// Ordering.  Top_K keeps the K components of largest magnitude (Section 1 of
// the paper); the library orders components by the pair (key descending, index
// ascending) with key = bits & 0x7fffffff.  Both are packed into one 64-bit
// "composite key"
//        ck = key << 32 | (0xffffffff - index)
// so that "larger ck" means "kept first" and no two components of a row
// compare equal.  Top_K is then: the K largest composite keys.
#pragma once

#include <cuda_runtime.h>
#include <cooperative_groups.h>
#include <stdint.h>

namespace tk {

namespace cg = cooperative_groups;

typedef unsigned int u32;
typedef unsigned long long u64;

constexpr int kHistBins = 2048;        // buckets of one refinement level
constexpr int kPredictCtas = 8;        // sampling CTAs per row
constexpr int kPredictThreads = 1024;
constexpr int kSampleSlots = kPredictCtas * kPredictThreads / 2;  // per-row sample maxima (one per thread pair)
constexpr int kPredictMaxTurns = 10;   // 16-byte loads one sampling thread issues, all at once
constexpr int kPredictLightTurns = 2;  // ... in the variant for many rows
// Streaming passes.  Measured on B200 (448 threads x 2 CTAs per SM, one wave): read bandwidth
// rises with the 16-byte loads a thread has in flight up to 8 (115 KB per SM: 5 -> 6 -> 8 loads take
// 4 and 7 us off the 0.57 ms kernel of the benchmark workload), is no better at 10, and falls with
// more resident threads (512 x 2) or fewer (320 .. 416 x 2 with 8 .. 10 loads).
#ifndef TK_FILTER_THREADS
#define TK_FILTER_THREADS 448
#endif
#ifndef TK_FILTER_CTAS
#define TK_FILTER_CTAS 2
#endif
#ifndef TK_STREAM_UNROLL
#define TK_STREAM_UNROLL 5
#endif
constexpr int kFilterThreads = TK_FILTER_THREADS;  // filter kernel: threads per CTA
constexpr int kFilterCtasPerSm = TK_FILTER_CTAS;   // filter kernel: resident CTAs per SM (grid = that x SMs)
constexpr int kGeneralThreads = 512;               // multi-pass kernel: threads per CTA
#ifndef TK_FILTER_UNROLL
#define TK_FILTER_UNROLL 8
#endif
constexpr int kFilterUnroll = TK_FILTER_UNROLL;    // filter kernel: 16-byte loads in flight per thread
constexpr int kStreamUnroll = TK_STREAM_UNROLL;    // multi-pass kernel: the same (512-thread CTAs; 8 measured 40 % slower there)
constexpr int kFilterTileVecs = kFilterThreads * kFilterUnroll;    // float4 per tile
constexpr int kGeneralTileVecs = kGeneralThreads * kStreamUnroll;
#ifndef TK_FILTER_EF_UNROLL
#define TK_FILTER_EF_UNROLL 2
#endif
constexpr int kFilterEfUnroll = TK_FILTER_EF_UNROLL;  // with error memories a thread has two loads in flight per float4
constexpr int kFilterEfTileVecs = kFilterThreads * kFilterEfUnroll;
#ifndef TK_FILTER_MIN_CPP
#define TK_FILTER_MIN_CPP 37
#endif
// The filter grid splits the tile space into ranges shared by at least this many CTAs each
// (8 ranges on 296 CTAs; 37 ranges of 8 CTAs measured 3 % slower on the 32-row workload).
constexpr int kFilterMinCpp = TK_FILTER_MIN_CPP;
#ifndef TK_FILTER_DYN_TILES
#define TK_FILTER_DYN_TILES 16
#endif
constexpr int kFilterDynTiles = TK_FILTER_DYN_TILES;  // tiles per CTA (on average) left to be claimed at the end of a tile range; 0: none
constexpr int kSelectThreads = 1024;   // cluster select: threads per CTA
#ifndef TK_SELECT_PER_THREAD
#define TK_SELECT_PER_THREAD 8
#endif
constexpr int kSelectPerThread = TK_SELECT_PER_THREAD;  // candidates per thread the cluster size aims at
#ifndef TK_RANK_MAX
#define TK_RANK_MAX 256
#endif
constexpr int kRankMax = TK_RANK_MAX;          // a bucket of at most this many candidates is ranked directly (cnt^2 compares) instead of refined
// Global scratch of the grid-wide select: three histograms, a counter (4 words) and a list of kRankMax
// composite keys; all but the list must be zero when the kernel starts, and are when it ends.
constexpr int kGridScratchWords = 3 * kHistBins + 4 + 2 * kRankMax;
constexpr int kMaxRowsPerLaunch = 4096;
constexpr u32 kRowGeneral = 1u;        // RowState.flags: row redone by the multi-pass path
constexpr u32 kRowNoFilter = 2u;       // RowState.flags: no filter pass has read this row
constexpr u32 kRowReused = 4u;         // RowState.flags: the row's bound was kept from its last selection, not sampled

// Per-row state of one batched selection.  Lives in global memory.
struct RowState {
    u64 lo;          // the row's candidates are exactly the components with ck >= lo
    u32 cand_count;  // how many components have ck >= lo (counted, even beyond capacity)
    u32 max_key;     // largest key among them (upper end of the selection's first range)
    u32 out_count;   // entries emitted by the final exact selection
    u32 flags;
    u32 ticket;      // sampling CTAs of this row that have finished
    u32 g_active;    // multi-pass path: still refining this row
    u64 g_lo;        // multi-pass path: known leading bits of the K-th composite key
    u32 g_need;      // multi-pass path: entries still to take inside the current bucket
    u32 g_level;
    // diagnostics (filled only when asked for)
    double sum_sq;   // sum of squares of the whole vector
    double sel_sq;   // sum of squares of the emitted entries
    u32 nnz;         // union list: entries whose value is not zero
    u32 tile_ticket; // streaming pass: tiles handed out so far from the claimed end of tile range number <this row's index>
    u32 bin_base;    // union: a key no unshared sum of this step lies below (see union_base)
    u32 bin_hint;    // union: where the previous step's downlink threshold puts the buckets (0: none yet); survives resets
    // warm start of the row's next selection (see predict_kernel); all of it survives resets
    u32 reuse_ok;    // next_lo_key may serve as the next selection's bound
    u32 next_lo_key; // the last threshold's key minus a margin
    u32 prev_T_key;  // key of the K-th largest of the last selection (0: none)
    u32 drift;       // how far, in keys, that key has recently moved from one selection to the next (decaying maximum)
    u32 reuse_wait;  // bit 0..15: selections to sample before a bound may be kept again; bits 16..31: the current
                     // back-off (doubles, up to 64, each time a warm-started bound fails; halves when one holds)
    // In the union's state the three words above gate the warm starts of ALL rows of the context's next
    // step (reuse_ok: allowed; reuse_wait: the same back-off, driven by reuse_fails), so that many rows
    // with unsteady thresholds cannot each spend a failed attempt in turn.
    u32 reuse_fails; // union: rows whose warm-started bound failed in this step
};

// Build with -DTK_PHASE_CLOCK=1 to make the kernels of a step leave device timestamps (the
// nanosecond global timer) where they start and end and at the milestones of the selections;
// tk_debug_phase_clock reads them.  Off in the ordinary build: a stamp costs two atomics per CTA.
#ifndef TK_PHASE_CLOCK
#define TK_PHASE_CLOCK 0
#endif
enum : int {
    kStampPredictStart = 0, kStampPredictEnd, kStampFilterStart, kStampFilterEnd, kStampVerifyStart, kStampVerifyEnd,
    // a selection: its predecessors have ended, candidates in registers, first level's bucket found,
    // threshold known, everything emitted
    kStampUpStart, kStampUpLoaded, kStampUpLevel, kStampUpThreshold, kStampUpEnd,
    kStampAggStart, kStampAggEnd,
    kStampDownStart, kStampDownLoaded, kStampDownLevel, kStampDownThreshold, kStampDownEnd,
    kStampCount
};

// Step-wide control block.
struct Ctrl {
    int status;        // sticky TK_ERR_* raised on the device
    u32 rows_general;  // rows the multi-pass path handled in the last selection
    u32 pad[6];
#if TK_PHASE_CLOCK
    u64 t_first[kStampCount];  // earliest / latest time any CTA passed each stamp
    u64 t_last[kStampCount];
#endif
};

// One thread per CTA calls.
__device__ __forceinline__ void phase_stamp(Ctrl* ctrl, int which) {
#if TK_PHASE_CLOCK
    u64 t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    atomicMin(&ctrl->t_first[which], t);
    atomicMax(&ctrl->t_last[which], t);
#endif
}

__device__ __forceinline__ u32 key_of(u32 bits) { return bits & 0x7fffffffu; }

// First level of the downlink selection, counted by the server sum as it appends the union:
// bucket 0 holds the keys below `base`, buckets 1 .. 2046 are 2^kUnionBinShift keys wide from
// `base` on, bucket 2047 everything above.  Where the buckets sit is only a matter of speed (the
// selection refines whatever bucket the K-th largest falls in): they are centred on the previous
// step's threshold (bin_hint: +-24 % in value, 0.02 % per bucket — consecutive steps of a
// training run have close thresholds, and then the bucket of the K-th holds few enough entries to
// be ranked directly); without one they start at the smallest p_q * |K-th value of row q|, below
// which no sum of a coordinate that only one worker sent can lie.
#ifndef TK_UNION_BIN_SHIFT
#define TK_UNION_BIN_SHIFT 11
#endif
constexpr int kUnionBinShift = TK_UNION_BIN_SHIFT;
__device__ __forceinline__ u32 union_base(const RowState* uni) { return uni->bin_hint ? uni->bin_hint : uni->bin_base; }
__device__ __forceinline__ u32 union_hint(u32 threshold_key) {  // the threshold in the middle bucket
    const u32 half = (u32)(kHistBins / 2 - 1) << kUnionBinShift;
    return threshold_key > half ? threshold_key - half : 1u;
}
__device__ __forceinline__ u32 union_bin(u32 key, u32 base) {
    if (key < base) return 0u;
    const u32 b = 1u + ((key - base) >> kUnionBinShift);
    return b > (u32)(kHistBins - 1) ? (u32)(kHistBins - 1) : b;
}

__device__ __forceinline__ u64 composite(u32 key, u32 idx) {
    return ((u64)key << 32) | (u64)(0xffffffffu - idx);
}

__device__ __forceinline__ void raise_status(Ctrl* ctrl, int code) {
    atomicCAS(&ctrl->status, 0, code);
}

// The vector a worker compresses.  Memory-free iteration: its gradient g.  With error
// memories (first worker line of Algorithm 1/2): a = eps + alpha * g, one rounding each.
struct EfArgs {
    float* eps;   // [rows][d] worker memories, NULL for the memory-free iteration
    float alpha;
};

__device__ __forceinline__ u32 compensated(u32 g_bits, u32 eps_bits, float alpha) {
    return __float_as_uint(__fadd_rn(__uint_as_float(eps_bits), __fmul_rn(alpha, __uint_as_float(g_bits))));
}

// 16-byte streaming load of data this kernel also writes (no L1 allocation, coherent path).
__device__ __forceinline__ uint4 ld_once(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// 16-byte read-only streaming load that does not allocate in L1.
__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

__device__ __forceinline__ u32 lane_id() { return threadIdx.x & 31; }

// Programmatic dependent launch.  A kernel launched with the programmatic-serialization
// attribute may become resident while its predecessor in the stream still runs; it must call
// dependency_wait() before it touches anything the predecessor produces (the call returns at
// once when the kernel was launched the ordinary way).  A predecessor calls
// allow_dependents() as early as it likes: the dependent's launch latency then overlaps the
// predecessor's run instead of following it.
__device__ __forceinline__ void dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void allow_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// *dst += sum over the warp of v, accumulated in double.  All lanes call.
__device__ __forceinline__ void warp_add_double(double* dst, double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if (lane_id() == 0 && v != 0.0) atomicAdd(dst, v);
}

__device__ __forceinline__ float sq4(uint4 v, float acc) {
    float a = __uint_as_float(v.x), b = __uint_as_float(v.y), c = __uint_as_float(v.z), e = __uint_as_float(v.w);
    return fmaf(a, a, fmaf(b, b, fmaf(c, c, fmaf(e, e, acc))));
}

// Slot filing of the server step (few workers), given what the compare-and-swap on head[idx]
// returned.  0: this entry e was the first at the coordinate and owns it (its value stays where it
// is, in the message); it says so in its own word of `mark` (bit 0).  Otherwise the word holds the
// owner's entry number + 1, and this entry marks the owner's word (bit 1: "shared"), sets its
// worker's bit in the 128-bit mask that opens the owner's row of the slot table and leaves its
// value in its worker's column of that row.  The marks are one word per entry (read back in entry
// order, unlike the coordinate words, which are scattered over a buffer far larger than L2); all
// of them are zero at rest.  Nothing here waits for a result.
constexpr u32 kMarkOwner = 1u, kMarkShared = 2u;
constexpr u32 kSlotMaskWords = 4;

__device__ __forceinline__ void file_in_slot(u32* mark, u32* slots, u32 row_words, u32 seen, u32 e, u32 worker, u32 bits) {
    if (seen == 0) {
        atomicOr(&mark[e], kMarkOwner);
        return;
    }
    atomicOr(&mark[seen - 1], kMarkShared);
    u32* row = slots + (size_t)(seen - 1) * row_words;
    atomicOr(row + (worker >> 5), 1u << (worker & 31u));
    row[kSlotMaskWords + worker] = bits;
}

// Append the lanes with `pred` to a list whose fill counter is *counter.
// Every lane of the warp must call.  The counter always advances by the number
// of appending lanes; entries that would land beyond `cap` are dropped (the
// caller detects that from the counter).  Returns the ballot.
__device__ __forceinline__ u32 warp_append(bool pred, u32 idx, u32 bits, u32* counter,
                                           uint2* list, u32 cap) {
    u32 m = __ballot_sync(0xffffffffu, pred);
    if (m == 0) return 0;
    u32 lane = lane_id();
    u32 base = 0;
    int leader = __ffs(m) - 1;
    if ((int)lane == leader) base = atomicAdd(counter, (u32)__popc(m));
    base = __shfl_sync(0xffffffffu, base, leader);
    if (pred) {
        u32 slot = base + (u32)__popc(m & ((1u << lane) - 1u));
        if (slot < cap) list[slot] = make_uint2(idx, bits);
    }
    return m;
}

// Inclusive scan of one u32 per thread over the whole block (blockDim.x a
// multiple of 32, at most 1024).  `scratch` holds 33 words.  Returns the
// inclusive prefix; *total receives the block sum.
__device__ __forceinline__ u32 block_inclusive_scan(u32 v, u32* scratch, u32* total) {
    u32 lane = lane_id(), warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    u32 x = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        u32 y = __shfl_up_sync(0xffffffffu, x, o);
        if (lane >= (u32)o) x += y;
    }
    __syncthreads();  // protects scratch against a previous use
    if (lane == 31) scratch[warp] = x;
    __syncthreads();
    if (warp == 0) {
        u32 w = lane < nwarps ? scratch[lane] : 0;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            u32 y = __shfl_up_sync(0xffffffffu, w, o);
            if (lane >= (u32)o) w += y;
        }
        if (lane < nwarps) scratch[lane] = w;
        if (lane == 31) scratch[32] = w;
    }
    __syncthreads();
    if (warp > 0) x += scratch[warp - 1];
    *total = scratch[32];
    return x;
}

// Given a histogram hist[0..nb) in shared memory and 1 <= need <= sum(hist),
// find the bucket b that holds the need-th entry counted from the TOP bucket
// downwards, and `above` = entries in buckets > b.  All threads call; the
// results are returned to every thread.  `res` holds 2 words, `scratch` 33.
template <int PER>
__device__ __forceinline__ void find_bucket(const u32* hist, int nb, u32 need, u32* scratch,
                                            u32* res, u32* b_out, u32* above_out) {
    // thread t owns the PER buckets nb-1-PER*t ... nb-PER-PER*t (descending)
    int top = nb - 1 - PER * (int)threadIdx.x;
    u32 local = 0;
#pragma unroll
    for (int i = 0; i < PER; ++i) {
        int b = top - i;
        if (b >= 0) local += hist[b];
    }
    u32 total;
    u32 incl = block_inclusive_scan(local, scratch, &total);
    u32 excl = incl - local;
    if (excl < need && need <= incl) {
        u32 run = excl;
#pragma unroll
        for (int i = 0; i < PER; ++i) {
            int b = top - i;
            if (b >= 0) {
                u32 h = hist[b];
                if (run < need && need <= run + h) { res[0] = (u32)b; res[1] = run; }
                run += h;
            }
        }
    }
    __syncthreads();
    *b_out = res[0];
    *above_out = res[1];
    __syncthreads();
}

}  // namespace tk
