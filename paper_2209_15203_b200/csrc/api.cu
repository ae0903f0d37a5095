// Host side of libtopk: argument checking, workspace layout, launch sequences.
// The C ABI is declared and documented in include/topk.h.
#include "../../include/topk.h"

#include <math.h>
#include <stddef.h>
#include <stdio.h>
#include <string.h>
#include <new>

#include "aggregate.cuh"
#include "common.cuh"
#include "diag.cuh"
#include "select.cuh"
#include "sort.cuh"

using namespace tk;

namespace {

constexpr size_t kAlign = 256;
constexpr int kMaxEvents = 256;

size_t align_up(size_t v) { return (v + kAlign - 1) / kAlign * kAlign; }

struct DeviceInfo {
    bool ready = false;
    int sms = 0;
    int general_grid = 0;  // co-resident CTAs of general_kernel
    int select_grid = 0;   // co-resident CTAs of the grid-wide select_kernel
};
DeviceInfo g_dev[64];

int device_info(DeviceInfo** out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return TK_ERR_CUDA;
    DeviceInfo& di = g_dev[dev];
    if (!di.ready) {
        int coop = 0, per_sm = 0;
        if (cudaDeviceGetAttribute(&di.sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return TK_ERR_CUDA;
        if (cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess || !coop) return TK_ERR_CUDA;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, general_kernel, kGeneralThreads, 0) != cudaSuccess ||
            per_sm < 1)
            return TK_ERR_CUDA;
        di.general_grid = per_sm * di.sms;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, select_kernel<true, false>, kSelectThreads, 0) != cudaSuccess ||
            per_sm < 1)
            return TK_ERR_CUDA;
        di.select_grid = per_sm * di.sms;
        di.ready = true;
    }
    *out = &di;
    return TK_OK;
}

// ---- buffers of one batched selection -------------------------------------------------------
struct SelectBufs {
    RowState* rs = nullptr;   // [rows]
    u32* hist = nullptr;      // [rows][kHistBins], zero at rest
    u32* smax = nullptr;      // [rows][kSampleSlots]
    uint2* cand = nullptr;    // [rows][cap]
    uint2* out = nullptr;     // [rows][K]
    u32 cap = 0;
    u32 tpr_filter = 0;       // tiles per row of the filter kernel / of the multi-pass kernel
    u32 tpr_filter_ef = 0;    // ... of the filter kernel with error memories (smaller tiles)
    u32 tpr_general = 0;
};

struct SelectLayout {
    size_t off_rs, off_hist, off_smax, off_cand, off_out, bytes;
    u32 cap, tpr_filter, tpr_filter_ef, tpr_general;
};

u32 candidate_capacity(int64_t d, int64_t K) {
    int64_t cap = 4 * K + 8192;
    if (cap > d) cap = d;
    return (u32)cap;
}

bool sampled_path(int64_t d, int64_t K, bool force_general) { return !force_general && d >= 131072 && K * 64 <= d; }

// The sample the prediction kernel takes of every row: ~128*d/K values (about 128 members of the top K;
// fewer when that would take more than the kernel's loads per thread), as whole 128-byte lines.
struct SamplePlan {
    int turns;        // 16-byte loads per sampling thread
    u64 stride_fp;    // 32.32 fixed-point distance between the sampled lines
    u32 rank;         // the bound is the rank-th largest of the per-thread-pair maxima
    double crowd;     // see below
};

// `light`: the two-CTAs-per-SM variant (many rows); `fused`: with error memories, two loads per value.
// crowd = 8 * rank / sampled fraction.  A thread pair keeps one maximum of 8 neighbouring sampled values,
// so when the K largest sit packed in one block of R values the sample holds about R*fraction/8 maxima
// from it; if that is below `rank` the bound drops to the level of the values outside and the whole
// block qualifies.  Lists of `crowd` entries (plus slack) still hold such a block, and a bigger block
// fills `rank` maxima by itself.
SamplePlan plan_sample(int64_t d, int64_t K, bool light, bool fused) {
    SamplePlan sp;
    const int64_t per_turn = 4 * 2 * (int64_t)kSampleSlots;          // values read per turn
    int64_t max_turns = light ? kPredictLightTurns : kPredictMaxTurns;
    if (fused) max_turns /= 2;
    int64_t want = (128 * (d / K) + per_turn - 1) / per_turn;
    int64_t lim = d / (8 * per_turn) < max_turns ? d / (8 * per_turn) : max_turns;
    sp.turns = (int)(want < 1 ? 1 : (want > lim ? lim : want));
    if (sp.turns < 1) sp.turns = 1;
    u64 lines = (u64)sp.turns * (2 * kSampleSlots / 8);
    sp.stride_fp = ((u64)(d - 32) << 32) / (lines - 1);                  // run g starts near g*(d-32)/(lines-1)
    double ks = (double)K * 32.0 * (double)lines / (double)d;          // expected top-K members in the sample
    double r = ceil(ks + 6.0 * sqrt(ks) + 4.0);
    sp.rank = (u32)(r > kSampleSlots / 2 ? kSampleSlots / 2 : r);
    sp.crowd = 8.0 * (double)sp.rank * (double)d / (32.0 * (double)lines);
    return sp;
}

constexpr int kSmsAssumed = 148;  // B200; only sizes the lists below (a wrong guess costs speed in a rare case, nothing else)

bool light_sampling(int64_t rows, int sms) { return rows * kPredictCtas > 2 * (int64_t)sms; }

// Candidate capacity per row of the batched selection: room for 4K + 8192 entries and, on the sampled
// path, for a block of large values the sample under-counts (plan_sample), at most 2^20 entries.
u32 wide_capacity(int64_t rows, int64_t d, int64_t K) {
    int64_t cap = candidate_capacity(d, K);
    if (!sampled_path(d, K, false)) return (u32)cap;
    bool light = light_sampling(rows, kSmsAssumed);
    double crowd = plan_sample(d, K, light, false).crowd, crowd_ef = plan_sample(d, K, light, true).crowd;
    if (crowd_ef > crowd) crowd = crowd_ef;
    int64_t want = (int64_t)(1.15 * crowd) + 2 * K;
    if (want > ((int64_t)1 << 20)) want = (int64_t)1 << 20;
    if (want > cap) cap = want;
    if (cap > d) cap = d;
    return (u32)cap;
}

SelectLayout select_layout(int64_t rows, int64_t d, int64_t K, bool wide = true) {
    SelectLayout L;
    L.cap = wide ? wide_capacity(rows, d, K) : candidate_capacity(d, K);
    int64_t nv = (d + 3) / 4;
    int64_t tf = (nv + kFilterTileVecs - 1) / kFilterTileVecs, tg = (nv + kGeneralTileVecs - 1) / kGeneralTileVecs;
    int64_t te = (nv + kFilterEfTileVecs - 1) / kFilterEfTileVecs;
    L.tpr_filter = (u32)(tf < 1 ? 1 : tf);
    L.tpr_filter_ef = (u32)(te < 1 ? 1 : te);
    L.tpr_general = (u32)(tg < 1 ? 1 : tg);
    size_t o = 0;
    L.off_rs = o;   o += align_up((size_t)rows * sizeof(RowState));
    L.off_hist = o; o += align_up((size_t)rows * kHistBins * sizeof(u32));
    L.off_smax = o; o += align_up((size_t)rows * kSampleSlots * sizeof(u32));
    L.off_cand = o; o += align_up((size_t)rows * L.cap * sizeof(uint2));
    L.off_out = o;  o += align_up((size_t)rows * (size_t)K * sizeof(uint2));
    L.bytes = o;
    return L;
}

SelectBufs bind(const SelectLayout& L, char* base) {
    SelectBufs b;
    b.rs = (RowState*)(base + L.off_rs);
    b.hist = (u32*)(base + L.off_hist);
    b.smax = (u32*)(base + L.off_smax);
    b.cand = (uint2*)(base + L.off_cand);
    b.out = (uint2*)(base + L.off_out);
    b.cap = L.cap;
    b.tpr_filter = L.tpr_filter;
    b.tpr_filter_ef = L.tpr_filter_ef;
    b.tpr_general = L.tpr_general;
    return b;
}

// ---- sort scratch ---------------------------------------------------------------------------
struct SortLayout {
    size_t off_tmp, off_cnt, bytes;
    u32 tiles;
};

SortLayout sort_layout(int64_t rows, int64_t n) {
    SortLayout L;
    L.tiles = (u32)((n + kSortTile - 1) / kSortTile);
    if (L.tiles < 1) L.tiles = 1;
    size_t o = 0;
    L.off_tmp = o; o += align_up((size_t)rows * (size_t)n * sizeof(uint2));
    L.off_cnt = o; o += align_up((size_t)rows * 256 * L.tiles * sizeof(u32));
    L.bytes = o;
    return L;
}

// ---- per-device scratch pool (tk_topk and the inspection calls) ------------------------------
// One region per device, shared by every user whatever its stream: a user makes its stream wait
// for the previous user's last kernel before it touches the region (pool_get) and leaves an event
// behind its own last kernel (pool_done).
struct Pool {
    char* base = nullptr;
    size_t bytes = 0;
    cudaEvent_t last = nullptr;  // recorded behind the last kernel of the most recent user
    bool pending = false;
};
Pool g_pool[64];

bool stream_is_capturing(cudaStream_t s) {
    cudaStreamCaptureStatus st = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(s, &st) != cudaSuccess) { cudaGetLastError(); return false; }
    return st != cudaStreamCaptureStatusNone;
}

int pool_get(size_t bytes, char** out, cudaStream_t stream) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return TK_ERR_CUDA;
    Pool& p = g_pool[dev];
    if (p.pending && !stream_is_capturing(stream)) {
        if (cudaStreamWaitEvent(stream, p.last, 0) != cudaSuccess) { cudaGetLastError(); return TK_ERR_CUDA; }
    }
    if (p.bytes < bytes) {
        if (p.base) {
            if (cudaDeviceSynchronize() != cudaSuccess) return TK_ERR_CUDA;
            cudaFree(p.base);
            p.base = nullptr;
            p.bytes = 0;
        }
        size_t want = bytes + bytes / 8;
        if (cudaMalloc((void**)&p.base, want) != cudaSuccess) {
            cudaGetLastError();
            p.base = nullptr;
            return TK_ERR_ALLOC;
        }
        p.bytes = want;
    }
    *out = p.base;
    return TK_OK;
}

// Call after the last kernel that uses the region has been enqueued on `stream`.
void pool_done(cudaStream_t stream) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return;
    Pool& p = g_pool[dev];
    if (stream_is_capturing(stream)) return;
    if (!p.last && cudaEventCreateWithFlags(&p.last, cudaEventDisableTiming) != cudaSuccess) {
        cudaGetLastError();
        p.last = nullptr;
        return;
    }
    if (cudaEventRecord(p.last, stream) == cudaSuccess) p.pending = true;
    else cudaGetLastError();
}

bool aligned4(const void* p) { return p != nullptr && ((uintptr_t)p & 3u) == 0; }

int bits_of(int64_t v) {  // number of significant bits of v >= 0
    int b = 0;
    while (v > 0) { ++b; v >>= 1; }
    return b;
}

// Candidate capacity under tk_set_cand_cap: never above what the buffers hold, never below K.
u32 capped(u32 laid_out, int64_t limit, int64_t K) {
    int64_t c = limit < K ? K : limit;
    return c < (int64_t)laid_out ? (u32)c : laid_out;
}

}  // namespace

// ---- the context ------------------------------------------------------------------------------
struct tk_ctx {
    int64_t d = 0, K_up = 0, K_down = 0;
    int32_t N = 0;
    cudaStream_t stream = nullptr;
    char* ws = nullptr;
    size_t ws_bytes = 0;
    // workspace views
    Ctrl* ctrl = nullptr;
    float* p = nullptr;
    SelectBufs up;             // uplink selection; up.out = the N uplink messages
    RowState* uni = nullptr;   // state of the union list / downlink selection
    u32* head = nullptr;       // [d] dense server buffer, zero at rest
    u32* next = nullptr;       // [N*K_up] chain links, or (slot scheme) one mark word per entry, zero at rest
    u32* slots = nullptr;      // [N*K_up][slot_row_words] slot table, zero at rest; NULL when the server step uses chains
    u32 slot_row_words = 0;
    uint2* U = nullptr;        // [ucap] aggregate over the union
    uint2* sel = nullptr;      // [ucap] downlink message (unordered)
    u32* ghist = nullptr;      // [kGridScratchWords] scratch of the grid-wide select, zero at rest
    u32 ucap = 0;
    // host state
    int force_general = 0;
    int bound_reuse = 1;       // tk_set_bound_reuse
    int64_t cand_cap = 0;      // tk_set_cand_cap: 0 = the capacity the workspace was laid out for
    int diagnostics = 0;
    int profile = 0;           // 0 = off, n = timestamp the streaming pass of every n-th step
    int64_t steps_seen = 0;
    int last_mode = -1;
    int64_t last_kdown = 0;
    int64_t launches = 0;
    cudaEvent_t ev[2 * kMaxEvents] = {};
    bool ev_ready = false;
    int ev_used = 0;
    float* stage_g = nullptr;  // tk_step_host staging
    float* stage_w = nullptr;
    // error memories (tk_ef_attach)
    float* eps = nullptr;      // [N][d]
    float* delta = nullptr;    // [d]
    SelectBufs down;           // selection over the dense server vector (1 row of d)
    int64_t ef_kdown = 0;      // largest K_down the attached buffers serve
    // gap-constant diagnostics (tk_set_diagnostics level 2): own allocation
    char* diag_mem = nullptr;
    float* diag_Da = nullptr;  // [d] dense sum of the compensated vectors (+ delta)
    float* diag_Z = nullptr;   // [d] scratch for sparse differences, zero at rest
    double* diag_sums = nullptr;  // [0] = squared denominator, [1] = squared numerator
    SelectBufs diag_sel;       // Top_K over diag_Da
    int64_t diag_kdown = 0;
    const uint2* diag_other_ef() const { return down.out; }
    // captured steps (tk_set_graph)
    struct StepKey {
        float* w; const float* g; float alpha; int mode; int64_t K_down; int force_general, diagnostics;
        float* eps;
        bool operator==(const StepKey& o) const {
            return w == o.w && g == o.g && memcmp(&alpha, &o.alpha, sizeof alpha) == 0 && mode == o.mode &&
                   K_down == o.K_down && force_general == o.force_general && diagnostics == o.diagnostics && eps == o.eps;
        }
    };
    struct StepGraph { StepKey key; cudaGraphExec_t exec; int64_t launches; uint64_t used; };
    static constexpr int kMaxGraphs = 16;
    StepGraph graphs[kMaxGraphs] = {};
    int n_graphs = 0;
    uint64_t graph_clock = 0;
    int use_graphs = 0;
};

namespace {

struct CtxLayout {
    size_t off_ctrl, off_p, off_sel_up, off_uni, off_head, off_next, off_slots, off_U, off_sel, off_ghist, bytes;
    size_t slot_words;  // 0: the server step uses chains
    u32 slot_row_words;
    SelectLayout up;
    u32 ucap;
};

#ifndef TK_SLOT_BUDGET
#define TK_SLOT_BUDGET ((size_t)1 << 30)
#endif
constexpr size_t kSlotBudget = TK_SLOT_BUDGET;  // largest slot table of the server step, bytes (0: always chains)

bool sizes_ok(int64_t d, int64_t N, int64_t K_up, int64_t K_down) {
    return d >= 1 && d < ((int64_t)1 << 31) && N >= 1 && N <= 65535 && K_up >= 1 && K_up <= d &&
           K_down >= 1 && K_down <= d && N * K_up < ((int64_t)1 << 31);
}

CtxLayout ctx_layout(int64_t d, int64_t N, int64_t K_up) {
    CtxLayout L;
    L.up = select_layout(N, d, K_up);
    int64_t ucap = N * K_up < d ? N * K_up : d;
    L.ucap = (u32)ucap;
    size_t o = 0;
    L.off_ctrl = o;   o += align_up(sizeof(Ctrl));
    L.off_p = o;      o += align_up((size_t)N * sizeof(float));
    L.off_sel_up = o; o += L.up.bytes;
    L.off_uni = o;    o += align_up(sizeof(RowState));
    L.off_head = o;   o += align_up((size_t)d * sizeof(u32));
    L.off_next = o;   o += align_up((size_t)(N * K_up) * sizeof(u32));
    // slot table of the server step: per uplink entry one row of a 128-bit mask plus one word per worker
    // (rounded up to 16 bytes), when the workers are few and the table stays within kSlotBudget bytes
    L.slot_row_words = 0;
    L.slot_words = 0;
    {
        size_t row_words = kSlotMaskWords + (size_t)((N + 3) / 4 * 4);
        if (N <= kSlotWorkers && row_words * (size_t)(N * K_up) * sizeof(u32) <= kSlotBudget) {
            L.slot_row_words = (u32)row_words;
            L.slot_words = row_words * (size_t)(N * K_up);
        }
    }
    L.off_slots = o;  o += align_up(L.slot_words * sizeof(u32));
    L.off_U = o;      o += align_up((size_t)ucap * sizeof(uint2));
    L.off_sel = o;    o += align_up((size_t)ucap * sizeof(uint2));
    L.off_ghist = o;  o += align_up((size_t)kGridScratchWords * sizeof(u32));
    L.bytes = o;
    return L;
}

// CTAs per row of the cluster select: the kernel issues a fixed string of instructions per
// register-held candidate and level, so few candidates per thread (about 4) on many SMs beats
// many per thread on few; at least 4 CTAs when there are few rows, but never so many that the
// clusters of all rows stop fitting in one wave.
int cluster_size_for(int64_t entries, int64_t rows, int sms) {
    // few rows (their clusters of 8 fill at most half the SMs): half as many candidates per thread — measured
    // on 8 rows of 25-35k candidates, clusters of 8 select 2 us faster than clusters of 4; on 16 rows 4 us slower
    const int per_thread = rows * 16 <= sms ? (kSelectPerThread + 1) / 2 : kSelectPerThread;
    int64_t per_cta = (int64_t)kSelectThreads * per_thread;
    int64_t need = (entries + per_cta - 1) / per_cta;
    int cs_need = 1;
    while (cs_need < 8 && cs_need < need) cs_need *= 2;
    int cs_fill = 1;
    while (cs_fill < 8 && (int64_t)cs_fill * 2 * rows <= sms) cs_fill *= 2;
    int floor4 = cs_fill < 4 ? cs_fill : 4;
    int cs = cs_need > floor4 ? cs_need : floor4;
    return cs < cs_fill ? cs : cs_fill;
}

#ifndef TK_PDL
#define TK_PDL 1
#endif
#ifndef TK_COOP_PDL
#define TK_COOP_PDL 1
#endif

// Launch with the programmatic-serialization attribute (the kernel calls dependency_wait()) and,
// optionally, a cluster size.
template <typename... KArgs, typename... Args>
int launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, int cluster,
                     Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    int n = 0;
    if (cluster > 0) {
        attr[n].id = cudaLaunchAttributeClusterDimension;
        attr[n].val.clusterDim.x = (unsigned)cluster;
        attr[n].val.clusterDim.y = 1;
        attr[n].val.clusterDim.z = 1;
        ++n;
    }
    if (TK_PDL) {
        attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n].val.programmaticStreamSerializationAllowed = 1;
        ++n;
    }
    cfg.attrs = attr;
    cfg.numAttrs = (unsigned)n;
    if (cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...) != cudaSuccess) {
        cudaGetLastError();
        return TK_ERR_CUDA;
    }
    return TK_OK;
}

#define TK_LAUNCH_CHECK()                                   \
    do {                                                    \
        if (cudaGetLastError() != cudaSuccess) return TK_ERR_CUDA; \
    } while (0)

int launch_select(cudaStream_t stream, int rows, int cs, const uint2* lists, size_t list_stride, u32 cap,
                  RowState* rs, u32 K, uint2* out, size_t out_stride, ApplyArgs apply, LinkArgs link, Ctrl* ctrl) {
    u32* no_ghist = nullptr;
    DenseArgs no_dense = {nullptr, nullptr, 0};
    return launch_dependent(select_kernel<false, false>, dim3((unsigned)(rows * cs)), dim3(kSelectThreads), 0, stream, cs, lists,
                            list_stride, cap, rs, K, out, out_stride, apply, link, ctrl, no_ghist, no_dense, 0);
}

// CTAs per row when the selection reads short rows directly: enough to keep (nearly) the whole row in
// registers (what does not fit is read again at every level).  0 when the row is too long for that or the
// clusters of all rows would not fit one wave — measured: 100 rows of 51k as 400 CTAs take longer than
// the multi-pass kernel, 20 rows of 29k as 80 CTAs take half as long.
int dense_cluster_size(int64_t d, int64_t rows, int sms) {
    const int64_t held = (int64_t)kSelectRegs * kSelectThreads;  // entries one CTA keeps in registers
    int cs = 1;
    while (cs < 8 && cs * held < d) cs *= 2;
    if (cs * held * 9 / 8 < d || rows * cs > (int64_t)sms) return 0;  // a remainder of an eighth may be re-read
    return cs;
}

// The same selection straight from short rows (no candidate lists, no bound).
int launch_select_dense(cudaStream_t stream, int rows, int cs, const float* x, int64_t d, RowState* rs, u32 K, uint2* out,
                        ApplyArgs apply, LinkArgs link, Ctrl* ctrl, RowState* also_reset, bool stats) {
    u32* no_ghist = nullptr;
    const uint2* no_lists = nullptr;
    DenseArgs dense = {x, also_reset, stats ? 1 : 0};
    return launch_dependent(select_kernel<false, true>, dim3((unsigned)(rows * cs)), dim3(kSelectThreads), 0, stream, cs, no_lists,
                            (size_t)d, (u32)d, rs, K, out, (size_t)K, apply, link, ctrl, no_ghist, dense, 0);
}

// One long list selected by the whole grid (cooperative launch).
int launch_select_grid(cudaStream_t stream, int ctas, const uint2* list, u32 cap, RowState* rs, u32 K, uint2* out,
                       ApplyArgs apply, Ctrl* ctrl, u32* ghist, bool stats, bool first_level_counted) {
    size_t stride = cap;
    LinkArgs nolink = {nullptr, nullptr, 0, 0, nullptr, 0, stats ? 1 : 0};
    DenseArgs no_dense = {nullptr, nullptr, 0};
    int prebuilt = first_level_counted ? 1 : 0;  // the server sum has counted the first level into ghist
    void* args[] = {(void*)&list, (void*)&stride, (void*)&cap, (void*)&rs,  (void*)&K,    (void*)&out,
                    (void*)&stride, (void*)&apply, (void*)&nolink, (void*)&ctrl, (void*)&ghist, (void*)&no_dense,
                    (void*)&prebuilt};
    if (cudaLaunchCooperativeKernel((void*)select_kernel<true, false>, dim3(ctas), dim3(kSelectThreads), args, 0, stream) !=
        cudaSuccess) {
        cudaGetLastError();
        return TK_ERR_CUDA;
    }
    return TK_OK;
}

// Exact Top_K of every row of x into b.out ([rows][K], arbitrary order).  ev0/ev1, when
// given, bracket the streaming pass.  *launches is advanced by the kernels enqueued.
//
// With error memories (ef.eps != NULL) the vector selected from is a = eps + alpha*x, which
// also replaces eps; the streaming pass computes it on the fly when x and eps are equally
// aligned, otherwise a separate pass does and the selection then reads eps alone.
int run_select(cudaStream_t stream, const float* x, int64_t rows, int64_t d, int64_t K, const SelectBufs& b,
               Ctrl* ctrl, bool force_general, cudaEvent_t ev0, cudaEvent_t ev1, int64_t* launches,
               RowState* also_reset = nullptr, LinkArgs link = LinkArgs{nullptr, nullptr, 0, 0},
               EfArgs ef = EfArgs{nullptr, 0.0f}, ApplyArgs apply = ApplyArgs{nullptr, 0.0f}, bool stats = false,
               bool reuse = false /* rows may keep the bound of their last selection (predict_kernel) */) {
    DeviceInfo* di = nullptr;
    int rc = device_info(&di);
    if (rc != TK_OK) return rc;
    const bool predict = sampled_path(d, K, force_general);
    bool fused = ef.eps != nullptr && predict && ((((uintptr_t)x) ^ ((uintptr_t)ef.eps)) & 15u) == 0;
    if (ef.eps && !fused) {
        size_t n = (size_t)rows * (size_t)d;
        size_t blocks = (n + 1023) / 1024;
        if (blocks > (size_t)di->sms * 16) blocks = (size_t)di->sms * 16;
        compensate_kernel<<<(unsigned)blocks, 256, 0, stream>>>(ef.eps, x, ef.alpha, n);
        TK_LAUNCH_CHECK();
        *launches += 1;
        x = ef.eps;            // from here on this is an ordinary selection over eps
        ef.eps = nullptr;
    }
    // rows too short for a sampled bound are selected from directly (unless the multi-pass path is forced)
    const int dense_cs = (!predict && !force_general) ? dense_cluster_size(d, rows < kMaxRowsPerLaunch ? rows : kMaxRowsPerLaunch, di->sms) : 0;
    const bool dense = dense_cs > 0;
    int turns = 1;
    u64 stride_fp = 0;
    u32 rank = 0;
    if (predict) {
        // many rows: the sampling CTAs of all rows should fit few waves, so cap the loads per thread at
        // what the two-CTAs-per-SM variant holds (the sample only sets how many candidates pass)
        SamplePlan sp = plan_sample(d, K, light_sampling(rows, di->sms), fused);
        turns = sp.turns;
        stride_fp = sp.stride_fp;
        rank = sp.rank;
    }
    for (int64_t r0 = 0; r0 < rows; r0 += kMaxRowsPerLaunch) {
        int nr = (int)(rows - r0 < kMaxRowsPerLaunch ? rows - r0 : kMaxRowsPerLaunch);
        const float* xb = x + (size_t)r0 * (size_t)d;
        RowState* rs = b.rs + r0;
        u32* hist = b.hist + (size_t)r0 * kHistBins;
        u32* smax = b.smax + (size_t)r0 * kSampleSlots;
        uint2* cand = b.cand + (size_t)r0 * b.cap;
        uint2* out = b.out + (size_t)r0 * (size_t)K;
        EfArgs efb = {fused ? ef.eps + (size_t)r0 * (size_t)d : nullptr, ef.alpha};
        if (predict) {
            RowState* ar = r0 == 0 ? also_reset : nullptr;
            const bool light = turns <= (fused ? kPredictLightTurns / 2 : kPredictLightTurns);
            dim3 pg(kPredictCtas, nr);
            if (fused && light)
                predict_kernel<true, true><<<pg, kPredictThreads, 0, stream>>>(xb, d, turns, stride_fp, rank, (u32)K, rs, smax, ar, efb, ctrl, reuse ? 1 : 0, (const RowState*)link.uni);
            else if (fused)
                predict_kernel<true, false><<<pg, kPredictThreads, 0, stream>>>(xb, d, turns, stride_fp, rank, (u32)K, rs, smax, ar, efb, ctrl, reuse ? 1 : 0, (const RowState*)link.uni);
            else if (light)
                predict_kernel<false, true><<<pg, kPredictThreads, 0, stream>>>(xb, d, turns, stride_fp, rank, (u32)K, rs, smax, ar, efb, ctrl, reuse ? 1 : 0, (const RowState*)link.uni);
            else
                predict_kernel<false, false><<<pg, kPredictThreads, 0, stream>>>(xb, d, turns, stride_fp, rank, (u32)K, rs, smax, ar, efb, ctrl, reuse ? 1 : 0, (const RowState*)link.uni);
            TK_LAUNCH_CHECK();
            if (ev0 && r0 == 0) cudaEventRecord(ev0, stream);
            u32 tprf = fused ? b.tpr_filter_ef : b.tpr_filter;
            u64 tiles = (u64)nr * tprf;
            u64 resident = (u64)di->sms * kFilterCtasPerSm;  // one wave: a second, partial wave runs at low occupancy
            u32 grid = (u32)(tiles < resident ? tiles : resident);
            u32 parts = 1;
            if (tiles >= 4 * resident) {  // about one range per row, but never fewer than kFilterMinCpp CTAs per range
                u32 most = grid / kFilterMinCpp;
                parts = (u32)nr < most ? (u32)nr : most;
                if (parts < 1) parts = 1;
            }
            u32 cpp = grid / parts;
            size_t shm = (size_t)nr * sizeof(u64);
            if (fused && stats)
                rc = launch_dependent(filter_kernel<true, true>, dim3(grid), dim3(kFilterThreads), shm, stream, 0, xb, nr, d, tprf,
                                      parts, cpp, rs, cand, b.cap, efb, ctrl);
            else if (fused)
                rc = launch_dependent(filter_kernel<true, false>, dim3(grid), dim3(kFilterThreads), shm, stream, 0, xb, nr, d, tprf,
                                      parts, cpp, rs, cand, b.cap, efb, ctrl);
            else if (stats)
                rc = launch_dependent(filter_kernel<false, true>, dim3(grid), dim3(kFilterThreads), shm, stream, 0, xb, nr, d, tprf,
                                      parts, cpp, rs, cand, b.cap, efb, ctrl);
            else
                rc = launch_dependent(filter_kernel<false, false>, dim3(grid), dim3(kFilterThreads), shm, stream, 0, xb, nr, d, tprf,
                                      parts, cpp, rs, cand, b.cap, efb, ctrl);
            if (rc != TK_OK) return rc;
            if (fused) xb = efb.eps;  // the compensated vector now sits in eps: what a re-filter must read
            if (ev1 && r0 == 0) cudaEventRecord(ev1, stream);
            *launches += 2;
        } else if (dense) {
            // short rows: one kernel selects straight from the rows
            LinkArgs lk = link;
            lk.row_base = (u32)r0;
            lk.stats = stats ? 1 : 0;
            if (lk.zero_src) lk.zero_src += (size_t)r0 * lk.zero_stride;
            if (ev0 && r0 == 0) cudaEventRecord(ev0, stream);
            rc = launch_select_dense(stream, nr, dense_cs, xb, d, rs, (u32)K, out, apply, lk, ctrl,
                                     r0 == 0 ? also_reset : nullptr, stats);
            if (rc != TK_OK) return rc;
            if (ev1 && r0 == 0) cudaEventRecord(ev1, stream);
            *launches += 1;
            continue;
        } else {
            reset_rows_kernel<<<(nr + 255) / 256, 256, 0, stream>>>(rs, nr, r0 == 0 ? also_reset : nullptr);
            TK_LAUNCH_CHECK();
            *launches += 1;
        }
        {
            u32 Ku = (u32)K, tpr = b.tpr_general, cap = b.cap;
            int st = stats ? 1 : 0;
            void* args[] = {(void*)&xb, (void*)&nr, (void*)&d, (void*)&Ku, (void*)&tpr, (void*)&cap,
                            (void*)&rs,  (void*)&hist, (void*)&cand, (void*)&ctrl, (void*)&st};
            // without a prediction the multi-pass kernel is the streaming pass that gets timed
            if (!predict && ev0 && r0 == 0) cudaEventRecord(ev0, stream);
            // no more CTAs than tiles: a grid-wide barrier costs more the more CTAs take part
            u64 gtiles = (u64)nr * b.tpr_general;
            unsigned ggrid = (unsigned)(gtiles < (u64)di->general_grid ? gtiles : (u64)di->general_grid);
            if (ggrid < 1) ggrid = 1;
#if TK_COOP_PDL
            {
                cudaLaunchConfig_t cfg = {};
                cfg.gridDim = dim3(ggrid);
                cfg.blockDim = dim3(kGeneralThreads);
                cfg.stream = stream;
                cudaLaunchAttribute attr[2];
                attr[0].id = cudaLaunchAttributeCooperative;
                attr[0].val.cooperative = 1;
                attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
                attr[1].val.programmaticStreamSerializationAllowed = 1;
                cfg.attrs = attr;
                cfg.numAttrs = 2;
                if (cudaLaunchKernelExC(&cfg, (const void*)general_kernel, args) != cudaSuccess) {
                    cudaGetLastError();
                    return TK_ERR_CUDA;
                }
            }
#else
            if (cudaLaunchCooperativeKernel((void*)general_kernel, dim3(ggrid), dim3(kGeneralThreads), args,
                                            0, stream) != cudaSuccess) {
                cudaGetLastError();
                return TK_ERR_CUDA;
            }
#endif
            if (!predict && ev1 && r0 == 0) cudaEventRecord(ev1, stream);
            *launches += 1;
        }
        int64_t expect = predict ? 2 * K : (int64_t)b.cap;
        LinkArgs lk = link;
        lk.row_base = (u32)r0;
        lk.stats = stats ? 1 : 0;
        if (lk.zero_src) lk.zero_src += (size_t)r0 * lk.zero_stride;
        rc = launch_select(stream, nr, cluster_size_for(expect, nr, di->sms), cand, b.cap, b.cap, rs, (u32)K, out, (size_t)K, apply,
                           lk, ctrl);
        if (rc != TK_OK) return rc;
        *launches += 1;
    }
    return TK_OK;
}

// Sort `rows` segments of (index, value) entries by index into idx_out / val_out.
// Segment r starts at src + r*stride and has min(n_fixed, counts[r*count_stride]) entries
// (n_fixed when counts is NULL).  tmp / cnt come from sort_layout(rows, n_fixed).
int run_sort(cudaStream_t stream, uint2* src, size_t stride, const u32* counts, size_t count_stride, u32 n_fixed,
             int64_t rows, int64_t d, uint2* tmp, u32* cnt, u32 tiles, int32_t* idx_out, float* val_out,
             size_t out_stride, int64_t* launches) {
    if (n_fixed == 0 || rows == 0) return TK_OK;
    int passes = (bits_of(d - 1) + 7) / 8;
    if (passes < 1) passes = 1;
    uint2* a = src;
    uint2* bbuf = tmp;
    for (int64_t r0 = 0; r0 < rows; r0 += 32768) {
        int nr = (int)(rows - r0 < 32768 ? rows - r0 : 32768);
        uint2* cur = a + (size_t)r0 * stride;
        uint2* oth = bbuf + (size_t)r0 * stride;
        const u32* cn = counts ? counts + (size_t)r0 * count_stride : nullptr;
        u32* c = cnt + (size_t)r0 * 256 * tiles;
        for (int p = 0; p < passes; ++p) {
            int shift = 8 * p;
            bool final_pass = p == passes - 1;
            sort_local_kernel<<<dim3(tiles, nr), kSortTile, 0, stream>>>(cur, stride, cn, count_stride, n_fixed, shift,
                                                                        tiles, c);
            TK_LAUNCH_CHECK();
            sort_scan_kernel<<<nr, 256, 0, stream>>>(c, tiles);
            TK_LAUNCH_CHECK();
            sort_scatter_kernel<<<dim3(tiles, nr), kSortTile, 0, stream>>>(
                cur, stride, cn, count_stride, n_fixed, shift, tiles, c, final_pass ? nullptr : oth,
                idx_out + (size_t)r0 * out_stride, val_out + (size_t)r0 * out_stride, out_stride);
            TK_LAUNCH_CHECK();
            *launches += 3;
            uint2* t = cur; cur = oth; oth = t;
        }
    }
    return TK_OK;
}

}  // namespace

namespace {
void drop_graphs(tk_ctx* c) {
    for (int i = 0; i < c->n_graphs; ++i) cudaGraphExecDestroy(c->graphs[i].exec);
    c->n_graphs = 0;
}

int diag_alloc(tk_ctx* c) {
    if (c->diag_mem && c->diag_kdown >= c->K_down) return TK_OK;
    drop_graphs(c);
    if (c->diag_mem) {
        cudaStreamSynchronize(c->stream);
        cudaFree(c->diag_mem);
        c->diag_mem = nullptr;
    }
    SelectLayout L = select_layout(1, c->d, c->K_down);
    size_t vec = align_up((size_t)c->d * sizeof(float));
    size_t bytes = 2 * vec + align_up(2 * sizeof(double)) + L.bytes;
    if (cudaMalloc((void**)&c->diag_mem, bytes) != cudaSuccess) {
        cudaGetLastError();
        c->diag_mem = nullptr;
        return TK_ERR_ALLOC;
    }
    c->diag_Da = (float*)c->diag_mem;
    c->diag_Z = (float*)(c->diag_mem + vec);
    c->diag_sums = (double*)(c->diag_mem + 2 * vec);
    c->diag_sel = bind(L, c->diag_mem + 2 * vec + align_up(2 * sizeof(double)));
    c->diag_kdown = c->K_down;
    if (cudaMemsetAsync(c->diag_Z, 0, vec, c->stream) != cudaSuccess ||
        cudaMemsetAsync(c->diag_sums, 0, 2 * sizeof(double), c->stream) != cudaSuccess ||
        cudaMemsetAsync(c->diag_sel.rs, 0, sizeof(RowState), c->stream) != cudaSuccess ||
        cudaMemsetAsync(c->diag_sel.hist, 0, (size_t)kHistBins * sizeof(u32), c->stream) != cudaSuccess ||
        cudaStreamSynchronize(c->stream) != cudaSuccess) {
        cudaGetLastError();
        return TK_ERR_CUDA;
    }
    return TK_OK;
}
}  // namespace

// ---- C ABI --------------------------------------------------------------------------------------
extern "C" {

size_t tk_workspace_bytes(int64_t d, int32_t N, int64_t K_up, int64_t K_down) {
    if (!sizes_ok(d, N, K_up, K_down)) return 0;
    return ctx_layout(d, N, K_up).bytes;
}

int tk_init(tk_ctx** out, int64_t d, int32_t N, int64_t K_up, int64_t K_down, const float* p_host,
            void* workspace_dev, size_t workspace_bytes, void* cuda_stream) {
    if (!out) return TK_ERR_INVALID;
    *out = nullptr;
    if (!sizes_ok(d, N, K_up, K_down) || !p_host || !workspace_dev) return TK_ERR_INVALID;
    if (((uintptr_t)workspace_dev & (kAlign - 1)) != 0) return TK_ERR_INVALID;
    for (int q = 0; q < N; ++q)
        if (!isfinite(p_host[q]) || p_host[q] < 0.0f) return TK_ERR_INVALID;
    CtxLayout L = ctx_layout(d, N, K_up);
    if (workspace_bytes < L.bytes) return TK_ERR_ALLOC;
    DeviceInfo* di = nullptr;
    int rc = device_info(&di);
    if (rc != TK_OK) return rc;
    tk_ctx* c = new (std::nothrow) tk_ctx();
    if (!c) return TK_ERR_ALLOC;
    c->d = d; c->N = N; c->K_up = K_up; c->K_down = K_down;
    c->stream = (cudaStream_t)cuda_stream;
    c->ws = (char*)workspace_dev;
    c->ws_bytes = workspace_bytes;
    c->ctrl = (Ctrl*)(c->ws + L.off_ctrl);
    c->p = (float*)(c->ws + L.off_p);
    c->up = bind(L.up, c->ws + L.off_sel_up);
    c->uni = (RowState*)(c->ws + L.off_uni);
    c->head = (u32*)(c->ws + L.off_head);
    c->next = (u32*)(c->ws + L.off_next);
    c->slots = L.slot_words ? (u32*)(c->ws + L.off_slots) : nullptr;
    c->slot_row_words = L.slot_row_words;
    c->U = (uint2*)(c->ws + L.off_U);
    c->sel = (uint2*)(c->ws + L.off_sel);
    c->ghist = (u32*)(c->ws + L.off_ghist);
    c->ucap = L.ucap;
    // state that must be zero at rest: control block, row states, histograms, the dense buffer
    bool ok = cudaMemsetAsync(c->ctrl, 0, sizeof(Ctrl), c->stream) == cudaSuccess &&
              cudaMemsetAsync(c->up.rs, 0, (size_t)N * sizeof(RowState), c->stream) == cudaSuccess &&
              cudaMemsetAsync(c->up.hist, 0, (size_t)N * kHistBins * sizeof(u32), c->stream) == cudaSuccess &&
              cudaMemsetAsync(c->uni, 0, sizeof(RowState), c->stream) == cudaSuccess &&
              cudaMemsetAsync(c->ghist, 0, (size_t)kGridScratchWords * sizeof(u32), c->stream) == cudaSuccess &&
              cudaMemsetAsync(c->head, 0, (size_t)d * sizeof(u32), c->stream) == cudaSuccess &&
              (!c->slots || cudaMemsetAsync(c->slots, 0, L.slot_words * sizeof(u32), c->stream) == cudaSuccess) &&
              cudaMemsetAsync(c->next, 0, (size_t)(N * K_up) * sizeof(u32), c->stream) == cudaSuccess &&
              cudaMemcpyAsync(c->p, p_host, (size_t)N * sizeof(float), cudaMemcpyHostToDevice, c->stream) ==
                  cudaSuccess &&
              cudaStreamSynchronize(c->stream) == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        delete c;
        return TK_ERR_CUDA;
    }
    *out = c;
    return TK_OK;
}

namespace {

// Stages 2-4 on the messages in c->up.out (already threaded onto their chains).
int run_server(tk_ctx* c, float* w_dev, float alpha, int mode) {
    const bool bidir = (mode & TK_MODE_BIDIR) != 0, with_ef = (mode & TK_MODE_EF) != 0;
    const bool diag = c->diagnostics != 0;
    cudaStream_t s = c->stream;
    // with memories the step size is already inside the messages
    const float scale = with_ef ? 1.0f : alpha;
    u32 total = (u32)(c->N * c->K_up);
    u32 blocks = (total + kAggThreads - 1) / kAggThreads;
    DeviceInfo* di = nullptr;
    int rc = device_info(&di);
    if (rc != TK_OK) return rc;
    // the downlink selection: the union can hold up to ucap entries, about 4096 per CTA, at most one
    // co-resident wave.  With more than one CTA its first level is counted by the server sum already.
#ifndef TK_DOWN_PER_CTA
#define TK_DOWN_PER_CTA 4096
#endif
    int ctas = (int)((c->ucap + TK_DOWN_PER_CTA - 1) / TK_DOWN_PER_CTA);
    if (ctas > di->select_grid) ctas = di->select_grid;
    if (ctas < 1) ctas = 1;
    const bool prebuilt = bidir && !with_ef && ctas > 1;
    rc = launch_dependent(agg_reduce_kernel, dim3(blocks), dim3(kAggThreads), 0, s, 0, (const uint2*)c->up.out, total,
                              (u32)c->K_up, (const float*)c->p, c->head, c->next, c->slots, c->slot_row_words, c->uni, c->U,
                              c->ucap, w_dev,
                              scale, bidir ? 0 : 1, (bidir && with_ef) ? c->delta : (float*)nullptr, c->ctrl, (u32)c->d,
                              diag ? 1 : 0, prebuilt ? c->ghist : (u32*)nullptr);
    if (rc != TK_OK) return rc;
    c->launches += 1;
    if (bidir && with_ef) {
        // Algorithm 2 with the server memory: delta now holds g = sum + delta everywhere; take
        // Top_K_down out of it (delta <- g - Top_K(g)) and apply it (w <- w - Top_K(g))
        LinkArgs zero = {nullptr, nullptr, 0, 0, c->delta, (size_t)c->d, 0};
        ApplyArgs ap = {w_dev, 1.0f};
        rc = run_select(s, c->delta, 1, c->d, c->K_down, c->down, c->ctrl, c->force_general != 0, nullptr, nullptr,
                        &c->launches, nullptr, zero, EfArgs{nullptr, 0.0f}, ap, diag);
        if (rc != TK_OK) return rc;
    } else if (bidir) {
        ApplyArgs ap = {w_dev, alpha};
        rc = launch_select_grid(s, ctas, c->U, c->ucap, c->uni, (u32)c->K_down, c->sel, ap, c->ctrl, c->ghist, diag, prebuilt);
        if (rc != TK_OK) return rc;
        c->launches += 1;
    }
    c->last_mode = mode;
    c->last_kdown = c->K_down;
    return TK_OK;
}

bool step_args_ok(tk_ctx* c, float alpha, int mode) {
    if (!c || !isfinite(alpha)) return false;
    if (mode < 0 || mode > (TK_MODE_BIDIR | TK_MODE_EF)) return false;
    if ((mode & TK_MODE_EF) && (!c->eps || c->K_down > c->ef_kdown)) return false;
    return true;
}

}  // namespace

namespace {
int enqueue_step(tk_ctx* c, float* w_dev, const float* grads_dev, float alpha, int mode, bool timed);
}  // namespace

int tk_step(tk_ctx* c, float* w_dev, const float* grads_dev, float alpha, int mode) {
    if (!step_args_ok(c, alpha, mode) || !aligned4(w_dev) || !aligned4(grads_dev)) return TK_ERR_INVALID;
    // Replay a captured graph of this very step (same buffers, same settings) when asked to.
    // Not for a step whose streaming pass is being timestamped, not on the legacy default stream (it
    // cannot be captured), not when the caller is itself capturing this stream.
    const bool timed = c->profile > 0 && (c->steps_seen++ % c->profile) == 0;
    if (c->use_graphs && !timed && c->stream != nullptr) {
        cudaStreamCaptureStatus st = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing(c->stream, &st) == cudaSuccess && st == cudaStreamCaptureStatusNone) {
            tk_ctx::StepKey key = {w_dev, grads_dev, alpha, mode, c->K_down, c->force_general, c->diagnostics,
                                   (mode & TK_MODE_EF) ? c->eps : nullptr};
            tk_ctx::StepGraph* hit = nullptr;
            for (int i = 0; i < c->n_graphs; ++i)
                if (c->graphs[i].key == key) hit = &c->graphs[i];
            if (!hit) {
                int64_t before = c->launches;
                if (cudaStreamBeginCapture(c->stream, cudaStreamCaptureModeRelaxed) != cudaSuccess) {
                    cudaGetLastError();
                    return TK_ERR_CUDA;
                }
                int rc = enqueue_step(c, w_dev, grads_dev, alpha, mode, false);
                cudaGraph_t graph = nullptr;
                cudaError_t ce = cudaStreamEndCapture(c->stream, &graph);
                int64_t per_step = c->launches - before;
                c->launches = before;
                if (rc != TK_OK || ce != cudaSuccess || !graph) {
                    if (graph) cudaGraphDestroy(graph);
                    cudaGetLastError();
                    return rc != TK_OK ? rc : TK_ERR_CUDA;
                }
                cudaGraphExec_t exec = nullptr;
                ce = cudaGraphInstantiate(&exec, graph, 0);
                cudaGraphDestroy(graph);
                if (ce != cudaSuccess) {
                    cudaGetLastError();
                    return TK_ERR_CUDA;
                }
                int slot = c->n_graphs;
                if (slot == tk_ctx::kMaxGraphs) {  // evict the least recently used
                    slot = 0;
                    for (int i = 1; i < c->n_graphs; ++i)
                        if (c->graphs[i].used < c->graphs[slot].used) slot = i;
                    cudaGraphExecDestroy(c->graphs[slot].exec);
                } else {
                    c->n_graphs += 1;
                }
                c->graphs[slot] = tk_ctx::StepGraph{key, exec, per_step, 0};
                hit = &c->graphs[slot];
            }
            hit->used = ++c->graph_clock;
            if (cudaGraphLaunch(hit->exec, c->stream) != cudaSuccess) {
                cudaGetLastError();
                return TK_ERR_CUDA;
            }
            c->launches += hit->launches;
            c->last_mode = mode;
            c->last_kdown = c->K_down;
            return TK_OK;
        }
    }
    return enqueue_step(c, w_dev, grads_dev, alpha, mode, timed);
}

namespace {
int enqueue_step(tk_ctx* c, float* w_dev, const float* grads_dev, float alpha, int mode, bool timed) {
    const bool with_ef = (mode & TK_MODE_EF) != 0;
    cudaStream_t s = c->stream;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    if (timed && c->ev_ready && c->ev_used < kMaxEvents) {
        e0 = c->ev[2 * c->ev_used];
        e1 = c->ev[2 * c->ev_used + 1];
        c->ev_used += 1;
    }
    // the first kernel of the selection also resets the state of the union / downlink selection
    // ... and its last kernel threads every uplink entry onto its coordinate's chain (and, with
    // error memories, zeroes the sent entries in eps)
    const bool diag = c->diagnostics != 0;
    const bool gap = c->diagnostics >= 2 && c->diag_mem && c->diag_kdown >= c->K_down;
    const bool bidir = (mode & TK_MODE_BIDIR) != 0;
    int rc = TK_OK;
    if (gap) {
        // before the memories change: the dense sums, and Top_K of (delta +) sum_q p_q a^q
        if (cudaMemsetAsync(c->diag_sums, 0, 2 * sizeof(double), s) != cudaSuccess) return TK_ERR_CUDA;
        DeviceInfo* di = nullptr;
        rc = device_info(&di);
        if (rc != TK_OK) return rc;
        dense_sums_kernel<<<di->sms * 8, 256, 0, s>>>(grads_dev, with_ef ? c->eps : nullptr,
                                                      (with_ef && bidir) ? c->delta : nullptr, c->p, c->N, (size_t)c->d,
                                                      alpha, with_ef ? alpha : 1.0f, c->diag_Da, c->diag_sums);
        TK_LAUNCH_CHECK();
        c->launches += 1;
        rc = run_select(s, c->diag_Da, 1, c->d, c->K_down, c->diag_sel, c->ctrl, c->force_general != 0, nullptr,
                        nullptr, &c->launches);
        if (rc != TK_OK) return rc;
    }
    LinkArgs link = {c->head, c->next, (u32)c->d, 0, with_ef ? c->eps : nullptr, (size_t)c->d, 0, c->slots, c->slot_row_words,
                     c->p, c->uni};
    EfArgs ef = {with_ef ? c->eps : nullptr, alpha};
    SelectBufs up = c->up;
    if (c->cand_cap > 0) up.cap = capped(up.cap, c->cand_cap, c->K_up);  // shorter lists, packed closer in the same buffer
    rc = run_select(s, grads_dev, c->N, c->d, c->K_up, up, c->ctrl, c->force_general != 0, e0, e1,
                    &c->launches, c->uni, link, ef, ApplyArgs{nullptr, 0.0f}, diag, c->bound_reuse != 0 && !with_ef);
    if (rc != TK_OK) return rc;
    rc = run_server(c, w_dev, alpha, mode);
    if (rc != TK_OK || !gap) return rc;
    // after the step: the other side of the difference is what the server actually sent
    const uint2* other = c->U;                      // unidirectional: S over the union
    const u32* other_count = &c->uni->cand_count;
    u32 other_cap = c->ucap;
    if (bidir && with_ef) { other = c->diag_other_ef(); other_count = nullptr; other_cap = (u32)c->K_down; }
    else if (bidir) { other = c->sel; other_count = &c->uni->out_count; other_cap = c->ucap; }
    u32 Kd = (u32)c->K_down, dd = (u32)c->d;
    diff_scatter_kernel<<<(Kd + 255) / 256, 256, 0, s>>>(c->diag_sel.out, nullptr, Kd, 1.0f, c->diag_Z, dd);
    diff_scatter_kernel<<<(other_cap + 255) / 256, 256, 0, s>>>(other, other_count, other_cap, -1.0f, c->diag_Z, dd);
    diff_norm_kernel<<<(Kd + 255) / 256, 256, 0, s>>>(c->diag_sel.out, nullptr, Kd, c->diag_Z, dd, c->diag_sums);
    diff_norm_kernel<<<(other_cap + 255) / 256, 256, 0, s>>>(other, other_count, other_cap, c->diag_Z, dd, c->diag_sums);
    TK_LAUNCH_CHECK();
    c->launches += 4;
    return TK_OK;
}
}  // namespace

int tk_step_uplink(tk_ctx* c, const float* grads_local_dev, int32_t row0, int32_t rows, float alpha, int mode) {
    if (!step_args_ok(c, alpha, mode) || !aligned4(grads_local_dev)) return TK_ERR_INVALID;
    if (row0 < 0 || rows < 1 || (int64_t)row0 + rows > c->N) return TK_ERR_INVALID;
    const bool with_ef = (mode & TK_MODE_EF) != 0;
    // this rank's slice of every per-row buffer
    SelectBufs b = c->up;
    if (c->cand_cap > 0) b.cap = capped(b.cap, c->cand_cap, c->K_up);
    b.rs += row0;
    b.hist += (size_t)row0 * kHistBins;
    b.smax += (size_t)row0 * kSampleSlots;
    b.cand += (size_t)row0 * b.cap;
    b.out += (size_t)row0 * (size_t)c->K_up;
    float* eps = with_ef ? c->eps + (size_t)row0 * (size_t)c->d : nullptr;
    // (the entries are filed after the exchange; the union's state gates the rows' warm starts as in tk_step)
    LinkArgs link = {nullptr, nullptr, 0, 0, eps, (size_t)c->d, 0, nullptr, 0, c->p, c->uni};
    EfArgs ef = {eps, alpha};
    // (the union's state is reset here too: the filing kernel of tk_step_server lowers its bin_base)
    return run_select(c->stream, grads_local_dev, rows, c->d, c->K_up, b, c->ctrl, c->force_general != 0, nullptr,
                      nullptr, &c->launches, c->uni, link, ef, ApplyArgs{nullptr, 0.0f}, c->diagnostics != 0,
                      c->bound_reuse != 0 && !with_ef);
}

int tk_messages(tk_ctx* c, void** msgs_dev, size_t* bytes_per_row) {
    if (!c || !msgs_dev) return TK_ERR_INVALID;
    *msgs_dev = c->up.out;
    if (bytes_per_row) *bytes_per_row = (size_t)c->K_up * sizeof(uint2);
    return TK_OK;
}

int tk_step_server(tk_ctx* c, float* w_dev, float alpha, int mode) {
    if (!step_args_ok(c, alpha, mode) || !aligned4(w_dev)) return TK_ERR_INVALID;
    u32 total = (u32)(c->N * c->K_up);
    agg_link_kernel<<<(total + 255) / 256, 256, 0, c->stream>>>(c->up.out, total, (u32)c->K_up, c->p, c->head, c->next, c->slots,
                                                                 c->slot_row_words, c->uni, c->ctrl, (u32)c->d);
    TK_LAUNCH_CHECK();
    c->launches += 1;
    return run_server(c, w_dev, alpha, mode);
}

int tk_step_host(tk_ctx* c, float* w_host, const float* grads_host, float alpha, int mode) {
    if (!c || !w_host || !grads_host) return TK_ERR_INVALID;
    size_t gbytes = (size_t)c->N * (size_t)c->d * sizeof(float), wbytes = (size_t)c->d * sizeof(float);
    if (!c->stage_g) {
        if (cudaMalloc((void**)&c->stage_g, gbytes) != cudaSuccess ||
            cudaMalloc((void**)&c->stage_w, wbytes) != cudaSuccess) {
            cudaGetLastError();
            if (c->stage_g) cudaFree(c->stage_g);
            c->stage_g = nullptr;
            c->stage_w = nullptr;
            return TK_ERR_ALLOC;
        }
    }
    if (cudaMemcpyAsync(c->stage_g, grads_host, gbytes, cudaMemcpyHostToDevice, c->stream) != cudaSuccess ||
        cudaMemcpyAsync(c->stage_w, w_host, wbytes, cudaMemcpyHostToDevice, c->stream) != cudaSuccess)
        return TK_ERR_CUDA;
    int rc = tk_step(c, c->stage_w, c->stage_g, alpha, mode);
    if (rc != TK_OK) return rc;
    if (cudaMemcpyAsync(w_host, c->stage_w, wbytes, cudaMemcpyDeviceToHost, c->stream) != cudaSuccess ||
        cudaStreamSynchronize(c->stream) != cudaSuccess)
        return TK_ERR_CUDA;
    return TK_OK;
}

int tk_topk(tk_ctx* c, const float* x_dev, int32_t rows, int64_t d, int64_t K, int32_t* idx_out_dev,
            float* val_out_dev) {
    if (!aligned4(x_dev) || !aligned4(idx_out_dev) || !aligned4(val_out_dev)) return TK_ERR_INVALID;
    if (rows < 1 || d < 1 || d >= ((int64_t)1 << 31) || K < 1 || K > d) return TK_ERR_INVALID;
    cudaStream_t s = c ? c->stream : nullptr;
    SelectLayout SL = select_layout(rows, d, K);
    SortLayout QL = sort_layout(rows, K);
    size_t off_ctrl = SL.bytes + QL.bytes;
    char* base = nullptr;
    int rc = pool_get(off_ctrl + align_up(sizeof(Ctrl)), &base, s);
    if (rc != TK_OK) return rc;
    SelectBufs b = bind(SL, base);
    Ctrl* ctrl = c ? c->ctrl : (Ctrl*)(base + off_ctrl);
    if (cudaMemsetAsync(b.rs, 0, (size_t)rows * sizeof(RowState), s) != cudaSuccess ||
        cudaMemsetAsync(b.hist, 0, (size_t)rows * kHistBins * sizeof(u32), s) != cudaSuccess ||
        (!c && cudaMemsetAsync(ctrl, 0, sizeof(Ctrl), s) != cudaSuccess))
        return TK_ERR_CUDA;
    int64_t local = 0;
    int64_t* launches = c ? &c->launches : &local;
    if (c && c->cand_cap > 0) b.cap = capped(b.cap, c->cand_cap, K);
    rc = run_select(s, x_dev, rows, d, K, b, ctrl, c ? c->force_general != 0 : false, nullptr, nullptr, launches);
    if (rc == TK_OK)
        rc = run_sort(s, b.out, (size_t)K, nullptr, 0, (u32)K, rows, d, (uint2*)(base + SL.bytes + QL.off_tmp),
                      (u32*)(base + SL.bytes + QL.off_cnt), QL.tiles, idx_out_dev, val_out_dev, (size_t)K, launches);
    pool_done(s);  // the next user of the pool, on whatever stream, waits for these kernels
    return rc;
}

size_t tk_ef_bytes(int64_t d, int32_t N, int64_t K_down) {
    if (!sizes_ok(d, N, 1, K_down)) return 0;
    size_t rows = align_up((size_t)N * (size_t)d * sizeof(float));
    return rows + align_up((size_t)d * sizeof(float)) + select_layout(1, d, K_down).bytes;
}

int tk_ef_attach(tk_ctx* c, void* mem_dev, size_t bytes) {
    if (!c || !mem_dev || ((uintptr_t)mem_dev & (kAlign - 1)) != 0) return TK_ERR_INVALID;
    size_t need = tk_ef_bytes(c->d, c->N, c->K_down);
    if (need == 0 || bytes < need) return TK_ERR_ALLOC;
    char* base = (char*)mem_dev;
    size_t off_delta = align_up((size_t)c->N * (size_t)c->d * sizeof(float));
    size_t off_down = off_delta + align_up((size_t)c->d * sizeof(float));
    SelectLayout L = select_layout(1, c->d, c->K_down);
    SelectBufs down = bind(L, base + off_down);
    // epsilon_0 = delta_0 = 0 (initialisation line of Algorithm 1/2); selection state zero at rest
    if (cudaMemsetAsync(base, 0, off_down, c->stream) != cudaSuccess ||
        cudaMemsetAsync(down.rs, 0, sizeof(RowState), c->stream) != cudaSuccess ||
        cudaMemsetAsync(down.hist, 0, (size_t)kHistBins * sizeof(u32), c->stream) != cudaSuccess ||
        cudaStreamSynchronize(c->stream) != cudaSuccess) {
        cudaGetLastError();
        return TK_ERR_CUDA;
    }
    drop_graphs(c);  // captured steps hold the old memories' addresses
    c->eps = (float*)base;
    c->delta = (float*)(base + off_delta);
    c->down = down;
    c->ef_kdown = c->K_down;
    return TK_OK;
}

int tk_ef_state(tk_ctx* c, float** eps_dev, float** delta_dev) {
    if (!c || !c->eps) return TK_ERR_INVALID;
    if (eps_dev) *eps_dev = c->eps;
    if (delta_dev) *delta_dev = c->delta;
    return TK_OK;
}

int tk_set_kdown(tk_ctx* c, int64_t K_down) {
    if (!c || K_down < 1 || K_down > c->d) return TK_ERR_INVALID;
    c->K_down = K_down;
    if (c->diagnostics >= 2) return diag_alloc(c);   // the dense selection of the diagnostics grows with K_down
    return TK_OK;
}

int tk_last_uplink(tk_ctx* c, int32_t* idx_out_dev, float* val_out_dev) {
    if (!c || !aligned4(idx_out_dev) || !aligned4(val_out_dev) || c->last_mode < 0) return TK_ERR_INVALID;
    SortLayout QL = sort_layout(c->N, c->K_up);
    char* base = nullptr;
    int rc = pool_get(QL.bytes, &base, c->stream);
    if (rc != TK_OK) return rc;
    rc = run_sort(c->stream, c->up.out, (size_t)c->K_up, nullptr, 0, (u32)c->K_up, c->N, c->d,
                  (uint2*)(base + QL.off_tmp), (u32*)(base + QL.off_cnt), QL.tiles, idx_out_dev, val_out_dev,
                  (size_t)c->K_up, &c->launches);
    if (rc != TK_OK) return rc;
    return cudaStreamSynchronize(c->stream) == cudaSuccess ? TK_OK : TK_ERR_CUDA;
}

int tk_last_aggregate(tk_ctx* c, int32_t* idx_out_dev, float* val_out_dev, int64_t* count_host) {
    if (!c || !aligned4(idx_out_dev) || !aligned4(val_out_dev) || !count_host || c->last_mode < 0)
        return TK_ERR_INVALID;
    RowState u;
    if (cudaMemcpyAsync(&u, c->uni, sizeof u, cudaMemcpyDeviceToHost, c->stream) != cudaSuccess ||
        cudaStreamSynchronize(c->stream) != cudaSuccess)
        return TK_ERR_CUDA;
    u32 n = u.cand_count < c->ucap ? u.cand_count : c->ucap;
    *count_host = n;
    if (n == 0) return TK_OK;
    SortLayout QL = sort_layout(1, n);
    char* base = nullptr;
    int rc = pool_get(QL.bytes, &base, c->stream);
    if (rc != TK_OK) return rc;
    rc = run_sort(c->stream, c->U, c->ucap, nullptr, 0, n, 1, c->d, (uint2*)(base + QL.off_tmp),
                  (u32*)(base + QL.off_cnt), QL.tiles, idx_out_dev, val_out_dev, n, &c->launches);
    if (rc != TK_OK) return rc;
    return cudaStreamSynchronize(c->stream) == cudaSuccess ? TK_OK : TK_ERR_CUDA;
}

int tk_last_downlink(tk_ctx* c, int32_t* idx_out_dev, float* val_out_dev, int64_t* count_host) {
    if (!c || c->last_mode < 0) return TK_ERR_INVALID;
    if (!(c->last_mode & TK_MODE_BIDIR)) return tk_last_aggregate(c, idx_out_dev, val_out_dev, count_host);
    if (!aligned4(idx_out_dev) || !aligned4(val_out_dev) || !count_host) return TK_ERR_INVALID;
    if (c->last_mode & TK_MODE_EF) {
        // selected from the dense server vector: already the exact K_down-entry message
        u32 Kd = (u32)c->last_kdown;
        SortLayout QL = sort_layout(1, Kd);
        char* base = nullptr;
        int rc = pool_get(QL.bytes, &base, c->stream);
        if (rc != TK_OK) return rc;
        *count_host = Kd;
        rc = run_sort(c->stream, c->down.out, Kd, nullptr, 0, Kd, 1, c->d, (uint2*)(base + QL.off_tmp),
                      (u32*)(base + QL.off_cnt), QL.tiles, idx_out_dev, val_out_dev, Kd, &c->launches);
        if (rc != TK_OK) return rc;
        return cudaStreamSynchronize(c->stream) == cudaSuccess ? TK_OK : TK_ERR_CUDA;
    }
    // The step selects among the union only.  The message proper has exactly K_down entries:
    // every selected entry of non-zero magnitude, then zero-valued entries at the lowest
    // indices that carry no such entry.
    RowState u;
    if (cudaMemcpyAsync(&u, c->uni, sizeof u, cudaMemcpyDeviceToHost, c->stream) != cudaSuccess ||
        cudaStreamSynchronize(c->stream) != cudaSuccess)
        return TK_ERR_CUDA;
    u32 nsel = u.out_count < c->ucap ? u.out_count : c->ucap;
    u32 Kd = (u32)c->last_kdown;
    SortLayout QL = sort_layout(1, Kd);
    size_t off_msg = QL.bytes;
    size_t off_flags = off_msg + align_up((size_t)Kd * sizeof(uint2));
    size_t off_cnt = off_flags + align_up((size_t)Kd);
    char* base = nullptr;
    int rc = pool_get(off_cnt + kAlign, &base, c->stream);
    if (rc != TK_OK) return rc;
    uint2* msg = (uint2*)(base + off_msg);
    unsigned char* flags = (unsigned char*)(base + off_flags);
    u32* msg_count = (u32*)(base + off_cnt);
    cudaStream_t s = c->stream;
    if (cudaMemsetAsync(flags, 0, Kd, s) != cudaSuccess || cudaMemsetAsync(msg_count, 0, sizeof(u32), s) != cudaSuccess)
        return TK_ERR_CUDA;
    u32 nz = 0;
    if (nsel) {
        msg_collect_kernel<<<(nsel + 255) / 256, 256, 0, s>>>(c->sel, nsel, msg, msg_count, flags, Kd);
        TK_LAUNCH_CHECK();
        c->launches += 1;
    }
    if (cudaMemcpyAsync(&nz, msg_count, sizeof nz, cudaMemcpyDeviceToHost, s) != cudaSuccess ||
        cudaStreamSynchronize(s) != cudaSuccess)
        return TK_ERR_CUDA;
    if (nz > Kd) return TK_ERR_INTERNAL;
    if (nz < Kd) {
        msg_pad_kernel<<<1, 1024, 0, s>>>(flags, Kd, Kd - nz, msg, nz);
        TK_LAUNCH_CHECK();
        c->launches += 1;
    }
    *count_host = Kd;
    rc = run_sort(s, msg, Kd, nullptr, 0, Kd, 1, c->d, (uint2*)(base + QL.off_tmp), (u32*)(base + QL.off_cnt),
                  QL.tiles, idx_out_dev, val_out_dev, Kd, &c->launches);
    if (rc != TK_OK) return rc;
    return cudaStreamSynchronize(s) == cudaSuccess ? TK_OK : TK_ERR_CUDA;
}

int tk_status(tk_ctx* c, tk_stats* out) {
    if (!c || !out) return TK_ERR_INVALID;
    memset(out, 0, sizeof *out);
    if (cudaStreamSynchronize(c->stream) != cudaSuccess) {
        cudaGetLastError();
        return TK_ERR_CUDA;
    }
    Ctrl ctrl;
    RowState u;
    RowState* rows = new (std::nothrow) RowState[c->N];
    if (!rows) return TK_ERR_ALLOC;
    bool ok = cudaMemcpy(&ctrl, c->ctrl, sizeof ctrl, cudaMemcpyDeviceToHost) == cudaSuccess &&
              cudaMemcpy(&u, c->uni, sizeof u, cudaMemcpyDeviceToHost) == cudaSuccess &&
              cudaMemcpy(rows, c->up.rs, (size_t)c->N * sizeof(RowState), cudaMemcpyDeviceToHost) == cudaSuccess;
    if (!ok) {
        delete[] rows;
        cudaGetLastError();
        return TK_ERR_CUDA;
    }
    out->device_status = ctrl.status;
    out->rows_general = (int32_t)ctrl.rows_general;
    out->union_size = u.cand_count;
    out->downlink_count = (c->last_mode >= 0 && (c->last_mode & TK_MODE_BIDIR)) ? u.out_count : u.cand_count;
    if (c->last_mode == (TK_MODE_BIDIR | TK_MODE_EF)) out->downlink_count = c->last_kdown;
    int64_t lo = INT64_MAX, hi = 0;
    for (int q = 0; q < c->N; ++q) {
        int64_t v = rows[q].cand_count;
        if (v < lo) lo = v;
        if (v > hi) hi = v;
    }
    out->cand_min = lo;
    out->cand_max = hi;
    delete[] rows;
    float sum = 0.0f;
    for (int i = 0; i < c->ev_used; ++i) {
        float ms = 0.0f;
        if (cudaEventElapsedTime(&ms, c->ev[2 * i], c->ev[2 * i + 1]) == cudaSuccess) sum += ms;
        else cudaGetLastError();
    }
    out->select_ms_sum = sum;
    out->select_samples = c->ev_used;
    c->ev_used = 0;
    return ctrl.status == 0 ? TK_OK : ctrl.status;
}

int tk_set_profile(tk_ctx* c, int on) {
    if (!c) return TK_ERR_INVALID;
    if (on && !c->ev_ready) {
        for (int i = 0; i < 2 * kMaxEvents; ++i)
            if (cudaEventCreate(&c->ev[i]) != cudaSuccess) return TK_ERR_CUDA;
        c->ev_ready = true;
    }
    c->profile = on > 0 ? on : 0;
    c->steps_seen = 0;
    c->ev_used = 0;
    return TK_OK;
}

int tk_set_diagnostics(tk_ctx* c, int level) {
    if (!c || level < 0 || level > 2) return TK_ERR_INVALID;
    if (level == 2) {
        int rc = diag_alloc(c);
        if (rc != TK_OK) return rc;
    }
    c->diagnostics = level;
    return TK_OK;
}

int tk_diagnostics(tk_ctx* c, tk_diag* out, double* one_minus_gamma_up_host) {
    if (!c || !out || c->last_mode < 0 || !c->diagnostics) return TK_ERR_INVALID;
    memset(out, 0, sizeof *out);
    if (cudaStreamSynchronize(c->stream) != cudaSuccess) {
        cudaGetLastError();
        return TK_ERR_CUDA;
    }
    RowState u, dn;
    memset(&dn, 0, sizeof dn);
    RowState* rows = new (std::nothrow) RowState[c->N];
    if (!rows) return TK_ERR_ALLOC;
    const bool ef_bidir = c->last_mode == (TK_MODE_BIDIR | TK_MODE_EF);
    bool ok = cudaMemcpy(&u, c->uni, sizeof u, cudaMemcpyDeviceToHost) == cudaSuccess &&
              cudaMemcpy(rows, c->up.rs, (size_t)c->N * sizeof(RowState), cudaMemcpyDeviceToHost) == cudaSuccess &&
              (!ef_bidir || cudaMemcpy(&dn, c->down.rs, sizeof dn, cudaMemcpyDeviceToHost) == cudaSuccess);
    if (!ok) {
        delete[] rows;
        cudaGetLastError();
        return TK_ERR_CUDA;
    }
    auto lost = [](double total, double kept) {   // ||Top_K(x) - x||^2 / ||x||^2
        if (!(total > 0.0)) return 0.0;
        double v = 1.0 - kept / total;
        return v < 0.0 ? 0.0 : v;
    };
    double worst = 0.0;
    for (int q = 0; q < c->N; ++q) {
        double v = lost(rows[q].sum_sq, rows[q].sel_sq);
        if (one_minus_gamma_up_host) one_minus_gamma_up_host[q] = v;
        if (v > worst) worst = v;
    }
    delete[] rows;
    out->one_minus_gamma_up_max = worst;
    out->union_fraction = (double)u.cand_count / (double)c->d;
    out->nonzero_fraction = (double)u.nnz / (double)c->d;
    out->compression_factor = (double)c->last_kdown / ((double)c->K_up * (double)c->N);
    if (ef_bidir) out->one_minus_gamma_down = lost(dn.sum_sq, dn.sel_sq);
    else if (c->last_mode & TK_MODE_BIDIR) out->one_minus_gamma_down = lost(u.sum_sq, u.sel_sq);
    out->rho = -1.0;
    if (c->diagnostics >= 2 && c->diag_mem) {
        double sums[2] = {0.0, 0.0};
        if (cudaMemcpy(sums, c->diag_sums, sizeof sums, cudaMemcpyDeviceToHost) != cudaSuccess) {
            cudaGetLastError();
            return TK_ERR_CUDA;
        }
        out->rho = sums[0] > 0.0 ? sqrt(sums[1]) / sqrt(sums[0]) : 0.0;
    }
    return TK_OK;
}

int tk_set_graph(tk_ctx* c, int on) {
    if (!c) return TK_ERR_INVALID;
    c->use_graphs = on ? 1 : 0;
    if (!on) drop_graphs(c);
    return TK_OK;
}

int tk_set_force_general(tk_ctx* c, int on) {
    if (!c) return TK_ERR_INVALID;
    c->force_general = on ? 1 : 0;
    return TK_OK;
}

int tk_set_bound_reuse(tk_ctx* c, int on) {
    if (!c) return TK_ERR_INVALID;
    if ((on != 0) != (c->bound_reuse != 0)) drop_graphs(c);  // captured steps carry the old setting
    c->bound_reuse = on ? 1 : 0;
    return TK_OK;
}

int tk_set_cand_cap(tk_ctx* c, int64_t cap) {
    if (!c || cap < 0) return TK_ERR_INVALID;
    if (cap != c->cand_cap) drop_graphs(c);  // captured steps carry the old capacity
    c->cand_cap = cap;
    return TK_OK;
}

int tk_comm_model(int32_t N, int64_t K_up, int64_t K_down, int64_t union_size, double alpha1, double beta1,
                  double alpha2, double beta2, tk_comm* out) {
    if (!out || N < 1 || K_up < 1 || K_down < 1 || (int64_t)N * K_up >= ((int64_t)1 << 31)) return TK_ERR_INVALID;
    if (union_size < -1 || union_size > (int64_t)N * K_up) return TK_ERR_INVALID;
    if (!isfinite(alpha1) || !isfinite(beta1) || !isfinite(alpha2) || !isfinite(beta2) || alpha1 < 0 || beta1 < 0 ||
        alpha2 < 0 || beta2 < 0)
        return TK_ERR_INVALID;
    memset(out, 0, sizeof *out);
    out->uplink_words = 2 * K_up;
    out->downlink_words_uni_max = 2 * (int64_t)N * K_up;
    out->downlink_words_uni = union_size < 0 ? -1 : 2 * union_size;
    out->downlink_words_bi = 2 * K_down;
    const double up = alpha1 + (double)out->uplink_words * beta1;
    out->time_uni = up + alpha2 + (double)out->downlink_words_uni_max * beta2;
    out->time_uni_union = union_size < 0 ? -1.0 : up + alpha2 + (double)out->downlink_words_uni * beta2;
    out->time_bi = up + alpha2 + (double)out->downlink_words_bi * beta2;
    out->compression_factor = (double)K_down / ((double)K_up * (double)N);
    return TK_OK;
}

int64_t tk_launch_count(tk_ctx* c) { return c ? c->launches : 0; }

int tk_debug_phase_clock(tk_ctx* c, double* first_us, double* last_us, int32_t n) {
#if TK_PHASE_CLOCK
    if (!c || !first_us || !last_us || n < 1) return TK_ERR_INVALID;
    if (cudaStreamSynchronize(c->stream) != cudaSuccess) { cudaGetLastError(); return TK_ERR_CUDA; }
    Ctrl ctrl;
    if (cudaMemcpy(&ctrl, c->ctrl, sizeof ctrl, cudaMemcpyDeviceToHost) != cudaSuccess) { cudaGetLastError(); return TK_ERR_CUDA; }
    u64 t0 = ~0ull;
    for (int i = 0; i < kStampCount; ++i)
        if (ctrl.t_last[i] != 0 && ctrl.t_first[i] < t0) t0 = ctrl.t_first[i];
    for (int i = 0; i < n; ++i) {
        bool seen = i < kStampCount && ctrl.t_last[i] != 0;
        first_us[i] = seen ? (double)(ctrl.t_first[i] - t0) * 1e-3 : -1.0;
        last_us[i] = seen ? (double)(ctrl.t_last[i] - t0) * 1e-3 : -1.0;
    }
    // re-arm: earliest stamps start at the largest value, latest ones at zero
    if (cudaMemset((char*)c->ctrl + offsetof(Ctrl, t_first), 0xff, sizeof ctrl.t_first) != cudaSuccess ||
        cudaMemset((char*)c->ctrl + offsetof(Ctrl, t_last), 0, sizeof ctrl.t_last) != cudaSuccess) {
        cudaGetLastError();
        return TK_ERR_CUDA;
    }
    return TK_OK;
#else
    (void)c; (void)first_us; (void)last_us; (void)n;
    return TK_ERR_INVALID;
#endif
}

void tk_destroy(tk_ctx* c) {
    if (!c) return;
    drop_graphs(c);
    if (c->ev_ready)
        for (int i = 0; i < 2 * kMaxEvents; ++i) cudaEventDestroy(c->ev[i]);
    if (c->stage_g) cudaFree(c->stage_g);
    if (c->stage_w) cudaFree(c->stage_w);
    if (c->diag_mem) cudaFree(c->diag_mem);
    delete c;
}

void tk_release_scratch(void) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return;
    if (g_pool[dev].base) {
        cudaDeviceSynchronize();
        cudaFree(g_pool[dev].base);
        g_pool[dev].base = nullptr;
        g_pool[dev].bytes = 0;
    }
}

// ---- tk_topk without allocation ----------------------------------------------------------------
// The scratch of tk_topk_noalloc.  In host code this name is only a handle for
// cudaGetSymbolAddress: the kernels get the device address looked up below.
static __device__ __align__(256) unsigned char g_noalloc_scratch[TK_NOALLOC_SCRATCH_BYTES];
static char* g_noalloc_addr[64];  // device address of the array, per device; NULL until looked up
// The last 256 bytes (more in a build with the phase clock) hold the control block with the sticky status word: zero when the library is
// loaded (static storage), written by the kernels' consistency checks, cleared only by
// tk_topk_noalloc_status.  Everything below it is per-call scratch.
constexpr size_t kNoallocCtrlOff = (size_t)TK_NOALLOC_SCRATCH_BYTES - (sizeof(Ctrl) + 255) / 256 * 256;

static int noalloc_base(char** out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return TK_ERR_CUDA;
    if (!g_noalloc_addr[dev]) {  // set-up, once per device, with that device current
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || !ptr) {
            cudaGetLastError();
            return TK_ERR_CUDA;
        }
        g_noalloc_addr[dev] = (char*)ptr;
    }
    *out = g_noalloc_addr[dev];
    return TK_OK;
}

int tk_topk_noalloc(const float* x_dev, int32_t rows, int64_t d, int64_t K, int32_t* idx_out_dev,
                    float* val_out_dev, void* cuda_stream) {
    if (!aligned4(x_dev) || !aligned4(idx_out_dev) || !aligned4(val_out_dev)) return TK_ERR_INVALID;
    if (rows < 1 || d < 1 || d >= ((int64_t)1 << 31) || K < 1 || K > d) return TK_ERR_INVALID;
    // size check first, in 64-bit arithmetic that cannot wrap for any accepted rows/d/K
    if ((double)rows * ((double)candidate_capacity(d, K) + 2.0 * (double)K) * 8.0 > (double)kNoallocCtrlOff)
        return TK_ERR_TOO_LARGE;
    SelectLayout SL = select_layout(rows, d, K, false);
    SortLayout QL = sort_layout(rows, K);
    if (SL.bytes + QL.bytes > kNoallocCtrlOff) return TK_ERR_TOO_LARGE;
    char* base = nullptr;
    int rc = noalloc_base(&base);
    if (rc != TK_OK) return rc;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    SelectBufs b = bind(SL, base);
    Ctrl* ctrl = (Ctrl*)(base + kNoallocCtrlOff);
    // the array still holds the previous call's data: clear what the kernels expect to be zero
    // (not the control block: its status word is sticky)
    if (cudaMemsetAsync(b.rs, 0, (size_t)rows * sizeof(RowState), s) != cudaSuccess ||
        cudaMemsetAsync(b.hist, 0, (size_t)rows * kHistBins * sizeof(u32), s) != cudaSuccess)
        return TK_ERR_CUDA;
    int64_t launches = 0;
    rc = run_select(s, x_dev, rows, d, K, b, ctrl, false, nullptr, nullptr, &launches);
    if (rc != TK_OK) return rc;
    return run_sort(s, b.out, (size_t)K, nullptr, 0, (u32)K, rows, d, (uint2*)(base + SL.bytes + QL.off_tmp),
                    (u32*)(base + SL.bytes + QL.off_cnt), QL.tiles, idx_out_dev, val_out_dev, (size_t)K, &launches);
}

int tk_topk_noalloc_status(void) {
    char* base = nullptr;
    int rc = noalloc_base(&base);
    if (rc != TK_OK) return rc;
    Ctrl ctrl;  // on the stack: nothing is allocated here either
    if (cudaDeviceSynchronize() != cudaSuccess ||
        cudaMemcpy(&ctrl, base + kNoallocCtrlOff, sizeof ctrl, cudaMemcpyDeviceToHost) != cudaSuccess) {
        cudaGetLastError();
        return TK_ERR_CUDA;
    }
    if (ctrl.status != 0 && cudaMemset(base + kNoallocCtrlOff, 0, sizeof(int)) != cudaSuccess) {
        cudaGetLastError();
        return TK_ERR_CUDA;
    }
    return ctrl.status;
}

const char* tk_strerror(int code) {
    switch (code) {
        case TK_OK: return "ok";
        case TK_ERR_INVALID: return "invalid argument";
        case TK_ERR_ALLOC: return "workspace too small or allocation failed";
        case TK_ERR_CUDA: return "CUDA runtime error";
        case TK_ERR_INTERNAL: return "device-side consistency check failed";
        case TK_ERR_TOO_LARGE: return "problem exceeds the built-in scratch of tk_topk_noalloc";
        default: return "unknown error";
    }
}

}  // extern "C"
