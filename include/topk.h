/*
 * libtopk — the per-step compression pipeline of bidirectional top_K SGD
 * (arXiv 2209.15203) on one NVIDIA B200 (sm_100a).
 *
 * The N workers of the parameter-server iteration are the N rows of one fp32
 * tensor on one GPU.  One step (tk_step) does, entirely on the device:
 *   1. uplink    Top_K_up of every row                (Algorithm 1/2, worker: SEND(Top_K(a^q)))
 *   2. server    g = sum_{q=1..N} p_q Top_K(a^q), summed in worker order
 *                                                     (Algorithm 1/2, server step)
 *   3. downlink  Top_K_down(g) when bidirectional     (Algorithm 2, server: SEND(Top_K(g)));
 *                g itself when unidirectional         (Algorithm 1, server: SEND(g))
 *   4. update    w <- w - alpha * message             (Algorithm 1/2, last worker step)
 * This is the iteration with the error memories epsilon, delta at zero (their
 * value at t = 1); the step size multiplies the message rather than the
 * gradient, which selects the same components because Top_K is positively
 * homogeneous.
 *
 * Top_K(x) keeps the K components of largest magnitude (Section 1).  Magnitudes
 * are compared through the integer key  bits(x) & 0x7fffffff  (so -0 == +0,
 * denormals are kept, NaN/Inf are ordered by bit pattern); among equal
 * magnitudes the LOWER index is kept.  A message always has exactly K entries
 * (zero-valued ones included when the vector has fewer than K non-zeros) and is
 * listed in ascending index order; values are the original signed values, bit
 * for bit.  All fp32 arithmetic is round-to-nearest with one rounding per
 * multiply and one per add/subtract (no fused multiply-add, no flush to zero).
 *
 * Conventions
 *   - "dev" pointers are device memory of the current CUDA device, "host"
 *     pointers are host memory.  The library never takes ownership of a
 *     caller's buffer.  fp32 / int32 buffers must be 4-byte aligned; rows of a
 *     [rows][d] tensor are contiguous (row r starts at element r*d).
 *   - Every function returns TK_OK (0) or a negative TK_ERR_* code; nothing
 *     throws or aborts.  tk_strerror() names a code.
 *   - Work is enqueued on the context's stream and the call returns without
 *     waiting, except where a function is documented to synchronise.
 *   - A context may be used by one host thread at a time.
 */
#ifndef TOPK_H_
#define TOPK_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct tk_ctx tk_ctx;

enum {
    TK_OK = 0,
    TK_ERR_INVALID = -1,  /* bad argument (range, NULL, alignment, size) */
    TK_ERR_ALLOC = -2,    /* workspace too small / allocation failed */
    TK_ERR_CUDA = -3,     /* a CUDA runtime call failed */
    /* -4 is not used: no kernel of the library waits on a flag (all device-side waiting is a
       cooperative-groups grid or cluster barrier), so there is no wait that could expire */
    TK_ERR_INTERNAL = -5, /* a device-side consistency check failed */
    TK_ERR_TOO_LARGE = -6 /* the problem does not fit the built-in scratch of tk_topk_noalloc */
};

enum {
    TK_MODE_UNI = 0,   /* Algorithm 1: the downlink carries the aggregate itself */
    TK_MODE_BIDIR = 1, /* Algorithm 2: the downlink carries Top_K_down of the aggregate */
    TK_MODE_EF = 2     /* flag, OR-ed in: keep the error memories epsilon^q and delta of
                          Algorithm 1/2 as printed (see tk_ef_attach) */
};

/* Counters of the last step / selection, filled by tk_status(). */
typedef struct tk_stats {
    int32_t device_status;    /* sticky TK_ERR_* raised by a kernel, 0 if none */
    int32_t rows_general;     /* rows the exact multi-pass path handled in the last selection: rows whose
                                 predicted threshold failed verification, or all rows when none was
                                 predicted (short rows, K > d/64, tk_set_force_general) */
    int64_t union_size;       /* |U|: distinct indices in the last aggregate (<= N*K_up);
                                 |U|/d is the non-zero fraction of Section 4.2 */
    int64_t downlink_count;   /* entries applied to w in the last step */
    int64_t cand_min;         /* fewest / most candidates any row kept in the last uplink */
    int64_t cand_max;
    float   select_ms_sum;    /* device time of the streaming selection passes recorded since the
                                 previous tk_status call, and how many were recorded (both 0 */
    int32_t select_samples;   /* unless tk_set_profile is on; at most 256 are kept) */
} tk_stats;

/* Bytes of device workspace tk_init needs for these sizes (0 if they are invalid). */
size_t tk_workspace_bytes(int64_t d, int32_t N, int64_t K_up, int64_t K_down);

/*
 * Create a context for N workers with vectors of length d (the problem of
 * Eq. 1: minimise sum_q p_q F^q(w), w in R^d).
 *   out             receives the context
 *   d               1 <= d < 2^31
 *   N               1 <= N <= 65535, with N * K_up < 2^31
 *   K_up, K_down    1 <= K <= d   (Section 4.2's K_uplink, K_downlink)
 *   p_host          [N] weights p_q, finite and >= 0 (copied; the sum is not checked)
 *   workspace_dev   device buffer of at least tk_workspace_bytes() bytes, 256-byte
 *                   aligned, owned by the caller and kept alive until tk_destroy;
 *                   the library keeps all per-step state in it and zeroes what
 *                   it needs here (this call synchronises the stream)
 *   cuda_stream     a cudaStream_t (NULL = the legacy default stream)
 */
int tk_init(tk_ctx** out, int64_t d, int32_t N, int64_t K_up, int64_t K_down,
            const float* p_host, void* workspace_dev, size_t workspace_bytes, void* cuda_stream);

/*
 * One iteration (stages 1-4 above).
 *   w_dev      [d]     parameters, updated in place
 *   grads_dev  [N][d]  the workers' vectors, read only
 *   alpha      finite step size
 *   mode       TK_MODE_UNI or TK_MODE_BIDIR, optionally | TK_MODE_EF (error memories, below)
 * Asynchronous.  Inputs are assumed finite.
 */
int tk_step(tk_ctx* ctx, float* w_dev, const float* grads_dev, float alpha, int mode);

/*
 * The same iteration with the workers spread over several GPUs (one process per GPU): the
 * uplink SEND / RECV of Algorithm 1/2 becomes one all-gather of the N messages.  Every process
 * creates its context with the FULL N and p, holds the gradients of its own rows only, and does
 *   tk_step_uplink(ctx, grads_local, row0, rows, alpha, mode)
 *        stage 1 for workers row0 .. row0+rows-1 (grads_local_dev: [rows][d]); their messages
 *        land in rows row0.. of the message buffer (with TK_MODE_EF only those rows' memories
 *        are used and updated)
 *   tk_messages(ctx, &msgs, &bytes_per_row)
 *        the message buffer: [N] rows of K_up entries of 8 bytes (int32 index, fp32 value), in
 *        the context's workspace.  The caller gathers it across processes so that every process
 *        holds all N rows (e.g. an in-place NCCL all-gather when every rank owns N/world rows).
 *   tk_step_server(ctx, w, alpha, mode)
 *        stages 2-4 on the gathered messages.  Every process computes the same sums in the same
 *        worker order, so the replicas of w (and of delta) stay bit-identical.
 * All three are asynchronous on the context's stream; order the exchange after it.
 * tk_step is tk_step_uplink over all rows followed by tk_step_server, fused.
 */
int tk_step_uplink(tk_ctx* ctx, const float* grads_local_dev, int32_t row0, int32_t rows, float alpha, int mode);
int tk_messages(tk_ctx* ctx, void** msgs_dev, size_t* bytes_per_row);
int tk_step_server(tk_ctx* ctx, float* w_dev, float alpha, int mode);

/*
 * The same iteration for callers whose data lives in host memory: copies
 * grads_host ([N][d]) and w_host ([d]) to staging buffers the context allocates
 * on first use (cudaMalloc, 4*(N+1)*d bytes), runs tk_step, copies w back and
 * synchronises.  Pinned host memory makes the copies fast but is not required.
 */
int tk_step_host(tk_ctx* ctx, float* w_host, const float* grads_host, float alpha, int mode);

/*
 * Top_K of every row of x (stage 1 alone; Section 1's compressor).
 *   ctx        a context (its stream is used), or NULL for the legacy default stream
 *   x_dev      [rows][d]
 *   idx_out_dev, val_out_dev   [rows][K], ascending index per row
 * rows, d, K need not match the context.  Scratch memory is taken from a
 * per-device pool that grows with cudaMalloc when a larger problem arrives
 * (tk_release_scratch frees it).  Asynchronous unless the pool has to grow.
 * The pool is one region shared by every tk_topk and tk_last_* call on the device, whatever
 * the context: the library orders its users itself (each call makes its stream wait for the
 * previous user's last kernel, through an event), so calls on different streams or contexts
 * may be issued back to back from one host thread.  Two host threads must not call into the
 * pool at the same time, and a call issued while its stream is being captured into a CUDA
 * graph is not ordered against other users (serialise those yourself).
 */
int tk_topk(tk_ctx* ctx, const float* x_dev, int32_t rows, int64_t d, int64_t K,
            int32_t* idx_out_dev, float* val_out_dev);

/*
 * tk_topk for callers that must not allocate.  (The paper has no counterpart:
 * this is a packaging variant of the call above, not another operation.)
 *
 * Who needs it: code that runs where device allocation is forbidden or
 * impossible — a plugin that lives inside somebody else's memory budget, a
 * real-time loop that may not take the allocator's locks or the implicit
 * device-wide synchronisation of cudaFree, a process whose memory was handed
 * out in full at start-up.  tk_topk would call cudaMalloc the first time (and
 * whenever a larger problem arrives); this entry point never calls cudaMalloc,
 * cudaFree or any other allocating routine.  All of its scratch memory (row
 * states, histograms, candidate lists, sort buffers) lives in one array of
 * TK_NOALLOC_SCRATCH_BYTES bytes that is part of the library image: every GPU
 * that loads the library holds that much memory until the process exits,
 * whether or not this function is ever called.
 *
 *   x_dev, rows, d, K, idx_out_dev, val_out_dev   exactly as for tk_topk; the
 *               caller still provides the input and both outputs
 *   cuda_stream a cudaStream_t (NULL = the legacy default stream)
 *
 * Limits and rules
 *   - The scratch a problem needs grows with rows*(min(d, 4K + 8192) + 2K) *
 *     8 bytes plus about 25 KB per row.  If that exceeds the array the call
 *     returns TK_ERR_TOO_LARGE and does nothing (for example rows = 8 with
 *     K = 4096 fits; K beyond about 80,000 does not fit even for one row).
 *   - The first call on each device looks up the array's device address (with
 *     that device current) and queries launch limits.  Make that first call
 *     before starting any stream capture.
 *   - All calls share the one array, which keeps whatever the previous call
 *     left in it; the function clears the parts that must start at zero.  Two
 *     calls whose GPU work overlaps (different streams, different host
 *     threads) race on it: serialise them.
 *   - The kernels' consistency checks (an entry outside its list, an empty bucket)
 *     report into a status word in the last 256 bytes of the array.  No call clears
 *     it, so it stays set until tk_topk_noalloc_status() reads it: that function
 *     waits for the device (cudaDeviceSynchronize), returns the word (TK_OK or a
 *     negative TK_ERR_* code) and puts it back to zero.  It allocates nothing either.
 * Asynchronous; results are identical to tk_topk's.
 */
#define TK_NOALLOC_SCRATCH_BYTES (4u << 20)
int tk_topk_noalloc(const float* x_dev, int32_t rows, int64_t d, int64_t K, int32_t* idx_out_dev,
                    float* val_out_dev, void* cuda_stream);
int tk_topk_noalloc_status(void);

/*
 * Error memories: the iteration exactly as Algorithm 1 / Algorithm 2 print it.
 *
 * With TK_MODE_EF set in `mode`, tk_step(w, grads, alpha, mode) does
 *   worker q:  a^q = epsilon^q + alpha * g^q;  SEND(Top_K_up(a^q));  epsilon^q <- a^q - Top_K_up(a^q)
 *   server:    S = sum_q p_q Top_K_up(a^q)  (worker order, from +0)
 *     TK_MODE_UNI | TK_MODE_EF    g = S, sent as it is;                     w <- w - g
 *     TK_MODE_BIDIR | TK_MODE_EF  g = S + delta; SEND(Top_K_down(g));
 *                                 delta <- g - Top_K_down(g);               w <- w - Top_K_down(g)
 * (the step size sits inside a^q, as in the paper; one rounding per multiply / add / subtract).
 * The memories live in device memory the caller provides once:
 *   tk_ef_bytes   bytes needed for N worker memories [N][d], the server memory [d] and the
 *                 scratch of the selection over the dense server vector (0 if the sizes are invalid)
 *   tk_ef_attach  mem_dev: at least tk_ef_bytes(d, N, K_down of the context) bytes, 256-byte
 *                 aligned, caller-owned, alive until tk_destroy; sets epsilon = delta = 0 (the
 *                 initialisation line of the algorithms) and synchronises.  Attaching again
 *                 restarts the memories.  After tk_set_kdown to a LARGER K_down, attach again
 *                 before the next TK_MODE_EF step (it is refused otherwise).
 *   tk_ef_state   device pointers to epsilon [N][d] and delta [d] (for checkpoints and tests;
 *                 stream-ordered with the steps).  Either output may be NULL.
 * tk_last_aggregate then reports S (without delta); tk_last_downlink the message sent.
 * Per step this path moves 12 bytes per gradient value (read g, read and write epsilon)
 * instead of 4, plus one pass over the d-long server vector when bidirectional.
 */
size_t tk_ef_bytes(int64_t d, int32_t N, int64_t K_down);
int tk_ef_attach(tk_ctx* ctx, void* mem_dev, size_t bytes);
int tk_ef_state(tk_ctx* ctx, float** eps_dev, float** delta_dev);

/* Change K_downlink of an existing context (1 <= K_down <= d). */
int tk_set_kdown(tk_ctx* ctx, int64_t K_down);

/*
 * Messages of the last tk_step, for inspection.  Each call synchronises, sorts the
 * message by index and writes it to caller-provided device buffers.  The step leaves its
 * messages in arbitrary order in the workspace and the sort permutes them there, in place
 * (the sets do not change and nothing reads their order afterwards; the next step overwrites
 * them).  Unlike a zero-copy accessor these calls hand out no pointer into the workspace:
 * the caller provides the buffers and receives the entry count.
 *   tk_last_uplink     the N uplink messages, [N][K_up]
 *   tk_last_aggregate  the aggregate g as (index, value) over the union U of the
 *                      uplink index sets (g is zero elsewhere); buffers of
 *                      min(N*K_up, d) entries; *count_host = |U|
 *   tk_last_downlink   the downlink message: Top_K_down(g) with exactly K_down
 *                      entries (bidirectional; buffers of K_down entries), or g on
 *                      U (unidirectional; buffers of min(N*K_up, d) entries)
 */
int tk_last_uplink(tk_ctx* ctx, int32_t* idx_out_dev, float* val_out_dev);
int tk_last_aggregate(tk_ctx* ctx, int32_t* idx_out_dev, float* val_out_dev, int64_t* count_host);
int tk_last_downlink(tk_ctx* ctx, int32_t* idx_out_dev, float* val_out_dev, int64_t* count_host);

/* Synchronise the stream and report counters and the sticky device status. */
int tk_status(tk_ctx* ctx, tk_stats* out);

/*
 * The paper's per-step diagnostics.
 *   tk_set_diagnostics(ctx, 1)  makes the following steps also accumulate sums of squares
 *        (one fused multiply-add per value in the streaming pass, fp32 per thread, double across
 *        threads) and count the non-zeros of the aggregate: cheap.
 *   tk_set_diagnostics(ctx, 2)  adds the estimate of the gap constant of the convergence analysis
 *        (rho_hat / rho, the paper's Table 1).  That needs what the method itself never forms,
 *        the dense sum of the workers' vectors and its Top_K: the gradients are read a second
 *        time and one more dense selection runs, so a step takes about twice as long.  The call
 *        allocates 8*d bytes plus selection scratch with cudaMalloc (freed by tk_destroy).
 *   tk_set_diagnostics(ctx, 0)  off (the default).
 *   tk_diagnostics              synchronises and reports, for the last step:
 */
typedef struct tk_diag {
    double nonzero_fraction;        /* nnz(sum_q p_q Top_K(a^q)) / d: the quantity of Fig. 5 / Section 4.2,
                                       which approaches K_up N / d */
    double union_fraction;          /* |U| / d (>= nonzero_fraction; they differ when entries cancel) */
    double compression_factor;      /* K_down / (K_up N): Section 4.2's bound on downlink size vs the aggregate */
    double one_minus_gamma_up_max;  /* max_q ||Top_K(a^q) - a^q||^2 / ||a^q||^2: the "1 - gamma" estimate of the
                                       appendix for the uplink compressions (<= (d - K_up)/d by Eq. "topk_bound") */
    double one_minus_gamma_down;    /* the same for the downlink compression Top_K_down(g); 0 when unidirectional */
    double rho;                     /* level 2 only (else -1).  With a^q the vector worker q compressed and K = K_down:
                                       unidirectional  || Top_K(sum_q p_q a^q) - sum_q p_q Top_K(a^q) || / || s sum_q p_q g^q ||
                                       bidirectional   || Top_K(delta + sum_q p_q a^q) - Top_K(delta + sum_q p_q Top_K(a^q)) ||
                                                       / || s sum_q p_q g^q ||   (delta: server memory before the step)
                                       (the two gap assumptions of Section 3; s = alpha with TK_MODE_EF, else 1: the
                                       step size cancels) */
} tk_diag;
/*   one_minus_gamma_up_host: NULL, or [N] doubles that receive the per-worker values. */
int tk_set_diagnostics(tk_ctx* ctx, int level);
int tk_diagnostics(tk_ctx* ctx, tk_diag* out, double* one_minus_gamma_up_host);

/*
 * Section 4.2's communication model of one iteration.  A sparse message costs two 32-bit words
 * per entry (index and value).  With alpha1 / alpha2 the uplink / downlink latency and beta1 /
 * beta2 the uplink / downlink transfer time of one 32-bit word (caller-supplied, any consistent
 * unit of time), the paper's two formulas are
 *     unidirectional   alpha1 + 2 K_up beta1 + alpha2 + 2 N K_up beta2
 *     bidirectional    alpha1 + 2 K_up beta1 + alpha2 + 2 K_down beta2
 * (the first takes the aggregate at its bound of N K_up non-zeros).
 *   N, K_up, K_down   as for tk_init (1 <= N, 1 <= K_up, 1 <= K_down)
 *   union_size        |U| of a step as tk_status reports it (tk_stats.union_size), 0 <= |U| <= N K_up,
 *                     or -1 when none is known
 * Pure host arithmetic: no context, no device.  Returns TK_ERR_INVALID for sizes out of range,
 * negative or non-finite latencies / word times, or a NULL out.
 */
typedef struct tk_comm {
    int64_t uplink_words;           /* 2 K_up: what one worker sends */
    int64_t downlink_words_uni_max; /* 2 N K_up: the unidirectional downlink at its bound */
    int64_t downlink_words_uni;     /* 2 |U|: what it actually carries (-1 if union_size was -1) */
    int64_t downlink_words_bi;      /* 2 K_down */
    double time_uni;                /* first formula */
    double time_uni_union;          /* first formula with 2 |U| in place of 2 N K_up (-1 if union_size was -1) */
    double time_bi;                 /* second formula */
    double compression_factor;      /* K_down / (K_up N): downlink size after compression relative to the bound */
} tk_comm;
int tk_comm_model(int32_t N, int64_t K_up, int64_t K_down, int64_t union_size, double alpha1, double beta1,
                  double alpha2, double beta2, tk_comm* out);

/* Record device timestamps around the streaming selection pass of every `every`-th tk_step
 * (0 = off, 1 = every step); tk_status reports their sum.  A timestamped step is always issued
 * as plain launches, also when tk_set_graph is on. */
int tk_set_profile(tk_ctx* ctx, int every);

/*
 * Replay steps as CUDA graphs (0/1, off by default).  A step is six to ten small dependent
 * launches around one long one; for small workloads the launch gaps are a tenth of the step.
 * With this on, the first tk_step with a given (w_dev, grads_dev, alpha, mode, K_down) captures
 * the launches into a graph and every later call with the same arguments replays it (up to 16
 * distinct argument sets are kept, least recently used dropped).  Needs a context created on a
 * non-default stream; bypassed for the steps tk_set_profile timestamps and while the caller is
 * itself capturing the stream.  Results are identical.
 */
int tk_set_graph(tk_ctx* ctx, int on);

/*
 * Testing aid: force every selection of this context down the exact multi-pass
 * path (1) or back to the predicted single-pass path with verification (0).
 * Both give identical results.
 */
int tk_set_force_general(tk_ctx* ctx, int on);

/*
 * Testing aid (host-side fault injection): cap the candidate list every row of this context's
 * uplink selections (tk_step, tk_step_uplink, tk_topk with this context) may use at `cap`
 * entries (values below K are raised to K; 0 restores the capacity the workspace was laid out
 * for).  With a cap near K every row overflows its list after the single streaming pass, fails
 * verification and is redone by the exact multi-pass path: the results are identical, only
 * slower.  Returns TK_ERR_INVALID for a negative cap.
 */
int tk_set_cand_cap(tk_ctx* ctx, int64_t cap);

/*
 * Bound reuse (on by default; no counterpart in the paper, which says nothing about how Top_K is
 * computed).  The uplink selection of a long row first needs a lower bound of the row's K-th
 * magnitude; normally it is estimated from a sample of the row at the start of every step.  With
 * reuse on, a row starts from the threshold its selection found in the context's last step, minus
 * a margin (1.5-3 % in value, four times the recent step-to-step movement of the row's threshold
 * if that is more; rows whose threshold moves by more than 6-12 % a step are sampled), and skips
 * the sampling — consecutive iterations of a training run have close thresholds.  Results are identical either way (every bound is verified
 * by the exact count of the components it admits, and a row whose bound fails is redone exactly
 * in the same step); only the time differs: a step whose vectors differ a lot in scale from the
 * step before pays one multi-pass redo, after which the context's rows are sampled for 2, 4, ...
 * up to 1024 steps before warm starts are tried again.  Steps with the error memories (TK_MODE_EF)
 * always sample: the compensated vectors pile up just under their thresholds, where a warm-started
 * bound admits too much.  tk_set_bound_reuse(ctx, 0) samples every step.
 */
int tk_set_bound_reuse(tk_ctx* ctx, int on);

/* Kernels launched on the context's stream since tk_init. */
int64_t tk_launch_count(tk_ctx* ctx);

/*
 * Developer aid, no counterpart in the paper: device timestamps of the last step's kernels.
 * Only a library compiled with -DTK_PHASE_CLOCK=1 records them (every CTA then does two atomics
 * per stamp); the ordinary build returns TK_ERR_INVALID.  Synchronises.  For each of the first n
 * stamps first_us / last_us [n] (host) receive the earliest and the latest time any CTA passed
 * it, in microseconds since the earliest stamp, -1 where no CTA passed.  The 18 stamps, in order:
 * sampling starts / ends; streaming pass starts / ends; verification starts / ends; uplink
 * selection: starts (its predecessors have ended), candidates loaded, first level done,
 * threshold known, ends; server sum starts / ends; downlink selection: the same five.
 * The call then re-arms the stamps, so call it once before the step to be measured.
 */
int tk_debug_phase_clock(tk_ctx* ctx, double* first_us, double* last_us, int32_t n);

/* Free the host-side context (and its staging buffers).  The workspace stays the caller's. */
void tk_destroy(tk_ctx* ctx);

/* Free the scratch pool used by tk_topk and the tk_last_* calls. */
void tk_release_scratch(void);

const char* tk_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* TOPK_H_ */
