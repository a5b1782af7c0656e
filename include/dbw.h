/*
 * dbw.h — C ABI of the cb-DyBW round library (consensus SGD with dynamic backup workers,
 * arXiv 2102.06280) for one NVIDIA B200.
 *
 * N workers are simulated together.  Row i of the row-major N x ld fp32 matrix X is worker
 * i's parameter vector w_i (the paper stores workers as columns of W; this is its transpose).
 * The communication graph is undirected, connected, without self loops, and is given once as
 * sorted CSR (rowptr[N+1], col[nnz]); deg_i = rowptr[i+1] - rowptr[i].  b_i is the number of
 * backup workers of i and p_i = deg_i - b_i the number of neighbours it waits for.
 *
 * Conventions for every entry point
 *   - returns DBW_OK (0) or a negative DBW_ERR_* detected on the host before anything is
 *     launched; nothing is printed.
 *   - pointers marked DEVICE are device memory owned by the caller (never freed, reallocated
 *     or retained past the call unless stated); pointers marked HOST are host memory.
 *   - all device work is enqueued on the `stream` argument (a cudaStream_t passed as void*)
 *     and is asynchronous; the caller synchronises.
 *   - dbw_round, dbw_grad, dbw_mix, dbw_select and dbw_update_backups allocate nothing after their
 *     first call on a handle (dbw_round's gradient workspace and a few kernel attributes are set up
 *     then), so later calls may be captured into a CUDA graph; what a call decides on the host
 *     (which kernel, whether a tracked bf16 copy is reused) is decided at capture time.
 *   - conditions that only the device can see (b_i outside [0, deg_i], NaN arrival time,
 *     a pipeline wait that ran out) set bits in a status word read by dbw_status(); the
 *     kernels clamp and continue, they never trap.
 */
#ifndef DBW_H
#define DBW_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct dbw_handle dbw_handle;

enum {
    DBW_OK = 0,
    DBW_ERR_NULL = -1,       /* a required pointer is NULL */
    DBW_ERR_BAD_GRAPH = -2,  /* CSR unsorted, asymmetric, self loop, index out of range, disconnected */
    DBW_ERR_BAD_SHAPE = -3,  /* N < 1, ld < d, ld % 4 != 0, pointer not 16-byte aligned, illegal aliasing */
    DBW_ERR_BAD_B = -4,      /* host-side b outside [0, deg] */
    DBW_ERR_BAD_MODEL = -5,  /* model descriptor inconsistent with d / ld, or no model / data set */
    DBW_ERR_CUDA = -6,       /* a CUDA runtime call failed; see dbw_last_cuda_error() */
    DBW_ERR_STATE = -7,      /* state blob of the wrong size or version */
    DBW_ERR_TOO_LARGE = -8   /* problem larger than a fixed-capacity entry point accepts */
};

/* flags of dbw_init */
#define DBW_WEIGHT_METROPOLIS 0u /* Assumption 1: w_ij = 1/(1+max{p_i,p_j}), w_ii = 1 - sum */
#define DBW_WEIGHT_UNIFORM 1u    /* w_ii = w_ij = 1/(1+p_i) over self and the kept neighbours */
#define DBW_ORDER_LOCAL_THEN_MIX 0u   /* Algorithm 1, Eqs. 4-5 */
#define DBW_ORDER_MIX_THEN_CORRECT 2u /* Eq. 3 restricted to the kept set */
#define DBW_GEMM_FP32 0u /* dense layers in fp32 on the CUDA cores */
#define DBW_GEMM_BF16 4u /* dense layers with BF16 operands on tcgen05 tensor cores, fp32 accumulate */

/* bits of the device status word */
#define DBW_STATUS_BAD_B 1u       /* some b_i was outside [0, deg_i] (clamped), or a kept mask given to dbw_mix
                                     does not hold deg_i - b_i entries for some i */
#define DBW_STATUS_NAN_TIME 2u    /* some arrival time was NaN (ordered last) */
#define DBW_STATUS_WAIT_TIMEOUT 4u /* a bounded pipeline wait expired; results of that call are invalid */
#define DBW_STATUS_BOUNDS 32u     /* bounds-checked build only (libdbw_dbg.so): an index a kernel read from its own data
                                     (graph, mixing plan, worker order) was out of range; the access was redirected */
#define DBW_STATUS_INTERNAL 16u   /* a kernel found its own precomputed data inconsistent (should not happen) */
#define DBW_STATUS_BAD_INDEX 8u   /* a batch index was outside [0, S) or a label outside [0, classes) (clamped) */

#define DBW_MAX_LAYERS 8

/*
 * Model: ReLU MLP dims[0] -> dims[1] -> ... -> dims[n_layers] with mean softmax cross-entropy
 * (Eq. 2: the mini-batch stochastic gradient g(w_j)).  Layer l (0-based) has W_l stored
 * row-major [dims[l+1]][dims[l]] at float offset w_off[l] of a parameter row and its bias at
 * b_off[l].  Offsets are multiples of 32 floats; the gaps and the tail up to ld are padding
 * that stays zero.  dbw_model_layout() fills a descriptor with the canonical padded layout.
 */
typedef struct {
    int32_t n_layers;
    int32_t dims[DBW_MAX_LAYERS + 1];
    int64_t w_off[DBW_MAX_LAYERS];
    int64_t b_off[DBW_MAX_LAYERS];
    int32_t batch; /* mini-batch size |C_j(k)| per worker */
} dbw_model_desc;

/* Canonical padded layout.  HOST in: dims[n_layers+1], batch; out: *desc, *d (logical
 * parameter count: sum of out*in + out), *ld (padded row length, multiple of 32). */
int dbw_model_layout(const int32_t* dims, int32_t n_layers, int32_t batch, dbw_model_desc* desc,
                     int64_t* d, int64_t* ld);

/*
 * Section 2.1 (graph, neighbourhoods) and Algorithm 2's input (the link set P).
 * Validates and copies the HOST CSR, builds P as the breadth-first spanning tree from worker 0
 * (neighbours in ascending index, links in discovery order), allocates the workspace on
 * `device` and returns the handle.  `model` may be NULL (mixing only: gradients are supplied
 * to dbw_round / dbw_mix).  The handle owns only its workspace.
 */
int dbw_init(dbw_handle** out, int32_t N, int64_t d, int64_t ld, const int32_t* h_rowptr,
             const int32_t* h_col, const dbw_model_desc* model, uint32_t flags, int device);
int dbw_destroy(dbw_handle* h);

/* Local data sets D_j (Section 2.1).  DEVICE feat [N][S][dims[0]] fp32, labels [N][S] int32 in
 * [0, dims[L]).  The pointers are retained (not copied) until replaced or the handle dies. */
int dbw_set_dataset(dbw_handle* h, const float* feat, const int32_t* labels, int32_t S);

/*
 * Section 2.2 (worker j waits for the first p_j updates) and Section 3.2.2 (T_j, T).
 * DEVICE in : t[N] f64 arrival time of each worker's update, b[N] int32.
 * DEVICE out: kept[nnz] uint8 aligned with col (1 = waited for, 0 = backup); ties in t go to
 *             the lower worker index;
 *             T_nbr[N]    max t over the kept neighbours (0.0 when p_i = 0);
 *             T_worker[N] max(t_i, T_nbr[i]) when p_i >= 1; t_i when i is only waited for by
 *                         others; 0.0 when i takes no part;
 *             T_round[1]  max of T_worker over the workers that take part (0.0 if none); without
 *                         per-link times this is the max of t over them.
 * Only comparisons are applied to t, so the outputs are bit-exact.  Any out pointer but kept
 * may be NULL.
 */
int dbw_select(dbw_handle* h, const double* t, const int32_t* b, uint8_t* kept, double* T_worker,
               double* T_nbr, double* T_round, void* stream);

/*
 * Per-link arrival times (a generalisation the paper leaves open: it takes the communication delay
 * as negligible, Section 4).  DEVICE t_edge[nnz], aligned with col: the update of worker col[e]
 * reaches worker i (the row of e) at t_edge[e].  While set, dbw_select / dbw_round / dbw_round_host
 * rank worker i's neighbours by these times (ties to the lower index), T_nbr is the latest kept
 * link time, T_worker[i] = max(t_i, T_nbr[i]) and T_round = max of T_worker over the workers that
 * take part.  The pointer is retained, not copied; pass NULL to return to per-worker times.  The
 * threshold rule (dbw_update_backups) keeps using the per-worker times.
 */
int dbw_set_edge_times(dbw_handle* h, const double* t_edge);

/*
 * dbw_select for callers that must not allocate.  (The paper has no counterpart: this is an
 * integration aid, not a step of the method.)
 *
 * Everything else in this library works through a handle, and dbw_init allocates the handle's
 * workspace with cudaMalloc.  Some callers cannot do that at the point where they need a
 * selection: code running inside a latency-critical loop where cudaMalloc's implicit device
 * synchronisation is not acceptable, plug-ins hosted by a framework whose caching allocator
 * already owns all of device memory, and callers that are handed a fixed memory budget and are
 * forbidden to grow it.  This entry point needs no handle and performs no cudaMalloc / cudaFree
 * (nor any other allocating call): the scratch the selection kernel needs (one flag and one
 * double per worker plus two counters, about 193 KB) is a fixed array compiled into the library,
 * which every GPU that loads the library holds until the process exits.
 *
 * DEVICE in : rowptr[N+1], col[nnz] — the same sorted, symmetric, self-loop-free CSR that
 *             dbw_init would take, but already on the device and NOT validated here;
 *             t[N], b[N] as in dbw_select.
 * DEVICE out: kept, T_worker, T_nbr, T_round exactly as dbw_select writes them (same kernel,
 *             so the results are bit-identical); status_out[1] (nullable) receives the
 *             DBW_STATUS_* bits of this call.
 * Limits and caveats
 *   - N <= DBW_SELECT_STATIC_MAX_N, otherwise DBW_ERR_TOO_LARGE and nothing is launched.
 *   - Works on the CURRENT device.  The first call on each device looks up the device address
 *     of the built-in array (cudaGetSymbolAddress); make that first call outside any stream
 *     capture.
 *   - All calls on a device share the one array, which still holds the previous call's
 *     contents; each call clears the part that must start at zero with a memset on `stream`.
 *     Two calls that may overlap on the GPU (different streams, no ordering between them) race
 *     on it and produce garbage: serialise them.
 */
#define DBW_SELECT_STATIC_MAX_N 16384
int dbw_select_static(int32_t N, const int32_t* rowptr, const int32_t* col, const double* t,
                      const int32_t* b, uint8_t* kept, double* T_worker, double* T_nbr,
                      double* T_round, uint32_t* status_out, void* stream);

/*
 * Eq. 2.  DEVICE in: X [N][ld]; batch_idx [N][batch] int32 sample indices into the data set.
 * DEVICE out: G [N][ld] fp32, g(w_i) in the layout of X (padding untouched: pass it zeroed);
 * loss [N] fp32 mean cross-entropy of each worker's batch (nullable).
 */
int dbw_grad(dbw_handle* h, const float* X, const int32_t* batch_idx, float* G, float* loss,
             void* stream);

/*
 * Assumption 1 (weights) + Eqs. 4-5 or Eq. 3 (update), every row read from the OLD X.
 * DEVICE in : X [N][ld], G [N][ld], kept[nnz], b[N]; lr scalar; lr_per_worker[N] fp32 nullable
 *             (eta_j; overrides lr).  G may be NULL: the gradients are taken as zero and nothing of G
 *             is read (the consensus-only iterations of the truncated model of Section 3.2.1, whose
 *             rows converge to their common mean by Corollary 1): 8 bytes per element instead of 12.
 *             With uniform weights the weight is 1 / (1 + number of entries set in kept's row i); with
 *             the weights of Assumption 1 the counts p = deg - b of both ends are used.  A row of kept
 *             that does not hold deg_i - b_i entries sets DBW_STATUS_BAD_B.
 * DEVICE out: X_out [N][ld].  X_out may alias X exactly (in place) when dbw_mix_in_place_ok()
 *             is 1; partial overlap is an error.  G is read only.
 * Summation order per element is fixed (self, then kept neighbours in CSR order), so results
 * are reproducible run to run.
 */
int dbw_mix(dbw_handle* h, const float* X, const float* G, const uint8_t* kept, const int32_t* b,
            float lr, const float* lr_per_worker, float* X_out, void* stream);
int dbw_mix_in_place_ok(const dbw_handle* h);
/* Expert knob: columns per shared-memory panel of the mix kernel: 0 = automatic, 16 / 32 / 64 /
 * 128 / 256 = fixed (falls back to the direct kernel when N * cols * 4 bytes exceed shared memory),
 * 1 = the tensor-memory staged kernel wherever it applies (64 <= N <= 1024; with the Metropolis
 *     weights degrees up to 62),
 * 2 = the tensor-core kernel wherever it applies (uniform weights, 256 <= N <= 1024): the mix as a
 *     dense product with the 0/1 selection matrix, every fp32 value split exactly into three BF16
 *     pieces, fp32 accumulation; with N > 512 it cannot run in place (dbw_mix_in_place_ok() = 0),
 *  3 = the structured-sparse tensor-core kernel wherever it applies (uniform weights, 256 <= N <= 1024, a
 *      2:4 order of the graph exists, see dbw_graph_order_2of4): the same product with the selection
 *      matrix compressed 2:4, at twice the dense tensor-core rate; in place only for N <= 512,
 * -1 = always the direct (L2 re-read, out-of-place only) kernel. */
int dbw_set_mix_panel(dbw_handle* h, int32_t cols);
/* Which mix kernel the current settings select: 0 = direct (L2 re-read), 1 = shared-memory panel,
 * 2 = tensor-memory staged, 3 = tensor-core, 4 = structured-sparse tensor-core.  Negative on error. */
int dbw_mix_kernel(const dbw_handle* h);

/*
 * Algorithm 1, one iteration: gradients (dbw_grad, or G_ext when batch_idx is NULL), selection
 * (dbw_select) and the update (dbw_mix) in one call.  Arguments as in those three; loss is
 * nullable; G_ext [N][ld] is used iff batch_idx == NULL, and when both are NULL the round is a
 * consensus-only one (G = 0, nothing of G read).  With batch_idx the selection kernel is
 * queued on a stream of the handle that waits for everything queued on `stream` so far and that
 * `stream` waits for before the mix: to the caller all work is still ordered on `stream`.
 */
int dbw_round(dbw_handle* h, const float* X, const double* t, const int32_t* b,
              const int32_t* batch_idx, const float* G_ext, float lr, const float* lr_per_worker,
              float* X_out, uint8_t* kept, double* T_worker, double* T_nbr, double* T_round,
              float* loss, void* stream);

/*
 * Single-launch round (Algorithm 1, one iteration, as ONE cooperative kernel launch).  For networks whose
 * round is bound by launch latency (an fp32 model and at most 64 workers) dbw_round with batch_idx runs
 * gather, forward, loss, backward, selection, weights, times and the mix inside one persistent kernel with
 * grid-wide barriers between dependent steps.  The results are bit-identical to the multi-launch path (the
 * same device functions in the same order per output element).  enable = -1 (the default) uses it where it
 * is the faster path (networks of up to about 6e7 multiply-adds per forward pass: above that the per-step
 * kernels, which put more blocks on an SM than a cooperative grid can, win), 1 wherever it applies, 0 never.
 * dbw_round_is_fused() tells which path dbw_round would take (1 = single launch).  With stage timing on, the
 * whole launch is reported under stage 0.
 */
int dbw_set_fused_round(dbw_handle* h, int enable);
int dbw_round_is_fused(const dbw_handle* h);

/*
 * Parameter tracking for chained rounds (tensor-core path; a no-op otherwise).  Each round the
 * BF16 GEMMs need a bf16 copy of the weights.  With tracking on, dbw_mix / dbw_round write that copy
 * next to X' (same values as a later cast, so results do not change), and the next dbw_grad /
 * dbw_round skips the cast when its X is the very X_out of the previous call.  The caller promises
 * not to modify that buffer in between; if it does (or passes other parameters at the same
 * address), it must turn tracking off and on again, which forgets the copy.  Off by default.
 */
int dbw_set_param_tracking(dbw_handle* h, int enable);

/*
 * The same round for callers whose per-round inputs live in HOST memory (pinned memory makes
 * the copies asynchronous).  X / X_out / G_ext stay DEVICE (the parameters are the state of the
 * simulation); h_t[N], h_b[N], h_batch_idx[N][batch] are copied to the device on `stream`, the
 * round runs, and h_kept[nnz], h_T_worker[N], h_T_round[1], h_loss[N], h_b_out[N] (each
 * nullable) are copied back on `stream`.  When h_b is NULL the backup counts come from the
 * threshold rule: dbw_update_backups runs on the copied times first (Algorithm 2 feeding
 * Algorithm 1) and h_b_out receives them.  The call does not synchronise.
 */
int dbw_round_host(dbw_handle* h, const float* X, const double* h_t, const int32_t* h_b,
                   const int32_t* h_batch_idx, const float* G_ext, float lr, float* X_out,
                   uint8_t* h_kept, double* h_T_worker, double* h_T_round, float* h_loss,
                   int32_t* h_b_out, void* stream);

/*
 * Section 4.1 (threshold rule) and Algorithm 2 (one iteration of the epoch).
 * DEVICE in : t_next[N] f64, the arrival times of the round about to run.
 * DEVICE out: b_out[N] int32, theta_out[1] f64 (nullable).
 * theta = the smallest max(t_u, t_v) over the links (u,v) of P not yet covered in this epoch
 * (first such link on ties); that link becomes covered; after |P| = N-1 calls the covered set
 * is emptied.  Then p_j = #{i in N_j : t_i <= theta} if t_j <= theta, else 0; b_j = deg_j - p_j.
 * The epoch state lives on the device and advances in stream order.
 */
int dbw_update_backups(dbw_handle* h, const double* t_next, int32_t* b_out, double* theta_out,
                       void* stream);
int dbw_reset_backups(dbw_handle* h, void* stream); /* empty the covered set, restart the epoch */

/* Epoch state (covered links, position in the epoch) as an opaque blob, for resuming a run.
 * HOST buf; *size in: capacity, out: bytes needed/written.  Both synchronise `stream`. */
int dbw_state_export(dbw_handle* h, void* buf, size_t* size, void* stream);
int dbw_state_import(dbw_handle* h, const void* buf, size_t size, void* stream);

/* Device status word (DBW_STATUS_* bits, accumulated since the last call); synchronises the
 * device.  Returns the bits (>= 0) or a negative error. */
int dbw_status(dbw_handle* h);

/* Spanning links P on the HOST: links[2*(N-1)] receives (u,v) pairs; returns N-1 or an error. */
int dbw_get_links(const dbw_handle* h, int32_t* links);

/*
 * Stage timing.  While enabled, every dbw_round / dbw_round_host records CUDA events around its
 * stages (0 = gradients, 1 = selection + plan, 2 = mix), up to 4096 rounds.  When the round computes
 * gradients the selection, which needs only t and b, runs beside them on a stream of the handle
 * (forked from and joined back into the caller's stream), so the three times may add up to more
 * than the round took.  dbw_profile_read() waits for the recorded events, adds their elapsed times to
 * ms[4] (HOST: the three stages, then ms[3] = the tensor-core GEMM launches inside the gradient stage, each
 * between events of its own; 0 on the fp32 path), stores the number of rounds in *rounds and clears the record.  Do not enable
 * it while the stream is being captured into a CUDA graph.
 */
int dbw_profile(dbw_handle* h, int enable);
int dbw_profile_read(dbw_handle* h, double* ms, int32_t* rounds);

/*
 * Self-test of the bounded waits of the tensor-core pipelines (no passage of the paper: a safety
 * property of this implementation).  Launches one small kernel in which a thread waits, with a limit of
 * `polls` polls (1 .. 2^20), on a barrier that nothing completes, then waits on it again.  DEVICE
 * out[3]: out[0] = 1 when the first wait gave up, out[1] = 1 when the second wait returned without
 * completing, out[2] = clock ticks the second wait took (it must not spin: the first expired wait makes
 * every later wait of the thread block return at once).  Sets DBW_STATUS_WAIT_TIMEOUT in the handle's
 * status word, as an expired wait in a real pipeline does; the context stays usable.
 */
int dbw_debug_wait_probe(dbw_handle* h, uint32_t polls, uint32_t* out, void* stream);

/*
 * Worker reordering for the structured-sparse tensor-core mix (Eq. 5 as the product of the 0/1 selection
 * matrix with the parameter matrix; the paper prescribes no order of the workers, so any order is the
 * same method).  HOST in: the sorted CSR of dbw_init.  HOST out: order[k], k < the returned count, is the
 * worker placed at input position k, or -1 for a position left empty.  The order is such that for every
 * worker i no aligned group of four consecutive positions holds more than two members of {i} + N_i, so
 * every row of every selection matrix the graph admits is 2:4 sparse.  Deterministic.  Returns the number
 * of positions used (a multiple of 128, at most 1024 and at most `capacity`), 0 when no such order was
 * found, or a negative error.  Needs no GPU.
 */
int dbw_graph_order_2of4(int32_t N, const int32_t* h_rowptr, const int32_t* h_col, int32_t* order, int32_t capacity);

/* Kernels launched by this library since it was loaded (for launch accounting). */
int64_t dbw_launch_count(void);
/* cudaError_t of the last failing runtime call in this library (0 if none). */
int dbw_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* DBW_H */
