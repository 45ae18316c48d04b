/*
 * powergossip.h - C ABI of the B200 PowerGossip library.
 *
 * PowerGossip (Vogels, Karimireddy, Jaggi, "Practical Low-Rank Communication
 * Compression in Decentralized Deep Learning"): every pair of neighbouring
 * workers (i, j) keeps a small warm-started vector and uses power-iteration
 * steps to build a low-rank approximation of the difference of their
 * parameter matrices, which replaces the full difference in the gossip
 * averaging update (Section 4, Eq. 2 and 3, Algorithm 2).
 *
 * This library simulates the whole decentralized network on ONE GPU: the
 * parameter stacks of all workers stay resident in device memory and the
 * "communication" between the two ends of an edge is an exchange of the small
 * vectors through device buffers.  All arithmetic of the method runs in CUDA
 * kernels; there is no CPU fallback.
 *
 * Conventions
 *   - Every call returns a pg_status (PG_OK == 0).  Nothing throws, aborts or
 *     traps across this boundary.  Out-parameters are written only on success.
 *   - "host" / "device" is stated for every pointer.  The library allocates no
 *     device memory: the caller passes one workspace of pg_workspace_bytes()
 *     bytes (cudaMalloc / torch.empty, 256-byte aligned) which must outlive the
 *     context.  Host-side tables are owned by the context.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *     One context is used from one host thread and one stream at a time.
 *   - Matrices are dense row-major fp32, rows x cols, on the host side of the
 *     API; inside the workspace rows are padded to a multiple of 4 floats.
 *   - Worker ids are 0..n_workers-1.  An edge is stored once, as (i, j), i < j.
 */
#ifndef POWERGOSSIP_H_
#define POWERGOSSIP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(PG_BUILDING_LIBRARY)
#define PG_API __attribute__((visibility("default")))
#else
#define PG_API
#endif

typedef enum pg_status {
    PG_OK = 0,
    PG_ERR_INVALID = 1,    /* bad argument, invalid topology or mixing matrix      */
    PG_ERR_WORKSPACE = 2,  /* workspace missing, misaligned, too small, not device */
    PG_ERR_CUDA = 3,       /* a CUDA runtime call failed                           */
    PG_ERR_STATE = 4,      /* call not allowed in the context's current state      */
    PG_ERR_TIMEOUT = 5,    /* a bounded device-side wait gave up                   */
    PG_ERR_NUMERIC = 6,    /* a norm was not finite (NaN / Inf in the parameters)  */
    PG_ERR_TOO_LARGE = 7,  /* problem exceeds the fixed scratch of a no-allocation call */
    PG_ERR_BOUNDS = 8      /* bounds-checked build only: a kernel computed an address outside its section */
} pg_status;

/* Graph kinds.  The paper's experiments use rings; Assumption A4 (Section 5.1)
 * allows any undirected connected graph, and Theorem 1 allows the compressors
 * (hence the graph) to change over time. */
enum {
    PG_RING = 0,      /* edges {i, (i+1) mod N}                                       */
    PG_TORUS = 1,     /* torus_rows x torus_cols grid with wrap-around, id = r*C + c   */
    PG_MATCHING = 2,  /* time-varying: a perfect matching re-drawn every round (N even) */
    PG_CUSTOM = 3     /* caller's edge list                                            */
};

/* How the gossip weight W_ij of an edge is chosen (Assumption A4: W symmetric,
 * doubly stochastic, non-zero only on edges; the self weight is 1 - row sum). */
enum {
    PG_W_UNIFORM = 0,     /* 1 / (max degree + 1)                                  */
    PG_W_METROPOLIS = 1,  /* 1 / (1 + max(deg_i, deg_j)); 1/2 on a matching        */
    PG_W_EXPLICIT = 2     /* the N x N matrix passed to pg_create                  */
};

typedef struct pg_topology {
    int32_t kind;                 /* PG_RING ... PG_CUSTOM                               */
    int32_t n_workers;            /* N >= 2                                              */
    int32_t torus_rows;           /* PG_TORUS only; rows * cols == N                     */
    int32_t torus_cols;
    int32_t weight_rule;          /* PG_W_*; ignored for PG_MATCHING (always 1/2)        */
    int32_t n_custom_edges;       /* PG_CUSTOM only                                      */
    const int32_t *custom_edges;  /* host, 2*n_custom_edges ints; copied by pg_create    */
} pg_topology;

typedef struct pg_layer_shape {
    int32_t rows;  /* output size (output channels for a convolution)               */
    int32_t cols;  /* input size (input channels x kernel height x kernel width)    */
} pg_layer_shape;

typedef struct pg_ctx pg_ctx;  /* opaque; host memory owned by the library */

/* Limits of the library as compiled. */
#define PG_MAX_RANK 4          /* columns per edge                                    */
#define PG_MAX_SLOTS 8         /* (max degree) * rank vectors handled per worker      */

/*
 * Size in bytes of the device workspace a context with these parameters needs
 * (parameters of all workers, per-pair vectors, exchange buffers, tables; on a
 * static graph of degree 2 at rank 1, and at rank 2 with layers the pair sweep
 * takes, a second copy of the parameters, see pg_round).  `shapes`: host, n_layers entries.  PG_ERR_INVALID for a bad topology, rank
 * outside 1..PG_MAX_RANK or degree*rank > PG_MAX_SLOTS.
 */
PG_API int pg_workspace_bytes(const pg_topology *topo, const pg_layer_shape *shapes, int32_t n_layers,
                       int32_t rank, size_t *bytes_out);

/*
 * Build a network (Algorithm 2, initialisation; Assumption A4).
 *   topo, shapes  host; copied.
 *   W_host        host, N x N row-major fp32 mixing matrix, required for
 *                 PG_W_EXPLICIT and ignored otherwise.  Checked against A4:
 *                 symmetric, off-diagonal entries >= 0 and non-zero only on
 *                 edges, every row sums to 1 within 1e-5; an edge weight of 0 is
 *                 accepted only for PG_CUSTOM (it freezes that edge's update).
 *   rank          columns of every per-edge factor (1 = the paper's Algorithm 2;
 *                 > 1 orthogonalises instead of normalising, Appendix "Changing
 *                 rank vs changing # power iterations").
 *   power_steps   power steps per round; one step = two consecutive iterations
 *                 of Algorithm 2 (X, then X transposed) followed by the update.
 *   seed          keys the per-pair standard-normal initial vectors (Philox4x32-10
 *                 + Box-Muller: entry e of column k of pair (i<j), layer l uses
 *                 counter (e/4, l, i, j*256+k)) and the per-round matchings.
 *   dev_workspace device, >= pg_workspace_bytes(), 256-byte aligned, on the
 *                 current device; zeroed and filled by this call (synchronous).
 * All parameters start at zero; load them with pg_write_params.
 */
PG_API int pg_create(const pg_topology *topo, const float *W_host, const pg_layer_shape *shapes,
              int32_t n_layers, int32_t rank, int32_t power_steps, uint64_t seed,
              void *dev_workspace, size_t workspace_bytes, pg_ctx **ctx_out);

/* Free the host side of a context (NULL is accepted).  The workspace stays the
 * caller's.  Does not synchronise: finish the stream first. */
PG_API void pg_destroy(pg_ctx *ctx);

/*
 * Copy one dense rows x cols fp32 matrix from host memory into worker
 * `worker`'s layer `layer` (Algorithm 1, input X_i^(0)).  Asynchronous on
 * `stream` when host_src is pinned; host_src must stay valid until the stream
 * reaches the copy.
 */
PG_API int pg_write_params(pg_ctx *ctx, int32_t worker, int32_t layer, const float *host_src, void *stream);

/*
 * Copy worker `worker`'s layer `layer` to host memory (dense rows x cols fp32),
 * then wait for `stream` and report the device status word: PG_ERR_NUMERIC if a
 * non-finite norm was met in any round since the context was created.
 */
PG_API int pg_read_params(pg_ctx *ctx, int32_t worker, int32_t layer, float *host_dst, void *stream);

/*
 * pg_read_params without the wait: the copy to host_dst (pinned memory, valid
 * until the stream reaches the copy) is only enqueued on `stream`, and the device
 * status word is not looked at - call pg_device_status when the results matter.
 * A correction still pending from the last round (see pg_round) is first applied
 * on `stream`, as in pg_read_params.  With it a caller can run the read-back of one
 * round's result (Algorithm 1's output X_i) on one stream beside the upload of the
 * next input on another, one matrix gated on the other by events of its own; the
 * context does not order streams against each other.
 */
PG_API int pg_read_params_async(pg_ctx *ctx, int32_t worker, int32_t layer, float *host_dst, void *stream);

/*
 * Device view of worker `worker`'s layer `layer` for local updates between
 * rounds - Algorithm 1's  - eta G  term: the caller subtracts its scaled
 * gradient in place with its own kernels.  *dev_ptr_out points at rows x cols
 * fp32 values with leading dimension *ld_out floats (cols rounded up to 4; the
 * padding columns must stay zero).  Any correction still pending is applied
 * first (enqueued on `stream`), and the cached forward product is dropped, so
 * the next pg_round starts from whatever the caller leaves there.  Work on the
 * view must be ordered after this call and before the next pg_round on the same
 * stream.  The pointer stays valid for the life of the workspace, but call this
 * again after every round before touching X.
 */
PG_API int pg_params_device(pg_ctx *ctx, int32_t worker, int32_t layer, void *stream, float **dev_ptr_out,
                            int64_t *ld_out);

/*
 * Enqueue one gossip round on `stream` (asynchronous): `power_steps` power
 * steps on every layer and every edge of this round's graph, each one
 *     Qh = unit columns of the pair's stored Q        (Algorithm 2, v / ||v||)
 *     P  = X_i Qh - X_j Qh,  Ph = orthonormalised P   (Eq. 3, odd iteration)
 *     Q' = X_i^T Ph - X_j^T Ph                        (Eq. 3, even iteration)
 *     X_i -= W_ij Ph Q'^T,  X_j += W_ij Ph Q'^T,  Q = Q'   (Eq. 2; Lemma 1)
 * with all edges of a step reading the same pre-update X.  Advances the round
 * counter.  At rank 1, on a matching and on static graphs of degree <= 2 without
 * isolated workers (rings, paths), layers may run through the "pair sweep": one
 * read of both ends of an edge gives p = D q-hat and D^T p, and the correction
 * of a step is applied to the copy of X in memory by the next step's sweep, or
 * by pg_read_params / pg_write_params / pg_params_device / pg_write_q /
 * pg_set_round, whichever comes first; every call of this API sees the fully
 * updated X.  On degree 2 a row has two readers, so the sweep writes corrected
 * rows to a second copy of the stack and the copies swap roles every step; the
 * calls above always leave the result in the copy pg_params_device points to.
 * There, all layers take the pair sweep when the stack is at most 48 MiB, else
 * only layers of at least 256 rows and 2^20 elements, and the kernels of the
 * other layers run on a stream of the library's own that is forked from and
 * joined to `stream` with events inside the call.  At rank 2 the pair sweep
 * exists for those graphs of degree 2 and layers of that size with rows of
 * 1025 to 5120 floats: one read gives P = D [q-hat_0 q-hat_1] and D^T P, and
 * the Gram-Schmidt step is applied afterwards as a 2 x 2 triangular map taken
 * from P^T P (same column order and same dependent-column rule).  PG_DISABLE_PAIR_SWEEP=1
 * in the environment at creation selects the general three-sweep path.
 * The kernels of a round are launched with programmatic stream serialisation
 * where that was measured to pay (each waits on the device for the kernel
 * before it, so results do not depend on it); PG_DEPENDENT_LAUNCH=0 in the
 * environment at creation gives plain launches.
 * Host-side errors are returned at once; device-side ones show up in
 * pg_read_params / pg_device_status.
 */
PG_API int pg_round(pg_ctx *ctx, void *stream);

/*
 * One round of Algorithm 1 with the local term: pg_round, and with the round's
 * last update every worker's matrices also lose eta * G (line 6 of Algorithm 1:
 * X_i <- X_i + sum_j W_ij C(X_j - X_i) - eta G_i, the gossip term computed from
 * the parameters the gradient was taken at).  The gradient is read in the sweep
 * that applies the update, so it costs one extra read of G (4 B per parameter)
 * and no pass of its own; on return (of the enqueued work) X in memory is
 * fully updated, ready for the next gradient evaluation.
 *   G_dev   device, caller-owned, pg_stack_elems floats, 16-byte aligned, laid out
 *           like the parameter stack: the rows x cols matrix of (worker, layer)
 *           starts at pg_stack_offset's offset, row-major with its leading
 *           dimension ld >= cols.  Only the rows x cols entries are read for
 *           their values; the padding may hold anything finite or not.  Must
 *           stay unchanged until the enqueued work has run.
 *   eta     finite step size.
 * In half-step and random-projection modes the gradient step is a pass of its
 * own after the round (12 B per parameter).  PG_ERR_INVALID for a null,
 * misaligned, host or other-device G or a non-finite eta; otherwise as pg_round.
 */
PG_API int pg_round_sgd(pg_ctx *ctx, const float *G_dev, float eta, void *stream);

/*
 * Shape of one copy of the parameter stack, for caller-owned buffers that
 * mirror it (gradients): total floats, and where (worker, layer) starts (in
 * floats from the start of the buffer) with its leading dimension.  Offsets are
 * multiples of 64 floats.  Host out-params, written only on PG_OK.
 */
PG_API int pg_stack_elems(pg_ctx *ctx, int64_t *elems_out);
PG_API int pg_stack_offset(pg_ctx *ctx, int32_t worker, int32_t layer, int64_t *offset_out, int64_t *ld_out);

/*
 * Algorithm 2 read literally ("half-step mode"): every iteration is ONE
 * mat-vec and one gossip update with that iteration's approximation, and the
 * stored vector alternates between R^cols and R^rows:
 *   k odd :  vh = v/||v||;  p = X_i vh - X_j vh;  X_i -= W p vh^T, X_j += W p vh^T;  v <- p
 *   k even:  the same with X transposed:  q = X_i^T vh - X_j^T vh;
 *            X_i -= W vh q^T, X_j += W vh q^T;  v <- q
 * `power_steps` then counts iterations per round (the algorithm's s), and one
 * iteration moves (rows+cols)/2 floats per edge direction on average, the count
 * behind the per-tensor compression ratios of the paper's parameter tables.  A
 * zero vector normalises to zero.  Call before the first round.  Needs rank 1
 * and a static graph (PG_ERR_INVALID otherwise; PG_ERR_STATE once rounds have
 * run).  Moves every layer to the three-sweep path for the life of the context.  In this mode pg_read_q / pg_write_q are only meaningful
 * after an even number of iterations, when the vector is back in R^cols.
 */
PG_API int pg_set_half_step(pg_ctx *ctx, int32_t on);

/*
 * Random-projection compressors instead of power iteration (Section 5.1, the
 * examples after Assumption A5; the paper's comparison "random projections vs
 * power iteration"):
 *   PG_RANDOM_RIGHT  C(X) = (X U) U^T,  U uniformly drawn orthonormal cols x rank   (delta = rank/cols)
 *   PG_RANDOM_LEFT   C(X) = V (V^T X),  V uniformly drawn orthonormal rows x rank   (delta = rank/rows)
 * Fresh directions for every edge, layer and power step, nothing warm-started:
 * Philox4x32-10 / Box-Muller normals as for the initial vectors, under the key
 * (seed_lo ^ low32(t+1), seed_hi ^ high32(t+1) ^ 0x52503031) for step t, then
 * Gram-Schmidt.  The stored per-pair vectors are overwritten by the directions.
 * Call before the first round; not available on PG_MATCHING (PG_ERR_INVALID),
 * nor together with half-step mode.  Moves every layer to the three-sweep path
 * for the life of the context.  A step costs one read of X
 * for the product and one read + write for the update (12 B per parameter).
 */
enum { PG_POWER_ITERATION = 0, PG_RANDOM_RIGHT = 1, PG_RANDOM_LEFT = 2 };
PG_API int pg_set_random_projection(pg_ctx *ctx, int32_t mode);

/*
 * Enqueue `n_rounds` rounds (same result as calling pg_round that many times).
 * When the graph is static and the whole stack is small enough to stay in L2
 * (at most 64 MiB of parameters, no layer on the pair sweep), all rounds run in ONE
 * cooperative kernel launch whose phases are separated by a grid barrier; the
 * barrier waits are bounded, and a wait that runs out ends the launch and sets
 * PG_ERR_TIMEOUT in the device status word.  Otherwise, on a static graph and
 * for four rounds or more, the first rounds are enqueued one by one until the
 * launches repeat, then two rounds are captured once as a CUDA graph (on a
 * stream of the library's own; nothing of the caller's is captured) and the graph
 * is launched into `stream` as often as needed; a remainder, and every round of
 * a time-varying graph, is enqueued one by one.  The same kernels run either way.
 * While `stream` itself is being captured by the caller, and with per-kernel
 * timing on (pg_timing_enable), only plain launches are used.
 */
PG_API int pg_rounds(pg_ctx *ctx, int32_t n_rounds, void *stream);

/*
 * Self-test of the bounded grid barrier (the paper has no counterpart): launches
 * a few CTAs on a barrier that expects one arrival more than will come.  Every
 * CTA must give up after about a millisecond; the call waits for `stream` and
 * returns PG_ERR_TIMEOUT when that happened (the expected outcome), PG_OK if the
 * wait was not reported.  The status word keeps the time-out bit afterwards and
 * the context refuses further rounds (PG_ERR_STATE), as after any time-out: use a
 * context of its own.
 */
PG_API int pg_selftest_barrier_timeout(pg_ctx *ctx, void *stream);

/*
 * Self-test of the bounds-checked build (the paper has no counterpart): a kernel asks the
 * check about a range that ends one float past the parameter section, without touching it.
 * Waits for `stream` and returns PG_ERR_BOUNDS from a library built with -DPG_BOUNDS_CHECK
 * (python -m paper_2008_01425_b200.build --checked), PG_OK from the regular one, where the
 * checks are compiled out.  The status word keeps the bit: use a context of its own.
 */
PG_API int pg_selftest_bounds_check(pg_ctx *ctx, void *stream);

/*
 * Wait for `stream` and return the device status word: PG_OK; PG_ERR_NUMERIC (a norm
 * was not finite); PG_ERR_TIMEOUT (a bounded device-side wait gave up: an mbarrier or
 * the grid barrier of pg_rounds); PG_ERR_BOUNDS (bounds-checked build only: a kernel
 * computed an address outside its section and skipped the access); PG_ERR_STATE (any other bit); PG_ERR_CUDA if the copy
 * or the wait failed.  The bits are sticky.  After PG_ERR_TIMEOUT a kernel has left in
 * the middle of a step, so X, Q and the cached products no longer belong together: the
 * context is marked failed, and pg_round, pg_round_sgd, pg_rounds and pg_set_round
 * return PG_ERR_STATE from then on (reading parameters still works; create a new
 * context to go on).  pg_read_params reports the same way.
 */
PG_API int pg_device_status(pg_ctx *ctx, void *stream);

/*
 * Edge list and weights of round `round` (Assumption A4's graph and W): writes
 * up to pg_max_edges() pairs (i<j, sorted) to edges_out (host, 2 ints per edge)
 * and their weights to w_out (host, may be NULL); *n_edges_out = count.
 */
PG_API int pg_get_schedule(pg_ctx *ctx, int64_t round, int32_t *edges_out, float *w_out, int32_t *n_edges_out);

/* Upper bound on the number of edges in any round of this context. */
PG_API int pg_max_edges(pg_ctx *ctx, int32_t *max_edges_out);

/*
 * Read / overwrite the stored right factor of the unordered pair {i, j} for
 * one layer (Algorithm 2's v_ij): host buffer of cols*rank floats, column k at
 * [k*cols, (k+1)*cols).  Synchronous with respect to `stream`.
 */
PG_API int pg_read_q(pg_ctx *ctx, int32_t i, int32_t j, int32_t layer, float *host_dst, void *stream);
PG_API int pg_write_q(pg_ctx *ctx, int32_t i, int32_t j, int32_t layer, const float *host_src, void *stream);

/* Round counter (the index of the next round): read it, or set it when
 * restoring a checkpoint {all X, all Q, round}.  Setting it first applies a
 * correction still pending from the last round (see pg_round), enqueued on
 * `stream`: pass the stream the rounds ran on, so that the correction is ordered
 * after them.  Does not wait. */
PG_API int pg_get_round(pg_ctx *ctx, int64_t *round_out);
PG_API int pg_set_round(pg_ctx *ctx, int64_t round, void *stream);

/*
 * Context-free, host-only view of the schedule builder: the edge list (i<j,
 * sorted) and weights that a context with this topology, mixing matrix and seed
 * uses in round `round` (Assumption A4; for PG_MATCHING a Fisher-Yates shuffle
 * of 0..N-1 whose draw at position k, from N-1 down to 1, is the low 64 bits of
 * Philox4x32-10 at counter (k, round_lo, round_hi, 0xFFFFFFFF) modulo k+1, with
 * consecutive entries paired).  edges_out: host, room for `capacity` pairs;
 * w_out: host, `capacity` floats, may be NULL.  PG_ERR_INVALID if the topology
 * or matrix is invalid or `capacity` is too small.  Touches no GPU.
 */
PG_API int pg_build_schedule(const pg_topology *topo, const float *W_host, uint64_t seed, int64_t round,
                             int32_t *edges_out, float *w_out, int32_t capacity, int32_t *n_edges_out);

/*
 * Host-only: column `col` of the standard-normal vector that pair (i<j) starts
 * with for layer `layer` (Algorithm 2, initialisation), m floats to host_dst.
 * This is what pg_create stores; exposed so the seeding can be checked without
 * a GPU.
 */
PG_API int pg_initial_vector(uint64_t seed, int32_t i, int32_t j, int32_t layer, int32_t col, int32_t m,
                             float *host_dst);

/*
 * Per-kernel device timing (measurement aid; the paper has no counterpart).
 * While enabled, pg_round brackets every kernel it launches with a pair of CUDA
 * events on the caller's stream.  pg_timing_read waits for the recorded events,
 * adds up, per kernel kind, the elapsed milliseconds, the launch counts and the
 * algorithmic bytes of those launches (4 B per parameter of the layers the
 * launch covers for every time it must read or write X once; 0 for the edge
 * steps, which touch vectors only) into ms_out / launches_out / bytes_out (host,
 * PG_KERNEL_KINDS entries each, indexed by the PG_KERNEL_* constants) and
 * forgets them.
 */
enum {
    PG_KERNEL_FORWARD = 0,         /* X q for all incident edges (first round only)     */
    PG_KERNEL_EDGE_LEFT = 1,       /* difference of the two ends, orthonormalisation    */
    PG_KERNEL_TRANSPOSED = 2,      /* X^T p-hat                                          */
    PG_KERNEL_EDGE_RIGHT = 3,      /* difference of the two ends, new stored vector      */
    PG_KERNEL_UPDATE_FORWARD = 4,  /* rank-r update of X fused with the next X q         */
    PG_KERNEL_PAIR_SWEEP = 5,      /* degree <= 2: pending update + X q + X^T p from one read */
    PG_KERNEL_PAIR_EDGE = 6,       /* its scalar edge step                               */
    PG_KERNEL_UPDATE_ONLY = 7,     /* applies a pending update before X is read or written */
    PG_KERNEL_KINDS = 8
};
PG_API int pg_timing_enable(pg_ctx *ctx, int32_t on);
/*
 * Algorithmic bytes of X that one steady-state round of this context moves (measurement
 * aid): per power step and parameter 8 B on layers the pair sweep takes (read once, written
 * once), 12 B on the three sweeps (read for the transposed product, read and written by the
 * update whose read doubles as the next forward product); 8 B per iteration in half-step
 * mode, 12 B per step with random projections.  *pair_fraction_out (may be NULL): share of
 * the parameters on the pair sweep.  Vectors and partial sums (under 1 %) are not counted.
 */
PG_API int pg_round_bytes(pg_ctx *ctx, double *bytes_out, double *pair_fraction_out);

PG_API int pg_timing_read(pg_ctx *ctx, double *ms_out, int64_t *launches_out, double *bytes_out);

/*
 * z = X^T p for one matrix, with no allocation of any kind (the paper has no
 * counterpart: this is a service entry point for callers that cannot allocate).
 *
 * Who needs it: code that runs where device memory cannot be obtained - inside
 * an allocator or memory-pool callback, in a process whose memory budget was
 * fixed at start-up, or on a latency path where cudaMalloc's implicit device
 * synchronisation would stall other streams.  Such callers cannot size and pass
 * the workspace that pg_create wants, so here the row-tile partial sums of the
 * transposed sweep live in a fixed array inside the library
 * (PG_NOALLOC_MAX_PARTIALS floats = 4 MiB, resident on every GPU that loads the
 * library until the process exits).  The call uses no cudaMalloc, cudaFree or
 * allocating library routine; the context-free call needs no pg_ctx.
 *
 *   X_dev   device, rows x cols fp32, row-major with leading dimension ld >= cols
 *           (floats).  16-byte rows (X_dev 16-byte aligned, cols and ld multiples
 *           of 4) take the vector path; anything else a scalar path, same result.
 *   p_dev   device, rows floats.        z_dev   device, cols floats (output).
 *   All three on the current device.  Asynchronous on `stream`.
 *
 * Limit: ceil(rows/256) * (cols rounded up to 4) <= PG_NOALLOC_MAX_PARTIALS,
 * e.g. 28000 x 650, 650 x 28000 or 8192 x 8192, and at most 65535 * 256 rows;
 * beyond either the call launches nothing, leaves z_dev alone and returns
 * PG_ERR_TOO_LARGE.
 * Set-up: the first call on each device looks up the device address of the
 * array (cudaGetSymbolAddress, once per device, with that device current); make
 * that first call outside any stream capture.
 * Sharing: all calls on a device use the same array, which keeps whatever the
 * last call left there.  Every cell a call reads it has written itself, so no
 * clearing is needed, but two calls that overlap on the GPU (different streams
 * or threads) race on the array: serialise them.
 */
#define PG_NOALLOC_MAX_PARTIALS (1 << 20)
PG_API int pg_transposed_product_noalloc(const float *X_dev, int32_t rows, int32_t cols, int64_t ld,
                                         const float *p_dev, float *z_dev, void *stream);

/*
 * Communication volume of Algorithm 2: what the two ends of an edge would send
 * each other if they sat on different machines (here the exchange is a read of
 * device buffers).  In iteration k (the algorithm's counter, from 1) each end
 * sends its product with the shared unit vector to the other end: rank * rows
 * floats of every tensor when k is odd (p = X v-hat), rank * cols when k is even
 * (the transposed iteration).  This is the count behind the per-tensor
 * "compression" column of the paper's parameter tables (Appendix "Network
 * architectures": rows * cols over (rows + cols) / 2 per iteration, "115/r x" for
 * 64 x 576) and behind the bytes-per-epoch columns of its result tables.
 *   pg_comm_floats        host only, no context: floats ONE end of ONE edge sends
 *                         over `iterations` iterations starting at counter
 *                         `first_iteration` >= 1, summed over the layers, to
 *                         *floats_out; *dense_out (may be NULL) gets rows * cols
 *                         summed over the layers, what one uncompressed exchange
 *                         (D-PSGD, Eq. 1) sends.
 *   pg_comm_floats_round  floats ALL workers of the context send in round `round`
 *                         (both ends of every edge of that round's graph).  A power
 *                         step is an odd and an even iteration; in half-step mode
 *                         the round's `power_steps` iterations continue the count
 *                         of the rounds before it; the random projections send the
 *                         product only (rank * rows for PG_RANDOM_RIGHT, rank * cols
 *                         for PG_RANDOM_LEFT per step; the directions are drawn
 *                         from the shared seed at both ends).
 * PG_ERR_INVALID for bad arguments.  Touches no GPU.
 */
PG_API int pg_comm_floats(const pg_layer_shape *shapes, int32_t n_layers, int32_t rank, int64_t first_iteration,
                          int64_t iterations, int64_t *floats_out, int64_t *dense_out);
PG_API int pg_comm_floats_round(pg_ctx *ctx, int64_t round, int64_t *floats_out, int64_t *dense_out);

/* Number of kernels this context has launched so far. */
PG_API int pg_kernel_launches(pg_ctx *ctx, int64_t *count_out);

/* Static string for a status code. */
PG_API const char *pg_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* POWERGOSSIP_H_ */
