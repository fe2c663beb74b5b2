/*
 * gcn_admm.h -- C ABI of the community-based ADMM trainer for graph convolutional networks
 * (single GPU, sm_100a).
 *
 * The calls follow the paper's statement of the problem: Algorithm 1 requires Y, Z_0, nu and
 * rho and returns Z_{l,m} and W_l; Problem 1 fixes the network (A~ = (D+I)^-1/2 (A+I) (D+I)^-1/2,
 * layer widths C_0..C_L, Z_l = f_l(A~ Z_{l-1} W_l)); Section 2 fixes the community split.
 *
 * General rules
 *  - Every function returns GCN_ADMM_OK (0) or a negative error code; no exception, abort or
 *    exit crosses this boundary.  After an error the handle stays valid for
 *    gcn_admm_last_error() and gcn_admm_destroy().
 *  - Pointers are plain host pointers unless a parameter says "host or device": those are
 *    classified with cudaPointerGetAttributes and copied accordingly.
 *  - All inputs are copied during gcn_admm_create(); the caller may free them afterwards.
 *    All outputs are caller-allocated and written in the caller's (original) node order; the
 *    community reordering is internal.
 *  - Matrices cross the boundary dense and row-major without padding.
 *  - A handle is not thread-safe; distinct handles are independent.  All device work of a
 *    handle is enqueued on the stream given at creation; calls return after that work has
 *    been enqueued, except where an output is a host buffer (then the call synchronises).
 *  - There is no CPU fallback: every call fails with GCN_ADMM_ERR_CUDA when no usable CUDA
 *    device is present.
 */
#ifndef GCN_ADMM_H
#define GCN_ADMM_H

#ifdef __cplusplus
extern "C" {
#endif

typedef struct gcn_admm gcn_admm; /* opaque, owned by the library */

enum {
  GCN_ADMM_OK = 0,
  GCN_ADMM_ERR_ARG = -1,       /* NULL pointer, non-positive size, unknown selector */
  GCN_ADMM_ERR_GRAPH = -2,     /* CSR not monotone / column out of range / unsorted or duplicate
                                  columns / not symmetric / more than 2^31-1 stored entries */
  GCN_ADMM_ERR_COMMUNITY = -3, /* community id outside 0..M-1, or an empty community */
  GCN_ADMM_ERR_WIDTHS = -4,    /* a width < 1, fewer than 1 layer, C_L > 128, label >= C_L, a width C_l above 1024 for some l >= 2,
                                  or n x (C_l rounded up to 4) of 2^34 elements or more for some layer l >= 1 */
  GCN_ADMM_ERR_ALLOC = -5,     /* host or device allocation failed */
  GCN_ADMM_ERR_CUDA = -6,      /* any CUDA runtime failure, including "no device" */
  GCN_ADMM_ERR_NONFINITE = -7  /* a NaN or infinity reached a step-size decision */
};

/* Parameters.  nu: penalty of the relaxed hidden-layer constraints (Problem 2).  rho: penalty of
 * the augmented Lagrangian (Eq. 1).  The remaining fields fix what the paper leaves open:
 *  tau0, theta0    initial step parameters of the quadratic approximations (Section 3.1, Eq. 8)
 *  bt_shrink       a search starts from max(previous * bt_shrink, 1e-12)
 *  bt_growth       and multiplies by bt_growth (> 1) until the condition of Section 3.1 / Eq. 9,
 *                  in the form f(x - g/t) <= f(x) - ||g||^2/(2t), holds
 *  bt_max_trials   at most this many trials (1..64); an exhausted block is left unchanged
 *  fista_iters     iterations of FISTA on the training rows of Eq. 7 (constant step
 *                  1/(loss_scale/2 + rho), t_1 = 1, warm start, no early exit)
 *  loss_scale      R = loss_scale * sum over training rows of the softmax cross-entropy
 *  dual_mode       0: Eq. 3 as printed (Z_L^k, Z_{L-1}^k, W_L^{k+1}); 1: the k+1 iterates
 *  tensor_cores    1: dense products with 8 <= K <= 2048 and at least 512 rows run on the tensor cores as an
 *                  error-compensated TF32 product (three passes, fp32 accumulation, relative error of a few
 *                  1e-7 of sum |a||b|); products of 16384 rows or more first split the weight operand once
 *                  into the staged layout and fetch it with bulk copies (smaller ones re-split it per row
 *                  tile, which is cheaper than another launch), and with at most 128 output columns they also
 *                  fetch the tiles of the row operand by tensor copies (products with 129 to 256 output columns
 *                  and K <= 128 run in that form as two groups of 128 columns); 2: the same kernels, pre-split
 *                  at every size; 0: fp32 FMA kernels everywhere
 *  use_graph       1: gcn_admm_step records one pass as a CUDA graph on first use and replays it (only when
 *                  the handle's stream is not the default stream and profiling is off); 2: the same, but
 *                  only for problems small enough for launch gaps to show (N x widest layer < 2^27);
 *                  0: plain launches
 *  schedule        0: Algorithm 1 (every W_l, then every Z_{l,m}, then U; Jacobi inside a pass);
 *                  1: the serial schedule of Section 4.1 (W_1, Z_1, .., W_L, Z_L, U one after the other,
 *                  each block reading the latest value of all others; the dual uses the new iterates)
 *  long_row        rows of A + I with more stored entries than this are cut into work items of at most
 *                  this many entries, each walked by a warp of its own, and the items' sums are added up
 *                  in a fixed order afterwards (the paper's graphs have power-law degrees; a hub row
 *                  walked by one warp would outlast the rest of the launch).  Same sums up to fp32
 *                  rounding order.  0: the default, 256; a value above the longest row switches it off
 *  w_init          L host pointers to row-major C_{l-1} x C_l matrices, or NULL: then every W_l is drawn
 *                  Glorot-uniform, entry (i, j) of W_l = a (2 u - 1) with a = sqrt(6 / (C_{l-1} + C_l)) and
 *                  u = (top 24 bits of splitmix64(seed + 2^32 l + i C_l + j)) / 2^24, where splitmix64(x) is
 *                  the output function of that generator applied to the state x + 0x9E3779B97F4A7C15 (the
 *                  paper does not say how W starts)
 *  seed            seed of that draw; ignored when w_init is given
 *  device          CUDA device ordinal;  stream: a cudaStream_t owned by the caller (NULL = the
 *                  default stream) */
typedef struct {
  float nu, rho;
  float tau0, theta0;
  float bt_growth, bt_shrink;
  int bt_max_trials;
  int fista_iters;
  float loss_scale;
  int dual_mode;
  int tensor_cores;
  int use_graph;
  int schedule;
  int long_row;
  unsigned long long seed;
  const float* const* w_init;
  int device;
  void* stream;
} gcn_admm_params;

/* Fills *p with the defaults: nu = rho = 1e-3, tau0 = theta0 = 1, growth 2, shrink 0.5,
 * 40 trials, 30 FISTA iterations, loss_scale 1, dual_mode 0, tensor_cores 1, use_graph 2, schedule 0, long_row 0, seed 0, w_init NULL,
 * device 0, stream NULL. */
void gcn_admm_default_params(gcn_admm_params* p);

/* Builds the problem of Algorithm 1 (its REQUIRE line) on the device.
 *  n                 number of nodes N
 *  row_ptr, col_idx  CSR pattern of the undirected, unweighted adjacency A (host or device):
 *                    row_ptr[n+1] ascending from 0, columns strictly ascending inside a row,
 *                    symmetric.  Diagonal entries are dropped; the identity of A~ is added here.
 *                    Range and order are checked entry by entry; symmetry by comparing the number
 *                    and two 64-bit fingerprints of the entries above and below the diagonal.
 *  X                 Z_0, n x C_0 (host or device)
 *  y                 class id per node, 0..C_L-1 (only rows with train_mask != 0 are read as labels)
 *  train_mask        n bytes, non-zero = the node's loss term is part of R
 *  n_layers, widths  L and C_0..C_L (widths has n_layers+1 entries)
 *  n_comm, community M and the community id 0..M-1 of every node (Section 2); every community
 *                    must be non-empty
 * Work done here (none of it is part of an ADMM iteration): community reordering (nodes sorted by
 * (community, original id)), A+I in that order with ascending columns, (D+I)^-1/2, the row-segment
 * table that splits each row by the community of its columns (the blocks A~_{m,r} of Section 2),
 * P_1 = A~ Z_0, and the initial state: W = w_init, Z from the forward pass of Problem 1, U = 0,
 * tau_l = tau0, theta_{l,m} = theta0.
 * On success *out receives the handle. */
int gcn_admm_create(gcn_admm** out, long long n, const long long* row_ptr, const int* col_idx,
                    const float* X, const int* y, const unsigned char* train_mask, int n_layers,
                    const int* widths, const gcn_admm_params* p, int n_comm, const int* community);

/* Runs n_iters passes of Algorithm 1: every W_l (Section 3.1), then every Z_{l,m} (Appendix A,
 * Eq. 5-10; Eq. 7 for l = L), then U (Eq. 3).  Updates inside a pass are Jacobi: each reads the
 * previous pass's Z and U and this pass's W.  Device work only; returns after enqueueing. */
int gcn_admm_step(gcn_admm* h, int n_iters);

/* out[0] = L_rho of Eq. 1, out[1] = R, out[2] = sum over l<L of (nu/2)||Z_l - f_l(A~ Z_{l-1} W_l)||^2,
 * out[3] = <U, r>, out[4] = (rho/2)||r||^2 with r = Z_L - A~ Z_{L-1} W_L, out[5] = training accuracy of
 * gcn_admm_predict.  Host pointer; synchronises. */
int gcn_admm_objective(gcn_admm* h, double out[6]);

/* Copies W_layer (1-based, C_{layer-1} x C_layer, row-major) to the host buffer out. */
int gcn_admm_weights(gcn_admm* h, int layer, float* out);

/* Forward pass of Problem 1 with the current W (not the auxiliary Z).  logits: n x C_L, labels: n
 * (row argmax, ties to the lowest class).  Either may be NULL.  Host pointers, original order. */
int gcn_admm_predict(gcn_admm* h, float* logits, int* labels);

void gcn_admm_destroy(gcn_admm* h);

/* Text of the last error of this handle (or of the last failed create when h is NULL). */
const char* gcn_admm_last_error(const gcn_admm* h);

/* ---- propagation alone (the product A~ X of Problem 1) ---------------------------------------
 * out = A~ x for an n x width matrix x in the original node order (host or device, both the same
 * kind; out may not alias x; width at most 2^24).  Uses the handle's graph only; the ADMM state is untouched. */
int gcn_admm_propagate(gcn_admm* h, const float* x, int width, float* out);

/* ---- the dense product alone (the contraction with W_l in Problem 1 and in every block update) ----
 * C = A B for device pointers A (m x k), B (k x n), C (m x n), dense row-major; tensor_cores selects
 * the kernel as the parameter of the same name does.  Allocates staging copies; synchronises. */
int gcn_admm_dense_product(gcn_admm* h, const float* A, const float* B, float* C, long long m, int n, int k,
                           int tensor_cores);

/* C = A^T B for device pointers A (rows x ka), B (rows x nb), C (ka x nb): the reduction over the node
 * dimension that forms the weight gradient P^T R (Section 3.1).  ka x (nb rounded up to 4) must fit
 * the handle's partial-sum scratch (it does for every layer shape of the handle).  Synchronises. */
int gcn_admm_dense_product_tn(gcn_admm* h, const float* A, const float* B, float* C, long long rows, int ka, int nb,
                              int tensor_cores);

/* ---- propagation for callers that cannot allocate ---------------------------------------------
 * (No counterpart in the paper: this is a packaging variant of gcn_admm_propagate.)
 * Same result as gcn_admm_propagate, for code that is not allowed to reserve device memory when it
 * calls: a real-time loop whose memory budget was fixed at start-up, a plug-in running inside
 * someone else's memory pool, a section between begin and end of a stream capture where cudaMalloc is
 * illegal.  gcn_admm_propagate stages x and the result in two padded matrices that it allocates and
 * frees on every call; this variant keeps those two matrices in an array compiled into the library
 * (32 MiB of device memory on every GPU that loads the library, held until the process ends), and
 * calls neither cudaMalloc nor cudaFree nor any allocating routine.
 *  - x and out are DEVICE pointers to n x width floats, original node order; out may not alias x.
 *  - its launches are counted by gcn_admm_launches but never timed by gcn_admm_profile (event
 *    creation reserves memory), whether profiling is on or off.
 *  - limit: n * (width rounded up to a multiple of 4) <= 4,194,304; larger sizes are refused with
 *    GCN_ADMM_ERR_ARG and a message naming the limit.
 *  - the first call on a device looks up the device address of the array (one runtime query, no
 *    allocation); make that first call before any stream capture begins.
 *  - the work is enqueued on the handle's stream and the call returns without synchronising.
 *  - all calls, from every handle, share the one array, which keeps whatever the last call left in
 *    it; each call overwrites all it later reads, so nothing needs clearing, but two calls whose
 *    kernels overlap on the GPU (different streams, different handles) race on it: serialise them. */
int gcn_admm_propagate_static(gcn_admm* h, const float* x, int width, float* out);

/* ---- index tables (Section 2; Appendix A first paragraph) ------------------------------------
 * Returns a pointer to a host int array owned by the handle (valid until the next call of this
 * function with the same selector, or destroy) and its length.  New ids = position after sorting
 * nodes by (community, original id).  comm is used by the per-community selectors only.
 *  GCN_ADMM_IX_PERM        new id -> original id            [n]
 *  GCN_ADMM_IX_INV_PERM    original id -> new id            [n]
 *  GCN_ADMM_IX_COMM_PTR    V_m = new ids comm_ptr[m]..comm_ptr[m+1]-1   [M+1]
 *  GCN_ADMM_IX_NBR         N_m, ascending                    (per community)
 *  GCN_ADMM_IX_HALO1       new ids outside V_m adjacent to V_m, ascending (first-order rows)
 *  GCN_ADMM_IX_HALO2       new ids outside V_m and HALO1 adjacent to HALO1, ascending (second order)
 *  GCN_ADMM_IX_CSR_ROW_PTR, GCN_ADMM_IX_CSR_COL   pattern of A+I in new ids  [n+1], [nnz]
 *  GCN_ADMM_IX_SEG_ROW_PTR [n+1], GCN_ADMM_IX_SEG_COMM [S], GCN_ADMM_IX_SEG_BEGIN [S+1]
 *       row i owns segments seg_row_ptr[i]..seg_row_ptr[i+1]-1; segment s covers positions
 *       seg_begin[s]..seg_begin[s+1]-1 of csr_col, whose columns all lie in community seg_comm[s]. */
enum {
  GCN_ADMM_IX_PERM = 0, GCN_ADMM_IX_INV_PERM, GCN_ADMM_IX_COMM_PTR, GCN_ADMM_IX_NBR,
  GCN_ADMM_IX_HALO1, GCN_ADMM_IX_HALO2, GCN_ADMM_IX_CSR_ROW_PTR, GCN_ADMM_IX_CSR_COL,
  GCN_ADMM_IX_SEG_ROW_PTR, GCN_ADMM_IX_SEG_COMM, GCN_ADMM_IX_SEG_BEGIN
};
int gcn_admm_index(gcn_admm* h, int which, int comm, const int** data, long long* len);

/* ---- plan for several GPUs (host only; Section 2: a community per agent; Appendix A, Eq. 4: the first-order
 * messages p and the second-order messages s) ----------------------------------------------------
 * This library runs a handle on one GPU and issues no collective.  For a caller that spreads the communities
 * over n_ranks GPUs it plans the split: rank r owns a contiguous range of communities (hence of rows in the
 * community order of gcn_admm_index), balanced by stored entries of A + I, and for every ordered pair
 * (receiver, sender) the rows of the sender that the receiver depends on.
 *  GCN_ADMM_SHARD_RANGES        [2 (n_ranks + 1)]: first community of every rank and one past the last,
 *                               then first row of every rank and one past the last (receiver, sender ignored)
 *  GCN_ADMM_SHARD_FIRST_ORDER   rows of `sender` adjacent to a row of `receiver`: the rows the receiver needs a
 *                               copy of before a pass (Z_{l-1} for its propagation; H_{l+1}, Z_{l+1}, U for the
 *                               gradient and the step-size search of its Z_{l,m} blocks).  The send list of
 *                               (sender -> receiver) is this same list.
 *  GCN_ADMM_SHARD_SECOND_ORDER  rows of `sender` that are neither the receiver's own nor first-order rows but
 *                               adjacent to one: their Z_l reaches the receiver only through a neighbour's
 *                               aggregate (the paper's second-order message); nothing is sent for them when
 *                               owners compute H_{l+1} for their own rows.
 * Lists are ascending new ids, owned by the handle, valid until the next call with another n_ranks or destroy.
 * n_ranks must lie between 1 and the number of communities. */
enum { GCN_ADMM_SHARD_RANGES = 0, GCN_ADMM_SHARD_FIRST_ORDER = 1, GCN_ADMM_SHARD_SECOND_ORDER = 2 };
int gcn_admm_shard_plan(gcn_admm* h, int n_ranks, int which, int receiver, int sender, const int** data,
                        long long* len);

/* The propagation A~ x (Problem 1; Section 2: every agent forms the rows of its own communities from its rows
 * and its neighbours' first-order rows) carried out the way the n_ranks ranks of that plan would, one rank
 * after the other on this handle's one device: for each rank, the rows it owns and, behind them, copies of
 * the first-order rows of every sender are gathered into a local matrix (on several devices that second
 * part is what the receives from the rows' owners fill), the rank's rows of A + I are renumbered to
 * positions in that local matrix, and the propagation kernel runs on those local tables alone and writes
 * the rank's rows of the result.  Entry order inside a row is kept, so a row is summed in the same order
 * as by gcn_admm_propagate (rows longer than `long_row` excepted: there the unsharded call adds partial
 * sums of pieces).  x, out: n x width, original node order, both host or both device; staged_rows (may be
 * NULL) receives the number of copied first-order rows summed over the ranks.  Allocates per rank and
 * synchronises; a check of the plan on the device, not a fast path.  No collective is issued. */
int gcn_admm_propagate_sharded(gcn_admm* h, int n_ranks, const float* x, int width, float* out,
                               long long* staged_rows);

/* ---- state access (checkpointing and single-block tests) -------------------------------------
 * Host buffers, dense row-major, original node order.
 *  GCN_ADMM_ST_W      layer 1..L   float  C_{l-1} x C_l
 *  GCN_ADMM_ST_Z      layer 1..L   float  n x C_l
 *  GCN_ADMM_ST_U      layer ignored float n x C_L
 *  GCN_ADMM_ST_TAU    layer 1..L   double [1]
 *  GCN_ADMM_ST_THETA  layer 1..L-1 double [M]
 *  GCN_ADMM_ST_PIPELINE_FLAG  layer ignored, int [1]: non-zero once a tensor-core product has given up one of
 *                     its bounded waits.  The next call that synchronises (objective, decisions, dense
 *                     products) then returns GCN_ADMM_ERR_CUDA once and clears the flag; the handle stays
 *                     usable.  Writable so that this path can be exercised without a failing kernel. */
enum { GCN_ADMM_ST_W = 0, GCN_ADMM_ST_Z, GCN_ADMM_ST_U, GCN_ADMM_ST_TAU, GCN_ADMM_ST_THETA, GCN_ADMM_ST_PIPELINE_FLAG };
int gcn_admm_get_state(gcn_admm* h, int which, int layer, void* out);
int gcn_admm_set_state(gcn_admm* h, int which, int layer, const void* in);

/* Runs one block family of Algorithm 1 on the current state and nothing else:
 *  GCN_ADMM_PHASE_W, layer l    W_l update (Section 3.1)
 *  GCN_ADMM_PHASE_Z, layer l<L  every Z_{l,m}, m = 1..M (Eq. 5/6, 8-10), with the stored W as W^{k+1}
 *  GCN_ADMM_PHASE_Z, layer L    Z_L (Eq. 7)
 *  GCN_ADMM_PHASE_U             U + rho (Z_L - A~ Z_{L-1} W_L) on the stored iterates (Eq. 3) */
enum { GCN_ADMM_PHASE_W = 0, GCN_ADMM_PHASE_Z = 1, GCN_ADMM_PHASE_U = 2 };
int gcn_admm_step_block(gcn_admm* h, int phase, int layer);

/* Step-size decisions of the most recent gcn_admm_step / gcn_admm_step_block call, oldest pass first
 * (at most the last 256 passes are kept).  trial: accepted trial index j (t = start * growth^j),
 * -1 = skipped (||g||^2 <= 1e-24 ||x||^2), -2 = exhausted, -3 = block not run in that pass.
 * q = (f(x) - f(x+)) / (||g||^2/(2t)) at the accepted trial (the condition is q >= 1).
 *  trial_w, q_w   [passes x L]           index pass*L + (l-1)
 *  trial_z, q_z   [passes x (L-1) x M]   index (pass*(L-1) + (l-1))*M + m
 * Any pointer may be NULL.  *n_passes receives the number of passes logged; the arrays must hold
 * max_passes passes and at most that many are written.  Synchronises. */
int gcn_admm_decisions(gcn_admm* h, int max_passes, int* n_passes, int* trial_w, double* q_w,
                       int* trial_z, double* q_z);

/* ---- accounting and timing ---------------------------------------------------------------------
 * gcn_admm_launches: number of kernels this handle has launched since it was created.
 * gcn_admm_profile(h, 1) clears the per-kernel table and starts bracketing every launch with CUDA
 * events on the handle's stream (this costs a little time, so leave it off when timing a whole step);
 * gcn_admm_profile(h, 0) stops.  gcn_admm_profile_read synchronises and returns one entry per kernel
 * kind ("spmm@256" = propagation at leading dimension 256, "gemm_nn@256x47" = K x N of the product, ...):
 * launches, summed device time in ms, and the algorithmic bytes and flops of the work those launches
 * did (what the operation must move / compute, not what the hardware moved).  names: max_entries x 48
 * chars.  Any output array may be NULL. */
int gcn_admm_launches(gcn_admm* h, long long* count);
int gcn_admm_profile(gcn_admm* h, int enable);
int gcn_admm_profile_read(gcn_admm* h, int max_entries, int* n_entries, char* names, long long* launches,
                          double* ms, double* bytes, double* flops);

#ifdef __cplusplus
}
#endif
#endif /* GCN_ADMM_H */
