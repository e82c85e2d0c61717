/*
 * gad.h - C boundary of the B200 (sm_100a) library for one training epoch of GAD
 * (Graph-Augmentation-based Distributed GCN, arXiv 2110.02987).
 *
 * What the library computes: K replicas of an L-layer GCN, one per augmented subgraph g'_k produced by
 * GAD-Partition, all batched on one GPU.  One call of gad_train_epoch is one pass of Algorithm 2 with one
 * subgraph per processor: forward propagation, loss, backward propagation (Section 3.3), the variance-based
 * subgraph importance zeta (Section 3.4.1) and the weighted global consensus over the K parameter copies
 * (Section 3.4.2).  The partition and the replicated-node lists are inputs (they are GAD-Partition's output,
 * Section 3.2); the library does not compute them.
 *
 * Conventions
 *   - Every function returns an int status: GAD_OK (0) or a negative GAD_ERR_* code.  Nothing throws.
 *     gad_last_error(ctx) gives a NUL-terminated message that belongs to the context.
 *   - "host" pointers are ordinary CPU memory owned by the caller; they are only read (or written) during the
 *     call.  "device" pointers are CUDA device memory of the current device.
 *   - The library allocates no device memory: the caller passes one device workspace (size from
 *     gad_workspace_bytes) and a CUDA stream; both must outlive the context.  Work is ordered as if it all ran on
 *     that stream; the context also owns two streams of its own (one for the host-to-device copies of
 *     gad_set_inputs, one for small kernels of an epoch that run beside the main sequence), tied to the caller's
 *     stream by events.  A context is not thread-safe.
 *   - Matrices are row-major.  One replica's parameters are the P floats
 *       [ W_0 (F_0 x F_1), b_0 (F_1), W_1 (F_1 x F_2), b_1 (F_2), ... ],  P = sum_l (F_l F_{l+1} + F_{l+1}).
 *   - "store row": the K augmented subgraphs are kept as one block-diagonal matrix.  Subgraph k owns the rows
 *     sub_off[k] .. sub_off[k+1]-1: first its core nodes in the order given, then its replicated nodes in the
 *     order given.  N' = sub_off[K], nnz' = stored entries of all A~_k.
 */
#ifndef GAD_H
#define GAD_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define GAD_OK 0
#define GAD_ERR_ARG (-1)            /* NULL pointer, non-positive size, bad flag                           */
#define GAD_ERR_RANGE (-2)          /* node id, column, label or split value out of range                  */
#define GAD_ERR_UNSORTED (-3)       /* a pointer array (rowptr, core_ptr, halo_ptr) is not non-decreasing   */
#define GAD_ERR_DUPLICATE (-4)      /* a node listed twice inside one subgraph, or in two core sets         */
#define GAD_ERR_OOM (-5)            /* workspace too small, or host allocation failed                       */
#define GAD_ERR_NONFINITE (-6)      /* a loss came out NaN or infinite (reported, never trapped)            */
#define GAD_ERR_DEVICE_TIMEOUT (-7) /* a bounded device-side wait ran out                                   */
#define GAD_ERR_CUDA (-8)           /* a CUDA call failed; see gad_last_error                               */
#define GAD_ERR_UNSUPPORTED (-9)    /* a documented option that this library does not implement             */

typedef struct gad_ctx gad_ctx;

/* The whole graph G = (V, E) in CSR form, host memory.  Columns need not be sorted; parallel edges are summed;
 * w == NULL means unit weights.  An undirected graph lists every edge in both directions. */
typedef struct {
    int32_t n;
    int64_t nnz;
    const int64_t* rowptr; /* [n+1] */
    const int32_t* col;    /* [nnz] */
    const float* w;        /* [nnz] or NULL */
} gad_csr;

/* GAD-Partition's output (Definition 1 and Algorithm 1): for subgraph k the core nodes
 * core_nodes[core_ptr[k] .. core_ptr[k+1]) (disjoint between subgraphs; they need not cover V) and the
 * replicated nodes halo_nodes[halo_ptr[k] .. halo_ptr[k+1]) (not in the same subgraph's core set; a node may
 * be replicated into several subgraphs).  Host memory. */
typedef struct {
    int32_t K;
    const int64_t* core_ptr;   /* [K+1] */
    const int32_t* core_nodes;
    const int64_t* halo_ptr;   /* [K+1] */
    const int32_t* halo_nodes;
} gad_partition;

typedef struct {
    int32_t L;            /* number of GCN layers, >= 1                                                      */
    const int32_t* dims;  /* [L+1] host: F_0 (input features) ... F_L (classes)                              */
    float lr;             /* eta of the update equation (Section 3.3 / 3.4.2)                                 */
    float dropout;        /* probability of dropping a hidden unit after the ReLU, in [0,1); 0 = none         */
    uint64_t seed;        /* seed of the dropout mask and of the default initialisation                       */
    int32_t gemm_mode;    /* 0: fp32-accurate transform (SIMT, or tensor cores with every operand split in two);  *
                           * 1: reduced-precision operands with fp32 accumulation: one TF32 pass on the tensor      *
                           *    cores, and the aggregation gathers a bfloat16 copy of its operand (tolerance 5e-2)  */
    int32_t zeta_mode;    /* 0: aggregate distance term; 1: literal pairwise form, O(n'^2 F_0) per subgraph, the  *
                           * squared distances from a Gram matrix on the tensor cores (any subgraph size; with   *
                           * flag bit 0 or 4 from the differences on the FP32 ALUs, GAD_ERR_UNSUPPORTED when a    *
                           * subgraph has more than 32768 rows); 2: the aggregate                               *
                           * term with the sum over layers of the variance equation (Section 3.4.1) kept: the  *
                           * squared distances are summed over the inputs H^(0) .. H^(L-1) of all layers, as   *
                           * the most recent forward pass left them, so zeta changes from epoch to epoch        */
    float beta;           /* beta of the importance weight (Section 3.4.1); the paper uses 1                  */
    int32_t weighted;     /* 1: weighted global consensus (Section 3.4.2); 0: plain average (Definition 3)    */
    int32_t flags;        /* bit 0: force the SIMT transform even where a tensor-core kernel exists;
                             bit 1: layer 0 aggregates first and keeps A~ H^(0) from one epoch to the next (it
                             changes only with the features, i.e. with gad_set_inputs);
                             bit 2: the backward pass of a layer of at most 16 output columns also goes through the
                             tensor-core transforms instead of the streaming FP32 kernel written for it (for
                             comparison);
                             bit 3: never replay an epoch as a CUDA graph (see gad_train_epoch);
                             bit 4: zeta_mode 1 on the FP32 ALUs (difference form) instead of the tensor cores;
                             bit 5: layers l >= 1 always transform before they aggregate (by default a layer whose
                             input is narrower than its output aggregates first, sigma((A~ H^(l)) W + b): the same
                             product in the other order, with both of its SpMMs at the narrower width);
                             bit 6: the last layer's backward aggregation reads every row (by default it runs over a
                             copy of the transposed store without the entries that read a row carrying no loss - a
                             replicated node, or a core node outside the training split, where d loss / d logits is
                             zero (the loss of Section 3.3 is taken over the subgraph's own training nodes): the same
                             sums without their zero terms; the copy costs up to 8 bytes per stored entry)           */
} gad_config;

/* Bytes of device workspace gad_create needs for these inputs.  Host-only; touches no GPU. */
int gad_workspace_bytes(const gad_csr* g, const gad_partition* part, const gad_config* cfg, size_t* bytes);

/* Builds the block-diagonal store of the augmented subgraphs g'_k = (v_k + v'_k, e_k + e'_k) (Algorithm 1,
 * last step): every edge of G with both endpoints in v_k + v'_k, a unit self-loop added where a node has none,
 * A~_k = D~^-1/2 (A'_k + I) D~^-1/2 with the degrees taken inside g'_k (the A~ of the forward equation,
 * Section 3.3); uploads it with the features, labels and split, and makes K identical parameter copies
 * (Algorithm 2: every processor starts from the same model).
 *   X            host [n x dims[0]]
 *   labels       host [n], values in 0 .. dims[L]-1
 *   split        host [n]: 0 train, 1 validation, 2 test.  Only core nodes with split 0 carry loss.
 *   init_params  host [P], or NULL for seeded Glorot-uniform W and zero b
 *   workspace    device, 256-byte aligned, at least gad_workspace_bytes; owned by the caller
 *   stream       a cudaStream_t (NULL = the default stream)
 * Synchronises the stream before returning.  On error *out is NULL. */
int gad_create(gad_ctx** out, const gad_csr* g, const gad_partition* part, const float* X, const int32_t* labels,
               const uint8_t* split, const gad_config* cfg, const float* init_params, void* workspace,
               size_t workspace_bytes, void* stream);

/* The parameters gad_create starts from when init_params is NULL, host [P] in the layout above: W_l uniform in (-a, a)
 * with a = sqrt(6 / (F_l + F_{l+1})) (Glorot), drawn from a splitmix64 stream of `seed`; biases zero.  Host-only.  (The
 * paper does not say how its models are initialised.) */
int gad_default_params(int32_t L, const int32_t* dims, uint64_t seed, float* out);

/* One pass of Algorithm 2 (one subgraph per processor): for every replica k
 *   forward   H^(l+1) = sigma(A~_k (H^(l) W_k^(l)) + b_k^(l)), sigma = ReLU (identity on the last layer), with
 *             the optional dropout after the ReLU                          (Section 3.3, forward equations)
 *   loss      softmax cross-entropy, mean over the core training nodes     (Section 3.3, loss equation)
 *   backward  gradients of every W_k^(l), b_k^(l) through A~_k^T           (Section 3.3, gradient equation)
 *   update    theta_k <- theta_k - eta * grad_k                            (Section 3.3, update equation)
 * then zeta_k and the weighted consensus theta_k <- sum_j w_j theta_j      (Sections 3.4.1, 3.4.2).
 * loss_out: host [K+1] = the K subgraph losses, then sum_k |T_k| L_k / sum_k |T_k|, all evaluated before the
 * update; the call then waits for the stream.  loss_out == NULL: the epoch is only enqueued (no wait, no
 * copy); read the losses later with gad_get_loss.  Returns GAD_ERR_NONFINITE if a loss is NaN or infinite
 * (detected when the losses are read).
 * From the second call on the launches of an epoch are replayed as one CUDA graph (captured on the context's
 * stream, thread-local mode) when nothing in them changes from epoch to epoch: dropout == 0, flag bits 1 and 3 clear,
 * per-kernel timing off, and a stream that can be captured (any stream but the legacy default one).  Otherwise, while
 * the caller is capturing that stream itself, or if the capture fails, they are enqueued one by one; the results are
 * the same either way. */
int gad_train_epoch(gad_ctx* ctx, float* loss_out);

/* Losses of the most recent epoch, host [K+1]; waits for the stream. */
int gad_get_loss(gad_ctx* ctx, float* loss_out);

/* Inference forward (no dropout) of replica k on subgraph k.  logits_out: host [n x dims[L]] in graph-node
 * order, filled for core nodes; rows that no subgraph owns are zero.  (Section 3.3, forward equations.) */
int gad_forward(gad_ctx* ctx, float* logits_out);

/* Variance-based importance of every subgraph (Section 3.4.1) and the consensus weights (Section 3.4.2):
 *   p_i = deg_k(i) / sum_j deg_k(j)  (degree inside g'_k without the self-loop; uniform if there are no edges)
 *   S_k = sum_{i<j} p_i p_j,   D_k = sqrt( sum_{i<j} p_i p_j |x_i - x_j|^2 / S_k )  on the input features
 *   zeta_k = S_k / (D_k + beta),   w_k = zeta_k / sum_j zeta_j   (1/K when weighted == 0 or all zeta are 0)
 * zeta_out, w_out: host [K], either may be NULL. */
int gad_subgraph_weights(gad_ctx* ctx, float* zeta_out, float* w_out);

/* Weighted global consensus on its own: theta_k <- sum_j w_j theta_j for every k (Section 3.4.2; Definition 3
 * when weighted == 0).  Enqueued on the stream. */
int gad_consensus(gad_ctx* ctx);

/* ---- Algorithm 2 with the subgraphs spread over several contexts --------------------------------------------
 * Algorithm 2 assigns z subgraphs to each of n processors: the processors train one subgraph each at the same time,
 * take the weighted consensus (Section 3.4.2) and go on to their next subgraph until all have been traversed (last
 * paragraph of Section 3.3).  One context holds the subgraphs that train at the same time on ONE GPU.  Two uses:
 *   - several GPUs: every GPU holds a context with its share of the subgraphs; per step each runs
 *     gad_train_epoch_local and gad_consensus_partial, the buffers are added over the GPUs (one all-reduce of
 *     gad_consensus_floats floats) and every GPU calls gad_consensus_apply with the sum;
 *   - rounds (z > 1): one context per round; after a round's gad_train_epoch its model goes to the next round's
 *     context with gad_export_params + gad_consensus_apply.
 * All contexts must have the same layer sizes.  The buffers are device memory of gad_consensus_floats floats,
 * 16-byte aligned, owned by the caller, in the library's padded parameter layout (opaque; the same for every context
 * with the same layer sizes).  Everything is enqueued on the context's stream and nothing waits. */

/* gad_train_epoch without the update and the consensus: forward, loss, backward, zeta.  Parameters unchanged,
 * gradients ready for gad_consensus_partial.  loss_out as in gad_train_epoch (the last entry is the mean over THIS
 * context's training rows). */
int gad_train_epoch_local(gad_ctx* ctx, float* loss_out);

/* |T_k|: the core training nodes of every subgraph, host [K] (the weights with which the subgraph losses combine
 * into the loss of an epoch over several contexts). */
int gad_get_train_counts(const gad_ctx* ctx, int64_t* counts);

/* Floats in a consensus buffer. */
int gad_consensus_floats(const gad_ctx* ctx, int64_t* count);

/* This context's share of the weighted consensus (Section 3.4.2):
 *   dev_out = sum over this context's replicas k of  w_k (theta_k - eta grad_k),   w_k = zeta_k / zeta_total,
 * with zeta_total the sum of zeta over the subgraphs of ALL contexts (from gad_subgraph_weights of each); with
 * weighted == 0 (Definition 3) w_k = 1 / zeta_total and zeta_total is the number of subgraphs of all contexts.
 * with_step == 0 leaves out the "- eta grad_k" (a consensus of the parameters as they are; zeta is evaluated
 * first).  with_step != 0 uses the gradients and zeta of the last gad_train_epoch_local.  The parameters are not
 * changed. */
int gad_consensus_partial(gad_ctx* ctx, double zeta_total, int32_t with_step, float* dev_out);

/* theta_k <- dev_in for every replica k of this context (the finished consensus, or another context's model). */
int gad_consensus_apply(gad_ctx* ctx, const float* dev_in);

/* Replica k's parameters into a consensus buffer (device to device). */
int gad_export_params(gad_ctx* ctx, int32_t k, float* dev_out);

/* Parameter copy / gradient of replica k, host [P] in the layout above.  Gradients are those of the most recent
 * epoch (d L_k / d theta_k).  These calls wait for the stream. */
int gad_get_params(gad_ctx* ctx, int32_t k, float* out);
int gad_set_params(gad_ctx* ctx, int32_t k, const float* in);
int gad_get_grads(gad_ctx* ctx, int32_t k, float* out);
int gad_param_count(const gad_ctx* ctx, int64_t* P);

/* The store as built (for checking the bookkeeping): sizes, then the arrays, all host.
 *   rowptr int64 [N'+1], col int32 [nnz'] (store-row ids, ascending inside a row), val float [nnz'],
 *   sub_off int32 [K+1], gid int32 [N'] (graph node of each store row), deg int32 [N'] (local degree without
 *   the self-loop).  Any array pointer may be NULL. */
int gad_store_sizes(const gad_ctx* ctx, int64_t* n_prime, int64_t* nnz_prime);
int gad_get_store(gad_ctx* ctx, int64_t* rowptr, int32_t* col, float* val, int32_t* sub_off, int32_t* gid,
                  int32_t* deg);

/* Activation H^(l) of the most recent forward pass, l = 0 .. L (l = L: logits), host [N' x dims[l]] in store-row
 * order.  Waits for the stream. */
int gad_get_activation(gad_ctx* ctx, int32_t l, float* out);

/* Replaces the node features and/or labels (either may be NULL), host arrays of the shapes given to
 * gad_create.  The host-to-device copies go out on a second stream that the context owns, into one of two staging
 * buffers, so they may overlap an epoch already enqueued on the context's stream; the reordering into store rows
 * then runs on the context's stream, after the copy, and every later call sees the new inputs.  The caller's
 * buffers must stay valid until a call that waits (gad_synchronize, gad_get_loss, ...) has returned; pinned memory
 * makes the copy asynchronous.  Not part of the paper's algorithm: it is how a training loop streams inputs. */
int gad_set_inputs(gad_ctx* ctx, const float* X, const int32_t* labels);

/* For a loop that never waits inside a step: enqueues the copy of the K+1 losses of the most recent epoch
 * (layout of gad_get_loss) into loss_out, host memory that must be pinned and stay valid until gad_synchronize has
 * returned.  No check for non-finite values is made.  gad_synchronize waits for all of the context's streams and
 * returns GAD_ERR_DEVICE_TIMEOUT if a bounded device-side wait ran out since the last check (the epoch in which that
 * happened has left the parameters as they were: the update and consensus kernels skip their work once the error
 * word is set); the error is cleared by reporting it. */
int gad_read_loss_async(gad_ctx* ctx, float* loss_out);
int gad_synchronize(gad_ctx* ctx);

/* Self-check of the device store (no counterpart in the paper; it stands in for a memory checker): one kernel tests every
 * index the aggregation kernels form - rows, entry ranges, scratch slots of the work lists, and every stored column against
 * the row range of its own subgraph (the store is block-diagonal) - for the store and, if there is one, its transposed copy.
 * *violations receives the count; returns GAD_ERR_RANGE if it is not zero.  Waits for the stream. */
int gad_check_store(gad_ctx* ctx, int64_t* violations);

/* For testing the time-out path without hanging anything (no counterpart in the paper): enqueues a one-thread kernel
 * that waits, with the same bounded wait the tensor-core transforms use and a limit of `polls` polls (1 .. 65536), on
 * a barrier that nothing ever arrives at.  The wait runs out, the kernel raises the context's error word and returns;
 * the next gad_get_loss / gad_train_epoch with loss_out / gad_synchronize reports GAD_ERR_DEVICE_TIMEOUT, and an epoch
 * enqueued in between leaves the parameters untouched. */
int gad_debug_expire_wait(gad_ctx* ctx, uint32_t polls);

/* Epoch counter (it indexes the dropout mask); set it to resume a run. */
int gad_get_epoch(const gad_ctx* ctx, int64_t* epoch);
int gad_set_epoch(gad_ctx* ctx, int64_t epoch);

/* Per-kernel timing with CUDA events on the context's stream.  While enabled, every kernel launch of the
 * epoch is bracketed by two events.  gad_profile_read waits for the stream and returns, for entry i of
 * gad_profile_count entries: a name (up to 63 chars + NUL), launches and total milliseconds since the last
 * gad_profile_reset, and the algorithmic bytes and flops of ONE launch. */
int gad_profile_enable(gad_ctx* ctx, int32_t on);
int gad_profile_reset(gad_ctx* ctx);
int gad_profile_count(const gad_ctx* ctx, int32_t* count);
int gad_profile_read(gad_ctx* ctx, int32_t i, char* name64, int64_t* launches, double* total_ms,
                     double* bytes_per_launch, double* flops_per_launch);

/* The subgraph importance and consensus weights of gad_subgraph_weights, for callers that cannot allocate.
 * (No counterpart in the paper: it computes the same zeta_k and w_k; only where the intermediate sums live differs.)
 *
 * Who needs it: code that runs where a cudaMalloc on its behalf is not possible - the device's memory already
 * belongs to the host application's own pool, the call comes from inside a framework whose allocator owns the
 * GPU, or an allocation (which may synchronise the device) has no place in a latency-critical loop.  This entry
 * point needs no context and no workspace: it takes device inputs and device outputs only, and keeps its partial
 * sums in a fixed 4 MiB array inside the library image.  Every GPU that loads the library holds that array until
 * the process exits.  It calls no cudaMalloc / cudaFree and no allocating library routine.
 *
 *   X        device [rows x ld] floats, 16-byte aligned, row r = features of store row r (columns F..ld-1 ignored)
 *   deg      device [rows]: degree of each row inside its subgraph, self-loop excluded
 *   sub_off  device [K+1]: subgraph k owns rows sub_off[k] .. sub_off[k+1]-1, sub_off[K] = rows
 *   zeta_out, w_out  device [K]
 *   stream   a cudaStream_t; the four kernels are enqueued on it, the call does not wait
 * Limits (the size of the fixed array): K <= 256, ld <= 4096, ld a multiple of 4, K * ld <= 16384; anything
 * larger returns GAD_ERR_RANGE and launches nothing.
 * The first call on a device looks up the array's device address (cudaGetSymbolAddress, with that device current);
 * make that first call outside any stream capture.  All calls share the one array and it keeps the previous
 * call's contents; every slot a call reads it has first rewritten itself, so nothing needs clearing, but two
 * calls whose kernels overlap on the GPU (different streams or host threads) race on it - keep them on one
 * stream or serialise them. */
int gad_subgraph_weights_static(const float* X, int64_t rows, int32_t F, int32_t ld, const int32_t* deg,
                                const int32_t* sub_off, int32_t K, float beta, int32_t weighted, float* zeta_out,
                                float* w_out, void* stream);

/* ---- Importance-based subgraph augmentation (Algorithm 1, Section 3.2.2) -----------------------------------------
 * Produces the replication-node lists that gad_create takes as halo_nodes, from a partition of G into K core sets:
 * for every subgraph, random walks of `steps` steps (the number of GCN layers, Property 1) start at uniformly drawn
 * boundary nodes; count[v] = walks that contain the outside node v (importance equation, I(v) = count[v] / n); after the
 * first d |B| walks (d = average degree of the boundary nodes) the number of walks n follows the Monte-Carlo error
 * equation, n = (zc sigma / (mean E))^2, at most cap times the first batch; walks are ranked by the sum of I over
 * their outside nodes and their nodes are taken in walk order until alpha (1 + density) |v_i| nodes are selected.
 * The boundary test, the density count, the walks, the counts, their statistics, the walk scores and the selection of
 * the leading walks (the few thousand best-ranked ones, all the selection loop normally reaches) run on the GPU; the
 * order among those and the selection loop, which is sequential by definition, on the host.  Every random number is mix(seed, subgraph, walk, step) (splitmix64 output
 * function), so the result is a pure function of the arguments. */
typedef struct {
    int32_t steps;   /* walk length l = number of GCN layers, 1 .. 8                                      */
    int32_t cap;     /* at most cap times the first batch of walks (>= 1)                                  */
    double alpha;    /* replication constant of n(g_i) = alpha (1 + d(g_i)) |v_i|; the paper uses 0.01     */
    double E;        /* Monte-Carlo error bound; the paper uses 0.05                                       */
    double zc;       /* confidence statistic; 1.96 for the paper's 95 % level                              */
    uint64_t seed;
    int32_t graph_resident; /* 0: copy g to the device; 1: the caller vouches that an earlier gad_augment call with   *
                             * this very workspace and the same g (n, nnz, rowptr, col unchanged) left it there:  *
                             * the copy is skipped (the graph sits at the start of the workspace)                   */
} gad_augment_config;

/* Bytes of device workspace gad_augment needs.  Host-only. */
int gad_augment_workspace_bytes(const gad_csr* g, int32_t K, const int64_t* core_ptr, const int32_t* core_nodes,
                                const gad_augment_config* cfg, size_t* bytes);

/* g (its weights are ignored), core_ptr [K+1], core_nodes: host.  workspace: device, 256-byte aligned, owned by the
 * caller.  Outputs, host: halo_ptr [K+1]; halo_nodes [halo_capacity], subgraph k's replication nodes in selection order
 * at halo_ptr[k] .. halo_ptr[k+1]-1 (GAD_ERR_OOM if the capacity is too small: sum_k alpha (1 + d_k) |v_k| always
 * suffices); walks_out [K] = walks drawn per subgraph, or NULL.  Waits for the stream.  After an error
 * gad_augment_last_error gives the message of the calling thread. */
int gad_augment(const gad_csr* g, int32_t K, const int64_t* core_ptr, const int32_t* core_nodes, const gad_augment_config* cfg,
                void* workspace, size_t workspace_bytes, void* stream, int64_t* halo_ptr, int32_t* halo_nodes,
                int64_t halo_capacity, int64_t* walks_out);
const char* gad_augment_last_error(void);

/* Number of CUDA kernels this library has launched in this process so far (all contexts). */
int gad_launch_count(int64_t* launches);

/* Message of the context's last error; with ctx == NULL, of the calling thread's last error (e.g. after a failed
 * gad_create). */
const char* gad_last_error(const gad_ctx* ctx);

/* Frees the context.  Frees nothing the caller allocated (workspace, stream). */
void gad_destroy(gad_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* GAD_H */
