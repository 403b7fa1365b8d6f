/*
 * gnnco -- partitioned-GNN training step for combinatorial optimisation on one GPU.
 *
 * C ABI of the CUDA library.  The calls follow the problem statement of the method
 * (Algorithm 1 takes the graph G, its subgraphs {G_i} and the QUBO matrix Q and returns a bit string x):
 *
 *   gnnco_partition_load   graph + partition  -> block-diagonal batch of subgraphs
 *                          (Section 3.3, first paragraph; Algorithm 1, Stage 2 masks)
 *   gnnco_train_step       one full-batch GCN training step over every subgraph
 *                          (Section 3.2, Eqs. 3-5; penalty term of Section 3.3;
 *                          Algorithm 1, Stage 1)
 *   gnnco_decode_boundary  threshold the probabilities and count conflicts on
 *                          cross-subgraph edges (Section 3.3; Algorithm 1, Stage 2 and
 *                          the first line of Stage 3)
 *
 * General rules
 *   - Every function returns a gnnco_status (0 = success, negative = error); nothing
 *     throws, aborts or traps the device.
 *   - All buffers are CALLER-OWNED.  The library allocates no device memory; sizes of
 *     work areas come from the *_workspace_bytes queries.  Work areas must be 256-byte
 *     aligned.
 *   - Unless a parameter says "host", pointers are DEVICE pointers of the current
 *     CUDA device.  `stream` is a cudaStream_t passed as void*.
 *   - Per-node arrays (X, p, x, pen, dX, z) are in the library's NEW node order, in
 *     which every subgraph is a contiguous id range; `perm` (new -> original) and
 *     `inv_perm` (original -> new) from gnnco_graph_info map back to the caller's ids.
 *   - Dense matrices are row-major.
 */
#ifndef GNNCO_H_
#define GNNCO_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define GNNCO_MAX_LAYERS 8

typedef enum {
  GNNCO_OK = 0,
  GNNCO_INVALID_ARGUMENT = -1,    /* null pointer, bad size, bad enum, misaligned work area */
  GNNCO_OUT_OF_RANGE = -2,        /* node id or partition id outside its range */
  GNNCO_NOT_SIMPLE_GRAPH = -3,    /* self loop or repeated edge */
  GNNCO_UNSUPPORTED = -4,         /* dtype / width combination not implemented */
  GNNCO_WORKSPACE_TOO_SMALL = -5,
  GNNCO_CUDA_ERROR = -6,
  GNNCO_INTERNAL = -7
} gnnco_status;

typedef enum { GNNCO_F32 = 0, GNNCO_BF16 = 1 } gnnco_dtype;

/* flags of gnnco_train_step */
#define GNNCO_WANT_DX 1u        /* also compute d loss / d X (runs the transposed aggregation of layer 1) */
#define GNNCO_FORWARD_ONLY 2u   /* stop after loss and p (Algorithm 1, Stage 2 needs one forward pass per subgraph) */
/* The embeddings X are fixed inputs (Section 3.2 updates the weights W only), so the
 * first layer's aggregated input  mean_{self + intra neighbours}(X)  of Eq. 3 is the same in
 * every step of a run.  With GNNCO_AX_STORE the step keeps it in gnnco_train_out.ax_cache;
 * with GNNCO_AX_REUSE the step skips that aggregation and reads ax_cache instead (the caller
 * vouches that graph and X are those of the storing step).  Both need L >= 2 and a non-NULL
 * ax_cache; results are bit-identical to the plain step. */
#define GNNCO_AX_STORE 4u
#define GNNCO_AX_REUSE 8u
/* bfloat16 features only.  A step that runs Adam writes, together with the updated master weights, the
 * bfloat16 copies of them that the matrix products of the NEXT step read (inside the work area).  With
 * GNNCO_WEIGHTS_UNTOUCHED the caller vouches that nobody but this library has written W[l] since the
 * previous gnnco_train_step on this handle returned, and that the work area is the same one and has not
 * been written either; the step then skips rounding the master weights again.  Without the flag (or when
 * the previous step left no copies: first step, forward only, no optimiser, other buffers) the copies
 * are rebuilt from W at the start of the step.  Results are bit-identical either way. */
#define GNNCO_WEIGHTS_UNTOUCHED 16u
/* Fine-tuning on the active subgraphs only; see gnnco_active_plan. */
#define GNNCO_ACTIVE_ONLY 32u
/* bfloat16 features, hidden layers of width 256 -> 256 only (ignored elsewhere).  Such a layer of Eq. 3 then
 * runs as ONE kernel: the aggregated rows are summed on chip straight into the operand of the matrix
 * product and never reach device memory.  Rows are added in the same order as in the separate aggregation
 * kernel, so the results are bit-identical to the plain step wherever no row has more than 256 neighbours.
 * Off by default: on B200 the two separate kernels are faster (the fused kernel can keep about 60 KB of
 * gathers in flight per SM beside its operands, the separate aggregation kernel more); the flag exists for
 * devices and graphs where saving the write and the re-read of the aggregated features pays. */
#define GNNCO_ONE_KERNEL_LAYERS 64u

typedef struct gnnco_handle gnnco_handle;

/* Input graph: undirected, unweighted, simple.  Edge e joins edge_u[e] and edge_v[e]
 * (each edge listed once, either orientation); part[i] in [0, S) is node i's subgraph. */
typedef struct {
  int64_t n;                /* nodes, 1 <= n < 2^31 */
  int64_t E;                /* undirected edges, 0 <= E, 2E < 2^31 */
  int32_t S;                /* subgraphs, 1 <= S <= n */
  const int32_t* edge_u;    /* [E] */
  const int32_t* edge_v;    /* [E] */
  const int32_t* part;      /* [n] */
} gnnco_graph_desc;

/* Read-only view of what gnnco_partition_load built (pointers live in the caller's
 * persistent work area and stay valid until gnnco_destroy). */
typedef struct {
  int64_t n;
  int32_t S;
  int64_t E_in;                 /* intra-subgraph edges */
  int64_t E_b;                  /* boundary (cross-subgraph) edges */
  int32_t max_row;              /* largest intra degree */
  const int32_t* perm;          /* [n]   new id -> original id */
  const int32_t* inv_perm;      /* [n]   original id -> new id */
  const int32_t* part_ptr;      /* [S+1] subgraph s owns new ids part_ptr[s] .. part_ptr[s+1]-1 */
  const int32_t* node_part;     /* [n]   subgraph of each new id */
  const int32_t* rowptr;        /* [n+1] CSR of intra edges, both directions, no self loops */
  const int32_t* colidx;        /* [2*E_in] ascending inside a row */
  const int32_t* bnd_u;         /* [E_b] boundary edges in new ids, bnd_u < bnd_v, sorted by (u, v) */
  const int32_t* bnd_v;         /* [E_b] */
  const float* inv_deg;         /* [n]   1 / (intra degree + 1), Eq. 3's normaliser */
  const uint8_t* is_boundary;   /* [n]   1 iff the node touches a boundary edge ("cross-node") */
} gnnco_graph_view;

/* GCN of L layers, widths dims[0] -> dims[1] -> ... -> dims[L] with dims[L] == 1
 * (Eq. 3 per layer, ReLU on hidden layers; Eq. 4 on the last layer's scalar).
 * W[l] is layer l's weight, [weight_sets x dims[l] x dims[l+1]] float32; weight_sets is
 * S (one model per subgraph, Algorithm 1 Stage 1) or 1 (one shared model).
 * feat_dtype is the storage type of X and of the activations the library keeps;
 * accumulation is always float32.  With GNNCO_BF16 the weights are rounded to bf16
 * for the matrix products while W itself (the master copy Adam updates) stays float32. */
typedef struct {
  int32_t L;
  int32_t dims[GNNCO_MAX_LAYERS + 1];
  int32_t feat_dtype;            /* gnnco_dtype */
  int32_t weight_sets;
  float* W[GNNCO_MAX_LAYERS];
} gnnco_model_desc;

/* Eq. 5 with the fine-tuning penalty of Section 3.3:
 *   loss_s = alpha * sum_{intra edges (i,j) of s} p_i p_j - beta * sum_{i in s} p_i
 *            + lambda * sum_{i in s} pen[i] * p_i
 * pen may be NULL (no penalty). */
typedef struct {
  float alpha, beta, lambda;
  const float* pen;              /* [n] or NULL */
} gnnco_objective;

/* Adam state (bias-corrected; eps outside the square root).  `step` is the 1-based
 * number of THIS update; the caller increments it between calls.  m[l], v[l] have the
 * shape of W[l].
 * `active` (device, [S] uint8, or NULL = all) restricts the update to the subgraphs that
 * are being fine-tuned (Section 3.3: an action fine-tunes the model of ONE endpoint's
 * subgraph; Algorithm 1, Stage 3 groups the actions per subgraph): weights and moments of
 * a subgraph with active[s] == 0 are left bit-for-bit unchanged.  It needs per-subgraph
 * weights (weight_sets == S); the bias correction uses `step` for every active subgraph.
 * `step_dev` (device, one int32, or NULL): when given, `step` is ignored; the step reads the number of
 * updates done so far from *step_dev, adds one and uses that.  Nothing in such a step then depends on a host
 * value that changes from step to step, so a run of steps recorded once in a CUDA graph (stream capture of
 * gnnco_train_step / gnnco_decode_boundary on the capturing stream; same buffers at every replay) can be
 * replayed any number of times -- for graphs of a few thousand nodes, where a step is tens of launches of a few
 * microseconds, that removes most of its cost. */
typedef struct {
  float lr, beta1, beta2, eps;
  int64_t step;
  float* m[GNNCO_MAX_LAYERS];
  float* v[GNNCO_MAX_LAYERS];
  const uint8_t* active;
  int32_t* step_dev;
} gnnco_adam_state;

/* Outputs of a training step.  loss and p are required; the rest may be NULL. */
typedef struct {
  float* loss;                   /* [S]  per-subgraph objective */
  float* p;                      /* [n]  selection probabilities (Eq. 4) */
  float* z;                      /* [n]  pre-sigmoid values, or NULL */
  float* dW[GNNCO_MAX_LAYERS];   /* gradient of sum_s loss_s wrt W[l], shape of W[l], or NULL */
  void* dX;                      /* [n x dims[0]] in feat_dtype; written only with GNNCO_WANT_DX */
  void* ax_cache;                /* [n x dims[0]] in feat_dtype; see GNNCO_AX_STORE / GNNCO_AX_REUSE; else NULL */
} gnnco_train_out;

typedef struct {
  int64_t set_size;              /* number of selected nodes */
  int64_t intra_viol;            /* intra edges with both ends selected */
  int64_t boundary_viol;         /* boundary edges with both ends selected */
} gnnco_counts;

const char* gnnco_status_string(int32_t status);

/* Sizes (bytes) of the two work areas of gnnco_partition_load for a graph of n nodes,
 * E edges and S subgraphs: `persistent` must outlive the handle, `scratch` may be
 * released when gnnco_partition_load returns.  `persistent` is about 41 n + 24 E bytes: the node
 * order, the CSR of the intra edges, the boundary list, a 16-byte head record per row, the per-row source list
 * of GNNCO_ONE_KERNEL_LAYERS (4 (n + 2 E) bytes) and the tile tables. */
int32_t gnnco_partition_workspace_bytes(int64_t n, int64_t E, int32_t S, size_t* persistent, size_t* scratch);

/* Build the block-diagonal batch (Section 3.3: split into subgraphs; cross edges set
 * aside).  New ids rank nodes by (part, original id); intra edges become a symmetric
 * CSR; boundary edges a sorted list.  All integer results are exactly defined (no
 * ordering freedom).  Runs on `stream` and synchronises it (sizes and the validation
 * result must reach the host).  On success *out receives a handle (host object, freed by
 * gnnco_destroy).  Errors: GNNCO_OUT_OF_RANGE, GNNCO_NOT_SIMPLE_GRAPH,
 * GNNCO_WORKSPACE_TOO_SMALL, GNNCO_INVALID_ARGUMENT, GNNCO_CUDA_ERROR. */
int32_t gnnco_partition_load(const gnnco_graph_desc* g, void* persistent_ws, size_t persistent_bytes,
                             void* scratch_ws, size_t scratch_bytes, void* stream, gnnco_handle** out);

int32_t gnnco_graph_info(const gnnco_handle* h, gnnco_graph_view* out);

/* Quality of the loaded partition in the terms of Section 3.1 (the quantities of Eq. 1), all device
 * outputs:  in_edges [S] int64 = edges with both ends in subgraph s;  tot [S] int64 = Sigma_tot, the
 * degree sum of its nodes in the whole graph;  Q = sum_s [ 2 in_edges(s) / 2m - (tot(s) / 2m)^2 ],
 * m = E, the modularity that the paper's partitioner maximises (float64; 0 when E = 0).  The
 * integers are exact.  Asynchronous on `stream`. */
int32_t gnnco_partition_quality(gnnco_handle* h, int64_t* in_edges, int64_t* tot, double* Q, void* stream);

/* Louvain partitioning (Section 3.1, Eqs. 1-2): the subgraphs that the method trains on.  The paper's
 * procedure moves nodes one by one in an order it does not fix, so its result is not unique; this is the
 * variant whose result is: every node of a level decides from the same frozen state (best gain of Eq. 2
 * over its own and its neighbours' communities, compared exactly in 64-bit integers, lowest community id
 * among equals, a move only on a strictly better gain, a node alone in its community never joins a
 * single node with a higher id), all moves of a sweep are applied together and kept only if the exact
 * modularity rises; then communities are contracted into the nodes of the next level, until a level moves
 * nothing.  Levels and sweeps per level are capped by max_levels / max_sweeps (32 and 64 are plenty).
 *   edge_u, edge_v [E] device: the graph as in gnnco_graph_desc (simple, undirected, each edge once)
 *   part [n] device int32 (out): community of every node, numbered 0 .. S-1; pass it to
 *        gnnco_partition_load with S = *S_out
 *   S_out, qnum_out, two_m_out, levels_out, sweeps_out: HOST values (the last four may be NULL): number of
 *        communities, exact modularity numerator and 2m (Q = qnum / two_m^2, Eq. 1's sum with Sigma_in counted
 *        from both ends), levels that moved a node, sweeps kept
 * ws: gnnco_louvain_workspace_bytes bytes, 256-byte aligned, free again when the call returns.  The call
 * synchronises `stream` several times per sweep (two integers decide whether a sweep is kept).
 * Errors: GNNCO_OUT_OF_RANGE, GNNCO_NOT_SIMPLE_GRAPH (self loop), GNNCO_WORKSPACE_TOO_SMALL. */
int32_t gnnco_louvain_workspace_bytes(int64_t n, int64_t E, size_t* bytes);
int32_t gnnco_louvain(int64_t n, int64_t E, const int32_t* edge_u, const int32_t* edge_v, int32_t max_levels,
                      int32_t max_sweeps, int32_t* part, int32_t* S_out, int64_t* qnum_out, int64_t* two_m_out,
                      int32_t* levels_out, int32_t* sweeps_out, void* ws, size_t ws_bytes, void* stream);

/* dst[i] = src[index[i]] for i < rows, rows of row_bytes bytes each (row_bytes a
 * multiple of 4).  With index = perm it brings a per-node array from the caller's
 * original order into the new order (Algorithm 1, Stage 2 uses the inverse to "map
 * local probs to global mask"): pass inv_perm to go back. */
int32_t gnnco_gather_rows(const gnnco_handle* h, const void* src, void* dst, const int32_t* index, int64_t rows,
                          int64_t row_bytes, void* stream);

/* Work-area size of gnnco_train_step for this graph and model. */
int32_t gnnco_train_workspace_bytes(const gnnco_handle* h, const gnnco_model_desc* m, uint32_t flags, size_t* bytes);

/* One training step over all subgraphs at once (Section 3.2):
 *   forward   per hidden layer  H' = ReLU( mean_{self + intra neighbours}(H) W_s )   (Eq. 3)
 *             last layer        z = mean_{self + intra neighbours}(H) w_s,  p = sigmoid(z)   (Eq. 4)
 *   objective loss_s as in gnnco_objective                                           (Eq. 5)
 *   backward  exact gradient of sum_s loss_s wrt every W (and X with GNNCO_WANT_DX)
 *   update    Adam on every W (skipped when opt == NULL or with GNNCO_FORWARD_ONLY)
 * X is [n x dims[0]] in feat_dtype, new node order, and is not modified.  Asynchronous
 * on `stream`; per-subgraph results are deterministic (no floating-point atomics). */
int32_t gnnco_train_step(gnnco_handle* h, const gnnco_model_desc* m, const void* X, const gnnco_objective* obj,
                         gnnco_adam_state* opt, const gnnco_train_out* out, uint32_t flags, void* ws,
                         size_t ws_bytes, void* stream);

/* Fine-tuning steps that cost what the ACTIVE subgraphs cost (Section 3.3: a conflict is resolved by
 * fine-tuning the model of one endpoint's subgraph; Algorithm 1, Stage 3 fine-tunes the subgraphs that
 * the grouped actions name -- typically a small share of all subgraphs).
 *
 * gnnco_active_plan reads `active` (device, [S] uint8, e.g. the vector written by gnnco_apply_actions)
 * and lays out, inside `plan_ws` (device, gnnco_active_plan_bytes bytes, 256-byte aligned, owned by the
 * caller and kept until the plan is replaced or the handle destroyed), the work lists of the active
 * subgraphs.  It synchronises `stream` (the flags must reach the host) and stores the number of active
 * subgraphs in *active_count (host, may be NULL).  A new call replaces the plan.
 *
 * gnnco_train_step with GNNCO_ACTIVE_ONLY then runs forward, objective, backward and Adam over those
 * subgraphs only.  It needs a plan, opt != NULL with opt->active equal to the pointer the plan was built
 * from (the caller vouches that the flags have not changed since), per-subgraph weights and L >= 2.
 * For every INACTIVE subgraph the step leaves loss[s], its rows of p, z and dX, its dW[l][s] and its
 * weights and moments exactly as they were; for every active subgraph all results are bit-identical to
 * those of a full step.  Not combined with GNNCO_AX_STORE / GNNCO_AX_REUSE. */
int32_t gnnco_active_plan_bytes(const gnnco_handle* h, size_t* bytes);
int32_t gnnco_active_plan(gnnco_handle* h, const uint8_t* active, void* plan_ws, size_t plan_bytes, void* stream,
                          int32_t* active_count);

/* Same step with HOST buffers for the per-step data: X_host [n x dims[0]] (feat_dtype,
 * new order; pinned memory recommended), pen_host [n] or NULL, loss_host [S], p_host [n].
 * Weights, Adam moments and the work area stay on the device.  `stream` is synchronised before
 * returning.  Inputs of 64 MB and more (L >= 2, S >= 2, no GNNCO_ACTIVE_ONLY) are uploaded in eight
 * ranges of subgraphs on a stream of the handle's own, ordered after whatever `stream` held at the call,
 * and the first hidden layer (Eq. 3 needs only a subgraph's own rows of X) runs on each range as it
 * arrives; smaller inputs are copied on `stream` itself.  Results are bit-identical to gnnco_train_step on
 * the same data either way.  ws must hold gnnco_train_host_workspace_bytes bytes. */
int32_t gnnco_train_host_workspace_bytes(const gnnco_handle* h, const gnnco_model_desc* m, uint32_t flags,
                                         size_t* bytes);
int32_t gnnco_train_step_host(gnnco_handle* h, const gnnco_model_desc* m, const void* X_host, float alpha,
                              float beta, float lambda, const float* pen_host, gnnco_adam_state* opt,
                              float* loss_host, float* p_host, uint32_t flags, void* ws, size_t ws_bytes,
                              void* stream);

/* Decode (Section 3.3): x[i] = (p[i] >= threshold) on the stored float32 value; a
 * boundary edge is violated when both ends are selected.
 *   x        [n] uint8, required          viol     [E_b] uint8 or NULL
 *   per_part [S] int32 or NULL: violated boundary edges touching subgraph s (an edge
 *            counts for both of its subgraphs, so the entries sum to 2*boundary_viol)
 *   counts   device gnnco_counts, required
 * Integer results are exact.  Asynchronous on `stream`; needs no work area. */
int32_t gnnco_decode_boundary(const gnnco_handle* h, const float* p, float threshold, uint8_t* x, uint8_t* viol,
                              int32_t* per_part, gnnco_counts* counts, void* stream);

/* Stage-3 glue (Section 3.3; Algorithm 1, Stage 3), the step right after decoding.
 *
 * gnnco_conflict_actions turns the per-edge flags of gnnco_decode_boundary into the
 * conflict set C and a non-learned base action for each conflict:
 *   conflict_idx [E_b] int32 (capacity): positions, in the sorted boundary list, of the
 *                violated edges, ASCENDING; only the first *count entries are written
 *   action       [E_b] uint8 (capacity) or NULL: for conflict c on the stored pair (u, v),
 *                u < v in the new order, 0 = push u below the threshold, 1 = push v.
 *                Section 3.3 gives every conflict exactly these two options.  Algorithm 1,
 *                Stage 3 starts the agent from a base action obtained with a cover heuristic
 *                that it does not spell out; this library SUBSTITUTES a rule of its own for
 *                it: the endpoint with the SMALLER probability p, and v when they are equal.
 *   count        device int32: |C|
 * viol [E_b] uint8 and p [n] float32 (new order) are inputs; p may be NULL iff action is.
 * ws must hold gnnco_conflict_workspace_bytes bytes.  Asynchronous on `stream`; no host
 * synchronisation (|C| stays on the device).  Results are exact and order-deterministic.
 *
 * gnnco_apply_actions turns (C, actions) into the inputs of the fine-tuning steps:
 *   pen    [n] float32: 1 for every chosen node, else 0 -- the node list of the added
 *          penalty term lambda * sum_k p_{i_k} (gnnco_objective.pen)
 *   active [S] uint8: 1 for every subgraph holding a chosen node (gnnco_adam_state.active)
 *   chosen device int32 or NULL: number of distinct chosen nodes
 * count is the DEVICE value written by gnnco_conflict_actions; action may come from there or
 * from the caller's own policy (any 0/1 vector of that length).  Asynchronous on `stream`. */
/*
 * gnnco_repair_boundary carries the chosen actions out on the mask itself, without any
 * fine-tuning -- the non-learned baseline of Stage 3 (Section 3.3: acting on a conflict takes
 * one of its two endpoints out of the candidate set):  x[i] <- 0 for every chosen node
 * (pen[i] != 0, the vector written by gnnco_apply_actions).  Afterwards no boundary edge has both
 * ends selected; intra-subgraph conflicts are not touched.  removed (device int32, or NULL)
 * receives the number of selected nodes that were cleared.  Asynchronous on `stream`. */
int32_t gnnco_repair_boundary(gnnco_handle* h, const float* pen, uint8_t* x, int32_t* removed, void* stream);
int32_t gnnco_conflict_workspace_bytes(const gnnco_handle* h, size_t* bytes);
int32_t gnnco_conflict_actions(gnnco_handle* h, const uint8_t* viol, const float* p, int32_t* conflict_idx,
                               uint8_t* action, int32_t* count, void* ws, size_t ws_bytes, void* stream);
int32_t gnnco_apply_actions(gnnco_handle* h, const int32_t* conflict_idx, const uint8_t* action,
                            const int32_t* count, float* pen, uint8_t* active, int32_t* chosen, void* stream);

/* Input embeddings (Section 3.2, subgraph training: the random initial node embeddings go
 * through a Gumbel-softmax before the first layer).
 *
 * gnnco_gumbel_softmax: X[i,:] = softmax( (E[i,:] + g[i,:]) / tau ) over the F features of node i,
 * with Gumbel noise g = -log(-log U) from uniforms U in (0, 1), exclusive, that the caller draws
 * (U == NULL: no noise).  The paper fixes neither the temperature, nor hard versus soft, nor
 * when the noise is redrawn; this is the soft form with one temperature, and the noise is an
 * input, so the call is deterministic.  E and X are [n x F] in feat_dtype (any node order, rows
 * are independent; E == X is allowed), U is [n x F] float32.  tau > 0.  Asynchronous on `stream`.
 *
 * gnnco_embedding_update: the variant in which the embeddings are trained (the paper only says
 * that W is updated; gnnco_train_step leaves X alone).  One Adam step, same rule as for the
 * weights, on the float32 master copy X_master [n x F] with the gradient dX [n x F] (feat_dtype)
 * that gnnco_train_step wrote under GNNCO_WANT_DX; m and v are its moments (float32, zero
 * before the first step), `step` is the 1-based number of this update.  X [n x F] (feat_dtype)
 * receives the updated embeddings in the type the next gnnco_train_step reads; a cached
 * first-layer aggregation (GNNCO_AX_REUSE) is stale after this call.  Asynchronous on `stream`. */
int32_t gnnco_gumbel_softmax(gnnco_handle* h, int32_t feat_dtype, int32_t F, const void* E, const float* U, float tau,
                             void* X, void* stream);
int32_t gnnco_embedding_update(gnnco_handle* h, int32_t feat_dtype, int32_t F, const void* dX, float* X_master,
                               float* m, float* v, void* X, float lr, float beta1, float beta2, float eps,
                               int64_t step, void* stream);

/* Objective only, for callers that cannot allocate device memory.  (The paper has no
 * counterpart to this call; it exists for the way the library is embedded.)
 *
 * Some users of this library run where no allocation is possible at the moment they need a
 * loss value: a coordination loop living inside another program's callback or plug-in
 * interface is handed `p` and a place for `loss` and nothing else -- it owns no allocator, the
 * host program's memory pool is not its to grow, and a cudaMalloc there would stall every
 * stream of the process.  gnnco_train_step cannot serve them, because it needs a work area.
 * This entry point evaluates the per-subgraph objective of gnnco_objective for GIVEN
 * probabilities `p` [n] (new node order) and writes loss [S]; it allocates nothing and takes
 * no work area.  Its only scratch, one float per objective work item, is a fixed array of
 * GNNCO_STATIC_OBJECTIVE_MAX_ITEMS floats (256 KiB) inside the library image, which every
 * GPU that loads the library holds until the process exits.
 *
 *  - A graph needs  sum_s ceil(|V_s| / 1024)  work items; if that exceeds the maximum the call
 *    returns GNNCO_WORKSPACE_TOO_SMALL and does nothing.
 *  - The first call on a device looks up the array's device address (once per device, with
 *    that device current); make that first call outside any stream capture.
 *  - All calls share the one array and it keeps what the last call left: the part a call
 *    uses is cleared and rewritten by that call, but two calls that overlap on the GPU
 *    (different streams, or another thread) race on it.  Serialise them.
 *  - The handle's device must be current.  Asynchronous on `stream`.  Results equal
 *    gnnco_train_step's loss for the same p to float32 rounding, and bit for bit when no row has
 *    more than 256 intra neighbours (longer rows are summed in another order here).
 */
#define GNNCO_STATIC_OBJECTIVE_MAX_ITEMS 65536
int32_t gnnco_objective_static(gnnco_handle* h, const float* p, const gnnco_objective* obj, float* loss,
                               void* stream);

/* Host read of the device-side status word (synchronises `stream`). */
int32_t gnnco_async_status(const gnnco_handle* h, void* stream, int32_t* status);

/* Per-kernel timing (a measurement aid; Section 4.1 reports runtime as a metric).
 * Between gnnco_profile_begin and gnnco_profile_end every kernel family of gnnco_train_step
 * and gnnco_decode_boundary is bracketed by CUDA events on the launching stream.
 * gnnco_profile_end synchronises `stream`, writes one entry per family that ran into
 * `entries` (host array of `capacity` elements) and their number into *count; it returns
 * GNNCO_WORKSPACE_TOO_SMALL if capacity was too small (*count then holds the need). */
typedef struct {
  char name[32];
  int64_t calls;       /* launcher calls (a call may issue more than one kernel) */
  double total_ms;     /* summed device time of those calls */
} gnnco_profile_entry;
int32_t gnnco_profile_begin(gnnco_handle* h);
int32_t gnnco_profile_end(gnnco_handle* h, void* stream, gnnco_profile_entry* entries, int32_t capacity,
                          int32_t* count);

/* Number of kernels this handle has launched so far (for launch accounting). */
int64_t gnnco_launch_count(const gnnco_handle* h);

int32_t gnnco_destroy(gnnco_handle* h);

#ifdef __cplusplus
}
#endif
#endif /* GNNCO_H_ */
