// Internal declarations shared by the translation units of libgnnco.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "gnnco.h"

#define GNNCO_CUDA_TRY(expr)                      \
  do {                                            \
    cudaError_t e__ = (expr);                     \
    if (e__ != cudaSuccess) return GNNCO_CUDA_ERROR; \
  } while (0)

#define GNNCO_LAUNCH_CHECK()                                   \
  do {                                                         \
    if (cudaPeekAtLastError() != cudaSuccess) { cudaGetLastError(); return GNNCO_CUDA_ERROR; } \
  } while (0)

constexpr int kGemmTileRows = 128;   // rows of one dense-transform tile (never straddles a subgraph)
constexpr int kLongRowDegree = 256;  // rows with more intra neighbours are aggregated by a whole block
constexpr int kLongRowSegment = 2048; // ... and in segments of this many neighbours, one block each
constexpr int kWgChunkMinRows = 2048; // a subgraph is split for the weight gradient only in runs at least this long
constexpr int kItemRows = 1024;      // rows of one objective work item (never straddles a subgraph)

// Kernel families, for launch accounting and per-kernel timing.
enum KernelKind {
  K_AGG_FWD, K_AGG_BWD, K_TRANSFORM_FWD, K_TRANSFORM_BWD, K_WEIGHT_GRAD, K_GEMV, K_WEIGHT_GRAD_VEC, K_RANK1,
  K_SUM_SETS, K_CAST, K_ADAM, K_OUT_FWD, K_OBJECTIVE, K_OUT_BWD, K_DECODE, K_STAGE3, K_AGG_RANK1, K_EMBED,
  K_AGG_TRANSFORM, K_KIND_COUNT
};

// Optional per-kernel timing: while `on`, every launcher brackets its launches with a pair
// of CUDA events on the launching stream; gnnco_profile_end turns the pairs into totals.
struct Profiler {
  struct Rec { int kind; cudaEvent_t a, b; };
  bool on = false;
  std::vector<cudaEvent_t> pool;
  size_t used = 0;
  std::vector<Rec> recs;
  cudaEvent_t get() {
    if (used == pool.size()) {
      cudaEvent_t e = nullptr;
      if (cudaEventCreate(&e) != cudaSuccess) return nullptr;
      pool.push_back(e);
    }
    return pool[used++];
  }
};

// Rows of a step that runs on SOME subgraphs only (fine-tuning, Section 3.3): the active subgraphs'
// row ranges cut into chunks of at most 256 rows.  row0 == nullptr means "all n rows".  A kernel that
// gives every block R rows (R divides 256) is launched with linear_rows() / R blocks and turns its linear
// row index into a row with chunk_row().
struct RowChunks {
  const int32_t* row0 = nullptr;
  const int32_t* rows = nullptr;
  int32_t count = 0;
};
__device__ __forceinline__ bool chunk_row(const RowChunks& rc, int64_t linear, int64_t n, int64_t& row) {
  if (!rc.row0) {
    row = linear;
    return linear < n;
  }
  const int64_t c = linear >> 8;
  const int off = (int)(linear & 255);
  if (c >= rc.count) return false;
  row = (int64_t)rc.row0[c] + off;
  return off < rc.rows[c];
}

// Work tables of the hidden layer that runs as one kernel (tc_gemm2.cu).  The double tiles are split into
// LIGHT ones (short rows only: the kernel's adders give every row to one warp) with each CTA's extent in the
// source list, cut into per-cluster ranges of about equal cost, and HEAVY ones (a long row or many entries),
// which go through the separate aggregation and transform kernels -- their tables have the format of the
// double-tile tables and of RowChunks.
struct FuseSet {
  int4* meta = nullptr;                 // [2 n_light] {tile's first row, this CTA's rows, list extent begin, end}
  int32_t* cluster_begin = nullptr;     // [clusters + 1] light tiles of each CTA pair
  int32_t *light_row0 = nullptr, *light_rows = nullptr, *heavy_row0 = nullptr, *heavy_rows = nullptr;
  int2* weights = nullptr;              // [tiles] scratch of the build: {list entries, longest row}
  int32_t n_light = 0, n_heavy = 0, clusters = 0;
  bool built = false;
};
constexpr int kFuseMaxClusters = 256;

// The per-graph work tables that the kernels of a step walk.  The handle holds the set for all
// subgraphs; gnnco_active_plan builds a second set for the active subgraphs only, and a step with
// GNNCO_ACTIVE_ONLY runs with that set swapped in.
struct WorkSet {
  int32_t *tile_row0 = nullptr, *tile_rows = nullptr, *pair_row0 = nullptr, *pair_rows = nullptr;
  int32_t *item_row0 = nullptr, *item_row1 = nullptr, *part_item_ptr = nullptr;
  int32_t *wg_begin = nullptr, *wg_end = nullptr, *wg_slot = nullptr;
  int32_t *wg_mpart = nullptr, *wg_mfirst = nullptr, *wg_mcount = nullptr;
  int32_t n_tiles = 0, n_pairs = 0, n_items = 0, n_wg_chunks = 0, n_wg_multi = 0;
  RowChunks row_chunks;
  FuseSet fuse;
};

// The host-buffer step lets layer 1 start on a range of subgraphs as soon as that range of X has been uploaded:
// per range the event its copy records and where its tiles and double tiles start in the tables.
constexpr int kArrivalGroups = 8;
struct ArrivalPlan {
  int groups = 0;
  cudaEvent_t ev[kArrivalGroups] = {};
  cudaEvent_t ev_rest = nullptr;                             // everything else the step uploads (the penalty mask)
  int32_t tile0[kArrivalGroups + 1] = {}, pair0[kArrivalGroups + 1] = {};
};

struct gnnco_handle {
  int64_t n = 0, E = 0, E_in = 0, E_b = 0;
  int32_t S = 0, max_row = 0;
  int device = 0, sm_count = 0;
  // device arrays inside the caller's persistent work area
  int32_t *perm = nullptr, *inv_perm = nullptr, *part_ptr = nullptr, *node_part = nullptr;
  int32_t *rowptr = nullptr, *colidx = nullptr, *bnd_u = nullptr, *bnd_v = nullptr;
  float* inv_deg = nullptr;
  uint8_t* is_boundary = nullptr;
  int32_t *tile_row0 = nullptr, *tile_rows = nullptr;      // dense-transform tiles
  int32_t *pair_row0 = nullptr, *pair_rows = nullptr;      // double tiles (up to 256 rows of one subgraph) for CTA pairs
  int32_t n_pairs = 0;
  int pair_clusters = -1;                                  // co-resident CTA pairs of the two-CTA transform (-1: not asked yet)
  int32_t *item_row0 = nullptr, *item_row1 = nullptr;      // objective work items
  int32_t* part_item_ptr = nullptr;                        // [S+1] items of each subgraph
  int32_t* status = nullptr;                               // device status word + counters
  FuseSet fuse;                                            // tables of the one-kernel layer for the running work set
  int32_t* src_list = nullptr;                             // per row: its own index, then its neighbours' (n + 2 E_in entries)
  int4* row_head = nullptr;                                // {first CSR slot, degree, first two neighbours} per row
  int32_t* long_rows = nullptr;                            // ids of rows with degree > kLongRowDegree, ascending
  // the long rows' neighbour lists cut into segments: CSR slots [seg_begin, seg_end) of each segment, and
  // for long row k its segments long_first_seg[k] .. long_first_seg[k+1]-1
  int32_t *seg_begin = nullptr, *seg_end = nullptr, *long_first_seg = nullptr;
  int32_t n_long_segs = 0;
  float* agg_partial = nullptr;                            // [n_long_segs x width] float32, set for the running step
  int32_t n_tiles = 0, n_items = 0, n_long = 0;
  // weight-gradient work: row ranges, output slot (>= 0 scratch slot, < 0 subgraph -(slot+1)), and the
  // subgraphs that were split (id, first slot, slot count)
  int32_t *wg_begin = nullptr, *wg_end = nullptr, *wg_slot = nullptr;
  int32_t *wg_mpart = nullptr, *wg_mfirst = nullptr, *wg_mcount = nullptr;
  int32_t n_wg_chunks = 0, n_wg_slots = 0, n_wg_multi = 0;
  std::vector<int32_t> h_part_ptr;
  // a step on the active subgraphs only: the rows it covers (nullptr: all), the plan built by
  // gnnco_active_plan and the device flags it was built from
  RowChunks row_chunks;
  WorkSet plan;
  const uint8_t* plan_active = nullptr;
  int32_t plan_active_count = -1;                            // -1: no plan
  int64_t launches = 0;
  Profiler prof;
  // bf16 copies of the weights that the last updating step left in its work area (GNNCO_WEIGHTS_UNTOUCHED):
  // which master weights and which copies they belong to; fresh[l] says whether layer l's copies are current
  const float* shadow_W[GNNCO_MAX_LAYERS] = {nullptr};
  const void* shadow_copy[GNNCO_MAX_LAYERS] = {nullptr};
  bool shadow_fresh[GNNCO_MAX_LAYERS] = {false};
  // long rows are aggregated on a side stream, concurrently with the short rows
  cudaStream_t side_stream = nullptr;
  // gnnco_train_step_host: the stream its uploads run on, their events, and (during such a step) the plan
  cudaStream_t copy_stream = nullptr;
  cudaEvent_t ev_arrive[kArrivalGroups] = {}, ev_rest = nullptr, ev_begin = nullptr;
  const ArrivalPlan* arrival = nullptr;
  // during a step whose Adam state keeps its step counter on the device: where adam_tick left 1 / (1 - beta^t)
  const float2* adam_bias = nullptr;
  cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
};

struct ProfScope {
  gnnco_handle* h;
  cudaStream_t st;
  Profiler::Rec rec{};
  bool on = false;
  ProfScope(gnnco_handle* h_, int kind, cudaStream_t st_) : h(h_), st(st_) {
    if (!h->prof.on) return;
    rec.kind = kind;
    rec.a = h->prof.get();
    rec.b = h->prof.get();
    if (!rec.a || !rec.b) return;
    on = cudaEventRecord(rec.a, st) == cudaSuccess;
  }
  ~ProfScope() {
    if (on && cudaEventRecord(rec.b, st) == cudaSuccess) h->prof.recs.push_back(rec);
  }
};

static inline size_t align_up(size_t x, size_t a = 256) { return (x + a - 1) / a * a; }

// rows a row-per-thread (or row-group-per-block) kernel has to cover in the running step
static inline int64_t linear_rows(const gnnco_handle* h) {
  return h->row_chunks.row0 ? (int64_t)h->row_chunks.count * 256 : h->n;
}

// Host side of the work tables: what partition_load uploads for all subgraphs and what
// gnnco_active_plan uploads for the active ones (active == nullptr: all).  Defined in partition.cu.
struct HostWorkTables {
  std::vector<int32_t> t0, tr, p0, pr, i0, i1, pip, wb, we, wsl, mp, mf, mc, c0, cr;
  int32_t n_wg_slots = 0;
};
void build_work_tables(const std::vector<int32_t>& part_ptr, int32_t S, int64_t n, int sm_count, const uint8_t* active,
                       HostWorkTables& out);

// A bump allocator over a caller-provided work area.
struct Carver {
  char* base;
  size_t off = 0, cap;
  Carver(void* p, size_t bytes) : base(static_cast<char*>(p)), cap(bytes) {}
  template <typename T>
  T* take(size_t count) {
    size_t bytes = align_up(count * sizeof(T));
    T* r = reinterpret_cast<T*>(base + off);
    off += bytes;
    return r;
  }
  bool ok() const { return off <= cap; }
};

// the arrays of a FuseSet for at most `tiles` double tiles
inline FuseSet carve_fuse_set(Carver& c, size_t tiles) {
  FuseSet f;
  f.meta = c.take<int4>(2 * tiles);
  f.cluster_begin = c.take<int32_t>(kFuseMaxClusters + 1);
  f.light_row0 = c.take<int32_t>(tiles);
  f.light_rows = c.take<int32_t>(tiles);
  f.heavy_row0 = c.take<int32_t>(tiles);
  f.heavy_rows = c.take<int32_t>(tiles);
  f.weights = c.take<int2>(tiles);
  return f;
}

// ---- partition.cu : device primitives (stable LSD radix sort of 64-bit keys on bits [bit_lo, bit_hi) with an
// optional 32-bit payload, exclusive scan of int32) and the sizes of their scratch arrays
int32_t device_exclusive_scan(int32_t* data, int64_t N, int32_t* tile_sums, cudaStream_t st);
int32_t device_radix_sort(uint64_t* a, uint64_t* b, int64_t N, int bit_lo, int bit_hi, int32_t* hist, int32_t* tile_sums,
                          cudaStream_t st, uint64_t** result, int32_t* va, int32_t* vb, int32_t** vresult);
void device_sort_scratch_sizes(int64_t N, size_t* hist_ints, size_t* tile_sum_ints);
void device_scan_scratch_size(int64_t N, size_t* tile_sum_ints);

// ---- spmm.cu : out[i] = scale[i] * (in[i] + sum_{j in row i} in[j]), optionally zeroed where mask[i,f] <= 0
int32_t launch_aggregate(gnnco_handle* h, int dtype, const void* in, void* out, int F, const float* row_scale,
                         const void* relu_mask, cudaStream_t st);
// out[i,f] = w_s[f] * sum_{j in {i} + row i} coef[j] * [H[j,f] > 0]: the transposed aggregation of
// D^-1 (g w_s^T * [H > 0]) with coef = D^-1 g, gathered straight from the saved activation H
int32_t launch_aggregate_rank1(gnnco_handle* h, int dtype, const void* H, const float* coef, const void* w,
                               int64_t w_stride, void* out, int F, cudaStream_t st);
// the same from the bits [H > 0] (n x F/8 bytes, element f of a row = bit f%8 of byte f/8) instead of H
// (H itself is still read for the few rows with more than kLongRowDegree neighbours)
bool aggregate_rank1_bits_supported(const gnnco_handle* h, int dtype, int F);
int32_t launch_aggregate_rank1_bits(gnnco_handle* h, int dtype, const uint8_t* bits, const void* H, const float* coef,
                                    const void* w, int64_t w_stride, void* out, int F, cudaStream_t st);

// ---- dense.cu
// Y[tile rows x N] = act( A[rows x K] * B_s ), B_s = W[s] (K x N) or, with transB, W[s]^T where W[s] is (N x K);
// with relu_mask (same shape as Y) the result is zeroed where relu_mask <= 0.
int32_t launch_transform(gnnco_handle* h, int dtype, const void* A, const void* W, int64_t w_stride, void* Y, int K,
                         int N, bool transB, bool relu, const float* row_scale, const void* relu_mask,
                         cudaStream_t st);
// u[i] = H[i,:] . w_s
int32_t launch_gemv(gnnco_handle* h, int dtype, const void* H, const void* w, int64_t w_stride, float* u, int F,
                    cudaStream_t st);
// dW[s] (K x N) = sum_{i in s} A[i,:]^T G[i,:]
int32_t launch_weight_grad(gnnco_handle* h, int dtype, const void* A, const void* G, float* dW, float* scratch, int K,
                           int N, cudaStream_t st);
// dw[s][f] = sum_{i in s} H[i,f] g[i]; scratch: F floats per slot of the weight-gradient chunk table.
// bits_out (optional, n x F/8 bytes): receives [H > 0], one bit per element, when the kernel that runs
// can produce it; *wrote_bits says whether it did.
int32_t launch_weight_grad_vec(gnnco_handle* h, int dtype, const void* H, const float* g, float* dw, float* scratch,
                               int F, uint8_t* bits_out, bool* wrote_bits, cudaStream_t st);
// dZ[i,f] = g[i] * w_s[f] where H[i,f] > 0, else 0 (H == nullptr: no mask)
int32_t launch_rank1_masked(gnnco_handle* h, int dtype, const float* g, const void* w, int64_t w_stride, const void* H,
                            void* dZ, int F, cudaStream_t st);
// dW[part] = sum of the scratch slots of every split subgraph, in slot order
int32_t launch_wg_combine(gnnco_handle* h, const float* scratch, float* dW, int64_t count, cudaStream_t st);
// out[q] = sum_s in[s][q]
int32_t launch_sum_over_sets(gnnco_handle* h, const float* in, float* out, int64_t count, int32_t sets, cudaStream_t st);
int32_t launch_cast_bf16(gnnco_handle* h, const float* in, __nv_bfloat16* out, int64_t count, cudaStream_t st);
// active (or nullptr): one byte per run of `per_set` consecutive elements; runs with a zero byte are skipped
int32_t launch_adam_tick(gnnco_handle* h, int32_t* step_dev, float b1, float b2, float2* bias, cudaStream_t st);
int32_t launch_adam(gnnco_handle* h, float* W, float* m, float* v, const float* g, int64_t count, float lr, float b1,
                    float b2, float eps, float c1, float c2, const uint8_t* active, int64_t per_set, cudaStream_t st);

// ---- tc_gemm.cu : the same transform on the tensor cores (bf16, widths 64/128/256)
bool tc_transform_supported(int dtype, int K, int N);
// Y = act(A B_s^T) * row_scale with A [n x K] and B [sets x N x K], K contiguous in both; zeroed where
// relu_mask [n x N] <= 0 when that is given
int32_t launch_transform_tc(gnnco_handle* h, const void* A, const void* B, int64_t b_stride, void* Y, int K, int N,
                            bool relu, const float* row_scale, const void* relu_mask, bool backward, const void* dot_w,
                            int64_t dot_stride, float* dot_out, cudaStream_t st);
// the same by pairs of CTAs (cluster of two, one 256-row double tile per pair; tc_gemm2.cu)
bool tc_pair_transform_supported(gnnco_handle* h, int dtype, int K, int N);
// modes: relu (optionally bits_out = [Y > 0], one bit per element, and the row dot product), plain, or
// row_scale + mask_bits (result zeroed where the bit of the saved activation is clear)
int32_t launch_transform_tc_pair(gnnco_handle* h, const void* A, const void* B, int64_t b_stride, int32_t b_sets, void* Y,
                                 int K, int N, bool relu, const float* row_scale, const uint8_t* mask_bits,
                                 uint8_t* bits_out, bool backward, const void* dot_w, int64_t dot_stride, float* dot_out,
                                 cudaStream_t st);
bool aggregate_transform_pair_supported(gnnco_handle* h, int dtype, int K, int N);
// Fills `fs` (whose arrays the caller has carved: meta 2 x tiles, cluster_begin kFuseMaxClusters + 1, the four
// row tables and weights `tiles` each) for the double tiles p0 / pr (host copies of d_pair_row0 / d_pair_rows).
// Synchronises `st`.  Leaves fs.built false where the one-kernel layer cannot run on this device or graph.
int32_t build_fuse_set(gnnco_handle* h, const int32_t* d_pair_row0, const int32_t* d_pair_rows,
                       const std::vector<int32_t>& p0, const std::vector<int32_t>& pr, FuseSet& fs, cudaStream_t st);
int32_t launch_aggregate_transform_pair(gnnco_handle* h, const void* Hin, const void* B, int64_t b_stride, int32_t b_sets,
                                        void* Y, int K, int N, const float* row_scale, uint8_t* bits_out, const void* dot_w,
                                        int64_t dot_stride, float* dot_out, cudaStream_t st);
bool tc_pair_weight_grad_supported(gnnco_handle* h, int dtype, int K, int N);
int32_t launch_weight_grad_tc_pair(gnnco_handle* h, const void* A, const void* G, float* dW, float* scratch, int K, int N,
                                   cudaStream_t st);
bool tc_weight_grad_supported(int dtype, int K, int N);
int32_t launch_weight_grad_tc(gnnco_handle* h, const void* A, const void* G, float* dW, float* scratch, int K, int N,
                              cudaStream_t st);
// Wc[s][k][n] = bf16(W[s][k][n]) and Wt[s][n][k] = bf16(W[s][k][n]) in one pass over W
int32_t launch_cast_both_bf16(gnnco_handle* h, const float* W, __nv_bfloat16* Wc, __nv_bfloat16* Wt, int K, int N,
                              int32_t sets, cudaStream_t st);
// Adam on W [sets x K x N] that also writes both bf16 copies of the updated weights (for the next step)
bool adam_cast_both_supported(const float* W, const float* m, const float* v, const float* g, const __nv_bfloat16* Wc,
                              const __nv_bfloat16* Wt, int K, int N, int32_t sets);
int32_t launch_adam_cast_both(gnnco_handle* h, float* W, float* m, float* v, const float* g, __nv_bfloat16* Wc,
                              __nv_bfloat16* Wt, int K, int N, int32_t sets, float lr, float b1, float b2, float eps,
                              float c1, float c2, const uint8_t* active, cudaStream_t st);
// Wt[s][n][k] = bf16(W[s][k][n])
int32_t launch_cast_transpose_bf16(gnnco_handle* h, const float* W, __nv_bfloat16* Wt, int K, int N, int32_t sets,
                                   cudaStream_t st);

// ---- tc_gemm_f32.cu : tensor-core path for float32 features (operands split into three bf16 limbs)
bool tc_f32_transform_supported(int K, int N);
bool tc_f32_weight_grad_supported(int K, int N);
int32_t launch_transform_tc_f32(gnnco_handle* h, const void* A, const void* B_limbs, int64_t b_stride,
                                int64_t b_limb_stride, void* Y, int K, int N, bool relu, const float* row_scale,
                                const void* relu_mask, bool backward, const void* dot_w, int64_t dot_stride,
                                float* dot_out, cudaStream_t st);
int32_t launch_weight_grad_tc_f32(gnnco_handle* h, const void* A, const void* G, float* dW, float* scratch, int K,
                                  int N, cudaStream_t st);
// three bf16 limb copies of W [sets x K x N] (transposed: [sets x N x K]); limb l at out + l*sets*K*N
int32_t launch_cast_split3(gnnco_handle* h, const float* W, __nv_bfloat16* out, int K, int N, int32_t sets,
                           bool transpose, cudaStream_t st);

// ---- chain.cu : the width-1 part of the step
int32_t launch_output_forward(gnnco_handle* h, const float* u, float* z, float* p, cudaStream_t st);
int32_t launch_objective(gnnco_handle* h, const float* p, const float* pen, float alpha, float beta, float lambda,
                         float* item_loss, float* loss, float* t, cudaStream_t st);
// g = t + sum of t over the row ( = A_hat^T dz ); coef (optional) = inv_deg * g
int32_t launch_output_backward(gnnco_handle* h, const float* t, float* g, float* coef, cudaStream_t st);

// ---- decode.cu
int32_t launch_decode(gnnco_handle* h, const float* p, float thr, uint8_t* x, uint8_t* viol, int32_t* per_part,
                      gnnco_counts* counts, cudaStream_t st);
