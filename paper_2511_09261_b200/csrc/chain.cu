// The width-1 tail of the training step: output-layer aggregation and sigmoid (Eq. 4),
// the relaxed objective with its per-subgraph reduction (Eq. 5 plus the fine-tuning
// penalty of Section 3.3), and the gradient that enters the backward pass.
//
//   z_i  = inv_deg_i * (u_i + sum_{j in N(i)} u_j),   p_i = 1 / (1 + exp(-z_i))
//   q_i  = sum_{j in N(i)} p_j
//   loss_s = sum_{i in s} ( alpha/2 * p_i q_i + c_i p_i ),  c_i = -beta + lambda * pen_i
//   dz_i = (alpha q_i + c_i) p_i (1 - p_i),  t_i = inv_deg_i dz_i
//   g_i  = t_i + sum_{j in N(i)} t_j            ( = (A_hat^T dz)_i, adjacency symmetric )
//   coef_i = inv_deg_i g_i                      ( row scale of the next transposed aggregation )
//
// All three passes are one thread per row; a row longer than 32 entries is instead summed
// by its whole warp, and a row longer than 2048 entries by its whole block, so a hub cannot
// stall its warp for thousands of dependent loads (with few, large subgraphs a power-law graph
// has rows of tens of thousands of entries, which would otherwise be the tail of these short
// kernels).
#include "internal.cuh"

namespace {

// Rows of more than kLongRowDegree entries, when the step has scratch for them: their entry
// lists are cut into segments (table built with the graph), a pre-pass sums val over every
// segment with one block each, and the row's owner only adds its segments up -- a hub's work
// is spread over many blocks instead of stalling the block that holds it (hubs are neighbours
// in the node order, so one block can hold dozens of them).
struct LongRows {
  const float* seg_sum = nullptr;          // [segments] pre-pass result; nullptr: not in use
  const int32_t* rows = nullptr;           // ids of the long rows, ascending
  const int32_t* first_seg = nullptr;      // [count + 1]
  int32_t count = 0;
};

__global__ void __launch_bounds__(256) long_row_segment_sums(const float* __restrict__ val,
                                                             const int32_t* __restrict__ colidx,
                                                             const int32_t* __restrict__ seg_begin,
                                                             const int32_t* __restrict__ seg_end,
                                                             float* __restrict__ seg_sum) {
  __shared__ float warp_part[8];
  const int32_t a = seg_begin[blockIdx.x], b = seg_end[blockIdx.x];
  float part = 0.0f;
  int32_t k = a + threadIdx.x;
  for (; k + 768 < b; k += 1024) {          // four independent gathers in flight per thread
    const int32_t c0 = __ldg(colidx + k), c1 = __ldg(colidx + k + 256), c2 = __ldg(colidx + k + 512),
                  c3 = __ldg(colidx + k + 768);
    const float v0 = __ldg(val + c0), v1 = __ldg(val + c1), v2 = __ldg(val + c2), v3 = __ldg(val + c3);
    part += (v0 + v1) + (v2 + v3);
  }
  for (; k < b; k += 256) part += __ldg(val + __ldg(colidx + k));
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) part += __shfl_xor_sync(0xffffffffu, part, d);
  if ((threadIdx.x & 31) == 0) warp_part[threadIdx.x >> 5] = part;
  __syncthreads();
  if (threadIdx.x == 0) {
    float tot = 0.0f;
#pragma unroll
    for (int w = 0; w < 8; ++w) tot += warp_part[w];
    seg_sum[blockIdx.x] = tot;
  }
}

constexpr int kLongRow = 32;       // longer rows are summed by the row's warp
constexpr int kBlockRow = 2048;    // ... and rows longer than this by the whole block

// Sum of val[col] over the CSR row [r0, r1) of each thread's own row.  Must be called by all
// 256 threads of the block (it contains block barriers); threads without a row pass
// active = false.  Every row's sum is formed in an order that depends only on the row.
__device__ __forceinline__ float row_sum(const float* __restrict__ val, const int32_t* __restrict__ colidx, int32_t r0,
                                         int32_t r1, bool active, int64_t row, const LongRows& lr) {
  __shared__ int32_t s_pick, s_a, s_b;
  __shared__ float s_part[8];
  const int lane = threadIdx.x & 31;
  float sum = 0.0f;
  // already summed by the pre-pass: find the row in the sorted list and add its segments in order
  const bool is_pre = active && lr.seg_sum && (r1 - r0 > kLongRowDegree);
  if (is_pre) {
    int32_t lo = 0, hi = lr.count - 1;
    while (lo < hi) {
      const int32_t mid = (lo + hi) >> 1;
      if ((int64_t)__ldg(lr.rows + mid) < row) lo = mid + 1;
      else hi = mid;
    }
    for (int32_t sg = __ldg(lr.first_seg + lo); sg < __ldg(lr.first_seg + lo + 1); ++sg) sum += __ldg(lr.seg_sum + sg);
  }
  const bool is_block = active && !is_pre && (r1 - r0 > kBlockRow);
  const bool is_long = active && !is_pre && !is_block && (r1 - r0 > kLongRow);
  if (active && !is_pre && !is_long && !is_block) {
    int32_t k = r0;
    for (; k + 4 <= r1; k += 4) {           // four independent gathers in flight
      const int32_t c0 = __ldg(colidx + k), c1 = __ldg(colidx + k + 1), c2 = __ldg(colidx + k + 2),
                    c3 = __ldg(colidx + k + 3);
      const float v0 = __ldg(val + c0), v1 = __ldg(val + c1), v2 = __ldg(val + c2), v3 = __ldg(val + c3);
      sum += (v0 + v1) + (v2 + v3);
    }
    for (; k < r1; ++k) sum += __ldg(val + __ldg(colidx + k));
  }
  uint32_t todo = __ballot_sync(0xffffffffu, is_long);
  while (todo) {
    const int src = __ffs(todo) - 1;
    todo &= todo - 1;
    const int32_t a = __shfl_sync(0xffffffffu, r0, src), b = __shfl_sync(0xffffffffu, r1, src);
    float part = 0.0f;
    int32_t k = a + lane;
    for (; k + 96 < b; k += 128) {          // four independent gathers in flight per lane
      const int32_t c0 = __ldg(colidx + k), c1 = __ldg(colidx + k + 32), c2 = __ldg(colidx + k + 64),
                    c3 = __ldg(colidx + k + 96);
      const float v0 = __ldg(val + c0), v1 = __ldg(val + c1), v2 = __ldg(val + c2), v3 = __ldg(val + c3);
      part += (v0 + v1) + (v2 + v3);
    }
    for (; k < b; k += 32) part += __ldg(val + __ldg(colidx + k));
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) part += __shfl_xor_sync(0xffffffffu, part, d);
    if (lane == src) sum = part;
  }
  // rows for the whole block, one at a time, owner with the lowest thread index first
  bool pending = is_block;
  while (__syncthreads_or(pending)) {
    if (threadIdx.x == 0) s_pick = 256;
    __syncthreads();
    if (pending) atomicMin(&s_pick, (int32_t)threadIdx.x);
    __syncthreads();
    const int owner = s_pick;
    if ((int)threadIdx.x == owner) { s_a = r0; s_b = r1; }
    __syncthreads();
    const int32_t a = s_a, b = s_b;
    float part = 0.0f;
    int32_t k = a + threadIdx.x;
    for (; k + 768 < b; k += 1024) {        // four independent gathers in flight per thread
      const int32_t c0 = __ldg(colidx + k), c1 = __ldg(colidx + k + 256), c2 = __ldg(colidx + k + 512),
                    c3 = __ldg(colidx + k + 768);
      const float v0 = __ldg(val + c0), v1 = __ldg(val + c1), v2 = __ldg(val + c2), v3 = __ldg(val + c3);
      part += (v0 + v1) + (v2 + v3);
    }
    for (; k < b; k += 256) part += __ldg(val + __ldg(colidx + k));
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) part += __shfl_xor_sync(0xffffffffu, part, d);
    if (lane == 0) s_part[threadIdx.x >> 5] = part;
    __syncthreads();
    if ((int)threadIdx.x == owner) {
      float tot = 0.0f;
#pragma unroll
      for (int w = 0; w < 8; ++w) tot += s_part[w];
      sum = tot;
      pending = false;
    }
  }
  return sum;
}

__global__ void __launch_bounds__(256) output_forward(const float* __restrict__ u, const int32_t* __restrict__ rowptr,
                                                      const int32_t* __restrict__ colidx,
                                                      const float* __restrict__ inv_deg, float* __restrict__ z_out,
                                                      float* __restrict__ p_out, int64_t n, const LongRows lr,
                                                      const RowChunks rc) {
  int64_t i;
  const bool active = chunk_row(rc, (int64_t)blockIdx.x * blockDim.x + threadIdx.x, n, i);
  int32_t r0 = 0, r1 = 0;
  if (active) { r0 = rowptr[i]; r1 = rowptr[i + 1]; }
  float s = row_sum(u, colidx, r0, r1, active, i, lr);
  if (!active) return;
  const float z = inv_deg[i] * (u[i] + s);
  if (z_out) z_out[i] = z;
  p_out[i] = 1.0f / (1.0f + expf(-z));
}

// One block per work item (at most kItemRows consecutive rows of one subgraph).
__global__ void __launch_bounds__(256) objective_items(const float* __restrict__ p, const float* __restrict__ pen,
                                                       const int32_t* __restrict__ rowptr,
                                                       const int32_t* __restrict__ colidx,
                                                       const float* __restrict__ inv_deg,
                                                       const int32_t* __restrict__ item_row0,
                                                       const int32_t* __restrict__ item_row1, float alpha, float beta,
                                                       float lambda, float* __restrict__ item_loss,
                                                       float* __restrict__ t_out, const LongRows lr) {
  __shared__ float warp_part[8];
  const int32_t a = item_row0[blockIdx.x], b = item_row1[blockIdx.x];
  float local = 0.0f;
  for (int32_t base = a; base < b; base += 256) {      // uniform trip count across the block
    const int32_t i = base + threadIdx.x;
    const bool active = i < b;
    int32_t r0 = 0, r1 = 0;
    if (active) { r0 = rowptr[i]; r1 = rowptr[i + 1]; }
    const float q = row_sum(p, colidx, r0, r1, active, i, lr);
    if (active) {
      const float pi = p[i];
      const float c = -beta + (pen ? lambda * pen[i] : 0.0f);
      local += 0.5f * alpha * pi * q + c * pi;
      if (t_out) t_out[i] = inv_deg[i] * ((alpha * q + c) * pi * (1.0f - pi));
    }
  }
  // fixed-shape tree: lanes, then warps in order
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) local += __shfl_xor_sync(0xffffffffu, local, d);
  if ((threadIdx.x & 31) == 0) warp_part[threadIdx.x >> 5] = local;
  __syncthreads();
  if (threadIdx.x == 0) {
    float tot = 0.0f;
#pragma unroll
    for (int w = 0; w < 8; ++w) tot += warp_part[w];
    item_loss[blockIdx.x] = tot;
  }
}

__global__ void sum_items_per_subgraph(const float* __restrict__ item_loss, const int32_t* __restrict__ part_item_ptr,
                                       float* __restrict__ loss, int32_t S, const uint8_t* __restrict__ only) {
  const int32_t s = blockIdx.x * blockDim.x + threadIdx.x;
  if (s >= S) return;
  if (only && !only[s]) return;             // a step on the active subgraphs leaves the other losses alone
  float tot = 0.0f;
  for (int32_t k = part_item_ptr[s]; k < part_item_ptr[s + 1]; ++k) tot += item_loss[k];
  loss[s] = tot;
}

__global__ void __launch_bounds__(256) output_backward(const float* __restrict__ t, const int32_t* __restrict__ rowptr,
                                                       const int32_t* __restrict__ colidx,
                                                       const float* __restrict__ inv_deg, float* __restrict__ g,
                                                       float* __restrict__ coef, int64_t n, const LongRows lr,
                                                       const RowChunks rc) {
  int64_t i;
  const bool active = chunk_row(rc, (int64_t)blockIdx.x * blockDim.x + threadIdx.x, n, i);
  int32_t r0 = 0, r1 = 0;
  if (active) { r0 = rowptr[i]; r1 = rowptr[i + 1]; }
  float s = row_sum(t, colidx, r0, r1, active, i, lr);
  if (active) {
    const float gi = t[i] + s;
    g[i] = gi;
    if (coef) coef[i] = inv_deg[i] * gi;
  }
}

// Pre-pass over the long rows of `val` when the running step has scratch for it (the first
// n_long_segs floats of the aggregation's segment area, which is idle between aggregations).
LongRows long_rows_prepass(gnnco_handle* h, const float* val, cudaStream_t st) {
  LongRows lr;
  if (!h->agg_partial || h->n_long_segs == 0) return lr;
  long_row_segment_sums<<<h->n_long_segs, 256, 0, st>>>(val, h->colidx, h->seg_begin, h->seg_end, h->agg_partial);
  h->launches += 1;
  lr.seg_sum = h->agg_partial;
  lr.rows = h->long_rows;
  lr.first_seg = h->long_first_seg;
  lr.count = h->n_long;
  return lr;
}

}  // namespace

int32_t launch_output_forward(gnnco_handle* h, const float* u, float* z, float* p, cudaStream_t st) {
  ProfScope prof_(h, K_OUT_FWD, st);
  unsigned grid = (unsigned)((linear_rows(h) + 255) / 256);
  const LongRows lr = long_rows_prepass(h, u, st);
  output_forward<<<grid, 256, 0, st>>>(u, h->rowptr, h->colidx, h->inv_deg, z, p, h->n, lr, h->row_chunks);
  h->launches += 1;
  GNNCO_LAUNCH_CHECK();
  return GNNCO_OK;
}

int32_t launch_objective(gnnco_handle* h, const float* p, const float* pen, float alpha, float beta, float lambda,
                         float* item_loss, float* loss, float* t, cudaStream_t st) {
  ProfScope prof_(h, K_OBJECTIVE, st);
  const LongRows lr = long_rows_prepass(h, p, st);
  if (h->n_items > 0)
    objective_items<<<h->n_items, 256, 0, st>>>(p, pen, h->rowptr, h->colidx, h->inv_deg, h->item_row0, h->item_row1,
                                                alpha, beta, lambda, item_loss, t, lr);
  sum_items_per_subgraph<<<(h->S + 255) / 256, 256, 0, st>>>(item_loss, h->part_item_ptr, loss, h->S,
                                                             h->row_chunks.row0 ? h->plan_active : nullptr);
  h->launches += 2;
  GNNCO_LAUNCH_CHECK();
  return GNNCO_OK;
}

int32_t launch_output_backward(gnnco_handle* h, const float* t, float* g, float* coef, cudaStream_t st) {
  ProfScope prof_(h, K_OUT_BWD, st);
  unsigned grid = (unsigned)((linear_rows(h) + 255) / 256);
  const LongRows lr = long_rows_prepass(h, t, st);
  output_backward<<<grid, 256, 0, st>>>(t, h->rowptr, h->colidx, h->inv_deg, g, coef, h->n, lr, h->row_chunks);
  h->launches += 1;
  GNNCO_LAUNCH_CHECK();
  return GNNCO_OK;
}

// ------------------------------------------------------------------------------------
// Objective evaluation for callers that cannot allocate device memory (see gnnco.h).
// The per-item partial sums, which launch_objective keeps in the caller's work area, live
// here in a fixed device array that is part of the library image.
namespace {

static __device__ __align__(256) float g_static_item_loss[GNNCO_STATIC_OBJECTIVE_MAX_ITEMS];

constexpr int kMaxDevices = 64;
float* g_static_item_loss_addr[kMaxDevices] = {nullptr};   // device address of the array, per device

// In host code the array's name is only a handle for the runtime, not a device address; the
// address a kernel can use has to be asked for, once per device, with that device current.
int32_t static_item_loss_address(float** out) {
  int dev = -1;
  GNNCO_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return GNNCO_UNSUPPORTED;
  if (!g_static_item_loss_addr[dev]) {
    void* ptr = nullptr;
    GNNCO_CUDA_TRY(cudaGetSymbolAddress(&ptr, g_static_item_loss));
    if (!ptr) return GNNCO_CUDA_ERROR;
    g_static_item_loss_addr[dev] = static_cast<float*>(ptr);
  }
  *out = g_static_item_loss_addr[dev];
  return GNNCO_OK;
}

}  // namespace

extern "C" int32_t gnnco_objective_static(gnnco_handle* h, const float* p, const gnnco_objective* obj, float* loss,
                                         void* stream) {
  if (!h || !p || !obj || !loss) return GNNCO_INVALID_ARGUMENT;
  if (h->n_items > GNNCO_STATIC_OBJECTIVE_MAX_ITEMS) return GNNCO_WORKSPACE_TOO_SMALL;
  int dev = -1;
  GNNCO_CUDA_TRY(cudaGetDevice(&dev));
  if (dev != h->device) return GNNCO_INVALID_ARGUMENT;
  float* item_loss = nullptr;
  int32_t rc = static_item_loss_address(&item_loss);
  if (rc != GNNCO_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // every slot that is read below is written first by objective_items; the clear only makes
  // sure nothing of an earlier call can be mistaken for a result
  if (h->n_items > 0) GNNCO_CUDA_TRY(cudaMemsetAsync(item_loss, 0, (size_t)h->n_items * sizeof(float), st));
  if (h->n_items > 0)
    objective_items<<<h->n_items, 256, 0, st>>>(p, obj->pen, h->rowptr, h->colidx, h->inv_deg, h->item_row0,
                                                h->item_row1, obj->alpha, obj->beta, obj->lambda, item_loss, nullptr,
                                                LongRows{});
  sum_items_per_subgraph<<<(h->S + 255) / 256, 256, 0, st>>>(item_loss, h->part_item_ptr, loss, h->S, nullptr);
  h->launches += 2;
  GNNCO_LAUNCH_CHECK();
  return GNNCO_OK;
}
