// Glue between decoding and the fine-tuning steps (Section 3.3; Algorithm 1, Stage 3):
// the violated boundary edges are compacted into the conflict set C in ascending order,
// every conflict gets a base action (which of its two endpoints is pushed below the
// threshold), and the chosen nodes become the node list of the penalty term plus the list
// of subgraphs whose models are fine-tuned.  Integer work only: results are exact and
// independent of scheduling (ordered compaction by count -> scan -> scatter; idempotent
// stores and one integer counter in the scatter of actions).
#include "internal.cuh"

namespace {

constexpr int kCompactThreads = 256;
constexpr int kEdgesPerThread = 16;
constexpr int kTileEdges = kCompactThreads * kEdgesPerThread;   // 4096 flags per block

// bit k of the result = flag of edge e0 + k is non-zero, for the 16 edges from e0 on
__device__ __forceinline__ uint32_t load_flags16(const uint8_t* __restrict__ viol, int64_t e0, int64_t E_b,
                                                 bool aligned) {
  uint32_t bits = 0;
  if (aligned && e0 + kEdgesPerThread <= E_b) {
    const uint4 q = __ldg(reinterpret_cast<const uint4*>(viol + e0));
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int b = 0; b < 4; ++b) bits |= ((w[i] >> (8 * b)) & 0xffu) ? (1u << (4 * i + b)) : 0u;
  } else {
    for (int k = 0; k < kEdgesPerThread; ++k)
      if (e0 + k < E_b && viol[e0 + k]) bits |= 1u << k;
  }
  return bits;
}

// exclusive prefix of `value` over the block's threads; *total receives the block sum
__device__ __forceinline__ int32_t block_exclusive(int32_t value, int32_t* total) {
  __shared__ int32_t warp_sum[kCompactThreads / 32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int32_t incl = value;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const int32_t up = __shfl_up_sync(0xffffffffu, incl, d);
    if (lane >= d) incl += up;
  }
  if (lane == 31) warp_sum[warp] = incl;
  __syncthreads();
  int32_t before = 0, all = 0;
#pragma unroll
  for (int w = 0; w < kCompactThreads / 32; ++w) {
    const int32_t s = warp_sum[w];
    before += w < warp ? s : 0;
    all += s;
  }
  *total = all;
  return before + incl - value;
}

__global__ void __launch_bounds__(kCompactThreads) count_conflicts_kernel(const uint8_t* __restrict__ viol,
                                                                          int64_t E_b, bool aligned,
                                                                          int32_t* __restrict__ tile_count) {
  const int64_t e0 = (int64_t)blockIdx.x * kTileEdges + (int64_t)threadIdx.x * kEdgesPerThread;
  const int32_t mine = e0 < E_b ? __popc(load_flags16(viol, e0, E_b, aligned)) : 0;
  int32_t total;
  block_exclusive(mine, &total);
  if (threadIdx.x == 0) tile_count[blockIdx.x] = total;
}

// in place: tile_count -> exclusive offsets; *count = total (one block)
__global__ void __launch_bounds__(kCompactThreads) scan_tile_counts_kernel(int32_t* __restrict__ tile_count,
                                                                           int32_t tiles, int32_t* __restrict__ count) {
  int32_t carry = 0;
  for (int32_t base = 0; base < tiles; base += kCompactThreads) {
    const int32_t t = base + threadIdx.x;
    const int32_t mine = t < tiles ? tile_count[t] : 0;
    int32_t total;
    const int32_t excl = block_exclusive(mine, &total);
    if (t < tiles) tile_count[t] = carry + excl;
    carry += total;
    __syncthreads();   // warp_sum is reused by the next round
  }
  if (threadIdx.x == 0) *count = carry;
}

__global__ void __launch_bounds__(kCompactThreads) scatter_conflicts_kernel(
    const uint8_t* __restrict__ viol, int64_t E_b, bool aligned, const int32_t* __restrict__ tile_offset,
    const int32_t* __restrict__ bnd_u, const int32_t* __restrict__ bnd_v, const float* __restrict__ p,
    int32_t* __restrict__ conflict_idx, uint8_t* __restrict__ action) {
  const int64_t e0 = (int64_t)blockIdx.x * kTileEdges + (int64_t)threadIdx.x * kEdgesPerThread;
  uint32_t bits = e0 < E_b ? load_flags16(viol, e0, E_b, aligned) : 0u;
  int32_t total;
  int32_t slot = tile_offset[blockIdx.x] + block_exclusive(__popc(bits), &total);
  while (bits) {
    const int k = __ffs(bits) - 1;
    bits &= bits - 1;
    const int64_t e = e0 + k;
    conflict_idx[slot] = (int32_t)e;
    if (action) {
      const float pu = __ldg(p + __ldg(bnd_u + e)), pv = __ldg(p + __ldg(bnd_v + e));
      action[slot] = pu < pv ? 0 : 1;
    }
    ++slot;
  }
}

__global__ void __launch_bounds__(256) apply_actions_kernel(const int32_t* __restrict__ conflict_idx,
                                                            const uint8_t* __restrict__ action,
                                                            const int32_t* __restrict__ count,
                                                            const int32_t* __restrict__ bnd_u,
                                                            const int32_t* __restrict__ bnd_v,
                                                            const int32_t* __restrict__ node_part, int64_t E_b,
                                                            float* __restrict__ pen, uint8_t* __restrict__ active,
                                                            int32_t* __restrict__ chosen) {
  const int32_t C = *count;
  int32_t fresh = 0;
  for (int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; c < C; c += (int64_t)gridDim.x * blockDim.x) {
    const int32_t e = conflict_idx[c];
    if (e < 0 || e >= E_b) continue;   // a caller-made list with a bad entry touches nothing
    const int32_t node = action[c] ? bnd_v[e] : bnd_u[e];
    // 1.0f as a bit pattern; the first writer of a node sees the cleared word
    const unsigned old = atomicExch(reinterpret_cast<unsigned*>(pen + node), 0x3f800000u);
    fresh += old == 0u ? 1 : 0;
    active[node_part[node]] = 1;
  }
  if (chosen) {
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) fresh += __shfl_xor_sync(0xffffffffu, fresh, d);
    if ((threadIdx.x & 31) == 0 && fresh) atomicAdd(chosen, fresh);
  }
}

// x[i] <- 0 for every chosen node (pen[i] != 0); counts the selected nodes that were removed
__global__ void __launch_bounds__(256) repair_kernel(const float* __restrict__ pen, uint8_t* __restrict__ x, int64_t n,
                                                     int32_t* __restrict__ removed) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  int32_t hit = 0;
  if (i < n && pen[i] != 0.0f && x[i]) {
    x[i] = 0;
    hit = 1;
  }
  if (removed) {
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) hit += __shfl_xor_sync(0xffffffffu, hit, d);
    if ((threadIdx.x & 31) == 0 && hit) atomicAdd(removed, hit);
  }
}

inline int32_t tiles_for(int64_t E_b) { return (int32_t)((E_b + kTileEdges - 1) / kTileEdges); }

}  // namespace

extern "C" int32_t gnnco_conflict_workspace_bytes(const gnnco_handle* h, size_t* bytes) {
  if (!h || !bytes) return GNNCO_INVALID_ARGUMENT;
  *bytes = align_up((size_t)(tiles_for(h->E_b) + 1) * sizeof(int32_t));
  return GNNCO_OK;
}

extern "C" int32_t gnnco_conflict_actions(gnnco_handle* h, const uint8_t* viol, const float* p, int32_t* conflict_idx,
                                         uint8_t* action, int32_t* count, void* ws, size_t ws_bytes, void* stream) {
  if (!h || !count) return GNNCO_INVALID_ARGUMENT;
  if (action && !p) return GNNCO_INVALID_ARGUMENT;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  ProfScope prof_(h, K_STAGE3, st);
  if (h->E_b == 0) {
    GNNCO_CUDA_TRY(cudaMemsetAsync(count, 0, sizeof(int32_t), st));
    return GNNCO_OK;
  }
  if (!viol || !conflict_idx || !ws) return GNNCO_INVALID_ARGUMENT;
  const int32_t tiles = tiles_for(h->E_b);
  if (ws_bytes < (size_t)(tiles + 1) * sizeof(int32_t) || ((uintptr_t)ws & 3)) return GNNCO_WORKSPACE_TOO_SMALL;
  int32_t* tile_count = static_cast<int32_t*>(ws);
  const bool aligned = ((uintptr_t)viol & 15) == 0;
  count_conflicts_kernel<<<tiles, kCompactThreads, 0, st>>>(viol, h->E_b, aligned, tile_count);
  scan_tile_counts_kernel<<<1, kCompactThreads, 0, st>>>(tile_count, tiles, count);
  scatter_conflicts_kernel<<<tiles, kCompactThreads, 0, st>>>(viol, h->E_b, aligned, tile_count, h->bnd_u, h->bnd_v, p,
                                                              conflict_idx, action);
  h->launches += 3;
  GNNCO_LAUNCH_CHECK();
  return GNNCO_OK;
}

extern "C" int32_t gnnco_apply_actions(gnnco_handle* h, const int32_t* conflict_idx, const uint8_t* action,
                                      const int32_t* count, float* pen, uint8_t* active, int32_t* chosen,
                                      void* stream) {
  if (!h || !pen || !active || !count) return GNNCO_INVALID_ARGUMENT;
  if (h->E_b > 0 && (!conflict_idx || !action)) return GNNCO_INVALID_ARGUMENT;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  ProfScope prof_(h, K_STAGE3, st);
  GNNCO_CUDA_TRY(cudaMemsetAsync(pen, 0, (size_t)h->n * sizeof(float), st));
  GNNCO_CUDA_TRY(cudaMemsetAsync(active, 0, (size_t)h->S, st));
  if (chosen) GNNCO_CUDA_TRY(cudaMemsetAsync(chosen, 0, sizeof(int32_t), st));
  if (h->E_b == 0) return GNNCO_OK;
  const int64_t want = (h->E_b + 255) / 256, cap = (int64_t)h->sm_count * 8;
  const unsigned grid = (unsigned)(want < cap ? want : cap);
  apply_actions_kernel<<<grid, 256, 0, st>>>(conflict_idx, action, count, h->bnd_u, h->bnd_v, h->node_part, h->E_b,
                                             pen, active, chosen);
  h->launches += 1;
  GNNCO_LAUNCH_CHECK();
  return GNNCO_OK;
}

extern "C" int32_t gnnco_repair_boundary(gnnco_handle* h, const float* pen, uint8_t* x, int32_t* removed, void* stream) {
  if (!h || !pen || !x) return GNNCO_INVALID_ARGUMENT;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  ProfScope prof_(h, K_STAGE3, st);
  if (removed) GNNCO_CUDA_TRY(cudaMemsetAsync(removed, 0, sizeof(int32_t), st));
  repair_kernel<<<(unsigned)((h->n + 255) / 256), 256, 0, st>>>(pen, x, h->n, removed);
  h->launches += 1;
  GNNCO_LAUNCH_CHECK();
  return GNNCO_OK;
}
