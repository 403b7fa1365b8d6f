// Thresholded decoding and integer conflict counts (Section 3.3: probabilities are
// binarised at 0.5 with ">=", and a cross edge whose two ends are both selected is a
// conflict; Section 4.1: set size and conflicts are the reported metrics).  All outputs
// are integers, accumulated with integer atomics, hence exact and order-independent.
#include "internal.cuh"

namespace {

__device__ __forceinline__ void block_add_u64(unsigned long long local, unsigned long long* dst) {
  __shared__ unsigned long long warp_part[8];
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) local += __shfl_xor_sync(0xffffffffu, local, d);
  if ((threadIdx.x & 31) == 0) warp_part[threadIdx.x >> 5] = local;
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned long long tot = 0;
#pragma unroll
    for (int w = 0; w < 8; ++w) tot += warp_part[w];
    if (tot) atomicAdd(dst, tot);
  }
}

__global__ void __launch_bounds__(256) threshold_kernel(const float* __restrict__ p, float thr, uint8_t* __restrict__ x,
                                                        int64_t n, unsigned long long* set_size) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  unsigned long long sel = 0;
  if (i < n) {
    sel = p[i] >= thr ? 1 : 0;
    x[i] = (uint8_t)sel;
  }
  block_add_u64(sel, set_size);
}

// intra edges with both ends selected, each counted from its lower endpoint
__global__ void __launch_bounds__(256) intra_conflicts_kernel(const uint8_t* __restrict__ x,
                                                              const int32_t* __restrict__ rowptr,
                                                              const int32_t* __restrict__ colidx, int64_t n,
                                                              unsigned long long* intra) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int lane = threadIdx.x & 31;
  int32_t r0 = 0, r1 = 0;
  bool sel = false;
  if (i < n) { sel = x[i] != 0; if (sel) { r0 = rowptr[i]; r1 = rowptr[i + 1]; } }
  const bool is_long = r1 - r0 > 32;
  unsigned long long cnt = 0;
  if (sel && !is_long)
    for (int32_t k = r0; k < r1; ++k) { int32_t j = colidx[k]; cnt += (j > i && x[j]) ? 1 : 0; }
  uint32_t todo = __ballot_sync(0xffffffffu, is_long);
  while (todo) {
    const int src = __ffs(todo) - 1;
    todo &= todo - 1;
    const int32_t a = __shfl_sync(0xffffffffu, r0, src), b = __shfl_sync(0xffffffffu, r1, src);
    const int64_t row = (i - lane) + src;
    for (int32_t k = a + lane; k < b; k += 32) { int32_t j = colidx[k]; cnt += (j > row && x[j]) ? 1 : 0; }
  }
  block_add_u64(cnt, intra);
}

// Four consecutive boundary edges per thread: the eight endpoint bits are gathered together
// (they are the kernel's only dependent loads), endpoints and flags move as 16- and 4-byte words.
__global__ void __launch_bounds__(256) boundary_conflicts_kernel(const uint8_t* __restrict__ x,
                                                                 const int32_t* __restrict__ bnd_u,
                                                                 const int32_t* __restrict__ bnd_v,
                                                                 const int32_t* __restrict__ node_part, int64_t E_b,
                                                                 uint8_t* __restrict__ viol,
                                                                 int32_t* __restrict__ per_part,
                                                                 unsigned long long* total, int vectorised) {
  const int64_t e0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
  const int lane = threadIdx.x & 31;
  int32_t a[4], b[4];
  if (vectorised && e0 + 4 <= E_b) {
    const int4 ua = __ldg(reinterpret_cast<const int4*>(bnd_u + e0)), va = __ldg(reinterpret_cast<const int4*>(bnd_v + e0));
    a[0] = ua.x; a[1] = ua.y; a[2] = ua.z; a[3] = ua.w;
    b[0] = va.x; b[1] = va.y; b[2] = va.z; b[3] = va.w;
  } else {
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      a[k] = e0 + k < E_b ? bnd_u[e0 + k] : -1;
      b[k] = e0 + k < E_b ? bnd_v[e0 + k] : -1;
    }
  }
  uint8_t xa[4], xb[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    xa[k] = a[k] >= 0 ? x[a[k]] : 0;
    xb[k] = b[k] >= 0 ? x[b[k]] : 0;
  }
  unsigned long long count = 0;
  uint8_t v[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    v[k] = (xa[k] & xb[k]) ? 1 : 0;
    count += v[k];
  }
  if (viol) {
    if (vectorised && e0 + 4 <= E_b) {
      *reinterpret_cast<uchar4*>(viol + e0) = make_uchar4(v[0], v[1], v[2], v[3]);
    } else {
#pragma unroll
      for (int k = 0; k < 4; ++k)
        if (e0 + k < E_b) viol[e0 + k] = v[k];
    }
  }
  if (per_part) {
    // edges are sorted by their lower endpoint, so neighbouring lanes mostly share su:
    // one atomic per distinct subgraph in the warp and edge slot
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int32_t su = v[k] ? node_part[a[k]] : -1, sv = v[k] ? node_part[b[k]] : -1;
      uint32_t peers = __match_any_sync(0xffffffffu, su);
      if (su >= 0 && lane == __ffs(peers) - 1) atomicAdd(per_part + su, __popc(peers));
      peers = __match_any_sync(0xffffffffu, sv);
      if (sv >= 0 && lane == __ffs(peers) - 1) atomicAdd(per_part + sv, __popc(peers));
    }
  }
  block_add_u64(count, total);
}

}  // namespace

int32_t launch_decode(gnnco_handle* h, const float* p, float thr, uint8_t* x, uint8_t* viol, int32_t* per_part,
                      gnnco_counts* counts, cudaStream_t st) {
  ProfScope prof_(h, K_DECODE, st);
  GNNCO_CUDA_TRY(cudaMemsetAsync(counts, 0, sizeof(gnnco_counts), st));
  if (per_part) GNNCO_CUDA_TRY(cudaMemsetAsync(per_part, 0, (size_t)h->S * sizeof(int32_t), st));
  unsigned long long* c = reinterpret_cast<unsigned long long*>(counts);
  unsigned grid = (unsigned)((h->n + 255) / 256);
  threshold_kernel<<<grid, 256, 0, st>>>(p, thr, x, h->n, c + 0);
  intra_conflicts_kernel<<<grid, 256, 0, st>>>(x, h->rowptr, h->colidx, h->n, c + 1);
  h->launches += 2;
  if (h->E_b > 0) {
    unsigned gb = (unsigned)((h->E_b + 1023) / 1024);
    const int vectorised = (((uintptr_t)h->bnd_u | (uintptr_t)h->bnd_v) & 15) == 0 && ((uintptr_t)viol & 3) == 0;
    boundary_conflicts_kernel<<<gb, 256, 0, st>>>(x, h->bnd_u, h->bnd_v, h->node_part, h->E_b, viol, per_part, c + 2,
                                                  vectorised);
    h->launches += 1;
  }
  GNNCO_LAUNCH_CHECK();
  return GNNCO_OK;
}

extern "C" int32_t gnnco_decode_boundary(const gnnco_handle* h, const float* p, float threshold, uint8_t* x,
                                        uint8_t* viol, int32_t* per_part, gnnco_counts* counts, void* stream) {
  if (!h || !p || !x || !counts) return GNNCO_INVALID_ARGUMENT;
  if ((uintptr_t)counts & 7) return GNNCO_INVALID_ARGUMENT;
  return launch_decode(const_cast<gnnco_handle*>(h), p, threshold, x, viol, per_part, counts,
                       static_cast<cudaStream_t>(stream));
}
