// Quality of the loaded partition in the terms of Section 3.1 (the quantities of Eq. 1): per
// subgraph the number of internal edges and Sigma_tot, the degree sum of its nodes, and the
// modularity  Q = sum_s [ Sigma_in(s)/2m - (Sigma_tot(s)/2m)^2 ]  with Sigma_in = 2 * internal
// edges and m = all edges.  Everything comes from what gnnco_partition_load built: a subgraph's
// internal edges are its slice of the CSR, and the degrees its nodes have outside it are the
// endpoints of the boundary list.  The integer parts are exact (integer atomics); Q is summed in
// float64 by one block in a fixed order.
#include "internal.cuh"

namespace {

__global__ void __launch_bounds__(256) quality_internal_kernel(const int32_t* __restrict__ part_ptr,
                                                               const int32_t* __restrict__ rowptr, int32_t S,
                                                               long long* __restrict__ in_edges,
                                                               unsigned long long* __restrict__ tot) {
  const int32_t s = blockIdx.x * blockDim.x + threadIdx.x;
  if (s >= S) return;
  const long long entries = (long long)rowptr[part_ptr[s + 1]] - (long long)rowptr[part_ptr[s]];
  in_edges[s] = entries / 2;                 // the CSR holds both directions of every internal edge
  tot[s] = (unsigned long long)entries;      // boundary endpoints are added by the next kernel
}

__global__ void __launch_bounds__(256) quality_boundary_kernel(const int32_t* __restrict__ bnd_u,
                                                               const int32_t* __restrict__ bnd_v,
                                                               const int32_t* __restrict__ node_part, int64_t E_b,
                                                               unsigned long long* __restrict__ tot) {
  const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int lane = threadIdx.x & 31;
  int32_t su = -1, sv = -1;
  if (e < E_b) {
    su = node_part[bnd_u[e]];
    sv = node_part[bnd_v[e]];
  }
  // the list is sorted by its lower endpoint: neighbouring lanes mostly share a subgraph
  uint32_t peers = __match_any_sync(0xffffffffu, su);
  if (su >= 0 && lane == __ffs(peers) - 1) atomicAdd(tot + su, (unsigned long long)__popc(peers));
  peers = __match_any_sync(0xffffffffu, sv);
  if (sv >= 0 && lane == __ffs(peers) - 1) atomicAdd(tot + sv, (unsigned long long)__popc(peers));
}

__global__ void __launch_bounds__(256) quality_modularity_kernel(const long long* __restrict__ in_edges,
                                                                 const unsigned long long* __restrict__ tot, int32_t S,
                                                                 long long E, double* __restrict__ Q) {
  __shared__ double warp_part[8];
  double local = 0.0;
  if (E > 0) {
    const double two_m = 2.0 * (double)E;
    for (int32_t s = threadIdx.x; s < S; s += 256) {
      const double share = (double)tot[s] / two_m;
      local += 2.0 * (double)in_edges[s] / two_m - share * share;
    }
  }
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) local += __shfl_xor_sync(0xffffffffu, local, d);
  if ((threadIdx.x & 31) == 0) warp_part[threadIdx.x >> 5] = local;
  __syncthreads();
  if (threadIdx.x == 0) {
    double q = 0.0;
#pragma unroll
    for (int w = 0; w < 8; ++w) q += warp_part[w];
    *Q = q;
  }
}

}  // namespace

extern "C" int32_t gnnco_partition_quality(gnnco_handle* h, int64_t* in_edges, int64_t* tot, double* Q, void* stream) {
  if (!h || !in_edges || !tot || !Q) return GNNCO_INVALID_ARGUMENT;
  if (((uintptr_t)in_edges | (uintptr_t)tot | (uintptr_t)Q) & 7) return GNNCO_INVALID_ARGUMENT;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  long long* ie = reinterpret_cast<long long*>(in_edges);
  unsigned long long* tt = reinterpret_cast<unsigned long long*>(tot);
  quality_internal_kernel<<<(h->S + 255) / 256, 256, 0, st>>>(h->part_ptr, h->rowptr, h->S, ie, tt);
  h->launches += 1;
  if (h->E_b > 0) {
    quality_boundary_kernel<<<(unsigned)((h->E_b + 255) / 256), 256, 0, st>>>(h->bnd_u, h->bnd_v, h->node_part, h->E_b, tt);
    h->launches += 1;
  }
  quality_modularity_kernel<<<1, 256, 0, st>>>(ie, tt, h->S, (long long)h->E, Q);
  h->launches += 1;
  GNNCO_LAUNCH_CHECK();
  return GNNCO_OK;
}
