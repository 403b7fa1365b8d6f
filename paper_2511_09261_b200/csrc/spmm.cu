// Neighbour aggregation over the block-diagonal CSR (Eq. 3's mean over a node and its
// intra-subgraph neighbours), and its transpose for the backward pass.
//
//   out[i,:] = scale[i] * ( in[i,:] + sum_{j in row i} in[j,:] )        (optionally masked)
//
// Forward:  scale = 1/(deg+1)  gives  M = A_hat H.
// Backward: the intra adjacency is symmetric, so A_hat^T G = (A + I)(D^-1 G); the
// producer of G folds D^-1 in, and this kernel runs with scale = NULL.  With `mask` the
// result is zeroed where mask[i,f] <= 0 (ReLU derivative taken from the saved activation).
//
// Mapping: a group of LPR lanes owns one row; every lane keeps VPL 16-byte vectors of the
// row in float32 registers, so a feature row is read with 128-bit loads and each
// neighbour row is one fully coalesced request.  Rows of one subgraph are adjacent in
// memory and are processed by neighbouring warps, so repeated neighbour reads hit in L2.
#include "internal.cuh"

namespace {

template <typename T>
struct Vec;
template <>
struct Vec<float> {
  static constexpr int N = 4;
  __device__ static void load(const float* p, float (&f)[4]) {
    float4 v = __ldg(reinterpret_cast<const float4*>(p));
    f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w;
  }
  __device__ static void store(float* p, const float (&f)[4]) {
    *reinterpret_cast<float4*>(p) = make_float4(f[0], f[1], f[2], f[3]);
  }
};
template <>
struct Vec<__nv_bfloat16> {
  static constexpr int N = 8;
  __device__ static void load(const __nv_bfloat16* p, float (&f)[8]) {
    uint4 v = __ldg(reinterpret_cast<const uint4*>(p));
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      f[2 * k] = __uint_as_float(w[k] << 16);
      f[2 * k + 1] = __uint_as_float(w[k] & 0xffff0000u);
    }
  }
  __device__ static void store(__nv_bfloat16* p, const float (&f)[8]) {
    uint32_t w[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      __nv_bfloat162 b = __floats2bfloat162_rn(f[2 * k], f[2 * k + 1]);
      w[k] = *reinterpret_cast<uint32_t*>(&b);
    }
    *reinterpret_cast<uint4*>(p) = make_uint4(w[0], w[1], w[2], w[3]);
  }
};

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ void from_f32(float& d, float x) { d = x; }
__device__ __forceinline__ void from_f32(__nv_bfloat16& d, float x) { d = __float2bfloat16_rn(x); }

// LPR lanes per row, VPL vectors per lane: row width F = LPR * VPL * Vec<T>::N elements.
template <typename T, int LPR, int VPL>
__global__ void __launch_bounds__(256) aggregate_vec(const T* __restrict__ in, T* __restrict__ out,
                                                     const int32_t* __restrict__ rowptr,
                                                     const int32_t* __restrict__ colidx,
                                                     const float* __restrict__ scale, const T* __restrict__ mask,
                                                     int64_t n, int F) {
  constexpr int VN = Vec<T>::N;
  constexpr int ROWS_PER_BLOCK = 256 / LPR;
  const int sub = threadIdx.x % LPR;
  const int64_t row = (int64_t)blockIdx.x * ROWS_PER_BLOCK + threadIdx.x / LPR;
  if (row >= n) return;
  const int32_t r0 = __ldg(rowptr + row), r1 = __ldg(rowptr + row + 1);
  float acc[VPL][VN];
#pragma unroll
  for (int v = 0; v < VPL; ++v) Vec<T>::load(in + row * F + (v * LPR + sub) * VN, acc[v]);
  int32_t k = r0;
  for (; k + 4 <= r1; k += 4) {
    int32_t j[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) j[u] = __ldg(colidx + k + u);
    float t[4][VPL][VN];
#pragma unroll
    for (int u = 0; u < 4; ++u)
#pragma unroll
      for (int v = 0; v < VPL; ++v) Vec<T>::load(in + (int64_t)j[u] * F + (v * LPR + sub) * VN, t[u][v]);
#pragma unroll
    for (int u = 0; u < 4; ++u)
#pragma unroll
      for (int v = 0; v < VPL; ++v)
#pragma unroll
        for (int e = 0; e < VN; ++e) acc[v][e] += t[u][v][e];
  }
  for (; k < r1; ++k) {
    const int64_t j = __ldg(colidx + k);
#pragma unroll
    for (int v = 0; v < VPL; ++v) {
      float t[VN];
      Vec<T>::load(in + j * F + (v * LPR + sub) * VN, t);
#pragma unroll
      for (int e = 0; e < VN; ++e) acc[v][e] += t[e];
    }
  }
  const float s = scale ? __ldg(scale + row) : 1.0f;
#pragma unroll
  for (int v = 0; v < VPL; ++v) {
    const int64_t off = row * F + (v * LPR + sub) * VN;
    if (mask) {
      float m[VN];
      Vec<T>::load(mask + off, m);
#pragma unroll
      for (int e = 0; e < VN; ++e) acc[v][e] = m[e] > 0.0f ? acc[v][e] * s : 0.0f;
    } else {
#pragma unroll
      for (int e = 0; e < VN; ++e) acc[v][e] *= s;
    }
    Vec<T>::store(out + off, acc[v]);
  }
}

// Any width: one warp per row, lanes stride over the features with scalar accesses.
template <typename T>
__global__ void __launch_bounds__(256) aggregate_any(const T* __restrict__ in, T* __restrict__ out,
                                                     const int32_t* __restrict__ rowptr,
                                                     const int32_t* __restrict__ colidx,
                                                     const float* __restrict__ scale, const T* __restrict__ mask,
                                                     int64_t n, int F) {
  const int lane = threadIdx.x & 31;
  const int64_t row = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  if (row >= n) return;
  const int32_t r0 = rowptr[row], r1 = rowptr[row + 1];
  const float s = scale ? scale[row] : 1.0f;
  for (int f = lane; f < F; f += 32) {
    float acc = to_f32(in[row * F + f]);
    for (int32_t k = r0; k < r1; ++k) acc += to_f32(in[(int64_t)colidx[k] * F + f]);
    acc *= s;
    if (mask && !(to_f32(mask[row * F + f]) > 0.0f)) acc = 0.0f;
    from_f32(out[row * F + f], acc);
  }
}

template <typename T, int LPR, int VPL>
void launch_vec(const T* in, T* out, const gnnco_handle* h, const float* scale, const T* mask, int F,
                cudaStream_t st) {
  constexpr int ROWS_PER_BLOCK = 256 / LPR;
  unsigned grid = (unsigned)((h->n + ROWS_PER_BLOCK - 1) / ROWS_PER_BLOCK);
  aggregate_vec<T, LPR, VPL><<<grid, 256, 0, st>>>(in, out, h->rowptr, h->colidx, scale, mask, h->n, F);
}

template <typename T>
int32_t aggregate_typed(gnnco_handle* h, const T* in, T* out, int F, const float* scale, const T* mask,
                        cudaStream_t st) {
  constexpr int VN = Vec<T>::N;
  bool aligned = !((uintptr_t)in & 15) && !((uintptr_t)out & 15) && !((uintptr_t)mask & 15);
  int vecs = F / VN;
  bool done = false;
  if (aligned && F % VN == 0) {
    done = true;
    switch (vecs) {
      case 1: launch_vec<T, 1, 1>(in, out, h, scale, mask, F, st); break;
      case 2: launch_vec<T, 2, 1>(in, out, h, scale, mask, F, st); break;
      case 4: launch_vec<T, 4, 1>(in, out, h, scale, mask, F, st); break;
      case 8: launch_vec<T, 8, 1>(in, out, h, scale, mask, F, st); break;
      case 16: launch_vec<T, 16, 1>(in, out, h, scale, mask, F, st); break;
      case 32: launch_vec<T, 32, 1>(in, out, h, scale, mask, F, st); break;
      case 64: launch_vec<T, 32, 2>(in, out, h, scale, mask, F, st); break;
      default: done = false;
    }
  }
  if (!done) {
    unsigned grid = (unsigned)((h->n + 7) / 8);
    aggregate_any<T><<<grid, 256, 0, st>>>(in, out, h->rowptr, h->colidx, scale, mask, h->n, F);
  }
  h->launches += 1;
  GNNCO_LAUNCH_CHECK();
  return GNNCO_OK;
}

}  // namespace

int32_t launch_aggregate(gnnco_handle* h, int dtype, const void* in, void* out, int F, const float* row_scale,
                         const void* relu_mask, cudaStream_t st) {
  ProfScope prof_(h, row_scale ? K_AGG_FWD : K_AGG_BWD, st);
  if (dtype == GNNCO_F32)
    return aggregate_typed<float>(h, (const float*)in, (float*)out, F, row_scale, (const float*)relu_mask, st);
  if (dtype == GNNCO_BF16)
    return aggregate_typed<__nv_bfloat16>(h, (const __nv_bfloat16*)in, (__nv_bfloat16*)out, F, row_scale,
                                          (const __nv_bfloat16*)relu_mask, st);
  return GNNCO_UNSUPPORTED;
}
