// Dense per-subgraph weight transform (Eq. 3's "... W"), its two gradients, and the
// element-wise kernels around it, on the FMA pipes.  Works for every width and both
// feature types; rows of a tile always belong to one subgraph, so one tile uses one
// weight set.
//
//   transform      Y = act( A W_s ) or A W_s^T, optional per-row scale (folds D^-1 into
//                  the tensor that feeds the transposed aggregation) and optional ReLU mask
//                  taken from a saved activation of the same shape
//   weight_grad    dW_s = A_s^T G_s        (one block per output tile, fixed row order)
//   gemv / weight_grad_vec / rank1_masked  the same three roles for the last layer,
//                  whose output width is 1 (Eq. 4)
//   adam           bias-corrected Adam on the float32 master weights
#include "internal.cuh"

namespace {

__device__ __forceinline__ float ld(const float* p) { return __ldg(p); }
__device__ __forceinline__ float ld(const __nv_bfloat16* p) {
  return __uint_as_float((uint32_t)__ldg(reinterpret_cast<const unsigned short*>(p)) << 16);
}
__device__ __forceinline__ void st(float* p, float x) { *p = x; }
__device__ __forceinline__ void st(__nv_bfloat16* p, float x) { *p = __float2bfloat16_rn(x); }

constexpr int BM = 128, BN = 64, BK = 16;

template <typename TA, typename TW, bool TRANSB>
__global__ void __launch_bounds__(256) transform_fma(const TA* __restrict__ A, const TW* __restrict__ W,
                                                     int64_t w_stride, TA* __restrict__ Y, int K, int N, int relu,
                                                     const float* __restrict__ row_scale,
                                                     const TA* __restrict__ relu_mask,
                                                     const int32_t* __restrict__ tile_row0,
                                                     const int32_t* __restrict__ tile_rows,
                                                     const int32_t* __restrict__ node_part) {
  __shared__ __align__(16) float As[BK][BM + 4];
  __shared__ __align__(16) float Bs[BK][BN + 4];
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int64_t row0 = tile_row0[blockIdx.x];
  const int rows = tile_rows[blockIdx.x];
  const int n0 = blockIdx.y * BN;
  const TW* Ws = W + (int64_t)node_part[row0] * w_stride;
  float acc[8][4];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.0f;
  for (int k0 = 0; k0 < K; k0 += BK) {
#pragma unroll
    for (int r = 0; r < (BM * BK) / 256; ++r) {
      int idx = tid + r * 256;
      int row = idx / BK, kk = idx % BK;
      float v = 0.0f;
      if (row < rows && k0 + kk < K) v = ld(A + (row0 + row) * K + k0 + kk);
      As[kk][row] = v;
    }
#pragma unroll
    for (int r = 0; r < (BN * BK) / 256; ++r) {
      int idx = tid + r * 256;
      float v = 0.0f;
      if (TRANSB) {
        int nn = idx / BK, kk = idx % BK;
        if (n0 + nn < N && k0 + kk < K) v = ld(Ws + (int64_t)(n0 + nn) * K + k0 + kk);
        Bs[kk][nn] = v;
      } else {
        int kk = idx / BN, nn = idx % BN;
        if (n0 + nn < N && k0 + kk < K) v = ld(Ws + (int64_t)(k0 + kk) * N + n0 + nn);
        Bs[kk][nn] = v;
      }
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      float a[8], b[4];
      const float4 a0 = *reinterpret_cast<const float4*>(&As[kk][ty * 8]);
      const float4 a1 = *reinterpret_cast<const float4*>(&As[kk][ty * 8 + 4]);
      const float4 b0 = *reinterpret_cast<const float4*>(&Bs[kk][tx * 4]);
      a[0] = a0.x; a[1] = a0.y; a[2] = a0.z; a[3] = a0.w; a[4] = a1.x; a[5] = a1.y; a[6] = a1.z; a[7] = a1.w;
      b[0] = b0.x; b[1] = b0.y; b[2] = b0.z; b[3] = b0.w;
#pragma unroll
      for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int row = ty * 8 + i;
    if (row >= rows) continue;
    const float s = row_scale ? row_scale[row0 + row] : 1.0f;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int col = n0 + tx * 4 + j;
      if (col >= N) continue;
      float v = acc[i][j] * s;
      if (relu) v = v > 0.0f ? v : 0.0f;
      if (relu_mask && !(ld(relu_mask + (row0 + row) * N + col) > 0.0f)) v = 0.0f;
      st(Y + (row0 + row) * N + col, v);
    }
  }
}

// One 64 x 64 tile of  sum over the rows of one chunk of A[i, k]^T G[i, n].  A chunk of the weight-gradient chunk
// table is a whole subgraph, or a run of rows of a very long one whose partial result goes to a scratch slot and
// is combined in chunk order afterwards (as in the tensor-core kernels): a partition into a few large
// subgraphs still gives the whole GPU work.
template <typename TA>
__global__ void __launch_bounds__(256) weight_grad_fma(const TA* __restrict__ A, const TA* __restrict__ G,
                                                       float* __restrict__ dW, float* __restrict__ scratch, int K, int N,
                                                       const int32_t* __restrict__ wg_begin,
                                                       const int32_t* __restrict__ wg_end,
                                                       const int32_t* __restrict__ wg_slot) {
  __shared__ __align__(16) float As[16][64 + 4];
  __shared__ __align__(16) float Gs[16][64 + 4];
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int c = blockIdx.x, k0 = blockIdx.y * 64, n0 = blockIdx.z * 64;
  const int64_t ra = wg_begin[c], rb = wg_end[c];
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.0f;
  for (int64_t r0 = ra; r0 < rb; r0 += 16) {
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      int idx = tid + r * 256;
      int rr = idx / 64, cc = idx % 64;
      bool in = r0 + rr < rb;
      As[rr][cc] = (in && k0 + cc < K) ? ld(A + (r0 + rr) * K + k0 + cc) : 0.0f;
      Gs[rr][cc] = (in && n0 + cc < N) ? ld(G + (r0 + rr) * N + n0 + cc) : 0.0f;
    }
    __syncthreads();
#pragma unroll
    for (int rr = 0; rr < 16; ++rr) {
      const float4 a = *reinterpret_cast<const float4*>(&As[rr][ty * 4]);
      const float4 g = *reinterpret_cast<const float4*>(&Gs[rr][tx * 4]);
      const float av[4] = {a.x, a.y, a.z, a.w}, gv[4] = {g.x, g.y, g.z, g.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], gv[j], acc[i][j]);
    }
    __syncthreads();
  }
  const int32_t slot = wg_slot[c];       // < 0: the whole subgraph -(slot + 1); >= 0: scratch slot of a split subgraph
  float* out = slot < 0 ? dW + (int64_t)(-(slot + 1)) * K * N : scratch + (int64_t)slot * K * N;
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      int k = k0 + ty * 4 + i, n = n0 + tx * 4 + j;
      if (k < K && n < N) out[(int64_t)k * N + n] = acc[i][j];
    }
}

template <typename TA, typename TW>
__global__ void __launch_bounds__(256) gemv_rows(const TA* __restrict__ H, const TW* __restrict__ w, int64_t w_stride,
                                                 const int32_t* __restrict__ node_part, float* __restrict__ u,
                                                 int64_t n, int F, const RowChunks rc) {
  const int lane = threadIdx.x & 31;
  int64_t row;
  if (!chunk_row(rc, (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5), n, row)) return;
  const TW* ws = w + (int64_t)node_part[row] * w_stride;
  float acc = 0.0f;
  for (int f = lane; f < F; f += 32) acc = fmaf(ld(H + row * F + f), ld(ws + f), acc);
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, d);
  if (lane == 0) u[row] = acc;
}

// dw[s][:] = sum_{i in s} H[i,:] g[i].  One block per row chunk of the weight-gradient chunk
// table (a whole subgraph, or a run of rows of a very long one whose partial result goes to a
// scratch slot and is combined in chunk order afterwards); LPR lanes cover a row with 16-byte
// loads, the 256/LPR row groups walk the chunk's rows interleaved (four rows in flight each)
// and meet in shared memory in a fixed order.  This pass reads every element of H exactly once,
// so (bfloat16) it can leave [H > 0] behind as one bit per element (bits_out: element f of a row
// = bit f%8 of byte f/8) for the rank-1 aggregation that follows, which then gathers 32 bytes
// a row instead of 512.
template <typename TA, int LPR>
__global__ void __launch_bounds__(256) weight_grad_vec_rows(const TA* __restrict__ H, const float* __restrict__ g,
                                                            float* __restrict__ dw, float* __restrict__ scratch,
                                                            uint8_t* __restrict__ bits_out, int F,
                                                            const int32_t* __restrict__ wg_begin,
                                                            const int32_t* __restrict__ wg_end,
                                                            const int32_t* __restrict__ wg_slot) {
  constexpr int VN = 16 / sizeof(TA);
  constexpr int RG = 256 / LPR;
  extern __shared__ float partial[];                       // [RG][F]
  const int sub = threadIdx.x % LPR, rg = threadIdx.x / LPR;
  const int64_t ra = wg_begin[blockIdx.x], rb = wg_end[blockIdx.x];
  const int32_t slot = wg_slot[blockIdx.x];
  float* out = slot < 0 ? dw + (int64_t)(-(slot + 1)) * F : scratch + (int64_t)slot * F;
  float acc[VN];
#pragma unroll
  for (int e = 0; e < VN; ++e) acc[e] = 0.0f;
  auto fma_row = [&](const uint4& v, float gi, int64_t row) {
    if (sizeof(TA) == 2 && bits_out) {
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
      uint32_t m = 0;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        m |= (__uint_as_float(w[k] << 16) > 0.0f ? 1u : 0u) << (2 * k);
        m |= (__uint_as_float(w[k] & 0xffff0000u) > 0.0f ? 1u : 0u) << (2 * k + 1);
      }
      if (LPR >= 32) {
        // a row group is one or two whole warps here (uniform trip counts): four lanes' bytes in one word
        m |= __shfl_down_sync(0xffffffffu, m, 1) << 8;
        m |= __shfl_down_sync(0xffffffffu, m, 2) << 16;
        if ((sub & 3) == 0) *reinterpret_cast<uint32_t*>(bits_out + row * (F >> 3) + sub) = m;
      } else {
        bits_out[row * (F >> 3) + sub] = (uint8_t)m;
      }
    }
    if (sizeof(TA) == 4) {
      acc[0] = fmaf(__uint_as_float(v.x), gi, acc[0]); acc[1] = fmaf(__uint_as_float(v.y), gi, acc[1]);
      acc[2] = fmaf(__uint_as_float(v.z), gi, acc[2]); acc[3] = fmaf(__uint_as_float(v.w), gi, acc[3]);
    } else {
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        acc[(2 * k) % VN] = fmaf(__uint_as_float(w[k] << 16), gi, acc[(2 * k) % VN]);
        acc[(2 * k + 1) % VN] = fmaf(__uint_as_float(w[k] & 0xffff0000u), gi, acc[(2 * k + 1) % VN]);
      }
    }
  };
  int64_t i = ra + rg;
  for (; i + 3 * RG < rb; i += 4 * RG) {
    uint4 v[4];
    float gi[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      v[u] = __ldg(reinterpret_cast<const uint4*>(H + (i + u * RG) * F + sub * VN));
      gi[u] = __ldg(g + i + u * RG);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) fma_row(v[u], gi[u], i + u * RG);
  }
  for (; i < rb; i += RG) fma_row(__ldg(reinterpret_cast<const uint4*>(H + i * F + sub * VN)), __ldg(g + i), i);
#pragma unroll
  for (int e = 0; e < VN; ++e) partial[rg * F + sub * VN + e] = acc[e];
  __syncthreads();
  for (int f = threadIdx.x; f < F; f += 256) {
    float tot = 0.0f;
    for (int r = 0; r < RG; ++r) tot += partial[r * F + f];
    out[f] = tot;
  }
}

// any width: one thread per column
template <typename TA>
__global__ void __launch_bounds__(256) weight_grad_vec_kernel(const TA* __restrict__ H, const float* __restrict__ g,
                                                              float* __restrict__ dw, float* __restrict__ scratch,
                                                              int F, const int32_t* __restrict__ wg_begin,
                                                              const int32_t* __restrict__ wg_end,
                                                              const int32_t* __restrict__ wg_slot) {
  const int f = blockIdx.y * 256 + threadIdx.x;
  if (f >= F) return;
  const int64_t ra = wg_begin[blockIdx.x], rb = wg_end[blockIdx.x];
  const int32_t slot = wg_slot[blockIdx.x];
  float* out = slot < 0 ? dw + (int64_t)(-(slot + 1)) * F : scratch + (int64_t)slot * F;
  float acc = 0.0f;
  for (int64_t i = ra; i < rb; ++i) acc = fmaf(ld(H + i * F + f), __ldg(g + i), acc);
  out[f] = acc;
}

template <typename TA, typename TW>
__global__ void __launch_bounds__(256) rank1_masked_kernel(const float* __restrict__ g, const TW* __restrict__ w,
                                                           int64_t w_stride, const int32_t* __restrict__ node_part,
                                                           const TA* __restrict__ H, TA* __restrict__ dZ, int64_t n,
                                                           int F) {
  const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= n * F) return;
  const int64_t i = t / F;
  const int f = (int)(t - i * F);
  const float hv = H ? ld(H + t) : 1.0f;
  const float v = hv > 0.0f ? __ldg(g + i) * ld(w + (int64_t)node_part[i] * w_stride + f) : 0.0f;
  st(dZ + t, v);
}

// float32, 4 features per thread (F a multiple of 4, 16-byte aligned rows)
__global__ void __launch_bounds__(256) rank1_masked_f32x4(const float* __restrict__ g, const float* __restrict__ w,
                                                          int64_t w_stride, const int32_t* __restrict__ node_part,
                                                          const float* __restrict__ H, float* __restrict__ dZ,
                                                          int64_t n, int F) {
  const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int groups = F >> 2;
  if (t >= n * groups) return;
  const int64_t i = t / groups;
  const int f = (int)(t - i * groups) << 2;
  const float gi = __ldg(g + i);
  const float4 wv = __ldg(reinterpret_cast<const float4*>(w + (int64_t)node_part[i] * w_stride + f));
  float4 hv = make_float4(1.f, 1.f, 1.f, 1.f);
  if (H) hv = __ldg(reinterpret_cast<const float4*>(H + i * F + f));
  *reinterpret_cast<float4*>(dZ + i * F + f) = make_float4(hv.x > 0.f ? gi * wv.x : 0.f, hv.y > 0.f ? gi * wv.y : 0.f,
                                                           hv.z > 0.f ? gi * wv.z : 0.f, hv.w > 0.f ? gi * wv.w : 0.f);
}

// bf16, 8 features per thread (F a multiple of 8, 16-byte aligned rows)
__global__ void __launch_bounds__(256) rank1_masked_bf16x8(const float* __restrict__ g,
                                                           const __nv_bfloat16* __restrict__ w, int64_t w_stride,
                                                           const int32_t* __restrict__ node_part,
                                                           const __nv_bfloat16* __restrict__ H,
                                                           __nv_bfloat16* __restrict__ dZ, int64_t n, int F) {
  const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;      // one 8-element group
  const int groups = F >> 3;
  if (t >= n * groups) return;
  const int64_t i = t / groups;
  const int f = (int)(t - i * groups) << 3;
  const float gi = __ldg(g + i);
  const uint4 wv = __ldg(reinterpret_cast<const uint4*>(w + (int64_t)node_part[i] * w_stride + f));
  uint4 hv = make_uint4(0x3f803f80u, 0x3f803f80u, 0x3f803f80u, 0x3f803f80u);   // ones when there is no mask
  if (H) hv = __ldg(reinterpret_cast<const uint4*>(H + i * F + f));
  const uint32_t wq[4] = {wv.x, wv.y, wv.z, wv.w}, hq[4] = {hv.x, hv.y, hv.z, hv.w};
  uint32_t o[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const float w0 = __uint_as_float(wq[k] << 16), w1 = __uint_as_float(wq[k] & 0xffff0000u);
    const float h0 = __uint_as_float(hq[k] << 16), h1 = __uint_as_float(hq[k] & 0xffff0000u);
    __nv_bfloat162 v = __floats2bfloat162_rn(h0 > 0.0f ? gi * w0 : 0.0f, h1 > 0.0f ? gi * w1 : 0.0f);
    o[k] = *reinterpret_cast<uint32_t*>(&v);
  }
  *reinterpret_cast<uint4*>(dZ + i * F + f) = make_uint4(o[0], o[1], o[2], o[3]);
}

__global__ void sum_over_sets_kernel(const float* __restrict__ in, float* __restrict__ out, int64_t count,
                                     int32_t sets) {
  const int64_t q = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (q >= count) return;
  float acc = 0.0f;
  for (int32_t s = 0; s < sets; ++s) acc += in[(int64_t)s * count + q];
  out[q] = acc;
}

__global__ void wg_combine_kernel(const float* __restrict__ scratch, float* __restrict__ dW, int64_t count,
                                  const int32_t* __restrict__ mpart, const int32_t* __restrict__ mfirst,
                                  const int32_t* __restrict__ mcount) {
  const int64_t q = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (q >= count) return;
  const int m = blockIdx.y;
  const float* src = scratch + (int64_t)mfirst[m] * count + q;
  float acc = 0.0f;
  for (int32_t c = 0; c < mcount[m]; ++c) acc += src[(int64_t)c * count];
  dW[(int64_t)mpart[m] * count + q] = acc;
}

__global__ void cast_bf16_kernel(const float* __restrict__ in, __nv_bfloat16* __restrict__ out, int64_t count) {
  const int64_t q = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (q < count) out[q] = __float2bfloat16_rn(in[q]);
}

__global__ void cast_bf16x8_kernel(const float4* __restrict__ in, uint4* __restrict__ out, int64_t groups) {
  const int64_t q = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (q >= groups) return;
  const float4 a = __ldg(in + 2 * q), b = __ldg(in + 2 * q + 1);
  __nv_bfloat162 v0 = __floats2bfloat162_rn(a.x, a.y), v1 = __floats2bfloat162_rn(a.z, a.w);
  __nv_bfloat162 v2 = __floats2bfloat162_rn(b.x, b.y), v3 = __floats2bfloat162_rn(b.z, b.w);
  out[q] = make_uint4(*reinterpret_cast<uint32_t*>(&v0), *reinterpret_cast<uint32_t*>(&v1),
                      *reinterpret_cast<uint32_t*>(&v2), *reinterpret_cast<uint32_t*>(&v3));
}

__global__ void adam_kernel(float* __restrict__ W, float* __restrict__ m, float* __restrict__ v,
                            const float* __restrict__ g, int64_t count, float lr, float b1, float b2, float eps,
                            float inv_c1, float inv_c2, const uint8_t* __restrict__ active, int64_t per_set,
                            const float2* __restrict__ bias) {
  const int64_t q = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (q >= count) return;
  if (bias) {            // bias corrections kept on the device (a step counter there: adam_tick)
    inv_c1 = bias->x;
    inv_c2 = bias->y;
  }
  if (active && !active[q / per_set]) return;   // this subgraph is not being fine-tuned
  const float gq = g[q];
  const float mq = b1 * m[q] + (1.0f - b1) * gq;
  const float vq = b2 * v[q] + (1.0f - b2) * gq * gq;
  m[q] = mq;
  v[q] = vq;
  W[q] -= lr * (mq * inv_c1) / (sqrtf(vq * inv_c2) + eps);
}

// the same update on four consecutive elements (count and per_set multiples of four, 16-byte aligned arrays)
__global__ void __launch_bounds__(256) adam_vec4_kernel(float4* __restrict__ W, float4* __restrict__ m,
                                                        float4* __restrict__ v, const float4* __restrict__ g,
                                                        int64_t quads, float lr, float b1, float b2, float eps,
                                                        float inv_c1, float inv_c2, const uint8_t* __restrict__ active,
                                                        int64_t quads_per_set, const float2* __restrict__ bias) {
  const int64_t q = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (q >= quads) return;
  if (bias) {
    inv_c1 = bias->x;
    inv_c2 = bias->y;
  }
  if (active && !active[q / quads_per_set]) return;
  const float4 gq = __ldg(g + q);
  float4 mq = m[q], vq = v[q], wq = W[q];
  const float gs[4] = {gq.x, gq.y, gq.z, gq.w};
  float* mp = reinterpret_cast<float*>(&mq);
  float* vp = reinterpret_cast<float*>(&vq);
  float* wp = reinterpret_cast<float*>(&wq);
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    mp[c] = b1 * mp[c] + (1.0f - b1) * gs[c];
    vp[c] = b2 * vp[c] + (1.0f - b2) * gs[c] * gs[c];
    wp[c] -= lr * (mp[c] * inv_c1) / (sqrtf(vp[c] * inv_c2) + eps);
  }
  m[q] = mq;
  v[q] = vq;
  W[q] = wq;
}

inline unsigned blocks_for(int64_t work, int threads) { return (unsigned)((work + threads - 1) / threads); }

}  // namespace

int32_t launch_transform(gnnco_handle* h, int dtype, const void* A, const void* W, int64_t w_stride, void* Y, int K,
                         int N, bool transB, bool relu, const float* row_scale, const void* relu_mask,
                         cudaStream_t stream) {
  ProfScope prof_(h, transB ? K_TRANSFORM_BWD : K_TRANSFORM_FWD, stream);
  if (h->n_tiles == 0) return GNNCO_OK;
  dim3 grid(h->n_tiles, (N + BN - 1) / BN);
  if (grid.y > 65535) return GNNCO_UNSUPPORTED;
#define GNNCO_TRANSFORM(TA, TW, TB)                                                                            \
  transform_fma<TA, TW, TB><<<grid, 256, 0, stream>>>((const TA*)A, (const TW*)W, w_stride, (TA*)Y, K, N, relu, \
                                                      row_scale, (const TA*)relu_mask, h->tile_row0, h->tile_rows, \
                                                      h->node_part)
  if (dtype == GNNCO_F32) {
    if (transB) GNNCO_TRANSFORM(float, float, true);
    else GNNCO_TRANSFORM(float, float, false);
  } else if (dtype == GNNCO_BF16) {
    if (transB) GNNCO_TRANSFORM(__nv_bfloat16, __nv_bfloat16, true);
    else GNNCO_TRANSFORM(__nv_bfloat16, __nv_bfloat16, false);
  } else {
    return GNNCO_UNSUPPORTED;
  }
#undef GNNCO_TRANSFORM
  h->launches += 1;
  GNNCO_LAUNCH_CHECK();
  return GNNCO_OK;
}

int32_t launch_gemv(gnnco_handle* h, int dtype, const void* H, const void* w, int64_t w_stride, float* u, int F,
                    cudaStream_t stream) {
  ProfScope prof_(h, K_GEMV, stream);
  unsigned grid = blocks_for(linear_rows(h), 8);
  if (dtype == GNNCO_F32)
    gemv_rows<float, float><<<grid, 256, 0, stream>>>((const float*)H, (const float*)w, w_stride, h->node_part, u,
                                                      h->n, F, h->row_chunks);
  else if (dtype == GNNCO_BF16)
    gemv_rows<__nv_bfloat16, __nv_bfloat16><<<grid, 256, 0, stream>>>(
        (const __nv_bfloat16*)H, (const __nv_bfloat16*)w, w_stride, h->node_part, u, h->n, F,
        h->row_chunks);
  else
    return GNNCO_UNSUPPORTED;
  h->launches += 1;
  GNNCO_LAUNCH_CHECK();
  return GNNCO_OK;
}

int32_t launch_weight_grad(gnnco_handle* h, int dtype, const void* A, const void* G, float* dW, float* scratch, int K,
                           int N, cudaStream_t stream) {
  ProfScope prof_(h, K_WEIGHT_GRAD, stream);
  if (h->n_wg_chunks <= 0) return GNNCO_OK;
  dim3 grid(h->n_wg_chunks, (K + 63) / 64, (N + 63) / 64);
  if (grid.y > 65535 || grid.z > 65535) return GNNCO_UNSUPPORTED;
  if (dtype == GNNCO_F32)
    weight_grad_fma<float><<<grid, 256, 0, stream>>>((const float*)A, (const float*)G, dW, scratch, K, N, h->wg_begin,
                                                     h->wg_end, h->wg_slot);
  else if (dtype == GNNCO_BF16)
    weight_grad_fma<__nv_bfloat16><<<grid, 256, 0, stream>>>((const __nv_bfloat16*)A, (const __nv_bfloat16*)G, dW, scratch,
                                                             K, N, h->wg_begin, h->wg_end, h->wg_slot);
  else
    return GNNCO_UNSUPPORTED;
  h->launches += 1;
  GNNCO_LAUNCH_CHECK();
  return launch_wg_combine(h, scratch, dW, (int64_t)K * N, stream);
}

int32_t launch_weight_grad_vec(gnnco_handle* h, int dtype, const void* H, const float* g, float* dw, float* scratch,
                               int F, uint8_t* bits_out, bool* wrote_bits, cudaStream_t stream) {
  ProfScope prof_(h, K_WEIGHT_GRAD_VEC, stream);
  if (wrote_bits) *wrote_bits = false;
  if (h->n_wg_slots > 0 && !scratch) return GNNCO_INTERNAL;
  const int vn = dtype == GNNCO_BF16 ? 8 : 4;
  const int lpr = F % vn == 0 ? F / vn : 0;
  const bool aligned = !((uintptr_t)H & 15);
  const size_t sm = (size_t)(lpr ? 256 / lpr : 0) * F * sizeof(float);
#define GNNCO_WGV(TT, L)                                                                                     \
  weight_grad_vec_rows<TT, L><<<h->n_wg_chunks, 256, sm, stream>>>((const TT*)H, g, dw, scratch, bits, F, \
                                                                   h->wg_begin, h->wg_end, h->wg_slot)
  bool done = aligned && (lpr == 8 || lpr == 16 || lpr == 32 || lpr == 64);
  uint8_t* bits = (done && dtype == GNNCO_BF16) ? bits_out : nullptr;   // every row is in exactly one chunk
  if (bits && wrote_bits) *wrote_bits = true;
  if (done && dtype == GNNCO_F32) {
    if (lpr == 8) GNNCO_WGV(float, 8); else if (lpr == 16) GNNCO_WGV(float, 16);
    else if (lpr == 32) GNNCO_WGV(float, 32); else GNNCO_WGV(float, 64);
  } else if (done && dtype == GNNCO_BF16) {
    if (lpr == 8) GNNCO_WGV(__nv_bfloat16, 8); else if (lpr == 16) GNNCO_WGV(__nv_bfloat16, 16);
    else if (lpr == 32) GNNCO_WGV(__nv_bfloat16, 32); else GNNCO_WGV(__nv_bfloat16, 64);
  } else {
    dim3 grid(h->n_wg_chunks, (F + 255) / 256);
    if (grid.y > 65535) return GNNCO_UNSUPPORTED;
    if (dtype == GNNCO_F32)
      weight_grad_vec_kernel<float><<<grid, 256, 0, stream>>>((const float*)H, g, dw, scratch, F, h->wg_begin,
                                                              h->wg_end, h->wg_slot);
    else if (dtype == GNNCO_BF16)
      weight_grad_vec_kernel<__nv_bfloat16><<<grid, 256, 0, stream>>>((const __nv_bfloat16*)H, g, dw, scratch, F,
                                                                      h->wg_begin, h->wg_end, h->wg_slot);
    else
      return GNNCO_UNSUPPORTED;
  }
#undef GNNCO_WGV
  h->launches += 1;
  GNNCO_LAUNCH_CHECK();
  return launch_wg_combine(h, scratch, dw, F, stream);
}

int32_t launch_rank1_masked(gnnco_handle* h, int dtype, const float* g, const void* w, int64_t w_stride, const void* H,
                            void* dZ, int F, cudaStream_t stream) {
  ProfScope prof_(h, K_RANK1, stream);
  unsigned grid = blocks_for(h->n * F, 256);
  if (dtype == GNNCO_F32 && F % 4 == 0 && w_stride % 4 == 0 && !(((uintptr_t)w | (uintptr_t)H | (uintptr_t)dZ) & 15))
    rank1_masked_f32x4<<<blocks_for(h->n * (F / 4), 256), 256, 0, stream>>>(g, (const float*)w, w_stride, h->node_part,
                                                                            (const float*)H, (float*)dZ, h->n, F);
  else if (dtype == GNNCO_F32)
    rank1_masked_kernel<float, float><<<grid, 256, 0, stream>>>(g, (const float*)w, w_stride, h->node_part,
                                                                (const float*)H, (float*)dZ, h->n, F);
  else if (dtype == GNNCO_BF16 && F % 8 == 0 && w_stride % 8 == 0 &&
           !(((uintptr_t)w | (uintptr_t)H | (uintptr_t)dZ) & 15))
    rank1_masked_bf16x8<<<blocks_for(h->n * (F / 8), 256), 256, 0, stream>>>(
        g, (const __nv_bfloat16*)w, w_stride, h->node_part, (const __nv_bfloat16*)H, (__nv_bfloat16*)dZ, h->n, F);
  else if (dtype == GNNCO_BF16)
    rank1_masked_kernel<__nv_bfloat16, __nv_bfloat16><<<grid, 256, 0, stream>>>(
        g, (const __nv_bfloat16*)w, w_stride, h->node_part, (const __nv_bfloat16*)H, (__nv_bfloat16*)dZ, h->n, F);
  else
    return GNNCO_UNSUPPORTED;
  h->launches += 1;
  GNNCO_LAUNCH_CHECK();
  return GNNCO_OK;
}

int32_t launch_wg_combine(gnnco_handle* h, const float* scratch, float* dW, int64_t count, cudaStream_t stream) {
  if (h->n_wg_multi == 0) return GNNCO_OK;
  ProfScope prof_(h, K_WEIGHT_GRAD, stream);
  dim3 grid(blocks_for(count, 256), h->n_wg_multi);
  if (grid.y > 65535) return GNNCO_UNSUPPORTED;
  wg_combine_kernel<<<grid, 256, 0, stream>>>(scratch, dW, count, h->wg_mpart, h->wg_mfirst, h->wg_mcount);
  h->launches += 1;
  GNNCO_LAUNCH_CHECK();
  return GNNCO_OK;
}

int32_t launch_sum_over_sets(gnnco_handle* h, const float* in, float* out, int64_t count, int32_t sets,
                             cudaStream_t stream) {
  ProfScope prof_(h, K_SUM_SETS, stream);
  sum_over_sets_kernel<<<blocks_for(count, 256), 256, 0, stream>>>(in, out, count, sets);
  h->launches += 1;
  GNNCO_LAUNCH_CHECK();
  return GNNCO_OK;
}

int32_t launch_cast_bf16(gnnco_handle* h, const float* in, __nv_bfloat16* out, int64_t count, cudaStream_t stream) {
  ProfScope prof_(h, K_CAST, stream);
  if (count % 8 == 0 && !(((uintptr_t)in | (uintptr_t)out) & 15))
    cast_bf16x8_kernel<<<blocks_for(count / 8, 256), 256, 0, stream>>>(reinterpret_cast<const float4*>(in),
                                                                       reinterpret_cast<uint4*>(out), count / 8);
  else
    cast_bf16_kernel<<<blocks_for(count, 256), 256, 0, stream>>>(in, out, count);
  h->launches += 1;
  GNNCO_LAUNCH_CHECK();
  return GNNCO_OK;
}

// One thread: the device-side step counter advances and the bias corrections of THIS update,
// 1 / (1 - beta^t), are left where the Adam kernels of the step read them.
__global__ void adam_tick(int32_t* __restrict__ step_dev, float b1, float b2, float2* __restrict__ bias) {
  const int32_t t = *step_dev + 1;
  *step_dev = t;
  const float c1 = (float)(1.0 - pow((double)b1, (double)t));
  const float c2 = (float)(1.0 - pow((double)b2, (double)t));
  *bias = make_float2(1.0f / c1, 1.0f / c2);
}

int32_t launch_adam_tick(gnnco_handle* h, int32_t* step_dev, float b1, float b2, float2* bias, cudaStream_t stream) {
  ProfScope prof_(h, K_ADAM, stream);
  adam_tick<<<1, 1, 0, stream>>>(step_dev, b1, b2, bias);
  h->launches += 1;
  GNNCO_LAUNCH_CHECK();
  return GNNCO_OK;
}

int32_t launch_adam(gnnco_handle* h, float* W, float* m, float* v, const float* g, int64_t count, float lr, float b1,
                    float b2, float eps, float c1, float c2, const uint8_t* active, int64_t per_set,
                    cudaStream_t stream) {
  ProfScope prof_(h, K_ADAM, stream);
  const bool vec = count % 4 == 0 && per_set % 4 == 0 &&
                   (((uintptr_t)W | (uintptr_t)m | (uintptr_t)v | (uintptr_t)g) & 15) == 0;
  if (vec)
    adam_vec4_kernel<<<blocks_for(count / 4, 256), 256, 0, stream>>>(
        reinterpret_cast<float4*>(W), reinterpret_cast<float4*>(m), reinterpret_cast<float4*>(v),
        reinterpret_cast<const float4*>(g), count / 4, lr, b1, b2, eps, 1.0f / c1, 1.0f / c2, active, per_set / 4,
        h->adam_bias);
  else
    adam_kernel<<<blocks_for(count, 256), 256, 0, stream>>>(W, m, v, g, count, lr, b1, b2, eps, 1.0f / c1, 1.0f / c2,
                                                          active, per_set, h->adam_bias);
  h->launches += 1;
  GNNCO_LAUNCH_CHECK();
  return GNNCO_OK;
}
