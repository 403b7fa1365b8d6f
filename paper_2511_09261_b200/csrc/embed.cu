// Input embeddings (Section 3.2, first paragraph on subgraph training): node embeddings start
// as random vectors and pass through a Gumbel-softmax before they enter the GCN layer of
// Eq. 3.  Two entry points:
//
//   gnnco_gumbel_softmax     x_i = softmax( (e_i + g_i) / tau ),  g = -log(-log u)
//   gnnco_embedding_update   Adam on a float32 master copy of the embeddings with the
//                            gradient dX of gnnco_train_step (the variant in which the
//                            embeddings are trained together with the weights)
//
// The paper gives neither temperature nor the hard/soft form nor a resampling rule; here:
// soft form, one temperature for all nodes, and the uniforms u are an input (drawn once by
// the caller), so the call is a pure function of its arguments.
#include <math.h>

#include "internal.cuh"

namespace {

__device__ __forceinline__ float load_f(const float* p) { return __ldg(p); }
__device__ __forceinline__ float load_f(const __nv_bfloat16* p) {
  return __uint_as_float((uint32_t)__ldg(reinterpret_cast<const unsigned short*>(p)) << 16);
}
__device__ __forceinline__ void store_f(float* p, float x) { *p = x; }
__device__ __forceinline__ void store_f(__nv_bfloat16* p, float x) { *p = __float2bfloat16_rn(x); }

template <typename T>
__device__ __forceinline__ float logit(const T* __restrict__ E, const float* __restrict__ U, int64_t at, float inv_tau) {
  float a = load_f(E + at);
  if (U) a += -logf(-logf(__ldg(U + at)));
  return a * inv_tau;
}

__device__ __forceinline__ float warp_max(float x) {
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, d));
  return x;
}
__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) x += __shfl_xor_sync(0xffffffffu, x, d);
  return x;
}

// One warp per row; lanes stride over the features (coalesced).  Rows of up to 32 * CACHE
// features keep their logits in registers (the two logarithms per element are evaluated
// once); longer rows recompute them in each of the three passes (max, sum, write).
template <typename T, int CACHE>
__global__ void __launch_bounds__(256) gumbel_softmax_kernel(const T* __restrict__ E, const float* __restrict__ U,
                                                             T* __restrict__ X, int64_t n, int F, float inv_tau) {
  const int lane = threadIdx.x & 31;
  const int64_t row = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  if (row >= n) return;
  const int64_t base = row * F;
  if (CACHE > 0) {
    float a[CACHE > 0 ? CACHE : 1];
    float mx = -INFINITY;
#pragma unroll
    for (int k = 0; k < CACHE; ++k) {
      const int f = lane + 32 * k;
      a[k] = f < F ? logit(E, U, base + f, inv_tau) : -INFINITY;
      mx = fmaxf(mx, a[k]);
    }
    mx = warp_max(mx);
    float sum = 0.0f;
#pragma unroll
    for (int k = 0; k < CACHE; ++k) {
      a[k] = lane + 32 * k < F ? expf(a[k] - mx) : 0.0f;
      sum += a[k];
    }
    sum = warp_sum(sum);
#pragma unroll
    for (int k = 0; k < CACHE; ++k) {
      const int f = lane + 32 * k;
      if (f < F) store_f(X + base + f, a[k] / sum);
    }
  } else {
    float mx = -INFINITY;
    for (int f = lane; f < F; f += 32) mx = fmaxf(mx, logit(E, U, base + f, inv_tau));
    mx = warp_max(mx);
    float sum = 0.0f;
    for (int f = lane; f < F; f += 32) sum += expf(logit(E, U, base + f, inv_tau) - mx);
    sum = warp_sum(sum);
    // a row is read completely before any of it is written, and an element is read before
    // it is written by the same lane, so E and X may be the same buffer
    for (int f = lane; f < F; f += 32) store_f(X + base + f, expf(logit(E, U, base + f, inv_tau) - mx) / sum);
  }
}

template <typename T>
__global__ void __launch_bounds__(256) embedding_adam_kernel(const T* __restrict__ dX, float* __restrict__ Xm,
                                                             float* __restrict__ m, float* __restrict__ v,
                                                             T* __restrict__ X, int64_t count, float lr, float b1,
                                                             float b2, float eps, float inv_c1, float inv_c2) {
  const int64_t q = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (q >= count) return;
  const float g = load_f(dX + q);
  const float mq = b1 * m[q] + (1.0f - b1) * g;
  const float vq = b2 * v[q] + (1.0f - b2) * g * g;
  m[q] = mq;
  v[q] = vq;
  const float x = Xm[q] - lr * (mq * inv_c1) / (sqrtf(vq * inv_c2) + eps);
  Xm[q] = x;
  store_f(X + q, x);
}

template <typename T>
int32_t gumbel_typed(gnnco_handle* h, const T* E, const float* U, T* X, int F, float tau, cudaStream_t st) {
  const unsigned grid = (unsigned)((h->n + 7) / 8);
  const float inv_tau = 1.0f / tau;
  if (F <= 32) gumbel_softmax_kernel<T, 1><<<grid, 256, 0, st>>>(E, U, X, h->n, F, inv_tau);
  else if (F <= 64) gumbel_softmax_kernel<T, 2><<<grid, 256, 0, st>>>(E, U, X, h->n, F, inv_tau);
  else if (F <= 128) gumbel_softmax_kernel<T, 4><<<grid, 256, 0, st>>>(E, U, X, h->n, F, inv_tau);
  else if (F <= 256) gumbel_softmax_kernel<T, 8><<<grid, 256, 0, st>>>(E, U, X, h->n, F, inv_tau);
  else gumbel_softmax_kernel<T, 0><<<grid, 256, 0, st>>>(E, U, X, h->n, F, inv_tau);
  h->launches += 1;
  GNNCO_LAUNCH_CHECK();
  return GNNCO_OK;
}

}  // namespace

extern "C" int32_t gnnco_gumbel_softmax(gnnco_handle* h, int32_t feat_dtype, int32_t F, const void* E, const float* U,
                                       float tau, void* X, void* stream) {
  if (!h || !E || !X || F < 1 || F > 65536 || !(tau > 0.0f)) return GNNCO_INVALID_ARGUMENT;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  ProfScope prof_(h, K_EMBED, st);
  if (feat_dtype == GNNCO_F32) return gumbel_typed<float>(h, (const float*)E, U, (float*)X, F, tau, st);
  if (feat_dtype == GNNCO_BF16)
    return gumbel_typed<__nv_bfloat16>(h, (const __nv_bfloat16*)E, U, (__nv_bfloat16*)X, F, tau, st);
  return GNNCO_UNSUPPORTED;
}

extern "C" int32_t gnnco_embedding_update(gnnco_handle* h, int32_t feat_dtype, int32_t F, const void* dX,
                                         float* X_master, float* m, float* v, void* X, float lr, float beta1,
                                         float beta2, float eps, int64_t step, void* stream) {
  if (!h || !dX || !X_master || !m || !v || !X || F < 1 || F > 65536 || step < 1) return GNNCO_INVALID_ARGUMENT;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  ProfScope prof_(h, K_EMBED, st);
  const int64_t count = h->n * (int64_t)F;
  const float c1 = (float)(1.0 - pow((double)beta1, (double)step));
  const float c2 = (float)(1.0 - pow((double)beta2, (double)step));
  const unsigned grid = (unsigned)((count + 255) / 256);
  if (feat_dtype == GNNCO_F32)
    embedding_adam_kernel<float><<<grid, 256, 0, st>>>((const float*)dX, X_master, m, v, (float*)X, count, lr, beta1,
                                                       beta2, eps, 1.0f / c1, 1.0f / c2);
  else if (feat_dtype == GNNCO_BF16)
    embedding_adam_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>((const __nv_bfloat16*)dX, X_master, m, v,
                                                               (__nv_bfloat16*)X, count, lr, beta1, beta2, eps,
                                                               1.0f / c1, 1.0f / c2);
  else
    return GNNCO_UNSUPPORTED;
  h->launches += 1;
  GNNCO_LAUNCH_CHECK();
  return GNNCO_OK;
}
