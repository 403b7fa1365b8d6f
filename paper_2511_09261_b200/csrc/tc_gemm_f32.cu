// Tensor-core dense transform and weight gradient for FLOAT32 features.
//
// The tensor cores multiply bf16 (8 significant bits), float32 has 24.  Every float32
// operand a is therefore split into three bf16 limbs a = a1 + a2 + a3 (each the rounding of
// what the previous ones left over; the subtractions are exact in float32), and a product
// is rebuilt from the six limb products whose weight is at least 2^-16 of the leading one:
//     a*b ~= a1 b1 + (a1 b2 + a2 b1) + (a1 b3 + a2 b2 + a3 b1)
// accumulated in float32 in TMEM.  What is dropped is below 2^-24 relative, i.e. float32
// rounding level, so results meet the float32 tolerance.  The leading products a1 b1 go to one
// accumulator and the five correction products to a second one, added once in the epilogue:
// every MMA rounds the running sum it adds to, and keeping the 5x more numerous corrections
// away from the large sum cuts the accumulated rounding error several times (measured).  Six bf16 MMAs cost as much tensor
// time as three tf32 ones and keep these kernels memory-bound at the widths in use (<= 128).
//
// Activations are split on the fly by the threads that stage them into shared memory; the
// weights' limbs are prepared once per step by a cast kernel.  Structure, shared-memory
// layouts and barriers are those of the bf16 kernels in tc_gemm.cu.
#include "internal.cuh"
#include "tc_common.cuh"

namespace {

constexpr int kTileM = 128;
constexpr int kThreads = 256;                // weight-gradient kernel
constexpr int kTfThreads = 384;              // transform kernel: 4 epilogue warps, 1 MMA warp, 7 producer warps
constexpr int kEpiWarps = 4;
constexpr int kMmaWarp = 4;
constexpr int kProdWarp0 = 5;
constexpr int kProdLanes = 224;              // splitting float32 into limbs is the producers' work: most warps do it
constexpr int kBatch = 5;                    // 32-byte source chunks a producer lane has in flight (a whole k-block)

__device__ __forceinline__ uint32_t pack_bf16x2(float a, float b) {
  __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float bf16_lo(uint32_t p) { return __uint_as_float(p << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t p) { return __uint_as_float(p & 0xffff0000u); }

// eight floats -> three 16-byte chunks of bf16 limbs
__device__ __forceinline__ void split3(const float4& x, const float4& y, uint4& l1, uint4& l2, uint4& l3) {
  const float f[8] = {x.x, x.y, x.z, x.w, y.x, y.y, y.z, y.w};
  uint32_t p1[4], p2[4], p3[4];
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const float a = f[2 * q], b = f[2 * q + 1];
    p1[q] = pack_bf16x2(a, b);
    const float ra = a - bf16_lo(p1[q]), rb = b - bf16_hi(p1[q]);
    p2[q] = pack_bf16x2(ra, rb);
    const float sa = ra - bf16_lo(p2[q]), sb = rb - bf16_hi(p2[q]);
    p3[q] = pack_bf16x2(sa, sb);
  }
  l1 = make_uint4(p1[0], p1[1], p1[2], p1[3]);
  l2 = make_uint4(p2[0], p2[1], p2[2], p2[3]);
  l3 = make_uint4(p3[0], p3[1], p3[2], p3[3]);
}

// ------------------------------------------------------------------------------ transform
// Shared memory: A slot of k-block kb = 3 limb tiles of 128 rows x 128 bytes (K-major SW128);
// B k-block kb = 3 limb tiles of NDIM rows x 128 bytes.
template <int KDIM, int NDIM>
__global__ void __launch_bounds__(kTfThreads, 1)
transform_tc_f32(const float* __restrict__ A, const __nv_bfloat16* __restrict__ B, int64_t b_stride,
                 int64_t b_limb_stride, float* __restrict__ Y, int relu, const float* __restrict__ row_scale,
                 const float* __restrict__ relu_mask, const float* __restrict__ dot_w, int64_t dot_stride, float* __restrict__ dot_out,
                 const int32_t* __restrict__ tile_row0, const int32_t* __restrict__ tile_rows,
                 const int32_t* __restrict__ node_part, int n_tiles, int tiles_per_cta, int32_t* status) {
  constexpr int KB = KDIM / 64;
  constexpr uint32_t A_LIMB = kTileM * 128, B_LIMB = NDIM * 128;
  constexpr uint32_t A_SLOT = 3 * A_LIMB, B_SLOT = 3 * B_LIMB;
  constexpr uint32_t A_BYTES = KB * A_SLOT, B_BYTES = KB * B_SLOT;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t sbase = (tc::smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sA = sbase, sB = sbase + A_BYTES;
  uint8_t* gen_base = smem_raw + (sbase - tc::smem_u32(smem_raw));
  uint64_t* full = reinterpret_cast<uint64_t*>(gen_base + A_BYTES + B_BYTES);
  uint64_t* empty = full + KB;
  uint64_t* acc_full = empty + KB;
  uint64_t* acc_empty = acc_full + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int t_begin = blockIdx.x * tiles_per_cta;
  const int t_end = min(n_tiles, t_begin + tiles_per_cta);
  if (t_begin >= t_end) return;

  if (threadIdx.x == 0) {
    for (int kb = 0; kb < KB; ++kb) {
      tc::mbar_init(full + kb, kProdLanes);
      tc::mbar_init(empty + kb, 1);
    }
    for (int i = 0; i < 2; ++i) {
      tc::mbar_init(acc_full + i, 1);
      tc::mbar_init(acc_empty + i, kEpiWarps * 32);
    }
    *abort_flag = 0;
    tc::fence_mbar_init();
  }
  if (warp == 0) tc::tmem_alloc(tmem_slot, 4 * NDIM);   // two buffers x (leading, correction) accumulators
  tc::tc_fence_before_sync();
  __syncthreads();
  tc::tc_fence_after_sync();
  const uint32_t tmem = *tmem_slot;

  if (warp >= kProdWarp0) {
    // ------------------------------------------------------------------- producers
    const int p = (warp - kProdWarp0) * 32 + lane;
    int cur_part = -1;
    for (int t = t_begin, j = 0; t < t_end && !*abort_flag; ++t, ++j) {
      const int64_t row0 = tile_row0[t];
      const int rows = tile_rows[t];
      const int part = node_part[row0];
      const bool new_b = part != cur_part;
      cur_part = part;
      // the operand loads below go through registers, a k-block at a time, so their latency is
      // on this pipeline's critical path: have the next tile's rows (contiguous) waiting in L2
      if (p == 0 && t + 1 < t_end)
        tc::prefetch_l2(A + (int64_t)tile_row0[t + 1] * KDIM, (uint32_t)tile_rows[t + 1] * KDIM * 4);
      for (int kb = 0; kb < KB; ++kb) {
        if (j > 0 && !tc::mbar_wait_bounded(empty + kb, (j - 1) & 1)) *abort_flag = 1;
        if (new_b) {
          // weight limbs are already bf16 in global memory: plain 16-byte copies
          for (int q = p; q < 3 * NDIM * 8; q += kProdLanes) {
            const int limb = q / (NDIM * 8), rem = q % (NDIM * 8);
            const int r = rem >> 3, cc = rem & 7;
            tc::cp_async16(sB + kb * B_SLOT + limb * B_LIMB + (r >> 3) * 1024 + (r & 7) * 128 + ((cc ^ (r & 7)) << 4),
                           B + limb * b_limb_stride + (int64_t)part * b_stride + (int64_t)r * KDIM + kb * 64 + cc * 8);
          }
        }
        // activations: 32 bytes of float32 -> one 16-byte chunk in each limb tile, a whole k-block in flight
        const float* src = A + row0 * KDIM + kb * 64;
        const uint32_t dstA = sA + kb * A_SLOT;
        for (int q0 = p; q0 < rows * 8; q0 += kBatch * kProdLanes) {
          float4 x[kBatch], y[kBatch];
#pragma unroll
          for (int u = 0; u < kBatch; ++u) {
            const int q = q0 + u * kProdLanes;
            if (q < rows * 8) {
              const float4* g = reinterpret_cast<const float4*>(src + (int64_t)(q >> 3) * KDIM + (q & 7) * 8);
              x[u] = __ldg(g);
              y[u] = __ldg(g + 1);
            }
          }
#pragma unroll
          for (int u = 0; u < kBatch; ++u) {
            const int q = q0 + u * kProdLanes;
            if (q < rows * 8) {
              const int r = q >> 3, cc = q & 7;
              uint4 l1, l2, l3;
              split3(x[u], y[u], l1, l2, l3);
              const uint32_t off = (r >> 3) * 1024 + (r & 7) * 128 + ((cc ^ (r & 7)) << 4);
              tc::st_shared16(dstA + off, l1.x, l1.y, l1.z, l1.w);
              tc::st_shared16(dstA + A_LIMB + off, l2.x, l2.y, l2.z, l2.w);
              tc::st_shared16(dstA + 2 * A_LIMB + off, l3.x, l3.y, l3.z, l3.w);
            }
          }
        }
        if (new_b) tc::cp_async_wait<0>();
        tc::fence_proxy_async_smem();
        tc::mbar_arrive(full + kb);
      }
    }
  } else if (warp == kMmaWarp) {
    // -------------------------------------------------------------------- MMA issuer
    constexpr uint32_t IDESC = tc::idesc_bf16_f32(kTileM, NDIM, false, false);
    for (int t = t_begin, j = 0; t < t_end && !*abort_flag; ++t, ++j) {
      const int buf = j & 1;
      if (j >= 2 && !tc::mbar_wait_bounded(acc_empty + buf, ((j >> 1) - 1) & 1)) *abort_flag = 1;
      for (int kb = 0; kb < KB; ++kb) {
        if (!tc::mbar_wait_bounded(full + kb, j & 1)) *abort_flag = 1;
        tc::fence_proxy_async_smem();
        tc::tc_fence_after_sync();
        if (lane == 0 && !*abort_flag) {
#pragma unroll
          for (int ks = 0; ks < 4; ++ks)
#pragma unroll
            for (int pr = 0; pr < 6; ++pr) {   // limb pairs, smallest products first: a3b1 a2b2 a1b3 a2b1 a1b2 a1b1
              const int la = pr == 0 ? 2 : (pr == 1 || pr == 3) ? 1 : 0;
              const int lb = pr == 0 ? 0 : pr == 1 ? 1 : pr == 2 ? 2 : pr == 3 ? 0 : pr == 4 ? 1 : 0;
              const uint64_t ad = tc::smem_desc_sw128(sA + kb * A_SLOT + la * A_LIMB + ks * 32, 16, 1024);
              const uint64_t bd = tc::smem_desc_sw128(sB + kb * B_SLOT + lb * B_LIMB + ks * 32, 16, 1024);
              if (pr == 5) tc::mma_bf16(tmem + buf * 2 * NDIM, ad, bd, IDESC, (kb | ks) != 0);
              else tc::mma_bf16(tmem + buf * 2 * NDIM + NDIM, ad, bd, IDESC, (kb | ks | pr) != 0);
            }
          tc::mma_commit(empty + kb);
          if (kb == KB - 1) tc::mma_commit(acc_full + buf);
        }
        __syncwarp();
      }
    }
  } else {
    // ---------------------------------------------------------------------- epilogue
    const int row = warp * 32 + lane;
    const uint32_t stage = sbase + A_BYTES + B_BYTES + 256 + warp * 4096;
    for (int t = t_begin, j = 0; t < t_end && !*abort_flag; ++t, ++j) {
      const int buf = j & 1;
      const int64_t row0 = tile_row0[t];
      const int rows = tile_rows[t];
      const bool valid = row < rows;
      const float s = (row_scale && valid) ? row_scale[row0 + row] : 1.0f;
      const float* wv = dot_out ? dot_w + (int64_t)node_part[row0] * dot_stride : nullptr;
      float dot = 0.0f;
      if (!tc::mbar_wait_bounded(acc_full + buf, (j >> 1) & 1)) { *abort_flag = 1; break; }
      tc::tc_fence_after_sync();
      const int rows_here = rows - warp * 32;
#pragma unroll 1
      for (int c0 = 0; c0 < NDIM; c0 += 32) {
        // ReLU-derivative mask, read where the result will be stored, requested before the accumulator
        float4 mk[8];
        if (relu_mask) {
#pragma unroll
          for (int it = 0; it < 8; ++it) {
            const int rr = it * 4 + (lane >> 3);
            mk[it] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (rr < rows_here)
              mk[it] = __ldg(reinterpret_cast<const float4*>(relu_mask + (row0 + warp * 32 + rr) * NDIM + c0 + (lane & 7) * 4));
          }
        }
        uint32_t r[32], rs[32];
        tc::tmem_ld_32x32(tmem + ((uint32_t)(warp * 32) << 16) + buf * 2 * NDIM + c0, r);
        tc::tmem_ld_32x32(tmem + ((uint32_t)(warp * 32) << 16) + buf * 2 * NDIM + NDIM + c0, rs);
        tc::tmem_ld_wait();
#pragma unroll
        for (int q = 0; q < 32; ++q) {
          float a = (__uint_as_float(r[q]) + __uint_as_float(rs[q])) * s;
          if (relu) a = a > 0.0f ? a : 0.0f;
          r[q] = __float_as_uint(a);
        }
        if (wv) {
#pragma unroll
          for (int q4 = 0; q4 < 8; ++q4) {
            const float4 w4 = __ldg(reinterpret_cast<const float4*>(wv + c0 + q4 * 4));
            dot = fmaf(__uint_as_float(r[4 * q4]), w4.x, dot);
            dot = fmaf(__uint_as_float(r[4 * q4 + 1]), w4.y, dot);
            dot = fmaf(__uint_as_float(r[4 * q4 + 2]), w4.z, dot);
            dot = fmaf(__uint_as_float(r[4 * q4 + 3]), w4.w, dot);
          }
        }
        __syncwarp();
#pragma unroll
        for (int pc = 0; pc < 8; ++pc)
          tc::st_shared16(stage + lane * 128 + ((pc ^ (lane & 7)) << 4), r[4 * pc], r[4 * pc + 1], r[4 * pc + 2],
                          r[4 * pc + 3]);
        __syncwarp();
#pragma unroll
        for (int it = 0; it < 8; ++it) {
          const int rr = it * 4 + (lane >> 3), pc = lane & 7;
          uint4 v = tc::ld_shared16(stage + rr * 128 + ((pc ^ (rr & 7)) << 4));
          if (relu_mask) {
            if (!(mk[it].x > 0.0f)) v.x = 0u;
            if (!(mk[it].y > 0.0f)) v.y = 0u;
            if (!(mk[it].z > 0.0f)) v.z = 0u;
            if (!(mk[it].w > 0.0f)) v.w = 0u;
          }
          if (rr < rows_here) *reinterpret_cast<uint4*>(Y + (row0 + warp * 32 + rr) * NDIM + c0 + pc * 4) = v;
        }
      }
      if (dot_out && valid) dot_out[row0 + row] = dot;
      tc::tc_fence_before_sync();
      tc::mbar_arrive(acc_empty + buf);
    }
  }
  if (*abort_flag && threadIdx.x == 0) atomicMin(status, (int32_t)GNNCO_INTERNAL);
  tc::tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) tc::tmem_dealloc(tmem, 4 * NDIM);
}

template <int KDIM, int NDIM>
int32_t launch_tf(gnnco_handle* h, const void* A, const void* B, int64_t b_stride, int64_t b_limb_stride, void* Y,
                  bool relu, const float* row_scale, const void* relu_mask, const void* dot_w, int64_t dot_stride,
                  float* dot_out, cudaStream_t st) {
  constexpr int KB = KDIM / 64;
  constexpr size_t smem = (size_t)KB * 3 * (kTileM + NDIM) * 128 + 256 + kEpiWarps * 4096 + 1024;
  static_assert(smem <= 232448, "tile does not fit in shared memory");
  GNNCO_CUDA_TRY(cudaFuncSetAttribute(transform_tc_f32<KDIM, NDIM>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)smem));
  int sms = h->sm_count > 0 ? h->sm_count : 148;
  int grid = h->n_tiles < sms ? h->n_tiles : sms;
  int per = (h->n_tiles + grid - 1) / grid;
  grid = (h->n_tiles + per - 1) / per;
  transform_tc_f32<KDIM, NDIM><<<grid, kTfThreads, smem, st>>>(
      (const float*)A, (const __nv_bfloat16*)B, b_stride, b_limb_stride, (float*)Y, relu ? 1 : 0, row_scale,
      (const float*)relu_mask, (const float*)dot_w, dot_stride, dot_out, h->tile_row0, h->tile_rows, h->node_part, h->n_tiles, per, h->status);
  h->launches += 1;
  GNNCO_LAUNCH_CHECK();
  return GNNCO_OK;
}

// -------------------------------------------------------------------------- weight gradient
// dW_s[KF x NF] = sum_{i in s} A[i,:]^T G[i,:], both float32, both split into limbs while
// they are staged (MN-major SW128, 64 rows per stage, two stages).
constexpr int kWgRows = 64;

template <int KF, int NF>
__global__ void __launch_bounds__(kThreads, 1)
weight_grad_tc_f32(const float* __restrict__ A, const float* __restrict__ G, float* __restrict__ dW,
                   float* __restrict__ scratch, const int32_t* __restrict__ wg_begin,
               const int32_t* __restrict__ wg_end, const int32_t* __restrict__ wg_slot, int32_t* status) {
  static_assert(KF == 128, "one 128-lane accumulator");
  constexpr uint32_t A_LIMB = KF * 128, G_LIMB = NF * 128;            // 64 rows x (DIM/64 blocks of 128 B)
  constexpr uint32_t STAGE = 3 * (A_LIMB + G_LIMB);
  constexpr int STAGES = 2;
  constexpr uint32_t TMEM_COLS = 2 * NF;                  // leading and correction accumulators
  extern __shared__ uint8_t smem_raw[];
  const uint32_t sbase = (tc::smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* gen_base = smem_raw + (sbase - tc::smem_u32(smem_raw));
  uint64_t* bars = reinterpret_cast<uint64_t*>(gen_base + STAGES * STAGE);        // [STAGES] consumed, [STAGES] all done
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + STAGES + 1);
  uint32_t* abort_flag = tmem_slot + 1;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // one block per chunk of rows; a chunk writes either a subgraph's result or a scratch slot
  const int64_t ra = wg_begin[blockIdx.x], rb = wg_end[blockIdx.x];
  const int32_t slot = wg_slot[blockIdx.x];
  float* out = slot < 0 ? dW + (int64_t)(-(slot + 1)) * KF * NF : scratch + (int64_t)slot * KF * NF;
  const int iters = (int)((rb - ra + kWgRows - 1) / kWgRows);
  if (iters == 0) {
    for (int q = threadIdx.x; q < KF * NF; q += kThreads) out[q] = 0.0f;
    return;
  }
  if (threadIdx.x == 0) {
    for (int i = 0; i <= STAGES; ++i) tc::mbar_init(bars + i, 1);
    *abort_flag = 0;
    tc::fence_mbar_init();
  }
  if (warp == 0) tc::tmem_alloc(tmem_slot, TMEM_COLS);
  tc::tc_fence_before_sync();
  __syncthreads();
  tc::tc_fence_after_sync();
  const uint32_t tmem = *tmem_slot;
  constexpr uint32_t IDESC = tc::idesc_bf16_f32(128, NF, true, true);
  constexpr int CA = KF / 8, CG = NF / 8;                 // 32-byte source chunks per row
  constexpr int CHUNKS = kWgRows * (CA + CG);
  constexpr int PER_THREAD = CHUNKS / kThreads;           // 8 (128+128) or 6 (128+64)
  static_assert(CHUNKS % kThreads == 0, "chunk count must divide evenly");
  bool failed = false;
  for (int it = 0; it < iters; ++it) {
    const int slot = it % STAGES;
    if (it >= STAGES) {
      const int prev = it - STAGES;
      if (!tc::mbar_wait_bounded(bars + slot, (prev / STAGES) & 1)) *abort_flag = 1;
    }
    const uint32_t sb = sbase + slot * STAGE;
    const int64_t r0 = ra + (int64_t)it * kWgRows;
    // the loads below go through registers and wait for their data: have the rows of the
    // iteration after next (contiguous in both operands) on their way into L2
    if (threadIdx.x < 2 && it + 2 < iters) {
      const int64_t rp = r0 + 2 * kWgRows;
      const uint32_t nrows = (uint32_t)min((int64_t)kWgRows, rb - rp);
      if (threadIdx.x == 0) tc::prefetch_l2(A + rp * KF, nrows * KF * 4);
      else tc::prefetch_l2(G + rp * NF, nrows * NF * 4);
    }
    // stage 64 rows of A and G: load float32, split, store the three limbs
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      float4 x[PER_THREAD / 2], y[PER_THREAD / 2];
#pragma unroll
      for (int u = 0; u < PER_THREAD / 2; ++u) {
        const int q = threadIdx.x + (half * (PER_THREAD / 2) + u) * kThreads;
        const bool isA = q < kWgRows * CA;
        const int qq = isA ? q : q - kWgRows * CA;
        const int k = isA ? qq / CA : qq / CG, c = isA ? qq % CA : qq % CG;
        x[u] = make_float4(0.f, 0.f, 0.f, 0.f);
        y[u] = x[u];
        if (r0 + k < rb) {
          const float4* g = reinterpret_cast<const float4*>((isA ? A + (r0 + k) * KF : G + (r0 + k) * NF) + c * 8);
          x[u] = __ldg(g);
          y[u] = __ldg(g + 1);
        }
      }
#pragma unroll
      for (int u = 0; u < PER_THREAD / 2; ++u) {
        const int q = threadIdx.x + (half * (PER_THREAD / 2) + u) * kThreads;
        const bool isA = q < kWgRows * CA;
        const int qq = isA ? q : q - kWgRows * CA;
        const int k = isA ? qq / CA : qq / CG, c = isA ? qq % CA : qq % CG;
        const int mb = c >> 3, cc = c & 7;
        uint4 l1, l2, l3;
        split3(x[u], y[u], l1, l2, l3);
        const uint32_t limb = isA ? A_LIMB : G_LIMB;
        const uint32_t dst = sb + (isA ? 0 : 3 * A_LIMB) + mb * (kWgRows * 128) + (k >> 3) * 1024 + (k & 7) * 128 +
                             ((cc ^ (k & 7)) << 4);
        tc::st_shared16(dst, l1.x, l1.y, l1.z, l1.w);
        tc::st_shared16(dst + limb, l2.x, l2.y, l2.z, l2.w);
        tc::st_shared16(dst + 2 * limb, l3.x, l3.y, l3.z, l3.w);
      }
    }
    tc::fence_proxy_async_smem();
    __syncthreads();
    if (*abort_flag) { failed = true; break; }
    if (threadIdx.x == 0) {
      tc::tc_fence_after_sync();
#pragma unroll
      for (int j = 0; j < kWgRows / 16; ++j)
#pragma unroll
        for (int pr = 0; pr < 6; ++pr) {
          const int la = pr == 0 ? 2 : (pr == 1 || pr == 3) ? 1 : 0;
          const int lb = pr == 0 ? 0 : pr == 1 ? 1 : pr == 2 ? 2 : pr == 3 ? 0 : pr == 4 ? 1 : 0;
          const uint64_t ad = tc::smem_desc_sw128(sb + la * A_LIMB + j * 2048, kWgRows * 128, 1024);
          const uint64_t gd = tc::smem_desc_sw128(sb + 3 * A_LIMB + lb * G_LIMB + j * 2048, kWgRows * 128, 1024);
          if (pr == 5) tc::mma_bf16(tmem, ad, gd, IDESC, (it | j) != 0);
          else tc::mma_bf16(tmem + NF, ad, gd, IDESC, (it | j | pr) != 0);
        }
      tc::mma_commit(bars + slot);
      if (it == iters - 1) tc::mma_commit(bars + STAGES);
    }
  }
  if (!failed) {
    if (!tc::mbar_wait_bounded(bars + STAGES, 0)) *abort_flag = 1;
    __syncthreads();
    failed = *abort_flag != 0;
  }
  if (failed) {
    if (threadIdx.x == 0) atomicMin(status, (int32_t)GNNCO_INTERNAL);
  } else {
    tc::tc_fence_after_sync();
    const int lg = warp & 3, ch = warp >> 2;
    constexpr int HALF = NF / 2;
    const int f = lg * 32 + lane;
#pragma unroll
    for (int c0 = 0; c0 < HALF; c0 += 32) {
      uint32_t r[32], rs[32];
      tc::tmem_ld_32x32(tmem + ((uint32_t)(lg * 32) << 16) + ch * HALF + c0, r);
      tc::tmem_ld_32x32(tmem + ((uint32_t)(lg * 32) << 16) + NF + ch * HALF + c0, rs);
      tc::tmem_ld_wait();
#pragma unroll
      for (int q = 0; q < 32; ++q) r[q] = __float_as_uint(__uint_as_float(r[q]) + __uint_as_float(rs[q]));
      uint4* dst = reinterpret_cast<uint4*>(out + (int64_t)f * NF + ch * HALF + c0);
#pragma unroll
      for (int j = 0; j < 8; ++j) dst[j] = make_uint4(r[4 * j], r[4 * j + 1], r[4 * j + 2], r[4 * j + 3]);
    }
  }
  tc::tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) tc::tmem_dealloc(tmem, TMEM_COLS);
}

template <int KF, int NF>
int32_t launch_wgf(gnnco_handle* h, const void* A, const void* G, float* dW, float* scratch, cudaStream_t st) {
  constexpr size_t smem = (size_t)2 * 3 * (KF + NF) * 128 + 128 + 1024;
  static_assert(smem <= 232448, "stages do not fit in shared memory");
  GNNCO_CUDA_TRY(cudaFuncSetAttribute(weight_grad_tc_f32<KF, NF>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)smem));
  weight_grad_tc_f32<KF, NF><<<h->n_wg_chunks, kThreads, smem, st>>>((const float*)A, (const float*)G, dW, scratch,
                                                                     h->wg_begin, h->wg_end, h->wg_slot, h->status);
  h->launches += 1;
  GNNCO_LAUNCH_CHECK();
  return launch_wg_combine(h, scratch, dW, (int64_t)KF * NF, st);
}

// W [sets][K][N] float32 -> three bf16 limb copies, either in place ([sets][K][N]) or
// transposed ([sets][N][K]); limb l starts at out + l * sets*K*N.
__global__ void cast_split3_kernel(const float* __restrict__ W, __nv_bfloat16* __restrict__ out, int K, int N,
                                   int64_t limb_stride, int transpose) {
  __shared__ float tile[32][33];
  const int64_t base = (int64_t)blockIdx.x * K * N;          // the set index is on x (no 65,535 limit there)
  const int k0 = blockIdx.y * 32, n0 = blockIdx.z * 32;
  for (int j = threadIdx.y; j < 32; j += 8) {
    int k = k0 + j, n = n0 + threadIdx.x;
    tile[j][threadIdx.x] = (k < K && n < N) ? W[base + (int64_t)k * N + n] : 0.0f;
  }
  __syncthreads();
  for (int j = threadIdx.y; j < 32; j += 8) {
    int64_t dst;
    float a;
    if (transpose) {
      int n = n0 + j, k = k0 + threadIdx.x;
      if (n >= N || k >= K) continue;
      a = tile[threadIdx.x][j];
      dst = base + (int64_t)n * K + k;
    } else {
      int k = k0 + j, n = n0 + threadIdx.x;
      if (n >= N || k >= K) continue;
      a = tile[j][threadIdx.x];
      dst = base + (int64_t)k * N + n;
    }
    const __nv_bfloat16 l1 = __float2bfloat16_rn(a);
    const float r1 = a - __bfloat162float(l1);
    const __nv_bfloat16 l2 = __float2bfloat16_rn(r1);
    const __nv_bfloat16 l3 = __float2bfloat16_rn(r1 - __bfloat162float(l2));
    out[dst] = l1;
    out[dst + limb_stride] = l2;
    out[dst + 2 * limb_stride] = l3;
  }
}

}  // namespace

bool tc_f32_transform_supported(int K, int N) { return (K == 64 || K == 128) && (N == 64 || N == 128); }
bool tc_f32_weight_grad_supported(int K, int N) { return K == 128 && (N == 64 || N == 128); }

// Y = act(A B_s^T) * row_scale, A float32 [n x K], B = three bf16 limb copies of [sets x N x K]
int32_t launch_transform_tc_f32(gnnco_handle* h, const void* A, const void* B_limbs, int64_t b_stride,
                                int64_t b_limb_stride, void* Y, int K, int N, bool relu, const float* row_scale,
                                const void* relu_mask, bool backward, const void* dot_w, int64_t dot_stride,
                                float* dot_out, cudaStream_t st) {
  if (h->n_tiles == 0) return GNNCO_OK;
  ProfScope prof_(h, backward ? K_TRANSFORM_BWD : K_TRANSFORM_FWD, st);
#define GNNCO_TF_CASE(KK, NN)    \
  if (K == KK && N == NN)        \
  return launch_tf<KK, NN>(h, A, B_limbs, b_stride, b_limb_stride, Y, relu, row_scale, relu_mask, dot_w, dot_stride, \
                           dot_out, st)
  GNNCO_TF_CASE(64, 64); GNNCO_TF_CASE(64, 128); GNNCO_TF_CASE(128, 64); GNNCO_TF_CASE(128, 128);
#undef GNNCO_TF_CASE
  return GNNCO_UNSUPPORTED;
}

int32_t launch_weight_grad_tc_f32(gnnco_handle* h, const void* A, const void* G, float* dW, float* scratch, int K,
                                  int N, cudaStream_t st) {
  ProfScope prof_(h, K_WEIGHT_GRAD, st);
  if (K == 128 && N == 64) return launch_wgf<128, 64>(h, A, G, dW, scratch, st);
  if (K == 128 && N == 128) return launch_wgf<128, 128>(h, A, G, dW, scratch, st);
  return GNNCO_UNSUPPORTED;
}

int32_t launch_cast_split3(gnnco_handle* h, const float* W, __nv_bfloat16* out, int K, int N, int32_t sets,
                           bool transpose, cudaStream_t st) {
  ProfScope prof_(h, K_CAST, st);
  dim3 grid(sets, (K + 31) / 32, (N + 31) / 32);
  if (grid.y > 65535 || grid.z > 65535) return GNNCO_UNSUPPORTED;
  cast_split3_kernel<<<grid, dim3(32, 8), 0, st>>>(W, out, K, N, (int64_t)sets * K * N, transpose ? 1 : 0);
  h->launches += 1;
  GNNCO_LAUNCH_CHECK();
  return GNNCO_OK;
}
