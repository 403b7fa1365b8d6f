// Dense per-subgraph transform on the sm_100a tensor cores (tcgen05 + TMEM), bf16 operands
// with float32 accumulation (Eq. 3's "... W" and its input gradient).
//
//   Y[tile, :] = act( A[tile, 0:K] * B_s^T ) * row_scale,    B_s = [N x K], K contiguous
//   (optionally zeroed where a saved activation of Y's shape is <= 0: the ReLU derivative)
//
// Forward uses B = W^T (bf16 copy, transposed), the input gradient uses B = W (bf16 copy), so
// both operands are K-major.  One CTA owns a run of consecutive 128-row tiles; consecutive
// tiles mostly belong to the same subgraph, so its weight matrix stays in shared memory.
// Operands are staged with 16-byte cp.async copies into the 128-byte-swizzled layout the
// tensor core expects; one thread issues the MMAs, the accumulator (128 lanes x N columns of
// TMEM) is read back by all eight warps, scaled / rectified, rounded to bf16 and stored.
// The copies of the next tile are in flight while the current accumulator is drained.
#include "internal.cuh"
#include "tc_common.cuh"

namespace {

constexpr int kTileM = 128;
constexpr int kThreads = 256;                // weight-gradient kernel
constexpr int kTfThreads = 384;              // transform kernel

// Roles of the twelve warps of the transform kernel.
constexpr int kEpiWarps = 8;                 // warps 0-7 drain the accumulator: TMEM lane quarter (warp % 4), column half (warp / 4)
constexpr int kMmaWarp = 8;                  // warp 8 issues the MMAs
constexpr int kProdWarp0 = 9;                // warps 9-11 stage operands with cp.async
constexpr int kProdLanes = 96;

constexpr uint32_t kTfMiscBytes = 1536;      // barriers (256 B) + two 128-float dot-product exchange buffers

// One 64-wide k-block of `rows` rows (row stride KDIM elements) -> K-major SW128 shared memory:
// row r at (r/8)*1024 + (r%8)*128, 16-byte chunk c at ((c ^ (r%8)) * 16).  Called by the 96
// producer lanes; p = producer lane index.
template <int KDIM>
__device__ __forceinline__ void stage_kblock(uint32_t sdst, const __nv_bfloat16* __restrict__ g, int rows, int p) {
  for (int q = p; q < rows * 8; q += kProdLanes) {
    const int r = q >> 3, cc = q & 7;
    tc::cp_async16(sdst + (r >> 3) * 1024 + (r & 7) * 128 + ((cc ^ (r & 7)) << 4), g + (int64_t)r * KDIM + cc * 8);
  }
}

// keep the bf16 halves of v where the matching halves of m are positive
__device__ __forceinline__ uint32_t keep_where_positive(uint32_t v, uint32_t m) {
  const uint32_t lo = __uint_as_float(m << 16) > 0.0f ? 0x0000ffffu : 0u;
  const uint32_t hi = __uint_as_float(m & 0xffff0000u) > 0.0f ? 0xffff0000u : 0u;
  return v & (lo | hi);
}

// Warp-specialised, persistent.  Shared memory: the subgraph's weight matrix (KB k-blocks of
// NDIM rows) and one 128-row operand tile as KB independently recycled k-block slots.
//   producers : wait until the MMAs that read slot kb are done, refill it (and the matching
//               weight k-block when the subgraph changes), arrive on full[kb] when the copies land
//   MMA warp  : for each k-block wait full[kb], issue 4 MMAs (K = 16 each) into accumulator
//               buffer (tile & 1), commit -> empty[kb]; after the last k-block commit -> acc_full
//   epilogue  : two warps per TMEM lane quarter, each owning half of the columns: request the
//               ReLU-mask lines of the tile (MASKED instantiation), wait acc_full, read the
//               accumulator (TMEM -> registers; without a mask the next chunk's read is issued
//               before the current chunk is stored, so its latency hides behind the stores),
//               scale / rectify / round to bf16, store; optionally the
//               next layer's row dot product (the two column halves meet in shared memory);
//               arrive acc_empty
// so the copies of tile t+1, the MMAs of tile t+1 and the drain of tile t overlap.
template <int KDIM, int NDIM, bool MASKED>
__global__ void __launch_bounds__(kTfThreads, 1)
transform_tc(const __nv_bfloat16* __restrict__ A, const __nv_bfloat16* __restrict__ B, int64_t b_stride,
             __nv_bfloat16* __restrict__ Y, int relu, const float* __restrict__ row_scale,
             const __nv_bfloat16* __restrict__ relu_mask, const __nv_bfloat16* __restrict__ dot_w, int64_t dot_stride, float* __restrict__ dot_out,
             const int32_t* __restrict__ tile_row0, const int32_t* __restrict__ tile_rows,
             const int32_t* __restrict__ node_part, int n_tiles, int tiles_per_cta, int32_t* status) {
  constexpr int KB = KDIM / 64;
  constexpr uint32_t A_SLOT = kTileM * 128, B_SLOT = NDIM * 128;
  constexpr uint32_t A_BYTES = KB * A_SLOT, B_BYTES = KB * B_SLOT;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t sbase = (tc::smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sA = sbase, sB = sbase + A_BYTES;
  uint8_t* gen_base = smem_raw + (sbase - tc::smem_u32(smem_raw));
  uint64_t* full = reinterpret_cast<uint64_t*>(gen_base + A_BYTES + B_BYTES);   // [KB]
  uint64_t* empty = full + KB;                                                  // [KB]
  uint64_t* acc_full = empty + KB;                                              // [2]
  uint64_t* acc_empty = acc_full + 2;                                           // [2]
  uint64_t* dot_bar = acc_empty + 2;                                            // [4 quarters][2 buffers]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(dot_bar + 8);
  volatile uint32_t* abort_flag = tmem_slot + 1;
  float* dot_x = reinterpret_cast<float*>(gen_base + A_BYTES + B_BYTES + 256);  // [2][128] upper column half's share

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
    for (int i = 0; i < 8; ++i) tc::mbar_init(dot_bar + i, 32);
    *abort_flag = 0;
    tc::fence_mbar_init();
  }
  if (warp == 0) tc::tmem_alloc(tmem_slot, 2 * NDIM);
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
      // (no L2 prefetch of later tiles here: the cp.async copies keep a whole tile in flight, and a
      // prefetch was measured to add 17-25 % DRAM reads -- lines evicted before use -- for no gain)
      for (int kb = 0; kb < KB; ++kb) {
        if (j > 0 && !tc::mbar_wait_bounded(empty + kb, (j - 1) & 1)) *abort_flag = 1;
        if (new_b) stage_kblock<KDIM>(sB + kb * B_SLOT, B + (int64_t)part * b_stride + kb * 64, NDIM, p);
        stage_kblock<KDIM>(sA + kb * A_SLOT, A + row0 * KDIM + kb * 64, rows, p);   // rows past `rows` keep old bits: they only reach output rows that are never stored
        tc::cp_async_arrive_noinc(full + kb);
      }
    }
    tc::cp_async_wait<0>();
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
          for (int ks = 0; ks < 4; ++ks) {
            const uint64_t ad = tc::smem_desc_sw128(sA + kb * A_SLOT + ks * 32, 16, 1024);
            const uint64_t bd = tc::smem_desc_sw128(sB + kb * B_SLOT + ks * 32, 16, 1024);
            tc::mma_bf16(tmem + buf * NDIM, ad, bd, IDESC, (kb | ks) != 0);
          }
          tc::mma_commit(empty + kb);
          if (kb == KB - 1) tc::mma_commit(acc_full + buf);
        }
        __syncwarp();
      }
    }
  } else {
    // ---------------------------------------------------------------------- epilogue
    constexpr int CHUNKS = NDIM / 64;                 // 64-column chunks of the tile
    constexpr int PER = (CHUNKS + 1) / 2;             // chunks per column half
    const int quarter = warp & 3, half = warp >> 2;
    const int ch_begin = half * PER, ch_end = min(CHUNKS, ch_begin + PER);
    const int row = quarter * 32 + lane;
    const uint32_t stage = sbase + A_BYTES + B_BYTES + kTfMiscBytes + warp * 4096;
    for (int t = t_begin, j = 0; t < t_end && !*abort_flag; ++t, ++j) {
      const int buf = j & 1;
      const int64_t row0 = tile_row0[t];
      const int rows = tile_rows[t];
      const bool valid = row < rows;
      const int rows_here = rows - quarter * 32;       // valid rows of this warp's 32
      // the mask is read where the result will be stored (whole lines); every line of the tile
      // that this warp needs is requested before the accumulator is waited for
      uint4 mk[MASKED ? PER : 1][8];
      if (MASKED) {
#pragma unroll
        for (int c = 0; c < PER; ++c)
#pragma unroll
          for (int it = 0; it < 8; ++it) {
            const int rr = it * 4 + (lane >> 3);
            mk[c][it] = make_uint4(0u, 0u, 0u, 0u);
            if (rr < rows_here && ch_begin + c < ch_end)
              mk[c][it] = __ldg(reinterpret_cast<const uint4*>(relu_mask + (row0 + quarter * 32 + rr) * NDIM +
                                                               (ch_begin + c) * 64 + (lane & 7) * 8));
          }
      }
      const float s = (row_scale && valid) ? row_scale[row0 + row] : 1.0f;
      const __nv_bfloat16* wv = nullptr;
      if (dot_out) wv = dot_w + (int64_t)node_part[row0] * dot_stride;
      float dot = 0.0f;
      if (!tc::mbar_wait_bounded(acc_full + buf, (j >> 1) & 1)) { *abort_flag = 1; break; }
      tc::tc_fence_after_sync();
      // the 64 columns of a chunk are read with two 32-column loads and one wait
      uint32_t ra[32], rb[32];
      auto read_chunk = [&](int c) {
        const uint32_t at = tmem + ((uint32_t)(quarter * 32) << 16) + buf * NDIM + (ch_begin + c) * 64;
        tc::tmem_ld_32x32(at, ra);
        tc::tmem_ld_32x32(at + 32, rb);
      };
      if (!MASKED && ch_begin < ch_end) read_chunk(0);
#pragma unroll
      for (int c = 0; c < PER; ++c) {
        if (ch_begin + c >= ch_end) break;
        const int c0 = (ch_begin + c) * 64;
        uint32_t o[32];                                // 64 bf16 of this thread's row, packed
        auto convert = [&](const uint32_t (&r)[32], int at) {
#pragma unroll
          for (int q = 0; q < 16; ++q) {
            float a = __uint_as_float(r[2 * q]) * s, b = __uint_as_float(r[2 * q + 1]) * s;
            if (relu) { a = a > 0.0f ? a : 0.0f; b = b > 0.0f ? b : 0.0f; }
            __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
            o[at + q] = *reinterpret_cast<uint32_t*>(&v);
          }
        };
        if (MASKED) {
          // the mask lines hold 64 registers: one 32-column read at a time
#pragma unroll
          for (int hh = 0; hh < 2; ++hh) {
            tc::tmem_ld_32x32(tmem + ((uint32_t)(quarter * 32) << 16) + buf * NDIM + c0 + hh * 32, ra);
            tc::tmem_ld_wait();
            convert(ra, hh * 16);
          }
        } else {
          tc::tmem_ld_wait();
          convert(ra, 0);
          convert(rb, 16);
          // the accumulator registers are free again: the next chunk's read goes out now and
          // lands while this chunk is being stored
          if (c + 1 < PER && ch_begin + c + 1 < ch_end) read_chunk(c + 1);
        }
        if (wv) {   // dot product of the STORED (rounded) row with the next layer's weight vector
#pragma unroll
          for (int q4 = 0; q4 < 8; ++q4) {
            const uint4 w8 = __ldg(reinterpret_cast<const uint4*>(wv + c0 + q4 * 8));
            const uint32_t wq[4] = {w8.x, w8.y, w8.z, w8.w};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const uint32_t hv = o[q4 * 4 + q];
              dot = fmaf(__uint_as_float(hv << 16), __uint_as_float(wq[q] << 16), dot);
              dot = fmaf(__uint_as_float(hv & 0xffff0000u), __uint_as_float(wq[q] & 0xffff0000u), dot);
            }
          }
        }
        // through a per-warp staging tile (32 rows x 128 bytes, pieces XOR-swizzled by row) so
        // that each store instruction writes whole 128-byte lines: 8 lanes per row, 4 rows
        __syncwarp();
#pragma unroll
        for (int pc = 0; pc < 8; ++pc)
          tc::st_shared16(stage + lane * 128 + ((pc ^ (lane & 7)) << 4), o[4 * pc], o[4 * pc + 1], o[4 * pc + 2],
                          o[4 * pc + 3]);
        __syncwarp();
#pragma unroll
        for (int it = 0; it < 8; ++it) {
          const int rr = it * 4 + (lane >> 3), pc = lane & 7;
          uint4 v = tc::ld_shared16(stage + rr * 128 + ((pc ^ (rr & 7)) << 4));
          if (MASKED) {
            v.x = keep_where_positive(v.x, mk[c][it].x); v.y = keep_where_positive(v.y, mk[c][it].y);
            v.z = keep_where_positive(v.z, mk[c][it].z); v.w = keep_where_positive(v.w, mk[c][it].w);
          }
          if (rr < rows_here)
            *reinterpret_cast<uint4*>(Y + (row0 + quarter * 32 + rr) * NDIM + c0 + pc * 8) = v;
        }
      }
      if (dot_out) {
        // lower column half + upper column half, in that order.  The exchange buffer of this
        // accumulator buffer is free again once the lower half has arrived on acc_empty below:
        // the upper half cannot reach its next write before the MMAs of tile j + 2 are done.
        if (CHUNKS > 1 && half == 1) {
          dot_x[buf * 128 + row] = dot;
          tc::mbar_arrive(dot_bar + quarter * 2 + buf);
        }
        if (half == 0) {
          if (CHUNKS > 1) {
            if (!tc::mbar_wait_bounded(dot_bar + quarter * 2 + buf, (j >> 1) & 1)) { *abort_flag = 1; break; }
            dot += dot_x[buf * 128 + row];
          }
          if (valid) dot_out[row0 + row] = dot;
        }
      }
      tc::tc_fence_before_sync();
      tc::mbar_arrive(acc_empty + buf);
    }
  }
  if (*abort_flag && threadIdx.x == 0) atomicMin(status, (int32_t)GNNCO_INTERNAL);
  tc::tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) tc::tmem_dealloc(tmem, 2 * NDIM);
}

template <int KDIM, int NDIM>
int32_t launch_tc(gnnco_handle* h, const void* A, const void* B, int64_t b_stride, void* Y, bool relu,
                  const float* row_scale, const void* relu_mask, const void* dot_w, int64_t dot_stride, float* dot_out,
                  cudaStream_t st) {
  constexpr int KB = KDIM / 64;
  // operands, barriers and dot-product exchange, one 4 KB staging tile per epilogue warp, alignment slack
  constexpr size_t smem = (size_t)KB * (kTileM + NDIM) * 128 + kTfMiscBytes + kEpiWarps * 4096 + 1024;
  static_assert(smem <= 232448, "tile does not fit in shared memory");
  GNNCO_CUDA_TRY(cudaFuncSetAttribute(transform_tc<KDIM, NDIM, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)smem));
  GNNCO_CUDA_TRY(cudaFuncSetAttribute(transform_tc<KDIM, NDIM, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)smem));
  int sms = h->sm_count > 0 ? h->sm_count : 148;
  int grid = h->n_tiles < sms ? h->n_tiles : sms;
  int per = (h->n_tiles + grid - 1) / grid;
  grid = (h->n_tiles + per - 1) / per;
  if (relu_mask)
    transform_tc<KDIM, NDIM, true><<<grid, kTfThreads, smem, st>>>(
      (const __nv_bfloat16*)A, (const __nv_bfloat16*)B, b_stride, (__nv_bfloat16*)Y, relu ? 1 : 0, row_scale,
      (const __nv_bfloat16*)relu_mask, (const __nv_bfloat16*)dot_w, dot_stride, dot_out, h->tile_row0, h->tile_rows, h->node_part, h->n_tiles, per,
      h->status);
  else
    transform_tc<KDIM, NDIM, false><<<grid, kTfThreads, smem, st>>>(
      (const __nv_bfloat16*)A, (const __nv_bfloat16*)B, b_stride, (__nv_bfloat16*)Y, relu ? 1 : 0, row_scale,
      (const __nv_bfloat16*)relu_mask, (const __nv_bfloat16*)dot_w, dot_stride, dot_out, h->tile_row0, h->tile_rows, h->node_part, h->n_tiles, per,
      h->status);
  h->launches += 1;
  GNNCO_LAUNCH_CHECK();
  return GNNCO_OK;
}

// ------------------------------------------------------------------------------------
// Weight gradient on the tensor cores:  dW_s[KF x NF] = sum_{i in s} A[i, :]^T G[i, :]
// (the reduction runs over the rows of subgraph s, so both operands are MN-major: a row of
// A or G is 128-byte lines of 64 features, indexed by the reduction index).
// One CTA per subgraph; rows stream through a 3-stage cp.async pipeline in chunks of 64;
// the KF x NF accumulator lives in TMEM (two 128-lane halves when KF = 256) and is written
// out in float32 once at the end, in a fixed order (deterministic, no atomics).
constexpr int kWgRows = 64;      // reduction rows per pipeline stage
constexpr int kWgStages = 3;

// rows [r0, r0+64) of a [.. x DIM] bf16 matrix -> MN-major SW128 stage: feature block mb
// (64 features) at mb*8192, row k at (k/8)*1024 + (k%8)*128, chunk c at ((c ^ (k%8)) * 16)
template <int DIM>
__device__ __forceinline__ void stage_mn_major(uint32_t sbase, const __nv_bfloat16* __restrict__ g, int64_t r0,
                                               int64_t r_end) {
  constexpr int CPR = DIM / 8;
  constexpr int total = kWgRows * CPR;
  for (int q = threadIdx.x; q < total; q += kThreads) {
    const int k = q / CPR, c = q % CPR;
    const int mb = c >> 3, cc = c & 7;
    const uint32_t dst = sbase + mb * (kWgRows * 128) + (k >> 3) * 1024 + (k & 7) * 128 + ((cc ^ (k & 7)) << 4);
    if (r0 + k < r_end) tc::cp_async16(dst, g + (r0 + k) * DIM + c * 8);
    else tc::st_shared_zero16(dst);
  }
}

template <int KF, int NF>
__global__ void __launch_bounds__(kThreads, 1)
weight_grad_tc(const __nv_bfloat16* __restrict__ A, const __nv_bfloat16* __restrict__ G, float* __restrict__ dW,
               float* __restrict__ scratch, const int32_t* __restrict__ wg_begin,
               const int32_t* __restrict__ wg_end, const int32_t* __restrict__ wg_slot, int32_t* status) {
  constexpr int MH = KF / 128;                          // accumulator halves of 128 rows
  constexpr uint32_t A_STAGE = KF * 128, G_STAGE = NF * 128;
  constexpr uint32_t STAGE = A_STAGE + G_STAGE;
  constexpr uint32_t TMEM_COLS = MH * NF < 32 ? 32 : MH * NF;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t sbase = (tc::smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* gen_base = smem_raw + (sbase - tc::smem_u32(smem_raw));
  uint64_t* bars = reinterpret_cast<uint64_t*>(gen_base + kWgStages * STAGE);      // [stages] consumed, [stages] = all done
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + kWgStages + 1);
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
    for (int i = 0; i <= kWgStages; ++i) tc::mbar_init(bars + i, 1);
    *abort_flag = 0;
    tc::fence_mbar_init();
  }
  if (warp == 0) tc::tmem_alloc(tmem_slot, TMEM_COLS);
  tc::tc_fence_before_sync();
  __syncthreads();
  tc::tc_fence_after_sync();
  const uint32_t tmem = *tmem_slot;
  constexpr uint32_t IDESC = tc::idesc_bf16_f32(128, NF, true, true);

  auto load_stage = [&](int it) {
    if (it < iters) {
      const uint32_t sb = sbase + (it % kWgStages) * STAGE;
      stage_mn_major<KF>(sb, A, ra + (int64_t)it * kWgRows, rb);
      stage_mn_major<NF>(sb + A_STAGE, G, ra + (int64_t)it * kWgRows, rb);
    }
    tc::cp_async_commit();            // always commit: keeps the group count uniform
  };
  for (int it = 0; it < kWgStages - 1; ++it) load_stage(it);
  bool failed = false;
  for (int it = 0; it < iters; ++it) {
    tc::cp_async_wait<kWgStages - 2>();
    tc::fence_proxy_async_smem();
    __syncthreads();
    if (threadIdx.x == 0) {
      tc::tc_fence_after_sync();
      const uint32_t sb = sbase + (it % kWgStages) * STAGE;
#pragma unroll
      for (int j = 0; j < kWgRows / 16; ++j) {
        const uint64_t gd = tc::smem_desc_sw128(sb + A_STAGE + j * 2048, kWgRows * 128, 1024);
#pragma unroll
        for (int hm = 0; hm < MH; ++hm) {
          const uint64_t ad = tc::smem_desc_sw128(sb + hm * 2 * (kWgRows * 128) + j * 2048, kWgRows * 128, 1024);
          tc::mma_bf16(tmem + hm * NF, ad, gd, IDESC, (it | j) != 0);
        }
      }
      tc::mma_commit(bars + (it % kWgStages));
      if (it == iters - 1) tc::mma_commit(bars + kWgStages);
    }
    // the slot that iteration it-1 used is free once its MMAs have completed; refill it
    if (it >= 1) {
      const int prev = it - 1;
      if (!tc::mbar_wait_bounded(bars + (prev % kWgStages), (prev / kWgStages) & 1)) *abort_flag = 1;
    }
    __syncthreads();
    if (*abort_flag) { failed = true; break; }
    load_stage(it + kWgStages - 1);
  }
  if (!failed) {
    if (!tc::mbar_wait_bounded(bars + kWgStages, 0)) *abort_flag = 1;
    __syncthreads();
    failed = *abort_flag != 0;
  }
  tc::cp_async_wait<0>();
  if (failed) {
    if (threadIdx.x == 0) atomicMin(status, (int32_t)GNNCO_INTERNAL);
  } else {
    tc::tc_fence_after_sync();
    const int lg = warp & 3, ch = warp >> 2;
    constexpr int HALF = NF / 2;
#pragma unroll
    for (int hm = 0; hm < MH; ++hm) {
      const int f = hm * 128 + lg * 32 + lane;
#pragma unroll
      for (int c0 = 0; c0 < HALF; c0 += 32) {
        uint32_t r[32];
        tc::tmem_ld_32x32(tmem + ((uint32_t)(lg * 32) << 16) + hm * NF + ch * HALF + c0, r);
        tc::tmem_ld_wait();
        uint4* dst = reinterpret_cast<uint4*>(out + (int64_t)f * NF + ch * HALF + c0);
#pragma unroll
        for (int j = 0; j < 8; ++j) dst[j] = make_uint4(r[4 * j], r[4 * j + 1], r[4 * j + 2], r[4 * j + 3]);
      }
    }
  }
  tc::tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) tc::tmem_dealloc(tmem, TMEM_COLS);
}

template <int KF, int NF>
int32_t launch_wg(gnnco_handle* h, const void* A, const void* G, float* dW, float* scratch, cudaStream_t st) {
  constexpr size_t smem = (size_t)kWgStages * (KF + NF) * 128 + 128 + 1024;
  GNNCO_CUDA_TRY(cudaFuncSetAttribute(weight_grad_tc<KF, NF>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  weight_grad_tc<KF, NF><<<h->n_wg_chunks, kThreads, smem, st>>>((const __nv_bfloat16*)A, (const __nv_bfloat16*)G, dW,
                                                                 scratch, h->wg_begin, h->wg_end, h->wg_slot, h->status);
  h->launches += 1;
  GNNCO_LAUNCH_CHECK();
  return launch_wg_combine(h, scratch, dW, (int64_t)KF * NF, st);
}

// W [sets][K][N] float32 -> Wt [sets][N][K] bf16
__global__ void cast_transpose_bf16_kernel(const float* __restrict__ W, __nv_bfloat16* __restrict__ Wt, int K, int N) {
  __shared__ float tile[32][33];
  const int64_t base = (int64_t)blockIdx.x * K * N;          // the set index is on x (no 65,535 limit there)
  const int k0 = blockIdx.y * 32, n0 = blockIdx.z * 32;
  for (int j = threadIdx.y; j < 32; j += 8) {
    int k = k0 + j, n = n0 + threadIdx.x;
    tile[j][threadIdx.x] = (k < K && n < N) ? W[base + (int64_t)k * N + n] : 0.0f;
  }
  __syncthreads();
  for (int j = threadIdx.y; j < 32; j += 8) {
    int n = n0 + j, k = k0 + threadIdx.x;
    if (n < N && k < K) Wt[base + (int64_t)n * K + k] = __float2bfloat16_rn(tile[threadIdx.x][j]);
  }
}

// One pass over W [sets][K][N] float32 (K, N multiples of 64) that writes both bf16 copies the
// tensor-core transforms read: Wc [sets][K][N] and Wt [sets][N][K].  A block owns a 64 x 64 tile.
__global__ void __launch_bounds__(256) cast_both_bf16_kernel(const float* __restrict__ W, __nv_bfloat16* __restrict__ Wc,
                                                             __nv_bfloat16* __restrict__ Wt, int K, int N) {
  __shared__ float tile[64][65];
  const int64_t base = (int64_t)blockIdx.x * K * N;          // the set index is on x (no 65,535 limit there)
  const int k0 = blockIdx.y * 64, n0 = blockIdx.z * 64;
  const int q = threadIdx.x & 15, r = threadIdx.x >> 4;   // 16 threads of four elements across, 16 rows per pass
#pragma unroll
  for (int pass = 0; pass < 4; ++pass) {
    const int k = r + 16 * pass;
    const int64_t at = base + (int64_t)(k0 + k) * N + n0 + 4 * q;
    const float4 v = __ldg(reinterpret_cast<const float4*>(W + at));
    __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
    *reinterpret_cast<uint2*>(Wc + at) = make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
    tile[k][4 * q + 0] = v.x; tile[k][4 * q + 1] = v.y; tile[k][4 * q + 2] = v.z; tile[k][4 * q + 3] = v.w;
  }
  __syncthreads();
#pragma unroll
  for (int pass = 0; pass < 4; ++pass) {
    const int n = r + 16 * pass;
    __nv_bfloat162 lo = __floats2bfloat162_rn(tile[4 * q + 0][n], tile[4 * q + 1][n]);
    __nv_bfloat162 hi = __floats2bfloat162_rn(tile[4 * q + 2][n], tile[4 * q + 3][n]);
    *reinterpret_cast<uint2*>(Wt + base + (int64_t)(n0 + n) * K + k0 + 4 * q) =
        make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
  }
}

// Adam (same rule as adam_vec4_kernel) on W [sets][K][N] that also leaves behind the two bf16 copies of the
// UPDATED weights which the next step's tensor-core transforms read (Wc [sets][K][N], Wt [sets][N][K]),
// so that the next step need not read the master weights again just to round them.  A block owns a
// 64 x 64 tile.  Subgraphs that are not being fine-tuned are skipped: W, m and v stay bit for bit, and
// their copies are current already (the step made or vouched for them before its first matrix product).
__global__ void __launch_bounds__(256) adam_cast_both_kernel(float* __restrict__ W, float* __restrict__ m,
                                                             float* __restrict__ v, const float* __restrict__ g,
                                                             __nv_bfloat16* __restrict__ Wc, __nv_bfloat16* __restrict__ Wt,
                                                             int K, int N, float lr, float b1, float b2, float eps,
                                                             float inv_c1, float inv_c2,
                                                             const uint8_t* __restrict__ active,
                                                             const float2* __restrict__ bias) {
  __shared__ float tile[64][65];
  if (bias) {            // bias corrections kept on the device (a step counter there: adam_tick)
    inv_c1 = bias->x;
    inv_c2 = bias->y;
  }
  const int64_t base = (int64_t)blockIdx.x * K * N;          // the set index is on x (no 65,535 limit there)
  const int k0 = blockIdx.y * 64, n0 = blockIdx.z * 64;
  const int q = threadIdx.x & 15, r = threadIdx.x >> 4;   // 16 threads of four elements across, 16 rows per pass
  if (active && !active[blockIdx.x]) return;                // uniform across the block
#pragma unroll
  for (int pass = 0; pass < 4; ++pass) {
    const int k = r + 16 * pass;
    const int64_t at = base + (int64_t)(k0 + k) * N + n0 + 4 * q;
    float4 wq = *reinterpret_cast<const float4*>(W + at);
    {
      const float4 gq = __ldg(reinterpret_cast<const float4*>(g + at));
      float4 mq = *reinterpret_cast<const float4*>(m + at), vq = *reinterpret_cast<const float4*>(v + at);
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
      *reinterpret_cast<float4*>(m + at) = mq;
      *reinterpret_cast<float4*>(v + at) = vq;
      *reinterpret_cast<float4*>(W + at) = wq;
    }
    __nv_bfloat162 lo = __floats2bfloat162_rn(wq.x, wq.y), hi = __floats2bfloat162_rn(wq.z, wq.w);
    *reinterpret_cast<uint2*>(Wc + at) = make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
    tile[k][4 * q + 0] = wq.x; tile[k][4 * q + 1] = wq.y; tile[k][4 * q + 2] = wq.z; tile[k][4 * q + 3] = wq.w;
  }
  __syncthreads();
#pragma unroll
  for (int pass = 0; pass < 4; ++pass) {
    const int n = r + 16 * pass;
    __nv_bfloat162 lo = __floats2bfloat162_rn(tile[4 * q + 0][n], tile[4 * q + 1][n]);
    __nv_bfloat162 hi = __floats2bfloat162_rn(tile[4 * q + 2][n], tile[4 * q + 3][n]);
    *reinterpret_cast<uint2*>(Wt + base + (int64_t)(n0 + n) * K + k0 + 4 * q) =
        make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
  }
}

}  // namespace

bool tc_transform_supported(int dtype, int K, int N) {
  auto ok = [](int d) { return d == 64 || d == 128 || d == 256; };
  return dtype == GNNCO_BF16 && ok(K) && ok(N);
}

// Y = act(A B_s^T) * row_scale with A [n x K], B [sets x N x K] (both bf16, K contiguous),
// zeroed where relu_mask [n x N] (bf16, optional) is not positive.
// With dot_out != nullptr also dot_out[i] = Y[i,:] . dot_w[s,:] (the width-1 output layer's
// product, taken on the rounded values that are stored).
int32_t launch_transform_tc(gnnco_handle* h, const void* A, const void* B, int64_t b_stride, void* Y, int K, int N,
                            bool relu, const float* row_scale, const void* relu_mask, bool backward, const void* dot_w,
                            int64_t dot_stride, float* dot_out, cudaStream_t st) {
  if (h->n_tiles == 0) return GNNCO_OK;
  ProfScope prof_(h, backward ? K_TRANSFORM_BWD : K_TRANSFORM_FWD, st);
#define GNNCO_TC_CASE(KK, NN) \
  if (K == KK && N == NN)       \
  return launch_tc<KK, NN>(h, A, B, b_stride, Y, relu, row_scale, relu_mask, dot_w, dot_stride, dot_out, st)
  GNNCO_TC_CASE(64, 64); GNNCO_TC_CASE(64, 128); GNNCO_TC_CASE(64, 256);
  GNNCO_TC_CASE(128, 64); GNNCO_TC_CASE(128, 128); GNNCO_TC_CASE(128, 256);
  GNNCO_TC_CASE(256, 64); GNNCO_TC_CASE(256, 128); GNNCO_TC_CASE(256, 256);
#undef GNNCO_TC_CASE
  return GNNCO_UNSUPPORTED;
}

bool tc_weight_grad_supported(int dtype, int K, int N) {
  return dtype == GNNCO_BF16 && (K == 128 || K == 256) && (N == 64 || N == 128 || N == 256);
}

// dW[s] (K x N, float32) = sum_{i in s} A[i,:]^T G[i,:], A [n x K], G [n x N] bf16
int32_t launch_weight_grad_tc(gnnco_handle* h, const void* A, const void* G, float* dW, float* scratch, int K, int N,
                              cudaStream_t st) {
  ProfScope prof_(h, K_WEIGHT_GRAD, st);
#define GNNCO_WG_CASE(KK, NN) \
  if (K == KK && N == NN) return launch_wg<KK, NN>(h, A, G, dW, scratch, st)
  GNNCO_WG_CASE(128, 64); GNNCO_WG_CASE(128, 128); GNNCO_WG_CASE(128, 256);
  GNNCO_WG_CASE(256, 64); GNNCO_WG_CASE(256, 128); GNNCO_WG_CASE(256, 256);
#undef GNNCO_WG_CASE
  return GNNCO_UNSUPPORTED;
}

int32_t launch_cast_both_bf16(gnnco_handle* h, const float* W, __nv_bfloat16* Wc, __nv_bfloat16* Wt, int K, int N,
                              int32_t sets, cudaStream_t st) {
  if ((K % 64) || (N % 64) || ((uintptr_t)W & 15) || ((uintptr_t)Wc & 7) || ((uintptr_t)Wt & 7)) {
    int32_t rc = launch_cast_bf16(h, W, Wc, (int64_t)K * N * sets, st);
    return rc != GNNCO_OK ? rc : launch_cast_transpose_bf16(h, W, Wt, K, N, sets, st);
  }
  ProfScope prof_(h, K_CAST, st);
  cast_both_bf16_kernel<<<dim3(sets, K / 64, N / 64), 256, 0, st>>>(W, Wc, Wt, K, N);
  h->launches += 1;
  GNNCO_LAUNCH_CHECK();
  return GNNCO_OK;
}

int32_t launch_cast_transpose_bf16(gnnco_handle* h, const float* W, __nv_bfloat16* Wt, int K, int N, int32_t sets,
                                   cudaStream_t st) {
  ProfScope prof_(h, K_CAST, st);
  dim3 grid(sets, (K + 31) / 32, (N + 31) / 32);
  if (grid.y > 65535 || grid.z > 65535) return GNNCO_UNSUPPORTED;
  cast_transpose_bf16_kernel<<<grid, dim3(32, 8), 0, st>>>(W, Wt, K, N);
  h->launches += 1;
  GNNCO_LAUNCH_CHECK();
  return GNNCO_OK;
}

bool adam_cast_both_supported(const float* W, const float* m, const float* v, const float* g, const __nv_bfloat16* Wc,
                              const __nv_bfloat16* Wt, int K, int N, int32_t sets) {
  return Wc && Wt && (K % 64) == 0 && (N % 64) == 0 && sets >= 1 &&
         !(((uintptr_t)W | (uintptr_t)m | (uintptr_t)v | (uintptr_t)g) & 15) && !(((uintptr_t)Wc | (uintptr_t)Wt) & 7);
}

int32_t launch_adam_cast_both(gnnco_handle* h, float* W, float* m, float* v, const float* g, __nv_bfloat16* Wc,
                              __nv_bfloat16* Wt, int K, int N, int32_t sets, float lr, float b1, float b2, float eps,
                              float c1, float c2, const uint8_t* active, cudaStream_t st) {
  if (!adam_cast_both_supported(W, m, v, g, Wc, Wt, K, N, sets)) return GNNCO_UNSUPPORTED;
  ProfScope prof_(h, K_ADAM, st);
  adam_cast_both_kernel<<<dim3(sets, K / 64, N / 64), 256, 0, st>>>(W, m, v, g, Wc, Wt, K, N, lr, b1, b2, eps, 1.0f / c1,
                                                                     1.0f / c2, active, h->adam_bias);
  h->launches += 1;
  GNNCO_LAUNCH_CHECK();
  return GNNCO_OK;
}
