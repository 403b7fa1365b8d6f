// The dense per-subgraph transform of tc_gemm.cu (Eq. 3's "... W" and its input gradient) by PAIRS of
// CTAs: a cluster of two CTAs owns a double tile of 256 rows of one subgraph.
//
//   Y[rows, :] = act( A[rows, 0:K] * B_s^T ) * row_scale,    B_s = [N x K], K contiguous
//
// Why pairs.  At width 256 the subgraph's weight matrix (128 KB in bf16) and one 128-row operand tile
// (64 KB) fill a CTA's shared memory, so a single CTA can stage only one tile and every k-block's
// load latency is serial with its MMAs.  With tcgen05's cta_group::2 form the two SMs of a pair
// share one B operand: each keeps HALF of the weight matrix (N/2 rows) next to its own 128 rows of
// A, the tensor cores of both SMs read both halves, and the freed 64 KB hold a second tile of A
// slots.  Each SM still streams only its own rows from HBM; B crosses the SM-to-SM link, not L2.
//
// Operands arrive by TMA (cp.async.bulk.tensor, 2-D boxes of 128 rows x 64 bf16 with the
// 128-byte swizzle that the MMA descriptors expect) issued by one thread per CTA; the tensor maps
// cover this GPU's own buffers and no load is multicast.  Roles per CTA (ten warps):
//   warp 9    one lane: waits for a free A slot, announces the bytes on the EVEN CTA's `full` barrier
//             (which counts the boxes of both CTAs) and issues the boxes: one A k-block per slot, plus
//             this CTA's half of the B k-block when the subgraph changes
//   warp 8    even CTA only, one lane: per k-block wait `full`, issue 4 MMAs of 256 x N x 16 for
//             the pair, commit -> `empty` of that slot in BOTH CTAs; after the last k-block commit
//             -> `acc_full` in both CTAs
//   warps 0-7 epilogue of this CTA's 128 rows, as in tc_gemm.cu (TMEM -> registers -> scale / ReLU /
//             mask / round -> staged 128-byte lines -> global; optional row dot product with the
//             next layer's weight vector); then one arrival per warp on the even CTA's `acc_empty`
// Every wait has a time limit; a CTA that gives up raises the handle's status word and still takes
// part in the cluster barriers at the end, so nothing is left waiting.
#include <cuda.h>

#include "internal.cuh"
#include "tc_common.cuh"

namespace {

constexpr int kPairThreads = 320;
constexpr int kPairEpiWarps = 8;
constexpr int kPairMmaWarp = 8;
constexpr int kPairTmaWarp = 9;
constexpr uint32_t kPairMisc = 1536;         // barriers (512 B) + two 128-float dot-product exchange buffers
constexpr uint32_t kPairSmemLimit = 232448;  // 227 KB

template <int KDIM, int NDIM>
struct PairCfg {
  static constexpr int KB = KDIM / 64;
  static constexpr uint32_t A_SLOT = 128 * 128;             // 128 rows x 64 bf16
  static constexpr uint32_t B_SLOT = (NDIM / 2) * 128;      // this CTA's N/2 rows of one k-block
  static constexpr uint32_t B_BYTES = KB * B_SLOT;
  static constexpr uint32_t EPI_BYTES = kPairEpiWarps * 4096;
  static constexpr int kFit = (int)((kPairSmemLimit - 1024 - kPairMisc - EPI_BYTES - B_BYTES) / A_SLOT);
  static constexpr int kTiles = (kFit / KB) < 4 ? (kFit / KB) : 4;      // tiles of A in flight (at most four)
  static constexpr int NSLOT = kTiles * KB;
  static constexpr uint32_t A_BYTES = NSLOT * A_SLOT;
  static constexpr size_t SMEM = 1024 + A_BYTES + B_BYTES + kPairMisc + EPI_BYTES;
  static_assert(kTiles >= 2, "the pair form needs at least two tiles of A slots");
  static_assert(NSLOT <= 16, "barrier area holds 16 slots");
};

// keep the bf16 halves of v where the matching halves of m are positive
__device__ __forceinline__ uint32_t keep_positive_pair(uint32_t v, uint32_t m) {
  const uint32_t lo = __uint_as_float(m << 16) > 0.0f ? 0x0000ffffu : 0u;
  const uint32_t hi = __uint_as_float(m & 0xffff0000u) > 0.0f ? 0xffff0000u : 0u;
  return v & (lo | hi);
}

template <int KDIM, int NDIM, bool MASKED>
__global__ void __launch_bounds__(kPairThreads, 1)
transform_tc_pair(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                  int32_t b_per_part, __nv_bfloat16* __restrict__ Y, int relu, const float* __restrict__ row_scale,
                  const __nv_bfloat16* __restrict__ relu_mask, const __nv_bfloat16* __restrict__ dot_w,
                  int64_t dot_stride, float* __restrict__ dot_out, const int32_t* __restrict__ pair_row0,
                  const int32_t* __restrict__ pair_rows, const int32_t* __restrict__ node_part, int n_pairs,
                  int pairs_per_cluster, int32_t* status) {
  using C = PairCfg<KDIM, NDIM>;
  constexpr int KB = C::KB, NSLOT = C::NSLOT;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t sbase = (tc::smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sA = sbase, sB = sbase + C::A_BYTES;
  uint8_t* gen_base = smem_raw + (sbase - tc::smem_u32(smem_raw));
  uint64_t* full = reinterpret_cast<uint64_t*>(gen_base + C::A_BYTES + C::B_BYTES);   // [16]  (even CTA's copy is used)
  uint64_t* empty = full + 16;                                                        // [16]  both CTAs
  uint64_t* acc_full = empty + 16;                                                    // [2]   both CTAs
  uint64_t* acc_empty = acc_full + 2;                                                 // [2]   even CTA's copy is used
  uint64_t* dot_bar = acc_empty + 2;                                                  // [4 quarters][2 buffers]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(dot_bar + 8);
  volatile uint32_t* abort_flag = tmem_slot + 1;
  float* dot_x = reinterpret_cast<float*>(gen_base + C::A_BYTES + C::B_BYTES + 512);  // [2][128]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = tc::cluster_ctarank();                 // 0 = even CTA (issues the MMAs), 1 = odd CTA
  const int cluster_id = blockIdx.x >> 1;
  const int t_begin = cluster_id * pairs_per_cluster;
  const int t_end = min(n_pairs, t_begin + pairs_per_cluster);
  if (t_begin >= t_end) return;                                // both CTAs of the cluster leave together

  if (threadIdx.x == 0) {
    for (int i = 0; i < NSLOT; ++i) {
      tc::mbar_init(full + i, 2);                              // one announcement per CTA; the boxes count as bytes
      tc::mbar_init(empty + i, 1);
    }
    for (int i = 0; i < 2; ++i) {
      tc::mbar_init(acc_full + i, 1);
      tc::mbar_init(acc_empty + i, 2 * kPairEpiWarps);         // one arrival per epilogue warp of both CTAs
    }
    for (int i = 0; i < 8; ++i) tc::mbar_init(dot_bar + i, 32);
    *abort_flag = 0;
    tc::fence_mbar_init();
  }
  if (warp == 0) tc::tmem_alloc_pair(tmem_slot, 2 * NDIM);
  tc::tc_fence_before_sync();
  __syncthreads();
  tc::cluster_sync_all();                                      // the other CTA's barriers exist before anything arrives there
  tc::tc_fence_after_sync();
  const uint32_t tmem = *tmem_slot;

  if (warp == kPairTmaWarp) {
    // ------------------------------------------------------------------- TMA producer
    if (lane == 0) {
      int cur_part = -1;
      for (int t = t_begin, j = 0; t < t_end && !*abort_flag; ++t, ++j) {
        const int32_t row0 = pair_row0[t];
        const int part = node_part[row0];
        const bool new_b = part != cur_part;
        cur_part = part;
        for (int kb = 0; kb < KB; ++kb) {
          const int g = j * KB + kb, slot = g % NSLOT, use = g / NSLOT;
          if (use > 0 && !tc::mbar_wait_bounded(empty + slot, (use - 1) & 1)) *abort_flag = 1;
          if (new_b && j > 0) {
            // B k-block kb was last read by the previous tile's MMAs of this k-block
            const int gp = g - KB;
            if (!tc::mbar_wait_bounded(empty + gp % NSLOT, (gp / NSLOT) & 1)) *abort_flag = 1;
          }
          if (*abort_flag) break;
          const uint32_t bar = tc::map_to_cta(tc::smem_u32(full + slot), 0);
          tc::mbar_arrive_expect_tx_cluster(bar, C::A_SLOT + (new_b ? C::B_SLOT : 0u));
          tc::tma_load_2d_pair(sA + slot * C::A_SLOT, &map_a, kb * 64, row0 + (int32_t)rank * 128, bar);
          if (new_b)
            tc::tma_load_2d_pair(sB + kb * C::B_SLOT, &map_b, kb * 64, part * b_per_part + (int32_t)rank * (NDIM / 2), bar);
        }
      }
    }
    __syncwarp();
  } else if (warp == kPairMmaWarp) {
    // -------------------------------------------------------------------- MMA issuer (even CTA)
    if (rank == 0) {
      constexpr uint32_t IDESC = tc::idesc_bf16_f32(256, NDIM, false, false);
      for (int t = t_begin, j = 0; t < t_end && !*abort_flag; ++t, ++j) {
        const int buf = j & 1;
        if (j >= 2 && !tc::mbar_wait_bounded(acc_empty + buf, ((j >> 1) - 1) & 1)) *abort_flag = 1;
        for (int kb = 0; kb < KB; ++kb) {
          const int g = j * KB + kb, slot = g % NSLOT, use = g / NSLOT;
          if (!tc::mbar_wait_bounded(full + slot, use & 1)) *abort_flag = 1;
          tc::tc_fence_after_sync();
          if (lane == 0 && !*abort_flag) {
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
              const uint64_t ad = tc::smem_desc_sw128(sA + slot * C::A_SLOT + ks * 32, 16, 1024);
              const uint64_t bd = tc::smem_desc_sw128(sB + kb * C::B_SLOT + ks * 32, 16, 1024);
              tc::mma_bf16_pair(tmem + buf * NDIM, ad, bd, IDESC, (kb | ks) != 0);
            }
            tc::mma_commit_pair(empty + slot, 3);
            if (kb == KB - 1) tc::mma_commit_pair(acc_full + buf, 3);
          }
          __syncwarp();
        }
      }
    }
  } else {
    // ---------------------------------------------------------------------- epilogue (this CTA's 128 rows)
    constexpr int CHUNKS = NDIM / 64;                 // 64-column chunks of the tile
    constexpr int PER = (CHUNKS + 1) / 2;             // chunks per column half
    const int quarter = warp & 3, half = warp >> 2;
    const int ch_begin = half * PER, ch_end = min(CHUNKS, ch_begin + PER);
    const int row = quarter * 32 + lane;
    const uint32_t stage = sbase + C::A_BYTES + C::B_BYTES + kPairMisc + warp * 4096;
    const uint32_t acc_empty_even = tc::map_to_cta(tc::smem_u32(acc_empty), 0);
    for (int t = t_begin, j = 0; t < t_end && !*abort_flag; ++t, ++j) {
      const int buf = j & 1;
      const int64_t row0 = (int64_t)pair_row0[t] + rank * 128;
      const int rows = max(0, min(128, pair_rows[t] - (int)rank * 128));
      const bool valid = row < rows;
      const int rows_here = rows - quarter * 32;       // valid rows of this warp's 32
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
      if (dot_out) wv = dot_w + (int64_t)node_part[pair_row0[t]] * dot_stride;
      float dot = 0.0f;
      if (!tc::mbar_wait_bounded(acc_full + buf, (j >> 1) & 1)) { *abort_flag = 1; break; }
      tc::tc_fence_after_sync();
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
            v.x = keep_positive_pair(v.x, mk[c][it].x); v.y = keep_positive_pair(v.y, mk[c][it].y);
            v.z = keep_positive_pair(v.z, mk[c][it].z); v.w = keep_positive_pair(v.w, mk[c][it].w);
          }
          if (rr < rows_here)
            *reinterpret_cast<uint4*>(Y + (row0 + quarter * 32 + rr) * NDIM + c0 + pc * 8) = v;
        }
      }
      if (dot_out) {
        // lower column half + upper column half, in that order (see tc_gemm.cu)
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
      __syncwarp();
      if (lane == 0) tc::mbar_arrive_cluster(acc_empty_even + buf * 8);
    }
  }
  if (*abort_flag && threadIdx.x == 0) atomicMin(status, (int32_t)GNNCO_INTERNAL);
  tc::tc_fence_before_sync();
  __syncthreads();
  tc::cluster_sync_all();            // the pair's MMAs have read this CTA's operands, its arrivals have landed
  if (warp == 0) tc::tmem_dealloc_pair(tmem, 2 * NDIM);
}

// ---- tensor maps (the driver's encoder is looked up through the runtime; nothing links against libcuda)
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled() {
  static EncodeTiledFn fn = nullptr;
  static bool asked = false;
  if (!asked) {
    asked = true;
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// [rows x KDIM] bf16 row-major, boxes of box_rows x 64 elements, 128-byte swizzle
bool make_map(CUtensorMap* m, const void* base, uint64_t rows, int kdim, int box_rows) {
  EncodeTiledFn enc = encode_tiled();
  if (!enc) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)kdim, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)kdim * 2};
  const cuuint32_t box[2] = {64u, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1u, 1u};
  return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int KDIM, int NDIM, bool MASKED>
int32_t launch_pair_kernel(gnnco_handle* h, const CUtensorMap& ma, const CUtensorMap& mb, int32_t b_per_part, void* Y,
                           bool relu, const float* row_scale, const void* relu_mask, const void* dot_w,
                           int64_t dot_stride, float* dot_out, int clusters, int per, cudaStream_t st) {
  using C = PairCfg<KDIM, NDIM>;
  auto kernel = transform_tc_pair<KDIM, NDIM, MASKED>;
  GNNCO_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)C::SMEM));
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(2 * clusters);
  cfg.blockDim = dim3(kPairThreads);
  cfg.dynamicSmemBytes = C::SMEM;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  GNNCO_CUDA_TRY(cudaLaunchKernelEx(&cfg, kernel, ma, mb, b_per_part, (__nv_bfloat16*)Y, relu ? 1 : 0, row_scale,
                                    (const __nv_bfloat16*)relu_mask, (const __nv_bfloat16*)dot_w, dot_stride, dot_out,
                                    (const int32_t*)h->pair_row0, (const int32_t*)h->pair_rows,
                                    (const int32_t*)h->node_part, (int)h->n_pairs, per, h->status));
  h->launches += 1;
  return GNNCO_OK;
}

// how many CTA pairs of the widest configuration can be resident at once (0: clusters of two cannot be launched)
template <int KDIM, int NDIM>
int resident_pairs() {
  using C = PairCfg<KDIM, NDIM>;
  auto kernel = transform_tc_pair<KDIM, NDIM, false>;
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)C::SMEM) != cudaSuccess) {
    cudaGetLastError();
    return 0;
  }
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(2 * 148);
  cfg.blockDim = dim3(kPairThreads);
  cfg.dynamicSmemBytes = C::SMEM;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, kernel, &cfg) != cudaSuccess) {
    cudaGetLastError();
    return 0;
  }
  return n;
}

template <int KDIM, int NDIM>
int32_t launch_pair(gnnco_handle* h, const void* A, const void* B, int64_t b_stride, int32_t b_sets, void* Y, bool relu,
                    const float* row_scale, const void* relu_mask, const void* dot_w, int64_t dot_stride,
                    float* dot_out, cudaStream_t st) {
  CUtensorMap ma, mb;
  // rows past the end of A read as zeros; B holds b_sets matrices of NDIM rows
  if (!make_map(&ma, A, (uint64_t)h->n, KDIM, 128)) return GNNCO_CUDA_ERROR;
  if (!make_map(&mb, B, (uint64_t)b_sets * NDIM, KDIM, NDIM / 2)) return GNNCO_CUDA_ERROR;
  int clusters = h->pair_clusters < h->n_pairs ? h->pair_clusters : h->n_pairs;
  const int per = (h->n_pairs + clusters - 1) / clusters;
  clusters = (h->n_pairs + per - 1) / per;
  const int32_t b_per_part = b_stride == 0 ? 0 : NDIM;
  if (relu_mask)
    return launch_pair_kernel<KDIM, NDIM, true>(h, ma, mb, b_per_part, Y, relu, row_scale, relu_mask, dot_w, dot_stride,
                                                dot_out, clusters, per, st);
  return launch_pair_kernel<KDIM, NDIM, false>(h, ma, mb, b_per_part, Y, relu, row_scale, relu_mask, dot_w, dot_stride,
                                               dot_out, clusters, per, st);
}

}  // namespace

// The pair form is used for the widths where a single CTA cannot hold a second operand tile.
bool tc_pair_transform_supported(gnnco_handle* h, int dtype, int K, int N) {
  if (dtype != GNNCO_BF16 || !(K == 256 && N == 256)) return false;
  if (h->n_pairs <= 0 || !encode_tiled()) return false;
  if (h->pair_clusters < 0) h->pair_clusters = resident_pairs<256, 256>();
  return h->pair_clusters > 0;
}

int32_t launch_transform_tc_pair(gnnco_handle* h, const void* A, const void* B, int64_t b_stride, int32_t b_sets, void* Y,
                                 int K, int N, bool relu, const float* row_scale, const void* relu_mask, bool backward,
                                 const void* dot_w, int64_t dot_stride, float* dot_out, cudaStream_t st) {
  if (!tc_pair_transform_supported(h, GNNCO_BF16, K, N)) return GNNCO_UNSUPPORTED;
  if (((uintptr_t)A & 15) || ((uintptr_t)B & 15) || (b_stride != 0 && b_stride != (int64_t)K * N)) return GNNCO_UNSUPPORTED;
  ProfScope prof_(h, backward ? K_TRANSFORM_BWD : K_TRANSFORM_FWD, st);
  return launch_pair<256, 256>(h, A, B, b_stride, b_sets, Y, relu, row_scale, relu_mask, dot_w, dot_stride, dot_out, st);
}
