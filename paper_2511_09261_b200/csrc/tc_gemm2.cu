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
// 128-byte swizzle that the MMA descriptors expect) issued by one thread per CTA; results leave by
// TMA too (boxes of 32 rows x 32 columns from a per-warp staging tile).  The tensor maps cover this
// GPU's own buffers and no load is multicast.  Roles per CTA (eighteen warps):
//   warp 17   one lane: waits for a free A slot, announces the bytes on the EVEN CTA's `full` barrier
//             (which counts the boxes of both CTAs) and issues the boxes: one A k-block per slot, plus
//             this CTA's half of the B k-block when the subgraph changes
//   warp 16   even CTA only, one lane: per k-block wait `full`, issue 4 MMAs of 256 x N x 16 for
//             the pair, commit -> `empty` of that slot in BOTH CTAs; after the last k-block commit
//             -> `acc_full` in both CTAs
//   warps 0-15 epilogue of this CTA's 128 rows: warp w owns TMEM lanes 32 (w % 4) .. +32 (one row per
//             lane) and columns 64 (w / 4) .. +64.  It copies its part of the accumulator to registers and
//             gives the accumulator buffer back AT ONCE (one arrival per warp on the even CTA's
//             `acc_empty`), so the next tile's MMAs never wait for conversions or stores; then, 32
//             columns at a time: scale / ReLU (inside the conversion to bf16) / mask (one bit per element of
//             the saved activation; a rectifying launch can leave those bits behind), optional dot
//             product with the next layer's weight vector, staging, one TMA store.  The last, ragged
//             tile of a subgraph is stored with plain stores (a TMA box would spill into the next subgraph).
// The drain used to be the bottleneck: with eight warps doing all of this the on-chip part alone took as
// long per tile as the tile's memory traffic, and the two did not overlap.
// Every wait has a time limit; a CTA that gives up raises the handle's status word and still takes
// part in the cluster barriers at the end, so nothing is left waiting.
#include <cuda.h>

#include "internal.cuh"
#include "tc_common.cuh"

namespace {

constexpr int kPairEpiWarps = 16;
constexpr int kPairMmaWarp = 16;
constexpr int kPairTmaWarp = 17;
constexpr int kPairThreads = 32 * 18;
constexpr uint32_t kPairStage = 2048;        // per epilogue warp: 32 rows x 32 bf16
constexpr uint32_t kPairMisc = 3584;         // barriers (512 B) + dot-product exchange [2 buffers][3 column groups][128 rows]
constexpr uint32_t kPairSmemLimit = 232448;  // 227 KB

// epilogue modes
constexpr int kModePlain = 0;                // Y = A B^T
constexpr int kModeRelu = 1;                 // Y = max(A B^T, 0), optional row dot product
constexpr int kModeScaledMasked = 2;         // Y = row_scale * (A B^T) where mask > 0, else 0

template <int KDIM, int NDIM>
struct PairCfg {
  static constexpr int KB = KDIM / 64;
  static constexpr uint32_t A_SLOT = 128 * 128;             // 128 rows x 64 bf16
  static constexpr uint32_t B_SLOT = (NDIM / 2) * 128;      // this CTA's N/2 rows of one k-block
  static constexpr uint32_t B_BYTES = KB * B_SLOT;
  static constexpr uint32_t EPI_BYTES = kPairEpiWarps * kPairStage;
  static constexpr int kFit = (int)((kPairSmemLimit - 1024 - kPairMisc - EPI_BYTES - B_BYTES) / A_SLOT);
  static constexpr int NSLOT = kFit < 4 * KB ? kFit : 4 * KB;           // k-block slots of A in flight (at most four tiles)
  static constexpr uint32_t A_BYTES = NSLOT * A_SLOT;
  static constexpr size_t SMEM = 1024 + A_BYTES + B_BYTES + EPI_BYTES + kPairMisc;
  static_assert(NDIM == 64 * (kPairEpiWarps / 4), "sixteen epilogue warps cover four column groups of 64");
  static_assert(NSLOT > KB, "the ring must hold more than one tile of A slots");
  static_assert(NSLOT <= 16, "barrier area holds 16 slots");
  static_assert(SMEM <= kPairSmemLimit, "does not fit in shared memory");
};

// two float32 -> packed bf16 pair (first argument in the low half), optionally rectified by the conversion itself
template <bool RELU>
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  uint32_t d;
  if (RELU) asm("cvt.rn.relu.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  else asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}

__device__ __forceinline__ void tma_store_2d(const void* tmap, uint32_t smem_src, int32_t x, int32_t y) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
               ::"l"(tmap), "r"(x), "r"(y), "r"(smem_src) : "memory");
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
// the bulk stores committed so far have read their shared-memory source
__device__ __forceinline__ void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
// ... and have been written
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

template <int KDIM, int NDIM, int MODE>
__global__ void __launch_bounds__(kPairThreads, 1)
transform_tc_pair(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                  const __grid_constant__ CUtensorMap map_y, int32_t b_per_part, __nv_bfloat16* __restrict__ Y,
                  const float* __restrict__ row_scale, const uint8_t* __restrict__ mask_bits,
                  uint8_t* __restrict__ bits_out, const __nv_bfloat16* __restrict__ dot_w, int64_t dot_stride, float* __restrict__ dot_out,
                  const int32_t* __restrict__ pair_row0, const int32_t* __restrict__ pair_rows,
                  const int32_t* __restrict__ node_part, int n_pairs, int pairs_per_cluster, int32_t* status) {
  using C = PairCfg<KDIM, NDIM>;
  constexpr int KB = C::KB, NSLOT = C::NSLOT;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t sbase = (tc::smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sA = sbase, sB = sbase + C::A_BYTES, sStage = sB + C::B_BYTES;
  uint8_t* gen_base = smem_raw + (sbase - tc::smem_u32(smem_raw));
  uint8_t* misc = gen_base + C::A_BYTES + C::B_BYTES + C::EPI_BYTES;
  uint64_t* full = reinterpret_cast<uint64_t*>(misc);          // [16]  (even CTA's copy is used)
  uint64_t* empty = full + 16;                                 // [16]  both CTAs
  uint64_t* acc_full = empty + 16;                             // [2]   both CTAs
  uint64_t* acc_empty = acc_full + 2;                          // [2]   even CTA's copy is used
  uint64_t* dot_bar = acc_empty + 2;                           // [4 quarters][2 buffers]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(dot_bar + 8);
  volatile uint32_t* abort_flag = tmem_slot + 1;
  float* dot_x = reinterpret_cast<float*>(misc + 512);         // [2 buffers][3 column groups][128 rows]

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
    for (int i = 0; i < 8; ++i) tc::mbar_init(dot_bar + i, 96);  // the three upper column groups of a lane quarter
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
    const int quarter = warp & 3, cg = warp >> 2;     // TMEM lane quarter, column group of 64
    const int row = quarter * 32 + lane;
    const int c0 = cg * 64;
    const uint32_t stage = sStage + warp * kPairStage;
    const uint32_t acc_empty_even = tc::map_to_cta(tc::smem_u32(acc_empty), 0);
    for (int t = t_begin, j = 0; t < t_end && !*abort_flag; ++t, ++j) {
      const int buf = j & 1;
      const int64_t row0 = (int64_t)pair_row0[t] + rank * 128;
      const int rows = max(0, min(128, pair_rows[t] - (int)rank * 128));
      const bool valid = row < rows;
      const int rows_here = rows - quarter * 32;       // valid rows of this warp's 32
      float s = 1.0f;
      uint2 mk = make_uint2(0u, 0u);
      if (MODE == kModeScaledMasked && valid) {
        // this row's scale and the 64 mask bits under this warp's columns, requested before the wait
        s = row_scale[row0 + row];
        mk = __ldg(reinterpret_cast<const uint2*>(mask_bits + (row0 + row) * (NDIM / 8) + c0 / 8));
      }
      const __nv_bfloat16* wv = nullptr;
      if (MODE == kModeRelu && dot_out) wv = dot_w + (int64_t)node_part[pair_row0[t]] * dot_stride + c0;
      float dot = 0.0f;
      uint32_t sign_words[2] = {0u, 0u};
      if (!tc::mbar_wait_bounded(acc_full + buf, (j >> 1) & 1)) { *abort_flag = 1; break; }
      tc::tc_fence_after_sync();
      uint32_t ra[32], rb[32];
      {
        const uint32_t at = tmem + ((uint32_t)(quarter * 32) << 16) + buf * NDIM + c0;
        tc::tmem_ld_32x32(at, ra);
        tc::tmem_ld_32x32(at + 32, rb);
        tc::tmem_ld_wait();
      }
      // the accumulator is in registers: hand the buffer back before converting and storing (the warps
      // that collect the row dot products do it after they have read the exchange slots of this buffer,
      // so that nobody can be two tiles ahead and overwrite them)
      const bool late_release = MODE == kModeRelu && dot_out && cg == 0;
      tc::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0 && !late_release) tc::mbar_arrive_cluster(acc_empty_even + buf * 8);
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        uint32_t o[16];                                // 32 bf16 of this thread's row, packed
#pragma unroll
        for (int q = 0; q < 16; ++q) {
          float a = __uint_as_float(hh ? rb[2 * q] : ra[2 * q]), b = __uint_as_float(hh ? rb[2 * q + 1] : ra[2 * q + 1]);
          if (MODE == kModeScaledMasked) {
            const uint32_t mw = hh ? mk.y : mk.x;          // bit k: column c0 + 32 hh + k of the saved activation was positive
            a = (mw >> (2 * q)) & 1u ? a * s : 0.0f;
            b = (mw >> (2 * q + 1)) & 1u ? b * s : 0.0f;
          }
          o[q] = pack_bf16<MODE == kModeRelu>(a, b);
        }
        if (MODE == kModeRelu && bits_out) {
          // [stored value > 0], one bit per element, for the backward pass (element f of a row = bit f % 8 of
          // byte f / 8): the 32 columns of this round are one word of the row
          uint32_t word = 0;
#pragma unroll
          for (int q = 0; q < 16; ++q) {
            word |= (o[q] & 0x0000ffffu) ? (1u << (2 * q)) : 0u;
            word |= (o[q] & 0xffff0000u) ? (2u << (2 * q)) : 0u;
          }
          sign_words[hh] = word;
          if (hh == 1 && valid)
            *reinterpret_cast<uint2*>(bits_out + (row0 + row) * (NDIM / 8) + c0 / 8) = make_uint2(sign_words[0], word);
        }
        if (wv) {   // dot product of the STORED (rounded) row with the next layer's weight vector
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) {
            const uint4 w8 = __ldg(reinterpret_cast<const uint4*>(wv + hh * 32) + q4);
            const uint32_t wq[4] = {w8.x, w8.y, w8.z, w8.w};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const uint32_t hv = o[q4 * 4 + q];
              dot = fmaf(__uint_as_float(hv << 16), __uint_as_float(wq[q] << 16), dot);
              dot = fmaf(__uint_as_float(hv & 0xffff0000u), __uint_as_float(wq[q] & 0xffff0000u), dot);
            }
          }
        }
        if (rows_here >= 32) {
          // staging tile: 32 rows of 64 bytes, dense; the previous store of this warp must have read it
          if (lane == 0) tma_store_wait_read();
          __syncwarp();
#pragma unroll
          for (int pc = 0; pc < 4; ++pc)
            tc::st_shared16(stage + lane * 64 + pc * 16, o[4 * pc], o[4 * pc + 1], o[4 * pc + 2], o[4 * pc + 3]);
          tc::fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) tma_store_2d(&map_y, stage, c0 + hh * 32, (int32_t)(row0 + quarter * 32));
        } else if (valid) {
          // ragged end of a subgraph: a box would reach into the next subgraph's rows
          uint4* dst = reinterpret_cast<uint4*>(Y + (row0 + row) * NDIM + c0 + hh * 32);
#pragma unroll
          for (int pc = 0; pc < 4; ++pc) dst[pc] = make_uint4(o[4 * pc], o[4 * pc + 1], o[4 * pc + 2], o[4 * pc + 3]);
        }
      }
      if (MODE == kModeRelu && dot_out) {
        // column groups are added in the order 0, 1, 2, 3
        if (cg > 0) {
          dot_x[(buf * 3 + cg - 1) * 128 + row] = dot;
          tc::mbar_arrive(dot_bar + quarter * 2 + buf);
        } else {
          if (!tc::mbar_wait_bounded(dot_bar + quarter * 2 + buf, (j >> 1) & 1)) { *abort_flag = 1; break; }
          dot += dot_x[(buf * 3 + 0) * 128 + row];
          dot += dot_x[(buf * 3 + 1) * 128 + row];
          dot += dot_x[(buf * 3 + 2) * 128 + row];
          if (valid) dot_out[row0 + row] = dot;
          __syncwarp();
          if (lane == 0) tc::mbar_arrive_cluster(acc_empty_even + buf * 8);
        }
      }
    }
    if (lane == 0) tma_store_wait_all();
    __syncwarp();
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

// [rows x width] bf16 row-major, boxes of box_rows x box_cols elements; operand boxes (64 columns) use the
// 128-byte swizzle of the MMA descriptors, result boxes are dense
bool make_map(CUtensorMap* m, const void* base, uint64_t rows, int width, int box_rows, int box_cols, bool swizzle) {
  EncodeTiledFn enc = encode_tiled();
  if (!enc) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)width, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)width * 2};
  const cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1u, 1u};
  return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
             CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int KDIM, int NDIM, int MODE>
int32_t launch_pair_kernel(gnnco_handle* h, const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& my,
                           int32_t b_per_part, void* Y, const float* row_scale, const uint8_t* mask_bits,
                           uint8_t* bits_out, const void* dot_w, int64_t dot_stride, float* dot_out, int clusters,
                           int per, cudaStream_t st) {
  using C = PairCfg<KDIM, NDIM>;
  auto kernel = transform_tc_pair<KDIM, NDIM, MODE>;
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
  GNNCO_CUDA_TRY(cudaLaunchKernelEx(&cfg, kernel, ma, mb, my, b_per_part, (__nv_bfloat16*)Y, row_scale, mask_bits,
                                    bits_out, (const __nv_bfloat16*)dot_w, dot_stride, dot_out,
                                    (const int32_t*)h->pair_row0, (const int32_t*)h->pair_rows,
                                    (const int32_t*)h->node_part, (int)h->n_pairs, per, h->status));
  h->launches += 1;
  return GNNCO_OK;
}

// how many CTA pairs of the widest configuration can be resident at once (0: clusters of two cannot be launched)
template <int KDIM, int NDIM>
int resident_pairs() {
  using C = PairCfg<KDIM, NDIM>;
  auto kernel = transform_tc_pair<KDIM, NDIM, kModePlain>;
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
                    const float* row_scale, const uint8_t* mask_bits, uint8_t* bits_out, const void* dot_w,
                    int64_t dot_stride, float* dot_out, cudaStream_t st) {
  int mode;
  if (relu && !row_scale && !mask_bits) mode = kModeRelu;
  else if (!relu && row_scale && mask_bits && !dot_out && !bits_out) mode = kModeScaledMasked;
  else if (!relu && !row_scale && !mask_bits && !dot_out && !bits_out) mode = kModePlain;
  else return GNNCO_UNSUPPORTED;
  CUtensorMap ma, mb, my;
  // rows past the end of A read as zeros; B holds b_sets matrices of NDIM rows; result boxes of 32 x 32
  if (!make_map(&ma, A, (uint64_t)h->n, KDIM, 128, 64, true)) return GNNCO_CUDA_ERROR;
  if (!make_map(&mb, B, (uint64_t)b_sets * NDIM, KDIM, NDIM / 2, 64, true)) return GNNCO_CUDA_ERROR;
  if (!make_map(&my, Y, (uint64_t)h->n, NDIM, 32, 32, false)) return GNNCO_CUDA_ERROR;
  int clusters = h->pair_clusters < h->n_pairs ? h->pair_clusters : h->n_pairs;
  const int per = (h->n_pairs + clusters - 1) / clusters;
  clusters = (h->n_pairs + per - 1) / per;
  const int32_t b_per_part = b_stride == 0 ? 0 : NDIM;
  if (mode == kModeRelu)
    return launch_pair_kernel<KDIM, NDIM, kModeRelu>(h, ma, mb, my, b_per_part, Y, row_scale, mask_bits, bits_out, dot_w,
                                                     dot_stride, dot_out, clusters, per, st);
  if (mode == kModeScaledMasked)
    return launch_pair_kernel<KDIM, NDIM, kModeScaledMasked>(h, ma, mb, my, b_per_part, Y, row_scale, mask_bits, bits_out,
                                                             dot_w, dot_stride, dot_out, clusters, per, st);
  return launch_pair_kernel<KDIM, NDIM, kModePlain>(h, ma, mb, my, b_per_part, Y, row_scale, mask_bits, bits_out, dot_w,
                                                    dot_stride, dot_out, clusters, per, st);
}

// ------------------------------------------------------------------------------------
// Weight gradient by pairs of CTAs:  dW_s[256 x 256] = sum_{i in s} A[i, :]^T G[i, :]  (A = layer input, G = Q_l).
//
// The single-CTA kernel (tc_gemm.cu) needs all 512 TMEM columns for one 256 x 256 float32 accumulator, so a
// subgraph's 256 KB result cannot leave while the next subgraph is being summed, and every subgraph pays an
// unhidden pipeline fill and drain (about a tenth of its time at 2,400 rows).  With cta_group::2 the pair owns
// one subgraph (or row chunk): each CTA stages, per 64 rows, only ITS 128 features of A (the M half) and ITS 128
// features of G (the N half), the pair's MMAs (256 x 256 x 16, both operands MN-major) leave 128 x 256 of the result
// in each CTA's TMEM -- 256 columns, so there are TWO accumulator buffers and a subgraph is written out while the
// next one is summed.  Persistent over the chunk table; six stages of 32 KB per CTA, filled by TMA across chunk
// boundaries.  A chunk's last, ragged stage lands on a private barrier; the producer warp zeroes the rows past the
// chunk's end (they belong to the next subgraph) before it announces the stage.
// Roles per CTA: warp 0 producer, warp 1 MMA issuer (even CTA), warps 2-9 write the result (TMEM lane quarter =
// warp % 4, column half by which of the two warps of that quarter).
constexpr int kWgpThreads = 320;
constexpr int kWgpStages = 6;
constexpr int kWgpRows = 64;                     // reduction rows per stage
constexpr uint32_t kWgpHalf = 128 * 128;         // one operand's share of a stage: 64 rows x 128 features x 2 B
constexpr uint32_t kWgpStage = 2 * kWgpHalf;     // A share + G share
constexpr size_t kWgpSmem = 1024 + kWgpStages * kWgpStage + 256;

__global__ void __launch_bounds__(kWgpThreads, 1)
weight_grad_tc_pair(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_g,
                    float* __restrict__ dW, float* __restrict__ scratch, const int32_t* __restrict__ wg_begin,
                    const int32_t* __restrict__ wg_end, const int32_t* __restrict__ wg_slot, int n_chunks,
                    int32_t* status) {
  constexpr int KF = 256, NF = 256;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t sbase = (tc::smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* gen_base = smem_raw + (sbase - tc::smem_u32(smem_raw));
  uint64_t* full = reinterpret_cast<uint64_t*>(gen_base + kWgpStages * kWgpStage);   // [6]  even CTA's copy is used
  uint64_t* empty = full + kWgpStages;                                                // [6]  both CTAs
  uint64_t* acc_full = empty + kWgpStages;                                            // [2]  both CTAs
  uint64_t* acc_empty = acc_full + 2;                                                 // [2]  even CTA's copy is used
  uint64_t* tail_bar = acc_empty + 2;                                                 // [1]  this CTA's ragged stages
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tail_bar + 1);
  volatile uint32_t* abort_flag = tmem_slot + 1;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = tc::cluster_ctarank();
  const int cluster_id = blockIdx.x >> 1, n_clusters = gridDim.x >> 1;
  if (cluster_id >= n_chunks) return;                            // both CTAs of the cluster leave together

  if (threadIdx.x == 0) {
    for (int i = 0; i < kWgpStages; ++i) {
      tc::mbar_init(full + i, 2);                                // one announcement per CTA
      tc::mbar_init(empty + i, 1);
    }
    for (int i = 0; i < 2; ++i) {
      tc::mbar_init(acc_full + i, 1);
      tc::mbar_init(acc_empty + i, 2 * 8);                       // one arrival per result warp of both CTAs
    }
    tc::mbar_init(tail_bar, 1);
    *abort_flag = 0;
    tc::fence_mbar_init();
  }
  if (warp == 0) tc::tmem_alloc_pair(tmem_slot, 512);
  tc::tc_fence_before_sync();
  __syncthreads();
  tc::cluster_sync_all();
  tc::tc_fence_after_sync();
  const uint32_t tmem = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------- producer
    int g = 0;                                                   // stages issued so far (ring position)
    int tails = 0;                                               // ragged stages so far (phase of tail_bar)
    for (int c = cluster_id; c < n_chunks && !*abort_flag; c += n_clusters) {
      const int32_t ra = wg_begin[c], rb = wg_end[c];
      for (int32_t r0 = ra; r0 < rb && !*abort_flag; r0 += kWgpRows, ++g) {
        const int slot = g % kWgpStages, use = g / kWgpStages;
        const uint32_t sa = sbase + slot * kWgpStage, sg = sa + kWgpHalf;
        const int valid = min(kWgpRows, rb - r0);
        const uint32_t bar = tc::map_to_cta(tc::smem_u32(full + slot), 0);
        if (use > 0 && !tc::mbar_wait_bounded(empty + slot, (use - 1) & 1)) *abort_flag = 1;
        if (*abort_flag) break;
        if (valid == kWgpRows) {
          if (lane == 0) {
            tc::mbar_arrive_expect_tx_cluster(bar, kWgpStage);
            tc::tma_load_2d_pair(sa, &map_a, (int32_t)rank * 128, r0, bar);
            tc::tma_load_2d_pair(sa + 8192, &map_a, (int32_t)rank * 128 + 64, r0, bar);
            tc::tma_load_2d_pair(sg, &map_g, (int32_t)rank * 128, r0, bar);
            tc::tma_load_2d_pair(sg + 8192, &map_g, (int32_t)rank * 128 + 64, r0, bar);
          }
        } else {
          // ragged end of the chunk: land on this CTA's own barrier, zero the rows past the end, then announce
          const uint32_t tb = tc::smem_u32(tail_bar);
          if (lane == 0) {
            tc::mbar_arrive_expect_tx_cluster(tb, kWgpStage);
            tc::tma_load_2d_pair(sa, &map_a, (int32_t)rank * 128, r0, tb);
            tc::tma_load_2d_pair(sa + 8192, &map_a, (int32_t)rank * 128 + 64, r0, tb);
            tc::tma_load_2d_pair(sg, &map_g, (int32_t)rank * 128, r0, tb);
            tc::tma_load_2d_pair(sg + 8192, &map_g, (int32_t)rank * 128 + 64, r0, tb);
          }
          if (!tc::mbar_wait_bounded(tail_bar, tails & 1)) *abort_flag = 1;
          ++tails;
          // row k of a 64-feature block is 128 bytes at (k/8)*1024 + (k%8)*128 whatever the swizzle does inside it
          for (int q = lane; q < (kWgpRows - valid) * 4 * 8; q += 32) {
            const int k = valid + q / 32, blk = (q / 8) & 3, piece = q & 7;
            tc::st_shared_zero16(sa + blk * 8192 + (k >> 3) * 1024 + (k & 7) * 128 + piece * 16);
          }
          tc::fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) tc::mbar_arrive_expect_tx_cluster(bar, 0);
        }
        __syncwarp();
      }
    }
  } else if (warp == 1) {
    // -------------------------------------------------------------------- MMA issuer (even CTA)
    if (rank == 0) {
      constexpr uint32_t IDESC = tc::idesc_bf16_f32(256, NF, true, true);
      int g = 0, j = 0;
      for (int c = cluster_id; c < n_chunks && !*abort_flag; c += n_clusters, ++j) {
        const int32_t ra = wg_begin[c], rb = wg_end[c];
        const int iters = (rb - ra + kWgpRows - 1) / kWgpRows;
        const int buf = j & 1;
        if (j >= 2 && !tc::mbar_wait_bounded(acc_empty + buf, ((j >> 1) - 1) & 1)) *abort_flag = 1;
        for (int it = 0; it < iters; ++it, ++g) {
          const int slot = g % kWgpStages, use = g / kWgpStages;
          if (!tc::mbar_wait_bounded(full + slot, use & 1)) *abort_flag = 1;
          tc::tc_fence_after_sync();
          if (lane == 0 && !*abort_flag) {
            const uint32_t sa = sbase + slot * kWgpStage, sg = sa + kWgpHalf;
#pragma unroll
            for (int q = 0; q < kWgpRows / 16; ++q) {
              const uint64_t ad = tc::smem_desc_sw128(sa + q * 2048, kWgpRows * 128, 1024);
              const uint64_t gd = tc::smem_desc_sw128(sg + q * 2048, kWgpRows * 128, 1024);
              tc::mma_bf16_pair(tmem + buf * NF, ad, gd, IDESC, (it | q) != 0);
            }
            tc::mma_commit_pair(empty + slot, 3);
          }
          __syncwarp();
        }
        if (lane == 0 && !*abort_flag) tc::mma_commit_pair(acc_full + buf, 3);
        __syncwarp();
      }
    }
  } else {
    // ---------------------------------------------------------------------- result writers
    const int quarter = warp & 3, half = (warp - 2) >> 2;        // warps 2..5 -> half 0, 6..9 -> half 1
    const uint32_t acc_empty_even = tc::map_to_cta(tc::smem_u32(acc_empty), 0);
    const int f = (int)rank * 128 + quarter * 32 + lane;          // this thread's row of dW
    int j = 0;
    for (int c = cluster_id; c < n_chunks && !*abort_flag; c += n_clusters, ++j) {
      const int buf = j & 1;
      const int32_t rows = wg_end[c] - wg_begin[c];
      const int32_t slot = wg_slot[c];
      float* out = slot < 0 ? dW + (int64_t)(-(slot + 1)) * KF * NF : scratch + (int64_t)slot * KF * NF;
      if (!tc::mbar_wait_bounded(acc_full + buf, (j >> 1) & 1)) { *abort_flag = 1; break; }
      tc::tc_fence_after_sync();
#pragma unroll
      for (int c0 = 0; c0 < NF / 2; c0 += 32) {
        uint32_t r[32];
        if (rows > 0) {
          tc::tmem_ld_32x32(tmem + ((uint32_t)(quarter * 32) << 16) + buf * NF + half * (NF / 2) + c0, r);
          tc::tmem_ld_wait();
        } else {
#pragma unroll
          for (int q = 0; q < 32; ++q) r[q] = 0u;                 // a chunk without rows: no MMA ran
        }
        uint4* dst = reinterpret_cast<uint4*>(out + (int64_t)f * NF + half * (NF / 2) + c0);
#pragma unroll
        for (int q = 0; q < 8; ++q) dst[q] = make_uint4(r[4 * q], r[4 * q + 1], r[4 * q + 2], r[4 * q + 3]);
      }
      tc::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) tc::mbar_arrive_cluster(acc_empty_even + buf * 8);
    }
  }
  if (*abort_flag && threadIdx.x == 0) atomicMin(status, (int32_t)GNNCO_INTERNAL);
  tc::tc_fence_before_sync();
  __syncthreads();
  tc::cluster_sync_all();
  if (warp == 0) tc::tmem_dealloc_pair(tmem, 512);
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
                                 int K, int N, bool relu, const float* row_scale, const uint8_t* mask_bits,
                                 uint8_t* bits_out, bool backward, const void* dot_w, int64_t dot_stride, float* dot_out,
                                 cudaStream_t st) {
  if (!tc_pair_transform_supported(h, GNNCO_BF16, K, N)) return GNNCO_UNSUPPORTED;
  if (((uintptr_t)A & 15) || ((uintptr_t)B & 15) || ((uintptr_t)Y & 15) || (b_stride != 0 && b_stride != (int64_t)K * N))
    return GNNCO_UNSUPPORTED;
  ProfScope prof_(h, backward ? K_TRANSFORM_BWD : K_TRANSFORM_FWD, st);
  if (((uintptr_t)mask_bits & 7) || ((uintptr_t)bits_out & 7)) return GNNCO_UNSUPPORTED;
  return launch_pair<256, 256>(h, A, B, b_stride, b_sets, Y, relu, row_scale, mask_bits, bits_out, dot_w, dot_stride, dot_out,
                               st);
}

bool tc_pair_weight_grad_supported(gnnco_handle* h, int dtype, int K, int N) {
  return K == 256 && N == 256 && tc_pair_transform_supported(h, dtype, 256, 256) && h->n_wg_chunks > 0;
}

// dW[s] (256 x 256, float32) = sum_{i in s} A[i,:]^T G[i,:], A, G [n x 256] bf16; chunks of split subgraphs land in
// `scratch` and are combined afterwards, as in the single-CTA kernel
int32_t launch_weight_grad_tc_pair(gnnco_handle* h, const void* A, const void* G, float* dW, float* scratch, int K, int N,
                                   cudaStream_t st) {
  if (!tc_pair_weight_grad_supported(h, GNNCO_BF16, K, N)) return GNNCO_UNSUPPORTED;
  if (((uintptr_t)A & 15) || ((uintptr_t)G & 15) || ((uintptr_t)dW & 15) || ((uintptr_t)scratch & 15)) return GNNCO_UNSUPPORTED;
  ProfScope prof_(h, K_WEIGHT_GRAD, st);
  CUtensorMap ma, mg;
  if (!make_map(&ma, A, (uint64_t)h->n, 256, kWgpRows, 64, true)) return GNNCO_CUDA_ERROR;
  if (!make_map(&mg, G, (uint64_t)h->n, 256, kWgpRows, 64, true)) return GNNCO_CUDA_ERROR;
  GNNCO_CUDA_TRY(cudaFuncSetAttribute(weight_grad_tc_pair, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kWgpSmem));
  const int clusters = h->pair_clusters < h->n_wg_chunks ? h->pair_clusters : h->n_wg_chunks;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(2 * clusters);
  cfg.blockDim = dim3(kWgpThreads);
  cfg.dynamicSmemBytes = kWgpSmem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  GNNCO_CUDA_TRY(cudaLaunchKernelEx(&cfg, weight_grad_tc_pair, ma, mg, dW, scratch, (const int32_t*)h->wg_begin,
                                    (const int32_t*)h->wg_end, (const int32_t*)h->wg_slot, (int)h->n_wg_chunks, h->status));
  h->launches += 1;
  return launch_wg_combine(h, scratch, dW, (int64_t)K * N, st);
}
