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

// What an epilogue warp does with its 32 rows x 64 columns of an accumulator tile once they are in registers
// (ra: columns c0 .. c0+31 of this thread's row, rb: the next 32): scale / ReLU (inside the conversion to bf16) /
// mask, optional sign bits of the stored values, optional dot product of the stored row with the next layer's
// weight vector (column groups are added in the order 0, 1, 2, 3; group 0 collects and writes), staging and one
// TMA store per 32 columns -- plain stores where the tile is ragged.  False: the wait for the other column
// groups' partial dot products ran out.
template <int NDIM, int MODE>
__device__ __forceinline__ bool convert_and_store(const uint32_t (&ra)[32], const uint32_t (&rb)[32], float s, uint2 mk,
                                                  const __nv_bfloat16* wv, uint8_t* __restrict__ bits_out,
                                                  float* __restrict__ dot_out, __nv_bfloat16* __restrict__ Y,
                                                  const CUtensorMap* map_y, uint32_t stage, int64_t row0, int row,
                                                  int quarter, int cg, int lane, int rows_here, bool valid, float* dot_x,
                                                  uint64_t* dot_bar, int buf, uint32_t dot_parity) {
  const int c0 = cg * 64;
  float dot = 0.0f;
  uint32_t sign_words[2] = {0u, 0u};
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
      if (lane == 0) tma_store_2d(map_y, stage, c0 + hh * 32, (int32_t)(row0 + quarter * 32));
    } else if (valid) {
      // ragged end of a subgraph: a box would reach into the next subgraph's rows
      uint4* dst = reinterpret_cast<uint4*>(Y + (row0 + row) * NDIM + c0 + hh * 32);
#pragma unroll
      for (int pc = 0; pc < 4; ++pc) dst[pc] = make_uint4(o[4 * pc], o[4 * pc + 1], o[4 * pc + 2], o[4 * pc + 3]);
    }
  }
  if (MODE == kModeRelu && dot_out) {
    if (cg > 0) {
      dot_x[(buf * 3 + cg - 1) * 128 + row] = dot;
      tc::mbar_arrive(dot_bar + quarter * 2 + buf);
    } else {
      if (!tc::mbar_wait_bounded(dot_bar + quarter * 2 + buf, dot_parity)) return false;
      dot += dot_x[(buf * 3 + 0) * 128 + row];
      dot += dot_x[(buf * 3 + 1) * 128 + row];
      dot += dot_x[(buf * 3 + 2) * 128 + row];
      if (valid) dot_out[row0 + row] = dot;
    }
  }
  return true;
}

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
      if (!convert_and_store<NDIM, MODE>(ra, rb, s, mk, wv, bits_out, dot_out, Y, &map_y, stage, row0, row, quarter, cg, lane,
                                         rows_here, valid, dot_x, dot_bar, buf, (j >> 1) & 1)) {
        *abort_flag = 1;
        break;
      }
      if (late_release) {
        __syncwarp();
        if (lane == 0) tc::mbar_arrive_cluster(acc_empty_even + buf * 8);
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
// Aggregation and transform of one hidden layer in ONE kernel (Eq. 3: H' = ReLU(D^-1 (A + I) H W_s)), by pairs of
// CTAs as above, for widths 256 -> 256.  The aggregated rows never exist in HBM: they are summed on chip straight
// into the A operand of the MMAs, which saves writing and re-reading one feature tensor per layer.
//
//   * A source list (built once per graph: every row's own index followed by its neighbours', rows in order) names
//     the feature rows a tile needs.  One warp walks it and gathers them with TMA, four named rows (2 KB) per
//     instruction, into a ring of shared memory; each instruction has its own `landed` / `consumed` barrier pair.
//     The ring (about 60 KB) is the memory parallelism of the kernel -- no warp waits on a global load of features.
//   * The sixteen epilogue warps are also the adders: warp w sums the landed source rows of the tile's rows w,
//     w + 16, ... in list order (float32, the order of the stand-alone aggregation kernel, hence the same bits),
//     scales by 1 / (degree + 1), rounds to bf16 and writes the row into the operand tile in the 128-byte-swizzled
//     layout of the MMA descriptors.  One arrival per warp of both CTAs on the even CTA's `a_full` starts the MMAs.
//   * The operand tile is single (64 KB; the weights' half and the ring take the rest).  Per tile the adders sum
//     their eight rows into REGISTERS while the previous tile's MMAs still read the operand tile, then wait for
//     those MMAs, store the rows, announce the tile and drain the previous accumulator (TMEM holds two) while
//     the tensor cores work on the new one.  The ring is emptied all the time except during the drain, a pause
//     that its 60 KB in flight cover, so the gathers never stop.
//   * Warp 16: one lane per CTA loads this CTA's half of the weights when the subgraph changes (after the previous
//     tile's MMAs); in the even CTA it then issues the pair's MMAs.
// A row is summed by ONE warp and the ring is a queue, so a long row would hold up the fifteen other warps; and
// the CTA pairs get fixed ranges of tiles, so a tile with many times the usual number of list entries would be
// the tail of the kernel.  Double tiles with a row of more than kFuseLongRow entries or more than kFuseHeavyTile
// entries in all ("heavy": a few percent of the tiles of a power-law graph, around its hubs) are therefore left
// to the separate aggregation and transform kernels, and the light tiles are dealt out to the CTA pairs in
// contiguous ranges of about equal cost (build_fuse_set).
constexpr int kFuseOps = 30;                         // gather instructions in flight: 30 x 4 rows x 512 B = 60 KB
constexpr int kFusePos = 4 * kFuseOps;               // ring positions (one source row each)
constexpr uint32_t kFuseRowBytes = 512;              // 256 bf16
constexpr uint32_t kFuseRing = kFuseOps * 4 * kFuseRowBytes;
constexpr uint32_t kFuseMisc = 4096;                 // barriers (1 KB) + dot-product exchange (3 KB)
constexpr uint32_t kFuseA = 4 * 128 * 128;           // four k-blocks of 128 rows x 64 bf16
constexpr uint32_t kFuseB = 4 * 128 * 128;           // this CTA's 128 of the 256 weight rows, four k-blocks
constexpr uint32_t kFuseEpi = kPairEpiWarps * kPairStage;
constexpr size_t kFuseSmem = 1024 + kFuseA + kFuseB + kFuseEpi + kFuseRing + kFuseMisc;
constexpr int kFuseLongRow = 64;                     // a double tile with a longer row (own entry included) is "heavy" ...
constexpr int kFuseHeavyTile = 2048;                 // ... and so is one with more list entries than this
constexpr int kFuseTileCost = 320;                   // fixed cost of a tile (MMAs, drain) in list entries, for the split
constexpr int kFusePrefetch = 4;                     // chunks of 32 gather instructions whose row names are read a tile ahead
static_assert(kFuseSmem <= kPairSmemLimit, "does not fit in shared memory");
static_assert(kFuseOps <= 32, "barrier area holds 32 gather slots");

// One CTA's share of a double tile, as the table built with the graph gives it: the double tile's first row,
// this CTA's row count (0 to 128) and the extent [beg, end) of its rows in the source list.
struct FuseTile {
  int32_t pair_r0, rows, beg, end;
};
__device__ __forceinline__ FuseTile fuse_tile(int t, int t_end, uint32_t rank, const int4* __restrict__ fuse_meta) {
  FuseTile m{0, 0, 0, 0};
  if (t < t_end) {
    const int4 v = __ldg(fuse_meta + 2 * (int64_t)t + rank);
    m.pair_r0 = v.x; m.rows = v.y; m.beg = v.z; m.end = v.w;
  }
  return m;
}
// gather instructions of a tile: its list extent, widened down to a multiple of four entries
__device__ __forceinline__ int fuse_ops(const FuseTile& m) {
  return m.rows > 0 ? (m.end - (m.beg & ~3) + 3) >> 2 : 0;
}

__global__ void __launch_bounds__(kPairThreads, 1)
aggregate_transform_pair(const __grid_constant__ CUtensorMap map_h, const __grid_constant__ CUtensorMap map_b,
                         const __grid_constant__ CUtensorMap map_y, int32_t b_per_part, __nv_bfloat16* __restrict__ Y,
                         const int32_t* __restrict__ src_list, const int4* __restrict__ row_head,
                         const float* __restrict__ row_scale, uint8_t* __restrict__ bits_out,
                         const __nv_bfloat16* __restrict__ dot_w, int64_t dot_stride, float* __restrict__ dot_out,
                         const int4* __restrict__ fuse_meta, const int32_t* __restrict__ cluster_begin,
                         const int32_t* __restrict__ node_part, int32_t oob_row, int32_t* status) {
  constexpr int NDIM = 256, KB = 4;
  constexpr uint32_t A_SLOT = 128 * 128, B_SLOT = 128 * 128;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t sbase = (tc::smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sA = sbase, sB = sA + kFuseA, sStage = sB + kFuseB, sRing = sStage + kFuseEpi;
  uint8_t* misc = smem_raw + (sbase - tc::smem_u32(smem_raw)) + kFuseA + kFuseB + kFuseEpi + kFuseRing;
  uint64_t* g_full = reinterpret_cast<uint64_t*>(misc);        // [32] a gather's four rows have landed
  uint64_t* g_empty = g_full + 32;                             // [32] ... and have been added (four arrivals)
  uint64_t* a_full = g_empty + 32;                             // operand tile written by both CTAs (even CTA's copy is used)
  uint64_t* b_full = a_full + 1;                               // both halves of the weights have landed (even CTA's copy)
  uint64_t* acc_full = b_full + 1;                             // [2] both CTAs
  uint64_t* dot_bar = acc_full + 2;                            // [4 quarters][2 buffers]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(dot_bar + 8);
  volatile uint32_t* abort_flag = tmem_slot + 1;
  volatile uint32_t* g_issued = reinterpret_cast<volatile uint32_t*>(misc + 640);   // [32] fills of each gather slot so far
  float* dot_x = reinterpret_cast<float*>(misc + 1024);        // [2 buffers][3 column groups][128 rows]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = tc::cluster_ctarank();
  const int cluster_id = blockIdx.x >> 1;
  const int t_begin = __ldg(cluster_begin + cluster_id), t_end = __ldg(cluster_begin + cluster_id + 1);
  if (t_begin >= t_end) return;                                // both CTAs of the cluster leave together

  if (threadIdx.x == 0) {
    for (int i = 0; i < kFuseOps; ++i) {
      tc::mbar_init(g_full + i, 1);
      tc::mbar_init(g_empty + i, 4);
      g_issued[i] = 0u;
    }
    tc::mbar_init(a_full, 2 * kPairEpiWarps);
    tc::mbar_init(b_full, 2);
    for (int i = 0; i < 2; ++i) tc::mbar_init(acc_full + i, 1);
    for (int i = 0; i < 8; ++i) tc::mbar_init(dot_bar + i, 96);
    *abort_flag = 0;
    tc::fence_mbar_init();
  }
  if (warp == 0) tc::tmem_alloc_pair(tmem_slot, 2 * NDIM);
  tc::tc_fence_before_sync();
  __syncthreads();
  tc::cluster_sync_all();
  tc::tc_fence_after_sync();
  const uint32_t tmem = *tmem_slot;

  if (warp == kPairTmaWarp) {
    // ------------------------------------------------------------------- gather producer (all lanes)
    FuseTile cur = fuse_tile(t_begin, t_end, rank, fuse_meta);
    FuseTile nxt = fuse_tile(t_begin + 1, t_end, rank, fuse_meta);
    // the four row names of gather `op` of a tile; list entries outside the tile's extent (the widening to a
    // multiple of four) name a row past the tensor, which reads as zeros and is added by nobody
    auto names = [&](const FuseTile& m, int op) -> int4 {
      int4 v = make_int4(oob_row, oob_row, oob_row, oob_row);
      const int64_t a = (int64_t)(m.beg & ~3) + 4 * (int64_t)op;
      if (m.rows > 0 && a < m.end) {
        v = __ldg(reinterpret_cast<const int4*>(src_list + a));
        if (a < m.beg || a >= m.end) v.x = oob_row;
        if (a + 1 < m.beg || a + 1 >= m.end) v.y = oob_row;
        if (a + 2 < m.beg || a + 2 >= m.end) v.z = oob_row;
        if (a + 3 < m.beg || a + 3 >= m.end) v.w = oob_row;
      }
      return v;
    };
    uint32_t qbase = 0;                                          // gathers issued by this CTA before this tile
    auto issue = [&](const int4 v, int op, int ops) {
      if (op >= ops || *abort_flag) return;
      const uint32_t q = qbase + (uint32_t)op, slot = q % kFuseOps, use = q / kFuseOps;
      if (use > 0 && !tc::mbar_wait_bounded(g_empty + slot, (use - 1) & 1)) { *abort_flag = 1; return; }
      // a name outside [0, n] would be a corrupt list: give up rather than hand it to the copy engine
      if ((uint32_t)v.x > (uint32_t)oob_row || (uint32_t)v.y > (uint32_t)oob_row || (uint32_t)v.z > (uint32_t)oob_row ||
          (uint32_t)v.w > (uint32_t)oob_row) {
        *abort_flag = 1;
        return;
      }
      const uint32_t dead = (v.x == oob_row) + (v.y == oob_row) + (v.z == oob_row) + (v.w == oob_row);
      g_issued[slot] = use + 1u;                                   // the slot's barrier is now in phase `use`
      tc::mbar_arrive_expect_tx_cluster(tc::smem_u32(g_full + slot), 4 * kFuseRowBytes);
      tc::tma_gather4_rows(sRing + slot * 4 * kFuseRowBytes, &map_h, 0, v.x, v.y, v.z, v.w, g_full + slot);
      if (dead) tc::mbar_arrive_count(g_empty + slot, dead);       // nobody will add those
    };
    // A chunk is one gather per lane for the first kFuseOps lanes: the slot a lane waits for was last filled by
    // the same lane one chunk earlier (or in an earlier tile), never by a lane of the chunk being issued --
    // lanes of one warp must not wait for one another.
    const bool issuer = lane < kFuseOps;
    int4 pre[kFusePrefetch];
#pragma unroll
    for (int c = 0; c < kFusePrefetch; ++c) pre[c] = names(cur, issuer ? c * kFuseOps + lane : 1 << 28);
    for (int t = t_begin; t < t_end && !*abort_flag; ++t) {
      // requested now, used one tile later: the tile after next's extent, the next tile's first row names
      const FuseTile after = fuse_tile(t + 2, t_end, rank, fuse_meta);
      int4 pre_next[kFusePrefetch];
#pragma unroll
      for (int c = 0; c < kFusePrefetch; ++c) pre_next[c] = names(nxt, issuer ? c * kFuseOps + lane : 1 << 28);
      const int ops = issuer ? fuse_ops(cur) : 0;
#pragma unroll
      for (int c = 0; c < kFusePrefetch; ++c) {
        issue(pre[c], c * kFuseOps + lane, ops);
        __syncwarp();
      }
      for (int c = kFusePrefetch; c * kFuseOps < fuse_ops(cur); ++c) {
        issue(names(cur, issuer ? c * kFuseOps + lane : 1 << 28), c * kFuseOps + lane, ops);
        __syncwarp();
      }
      qbase += (uint32_t)fuse_ops(cur);
      cur = nxt;
      nxt = after;
#pragma unroll
      for (int c = 0; c < kFusePrefetch; ++c) pre[c] = pre_next[c];
    }
    __syncwarp();
  } else if (warp == kPairMmaWarp) {
    // ---------------------------------------------------- weights (each CTA its half) and MMAs (even CTA)
    if (lane == 0) {
      constexpr uint32_t IDESC = tc::idesc_bf16_f32(256, NDIM, false, false);
      const uint32_t b_full_even = tc::map_to_cta(tc::smem_u32(b_full), 0);
      int cur_part = -1, loads = 0;
      for (int t = t_begin, j = 0; t < t_end && !*abort_flag; ++t, ++j) {
        const int buf = j & 1;
        const int part = node_part[__ldg(fuse_meta + 2 * (int64_t)t).x];
        const bool new_b = part != cur_part;
        cur_part = part;
        // Every tile's completion is observed, in order, whether or not the weights change: a parity wait names a
        // phase only to somebody who has seen the one before it (the odd CTA's lane has nothing else to pace it).
        if (j > 0 && !tc::mbar_wait_bounded(acc_full + (buf ^ 1), ((j - 1) >> 1) & 1)) { *abort_flag = 1; break; }
        if (new_b) {
          // the previous tile's MMAs (of both CTAs) have read the weights that are about to be replaced
          tc::mbar_arrive_expect_tx_cluster(b_full_even, kFuseB);
#pragma unroll
          for (int kb = 0; kb < KB; ++kb)
            tc::tma_load_2d_pair(sB + kb * B_SLOT, &map_b, kb * 64, part * b_per_part + (int32_t)rank * (NDIM / 2),
                                 b_full_even);
        }
        if (rank == 0) {
          if (new_b) {
            if (!tc::mbar_wait_bounded(b_full, loads & 1)) { *abort_flag = 1; break; }
            ++loads;
          }
          if (!tc::mbar_wait_bounded(a_full, j & 1)) { *abort_flag = 1; break; }
          tc::tc_fence_after_sync();
#pragma unroll
          for (int kb = 0; kb < KB; ++kb) {
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
              const uint64_t ad = tc::smem_desc_sw128(sA + kb * A_SLOT + ks * 32, 16, 1024);
              const uint64_t bd = tc::smem_desc_sw128(sB + kb * B_SLOT + ks * 32, 16, 1024);
              tc::mma_bf16_pair(tmem + buf * NDIM, ad, bd, IDESC, (kb | ks) != 0);
            }
          }
          tc::mma_commit_pair(acc_full + buf, 3);
        }
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------- adders and epilogue (this CTA's 128 rows)
    const int quarter = warp & 3, cg = warp >> 2;
    const int row = quarter * 32 + lane;
    const uint32_t stage = sStage + warp * kPairStage;
    const uint32_t a_full_even = tc::map_to_cta(tc::smem_u32(a_full), 0);
    // drain of tile (jd, row0d, rowsd, partd): its accumulator is known to be complete
    auto drain = [&](int jd, int64_t row0d, int rowsd, int partd) -> bool {
      const int buf = jd & 1;
      const bool valid = row < rowsd;
      const __nv_bfloat16* wv = dot_out ? dot_w + (int64_t)partd * dot_stride + cg * 64 : nullptr;
      uint32_t ra[32], rb[32];
      const uint32_t at = tmem + ((uint32_t)(quarter * 32) << 16) + buf * NDIM + cg * 64;
      tc::tmem_ld_32x32(at, ra);
      tc::tmem_ld_32x32(at + 32, rb);
      tc::tmem_ld_wait();
      tc::tc_fence_before_sync();
      return convert_and_store<NDIM, kModeRelu>(ra, rb, 1.0f, make_uint2(0u, 0u), wv, bits_out, dot_out, Y, &map_y, stage,
                                                row0d, row, quarter, cg, lane, rowsd - quarter * 32, valid, dot_x, dot_bar,
                                                buf, (jd >> 1) & 1);
    };
    FuseTile cur = fuse_tile(t_begin, t_end, rank, fuse_meta);
    FuseTile nxt = fuse_tile(t_begin + 1, t_end, rank, fuse_meta);
    uint32_t qbase = 0;
    // lane k < 8 holds the extent of row warp + 16 k of the tile: first ring position, entries (0: no such row),
    // scale
    auto extent = [&](const FuseTile& m, uint32_t q0, uint32_t& pos, int& cnt, float& sc) {
      pos = 0; cnt = 0; sc = 0.0f;
      const int rr = warp + 16 * lane;
      if (lane < 8 && rr < m.rows) {
        const int32_t r = m.pair_r0 + (int32_t)rank * 128 + rr;
        const int4 hd = __ldg(row_head + r);
        pos = (uint32_t)(hd.x + r - (m.beg & ~3)) + 4u * q0;
        cnt = hd.y + 1;
        sc = __ldg(row_scale + r);
      }
    };
    uint32_t pos, pos_n;
    int cnt, cnt_n;
    float sc, sc_n;
    extent(cur, 0u, pos, cnt, sc);
    int part = dot_out ? __ldg(node_part + cur.pair_r0) : 0, part_n = 0;
    int64_t prev_row0 = 0;
    int prev_rows = 0, prev_part = 0, j = 0;
    bool ok = true;
    for (int t = t_begin; t < t_end && ok && !*abort_flag; ++t, ++j) {
      // requested now, used one tile later
      const FuseTile after = fuse_tile(t + 2, t_end, rank, fuse_meta);
      const uint32_t qnext = qbase + (uint32_t)fuse_ops(cur);
      extent(nxt, qnext, pos_n, cnt_n, sc_n);
      if (dot_out && t + 1 < t_end) part_n = __ldg(node_part + nxt.pair_r0);
      // The rows are summed into registers FIRST, while the previous tile's MMAs still read the operand tile: the
      // ring is emptied (and refilled) all the time except during the drain below, which its 60 KB cover.
      uint4 packed[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const uint32_t p = __shfl_sync(0xffffffffu, pos, k);
        int c = __shfl_sync(0xffffffffu, cnt, k);
        const float s = __shfl_sync(0xffffffffu, sc, k);
        float acc[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] = 0.0f;
        uint32_t ri = p % kFusePos, use = p / kFusePos;       // ring position and how often the ring has gone round
        while (c > 0 && ok) {
          const uint32_t o = ri >> 2;
          const int take = min(c, 4 - (int)(ri & 3u));
          // A parity names a phase only to somebody who knows which phase the barrier is in, and an adder that
          // waits behind a long row may not have looked at this slot for many turns of the ring.  The producer
          // counts the fills of every slot: once fill `use` has been issued the barrier is in phase `use` (the
          // next fill needs this warp's arrival), and the parity wait is exact.
          bool landed = true;
          if (g_issued[o] <= use) {
            const long long t0 = clock64();
            while (g_issued[o] <= use) {
              if (*abort_flag || clock64() - t0 > 4000000000ll) { landed = false; break; }
            }
          }
          landed = landed && tc::mbar_wait_bounded(g_full + o, use & 1u);
          if (!__all_sync(0xffffffffu, landed)) { ok = false; break; }
          const uint32_t src = sRing + ri * kFuseRowBytes + lane * 16;
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            if (i < take) {
              const uint4 v = tc::ld_shared16(src + i * kFuseRowBytes);
              const uint32_t w4[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                acc[2 * e] += __uint_as_float(w4[e] << 16);
                acc[2 * e + 1] += __uint_as_float(w4[e] & 0xffff0000u);
              }
            }
          }
          __syncwarp();
          if (lane == 0) tc::mbar_arrive_count(g_empty + o, (uint32_t)take);
          ri += (uint32_t)take;
          c -= take;
          if (ri == kFusePos) { ri = 0; ++use; }
        }
        packed[k] = make_uint4(pack_bf16<false>(acc[0] * s, acc[1] * s), pack_bf16<false>(acc[2] * s, acc[3] * s),
                               pack_bf16<false>(acc[4] * s, acc[5] * s), pack_bf16<false>(acc[6] * s, acc[7] * s));
      }
      if (!ok) break;
      if (j > 0) {
        // the previous tile's MMAs are done: the operand tile is free and that accumulator can be drained
        if (!__all_sync(0xffffffffu, tc::mbar_wait_bounded(acc_full + ((j - 1) & 1), ((j - 1) >> 1) & 1))) {
          ok = false;
          break;
        }
        tc::tc_fence_after_sync();
      }
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        // 16 bytes of row rr: k-block lane / 8, piece lane % 8, XORed with rr % 8 (the 128-byte swizzle)
        const int rr = warp + 16 * k;
        if (rr < cur.rows) {
          const uint32_t dst = sA + (uint32_t)(lane >> 3) * A_SLOT + rr * 128 + (((lane & 7) ^ (rr & 7)) << 4);
          tc::st_shared16(dst, packed[k].x, packed[k].y, packed[k].z, packed[k].w);
        }
      }
      tc::fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) tc::mbar_arrive_release_cluster(a_full_even);
      if (j > 0 && !drain(j - 1, prev_row0, prev_rows, prev_part)) { ok = false; break; }
      prev_row0 = (int64_t)cur.pair_r0 + (int64_t)rank * 128;
      prev_rows = cur.rows;
      prev_part = part;
      part = part_n;
      qbase = qnext;
      cur = nxt;
      nxt = after;
      pos = pos_n; cnt = cnt_n; sc = sc_n;
    }
    if (ok && !*abort_flag) {
      // the last tile
      if (!__all_sync(0xffffffffu, tc::mbar_wait_bounded(acc_full + ((j - 1) & 1), ((j - 1) >> 1) & 1))) ok = false;
      tc::tc_fence_after_sync();
      if (ok && !drain(j - 1, prev_row0, prev_rows, prev_part)) ok = false;
    }
    if (!ok) *abort_flag = 1;
    if (lane == 0) tma_store_wait_all();
    __syncwarp();
  }
  if (*abort_flag) {
    // a wait ran out: give the gathers, weight boxes and MMAs already in flight (microseconds of work) time to
    // finish before this CTA's shared memory and TMEM are handed back
    if (threadIdx.x == 0) atomicMin(status, (int32_t)GNNCO_INTERNAL);
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000ll) {}
  }
  tc::tc_fence_before_sync();
  __syncthreads();
  tc::cluster_sync_all();
  if (warp == 0) tc::tmem_dealloc_pair(tmem, 2 * NDIM);
}

// Per-tile figures for the split into light and heavy double tiles: entries of the source list and the longest row.
__global__ void fuse_tile_weights(const int32_t* __restrict__ pair_row0, const int32_t* __restrict__ pair_rows, int n_pairs,
                                  const int4* __restrict__ row_head, int2* __restrict__ out) {
  const int t = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (t >= n_pairs) return;
  const int32_t r0 = pair_row0[t], rows = pair_rows[t];
  int total = 0, longest = 0;
  for (int r = lane; r < rows; r += 32) {
    const int c = row_head[r0 + r].y + 1;
    total += c;
    longest = max(longest, c);
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    total += __shfl_xor_sync(0xffffffffu, total, off);
    longest = max(longest, __shfl_xor_sync(0xffffffffu, longest, off));
  }
  if (lane == 0) out[t] = make_int2(total, longest);
}

// {double tile's first row, this CTA's rows, extent of those rows in the source list} for both CTAs of each light tile
__global__ void fuse_tile_meta(const int32_t* __restrict__ row0, const int32_t* __restrict__ rows, int n_tiles,
                               const int4* __restrict__ row_head, int4* __restrict__ meta) {
  const int g = blockIdx.x * blockDim.x + threadIdx.x;
  if (g >= 2 * n_tiles) return;
  const int t = g >> 1, rank = g & 1;
  const int32_t pr0 = row0[t], r0 = pr0 + rank * 128;
  const int32_t cnt = max(0, min(128, rows[t] - rank * 128));
  int4 m = make_int4(pr0, cnt, 0, 0);
  if (cnt > 0) {
    const int4 h0 = row_head[r0], h1 = row_head[r0 + cnt - 1];
    m.z = h0.x + r0;                                   // row i starts at rowptr[i] + i: one own entry per row
    m.w = h1.x + h1.y + r0 + cnt;
  }
  meta[g] = m;
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

// co-resident CTA pairs of the one-kernel layer (0: clusters of two cannot be launched)
static int resident_fuse_pairs() {
  auto kernel = aggregate_transform_pair;
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kFuseSmem) != cudaSuccess) {
    cudaGetLastError();
    return 0;
  }
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(2 * 148);
  cfg.blockDim = dim3(kPairThreads);
  cfg.dynamicSmemBytes = kFuseSmem;
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

int32_t build_fuse_set(gnnco_handle* h, const int32_t* d_pair_row0, const int32_t* d_pair_rows,
                       const std::vector<int32_t>& p0, const std::vector<int32_t>& pr, FuseSet& fs, cudaStream_t st) {
  fs.built = false;
  fs.n_light = fs.n_heavy = fs.clusters = 0;
  const int n_pairs = (int)p0.size();
  // list positions are 32-bit in the kernel
  if (n_pairs == 0 || !h->src_list || !encode_tiled() || h->n + 2 * h->E_in >= ((int64_t)1 << 31) - 8) return GNNCO_OK;
  static int resident = -1;
  if (resident < 0) resident = resident_fuse_pairs();
  if (resident <= 0) return GNNCO_OK;
  fuse_tile_weights<<<(n_pairs + 7) / 8, 256, 0, st>>>(d_pair_row0, d_pair_rows, n_pairs, h->row_head, fs.weights);
  h->launches += 1;
  std::vector<int2> wt((size_t)n_pairs);
  GNNCO_CUDA_TRY(cudaMemcpyAsync(wt.data(), fs.weights, wt.size() * sizeof(int2), cudaMemcpyDeviceToHost, st));
  GNNCO_CUDA_TRY(cudaStreamSynchronize(st));
  std::vector<int32_t> l0, lr, h0, hr;
  std::vector<int64_t> cost;                    // of the light tiles: list entries plus a fixed part for the MMAs and the drain
  int64_t total = 0;
  for (int t = 0; t < n_pairs; ++t) {
    if (wt[t].y > kFuseLongRow || wt[t].x > kFuseHeavyTile) {
      h0.push_back(p0[t]);
      hr.push_back(pr[t]);
    } else {
      l0.push_back(p0[t]);
      lr.push_back(pr[t]);
      cost.push_back((int64_t)wt[t].x + kFuseTileCost);
      total += cost.back();
    }
  }
  fs.n_light = (int32_t)l0.size();
  fs.n_heavy = (int32_t)h0.size();
  int clusters = resident < kFuseMaxClusters ? resident : kFuseMaxClusters;
  if (clusters > fs.n_light) clusters = fs.n_light;
  std::vector<int32_t> cb((size_t)clusters + 1, 0);
  {
    // contiguous ranges of about total / clusters each (a subgraph's tiles stay together: one load of its weights)
    int64_t seen = 0;
    int c = 1;
    for (int t = 0; t < fs.n_light && c < clusters; ++t) {
      seen += cost[t];
      while (c < clusters && seen * clusters >= total * c) cb[c++] = t + 1;
    }
    while (c <= clusters) cb[c++] = fs.n_light;
    if (clusters > 0) cb[clusters] = fs.n_light;
  }
  fs.clusters = clusters;
  auto up = [&](int32_t* dst, const std::vector<int32_t>& v) {
    return v.empty() ? cudaSuccess : cudaMemcpyAsync(dst, v.data(), v.size() * sizeof(int32_t), cudaMemcpyHostToDevice, st);
  };
  GNNCO_CUDA_TRY(up(fs.light_row0, l0));
  GNNCO_CUDA_TRY(up(fs.light_rows, lr));
  GNNCO_CUDA_TRY(up(fs.heavy_row0, h0));
  GNNCO_CUDA_TRY(up(fs.heavy_rows, hr));
  GNNCO_CUDA_TRY(up(fs.cluster_begin, cb));
  if (fs.n_light > 0) {
    fuse_tile_meta<<<(2 * fs.n_light + 255) / 256, 256, 0, st>>>(fs.light_row0, fs.light_rows, fs.n_light, h->row_head, fs.meta);
    h->launches += 1;
  }
  GNNCO_CUDA_TRY(cudaStreamSynchronize(st));      // the host vectors go out of scope
  GNNCO_CUDA_TRY(cudaGetLastError());
  fs.built = true;
  return GNNCO_OK;
}

// The one-kernel layer needs the tables that build_fuse_set made for the running work set.
bool aggregate_transform_pair_supported(gnnco_handle* h, int dtype, int K, int N) {
  return tc_pair_transform_supported(h, dtype, K, N) && h->src_list && h->fuse.built;
}

// Y = ReLU( (row_scale * (A + I) Hin) B_s^T ) on the LIGHT double tiles of the running work set, Hin and Y
// [n x 256] bf16, B as in launch_transform_tc_pair; optional sign bits of Y and dot products of Y's rows with
// dot_w, as there.  The heavy double tiles (h->fuse.heavy_*) are the caller's to run through the separate kernels.
int32_t launch_aggregate_transform_pair(gnnco_handle* h, const void* Hin, const void* B, int64_t b_stride, int32_t b_sets,
                                        void* Y, int K, int N, const float* row_scale, uint8_t* bits_out, const void* dot_w,
                                        int64_t dot_stride, float* dot_out, cudaStream_t st) {
  if (!aggregate_transform_pair_supported(h, GNNCO_BF16, K, N) || !row_scale) return GNNCO_UNSUPPORTED;
  if (((uintptr_t)Hin & 15) || ((uintptr_t)B & 15) || ((uintptr_t)Y & 15) || ((uintptr_t)bits_out & 7) ||
      ((uintptr_t)h->src_list & 15) || (b_stride != 0 && b_stride != (int64_t)K * N))
    return GNNCO_UNSUPPORTED;
  if (h->fuse.n_light == 0 || h->fuse.clusters == 0) return GNNCO_OK;
  ProfScope prof_(h, K_AGG_TRANSFORM, st);
  CUtensorMap mh, mb, my;
  // gathered rows: boxes of one whole row, dense; weights and results as in the plain pair kernel
  if (!make_map(&mh, Hin, (uint64_t)h->n, 256, 1, 256, false)) return GNNCO_CUDA_ERROR;
  if (!make_map(&mb, B, (uint64_t)b_sets * 256, 256, 128, 64, true)) return GNNCO_CUDA_ERROR;
  if (!make_map(&my, Y, (uint64_t)h->n, 256, 32, 32, false)) return GNNCO_CUDA_ERROR;
  auto kernel = aggregate_transform_pair;
  GNNCO_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kFuseSmem));
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(2 * h->fuse.clusters);
  cfg.blockDim = dim3(kPairThreads);
  cfg.dynamicSmemBytes = kFuseSmem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const int32_t b_per_part = b_stride == 0 ? 0 : 256;
  GNNCO_CUDA_TRY(cudaLaunchKernelEx(&cfg, kernel, mh, mb, my, b_per_part, (__nv_bfloat16*)Y, (const int32_t*)h->src_list,
                                    (const int4*)h->row_head, row_scale, bits_out, (const __nv_bfloat16*)dot_w, dot_stride,
                                    dot_out, (const int4*)h->fuse.meta, (const int32_t*)h->fuse.cluster_begin,
                                    (const int32_t*)h->node_part, (int32_t)h->n, h->status));
  h->launches += 1;
  return GNNCO_OK;
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
