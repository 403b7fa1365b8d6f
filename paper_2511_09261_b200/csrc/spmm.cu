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
// Rank-1 mode (template flag R1), for the layer below the width-1 output layer: its incoming
// gradient is dZ[j,f] = g_j w_s[f] [H[j,f] > 0], so the transposed aggregation of D^-1 dZ is
//   out[i,f] = w_s[f] * sum_{j in {i} + row i} coef[j] [H[j,f] > 0],     coef = D^-1 g,
// which gathers the saved activation H directly; dZ itself is never written.
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
  __device__ static uint4 load_raw(const float* p) { return __ldg(reinterpret_cast<const uint4*>(p)); }
  __device__ static void unpack(const uint4& v, float (&f)[4]) {
    f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y); f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
  }
  __device__ static void add_raw(float (&acc)[4], const uint4& v) {
    acc[0] += __uint_as_float(v.x); acc[1] += __uint_as_float(v.y);
    acc[2] += __uint_as_float(v.z); acc[3] += __uint_as_float(v.w);
  }
  // acc[e] += c where the element is positive
  __device__ static void add_where_positive(float (&acc)[4], const uint4& v, float c) {
    acc[0] += __uint_as_float(v.x) > 0.0f ? c : 0.0f; acc[1] += __uint_as_float(v.y) > 0.0f ? c : 0.0f;
    acc[2] += __uint_as_float(v.z) > 0.0f ? c : 0.0f; acc[3] += __uint_as_float(v.w) > 0.0f ? c : 0.0f;
  }
  __device__ static void store(float* p, const float (&f)[4]) {
    // streaming store: an output row is not read again by this kernel, the gathered rows are
    __stcs(reinterpret_cast<float4*>(p), make_float4(f[0], f[1], f[2], f[3]));
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
  __device__ static uint4 load_raw(const __nv_bfloat16* p) { return __ldg(reinterpret_cast<const uint4*>(p)); }
  __device__ static void unpack(const uint4& v, float (&f)[8]) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      f[2 * k] = __uint_as_float(w[k] << 16);
      f[2 * k + 1] = __uint_as_float(w[k] & 0xffff0000u);
    }
  }
  // acc[e] += element e.  The mixed-precision add takes the bfloat16 halves of a word as they are instead of a
  // shift or mask plus an add per element; same bits.  The aggregation kernel is bound by instruction issue
  // (85 % of the issue slots busy, 168 warp instructions per 256-wide row before this; 134 with this and the
  // compile-time row width), so instructions saved are time saved: this loop alone 1.78 against 2.94 ms.
  __device__ static void add_raw(float (&acc)[8], const uint4& v) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int k = 0; k < 4; ++k)
      asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %2;\n\t"
          "add.rn.f32.bf16 %0, lo, %0;\n\tadd.rn.f32.bf16 %1, hi, %1;\n\t}"
          : "+f"(acc[2 * k]), "+f"(acc[2 * k + 1])
          : "r"(w[k]));
  }
  __device__ static void add_where_positive(float (&acc)[8], const uint4& v, float c) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      acc[2 * k] += __uint_as_float(w[k] << 16) > 0.0f ? c : 0.0f;
      acc[2 * k + 1] += __uint_as_float(w[k] & 0xffff0000u) > 0.0f ? c : 0.0f;
    }
  }
  __device__ static void store(__nv_bfloat16* p, const float (&f)[8]) {
    uint32_t w[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      __nv_bfloat162 b = __floats2bfloat162_rn(f[2 * k], f[2 * k + 1]);
      w[k] = *reinterpret_cast<uint32_t*>(&b);
    }
    __stcs(reinterpret_cast<uint4*>(p), make_uint4(w[0], w[1], w[2], w[3]));
  }
};

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ void from_f32(float& d, float x) { d = x; }
__device__ __forceinline__ void from_f32(__nv_bfloat16& d, float x) { d = __float2bfloat16_rn(x); }

// Arguments of the rank-1 mode.
template <typename T>
struct Rank1Args {
  const float* coef;            // D^-1 g, one value per node
  const T* w;                   // output-layer weight vectors [sets x F], in the features' type
  int64_t w_stride;             // 0 when all subgraphs share one vector
  const int32_t* node_part;
};

template <typename T, bool R1>
__device__ __forceinline__ void accumulate(float (&acc)[Vec<T>::N], const uint4& v, float c) {
  if constexpr (R1) Vec<T>::add_where_positive(acc, v, c);
  else Vec<T>::add_raw(acc, v);
}

// LPR lanes per row, VPL vectors per lane: row width F = LPR * VPL * Vec<T>::N elements.
// Threads per block of the row-per-warp aggregation.  Measured on B200 (width 256, bfloat16, alternating runs on one device): 128
// threads 1.95-1.97 ms, 256 threads 1.99-2.01 ms, 64 threads 2.81-2.85 ms per launch of 10 M rows.
constexpr int kAggThreads = 128;

// row_head[i] = {first CSR slot, degree, first neighbour, second neighbour}: one 16-byte load
// tells a row its extent AND its first two neighbours, so for the many rows of degree <= 2
// the neighbour features are only one round trip behind the head instead of two.
template <typename T, int LPR, int VPL, bool R1>
__global__ void __launch_bounds__(kAggThreads) aggregate_vec(const T* __restrict__ in, T* __restrict__ out,
                                                     const int4* __restrict__ row_head,
                                                     const int32_t* __restrict__ colidx,
                                                     const float* __restrict__ scale, const T* __restrict__ mask,
                                                     const Rank1Args<T> r1, int64_t n, int F_unused, int skip_long,
                                                     int prefetch_blocks, const RowChunks rc) {
  constexpr int VN = Vec<T>::N;
  constexpr int F = LPR * VPL * VN;                  // the row width is fixed by the instantiation: row offsets are shifts
  constexpr int ROWS_PER_BLOCK = kAggThreads / LPR;
  const int sub = threadIdx.x % LPR;
  int64_t row;
  const bool has_row = chunk_row(rc, (int64_t)blockIdx.x * ROWS_PER_BLOCK + threadIdx.x / LPR, n, row);
  // Blocks are dispatched roughly in index order, so the block `prefetch_blocks` further on
  // will run a few microseconds from now: ask for its rows and head records to be brought
  // into L2 (no data returns to the SM, nothing to wait for), so that its first round trip
  // is an L2 hit instead of a DRAM access.
  if (threadIdx.x == 0 && prefetch_blocks > 0 && !rc.row0) {
    const int64_t r0 = ((int64_t)blockIdx.x + prefetch_blocks) * ROWS_PER_BLOCK;
    if (r0 + ROWS_PER_BLOCK <= n) {
      asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(in + r0 * F),
                   "r"((uint32_t)(ROWS_PER_BLOCK * VPL * LPR * 16)) : "memory");
      asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(row_head + r0),
                   "r"((uint32_t)(ROWS_PER_BLOCK * 16)) : "memory");
      // per-row scalars: 4 bytes a row; the instruction wants 16-byte granules
      auto prefetch_words = [&](const void* base) {
        const char* a = static_cast<const char*>(base) + r0 * 4;
        if ((ROWS_PER_BLOCK * 4) % 16 == 0 && ((uintptr_t)a & 15) == 0)
          asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(a), "r"((uint32_t)(ROWS_PER_BLOCK * 4))
                       : "memory");
      };
      if constexpr (R1) {
        prefetch_words(r1.coef);
        prefetch_words(r1.node_part);
      } else if (scale) {
        prefetch_words(scale);
      }
    }
  }
  if (!has_row) return;
  // the row's own features are requested before its CSR extent is known, so the two round
  // trips overlap
  float acc[VPL][VN];
  uint4 own[VPL];
#pragma unroll
  for (int v = 0; v < VPL; ++v) own[v] = Vec<T>::load_raw(in + row * F + (v * LPR + sub) * VN);
  float c_own = 0.0f, s = 1.0f;
  int32_t part = 0;
  if constexpr (R1) {
    c_own = __ldg(r1.coef + row);
    part = __ldg(r1.node_part + row);
  } else if (scale) {
    s = __ldg(scale + row);                          // with the first round trip, not after the last
  }
  const int4 head = __ldg(row_head + row);
  const int32_t deg = head.y;
  if (skip_long && deg > kLongRowDegree) return;   // a whole block takes this row
  {
    uint4 t[2][VPL];
    float c[2] = {0.0f, 0.0f};
    if (deg > 0) {
#pragma unroll
      for (int v = 0; v < VPL; ++v) t[0][v] = Vec<T>::load_raw(in + (int64_t)head.z * F + (v * LPR + sub) * VN);
      if constexpr (R1) c[0] = __ldg(r1.coef + head.z);
    }
    if (deg > 1) {
#pragma unroll
      for (int v = 0; v < VPL; ++v) t[1][v] = Vec<T>::load_raw(in + (int64_t)head.w * F + (v * LPR + sub) * VN);
      if constexpr (R1) c[1] = __ldg(r1.coef + head.w);
    }
#pragma unroll
    for (int v = 0; v < VPL; ++v) {
#pragma unroll
      for (int e = 0; e < VN; ++e) acc[v][e] = 0.0f;
      accumulate<T, R1>(acc[v], own[v], c_own);
    }
    if (deg > 0) {
#pragma unroll
      for (int v = 0; v < VPL; ++v) accumulate<T, R1>(acc[v], t[0][v], c[0]);
    }
    if (deg > 1) {
#pragma unroll
      for (int v = 0; v < VPL; ++v) accumulate<T, R1>(acc[v], t[1][v], c[1]);
    }
  }
  // rank-1 mode: this lane's piece of the subgraph's weight vector, requested while the
  // neighbour rows are still in flight
  uint4 wraw[VPL];
  if constexpr (R1) {
    const T* wv = r1.w + (int64_t)part * r1.w_stride;
#pragma unroll
    for (int v = 0; v < VPL; ++v) wraw[v] = Vec<T>::load_raw(wv + (v * LPR + sub) * VN);
  }
  const int32_t r1_end = head.x + deg;
  int32_t k = head.x + 2;
  constexpr int U = 4;                               // neighbour rows in flight
  if (deg > 2) {                                     // most rows end before this: one test instead of two loop heads
    for (; k + U <= r1_end; k += U) {
      int32_t j[U];
  #pragma unroll
      for (int u = 0; u < U; ++u) j[u] = __ldg(colidx + k + u);
      uint4 t[U][VPL];
      float c[U];
  #pragma unroll
      for (int u = 0; u < U; ++u) {
  #pragma unroll
        for (int v = 0; v < VPL; ++v) t[u][v] = Vec<T>::load_raw(in + (int64_t)j[u] * F + (v * LPR + sub) * VN);
        c[u] = 0.0f;
        if constexpr (R1) c[u] = __ldg(r1.coef + j[u]);
      }
  #pragma unroll
      for (int u = 0; u < U; ++u)
  #pragma unroll
        for (int v = 0; v < VPL; ++v) accumulate<T, R1>(acc[v], t[u][v], c[u]);
    }
    for (; k < r1_end; ++k) {
      const int64_t j = __ldg(colidx + k);
      float c = 0.0f;
      if constexpr (R1) c = __ldg(r1.coef + j);
  #pragma unroll
      for (int v = 0; v < VPL; ++v)
        accumulate<T, R1>(acc[v], Vec<T>::load_raw(in + j * F + (v * LPR + sub) * VN), c);
    }
  }
  if constexpr (R1) {
#pragma unroll
    for (int v = 0; v < VPL; ++v) {
      float wf[VN];
      Vec<T>::unpack(wraw[v], wf);
#pragma unroll
      for (int e = 0; e < VN; ++e) acc[v][e] *= wf[e];
      Vec<T>::store(out + row * F + (v * LPR + sub) * VN, acc[v]);
    }
  } else {
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
}

// Rank-1 mode from mask bits: the pass that reads H just before (the last layer's weight
// gradient) can leave [H > 0] as one bit per element (element f of a row = bit f%8 of byte
// f/8, F/8 bytes a row).  The gather then moves 1/16 (bfloat16) of the bytes of an activation
// row.  Same sums in the same order as the activation-gathering mode.
template <int VN>
__device__ __forceinline__ void add_where_bits(float (&acc)[VN], uint32_t m, float c) {
#pragma unroll
  for (int e = 0; e < VN; ++e) acc[e] += ((m >> e) & 1u) ? c : 0.0f;
}

// The same for a byte of bits, written so that the seven low bits become seven predicates at once
// (the assembler turns tests of the low bits 1, 2, 4 ... 64 of one register into a single
// register-to-predicates move) and every element costs one predicated add.  Measured on B200:
// 10 issue cycles per byte against 21 for the shift-mask-select form above; the batched kernel is
// bound by its integer pipe, so this is what its speed hangs on.
__device__ __forceinline__ void add_where_bits8(float (&acc)[8], uint32_t m, float c) {
  asm("{\n\t.reg .pred p<7>;\n\t.reg .b32 t<7>;\n\t"
      "and.b32 t0, %7, 1;\n\tand.b32 t1, %7, 2;\n\tand.b32 t2, %7, 4;\n\tand.b32 t3, %7, 8;\n\t"
      "and.b32 t4, %7, 16;\n\tand.b32 t5, %7, 32;\n\tand.b32 t6, %7, 64;\n\t"
      "setp.ne.b32 p0, t0, 0;\n\tsetp.ne.b32 p1, t1, 0;\n\tsetp.ne.b32 p2, t2, 0;\n\tsetp.ne.b32 p3, t3, 0;\n\t"
      "setp.ne.b32 p4, t4, 0;\n\tsetp.ne.b32 p5, t5, 0;\n\tsetp.ne.b32 p6, t6, 0;\n\t"
      "@p0 add.f32 %0, %0, %8;\n\t@p1 add.f32 %1, %1, %8;\n\t@p2 add.f32 %2, %2, %8;\n\t@p3 add.f32 %3, %3, %8;\n\t"
      "@p4 add.f32 %4, %4, %8;\n\t@p5 add.f32 %5, %5, %8;\n\t@p6 add.f32 %6, %6, %8;\n\t}"
      : "+f"(acc[0]), "+f"(acc[1]), "+f"(acc[2]), "+f"(acc[3]), "+f"(acc[4]), "+f"(acc[5]), "+f"(acc[6])
      : "r"(m), "f"(c));
  acc[7] += (m & 128u) ? c : 0.0f;
}

template <typename T, int LPR, int VPL>
__global__ void __launch_bounds__(256) aggregate_rank1_bits(const uint8_t* __restrict__ bits, T* __restrict__ out,
                                                            const int4* __restrict__ row_head,
                                                            const int32_t* __restrict__ colidx,
                                                            const Rank1Args<T> r1, int64_t n, int F,
                                                            int prefetch_blocks, const RowChunks rc) {
  constexpr int VN = Vec<T>::N;
  constexpr int ROWS_PER_BLOCK = 256 / LPR;
  constexpr uint32_t PIECE = (1u << VN) - 1u;
  const int sub = threadIdx.x % LPR;
  int64_t row;
  const bool has_row = chunk_row(rc, (int64_t)blockIdx.x * ROWS_PER_BLOCK + threadIdx.x / LPR, n, row);
  const int64_t rb = F >> 3;                                   // bytes of bits per row
  if (threadIdx.x == 0 && prefetch_blocks > 0 && !rc.row0) {   // see aggregate_vec
    const int64_t r0 = ((int64_t)blockIdx.x + prefetch_blocks) * ROWS_PER_BLOCK;
    if (r0 + ROWS_PER_BLOCK <= n) {
      asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(row_head + r0),
                   "r"((uint32_t)(ROWS_PER_BLOCK * 16)) : "memory");
      const uint8_t* b0 = bits + r0 * rb;
      const uint32_t nb = (uint32_t)(ROWS_PER_BLOCK * rb);
      if ((nb & 15u) == 0 && ((uintptr_t)b0 & 15) == 0)
        asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(b0), "r"(nb) : "memory");
    }
  }
  if (!has_row) return;
  // piece v of this lane: elements (v*LPR + sub)*VN .. +VN  ->  VN bits inside one byte
  int byte_of[VPL], shift_of[VPL];
#pragma unroll
  for (int v = 0; v < VPL; ++v) {
    const int off = (v * LPR + sub) * VN;
    byte_of[v] = off >> 3;
    shift_of[v] = off & 7;
  }
  uint32_t own[VPL];
#pragma unroll
  for (int v = 0; v < VPL; ++v) own[v] = __ldg(bits + row * rb + byte_of[v]);
  const float c_own = __ldg(r1.coef + row);
  const int32_t part = __ldg(r1.node_part + row);
  const int4 head = __ldg(row_head + row);
  const int32_t deg = head.y;
  float acc[VPL][VN];
  {
    uint32_t t[2][VPL];
    float c[2] = {0.0f, 0.0f};
    if (deg > 0) {
#pragma unroll
      for (int v = 0; v < VPL; ++v) t[0][v] = __ldg(bits + (int64_t)head.z * rb + byte_of[v]);
      c[0] = __ldg(r1.coef + head.z);
    }
    if (deg > 1) {
#pragma unroll
      for (int v = 0; v < VPL; ++v) t[1][v] = __ldg(bits + (int64_t)head.w * rb + byte_of[v]);
      c[1] = __ldg(r1.coef + head.w);
    }
#pragma unroll
    for (int v = 0; v < VPL; ++v) {
#pragma unroll
      for (int e = 0; e < VN; ++e) acc[v][e] = 0.0f;
      add_where_bits<VN>(acc[v], (own[v] >> shift_of[v]) & PIECE, c_own);
    }
    if (deg > 0) {
#pragma unroll
      for (int v = 0; v < VPL; ++v) add_where_bits<VN>(acc[v], (t[0][v] >> shift_of[v]) & PIECE, c[0]);
    }
    if (deg > 1) {
#pragma unroll
      for (int v = 0; v < VPL; ++v) add_where_bits<VN>(acc[v], (t[1][v] >> shift_of[v]) & PIECE, c[1]);
    }
  }
  // this lane's piece of the subgraph's weight vector, requested while the rest of the row is walked
  uint4 wraw[VPL];
  {
    const T* wv = r1.w + (int64_t)part * r1.w_stride;
#pragma unroll
    for (int v = 0; v < VPL; ++v) wraw[v] = Vec<T>::load_raw(wv + (v * LPR + sub) * VN);
  }
  const int32_t r_end = head.x + deg;
  int32_t k = head.x + 2;
  constexpr int U = 8;                                         // neighbour rows in flight
  for (; k + U <= r_end; k += U) {
    int32_t j[U];
#pragma unroll
    for (int u = 0; u < U; ++u) j[u] = __ldg(colidx + k + u);
    uint32_t t[U][VPL];
    float c[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
#pragma unroll
      for (int v = 0; v < VPL; ++v) t[u][v] = __ldg(bits + (int64_t)j[u] * rb + byte_of[v]);
      c[u] = __ldg(r1.coef + j[u]);
    }
#pragma unroll
    for (int u = 0; u < U; ++u)
#pragma unroll
      for (int v = 0; v < VPL; ++v) add_where_bits<VN>(acc[v], (t[u][v] >> shift_of[v]) & PIECE, c[u]);
  }
  for (; k < r_end; ++k) {
    const int64_t j = __ldg(colidx + k);
    const float cj = __ldg(r1.coef + j);
#pragma unroll
    for (int v = 0; v < VPL; ++v)
      add_where_bits<VN>(acc[v], ((uint32_t)__ldg(bits + j * rb + byte_of[v]) >> shift_of[v]) & PIECE, cj);
  }
#pragma unroll
  for (int v = 0; v < VPL; ++v) {
    float wf[VN];
    Vec<T>::unpack(wraw[v], wf);
#pragma unroll
    for (int e = 0; e < VN; ++e) acc[v][e] *= wf[e];
    Vec<T>::store(out + row * F + (v * LPR + sub) * VN, acc[v]);
  }
}

// Rank-1 mode from mask bits, rows in batches (row widths of 256 and 512 elements: NB = 32 or 64
// bytes of bits a row).  The kernel above gives every row a warp that walks head record ->
// neighbour bits -> store as a chain of dependent round trips; with 64 warps on an SM only 64 rows
// are in flight and the pass is bound by that chain, not by its bytes.  Here a warp owns 32
// consecutive rows and works in two phases:
//   gather   lane = row: head record, coefficient, subgraph id and the row's own bits in one round
//            trip (the bits of 32 consecutive rows are one contiguous kilobyte), the bits and
//            coefficients of the first two neighbours (named by the head record) in a second one;
//            everything is parked in shared memory.  32 rows per warp are in flight.
//   reduce   lane = 8 (or 16) features: row after row, the parked bits are expanded, neighbours
//            beyond the second are fetched 32 at a time (lane = neighbour, parked the same way)
//            and added in CSR order, the sum is scaled by the subgraph's weight vector and stored
//            as one 512-byte (1 KB) line per row.
// Sums are taken in the same order as in the kernel above, so the results are bit-identical.
// Rows with more than kLongRowDegree neighbours are left to the block-per-segment kernels (which gather
// the activation itself): hubs are neighbours in the node order, and a warp that met a run of them
// would walk tens of thousands of neighbours on its own while the rest of the GPU idles.
template <int NB>
__global__ void __launch_bounds__(256) aggregate_rank1_bits_batch(const uint8_t* __restrict__ bits,
                                                                  __nv_bfloat16* __restrict__ out,
                                                                  const int4* __restrict__ row_head,
                                                                  const int32_t* __restrict__ colidx,
                                                                  const Rank1Args<__nv_bfloat16> r1, int64_t n,
                                                                  int skip_long, int prefetch_blocks,
                                                                  const RowChunks rc) {
  using T = __nv_bfloat16;
  constexpr int F = NB * 8, VPL = NB / 32, Q = NB / 16;
  constexpr int kWarpBytes = 4 * 32 * NB + 7 * 32 * 4;       // own + two neighbours + tail bits, 7 words of per-row scalars
  extern __shared__ uint4 smem_r1b[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0 && prefetch_blocks > 0 && !rc.row0) {   // see aggregate_vec
    const int64_t r0 = ((int64_t)blockIdx.x + prefetch_blocks) * 256;
    if (r0 + 256 <= n) {
      asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(row_head + r0), "r"(256u * 16u) : "memory");
      const uint8_t* b0 = bits + r0 * NB;
      if (((uintptr_t)b0 & 15) == 0)
        asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(b0), "r"(256u * (uint32_t)NB) : "memory");
      if ((((uintptr_t)(r1.coef + r0)) & 15) == 0)
        asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(r1.coef + r0), "r"(1024u) : "memory");
      if ((((uintptr_t)(r1.node_part + r0)) & 15) == 0)
        asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(r1.node_part + r0), "r"(1024u) : "memory");
    }
  }
  // the warp's 32 consecutive rows: of the whole graph, or of one 256-row chunk of an active subgraph
  int64_t row0 = (int64_t)blockIdx.x * 256 + warp * 32, row_end = n;
  if (rc.row0) {
    row0 = (int64_t)rc.row0[blockIdx.x] + warp * 32;
    row_end = (int64_t)rc.row0[blockIdx.x] + rc.rows[blockIdx.x];
  }
  if (row0 >= row_end) return;                                 // whole warp; no block-wide barrier below
  uint8_t* wbase = reinterpret_cast<uint8_t*>(smem_r1b) + warp * kWarpBytes;
  uint8_t* sb = wbase;                                         // [3][32 rows][NB]: own, first, second neighbour
  uint8_t* tb = wbase + 3 * 32 * NB;                           // [32 neighbours][NB]
  float* sc = reinterpret_cast<float*>(wbase + 4 * 32 * NB);   // [3][32] coefficients
  int32_t* sdeg = reinterpret_cast<int32_t*>(sc + 96);
  int32_t* sfirst = sdeg + 32;
  int32_t* spart = sfirst + 32;
  float* tcf = reinterpret_cast<float*>(spart + 32);           // [32] coefficients of the parked neighbours
  // ---- gather, lane = row
  {
    const int64_t row = row0 + lane;
    const bool valid = row < row_end;
    int4 head = make_int4(0, 0, 0, 0);
    float c_own = 0.0f, c0 = 0.0f, c1 = 0.0f;
    int32_t part = 0;
    uint4 own[Q], b0[Q], b1[Q];
#pragma unroll
    for (int q = 0; q < Q; ++q) own[q] = b0[q] = b1[q] = make_uint4(0u, 0u, 0u, 0u);
    if (valid) {
      head = __ldg(row_head + row);
      c_own = __ldg(r1.coef + row);
      part = __ldg(r1.node_part + row);
#pragma unroll
      for (int q = 0; q < Q; ++q) own[q] = __ldg(reinterpret_cast<const uint4*>(bits + row * NB) + q);
      if (head.y > 0) {
#pragma unroll
        for (int q = 0; q < Q; ++q) b0[q] = __ldg(reinterpret_cast<const uint4*>(bits + (int64_t)head.z * NB) + q);
        c0 = __ldg(r1.coef + head.z);
      }
      if (head.y > 1) {
#pragma unroll
        for (int q = 0; q < Q; ++q) b1[q] = __ldg(reinterpret_cast<const uint4*>(bits + (int64_t)head.w * NB) + q);
        c1 = __ldg(r1.coef + head.w);
      }
    }
#pragma unroll
    for (int q = 0; q < Q; ++q) {
      reinterpret_cast<uint4*>(sb + (0 * 32 + lane) * NB)[q] = own[q];
      reinterpret_cast<uint4*>(sb + (1 * 32 + lane) * NB)[q] = b0[q];
      reinterpret_cast<uint4*>(sb + (2 * 32 + lane) * NB)[q] = b1[q];
    }
    sc[lane] = c_own; sc[32 + lane] = c0; sc[64 + lane] = c1;
    sdeg[lane] = head.y; sfirst[lane] = head.x; spart[lane] = part;
  }
  __syncwarp();
  // ---- reduce, lane = VPL pieces of 8 features
  const int rows_here = (int)min((int64_t)32, row_end - row0);
  int cur_part = -1;
  float wf[VPL][8];                                            // this lane's pieces of the subgraph's weight vector
  for (int r = 0; r < rows_here; ++r) {
    const int deg = sdeg[r];
    if (skip_long && deg > kLongRowDegree) continue;           // a block (or one per segment) takes this row
    float acc[VPL][8];
#pragma unroll
    for (int v = 0; v < VPL; ++v) {
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[v][e] = 0.0f;
      add_where_bits8(acc[v], sb[(0 * 32 + r) * NB + v * 32 + lane], sc[r]);
    }
    if (deg > 0) {
#pragma unroll
      for (int v = 0; v < VPL; ++v) add_where_bits8(acc[v], sb[(1 * 32 + r) * NB + v * 32 + lane], sc[32 + r]);
    }
    if (deg > 1) {
#pragma unroll
      for (int v = 0; v < VPL; ++v) add_where_bits8(acc[v], sb[(2 * 32 + r) * NB + v * 32 + lane], sc[64 + r]);
    }
    if (deg > 2) {
      const int32_t r_end = sfirst[r] + deg;
      for (int32_t k0 = sfirst[r] + 2; k0 < r_end; k0 += 32) {
        const int32_t k = k0 + lane;
        uint4 tbits[Q];
        float cj = 0.0f;
#pragma unroll
        for (int q = 0; q < Q; ++q) tbits[q] = make_uint4(0u, 0u, 0u, 0u);
        if (k < r_end) {
          const int64_t j = __ldg(colidx + k);
          cj = __ldg(r1.coef + j);
#pragma unroll
          for (int q = 0; q < Q; ++q) tbits[q] = __ldg(reinterpret_cast<const uint4*>(bits + j * NB) + q);
        }
        __syncwarp();                                          // readers of the previous 32 are done
#pragma unroll
        for (int q = 0; q < Q; ++q) reinterpret_cast<uint4*>(tb + lane * NB)[q] = tbits[q];
        tcf[lane] = cj;
        __syncwarp();
        const int cnt = min(32, r_end - k0);
        for (int t = 0; t < cnt; ++t) {
          const float c = tcf[t];
#pragma unroll
          for (int v = 0; v < VPL; ++v) add_where_bits8(acc[v], tb[t * NB + v * 32 + lane], c);
        }
      }
    }
    const int part = spart[r];
    if (part != cur_part) {                                    // uniform across the warp
      cur_part = part;
      const T* wv = r1.w + (int64_t)part * r1.w_stride;
#pragma unroll
      for (int v = 0; v < VPL; ++v) Vec<T>::load(wv + (v * 32 + lane) * 8, wf[v]);
    }
#pragma unroll
    for (int v = 0; v < VPL; ++v) {
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[v][e] *= wf[v][e];
      Vec<T>::store(out + (row0 + r) * F + (v * 32 + lane) * 8, acc[v]);
    }
  }
}

// A row with more than kLongRowDegree neighbours: one block per row.  Each of the 8 warps sums
// a contiguous eighth of the neighbour list with eight rows in flight, the partial sums
// meet in shared memory in warp order (deterministic), and the block finishes the row.
// With a segment table (seg_out != nullptr) a block instead sums ONE SEGMENT of a long row's
// neighbour list (at most kLongRowSegment entries) into seg_out[segment][F], float32, and
// aggregate_long_finish adds a row's segments up in order: a hub of tens of thousands of
// neighbours then occupies a dozen blocks for a moment instead of one block for a millisecond.
template <typename T, int LPR, int VPL, bool R1>
__global__ void __launch_bounds__(256) aggregate_long_row(const T* __restrict__ in, T* __restrict__ out,
                                                          const int32_t* __restrict__ rowptr,
                                                          const int32_t* __restrict__ colidx,
                                                          const float* __restrict__ scale,
                                                          const T* __restrict__ mask, const Rank1Args<T> r1,
                                                          const int32_t* __restrict__ long_rows, int F,
                                                          const int32_t* __restrict__ seg_begin,
                                                          const int32_t* __restrict__ seg_end,
                                                          float* __restrict__ seg_out) {
  constexpr int VN = Vec<T>::N;
  constexpr int GROUPS = 256 / LPR;               // lane groups, each walks its own slice of the row
  extern __shared__ float partial[];              // [GROUPS][F]
  const int64_t row = seg_out ? 0 : long_rows[blockIdx.x];
  const int sub = threadIdx.x % LPR, grp = threadIdx.x / LPR;
  const int32_t r0 = seg_out ? seg_begin[blockIdx.x] : rowptr[row];
  const int32_t r1_end = seg_out ? seg_end[blockIdx.x] : rowptr[row + 1];
  const int32_t len = (r1_end - r0 + GROUPS - 1) / GROUPS;
  const int32_t a = r0 + grp * len, b = min(r1_end, a + len);
  float acc[VPL][VN];
#pragma unroll
  for (int v = 0; v < VPL; ++v)
#pragma unroll
    for (int e = 0; e < VN; ++e) acc[v][e] = 0.0f;
  for (int32_t k = a; k < b; k += 8) {
    uint4 t[8][VPL];
    float c[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      c[u] = 0.0f;
      if (k + u < b) {
        const int64_t col = __ldg(colidx + k + u);
#pragma unroll
        for (int v = 0; v < VPL; ++v) t[u][v] = Vec<T>::load_raw(in + col * F + (v * LPR + sub) * VN);
        if constexpr (R1) c[u] = __ldg(r1.coef + col);
      }
    }
#pragma unroll
    for (int u = 0; u < 8; ++u)
      if (k + u < b) {
#pragma unroll
        for (int v = 0; v < VPL; ++v) accumulate<T, R1>(acc[v], t[u][v], c[u]);
      }
  }
#pragma unroll
  for (int v = 0; v < VPL; ++v)
#pragma unroll
    for (int e = 0; e < VN; ++e) partial[grp * F + (v * LPR + sub) * VN + e] = acc[v][e];
  __syncthreads();
  if (seg_out) {
    for (int f = threadIdx.x; f < F; f += 256) {
      float tot = 0.0f;
      for (int g = 0; g < GROUPS; ++g) tot += partial[g * F + f];
      seg_out[(int64_t)blockIdx.x * F + f] = tot;
    }
    return;
  }
  if constexpr (R1) {
    const float ci = r1.coef[row];
    const T* wv = r1.w + (int64_t)r1.node_part[row] * r1.w_stride;
    for (int f = threadIdx.x; f < F; f += 256) {
      float tot = to_f32(in[row * F + f]) > 0.0f ? ci : 0.0f;
      for (int g = 0; g < GROUPS; ++g) tot += partial[g * F + f];
      from_f32(out[row * F + f], tot * to_f32(wv[f]));
    }
  } else {
    const float sc = scale ? scale[row] : 1.0f;
    for (int f = threadIdx.x; f < F; f += 256) {
      float tot = to_f32(in[row * F + f]);
      for (int g = 0; g < GROUPS; ++g) tot += partial[g * F + f];
      tot *= sc;
      if (mask && !(to_f32(mask[row * F + f]) > 0.0f)) tot = 0.0f;
      from_f32(out[row * F + f], tot);
    }
  }
}

// Second half of the segmented long rows: one block per long row adds the row's own features
// and its segments' partial sums (in segment order) and applies the epilogue of the mode.
template <typename T, bool R1>
__global__ void __launch_bounds__(256) aggregate_long_finish(const T* __restrict__ in, T* __restrict__ out,
                                                             const float* __restrict__ scale,
                                                             const T* __restrict__ mask, const Rank1Args<T> r1,
                                                             const int32_t* __restrict__ long_rows,
                                                             const int32_t* __restrict__ long_first_seg,
                                                             const float* __restrict__ seg_part, int F) {
  const int64_t row = long_rows[blockIdx.x];
  const int32_t s0 = long_first_seg[blockIdx.x], s1 = long_first_seg[blockIdx.x + 1];
  for (int f = threadIdx.x; f < F; f += 256) {
    float tot;
    if constexpr (R1) tot = to_f32(in[row * F + f]) > 0.0f ? r1.coef[row] : 0.0f;
    else tot = to_f32(in[row * F + f]);
    for (int32_t sg = s0; sg < s1; ++sg) tot += seg_part[(int64_t)sg * F + f];
    if constexpr (R1) {
      tot *= to_f32(r1.w[(int64_t)r1.node_part[row] * r1.w_stride + f]);
    } else {
      tot *= scale ? scale[row] : 1.0f;
      if (mask && !(to_f32(mask[row * F + f]) > 0.0f)) tot = 0.0f;
    }
    from_f32(out[row * F + f], tot);
  }
}

// Any width: one warp per row, lanes stride over the features with scalar accesses.
template <typename T, bool R1>
__global__ void __launch_bounds__(256) aggregate_any(const T* __restrict__ in, T* __restrict__ out,
                                                     const int32_t* __restrict__ rowptr,
                                                     const int32_t* __restrict__ colidx,
                                                     const float* __restrict__ scale, const T* __restrict__ mask,
                                                     const Rank1Args<T> r1, int64_t n, int F, const RowChunks rc) {
  const int lane = threadIdx.x & 31;
  int64_t row;
  if (!chunk_row(rc, (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5), n, row)) return;
  const int32_t r0 = rowptr[row], r1_end = rowptr[row + 1];
  if constexpr (R1) {
    const float ci = r1.coef[row];
    const T* wv = r1.w + (int64_t)r1.node_part[row] * r1.w_stride;
    for (int f = lane; f < F; f += 32) {
      float acc = to_f32(in[row * F + f]) > 0.0f ? ci : 0.0f;
      for (int32_t k = r0; k < r1_end; ++k) {
        const int64_t j = colidx[k];
        acc += to_f32(in[j * F + f]) > 0.0f ? r1.coef[j] : 0.0f;
      }
      from_f32(out[row * F + f], acc * to_f32(wv[f]));
    }
  } else {
    const float s = scale ? scale[row] : 1.0f;
    for (int f = lane; f < F; f += 32) {
      float acc = to_f32(in[row * F + f]);
      for (int32_t k = r0; k < r1_end; ++k) acc += to_f32(in[(int64_t)colidx[k] * F + f]);
      acc *= s;
      if (mask && !(to_f32(mask[row * F + f]) > 0.0f)) acc = 0.0f;
      from_f32(out[row * F + f], acc);
    }
  }
}

// The rows with more than kLongRowDegree neighbours, one block per row (or per segment of a row when the
// step has scratch for the partial sums), on the handle's side stream so that they run beside the kernel
// that the caller launches next on `st`.  Returns whether the side stream was used; the caller then
// makes `st` wait for ev_join.
template <typename T, int LPR, int VPL, bool R1>
bool fork_long_rows(gnnco_handle* h, const T* in, T* out, const float* scale, const T* mask, const Rank1Args<T>& r1,
                    int F, cudaStream_t st) {
  const size_t long_smem = (size_t)(256 / LPR) * F * sizeof(float);
  const bool fork = h->side_stream && h->ev_fork && h->ev_join && cudaEventRecord(h->ev_fork, st) == cudaSuccess &&
                    cudaStreamWaitEvent(h->side_stream, h->ev_fork, 0) == cudaSuccess;
  cudaStream_t ls = fork ? h->side_stream : st;
  if (h->agg_partial && h->n_long_segs > 0) {
    // long rows cut into segments: partial sums by one block per segment, then one block per row
    aggregate_long_row<T, LPR, VPL, R1><<<h->n_long_segs, 256, long_smem, ls>>>(
        in, out, h->rowptr, h->colidx, scale, mask, r1, h->long_rows, F, h->seg_begin, h->seg_end, h->agg_partial);
    aggregate_long_finish<T, R1><<<h->n_long, 256, 0, ls>>>(in, out, scale, mask, r1, h->long_rows, h->long_first_seg,
                                                            h->agg_partial, F);
    h->launches += 2;
  } else {
    aggregate_long_row<T, LPR, VPL, R1><<<h->n_long, 256, long_smem, ls>>>(in, out, h->rowptr, h->colidx, scale, mask,
                                                                            r1, h->long_rows, F, nullptr, nullptr, nullptr);
    h->launches += 1;
  }
  if (fork) cudaEventRecord(h->ev_join, h->side_stream);
  return fork;
}

template <typename T, int LPR, int VPL, bool R1>
void launch_vec(const T* in, T* out, gnnco_handle* h, const float* scale, const T* mask, const Rank1Args<T>& r1, int F,
                cudaStream_t st) {
  constexpr int ROWS_PER_BLOCK = kAggThreads / LPR;
  const unsigned main_blocks = (unsigned)((linear_rows(h) + ROWS_PER_BLOCK - 1) / ROWS_PER_BLOCK);
  // L2 prefetch distance: one full wave of resident blocks ahead; pointless on small grids
  const int sms = h->sm_count > 0 ? h->sm_count : 148;
  constexpr int kWave = 2048 / kAggThreads;               // resident blocks per SM
  const int pf_blocks = main_blocks > 4u * kWave * (unsigned)sms ? kWave * sms : 0;
  if (h->n_long == 0) {
    aggregate_vec<T, LPR, VPL, R1><<<main_blocks, kAggThreads, 0, st>>>(in, out, h->row_head, h->colidx, scale, mask, r1, h->n,
                                                                F, 0, pf_blocks, h->row_chunks);
    return;
  }
  // A single warp walks a row of max_row entries in about max_row/4 dependent round trips of
  // roughly a microsecond.  When streaming all rows takes several times longer than that, the
  // long rows stay where they are (scattered through the grid, each a lightweight warp that
  // overlaps with the streaming of its neighbours); otherwise (small or hub-dominated graphs,
  // where one such walk would be the tail of the kernel) they get a block each, on a side
  // stream, beside the short rows.
  const double stream_us = 2.0 * (double)linear_rows(h) * F * sizeof(T) / 4.0e6;   // at ~4 TB/s
  const double walk_us = (double)h->max_row / 4.0;
  const bool inline_first = stream_us > 3.0 * walk_us;
  if (inline_first) {
    aggregate_vec<T, LPR, VPL, R1><<<main_blocks, kAggThreads, 0, st>>>(in, out, h->row_head, h->colidx, scale, mask, r1, h->n,
                                                                F, 0, pf_blocks, h->row_chunks);
    return;
  }
  const bool fork = fork_long_rows<T, LPR, VPL, R1>(h, in, out, scale, mask, r1, F, st);
  aggregate_vec<T, LPR, VPL, R1><<<main_blocks, kAggThreads, 0, st>>>(in, out, h->row_head, h->colidx, scale, mask, r1, h->n, F,
                                                              1, pf_blocks, h->row_chunks);
  if (fork) cudaStreamWaitEvent(st, h->ev_join, 0);
}

template <typename T, bool R1>
int32_t aggregate_typed(gnnco_handle* h, const T* in, T* out, int F, const float* scale, const T* mask,
                        const Rank1Args<T>& r1, cudaStream_t st) {
  constexpr int VN = Vec<T>::N;
  bool aligned = !((uintptr_t)in & 15) && !((uintptr_t)out & 15) && !((uintptr_t)mask & 15);
  if (R1) aligned = aligned && !((uintptr_t)r1.w & 15) && (r1.w_stride % VN == 0);
  int vecs = F / VN;
  bool done = false;
  if (aligned && F % VN == 0) {
    done = true;
    switch (vecs) {
      case 1: launch_vec<T, 1, 1, R1>(in, out, h, scale, mask, r1, F, st); break;
      case 2: launch_vec<T, 2, 1, R1>(in, out, h, scale, mask, r1, F, st); break;
      case 4: launch_vec<T, 4, 1, R1>(in, out, h, scale, mask, r1, F, st); break;
      case 8: launch_vec<T, 8, 1, R1>(in, out, h, scale, mask, r1, F, st); break;
      case 16: launch_vec<T, 16, 1, R1>(in, out, h, scale, mask, r1, F, st); break;
      case 32: launch_vec<T, 32, 1, R1>(in, out, h, scale, mask, r1, F, st); break;
      case 64: launch_vec<T, 32, 2, R1>(in, out, h, scale, mask, r1, F, st); break;
      default: done = false;
    }
  }
  if (!done) {
    unsigned grid = (unsigned)((linear_rows(h) + 7) / 8);
    aggregate_any<T, R1><<<grid, 256, 0, st>>>(in, out, h->rowptr, h->colidx, scale, mask, r1, h->n, F, h->row_chunks);
  }
  h->launches += 1;
  GNNCO_LAUNCH_CHECK();
  return GNNCO_OK;
}

}  // namespace

int32_t launch_aggregate(gnnco_handle* h, int dtype, const void* in, void* out, int F, const float* row_scale,
                         const void* relu_mask, cudaStream_t st) {
  if (h->n == 0) return GNNCO_OK;
  ProfScope prof_(h, row_scale ? K_AGG_FWD : K_AGG_BWD, st);
  if (dtype == GNNCO_F32)
    return aggregate_typed<float, false>(h, (const float*)in, (float*)out, F, row_scale, (const float*)relu_mask,
                                         Rank1Args<float>{}, st);
  if (dtype == GNNCO_BF16)
    return aggregate_typed<__nv_bfloat16, false>(h, (const __nv_bfloat16*)in, (__nv_bfloat16*)out, F, row_scale,
                                                 (const __nv_bfloat16*)relu_mask, Rank1Args<__nv_bfloat16>{}, st);
  return GNNCO_UNSUPPORTED;
}

int32_t launch_aggregate_rank1(gnnco_handle* h, int dtype, const void* H, const float* coef, const void* w,
                               int64_t w_stride, void* out, int F, cudaStream_t st) {
  if (h->n == 0) return GNNCO_OK;
  ProfScope prof_(h, K_AGG_RANK1, st);
  if (dtype == GNNCO_F32)
    return aggregate_typed<float, true>(h, (const float*)H, (float*)out, F, nullptr, nullptr,
                                        Rank1Args<float>{coef, (const float*)w, w_stride, h->node_part}, st);
  if (dtype == GNNCO_BF16)
    return aggregate_typed<__nv_bfloat16, true>(
        h, (const __nv_bfloat16*)H, (__nv_bfloat16*)out, F, nullptr, nullptr,
        Rank1Args<__nv_bfloat16>{coef, (const __nv_bfloat16*)w, w_stride, h->node_part}, st);
  return GNNCO_UNSUPPORTED;
}

namespace {

// The bit-gathering kernel walks every row inline, so it is used where the plain kernel would
// do the same (no separate pass for long rows).
bool rows_stay_inline(const gnnco_handle* h, int F, size_t elem) {
  if (h->n_long == 0) return true;
  const double stream_us = 2.0 * (double)h->n * F * elem / 4.0e6;
  const double walk_us = (double)h->max_row / 4.0;
  return stream_us > 3.0 * walk_us;
}

template <typename T>
int32_t rank1_bits_typed(gnnco_handle* h, const uint8_t* bits, const T* H, T* out, int F, const Rank1Args<T>& r1,
                         cudaStream_t st) {
  constexpr int VN = Vec<T>::N;
  const int sms = h->sm_count > 0 ? h->sm_count : 148;
#define GNNCO_R1B(LPR, VPL)                                                                                      \
  do {                                                                                                           \
    const unsigned blocks = (unsigned)((linear_rows(h) + (256 / LPR) - 1) / (256 / LPR));                        \
    const int pf = blocks > 4u * 8u * (unsigned)sms ? 8 * sms : 0;                                               \
    aggregate_rank1_bits<T, LPR, VPL><<<blocks, 256, 0, st>>>(bits, out, h->row_head, h->colidx, r1, h->n, F, pf, \
                                                              h->row_chunks);                                    \
  } while (0)
  if (F == 256 || F == 512) {
    // rows in batches of 32 per warp (see aggregate_rank1_bits_batch); long rows beside them
    const unsigned blocks = (unsigned)((linear_rows(h) + 255) / 256);
    const int pf = blocks > 4u * 5u * (unsigned)sms ? 5 * sms : 0;      // one wave of resident blocks ahead
    const int skip = h->n_long > 0 ? 1 : 0;
    bool fork = false;
    if (F == 256) {
      constexpr int smem = 8 * (4 * 32 * 32 + 7 * 32 * 4);
      if (skip) fork = fork_long_rows<T, 32, 1, true>(h, H, out, nullptr, nullptr, r1, F, st);
      aggregate_rank1_bits_batch<32><<<blocks, 256, smem, st>>>(bits, out, h->row_head, h->colidx, r1, h->n, skip, pf,
                                                                h->row_chunks);
    } else {
      constexpr int smem = 8 * (4 * 32 * 64 + 7 * 32 * 4);
      GNNCO_CUDA_TRY(cudaFuncSetAttribute(aggregate_rank1_bits_batch<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
      if (skip) fork = fork_long_rows<T, 32, 2, true>(h, H, out, nullptr, nullptr, r1, F, st);
      aggregate_rank1_bits_batch<64><<<blocks, 256, smem, st>>>(bits, out, h->row_head, h->colidx, r1, h->n, skip, pf,
                                                                h->row_chunks);
    }
    if (fork) cudaStreamWaitEvent(st, h->ev_join, 0);
    h->launches += 1;
    GNNCO_LAUNCH_CHECK();
    return GNNCO_OK;
  }
  switch (F / VN) {
    case 1: GNNCO_R1B(1, 1); break;
    case 2: GNNCO_R1B(2, 1); break;
    case 4: GNNCO_R1B(4, 1); break;
    case 8: GNNCO_R1B(8, 1); break;
    case 16: GNNCO_R1B(16, 1); break;
    case 32: GNNCO_R1B(32, 1); break;
    case 64: GNNCO_R1B(32, 2); break;
    default: return GNNCO_UNSUPPORTED;
  }
#undef GNNCO_R1B
  h->launches += 1;
  GNNCO_LAUNCH_CHECK();
  return GNNCO_OK;
}

}  // namespace

bool aggregate_rank1_bits_supported(const gnnco_handle* h, int dtype, int F) {
  if (dtype != GNNCO_BF16) return false;
  if (F % 8) return false;
  const int vecs = F / 8;
  if (!(vecs == 1 || vecs == 2 || vecs == 4 || vecs == 8 || vecs == 16 || vecs == 32 || vecs == 64)) return false;
  if (F == 256 || F == 512) return true;          // the batched kernel hands its long rows to a block each
  return rows_stay_inline(h, F, 2);
}

int32_t launch_aggregate_rank1_bits(gnnco_handle* h, int dtype, const uint8_t* bits, const void* H, const float* coef,
                                    const void* w, int64_t w_stride, void* out, int F, cudaStream_t st) {
  if (!aggregate_rank1_bits_supported(h, dtype, F)) return GNNCO_UNSUPPORTED;
  if (((uintptr_t)out & 15) || ((uintptr_t)w & 15) || (w_stride % 8) || ((uintptr_t)bits & 15) || ((uintptr_t)H & 15))
    return GNNCO_UNSUPPORTED;
  ProfScope prof_(h, K_AGG_RANK1, st);
  return rank1_bits_typed<__nv_bfloat16>(
      h, bits, (const __nv_bfloat16*)H, (__nv_bfloat16*)out, F,
      Rank1Args<__nv_bfloat16>{coef, (const __nv_bfloat16*)w, w_stride, h->node_part}, st);
}
