// gnnco_partition_load: integer bookkeeping that turns (graph, partition) into the
// block-diagonal batch -- new node ids ranked by (part, id), symmetric CSR of the intra
// edges, sorted list of boundary edges (Section 3.3: subgraphs are trained on their own
// edges, cross edges are kept for conflict detection).
//
// Everything is built from three device primitives written here: an exclusive scan, a
// stable least-significant-digit radix sort of 64-bit keys, and "segment starts of a
// sorted key array".  Slot allocation for the two edge classes uses integer atomics, but
// both lists are sorted afterwards, so every output is uniquely defined.
#include <algorithm>
#include <new>

#include "internal.cuh"

namespace {

// ------------------------------------------------------------------ exclusive scan
constexpr int kScanThreads = 256;
constexpr int kScanPerThread = 8;
constexpr int kScanTile = kScanThreads * kScanPerThread;

__global__ void scan_tiles(int32_t* data, int64_t N, int32_t* tile_sums) {
  __shared__ int32_t warp_tot[kScanThreads / 32];
  int64_t base = (int64_t)blockIdx.x * kScanTile + (int64_t)threadIdx.x * kScanPerThread;
  int32_t v[kScanPerThread];
  int32_t sum = 0;
#pragma unroll
  for (int k = 0; k < kScanPerThread; ++k) {
    v[k] = (base + k < N) ? data[base + k] : 0;
    sum += v[k];
  }
  int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int32_t incl = sum;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    int32_t o = __shfl_up_sync(0xffffffffu, incl, d);
    if (lane >= d) incl += o;
  }
  if (lane == 31) warp_tot[warp] = incl;
  __syncthreads();
  int32_t warp_off = 0, total = 0;
#pragma unroll
  for (int w = 0; w < kScanThreads / 32; ++w) {
    if (w < warp) warp_off += warp_tot[w];
    total += warp_tot[w];
  }
  int32_t run = warp_off + incl - sum;
#pragma unroll
  for (int k = 0; k < kScanPerThread; ++k) {
    if (base + k < N) data[base + k] = run;
    run += v[k];
  }
  if (threadIdx.x == 0) tile_sums[blockIdx.x] = total;
}

__global__ void scan_tile_sums(int32_t* sums, int32_t count) {
  // one block; walks the array in chunks of blockDim.x, carrying the running total
  __shared__ int32_t warp_tot[32];
  __shared__ int32_t carry_s;
  if (threadIdx.x == 0) carry_s = 0;
  __syncthreads();
  int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
  for (int32_t start = 0; start < count; start += blockDim.x) {
    int32_t i = start + threadIdx.x;
    int32_t x = i < count ? sums[i] : 0;
    int32_t incl = x;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      int32_t o = __shfl_up_sync(0xffffffffu, incl, d);
      if (lane >= d) incl += o;
    }
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    int32_t off = carry_s, tot = 0;
    for (int w = 0; w < nwarp; ++w) {
      if (w < warp) off += warp_tot[w];
      tot += warp_tot[w];
    }
    if (i < count) sums[i] = off + incl - x;
    __syncthreads();
    if (threadIdx.x == 0) carry_s += tot;
    __syncthreads();
  }
}

__global__ void scan_add_offsets(int32_t* data, int64_t N, const int32_t* tile_sums) {
  int64_t base = (int64_t)blockIdx.x * kScanTile + (int64_t)threadIdx.x * kScanPerThread;
  int32_t off = tile_sums[blockIdx.x];
#pragma unroll
  for (int k = 0; k < kScanPerThread; ++k)
    if (base + k < N) data[base + k] += off;
}

int32_t exclusive_scan(gnnco_handle* h, int32_t* data, int64_t N, int32_t* tile_sums, cudaStream_t st) {
  if (N <= 0) return GNNCO_OK;
  int32_t tiles = (int32_t)((N + kScanTile - 1) / kScanTile);
  scan_tiles<<<tiles, kScanThreads, 0, st>>>(data, N, tile_sums);
  scan_tile_sums<<<1, 1024, 0, st>>>(tile_sums, tiles);
  scan_add_offsets<<<tiles, kScanThreads, 0, st>>>(data, N, tile_sums);
  if (h) h->launches += 3;
  GNNCO_LAUNCH_CHECK();
  return GNNCO_OK;
}

// ---------------------------------------------------------------------- radix sort
constexpr int kSortThreads = 256;
constexpr int kSortWarps = kSortThreads / 32;
constexpr int kSortRounds = 8;                               // 32 keys per warp per round
constexpr int kSortKeysPerWarp = 32 * kSortRounds;
constexpr int kSortTile = kSortWarps * kSortKeysPerWarp;     // 2048 keys per block

__device__ __forceinline__ void count_warp_digits(const uint64_t* keys, int64_t N, int64_t warp_base, int shift,
                                                  int32_t* cnt, int lane) {
#pragma unroll
  for (int r = 0; r < kSortRounds; ++r) {
    int64_t idx = warp_base + r * 32 + lane;
    bool valid = idx < N;
    uint32_t d = valid ? (uint32_t)((keys[idx] >> shift) & 255u) : 256u;
    uint32_t peers = __match_any_sync(0xffffffffu, d);
    if (valid && lane == __ffs(peers) - 1) cnt[d] += __popc(peers);
    __syncwarp();
  }
}

__global__ void sort_histogram(const uint64_t* keys, int64_t N, int shift, int32_t* hist, int32_t nblocks) {
  __shared__ int32_t cnt[kSortWarps][256];
  for (int i = threadIdx.x; i < kSortWarps * 256; i += kSortThreads) (&cnt[0][0])[i] = 0;
  __syncthreads();
  int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  count_warp_digits(keys, N, (int64_t)blockIdx.x * kSortTile + warp * kSortKeysPerWarp, shift, cnt[warp], lane);
  __syncthreads();
  int32_t total = 0;
#pragma unroll
  for (int w = 0; w < kSortWarps; ++w) total += cnt[w][threadIdx.x];
  hist[(int64_t)threadIdx.x * nblocks + blockIdx.x] = total;   // digit-major: a flat scan gives global offsets
}

__global__ void sort_scatter(const uint64_t* keys, uint64_t* out, int64_t N, int shift, const int32_t* offs,
                             int32_t nblocks, const int32_t* vals, int32_t* vals_out) {
  __shared__ int32_t cnt[kSortWarps][256];
  for (int i = threadIdx.x; i < kSortWarps * 256; i += kSortThreads) (&cnt[0][0])[i] = 0;
  __syncthreads();
  int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int64_t warp_base = (int64_t)blockIdx.x * kSortTile + warp * kSortKeysPerWarp;
  count_warp_digits(keys, N, warp_base, shift, cnt[warp], lane);
  __syncthreads();
  {
    int32_t base = offs[(int64_t)threadIdx.x * nblocks + blockIdx.x];
#pragma unroll
    for (int w = 0; w < kSortWarps; ++w) {
      int32_t c = cnt[w][threadIdx.x];
      cnt[w][threadIdx.x] = base;        // first output slot of (warp w, this digit)
      base += c;
    }
  }
  __syncthreads();
  // keys of one warp are visited in index order, lanes in order: equal digits keep their order
#pragma unroll
  for (int r = 0; r < kSortRounds; ++r) {
    int64_t idx = warp_base + r * 32 + lane;
    bool valid = idx < N;
    uint64_t key = valid ? keys[idx] : 0ull;
    uint32_t d = valid ? (uint32_t)((key >> shift) & 255u) : 256u;
    uint32_t peers = __match_any_sync(0xffffffffu, d);
    int rank = __popc(peers & ((1u << lane) - 1u));
    int32_t pos = valid ? cnt[warp][d] + rank : 0;
    __syncwarp();
    if (valid && rank == 0) cnt[warp][d] += __popc(peers);
    __syncwarp();
    if (valid) {
      out[pos] = key;
      if (vals) vals_out[pos] = vals[idx];        // optional 32-bit payload travels with its key
    }
  }
}

// Stable sort of keys on bits [bit_lo, bit_hi), optionally with a 32-bit payload per key (va / vb ping-pong
// like the keys).  Returns the buffers that hold the result.
int32_t radix_sort(gnnco_handle* h, uint64_t* a, uint64_t* b, int64_t N, int bit_lo, int bit_hi, int32_t* hist,
                   int32_t* tile_sums, cudaStream_t st, uint64_t** result, int32_t* va = nullptr, int32_t* vb = nullptr,
                   int32_t** vresult = nullptr) {
  *result = a;
  if (vresult) *vresult = va;
  if (N <= 1) return GNNCO_OK;
  int32_t nblocks = (int32_t)((N + kSortTile - 1) / kSortTile);
  for (int shift = bit_lo; shift < bit_hi; shift += 8) {
    sort_histogram<<<nblocks, kSortThreads, 0, st>>>(a, N, shift, hist, nblocks);
    if (h) h->launches += 1;
    int32_t rc = exclusive_scan(h, hist, (int64_t)256 * nblocks, tile_sums, st);
    if (rc != GNNCO_OK) return rc;
    sort_scatter<<<nblocks, kSortThreads, 0, st>>>(a, b, N, shift, hist, nblocks, va, vb);
    if (h) h->launches += 1;
    GNNCO_LAUNCH_CHECK();
    uint64_t* t = a; a = b; b = t;
    int32_t* tv = va; va = vb; vb = tv;
  }
  *result = a;
  if (vresult) *vresult = va;
  return GNNCO_OK;
}

// ptr[s] = first index k whose segment id (key >> 32) is >= s, for s in [0, nseg]
__global__ void segment_starts(const uint64_t* keys, int64_t N, int32_t nseg, int32_t* ptr) {
  int64_t k = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (k > N) return;
  int64_t prev = k == 0 ? -1 : (int64_t)(keys[k - 1] >> 32);
  int64_t cur = k == N ? nseg : (int64_t)(keys[k] >> 32);
  for (int64_t s = prev + 1; s <= cur; ++s) ptr[s] = (int32_t)k;
}

// ----------------------------------------------------------------------- the steps
enum { kStatus = 0, kCntIn = 1, kCntB = 2, kMaxRow = 3, kSelfLoop = 4, kLongCnt = 5, kStatusWords = 16 };

__global__ void check_parts_make_keys(const int32_t* part, int64_t n, int32_t S, uint64_t* keys, int32_t* status) {
  int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  int32_t s = part[i];
  if (s < 0 || s >= S) {
    atomicMin(&status[kStatus], (int32_t)GNNCO_OUT_OF_RANGE);
    s = 0;
  }
  keys[i] = ((uint64_t)(uint32_t)s << 32) | (uint64_t)i;
}

__global__ void check_edges(const int32_t* eu, const int32_t* ev, int64_t E, int64_t n, int32_t* status) {
  int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= E) return;
  int32_t u = eu[e], v = ev[e];
  if (u < 0 || u >= n || v < 0 || v >= n) atomicMin(&status[kStatus], (int32_t)GNNCO_OUT_OF_RANGE);
  else if (u == v) atomicMax(&status[kSelfLoop], 1);    // self loop seen (reported if ids are all in range)
}

__global__ void unpack_node_order(const uint64_t* keys, int64_t n, int32_t* perm, int32_t* inv_perm,
                                  int32_t* node_part) {
  int64_t k = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (k >= n) return;
  uint64_t key = keys[k];
  int32_t orig = (int32_t)(key & 0xffffffffu);
  perm[k] = orig;
  inv_perm[orig] = (int32_t)k;
  node_part[k] = (int32_t)(key >> 32);
}

__global__ void classify_edges(const int32_t* eu, const int32_t* ev, int64_t E, const int32_t* inv_perm,
                               const int32_t* node_part, uint64_t* intra_keys, uint64_t* bnd_keys,
                               uint8_t* is_boundary, int32_t* status) {
  int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= E) return;
  uint32_t a = (uint32_t)inv_perm[eu[e]], b = (uint32_t)inv_perm[ev[e]];
  if (node_part[a] == node_part[b]) {
    int32_t slot = atomicAdd(&status[kCntIn], 1);
    intra_keys[2 * (int64_t)slot] = ((uint64_t)a << 32) | b;
    intra_keys[2 * (int64_t)slot + 1] = ((uint64_t)b << 32) | a;
  } else {
    int32_t slot = atomicAdd(&status[kCntB], 1);
    uint32_t lo = a < b ? a : b, hi = a < b ? b : a;
    bnd_keys[slot] = ((uint64_t)lo << 32) | hi;
    is_boundary[a] = 1;
    is_boundary[b] = 1;
  }
}

__global__ void unpack_pairs(const uint64_t* keys, int64_t N, int32_t* hi_out, int32_t* lo_out, int32_t* status) {
  int64_t k = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (k >= N) return;
  uint64_t key = keys[k];
  if (k > 0 && keys[k - 1] == key) atomicMin(&status[kStatus], (int32_t)GNNCO_NOT_SIMPLE_GRAPH);   // repeated edge
  if (hi_out) hi_out[k] = (int32_t)(key >> 32);
  lo_out[k] = (int32_t)(key & 0xffffffffu);
}

__global__ void degree_scale(const int32_t* rowptr, int64_t n, float* inv_deg, int32_t* status) {
  int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  int32_t deg = rowptr[i + 1] - rowptr[i];
  inv_deg[i] = __fdiv_rn(1.0f, (float)(deg + 1));
  int32_t m = deg;
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, d));
  if ((threadIdx.x & 31) == 0) atomicMax(&status[kMaxRow], m);
}

// row_head[i] = {rowptr[i], degree, first neighbour or -1, second neighbour or -1}
__global__ void build_row_heads(const int32_t* rowptr, const int32_t* colidx, int64_t n, int4* row_head) {
  int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const int32_t a = rowptr[i], d = rowptr[i + 1] - a;
  row_head[i] = make_int4(a, d, d > 0 ? colidx[a] : -1, d > 1 ? colidx[a + 1] : -1);
}

// rows longer than kLongRowDegree, in no particular order (each is processed on its own)
__global__ void collect_long_rows(const int32_t* rowptr, int64_t n, int32_t* long_rows, int32_t capacity,
                                  int32_t* status) {
  int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  if (rowptr[i + 1] - rowptr[i] > kLongRowDegree) {
    int32_t slot = atomicAdd(&status[kLongCnt], 1);
    if (slot < capacity) long_rows[slot] = (int32_t)i;
  }
}

// extents of the listed rows: ext[2k] = rowptr[rows[k]], ext[2k+1] = rowptr[rows[k] + 1]
__global__ void gather_extents(const int32_t* rows, const int32_t* rowptr, int32_t count, int32_t* ext) {
  const int32_t k = blockIdx.x * blockDim.x + threadIdx.x;
  if (k >= count) return;
  ext[2 * k] = rowptr[rows[k]];
  ext[2 * k + 1] = rowptr[rows[k] + 1];
}

template <int VEC>
__global__ void gather_rows_kernel(const char* src, char* dst, const int32_t* index, int64_t rows, int64_t units) {
  int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= rows * units) return;
  int64_t i = t / units, w = t - i * units;
  int64_t s = (int64_t)index[i] * units + w;
  if (VEC == 16) reinterpret_cast<uint4*>(dst)[t] = reinterpret_cast<const uint4*>(src)[s];
  else reinterpret_cast<uint32_t*>(dst)[t] = reinterpret_cast<const uint32_t*>(src)[s];
}

// src[rowptr[i] + i] = i, then row i's neighbours: what the fused aggregation + transform gathers for row i, in
// the order the aggregation kernels add.  Four threads per row.
__global__ void build_source_list(const int32_t* rowptr, const int32_t* colidx, int64_t n, int32_t* src) {
  const int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t i = g >> 2;
  const int sub = (int)(g & 3);
  if (i >= n) return;
  const int32_t a = rowptr[i], b = rowptr[i + 1];
  int32_t* dst = src + a + i;
  if (sub == 0) dst[0] = (int32_t)i;
  for (int32_t k = a + sub; k < b; k += 4) dst[1 + k - a] = colidx[k];
}

inline int bits_for(int64_t count) {   // bits needed to hold ids 0..count-1
  int b = 0;
  while (b < 32 && ((int64_t)1 << b) < count) ++b;
  return b;
}

inline unsigned grid_for(int64_t work, int threads) { return (unsigned)((work + threads - 1) / threads); }

struct PersistentLayout {
  int32_t *perm, *inv_perm, *node_part, *part_ptr, *rowptr, *colidx, *bnd_u, *bnd_v;
  float* inv_deg;
  uint8_t* is_boundary;
  int32_t *pair_row0, *pair_rows;
  int32_t *tile_row0, *tile_rows, *item_row0, *item_row1, *part_item_ptr, *status, *long_rows, *seg_begin, *seg_end, *long_first_seg;
  int4* row_head;
  int32_t* src_list;
  FuseSet fuse;
  int32_t *wg_begin, *wg_end, *wg_slot, *wg_mpart, *wg_mfirst, *wg_mcount;
  int64_t max_chunks;
  int64_t max_tiles, max_items, max_long, max_segs;
  size_t bytes;
};

PersistentLayout carve_persistent(void* base, int64_t n, int64_t E, int32_t S) {
  PersistentLayout L;
  Carver c(base, ~(size_t)0);
  L.max_tiles = n / kGemmTileRows + S + 1;
  L.max_items = n / kItemRows + S + 1;
  L.status = c.take<int32_t>(kStatusWords);
  L.perm = c.take<int32_t>(n);
  L.inv_perm = c.take<int32_t>(n);
  L.node_part = c.take<int32_t>(n);
  L.part_ptr = c.take<int32_t>((size_t)S + 1);
  L.rowptr = c.take<int32_t>(n + 1);
  L.colidx = c.take<int32_t>(2 * E + 1);
  L.bnd_u = c.take<int32_t>(E + 1);
  L.bnd_v = c.take<int32_t>(E + 1);
  L.inv_deg = c.take<float>(n);
  L.is_boundary = c.take<uint8_t>(n);
  L.tile_row0 = c.take<int32_t>(L.max_tiles);
  L.tile_rows = c.take<int32_t>(L.max_tiles);
  L.pair_row0 = c.take<int32_t>(L.max_tiles);
  L.pair_rows = c.take<int32_t>(L.max_tiles);
  L.item_row0 = c.take<int32_t>(L.max_items);
  L.item_row1 = c.take<int32_t>(L.max_items);
  L.part_item_ptr = c.take<int32_t>((size_t)S + 1);
  L.max_long = 2 * E / kLongRowDegree + 1;
  L.long_rows = c.take<int32_t>(L.max_long);
  L.max_segs = 2 * E / kLongRowSegment + L.max_long + 1;
  L.seg_begin = c.take<int32_t>(L.max_segs);
  L.seg_end = c.take<int32_t>(L.max_segs);
  L.long_first_seg = c.take<int32_t>(L.max_long + 1);
  L.row_head = c.take<int4>(n);
  L.src_list = c.take<int32_t>((size_t)n + 2 * E + 8);
  L.fuse = carve_fuse_set(c, (size_t)L.max_tiles);
  L.max_chunks = (int64_t)S + n / kWgChunkMinRows + 1;
  L.wg_begin = c.take<int32_t>(L.max_chunks);
  L.wg_end = c.take<int32_t>(L.max_chunks);
  L.wg_slot = c.take<int32_t>(L.max_chunks);
  L.wg_mpart = c.take<int32_t>((size_t)S);
  L.wg_mfirst = c.take<int32_t>((size_t)S);
  L.wg_mcount = c.take<int32_t>((size_t)S);
  L.bytes = c.off;
  return L;
}

struct ScratchLayout {
  uint64_t *keys_a, *keys_b, *bkeys_a, *bkeys_b;
  int32_t *hist, *tile_sums;
  size_t bytes;
};

ScratchLayout carve_scratch(void* base, int64_t n, int64_t E) {
  ScratchLayout L;
  Carver c(base, ~(size_t)0);
  int64_t big = n > 2 * E ? n : 2 * E;
  int64_t nblocks = (big + kSortTile - 1) / kSortTile + 1;
  L.keys_a = c.take<uint64_t>(big + 1);
  L.keys_b = c.take<uint64_t>(big + 1);
  L.bkeys_a = c.take<uint64_t>(E + 1);
  L.bkeys_b = c.take<uint64_t>(E + 1);
  L.hist = c.take<int32_t>(256 * nblocks);
  L.tile_sums = c.take<int32_t>((256 * nblocks + kScanTile - 1) / kScanTile + 1);
  L.bytes = c.off;
  return L;
}

bool valid_sizes(int64_t n, int64_t E, int32_t S) {
  return n >= 1 && n < ((int64_t)1 << 31) - 1 && E >= 0 && 2 * E < ((int64_t)1 << 31) - 1 && S >= 1 && S <= n;
}

}  // namespace

// The sort and scan primitives for the other translation units (louvain.cu).
int32_t device_exclusive_scan(int32_t* data, int64_t N, int32_t* tile_sums, cudaStream_t st) {
  return exclusive_scan(nullptr, data, N, tile_sums, st);
}
int32_t device_radix_sort(uint64_t* a, uint64_t* b, int64_t N, int bit_lo, int bit_hi, int32_t* hist, int32_t* tile_sums,
                          cudaStream_t st, uint64_t** result, int32_t* va, int32_t* vb, int32_t** vresult) {
  return radix_sort(nullptr, a, b, N, bit_lo, bit_hi, hist, tile_sums, st, result, va, vb, vresult);
}
void device_sort_scratch_sizes(int64_t N, size_t* hist_ints, size_t* tile_sum_ints) {
  const int64_t nblocks = (N + kSortTile - 1) / kSortTile + 1;
  *hist_ints = (size_t)(256 * nblocks);
  *tile_sum_ints = (size_t)((256 * nblocks + kScanTile - 1) / kScanTile + 1);
}
void device_scan_scratch_size(int64_t N, size_t* tile_sum_ints) { *tile_sum_ints = (size_t)((N + kScanTile - 1) / kScanTile + 1); }

// Work tables of the subgraphs with active[s] != 0 (all when active == nullptr), in subgraph order:
//   tiles of 128 rows and double tiles of 256 rows of one subgraph (dense transforms), objective work items
//   of kItemRows rows with the item range of every subgraph (empty for an inactive one), row chunks of
//   256 rows, and the weight-gradient chunks: a subgraph is one chunk unless it is so long that too few
//   blocks would be busy; then it is cut into runs of chunk_rows rows whose partial results meet in a
//   scratch area (slot >= 0) and are summed in chunk order afterwards; slot = -(s+1) means "write
//   subgraph s's result directly".  Scratch slots are numbered over ALL subgraphs, so a plan for some
//   subgraphs uses the same slots as the full set.
void build_work_tables(const std::vector<int32_t>& part_ptr, int32_t S, int64_t n, int sm_count, const uint8_t* active,
                       HostWorkTables& o) {
  o = HostWorkTables();
  o.pip.assign((size_t)S + 1, 0);
  const int64_t sms = sm_count > 0 ? sm_count : 148;
  const int64_t per = (n + 4 * sms - 1) / (4 * sms);
  int64_t chunk_rows = (per + 63) / 64 * 64;
  if (chunk_rows < kWgChunkMinRows) chunk_rows = kWgChunkMinRows;
  int32_t slots = 0;
  for (int32_t s = 0; s < S; ++s) {
    const int32_t a = part_ptr[s], b = part_ptr[s + 1];
    const bool on = !active || active[s];
    o.pip[s] = (int32_t)o.i0.size();
    const bool split = b - a > chunk_rows;
    int32_t first_slot = slots;
    if (split) slots += (int32_t)((b - a + chunk_rows - 1) / chunk_rows);
    if (!on) continue;
    for (int32_t r = a; r < b; r += kGemmTileRows) {
      o.t0.push_back(r);
      o.tr.push_back(b - r < kGemmTileRows ? b - r : kGemmTileRows);
    }
    for (int32_t r = a; r < b; r += 2 * kGemmTileRows) {
      o.p0.push_back(r);
      o.pr.push_back(b - r < 2 * kGemmTileRows ? b - r : 2 * kGemmTileRows);
    }
    for (int32_t r = a; r < b; r += 256) {
      o.c0.push_back(r);
      o.cr.push_back(b - r < 256 ? b - r : 256);
    }
    for (int32_t r = a; r < b; r += kItemRows) {
      o.i0.push_back(r);
      o.i1.push_back(b - r < kItemRows ? b : r + kItemRows);
    }
    if (!split) {
      o.wb.push_back(a); o.we.push_back(b); o.wsl.push_back(-(s + 1));
    } else {
      o.mp.push_back(s); o.mf.push_back(first_slot);
      int32_t cnt = 0;
      for (int64_t r = a; r < b; r += chunk_rows) {
        o.wb.push_back((int32_t)r);
        o.we.push_back((int32_t)(r + chunk_rows < b ? r + chunk_rows : b));
        o.wsl.push_back(first_slot + cnt);
        ++cnt;
      }
      o.mc.push_back(cnt);
    }
  }
  o.pip[S] = (int32_t)o.i0.size();
  o.n_wg_slots = slots;
}

extern "C" const char* gnnco_status_string(int32_t status) {
  switch (status) {
    case GNNCO_OK: return "ok";
    case GNNCO_INVALID_ARGUMENT: return "invalid argument";
    case GNNCO_OUT_OF_RANGE: return "node or partition id out of range";
    case GNNCO_NOT_SIMPLE_GRAPH: return "graph has a self loop or a repeated edge";
    case GNNCO_UNSUPPORTED: return "unsupported dtype or width";
    case GNNCO_WORKSPACE_TOO_SMALL: return "work area too small";
    case GNNCO_CUDA_ERROR: return "CUDA error";
    case GNNCO_INTERNAL: return "internal error";
    default: return "unknown status";
  }
}

extern "C" int32_t gnnco_partition_workspace_bytes(int64_t n, int64_t E, int32_t S, size_t* persistent,
                                                  size_t* scratch) {
  if (!persistent || !scratch || !valid_sizes(n, E, S)) return GNNCO_INVALID_ARGUMENT;
  *persistent = carve_persistent(nullptr, n, E, S).bytes;
  *scratch = carve_scratch(nullptr, n, E).bytes;
  return GNNCO_OK;
}

extern "C" int32_t gnnco_partition_load(const gnnco_graph_desc* g, void* persistent_ws, size_t persistent_bytes,
                                       void* scratch_ws, size_t scratch_bytes, void* stream, gnnco_handle** out) {
  if (!g || !out || !persistent_ws || !scratch_ws) return GNNCO_INVALID_ARGUMENT;
  *out = nullptr;
  const int64_t n = g->n, E = g->E;
  const int32_t S = g->S;
  if (!valid_sizes(n, E, S) || !g->part || (E > 0 && (!g->edge_u || !g->edge_v))) return GNNCO_INVALID_ARGUMENT;
  if (((uintptr_t)persistent_ws & 255) || ((uintptr_t)scratch_ws & 255)) return GNNCO_INVALID_ARGUMENT;
  PersistentLayout P = carve_persistent(persistent_ws, n, E, S);
  ScratchLayout W = carve_scratch(scratch_ws, n, E);
  if (P.bytes > persistent_bytes || W.bytes > scratch_bytes) return GNNCO_WORKSPACE_TOO_SMALL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  gnnco_handle* h = new (std::nothrow) gnnco_handle();
  if (!h) return GNNCO_INTERNAL;
  struct Guard {
    gnnco_handle* h;
    ~Guard() { if (h) gnnco_destroy(h); }
  } guard{h};
  GNNCO_CUDA_TRY(cudaGetDevice(&h->device));
  GNNCO_CUDA_TRY(cudaDeviceGetAttribute(&h->sm_count, cudaDevAttrMultiProcessorCount, h->device));
  h->n = n; h->E = E; h->S = S;
  h->perm = P.perm; h->inv_perm = P.inv_perm; h->node_part = P.node_part; h->part_ptr = P.part_ptr;
  h->rowptr = P.rowptr; h->colidx = P.colidx; h->bnd_u = P.bnd_u; h->bnd_v = P.bnd_v;
  h->inv_deg = P.inv_deg; h->is_boundary = P.is_boundary;
  h->pair_row0 = P.pair_row0; h->pair_rows = P.pair_rows;
  h->tile_row0 = P.tile_row0; h->tile_rows = P.tile_rows; h->item_row0 = P.item_row0; h->item_row1 = P.item_row1;
  h->part_item_ptr = P.part_item_ptr; h->status = P.status; h->long_rows = P.long_rows; h->seg_begin = P.seg_begin; h->seg_end = P.seg_end;
  h->long_first_seg = P.long_first_seg; h->row_head = P.row_head; h->src_list = P.src_list;
  h->wg_begin = P.wg_begin; h->wg_end = P.wg_end; h->wg_slot = P.wg_slot;
  h->wg_mpart = P.wg_mpart; h->wg_mfirst = P.wg_mfirst; h->wg_mcount = P.wg_mcount;

  const int T = 256;
  int32_t hs[kStatusWords];
  GNNCO_CUDA_TRY(cudaMemsetAsync(P.status, 0, kStatusWords * sizeof(int32_t), st));
  GNNCO_CUDA_TRY(cudaMemsetAsync(P.is_boundary, 0, (size_t)n, st));
  // 1. validate ids; node keys (part, id)
  check_parts_make_keys<<<grid_for(n, T), T, 0, st>>>(g->part, n, S, W.keys_a, P.status);
  h->launches += 1;
  if (E > 0) {
    check_edges<<<grid_for(E, T), T, 0, st>>>(g->edge_u, g->edge_v, E, n, P.status);
    h->launches += 1;
  }
  GNNCO_LAUNCH_CHECK();
  GNNCO_CUDA_TRY(cudaMemcpyAsync(hs, P.status, sizeof(hs), cudaMemcpyDeviceToHost, st));
  GNNCO_CUDA_TRY(cudaStreamSynchronize(st));
  if (hs[kStatus] != GNNCO_OK) return hs[kStatus];
  if (hs[kSelfLoop] != 0) return GNNCO_NOT_SIMPLE_GRAPH;

  // 2. new node order: stable sort of (part, id) on the part bits
  uint64_t* sorted = nullptr;
  int32_t rc = radix_sort(h, W.keys_a, W.keys_b, n, 32, 32 + bits_for(S), W.hist, W.tile_sums, st, &sorted);
  if (rc != GNNCO_OK) return rc;
  unpack_node_order<<<grid_for(n, T), T, 0, st>>>(sorted, n, P.perm, P.inv_perm, P.node_part);
  segment_starts<<<grid_for(n + 1, T), T, 0, st>>>(sorted, n, S, P.part_ptr);
  h->launches += 2;

  // 3. split edges
  if (E > 0) {
    classify_edges<<<grid_for(E, T), T, 0, st>>>(g->edge_u, g->edge_v, E, P.inv_perm, P.node_part, W.keys_a,
                                                 W.bkeys_a, P.is_boundary, P.status);
    h->launches += 1;
  }
  GNNCO_LAUNCH_CHECK();
  GNNCO_CUDA_TRY(cudaMemcpyAsync(hs, P.status, sizeof(hs), cudaMemcpyDeviceToHost, st));
  h->h_part_ptr.resize((size_t)S + 1);
  GNNCO_CUDA_TRY(cudaMemcpyAsync(h->h_part_ptr.data(), P.part_ptr, ((size_t)S + 1) * sizeof(int32_t),
                                 cudaMemcpyDeviceToHost, st));
  GNNCO_CUDA_TRY(cudaStreamSynchronize(st));
  h->E_in = hs[kCntIn];
  h->E_b = hs[kCntB];
  if (h->E_in + h->E_b != E) return GNNCO_INTERNAL;

  // 4. CSR of intra edges: sort (row, col) keys; boundary list: sort (lo, hi) keys
  const int nb = bits_for(n);
  const int64_t nnz = 2 * h->E_in;
  uint64_t* csr_keys = nullptr;
  rc = radix_sort(h, W.keys_a, W.keys_b, nnz, 0, nb, W.hist, W.tile_sums, st, &csr_keys);
  if (rc != GNNCO_OK) return rc;
  uint64_t* other = csr_keys == W.keys_a ? W.keys_b : W.keys_a;
  rc = radix_sort(h, csr_keys, other, nnz, 32, 32 + nb, W.hist, W.tile_sums, st, &csr_keys);
  if (rc != GNNCO_OK) return rc;
  if (nnz > 0) {
    unpack_pairs<<<grid_for(nnz, T), T, 0, st>>>(csr_keys, nnz, nullptr, P.colidx, P.status);
    h->launches += 1;
  }
  segment_starts<<<grid_for(nnz + 1, T), T, 0, st>>>(csr_keys, nnz, (int32_t)n, P.rowptr);
  h->launches += 1;
  uint64_t* bkeys = nullptr;
  rc = radix_sort(h, W.bkeys_a, W.bkeys_b, h->E_b, 0, nb, W.hist, W.tile_sums, st, &bkeys);
  if (rc != GNNCO_OK) return rc;
  other = bkeys == W.bkeys_a ? W.bkeys_b : W.bkeys_a;
  rc = radix_sort(h, bkeys, other, h->E_b, 32, 32 + nb, W.hist, W.tile_sums, st, &bkeys);
  if (rc != GNNCO_OK) return rc;
  if (h->E_b > 0) {
    unpack_pairs<<<grid_for(h->E_b, T), T, 0, st>>>(bkeys, h->E_b, P.bnd_u, P.bnd_v, P.status);
    h->launches += 1;
  }
  degree_scale<<<grid_for(n, T), T, 0, st>>>(P.rowptr, n, P.inv_deg, P.status);
  collect_long_rows<<<grid_for(n, T), T, 0, st>>>(P.rowptr, n, P.long_rows, (int32_t)P.max_long, P.status);
  build_row_heads<<<grid_for(n, T), T, 0, st>>>(P.rowptr, P.colidx, n, P.row_head);
  build_source_list<<<grid_for(n * 4, T), T, 0, st>>>(P.rowptr, P.colidx, n, P.src_list);
  h->launches += 4;
  GNNCO_LAUNCH_CHECK();

  // 5. host-built tables: dense-transform tiles, objective work items, weight-gradient chunks (from part_ptr)
  HostWorkTables tab;
  build_work_tables(h->h_part_ptr, S, n, h->sm_count, nullptr, tab);
  const std::vector<int32_t>&t0 = tab.t0, &tr = tab.tr, &p0 = tab.p0, &pr = tab.pr, &i0 = tab.i0, &i1 = tab.i1, &pip = tab.pip,
                            &wb = tab.wb, &we = tab.we, &wsl = tab.wsl, &mp = tab.mp, &mf = tab.mf, &mc = tab.mc;
  h->n_wg_chunks = (int32_t)wb.size();
  h->n_wg_slots = tab.n_wg_slots;
  h->n_wg_multi = (int32_t)mp.size();
  if (h->n_wg_chunks > P.max_chunks) return GNNCO_INTERNAL;
  h->n_tiles = (int32_t)t0.size();
  h->n_pairs = (int32_t)p0.size();
  h->n_items = (int32_t)i0.size();
  if (h->n_tiles > P.max_tiles || h->n_items > P.max_items) return GNNCO_INTERNAL;
  auto up = [&](int32_t* dst, const std::vector<int32_t>& v) {
    return v.empty() ? cudaSuccess
                     : cudaMemcpyAsync(dst, v.data(), v.size() * sizeof(int32_t), cudaMemcpyHostToDevice, st);
  };
  GNNCO_CUDA_TRY(up(P.tile_row0, t0));
  GNNCO_CUDA_TRY(up(P.tile_rows, tr));
  GNNCO_CUDA_TRY(up(P.pair_row0, p0));
  GNNCO_CUDA_TRY(up(P.pair_rows, pr));
  GNNCO_CUDA_TRY(up(P.item_row0, i0));
  GNNCO_CUDA_TRY(up(P.item_row1, i1));
  GNNCO_CUDA_TRY(up(P.part_item_ptr, pip));
  GNNCO_CUDA_TRY(up(P.wg_begin, wb));
  GNNCO_CUDA_TRY(up(P.wg_end, we));
  GNNCO_CUDA_TRY(up(P.wg_slot, wsl));
  GNNCO_CUDA_TRY(up(P.wg_mpart, mp));
  GNNCO_CUDA_TRY(up(P.wg_mfirst, mf));
  GNNCO_CUDA_TRY(up(P.wg_mcount, mc));
  GNNCO_CUDA_TRY(cudaMemcpyAsync(hs, P.status, sizeof(hs), cudaMemcpyDeviceToHost, st));
  GNNCO_CUDA_TRY(cudaStreamSynchronize(st));
  if (hs[kStatus] != GNNCO_OK) return hs[kStatus];
  h->max_row = hs[kMaxRow];
  GNNCO_CUDA_TRY(cudaStreamCreateWithFlags(&h->side_stream, cudaStreamNonBlocking));
  GNNCO_CUDA_TRY(cudaEventCreateWithFlags(&h->ev_fork, cudaEventDisableTiming));
  GNNCO_CUDA_TRY(cudaEventCreateWithFlags(&h->ev_join, cudaEventDisableTiming));
  h->n_long = hs[kLongCnt];
  if (h->n_long > P.max_long) return GNNCO_INTERNAL;
  if (h->n_long > 0) {
    // The long rows were collected in no particular order: sort them, then cut every row's
    // neighbour list into segments of at most kLongRowSegment entries (one block each in the
    // aggregation; a row's segments are consecutive, so its partial sums are added in a fixed order).
    std::vector<int32_t> lr((size_t)h->n_long), ext(2 * (size_t)h->n_long);
    GNNCO_CUDA_TRY(cudaMemcpyAsync(lr.data(), P.long_rows, lr.size() * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    GNNCO_CUDA_TRY(cudaStreamSynchronize(st));
    std::sort(lr.begin(), lr.end());
    GNNCO_CUDA_TRY(cudaMemcpyAsync(P.long_rows, lr.data(), lr.size() * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    // 2 * n_long <= 2 * max_long <= max_segs + max_long: seg_begin is large enough to hold the extents for a moment
    if (2 * (int64_t)h->n_long > P.max_segs) return GNNCO_INTERNAL;
    gather_extents<<<grid_for(h->n_long, T), T, 0, st>>>(P.long_rows, P.rowptr, h->n_long, P.seg_begin);
    h->launches += 1;
    GNNCO_CUDA_TRY(cudaMemcpyAsync(ext.data(), P.seg_begin, ext.size() * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    GNNCO_CUDA_TRY(cudaStreamSynchronize(st));
    std::vector<int32_t> sb, se, first((size_t)h->n_long + 1);
    for (int32_t k = 0; k < h->n_long; ++k) {
      first[k] = (int32_t)sb.size();
      for (int64_t a = ext[2 * k]; a < ext[2 * k + 1]; a += kLongRowSegment) {
        sb.push_back((int32_t)a);
        se.push_back((int32_t)(a + kLongRowSegment < ext[2 * k + 1] ? a + kLongRowSegment : ext[2 * k + 1]));
      }
    }
    first[h->n_long] = (int32_t)sb.size();
    if ((int64_t)sb.size() > P.max_segs) return GNNCO_INTERNAL;
    h->n_long_segs = (int32_t)sb.size();
    GNNCO_CUDA_TRY(up(P.seg_begin, sb));
    GNNCO_CUDA_TRY(up(P.seg_end, se));
    GNNCO_CUDA_TRY(up(P.long_first_seg, first));
    GNNCO_CUDA_TRY(cudaStreamSynchronize(st));      // the host vectors go out of scope
  }
  // tables of the hidden layer that runs as one kernel (light / heavy double tiles, per-cluster ranges)
  h->fuse = P.fuse;
  rc = build_fuse_set(h, P.pair_row0, P.pair_rows, p0, pr, h->fuse, st);
  if (rc != GNNCO_OK) return rc;
  guard.h = nullptr;
  *out = h;
  return GNNCO_OK;
}

extern "C" int32_t gnnco_graph_info(const gnnco_handle* h, gnnco_graph_view* out) {
  if (!h || !out) return GNNCO_INVALID_ARGUMENT;
  out->n = h->n; out->S = h->S; out->E_in = h->E_in; out->E_b = h->E_b; out->max_row = h->max_row;
  out->perm = h->perm; out->inv_perm = h->inv_perm; out->part_ptr = h->part_ptr; out->node_part = h->node_part;
  out->rowptr = h->rowptr; out->colidx = h->colidx; out->bnd_u = h->bnd_u; out->bnd_v = h->bnd_v;
  out->inv_deg = h->inv_deg; out->is_boundary = h->is_boundary;
  return GNNCO_OK;
}

extern "C" int32_t gnnco_gather_rows(const gnnco_handle* h, const void* src, void* dst, const int32_t* index,
                                    int64_t rows, int64_t row_bytes, void* stream) {
  if (!h || !src || !dst || !index || rows < 0 || row_bytes <= 0 || (row_bytes & 3)) return GNNCO_INVALID_ARGUMENT;
  if (rows == 0) return GNNCO_OK;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  bool v16 = (row_bytes % 16 == 0) && !((uintptr_t)src & 15) && !((uintptr_t)dst & 15);
  int64_t units = row_bytes / (v16 ? 16 : 4);
  unsigned grid = grid_for(rows * units, 256);
  if (v16) gather_rows_kernel<16><<<grid, 256, 0, st>>>((const char*)src, (char*)dst, index, rows, units);
  else gather_rows_kernel<4><<<grid, 256, 0, st>>>((const char*)src, (char*)dst, index, rows, units);
  const_cast<gnnco_handle*>(h)->launches += 1;
  GNNCO_LAUNCH_CHECK();
  return GNNCO_OK;
}

extern "C" int32_t gnnco_async_status(const gnnco_handle* h, void* stream, int32_t* status) {
  if (!h || !status) return GNNCO_INVALID_ARGUMENT;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  GNNCO_CUDA_TRY(cudaMemcpyAsync(status, h->status, sizeof(int32_t), cudaMemcpyDeviceToHost, st));
  GNNCO_CUDA_TRY(cudaStreamSynchronize(st));
  return GNNCO_OK;
}

extern "C" int64_t gnnco_launch_count(const gnnco_handle* h) { return h ? h->launches : 0; }

extern "C" int32_t gnnco_destroy(gnnco_handle* h) {
  if (h) {
    for (cudaEvent_t e : h->prof.pool) cudaEventDestroy(e);
    if (h->ev_fork) cudaEventDestroy(h->ev_fork);
    if (h->ev_join) cudaEventDestroy(h->ev_join);
    if (h->side_stream) cudaStreamDestroy(h->side_stream);
    if (h->copy_stream) cudaStreamDestroy(h->copy_stream);
    for (cudaEvent_t e : h->ev_arrive)
      if (e) cudaEventDestroy(e);
    if (h->ev_rest) cudaEventDestroy(h->ev_rest);
    if (h->ev_begin) cudaEventDestroy(h->ev_begin);
  }
  delete h;
  return GNNCO_OK;
}
