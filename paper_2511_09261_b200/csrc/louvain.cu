// Louvain partitioning on the GPU (Section 3.1, Eqs. 1-2): the step that produces the subgraphs which
// gnnco_partition_load turns into the block-diagonal batch.
//
// The visiting order of the textbook procedure is not fixed by the paper, so its result is not unique.
// This is the variant whose result IS unique, so that it can be held bit-exact against a CPU
// restatement:
//   level graph  nodes 0..N-1, directed entries (a, b, w) for every neighbour b != a (both directions),
//                self-loop weights loop[a]; k[a] = sum_b w(a,b) + 2 loop[a]; 2m is the same on every level
//   sweep        from the frozen state every node scores its own community and every neighbouring one with
//                Eq. 2 times 2 m^2 in 64-bit integers,  score(c) = 2m kin[c] - (tot[c] - [c == own] k) k,
//                and picks the best, the lowest id among equals; it moves only on a strictly better score,
//                and a node alone in its community never moves to a community of one node with a higher id
//   acceptance   all moves of a sweep are applied together; the sweep is kept only if the exact modularity
//                numerator  sum_c [ 2m in2(c) - tot(c)^2 ]  rises strictly, otherwise it is undone and the level
//                ends (as it does without a move or at the sweep limit)
//   contraction  communities in ascending id order become the nodes of the next level; weights add up
// Per sweep: one key per entry, (node, community of the neighbour), sorted with the entry index as payload;
// a node's keys stay one contiguous run (runs are by node), inside which equal communities are adjacent,
// so one pass per node yields every kin[c] and the best community.  All sums are integer (atomics are
// order-free), so nothing depends on scheduling.  The host drives the loop and reads two integers back per
// sweep (moves, new numerator).
#include "internal.cuh"

namespace {

constexpr int kT = 256;
inline unsigned blocks_of(int64_t work) { return (unsigned)((work + kT - 1) / kT); }
inline int bits_needed(int64_t count) {
  int b = 1;
  while (b < 32 && ((int64_t)1 << b) < count) ++b;
  return b;
}

typedef unsigned long long u64;

__global__ void lv_check_edges(const int32_t* eu, const int32_t* ev, int64_t E, int64_t n, int32_t* status) {
  const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= E) return;
  const int32_t u = eu[e], v = ev[e];
  if (u < 0 || u >= n || v < 0 || v >= n) atomicMin(status, (int32_t)GNNCO_OUT_OF_RANGE);
  else if (u == v) atomicMax(status + 1, 1);
}

// level 0: both directions of every edge as keys (a << 32 | b), payload = unit weight marker
__global__ void lv_edge_keys(const int32_t* eu, const int32_t* ev, int64_t E, uint64_t* keys) {
  const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= E) return;
  const uint32_t u = (uint32_t)eu[e], v = (uint32_t)ev[e];
  keys[2 * e] = ((uint64_t)u << 32) | v;
  keys[2 * e + 1] = ((uint64_t)v << 32) | u;
}

__global__ void lv_unpack_entries(const uint64_t* keys, int64_t M, int32_t* src, int32_t* dst) {
  const int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (p >= M) return;
  src[p] = (int32_t)(keys[p] >> 32);
  dst[p] = (int32_t)(keys[p] & 0xffffffffu);
}

// row extents of the entry list sorted by source: rowp[a] = first entry of node a
__global__ void lv_row_starts(const int32_t* src, int64_t M, int64_t N, int64_t* rowp) {
  const int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (p > M) return;
  const int64_t prev = p == 0 ? -1 : src[p - 1];
  const int64_t cur = p == M ? N : src[p];
  for (int64_t a = prev + 1; a <= cur; ++a) rowp[a] = p;
}

__global__ void lv_fill_i64(int64_t* a, int64_t N, int64_t v) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < N) a[i] = v;
}
__global__ void lv_iota(int32_t* a, int64_t N) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < N) a[i] = (int32_t)i;
}

// k[a] = sum of the weights of a's entries + 2 loop[a]
__global__ void lv_degrees(const int64_t* rowp, const int64_t* w, const int64_t* loop, int64_t N, int64_t* k) {
  const int64_t a = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (a >= N) return;
  int64_t s = 2 * loop[a];
  for (int64_t p = rowp[a]; p < rowp[a + 1]; ++p) s += w[p];
  k[a] = s;
}

__global__ void lv_community_totals(const int32_t* comm, const int64_t* k, int64_t N, int64_t* tot, int32_t* size) {
  const int64_t a = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (a >= N) return;
  atomicAdd(reinterpret_cast<u64*>(tot + comm[a]), (u64)k[a]);
  if (size) atomicAdd(size + comm[a], 1);
}

__global__ void lv_sweep_keys(const int32_t* src, const int32_t* dst, const int32_t* comm, int64_t M, uint64_t* keys,
                              int32_t* idx) {
  const int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (p >= M) return;
  keys[p] = ((uint64_t)(uint32_t)src[p] << 32) | (uint32_t)comm[dst[p]];
  idx[p] = (int32_t)p;
}

// One thread per node walks its run of keys (sorted by community): kin of each neighbouring community
// in turn, best community as defined at the top of the file.
__global__ void lv_decide(const uint64_t* keys, const int32_t* idx, const int64_t* w, const int64_t* rowp,
                          const int32_t* comm, const int64_t* k, const int64_t* tot, const int32_t* size, int64_t two_m,
                          int64_t N, int32_t* next, int32_t* moves) {
  const int64_t a = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (a >= N) return;
  const int32_t own = comm[a];
  const int64_t ka = k[a];
  int64_t kin_own = 0, best_score = 0;
  int32_t best = -1;
  int64_t p = rowp[a];
  const int64_t end = rowp[a + 1];
  while (p < end) {
    const int32_t c = (int32_t)(keys[p] & 0xffffffffu);
    int64_t kin = 0;
    while (p < end && (int32_t)(keys[p] & 0xffffffffu) == c) {
      kin += w[idx[p]];
      ++p;
    }
    if (c == own) {
      kin_own = kin;
    } else {
      const int64_t sc = two_m * kin - tot[c] * ka;
      if (best < 0 || sc > best_score) {          // communities arrive in ascending id: the lowest id wins ties
        best = c;
        best_score = sc;
      }
    }
  }
  const int64_t own_score = two_m * kin_own - (tot[own] - ka) * ka;
  int32_t to = own;
  if (best >= 0 && best_score > own_score && !(size[own] == 1 && size[best] == 1 && best > own)) to = best;
  next[a] = to;
  if (to != own) atomicAdd(moves, 1);
}

// in2[c] += w for every entry whose two ends share community c (each undirected edge is seen from both
// ends), plus twice the self loops
__global__ void lv_internal_entries(const int32_t* src, const int32_t* dst, const int64_t* w, const int32_t* comm,
                                    int64_t M, int64_t* in2) {
  const int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (p >= M) return;
  const int32_t c = comm[src[p]];
  if (comm[dst[p]] == c) atomicAdd(reinterpret_cast<u64*>(in2 + c), (u64)w[p]);
}
__global__ void lv_internal_loops(const int64_t* loop, const int32_t* comm, int64_t N, int64_t* in2) {
  const int64_t a = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (a >= N) return;
  if (loop[a]) atomicAdd(reinterpret_cast<u64*>(in2 + comm[a]), (u64)(2 * loop[a]));
}
__global__ void lv_numerator(const int64_t* in2, const int64_t* tot, int64_t N, int64_t two_m, int64_t* out) {
  const int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  int64_t v = 0;
  if (c < N) v = two_m * in2[c] - tot[c] * tot[c];
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
  if ((threadIdx.x & 31) == 0 && v != 0) atomicAdd(reinterpret_cast<u64*>(out), (u64)v);
}

// contraction
__global__ void lv_mark_used(const int32_t* comm, int64_t N, int32_t* used) {
  const int64_t a = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (a < N) used[comm[a]] = 1;
}
__global__ void lv_relabel_part(int32_t* part, int64_t n, const int32_t* comm, const int32_t* newid) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) part[i] = newid[comm[part[i]]];
}
// entries between different communities keep a key (ca << 32 | cb) and their weight index; entries inside
// a community add to its self loop (both directions are present, so that sum is halved afterwards, and the
// members' own self loops are added to it once)
__global__ void lv_cross_flags(const int32_t* src, const int32_t* dst, const int32_t* comm, int64_t M, int32_t* flag) {
  const int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (p < M) flag[p] = comm[src[p]] != comm[dst[p]] ? 1 : 0;
}
__global__ void lv_cross_scatter(const int32_t* src, const int32_t* dst, const int64_t* w, const int32_t* comm,
                                 const int32_t* newid, const int32_t* pos, int64_t M, uint64_t* keys, int32_t* idx,
                                 int64_t* loop2) {
  const int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (p >= M) return;
  const int32_t ca = newid[comm[src[p]]], cb = newid[comm[dst[p]]];
  if (ca != cb) {
    keys[pos[p]] = ((uint64_t)(uint32_t)ca << 32) | (uint32_t)cb;
    idx[pos[p]] = (int32_t)p;
  } else {
    atomicAdd(reinterpret_cast<u64*>(loop2 + ca), (u64)w[p]);
  }
}
__global__ void lv_loops_down(const int64_t* loop, const int32_t* comm, const int32_t* newid, int64_t N, int64_t* loop2) {
  const int64_t a = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (a >= N) return;
  if (loop[a]) atomicAdd(reinterpret_cast<u64*>(loop2 + newid[comm[a]]), (u64)loop[a]);
}
__global__ void lv_halve(int64_t* a, int64_t N) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < N) a[i] /= 2;
}
__global__ void lv_head_flags(const uint64_t* keys, int64_t M, int32_t* flag) {
  const int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (p < M) flag[p] = (p == 0 || keys[p] != keys[p - 1]) ? 1 : 0;
}
// after an exclusive scan of the head flags, group(p) = scan[p] + flag-of-p - 1; every entry adds its weight
// to its group, the head also writes the group's endpoints
__global__ void lv_merge_entries(const uint64_t* keys, const int32_t* idx, const int64_t* w, const int32_t* scan,
                                 int64_t M, int32_t* src2, int32_t* dst2, int64_t* w2) {
  const int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (p >= M) return;
  const bool head = p == 0 || keys[p] != keys[p - 1];
  const int32_t g = scan[p] + (head ? 1 : 0) - 1;
  atomicAdd(reinterpret_cast<u64*>(w2 + g), (u64)w[idx[p]]);
  if (head) {
    src2[g] = (int32_t)(keys[p] >> 32);
    dst2[g] = (int32_t)(keys[p] & 0xffffffffu);
  }
}

struct LvLayout {
  uint64_t *key_a, *key_b;
  int32_t *idx_a, *idx_b, *src, *dst, *src2, *dst2, *flag, *comm, *next, *size, *used, *hist, *tile_sums, *counters;
  int64_t *w, *w2, *rowp, *loop, *loop2, *k, *tot, *in2, *qnum;
  size_t bytes;
};

LvLayout carve_lv(void* base, int64_t n, int64_t E) {
  LvLayout L;
  Carver c(base, ~(size_t)0);
  const size_t M = (size_t)(2 * E + 1), N = (size_t)(n + 1);
  size_t hist_ints, tile_ints, scan_ints;
  device_sort_scratch_sizes((int64_t)M, &hist_ints, &tile_ints);
  device_scan_scratch_size((int64_t)(M > N ? M : N), &scan_ints);
  L.key_a = c.take<uint64_t>(M); L.key_b = c.take<uint64_t>(M);
  L.idx_a = c.take<int32_t>(M); L.idx_b = c.take<int32_t>(M);
  L.src = c.take<int32_t>(M); L.dst = c.take<int32_t>(M); L.src2 = c.take<int32_t>(M); L.dst2 = c.take<int32_t>(M);
  L.flag = c.take<int32_t>(M > N ? M : N);
  L.w = c.take<int64_t>(M); L.w2 = c.take<int64_t>(M);
  L.rowp = c.take<int64_t>(N + 1);
  L.loop = c.take<int64_t>(N); L.loop2 = c.take<int64_t>(N);
  L.k = c.take<int64_t>(N); L.tot = c.take<int64_t>(N); L.in2 = c.take<int64_t>(N);
  L.comm = c.take<int32_t>(N); L.next = c.take<int32_t>(N); L.size = c.take<int32_t>(N); L.used = c.take<int32_t>(N);
  L.hist = c.take<int32_t>(hist_ints);
  L.tile_sums = c.take<int32_t>(tile_ints > scan_ints ? tile_ints : scan_ints);
  L.counters = c.take<int32_t>(16);
  L.qnum = c.take<int64_t>(4);
  L.bytes = c.off;
  return L;
}

bool lv_sizes_ok(int64_t n, int64_t E) { return n >= 1 && n < ((int64_t)1 << 31) - 1 && E >= 0 && 2 * E < ((int64_t)1 << 31) - 1; }

}  // namespace

extern "C" int32_t gnnco_louvain_workspace_bytes(int64_t n, int64_t E, size_t* bytes) {
  if (!bytes || !lv_sizes_ok(n, E)) return GNNCO_INVALID_ARGUMENT;
  *bytes = carve_lv(nullptr, n, E).bytes;
  return GNNCO_OK;
}

extern "C" int32_t gnnco_louvain(int64_t n, int64_t E, const int32_t* edge_u, const int32_t* edge_v, int32_t max_levels,
                                int32_t max_sweeps, int32_t* part, int32_t* S_out, int64_t* qnum_out, int64_t* two_m_out,
                                int32_t* levels_out, int32_t* sweeps_out, void* ws, size_t ws_bytes, void* stream) {
  if (!lv_sizes_ok(n, E) || !part || !S_out || !ws || max_levels < 1 || max_sweeps < 1) return GNNCO_INVALID_ARGUMENT;
  if (E > 0 && (!edge_u || !edge_v)) return GNNCO_INVALID_ARGUMENT;
  if ((uintptr_t)ws & 255) return GNNCO_INVALID_ARGUMENT;
  LvLayout L = carve_lv(ws, n, E);
  if (L.bytes > ws_bytes) return GNNCO_WORKSPACE_TOO_SMALL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int64_t two_m = 2 * E;
  int32_t hc[4] = {0, 0, 0, 0};
  // ---- level 0: validate, then both directions of every edge sorted by (a, b)
  GNNCO_CUDA_TRY(cudaMemsetAsync(L.counters, 0, 16 * sizeof(int32_t), st));
  if (E > 0) {
    lv_check_edges<<<blocks_of(E), kT, 0, st>>>(edge_u, edge_v, E, n, L.counters);
    GNNCO_LAUNCH_CHECK();
  }
  GNNCO_CUDA_TRY(cudaMemcpyAsync(hc, L.counters, 2 * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
  GNNCO_CUDA_TRY(cudaStreamSynchronize(st));
  if (hc[0] != GNNCO_OK) return hc[0];
  if (hc[1] != 0) return GNNCO_NOT_SIMPLE_GRAPH;
  int64_t N = n, M = 2 * E;
  int32_t rc;
  if (E > 0) {
    lv_edge_keys<<<blocks_of(E), kT, 0, st>>>(edge_u, edge_v, E, L.key_a);
    uint64_t* sorted = nullptr;
    const int nb = bits_needed(n);
    rc = device_radix_sort(L.key_a, L.key_b, M, 0, nb, L.hist, L.tile_sums, st, &sorted, nullptr, nullptr, nullptr);
    if (rc != GNNCO_OK) return rc;
    uint64_t* other = sorted == L.key_a ? L.key_b : L.key_a;
    rc = device_radix_sort(sorted, other, M, 32, 32 + nb, L.hist, L.tile_sums, st, &sorted, nullptr, nullptr, nullptr);
    if (rc != GNNCO_OK) return rc;
    lv_unpack_entries<<<blocks_of(M), kT, 0, st>>>(sorted, M, L.src, L.dst);
    lv_fill_i64<<<blocks_of(M), kT, 0, st>>>(L.w, M, 1);
    GNNCO_LAUNCH_CHECK();
  }
  lv_fill_i64<<<blocks_of(N), kT, 0, st>>>(L.loop, N, 0);
  lv_iota<<<blocks_of(n), kT, 0, st>>>(part, n);
  GNNCO_LAUNCH_CHECK();
  int32_t levels = 0, sweeps_total = 0;
  int64_t qnum = 0;
  for (int32_t level = 0; level < max_levels; ++level) {
    lv_row_starts<<<blocks_of(M + 1), kT, 0, st>>>(L.src, M, N, L.rowp);
    lv_degrees<<<blocks_of(N), kT, 0, st>>>(L.rowp, L.w, L.loop, N, L.k);
    lv_iota<<<blocks_of(N), kT, 0, st>>>(L.comm, N);
    GNNCO_LAUNCH_CHECK();
    // numerator of the starting assignment (every node alone): sum_a [ 2m * 2 loop(a) - k(a)^2 ]
    auto numerator_of = [&](const int32_t* assign, int64_t* host_value) -> int32_t {
      GNNCO_CUDA_TRY(cudaMemsetAsync(L.tot, 0, (size_t)N * sizeof(int64_t), st));
      GNNCO_CUDA_TRY(cudaMemsetAsync(L.in2, 0, (size_t)N * sizeof(int64_t), st));
      GNNCO_CUDA_TRY(cudaMemsetAsync(L.qnum, 0, sizeof(int64_t), st));
      lv_community_totals<<<blocks_of(N), kT, 0, st>>>(assign, L.k, N, L.tot, nullptr);
      if (M > 0) lv_internal_entries<<<blocks_of(M), kT, 0, st>>>(L.src, L.dst, L.w, assign, M, L.in2);
      lv_internal_loops<<<blocks_of(N), kT, 0, st>>>(L.loop, assign, N, L.in2);
      lv_numerator<<<blocks_of(N), kT, 0, st>>>(L.in2, L.tot, N, two_m, L.qnum);
      GNNCO_LAUNCH_CHECK();
      GNNCO_CUDA_TRY(cudaMemcpyAsync(host_value, L.qnum, sizeof(int64_t), cudaMemcpyDeviceToHost, st));
      return GNNCO_OK;
    };
    rc = numerator_of(L.comm, &qnum);
    if (rc != GNNCO_OK) return rc;
    GNNCO_CUDA_TRY(cudaStreamSynchronize(st));
    bool moved_this_level = false;
    const int nbN = bits_needed(N);
    for (int32_t sweep = 0; sweep < max_sweeps && M > 0; ++sweep) {
      GNNCO_CUDA_TRY(cudaMemsetAsync(L.tot, 0, (size_t)N * sizeof(int64_t), st));
      GNNCO_CUDA_TRY(cudaMemsetAsync(L.size, 0, (size_t)N * sizeof(int32_t), st));
      GNNCO_CUDA_TRY(cudaMemsetAsync(L.counters, 0, 16 * sizeof(int32_t), st));
      lv_community_totals<<<blocks_of(N), kT, 0, st>>>(L.comm, L.k, N, L.tot, L.size);
      lv_sweep_keys<<<blocks_of(M), kT, 0, st>>>(L.src, L.dst, L.comm, M, L.key_a, L.idx_a);
      GNNCO_LAUNCH_CHECK();
      // entries are already grouped by node (high word); a stable sort on the community bits keeps the runs
      uint64_t* sk = nullptr;
      int32_t* si = nullptr;
      rc = device_radix_sort(L.key_a, L.key_b, M, 0, nbN, L.hist, L.tile_sums, st, &sk, L.idx_a, L.idx_b, &si);
      if (rc != GNNCO_OK) return rc;
      uint64_t* ok2 = sk == L.key_a ? L.key_b : L.key_a;
      int32_t* oi2 = si == L.idx_a ? L.idx_b : L.idx_a;
      rc = device_radix_sort(sk, ok2, M, 32, 32 + nbN, L.hist, L.tile_sums, st, &sk, si, oi2, &si);
      if (rc != GNNCO_OK) return rc;
      lv_decide<<<blocks_of(N), kT, 0, st>>>(sk, si, L.w, L.rowp, L.comm, L.k, L.tot, L.size, two_m, N, L.next, L.counters);
      GNNCO_LAUNCH_CHECK();
      GNNCO_CUDA_TRY(cudaMemcpyAsync(hc, L.counters, sizeof(int32_t), cudaMemcpyDeviceToHost, st));
      int64_t q_new = 0;
      rc = numerator_of(L.next, &q_new);
      if (rc != GNNCO_OK) return rc;
      GNNCO_CUDA_TRY(cudaStreamSynchronize(st));
      if (hc[0] == 0) break;
      if (q_new <= qnum) break;                       // the sweep as a whole did not help: undone
      GNNCO_CUDA_TRY(cudaMemcpyAsync(L.comm, L.next, (size_t)N * sizeof(int32_t), cudaMemcpyDeviceToDevice, st));
      qnum = q_new;
      moved_this_level = true;
      ++sweeps_total;
    }
    if (!moved_this_level) break;
    ++levels;
    // ---- contraction
    GNNCO_CUDA_TRY(cudaMemsetAsync(L.used, 0, (size_t)(N + 1) * sizeof(int32_t), st));
    lv_mark_used<<<blocks_of(N), kT, 0, st>>>(L.comm, N, L.used);
    GNNCO_LAUNCH_CHECK();
    rc = device_exclusive_scan(L.used, N + 1, L.tile_sums, st);         // used[c] -> new id of c; used[N] -> Nc
    if (rc != GNNCO_OK) return rc;
    int32_t Nc = 0;
    GNNCO_CUDA_TRY(cudaMemcpyAsync(&Nc, L.used + N, sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    lv_relabel_part<<<blocks_of(n), kT, 0, st>>>(part, n, L.comm, L.used);
    GNNCO_CUDA_TRY(cudaMemsetAsync(L.loop2, 0, (size_t)N * sizeof(int64_t), st));
    lv_cross_flags<<<blocks_of(M), kT, 0, st>>>(L.src, L.dst, L.comm, M, L.flag);
    GNNCO_LAUNCH_CHECK();
    int32_t last_flag = 0, last_pos = 0;
    GNNCO_CUDA_TRY(cudaMemcpyAsync(&last_flag, L.flag + (M - 1), sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    rc = device_exclusive_scan(L.flag, M, L.tile_sums, st);
    if (rc != GNNCO_OK) return rc;
    GNNCO_CUDA_TRY(cudaMemcpyAsync(&last_pos, L.flag + (M - 1), sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    lv_cross_scatter<<<blocks_of(M), kT, 0, st>>>(L.src, L.dst, L.w, L.comm, L.used, L.flag, M, L.key_a, L.idx_a, L.loop2);
    lv_halve<<<blocks_of(N), kT, 0, st>>>(L.loop2, N);
    lv_loops_down<<<blocks_of(N), kT, 0, st>>>(L.loop, L.comm, L.used, N, L.loop2);
    GNNCO_LAUNCH_CHECK();
    GNNCO_CUDA_TRY(cudaStreamSynchronize(st));
    const int64_t Mc = (int64_t)last_pos + last_flag;            // entries between different communities
    int64_t M2 = 0;
    if (Mc > 0) {
      const int nbc = bits_needed(Nc);
      uint64_t* sk = nullptr;
      int32_t* si = nullptr;
      rc = device_radix_sort(L.key_a, L.key_b, Mc, 0, nbc, L.hist, L.tile_sums, st, &sk, L.idx_a, L.idx_b, &si);
      if (rc != GNNCO_OK) return rc;
      uint64_t* ok2 = sk == L.key_a ? L.key_b : L.key_a;
      int32_t* oi2 = si == L.idx_a ? L.idx_b : L.idx_a;
      rc = device_radix_sort(sk, ok2, Mc, 32, 32 + nbc, L.hist, L.tile_sums, st, &sk, si, oi2, &si);
      if (rc != GNNCO_OK) return rc;
      lv_head_flags<<<blocks_of(Mc), kT, 0, st>>>(sk, Mc, L.flag);
      GNNCO_LAUNCH_CHECK();
      int32_t lf = 0, lp = 0;
      GNNCO_CUDA_TRY(cudaMemcpyAsync(&lf, L.flag + (Mc - 1), sizeof(int32_t), cudaMemcpyDeviceToHost, st));
      rc = device_exclusive_scan(L.flag, Mc, L.tile_sums, st);
      if (rc != GNNCO_OK) return rc;
      GNNCO_CUDA_TRY(cudaMemcpyAsync(&lp, L.flag + (Mc - 1), sizeof(int32_t), cudaMemcpyDeviceToHost, st));
      GNNCO_CUDA_TRY(cudaMemsetAsync(L.w2, 0, (size_t)Mc * sizeof(int64_t), st));
      lv_merge_entries<<<blocks_of(Mc), kT, 0, st>>>(sk, si, L.w, L.flag, Mc, L.src2, L.dst2, L.w2);
      GNNCO_LAUNCH_CHECK();
      GNNCO_CUDA_TRY(cudaStreamSynchronize(st));
      M2 = (int64_t)lp + lf;
    }
    // the contracted graph becomes the level graph
    { int32_t* t = L.src; L.src = L.src2; L.src2 = t; }
    { int32_t* t = L.dst; L.dst = L.dst2; L.dst2 = t; }
    { int64_t* t = L.w; L.w = L.w2; L.w2 = t; }
    { int64_t* t = L.loop; L.loop = L.loop2; L.loop2 = t; }
    N = Nc;
    M = M2;
  }
  GNNCO_CUDA_TRY(cudaStreamSynchronize(st));
  *S_out = (int32_t)N;
  if (qnum_out) *qnum_out = qnum;
  if (two_m_out) *two_m_out = two_m;
  if (levels_out) *levels_out = levels;
  if (sweeps_out) *sweeps_out = sweeps_total;
  return GNNCO_OK;
}
