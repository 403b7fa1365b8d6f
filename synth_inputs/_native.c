/*
 * Seeded synthetic-input helpers (graph partition growth and random fills).
 *
 * This file holds input generation only: no step of the GNN method (aggregation,
 * transform, objective, decoding, bookkeeping of intra/boundary edges) lives here.
 * Both the CUDA library's tests and the CPU oracle's tests are fed from it.
 *
 * Random numbers come from the SplitMix64 sequence (Steele, Lea, Flood 2014,
 * "Fast splittable pseudorandom number generators"): the k-th output of a stream
 * with start state `seed` is mix(seed + (k+1)*GAMMA).  Because the state advance is
 * a plain addition the sequence is random-access, which lets any slice of a large
 * tensor be regenerated on its own.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>

static inline uint64_t splitmix64_at(uint64_t seed, uint64_t k) {
  uint64_t z = seed + (k + 1ull) * 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

/* k-th raw 64-bit output, exported so Python can use the same stream. */
void synth_u64(uint64_t seed, uint64_t start, int64_t count, uint64_t* out) {
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < count; ++i) out[i] = splitmix64_at(seed, start + (uint64_t)i);
}

/* Standard normal for element index e: Box-Muller on draw e/2, cosine branch for
 * even e and sine branch for odd e. */
static inline float normal_at(uint64_t seed, uint64_t e) {
  uint64_t z = splitmix64_at(seed, e >> 1);
  double u1 = ((double)(z >> 40) + 1.0) * (1.0 / 16777216.0);          /* (0,1] */
  double u2 = (double)((z >> 8) & 0xFFFFFFull) * (1.0 / 16777216.0);   /* [0,1) */
  double r = sqrt(-2.0 * log(u1));
  double a = 6.283185307179586476925286766559 * u2;
  return (float)((e & 1ull) ? r * sin(a) : r * cos(a));
}

void synth_fill_normal_f32(uint64_t seed, uint64_t start, int64_t count, float* out) {
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < count; ++i) out[i] = normal_at(seed, start + (uint64_t)i);
}

static inline uint16_t f32_to_bf16_rne(float f) {
  uint32_t u;
  memcpy(&u, &f, 4);
  uint32_t lsb = (u >> 16) & 1u;
  u += 0x7FFFu + lsb;
  return (uint16_t)(u >> 16);
}

/* Same normals, rounded to nearest-even bfloat16 and stored as raw 16-bit patterns. */
void synth_fill_normal_bf16(uint64_t seed, uint64_t start, int64_t count, uint16_t* out) {
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < count; ++i) out[i] = f32_to_bf16_rne(normal_at(seed, start + (uint64_t)i));
}

/* Uniform in [lo, hi) for element index e. */
void synth_fill_uniform_f32(uint64_t seed, uint64_t start, int64_t count, float lo, float hi, float* out) {
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < count; ++i) {
    uint64_t z = splitmix64_at(seed, start + (uint64_t)i);
    double u = (double)(z >> 11) * (1.0 / 9007199254740992.0);
    out[i] = (float)((double)lo + u * ((double)hi - (double)lo));
  }
}

/*
 * Breadth-first grown, balanced partition of an undirected graph.
 *   - a part grows by a FIFO breadth-first search (neighbours visited in ascending id)
 *     from the lowest unassigned node id until it holds ceil(n/S) nodes;
 *   - if the search runs dry first, it restarts inside the same part from the lowest
 *     unassigned id;
 *   - when a part is full, the nodes still waiting in the queue are released and the
 *     next part starts a fresh search from the lowest unassigned id.
 * part_out[i] receives the part of node i.  Returns 0, or -1 on allocation failure
 * or an edge endpoint outside [0, n).
 */
int synth_bfs_partition(int64_t n, int64_t E, const int32_t* eu, const int32_t* ev, int32_t S, int32_t* part_out) {
  if (n <= 0 || S <= 0) return -1;
  int64_t* ptr = (int64_t*)calloc((size_t)n + 1, sizeof(int64_t));
  int32_t* adj = (int32_t*)malloc((size_t)(2 * E + 1) * sizeof(int32_t));
  int32_t* tmp = (int32_t*)malloc((size_t)(2 * E + 1) * sizeof(int32_t));
  int32_t* tmp_row = (int32_t*)malloc((size_t)(2 * E + 1) * sizeof(int32_t));
  int32_t* queue = (int32_t*)malloc((size_t)n * sizeof(int32_t));
  uint8_t* seen = (uint8_t*)calloc((size_t)n, 1);
  uint8_t* done_ = (uint8_t*)calloc((size_t)n, 1);
  int rc = -1;
  if (!ptr || !adj || !tmp || !tmp_row || !queue || !seen || !done_) goto done;
  for (int64_t e = 0; e < E; ++e)
    if (eu[e] < 0 || eu[e] >= n || ev[e] < 0 || ev[e] >= n) goto done;
  /* pass 1: stable counting sort of the 2E directed pairs by neighbour id */
  {
    int64_t* cnt = (int64_t*)calloc((size_t)n + 1, sizeof(int64_t));
    if (!cnt) goto done;
    for (int64_t e = 0; e < E; ++e) { cnt[ev[e] + 1]++; cnt[eu[e] + 1]++; }
    for (int64_t i = 0; i < n; ++i) cnt[i + 1] += cnt[i];
    for (int64_t e = 0; e < E; ++e) {
      int64_t a = cnt[ev[e]]++; tmp_row[a] = eu[e]; tmp[a] = ev[e];   /* row u, neighbour v */
      int64_t b = cnt[eu[e]]++; tmp_row[b] = ev[e]; tmp[b] = eu[e];   /* row v, neighbour u */
    }
    free(cnt);
  }
  /* pass 2: stable counting sort by row -> rows hold neighbours in ascending id */
  for (int64_t k = 0; k < 2 * E; ++k) ptr[tmp_row[k] + 1]++;
  for (int64_t i = 0; i < n; ++i) ptr[i + 1] += ptr[i];
  {
    int64_t* fill = (int64_t*)malloc((size_t)n * sizeof(int64_t));
    if (!fill) goto done;
    memcpy(fill, ptr, (size_t)n * sizeof(int64_t));
    for (int64_t k = 0; k < 2 * E; ++k) adj[fill[tmp_row[k]]++] = tmp[k];
    free(fill);
  }
  {
    int64_t target = (n + S - 1) / S, filled = 0, head = 0, tail = 0, next_seed = 0;
    int32_t cur = 0;
    int64_t assigned = 0;
    while (assigned < n) {
      if (head == tail) {
        while (done_[next_seed]) ++next_seed;
        seen[next_seed] = 1;
        queue[tail++] = (int32_t)next_seed;
      }
      if (filled == target && cur < S - 1) {
        /* part complete: release the waiting nodes, start the next part afresh */
        for (int64_t k = head; k < tail; ++k) seen[queue[k]] = 0;
        head = tail = 0;
        ++cur; filled = 0;
        continue;
      }
      int32_t v = queue[head++];
      part_out[v] = cur; done_[v] = 1;
      ++filled; ++assigned;
      for (int64_t k = ptr[v]; k < ptr[v + 1]; ++k) {
        int32_t w = adj[k];
        if (!seen[w]) { seen[w] = 1; queue[tail++] = w; }
      }
    }
  }
  rc = 0;
done:
  free(ptr); free(adj); free(tmp); free(tmp_row); free(queue); free(seen); free(done_);
  return rc;
}
