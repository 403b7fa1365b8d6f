/*
 * CPU oracle for the partitioned-GNN train step.  TEST INFRASTRUCTURE ONLY.
 *
 * Plain, slow, double-precision restatement of what the hot path computes, written
 * from the paper's definitions.  It shares no code, header, table or helper with the
 * CUDA library; only tests, the smoke check and the benchmark's CPU-baseline leg may
 * call it.  Every function cites the passage it follows.
 *
 * Conventions
 *   - nodes are renumbered so that each subgraph (partition) is a contiguous id range;
 *     `part_ptr[s] .. part_ptr[s+1]` is subgraph s;
 *   - only intra-subgraph edges take part in training (Section 3.3: each subgraph is
 *     trained on its own, edges to other subgraphs play no part); cross edges are kept aside as
 *     the boundary list that decoding inspects;
 *   - dense matrices are row-major.
 *
 * Pins (see tests, "not gpu"): finite differences for every gradient, closed forms at
 * W = 0, row-stochastic aggregation, per-subgraph runs equal the batched run, brute
 * force on graphs of at most 16 nodes, hand-computed Adam steps, brute-force decode;
 * the bfloat16-storage mode: exact rational rounding, a dense restatement with the rounding
 * written out at the stored tensors, and bit-equality with the plain mode on inputs whose
 * stored values are all bfloat16 numbers.
 * Parity unpinned: nothing here can be compared with the paper's result tables
 * (they need the original datasets, trained weights and the RL stage).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORACLE_OK = 0, ORACLE_BAD_ARG = -1, ORACLE_OUT_OF_RANGE = -2, ORACLE_NOT_SIMPLE = -3, ORACLE_NOMEM = -6 };

static int cmp_i32(const void* a, const void* b) {
  int32_t x = *(const int32_t*)a, y = *(const int32_t*)b;
  return (x > y) - (x < y);
}
static int cmp_pair(const void* a, const void* b) {
  const int32_t* x = (const int32_t*)a;
  const int32_t* y = (const int32_t*)b;
  if (x[0] != y[0]) return (x[0] > y[0]) - (x[0] < y[0]);
  return (x[1] > y[1]) - (x[1] < y[1]);
}

/* Round a double to bfloat16 the way a value that was accumulated in float32 and is then STORED
 * in bfloat16 gets there: first to the nearest float (ties to even), then that float to the
 * nearest bfloat16 (8 significant bits, float's exponent range; ties to even; overflow gives
 * infinity), returned as double.  Used only where a workload fixes bfloat16 storage of
 * activations with float32 accumulation. */
static double round_bf16(double x) {
  float f = (float)x;
  uint32_t u;
  memcpy(&u, &f, 4);
  if ((u & 0x7F800000u) == 0x7F800000u) return (double)f;      /* inf / nan unchanged */
  u += 0x7FFFu + ((u >> 16) & 1u);
  u &= 0xFFFF0000u;
  memcpy(&f, &u, 4);
  return (double)f;
}

/* round_bf16 for the pins (exact rational arithmetic checks it from outside). */
double oracle_round_bf16(double x) { return round_bf16(x); }

/*
 * Bookkeeping (Section 3.3, first paragraph: the graph is split into subgraphs, and
 * "cross-nodes" are the endpoints of edges whose ends lie in different subgraphs;
 * Algorithm 1, Stage 2: global mask and cross-node mask).
 *
 *   new id of a node   = its rank under the key (part, original id)
 *   perm[new] = original id, inv_perm[original] = new id
 *   intra edge         = part[u] == part[v]: stored in both directions in a CSR with
 *                        ascending columns and no self loops
 *   boundary edge      = otherwise: stored once as (min, max) of the new ids, the list
 *                        sorted lexicographically
 *   inv_deg[i]         = 1 / (intra degree of i + 1)   (Eq. 3's 1/(|N(i)|+1)), in float
 *   is_boundary[i]     = 1 iff i is an endpoint of a boundary edge
 * colidx must hold 2E entries and bnd_u/bnd_v E entries (worst case).
 */
int oracle_bookkeeping(int64_t n, int64_t E, const int32_t* eu, const int32_t* ev, const int32_t* part, int32_t S,
                       int32_t* perm, int32_t* inv_perm, int32_t* part_ptr, int32_t* node_part, int32_t* rowptr,
                       int32_t* colidx, int32_t* bnd_u, int32_t* bnd_v, float* inv_deg, uint8_t* is_boundary,
                       int64_t* E_in_out, int64_t* E_b_out) {
  if (n <= 0 || E < 0 || S <= 0) return ORACLE_BAD_ARG;
  for (int64_t i = 0; i < n; ++i)
    if (part[i] < 0 || part[i] >= S) return ORACLE_OUT_OF_RANGE;
  for (int64_t e = 0; e < E; ++e) {
    if (eu[e] < 0 || eu[e] >= n || ev[e] < 0 || ev[e] >= n) return ORACLE_OUT_OF_RANGE;
    if (eu[e] == ev[e]) return ORACLE_NOT_SIMPLE;
  }
  /* subgraph sizes -> start offsets */
  for (int32_t s = 0; s <= S; ++s) part_ptr[s] = 0;
  for (int64_t i = 0; i < n; ++i) part_ptr[part[i] + 1]++;
  for (int32_t s = 0; s < S; ++s) part_ptr[s + 1] += part_ptr[s];
  /* rank under (part, original id): walk original ids upward, append to the node's part */
  int32_t* fill = (int32_t*)malloc((size_t)S * sizeof(int32_t));
  if (!fill) return ORACLE_NOMEM;
  memcpy(fill, part_ptr, (size_t)S * sizeof(int32_t));
  for (int64_t i = 0; i < n; ++i) {
    int32_t id = fill[part[i]]++;
    inv_perm[i] = id;
    perm[id] = (int32_t)i;
    node_part[id] = part[i];
  }
  free(fill);
  /* classify edges, count intra degree */
  for (int64_t i = 0; i <= n; ++i) rowptr[i] = 0;
  memset(is_boundary, 0, (size_t)n);
  int64_t E_in = 0, E_b = 0;
  int32_t* bpairs = (int32_t*)malloc((size_t)(2 * E + 2) * sizeof(int32_t));
  if (!bpairs) return ORACLE_NOMEM;
  for (int64_t e = 0; e < E; ++e) {
    int32_t a = inv_perm[eu[e]], b = inv_perm[ev[e]];
    if (part[eu[e]] == part[ev[e]]) {
      rowptr[a + 1]++; rowptr[b + 1]++; ++E_in;
    } else {
      bpairs[2 * E_b] = a < b ? a : b;
      bpairs[2 * E_b + 1] = a < b ? b : a;
      is_boundary[a] = 1; is_boundary[b] = 1;
      ++E_b;
    }
  }
  for (int64_t i = 0; i < n; ++i) rowptr[i + 1] += rowptr[i];
  int32_t* pos = (int32_t*)malloc((size_t)n * sizeof(int32_t));
  if (!pos) { free(bpairs); return ORACLE_NOMEM; }
  memcpy(pos, rowptr, (size_t)n * sizeof(int32_t));
  for (int64_t e = 0; e < E; ++e) {
    if (part[eu[e]] != part[ev[e]]) continue;
    int32_t a = inv_perm[eu[e]], b = inv_perm[ev[e]];
    colidx[pos[a]++] = b;
    colidx[pos[b]++] = a;
  }
  free(pos);
  int status = ORACLE_OK;
  for (int64_t i = 0; i < n; ++i) {
    int32_t lo = rowptr[i], hi = rowptr[i + 1];
    qsort(colidx + lo, (size_t)(hi - lo), sizeof(int32_t), cmp_i32);
    for (int32_t k = lo + 1; k < hi; ++k)
      if (colidx[k] == colidx[k - 1]) status = ORACLE_NOT_SIMPLE;   /* repeated edge */
    inv_deg[i] = 1.0f / (float)(hi - lo + 1);
  }
  qsort(bpairs, (size_t)E_b, 2 * sizeof(int32_t), cmp_pair);
  for (int64_t k = 0; k < E_b; ++k) {
    bnd_u[k] = bpairs[2 * k];
    bnd_v[k] = bpairs[2 * k + 1];
    if (k > 0 && bnd_u[k] == bnd_u[k - 1] && bnd_v[k] == bnd_v[k - 1]) status = ORACLE_NOT_SIMPLE;
  }
  free(bpairs);
  *E_in_out = E_in;
  *E_b_out = E_b;
  return status;
}

/*
 * One subgraph, standalone (local node ids 0..ns-1, local CSR): forward (Eq. 3 per
 * hidden layer, Eq. 4 on the last layer's scalar output), objective (Eq. 5 plus the
 * fine-tuning penalty of Section 3.3), and the exact reverse-mode derivative of that
 * scalar with respect to every weight matrix and, optionally, the input embeddings.
 *
 * Readings of the paper taken here:
 *   - hidden layers: h = ReLU( mean_{self+neighbours}(h_prev) W )          (Eq. 3)
 *   - last layer (output width 1): z = mean_{self+neighbours}(h_prev) w, no ReLU;
 *     p = 1/(1+exp(-z))                                                     (Eq. 4)
 *   - loss = alpha * sum_{edges, each once} p_i p_j - beta * sum_i p_i
 *            + lambda * sum_i pen_i p_i                                     (Eq. 5, penalty)
 *   - ReLU derivative is 1 where the pre-activation is > 0, else 0.
 * W[l] points at this subgraph's F_l x F_{l+1} matrix of layer l (0-based).
 * dW[l] (if dW != NULL) receives the gradient; dX (if != NULL) receives d loss / d X.
 * Zsave[l] (if Zsave != NULL), l < L-1, receives the pre-activations of hidden layer l.
 *
 * store_bf16 != 0 models a workload whose activations are STORED in bfloat16 while all
 * sums are carried at higher precision (the "bf16 embeddings, fp32 accumulation"
 * benchmark configuration): the aggregated input M_l and the activation H_l of every
 * hidden layer are rounded to the nearest bfloat16 before they are used again.  The
 * ReLU mask is a 0/1 decision taken from floating point, so it must be taken on values
 * of the same precision on both sides of a comparison.  Everything else stays double.
 */
static int subgraph_step(int32_t ns, const int32_t* rp, const int32_t* ci, int32_t L, const int32_t* dims,
                         const double* X, const double* const* W, double alpha, double beta, double lambda,
                         const double* pen, double* loss_out, double* z_out, double* p_out, double* const* dW,
                         double* dX, double* const* Zsave, int store_bf16) {
  int rc = ORACLE_OK;
  double** H = (double**)calloc((size_t)L + 1, sizeof(double*));   /* H[0] = X, H[l] = output of layer l */
  double** M = (double**)calloc((size_t)L + 1, sizeof(double*));   /* M[l] = aggregated input of layer l (1-based) */
  double** Z = (double**)calloc((size_t)L + 1, sizeof(double*));   /* Z[l] = M[l] W[l-1] */
  if (!H || !M || !Z) { rc = ORACLE_NOMEM; goto done; }
  H[0] = (double*)X;
  for (int32_t l = 1; l <= L; ++l) {
    int32_t fi = dims[l - 1], fo = dims[l];
    M[l] = (double*)calloc((size_t)ns * fi + 1, sizeof(double));
    Z[l] = (double*)calloc((size_t)ns * fo + 1, sizeof(double));
    if (l < L) H[l] = (double*)calloc((size_t)ns * fo + 1, sizeof(double));
    if (!M[l] || !Z[l] || (l < L && !H[l])) { rc = ORACLE_NOMEM; goto done; }
    const double* Hp = H[l - 1];
    const double* Wl = W[l - 1];
    for (int32_t i = 0; i < ns; ++i) {
      double* m = M[l] + (size_t)i * fi;
      for (int32_t f = 0; f < fi; ++f) m[f] = Hp[(size_t)i * fi + f];
      for (int32_t k = rp[i]; k < rp[i + 1]; ++k) {
        const double* hj = Hp + (size_t)ci[k] * fi;
        for (int32_t f = 0; f < fi; ++f) m[f] += hj[f];
      }
      double inv = 1.0 / (double)(rp[i + 1] - rp[i] + 1);
      for (int32_t f = 0; f < fi; ++f) m[f] *= inv;
      if (store_bf16 && l < L)
        for (int32_t f = 0; f < fi; ++f) m[f] = round_bf16(m[f]);     /* aggregated tensor is stored */
      double* zr = Z[l] + (size_t)i * fo;
      for (int32_t f = 0; f < fi; ++f) {
        double mf = m[f];
        const double* wrow = Wl + (size_t)f * fo;
        for (int32_t h = 0; h < fo; ++h) zr[h] += mf * wrow[h];
      }
      if (l < L) {
        double* hr = H[l] + (size_t)i * fo;
        for (int32_t h = 0; h < fo; ++h) hr[h] = zr[h] > 0.0 ? zr[h] : 0.0;
        if (store_bf16)
          for (int32_t h = 0; h < fo; ++h) hr[h] = round_bf16(hr[h]);   /* activation is stored */
      }
    }
    if (l < L && Zsave && Zsave[l - 1]) memcpy(Zsave[l - 1], Z[l], (size_t)ns * fo * sizeof(double));
  }
  if (dims[L] != 1) { rc = ORACLE_BAD_ARG; goto done; }
  {
    double* p = p_out;
    for (int32_t i = 0; i < ns; ++i) {
      double z = Z[L][i];
      if (z_out) z_out[i] = z;
      p[i] = 1.0 / (1.0 + exp(-z));
    }
    double edge_term = 0.0, node_term = 0.0, pen_term = 0.0;
    for (int32_t i = 0; i < ns; ++i) {
      for (int32_t k = rp[i]; k < rp[i + 1]; ++k)
        if (ci[k] > i) edge_term += p[i] * p[ci[k]];
      node_term += p[i];
      if (pen) pen_term += pen[i] * p[i];
    }
    *loss_out = alpha * edge_term - beta * node_term + lambda * pen_term;
    if (!dW && !dX) goto done;
    /* backward */
    double* dZ = (double*)calloc((size_t)ns + 1, sizeof(double));   /* gradient wrt Z[L] */
    if (!dZ) { rc = ORACLE_NOMEM; goto done; }
    for (int32_t i = 0; i < ns; ++i) {
      double nb = 0.0;
      for (int32_t k = rp[i]; k < rp[i + 1]; ++k) nb += p[ci[k]];
      double dp = alpha * nb - beta + (pen ? lambda * pen[i] : 0.0);
      dZ[i] = dp * p[i] * (1.0 - p[i]);
    }
    for (int32_t l = L; l >= 1; --l) {
      int32_t fi = dims[l - 1], fo = dims[l];
      const double* Wl = W[l - 1];
      if (dW && dW[l - 1]) {
        double* g = dW[l - 1];
        for (size_t q = 0; q < (size_t)fi * fo; ++q) g[q] = 0.0;
        for (int32_t i = 0; i < ns; ++i)
          for (int32_t f = 0; f < fi; ++f) {
            double mf = M[l][(size_t)i * fi + f];
            for (int32_t h = 0; h < fo; ++h) g[(size_t)f * fo + h] += mf * dZ[(size_t)i * fo + h];
          }
      }
      if (l == 1 && !dX) break;
      /* dM = dZ W^T, then through the transpose of the mean aggregation */
      double* dH = (double*)calloc((size_t)ns * fi + 1, sizeof(double));
      double* dm = (double*)malloc((size_t)fi * sizeof(double) + 8);
      if (!dH || !dm) { free(dH); free(dm); free(dZ); rc = ORACLE_NOMEM; goto done; }
      for (int32_t i = 0; i < ns; ++i) {
        for (int32_t f = 0; f < fi; ++f) {
          double acc = 0.0;
          for (int32_t h = 0; h < fo; ++h) acc += dZ[(size_t)i * fo + h] * Wl[(size_t)f * fo + h];
          dm[f] = acc / (double)(rp[i + 1] - rp[i] + 1);
        }
        /* row i of the mean used itself and each neighbour with the same weight */
        for (int32_t f = 0; f < fi; ++f) dH[(size_t)i * fi + f] += dm[f];
        for (int32_t k = rp[i]; k < rp[i + 1]; ++k) {
          double* dj = dH + (size_t)ci[k] * fi;
          for (int32_t f = 0; f < fi; ++f) dj[f] += dm[f];
        }
      }
      free(dm);
      free(dZ);
      if (l == 1) {
        memcpy(dX, dH, (size_t)ns * fi * sizeof(double));
        free(dH);
        dZ = NULL;
      } else {
        for (size_t q = 0; q < (size_t)ns * fi; ++q)
          if (!(Z[l - 1][q] > 0.0)) dH[q] = 0.0;
        dZ = dH;
      }
    }
    free(dZ);
  }
done:
  if (H) for (int32_t l = 1; l <= L; ++l) free(H[l]);
  if (M) for (int32_t l = 1; l <= L; ++l) free(M[l]);
  if (Z) for (int32_t l = 1; l <= L; ++l) free(Z[l]);
  free(H); free(M); free(Z);
  return rc;
}

/* Standalone single-subgraph entry (used by the "batch equals per-subgraph runs" pin). */
int oracle_subgraph_step(int32_t ns, const int32_t* rowptr, const int32_t* colidx, int32_t L, const int32_t* dims,
                         const double* X, const double* const* W, double alpha, double beta, double lambda,
                         const double* pen, double* loss, double* z, double* p, double* const* dW, double* dX,
                         double* const* Zsave, int32_t store_bf16) {
  if (ns <= 0 || L < 1) return ORACLE_BAD_ARG;
  return subgraph_step(ns, rowptr, colidx, L, dims, X, W, alpha, beta, lambda, pen, loss, z, p, dW, dX, Zsave,
                       store_bf16);
}

/*
 * Block-diagonal batch: every subgraph of the partitioned graph, each with its own
 * weight set (Algorithm 1, Stage 1: one model per subgraph) or all sharing one
 * (weight_sets == 1, gradients summed over subgraphs).
 *   X [n x F_0], z/p [n], loss [S]; W[l] is [weight_sets x F_l x F_{l+1}];
 *   dW[l] the same shape; dX [n x F_0]; Zsave[l] [n x F_{l+1}] for hidden layers.
 * Subgraphs are independent, so the outer loop may run on several threads; the
 * arithmetic inside one subgraph is untouched.  Returns the thread count used (> 0)
 * or a negative error.
 */
int oracle_train_step(int64_t n, int32_t S, const int32_t* part_ptr, const int32_t* rowptr, const int32_t* colidx,
                      int32_t L, const int32_t* dims, int32_t weight_sets, const double* X, const double* const* W,
                      double alpha, double beta, double lambda, const double* pen, double* loss, double* z, double* p,
                      double* const* dW, double* dX, double* const* Zsave, int32_t threads, int32_t store_bf16) {
  if (n <= 0 || S <= 0 || L < 1 || L > 16 || (weight_sets != 1 && weight_sets != S)) return ORACLE_BAD_ARG;
  int rc = ORACLE_OK;
  int used = 1;
  if (dW && weight_sets == 1)
    for (int32_t l = 0; l < L; ++l)
      if (dW[l]) memset(dW[l], 0, (size_t)dims[l] * dims[l + 1] * sizeof(double));
#ifdef _OPENMP
  if (threads < 1) threads = 1;
#pragma omp parallel for schedule(dynamic, 1) num_threads(threads)
#endif
  for (int32_t s = 0; s < S; ++s) {
#ifdef _OPENMP
    if (s == 0 || omp_get_thread_num() == 0) {
#pragma omp atomic write
      used = omp_get_num_threads();
    }
#endif
    int32_t r0 = part_ptr[s], r1 = part_ptr[s + 1], ns = r1 - r0;
    if (ns <= 0) { loss[s] = 0.0; continue; }
    int32_t base = rowptr[r0];
    int32_t nnz = rowptr[r1] - base;
    int32_t* rp = (int32_t*)malloc((size_t)(ns + 1) * sizeof(int32_t));
    int32_t* ci = (int32_t*)malloc((size_t)(nnz + 1) * sizeof(int32_t));
    const double* Ws[16];
    double* dWs[16];
    double* Zs[16];
    int bad = (!rp || !ci);
    if (!bad) {
      for (int32_t i = 0; i <= ns; ++i) rp[i] = rowptr[r0 + i] - base;
      for (int32_t k = 0; k < nnz; ++k) {
        ci[k] = colidx[base + k] - r0;
        if (ci[k] < 0 || ci[k] >= ns) bad = 1;   /* an intra edge must stay inside its subgraph */
      }
    }
    if (bad) {
#pragma omp critical
      rc = ORACLE_BAD_ARG;
      free(rp); free(ci);
      continue;
    }
    for (int32_t l = 0; l < L; ++l) {
      size_t wsz = (size_t)dims[l] * dims[l + 1];
      Ws[l] = W[l] + (weight_sets == 1 ? 0 : (size_t)s * wsz);
      dWs[l] = NULL;
      if (dW && dW[l]) dWs[l] = weight_sets == 1 ? (double*)malloc(wsz * sizeof(double)) : dW[l] + (size_t)s * wsz;
      Zs[l] = (Zsave && l < L - 1 && Zsave[l]) ? Zsave[l] + (size_t)r0 * dims[l + 1] : NULL;
    }
    int r = subgraph_step(ns, rp, ci, L, dims, X + (size_t)r0 * dims[0], Ws, alpha, beta, lambda,
                          pen ? pen + r0 : NULL, loss + s, z ? z + r0 : NULL, p + r0, dW ? dWs : NULL,
                          dX ? dX + (size_t)r0 * dims[0] : NULL, Zsave ? Zs : NULL, store_bf16);
    if (r != ORACLE_OK) {
#pragma omp critical
      rc = r;
    }
    if (dW && weight_sets == 1) {
      for (int32_t l = 0; l < L; ++l) {
        if (!dWs[l]) continue;
        size_t wsz = (size_t)dims[l] * dims[l + 1];
#pragma omp critical
        for (size_t q = 0; q < wsz; ++q) dW[l][q] += dWs[l][q];
        free(dWs[l]);
      }
    }
    free(rp); free(ci);
  }
  return rc != ORACLE_OK ? rc : used;
}

/*
 * Adam with bias correction (Section 3.2 only says that W is updated by backpropagation
 * and names no optimiser; the benchmark configurations
 * fix Adam).  t is the 1-based step number.
 *   m <- b1 m + (1-b1) g;  v <- b2 v + (1-b2) g^2
 *   W <- W - lr * (m / (1-b1^t)) / (sqrt(v / (1-b2^t)) + eps)
 */
void oracle_adam(int64_t count, double* W, double* m, double* v, const double* g, double lr, double b1, double b2,
                 double eps, int64_t t) {
  double c1 = 1.0 - pow(b1, (double)t), c2 = 1.0 - pow(b2, (double)t);
  for (int64_t q = 0; q < count; ++q) {
    m[q] = b1 * m[q] + (1.0 - b1) * g[q];
    v[q] = b2 * v[q] + (1.0 - b2) * g[q] * g[q];
    W[q] -= lr * (m[q] / c1) / (sqrt(v[q] / c2) + eps);
  }
}

/*
 * Decoding and conflict counting (Section 3.3: a probability of at least 0.5 becomes one, anything
 * below zero; a cross edge whose two endpoints are both selected is a conflict; Section 4.1: MIS size and conflicts are the reported metrics).
 *   x[i]        = p[i] >= threshold   (compared on the stored float value)
 *   viol[e]     = x[bnd_u[e]] & x[bnd_v[e]]
 *   per_part[s] = number of violated boundary edges with an endpoint in s (an edge
 *                 counts once for each of its two subgraphs)
 *   counts      = { sum x, violated intra edges (each once), violated boundary edges }
 */
void oracle_decode(int64_t n, int32_t S, const int32_t* node_part, const int32_t* rowptr, const int32_t* colidx,
                   int64_t E_b, const int32_t* bnd_u, const int32_t* bnd_v, const float* p, float threshold,
                   uint8_t* x, uint8_t* viol, int32_t* per_part, int64_t* counts) {
  int64_t set_size = 0, intra = 0, bviol = 0;
  for (int64_t i = 0; i < n; ++i) {
    x[i] = p[i] >= threshold ? 1 : 0;
    set_size += x[i];
  }
  for (int64_t i = 0; i < n; ++i)
    for (int32_t k = rowptr[i]; k < rowptr[i + 1]; ++k)
      if (colidx[k] > i && x[i] && x[colidx[k]]) ++intra;
  for (int32_t s = 0; s < S; ++s) per_part[s] = 0;
  for (int64_t e = 0; e < E_b; ++e) {
    uint8_t v = (uint8_t)(x[bnd_u[e]] & x[bnd_v[e]]);
    if (viol) viol[e] = v;
    if (v) {
      ++bviol;
      per_part[node_part[bnd_u[e]]]++;
      per_part[node_part[bnd_v[e]]]++;
    }
  }
  counts[0] = set_size;
  counts[1] = intra;
  counts[2] = bviol;
}

/*
 * Stage-3 glue (Algorithm 1, Stage 3, first lines; Section 3.3).
 *
 * Conflict list: the boundary edges whose two endpoints are both selected, as ascending
 * indices into the boundary list (Algorithm 1, Stage 3 derives them from the global mask; the set C of Section 3.3).
 * Returns their number.
 */
int64_t oracle_conflict_list(int64_t E_b, const uint8_t* viol, int32_t* conflict_idx) {
  int64_t c = 0;
  for (int64_t e = 0; e < E_b; ++e)
    if (viol[e]) conflict_idx[c++] = (int32_t)e;
  return c;
}

/*
 * Base action (Algorithm 1, Stage 3 starts the agent from one, obtained with a cover heuristic it
 * does not spell out).  A rule of this build's own stands in for it: for every conflict edge (u, v) the endpoint with the SMALLER probability is
 * the one to push below the threshold; on equal probabilities the endpoint with the larger
 * id.  action = 0 chooses u (the lower id of the stored pair), 1 chooses v.  Every conflict
 * loses one endpoint, so removing all chosen nodes leaves no violated boundary edge.
 */
void oracle_base_action(int64_t count, const int32_t* conflict_idx, const int32_t* bnd_u, const int32_t* bnd_v,
                        const float* p, uint8_t* action) {
  for (int64_t c = 0; c < count; ++c) {
    int32_t u = bnd_u[conflict_idx[c]], v = bnd_v[conflict_idx[c]];
    action[c] = p[u] < p[v] ? 0 : 1;
  }
}

/*
 * Actions -> fine-tuning inputs (Section 3.3: each conflict offers two options, fine-tune the
 * subgraph of node i or of node j so that this node's probability falls below the threshold;
 * Algorithm 1, Stage 3 then groups the actions by subgraph).  pen[i] = 1 for every chosen node (the node
 * list of the penalty term), 0 elsewhere; active[s] = 1 for every subgraph that holds a chosen
 * node (the subgraphs whose models are fine-tuned).  Returns the number of distinct chosen nodes.
 */
int64_t oracle_apply_actions(int64_t n, int32_t S, int64_t count, const int32_t* conflict_idx, const uint8_t* action,
                             const int32_t* bnd_u, const int32_t* bnd_v, const int32_t* node_part, float* pen,
                             uint8_t* active) {
  for (int64_t i = 0; i < n; ++i) pen[i] = 0.0f;
  for (int32_t s = 0; s < S; ++s) active[s] = 0;
  int64_t chosen = 0;
  for (int64_t c = 0; c < count; ++c) {
    int32_t node = action[c] ? bnd_v[conflict_idx[c]] : bnd_u[conflict_idx[c]];
    if (pen[node] == 0.0f) ++chosen;
    pen[node] = 1.0f;
    active[node_part[node]] = 1;
  }
  return chosen;
}

/*
 * Non-learned repair (Section 3.3: acting on conflict (i, j) takes node i, or node j, out of the
 * candidate set and so removes the conflict; Algorithm 1, Stage 3 starts from a base action).  Carrying the chosen actions out on the bit mask itself, without fine-tuning:
 * x[i] <- 0 for every chosen node i (pen[i] != 0).  Returns how many selected nodes were removed.
 */
int64_t oracle_repair(int64_t n, const float* pen, uint8_t* x) {
  int64_t removed = 0;
  for (int64_t i = 0; i < n; ++i)
    if (pen[i] != 0.0f && x[i]) {
      x[i] = 0;
      ++removed;
    }
  return removed;
}

/*
 * Quality of a partition in the terms of Section 3.1 (the quantities of Eq. 1): for every
 * community s, in_edges[s] = number of edges with both ends in s and tot[s] = Sigma_tot = sum of
 * the degrees of its nodes; m = E.  With Sigma_in = 2 * in_edges (every internal edge seen from
 * both ends, the convention under which a bracket of Eq. 1 is one community's share), the
 * modularity is  Q = sum_s [ Sigma_in(s) / 2m - (Sigma_tot(s) / 2m)^2 ].  Works on the ORIGINAL
 * edge list and part vector.  Returns Q (0 for a graph without edges).
 */
double oracle_partition_quality(int64_t E, const int32_t* eu, const int32_t* ev, const int32_t* part, int32_t S,
                                int64_t* in_edges, int64_t* tot) {
  for (int32_t s = 0; s < S; ++s) in_edges[s] = tot[s] = 0;
  for (int64_t e = 0; e < E; ++e) {
    int32_t a = part[eu[e]], b = part[ev[e]];
    if (a == b) in_edges[a] += 1;
    tot[a] += 1;
    tot[b] += 1;
  }
  if (E == 0) return 0.0;
  double two_m = 2.0 * (double)E, q = 0.0;
  for (int32_t s = 0; s < S; ++s) {
    double share = (double)tot[s] / two_m;
    q += 2.0 * (double)in_edges[s] / two_m - share * share;
  }
  return q;
}

/*
 * Louvain partitioning (Section 3.1, Eqs. 1-2), in a form whose result is uniquely defined.
 *
 * The method of Section 3.1 repeats two phases: nodes move, one by one, to the neighbouring
 * community with the largest modularity gain (Eq. 2), and then every community is contracted
 * into one node of a smaller weighted graph.  The one-by-one phase depends on a visiting order
 * that the paper does not fix, so its result is not unique.  The reading taken here makes every
 * sweep a function of the state before it (all nodes decide from the same frozen state, then
 * all moves are applied together) and compares gains exactly:
 *
 *   level graph   nodes 0..N-1, integer edge weights w(a,b) (1 on the input graph), self-loop
 *                 weights loop(a) (0 on the input graph); degree k_a = sum_{b != a} w(a,b) + 2 loop(a);
 *                 2m = sum_a k_a, the same on every level.
 *   sweep         every node a starts a level in its own community.  With the state frozen
 *                 (comm, tot[c] = sum of k over c, size[c]), node a collects kin[c] = sum of w(a,b)
 *                 over neighbours b != a with comm[b] = c, and scores its own community and every
 *                 community with kin > 0 by Eq. 2 times 2 m^2, an integer:
 *                     score(c) = 2m * kin[c] - (tot[c] - [c == comm[a]] k_a) * k_a
 *                 (the node is taken out of its own community first).  It moves to the best-scoring
 *                 community, the LOWEST id among equals, if that is not its own and scores strictly
 *                 higher than its own; a node alone in its community does not move to a community of
 *                 one node with a HIGHER id (two single nodes would swap places for ever otherwise).
 *   acceptance    after the moves of a sweep are applied the modularity numerator
 *                     Qnum = sum_c [ 2m * in2(c) - tot(c)^2 ],   Q = Qnum / (2m)^2,
 *                 in2(c) = twice the weight inside c (Eq. 1's Sigma_in counted from both ends, self loops
 *                 twice), is recomputed exactly; a sweep that does not raise it strictly is undone and
 *                 ends the level, as does a sweep without a move or the sweep limit.
 *   contraction   communities that are not empty become the nodes of the next level, numbered in
 *                 ascending order of their ids; weights between two communities add up, weight inside a
 *                 community becomes its self loop.  The procedure ends when a level moves nothing (or at
 *                 the level limit).
 *
 * Input: simple undirected graph as an edge list (each edge once).  Output: part[i] in [0, S) for the
 * original nodes, S (returned), and *qnum_out / *two_m_out so that Q = qnum / two_m^2.
 * levels_out / sweeps_out (optional) receive the number of levels that moved something and the
 * number of accepted sweeps.  Returns S, or a negative error.
 */
typedef struct {
  int64_t N;
  int64_t* rp;      /* [N+1] */
  int32_t* ci;      /* neighbours b != a */
  int64_t* w;       /* weights */
  int64_t* loop;    /* [N] */
} lv_graph;

static void lv_free(lv_graph* g) { free(g->rp); free(g->ci); free(g->w); free(g->loop); g->rp = NULL; g->ci = NULL; g->w = NULL; g->loop = NULL; }

/* level graph from a list of M undirected weighted edges (a != b allowed to repeat: weights add up;
 * a == b goes to the self loop) */
static int lv_build(int64_t N, int64_t M, const int32_t* ea, const int32_t* eb, const int64_t* ew, lv_graph* g) {
  g->N = N;
  g->rp = (int64_t*)calloc((size_t)N + 1, sizeof(int64_t));
  g->loop = (int64_t*)calloc((size_t)N + 1, sizeof(int64_t));
  if (!g->rp || !g->loop) return ORACLE_NOMEM;
  for (int64_t e = 0; e < M; ++e) {
    if (ea[e] == eb[e]) { g->loop[ea[e]] += ew[e]; continue; }
    g->rp[ea[e] + 1]++; g->rp[eb[e] + 1]++;
  }
  for (int64_t a = 0; a < N; ++a) g->rp[a + 1] += g->rp[a];
  int64_t nnz = g->rp[N];
  int32_t* tci = (int32_t*)malloc((size_t)(nnz + 1) * sizeof(int32_t));
  int64_t* tw = (int64_t*)malloc((size_t)(nnz + 1) * sizeof(int64_t));
  int64_t* pos = (int64_t*)malloc((size_t)(N + 1) * sizeof(int64_t));
  if (!tci || !tw || !pos) { free(tci); free(tw); free(pos); return ORACLE_NOMEM; }
  memcpy(pos, g->rp, (size_t)N * sizeof(int64_t));
  for (int64_t e = 0; e < M; ++e) {
    if (ea[e] == eb[e]) continue;
    tci[pos[ea[e]]] = eb[e]; tw[pos[ea[e]]++] = ew[e];
    tci[pos[eb[e]]] = ea[e]; tw[pos[eb[e]]++] = ew[e];
  }
  free(pos);
  g->ci = tci; g->w = tw;
  return ORACLE_OK;
}

static int64_t lv_qnum(const lv_graph* g, const int32_t* comm, int64_t two_m, int64_t* in2, int64_t* tot) {
  int64_t N = g->N;
  for (int64_t c = 0; c < N; ++c) in2[c] = tot[c] = 0;
  for (int64_t a = 0; a < N; ++a) {
    int64_t k = 2 * g->loop[a];
    in2[comm[a]] += 2 * g->loop[a];
    for (int64_t q = g->rp[a]; q < g->rp[a + 1]; ++q) {
      k += g->w[q];
      if (comm[g->ci[q]] == comm[a]) in2[comm[a]] += g->w[q];      /* seen from both ends over the loop */
    }
    tot[comm[a]] += k;
  }
  int64_t num = 0;
  for (int64_t c = 0; c < N; ++c) num += two_m * in2[c] - tot[c] * tot[c];
  return num;
}

/* One frozen-state sweep: next[a] for every node of the level graph (see above).  tot and size
 * describe comm; kin (all zero on entry and on exit) and touched are scratch.  Returns the number
 * of nodes that move. */
static int64_t lv_decide(const lv_graph* g, const int32_t* comm, const int64_t* k, const int64_t* tot,
                         const int64_t* size, int64_t two_m, int64_t* kin, int32_t* touched, int32_t* next) {
  int64_t moves = 0;
  for (int64_t a = 0; a < g->N; ++a) {
    const int32_t own = comm[a];
    int64_t nt = 0;
    for (int64_t q = g->rp[a]; q < g->rp[a + 1]; ++q) {
      int32_t c = comm[g->ci[q]];
      if (kin[c] == 0) touched[nt++] = c;
      kin[c] += g->w[q];
    }
    const int64_t own_score = two_m * kin[own] - (tot[own] - k[a]) * k[a];
    int64_t best_score = own_score;
    int32_t best = own;
    for (int64_t t = 0; t < nt; ++t) {
      int32_t c = touched[t];
      if (c == own) continue;
      int64_t sc = two_m * kin[c] - tot[c] * k[a];
      if (sc > best_score || (sc == best_score && best != own && c < best)) { best_score = sc; best = c; }
    }
    for (int64_t t = 0; t < nt; ++t) kin[touched[t]] = 0;
    if (best != own && best_score > own_score && !(size[own] == 1 && size[best] == 1 && best > own)) {
      next[a] = best;
      ++moves;
    } else {
      next[a] = own;
    }
  }
  return moves;
}

int64_t oracle_louvain(int64_t n, int64_t E, const int32_t* eu, const int32_t* ev, int32_t max_levels,
                       int32_t max_sweeps, int32_t* part, int64_t* qnum_out, int64_t* two_m_out,
                       int32_t* levels_out, int32_t* sweeps_out) {
  if (n <= 0 || E < 0 || max_levels < 1 || max_sweeps < 1) return ORACLE_BAD_ARG;
  for (int64_t e = 0; e < E; ++e) {
    if (eu[e] < 0 || eu[e] >= n || ev[e] < 0 || ev[e] >= n) return ORACLE_OUT_OF_RANGE;
    if (eu[e] == ev[e]) return ORACLE_NOT_SIMPLE;
  }
  const int64_t two_m = 2 * E;
  int64_t* ones = (int64_t*)malloc((size_t)(E + 1) * sizeof(int64_t));
  if (!ones) return ORACLE_NOMEM;
  for (int64_t e = 0; e < E; ++e) ones[e] = 1;
  lv_graph g;
  int rc = lv_build(n, E, eu, ev, ones, &g);
  free(ones);
  if (rc != ORACLE_OK) { lv_free(&g); return rc; }
  for (int64_t i = 0; i < n; ++i) part[i] = (int32_t)i;      /* level-0 node of every original node */
  int32_t levels = 0, sweeps_total = 0;
  int64_t qnum = 0;
  int64_t S = n;
  for (int32_t level = 0; level < max_levels; ++level) {
    const int64_t N = g.N;
    int32_t* comm = (int32_t*)malloc((size_t)N * sizeof(int32_t));
    int32_t* next = (int32_t*)malloc((size_t)N * sizeof(int32_t));
    int64_t* k = (int64_t*)malloc((size_t)N * sizeof(int64_t));
    int64_t* tot = (int64_t*)malloc((size_t)N * sizeof(int64_t));
    int64_t* in2 = (int64_t*)malloc((size_t)N * sizeof(int64_t));
    int64_t* size = (int64_t*)malloc((size_t)N * sizeof(int64_t));
    int64_t* kin = (int64_t*)calloc((size_t)N, sizeof(int64_t));
    int32_t* touched = (int32_t*)malloc((size_t)N * sizeof(int32_t));
    if (!comm || !next || !k || !tot || !in2 || !size || !kin || !touched) {
      free(comm); free(next); free(k); free(tot); free(in2); free(size); free(kin); free(touched); lv_free(&g);
      return ORACLE_NOMEM;
    }
    for (int64_t a = 0; a < N; ++a) {
      comm[a] = (int32_t)a;
      k[a] = 2 * g.loop[a];
      for (int64_t q = g.rp[a]; q < g.rp[a + 1]; ++q) k[a] += g.w[q];
    }
    qnum = lv_qnum(&g, comm, two_m, in2, tot);
    int moved_this_level = 0;
    for (int32_t sweep = 0; sweep < max_sweeps; ++sweep) {
      for (int64_t c = 0; c < N; ++c) tot[c] = size[c] = 0;
      for (int64_t a = 0; a < N; ++a) { tot[comm[a]] += k[a]; size[comm[a]] += 1; }
      const int64_t moves = lv_decide(&g, comm, k, tot, size, two_m, kin, touched, next);
      if (moves == 0) break;
      int64_t q_new = lv_qnum(&g, next, two_m, in2, tot);
      if (q_new <= qnum) break;                         /* the sweep as a whole did not help: undone */
      memcpy(comm, next, (size_t)N * sizeof(int32_t));
      qnum = q_new;
      moved_this_level = 1;
      ++sweeps_total;
    }
    free(next); free(k); free(tot); free(in2); free(size); free(kin); free(touched);
    if (!moved_this_level) { free(comm); break; }
    ++levels;
    /* contraction: communities in ascending id order become nodes 0..Nc-1 */
    int32_t* newid = (int32_t*)malloc((size_t)N * sizeof(int32_t));
    if (!newid) { free(comm); lv_free(&g); return ORACLE_NOMEM; }
    for (int64_t c = 0; c < N; ++c) newid[c] = -1;
    for (int64_t a = 0; a < N; ++a) newid[comm[a]] = 0;
    int64_t Nc = 0;
    for (int64_t c = 0; c < N; ++c) if (newid[c] == 0) newid[c] = (int32_t)Nc++;
    for (int64_t i = 0; i < n; ++i) part[i] = newid[comm[part[i]]];
    /* every undirected edge once (a < b) plus the self loops, relabelled; lv_build adds weights up */
    int64_t M = N;
    for (int64_t a = 0; a < N; ++a)
      for (int64_t q = g.rp[a]; q < g.rp[a + 1]; ++q) if (g.ci[q] > a) ++M;
    int32_t* ea = (int32_t*)malloc((size_t)(M + 1) * sizeof(int32_t));
    int32_t* eb = (int32_t*)malloc((size_t)(M + 1) * sizeof(int32_t));
    int64_t* ew = (int64_t*)malloc((size_t)(M + 1) * sizeof(int64_t));
    if (!ea || !eb || !ew) { free(ea); free(eb); free(ew); free(newid); free(comm); lv_free(&g); return ORACLE_NOMEM; }
    int64_t t = 0;
    for (int64_t a = 0; a < N; ++a) {
      ea[t] = eb[t] = newid[comm[a]]; ew[t++] = g.loop[a];
      for (int64_t q = g.rp[a]; q < g.rp[a + 1]; ++q)
        if (g.ci[q] > a) { ea[t] = newid[comm[a]]; eb[t] = newid[comm[g.ci[q]]]; ew[t++] = g.w[q]; }
    }
    free(newid); free(comm);
    lv_free(&g);
    /* merge parallel edges so that the next level's adjacency lists hold every neighbour once */
    {
      /* sort (min, max) pairs by a simple two-pass counting approach: build, then compact rows */
      lv_graph raw;
      for (int64_t e = 0; e < t; ++e)
        if (ea[e] > eb[e]) { int32_t s = ea[e]; ea[e] = eb[e]; eb[e] = s; }
      rc = lv_build(Nc, t, ea, eb, ew, &raw);
      free(ea); free(eb); free(ew);
      if (rc != ORACLE_OK) { lv_free(&raw); return rc; }
      int64_t* acc = (int64_t*)calloc((size_t)Nc, sizeof(int64_t));
      int32_t* seen = (int32_t*)malloc((size_t)Nc * sizeof(int32_t));
      int64_t* nrp = (int64_t*)calloc((size_t)Nc + 1, sizeof(int64_t));
      if (!acc || !seen || !nrp) { free(acc); free(seen); free(nrp); lv_free(&raw); return ORACLE_NOMEM; }
      int64_t out = 0;
      for (int64_t a = 0; a < Nc; ++a) {
        int64_t ns = 0;
        for (int64_t q = raw.rp[a]; q < raw.rp[a + 1]; ++q) {
          int32_t b = raw.ci[q];
          if (acc[b] == 0) seen[ns++] = b;
          acc[b] += raw.w[q];
        }
        qsort(seen, (size_t)ns, sizeof(int32_t), cmp_i32);
        for (int64_t s = 0; s < ns; ++s) { raw.ci[out] = seen[s]; raw.w[out++] = acc[seen[s]]; acc[seen[s]] = 0; }
        nrp[a + 1] = out;
      }
      free(acc); free(seen);
      free(raw.rp);
      raw.rp = nrp;
      g = raw;
    }
    S = Nc;
  }
  lv_free(&g);
  if (qnum_out) *qnum_out = qnum;
  if (two_m_out) *two_m_out = two_m;
  if (levels_out) *levels_out = levels;
  if (sweeps_out) *sweeps_out = sweeps_total;
  return S;
}

/* One frozen-state sweep on the input graph from a GIVEN community vector (no acceptance test, no
 * contraction): next[i] as defined above.  Lets a test look at a single sweep. */
int64_t oracle_louvain_sweep(int64_t n, int64_t E, const int32_t* eu, const int32_t* ev, const int32_t* comm,
                             int32_t* next) {
  int64_t* ones = (int64_t*)malloc((size_t)(E + 1) * sizeof(int64_t));
  if (!ones) return ORACLE_NOMEM;
  for (int64_t e = 0; e < E; ++e) ones[e] = 1;
  lv_graph g;
  int rc = lv_build(n, E, eu, ev, ones, &g);
  free(ones);
  if (rc != ORACLE_OK) { lv_free(&g); return rc; }
  const int64_t two_m = 2 * E;
  int64_t* k = (int64_t*)calloc((size_t)n, sizeof(int64_t));
  int64_t* tot = (int64_t*)calloc((size_t)n, sizeof(int64_t));
  int64_t* size = (int64_t*)calloc((size_t)n, sizeof(int64_t));
  int64_t* kin = (int64_t*)calloc((size_t)n, sizeof(int64_t));
  int32_t* touched = (int32_t*)malloc((size_t)n * sizeof(int32_t));
  if (!k || !tot || !size || !kin || !touched) { free(k); free(tot); free(size); free(kin); free(touched); lv_free(&g); return ORACLE_NOMEM; }
  for (int64_t a = 0; a < n; ++a) {
    for (int64_t q = g.rp[a]; q < g.rp[a + 1]; ++q) k[a] += g.w[q];
    tot[comm[a]] += k[a];
    size[comm[a]] += 1;
  }
  const int64_t moves = lv_decide(&g, comm, k, tot, size, two_m, kin, touched, next);
  free(k); free(tot); free(size); free(kin); free(touched);
  lv_free(&g);
  return moves;
}
