// gnnco_train_step: host-side plan of one full-batch training step over the
// block-diagonal batch (Section 3.2, Eqs. 3-5; Algorithm 1, Stage 1).  Only kernel
// launches happen here; every arithmetic step runs on the device.
//
// Forward, hidden layer l (1-based, widths d_{l-1} -> d_l):
//     M_l = A_hat H_{l-1}            aggregate   (spmm.cu; M_l is a temporary, not kept)
//     H_l = ReLU(M_l W_l)            transform   (dense.cu / tc_gemm*.cu)
// Output layer:  u = H_{L-1} w_L ;  z = A_hat u ;  p = sigmoid(z)      (chain.cu)
// Objective:     q = A p, per-subgraph loss, t = D^-1 dz ;  g = (A+I) t = A_hat^T dz
// Backward.  With Q_l = A_hat^T dZ_l = (A+I)(D^-1 dZ_l) the chain rule through
// Z_l = A_hat H_{l-1} W_l reads  dW_l = H_{l-1}^T Q_l  and  dH_{l-1} = Q_l W_l^T, so only the
// activations H_l are kept from the forward pass:
//     dw_L = H_{L-1}^T g
//     Q_{L-1} = (A+I) D^-1 (g w_L^T * [H_{L-1} > 0])                  aggregate, rank-1 mode
//     for l = L-1 .. 1:  R = D^-1 ((Q_l W_l^T) * [H_{l-1} > 0])       transform with mask (dX = Q_1 W_1^T when l = 1)
//                        dW_l = H_{l-1}^T Q_l ;  Adam on W_l
//                        Q_{l-1} = (A+I) R                            aggregate
// The transposed aggregation reuses the forward CSR because the intra adjacency is
// symmetric: A_hat^T G = (A+I)(D^-1 G).
#include <math.h>

#include "internal.cuh"

namespace {

struct TrainLayout {
  void* H[GNNCO_MAX_LAYERS];          // H[l], l = 1..L-1: activation of hidden layer l
  void* Ga;                           // n x max width: aggregated input M_l (forward), then gradient ping-pong
  void* Gb;                           // second gradient buffer (three or more layers, backward)
  float *u, *t, *g, *item_loss;
  float* dW_scratch;                  // one layer's gradient (all sets), when the caller wants none
  float* dW_sets;                     // per-subgraph partials when the model shares one weight set
  float* wg_scratch;                  // partial weight gradients of subgraphs that were split into row chunks
  float2* adam_bias;                  // 1 / (1 - beta^t) of this update when the step counter lives on the device
  float* agg_partial;                 // partial sums of the segments of long rows (aggregation)
  uint8_t* Hbits[GNNCO_MAX_LAYERS];   // [H_l > 0], one bit per element (bfloat16; written by the transform that makes H_l,
                                      // or, for the last hidden layer, by the output layer's weight gradient)
  __nv_bfloat16* W_lp[GNNCO_MAX_LAYERS];   // bf16 copies of the weights (bf16 features only)
  __nv_bfloat16* W_lp_t[GNNCO_MAX_LAYERS]; // transposed bf16 copies [sets x F_out x F_in] for the tensor-core forward
  __nv_bfloat16* W3[GNNCO_MAX_LAYERS];     // float32 features: three bf16 limbs of W (input-gradient operand)
  __nv_bfloat16* W3_t[GNNCO_MAX_LAYERS];   // ... and of W^T (forward operand)
  // host-variant staging
  void* X_stage;
  float *pen_stage, *loss_stage, *p_stage;
  size_t bytes;
};

size_t elem_size(int dtype) { return dtype == GNNCO_BF16 ? 2 : 4; }

int32_t check_model(const gnnco_handle* h, const gnnco_model_desc* m, bool need_ptrs) {
  if (!h || !m) return GNNCO_INVALID_ARGUMENT;
  if (m->L < 1 || m->L > GNNCO_MAX_LAYERS) return GNNCO_INVALID_ARGUMENT;
  if (m->feat_dtype != GNNCO_F32 && m->feat_dtype != GNNCO_BF16) return GNNCO_UNSUPPORTED;
  if (m->weight_sets != 1 && m->weight_sets != h->S) return GNNCO_INVALID_ARGUMENT;
  for (int l = 0; l <= m->L; ++l)
    if (m->dims[l] < 1 || m->dims[l] > 65536) return GNNCO_INVALID_ARGUMENT;
  if (m->dims[m->L] != 1) return GNNCO_INVALID_ARGUMENT;
  if (m->feat_dtype == GNNCO_BF16)
    for (int l = 0; l < m->L; ++l)
      if (m->dims[l] % 2) return GNNCO_UNSUPPORTED;     // bf16 rows must stay 4-byte aligned
  if (need_ptrs)
    for (int l = 0; l < m->L; ++l)
      if (!m->W[l]) return GNNCO_INVALID_ARGUMENT;
  return GNNCO_OK;
}

TrainLayout carve_train(const gnnco_handle* h, const gnnco_model_desc* m, uint32_t flags, void* base, bool host) {
  TrainLayout T{};
  Carver c(base, ~(size_t)0);
  const size_t es = elem_size(m->feat_dtype);
  const size_t n = (size_t)h->n;
  const int L = m->L;
  int maxw = 1;
  size_t max_wcount = 0;
  for (int l = 0; l < L; ++l) {
    if (m->dims[l] > maxw) maxw = m->dims[l];
    size_t wc = (size_t)m->dims[l] * m->dims[l + 1];
    if (wc > max_wcount) max_wcount = wc;
  }
  for (int l = 1; l < L; ++l) T.H[l] = c.take<char>(n * m->dims[l] * es);
  if (L > 1) T.Ga = c.take<char>(n * maxw * es);
  T.u = c.take<float>(n);
  T.t = c.take<float>(n);
  T.g = c.take<float>(n);
  T.item_loss = c.take<float>((size_t)h->n_items + 1);
  T.agg_partial = h->n_long_segs > 0 ? c.take<float>((size_t)h->n_long_segs * maxw) : nullptr;
  if (!(flags & GNNCO_FORWARD_ONLY)) {
    if (m->feat_dtype == GNNCO_BF16)
      for (int l = 1; l < L; ++l)
        if (m->dims[l] % 8 == 0) T.Hbits[l] = c.take<uint8_t>(n * (size_t)(m->dims[l] / 8));
    if (L > 2) T.Gb = c.take<char>(n * maxw * es);
    T.dW_scratch = c.take<float>(max_wcount * m->weight_sets);
    if (m->weight_sets == 1) T.dW_sets = c.take<float>(max_wcount * (size_t)h->S);
    T.wg_scratch = c.take<float>(max_wcount * (size_t)h->n_wg_slots + 1);
    T.adam_bias = c.take<float2>(1);
  }
  if (m->feat_dtype == GNNCO_BF16)
    for (int l = 0; l < L; ++l)
      T.W_lp[l] = c.take<__nv_bfloat16>((size_t)m->dims[l] * m->dims[l + 1] * m->weight_sets);
  for (int l = 0; l + 1 < L; ++l)
    if (tc_transform_supported(m->feat_dtype, m->dims[l], m->dims[l + 1]))
      T.W_lp_t[l] = c.take<__nv_bfloat16>((size_t)m->dims[l] * m->dims[l + 1] * m->weight_sets);
  if (m->feat_dtype == GNNCO_F32)
    for (int l = 0; l + 1 < L; ++l) {
      const size_t wc3 = (size_t)3 * m->dims[l] * m->dims[l + 1] * m->weight_sets;
      if (tc_f32_transform_supported(m->dims[l], m->dims[l + 1])) T.W3_t[l] = c.take<__nv_bfloat16>(wc3);
      if (!(flags & GNNCO_FORWARD_ONLY) && tc_f32_transform_supported(m->dims[l + 1], m->dims[l]))
        T.W3[l] = c.take<__nv_bfloat16>(wc3);
    }
  if (host) {
    T.X_stage = c.take<char>(n * m->dims[0] * es);
    T.pen_stage = c.take<float>(n);
    T.loss_stage = c.take<float>((size_t)h->S);
    T.p_stage = c.take<float>(n);
  }
  T.bytes = c.off;
  return T;
}

int32_t run_step_on(gnnco_handle* h, const gnnco_model_desc* m, const void* X, const gnnco_objective* obj,
                    gnnco_adam_state* opt, const gnnco_train_out* out, uint32_t flags, const TrainLayout& T,
                    cudaStream_t st);

WorkSet capture_work(const gnnco_handle* h) {
  WorkSet w;
  w.tile_row0 = h->tile_row0; w.tile_rows = h->tile_rows; w.pair_row0 = h->pair_row0; w.pair_rows = h->pair_rows;
  w.item_row0 = h->item_row0; w.item_row1 = h->item_row1; w.part_item_ptr = h->part_item_ptr;
  w.wg_begin = h->wg_begin; w.wg_end = h->wg_end; w.wg_slot = h->wg_slot;
  w.wg_mpart = h->wg_mpart; w.wg_mfirst = h->wg_mfirst; w.wg_mcount = h->wg_mcount;
  w.n_tiles = h->n_tiles; w.n_pairs = h->n_pairs; w.n_items = h->n_items; w.n_wg_chunks = h->n_wg_chunks;
  w.n_wg_multi = h->n_wg_multi;
  w.row_chunks = h->row_chunks;
  w.fuse = h->fuse;
  return w;
}

void apply_work(gnnco_handle* h, const WorkSet& w) {
  h->tile_row0 = w.tile_row0; h->tile_rows = w.tile_rows; h->pair_row0 = w.pair_row0; h->pair_rows = w.pair_rows;
  h->item_row0 = w.item_row0; h->item_row1 = w.item_row1; h->part_item_ptr = w.part_item_ptr;
  h->wg_begin = w.wg_begin; h->wg_end = w.wg_end; h->wg_slot = w.wg_slot;
  h->wg_mpart = w.wg_mpart; h->wg_mfirst = w.wg_mfirst; h->wg_mcount = w.wg_mcount;
  h->n_tiles = w.n_tiles; h->n_pairs = w.n_pairs; h->n_items = w.n_items; h->n_wg_chunks = w.n_wg_chunks;
  h->n_wg_multi = w.n_wg_multi;
  h->row_chunks = w.row_chunks;
  h->fuse = w.fuse;
}

// A step over all subgraphs, or (GNNCO_ACTIVE_ONLY) the same launch sequence with the plan's work tables
// swapped in for its duration.
int32_t run_step(gnnco_handle* h, const gnnco_model_desc* m, const void* X, const gnnco_objective* obj,
                 gnnco_adam_state* opt, const gnnco_train_out* out, uint32_t flags, const TrainLayout& T,
                 cudaStream_t st) {
  if (!(flags & GNNCO_ACTIVE_ONLY)) return run_step_on(h, m, X, obj, opt, out, flags, T, st);
  if (h->plan.row_chunks.count == 0) return GNNCO_OK;          // no active subgraph has a node: nothing to do
  const WorkSet full = capture_work(h);
  apply_work(h, h->plan);
  const int32_t rc = run_step_on(h, m, X, obj, opt, out, flags, T, st);
  apply_work(h, full);
  return rc;
}

int32_t run_step_on(gnnco_handle* h, const gnnco_model_desc* m, const void* X, const gnnco_objective* obj,
                    gnnco_adam_state* opt, const gnnco_train_out* out, uint32_t flags, const TrainLayout& T,
                    cudaStream_t st) {
  const int L = m->L, dt = m->feat_dtype;
  const bool bf16 = dt == GNNCO_BF16;
  h->agg_partial = T.agg_partial;       // where this step's aggregations keep the segments of long rows
  h->adam_bias = nullptr;
  const int32_t sets = m->weight_sets;
  int32_t rc;
#define GNNCO_TRY(call) do { rc = (call); if (rc != GNNCO_OK) return rc; } while (0)
  // weights as the matrix products see them
  const void* Wc[GNNCO_MAX_LAYERS];
  int64_t wstride[GNNCO_MAX_LAYERS];
  for (int l = 0; l < L; ++l) {
    const int64_t wc = (int64_t)m->dims[l] * m->dims[l + 1];
    wstride[l] = sets == 1 ? 0 : wc;
    if (bf16) {
      // copies that the previous step's Adam left behind are used as they are when the caller vouches for them
      const bool fresh = (flags & GNNCO_WEIGHTS_UNTOUCHED) && h->shadow_fresh[l] && h->shadow_W[l] == m->W[l] &&
                         h->shadow_copy[l] == (const void*)T.W_lp[l];
      h->shadow_fresh[l] = false;
      if (fresh) {
      } else if (T.W_lp_t[l])
        GNNCO_TRY(launch_cast_both_bf16(h, m->W[l], T.W_lp[l], T.W_lp_t[l], m->dims[l], m->dims[l + 1], sets, st));
      else
        GNNCO_TRY(launch_cast_bf16(h, m->W[l], T.W_lp[l], wc * sets, st));
      Wc[l] = T.W_lp[l];
    } else {
      Wc[l] = m->W[l];
      if (T.W3_t[l]) GNNCO_TRY(launch_cast_split3(h, m->W[l], T.W3_t[l], m->dims[l], m->dims[l + 1], sets, true, st));
      const bool need_bwd = !(flags & GNNCO_FORWARD_ONLY) && (l > 0 || (flags & GNNCO_WANT_DX));
      if (T.W3[l] && need_bwd)
        GNNCO_TRY(launch_cast_split3(h, m->W[l], T.W3[l], m->dims[l], m->dims[l + 1], sets, false, st));
    }
  }
  // ---- forward
  const void* Hprev = X;
  bool u_done = false;
  bool bits_written[GNNCO_MAX_LAYERS] = {false};
  // hidden layer l of the forward pass over the work tables that the handle holds at the moment
  auto forward_layer = [&](int l, const void* Hprev) -> int32_t {
    // aggregated input M_l; the first layer's can be kept across steps (X does not change)
    const void* Min = T.Ga;
    const bool cached_first = l == 1 && (flags & (GNNCO_AX_STORE | GNNCO_AX_REUSE));
    if (cached_first) Min = out->ax_cache;
    // on request, aggregation and transform in one kernel where there is one: M_l never reaches HBM (the
    // backward pass does not need it: dW_l = H_{l-1}^T Q_l)
    const bool one_kernel = (flags & GNNCO_ONE_KERNEL_LAYERS) && !cached_first && !(l == 1 && h->arrival) && T.W_lp_t[l - 1] &&
                            aggregate_transform_pair_supported(h, dt, m->dims[l - 1], m->dims[l]) &&
                            !((uintptr_t)Hprev & 15);
    if (one_kernel) {
      const bool fuse = (l == L - 1);
      uint8_t* bits = l < L - 1 ? T.Hbits[l] : nullptr;
      if (h->fuse.n_light > 0)
        GNNCO_TRY(launch_aggregate_transform_pair(h, Hprev, T.W_lp_t[l - 1], wstride[l - 1], sets, T.H[l], m->dims[l - 1],
                                                  m->dims[l], h->inv_deg, bits, fuse ? Wc[L - 1] : nullptr, wstride[L - 1],
                                                  fuse ? T.u : nullptr, st));
      if (h->fuse.n_heavy > 0) {
        // double tiles with a long row or very many entries: the two separate kernels, over those tiles only
        // (their table has the format of the double-tile table and of the row chunks)
        const WorkSet all = capture_work(h);
        h->pair_row0 = h->fuse.heavy_row0; h->pair_rows = h->fuse.heavy_rows; h->n_pairs = h->fuse.n_heavy;
        h->row_chunks.row0 = h->fuse.heavy_row0; h->row_chunks.rows = h->fuse.heavy_rows;
        h->row_chunks.count = h->fuse.n_heavy;
        rc = launch_aggregate(h, dt, Hprev, T.Ga, m->dims[l - 1], h->inv_deg, nullptr, st);
        if (rc == GNNCO_OK)
          rc = launch_transform_tc_pair(h, T.Ga, T.W_lp_t[l - 1], wstride[l - 1], sets, T.H[l], m->dims[l - 1], m->dims[l],
                                        true, nullptr, nullptr, bits, false, fuse ? Wc[L - 1] : nullptr, wstride[L - 1],
                                        fuse ? T.u : nullptr, st);
        apply_work(h, all);
        if (rc != GNNCO_OK) return rc;
      }
      bits_written[l] = bits != nullptr;
      u_done = fuse;
      return GNNCO_OK;
    }
    if (!(l == 1 && (flags & GNNCO_AX_REUSE)))
      GNNCO_TRY(launch_aggregate(h, dt, Hprev, const_cast<void*>(Min), m->dims[l - 1], h->inv_deg, nullptr, st));
    if (T.W_lp_t[l - 1]) {
      // the last hidden layer also produces u = H w_L in its epilogue
      const bool fuse = (l == L - 1) && (m->dims[l] % 8 == 0);
      if (tc_pair_transform_supported(h, dt, m->dims[l - 1], m->dims[l])) {
        // The pair kernel can leave [H_l > 0] behind as bits for the masked input gradient of layer l + 1.  The
        // last hidden layer's bits are left to the output layer's weight gradient, which reads H_{L-1} anyway:
        // measured in one run, 0.22 ms more here against 0.21 ms more there, and the drain of this kernel is the
        // scarcer resource.
        uint8_t* bits = l < L - 1 ? T.Hbits[l] : nullptr;
        GNNCO_TRY(launch_transform_tc_pair(h, Min, T.W_lp_t[l - 1], wstride[l - 1], sets, T.H[l], m->dims[l - 1],
                                           m->dims[l], true, nullptr, nullptr, bits, false, fuse ? Wc[L - 1] : nullptr,
                                           wstride[L - 1], fuse ? T.u : nullptr, st));
        bits_written[l] = bits != nullptr;
      } else
        GNNCO_TRY(launch_transform_tc(h, Min, T.W_lp_t[l - 1], wstride[l - 1], T.H[l], m->dims[l - 1], m->dims[l], true,
                                      nullptr, nullptr, false, fuse ? Wc[L - 1] : nullptr, wstride[L - 1],
                                      fuse ? T.u : nullptr, st));
      u_done = fuse;
    } else if (T.W3_t[l - 1]) {
      const bool fuse = (l == L - 1) && (m->dims[l] % 4 == 0);
      GNNCO_TRY(launch_transform_tc_f32(h, Min, T.W3_t[l - 1], wstride[l - 1],
                                        (int64_t)m->dims[l - 1] * m->dims[l] * sets, T.H[l], m->dims[l - 1], m->dims[l],
                                        true, nullptr, nullptr, false, fuse ? Wc[L - 1] : nullptr, wstride[L - 1],
                                        fuse ? T.u : nullptr, st));
      u_done = fuse;
    } else
      GNNCO_TRY(launch_transform(h, dt, Min, Wc[l - 1], wstride[l - 1], T.H[l], m->dims[l - 1], m->dims[l], false,
                                 true, nullptr, nullptr, st));
    return GNNCO_OK;
  };
  for (int l = 1; l < L; ++l) {
    const ArrivalPlan* ap = l == 1 ? h->arrival : nullptr;
    if (ap && ap->groups > 1) {
      // the host variant: X arrives in ranges of subgraphs on another stream; layer 1 follows range by range
      // (the tables are ordered by subgraph, so a range of subgraphs is a range of each table)
      const WorkSet all = capture_work(h);
      rc = GNNCO_OK;
      for (int g = 0; g < ap->groups && rc == GNNCO_OK; ++g) {
        if (cudaStreamWaitEvent(st, ap->ev[g], 0) != cudaSuccess) { rc = GNNCO_CUDA_ERROR; break; }
        h->tile_row0 = all.tile_row0 + ap->tile0[g]; h->tile_rows = all.tile_rows + ap->tile0[g];
        h->n_tiles = ap->tile0[g + 1] - ap->tile0[g];
        h->pair_row0 = all.pair_row0 + ap->pair0[g]; h->pair_rows = all.pair_rows + ap->pair0[g];
        h->n_pairs = ap->pair0[g + 1] - ap->pair0[g];
        h->row_chunks.row0 = h->pair_row0; h->row_chunks.rows = h->pair_rows; h->row_chunks.count = h->n_pairs;
        if (h->n_pairs > 0) rc = forward_layer(1, Hprev);
      }
      apply_work(h, all);
      if (rc != GNNCO_OK) return rc;
      if (cudaStreamWaitEvent(st, ap->ev_rest, 0) != cudaSuccess) return GNNCO_CUDA_ERROR;
    } else {
      GNNCO_TRY(forward_layer(l, Hprev));
    }
    Hprev = T.H[l];
  }
  const int FL = m->dims[L - 1];
  if (!u_done) GNNCO_TRY(launch_gemv(h, dt, Hprev, Wc[L - 1], wstride[L - 1], T.u, FL, st));
  GNNCO_TRY(launch_output_forward(h, T.u, out->z, out->p, st));
  const bool fwd_only = (flags & GNNCO_FORWARD_ONLY) != 0;
  GNNCO_TRY(launch_objective(h, out->p, obj->pen, obj->alpha, obj->beta, obj->lambda, T.item_loss, out->loss,
                             fwd_only ? nullptr : T.t, st));
  if (fwd_only) return GNNCO_OK;
  // ---- backward
  // coef = D^-1 g takes the place of u, which the forward pass is done with
  GNNCO_TRY(launch_output_backward(h, T.t, T.g, L > 1 ? T.u : nullptr, st));
  float c1 = 1.0f, c2 = 1.0f;
  h->adam_bias = nullptr;
  if (opt && opt->step_dev) {
    // step counter on the device: one thread advances it and leaves this update's bias corrections for the Adam
    // kernels (nothing below then depends on a host value that changes from step to step)
    GNNCO_TRY(launch_adam_tick(h, opt->step_dev, opt->beta1, opt->beta2, T.adam_bias, st));
    h->adam_bias = T.adam_bias;
  } else if (opt) {
    c1 = (float)(1.0 - pow((double)opt->beta1, (double)opt->step));
    c2 = (float)(1.0 - pow((double)opt->beta2, (double)opt->step));
  }
  auto finish_layer = [&](int l, float* grad_sets_or_final) -> int32_t {
    // grad_sets_or_final holds [sets x ...] already reduced; run Adam on layer l (0-based)
    const int64_t wc = (int64_t)m->dims[l] * m->dims[l + 1] * sets;
    if (!opt) return GNNCO_OK;
    if (bf16 && T.W_lp_t[l] &&
        adam_cast_both_supported(m->W[l], opt->m[l], opt->v[l], grad_sets_or_final, T.W_lp[l], T.W_lp_t[l], m->dims[l],
                                 m->dims[l + 1], sets)) {
      // everything that reads this layer's bf16 copies in this step has been launched before this point
      int32_t rc2 = launch_adam_cast_both(h, m->W[l], opt->m[l], opt->v[l], grad_sets_or_final, T.W_lp[l], T.W_lp_t[l],
                                          m->dims[l], m->dims[l + 1], sets, opt->lr, opt->beta1, opt->beta2, opt->eps,
                                          c1, c2, opt->active, st);
      if (rc2 == GNNCO_OK) {
        h->shadow_W[l] = m->W[l];
        h->shadow_copy[l] = T.W_lp[l];
        h->shadow_fresh[l] = true;
      }
      return rc2;
    }
    return launch_adam(h, m->W[l], opt->m[l], opt->v[l], grad_sets_or_final, wc, opt->lr, opt->beta1, opt->beta2,
                       opt->eps, c1, c2, opt->active, wc / sets, st);
  };
  // gradient target of layer l: the caller's buffer or the scratch
  auto grad_target = [&](int l) -> float* { return out->dW[l] ? out->dW[l] : T.dW_scratch; };
  void* Q = T.Ga;          // Q_l = A_hat^T dZ_l of the layer being processed
  void* other = T.Gb;
  {
    // last layer (0-based index L-1): dw = H^T g
    float* target = grad_target(L - 1);
    bool have_bits = false;
    uint8_t* wgv_bits = (L > 1 && !bits_written[L - 1]) ? T.Hbits[L - 1] : nullptr;
    if (sets == 1) {
      GNNCO_TRY(launch_weight_grad_vec(h, dt, Hprev, T.g, T.dW_sets, T.wg_scratch, FL, wgv_bits, &have_bits, st));
      GNNCO_TRY(launch_sum_over_sets(h, T.dW_sets, target, FL, h->S, st));
    } else {
      GNNCO_TRY(launch_weight_grad_vec(h, dt, Hprev, T.g, target, T.wg_scratch, FL, wgv_bits, &have_bits, st));
    }
    if (L > 1 && bits_written[L - 1]) have_bits = true;
    // everything that reads the weights of a layer runs before that layer's Adam update
    if (L > 1) {
      // from the mask bits that the weight-gradient pass above left behind, where it could
      const bool from_bits = have_bits && aggregate_rank1_bits_supported(h, dt, FL) &&
                             !((uintptr_t)Wc[L - 1] & 15) && wstride[L - 1] % 8 == 0 && !((uintptr_t)Q & 15) &&
                             !((uintptr_t)Hprev & 15);
      if (from_bits)
        GNNCO_TRY(launch_aggregate_rank1_bits(h, dt, T.Hbits[L - 1], Hprev, T.u, Wc[L - 1], wstride[L - 1], Q, FL, st));
      else
        GNNCO_TRY(launch_aggregate_rank1(h, dt, Hprev, T.u, Wc[L - 1], wstride[L - 1], Q, FL, st));
    }
    else if (flags & GNNCO_WANT_DX)
      // L == 1: dX = A_hat^T (dz w_s^T) and w_s is constant inside a subgraph, so dX[i,:] = g_i w_s^T
      GNNCO_TRY(launch_rank1_masked(h, dt, T.g, Wc[0], wstride[0], nullptr, out->dX, FL, st));
    GNNCO_TRY(finish_layer(L - 1, target));
  }
  for (int l = L - 1; l >= 1; --l) {
    // hidden layer l uses weight index l-1: widths d_{l-1} -> d_l
    const int K = m->dims[l - 1], N = m->dims[l];
    const void* Hin = l > 1 ? T.H[l - 1] : X;
    const bool need_input_grad = (l > 1) || (flags & GNNCO_WANT_DX);
    if (need_input_grad) {
      // l > 1: R = D^-1 ((Q W^T) * [H_{l-1} > 0]);  l == 1: dX = Q W^T
      void* dst = l > 1 ? other : out->dX;
      const float* scale = l > 1 ? h->inv_deg : nullptr;
      const void* mask = l > 1 ? T.H[l - 1] : nullptr;
      if (tc_pair_transform_supported(h, dt, N, K) && (l == 1 || bits_written[l - 1]))
        GNNCO_TRY(launch_transform_tc_pair(h, Q, Wc[l - 1], wstride[l - 1], sets, dst, N, K, false, scale,
                                           l > 1 ? T.Hbits[l - 1] : nullptr, nullptr, true, nullptr, 0, nullptr, st));
      else if (tc_transform_supported(dt, N, K))
        GNNCO_TRY(launch_transform_tc(h, Q, Wc[l - 1], wstride[l - 1], dst, N, K, false, scale, mask, true, nullptr, 0,
                                      nullptr, st));
      else if (T.W3[l - 1])
        GNNCO_TRY(launch_transform_tc_f32(h, Q, T.W3[l - 1], wstride[l - 1], (int64_t)K * N * sets, dst, N, K, false,
                                          scale, mask, true, nullptr, 0, nullptr, st));
      else
        GNNCO_TRY(launch_transform(h, dt, Q, Wc[l - 1], wstride[l - 1], dst, N, K, true, false, scale, mask, st));
    }
    float* target = grad_target(l - 1);
    float* wg_out = sets == 1 ? T.dW_sets : target;
    if (tc_pair_weight_grad_supported(h, dt, K, N))
      GNNCO_TRY(launch_weight_grad_tc_pair(h, Hin, Q, wg_out, T.wg_scratch, K, N, st));
    else if (tc_weight_grad_supported(dt, K, N))
      GNNCO_TRY(launch_weight_grad_tc(h, Hin, Q, wg_out, T.wg_scratch, K, N, st));
    else if (dt == GNNCO_F32 && tc_f32_weight_grad_supported(K, N))
      GNNCO_TRY(launch_weight_grad_tc_f32(h, Hin, Q, wg_out, T.wg_scratch, K, N, st));
    else GNNCO_TRY(launch_weight_grad(h, dt, Hin, Q, wg_out, T.wg_scratch, K, N, st));
    if (sets == 1) GNNCO_TRY(launch_sum_over_sets(h, T.dW_sets, target, (int64_t)K * N, h->S, st));
    GNNCO_TRY(finish_layer(l - 1, target));
    if (l > 1) GNNCO_TRY(launch_aggregate(h, dt, other, Q, K, nullptr, nullptr, st));   // Q_{l-1} = (A+I) R
  }
#undef GNNCO_TRY
  return GNNCO_OK;
}

int32_t check_step_args(const gnnco_handle* h, const gnnco_model_desc* m, const gnnco_adam_state* opt,
                        uint32_t flags) {
  int32_t rc = check_model(h, m, true);
  if (rc != GNNCO_OK) return rc;
  if (flags & ~(GNNCO_WANT_DX | GNNCO_FORWARD_ONLY | GNNCO_AX_STORE | GNNCO_AX_REUSE | GNNCO_WEIGHTS_UNTOUCHED |
                GNNCO_ACTIVE_ONLY | GNNCO_ONE_KERNEL_LAYERS))
    return GNNCO_INVALID_ARGUMENT;
  if (flags & GNNCO_ACTIVE_ONLY) {
    if (flags & (GNNCO_AX_STORE | GNNCO_AX_REUSE)) return GNNCO_INVALID_ARGUMENT;
    if (h->plan_active_count < 0 || !opt || opt->active != h->plan_active || m->weight_sets != h->S || m->L < 2)
      return GNNCO_INVALID_ARGUMENT;
  }
  if ((flags & GNNCO_AX_STORE) && (flags & GNNCO_AX_REUSE)) return GNNCO_INVALID_ARGUMENT;
  if ((flags & (GNNCO_AX_STORE | GNNCO_AX_REUSE)) && m->L < 2) return GNNCO_INVALID_ARGUMENT;
  if (opt && !(flags & GNNCO_FORWARD_ONLY)) {
    if (opt->step < 1) return GNNCO_INVALID_ARGUMENT;
    if (opt->active && m->weight_sets != h->S) return GNNCO_INVALID_ARGUMENT;
    for (int l = 0; l < m->L; ++l)
      if (!opt->m[l] || !opt->v[l]) return GNNCO_INVALID_ARGUMENT;
  }
  return GNNCO_OK;
}

}  // namespace

extern "C" int32_t gnnco_train_workspace_bytes(const gnnco_handle* h, const gnnco_model_desc* m, uint32_t flags,
                                              size_t* bytes) {
  if (!bytes) return GNNCO_INVALID_ARGUMENT;
  int32_t rc = check_model(h, m, false);
  if (rc != GNNCO_OK) return rc;
  *bytes = carve_train(h, m, flags, nullptr, false).bytes;
  return GNNCO_OK;
}

extern "C" int32_t gnnco_train_host_workspace_bytes(const gnnco_handle* h, const gnnco_model_desc* m, uint32_t flags,
                                                   size_t* bytes) {
  if (!bytes) return GNNCO_INVALID_ARGUMENT;
  int32_t rc = check_model(h, m, false);
  if (rc != GNNCO_OK) return rc;
  *bytes = carve_train(h, m, flags, nullptr, true).bytes;
  return GNNCO_OK;
}

extern "C" int32_t gnnco_train_step(gnnco_handle* h, const gnnco_model_desc* m, const void* X,
                                   const gnnco_objective* obj, gnnco_adam_state* opt, const gnnco_train_out* out,
                                   uint32_t flags, void* ws, size_t ws_bytes, void* stream) {
  if (!h || !m || !X || !obj || !out || !ws || !out->loss || !out->p) return GNNCO_INVALID_ARGUMENT;
  int32_t rc = check_step_args(h, m, opt, flags);
  if (rc != GNNCO_OK) return rc;
  if ((flags & GNNCO_WANT_DX) && !out->dX) return GNNCO_INVALID_ARGUMENT;
  if ((flags & (GNNCO_AX_STORE | GNNCO_AX_REUSE)) && !out->ax_cache) return GNNCO_INVALID_ARGUMENT;
  if ((uintptr_t)ws & 255) return GNNCO_INVALID_ARGUMENT;
  TrainLayout T = carve_train(h, m, flags, ws, false);
  if (T.bytes > ws_bytes) return GNNCO_WORKSPACE_TOO_SMALL;
  return run_step(h, m, X, obj, opt, out, flags, T, static_cast<cudaStream_t>(stream));
}

extern "C" int32_t gnnco_train_step_host(gnnco_handle* h, const gnnco_model_desc* m, const void* X_host, float alpha,
                                        float beta, float lambda, const float* pen_host, gnnco_adam_state* opt,
                                        float* loss_host, float* p_host, uint32_t flags, void* ws, size_t ws_bytes,
                                        void* stream) {
  if (!h || !m || !X_host || !loss_host || !p_host || !ws) return GNNCO_INVALID_ARGUMENT;
  int32_t rc = check_step_args(h, m, opt, flags);
  if (rc != GNNCO_OK) return rc;
  // the host variant returns loss and p only and takes fresh inputs every step
  if (flags & (GNNCO_WANT_DX | GNNCO_AX_STORE | GNNCO_AX_REUSE)) return GNNCO_UNSUPPORTED;
  if ((uintptr_t)ws & 255) return GNNCO_INVALID_ARGUMENT;
  TrainLayout T = carve_train(h, m, flags, ws, true);
  if (T.bytes > ws_bytes) return GNNCO_WORKSPACE_TOO_SMALL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t n = (size_t)h->n;
  const size_t row_bytes = (size_t)m->dims[0] * elem_size(m->feat_dtype);
  gnnco_objective obj{alpha, beta, lambda, nullptr};
  if (pen_host) obj.pen = T.pen_stage;
  gnnco_train_out out{};
  out.loss = T.loss_stage;
  out.p = T.p_stage;
  // Large inputs arrive in ranges of subgraphs on a second stream, and the first hidden layer (which needs nothing
  // but a subgraph's own rows of X) follows them range by range; the rest of the step starts when all are there.
  // Results are those of the plain order bit for bit: every subgraph is cut into the same tiles.
  ArrivalPlan plan;
  const bool in_ranges = m->L >= 2 && h->S >= 2 && !(flags & GNNCO_ACTIVE_ONLY) && n * row_bytes >= ((size_t)64 << 20);
  if (in_ranges) {
    if (!h->copy_stream) {
      GNNCO_CUDA_TRY(cudaStreamCreateWithFlags(&h->copy_stream, cudaStreamNonBlocking));
      for (cudaEvent_t& e : h->ev_arrive) GNNCO_CUDA_TRY(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
      GNNCO_CUDA_TRY(cudaEventCreateWithFlags(&h->ev_rest, cudaEventDisableTiming));
      GNNCO_CUDA_TRY(cudaEventCreateWithFlags(&h->ev_begin, cudaEventDisableTiming));
    }
    // whatever the caller queued on `stream` before this call comes first
    GNNCO_CUDA_TRY(cudaEventRecord(h->ev_begin, st));
    GNNCO_CUDA_TRY(cudaStreamWaitEvent(h->copy_stream, h->ev_begin, 0));
    const std::vector<int32_t>& pp = h->h_part_ptr;
    int32_t tiles = 0, pairs = 0, s = 0;
    for (int g = 0; g < kArrivalGroups; ++g) {
      plan.tile0[g] = tiles;
      plan.pair0[g] = pairs;
      const int32_t s_begin = s;
      const int64_t until = g + 1 == kArrivalGroups ? (int64_t)n : (int64_t)n * (g + 1) / kArrivalGroups;
      while (s < h->S && (pp[s + 1] <= until || g + 1 == kArrivalGroups)) {
        const int32_t rows = pp[s + 1] - pp[s];
        tiles += (rows + kGemmTileRows - 1) / kGemmTileRows;
        pairs += (rows + 2 * kGemmTileRows - 1) / (2 * kGemmTileRows);
        ++s;
      }
      const size_t r0 = (size_t)pp[s_begin], r1 = (size_t)pp[s];
      if (r1 > r0)
        GNNCO_CUDA_TRY(cudaMemcpyAsync(static_cast<char*>(T.X_stage) + r0 * row_bytes,
                                       static_cast<const char*>(X_host) + r0 * row_bytes, (r1 - r0) * row_bytes,
                                       cudaMemcpyHostToDevice, h->copy_stream));
      plan.ev[g] = h->ev_arrive[g];
      GNNCO_CUDA_TRY(cudaEventRecord(plan.ev[g], h->copy_stream));
    }
    plan.tile0[kArrivalGroups] = tiles;
    plan.pair0[kArrivalGroups] = pairs;
    plan.groups = kArrivalGroups;
    if (tiles != h->n_tiles || pairs != h->n_pairs) return GNNCO_INTERNAL;
    if (pen_host)
      GNNCO_CUDA_TRY(cudaMemcpyAsync(T.pen_stage, pen_host, n * sizeof(float), cudaMemcpyHostToDevice, h->copy_stream));
    plan.ev_rest = h->ev_rest;
    GNNCO_CUDA_TRY(cudaEventRecord(plan.ev_rest, h->copy_stream));
    h->arrival = &plan;
    rc = run_step(h, m, T.X_stage, &obj, opt, &out, flags, T, st);
    h->arrival = nullptr;
  } else {
    GNNCO_CUDA_TRY(cudaMemcpyAsync(T.X_stage, X_host, n * row_bytes, cudaMemcpyHostToDevice, st));
    if (pen_host)
      GNNCO_CUDA_TRY(cudaMemcpyAsync(T.pen_stage, pen_host, n * sizeof(float), cudaMemcpyHostToDevice, st));
    rc = run_step(h, m, T.X_stage, &obj, opt, &out, flags, T, st);
  }
  if (rc != GNNCO_OK) {
    cudaStreamSynchronize(st);                      // nothing of this call is in flight when it returns an error
    if (h->copy_stream) cudaStreamSynchronize(h->copy_stream);
    return rc;
  }
  GNNCO_CUDA_TRY(cudaMemcpyAsync(loss_host, T.loss_stage, (size_t)h->S * sizeof(float), cudaMemcpyDeviceToHost, st));
  GNNCO_CUDA_TRY(cudaMemcpyAsync(p_host, T.p_stage, n * sizeof(float), cudaMemcpyDeviceToHost, st));
  GNNCO_CUDA_TRY(cudaStreamSynchronize(st));
  return GNNCO_OK;
}
