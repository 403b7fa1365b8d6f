// Fine-tuning on SOME subgraphs (Section 3.3: resolving a conflict fine-tunes the model of ONE endpoint's
// subgraph; Algorithm 1, Stage 3 groups the chosen actions by subgraph and fine-tunes those).  A
// training step costs what its rows cost, so a fine-tuning step should cost what the ACTIVE subgraphs'
// rows cost.  gnnco_active_plan turns the device flags `active` [S] into a second set of work tables
// (tiles, double tiles, objective items, weight-gradient chunks, 256-row chunks) that lists the active
// subgraphs only; a gnnco_train_step with GNNCO_ACTIVE_ONLY then runs every kernel over that set.
// The tables are built on the host from the subgraph boundaries that partition_load kept (the same
// code that builds the full set), so an active subgraph is cut into exactly the same tiles, items and
// chunks as in a full step and its results are bit-identical.
#include "internal.cuh"

namespace {

struct PlanLayout {
  int32_t *tile_row0, *tile_rows, *pair_row0, *pair_rows, *item_row0, *item_row1, *part_item_ptr;
  int32_t *wg_begin, *wg_end, *wg_slot, *wg_mpart, *wg_mfirst, *wg_mcount, *chunk_row0, *chunk_rows;
  FuseSet fuse;
  size_t bytes;
};

// worst case: every subgraph active
PlanLayout carve_plan(void* base, int64_t n, int32_t S) {
  PlanLayout L;
  Carver c(base, ~(size_t)0);
  const size_t tiles = (size_t)(n / kGemmTileRows + S + 1);
  const size_t items = (size_t)(n / kItemRows + S + 1);
  const size_t chunks = (size_t)(S + n / kWgChunkMinRows + 1);
  const size_t rows256 = (size_t)(n / 256 + S + 1);
  L.tile_row0 = c.take<int32_t>(tiles);
  L.tile_rows = c.take<int32_t>(tiles);
  L.pair_row0 = c.take<int32_t>(tiles);
  L.pair_rows = c.take<int32_t>(tiles);
  L.item_row0 = c.take<int32_t>(items);
  L.item_row1 = c.take<int32_t>(items);
  L.part_item_ptr = c.take<int32_t>((size_t)S + 1);
  L.wg_begin = c.take<int32_t>(chunks);
  L.wg_end = c.take<int32_t>(chunks);
  L.wg_slot = c.take<int32_t>(chunks);
  L.wg_mpart = c.take<int32_t>((size_t)S);
  L.wg_mfirst = c.take<int32_t>((size_t)S);
  L.wg_mcount = c.take<int32_t>((size_t)S);
  L.chunk_row0 = c.take<int32_t>(rows256);
  L.chunk_rows = c.take<int32_t>(rows256);
  L.fuse = carve_fuse_set(c, tiles);
  L.bytes = c.off;
  return L;
}

}  // namespace

extern "C" int32_t gnnco_active_plan_bytes(const gnnco_handle* h, size_t* bytes) {
  if (!h || !bytes) return GNNCO_INVALID_ARGUMENT;
  *bytes = carve_plan(nullptr, h->n, h->S).bytes;
  return GNNCO_OK;
}

extern "C" int32_t gnnco_active_plan(gnnco_handle* h, const uint8_t* active, void* plan_ws, size_t plan_bytes,
                                    void* stream, int32_t* active_count) {
  if (!h || !active || !plan_ws) return GNNCO_INVALID_ARGUMENT;
  if ((uintptr_t)plan_ws & 255) return GNNCO_INVALID_ARGUMENT;
  PlanLayout P = carve_plan(plan_ws, h->n, h->S);
  if (P.bytes > plan_bytes) return GNNCO_WORKSPACE_TOO_SMALL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  h->plan_active_count = -1;
  std::vector<uint8_t> flags((size_t)h->S);
  GNNCO_CUDA_TRY(cudaMemcpyAsync(flags.data(), active, flags.size(), cudaMemcpyDeviceToHost, st));
  GNNCO_CUDA_TRY(cudaStreamSynchronize(st));
  HostWorkTables tab;
  build_work_tables(h->h_part_ptr, h->S, h->n, h->sm_count, flags.data(), tab);
  auto up = [&](int32_t* dst, const std::vector<int32_t>& v) {
    return v.empty() ? cudaSuccess
                     : cudaMemcpyAsync(dst, v.data(), v.size() * sizeof(int32_t), cudaMemcpyHostToDevice, st);
  };
  GNNCO_CUDA_TRY(up(P.tile_row0, tab.t0));
  GNNCO_CUDA_TRY(up(P.tile_rows, tab.tr));
  GNNCO_CUDA_TRY(up(P.pair_row0, tab.p0));
  GNNCO_CUDA_TRY(up(P.pair_rows, tab.pr));
  GNNCO_CUDA_TRY(up(P.item_row0, tab.i0));
  GNNCO_CUDA_TRY(up(P.item_row1, tab.i1));
  GNNCO_CUDA_TRY(up(P.part_item_ptr, tab.pip));
  GNNCO_CUDA_TRY(up(P.wg_begin, tab.wb));
  GNNCO_CUDA_TRY(up(P.wg_end, tab.we));
  GNNCO_CUDA_TRY(up(P.wg_slot, tab.wsl));
  GNNCO_CUDA_TRY(up(P.wg_mpart, tab.mp));
  GNNCO_CUDA_TRY(up(P.wg_mfirst, tab.mf));
  GNNCO_CUDA_TRY(up(P.wg_mcount, tab.mc));
  GNNCO_CUDA_TRY(up(P.chunk_row0, tab.c0));
  GNNCO_CUDA_TRY(up(P.chunk_rows, tab.cr));
  GNNCO_CUDA_TRY(cudaStreamSynchronize(st));      // the host vectors go out of scope
  WorkSet& w = h->plan;
  w.tile_row0 = P.tile_row0; w.tile_rows = P.tile_rows; w.pair_row0 = P.pair_row0; w.pair_rows = P.pair_rows;
  w.item_row0 = P.item_row0; w.item_row1 = P.item_row1; w.part_item_ptr = P.part_item_ptr;
  w.wg_begin = P.wg_begin; w.wg_end = P.wg_end; w.wg_slot = P.wg_slot;
  w.wg_mpart = P.wg_mpart; w.wg_mfirst = P.wg_mfirst; w.wg_mcount = P.wg_mcount;
  w.n_tiles = (int32_t)tab.t0.size(); w.n_pairs = (int32_t)tab.p0.size(); w.n_items = (int32_t)tab.i0.size();
  w.n_wg_chunks = (int32_t)tab.wb.size(); w.n_wg_multi = (int32_t)tab.mp.size();
  w.row_chunks.row0 = P.chunk_row0; w.row_chunks.rows = P.chunk_rows; w.row_chunks.count = (int32_t)tab.c0.size();
  w.fuse = P.fuse;
  {
    const int32_t rc = build_fuse_set(h, P.pair_row0, P.pair_rows, tab.p0, tab.pr, w.fuse, st);
    if (rc != GNNCO_OK) return rc;
  }
  int32_t count = 0;
  for (uint8_t f : flags) count += f ? 1 : 0;
  h->plan_active = active;
  h->plan_active_count = count;
  if (active_count) *active_count = count;
  return GNNCO_OK;
}
