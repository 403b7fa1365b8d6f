// Per-kernel timing of the training step and decoding (a measurement aid: the method's
// evaluation reports runtime, Section 4.1; this breaks a step's time down by kernel family).
#include <string.h>

#include "internal.cuh"

namespace {
const char* kKindNames[K_KIND_COUNT] = {
    "aggregate_fwd", "aggregate_bwd", "transform_fwd", "transform_bwd", "weight_grad", "gemv", "weight_grad_vec",
    "rank1_masked", "sum_over_sets", "cast_bf16", "adam", "output_forward", "objective", "output_backward", "decode",
    "stage3_glue", "aggregate_rank1", "embeddings", "aggregate_transform"};
}

extern "C" int32_t gnnco_profile_begin(gnnco_handle* h) {
  if (!h) return GNNCO_INVALID_ARGUMENT;
  h->prof.recs.clear();
  h->prof.used = 0;
  h->prof.on = true;
  return GNNCO_OK;
}

extern "C" int32_t gnnco_profile_end(gnnco_handle* h, void* stream, gnnco_profile_entry* entries, int32_t capacity,
                                    int32_t* count) {
  if (!h || !count || (capacity > 0 && !entries)) return GNNCO_INVALID_ARGUMENT;
  h->prof.on = false;
  GNNCO_CUDA_TRY(cudaStreamSynchronize(static_cast<cudaStream_t>(stream)));
  double total[K_KIND_COUNT] = {0};
  int64_t calls[K_KIND_COUNT] = {0};
  for (const Profiler::Rec& r : h->prof.recs) {
    float ms = 0.0f;
    GNNCO_CUDA_TRY(cudaEventElapsedTime(&ms, r.a, r.b));
    total[r.kind] += ms;
    calls[r.kind] += 1;
  }
  h->prof.recs.clear();
  h->prof.used = 0;
  int32_t k = 0;
  for (int kind = 0; kind < K_KIND_COUNT; ++kind) {
    if (!calls[kind]) continue;
    if (k < capacity) {
      memset(&entries[k], 0, sizeof(entries[k]));
      strncpy(entries[k].name, kKindNames[kind], sizeof(entries[k].name) - 1);
      entries[k].calls = calls[kind];
      entries[k].total_ms = total[kind];
    }
    ++k;
  }
  *count = k;
  return k <= capacity ? GNNCO_OK : GNNCO_WORKSPACE_TOO_SMALL;
}
