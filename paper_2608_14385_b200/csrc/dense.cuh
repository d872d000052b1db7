// Tensor-core (tcgen05 / TMEM) kernels for the stages whose token buckets are dense at larger
// batches: the department matrices (Section 3.2, first and last step) and the shared expert.
#pragma once
#include "deamoe_internal.cuh"

namespace deamoe {

struct DensePlan;

// Batches from this size on take the dense schedule when the layer has one (DEAMOE_SCHED_AUTO).
// Measured crossover: about 28 tokens on the DeepSeek-V3 shape, 16 - 32 on the layers of the paper's Table 1
// (256 - 1280 experts); a 7B-class layer of 4 x 4 experts crosses over near 64 (its first stage has fewer tile
// jobs than the device has CTAs), so layers of fewer than DENSE_SMALL_ROUTER experts switch at twice the size.
constexpr int DENSE_MIN_BATCH = 32;
constexpr int DENSE_SMALL_ROUTER = 64;

// True if the layer's shapes and dtypes fit the dense kernels (bf16 weights and activations, a
// DeaMoE layer with private matrices, h a multiple of 256, f and shared_ffn of 128).
bool dense_supported(const LayerDev& L);

// Copies the department and shared-expert matrices into the tile layout of the dense kernels
// (enqueued on `s`).  *bytes receives the device memory taken.
deamoe_status_t dense_plan_create(const LayerDev& L, const deamoe_weights_t& w, cudaStream_t s, DensePlan** out,
                                  uint64_t* bytes);
void dense_plan_destroy(DensePlan* p);

// Failure-detection tests: poll limit of the kernel's bounded waits (0 = default); withhold = 1: the
// copy role issues no copies, so the MMA role's wait for the ring must expire.
void dense_set_failure_test(DensePlan& p, unsigned spin_limit, int withhold);

// Enqueue one launch that runs the given stages (at most two, independent of each other) of one
// step.  in / out planes are the bf16 activation planes of the streaming schedule.  Returns the
// number of kernels launched or -1.
struct DenseIO {
  const __nv_bfloat16* tokens;  // [B, h]
  __nv_bfloat16* GU;            // [token-departments, 2f]
  const __nv_bfloat16* Z;       // [pairs, f]
  __nv_bfloat16* Ysh;           // [B, fs]
  int32_t* s1_done;             // per department: counts DENSE_S1_ARRIVALS per finished tile of its first stage
  const int32_t* routed_flag;   // set by the routing kernel once the departments' token lists are published
  int32_t* gathered;            // cleared by the step's router kernel: CTAs of the gather kernel that are done
  unsigned spin_limit;          // polls after which the wait for that flag gives up
};
// Tile height of the dense kernels and what one finished first-stage tile adds to its department's counter: a
// department's first stage is complete at DENSE_S1_ARRIVALS * (2 f / DENSE_TILE_ROWS).
constexpr int DENSE_TILE_ROWS = 128;
constexpr int DENSE_S1_ARRIVALS = 4;
int dense_launch(DensePlan& p, const LayerDev& L, const DenseIO& io, const int* stages, int n_stages, int B,
                 cudaStream_t s);

}  // namespace deamoe
