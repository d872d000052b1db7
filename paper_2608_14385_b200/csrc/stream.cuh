// Weight-streaming schedules (bf16): packed weights, device-built work list, persistent kernel.
#pragma once
#include "deamoe_internal.cuh"

namespace deamoe {

struct StreamPlan;

// The schedule DEAMOE_SCHED_AUTO resolves to for streamable bf16 layers.
int stream_default_schedule();

// Re-pack the canonical weights into the streaming layout (enqueued on `s`) and allocate the
// work-list buffers.  *bytes receives the device memory taken.
// dense_mode: 0 = never, 1 = from DENSE_MIN_BATCH tokens on (when the layer supports it), 2 = always (the
// layer must support it) take the dense schedule (tcgen05 kernels for the department and shared-expert stages).
deamoe_status_t stream_plan_create(const LayerDev& L, const deamoe_weights_t& w, int schedule, int dense_mode,
                                   cudaStream_t s, StreamPlan** out, uint64_t* bytes);
void stream_plan_destroy(StreamPlan* p);

// Routing for the streaming schedules: router logits, then ONE kernel for top-k + gate weights,
// bucketing and the work list.  Returns the number of kernels launched or -1.
// The completion counter of the shared expert's first stage when the fused schedule runs the
// shared expert ahead of the routing (else null).  The last kernel of a step must zero it.
int32_t* stream_shared_counter(StreamPlan& p);

int stream_route(StreamPlan& p, const LayerDev& L, const void* tokens, int B, cudaStream_t s, int kslices,
                 int32_t* user_idx, float* user_w);

// Enqueue all stages of one step.  Returns the number of kernels launched or -1.
int stream_forward(StreamPlan& p, const LayerDev& L, int B, cudaStream_t s);

// Failure-detection tests: poll limit of the bounded waits (0 = default) and withheld hand-overs
// (bit 0: the routing tail raises no flag for the fused streaming kernel; bit 1: the dense kernel's
// copy role issues nothing; bit 2: the routing tail publishes an out-of-range pair slot for the
// combine's consistency check).  False if the plan has no such hand-over.
bool stream_set_failure_test(StreamPlan& p, unsigned spin_limit, int withhold);

// Event pair around the streaming launches of stream_forward (measurement aid).
cudaError_t stream_profile_enable(StreamPlan& p, bool on);
cudaError_t stream_profile_last_ms(StreamPlan& p, float* ms);

#ifdef DEAMOE_TRACE
// Trace builds only: per-CTA cycle counters of the last streaming launch.
int stream_read_trace(StreamPlan& p, long long* host, int max_ctas);
#endif

}  // namespace deamoe
