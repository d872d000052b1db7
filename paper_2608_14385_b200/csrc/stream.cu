#include "stream.cuh"

namespace deamoe {
struct StreamPlan { int dummy; };
int stream_default_schedule() { return DEAMOE_SCHED_PLAIN; }
deamoe_status_t stream_plan_create(const LayerDev&, const deamoe_weights_t&, int, cudaStream_t, StreamPlan**,
                                   uint64_t*) {
  return DEAMOE_ERR_UNSUPPORTED;
}
void stream_plan_destroy(StreamPlan*) {}
int stream_build_worklist(StreamPlan&, const LayerDev&, int, cudaStream_t) { return -1; }
int stream_forward(StreamPlan&, const LayerDev&, int, cudaStream_t) { return -1; }
}  // namespace deamoe
