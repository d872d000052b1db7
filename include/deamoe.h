/*
 * deamoe.h -- C ABI of the B200 (sm_100a) decode forward of one DeaMoE layer.
 *
 * One layer = a router, m departments that each own three large SwiGLU matrices
 * shared by their experts, and n = m*g experts that each own three small private
 * matrices (paper Section 3.1, Eq. (4)).  A decode step routes B tokens to their
 * top-k experts (Eq. (2)), gathers the tokens of every department once, streams the
 * department's matrices from HBM once for all of them, applies the selected experts'
 * private matrices, and combines with the gate weights (Eq. (3)) -- the two-stage
 * schedule of Section 3.2.  The same library builds the standard MoE layer of
 * Eq. (1)-(3) at the same shape as a comparator.
 *
 * Conventions that hold for every entry point:
 *  - Pointers marked DEVICE are CUDA device pointers of the current device; pointers
 *    marked HOST are ordinary host pointers.  `cuda_stream` is a cudaStream_t passed as
 *    void* (NULL = the legacy default stream).
 *  - All matrices are dense, row-major, 16-byte aligned.  A device pointer to tokens, outputs or a
 *    router matrix that is not 16-byte aligned is rejected with DEAMOE_ERR_INVALID_ARG (the kernels
 *    use 16-byte accesses and bulk copies); topk_idx / topk_w need 4-byte alignment.
 *  - Every call returns a deamoe_status_t; nothing aborts, traps or throws.  Argument
 *    errors are detected on the host before anything is enqueued.
 *  - deamoe_route / deamoe_forward only ENQUEUE work on the given stream; they never
 *    synchronise and never allocate (all workspace is sized at create for max_batch).
 *    Calls on one layer must be enqueued on one stream (or otherwise ordered): a layer has one
 *    workspace.  A step keeps no per-step state on the host, so it may be captured into a CUDA
 *    graph and replayed (Section 5 of the paper runs its steps that way).
 *  - The weight-streaming and dense kernels are PERSISTENT grids sized to fill the device (every
 *    SM, two thread blocks each) whose blocks wait for one another's results, so all blocks of a
 *    launch must be resident at the same time; consecutive kernels of one step are launched
 *    programmatically and run beside one another, handing over through counters in device memory
 *    rather than at kernel boundaries.  Run one such step per device at a time: if another
 *    kernel holds SMs while a step runs (a second layer driven from another stream, another process
 *    under MPS, a long-running communication kernel), blocks that cannot become resident keep the
 *    others waiting.  Nothing hangs or faults in that case -- every device-side wait is bounded --
 *    but when a wait expires the step's output is invalid and deamoe_get_stats reports
 *    DEAMOE_ERR_TIMEOUT in the device status word; the layer is usable again for the next call.
 *    Layers enqueued one after another on ONE stream (a model's stack) are the intended use.
 *  - There is no CPU fallback and no other backend: without a CUDA device the create
 *    calls fail with DEAMOE_ERR_CUDA.
 */
#ifndef DEAMOE_H
#define DEAMOE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct deamoe_layer deamoe_layer_t; /* opaque, owned by the library */

typedef enum {
  DEAMOE_OK = 0,
  DEAMOE_ERR_INVALID_ARG = 1, /* NULL pointer, inconsistent or non-positive sizes */
  DEAMOE_ERR_UNSUPPORTED = 2, /* a valid request this build has no kernel for */
  DEAMOE_ERR_ALLOC = 3,       /* device or host allocation failed */
  DEAMOE_ERR_CUDA = 4,        /* a CUDA runtime call failed (no device, launch error) */
  DEAMOE_ERR_BATCH = 5,       /* B < 0 or B > max_batch */
  DEAMOE_ERR_TIMEOUT = 6,     /* a bounded device-side wait expired (reported by get_stats) */
  DEAMOE_ERR_INTERNAL = 7     /* a device-side consistency check failed; the access was skipped (get_stats) */
} deamoe_status_t;

typedef enum { DEAMOE_F32 = 0, DEAMOE_BF16 = 1 } deamoe_dtype_t;

/* sigma of Section 3.1: the non-linearity between department and expert projections */
typedef enum {
  DEAMOE_SIGMA_NONE = 0,
  DEAMOE_SIGMA_SILU = 1,    /* the paper's choice (Section 3.4) */
  DEAMOE_SIGMA_GELU = 2,
  DEAMOE_SIGMA_RMSNORM = 3  /* v / sqrt(mean(v^2) + 1e-6) over the whole length-f vector, no gain; needs priv > 0 */
} deamoe_sigma_t;

/* how one forward is issued */
typedef enum {
  DEAMOE_SCHED_AUTO = 0,   /* the library's best schedule for the dtype */
  DEAMOE_SCHED_PLAIN = 1,  /* one simple kernel per stage on the canonical layouts (any dtype) */
  DEAMOE_SCHED_STAGED = 2, /* bf16 weight-streaming kernel, one launch per stage */
  DEAMOE_SCHED_FUSED = 3,  /* bf16 weight-streaming kernel, one persistent launch for all stages */
  DEAMOE_SCHED_DENSE = 4   /* larger batches, where a department's token bucket X^j (Section 3.2) is a
                              dense tile: department and shared-expert matrices on the tcgen05 tensor
                              cores, private matrices in the streaming kernel.  bf16 weights and
                              tokens, a DeaMoE layer with private matrices, h a multiple of 256,
                              f and shared_ffn of 128; else UNSUPPORTED.  AUTO takes this schedule by
                              itself for calls of 32 tokens and more (64 and more on layers of fewer than 64 experts) on
                              layers that support it. */
} deamoe_schedule_t;

/*
 * Layer description (Section 3.1 / 3.2; Table 1 uses the same symbols).
 * Expert i belongs to department i / experts_per_dept.
 */
typedef struct {
  int32_t hidden;           /* h */
  int32_t n_dept;           /* m */
  int32_t experts_per_dept; /* g; n = m*g experts */
  int32_t ffn;              /* f = h_ffn: department (and standard expert) intermediate size */
  int32_t priv;             /* r: private matrices A_g, A_u, A_d are [r, f].  r == f is the paper's
                               square form.  0 = no private parameters (A = identity, nothing is
                               stored or loaded; sigma is still applied as configured). */
  int32_t top_k;            /* k_expert of Eq. (2) */
  int32_t k_dept;           /* 0 = flat top-k.  > 0 = group-limited routing (Section 3.3): only the
                               k_dept departments with the largest best logit stay eligible. */
  int32_t n_shared;         /* 0 or 1 always-on shared SwiGLU expert (Eq. (1), weight 1) */
  int32_t shared_ffn;       /* its intermediate size */
  int32_t sigma;            /* deamoe_sigma_t */
  int32_t norm_topk;        /* 1: p = softmax over the k selected logits; 0: softmax over all n, not
                               renormalised; 2 (a variant the paper does not have): logistic
                               function of the k selected logits divided by their sum.  The
                               selection is by raw logit (Eq. (2)) in every case. */
  int32_t weight_dtype;     /* deamoe_dtype_t of department / private / shared matrices */
  int32_t act_dtype;        /* deamoe_dtype_t of tokens and out */
  int32_t residual;         /* 1: out = tokens + layer(tokens) */
  int32_t max_batch;        /* largest B any later call may pass (1..DEAMOE_MAX_BATCH) */
  int32_t schedule;         /* deamoe_schedule_t */
  float route_scale;        /* gate weights are multiplied by this (Eq. (3) "scaling") */
  int32_t strict_dept;      /* 1 (with k_dept > 0): strict department coverage, the variant Section 3.3
                               evaluates and rejects: while a token's selection spans fewer than
                               min(k_dept, k) departments, its lowest-ranked selected expert whose
                               department holds another selected expert is replaced, in place, by
                               the expert with the largest logit (ties: lowest index) of the
                               departments not yet covered.  Needs n_dept <= 64.  0: the soft cap. */
  int32_t dept_begin, dept_end; /* 0, 0: the whole layer.  Otherwise this object is the SLICE of the layer
                               that holds departments [dept_begin, dept_end) and their experts -- a
                               department with its experts' private matrices is an independent unit
                               (Section 3.1 / 3.2), so a layer can be spread over several GPUs by
                               department.  See deamoe_forward_partial. */
} deamoe_config_t;

#define DEAMOE_MAX_BATCH 128
#define DEAMOE_MAX_TOPK 32
#define DEAMOE_MAX_EXPERTS 2048

/*
 * Weights in their canonical layouts.  All DEVICE pointers, caller-owned, read only
 * during create (the library keeps its own re-packed copy, so the caller may free
 * them as soon as create returns and the stream has been synchronised).
 *
 *   router                       [n, h]  fp32 always (Eq. (2))
 *   dept_gate, dept_up           [m, f, h]   W_g^j, W_u^j
 *   dept_down                    [m, f, h]   W_d^j, applied transposed: (W_d^j)^T z
 *   priv_gate, priv_up           [n, r, f]   A_g^i, A_u^i
 *   priv_down                    [n, r, f]   A_d^i, applied transposed: (A_d^i)^T y
 *   shared_gate/up/down          [shared_ffn, h]
 * priv_* must be NULL iff priv == 0; shared_* must be NULL iff n_shared == 0.
 * For a department slice (dept_begin, dept_end) the router is still the whole [n, h] matrix (every
 * slice routes all tokens, identically), while dept_* hold only the slice's departments,
 * [dept_end - dept_begin, f, h], and priv_* only their experts, [(dept_end - dept_begin) * g, r, f].
 * For deamoe_vanilla_create the dept_* pointers hold the n standard experts, [n, f, h].
 */
typedef struct {
  const float *router;
  const void *dept_gate, *dept_up, *dept_down;
  const void *priv_gate, *priv_up, *priv_down;
  const void *shared_gate, *shared_up, *shared_down;
} deamoe_weights_t;

/*
 * Build a DeaMoE layer (Section 3.1).  Allocates the library's weight copy and all
 * workspace for max_batch tokens, enqueues the re-packing on `cuda_stream` and
 * synchronises it before returning.  *out is set only on DEAMOE_OK.
 * Errors: INVALID_ARG (NULL, sizes <= 0, top_k > n, priv/shared pointers inconsistent with
 * the sizes), UNSUPPORTED (bf16 streaming schedules need h, f, r, shared_ffn to be multiples
 * of 16; n > DEAMOE_MAX_EXPERTS; top_k > DEAMOE_MAX_TOPK), BATCH, ALLOC, CUDA.
 */
deamoe_status_t deamoe_layer_create(const deamoe_config_t *cfg, const deamoe_weights_t *weights,
                                    void *cuda_stream, deamoe_layer_t **out);

/* Standard MoE comparator, Eq. (1)-(3): n experts of three [f, h] matrices, same router
 * semantics, same optional shared expert.  cfg->priv must be 0; sigma is ignored. */
deamoe_status_t deamoe_vanilla_create(const deamoe_config_t *cfg, const deamoe_weights_t *weights,
                                      void *cuda_stream, deamoe_layer_t **out);

/* Frees everything the layer owns.  The caller must make sure no work of this layer is
 * still running.  NULL is accepted. */
deamoe_status_t deamoe_layer_destroy(deamoe_layer_t *layer);

/*
 * Routing only (Eq. (2), gate weights of Eq. (3), department sets of Section 3.2).
 * tokens: DEVICE [B, h] in act_dtype.  Fills the layer's device-side routing state and, where
 * non-NULL, the caller's DEVICE outputs topk_idx [B, k] (experts in order of decreasing logit,
 * ties to the lower index) and topk_w [B, k] fp32.  B == 0 is a no-op.
 */
deamoe_status_t deamoe_route(deamoe_layer_t *layer, void *cuda_stream, const void *tokens, int32_t B,
                             int32_t *topk_idx, float *topk_w);

/*
 * One decode step of the layer: out[B, h] = sum_{i in S(x)} p_i Expert_i(x) (+ shared expert)
 * (+ x if residual), Eq. (3) with Eq. (4) (DeaMoE layer) or Eq. (1) (vanilla layer), evaluated
 * with the two-stage schedule of Section 3.2.  tokens, out: DEVICE [B, h] in act_dtype; out must
 * not alias tokens.  Includes routing.  B == 0 is a no-op.
 */
deamoe_status_t deamoe_forward(deamoe_layer_t *layer, void *cuda_stream, const void *tokens, int32_t B,
                               void *out);

/*
 * Department-sharded execution (Section 3.1 / 3.2: the departments are independent units; Eq. (3) is a
 * sum over the selected experts, so it splits over any partition of the departments).  Every GPU
 * creates the slice of the layer that holds its departments (cfg.dept_begin / dept_end; exactly one
 * slice is created with the shared expert, if there is one), gets the same tokens, and calls
 *
 *   deamoe_forward_partial: partial[B, h] (DEVICE, fp32, 16-byte aligned) =
 *       sum over the token's selected experts THAT LIVE IN THIS SLICE of p_i Expert_i(x)
 *       (+ the shared expert if this slice has it); no residual, no rounding to the activation dtype.
 *       Routing is computed in full by every slice (same router, same tokens, same result); its
 *       department sets, token lists and byte counters (deamoe_get_routing / deamoe_get_stats)
 *       cover the slice's own departments only.
 *
 * The caller adds the partial sums of all slices element by element (one all-reduce of B * h
 * floats; any order is correct up to fp32 rounding) and calls, on any slice object,
 *
 *   deamoe_finish_partial: out[B, h] (DEVICE, act_dtype) = sum (+ tokens if cfg.residual).
 *
 * Both only enqueue on the stream.  deamoe_forward_partial also works on a whole (unsliced) DeaMoE
 * layer; deamoe_forward on a slice is INVALID_ARG (a slice alone does not compute the layer).
 */
deamoe_status_t deamoe_forward_partial(deamoe_layer_t *layer, void *cuda_stream, const void *tokens, int32_t B,
                                       float *partial);
deamoe_status_t deamoe_finish_partial(deamoe_layer_t *layer, void *cuda_stream, const float *sum,
                                      const void *tokens, int32_t B, void *out);

/* The same step for a layer made by deamoe_vanilla_create (INVALID_ARG for a DeaMoE layer). */
deamoe_status_t deamoe_vanilla_forward(deamoe_layer_t *layer, void *cuda_stream, const void *tokens,
                                       int32_t B, void *out);

/*
 * End-to-end step on HOST buffers: copies tokens (HOST [B, h], act_dtype, ideally pinned) to a
 * device staging buffer owned by the layer, runs deamoe_forward, brings the result to `out`
 * (HOST [B, h]) and synchronises the stream before returning.  When `out` is pinned memory the
 * device can address, the last kernel of the step writes into it directly; otherwise the result is
 * copied from a staging buffer.
 */
deamoe_status_t deamoe_forward_host(deamoe_layer_t *layer, void *cuda_stream, const void *tokens,
                                    int32_t B, void *out);

/*
 * Copy the routing state of the LAST route/forward call to HOST buffers (synchronises the
 * given stream first).  Any pointer may be NULL.  Sizes: topk_idx/topk_w [B*k]; dept_mask
 * [ceil(m/64)] (bit j of word j/64 = department j active); dept_off [m+1] and dept_tok
 * [dept_off[m]] = the distinct tokens of each department, ascending (X^j of Section 3.2);
 * expert_off [n+1] and expert_tok [B*k] likewise per expert.
 */
deamoe_status_t deamoe_get_routing(deamoe_layer_t *layer, void *cuda_stream, int32_t *topk_idx,
                                   float *topk_w, uint64_t *dept_mask, int32_t *dept_off,
                                   int32_t *dept_tok, int32_t *expert_off, int32_t *expert_tok);

/*
 * Counters of the LAST route/forward call (synchronises the stream first), HOST outputs, any may
 * be NULL: active departments |D|, active experts |E|, (token, department) pairs, the unique weight
 * bytes the step had to load (|D|*3hf*s + |E|*3rf*s + shared + 4nh for DeaMoE; |E|*3hf*s + shared +
 * 4nh for vanilla), and the device status word (DEAMOE_OK, DEAMOE_ERR_TIMEOUT or DEAMOE_ERR_INTERNAL).
 */
deamoe_status_t deamoe_get_stats(deamoe_layer_t *layer, void *cuda_stream, int32_t *n_active_dept,
                                 int32_t *n_active_expert, int32_t *n_token_dept_pairs,
                                 uint64_t *unique_weight_bytes, int32_t *device_status);

/*
 * Measurement aid.  With profiling enabled the forward calls of this layer record a CUDA event on
 * their stream before the first and after the last weight-streaming launch (the stages of
 * Section 3.2; routing, bucketing and the final combine of Eq. (3) lie outside the pair).
 * deamoe_profile_last_ms synchronises on the second event and returns the time between them in
 * *ms (HOST).  Errors: INVALID_ARG (NULL, profiling off, or no forward since it was enabled),
 * UNSUPPORTED for the plain schedule, CUDA.
 */
deamoe_status_t deamoe_profile_enable(deamoe_layer_t *layer, int32_t enable);
deamoe_status_t deamoe_profile_last_ms(deamoe_layer_t *layer, float *ms);

/*
 * Routing for callers that must not allocate.  (The paper has no counterpart: this is an
 * integration convenience of the library, not part of the method.)
 *
 * Some hosts of this library cannot call cudaMalloc at the point where they need a routing
 * decision: code that runs while a stream is being captured into a CUDA graph, a latency-critical
 * serving loop in which an allocation would synchronise the whole device, or a plug-in that is
 * handed a stream and pre-allocated buffers by a framework that owns all device memory.  A layer
 * object (deamoe_layer_create) is out of reach for them because it allocates its workspace.  This
 * entry point computes the same routing -- Eq. (2) top-k, ties to the lower index, and the gate
 * weights of Eq. (3), flat top-k only -- without creating anything: the partial logits, the one
 * piece of scratch the two routing kernels need, live in a fixed array of
 * DEAMOE_STATIC_ROUTE_SCRATCH_BYTES inside the library image (every GPU that loads the library
 * holds those bytes until the process exits).
 *
 *   router   DEVICE [n, hidden] fp32,  n = n_dept * experts_per_dept
 *   tokens   DEVICE [B, hidden] fp32 (16-byte aligned)
 *   topk_idx DEVICE [B, top_k] out, topk_w DEVICE [B, top_k] out (fp32)
 *
 * Limits: slices * B * n * 4 bytes must fit the fixed array, where slices (1, 2, 4, 8 or 16) is the
 * number of column slices the logits kernel uses for this n and hidden -- the same rule as a layer
 * object's: doubled while a slice is wider than 512 columns and (n / 4) * slices, doubled, stays at or
 * below 740.  A larger request returns DEAMOE_ERR_BATCH and enqueues nothing.  (DeepSeek-V3 layout,
 * n = 256, hidden = 7168: 8 slices, B up to 512; n = 2048, hidden = 7168: 1 slice, B up to 512;
 * hidden <= 512: 1 slice.)  Other errors as for deamoe_route.
 *
 * The first call on each device resolves the array's device address and sets one kernel
 * attribute (the device must be current); make that first call before any stream capture begins.
 * Later calls only enqueue two kernels on `cuda_stream`.  All calls share the one array and it
 * keeps the previous call's contents: nothing has to be cleared, because every entry a call reads
 * it has first written itself, but two calls that overlap on the GPU (different streams, or the
 * same array used from two threads) race on it -- serialise them.  The one-time set-up itself is
 * safe to reach from several host threads at once.
 */
#define DEAMOE_STATIC_ROUTE_SCRATCH_BYTES (4u << 20)
deamoe_status_t deamoe_route_static(void *cuda_stream, const float *router, const float *tokens,
                                    int32_t n_dept, int32_t experts_per_dept, int32_t hidden, int32_t top_k,
                                    int32_t norm_topk, float route_scale, int32_t B, int32_t *topk_idx,
                                    float *topk_w);

/*
 * Measurement aid.  (The paper has no counterpart.)  Enqueues one kernel that reads `bytes` bytes
 * of `buf` (DEVICE, 16-byte aligned; a trailing remainder of fewer than 16 bytes is ignored) exactly
 * once with plain 16-byte loads and writes one word per thread block to sink (DEVICE,
 * DEAMOE_PROBE_BLOCKS words, caller-owned).  Timed by the caller with events on a buffer much
 * larger than the L2, it gives the read-only HBM bandwidth of this GPU: the ceiling a
 * weight-streaming step is set against (the usual copy benchmark reads AND writes).  No layer needed.
 */
#define DEAMOE_PROBE_BLOCKS 2368
deamoe_status_t deamoe_probe_read(void *cuda_stream, const void *buf, uint64_t bytes, uint32_t *sink);

/*
 * Failure-detection test aid.  (The paper has no counterpart.)  Every device-side wait of the
 * library is bounded: after a number of polls it gives up, the kernel records DEAMOE_ERR_TIMEOUT
 * in the device status word, waits (bounded) for its copies in flight, frees its tensor memory
 * and returns.  This call lets a test see that path without faulting or hanging anything:
 *   wait_limit  polls after which a wait gives up in later calls on this layer (0 = the default);
 *   withhold    bit 0: the routing kernel does not raise the flags that hand the work list to the
 *               fused streaming kernel, so that kernel's planners wait until the limit expires;
 *               bit 1: the copy role of the dense (tcgen05) kernel issues no copies, so its MMA role
 *               waits for the ring until the limit expires;
 *               bit 2: the routing kernel publishes an out-of-range slot for the first (token,
 *               expert) pair, which the combine kernel's consistency check must skip and report
 *               as DEAMOE_ERR_INTERNAL (that pair's term is then missing from the output).
 *               0 = normal operation.
 * A step run with a withheld hand-over returns garbage in `out` and DEAMOE_ERR_TIMEOUT from
 * deamoe_get_stats; after deamoe_failure_test(layer, 0, 0) the layer works normally again.
 * Errors: INVALID_ARG; UNSUPPORTED if the layer's schedule has no such hand-over (plain / staged
 * schedule for bit 0, no dense schedule for bit 1).
 */
deamoe_status_t deamoe_failure_test(deamoe_layer_t *layer, int32_t wait_limit, int32_t withhold);

/* Number of kernels the last forward/route call of this layer launched (host-side count). */
int32_t deamoe_last_launches(const deamoe_layer_t *layer);

/* Bytes of device memory the layer owns (weights copy + workspace). */
uint64_t deamoe_device_bytes(const deamoe_layer_t *layer);

/* Static, never NULL. */
const char *deamoe_status_string(deamoe_status_t status);

#ifdef __cplusplus
}
#endif
#endif /* DEAMOE_H */
