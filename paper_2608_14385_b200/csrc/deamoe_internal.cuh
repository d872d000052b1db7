// Internal declarations shared by the translation units of libdeamoe.so.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "deamoe.h"


namespace deamoe {

#ifdef DEAMOE_TRACE
static __device__ __forceinline__ unsigned long long gtime() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
#define TS_MIN(L, i) do { if (threadIdx.x == 0 && (L).ts) atomicMin((L).ts + (i), gtime()); } while (0)
#define TS_MAX(L, i) do { if (threadIdx.x == 0 && (L).ts) atomicMax((L).ts + (i), gtime()); } while (0)
#define TS_PARAM , unsigned long long* ts
#define TS_ARG(L) , (L).ts
#else
#define TS_PARAM
#define TS_ARG(L)
#define TS_MIN(L, i) ((void)0)
#define TS_MAX(L, i) ((void)0)
#endif

// Stages of one decode step (Section 3.2 of the paper; SH* = shared expert, V* = vanilla MoE).
enum Stage : int {
  ST_S1 = 0,   // department gate/up:  GU = sigma([W_g; W_u] X^j)
  ST_S2 = 1,   // private gate/up:     Y = SiLU(A_g G) * (A_u U)
  ST_S3 = 2,   // private down:        Z = sigma(A_d^T Y)
  ST_S4 = 3,   // department down:     O = W_d^T Z
  ST_SH1 = 4,  // shared expert gate/up: Ysh = SiLU(W_sg x) * (W_su x)
  ST_SH2 = 5,  // shared expert down:    Osh = W_sd^T Ysh
  ST_V1 = 6,   // vanilla expert gate/up: Y = SiLU(W_gate x) * (W_up x)
  ST_V2 = 7,   // vanilla expert down:    O = W_down^T Y
  ST_COUNT = 8
};

enum Counter : int {
  CNT_ACTIVE_DEPT = 0,
  CNT_ACTIVE_EXPERT = 1,
  CNT_TOKEN_DEPT = 2,
  CNT_PAIRS = 3,
  CNT_STATUS = 4,
  CNT_NSEG = 5,
  CNT_NITEMS = 6,
  CNT_COUNT = 16
};

// Everything a kernel needs to know about the layer; passed by value.
struct LayerDev {
#ifdef DEAMOE_TRACE
  unsigned long long* ts;  // trace builds: globaltimer stamps of the kernels of one step
#endif
  // sizes
  int h, m, g, n, f, r, k, k_dept, n_shared, fs, sigma, norm_topk, residual, vanilla;
  int wdt, adt, max_batch;
  int strict_dept;  // 1: strict department coverage routing (with k_dept > 0)
  int dept_lo, dept_hi;  // departments [dept_lo, dept_hi) live in this layer object (all of them: 0, m); the
                         // weight arrays hold only those, the routing state lists only their tokens
  int rp;  // rows of Y per pair: r, or f when there are no private parameters
  float route_scale;
  // canonical weights (PLAIN schedule and fp32); element type per wdt
  const float* router;
  // the router matrix once more, for the tensor-core logits kernel of bf16-token layers: every fp32 value as
  // the exact sum of three bf16 pieces, in mma fragment order (k_pack_router3 in route.cu); or null
  const __nv_bfloat16* router3;
  int router3_slices;   // column slices that kernel uses (its partial-logit arrays)
  const void *dept_gate, *dept_up, *dept_down;
  const void *priv_gate, *priv_up, *priv_down;
  const void *shared_gate, *shared_up, *shared_down;
  // workspace
  const void* tokens_raw;  // the caller's tokens of this call, in act dtype
  float* x32;          // [MB, h] tokens widened to fp32 (aliases the caller's tokens when fp32)
  float* logit_part;   // [KS, MB, n]
  int32_t* topk_idx;   // [MB, k]
  float* topk_w;       // [MB, k]
  uint64_t* dept_mask; // [ceil(m/64)]
  int32_t* dept_off;   // [m+1]
  int32_t* dept_tok;   // [MB*min(k,m)]
  int32_t* expert_off; // [n+1]
  int32_t* expert_tok; // [MB*k]
  int32_t* pair_slot;  // [MB, k] slot of (t, q) in expert-major pair order
  int32_t* pair_gurow; // [MB*k] pair slot -> row of GU (its (token, department) row)
  int32_t* active_dept;   // [m]
  int32_t* active_expert; // [n]
  int32_t* counts;     // [CNT_COUNT]
  float* GU;           // [MB*min(k,m), 2f]
  float* Y;            // [MB*k, rp]   (vanilla: [MB*k, f])
  float* Z;            // [MB*k, f]
  float* O;            // [MB*k, h]
  float* Ysh;          // [MB, fs]
  float* Osh;          // [MB, h]
  int32_t* sh_done;    // counter the combine kernel resets at the end of a step, or null
  // sigma = RMSNorm: sums of squares of the un-normalised vectors, zeroed by the routing tail
  unsigned long long* ss_gu;  // [MB*min(k,m), 2]: G and U of every (token, department) row (fixed point, see ss_fixed)
  unsigned long long* ss_z;   // [MB*k]: Z of every pair
};

constexpr float RMS_EPS = 1e-6f;
// 1 / sqrt(mean(v^2) + eps) from a sum of squares over `width` elements
static __device__ __forceinline__ float rms_scale(float ss, int width) { return rsqrtf(ss / (float)width + RMS_EPS); }
// The streaming and dense kernels add the squares of a vector tile by tile, from many thread blocks
// in no fixed order.  The partial sums are therefore accumulated as 64-bit fixed-point integers
// (2^-30 resolution): integer addition is associative, so the total -- and with it the layer's
// output -- does not depend on the order of arrival.  A vector of f values loses at most
// f / 16 * 2^-31 of its sum of squares to the rounding of the partial sums, far below RMS_EPS * f.
constexpr float SS_FIXED_ONE = 1073741824.f;  // 2^30
static __device__ __forceinline__ unsigned long long ss_fixed(float sq) {
  return __float2ull_rn(fminf(sq * SS_FIXED_ONE, 4.0e18f));
}
static __device__ __forceinline__ float rms_scale_fixed(unsigned long long ss, int width) {
  return rms_scale(__ull2float_rn(ss) * (1.0f / SS_FIXED_ONE), width);
}

// Programmatic dependent launch: a kernel launched with launch_pdl() may start while its
// predecessor in the stream is still running (after the predecessor called pdl_trigger()); it must
// call pdl_wait() before touching anything the predecessor wrote.  Both are no-ops for a kernel that
// was launched the ordinary way.
static __device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
static __device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
static cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                              Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// Column slices of the router product (one grid row of k_router_logits per slice, one array of partial logits
// each): doubled while a slice is wider than 512 columns and the grid, blocks of four router rows times the slices,
// still fits the device in ONE wave (the 128-thread blocks are resident five to an SM, by their registers: 740 on a
// B200).  Measured on routers of 256 / 864 / 1280 experts and 7168 columns: 8 / 2 / 2 slices bring the logits in
// 3.9 / 8.9 / 10.9 us, the 16 / 8 / 4 of a second wave in 4.9 / 10.1 / 12.2 (and every slice is one more array
// the top-k has to read back).  The slices' partial sums are added in slice order, so every caller that wants the
// same fp32 logits must use the same count: the layer object and deamoe_route_static both call this.
static inline int router_kslices(int n, int h) {
  int ks = 1;
  while (ks < 16 && h / ks > 512 && (n / 4) * (2 * ks) <= 740) ks *= 2;
  return ks;
}

// The kernels read tokens and write outputs with 16-byte vector accesses and bulk copies.
static inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static __device__ __forceinline__ float silu_f(float v) { return v / (1.0f + __expf(-v)); }

static __device__ __forceinline__ float sigma_f(int kind, float v) {
  if (kind == DEAMOE_SIGMA_SILU) return silu_f(v);
  if (kind == DEAMOE_SIGMA_GELU) return 0.5f * v * (1.0f + erff(v * 0.70710678118654752f));
  return v;  // none; RMSNorm: the vector is stored un-normalised, its consumer applies rms_scale()
}

// host-side launchers (each returns the number of kernels it launched, or -1 on a launch error)
int launch_route(const LayerDev& L, const void* tokens, int B, cudaStream_t s, int kslices, int32_t* user_idx,
                 float* user_w);
size_t bucket_smem_bytes(const LayerDev& L, int B);
int launch_router_logits(const LayerDev& L, const void* tokens, int B, cudaStream_t s, int kslices,
                         int32_t* step_flag = nullptr);
cudaError_t route_configure(const LayerDev& L);
// Tensor-core router product (bf16 tokens): elements of the packed three-piece router, the column slices it is run
// with, and the packing itself (enqueued on s).
size_t router3_elems(int n, int h);
int router3_kslices(int n, int h);
cudaError_t pack_router3(const float* router, __nv_bfloat16* out, int n, int h, cudaStream_t s);
int launch_plain_forward(const LayerDev& L, int B, cudaStream_t s);
// partial != 0: fp32 output without the residual (the partial sum of a department-sharded layer)
int launch_combine(const LayerDev& L, const void* tokens, int B, void* out, cudaStream_t s, int partial = 0);
int launch_finish_partial(const LayerDev& L, const float* sum, const void* tokens, int B, void* out, cudaStream_t s);
int launch_probe_read(const void* src, size_t bytes, uint32_t* sink, int blocks, cudaStream_t s);

}  // namespace deamoe
