// Router (Eq. (2)), gate weights (Eq. (3)) and the department / expert token lists of
// Section 3.2, all on the device with no host round trip.
#include <atomic>
#include <cstring>
#include <mutex>

#include "deamoe_internal.cuh"
#include "route_device.cuh"

namespace deamoe {

// ---------------------------------------------------------------- tokens -> fp32
__global__ void k_widen_tokens(const __nv_bfloat16* __restrict__ tok, float* __restrict__ x32, size_t count) {
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  size_t stride = (size_t)gridDim.x * blockDim.x;
  for (; i < count; i += stride) x32[i] = __bfloat162float(tok[i]);
}

// ---------------------------------------------------------------- logits = W_r x   (fp32)
// CTA (bx, by): router rows [bx*RG, bx*RG+RG), columns [by*kslice, by*kslice+kslice).
// Partial sums go to part[by][t][row]; the top-k kernel adds the slices in a fixed order.
constexpr int RG = 4;   // router rows per CTA
constexpr int TG = 8;   // tokens per register tile
constexpr int ROUTER_THREADS = 128;

static __device__ __forceinline__ float4 load_x4(const float* p) { return *reinterpret_cast<const float4*>(p); }
static __device__ __forceinline__ float4 load_x4(const __nv_bfloat16* p) {
  const uint2 raw = *reinterpret_cast<const uint2*>(p);
  const __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162*>(&raw.x);
  const __nv_bfloat162 b = *reinterpret_cast<const __nv_bfloat162*>(&raw.y);
  return make_float4(__bfloat162float(a.x), __bfloat162float(a.y), __bfloat162float(b.x), __bfloat162float(b.y));
}

// XT = float: tokens already fp32; XT = bf16: tokens widened on the fly (exact).
template <typename XT>
__global__ void __launch_bounds__(ROUTER_THREADS)
k_router_logits(const float* __restrict__ Wr, const XT* __restrict__ x32, float* __restrict__ part,
                int n, int h, int B, int kslice, int32_t* __restrict__ step_flag TS_PARAM) {
#ifdef DEAMOE_TRACE
  if (threadIdx.x == 0 && ts) atomicMin(ts + 0, gtime());
#endif
  // step_flag (may be null): the word through which the routing tail tells the streaming kernel
  // that the first stage's records exist.  It is cleared here, before this grid releases its
  // dependents, so a streaming kernel can never see the value of the step before.
  if (step_flag && blockIdx.x == 0 && blockIdx.y == 0) {
    if (threadIdx.x == 0) {
      step_flag[0] = 0;
      step_flag[2] = 0;  // two words further: the flag that the rest of the work list exists
      step_flag[3] = 0;  // and the dense schedule's count of finished CTAs of its gather kernel
      __threadfence();
    }
    __syncthreads();
  }
  // Kernels launched behind this one with programmatic stream serialization (the routing tail, and
  // through it the streaming kernel with the routing-independent shared expert) may become
  // resident right away; they wait for this grid's results themselves.
  pdl_trigger();
  const int row0 = blockIdx.x * RG;
  const int c0 = blockIdx.y * kslice;
  const int c1 = min(h, c0 + kslice);
  __shared__ float red[ROUTER_THREADS / 32][RG][TG];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int t0 = 0; t0 < B; t0 += TG) {
    float acc[RG][TG];
#pragma unroll
    for (int a = 0; a < RG; ++a)
#pragma unroll
      for (int b = 0; b < TG; ++b) acc[a][b] = 0.f;
    for (int c = c0 + threadIdx.x * 4; c < c1; c += ROUTER_THREADS * 4) {
      float4 w[RG];
#pragma unroll
      for (int a = 0; a < RG; ++a) {
        const int row = min(row0 + a, n - 1);
        w[a] = __ldg(reinterpret_cast<const float4*>(Wr + (size_t)row * h + c));
      }
#pragma unroll
      for (int b = 0; b < TG; ++b) {
        const int t = min(t0 + b, B - 1);
        const float4 x = load_x4(x32 + (size_t)t * h + c);
#pragma unroll
        for (int a = 0; a < RG; ++a) {
          acc[a][b] = fmaf(w[a].x, x.x, acc[a][b]);
          acc[a][b] = fmaf(w[a].y, x.y, acc[a][b]);
          acc[a][b] = fmaf(w[a].z, x.z, acc[a][b]);
          acc[a][b] = fmaf(w[a].w, x.w, acc[a][b]);
        }
      }
    }
    // Warp reduction of the 32 accumulators by recursive halving: in the step with distance d a
    // lane keeps the half of its values that matches its lane bit d and adds the partner's, so
    // after five steps lane l holds the warp's total of accumulator l (31 shuffles, not 160).
    static_assert(RG * TG == 32, "one accumulator per lane after the reduction");
    float v[32];
#pragma unroll
    for (int a = 0; a < RG; ++a)
#pragma unroll
      for (int b = 0; b < TG; ++b) v[a * TG + b] = acc[a][b];
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
      const bool up = (lane & d) != 0;
#pragma unroll
      for (int i = 0; i < d; ++i) {
        const float send = up ? v[i] : v[i + d];
        const float keep = up ? v[i + d] : v[i];
        v[i] = keep + __shfl_xor_sync(0xffffffffu, send, d);
      }
    }
    red[warp][lane / TG][lane % TG] = v[0];
    __syncthreads();
    if (threadIdx.x < RG * TG) {
      const int a = threadIdx.x / TG, b = threadIdx.x % TG;
      float v = 0.f;
#pragma unroll
      for (int w = 0; w < ROUTER_THREADS / 32; ++w) v += red[w][a][b];
      if (row0 + a < n && t0 + b < B)
        part[((size_t)blockIdx.y * B + (t0 + b)) * n + row0 + a] = v;
    }
    __syncthreads();
  }
#ifdef DEAMOE_TRACE
  if (threadIdx.x == 0 && ts) atomicMax(ts + 1, gtime());
#endif
}

// ---------------------------------------------------------------- logits = W_r x on the tensor cores
// For bf16 tokens the fp32 product of Eq. (2) can run on mma.sync without losing a bit of the router: at
// create every fp32 router value w is split into three bf16 pieces, w = hi + mid + lo exactly (8 + 8 + 8
// mantissa bits), stored in the per-lane order of the m16n8k16 A fragment.  A bf16 token times a bf16 piece
// is exact in fp32, so the only rounding is the fp32 accumulation, as in the scalar kernel above (in a
// different, equally fixed order).  One CTA takes 16 router rows x all tokens x one column slice; its four
// warps split the slice's 16-column steps, each accumulating 16 x B partial logits in registers (B / 8
// accumulator tiles), which are then added across the warps through shared memory in a fixed order.
// The scalar kernel needs ~1.5 us of dependent latency per group of 8 tokens (44 us at 128 tokens, 13 at
// 32); this one issues three 16-byte loads and 2 x B / 8 4-byte loads per step and has no per-token-group
// barrier.  It is used for calls of more than 16 tokens.
constexpr int R3_ROWS = 16, R3_WARPS = 4;

size_t router3_elems(int n, int h) { return (size_t)((n + R3_ROWS - 1) / R3_ROWS) * (h / 16) * 3 * 32 * 8; }

int router3_kslices(int n, int h) {
  const int tiles = (n + R3_ROWS - 1) / R3_ROWS, ksteps = h / 16;
  int ks = 1;
  // more slices while every warp keeps at least two 16-column steps and the grid stays within ~256 CTAs; at
  // most 16, because every slice is one more array of partial logits for the top-k to add up
  while (ks < 16 && ksteps / (2 * ks) >= 2 * R3_WARPS && tiles * (2 * ks) <= 256) ks *= 2;
  return ks;
}

// out[((tile * (h / 16) + kt) * 3 + piece) * 32 + lane][8]: the A fragment (rows tile * 16 .., columns kt * 16 ..)
// of piece `piece` of the router; rows beyond n are zero.
__global__ void k_pack_router3(const float* __restrict__ Wr, __nv_bfloat16* __restrict__ out, int n, int h) {
  const int nk = h / 16;
  const long long total = (long long)((n + R3_ROWS - 1) / R3_ROWS) * nk * 32;
  for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (long long)gridDim.x * blockDim.x) {
    const int lane = (int)(idx & 31);
    const long long tk = idx >> 5;
    const int kt = (int)(tk % nk), tile = (int)(tk / nk);
    const int g = lane >> 2, tig = lane & 3;
    const int rr[4] = {tile * 16 + g, tile * 16 + g + 8, tile * 16 + g, tile * 16 + g + 8};
    const int kk[4] = {kt * 16 + tig * 2, kt * 16 + tig * 2, kt * 16 + tig * 2 + 8, kt * 16 + tig * 2 + 8};
    __align__(16) __nv_bfloat16 v[3][8];
#pragma unroll
    for (int e = 0; e < 4; ++e)
#pragma unroll
      for (int d = 0; d < 2; ++d) {
        const float w = rr[e] < n ? Wr[(size_t)rr[e] * h + kk[e] + d] : 0.f;
        const __nv_bfloat16 hi = __float2bfloat16_rn(w);
        const float r1 = w - __bfloat162float(hi);          // exact: at most 16 significant bits are left
        const __nv_bfloat16 mid = __float2bfloat16_rn(r1);
        const float r2 = r1 - __bfloat162float(mid);        // exact: at most 8 are left, so lo is exact too
        v[0][e * 2 + d] = hi; v[1][e * 2 + d] = mid; v[2][e * 2 + d] = __float2bfloat16_rn(r2);
      }
    const size_t base = (((size_t)tile * nk + kt) * 3) * 32 + lane;
#pragma unroll
    for (int pc = 0; pc < 3; ++pc)
      *reinterpret_cast<uint4*>(out + (base + (size_t)pc * 32) * 8) = *reinterpret_cast<const uint4*>(v[pc]);
  }
}

cudaError_t pack_router3(const float* router, __nv_bfloat16* out, int n, int h, cudaStream_t s) {
  const long long total = (long long)((n + R3_ROWS - 1) / R3_ROWS) * (h / 16) * 32;
  int blocks = (int)((total + 255) / 256);
  if (blocks > 2048) blocks = 2048;
  k_pack_router3<<<blocks, 256, 0, s>>>(router, out, n, h);
  return cudaGetLastError();
}

static __device__ __forceinline__ void mma_bf16_16816(float (&d)[4], const uint4& a, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a.x), "r"(a.y), "r"(a.z), "r"(a.w), "r"(b0), "r"(b1));
}

// NT = accumulator tiles of 8 tokens (a power of two, ceil(B / 8) rounded up).
template <int NT>
__global__ void __launch_bounds__(R3_WARPS * 32)
k_router_logits_mma(const __nv_bfloat16* __restrict__ W3, const __nv_bfloat16* __restrict__ X, float* __restrict__ part,
                    int n, int h, int B, int ksteps_per_slice, int32_t* __restrict__ step_flag TS_PARAM) {
#ifdef DEAMOE_TRACE
  if (threadIdx.x == 0 && ts) atomicMin(ts + 0, gtime());
#endif
  if (step_flag && blockIdx.x == 0 && blockIdx.y == 0) {  // see k_router_logits
    if (threadIdx.x == 0) {
      step_flag[0] = 0;
      step_flag[2] = 0;
      step_flag[3] = 0;
      __threadfence();
    }
    __syncthreads();
  }
  pdl_trigger();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, g = lane >> 2, tig = lane & 3;
  const int nk = h / 16;
  const int k_begin = blockIdx.y * ksteps_per_slice, k_end = min(nk, k_begin + ksteps_per_slice);
  float acc[NT][4];
#pragma unroll
  for (int t = 0; t < NT; ++t)
#pragma unroll
    for (int x = 0; x < 4; ++x) acc[t][x] = 0.f;
  const uint4* wp = reinterpret_cast<const uint4*>(W3) + ((size_t)blockIdx.x * nk * 3) * 32 + lane;
  // token row of this lane in accumulator tile t: 8 t + g (clamped; rows past B are never stored)
  const __nv_bfloat16* xrow[NT];
#pragma unroll
  for (int t = 0; t < NT; ++t) xrow[t] = X + (size_t)min(8 * t + g, B - 1) * h + 2 * tig;
  // G steps at a time: every load of the group is issued before its first MMA (the router comes from HBM,
  // the tokens from the L2; with few tokens a warp's steps would otherwise be a chain of memory latencies)
  constexpr int G = NT <= 2 ? 4 : (NT <= 4 ? 2 : 1);
  for (int kt0 = k_begin + warp; kt0 < k_end; kt0 += R3_WARPS * G) {
    uint4 a[G][3];
    uint32_t b0[G][NT], b1[G][NT];
#pragma unroll
    for (int u = 0; u < G; ++u) {
      const int kt = min(kt0 + u * R3_WARPS, k_end - 1);  // clamped: a step past the end is loaded but not used
#pragma unroll
      for (int pc = 0; pc < 3; ++pc) a[u][pc] = __ldg(wp + (size_t)kt * 96 + pc * 32);
#pragma unroll
      for (int t = 0; t < NT; ++t) {
        b0[u][t] = *reinterpret_cast<const uint32_t*>(xrow[t] + kt * 16);
        b1[u][t] = *reinterpret_cast<const uint32_t*>(xrow[t] + kt * 16 + 8);
      }
    }
#pragma unroll
    for (int u = 0; u < G; ++u) {
      if (kt0 + u * R3_WARPS < k_end) {
#pragma unroll
        for (int t = 0; t < NT; ++t) {
          mma_bf16_16816(acc[t], a[u][0], b0[u][t], b1[u][t]);
          mma_bf16_16816(acc[t], a[u][1], b0[u][t], b1[u][t]);
          mma_bf16_16816(acc[t], a[u][2], b0[u][t], b1[u][t]);
        }
      }
    }
  }
  // add the four warps' partial sums in warp order and store part[slice][token][row]
  __shared__ float red[R3_WARPS][R3_ROWS][NT * 8 + 1];
#pragma unroll
  for (int t = 0; t < NT; ++t) {
    red[warp][g][t * 8 + 2 * tig] = acc[t][0];
    red[warp][g][t * 8 + 2 * tig + 1] = acc[t][1];
    red[warp][g + 8][t * 8 + 2 * tig] = acc[t][2];
    red[warp][g + 8][t * 8 + 2 * tig + 1] = acc[t][3];
  }
  __syncthreads();
  const int row0 = blockIdx.x * R3_ROWS;
  for (int i = threadIdx.x; i < R3_ROWS * B; i += R3_WARPS * 32) {
    const int row = i % R3_ROWS, t = i / R3_ROWS;
    if (row0 + row < n) {
      float v = red[0][row][t];
#pragma unroll
      for (int w = 1; w < R3_WARPS; ++w) v += red[w][row][t];
      part[((size_t)blockIdx.y * B + t) * n + row0 + row] = v;
    }
  }
#ifdef DEAMOE_TRACE
  if (threadIdx.x == 0 && ts) atomicMax(ts + 1, gtime());
#endif
}

// ---------------------------------------------------------------- top-k, gate weights, bucketing
__global__ void __launch_bounds__(TOPK_WARPS * 32)
k_topk(LayerDev L, int B, int kslices, int32_t* __restrict__ user_idx, float* __restrict__ user_w) {
  extern __shared__ float s_log[];  // [TOPK_WARPS][n] logits, then [TOPK_WARPS][n] bytes "dead"
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int t = blockIdx.x * TOPK_WARPS + warp;
  if (t >= B) return;
  topk_one_token(L, t, B, kslices, s_log + (size_t)warp * L.n,
                 reinterpret_cast<unsigned char*>(s_log + (size_t)TOPK_WARPS * L.n) + (size_t)warp * L.n, lane, user_idx,
                 user_w);
}

__global__ void __launch_bounds__(BUCKET_THREADS) k_bucket(LayerDev L, int B) {
  extern __shared__ uint32_t s_bucket[];
  bucket_block(L, B, s_bucket, BUCKET_THREADS);
}

size_t bucket_smem_bytes(const LayerDev& L, int B) { return bucket_smem_words(L.n, L.m, B) * sizeof(uint32_t); }

cudaError_t route_configure(const LayerDev& L) {
  // the bucketing kernel may need more than the default 48 KB of dynamic shared memory
  const size_t need = bucket_smem_bytes(L, L.max_batch);
  if (need > 200 * 1024) return cudaErrorInvalidValue;
  cudaError_t e = cudaFuncSetAttribute(k_bucket, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(k_topk, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * 1024);
}

// Router logits straight from the caller's tokens (no fp32 copy): used by the streaming schedules.
// Returns the number of column slices written (the second grid dimension), or -1.
int launch_router_logits(const LayerDev& L, const void* tokens, int B, cudaStream_t s, int kslices, int32_t* step_flag) {
  // More than 16 tokens (three and more groups of eight for the scalar kernel, whose time grows by ~1.5 us per
  // group: 13 us at 32 tokens, 44 at 128): the tensor-core product on the three-piece router, 7.5 us at 32
  // tokens.  Up to 16 tokens the scalar kernel's 1024 small CTAs bring the router in faster (4.9 against 6.3 us
  // for one token on the DeepSeek-V3 shape).
  if (L.adt == DEAMOE_BF16 && L.router3 && B > 16) {
    const int nk = L.h / 16, ks = L.router3_slices;
    const int per = (nk + ks - 1) / ks;
    dim3 grid((L.n + R3_ROWS - 1) / R3_ROWS, (nk + per - 1) / per);
    const __nv_bfloat16* X = reinterpret_cast<const __nv_bfloat16*>(tokens);
    const int nt = (B + 7) / 8;
#define DEAMOE_R3(NT) k_router_logits_mma<NT><<<grid, R3_WARPS * 32, 0, s>>>(L.router3, X, L.logit_part, L.n, L.h, B, per, step_flag TS_ARG(L))
    if (nt <= 1) DEAMOE_R3(1);
    else if (nt <= 2) DEAMOE_R3(2);
    else if (nt <= 4) DEAMOE_R3(4);
    else if (nt <= 8) DEAMOE_R3(8);
    else DEAMOE_R3(16);
#undef DEAMOE_R3
    return cudaGetLastError() == cudaSuccess ? (int)grid.y : -1;
  }
  const int kslice = (((L.h + kslices - 1) / kslices) + 3) & ~3;
  dim3 grid((L.n + RG - 1) / RG, (L.h + kslice - 1) / kslice);
  if (L.adt == DEAMOE_BF16)
    k_router_logits<__nv_bfloat16><<<grid, ROUTER_THREADS, 0, s>>>(L.router, reinterpret_cast<const __nv_bfloat16*>(tokens),
                                                                  L.logit_part, L.n, L.h, B, kslice, step_flag TS_ARG(L));
  else
    k_router_logits<float><<<grid, ROUTER_THREADS, 0, s>>>(L.router, reinterpret_cast<const float*>(tokens), L.logit_part,
                                                          L.n, L.h, B, kslice, step_flag TS_ARG(L));
  return cudaGetLastError() == cudaSuccess ? (int)grid.y : -1;
}

int launch_route(const LayerDev& L, const void* tokens, int B, cudaStream_t s, int kslices, int32_t* user_idx,
                 float* user_w) {
  int launches = 0;
  if (L.adt == DEAMOE_BF16) {
    const size_t count = (size_t)B * L.h;
    const int blocks = (int)((count + 1023) / 1024);
    k_widen_tokens<<<blocks < 592 ? blocks : 592, 256, 0, s>>>((const __nv_bfloat16*)tokens, L.x32, count);
    ++launches;
  }
  const int kslice = (((L.h + kslices - 1) / kslices) + 3) & ~3;
  dim3 grid((L.n + RG - 1) / RG, (L.h + kslice - 1) / kslice);
  k_router_logits<float><<<grid, ROUTER_THREADS, 0, s>>>(L.router, L.x32, L.logit_part, L.n, L.h, B, kslice, nullptr TS_ARG(L));
  ++launches;
  const size_t topk_smem = (size_t)TOPK_WARPS * L.n * (sizeof(float) + 1);
  k_topk<<<(B + TOPK_WARPS - 1) / TOPK_WARPS, TOPK_WARPS * 32, topk_smem, s>>>(L, B, (int)grid.y, user_idx, user_w);
  ++launches;
  k_bucket<<<1, BUCKET_THREADS, bucket_smem_bytes(L, B), s>>>(L, B);
  ++launches;
  return cudaGetLastError() == cudaSuccess ? launches : -1;
}

}  // namespace deamoe

// ---------------------------------------------------------------- routing without any allocation
// deamoe_route_static: the router logits + top-k pair for callers that may not allocate.  The
// partial logits, which the layer object normally keeps in cudaMalloc'ed workspace, live in a
// fixed array inside the library image instead.
namespace {

constexpr size_t STATIC_SCRATCH_FLOATS = DEAMOE_STATIC_ROUTE_SCRATCH_BYTES / sizeof(float);
static __device__ __align__(256) float g_route_scratch[STATIC_SCRATCH_FLOATS];

constexpr int MAX_DEVICES = 64;
float* g_route_scratch_ptr[MAX_DEVICES];  // device address of the array, per device, after set-up
std::atomic<bool> g_route_ready[MAX_DEVICES];
std::mutex g_route_setup_mutex;           // first calls from several host threads set up one at a time

// Once per device, with that device current: resolve the array's device address (in host code the
// symbol is only a handle) and let the top-k kernel use its full dynamic shared memory.
deamoe_status_t static_route_setup(int dev) {
  if (g_route_ready[dev].load(std::memory_order_acquire)) return DEAMOE_OK;
  std::lock_guard<std::mutex> lock(g_route_setup_mutex);
  if (g_route_ready[dev].load(std::memory_order_relaxed)) return DEAMOE_OK;
  float* p = nullptr;
  if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_route_scratch) != cudaSuccess || !p) {
    cudaGetLastError();
    return DEAMOE_ERR_CUDA;
  }
  if (cudaFuncSetAttribute(deamoe::k_topk, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * 1024) != cudaSuccess) {
    cudaGetLastError();
    return DEAMOE_ERR_CUDA;
  }
  g_route_scratch_ptr[dev] = p;
  g_route_ready[dev].store(true, std::memory_order_release);
  return DEAMOE_OK;
}

}  // namespace

extern "C" deamoe_status_t deamoe_route_static(void* cuda_stream, const float* router, const float* tokens,
                                               int32_t n_dept, int32_t experts_per_dept, int32_t hidden,
                                               int32_t top_k, int32_t norm_topk, float route_scale, int32_t B,
                                               int32_t* topk_idx, float* topk_w) {
  using namespace deamoe;
  if (n_dept <= 0 || experts_per_dept <= 0 || hidden <= 0 || top_k <= 0 || B < 0) return DEAMOE_ERR_INVALID_ARG;
  const long long n = (long long)n_dept * experts_per_dept;
  if (top_k > n || !(route_scale == route_scale) || norm_topk < 0 || norm_topk > 2) return DEAMOE_ERR_INVALID_ARG;
  if (n > DEAMOE_MAX_EXPERTS || top_k > DEAMOE_MAX_TOPK || (hidden & 3)) return DEAMOE_ERR_UNSUPPORTED;
  if (B == 0) return DEAMOE_OK;
  if (!router || !tokens || !topk_idx || !topk_w) return DEAMOE_ERR_INVALID_ARG;
  // the logits kernel reads router rows and tokens as 16-byte vectors; the outputs are 4-byte words
  if (!aligned16(router) || !aligned16(tokens)) return DEAMOE_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(topk_idx) | reinterpret_cast<uintptr_t>(topk_w)) & 3u) return DEAMOE_ERR_INVALID_ARG;
  // column slices of the logits kernel: the same rule as the layer object, so that the partial sums
  // are added in the same grouping and the fp32 logits (hence near-ties and gate weights) are the same
  const int kslices = router_kslices((int)n, hidden);
  const int kslice = (((hidden + kslices - 1) / kslices) + 3) & ~3;
  const int ny = (hidden + kslice - 1) / kslice;
  if ((size_t)ny * (size_t)B * (size_t)n > STATIC_SCRATCH_FLOATS) return DEAMOE_ERR_BATCH;  // beyond the fixed scratch
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) {
    cudaGetLastError();
    return DEAMOE_ERR_CUDA;
  }
  const deamoe_status_t st = static_route_setup(dev);
  if (st != DEAMOE_OK) return st;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(cuda_stream);
  LayerDev L;
  memset(&L, 0, sizeof(L));
  L.h = hidden; L.m = n_dept; L.g = experts_per_dept; L.n = (int)n; L.k = top_k; L.k_dept = 0;
  L.norm_topk = norm_topk; L.route_scale = route_scale;
  L.logit_part = g_route_scratch_ptr[dev];   // every (slice, token, expert) entry used below is overwritten
  L.topk_idx = topk_idx; L.topk_w = topk_w;  // results go straight to the caller's buffers
  dim3 grid((L.n + RG - 1) / RG, ny);
  k_router_logits<float><<<grid, ROUTER_THREADS, 0, s>>>(router, tokens, L.logit_part, L.n, hidden, B, kslice, nullptr TS_ARG(L));
  const size_t topk_smem = (size_t)TOPK_WARPS * L.n * (sizeof(float) + 1);
  k_topk<<<(B + TOPK_WARPS - 1) / TOPK_WARPS, TOPK_WARPS * 32, topk_smem, s>>>(L, B, ny, nullptr, nullptr);
  return cudaGetLastError() == cudaSuccess ? DEAMOE_OK : DEAMOE_ERR_CUDA;
}
