// Router (Eq. (2)), gate weights (Eq. (3)) and the department / expert token lists of
// Section 3.2, all on the device with no host round trip.
#include <cstring>

#include "deamoe_internal.cuh"

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

__global__ void __launch_bounds__(ROUTER_THREADS)
k_router_logits(const float* __restrict__ Wr, const float* __restrict__ x32, float* __restrict__ part,
                int n, int h, int B, int kslice) {
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
        const float4 x = *reinterpret_cast<const float4*>(x32 + (size_t)t * h + c);
#pragma unroll
        for (int a = 0; a < RG; ++a) {
          acc[a][b] = fmaf(w[a].x, x.x, acc[a][b]);
          acc[a][b] = fmaf(w[a].y, x.y, acc[a][b]);
          acc[a][b] = fmaf(w[a].z, x.z, acc[a][b]);
          acc[a][b] = fmaf(w[a].w, x.w, acc[a][b]);
        }
      }
    }
#pragma unroll
    for (int a = 0; a < RG; ++a)
#pragma unroll
      for (int b = 0; b < TG; ++b) {
        float v = acc[a][b];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if (lane == 0) red[warp][a][b] = v;
      }
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
}

// ---------------------------------------------------------------- top-k + gate weights
// One warp per token.  Order: logit descending, ties to the lower expert index.
constexpr int TOPK_WARPS = 4;

static __device__ __forceinline__ bool better(float v, int i, float bv, int bi) {
  return (v > bv) || (v == bv && i < bi);
}

__global__ void __launch_bounds__(TOPK_WARPS * 32)
k_topk(LayerDev L, int B, int kslices, int32_t* __restrict__ user_idx, float* __restrict__ user_w) {
  extern __shared__ float s_log[];  // [TOPK_WARPS][n] logits, then [TOPK_WARPS][n] bytes "dead"
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int t = blockIdx.x * TOPK_WARPS + warp;
  const int n = L.n, g = L.g, m = L.m, k = L.k;
  float* lg = s_log + (size_t)warp * n;
  unsigned char* dead = reinterpret_cast<unsigned char*>(s_log + (size_t)TOPK_WARPS * n) + (size_t)warp * n;
  if (t >= B) return;
  float mx_all = -INFINITY;
  for (int i = lane; i < n; i += 32) {
    float v = 0.f;
    for (int s = 0; s < kslices; ++s) v += L.logit_part[((size_t)s * B + t) * n + i];
    lg[i] = v;
    dead[i] = 0;
    mx_all = fmaxf(mx_all, v);
  }
  __syncwarp();
  if (L.k_dept > 0 && L.k_dept < m) {
    // group limit: only the k_dept departments with the largest best logit stay eligible.
    // A department is eliminated if at least k_dept departments rank ahead of it.
    for (int j = lane; j < m; j += 32) {
      float best = lg[(size_t)j * g];
      for (int e = 1; e < g; ++e) best = fmaxf(best, lg[(size_t)j * g + e]);
      int ahead = 0;
      for (int j2 = 0; j2 < m; ++j2) {
        float b2 = lg[(size_t)j2 * g];
        for (int e = 1; e < g; ++e) b2 = fmaxf(b2, lg[(size_t)j2 * g + e]);
        ahead += better(b2, j2, best, j) ? 1 : 0;
      }
      if (ahead >= L.k_dept)
        for (int e = 0; e < g; ++e) dead[(size_t)j * g + e] = 1;
    }
    __syncwarp();
  }
  float den_all = 0.f;
  if (!L.norm_topk) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx_all = fmaxf(mx_all, __shfl_xor_sync(0xffffffffu, mx_all, o));
    for (int i = lane; i < n; i += 32) den_all += expf(lg[i] - mx_all);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) den_all += __shfl_xor_sync(0xffffffffu, den_all, o);
  }
  float my_v = 0.f;  // lane q keeps the q-th selected logit (k <= 32)
  int my_i = 0;
  for (int q = 0; q < k; ++q) {
    float bv = -INFINITY;
    int bi = 0x7fffffff;
    for (int i = lane; i < n; i += 32)
      if (!dead[i] && better(lg[i], i, bv, bi)) { bv = lg[i]; bi = i; }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
      const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
      if (better(ov, oi, bv, bi)) { bv = ov; bi = oi; }
    }
    if (lane == q) { my_v = bv; my_i = bi; }
    if (lane == 0 && bi < n) dead[bi] = 1;
    __syncwarp();
  }
  // gate weights
  const float top = __shfl_sync(0xffffffffu, my_v, 0);
  float e, den;
  if (L.norm_topk) {
    e = (lane < k) ? expf(my_v - top) : 0.f;
    den = e;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) den += __shfl_xor_sync(0xffffffffu, den, o);
  } else {
    e = (lane < k) ? expf(my_v - mx_all) : 0.f;
    den = den_all;
  }
  if (lane < k) {
    const float p = L.route_scale * e / den;
    L.topk_idx[(size_t)t * k + lane] = my_i;
    L.topk_w[(size_t)t * k + lane] = p;
    if (user_idx) user_idx[(size_t)t * k + lane] = my_i;
    if (user_w) user_w[(size_t)t * k + lane] = p;
  }
}

// ---------------------------------------------------------------- department bucketing
// One CTA.  Token-membership bitmasks per department and per expert are built with shared
// atomics, then counts, offsets (warp ballot/popc scans), ascending token lists, the pair
// order (expert-major) and the (token, department) row of every pair.
constexpr int BUCKET_THREADS = 512;

static __device__ __forceinline__ int warp_exclusive_offsets(const int* cnt, int count, int32_t* off,
                                                             int32_t* active, int lane, int* n_active) {
  // exclusive prefix sum of cnt[0..count) into off[0..count], compaction of the non-empty
  // indices into active[]; executed by one warp.
  int run = 0, nact = 0;
  for (int base = 0; base < count; base += 32) {
    const int i = base + lane;
    const int c = (i < count) ? cnt[i] : 0;
    int incl = c;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += v;
    }
    if (i < count) off[i] = run + incl - c;
    const unsigned live = __ballot_sync(0xffffffffu, c > 0);
    if (c > 0) active[nact + __popc(live & ((1u << lane) - 1u))] = i;
    nact += __popc(live);
    run += __shfl_sync(0xffffffffu, incl, 31);
  }
  if (lane == 0) { off[count] = run; *n_active = nact; }
  return run;
}

__global__ void __launch_bounds__(BUCKET_THREADS) k_bucket(LayerDev L, int B) {
  extern __shared__ uint32_t s_u32[];
  const int n = L.n, m = L.m, g = L.g, k = L.k;
  const int W = (B + 31) / 32;
  uint32_t* emask = s_u32;                    // [n][W]
  uint32_t* dmask = emask + (size_t)n * W;    // [m][W]
  int* ecnt = reinterpret_cast<int*>(dmask + (size_t)m * W);  // [n]
  int* dcnt = ecnt + n;                                        // [m]
  int* s_eoff = dcnt + m;                                      // [n+1]
  int* s_doff = s_eoff + n + 1;                                // [m+1]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int i = tid; i < (n + m) * W; i += BUCKET_THREADS) s_u32[i] = 0u;
  __syncthreads();
  for (int p = tid; p < B * k; p += BUCKET_THREADS) {
    const int t = p / k;
    const int i = L.topk_idx[p];
    atomicOr(&emask[(size_t)i * W + (t >> 5)], 1u << (t & 31));
    atomicOr(&dmask[(size_t)(i / g) * W + (t >> 5)], 1u << (t & 31));
  }
  __syncthreads();
  for (int i = tid; i < n; i += BUCKET_THREADS) {
    int c = 0;
    for (int w = 0; w < W; ++w) c += __popc(emask[(size_t)i * W + w]);
    ecnt[i] = c;
  }
  for (int j = tid; j < m; j += BUCKET_THREADS) {
    int c = 0;
    for (int w = 0; w < W; ++w) c += __popc(dmask[(size_t)j * W + w]);
    dcnt[j] = c;
  }
  for (int w = tid; w < (m + 63) / 64; w += BUCKET_THREADS) {
    uint64_t bits = 0;
    for (int b = 0; b < 64 && w * 64 + b < m; ++b) {
      bool any = false;
      for (int q = 0; q < W; ++q) any |= dmask[(size_t)(w * 64 + b) * W + q] != 0u;
      if (any) bits |= (uint64_t)1 << b;
    }
    L.dept_mask[w] = bits;
  }
  __syncthreads();
  if (warp == 0) {
    warp_exclusive_offsets(dcnt, m, s_doff, L.active_dept, lane, &L.counts[CNT_ACTIVE_DEPT]);
  } else if (warp == 1) {
    warp_exclusive_offsets(ecnt, n, s_eoff, L.active_expert, lane, &L.counts[CNT_ACTIVE_EXPERT]);
  }
  __syncthreads();
  for (int i = tid; i <= n; i += BUCKET_THREADS) L.expert_off[i] = s_eoff[i];
  for (int j = tid; j <= m; j += BUCKET_THREADS) L.dept_off[j] = s_doff[j];
  if (tid == 0) {
    L.counts[CNT_STATUS] = 0;
    L.counts[CNT_TOKEN_DEPT] = s_doff[m];
    L.counts[CNT_PAIRS] = s_eoff[n];
  }
  // ascending token lists
  for (int i = tid; i < n; i += BUCKET_THREADS) {
    int pos = s_eoff[i];
    for (int w = 0; w < W; ++w) {
      uint32_t bits = emask[(size_t)i * W + w];
      while (bits) {
        const int b = __ffs(bits) - 1;
        bits &= bits - 1;
        L.expert_tok[pos++] = w * 32 + b;
      }
    }
  }
  for (int j = tid; j < m; j += BUCKET_THREADS) {
    int pos = s_doff[j];
    for (int w = 0; w < W; ++w) {
      uint32_t bits = dmask[(size_t)j * W + w];
      while (bits) {
        const int b = __ffs(bits) - 1;
        bits &= bits - 1;
        L.dept_tok[pos++] = w * 32 + b;
      }
    }
  }
  // pair order and the GU row of every pair
  for (int p = tid; p < B * k; p += BUCKET_THREADS) {
    const int t = p / k;
    const int i = L.topk_idx[p];
    const int j = i / g;
    int re = 0, rd = 0;
    for (int w = 0; w < (t >> 5); ++w) {
      re += __popc(emask[(size_t)i * W + w]);
      rd += __popc(dmask[(size_t)j * W + w]);
    }
    const uint32_t below = (1u << (t & 31)) - 1u;
    re += __popc(emask[(size_t)i * W + (t >> 5)] & below);
    rd += __popc(dmask[(size_t)j * W + (t >> 5)] & below);
    const int slot = s_eoff[i] + re;
    L.pair_slot[p] = slot;
    L.pair_gurow[slot] = s_doff[j] + rd;
  }
}

size_t bucket_smem_bytes(const LayerDev& L, int B) {
  const int W = (B + 31) / 32;
  return ((size_t)(L.n + L.m) * W + (size_t)L.n + L.m + (L.n + 1) + (L.m + 1)) * sizeof(uint32_t);
}

cudaError_t route_configure(const LayerDev& L) {
  // the bucketing kernel may need more than the default 48 KB of dynamic shared memory
  const size_t need = bucket_smem_bytes(L, L.max_batch);
  if (need > 200 * 1024) return cudaErrorInvalidValue;
  cudaError_t e = cudaFuncSetAttribute(k_bucket, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(k_topk, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * 1024);
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
  k_router_logits<<<grid, ROUTER_THREADS, 0, s>>>(L.router, L.x32, L.logit_part, L.n, L.h, B, kslice);
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
bool g_route_ready[MAX_DEVICES];

// Once per device, with that device current: resolve the array's device address (in host code the
// symbol is only a handle) and let the top-k kernel use its full dynamic shared memory.
deamoe_status_t static_route_setup(int dev) {
  if (g_route_ready[dev]) return DEAMOE_OK;
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
  g_route_ready[dev] = true;
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
  if (top_k > n || !(route_scale == route_scale)) return DEAMOE_ERR_INVALID_ARG;
  if (n > DEAMOE_MAX_EXPERTS || top_k > DEAMOE_MAX_TOPK || (hidden & 3)) return DEAMOE_ERR_UNSUPPORTED;
  if (B == 0) return DEAMOE_OK;
  if (!router || !tokens || !topk_idx || !topk_w) return DEAMOE_ERR_INVALID_ARG;
  // column slices of the logits kernel, chosen as the layer object does
  int kslices = 1;
  while (kslices < 16 && ((n + 3) / 4) * kslices < 296 && hidden / (kslices * 2) >= 512) kslices *= 2;
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
  k_router_logits<<<grid, ROUTER_THREADS, 0, s>>>(router, tokens, L.logit_part, L.n, hidden, B, kslice);
  const size_t topk_smem = (size_t)TOPK_WARPS * L.n * (sizeof(float) + 1);
  k_topk<<<(B + TOPK_WARPS - 1) / TOPK_WARPS, TOPK_WARPS * 32, topk_smem, s>>>(L, B, ny, nullptr, nullptr);
  return cudaGetLastError() == cudaSuccess ? DEAMOE_OK : DEAMOE_ERR_CUDA;
}
