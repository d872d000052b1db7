// PLAIN schedule: one simple kernel per stage of Section 3.2, reading the canonical layouts.
// It is the path for fp32 weights (the tiny configuration) and a cross-check for the bf16
// streaming kernels; it makes no attempt to reach the HBM roofline.
#include "deamoe_internal.cuh"

namespace deamoe {

// One unit of a stage = one active department, one active expert, or the shared expert.
struct UnitView {
  const void* Wa;         // first matrix
  const void* Wb;         // second matrix (paired gate/up stages) or nullptr
  int rows, cols;         // matrix shape [rows, cols] as stored (row-major)
  int T;                  // token rows of this unit
  const float* in_a;      // input of Wa: row s at in_a + in_row(s) * in_stride
  const float* in_b;      // input of Wb
  int in_stride;
  const int32_t* in_rows; // gathered input rows, or nullptr for in_row0 + s
  int in_row0;
  float* out;             // output row s at out + (out_row0 + s) * out_stride
  int out_stride, out_row0;
  int epi;                // 0: sigma(a)   1: SiLU(a) * b   2: a
};

static __device__ __forceinline__ size_t wsize(int wdt) { return wdt == DEAMOE_F32 ? 4 : 2; }

static __device__ __forceinline__ const void* woff(const void* base, int wdt, size_t elems) {
  return reinterpret_cast<const char*>(base) + elems * wsize(wdt);
}

// Resolve unit `u` (an index into the active list of the stage) of `stage`.
static __device__ bool resolve(const LayerDev& L, int stage, int u, int B, UnitView& v) {
  const size_t fh = (size_t)L.f * L.h, rf = (size_t)L.r * L.f;
  const int e_lo = L.dept_lo * L.g;  // the weight arrays start at department dept_lo / expert e_lo
  v.Wb = nullptr; v.in_b = nullptr; v.in_rows = nullptr; v.in_row0 = 0; v.out_row0 = 0;
  switch (stage) {
    case ST_S1: {  // rows [0,f): W_g^j, rows [f,2f): W_u^j  (handled as two matrices of f rows)
      if (u >= L.counts[CNT_ACTIVE_DEPT]) return false;
      const int j = L.active_dept[u];
      v.Wa = woff(L.dept_gate, L.wdt, (j - L.dept_lo) * fh); v.Wb = woff(L.dept_up, L.wdt, (j - L.dept_lo) * fh);
      v.rows = L.f; v.cols = L.h;
      v.T = L.dept_off[j + 1] - L.dept_off[j];
      v.in_a = L.x32; v.in_b = L.x32; v.in_stride = L.h; v.in_rows = L.dept_tok + L.dept_off[j];
      v.out = L.GU; v.out_stride = 2 * L.f; v.out_row0 = L.dept_off[j];
      v.epi = 0;
      return true;
    }
    case ST_S2: {
      if (u >= L.counts[CNT_ACTIVE_EXPERT]) return false;
      const int i = L.active_expert[u];
      v.Wa = woff(L.priv_gate, L.wdt, (i - e_lo) * rf); v.Wb = woff(L.priv_up, L.wdt, (i - e_lo) * rf);
      v.rows = L.r; v.cols = L.f;
      v.T = L.expert_off[i + 1] - L.expert_off[i];
      v.in_a = L.GU; v.in_b = L.GU + L.f; v.in_stride = 2 * L.f; v.in_rows = L.pair_gurow + L.expert_off[i];
      v.out = L.Y; v.out_stride = L.rp; v.out_row0 = L.expert_off[i];
      v.epi = 1;
      return true;
    }
    case ST_S3: {  // Z = sigma(A_d^T Y): A_d stored [r, f]
      if (u >= L.counts[CNT_ACTIVE_EXPERT]) return false;
      const int i = L.active_expert[u];
      v.Wa = woff(L.priv_down, L.wdt, (i - e_lo) * rf);
      v.rows = L.r; v.cols = L.f;
      v.T = L.expert_off[i + 1] - L.expert_off[i];
      v.in_a = L.Y; v.in_stride = L.rp; v.in_row0 = L.expert_off[i];
      v.out = L.Z; v.out_stride = L.f; v.out_row0 = L.expert_off[i];
      v.epi = 0;
      return true;
    }
    case ST_S4: {  // O = W_d^T Z over the pairs of the department (contiguous in pair order)
      if (u >= L.counts[CNT_ACTIVE_DEPT]) return false;
      const int j = L.active_dept[u];
      v.Wa = woff(L.dept_down, L.wdt, (j - L.dept_lo) * fh);
      v.rows = L.f; v.cols = L.h;
      const int p0 = L.expert_off[j * L.g], p1 = L.expert_off[(j + 1) * L.g];
      v.T = p1 - p0;
      v.in_a = L.Z; v.in_stride = L.f; v.in_row0 = p0;
      v.out = L.O; v.out_stride = L.h; v.out_row0 = p0;
      v.epi = 2;
      return true;
    }
    case ST_SH1: {
      if (u >= 1) return false;
      v.Wa = L.shared_gate; v.Wb = L.shared_up; v.rows = L.fs; v.cols = L.h; v.T = B;
      v.in_a = L.x32; v.in_b = L.x32; v.in_stride = L.h;
      v.out = L.Ysh; v.out_stride = L.fs;
      v.epi = 1;
      return true;
    }
    case ST_SH2: {
      if (u >= 1) return false;
      v.Wa = L.shared_down; v.rows = L.fs; v.cols = L.h; v.T = B;
      v.in_a = L.Ysh; v.in_stride = L.fs;
      v.out = L.Osh; v.out_stride = L.h;
      v.epi = 2;
      return true;
    }
    case ST_V1: {
      if (u >= L.counts[CNT_ACTIVE_EXPERT]) return false;
      const int i = L.active_expert[u];
      v.Wa = woff(L.dept_gate, L.wdt, i * fh); v.Wb = woff(L.dept_up, L.wdt, i * fh);
      v.rows = L.f; v.cols = L.h;
      v.T = L.expert_off[i + 1] - L.expert_off[i];
      v.in_a = L.x32; v.in_b = L.x32; v.in_stride = L.h; v.in_rows = L.expert_tok + L.expert_off[i];
      v.out = L.Y; v.out_stride = L.f; v.out_row0 = L.expert_off[i];
      v.epi = 1;
      return true;
    }
    case ST_V2: {
      if (u >= L.counts[CNT_ACTIVE_EXPERT]) return false;
      const int i = L.active_expert[u];
      v.Wa = woff(L.dept_down, L.wdt, i * fh);
      v.rows = L.f; v.cols = L.h;
      v.T = L.expert_off[i + 1] - L.expert_off[i];
      v.in_a = L.Y; v.in_stride = L.f; v.in_row0 = L.expert_off[i];
      v.out = L.O; v.out_stride = L.h; v.out_row0 = L.expert_off[i];
      v.epi = 2;
      return true;
    }
  }
  return false;
}

template <typename WT> static __device__ __forceinline__ float wval(const WT* p, size_t i);
template <> __device__ __forceinline__ float wval<float>(const float* p, size_t i) { return __ldg(p + i); }
template <> __device__ __forceinline__ float wval<__nv_bfloat16>(const __nv_bfloat16* p, size_t i) {
  return __bfloat162float(p[i]);
}

constexpr int PLAIN_THREADS = 256;
constexpr int PLAIN_TT = 4;  // tokens per pass

// out[s][row] = epi( Wa[row,:] . in_a[s,:],  Wb[row,:] . in_b[s,:] ); one warp per matrix row.
// For ST_S1 the two matrices are independent outputs: row < f -> gate, row >= f -> up.
template <typename WT>
__global__ void __launch_bounds__(PLAIN_THREADS) k_plain_rows(LayerDev L, int stage, int B) {
  UnitView v;
  if (!resolve(L, stage, blockIdx.y, B, v)) return;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const bool split = (stage == ST_S1);  // two independent matrices stacked
  const int total_rows = split ? 2 * v.rows : v.rows;
  const int row = blockIdx.x * (PLAIN_THREADS / 32) + warp;
  if (row >= total_rows) return;
  const bool second = split && row >= v.rows;
  const int mrow = second ? row - v.rows : row;
  const WT* wa = reinterpret_cast<const WT*>(second ? v.Wb : v.Wa) + (size_t)mrow * v.cols;
  const WT* wb = (!split && v.Wb) ? reinterpret_cast<const WT*>(v.Wb) + (size_t)mrow * v.cols : nullptr;
  for (int s0 = 0; s0 < v.T; s0 += PLAIN_TT) {
    float a[PLAIN_TT], b[PLAIN_TT];
    const float* xa[PLAIN_TT];
    const float* xb[PLAIN_TT];
#pragma unroll
    for (int q = 0; q < PLAIN_TT; ++q) {
      const int s = min(s0 + q, v.T - 1);
      const int ir = v.in_rows ? v.in_rows[s] : v.in_row0 + s;
      xa[q] = (second ? v.in_b : v.in_a) + (size_t)ir * v.in_stride;
      xb[q] = wb ? v.in_b + (size_t)ir * v.in_stride : nullptr;
      a[q] = 0.f; b[q] = 0.f;
    }
    for (int c = lane; c < v.cols; c += 32) {
      const float w1 = wval<WT>(wa, c);
      const float w2 = wb ? wval<WT>(wb, c) : 0.f;
#pragma unroll
      for (int q = 0; q < PLAIN_TT; ++q) {
        a[q] = fmaf(w1, xa[q][c], a[q]);
        if (wb) b[q] = fmaf(w2, xb[q][c], b[q]);
      }
    }
#pragma unroll
    for (int q = 0; q < PLAIN_TT; ++q) {
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        a[q] += __shfl_xor_sync(0xffffffffu, a[q], o);
        b[q] += __shfl_xor_sync(0xffffffffu, b[q], o);
      }
      if (lane == 0 && s0 + q < v.T) {
        float r;
        if (v.epi == 0) r = sigma_f(L.sigma, a[q]);
        else if (v.epi == 1) r = silu_f(a[q]) * b[q];
        else r = a[q];
        v.out[(size_t)(v.out_row0 + s0 + q) * v.out_stride + row] = r;
      }
    }
  }
}

// out[s][c] = epi( sum_q W[q, c] * in[s, q] ) for the transposed ("down") matrices; one thread
// per output column, adjacent threads read adjacent columns of a matrix row.
template <typename WT>
__global__ void __launch_bounds__(PLAIN_THREADS) k_plain_cols(LayerDev L, int stage, int B) {
  UnitView v;
  if (!resolve(L, stage, blockIdx.y, B, v)) return;
  const int c = blockIdx.x * PLAIN_THREADS + threadIdx.x;
  if (c >= v.cols) return;
  const WT* w = reinterpret_cast<const WT*>(v.Wa);
  for (int s0 = 0; s0 < v.T; s0 += PLAIN_TT) {
    float a[PLAIN_TT];
    const float* x[PLAIN_TT];
#pragma unroll
    for (int q = 0; q < PLAIN_TT; ++q) {
      const int s = min(s0 + q, v.T - 1);
      x[q] = v.in_a + (size_t)(v.in_row0 + s) * v.in_stride;
      a[q] = 0.f;
    }
    for (int q2 = 0; q2 < v.rows; ++q2) {
      const float wv = wval<WT>(w, (size_t)q2 * v.cols + c);
#pragma unroll
      for (int q = 0; q < PLAIN_TT; ++q) a[q] = fmaf(wv, x[q][q2], a[q]);
    }
#pragma unroll
    for (int q = 0; q < PLAIN_TT; ++q)
      if (s0 + q < v.T) {
        const float r = (v.epi == 0) ? sigma_f(L.sigma, a[q]) : a[q];
        v.out[(size_t)(v.out_row0 + s0 + q) * v.out_stride + c] = r;
      }
  }
}

// priv == 0: A = identity, so Y = SiLU(G) * U and Z = sigma(Y) element by element.
__global__ void k_plain_identity_private(LayerDev L) {
  const int pairs = L.counts[CNT_PAIRS];
  const size_t total = (size_t)pairs * L.f;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    const int p = (int)(i / L.f), c = (int)(i % L.f);
    const float* gu = L.GU + (size_t)L.pair_gurow[p] * 2 * L.f;
    const float y = silu_f(gu[c]) * gu[L.f + c];
    L.Y[(size_t)p * L.rp + c] = y;
    L.Z[(size_t)p * L.f + c] = sigma_f(L.sigma, y);
  }
}

// sigma = RMSNorm (plain schedule): normalise, in place, the `parts` vectors of `width` floats that
// make up every row of `buf`; the number of rows is counter `count_idx` of the routing state.
// One block per (row, part).
__global__ void k_plain_rmsnorm(LayerDev L, float* __restrict__ buf, int count_idx, int parts, int width) {
  __shared__ float s_part[32];
  const int rows = L.counts[count_idx];
  for (int v = (int)blockIdx.x; v < rows * parts; v += (int)gridDim.x) {
    float* p = buf + (size_t)v * width;
    float ss = 0.f;
    for (int i = (int)threadIdx.x; i < width; i += (int)blockDim.x) ss = fmaf(p[i], p[i], ss);
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = ss;
    __syncthreads();
    if (threadIdx.x < 32) {
      float t = (threadIdx.x < (blockDim.x >> 5)) ? s_part[threadIdx.x] : 0.f;
      for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
      if (threadIdx.x == 0) s_part[0] = t;
    }
    __syncthreads();
    const float sc = rms_scale(s_part[0], width);
    for (int i = (int)threadIdx.x; i < width; i += (int)blockDim.x) p[i] *= sc;
    __syncthreads();
  }
}

// Eq. (3): out[t] = sum_q p[t,q] * O[slot(t,q)] (+ shared expert) (+ x[t]), written in act dtype.
// partial != 0 (department-sharded layer): the sum over this layer object's pairs only (+ its shared
// expert if it has one), written as fp32 without the residual; the partial sums of all shards are
// added by the caller (an all-reduce) and finished by k_finish_partial.
__global__ void k_combine(LayerDev L, int B, const float* __restrict__ x32, void* __restrict__ out, int partial) {
  TS_MIN(L, 8);
  pdl_wait();  // stage outputs of the preceding kernel
  TS_MIN(L, 9);
  if (L.sh_done && blockIdx.x == 0 && threadIdx.x == 0) *L.sh_done = 0;  // nothing of this step reads it any more
  // four consecutive columns per thread (h is a multiple of 4 in every accepted configuration)
  const int h4 = L.h >> 2;
  const size_t total = (size_t)B * h4;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    const int t = (int)(i / h4), c4 = (int)(i % h4);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int q = 0; q < L.k; ++q) {
      const int slot = L.pair_slot[t * L.k + q];
      if (slot == -1) continue;  // the pair's department lives in another layer object (sharded layer)
      if ((unsigned)slot >= (unsigned)(L.max_batch * L.k)) {  // consistency check: skip the access, report
        L.counts[CNT_STATUS] = DEAMOE_ERR_INTERNAL;
        continue;
      }
      const float p = L.topk_w[t * L.k + q];
      const float4 o = __ldcg(reinterpret_cast<const float4*>(L.O + (size_t)slot * L.h) + c4);
      acc.x = fmaf(p, o.x, acc.x); acc.y = fmaf(p, o.y, acc.y); acc.z = fmaf(p, o.z, acc.z); acc.w = fmaf(p, o.w, acc.w);
    }
    if (L.n_shared) {
      const float4 o = __ldcg(reinterpret_cast<const float4*>(L.Osh) + i);
      acc.x += o.x; acc.y += o.y; acc.z += o.z; acc.w += o.w;
    }
    if (partial) {
      reinterpret_cast<float4*>(out)[i] = acc;
      continue;
    }
    if (L.residual) {
      if (L.adt == DEAMOE_F32) {
        const float4 x = reinterpret_cast<const float4*>(L.tokens_raw)[i];
        acc.x += x.x; acc.y += x.y; acc.z += x.z; acc.w += x.w;
      } else {
        const uint2 raw = reinterpret_cast<const uint2*>(L.tokens_raw)[i];
        const __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162*>(&raw.x);
        const __nv_bfloat162 b = *reinterpret_cast<const __nv_bfloat162*>(&raw.y);
        acc.x += __bfloat162float(a.x); acc.y += __bfloat162float(a.y);
        acc.z += __bfloat162float(b.x); acc.w += __bfloat162float(b.y);
      }
    }
    if (L.adt == DEAMOE_F32) {
      reinterpret_cast<float4*>(out)[i] = acc;
    } else {
      const __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y), hi = __floats2bfloat162_rn(acc.z, acc.w);
      uint2 pk;
      pk.x = *reinterpret_cast<const uint32_t*>(&lo);
      pk.y = *reinterpret_cast<const uint32_t*>(&hi);
      reinterpret_cast<uint2*>(out)[i] = pk;
    }
  }
  TS_MAX(L, 10);
}

// Measurement aid: read `n16` 16-byte words once, with plain vectorised loads that bypass L1, eight
// independent loads in flight per thread; the xor of everything read goes to sink[block] so that the
// loads cannot be dropped.  What a read-only stream of this GPU's HBM can reach without any of the
// layer's machinery: the yardstick the weight-streaming kernel is set against.
__global__ void __launch_bounds__(256) k_probe_read(const uint4* __restrict__ src, size_t n16, uint32_t* __restrict__ sink) {
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  uint32_t acc = 0;
  auto ld = [](const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
  };
  for (; i + 7 * stride < n16; i += 8 * stride) {
    uint4 v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) v[u] = ld(src + i + u * stride);
#pragma unroll
    for (int u = 0; u < 8; ++u) acc ^= v[u].x ^ v[u].y ^ v[u].z ^ v[u].w;
  }
  for (; i < n16; i += stride) {
    const uint4 v = ld(src + i);
    acc ^= v.x ^ v.y ^ v.z ^ v.w;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc ^= __shfl_xor_sync(0xffffffffu, acc, o);
  __shared__ uint32_t s_acc[8];
  if ((threadIdx.x & 31) == 0) s_acc[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    uint32_t a = 0;
    for (int w = 0; w < 8; ++w) a ^= s_acc[w];
    sink[blockIdx.x] = a;
  }
}

int launch_probe_read(const void* src, size_t bytes, uint32_t* sink, int blocks, cudaStream_t s) {
  k_probe_read<<<blocks, 256, 0, s>>>(reinterpret_cast<const uint4*>(src), bytes / 16, sink);
  return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

template <typename WT>
static int plain_forward_t(const LayerDev& L, int B, cudaStream_t s) {
  int launches = 0;
  const int wpb = PLAIN_THREADS / 32;
  auto rows_grid = [&](int rows, int units) { return dim3((rows + wpb - 1) / wpb, units); };
  auto cols_grid = [&](int cols, int units) { return dim3((cols + PLAIN_THREADS - 1) / PLAIN_THREADS, units); };
  const int max_dept = L.m < B * L.k ? L.m : B * L.k;
  const int max_exp = L.n < B * L.k ? L.n : B * L.k;
  if (L.n_shared) {
    k_plain_rows<WT><<<rows_grid(L.fs, 1), PLAIN_THREADS, 0, s>>>(L, ST_SH1, B);
    k_plain_cols<WT><<<cols_grid(L.h, 1), PLAIN_THREADS, 0, s>>>(L, ST_SH2, B);
    launches += 2;
  }
  if (L.vanilla) {
    k_plain_rows<WT><<<rows_grid(L.f, max_exp), PLAIN_THREADS, 0, s>>>(L, ST_V1, B);
    k_plain_cols<WT><<<cols_grid(L.h, max_exp), PLAIN_THREADS, 0, s>>>(L, ST_V2, B);
    launches += 2;
  } else {
    k_plain_rows<WT><<<rows_grid(2 * L.f, max_dept), PLAIN_THREADS, 0, s>>>(L, ST_S1, B);
    ++launches;
    const bool rms = L.sigma == DEAMOE_SIGMA_RMSNORM;
    if (rms) {  // G and U of every (token, department) row
      k_plain_rmsnorm<<<296, 256, 0, s>>>(L, L.GU, CNT_TOKEN_DEPT, 2, L.f);
      ++launches;
    }
    if (L.r > 0) {
      k_plain_rows<WT><<<rows_grid(L.r, max_exp), PLAIN_THREADS, 0, s>>>(L, ST_S2, B);
      k_plain_cols<WT><<<cols_grid(L.f, max_exp), PLAIN_THREADS, 0, s>>>(L, ST_S3, B);
      launches += 2;
      if (rms) {  // Z of every pair
        k_plain_rmsnorm<<<296, 256, 0, s>>>(L, L.Z, CNT_PAIRS, 1, L.f);
        ++launches;
      }
    } else {
      k_plain_identity_private<<<148, 256, 0, s>>>(L);
      ++launches;
    }
    k_plain_cols<WT><<<cols_grid(L.h, max_dept), PLAIN_THREADS, 0, s>>>(L, ST_S4, B);
    ++launches;
  }
  return cudaGetLastError() == cudaSuccess ? launches : -1;
}

int launch_plain_forward(const LayerDev& L, int B, cudaStream_t s) {
  return L.wdt == DEAMOE_F32 ? plain_forward_t<float>(L, B, s) : plain_forward_t<__nv_bfloat16>(L, B, s);
}

int launch_combine(const LayerDev& L, const void* tokens, int B, void* out, cudaStream_t s, int partial) {
  (void)tokens;
  const size_t total = (size_t)B * (L.h / 4);  // four columns per thread
  int blocks = (int)((total + 255) / 256);
  if (blocks > 148 * 8) blocks = 148 * 8;
  const cudaError_t e = launch_pdl(k_combine, dim3(blocks), dim3(256), 0, s, L, B, (const float*)L.x32, out, partial);
  return (e == cudaSuccess && cudaGetLastError() == cudaSuccess) ? 1 : -1;
}

// out[t] = sum[t] (+ x[t] if residual), written in the activation dtype: the last step of Eq. (3) for a
// department-sharded layer, after the shards' partial sums have been added.
__global__ void k_finish_partial(LayerDev L, int B, const float* __restrict__ sum, void* __restrict__ out) {
  const size_t total = (size_t)B * (L.h >> 2);
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    float4 acc = reinterpret_cast<const float4*>(sum)[i];
    if (L.residual) {
      if (L.adt == DEAMOE_F32) {
        const float4 x = reinterpret_cast<const float4*>(L.tokens_raw)[i];
        acc.x += x.x; acc.y += x.y; acc.z += x.z; acc.w += x.w;
      } else {
        const uint2 raw = reinterpret_cast<const uint2*>(L.tokens_raw)[i];
        const __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162*>(&raw.x);
        const __nv_bfloat162 b = *reinterpret_cast<const __nv_bfloat162*>(&raw.y);
        acc.x += __bfloat162float(a.x); acc.y += __bfloat162float(a.y);
        acc.z += __bfloat162float(b.x); acc.w += __bfloat162float(b.y);
      }
    }
    if (L.adt == DEAMOE_F32) {
      reinterpret_cast<float4*>(out)[i] = acc;
    } else {
      const __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y), hi = __floats2bfloat162_rn(acc.z, acc.w);
      uint2 pk;
      pk.x = *reinterpret_cast<const uint32_t*>(&lo);
      pk.y = *reinterpret_cast<const uint32_t*>(&hi);
      reinterpret_cast<uint2*>(out)[i] = pk;
    }
  }
}

int launch_finish_partial(const LayerDev& L, const float* sum, const void* tokens, int B, void* out, cudaStream_t s) {
  (void)tokens;
  const size_t total = (size_t)B * (L.h / 4);
  int blocks = (int)((total + 255) / 256);
  if (blocks > 148 * 8) blocks = 148 * 8;
  k_finish_partial<<<blocks, 256, 0, s>>>(L, B, sum, out);
  return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

}  // namespace deamoe
