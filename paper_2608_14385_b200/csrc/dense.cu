// Dense schedule: the department matrices (W_g, W_u, W_d of Section 3.2) and the shared expert
// (Eq. (1)) on the fifth-generation tensor cores.
//
// From a few dozen tokens on, a department's token bucket X^j is a dense tile (16 and more rows),
// and the per-warp mma.sync path of the streaming kernel becomes issue-bound.  Here one
// tcgen05.mma covers 128 weight rows x all tokens of the bucket (N up to 64) x 16 columns, with the
// accumulator in tensor memory, so the kernel is again bound by the weight stream:
//
//   D[128 weight rows, N tokens] += W_tile[128, K] . X^j[N, K]^T
//
// Roles of a CTA (one CTA per SM, persistent over a list of (unit, 128-row tile) jobs):
//   warps 0-3   epilogue: tcgen05.ld of the finished accumulator, sigma / SwiGLU, stores
//   warp  4     one thread issues the bulk copies of the weight chunks (16 KB each) into the ring
//   warp  5     one thread issues the MMAs and the commits that free ring stages / publish accumulators
//   warps 6-13  loaders: copy the tokens' activation rows of a chunk from their row-major planes
//               into the core-matrix layout the MMA reads (warp w serves ring stage w)
// Weights are stored at create time in that same layout, tile by tile and chunk by chunk, so a
// chunk is one contiguous bulk copy.  Layout of an operand chunk (R rows x BK columns, bf16, "K-major,
// no swizzle"): 8 x 8 core matrices of 128 contiguous bytes; byte offset of element (r, k) =
// (r / 8) * (BK * 16) + (k / 8) * 128 + (r % 8) * 16 + (k % 8) * 2.
#include "dense.cuh"

#include <cstring>
#include <new>

namespace deamoe {

namespace {

constexpr int DN_NST = 8;                   // ring stages = loader warps
constexpr int DN_NMAX = 64;                 // token columns of one accumulator
constexpr int DN_A_BYTES = 16 * 1024;       // weights per stage: 128 rows x 64 k, or 2 x (128 x 32)
constexpr int DN_B_BYTES = DN_NMAX * 128;   // activations per stage: 64 tokens x 64 k
constexpr int DN_STAGE_BYTES = DN_A_BYTES + DN_B_BYTES;
constexpr int DN_WARP_TMA = 4, DN_WARP_MMA = 5, DN_WARP_LOAD0 = 6;
constexpr int DN_THREADS = (DN_WARP_LOAD0 + DN_NST) * 32;
constexpr int DN_TMEM_COLS = 256;           // 2 accumulator buffers x 2 matrices x 64 columns
constexpr size_t DN_SMEM = (size_t)DN_NST * DN_STAGE_BYTES + 1024 /* alignment */ + 512 /* barriers, control */;
constexpr unsigned DN_SPIN_LIMIT = 1u << 22;  // bounded waits; then an error status, never a hang
static_assert(DN_SMEM <= 227 * 1024, "shared memory budget");
// More than half of an SM's shared memory: two of these CTAs never share an SM, so the tensor
// memory allocation below never waits for another CTA.
static_assert(DN_SMEM > 114 * 1024, "one CTA per SM is relied upon by the tensor-memory allocation");

enum DenseEpi : int { DE_SIGMA = 0, DE_SWIGLU = 1, DE_NONE = 2 };

struct DensePhase {
  int stage;      // ST_S1, ST_S4, ST_SH1 or ST_SH2
  int K, tiles;   // contraction length; 128-row tiles of a unit
  int dual;       // a tile is 128 rows of w and the same rows of w1; epilogue SiLU(a) * b; BK = 32
  int epi;
  int in_stride, out_stride;
  const __nv_bfloat16* w;
  const __nv_bfloat16* w1;
  unsigned long long unit_elems;
  const __nv_bfloat16* in;
  __nv_bfloat16* outh;
  float* outf;
};
struct DenseArgs {
  DensePhase ph[2];
  int nph;
};

// ---------------------------------------------------------------- PTX helpers
__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void bar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count));
}
__device__ __forceinline__ void bar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}
__device__ __forceinline__ void bar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool bar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t done;
  asm volatile(
      "{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
      : "=r"(done) : "r"(smem_addr(bar)), "r"(parity) : "memory");
  return done != 0;
}
// Bounded wait.  On expiry (or when another role has given up) the abort flag is raised and false
// is returned; the caller leaves its loop and the CTA runs to its common end.
__device__ __forceinline__ bool bar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  for (unsigned it = 0; it < DN_SPIN_LIMIT; ++it) {
    if (bar_try_wait(bar, parity)) return true;
    if ((it & 63u) == 63u && *abort_flag) return false;
  }
  *abort_flag = 1;
  return false;
}
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
      ::"r"(smem_addr(dst)), "l"(src), "r"(bytes), "r"(smem_addr(bar)), "l"(pol) : "memory");
}
__device__ __forceinline__ uint64_t policy_stream() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// Shared-memory matrix descriptor, K-major without swizzle: `lbo` = bytes between core matrices that
// are neighbours along K, `sbo` = bytes between 8-row groups.
__device__ __forceinline__ uint64_t umma_smem_desc(uint32_t saddr, uint32_t lbo, uint32_t sbo) {
  uint64_t d = (uint64_t)((saddr & 0x3ffffu) >> 4);
  d |= (uint64_t)((lbo >> 4) & 0x3fffu) << 16;
  d |= (uint64_t)((sbo >> 4) & 0x3fffu) << 32;
  d |= 1ull << 46;  // descriptor version of this architecture
  return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M x N.
__device__ __forceinline__ uint32_t umma_instr_desc(int M, int N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
__device__ __forceinline__ void umma(uint32_t d_tmem, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
      ::"r"(d_tmem), "l"(da), "l"(db), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_addr(bar)) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// ---------------------------------------------------------------- job decoding (all roles alike)
struct Job {
  int phase, tile;
  int T;          // token rows of the unit
  int row0;       // first output row of the unit (and first input row when the rows are contiguous)
  const int32_t* in_list;  // gathered input rows, or null
  size_t woff;    // element offset of the unit's weights
};

__device__ __forceinline__ int phase_units(const LayerDev& L, const DensePhase& ph) {
  return (ph.stage == ST_S1 || ph.stage == ST_S4) ? L.counts[CNT_ACTIVE_DEPT] : 1;
}

__device__ __forceinline__ Job decode_job(const LayerDev& L, const DenseArgs& A, int job, int jobs0, int B) {
  Job j;
  j.phase = (job >= jobs0) ? 1 : 0;
  const DensePhase& ph = A.ph[j.phase];
  const int local = job - (j.phase ? jobs0 : 0);
  const int u = local / ph.tiles;
  j.tile = local - u * ph.tiles;
  j.in_list = nullptr;
  j.woff = 0;
  if (ph.stage == ST_S1) {
    const int id = L.active_dept[u];
    j.row0 = L.dept_off[id];
    j.T = L.dept_off[id + 1] - j.row0;
    j.in_list = L.dept_tok + j.row0;
    j.woff = (size_t)id * ph.unit_elems;
  } else if (ph.stage == ST_S4) {
    const int id = L.active_dept[u];
    j.row0 = L.expert_off[id * L.g];
    j.T = L.expert_off[(id + 1) * L.g] - j.row0;
    j.woff = (size_t)id * ph.unit_elems;
  } else {
    j.row0 = 0;
    j.T = B;
  }
  return j;
}

// ---------------------------------------------------------------- the kernel
__global__ void __launch_bounds__(DN_THREADS, 1) k_dense(LayerDev L, DenseArgs A, int B) {
  extern __shared__ unsigned char dn_smem_raw[];
  unsigned char* smem =
      reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(dn_smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + (size_t)DN_NST * DN_STAGE_BYTES);
  uint64_t* empty_bar = full_bar + DN_NST;
  uint64_t* acc_full = empty_bar + DN_NST;
  uint64_t* acc_empty = acc_full + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    for (int s = 0; s < DN_NST; ++s) { bar_init(&full_bar[s], 2); bar_init(&empty_bar[s], 1); }
    for (int b = 0; b < 2; ++b) { bar_init(&acc_full[b], 1); bar_init(&acc_empty[b], 4); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_addr(tmem_slot)),
                 "r"(DN_TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  const int jobs0 = phase_units(L, A.ph[0]) * A.ph[0].tiles;
  const int jobs = jobs0 + (A.nph > 1 ? phase_units(L, A.ph[1]) * A.ph[1].tiles : 0);
  const int G = (int)gridDim.x;

  if (warp == DN_WARP_TMA) {
    // ============================================================ weight chunks -> ring
    if (lane == 0) {
      const uint64_t pol = policy_stream();
      uint32_t g = 0;
      bool ok = true;
      for (int job = (int)blockIdx.x; ok && job < jobs; job += G) {
        const Job j = decode_job(L, A, job, jobs0, B);
        const DensePhase& ph = A.ph[j.phase];
        const int bk = ph.dual ? 32 : 64, nch = ph.K / bk;
        const size_t tile_off = j.woff + (size_t)j.tile * 128 * ph.K;
        const int groups = (j.T + DN_NMAX - 1) / DN_NMAX;
        for (int gi = 0; ok && gi < groups; ++gi) {
          for (int c = 0; c < nch; ++c, ++g) {
            const int s = (int)(g % DN_NST);
            if (!bar_wait(&empty_bar[s], ((g / DN_NST) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
            unsigned char* sa = smem + (size_t)s * DN_STAGE_BYTES;
            bar_arrive_expect_tx(&full_bar[s], DN_A_BYTES);
            if (ph.dual) {
              bulk_load(sa, ph.w + tile_off + (size_t)c * 128 * bk, DN_A_BYTES / 2, &full_bar[s], pol);
              bulk_load(sa + DN_A_BYTES / 2, ph.w1 + tile_off + (size_t)c * 128 * bk, DN_A_BYTES / 2, &full_bar[s], pol);
            } else {
              bulk_load(sa, ph.w + tile_off + (size_t)c * 128 * bk, DN_A_BYTES, &full_bar[s], pol);
            }
          }
        }
      }
    }
  } else if (warp == DN_WARP_MMA) {
    // ============================================================ MMA issue
    if (lane == 0) {
      uint32_t g = 0, a = 0;
      bool ok = true;
      for (int job = (int)blockIdx.x; ok && job < jobs; job += G) {
        const Job j = decode_job(L, A, job, jobs0, B);
        const DensePhase& ph = A.ph[j.phase];
        const int bk = ph.dual ? 32 : 64, nch = ph.K / bk;
        const uint32_t sbo = (uint32_t)bk * 16u;
        const int groups = (j.T + DN_NMAX - 1) / DN_NMAX;
        for (int gi = 0; ok && gi < groups; ++gi, ++a) {
          const int Tg = min(DN_NMAX, j.T - gi * DN_NMAX);
          const int npad = (Tg + 15) & ~15;
          const uint32_t idesc = umma_instr_desc(128, npad);
          const uint32_t buf = a & 1u;
          if (!bar_wait(&acc_empty[buf], ((a >> 1) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t d0 = tmem_base + buf * 128u, d1 = d0 + 64u;
          for (int c = 0; c < nch; ++c, ++g) {
            const int s = (int)(g % DN_NST);
            if (!bar_wait(&full_bar[s], (g / DN_NST) & 1u, abort_flag)) { ok = false; break; }
            tc_fence_after();
            const uint32_t sa = smem_addr(smem + (size_t)s * DN_STAGE_BYTES), sb = sa + DN_A_BYTES;
            for (int ks = 0; ks < bk / 16; ++ks) {
              const uint64_t db = umma_smem_desc(sb + ks * 256, 128, sbo);
              const uint32_t acc = (c | ks) ? 1u : 0u;
              umma(d0, umma_smem_desc(sa + ks * 256, 128, sbo), db, idesc, acc);
              if (ph.dual) umma(d1, umma_smem_desc(sa + DN_A_BYTES / 2 + ks * 256, 128, sbo), db, idesc, acc);
            }
            umma_commit(&empty_bar[s]);  // the stage is free once these MMAs have read it
          }
          if (ok) umma_commit(&acc_full[buf]);
        }
      }
    }
  } else if (warp >= DN_WARP_LOAD0) {
    // ============================================================ activation rows -> ring (stage = w)
    const int w = warp - DN_WARP_LOAD0;
    uint32_t g0 = 0;  // chunk counter at the start of the current (job, token group)
    bool ok = true;
    for (int job = (int)blockIdx.x; ok && job < jobs; job += G) {
      const Job j = decode_job(L, A, job, jobs0, B);
      const DensePhase& ph = A.ph[j.phase];
      const int bk = ph.dual ? 32 : 64, nch = ph.K / bk;
      const int pr = bk / 8;                      // 16-byte pieces per row and chunk
      const int pr_shift = ph.dual ? 2 : 3;
      const uint32_t sbo = (uint32_t)bk * 16u;
      const int groups = (j.T + DN_NMAX - 1) / DN_NMAX;
      for (int gi = 0; ok && gi < groups; ++gi) {
        const int n0 = gi * DN_NMAX, Tg = min(DN_NMAX, j.T - n0);
        // input row of token n0 + lane and n0 + lane + 32, handed around with shuffles below
        int rowA = 0, rowB = 0;
        if (lane < Tg) rowA = j.in_list ? j.in_list[n0 + lane] : j.row0 + n0 + lane;
        if (lane + 32 < Tg) rowB = j.in_list ? j.in_list[n0 + lane + 32] : j.row0 + n0 + lane + 32;
        const int pieces = Tg * pr;
        const int first = (int)((w + DN_NST - (g0 % DN_NST)) % DN_NST);
        for (int c = first; ok && c < nch; c += DN_NST) {
          const uint32_t g = g0 + (uint32_t)c;
          if (lane == 0 && !bar_wait(&empty_bar[w], ((g / DN_NST) & 1u) ^ 1u, abort_flag)) ok = false;
          ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
          if (!ok) break;
          unsigned char* sb = smem + (size_t)w * DN_STAGE_BYTES + DN_A_BYTES;
          const __nv_bfloat16* src = ph.in + (size_t)c * bk;
          for (int i0 = 0; i0 < pieces; i0 += 128) {  // four pieces per lane in flight
            int4 v[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const int i = i0 + q * 32 + lane;
              const int n = i >> pr_shift, kg = i & (pr - 1);
              const int ra = __shfl_sync(0xffffffffu, rowA, n & 31), rb = __shfl_sync(0xffffffffu, rowB, n & 31);
              const int rsel = (n & 32) ? rb : ra;
              v[q] = make_int4(0, 0, 0, 0);
              if (i < pieces) v[q] = __ldcg(reinterpret_cast<const int4*>(src + (size_t)rsel * ph.in_stride + kg * 8));
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const int i = i0 + q * 32 + lane;
              const int n = i >> pr_shift, kg = i & (pr - 1);
              if (i < pieces) *reinterpret_cast<int4*>(sb + (n >> 3) * sbo + kg * 128 + (n & 7) * 16) = v[q];
            }
          }
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic-proxy stores, read by the MMA
          __syncwarp();
          if (lane == 0) bar_arrive(&full_bar[w]);
        }
        g0 += (uint32_t)nch;
      }
    }
  } else {
    // ============================================================ epilogue (warp e owns TMEM lanes 32e..32e+31)
    const int e = warp;
    uint32_t a = 0;
    bool ok = true;
    for (int job = (int)blockIdx.x; ok && job < jobs; job += G) {
      const Job j = decode_job(L, A, job, jobs0, B);
      const DensePhase& ph = A.ph[j.phase];
      const int groups = (j.T + DN_NMAX - 1) / DN_NMAX;
      const int col = j.tile * 128 + e * 32 + lane;  // output column = weight row of the unit
      for (int gi = 0; ok && gi < groups; ++gi, ++a) {
        const int n0 = gi * DN_NMAX, Tg = min(DN_NMAX, j.T - n0);
        const uint32_t buf = a & 1u;
        if (lane == 0 && !bar_wait(&acc_full[buf], (a >> 1) & 1u, abort_flag)) ok = false;
        ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
        if (!ok) break;
        tc_fence_after();
        const uint32_t t0 = tmem_base + ((uint32_t)(e * 32) << 16) + buf * 128u;
        for (int c0 = 0; c0 < Tg; c0 += 16) {
          uint32_t r0[16], r1[16];
          tmem_ld16(t0 + c0, r0);
          if (ph.dual) tmem_ld16(t0 + 64u + c0, r1);
          tmem_ld_wait();
#pragma unroll
          for (int q = 0; q < 16; ++q) {
            const int n = c0 + q;
            if (n < Tg) {
              float v = __uint_as_float(r0[q]);
              if (ph.epi == DE_SWIGLU) v = silu_f(v) * __uint_as_float(r1[q]);
              else if (ph.epi == DE_SIGMA) v = sigma_f(L.sigma, v);
              const size_t o = (size_t)(j.row0 + n0 + n) * ph.out_stride + col;
              if (ph.outf) ph.outf[o] = v;
              else ph.outh[o] = __float2bfloat16_rn(v);
            }
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) bar_arrive(&acc_empty[buf]);
      }
    }
  }

  // common end: every role arrives here, also after an abort
  tc_fence_before();
  __syncthreads();
  if (tid == 0 && *abort_flag) L.counts[CNT_STATUS] = DEAMOE_ERR_TIMEOUT;
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(DN_TMEM_COLS) : "memory");
  }
}

// Copies `units` matrices [rows, K] (element (r, k) of unit u at src[u * src_unit + r * rs + k * cs])
// into the tile layout: unit u at dst + u * dst_unit; tile t (128 rows) and chunk c (bk columns) at
// (t * (K / bk) + c) * 128 * bk elements; inside, the core-matrix layout described at the top.
// One thread per 16-byte piece (8 consecutive k of one row), in destination order.
__global__ void k_pack_tiles(const __nv_bfloat16* __restrict__ src, __nv_bfloat16* __restrict__ dst, int rows, int K,
                             long long rs, long long cs, long long src_unit, long long dst_unit, int bk) {
  const int pr = bk / 8, nch = K / bk;
  const long long pieces = (long long)rows * (K / 8);
  const __nv_bfloat16* s = src + (long long)blockIdx.y * src_unit;
  __nv_bfloat16* d = dst + (long long)blockIdx.y * dst_unit;
  for (long long p = (long long)blockIdx.x * blockDim.x + threadIdx.x; p < pieces; p += (long long)gridDim.x * blockDim.x) {
    long long x = p;
    const int r8 = (int)(x % 8); x /= 8;
    const int kg = (int)(x % pr); x /= pr;
    const int rg = (int)(x % 16); x /= 16;
    const int c = (int)(x % nch); x /= nch;
    const int t = (int)x;
    const long long r = (long long)t * 128 + rg * 8 + r8, k0 = (long long)c * bk + kg * 8;
    __align__(16) __nv_bfloat16 v[8];
#pragma unroll
    for (int e2 = 0; e2 < 8; ++e2) v[e2] = s[r * rs + (k0 + e2) * cs];
    *reinterpret_cast<int4*>(d + p * 8) = *reinterpret_cast<const int4*>(v);
  }
}

}  // namespace

struct DensePlan {
  __nv_bfloat16* tiles;    // all matrices in the tile layout
  size_t o_gu, o_d, o_sg, o_su, o_sd;  // element offsets: stacked gate;up / down^T of the departments, shared expert
  size_t e_gu, e_d;        // elements per department
  int n_sm;
};

bool dense_supported(const LayerDev& L) {
  if (L.vanilla || L.r <= 0) return false;
  if (L.wdt != DEAMOE_BF16 || L.adt != DEAMOE_BF16) return false;
  if (L.h % 128 || L.f % 128) return false;
  if (L.n_shared && (L.fs % 128)) return false;
  return true;
}

deamoe_status_t dense_plan_create(const LayerDev& L, const deamoe_weights_t& w, cudaStream_t s, DensePlan** out,
                                  uint64_t* bytes) {
  if (!dense_supported(L)) return DEAMOE_ERR_UNSUPPORTED;
  DensePlan* p = new (std::nothrow) DensePlan();
  if (!p) return DEAMOE_ERR_ALLOC;
  std::memset(p, 0, sizeof(*p));
  int dev = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&p->n_sm, cudaDevAttrMultiProcessorCount, dev);
  if (p->n_sm <= 0) p->n_sm = 148;
  const size_t fh = (size_t)L.f * L.h;
  p->e_gu = 2 * fh; p->e_d = fh;
  size_t total = 0;
  p->o_gu = total; total += (size_t)L.m * p->e_gu;
  p->o_d = total; total += (size_t)L.m * p->e_d;
  if (L.n_shared) {
    const size_t sh = (size_t)L.fs * L.h;
    p->o_sg = total; total += sh;
    p->o_su = total; total += sh;
    p->o_sd = total; total += sh;
  }
  if (cudaMalloc(&p->tiles, total * 2) != cudaSuccess) {
    cudaGetLastError();
    delete p;
    return DEAMOE_ERR_ALLOC;
  }
  auto pack = [&](const void* src, size_t off, int rows, int K, long long rs, long long cs, long long su, long long du,
                  int units, int bk) {
    const long long pieces = (long long)rows * (K / 8);
    int bx = (int)((pieces + 255) / 256);
    if (bx > 8192) bx = 8192;
    k_pack_tiles<<<dim3(bx, units), 256, 0, s>>>(reinterpret_cast<const __nv_bfloat16*>(src), p->tiles + off, rows, K, rs,
                                                 cs, su, du, bk);
  };
  // departments: gate rows [0, f) and up rows [f, 2f) of one stacked matrix; down applied as W_d^T
  pack(w.dept_gate, p->o_gu, L.f, L.h, L.h, 1, (long long)fh, (long long)p->e_gu, L.m, 64);
  pack(w.dept_up, p->o_gu + fh, L.f, L.h, L.h, 1, (long long)fh, (long long)p->e_gu, L.m, 64);
  pack(w.dept_down, p->o_d, L.h, L.f, 1, L.h, (long long)fh, (long long)p->e_d, L.m, 64);
  if (L.n_shared) {
    pack(w.shared_gate, p->o_sg, L.fs, L.h, L.h, 1, 0, 0, 1, 32);
    pack(w.shared_up, p->o_su, L.fs, L.h, L.h, 1, 0, 0, 1, 32);
    pack(w.shared_down, p->o_sd, L.h, L.fs, 1, L.h, 0, 0, 1, 64);
  }
  cudaError_t e = cudaGetLastError();
  if (e == cudaSuccess) e = cudaFuncSetAttribute(k_dense, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)DN_SMEM);
  if (e != cudaSuccess) {
    cudaGetLastError();
    dense_plan_destroy(p);
    return DEAMOE_ERR_CUDA;
  }
  *out = p;
  *bytes = total * 2;
  return DEAMOE_OK;
}

void dense_plan_destroy(DensePlan* p) {
  if (!p) return;
  if (p->tiles) cudaFree(p->tiles);
  delete p;
}

int dense_launch(DensePlan& p, const LayerDev& L, const DenseIO& io, const int* stages, int n_stages, int B,
                 cudaStream_t s) {
  if (n_stages < 1 || n_stages > 2) return -1;
  DenseArgs A;
  std::memset(&A, 0, sizeof(A));
  A.nph = n_stages;
  for (int i = 0; i < n_stages; ++i) {
    DensePhase& ph = A.ph[i];
    ph.stage = stages[i];
    switch (stages[i]) {
      case ST_S1:
        ph.K = L.h; ph.tiles = 2 * L.f / 128; ph.dual = 0; ph.epi = DE_SIGMA;
        ph.w = p.tiles + p.o_gu; ph.unit_elems = p.e_gu;
        ph.in = io.tokens; ph.in_stride = L.h; ph.outh = io.GU; ph.out_stride = 2 * L.f;
        break;
      case ST_S4:
        ph.K = L.f; ph.tiles = L.h / 128; ph.dual = 0; ph.epi = DE_NONE;
        ph.w = p.tiles + p.o_d; ph.unit_elems = p.e_d;
        ph.in = io.Z; ph.in_stride = L.f; ph.outf = L.O; ph.out_stride = L.h;
        break;
      case ST_SH1:
        ph.K = L.h; ph.tiles = L.fs / 128; ph.dual = 1; ph.epi = DE_SWIGLU;
        ph.w = p.tiles + p.o_sg; ph.w1 = p.tiles + p.o_su;
        ph.in = io.tokens; ph.in_stride = L.h; ph.outh = io.Ysh; ph.out_stride = L.fs;
        break;
      case ST_SH2:
        ph.K = L.fs; ph.tiles = L.h / 128; ph.dual = 0; ph.epi = DE_NONE;
        ph.w = p.tiles + p.o_sd;
        ph.in = io.Ysh; ph.in_stride = L.fs; ph.outf = L.Osh; ph.out_stride = L.h;
        break;
      default:
        return -1;
    }
  }
  k_dense<<<p.n_sm, DN_THREADS, DN_SMEM, s>>>(L, A, B);
  return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

}  // namespace deamoe
