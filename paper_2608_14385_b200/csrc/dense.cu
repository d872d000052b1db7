// Dense schedule: the department matrices (W_g, W_u, W_d of Section 3.2) and the shared expert
// (Eq. (1)) on the fifth-generation tensor cores.
//
// From a few dozen tokens on, a department's token bucket X^j is a dense tile (16 and more rows),
// and the per-warp mma.sync path of the streaming kernel becomes issue-bound.  Here one
// tcgen05.mma covers up to 64 tokens of the bucket x 128 weight rows x 16 columns, with the
// accumulator in tensor memory:
//
//   D[64 tokens, 128 weight rows] += X^j[64, K] . W_tile[128, K]^T
//
// The tokens are the M operand and the weights the N operand.  What limits such a kernel first is
// the one thread that issues the MMAs: an MMA costs it about 125 cycles whatever its shape, a wait
// or a commit 60 to 250, and the weight stream leaves about 700 cycles per 16 KB and SM.  With one
// CTA per SM and 128-row MMAs (4 KB of weights each) that thread was the bottleneck at half the HBM
// rate; either 256-row MMAs or, as here, two CTAs per SM (two issuing threads, each with twice the
// time per chunk, and two independent copy / MMA chains whose stalls overlap) remove it.
// An M = 64 accumulator lives in lanes 32 (r / 16) + r % 16 of tensor memory (row r), so each of
// the four epilogue warps owns 16 tokens and a token's outputs are one contiguous run.
//
// Roles of a CTA (two CTAs per SM, persistent over a list of (unit, 128-row tile) jobs):
//   warps 0-3   epilogue: tcgen05.ld of the finished accumulator, sigma / SwiGLU, stores
//   warp  4     one thread issues the copies of a chunk into the ring: the weights (one 16 KB bulk
//               copy) and the bucket's activation rows (one tiled TMA copy, 64 rows x 64 columns)
//   warp  5     one thread issues the MMAs and the commits that free ring stages / publish accumulators
// The ring has 4 stages of 16 KB weights + 8 KB activation rows.  The activation rows are fetched
// by TMA, not by loads of a warp: while the weights stream at full rate an ordinary load from this
// SM waits 2 to 4 us behind the bulk copies in flight (measured, L2 hit or not), and a warp that
// has to wait that long per chunk cannot keep up, however far ahead it fetches.  The rows' tensor
// map views a row-major [rows, K] plane as [K / 8][rows][8]; a box of 8 x 64 x 8 lands in shared
// memory as 8 column blocks of 64 rows x 16 bytes, which is the core-matrix layout with 128 bytes
// between 8-row groups and 1024 bytes between neighbours along K.  The box is 16, 32 or 64 rows
// high, whichever holds the group's rows (three tensor maps per input plane; the MMA always reads
// 64 rows: the ones past the box are stale shared memory of the same stage and feed accumulator
// rows nobody reads; a box of R rows puts R x 16 bytes between neighbours along K).  The rows
// come through the same per-SM path as the weights, and a 64-row box for a 15-row bucket would
// take a third of that path.  The rows of a bucket are
// contiguous in every input plane (the first stage's tokens are gathered into bucket order by a
// small kernel first); a box may run past the bucket's end, into rows that no output depends on.
// Weights are stored at create time tile by tile and chunk by chunk in the layout the MMA reads,
// so a chunk is one contiguous bulk copy.  Layout of an operand chunk (R rows x 64 columns, bf16,
// "K-major, no swizzle"): 8 x 8 core matrices of 128 contiguous bytes; byte offset of element
// (r, k) = (r / 8) * 1024 + (k / 8) * 128 + (r % 8) * 16 + (k % 8) * 2.
// A job is one tile of one unit.  The CTAs claim the jobs from a counter, one at a time and shortly
// before their current job's last chunks are issued: CTAs are not served by the memory system at
// one rate (dealt round-robin, the first CTA was done 95 us before the last of a 320 us launch), and
// a claimed list ends when the work ends.  The copy role claims and posts each job to the other
// roles through a small queue in shared memory; the last CTA to finish clears the counter.
//
// The first launch of a step (shared expert's and departments' gate / up) is launched programmatically behind the
// kernel that gathers the token rows, which itself sits behind the routing kernel: its CTAs are resident while the
// routing runs, do the shared expert's jobs (they need nothing of the routing) and start the departments' jobs when
// every CTA of the gather kernel has counted itself done.  Every finished department tile is counted into that
// department's completion counter, which the streaming kernel of the private stages, resident as this grid's CTAs
// leave, tests expert by expert.  The second launch (down projections) is an ordinary launch.
#include "dense.cuh"

#include <cuda.h>  // CUtensorMap and the encode function's signature; the entry point is looked up at run time

#include <cstring>
#include <new>

namespace deamoe {

namespace {

constexpr int DN_AST = 4;                   // ring stages
constexpr int DN_CTAS_PER_SM = 2;
constexpr int DN_NMAX = 64;                 // token rows of one accumulator (the MMA's M) = rows of a bucket per pass
constexpr int DN_BK = 64;                   // columns of a chunk
constexpr int DN_TILE = 128;                // weight rows of a tile (the MMA's N)
constexpr int DN_A_BYTES = DN_TILE * DN_BK * 2;   // 16 KB
constexpr int DN_B_BYTES = DN_NMAX * DN_BK * 2;   // 8 KB
constexpr int DN_STAGE_BYTES = DN_A_BYTES + DN_B_BYTES;
constexpr int DN_WARP_TMA = 4, DN_WARP_MMA = 5;
constexpr int DN_THREADS = (DN_WARP_MMA + 1) * 32;
constexpr int DN_GATHER_CTAS_PER_SM = 2;     // CTAs (of 256 threads) of the kernel that gathers the token rows: all resident at once
constexpr int DN_JQ = 4;                    // slots of the CTA's queue of claimed jobs
constexpr int DN_CLAIM_AHEAD = 6;           // chunks left to issue of a job when the copy role claims the next one
constexpr int DN_TMEM_COLS = 2 * DN_TILE;   // 2 accumulator buffers; the CTAs of an SM share its 512 columns
static_assert(DN_TILE == DENSE_TILE_ROWS, "tile height");
constexpr size_t DN_SMEM = (size_t)DN_AST * DN_STAGE_BYTES + 512 /* barriers, control */;
constexpr unsigned DN_SPIN_LIMIT = 1u << 22;  // bounded waits (default poll limit); then an error status, never a hang
static_assert((DN_SMEM + 1024) * DN_CTAS_PER_SM <= 228 * 1024, "shared memory budget");
// No more than DN_CTAS_PER_SM of these CTAs fit an SM's shared memory, and together they ask for no
// more tensor memory than an SM has: the allocation below never waits for another CTA.
static_assert((DN_SMEM + 1024) * (DN_CTAS_PER_SM + 1) > 228 * 1024 && DN_TMEM_COLS * DN_CTAS_PER_SM <= 512,
              "tensor-memory allocation must never block");

#ifdef DEAMOE_TRACE
__device__ long long dn_trace[512 * 16];  // trace builds: per-CTA cycle counters of the last launch
#define DN_T0() const long long dn_t0 = clock64()
#define DN_ADD(k) dn_acc[k] += clock64() - dn_t0
#else
#define DN_T0() ((void)0)
#define DN_ADD(k) ((void)0)
#endif

enum DenseEpi : int { DE_SIGMA = 0, DE_SWIGLU = 1, DE_NONE = 2 };

struct DensePhase {
  int stage;      // ST_S1, ST_S4, ST_SH1 or ST_SH2
  int K, tiles;   // contraction length; DN_TILE-row tiles of a unit
  int dual;       // a tile is half a tile of gate rows followed by the same rows of the up matrix;
                  // epilogue SiLU(a) * b, DN_TILE / 2 outputs per tile
  int epi;
  int out_stride, pad;
  const __nv_bfloat16* w;
  unsigned long long unit_elems;
  __nv_bfloat16* outh;
  float* outf;
};
struct DenseArgs {
  DensePhase ph[2];
  int nph;
  unsigned spin_limit;  // polls after which a bounded wait gives up
  int withhold;         // failure tests: the copy role issues nothing
  int32_t* claim;       // [0]: next job of this launch; [1]: CTAs that have finished (the last one clears both)
  int32_t* s1_done;     // first stage: per department, every epilogue warp adds one per finished tile (null: nobody listens)
  const int32_t* gathered;  // launched beside the routing: CTAs of the gather kernel that are done (null: an ordinary launch)
  int gather_ctas;
};
// tensor maps of the phases' input planes: [phase][box height 16 / 32 / 64 rows]
struct DenseMaps {
  CUtensorMap tm[2][3];
};
// box height index for a group of Tg rows
__host__ __device__ __forceinline__ int box_index(int Tg) { return Tg <= 16 ? 0 : (Tg <= 32 ? 1 : 2); }

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
__device__ __forceinline__ bool bar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag, unsigned limit) {
  for (unsigned it = 0; it < limit; ++it) {
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
// Tiled TMA load of one box of a 3-D tensor map into this CTA only; x is the innermost coordinate.
__device__ __forceinline__ void tensor_load_3d(void* dst, const CUtensorMap* tm, int x, int y, int z, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(smem_addr(dst)), "l"(reinterpret_cast<uint64_t>(tm)), "r"(x), "r"(y), "r"(z), "r"(smem_addr(bar)) : "memory");
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
__device__ __forceinline__ int ld_acquire_gpu(const int32_t* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// ---------------------------------------------------------------- job decoding (all roles alike)
struct Sched {
  int free_jobs;  // jobs at the head of the list that need nothing of the routing (the shared expert's, as phase 0)
  int jobs0;      // tile jobs of phase 0
  int jobs;       // tile jobs of both phases, claimed in this order
};
struct Job {
  int phase;
  int unit;       // department of the job (first and last stage)
  int T;          // token rows of the unit (0: nothing to do)
  int row0;       // first row of the unit's bucket, in its input plane and in its output
  int ncols;      // weight rows of the job = accumulator columns (DN_TILE)
  int col0;       // output column of accumulator column 0
  const __nv_bfloat16* w;    // the job's part of the tile's first chunk; the next chunk is DN_TILE * DN_BK further
};

__device__ __forceinline__ void put_job(volatile Job* q, const Job& j) {
  q->phase = j.phase; q->unit = j.unit; q->T = j.T; q->row0 = j.row0; q->ncols = j.ncols; q->col0 = j.col0; q->w = j.w;
}
__device__ __forceinline__ Job get_job(const volatile Job* q) {
  Job j;
  j.phase = q->phase; j.unit = q->unit; j.T = q->T; j.row0 = q->row0; j.ncols = q->ncols; j.col0 = q->col0; j.w = q->w;
  return j;
}

// Units of a phase: the active departments, or, for the shared expert, the groups of DN_NMAX tokens
// of the batch.  (A department's bucket of more than DN_NMAX rows is rare and stays one job that
// passes over its tile once per group; the shared expert sees every token, so from 65 tokens on
// each of its groups is a job of its own: jobs of one length deal out evenly.)
__device__ __forceinline__ bool phase_routed(const DensePhase& ph) { return ph.stage == ST_S1 || ph.stage == ST_S4; }
__device__ __forceinline__ int phase_units(const LayerDev& L, const DensePhase& ph, int B) {
  return phase_routed(ph) ? __ldcg(L.counts + CNT_ACTIVE_DEPT) : (B + DN_NMAX - 1) / DN_NMAX;
}

// The list as far as it is known before the routing: the shared expert's jobs, if they come first.
__device__ __forceinline__ Sched head_sched(const LayerDev& L, const DenseArgs& A, int B) {
  Sched s;
  s.free_jobs = phase_routed(A.ph[0]) ? 0 : phase_units(L, A.ph[0], B) * A.ph[0].tiles;
  s.jobs0 = s.free_jobs;
  s.jobs = s.free_jobs;
  return s;
}
// The whole list (reads the routing state).
__device__ __forceinline__ Sched make_sched(const LayerDev& L, const DenseArgs& A, int B) {
  Sched s = head_sched(L, A, B);
  s.jobs0 = phase_units(L, A.ph[0], B) * A.ph[0].tiles;
  s.jobs = s.jobs0 + (A.nph > 1 ? phase_units(L, A.ph[1], B) * A.ph[1].tiles : 0);
  return s;
}

__device__ __forceinline__ Job decode_job(const LayerDev& L, const DenseArgs& A, const Sched& sc, int tjob, int B) {
  Job j;
  j.phase = (tjob >= sc.jobs0) ? 1 : 0;
  const DensePhase& ph = A.ph[j.phase];
  const int local = tjob - (j.phase ? sc.jobs0 : 0);
  const int u = local / ph.tiles, tile = local - u * ph.tiles;
  size_t woff = 0;
  j.unit = 0;
  if (ph.stage == ST_S1) {
    const int id = __ldcg(L.active_dept + u);
    j.unit = id;
    j.row0 = __ldcg(L.dept_off + id);
    j.T = __ldcg(L.dept_off + id + 1) - j.row0;
    woff = (size_t)(id - L.dept_lo) * ph.unit_elems;  // the tile arrays start at this object's first department
  } else if (ph.stage == ST_S4) {
    const int id = __ldcg(L.active_dept + u);
    j.unit = id;
    j.row0 = __ldcg(L.expert_off + id * L.g);
    j.T = __ldcg(L.expert_off + (id + 1) * L.g) - j.row0;
    woff = (size_t)(id - L.dept_lo) * ph.unit_elems;
  } else {
    j.row0 = u * DN_NMAX;  // shared expert: unit u = token group u
    j.T = min(DN_NMAX, B - j.row0);
  }
  j.w = ph.w + woff + (size_t)tile * DN_TILE * ph.K;
  j.ncols = DN_TILE;
  j.col0 = ph.dual ? tile * (DN_TILE / 2) : tile * DN_TILE;
  return j;
}

// ---------------------------------------------------------------- the kernel
__global__ void __launch_bounds__(DN_THREADS, DN_CTAS_PER_SM) k_dense(LayerDev L, DenseArgs A, int B, const __grid_constant__ DenseMaps maps) {
  extern __shared__ __align__(1024) unsigned char smem[];
  unsigned char* ring = smem;  // stage s: weights at s * DN_STAGE_BYTES, activation rows DN_A_BYTES further
  uint64_t* a_full = reinterpret_cast<uint64_t*>(ring + (size_t)DN_AST * DN_STAGE_BYTES);
  uint64_t* a_empty = a_full + DN_AST;
  uint64_t* acc_full = a_empty + DN_AST;
  uint64_t* acc_empty = acc_full + 2;
  uint64_t* jq_full = acc_empty + 2;     // queue of claimed jobs: the copy role posts, the five other warps read
  uint64_t* jq_empty = jq_full + DN_JQ;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(jq_empty + DN_JQ);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  // [DN_JQ] decoded jobs (phase -1: no more jobs): the copy role reads the routing state, the other roles
  // have no global-memory latency at a job's start
  volatile Job* jq = reinterpret_cast<volatile Job*>(abort_flag + 1);
  static_assert(sizeof(Job) == 32 && (2 * DN_AST + 4 + 2 * DN_JQ) * 8 + 8 + sizeof(Job) * DN_JQ <= 512, "control region");

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // The kernel behind this one in the stream may become resident as this grid's CTAs leave (it waits for
  // what it needs of this grid's results through counters, or for the whole grid).
  pdl_trigger();
  if (tid == 0) {
    for (int s = 0; s < DN_AST; ++s) { bar_init(&a_full[s], 1); bar_init(&a_empty[s], 1); }
    for (int b = 0; b < 2; ++b) { bar_init(&acc_full[b], 1); bar_init(&acc_empty[b], 4); }
    for (int q = 0; q < DN_JQ; ++q) { bar_init(&jq_full[q], 1); bar_init(&jq_empty[q], 5); }
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

  const int G = (int)gridDim.x;
  // Launched programmatically behind the kernel that gathers the first stage's token rows, this grid may be
  // running before the routing is done.  It starts with the jobs that need nothing of the routing; before the
  // first job that does, the copy role waits (bounded) until every CTA of the gather kernel has counted itself
  // done, which also says that the departments' token lists are published.  (Not griddepcontrol.wait: that
  // waits for the routing kernel's end as well, and the first stage needs only what that kernel publishes early.)
  // The other roles learn of a job from the copy role, so what it has seen they may read.
  Sched sc = head_sched(L, A, B);
  bool routed = false;

  if (warp == DN_WARP_TMA) {
    // ============================================================ weight chunks -> weight ring
    if (lane == 0) {
      const uint64_t pol = policy_stream();
      uint32_t g = 0;
      bool ok = true;
#ifdef DEAMOE_TRACE
      long long dn_acc[2] = {0, 0};
      const long long dn_start = clock64();
#endif
      // failure test: nothing is claimed, posted or copied, and the other roles' wait for a job expires
      if (A.withhold) ok = false;
      int idx = ok ? atomicAdd(A.claim, 1) : 0;
      for (uint32_t jn = 0; ok; ++jn) {
        // post the claimed job (or the end of the list) to the other roles
        const int q = (int)(jn % DN_JQ);
        if (!bar_wait(&jq_empty[q], ((jn / DN_JQ) & 1u) ^ 1u, abort_flag, A.spin_limit)) { ok = false; break; }
        if (idx >= sc.free_jobs && !routed) {
          if (A.gathered) {
            unsigned spins = 0;
            while (ld_acquire_gpu(A.gathered) < A.gather_ctas) {
              __nanosleep(64);
              if (++spins > A.spin_limit / 16 || *abort_flag) { *abort_flag = 1; ok = false; break; }
            }
            if (!ok) break;
            asm volatile("fence.proxy.async;" ::: "memory");  // the gathered rows were stored, the boxes are read by TMA
          }
          routed = true;
          sc = make_sched(L, A, B);
        }
        Job j;
        j.phase = -1;
        if (idx < sc.jobs) j = decode_job(L, A, sc, idx, B);
        put_job(&jq[q], j);
        bar_arrive(&jq_full[q]);
        if (j.phase < 0) break;
        const int nch = A.ph[j.phase].K / DN_BK;
        const uint32_t bytes = (uint32_t)j.ncols * DN_BK * 2;
        const int groups = (j.T + DN_NMAX - 1) / DN_NMAX;
        int left = groups * nch;   // chunks of this job still to issue
        int next = -1;
        for (int gi = 0; ok && gi < groups; ++gi) {
          const int bi = box_index(min(DN_NMAX, j.T - gi * DN_NMAX));
          const CUtensorMap* tm = &maps.tm[j.phase][bi];
          const uint32_t box_bytes = (16u << bi) * DN_BK * 2;
          for (int c = 0; c < nch; ++c, ++g, --left) {
            // the next job is claimed shortly before this one's last chunks are issued: late enough that the
            // CTAs share the end of the list by their speed, early enough that the answer is there in time
            if (left == DN_CLAIM_AHEAD) next = atomicAdd(A.claim, 1);
            const int s = (int)(g % DN_AST);
            { DN_T0();
            if (!bar_wait(&a_empty[s], ((g / DN_AST) & 1u) ^ 1u, abort_flag, A.spin_limit)) { ok = false; break; }
            DN_ADD(0); }
            unsigned char* st = ring + (size_t)s * DN_STAGE_BYTES;
            bar_arrive_expect_tx(&a_full[s], bytes + box_bytes);
            bulk_load(st, j.w + (size_t)c * DN_TILE * DN_BK, bytes, &a_full[s], pol);
            tensor_load_3d(st + DN_A_BYTES, tm, 0, j.row0 + gi * DN_NMAX, c * (DN_BK / 8), &a_full[s]);
          }
        }
        idx = next >= 0 ? next : atomicAdd(A.claim, 1);  // (a job of fewer chunks than the claim runs ahead)
      }
#ifdef DEAMOE_TRACE
      dn_trace[blockIdx.x * 16 + 0] = dn_acc[0];
      dn_trace[blockIdx.x * 16 + 1] = clock64() - dn_start;
      dn_trace[blockIdx.x * 16 + 7] = g;
#endif
    }
  } else if (warp == DN_WARP_MMA) {
    // ============================================================ MMA issue
    if (lane == 0) {
      uint32_t g = 0, a = 0;
      bool ok = true;
#ifdef DEAMOE_TRACE
      long long dn_acc[4] = {0, 0, 0, 0};
      const long long dn_start = clock64();
#endif
      // descriptors of stage 0, first k-step; a k-step of 16 columns is two core matrices (256
      // bytes) further, which adds 16 to the descriptor's address field
      const uint64_t desc0_w = umma_smem_desc(smem_addr(ring), 128, DN_BK * 16);
      // activation rows as the TMA box leaves them: (box rows x 16) bytes between neighbours along K,
      // 128 between 8-row groups; built per token group below
      for (uint32_t jn = 0; ok; ++jn) {
        const int q = (int)(jn % DN_JQ);
        if (!bar_wait(&jq_full[q], (jn / DN_JQ) & 1u, abort_flag, A.spin_limit)) { ok = false; break; }
        const Job j = get_job(&jq[q]);
        bar_arrive(&jq_empty[q]);
        if (j.phase < 0) break;
        const int nch = A.ph[j.phase].K / DN_BK;
        const uint32_t idesc = umma_instr_desc(DN_NMAX, j.ncols);  // tokens: M operand; weight rows: N operand
        const int groups = (j.T + DN_NMAX - 1) / DN_NMAX;
        for (int gi = 0; ok && gi < groups; ++gi, ++a) {
          const uint32_t box_rows = 16u << box_index(min(DN_NMAX, j.T - gi * DN_NMAX));
          const uint64_t desc0_x = umma_smem_desc(smem_addr(ring + DN_A_BYTES), box_rows * 16, 128);
          const uint32_t xstep = (2 * box_rows * 16) >> 4;  // a k-step of 16 columns = two column blocks of the rows
          const uint32_t buf = a & 1u;
          if (!bar_wait(&acc_empty[buf], ((a >> 1) & 1u) ^ 1u, abort_flag, A.spin_limit)) { ok = false; break; }
          tc_fence_after();
          const uint32_t d0 = tmem_base + buf * (uint32_t)DN_TILE;
          for (int c = 0; c < nch; ++c, ++g) {
            const int sa_i = (int)(g % DN_AST);
            { DN_T0();
            if (!bar_wait(&a_full[sa_i], (g / DN_AST) & 1u, abort_flag, A.spin_limit)) { ok = false; break; }
            DN_ADD(1); }
            // (no tcgen05 fence here: the barrier wait orders the copies' writes before the MMAs)
            DN_T0();
            const uint64_t dw = desc0_w + (uint64_t)(sa_i * (DN_STAGE_BYTES >> 4));
            const uint64_t dx = desc0_x + (uint64_t)(sa_i * (DN_STAGE_BYTES >> 4));
            // a k-step of 16 columns: two core matrices further, 256 bytes in the weights
#pragma unroll
            for (int ks = 0; ks < DN_BK / 16; ++ks) umma(d0, dx + xstep * ks, dw + 16 * ks, idesc, (c | ks) ? 1u : 0u);
            DN_ADD(2);
            { DN_T0();
            umma_commit(&a_empty[sa_i]);  // the stage is free once these MMAs have read it
            DN_ADD(3); }
          }
          if (ok) umma_commit(&acc_full[buf]);
        }
      }
#ifdef DEAMOE_TRACE
      dn_trace[blockIdx.x * 16 + 2] = dn_acc[0];
      dn_trace[blockIdx.x * 16 + 3] = dn_acc[1];
      dn_trace[blockIdx.x * 16 + 4] = dn_acc[2];
      dn_trace[blockIdx.x * 16 + 5] = clock64() - dn_start;
      dn_trace[blockIdx.x * 16 + 6] = dn_acc[3];
#endif
    }
  } else if (warp < 4) {
    // ============================================================ epilogue
    // Warp e reads TMEM lanes 32e..32e+31, of which the first 16 hold tokens 16e..16e+15 of the group.
    const int e = warp;
    uint32_t a = 0;
    bool ok = true;
    for (uint32_t jn = 0; ok; ++jn) {
      const int q = (int)(jn % DN_JQ);
      if (lane == 0 && !bar_wait(&jq_full[q], (jn / DN_JQ) & 1u, abort_flag, A.spin_limit)) ok = false;
      ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;   // (also orders lane 0's wait before every lane's read)
      if (!ok) break;
      const Job j = get_job(&jq[q]);
      __syncwarp();
      if (lane == 0) bar_arrive(&jq_empty[q]);
      if (j.phase < 0) break;
      const DensePhase& ph = A.ph[j.phase];
      const int groups = (j.T + DN_NMAX - 1) / DN_NMAX;
      const int nout = ph.dual ? DN_TILE / 2 : j.ncols;  // outputs per token
      for (int gi = 0; ok && gi < groups; ++gi, ++a) {
        const int n0 = gi * DN_NMAX, Tg = min(DN_NMAX, j.T - n0);
        const uint32_t buf = a & 1u;
        if (lane == 0 && !bar_wait(&acc_full[buf], (a >> 1) & 1u, abort_flag, A.spin_limit)) ok = false;
        ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
        if (!ok) break;
        tc_fence_after();
        const int n = 16 * e + lane;                      // token of this lane (lanes 16..31: none)
        const bool mine = lane < 16 && n < Tg;
        // sigma = RMSNorm: the first stage stores G and U un-normalised and adds their squares to
        // the row's two sums; the last stage scales its result by the pair's 1 / rms(Z)
        const bool rms = L.sigma == DEAMOE_SIGMA_RMSNORM;
        const int grow = j.row0 + n0 + n;                 // row of this lane's token in the stage's planes
        float zscale = 1.f;
        if (rms && mine && ph.stage == ST_S4) zscale = rms_scale_fixed(__ldcg(L.ss_z + grow), L.f);
        if (16 * e < Tg) {                                // warp-uniform: some lane of the warp has a token
          const uint32_t t0 = tmem_base + ((uint32_t)(e * 32) << 16) + buf * (uint32_t)DN_TILE;
          const size_t o0 = (size_t)(j.row0 + n0 + n) * ph.out_stride + (size_t)j.col0;
          for (int c0 = 0; c0 < nout; c0 += 16) {
            uint32_t r0[16], r1[16];
            tmem_ld16(t0 + c0, r0);
            if (ph.dual) tmem_ld16(t0 + (uint32_t)(DN_TILE / 2) + c0, r1);
            tmem_ld_wait();
            if (mine) {
              float v[16];
#pragma unroll
              for (int q = 0; q < 16; ++q) {
                v[q] = __uint_as_float(r0[q]) * zscale;
                if (ph.epi == DE_SWIGLU) v[q] = silu_f(v[q]) * __uint_as_float(r1[q]);
                else if (ph.epi == DE_SIGMA) v[q] = sigma_f(L.sigma, v[q]);
              }
              if (rms && ph.stage == ST_S1) {  // 16 columns of one half (f is a multiple of 128)
                float sq = 0.f;
#pragma unroll
                for (int q = 0; q < 16; ++q) sq = fmaf(v[q], v[q], sq);
                atomicAdd(L.ss_gu + (size_t)grow * 2 + ((j.col0 + c0) >= L.f ? 1 : 0), ss_fixed(sq));
              }
              if (ph.outf) {
                float4* dst = reinterpret_cast<float4*>(ph.outf + o0 + c0);
#pragma unroll
                for (int q = 0; q < 4; ++q) dst[q] = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
              } else {
                uint32_t pk[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                  const __nv_bfloat162 h2 = __floats2bfloat162_rn(v[2 * q], v[2 * q + 1]);
                  pk[q] = *reinterpret_cast<const uint32_t*>(&h2);
                }
                uint4* dst = reinterpret_cast<uint4*>(ph.outh + o0 + c0);
                dst[0] = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                dst[1] = make_uint4(pk[4], pk[5], pk[6], pk[7]);
              }
            }
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) bar_arrive(&acc_empty[buf]);
      }
      // a finished tile of the first stage counts towards its department: the streaming kernel that runs the
      // private stages may already be resident and starts an expert when its department's rows are complete
      if (ok && A.s1_done && ph.stage == ST_S1) {
        __threadfence();
        __syncwarp();
        if (lane == 0) atomicAdd(A.s1_done + j.unit, 1);
      }
    }
  }

  // common end: every role arrives here, also after an abort
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    // giving up: copies issued into the ring may still be in flight; stay (bounded: about 64 us)
    // until they have landed before the CTA's shared memory is released
#pragma unroll 1
    for (int i = 0; i < 64; ++i) __nanosleep(1000);
  }
  if (tid == 0 && *abort_flag) L.counts[CNT_STATUS] = DEAMOE_ERR_TIMEOUT;
  if (tid == 0 && atomicAdd(A.claim + 1, 1) == G - 1) {  // the last CTA to finish: nobody claims any more
    A.claim[0] = 0;
    A.claim[1] = 0;
  }
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(DN_TMEM_COLS) : "memory");
  }
}

// Copies `units` matrices [rows, K] (element (r, k) of unit u at src[u * src_unit + r * rs + k * cs])
// into the tile layout of unit u at dst + u * dst_unit.  Source row r becomes row
// R = dst_row0 + (r / spt) * tstride + r % spt of the unit's stacked matrix (two matrices can be
// stacked, or interleaved half a tile at a time); tile R / DN_TILE and chunk k / 64 start at
// ((R / DN_TILE) * (K / 64) + k / 64) * DN_TILE * 64 elements; inside, the core-matrix layout described at
// the top.  One thread per 16-byte piece (8 consecutive k of one row).
__global__ void k_pack_tiles(const __nv_bfloat16* __restrict__ src, __nv_bfloat16* __restrict__ dst, int rows, int K,
                             long long rs, long long cs, long long src_unit, long long dst_unit, int dst_row0, int spt,
                             int tstride) {
  const int k8n = K / 8, nch = K / DN_BK;
  const long long pieces = (long long)rows * k8n;
  const __nv_bfloat16* s = src + (long long)blockIdx.y * src_unit;
  __nv_bfloat16* d = dst + (long long)blockIdx.y * dst_unit;
  for (long long p = (long long)blockIdx.x * blockDim.x + threadIdx.x; p < pieces; p += (long long)gridDim.x * blockDim.x) {
    const int r = (int)(p / k8n), k8 = (int)(p % k8n);
    const int R = dst_row0 + (r / spt) * tstride + r % spt;
    const int t = R / DN_TILE, rg = (R % DN_TILE) / 8, r8 = R % 8, c = k8 / 8, kg = k8 % 8;
    __align__(16) __nv_bfloat16 v[8];
#pragma unroll
    for (int e2 = 0; e2 < 8; ++e2) v[e2] = s[(long long)r * rs + ((long long)k8 * 8 + e2) * cs];
    const size_t o = ((((size_t)t * nch + c) * (DN_TILE / 8) + rg) * 8 + kg) * 64 + (size_t)r8 * 8;
    *reinterpret_cast<int4*>(d + o) = *reinterpret_cast<const int4*>(v);
  }
}

// First stage's input: the tokens of every department's bucket X^j (Section 3.2), in bucket order.
// Row r of Xg = token dept_tok[r]; one block per row, 16 bytes per thread and step.
// Launched programmatically behind the routing kernel: waits (bounded) for that kernel's word that the
// departments' token lists are published, which is well before its end.
__global__ void k_gather_buckets(LayerDev L, const __nv_bfloat16* __restrict__ tokens, __nv_bfloat16* __restrict__ Xg,
                                 const int32_t* __restrict__ routed_flag, int32_t* __restrict__ gathered,
                                 unsigned spin_limit) {
  pdl_trigger();
  __shared__ int s_ok;
  if (threadIdx.x == 0) {
    int ok = 1;
    unsigned spins = 0;
    while (routed_flag && ld_acquire_gpu(routed_flag) == 0) {
      __nanosleep(64);
      if (++spins > spin_limit / 16) { ok = 0; break; }
    }
    if (!ok) L.counts[CNT_STATUS] = DEAMOE_ERR_TIMEOUT;
    s_ok = ok;
  }
  __syncthreads();
  if (!s_ok) return;
  const int rows = __ldcg(L.counts + CNT_TOKEN_DEPT);
  const int v = L.h / 8;
  for (int r = (int)blockIdx.x; r < rows; r += (int)gridDim.x) {
    const int4* src = reinterpret_cast<const int4*>(tokens + (size_t)__ldcg(L.dept_tok + r) * L.h);
    int4* dst = reinterpret_cast<int4*>(Xg + (size_t)r * L.h);
    for (int i = (int)threadIdx.x; i < v; i += (int)blockDim.x) dst[i] = src[i];
  }
  if (gathered) {  // this CTA's rows are stored: count it in for the tensor-core kernel that may already be waiting
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) atomicAdd(gathered, 1);
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

}  // namespace

struct DensePlan {
  __nv_bfloat16* tiles;    // all matrices in the tile layout
  __nv_bfloat16* Xg;       // [max_batch * min(k, m), h] tokens in bucket order
  int xg_rows;
  EncodeTiledFn encode;    // cuTensorMapEncodeTiled, looked up through the runtime
  size_t o_gu, o_d, o_sgu, o_sd;  // element offsets: stacked gate;up / down^T of the departments, shared expert
  size_t e_gu, e_d;        // elements per department
  int n_sm;
  unsigned spin_limit;     // DN_SPIN_LIMIT unless a failure test lowered it
  int withhold;
  int32_t* claim;          // the launches' job counter and count of finished CTAs (zero between launches)
};

bool dense_supported(const LayerDev& L) {
  if (L.vanilla || L.r <= 0) return false;
  if (L.wdt != DEAMOE_BF16 || L.adt != DEAMOE_BF16) return false;
  if (L.h % 256 || L.f % 128) return false;   // whole tiles of [2f, h] and of [h, f]; 64-column chunks
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
  p->spin_limit = DN_SPIN_LIMIT;
  const size_t fh = (size_t)L.f * L.h;
  p->e_gu = 2 * fh; p->e_d = fh;
  size_t total = 0;
  const int m_loc = L.dept_hi - L.dept_lo;  // departments this layer object holds
  p->o_gu = total; total += (size_t)m_loc * p->e_gu;
  p->o_d = total; total += (size_t)m_loc * p->e_d;
  if (L.n_shared) {
    const size_t sh = (size_t)L.fs * L.h;
    p->o_sgu = total; total += 2 * sh;
    p->o_sd = total; total += sh;
  }
  p->xg_rows = L.max_batch * (L.k < L.m ? L.k : L.m);
  if (cudaMalloc(&p->tiles, total * 2) != cudaSuccess ||
      cudaMalloc(&p->Xg, (size_t)p->xg_rows * L.h * 2) != cudaSuccess ||
      cudaMalloc(&p->claim, 2 * sizeof(int32_t)) != cudaSuccess ||
      cudaMemset(p->claim, 0, 2 * sizeof(int32_t)) != cudaSuccess) {
    cudaGetLastError();
    dense_plan_destroy(p);
    return DEAMOE_ERR_ALLOC;
  }
  {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qr = cudaDriverEntryPointSymbolNotFound;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qr) != cudaSuccess ||
        qr != cudaDriverEntryPointSuccess || !fn) {
      cudaGetLastError();
      dense_plan_destroy(p);
      return DEAMOE_ERR_CUDA;
    }
    p->encode = reinterpret_cast<EncodeTiledFn>(fn);
  }
  const int NOSPLIT = 1 << 30;
  auto pack = [&](const void* src, size_t off, int rows, int K, long long rs, long long cs, long long su, long long du,
                  int units, int dst_row0, int spt, int tstride) {
    const long long pieces = (long long)rows * (K / 8);
    int bx = (int)((pieces + 255) / 256);
    if (bx > 8192) bx = 8192;
    k_pack_tiles<<<dim3(bx, units), 256, 0, s>>>(reinterpret_cast<const __nv_bfloat16*>(src), p->tiles + off, rows, K, rs,
                                                 cs, su, du, dst_row0, spt, tstride);
  };
  // departments: gate rows [0, f) and up rows [f, 2f) of one stacked matrix; down applied as W_d^T
  pack(w.dept_gate, p->o_gu, L.f, L.h, L.h, 1, (long long)fh, (long long)p->e_gu, m_loc, 0, NOSPLIT, 0);
  pack(w.dept_up, p->o_gu, L.f, L.h, L.h, 1, (long long)fh, (long long)p->e_gu, m_loc, L.f, NOSPLIT, 0);
  pack(w.dept_down, p->o_d, L.h, L.f, 1, L.h, (long long)fh, (long long)p->e_d, m_loc, 0, NOSPLIT, 0);
  if (L.n_shared) {
    // shared expert: tile t = half a tile of gate rows followed by the same rows of up
    pack(w.shared_gate, p->o_sgu, L.fs, L.h, L.h, 1, 0, 0, 1, 0, DN_TILE / 2, DN_TILE);
    pack(w.shared_up, p->o_sgu, L.fs, L.h, L.h, 1, 0, 0, 1, DN_TILE / 2, DN_TILE / 2, DN_TILE);
    pack(w.shared_down, p->o_sd, L.h, L.fs, 1, L.h, 0, 0, 1, 0, NOSPLIT, 0);
  }
  cudaError_t e = cudaGetLastError();
  if (e == cudaSuccess) e = cudaFuncSetAttribute(k_dense, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)DN_SMEM);
  if (e != cudaSuccess) {
    cudaGetLastError();
    dense_plan_destroy(p);
    return DEAMOE_ERR_CUDA;
  }
  *out = p;
  *bytes = total * 2 + (size_t)p->xg_rows * L.h * 2;
  return DEAMOE_OK;
}

void dense_set_failure_test(DensePlan& p, unsigned spin_limit, int withhold) {
  p.spin_limit = spin_limit ? spin_limit : DN_SPIN_LIMIT;
  p.withhold = withhold;
}

void dense_plan_destroy(DensePlan* p) {
  if (!p) return;
  if (p->tiles) cudaFree(p->tiles);
  if (p->Xg) cudaFree(p->Xg);
  if (p->claim) cudaFree(p->claim);
  delete p;
}

// Tensor map over a row-major bf16 plane [rows, K], viewed as [K / 8][rows][8]; box 8 x box_rows x 8.
static bool encode_rows_map(const DensePlan& p, CUtensorMap* tm, const void* base, int rows, int K, int box_rows) {
  const cuuint64_t dims[3] = {8, (cuuint64_t)rows, (cuuint64_t)(K / 8)};
  const cuuint64_t strides[2] = {(cuuint64_t)K * 2, 16};  // bytes between rows, between 8-column groups
  const cuuint32_t box[3] = {8, (cuuint32_t)box_rows, DN_BK / 8};
  const cuuint32_t estr[3] = {1, 1, 1};
  return p.encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int dense_launch(DensePlan& p, const LayerDev& L, const DenseIO& io, const int* stages, int n_stages, int B,
                 cudaStream_t s) {
  if (n_stages < 1 || n_stages > 2) return -1;
  DenseArgs A;
  std::memset(&A, 0, sizeof(A));
  A.nph = n_stages;
  A.spin_limit = p.spin_limit; A.withhold = p.withhold;
  A.claim = p.claim;
  A.s1_done = io.s1_done;
  DenseMaps maps;
  std::memset(&maps, 0, sizeof(maps));
  int launches = 0;
  bool chained = false;
  for (int i = 0; i < n_stages; ++i) {
    DensePhase& ph = A.ph[i];
    ph.stage = stages[i];
    const void* in = nullptr;
    int in_rows = 0;
    switch (stages[i]) {
      case ST_S1:
        ph.K = L.h; ph.tiles = 2 * L.f / DN_TILE; ph.dual = 0; ph.epi = DE_SIGMA;
        ph.w = p.tiles + p.o_gu; ph.unit_elems = p.e_gu;
        in = p.Xg; in_rows = p.xg_rows; ph.outh = io.GU; ph.out_stride = 2 * L.f;
        if (launch_pdl(k_gather_buckets, dim3(DN_GATHER_CTAS_PER_SM * p.n_sm), dim3(256), 0, s, L, io.tokens, p.Xg, io.routed_flag,
                       io.gathered, io.spin_limit ? io.spin_limit : DN_SPIN_LIMIT) != cudaSuccess)
          return -1;
        chained = io.routed_flag != nullptr && io.gathered != nullptr;
        if (chained) { A.gathered = io.gathered; A.gather_ctas = DN_GATHER_CTAS_PER_SM * p.n_sm; }
        ++launches;
        break;
      case ST_S4:
        ph.K = L.f; ph.tiles = L.h / DN_TILE; ph.dual = 0; ph.epi = DE_NONE;
        ph.w = p.tiles + p.o_d; ph.unit_elems = p.e_d;
        in = io.Z; in_rows = L.max_batch * L.k; ph.outf = L.O; ph.out_stride = L.h;
        break;
      case ST_SH1:
        ph.K = L.h; ph.tiles = L.fs / (DN_TILE / 2); ph.dual = 1; ph.epi = DE_SWIGLU;
        ph.w = p.tiles + p.o_sgu;
        in = io.tokens; in_rows = B; ph.outh = io.Ysh; ph.out_stride = L.fs;
        break;
      case ST_SH2:
        ph.K = L.fs; ph.tiles = L.h / DN_TILE; ph.dual = 0; ph.epi = DE_NONE;
        ph.w = p.tiles + p.o_sd;
        in = io.Ysh; in_rows = L.max_batch; ph.outf = L.Osh; ph.out_stride = L.h;
        break;
      default:
        return -1;
    }
    for (int b = 0; b < 3; ++b)
      if (!encode_rows_map(p, &maps.tm[i][b], in, in_rows, ph.K, 16 << b)) return -1;
  }
  if (n_stages == 1) std::memcpy(maps.tm[1], maps.tm[0], sizeof(maps.tm[0]));
  if (chained) {  // behind the gather kernel, possibly beside the end of the routing
    if (launch_pdl(k_dense, dim3(p.n_sm * DN_CTAS_PER_SM), dim3(DN_THREADS), DN_SMEM, s, L, A, B, maps) != cudaSuccess) return -1;
  } else {
    k_dense<<<p.n_sm * DN_CTAS_PER_SM, DN_THREADS, DN_SMEM, s>>>(L, A, B, maps);
  }
  ++launches;
  return cudaGetLastError() == cudaSuccess ? launches : -1;
}

}  // namespace deamoe

#ifdef DEAMOE_TRACE
extern "C" int deamoe_debug_dense(long long* host, int n) {  // trace builds: counters of the last dense launch
  cudaDeviceSynchronize();
  return (int)cudaMemcpyFromSymbol(host, deamoe::dn_trace, (size_t)n * sizeof(long long));
}
#endif
