// Weight-streaming schedules for bf16 layers.
//
// Every stage of Section 3.2 (department gate/up, private gate/up, private down, department
// down, and the shared / vanilla experts of Eq. (1)) is the same operation: a few token rows
// times a weight matrix that is read exactly once.  At create the matrices are re-packed so
// that one 16-row tile of a matrix is a contiguous stream whose 512-byte pieces are the
// per-lane A fragments of mma.sync.m16n8k16.  One persistent kernel (CTAS_PER_SM co-resident
// CTAs on every SM) then works through a device-built list of items (one or two 16-row tiles x
// the full contraction length).  Warp roles inside a CTA:
//
//   planner warp  : picks the CTA's items (the first stage is dealt out, the rest is claimed in
//                   list order from a global counter), checks their records, resolves all source
//                   pointers and queues a descriptor in shared memory;
//   issue warp    : moves weight chunks (HBM, evict-first) into a shared-memory ring with
//                   cp.async.bulk as soon as a slot is free, and the matching activation rows
//                   (L2) once the item's inputs exist; completion on mbarriers;
//   consumer warps: split each chunk's k-tiles, accumulate in fp32 with mma.sync on bf16
//                   activations (one plane, or hi + lo planes for fp32 tokens) and hand their
//                   partial sums of a finished item to
//   epilogue warp : sums the partials, applies the stage's epilogue (sigma, SwiGLU), stores the
//                   result as the next stage's bf16 planes (or fp32 for the last stage) and
//                   publishes the item's completion with one fence per batch of items.
//
// Weights never depend on earlier stages, so the ring keeps the HBM pipe full across item and
// stage boundaries; only the (tiny) activations wait for their producers.  Two small CTAs per SM
// measured faster than one large one: a CTA's chunks are consumed strictly one after another, so
// the fixed latency of a chunk (barrier wait, header, fragment loads, dependent MMAs, release)
// bounds its rate, and two independent streams per SM hide that latency behind one another.
#include <cstddef>
#include <cstdlib>
#include <cstring>
#include <new>

#include "route_device.cuh"
#include "stream.cuh"
#include "dense.cuh"

namespace deamoe {

constexpr int CTAS_PER_SM = 2;                   // co-resident CTAs of the streaming kernel per SM
constexpr int CONSUMER_WARPS = 4;
constexpr int ISSUE_WARPS = 1;                   // copy-issue warps per CTA (two CTAs per SM, so two per SM)
constexpr int WARP_ISSUE = CONSUMER_WARPS;       // first of the warps that issue the bulk copies
constexpr int WARP_PLAN = WARP_ISSUE + ISSUE_WARPS;  // picks items, fetches records, queues descriptors
constexpr int WARP_EPI = WARP_PLAN + 1;          // reduces, applies epilogues, publishes completions
constexpr int STREAM_THREADS = (WARP_EPI + 1) * 32;
constexpr int DESC_DEPTH = 8;                    // item descriptors queued between planner and epilogue
constexpr int DESC_BYTES = 1024;                 // Seg | tail | weight sources | activation row sources
constexpr int DESC_TAIL = 224, DESC_WSRC = 256, DESC_ASRC = 272;
constexpr int MAX_CAT_INTS_PAD = 8;             // cat_tab: 4 ints for each of 8 categories = 16 B x 8
#ifndef PREFIX_LAST_STAGE
#define PREFIX_LAST_STAGE ST_SH1  // the shared expert's second stage waits for all of the first: it runs from the list
#endif
constexpr int CLAIM_MIN_PER_CTA = 16;            // lists with fewer items per CTA are dealt out, not claimed
constexpr int PREFETCH_BYTES = 512 * 1024;       // per CTA: at most this much of its likely first routed item goes to L2 during the routing
constexpr int CLAIM_AHEAD = 4;                   // unfinished items a CTA may hold while it claims from the last category
constexpr int NRED = 2;                          // reduction buffers between consumers and epilogue warp
constexpr int SLOT_BYTES = 32 * 1024;
constexpr int SLOT_HDR = 128;
constexpr int NSLOT = 3;
constexpr int ACT_PAD = 8;   // floats of padding per activation row in shared memory
constexpr int MAX_QP = 2;    // 8-token passes a consumer warp accumulates for its tile (16 tokens per segment)
constexpr int SEG_TOKENS = 8 * MAX_QP;   // token rows of a segment: a warp accumulates up to MAX_QP passes of 8 tokens for its tile
constexpr int RED_FLOATS = CONSUMER_WARPS * MAX_QP * 128;
constexpr size_t STREAM_SMEM =
    (size_t)NSLOT * SLOT_BYTES + (size_t)NRED * RED_FLOATS * 4 + (size_t)DESC_DEPTH * DESC_BYTES + 1024;
static_assert((STREAM_SMEM + 1024) * CTAS_PER_SM <= 228 * 1024, "shared memory budget");
static_assert((2 * NSLOT + 2 * DESC_DEPTH + 2 * NRED) * 8 + 16 * MAX_CAT_INTS_PAD + 16 * NRED + 32 + 224 <= 1024, "control region");
constexpr unsigned SPIN_LIMIT = 1u << 24;  // bounded waits (default poll limit); then an error status, never a hang
constexpr int MAX_CAT = 8;

enum Epi : int { EPI_SIGMA = 0, EPI_SWIGLU = 1, EPI_NONE = 2 };

// layout of the int32 `sync` array
enum SyncSlot : int {
  SY_NCAT = 0, SY_NSEG = 1, SY_NITEMS = 2,
  SY_CAT = 8,                     // MAX_CAT x {item_base, seg_base, items_per_seg, stage}
  SY_CLAIM = SY_CAT + 4 * MAX_CAT,  // MAX_CAT + 1 claim counters (one per launch)
  SY_DEP = SY_CLAIM + MAX_CAT + 8   // dependency counters
};

// static description of a stage (host-built at create)
struct StageCfg {
  const __nv_bfloat16* w0;  // packed matrix of unit 0
  const __nv_bfloat16* w1;  // second packed matrix of paired stages
  unsigned long long unit_elems;  // packed elements per unit
  int C, rows, n_tiles;     // contraction length, output rows, ceil(rows / 16)
  int paired;               // item = (tile of w0, same tile of w1), epilogue SiLU(a) * b
  int q;                    // tiles per item
  int epi, tg;              // epilogue, max token rows per segment
  int items_per_seg;
  int enabled, pad;
};

// one unit (department / expert / shared expert) x one token group of a stage
struct Seg {
  int item0, n_items, stage, epi;
  int T, q, paired, nB;
  int kc, C, rows, n_tiles;
  int in_stride, out_stride, out_row0, dep_idx;   // dep_idx / dep_target are ints 15 / 16 (planner)
  int dep_target, done_idx, planes, pad0;
  const __nv_bfloat16* w0;
  const __nv_bfloat16* w1;
  const __nv_bfloat16* in0h;   // activations: bf16 "hi" plane, row-major
  const __nv_bfloat16* in0l;   // optional "lo" plane (x - hi), planes == 2
  const __nv_bfloat16* in1h;   // second input of stages whose two matrices read different vectors
  const __nv_bfloat16* in1l;
  __nv_bfloat16* outh;         // output planes of stages that feed another stage
  __nv_bfloat16* outl;
  float* outf;                 // fp32 output of the last stage (read by the combine)
  unsigned long long pad1;
  uint16_t rows16[32];         // input row of each of the T tokens
};
static_assert(sizeof(Seg) == 224, "Seg layout is relied upon by the planner warp");
constexpr int SEG_VEC = sizeof(Seg) / 16;
static_assert(sizeof(Seg) % 16 == 0, "Seg is copied with 16-byte loads");

struct StreamDev {
  StageCfg st[ST_COUNT];
  Seg* segs;
  int32_t* sync;
  int max_segs;
  int dep_s1, dep_s2, dep_s3, dep_sh1, n_dep;  // offsets relative to SY_DEP
  const __nv_bfloat16* packed_lo;  // packed weights: first element and element count (record checks)
  size_t packed_elems;
  int sh_prefix;  // fused schedule with a shared expert: its items are not in the work list
  int early;      // fused DeaMoE layers: the first stage's records are handed over ahead of the rest
  int claim_items;              // fused schedule: the items of the list are claimed, not dealt
  int dense;                    // dense schedule: the list holds the private stages only (the rest runs on tcgen05 kernels)
  int early_stage;              // the stage handed over early (ST_S1 or ST_V1)
  int early_flag, early_items;  // slots (relative to SY_DEP, outside the zeroed range): flag, item count;
                                // early_flag + 2: flag that the rest of the work list exists
  int planes;                  // 1: activations carried as bf16; 2: as bf16 hi + lo (fp32 activations)
  unsigned spin_limit;         // polls after which a bounded wait gives up (SPIN_LIMIT; lower only in failure tests)
  int withhold;                // failure tests: bit 0 = the routing tail raises no hand-over flag; bit 2 = it
                               // publishes an out-of-range slot for the first (token, expert) pair
  // activations between stages, bf16 planes ([rows, width] each)
  __nv_bfloat16 *xh, *xl;      // tokens split (fp32 activations only; bf16 tokens are read in place)
  __nv_bfloat16 *GUh, *GUl, *Yh, *Yl, *Zh, *Zl, *Yshh, *Yshl;
  long long* trace;  // per-CTA cycle counters, only in -DDEAMOE_TRACE builds (else nullptr)
};

#ifdef DEAMOE_TRACE
#define TR_NOW() clock64()
#define TR_ADD(k, t0) tr[k] += clock64() - (t0)
#else
#define TR_NOW() 0ll
#define TR_ADD(k, t0) ((void)(t0))
#endif
enum TraceSlot : int { TR_META = 0, TR_DEP, TR_EMPTY, TR_ISSUE, TR_ITEMS, TR_CHUNKS, TR_PTOTAL, TR_FULL = 8, TR_COMPUTE,
                       TR_EPI, TR_CTOTAL, TR_SLOTS = 16 };

struct StreamPlan {
  StreamDev dev;
  StreamDev dev_dense;  // the view of `dev` that the dense schedule's routing and streaming launches get
  DensePlan* dense;     // tcgen05 kernels for the department / shared-expert stages, or null
  int dense_min;        // batches from this size on take the dense schedule
  int schedule;
  int n_sm;
  int grid;  // CTAs of the streaming kernel: all of them must be resident at once
  void* packed;
  uint64_t bytes;
  cudaEvent_t ev0, ev1;   // profiling event pair (null when profiling is off)
  int ev_recorded;
};

static_assert(sizeof(Seg) == DESC_TAIL && DESC_ASRC + 64 * 8 <= DESC_BYTES, "descriptor layout");


// ---------------------------------------------------------------- PTX wrappers
static __device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
static __device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
static __device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}
static __device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
static __device__ __forceinline__ bool mbar_test_wait(uint64_t* bar, uint32_t parity) {  // never blocks
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
static __device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false if the limit expired or the CTA was told to stop.
// `sleep_ns` > 0 backs off between polls: used by the roles whose wake-up latency is not critical,
// so that their polling does not compete with the consumers for issue slots.
// abort_flag points at the CTA's control words: [0] the abort flag, [CTL_LIMIT] the poll limit of
// this launch (SPIN_LIMIT unless a test lowered it).
constexpr int CTL_LIMIT = 4;
static __device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                                 unsigned sleep_ns = 0) {
  const unsigned limit = (unsigned)abort_flag[CTL_LIMIT];
  for (unsigned it = 0; it < limit; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if (sleep_ns) __nanosleep(sleep_ns);
    if ((it & 1023u) == 1023u && *abort_flag) return false;
  }
  return false;
}
// One lane polls for the whole warp; the other lanes wait at the warp barrier without touching
// the shared-memory pipe.  Every lane then observes the completed phase itself (acquire).
static __device__ __forceinline__ bool mbar_wait_warp(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                                      int lane, unsigned sleep_ns = 0) {
  bool ok = true;
  if (lane == 0) ok = mbar_wait(bar, parity, abort_flag, sleep_ns);
  ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
  __syncwarp();  // orders the other lanes' reads after lane 0's acquire
  return ok;
}
static __device__ __forceinline__ uint64_t policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
static __device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(dst)),
               "l"(src), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
static __device__ __forceinline__ void bulk_g2s_hint(void* dst, const void* src, uint32_t bytes, uint64_t* bar,
                                                     uint64_t policy) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::
          "r"(smem_u32(dst)),
      "l"(src), "r"(bytes), "r"(smem_u32(bar)), "l"(policy)
      : "memory");
}
static __device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async;" ::: "memory"); }
static __device__ __forceinline__ void st_release(int32_t* p, int v) {
  asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
static __device__ __forceinline__ int ld_acquire(const int32_t* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
static __device__ __forceinline__ void mma_bf16(float (&d)[4], const uint4& a, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a.x), "r"(a.y), "r"(a.z), "r"(a.w), "r"(b0), "r"(b1));
}
// ---------------------------------------------------------------- weight re-packing (create)
// dst: [unit][tile][k-tile][lane][8 bf16]; element (row, k) of the logical matrix is read from
// src[unit*src_unit + row*row_stride + k*col_stride].  Rows beyond `rows` are zero.
__global__ void k_pack(const __nv_bfloat16* __restrict__ src, __nv_bfloat16* __restrict__ dst, int rows, int C,
                       long long row_stride, long long col_stride, long long src_unit, long long dst_unit,
                       int n_tiles) {
  const long long per_unit = (long long)n_tiles * (C / 16) * 32;
  const long long src_base = (long long)blockIdx.y * src_unit;
  __nv_bfloat16* out_base = dst + (long long)blockIdx.y * dst_unit;
  for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < per_unit;
       idx += (long long)gridDim.x * blockDim.x) {
    const int lane = (int)(idx & 31);
    const long long tk = idx >> 5;
    const int kt = (int)(tk % (C / 16));
    const int tile = (int)(tk / (C / 16));
    const int g = lane >> 2, tig = lane & 3;
    const int r_lo = tile * 16 + g, r_hi = r_lo + 8;
    const int k0 = kt * 16 + tig * 2;
    __align__(16) __nv_bfloat16 v[8];
    const int rr[4] = {r_lo, r_hi, r_lo, r_hi};
    const int kk[4] = {k0, k0, k0 + 8, k0 + 8};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
#pragma unroll
      for (int d = 0; d < 2; ++d) {
        v[e * 2 + d] = (rr[e] < rows)
                           ? src[src_base + (long long)rr[e] * row_stride + (long long)(kk[e] + d) * col_stride]
                           : __float2bfloat16(0.f);
      }
    }
    *reinterpret_cast<uint4*>(out_base + idx * 8) = *reinterpret_cast<const uint4*>(v);
  }
}

// ---------------------------------------------------------------- work list (every step)
struct CatInfo {
  int stage;
  int unit_kind;  // 0 single unit, 1 active departments, 2 active experts
};

static __device__ __forceinline__ int category_list(const LayerDev& L, const StreamDev& P, CatInfo* cats) {
  int n = 0;
  if (P.dense) {  // department and shared-expert stages run in the dense kernels, between which this list runs
    cats[n++] = {ST_S2, 2};
    cats[n++] = {ST_S3, 2};
    return n;
  }
  // with sh_prefix the streaming kernel generates the shared expert's first stage itself
  if (L.n_shared && !P.sh_prefix) cats[n++] = {ST_SH1, 0};
  const bool sh = L.n_shared;
  if (L.vanilla) {
    cats[n++] = {ST_V1, 2};
    if (sh) cats[n++] = {ST_SH2, 0};
    cats[n++] = {ST_V2, 2};
  } else {
    cats[n++] = {ST_S1, 1};
    if (sh) cats[n++] = {ST_SH2, 0};
    if (L.r > 0) {
      cats[n++] = {ST_S2, 2};
      cats[n++] = {ST_S3, 2};
    }
    cats[n++] = {ST_S4, 1};
  }
  return n;
}

static __device__ __forceinline__ int unit_count(const LayerDev& L, int kind) {
  return kind == 0 ? 1 : (kind == 1 ? L.counts[CNT_ACTIVE_DEPT] : L.counts[CNT_ACTIVE_EXPERT]);
}
static __device__ __forceinline__ int unit_id(const LayerDev& L, int kind, int u) {
  return kind == 0 ? 0 : (kind == 1 ? L.active_dept[u] : L.active_expert[u]);
}
// token rows of unit `id` in `stage`
static __device__ __forceinline__ int unit_tokens(const LayerDev& L, int stage, int id, int B) {
  switch (stage) {
    case ST_S1: return L.dept_off[id + 1] - L.dept_off[id];
    case ST_S4: return L.expert_off[(id + 1) * L.g] - L.expert_off[id * L.g];
    case ST_SH1:
    case ST_SH2: return B;
    default: return L.expert_off[id + 1] - L.expert_off[id];
  }
}
static __device__ __forceinline__ int groups_of(int T, int tg) { return (T + tg - 1) / tg; }
static __device__ __forceinline__ int stage_kind(int stage) {  // 0 single unit, 1 departments, 2 experts
  return (stage == ST_SH1 || stage == ST_SH2) ? 0 : ((stage == ST_S1 || stage == ST_S4) ? 1 : 2);
}

static __device__ __forceinline__ int chunk_k(int C, int q, int act_rows) {
  const int avail = SLOT_BYTES - SLOT_HDR - act_rows * ACT_PAD * 2;
  int kc = (avail / (q * 32 + act_rows * 2)) & ~15;   // largest chunk a slot can hold
  if (kc > C) kc = C;
  const int nch = (C + kc - 1) / kc;                   // then balance the chunks of one item
  kc = (((C + nch - 1) / nch) + 15) & ~15;
  return kc;
}

// Fills the record of (stage, unit id, token group gi).  Everything is computed in registers and
// stored as fourteen 16-byte words, so that `dst` may be global or shared memory and nothing
// passes through per-thread local memory (that cost microseconds per record: this code runs once
// per step, with cold caches).
static_assert(offsetof(Seg, w0) == 80 && offsetof(Seg, outf) == 144 && offsetof(Seg, rows16) == 160, "Seg layout");
static_assert(MAX_QP * 8 <= 16, "build_seg writes at most 16 token rows");
static __device__ void build_seg(const LayerDev& L, const StreamDev& P, int stage, int id, int gi, int B, int item0,
                                 Seg& dst) {
  const StageCfg& sc = P.st[stage];
  const int Tall = unit_tokens(L, stage, id, B);
  const int t0 = gi * SEG_TOKENS;
  const int T = min(SEG_TOKENS, Tall - t0);
  int nB = 1, in_stride = 0, out_stride = 0, out_row0 = 0, dep_idx = -1, dep_target = 0, done_idx = -1, in_row0 = 0;
  const __nv_bfloat16* in0h = nullptr; const __nv_bfloat16* in0l = nullptr;
  const __nv_bfloat16* in1h = nullptr; const __nv_bfloat16* in1l = nullptr;
  __nv_bfloat16* outh = nullptr; __nv_bfloat16* outl = nullptr;
  float* outf = nullptr;
  const int32_t* in_list = nullptr;  // gathered input rows, or in_row0 + token
  // tokens: bf16 tokens are their own (only) plane; fp32 tokens were split by k_split_tokens
  const __nv_bfloat16* tokh = (L.adt == DEAMOE_BF16) ? reinterpret_cast<const __nv_bfloat16*>(L.tokens_raw) : P.xh;
  const __nv_bfloat16* tokl = (L.adt == DEAMOE_BF16) ? nullptr : P.xl;
  const int j = (stage == ST_S2 || stage == ST_S3) ? id / L.g : id;
  switch (stage) {
    case ST_S1:
      in0h = tokh; in0l = tokl; in_stride = L.h; in_list = L.dept_tok + L.dept_off[id] + t0;
      outh = P.GUh; outl = P.GUl; out_stride = 2 * L.f; out_row0 = L.dept_off[id] + t0;
      done_idx = P.dep_s1 + id;
      break;
    case ST_S2:
      in0h = P.GUh; in0l = P.GUl; in1h = P.GUh + L.f; in1l = P.GUl + L.f; nB = 2;
      in_stride = 2 * L.f;
      in_list = L.pair_gurow + L.expert_off[id] + t0;
      outh = P.Yh; outl = P.Yl; out_stride = L.rp; out_row0 = L.expert_off[id] + t0;
      dep_idx = P.dep_s1 + j;
      if (P.dense)  // the first stage runs in the tensor-core kernel, which may still be running: its count per department
        dep_target = DENSE_S1_ARRIVALS * (2 * L.f / DENSE_TILE_ROWS);
      else
        dep_target = groups_of(unit_tokens(L, ST_S1, j, B), SEG_TOKENS) * P.st[ST_S1].n_tiles;
      done_idx = P.dep_s2 + id;
      break;
    case ST_S3:
      in0h = P.Yh; in0l = P.Yl; in_stride = L.rp; in_row0 = L.expert_off[id] + t0;
      outh = P.Zh; outl = P.Zl; out_stride = L.f; out_row0 = in_row0;
      dep_idx = P.dep_s2 + id;
      dep_target = groups_of(Tall, SEG_TOKENS) * P.st[ST_S2].n_tiles;
      // (dense schedule: the last stage runs in a later kernel, nobody polls this counter, and an item
      // without one spares the epilogue warp its fence and atomic)
      done_idx = P.dense ? -1 : P.dep_s3 + j;
      break;
    case ST_S4: {
      const int p0 = L.expert_off[id * L.g];
      in0h = P.Zh; in0l = P.Zl; in_stride = L.f; in_row0 = p0 + t0;
      outf = L.O; out_stride = L.h; out_row0 = p0 + t0;
      if (L.r > 0) {
#pragma unroll 1
        for (int e = 0; e < L.g; ++e) {
          const int Te = L.expert_off[id * L.g + e + 1] - L.expert_off[id * L.g + e];
          dep_target += groups_of(Te, SEG_TOKENS) * P.st[ST_S3].n_tiles;
        }
        dep_idx = P.dep_s3 + id;
      }
      break;
    }
    case ST_SH1:
      in0h = tokh; in0l = tokl; in_stride = L.h; in_row0 = t0;
      outh = P.Yshh; outl = P.Yshl; out_stride = L.fs; out_row0 = t0;
      done_idx = P.dep_sh1;
      break;
    case ST_SH2:
      in0h = P.Yshh; in0l = P.Yshl; in_stride = L.fs; in_row0 = t0;
      outf = L.Osh; out_stride = L.h; out_row0 = t0;
      dep_idx = P.dep_sh1;
      dep_target = groups_of(B, SEG_TOKENS) * P.st[ST_SH1].n_tiles;
      break;
    case ST_V1:
      in0h = tokh; in0l = tokl; in_stride = L.h; in_list = L.expert_tok + L.expert_off[id] + t0;
      outh = P.Yh; outl = P.Yl; out_stride = L.f; out_row0 = L.expert_off[id] + t0;
      done_idx = P.dep_s2 + id;
      break;
    case ST_V2:
      in0h = P.Yh; in0l = P.Yl; in_stride = L.f; in_row0 = L.expert_off[id] + t0;
      outf = L.O; out_stride = L.h; out_row0 = in_row0;
      dep_idx = P.dep_s2 + id;
      dep_target = groups_of(Tall, SEG_TOKENS) * P.st[ST_V1].n_tiles;
      break;
  }
  const int planes = in0l ? P.planes : 1;
  const int kc = chunk_k(sc.C, sc.q, planes * nB * T);
  uint32_t rw[8];  // rows16[0..15], two per word
#pragma unroll
  for (int w = 0; w < 8; ++w) {
    const int ta = 2 * w, tb = 2 * w + 1;
    const uint32_t ra = (ta < T) ? (uint32_t)(in_list ? in_list[ta] : in_row0 + ta) : 0u;
    const uint32_t rb = (tb < T) ? (uint32_t)(in_list ? in_list[tb] : in_row0 + tb) : 0u;
    rw[w] = (ra & 0xffffu) | (rb << 16);
  }
  auto ptr2 = [](const void* a, const void* b) {
    const unsigned long long x = reinterpret_cast<unsigned long long>(a), y = reinterpret_cast<unsigned long long>(b);
    return make_int4((int)(x & 0xffffffffull), (int)(x >> 32), (int)(y & 0xffffffffull), (int)(y >> 32));
  };
  int4* o = reinterpret_cast<int4*>(&dst);
  o[0] = make_int4(item0, sc.items_per_seg, stage, sc.epi);
  o[1] = make_int4(T, sc.q, sc.paired, nB);
  o[2] = make_int4(kc, sc.C, sc.rows, sc.n_tiles);
  o[3] = make_int4(in_stride, out_stride, out_row0, dep_idx);
  o[4] = make_int4(dep_target, done_idx, planes, 0);
  // the packed arrays hold only this layer object's departments [dept_lo, dept_hi) and their experts
  const int sk = stage_kind(stage);
  const size_t wu = (size_t)(id - (sk == 1 ? L.dept_lo : (sk == 2 ? L.dept_lo * L.g : 0)));
  o[5] = ptr2(sc.w0 + wu * sc.unit_elems, sc.w1 ? sc.w1 + wu * sc.unit_elems : nullptr);
  o[6] = ptr2(in0h, in0l);
  o[7] = ptr2(in1h, in1l);
  o[8] = ptr2(outh, outl);
  o[9] = ptr2(outf, nullptr);
  o[10] = make_int4((int)rw[0], (int)rw[1], (int)rw[2], (int)rw[3]);
  o[11] = make_int4((int)rw[4], (int)rw[5], (int)rw[6], (int)rw[7]);
  o[12] = make_int4(0, 0, 0, 0);
  o[13] = make_int4(0, 0, 0, 0);
}

static __device__ void write_seg(const LayerDev& L, const StreamDev& P, int stage, int id, int gi, int B,
                                 int seg_index, int item0) {
  if (seg_index < P.max_segs) build_seg(L, P, stage, id, gi, B, item0, P.segs[seg_index]);
}

// Work-list construction by one CTA (any multiple of 32 threads, at most 1024).  One thread per
// unit (department / expert / shared expert) of every category: the units are numbered
// category after category, a block-wide exclusive scan of their token-group counts gives each
// unit the index of its first segment record, and the thread writes the unit's records.
// `s_excl` is shared-memory scratch for one int per unit (at most 2 m + 2 n + 2 of them).
static __device__ void worklist_block(const LayerDev& L, const StreamDev& P, int B, int* s_excl, bool counters_zeroed,
                                      bool early_done) {
  __shared__ int s_ubase[MAX_CAT + 1], s_segbase[MAX_CAT + 1], s_itembase[MAX_CAT + 1], s_wsum[32], s_carry;
  // the category list lives in shared memory: a per-thread array indexed with a run-time index would
  // sit in local memory and give the kernel a stack frame
  __shared__ CatInfo cats[MAX_CAT];
  __shared__ int s_ncat;
  const int tid = threadIdx.x, nthr = blockDim.x, warp = tid >> 5, lane = tid & 31, nwarp = nthr >> 5;
  if (tid == 0) s_ncat = category_list(L, P, cats);
  __syncthreads();
  const int ncat = s_ncat;
  if (!counters_zeroed)  // else an early hand-over has zeroed the counters, and the first stage may be running
#pragma unroll 1
    for (int i = tid; i < P.n_dep + MAX_CAT + 8; i += nthr) P.sync[SY_CLAIM + i] = 0;
  if (tid == 0) {
    int ub = 0;
#pragma unroll 1
    for (int c = 0; c < ncat; ++c) { s_ubase[c] = ub; ub += unit_count(L, cats[c].unit_kind); }
    s_ubase[ncat] = ub;
    s_carry = 0;
  }
  __syncthreads();
  const int total = s_ubase[ncat];
  auto category_of = [&](int flat) {
    int c = 0;
#pragma unroll 1
    for (int q2 = 1; q2 < ncat; ++q2)
      if (flat >= s_ubase[q2]) c = q2;
    return c;
  };
  // pass 1: exclusive scan of the group counts over all units
#pragma unroll 1
  for (int base = 0; base < total; base += nthr) {
    const int flat = base + tid;
    int gc = 0;
    if (flat < total) {
      const int c = category_of(flat);
      const int stage = cats[c].stage;
      gc = groups_of(unit_tokens(L, stage, unit_id(L, cats[c].unit_kind, flat - s_ubase[c]), B), SEG_TOKENS);
    }
    int incl = gc;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += v;
    }
    if (lane == 31) s_wsum[warp] = incl;
    __syncthreads();
    if (warp == 0) {
      const int w = (lane < nwarp) ? s_wsum[lane] : 0;
      int wi = w;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, wi, o);
        if (lane >= o) wi += v;
      }
      s_wsum[lane] = wi - w;  // exclusive offset of warp `lane`
      if (lane == 31) s_excl[total] = wi;  // chunk total, parked after the units
    }
    __syncthreads();
    const int carry = s_carry;
    if (flat < total) s_excl[flat] = carry + s_wsum[warp] + incl - gc;
    __syncthreads();
    if (tid == 0) s_carry = carry + s_excl[total];
    __syncthreads();
  }
  if (tid == 0) {
    const int nseg = s_carry;
    int ib = 0;
#pragma unroll 1
    for (int c = 0; c < ncat; ++c) {
      const int sb = (s_ubase[c] < total) ? s_excl[s_ubase[c]] : nseg;
      const int sb_next = (c + 1 < ncat && s_ubase[c + 1] < total) ? s_excl[s_ubase[c + 1]] : nseg;
      const int ips = P.st[cats[c].stage].items_per_seg;
      s_segbase[c] = sb; s_itembase[c] = ib;
      P.sync[SY_CAT + 4 * c + 0] = ib;
      P.sync[SY_CAT + 4 * c + 1] = sb;
      P.sync[SY_CAT + 4 * c + 2] = ips;
      P.sync[SY_CAT + 4 * c + 3] = cats[c].stage;
      ib += (sb_next - sb) * ips;
    }
#pragma unroll 1
    for (int c = ncat; c < MAX_CAT; ++c) {
      P.sync[SY_CAT + 4 * c + 0] = ib;
      P.sync[SY_CAT + 4 * c + 1] = nseg;
      P.sync[SY_CAT + 4 * c + 2] = 1;
      P.sync[SY_CAT + 4 * c + 3] = -1;
    }
    P.sync[SY_NCAT] = ncat; P.sync[SY_NSEG] = nseg; P.sync[SY_NITEMS] = ib;
    L.counts[CNT_NSEG] = nseg; L.counts[CNT_NITEMS] = ib;
    if (nseg > P.max_segs) L.counts[CNT_STATUS] = DEAMOE_ERR_UNSUPPORTED;
  }
  __syncthreads();
  TS_MIN(L, 14);
  // pass 2: every unit's records.  A warp stays with one category (warp w takes category w mod the
  // number of categories, and with the other warps of that category every unit of it): the record
  // code differs by stage, and a warp whose lanes held units of different stages would run the
  // stages' code one after the other, from a cold instruction cache.
  const int first_c = (early_done && ncat > 1) ? 1 : 0;  // category 0 was written by early_first_stage()
  const int nc = ncat - first_c;
#pragma unroll 1
  for (int c0 = warp % (nc > 0 ? nc : 1); c0 < nc; c0 += nwarp) {  // (one pass unless there are fewer warps than categories)
    const int c = first_c + c0;
    const bool shared = nwarp >= nc;  // several warps share a category
    const int rank = shared ? warp / nc : 0;
    const int per_c = shared ? (nwarp - c0 + nc - 1) / nc : 1;  // this warp's place among the category's warps
    if (!(early_done && c == 0)) {
      const int stage = cats[c].stage;
      const int nu = s_ubase[c + 1] - s_ubase[c];
      const int ips = P.st[stage].items_per_seg;
#pragma unroll 1
      for (int u = rank * 32 + lane; u < nu; u += per_c * 32) {
        const int flat = s_ubase[c] + u;
        const int id = unit_id(L, cats[c].unit_kind, u);
        const int gc = groups_of(unit_tokens(L, stage, id, B), SEG_TOKENS);
#pragma unroll 1
        for (int gi = 0; gi < gc; ++gi) {
          const int si = s_excl[flat] + gi;
          write_seg(L, P, stage, id, gi, B, si, s_itembase[c] + (si - s_segbase[c]) * ips);
        }
      }
    }
  }
}


// Hand the first stage (department gate / up; for the vanilla layer the experts' gate / up) to the
// streaming kernel as soon as its token lists exist: zero the dependency counters, write the stage's segment records (the same
// numbering worklist_block() gives them: category 0, units in active-department order), publish
// the item count and raise the flag with this step's number.  scr: A + 1 ints of shared memory.
template <int STAGE>  // ST_S1 or ST_V1: a compile-time stage keeps only that stage's record code (this runs cold)
static __device__ void early_first_stage(const LayerDev& L, const StreamDev& P, int B, int* scr) {
  constexpr int stage = STAGE;
  const int kind = stage_kind(stage);
  __shared__ int s_w[33];
  const int tid = threadIdx.x, nthr = blockDim.x, warp = tid >> 5, lane = tid & 31, nwarp = nthr >> 5;
#pragma unroll 1
  for (int i = tid; i < P.n_dep + MAX_CAT + 8; i += nthr) P.sync[SY_CLAIM + i] = 0;
  const int A = unit_count(L, kind);
  const int tg = SEG_TOKENS, ips = P.st[stage].items_per_seg;
  int carry = 0;  // exclusive scan of the departments' group counts, 'nthr' departments at a time
#pragma unroll 1
  for (int base = 0; base < A; base += nthr) {
    const int a = base + tid;
    const int gc = (a < A) ? groups_of(unit_tokens(L, stage, unit_id(L, kind, a), B), tg) : 0;
    int incl = gc;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += y;
    }
    if (lane == 31) s_w[warp] = incl;
    __syncthreads();
    if (warp == 0) {
      const int w = (lane < nwarp) ? s_w[lane] : 0;
      int wi = w;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int y = __shfl_up_sync(0xffffffffu, wi, o);
        if (lane >= o) wi += y;
      }
      s_w[lane] = wi - w;
      if (lane == 31) s_w[32] = wi;
    }
    __syncthreads();
    if (a < A) scr[a] = carry + s_w[warp] + incl - gc;
    carry += s_w[32];
    __syncthreads();
  }
  if (tid == 0) scr[A] = carry;
  __syncthreads();
  TS_MIN(L, 18);
#pragma unroll 1
  for (int a = tid; a < A; a += nthr) {
    const int id = unit_id(L, kind, a);
    const int gc = scr[a + 1] - scr[a];
#pragma unroll 1
    for (int gi = 0; gi < gc; ++gi) write_seg(L, P, stage, id, gi, B, scr[a] + gi, (scr[a] + gi) * ips);
  }
  TS_MIN(L, 19);
  __threadfence();  // every thread's records and zeroed counters, before the flag
  __syncthreads();
  TS_MIN(L, 20);
  if (tid == 0) {
    // the flag carries the item count (+ 1, so that it is never 0), which saves the streaming kernel
    // a dependent load; it is cleared again by the next step's router kernel
    const int items = (carry <= P.max_segs) ? carry * ips : 0;
    P.sync[SY_DEP + P.early_items] = items;
    if (!(P.withhold & 1))  // (a failure test withholds the flag: the streaming kernel's bounded wait must expire)
      st_release(P.sync + SY_DEP + P.early_flag, items + 1);
  }
}

// The top-k keeps a token's logits in registers (up to 32 per lane) unless the layer is too wide or
// its group limit spans more departments than a warp has lanes; then the shared-memory variant runs.
static __host__ __device__ inline bool topk_in_registers(const LayerDev& L) {
  const bool grouped = L.k_dept > 0 && L.k_dept < L.m;
  return L.n <= 1024 && (!grouped || L.m <= 32);
}

// Routing tail in one CTA: top-k + gate weights (warp per token), bucketing, work list.  The
// routing state (selection, gate weights, offsets, token lists, counters) is built in shared
// memory -- the three steps read each other's results from there, not through L2 -- and copied
// to the layer's global arrays at the end for the later kernels and for deamoe_get_routing.
constexpr int FINISH_THREADS = 512;

struct FinishSmem {  // element counts of the shared-memory copy of the routing state
  int idx, w, dept_off, dept_tok, expert_off, expert_tok, pair_slot, pair_gurow, active_dept, active_expert, counts,
      dept_mask, total;
};
static __host__ __device__ FinishSmem finish_layout(int n, int m, int k, int B) {
  FinishSmem f;
  const int pk = B * k, td = B * (k < m ? k : m);
  int o = 0;
  f.idx = o; o += pk; f.w = o; o += pk; f.dept_off = o; o += m + 1; f.dept_tok = o; o += td;
  f.expert_off = o; o += n + 1; f.expert_tok = o; o += pk; f.pair_slot = o; o += pk; f.pair_gurow = o; o += pk;
  f.active_dept = o; o += m; f.active_expert = o; o += n; f.counts = o; o += CNT_COUNT;
  o = (o + 1) & ~1;
  f.dept_mask = o; o += 2 * ((m + 63) / 64);
  f.total = (o + 3) & ~3;
  return f;
}

// Dense schedule: the tensor-core kernel of the first stage needs the departments' token lists and nothing
// else of the routing.  Publish those as soon as they exist (the rest of the routing state follows at this
// kernel's end, as always), zero the step's counters, which that kernel counts into, and raise the flag that
// the kernels queued behind this one wait for.  S: the routing arrays in shared memory; L: in global memory.
static __device__ void dense_hand_over(const LayerDev& S, const LayerDev& L, const StreamDev& P) {
  const int tid = threadIdx.x, nthr = blockDim.x;
#pragma unroll 1
  for (int i = tid; i < P.n_dep + MAX_CAT + 8; i += nthr) P.sync[SY_CLAIM + i] = 0;
  const int td = S.counts[CNT_TOKEN_DEPT], na = S.counts[CNT_ACTIVE_DEPT];
#pragma unroll 1
  for (int j = tid; j <= L.m; j += nthr) L.dept_off[j] = S.dept_off[j];
#pragma unroll 1
  for (int j = tid; j < td; j += nthr) L.dept_tok[j] = S.dept_tok[j];
#pragma unroll 1
  for (int j = tid; j < na; j += nthr) L.active_dept[j] = S.active_dept[j];
  if (tid == 0) { L.counts[CNT_ACTIVE_DEPT] = na; L.counts[CNT_TOKEN_DEPT] = td; }
  __threadfence();
  __syncthreads();
  if (tid == 0) st_release(P.sync + SY_DEP + P.early_flag, 1);  // cleared again by the next step's router kernel
}

// Top-k + gate weights in a grid of their own: one warp per token over as many CTAs as it takes,
// instead of the routing tail's one CTA ranking its tokens sixteen at a time.  Used when a call has
// more tokens than the tail has warps, in the dense schedule, and for routers of more than 256
// experts (16 or 32 logits per lane: inside the 512-thread tail those variants are short of
// registers; the widest measured 4 us slower per token round there).  Writes the layer's global selection arrays; the routing
// tail that follows (topk_warps == 0) reads them from there.
constexpr int TOPK_CTA_WARPS = 4;
__global__ void __launch_bounds__(TOPK_CTA_WARPS * 32)
k_topk_tokens(LayerDev L, int B, int kslices, int32_t* __restrict__ user_idx, float* __restrict__ user_w) {
  pdl_trigger();
  pdl_wait();  // the router logits of the preceding kernel
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int t = (int)blockIdx.x * TOPK_CTA_WARPS + warp;
  if (t >= B) return;
  if (L.n <= 256) topk_one_token_regs<8>(L, t, B, kslices, lane, user_idx, user_w);
  else if (L.n <= 512) topk_one_token_regs<16>(L, t, B, kslices, lane, user_idx, user_w);
  else topk_one_token_regs<32>(L, t, B, kslices, lane, user_idx, user_w);
}

// The same for routers of more than 256 experts: one CTA per token (see topk_one_token_wide).
__global__ void __launch_bounds__(WIDE_MAX_WARPS * 32)
k_topk_wide(LayerDev L, int B, int kslices, int32_t* __restrict__ user_idx, float* __restrict__ user_w) {
  pdl_trigger();
  pdl_wait();  // the router logits of the preceding kernel
  topk_one_token_wide(L, (int)blockIdx.x, B, kslices, user_idx, user_w);
}

// TOPK: who selects (0: a kernel in front of this one; 1: this kernel's warps with the logits in registers; 2: with
// the logits in shared memory; 3: as 1 on a layer without group limit, strict coverage or softmax over all experts,
// whose code is then left out); VAN: a vanilla layer.  Compile-time, so that an instantiation holds only the code its
// steps run: the kernel waits for its instructions most of the time (a step runs it once, from cold caches), and
// code that is never executed but sits between code that is costs fetches.
template <int TOPK, bool VAN>
__global__ void __launch_bounds__(FINISH_THREADS, 1)
k_route_finish(LayerDev L, StreamDev P, int B, int kslices, int topk_warps, int scratch_words,
               int32_t* __restrict__ user_idx, float* __restrict__ user_w) {
  extern __shared__ uint32_t s_dyn[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, tid = threadIdx.x;
  TS_MIN(L, 2);
  pdl_trigger();  // the streaming kernel may be launched now; it waits for this grid before reading
  pdl_wait();     // the router logits of the preceding kernel
  TS_MIN(L, 3);
  const FinishSmem fl = finish_layout(L.n, L.m, L.k, B);
  uint32_t* state = s_dyn + scratch_words;  // persistent part, after the scratch of top-k / bucketing
  // a view of the layer whose routing arrays live in shared memory
  LayerDev S = L;
  S.topk_idx = reinterpret_cast<int32_t*>(state + fl.idx);
  S.topk_w = reinterpret_cast<float*>(state + fl.w);
  S.dept_off = reinterpret_cast<int32_t*>(state + fl.dept_off);
  S.dept_tok = reinterpret_cast<int32_t*>(state + fl.dept_tok);
  S.expert_off = reinterpret_cast<int32_t*>(state + fl.expert_off);
  S.expert_tok = reinterpret_cast<int32_t*>(state + fl.expert_tok);
  S.pair_slot = reinterpret_cast<int32_t*>(state + fl.pair_slot);
  S.pair_gurow = reinterpret_cast<int32_t*>(state + fl.pair_gurow);
  S.active_dept = reinterpret_cast<int32_t*>(state + fl.active_dept);
  S.active_expert = reinterpret_cast<int32_t*>(state + fl.active_expert);
  S.counts = reinterpret_cast<int32_t*>(state + fl.counts);
  S.dept_mask = reinterpret_cast<uint64_t*>(state + fl.dept_mask);
#ifdef DEAMOE_TRACE
  long long tt0 = clock64();
  TS_MIN(L, 11);
#endif
  for (int i = tid; i < CNT_COUNT; i += FINISH_THREADS) S.counts[i] = 0;
  // The status word of the step starts at "ok" here; the streaming kernel may report into the
  // global word while this kernel is still running, so the publication at the end only ever
  // writes an error of this kernel's own into it.
  if (tid == 0) L.counts[CNT_STATUS] = 0;
  if (L.sigma == DEAMOE_SIGMA_RMSNORM) {  // sums of squares of this step's G, U and Z vectors
    const int ngu = 2 * B * (L.k < L.m ? L.k : L.m), nz = B * L.k;
#pragma unroll 1
    for (int i = tid; i < ngu + nz; i += FINISH_THREADS) (i < ngu ? L.ss_gu[i] : L.ss_z[i - ngu]) = 0ull;
  }
  if (TOPK == 0) {  // the selection was made by a kernel of its own
#pragma unroll 1
    for (int i = tid; i < B * L.k; i += FINISH_THREADS) {
      S.topk_idx[i] = __ldcg(L.topk_idx + i);
      S.topk_w[i] = __ldcg(L.topk_w + i);
    }
  } else if (warp < topk_warps) {
    const int per_warp = (L.n * 5 + 15) & ~15;  // n fp32 logits + n flag bytes (memory path only)
    unsigned char* base = reinterpret_cast<unsigned char*>(s_dyn) + (size_t)warp * per_warp;
#pragma unroll 1
    for (int t = warp; t < B; t += topk_warps) {
      // (wider routers that fit the register variants are ranked by k_topk_tokens: their 16 and 32
      // logits per lane would set this kernel's register budget and give it a stack frame)
      if (TOPK == 3) topk_one_token_regs<8, 0>(S, t, B, kslices, lane, user_idx, user_w);
      else if (TOPK == 1) topk_one_token_regs<8, 1>(S, t, B, kslices, lane, user_idx, user_w);
      else topk_one_token(S, t, B, kslices, reinterpret_cast<float*>(base), base + (size_t)L.n * 4, lane, user_idx, user_w);
    }
  }
  __syncthreads();
#ifdef DEAMOE_TRACE
  long long tt1 = clock64();
  TS_MIN(L, 12);
#endif
  bucket_departments(S, B, s_dyn, FINISH_THREADS);
  TS_MIN(L, 17);
  int* early_scr = reinterpret_cast<int*>(s_dyn) + bucket_smem_words(L.n, L.m, B);  // after the masks and offsets
  if (P.dense) dense_hand_over(S, L, P);
  if (!VAN && P.early) early_first_stage<ST_S1>(S, P, B, early_scr);
  bucket_experts(S, B, s_dyn, FINISH_THREADS);
  __syncthreads();
  if (VAN && P.early) early_first_stage<ST_V1>(S, P, B, early_scr);
#ifdef DEAMOE_TRACE
  long long tt2 = clock64();
  TS_MIN(L, 13);
#endif
  worklist_block(S, P, B, reinterpret_cast<int*>(s_dyn), P.early != 0 || P.dense != 0, P.early != 0);
  if (P.early || P.dense) {
    // the rest of the work list is complete: tell the streaming kernel now rather than through this
    // kernel's completion, which comes only after the routing state has been published (on a small
    // layer the streaming kernel has finished the first stage by then and would wait)
    __threadfence();  // every thread's records, before the flag
    __syncthreads();
    if (tid == 0 && !(P.withhold & 1))
      st_release(P.sync + SY_DEP + P.early_flag + 2, 1);  // cleared again by the next step's router kernel
  }
  __syncthreads();
  TS_MIN(L, 15);
  // publish the routing state: every array is a run of 32-bit words in the shared-memory copy.
  // One rolled loop over a small table, so that this once-per-step code stays short.
  __shared__ uint32_t* s_dst[13];
  __shared__ int s_src[13], s_cnt[13];
  if (tid == 0) {
    const int pk = B * L.k;
    int e = 0;
    auto add = [&](void* dst, int src, int cnt) { s_dst[e] = reinterpret_cast<uint32_t*>(dst); s_src[e] = src; s_cnt[e] = cnt; ++e; };
    add(L.topk_idx, fl.idx, pk);
    add(L.topk_w, fl.w, pk);
    add(L.expert_tok, fl.expert_tok, pk);
    add(L.pair_slot, fl.pair_slot, pk);
    add(L.pair_gurow, fl.pair_gurow, pk);
    add(L.dept_tok, fl.dept_tok, S.counts[CNT_TOKEN_DEPT]);
    add(L.dept_off, fl.dept_off, L.m + 1);
    add(L.expert_off, fl.expert_off, L.n + 1);
    add(L.active_dept, fl.active_dept, L.m);
    add(L.active_expert, fl.active_expert, L.n);
    add(L.dept_mask, fl.dept_mask, 2 * ((L.m + 63) / 64));
    add(L.counts, fl.counts, CNT_STATUS);                                              // counts below the status word
    add(L.counts + CNT_STATUS + 1, fl.counts + CNT_STATUS + 1, CNT_COUNT - CNT_STATUS - 1);  // and above it
    if (S.counts[CNT_STATUS] != 0) L.counts[CNT_STATUS] = S.counts[CNT_STATUS];
  }
  __syncthreads();
#pragma unroll 1
  for (int e = 0; e < 13; ++e) {
    uint32_t* dst = s_dst[e];
    const uint32_t* src = state + s_src[e];
    const int cnt = s_cnt[e];
#pragma unroll 1
    for (int i = tid; i < cnt; i += FINISH_THREADS) dst[i] = src[i];
  }
  if (P.withhold & 4) {  // failure test: an out-of-range pair slot, which the combine must skip and report
    __syncthreads();
    if (tid == 0) L.pair_slot[0] = 0x7fff0000;
  }
#ifdef DEAMOE_TRACE
  __syncthreads();
  TS_MAX(L, 4);
  if (threadIdx.x == 0) {
    L.counts[8] = (int)(tt1 - tt0); L.counts[9] = (int)(tt2 - tt1); L.counts[10] = (int)(clock64() - tt2);
    L.counts[11] = S.counts[11]; L.counts[12] = (int)((S.counts[12] - (int)(tt0 & 0x7fffffff)));
  }
#endif
}

// ---------------------------------------------------------------- inner loop of the consumers
// One ring slot holds q weight tiles x kc columns (per-lane A fragments, 512 B per k-tile and tile)
// followed by the activation rows [plane][input][token] x (kc + ACT_PAD) bf16.  A consumer warp
// works on ONE tile: with two tiles in the slot the first half of the consumer warps takes the
// first tile and the second half the second, with one tile all of them share it; the warps on a
// tile split its k-tiles round-robin.  The warp's
// k-tiles are handled G at a time: every shared-memory load of the group is issued before its
// first MMA, so the load latencies overlap.  acc[p] accumulates tokens 8p..8p+7.
template <int NPASS, int PLANES>
static __device__ __forceinline__ void consume_chunk(float (&acc)[MAX_QP][4], const unsigned char* wtile,
                                                     const uint32_t* act, int lo, int kc, int T, int ks, int kw,
                                                     int lane) {
  constexpr int G = (NPASS * PLANES <= 2) ? 4 : 2;
  const int g = lane >> 2, tig = lane & 3;
  const int nkt = kc >> 4;
  const int aw = (kc + ACT_PAD) >> 1;                       // activation row stride in 32-bit words
  const uint4* w0 = reinterpret_cast<const uint4*>(wtile) + lane;
  const uint32_t* rb[NPASS];
#pragma unroll
  for (int p = 0; p < NPASS; ++p) rb[p] = act + min(p * 8 + g, T - 1) * aw + tig;
  const int mine = (nkt > ks) ? (nkt - ks + kw - 1) / kw : 0;  // k-tiles ks, ks+kw, ... of this warp
  for (int i0 = 0; i0 < mine; i0 += G) {
    uint4 A[G];
    uint32_t B[G][NPASS][PLANES][2];
#pragma unroll
    for (int u = 0; u < G; ++u) {
      const int kt = ks + min(i0 + u, mine - 1) * kw;       // clamped: the tail re-reads a valid tile
      A[u] = w0[kt * 32];
#pragma unroll
      for (int p = 0; p < NPASS; ++p)
#pragma unroll
        for (int pl = 0; pl < PLANES; ++pl) {
          const uint32_t* r = rb[p] + kt * 8 + pl * lo;
          B[u][p][pl][0] = r[0];
          B[u][p][pl][1] = r[4];
        }
    }
#pragma unroll
    for (int u = 0; u < G; ++u) {
      if (i0 + u < mine) {
#pragma unroll
        for (int p = 0; p < NPASS; ++p)
#pragma unroll
          for (int pl = 0; pl < PLANES; ++pl) mma_bf16(acc[p], A[u], B[u][p][pl][0], B[u][p][pl][1]);
      }
    }
  }
}

// ---------------------------------------------------------------- the streaming kernel
struct __align__(16) ItemCtx {  // producer-side view of one claimed item
  int seg, item_in_seg;
};

__global__ void __launch_bounds__(STREAM_THREADS, CTAS_PER_SM)
k_stream(LayerDev L, StreamDev P, int B, int cat, int check_deps) {
  extern __shared__ __align__(128) unsigned char smem[];
  unsigned char* ring = smem;
  float* red = reinterpret_cast<float*>(smem + (size_t)NSLOT * SLOT_BYTES);
  unsigned char* descs = reinterpret_cast<unsigned char*>(red) + (size_t)NRED * RED_FLOATS * 4;
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(descs + (size_t)DESC_DEPTH * DESC_BYTES);
  uint64_t* empty_bar = full_bar + NSLOT;
  uint64_t* dq_full = empty_bar + NSLOT;
  uint64_t* dq_empty = dq_full + DESC_DEPTH;
  uint64_t* red_full = dq_empty + DESC_DEPTH;
  uint64_t* red_empty = red_full + NRED;
  int* cat_tab = reinterpret_cast<int*>(red_empty + NRED);             // 4 * MAX_CAT ints
  int* red_info = cat_tab + 4 * MAX_CAT;                               // NRED x {e | tile0 << 8, q, T, 0}
  volatile int* ctl = red_info + 4 * NRED;  // [0] abort, [1] closed, [2] items produced, [3] items completed, [4] poll limit
  volatile int* abort_flag = ctl;
  unsigned char* seg_stage = reinterpret_cast<unsigned char*>(red_info + 4 * NRED + 8);  // one Seg, planner only
  const unsigned spin_limit = P.spin_limit;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int32_t* sy = P.sync;
  if (tid == 0) {
    for (int s = 0; s < NSLOT; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], CONSUMER_WARPS); }
    for (int s = 0; s < DESC_DEPTH; ++s) { mbar_init(&dq_full[s], 1); mbar_init(&dq_empty[s], 1); }
    for (int s = 0; s < NRED; ++s) { mbar_init(&red_full[s], CONSUMER_WARPS); mbar_init(&red_empty[s], 1); }
    ctl[0] = 0; ctl[1] = 0; ctl[2] = 0; ctl[3] = 0; ctl[CTL_LIMIT] = (int)spin_limit;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  TS_MIN(L, 5);
  pdl_trigger();  // the combine kernel may be launched; it waits for this grid to finish

  if (warp == WARP_PLAN) {
    // ================================================================ planner warp
    // Runs ahead of the copy issue.  The items of a CTA are fixed by its index, so their records
    // can be read ahead; the planner waits (bounded) until an item's inputs exist, resolves every
    // source pointer and queues a ready-to-issue descriptor in shared memory.  All global
    // memory latency of the bookkeeping is paid here, off the streaming path.  It is the only
    // warp that reads what the routing kernel wrote, so it alone waits for that kernel.
#ifdef DEAMOE_TRACE
    long long ptr_q = 0, ptr_dep = 0;
#endif
    const int G = (int)gridDim.x;
    int e = 0;
    uint32_t eph = 0;
    bool ok = true;
    // Queue the item `it` of the segment record held as one int4 per lane (lane l < SEG_VEC holds
    // bytes [16 l, 16 l + 16)).  The item is queued before its inputs exist: the issue warp
    // starts the item's weights at once and holds back only its activation rows, until this warp
    // has seen the item's dependency counter at its target and says so in the descriptor.  The
    // poll is done here because an acquire load next to the SM's bulk copies takes microseconds
    // to return, during which the issue warp would not refill the ring.  The next item is queued
    // only after that: the ring holds less than one item's weights beyond the one that waits, and
    // a CTA that claims its items should not hold more of them while it waits (queueing one item
    // beyond the awaited one was measured 1-3 % slower at 16 and 32 tokens).
    int queued = 0;  // items this planner has queued
    int dep_seen = -1;  // dependency counter last seen at its target
    // wait for a queued item's inputs, then release its activation rows (`word` of its descriptor)
    auto await_inputs = [&](volatile int* word, int dep_idx, int dep_target) -> bool {
#ifdef DEAMOE_TRACE
      const long long td0 = clock64();
#endif
      bool seen = true;
      if (lane == 0) {
        unsigned spins = 0;
        while (ld_acquire(P.sync + SY_DEP + dep_idx) < dep_target) {
          __nanosleep(32);
          if (++spins > spin_limit / 16 || *abort_flag) { seen = false; break; }
        }
        if (seen) {
          __threadfence_block();  // what the acquire made visible, before the word the issue warp polls
          *word = 1;
        }
      }
      seen = __shfl_sync(0xffffffffu, (int)seen, 0) != 0;
      dep_seen = dep_idx;
#ifdef DEAMOE_TRACE
      ptr_dep += clock64() - td0;
#endif
      return seen;
    };
    auto emit = [&](const int4 v, const int it) -> bool {
#ifdef DEAMOE_TRACE
      const long long tpq0 = clock64();
#endif
      if (!mbar_wait_warp(&dq_empty[e], eph ^ 1u, abort_flag, lane, 200)) return false;
#ifdef DEAMOE_TRACE
      ptr_q += clock64() - tpq0;
#endif
      unsigned char* ent = descs + (size_t)e * DESC_BYTES;
      if (lane < SEG_VEC) reinterpret_cast<int4*>(ent)[lane] = v;
      __syncwarp();
      const Seg* sg = reinterpret_cast<const Seg*>(ent);
      const int T = sg->T, paired = sg->paired, nB = sg->nB, C = sg->C;
      {
        // consistency check of the record before anything is copied on its behalf
        const size_t woff = (size_t)(sg->w0 - P.packed_lo);
        const bool good = (unsigned)sg->stage < 8u && T >= 1 && T <= MAX_QP * 8 && (nB == 1 || nB == 2) &&
                          (sg->q == 1 || sg->q == 2) && (sg->planes == 1 || sg->planes == 2) && C >= 16 &&
                          sg->kc >= 16 && (sg->kc & 15) == 0 && sg->kc <= C && sg->n_tiles >= 1 &&
                          it >= 0 && it < sg->n_items && sg->in0h != nullptr && woff < P.packed_elems;
        if (!good) {
          if (lane == 0) {
            L.counts[CNT_STATUS] = DEAMOE_ERR_INTERNAL;
            L.counts[8] = sg->stage; L.counts[9] = T; L.counts[10] = sg->kc; L.counts[11] = it; L.counts[12] = C;
            *abort_flag = 1;
          }
          return false;
        }
      }
      const int tile0 = paired ? it : it * sg->q;
      const int q_eff = paired ? 2 : min(sg->q, sg->n_tiles - tile0);
      const int nrows = sg->planes * nB * T;
      const int dep_idx = sg->dep_idx, dep_target = sg->dep_target;
      const bool inputs_exist = !(check_deps & 1) || dep_idx < 0 || dep_idx == dep_seen;
      if (lane == 31) {
        int* tail = reinterpret_cast<int*>(ent + DESC_TAIL);
        tail[0] = 0;      // kind: work
        tail[1] = tile0;
        tail[2] = inputs_exist ? 1 : 0;  // set below otherwise
        tail[3] = q_eff;
        tail[4] = nrows;
      }
      if (lane < 2) {  // weight stream of tile `lane` of the item
        const __nv_bfloat16* wsrc = (lane == 0 || !paired) ? sg->w0 + (size_t)(tile0 + lane) * (C / 16) * 256
                                                           : sg->w1 + (size_t)tile0 * (C / 16) * 256;
        reinterpret_cast<const __nv_bfloat16**>(ent + DESC_WSRC)[lane] = wsrc;
      }
#pragma unroll
      for (int u = 0; u < 2; ++u) {  // activation rows, ordered [plane][input][token]
        const int rr = lane + 32 * u;
        if (rr < nrows) {
          const int pn = rr / T, s = rr - pn * T;
          const int pl = pn / nB, nb = pn - pl * nB;
          const __nv_bfloat16* base = pl ? (nb ? sg->in1l : sg->in0l) : (nb ? sg->in1h : sg->in0h);
          reinterpret_cast<const __nv_bfloat16**>(ent + DESC_ASRC)[rr] = base + (size_t)sg->rows16[s] * sg->in_stride;
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&dq_full[e]);
      const bool seen = inputs_exist || await_inputs(reinterpret_cast<volatile int*>(ent + DESC_TAIL) + 2, dep_idx, dep_target);
      if (++e == DESC_DEPTH) { e = 0; eph ^= 1u; }
      ++queued;
      return seen;
    };

    // The shared expert (Eq. (1)) does not depend on the routing: in the fused schedule its items
    // are generated here, from the batch size alone, and stream while the routing kernel that
    // precedes this grid is still running.
    int first_cta = 0;  // the CTA that takes the next dealt item
    if (P.sh_prefix && cat < 0) {
      Seg* stage_seg = reinterpret_cast<Seg*>(seg_stage);
      for (int st = ST_SH1; ok && st <= PREFIX_LAST_STAGE; ++st) {
        const int ips = P.st[st].items_per_seg;
        const int n_items = groups_of(B, SEG_TOKENS) * ips;
        int have_seg = -1;
        int4 v = make_int4(0, 0, 0, 0);
        for (int x = ((int)blockIdx.x - first_cta + G) % G; ok && x < n_items; x += G) {
          const int gi = x / ips;
          if (gi != have_seg) {
            __syncwarp();
            if (lane == 0) build_seg(L, P, st, 0, gi, B, 0, *stage_seg);
            __syncwarp();
            if (lane < SEG_VEC) v = reinterpret_cast<const int4*>(stage_seg)[lane];
            have_seg = gi;
          }
          ok = emit(v, x - gi * ips);
        }
        first_cta = (first_cta + n_items) % G;
      }
    }

    // The list is walked in up to two phases.  Phase 1 (fused schedule of DeaMoE layers): the
    // routing kernel publishes the records of the first stage as soon as the department token
    // lists exist and raises a flag carrying this step's number; the first stage is by far the
    // longest, so the rest of the routing (expert lists, the other stages' records) hides behind
    // it.  Phase 2, after the routing kernel has completed: everything else.
    int ncat = 0, item_end = 0;
    // Item i of the launch's range goes to CTA (first_cta + i) mod grid: the dealing continues behind
    // the CTAs that took the shared expert's prefix items (equal in size to the first stage's), so
    // those do not start the routed stages one item behind the others.
    int cur_i = ((int)blockIdx.x - first_cta + G) % G;
    auto seg_of = [&](int k, int item, int& it) -> const Seg* {
      const int ib = cat_tab[4 * k + 0], sb = cat_tab[4 * k + 1], ips = cat_tab[4 * k + 2];
      it = (item - ib) % ips;
      return P.segs + sb + (item - ib) / ips;
    };
    // Dealing the items out (rather than giving a CTA one contiguous stretch per category)
    // completes the units one after another, so dependent items of later categories become ready
    // early; contiguous stretches were measured 25-35 % slower for that reason.
    // Fused schedule: the items are not dealt out but CLAIMED, one by one and in list order, from a
    // global counter, and a CTA claims only while fewer than CLAIM_AHEAD of its items are
    // unfinished.  The CTAs move through the list at different speeds (the shared expert's items,
    // stalls at stage boundaries, unequal items); claiming lets the fast ones take what the slow
    // ones would have been left with, and because claims follow the list order an item still
    // depends only on items claimed before it.  The first stage (phase 1) is dealt out, item i to
    // CTA i mod grid, like the categories of a staged launch; claiming starts with the second
    // category.  A short list (fewer than CLAIM_MIN_PER_CTA items per CTA: a single token, a small
    // layer) is dealt out entirely: it loses more to the claim's latency than it gains (171 against
    // 164 us for one token on the DeepSeek-V3 shape).
    int claim_base = 0x7fffffff;  // first claimed item (set in phase 2 of a fused launch)
    bool claiming = false;        // the dealt items before claim_base are used up
    auto next_item = [&](int& k) -> int {  // next item of this CTA, -1 at the end of the phase
      int item = -1;
      if (!claiming) {
        if (cur_i >= item_end) return -1;
        item = cur_i;
        cur_i += G;
        if (item >= claim_base) { claiming = true; item = -1; }
      }
      if (claiming) {
        if (lane == 0) {
          unsigned spins = 0;
          while (queued - ctl[3] >= CLAIM_AHEAD) {  // throttle: stay close to what is actually finished
            __nanosleep(100);
            if (++spins > spin_limit / 16 || *abort_flag) break;
          }
          item = claim_base + atomicAdd(P.sync + SY_CLAIM, 1);
        }
        item = __shfl_sync(0xffffffffu, item, 0);
        if (item >= item_end) { cur_i = item_end; return -1; }
      }
      k = 0;
      for (int q2 = 1; q2 < ncat; ++q2)
        if (item >= cat_tab[4 * q2]) k = q2;
      return item;
    };
    // Three segment records are in flight (this item's and the next two), so the planner pays one
    // L2 latency per three items, not per item.
    auto walk = [&]() {
      const Seg* sp0 = nullptr; const Seg* sp1 = nullptr; const Seg* sp2 = nullptr;
      int it0 = 0, it1 = 0, it2 = 0;
      int4 v0 = make_int4(0, 0, 0, 0), v1 = v0, v2 = v0;  // lane l < SEG_VEC holds bytes [16l, 16l+16) of a record
      auto fetch = [&](const Seg*& sp, int& it, int4& v) {
        sp = nullptr;
        int k = 0;
        const int item = next_item(k);
        if (item >= 0) {
          sp = seg_of(k, item, it);
          // L2 load: in phase 1 the records were written while this kernel was already running
          if (lane < SEG_VEC) v = __ldcg(reinterpret_cast<const int4*>(sp) + lane);
        }
      };
      fetch(sp0, it0, v0);
      if (!claiming) fetch(sp1, it1, v1);
      if (!claiming) fetch(sp2, it2, v2);
      while (ok && sp0) {
        const Seg* sp3 = nullptr; int it3 = 0; int4 v3 = make_int4(0, 0, 0, 0);
        if (!claiming) fetch(sp3, it3, v3);  // read ahead: the record of the item three ahead
        ok = emit(v0, it0);
        // rotate the record pipeline
        sp0 = sp1; it0 = it1; v0 = v1;
        sp1 = sp2; it1 = it2; v1 = v2;
        sp2 = sp3; it2 = it3; v2 = v3;
        if (ok && !sp0 && claiming) fetch(sp0, it0, v0);  // no read-ahead while claiming: a claimed item is a held item
      }
    };

    if (P.early && cat < 0 && ok) {
      // While the routing is still in progress HBM is nearly idle.  When almost every department
      // will be active anyway (the host decides from the batch size), bring the weights of the
      // item this CTA gets if the first departments are active into L2: whichever CTA ends up
      // with an item of those departments then streams it from L2.  A wrong guess only costs
      // reads nobody was waiting for.
      // (The vanilla layer does the same with its experts when nearly all of them will be active.)
      if ((check_deps & 4) && lane == 0) {
        const StageCfg& sc = P.st[P.early_stage];
        const int x = ((int)blockIdx.x - first_cta + G) % G;
        const int unit = x / sc.items_per_seg, it = x - unit * sc.items_per_seg;
        if (unit < (L.vanilla ? L.n : L.dept_hi - L.dept_lo)) {  // (offsets below are relative to this object's first unit)
          const int tile0 = sc.paired ? it : it * sc.q;
          const int ntile = sc.paired ? 1 : min(sc.q, sc.n_tiles - tile0);
          const size_t tile_bytes = (size_t)(sc.C / 16) * 512;
          const size_t off = (size_t)unit * sc.unit_elems * 2 + (size_t)tile0 * tile_bytes;
          size_t bytes = (size_t)ntile * tile_bytes;
          const size_t cap = sc.paired ? PREFETCH_BYTES / 2 : PREFETCH_BYTES;  // a paired item has a tile of each matrix
          if (bytes > cap) bytes = cap;
#pragma unroll 1
          for (size_t o = 0; o < bytes; o += 32768) {
            const unsigned chunk = (unsigned)((bytes - o < 32768) ? (bytes - o) : 32768);
            asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(reinterpret_cast<const char*>(sc.w0) + off + o), "r"(chunk) : "memory");
            if (sc.paired)
              asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(reinterpret_cast<const char*>(sc.w1) + off + o), "r"(chunk) : "memory");
          }
        }
      }
      int n1 = 0;
      if (lane == 0) {
        const int32_t* flag = P.sync + SY_DEP + P.early_flag;
        unsigned spins = 0;
        bool seen = true;
        int fv;
        while ((fv = ld_acquire(flag)) == 0) {
          __nanosleep(64);
          if (++spins > spin_limit / 16 || *abort_flag) { seen = false; break; }
        }
        n1 = seen ? fv - 1 : -1;  // the flag is the first stage's item count + 1
      }
      n1 = __shfl_sync(0xffffffffu, n1, 0);
      if (n1 < 0) {
        ok = false;
      } else {
        if (lane == 0) {
          cat_tab[0] = 0; cat_tab[1] = 0; cat_tab[2] = P.st[P.early_stage].items_per_seg; cat_tab[3] = P.early_stage;
        }
        __syncwarp();
        ncat = 1; item_end = n1;
        walk();
      }
    }

    // The rest of the work list is complete when the routing kernel says so (fused schedule of a
    // layer with the early hand-over: a second flag) or when it has completed.
    bool waited = false;  // for the routing kernel's completion
    if ((P.early && cat < 0) || (check_deps & 16)) {
      // (dense schedule, check_deps & 16: the kernel in front of this one is the first tensor-core launch, which
      // runs beside the end of the routing; what the items need of that launch they await item by item)
      if (lane == 0) {
        const int32_t* flag = P.sync + SY_DEP + P.early_flag + 2;
        unsigned spins = 0;
        while (ld_acquire(flag) == 0) {
          __nanosleep(64);
          if (++spins > spin_limit / 16 || *abort_flag) { ok = false; break; }
        }
      }
      ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
    } else {
      pdl_wait();
      waited = true;
    }
    cat_tab[lane] = __ldcg(sy + SY_CAT + lane);  // 4 * MAX_CAT == 32 entries
    __syncwarp();
    // item range of this launch: one category (staged) or everything (fused)
    ncat = __ldcg(sy + SY_NCAT);
    if (cat >= 0) cur_i = cat_tab[4 * cat] + (int)blockIdx.x;
    item_end = (cat >= 0) ? cat_tab[4 * (cat + 1)] : __ldcg(sy + SY_NITEMS);
    if (*abort_flag && lane == 0) L.counts[CNT_STATUS] = DEAMOE_ERR_TIMEOUT;  // set before the routing kernel reset it
    if (cat < 0 && P.claim_items && ncat >= 2 && item_end >= CLAIM_MIN_PER_CTA * G) claim_base = cat_tab[4];
    if (ok) walk();
#ifdef DEAMOE_TRACE
    if (lane == 0 && P.trace) {
      P.trace[(size_t)blockIdx.x * TR_SLOTS + 15] = ptr_q;
      P.trace[(size_t)blockIdx.x * TR_SLOTS + 7] = ptr_dep;
    }
#endif
    if (!ok && lane == 0) { L.counts[CNT_STATUS] = DEAMOE_ERR_TIMEOUT; *abort_flag = 1; }
    // end marker (also after an abort, so the downstream warps leave their loops)
    mbar_wait_warp(&dq_empty[e], eph ^ 1u, abort_flag, lane);
    if (lane == 0) {
      reinterpret_cast<int*>(descs + (size_t)e * DESC_BYTES + DESC_TAIL)[0] = 1;
      mbar_arrive(&dq_full[e]);
    }
    // This grid must not complete before the routing kernel has: the combine kernel behind it
    // reads the routing state that kernel publishes last.
    if (!waited) pdl_wait();
    return;
  }

  if (warp == WARP_ISSUE) {
    // ================================================================ copy-issue warp
    // Two cursors walk the CTA's chunk stream.  The WEIGHT cursor runs ahead: weights depend on
    // nothing, so a chunk's header and weight tiles are issued as soon as a ring slot is free,
    // also while the item's inputs do not exist yet.  The ACTIVATION cursor follows: the (tiny)
    // activation rows of a chunk are copied once the planner warp has seen the dependency counter
    // of its item at its target and set the descriptor's word (then a proxy fence, because the
    // rows were written with ordinary stores by other CTAs).  So at a stage boundary the HBM pipe keeps running and
    // a waiting item costs only the latency of its activation rows, not of its weights.
    // Issuing a chunk's copies keeps the warp busy for 600-1000 cycles (about 270 for a bulk-copy
    // instruction plus 55 for every further lane that takes part).
    static_assert(ISSUE_WARPS == 1, "the two-cursor issue loop is written for one issue warp per CTA");
    const uint64_t pol = policy_evict_first();
    // weight cursor
    int e_w = 0, cw = 0, ch_w = 0, nch_w = 0, kc0_w = 0, C_w = 0, T_w = 0, tile0_w = 0, qeff_w = 0, nrows_w = 0, hflags_w = 0;
    uint32_t eph_w = 0;
    bool w_loaded = false, end_seen = false;
    const __nv_bfloat16* wsrc_w = nullptr;
    // activation cursor
    int e_a = 0, ca = 0, ch_a = 0, nch_a = 0, kc0_a = 0, C_a = 0, qeff_a = 0, nrows_a = 0, dep_idx_a = -1;
    bool a_loaded = false, a_ready = false;
    const volatile int* ready_a = nullptr;
    const __nv_bfloat16* asrc_a[2] = {nullptr, nullptr};
    int dep_ok = -1;  // dependency counter behind whose completion this warp has fenced
    unsigned idle = 0;
    bool ok = true;
#ifdef DEAMOE_TRACE
    bool routed_seen = false;
    long long tr[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    const long long tp0 = clock64();
#endif
    while (ok) {
      bool progressed = false;
      // ---- weights of chunk cw
      if (!end_seen && !w_loaded) {
        const bool have = __shfl_sync(0xffffffffu, (lane == 0) ? (int)mbar_test_wait(&dq_full[e_w], eph_w) : 0, 0) != 0;
        if (have) {
          __syncwarp();
          const unsigned char* ent = descs + (size_t)e_w * DESC_BYTES;
          const Seg* sg = reinterpret_cast<const Seg*>(ent);
          const int* tail = reinterpret_cast<const int*>(ent + DESC_TAIL);
          if (tail[0] != 0) {
            end_seen = true;
          } else {
            tile0_w = tail[1]; qeff_w = tail[3]; nrows_w = tail[4];
            T_w = sg->T; kc0_w = sg->kc; C_w = sg->C;
            hflags_w = (qeff_w << 4) | (sg->planes << 8) | (sg->nB << 12);
            wsrc_w = (lane < 2) ? reinterpret_cast<const __nv_bfloat16* const*>(ent + DESC_WSRC)[lane] : nullptr;
            nch_w = (C_w + kc0_w - 1) / kc0_w;
            ch_w = 0;
            w_loaded = true;
#ifdef DEAMOE_TRACE
            tr[TR_ITEMS] += 1; tr[TR_CHUNKS] += nch_w;
#endif
          }
        }
      }
      if (w_loaded) {
        const int slot = cw % NSLOT;
        const uint32_t phase = (uint32_t)(cw / NSLOT) & 1u;
        const bool free_slot =
            __shfl_sync(0xffffffffu, (lane == 0) ? (int)mbar_test_wait(&empty_bar[slot], phase ^ 1u) : 0, 0) != 0;
        if (free_slot) {
          __syncwarp();
          const int k0 = ch_w * kc0_w;
          const int kc = min(kc0_w, C_w - k0);
          unsigned char* sbase = ring + (size_t)slot * SLOT_BYTES;
          const uint32_t wbytes = (uint32_t)kc * 32u;
          if (lane == 0) {
            *reinterpret_cast<int4*>(sbase) = make_int4(0, hflags_w | (ch_w == 0 ? 1 : 0) | (ch_w == nch_w - 1 ? 2 : 0),
                                                        kc | (T_w << 16), e_w | (tile0_w << 8));
            mbar_arrive_expect_tx(&full_bar[slot], (uint32_t)qeff_w * wbytes + (uint32_t)nrows_w * (uint32_t)kc * 2u);
          }
          __syncwarp();
          if (lane < qeff_w)
            bulk_g2s_hint(sbase + SLOT_HDR + (size_t)lane * wbytes, wsrc_w + (size_t)(k0 / 16) * 256, wbytes,
                          &full_bar[slot], pol);
          ++cw;
          progressed = true;
          if (++ch_w == nch_w) {
            w_loaded = false;
            if (++e_w == DESC_DEPTH) { e_w = 0; eph_w ^= 1u; }
          }
        }
      }
      // ---- activation rows of chunk ca (its weights have been issued)
      if (ca < cw) {
        if (!a_loaded) {
          const unsigned char* ent = descs + (size_t)e_a * DESC_BYTES;
          const Seg* sg = reinterpret_cast<const Seg*>(ent);
          const int* tail = reinterpret_cast<const int*>(ent + DESC_TAIL);
          qeff_a = tail[3]; nrows_a = tail[4];
          kc0_a = sg->kc; C_a = sg->C;
          dep_idx_a = sg->dep_idx;
#pragma unroll
          for (int u = 0; u < 2; ++u)
            asrc_a[u] = (lane + 32 * u < nrows_a)
                            ? reinterpret_cast<const __nv_bfloat16* const*>(ent + DESC_ASRC)[lane + 32 * u] : nullptr;
          nch_a = (C_a + kc0_a - 1) / kc0_a;
          ch_a = 0;
          a_loaded = true;
          a_ready = !(check_deps & 1) || dep_idx_a < 0 || dep_idx_a == dep_ok;
          ready_a = reinterpret_cast<const volatile int*>(tail + 2);
#ifdef DEAMOE_TRACE
          if (lane == 0 && !routed_seen && sg->stage != ST_SH1 && sg->stage != ST_SH2 && L.ts) {
            routed_seen = true;
            const unsigned long long g = gtime();
            atomicMin(L.ts + 6, g); atomicMax(L.ts + 16, g);
          }
#endif
        }
        if (!a_ready) {
#ifdef DEAMOE_TRACE
          const long long td0 = clock64();
#endif
          // the planner warp polls the counter and sets this word of the descriptor
          const int seen = __shfl_sync(0xffffffffu, (lane == 0) ? *ready_a : 0, 0);
          if (seen) {
            __threadfence_block();
            dep_ok = dep_idx_a;
            fence_proxy_async();  // the rows were written through the generic proxy; the copies read through the async proxy
            a_ready = true;
          }
#ifdef DEAMOE_TRACE
          tr[TR_DEP] += clock64() - td0;
#endif
        }
        if (a_ready) {
          const int slot = ca % NSLOT;
          const int k0 = ch_a * kc0_a;
          const int kc = min(kc0_a, C_a - k0);
          unsigned char* abase = ring + (size_t)slot * SLOT_BYTES + SLOT_HDR + (size_t)qeff_a * kc * 32;
          const int astride = kc + ACT_PAD;
#pragma unroll
          for (int u = 0; u < 2; ++u) {
            const int rr = lane + 32 * u;
            if (rr < nrows_a)
              bulk_g2s(abase + (size_t)rr * astride * 2, asrc_a[u] + k0, (uint32_t)kc * 2u, &full_bar[slot]);
          }
          ++ca;
          progressed = true;
          if (++ch_a == nch_a) {
            a_loaded = false;
            if (++e_a == DESC_DEPTH) e_a = 0;
          }
        }
      }
      if (end_seen && ca == cw) break;
      if (progressed) {
        idle = 0;
      } else {
        if (++idle > spin_limit || *abort_flag) { ok = false; break; }
        __nanosleep(20);
      }
    }
    if (!ok && lane == 0) { L.counts[CNT_STATUS] = DEAMOE_ERR_TIMEOUT; *abort_flag = 1; }
    if (!ok) {
      // giving up: the bulk copies this warp has issued may still be in flight towards the ring;
      // stay (bounded: about 64 us, many times a copy's latency) until they have landed, so that
      // the CTA's shared memory is not released under them
#pragma unroll 1
      for (int i = 0; i < 64; ++i) __nanosleep(1000);
    }
#ifdef DEAMOE_TRACE
    tr[TR_PTOTAL] = clock64() - tp0;
    if (lane == 0 && P.trace)
      for (int i = 0; i < 7; ++i) P.trace[(size_t)blockIdx.x * TR_SLOTS + i] = tr[i];
#endif
    // end-of-work marker for the consumers, in the slot after the last chunk
    const int slot = cw % NSLOT;
    const uint32_t phase = (uint32_t)(cw / NSLOT) & 1u;
    if (mbar_wait_warp(&empty_bar[slot], phase ^ 1u, abort_flag, lane) && lane == 0) {
      *reinterpret_cast<int4*>(ring + (size_t)slot * SLOT_BYTES) = make_int4(1, 0, 0, 0);
      mbar_arrive(&full_bar[slot]);
    }
    return;
  }

  if (warp == WARP_EPI) {
    // ================================================================ epilogue warp
    // Sums the consumers' partial accumulators of a finished item, applies the stage's epilogue,
    // stores the outputs and publishes the completion: one gpu-scope fence covers every item
    // finished since the previous fence.  The consumers never wait for any of this.
    int n = 0;                    // items processed
    int pend = 0;                 // completions not yet published
    int32_t* pend_ptr[NRED];
    int pend_cnt[NRED];
    unsigned idle = 0;
    while (true) {
      const int rb = n % NRED;
      const uint32_t par = (uint32_t)(n / NRED) & 1u;
      // A test that never blocks: `mbarrier.try_wait` may suspend the thread for microseconds before it
      // reports "not yet", and the completions of the items already finished would wait that long.
      const bool have = __shfl_sync(0xffffffffu, (lane == 0) ? (int)mbar_test_wait(&red_full[rb], par) : 0, 0) != 0;
      __syncwarp();  // orders the other lanes' reads after lane 0's acquire
      if (!have) {
        if (pend) {  // nothing ready: publish what is finished
          __syncwarp();
          if (lane == 0) {
            __threadfence();
#pragma unroll
            for (int i = 0; i < NRED; ++i)
              if (i < pend) atomicAdd(pend_ptr[i], pend_cnt[i]);
          }
          pend = 0;
          continue;
        }
        if ((ctl[1] && n >= ctl[2]) || *abort_flag || ++idle > spin_limit) break;
        __nanosleep(32);
        continue;
      }
      idle = 0;
      const int info_w = red_info[4 * rb + 0], q = red_info[4 * rb + 1], T = red_info[4 * rb + 2];
      const int e = info_w & 0xff, tile0 = info_w >> 8;
      const Seg* sg = reinterpret_cast<const Seg*>(descs + (size_t)e * DESC_BYTES);
      const int paired = sg->paired, epi = sg->epi, rows = sg->rows;
      const int out_stride = sg->out_stride, out_row0 = sg->out_row0;
      __nv_bfloat16* outh = sg->outh;
      __nv_bfloat16* outl = sg->outl;
      float* outf = sg->outf;
      int32_t* done = (sg->done_idx >= 0) ? P.sync + SY_DEP + sg->done_idx : nullptr;
      const float* rbuf = red + (size_t)rb * RED_FLOATS;
      // Only the real outputs are reduced: (tile a, row rr of 16, token s < T).  In the MMA D
      // fragment that element is register reg = (rr >= 8 ? 2 : 0) + (s & 1) of lane (rr % 8) * 4 +
      // (s % 8) / 2 in pass s / 8.  Consecutive lanes of this warp take consecutive rows, so the
      // stores of one token are contiguous.
      const int ntile = paired ? 1 : q;
      const int count = ntile * T * 16;
      // sigma = RMSNorm: a stage that ends in sigma stores its vector un-normalised and adds the
      // squares to the vector's sum; the stage that reads the vector scales its own result (the
      // matrix product in between is linear).  The sums are complete when the dependency counter
      // that lets the reader start is: both are published behind the same fence.
      const bool rms = L.sigma == DEAMOE_SIGMA_RMSNORM;
      const int stage = sg->stage;
      for (int x0 = 0; x0 < count; x0 += 32) {
        const int x = x0 + lane;
        const int rr = x & 15, s = (x >> 4) % T, a = x / (16 * T);
        const int p = s >> 3, reg = ((rr & 8) ? 2 : 0) + (s & 1), ln = (rr & 7) * 4 + ((s & 7) >> 1);
        const int rem = (p * 4 + reg) * 32 + ln;
        float v0 = 0.f, v1 = 0.f;
        if (x >= count) {
          // (a lane past the end only takes part in the shuffles below)
        } else if (q == 2) {
          constexpr int HW = CONSUMER_WARPS / 2;
#pragma unroll
          for (int w = 0; w < HW; ++w) {
            v0 += rbuf[(size_t)(a * HW + w) * (MAX_QP * 128) + rem];
            if (paired) v1 += rbuf[(size_t)(HW + w) * (MAX_QP * 128) + rem];
          }
        } else {
#pragma unroll
          for (int w = 0; w < CONSUMER_WARPS; ++w) v0 += rbuf[(size_t)w * (MAX_QP * 128) + rem];
        }
        const int row = tile0 * 16 + a * 16 + rr;
        const bool live = x < count && row < rows && s < T;
        if (rms && epi == EPI_SIGMA) {  // 16 consecutive lanes hold 16 rows of one token and tile
          float sq = live ? v0 * v0 : 0.f;
#pragma unroll
          for (int o = 8; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
          if ((lane & 15) == 0 && x < count && s < T) {
            if (stage == ST_S1) atomicAdd(L.ss_gu + (size_t)(out_row0 + s) * 2 + (row >= L.f ? 1 : 0), ss_fixed(sq));
            else atomicAdd(L.ss_z + (out_row0 + s), ss_fixed(sq));
          }
        }
        if (live) {
          float r;
          if (epi == EPI_SIGMA) r = sigma_f(L.sigma, v0);
          else if (epi == EPI_SWIGLU) {
            if (rms && stage == ST_S2) {  // inputs were the un-normalised G and U of this pair's row
              const unsigned long long* ss = L.ss_gu + (size_t)sg->rows16[s] * 2;
              v0 *= rms_scale_fixed(__ldcg(ss), L.f);
              v1 *= rms_scale_fixed(__ldcg(ss + 1), L.f);
            }
            r = silu_f(v0) * v1;
          } else {
            r = v0;
            if (rms && stage == ST_S4) r *= rms_scale_fixed(__ldcg(L.ss_z + sg->rows16[s]), L.f);
          }
          const size_t o = (size_t)(out_row0 + s) * out_stride + row;
          if (outf) {
            outf[o] = r;
          } else {
            const __nv_bfloat16 hi = __float2bfloat16_rn(r);
            outh[o] = hi;
            if (outl) outl[o] = __float2bfloat16_rn(r - __bfloat162float(hi));
          }
        }
      }
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(&red_empty[rb]);
        mbar_arrive(&dq_empty[e]);  // the descriptor may be reused
        ctl[3] = n + 1;             // items completed (read by the planner while it claims items)
      }
      if (done) {
#pragma unroll
        for (int i = 0; i < NRED; ++i)
          if (i == pend) { pend_ptr[i] = done; pend_cnt[i] = paired ? 1 : q; }
        ++pend;
      }
      ++n;
      if (pend == NRED) {
        __syncwarp();
        if (lane == 0) {
          __threadfence();
#pragma unroll
          for (int i = 0; i < NRED; ++i) atomicAdd(pend_ptr[i], pend_cnt[i]);
        }
        pend = 0;
      }
    }
    if (pend) {
      __syncwarp();
      if (lane == 0) {
        __threadfence();
#pragma unroll
        for (int i = 0; i < NRED; ++i)
          if (i < pend) atomicAdd(pend_ptr[i], pend_cnt[i]);
      }
    }
    return;
  }

  // ================================================================ consumers
  // Pure streaming role: wait for a chunk, multiply, release the slot.  On an item's last chunk
  // the partial accumulators go to a reduction buffer for the epilogue warp (an mbarrier
  // arrival, never a CTA barrier).
  float acc[MAX_QP][4];
  int slot = 0, items = 0;
  uint32_t phase = 0;
#ifdef DEAMOE_TRACE
  long long tr[16] = {0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0};
#endif
  const long long tc0 = TR_NOW();
  (void)tc0;
  while (true) {
    const long long tf0 = TR_NOW();
    if (!mbar_wait_warp(&full_bar[slot], phase, abort_flag, lane)) {
      if (lane == 0) { L.counts[CNT_STATUS] = DEAMOE_ERR_TIMEOUT; *abort_flag = 1; }
      break;
    }
    TR_ADD(TR_FULL, tf0);
    const long long tk0 = TR_NOW();
    const unsigned char* sbase = ring + (size_t)slot * SLOT_BYTES;
    const int4 hw = *reinterpret_cast<const int4*>(sbase);
    if (hw.x != 0) break;
    const bool first = hw.y & 1, last = hw.y & 2;
    const int q = (hw.y >> 4) & 15, planes = (hw.y >> 8) & 15, nB = (hw.y >> 12) & 15;
    const int kc = hw.z & 0xffff, T = hw.z >> 16;
    const int npass = (T + 7) >> 3;
    if (first) {
#pragma unroll
      for (int p = 0; p < MAX_QP; ++p)
#pragma unroll
        for (int x = 0; x < 4; ++x) acc[p][x] = 0.f;
    }
    TR_ADD(12, tk0);
    const long long tl0 = TR_NOW();
#ifdef DEAMOE_TRACE
    tr[14] += kc >> 4;
    if ((check_deps >> 8) != 1)
#endif
    {
      // this warp's tile and its share of the k-tiles; one specialised loop per (passes, planes)
      const int a = (q == 2) ? (warp / (CONSUMER_WARPS / 2)) : 0;
      const int kw = (q == 2) ? CONSUMER_WARPS / 2 : CONSUMER_WARPS;
      const int ks = (q == 2) ? (warp % (CONSUMER_WARPS / 2)) : warp;
      const int aw = (kc + ACT_PAD) >> 1;
      const unsigned char* wtile = sbase + SLOT_HDR + (size_t)a * kc * 32;
      const uint32_t* act = reinterpret_cast<const uint32_t*>(sbase + SLOT_HDR + (size_t)q * kc * 32) +
                            (size_t)((nB == 2) ? a : 0) * T * aw;
      const int lo = nB * T * aw;  // offset of the lo plane
#define DEAMOE_CASE(NP, PL) \
  case (NP * 4 + PL): consume_chunk<NP, PL>(acc, wtile, act, lo, kc, T, ks, kw, lane); break;
      switch (npass * 4 + planes) {
        DEAMOE_CASE(1, 1) DEAMOE_CASE(2, 1)
        DEAMOE_CASE(1, 2) DEAMOE_CASE(2, 2)
        default: break;
      }
#undef DEAMOE_CASE
    }
    TR_ADD(13, tl0);
    __syncwarp();
    if (lane == 0) mbar_arrive(&empty_bar[slot]);
    if (++slot == NSLOT) { slot = 0; phase ^= 1u; }
    TR_ADD(TR_COMPUTE, tk0);
    const long long tq0 = TR_NOW();

    if (last) {
      // hand the partial sums of this item to the epilogue warp
      const int rb = items % NRED;
      const uint32_t par = ((uint32_t)(items / NRED) & 1u) ^ 1u;
      if (!mbar_wait_warp(&red_empty[rb], par, abort_flag, lane)) {
        if (lane == 0) { L.counts[CNT_STATUS] = DEAMOE_ERR_TIMEOUT; *abort_flag = 1; }
        break;
      }
      float* mine = red + (size_t)rb * RED_FLOATS + (size_t)warp * (MAX_QP * 128);
#pragma unroll
      for (int p = 0; p < MAX_QP; ++p)
        if (p < npass) {
#pragma unroll
          for (int x = 0; x < 4; ++x) mine[(p * 4 + x) * 32 + lane] = acc[p][x];
        }
      if (tid == 0) {
        red_info[4 * rb + 0] = hw.w;
        red_info[4 * rb + 1] = q;
        red_info[4 * rb + 2] = T;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&red_full[rb]);
      ++items;
      TR_ADD(TR_EPI, tq0);
    }
  }
  if (tid == 0) {
    ctl[2] = items;
    __threadfence_block();
    ctl[1] = 1;
  }
#ifdef DEAMOE_TRACE
  tr[TR_CTOTAL] = clock64() - tc0;
  TS_MAX(L, 7);
  if (tid == 0 && P.trace)
    for (int i = 8; i < 15; ++i) P.trace[(size_t)blockIdx.x * TR_SLOTS + i] = tr[i];
#endif
}

// ---------------------------------------------------------------- host side
int stream_default_schedule() { return DEAMOE_SCHED_FUSED; }

static void fill_stage(StageCfg& s, const __nv_bfloat16* w0, const __nv_bfloat16* w1, size_t unit_elems, int C,
                       int rows, int paired, int epi) {
  s.w0 = w0; s.w1 = w1; s.unit_elems = unit_elems; s.C = C; s.rows = rows;
  s.n_tiles = (rows + 15) / 16;
  s.paired = paired;
  s.q = 2;                      // two 16-row tiles per item: (gate, up) of paired stages, else rows r, r+16
  s.epi = epi;
  s.tg = SEG_TOKENS;            // (the kernels use the constant: a run-time divisor costs a division per use)
  s.items_per_seg = paired ? s.n_tiles : (s.n_tiles + s.q - 1) / s.q;
  s.enabled = 1; s.pad = 0;
}

static size_t packed_elems(int rows, int C) { return (size_t)((rows + 15) / 16) * 16 * C; }

static cudaError_t pack(const void* src, __nv_bfloat16* dst, int rows, int C, long long rs, long long cs,
                        long long src_unit, long long dst_unit, int units, cudaStream_t s) {
  const long long per_unit = (long long)((rows + 15) / 16) * (C / 16) * 32;
  int bx = (int)((per_unit + 255) / 256);
  if (bx > 4096) bx = 4096;
  k_pack<<<dim3(bx, units), 256, 0, s>>>(reinterpret_cast<const __nv_bfloat16*>(src), dst, rows, C, rs, cs, src_unit,
                                         dst_unit, (rows + 15) / 16);
  return cudaGetLastError();
}

static cudaError_t finish_smem_attribute() {  // every instantiation may need more than the default 48 KB
  cudaError_t e = cudaSuccess;
#define DEAMOE_ATTR(T, V) if (e == cudaSuccess) e = cudaFuncSetAttribute(k_route_finish<T, V>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024)
  DEAMOE_ATTR(0, false); DEAMOE_ATTR(1, false); DEAMOE_ATTR(2, false); DEAMOE_ATTR(3, false);
  DEAMOE_ATTR(0, true); DEAMOE_ATTR(1, true); DEAMOE_ATTR(2, true); DEAMOE_ATTR(3, true);
#undef DEAMOE_ATTR
  return e;
}

deamoe_status_t stream_plan_create(const LayerDev& L, const deamoe_weights_t& w, int schedule, int dense_mode,
                                   cudaStream_t s, StreamPlan** out, uint64_t* bytes) {
  StreamPlan* p = new (std::nothrow) StreamPlan();
  if (!p) return DEAMOE_ERR_ALLOC;
  std::memset(p, 0, sizeof(*p));
  p->schedule = schedule;
  int dev = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&p->n_sm, cudaDevAttrMultiProcessorCount, dev);
  if (p->n_sm <= 0) p->n_sm = 148;
  const int m_loc = L.dept_hi - L.dept_lo, n_loc = m_loc * L.g;  // departments / experts this object holds
  const size_t units = L.vanilla ? (size_t)L.n : (size_t)m_loc;
  const size_t e_gu = packed_elems(2 * L.f, L.h);  // stacked gate;up (DeaMoE stage 1)
  const size_t e_fh = packed_elems(L.f, L.h), e_hf = packed_elems(L.h, L.f);
  const size_t e_rf = packed_elems(L.r, L.f), e_fr = packed_elems(L.f, L.r);
  const size_t e_sh = packed_elems(L.fs, L.h), e_hs = packed_elems(L.h, L.fs);
  size_t total = 0;
  size_t o_a = 0, o_b = 0, o_c = 0, o_pg = 0, o_pu = 0, o_pd = 0, o_sg = 0, o_su = 0, o_sd = 0;
  if (L.vanilla) {
    o_a = total; total += units * e_fh;  // gate
    o_b = total; total += units * e_fh;  // up
    o_c = total; total += units * e_hf;  // down^T
  } else {
    o_a = total; total += units * e_gu;
    o_c = total; total += units * e_hf;
    if (L.r > 0) {
      o_pg = total; total += (size_t)n_loc * e_rf;
      o_pu = total; total += (size_t)n_loc * e_rf;
      o_pd = total; total += (size_t)n_loc * e_fr;
    }
  }
  if (L.n_shared) {
    o_sg = total; total += e_sh;
    o_su = total; total += e_sh;
    o_sd = total; total += e_hs;
  }
  __nv_bfloat16* base = nullptr;
  if (cudaMalloc(&base, total * 2 + 16) != cudaSuccess) {
    cudaGetLastError();
    delete p;
    return DEAMOE_ERR_ALLOC;
  }
  p->packed = base;
  p->bytes = total * 2 + 16;
  p->dev.packed_lo = base;
  p->dev.packed_elems = total;
  cudaError_t e = cudaSuccess;
  auto P = [&](const void* src, size_t off, int rows, int C, long long rs, long long cs, long long su, long long du,
               int nu) {
    if (e == cudaSuccess) e = pack(src, base + off, rows, C, rs, cs, su, du, nu, s);
  };
  StreamDev& d = p->dev;
  const long long fh = (long long)L.f * L.h, rf = (long long)L.r * L.f;
  if (L.vanilla) {
    P(w.dept_gate, o_a, L.f, L.h, L.h, 1, fh, (long long)e_fh, (int)units);
    P(w.dept_up, o_b, L.f, L.h, L.h, 1, fh, (long long)e_fh, (int)units);
    P(w.dept_down, o_c, L.h, L.f, 1, L.h, fh, (long long)e_hf, (int)units);
    fill_stage(d.st[ST_V1], base + o_a, base + o_b, e_fh, L.h, L.f, 1, EPI_SWIGLU);
    fill_stage(d.st[ST_V2], base + o_c, nullptr, e_hf, L.f, L.h, 0, EPI_NONE);
  } else {
    P(w.dept_gate, o_a, L.f, L.h, L.h, 1, fh, (long long)e_gu, (int)units);
    P(w.dept_up, o_a + (size_t)L.f * L.h, L.f, L.h, L.h, 1, fh, (long long)e_gu, (int)units);
    P(w.dept_down, o_c, L.h, L.f, 1, L.h, fh, (long long)e_hf, (int)units);
    fill_stage(d.st[ST_S1], base + o_a, nullptr, e_gu, L.h, 2 * L.f, 0, EPI_SIGMA);
    fill_stage(d.st[ST_S4], base + o_c, nullptr, e_hf, L.f, L.h, 0, EPI_NONE);
    if (L.r > 0) {
      P(w.priv_gate, o_pg, L.r, L.f, L.f, 1, rf, (long long)e_rf, n_loc);
      P(w.priv_up, o_pu, L.r, L.f, L.f, 1, rf, (long long)e_rf, n_loc);
      P(w.priv_down, o_pd, L.f, L.r, 1, L.f, rf, (long long)e_fr, n_loc);
      fill_stage(d.st[ST_S2], base + o_pg, base + o_pu, e_rf, L.f, L.r, 1, EPI_SWIGLU);
      fill_stage(d.st[ST_S3], base + o_pd, nullptr, e_fr, L.r, L.f, 0, EPI_SIGMA);
    }
  }
  if (L.n_shared) {
    P(w.shared_gate, o_sg, L.fs, L.h, L.h, 1, 0, 0, 1);
    P(w.shared_up, o_su, L.fs, L.h, L.h, 1, 0, 0, 1);
    P(w.shared_down, o_sd, L.h, L.fs, 1, L.h, 0, 0, 1);
    fill_stage(d.st[ST_SH1], base + o_sg, base + o_su, e_sh, L.h, L.fs, 1, EPI_SWIGLU);
    fill_stage(d.st[ST_SH2], base + o_sd, nullptr, e_hs, L.fs, L.h, 0, EPI_NONE);
  }
  // work-list storage
  const int MB = L.max_batch;
  d.max_segs = 8 + 2 * L.m + 2 * L.n + MB * L.k + 2 * MB;
  d.dep_s1 = 0; d.dep_s2 = L.m; d.dep_s3 = L.m + L.n; d.dep_sh1 = 2 * L.m + L.n; d.n_dep = 2 * L.m + L.n + 1;
  // Fused schedule: the shared expert's items run before the routing kernel has finished, which
  // zeroes counters [0, n_dep); theirs is the first counter after that range, and the combine
  // kernel, the last of a step, resets it.
  d.sh_prefix = (schedule == DEAMOE_SCHED_FUSED && L.n_shared && (L.vanilla || L.r > 0)) ? 1 : 0;
  if (d.sh_prefix) d.dep_sh1 = d.n_dep;
  d.early = (schedule == DEAMOE_SCHED_FUSED && (L.vanilla || L.r > 0) && (!L.n_shared || d.sh_prefix)) ? 1 : 0;
  d.early_stage = L.vanilla ? ST_V1 : ST_S1;
  d.claim_items = (schedule == DEAMOE_SCHED_FUSED && (L.vanilla || L.r > 0)) ? 1 : 0;
  d.early_flag = d.n_dep + 1; d.early_items = d.n_dep + 2;  // the allocation has 8 spare counters
  d.planes = (L.adt == DEAMOE_F32) ? 2 : 1;
  d.spin_limit = SPIN_LIMIT; d.withhold = 0;
  {
    // activation planes between stages
    const size_t tdmax = (size_t)MB * (L.k < L.m ? L.k : L.m), pmax = (size_t)MB * L.k;
    struct { __nv_bfloat16** h; __nv_bfloat16** l; size_t elems; } bufs[] = {
        {&d.xh, &d.xl, L.adt == DEAMOE_F32 ? (size_t)MB * L.h : 0},
        {&d.GUh, &d.GUl, L.vanilla ? 0 : tdmax * 2 * L.f},
        {&d.Yh, &d.Yl, pmax * (size_t)(L.vanilla ? L.f : L.rp)},
        {&d.Zh, &d.Zl, L.vanilla ? 0 : pmax * (size_t)L.f},
        {&d.Yshh, &d.Yshl, L.n_shared ? (size_t)MB * L.fs : 0},
    };
    for (auto& b : bufs) {
      if (!b.elems) continue;
      if (e == cudaSuccess) e = cudaMalloc(b.h, b.elems * 2);
      if (e == cudaSuccess && d.planes > 1) e = cudaMalloc(b.l, b.elems * 2);
      p->bytes += b.elems * 2 * d.planes;
    }
  }
  const size_t seg_bytes = (size_t)d.max_segs * sizeof(Seg);
  const size_t sync_bytes = (size_t)(SY_DEP + d.n_dep + 8) * sizeof(int32_t);
  if (e == cudaSuccess) e = cudaMalloc(&d.segs, seg_bytes);
  if (e == cudaSuccess) e = cudaMalloc(&d.sync, sync_bytes);
#ifdef DEAMOE_TRACE
  if (e == cudaSuccess) e = cudaMalloc(&d.trace, (size_t)p->n_sm * CTAS_PER_SM * TR_SLOTS * sizeof(long long));
  if (e == cudaSuccess) e = cudaMemsetAsync(d.trace, 0, (size_t)p->n_sm * CTAS_PER_SM * TR_SLOTS * sizeof(long long), s);
#endif
  if (e == cudaSuccess) e = cudaMemsetAsync(d.sync, 0, sync_bytes, s);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(k_stream, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)STREAM_SMEM);
  if (e == cudaSuccess) {
    // The CTAs wait on one another's results, so the grid may hold only as many as fit on the
    // device at once: the occupancy the runtime reports, at most CTAS_PER_SM per SM.
    int occ = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, k_stream, STREAM_THREADS, STREAM_SMEM);
    if (e == cudaSuccess && occ < 1) e = cudaErrorLaunchOutOfResources;
    const int per_sm = occ < CTAS_PER_SM ? occ : CTAS_PER_SM;
    p->grid = p->n_sm * per_sm;
    // Fused schedule: the routing tail (one CTA that fills an SM's register file) is still running
    // when this grid starts, and the CTAs that would share its SM could only start when it exits,
    // tens of microseconds after the others, and would finish the step that much later.  The
    // grid leaves that SM out (the stream is bound by HBM, not by the number of SMs).
    if (schedule == DEAMOE_SCHED_FUSED && p->n_sm > 1) p->grid -= per_sm;
  }
  if (e == cudaSuccess)
    e = finish_smem_attribute();
  p->bytes += seg_bytes + sync_bytes;
  if (e != cudaSuccess) {
    cudaGetLastError();
    stream_plan_destroy(p);
    return e == cudaErrorMemoryAllocation ? DEAMOE_ERR_ALLOC : DEAMOE_ERR_CUDA;
  }
  // Dense schedule: always (dense_mode 2) or from DENSE_MIN_BATCH tokens on (dense_mode 1, layers
  // that can be called with that many).  Its routing and its streaming launch see the plan with
  // the fused schedule's hand-overs switched off and the private stages as the whole list.
  p->dense_min = dense_mode == 2 ? 1 : (L.n >= DENSE_SMALL_ROUTER ? DENSE_MIN_BATCH : 2 * DENSE_MIN_BATCH);
  if (dense_mode == 2 || (dense_mode == 1 && dense_supported(L) && L.max_batch >= p->dense_min)) {
    uint64_t db = 0;
    const deamoe_status_t ds = dense_plan_create(L, w, s, &p->dense, &db);
    if (ds != DEAMOE_OK) {
      stream_plan_destroy(p);
      return ds;
    }
    p->bytes += db;
    p->dev_dense = p->dev;
    p->dev_dense.dense = 1;
    p->dev_dense.early = 0; p->dev_dense.sh_prefix = 0;  // (items of the second private stage are still claimed)
  }
  *out = p;
  *bytes = p->bytes;
  return DEAMOE_OK;
}

void stream_plan_destroy(StreamPlan* p) {
  if (!p) return;
  stream_profile_enable(*p, false);
  if (p->packed) cudaFree(p->packed);
  if (p->dense) dense_plan_destroy(p->dense);
  if (p->dev.segs) cudaFree(p->dev.segs);
  if (p->dev.sync) cudaFree(p->dev.sync);
  if (p->dev.trace) cudaFree(p->dev.trace);
  __nv_bfloat16* planes[] = {p->dev.xh, p->dev.xl, p->dev.GUh, p->dev.GUl, p->dev.Yh, p->dev.Yl,
                             p->dev.Zh, p->dev.Zl, p->dev.Yshh, p->dev.Yshl};
  for (__nv_bfloat16* q : planes)
    if (q) cudaFree(q);
  delete p;
}

int32_t* stream_shared_counter(StreamPlan& p) {
  return p.dev.sh_prefix ? p.dev.sync + SY_DEP + p.dev.dep_sh1 : nullptr;
}

static bool takes_dense(const StreamPlan& p, int B) { return p.dense && B >= p.dense_min; }

int stream_route(StreamPlan& p, const LayerDev& L, const void* tokens, int B, cudaStream_t s, int kslices,
                 int32_t* user_idx, float* user_w) {
  const StreamDev& dv = takes_dense(p, B) ? p.dev_dense : p.dev;
  const int ny = launch_router_logits(L, tokens, B, s, kslices,
                                      (dv.early || dv.dense) ? dv.sync + SY_DEP + dv.early_flag : nullptr);
  if (ny < 0) return -1;
  const int per_warp = (L.n * 5 + 15) & ~15;
  const bool in_regs = topk_in_registers(L);
  int topk_warps = in_regs ? FINISH_THREADS / 32 : (48 * 1024) / per_warp;
  if (topk_warps > FINISH_THREADS / 32) topk_warps = FINISH_THREADS / 32;
  if (topk_warps > B) topk_warps = B;
  if (topk_warps < 1) topk_warps = 1;
  int extra = 0;
  if (topk_wide_fits(L)) {  // wide router: the selection by one CTA per token, in a grid of its own
    launch_pdl(k_topk_wide, dim3(B), dim3(((L.n + 255) / 256) * 32), 0, s, L, B, ny, user_idx, user_w);
    topk_warps = 0;
    extra = 1;
  } else if ((takes_dense(p, B) || B > FINISH_THREADS / 32 || L.n > 256) && in_regs) {  // the selection gets a grid of its own
    launch_pdl(k_topk_tokens, dim3((B + TOPK_CTA_WARPS - 1) / TOPK_CTA_WARPS), dim3(TOPK_CTA_WARPS * 32), 0, s, L, B, ny,
               user_idx, user_w);
    topk_warps = 0;
    extra = 1;
  }
  size_t scratch = (in_regs || topk_warps == 0) ? 0 : (size_t)topk_warps * per_warp;   // top-k scratch, reused by the bucketing masks
  const size_t bs = bucket_smem_bytes(L, B) + (size_t)((L.vanilla ? L.n : L.m) + 2) * sizeof(int);  // + early_first_stage()'s scan
  if (bs > scratch) scratch = bs;
  scratch = (scratch + 15) & ~(size_t)15;
  const FinishSmem fl = finish_layout(L.n, L.m, L.k, B);
  const size_t smem = scratch + (size_t)fl.total * 4;
  if (smem > 200 * 1024) return -1;
  const bool plain_router = !(L.k_dept > 0 && L.k_dept < L.m) && !(L.strict_dept && L.k_dept > 0) && L.norm_topk != 0;
  const int mode = topk_warps == 0 ? 0 : ((in_regs && L.n <= 256) ? (plain_router ? 3 : 1) : 2);
#define DEAMOE_FINISH(T, V) launch_pdl(k_route_finish<T, V>, dim3(1), dim3(FINISH_THREADS), smem, s, L, dv, B, ny, topk_warps, \
                                       (int)(scratch / 4), user_idx, user_w)
  if (L.vanilla) {
    if (mode == 0) DEAMOE_FINISH(0, true); else if (mode == 1) DEAMOE_FINISH(1, true); else if (mode == 2) DEAMOE_FINISH(2, true);
    else DEAMOE_FINISH(3, true);
  } else {
    if (mode == 0) DEAMOE_FINISH(0, false); else if (mode == 1) DEAMOE_FINISH(1, false); else if (mode == 2) DEAMOE_FINISH(2, false);
    else DEAMOE_FINISH(3, false);
  }
#undef DEAMOE_FINISH
  return cudaGetLastError() == cudaSuccess ? 2 + extra : -1;
}

// category order as built by category_list(), host copy
static int host_categories(const LayerDev& L, int* stages) {
  int n = 0;
  if (L.n_shared) stages[n++] = ST_SH1;
  if (L.vanilla) {
    stages[n++] = ST_V1;
    if (L.n_shared) stages[n++] = ST_SH2;
    stages[n++] = ST_V2;
  } else {
    stages[n++] = ST_S1;
    if (L.n_shared) stages[n++] = ST_SH2;
    if (L.r > 0) { stages[n++] = ST_S2; stages[n++] = ST_S3; }
    stages[n++] = ST_S4;
  }
  return n;
}

__global__ void k_identity_private(LayerDev L, StreamDev P);  // defined below
__global__ void k_split_tokens(const float* x, __nv_bfloat16* xh, __nv_bfloat16* xl, size_t count);

int stream_forward(StreamPlan& p, const LayerDev& L, int B, cudaStream_t s) {
  int stages[MAX_CAT];
  const int ncat = host_categories(L, stages);
  int launches = 0;
  if (p.ev0) cudaEventRecord(p.ev0, s);
  if (L.adt == DEAMOE_F32) {
    const size_t count = (size_t)B * L.h;
    int blocks = (int)((count + 255) / 256);
    if (blocks > 4 * p.n_sm) blocks = 4 * p.n_sm;
    k_split_tokens<<<blocks, 256, 0, s>>>(L.x32, p.dev.xh, p.dev.xl, count);
    ++launches;
  }
  const bool fused = p.schedule == DEAMOE_SCHED_FUSED && (L.vanilla || L.r > 0);
  if (takes_dense(p, B)) {
    // department gate / up (+ shared expert gate / up) on the tensor cores; the private stages in
    // the streaming kernel; department down (+ shared expert down) on the tensor cores
    DenseIO io;
    io.tokens = reinterpret_cast<const __nv_bfloat16*>(L.tokens_raw);
    io.GU = p.dev.GUh; io.Z = p.dev.Zh; io.Ysh = p.dev.Yshh;
    io.s1_done = p.dev.sync + SY_DEP + p.dev.dep_s1;
    io.routed_flag = p.dev.sync + SY_DEP + p.dev.early_flag;
    io.gathered = p.dev.sync + SY_DEP + p.dev.early_flag + 3;  // cleared by the step's router kernel, like the flags
    io.spin_limit = p.dev_dense.spin_limit;
    // (the shared expert's tiles first: every token passes through them, which makes them the longest jobs, and
    // jobs claimed from a counter finish closest together when the longest are claimed first)
    const int first[2] = {ST_SH1, ST_S1}, last[2] = {ST_SH2, ST_S4};
    const int o = L.n_shared ? 0 : 1;
    const int n1 = dense_launch(*p.dense, L, io, first + o, 2 - o, B, s);
    if (n1 < 0) return -1;
    // resident as soon as the tensor-core kernel's CTAs leave room; an expert's items wait for its department's rows
    launch_pdl(k_stream, dim3(p.grid), dim3(STREAM_THREADS), STREAM_SMEM, s, L, p.dev_dense, B, -1, 1 | 16);
    const int n2 = dense_launch(*p.dense, L, io, last + o, 2 - o, B, s);
    if (n2 < 0) return -1;
    launches += n1 + 1 + n2;
  } else if (fused) {
    int dbgflag = 0;
#ifdef DEAMOE_TRACE
    if (const char* ev = getenv("DEAMOE_DBG")) dbgflag = atoi(ev) << 8;
#endif
    // expected share of active departments under uniform routing: prefetch when it is at least 0.65
    // (measured on the DeepSeek-V3 shape: a gain from 4 tokens on, share 0.68; a loss at 2, share 0.44)
    int pf = 0;
    {
      const int units = L.vanilla ? L.n : L.m;  // the first stage's units: experts (vanilla) or departments
      const int c = L.vanilla ? L.k : ((L.k_dept > 0 && L.k_dept < L.m) ? L.k_dept : (L.k < L.m ? L.k : L.m));
      double miss = 1.0;
      for (int t = 0; t < B; ++t) miss *= 1.0 - (double)c / units;
      pf = (miss <= 0.35) ? 4 : 0;
    }
    launch_pdl(k_stream, dim3(p.grid), dim3(STREAM_THREADS), STREAM_SMEM, s, L, p.dev, B, -1, 1 | pf | dbgflag);
    ++launches;
  } else {
    for (int c = 0; c < ncat; ++c) {
      if (stages[c] == ST_S4 && !L.vanilla && L.r == 0) {
        k_identity_private<<<p.n_sm, 256, 0, s>>>(L, p.dev);
        ++launches;
      }
      k_stream<<<p.grid, STREAM_THREADS, STREAM_SMEM, s>>>(L, p.dev, B, c, 0);
      ++launches;
    }
  }
  if (p.ev1) { cudaEventRecord(p.ev1, s); p.ev_recorded = 1; }
  return cudaGetLastError() == cudaSuccess ? launches : -1;
}

// Failure tests: lower the poll limit of every bounded wait and / or withhold a hand-over.
// spin_limit 0 restores the default.  Returns false if the plan cannot honour `withhold`.
bool stream_set_failure_test(StreamPlan& p, unsigned spin_limit, int withhold) {
  if ((withhold & 1) && !p.dev.early) return false;   // only the fused schedule hands over through flags
  if ((withhold & 2) && !p.dense) return false;
  const unsigned lim = spin_limit ? spin_limit : SPIN_LIMIT;
  p.dev.spin_limit = lim; p.dev.withhold = withhold & 5;
  p.dev_dense.spin_limit = lim; p.dev_dense.withhold = withhold & 4;
  if (p.dense) dense_set_failure_test(*p.dense, spin_limit, (withhold & 2) ? 1 : 0);
  return true;
}

cudaError_t stream_profile_enable(StreamPlan& p, bool on) {
  if (on && !p.ev0) {
    cudaError_t e = cudaEventCreate(&p.ev0);
    if (e == cudaSuccess) e = cudaEventCreate(&p.ev1);
    p.ev_recorded = 0;
    return e;
  }
  if (!on && p.ev0) {
    cudaEventDestroy(p.ev0); cudaEventDestroy(p.ev1);
    p.ev0 = nullptr; p.ev1 = nullptr; p.ev_recorded = 0;
  }
  return cudaSuccess;
}

cudaError_t stream_profile_last_ms(StreamPlan& p, float* ms) {
  if (!p.ev0 || !p.ev_recorded) return cudaErrorInvalidValue;
  cudaError_t e = cudaEventSynchronize(p.ev1);
  if (e == cudaSuccess) e = cudaEventElapsedTime(ms, p.ev0, p.ev1);
  return e;
}

// priv == 0: A = identity, so Y = SiLU(G) * U and Z = sigma(Y) element by element.
__global__ void k_identity_private(LayerDev L, StreamDev P) {
  const int pairs = L.counts[CNT_PAIRS];
  const size_t total = (size_t)pairs * L.f;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    const int pr = (int)(i / L.f), c = (int)(i % L.f);
    const size_t o = (size_t)L.pair_gurow[pr] * 2 * L.f + c;
    float gv = __bfloat162float(P.GUh[o]), uv = __bfloat162float(P.GUh[o + L.f]);
    if (P.planes > 1) {
      gv += __bfloat162float(P.GUl[o]);
      uv += __bfloat162float(P.GUl[o + L.f]);
    }
    const float z = sigma_f(L.sigma, silu_f(gv) * uv);
    const __nv_bfloat16 hi = __float2bfloat16_rn(z);
    P.Zh[i] = hi;
    if (P.planes > 1) P.Zl[i] = __float2bfloat16_rn(z - __bfloat162float(hi));
  }
}

// fp32 tokens -> bf16 hi + lo planes (x = hi + lo up to ~2^-17 relative)
__global__ void k_split_tokens(const float* __restrict__ x, __nv_bfloat16* __restrict__ xh,
                               __nv_bfloat16* __restrict__ xl, size_t count) {
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (size_t)gridDim.x * blockDim.x) {
    const float v = x[i];
    const __nv_bfloat16 hi = __float2bfloat16_rn(v);
    xh[i] = hi;
    xl[i] = __float2bfloat16_rn(v - __bfloat162float(hi));
  }
}

}  // namespace deamoe

#ifdef DEAMOE_TRACE
// Trace builds only: copy the per-CTA cycle counters of the last k_stream launch to the host.
namespace deamoe {
int stream_read_trace(StreamPlan& p, long long* host, int max_ctas) {
  const int n = p.grid < max_ctas ? p.grid : max_ctas;
  cudaDeviceSynchronize();
  cudaMemcpy(host, p.dev.trace, (size_t)n * TR_SLOTS * sizeof(long long), cudaMemcpyDeviceToHost);
  return n;
}
}  // namespace deamoe
#endif
