// Weight-streaming schedules for bf16 layers.
//
// Every stage of Section 3.2 (department gate/up, private gate/up, private down, department
// down, and the shared / vanilla experts of Eq. (1)) is the same operation: a few token rows
// times a weight matrix that is read exactly once.  At create the matrices are re-packed so
// that one 16-row tile of a matrix is a contiguous stream whose 512-byte pieces are the
// per-lane A fragments of mma.sync.m16n8k16.  One persistent kernel then works through a
// device-built list of items (one or two 16-row tiles x the full contraction length):
//
//   producer warp   : claims items, waits (bounded) until the item's inputs exist, and moves
//                     weight chunks (HBM) and the matching activation chunks (L2) into a
//                     shared-memory ring with cp.async.bulk, completion on mbarriers;
//   8 consumer warps: split each chunk's k-tiles, build bf16 hi/lo B fragments from the fp32
//                     activations (products keep ~16 mantissa bits), accumulate in fp32 with
//                     mma.sync, and on the item's last chunk reduce across warps, apply the
//                     stage's epilogue and signal completion.
//
// Weights never depend on earlier stages, so the ring keeps the HBM pipe full across item and
// stage boundaries; only the (tiny) activations wait for their producers.
#include <cstring>
#include <new>

#include "stream.cuh"

namespace deamoe {

constexpr int CONSUMER_WARPS = 8;
constexpr int CONSUMER_THREADS = CONSUMER_WARPS * 32;
constexpr int STREAM_THREADS = CONSUMER_THREADS + 32;
constexpr int SLOT_BYTES = 32 * 1024;
constexpr int SLOT_HDR = 128;
constexpr int NSLOT = 6;
constexpr int ACT_PAD = 8;   // floats of padding per activation row in shared memory
constexpr int MAX_QP = 4;    // (tiles per item) x (8-token passes) held in accumulators
constexpr int RED_FLOATS = CONSUMER_WARPS * MAX_QP * 128;
constexpr size_t STREAM_SMEM = (size_t)NSLOT * SLOT_BYTES + (size_t)RED_FLOATS * 4 + 256;
constexpr unsigned SPIN_LIMIT = 1u << 24;  // bounded waits; then an error status, never a hang
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
  int in_stride, in_row0, out_stride, out_row0;
  int dep_idx, dep_target, done_idx, use_lo;
  const __nv_bfloat16* w0;
  const __nv_bfloat16* w1;
  const float* in0;
  const float* in1;
  const int32_t* in_rows;
  float* out;
};

struct StreamDev {
  StageCfg st[ST_COUNT];
  Seg* segs;
  int32_t* sync;
  int max_segs;
  int dep_s1, dep_s2, dep_s3, dep_sh1, n_dep;  // offsets relative to SY_DEP
};

struct StreamPlan {
  StreamDev dev;
  int schedule;
  int n_sm;
  void* packed;
  uint64_t bytes;
};

// chunk header written by the producer at the start of a ring slot
struct SlotHdr {
  int kind;  // 0 data, 1 end of work
  int first, last, kc;
  int T, q, paired, nB;
  int epi, use_lo, row0, rows;
  int out_stride, out_row0, npass, pad;
  float* out;
  int32_t* done;
};
static_assert(sizeof(SlotHdr) <= SLOT_HDR, "slot header too large");

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
static __device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  for (unsigned it = 0; it < SPIN_LIMIT; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 1023u) == 1023u && *abort_flag) return false;
  }
  return false;
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
static __device__ __forceinline__ int ld_acquire(const int32_t* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
static __device__ __forceinline__ void consumer_sync() {
  asm volatile("bar.sync 1, %0;" ::"n"(CONSUMER_THREADS) : "memory");
}
static __device__ __forceinline__ void mma_bf16(float (&d)[4], const uint4& a, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a.x), "r"(a.y), "r"(a.z), "r"(a.w), "r"(b0), "r"(b1));
}
// two fp32 -> packed bf16 pair (first value in the low half) and the rounding remainders
static __device__ __forceinline__ uint32_t pack_hi(float x, float y, float& rx, float& ry) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(x, y);
  rx = x - __bfloat162float(h.x);
  ry = y - __bfloat162float(h.y);
  return *reinterpret_cast<const uint32_t*>(&h);
}
static __device__ __forceinline__ uint32_t pack_bf(float x, float y) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(x, y);
  return *reinterpret_cast<const uint32_t*>(&h);
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
  if (L.n_shared) cats[n++] = {ST_SH1, 0};
  if (L.vanilla) {
    cats[n++] = {ST_V1, 2};
    if (L.n_shared) cats[n++] = {ST_SH2, 0};
    cats[n++] = {ST_V2, 2};
  } else {
    cats[n++] = {ST_S1, 1};
    if (L.n_shared) cats[n++] = {ST_SH2, 0};
    if (L.r > 0) {
      cats[n++] = {ST_S2, 2};
      cats[n++] = {ST_S3, 2};
    }
    cats[n++] = {ST_S4, 1};
  }
  (void)P;
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

static __device__ __forceinline__ int chunk_k(int C, int q, int nB, int T) {
  const int avail = SLOT_BYTES - SLOT_HDR - nB * T * ACT_PAD * 4;
  int kc = avail / (q * 32 + nB * T * 4);
  if (kc > C) kc = C;
  kc = (kc >= 128) ? (kc & ~127) : (kc & ~15);
  return kc;
}

static __device__ void write_seg(const LayerDev& L, const StreamDev& P, int stage, int id, int gi, int B,
                                 int seg_index, int item0) {
  const StageCfg& sc = P.st[stage];
  const int Tall = unit_tokens(L, stage, id, B);
  const int t0 = gi * sc.tg;
  Seg s;
  s.item0 = item0; s.n_items = sc.items_per_seg; s.stage = stage; s.epi = sc.epi;
  s.T = min(sc.tg, Tall - t0); s.q = sc.q; s.paired = sc.paired; s.nB = 1;
  s.C = sc.C; s.rows = sc.rows; s.n_tiles = sc.n_tiles;
  s.w0 = sc.w0 + (size_t)id * sc.unit_elems;
  s.w1 = sc.w1 ? sc.w1 + (size_t)id * sc.unit_elems : nullptr;
  s.in1 = nullptr; s.in_rows = nullptr; s.in_row0 = 0;
  s.dep_idx = -1; s.dep_target = 0; s.done_idx = -1;
  s.use_lo = 1;
  const int j = (stage == ST_S2 || stage == ST_S3) ? id / L.g : id;
  switch (stage) {
    case ST_S1:
      s.in0 = L.x32; s.in_stride = L.h; s.in_rows = L.dept_tok + L.dept_off[id] + t0;
      s.out = L.GU; s.out_stride = 2 * L.f; s.out_row0 = L.dept_off[id] + t0;
      s.done_idx = P.dep_s1 + id; s.use_lo = (L.adt == DEAMOE_F32);
      break;
    case ST_S2:
      s.in0 = L.GU; s.in1 = L.GU + L.f; s.nB = 2; s.in_stride = 2 * L.f;
      s.in_rows = L.pair_gurow + L.expert_off[id] + t0;
      s.out = L.Y; s.out_stride = L.rp; s.out_row0 = L.expert_off[id] + t0;
      s.dep_idx = P.dep_s1 + j;
      s.dep_target = groups_of(unit_tokens(L, ST_S1, j, B), P.st[ST_S1].tg) * P.st[ST_S1].items_per_seg;
      s.done_idx = P.dep_s2 + id;
      break;
    case ST_S3:
      s.in0 = L.Y; s.in_stride = L.rp; s.in_row0 = L.expert_off[id] + t0;
      s.out = L.Z; s.out_stride = L.f; s.out_row0 = L.expert_off[id] + t0;
      s.dep_idx = P.dep_s2 + id;
      s.dep_target = groups_of(Tall, P.st[ST_S2].tg) * P.st[ST_S2].items_per_seg;
      s.done_idx = P.dep_s3 + j;
      break;
    case ST_S4: {
      const int p0 = L.expert_off[id * L.g];
      s.in0 = L.Z; s.in_stride = L.f; s.in_row0 = p0 + t0;
      s.out = L.O; s.out_stride = L.h; s.out_row0 = p0 + t0;
      if (L.r > 0) {
        int target = 0;
        for (int e = 0; e < L.g; ++e) {
          const int Te = L.expert_off[id * L.g + e + 1] - L.expert_off[id * L.g + e];
          target += groups_of(Te, P.st[ST_S3].tg) * P.st[ST_S3].items_per_seg;
        }
        s.dep_idx = P.dep_s3 + id; s.dep_target = target;
      }
      break;
    }
    case ST_SH1:
      s.in0 = L.x32; s.in_stride = L.h; s.in_row0 = t0;
      s.out = L.Ysh; s.out_stride = L.fs; s.out_row0 = t0;
      s.done_idx = P.dep_sh1; s.use_lo = (L.adt == DEAMOE_F32);
      break;
    case ST_SH2:
      s.in0 = L.Ysh; s.in_stride = L.fs; s.in_row0 = t0;
      s.out = L.Osh; s.out_stride = L.h; s.out_row0 = t0;
      s.dep_idx = P.dep_sh1;
      s.dep_target = groups_of(B, P.st[ST_SH1].tg) * P.st[ST_SH1].items_per_seg;
      break;
    case ST_V1:
      s.in0 = L.x32; s.in_stride = L.h; s.in_rows = L.expert_tok + L.expert_off[id] + t0;
      s.out = L.Y; s.out_stride = L.f; s.out_row0 = L.expert_off[id] + t0;
      s.done_idx = P.dep_s2 + id; s.use_lo = (L.adt == DEAMOE_F32);
      break;
    case ST_V2:
      s.in0 = L.Y; s.in_stride = L.f; s.in_row0 = L.expert_off[id] + t0;
      s.out = L.O; s.out_stride = L.h; s.out_row0 = L.expert_off[id] + t0;
      s.dep_idx = P.dep_s2 + id;
      s.dep_target = groups_of(Tall, P.st[ST_V1].tg) * P.st[ST_V1].items_per_seg;
      break;
  }
  s.kc = chunk_k(s.C, s.q, s.nB, s.T);
  if (seg_index < P.max_segs) P.segs[seg_index] = s;
}

constexpr int BUILD_THREADS = 32 * MAX_CAT;

__global__ void __launch_bounds__(BUILD_THREADS) k_build_worklist(LayerDev L, StreamDev P, int B) {
  __shared__ int s_nseg[MAX_CAT], s_segbase[MAX_CAT + 1], s_itembase[MAX_CAT + 1];
  CatInfo cats[MAX_CAT];
  const int ncat = category_list(L, P, cats);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int i = threadIdx.x; i < P.n_dep + MAX_CAT + 8; i += BUILD_THREADS) P.sync[SY_CLAIM + i] = 0;
  if (warp < ncat) {
    const int stage = cats[warp].stage, kind = cats[warp].unit_kind;
    const int U = unit_count(L, kind);
    int cnt = 0;
    for (int u = lane; u < U; u += 32)
      cnt += groups_of(unit_tokens(L, stage, unit_id(L, kind, u), B), P.st[stage].tg);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
    if (lane == 0) s_nseg[warp] = cnt;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int sb = 0, ib = 0;
    for (int c = 0; c < ncat; ++c) {
      s_segbase[c] = sb; s_itembase[c] = ib;
      const int ips = P.st[cats[c].stage].items_per_seg;
      P.sync[SY_CAT + 4 * c + 0] = ib;
      P.sync[SY_CAT + 4 * c + 1] = sb;
      P.sync[SY_CAT + 4 * c + 2] = ips;
      P.sync[SY_CAT + 4 * c + 3] = cats[c].stage;
      sb += s_nseg[c];
      ib += s_nseg[c] * ips;
    }
    s_segbase[ncat] = sb; s_itembase[ncat] = ib;
    for (int c = ncat; c < MAX_CAT; ++c) {
      P.sync[SY_CAT + 4 * c + 0] = ib;
      P.sync[SY_CAT + 4 * c + 1] = sb;
      P.sync[SY_CAT + 4 * c + 2] = 1;
      P.sync[SY_CAT + 4 * c + 3] = -1;
    }
    P.sync[SY_NCAT] = ncat; P.sync[SY_NSEG] = sb; P.sync[SY_NITEMS] = ib;
    L.counts[CNT_NSEG] = sb; L.counts[CNT_NITEMS] = ib;
    if (sb > P.max_segs) L.counts[CNT_STATUS] = DEAMOE_ERR_UNSUPPORTED;
  }
  __syncthreads();
  if (warp < ncat) {
    const int stage = cats[warp].stage, kind = cats[warp].unit_kind;
    const int U = unit_count(L, kind);
    const int ips = P.st[stage].items_per_seg;
    int running = 0;
    for (int base = 0; base < U; base += 32) {
      const int u = base + lane;
      const int id = (u < U) ? unit_id(L, kind, u) : 0;
      const int gc = (u < U) ? groups_of(unit_tokens(L, stage, id, B), P.st[stage].tg) : 0;
      int incl = gc;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
      }
      const int first = running + incl - gc;
      for (int gi = 0; gi < gc; ++gi) {
        const int si = s_segbase[warp] + first + gi;
        write_seg(L, P, stage, id, gi, B, si, s_itembase[warp] + (first + gi) * ips);
      }
      running += __shfl_sync(0xffffffffu, incl, 31);
    }
  }
}

// ---------------------------------------------------------------- the streaming kernel
struct __align__(16) ItemCtx {  // producer-side view of one claimed item
  int seg, item_in_seg;
};

__global__ void __launch_bounds__(STREAM_THREADS, 1)
k_stream(LayerDev L, StreamDev P, int launch_id, int cat, int check_deps) {
  extern __shared__ __align__(128) unsigned char smem[];
  unsigned char* ring = smem;
  float* red = reinterpret_cast<float*>(smem + (size_t)NSLOT * SLOT_BYTES);
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + (size_t)NSLOT * SLOT_BYTES + (size_t)RED_FLOATS * 4);
  uint64_t* empty_bar = full_bar + NSLOT;
  volatile int* abort_flag = reinterpret_cast<volatile int*>(empty_bar + NSLOT);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    for (int s = 0; s < NSLOT; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], CONSUMER_WARPS);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  // item range of this launch: one category (staged) or everything (fused)
  const int32_t* sy = P.sync;
  const int item_begin = (cat >= 0) ? sy[SY_CAT + 4 * cat + 0] : 0;
  const int item_end = (cat >= 0) ? sy[SY_CAT + 4 * (cat + 1) + 0] : sy[SY_NITEMS];
  const int ncat = sy[SY_NCAT];

  if (warp == CONSUMER_WARPS) {
    // ================================================================ producer
    const uint64_t pol = policy_evict_first();
    int slot = 0;
    uint32_t phase = 0;
    bool ok = true;
    int32_t* claim = P.sync + SY_CLAIM + launch_id;
    while (ok) {
      int item = 0;
      if (lane == 0) item = item_begin + atomicAdd(claim, 1);
      item = __shfl_sync(0xffffffffu, item, 0);
      if (item >= item_end) break;
      // category -> segment -> item within the segment
      int c = 0;
      for (int q = 1; q < ncat; ++q)
        if (item >= sy[SY_CAT + 4 * q + 0]) c = q;
      const int ib = sy[SY_CAT + 4 * c + 0], sb = sy[SY_CAT + 4 * c + 1], ips = sy[SY_CAT + 4 * c + 2];
      const Seg* sg = P.segs + sb + (item - ib) / ips;
      const int it = (item - ib) % ips;
      const int T = sg->T, q = sg->q, paired = sg->paired, nB = sg->nB, kc0 = sg->kc, C = sg->C;
      const int tile0 = paired ? it : it * q;
      const int q_eff = paired ? 2 : min(q, sg->n_tiles - tile0);
      // lane a < q_eff moves tile a of the item
      const __nv_bfloat16* wsrc = (lane == 0 || !paired) ? sg->w0 + (size_t)(tile0 + (lane == 0 ? 0 : 1)) * (C / 16) * 256
                                                         : sg->w1 + (size_t)tile0 * (C / 16) * 256;
      const float* in0 = sg->in0;
      const float* in1 = sg->in1;
      const int in_stride = sg->in_stride;
      // activation rows handled by this lane (row s = lane, lane + 32, ... of nB*T rows)
      // dependency: the inputs of this item must have been produced
      if (check_deps && sg->dep_idx >= 0) {
        const int32_t* dep = P.sync + SY_DEP + sg->dep_idx;
        const int target = sg->dep_target;
        unsigned spins = 0;
        bool ready = false;
        while (!ready) {
          ready = __all_sync(0xffffffffu, ld_acquire(dep) >= target);
          if (!ready) {
            __nanosleep(64);
            if (++spins > SPIN_LIMIT / 16) break;
          }
        }
        if (!ready) {
          if (lane == 0) { L.counts[CNT_STATUS] = DEAMOE_ERR_TIMEOUT; *abort_flag = 1; }
          ok = false;
          break;
        }
        fence_proxy_async();
      }
      const int nchunks = (C + kc0 - 1) / kc0;
      for (int ch = 0; ch < nchunks && ok; ++ch) {
        const int k0 = ch * kc0;
        const int kc = min(kc0, C - k0);
        bool free_slot = true;
        if (lane == 0) free_slot = mbar_wait(&empty_bar[slot], phase ^ 1u, abort_flag);
        free_slot = __shfl_sync(0xffffffffu, (int)free_slot, 0) != 0;
        if (!free_slot) {
          if (lane == 0) { L.counts[CNT_STATUS] = DEAMOE_ERR_TIMEOUT; *abort_flag = 1; }
          ok = false;
          break;
        }
        unsigned char* sbase = ring + (size_t)slot * SLOT_BYTES;
        const uint32_t wbytes = (uint32_t)kc * 32u;
        const int astride = kc + ACT_PAD;
        if (lane == 0) {
          SlotHdr* h = reinterpret_cast<SlotHdr*>(sbase);
          h->kind = 0; h->first = (ch == 0); h->last = (ch == nchunks - 1); h->kc = kc;
          h->T = T; h->q = q_eff; h->paired = paired; h->nB = nB;
          h->epi = sg->epi; h->use_lo = sg->use_lo; h->row0 = tile0 * 16; h->rows = sg->rows;
          h->out_stride = sg->out_stride; h->out_row0 = sg->out_row0; h->npass = (T + 7) / 8;
          h->out = sg->out;
          h->done = (sg->done_idx >= 0) ? P.sync + SY_DEP + sg->done_idx : nullptr;
          mbar_arrive_expect_tx(&full_bar[slot], (uint32_t)q_eff * wbytes + (uint32_t)(nB * T) * (uint32_t)kc * 4u);
        }
        __syncwarp();
        if (lane < q_eff)
          bulk_g2s_hint(sbase + SLOT_HDR + (size_t)lane * wbytes, wsrc + (size_t)(k0 / 16) * 256, wbytes,
                        &full_bar[slot], pol);
        unsigned char* abase = sbase + SLOT_HDR + (size_t)q_eff * wbytes;
        for (int rr = lane; rr < nB * T; rr += 32) {
          const int nb = rr / T, s = rr - nb * T;
          const int row = sg->in_rows ? sg->in_rows[s] : sg->in_row0 + s;
          const float* src = (nb ? in1 : in0) + (size_t)row * in_stride + k0;
          bulk_g2s(abase + (size_t)rr * astride * 4, src, (uint32_t)kc * 4u, &full_bar[slot]);
        }
        if (++slot == NSLOT) { slot = 0; phase ^= 1u; }
      }
    }
    // end-of-work marker (also sent after an abort so the consumers leave their loop)
    {
      bool free_slot = true;
      if (lane == 0) free_slot = mbar_wait(&empty_bar[slot], phase ^ 1u, abort_flag);
      if (lane == 0 && free_slot) {
        SlotHdr* h = reinterpret_cast<SlotHdr*>(ring + (size_t)slot * SLOT_BYTES);
        h->kind = 1;
        mbar_arrive(&full_bar[slot]);
      }
    }
    return;
  }

  // ================================================================ consumers
  const int g = lane >> 2, tig = lane & 3;
  float acc[2][4][4];
  int slot = 0;
  uint32_t phase = 0;
  while (true) {
    if (!mbar_wait(&full_bar[slot], phase, abort_flag)) {
      if (lane == 0) { L.counts[CNT_STATUS] = DEAMOE_ERR_TIMEOUT; *abort_flag = 1; }
      break;
    }
    const unsigned char* sbase = ring + (size_t)slot * SLOT_BYTES;
    const SlotHdr hd = *reinterpret_cast<const SlotHdr*>(sbase);
    if (hd.kind != 0) break;
    if (hd.first) {
#pragma unroll
      for (int a = 0; a < 2; ++a)
#pragma unroll
        for (int p = 0; p < 4; ++p)
#pragma unroll
          for (int e = 0; e < 4; ++e) acc[a][p][e] = 0.f;
    }
    const int kc = hd.kc, T = hd.T, q = hd.q, npass = hd.npass;
    const int astride = kc + ACT_PAD;
    const uint4* wt0 = reinterpret_cast<const uint4*>(sbase + SLOT_HDR);
    const uint4* wt1 = reinterpret_cast<const uint4*>(sbase + SLOT_HDR + (size_t)kc * 32);
    const float* act = reinterpret_cast<const float*>(sbase + SLOT_HDR + (size_t)q * kc * 32);
    const int nkt = kc >> 4;
    for (int kt = warp; kt < nkt; kt += CONSUMER_WARPS) {
      const uint4 A0 = wt0[kt * 32 + lane];
      uint4 A1 = make_uint4(0u, 0u, 0u, 0u);
      if (q > 1) A1 = wt1[kt * 32 + lane];
#pragma unroll
      for (int p = 0; p < 4; ++p) {
        if (p < npass) {
          const int s = min(p * 8 + g, T - 1);
          uint32_t bh[2][2], bl[2][2];
#pragma unroll
          for (int nb = 0; nb < 2; ++nb) {
            if (nb < hd.nB) {
              const float* xr = act + (size_t)(nb * T + s) * astride + kt * 16 + tig * 2;
              const float2 x0 = *reinterpret_cast<const float2*>(xr);
              const float2 x1 = *reinterpret_cast<const float2*>(xr + 8);
              float r0, r1, r2, r3;
              bh[nb][0] = pack_hi(x0.x, x0.y, r0, r1);
              bh[nb][1] = pack_hi(x1.x, x1.y, r2, r3);
              bl[nb][0] = pack_bf(r0, r1);
              bl[nb][1] = pack_bf(r2, r3);
            } else {
              bh[nb][0] = bh[0][0]; bh[nb][1] = bh[0][1];
              bl[nb][0] = bl[0][0]; bl[nb][1] = bl[0][1];
            }
          }
          mma_bf16(acc[0][p], A0, bh[0][0], bh[0][1]);
          if (hd.use_lo) mma_bf16(acc[0][p], A0, bl[0][0], bl[0][1]);
          if (q > 1 && p < 2) {
            mma_bf16(acc[1][p], A1, bh[1][0], bh[1][1]);
            if (hd.use_lo) mma_bf16(acc[1][p], A1, bl[1][0], bl[1][1]);
          }
        }
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&empty_bar[slot]);
    if (++slot == NSLOT) { slot = 0; phase ^= 1u; }

    if (hd.last) {
      // cross-warp reduction, epilogue, completion signal
      float* mine = red + (size_t)warp * (MAX_QP * 128);
#pragma unroll
      for (int a = 0; a < 2; ++a)
#pragma unroll
        for (int p = 0; p < 4; ++p)
          if (a < q && p < npass && (a == 0 || p < 2)) {
#pragma unroll
            for (int e = 0; e < 4; ++e) mine[((a * npass + p) * 4 + e) * 32 + lane] = acc[a][p][e];
          }
      consumer_sync();
      const int per_tile = npass * 128;
      const int count = hd.paired ? per_tile : q * per_tile;
      for (int e = tid; e < count; e += CONSUMER_THREADS) {
        const int a = e / per_tile, rem = e - a * per_tile;
        const int p = rem >> 7, reg = (rem >> 5) & 3, ln = rem & 31;
        float v0 = 0.f, v1 = 0.f;
#pragma unroll
        for (int w = 0; w < CONSUMER_WARPS; ++w) {
          v0 += red[(size_t)w * (MAX_QP * 128) + a * per_tile + rem];
          if (hd.paired) v1 += red[(size_t)w * (MAX_QP * 128) + per_tile + rem];
        }
        const int row = hd.row0 + a * 16 + (ln >> 2) + ((reg & 2) ? 8 : 0);
        const int s = p * 8 + (ln & 3) * 2 + (reg & 1);
        if (row < hd.rows && s < T) {
          float r;
          if (hd.epi == EPI_SIGMA) r = sigma_f(L.sigma, v0);
          else if (hd.epi == EPI_SWIGLU) r = silu_f(v0) * v1;
          else r = v0;
          hd.out[(size_t)(hd.out_row0 + s) * hd.out_stride + row] = r;
        }
      }
      __threadfence();
      consumer_sync();
      if (tid == 0 && hd.done) {
        __threadfence();
        atomicAdd(hd.done, 1);
      }
    }
  }
}

// ---------------------------------------------------------------- host side
int stream_default_schedule() { return DEAMOE_SCHED_STAGED; }

static void fill_stage(StageCfg& s, const __nv_bfloat16* w0, const __nv_bfloat16* w1, size_t unit_elems, int C,
                       int rows, int paired, int epi) {
  s.w0 = w0; s.w1 = w1; s.unit_elems = unit_elems; s.C = C; s.rows = rows;
  s.n_tiles = (rows + 15) / 16;
  s.paired = paired;
  s.q = paired ? 2 : 1;
  s.epi = epi;
  s.tg = 8 * (MAX_QP / s.q);
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

deamoe_status_t stream_plan_create(const LayerDev& L, const deamoe_weights_t& w, int schedule, cudaStream_t s,
                                   StreamPlan** out, uint64_t* bytes) {
  StreamPlan* p = new (std::nothrow) StreamPlan();
  if (!p) return DEAMOE_ERR_ALLOC;
  std::memset(p, 0, sizeof(*p));
  p->schedule = schedule;
  int dev = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&p->n_sm, cudaDevAttrMultiProcessorCount, dev);
  if (p->n_sm <= 0) p->n_sm = 148;
  const size_t units = L.vanilla ? (size_t)L.n : (size_t)L.m;
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
      o_pg = total; total += (size_t)L.n * e_rf;
      o_pu = total; total += (size_t)L.n * e_rf;
      o_pd = total; total += (size_t)L.n * e_fr;
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
      P(w.priv_gate, o_pg, L.r, L.f, L.f, 1, rf, (long long)e_rf, L.n);
      P(w.priv_up, o_pu, L.r, L.f, L.f, 1, rf, (long long)e_rf, L.n);
      P(w.priv_down, o_pd, L.f, L.r, 1, L.f, rf, (long long)e_fr, L.n);
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
  const size_t seg_bytes = (size_t)d.max_segs * sizeof(Seg);
  const size_t sync_bytes = (size_t)(SY_DEP + d.n_dep + 8) * sizeof(int32_t);
  if (e == cudaSuccess) e = cudaMalloc(&d.segs, seg_bytes);
  if (e == cudaSuccess) e = cudaMalloc(&d.sync, sync_bytes);
  if (e == cudaSuccess) e = cudaMemsetAsync(d.sync, 0, sync_bytes, s);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(k_stream, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)STREAM_SMEM);
  p->bytes += seg_bytes + sync_bytes;
  if (e != cudaSuccess) {
    cudaGetLastError();
    stream_plan_destroy(p);
    return e == cudaErrorMemoryAllocation ? DEAMOE_ERR_ALLOC : DEAMOE_ERR_CUDA;
  }
  *out = p;
  *bytes = p->bytes;
  return DEAMOE_OK;
}

void stream_plan_destroy(StreamPlan* p) {
  if (!p) return;
  if (p->packed) cudaFree(p->packed);
  if (p->dev.segs) cudaFree(p->dev.segs);
  if (p->dev.sync) cudaFree(p->dev.sync);
  delete p;
}

int stream_build_worklist(StreamPlan& p, const LayerDev& L, int B, cudaStream_t s) {
  k_build_worklist<<<1, BUILD_THREADS, 0, s>>>(L, p.dev, B);
  return cudaGetLastError() == cudaSuccess ? 1 : -1;
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

__global__ void k_identity_private(LayerDev L);  // defined below

int stream_forward(StreamPlan& p, const LayerDev& L, int B, cudaStream_t s) {
  (void)B;
  int stages[MAX_CAT];
  const int ncat = host_categories(L, stages);
  int launches = 0;
  const bool fused = p.schedule == DEAMOE_SCHED_FUSED && (L.vanilla || L.r > 0);
  if (fused) {
    k_stream<<<p.n_sm, STREAM_THREADS, STREAM_SMEM, s>>>(L, p.dev, MAX_CAT, -1, 1);
    ++launches;
  } else {
    for (int c = 0; c < ncat; ++c) {
      if (stages[c] == ST_S4 && !L.vanilla && L.r == 0) {
        k_identity_private<<<p.n_sm, 256, 0, s>>>(L);
        ++launches;
      }
      k_stream<<<p.n_sm, STREAM_THREADS, STREAM_SMEM, s>>>(L, p.dev, c, c, 0);
      ++launches;
    }
  }
  return cudaGetLastError() == cudaSuccess ? launches : -1;
}

// priv == 0: A = identity, so Y = SiLU(G) * U and Z = sigma(Y) element by element.
__global__ void k_identity_private(LayerDev L) {
  const int pairs = L.counts[CNT_PAIRS];
  const size_t total = (size_t)pairs * L.f;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    const int pr = (int)(i / L.f), c = (int)(i % L.f);
    const float* gu = L.GU + (size_t)L.pair_gurow[pr] * 2 * L.f;
    L.Z[i] = sigma_f(L.sigma, silu_f(gu[c]) * gu[L.f + c]);
  }
}

}  // namespace deamoe
