// Device-side pieces of the routing step shared by the stand-alone kernels (route.cu) and the
// fused routing kernel of the streaming schedules (stream.cu).
#pragma once
#include "deamoe_internal.cuh"

namespace deamoe {

// ---------------------------------------------------------------- top-k + gate weights
// One warp per token.  Order: logit descending, ties to the lower expert index.
constexpr int TOPK_WARPS = 4;

static __device__ __forceinline__ bool better(float v, int i, float bv, int bi) {
  return (v > bv) || (v == bv && i < bi);
}

// Strict department coverage (the variant Section 3.3 evaluates in its last paragraph), applied by
// one warp to the selection it holds (lane q < k: the q-th selected expert my_i and its logit
// my_v): while the selection spans fewer than min(k_dept, k) departments, the lowest-ranked
// selected expert whose department holds another selected expert is replaced, in place, by the
// expert with the largest logit (ties: lowest index) of the departments not yet covered.
// find(covered, v, i) returns that expert to every lane (i = 0x7fffffff: none).  m <= 64.
template <typename Find>
static __device__ __forceinline__ void strict_coverage(const LayerDev& L, int lane, float& my_v, int& my_i, Find find) {
  const int k = L.k, g = L.g;
  const int target = min(min(L.k_dept, k), L.m);
#pragma unroll 1
  for (int round = 0; round < target; ++round) {
    const int md = (lane < k) ? my_i / g : -1 - lane;  // lanes without a selection match nobody
    const unsigned long long bit = (lane < k) ? (1ull << md) : 0ull;
    const unsigned long long covered =
        (unsigned long long)__reduce_or_sync(0xffffffffu, (unsigned)bit) |
        ((unsigned long long)__reduce_or_sync(0xffffffffu, (unsigned)(bit >> 32)) << 32);
    if (__popcll(covered) >= target) break;
    const unsigned same = __match_any_sync(0xffffffffu, md);
    const int victim = __reduce_max_sync(0xffffffffu, (lane < k && (same & ~(1u << lane))) ? lane : -1);
    if (victim < 0) break;
    float cv;
    int ci;
    find(covered, cv, ci);
    if (ci == 0x7fffffff) break;
    if (lane == victim) { my_v = cv; my_i = ci; }
  }
}

// Top-k and gate weights of token t by one warp.  lg: n floats, dead: n bytes of shared memory.
static __device__ void topk_one_token(const LayerDev& L, int t, int B, int kslices, float* lg, unsigned char* dead,
                                      int lane, int32_t* __restrict__ user_idx, float* __restrict__ user_w) {
  const int n = L.n, g = L.g, m = L.m, k = L.k;
  float mx_all = -INFINITY;
  for (int i = lane; i < n; i += 32) {
    float v = 0.f;
    for (int s = 0; s < kslices; ++s) v += L.logit_part[((size_t)s * B + t) * n + i];
    if (!(v == v)) v = -INFINITY;  // a NaN logit (non-finite input) must still yield valid indices
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
  if (L.strict_dept && L.k_dept > 0)
    strict_coverage(L, lane, my_v, my_i, [&](unsigned long long covered, float& cv, int& ci) {
      float bv = -INFINITY;
      int bi = 0x7fffffff;
      for (int i = lane; i < n; i += 32)
        if (!((covered >> (i / g)) & 1ull) && better(lg[i], i, bv, bi)) { bv = lg[i]; bi = i; }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (better(ov, oi, bv, bi)) { bv = ov; bi = oi; }
      }
      cv = bv; ci = bi;
    });
  // gate weights
  const float top = __shfl_sync(0xffffffffu, my_v, 0);
  float e, den;
  if (L.norm_topk) {  // 1: softmax over the selection; 2: logistic scores normalised over the selection
    e = (lane < k) ? (L.norm_topk == 2 ? 1.f / (1.f + expf(-my_v)) : expf(my_v - top)) : 0.f;
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


// Same result with the logits held in registers (n <= 32 * VPL, flat top-k): every partial-logit
// load is issued before the first use, and the k selection rounds touch no memory at all.
// Largest key of the eight keys of group GI that are not masked by `taken`, and the lowest index
// that holds it (strict compare).  GI is a template argument so that key[] is only ever indexed
// with constants and stays in registers.
template <int GI, int VPL>
static __device__ __forceinline__ void rescan_group(const unsigned (&key)[VPL], unsigned taken, unsigned& mx_out,
                                                    int& mj_out) {
  unsigned mx = 0u;
  int mj = GI * 8;
#pragma unroll
  for (int jj = 0; jj < 8; ++jj) {
    const unsigned kq = ((taken >> (GI * 8 + jj)) & 1u) ? 0u : key[GI * 8 + jj];
    if (kq > mx) { mx = kq; mj = GI * 8 + jj; }
  }
  mx_out = mx;
  mj_out = mj;
}

// FEAT: 0 = neither a group limit nor strict coverage nor the softmax over all experts can occur (their code is
// left out of the instantiation); 1 = whatever the layer's configuration says.
template <int VPL, int FEAT = 1>
static __device__ void topk_one_token_regs(const LayerDev& L, int t, int B, int kslices, int lane,
                                           int32_t* __restrict__ user_idx, float* __restrict__ user_w) {
  const int n = L.n, k = L.k;
  float v[VPL];
  unsigned taken = 0;
  {
    // Slices are added in the fixed order 0, 1, ...; four (two for the wider variants) slices'
    // loads are in flight at a time.  The loop stays rolled: this runs once per step from a cold instruction
    // cache, where a short loop beats a long unrolled run of loads.
#pragma unroll
    for (int j = 0; j < VPL; ++j) v[j] = 0.f;
    const float* __restrict__ src = L.logit_part + (size_t)t * n;
    const size_t slice = (size_t)B * n;
    if (VPL <= 8) {
#pragma unroll 4
      for (int sl = 0; sl < kslices; ++sl, src += slice) {
#pragma unroll
        for (int j = 0; j < VPL; ++j) v[j] += __ldg(src + min(lane + 32 * j, n - 1));
      }
    } else {
#pragma unroll 2
      for (int sl = 0; sl < kslices; ++sl, src += slice) {
#pragma unroll
        for (int j = 0; j < VPL; ++j) v[j] += __ldg(src + min(lane + 32 * j, n - 1));
      }
    }
#pragma unroll
    for (int j = 0; j < VPL; ++j) {
      if (!(v[j] == v[j])) v[j] = -INFINITY;  // a NaN logit (non-finite input) must still yield valid indices
      if (lane + 32 * j >= n) { v[j] = -INFINITY; taken |= 1u << j; }
    }
  }
#ifdef DEAMOE_TRACE
  float chk = 0.f;
#pragma unroll
  for (int j = 0; j < VPL; ++j) chk += v[j];
  long long ta = clock64();
  if (chk == 12345.678f) L.counts[15] = 1;
#endif
  float mx_all = -INFINITY, den_all = 0.f;
  if (FEAT && !L.norm_topk) {
#pragma unroll
    for (int j = 0; j < VPL; ++j) mx_all = fmaxf(mx_all, v[j]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx_all = fmaxf(mx_all, __shfl_xor_sync(0xffffffffu, mx_all, o));
#pragma unroll
    for (int j = 0; j < VPL; ++j)
      if (!((taken >> j) & 1u)) den_all += expf(v[j] - mx_all);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) den_all += __shfl_xor_sync(0xffffffffu, den_all, o);
  }
  if (FEAT && L.k_dept > 0 && L.k_dept < L.m) {
    // Group limit (Section 3.3; needs m <= 32): the score of a department is its largest logit;
    // a department is dropped when at least k_dept departments rank ahead of it (score
    // descending, index ascending).  Lane d ends up holding the score of department d.
    const int g = L.g, m = L.m;
    float dscore = -INFINITY;
#pragma unroll 1
    for (int d = 0; d < m; ++d) {
      const int lo = d * g, hi = lo + g;
      float loc = -INFINITY;
#pragma unroll
      for (int j = 0; j < VPL; ++j) {
        const int idx = lane + 32 * j;
        if (idx >= lo && idx < hi && idx < n) loc = fmaxf(loc, v[j]);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) loc = fmaxf(loc, __shfl_xor_sync(0xffffffffu, loc, o));
      if (lane == d) dscore = loc;
    }
    int ahead = 0;
#pragma unroll 1
    for (int d2 = 0; d2 < m; ++d2) {
      const float s2 = __shfl_sync(0xffffffffu, dscore, d2);
      ahead += better(s2, d2, dscore, lane) ? 1 : 0;
    }
    const unsigned alive = __ballot_sync(0xffffffffu, lane < m && ahead < L.k_dept);
    const unsigned inv = (g > 1) ? (unsigned)((0x100000000ull + (unsigned)g - 1u) / (unsigned)g) : 0u;  // ceil(2^32 / g)
#pragma unroll
    for (int j = 0; j < VPL; ++j) {
      const unsigned idx = (unsigned)(lane + 32 * j);
      const unsigned d = (g > 1) ? __umulhi(idx, inv) : idx;  // idx / g, exact for idx * g < 2^32
      if (idx < (unsigned)n && !((alive >> d) & 1u)) taken |= 1u << j;
    }
  }
  // Selection on order-preserving integer keys (larger logit <=> larger key, equal logits <=> equal
  // keys; 0 stands for "not a candidate").  A lane keeps the maximum of each group of eight of its
  // keys, so a round costs a handful of compares, two warp reductions (largest key, then the
  // lowest index that holds it: ties go to the lower expert index) and, in the winning lane only,
  // the rescan of one group.  The keys are never modified: selected and excluded elements are
  // masked through `taken`.
  static_assert(VPL % 8 == 0 && VPL <= 32, "keys are grouped by eight, at most four groups");
  constexpr int NG = VPL / 8;
  unsigned key[VPL];
#pragma unroll
  for (int j = 0; j < VPL; ++j) {
    const unsigned bits = __float_as_uint(v[j] + 0.f);  // + 0.f: -0 and +0 are one value, so they get one key
    key[j] = (bits & 0x80000000u) ? ~bits : (bits | 0x80000000u);
  }
  unsigned gmax[NG];
  int gj[NG];
#define DEAMOE_EACH_GROUP(OP) \
  { if (NG > 0) { OP(0) } if (NG > 1) { OP(1) } if (NG > 2) { OP(2) } if (NG > 3) { OP(3) } }
#define DEAMOE_GI(GI) ((GI) < NG ? (GI) : 0)
#define DEAMOE_RESCAN(GI) rescan_group<DEAMOE_GI(GI), VPL>(key, taken, gmax[DEAMOE_GI(GI)], gj[DEAMOE_GI(GI)]);
#define DEAMOE_RESCAN_IF(GI) if ((js >> 3) == (GI)) { DEAMOE_RESCAN(GI) }
  DEAMOE_EACH_GROUP(DEAMOE_RESCAN)
  float my_v = 0.f;  // lane q keeps the q-th selected logit (k <= 32)
  int my_i = 0;
#pragma unroll 1
  for (int q = 0; q < k; ++q) {
    unsigned best = gmax[0];
    int bj = gj[0];
#pragma unroll
    for (int gi = 1; gi < NG; ++gi)
      if (gmax[gi] > best) { best = gmax[gi]; bj = gj[gi]; }
    const unsigned wmax = __reduce_max_sync(0xffffffffu, best);
    const unsigned cand = (best == wmax && wmax != 0u) ? (unsigned)(lane + 32 * bj) : 0x7fffffffu;
    const unsigned widx = __reduce_min_sync(0xffffffffu, cand);
    if (lane == q) {
      my_i = (int)widx;
      my_v = __uint_as_float((wmax & 0x80000000u) ? (wmax ^ 0x80000000u) : ~wmax);
    }
    if (widx != 0x7fffffffu && lane == (int)(widx & 31u)) {  // the owner masks the element and rescans its group
      const int js = (int)(widx >> 5);
      taken |= 1u << js;
      DEAMOE_EACH_GROUP(DEAMOE_RESCAN_IF)
    }
  }
#undef DEAMOE_RESCAN_IF
#undef DEAMOE_RESCAN
#undef DEAMOE_GI
#undef DEAMOE_EACH_GROUP
#ifdef DEAMOE_TRACE
  if (lane == 0 && t == 0) { L.counts[11] = (int)(clock64() - ta); L.counts[12] = (int)(ta & 0x7fffffff); }
#endif
  if (FEAT && L.strict_dept && L.k_dept > 0)
    strict_coverage(L, lane, my_v, my_i, [&](unsigned long long covered, float& cv, int& ci) {
      float bv = -INFINITY;
      int bi = 0x7fffffff;
#pragma unroll
      for (int j = 0; j < VPL; ++j) {
        const int idx = lane + 32 * j;
        if (idx < n && !((covered >> (idx / L.g)) & 1ull) && better(v[j], idx, bv, bi)) { bv = v[j]; bi = idx; }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (better(ov, oi, bv, bi)) { bv = ov; bi = oi; }
      }
      cv = bv; ci = bi;
    });
  const float top = __shfl_sync(0xffffffffu, my_v, 0);
  float e, den;
  if (!FEAT || L.norm_topk) {  // 1: softmax over the selection; 2: logistic scores normalised over the selection
    e = (lane < k) ? (L.norm_topk == 2 ? 1.f / (1.f + expf(-my_v)) : expf(my_v - top)) : 0.f;
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

// Wide routers (more than 256 experts): a token's top-k by ONE CTA of ceil(n / 256) warps.  Warp w holds experts
// 256 w ... 256 w + 255, eight per lane, and picks its own k best; warp 0 then picks the k best of the warps'
// candidates.  Same selection as topk_one_token_regs (largest logit first, ties to the lower expert index, the same
// fixed-order sums of the partial logits), but every loop over more than eight values is rolled: the 16- and
// 32-logits-per-lane variants of the one-warp routine are 30 - 60 KB of straight-line code, and a step starts with
// cold instruction caches (they took 13 - 25 us, of which the warps stood waiting for instructions five cycles in
// six).  Not for strict department coverage, whose repair step scans all logits.
constexpr int WIDE_MAX_WARPS = 8;
static __host__ __device__ inline bool topk_wide_fits(const LayerDev& L) {
  const bool grouped = L.k_dept > 0 && L.k_dept < L.m;
  return L.n > 256 && L.n <= 256 * WIDE_MAX_WARPS && L.k <= 32 && (!grouped || L.m <= 32) &&
         !(L.strict_dept && L.k_dept > 0);
}
static __device__ void topk_one_token_wide(const LayerDev& L, int t, int B, int kslices, int32_t* __restrict__ user_idx,
                                           float* __restrict__ user_w) {
  __shared__ float s_dmax[WIDE_MAX_WARPS][32];
  __shared__ float s_mx[WIDE_MAX_WARPS], s_den[WIDE_MAX_WARPS];
  __shared__ unsigned s_ckey[WIDE_MAX_WARPS][32];
  __shared__ int s_cidx[WIDE_MAX_WARPS][32];
  const int n = L.n, k = L.k;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
  const int base = 256 * warp;
  float v[8];
  unsigned taken = 0;
  {
#pragma unroll
    for (int j = 0; j < 8; ++j) v[j] = 0.f;
    const float* __restrict__ src = L.logit_part + (size_t)t * n;
    const size_t slice = (size_t)B * n;
    // (eight slices' loads in flight at a time: a round of loads costs 1.5 us here, right behind the kernel that
    // wrote the partial logits, whatever its width)
#pragma unroll 8
    for (int sl = 0; sl < kslices; ++sl, src += slice) {
#pragma unroll
      for (int j = 0; j < 8; ++j) v[j] += __ldg(src + min(base + lane + 32 * j, n - 1));
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      if (!(v[j] == v[j])) v[j] = -INFINITY;  // a NaN logit (non-finite input) must still yield valid indices
      if (base + lane + 32 * j >= n) { v[j] = -INFINITY; taken |= 1u << j; }
    }
  }
  float mx_all = -INFINITY, den_all = 0.f;
  if (!L.norm_topk) {  // gate weights by softmax over ALL experts: maximum and denominator across the warps
    float mx = -INFINITY;
#pragma unroll
    for (int j = 0; j < 8; ++j) mx = fmaxf(mx, v[j]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    if (lane == 0) s_mx[warp] = mx;
    __syncthreads();
#pragma unroll 1
    for (int w = 0; w < nw; ++w) mx_all = fmaxf(mx_all, s_mx[w]);
    float den = 0.f;
#pragma unroll
    for (int j = 0; j < 8; ++j)
      if (!((taken >> j) & 1u)) den += expf(v[j] - mx_all);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) den += __shfl_xor_sync(0xffffffffu, den, o);
    if (lane == 0) s_den[warp] = den;
    __syncthreads();
#pragma unroll 1
    for (int w = 0; w < nw; ++w) den_all += s_den[w];  // warp order: the same sum on every run
  }
  if (L.k_dept > 0 && L.k_dept < L.m) {
    // Group limit (Section 3.3; m <= 32): the score of a department is its largest logit; a department is dropped
    // when at least k_dept departments rank ahead of it (score descending, index ascending).
    const int g = L.g, m = L.m;
    float dloc = -INFINITY;  // lane d: largest logit of department d among this warp's experts
#pragma unroll 1
    for (int d = 0; d < m; ++d) {
      const int lo = d * g, hi = lo + g;
      if (hi <= base || lo >= base + 256) continue;  // (warp-uniform) none of this warp's experts
      float loc = -INFINITY;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int idx = base + lane + 32 * j;
        if (idx >= lo && idx < hi && idx < n) loc = fmaxf(loc, v[j]);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) loc = fmaxf(loc, __shfl_xor_sync(0xffffffffu, loc, o));
      if (lane == d) dloc = loc;
    }
    s_dmax[warp][lane] = dloc;
    __syncthreads();
    float dscore = -INFINITY;
#pragma unroll 1
    for (int w = 0; w < nw; ++w) dscore = fmaxf(dscore, s_dmax[w][lane]);
    int ahead = 0;
#pragma unroll 1
    for (int d2 = 0; d2 < m; ++d2) {
      const float s2 = __shfl_sync(0xffffffffu, dscore, d2);
      ahead += better(s2, d2, dscore, lane) ? 1 : 0;
    }
    const unsigned alive = __ballot_sync(0xffffffffu, lane < m && ahead < L.k_dept);
    const unsigned inv = (g > 1) ? (unsigned)((0x100000000ull + (unsigned)g - 1u) / (unsigned)g) : 0u;  // ceil(2^32 / g)
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const unsigned idx = (unsigned)(base + lane + 32 * j);
      const unsigned d = (g > 1) ? __umulhi(idx, inv) : idx;  // idx / g, exact for idx * g < 2^32
      if (idx < (unsigned)n && !((alive >> d) & 1u)) taken |= 1u << j;
    }
  }
  // this warp's k best (order-preserving integer keys, 0 = not a candidate)
  unsigned key[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const unsigned bits = __float_as_uint(v[j] + 0.f);  // + 0.f: -0 and +0 are one value, so they get one key
    key[j] = (bits & 0x80000000u) ? ~bits : (bits | 0x80000000u);
  }
  {
    unsigned gmax;
    int gj;
    rescan_group<0, 8>(key, taken, gmax, gj);
    unsigned ck = 0u;
    int ci = 0x7fffffff;
#pragma unroll 1
    for (int q = 0; q < k; ++q) {
      const unsigned wmax = __reduce_max_sync(0xffffffffu, gmax);
      if (wmax == 0u) break;  // (warp-uniform) this warp has no candidate left
      const unsigned cand = (gmax == wmax) ? (unsigned)(base + lane + 32 * gj) : 0x7fffffffu;
      const unsigned widx = __reduce_min_sync(0xffffffffu, cand);
      if (lane == q) { ck = wmax; ci = (int)widx; }
      if (lane == (int)((widx - (unsigned)base) & 31u)) {  // the owner masks the element and rescans
        taken |= 1u << ((widx - (unsigned)base) >> 5);
        rescan_group<0, 8>(key, taken, gmax, gj);
      }
    }
    s_ckey[warp][lane] = ck;
    s_cidx[warp][lane] = ci;
  }
  __syncthreads();
  if (warp != 0) return;
  // warp 0: the k best of the warps' candidates.  Lane l holds every warp's l-th candidate; the warps' expert
  // ranges ascend, so among equal keys the first one in a lane's scan is the lower expert index.
  unsigned ckey[WIDE_MAX_WARPS];
  int cidx[WIDE_MAX_WARPS];
#pragma unroll
  for (int w = 0; w < WIDE_MAX_WARPS; ++w) {
    ckey[w] = (w < nw) ? s_ckey[w][lane] : 0u;
    cidx[w] = (w < nw) ? s_cidx[w][lane] : 0x7fffffff;
  }
  unsigned used = 0;
  auto scan = [&](unsigned& bk, int& bi) {
    bk = 0u; bi = 0x7fffffff;
#pragma unroll
    for (int w = 0; w < WIDE_MAX_WARPS; ++w) {
      const unsigned kq = ((used >> w) & 1u) ? 0u : ckey[w];
      if (kq > bk) { bk = kq; bi = cidx[w]; }
    }
  };
  unsigned bk;
  int bi;
  scan(bk, bi);
  float my_v = 0.f;  // lane q keeps the q-th selected logit (k <= 32)
  int my_i = 0;
#pragma unroll 1
  for (int q = 0; q < k; ++q) {
    const unsigned wmax = __reduce_max_sync(0xffffffffu, bk);
    const unsigned cand = (bk == wmax && wmax != 0u) ? (unsigned)bi : 0x7fffffffu;
    const unsigned widx = __reduce_min_sync(0xffffffffu, cand);
    if (lane == q) {
      my_i = (int)widx;
      my_v = __uint_as_float((wmax & 0x80000000u) ? (wmax ^ 0x80000000u) : ~wmax);
    }
    if (widx != 0x7fffffffu && bk == wmax && (unsigned)bi == widx) {  // the owner drops the candidate and rescans
#pragma unroll
      for (int w = 0; w < WIDE_MAX_WARPS; ++w)
        if (cidx[w] == (int)widx) used |= 1u << w;
      scan(bk, bi);
    }
  }
  // gate weights
  const float top = __shfl_sync(0xffffffffu, my_v, 0);
  float e, den;
  if (L.norm_topk) {  // 1: softmax over the selection; 2: logistic scores normalised over the selection
    e = (lane < k) ? (L.norm_topk == 2 ? 1.f / (1.f + expf(-my_v)) : expf(my_v - top)) : 0.f;
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
#pragma unroll 1
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

// Bucketing for one CTA of `nthr` threads (a multiple of 64); s_u32: bucket_smem_bytes() of shared
// memory that must stay untouched between the two parts.  Executed once per step by one CTA,
// usually with a cold instruction cache: the loops are kept rolled so that the code stays small.
//
// Part 1, departments: membership bit masks of tokens per expert and per department (atomicOr),
// department counts, active-department mask (warp ballot) and list, CSR offsets (warp scan) and
// the ascending token list X^j of every department.  This is all the first stage of the layer
// needs, so a caller may hand that stage its work before running part 2.
// 32-bit words of shared memory the bucketing needs
static __host__ __device__ inline size_t bucket_smem_words(int n, int m, int B) {
  const int W = (B + 31) / 32;
  return (size_t)(n + m) * W + (size_t)n + m + (n + 1) + (m + 1);
}

struct BucketSmem {
  uint32_t *emask, *dmask;
  int *ecnt, *dcnt, *eoff, *doff;
  int W;
};
static __device__ __forceinline__ BucketSmem bucket_smem(const LayerDev& L, int B, uint32_t* s_u32) {
  BucketSmem b;
  b.W = (B + 31) / 32;
  b.emask = s_u32;                                            // [n][W]
  b.dmask = b.emask + (size_t)L.n * b.W;                      // [m][W]
  b.ecnt = reinterpret_cast<int*>(b.dmask + (size_t)L.m * b.W);  // [n]
  b.dcnt = b.ecnt + L.n;                                      // [m]
  b.eoff = b.dcnt + L.m;                                      // [n+1]
  b.doff = b.eoff + L.n + 1;                                  // [m+1]
  return b;
}

static __device__ void bucket_departments(const LayerDev& L, int B, uint32_t* s_u32, int nthr) {
  const int n = L.n, m = L.m, g = L.g, k = L.k;
  const BucketSmem b = bucket_smem(L, B, s_u32);
  const int W = b.W;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
#pragma unroll 1
  for (int i = tid; i < (n + m) * W; i += nthr) s_u32[i] = 0u;
  __syncthreads();
#pragma unroll 1
  for (int p = tid; p < B * k; p += nthr) {
    const int t = p / k;
    const int i = L.topk_idx[p];
    const int j = i / g;
    if (j < L.dept_lo || j >= L.dept_hi) continue;  // a department another layer object (another GPU) holds
    atomicOr(&b.emask[(size_t)i * W + (t >> 5)], 1u << (t & 31));
    atomicOr(&b.dmask[(size_t)j * W + (t >> 5)], 1u << (t & 31));
  }
  __syncthreads();
  // department counts; the active-department bitmask falls out of a warp ballot (32 departments
  // per warp iteration, written as the two 32-bit halves of the 64-bit words)
#pragma unroll 1
  for (int j = tid; j < ((m + 63) & ~63); j += nthr) {
    int c = 0;
    if (j < m) {
#pragma unroll 1
      for (int w = 0; w < W; ++w) c += __popc(b.dmask[(size_t)j * W + w]);
      b.dcnt[j] = c;
    }
    const unsigned live = __ballot_sync(0xffffffffu, c > 0);
    if ((tid & 31) == 0) reinterpret_cast<uint32_t*>(L.dept_mask)[j >> 5] = live;
  }
  __syncthreads();
  if (warp == 0) warp_exclusive_offsets(b.dcnt, m, b.doff, L.active_dept, lane, &L.counts[CNT_ACTIVE_DEPT]);
  __syncthreads();
#pragma unroll 1
  for (int j = tid; j <= m; j += nthr) L.dept_off[j] = b.doff[j];
  if (tid == 0) {
    L.counts[CNT_STATUS] = 0;
    L.counts[CNT_TOKEN_DEPT] = b.doff[m];
  }
#pragma unroll 1
  for (int j = tid; j < m; j += nthr) {
    int pos = b.doff[j];
#pragma unroll 1
    for (int w = 0; w < W; ++w) {
      uint32_t bits = b.dmask[(size_t)j * W + w];
#pragma unroll 1
      while (bits) {
        const int bb = __ffs(bits) - 1;
        bits &= bits - 1;
        L.dept_tok[pos++] = w * 32 + bb;
      }
    }
  }
  __syncthreads();
}

// Part 2, experts: counts, active list, CSR offsets and ascending token lists per expert, the slot
// of every (token, expert) pair in expert-major order and the department row each pair reads.
static __device__ void bucket_experts(const LayerDev& L, int B, uint32_t* s_u32, int nthr) {
  const int n = L.n, g = L.g, k = L.k;
  const BucketSmem b = bucket_smem(L, B, s_u32);
  const int W = b.W;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
#pragma unroll 1
  for (int i = tid; i < n; i += nthr) {
    int c = 0;
#pragma unroll 1
    for (int w = 0; w < W; ++w) c += __popc(b.emask[(size_t)i * W + w]);
    b.ecnt[i] = c;
  }
  __syncthreads();
  if (warp == 0) warp_exclusive_offsets(b.ecnt, n, b.eoff, L.active_expert, lane, &L.counts[CNT_ACTIVE_EXPERT]);
  __syncthreads();
#pragma unroll 1
  for (int i = tid; i <= n; i += nthr) L.expert_off[i] = b.eoff[i];
  if (tid == 0) L.counts[CNT_PAIRS] = b.eoff[n];
#pragma unroll 1
  for (int i = tid; i < n; i += nthr) {
    int pos = b.eoff[i];
#pragma unroll 1
    for (int w = 0; w < W; ++w) {
      uint32_t bits = b.emask[(size_t)i * W + w];
#pragma unroll 1
      while (bits) {
        const int bb = __ffs(bits) - 1;
        bits &= bits - 1;
        L.expert_tok[pos++] = w * 32 + bb;
      }
    }
  }
  // pair order and the GU row of every pair
#pragma unroll 1
  for (int p = tid; p < B * k; p += nthr) {
    const int t = p / k;
    const int i = L.topk_idx[p];
    const int j = i / g;
    if (j < L.dept_lo || j >= L.dept_hi) {  // not this layer object's pair: the combine skips it
      L.pair_slot[p] = -1;
      continue;
    }
    int re = 0, rd = 0;
#pragma unroll 1
    for (int w = 0; w < (t >> 5); ++w) {
      re += __popc(b.emask[(size_t)i * W + w]);
      rd += __popc(b.dmask[(size_t)j * W + w]);
    }
    const uint32_t below = (1u << (t & 31)) - 1u;
    re += __popc(b.emask[(size_t)i * W + (t >> 5)] & below);
    rd += __popc(b.dmask[(size_t)j * W + (t >> 5)] & below);
    const int slot = b.eoff[i] + re;
    L.pair_slot[p] = slot;
    L.pair_gurow[slot] = b.doff[j] + rd;
  }
}

static __device__ void bucket_block(const LayerDev& L, int B, uint32_t* s_u32, int nthr) {
  bucket_departments(L, B, s_u32, nthr);
  bucket_experts(L, B, s_u32, nthr);
}


}  // namespace deamoe
