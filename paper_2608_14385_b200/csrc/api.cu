// C ABI of libdeamoe.so: argument checking, ownership, and the order in which the stages of
// one decode step are enqueued.  All arithmetic lives in the kernels of the other files.
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "deamoe_internal.cuh"
#include "stream.cuh"

using namespace deamoe;

struct deamoe_layer {
  deamoe_config_t cfg;
  LayerDev dev;                 // device view (weights + workspace)
  StreamPlan* plan = nullptr;   // packed weights + work-list machinery of the streaming schedules
  std::vector<void*> owned;     // every device allocation of this layer
  uint64_t device_bytes = 0;
  int schedule = DEAMOE_SCHED_PLAIN;
  int kslices = 1;
  int last_launches = 0;
  int last_B = 0;
  void* stage_tokens = nullptr; // device staging for deamoe_forward_host
  void* stage_out = nullptr;
};

namespace {

size_t dtype_size(int dt) { return dt == DEAMOE_F32 ? 4 : 2; }

template <typename T>
deamoe_status_t dev_alloc(deamoe_layer* L, T** p, size_t count) {
  void* q = nullptr;
  const size_t bytes = (count ? count : 1) * sizeof(T);
  if (cudaMalloc(&q, bytes) != cudaSuccess) {
    cudaGetLastError();
    return DEAMOE_ERR_ALLOC;
  }
  L->owned.push_back(q);
  L->device_bytes += bytes;
  *p = reinterpret_cast<T*>(q);
  return DEAMOE_OK;
}

deamoe_status_t dev_copy(deamoe_layer* L, const void** dst, const void* src, size_t bytes, cudaStream_t s) {
  char* q = nullptr;
  deamoe_status_t st = dev_alloc(L, &q, bytes);
  if (st != DEAMOE_OK) return st;
  if (cudaMemcpyAsync(q, src, bytes, cudaMemcpyDeviceToDevice, s) != cudaSuccess) return DEAMOE_ERR_CUDA;
  *dst = q;
  return DEAMOE_OK;
}

deamoe_status_t check_config(const deamoe_config_t* c, const deamoe_weights_t* w, bool vanilla) {
  if (!c || !w) return DEAMOE_ERR_INVALID_ARG;
  if (c->hidden <= 0 || c->n_dept <= 0 || c->experts_per_dept <= 0 || c->ffn <= 0 || c->priv < 0 ||
      c->top_k <= 0 || c->k_dept < 0 || c->n_shared < 0 || c->n_shared > 1)
    return DEAMOE_ERR_INVALID_ARG;
  const long long n = (long long)c->n_dept * c->experts_per_dept;
  if (c->top_k > n) return DEAMOE_ERR_INVALID_ARG;
  if (c->k_dept > 0 && (long long)c->k_dept * c->experts_per_dept < c->top_k) return DEAMOE_ERR_INVALID_ARG;
  if (c->n_shared && c->shared_ffn <= 0) return DEAMOE_ERR_INVALID_ARG;
  if (c->weight_dtype != DEAMOE_F32 && c->weight_dtype != DEAMOE_BF16) return DEAMOE_ERR_INVALID_ARG;
  if (c->act_dtype != DEAMOE_F32 && c->act_dtype != DEAMOE_BF16) return DEAMOE_ERR_INVALID_ARG;
  if (c->sigma < DEAMOE_SIGMA_NONE || c->sigma > DEAMOE_SIGMA_RMSNORM) return DEAMOE_ERR_INVALID_ARG;
  if (c->norm_topk < 0 || c->norm_topk > 2) return DEAMOE_ERR_INVALID_ARG;
  if (!vanilla && c->sigma == DEAMOE_SIGMA_RMSNORM && c->priv <= 0) return DEAMOE_ERR_UNSUPPORTED;
  if (c->schedule < DEAMOE_SCHED_AUTO || c->schedule > DEAMOE_SCHED_DENSE) return DEAMOE_ERR_INVALID_ARG;
  if (!(c->route_scale == c->route_scale)) return DEAMOE_ERR_INVALID_ARG;
  if (c->strict_dept != 0 && c->strict_dept != 1) return DEAMOE_ERR_INVALID_ARG;
  if (c->strict_dept && c->k_dept > 0 && c->n_dept > 64) return DEAMOE_ERR_UNSUPPORTED;
  if (c->dept_begin != 0 || c->dept_end != 0) {  // a department slice of the layer (0, 0 = all of it)
    if (vanilla) return DEAMOE_ERR_INVALID_ARG;
    if (c->dept_begin < 0 || c->dept_end <= c->dept_begin || c->dept_end > c->n_dept) return DEAMOE_ERR_INVALID_ARG;
  }
  if (c->max_batch < 1 || c->max_batch > DEAMOE_MAX_BATCH) return DEAMOE_ERR_BATCH;
  if (!w->router || !w->dept_gate || !w->dept_up || !w->dept_down) return DEAMOE_ERR_INVALID_ARG;
  if (vanilla && c->priv != 0) return DEAMOE_ERR_INVALID_ARG;
  const bool has_priv = w->priv_gate && w->priv_up && w->priv_down;
  const bool no_priv = !w->priv_gate && !w->priv_up && !w->priv_down;
  if (c->priv > 0 ? !has_priv : !no_priv) return DEAMOE_ERR_INVALID_ARG;
  const bool has_sh = w->shared_gate && w->shared_up && w->shared_down;
  const bool no_sh = !w->shared_gate && !w->shared_up && !w->shared_down;
  if (c->n_shared ? !has_sh : !no_sh) return DEAMOE_ERR_INVALID_ARG;
  if (n > DEAMOE_MAX_EXPERTS || c->top_k > DEAMOE_MAX_TOPK) return DEAMOE_ERR_UNSUPPORTED;
  if ((c->hidden | c->ffn | c->priv | c->shared_ffn) & 3) return DEAMOE_ERR_UNSUPPORTED;
  return DEAMOE_OK;
}

deamoe_status_t create_impl(const deamoe_config_t* cfg, const deamoe_weights_t* w, void* stream,
                            deamoe_layer_t** out, bool vanilla) {
  if (!out) return DEAMOE_ERR_INVALID_ARG;
  deamoe_status_t st = check_config(cfg, w, vanilla);
  if (st != DEAMOE_OK) return st;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev == 0) {
    cudaGetLastError();
    return DEAMOE_ERR_CUDA;
  }
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  deamoe_layer* L = new (std::nothrow) deamoe_layer();
  if (!L) return DEAMOE_ERR_ALLOC;
  L->cfg = *cfg;
  LayerDev& d = L->dev;
  std::memset(&d, 0, sizeof(d));
  d.h = cfg->hidden; d.m = cfg->n_dept; d.g = cfg->experts_per_dept; d.n = d.m * d.g;
  d.f = cfg->ffn; d.r = vanilla ? 0 : cfg->priv; d.k = cfg->top_k; d.k_dept = cfg->k_dept;
  d.n_shared = cfg->n_shared; d.fs = cfg->n_shared ? cfg->shared_ffn : 0;
  d.sigma = vanilla ? DEAMOE_SIGMA_NONE : cfg->sigma; d.norm_topk = cfg->norm_topk;
  d.residual = cfg->residual; d.vanilla = vanilla ? 1 : 0;
  d.wdt = cfg->weight_dtype; d.adt = cfg->act_dtype; d.max_batch = cfg->max_batch;
  d.strict_dept = cfg->strict_dept;
  d.dept_lo = 0; d.dept_hi = d.m;
  if (cfg->dept_end > 0) { d.dept_lo = cfg->dept_begin; d.dept_hi = cfg->dept_end; }
  d.rp = d.r > 0 ? d.r : d.f;
  d.route_scale = cfg->route_scale;

  int sched = cfg->schedule;
  const bool streamable = cfg->weight_dtype == DEAMOE_BF16 &&
                          ((cfg->hidden | cfg->ffn | cfg->priv | cfg->shared_ffn) & 15) == 0;
  // the dense schedule rides on a fused plan: AUTO switches to it by batch size, DENSE always takes it
  const int dense_mode = sched == DEAMOE_SCHED_DENSE ? 2 : (sched == DEAMOE_SCHED_AUTO ? 1 : 0);
  if (sched == DEAMOE_SCHED_DENSE) sched = DEAMOE_SCHED_FUSED;
  if (sched == DEAMOE_SCHED_AUTO) sched = streamable ? stream_default_schedule() : DEAMOE_SCHED_PLAIN;
  if ((sched == DEAMOE_SCHED_STAGED || sched == DEAMOE_SCHED_FUSED) && !streamable) {
    delete L;
    return DEAMOE_ERR_UNSUPPORTED;
  }
  L->schedule = sched;

  const int MB = cfg->max_batch, k = d.k;
  const int tdmax = MB * (k < d.m ? k : d.m);  // (token, department) rows
  const int pmax = MB * k;                     // (token, expert) pairs
  L->kslices = router_kslices(d.n, d.h);

  bool ok = true;
  auto A = [&](deamoe_status_t r) { if (r != DEAMOE_OK && ok) { ok = false; st = r; } };
  const size_t ws = dtype_size(d.wdt);
  const size_t units = vanilla ? (size_t)d.n : (size_t)(d.dept_hi - d.dept_lo);
  const size_t n_loc = (size_t)(d.dept_hi - d.dept_lo) * d.g;  // experts whose private matrices this object holds
  A(dev_copy(L, reinterpret_cast<const void**>(&d.router), w->router, (size_t)d.n * d.h * 4, s));
  if (ok && sched == DEAMOE_SCHED_PLAIN) {
    A(dev_copy(L, &d.dept_gate, w->dept_gate, units * d.f * d.h * ws, s));
    A(dev_copy(L, &d.dept_up, w->dept_up, units * d.f * d.h * ws, s));
    A(dev_copy(L, &d.dept_down, w->dept_down, units * d.f * d.h * ws, s));
    if (d.r > 0) {
      A(dev_copy(L, &d.priv_gate, w->priv_gate, n_loc * d.r * d.f * ws, s));
      A(dev_copy(L, &d.priv_up, w->priv_up, n_loc * d.r * d.f * ws, s));
      A(dev_copy(L, &d.priv_down, w->priv_down, n_loc * d.r * d.f * ws, s));
    }
    if (d.n_shared) {
      A(dev_copy(L, &d.shared_gate, w->shared_gate, (size_t)d.fs * d.h * ws, s));
      A(dev_copy(L, &d.shared_up, w->shared_up, (size_t)d.fs * d.h * ws, s));
      A(dev_copy(L, &d.shared_down, w->shared_down, (size_t)d.fs * d.h * ws, s));
    }
  }
  if (ok) {
    if (d.adt == DEAMOE_BF16) A(dev_alloc(L, &d.x32, (size_t)MB * d.h));
    // bf16 tokens on a streaming schedule: the router product runs on the tensor cores, on a three-piece
    // bf16 copy of the router (route.cu); its partial-logit arrays may be more than the scalar kernel's
    int part_slices = L->kslices;
    if (sched != DEAMOE_SCHED_PLAIN && d.adt == DEAMOE_BF16 && (d.h & 15) == 0) {
      __nv_bfloat16* r3 = nullptr;
      A(dev_alloc(L, &r3, router3_elems(d.n, d.h)));
      if (ok && pack_router3(d.router, r3, d.n, d.h, s) != cudaSuccess) A(DEAMOE_ERR_CUDA);
      d.router3 = r3;
      d.router3_slices = router3_kslices(d.n, d.h);
      if (d.router3_slices > part_slices) part_slices = d.router3_slices;
    }
    A(dev_alloc(L, &d.logit_part, (size_t)part_slices * MB * d.n));
    A(dev_alloc(L, &d.topk_idx, (size_t)pmax));
    A(dev_alloc(L, &d.topk_w, (size_t)pmax));
    A(dev_alloc(L, &d.dept_mask, (size_t)(d.m + 63) / 64));
    A(dev_alloc(L, &d.dept_off, (size_t)d.m + 1));
    A(dev_alloc(L, &d.dept_tok, (size_t)tdmax));
    A(dev_alloc(L, &d.expert_off, (size_t)d.n + 1));
    A(dev_alloc(L, &d.expert_tok, (size_t)pmax));
    A(dev_alloc(L, &d.pair_slot, (size_t)pmax));
    A(dev_alloc(L, &d.pair_gurow, (size_t)pmax));
    A(dev_alloc(L, &d.active_dept, (size_t)d.m));
    A(dev_alloc(L, &d.active_expert, (size_t)d.n));
    A(dev_alloc(L, &d.counts, (size_t)CNT_COUNT));
#ifdef DEAMOE_TRACE
    A(dev_alloc(L, &d.ts, (size_t)24));
#endif
    if (sched == DEAMOE_SCHED_PLAIN) {  // fp32 intermediates of the plain kernels
      if (!vanilla) {
        A(dev_alloc(L, &d.GU, (size_t)tdmax * 2 * d.f));
        A(dev_alloc(L, &d.Z, (size_t)pmax * d.f));
      }
      A(dev_alloc(L, &d.Y, (size_t)pmax * (vanilla ? d.f : d.rp)));
      if (d.n_shared) A(dev_alloc(L, &d.Ysh, (size_t)MB * d.fs));
    }
    if (d.sigma == DEAMOE_SIGMA_RMSNORM) {
      A(dev_alloc(L, &d.ss_gu, (size_t)tdmax * 2));
      A(dev_alloc(L, &d.ss_z, (size_t)pmax));
    }
    A(dev_alloc(L, &d.O, (size_t)pmax * d.h));
    if (d.n_shared) A(dev_alloc(L, &d.Osh, (size_t)MB * d.h));
    const size_t io = (size_t)MB * d.h * dtype_size(d.adt);
    A(dev_alloc(L, reinterpret_cast<char**>(&L->stage_tokens), io));
    A(dev_alloc(L, reinterpret_cast<char**>(&L->stage_out), io));
  }
  if (ok && cudaMemsetAsync(d.counts, 0, CNT_COUNT * sizeof(int32_t), s) != cudaSuccess) A(DEAMOE_ERR_CUDA);
  if (ok && route_configure(d) != cudaSuccess) A(DEAMOE_ERR_CUDA);
  if (ok && sched != DEAMOE_SCHED_PLAIN) {
    uint64_t plan_bytes = 0;
    A(stream_plan_create(d, *w, sched, dense_mode, s, &L->plan, &plan_bytes));
    L->device_bytes += plan_bytes;
    if (ok) d.sh_done = stream_shared_counter(*L->plan);
  }
  if (ok && cudaStreamSynchronize(s) != cudaSuccess) A(DEAMOE_ERR_CUDA);
  if (!ok) {
    cudaGetLastError();
    deamoe_layer_destroy(L);
    return st;
  }
  *out = L;
  return DEAMOE_OK;
}

deamoe_status_t check_call(deamoe_layer_t* L, const void* tokens, int B) {
  if (!L) return DEAMOE_ERR_INVALID_ARG;
  if (B < 0 || B > L->cfg.max_batch) return DEAMOE_ERR_BATCH;
  if (B > 0 && !tokens) return DEAMOE_ERR_INVALID_ARG;
  return DEAMOE_OK;
}

// Device buffers are read and written with 16-byte accesses: a misaligned pointer is an argument
// error reported here, before anything is enqueued, never a fault on the device.
deamoe_status_t check_device_ptr(const void* p) { return aligned16(p) ? DEAMOE_OK : DEAMOE_ERR_INVALID_ARG; }

LayerDev call_view(deamoe_layer_t* L, const void* tokens) {
  LayerDev d = L->dev;
  d.tokens_raw = tokens;
  if (d.adt == DEAMOE_F32) d.x32 = const_cast<float*>(reinterpret_cast<const float*>(tokens));
  return d;
}

}  // namespace

extern "C" {

deamoe_status_t deamoe_layer_create(const deamoe_config_t* cfg, const deamoe_weights_t* weights, void* cuda_stream,
                                    deamoe_layer_t** out) {
  return create_impl(cfg, weights, cuda_stream, out, false);
}

deamoe_status_t deamoe_vanilla_create(const deamoe_config_t* cfg, const deamoe_weights_t* weights,
                                      void* cuda_stream, deamoe_layer_t** out) {
  return create_impl(cfg, weights, cuda_stream, out, true);
}

deamoe_status_t deamoe_layer_destroy(deamoe_layer_t* L) {
  if (!L) return DEAMOE_OK;
  if (L->plan) stream_plan_destroy(L->plan);
  for (void* p : L->owned) cudaFree(p);
  delete L;
  return DEAMOE_OK;
}

deamoe_status_t deamoe_route(deamoe_layer_t* L, void* cuda_stream, const void* tokens, int32_t B, int32_t* topk_idx,
                             float* topk_w) {
  deamoe_status_t st = check_call(L, tokens, B);
  if (st != DEAMOE_OK) return st;
  if (B > 0 && check_device_ptr(tokens) != DEAMOE_OK) return DEAMOE_ERR_INVALID_ARG;
  if (B > 0 && ((reinterpret_cast<uintptr_t>(topk_idx) | reinterpret_cast<uintptr_t>(topk_w)) & 3u))
    return DEAMOE_ERR_INVALID_ARG;
  L->last_B = B;
  L->last_launches = 0;
  if (B == 0) return DEAMOE_OK;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(cuda_stream);
  LayerDev d = call_view(L, tokens);
  const int nl = L->plan ? stream_route(*L->plan, d, tokens, B, s, L->kslices, topk_idx, topk_w)
                         : launch_route(d, tokens, B, s, L->kslices, topk_idx, topk_w);
  if (nl < 0) return DEAMOE_ERR_CUDA;
  L->last_launches = nl;
  return DEAMOE_OK;
}

static deamoe_status_t forward_impl(deamoe_layer_t* L, void* cuda_stream, const void* tokens, int32_t B, void* out,
                                    int partial);

deamoe_status_t deamoe_forward(deamoe_layer_t* L, void* cuda_stream, const void* tokens, int32_t B, void* out) {
  // a department slice alone does not compute the layer's output: its partial sum goes through
  // deamoe_forward_partial, an all-reduce over the slices, and deamoe_finish_partial
  if (L && (L->dev.dept_lo != 0 || L->dev.dept_hi != L->dev.m)) return DEAMOE_ERR_INVALID_ARG;
  return forward_impl(L, cuda_stream, tokens, B, out, 0);
}

deamoe_status_t deamoe_forward_partial(deamoe_layer_t* L, void* cuda_stream, const void* tokens, int32_t B,
                                       float* partial) {
  if (L && L->dev.vanilla) return DEAMOE_ERR_INVALID_ARG;
  return forward_impl(L, cuda_stream, tokens, B, partial, 1);
}

deamoe_status_t deamoe_finish_partial(deamoe_layer_t* L, void* cuda_stream, const float* sum, const void* tokens,
                                      int32_t B, void* out) {
  deamoe_status_t st = check_call(L, tokens, B);
  if (st != DEAMOE_OK) return st;
  if (B == 0) return DEAMOE_OK;
  if (!sum || !out || out == tokens || out == (const void*)sum) return DEAMOE_ERR_INVALID_ARG;
  if (check_device_ptr(tokens) != DEAMOE_OK || check_device_ptr(out) != DEAMOE_OK || check_device_ptr(sum) != DEAMOE_OK)
    return DEAMOE_ERR_INVALID_ARG;
  LayerDev d = call_view(L, tokens);
  return launch_finish_partial(d, sum, tokens, B, out, reinterpret_cast<cudaStream_t>(cuda_stream)) > 0 ? DEAMOE_OK
                                                                                                         : DEAMOE_ERR_CUDA;
}

static deamoe_status_t forward_impl(deamoe_layer_t* L, void* cuda_stream, const void* tokens, int32_t B, void* out,
                                    int partial) {
  deamoe_status_t st = check_call(L, tokens, B);
  if (st != DEAMOE_OK) return st;
  if (B > 0 && (!out || out == tokens)) return DEAMOE_ERR_INVALID_ARG;
  if (B > 0 && (check_device_ptr(tokens) != DEAMOE_OK || check_device_ptr(out) != DEAMOE_OK))
    return DEAMOE_ERR_INVALID_ARG;
  st = deamoe_route(L, cuda_stream, tokens, B, nullptr, nullptr);
  if (st != DEAMOE_OK || B == 0) return st;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(cuda_stream);
  LayerDev d = call_view(L, tokens);
  int nl;
  if (L->schedule == DEAMOE_SCHED_PLAIN) {
    nl = launch_plain_forward(d, B, s);
  } else {
    nl = stream_forward(*L->plan, d, B, s);
  }
  if (nl < 0) return DEAMOE_ERR_CUDA;
  const int nc = launch_combine(d, tokens, B, out, s, partial);
  if (nc < 0) return DEAMOE_ERR_CUDA;
  L->last_launches += nl + nc;
  return DEAMOE_OK;
}

deamoe_status_t deamoe_vanilla_forward(deamoe_layer_t* L, void* cuda_stream, const void* tokens, int32_t B,
                                       void* out) {
  if (!L || !L->dev.vanilla) return DEAMOE_ERR_INVALID_ARG;
  return deamoe_forward(L, cuda_stream, tokens, B, out);
}

deamoe_status_t deamoe_forward_host(deamoe_layer_t* L, void* cuda_stream, const void* tokens, int32_t B, void* out) {
  deamoe_status_t st = check_call(L, tokens, B);
  if (st != DEAMOE_OK) return st;
  if (B == 0) return DEAMOE_OK;
  if (!out) return DEAMOE_ERR_INVALID_ARG;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(cuda_stream);
  const size_t bytes = (size_t)B * L->dev.h * dtype_size(L->dev.adt);
  if (cudaMemcpyAsync(L->stage_tokens, tokens, bytes, cudaMemcpyHostToDevice, s) != cudaSuccess)
    return DEAMOE_ERR_CUDA;
  // If `out` is pinned host memory that the device can address (cudaHostAlloc / cudaHostRegister under
  // unified addressing), the combine kernel writes the result straight into it: one pass of B * h
  // values over the bus, and no separate copy behind the step.  Pageable memory takes the copy.
  void* direct = nullptr;
  {
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, out) == cudaSuccess && at.type == cudaMemoryTypeHost && at.devicePointer &&
        aligned16(at.devicePointer))
      direct = at.devicePointer;
    else
      cudaGetLastError();
  }
  st = deamoe_forward(L, cuda_stream, L->stage_tokens, B, direct ? direct : L->stage_out);
  if (st != DEAMOE_OK) return st;
  if (!direct && cudaMemcpyAsync(out, L->stage_out, bytes, cudaMemcpyDeviceToHost, s) != cudaSuccess)
    return DEAMOE_ERR_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return DEAMOE_ERR_CUDA;
  return DEAMOE_OK;
}

deamoe_status_t deamoe_get_routing(deamoe_layer_t* L, void* cuda_stream, int32_t* topk_idx, float* topk_w,
                                   uint64_t* dept_mask, int32_t* dept_off, int32_t* dept_tok, int32_t* expert_off,
                                   int32_t* expert_tok) {
  if (!L) return DEAMOE_ERR_INVALID_ARG;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(cuda_stream);
  if (cudaStreamSynchronize(s) != cudaSuccess) return DEAMOE_ERR_CUDA;
  const LayerDev& d = L->dev;
  const int B = L->last_B, k = d.k;
  bool ok = true;
  auto G = [&](void* dst, const void* src, size_t bytes) {
    if (dst && bytes && cudaMemcpy(dst, src, bytes, cudaMemcpyDeviceToHost) != cudaSuccess) ok = false;
  };
  G(topk_idx, d.topk_idx, (size_t)B * k * 4);
  G(topk_w, d.topk_w, (size_t)B * k * 4);
  if (B == 0) {
    if (dept_mask) std::memset(dept_mask, 0, ((d.m + 63) / 64) * 8);
    if (dept_off) std::memset(dept_off, 0, (d.m + 1) * 4);
    if (expert_off) std::memset(expert_off, 0, (d.n + 1) * 4);
    return DEAMOE_OK;
  }
  G(dept_mask, d.dept_mask, (size_t)((d.m + 63) / 64) * 8);
  std::vector<int32_t> doff(d.m + 1);
  G(doff.data(), d.dept_off, (size_t)(d.m + 1) * 4);
  if (dept_off && ok) std::memcpy(dept_off, doff.data(), (size_t)(d.m + 1) * 4);
  if (ok) G(dept_tok, d.dept_tok, (size_t)doff[d.m] * 4);
  G(expert_off, d.expert_off, (size_t)(d.n + 1) * 4);
  G(expert_tok, d.expert_tok, (size_t)B * k * 4);
  return ok ? DEAMOE_OK : DEAMOE_ERR_CUDA;
}

deamoe_status_t deamoe_get_stats(deamoe_layer_t* L, void* cuda_stream, int32_t* n_active_dept,
                                 int32_t* n_active_expert, int32_t* n_token_dept_pairs,
                                 uint64_t* unique_weight_bytes, int32_t* device_status) {
  if (!L) return DEAMOE_ERR_INVALID_ARG;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(cuda_stream);
  if (cudaStreamSynchronize(s) != cudaSuccess) return DEAMOE_ERR_CUDA;
  int32_t c[CNT_COUNT] = {0};
  if (L->last_B > 0 && cudaMemcpy(c, L->dev.counts, sizeof(c), cudaMemcpyDeviceToHost) != cudaSuccess)
    return DEAMOE_ERR_CUDA;
  const LayerDev& d = L->dev;
  if (n_active_dept) *n_active_dept = c[CNT_ACTIVE_DEPT];
  if (n_active_expert) *n_active_expert = c[CNT_ACTIVE_EXPERT];
  if (n_token_dept_pairs) *n_token_dept_pairs = c[CNT_TOKEN_DEPT];
  if (unique_weight_bytes) {
    const uint64_t s_w = dtype_size(d.wdt);
    const uint64_t big = (uint64_t)3 * d.h * d.f * s_w, small = (uint64_t)3 * d.r * d.f * s_w;
    uint64_t b = (uint64_t)d.n * d.h * 4 + (uint64_t)d.n_shared * 3 * d.h * d.fs * s_w;
    if (L->last_B > 0) {
      if (d.vanilla) b += (uint64_t)c[CNT_ACTIVE_EXPERT] * big;
      else b += (uint64_t)c[CNT_ACTIVE_DEPT] * big + (uint64_t)c[CNT_ACTIVE_EXPERT] * small;
    }
    *unique_weight_bytes = b;
  }
  if (device_status) *device_status = c[CNT_STATUS];
  return DEAMOE_OK;
}

deamoe_status_t deamoe_profile_enable(deamoe_layer_t* L, int32_t enable) {
  if (!L) return DEAMOE_ERR_INVALID_ARG;
  if (!L->plan) return DEAMOE_ERR_UNSUPPORTED;
  return stream_profile_enable(*L->plan, enable != 0) == cudaSuccess ? DEAMOE_OK : DEAMOE_ERR_CUDA;
}

deamoe_status_t deamoe_profile_last_ms(deamoe_layer_t* L, float* ms) {
  if (!L || !ms) return DEAMOE_ERR_INVALID_ARG;
  if (!L->plan) return DEAMOE_ERR_UNSUPPORTED;
  const cudaError_t e = stream_profile_last_ms(*L->plan, ms);
  if (e == cudaErrorInvalidValue) return DEAMOE_ERR_INVALID_ARG;
  return e == cudaSuccess ? DEAMOE_OK : DEAMOE_ERR_CUDA;
}

deamoe_status_t deamoe_failure_test(deamoe_layer_t* L, int32_t wait_limit, int32_t withhold) {
  if (!L || wait_limit < 0 || withhold < 0 || withhold > 7) return DEAMOE_ERR_INVALID_ARG;
  if (!L->plan) return withhold ? DEAMOE_ERR_UNSUPPORTED : DEAMOE_OK;  // the plain schedule has no device-side waits
  return stream_set_failure_test(*L->plan, (unsigned)wait_limit, withhold) ? DEAMOE_OK : DEAMOE_ERR_UNSUPPORTED;
}

deamoe_status_t deamoe_probe_read(void* cuda_stream, const void* buf, uint64_t bytes, uint32_t* sink) {
  if (!buf || !sink || bytes < 16 || !aligned16(buf) || (reinterpret_cast<uintptr_t>(sink) & 3u)) return DEAMOE_ERR_INVALID_ARG;
  return launch_probe_read(buf, (size_t)bytes, sink, DEAMOE_PROBE_BLOCKS, reinterpret_cast<cudaStream_t>(cuda_stream)) > 0
             ? DEAMOE_OK : DEAMOE_ERR_CUDA;
}

int32_t deamoe_last_launches(const deamoe_layer_t* L) { return L ? L->last_launches : 0; }

uint64_t deamoe_device_bytes(const deamoe_layer_t* L) { return L ? L->device_bytes : 0; }

#ifdef DEAMOE_TRACE
int deamoe_debug_ts(deamoe_layer_t* L, unsigned long long* host) {  // read and reset the step's stamps
  cudaDeviceSynchronize();
  cudaMemcpy(host, L->dev.ts, 24 * sizeof(unsigned long long), cudaMemcpyDeviceToHost);
  unsigned long long init[24];
  for (int i = 0; i < 24; ++i) init[i] = (i == 1 || i == 4 || i == 7 || i == 10 || i == 16) ? 0ull : ~0ull;
  cudaMemcpy(L->dev.ts, init, sizeof(init), cudaMemcpyHostToDevice);
  return 0;
}
int deamoe_debug_counts(deamoe_layer_t* L, int* host) {
  cudaDeviceSynchronize();
  cudaMemcpy(host, L->dev.counts, CNT_COUNT * sizeof(int), cudaMemcpyDeviceToHost);
  return 0;
}
int deamoe_debug_trace(deamoe_layer_t* L, long long* host, int max_ctas) {
  return (L && L->plan) ? deamoe::stream_read_trace(*L->plan, host, max_ctas) : 0;
}
#endif

const char* deamoe_status_string(deamoe_status_t st) {
  switch (st) {
    case DEAMOE_OK: return "ok";
    case DEAMOE_ERR_INTERNAL: return "device-side consistency check failed";
    case DEAMOE_ERR_INVALID_ARG: return "invalid argument";
    case DEAMOE_ERR_UNSUPPORTED: return "unsupported configuration";
    case DEAMOE_ERR_ALLOC: return "allocation failed";
    case DEAMOE_ERR_CUDA: return "CUDA runtime error";
    case DEAMOE_ERR_BATCH: return "batch size out of range";
    case DEAMOE_ERR_TIMEOUT: return "device-side wait timed out";
  }
  return "unknown status";
}

}  // extern "C"
