"""Thin ctypes binding of libdeamoe.so: argument marshalling only.

Every step of the layer runs in the library's CUDA kernels.  torch is used here for device
memory (tensors handed in by the caller) and for the current stream, nothing else.  If the
library has not been built the import of `lib()` raises -- there is no fallback.
"""
import ctypes as C
import os

import torch


_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdeamoe.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_ALLOC, ERR_CUDA, ERR_BATCH, ERR_TIMEOUT, ERR_INTERNAL = range(8)
DENSE_MIN_BATCH = 32   # calls of this many tokens and more take the dense schedule under SCHED_AUTO (csrc/dense.cuh) ...
DENSE_SMALL_ROUTER = 64  # ... twice as many on layers of fewer experts than this

F32, BF16 = 0, 1
SIGMA_NONE, SIGMA_SILU, SIGMA_GELU, SIGMA_RMSNORM = 0, 1, 2, 3
SCHED_AUTO, SCHED_PLAIN, SCHED_STAGED, SCHED_FUSED, SCHED_DENSE = 0, 1, 2, 3, 4


def dense_min_batch(shape):
    """Smallest call that SCHED_AUTO runs in the dense schedule on a layer of this shape (if it supports it)."""
    n = shape.n_dept * shape.experts_per_dept
    return DENSE_MIN_BATCH if n >= DENSE_SMALL_ROUTER else 2 * DENSE_MIN_BATCH


# every symbol include/deamoe.h declares
SYMBOLS = ("deamoe_layer_create", "deamoe_vanilla_create", "deamoe_layer_destroy", "deamoe_route",
           "deamoe_forward", "deamoe_vanilla_forward", "deamoe_forward_host", "deamoe_forward_partial",
           "deamoe_finish_partial", "deamoe_get_routing",
           "deamoe_get_stats", "deamoe_profile_enable", "deamoe_profile_last_ms", "deamoe_route_static", "deamoe_failure_test", "deamoe_probe_read",
           "deamoe_last_launches", "deamoe_device_bytes", "deamoe_status_string")


class Config(C.Structure):
    _fields_ = [(k, C.c_int32) for k in (
        "hidden", "n_dept", "experts_per_dept", "ffn", "priv", "top_k", "k_dept", "n_shared",
        "shared_ffn", "sigma", "norm_topk", "weight_dtype", "act_dtype", "residual", "max_batch",
        "schedule")] + [("route_scale", C.c_float), ("strict_dept", C.c_int32), ("dept_begin", C.c_int32),
                        ("dept_end", C.c_int32)]


class Weights(C.Structure):
    _fields_ = [(k, C.c_void_p) for k in (
        "router", "dept_gate", "dept_up", "dept_down", "priv_gate", "priv_up", "priv_down",
        "shared_gate", "shared_up", "shared_down")]


class DeaMoEError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status})")


_lib = None


def lib():
    """Load libdeamoe.so (built in-tree by build.py); raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2608_14385_b200.build` "
                              "(there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        for name in SYMBOLS:
            getattr(L, name)
        L.deamoe_status_string.restype = C.c_char_p
        L.deamoe_status_string.argtypes = [C.c_int]
        L.deamoe_last_launches.restype = C.c_int32
        L.deamoe_last_launches.argtypes = [C.c_void_p]
        L.deamoe_device_bytes.restype = C.c_uint64
        L.deamoe_device_bytes.argtypes = [C.c_void_p]
        for name in ("deamoe_layer_create", "deamoe_vanilla_create"):
            getattr(L, name).argtypes = [C.POINTER(Config), C.POINTER(Weights), C.c_void_p,
                                         C.POINTER(C.c_void_p)]
        L.deamoe_layer_destroy.argtypes = [C.c_void_p]
        L.deamoe_route.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]
        for name in ("deamoe_forward", "deamoe_vanilla_forward", "deamoe_forward_host"):
            getattr(L, name).argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p]
        L.deamoe_forward_partial.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p]
        L.deamoe_finish_partial.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p]
        L.deamoe_get_routing.argtypes = [C.c_void_p] * 9
        L.deamoe_get_stats.argtypes = [C.c_void_p] * 7
        L.deamoe_route_static.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32,
                                          C.c_int32, C.c_int32, C.c_float, C.c_int32, C.c_void_p, C.c_void_p]
        L.deamoe_failure_test.argtypes = [C.c_void_p, C.c_int32, C.c_int32]
        L.deamoe_probe_read.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_void_p]
        L.deamoe_profile_enable.argtypes = [C.c_void_p, C.c_int32]
        L.deamoe_profile_last_ms.argtypes = [C.c_void_p, C.POINTER(C.c_float)]
        _lib = L
    return _lib


def status_string(status):
    return lib().deamoe_status_string(int(status)).decode()


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _dptr(t):
    return C.c_void_p(t.data_ptr()) if t is not None else None


def make_config(shape, max_batch, schedule=SCHED_AUTO, dept_range=None):
    d = shape.asdict() if hasattr(shape, "asdict") else dict(shape)
    lo, hi = dept_range if dept_range is not None else (0, 0)
    return Config(d["hidden"], d["n_dept"], d["experts_per_dept"], d["ffn"], d["priv"], d["top_k"],
                  d.get("k_dept", 0), d.get("n_shared", 0), d.get("shared_ffn", 0), d.get("sigma", 1),
                  d.get("norm_topk", 1), d.get("weight_dtype", 1), d.get("act_dtype", 1),
                  d.get("residual", 0), int(max_batch), int(schedule), float(d.get("route_scale", 1.0)),
                  int(d.get("strict_dept", 0)), int(lo), int(hi))


STATIC_ROUTE_SCRATCH_BYTES = 4 << 20
PROBE_BLOCKS = 2368


def probe_read(buf, sink):
    """Enqueue one plain read of the CUDA tensor `buf` (deamoe_probe_read); sink: int32 CUDA tensor of
    at least PROBE_BLOCKS elements.  The caller times it with events."""
    assert buf.is_cuda and buf.is_contiguous() and sink.is_cuda and sink.numel() >= PROBE_BLOCKS
    st = lib().deamoe_probe_read(_stream(), _dptr(buf), buf.numel() * buf.element_size(), _dptr(sink))
    if st != OK:
        raise DeaMoEError(st, "deamoe_probe_read")



def route_static(router, tokens, n_dept, experts_per_dept, top_k, norm_topk=1, route_scale=1.0, idx=None, w=None):
    """Allocation-free routing (deamoe_route_static): for hosts that cannot create a layer object
    because they may not allocate device memory (graph capture, latency-critical loops, plug-ins
    working inside someone else's memory pool).  router [n, h] and tokens [B, h] are fp32 CUDA
    tensors; idx [B, k] int32 and w [B, k] fp32 are caller-provided outputs (made here only when
    omitted, for convenience in tests).  All calls share one fixed scratch array inside the library:
    do not overlap two calls on the GPU."""
    assert router.is_cuda and tokens.is_cuda and router.dtype == torch.float32 and tokens.dtype == torch.float32
    B, h = tokens.shape
    if idx is None:
        idx = torch.empty((B, top_k), dtype=torch.int32, device=tokens.device)
    if w is None:
        w = torch.empty((B, top_k), dtype=torch.float32, device=tokens.device)
    st = lib().deamoe_route_static(_stream(), _dptr(router), _dptr(tokens), n_dept, experts_per_dept, h, top_k,
                                   norm_topk, float(route_scale), B, _dptr(idx), _dptr(w))
    if st != OK:
        raise DeaMoEError(st, "deamoe_route_static")
    return idx, w


class Layer:
    """One DeaMoE (or vanilla MoE) layer living on the current CUDA device."""

    def __init__(self, shape, weights, max_batch, schedule=SCHED_AUTO, vanilla=False, dept_range=None):
        """weights: dict of CUDA tensors in the canonical layouts of include/deamoe.h.
        dept_range = (begin, end): this object is the slice of the layer holding those departments
        (the dept_* / priv_* tensors then hold only them); use forward_partial / finish_partial."""
        self.shape = shape
        self.vanilla = vanilla
        self.cfg = make_config(shape, max_batch, schedule, dept_range)
        if vanilla:
            self.cfg.priv = 0
        w = Weights()
        for name, _ in Weights._fields_:
            t = weights.get(name)
            if vanilla and name.startswith("priv_"):
                t = None
            if t is not None:
                assert t.is_cuda and t.is_contiguous(), name
            setattr(w, name, t.data_ptr() if t is not None else None)
        self._h = C.c_void_p()
        fn = lib().deamoe_vanilla_create if vanilla else lib().deamoe_layer_create
        st = fn(C.byref(self.cfg), C.byref(w), _stream(), C.byref(self._h))
        if st != OK:
            self._h = C.c_void_p()
            raise DeaMoEError(st, "deamoe_vanilla_create" if vanilla else "deamoe_layer_create")
        self.act = torch.float32 if self.cfg.act_dtype == F32 else torch.bfloat16

    def close(self):
        h = getattr(self, "_h", None)
        if h is not None and h.value and _lib is not None:
            _lib.deamoe_layer_destroy(h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check_tokens(self, tokens):
        assert tokens.is_cuda and tokens.is_contiguous() and tokens.dtype == self.act
        assert tokens.dim() == 2 and tokens.shape[1] == self.cfg.hidden
        return tokens.shape[0]

    def route(self, tokens, want_outputs=True):
        B = self._check_tokens(tokens)
        k = self.cfg.top_k
        idx = torch.empty((B, k), dtype=torch.int32, device=tokens.device) if want_outputs else None
        w = torch.empty((B, k), dtype=torch.float32, device=tokens.device) if want_outputs else None
        st = lib().deamoe_route(self._h, _stream(), _dptr(tokens), B, _dptr(idx), _dptr(w))
        if st != OK:
            raise DeaMoEError(st, "deamoe_route")
        return idx, w

    def forward(self, tokens, out=None):
        B = self._check_tokens(tokens)
        if out is None:
            out = torch.empty_like(tokens)
        fn = lib().deamoe_vanilla_forward if self.vanilla else lib().deamoe_forward
        st = fn(self._h, _stream(), _dptr(tokens), B, _dptr(out))
        if st != OK:
            raise DeaMoEError(st, "deamoe_forward")
        return out

    def forward_partial(self, tokens, partial=None):
        """fp32 partial sum of this layer object (a department slice, or a whole layer): [B, h]."""
        B = self._check_tokens(tokens)
        if partial is None:
            partial = torch.empty(tokens.shape, dtype=torch.float32, device=tokens.device)
        assert partial.is_cuda and partial.is_contiguous() and partial.dtype == torch.float32
        st = lib().deamoe_forward_partial(self._h, _stream(), _dptr(tokens), B, _dptr(partial))
        if st != OK:
            raise DeaMoEError(st, "deamoe_forward_partial")
        return partial

    def finish_partial(self, total, tokens, out=None):
        """out = total (+ tokens if residual) in the activation dtype; total: the slices' partial sums added."""
        B = self._check_tokens(tokens)
        if out is None:
            out = torch.empty_like(tokens)
        assert total.is_cuda and total.is_contiguous() and total.dtype == torch.float32
        st = lib().deamoe_finish_partial(self._h, _stream(), _dptr(total), _dptr(tokens), B, _dptr(out))
        if st != OK:
            raise DeaMoEError(st, "deamoe_finish_partial")
        return out

    def forward_host(self, tokens, out):
        """tokens/out: CPU tensors (pinned for speed) [B, h] in the activation dtype."""
        assert not tokens.is_cuda and not out.is_cuda and tokens.is_contiguous() and out.is_contiguous()
        st = lib().deamoe_forward_host(self._h, _stream(), C.c_void_p(tokens.data_ptr()), tokens.shape[0],
                                       C.c_void_p(out.data_ptr()))
        if st != OK:
            raise DeaMoEError(st, "deamoe_forward_host")
        return out

    def routing(self, B):
        """Host copy of the last call's routing state as numpy arrays."""
        import numpy as np
        m, n, k = self.cfg.n_dept, self.cfg.n_dept * self.cfg.experts_per_dept, self.cfg.top_k
        idx = np.zeros((B, k), np.int32)
        w = np.zeros((B, k), np.float32)
        mask = np.zeros(((m + 63) // 64,), np.uint64)
        doff = np.zeros((m + 1,), np.int32)
        dtok = np.full((max(1, B * min(k, m)),), -1, np.int32)
        eoff = np.zeros((n + 1,), np.int32)
        etok = np.full((max(1, B * k),), -1, np.int32)
        st = lib().deamoe_get_routing(self._h, _stream(), *(C.c_void_p(a.ctypes.data)
                                                           for a in (idx, w, mask, doff, dtok, eoff, etok)))
        if st != OK:
            raise DeaMoEError(st, "deamoe_get_routing")
        return {"idx": idx, "w": w, "dept_mask": mask, "dept_off": doff, "dept_tok": dtok[:doff[m]],
                "expert_off": eoff, "expert_tok": etok[:eoff[n]]}

    def stats(self):
        nd, ne, ntd, st_ = C.c_int32(), C.c_int32(), C.c_int32(), C.c_int32()
        ub = C.c_uint64()
        st = lib().deamoe_get_stats(self._h, _stream(), C.byref(nd), C.byref(ne), C.byref(ntd), C.byref(ub),
                                    C.byref(st_))
        if st != OK:
            raise DeaMoEError(st, "deamoe_get_stats")
        return {"active_dept": nd.value, "active_expert": ne.value, "token_dept_pairs": ntd.value,
                "unique_weight_bytes": ub.value, "device_status": st_.value}

    def failure_test(self, wait_limit=0, withhold=0):
        """Test aid (deamoe_failure_test): lower the poll limit of the bounded device-side waits
        and / or withhold a hand-over so that a wait expires; (0, 0) restores normal operation."""
        st = lib().deamoe_failure_test(self._h, int(wait_limit), int(withhold))
        if st != OK:
            raise DeaMoEError(st, "deamoe_failure_test")

    def profile(self, enable=True):
        """Record CUDA events around the weight-streaming launches of later forward calls."""
        st = lib().deamoe_profile_enable(self._h, 1 if enable else 0)
        if st != OK:
            raise DeaMoEError(st, "deamoe_profile_enable")

    def last_stream_ms(self):
        """Milliseconds between those events for the last forward (synchronises on it)."""
        ms = C.c_float()
        st = lib().deamoe_profile_last_ms(self._h, C.byref(ms))
        if st != OK:
            raise DeaMoEError(st, "deamoe_profile_last_ms")
        return ms.value

    @property
    def last_launches(self):
        return lib().deamoe_last_launches(self._h)

    @property
    def device_bytes(self):
        return lib().deamoe_device_bytes(self._h)
