"""ctypes front end of the fp64 CPU oracle -- TEST INFRASTRUCTURE.

Builds `deamoe_oracle.c` with gcc on first use and exposes its entry points on
numpy arrays.  bf16 data is passed as uint16 bit patterns (numpy has no bf16);
fp32 data as float32.  Only tests, the smoke check and the benchmark's
cpu_baseline leg may import this module; it imports nothing from the CUDA
package.
"""
import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "deamoe_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")

F32, BF16 = 0, 1
SIGMA_NONE, SIGMA_SILU, SIGMA_GELU, SIGMA_RMSNORM = 0, 1, 2, 3


class OracleConfig(C.Structure):
    _fields_ = [(k, C.c_int32) for k in (
        "hidden", "n_dept", "experts_per_dept", "ffn", "priv", "top_k", "k_dept", "n_shared",
        "shared_ffn", "sigma", "norm_topk", "weight_dtype", "act_dtype", "residual", "strict_dept")] + [
        ("route_scale", C.c_double), ("dept_begin", C.c_int32), ("dept_end", C.c_int32)]


class OracleWeights(C.Structure):
    _fields_ = [("router", C.c_void_p)] + [
        (k, C.POINTER(C.c_void_p)) for k in (
            "dept_gate", "dept_up", "dept_down", "priv_gate", "priv_up", "priv_down")] + [
        (k, C.c_void_p) for k in ("shared_gate", "shared_up", "shared_down")]


def build(force=False):
    """Compile the oracle with gcc (plain -O2, OpenMP for the row loops)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-shared", "-fPIC",
                               "-o", _LIB, _SRC, "-lm"])
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.oracle_set_threads.restype = C.c_int
        _lib.oracle_get_threads.restype = C.c_int
    return _lib


def set_threads(t):
    return lib().oracle_set_threads(int(t))


def host_cores():
    return len(os.sched_getaffinity(0))


def make_config(hidden, n_dept, experts_per_dept, ffn, priv, top_k, k_dept=0, n_shared=0,
                shared_ffn=0, sigma=SIGMA_SILU, norm_topk=1, weight_dtype=BF16, act_dtype=BF16,
                residual=0, route_scale=1.0, strict_dept=0, dept_range=None, **_ignored):
    """dept_range = (begin, end): the partial sum of that department slice (see deamoe_oracle.c)."""
    lo, hi = dept_range if dept_range is not None else (0, 0)
    return OracleConfig(hidden, n_dept, experts_per_dept, ffn, priv, top_k, k_dept, n_shared,
                        shared_ffn, sigma, norm_topk, weight_dtype, act_dtype, residual, strict_dept,
                        float(route_scale), int(lo), int(hi))


def _check(arr, dtype_code, what):
    want = np.float32 if dtype_code == F32 else np.uint16
    if arr.dtype != want or not arr.flags["C_CONTIGUOUS"]:
        raise TypeError(f"{what}: expected C-contiguous {want.__name__}, got {arr.dtype}")
    return arr


def _ptr(arr):
    return C.c_void_p(arr.ctypes.data)


def _table(entries, count, dtype_code, what):
    """entries: one [count, ...] array, or a sequence of `count` arrays / None."""
    tab = (C.c_void_p * count)()
    keep = []
    if entries is None:
        return None, keep
    for q in range(count):
        a = entries[q]
        if a is None:
            tab[q] = None
        else:
            a = _check(np.ascontiguousarray(a), dtype_code, what)
            keep.append(a)
            tab[q] = a.ctypes.data
    return tab, keep


def make_weights(cfg, w, per_expert_dept_tables=False):
    """w: dict with router [n,h] f32, dept_gate/up/down, priv_gate/up/down
    (arrays or sequences, entries may be None), shared_gate/up/down."""
    m, g = cfg.n_dept, cfg.experts_per_dept
    n = m * g
    keep = []
    ow = OracleWeights()
    router = _check(np.ascontiguousarray(w["router"]), F32, "router")
    keep.append(router)
    ow.router = router.ctypes.data
    n_dept_entries = n if per_expert_dept_tables else m
    for name in ("dept_gate", "dept_up", "dept_down"):
        tab, k2 = _table(w[name], n_dept_entries, cfg.weight_dtype, name)
        keep += k2 + [tab]
        setattr(ow, name, C.cast(tab, C.POINTER(C.c_void_p)))
    for name in ("priv_gate", "priv_up", "priv_down"):
        tab, k2 = _table(w.get(name) if cfg.priv > 0 else None, n, cfg.weight_dtype, name)
        keep += k2 + [tab]
        if tab is not None:
            setattr(ow, name, C.cast(tab, C.POINTER(C.c_void_p)))
    for name in ("shared_gate", "shared_up", "shared_down"):
        if cfg.n_shared:
            a = _check(np.ascontiguousarray(w[name]), cfg.weight_dtype, name)
            keep.append(a)
            setattr(ow, name, a.ctypes.data)
    return ow, keep


def route(cfg, router, tokens, want_logits=False):
    """Eq. (2) + gate weights.  Returns dict(idx [B,k] i32, w [B,k] f64, gap [B] f64, gap_parts [B,3]
    f64, logits?).  gap is the smallest margin of any comparison that decided the token's selection
    (gap_parts: among the sorted candidates / at the department cut / at a strict-coverage
    replacement); a test that compares an fp32 router bit for bit requires it to be clear of zero."""
    tokens = _check(np.ascontiguousarray(tokens), cfg.act_dtype, "tokens")
    router = _check(np.ascontiguousarray(router), F32, "router")
    B, k, n = tokens.shape[0], cfg.top_k, cfg.n_dept * cfg.experts_per_dept
    idx = np.zeros((B, k), np.int32)
    p = np.zeros((B, k), np.float64)
    gap = np.zeros((B,), np.float64)
    parts = np.zeros((B, 3), np.float64)
    logits = np.zeros((B, n), np.float64) if want_logits else None
    rc = lib().oracle_route(C.byref(cfg), _ptr(router), _ptr(tokens), C.c_int(B), _ptr(idx), _ptr(p),
                            _ptr(logits) if want_logits else None, _ptr(gap), _ptr(parts))
    if rc:
        raise RuntimeError(f"oracle_route failed: {rc}")
    out = {"idx": idx, "w": p, "gap": gap, "gap_parts": parts}
    if want_logits:
        out["logits"] = logits
    return out


def bucket(cfg, topk_idx):
    """Section 3.2 department / expert token lists."""
    topk_idx = np.ascontiguousarray(topk_idx, np.int32)
    B, k = topk_idx.shape
    m, n = cfg.n_dept, cfg.n_dept * cfg.experts_per_dept
    mask = np.zeros(((m + 63) // 64,), np.uint64)
    dept_off = np.zeros((m + 1,), np.int32)
    dept_tok = np.full((max(1, B * min(k, m)),), -1, np.int32)
    expert_off = np.zeros((n + 1,), np.int32)
    expert_tok = np.full((max(1, B * k),), -1, np.int32)
    rc = lib().oracle_bucket(C.byref(cfg), _ptr(topk_idx), C.c_int(B), _ptr(mask), _ptr(dept_off),
                             _ptr(dept_tok), _ptr(expert_off), _ptr(expert_tok))
    if rc:
        raise RuntimeError(f"oracle_bucket failed: {rc}")
    return {"dept_mask": mask, "dept_off": dept_off, "dept_tok": dept_tok[:dept_off[m]],
            "expert_off": expert_off, "expert_tok": expert_tok[:expert_off[n]]}


def _forward(fn, cfg, w, tokens, rows, per_expert):
    tokens = _check(np.ascontiguousarray(tokens), cfg.act_dtype, "tokens")
    B, h, k = tokens.shape[0], cfg.hidden, cfg.top_k
    ow, keep = make_weights(cfg, w, per_expert_dept_tables=per_expert)
    out = np.zeros((B, h), np.float64)
    idx = np.zeros((B, k), np.int32)
    p = np.zeros((B, k), np.float64)
    if rows is not None:
        rows = np.ascontiguousarray(rows, np.int32)
    rc = fn(C.byref(cfg), C.byref(ow), _ptr(tokens), C.c_int(B),
            _ptr(rows) if rows is not None else None,
            C.c_int(0 if rows is None else len(rows)), _ptr(out), _ptr(idx), _ptr(p))
    del keep
    if rc:
        raise RuntimeError(f"oracle forward failed: {rc} (2 = a needed weight entry was None)")
    return {"out": out, "idx": idx, "w": p}


def deamoe_forward(cfg, w, tokens, rows=None):
    """DeaMoE layer output [B,h] fp64 (rows: optional subset of tokens to evaluate)."""
    return _forward(lib().oracle_deamoe_forward, cfg, w, tokens, rows, False)


def vanilla_forward(cfg, w, tokens, rows=None):
    """Standard MoE layer; w['dept_*'] hold n per-expert matrices."""
    return _forward(lib().oracle_vanilla_forward, cfg, w, tokens, rows, True)


def swiglu(Wg, Wu, Wd, dtype_code, x):
    """Eq. (1) on one fp64 vector."""
    f, h = Wg.shape
    x = np.ascontiguousarray(x, np.float64)
    out = np.zeros((h,), np.float64)
    arrs = [_check(np.ascontiguousarray(a), dtype_code, "W") for a in (Wg, Wu, Wd)]
    rc = lib().oracle_swiglu(_ptr(arrs[0]), _ptr(arrs[1]), _ptr(arrs[2]), C.c_int(dtype_code),
                             C.c_int(h), C.c_int(f), _ptr(x), _ptr(out))
    if rc:
        raise RuntimeError(f"oracle_swiglu failed: {rc}")
    return out


def deamoe_expert(cfg, Wg, Wu, Wd, Ag, Au, Ad, x, taps=False):
    """Eq. (4) on one fp64 vector; with taps also G, U, Y, Z of Section 3.2."""
    h, f = cfg.hidden, cfg.ffn
    r = cfg.priv if cfg.priv > 0 else f
    x = np.ascontiguousarray(x, np.float64)
    out = np.zeros((h,), np.float64)
    dt = cfg.weight_dtype
    arrs = [None if a is None else _check(np.ascontiguousarray(a), dt, "W")
            for a in (Wg, Wu, Wd, Ag, Au, Ad)]
    ptrs = [None if a is None else _ptr(a) for a in arrs]
    G, U, Y, Z = (np.zeros((f,)), np.zeros((f,)), np.zeros((r,)), np.zeros((f,)))
    rc = lib().oracle_deamoe_expert(C.byref(cfg), *ptrs, _ptr(x), _ptr(out),
                                    *([_ptr(G), _ptr(U), _ptr(Y), _ptr(Z)] if taps else [None] * 4))
    if rc:
        raise RuntimeError(f"oracle_deamoe_expert failed: {rc}")
    return (out, G, U, Y, Z) if taps else out
