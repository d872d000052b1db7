"""The C-ABI library loads and exports every symbol the header declares (no GPU needed)."""
import ctypes
import os
import re

from paper_2608_14385_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "deamoe.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(deamoe_[a-z_]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    path = build.build()
    lib = ctypes.CDLL(path)
    names = _declared()
    assert len(names) >= 12
    for name in names:
        assert hasattr(lib, name), name
    assert sorted(binding.SYMBOLS) == names


def test_status_strings_and_host_side_argument_errors():
    L = binding.lib()
    assert binding.status_string(binding.OK) == "ok"
    for code in range(1, 7):
        assert binding.status_string(code) not in ("", "ok")
    # NULL arguments are rejected on the host before any CUDA call
    out = ctypes.c_void_p()
    assert L.deamoe_layer_create(None, None, None, ctypes.byref(out)) == binding.ERR_INVALID_ARG
    assert L.deamoe_forward(None, None, None, 1, None) == binding.ERR_INVALID_ARG
    assert L.deamoe_layer_destroy(None) == binding.OK
    cfg = binding.Config(hidden=64, n_dept=2, experts_per_dept=2, ffn=32, priv=16, top_k=5, max_batch=4)
    w = binding.Weights(router=1, dept_gate=1, dept_up=1, dept_down=1, priv_gate=1, priv_up=1, priv_down=1)
    assert L.deamoe_layer_create(ctypes.byref(cfg), ctypes.byref(w), None, ctypes.byref(out)) == binding.ERR_INVALID_ARG
    cfg.top_k = 2
    cfg.max_batch = 100000
    assert L.deamoe_layer_create(ctypes.byref(cfg), ctypes.byref(w), None, ctypes.byref(out)) == binding.ERR_BATCH
    cfg.max_batch = 4
    w.priv_gate = None
    assert L.deamoe_layer_create(ctypes.byref(cfg), ctypes.byref(w), None, ctypes.byref(out)) == binding.ERR_INVALID_ARG
    w.priv_gate = 1
    for field, bad in (("norm_topk", 3), ("norm_topk", -1), ("sigma", 4)):
        good = getattr(cfg, field)
        setattr(cfg, field, bad)
        assert L.deamoe_layer_create(ctypes.byref(cfg), ctypes.byref(w), None, ctypes.byref(out)) == binding.ERR_INVALID_ARG
        setattr(cfg, field, good)


def test_misaligned_device_pointers_are_argument_errors_without_a_gpu():
    """deamoe_route_static checks its arguments before it touches CUDA: pointers that are not
    aligned for the kernels' 16-byte accesses come back as INVALID_ARG and nothing is enqueued (the
    same check in deamoe_route / deamoe_forward needs a layer object and runs in the GPU tests)."""
    L = binding.lib()
    p = ctypes.c_void_p

    def call(router, tokens, idx, w):
        return L.deamoe_route_static(None, p(router), p(tokens), 4, 4, 1024, 2, 1, 1.0, 4, p(idx), p(w))
    assert call(4096 + 4, 8192, 12288, 16384) == binding.ERR_INVALID_ARG      # router
    assert call(4096, 8192 + 8, 12288, 16384) == binding.ERR_INVALID_ARG      # tokens
    assert call(4096, 8192, 12288 + 2, 16384) == binding.ERR_INVALID_ARG      # topk_idx
    assert call(4096, 8192, 12288, 16384 + 1) == binding.ERR_INVALID_ARG      # topk_w
    assert binding.ERR_INTERNAL == 7 and binding.status_string(binding.ERR_INTERNAL) not in ("", "ok", "unknown status")
