"""deamoe_route_static: routing for hosts that cannot allocate device memory.

Some users of the library only have a stream and buffers they were given -- they run inside a CUDA
graph capture, inside a serving loop where an allocation would stall the device, or inside another
framework's memory pool -- so they cannot build a layer object, which allocates its workspace.  The
allocation-free entry point keeps its only scratch (the partial router logits) in a fixed array inside
the library.  This test calls it through the C ABI and checks it against the ordinary entry point
(deamoe_route on a layer object) on the same router and tokens: expert indices bit for bit, gate
weights within the 1e-5 the routing tests use.  It runs two calls back to back on different batches,
so the second call sees the first call's leftovers in the shared scratch.  The file is named to be
collected last: a failure here cannot hide a failure of any other test in a run that stops early.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2608_14385_b200 import binding, synth

pytestmark = pytest.mark.gpu

SHAPE = synth.LayerShape("noalloc", hidden=512, n_dept=8, experts_per_dept=8, ffn=64, priv=16, top_k=6,
                         act_dtype=0)


def _reference(layer, tokens):
    idx, w = layer.route(tokens)
    torch.cuda.synchronize()
    return idx.cpu().numpy(), w.cpu().numpy()


def test_static_routing_matches_layer_routing_on_two_consecutive_calls():
    dev = torch.device("cuda:0")
    weights = synth.make_deamoe_weights(SHAPE, 21, dev)
    layer = binding.Layer(SHAPE, weights, 32)
    try:
        batches = [synth.make_tokens(SHAPE, 32, 22, dev), synth.make_tokens(SHAPE, 5, 23, dev)]
        want = [_reference(layer, b) for b in batches]
        # caller-owned outputs, made before the calls: the entry point itself allocates nothing
        outs = [(torch.full((b.shape[0], SHAPE.top_k), -1, dtype=torch.int32, device=dev),
                 torch.full((b.shape[0], SHAPE.top_k), -1.0, dtype=torch.float32, device=dev)) for b in batches]
        for b, (idx, w) in zip(batches, outs):        # two calls in a row, no synchronisation between them
            binding.route_static(weights["router"], b, SHAPE.n_dept, SHAPE.experts_per_dept, SHAPE.top_k,
                                 idx=idx, w=w)
        torch.cuda.synchronize()
        for (idx, w), (widx, ww) in zip(outs, want):
            assert (idx.cpu().numpy() == widx).all()
            assert np.abs(w.cpu().numpy() - ww).max() <= 1e-5
            assert np.abs(w.cpu().numpy().sum(axis=1) - 1.0).max() <= 1e-5
    finally:
        layer.close()


def test_static_routing_rejects_what_does_not_fit_and_bad_arguments():
    dev = torch.device("cuda:0")
    L = binding.lib()
    router = torch.zeros((2048, 1024), dtype=torch.float32, device=dev)
    tokens = torch.zeros((1024, 1024), dtype=torch.float32, device=dev)
    idx = torch.zeros((1024, 4), dtype=torch.int32, device=dev)
    w = torch.zeros((1024, 4), dtype=torch.float32, device=dev)

    def call(n_dept, g, h, k, B, r=router, t=tokens):
        return L.deamoe_route_static(None, ctypes.c_void_p(r.data_ptr()), ctypes.c_void_p(t.data_ptr()), n_dept, g, h,
                                     k, 1, 1.0, B, ctypes.c_void_p(idx.data_ptr()), ctypes.c_void_p(w.data_ptr()))
    assert call(256, 8, 1024, 4, 1024) == binding.ERR_BATCH          # 2048 experts x 1024 tokens: beyond the array
    assert call(256, 8, 1024, 4, 0) == binding.OK                    # empty batch: nothing to do
    assert call(0, 8, 1024, 4, 4) == binding.ERR_INVALID_ARG
    assert call(2, 2, 1024, 5, 4) == binding.ERR_INVALID_ARG         # top_k > n
    assert call(256, 8, 1022, 4, 4) == binding.ERR_UNSUPPORTED       # hidden not a multiple of 4
    assert L.deamoe_route_static(None, None, None, 4, 4, 1024, 2, 1, 1.0, 4, None, None) == binding.ERR_INVALID_ARG
    torch.cuda.synchronize()
