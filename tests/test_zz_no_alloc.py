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

from oracle import ref
from paper_2608_14385_b200 import binding, synth
from tests.common import oracle_cfg

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
        cfg = oracle_cfg(SHAPE)
        for b, (idx, w), (widx, ww) in zip(batches, outs, want):
            assert (idx.cpu().numpy() == widx).all()
            assert np.abs(w.cpu().numpy() - ww).max() <= 1e-5
            assert np.abs(w.cpu().numpy().sum(axis=1) - 1.0).max() <= 1e-5
            # ... and against the fp64 oracle (Eq. (2), ties to the lower index; gate weights of Eq. (3))
            o = ref.route(cfg, synth.to_numpy(weights["router"]), synth.to_numpy(b), want_logits=True)
            assert (o["gap"] > 1e-5 * np.abs(o["logits"]).max(axis=1)).all(), "seed too close to a routing tie"
            assert (idx.cpu().numpy() == o["idx"]).all()
            assert np.abs(w.cpu().numpy().astype(np.float64) - o["w"]).max() <= 1e-5
    finally:
        layer.close()


def test_static_routing_on_the_multi_slice_layout_against_the_oracle():
    """The documented large use: the DeepSeek-V3 router (256 experts, hidden 7168, top-8) takes 8
    column slices, so the fixed array holds part[slice][B][n] with a stride that depends on the call's
    B.  512 tokens fill the 4 MiB exactly; a call with 3 tokens right behind it (no synchronisation)
    reads slices that lie between leftovers of the first.  Both are compared bit for bit with the
    oracle and with a layer object's routing (same slice rule, so the same fp32 sums); 513 tokens do
    not fit and are refused."""
    shape = synth.LayerShape("noalloc-dsv3", hidden=7168, n_dept=32, experts_per_dept=8, ffn=16, priv=16, top_k=8,
                             act_dtype=0)
    dev = torch.device("cuda:0")
    weights = synth.make_deamoe_weights(shape, 24, dev)
    big, small = synth.make_tokens(shape, 512, 25, dev), synth.make_tokens(shape, 3, 26, dev)
    outs = [(torch.full((b.shape[0], shape.top_k), -1, dtype=torch.int32, device=dev),
             torch.full((b.shape[0], shape.top_k), -1.0, dtype=torch.float32, device=dev)) for b in (big, small)]
    for b, (idx, w) in zip((big, small), outs):
        binding.route_static(weights["router"], b, shape.n_dept, shape.experts_per_dept, shape.top_k, idx=idx, w=w)
    torch.cuda.synchronize()
    cfg = oracle_cfg(shape)
    layer = binding.Layer(shape, weights, 128)
    try:
        for b, (idx, w) in zip((big, small), outs):
            o = ref.route(cfg, synth.to_numpy(weights["router"]), synth.to_numpy(b), want_logits=True)
            safe = o["gap"] > 1e-5 * np.abs(o["logits"]).max(axis=1)
            assert safe.mean() > 0.97                  # 512 tokens: a few may sit within rounding of a tie
            assert (idx.cpu().numpy()[safe] == o["idx"][safe]).all()
            assert np.abs(w.cpu().numpy().astype(np.float64) - o["w"])[safe].max() <= 1e-5
            for s0 in range(0, b.shape[0], 128):       # the layer object takes at most 128 tokens per call
                part = b[s0:s0 + 128].contiguous()
                lidx, lw = layer.route(part)
                torch.cuda.synchronize()
                assert torch.equal(lidx, idx[s0:s0 + 128])
                assert (lw - w[s0:s0 + 128]).abs().max().item() <= 1e-6
    finally:
        layer.close()
    too_many = torch.zeros((513, shape.hidden), dtype=torch.float32, device=dev)
    with pytest.raises(binding.DeaMoEError) as e:
        binding.route_static(weights["router"], too_many, shape.n_dept, shape.experts_per_dept, shape.top_k)
    assert e.value.status == binding.ERR_BATCH


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
