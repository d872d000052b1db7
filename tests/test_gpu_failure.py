"""Failure detection on the device, without faulting or hanging anything.

Every device-side wait of the library is bounded.  These tests make such a wait run out in the only
way that needs no fault: the host withholds a hand-over (deamoe_failure_test) and lowers the poll
limit, the kernel gives up by itself, and the host reads DEAMOE_ERR_TIMEOUT from the status word.
The context stays usable: the same layer, switched back to normal operation, and a fresh layer both
give correct results afterwards."""
import ctypes

import numpy as np
import pytest
import torch

from paper_2608_14385_b200 import binding, synth
from tests.gpu_common import run_case

pytestmark = pytest.mark.gpu

SHAPE = synth.LayerShape("fail", hidden=256, n_dept=4, experts_per_dept=4, ffn=128, priv=64, top_k=3,
                         n_shared=1, shared_ffn=128)


def _weights(shape, seed):
    w = synth.make_deamoe_weights(shape, seed, "cuda:0")
    for k in w:
        w[k] = (w[k].float() * 12.0).to(w[k].dtype) if k != "router" else w[k] * 4.0
    return w


@pytest.mark.parametrize("shared", [1, 0])
def test_streaming_kernel_wait_expires_when_the_work_list_is_withheld(shared):
    """Fused schedule: the routing kernel normally raises two flags that hand the work list to the
    persistent streaming kernel.  Withheld, the kernel's planners poll until the (lowered) limit,
    report DEAMOE_ERR_TIMEOUT and every role of every thread block leaves."""
    shape = SHAPE.with_(n_shared=shared, shared_ffn=128 if shared else 0)
    w = _weights(shape, 31)
    layer = binding.Layer(shape, w, 8, binding.SCHED_FUSED)
    try:
        tokens = synth.make_tokens(shape, 5, 31, "cuda:0")
        good = layer.forward(tokens).clone()
        torch.cuda.synchronize()
        assert layer.stats()["device_status"] == binding.OK
        layer.failure_test(wait_limit=1 << 14, withhold=1)
        layer.forward(tokens)
        torch.cuda.synchronize()                      # the kernel returns by itself
        assert layer.stats()["device_status"] == binding.ERR_TIMEOUT
        layer.failure_test(0, 0)                      # back to normal: the same layer is usable again
        again = layer.forward(tokens)
        torch.cuda.synchronize()
        assert layer.stats()["device_status"] == binding.OK
        assert torch.equal(again, good)
        run_case(shape, 5, weights=w, tokens=tokens, layer=layer)
    finally:
        layer.close()
    run_case(shape, 7, seed=32, weights=w, schedule=binding.SCHED_FUSED)     # a fresh layer after the failure


def test_dense_kernel_wait_expires_when_its_copies_are_withheld():
    """Dense schedule: the copy role of the tcgen05 kernel issues nothing, so the role that issues the
    MMAs waits for the ring until the limit, the kernel reports DEAMOE_ERR_TIMEOUT, frees its tensor
    memory and returns."""
    shape = synth.LayerShape("faild", hidden=256, n_dept=2, experts_per_dept=4, ffn=128, priv=64, top_k=2,
                             n_shared=1, shared_ffn=128)
    w = _weights(shape, 33)
    layer = binding.Layer(shape, w, 64, binding.SCHED_DENSE)
    try:
        tokens = synth.make_tokens(shape, 64, 33, "cuda:0")
        good = layer.forward(tokens).clone()
        torch.cuda.synchronize()
        assert layer.stats()["device_status"] == binding.OK
        layer.failure_test(wait_limit=1 << 12, withhold=2)
        layer.forward(tokens)
        torch.cuda.synchronize()
        assert layer.stats()["device_status"] == binding.ERR_TIMEOUT
        layer.failure_test(0, 0)
        again = layer.forward(tokens)
        torch.cuda.synchronize()
        assert layer.stats()["device_status"] == binding.OK
        assert torch.equal(again, good)               # tensor memory was freed: the next launch allocates it again
        run_case(shape, 64, weights=w, tokens=tokens, layer=layer)
    finally:
        layer.close()


@pytest.mark.parametrize("schedule", [binding.SCHED_STAGED, binding.SCHED_FUSED])
def test_out_of_range_pair_slot_is_skipped_and_reported(schedule):
    """The combine kernel checks every pair slot before it uses it as a row index.  With a planted
    out-of-range slot for pair (token 0, first expert) it must skip that row (no access), report
    DEAMOE_ERR_INTERNAL, and leave every other token's output exactly as in a normal step."""
    w = _weights(SHAPE, 36)
    layer = binding.Layer(SHAPE, w, 8, schedule)
    try:
        tokens = synth.make_tokens(SHAPE, 6, 36, "cuda:0")
        good = layer.forward(tokens).clone()
        torch.cuda.synchronize()
        layer.failure_test(0, 4)
        bad = layer.forward(tokens).clone()
        torch.cuda.synchronize()
        assert layer.stats()["device_status"] == binding.ERR_INTERNAL
        assert torch.equal(bad[1:], good[1:])             # the other tokens are untouched
        assert not torch.equal(bad[0], good[0])           # token 0 lost one expert's term
        assert torch.isfinite(bad.float()).all()
        layer.failure_test(0, 0)
        assert torch.equal(layer.forward(tokens), good)
        torch.cuda.synchronize()
        assert layer.stats()["device_status"] == binding.OK
    finally:
        layer.close()


def test_failure_test_is_refused_where_there_is_no_such_hand_over():
    w = _weights(SHAPE, 34)
    for sched, withhold in ((binding.SCHED_PLAIN, 1), (binding.SCHED_STAGED, 1), (binding.SCHED_FUSED, 2)):
        layer = binding.Layer(SHAPE, w, 8, sched)
        try:
            with pytest.raises(binding.DeaMoEError) as e:
                layer.failure_test(1 << 12, withhold)
            assert e.value.status == binding.ERR_UNSUPPORTED
            layer.failure_test(1 << 20, 0)            # a lower limit alone is accepted and changes no result
            run_case(SHAPE, 4, weights=w, layer=layer)
        finally:
            layer.close()
    assert binding.lib().deamoe_failure_test(None, 0, 0) == binding.ERR_INVALID_ARG


def test_misaligned_device_pointers_are_rejected_before_anything_is_enqueued():
    """Tokens and outputs are read and written with 16-byte accesses; a pointer that is not 16-byte
    aligned is an argument error on the host, not a fault on the device."""
    shape = SHAPE
    w = _weights(shape, 35)
    layer = binding.Layer(shape, w, 8)
    try:
        B, h = 4, shape.hidden
        flat = torch.zeros(B * h + 16, dtype=torch.bfloat16, device="cuda:0")
        good_in, good_out = flat[:B * h].view(B, h), torch.empty((B, h), dtype=torch.bfloat16, device="cuda:0")
        bad = flat[1:1 + B * h].view(B, h)            # 2 bytes off
        L = binding.lib()
        p = lambda t: ctypes.c_void_p(t.data_ptr())
        assert L.deamoe_forward(layer._h, None, p(bad), B, p(good_out)) == binding.ERR_INVALID_ARG
        assert L.deamoe_forward(layer._h, None, p(good_in), B, p(bad)) == binding.ERR_INVALID_ARG
        assert L.deamoe_route(layer._h, None, p(bad), B, None, None) == binding.ERR_INVALID_ARG
        idx = torch.zeros(B * shape.top_k + 2, dtype=torch.int16, device="cuda:0")
        assert L.deamoe_route(layer._h, None, p(good_in), B, p(idx[1:]), None) == binding.ERR_INVALID_ARG
        assert L.deamoe_forward(layer._h, None, p(good_in), B, p(good_out)) == binding.OK
        torch.cuda.synchronize()
        assert layer.stats()["device_status"] == binding.OK
    finally:
        layer.close()
