"""Department-sharded execution on the GPU: the slices of a layer (paper Section 3.1: a department and
its experts' private matrices are an independent unit) are created as separate layer objects, each from
ITS slice of the weights only; here they run one after another on one GPU (they do not wait on one
another: the only exchange is the sum of their fp32 partial outputs, which an all-reduce does across
GPUs and a plain addition does here).  Every slice's partial sum is compared with the oracle's partial
sum of the same slice, the finished output with the oracle's unsharded layer."""
import ctypes

import numpy as np
import pytest
import torch

from oracle import accounting, ref
from paper_2608_14385_b200 import binding, shard, synth
from tests.common import within_tolerance

pytestmark = pytest.mark.gpu

SHAPE = synth.LayerShape("shard", hidden=256, n_dept=5, experts_per_dept=4, ffn=128, priv=64, top_k=4,
                         n_shared=1, shared_ffn=128, residual=1)


def _scale(w):
    for k in w:
        w[k] = (w[k].float() * 12.0).to(w[k].dtype) if k != "router" else w[k] * 4.0
    return w


def _host_tables(shape, w, lo, hi):
    g = shape.experts_per_dept
    host = {"router": synth.to_numpy(w["router"])}
    for name in ("gate", "up", "down"):
        host[f"dept_{name}"] = [synth.to_numpy(w[f"dept_{name}"][j - lo]) if lo <= j < hi else None
                                for j in range(shape.n_dept)]
        if shape.priv > 0:
            host[f"priv_{name}"] = [synth.to_numpy(w[f"priv_{name}"][i - lo * g]) if lo <= i // g < hi else None
                                    for i in range(shape.n_expert)]
        if f"shared_{name}" in w:
            host[f"shared_{name}"] = synth.to_numpy(w[f"shared_{name}"])
    return host


def _run_sharded(shape, world, B, schedule, seed, max_batch=None):
    dev = torch.device("cuda:0")
    tokens = synth.make_tokens(shape, B, seed, dev)
    whole = _scale(synth.make_deamoe_weights(shape, seed, dev))
    full = ref.deamoe_forward(ref.make_config(**shape.asdict()), {k: synth.to_numpy(v) for k, v in whole.items()},
                              synth.to_numpy(tokens))
    g = shape.experts_per_dept
    total = torch.zeros((B, shape.hidden), dtype=torch.float32, device=dev)
    layers, stats = [], []
    try:
        for r in range(world):
            my_shape, (lo, hi) = shard.slice_shape(shape, r, world)
            w = _scale(synth.make_deamoe_weights(my_shape, seed, dev, dept_range=(lo, hi)))
            layer = binding.Layer(my_shape, w, max_batch or B, schedule, dept_range=(lo, hi))
            layers.append(layer)
            part = layer.forward_partial(tokens)
            torch.cuda.synchronize()
            st = layer.stats()
            assert st["device_status"] == 0
            rt = layer.routing(B)
            assert (rt["idx"] == full["idx"]).all()                               # every slice routes alike
            mine = [[int(i) for i in row if lo <= int(i) // g < hi] for row in full["idx"]]
            nd, ne, pairs = accounting.count_active(mine, g)
            assert (st["active_dept"], st["active_expert"], st["token_dept_pairs"]) == (nd, ne, pairs)
            assert st["unique_weight_bytes"] == accounting.unique_bytes_deamoe(
                nd, ne, shape.hidden, shape.ffn, shape.priv, shape.n_expert, 2, my_shape.n_shared, my_shape.shared_ffn)
            # this slice's department sets and token lists: the oracle's bucketing of its own pairs
            for j in range(shape.n_dept):
                toks = rt["dept_tok"][rt["dept_off"][j]:rt["dept_off"][j + 1]]
                want = [t for t in range(B) if any(int(i) // g == j for i in mine[t])]
                assert list(toks) == want
            want_part = ref.deamoe_forward(
                ref.make_config(**my_shape.with_(residual=0).asdict(), dept_range=(lo, hi)),
                _host_tables(my_shape, w, lo, hi), synth.to_numpy(tokens))
            ok, err, bound = within_tolerance(part.cpu().numpy(), want_part["out"],
                                              abs_=1e-3 + 1e-2 * float(np.abs(full["out"]).max()))
            assert ok, (r, err, bound)
            total += part                                                         # across GPUs: the all-reduce
            stats.append(st)
        out = layers[0].finish_partial(total, tokens)
        torch.cuda.synchronize()
        ok, err, bound = within_tolerance(out.float().cpu().numpy(), full["out"])
        assert ok, (err, bound)
        return out, stats, layers
    finally:
        for layer in layers:
            layer.close()


@pytest.mark.parametrize("schedule", [binding.SCHED_PLAIN, binding.SCHED_STAGED, binding.SCHED_FUSED])
@pytest.mark.parametrize("world,B", [(2, 6), (3, 1), (5, 9)])
def test_slices_of_a_layer_add_up_to_the_layer(schedule, world, B):
    """2, 3 and 5 slices of a 5-department layer (the last with one department each; with one token
    some slices receive nothing at all)."""
    _run_sharded(SHAPE, world, B, schedule, seed=40 + world)


def test_slices_on_the_dense_schedule():
    shape = SHAPE.with_(n_dept=4, top_k=3)
    _run_sharded(shape, 2, 64, binding.SCHED_DENSE, seed=45, max_batch=64)


def test_slices_of_a_benchmark_sized_cut():
    """Two slices of the 1.1 GB cut of the DeepSeek-V3 shape (8 departments x 4 experts, shared expert)."""
    _run_sharded(synth.DSV3_MINI.with_(residual=1), 2, 8, binding.SCHED_AUTO, seed=46)


def test_slice_objects_refuse_what_only_a_whole_layer_can_do():
    dev = torch.device("cuda:0")
    my_shape, (lo, hi) = shard.slice_shape(SHAPE, 0, 2)
    w = _scale(synth.make_deamoe_weights(my_shape, 47, dev, dept_range=(lo, hi)))
    layer = binding.Layer(my_shape, w, 4, dept_range=(lo, hi))
    try:
        tokens = synth.make_tokens(SHAPE, 4, 47, dev)
        with pytest.raises(binding.DeaMoEError) as e:
            layer.forward(tokens)
        assert e.value.status == binding.ERR_INVALID_ARG
    finally:
        layer.close()
    for bad in ((2, 2), (3, 2), (0, 6), (-1, 2)):
        with pytest.raises(binding.DeaMoEError) as e:
            binding.Layer(my_shape, w, 4, dept_range=bad)
        assert e.value.status == binding.ERR_INVALID_ARG
    # a whole layer's partial output + finish equals its ordinary output
    whole = _scale(synth.make_deamoe_weights(SHAPE, 47, dev))
    layer = binding.Layer(SHAPE, whole, 4)
    try:
        tokens = synth.make_tokens(SHAPE, 4, 47, dev)
        direct = layer.forward(tokens).clone()
        via = layer.finish_partial(layer.forward_partial(tokens), tokens)
        torch.cuda.synchronize()
        assert torch.equal(direct, via)
    finally:
        layer.close()
