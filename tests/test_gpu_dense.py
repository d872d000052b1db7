"""Dense schedule (tcgen05 kernels for the department and shared-expert matrices, Section 3.2 at
larger batches): element-by-element parity with the fp64 oracle, and agreement with the streaming
schedule."""
import numpy as np
import pytest
import torch

from paper_2608_14385_b200 import binding, synth
from tests.common import within_tolerance
from tests.gpu_common import run_case

pytestmark = pytest.mark.gpu

# h a multiple of the 256-row tile, f and shared_ffn of 128; three departments, so 100 tokens put more
# than 64 (one accumulator's worth of) rows into a department's bucket and into the shared expert's.
# So few tiles that all of them are split into half-tile jobs.
DENSE_SMALL = synth.LayerShape("dense-small", hidden=256, n_dept=3, experts_per_dept=4, ffn=128, priv=32, top_k=3,
                               n_shared=1, shared_ffn=256)
# several row tiles per matrix, a contraction that spans the ring more than once, f not a multiple of
# 256 (a tile of the stacked gate / up matrix holds rows of both)
DENSE_WIDE = synth.LayerShape("dense-wide", hidden=1024, n_dept=4, experts_per_dept=4, ffn=384, priv=64, top_k=4,
                              n_shared=1, shared_ffn=128)


def _scaled(shape, seed, scale=12.0):
    dev = torch.device("cuda:0")
    w = synth.make_deamoe_weights(shape, seed, dev)
    for k in w:
        w[k] = (w[k].float() * scale).to(w[k].dtype) if k != "router" else w[k] * 4.0
    return w


@pytest.mark.parametrize("B", [1, 7, 16, 17, 48, 64, 65, 100, 128])
def test_dense_schedule_small_layer(B):
    """Buckets of 1 to 128 rows: one ragged group, exactly one accumulator, two groups."""
    run_case(DENSE_SMALL, B, seed=11, schedule=binding.SCHED_DENSE, weights=_scaled(DENSE_SMALL, 11))


@pytest.mark.parametrize("B", [5, 40, 96])
def test_dense_schedule_wide_layer(B):
    run_case(DENSE_WIDE, B, seed=12, schedule=binding.SCHED_DENSE, weights=_scaled(DENSE_WIDE, 12, scale=6.0))


@pytest.mark.parametrize("variant", ["no_shared", "sigma_none", "gelu", "rmsnorm", "group_limited", "strict_rmsnorm",
                                     "residual"])
def test_dense_schedule_variants(variant):
    shape = {
        "no_shared": DENSE_SMALL.with_(n_shared=0, shared_ffn=0),
        "sigma_none": DENSE_SMALL.with_(sigma=0),
        "gelu": DENSE_SMALL.with_(sigma=2),
        "rmsnorm": DENSE_SMALL.with_(sigma=3),
        "group_limited": DENSE_SMALL.with_(n_dept=4, top_k=4, k_dept=2),
        "strict_rmsnorm": DENSE_SMALL.with_(n_dept=6, experts_per_dept=6, top_k=4, k_dept=4, strict_dept=1, sigma=3),
        "residual": DENSE_SMALL.with_(residual=1),
    }[variant]
    run_case(shape, 50, seed=13, schedule=binding.SCHED_DENSE, weights=_scaled(shape, 13))


def test_dense_schedule_is_refused_for_layers_it_cannot_run():
    dev = torch.device("cuda:0")
    for shape, vanilla in ((DENSE_SMALL.with_(priv=0), False), (DENSE_SMALL.with_(hidden=192), False),
                           (DENSE_SMALL.with_(act_dtype=0), False), (DENSE_SMALL.with_(priv=0), True)):
        w = (synth.make_vanilla_weights if vanilla else synth.make_deamoe_weights)(shape, 1, dev)
        with pytest.raises(binding.DeaMoEError) as e:
            binding.Layer(shape, w, 8, binding.SCHED_DENSE, vanilla=vanilla)
        assert e.value.status == binding.ERR_UNSUPPORTED


def test_auto_switches_to_the_dense_schedule_by_batch_and_both_agree():
    """One AUTO layer sized for 128 tokens: below `binding.dense_min_batch(shape)` tokens (64 for this 16-expert layer) calls take the streaming schedule, from there on the dense one;
    each agrees with a layer fixed to that schedule bit for bit, and the two schedules agree within
    the tolerance (they round intermediates alike but sum in different orders)."""
    shape = DENSE_WIDE
    w = _scaled(shape, 14, scale=6.0)
    auto = binding.Layer(shape, w, 128, binding.SCHED_AUTO)
    fused = binding.Layer(shape, w, 128, binding.SCHED_FUSED)
    dense = binding.Layer(shape, w, 128, binding.SCHED_DENSE)
    try:
        for B in (16, 32, 63, 64, 128):
            x = synth.make_tokens(shape, B, 14 + B, torch.device("cuda:0"))
            oa, of, od = auto.forward(x).float(), fused.forward(x).float(), dense.forward(x).float()
            torch.cuda.synchronize()
            for layer in (auto, fused, dense):
                assert layer.stats()["device_status"] == 0
            same = of if B < binding.dense_min_batch(shape) else od
            assert torch.equal(oa, same)
            ok, err, bound = within_tolerance(od.cpu().numpy().astype(np.float64), of.cpu().numpy().astype(np.float64))
            assert ok, f"{err:.3e} > {bound:.3e}"
    finally:
        auto.close(); fused.close(); dense.close()


def test_dense_schedule_deepseek_v3_cut_sampled_rows():
    """The benchmark's matrices (h 7168, f 2048, r 896, shared expert; 8 x 4 experts) at 64 tokens,
    oracle on sampled token rows."""
    run_case(synth.DSV3_MINI, 64, seed=3, schedule=binding.SCHED_DENSE, rows=[0, 31, 63])


def test_dense_step_can_be_captured_in_a_cuda_graph_and_replayed():
    """The dense step (routing, bucket gather, three tensor-core / streaming launches, combine)
    allocates nothing and builds its tensor maps on the host from pointers that do not change, so
    it can be captured once and replayed on new token values in the same buffer."""
    shape = DENSE_WIDE
    w = _scaled(shape, 15, scale=6.0)
    layer = binding.Layer(shape, w, 96, binding.SCHED_DENSE)
    try:
        x = synth.make_tokens(shape, 70, 41, "cuda:0")
        out = torch.empty_like(x)
        layer.forward(x, out)
        torch.cuda.synchronize()
        side = torch.cuda.Stream()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(graph, stream=side):
                layer.forward(x, out)
        torch.cuda.synchronize()
        for seed in (42, 43):
            new = synth.make_tokens(shape, 70, seed, "cuda:0")
            want = layer.forward(new).clone()
            torch.cuda.synchronize()
            x.copy_(new)
            graph.replay()
            torch.cuda.synchronize()
            assert torch.equal(out, want), seed
        assert layer.stats()["device_status"] == 0
    finally:
        layer.close()


def test_dense_steps_of_changing_batch_on_one_layer_leave_no_state_behind():
    """Steps of very different token counts queued on one dense layer without a synchronisation in between:
    the hand-over words of a step (the routing kernel's flags, the count of finished gather CTAs, the job
    counter of the tensor-core launches, the departments' completion counters) are all reused by the next,
    which may start while the previous step's last kernels drain.  Every output must equal, bit for bit, the
    one a fresh layer gives for that batch alone."""
    shape = DENSE_WIDE
    w = _scaled(shape, 16, scale=6.0)
    seq = [(100, 61), (5, 62), (64, 63), (33, 64), (128, 65), (1, 66), (128, 67), (17, 68)]
    xs = [synth.make_tokens(shape, B, seed, "cuda:0") for B, seed in seq]
    # DENSE: every step takes the dense schedule; AUTO: the steps of fewer than 64 tokens (a 16-expert layer) take the fused one, whose
    # hand-over flags are the same words with another meaning
    for sched in (binding.SCHED_DENSE, binding.SCHED_AUTO):
        layer = binding.Layer(shape, w, 128, sched)
        try:
            outs = [layer.forward(x).clone() for x in xs]     # (clone is enqueued on the same stream)
            torch.cuda.synchronize()
            assert layer.stats()["device_status"] == 0
            for (B, seed), x, got in zip(seq, xs, outs):
                fresh = binding.Layer(shape, w, 128, sched)
                try:
                    want = fresh.forward(x).clone()
                    torch.cuda.synchronize()
                finally:
                    fresh.close()
                assert torch.equal(got, want), (sched, B, seed)
            run_case(shape, 128, weights=w, tokens=xs[4], layer=layer)   # and the layer still agrees with the oracle
        finally:
            layer.close()


def test_many_steps_of_random_batch_sizes_repeat_bit_for_bit():
    """400 steps of random token counts (1 - 128) on one AUTO layer, queued without a synchronisation, a second
    layer's steps in between: every (batch, tokens) pair must give the same bits each time it comes up, and the
    device status must stay 0.  (The chained kernels of a step overlap differently from step to step; nothing
    they hand over may depend on that.)"""
    import random
    shape = DENSE_WIDE
    a = binding.Layer(shape, _scaled(shape, 17, scale=6.0), 128, binding.SCHED_AUTO)
    b = binding.Layer(DENSE_SMALL, _scaled(DENSE_SMALL, 18), 128, binding.SCHED_DENSE)
    try:
        rng = random.Random(5)
        sizes = [1, 2, 7, 16, 31, 32, 33, 63, 64, 65, 100, 128]
        pool = {(B, i): synth.make_tokens(shape, B, 300 + 10 * B + i, "cuda:0") for B in sizes for i in range(2)}
        pool_b = {B: synth.make_tokens(DENSE_SMALL, B, 500 + B, "cuda:0") for B in sizes}
        first, first_b = {}, {}
        for _ in range(400):
            key = (rng.choice(sizes), rng.randrange(2))
            out = a.forward(pool[key])
            if key not in first:
                first[key] = out.clone()
            else:
                assert torch.equal(out, first[key]), key
            if rng.random() < 0.3:
                B = rng.choice(sizes)
                out = b.forward(pool_b[B])
                if B not in first_b:
                    first_b[B] = out.clone()
                else:
                    assert torch.equal(out, first_b[B]), B
        torch.cuda.synchronize()
        assert a.stats()["device_status"] == 0 and b.stats()["device_status"] == 0
    finally:
        a.close(); b.close()


def test_layers_of_both_schedules_enqueued_back_to_back():
    """Dense and streaming steps of different layers queued on one stream without a synchronisation
    in between (a decoder stack): every output equals the one the layer gives when run alone."""
    shape = DENSE_WIDE
    layers = [binding.Layer(shape, _scaled(shape, 20 + i, scale=6.0), 96, binding.SCHED_AUTO) for i in range(3)]
    try:
        for B in (8, 80):
            x = synth.make_tokens(shape, B, 50 + B, "cuda:0")
            alone = []
            for layer in layers:
                alone.append(layer.forward(x).clone())
                torch.cuda.synchronize()
            outs = [torch.empty_like(x) for _ in layers]
            for layer, o in zip(layers, outs):
                layer.forward(x, o)
            torch.cuda.synchronize()
            for o, a in zip(outs, alone):
                assert torch.equal(o, a)
    finally:
        for layer in layers:
            layer.close()


def test_7b_class_layer_dense_every_element():
    """7B-class layer (h 4096, f 1408: a stacked gate / up tile holds rows of both matrices), 64
    tokens, every output element against the oracle."""
    run_case(synth.MOE7B, 64, seed=2, schedule=binding.SCHED_DENSE)
