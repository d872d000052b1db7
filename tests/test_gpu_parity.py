"""GPU parity: the CUDA library against the fp64 oracle, through the C ABI, on the same seeded inputs.

Routing indices, department sets and token lists must be bit-exact; gate weights within 1e-5;
outputs within max|diff| <= 1e-2 * max|ref| + 1e-3 (bf16 weights, fp32 accumulation)."""
import ctypes

import numpy as np
import pytest
import torch

from oracle import ref
from paper_2608_14385_b200 import binding, synth
from tests.common import oracle_cfg, within_tolerance
from tests.gpu_common import check_routing, run_case

pytestmark = pytest.mark.gpu

SMALL = synth.LayerShape("small", hidden=64, n_dept=3, experts_per_dept=4, ffn=48, priv=32, top_k=3)
RAGGED = synth.LayerShape("ragged", hidden=208, n_dept=5, experts_per_dept=3, ffn=176, priv=80, top_k=4,
                          n_shared=1, shared_ffn=112)

ALL_SCHEDULES = [binding.SCHED_PLAIN, binding.SCHED_STAGED, binding.SCHED_FUSED]


def _scaled(shape, seed, scale=12.0, vanilla=False):
    """Weights of std 0.02*scale: small layers need larger weights for non-trivial outputs."""
    dev = torch.device("cuda:0")
    w = (synth.make_vanilla_weights if vanilla else synth.make_deamoe_weights)(shape, seed, dev)
    for k in w:
        w[k] = (w[k].float() * scale).to(w[k].dtype) if k != "router" else w[k] * 4.0
    return w


def test_tiny_fp32_config():
    """Benchmark configuration 1: h 256, 2 x 4 experts, f 512, r 32, top-2, 4 tokens, all fp32."""
    res = run_case(synth.TINY, 4, seed=0)
    assert res["err"] <= 1e-4 * np.abs(res["want"]["out"]).max() + 1e-6   # fp32 end to end is far tighter


@pytest.mark.parametrize("schedule", ALL_SCHEDULES)
@pytest.mark.parametrize("B", [1, 3, 8, 17])
def test_small_bf16_layer_all_schedules(schedule, B):
    w = _scaled(SMALL, 1)
    run_case(SMALL, B, seed=1, schedule=schedule, weights=w)


@pytest.mark.parametrize("schedule", ALL_SCHEDULES)
def test_ragged_sizes_with_shared_expert_and_residual(schedule):
    """Sizes that are not multiples of the kernel tiles (rows 176/80/112, k-extent 208), shared
    expert, residual add, batch not a multiple of the token tile."""
    shape = RAGGED.with_(residual=1)
    run_case(shape, 11, seed=2, schedule=schedule, weights=_scaled(shape, 2))


@pytest.mark.parametrize("schedule", ALL_SCHEDULES)
def test_vanilla_comparator(schedule):
    shape = RAGGED
    run_case(shape, 9, seed=3, schedule=schedule, vanilla=True, weights=_scaled(shape, 3, vanilla=True))


@pytest.mark.parametrize("schedule", ALL_SCHEDULES)
@pytest.mark.parametrize("variant", ["no_private", "sigma_none", "gelu", "rmsnorm", "rmsnorm_shared_f32", "square_private", "g1", "k_eq_n",
                                     "norm_all", "sigmoid_gates", "group_limited", "strict_coverage", "f32_tokens"])
def test_variants(schedule, variant):
    shape = {
        "no_private": SMALL.with_(priv=0),
        "sigma_none": SMALL.with_(sigma=0),
        "gelu": SMALL.with_(sigma=2),
        "rmsnorm": SMALL.with_(sigma=3),
        "rmsnorm_shared_f32": RAGGED.with_(sigma=3, act_dtype=0),
        "square_private": SMALL.with_(priv=48),
        "g1": SMALL.with_(n_dept=12, experts_per_dept=1),
        "k_eq_n": SMALL.with_(n_dept=2, experts_per_dept=2, top_k=4),
        "norm_all": SMALL.with_(norm_topk=0, route_scale=2.5),
        "sigmoid_gates": SMALL.with_(norm_topk=2, route_scale=2.5),
        "group_limited": SMALL.with_(n_dept=4, experts_per_dept=4, top_k=4, k_dept=2),
        "strict_coverage": SMALL.with_(n_dept=6, experts_per_dept=6, top_k=4, k_dept=4, strict_dept=1),
        "f32_tokens": RAGGED.with_(act_dtype=0),
    }[variant]
    run_case(shape, 6, seed=4, schedule=schedule, weights=_scaled(shape, 4))


@pytest.mark.parametrize("schedule", ALL_SCHEDULES)
def test_all_tokens_identical_and_max_batch(schedule):
    """Degenerate routing: every token picks the same experts (one department bucket holds the
    whole batch); batch equal to max_batch."""
    shape = SMALL
    w = _scaled(shape, 5)
    one = synth.make_tokens(shape, 1, 5, "cuda:0")
    tokens = one.expand(32, shape.hidden).contiguous()
    res = run_case(shape, 32, seed=5, schedule=schedule, weights=w, tokens=tokens, max_batch=32)
    assert res["stats"]["active_expert"] == shape.top_k


def test_exact_ties_break_to_lowest_index():
    """Integer-valued router and tokens: logits are exact in fp32 whatever the summation order, so
    equal logits are true ties and the selection must still match the oracle bit for bit."""
    shape = SMALL.with_(n_dept=4, experts_per_dept=4, top_k=5)
    dev = torch.device("cuda:0")
    w = _scaled(shape, 6)
    ints = torch.tensor(synth.uniform_ints(16 * 64, 3, 6, "ri"), dtype=torch.float32).reshape(16, 64) - 1.0
    ints[5] = ints[2]
    ints[9] = ints[2]
    ints[12] = ints[0]
    w["router"] = ints.to(dev)
    tok = torch.tensor(synth.uniform_ints(7 * 64, 5, 6, "ti"), dtype=torch.float32).reshape(7, 64) - 2.0
    tok[3] = 0.0                                           # all logits equal (zero)
    tokens = tok.to(torch.bfloat16).to(dev)
    layer = binding.Layer(shape, w, 8, binding.SCHED_PLAIN)
    try:
        layer.forward(tokens)
        want, _ = check_routing(shape, layer, w, tokens, 7, require_guard=False)
        assert (want["gap"] == 0).any()
        assert list(want["idx"][3]) == [0, 1, 2, 3, 4]
    finally:
        layer.close()


def test_route_entry_point_and_empty_batch():
    shape = SMALL
    w = _scaled(shape, 7)
    layer = binding.Layer(shape, w, 8)
    try:
        tokens = synth.make_tokens(shape, 5, 7, "cuda:0")
        idx, p = layer.route(tokens)
        torch.cuda.synchronize()
        want, _ = check_routing(shape, layer, w, tokens, 5)
        assert (idx.cpu().numpy() == want["idx"]).all()
        assert np.abs(p.cpu().numpy() - want["w"]).max() <= 1e-5
        empty = tokens[:0].contiguous()
        out = layer.forward(empty)
        assert out.shape == (0, shape.hidden)
        st = layer.stats()
        assert st["active_dept"] == 0 and st["active_expert"] == 0 and st["device_status"] == 0
        r = layer.routing(0)
        assert (r["dept_off"] == 0).all() and (r["expert_off"] == 0).all() and r["dept_mask"][0] == 0
        with pytest.raises(binding.DeaMoEError) as e:
            layer.forward(synth.make_tokens(shape, 9, 7, "cuda:0"))
        assert e.value.status == binding.ERR_BATCH
        st_alias = binding.lib().deamoe_forward(layer._h, None, ctypes.c_void_p(tokens.data_ptr()), 5,
                                                ctypes.c_void_p(tokens.data_ptr()))
        assert st_alias == binding.ERR_INVALID_ARG
    finally:
        layer.close()


def test_forward_host_matches_device_forward():
    shape = RAGGED
    w = _scaled(shape, 8)
    layer = binding.Layer(shape, w, 8)
    try:
        tokens = synth.make_tokens(shape, 6, 8, "cuda:0")
        dev_out = layer.forward(tokens).cpu()
        host_in = tokens.cpu().pin_memory()
        host_out = torch.empty_like(host_in).pin_memory()
        layer.forward_host(host_in, host_out)
        assert torch.equal(host_out, dev_out)
    finally:
        layer.close()


def test_repeated_calls_are_bit_reproducible_and_state_is_reset():
    """Two different batches alternately through one layer: each result must be identical every
    time (no stale routing state, no order-dependent accumulation)."""
    shape = RAGGED
    w = _scaled(shape, 9)
    layer = binding.Layer(shape, w, 16)
    try:
        a = synth.make_tokens(shape, 16, 9, "cuda:0")
        b = synth.make_tokens(shape, 3, 10, "cuda:0")
        ra, rb = layer.forward(a).clone(), layer.forward(b).clone()
        for _ in range(3):
            assert torch.equal(layer.forward(a), ra)
            assert torch.equal(layer.forward(b), rb)
    finally:
        layer.close()


@pytest.mark.parametrize("schedule", [binding.SCHED_STAGED, binding.SCHED_FUSED, binding.SCHED_DENSE])
def test_rmsnorm_sigma_is_bit_reproducible(schedule):
    """sigma = RMSNorm adds the squares of a vector tile by tile, from many thread blocks in no fixed
    order; the sums are kept as fixed-point integers, so the result must not depend on that order:
    repeated calls on alternating batches give identical bits."""
    shape = synth.LayerShape("rmsrep", hidden=256, n_dept=3, experts_per_dept=4, ffn=384, priv=128, top_k=4,
                             n_shared=1, shared_ffn=128, sigma=binding.SIGMA_RMSNORM)
    w = _scaled(shape, 12)
    nb = 64 if schedule == binding.SCHED_DENSE else 16
    layer = binding.Layer(shape, w, nb, schedule)
    try:
        a = synth.make_tokens(shape, nb, 12, "cuda:0")
        b = synth.make_tokens(shape, 5, 13, "cuda:0")
        ra, rb = layer.forward(a).clone(), layer.forward(b).clone()
        for _ in range(5):
            assert torch.equal(layer.forward(a), ra)
            assert torch.equal(layer.forward(b), rb)
        run_case(shape, nb, weights=w, tokens=a, layer=layer)
    finally:
        layer.close()


@pytest.mark.parametrize("B", [1, 4, 16])
def test_7b_class_layer(B):
    """Benchmark configuration 2 at full size, every output element compared."""
    run_case(synth.MOE7B, B, seed=0)


@pytest.mark.parametrize("B", [1, 4, 16])
def test_7b_class_vanilla(B):
    """The comparator of benchmark configuration 2 at the batch sizes `bench.py` times, every element."""
    run_case(synth.MOE7B, B, seed=0, vanilla=True, max_batch=16)


def test_dsv3_shape_vanilla_sampled_row():
    run_case(synth.DSV3, 4, seed=0, vanilla=True, rows=[2], max_batch=32)


def test_unsupported_and_invalid_creates_are_reported():
    dev = torch.device("cuda:0")
    shape = SMALL.with_(hidden=66)                         # not a multiple of 4
    w = {k: torch.zeros(1, device=dev) for k in ("router", "dept_gate", "dept_up", "dept_down",
                                                 "priv_gate", "priv_up", "priv_down")}
    with pytest.raises(binding.DeaMoEError) as e:
        binding.Layer(shape, w, 4)
    assert e.value.status == binding.ERR_UNSUPPORTED
    with pytest.raises(binding.DeaMoEError) as e:
        binding.Layer(SMALL.with_(weight_dtype=0), w, 4, binding.SCHED_FUSED)   # fp32 cannot stream
    assert e.value.status == binding.ERR_UNSUPPORTED
    with pytest.raises(binding.DeaMoEError) as e:
        binding.Layer(SMALL.with_(sigma=3, priv=0), w, 4, binding.SCHED_PLAIN)   # RMSNorm needs private matrices
    assert e.value.status == binding.ERR_UNSUPPORTED


def test_non_finite_tokens_keep_indices_valid():
    """Inputs must be finite for the results to mean anything, but a NaN / Inf token row must not
    turn into an invalid expert index (that would be an out-of-range access): the call completes,
    every index is a valid expert, and the finite rows are unaffected."""
    shape = RAGGED
    w = _scaled(shape, 4)
    layer = binding.Layer(shape, w, 8)
    try:
        good = synth.make_tokens(shape, 6, 21, "cuda:0")
        bad = good.clone()
        bad[1, :] = float("nan")
        bad[4, 3] = float("inf")
        ref_out = layer.forward(good).clone()
        out = layer.forward(bad)
        torch.cuda.synchronize()
        st = layer.stats()
        assert st["device_status"] == 0
        idx = layer.routing(6)["idx"]
        assert idx.min() >= 0 and idx.max() < shape.n_expert
        for t in range(6):
            assert len(set(int(i) for i in idx[t])) == shape.top_k
        keep = [0, 2, 3, 5]
        a, b = out[keep].float().cpu().numpy(), ref_out[keep].float().cpu().numpy()
        assert np.isfinite(a).all()
        ok, err, bound = within_tolerance(a, b)
        assert ok, (err, bound)
    finally:
        layer.close()


def test_fused_step_can_be_captured_in_a_cuda_graph_and_replayed():
    """A step allocates nothing and keeps no per-step state on the host, so it can be captured once
    and replayed on new token values in the same buffer; every replay must equal the eager result."""
    shape = RAGGED
    w = _scaled(shape, 6)
    layer = binding.Layer(shape, w, 8, binding.SCHED_FUSED)
    try:
        x = synth.make_tokens(shape, 5, 31, "cuda:0")
        out = torch.empty_like(x)
        layer.forward(x, out)                      # warm-up outside the capture
        torch.cuda.synchronize()
        side = torch.cuda.Stream()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(graph, stream=side):
                layer.forward(x, out)
        torch.cuda.synchronize()
        for seed in (32, 33, 34):
            new = synth.make_tokens(shape, 5, seed, "cuda:0")
            want = layer.forward(new).clone()
            torch.cuda.synchronize()
            x.copy_(new)
            graph.replay()
            torch.cuda.synchronize()
            assert torch.equal(out, want), seed
        assert layer.stats()["device_status"] == 0
    finally:
        layer.close()


@pytest.mark.parametrize("vanilla", [False, True])
def test_fused_and_staged_schedules_agree_bit_for_bit_over_random_batches(vanilla):
    """The fused schedule overlaps the routing with the first streams, hands work over through
    flags and claims items dynamically; the staged schedule launches one stage at a time.  Both run
    the same arithmetic per item, so their outputs must be identical for any batch, also when the
    calls are enqueued back to back."""
    import random
    rnd = random.Random(5)
    shape = synth.LayerShape("mix", hidden=512, n_dept=8, experts_per_dept=4, ffn=256, priv=64, top_k=6,
                             n_shared=1, shared_ffn=256)
    w = (synth.make_vanilla_weights if vanilla else synth.make_deamoe_weights)(shape, 3, "cuda:0")
    for key in w:
        if key != "router":
            w[key] = (w[key].float() * 4).to(w[key].dtype)
    fused = binding.Layer(shape, w, 32, binding.SCHED_FUSED, vanilla=vanilla)
    staged = binding.Layer(shape, w, 32, binding.SCHED_STAGED, vanilla=vanilla)
    try:
        pending = []
        for it in range(60):
            B = rnd.choice([1, 1, 2, 3, 4, 7, 8, 13, 16, 17, 31, 32])
            x = synth.make_tokens(shape, B, 1000 + it, "cuda:0")
            a = fused.forward(x)
            if it % 3 == 0:
                torch.cuda.synchronize()
            pending.append((a, staged.forward(x), B))
            if len(pending) == 6:
                torch.cuda.synchronize()
                for fa, sa, b in pending:
                    assert torch.equal(fa, sa), b
                pending = []
        torch.cuda.synchronize()
        assert fused.stats()["device_status"] == 0 and staged.stats()["device_status"] == 0
    finally:
        fused.close()
        staged.close()
