"""GPU parity where the numbers are quoted: the DeepSeek-V3-shaped layer at full size, created the way
`bench.py` creates it (AUTO schedule, sized for 128 tokens), at every batch size of the benchmark's
sweep; and the routing-locality sweep (benchmark configuration 4) on that same layer."""
import numpy as np
import pytest
import torch

from oracle import accounting, ref
from paper_2608_14385_b200 import binding, synth
from tests.common import oracle_cfg
from tests.gpu_common import deep_rows, run_case

pytestmark = pytest.mark.gpu

SHAPE = synth.DSV3


@pytest.fixture(scope="module")
def dsv3():
    """One full-size layer (5.7 GB of weights + the dense schedule's 2.9 GB) for the whole module."""
    dev = torch.device("cuda:0")
    w = synth.make_deamoe_weights(SHAPE, 0, dev)
    layer = binding.Layer(SHAPE, w, 128, binding.SCHED_AUTO)
    yield w, layer
    layer.close()


@pytest.mark.parametrize("B", [1, 2, 4, 8, 16])
def test_dsv3_shape_every_token_row(dsv3, B):
    """Benchmark configuration 3 at the batch sizes of its target range (the headline number is
    B = 16): routing, department sets and token lists bit-exact, and EVERY token row of the output
    against the oracle (which evaluates Eq. (4) per selected expert and Eq. (3) per token)."""
    w, layer = dsv3
    res = run_case(SHAPE, B, weights=w, tokens=synth.make_tokens(SHAPE, B, 100, "cuda:0"), layer=layer)
    assert res["rows"] == list(range(B))
    st = res["stats"]
    assert st["unique_weight_bytes"] == accounting.unique_bytes_deamoe(
        st["active_dept"], st["active_expert"], SHAPE.hidden, SHAPE.ffn, SHAPE.priv, SHAPE.n_expert, 2,
        SHAPE.n_shared, SHAPE.shared_ffn)


@pytest.mark.parametrize("B,count,min_depth", [(32, 8, 8), (64, 8, 16), (128, 10, 30)])
def test_dsv3_shape_larger_batches_deep_rows(dsv3, B, count, min_depth):
    """32 tokens (streaming schedule: buckets of more than 8 tokens take a second 8-token pass per
    tile) and 64 / 128 tokens (dense schedule on the tensor cores: buckets of 16 and more rows).
    Routing and lists for the whole batch; output values on the token rows that sit deepest in their
    department's token list, plus the first and last token."""
    w, layer = dsv3
    res = run_case(SHAPE, B, weights=w, tokens=synth.make_tokens(SHAPE, B, 100, "cuda:0"), layer=layer,
                   rows=deep_rows(count))
    assert len(res["rows"]) >= count - 1 and res["deepest"] >= min_depth


@pytest.mark.parametrize("c", [1, 2, 4, 8])
@pytest.mark.parametrize("B", [1, 16])
def test_locality_sweep_on_the_full_shape(dsv3, c, B):
    """Benchmark configuration 4: every token's top-8 is planted (through the real router) in exactly
    c departments.  The oracle must confirm the planted selection; the GPU routing must match it bit
    for bit; the counted unique bytes must equal the closed form on the planted sets; output values on
    the first and last token."""
    w, layer = dsv3
    g = SHAPE.experts_per_dept
    for attempt in range(8):    # the first seed whose planted logits stay clear of a tie (decided by the oracle alone)
        tokens, chosen = synth.plant_locality(SHAPE, w["router"],
                                              synth.make_tokens(SHAPE, B, 200 + c + 100 * attempt, "cuda:0"), c,
                                              seed=10 * c + B + 100 * attempt)
        want = ref.route(oracle_cfg(SHAPE), synth.to_numpy(w["router"]), synth.to_numpy(tokens), want_logits=True)
        if (want["gap"] > 1e-5 * np.abs(want["logits"]).max(axis=1)).all():
            break
    for t in range(B):
        assert sorted(int(i) for i in want["idx"][t]) == chosen[t]
        assert len({i // g for i in chosen[t]}) == c
    res = run_case(SHAPE, B, weights=w, tokens=tokens, layer=layer, rows=sorted({0, B - 1}))
    nd, ne, pairs = accounting.count_active(chosen, g)
    st = res["stats"]
    assert (st["active_dept"], st["active_expert"], st["token_dept_pairs"]) == (nd, ne, pairs) and pairs == B * c
    assert st["unique_weight_bytes"] == accounting.unique_bytes_deamoe(
        nd, ne, SHAPE.hidden, SHAPE.ffn, SHAPE.priv, SHAPE.n_expert, 2, SHAPE.n_shared, SHAPE.shared_ffn)


@pytest.fixture(scope="module")
def dsv3_vanilla():
    """The comparator `bench.py` times beside the layer: 256 standard experts, 22.6 GB, sized for 128 tokens."""
    dev = torch.device("cuda:0")
    w = synth.make_vanilla_weights(SHAPE, 0, dev)
    layer = binding.Layer(SHAPE, w, 128, binding.SCHED_AUTO, vanilla=True)
    yield w, layer
    layer.close()


@pytest.mark.parametrize("B,count", [(1, None), (4, None), (16, None), (64, 6)])
def test_vanilla_comparator_at_the_benchmark_points(dsv3_vanilla, B, count):
    """The in-library vanilla MoE layer (Eq. (1)-(3)) the speed-up is quoted against, at full size: routing and
    token lists for the whole batch, every token row at B = 1, 4, 16 (the headline's comparator), sampled
    deep rows at 64 tokens."""
    w, layer = dsv3_vanilla
    res = run_case(SHAPE, B, weights=w, tokens=synth.make_tokens(SHAPE, B, 100, "cuda:0"), layer=layer, vanilla=True,
                   rows=None if count is None else deep_rows(count))
    st = res["stats"]
    assert st["unique_weight_bytes"] == accounting.unique_bytes_vanilla(
        st["active_expert"], SHAPE.hidden, SHAPE.ffn, SHAPE.n_expert, 2, SHAPE.n_shared, SHAPE.shared_ffn)


@pytest.mark.parametrize("B,count", [(4, None), (16, 8), (64, 8)])
def test_paper_row_and_its_baseline_at_the_benchmark_points(B, count):
    """The paper's own DeepSeek-V3-matched row (Table 1: 8 x 108 experts, square private matrices, top-10 in at most
    5 departments) and the standard layer it is matched to (256 experts, top-8, no shared expert), at the token
    counts of `bench.py`'s rows for them, both created as `bench.py` creates them (sized for 64 tokens)."""
    rows = None if count is None else deep_rows(count)
    shape = synth.DSV3_PAPER
    res = run_case(shape, B, seed=0, rows=rows, max_batch=64)
    st = res["stats"]
    assert st["unique_weight_bytes"] == accounting.unique_bytes_deamoe(
        st["active_dept"], st["active_expert"], shape.hidden, shape.ffn, shape.priv, shape.n_expert, 2)
    base = synth.PAPER_BASELINES[shape.name]
    run_case(base, B, seed=0, vanilla=True, rows=rows, max_batch=64)


def test_two_slices_of_the_benchmark_layer():
    """The department-sharded layout at the benchmark's size: two slices of 16 departments each (the second
    with the shared expert), B = 16, run one after the other on this GPU; the sum of their partial outputs,
    finished, against the oracle's unsharded layer on every token row; each slice's byte count against the closed
    form on its own active sets."""
    from paper_2608_14385_b200 import shard
    dev = torch.device("cuda:0")
    B = 16
    tokens = synth.make_tokens(SHAPE, B, 100, dev)
    g = SHAPE.experts_per_dept
    total = torch.zeros((B, SHAPE.hidden), dtype=torch.float32, device=dev)
    host = {"router": None}
    want_idx = None
    tables = {name: [None] * SHAPE.n_dept for name in ("dept_gate", "dept_up", "dept_down")}
    tables.update({name: [None] * SHAPE.n_expert for name in ("priv_gate", "priv_up", "priv_down")})
    last = None
    for r in range(2):
        my_shape, (lo, hi) = shard.slice_shape(SHAPE, r, 2)
        w = synth.make_deamoe_weights(my_shape, 0, dev, dept_range=(lo, hi))
        layer = binding.Layer(my_shape, w, 32, binding.SCHED_AUTO, dept_range=(lo, hi))
        part = layer.forward_partial(tokens)
        torch.cuda.synchronize()
        st = layer.stats()
        assert st["device_status"] == 0
        idx = layer.routing(B)["idx"]
        if want_idx is None:
            want_idx = ref.route(oracle_cfg(SHAPE), synth.to_numpy(w["router"]), synth.to_numpy(tokens))["idx"]
            host["router"] = synth.to_numpy(w["router"])
        assert (idx == want_idx).all()
        mine = [[int(i) for i in row if lo <= int(i) // g < hi] for row in want_idx]
        nd, ne, pairs = accounting.count_active(mine, g)
        assert (st["active_dept"], st["active_expert"], st["token_dept_pairs"]) == (nd, ne, pairs)
        assert st["unique_weight_bytes"] == accounting.unique_bytes_deamoe(
            nd, ne, SHAPE.hidden, SHAPE.ffn, SHAPE.priv, SHAPE.n_expert, 2, my_shape.n_shared, my_shape.shared_ffn)
        for row in mine:                                   # host copies of exactly what the oracle will touch
            for i in row:
                j = i // g
                for name in ("gate", "up", "down"):
                    if tables[f"dept_{name}"][j] is None:
                        tables[f"dept_{name}"][j] = synth.to_numpy(w[f"dept_{name}"][j - lo])
                    if tables[f"priv_{name}"][i] is None:
                        tables[f"priv_{name}"][i] = synth.to_numpy(w[f"priv_{name}"][i - lo * g])
        if my_shape.n_shared:
            for name in ("gate", "up", "down"):
                host[f"shared_{name}"] = synth.to_numpy(w[f"shared_{name}"])
        total += part
        if last is not None:
            last.close()
        last = layer
        del w
    try:
        out = last.finish_partial(total, tokens)
        torch.cuda.synchronize()
        host.update(tables)
        want = ref.deamoe_forward(oracle_cfg(SHAPE), host, synth.to_numpy(tokens))
        from tests.common import within_tolerance
        ok, err, bound = within_tolerance(out.float().cpu().numpy(), want["out"])
        assert ok, (err, bound)
    finally:
        last.close()
