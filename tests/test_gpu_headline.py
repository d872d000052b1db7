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
