"""GPU parity for the benchmark's structured workloads: routing-locality sweep (configuration 4) and a
stack of consecutive layers with a residual add (configuration 5)."""
import numpy as np
import pytest
import torch

from oracle import accounting, ref
from paper_2608_14385_b200 import binding, synth
from tests.common import oracle_cfg, within_tolerance
from tests.gpu_common import check_routing, lazy_oracle_weights, run_case

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("c", [1, 2, 4])
def test_locality_sweep_planted_routing(c):
    """Tokens whose top-k picks are planted in exactly c departments (through the real router): the
    oracle must confirm the planted selection, the GPU routing must match it bit for bit, the unique
    weight bytes must equal the closed form on the counted sets, and outputs must be in tolerance."""
    shape = synth.DSV3_MINI
    dev = torch.device("cuda:0")
    B = 8
    w = synth.make_deamoe_weights(shape, 0, dev)
    tokens, chosen = synth.plant_locality(shape, w["router"], synth.make_tokens(shape, B, 1, dev), c, seed=c)
    want = ref.route(oracle_cfg(shape), synth.to_numpy(w["router"]), synth.to_numpy(tokens))
    for t in range(B):
        assert sorted(int(i) for i in want["idx"][t]) == chosen[t]
        assert len({i // shape.experts_per_dept for i in chosen[t]}) == c
    res = run_case(shape, B, weights=w, tokens=tokens, rows=[0, B - 1], max_batch=8)
    nd, ne, _ = accounting.count_active(chosen, shape.experts_per_dept)
    assert res["stats"]["active_dept"] == nd and res["stats"]["active_expert"] == ne
    assert res["stats"]["unique_weight_bytes"] == accounting.unique_bytes_deamoe(
        nd, ne, shape.hidden, shape.ffn, shape.priv, shape.n_expert, 2, shape.n_shared, shape.shared_ffn)


@pytest.mark.parametrize("B", [1, 8])
def test_stack_of_32_layers_teacher_forced(B):
    """Benchmark configuration 5 at its full depth: 32 consecutive 7B-class layers with a residual add,
    every layer with its own seeded weights, tokens scaled as `bench.py` scales them (1/16, so that the
    un-normalised stack stays finite).  Teacher forced: GPU layer l gets the oracle's x_l rounded to
    bf16; routing bit-exact (on tokens clear of a tie) and every output element in tolerance, layer by
    layer."""
    n_layers = 32
    shape = synth.MOE7B.with_(residual=1)
    dev = torch.device("cuda:0")
    cfg = oracle_cfg(shape)
    x = (synth.make_tokens(shape, B, 300, dev).float() / 16).to(torch.bfloat16)
    worst = 0.0
    for l in range(n_layers):
        w = synth.make_deamoe_weights(shape, 0, dev, layer=l)
        layer = binding.Layer(shape, w, 8)
        try:
            hostw = {k: synth.to_numpy(v) for k, v in w.items()}
            want = ref.deamoe_forward(cfg, hostw, synth.to_numpy(x))
            r = ref.route(cfg, hostw["router"], synth.to_numpy(x), want_logits=True)
            safe = r["gap"] > 1e-5 * np.abs(r["logits"]).max(axis=1)
            got = layer.forward(x)
            torch.cuda.synchronize()
            assert layer.stats()["device_status"] == 0
            assert (layer.routing(B)["idx"][safe] == want["idx"][safe]).all(), f"layer {l}"
            ok, err, bound = within_tolerance(got.float().cpu().numpy()[safe], want["out"][safe])
            assert ok, (l, err, bound)
            worst = max(worst, err / bound)
            assert safe.mean() >= 0.75
            x = torch.from_numpy(want["out"]).to(torch.bfloat16).to(dev)
            assert torch.isfinite(x.float()).all()
        finally:
            layer.close()
        del w
    assert worst <= 1.0


@pytest.mark.parametrize("B", [1, 8])
def test_stack_of_layers_teacher_forced_and_free_running(B):
    """x_{l+1} = x_l + Layer_l(x_l), every layer with its own seeded weights.  Teacher forced: GPU layer l
    is fed the oracle's x_l (rounded to the activation dtype) and must match routing bit-exactly and
    the output in tolerance.  Free running: the GPU feeds its own outputs forward; the final rows are
    compared only for tokens whose routing agreed in every layer."""
    n_layers = 8
    shape = synth.MOE7B.with_(residual=1)
    dev = torch.device("cuda:0")
    cfg = oracle_cfg(shape)
    layers, hostw = [], []
    for l in range(n_layers):
        w = synth.make_deamoe_weights(shape, 0, dev, layer=l)
        layers.append(binding.Layer(shape, w, 8))
        hostw.append({k: synth.to_numpy(v) for k, v in w.items()})
        del w
    try:
        x_forced = synth.make_tokens(shape, B, 3, dev)
        x_free = x_forced.clone()
        agree = np.ones(B, bool)
        for l in range(n_layers):
            want = ref.deamoe_forward(cfg, hostw[l], synth.to_numpy(x_forced))
            got = layers[l].forward(x_forced)
            torch.cuda.synchronize()
            r = layers[l].routing(B)
            assert (r["idx"] == want["idx"]).all(), f"layer {l}"
            ok, err, bound = within_tolerance(got.float().cpu().numpy(), want["out"])
            assert ok, (l, err, bound)
            free_out = layers[l].forward(x_free)
            torch.cuda.synchronize()
            agree &= (layers[l].routing(B)["idx"] == want["idx"]).all(axis=1)
            x_free = free_out
            x_forced = torch.from_numpy(want["out"]).to(torch.bfloat16).to(dev)
        assert agree.any()
        a = x_free.float().cpu().numpy()[agree]
        b = x_forced.float().cpu().numpy()[agree]
        ok, err, bound = within_tolerance(a, b, rel=3e-2, abs_=1e-2)   # rounding accumulates over the stack
        assert ok, (err, bound, int(agree.sum()))
    finally:
        for layer in layers:
            layer.close()


@pytest.mark.parametrize("B,rows", [(4, [1]), (64, [40])])
def test_paper_deepseek_v3_row_group_limited(B, rows):
    """The paper's own DeepSeek-V3-matched configuration (Table 1, first row): 8 departments x 108
    experts, square private matrices (r = f), top-10 limited to 5 departments (Section 3.3).
    Routing and buckets bit-exact for the whole batch, values on a sampled row, every token inside
    its department cap, unique bytes equal to the closed form on the counted sets."""
    shape = synth.DSV3_PAPER
    res = run_case(shape, B, seed=0, rows=rows, max_batch=64)
    st = res["stats"]
    assert st["active_dept"] <= shape.n_dept and st["active_expert"] <= B * shape.top_k
    assert st["unique_weight_bytes"] == accounting.unique_bytes_deamoe(
        st["active_dept"], st["active_expert"], shape.hidden, shape.ffn, shape.priv, shape.n_expert, 2)


@pytest.mark.parametrize("name,B,rows", [("qwen3-paper", 16, [3, 15]), ("b7-paper", 64, [0, 40, 63]),
                                         ("dsv2-paper", 8, [5]), ("kimi-k2-paper", 4, [2])])
def test_other_table1_rows(name, B, rows):
    """Further rows of Table 1 at full size (Qwen3-235B-, Baseline-7B- and DeepSeek-V2-matched DeaMoE
    configurations): routing and lists for the whole batch, values on sampled rows, unique bytes
    equal to the closed form on the counted sets."""
    shape = synth.SHAPES[name]
    res = run_case(shape, B, seed=1, rows=rows, max_batch=64)
    st = res["stats"]
    assert st["unique_weight_bytes"] == accounting.unique_bytes_deamoe(
        st["active_dept"], st["active_expert"], shape.hidden, shape.ffn, shape.priv, shape.n_expert, 2)


def test_table1_baselines_as_vanilla_layers():
    """The standard MoE layers the Table 1 rows are matched to run as vanilla layers (flat top-k)."""
    for name, B in (("qwen3-paper", 8), ("b7-paper", 16)):
        base = synth.PAPER_BASELINES[name]
        run_case(base, B, seed=2, vanilla=True, rows=[B - 1], max_batch=16)


def test_paper_row_department_cap_holds_for_every_token():
    shape = synth.DSV3_PAPER
    dev = torch.device("cuda:0")
    B = 32
    w = synth.make_deamoe_weights(shape, 1, dev)
    layer = binding.Layer(shape, w, B, binding.SCHED_AUTO)
    try:
        tokens = synth.make_tokens(shape, B, 6, dev)  # seed 5 puts one token within 1e-5 of a routing tie
        layer.route(tokens, want_outputs=False)
        torch.cuda.synchronize()
        idx = layer.routing(B)["idx"]
        for t in range(B):
            assert len({int(i) // shape.experts_per_dept for i in idx[t]}) <= shape.k_dept
            assert len(set(int(i) for i in idx[t])) == shape.top_k
        want, _ = check_routing(shape, layer, w, tokens, B)
    finally:
        layer.close()


@pytest.mark.parametrize("vanilla", [False, True])
def test_layers_enqueued_back_to_back_match_layers_run_one_by_one(vanilla):
    """A stack is normally enqueued without waiting for each layer: the kernels of consecutive layers
    then follow each other directly in the stream (programmatic dependent launches inside a layer,
    ordinary dependencies between layers).  The result must equal, bit for bit, the result of running
    the layers one at a time."""
    n_layers, B = 6, 8
    shape = synth.MOE7B.with_(residual=1)
    dev = torch.device("cuda:0")
    layers = []
    for l in range(n_layers):
        w = (synth.make_vanilla_weights if vanilla else synth.make_deamoe_weights)(shape, 0, dev, layer=l)
        layers.append(binding.Layer(shape, w, 8, vanilla=vanilla))
        del w
    try:
        x0 = (synth.make_tokens(shape, B, 11, dev).float() / 16).to(torch.bfloat16)
        bufs = [torch.empty_like(x0), torch.empty_like(x0)]

        def run(sync):
            cur = x0
            for l, layer in enumerate(layers):
                layer.forward(cur, bufs[l & 1])
                if sync:
                    torch.cuda.synchronize()
                cur = bufs[l & 1]
            torch.cuda.synchronize()
            return cur.clone()
        one_by_one = run(True)
        for _ in range(3):
            assert torch.equal(run(False), one_by_one)
        assert torch.isfinite(one_by_one.float()).all()
        assert all(layer.stats()["device_status"] == 0 for layer in layers)
    finally:
        for layer in layers:
            layer.close()


WIDE_ROUTERS = [
    # n_dept, experts_per_dept, top_k, k_dept, strict department coverage
    (6, 16, 6, 0, 0),       # 96 experts: 8 logits per lane
    (10, 32, 10, 0, 0),     # 320 experts: the wide top-k (one CTA of two warps per token)
    (10, 32, 10, 4, 0),     # group limited
    (8, 108, 10, 5, 0),     # the paper's DeepSeek-V3 router (Table 1)
    (8, 64, 10, 5, 0),      # ... DeepSeek-V2 router
    (8, 40, 8, 5, 0),       # ... Qwen3-235B router
    (16, 80, 10, 5, 0),     # ... Kimi-K2 router: 1280 experts, five warps per token, with a group limit
    (8, 84, 10, 4, 0),      # ... Baseline-7B router
    (32, 32, 32, 0, 0),     # 1024 experts, top-32: every lane of the merging warp holds a selection
    (32, 32, 8, 3, 0),
    (40, 40, 8, 6, 0),      # 1600 experts, a group limit over 40 departments (more than a warp has lanes): the shared-memory top-k
    (32, 64, 8, 0, 0),      # 2048 experts: the most a layer may have (eight warps per token)
    (6, 16, 6, 4, 1),       # strict department coverage (Section 3.3, last paragraph)
    (8, 108, 10, 5, 1),     # ... on the paper's DeepSeek-V3 router
    (40, 40, 8, 6, 1),      # ... in the shared-memory top-k
]


@pytest.mark.parametrize("m,g,k,k_dept,strict", WIDE_ROUTERS)
def test_routing_of_wide_and_group_limited_routers(m, g, k, k_dept, strict):
    """Routing only (indices, gate weights, department and expert lists) on layers with tiny experts but
    wide routers, so that every top-k variant (one warp with 8 logits per lane; the wide kernel of 2 - 8 warps per
    token, with and without a group limit; the one-warp variants with 16 / 32 logits per lane, which strict
    coverage still takes; the shared-memory fallback) is compared with the oracle, with random logits and with
    exact ties."""
    shape = synth.LayerShape(f"wide{m}x{g}", hidden=256, n_dept=m, experts_per_dept=g, ffn=16, priv=16, top_k=k,
                             k_dept=k_dept, strict_dept=strict)
    dev = torch.device("cuda:0")
    w = synth.make_deamoe_weights(shape, 2, dev)
    layer = binding.Layer(shape, w, 40)
    try:
        cfg = oracle_cfg(shape)
        for B, seed in ((1, 3), (5, 4), (33, 5), (40, 6)):
            tokens = synth.make_tokens(shape, B, seed, dev)
            layer.route(tokens, want_outputs=False)
            torch.cuda.synchronize()
            want = ref.route(cfg, synth.to_numpy(w["router"]), synth.to_numpy(tokens), want_logits=True)
            safe = want["gap"] > 1e-5 * np.abs(want["logits"]).max(axis=1)
            got = layer.routing(B)
            assert safe.mean() > 0.5
            assert (got["idx"][safe] == want["idx"][safe]).all()
            assert np.abs(got["w"][safe].astype(np.float64) - want["w"][safe]).max() <= 1e-5
            if safe.all():
                bk = ref.bucket(cfg, want["idx"])
                for key in ("dept_mask", "dept_off", "dept_tok", "expert_off", "expert_tok"):
                    assert (got[key] == bk[key]).all(), key
        # exact ties: small integers in the router and the tokens make every logit an exact integer in
        # fp32 and fp64 alike, with many equal values; the order must be (logit descending, index ascending)
        gen = torch.Generator(device="cpu").manual_seed(7)
        router = torch.randint(-2, 3, (shape.n_expert, shape.hidden), generator=gen).float()
        w2 = dict(w)
        w2["router"] = router.to(dev)
        tied = binding.Layer(shape, w2, 8)
        try:
            tokens = torch.randint(-2, 3, (8, shape.hidden), generator=gen).to(torch.bfloat16).to(dev)
            tied.route(tokens, want_outputs=False)
            torch.cuda.synchronize()
            want = ref.route(cfg, synth.to_numpy(w2["router"]), synth.to_numpy(tokens))
            got = tied.routing(8)
            assert (got["idx"] == want["idx"]).all()
            bk = ref.bucket(cfg, want["idx"])
            for key in ("dept_off", "dept_tok", "expert_off", "expert_tok"):
                assert (got[key] == bk[key]).all(), key
        finally:
            tied.close()
    finally:
        layer.close()


@pytest.mark.parametrize("m,g,k,norm,k_dept", [(6, 16, 6, 2, 0), (40, 40, 8, 2, 0), (10, 32, 10, 0, 0),
                                                (16, 80, 10, 0, 5), (40, 40, 8, 2, 6), (40, 40, 8, 0, 6)])
def test_gate_variants_on_every_topk_path(m, g, k, norm, k_dept):
    """The gate-weight variants (logistic scores normalised over the selection; full softmax without
    renormalisation) through the one-warp register top-k (inside the routing tail and, for more tokens than it
    has warps, in the grid of its own), through the wide kernel of several warps per token (whose softmax over all
    experts sums across warps; with and without a group limit) and through the shared-memory top-k."""
    shape = synth.LayerShape(f"gate{m}x{g}", hidden=256, n_dept=m, experts_per_dept=g, ffn=16, priv=16, top_k=k,
                             norm_topk=norm, route_scale=1.5, k_dept=k_dept)
    dev = torch.device("cuda:0")
    w = synth.make_deamoe_weights(shape, 3, dev)
    w["router"] = w["router"] * 8.0  # logits of order one, so the variants differ visibly
    layer = binding.Layer(shape, w, 40)
    try:
        cfg = oracle_cfg(shape)
        for B, seed in ((3, 8), (40, 9)):
            tokens = synth.make_tokens(shape, B, seed, dev)
            layer.route(tokens, want_outputs=False)
            torch.cuda.synchronize()
            want = ref.route(cfg, synth.to_numpy(w["router"]), synth.to_numpy(tokens), want_logits=True)
            safe = want["gap"] > 1e-5 * np.abs(want["logits"]).max(axis=1)
            got = layer.routing(B)
            assert safe.mean() > 0.5
            assert (got["idx"][safe] == want["idx"][safe]).all()
            assert np.abs(got["w"][safe].astype(np.float64) - want["w"][safe]).max() <= 1e-5
        assert layer.stats()["device_status"] == 0
    finally:
        layer.close()

