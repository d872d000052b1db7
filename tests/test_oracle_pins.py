"""Pins for the fp64 oracle: each test ties it to something other than itself --
a reduction between the paper's own definitions, an independently written dense
numpy routine on a special case, brute force on tiny inputs, or an invariant."""
import itertools
import os

import numpy as np
import pytest
import torch

from oracle import ref
from paper_2608_14385_b200 import synth
from tests.common import oracle_cfg, oracle_weights, silu, widen

SMALL = synth.LayerShape("small", hidden=48, n_dept=3, experts_per_dept=4, ffn=40, priv=24, top_k=3,
                         weight_dtype=1, act_dtype=1)


def _layer(shape, seed=0, std=None):
    w = synth.make_deamoe_weights(shape, seed)
    if std is not None:       # larger weights so that non-linearities matter in small layers
        for k in w:
            if k != "router":
                w[k] = (w[k].float() * (std / synth.W_STD)).to(w[k].dtype)
    return w


# ---------------------------------------------------------------- routing (Eq. 2, gate weights)

def test_topk_is_max_sum_subset_bruteforce():
    """Eq. (2): on tiny inputs the selected set must be the k-subset with the largest logit sum."""
    shape = synth.LayerShape("t", hidden=16, n_dept=2, experts_per_dept=4, ffn=8, priv=0, top_k=3,
                             weight_dtype=0, act_dtype=0)
    cfg = oracle_cfg(shape)
    for seed in range(5):
        router = synth.normal((8, 16), 1.0, seed, "r").numpy()
        tokens = synth.normal((6, 16), 1.0, seed, "x").numpy()
        got = ref.route(cfg, router, tokens, want_logits=True)
        np.testing.assert_allclose(got["logits"], tokens.astype(np.float64) @ router.astype(np.float64).T,
                                   rtol=1e-12, atol=1e-12)
        for t in range(6):
            l = got["logits"][t]
            best = max(itertools.combinations(range(8), 3), key=lambda s: sum(l[list(s)]))
            assert set(got["idx"][t]) == set(best)
            assert list(l[got["idx"][t]]) == sorted(l[got["idx"][t]], reverse=True)


def test_topk_ties_go_to_lowest_index_all_permutations():
    """Exactly representable logits with repeated values, every ordering of the experts."""
    shape = synth.LayerShape("t", hidden=4, n_dept=1, experts_per_dept=5, ffn=8, priv=0, top_k=3,
                             weight_dtype=0, act_dtype=0)
    cfg = oracle_cfg(shape)
    values = [2.0, 1.0, 1.0, 1.0, 0.5]
    tokens = np.array([[1.0, 0.0, 0.0, 0.0]], np.float32)
    for perm in itertools.permutations(range(5)):
        router = np.zeros((5, 4), np.float32)
        for slot, src in enumerate(perm):
            router[slot, 0] = values[src]
        got = ref.route(cfg, router, tokens)["idx"][0]
        order = sorted(range(5), key=lambda i: (-router[i, 0], i))[:3]
        assert list(got) == order
    # all logits equal: the first k indices in order
    got = ref.route(cfg, np.ones((5, 4), np.float32), tokens)
    assert list(got["idx"][0]) == [0, 1, 2]
    assert got["gap"][0] == 0.0


def test_gate_weights_are_renormalised_full_softmax():
    """p over the selection == softmax over all n followed by renormalisation; sum == route_scale;
    norm_topk = 0 returns the plain full-softmax entries."""
    shape = SMALL.with_(route_scale=2.5)
    cfg = oracle_cfg(shape)
    router = synth.normal((12, 48), 0.3, 1, "r").numpy()
    tokens = synth.to_numpy(synth.make_tokens(shape, 5, 1))
    got = ref.route(cfg, router, tokens, want_logits=True)
    full = np.exp(got["logits"] - got["logits"].max(1, keepdims=True))
    full /= full.sum(1, keepdims=True)
    for t in range(5):
        sel = full[t, got["idx"][t]]
        np.testing.assert_allclose(got["w"][t], 2.5 * sel / sel.sum(), rtol=1e-12)
        assert abs(got["w"][t].sum() - 2.5) < 1e-12
    cfg0 = oracle_cfg(shape.with_(norm_topk=0, route_scale=1.0))
    got0 = ref.route(cfg0, router, tokens)
    for t in range(5):
        np.testing.assert_allclose(got0["w"][t], full[t, got0["idx"][t]], rtol=1e-12)


def test_sigmoid_gate_variant_against_the_library_routine_and_its_limits():
    """norm_topk = 2 (a variant the paper does not have): the selection is unchanged, the weights
    are the logistic function of the selected logits (scipy's routine) normalised over the
    selection; they sum to route_scale, are ordered like the logits, and for very negative logits
    (where the logistic function tends to exp) they tend to the softmax weights."""
    from scipy.special import expit
    shape = SMALL.with_(route_scale=2.5, norm_topk=2)
    router = synth.normal((12, 48), 0.3, 1, "r").numpy()
    tokens = synth.to_numpy(synth.make_tokens(shape, 5, 1))
    got = ref.route(oracle_cfg(shape), router, tokens, want_logits=True)
    soft = ref.route(oracle_cfg(shape.with_(norm_topk=1)), router, tokens)
    assert (got["idx"] == soft["idx"]).all()
    for t in range(5):
        s = expit(got["logits"][t, got["idx"][t]])
        np.testing.assert_allclose(got["w"][t], 2.5 * s / s.sum(), rtol=1e-12)
        assert abs(got["w"][t].sum() - 2.5) < 1e-12
        assert (np.diff(got["w"][t]) <= 0).all()  # selection order is logit descending
        assert not np.allclose(got["w"][t], soft["w"][t], rtol=1e-3)
    # shift every logit by -40 through one extra input column: logistic(l) -> exp(l) (1 - O(e^-40))
    router2 = np.concatenate([router, np.full((12, 1), -40.0, np.float32)], axis=1)
    tokens2 = np.concatenate([synth.normal((5, 48), 1.0, 2, "x").numpy(), np.ones((5, 1), np.float32)], axis=1)
    shape2 = shape.with_(hidden=49, act_dtype=0)
    far = ref.route(oracle_cfg(shape2), router2, tokens2)
    far_soft = ref.route(oracle_cfg(shape2.with_(norm_topk=1)), router2, tokens2)
    np.testing.assert_allclose(far["w"], far_soft["w"], rtol=1e-12)


def test_group_limited_routing_bruteforce():
    """k_dept cap: the selection is the flat top-k restricted to the k_dept departments with the
    largest best logit, so it never spans more than k_dept departments; k_dept = m changes nothing."""
    shape = synth.LayerShape("t", hidden=16, n_dept=4, experts_per_dept=3, ffn=8, priv=0, top_k=4,
                             k_dept=2, weight_dtype=0, act_dtype=0)
    router = synth.normal((12, 16), 1.0, 3, "r").numpy()
    tokens = synth.normal((9, 16), 1.0, 3, "x").numpy()
    got = ref.route(oracle_cfg(shape), router, tokens, want_logits=True)
    flat = ref.route(oracle_cfg(shape.with_(k_dept=4)), router, tokens)
    free = ref.route(oracle_cfg(shape.with_(k_dept=0)), router, tokens)
    assert (flat["idx"] == free["idx"]).all()
    for t in range(9):
        l = got["logits"][t]
        score = [max(l[j * 3:(j + 1) * 3]) for j in range(4)]
        keep = sorted(range(4), key=lambda j: (-score[j], j))[:2]
        cand = [i for i in range(12) if i // 3 in keep]
        want = sorted(cand, key=lambda i: (-l[i], i))[:4]
        assert list(got["idx"][t]) == want
        assert len({i // 3 for i in got["idx"][t]}) <= 2


def test_strict_department_coverage_properties():
    """The strict variant of Section 3.3: every token ends up with exactly min(k_dept, k)
    departments; a token whose soft selection already has that many is untouched; otherwise only
    lowest-ranked duplicates leave (the highest-ranked expert of every covered department stays, the
    number of swaps is the number of missing departments), and every newcomer is the best expert of
    its department, taken from the best-scoring uncovered departments."""
    shape = synth.LayerShape("t", hidden=16, n_dept=6, experts_per_dept=6, ffn=8, priv=0, top_k=4,
                             k_dept=4, weight_dtype=0, act_dtype=0)
    g, m, k, kd = 6, 6, 4, 4
    router = synth.normal((36, 16), 1.0, 7, "r").numpy()
    tokens = synth.normal((64, 16), 1.0, 7, "x").numpy()
    soft = ref.route(oracle_cfg(shape), router, tokens, want_logits=True)
    strict = ref.route(oracle_cfg(shape.with_(strict_dept=1)), router, tokens)
    changed_tokens = 0
    for t in range(64):
        l = soft["logits"][t]
        a, b = list(soft["idx"][t]), list(strict["idx"][t])
        da, db = [i // g for i in a], [i // g for i in b]
        assert len(set(b)) == k and len(set(db)) == min(kd, k)
        missing = min(kd, k) - len(set(da))
        assert sum(x != y for x, y in zip(a, b)) == missing
        if missing == 0:
            continue
        changed_tokens += 1
        for q, (x, y) in enumerate(zip(a, b)):
            if x != y:
                assert da[q] in da[:q]                       # a lower-ranked duplicate left ...
                assert y == max(range(db[q] * g, db[q] * g + g), key=lambda i: (l[i], -i))   # ... for a department's best
                assert db[q] not in da
        # the departments that came in are the best-scoring uncovered ones
        score = {j: max(l[j * g:(j + 1) * g]) for j in range(m) if j not in da}
        came = sorted(set(db) - set(da))
        assert came == sorted(sorted(score, key=lambda j: (-score[j], j))[:missing])
        # no higher-ranked duplicate stayed while a lower-ranked one of another department left
        left = [q for q in range(k) if a[q] != b[q]]
        stay_dups = [q for q in range(k) if a[q] == b[q] and da[q] in da[:q]]
        assert all(q < min(left) for q in stay_dups)
    assert changed_tokens >= 5                               # the case is exercised
    w_sum = strict["w"].sum(axis=1)
    np.testing.assert_allclose(w_sum, 1.0, rtol=1e-12)
    off = ref.route(oracle_cfg(shape.with_(strict_dept=1, k_dept=0)), router, tokens)   # no cap: nothing to enforce
    free = ref.route(oracle_cfg(shape.with_(k_dept=0)), router, tokens)
    assert (off["idx"] == free["idx"]).all()


# ---------------------------------------------------------------- Section 3.2 sets and lists

def test_bucketing_matches_python_sets():
    shape = SMALL
    cfg = oracle_cfg(shape)
    g, m, n = shape.experts_per_dept, shape.n_dept, shape.n_expert
    for seed in range(4):
        B = 1 + 3 * seed
        picks = synth.uniform_ints(B * n, 1 << 20, seed, "pick")
        idx = np.array([sorted(range(n), key=lambda i: (picks[t * n + i], i))[:shape.top_k]
                        for t in range(B)], np.int32)
        got = ref.bucket(cfg, idx)
        for j in range(m):
            want = [t for t in range(B) if any(i // g == j for i in idx[t])]
            assert list(got["dept_tok"][got["dept_off"][j]:got["dept_off"][j + 1]]) == want
            assert bool(int(got["dept_mask"][0]) >> j & 1) == bool(want)
        for i in range(n):
            want = [t for t in range(B) if i in idx[t]]
            assert list(got["expert_tok"][got["expert_off"][i]:got["expert_off"][i + 1]]) == want
        assert got["expert_off"][n] == B * shape.top_k


# ---------------------------------------------------------------- reductions of Eq. (4)

def test_one_expert_per_department_without_private_parts_is_vanilla_moe():
    """g = 1, no private parameters, no interface non-linearity: Eq. (4) is Eq. (1), and the
    DeaMoE layer must equal the standard MoE layer on the same matrices."""
    shape = synth.LayerShape("p1", hidden=32, n_dept=6, experts_per_dept=1, ffn=24, priv=0, top_k=2,
                             sigma=0, n_shared=1, shared_ffn=16)
    cfg = oracle_cfg(shape)
    w = oracle_weights(_layer(shape, 2, std=0.3))
    tokens = synth.to_numpy(synth.make_tokens(shape, 5, 2))
    a = ref.deamoe_forward(cfg, w, tokens)
    b = ref.vanilla_forward(cfg, w, tokens)
    assert (a["idx"] == b["idx"]).all()
    np.testing.assert_allclose(a["out"], b["out"], rtol=1e-13, atol=1e-15)
    assert np.abs(a["out"]).max() > 1e-3


def _dense_swiglu(Wg, Wu, Wd, x):
    """Eq. (1) with numpy matmuls on torch-widened matrices (independent of the oracle's loops)."""
    return Wd.T @ (silu(Wg @ x) * (Wu @ x))


def test_no_private_parameters_collapse_to_department_ffn():
    """priv = 0 and sigma = none: every selected expert is its department's plain SwiGLU FFN, so
    out_t = sum_j (sum of p over the picks in department j) * SwiGLU_j(x_t) (+ shared expert)."""
    shape = SMALL.with_(priv=0, sigma=0, n_shared=1, shared_ffn=20)
    cfg = oracle_cfg(shape)
    wt = _layer(shape, 3, std=0.25)
    tokens_t = synth.make_tokens(shape, 6, 3)
    got = ref.deamoe_forward(cfg, oracle_weights(wt), synth.to_numpy(tokens_t))
    X = widen(tokens_t)
    Wg, Wu, Wd = (widen(wt[f"dept_{k}"]) for k in ("gate", "up", "down"))
    Sg, Su, Sd = (widen(wt[f"shared_{k}"]) for k in ("gate", "up", "down"))
    for t in range(6):
        want = _dense_swiglu(Sg, Su, Sd, X[t])
        for i, p in zip(got["idx"][t], got["w"][t]):
            j = i // shape.experts_per_dept
            want = want + p * _dense_swiglu(Wg[j], Wu[j], Wd[j], X[t])
        np.testing.assert_allclose(got["out"][t], want, rtol=1e-11, atol=1e-14)
    assert np.abs(got["out"]).max() > 1e-3


def test_identity_private_matrices_give_the_department_backbone_and_zero_gives_zero():
    """Square A = I with SiLU interfaces: every expert of department j computes
    Wd^T SiLU( SiLU(SiLU(Wg x)) * SiLU(Wu x) ) -- the identity-initialisation property --
    and equals the priv = 0 shorthand; A = 0 gives exactly 0."""
    f = 40
    shape = SMALL.with_(priv=f)
    cfg = oracle_cfg(shape)
    wt = _layer(shape, 4, std=0.3)
    eye = torch.eye(f).to(torch.bfloat16).expand(shape.n_expert, f, f).contiguous()
    for k in ("gate", "up", "down"):
        wt[f"priv_{k}"] = eye
    tokens_t = synth.make_tokens(shape, 4, 4)
    tokens = synth.to_numpy(tokens_t)
    got = ref.deamoe_forward(cfg, oracle_weights(wt), tokens)
    X = widen(tokens_t)
    Wg, Wu, Wd = (widen(wt[f"dept_{k}"]) for k in ("gate", "up", "down"))
    for t in range(4):
        want = np.zeros(shape.hidden)
        for i, p in zip(got["idx"][t], got["w"][t]):
            j = i // shape.experts_per_dept
            want += p * (Wd[j].T @ silu(silu(silu(Wg[j] @ X[t])) * silu(Wu[j] @ X[t])))
        np.testing.assert_allclose(got["out"][t], want, rtol=1e-11, atol=1e-14)
    short = ref.deamoe_forward(oracle_cfg(shape.with_(priv=0)), oracle_weights(wt), tokens)
    np.testing.assert_allclose(short["out"], got["out"], rtol=1e-13, atol=1e-16)
    for k in ("gate", "up", "down"):
        wt[f"priv_{k}"] = torch.zeros_like(eye)
    zero = ref.deamoe_forward(cfg, oracle_weights(wt), tokens)
    assert np.all(zero["out"] == 0.0)


def test_selection_matrices_pin_orientation_of_private_transforms():
    """Private matrices that are 0/1 selections: A_g picks G[pg], A_u picks U[pu] and A_d^T scatters
    Y into Z, so Eq. (4) can be written with index arithmetic only.  Catches a transposed A_d, a
    gate/up swap and a misplaced non-linearity."""
    shape = SMALL.with_(n_dept=1, experts_per_dept=2, top_k=1)
    cfg = oracle_cfg(shape)
    h, f, r = shape.hidden, shape.ffn, shape.priv
    wt = _layer(shape, 5, std=0.4)
    pg = np.array(synth.uniform_ints(r, f, 5, "pg"))
    pu = np.array(synth.uniform_ints(r, f, 5, "pu"))
    pd = np.array(synth.uniform_ints(r, f, 5, "pd"))

    def sel(p):
        a = np.zeros((r, f), np.float32)
        a[np.arange(r), p] = 1.0
        return synth.to_numpy(torch.from_numpy(a).to(torch.bfloat16))
    Wg, Wu, Wd = (widen(wt[f"dept_{k}"][0]) for k in ("gate", "up", "down"))
    w0 = [synth.to_numpy(wt[f"dept_{k}"][0]) for k in ("gate", "up", "down")]
    x = widen(synth.make_tokens(shape, 1, 5))[0]
    out, G, U, Y, Z = ref.deamoe_expert(cfg, *w0, sel(pg), sel(pu), sel(pd), x, taps=True)
    G_w, U_w = silu(Wg @ x), silu(Wu @ x)
    Y_w = silu(G_w[pg]) * U_w[pu]
    Zpre = np.zeros(f)
    np.add.at(Zpre, pd, Y_w)
    np.testing.assert_allclose(G, G_w, rtol=1e-12)
    np.testing.assert_allclose(U, U_w, rtol=1e-12)
    np.testing.assert_allclose(Y, Y_w, rtol=1e-12)
    np.testing.assert_allclose(Z, silu(Zpre), rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(out, Wd.T @ silu(Zpre), rtol=1e-11, atol=1e-14)


# ---------------------------------------------------------------- invariants

def test_layer_invariants():
    """Row t of a batch equals the layer on token t alone; permuting tokens permutes rows;
    relabelling the experts inside a department (router rows and private matrices together)
    leaves the output unchanged; the routed part is linear in route_scale."""
    shape = SMALL
    cfg = oracle_cfg(shape)
    wt = _layer(shape, 6, std=0.3)
    w = oracle_weights(wt)
    tok_t = synth.make_tokens(shape, 5, 6)
    tok = synth.to_numpy(tok_t)
    full = ref.deamoe_forward(cfg, w, tok)
    assert np.abs(full["out"]).max() > 1e-4
    for t in range(5):
        one = ref.deamoe_forward(cfg, w, tok[t:t + 1])
        assert (one["out"][0] == full["out"][t]).all()
    sub = ref.deamoe_forward(cfg, w, tok, rows=[3, 1])
    assert (sub["out"][[3, 1]] == full["out"][[3, 1]]).all() and (sub["out"][0] == 0).all()
    perm = [4, 2, 0, 3, 1]
    pf = ref.deamoe_forward(cfg, w, tok[perm])
    assert (pf["out"] == full["out"][perm]).all()
    # relabel experts inside each department
    g = shape.experts_per_dept
    relabel = np.concatenate([j * g + np.array([2, 0, 3, 1]) for j in range(shape.n_dept)])
    w2 = dict(w)
    for k in ("router", "priv_gate", "priv_up", "priv_down"):
        w2[k] = np.ascontiguousarray(w[k][relabel])
    rf = ref.deamoe_forward(cfg, w2, tok)
    np.testing.assert_allclose(rf["out"], full["out"], rtol=1e-12, atol=1e-16)
    assert (relabel[rf["idx"]] == full["idx"]).all()
    scaled = ref.deamoe_forward(oracle_cfg(shape.with_(route_scale=3.0)), w, tok)
    np.testing.assert_allclose(scaled["out"], 3.0 * full["out"], rtol=1e-12)
    res = ref.deamoe_forward(oracle_cfg(shape.with_(residual=1)), w, tok)
    np.testing.assert_allclose(res["out"], full["out"] + widen(tok_t), rtol=1e-12)


def test_bf16_and_fp32_storage_agree_on_the_same_numbers():
    """The same bf16-representable numbers stored as fp32 give the same output bit for bit."""
    shape = SMALL
    wt = _layer(shape, 7, std=0.3)
    tok_t = synth.make_tokens(shape, 3, 7)
    a = ref.deamoe_forward(oracle_cfg(shape), oracle_weights(wt), synth.to_numpy(tok_t))
    w32 = {k: v.float() for k, v in wt.items()}
    b = ref.deamoe_forward(oracle_cfg(shape.with_(weight_dtype=0, act_dtype=0)), oracle_weights(w32),
                           synth.to_numpy(tok_t.float()))
    assert (a["out"] == b["out"]).all()


# ---------------------------------------------------------------- accounting (Table 1, Fig. 2)

def _golden(name):
    path = os.path.join(os.path.dirname(__file__), "golden", name)
    return [ln.split() for ln in open(path) if ln.strip() and not ln.startswith("#")]


def test_table1_budget_ratios_reproduce_to_the_printed_digit():
    from oracle import accounting as acc
    for name, kb, h, f, nb, m, n, kd, k, fx, px in _golden("table1_budget_ratios.txt"):
        kb, h, f, nb, m, n, kd, k = map(int, (kb, h, f, nb, m, n, kd, k))
        params = acc.deamoe_params(h, f, m, n) / acc.baseline_params(h, f, nb)
        flops = acc.deamoe_flops(h, f, n, kd, k) / acc.baseline_flops(h, f, nb, kb)
        assert abs(params - float(px)) <= 0.00051, (name, params)
        if fx != "-":
            assert abs(flops - float(fx)) <= 0.00051, (name, flops)


def test_fig2_loading_ratio_range_for_the_deepseek_v3_row():
    from oracle import accounting as acc
    gold = {k: float(v) for k, v in _golden("fig2_loading_ratio.txt")}
    ratios = [acc.expected_loading_ratio(T, 7168, 2048, 256, 8, 8, 864, 5, 10) for T in range(4, 65)]
    assert abs(min(ratios) - gold["min_ratio_tokens_4_to_64"]) < 0.00051
    assert abs(max(ratios) - gold["max_ratio_tokens_4_to_64"]) < 0.00051
    assert abs((1 - min(ratios)) - gold["max_reduction"]) < 0.00051
    # non-monotone: falls from 4 tokens to its minimum, then rises again towards 1
    lo = ratios.index(min(ratios))
    assert 0 < lo < len(ratios) - 1
    assert acc.expected_loading_ratio(4096, 7168, 2048, 256, 8, 8, 864, 5, 10) > 0.97


def test_expected_active_departments_matches_counted_routings():
    """Hypergeometric closed form for flat uniform top-k against Monte-Carlo counting with the
    oracle's own bucketing, at the DeepSeek-V3 benchmark layout (32 x 8 experts, top-8)."""
    from oracle import accounting as acc
    n, g, k, B, trials = 256, 8, 8, 8, 300
    shape = synth.LayerShape("t", hidden=8, n_dept=32, experts_per_dept=8, ffn=8, priv=0, top_k=8)
    cfg = oracle_cfg(shape)
    rnd = synth.uniform_ints(trials * B * n, 1 << 30, 11, "mc")
    tot_d = tot_e = 0
    for s in range(trials):
        idx = []
        for t in range(B):
            v = rnd[(s * B + t) * n:(s * B + t + 1) * n]
            idx.append(sorted(range(n), key=lambda i: (v[i], i))[:k])
        got = ref.bucket(cfg, np.array(idx, np.int32))
        nd, ne, _ = acc.count_active(idx, g)
        assert nd == bin(int(got["dept_mask"][0])).count("1")
        assert ne == int((np.diff(got["expert_off"]) > 0).sum())
        tot_d += nd
        tot_e += ne
    assert abs(tot_d / trials - acc.expected_active_depts(n, g, k, B)) < 0.25
    assert abs(tot_e / trials - acc.expected_unique(n, k, B)) < 0.6
    assert abs(acc.dept_miss_probability(256, 8, 8) - 0.7729) < 1e-4


def test_unique_bytes_closed_form_against_vanilla():
    from oracle import accounting as acc
    h, f, r, n = 7168, 2048, 896, 256
    dea = acc.unique_bytes_deamoe(7, 8, h, f, r, n, 2, 1, 2048)
    van = acc.unique_bytes_vanilla(8, h, f, n, 2, 1, 2048)
    assert dea == 7 * 88080384 + 8 * 11010048 + 88080384 + 7340032
    assert van == 8 * 88080384 + 88080384 + 7340032


# ---------------------------------------------------------------- sigma = RMSNorm (Section 3.4, Table 4)

def test_rmsnorm_sigma_against_the_library_routine_and_its_invariants():
    """sigma = RMSNorm normalises the three length-f vectors of Eq. (4).  Pinned by (1) the taps
    G, U, Z against torch.nn.functional.rms_norm applied to the un-normalised vectors (sigma = none
    taps, re-built here with dense numpy for Z), (2) unit mean square of each tap, (3) invariance of
    the expert's output under scaling W_g, W_u or A_d by powers of two (exact in bf16), which
    element-wise operators do not have."""
    shape = SMALL.with_(sigma=ref.SIGMA_RMSNORM)
    cfg = oracle_cfg(shape)
    wt = _layer(shape, 8, std=0.3)
    x = widen(synth.make_tokens(shape, 1, 8))[0]
    j, i = 1, 1 * shape.experts_per_dept + 2
    Wg, Wu, Wd = (synth.to_numpy(wt[f"dept_{k}"][j]) for k in ("gate", "up", "down"))
    Ag, Au, Ad = (synth.to_numpy(wt[f"priv_{k}"][i]) for k in ("gate", "up", "down"))
    out, G, U, Y, Z = ref.deamoe_expert(cfg, Wg, Wu, Wd, Ag, Au, Ad, x, taps=True)
    raw_cfg = oracle_cfg(shape.with_(sigma=ref.SIGMA_NONE))
    _, G0, U0, _, _ = ref.deamoe_expert(raw_cfg, Wg, Wu, Wd, Ag, Au, Ad, x, taps=True)

    def lib_rms(v):
        return torch.nn.functional.rms_norm(torch.from_numpy(v), (v.size,), eps=1e-6).numpy()

    np.testing.assert_allclose(G, lib_rms(G0), rtol=1e-12)
    np.testing.assert_allclose(U, lib_rms(U0), rtol=1e-12)
    Z0 = widen(wt["priv_down"][i]).T @ Y          # (A_d)^T Y, before the last sigma
    np.testing.assert_allclose(Z, lib_rms(Z0), rtol=1e-11)
    np.testing.assert_allclose(out, widen(wt["dept_down"][j]).T @ Z, rtol=1e-11, atol=1e-14)
    for v, v0 in ((G, G0), (U, U0), (Z, Z0)):
        ms0 = np.mean(v0 * v0)
        assert abs(np.mean(v * v) - ms0 / (ms0 + 1e-6)) < 1e-12
    # scale invariance (up to the epsilon): doubling W_g, quartering W_u, doubling A_d
    wt2 = {k: v.clone() for k, v in wt.items()}
    wt2["dept_gate"] = (wt["dept_gate"].float() * 2).to(torch.bfloat16)
    wt2["dept_up"] = (wt["dept_up"].float() * 0.25).to(torch.bfloat16)
    wt2["priv_down"] = (wt["priv_down"].float() * 2).to(torch.bfloat16)
    out2 = ref.deamoe_expert(cfg, synth.to_numpy(wt2["dept_gate"][j]), synth.to_numpy(wt2["dept_up"][j]), Wd,
                             Ag, Au, synth.to_numpy(wt2["priv_down"][i]), x)
    np.testing.assert_allclose(out2, out, rtol=2e-5, atol=1e-9)
    # ... which SiLU does not have
    s_cfg = oracle_cfg(shape.with_(sigma=ref.SIGMA_SILU))
    a = ref.deamoe_expert(s_cfg, Wg, Wu, Wd, Ag, Au, Ad, x)
    b = ref.deamoe_expert(s_cfg, synth.to_numpy(wt2["dept_gate"][j]), Wu, Wd, Ag, Au, Ad, x)
    assert np.abs(a - b).max() > 1e-3 * np.abs(a).max()


# ---------------------------------------------------------------- sigma = GeLU (Section 3.4, Table 4)

def test_gelu_sigma_against_the_library_routine_and_textbook_values():
    """sigma = GeLU is the exact (erf) form x Phi(x).  Pinned by (1) the taps G, U, Z against
    torch.nn.functional.gelu(approximate="none") and scipy's normal CDF applied to the
    un-transformed vectors (sigma = none taps; Z re-built with dense numpy), (2) textbook values
    of the standard normal CDF: GeLU(1) = Phi(1) = 0.8413447460685429, which the tanh
    approximation (0.8411919906082768) misses in the fourth digit, so neither a switch to that
    form nor a wrong 1/sqrt(2) passes."""
    from scipy.special import ndtr
    shape = SMALL.with_(sigma=ref.SIGMA_GELU)
    cfg = oracle_cfg(shape)
    wt = _layer(shape, 9, std=0.3)
    x = widen(synth.make_tokens(shape, 1, 9))[0]
    j, i = 2, 2 * shape.experts_per_dept + 1
    Wg, Wu, Wd = (synth.to_numpy(wt[f"dept_{k}"][j]) for k in ("gate", "up", "down"))
    Ag, Au, Ad = (synth.to_numpy(wt[f"priv_{k}"][i]) for k in ("gate", "up", "down"))
    out, G, U, Y, Z = ref.deamoe_expert(cfg, Wg, Wu, Wd, Ag, Au, Ad, x, taps=True)
    raw_cfg = oracle_cfg(shape.with_(sigma=ref.SIGMA_NONE))
    _, G0, U0, _, _ = ref.deamoe_expert(raw_cfg, Wg, Wu, Wd, Ag, Au, Ad, x, taps=True)

    def lib_gelu(v):
        return torch.nn.functional.gelu(torch.from_numpy(v), approximate="none").numpy()

    assert np.abs(G0).max() > 1.0 and np.abs(U0).max() > 1.0      # arguments where the forms differ
    np.testing.assert_allclose(G, lib_gelu(G0), rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(U, lib_gelu(U0), rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(G, G0 * ndtr(G0), rtol=1e-12, atol=1e-15)
    Z0 = widen(wt["priv_down"][i]).T @ Y          # (A_d)^T Y, before the last sigma
    np.testing.assert_allclose(Z, lib_gelu(Z0), rtol=1e-10, atol=1e-14)
    np.testing.assert_allclose(out, widen(wt["dept_down"][j]).T @ Z, rtol=1e-11, atol=1e-14)
    tanh_form = 0.5 * G0 * (1.0 + np.tanh(np.sqrt(2.0 / np.pi) * (G0 + 0.044715 * G0 ** 3)))
    assert np.abs(G - tanh_form).max() > 1e-5      # the approximation is told apart
    # textbook values through the oracle itself: identity department matrices (fp32, no private part),
    # so the tap G is sigma applied to the token
    eye = synth.LayerShape("eye", hidden=4, n_dept=1, experts_per_dept=1, ffn=4, priv=0, top_k=1,
                           sigma=ref.SIGMA_GELU, weight_dtype=0, act_dtype=0)
    I4 = np.eye(4, dtype=np.float32)
    xs = np.array([1.0, -1.0, 0.5, 2.0])
    _, Gt, Ut, _, _ = ref.deamoe_expert(oracle_cfg(eye), I4, I4, I4, None, None, None, xs, taps=True)
    phi = np.array([0.8413447460685429, 0.15865525393145707, 0.6914624612740131, 0.9772498680518208])
    np.testing.assert_allclose(Gt, xs * phi, rtol=1e-14)
    np.testing.assert_allclose(Ut, xs * phi, rtol=1e-14)
    assert abs(Gt[0] - 0.8411919906082768) > 1e-4   # not the tanh form


# ---------------------------------------------------------------- the tie-guard diagnostics

def test_routing_gaps_report_every_comparison_that_decides_a_selection():
    """oracle.ref.route reports, per token, the smallest margin of any comparison its selection
    rests on: neighbours among the sorted candidates, the department cut of the group limit
    (Section 3.3) and the choice of a newcomer under strict coverage.  Hand-built logits (the router
    is the identity, so the logits are the token) put a near-tie at each place in turn."""
    g, m, k = 3, 4, 3
    n = g * m
    base = synth.LayerShape("gaps", hidden=n, n_dept=m, experts_per_dept=g, ffn=8, priv=0, top_k=k,
                            weight_dtype=0, act_dtype=0)
    router = np.eye(n, dtype=np.float32)
    #          dept 0          dept 1          dept 2          dept 3
    l = np.array([[9.0, 8.0, 1.0, 7.0, 0.5, 0.25, 6.5, 0.1, 0.2, 6.25, 0.3, 0.4]], np.float32)
    flat = ref.route(oracle_cfg(base), router, l)
    assert list(flat["idx"][0]) == [0, 1, 3]
    np.testing.assert_allclose(flat["gap_parts"][0], [0.5, np.inf, np.inf])      # 7.0 against 6.5 left out
    assert flat["gap"][0] == 0.5
    cut = ref.route(oracle_cfg(base.with_(k_dept=2)), router, l)                 # departments 0, 1 stay (9, 7 | 6.5)
    assert list(cut["idx"][0]) == [0, 1, 3]
    np.testing.assert_allclose(cut["gap_parts"][0], [1.0, 0.5, np.inf])          # candidates 9 8 7 | 1; cut 7 - 6.5
    assert cut["gap"][0] == 0.5
    l2 = l.copy()
    l2[0, 6] = np.float32(7.0) - np.float32(2.0 ** -20)                          # department 2 almost ties department 1
    near = ref.route(oracle_cfg(base.with_(k_dept=2)), router, l2)
    assert near["gap_parts"][0, 1] == pytest.approx(2.0 ** -20) and near["gap"][0] == near["gap_parts"][0, 1]
    assert near["gap_parts"][0, 0] == 1.0                                        # the flat candidates are far apart
    # strict coverage with k_dept = 3: selection 0, 1, 3 covers two departments; expert 1 (the lower
    # duplicate of department 0) is replaced by the best expert of departments 2, 3: 6.5 against 6.25
    strict = ref.route(oracle_cfg(base.with_(k_dept=3, strict_dept=1)), router, l)
    assert list(strict["idx"][0]) == [0, 6, 3]
    np.testing.assert_allclose(strict["gap_parts"][0], [0.5, 0.25, 0.25])        # 7 - 6.5; cut 6.5 - 6.25; newcomer 6.5 - 6.25
    l3 = l.copy()
    l3[0, 9] = 6.5                                                               # exact tie for the newcomer
    tied = ref.route(oracle_cfg(base.with_(k_dept=4, strict_dept=1)), router, l3)
    assert list(tied["idx"][0]) == [0, 6, 3]
    assert tied["gap_parts"][0, 2] == 0.0 and tied["gap"][0] == 0.0
    assert 9 not in tied["idx"][0]                                               # ties go to the lower index


# ---------------------------------------------------------------- department slices (sharded layer)

def test_department_slices_add_up_to_the_layer():
    """Eq. (3) is a sum over the selected experts and the departments are independent units
    (Section 3.1), so for ANY partition of the departments the slices' partial sums (the shared expert
    on exactly one of them, the residual on none) add up to the layer's output.  Also: a slice that
    holds no selected expert of a token contributes exactly zero for it, and the slice generator gives
    the same numbers as indexing the full tensors."""
    shape = synth.LayerShape("sl", hidden=48, n_dept=5, experts_per_dept=3, ffn=40, priv=24, top_k=4,
                             n_shared=1, shared_ffn=32, residual=1)
    wt = _layer(shape, 11, std=0.3)
    w = oracle_weights(wt)
    tokens = synth.to_numpy(synth.make_tokens(shape, 6, 11))
    full = ref.deamoe_forward(oracle_cfg(shape), w, tokens)
    x = widen(synth.make_tokens(shape, 6, 11))
    for cuts in ([0, 2, 5], [0, 1, 2, 5], [0, 5], [0, 4, 5]):
        total = np.zeros_like(full["out"])
        for r, (lo, hi) in enumerate(zip(cuts[:-1], cuts[1:])):
            own_shared = r == len(cuts) - 2
            sl = shape.with_(n_shared=1 if own_shared else 0, residual=0)
            cfg = ref.make_config(**sl.asdict(), dept_range=(lo, hi))
            wr = dict(w)
            for name in ("dept_gate", "dept_up", "dept_down"):        # a slice only has its own departments
                wr[name] = [w[name][j] if lo <= j < hi else None for j in range(shape.n_dept)]
            for name in ("priv_gate", "priv_up", "priv_down"):
                wr[name] = [w[name][i] if lo <= i // 3 < hi else None for i in range(shape.n_expert)]
            part = ref.deamoe_forward(cfg, wr, tokens)
            assert (part["idx"] == full["idx"]).all()                 # every slice routes all tokens alike
            for t in range(6):
                if not any(lo <= i // 3 < hi for i in full["idx"][t]) and not own_shared:
                    assert (part["out"][t] == 0).all()
            total += part["out"]
        np.testing.assert_allclose(total + x, full["out"], rtol=1e-12, atol=1e-13)
    sliced = synth.make_deamoe_weights(shape, 11, dept_range=(1, 4))
    whole = synth.make_deamoe_weights(shape, 11)
    assert torch.equal(sliced["dept_down"], whole["dept_down"][1:4])
    assert torch.equal(sliced["priv_gate"], whole["priv_gate"][3:12])
    assert torch.equal(sliced["router"], whole["router"])
