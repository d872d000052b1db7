"""Parity harness: run the CUDA library and the fp64 oracle on the same seeded layer."""
import numpy as np
import torch

from oracle import ref
from paper_2608_14385_b200 import binding, synth
from tests.common import oracle_cfg, within_tolerance

GAP_GUARD = 1e-5   # relative distance from a routing tie below which fp32 and fp64 may disagree


def lazy_oracle_weights(shape, w, needed_depts, needed_experts, vanilla=False):
    """Host copies of only the department / expert slices the oracle will touch."""
    m, n = shape.n_dept, shape.n_expert
    out = {"router": synth.to_numpy(w["router"])}
    units = n if vanilla else m
    need_units = needed_experts if vanilla else needed_depts
    for name in ("dept_gate", "dept_up", "dept_down"):
        out[name] = [synth.to_numpy(w[name][u]) if u in need_units else None for u in range(units)]
    if not vanilla and shape.priv > 0:
        for name in ("priv_gate", "priv_up", "priv_down"):
            out[name] = [synth.to_numpy(w[name][i]) if i in needed_experts else None for i in range(n)]
    if shape.n_shared:
        for name in ("shared_gate", "shared_up", "shared_down"):
            out[name] = synth.to_numpy(w[name])
    return out


def check_routing(shape, layer, w, tokens, B, require_guard=True):
    """Routing indices, department sets and token lists bit-exact; gate weights within 1e-5."""
    cfg = oracle_cfg(shape)
    want = ref.route(cfg, synth.to_numpy(w["router"]), synth.to_numpy(tokens), want_logits=True)
    scale = np.abs(want["logits"]).max(axis=1) if B else np.zeros(0)
    if require_guard:
        # gap = the smallest margin of ANY comparison the selection rests on (sorted candidates, the
        # department cut of the group limit, a strict-coverage newcomer), so no bit-exact comparison
        # below can hinge on an fp32 / fp64 rounding difference
        assert (want["gap_parts"] > GAP_GUARD * scale[:, None]).all(), "seed too close to a routing tie: pick another"
        assert (want["gap"] == want["gap_parts"].min(axis=1)).all()
    got = layer.routing(B)
    assert (got["idx"] == want["idx"]).all()
    assert np.abs(got["w"].astype(np.float64) - want["w"]).max(initial=0.0) <= 1e-5 * max(1.0, shape.route_scale)
    bk = ref.bucket(cfg, want["idx"])
    for key in ("dept_mask", "dept_off", "dept_tok", "expert_off", "expert_tok"):
        assert got[key].shape == bk[key].shape and (got[key] == bk[key]).all(), key
    return want, bk


def deep_rows(count):
    """Row chooser for run_case: the `count` tokens that sit deepest in a department's token list
    X^j (position 8 and beyond is the second 8-token pass of the streaming kernel's tiles, position 16
    and beyond a second token group), always with the first and the last token of the batch."""
    def choose(want_r, bk):
        B = want_r["idx"].shape[0]
        depth = np.zeros(B, np.int64)
        off = bk["dept_off"]
        for j in range(len(off) - 1):
            toks = bk["dept_tok"][off[j]:off[j + 1]]
            depth[toks] = np.maximum(depth[toks], np.arange(len(toks)))
        order = sorted(range(B), key=lambda t: (-depth[t], t))
        rows = sorted(set(order[:max(0, count - 2)]) | {0, B - 1})
        return rows, int(depth[rows].max())
    return choose


def run_case(shape, B, seed=0, schedule=binding.SCHED_AUTO, vanilla=False, rows=None, max_batch=None,
             weights=None, tokens=None, layer=None, require_guard=True):
    """Build (or reuse) a layer on cuda:0, run one forward, compare with the oracle.
    rows: optional subset of token rows for the (expensive) oracle values."""
    dev = torch.device("cuda:0")
    if weights is None:
        weights = (synth.make_vanilla_weights if vanilla else synth.make_deamoe_weights)(shape, seed, dev)
    if tokens is None:
        tokens = synth.make_tokens(shape, B, seed, dev)
    own = layer is None
    if own:
        layer = binding.Layer(shape, weights, max_batch or max(B, 1), schedule, vanilla=vanilla)
    try:
        out = layer.forward(tokens)
        torch.cuda.synchronize()
        st = layer.stats()
        assert st["device_status"] == 0
        if B == 0:
            return {"out": out, "stats": st}
        want_r, bk = check_routing(shape, layer, weights, tokens, B, require_guard)
        depts = {int(j) for j in np.nonzero(np.diff(bk["dept_off"]))[0]}
        experts = {int(i) for i in np.nonzero(np.diff(bk["expert_off"]))[0]}
        assert st["active_dept"] == len(depts) and st["active_expert"] == len(experts)
        assert st["token_dept_pairs"] == int(bk["dept_off"][-1])
        deepest = None
        if callable(rows):
            rows, deepest = rows(want_r, bk)
        if rows is not None:
            sel = want_r["idx"][rows].reshape(-1)
            experts_needed = {int(i) for i in sel}
            depts_needed = {int(i) // shape.experts_per_dept for i in sel}
        else:
            experts_needed, depts_needed = experts, depts
        ow = lazy_oracle_weights(shape, weights, depts_needed, experts_needed, vanilla)
        cfg = oracle_cfg(shape)
        fwd = ref.vanilla_forward if vanilla else ref.deamoe_forward
        want = fwd(cfg, ow, synth.to_numpy(tokens), rows=rows)
        got = out.float().cpu().numpy().astype(np.float64)
        r = list(range(B)) if rows is None else list(rows)
        ok, err, bound = within_tolerance(got[r], want["out"][r])
        assert ok, f"max|diff| {err:.3e} > {bound:.3e}"
        assert np.abs(want["out"][r]).max() > 0
        return {"out": out, "stats": st, "err": err, "bound": bound, "want": want, "layer": layer, "rows": r,
                "deepest": deepest}
    finally:
        if own:
            layer.close()
