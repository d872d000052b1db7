"""Department-sharded execution, host side, with two CPU ranks (gloo).

Each rank owns a contiguous range of departments (paper Section 3.1: a department and its experts'
private matrices are an independent unit), generates ONLY its slice of the weights, evaluates the
partial sum of Eq. (3) over its own experts with the oracle, and one all-reduce of the [B, h] partial
sums completes the layer.  Checked: the partition arithmetic, that the reduced output equals the
unsharded oracle, that the department sets / token lists of the ranks partition the layer's, and the
per-rank count of unique weight bytes."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

def _shape():
    from paper_2608_14385_b200 import synth
    return synth.LayerShape("shard", hidden=64, n_dept=5, experts_per_dept=3, ffn=48, priv=32, top_k=4,
                            n_shared=1, shared_ffn=32, residual=1)


def _rank(rank, world, port, out):
    sys.path.insert(0, ROOT)
    from oracle import accounting, ref
    from paper_2608_14385_b200 import shard, synth
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    shape = _shape()
    B, g = 7, shape.experts_per_dept
    my_shape, (lo, hi) = shard.slice_shape(shape, rank, world)
    w = synth.make_deamoe_weights(my_shape, 5, dept_range=(lo, hi))          # this rank's slice only
    for k in w:
        if k != "router":
            w[k] = (w[k].float() * 12.0).to(w[k].dtype)
    tokens = synth.make_tokens(shape, B, 5)                                  # replicated
    host = {"router": synth.to_numpy(w["router"])}
    for name in ("gate", "up", "down"):
        host[f"dept_{name}"] = [synth.to_numpy(w[f"dept_{name}"][j - lo]) if lo <= j < hi else None
                                for j in range(shape.n_dept)]
        host[f"priv_{name}"] = [synth.to_numpy(w[f"priv_{name}"][i - lo * g]) if lo <= i // g < hi else None
                                for i in range(shape.n_expert)]
        if my_shape.n_shared:
            host[f"shared_{name}"] = synth.to_numpy(w[f"shared_{name}"])
    cfg = ref.make_config(**my_shape.with_(residual=0).asdict(), dept_range=(lo, hi))
    part = ref.deamoe_forward(cfg, host, synth.to_numpy(tokens))
    total = torch.from_numpy(part["out"].copy())
    dist.all_reduce(total)                                                   # the one collective of the path
    final = total.numpy() + tokens.to(torch.float64).numpy()                 # finish: + residual
    # routing state of this slice: only its own departments' pairs
    mine = [[int(i) for i in row if lo <= int(i) // g < hi] for row in part["idx"]]
    nd, ne, pairs = accounting.count_active(mine, g)
    ub = accounting.unique_bytes_deamoe(nd, ne, shape.hidden, shape.ffn, shape.priv, shape.n_expert, 2,
                                        my_shape.n_shared, my_shape.shared_ffn)
    np.save(os.path.join(out, f"final{rank}.npy"), final)
    np.save(os.path.join(out, f"idx{rank}.npy"), part["idx"])
    open(os.path.join(out, f"meta{rank}.txt"), "w").write(f"{lo} {hi} {nd} {ne} {pairs} {ub} {my_shape.n_shared}")
    dist.barrier()
    dist.destroy_process_group()


def _free_port():
    import socket
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def test_two_ranks_each_holding_half_the_departments_reduce_to_the_layer(tmp_path):
    sys.path.insert(0, ROOT)
    from oracle import accounting, ref
    from paper_2608_14385_b200 import synth
    world = 2
    mp.spawn(_rank, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    shape = _shape()
    w = synth.make_deamoe_weights(shape, 5)
    for k in w:
        if k != "router":
            w[k] = (w[k].float() * 12.0).to(w[k].dtype)
    tokens = synth.make_tokens(shape, 7, 5)
    full = ref.deamoe_forward(ref.make_config(**shape.asdict()), {k: synth.to_numpy(v) for k, v in w.items()},
                              synth.to_numpy(tokens))
    metas = [open(tmp_path / f"meta{r}.txt").read().split() for r in range(world)]
    for r in range(world):
        np.testing.assert_allclose(np.load(tmp_path / f"final{r}.npy"), full["out"], rtol=1e-12, atol=1e-12)
        assert (np.load(tmp_path / f"idx{r}.npy") == full["idx"]).all()
    assert [(int(m[0]), int(m[1])) for m in metas] == [(0, 3), (3, 5)]
    g = shape.experts_per_dept
    nd, ne, pairs = accounting.count_active(full["idx"].tolist(), g)
    assert sum(int(m[2]) for m in metas) == nd and sum(int(m[3]) for m in metas) == ne
    assert sum(int(m[4]) for m in metas) == pairs
    assert [int(m[6]) for m in metas] == [0, 1]                               # one owner of the shared expert
    whole = accounting.unique_bytes_deamoe(nd, ne, shape.hidden, shape.ffn, shape.priv, shape.n_expert, 2, 1,
                                           shape.shared_ffn)
    router_bytes = shape.n_expert * shape.hidden * 4
    assert sum(int(m[5]) for m in metas) == whole + (world - 1) * router_bytes   # the router is read on every rank


def test_department_partition_arithmetic():
    sys.path.insert(0, ROOT)
    from paper_2608_14385_b200 import shard
    import pytest
    for m in (1, 4, 5, 8, 32):
        for world in range(1, m + 1):
            cuts = [shard.dept_slice(m, r, world) for r in range(world)]
            assert cuts[0][0] == 0 and cuts[-1][1] == m
            assert all(a[1] == b[0] for a, b in zip(cuts[:-1], cuts[1:]))
            sizes = [hi - lo for lo, hi in cuts]
            assert max(sizes) - min(sizes) <= 1 and min(sizes) >= 1
            assert sizes[shard.shared_expert_owner(world)] == min(sizes)
    with pytest.raises(ValueError):
        shard.dept_slice(4, 0, 5)
