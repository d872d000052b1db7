"""Closed-form parameter, FLOP and loaded-weight accounting -- TEST INFRASTRUCTURE.

Plain fp64 Python restating the paper's budget accounting (Section 3.3: total
parameters and per-token FLOPs of a DeaMoE configuration against its standard
MoE baseline, the router included on both sides, Table 1) and the expected
amount of weights loaded per decoding step as a function of the number of
tokens (Fig. 2), plus the exact per-step count for a given routing.

Nothing here is used by the CUDA library.
"""
from math import comb


# ---- Table 1: budget matching (the paper's private matrices are [f, f]) ----

def baseline_params(h, f, n):
    """n independent experts of three [f, h] matrices + router [n, h]."""
    return n * 3 * h * f + n * h


def baseline_flops(h, f, n, k):
    """per-token FLOPs: k experts + router (2 flops per multiply-add)."""
    return 2 * (k * 3 * h * f + n * h)


def deamoe_params(h, f, m, n, r=None):
    """m departments of three [f, h] matrices, n experts of three [r, f], router [n, h]."""
    r = f if r is None else r
    return m * 3 * h * f + n * 3 * r * f + n * h


def deamoe_flops(h, f, n, k_dept, k, r=None):
    """per-token FLOPs with at most k_dept departments and k experts active."""
    r = f if r is None else r
    return 2 * (k_dept * 3 * h * f + k * 3 * r * f + n * h)


# ---- Fig. 2: expected loaded weights per step ----

def expected_unique(total, picks, tokens):
    """E[number of distinct units touched] when each of `tokens` independent
    tokens touches `picks` of `total` units uniformly: total*(1-(1-picks/total)^T)."""
    return total * (1.0 - (1.0 - picks / total) ** tokens)


def expected_loading_ratio(tokens, h, f, n_base, k_base, m, n_dea, k_dept, k_dea, r=None):
    """Expected DeaMoE weights loaded per step / expected baseline weights
    loaded per step, router weights included on both sides (Fig. 2)."""
    r = f if r is None else r
    base = expected_unique(n_base, k_base, tokens) * 3 * h * f + n_base * h
    dea = (expected_unique(m, k_dept, tokens) * 3 * h * f
           + expected_unique(n_dea, k_dea, tokens) * 3 * r * f + n_dea * h)
    return dea / base


def dept_miss_probability(n, g, k):
    """Flat uniform top-k over n experts: probability that one token's k
    distinct experts all fall outside a given department of g experts
    (hypergeometric): C(n-g, k) / C(n, k)."""
    return comb(n - g, k) / comb(n, k)


def expected_active_depts(n, g, k, tokens):
    m = n // g
    return m * (1.0 - dept_miss_probability(n, g, k) ** tokens)


# ---- exact per-step unique bytes for a given routing ----

def unique_bytes_deamoe(n_active_dept, n_active_expert, h, f, r, n, s_w, n_shared=0, shared_ffn=0):
    """|D|*3hf*s_w + |E|*3rf*s_w + shared + fp32 router."""
    return (n_active_dept * 3 * h * f * s_w + n_active_expert * 3 * r * f * s_w
            + n_shared * 3 * h * shared_ffn * s_w + n * h * 4)


def unique_bytes_vanilla(n_active_expert, h, f, n, s_w, n_shared=0, shared_ffn=0):
    return n_active_expert * 3 * h * f * s_w + n_shared * 3 * h * shared_ffn * s_w + n * h * 4


def count_active(topk_idx, g):
    """(|D|, |E|, sum_t |D_t|) from a [B][k] selection given as nested lists."""
    experts, depts, pairs = set(), set(), 0
    for row in topk_idx:
        dt = set(int(i) // g for i in row)
        pairs += len(dt)
        depts |= dt
        experts |= set(int(i) for i in row)
    return len(depts), len(experts), pairs
