"""Helpers shared by the tests: turn a synthetic layer into what each side takes."""
import numpy as np
import torch

from oracle import ref
from paper_2608_14385_b200 import synth


def oracle_cfg(shape):
    return ref.make_config(**shape.asdict())


def oracle_weights(w):
    """dict of torch tensors -> dict of numpy arrays (fp32 / bf16 bits) for the oracle."""
    return {k: synth.to_numpy(v) for k, v in w.items()}


def widen(t):
    """torch tensor (fp32/bf16) -> float64 numpy, using torch's own conversion."""
    return t.detach().cpu().to(torch.float64).numpy()


def silu(v):
    return v / (1.0 + np.exp(-v))


def within_tolerance(got, want, rel=1e-2, abs_=1e-3):
    """max|got - want| <= rel * max|want| + abs_  (the output tolerance of the layer)."""
    got = np.asarray(got, np.float64)
    want = np.asarray(want, np.float64)
    err = float(np.max(np.abs(got - want))) if got.size else 0.0
    bound = rel * (float(np.max(np.abs(want))) if want.size else 0.0) + abs_
    return err <= bound, err, bound
