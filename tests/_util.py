"""Helpers shared by the GPU parity tests: oracle calls on torch inputs and the error metric."""
import numpy as np
import torch

from oracle import lasad_oracle as orc

TOL = {torch.float32: 1e-4, torch.bfloat16: 2e-2}   # max|err| / max|ref|: fp32 I/O; bf16 I/O with fp32 accumulation


def to64(t):
    return None if t is None else t.detach().to("cpu", torch.float64).numpy()


def oracle(q, k, v, decay, grid_w, prefix_len=0, t0=0, scale=1.0, state_in=None, form="recurrent"):
    """Oracle on the exact values the kernel saw (bf16 inputs are up-converted, not re-drawn)."""
    fn = orc.recurrent if form == "recurrent" else orc.quadratic
    return fn(to64(q), to64(k), to64(v), to64(decay), grid_w, prefix_len, t0, scale, to64(state_in))


def rel_err(got, ref):
    got = to64(got) if isinstance(got, torch.Tensor) else np.asarray(got, dtype=np.float64)
    denom = np.abs(ref).max()
    if denom == 0:
        return float(np.abs(got).max())
    return float(np.abs(got - ref).max() / denom)
