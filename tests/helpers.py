"""Shared test helpers: array conversion between the seeded inputs and the two sides."""
import numpy as np
import torch


def to_np(t):
    """torch tensor (bf16/fp32/int) -> numpy (fp32 / int), exact."""
    if isinstance(t, torch.Tensor):
        t = t.detach().cpu()
        if t.dtype == torch.bfloat16:
            t = t.to(torch.float32)
        return t.numpy()
    return np.asarray(t)


def weights_to_np(W):
    out = {k: to_np(v) for k, v in W.items() if k != "layers"}
    out["layers"] = [{k: to_np(v) for k, v in lw.items()} for lw in W["layers"]]
    return out


def rel_err(a, b):
    """max|a-b| / max|b| (the per-tensor norm the tolerances are stated in)."""
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    return float(np.max(np.abs(a - b)) / max(np.max(np.abs(b)), 1e-300))
