"""Helpers shared by the tests: weight conversion and side-by-side drivers of the oracle and the CUDA path."""
import numpy as np
import torch


def oracle_weights(w):
    """fp32 tensors -> numpy, bf16 tensors stay CPU torch tensors (both expose raw pointers)."""
    def conv(t):
        t = t.detach().cpu().contiguous()
        return t.numpy() if t.dtype == torch.float32 else t
    return {k: [conv(t) for t in v] if isinstance(v, list) else conv(v) for k, v in w.items()}


def rel_margin_ok(mg, tol_logit):
    """A decision may legitimately differ between two sets of logits that agree within tol_logit when
    its deciding comparison was that close (a logit change d scales a probability by about e^d)."""
    lim = np.expm1(2 * tol_logit) * 2
    return min(mg.accept_rel, mg.sample_rel) <= lim or mg.greedy_gap <= 2 * tol_logit
