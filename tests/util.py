"""Helpers shared by the tests: weight conversion and side-by-side drivers of the oracle and the CUDA path."""
import numpy as np
import torch


def oracle_weights(w):
    """fp32 tensors -> numpy, bf16 tensors stay CPU torch tensors (both expose raw pointers)."""
    def conv(t):
        t = t.detach().cpu().contiguous()
        return t.numpy() if t.dtype == torch.float32 else t
    return {k: [conv(t) for t in v] if isinstance(v, list) else conv(v) for k, v in w.items()}


def rel_margin_ok(mg, eps):
    """May a decision differ between two sets of logits that are within eps of each other (max abs)?  Only if its
    deciding comparison was close enough for eps to move it.  Logits within eps give probabilities within a factor
    e^(2 eps) (numerator and normaliser each move by at most e^eps), so
      * an accept test u q(d) < p(d) can flip only if its two sides are within e^(2 eps) - 1 of each other, relatively;
      * a boundary of the sampling CDF moves by at most e^(2 eps) - 1 of the row's mass, i.e. by that over the
        fraction of the mass the token is drawn from (the rejected mass after a rejection), doubled because weights
        and their total both move;
      * a greedy argmax can flip only if the top two logits are within 2 eps.
    Pass the deviation that was actually measured on the request's rows, not a blanket tolerance: with the blanket
    value almost any sampled token over a large vocabulary would count as explained."""
    lim = float(np.expm1(2 * eps))
    return (mg.accept_rel <= lim or mg.sample_rel <= 2 * lim / max(mg.draw_mass, 1e-300) or mg.greedy_gap <= 2 * eps)
