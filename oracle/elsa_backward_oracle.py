"""Oracle of the backward pass of the masked linear (test infrastructure; shares no code with the library).
Only tests/, __graft_entry__.smoke() and bench.py's cpu_baseline leg may import it.

What it follows (ELSA, arXiv 2409.09708, Alg. 2, supernet training): each step derives the sparse weights
W(alpha) from the shared weights by the N:M projection of Sec. 3.1, computes the gradient of the loss with respect
to those sparse weights, and applies it to the shared weights.  For one linear module
    Y = X Wm^T + b,   Wm = mask .* W   (mask = the projection's keep-mask, a constant of the step)
the chain rule gives, with dY the gradient arriving at Y,
    dX = dY Wm              [rows, in]
    dW = mask .* (dY^T X)   [out, in]     (a pruned weight takes no part in the product: its derivative is zero)
    db = sum over rows of dY [out]

Reading: the paper writes g_t = grad L(X, W(alpha), W) and does not spell out the derivative at pruned
positions.  Differentiating with respect to W(alpha) = mask .* W gives zero there, which is what is written
here; a straight-through estimator (the dense dY^T X at pruned positions too) is the method of other work the
paper cites, not something Alg. 2 states.

Plain numpy in fp64 from the 16-bit inputs: the mask is oracle/elsa_oracle.c's, the three contractions are numpy
matmul / sum (library routines serving as steps); the caller rounds each result once to the 16-bit type.
"""
import numpy as np
import torch

from oracle import elsa_oracle as eo


def _f64(bits, code):
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16))
    return t.view(torch.float16 if code == eo.F16 else torch.bfloat16).to(torch.float64).numpy()


def linear_backward_f64(dY_bits, X_bits, W_bits, N, M, code):
    """dY [rows, out], X [rows, in], W [out, in] as uint16 bit patterns.  Returns fp64 (dX, dW, db)."""
    mask = eo.nm_mask(W_bits, N, M).astype(np.float64)
    dY, X, W = _f64(dY_bits, code), _f64(X_bits, code), _f64(W_bits, code)
    Wm = mask * W
    dX = dY @ Wm
    dW = mask * (dY.T @ X)
    db = dY.sum(axis=0)
    return dX, dW, db
