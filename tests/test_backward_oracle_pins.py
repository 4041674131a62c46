"""Pins of the backward oracle (no GPU): autograd in fp64 on a masked dense weight, exact finite differences of
the forward oracle on integer-valued inputs, a hand-worked case, and planted mistakes."""
import numpy as np
import torch

from oracle import elsa_backward_oracle as bwo
from oracle import elsa_oracle as eo
from paper_2409_09708_b200 import synth


def _case(rows, in_, out, seed, dtype=torch.bfloat16):
    X = synth.randn((rows, in_), seed, 1.0, dtype)
    W = synth.randn((out, in_), seed + 1, 0.1, dtype)
    dY = synth.randn((rows, out), seed + 2, 0.5, dtype)
    return X, W, dY


def test_against_autograd_in_fp64():
    for (N, M), dtype in [((2, 8), torch.bfloat16), ((1, 4), torch.float16), ((8, 8), torch.bfloat16), ((3, 16), torch.float16)]:
        code = eo.F16 if dtype == torch.float16 else eo.BF16
        X, W, dY = _case(11, 32, 6, 3, dtype)
        mask = torch.from_numpy(eo.nm_mask(synth.bits(W), N, M).astype(np.float64))
        x = X.double().requires_grad_()
        w = W.double().requires_grad_()
        b = torch.zeros(6, dtype=torch.float64, requires_grad=True)
        y = torch.nn.functional.linear(x, w * mask, b)
        (y * dY.double()).sum().backward()
        dX, dW, db = bwo.linear_backward_f64(synth.bits(dY), synth.bits(X), synth.bits(W), N, M, code)
        assert np.allclose(dX, x.grad.numpy(), rtol=1e-13, atol=1e-13)
        assert np.allclose(dW, w.grad.numpy(), rtol=1e-13, atol=1e-13)
        assert np.allclose(db, b.grad.numpy(), rtol=1e-13, atol=1e-13)
        assert (dW[mask.numpy() == 0] == 0).all()                  # pruned weights receive exactly zero


def test_exact_finite_differences_of_the_forward_oracle():
    # integer-valued tensors: the forward product is exact, the loss sum(G .* Y) is linear in X and in each kept
    # weight, so a unit step gives the derivative exactly
    rng = np.random.default_rng(0)
    rows, in_, out, N, M = 5, 16, 4, 2, 8
    dtype, code = torch.bfloat16, eo.BF16
    X = torch.from_numpy(rng.integers(-4, 5, (rows, in_)).astype(np.float32)).to(dtype)
    # distinct magnitudes inside every group, so that a unit step away from zero never changes the mask
    Wn = np.stack([np.concatenate([rng.permutation(np.arange(2, 2 + 2 * M, 2)) for _ in range(in_ // M)]) for _ in range(out)])
    Wn = Wn * rng.choice([-1, 1], Wn.shape)
    W = torch.from_numpy(Wn.astype(np.float32)).to(dtype)
    G = torch.from_numpy(rng.integers(-3, 4, (rows, out)).astype(np.float32)).to(dtype)
    mask = eo.nm_mask(synth.bits(W), N, M)

    def loss(Xt, Wt):
        vals, idx, _ = eo.nm_compress(synth.bits(Wt), N, M)
        Y = eo.nm_linear_f64(synth.bits(Xt), vals, idx, None, out, in_, N, M, code)
        return float((Y * G.double().numpy()).sum())

    dX, dW, db = bwo.linear_backward_f64(synth.bits(G), synth.bits(X), synth.bits(W), N, M, code)
    base = loss(X, W)
    for r, k in [(0, 0), (2, 7), (4, 15), (3, 9)]:
        Xp = X.clone()
        Xp[r, k] += 1
        assert loss(Xp, W) - base == dX[r, k]
    kept = np.argwhere(mask == 1)
    for o, k in kept[::3]:
        Wp = W.clone()
        Wp[o, k] += 1.0 if W[o, k] > 0 else -1.0                    # away from zero: still kept
        step = loss(X, Wp) - base
        assert step == (dW[o, k] if W[o, k] > 0 else -dW[o, k])
    pruned = np.argwhere(mask == 0)
    for o, k in pruned[::5]:
        Wp = W.clone()
        Wp[o, k] -= 1.0 if W[o, k] > 0 else -1.0                    # towards zero: still pruned
        assert loss(X, Wp) == base and dW[o, k] == 0
    assert np.array_equal(db, G.double().numpy().sum(axis=0))


def test_hand_worked_case():
    # one group of four, 2:4: W = [3, -1, 0.5, -4] keeps positions 0 and 3
    dtype, code = torch.bfloat16, eo.BF16
    W = torch.tensor([[3.0, -1.0, 0.5, -4.0]]).to(dtype)
    X = torch.tensor([[1.0, 2.0, 3.0, 4.0], [0.5, -1.0, 2.0, 0.0]]).to(dtype)
    dY = torch.tensor([[2.0], [-1.0]]).to(dtype)
    dX, dW, db = bwo.linear_backward_f64(synth.bits(dY), synth.bits(X), synth.bits(W), 2, 4, code)
    assert np.array_equal(dX, [[6.0, 0.0, 0.0, -8.0], [-3.0, 0.0, 0.0, 4.0]])      # dY * [3, 0, 0, -4]
    assert np.array_equal(dW, [[2 * 1 - 0.5, 0.0, 0.0, 2 * 4 - 0.0]])              # dY^T X at the kept positions
    assert np.array_equal(db, [1.0])


def test_planted_mistakes_are_caught():
    X, W, dY = _case(6, 8, 8, 9)                                     # square weight: a transposed operand still has a shape
    N, M = 2, 8
    mask = eo.nm_mask(synth.bits(W), N, M).astype(np.float64)
    dX, dW, db = bwo.linear_backward_f64(synth.bits(dY), synth.bits(X), synth.bits(W), N, M, eo.BF16)
    Wm = mask * W.double().numpy()
    assert not np.allclose(dX, dY.double().numpy() @ Wm.T)           # transposed weight
    assert not np.allclose(dX, dY.double().numpy() @ W.double().numpy())   # unmasked weight
    assert not np.allclose(dW, dY.double().numpy().T @ X.double().numpy())  # straight-through (dense) gradient
    assert not np.allclose(dW, mask * (X.double().numpy().T @ dY.double().numpy()))   # dW transposed
