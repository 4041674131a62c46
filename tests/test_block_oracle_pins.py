"""Pins of the chained-block oracle (no GPU): LayerNorm and GELU against closed forms and hand-worked values, the
whole chain against the library routines of torch in fp64 on a masked dense weight."""
import math

import numpy as np
import torch

from oracle import elsa_block_oracle as bo
from oracle import elsa_oracle as eo
from paper_2409_09708_b200 import synth


def test_layer_norm_closed_forms():
    x = np.array([[1.0, 2.0, 3.0, 6.0], [5.0, 5.0, 5.0, 5.0]])
    g = np.array([1.0, 1.0, 2.0, 1.0])
    b = np.array([0.0, 0.5, 0.0, 0.0])
    y = bo.layer_norm(x, g, b, 0.0 + 1e-12)
    # row 0: mean 3, biased variance (4 + 1 + 0 + 9) / 4 = 3.5
    s = math.sqrt(3.5)
    assert np.allclose(y[0], [-2 / s, -1 / s + 0.5, 0.0, 3 / s], atol=1e-9)
    # a constant row has zero variance: the normalised row is 0 (eps keeps the division finite), leaving the bias
    assert np.allclose(y[1], b, atol=1e-6)
    z = bo.layer_norm(np.random.default_rng(0).standard_normal((5, 64)), np.ones(64), np.zeros(64), 0.0)
    assert np.allclose(z.mean(axis=1), 0, atol=1e-12) and np.allclose(z.var(axis=1), 1, atol=1e-12)


def test_gelu_is_the_exact_form():
    assert bo.gelu(np.array([0.0]))[0] == 0.0
    # Phi(1) = 0.8413447460685429, Phi(-1) = 1 - Phi(1): standard normal table values
    assert abs(bo.gelu(np.array([1.0]))[0] - 0.8413447460685429) < 1e-15
    assert abs(bo.gelu(np.array([-1.0]))[0] + 0.15865525393145707) < 1e-15
    v = np.linspace(-6, 6, 101)
    assert np.allclose(bo.gelu(v) - bo.gelu(-v), v, atol=1e-12)              # v Phi(v) + v Phi(-v) = v
    tanh_form = 0.5 * v * (1 + np.tanh(math.sqrt(2 / math.pi) * (v + 0.044715 * v ** 3)))
    assert np.abs(bo.gelu(v) - tanh_form).max() > 1e-4                        # not the approximation
    assert np.allclose(bo.gelu(v), torch.nn.functional.gelu(torch.from_numpy(v)).numpy(), atol=1e-15)


def test_block_chain_against_torch_fp64_routines():
    dtype = torch.bfloat16
    rows, dim, mlp = 24, 64, 256
    x = synth.randn((rows, dim), 1, 1.0, dtype)
    p, tp = {}, {}
    shapes = {"qkv": (3 * dim, dim), "proj": (dim, dim), "fc1": (mlp, dim), "fc2": (dim, mlp)}
    levels = {"qkv": (4, 8), "proj": (2, 8), "fc1": (2, 4), "fc2": (1, 4)}
    for i, (name, (o, k)) in enumerate(shapes.items()):
        W = synth.randn((o, k), 10 + i, 0.08, dtype)
        b = synth.randn((o,), 20 + i, 0.02, dtype)
        p["W_" + name], p["b_" + name], p["level_" + name] = synth.bits(W), synth.bits(b), levels[name]
        mask = eo.nm_mask(synth.bits(W), *levels[name])
        tp[name] = (W.double() * torch.from_numpy(mask.astype(np.float64)), b.double())
    for i, name in enumerate(("ln1_g", "ln1_b", "ln2_g", "ln2_b")):
        t = synth.randn((dim,), 30 + i, 0.1, dtype) + (1.0 if name.endswith("g") else 0.0)
        p[name] = synth.bits(t.to(dtype))
        tp[name] = t.to(dtype).double()
    got = bo.block_forward(synth.bits(x), p, eo.BF16, eps=1e-6)

    F = torch.nn.functional
    r = lambda t: t.to(dtype).double()                                  # a stage boundary: one rounding to 16 bits
    xt = x.double()
    x1 = r(F.layer_norm(xt, (dim,), tp["ln1_g"], tp["ln1_b"], 1e-6))
    qkv = r(F.linear(x1, *tp["qkv"]))
    a = qkv[:, 2 * dim:]
    x2 = r(xt + F.linear(a, *tp["proj"]))
    x3 = r(F.layer_norm(x2, (dim,), tp["ln2_g"], tp["ln2_b"], 1e-6))
    h = r(F.gelu(F.linear(x3, *tp["fc1"])))
    y = r(x2 + F.linear(h, *tp["fc2"]))
    for name, ref in (("x1", x1), ("qkv", qkv), ("a", a), ("x2", x2), ("x3", x3), ("h", h), ("y", y)):
        ref = ref.numpy()
        # summation order differs between the two fp64 products: a value next to a rounding boundary may land on
        # the neighbouring 16-bit number, nothing more
        close = np.abs(got[name] - ref) <= 2.0 ** -7 * np.abs(ref) + 1e-30
        assert close.all(), name
        assert (got[name] == ref).mean() > 0.98, name
    # a mistake anywhere shows: dropping a residual, the wrong GELU, or the wrong third of qkv
    assert np.abs(got["x2"] - (got["x2"] - x.double().numpy())).max() > 0.1
    assert not np.array_equal(got["a"], got["qkv"][:, :dim])


def test_attention_against_torch_and_closed_forms():
    rng = np.random.default_rng(3)
    images, tokens, heads, d = 3, 7, 2, 4
    dim = heads * d
    qkv = rng.standard_normal((images * tokens, 3 * dim))
    got = bo.attention(qkv, tokens, heads)
    # torch's fused routine in fp64 on [images, heads, tokens, d] views
    t = torch.from_numpy(qkv).view(images, tokens, 3, heads, d).permute(2, 0, 3, 1, 4)
    ref = torch.nn.functional.scaled_dot_product_attention(t[0], t[1], t[2]).permute(0, 2, 1, 3).reshape(images * tokens, dim)
    assert np.allclose(got, ref.numpy(), rtol=1e-12, atol=1e-12)
    # hand-worked: one image, one head, two tokens, d = 1: scores q_i k_j, weights by softmax
    q, k, v = np.array([1.0, 0.0]), np.array([2.0, -1.0]), np.array([10.0, 20.0])
    w0 = math.exp(2.0) / (math.exp(2.0) + math.exp(-1.0))
    hand = bo.attention(np.stack([q, k, v], axis=1), 2, 1)
    assert np.allclose(hand[:, 0], [w0 * 10 + (1 - w0) * 20, 15.0], atol=1e-12)     # q = 0 attends uniformly
    # zero queries: every token gets the mean of its own image's values, never another image's
    z = qkv.copy()
    z[:, :dim] = 0.0
    mean_v = z[:, 2 * dim:].reshape(images, tokens, dim).mean(axis=1)
    assert np.allclose(bo.attention(z, tokens, heads).reshape(images, tokens, dim), mean_v[:, None, :], atol=1e-12)
    # the keys' order inside an image does not matter; the 1 / sqrt d scale does
    perm = rng.permutation(tokens)
    shuffled = qkv.reshape(images, tokens, 3 * dim).copy()
    shuffled[:, :, dim:] = shuffled[:, perm, dim:]
    assert np.allclose(bo.attention(shuffled.reshape(-1, 3 * dim), tokens, heads), got, atol=1e-12)
    unscaled = qkv.copy()
    unscaled[:, :dim] *= math.sqrt(d)
    assert not np.allclose(bo.attention(unscaled, tokens, heads), got, atol=1e-3)
    # a shift common to all keys cancels in the softmax
    shifted = qkv.copy()
    shifted[:, dim:2 * dim] += 1.0
    assert np.allclose(bo.attention(shifted, tokens, heads), got, atol=1e-12)
    # heads are independent: changing head 1's keys leaves head 0's output alone
    other = qkv.copy()
    other[:, dim + d:2 * dim] *= 2.0
    assert np.allclose(bo.attention(other, tokens, heads)[:, :d], got[:, :d], atol=1e-12)
    assert not np.allclose(bo.attention(other, tokens, heads)[:, d:], got[:, d:], atol=1e-3)


def test_block_chain_with_attention_against_torch():
    dtype = torch.bfloat16
    images, tokens, heads, dim, mlp = 2, 5, 2, 16, 32
    rows = images * tokens
    x = synth.randn((rows, dim), 41, 1.0, dtype)
    p = {}
    shapes = {"qkv": (3 * dim, dim), "proj": (dim, dim), "fc1": (mlp, dim), "fc2": (dim, mlp)}
    for i, (name, (o, k)) in enumerate(shapes.items()):
        p["W_" + name] = synth.bits(synth.randn((o, k), 50 + i, 0.2, dtype))
        p["b_" + name] = synth.bits(synth.randn((o,), 60 + i, 0.02, dtype))
        p["level_" + name] = (2, 4)
    for i, name in enumerate(("ln1_g", "ln1_b", "ln2_g", "ln2_b")):
        p[name] = synth.bits((synth.randn((dim,), 70 + i, 0.1, dtype) + (1.0 if name.endswith("g") else 0.0)).to(dtype))
    got = bo.block_forward(synth.bits(x), p, eo.BF16, attn="softmax", tokens=tokens, heads=heads)
    qkv = torch.from_numpy(got["qkv"]).view(images, tokens, 3, heads, dim // heads).permute(2, 0, 3, 1, 4)
    a = torch.nn.functional.scaled_dot_product_attention(qkv[0], qkv[1], qkv[2]).permute(0, 2, 1, 3).reshape(rows, dim)
    a16 = a.to(dtype).double().numpy()
    assert (np.abs(got["a"] - a16) <= 2.0 ** -7 * np.abs(a16) + 1e-30).all() and (got["a"] == a16).mean() > 0.95
    assert not np.allclose(got["a"], got["qkv"][:, 2 * dim:])            # not the stand-in


def _swin_reference(qkv, B, H, W, ws, shift, heads, rel_bias):
    """The backbone's formulation with torch's own roll / view / permute and its fused attention, in fp64."""
    dim = qkv.shape[1] // 3
    d = dim // heads
    t = torch.from_numpy(qkv).view(B, H, W, 3 * dim)
    if shift:
        t = torch.roll(t, shifts=(-shift, -shift), dims=(1, 2))
    t = t.view(B, H // ws, ws, W // ws, ws, 3 * dim).permute(0, 1, 3, 2, 4, 5).reshape(-1, ws * ws, 3, heads, d)
    q, k, v = (t[:, :, i].permute(0, 2, 1, 3) for i in range(3))                    # [windows, heads, tokens, d]
    bias = torch.from_numpy(rel_bias)[None]                                          # [1, heads, T, T]
    if shift:
        img = torch.zeros(1, H, W, 1, dtype=torch.float64)
        cnt = 0
        for hs in (slice(0, -ws), slice(-ws, -shift), slice(-shift, None)):
            for wsl in (slice(0, -ws), slice(-ws, -shift), slice(-shift, None)):
                img[:, hs, wsl, :] = cnt
                cnt += 1
        mw = img.view(1, H // ws, ws, W // ws, ws, 1).permute(0, 1, 3, 2, 4, 5).reshape(-1, ws * ws)
        m = (mw[:, None, :] - mw[:, :, None] != 0).double() * -100.0                 # [nW, T, T]
        bias = bias + m.repeat(B, 1, 1)[:, None]
    o = torch.nn.functional.scaled_dot_product_attention(q, k, v, attn_mask=bias)
    o = o.permute(0, 2, 1, 3).reshape(B, H // ws, W // ws, ws, ws, dim).permute(0, 1, 3, 2, 4, 5).reshape(B, H, W, dim)
    if shift:
        o = torch.roll(o, shifts=(shift, shift), dims=(1, 2))
    return o.reshape(B * H * W, dim).numpy()


def test_window_attention_against_the_backbones_formulation():
    rng = np.random.default_rng(5)
    for (B, H, W, ws, shift, heads, d) in [(2, 6, 6, 3, 0, 2, 4), (2, 6, 6, 3, 1, 2, 4), (1, 8, 4, 4, 2, 1, 8), (3, 14, 14, 7, 3, 2, 4)]:
        dim = heads * d
        qkv = rng.standard_normal((B * H * W, 3 * dim))
        rel_bias = rng.standard_normal((heads, ws * ws, ws * ws))
        got = bo.window_attention(qkv, H, W, ws, shift, heads, rel_bias)
        assert np.allclose(got, _swin_reference(qkv, B, H, W, ws, shift, heads, rel_bias), rtol=1e-10, atol=1e-10)
    # one window covering the whole image, no shift, no bias: plain attention over the image
    qkv = rng.standard_normal((2 * 16, 3 * 8))
    assert np.allclose(bo.window_attention(qkv, 4, 4, 4, 0, 2, np.zeros((2, 16, 16))), bo.attention(qkv, 16, 2), atol=1e-12)
    # the order of windows: every token exactly once, windows are ws x ws patches of the rolled grid
    order = bo.window_order(6, 9, 3, 1)
    assert sorted(order.ravel().tolist()) == list(range(54))
    assert order[0].tolist() == [10, 11, 12, 19, 20, 21, 28, 29, 30]               # rows 1..3, columns 1..3
    assert order[-1].tolist() == [43, 44, 36, 52, 53, 45, 7, 8, 0]                 # the wrapped corner
    # the mask: nothing is masked inside the windows away from the seam; the last window mixes four regions
    m = bo.shift_mask(6, 9, 3, 1)
    assert (m[0] == 0).all() and (m[-1] != 0).any()
    r_last = np.array([0, 0, 1, 0, 0, 1, 2, 2, 3])                                # regions of the last window's tokens
    assert np.array_equal(m[-1] != 0, r_last[:, None] != r_last[None, :])
    # tokens from different regions of a window do not influence each other
    B, H, W, ws, shift, heads, d = 1, 6, 6, 3, 1, 1, 4
    qkv = rng.standard_normal((36, 12))
    bias = np.zeros((1, 9, 9))
    base = bo.window_attention(qkv, H, W, ws, shift, heads, bias)
    changed = qkv.copy()
    changed[0, 4:] += 5.0                        # token (0, 0) ends up alone in its region of the last window
    after = bo.window_attention(changed, H, W, ws, shift, heads, bias)
    others = np.ones(36, bool)
    others[0] = False
    assert np.allclose(after[others], base[others], atol=1e-12) and not np.allclose(after[0], base[0], atol=1e-3)
