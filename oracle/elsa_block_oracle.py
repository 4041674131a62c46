"""Oracle of the chained transformer block around the four N:M linears (test infrastructure; shares no code
with the library).  Only tests/, __graft_entry__.smoke() and bench.py's cpu_baseline leg may import it.

What it follows: the ViT encoder block the paper prunes (ELSA, arXiv 2409.09708, Sec. 3: the linear modules
qkv, proj, fc1, fc2 of every block take one N:M level each; Sec. 4.2 quotes end-to-end speed-ups of whole
models).  The block is the standard pre-norm one of DeiT:
    x1 = LayerNorm1(x);  qkv = Linear_qkv(x1);  a = attention(qkv)
    x2 = x + Linear_proj(a);  x3 = LayerNorm2(x2);  h = GELU(Linear_fc1(x3));  y = x2 + Linear_fc2(h)
with LayerNorm over the feature dimension (biased variance, eps inside the square root, elementwise gain and
bias) and GELU(v) = v * Phi(v) = 0.5 * v * (1 + erf(v / sqrt 2)), the exact form (not the tanh approximation).
`attention` comes in two forms.  "copy_v": the stated stand-in a = V, the last third of qkv copied through, with
which the linear and elementwise path can be checked and timed alone.  "softmax": the multi-head self-attention
of the ViT / DeiT backbones the paper prunes (the paper leaves the attention products unpruned and gives no
formula of its own: this is the standard one): per image and head, with q, k, v the head's slices of the three
thirds of qkv and d the head dimension, a = softmax(q k^T / sqrt d) v, the softmax over the keys of the same image;
heads are laid side by side in a's columns.  All tokens of an image attend to each other (no mask, no dropout).
"window": the shifted-window attention of the Swin backbones the paper also prunes (Table 1, Swin-S / Swin-B; again
the paper gives no formula, this is the backbone's): the H x W token grid of an image is rolled by -shift along both
axes, cut into windows of ws x ws tokens, every window attends within itself as above with a per-head additive
bias [ws^2, ws^2] on the scores (the relative-position bias, given as a dense table) and, when shift > 0, with
-100 added where two tokens of a window come from different sides of the roll's seam (the three bands
[0, H - ws), [H - ws, H - shift), [H - shift, H) of each axis number the regions); the result is put back and rolled
by +shift.

Every tensor that crosses a stage boundary is a 16-bit tensor (the library writes it to memory in the block's
dtype), so every stage here computes in fp64 from its 16-bit inputs and rounds its result once, to nearest
even, to the 16-bit type; the linears are oracle/elsa_oracle.c's (mask, pack, unpack, fp64 product).
"""
import math

import numpy as np
import torch

from oracle import elsa_oracle as eo


def _round16(a64, torch_dtype):
    """fp64 array -> 16-bit type (one rounding to nearest even) -> fp64."""
    return torch.from_numpy(np.ascontiguousarray(a64)).to(torch_dtype).to(torch.float64).numpy()


def _bits(a64, torch_dtype):
    return torch.from_numpy(np.ascontiguousarray(a64)).to(torch_dtype).contiguous().view(torch.int16).numpy().view(np.uint16)


def layer_norm(x, gain, bias, eps):
    """fp64: rows normalised to zero mean and unit (biased) variance, then gain and bias per feature."""
    mean = x.mean(axis=1, keepdims=True)
    var = ((x - mean) ** 2).mean(axis=1, keepdims=True)
    return (x - mean) / np.sqrt(var + eps) * gain[None, :] + bias[None, :]


_erf = np.vectorize(math.erf, otypes=[np.float64])


def gelu(v):
    return 0.5 * v * (1.0 + _erf(v / math.sqrt(2.0)))


def sparse_linear(x16, W_bits, bias_bits, N, M, code):
    """fp64 product of 16-bit activations (fp64 array of 16-bit values) with the N:M projection of W."""
    vals, idx, _ = eo.nm_compress(W_bits, N, M)
    torch_dtype = torch.float16 if code == eo.F16 else torch.bfloat16
    return eo.nm_linear_f64(_bits(x16, torch_dtype), vals, idx, bias_bits, W_bits.shape[0], W_bits.shape[1], N, M, code)


def attention(qkv, tokens, heads):
    """fp64 multi-head self-attention.  qkv: [images * tokens, 3 * dim] (q | k | v thirds, heads side by side in
    each); returns [images * tokens, dim].  Plain loops over images and heads; softmax written out."""
    rows, three_dim = qkv.shape
    dim = three_dim // 3
    d = dim // heads
    out = np.zeros((rows, dim))
    for b in range(rows // tokens):
        r = slice(b * tokens, (b + 1) * tokens)
        for h in range(heads):
            q = qkv[r, h * d:(h + 1) * d]
            k = qkv[r, dim + h * d:dim + (h + 1) * d]
            v = qkv[r, 2 * dim + h * d:2 * dim + (h + 1) * d]
            s = q @ k.T / math.sqrt(d)
            e = np.exp(s - s.max(axis=1, keepdims=True))
            out[r, h * d:(h + 1) * d] = (e / e.sum(axis=1, keepdims=True)) @ v
    return out


def window_order(H, W, ws, shift):
    """Row index, inside one image's H * W tokens, of every window token: [windows, ws * ws] in the order
    (window row, window column; token row, token column) of the grid rolled by -shift."""
    i, j = np.meshgrid(np.arange(H), np.arange(W), indexing="ij")
    src = ((i + shift) % H) * W + (j + shift) % W          # rolled[i, j] = x[(i + shift) % H, (j + shift) % W]
    return src.reshape(H // ws, ws, W // ws, ws).transpose(0, 2, 1, 3).reshape(-1, ws * ws)


def shift_mask(H, W, ws, shift):
    """[windows, ws * ws, ws * ws]: 0 where two tokens of a window may attend to each other, -100 where the roll
    brought them together from different regions."""
    region = np.zeros((H, W))
    bands = lambda n: (slice(0, n - ws), slice(n - ws, n - shift), slice(n - shift, n))
    k = 0
    for hs in bands(H):
        for wsl in bands(W):
            region[hs, wsl] = k
            k += 1
    r = region.reshape(H // ws, ws, W // ws, ws).transpose(0, 2, 1, 3).reshape(-1, ws * ws)
    return np.where(r[:, :, None] != r[:, None, :], -100.0, 0.0)


def window_attention(qkv, H, W, ws, shift, heads, rel_bias):
    """fp64 shifted-window attention.  qkv: [images * H * W, 3 * dim] in the images' own token order; rel_bias:
    [heads, ws * ws, ws * ws]; returns [images * H * W, dim] in the same token order."""
    rows, three_dim = qkv.shape
    dim = three_dim // 3
    d = dim // heads
    order = window_order(H, W, ws, shift)
    mask = shift_mask(H, W, ws, shift) if shift > 0 else np.zeros((order.shape[0], ws * ws, ws * ws))
    out = np.zeros((rows, dim))
    for b in range(rows // (H * W)):
        for w in range(order.shape[0]):
            r = b * H * W + order[w]
            for h in range(heads):
                q = qkv[r, h * d:(h + 1) * d]
                k = qkv[r, dim + h * d:dim + (h + 1) * d]
                v = qkv[r, 2 * dim + h * d:2 * dim + (h + 1) * d]
                s = q @ k.T / math.sqrt(d) + rel_bias[h] + mask[w]
                e = np.exp(s - s.max(axis=1, keepdims=True))
                out[r, h * d:(h + 1) * d] = (e / e.sum(axis=1, keepdims=True)) @ v
    return out


def block_forward(x_bits, p, code, eps=1e-6, attn="copy_v", tokens=None, heads=None, window=None):
    """x_bits: uint16 [rows, dim].  p: dict with ln1_g, ln1_b, ln2_g, ln2_b (uint16 [dim]) and, for each of qkv,
    proj, fc1, fc2: W_<name> (uint16 [out, in]), b_<name> (uint16 [out]), level_<name> = (N, M).
    attn: "copy_v", "softmax" (then tokens per image and heads are required; rows = images * tokens) or "window"
    (then heads and window = dict(H, W, ws, shift, rel_bias [heads, ws^2, ws^2] fp64); rows = images * H * W).
    Returns a dict of every stage's 16-bit result as fp64 arrays: x1, qkv, a, x2, x3, h, y."""
    torch_dtype = torch.float16 if code == eo.F16 else torch.bfloat16

    def f64(bits):
        return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch_dtype).to(torch.float64).numpy()

    x = f64(x_bits)
    dim = x.shape[1]
    out = {}
    out["x1"] = _round16(layer_norm(x, f64(p["ln1_g"]), f64(p["ln1_b"]), eps), torch_dtype)
    out["qkv"] = _round16(sparse_linear(out["x1"], p["W_qkv"], p["b_qkv"], *p["level_qkv"], code), torch_dtype)
    if attn == "copy_v":
        out["a"] = out["qkv"][:, 2 * dim:3 * dim].copy()             # the stated stand-in for attention: a = V
    elif attn == "window":
        out["a"] = _round16(window_attention(out["qkv"], window["H"], window["W"], window["ws"], window["shift"], heads,
                                             window["rel_bias"]), torch_dtype)
    else:
        out["a"] = _round16(attention(out["qkv"], tokens, heads), torch_dtype)
    out["x2"] = _round16(x + sparse_linear(out["a"], p["W_proj"], p["b_proj"], *p["level_proj"], code), torch_dtype)
    out["x3"] = _round16(layer_norm(out["x2"], f64(p["ln2_g"]), f64(p["ln2_b"]), eps), torch_dtype)
    out["h"] = _round16(gelu(sparse_linear(out["x3"], p["W_fc1"], p["b_fc1"], *p["level_fc1"], code)), torch_dtype)
    out["y"] = _round16(out["x2"] + sparse_linear(out["h"], p["W_fc2"], p["b_fc2"], *p["level_fc2"], code), torch_dtype)
    return out
