"""Oracle of the INT8 form of the N:M path (test infrastructure; shares no code with the library).

Only tests/, __graft_entry__.smoke() and bench.py's cpu_baseline leg may import it.

What it follows (ELSA, arXiv 2409.09708): the same projection and packed form as the 16-bit oracle
(Sec. 3.1 / Eq. 1 with saliency |w|; Sec. 1 and Sec. 2: N of every M kept, one log2(M)-bit index each), applied
to signed 8-bit weights, and the product of Sec. 2 on integers; Table 6 is the paper's use of 8-bit
quantisation on top of the searched N:M models (the quantiser, PTQ4ViT, supplies integers and scales and is
not restated here).

Readings (the paper is silent on all of them): |w| is the integer magnitude, so -128 (magnitude 128) outranks
127; ties go to the lowest position; the index stream is the 16-bit form's (field t of group g of a row at bit
(g * N + t) * log2 M, LSB first in little-endian 32-bit words, rows word-aligned, pad bits zero).  The product
is exact in integers; the result leaves the integer domain as
    y = fl32(fl32(fl32(acc) * fl32(x_scale * w_scale[o])) + bias[o])
(fl32 = round to nearest even in binary32: the precision the kernel computes its epilogue in), and the caller
rounds y once to the 16-bit output type.

Plain numpy: N rounds of "first arg-max among the not yet taken" per group; bits placed one at a time; the
integer product as a float64 matmul (exact: every partial sum is an integer far below 2^53).
"""
import numpy as np

_BITS = {4: 2, 8: 3, 16: 4}


def nm_mask(W, N, M):
    """W: int8 [out, in].  1 where kept."""
    out, in_ = W.shape
    mag = np.abs(W.astype(np.int16)).reshape(out, in_ // M, M)
    taken = np.zeros_like(mag, dtype=bool)
    for _ in range(N):
        cand = np.where(taken, -1, mag)
        first = np.argmax(cand, axis=2)                  # the first position of the largest magnitude
        np.put_along_axis(taken, first[..., None], True, axis=2)
    return taken.reshape(out, in_).astype(np.uint8)


def index_words_per_row(in_, N, M):
    return 0 if N == M else -(-(in_ // M * N * _BITS[M]) // 32)


def nm_pack(W, mask, N, M):
    """Kept bytes in ascending position and the index words.  Pure-Python loops: small cases only."""
    out, in_ = W.shape
    b = _BITS[M]
    vals = np.zeros((out, in_ // M * N), dtype=np.int8)
    words = index_words_per_row(in_, N, M)
    idx = np.zeros((out, words), dtype=np.uint32)
    for o in range(out):
        for g in range(in_ // M):
            t = 0
            for i in range(M):
                if mask[o, g * M + i]:
                    vals[o, g * N + t] = W[o, g * M + i]
                    if words:
                        for bit in range(b):
                            if (i >> bit) & 1:
                                pos = (g * N + t) * b + bit
                                idx[o, pos >> 5] |= np.uint32(1 << (pos & 31))
                    t += 1
            assert t == N
    return vals, idx


def nm_unpack(vals, idx, out, in_, N, M):
    b = _BITS[M]
    W = np.zeros((out, in_), dtype=np.int8)
    for o in range(out):
        for g in range(in_ // M):
            for t in range(N):
                if N == M:
                    i = t
                else:
                    i = 0
                    for bit in range(b):
                        pos = (g * N + t) * b + bit
                        i |= ((int(idx[o, pos >> 5]) >> (pos & 31)) & 1) << bit
                W[o, g * M + i] = vals[o, g * N + t]
    return W


def linear_f32(X, x_scale, Wm, w_scale, bias_f32):
    """X int8 [rows, in], Wm int8 [out, in] (masked weight), w_scale float32 [out], bias_f32 float32 [out] or None.
    Returns y as float32, before the final rounding to 16 bits."""
    acc = X.astype(np.float64) @ Wm.astype(np.float64).T             # exact integers
    assert np.abs(acc).max() < 2 ** 31
    s = np.float32(x_scale) * w_scale.astype(np.float32)              # one fp32 product per feature
    y = acc.astype(np.float32) * s[None, :]                           # int -> fp32 (RNE), fp32 product
    if bias_f32 is not None:
        y = y + bias_f32.astype(np.float32)[None, :]                  # fp32 sum
    return y.astype(np.float32)
