"""INT8 form of the N:M path: pins of its oracle (no GPU) and parity of the library against it (GPU)."""
import numpy as np
import pytest
import torch

from oracle import elsa_int8_oracle as io


# ------------------------------------------------------------------ pins of the oracle (no GPU)

def _stable_sort_mask(W, N, M):
    """Independent restatement: the N kept positions are the first N of a stable sort by descending magnitude."""
    out, in_ = W.shape
    mask = np.zeros((out, in_), dtype=np.uint8)
    mag = np.abs(W.astype(np.int16))
    for o in range(out):
        for g in range(in_ // M):
            order = np.argsort(-mag[o, g * M:(g + 1) * M], kind="stable")
            mask[o, g * M + order[:N]] = 1
    return mask


def test_oracle_mask_keeps_the_n_largest_magnitudes_lowest_position_first():
    rng = np.random.default_rng(1)
    W = rng.integers(-128, 128, (12, 64)).astype(np.int8)
    W[0, :8] = [-128, 127, 127, -128, 0, 0, 5, -5]          # |-128| outranks 127; equal magnitudes of both signs
    W[1, :16] = 3                                            # an all-equal stretch keeps positions 0..N-1
    for N, M in [(1, 4), (2, 4), (3, 4), (1, 8), (2, 8), (4, 8), (7, 8), (2, 16), (8, 16), (4, 4)]:
        mask = io.nm_mask(W, N, M)
        assert (mask.reshape(12, -1, M).sum(axis=2) == N).all()
        assert (mask == _stable_sort_mask(W, N, M)).all(), (N, M)
    assert list(io.nm_mask(W, 2, 8)[0, :8]) == [1, 0, 0, 1, 0, 0, 0, 0]
    assert list(io.nm_mask(W, 3, 8)[0, :8]) == [1, 1, 0, 1, 0, 0, 0, 0]
    assert list(io.nm_mask(W, 2, 8)[1, :8]) == [1, 1, 0, 0, 0, 0, 0, 0]
    # nesting across N (Sec. 3.1, subset-superset relation)
    for M in (4, 8, 16):
        prev = np.zeros_like(W, dtype=np.uint8)
        for N in range(1, M + 1):
            cur = io.nm_mask(W, N, M)
            assert ((prev & cur) == prev).all()
            prev = cur


def test_oracle_pack_is_the_hand_worked_stream_and_unpack_inverts_it():
    # one row, 3:8: groups (9, -7, 0, 1, -128, 2, 3, -4) and (1, 1, 1, 1, 1, 1, 1, 2)
    W = np.array([[9, -7, 0, 1, -128, 2, 3, -4, 1, 1, 1, 1, 1, 1, 1, 2]], dtype=np.int8)
    mask = io.nm_mask(W, 3, 8)
    assert list(mask[0]) == [1, 1, 0, 0, 1, 0, 0, 0, 1, 1, 0, 0, 0, 0, 0, 1]
    vals, idx = io.nm_pack(W, mask, 3, 8)
    assert list(vals[0]) == [9, -7, -128, 1, 1, 2]
    # fields 0, 1, 4, 0, 1, 7 of three bits, LSB first: 0 | 1<<3 | 4<<6 | 0<<9 | 1<<12 | 7<<15
    assert idx.shape == (1, 1) and int(idx[0, 0]) == (1 << 3) | (4 << 6) | (1 << 12) | (7 << 15)
    assert (io.nm_unpack(vals, idx, 1, 16, 3, 8) == np.where(mask == 1, W, 0)).all()
    rng = np.random.default_rng(2)
    Wr = rng.integers(-128, 128, (5, 48)).astype(np.int8)
    for N, M in [(1, 4), (3, 4), (2, 8), (5, 8), (8, 8), (3, 16)]:
        m = io.nm_mask(Wr, N, M)
        v, ix = io.nm_pack(Wr, m, N, M)
        assert ix.shape[1] == io.index_words_per_row(48, N, M)
        assert (io.nm_unpack(v, ix, 5, 48, N, M) == np.where(m == 1, Wr, 0)).all()


def test_oracle_linear_is_the_integer_product_with_fp32_scaling():
    rng = np.random.default_rng(3)
    X = rng.integers(-128, 128, (7, 32)).astype(np.int8)
    W = rng.integers(-128, 128, (5, 32)).astype(np.int8)
    ws = rng.random(5).astype(np.float32) * 0.01
    bias = rng.standard_normal(5).astype(np.float32)
    y = io.linear_f32(X, 0.05, W, ws, bias)
    acc = X.astype(np.int64) @ W.astype(np.int64).T                   # integer matmul, no floating point at all
    for r in range(7):
        for o in range(5):
            s = np.float32(0.05) * ws[o]
            assert y[r, o] == np.float32(np.float32(np.float32(acc[r, o]) * s) + bias[o])
    # scale one and no bias: the integers themselves
    assert (io.linear_f32(X, 1.0, W, np.ones(5, np.float32), None) == acc.astype(np.float32)).all()


# ------------------------------------------------------------------ the library against the oracle (GPU)

@pytest.fixture(scope="module")
def lib():
    from paper_2409_09708_b200 import build
    build.build()
    from paper_2409_09708_b200 import binding
    return binding


def _idx_words(idx, rows, words):
    if idx is None:
        return np.zeros((rows, 0), dtype=np.uint32)
    return idx.cpu().numpy().view(np.uint32)[:, :words]


@pytest.mark.gpu
@pytest.mark.parametrize("shape", [(768, 768), (16, 64), (40, 1008), (8, 4096)])
def test_int8_compress_and_unpack_match_the_oracle_bit_for_bit(lib, shape):
    out, in_ = shape
    rng = np.random.default_rng(out + in_)
    W = rng.integers(-128, 128, (out, in_)).astype(np.int8)
    W[0, :8] = [-128, 127, 127, -128, 0, 0, 5, -5]
    W[1, :16] = 3
    Wd = torch.from_numpy(W).cuda()
    small = out * in_ <= 16 * 1024
    for N, M in [(1, 4), (2, 4), (3, 4), (4, 4), (1, 8), (2, 8), (4, 8), (7, 8), (8, 8), (1, 16), (2, 16), (8, 16)]:
        if in_ % M:
            continue
        vals, idx = lib.elsa_nm_compress_i8(Wd, N, M)
        Wm = lib.elsa_nm_unpack_i8(vals, idx, out, in_, N, M)
        torch.cuda.synchronize()
        mask = io.nm_mask(W, N, M)
        assert (Wm.cpu().numpy() == np.where(mask == 1, W, 0)).all(), (N, M)
        # kept bytes in ascending position: the masked weight with the pruned positions squeezed out
        keep_sorted = np.sort(np.where(mask.reshape(out, -1, M) == 1, np.arange(M), M), axis=2)[:, :, :N]
        expect_vals = np.take_along_axis(W.reshape(out, -1, M), keep_sorted, axis=2).reshape(out, -1)
        assert (vals.cpu().numpy() == expect_vals).all(), (N, M)
        if small:                                     # the index stream bit for bit (python loops in the oracle)
            ovals, oidx = io.nm_pack(W, mask, N, M)
            assert (vals.cpu().numpy() == ovals).all()
            assert (_idx_words(idx, out, oidx.shape[1]) == oidx).all(), (N, M)


INT8_LINEAR_CASES = [
    # rows, in, out, N, M: ragged rows and features, K not a multiple of the 128-element stage, dense level
    (197, 768, 768, 4, 8), (300, 208, 136, 2, 4), (1, 128, 8, 1, 4), (515, 512, 1000, 2, 16), (257, 1024, 264, 8, 8),
    (5000, 3072, 768, 2, 8), (4100, 768, 2304, 1, 8),
]


@pytest.mark.gpu
@pytest.mark.parametrize("out_dtype", [torch.float16, torch.bfloat16])
@pytest.mark.parametrize("case", INT8_LINEAR_CASES)
def test_int8_linear_matches_the_oracle_bit_for_bit(lib, case, out_dtype):
    rows, in_, out, N, M = case
    rng = np.random.default_rng(rows * 7 + in_ + out)
    X = rng.integers(-128, 128, (rows, in_)).astype(np.int8)
    W = rng.integers(-128, 128, (out, in_)).astype(np.int8)
    ws = (rng.random(out).astype(np.float32) + 0.5) * np.float32(2e-4)
    x_scale = 0.03
    bias = torch.from_numpy(rng.standard_normal(out).astype(np.float32) * 0.5).to(out_dtype)
    Wd = torch.from_numpy(W).cuda()
    vals, idx = lib.elsa_nm_compress_i8(Wd, N, M)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    Y = lib.elsa_nm_linear_i8(torch.from_numpy(X).cuda(), x_scale, vals, idx, torch.from_numpy(ws).cuda(), bias.cuda(), out,
                              in_, N, M, out_dtype, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    Wm = np.where(io.nm_mask(W, N, M) == 1, W, 0).astype(np.int8)
    pick = np.arange(rows) if rows <= 600 else np.unique(np.concatenate([[0, rows - 1], rng.integers(0, rows, 300)]))
    ref = io.linear_f32(X[pick], x_scale, Wm, ws, bias.to(torch.float32).numpy())
    expect = torch.from_numpy(ref).to(out_dtype)                     # the one rounding to 16 bits
    got = Y.cpu()[torch.from_numpy(pick)]
    assert torch.equal(got.view(torch.int16), expect.view(torch.int16)), (case, out_dtype)


@pytest.mark.gpu
def test_int8_linear_refuses_bad_arguments(lib):
    W = torch.zeros((64, 128), dtype=torch.int8, device="cuda")
    vals, idx = lib.elsa_nm_compress_i8(W, 2, 4)
    ws = torch.ones(64, device="cuda")
    X = torch.zeros((8, 128), dtype=torch.int8, device="cuda")
    with pytest.raises(lib.ElsaError):
        lib.elsa_nm_linear_i8(X, 1.0, vals, None, ws, None, 64, 128, 2, 4, torch.bfloat16)      # idx missing
    with pytest.raises(lib.ElsaError):
        lib.elsa_nm_compress_i8(torch.zeros((64, 24), dtype=torch.int8, device="cuda"), 2, 4)    # in % 16 != 0
    with pytest.raises(lib.ElsaError):
        lib.elsa_nm_compress_i8(W, 5, 4)                                                        # N > M
