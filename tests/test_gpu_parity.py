"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the same
seeded bytes.  Masks, packed values and index words must match bit for bit; linear outputs must
stay within relative Frobenius error 5e-3 and |err| <= 1e-2 * (|ref| + 1) of the fp64 oracle."""
import numpy as np
import pytest
import torch

from oracle import elsa_oracle as eo
from paper_2409_09708_b200 import synth

pytestmark = pytest.mark.gpu

REL_FRO_TOL = 5e-3
ELEM_TOL = 1e-2


@pytest.fixture(scope="module")
def lib():
    from paper_2409_09708_b200 import build
    build.build()
    from paper_2409_09708_b200 import binding
    return binding


def ocode(dtype):
    return eo.F16 if dtype == torch.float16 else eo.BF16


def idx_bits(idx, like=None):
    if idx is None:          # the dense level stores no indices
        return np.zeros(like.shape if like is not None else (0, 0), np.uint32)
    return idx.cpu().numpy().view(np.uint32)


def check_close(Y_gpu, ref):
    got = Y_gpu.detach().to(torch.float64).cpu().numpy()
    assert np.isfinite(got).all()
    err = got - ref
    rel = np.linalg.norm(err) / max(np.linalg.norm(ref), 1e-30)
    worst = np.max(np.abs(err) / (np.abs(ref) + 1.0))
    assert rel <= REL_FRO_TOL, "relative Frobenius error %g" % rel
    assert worst <= ELEM_TOL, "per-element error %g" % worst
    return rel, worst


def oracle_linear(X, W, bias, N, M, dtype):
    vals, idx, _ = eo.nm_compress(synth.bits(W), N, M)
    return eo.nm_linear_f64(synth.bits(X), vals, idx, None if bias is None else synth.bits(bias),
                            W.shape[0], W.shape[1], N, M, ocode(dtype))


# ------------------------------------------------------------------ compress / unpack

COMPRESS_SHAPES = [(768, 768), (16, 64), (40, 1008), (24, 16 * 23), (8, 4096)]
LEVELS = [(1, 4), (2, 4), (3, 4), (4, 4), (1, 8), (2, 8), (3, 8), (4, 8), (7, 8), (8, 8),
          (1, 16), (2, 16), (4, 16), (8, 16), (15, 16), (16, 16)]


@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
@pytest.mark.parametrize("shape", COMPRESS_SHAPES)
def test_compress_and_unpack_match_oracle_bit_for_bit(lib, shape, dtype):
    out, in_ = shape
    W = synth.randn((out, in_), 900 + out + in_, synth.W_STD, dtype)
    Wb = synth.bits(W).copy()
    Wb[0, :8] = [0x8000, 0, 0x8000, 0, 0, 0, 0, 0x8000]           # signed zeros
    Wb[1, :16] = Wb[1, 0]                                           # an all-equal stretch
    # patterns outside the contract of the linear, inside that of compress / unpack (compare domain: the 15
    # magnitude bits as an integer, so NaN > Inf > finite and a subnormal is just a small magnitude): infinities of
    # both signs, quiet and signalling NaNs with different payloads, the largest finite value, subnormals, and
    # ties among them
    inf = 0x7C00 if dtype == torch.float16 else 0x7F80
    sub = [0x0001, 0x8001, 0x03FF, 0x0200] if dtype == torch.float16 else [0x0001, 0x8001, 0x007F, 0x0040]
    special = [inf, inf | 0x8000, inf + 1, (inf + 1) | 0x8000, 0x7FFF, 0xFFFF, inf - 1, (inf - 1) | 0x8000] + sub + [inf, 0, inf | 0x8000, sub[0]]
    Wb[2, :16] = special
    Wb[3, :16] = special[::-1]
    rng = np.random.default_rng(out * 7 + in_)
    where = rng.choice(out * in_, size=max(8, out * in_ // 64), replace=False)      # and scattered through the matrix
    Wb.reshape(-1)[where] = rng.choice(np.asarray(special, dtype=Wb.dtype), size=where.size)
    Wd = synth.from_bits(Wb, dtype).cuda()                           # exact bit patterns, no conversion
    for N, M in LEVELS:
        if in_ % M:
            continue
        vals, idx = lib.elsa_nm_compress(Wd, N, M)
        torch.cuda.synchronize()
        ovals, oidx, omask = eo.nm_compress(Wb, N, M)
        assert (synth.bits(vals) == ovals).all(), (N, M)
        assert (idx_bits(idx, oidx) == oidx).all(), (N, M)
        Wm = lib.elsa_nm_unpack(vals, idx, out, in_, N, M)
        torch.cuda.synchronize()
        assert (synth.bits(Wm) == eo.nm_unpack(ovals, oidx, out, in_, N, M)).all(), (N, M)
        assert (synth.bits(Wm) == np.where(omask == 1, Wb, 0)).all()


def test_compress_weight_shapes_of_the_workloads(lib):
    """Every distinct weight shape and level of the DeiT-B and Swin-B tables, checked in full."""
    seen = set()
    for name in ("deit_b_block_b64", "deit_b_stack_b256", "swin_b_stack_b128"):
        layers, dt = synth.workload(name)
        dtype = synth.torch_dtype(dt)
        for l in layers:
            key = (l.out, l.in_, l.N, l.M, dt)
            if key in seen:
                continue
            seen.add(key)
            W = synth.randn((l.out, l.in_), l.seed_w, synth.W_STD, dtype)
            vals, idx = lib.elsa_nm_compress(W.cuda(), l.N, l.M)
            ovals, oidx, _ = eo.nm_compress(synth.bits(W), l.N, l.M)
            assert (synth.bits(vals) == ovals).all(), key
            assert (idx_bits(idx, oidx) == oidx).all(), key
    assert len(seen) > 20


# ------------------------------------------------------------------ linear

def run_linear(lib, X, W, bias, N, M, variant):
    lib.elsa_set_linear_variant(variant)
    try:
        Wd = W.cuda()
        vals, idx = lib.elsa_nm_compress(Wd, N, M)
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        Y = lib.elsa_nm_linear(X.cuda(), vals, idx, None if bias is None else bias.cuda(),
                               W.shape[0], W.shape[1], N, M, dev_status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0, "device status %#x" % int(status.item())
        return Y
    finally:
        lib.elsa_set_linear_variant(lib.VARIANT_AUTO)


VARIANTS = ["simt", "tc_dense", "tc_pair"]


def variant_code(lib, name):
    return {"simt": lib.VARIANT_SIMT, "tc_dense": lib.VARIANT_TC_DENSE, "tc_pair": lib.VARIANT_TC_PAIR,
            "tc_sparse": lib.VARIANT_TC_SPARSE, "tc_sparse_pair": lib.VARIANT_TC_SPARSE_PAIR,
            "tc_sparse_ws": lib.VARIANT_TC_SPARSE_WS, "tc_sparse_st": lib.VARIANT_TC_SPARSE_ST,
            "auto": lib.VARIANT_AUTO}[name]


LINEAR_CASES = [
    # rows, in, out, N, M   (ragged row tiles, several K blocks, feature tiles of every width)
    (197, 768, 768, 4, 8),
    (130, 64, 128, 2, 4),
    (1, 128, 64, 1, 4),
    (300, 200, 384, 3, 8),      # K not a multiple of 64, 192-wide feature tile
    (257, 1024, 136, 8, 8),     # dense level, out not a multiple of the chunk width
    (515, 512, 1000, 2, 16),
    (1024, 3072, 768, 1, 8),
    (700, 256, 2304, 4, 16),
]


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
@pytest.mark.parametrize("case", LINEAR_CASES)
def test_linear_matches_oracle(lib, case, dtype, variant):
    rows, in_, out, N, M = case
    X = synth.randn((rows, in_), 11 * rows + in_, synth.X_STD, dtype)
    W = synth.randn((out, in_), 13 * out + in_, synth.W_STD, dtype)
    bias = synth.randn((out,), 17 * out, synth.B_STD, dtype)
    Y = run_linear(lib, X, W, bias, N, M, variant_code(lib, variant))
    check_close(Y, oracle_linear(X, W, bias, N, M, dtype))


@pytest.mark.parametrize("variant", VARIANTS)
def test_identity_activations_give_the_masked_weight_exactly(lib, variant):
    """X = I: Y must be W_masked^T + bias rounded once -- no tolerance, pins indexing and layout."""
    dtype = torch.float16
    in_, out = 256, 320
    W = synth.randn((out, in_), 5, synth.W_STD, dtype)
    bias = synth.randn((out,), 6, synth.B_STD, dtype)
    X = torch.eye(in_, dtype=dtype)
    for N, M in [(2, 8), (1, 4), (3, 8), (8, 8)]:
        Y = run_linear(lib, X, W, bias, N, M, variant_code(lib, variant))
        ref = oracle_linear(X, W, bias, N, M, dtype)
        expect = torch.from_numpy(ref).to(dtype)            # one rounding of the exact value
        assert torch.equal(Y.cpu(), expect), (N, M)


@pytest.mark.parametrize("variant", VARIANTS)
def test_integer_inputs_are_exact(lib, variant):
    """Small integers: every product and partial sum is exact in fp32, so is the result."""
    rng = np.random.default_rng(3)
    rows, in_, out = 200, 192, 96
    X = torch.from_numpy(rng.integers(-4, 5, (rows, in_))).to(torch.bfloat16)
    W = torch.from_numpy(rng.integers(-8, 9, (out, in_))).to(torch.bfloat16)
    for N, M in [(4, 8), (2, 4), (1, 16)]:
        Y = run_linear(lib, X, W, None, N, M, variant_code(lib, variant))
        ref = oracle_linear(X, W, None, N, M, torch.bfloat16)
        # the exact integer result, rounded once to bf16 (integers up to 256 are unchanged)
        assert torch.equal(Y.cpu(), torch.from_numpy(ref).to(torch.bfloat16)), (N, M)


SPARSE_CASES = [
    # rows, in, out, N, M: every level the 2:4 sparse MMA can carry, ragged rows and features
    (197, 768, 768, 2, 8), (500, 128, 384, 1, 4), (225, 64, 128, 2, 4), (1000, 3072, 768, 1, 8),
    (449, 512, 200, 2, 16), (300, 1024, 136, 1, 16), (7, 48, 8, 2, 4), (2300, 768, 2304, 2, 8),
]


SPARSE_VARIANTS = ["tc_sparse", "tc_sparse_pair"]


@pytest.mark.parametrize("variant", SPARSE_VARIANTS)
@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
@pytest.mark.parametrize("case", SPARSE_CASES)
def test_sparse_mma_variant_matches_oracle(lib, case, dtype, variant):
    rows, in_, out, N, M = case
    X = synth.randn((rows, in_), 19 * rows + in_, synth.X_STD, dtype)
    W = synth.randn((out, in_), 23 * out + in_, synth.W_STD, dtype)
    bias = synth.randn((out,), 29 * out, synth.B_STD, dtype)
    Y = run_linear(lib, X, W, bias, N, M, variant_code(lib, variant))
    check_close(Y, oracle_linear(X, W, bias, N, M, dtype))


@pytest.mark.parametrize("variant", SPARSE_VARIANTS)
def test_sparse_mma_variant_exact_cases_and_refusals(lib, variant):
    code = variant_code(lib, variant)
    dtype = torch.float16
    W = synth.randn((320, 256), 5, synth.W_STD, dtype)
    bias = synth.randn((320,), 6, synth.B_STD, dtype)
    X = torch.eye(256, dtype=dtype)
    for N, M in [(2, 8), (1, 4), (2, 4), (1, 16)]:
        Y = run_linear(lib, X, W, bias, N, M, code)
        expect = torch.from_numpy(oracle_linear(X, W, bias, N, M, dtype)).to(dtype)
        assert torch.equal(Y.cpu(), expect), (N, M)
    rng = np.random.default_rng(5)
    Xi = torch.from_numpy(rng.integers(-4, 5, (300, 192))).to(torch.bfloat16)
    Wi = torch.from_numpy(rng.integers(-8, 9, (96, 192))).to(torch.bfloat16)
    for N, M in [(2, 4), (1, 8), (2, 16)]:
        Y = run_linear(lib, Xi, Wi, None, N, M, code)
        ref = oracle_linear(Xi, Wi, None, N, M, torch.bfloat16)
        assert torch.equal(Y.cpu(), torch.from_numpy(ref).to(torch.bfloat16)), (N, M)
    for N, M in [(4, 8), (3, 4), (8, 8)]:                      # more than 2 per chunk possible: refused
        with pytest.raises(lib.ElsaError):
            run_linear(lib, X, W, bias, N, M, code)


WS_CASES = [
    # rows, in, out, N, M: weight block resident in tensor memory (in % 128 == 0, in <= 1024); ragged row
    # tiles, a half-empty feature block, more row tiles than row groups, the narrower tile of in = 1024
    (197, 768, 768, 2, 8), (500, 128, 384, 1, 4), (449, 512, 200, 2, 16), (300, 1024, 136, 1, 16),
    (2300, 768, 2304, 2, 8), (40000, 256, 520, 2, 4), (9000, 1024, 1024, 1, 8), (1, 128, 8, 1, 4),
]


@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
@pytest.mark.parametrize("case", WS_CASES)
def test_weight_stationary_sparse_variant_matches_oracle(lib, case, dtype):
    rows, in_, out, N, M = case
    X = synth.randn((rows, in_), 31 * rows + in_, synth.X_STD, dtype)
    W = synth.randn((out, in_), 37 * out + in_, synth.W_STD, dtype)
    bias = synth.randn((out,), 41 * out, synth.B_STD, dtype)
    Y = run_linear(lib, X, W, bias, N, M, lib.VARIANT_TC_SPARSE_WS)
    if rows <= 4096:
        check_close(Y, oracle_linear(X, W, bias, N, M, dtype))
    else:                                                   # sampled rows: first, last, and a seeded spread
        pick = torch.from_numpy(synth.sample_rows(rows, 512, 7))
        check_close(Y.cpu()[pick], oracle_linear(X[pick], W, bias, N, M, dtype))


def test_weight_stationary_sparse_variant_exact_cases_and_refusals(lib):
    code = lib.VARIANT_TC_SPARSE_WS
    dtype = torch.float16
    W = synth.randn((320, 256), 5, synth.W_STD, dtype)
    bias = synth.randn((320,), 6, synth.B_STD, dtype)
    X = torch.eye(256, dtype=dtype)
    for N, M in [(2, 8), (1, 4), (2, 4), (1, 16)]:
        Y = run_linear(lib, X, W, bias, N, M, code)
        expect = torch.from_numpy(oracle_linear(X, W, bias, N, M, dtype)).to(dtype)
        assert torch.equal(Y.cpu(), expect), (N, M)
    rng = np.random.default_rng(5)
    Xi = torch.from_numpy(rng.integers(-4, 5, (300, 384))).to(torch.bfloat16)
    Wi = torch.from_numpy(rng.integers(-8, 9, (96, 384))).to(torch.bfloat16)
    for N, M in [(2, 4), (1, 8), (2, 16)]:
        Y = run_linear(lib, Xi, Wi, None, N, M, code)
        ref = oracle_linear(Xi, Wi, None, N, M, torch.bfloat16)
        assert torch.equal(Y.cpu(), torch.from_numpy(ref).to(torch.bfloat16)), (N, M)
    for N, M in [(4, 8), (3, 4), (8, 8)]:                      # more than 2 per chunk possible: refused
        with pytest.raises(lib.ElsaError):
            run_linear(lib, X, W, bias, N, M, code)
    with pytest.raises(lib.ElsaError):                         # K block of 128 does not divide in
        run_linear(lib, torch.eye(192, dtype=dtype), synth.randn((64, 192), 7, synth.W_STD, dtype), None, 2, 4, code)
    with pytest.raises(lib.ElsaError):                         # weight block larger than tensor memory
        run_linear(lib, torch.zeros((8, 2048), dtype=dtype), synth.randn((64, 2048), 8, synth.W_STD, dtype), None, 2, 4, code)


ST_CASES = [
    # rows, in, out, N, M: weight streaming through tensor memory in K chunks of 256 (in % 128 == 0, any length);
    # ragged row tiles, a half-empty feature block, a last chunk of 128, more chunks than slots, one chunk only
    (197, 3072, 768, 1, 8), (500, 1152, 384, 2, 4), (449, 2048, 200, 2, 16), (300, 1024, 136, 1, 16),
    (2300, 768, 2304, 2, 8), (9000, 4096, 1024, 1, 8), (1, 128, 8, 1, 4), (40000, 256, 520, 2, 4),
]


@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
@pytest.mark.parametrize("case", ST_CASES)
def test_streaming_sparse_variant_matches_oracle(lib, case, dtype):
    rows, in_, out, N, M = case
    X = synth.randn((rows, in_), 43 * rows + in_, synth.X_STD, dtype)
    W = synth.randn((out, in_), 47 * out + in_, synth.W_STD, dtype)
    bias = synth.randn((out,), 53 * out, synth.B_STD, dtype)
    Y = run_linear(lib, X, W, bias, N, M, lib.VARIANT_TC_SPARSE_ST)
    if rows <= 4096:
        check_close(Y, oracle_linear(X, W, bias, N, M, dtype))
    else:                                                   # sampled rows: first, last, and a seeded spread
        pick = torch.from_numpy(synth.sample_rows(rows, 256, 9))
        check_close(Y.cpu()[pick], oracle_linear(X[pick], W, bias, N, M, dtype))


def test_streaming_sparse_variant_exact_cases_and_refusals(lib):
    code = lib.VARIANT_TC_SPARSE_ST
    dtype = torch.float16
    W = synth.randn((320, 1280), 15, synth.W_STD, dtype)
    bias = synth.randn((320,), 16, synth.B_STD, dtype)
    X = torch.eye(1280, dtype=dtype)                            # Y = masked W^T + bias, one rounding at most
    for N, M in [(2, 8), (1, 4), (2, 4), (1, 16)]:
        Y = run_linear(lib, X, W, bias, N, M, code)
        expect = torch.from_numpy(oracle_linear(X, W, bias, N, M, dtype)).to(dtype)
        assert torch.equal(Y.cpu(), expect), (N, M)
    rng = np.random.default_rng(15)
    Xi = torch.from_numpy(rng.integers(-4, 5, (300, 896))).to(torch.bfloat16)
    Wi = torch.from_numpy(rng.integers(-8, 9, (96, 896))).to(torch.bfloat16)
    for N, M in [(2, 4), (1, 8), (2, 16)]:                      # integer products: fp32 accumulation is exact
        Y = run_linear(lib, Xi, Wi, None, N, M, code)
        ref = oracle_linear(Xi, Wi, None, N, M, torch.bfloat16)
        assert torch.equal(Y.cpu(), torch.from_numpy(ref).to(torch.bfloat16)), (N, M)
    for N, M in [(4, 8), (3, 4), (8, 8)]:                      # more than 2 per chunk possible: refused
        with pytest.raises(lib.ElsaError):
            run_linear(lib, X, W, bias, N, M, code)
    with pytest.raises(lib.ElsaError):                         # in is not a multiple of 128
        run_linear(lib, torch.eye(192, dtype=dtype), synth.randn((64, 192), 17, synth.W_STD, dtype), None, 2, 4, code)


def test_no_bias_and_zero_rows_of_padding(lib):
    dtype = torch.bfloat16
    X = synth.randn((129, 128), 1, 1.0, dtype)
    W = synth.randn((64, 128), 2, synth.W_STD, dtype)
    Yc = torch.full((129 + 8, 64), 7.0, dtype=dtype, device="cuda")      # guard rows after Y
    Wd = W.cuda()
    vals, idx = lib.elsa_nm_compress(Wd, 2, 4)
    lib.elsa_nm_linear(X.cuda(), vals, idx, None, 64, 128, 2, 4, Y=Yc[:129])
    torch.cuda.synchronize()
    check_close(Yc[:129], oracle_linear(X, W, None, 2, 4, dtype))
    assert (Yc[129:] == 7.0).all()                                       # nothing written past the last row


def test_single_layer_config(lib):
    """197 x 768 activations, 768 x 768 weight at 4:8, fp16, seed 0: checked in full."""
    (layer,), dt = synth.workload("single_layer")
    dtype = synth.torch_dtype(dt)
    X, W, b = synth.layer_tensors(layer, dtype)
    ref = oracle_linear(X, W, b, layer.N, layer.M, dtype)
    for v in ("auto", "simt", "tc_dense", "tc_pair"):
        check_close(run_linear(lib, X, W, b, layer.N, layer.M, variant_code(lib, v)), ref)


ROW_TILE_HEIGHTS = (144, 224, 256)    # weight-stationary, streaming / sparse pair, dense pair kernels


def stack_check(lib, layers, dtype, rows_sampled, seed, every_tile=False):
    """Run a table through elsa_vit_compress + elsa_vit_linears and check the packed weights in full and
    sampled rows of every layer against the oracle."""
    code = lib.dtype_code(dtype)
    dev = []
    for l in layers:
        X, W, b = synth.layer_tensors(l, dtype, device="cuda")
        vals, idx = lib.alloc_packed(l.out, l.in_, l.N, l.M, dtype)
        Y = torch.empty((l.rows, l.out), dtype=dtype, device="cuda")
        dev.append(dict(X=X, Y=Y, W=W, vals=vals, idx=idx, bias=b, N=l.N, M=l.M))
    lib.elsa_vit_compress(lib.make_weight_table(dev), code)
    table = lib.make_layer_table(dev)
    ws = lib.alloc_workspace(lib.elsa_vit_workspace_bytes(table, code))
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    lib.elsa_vit_linears(table, code, ws, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    for i, (l, d) in enumerate(zip(layers, dev)):
        pick = synth.sample_rows(l.rows, rows_sampled, seed + i)
        if every_tile:
            # one seeded row inside every row tile, for each tile height the kernels use: a persistent launch
            # walks one tile sequence over many layers, and a wrong tile anywhere in it must show
            rng = np.random.default_rng(seed + 1000 + i)
            extra = [np.minimum(np.arange(0, l.rows, t) + rng.integers(0, t, size=-(-l.rows // t)), l.rows - 1)
                     for t in ROW_TILE_HEIGHTS]
            pick = np.unique(np.concatenate([pick] + extra))
        sel = torch.from_numpy(pick).cuda()
        Xs = d["X"][sel].cpu()
        ovals, oidx, _ = eo.nm_compress(synth.bits(d["W"]), l.N, l.M)
        assert (synth.bits(d["vals"]) == ovals).all() and (idx_bits(d["idx"], oidx) == oidx).all(), l.name
        ref = eo.nm_linear_f64(synth.bits(Xs), ovals, oidx, synth.bits(d["bias"]), l.out, l.in_, l.N, l.M,
                               ocode(dtype))
        check_close(d["Y"][sel], ref)
        del d["X"], d["Y"]


def test_deit_b_block_layers_sampled_rows(lib):
    """One DeiT-B block at batch 64 (qkv 4:8, proj 2:8, fc1 2:8, fc2 1:8), full size on the GPU,
    sampled rows against the oracle, weights compared in full."""
    layers, dt = synth.workload("deit_b_block_b64")
    stack_check(lib, layers, synth.torch_dtype(dt), 160, 21)


def test_deit_b_stack_full_size_sampled_rows(lib):
    """All 48 DeiT-B linears at batch 256, the configuration the benchmark times."""
    layers, dt = synth.workload("deit_b_stack_b256")
    dtype = synth.torch_dtype(dt)
    # run the whole table in one call, a few layers' worth of memory at a time is not needed: 15 GB fits
    stack_check(lib, layers, dtype, 24, 31, every_tile=True)


def test_swin_b_stack_full_size_sampled_rows(lib):
    layers, dt = synth.workload("swin_b_stack_b128")
    stack_check(lib, layers, synth.torch_dtype(dt), 24, 41, every_tile=True)


def test_streaming_layers_share_one_launch(lib):
    """A table whose layers all take the streaming sparse kernel under the automatic rule (N <= 2, in > 768,
    in % 128 == 0): reductions of 4, 4.5, 8 and 12 chunks, a last feature block of only 8 features, ragged row
    tiles; one launch carries them all, its tiles forming one sequence."""
    dtype = torch.bfloat16
    layers = [synth.Layer("a", 6000, 1024, 1280, 1, 8, 601, 602, 603),
              synth.Layer("b", 5001, 1152, 1024, 2, 8, 611, 612, 613),
              synth.Layer("c", 4100, 2048, 2312, 2, 4, 621, 622, 623),
              synth.Layer("d", 7777, 3072, 768, 1, 16, 631, 632, 633)]
    lib.elsa_profile_start()
    stack_check(lib, layers, dtype, 96, 61, every_tile=True)
    recs = lib.elsa_profile_stop()
    assert [k for (k, _, _) in recs if k.startswith("linear")] == ["linear_tc_sp24_st"], recs


def test_weight_stationary_layers_share_one_launch(lib):
    """A table whose layers all take the weight-stationary sparse kernel under the automatic rule
    (N <= 2, in of 768-896, out >= 1024): feature blocks that do not divide the CTA pairs (5 and 10 blocks),
    a last block of only 8 features, ragged row tiles, two different K; one launch carries them all."""
    dtype = torch.bfloat16
    layers = [synth.Layer("a", 6000, 896, 1280, 1, 8, 501, 502, 503),
              synth.Layer("b", 5001, 768, 1024, 2, 8, 511, 512, 513),
              synth.Layer("c", 4100, 768, 2312, 2, 4, 521, 522, 523),
              synth.Layer("d", 7777, 896, 3072, 1, 16, 531, 532, 533)]
    lib.elsa_profile_start()
    stack_check(lib, layers, dtype, 96, 51)
    recs = lib.elsa_profile_stop()
    assert [k for (k, _, _) in recs if k.startswith("linear")] == ["linear_tc_sp24_ws"], recs


def test_shared_launches_give_the_same_bits_as_one_launch_per_layer(lib):
    """elsa_vit_linears with per-layer scratch (layers share persistent launches) against the same
    table run layer by layer, on a table that mixes all three tensor-core families."""
    dtype = torch.bfloat16
    code = lib.dtype_code(dtype)
    layers = [synth.Layer("sparse_a", 9000, 768, 768, 2, 8, 201, 202, 203),
              synth.Layer("dense_pair_a", 19000, 256, 384, 4, 8, 204, 205, 206),
              synth.Layer("small", 150, 128, 64, 1, 4, 207, 208, 209),
              synth.Layer("dense_level", 19000, 512, 256, 8, 8, 210, 211, 212),
              synth.Layer("sparse_b", 9000, 1024, 512, 1, 16, 213, 214, 215),
              synth.Layer("dense_pair_b", 20000, 128, 1000, 3, 8, 216, 217, 218)]
    dev = []
    for l in layers:
        X, W, b = synth.layer_tensors(l, dtype, device="cuda")
        vals, idx = lib.elsa_nm_compress(W, l.N, l.M)
        dev.append(dict(X=X, W=W, vals=vals, idx=idx, bias=b, N=l.N, M=l.M,
                        Y=torch.empty((l.rows, l.out), dtype=dtype, device="cuda")))
    table = lib.make_layer_table(dev)
    ws = lib.alloc_workspace(lib.elsa_vit_workspace_bytes(table, code))
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    lib.elsa_vit_linears(table, code, ws, dev_status=status)
    torch.cuda.synchronize()
    shared = [d["Y"].clone() for d in dev]
    for d in dev:
        d["Y"].zero_()
    lib.elsa_set_grouping(False)
    try:
        lib.elsa_vit_linears(table, code, ws, dev_status=status)
        torch.cuda.synchronize()
    finally:
        lib.elsa_set_grouping(True)
    assert int(status.item()) == 0
    for l, d, y in zip(layers, dev, shared):
        assert torch.equal(d["Y"], y), l.name
        pick = torch.from_numpy(synth.sample_rows(l.rows, 40, 77)).cuda()
        check_close(y[pick], oracle_linear(d["X"][pick].cpu(), d["W"].cpu(), d["bias"].cpu(), l.N, l.M, dtype))
    # a scratch of only the largest layer's size still works: the layers then run one after the other
    small_ws = lib.alloc_workspace(max(lib.elsa_workspace_bytes(l.rows, l.in_, l.out, l.N, l.M, code) for l in layers))
    for d in dev:
        d["Y"].zero_()
    lib.elsa_vit_linears(table, code, small_ws, dev_status=status)
    torch.cuda.synchronize()
    for d, y in zip(dev, shared):
        assert torch.equal(d["Y"], y)


def test_host_memory_entry_point_matches_device_entry_point(lib):
    dtype = torch.float16
    layers = [synth.Layer("a", 300, 256, 384, 2, 8, 1, 2, 3), synth.Layer("b", 300, 384, 128, 4, 4, 4, 5, 6),
              synth.Layer("c", 77, 128, 256, 1, 16, 7, 8, 9)]
    host, dev_out = [], []
    for l in layers:
        X, W, b = synth.layer_tensors(l, dtype)
        Y = torch.empty((l.rows, l.out), dtype=dtype).pin_memory()
        host.append(dict(X=X.pin_memory(), Y=Y, W=W.pin_memory(), bias=b.pin_memory(), N=l.N, M=l.M))
        dev_out.append(run_linear(lib, X, W, b, l.N, l.M, lib.VARIANT_AUTO).cpu())
    table = lib.make_host_layer_table(host)
    code = lib.dtype_code(dtype)
    mem = lib.alloc_workspace(lib.elsa_vit_host_device_bytes(table, code))
    lib.elsa_vit_linears_host(table, code, mem)
    torch.cuda.synchronize()
    for h, y in zip(host, dev_out):
        assert torch.equal(h["Y"], y)


@pytest.mark.parametrize("dt", ["f16", "bf16"])
def test_sweep_points_sampled_rows(lib, dt):
    """Every (rows, K, O, level) point of the shape / sparsity sweep at full size: packed weight
    compared in full once per weight, 12 sampled rows of Y per point against the oracle."""
    dtype = synth.torch_dtype(dt)
    packed = {}
    for i, l in enumerate(synth.sweep()):
        key = (l.in_, l.out, l.N, l.M)
        if key not in packed:
            W = synth.randn((l.out, l.in_), 7000 + len(packed), synth.W_STD, dtype, "cuda")
            vals, idx = lib.elsa_nm_compress(W, l.N, l.M)
            ovals, oidx, _ = eo.nm_compress(synth.bits(W), l.N, l.M)
            assert (synth.bits(vals) == ovals).all() and (idx_bits(idx, oidx) == oidx).all(), key
            packed[key] = (vals, idx, ovals, oidx)
        vals, idx, ovals, oidx = packed[key]
        X = synth.randn((l.rows, l.in_), l.seed_x, synth.X_STD, dtype, "cuda")
        b = synth.randn((l.out,), l.seed_b, synth.B_STD, dtype, "cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        Y = lib.elsa_nm_linear(X, vals, idx, b, l.out, l.in_, l.N, l.M, dev_status=status)
        pick = torch.from_numpy(synth.sample_rows(l.rows, 12, 900 + i, tile=256)).cuda()
        ref = eo.nm_linear_f64(synth.bits(X[pick]), ovals, oidx, synth.bits(b), l.out, l.in_, l.N, l.M, ocode(dtype))
        assert int(status.item()) == 0
        check_close(Y[pick], ref)


# ------------------------------------------------------------------ supernet-side forms (Sec. 3.1)

@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
@pytest.mark.parametrize("M,N_list", [(4, [1, 2, 3, 4]), (8, [1, 2, 3, 4, 8]), (16, [1, 2, 4, 8, 15, 16])])
def test_all_levels_in_one_pass_match_the_oracle(lib, M, N_list, dtype):
    """Shared weight, every level of the search space from one read: each level's packed form is the
    oracle's, bit for bit (and the kept sets nest, Sec. 3.1)."""
    W = synth.randn((72, 16 * 23), 300 + M, synth.W_STD, dtype)
    Wb = synth.bits(W)
    packed = lib.elsa_nm_compress_levels(W.cuda(), N_list, M)
    torch.cuda.synchronize()
    prev = None
    for N, (vals, idx) in zip(N_list, packed):
        ovals, oidx, omask = eo.nm_compress(Wb, N, M)
        assert (synth.bits(vals) == ovals).all(), (N, M)
        assert (idx_bits(idx, oidx) == oidx).all(), (N, M)
        if prev is not None:
            assert (omask >= prev).all()
        prev = omask


MASKED_CASES = [
    # rows, in, out, N, M -> kernel family the automatic dispatch takes
    (9000, 768, 512, 2, 8),      # 2:4 sparse MMA on CTA pairs, re-encoded from the dense weight
    (9000, 1024, 256, 1, 16),    # the same, M = 16
    (19000, 256, 384, 4, 8),     # dense-rate pair kernel on the masked image
    (19000, 512, 256, 8, 8),     # dense level: the shared weight as it is
    (197, 768, 768, 3, 8),       # small: one CTA per tile
]


@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
@pytest.mark.parametrize("case", MASKED_CASES)
def test_mask_on_load_linear_matches_oracle_and_packed_path(lib, case, dtype):
    rows, in_, out, N, M = case
    X = synth.randn((rows, in_), 31 * rows + in_, synth.X_STD, dtype, "cuda")
    W = synth.randn((out, in_), 37 * out + in_, synth.W_STD, dtype, "cuda")
    bias = synth.randn((out,), 41 * out, synth.B_STD, dtype, "cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    Y = lib.elsa_nm_linear_masked(X, W, bias, N, M, dev_status=status)
    vals, idx = lib.elsa_nm_compress(W, N, M)
    Y_packed = lib.elsa_nm_linear(X, vals, idx, bias, out, in_, N, M, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.equal(Y, Y_packed)                      # same projection, same kernels
    pick = torch.from_numpy(synth.sample_rows(rows, 48, 5)).cuda()
    check_close(Y[pick], oracle_linear(X[pick].cpu(), W.cpu(), bias.cpu(), N, M, dtype))


def test_a_wait_that_runs_out_reports_and_leaves_the_device_usable(lib):
    """The failure path every tensor-core kernel shares: a bounded wait on a barrier nobody arrives at gives up
    after its limit (here one millisecond), records ELSA_ERR_TIMEOUT with the site of the wait, and the kernel
    returns.  Nothing faults and nothing hangs: the next ordinary call runs and is correct."""
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    lib.elsa_selftest_wait_timeout(1_000_000, status)
    t1.record()
    torch.cuda.synchronize()
    code = int(status.item())
    assert code & 0xFF == 8 and (code >> 8) == 15, "device status %#x" % code      # ELSA_ERR_TIMEOUT | site << 8
    assert 0.9 <= t0.elapsed_time(t1) < 100.0                                       # the limit, not the kernels' 2 s
    # a status that is already set is kept (first failure wins)
    lib.elsa_selftest_wait_timeout(200_000, status)
    torch.cuda.synchronize()
    assert int(status.item()) == code
    with pytest.raises(lib.ElsaError):
        lib.elsa_selftest_wait_timeout(0, status)
    # the device is as usable as before
    dtype = torch.bfloat16
    X = synth.randn((300, 768), 71, synth.X_STD, dtype)
    W = synth.randn((256, 768), 72, synth.W_STD, dtype)
    bias = synth.randn((256,), 73, synth.B_STD, dtype)
    Y = run_linear(lib, X, W, bias, 2, 8, lib.VARIANT_AUTO)
    check_close(Y, oracle_linear(X, W, bias, 2, 8, dtype))
