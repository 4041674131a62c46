"""The chained transformer block (elsa_vit_block and its two phases) against oracle/elsa_block_oracle.py.

Two comparisons per case.  Stage by stage: every stage's stored 16-bit result against the oracle's fp64 result of
that stage computed from the library's own stored inputs, so each kernel is held to one rounding.  Whole chain:
the library's results against block_forward from x alone, where the stages' roundings compound.

Tolerance of a stage, |got - ref| <= u * (|ref| + |lin|) + 5e-4 with u one unit in the last place of the 16-bit
type relative to the value (2^-7 bf16, 2^-10 fp16): the library computes in fp32 and rounds once where the
oracle computes in fp64 and rounds once, so the two can land on neighbouring 16-bit values; |lin| is the
magnitude of the linear's own output at the stages that add a residual or apply GELU (a kernel whose epilogue
cannot take the residual or the activation rounds the linear's output first; GELU's slope is at most 1.13); 5e-4 is above the fp32 accumulation bound
K * 2^-24 * max|x w| ~ 1e-4 of the longest reduction here.  In the chain a stage also inherits the rounding
of its inputs, which LayerNorm and the linears carry from the large elements of a row to its small ones: each
element is held to four times the stage tolerance with the largest |ref| of its row added to |ref|, and every
stage as a whole to a relative Frobenius error of 5e-3 (the bound of the single linears' parity tests).

Attention (elsa_attention, and the block run with it): the kernel keeps fp32 scores and row sums and rounds the
probabilities to the 16-bit type for the second product, so |err| <= u |ref| + (u / 2) max|v| + 1e-5 with max|v|
over the head's values in the image (sum of p |v| <= max|v|; a probability's rounding is u / 4 relative).
"""
import numpy as np
import pytest
import torch

from oracle import elsa_block_oracle as bo
from oracle import elsa_oracle as eo
from paper_2409_09708_b200 import synth

STAGES = ("x1", "qkv", "a", "x2", "x3", "h", "y")
NAMES = ("qkv", "proj", "fc1", "fc2")


def shapes_of(dim, mlp):
    return {"qkv": (3 * dim, dim), "proj": (dim, dim), "fc1": (mlp, dim), "fc2": (dim, mlp)}


def make_params(dim, mlp, levels, dtype, seed):
    """Host tensors of one block: weights N(0, 0.02 .. 0.08), biases, LayerNorm gains near 1."""
    host = {}
    for i, (name, (o, k)) in enumerate(shapes_of(dim, mlp).items()):
        host["W_" + name] = synth.randn((o, k), seed + i, 2.0 / np.sqrt(k), dtype)
        host["b_" + name] = synth.randn((o,), seed + 10 + i, 0.02, dtype)
    for i, name in enumerate(("ln1_g", "ln1_b", "ln2_g", "ln2_b")):
        t = synth.randn((dim,), seed + 20 + i, 0.1, dtype).float() + (1.0 if name.endswith("g") else 0.0)
        host[name] = t.to(dtype)
    p = {k: synth.bits(v) for k, v in host.items()}
    for name in NAMES:
        p["level_" + name] = levels[name]
    return host, p


def test_scratch_layout_is_host_arithmetic():
    from paper_2409_09708_b200 import build
    build.build()
    from paper_2409_09708_b200 import binding as lib
    w = lib.ElsaBlockWeights()
    for name, (N, M) in zip(NAMES, [(8, 8), (2, 8), (4, 8), (1, 8)]):
        setattr(w, name, lib.ElsaBlockLinear(None, None, None, N, M))
    rows, dim, mlp = 1000, 768, 3072
    total, off = lib.elsa_vit_block_scratch_bytes(rows, dim, mlp, w, lib.BF16)
    sizes = {"x1": dim, "qkv": 3 * dim, "a": dim, "x2": dim, "x3": dim, "h": mlp, "t": dim}
    at = 0
    for name in lib.BLOCK_REGIONS[:-1]:
        assert off[name] == at and at % 256 == 0
        at += -(-rows * sizes[name] * 2 // 256) * 256
    assert off["workspace"] == at
    ws = sum(-(-lib.elsa_workspace_bytes(rows, k, o, N, M, lib.BF16) // 256) * 256
             for (o, k), (N, M) in zip(shapes_of(dim, mlp).values(), [(8, 8), (2, 8), (4, 8), (1, 8)]))
    assert total == at + ws
    assert lib.elsa_vit_block_scratch_bytes(rows, 772, mlp, w, lib.BF16)[0] == 0       # dim % 8 != 0
    w.fc2 = lib.ElsaBlockLinear(None, None, None, 9, 8)
    assert lib.elsa_vit_block_scratch_bytes(rows, dim, mlp, w, lib.BF16)[0] == 0       # N > M


# ------------------------------------------------------------------------------------------------ GPU

def run_block(lib, x, host, levels, mlp, variant=None, phase="both", attn=None):
    """Compresses the four weights, runs the block; returns ({stage: fp64 array}, {stage: bits}, weights)."""
    dtype = x.dtype
    rows, dim = x.shape
    dev = {k: v.cuda() for k, v in host.items()}
    lin = {}
    for name in NAMES:
        N, M = levels[name]
        vals, idx = lib.elsa_nm_compress(dev["W_" + name], N, M)
        lin[name] = (vals, idx, dev["b_" + name], N, M)
    w, keep = lib.make_block_weights(dev["ln1_g"], dev["ln1_b"], dev["ln2_g"], dev["ln2_b"], lin, eps=1e-6)
    code = lib.dtype_code(dtype)
    total, off = lib.elsa_vit_block_scratch_bytes(rows, dim, mlp, w, code)
    scratch = torch.zeros(total, dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    xd = x.cuda()
    if variant is not None:
        lib.elsa_set_linear_variant(variant)
    try:
        if phase == "both" and attn:
            y, _ = lib.elsa_vit_block(xd, mlp, w, scratch=scratch, dev_status=status, tokens=attn[0], heads=attn[1])
        elif phase == "both":
            y, _ = lib.elsa_vit_block(xd, mlp, w, scratch=scratch, dev_status=status)
        else:
            lib.elsa_vit_block(xd, mlp, w, scratch=scratch, dev_status=status, phase="qkv")
            qkv = lib.block_region(scratch, off, "qkv", rows, 3 * dim, dtype)
            lib.block_region(scratch, off, "a", rows, dim, dtype).copy_(qkv[:, 2 * dim:])   # the caller's "attention"
            y, _ = lib.elsa_vit_block(xd, mlp, w, scratch=scratch, dev_status=status, phase="rest")
        torch.cuda.synchronize()
    finally:
        lib.elsa_set_linear_variant(lib.VARIANT_AUTO)
    assert int(status.item()) == 0, "device status %#x" % int(status.item())
    cols = {"x1": dim, "qkv": 3 * dim, "a": dim, "x2": dim, "x3": dim, "h": mlp}
    got = {s: lib.block_region(scratch, off, s, rows, cols[s], dtype).cpu() for s in cols}
    got["y"] = y.cpu()
    return got


def stage_tolerance(ref, lin, dtype):
    u = 2.0 ** -7 if dtype == torch.bfloat16 else 2.0 ** -10
    return u * (np.abs(ref) + (0 if lin is None else np.abs(lin))) + 5e-4


def attention_tolerance(ref, v, tokens, heads, dtype):
    """ref, v: [rows, dim] fp64 (v = the value third of qkv); per element u |ref| + u / 2 max|v| of its head and image."""
    u = 2.0 ** -7 if dtype == torch.bfloat16 else 2.0 ** -10
    rows, dim = v.shape
    vmax = np.abs(v).reshape(rows // tokens, tokens, heads, dim // heads).max(axis=(1, 3), keepdims=True)
    vmax = np.broadcast_to(vmax, (rows // tokens, tokens, heads, dim // heads)).reshape(rows, dim)
    return u * np.abs(ref) + 0.5 * u * vmax + 1e-5


def check_rows(got, x, p, dtype, rows_idx, attn=None):
    """Both comparisons on the given rows (the block treats token rows independently; with attention the rows
    must be whole images)."""
    code = eo.F16 if dtype == torch.float16 else eo.BF16
    f64 = lambda t: t[rows_idx].to(torch.float64).numpy()
    bits = lambda t: synth.bits(t[rows_idx].contiguous())
    g = {s: f64(got[s]) for s in STAGES}
    for s in STAGES:
        assert np.isfinite(g[s]).all(), s
    dim = x.shape[1]
    r16 = lambda a: bo._round16(a, dtype)
    pf = lambda key: torch.from_numpy(p[key].view(np.int16)).view(dtype).to(torch.float64).numpy()
    lin = lambda name, inp: bo.sparse_linear(inp, p["W_" + name], p["b_" + name], *p["level_" + name], code)
    xs = f64(x)
    # stage by stage, from the library's own stored inputs
    proj, fc1, fc2 = lin("proj", g["a"]), lin("fc1", g["x3"]), lin("fc2", g["h"])
    stage_ref = {
        "x1": (r16(bo.layer_norm(xs, pf("ln1_g"), pf("ln1_b"), 1e-6)), None),
        "qkv": (r16(lin("qkv", g["x1"])), None),
        "x2": (r16(xs + proj), proj),
        "x3": (r16(bo.layer_norm(g["x2"], pf("ln2_g"), pf("ln2_b"), 1e-6)), None),
        "h": (r16(bo.gelu(fc1)), 1.13 * fc1),
        "y": (r16(g["x2"] + fc2), fc2),
    }
    if attn is None:
        assert np.array_equal(bits(got["a"]), bits(got["qkv"][:, 2 * dim:3 * dim]))  # the stand-in copies V through
    elif isinstance(attn, dict):                                                      # Swin's windows
        ref = r16(bo.window_attention(g["qkv"], attn["H"], attn["W"], attn["ws"], attn["shift"], attn["heads"], attn["rel_bias"]))
        u = 2.0 ** -7 if dtype == torch.bfloat16 else 2.0 ** -10
        tol = u * np.abs(ref) + 0.5 * u * np.abs(g["qkv"][:, 2 * dim:]).max() + 1e-5
        err = np.abs(g["a"] - ref)
        worst = (err - tol).argmax()
        assert (err <= tol).all(), "stage a: error %g at tolerance %g" % (err.flat[worst], tol.flat[worst])
    else:
        ref = r16(bo.attention(g["qkv"], *attn))
        tol = attention_tolerance(ref, g["qkv"][:, 2 * dim:], attn[0], attn[1], dtype)
        err = np.abs(g["a"] - ref)
        worst = (err - tol).argmax()
        assert (err <= tol).all(), "stage a: error %g at tolerance %g" % (err.flat[worst], tol.flat[worst])
    for s, (ref, mag) in stage_ref.items():
        err = np.abs(g[s] - ref)
        tol = stage_tolerance(ref, mag, dtype)
        worst = (err - tol).argmax()
        assert (err <= tol).all(), "stage %s: error %g at tolerance %g" % (s, err.flat[worst], tol.flat[worst])
    # the whole chain from x alone
    if attn is None:
        how = {}
    elif isinstance(attn, dict):
        how = dict(attn="window", heads=attn["heads"], window=attn)
    else:
        how = dict(attn="softmax", tokens=attn[0], heads=attn[1])
    chain = bo.block_forward(bits(x), p, code, eps=1e-6, **how)
    for s in STAGES:
        mag = chain["x2"] - xs if s == "x2" else chain["y"] - chain["x2"] if s == "y" else 1.13 * fc1 if s == "h" else None
        err = np.abs(g[s] - chain[s])
        row_max = np.abs(chain[s]).max(axis=1, keepdims=True)
        tol = 4 * stage_tolerance(chain[s], row_max if mag is None else np.abs(mag) + row_max, dtype)
        worst = (err - tol).argmax()
        assert (err <= tol).all(), "chain %s: error %g at tolerance %g" % (s, err.flat[worst], tol.flat[worst])
        assert np.linalg.norm(g[s] - chain[s]) <= 5e-3 * np.linalg.norm(chain[s]), s


@pytest.fixture(scope="module")
def lib():
    from paper_2409_09708_b200 import build
    build.build()
    from paper_2409_09708_b200 import binding
    return binding


SPARSE_LEVELS = {"qkv": (2, 8), "proj": (1, 8), "fc1": (2, 4), "fc2": (1, 4)}
MIXED_LEVELS = {"qkv": (8, 8), "proj": (4, 8), "fc1": (2, 8), "fc2": (3, 4)}
SMALL = [("simt", MIXED_LEVELS), ("tc_dense", MIXED_LEVELS), ("tc_pair", MIXED_LEVELS), ("tc_pair", SPARSE_LEVELS),
         ("tc_sparse_pair", SPARSE_LEVELS), ("tc_sparse_ws", SPARSE_LEVELS), ("tc_sparse_st", SPARSE_LEVELS),
         ("auto", MIXED_LEVELS)]


@pytest.mark.gpu
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float16], ids=["bf16", "f16"])
@pytest.mark.parametrize("variant,levels", SMALL, ids=["%s-%s" % (v, "sparse" if l is SPARSE_LEVELS else "mixed") for v, l in SMALL])
def test_block_matches_oracle_on_every_kernel_family(lib, variant, levels, dtype):
    rows, dim, mlp = 333, 256, 1024                 # a ragged last tile for every kernel's row tile
    host, p = make_params(dim, mlp, levels, dtype, 100)
    x = synth.randn((rows, dim), 7, 1.5, dtype)
    x[5] = 0.75                                      # a constant row: zero variance, LayerNorm leaves its bias
    x[6] = 0.0
    code = {"simt": lib.VARIANT_SIMT, "tc_dense": lib.VARIANT_TC_DENSE, "tc_pair": lib.VARIANT_TC_PAIR,
            "tc_sparse_pair": lib.VARIANT_TC_SPARSE_PAIR, "tc_sparse_ws": lib.VARIANT_TC_SPARSE_WS,
            "tc_sparse_st": lib.VARIANT_TC_SPARSE_ST, "auto": lib.VARIANT_AUTO}[variant]
    got = run_block(lib, x, host, levels, mlp, variant=code)
    check_rows(got, x, p, dtype, np.arange(rows))


@pytest.mark.gpu
@pytest.mark.parametrize("levels", [SPARSE_LEVELS, MIXED_LEVELS], ids=["sparse", "mixed"])
@pytest.mark.parametrize("dim", [128, 512, 768, 1024])
def test_row_widths_of_the_row_wise_kernels(lib, dim, levels):
    # 128, 256 (above), 512 and 1024 take the several-rows-per-warp LayerNorm, 768 the one-row-per-warp one; 77 rows
    # leave a ragged last step for every rows-per-step (8, 4, 2); sparse proj / fc2 make the add-and-normalise form run
    dtype = torch.bfloat16
    rows, mlp = 77, 512
    host, p = make_params(dim, mlp, levels, dtype, 310 + dim)
    x = synth.randn((rows, dim), 9, 1.25, dtype)
    x[3] = -0.5
    got = run_block(lib, x, host, levels, mlp)
    check_rows(got, x, p, dtype, np.arange(rows))


@pytest.mark.gpu
def test_rows_longer_than_the_register_cache(lib):
    # dim > 1024: LayerNorm re-reads the part of the row it does not keep in registers
    dtype = torch.bfloat16
    rows, dim, mlp = 70, 1536, 512
    host, p = make_params(dim, mlp, MIXED_LEVELS, dtype, 300)
    x = synth.randn((rows, dim), 8, 1.0, dtype)
    got = run_block(lib, x, host, MIXED_LEVELS, mlp)
    check_rows(got, x, p, dtype, np.arange(rows))


@pytest.mark.gpu
def test_two_phases_with_the_callers_attention_give_the_same_bits(lib):
    dtype = torch.bfloat16
    rows, dim, mlp = 400, 256, 1024
    host, _ = make_params(dim, mlp, MIXED_LEVELS, dtype, 500)
    x = synth.randn((rows, dim), 9, 1.0, dtype)
    whole = run_block(lib, x, host, MIXED_LEVELS, mlp)
    split = run_block(lib, x, host, MIXED_LEVELS, mlp, phase="split")
    for s in STAGES:
        assert torch.equal(whole[s].view(torch.int16), split[s].view(torch.int16)), s


DEIT_LEVELS = [{"qkv": (2, 8), "proj": (1, 8), "fc1": (4, 8), "fc2": (2, 8)},     # WS, WS, dense pair + image, ST
               {"qkv": (8, 8), "proj": (4, 8), "fc1": (1, 8), "fc2": (8, 8)}]     # dense pair (fused residuals), WS


@pytest.mark.gpu
@pytest.mark.parametrize("levels", DEIT_LEVELS, ids=["sparse_heavy", "dense_heavy"])
def test_deit_b_block_full_size_sampled_rows(lib, levels):
    # the block at the size the timing runs (batch 256 x 197 tokens, dim 768, mlp 3072), AUTO kernel choice;
    # the oracle follows 40 token rows, among them the first and last row of row tiles of every kernel
    dtype = torch.bfloat16
    rows, dim, mlp = 256 * 197, 768, 3072
    host, p = make_params(dim, mlp, levels, dtype, 700)
    x = synth.randn((rows, dim), 11, 1.0, dtype, "cuda").cpu()
    got = run_block(lib, x, host, levels, mlp)
    rng = np.random.default_rng(5)
    edges = [0, 143, 144, 223, 224, 255, 256, rows - 1, rows - 145, (rows // 224) * 224, (rows // 144) * 144]
    pick = np.unique(np.concatenate([np.array(edges), rng.integers(0, rows, 29)]))
    check_rows(got, x, p, dtype, pick)


@pytest.mark.gpu
def test_block_validation(lib):
    dtype = torch.bfloat16
    rows, dim, mlp = 64, 256, 512
    host, _ = make_params(dim, mlp, MIXED_LEVELS, dtype, 900)
    dev = {k: v.cuda() for k, v in host.items()}
    lin = {}
    for name in NAMES:
        N, M = MIXED_LEVELS[name]
        vals, idx = lib.elsa_nm_compress(dev["W_" + name], N, M)
        lin[name] = (vals, idx, dev["b_" + name], N, M)
    w, keep = lib.make_block_weights(dev["ln1_g"], dev["ln1_b"], dev["ln2_g"], dev["ln2_b"], lin)
    x = synth.randn((rows, dim), 1, 1.0, dtype).cuda()
    total, _ = lib.elsa_vit_block_scratch_bytes(rows, dim, mlp, w, lib.BF16)
    before = lib.elsa_launch_count()
    with pytest.raises(lib.ElsaError) as e:
        lib.elsa_vit_block(x, mlp, w, scratch=torch.empty(total - 256, dtype=torch.uint8, device="cuda"))
    assert e.value.status == 6                                   # ELSA_ERR_WORKSPACE
    with pytest.raises(lib.ElsaError) as e:
        lib.elsa_vit_block(x, mlp, w, y=x)
    assert e.value.status == 5                                   # y aliases x
    w.fc1.idx = None
    with pytest.raises(lib.ElsaError) as e:
        lib.elsa_vit_block(x, mlp, w)
    assert e.value.status == 1 and "fc1" in str(e.value)
    assert lib.elsa_launch_count() == before                     # nothing was enqueued


ATTN_CASES = [(3, 197, 2, 1.0), (2, 64, 1, 1.0), (5, 49, 3, 1.0), (2, 256, 2, 1.0), (3, 130, 1, 1.0), (1, 16, 1, 1.0),
              (2, 7, 2, 1.0), (2, 197, 1, 4.0)]


@pytest.mark.gpu
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float16], ids=["bf16", "f16"])
@pytest.mark.parametrize("case", ATTN_CASES, ids=["%dx%dx%d_s%g" % c for c in ATTN_CASES])
def test_attention_matches_oracle(lib, case, dtype):
    images, tokens, heads, scale = case              # scale 4: scores up to +-60, the row maximum matters
    dim = 64 * heads
    qkv = synth.randn((images * tokens, 3 * dim), 17, scale, dtype)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    guard = torch.full((images * tokens + 64, dim), 7.0, dtype=dtype, device="cuda")   # rows after the last image stay
    a = guard[:images * tokens]
    lib.elsa_attention(qkv.cuda(), tokens, heads, a=a, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0, "device status %#x" % int(status.item())
    assert (guard[images * tokens:] == 7.0).all()
    q64 = qkv.double().numpy()
    ref = bo._round16(bo.attention(q64, tokens, heads), dtype)
    got = a.double().cpu().numpy()
    assert np.isfinite(got).all()
    tol = attention_tolerance(ref, q64[:, 2 * dim:], tokens, heads, dtype)
    err = np.abs(got - ref)
    worst = (err - tol).argmax()
    assert (err <= tol).all(), "error %g at tolerance %g" % (err.flat[worst], tol.flat[worst])


@pytest.mark.gpu
def test_attention_refuses_shapes_it_does_not_cover(lib):
    qkv = torch.zeros((300, 3 * 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(lib.ElsaError) as e:
        lib.elsa_attention(qkv, 300, 1)                 # more than 256 tokens per image
    assert e.value.status == 2
    qkv = torch.zeros((64, 3 * 96), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(lib.ElsaError) as e:
        lib.elsa_attention(qkv, 64, 1)                  # head dimension 96
    assert e.value.status == 2


@pytest.mark.gpu
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float16], ids=["bf16", "f16"])
def test_block_with_attention_matches_oracle(lib, dtype):
    images, tokens, heads, mlp = 3, 197, 4, 1024
    dim = 64 * heads
    host, p = make_params(dim, mlp, MIXED_LEVELS, dtype, 1100)
    x = synth.randn((images * tokens, dim), 12, 1.0, dtype)
    got = run_block(lib, x, host, MIXED_LEVELS, mlp, attn=(tokens, heads))
    check_rows(got, x, p, dtype, np.arange(images * tokens), attn=(tokens, heads))


@pytest.mark.gpu
def test_deit_b_block_with_attention_full_size_sampled_images(lib):
    dtype = torch.bfloat16
    images, tokens, heads, dim, mlp = 256, 197, 12, 768, 3072
    levels = DEIT_LEVELS[0]
    host, p = make_params(dim, mlp, levels, dtype, 1300)
    x = synth.randn((images * tokens, dim), 13, 1.0, dtype, "cuda").cpu()
    got = run_block(lib, x, host, levels, mlp, attn=(tokens, heads))
    pick = np.concatenate([np.arange(i * tokens, (i + 1) * tokens) for i in (0, 101, 255)])   # whole images
    check_rows(got, x, p, dtype, pick, attn=(tokens, heads))


def _encoder_case(lib, dtype, images, tokens, heads, mlp, level_sets, seed):
    dim = 64 * heads
    x = synth.randn((images * tokens, dim), seed, 1.0, dtype)
    blocks, params, keep = [], [], []
    for b, levels in enumerate(level_sets):
        host, p = make_params(dim, mlp, levels, dtype, seed + 100 * (b + 1))
        dev = {k: v.cuda() for k, v in host.items()}
        lin = {}
        for name in NAMES:
            N, M = levels[name]
            vals, idx = lib.elsa_nm_compress(dev["W_" + name], N, M)
            lin[name] = (vals, idx, dev["b_" + name], N, M)
        w, k = lib.make_block_weights(dev["ln1_g"], dev["ln1_b"], dev["ln2_g"], dev["ln2_b"], lin, eps=1e-6)
        blocks.append(w)
        params.append(p)
        keep.append((dev, lin, k))
    return x, blocks, params, keep


@pytest.mark.gpu
@pytest.mark.parametrize("variant", ["auto", "tc_pair", "tc_sparse_ws"])
def test_encoder_equals_block_by_block_and_follows_the_oracle(lib, variant):
    # auto at this size: kernels without a residual epilogue, so every block hands its last add to the next LayerNorm;
    # tc_pair: every residual fused; tc_sparse_ws: proj and fc2 unfused, fc1's GELU fused
    dtype = torch.bfloat16
    images, tokens, heads, mlp = 3, 50, 2, 256
    sets = [SPARSE_LEVELS, {"qkv": (1, 8), "proj": (2, 8), "fc1": (1, 4), "fc2": (2, 4)}, SPARSE_LEVELS] if variant == "tc_sparse_ws" \
        else [MIXED_LEVELS, SPARSE_LEVELS, {"qkv": (2, 4), "proj": (8, 8), "fc1": (4, 8), "fc2": (1, 16)}]
    x, blocks, params, keep = _encoder_case(lib, dtype, images, tokens, heads, mlp, sets, 2000)
    code = {"auto": lib.VARIANT_AUTO, "tc_pair": lib.VARIANT_TC_PAIR, "tc_sparse_ws": lib.VARIANT_TC_SPARSE_WS}[variant]
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    fg = (synth.randn((64 * heads,), 31, 0.1, dtype).float() + 1.0).to(dtype).cuda()
    fb = synth.randn((64 * heads,), 32, 0.1, dtype).cuda()
    lib.elsa_set_linear_variant(code)
    try:
        cur = x.cuda()
        for w in blocks:
            cur, _ = lib.elsa_vit_block(cur, mlp, w, dev_status=status, tokens=tokens, heads=heads)
        table = lib.make_encoder_table(blocks)
        y_plain, _ = lib.elsa_vit_encoder(x.cuda(), tokens, heads, mlp, table, dev_status=status)
        y_norm, _ = lib.elsa_vit_encoder(x.cuda(), tokens, heads, mlp, table, final_gain=fg, final_bias=fb, dev_status=status)
        torch.cuda.synchronize()
    finally:
        lib.elsa_set_linear_variant(lib.VARIANT_AUTO)
    assert int(status.item()) == 0, "device status %#x" % int(status.item())
    assert torch.equal(y_plain.view(torch.int16), cur.view(torch.int16))         # bit for bit the block-by-block result
    # the final LayerNorm, from the library's own block output
    ref_norm = bo._round16(bo.layer_norm(cur.double().cpu().numpy(), fg.double().cpu().numpy(), fb.double().cpu().numpy(), 1e-6), dtype)
    err = np.abs(y_norm.double().cpu().numpy() - ref_norm)
    assert (err <= stage_tolerance(ref_norm, None, dtype)).all()
    # the oracle's chain of the same blocks
    bits = synth.bits(x)
    for p in params:
        out = bo.block_forward(bits, p, eo.BF16, eps=1e-6, attn="softmax", tokens=tokens, heads=heads)
        bits = bo._bits(out["y"], dtype)
    got = cur.double().cpu().numpy()
    assert np.linalg.norm(got - out["y"]) <= 1e-2 * np.linalg.norm(out["y"])     # three blocks of seven 16-bit stages each


@pytest.mark.gpu
def test_encoder_validates_every_block_before_launching(lib):
    dtype = torch.bfloat16
    x, blocks, params, keep = _encoder_case(lib, dtype, 2, 20, 1, 128, [MIXED_LEVELS, MIXED_LEVELS], 2500)
    blocks[1].fc2.idx = None
    before = lib.elsa_launch_count()
    with pytest.raises(lib.ElsaError) as e:
        lib.elsa_vit_encoder(x.cuda(), 20, 1, 128, lib.make_encoder_table(blocks))
    assert e.value.status == 1 and "block 1" in str(e.value)
    assert lib.elsa_launch_count() == before


WINDOW_CASES = [(2, 14, 14, 7, 0, 2, 32), (2, 14, 14, 7, 3, 2, 32), (1, 28, 14, 7, 3, 4, 32), (2, 14, 14, 7, 3, 1, 64),
                (3, 8, 8, 4, 2, 3, 32), (1, 16, 16, 16, 5, 2, 32)]


@pytest.mark.gpu
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float16], ids=["bf16", "f16"])
@pytest.mark.parametrize("case", WINDOW_CASES, ids=["%dx%dx%d_w%d_s%d_h%d_d%d" % c for c in WINDOW_CASES])
def test_window_attention_matches_oracle(lib, case, dtype):
    B, H, W, ws, shift, heads, d = case
    dim, T = heads * d, ws * ws
    qkv = synth.randn((B * H * W, 3 * dim), 23, 1.0, dtype)
    rel_bias = np.random.default_rng(7).standard_normal((heads, T, T)) * 0.5
    # the rows in window order: what the block's first LayerNorm writes
    order = bo.window_order(H, W, ws, shift)
    perm = np.concatenate([b * H * W + order.ravel() for b in range(B)])
    mask = bo.shift_mask(H, W, ws, shift) if shift else None
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    a_win = lib.elsa_window_attention(qkv[perm].contiguous().cuda(), T, heads,
                                      lib.pad_score_table(torch.from_numpy(rel_bias).float().cuda()),
                                      None if mask is None else lib.pad_score_table(torch.from_numpy(mask).float().cuda()),
                                      dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0, "device status %#x" % int(status.item())
    q64 = qkv.double().numpy()
    ref = bo._round16(bo.window_attention(q64, H, W, ws, shift, heads, rel_bias), dtype)[perm]
    got = a_win.double().cpu().numpy()
    assert np.isfinite(got).all()
    tol = attention_tolerance(ref, q64[perm][:, 2 * dim:], T, heads, dtype)
    err = np.abs(got - ref)
    worst = (err - tol).argmax()
    assert (err <= tol).all(), "error %g at tolerance %g" % (err.flat[worst], tol.flat[worst])


def test_swin_mask_is_the_oracles():
    from paper_2409_09708_b200 import build
    build.build()
    from paper_2409_09708_b200 import binding as lib
    for H, W, ws, shift in [(14, 14, 7, 3), (6, 9, 3, 1), (28, 14, 7, 3), (8, 8, 4, 2)]:
        got = lib.elsa_swin_mask(H, W, ws, shift, pitch=ws * ws).numpy()
        ref = bo.shift_mask(H, W, ws, shift).astype(np.float32)
        assert np.array_equal(got, ref)
        padded = lib.elsa_swin_mask(H, W, ws, shift, pitch=ws * ws + 7).numpy()
        assert np.array_equal(padded[:, :, :ws * ws], got) and (padded[:, :, ws * ws:] == 0).all()
        # two windows per item: the seam masks on the diagonal blocks, nothing (the bias table separates the windows) elsewhere
        T = ws * ws
        two = lib.elsa_swin_mask(H, W, ws, shift, pitch=2 * T, pack=2).numpy()
        assert two.shape == (ref.shape[0] // 2, 2 * T, 2 * T)
        assert np.array_equal(two[:, :T, :T], ref[0::2]) and np.array_equal(two[:, T:, T:], ref[1::2])
        assert (two[:, :T, T:] == 0).all() and (two[:, T:, :T] == 0).all()
    bias = torch.from_numpy(np.random.default_rng(1).standard_normal((3, 9, 9)).astype(np.float32))
    packed = lib.elsa_swin_pack_bias(bias, 3, pack=2, pitch=20).numpy()
    assert np.array_equal(packed[:, :9, :9], bias.numpy()) and np.array_equal(packed[:, 9:, 9:18], bias.numpy())
    assert (packed[:, :9, 9:18] == -30000).all() and (packed[:, 9:, :9] == -30000).all() and (packed[:, :, 18:] == 0).all()


SWIN_CASES = [(2, 14, 14, 7, 0, 2, 32), (2, 14, 14, 7, 3, 2, 32), (1, 28, 28, 7, 3, 4, 32), (2, 14, 14, 7, 3, 1, 64)]


@pytest.mark.gpu
@pytest.mark.parametrize("pack", [1, 2])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float16], ids=["bf16", "f16"])
@pytest.mark.parametrize("case", SWIN_CASES, ids=["%dx%dx%d_w%d_s%d_h%d_d%d" % c for c in SWIN_CASES])
def test_swin_block_matches_oracle(lib, case, dtype, pack):
    run_swin_case(lib, case, dtype, pack, MIXED_LEVELS)


# the grids, widths and head counts of Swin-B's stages 1, 3 and 4 (window 7; stage 4's grid is one window, so it is
# never shifted), a few images each: 64 window positions with their own masks, rows of 128 / 512 / 1024 values
SWIN_B_STAGE_CASES = [(4, 56, 56, 7, 3, 4, 32), (16, 14, 14, 7, 3, 16, 32), (32, 7, 7, 7, 0, 32, 32)]


@pytest.mark.gpu
@pytest.mark.parametrize("levels", [SPARSE_LEVELS, MIXED_LEVELS], ids=["sparse", "mixed"])
@pytest.mark.parametrize("case", SWIN_B_STAGE_CASES, ids=["%dx%dx%d_w%d_s%d_h%d_d%d" % c for c in SWIN_B_STAGE_CASES])
def test_swin_b_stage_shapes_match_oracle(lib, case, levels):
    run_swin_case(lib, case, torch.bfloat16, 1, levels)


def run_swin_case(lib, case, dtype, pack, levels):
    B, H, W, ws, shift, heads, d = case
    dim, T, mlp = heads * d, ws * ws, 4 * heads * d
    rows = B * H * W
    host, p = make_params(dim, mlp, levels, dtype, 3100)
    x = synth.randn((rows, dim), 14, 1.0, dtype)
    rel_bias = np.random.default_rng(9).standard_normal((heads, T, T)) * 0.5
    dev = {k: v.cuda() for k, v in host.items()}
    lin = {}
    for name in NAMES:
        N, M = levels[name]
        vals, idx = lib.elsa_nm_compress(dev["W_" + name], N, M)
        lin[name] = (vals, idx, dev["b_" + name], N, M)
    w, keep = lib.make_block_weights(dev["ln1_g"], dev["ln1_b"], dev["ln2_g"], dev["ln2_b"], lin, eps=1e-6)
    code = lib.dtype_code(dtype)
    total, off = lib.elsa_vit_block_scratch_bytes(rows, dim, mlp, w, code)
    scratch = torch.zeros(total, dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    mask = lib.elsa_swin_mask(H, W, ws, shift, pack=pack).cuda() if shift else None
    bias_table = lib.elsa_swin_pack_bias(torch.from_numpy(rel_bias), ws, pack=pack).cuda()
    y, _ = lib.elsa_swin_block(x.cuda(), H, W, ws, shift, heads, mlp, w, bias_table, mask, scratch=scratch, dev_status=status,
                               pack=pack)
    torch.cuda.synchronize()
    assert int(status.item()) == 0, "device status %#x" % int(status.item())
    cols = {"x1": dim, "qkv": 3 * dim, "a": dim, "x2": dim, "x3": dim, "h": mlp}
    got = {s: lib.block_region(scratch, off, s, rows, cols[s], dtype).cpu() for s in cols}
    got["y"] = y.cpu()
    # x1, qkv and a are stored in window order: bring them back to the grid's order for the comparison
    order = bo.window_order(H, W, ws, shift)
    perm = torch.from_numpy(np.concatenate([b * H * W + order.ravel() for b in range(B)]))
    for s in ("x1", "qkv", "a"):
        back = torch.empty_like(got[s])
        back[perm] = got[s]
        got[s] = back
    check_rows(got, x, p, dtype, np.arange(rows), attn=dict(H=H, W=W, ws=ws, shift=shift, heads=heads, rel_bias=rel_bias))
