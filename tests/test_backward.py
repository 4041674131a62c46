"""Backward pass of the masked linear (elsa_nm_linear_backward) against oracle/elsa_backward_oracle.py: every
output element by element at small sizes, sampled token rows (dX) and sampled output features (dW, db) at the
size of a DeiT-B layer.  Tolerances are the forward linear's: relative Frobenius error 5e-3 and
|err| <= 1e-2 * (|ref| + 1) per element; pruned positions of dW must be exact zeros."""
import numpy as np
import pytest
import torch

from oracle import elsa_backward_oracle as bwo
from oracle import elsa_oracle as eo
from paper_2409_09708_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def lib():
    from paper_2409_09708_b200 import build
    build.build()
    from paper_2409_09708_b200 import binding
    return binding


def check_close(got, ref):
    got = got.detach().to(torch.float64).cpu().numpy()
    assert np.isfinite(got).all()
    err = got - ref
    assert np.linalg.norm(err) <= 5e-3 * max(np.linalg.norm(ref), 1e-30)
    assert (np.abs(err) <= 1e-2 * (np.abs(ref) + 1.0)).all()


def run(lib, dY, X, W, N, M, want=("dX", "dW", "db"), variant=None):
    Wd = W.cuda()
    vals, idx = lib.elsa_nm_compress(Wd, N, M)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    if variant is not None:
        lib.elsa_set_linear_variant(variant)
    try:
        out = lib.elsa_nm_linear_backward(dY.cuda(), X.cuda(), vals, idx, W.shape[0], W.shape[1], N, M, want=want,
                                          dev_status=status)
        torch.cuda.synchronize()
    finally:
        lib.elsa_set_linear_variant(lib.VARIANT_AUTO)
    assert int(status.item()) == 0, "device status %#x" % int(status.item())
    return out


CASES = [(333, 256, 192, 2, 8), (70, 64, 40, 1, 4), (1000, 768, 768, 4, 8), (129, 128, 264, 8, 8), (200, 96, 64, 3, 16),
         (65, 24, 8, 3, 8), (5000, 768, 768, 1, 8)]     # the last: nine 256 x 256 tiles, so the rows are cut into eight uneven ranges


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float16], ids=["bf16", "f16"])
@pytest.mark.parametrize("case", CASES, ids=["%dx%dx%d_%d:%d" % c for c in CASES])
def test_backward_matches_oracle(lib, case, dtype):
    rows, in_, out, N, M = case
    code = eo.F16 if dtype == torch.float16 else eo.BF16
    X = synth.randn((rows, in_), 1, 1.0, dtype)
    W = synth.randn((out, in_), 2, 0.05, dtype)
    dY = synth.randn((rows, out), 3, 0.25, dtype)
    dX, dW, db = run(lib, dY, X, W, N, M)
    rX, rW, rb = bwo.linear_backward_f64(synth.bits(dY), synth.bits(X), synth.bits(W), N, M, code)
    check_close(dX, rX)
    check_close(dW, rW)
    check_close(db, rb)
    mask = eo.nm_mask(synth.bits(W), N, M)
    assert (synth.bits(dW)[mask == 0] == 0).all()                    # +0.0 bit patterns at the pruned positions


def test_each_output_alone_and_both_gemm_kernels(lib):
    dtype, code = torch.bfloat16, eo.BF16
    rows, in_, out, N, M = 520, 128, 256, 2, 8
    X = synth.randn((rows, in_), 4, 1.0, dtype)
    W = synth.randn((out, in_), 5, 0.05, dtype)
    dY = synth.randn((rows, out), 6, 0.25, dtype)
    rX, rW, rb = bwo.linear_backward_f64(synth.bits(dY), synth.bits(X), synth.bits(W), N, M, code)
    for variant in (lib.VARIANT_TC_DENSE, lib.VARIANT_TC_PAIR):
        dX, dW, db = run(lib, dY, X, W, N, M, variant=variant)
        check_close(dX, rX), check_close(dW, rW), check_close(db, rb)
    dX, dW, db = run(lib, dY, X, W, N, M, want=("dX",))
    assert dW is None and db is None
    check_close(dX, rX)
    dX, dW, db = run(lib, dY, X, W, N, M, want=("db",))
    check_close(db, rb)
    dX, dW, db = run(lib, dY, X, W, N, M, want=("dW",))
    check_close(dW, rW)


def test_integer_inputs_are_exact(lib):
    # small integers: every product and sum is exact in fp32 and representable in bf16
    rng = np.random.default_rng(1)
    dtype, code = torch.bfloat16, eo.BF16
    rows, in_, out, N, M = 96, 64, 48, 2, 4
    X = torch.from_numpy(rng.integers(-2, 3, (rows, in_)).astype(np.float32)).to(dtype)
    W = torch.from_numpy(rng.integers(-3, 4, (out, in_)).astype(np.float32)).to(dtype)
    dY = torch.from_numpy(rng.integers(-1, 2, (rows, out)).astype(np.float32)).to(dtype)
    dX, dW, db = run(lib, dY, X, W, N, M)
    rX, rW, rb = bwo.linear_backward_f64(synth.bits(dY), synth.bits(X), synth.bits(W), N, M, code)
    assert np.array_equal(dX.double().cpu().numpy(), rX)
    assert np.array_equal(dW.double().cpu().numpy(), rW)
    assert np.array_equal(db.double().cpu().numpy(), rb)


def test_deit_b_fc1_full_size_sampled(lib):
    dtype, code = torch.bfloat16, eo.BF16
    rows, in_, out, N, M = 256 * 197, 768, 3072, 2, 8
    X = synth.randn((rows, in_), 7, 1.0, dtype, "cuda").cpu()
    W = synth.randn((out, in_), 8, 0.02, dtype)
    dY = synth.randn((rows, out), 9, 0.05, dtype, "cuda").cpu()
    dX, dW, db = run(lib, dY, X, W, N, M)
    rng = np.random.default_rng(2)
    pick_r = np.unique(np.concatenate([[0, 255, 256, rows - 1], rng.integers(0, rows, 28)]))
    rX, _, _ = bwo.linear_backward_f64(synth.bits(dY[pick_r].contiguous()), synth.bits(X[pick_r].contiguous()), synth.bits(W), N, M, code)
    check_close(dX.cpu()[pick_r], rX)
    pick_o = np.unique(np.concatenate([[0, 127, 128, 255, 256, out - 1], rng.integers(0, out, 10)]))
    _, rW, rb = bwo.linear_backward_f64(synth.bits(dY[:, pick_o].contiguous()), synth.bits(X), synth.bits(W[pick_o].contiguous()), N, M, code)
    check_close(dW.cpu()[pick_o], rW)
    check_close(db.cpu()[pick_o], rb)


def test_backward_validation(lib):
    dtype = torch.bfloat16
    X = synth.randn((64, 64), 1, 1.0, dtype).cuda()
    W = synth.randn((32, 64), 2, 0.1, dtype).cuda()
    dY = synth.randn((64, 32), 3, 1.0, dtype).cuda()
    vals, idx = lib.elsa_nm_compress(W, 2, 8)
    with pytest.raises(lib.ElsaError) as e:
        lib.elsa_nm_linear_backward(dY, X, vals, idx, 32, 64, 2, 8, workspace=torch.empty(256, dtype=torch.uint8, device="cuda"))
    assert e.value.status == 6
    with pytest.raises(lib.ElsaError) as e:
        lib.elsa_nm_linear_backward(dY, None, vals, idx, 32, 64, 2, 8)
    assert e.value.status == 1
    with pytest.raises(lib.ElsaError) as e:
        lib.elsa_nm_linear_backward(dY, X, vals, None, 32, 64, 2, 8)
    assert e.value.status == 1
