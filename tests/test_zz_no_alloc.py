"""The allocation-free entry point, elsa_nm_linear_static, against elsa_nm_linear and the CPU oracle.

Some users of the library call it from places where device memory cannot be allocated (a
runtime plugin's enqueue hook, a process whose framework already owns all of the GPU's memory, a
loop that must not stall on an allocation).  For them the library keeps the scratch it needs in
a fixed built-in array.  This file checks, through the C ABI, that the variant returns what the
ordinary call returns -- on two calls in a row that share the array, the second with a different
and smaller weight so that leftovers of the first would show --, that both agree with the fp64
oracle within the parity tolerances, and that a weight too large for the array is refused with a
clear message instead of being run.

It is collected last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import numpy as np
import pytest
import torch

from oracle import elsa_oracle as eo
from paper_2409_09708_b200 import synth

pytestmark = pytest.mark.gpu

REL_FRO_TOL = 5e-3     # the tolerances of the parity tests
ELEM_TOL = 1e-2


@pytest.fixture(scope="module")
def lib():
    from paper_2409_09708_b200 import build
    build.build()
    from paper_2409_09708_b200 import binding
    return binding


def both_ways(lib, layer, dtype):
    """Y of the allocation-free call, Y of elsa_nm_linear forced onto the kernel the allocation-free call
    always uses (so that bit-equality does not hang on the dispatch rule), and the oracle on sampled rows."""
    X, W, b = synth.layer_tensors(layer, dtype, device="cuda")
    vals, idx = lib.elsa_nm_compress(W, layer.N, layer.M)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    lib.elsa_set_linear_variant(lib.VARIANT_TC_DENSE)
    try:
        Y_ref = lib.elsa_nm_linear(X, vals, idx, b, layer.out, layer.in_, layer.N, layer.M, dev_status=status)
    finally:
        lib.elsa_set_linear_variant(lib.VARIANT_AUTO)
    Y = torch.full((layer.rows, layer.out), float("nan"), dtype=dtype, device="cuda")   # caller-owned output
    lib.elsa_nm_linear_static(X, vals, idx, b, layer.out, layer.in_, layer.N, layer.M, Y, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    pick = synth.sample_rows(layer.rows, 64, layer.seed_x)
    code = eo.F16 if dtype == torch.float16 else eo.BF16
    ovals, oidx, _ = eo.nm_compress(synth.bits(W), layer.N, layer.M)
    ref = eo.nm_linear_f64(synth.bits(X.cpu()[torch.from_numpy(pick)]), ovals, oidx, synth.bits(b), layer.out, layer.in_,
                           layer.N, layer.M, code)
    got = Y.cpu()[torch.from_numpy(pick)].to(torch.float64).numpy()
    assert np.linalg.norm(got - ref) <= REL_FRO_TOL * np.linalg.norm(ref), layer.name
    assert np.max(np.abs(got - ref) / (np.abs(ref) + 1.0)) <= ELEM_TOL, layer.name
    return Y, Y_ref


def assert_within_tolerance(Y, Y_ref):
    got = Y.to(torch.float64).cpu().numpy()
    ref = Y_ref.to(torch.float64).cpu().numpy()
    assert np.isfinite(got).all()
    assert np.linalg.norm(got - ref) <= REL_FRO_TOL * np.linalg.norm(ref)
    assert np.max(np.abs(got - ref) / (np.abs(ref) + 1.0)) <= ELEM_TOL


def test_two_calls_in_a_row_match_the_workspace_entry_point(lib):
    first = synth.Layer("first", 1000, 1024, 768, 2, 8, 101, 102, 103)     # 1.5 MB image
    second = synth.Layer("second", 333, 256, 320, 3, 8, 104, 105, 106)     # smaller: sits inside the first's bytes
    for layer, dtype in ((first, torch.bfloat16), (second, torch.float16)):
        Y, Y_ref = both_ways(lib, layer, dtype)
        assert_within_tolerance(Y, Y_ref)
        assert torch.equal(Y, Y_ref)            # same kernels on the same image: identical, in fact


def test_dense_level_and_largest_supported_weight(lib):
    dense = synth.Layer("dense", 200, 512, 256, 8, 8, 111, 112, 113)        # N == M: no scratch involved
    Y, Y_ref = both_ways(lib, dense, torch.bfloat16)
    assert_within_tolerance(Y, Y_ref)
    full = synth.Layer("full", 256, 4096, 1024, 1, 16, 114, 115, 116)       # exactly the 8 MiB limit
    assert full.out * full.in_ * 2 == lib.STATIC_SCRATCH_BYTES
    Y, Y_ref = both_ways(lib, full, torch.float16)
    assert_within_tolerance(Y, Y_ref)


def test_weight_beyond_the_built_in_scratch_is_refused(lib):
    layer = synth.Layer("big", 64, 4096, 1032, 2, 8, 121, 122, 123)         # 8 rows past the limit
    X, W, b = synth.layer_tensors(layer, torch.bfloat16, device="cuda")
    vals, idx = lib.elsa_nm_compress(W, layer.N, layer.M)
    Y = torch.zeros((layer.rows, layer.out), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(lib.ElsaError) as err:
        lib.elsa_nm_linear_static(X, vals, idx, b, layer.out, layer.in_, layer.N, layer.M, Y)
    assert err.value.status == 6 and "exceeds the built-in scratch" in str(err.value)
    torch.cuda.synchronize()
    assert (Y == 0).all()                       # nothing was launched
