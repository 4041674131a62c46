"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the
header declares, sizes follow the closed forms, and bad arguments are refused before any launch."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "elsa.h")


@pytest.fixture(scope="module")
def lib():
    from paper_2409_09708_b200 import build
    build.build()
    from paper_2409_09708_b200 import binding
    return binding


def declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(elsa_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert {"elsa_nm_compress", "elsa_nm_unpack", "elsa_nm_linear", "elsa_vit_linears",
            "elsa_vit_linears_host", "elsa_last_error"} <= set(names)
    cdll = ctypes.CDLL(lib.LIB_PATH)
    for n in names:
        assert hasattr(cdll, n), n


def test_packed_sizes_follow_the_closed_form(lib):
    # Sec. 1: N of every M values kept, log2(M) index bits each; rows start on a word boundary
    for out, in_, N, M, b in [(768, 768, 4, 8, 3), (768, 768, 2, 8, 3), (3072, 768, 1, 8, 3), (128, 512, 1, 4, 2),
                              (1024, 4096, 2, 16, 4), (16, 24, 3, 8, 3), (8, 368, 1, 16, 4)]:
        assert lib.elsa_nm_values_bytes(out, in_, N, M) == out * (in_ // M) * N * 2
        assert lib.elsa_nm_index_bytes(out, in_, N, M) == out * (-(-(in_ // M * N * b) // 32)) * 4
    assert lib.elsa_nm_index_bytes(768, 768, 8, 8) == 0
    assert lib.elsa_nm_values_bytes(768, 768, 8, 8) == 768 * 768 * 2
    # 768 x 768 at 4:8: 590 KB of values + 110 KB of indices against 1.18 MB dense
    assert lib.elsa_nm_values_bytes(768, 768, 4, 8) == 589824 and lib.elsa_nm_index_bytes(768, 768, 4, 8) == 110592
    assert lib.elsa_nm_values_bytes(768, 770, 4, 8) == 0          # invalid -> 0
    assert lib.elsa_workspace_bytes(197, 768, 768, 8, 8) == 0
    assert lib.elsa_workspace_bytes(197, 768, 768, 4, 8) >= 768 * 768 * 2


FAKE = 0x10000  # a non-NULL, 16-byte aligned value that is never dereferenced: validation fails first


def test_compress_argument_errors(lib):
    c = lib._compress
    assert c(None, 8, 8, 2, 4, 0, FAKE, FAKE, None) == 1                       # NULL W
    assert c(FAKE, 8, 8, 2, 4, 0, FAKE, None, None) == 1                       # NULL idx with N < M
    assert c(FAKE, 0, 8, 2, 4, 0, FAKE, FAKE, None) == 2                       # out <= 0
    assert c(FAKE, 8, 24, 2, 16, 0, FAKE, FAKE, None) == 2                     # in % M != 0
    assert c(FAKE, 8, 8, 2, 5, 0, FAKE, FAKE, None) == 3                       # M unsupported
    assert c(FAKE, 8, 8, 5, 4, 0, FAKE, FAKE, None) == 3                       # N > M
    assert c(FAKE, 8, 8, 0, 4, 0, FAKE, FAKE, None) == 3                       # N < 1
    assert c(FAKE, 8, 8, 2, 4, 7, FAKE, FAKE, None) == 4                       # dtype
    assert c(FAKE + 2, 8, 8, 2, 4, 0, FAKE, FAKE, None) == 5                   # misaligned W
    assert c(FAKE, 8, 12, 2, 4, 0, FAKE, FAKE, None) == 5                      # in % 8 != 0
    assert "multiple" in lib.elsa_last_error()


def test_linear_argument_errors(lib):
    f = lib._linear
    ok = dict(X=FAKE, rows=4, vals=FAKE, idx=FAKE, bias=None, out=8, in_=8, N=2, M=4, dt=0, Y=FAKE, ws=0x20000,
              wsb=1 << 20, st=None, stream=None)

    def call(**kw):
        a = dict(ok, **kw)
        return f(a["X"], a["rows"], a["vals"], a["idx"], a["bias"], a["out"], a["in_"], a["N"], a["M"], a["dt"],
                 a["Y"], a["ws"], a["wsb"], a["st"], a["stream"])

    assert call(X=None) == 1 and call(Y=None) == 1 and call(vals=None) == 1 and call(idx=None) == 1
    assert call(rows=0) == 2 and call(in_=6) in (2, 5) and call(in_=24, M=16, N=2) == 2
    assert call(M=3) == 3 and call(N=9, M=8) == 3
    assert call(dt=2) == 4
    assert call(Y=FAKE + 8) == 5 and call(out=12) == 5 and call(ws=0x20010) == 5
    assert call(ws=None) == 6 and call(wsb=16) == 6
    assert "workspace" in lib.elsa_last_error()


def test_vit_linears_reports_the_layer(lib):
    table = (lib.ElsaLayer * 2)()
    for t in table:
        t.X, t.Y, t.vals, t.idx, t.bias = FAKE, FAKE, FAKE, FAKE, None
        t.rows, t.in_, t.out, t.N, t.M = 4, 8, 8, 2, 4
    table[1].M = 7
    assert lib._vit(table, 2, 0, 0x20000, 1 << 20, None, None) == 3
    assert lib.elsa_last_error().startswith("layer 1:")
    assert lib._vit(None, 2, 0, 0x20000, 1 << 20, None, None) == 1
    assert lib._vit(table, 0, 0, 0x20000, 1 << 20, None, None) == 2
    assert lib.elsa_vit_workspace_bytes(table, 0) == lib.elsa_workspace_bytes(4, 8, 8, 2, 4)


def test_vit_compress_reports_the_weight(lib):
    table = (lib.ElsaWeight * 3)()
    for t in table:
        t.W, t.vals, t.idx = FAKE, FAKE, FAKE
        t.out, t.in_, t.N, t.M = 8, 16, 2, 8
    table[2].in_ = 20                                       # not a multiple of M
    assert lib._vit_compress(table, 3, 0, None) == 2
    assert lib.elsa_last_error().startswith("weight 2:")
    table[2].in_ = 16
    table[1].idx = None
    assert lib._vit_compress(table, 3, 0, None) == 1 and lib.elsa_last_error().startswith("weight 1:")
    assert lib._vit_compress(None, 3, 0, None) == 1
    assert lib._vit_compress(table, 0, 0, None) == 2


def test_supernet_side_entry_points_validate_their_arguments(lib):
    import ctypes
    n = 2
    Ns = (ctypes.c_int * n)(1, 2)
    vals = (ctypes.c_void_p * n)(FAKE, FAKE)
    idx = (ctypes.c_void_p * n)(FAKE, FAKE)
    f = lib._compress_levels
    assert f(None, 8, 16, 8, Ns, n, 0, vals, idx, None) == 1
    assert f(FAKE, 8, 16, 8, Ns, 0, 0, vals, idx, None) == 2
    assert f(FAKE, 8, 16, 8, Ns, 17, 0, vals, idx, None) == 2
    assert f(FAKE, 8, 20, 8, Ns, n, 0, vals, idx, None) == 2 and lib.elsa_last_error().startswith("level 0:")
    bad = (ctypes.c_int * n)(1, 9)
    assert f(FAKE, 8, 16, 8, bad, n, 0, vals, idx, None) == 3 and lib.elsa_last_error().startswith("level 1:")
    noidx = (ctypes.c_void_p * n)(FAKE, None)
    assert f(FAKE, 8, 16, 8, Ns, n, 0, vals, noidx, None) == 1
    g = lib._linear_masked
    assert g(FAKE, 4, None, None, 8, 8, 2, 4, 0, FAKE, 0x20000, 1 << 20, None, None) == 1
    assert g(FAKE, 4, FAKE, None, 8, 8, 5, 4, 0, FAKE, 0x20000, 1 << 20, None, None) == 3
    assert g(FAKE, 4, FAKE, None, 8, 8, 2, 4, 0, FAKE, None, 0, None, None) == 6


def test_variant_switch_and_launch_counter(lib):
    assert lib.elsa_get_linear_variant() == lib.VARIANT_AUTO
    lib.elsa_set_linear_variant(lib.VARIANT_SIMT)
    assert lib.elsa_get_linear_variant() == lib.VARIANT_SIMT
    lib.elsa_set_linear_variant(lib.VARIANT_AUTO)
    with pytest.raises(lib.ElsaError):
        lib.elsa_set_linear_variant(17)
    assert lib.elsa_launch_count() >= 0


def test_binding_module_refuses_to_import_without_the_library(tmp_path):
    """No fallback: with no libelsa.so beside it the binding raises instead of degrading."""
    import shutil
    import subprocess
    import sys
    pkg = tmp_path / "paper_2409_09708_b200"
    pkg.mkdir()
    src = os.path.join(ROOT, "paper_2409_09708_b200")
    for f in ("__init__.py", "binding.py", "synth.py"):
        shutil.copy(os.path.join(src, f), pkg / f)
    r = subprocess.run([sys.executable, "-c", "import paper_2409_09708_b200.binding"], cwd=tmp_path,
                       capture_output=True, text=True)
    assert r.returncode != 0 and "libelsa.so is missing" in r.stderr
