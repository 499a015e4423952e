"""Host-only checks of the C-ABI library: it builds, loads, exports every symbol
the header declares, validates arguments before touching a device, and its
workspace has no frames-by-vocabulary term."""

import ctypes
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    names = set()
    inc = os.path.join(ROOT, "include")
    for f in os.listdir(inc):
        if not f.endswith(".h"):
            continue
        text = open(os.path.join(inc, f)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        for m in re.finditer(r"\b(pctc_status_t|const char\*|int32_t)\s+(\w+)\s*\(", text):
            names.add(m.group(2))
    return names


def test_library_exports_every_declared_symbol(lib):
    cdll = lib.load()
    names = declared_functions()
    assert {"pruned_ctc_fwd_bwd", "pctc_workspace_bytes"} <= names
    for name in names:
        assert hasattr(cdll, name), name
    assert set(lib.EXPORTS) <= names


def test_status_strings(lib):
    assert lib.status_string(0) == "ok"
    assert "workspace" in lib.status_string(2)


def _prob(lib, **kw):
    d = dict(N=2, T=50, D=64, V=1000, dtype=lib.PCTC_FP32, blank_id=0, beam=0.0, chunk=0, target_stride=10,
             gemm_path=0)
    d.update(kw)
    return lib.make_problem(**d)


def test_workspace_has_no_M_times_V_term(lib):
    il, tl = [50, 40], [10, 3]
    small = lib.workspace_bytes(_prob(lib, V=100000, dtype=lib.PCTC_BF16), il, tl)
    big = lib.workspace_bytes(_prob(lib, V=200000, dtype=lib.PCTC_BF16), il, tl)
    # only the O(V) index tables grow: 4 bytes (class map) + 2 bits (bitmap, rank) per class
    assert 0 < big - small <= 100000 * 4.5 + 4096
    # and it is well below one fp32 [M, V] array
    assert big < 90 * 200000 * 4
    # beam adds the best-alignment arrays
    assert lib.workspace_bytes(_prob(lib, beam=8.0), il, tl) > lib.workspace_bytes(_prob(lib), il, tl)


@pytest.mark.parametrize("kw,il,want", [
    (dict(dtype=1), [50, 40], (1000, 1)),                           # fp32: 4,096, capped by V
    (dict(dtype=1, V=10000), [50, 40], (4096, 3)),
    (dict(dtype=0, D=512, V=180000), [50, 40], (56832, 4)),         # narrow head: 3 x 74 x 256 columns
    (dict(dtype=0, D=512, V=180000, N=2, T=6400), [6399, 1], (37888, 5)),      # c2's frame count: 2 x 74 x 256
    (dict(dtype=0, D=1024, V=151936, N=2, T=4470), [4469, 1], (56832, 3)),     # c3's
    (dict(dtype=0, D=512, V=180000, N=2, T=14000), [13999, 1], (18944, 10)),
    (dict(dtype=0, D=2048, V=180000), [50, 40], (16384, 11)),
    (dict(dtype=0, D=4096, V=151936), [50, 40], (16384, 10)),
    (dict(dtype=0, D=4096, V=151936, N=2, T=20000), [20000, 1], (8192, 19)),     # 512 MiB rule
    (dict(dtype=0, D=512, V=180000, N=2, T=16000), [16000, 1], (16384, 11)),   # [M, C] temporary <= 512 MiB
    (dict(dtype=0, D=512, V=180000, N=2, T=64000), [64000, 1], (8192, 22)),
    (dict(dtype=0, D=512, V=180000, chunk=1000), [50, 40], (1024, 176)),       # rounded up to the tile width
    (dict(dtype=0, D=512, V=180000, chunk=1000, gemm_path=1), [50, 40], (1000, 180)),
])
def test_chunk_width_default_and_rounding(lib, kw, il, want):
    assert lib.chunk_width(_prob(lib, **kw), il, [10, 3]) == want


@pytest.mark.parametrize("kw,il,tl", [
    (dict(N=0), [50, 50], [3, 3]),
    (dict(V=0), [50, 50], [3, 3]),
    (dict(blank_id=1000), [50, 50], [3, 3]),
    (dict(blank_id=-1), [50, 50], [3, 3]),
    (dict(), [51, 50], [3, 3]),       # T_n > T
    (dict(), [0, 50], [3, 3]),        # T_n = 0
    (dict(), [50, 50], [11, 3]),      # U_n > stride
    (dict(), [50, 50], [-1, 3]),
    (dict(dtype=7), [50, 50], [3, 3]),
    (dict(beam=float("nan")), [50, 50], [3, 3]),
    (dict(gemm_path=9), [50, 50], [3, 3]),
    (dict(target_stride=3000), [50, 50], [2500, 3]),   # trellis wider than the DP kernels cover
])
def test_invalid_problems_are_rejected_on_the_host(lib, kw, il, tl):
    with pytest.raises(lib.PctcError) as ei:
        lib.workspace_bytes(_prob(lib, **kw), il, tl)
    assert ei.value.status in (1, 3)


def test_fwd_bwd_rejects_null_and_short_workspace_before_any_launch(lib):
    cdll = lib.load()
    prob = _prob(lib)
    il = np.array([50, 40], dtype=np.int32)
    tl = np.array([10, 3], dtype=np.int32)
    p = lambda a: a.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))
    fake = ctypes.c_void_p(256 * 4096)      # non-null, aligned, never dereferenced on these paths
    args = [ctypes.byref(prob), fake, fake, None, fake, p(il), p(tl), fake, fake, fake, None,
            None, None, None, None, fake, ctypes.c_size_t(16), None]
    assert cdll.pruned_ctc_fwd_bwd(*args) == 2          # workspace too small
    args[1] = None
    assert cdll.pruned_ctc_fwd_bwd(*args) == 1          # null hidden
    assert cdll.pctc_gemm_bf16(None, fake, fake, 8, 8, 8, 0, 0, 0, None, None) == 1


def test_topk_workspace_query_validates_k_and_has_no_frames_by_vocabulary_term(lib):
    il = np.array([50, 40], dtype=np.int32)
    ptr = il.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))
    out = ctypes.c_size_t(0)
    cdll = lib.load()
    prob = _prob(lib, dtype=0, D=512, V=180000)
    for k in (0, 3, 5, 16, -1):
        assert cdll.pctc_topk_workspace_bytes(ctypes.byref(prob), ptr, k, ctypes.byref(out)) == 1
    sizes = []
    for V in (180000, 90000):
        p = _prob(lib, dtype=0, D=512, V=V)
        assert cdll.pctc_topk_workspace_bytes(ctypes.byref(p), ptr, 8, ctypes.byref(out)) == 0
        sizes.append(out.value)
    assert sizes[0] == sizes[1] < 90 * 180000          # one 4,096-column block of logits, whatever V
