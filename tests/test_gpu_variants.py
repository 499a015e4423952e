"""Two test builds of the library (same sources, extra compile-time definitions; see build.VARIANTS).

shortwait: every bounded device wait gives up after about 3,000 cycles.  An ordinary contraction
then cannot finish its first tile in time: a wait runs out on a normal run, the kernel records which
one in the status word, drains what it has in flight and returns.  Nothing is provoked to hang.

bounds: every index a kernel gathers or scatters through is range-checked before use.  The parity
cases must give the same results and an untouched status word.
"""

import ctypes

import numpy as np
import pytest

from paper_2609_33645_b200 import workloads as wl
from tests import helpers as H

pytestmark = pytest.mark.gpu


def test_a_wait_that_runs_out_is_reported_and_the_kernel_returns(lib):
    import torch
    from paper_2609_33645_b200 import build
    short = lib.load_variant(build.build_variant("shortwait"))
    dev = torch.device("cuda:0")
    m, n, k = 256, 256, 8192                       # one tile for one pair of CTAs; 128 k-blocks: far beyond the limit
    g = torch.Generator(device="cpu").manual_seed(3)
    A = torch.randn(m, k, generator=g).to(torch.bfloat16).to(dev)
    B = torch.randn(n, k, generator=g).to(torch.bfloat16).to(dev)
    C = torch.zeros((m, n), dtype=torch.float32, device=dev)
    word = torch.zeros(64, dtype=torch.int32, device=dev)
    stream = ctypes.c_void_p(torch.cuda.current_stream(dev).cuda_stream)
    vp = ctypes.c_void_p
    st = short.pctc_gemm_bf16(vp(A.data_ptr()), vp(B.data_ptr()), vp(C.data_ptr()), m, n, k, 0, 0, 0,
                              vp(word.data_ptr()), stream)
    assert st == 0                                  # the launch itself is fine
    host = ctypes.c_int32(0)
    rc = short.pctc_workspace_status(vp(word.data_ptr()), stream, ctypes.byref(host))
    assert rc == 6 and short.pctc_status_string(rc) == b"bounded device wait gave up"
    assert host.value in (1, 2, 3, 4), host.value   # which wait gave up: producer, accumulator, operands, epilogue
    torch.cuda.synchronize()                        # the kernel has returned and the context is intact
    # the regular library computes the same product right afterwards
    got = lib.gemm_bf16(A, B, m, n, k).cpu().numpy().astype(np.float64)
    ref = A.float().cpu().numpy().astype(np.float64) @ B.float().cpu().numpy().astype(np.float64).T
    assert H.rel_fro(got, ref) < 1e-5


@pytest.mark.parametrize("case", ["bf16-tensor", "bf16-fma-bias", "fp32-beam", "excluded"])
def test_bounds_checked_build_gives_the_same_results_and_reports_nothing(lib, case):
    from paper_2609_33645_b200 import build
    chk = lib.load_variant(build.build_variant("bounds"))
    kw = {}
    if case == "bf16-tensor":
        batch = wl.make_batch(wl.reduced(wl.CONFIGS["c2"], name="b1", V=8192 + 40, N=6, T_div=4), permute_ids=True,
                              poison_padding=True)
        kw = dict(chunk=4096)
    elif case == "bf16-fma-bias":
        batch = wl.make_batch(wl.reduced(wl.CONFIGS["c3"], name="b2", V=5001, D=192, N=5, T_div=6, U_div=3, blank=4097),
                              with_bias=True, permute_ids=True)
        kw = dict(gemm_path=1, chunk=2048)
    elif case == "fp32-beam":
        import dataclasses
        batch = wl.make_batch(dataclasses.replace(wl.CONFIGS["c1"], name="b3", N=4, T_lo=30, T_hi=90, V=777, seed=5))
        kw = dict(beam=6.0)
    else:
        batch = wl.make_batch(wl.reduced(wl.CONFIGS["c2"], name="b4", V=4096, D=64, N=5, T_div=8, U_div=2))
        batch.targets[1, 0] = batch.blank                     # bad target
        batch.input_lengths[2] = 3                            # too few frames for its labels
        batch.targets[3, :4] = 9                              # repeated labels
    gpu = H.run_gpu(lib, batch, lib_handle=chk, check_status=True, **kw)
    regular = H.run_gpu(lib, batch, **kw)
    for k in ("loss", "dH", "dW", "subset", "relabeled", "flags"):
        np.testing.assert_array_equal(gpu[k], regular[k])
    ref = H.run_oracle(batch, beam=kw.get("beam"))
    H.assert_parity(gpu, ref, batch, tol=(1e-5, 5e-4) if case == "fp32-beam" else None)
