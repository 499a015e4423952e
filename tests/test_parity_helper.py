"""The parity helper must not be able to miss a wrong part of a gradient.

The whole-matrix Frobenius norm of dW is dominated by the K selected rows (they carry the occupancy
term of Eq. "grad-full"); the other rows, i.e. the dense softmax term, are a few percent of it, so a
dead tile there would pass a whole-matrix check at the 1e-2 tolerance.  These CPU tests feed
`assert_parity` the oracle's own outputs, rounded to bf16 the way the library rounds them, with one
defect planted, and require a failure for every defect (and a pass without one)."""

import copy

import ml_dtypes
import numpy as np
import pytest

from paper_2609_33645_b200 import workloads as wl
from tests import helpers as H


def _bf16(x):
    return np.asarray(x, dtype=np.float32).astype(ml_dtypes.bfloat16).astype(np.float64)


@pytest.fixture(scope="module")
def case():
    cfg = wl.reduced(wl.CONFIGS["c2"], name="c2-small", V=8192, N=6, T_div=4)     # the shape of test_bf16_reduced_configs
    batch = wl.make_batch(cfg, permute_ids=True, with_bias=True)
    ref = H.run_oracle(batch)
    gpu = dict(K=np.array([ref["K"]]), subset=np.asarray(ref["U"]).copy(), relabeled=ref["relabeled"].copy(),
               flags=ref["flags"].copy(), loss=ref["loss"].astype(np.float32),
               dH=_bf16(ref["dH"]), dW=_bf16(ref["dW"]), dbias=_bf16(ref["db"]))
    return batch, ref, gpu


def test_faithful_outputs_pass(case):
    batch, ref, gpu = case
    errs = H.assert_parity(gpu, ref, batch)
    assert errs["dW"] < 5e-3 and errs["dW off-support"] < 5e-3


def _off_support_rows(ref, V, lo, hi):
    off = np.ones(V, dtype=bool)
    off[np.asarray(ref["U"], dtype=np.int64)] = False
    rows = np.arange(lo, hi)
    return rows[off[lo:hi]]


def test_a_dead_tile_of_the_dense_term_is_caught(case):
    batch, ref, gpu = case
    V = batch.cfg.V
    bad = copy.deepcopy(gpu)
    bad["dW"][_off_support_rows(ref, V, V - 256, V)] = 0.0
    # the whole-matrix error of this defect is under the tolerance: that is the blind spot
    assert H.rel_fro(bad["dW"], ref["dW"]) < 1e-2
    with pytest.raises(AssertionError):
        H.assert_parity(bad, ref, batch)


def test_a_dead_column_block_of_dH_is_caught(case):
    batch, ref, gpu = case
    bad = copy.deepcopy(gpu)
    bad["dH"][:, :, 256:288] = 0.0            # 32 of 512 columns: 6% of the entries
    with pytest.raises(AssertionError):
        H.assert_parity(bad, ref, batch)


def test_one_utterance_scaled_by_two_percent_is_caught(case):
    batch, ref, gpu = case
    bad = copy.deepcopy(gpu)
    n = int(np.argmin(batch.input_lengths))   # the shortest utterance weighs least in the whole-tensor norm
    bad["dH"][n] *= 1.02
    assert H.rel_fro(bad["dH"], ref["dH"]) < 1e-2
    with pytest.raises(AssertionError):
        H.assert_parity(bad, ref, batch)


def test_a_dead_stretch_of_dbias_is_caught(case):
    batch, ref, gpu = case
    V = batch.cfg.V
    bad = copy.deepcopy(gpu)
    bad["dbias"][_off_support_rows(ref, V, 4096, 4096 + 256)] = 0.0
    with pytest.raises(AssertionError):
        H.assert_parity(bad, ref, batch)


def test_a_wrong_selected_row_is_caught(case):
    batch, ref, gpu = case
    bad = copy.deepcopy(gpu)
    j = int(ref["U"][ref["K"] // 2])
    bad["dW"][j] *= 1.5                       # one row of the occupancy term
    with pytest.raises(AssertionError):
        H.assert_parity(bad, ref, batch)
