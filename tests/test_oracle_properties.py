"""Property tests of the oracle on random tiny problems (hypothesis): what must hold for ANY input,
checked on hundreds of drawn shapes, label sequences (repeats, empty targets, too few frames), blank
positions and beams.  A dropped term, a wrong sign or a wrong index in the recursions breaks one of them."""

import numpy as np
import pytest

hyp = pytest.importorskip("hypothesis")
from hypothesis import given, settings, strategies as st   # noqa: E402

from oracle import pruned_ctc_oracle as O   # noqa: E402


@st.composite
def problems(draw):
    V = draw(st.integers(2, 7))
    D = draw(st.integers(1, 4))
    N = draw(st.integers(1, 3))
    T = draw(st.integers(1, 7))
    blank = draw(st.integers(0, V - 1))
    seed = draw(st.integers(0, 2 ** 31 - 1))
    rng = np.random.default_rng(seed)
    labels = [v for v in range(V) if v != blank]
    Tn = [draw(st.integers(1, T)) for _ in range(N)]
    ys = [draw(st.lists(st.sampled_from(labels), min_size=0, max_size=4)) for _ in range(N)]
    stride = max(1, max(len(y) for y in ys))
    targets = np.full((N, stride), -1, dtype=np.int32)
    for n, y in enumerate(ys):
        targets[n, : len(y)] = y
    H = rng.standard_normal((N, T, D))
    W = rng.standard_normal((V, D))
    b = rng.standard_normal(V) if draw(st.booleans()) else None
    return dict(H=H, W=W, b=b, targets=targets, Tn=np.array(Tn, dtype=np.int32),
                tl=np.array([len(y) for y in ys], dtype=np.int32), blank=blank, ys=ys)


@settings(max_examples=150, deadline=None)
@given(problems())
def test_loss_gradient_and_exclusion_invariants(p):
    out = O.pruned_ctc_reference(p["H"], p["W"], p["b"], p["targets"], p["Tn"], p["tl"], p["blank"])
    N = p["H"].shape[0]
    for n in range(N):
        feasible = O.is_feasible(p["ys"][n], int(p["Tn"][n]))
        assert (out["flags"][n] == 0) == feasible
        if not feasible:
            assert out["loss"][n] == 0.0 and np.all(out["dH"][n] == 0.0)
        else:
            assert out["loss"][n] > 0.0                    # minus the log of a probability below one
        assert np.all(out["dH"][n, int(p["Tn"][n]):] == 0.0)
    # every frame's dlogits sum to zero (Section 3.2): so do the bias gradient and the columns of dW
    assert abs(out["db"].sum()) < 1e-10
    np.testing.assert_allclose(out["dW"].sum(axis=0), 0.0, atol=1e-10)
    # U: blank first, then strictly increasing, and it indexes back to the targets
    U = out["U"]
    assert U[0] == p["blank"] and np.all(np.diff(U[1:]) > 0)
    for n in range(N):
        for i in range(int(p["tl"][n])):
            assert U[out["relabeled"][n, i]] == p["targets"][n, i]


@settings(max_examples=80, deadline=None)
@given(problems())
def test_proposition_1_on_random_problems(p):
    full = O.pruned_ctc_reference(p["H"], p["W"], p["b"], p["targets"], p["Tn"], p["tl"], p["blank"])
    grouped = O.grouped_reference(p["H"], p["W"], p["b"], p["targets"], p["Tn"], p["tl"], p["blank"])
    np.testing.assert_allclose(grouped["loss"], full["loss"], rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(grouped["dH"], full["dH"], rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(grouped["dW"], full["dW"], rtol=1e-9, atol=1e-11)


@settings(max_examples=80, deadline=None)
@given(problems(), st.floats(0.05, 30.0))
def test_beam_bounds_on_random_problems(p, beam):
    exact = O.pruned_ctc_reference(p["H"], p["W"], p["b"], p["targets"], p["Tn"], p["tl"], p["blank"])
    pruned = O.pruned_ctc_reference(p["H"], p["W"], p["b"], p["targets"], p["Tn"], p["tl"], p["blank"], beam=beam)
    for n in range(p["H"].shape[0]):
        if exact["flags"][n] != 0:
            continue
        assert pruned["flags"][n] == 0                     # the best alignment always survives
        # the retained lattice is a subset of the alignments: L_beta >= L (Appendix B.3)
        assert pruned["loss"][n] >= exact["loss"][n] - 1e-10
        assert pruned["exact_loss"][n] == pytest.approx(exact["loss"][n], rel=1e-12)
    # still a gradient of a softmax minus a distribution: rows of dlogits sum to zero
    assert abs(pruned["db"].sum()) < 1e-10
    # a beam wider than any score gap prunes nothing
    wide = O.pruned_ctc_reference(p["H"], p["W"], p["b"], p["targets"], p["Tn"], p["tl"], p["blank"], beam=1e6)
    np.testing.assert_allclose(wide["loss"], exact["loss"], rtol=1e-12)
    np.testing.assert_allclose(wide["dW"], exact["dW"], rtol=1e-10, atol=1e-13)
