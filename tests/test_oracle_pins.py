"""Pins for the float64 oracle: each test checks it against something fixed by
the paper or by mathematics, not against itself."""

import itertools
import math

import numpy as np
import pytest

from oracle import pruned_ctc_oracle as O


def collapse(path, blank):
    """The map B of Section 3.1: merge repeats, then drop blanks."""
    out = []
    prev = None
    for p in path:
        if p != prev and p != blank:
            out.append(p)
        prev = p
    return out


def brute_force(logp, y, blank):
    """Sum over every label sequence in V^T that collapses to y (Eq. "ctc")."""
    T, V = logp.shape
    total = 0.0
    occ = np.zeros((T, V))
    for path in itertools.product(range(V), repeat=T):
        if collapse(path, blank) != list(y):
            continue
        p = math.exp(sum(logp[t, v] for t, v in enumerate(path)))
        total += p
        for t, v in enumerate(path):
            occ[t, v] += p
    return total, occ


def random_logp(rng, T, V):
    Z = rng.standard_normal((T, V)) * 1.5
    return Z - O.log_normalizer(Z)[:, None], Z


@pytest.mark.parametrize("y,blank", [([1, 2], 0), ([2, 2], 0), ([3, 1], 4), ([1], 0), ([], 0), ([1, 1, 1], 0)])
def test_loss_and_occupancy_match_brute_force(y, blank):
    rng = np.random.default_rng(7)
    T, V = 6, 5
    logp, _ = random_logp(rng, T, V)
    loss, gamma, flags, exact = O.ctc_occupancy(logp, y, blank)
    total, occ = brute_force(logp, y, blank)
    if total == 0.0:
        assert flags == O.FLAG_INFEASIBLE and loss == 0.0 and gamma is None
        return
    assert flags == 0
    assert loss == pytest.approx(-math.log(total), rel=1e-12)
    np.testing.assert_allclose(gamma, occ / total, atol=1e-12)
    assert exact == loss


def test_alignment_counts_by_enumeration():
    # distinct pair on T=6 has 70 alignments over {blank, a, b}; a repeated pair has 35
    for y, expect in (([1, 2], 70), ([1, 1], 35)):
        n = sum(1 for p in itertools.product(range(3), repeat=6) if collapse(p, 0) == y)
        assert n == expect
        assert n == math.comb(6 + 2 - O.adjacent_repeats(y), 4)


@pytest.mark.parametrize("T,y", [(6, [1, 2]), (6, [2, 2]), (9, [1, 1, 2, 3, 3]), (5, []), (12, [4, 4, 4]),
                                 (4, [1, 1, 1])])
def test_equal_logits_closed_form(T, y):
    # with all logits equal every alignment has probability V^-T, so
    # loss = T log V - log(#alignments), #alignments = C(T + U - r, 2U)
    V, D = 7, 3
    H = np.zeros((1, T, D))
    W = np.ones((V, D))
    targets = np.array([y + [0] * (6 - len(y))], dtype=np.int32)
    out = O.pruned_ctc_reference(H, W, None, targets, [T], [len(y)], blank=0)
    r = O.adjacent_repeats(y)
    count = math.comb(T + len(y) - r, 2 * len(y)) if T >= len(y) + r else 0
    if count == 0:
        assert out["loss"][0] == 0.0 and out["flags"][0] == O.FLAG_INFEASIBLE
        assert np.all(out["dW"] == 0) and np.all(out["dH"] == 0)
    else:
        assert out["loss"][0] == pytest.approx(T * math.log(V) - math.log(count), rel=1e-13)


def test_single_alignment_and_empty_target():
    rng = np.random.default_rng(3)
    logp, _ = random_logp(rng, 5, 6)
    # T = U + r: exactly one alignment (1, blank, 1, 2, 3)
    y = [1, 1, 2, 3]
    loss, gamma, _, _ = O.ctc_occupancy(logp, y, 0)
    path = [1, 0, 1, 2, 3]
    assert loss == pytest.approx(-sum(logp[t, v] for t, v in enumerate(path)), rel=1e-13)
    expect = np.zeros_like(logp)
    for t, v in enumerate(path):
        expect[t, v] = 1.0
    np.testing.assert_allclose(gamma, expect, atol=1e-13)
    # U = 0: only the all-blank alignment
    loss0, gamma0, _, _ = O.ctc_occupancy(logp, [], 2)
    assert loss0 == pytest.approx(-logp[:, 2].sum(), rel=1e-13)
    assert np.allclose(gamma0[:, 2], 1.0) and np.allclose(np.delete(gamma0, 2, axis=1), 0.0)
    # one frame short: infeasible
    assert O.ctc_occupancy(logp[:4], y, 0)[2] == O.FLAG_INFEASIBLE


def _small_batch(rng, N=3, T=9, D=5, V=11, blank=0, with_bias=True):
    Tn = np.array([T, T - 2, T - 4][:N], dtype=np.int32)
    tl = np.array([3, 2, 4][:N], dtype=np.int32)
    targets = np.zeros((N, 4), dtype=np.int32)
    for n in range(N):
        toks = rng.integers(0, V - 1, size=4)
        toks = np.where(toks >= blank, toks + 1, toks)      # skip the blank id
        targets[n] = toks
    targets[0, 1] = targets[0, 0]                            # an adjacent repeat
    H = rng.standard_normal((N, T, D))
    W = rng.standard_normal((V, D)) * 0.7
    b = rng.standard_normal(V) * 0.3 if with_bias else None
    return H, W, b, targets, Tn, tl


@pytest.mark.parametrize("blank", [0, 4])
def test_matches_torch_ctc_loss_and_autograd(blank):
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(11)
    H, W, b, targets, Tn, tl = _small_batch(rng, blank=blank)
    out = O.pruned_ctc_reference(H, W, b, targets, Tn, tl, blank)
    Ht = torch.tensor(H, dtype=torch.float64, requires_grad=True)
    Wt = torch.tensor(W, dtype=torch.float64, requires_grad=True)
    bt = torch.tensor(b, dtype=torch.float64, requires_grad=True)
    logp = torch.log_softmax(Ht @ Wt.T + bt, dim=-1)          # [N,T,V]
    losses = torch.nn.functional.ctc_loss(
        logp.transpose(0, 1), torch.tensor(targets, dtype=torch.long), torch.tensor(Tn, dtype=torch.long),
        torch.tensor(tl, dtype=torch.long), blank=blank, reduction="none", zero_infinity=True)
    losses.sum().backward()
    np.testing.assert_allclose(out["loss"], losses.detach().numpy(), rtol=1e-12)
    np.testing.assert_allclose(out["dH"], Ht.grad.numpy(), atol=1e-11)
    np.testing.assert_allclose(out["dW"], Wt.grad.numpy(), atol=1e-11)
    np.testing.assert_allclose(out["db"], bt.grad.numpy(), atol=1e-11)


def test_gradients_match_finite_differences():
    rng = np.random.default_rng(5)
    H, W, b, targets, Tn, tl = _small_batch(rng, N=2, T=7, D=4, V=9, blank=2)
    out = O.pruned_ctc_reference(H, W, b, targets, Tn, tl, 2)

    def total(Hx, Wx, bx):
        return O.pruned_ctc_reference(Hx, Wx, bx, targets, Tn, tl, 2, want_dW=False)["loss"].sum()

    h = 1e-6
    for arr, grad, which in ((H, out["dH"], 0), (W, out["dW"], 1), (b, out["db"], 2)):
        idxs = [tuple(rng.integers(0, s) for s in arr.shape) for _ in range(12)]
        if which == 0:
            idxs.append((1, 6, 0))          # a padded frame of utterance 1 (T_1 = 5)
        for idx in idxs:
            plus, minus = arr.copy(), arr.copy()
            plus[idx] += h
            minus[idx] -= h
            args_p = [H, W, b]
            args_m = [H, W, b]
            args_p[which], args_m[which] = plus, minus
            fd = (total(*args_p) - total(*args_m)) / (2 * h)
            assert grad[idx] == pytest.approx(fd, rel=2e-6, abs=2e-8)


def test_utterance_weights_are_upstream_gradients():
    # gradients of sum_n c_n L_n by central differences; losses stay unweighted
    rng = np.random.default_rng(6)
    H, W, b, targets, Tn, tl = _small_batch(rng, N=3, T=8, D=4, V=9, blank=0)
    c = np.array([0.5, -1.25, 3.0])
    out = O.pruned_ctc_reference(H, W, b, targets, Tn, tl, 0, utt_weights=c)
    plain = O.pruned_ctc_reference(H, W, b, targets, Tn, tl, 0)
    np.testing.assert_array_equal(out["loss"], plain["loss"])

    def total(Wx):
        return float(np.dot(c, O.pruned_ctc_reference(H, Wx, b, targets, Tn, tl, 0, want_dW=False)["loss"]))

    h = 1e-6
    for idx in [(0, 0), (3, 2), (8, 1), (5, 3)]:
        p, m = W.copy(), W.copy()
        p[idx] += h
        m[idx] -= h
        assert out["dW"][idx] == pytest.approx((total(p) - total(m)) / (2 * h), rel=2e-6, abs=2e-8)
    for n in range(3):
        np.testing.assert_allclose(out["dH"][n], c[n] * plain["dH"][n], rtol=1e-13, atol=1e-15)


def test_invariants_and_exclusions():
    rng = np.random.default_rng(9)
    H, W, b, targets, Tn, tl = _small_batch(rng, N=3, T=9, D=5, V=11)
    # make utterance 2 infeasible: 4 labels incl. repeats on 5 frames
    targets[2] = [3, 3, 3, 3]
    out = O.pruned_ctc_reference(H, W, b, targets, Tn, tl, 0)
    assert list(out["flags"]) == [0, 0, O.FLAG_INFEASIBLE]
    assert out["loss"][2] == 0.0 and np.all(out["dH"][2] == 0.0)
    for n in range(2):
        assert np.all(out["dH"][n, Tn[n]:] == 0.0)
    # every valid row of dZ sums to zero => db sums to zero; occupancies are distributions
    assert abs(out["db"].sum()) < 1e-12
    Z = O.head_logits(H[0, :Tn[0]], W, b)
    logp = Z - O.log_normalizer(Z)[:, None]
    np.testing.assert_allclose(np.exp(logp).sum(1), 1.0, atol=1e-13)
    _, gamma, _, _ = O.ctc_occupancy(logp, list(targets[0, :tl[0]]), 0)
    np.testing.assert_allclose(gamma.sum(1), 1.0, atol=1e-12)
    assert gamma.min() >= 0.0
    # shift invariance: a constant added to every bias entry changes nothing
    out2 = O.pruned_ctc_reference(H, W, b + 3.25, targets, Tn, tl, 0)
    np.testing.assert_allclose(out2["loss"], out["loss"], rtol=1e-12)
    np.testing.assert_allclose(out2["dW"], out["dW"], atol=1e-12)
    # infeasible utterances still contribute their labels to U
    assert 3 in out["U"]


def test_log_normalizer_against_scipy():
    sp = pytest.importorskip("scipy.special")
    rng = np.random.default_rng(2)
    Z = rng.standard_normal((17, 301)) * 20
    np.testing.assert_allclose(O.log_normalizer(Z), sp.logsumexp(Z, axis=1), rtol=1e-14)
    a, b = rng.standard_normal(9), rng.standard_normal(9)
    np.testing.assert_allclose(O.lse(a, b, np.full(9, -np.inf)), np.logaddexp(a, b), rtol=1e-14)
    assert np.all(np.isneginf(O.lse(np.full(3, -np.inf), np.full(3, -np.inf))))


@pytest.mark.parametrize("blank", [0, 5])
def test_proposition_1_grouped_equals_full(blank):
    rng = np.random.default_rng(13)
    H, W, b, targets, Tn, tl = _small_batch(rng, N=3, T=10, D=6, V=23, blank=blank)
    full = O.pruned_ctc_reference(H, W, b, targets, Tn, tl, blank)
    grp = O.grouped_reference(H, W, b, targets, Tn, tl, blank)
    np.testing.assert_allclose(grp["loss"], full["loss"], rtol=1e-12)
    for k in ("dH", "dW", "db"):
        np.testing.assert_allclose(grp[k], full[k], atol=1e-12)


def test_proposition_1_empty_complement():
    rng = np.random.default_rng(14)
    V = 4
    H = rng.standard_normal((1, 8, 3))
    W = rng.standard_normal((V, 3))
    targets = np.array([[1, 2, 3, 1]], dtype=np.int32)
    full = O.pruned_ctc_reference(H, W, None, targets, [8], [4], 0)
    grp = O.grouped_reference(H, W, None, targets, [8], [4], 0)
    assert grp["K"] == V
    np.testing.assert_allclose(grp["loss"], full["loss"], rtol=1e-12)
    np.testing.assert_allclose(grp["dW"], full["dW"], atol=1e-12)


def test_subset_definition():
    rng = np.random.default_rng(21)
    V, blank = 50, 7
    tl = np.array([5, 0, 9, 3], dtype=np.int32)
    targets = rng.integers(0, V, size=(4, 9)).astype(np.int32)
    targets[targets == blank] = 8
    U, rel, bad = O.subset_and_relabel(targets, tl, blank, V)
    used = np.concatenate([targets[n, :tl[n]] for n in range(4)])
    assert U[0] == blank
    np.testing.assert_array_equal(U[1:], np.unique(used))
    assert np.all(np.diff(U[1:]) > 0)
    assert not bad.any()
    for n in range(4):
        np.testing.assert_array_equal(U[rel[n, :tl[n]]], targets[n, :tl[n]])
        assert np.all(rel[n, :tl[n]] >= 1) and np.all(rel[n, tl[n]:] == -1)
    assert len(U) <= 1 + tl.sum()
    # bad targets: blank inside a target, id out of range
    targets[0, 2] = blank
    targets[2, 0] = V
    U2, rel2, bad2 = O.subset_and_relabel(targets, tl, blank, V)
    assert list(bad2) == [True, False, True, False]
    assert rel2[0, 2] == -1 and rel2[2, 0] == -1 and V not in U2 and list(U2).count(blank) == 1


# ----------------------------------------------------------------------------
# finite-beam option (Section 3.3, Appendix B.3)
# ----------------------------------------------------------------------------

def enumerate_state_paths(T, L, skip):
    """All trellis paths: start in {0,1}, step by 0, 1 or (where allowed) 2, end in {L-2, L-1}."""
    paths = []

    def rec(path):
        if len(path) == T:
            if path[-1] >= L - 2:
                paths.append(tuple(path))
            return
        s = path[-1]
        for k in (0, 1, 2):
            s2 = s + k
            if s2 >= L or (k == 2 and not skip[s2]):
                continue
            rec(path + [s2])

    for s0 in range(min(2, L)):
        rec([s0])
    return paths


def brute_force_beam(E, skip, beam):
    T, L = E.shape
    paths = enumerate_state_paths(T, L, skip)
    score = {p: sum(E[t, s] for t, s in enumerate(p)) for p in paths}
    best = max(score.values())

    def arcs_of(p):
        a = [("in", p[0])]
        a += [(t, p[t - 1], p[t]) for t in range(1, T)]
        a.append(("out", p[-1]))
        return a

    through = {}
    for p in paths:
        for a in arcs_of(p):
            through[a] = max(through.get(a, -np.inf), score[p])
    kept_arcs = {a for a, sc in through.items() if sc >= best - beam}
    kept = [p for p in paths if all(a in kept_arcs for a in arcs_of(p))]
    within = [p for p in paths if score[p] >= best - beam]
    tot = sum(math.exp(score[p]) for p in kept)
    occ = np.zeros((T, L))
    for p in kept:
        for t, s in enumerate(p):
            occ[t, s] += math.exp(score[p]) / tot
    return -math.log(tot), occ, len(kept), len(within), len(paths)


@pytest.mark.parametrize("beam", [0.5, 1.0, 2.0, 4.0, 8.0, 50.0])
def test_beam_matches_arc_filtered_brute_force(beam):
    rng = np.random.default_rng(17)
    T, V, blank = 7, 6, 0
    y = [2, 2, 4]
    logp, _ = random_logp(rng, T, V)
    logp = logp * 2.0      # spread the scores so that small beams prune
    ext = O.extended_labels(y, blank)
    skip = O.skip_allowed(ext, blank)
    E = logp[:, ext]
    loss_b, occ, n_kept, n_within, n_all = brute_force_beam(E, skip, beam)
    loss, gamma, flags, exact = O.ctc_occupancy(logp, y, blank, beam=beam)
    assert flags == 0
    assert loss == pytest.approx(loss_b, rel=1e-12)
    expect = np.zeros((T, V))
    for s, v in enumerate(ext):
        expect[:, v] += occ[:, s]
    np.testing.assert_allclose(gamma, expect, atol=1e-12)
    assert n_kept >= n_within            # retained arcs can recombine into worse alignments
    # bounds of Appendix B.3
    _, gamma_full, _, _ = O.ctc_occupancy(logp, y, blank)
    Delta, delta = O.discarded_mass(loss, exact)
    assert Delta >= -1e-12
    assert np.max(np.abs(gamma - gamma_full)) <= delta + 1e-12
    assert np.max(np.abs(gamma - gamma_full).sum(1)) <= 2 * delta + 1e-12
    if beam >= 50:
        assert n_kept == n_all and loss == pytest.approx(exact, rel=1e-13)


def test_beam_recombination_exceeds_within_beam_paths():
    # some beam keeps strictly more alignments than score within the beam of the best one
    rng = np.random.default_rng(17)
    logp, _ = random_logp(rng, 7, 6)
    logp = logp * 2.0
    ext = O.extended_labels([2, 2, 4], 0)
    skip = O.skip_allowed(ext, 0)
    counts = [brute_force_beam(logp[:, ext], skip, b)[2:4] for b in (1.0, 2.0, 4.0, 8.0)]
    assert any(k > w for k, w in counts)


def test_beam_monotone_and_off_encodings():
    rng = np.random.default_rng(19)
    logp, _ = random_logp(rng, 12, 9)
    logp = logp * 3.0
    y = [1, 5, 5, 2, 7]
    exact = O.ctc_occupancy(logp, y, 0)[0]
    prev = np.inf
    for beam in (0.25, 1, 2, 4, 8, 16, 32, 64):
        l = O.ctc_occupancy(logp, y, 0, beam=beam)[0]
        assert l >= exact - 1e-12 and l <= prev + 1e-12
        prev = l
    assert prev == pytest.approx(exact, rel=1e-13)
    for off in (None, 0.0, -1.0, float("inf")):
        assert O.ctc_occupancy(logp, y, 0, beam=off)[0] == exact
    # the best alignment always survives: the loss stays finite at any positive beam
    assert np.isfinite(O.ctc_occupancy(logp, y, 0, beam=1e-9)[0])


def test_feasibility_rule_fixture():
    # tests/golden/feasibility_cases.txt: the paper's rule T >= |y| + (adjacent equal pairs), Appendix B.1
    import os
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "feasibility_cases.txt")
    rows = [ln.split("|") for ln in open(path) if ln.strip() and not ln.startswith("#")]
    assert len(rows) >= 10
    rng = np.random.default_rng(0)
    for T, toks, ok in rows:
        T, ok = int(T), int(ok)
        y = [] if toks.strip() == "-" else [int(t) for t in toks.split()]
        assert O.is_feasible(y, T) == bool(ok)
        logp, _ = random_logp(rng, T, 9)
        loss, gamma, flags, _ = O.ctc_occupancy(logp, y, 0)
        assert (flags == 0) == bool(ok)
        if not ok:
            assert loss == 0.0 and gamma is None


def test_stored_c1_values_match_the_oracle():
    # the stored file is written by tests/golden/make_c1_golden.py (oracle only); it guards the
    # oracle and the generator against silent changes
    import json, os
    from paper_2609_33645_b200 import workloads as wl
    gold = json.load(open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "c1_oracle.json")))
    batch = wl.make_batch(wl.CONFIGS["c1"])
    ref = O.pruned_ctc_reference(batch.hidden, batch.W, None, batch.targets, batch.input_lengths,
                                 batch.target_lengths, batch.blank)
    np.testing.assert_allclose(ref["loss"], gold["loss"], rtol=1e-12)
    assert ref["K"] == gold["K"] and list(ref["U"]) == gold["U"]
    assert np.linalg.norm(ref["dW"]) == pytest.approx(gold["dW_fro"], rel=1e-12)
    np.testing.assert_allclose(ref["dW"][0, :8], gold["dW_row_blank"], rtol=1e-10)


def test_collapse_map_and_greedy_decode():
    # B merges repeats first, then drops blanks (Section 3.1): a blank between equal labels keeps both
    assert O.collapse([0, 3, 3, 0, 3, 5, 5, 0, 0, 2], 0) == [3, 3, 5, 2]
    assert O.collapse([4, 4, 4], 4) == [] and O.collapse([], 0) == []
    assert collapse([0, 3, 3, 0, 3, 5, 5, 0, 0, 2], 0) == [3, 3, 5, 2]     # the test's own B agrees
    rng = np.random.default_rng(8)
    H = rng.standard_normal((2, 7, 4))
    W = rng.standard_normal((6, 4))
    frames, hyps, logits = O.greedy_decode(H, W, None, [7, 5], 2)
    for n, Tn in enumerate((7, 5)):
        Z = H[n, :Tn] @ W.T
        assert list(frames[n]) == [int(np.argmax(z)) for z in Z]
        assert hyps[n] == collapse(list(frames[n]), 2)
    # a planted answer: orthonormal class vectors, every frame a multiple of its class's vector plus a
    # little noise, so the top class of each frame is known without taking any arg-max
    V = D = 9
    Q, _ = np.linalg.qr(rng.standard_normal((D, D)))
    planted = [[3, 3, 0, 0, 3, 7, 7, 0, 1, 1, 1, 8], [0, 0, 5, 0, 5, 5, 2]]
    Hp = np.zeros((2, 12, D))
    for n, labs in enumerate(planted):
        for t, v in enumerate(labs):
            Hp[n, t] = 4.0 * Q[v] + 0.05 * rng.standard_normal(D)
    frames, hyps, _ = O.greedy_decode(Hp, Q, None, [12, 7], 0)
    assert [list(f) for f in frames] == planted
    assert hyps == [[3, 3, 7, 1, 8], [5, 5, 2]]                  # worked by hand from the planted frames
    # equal logits: the smallest class index wins (two identical head rows)
    W2 = np.array([[0.0, 1.0], [1.0, 0.0], [1.0, 0.0], [0.5, 0.5]])
    frames, _, _ = O.greedy_decode(np.array([[[2.0, 0.0], [0.0, 3.0]]]), W2, None, [2], 0)
    assert list(frames[0]) == [1, 0]
    # a bias can overturn the projection's winner
    frames, _, _ = O.greedy_decode(np.array([[[2.0, 0.0]]]), W2, np.array([0.0, 0.0, 0.0, 1.5]), [1], 0)
    assert list(frames[0]) == [3]


def test_topk_decode_against_planted_answers():
    # orthonormal class vectors; a frame is 4 q_a + 2 q_b + 1 q_c + noise, so its three best classes are
    # a, b, c in that order by construction, with logits close to 4, 2, 1 and all others close to 0
    rng = np.random.default_rng(11)
    V = D = 12
    Q, _ = np.linalg.qr(rng.standard_normal((D, D)))
    triples = [[(3, 7, 1), (0, 2, 11), (5, 4, 9), (9, 0, 3)], [(8, 1, 2), (6, 10, 0)]]
    Hp = np.zeros((2, 4, D))
    for n, frames in enumerate(triples):
        for t, (a, b, c) in enumerate(frames):
            Hp[n, t] = 4.0 * Q[a] + 2.0 * Q[b] + 1.0 * Q[c] + 0.01 * rng.standard_normal(D)
    cls, lp = O.topk_decode(Hp, Q, None, [4, 2], 4)
    for n, frames in enumerate(triples):
        assert [tuple(r[:3]) for r in cls[n]] == frames
        # log-probabilities: decreasing, differences equal to the planted logit gaps, and consistent with
        # a softmax that sums to one over all classes
        assert np.all(np.diff(lp[n], axis=1) <= 0)
        np.testing.assert_allclose(lp[n][:, 0] - lp[n][:, 1], 2.0, atol=0.05)
        np.testing.assert_allclose(lp[n][:, 1] - lp[n][:, 2], 1.0, atol=0.05)
        full_cls, full_lp = O.topk_decode(Hp[n:n + 1], Q, None, [len(frames)], V)
        np.testing.assert_allclose(np.exp(full_lp[0]).sum(axis=1), 1.0, rtol=1e-12)
        assert sorted(full_cls[0][0]) == list(range(V))
    # rank one is the greedy decoder's frame label
    frames_greedy, _, _ = O.greedy_decode(Hp, Q, None, [4, 2], 0)
    for n in range(2):
        assert list(cls[n][:, 0]) == list(frames_greedy[n])
    # equal logits: the smaller class index first; more ranks than classes: -1 and -inf
    W2 = np.array([[1.0, 0.0], [1.0, 0.0], [0.0, 1.0]])
    cls, lp = O.topk_decode(np.array([[[2.0, 1.0]]]), W2, None, [1], 4)
    assert list(cls[0][0]) == [0, 1, 2, -1] and lp[0][0, 3] == -np.inf and lp[0][0, 0] == lp[0][0, 1]
