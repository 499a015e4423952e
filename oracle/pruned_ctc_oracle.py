"""Float64 CPU oracle for the Pruned-CTC head-and-loss computation.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
CUDA library is compared against.  It shares no code with the CUDA path and is
imported only by the tests, by the smoke check and by the bench's CPU-baseline
leg; the product never routes through it.

What it computes is the *standard* CTC objective on the full vocabulary
(Section 3.1, Eq. "lognorm" and Eq. "ctc"): it materialises the logits and the
log-softmax over all V classes for one utterance at a time, runs the textbook
alpha/beta recursion on the original token ids, and forms the logit gradient
p - gamma (Eq. "grad-full") and its products with the head.  By Proposition 1
this is exactly what the pruned method must reproduce, so the oracle is the
definition written out, not a restatement of Algorithm 1.

Conventions follow Section 3.1: class indices are 0-based.  The paper counts
frames t and trellis positions s from 1; the arrays here are 0-based, so
paper position s is index s-1 and "odd s is blank" becomes "even index is
blank".

Pins (tests/test_oracle_*.py): brute-force enumeration of all alignments on
tiny inputs, the closed form for equal logits, single-alignment and empty-target
special cases, torch's CPU float64 ctc_loss, central finite differences,
per-frame invariants, and Proposition 1 through `grouped_reference`.
The finite-beam rule (`beam=`) follows Appendix B.3 as one sentence of prose;
it is pinned by brute force over arc-filtered paths and by the bounds of
Appendix B.3, but its agreement with the k2 library's retained set is
**parity unpinned** (k2 is not available).
"""

from __future__ import annotations

import numpy as np

NEG_INF = -np.inf

FLAG_INFEASIBLE = 1
FLAG_NONFINITE = 2
FLAG_BAD_TARGET = 4


# ----------------------------------------------------------------------------
# Section 3.1, Eq. "lognorm": logits, normaliser, log-probabilities
# ----------------------------------------------------------------------------

def head_logits(X, W, b=None):
    """Z = X W^T + 1 b^T  (Section 3.1)."""
    Z = np.asarray(X, dtype=np.float64) @ np.asarray(W, dtype=np.float64).T
    if b is not None:
        Z = Z + np.asarray(b, dtype=np.float64)[None, :]
    return Z


def log_normalizer(Z):
    """lambda_m = log sum_u exp Z[m,u]  (Eq. "lognorm"), shifted by the row maximum."""
    mx = np.max(Z, axis=1, keepdims=True)
    mx = np.where(np.isfinite(mx), mx, 0.0)
    return (mx + np.log(np.sum(np.exp(Z - mx), axis=1, keepdims=True)))[:, 0]


def lse(*terms):
    """Elementwise log(sum_i exp(term_i)) with -inf as the empty sum."""
    stack = np.stack([np.asarray(t, dtype=np.float64) for t in terms], axis=0)
    mx = np.max(stack, axis=0)
    safe = np.where(np.isfinite(mx), mx, 0.0)
    with np.errstate(divide="ignore"):
        out = safe + np.log(np.sum(np.exp(stack - safe), axis=0))
    return np.where(np.isneginf(mx), NEG_INF, out)


# ----------------------------------------------------------------------------
# Algorithm 1, lines 2-3: batch-union subset and relabelling
# ----------------------------------------------------------------------------

def subset_and_relabel(targets, target_lengths, blank, V):
    """U = blank followed by the ascending distinct labels of all targets.

    Returns (U [K] int32, relabelled targets with the same shape as `targets`,
    entries beyond a row's length set to -1, and per-utterance bad-target mask).
    A token equal to `blank` or outside [0, V) is a bad target: it is left out
    of U, relabelled -1, and marks its utterance.
    """
    targets = np.asarray(targets)
    N = targets.shape[0]
    good = []
    bad = np.zeros(N, dtype=bool)
    for n in range(N):
        for i in range(int(target_lengths[n])):
            tok = int(targets[n, i])
            if tok == blank or tok < 0 or tok >= V:
                bad[n] = True
            else:
                good.append(tok)
    labels = sorted(set(good))
    U = np.array([blank] + labels, dtype=np.int32)
    index = {tok: 1 + k for k, tok in enumerate(labels)}
    rel = np.full(targets.shape, -1, dtype=np.int32)
    for n in range(N):
        for i in range(int(target_lengths[n])):
            rel[n, i] = index.get(int(targets[n, i]), -1)
    return U, rel, bad


# ----------------------------------------------------------------------------
# Appendix B.1: structural feasibility
# ----------------------------------------------------------------------------

def adjacent_repeats(y):
    y = list(y)
    return sum(1 for i in range(1, len(y)) if y[i] == y[i - 1])


def is_feasible(y, T):
    """An utterance has an alignment iff T >= |y| + (number of adjacent equal pairs)."""
    return T >= len(y) + adjacent_repeats(y)


# ----------------------------------------------------------------------------
# Textbook CTC alpha/beta on the extended label sequence
# ----------------------------------------------------------------------------

def extended_labels(y, blank):
    """l' = (blank, y_1, blank, ..., y_U, blank), length 2U+1."""
    ext = [blank]
    for tok in y:
        ext += [int(tok), blank]
    return np.array(ext, dtype=np.int64)


def skip_allowed(ext, blank):
    """skip[s] is True where the transition s-2 -> s exists: l'_s non-blank and != l'_{s-2}."""
    L = len(ext)
    ok = np.zeros(L, dtype=bool)
    for s in range(2, L):
        ok[s] = ext[s] != blank and ext[s] != ext[s - 2]
    return ok


def _shift(v, k):
    """v delayed by k positions (out[s] = v[s-k]), -inf shifted in."""
    out = np.full_like(v, NEG_INF)
    if k == 0:
        out[:] = v
    elif k < len(v):
        out[k:] = v[:-k]
    return out


def _advance(v, k):
    """out[s] = v[s+k], -inf shifted in."""
    out = np.full_like(v, NEG_INF)
    if k == 0:
        out[:] = v
    elif k < len(v):
        out[:-k] = v[k:]
    return out


def _reduce(v, semiring):
    """Sum (log semiring) or best (max semiring) of a vector of log-scores."""
    mx = np.max(v)
    if semiring == "max" or np.isneginf(mx):
        return mx
    return mx + np.log(np.sum(np.exp(v - mx)))


def trellis_sweeps(E, skip, semiring="log", keep=None):
    """Forward and backward recursions over the T x L trellis.

    E[t,s] is the emission log-score of position s at frame t.  Both recursions
    include E[t,s] in their value at (t,s).  `semiring` is "log" (sum over
    alignments) or "max" (best alignment).  `keep`, if given, is a dict of
    boolean arrays restricting the arcs: keep["in"][s] (entry arcs at the first
    frame), keep["out"][s] (exit arcs at the last frame) and keep[k][t,s] for
    k in 0,1,2: the arc (t-1, s-k) -> (t, s), rows t >= 1.
    Returns alpha, beta, total.
    """
    T, L = E.shape
    comb = lse if semiring == "log" else (lambda *a: np.max(np.stack(a, 0), axis=0))
    entry = np.zeros(L, dtype=bool)
    entry[0] = True
    if L >= 2:
        entry[1] = True
    exit_ = np.zeros(L, dtype=bool)
    exit_[L - 1] = True
    if L >= 2:
        exit_[L - 2] = True
    if keep is not None:
        entry = entry & keep["in"]
        exit_ = exit_ & keep["out"]

    def masked(v, m):
        return np.where(m, v, NEG_INF)

    alpha = np.full((T, L), NEG_INF)
    alpha[0] = masked(E[0], entry)
    for t in range(1, T):
        a0 = _shift(alpha[t - 1], 0)
        a1 = _shift(alpha[t - 1], 1)
        a2 = masked(_shift(alpha[t - 1], 2), skip)
        if keep is not None:
            a0, a1, a2 = masked(a0, keep[0][t]), masked(a1, keep[1][t]), masked(a2, keep[2][t])
        alpha[t] = E[t] + comb(a0, a1, a2)
    total = _reduce(masked(alpha[T - 1], exit_), semiring)

    beta = np.full((T, L), NEG_INF)
    beta[T - 1] = masked(E[T - 1], exit_)
    for t in range(T - 2, -1, -1):
        nxt = beta[t + 1]
        if keep is not None:
            b0 = _advance(masked(nxt, keep[0][t + 1]), 0)
            b1 = _advance(masked(nxt, keep[1][t + 1]), 1)
            b2 = _advance(masked(masked(nxt, skip), keep[2][t + 1]), 2)
        else:
            b0 = _advance(nxt, 0)
            b1 = _advance(nxt, 1)
            b2 = _advance(masked(nxt, skip), 2)
        beta[t] = E[t] + comb(b0, b1, b2)
    return alpha, beta, float(total)


def retained_arcs(E, skip, beam):
    """Arc retention of the finite-beam option (Section 3.3, Appendix B.3).

    With a[t,s] / b[t,s] the best-alignment (max-semiring) forward / backward
    scores, the best alignment through the arc (t-1,s') -> (t,s) scores
    a[t-1,s'] + b[t,s]; the arc is kept iff that is within `beam` of the best
    alignment overall (inclusive).  Entry arcs use b at the first frame, exit
    arcs use a at the last frame.
    """
    T, L = E.shape
    a, b, best = trellis_sweeps(E, skip, semiring="max")
    thr = best - beam
    keep = {"in": b[0] >= thr, "out": a[T - 1] >= thr}
    for k in (0, 1, 2):
        m = np.zeros((T, L), dtype=bool)
        for t in range(1, T):
            m[t] = _shift(a[t - 1], k) + b[t] >= thr
        if k == 2:
            m &= skip[None, :]
        keep[k] = m
    return keep, best


def beam_is_off(beam):
    return beam is None or not (beam > 0) or np.isinf(beam)


def ctc_occupancy(logp, y, blank, beam=None):
    """Loss and label occupancies gamma[t,v] of one utterance.

    logp: [T, V] log-probabilities of the utterance's frames.  Returns
    (loss, gamma [T,V], flags, exact_loss) where exact_loss is the unpruned loss
    (equal to loss when no beam is set).  Infeasible or non-finite utterances
    give loss 0 and gamma None (their frames get zero gradient).
    """
    T, V = logp.shape
    if not is_feasible(y, T):
        return 0.0, None, FLAG_INFEASIBLE, 0.0
    ext = extended_labels(y, blank)
    skip = skip_allowed(ext, blank)
    E = logp[:, ext]
    alpha, beta, total = trellis_sweeps(E, skip, "log")
    exact_loss = -total
    if not beam_is_off(beam):
        keep, _ = retained_arcs(E, skip, float(beam))
        alpha, beta, total = trellis_sweeps(E, skip, "log", keep=keep)
    loss = -total
    if not np.isfinite(loss):
        return 0.0, None, FLAG_NONFINITE, 0.0
    with np.errstate(invalid="ignore"):
        g_state = np.exp(alpha + beta - E - total)
    g_state = np.where(np.isfinite(g_state), g_state, 0.0)
    gamma = np.zeros((T, V))
    for s, v in enumerate(ext):
        gamma[:, v] += g_state[:, s]
    return loss, gamma, 0, exact_loss


# ----------------------------------------------------------------------------
# The whole computation, one utterance at a time
# ----------------------------------------------------------------------------

def utterance_fwd_bwd(Hn, W, b, y, blank, beam=None, bad=False):
    """Returns (loss, dZ [T_n,V] or None, flags, exact_loss, lambda [T_n])."""
    Z = head_logits(Hn, W, b)
    lam = log_normalizer(Z)
    if bad:
        return 0.0, None, FLAG_BAD_TARGET, 0.0, lam
    if not np.all(np.isfinite(lam)):
        return 0.0, None, FLAG_NONFINITE, 0.0, lam
    logp = Z - lam[:, None]
    loss, gamma, flags, exact = ctc_occupancy(logp, y, blank, beam)
    if gamma is None:
        return 0.0, None, flags, 0.0, lam
    dZ = np.exp(logp) - gamma                     # Eq. "grad-full"
    return loss, dZ, flags, exact, lam


def pruned_ctc_reference(hidden, W, bias, targets, input_lengths, target_lengths, blank,
                         beam=None, want_dW=True, dW_rows=None, dH_for=None, utt_weights=None):
    """Full-vocabulary CTC loss and gradients of the sum of utterance losses.

    hidden [N,T,D], W [V,D], bias [V] or None, targets [N,stride] int,
    input_lengths [N], target_lengths [N].  Returns a dict with
    loss [N], dH [N,T,D] (padded frames zero), dW [V,D] (or only the rows in
    `dW_rows`), db [V], U, K, relabeled, flags [N], exact_loss [N],
    lam (list of per-utterance normalisers).  `dH_for`, if given, lists the
    utterances whose dH is wanted (the others are left zero): sampled checks at
    full size skip the products they do not look at.  `utt_weights` [N] are
    upstream gradients c_n of the utterance losses (Appendix B.1: the row sums of
    G account for loss scaling): gradients are then those of sum_n c_n L_n, the
    returned losses stay unweighted.
    """
    hidden = np.asarray(hidden, dtype=np.float64)
    W64 = np.asarray(W, dtype=np.float64)
    b64 = None if bias is None else np.asarray(bias, dtype=np.float64)
    N, T, D = hidden.shape
    V = W64.shape[0]
    U, rel, bad = subset_and_relabel(targets, target_lengths, blank, V)
    loss = np.zeros(N)
    exact = np.zeros(N)
    flags = np.zeros(N, dtype=np.int32)
    dH = np.zeros((N, T, D))
    rows = None if dW_rows is None else np.asarray(dW_rows, dtype=np.int64)
    if want_dW:
        dW = np.zeros((V, D)) if rows is None else np.zeros((len(rows), D))
    else:
        dW = None
    db = np.zeros(V)
    lams = []
    for n in range(N):
        Tn = int(input_lengths[n])
        y = [int(v) for v in targets[n, : int(target_lengths[n])]]
        Hn = hidden[n, :Tn]
        l, dZ, f, ex, lam = utterance_fwd_bwd(Hn, W64, b64, y, blank, beam, bad=bool(bad[n]))
        lams.append(lam)
        loss[n], flags[n], exact[n] = l, f, ex
        if dZ is None:
            continue
        if utt_weights is not None:
            dZ = dZ * float(utt_weights[n])
        if dH_for is None or n in dH_for:
            dH[n, :Tn] = dZ @ W64
        if want_dW:
            if rows is None:
                dW += dZ.T @ Hn
            else:
                dW += dZ[:, rows].T @ Hn
        db += dZ.sum(axis=0)
    return dict(loss=loss, dH=dH, dW=dW, db=db, U=U, K=int(len(U)), relabeled=rel,
                flags=flags, exact_loss=exact, lam=lams)


# ----------------------------------------------------------------------------
# Proposition 1: the grouped ("other class") formulation, Eq. "grouped",
# Eq. "grad-grouped" and Eq. "offsupport"
# ----------------------------------------------------------------------------

def grouped_reference(hidden, W, bias, targets, input_lengths, target_lengths, blank):
    """Unpruned reduced CTC: CTC on log_softmax(R) with relabelled targets.

    R holds the K selected logits and, when the complement is non-empty, one
    extra column with the log-sum-exp of the complement.  The gradient is pushed
    back through R to the full logits.  Same return keys as
    `pruned_ctc_reference` (loss, dH, dW, db).
    """
    hidden = np.asarray(hidden, dtype=np.float64)
    W64 = np.asarray(W, dtype=np.float64)
    b64 = None if bias is None else np.asarray(bias, dtype=np.float64)
    N, T, D = hidden.shape
    V = W64.shape[0]
    U, rel, bad = subset_and_relabel(targets, target_lengths, blank, V)
    K = len(U)
    comp = np.setdiff1d(np.arange(V), U)
    loss = np.zeros(N)
    dH = np.zeros((N, T, D))
    dW = np.zeros((V, D))
    db = np.zeros(V)
    for n in range(N):
        Tn = int(input_lengths[n])
        Hn = hidden[n, :Tn]
        Z = head_logits(Hn, W64, b64)
        if len(comp):
            other = log_normalizer(Z[:, comp])
            R = np.concatenate([Z[:, U], other[:, None]], axis=1)
        else:
            R = Z[:, U]
        logpbar = R - log_normalizer(R)[:, None]
        ytil = [int(v) for v in rel[n, : int(target_lengths[n])]]
        if bad[n]:
            continue
        l, gam, f, _ = ctc_occupancy(logpbar, ytil, 0, None)   # blank is index 0 of U
        if gam is None:
            continue
        loss[n] = l
        dR = np.exp(logpbar) - gam                               # Eq. "grad-grouped"
        dZ = np.zeros_like(Z)
        dZ[:, U] = dR[:, :K]
        if len(comp):
            dZ[:, comp] = dR[:, K:K + 1] * np.exp(Z[:, comp] - other[:, None])   # Eq. "offsupport"
        dH[n, :Tn] = dZ @ W64
        dW += dZ.T @ Hn
        db += dZ.sum(axis=0)
    return dict(loss=loss, dH=dH, dW=dW, db=db, U=U, K=K, relabeled=rel)


# ----------------------------------------------------------------------------
# Greedy recognition (Section 5.1; Appendix D): frame-wise arg-max, then the
# collapse map B of Section 3.1
# ----------------------------------------------------------------------------

def collapse(labels, blank):
    """B: merge consecutive repetitions, then remove blanks."""
    out = []
    prev = None
    for v in labels:
        v = int(v)
        if v != prev and v != blank:
            out.append(v)
        prev = v
    return out


def greedy_decode(hidden, W, bias, input_lengths, blank):
    """Per utterance: arg-max class of every valid frame (first index on ties), the collapsed
    hypothesis, and the full logits' top value per frame (for near-tie checks)."""
    hidden = np.asarray(hidden, dtype=np.float64)
    W64 = np.asarray(W, dtype=np.float64)
    b64 = None if bias is None else np.asarray(bias, dtype=np.float64)
    frames, hyps, logits = [], [], []
    for n in range(hidden.shape[0]):
        Z = head_logits(hidden[n, : int(input_lengths[n])], W64, b64)
        lab = np.argmax(Z, axis=1)
        frames.append(lab)
        hyps.append(collapse(lab, blank))
        logits.append(Z)
    return frames, hyps, logits


def topk_decode(hidden, W, bias, input_lengths, k):
    """Per utterance: the k classes with the largest logits of every valid frame (descending; the
    smaller class index first among equal logits) and their log-probabilities under the
    full-vocabulary softmax (Eq. "lognorm"): what a prefix beam search (Section 5.1) reads per frame."""
    hidden = np.asarray(hidden, dtype=np.float64)
    W64 = np.asarray(W, dtype=np.float64)
    b64 = None if bias is None else np.asarray(bias, dtype=np.float64)
    classes, logprobs = [], []
    for n in range(hidden.shape[0]):
        Z = head_logits(hidden[n, : int(input_lengths[n])], W64, b64)
        logp = Z - log_normalizer(Z)[:, None]
        V = Z.shape[1]
        cls = np.full((Z.shape[0], k), -1, dtype=np.int64)
        lp = np.full((Z.shape[0], k), -np.inf)
        for t in range(Z.shape[0]):
            order = np.lexsort((np.arange(V), -Z[t]))[:k]      # by logit, descending; ties by class index
            cls[t, : len(order)] = order
            lp[t, : len(order)] = logp[t, order]
        classes.append(cls)
        logprobs.append(lp)
    return classes, logprobs


def discarded_mass(loss_beam, loss_exact):
    """Delta_n = L_beta,n - L_n and delta_n = 1 - exp(-Delta_n)  (Appendix B.3)."""
    delta_big = np.asarray(loss_beam, dtype=np.float64) - np.asarray(loss_exact, dtype=np.float64)
    return delta_big, -np.expm1(-delta_big)
