"""Parity at full size: the bf16 configurations c2-c5 exactly as bench.py launches them
(default chunk; c4 is the bench default: D=4096, V=151,936, about 8,000 frames) and the smallest
workload of the paper's own grid (g16k: 160 utterances of 100 frames, D=512, V=180,000), checked on
outputs the oracle can compute one by one (integer outputs, every per-utterance loss, dH of
two utterances, sampled rows of dW) and on identities that hold at any size.  c1 (fp32) is
compared in full in test_gpu_parity.py."""

import time

import numpy as np
import pytest

from paper_2609_33645_b200 import workloads as wl
from tests import helpers as H

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", ["c2", "c3", "c4", "c5", "g16k"])
def test_full_size_sampled_parity(lib, name):
    check_sampled_parity(lib, wl.CONFIGS[name])


def test_chunk_buffer_beyond_2_to_31_elements(lib):
    # 64 utterances of about 4,200 frames: M x C = 268,000 x 8,192 > 2^31 elements in the dlogits chunk,
    # so every index into it has to be 64-bit; narrow head and small vocabulary keep the oracle quick
    cfg = wl.Config("bigM", N=64, T_lo=4150, T_hi=4250, D=256, V=8192 + 40, dtype="bf16", U_lo=5, U_hi=20,
                    zipf_s=1.1, seed=1777)
    check_sampled_parity(lib, cfg)


@pytest.mark.parametrize("beam", [8.0, 16.0])
def test_c5_full_size_gradients_under_a_beam(lib, beam):
    """Section 3.3 at full size (T up to 3000, about 1,200 trellis positions): the gradients p - gamma^beta
    against the oracle AT THE SAME BEAM.  At these beams gamma^beta differs strongly from the exact
    occupancy (Appendix B.3: most of the exact lattice's mass is discarded), so this is a check of the
    arc-masked sweeps, not of the unpruned ones."""
    check_sampled_parity(lib, wl.CONFIGS["c5"], beam=beam, n_dH=1)


def check_sampled_parity(lib, cfg, beam=0.0, n_dH=2):
    import torch
    batch = wl.make_batch(cfg)
    assert batch.M * min(cfg.V, 8192) > 2 ** 31 or cfg.name != "bigM"
    dev = torch.device("cuda:0")
    hidden = torch.from_numpy(batch.hidden).to(dev).to(torch.bfloat16)
    W = torch.from_numpy(batch.W).to(dev).to(torch.bfloat16)
    targets = torch.from_numpy(batch.targets).to(dev)
    res = lib.pruned_ctc_fwd_bwd(hidden, W, None, targets, batch.input_lengths, batch.target_lengths, batch.blank,
                                 beam=beam, check_status=True)
    torch.cuda.synchronize()

    # ---- identities that hold at any size (computed from the GPU outputs alone) ----
    dW = res["dW"].float()
    dH = res["dH"].float()
    # every frame's dlogits sum to zero  =>  the rows of dW sum to the zero vector
    col = dW.double().sum(0)
    scale = dW.double().abs().sum(0)
    assert float((col.abs() / scale).max()) < 2e-2
    # <dW, W> = <dH, X> (both equal sum dZ * Z when there is no bias)
    lhs = float((dW.double() * W.double()).sum())
    rhs = float((dH.double() * hidden.double()).sum())
    assert abs(lhs - rhs) <= 1e-2 * max(abs(lhs), abs(rhs)), (lhs, rhs)
    for n in range(cfg.N):
        assert bool((dH[n, int(batch.input_lengths[n]):] == 0).all())

    # ---- oracle on sampled outputs ----
    rng = np.random.default_rng(4)
    loss = res["loss"].cpu().numpy()
    flags_gpu = res["flags"].cpu().numpy()
    from oracle import pruned_ctc_oracle as O
    U, rel, bad = O.subset_and_relabel(batch.targets, batch.target_lengths, batch.blank, cfg.V)
    K = len(U)
    assert int(res["K"].item()) == K
    np.testing.assert_array_equal(res["subset"].cpu().numpy()[:K], U)
    np.testing.assert_array_equal(res["relabeled"].cpu().numpy(), rel)
    rows = np.unique(np.concatenate([
        U[:8], U[rng.integers(0, K, 16)],                          # selected classes (gamma term)
        rng.integers(0, cfg.V, 24),                                # any class
        np.arange(cfg.V - 4, cfg.V), [8191, 8192, 4095, 4096],     # chunk and tile edges, ragged last chunk
    ])).astype(np.int64)
    del res
    torch.cuda.empty_cache()
    order = np.argsort(batch.input_lengths)
    dH_for = [int(order[k]) for k in range(n_dH)]
    t0 = time.time()
    ref = H.run_oracle(batch, beam=beam if beam > 0 else None, dW_rows=rows, dH_for=dH_for)
    print(f"oracle (sampled) took {time.time() - t0:.1f} s")
    np.testing.assert_array_equal(flags_gpu, ref["flags"])
    assert np.all(np.abs(loss - ref["loss"]) <= 2e-3 * np.abs(ref["loss"])), (loss, ref["loss"])
    for n in dH_for:
        err = H.rel_fro(dH[n].cpu().numpy(), ref["dH"][n])
        assert err <= 1e-2, (n, err)
    got_rows = dW[torch.from_numpy(rows).to(dev)].cpu().numpy()
    err = H.rel_fro(got_rows, ref["dW"])
    assert err <= 1e-2, err
    # row by row as well, so that a single wrong row cannot hide in the norm
    for k, v in enumerate(rows):
        e = H.rel_fro(got_rows[k], ref["dW"][k])
        assert e <= 3e-2, (int(v), e)


def test_c5_full_size_losses_and_beam_gap(lib):
    """c5 (D=5120, V=151,936, T up to 3000, up to 600 labels): per-utterance loss without a beam and at
    beams 16 and 8 against the oracle at the same beam; the gap Delta_n = L_beta,n - L_n >= 0 and the
    discarded mass delta_n = 1 - exp(-Delta_n) of Appendix B.3 are printed for the record."""
    import torch
    from oracle import pruned_ctc_oracle as O
    cfg = wl.CONFIGS["c5"]
    batch = wl.make_batch(cfg)
    dev = torch.device("cuda:0")
    hidden = torch.from_numpy(batch.hidden).to(dev).to(torch.bfloat16)
    W = torch.from_numpy(batch.W).to(dev).to(torch.bfloat16)
    targets = torch.from_numpy(batch.targets).to(dev)
    gpu = {}
    res = None
    for beam in (0.0, 16.0, 8.0):
        res = lib.pruned_ctc_fwd_bwd(hidden, W, None, targets, batch.input_lengths, batch.target_lengths,
                                     batch.blank, beam=beam, check_status=True,
                                     workspace=None if res is None else res["workspace"])
        torch.cuda.synchronize()
        gpu[beam] = res["loss"].cpu().numpy().astype(np.float64)
        assert int(res["flags"].abs().sum().item()) == 0
    del res
    torch.cuda.empty_cache()

    # oracle: full-vocabulary normaliser per utterance, then the alignment sums on the selected classes
    # (by Proposition 1 the selected log-probabilities with relabelled targets give the same loss)
    t0 = time.time()
    W64 = batch.W.astype(np.float64)
    ref = {0.0: [], 16.0: [], 8.0: []}
    for n in range(cfg.N):
        Tn, Un = int(batch.input_lengths[n]), int(batch.target_lengths[n])
        y = [int(v) for v in batch.targets[n, :Un]]
        Z = O.head_logits(batch.hidden[n, :Tn], W64)
        lam = O.log_normalizer(Z)
        cols = np.array([batch.blank] + sorted(set(y)), dtype=np.int64)
        logp = Z[:, cols] - lam[:, None]
        del Z
        ytil = [int(np.searchsorted(cols[1:], v)) + 1 for v in y]
        for beam in ref:
            ref[beam].append(O.ctc_occupancy(logp, ytil, 0, beam=beam if beam > 0 else None)[0])
    print(f"oracle took {time.time() - t0:.1f} s")
    for beam in ref:
        r = np.array(ref[beam])
        rel = np.abs(gpu[beam] - r) / np.abs(r)
        print(f"beam {beam}: oracle {r}, gpu {gpu[beam]}, rel err {rel}")
        assert np.all(rel <= 2e-3)
    exact = np.array(ref[0.0])
    for beam in (16.0, 8.0):
        Delta, delta = O.discarded_mass(ref[beam], exact)
        Delta_gpu = gpu[beam] - gpu[0.0]
        print(f"beam {beam}: Delta_n oracle {Delta}, gpu {Delta_gpu}, delta_n {delta}")
        assert np.all(Delta >= -1e-9)
        assert np.all(Delta_gpu >= -2e-3 * exact)          # within the loss tolerance of being an upper bound
        assert np.all(np.abs(Delta_gpu - Delta) <= 2e-3 * exact)
