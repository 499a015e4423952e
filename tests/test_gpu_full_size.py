"""Parity at full size: the workload and launch configuration that bench.py times
(c4: D=4096, V=151,936, about 8,000 frames, default chunk), checked on outputs the
oracle can compute one by one (integer outputs, every per-utterance loss, dH of two
utterances, sampled rows of dW) and on identities that hold at any size."""

import time

import numpy as np
import pytest

from paper_2609_33645_b200 import workloads as wl
from tests import helpers as H

pytestmark = pytest.mark.gpu


def test_c4_full_size_sampled_parity(lib):
    import torch
    cfg = wl.CONFIGS["c4"]
    batch = wl.make_batch(cfg)
    dev = torch.device("cuda:0")
    hidden = torch.from_numpy(batch.hidden).to(dev).to(torch.bfloat16)
    W = torch.from_numpy(batch.W).to(dev).to(torch.bfloat16)
    targets = torch.from_numpy(batch.targets).to(dev)
    res = lib.pruned_ctc_fwd_bwd(hidden, W, None, targets, batch.input_lengths, batch.target_lengths, batch.blank,
                                 check_status=True)
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
    order = np.argsort(batch.input_lengths)
    dH_for = [int(order[0]), int(order[1])]
    t0 = time.time()
    ref = H.run_oracle(batch, dW_rows=rows, dH_for=dH_for)
    print(f"oracle (sampled) took {time.time() - t0:.1f} s")
    loss = res["loss"].cpu().numpy()
    np.testing.assert_array_equal(res["flags"].cpu().numpy(), ref["flags"])
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
