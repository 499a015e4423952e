"""The entry point for callers that cannot allocate device memory.

Some users of this library run where cudaMalloc is not available to them (a
memory-pool callback, a process that handed out all device memory at start-up,
a loop that must stay clear of the allocator).  pctc_subset_relabel_noalloc
serves them: it keeps its scratch in a fixed array inside the library.  This
test calls it through the C ABI twice in a row, on two different batches, and
requires the same subset, K and relabelled targets, bit for bit, as the regular
entry point (which uses a caller-provided workspace) returns.

Collected last on purpose, so that a failure here cannot hide the other tests
in a run that stops at the first failure; it also passes on its own in a fresh
process.
"""

import numpy as np
import pytest

from paper_2609_33645_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _regular(lib, batch):
    import torch
    dev = torch.device("cuda:0")
    hidden = torch.from_numpy(batch.hidden).to(dev).to(torch.bfloat16)
    W = torch.from_numpy(batch.W).to(dev).to(torch.bfloat16)
    targets = torch.from_numpy(batch.targets).to(dev)
    res = lib.pruned_ctc_fwd_bwd(hidden, W, None, targets, batch.input_lengths, batch.target_lengths, batch.blank)
    torch.cuda.synchronize()
    return res, targets


def test_no_alloc_entry_point_matches_regular_entry_point_twice(lib):
    import torch
    dev = torch.device("cuda:0")
    cases = [
        wl.make_batch(wl.reduced(wl.CONFIGS["c2"], V=8192, D=64, N=6, T_div=8, name="na1"), permute_ids=True),
        wl.make_batch(wl.reduced(wl.CONFIGS["c3"], V=200000, D=8, N=5, T_div=16, U_div=2, name="na2", blank=77)),
    ]
    cases[1].targets[2, 1] = cases[1].blank          # a bad target: flagged, left out of U
    for batch in cases:                              # two calls in a row share the library's scratch
        ref, targets = _regular(lib, batch)
        N, stride = batch.targets.shape
        tl = torch.from_numpy(batch.target_lengths).to(dev)
        out = dict(subset=torch.full_like(ref["subset"], -1), K=torch.zeros(1, dtype=torch.int32, device=dev),
                   relabeled=torch.zeros((N, stride), dtype=torch.int32, device=dev),
                   flags=torch.zeros(N, dtype=torch.int32, device=dev))
        before = torch.cuda.memory_allocated(dev)
        lib.subset_relabel_noalloc(targets, tl, batch.cfg.V, batch.blank, out)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated(dev) == before
        K = int(ref["K"].item())
        assert int(out["K"].item()) == K
        np.testing.assert_array_equal(out["subset"].cpu().numpy()[:K], ref["subset"].cpu().numpy()[:K])
        np.testing.assert_array_equal(out["relabeled"].cpu().numpy(), ref["relabeled"].cpu().numpy())
        np.testing.assert_array_equal(out["flags"].cpu().numpy() & 4, ref["flags"].cpu().numpy() & 4)


def test_no_alloc_entry_point_rejects_oversized_vocabulary(lib):
    import torch
    dev = torch.device("cuda:0")
    t = torch.ones((1, 2), dtype=torch.int32, device=dev)
    out = dict(subset=torch.zeros(3, dtype=torch.int32, device=dev), K=torch.zeros(1, dtype=torch.int32, device=dev),
               relabeled=torch.zeros((1, 2), dtype=torch.int32, device=dev),
               flags=torch.zeros(1, dtype=torch.int32, device=dev))
    with pytest.raises(lib.PctcError) as ei:
        lib.subset_relabel_noalloc(t, torch.tensor([2], dtype=torch.int32, device=dev), lib.NOALLOC_MAX_V + 1, 0, out)
    assert ei.value.status == 3
