"""The entry point for callers that cannot allocate device memory.

Some users of this library run where cudaMalloc is not available to them (a
memory-pool callback, a process that handed out all device memory at start-up,
a loop that must stay clear of the allocator).  pctc_subset_relabel_noalloc
serves them: it keeps its scratch in a fixed array inside the library.  This
test calls it through the C ABI twice in a row, on two different batches, and
requires the same subset, K and relabelled targets, bit for bit, as the regular
entry point (which uses a caller-provided workspace) returns and as the oracle
defines; it also checks that the device's free memory does not move across a call.
"""

import numpy as np
import pytest

from oracle import pruned_ctc_oracle as O
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


def _outputs(N, stride, cap, dev):
    import torch
    return dict(subset=torch.full((cap,), -1, dtype=torch.int32, device=dev),
                K=torch.zeros(1, dtype=torch.int32, device=dev),
                relabeled=torch.zeros((N, stride), dtype=torch.int32, device=dev),
                flags=torch.zeros(N, dtype=torch.int32, device=dev))


def test_no_alloc_entry_point_matches_regular_entry_point_twice(lib):
    import torch
    dev = torch.device("cuda:0")
    cases = [
        wl.make_batch(wl.reduced(wl.CONFIGS["c2"], V=8192, D=64, N=6, T_div=8, name="na1"), permute_ids=True),
        wl.make_batch(wl.reduced(wl.CONFIGS["c3"], V=200000, D=8, N=5, T_div=16, U_div=2, name="na2", blank=77)),
    ]
    cases[1].targets[2, 1] = cases[1].blank          # a bad target: flagged, left out of U
    for i, batch in enumerate(cases):                # two calls in a row share the library's scratch
        ref, targets = _regular(lib, batch)
        N, stride = batch.targets.shape
        tl = torch.from_numpy(batch.target_lengths).to(dev)
        out = _outputs(N, stride, ref["subset"].numel(), dev)
        if i == 0:                                   # module loading and the address look-up happen at the first call
            lib.subset_relabel_noalloc(targets, tl, batch.cfg.V, batch.blank, out)
            torch.cuda.synchronize()
            out = _outputs(N, stride, ref["subset"].numel(), dev)
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info(dev)     # the driver's count: sees any cudaMalloc, not only torch's
        before = torch.cuda.memory_allocated(dev)
        lib.subset_relabel_noalloc(targets, tl, batch.cfg.V, batch.blank, out)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated(dev) == before
        assert torch.cuda.mem_get_info(dev)[0] == free_before
        K = int(ref["K"].item())
        assert int(out["K"].item()) == K
        np.testing.assert_array_equal(out["subset"].cpu().numpy()[:K], ref["subset"].cpu().numpy()[:K])
        np.testing.assert_array_equal(out["relabeled"].cpu().numpy(), ref["relabeled"].cpu().numpy())
        np.testing.assert_array_equal(out["flags"].cpu().numpy() & 4, ref["flags"].cpu().numpy() & 4)
        # and against the definition itself (Algorithm 1 lines 2-3)
        U, rel, bad = O.subset_and_relabel(batch.targets, batch.target_lengths, batch.blank, batch.cfg.V)
        assert K == len(U)
        np.testing.assert_array_equal(out["subset"].cpu().numpy()[:K], U)
        np.testing.assert_array_equal(out["relabeled"].cpu().numpy(), rel)
        np.testing.assert_array_equal((out["flags"].cpu().numpy() & 4) != 0, np.asarray(bad, dtype=bool))


def test_no_alloc_entry_point_at_its_largest_vocabulary(lib):
    """V equal to the limit: the last word of the bit map, of the rank table and the last entry of the
    class map (the ends of the three regions of the fixed array) are all in use."""
    import torch
    dev = torch.device("cuda:0")
    V = lib.NOALLOC_MAX_V
    rng = np.random.default_rng(5)
    N, stride, blank = 3, 40, V - 7
    targets = rng.integers(0, V, size=(N, stride)).astype(np.int32)
    targets[targets == blank] = 0
    targets[0, :4] = [V - 1, V - 2, 0, V - 32]       # both ends of the class range
    lengths = np.array([40, 17, 0], dtype=np.int32)
    U, rel, bad = O.subset_and_relabel(targets, lengths, blank, V)
    out = _outputs(N, stride, 1 + int(lengths.sum()), dev)
    for _ in range(2):
        lib.subset_relabel_noalloc(torch.from_numpy(targets).to(dev), torch.from_numpy(lengths).to(dev), V, blank, out)
        torch.cuda.synchronize()
        assert int(out["K"].item()) == len(U)
        np.testing.assert_array_equal(out["subset"].cpu().numpy()[:len(U)], U)
        np.testing.assert_array_equal(out["relabeled"].cpu().numpy(), rel)
        assert not out["flags"].cpu().numpy().any() and not np.any(bad)


def test_no_alloc_entry_point_rejects_oversized_vocabulary(lib):
    import torch
    dev = torch.device("cuda:0")
    t = torch.ones((1, 2), dtype=torch.int32, device=dev)
    out = _outputs(1, 2, 3, dev)
    with pytest.raises(lib.PctcError) as ei:
        lib.subset_relabel_noalloc(t, torch.tensor([2], dtype=torch.int32, device=dev), lib.NOALLOC_MAX_V + 1, 0, out)
    assert ei.value.status == 3
