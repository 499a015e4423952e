"""Host logic of the utterance-sharded data-parallel step, on CPU: the sharding, the chunk row
ranges, and the per-chunk all-reduce of dW over two gloo ranks.  The ranks compute their shard's
gradients with the float64 oracle; the sum over ranks must be the gradient of the whole batch
(the loss is a sum over utterances), and losses and dH must be the shard's rows of the whole."""

import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from paper_2609_33645_b200 import data_parallel as dp  # noqa: E402
from paper_2609_33645_b200 import workloads as wl  # noqa: E402


@pytest.mark.parametrize("world", [1, 2, 3, 8])
def test_sharding_is_a_partition_and_balances_frames(world):
    rng = np.random.default_rng(world)
    T = rng.integers(100, 3000, size=37)
    shards = dp.shard_utterances(T, world)
    assert len(shards) == world
    allidx = np.concatenate(shards)
    assert sorted(allidx.tolist()) == list(range(37))
    loads = np.array([T[s].sum() for s in shards])
    # greedy longest-first: no rank exceeds the mean by more than one utterance
    assert loads.max() - T.sum() / world <= T.max()
    for s in shards:
        assert np.all(np.diff(s) > 0)


def test_more_ranks_than_utterances_leaves_ranks_empty():
    shards = dp.shard_utterances([5, 9], 4)
    assert sorted(len(s) for s in shards) == [0, 0, 1, 1]


def test_chunk_rows_cover_the_vocabulary_once():
    rows = dp.chunk_rows(151936, 8192)
    assert rows[0] == (0, 8192) and rows[-1] == (147456, 151936) and len(rows) == 19
    assert all(a[1] == b[0] for a, b in zip(rows, rows[1:]))
    assert dp.chunk_rows(100, 4096) == [(0, 100)]
    with pytest.raises(ValueError):
        dp.chunk_rows(100, 0)


def test_take_utterances_trims_padding():
    cfg = wl.reduced(wl.CONFIGS["c2"], V=64, D=8, N=5, T_div=20, U_div=10, name="tk")
    b = wl.make_batch(cfg)
    idx = [3, 1]
    h, t, il, tl = dp.take_utterances(idx, b.hidden, b.targets, b.input_lengths, b.target_lengths)
    assert h.shape == (2, int(il.max()), 8) and t.shape[1] == max(1, int(tl.max()))
    np.testing.assert_array_equal(h[0, : il[0]], b.hidden[3, : il[0]])
    np.testing.assert_array_equal(t[1, : tl[1]], b.targets[1, : tl[1]])
    ht, tt, _, _ = dp.take_utterances(idx, torch.from_numpy(b.hidden), torch.from_numpy(b.targets),
                                      b.input_lengths, b.target_lengths)
    np.testing.assert_array_equal(ht.numpy(), h)
    np.testing.assert_array_equal(tt.numpy(), t)


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    from oracle import pruned_ctc_oracle as O
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfg = wl.reduced(wl.CONFIGS["c2"], V=96, D=12, N=5, T_div=12, U_div=8, name="dp")
    b = wl.make_batch(cfg, with_bias=True, permute_ids=True)
    mine = dp.shard_utterances(b.input_lengths, world)[rank]
    h, t, il, tl = dp.take_utterances(mine, b.hidden, b.targets, b.input_lengths, b.target_lengths)
    ref = O.pruned_ctc_reference(h, b.W, b.bias, t, il, tl, b.blank)
    dW = torch.from_numpy(ref["dW"].copy())
    db = torch.from_numpy(ref["db"].copy())
    dp.allreduce_rows(dW, dp.chunk_rows(cfg.V, 40), dbias=db)      # three chunks, the last one ragged
    out[rank] = dict(idx=mine, loss=ref["loss"], dH=ref["dH"], dW=dW.numpy(), db=db.numpy(), U=ref["U"])
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_sum_dW_per_chunk_and_keep_loss_and_dH_local():
    from oracle import pruned_ctc_oracle as O
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Manager().dict()
    port = 31500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(180)
        assert p.exitcode == 0
    cfg = wl.reduced(wl.CONFIGS["c2"], V=96, D=12, N=5, T_div=12, U_div=8, name="dp")
    b = wl.make_batch(cfg, with_bias=True, permute_ids=True)
    full = O.pruned_ctc_reference(b.hidden, b.W, b.bias, b.targets, b.input_lengths, b.target_lengths, b.blank)
    for r in range(world):
        o = out[r]
        np.testing.assert_allclose(o["dW"], full["dW"], rtol=1e-10, atol=1e-12)   # every rank holds the sum
        np.testing.assert_allclose(o["db"], full["db"], rtol=1e-10, atol=1e-12)
        np.testing.assert_allclose(o["loss"], full["loss"][o["idx"]], rtol=1e-12)
        for k, n in enumerate(o["idx"]):
            Tn = int(b.input_lengths[n])
            np.testing.assert_allclose(o["dH"][k, :Tn], full["dH"][n, :Tn], rtol=1e-10, atol=1e-14)
        assert set(o["U"].tolist()) <= set(full["U"].tolist())      # a rank's subset is its own, smaller one
    assert set(out[0]["U"].tolist()) != set(out[1]["U"].tolist())
