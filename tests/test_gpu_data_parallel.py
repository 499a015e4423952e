"""The data-parallel step on one GPU: a one-rank NCCL group runs the whole mechanism (events after
each chunk's dW kernel, the communication stream, one collective per chunk), and with one rank the
sum over ranks is the identity, so every output must equal the plain call's bit for bit."""

import os
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from paper_2609_33645_b200 import workloads as wl  # noqa: E402

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def group():
    import torch
    import torch.distributed as dist
    os.environ.setdefault("NCCL_NVLS_ENABLE", "0")
    port = 33500 + os.getpid() % 2000
    dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1,
                            device_id=torch.device("cuda", 0))
    yield dist.group.WORLD
    torch.cuda.synchronize()
    dist.destroy_process_group()


@pytest.mark.parametrize("chunk,with_bias,frozen", [(2048, True, False), (0, False, False), (1024, True, True)])
def test_one_rank_group_equals_plain_call(group, chunk, with_bias, frozen):
    import torch
    from paper_2609_33645_b200 import binding, data_parallel as dp
    binding.load()
    cfg = wl.reduced(wl.CONFIGS["c3"], V=8192 + 384, D=256, N=4, T_div=4, U_div=2, name="dp1")
    b = wl.make_batch(cfg, with_bias=with_bias, permute_ids=True)
    dev = torch.device("cuda:0")
    hidden = torch.from_numpy(b.hidden).to(dev).to(torch.bfloat16)
    W = torch.from_numpy(b.W).to(dev).to(torch.bfloat16)
    bias = None if b.bias is None else torch.from_numpy(b.bias).to(dev).to(torch.bfloat16)
    targets = torch.from_numpy(b.targets).to(dev)
    args = (hidden, W, bias, targets, b.input_lengths, b.target_lengths, b.blank)
    plain = binding.pruned_ctc_fwd_bwd(*args, chunk=chunk, skip_dW=frozen, check_status=True)
    torch.cuda.synchronize()
    comm = torch.cuda.Stream(dev)
    trace = None
    for _ in range(2):                                   # the second step reuses the events of the first
        res = dp.pruned_ctc_fwd_bwd_data_parallel(*args, group=group, comm_stream=comm, trace=trace, chunk=chunk,
                                                  skip_dW=frozen)
        trace = res["trace"]
        torch.cuda.synchronize()
        for k in ("loss", "dH", "dW", "dbias", "flags"):
            if plain[k] is None:
                assert res[k] is None
            else:
                assert torch.equal(res[k], plain[k]), k
    if not frozen:
        C, nchunks = binding.chunk_width(binding.make_problem(cfg.N, hidden.shape[1], cfg.D, cfg.V, binding.PCTC_BF16,
                                                               b.blank, 0.0, chunk, targets.shape[1]),
                                         b.input_lengths, b.target_lengths)
        assert len(dp.dw_ready_events(trace)) == nchunks == len(dp.chunk_rows(cfg.V, C))
