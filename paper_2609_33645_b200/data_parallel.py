"""Utterance-sharded data parallelism for the Pruned-CTC head (one process per GPU).

Every rank holds the full head W[V, D] (the head is replicated, not sharded:
Appendix B.1) and a slice of the batch's utterances.  A rank builds the selected
class set U of *its own* utterances: by Proposition 1 any superset of an
utterance's labels gives that utterance's exact loss and gradient, so per-rank
subsets change nothing.  Losses and dH stay local.  The one exchange step is the
sum over ranks of dW (and db): the rows of a vocabulary chunk are final as soon
as that chunk's dW kernel has finished (Algorithm 1, line 15), so their all-reduce
is issued on a communication stream right then and overlaps the chunks that
are still being computed.  With a frozen head (Section 4.2) nothing is exchanged.

torch.distributed carries the collective (NCCL between GPUs; gloo on CPU tensors,
which is how the host logic here is tested without a GPU).
"""

from __future__ import annotations

from typing import List, Optional, Sequence, Tuple

import numpy as np

from . import binding

PHASE_DW = binding.PHASES.index("dw")


def shard_utterances(input_lengths: Sequence[int], world: int) -> List[np.ndarray]:
    """Split utterances over ranks so that the frame counts per rank are as even as a greedy pass gets.

    The step time of a rank grows with its number of frames M_r and the job waits for the slowest
    rank, so the longest utterances are placed first, each on the rank that holds the fewest frames
    so far (ties: lowest rank).  Returns, per rank, the ascending utterance indices it owns; every
    utterance is owned exactly once.  Ranks may end up empty only when world > N.
    """
    T = np.asarray(input_lengths, dtype=np.int64)
    if world < 1:
        raise ValueError("world must be >= 1")
    load = np.zeros(world, dtype=np.int64)
    owned: List[List[int]] = [[] for _ in range(world)]
    for n in sorted(range(T.shape[0]), key=lambda i: (-int(T[i]), i)):
        r = int(np.argmin(load))
        owned[r].append(n)
        load[r] += T[n]
    return [np.array(sorted(o), dtype=np.int64) for o in owned]


def take_utterances(idx, hidden, targets, input_lengths, target_lengths):
    """The slice of a batch owned by one rank, trimmed to its own longest utterance and transcript.

    Works on numpy arrays and on torch tensors alike (hidden [N,T,D], targets [N,stride]); lengths
    are host integer sequences.  Returns (hidden, targets, input_lengths, target_lengths).
    """
    idx = np.asarray(idx, dtype=np.int64)
    il = np.asarray(input_lengths, dtype=np.int32)[idx]
    tl = np.asarray(target_lengths, dtype=np.int32)[idx]
    if idx.size == 0:
        raise ValueError("a rank needs at least one utterance")
    Tmax, Umax = int(il.max()), max(1, int(tl.max()))
    sel = idx if isinstance(hidden, np.ndarray) else idx.tolist()
    h = hidden[sel][:, :Tmax]
    t = targets[sel][:, :Umax]
    if not isinstance(hidden, np.ndarray):
        h, t = h.contiguous(), t.contiguous()
    else:
        h, t = np.ascontiguousarray(h), np.ascontiguousarray(t)
    return h, t, il, tl


def chunk_rows(V: int, chunk: int) -> List[Tuple[int, int]]:
    """Row ranges [v0, v1) of dW written by the successive vocabulary chunks."""
    if V <= 0 or chunk <= 0:
        raise ValueError("V and chunk must be positive")
    return [(v0, min(V, v0 + chunk)) for v0 in range(0, V, chunk)]


def dw_ready_events(trace: "binding.Trace") -> list:
    """For each vocabulary chunk, the event of the last call's timeline that follows its dW kernel."""
    n = trace.struct.used
    return [trace.events[i + 1] for i in range(n - 1) if int(trace._kinds[i]) == PHASE_DW]


def allreduce_rows(dW, rows: Sequence[Tuple[int, int]], ready: Optional[Sequence] = None, *, group=None,
                   comm_stream=None, dbias=None):
    """Sum dW over the ranks of `group`, one collective per chunk of rows, each as early as it may start.

    dW: [V, D] tensor (reduced in place).  rows: the chunks' row ranges.  ready: for CUDA tensors, one
    event per chunk after which those rows are final; the collective of a chunk waits for its event
    on `comm_stream`, not for the whole backward pass, and the current stream waits for the
    communication stream at the end.  CPU tensors are reduced in order with no stream logic.  dbias,
    if given, is reduced whole after the last chunk.  Sums in dW's own dtype (bf16 stays bf16, as a
    bf16 trainer's gradient all-reduce does).
    """
    import torch
    import torch.distributed as dist

    if not dW.is_cuda:
        for v0, v1 in rows:
            dist.all_reduce(dW[v0:v1], group=group)
        if dbias is not None:
            dist.all_reduce(dbias, group=group)
        return
    if ready is None or len(ready) != len(rows):
        raise ValueError("one ready-event per chunk of rows is required for CUDA tensors")
    cur = torch.cuda.current_stream(dW.device)
    comm = comm_stream if comm_stream is not None else torch.cuda.Stream(dW.device)
    for (v0, v1), ev in zip(rows, ready):
        comm.wait_event(ev)
        with torch.cuda.stream(comm):
            dist.all_reduce(dW[v0:v1], group=group)
    if dbias is not None:
        comm.wait_stream(cur)
        with torch.cuda.stream(comm):
            dist.all_reduce(dbias, group=group)
    dW.record_stream(comm)
    cur.wait_stream(comm)


def pruned_ctc_fwd_bwd_data_parallel(hidden, W, bias, targets, input_lengths, target_lengths, blank_id, *,
                                     group=None, comm_stream=None, trace: Optional["binding.Trace"] = None,
                                     sync: bool = True, **kw):
    """Algorithm 1 on this rank's utterances, then dW (and db) summed over the ranks of `group`.

    Arguments and result as `binding.pruned_ctc_fwd_bwd` (this rank's slice of the batch; W and bias
    are the full, replicated head).  `sync=False` skips the exchange (a micro-batch of a gradient
    accumulation that is not the last one: pass accumulate_dW=True and reduce once at the end).
    With skip_dW or forward_only there is nothing to exchange except db.  `trace` may be passed to
    reuse its events between steps; it needs `Trace.capacity_for(V, chunk)` entries.
    """
    import torch
    import torch.distributed as dist

    V = W.shape[0]
    N, T, D = hidden.shape
    dt = binding.PCTC_BF16 if hidden.dtype == torch.bfloat16 else binding.PCTC_FP32
    prob = binding.make_problem(N, T, D, V, dt, blank_id, kw.get("beam", 0.0), kw.get("chunk", 0),
                                targets.shape[1], kw.get("gemm_path", binding.GEMM_AUTO))
    chunk, nchunks = binding.chunk_width(prob, input_lengths, target_lengths)
    if trace is None:
        trace = binding.Trace(12 + 4 * nchunks)
    res = binding.pruned_ctc_fwd_bwd(hidden, W, bias, targets, input_lengths, target_lengths, blank_id,
                                     trace=trace, **kw)
    res["trace"] = trace
    if not sync or kw.get("forward_only") or not dist.is_initialized():
        return res
    if res.get("dW") is not None:
        ready = dw_ready_events(trace)
        allreduce_rows(res["dW"], chunk_rows(V, chunk), ready, group=group, comm_stream=comm_stream,
                       dbias=res.get("dbias"))
    elif res.get("dbias") is not None:
        dist.all_reduce(res["dbias"], group=group)
    return res
