"""ctypes binding of libprunedctc: argument marshalling only.

Every step of the computation runs in the library's CUDA kernels; torch is
used for device memory and the current stream.  There is no CPU path: calls
raise if the library is missing or returns an error status.
"""

from __future__ import annotations

import ctypes
import os
from typing import Optional

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libprunedctc.so")

PCTC_BF16, PCTC_FP32 = 0, 1
GEMM_AUTO, GEMM_SIMT = 0, 1
UTT_INFEASIBLE, UTT_NONFINITE, UTT_BAD_TARGET, UTT_SUBSET_OVERFLOW = 1, 2, 4, 8

EXPORTS = ("pctc_workspace_bytes", "pctc_chunk_width", "pruned_ctc_fwd_bwd", "pruned_ctc_fwd_bwd_traced", "pctc_gemm_bf16",
           "pctc_workspace_status", "pctc_status_string", "pctc_host_call_scratch_bytes",
           "pruned_ctc_fwd_bwd_host", "pctc_subset_relabel_noalloc", "pctc_greedy_workspace_bytes",
           "pctc_greedy_decode", "pctc_topk_workspace_bytes", "pctc_topk_decode")
NOALLOC_MAX_V = 262144

PHASES = ("prep", "lse", "subset_logp", "dp", "dlogits", "dh", "dw", "dbias", "finish")


class Problem(ctypes.Structure):
    _fields_ = [
        ("N", ctypes.c_int32), ("T", ctypes.c_int32), ("D", ctypes.c_int32),
        ("V", ctypes.c_int64),
        ("dtype", ctypes.c_int32), ("blank_id", ctypes.c_int32),
        ("beam", ctypes.c_float),
        ("chunk", ctypes.c_int32), ("target_stride", ctypes.c_int32), ("gemm_path", ctypes.c_int32),
        ("skip_dW", ctypes.c_int32), ("accumulate_dW", ctypes.c_int32), ("forward_only", ctypes.c_int32),
        ("max_K", ctypes.c_int32),
        ("utt_weights", ctypes.c_void_p),
    ]


class TraceStruct(ctypes.Structure):
    _fields_ = [("events", ctypes.POINTER(ctypes.c_void_p)), ("capacity", ctypes.c_int32),
                ("used", ctypes.c_int32), ("kinds", ctypes.POINTER(ctypes.c_int32))]


class Trace:
    """Caller-owned CUDA events for pruned_ctc_fwd_bwd_traced (one timeline per call)."""

    def __init__(self, capacity: int):
        import torch

        self.capacity = int(capacity)
        self.events = [torch.cuda.Event(enable_timing=True) for _ in range(self.capacity)]
        for e in self.events:          # torch creates the CUDA event at its first record
            e.record()
        torch.cuda.synchronize()
        self._handles = (ctypes.c_void_p * self.capacity)(*[int(e.cuda_event) for e in self.events])
        self._kinds = (ctypes.c_int32 * self.capacity)()
        self.struct = TraceStruct(ctypes.cast(self._handles, ctypes.POINTER(ctypes.c_void_p)), self.capacity, 0,
                                  ctypes.cast(self._kinds, ctypes.POINTER(ctypes.c_int32)))

    def spans(self):
        """[(phase index, milliseconds)] of the last call; synchronise the stream first."""
        n = self.struct.used
        return [(int(self._kinds[i]), self.events[i].elapsed_time(self.events[i + 1])) for i in range(n - 1)]

    @staticmethod
    def capacity_for(V: int, chunk: int) -> int:
        return 12 + 4 * ((V + chunk - 1) // chunk)


class PctcError(RuntimeError):
    def __init__(self, status: int, what: str):
        super().__init__(f"{what}: status {status} ({status_string(status)})")
        self.status = status


_lib = None


def load() -> ctypes.CDLL:
    """Load the shared library (no build here; see build.build())."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: run paper_2609_33645_b200.build.build() first; "
                           "there is no fallback implementation")
    _lib = _configure(ctypes.CDLL(LIB_PATH))
    return _lib


def load_variant(path: str) -> ctypes.CDLL:
    """A test variant of the library (build.build_variant), loaded beside the regular one: call its
    entry points directly, e.g. ``gemm_bf16(..., lib=load_variant(path))``."""
    if not os.path.exists(path):
        raise RuntimeError(f"{path} is missing: run paper_2609_33645_b200.build.build_variant() first")
    return _configure(ctypes.CDLL(path))


def _configure(lib: ctypes.CDLL) -> ctypes.CDLL:
    vp, i32p = ctypes.c_void_p, ctypes.POINTER(ctypes.c_int32)
    lib.pctc_workspace_bytes.restype = ctypes.c_int
    lib.pctc_workspace_bytes.argtypes = [ctypes.POINTER(Problem), i32p, i32p, ctypes.POINTER(ctypes.c_size_t)]
    lib.pctc_chunk_width.restype = ctypes.c_int
    lib.pctc_chunk_width.argtypes = [ctypes.POINTER(Problem), i32p, i32p, i32p, i32p]
    lib.pruned_ctc_fwd_bwd.restype = ctypes.c_int
    lib.pruned_ctc_fwd_bwd.argtypes = [ctypes.POINTER(Problem), vp, vp, vp, vp, i32p, i32p,
                                       vp, vp, vp, vp, vp, vp, vp, vp, vp, ctypes.c_size_t, vp]
    lib.pruned_ctc_fwd_bwd_traced.restype = ctypes.c_int
    lib.pruned_ctc_fwd_bwd_traced.argtypes = lib.pruned_ctc_fwd_bwd.argtypes + [ctypes.POINTER(TraceStruct)]
    lib.pruned_ctc_fwd_bwd_host.restype = ctypes.c_int
    lib.pruned_ctc_fwd_bwd_host.argtypes = lib.pruned_ctc_fwd_bwd.argtypes
    lib.pctc_host_call_scratch_bytes.restype = ctypes.c_int
    lib.pctc_host_call_scratch_bytes.argtypes = [ctypes.POINTER(Problem), i32p, i32p, ctypes.c_int32,
                                                 ctypes.POINTER(ctypes.c_size_t)]
    lib.pctc_subset_relabel_noalloc.restype = ctypes.c_int
    lib.pctc_subset_relabel_noalloc.argtypes = [vp, vp, ctypes.c_int32, ctypes.c_int32, ctypes.c_int64,
                                                ctypes.c_int32, vp, vp, vp, vp, vp]
    lib.pctc_greedy_workspace_bytes.restype = ctypes.c_int
    lib.pctc_greedy_workspace_bytes.argtypes = [ctypes.POINTER(Problem), i32p, ctypes.POINTER(ctypes.c_size_t)]
    lib.pctc_greedy_decode.restype = ctypes.c_int
    lib.pctc_greedy_decode.argtypes = [ctypes.POINTER(Problem), vp, vp, vp, i32p, vp, vp, vp, vp, ctypes.c_size_t, vp]
    lib.pctc_topk_workspace_bytes.restype = ctypes.c_int
    lib.pctc_topk_workspace_bytes.argtypes = [ctypes.POINTER(Problem), i32p, ctypes.c_int32,
                                              ctypes.POINTER(ctypes.c_size_t)]
    lib.pctc_topk_decode.restype = ctypes.c_int
    lib.pctc_topk_decode.argtypes = [ctypes.POINTER(Problem), vp, vp, vp, i32p, ctypes.c_int32, vp, vp, vp,
                                     ctypes.c_size_t, vp]
    lib.pctc_gemm_bf16.restype = ctypes.c_int
    lib.pctc_gemm_bf16.argtypes = [vp, vp, vp, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
                                   ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, vp, vp]
    lib.pctc_workspace_status.restype = ctypes.c_int
    lib.pctc_workspace_status.argtypes = [vp, vp, i32p]
    lib.pctc_status_string.restype = ctypes.c_char_p
    lib.pctc_status_string.argtypes = [ctypes.c_int]
    return lib


def status_string(status: int) -> str:
    return load().pctc_status_string(int(status)).decode()


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a), dtype=np.int32)


def _ptr_i32(a: np.ndarray):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))


def make_problem(N, T, D, V, dtype, blank_id, beam=0.0, chunk=0, target_stride=0, gemm_path=GEMM_AUTO,
                 skip_dW=False, accumulate_dW=False, utt_weights_ptr=None, max_K=0, forward_only=False) -> Problem:
    return Problem(int(N), int(T), int(D), int(V), int(dtype), int(blank_id), float(beam), int(chunk),
                   int(target_stride), int(gemm_path), int(bool(skip_dW)), int(bool(accumulate_dW)),
                   int(bool(forward_only)), int(max_K), utt_weights_ptr)


def workspace_bytes(problem: Problem, input_lengths, target_lengths) -> int:
    il, tl = _i32(input_lengths), _i32(target_lengths)
    out = ctypes.c_size_t(0)
    st = load().pctc_workspace_bytes(ctypes.byref(problem), _ptr_i32(il), _ptr_i32(tl), ctypes.byref(out))
    if st != 0:
        raise PctcError(st, "pctc_workspace_bytes")
    return int(out.value)


def chunk_width(problem: Problem, input_lengths, target_lengths):
    """(C, number of chunks) the library will use for this problem (its default when problem.chunk is 0)."""
    il, tl = _i32(input_lengths), _i32(target_lengths)
    c, n = ctypes.c_int32(0), ctypes.c_int32(0)
    st = load().pctc_chunk_width(ctypes.byref(problem), _ptr_i32(il), _ptr_i32(tl), ctypes.byref(c), ctypes.byref(n))
    if st != 0:
        raise PctcError(st, "pctc_chunk_width")
    return int(c.value), int(n.value)


def _dptr(t) -> Optional[int]:
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def pruned_ctc_fwd_bwd(hidden, W, bias, targets, input_lengths, target_lengths, blank_id, *, beam=0.0,
                       chunk=0, gemm_path=GEMM_AUTO, workspace=None, out=None, check_status=False,
                       trace: Optional[Trace] = None, skip_dW=False, accumulate_dW=False, utt_weights=None,
                       max_K=0, forward_only=False, lib_handle=None):
    """Algorithm 1 on CUDA tensors.

    hidden [N,T,D], W [V,D], bias [V] or None (bf16 or fp32, same dtype), targets
    [N,stride] int32 on the device; input_lengths / target_lengths are host
    integer sequences.  Returns a dict of device tensors: loss [N] fp32, dH, dW,
    dbias (or None), subset [1+sum U], K [1], relabeled [N,stride], flags [N],
    plus "workspace" (reusable) and "workspace_bytes".  `out` may carry
    preallocated tensors from an earlier call with the same shapes.
    skip_dW: frozen head, dW is None.  accumulate_dW: add into out["dW"] / out["dbias"].
    utt_weights: fp32 CUDA tensor [N] of upstream gradients of the utterance losses.
    lib_handle: a test variant of the library from load_variant() instead of the regular one.
    """
    import torch

    lib = lib_handle or load()
    if not (hidden.is_cuda and W.is_cuda and hidden.is_contiguous() and W.is_contiguous()):
        raise ValueError("hidden and W must be contiguous CUDA tensors")
    if hidden.dtype != W.dtype or hidden.dtype not in (torch.bfloat16, torch.float32):
        raise ValueError("hidden and W must both be bf16 or both fp32")
    dt = PCTC_BF16 if hidden.dtype == torch.bfloat16 else PCTC_FP32
    N, T, D = hidden.shape
    V = W.shape[0]
    il, tl = _i32(input_lengths), _i32(target_lengths)
    if targets is None:
        targets = torch.zeros((N, 1), dtype=torch.int32, device=hidden.device)
    if targets.dtype != torch.int32 or not targets.is_contiguous():
        raise ValueError("targets must be a contiguous int32 CUDA tensor")
    stride = targets.shape[1]
    if utt_weights is not None and (utt_weights.dtype != torch.float32 or tuple(utt_weights.shape) != (N,)):
        raise ValueError("utt_weights must be an fp32 CUDA tensor of shape [N]")
    prob = make_problem(N, T, D, V, dt, blank_id, beam, chunk, stride, gemm_path, skip_dW, accumulate_dW,
                        None if utt_weights is None else utt_weights.data_ptr(), max_K, forward_only)
    need = workspace_bytes(prob, il, tl)          # host-only arithmetic, the same in every variant
    dev = hidden.device
    if workspace is None or workspace.numel() < need:
        workspace = torch.empty(need, dtype=torch.uint8, device=dev)
    o = out or {}

    def buf(name, shape, dtype):
        t = o.get(name)
        if t is None or tuple(t.shape) != tuple(shape) or t.dtype != dtype:
            t = torch.empty(shape, dtype=dtype, device=dev)
        return t

    ksum = int(tl.sum()) + 1
    if max_K:
        ksum = min(ksum, int(max_K))
    res = dict(
        loss=buf("loss", (N,), torch.float32),
        dH=None if forward_only else buf("dH", (N, T, D), hidden.dtype),
        dW=None if (skip_dW or forward_only) else buf("dW", (V, D), hidden.dtype),
        dbias=buf("dbias", (V,), hidden.dtype) if (bias is not None and not forward_only) else None,
        subset=buf("subset", (ksum,), torch.int32),
        K=buf("K", (1,), torch.int32),
        relabeled=buf("relabeled", (N, stride), torch.int32),
        flags=buf("flags", (N,), torch.int32),
        workspace=workspace, workspace_bytes=need,
    )
    stream = ctypes.c_void_p(torch.cuda.current_stream(dev).cuda_stream)
    args = [ctypes.byref(prob), _dptr(hidden), _dptr(W), _dptr(bias), _dptr(targets), _ptr_i32(il), _ptr_i32(tl),
            _dptr(res["loss"]), _dptr(res["dH"]), _dptr(res["dW"]), _dptr(res["dbias"]),
            _dptr(res["subset"]), _dptr(res["K"]), _dptr(res["relabeled"]), _dptr(res["flags"]),
            _dptr(workspace), ctypes.c_size_t(workspace.numel()), stream]
    if trace is None:
        st = lib.pruned_ctc_fwd_bwd(*args)
    else:
        st = lib.pruned_ctc_fwd_bwd_traced(*args, ctypes.byref(trace.struct))
    if st != 0:
        raise PctcError(st, "pruned_ctc_fwd_bwd")
    if check_status:
        code = workspace_status(workspace, lib_handle=lib)
        if code != 0:
            raise PctcError(6 if code < 0x100 else 1, f"device status word {code:#x}")
    return res


def workspace_status(workspace, lib_handle=None) -> int:
    """Synchronise the current stream and return the device status word: 0 nothing to report, 1-4 a
    bounded wait gave up, 0x100 more selected classes than max_K, 0x201.. (debug build) a bad index."""
    import torch

    host = ctypes.c_int32(0)
    stream = ctypes.c_void_p(torch.cuda.current_stream(workspace.device).cuda_stream)
    st = (lib_handle or load()).pctc_workspace_status(_dptr(workspace), stream, ctypes.byref(host))
    if st not in (0, 1, 6):
        raise PctcError(st, "pctc_workspace_status")
    return int(host.value)


def gemm_bf16(A, B, m, n, k, a_mn_major=False, b_mn_major=False, gemm_path=GEMM_AUTO):
    """C[m,n] (fp32) = sum_k A(i,k) B(j,k) for bf16 CUDA tensors; see prunedctc.h."""
    import torch

    C = torch.empty((m, n), dtype=torch.float32, device=A.device)
    status = torch.zeros(64, dtype=torch.int32, device=A.device)
    stream = ctypes.c_void_p(torch.cuda.current_stream(A.device).cuda_stream)
    st = load().pctc_gemm_bf16(_dptr(A), _dptr(B), _dptr(C), m, n, k, int(a_mn_major), int(b_mn_major),
                               int(gemm_path), _dptr(status), stream)
    if st != 0:
        raise PctcError(st, "pctc_gemm_bf16")
    code = int(status[0].item())
    if code != 0:
        raise PctcError(6, f"device status word {code}")
    return C


def pruned_ctc_fwd_bwd_host(hidden, W, bias, targets, input_lengths, target_lengths, blank_id, *, beam=0.0,
                            chunk=0, gemm_path=GEMM_AUTO, scratch=None, out=None, device=None):
    """Algorithm 1 on HOST tensors (pinned torch CPU tensors): copies in, computes, copies out.

    Returns host tensors loss, dH, dW, dbias, subset, K, relabeled, flags (pinned; valid after the
    current stream has been synchronised) plus "scratch", the reusable device buffer.
    """
    import torch

    lib = load()
    dev = torch.device(device or "cuda:0")
    if hidden.is_cuda or W.is_cuda:
        raise ValueError("the host entry point takes CPU tensors")
    dt = PCTC_BF16 if hidden.dtype == torch.bfloat16 else PCTC_FP32
    N, T, D = hidden.shape
    V = W.shape[0]
    il, tl = _i32(input_lengths), _i32(target_lengths)
    stride = targets.shape[1]
    prob = make_problem(N, T, D, V, dt, blank_id, beam, chunk, stride, gemm_path)
    need = ctypes.c_size_t(0)
    st = lib.pctc_host_call_scratch_bytes(ctypes.byref(prob), _ptr_i32(il), _ptr_i32(tl),
                                          int(bias is not None), ctypes.byref(need))
    if st != 0:
        raise PctcError(st, "pctc_host_call_scratch_bytes")
    if scratch is None or scratch.numel() < need.value:
        scratch = torch.empty(need.value, dtype=torch.uint8, device=dev)
    o = out or {}

    def buf(name, shape, dtype):
        t = o.get(name)
        if t is None or tuple(t.shape) != tuple(shape) or t.dtype != dtype:
            t = torch.empty(shape, dtype=dtype, pin_memory=True)
        return t

    res = dict(
        loss=buf("loss", (N,), torch.float32), dH=buf("dH", (N, T, D), hidden.dtype),
        dW=buf("dW", (V, D), hidden.dtype),
        dbias=buf("dbias", (V,), hidden.dtype) if bias is not None else None,
        subset=buf("subset", (int(tl.sum()) + 1,), torch.int32), K=buf("K", (1,), torch.int32),
        relabeled=buf("relabeled", (N, stride), torch.int32), flags=buf("flags", (N,), torch.int32),
        scratch=scratch, scratch_bytes=int(need.value),
    )
    stream = ctypes.c_void_p(torch.cuda.current_stream(dev).cuda_stream)
    st = lib.pruned_ctc_fwd_bwd_host(
        ctypes.byref(prob), _dptr(hidden), _dptr(W), _dptr(bias), _dptr(targets), _ptr_i32(il), _ptr_i32(tl),
        _dptr(res["loss"]), _dptr(res["dH"]), _dptr(res["dW"]), _dptr(res["dbias"]),
        _dptr(res["subset"]), _dptr(res["K"]), _dptr(res["relabeled"]), _dptr(res["flags"]),
        _dptr(scratch), ctypes.c_size_t(scratch.numel()), stream)
    if st != 0:
        raise PctcError(st, "pruned_ctc_fwd_bwd_host")
    return res


def subset_relabel_noalloc(targets, target_lengths, V, blank_id, out):
    """Algorithm 1 lines 2-3 through the entry point that allocates nothing.

    For callers that may not allocate device memory: every buffer, including the
    outputs in `out` (subset, K, relabeled, flags: int32 CUDA tensors), is the
    caller's; the library's own scratch is a fixed array inside it, so V may be
    at most NOALLOC_MAX_V.  targets [N,stride] and target_lengths [N] are int32
    CUDA tensors.  Runs on the current stream; returns `out`.
    """
    import torch

    N, stride = targets.shape
    stream = ctypes.c_void_p(torch.cuda.current_stream(targets.device).cuda_stream)
    st = load().pctc_subset_relabel_noalloc(_dptr(targets), _dptr(target_lengths), int(N), int(stride), int(V),
                                            int(blank_id), _dptr(out["subset"]), _dptr(out["K"]),
                                            _dptr(out["relabeled"]), _dptr(out["flags"]), stream)
    if st != 0:
        raise PctcError(st, "pctc_subset_relabel_noalloc")
    return out


def greedy_decode(hidden, W, bias, input_lengths, blank_id, *, gemm_path=GEMM_AUTO, workspace=None):
    """Greedy CTC recognition: frame arg-max of the head, repeats merged, blanks dropped.

    Returns device tensors frame_labels [N,T] (-1 on padded frames), tokens [N,T] (padded with
    -1), token_lengths [N], and the reusable workspace.
    """
    import torch

    lib = load()
    dt = PCTC_BF16 if hidden.dtype == torch.bfloat16 else PCTC_FP32
    N, T, D = hidden.shape
    V = W.shape[0]
    il = _i32(input_lengths)
    prob = make_problem(N, T, D, V, dt, blank_id, gemm_path=gemm_path)
    need = ctypes.c_size_t(0)
    st = lib.pctc_greedy_workspace_bytes(ctypes.byref(prob), _ptr_i32(il), ctypes.byref(need))
    if st != 0:
        raise PctcError(st, "pctc_greedy_workspace_bytes")
    dev = hidden.device
    if workspace is None or workspace.numel() < need.value:
        workspace = torch.empty(need.value, dtype=torch.uint8, device=dev)
    frame_labels = torch.empty((N, T), dtype=torch.int32, device=dev)
    tokens = torch.empty((N, T), dtype=torch.int32, device=dev)
    token_lengths = torch.empty((N,), dtype=torch.int32, device=dev)
    stream = ctypes.c_void_p(torch.cuda.current_stream(dev).cuda_stream)
    st = lib.pctc_greedy_decode(ctypes.byref(prob), _dptr(hidden), _dptr(W), _dptr(bias), _ptr_i32(il),
                                _dptr(frame_labels), _dptr(tokens), _dptr(token_lengths), _dptr(workspace),
                                ctypes.c_size_t(workspace.numel()), stream)
    if st != 0:
        raise PctcError(st, "pctc_greedy_decode")
    return dict(frame_labels=frame_labels, tokens=tokens, token_lengths=token_lengths, workspace=workspace)


def topk_decode(hidden, W, bias, input_lengths, k, *, chunk=0, gemm_path=GEMM_AUTO, workspace=None):
    """The k best classes of every frame (k in 1, 2, 4, 8) and their log-probabilities under the
    full-vocabulary softmax: device tensors classes [N,T,k] int32 (-1 on padded frames) and logprobs
    [N,T,k] fp32 (-inf there), plus the reusable workspace."""
    import torch

    lib = load()
    dt = PCTC_BF16 if hidden.dtype == torch.bfloat16 else PCTC_FP32
    N, T, D = hidden.shape
    V = W.shape[0]
    il = _i32(input_lengths)
    prob = make_problem(N, T, D, V, dt, 0, chunk=chunk, gemm_path=gemm_path)
    need = ctypes.c_size_t(0)
    st = lib.pctc_topk_workspace_bytes(ctypes.byref(prob), _ptr_i32(il), int(k), ctypes.byref(need))
    if st != 0:
        raise PctcError(st, "pctc_topk_workspace_bytes")
    dev = hidden.device
    if workspace is None or workspace.numel() < need.value:
        workspace = torch.empty(need.value, dtype=torch.uint8, device=dev)
    classes = torch.empty((N, T, k), dtype=torch.int32, device=dev)
    logprobs = torch.empty((N, T, k), dtype=torch.float32, device=dev)
    stream = ctypes.c_void_p(torch.cuda.current_stream(dev).cuda_stream)
    st = lib.pctc_topk_decode(ctypes.byref(prob), _dptr(hidden), _dptr(W), _dptr(bias), _ptr_i32(il), int(k),
                              _dptr(classes), _dptr(logprobs), _dptr(workspace), ctypes.c_size_t(workspace.numel()),
                              stream)
    if st != 0:
        raise PctcError(st, "pctc_topk_decode")
    return dict(classes=classes, logprobs=logprobs, workspace=workspace)
