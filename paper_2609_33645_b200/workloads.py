"""Seeded synthetic batches with the shapes of the paper's workloads.

This module is input generation only: it holds none of the method's
arithmetic and is the one piece of code that both the CPU oracle's tests and
the CUDA path's tests/bench use, so that both see the same bits.

The paper measures on speech corpora with trained or randomly initialised
models; those are replaced here by random states and heads of the same shape:
head widths and vocabularies of the Zipformer-M head (D=512, V up to 180,000)
and of the Qwen3 family (D = 1,024 / 4,096 / 5,120, V = 151,936), frame counts
and transcript lengths in the ranges of each configuration, and Zipf-distributed
token ids so that the batch-union subset has a few hundred to a few thousand
classes and adjacent repeated labels occur.

Draw order for a batch (fixed, so a seed defines the batch):
frame counts T_n, target lengths U_n, tokens of each utterance in order,
hidden states, head weight, (bias, if requested).  Hidden states and weights
of bf16 configurations are rounded to bf16 (round to nearest even) and
returned as float32 arrays holding exactly those values.
"""

from __future__ import annotations

import dataclasses
from typing import Optional

import numpy as np


@dataclasses.dataclass(frozen=True)
class Config:
    name: str
    N: int
    T_lo: int
    T_hi: int
    D: int
    V: int
    dtype: str            # "bf16" or "fp32"
    U_lo: int
    U_hi: int
    zipf_s: Optional[float]   # None => uniform tokens on [1, V)
    rms_norm: bool = False    # per-frame RMS normalisation of hidden
    blank: int = 0
    seed: int = 0


# The five benchmark configurations (index i has seed 1000 + i).
CONFIGS = {
    "c1": Config("c1", N=2, T_lo=50, T_hi=50, D=64, V=1000, dtype="fp32",
                 U_lo=3, U_hi=10, zipf_s=None, seed=1001),
    "c2": Config("c2", N=16, T_lo=300, T_hi=500, D=512, V=180000, dtype="bf16",
                 U_lo=20, U_hi=100, zipf_s=1.1, seed=1002),
    "c3": Config("c3", N=8, T_lo=400, T_hi=750, D=1024, V=151936, dtype="bf16",
                 U_lo=50, U_hi=150, zipf_s=1.1, rms_norm=True, seed=1003),
    "c4": Config("c4", N=8, T_lo=800, T_hi=1500, D=4096, V=151936, dtype="bf16",
                 U_lo=100, U_hi=300, zipf_s=1.1, rms_norm=True, seed=1004),
    "c5": Config("c5", N=4, T_lo=1500, T_hi=3000, D=5120, V=151936, dtype="bf16",
                 U_lo=300, U_hi=600, zipf_s=1.0, rms_norm=True, seed=1005),
    # The paper's own resource benchmark (Appendix C.2): utterances of exactly 100 encoder frames,
    # 160 / 320 / 640 of them (16k / 32k / 64k frames), Zipformer-M head width, vocabulary swept
    # from 500 to 180,000 (use `reduced(cfg, V=...)` for the sweep).  Transcript lengths are not
    # stated; 10-30 tokens is about four seconds of speech at the usual subword rates.
    "g16k": Config("g16k", N=160, T_lo=100, T_hi=100, D=512, V=180000, dtype="bf16",
                   U_lo=10, U_hi=30, zipf_s=1.1, seed=1016),
    "g32k": Config("g32k", N=320, T_lo=100, T_hi=100, D=512, V=180000, dtype="bf16",
                   U_lo=10, U_hi=30, zipf_s=1.1, seed=1032),
    "g64k": Config("g64k", N=640, T_lo=100, T_hi=100, D=512, V=180000, dtype="bf16",
                   U_lo=10, U_hi=30, zipf_s=1.1, seed=1064),
}


def reduced(cfg: Config, *, V: Optional[int] = None, D: Optional[int] = None,
            N: Optional[int] = None, T_div: int = 1, U_div: int = 1,
            name: Optional[str] = None, **kw) -> Config:
    """A smaller variant of ``cfg`` (same distributions) for oracle-sized parity cases."""
    return dataclasses.replace(
        cfg,
        name=name or (cfg.name + "-reduced"),
        V=V or cfg.V, D=D or cfg.D, N=N or cfg.N,
        T_lo=max(1, cfg.T_lo // T_div), T_hi=max(1, cfg.T_hi // T_div),
        U_lo=max(0, cfg.U_lo // U_div), U_hi=max(0, cfg.U_hi // U_div),
        **kw)


@dataclasses.dataclass
class Batch:
    cfg: Config
    hidden: np.ndarray          # [N, T, D] float32 (bf16-representable for bf16 configs)
    W: np.ndarray               # [V, D]   float32 (same)
    bias: Optional[np.ndarray]  # [V] float32 or None
    targets: np.ndarray         # [N, stride] int32, rows padded with `pad_token`
    input_lengths: np.ndarray   # [N] int32
    target_lengths: np.ndarray  # [N] int32
    blank: int

    @property
    def M(self) -> int:
        return int(self.input_lengths.sum())

    @property
    def T(self) -> int:
        return int(self.hidden.shape[1])


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bf16 (ties to even); result stays float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    bits = x.view(np.uint32).astype(np.uint64)
    lsb = (bits >> 16) & 1
    rounded = ((bits + 0x7FFF + lsb) >> 16) << 16
    return rounded.astype(np.uint32).view(np.float32).reshape(x.shape)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """The uint16 bit patterns of bf16-representable float32 values."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    return (x.view(np.uint32) >> 16).astype(np.uint16).reshape(x.shape)


def _zipf_tokens(rng: np.random.Generator, cdf: np.ndarray, count: int) -> np.ndarray:
    u = rng.random(count)
    rank = np.searchsorted(cdf, u, side="left") + 1     # ranks 1..V-1
    return np.minimum(rank, cdf.shape[0]).astype(np.int64)


def make_batch(cfg: Config, *, seed: Optional[int] = None, with_bias: bool = False,
               permute_ids: bool = False, poison_padding: bool = False,
               target_stride: Optional[int] = None, pad_token: int = -1,
               normal_chunk: int = 1 << 24) -> Batch:
    """Generate one batch.

    ``permute_ids`` maps the non-blank ids through a seeded permutation so that
    the frequent tokens land in every vocabulary chunk instead of the first
    one.  ``poison_padding`` fills padded frames of ``hidden`` with large finite
    values (they must never influence a result); otherwise they are zero.
    With ``cfg.blank != 0`` the drawn id ``blank`` is swapped with id 0 so that
    targets stay blank-free.
    """
    rng = np.random.Generator(np.random.PCG64(cfg.seed if seed is None else seed))
    N, D, V = cfg.N, cfg.D, cfg.V

    T_n = rng.integers(cfg.T_lo, cfg.T_hi, size=N, endpoint=True).astype(np.int32)
    U_n = rng.integers(cfg.U_lo, cfg.U_hi, size=N, endpoint=True).astype(np.int32)

    if cfg.zipf_s is not None:
        w = np.arange(1, V, dtype=np.float64) ** (-cfg.zipf_s)
        cdf = np.cumsum(w)
        cdf /= cdf[-1]
    rows = []
    for n in range(N):
        u = int(U_n[n])
        if cfg.zipf_s is None:
            tok = rng.integers(1, V, size=u).astype(np.int64)
        else:
            tok = _zipf_tokens(rng, cdf, u)
        rows.append(tok)

    T = int(T_n.max())
    hidden = np.zeros((N, T, D), dtype=np.float32)
    for n in range(N):
        t = int(T_n[n])
        h = rng.standard_normal((t, D), dtype=np.float32)
        if cfg.rms_norm:
            h = h / np.sqrt(np.mean(h.astype(np.float64) ** 2, axis=1, keepdims=True)).astype(np.float32)
        hidden[n, :t] = h

    W = np.empty((V, D), dtype=np.float32)
    scale = np.float32(D ** -0.5)
    flat = W.reshape(-1)
    for s in range(0, flat.shape[0], normal_chunk):
        e = min(flat.shape[0], s + normal_chunk)
        flat[s:e] = rng.standard_normal(e - s, dtype=np.float32) * scale

    bias = None
    if with_bias:
        bias = (rng.standard_normal(V, dtype=np.float32) * np.float32(0.5))

    if permute_ids:
        perm = np.concatenate([[0], 1 + rng.permutation(V - 1)]).astype(np.int64)
        rows = [perm[r] for r in rows]
    if cfg.blank != 0:
        b = cfg.blank
        rows = [np.where(r == b, 0, r) for r in rows]   # id `blank` <-> id 0

    if poison_padding:
        for n in range(N):
            hidden[n, int(T_n[n]):] = np.float32(3.0e4) * (1 - 2 * (n % 2))

    if cfg.dtype == "bf16":
        hidden = round_to_bf16(hidden)
        W = round_to_bf16(W)
        if bias is not None:
            bias = round_to_bf16(bias)

    stride = int(target_stride if target_stride is not None else max(1, int(U_n.max())))
    targets = np.full((N, stride), pad_token, dtype=np.int32)
    for n in range(N):
        targets[n, : int(U_n[n])] = rows[n].astype(np.int32)

    return Batch(cfg=cfg, hidden=hidden, W=W, bias=bias, targets=targets,
                 input_lengths=T_n, target_lengths=U_n, blank=cfg.blank)
