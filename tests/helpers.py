"""Shared helpers of the GPU parity tests: run a generated batch through the
C-ABI library and through the oracle, and measure the errors the way the
paper's validation does (Appendix B.2: norm of the difference over the norm of
the reference; Frobenius for matrices)."""

import numpy as np

from oracle import pruned_ctc_oracle as O

TOL = {  # (per-utterance loss relative error, gradient relative Frobenius error)
    "bf16": (2e-3, 1e-2),
    "fp32": (1e-5, 1e-4),
}


def rel_fro(x, ref):
    x = np.asarray(x, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    den = np.linalg.norm(ref.ravel())
    num = np.linalg.norm((x - ref).ravel())
    return num / den if den > 0 else num


def run_gpu(binding, batch, *, beam=0.0, chunk=0, gemm_path=0, check_status=True, utt_weights=None, **kw):
    """kw goes to binding.pruned_ctc_fwd_bwd (skip_dW, max_K, lib_handle, ...)."""
    import torch

    dev = torch.device("cuda:0")
    tdt = torch.bfloat16 if batch.cfg.dtype == "bf16" else torch.float32
    hidden = torch.from_numpy(batch.hidden).to(dev).to(tdt).contiguous()
    W = torch.from_numpy(batch.W).to(dev).to(tdt).contiguous()
    bias = None if batch.bias is None else torch.from_numpy(batch.bias).to(dev).to(tdt).contiguous()
    targets = torch.from_numpy(batch.targets).to(dev).contiguous()
    if utt_weights is not None:
        utt_weights = torch.tensor(np.asarray(utt_weights), dtype=torch.float32, device=dev)
    res = binding.pruned_ctc_fwd_bwd(hidden, W, bias, targets, batch.input_lengths, batch.target_lengths,
                                     batch.blank, beam=beam, chunk=chunk, gemm_path=gemm_path,
                                     check_status=check_status, utt_weights=utt_weights, **kw)
    torch.cuda.synchronize()
    out = {}
    for k, v in res.items():
        if hasattr(v, "detach") and k != "workspace":
            out[k] = v.detach().float().cpu().numpy() if v.is_floating_point() else v.cpu().numpy()
        else:
            out[k] = v
    return out


def run_oracle(batch, *, beam=None, **kw):
    """kw: utt_weights, dW_rows, dH_for, want_dW (see the oracle)."""
    return O.pruned_ctc_reference(batch.hidden, batch.W, batch.bias, batch.targets, batch.input_lengths,
                                  batch.target_lengths, batch.blank, beam=beam, **kw)


BLOCK = 256          # rows of dW / columns of dH per block of the block-wise checks
BLOCK_SLACK = 3.0    # a block may miss the whole-matrix tolerance by this factor
BLOCK_FLOOR = 1e-3   # blocks whose reference norm is below this share of an average block's are skipped


def _blockwise(x, ref, axis, what, tol, errs):
    """Relative Frobenius error of every BLOCK-wide slab of `x` along `axis` (Appendix B.2's metric,
    applied to parts of the matrix so that a part that is wrong cannot hide in the norm of the whole)."""
    x = np.asarray(x, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    n = ref.shape[axis]
    nblocks = (n + BLOCK - 1) // BLOCK
    whole = np.linalg.norm(ref.ravel())
    floor = BLOCK_FLOOR * whole / np.sqrt(max(1, nblocks))
    worst = 0.0
    for b in range(nblocks):
        sl = [slice(None)] * ref.ndim
        sl[axis] = slice(b * BLOCK, min(n, (b + 1) * BLOCK))
        r = ref[tuple(sl)]
        den = np.linalg.norm(r.ravel())
        if den <= floor:
            continue
        e = np.linalg.norm((x[tuple(sl)] - r).ravel()) / den
        worst = max(worst, e)
        assert e <= tol, (what, "block", b, e)
    errs[what + " worst block"] = worst


def assert_parity(gpu, ref, batch, *, tol=None, check_db=True, chunk=None):
    """Comparison of everything the call returns with the oracle.

    Integer outputs bit for bit; every per-utterance loss; the gradients by relative Frobenius error
    of the whole matrix AND of its parts, since the whole-matrix norm is dominated by the few selected
    rows of dW (Eq. "grad-full": the rows outside U carry only the dense softmax term):
      dW  restricted to the rows outside U, at the whole-matrix tolerance;
          every block of 256 rows, and the rows outside U of every such block, at 3x the tolerance;
      dH  every utterance at the whole-matrix tolerance; every block of 256 columns at 3x;
      db  (with a bias) the classes outside U, and every block of `chunk` classes (256 if not given).
    Blocks whose reference norm is negligible next to an average block are skipped.
    """
    loss_tol, grad_tol = tol or TOL[batch.cfg.dtype]
    K = ref["K"]
    # integer outputs: bit-exact
    assert int(gpu["K"][0]) == K
    np.testing.assert_array_equal(gpu["subset"][:K], ref["U"])
    np.testing.assert_array_equal(gpu["relabeled"], ref["relabeled"])
    np.testing.assert_array_equal(gpu["flags"], ref["flags"])
    # per-utterance loss
    for n in range(batch.cfg.N):
        if ref["loss"][n] == 0.0:
            assert gpu["loss"][n] == 0.0
        else:
            assert abs(gpu["loss"][n] - ref["loss"][n]) <= loss_tol * abs(ref["loss"][n]), (n, gpu["loss"][n], ref["loss"][n])
    errs = {"dH": rel_fro(gpu["dH"], ref["dH"])}
    if gpu.get("dW") is not None:
        errs["dW"] = rel_fro(gpu["dW"], ref["dW"])
    if check_db and batch.bias is not None:
        errs["db"] = rel_fro(gpu["dbias"], ref["db"])
    for k, e in errs.items():
        assert e <= grad_tol, (k, e)

    # ---- the parts ----
    off = np.ones(batch.cfg.V, dtype=bool)          # classes outside U
    off[np.asarray(ref["U"], dtype=np.int64)] = False
    block_tol = BLOCK_SLACK * grad_tol
    if gpu.get("dW") is not None:
        gW = np.asarray(gpu["dW"], dtype=np.float64)
        rW = np.asarray(ref["dW"], dtype=np.float64)
        if off.any() and np.linalg.norm(rW[off]) > 0:
            errs["dW off-support"] = rel_fro(gW[off], rW[off])
            assert errs["dW off-support"] <= grad_tol, ("dW off-support", errs["dW off-support"])
        _blockwise(gW, rW, 0, "dW", block_tol, errs)
        _blockwise(gW * off[:, None], rW * off[:, None], 0, "dW off-support", block_tol, errs)
    worst = 0.0
    for n in range(batch.cfg.N):
        if np.linalg.norm(ref["dH"][n]) > 0:
            e = rel_fro(gpu["dH"][n], ref["dH"][n])
            worst = max(worst, e)
            assert e <= grad_tol, ("dH utterance", n, e)
    errs["dH worst utterance"] = worst
    _blockwise(gpu["dH"], ref["dH"], 2, "dH", block_tol, errs)
    if check_db and batch.bias is not None:
        gb = np.asarray(gpu["dbias"], dtype=np.float64)
        rb = np.asarray(ref["db"], dtype=np.float64)
        if off.any() and np.linalg.norm(rb[off]) > 0:
            errs["db off-support"] = rel_fro(gb[off], rb[off])
            assert errs["db off-support"] <= grad_tol, ("db off-support", errs["db off-support"])
        # db[v] = sum over frames of w_m (p - gamma): with utterance weights of both signs a block can cancel
        # to far below the size of its terms, so a block's error is taken relative to its own norm or to an
        # average block's, whichever is larger (a dead stretch of typical size still reads an error of one)
        step = int(chunk) if chunk else BLOCK
        nblocks = max(1, (batch.cfg.V + step - 1) // step)
        avg = np.linalg.norm(rb) / np.sqrt(nblocks)
        for v0 in range(0, batch.cfg.V, step):
            r = rb[v0:v0 + step]
            den = max(np.linalg.norm(r), avg)
            if den > 0:
                e = np.linalg.norm(gb[v0:v0 + step] - r) / den
                assert e <= block_tol, ("db block", v0, e)

    # padded frames and frames of excluded utterances are exactly zero
    for n in range(batch.cfg.N):
        Tn = int(batch.input_lengths[n])
        assert np.all(gpu["dH"][n, Tn:] == 0.0)
        if ref["flags"][n] != 0:
            assert np.all(gpu["dH"][n] == 0.0)
    return errs
