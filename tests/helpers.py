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


def assert_parity(gpu, ref, batch, *, tol=None, check_db=True):
    """Element-wise comparison of everything the call returns."""
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
    # padded frames and frames of excluded utterances are exactly zero
    for n in range(batch.cfg.N):
        Tn = int(batch.input_lengths[n])
        assert np.all(gpu["dH"][n, Tn:] == 0.0)
        if ref["flags"][n] != 0:
            assert np.all(gpu["dH"][n] == 0.0)
    return errs
