"""GPU parity: the CUDA library against the float64 oracle, element by element,
on seeded batches small enough for the oracle (several tiles and ragged tails in
every dimension), for both arithmetic paths and the edge cases of the method."""

import dataclasses

import numpy as np
import pytest

from paper_2609_33645_b200 import workloads as wl
from tests import helpers as H

pytestmark = pytest.mark.gpu

SIMT, AUTO = 1, 0


def small(name, **kw):
    return wl.reduced(wl.CONFIGS[name], name=name + "-small", **kw)


def test_c1_fp32_full_config(lib):
    batch = wl.make_batch(wl.CONFIGS["c1"])
    gpu = H.run_gpu(lib, batch)
    ref = H.run_oracle(batch)
    errs = H.assert_parity(gpu, ref, batch)
    assert max(errs.values()) < 1e-4
    # and against the stored oracle values (tests/golden/c1_oracle.json)
    import json, os
    gold = json.load(open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "c1_oracle.json")))
    np.testing.assert_allclose(gpu["loss"], gold["loss"], rtol=1e-5)
    assert list(gpu["subset"][: gold["K"]]) == gold["U"]


def test_fp32_with_bias_ragged_chunks_blank_nonzero(lib):
    cfg = dataclasses.replace(wl.CONFIGS["c1"], name="c1-var", N=5, T_lo=9, T_hi=70, V=1531, D=72, blank=17,
                              U_lo=0, U_hi=12, seed=77)
    batch = wl.make_batch(cfg, with_bias=True, poison_padding=True)
    gpu = H.run_gpu(lib, batch, chunk=500)
    ref = H.run_oracle(batch)
    H.assert_parity(gpu, ref, batch)
    assert abs(float(gpu["dbias"].sum())) < 1e-3       # every frame's dlogits sum to zero


@pytest.mark.parametrize("path", [SIMT, AUTO])
@pytest.mark.parametrize("name,kw,chunk", [
    ("c2", dict(V=8192, N=6, T_div=4), 0),              # D=512, several row and column tiles, default chunk
    ("c3", dict(V=12288 + 384, D=256, N=4, T_div=4, U_div=2), 4096),   # ragged last chunk, RMS-normalised frames
])
def test_bf16_reduced_configs(lib, path, name, kw, chunk):
    batch = wl.make_batch(small(name, **kw), permute_ids=True, poison_padding=True)
    gpu = H.run_gpu(lib, batch, gemm_path=path, chunk=chunk)
    ref = H.run_oracle(batch)
    H.assert_parity(gpu, ref, batch)


@pytest.mark.parametrize("path", [SIMT, AUTO])
def test_bf16_bias_blank_nonzero_small_chunk(lib, path):
    cfg = small("c2", V=5001, D=192, N=5, T_div=6, U_div=3, blank=4097)      # odd V: ragged last chunk of 905
    batch = wl.make_batch(cfg, with_bias=True, permute_ids=True, poison_padding=True)
    gpu = H.run_gpu(lib, batch, gemm_path=path, chunk=1024)
    ref = H.run_oracle(batch)
    H.assert_parity(gpu, ref, batch)


@pytest.mark.parametrize("V", [1001, 257, 9])
def test_bf16_odd_vocabulary_narrower_than_one_chunk(lib, V):
    cfg = small("c2", V=V, D=64, N=4, T_div=10, U_div=8, zipf_s=None)
    batch = wl.make_batch(cfg, with_bias=True)
    gpu = H.run_gpu(lib, batch)
    H.assert_parity(gpu, H.run_oracle(batch), batch)


@pytest.mark.parametrize("path", [SIMT, AUTO])
def test_edge_cases_excluded_utterances(lib, path):
    cfg = small("c2", V=2048, D=64, N=6, T_div=20, U_div=6)
    batch = wl.make_batch(cfg, poison_padding=True)
    tl, il, tg = batch.target_lengths, batch.input_lengths, batch.targets
    tl[0] = 0                                   # empty target: only the all-blank alignment
    tg[1, :tl[1]] = 7                           # all labels equal: needs 2U-1 frames
    il[1] = 2 * tl[1] - 2                       # one frame short -> infeasible
    batch.hidden[1, il[1]:] = 3e4
    tg[2, 1] = batch.blank                      # blank inside a target -> bad target
    tg[3, 0] = cfg.V + 5                        # id out of range -> bad target
    il[4] = tl[4]                               # T = U with no repeats: exactly one alignment ...
    row = np.arange(1, tl[4] + 1) * 3
    tg[4, :tl[4]] = row                         # ... (distinct labels)
    batch.hidden[4, il[4]:] = -3e4
    gpu = H.run_gpu(lib, batch, gemm_path=path)
    ref = H.run_oracle(batch)
    assert list(ref["flags"]) == [0, 1, 4, 4, 0, 0]
    H.assert_parity(gpu, ref, batch)


def test_single_frame_and_single_utterance(lib):
    cfg = dataclasses.replace(wl.CONFIGS["c1"], name="one", N=1, T_lo=1, T_hi=1, U_lo=1, U_hi=1, V=264, D=8, seed=5)
    batch = wl.make_batch(cfg)
    gpu = H.run_gpu(lib, batch)
    ref = H.run_oracle(batch)
    H.assert_parity(gpu, ref, batch)


@pytest.mark.parametrize("U,T", [(14, 40), (30, 90), (60, 150), (120, 300), (250, 520), (500, 1010), (1000, 2005),
                                 (2047, 4100)])
def test_every_trellis_width_of_the_dp(lib, U, T):
    # one utterance per DP kernel configuration (32 ... 4096 positions, the widest the library takes:
    # 2 * 2047 + 1 = 4095), with adjacent repeats
    cfg = dataclasses.replace(wl.CONFIGS["c1"], name=f"dp{U}", N=2, T_lo=T - 3, T_hi=T, U_lo=U - 2, U_hi=U,
                              V=300, D=16, zipf_s=1.0, seed=U)
    batch = wl.make_batch(cfg)
    gpu = H.run_gpu(lib, batch)
    ref = H.run_oracle(batch)
    H.assert_parity(gpu, ref, batch, tol=(1e-5, 2e-4))


@pytest.mark.parametrize("beam", [2.0, 8.0, 16.0, 64.0])
@pytest.mark.parametrize("path", [SIMT])
def test_finite_beam_matches_oracle_at_the_same_beam(lib, beam, path):
    cfg = dataclasses.replace(wl.CONFIGS["c1"], name="beam", N=4, T_lo=60, T_hi=140, U_lo=5, U_hi=40,
                              V=1000, D=64, zipf_s=1.0, seed=31)
    batch = wl.make_batch(cfg)
    batch.hidden *= 3.0                      # sharper posteriors so that the beams prune
    gpu = H.run_gpu(lib, batch, beam=beam, gemm_path=path)
    ref = H.run_oracle(batch, beam=beam)
    H.assert_parity(gpu, ref, batch, tol=(1e-5, 5e-4))
    exact = H.run_oracle(batch)
    Delta, delta = H.O.discarded_mass(ref["loss"], exact["loss"])
    assert np.all(Delta >= -1e-9)
    if beam <= 2.0:
        assert Delta.max() > 1e-6            # the case does prune
    # loss stays an upper bound of the exact loss on the GPU too
    assert np.all(gpu["loss"] >= exact["loss"] * (1 - 1e-5))


def test_beam_bf16_reduced_c5_shape(lib):
    cfg = small("c5", V=4096, D=128, N=3, T_div=10, U_div=10)
    batch = wl.make_batch(cfg)
    for beam in (8.0, 16.0):
        gpu = H.run_gpu(lib, batch, beam=beam)
        ref = H.run_oracle(batch, beam=beam)
        H.assert_parity(gpu, ref, batch)


def test_two_calls_are_bitwise_identical_and_workspace_is_reusable(lib):
    import torch
    # with a bias (two-stage column sums) and few output tiles (the dX contraction is cut along k)
    batch = wl.make_batch(small("c2", V=4096, D=128, N=4, T_div=8, U_div=4), with_bias=True)
    a = H.run_gpu(lib, batch)
    b = H.run_gpu(lib, batch)
    for k in ("loss", "dH", "dW", "dbias", "subset", "relabeled"):
        np.testing.assert_array_equal(a[k], b[k])
    torch.cuda.synchronize()


def test_repeated_labels_pool_in_a_fixed_order(lib):
    """The occupancy of a class sums over the positions that carry it (Section 3.2).  One utterance
    whose labels are all the same token, one that cycles through three tokens (many scattered
    repeats), one ordinary: parity with the oracle, and three calls must agree bit for bit."""
    cfg = small("c2", V=2048, D=64, N=3, T_div=2, U_div=1)
    batch = wl.make_batch(cfg, permute_ids=True)
    U0 = min(int(batch.target_lengths[0]), int(batch.input_lengths[0]) // 2 - 1)
    batch.target_lengths[0] = U0
    batch.targets[0, :U0] = 777                                   # T >= 2 U - 1 keeps it feasible
    U1 = int(batch.target_lengths[1])
    batch.targets[1, :U1] = np.array([5, 1500, 31])[np.arange(U1) % 3]
    runs = [H.run_gpu(lib, batch) for _ in range(3)]
    ref = H.run_oracle(batch)
    assert not ref["flags"].any()
    H.assert_parity(runs[0], ref, batch)
    for other in runs[1:]:
        for k in ("loss", "dH", "dW"):
            np.testing.assert_array_equal(runs[0][k], other[k])


@pytest.mark.parametrize("path", [SIMT, AUTO])
def test_frozen_head_utterance_weights_and_accumulation(lib, path):
    import torch
    cfg = small("c3", V=8192 + 384, D=256, N=4, T_div=4, U_div=2)
    batch = wl.make_batch(cfg, with_bias=True, permute_ids=True)
    c = np.array([0.25, 1.0, 2.0, 0.5], dtype=np.float32)
    ref = H.run_oracle(batch, utt_weights=c)
    # weighted gradients, full outputs
    full = H.run_gpu(lib, batch, gemm_path=path, utt_weights=c, chunk=2048)
    H.assert_parity(full, ref, batch)
    # frozen head: dH and dbias as before, dW not produced
    frozen = H.run_gpu(lib, batch, gemm_path=path, utt_weights=c, chunk=2048, skip_dW=True)
    assert frozen["dW"] is None
    np.testing.assert_array_equal(frozen["dH"], full["dH"])
    np.testing.assert_array_equal(frozen["dbias"], full["dbias"])
    np.testing.assert_array_equal(frozen["loss"], full["loss"])
    # accumulation over two micro-batches: the second call adds to dW / dbias of the first
    dev = torch.device("cuda:0")
    hidden = torch.from_numpy(batch.hidden).to(dev).to(torch.bfloat16)
    W = torch.from_numpy(batch.W).to(dev).to(torch.bfloat16)
    bias = torch.from_numpy(batch.bias).to(dev).to(torch.bfloat16)
    targets = torch.from_numpy(batch.targets).to(dev)
    cw = torch.from_numpy(c).to(dev)
    args = (hidden, W, bias, targets, batch.input_lengths, batch.target_lengths, batch.blank)
    out = lib.pruned_ctc_fwd_bwd(*args, gemm_path=path, chunk=2048, utt_weights=cw)
    out = lib.pruned_ctc_fwd_bwd(*args, gemm_path=path, chunk=2048, utt_weights=cw, accumulate_dW=True,
                                 workspace=out["workspace"], out=out)
    torch.cuda.synchronize()
    assert H.rel_fro(out["dW"].float().cpu().numpy(), 2.0 * ref["dW"]) <= 1e-2
    assert H.rel_fro(out["dbias"].float().cpu().numpy(), 2.0 * ref["db"]) <= 1e-2
    np.testing.assert_array_equal(out["dH"].float().cpu().numpy(), full["dH"])   # dH is never accumulated


@pytest.mark.parametrize("a_mn", [False, True])
@pytest.mark.parametrize("b_mn", [False, True])
@pytest.mark.parametrize("m,n,k", [(128, 256, 64), (200, 264, 328), (1000, 520, 1032), (72, 8, 4096)])
def test_tensor_core_contraction_all_operand_layouts(lib, a_mn, b_mn, m, n, k):
    import torch
    g = torch.Generator(device="cpu").manual_seed(m * 7 + n * 3 + k)
    A = torch.randn((m, k), generator=g).to(torch.bfloat16)
    B = torch.randn((n, k), generator=g).to(torch.bfloat16)
    ref = A.double() @ B.double().T
    Ad = (A.T.contiguous() if a_mn else A).cuda()
    Bd = (B.T.contiguous() if b_mn else B).cuda()
    if (a_mn and m % 8) or (b_mn and n % 8):
        pytest.skip("contiguous extent must be a multiple of 8")
    for path in (SIMT, AUTO):
        C = lib.gemm_bf16(Ad, Bd, m, n, k, a_mn, b_mn, gemm_path=path).cpu().double()
        err = (C - ref).abs().max().item()
        assert err <= 2e-3 * (k ** 0.5), (path, err)


def test_max_K_promise_kept_and_broken(lib):
    cfg = small("c2", V=4096, D=64, N=6, T_div=10, U_div=4)
    batch = wl.make_batch(cfg, permute_ids=True)
    ref = H.run_oracle(batch)
    K = ref["K"]
    kept = H.run_gpu(lib, batch, max_K=K)                 # exact promise: same result, smaller buffers
    H.assert_parity(kept, ref, batch)
    assert kept["workspace_bytes"] < H.run_gpu(lib, batch)["workspace_bytes"]
    broken = H.run_gpu(lib, batch, max_K=K - 3, check_status=False)   # promise broken: flagged, nothing faults
    assert np.all(broken["flags"] & 8)
    assert np.all(broken["loss"] == 0) and np.all(broken["dH"] == 0) and np.all(broken["dW"] == 0)
    assert int(broken["K"][0]) == K - 3
    np.testing.assert_array_equal(broken["subset"][: K - 3], ref["U"][: K - 3])


def test_paper_grid_shape_many_short_utterances(lib):
    # the paper's benchmark grid: every utterance exactly 100 frames, many utterances, D = 512
    cfg = wl.reduced(wl.CONFIGS["g16k"], V=8192, N=24, name="g-small")
    batch = wl.make_batch(cfg, permute_ids=True)
    gpu = H.run_gpu(lib, batch)
    H.assert_parity(gpu, H.run_oracle(batch), batch)


def test_forward_only_matches_full_call(lib):
    batch = wl.make_batch(small("c3", V=8192, D=256, N=4, T_div=4, U_div=2), permute_ids=True)
    full = H.run_gpu(lib, batch)
    fwd = H.run_gpu(lib, batch, forward_only=True)
    assert fwd["dH"] is None and fwd["dW"] is None
    np.testing.assert_array_equal(fwd["loss"], full["loss"])
    np.testing.assert_array_equal(fwd["subset"], full["subset"])
    fwd_beam = H.run_gpu(lib, batch, forward_only=True, beam=8.0)
    np.testing.assert_array_equal(fwd_beam["loss"], H.run_gpu(lib, batch, beam=8.0)["loss"])


@pytest.mark.parametrize("path,dtype", [(SIMT, "fp32"), (SIMT, "bf16"), (AUTO, "bf16")])
def test_greedy_recognition_matches_oracle(lib, path, dtype):
    import torch
    from oracle import pruned_ctc_oracle as O
    cfg = dataclasses.replace(wl.CONFIGS["c2"], name="greedy", N=5, T_lo=40, T_hi=90, D=64, V=5000 - 5000 % 8,
                              dtype=dtype, blank=3, seed=99)
    batch = wl.make_batch(cfg, with_bias=True)
    batch.W[batch.blank] *= 3.0                      # make blanks and repeats frequent enough to matter
    for t in range(0, batch.T - 1, 3):
        batch.hidden[:, t + 1] = batch.hidden[:, t]  # repeated frames, so that merging repeats matters
    if dtype == "bf16":
        batch.W = wl.round_to_bf16(batch.W)
    dev = torch.device("cuda:0")
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    out = lib.greedy_decode(torch.from_numpy(batch.hidden).to(dev).to(tdt), torch.from_numpy(batch.W).to(dev).to(tdt),
                            torch.from_numpy(batch.bias).to(dev).to(tdt), batch.input_lengths, batch.blank,
                            gemm_path=path)
    torch.cuda.synchronize()
    fl = out["frame_labels"].cpu().numpy()
    tok = out["tokens"].cpu().numpy()
    tlen = out["token_lengths"].cpu().numpy()
    frames, hyps, logits = O.greedy_decode(batch.hidden, batch.W, batch.bias, batch.input_lengths, batch.blank)
    tol = 1e-4 if dtype == "fp32" else 1e-3
    exact = 0
    for n in range(cfg.N):
        Tn = int(batch.input_lengths[n])
        assert np.all(fl[n, Tn:] == -1)
        got = fl[n, :Tn]
        # the arg-max is unique up to rounding: where it differs from the oracle's, the logit of the
        # class the GPU chose must be within the arithmetic's rounding of the largest logit
        z = logits[n]
        assert np.all(z[np.arange(Tn), got] >= z.max(axis=1) - tol)
        exact += int(np.sum(got == frames[n]))
        # the hypothesis is the collapse of the frame labels the GPU itself chose (bit-exact), and
        # equals the oracle's hypothesis whenever the frame labels agree
        mine = O.collapse(got, batch.blank)
        assert int(tlen[n]) == len(mine) and list(tok[n, : tlen[n]]) == mine and np.all(tok[n, tlen[n]:] == -1)
        if np.array_equal(got, frames[n]):
            assert mine == hyps[n]
    assert exact >= 0.999 * int(batch.input_lengths.sum())
    assert sum(len(h) for h in hyps) > 0


@pytest.mark.parametrize("path", [SIMT, AUTO])
@pytest.mark.parametrize("case", range(12))
def test_random_small_shapes(lib, path, case):
    # seeded sweep over odd shapes: single frames, empty targets, heavy repeats, any blank id,
    # vocabularies smaller than a tile, widths that are no multiple of a tile, bias on or off, beams
    rng = np.random.default_rng(1000 + case)
    N = int(rng.integers(1, 7))
    D = int(rng.choice([8, 24, 64, 136, 200]))
    V = int(rng.integers(9, 2100))                       # any vocabulary size, odd ones included
    T_hi = int(rng.integers(1, 70))
    U_hi = int(rng.integers(0, max(1, min(T_hi, 40)) + 1))
    dtype = "bf16" if (path == AUTO or case % 2) else "fp32"
    cfg = dataclasses.replace(wl.CONFIGS["c1"], name=f"rnd{case}", N=N, T_lo=max(1, T_hi // 3), T_hi=T_hi, D=D, V=V,
                              dtype=dtype, U_lo=0, U_hi=U_hi, zipf_s=1.0 if case % 3 else None,
                              blank=int(rng.integers(0, V)), seed=5000 + case)
    batch = wl.make_batch(cfg, with_bias=bool(case % 2), poison_padding=True, permute_ids=bool(case % 4 == 1))
    for n in range(N):                                   # inject runs of equal labels
        u = int(batch.target_lengths[n])
        if u >= 3 and rng.random() < 0.6:
            s0 = int(rng.integers(0, u - 2))
            batch.targets[n, s0:s0 + 3] = batch.targets[n, s0]
    beam = [0.0, 0.0, 4.0, 32.0][case % 4]
    chunk = [0, 64, 128, 1024][case % 4]
    gpu = H.run_gpu(lib, batch, gemm_path=path, beam=beam, chunk=chunk)
    ref = H.run_oracle(batch, beam=beam if beam > 0 else None)
    tol = (2e-3, 1e-2) if dtype == "bf16" else (2e-5, 5e-4)
    H.assert_parity(gpu, ref, batch, tol=tol)


@pytest.mark.parametrize("path", [SIMT, AUTO])
def test_zero_and_negative_utterance_weights(lib, path):
    # c_n = 0 switches an utterance's gradient off without flagging it; a negative c_n flips its sign
    cfg = small("c3", V=4096 + 77, D=128, N=5, T_div=8, U_div=4)
    batch = wl.make_batch(cfg, with_bias=True, permute_ids=True)
    c = np.array([0.0, -1.0, 1.0, 3.0, -0.5], dtype=np.float32)
    gpu = H.run_gpu(lib, batch, gemm_path=path, utt_weights=c, chunk=1024)
    ref = H.run_oracle(batch, utt_weights=c)
    H.assert_parity(gpu, ref, batch)
    assert np.all(gpu["dH"][0] == 0.0) and gpu["flags"][0] == 0 and gpu["loss"][0] > 0


# one upload / four segments of W; and a strongly negative bias: every logit of a frame then lies far
# below zero, so the normaliser must not be anchored at the value an unused partial slot holds
@pytest.mark.parametrize("V,D,bias_shift", [(8192 + 384, 256, 0.0), (4 * 4096 + 1000, 64, 0.0),
                                            (4 * 4096 + 1000, 64, -200.0)])
def test_host_buffer_entry_point_matches_device_entry_point(lib, V, D, bias_shift):
    import torch
    batch = wl.make_batch(small("c3", V=V, D=D, N=4, T_div=4, U_div=2), with_bias=True, permute_ids=True)
    if bias_shift:
        batch.bias = wl.round_to_bf16(batch.bias + np.float32(bias_shift))
    dev_out = H.run_gpu(lib, batch, chunk=2048)
    tdt = torch.bfloat16
    hid = torch.from_numpy(batch.hidden).to(tdt).pin_memory()
    W = torch.from_numpy(batch.W).to(tdt).pin_memory()
    bias = torch.from_numpy(batch.bias).to(tdt).pin_memory()
    tg = torch.from_numpy(batch.targets).pin_memory()
    res = None
    for _ in range(2):                                   # the scratch buffer and outputs are reusable
        res = lib.pruned_ctc_fwd_bwd_host(hid, W, bias, tg, batch.input_lengths, batch.target_lengths, batch.blank,
                                          chunk=2048, scratch=None if res is None else res["scratch"], out=res)
        torch.cuda.synchronize()
        for k in ("loss", "dH", "dW", "dbias"):
            got = res[k].float().numpy()
            if V < 4 * 4096:
                np.testing.assert_array_equal(got, dev_out[k])
            else:
                # W arrives in four segments and the normaliser is summed per segment: another
                # summation order, so the last bits of lambda (and a few bf16 roundings) may differ
                assert H.rel_fro(got, dev_out[k]) <= 1e-3
        K = int(res["K"][0])
        np.testing.assert_array_equal(res["subset"].numpy()[:K], dev_out["subset"][:K])
        np.testing.assert_array_equal(res["relabeled"].numpy(), dev_out["relabeled"])
        np.testing.assert_array_equal(res["flags"].numpy(), dev_out["flags"])
    ref = H.run_oracle(batch)
    host = {k: (v.float().numpy() if v.is_floating_point() else v.numpy()) for k, v in res.items()
            if hasattr(v, "numpy") and k != "scratch"}
    H.assert_parity(host, ref, batch)


@pytest.mark.parametrize("path", [SIMT, AUTO])
def test_non_finite_states_exclude_only_their_utterance(lib, path):
    cfg = small("c2", V=4096, D=128, N=4, T_div=8, U_div=4)
    batch = wl.make_batch(cfg, with_bias=True)
    clean = wl.make_batch(cfg, with_bias=True)
    batch.hidden[1, 3, 5] = np.nan                     # one NaN state in utterance 1
    batch.hidden[2, 0, :4] = np.inf                    # Inf states in utterance 2
    gpu = H.run_gpu(lib, batch, gemm_path=path)
    assert list(gpu["flags"]) == [0, 2, 2, 0]
    assert gpu["loss"][1] == 0 and gpu["loss"][2] == 0
    assert np.all(gpu["dH"][1] == 0) and np.all(gpu["dH"][2] == 0)
    assert np.isfinite(gpu["dW"]).all() and np.isfinite(gpu["dbias"]).all() and np.isfinite(gpu["dH"]).all()
    # the other utterances are untouched: same result as a batch that holds only them
    keep = [0, 3]
    sub = dataclasses.replace(clean, hidden=clean.hidden[keep], targets=clean.targets[keep],
                              input_lengths=clean.input_lengths[keep], target_lengths=clean.target_lengths[keep],
                              cfg=dataclasses.replace(cfg, N=2))
    ref = H.run_oracle(sub)
    np.testing.assert_allclose(gpu["loss"][keep], ref["loss"], rtol=2e-3)
    assert H.rel_fro(gpu["dW"], ref["dW"]) <= 1e-2
    assert H.rel_fro(gpu["dH"][keep][:, : sub.hidden.shape[1]], ref["dH"]) <= 1e-2


def test_workspace_guards_stay_intact_and_trace_is_well_formed(lib):
    import torch
    batch = wl.make_batch(small("c3", V=8192 + 384, D=256, N=4, T_div=4, U_div=2), with_bias=True, permute_ids=True)
    dev = torch.device("cuda:0")
    hidden = torch.from_numpy(batch.hidden).to(dev).to(torch.bfloat16)
    W = torch.from_numpy(batch.W).to(dev).to(torch.bfloat16)
    bias = torch.from_numpy(batch.bias).to(dev).to(torch.bfloat16)
    targets = torch.from_numpy(batch.targets).to(dev)
    N, T, D = hidden.shape
    for beam in (0.0, 8.0):
        prob = lib.make_problem(N, T, D, W.shape[0], lib.PCTC_BF16, batch.blank, beam, 2048, targets.shape[1])
        need = lib.workspace_bytes(prob, batch.input_lengths, batch.target_lengths)
        guard = 4096
        buf = torch.full((guard + need + guard,), 0xA5, dtype=torch.uint8, device=dev)
        ws = buf[guard:guard + need]                      # the library is told about exactly `need` bytes
        trace = lib.Trace(lib.Trace.capacity_for(W.shape[0], 2048))
        res = lib.pruned_ctc_fwd_bwd(hidden, W, bias, targets, batch.input_lengths, batch.target_lengths,
                                     batch.blank, beam=beam, chunk=2048, workspace=ws, trace=trace, check_status=True)
        torch.cuda.synchronize()
        assert res["workspace"].data_ptr() == ws.data_ptr()
        assert bool((buf[:guard] == 0xA5).all()) and bool((buf[guard + need:] == 0xA5).all())
        spans = trace.spans()
        kinds = [k for k, _ in spans if k >= 0]
        names = [lib.PHASES[k] for k in kinds]
        nchunks = (W.shape[0] + 2047) // 2048
        assert names.count("dlogits") == nchunks and names.count("dh") == nchunks and names.count("dw") == nchunks
        assert names.count("dbias") == nchunks and names.count("lse") == 1 and names.count("dp") == 1
        assert all(ms >= 0 for k, ms in spans if k >= 0)
    ref = H.run_oracle(batch, beam=8.0)
    np.testing.assert_allclose(res["loss"].cpu().numpy(), ref["loss"], rtol=2e-3)


def test_bf16_shapes_the_tensor_core_path_does_not_cover_fall_to_the_fma_kernels(lib):
    # V and D that are no multiples of 8: TMA row pitches would be misaligned, so AUTO uses the FMA kernels
    cfg = small("c2", V=5003, D=100, N=3, T_div=10, U_div=5)
    batch = wl.make_batch(cfg, with_bias=True, permute_ids=True)
    gpu = H.run_gpu(lib, batch, gemm_path=AUTO)
    H.assert_parity(gpu, H.run_oracle(batch), batch)


def test_call_returns_to_the_host_while_the_stream_is_still_busy(lib):
    """No hidden synchronisation: with tens of milliseconds of earlier work still queued on the stream,
    a call on the paper-grid shape with the most frames (640 utterances of 100 frames, vocabulary
    reduced) must hand control back to the host at once, and give the same bits as an idle-stream call."""
    import time
    import torch
    cfg = wl.reduced(wl.CONFIGS["g64k"], V=4096, D=128, name="g64k-small")
    batch = wl.make_batch(cfg)
    assert batch.M == 64000
    dev = torch.device("cuda:0")
    hidden = torch.from_numpy(batch.hidden).to(dev).to(torch.bfloat16)
    W = torch.from_numpy(batch.W).to(dev).to(torch.bfloat16)
    targets = torch.from_numpy(batch.targets).to(dev)
    args = (hidden, W, None, targets, batch.input_lengths, batch.target_lengths, batch.blank)
    first = lib.pruned_ctc_fwd_bwd(*args, check_status=True)
    torch.cuda.synchronize()
    want = {k: first[k].clone() for k in ("loss", "dH", "dW", "subset", "relabeled", "flags")}
    a = torch.randn(8192, 8192, device=dev, dtype=torch.bfloat16)
    c = torch.empty_like(a)
    torch.matmul(a, a, out=c)
    torch.cuda.synchronize()
    busy = torch.cuda.Event()
    t_busy = time.perf_counter()
    for _ in range(120):                               # about 0.1 s of queued work (0.7 ms or more each)
        torch.matmul(a, a, out=c)
    busy.record()
    t0 = time.perf_counter()
    res = lib.pruned_ctc_fwd_bwd(*args, workspace=first["workspace"], out=first)
    t1 = time.perf_counter()
    still_busy = not busy.query()
    torch.cuda.synchronize()
    t_done = time.perf_counter()
    print(f"host time of the call {1e3 * (t1 - t0):.2f} ms; queued work took {1e3 * (t_done - t_busy):.1f} ms")
    assert still_busy, "the earlier work had finished before the call returned: the call waited for the stream"
    assert t1 - t0 < 0.010
    for k, v in want.items():
        assert torch.equal(res[k], v), k
    assert lib.workspace_status(res["workspace"]) == 0


def test_capturing_stream_is_refused_before_anything_is_enqueued(lib):
    # the call uploads per-call index tables from temporary host memory, which a graph replay would
    # read again after it is gone: a capturing stream gets "unsupported" and an empty capture
    import torch
    batch = wl.make_batch(small("c2", V=2048, D=64, N=3, T_div=10, U_div=4))
    dev = torch.device("cuda:0")
    hidden = torch.from_numpy(batch.hidden).to(dev).to(torch.bfloat16)
    W = torch.from_numpy(batch.W).to(dev).to(torch.bfloat16)
    targets = torch.from_numpy(batch.targets).to(dev)
    args = (hidden, W, None, targets, batch.input_lengths, batch.target_lengths, batch.blank)
    eager = lib.pruned_ctc_fwd_bwd(*args, check_status=True)
    torch.cuda.synchronize()
    loss0 = eager["loss"].clone()
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    with pytest.raises(lib.PctcError) as ei:
        with torch.cuda.graph(g, stream=s):
            lib.pruned_ctc_fwd_bwd(*args, workspace=eager["workspace"], out=eager)
    assert ei.value.status == 3
    torch.cuda.synchronize()
    again = lib.pruned_ctc_fwd_bwd(*args, workspace=eager["workspace"], out=eager, check_status=True)   # still usable
    torch.cuda.synchronize()
    assert torch.equal(again["loss"], loss0)


def test_million_class_vocabulary(lib):
    # V = 1,000,003 (odd, 123 chunks of 8,192 on the tensor-core path): bitmap ranking over 31k words,
    # class map of 4 MB, many column splits of the normaliser, a ragged last chunk of 579 classes
    cfg = dataclasses.replace(wl.CONFIGS["c2"], name="v1m", N=3, T_lo=30, T_hi=48, D=32, V=1_000_003,
                              U_lo=4, U_hi=12, zipf_s=1.05, seed=4242)
    batch = wl.make_batch(cfg, permute_ids=True)
    gpu = H.run_gpu(lib, batch, chunk=8192)
    ref = H.run_oracle(batch)
    H.assert_parity(gpu, ref, batch)


@pytest.mark.parametrize("case", range(40))
def test_random_wide_shapes(lib, case):
    # a wider seeded sweep: head widths up to 1024 (including widths that are no multiple of 64), odd
    # vocabularies up to 40,000, up to 500 frames, any chunk width, optional bias, beam, signed utterance
    # weights and frozen head, mostly on the tensor-core path
    rng = np.random.default_rng(77000 + case)
    N = int(rng.integers(1, 9))
    D = int(rng.choice([8, 16, 64, 72, 128, 256, 512, 520, 1024]))
    V = int(rng.choice([rng.integers(2, 300), rng.integers(300, 5000), rng.integers(5000, 40000)]))
    T_hi = int(rng.choice([rng.integers(1, 20), rng.integers(20, 200), rng.integers(200, 500)]))
    U_hi = int(rng.integers(0, max(1, min(T_hi, 120)) + 1))
    path = SIMT if int(rng.integers(0, 4)) == 0 else AUTO
    dtype = "fp32" if (path == SIMT and rng.random() < 0.5) else "bf16"
    cfg = dataclasses.replace(wl.CONFIGS["c1"], name=f"wide{case}", N=N, T_lo=max(1, T_hi // 3), T_hi=T_hi, D=D, V=V,
                              dtype=dtype, U_lo=0, U_hi=U_hi, zipf_s=[None, 1.0, 1.3][case % 3],
                              blank=int(rng.integers(0, V)), seed=9000 + case, rms_norm=bool(case % 2))
    batch = wl.make_batch(cfg, with_bias=bool(rng.integers(0, 2)), poison_padding=True,
                          permute_ids=bool(rng.integers(0, 2)))
    for n in range(N):
        u = int(batch.target_lengths[n])
        if u >= 3 and rng.random() < 0.5:
            s0 = int(rng.integers(0, u - 2))
            batch.targets[n, s0:s0 + 3] = batch.targets[n, s0]
    beam = float(rng.choice([0.0, 0.0, 3.0, 12.0, 40.0]))
    chunk = int(rng.choice([0, 0, 64, 200, 1024, 2048, 4096, 8192]))
    w = rng.choice([0.0, 0.5, 1.0, 2.0], size=N).astype(np.float32) if rng.random() < 0.3 else None
    frozen = bool(rng.random() < 0.2)
    gpu = H.run_gpu(lib, batch, gemm_path=path, beam=beam, chunk=chunk, utt_weights=w, skip_dW=frozen)
    ref = H.run_oracle(batch, beam=beam if beam > 0 else None, utt_weights=w)
    tol = (2e-3, 1e-2) if dtype == "bf16" else (2e-5, 5e-4)
    H.assert_parity(gpu, ref, batch, tol=tol)


def test_tall_dw_tiles_ragged_chunk_and_accumulation(lib):
    # D = 512, about 2,400 frames, one 16,384-column chunk plus a ragged one: the dW contraction of the
    # first chunk runs on 512 x 256 tiles (long contraction, 64 such tiles fill one wave); the rows of dW
    # must match the oracle across the chunk boundary, and a second call with accumulate_dW doubles them
    import torch
    cfg = small("c2", V=16384 + 300, D=512, N=6, T_div=1, U_div=2)
    batch = wl.make_batch(cfg, permute_ids=True)
    assert batch.M > 2048
    ref = H.run_oracle(batch)
    gpu = H.run_gpu(lib, batch, chunk=16384)
    H.assert_parity(gpu, ref, batch)
    dev = torch.device("cuda:0")
    hidden = torch.from_numpy(batch.hidden).to(dev).to(torch.bfloat16)
    W = torch.from_numpy(batch.W).to(dev).to(torch.bfloat16)
    targets = torch.from_numpy(batch.targets).to(dev)
    args = (hidden, W, None, targets, batch.input_lengths, batch.target_lengths, batch.blank)
    out = lib.pruned_ctc_fwd_bwd(*args, chunk=16384)
    out = lib.pruned_ctc_fwd_bwd(*args, chunk=16384, accumulate_dW=True, workspace=out["workspace"], out=out)
    torch.cuda.synchronize()
    assert H.rel_fro(out["dW"].float().cpu().numpy(), 2.0 * ref["dW"]) <= 1e-2


@pytest.mark.parametrize("path,dtype,k,chunk", [(SIMT, "fp32", 4, 300), (SIMT, "bf16", 8, 0), (AUTO, "bf16", 8, 1024),
                                                (AUTO, "bf16", 1, 0), (AUTO, "bf16", 2, 4096)])
def test_topk_recognition_matches_oracle(lib, path, dtype, k, chunk):
    """The k best classes of every frame and their log-probabilities (the per-frame input of a prefix beam
    search): classes must agree with the oracle wherever the oracle's neighbouring ranks are not near-ties,
    log-probabilities rank by rank."""
    import torch
    from oracle import pruned_ctc_oracle as O
    if dtype == "fp32":
        cfg = dataclasses.replace(wl.CONFIGS["c1"], name="tk32", N=3, T_lo=10, T_hi=40, V=1531, D=72, seed=21)
    else:
        cfg = small("c3", V=9000 + 37, D=256, N=3, T_div=6)
    batch = wl.make_batch(cfg, with_bias=True, poison_padding=True)
    dev = torch.device("cuda:0")
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    hidden = torch.from_numpy(batch.hidden).to(dev).to(tdt)
    W = torch.from_numpy(batch.W).to(dev).to(tdt)
    bias = torch.from_numpy(batch.bias).to(dev).to(tdt)
    res = lib.topk_decode(hidden, W, bias, batch.input_lengths, k, chunk=chunk, gemm_path=path)
    torch.cuda.synchronize()
    cls_g = res["classes"].cpu().numpy()
    lp_g = res["logprobs"].cpu().numpy().astype(np.float64)
    cls_r, lp_r = O.topk_decode(batch.hidden, batch.W, batch.bias, batch.input_lengths, k)
    # full top-(k+1) of the oracle gives the gap below the last rank too
    _, lp_r1 = O.topk_decode(batch.hidden, batch.W, batch.bias, batch.input_lengths, k + 1)
    tol = 1e-4 if dtype == "fp32" else 2e-3
    checked = 0
    for n in range(cfg.N):
        Tn = int(batch.input_lengths[n])
        assert np.all(cls_g[n, Tn:] == -1) and np.all(np.isneginf(lp_g[n, Tn:]))
        np.testing.assert_allclose(lp_g[n, :Tn], lp_r[n], atol=tol, rtol=0)      # rank by rank
        gaps = -np.diff(lp_r1[n], axis=1)                                        # [Tn, k]: rank r to rank r+1
        for t in range(Tn):
            for r in range(k):
                clear = gaps[t, r] > 4 * tol and (r == 0 or gaps[t, r - 1] > 4 * tol)
                if clear:
                    assert cls_g[n, t, r] == cls_r[n][t, r], (n, t, r)
                    checked += 1
    assert checked > 0.6 * k * batch.M      # most ranks are clear of their neighbours by more than the tolerance
    # rank one is the greedy decoder's label
    greedy = lib.greedy_decode(hidden, W, bias, batch.input_lengths, 0, gemm_path=path)
    fl = greedy["frame_labels"].cpu().numpy()
    for n in range(cfg.N):
        Tn = int(batch.input_lengths[n])
        same = fl[n, :Tn] == cls_g[n, :Tn, 0]
        assert same.mean() > 0.98          # the two take their maxima over different chunkings of V: near-ties may differ


@pytest.mark.parametrize("path", [SIMT, AUTO])
def test_more_utterances_than_one_length_slice(lib, path):
    """2,100 very short utterances: the lengths reach the device in three kernel-parameter slices of 1,024,
    and the prefix sums over the utterances run over more than one utterance per thread."""
    cfg = wl.Config("manyutt", N=2100, T_lo=2, T_hi=6, D=16, V=96, dtype="bf16", U_lo=0, U_hi=3, zipf_s=1.1, seed=4242)
    batch = wl.make_batch(cfg, poison_padding=True)
    gpu = H.run_gpu(lib, batch, gemm_path=path)
    ref = H.run_oracle(batch)
    assert (ref["flags"] == 1).any() and (ref["flags"] == 0).any()      # some utterances have too few frames
    H.assert_parity(gpu, ref, batch)
    import torch
    dev = torch.device("cuda:0")
    greedy = lib.greedy_decode(torch.from_numpy(batch.hidden).to(dev).to(torch.bfloat16),
                               torch.from_numpy(batch.W).to(dev).to(torch.bfloat16), None, batch.input_lengths, 0,
                               gemm_path=path)
    fl = greedy["frame_labels"].cpu().numpy()
    for n in (0, 1023, 1024, 2047, 2048, 2099):
        assert np.all(fl[n, : batch.input_lengths[n]] >= 0) and np.all(fl[n, batch.input_lengths[n]:] == -1)


@pytest.mark.parametrize("V,chunk", [(2 * 3072 + 520, 3072), (3 * 2560, 2560)])
def test_wide_head_many_output_tiles_of_dx(lib, V, chunk):
    """A head wide enough that dX += dZ_c W_c has more output tiles (11 x 13 of 256 x 256) than the GPU has CTA
    pairs, with a ragged last chunk shorter than the others in the first case.  Three calls must agree bit
    for bit."""
    cfg = wl.Config("widehead", N=6, T_lo=400, T_hi=480, D=3328, V=V, dtype="bf16", U_lo=20, U_hi=60, zipf_s=1.1,
                    rms_norm=True, seed=808)
    batch = wl.make_batch(cfg, permute_ids=True, poison_padding=True)
    runs = [H.run_gpu(lib, batch, chunk=chunk) for _ in range(3)]
    ref = H.run_oracle(batch)
    H.assert_parity(runs[0], ref, batch)
    for other in runs[1:]:
        for k in ("loss", "dH", "dW"):
            np.testing.assert_array_equal(runs[0][k], other[k])
