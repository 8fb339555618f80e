"""Parity at the benchmark's full sizes, in the launch configuration bench.py times (default tile policy).

Every config is compared in full against the oracle: every element of C, the whole flag bitmap, the header
counts and the site log of a GEMM with 16 or more sites of the config's mix, then the campaign's records (the
oracle's GEMM takes seconds at these sizes on the host cores, about half a minute for the 8192^3 one). The
sampled-output test that follows adds properties that hold at any size (flag count = popcount of the bitmap,
untouched rows / columns bit-identical to the fault-free run).
"""
import numpy as np
import pytest
import torch

import oracle as orc
import paper_2311_05782_b200 as mpg
import synth
from parity import (TOL, absprod_fast, bits_f32, check_campaign_against_oracle, check_gemm_against_oracle,
                    check_operand_trial, close, run_gpu_campaign, run_gpu_gemm, to_dev)

pytestmark = pytest.mark.gpu


def widen_np(dtype, bits):
    """Library conversions only (numpy half, bit shifts): the test's own view of the operand values."""
    if dtype == orc.FP16:
        return bits.view(np.float16).astype(np.float64)
    if dtype == orc.BF16:
        return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    return (bits & np.uint32(0xFFFFE000)).view(np.float32).astype(np.float64)


def absprod_np(dtype, A, Bt):
    return np.abs(widen_np(dtype, A)) @ np.abs(widen_np(dtype, Bt)).T


def test_c2_full_size_gemm_and_campaign():
    w = synth.make_workload("c2")
    M, N, K = w.M, w.N, w.K
    sites = w.sites[:6]
    Cg, hdr, log, bm = run_gpu_gemm(w.dtype, w.A, w.Bt, sites, w.detect_mode)
    assert hdr[0] == 0 and hdr[3] == len(sites)
    Co, hdr_o, log_o, bm_o = orc.gemm(w.dtype, w.A, w.Bt, sites, w.detect_mode)
    A2, B2 = w.A.copy(), w.Bt.copy()
    for s in sites:
        if s["kind"] == orc.KIND_A:
            A2[s["row"], s["k"]] = orc.flip_operand(w.dtype, int(A2[s["row"], s["k"]]), int(s["xor_mask"]))
        else:
            B2[s["col"], s["k"]] = orc.flip_operand(w.dtype, int(B2[s["col"], s["k"]]), int(s["xor_mask"]))
    tol = TOL * absprod_np(w.dtype, A2, B2)
    ok = close(Cg, Co, tol)
    assert ok.all(), f"{(~ok).sum()} of {ok.size} elements out of tolerance"
    assert np.array_equal(bm, bm_o) and hdr[1] == hdr_o[1] and hdr[2] == hdr_o[2]
    assert np.array_equal(log.view(np.uint32), log_o.view(np.uint32))
    # campaign: all 1024 trials; the oracle recomputes each affected row / column in full
    Cc, rec = run_gpu_campaign(w.dtype, w.A, w.Bt, w.sites, w.detect_mode)
    Cclean, *_ = orc.gemm(w.dtype, w.A, w.Bt)
    assert close(Cc, Cclean, TOL * absprod_np(w.dtype, w.A, w.Bt)).all()
    ro = orc.campaign(w.dtype, w.A, w.Bt, Cclean, w.sites, w.detect_mode)
    for f in ("kind", "primary_index", "before_bits", "after_bits", "final_bits", "n_affected"):
        assert np.array_equal(rec[f], ro[f]), f
    assert (rec["n_detected"] > 0).sum() > 20        # exponent-MSB flips of an operand light up a whole row/column
    # every trial: bit for bit against Eq. 1-2 on the device's clean C; against the recompute the detected sets, the
    # status bits and the largest deviation, element by element wherever the two records are not identical (and on
    # every 64th trial regardless)
    rw = orc.campaign(w.dtype, w.A, w.Bt, Cc, w.sites, w.detect_mode, operand_form=1)
    for t, st in enumerate(w.sites):
        check_operand_trial(w.dtype, w.A, w.Bt, st, w.detect_mode, Cc, Cclean, rec[t], ro[t], rw[t], deep=t % 64 == 0)


def test_c1_full_size_all_trials_in_one_gemm_and_as_campaign():
    from parity import check_campaign_against_oracle, check_gemm_against_oracle
    w = synth.make_workload("c1")
    check_gemm_against_oracle(w.dtype, w.A, w.Bt, w.sites, w.detect_mode, max_fragile=1)
    check_campaign_against_oracle(w.dtype, w.A, w.Bt, w.sites, w.detect_mode, max_fragile=1)


@pytest.mark.parametrize("name,n_sites,n_trials", [("c3a", 24, 4096), ("c3b", 24, 4096), ("c4", 16, 2048), ("c5", 48, 2048)])
def test_large_configs_whole(name, n_sites, n_trials):
    """The whole output of a faulty GEMM at the benchmark's size and default launch policy (so with the tile order and,
    where it applies, the cut last round that bench.py times): every element within tolerance of the oracle's, flag
    bitmap, header and site log word for word; then the campaign's records for the config's trial table (c5: the
    first 2048 of its 100000 trials -- a column trial costs the oracle half a billion multiply-adds)."""
    w = synth.make_workload(name, trials=max(n_trials, n_sites))
    sites = w.sites[:n_sites].copy()
    # sites at tile corners and seams as well as where the generator put them
    M, N = w.M, w.N
    corners = [(0, 0), (M - 1, N - 1), (127, N - 1), (128, 0), (255, min(255, N - 1)), (256, min(256, N - 1)), (M - 129, N // 2)]
    movable = [t for t in range(n_sites) if int(sites["kind"][t]) in (orc.KIND_OUT, orc.KIND_ACC)][:len(corners)]
    for t, (i, j) in zip(movable, corners):
        sites["row"][t] = i; sites["col"][t] = j
    check_gemm_against_oracle(w.dtype, w.A, w.Bt, sites, w.detect_mode, max_fragile=1, fast_tol=True)
    Cclean, *_ = orc.gemm(w.dtype, w.A, w.Bt)
    check_campaign_against_oracle(w.dtype, w.A, w.Bt, w.sites[:n_trials], w.detect_mode, max_fragile=2, Cclean=Cclean,
                                  ap=absprod_fast(w.dtype, w.A, w.Bt), deep_every=0 if name != "c5" else 500)


@pytest.mark.parametrize("name", ["c3a", "c3b", "c4", "c5"])
def test_large_configs_on_sampled_outputs(name):
    w = synth.make_workload(name, trials=256)
    M, N, K = w.M, w.N, w.K
    a, b = to_dev(w.A, w.dtype), to_dev(w.Bt, w.dtype)
    # fault-free run, then a run with the first sites of the table
    C0, f0 = mpg.gemm(w.dtype, a, b, None, w.detect_mode)
    n_sites = 16
    sites = w.sites[:n_sites]
    C1, f1 = mpg.gemm(w.dtype, a, b, sites, w.detect_mode)
    torch.cuda.synchronize()
    hdr0, _, bm0 = mpg.split_flags(f0, M, N, 0)
    hdr1, log1, bm1 = mpg.split_flags(f1, M, N, n_sites)
    assert hdr0[0] == 0 and hdr0[1] == 0 and not bm0.any()          # clean workloads raise no flag
    assert hdr1[0] == 0 and hdr1[3] == n_sites
    assert sum(int(x) for x in np.bitwise_count(bm1).reshape(-1)) == hdr1[1]
    # sampled clean outputs against the oracle, tile corners and tails included
    rng = np.random.default_rng(5)
    si = np.concatenate([rng.integers(0, M, 3000), [0, M - 1, 0, M - 1, 127, 128, 255, 256]]).astype(np.uint32)
    sj = np.concatenate([rng.integers(0, N, 3000), [0, N - 1, N - 1, 0, N - 1, 0, 63, 32]]).astype(np.uint32)
    ref, ap = orc.sample(w.dtype, w.A, w.Bt, si, sj)
    got0 = C0[torch.from_numpy(si.astype(np.int64)).cuda(), torch.from_numpy(sj.astype(np.int64)).cuda()].cpu().numpy()
    assert close(got0, ref, TOL * ap).all()
    # the faulty run: rows / columns / elements no site reaches are bit-identical to the fault-free run
    hit_rows = set(int(s["row"]) for s in sites if s["kind"] != orc.KIND_B)
    hit_cols = set(int(s["col"]) for s in sites if s["kind"] == orc.KIND_B)
    same = (C0 == C1) | (torch.isnan(C0) & torch.isnan(C1))
    rows_ok = torch.ones(M, dtype=torch.bool, device="cuda"); rows_ok[list(hit_rows)] = False
    cols_ok = torch.ones(N, dtype=torch.bool, device="cuda")
    if hit_cols:
        cols_ok[list(hit_cols)] = False
    assert bool(same[rows_ok][:, cols_ok].all())
    # each site against the oracle's element-level view
    for t, s in enumerate(sites):
        kind, i, j = int(s["kind"]), int(s["row"]), int(s["col"])
        lg = log1[t]
        assert lg["status"] & 1
        if kind in (orc.KIND_A, orc.KIND_B):
            src = w.A[i, s["k"]] if kind == orc.KIND_A else w.Bt[j, s["k"]]
            assert lg["before_bits"] == int(src) and lg["after_bits"] == orc.flip_operand(w.dtype, int(src), int(s["xor_mask"]))
            # a few elements of the affected row / column, recomputed by the oracle with the faulty operand
            other = rng.integers(0, N if kind == orc.KIND_A else M, 64).astype(np.uint32)
            fix = np.full(64, i if kind == orc.KIND_A else j, dtype=np.uint32)
            ri, rj = (fix, other) if kind == orc.KIND_A else (other, fix)
            ref1, ap1 = orc.sample(w.dtype, w.A, w.Bt, ri, rj, sites)
            got1 = C1[torch.from_numpy(ri.astype(np.int64)).cuda(), torch.from_numpy(rj.astype(np.int64)).cuda()].cpu().numpy()
            if w.detect_mode & orc.CORRECT:
                ref1 = np.array([bits_f32(orc.boundcheck_correct(int(x))) for x in ref1.view(np.uint32)], dtype=np.float32)
            assert close(got1, ref1, TOL * ap1).all()
        else:
            assert lg["after_bits"] == lg["before_bits"] ^ s["xor_mask"]
            stored = int(C1[i, j].cpu().numpy().view(np.uint32))
            flagged = bool((bm1[i, j // 32] >> (j % 32)) & 1)
            if kind == orc.KIND_OUT:
                r0, a0 = orc.sample(w.dtype, w.A, w.Bt, np.array([i], np.uint32), np.array([j], np.uint32))
                assert close(bits_f32(lg["before_bits"]), r0[0], TOL * a0[0])
                want = orc.boundcheck_correct(int(lg["after_bits"])) if w.detect_mode & orc.CORRECT else int(lg["after_bits"])
                assert stored == want and flagged == bool(orc.boundcheck_detect(int(lg["after_bits"])))
            elif not (w.detect_mode & orc.CORRECT):
                assert flagged == bool(orc.boundcheck_detect(stored))
    # campaign on the same table: single-element trials are exact against the oracle's element evaluation
    Cc, rec = run_gpu_campaign(w.dtype, w.A, w.Bt, w.sites, w.detect_mode)
    elem = np.isin(w.sites["kind"], [orc.KIND_ACC, orc.KIND_TERM])
    if elem.any():
        idx = np.nonzero(elem)[0][:64]
        for t in idx:
            s = w.sites[t]
            i, j = int(s["row"]), int(s["col"])
            # the oracle on the 1 x 1 problem made of row i of A and row j of Bt is the same dot product
            sub = s.copy().reshape(1); sub["row"] = 0; sub["col"] = 0
            Cs, *_ = orc.gemm(w.dtype, w.A[i:i + 1], w.Bt[j:j + 1])
            ro = orc.campaign(w.dtype, w.A[i:i + 1], w.Bt[j:j + 1], Cs, sub, w.detect_mode)[0]
            raw = orc.campaign(w.dtype, w.A[i:i + 1], w.Bt[j:j + 1], Cs, sub, w.detect_mode & ~orc.CORRECT)[0]
            g = rec[t]
            assert g["before_bits"] == ro["before_bits"] and g["after_bits"] == ro["after_bits"]
            assert g["n_detected"] == ro["n_detected"] and (g["status"] & 7) == (ro["status"] & 7)
            if not np.isnan(bits_f32(raw["final_bits"])):      # NaN payloads are not part of parity
                assert g["final_bits"] == ro["final_bits"] and g["max_abs_dev"] == ro["max_abs_dev"]
    out = w.sites["kind"] == orc.KIND_OUT
    for t in np.nonzero(out)[0][:64]:
        s = w.sites[t]
        g = rec[t]
        assert g["before_bits"] == int(Cc[int(s["row"]), int(s["col"])].view(np.uint32))
        assert g["after_bits"] == g["before_bits"] ^ s["xor_mask"]
        assert g["n_detected"] == orc.boundcheck_detect(int(g["after_bits"]))


@pytest.mark.parametrize("name", ["c2", "c3a", "c4", "c5"])
def test_full_size_addend_on_sampled_outputs(name):
    """D = A x B + C_in at the benchmark's sizes and default launch configuration: sampled outputs against the oracle's
    chains that start from the addend, no flags on a clean workload with a small addend, and the elements of an
    accumulator / output site met by the addend-bearing sum."""
    w = synth.make_workload(name, trials=16)
    M, N, K = w.M, w.N, w.K
    a, b = to_dev(w.A, w.dtype), to_dev(w.Bt, w.dtype)
    g = torch.Generator(device="cuda"); g.manual_seed(99)
    cin = torch.randn((M, N), dtype=torch.float32, device="cuda", generator=g)
    kt = synth.kstep(w.dtype)
    sites = np.zeros(2, dtype=orc.SITE)
    sites["kind"] = [orc.KIND_ACC, orc.KIND_OUT]
    sites["row"] = [M - 3, 130]; sites["col"] = [N - 2, 33]; sites["k"] = [kt, 0]; sites["xor_mask"] = [1 << 21, 1 << 31]
    D, f = mpg.gemm(w.dtype, a, b, sites, w.detect_mode, addend=cin)
    torch.cuda.synchronize()
    hdr, log, bm = mpg.split_flags(f, M, N, 2)
    assert hdr[0] == 0 and hdr[1] == 0 and hdr[3] == 2 and not bm.any()
    rng = np.random.default_rng(6)
    si = np.concatenate([rng.integers(0, M, 3000), [0, M - 1, 0, M - 1, 127, 128, 255, 256]]).astype(np.uint32)
    sj = np.concatenate([rng.integers(0, N, 3000), [0, N - 1, N - 1, 0, N - 1, 0, 63, 32]]).astype(np.uint32)
    ti, tj = torch.from_numpy(si.astype(np.int64)).cuda(), torch.from_numpy(sj.astype(np.int64)).cuda()
    start = cin[ti, tj].cpu().numpy()
    ref, ap = orc.sample(w.dtype, w.A, w.Bt, si, sj, start=start)
    got = D[ti, tj].cpu().numpy()
    hit = ((si == M - 3) & (sj == N - 2)) | ((si == 130) & (sj == 33))
    assert close(got, ref, TOL * ap)[~hit].all()
    # the accumulator site met addend + the first k-step's products; the output site the finished sum
    i, j = M - 3, N - 2
    c0 = np.array([float(cin[i, j].cpu())], dtype=np.float32)
    r_acc, a_acc = orc.sample(w.dtype, np.ascontiguousarray(w.A[i:i + 1, :kt]), np.ascontiguousarray(w.Bt[j:j + 1, :kt]),
                              np.zeros(1, np.uint32), np.zeros(1, np.uint32), start=c0)
    assert close(bits_f32(log[0]["before_bits"]), r_acc[0], TOL * a_acc[0])
    assert log[0]["after_bits"] == log[0]["before_bits"] ^ (1 << 21)
    r_out, a_out = orc.sample(w.dtype, w.A, w.Bt, np.array([130], np.uint32), np.array([33], np.uint32),
                              start=np.array([float(cin[130, 33].cpu())], dtype=np.float32))
    assert close(bits_f32(log[1]["before_bits"]), r_out[0], TOL * a_out[0])
    assert int(D[130, 33].cpu().numpy().view(np.uint32)) == int(log[1]["before_bits"]) ^ (1 << 31)
