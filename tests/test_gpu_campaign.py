"""GPU parity: mpgemmfi_campaign through the C ABI against the oracle's incremental trial evaluation."""
import numpy as np
import pytest
import torch

import oracle as orc
import paper_2311_05782_b200 as mpg
import synth
from parity import check_campaign_against_oracle, run_gpu_campaign, run_gpu_gemm, to_dev

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,shape,trials", [
    ("c1", (256, 256, 256), 64),
    ("c2", (384, 640, 512), 128),
    ("c3a", (512, 384, 256), 256),
    ("c3b", (512, 256, 512), 256),
    ("c4", (256, 384, 544), 128),
    ("c5", (3000, 64, 576), 300),
])
def test_campaign_records_on_config_mixes(name, shape, trials):
    M, N, K = shape
    w = synth.make_workload(name, M, N, K, trials=trials)
    check_campaign_against_oracle(w.dtype, w.A, w.Bt, w.sites, w.detect_mode, max_fragile=2)


@pytest.mark.parametrize("tech", [orc.T_NONE, orc.T_BOUND, orc.T_RMAX, orc.T_RFLIP])
@pytest.mark.parametrize("nbits", [1, 2, 4])
def test_campaign_term_trials(tech, nbits):
    """The paper's own fault (1, 2 or 4 bits of one product, Section IV-C) under each technique."""
    M, N, K = 256, 256, 256
    A, Bt = synth.make_operands("c2", M, N, K)
    sites = synth.make_sites("term", orc.BF16, M, N, K, 256, 77 + nbits, nbits=nbits)
    check_campaign_against_oracle(orc.BF16, A, Bt, sites, tech | orc.CORRECT)
    check_campaign_against_oracle(orc.BF16, A, Bt, sites, tech)


def test_campaign_record_matches_single_site_gemm():
    """Consistency inside the CUDA path: a trial's record against mpgemmfi_gemm run with that one site."""
    w = synth.make_workload("c5", 1024, 64, 576, trials=60)
    Cc, rec = run_gpu_campaign(w.dtype, w.A, w.Bt, w.sites, w.detect_mode)
    for t in range(0, 60, 3):
        s = w.sites[t:t + 1]
        Cg, hdr, log, bm = run_gpu_gemm(w.dtype, w.A, w.Bt, s, w.detect_mode)
        kind = int(s["kind"][0])
        if kind == orc.KIND_OUT:
            assert rec[t]["before_bits"] == log["before_bits"][0] and rec[t]["after_bits"] == log["after_bits"][0]
            assert rec[t]["final_bits"] == log["final_bits"][0]
            assert rec[t]["n_detected"] == hdr[1]
        elif kind in (orc.KIND_A, orc.KIND_B):
            assert rec[t]["before_bits"] == log["before_bits"][0] and rec[t]["after_bits"] == log["after_bits"][0]
            assert abs(int(rec[t]["n_detected"]) - int(hdr[1])) <= 1
        else:
            assert abs(int(rec[t]["n_detected"]) - int(hdr[1])) <= 1


def test_campaign_edge_cases():
    A, Bt = synth.make_operands("c1", 128, 128, 64)
    a, b = to_dev(A, orc.FP16), to_dev(Bt, orc.FP16)
    # no trials: only the clean product is written
    Cc, rec = mpg.campaign(orc.FP16, a, b, None, orc.T_BOUND)
    torch.cuda.synchronize()
    Co, *_ = orc.gemm(orc.FP16, A, Bt)
    assert np.allclose(Cc.cpu().numpy(), Co, atol=1e-5) and rec.shape[0] == 0
    # invalid sites are reported in the record, valid ones still evaluated
    s = np.zeros(3, dtype=orc.SITE)
    s["kind"] = [orc.KIND_OUT, orc.KIND_ACC, 9]
    s["row"] = [500, 1, 0]; s["k"] = [0, 33, 0]; s["xor_mask"] = 1 << 30
    _, rec = run_gpu_campaign(orc.FP16, A, Bt, s, orc.T_BOUND)
    assert all(r["status"] & 0x100 for r in rec)
    # workspace too small / misaligned
    c = torch.empty((128, 128), dtype=torch.float32, device="cuda")
    r = torch.empty((4, 12), dtype=torch.int32, device="cuda")
    ws = torch.empty(4096, dtype=torch.uint8, device="cuda")
    st = torch.from_numpy(s.view(np.int32).reshape(3, 8)).cuda()
    cs = torch.cuda.current_stream().cuda_stream
    assert mpg.mpgemmfi_campaign(0, 128, 128, 64, a.data_ptr(), b.data_ptr(), c.data_ptr(), st.data_ptr(), 3, 1,
                                 r.data_ptr(), ws.data_ptr(), 16, cs) == -5
    assert mpg.mpgemmfi_campaign(0, 128, 128, 64, a.data_ptr(), b.data_ptr(), c.data_ptr(), st.data_ptr(), 3, 1,
                                 r.data_ptr(), ws.data_ptr() + 8, 2048, cs) == -5
    torch.cuda.synchronize()


@pytest.mark.parametrize("name,shape,trials", [("c5", (2048, 64, 576), 400), ("c2", (256, 384, 256), 200), ("c4", (256, 256, 256), 150)])
def test_campaign_summary_matches_oracle_reduction(name, shape, trials):
    """The device reduction of the records (zero-difference share, deviation histogram) against the oracle's."""
    M, N, K = shape
    w = synth.make_workload(name, M, N, K, trials=trials)
    sites = w.sites.copy()
    sites["kind"][3] = 9                                        # an invalid site must be left out of the counts
    view = np.int32 if w.dtype == orc.TF32 else np.int16
    a = torch.from_numpy(w.A.view(view)).cuda(); b = torch.from_numpy(w.Bt.view(view)).cuda()
    Cc, rec = mpg.campaign(w.dtype, a, b, sites, w.detect_mode)
    got = mpg.campaign_summary(rec)
    host = rec.cpu().numpy().view(np.uint32).reshape(-1).view(mpg.RECORD_DTYPE)
    want = orc.summary(host)                                    # same records: the reduction itself is bit-exact
    flat = np.concatenate([[got["n_trials"], got["n_invalid"], got["n_zero_diff"], got["n_detected"], got["n_corrected"],
                            got["n_nonfinite"]], got["kind_trials"], got["kind_zero_diff"], got["dev_exponent_hist"]])
    assert np.array_equal(flat.astype(np.uint32), want)
    assert got["n_invalid"] == 1 and got["n_trials"] == trials
    # and end to end against the oracle's own campaign: same zero-difference share for the exactly reproducible kinds
    Cclean, *_ = orc.gemm(w.dtype, w.A, w.Bt)
    ro = orc.campaign(w.dtype, w.A, w.Bt, Cclean, sites, w.detect_mode)
    so = orc.summary(ro)
    for kind in (orc.KIND_ACC, orc.KIND_TERM):
        assert got["kind_trials"][kind] == so[6 + kind] and got["kind_zero_diff"][kind] == so[11 + kind]
    assert np.array_equal(got["kind_trials"], so[6:11])
    # empty input
    empty = mpg.campaign_summary(rec[:0])
    assert empty["n_trials"] == 0 and empty["dev_exponent_hist"].sum() == 0


@pytest.mark.parametrize("dtype,name", [(orc.FP16, "c1"), (orc.BF16, "c2"), (orc.TF32, "c4")])
@pytest.mark.parametrize("nbits", [1, 2, 4])
def test_campaign_term_trials_at_hmma_granularity(dtype, name, nbits):
    """The paper's own trial (Section IV-A): uniform element, uniform term, 1/2/4 flipped bits of the product,
    written back into the sum that one HMMA leaves (16 terms for FP16/BF16, 8 for TF32)."""
    M, N, K = 192, 160, 208
    A, Bt = synth.make_operands(name, M, N, K)
    sites = synth.make_sites("term", dtype, M, N, K, 300, 99 + nbits, nbits=nbits)
    step = 8 if dtype == orc.TF32 else 16
    for tech in (orc.T_NONE, orc.T_BOUND | orc.CORRECT, orc.T_RMAX | orc.CORRECT, orc.T_RFLIP | orc.CORRECT):
        _, rg = run_gpu_campaign(dtype, A, Bt, sites, tech | mpg.TERM_HMMA_STEP)
        Cclean, *_ = orc.gemm(dtype, A, Bt)
        ro = orc.campaign(dtype, A, Bt, Cclean, sites, tech, kstep=step)
        raw = orc.campaign(dtype, A, Bt, Cclean, sites, tech & ~orc.CORRECT, kstep=step)
        nan_made = np.isnan(raw["final_bits"].view(np.float32))
        for f in rg.dtype.names:
            same = rg[f] == ro[f]
            if f in ("final_bits", "max_abs_dev"):
                same |= nan_made                                 # NaN payloads are not part of parity
            assert same.all(), (f, np.nonzero(~same)[0][:5])
        # the granularity matters: with the GEMM's k-step some of these trials end differently
        _, rk = run_gpu_campaign(dtype, A, Bt, sites, tech)
        assert np.array_equal(rk["before_bits"], rg["before_bits"])
    # the flag is a campaign-only option
    a, b = to_dev(A, dtype), to_dev(Bt, dtype)
    with pytest.raises(mpg.MpgemmfiError):
        mpg.gemm(dtype, a, b, sites[:1], mpg.TERM_HMMA_STEP)


def test_campaign_single_element_trials_with_special_values():
    """ACC / TERM / OUT trials on operands that hold zeros, Inf, NaN and huge values: both sides walk the same
    sums in the same order, so the records agree bit for bit (NaN payloads aside)."""
    M, N, K = 96, 80, 200
    rng = np.random.default_rng(51)
    a = rng.standard_normal((M, K)).astype(np.float32); b = rng.standard_normal((N, K)).astype(np.float32)
    a[rng.random((M, K)) < 0.4] = 0.0
    a[5, 17] = np.inf; a[9, 3] = np.nan; a[20, 100] = 1e30; b[7, 17] = -np.inf; b[30, 100] = 1e30; b[11, :] = 0.0
    A, Bt = synth.round_to_storage(a, orc.BF16), synth.round_to_storage(b, orc.BF16)
    parts = []
    for mix, seed in (("acc", 1), ("term", 2), ("out", 3)):
        s = synth.make_sites(mix, orc.BF16, M, N, K, 200, seed, nbits=2)
        parts.append(s)
    sites = np.concatenate(parts)
    sites["row"][:12] = [5, 5, 9, 9, 20, 20, 5, 9, 20, 5, 9, 20]          # make sure the special rows / columns are hit
    sites["col"][:12] = [7, 30, 7, 11, 30, 11, 0, 1, 2, 11, 30, 7]
    for mode in (orc.T_BOUND | orc.CORRECT, orc.T_RMAX | orc.CORRECT, orc.T_NONE):
        Cg, rg = run_gpu_campaign(orc.BF16, A, Bt, sites, mode)
        Cclean, *_ = orc.gemm(orc.BF16, A, Bt)
        elem = sites["kind"] != orc.KIND_OUT
        ro = orc.campaign(orc.BF16, A, Bt, Cclean, sites, mode)
        raw = orc.campaign(orc.BF16, A, Bt, Cclean, sites, mode & ~orc.CORRECT)
        nan_made = np.isnan(raw["final_bits"].view(np.float32)) | np.isnan(raw["before_bits"].view(np.float32))
        for f in rg.dtype.names:
            same = (rg[f] == ro[f])
            if f in ("final_bits", "max_abs_dev", "before_bits", "after_bits"):
                same |= nan_made
            if f == "max_abs_dev":
                same |= np.isnan(rg[f]) & np.isnan(ro[f])
            if f == "status":
                # "changed" compares bit patterns: between two NaNs it depends on payloads, which are not part of parity
                clean_nan = np.isnan(Cclean.reshape(-1)[np.minimum(ro["primary_index"], M * N - 1)])
                same |= ((rg[f] ^ ro[f]) == 1) & (nan_made | clean_nan)
            assert same[elem].all(), (mode, f, np.nonzero(~same & elem)[0][:5])
        out = ~elem
        assert np.array_equal(rg["after_bits"][out], rg["before_bits"][out] ^ sites["xor_mask"][out])
        assert np.array_equal(rg["n_detected"][out], np.array([orc.boundcheck_detect(int(x)) if (mode & 3) == 1 else 0
                                                               for x in rg["after_bits"][out]]))


@pytest.mark.parametrize("seed", range(12))
def test_campaign_random_shapes_mixes_and_modes(seed):
    """Differential fuzz of the campaign against the oracle's incremental evaluation (finite operands)."""
    rng = np.random.default_rng(3000 + seed)
    dtype = int(rng.integers(0, 3))
    unit = 4 if dtype == orc.TF32 else 8
    M = int(rng.integers(1, 500)); N = int(rng.integers(1, 300)); K = unit * int(rng.integers(1, 50))
    if seed % 4 == 0:
        M, N, K = int(rng.integers(2100, 2600)), int(rng.integers(8, 70)), unit * int(rng.integers(8, 40))   # panel path
    mode = int(rng.choice([orc.T_NONE, orc.T_BOUND, orc.T_BOUND | orc.CORRECT, orc.T_RMAX | orc.CORRECT]))
    a = (rng.standard_normal((M, K)) * rng.choice([0.05, 1.0])).astype(np.float32)
    b = (rng.standard_normal((N, K)) * rng.choice([0.05, 1.0])).astype(np.float32)
    a[rng.random((M, K)) < 0.2] = 0.0
    A, Bt = synth.round_to_storage(a, dtype), synth.round_to_storage(b, dtype)
    parts = [synth.make_sites(mix, dtype, M, N, K, 40, 4000 + seed + i, nbits=int(rng.choice([1, 2, 4])))
             for i, mix in enumerate(("mixed", "term", "operand"))]
    sites = np.concatenate(parts)
    sites["kind"][5] = 11                                   # an invalid entry
    check_campaign_against_oracle(dtype, A, Bt, sites, mode, max_fragile=3)


def _widen_np(dtype, bits):
    """Library conversions only: numpy's half type, or the storage word moved into a float32 word."""
    bits = np.asarray(bits)
    if dtype == orc.FP16:
        return bits.astype(np.uint16).view(np.float16).astype(np.float32)
    if dtype == orc.BF16:
        return (bits.astype(np.uint32) << 16).view(np.float32)
    return (bits.astype(np.uint32) & np.uint32(0xFFFFE000)).view(np.float32)


@pytest.mark.parametrize("dtype,shape,n", [(orc.FP16, (8192, 64, 128), 160), (orc.BF16, (8192, 64, 128), 160),
                                           (orc.FP16, (700, 520, 72), 160), (orc.TF32, (600, 200, 64), 160),
                                           (orc.FP16, (4608, 64, 576), 5000), (orc.TF32, (2048, 40, 64), 2500)])
@pytest.mark.parametrize("mode", [orc.T_NONE, orc.T_BOUND | orc.CORRECT])
def test_operand_trials_are_eq1_eq2_on_the_clean_sum_bit_for_bit(dtype, shape, n, mode):
    """An operand trial's statistics are those of Eq. 1-2 applied to the device's own clean C with every product and
    every sum rounded to FP32, bit for bit: first against the oracle's write-back form (all record fields), then
    against numpy float32 arithmetic (one rounding per operation) restated here.
    Covers the row-panel kernel (long columns: the first two and the last two shapes, the last two with several groups of
    1024 column trials, so that full and partial groups and their bank-wise dealing to warps all occur) and the
    one-CTA-per-trial kernel."""
    M, N, K = shape
    rng = np.random.default_rng(91)
    A = synth.round_to_storage(np.maximum(rng.standard_normal((M, K)), 0).astype(np.float32), dtype)   # zeros among the values
    Bt = synth.round_to_storage((rng.standard_normal((N, K)) * 0.1).astype(np.float32), dtype)
    s = np.zeros(n, dtype=orc.SITE)
    s["kind"] = rng.integers(0, 2, n)
    s["row"] = rng.integers(0, M, n); s["col"] = rng.integers(0, N, n); s["k"] = rng.integers(0, K, n)
    width = 19 if dtype == orc.TF32 else 16
    s["xor_mask"] = [1 << int(b) for b in rng.integers(0, width, n)]
    Cg, rec = run_gpu_campaign(dtype, A, Bt, s, mode)
    # the oracle's form of the same thing: Eq. 1-2 on the finished sums of the clean C the device produced
    rw = orc.campaign(dtype, A, Bt, Cg, s, mode, operand_form=1)
    # a faulty operand that is Inf or NaN puts NaNs among the values (Inf * 0); what the correction makes of a NaN
    # depends on its payload, which is left open
    special = ~np.isfinite(np.array([orc.widen(dtype, int(x)) for x in rw["after_bits"]]))
    for f in rec.dtype.names:
        same = rec[f] == rw[f]
        if f in ("max_abs_dev", "status"):
            same |= special
        assert same.all(), (f, np.nonzero(~same)[0][:5], rec[~same][:2], rw[~same][:2])
    HASH_MUL = 0x9E3779B97F4A7C15
    with np.errstate(all="ignore"):
        for t in range(n):
            is_a = int(s["kind"][t]) == orc.KIND_A
            i, j, k = int(s["row"][t]), int(s["col"][t]), int(s["k"][t])
            w_clean = int(A[i, k]) if is_a else int(Bt[j, k])
            x = _widen_np(dtype, np.array([w_clean]))[0]
            xf = _widen_np(dtype, np.array([orc.flip_operand(dtype, w_clean, int(s["xor_mask"][t]))]))[0]
            y = _widen_np(dtype, Bt[:, k] if is_a else A[:, k])
            c = Cg[i, :] if is_a else Cg[:, j]
            lin = (i * N + np.arange(N)) if is_a else (np.arange(M) * N + j)
            cf = (c - x * y).astype(np.float32) + (xf * y).astype(np.float32)       # Eq. 1, Eq. 2: four roundings
            fin = cf.view(np.uint32).copy()
            det = np.zeros(len(c), dtype=bool)
            if (mode & 3) == orc.T_BOUND:
                det = ~(np.abs(cf) < np.float32(131072.0))
                if mode & orc.CORRECT:
                    fin[det] &= np.uint32(~(7 << 27) & 0xFFFFFFFF)
            g = rec[t]
            assert g["n_affected"] == len(c) and g["n_detected"] == det.sum(), t
            if np.isnan(cf).any():
                continue                      # NaN payloads are not part of parity
            dev = np.abs(fin.view(np.float32) - c)
            assert g["max_abs_dev"].view(np.uint32) == np.float32(dev.max()).view(np.uint32), (t, g["max_abs_dev"], dev.max())
            assert bool(g["status"] & 1) == bool((fin != c.view(np.uint32)).any())
            if det.any():
                assert g["first_detected"] == lin[det].min()
                assert int(g["idx_hash"]) == sum((int(l) + 1) * HASH_MUL for l in lin[det]) & ((1 << 64) - 1)


@pytest.mark.parametrize("workload,fmt,nbits,mode", [("relu_k576", orc.FP16, 1, 0), ("relu_k576", orc.BF16, 4, orc.T_BOUND | orc.CORRECT),
                                                     ("gelu_k4096", orc.TF32, 2, orc.T_RMAX | orc.CORRECT),
                                                     ("gelu_k4096", orc.FP16, 4, orc.T_RFLIP | orc.CORRECT)])
def test_deviation_study_cell_against_the_oracle(workload, fmt, nbits, mode):
    """A cell of the deviation study (term trials at HMMA granularity, reduced on the device) against the oracle's
    campaign and summary on the same operands and trial table: the whole summary, word for word."""
    from paper_2311_05782_b200 import deviation_study as ds
    trials = 600
    summ, cell = ds.run_cell(mpg, synth, torch, workload, fmt, nbits, mode, trials)
    cfg, M, N, K = ds.WORKLOADS[workload]
    A, Bt = synth.make_operands(cfg, M, N, K, dtype=fmt)
    sites = synth.make_sites("term", fmt, M, N, K, trials, synth.config_seed(cfg) + 100 * nbits + 1, nbits=nbits)
    # the oracle needs only the rows of A and Bt that the trials touch: one 1 x 1 problem per trial
    rec = np.zeros(trials, dtype=orc.RECORD)
    for t, s in enumerate(sites):
        i, j = int(s["row"]), int(s["col"])
        one = s.copy().reshape(1); one["row"] = 0; one["col"] = 0
        Cs, *_ = orc.gemm(fmt, A[i:i + 1], Bt[j:j + 1])
        rec[t] = orc.campaign(fmt, A[i:i + 1], Bt[j:j + 1], Cs, one, mode, kstep=8 if fmt == orc.TF32 else 16)[0]
    want = orc.summary(rec)
    raw = np.zeros(trials, dtype=orc.RECORD)
    got = np.concatenate([[summ["n_trials"], summ["n_invalid"], summ["n_zero_diff"], summ["n_detected"], summ["n_corrected"],
                           summ["n_nonfinite"]], summ["kind_trials"], summ["kind_zero_diff"], summ["dev_exponent_hist"]]).astype(np.uint32)
    # a NaN that a fault creates keeps an unspecified payload through the later additions; what a correction makes of it
    # is then not unique: such trials can sit in different bins on the two sides, all others must agree
    nan_made = sum(1 for r in rec if np.isnan(np.uint32(r["final_bits"]).view(np.float32)) or np.isinf(r["max_abs_dev"]))
    diff = np.abs(got.astype(np.int64) - want.astype(np.int64))
    assert diff[:5].sum() == 0 and diff[6:16].sum() == 0, (got[:16], want[:16])
    assert diff[16:].sum() <= 2 * nan_made and diff[5] <= nan_made
    assert cell["trials"] == trials and abs(cell["zero_diff_pct"] - 100.0 * want[2] / trials) < 1e-9


@pytest.mark.parametrize("dtype,name", [(orc.FP16, "c5"), (orc.BF16, "c2"), (orc.TF32, "c4")])
@pytest.mark.parametrize("nbits", [1, 2, 4])
def test_campaign_term_trials_with_the_product_in_the_operand_format(dtype, name, nbits):
    """MPGEMMFI_TERM_IN_FORMAT: the product rounded to the operand format, flipped there, written back by Eq. 1-2.
    Both sides walk the same sums in the same order: the records agree bit for bit (NaN payloads aside), at the GEMM's
    k-step and at HMMA granularity, under every technique."""
    M, N, K = 192, 160, 208
    A, Bt = synth.make_operands(name, M, N, K, dtype=dtype)
    sites = synth.make_sites("term_op", dtype, M, N, K, 300, 199 + nbits, nbits=nbits)
    step = 8 if dtype == orc.TF32 else 16
    Cclean, *_ = orc.gemm(dtype, A, Bt)
    for tech in (orc.T_NONE, orc.T_BOUND | orc.CORRECT, orc.T_RMAX | orc.CORRECT, orc.T_RFLIP | orc.CORRECT, orc.T_RMAX):
        for hmma in (True, False):
            _, rg = run_gpu_campaign(dtype, A, Bt, sites, tech | mpg.TERM_IN_FORMAT | (mpg.TERM_HMMA_STEP if hmma else 0))
            ro = orc.campaign(dtype, A, Bt, Cclean, sites, tech | orc.TERM_IN_FORMAT, kstep=step if hmma else None)
            raw = orc.campaign(dtype, A, Bt, Cclean, sites, (tech & ~orc.CORRECT) | orc.TERM_IN_FORMAT, kstep=step if hmma else None)
            nan_made = np.isnan(raw["final_bits"].view(np.float32))
            for f in rg.dtype.names:
                same = rg[f] == ro[f]
                if f in ("final_bits", "max_abs_dev"):
                    same |= nan_made
                if f == "max_abs_dev":
                    same |= np.isnan(rg[f]) & np.isnan(ro[f])
                assert same.all(), (tech, hmma, f, np.nonzero(~same)[0][:5], rg[~same][:2], ro[~same][:2])
    # it changes what a trial does: an FP16 zero product with a flipped mantissa bit now shows in the sum
    if dtype == orc.FP16:
        _, r32 = run_gpu_campaign(dtype, A, Bt, sites, mpg.TERM_HMMA_STEP)
        _, r16 = run_gpu_campaign(dtype, A, Bt, sites, mpg.TERM_HMMA_STEP | mpg.TERM_IN_FORMAT)
        assert (r16["status"] & 1).sum() > (r32["status"] & 1).sum()
    # the GEMM entry point does not take the flag
    with pytest.raises(mpg.MpgemmfiError):
        mpg.gemm(dtype, to_dev(A, dtype), to_dev(Bt, dtype), sites[:1], mpg.TERM_IN_FORMAT)
