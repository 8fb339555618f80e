"""Pins for the oracle's GEMM, fault application and records (CPU only)."""
import struct

import numpy as np
import pytest

import oracle as orc
import synth

HASH_MUL = 0x9E3779B97F4A7C15
MASK64 = (1 << 64) - 1


def f32_bits(x):
    return struct.unpack("<I", struct.pack("<f", x))[0]


def bits_f32(u):
    return struct.unpack("<f", struct.pack("<I", u & 0xFFFFFFFF))[0]


def int_operands(dtype, M, N, K, seed, lo=-8, hi=9):
    """Small integers: every product and partial sum is exact in FP32 and in all three formats."""
    rng = np.random.default_rng(seed)
    a = rng.integers(lo, hi, size=(M, K)).astype(np.float32)
    b = rng.integers(lo, hi, size=(N, K)).astype(np.float32)
    return a, b, synth.round_to_storage(a, dtype), synth.round_to_storage(b, dtype)


def site(kind, row=0, col=0, k=0, mask=0):
    s = np.zeros(1, dtype=orc.SITE)
    s["kind"], s["row"], s["col"], s["k"], s["xor_mask"] = kind, row, col, k, mask
    return s


@pytest.mark.parametrize("dtype", [orc.FP16, orc.BF16, orc.TF32])
def test_exact_integer_gemm_nonsquare(dtype):
    """C = A x B exactly for small integers; non-square shapes catch a transposed operand or swapped index."""
    M, N, K = 5, 7, 11
    a, b, A, Bt = int_operands(dtype, M, N, K, 1)
    Cm, hdr, _, bm = orc.gemm(dtype, A, Bt)
    ref = a.astype(np.int64) @ b.astype(np.int64).T
    assert np.array_equal(Cm.astype(np.int64), ref) and Cm.shape == (M, N)
    assert hdr[1] == 0 and not bm.any()


def test_k1_and_identity_special_cases():
    rng = np.random.default_rng(2)
    x = rng.standard_normal((6, 1)).astype(np.float32)
    y = rng.standard_normal((4, 1)).astype(np.float32)
    A, Bt = synth.round_to_storage(x, orc.BF16), synth.round_to_storage(y, orc.BF16)
    Cm, *_ = orc.gemm(orc.BF16, A, Bt)
    xa = (A.astype(np.uint32) << 16).view(np.float32)
    ya = (Bt.astype(np.uint32) << 16).view(np.float32)
    assert np.array_equal(Cm, xa @ ya.T)           # one exact product per element
    # B = identity: C reproduces A (widened) exactly
    a = rng.standard_normal((5, 8)).astype(np.float32)
    A = synth.round_to_storage(a, orc.FP16)
    I = synth.round_to_storage(np.eye(8, dtype=np.float32), orc.FP16)
    Cm, *_ = orc.gemm(orc.FP16, A, I)
    assert np.array_equal(Cm, A.view(np.float16).astype(np.float32))


@pytest.mark.parametrize("dtype", [orc.FP16, orc.BF16, orc.TF32])
def test_random_gemm_against_float64_and_sequential_float32(dtype):
    """Within K*2^-24*(|A||B|) of the exact product; bit-equal to a scalar float32 loop in k order."""
    M, N, K = 6, 5, 37
    rng = np.random.default_rng(3)
    A = synth.round_to_storage(rng.standard_normal((M, K)).astype(np.float32), dtype)
    Bt = synth.round_to_storage(rng.standard_normal((N, K)).astype(np.float32), dtype)
    af = np.array([[orc.widen(dtype, int(v)) for v in r] for r in A], dtype=np.float32)
    bf = np.array([[orc.widen(dtype, int(v)) for v in r] for r in Bt], dtype=np.float32)
    Cm, *_ = orc.gemm(dtype, A, Bt)
    exact = af.astype(np.float64) @ bf.astype(np.float64).T
    ap = np.abs(af).astype(np.float64) @ np.abs(bf).astype(np.float64).T
    assert np.all(np.abs(Cm - exact) <= K * 2.0 ** -24 * ap)
    assert np.allclose(orc.absprod(dtype, A, Bt), ap, rtol=1e-12)
    for i in range(M):
        for j in range(N):
            acc = np.float32(0.0)
            for k in range(K):
                acc = np.float32(acc + np.float32(af[i, k] * bf[j, k]))
            assert f32_bits(float(acc)) == f32_bits(float(Cm[i, j]))
    si = np.array([0, 3, 5], dtype=np.uint32); sj = np.array([4, 0, 2], dtype=np.uint32)
    sc, sap = orc.sample(dtype, A, Bt, si, sj)
    assert np.array_equal(sc, Cm[si, sj]) and np.allclose(sap, ap[si, sj], rtol=1e-12)


@pytest.mark.parametrize("dtype", [orc.FP16, orc.BF16, orc.TF32])
def test_operand_sites_are_linear_and_local(dtype):
    """An A[i,k] fault changes only row i, by exactly delta*B[k,:]; a B[k,j] fault only column j."""
    M, N, K = 6, 7, 9
    a, b, A, Bt = int_operands(dtype, M, N, K, 4, lo=1, hi=5)
    C0, *_ = orc.gemm(dtype, A, Bt)
    i, k, j = 2, 5, 3
    # flip the lowest mantissa bit that keeps the operand an integer: use the sign bit and an exponent bit
    sign = 18 if dtype == orc.TF32 else 15
    exp_lsb = {orc.FP16: 10, orc.BF16: 7, orc.TF32: 10}[dtype]
    for mask in (1 << sign, 1 << exp_lsb):
        C1, hdr, log, _ = orc.gemm(dtype, A, Bt, site(orc.KIND_A, row=i, k=k, mask=mask))
        a_new = orc.widen(dtype, orc.flip_operand(dtype, int(A[i, k]), mask))
        assert log["before_bits"][0] == int(A[i, k]) and hdr[3] == 1
        delta = a_new - a[i, k]
        rows = np.arange(M) != i
        assert np.array_equal(C1[rows], C0[rows])
        assert np.array_equal(C1[i], C0[i] + np.float32(delta) * b[:, k])
        C2, *_ = orc.gemm(dtype, A, Bt, site(orc.KIND_B, col=j, k=k, mask=mask))
        b_new = orc.widen(dtype, orc.flip_operand(dtype, int(Bt[j, k]), mask))
        cols = np.arange(N) != j
        assert np.array_equal(C2[:, cols], C0[:, cols])
        assert np.array_equal(C2[:, j], C0[:, j] + a[:, k] * np.float32(b_new - b[j, k]))
    # the same fault twice cancels
    two = np.concatenate([site(orc.KIND_A, row=i, k=k, mask=0x21), site(orc.KIND_A, row=i, k=k, mask=0x21)])
    C3, *_ = orc.gemm(dtype, A, Bt, two)
    assert np.array_equal(C3, C0)


def test_acc_site_flips_the_running_sum_at_its_boundary():
    M, N, K = 3, 4, 12
    a, b, A, Bt = int_operands(orc.BF16, M, N, K, 5)
    C0, *_ = orc.gemm(orc.BF16, A, Bt)
    i, j = 1, 2
    for kb in (1, 4, 8, 12):
        prefix = np.float32(np.dot(a[i, :kb], b[j, :kb]))
        rest = np.float32(np.dot(a[i, kb:], b[j, kb:]))
        for mask in (0, 1 << 31, 1 << 23, 0x00400000, 3 << 20):
            C1, _, log, _ = orc.gemm(orc.BF16, A, Bt, site(orc.KIND_ACC, i, j, kb, mask), 0, kstep=4)
            assert log["before_bits"][0] == f32_bits(float(prefix))
            assert log["after_bits"][0] == f32_bits(float(prefix)) ^ mask
            flipped = np.float32(bits_f32(f32_bits(float(prefix)) ^ mask))
            want = flipped
            for k in range(kb, K):     # continue the sequential accumulation from the flipped value
                want = np.float32(want + np.float32(a[i, k] * b[j, k]))
            assert f32_bits(float(C1[i, j])) == f32_bits(float(want))
            C1[i, j] = C0[i, j]
            assert np.array_equal(C1, C0)       # nothing else moved; mask 0 is a bitwise no-op
            if mask == 0:
                assert prefix + rest == C0[i, j]


def test_term_site_write_back_is_exact_on_integers():
    """Eq. 1-2 with no rounding: re'_sum - re_sum = re_err - re_2; applied at the boundary ending k's tile."""
    M, N, K = 3, 3, 16
    a, b, A, Bt = int_operands(orc.FP16, M, N, K, 6, lo=1, hi=4)
    C0, *_ = orc.gemm(orc.FP16, A, Bt)
    i, j = 2, 1
    for k in (0, 3, 4, 15):
        re2 = np.float32(a[i, k] * b[j, k])
        for mask in (1 << 31, 1 << 22, 1 << 23):
            C1, _, log, _ = orc.gemm(orc.FP16, A, Bt, site(orc.KIND_TERM, i, j, k, mask), 0, kstep=4)
            re_err = np.float32(bits_f32(f32_bits(float(re2)) ^ mask))
            assert log["before_bits"][0] == f32_bits(float(re2))
            assert float(C1[i, j]) - float(C0[i, j]) == float(re_err) - float(re2)
    # mask 0 away from exact data: at most two roundings of the running sum
    rng = np.random.default_rng(7)
    A = synth.round_to_storage(rng.standard_normal((2, 40)).astype(np.float32), orc.BF16)
    Bt = synth.round_to_storage(rng.standard_normal((2, 40)).astype(np.float32), orc.BF16)
    C0, *_ = orc.gemm(orc.BF16, A, Bt)
    ap = orc.absprod(orc.BF16, A, Bt)
    C1, *_ = orc.gemm(orc.BF16, A, Bt, site(orc.KIND_TERM, 1, 0, 17, 0), 0, kstep=8)
    assert abs(float(C1[1, 0]) - float(C0[1, 0])) <= 2 * 2.0 ** -23 * ap[1, 0]
    # the boundary matters: with kstep 8 the term k=17 is rewritten after k=23, not after k=17
    af = (A.astype(np.uint32) << 16).view(np.float32); bf = (Bt.astype(np.uint32) << 16).view(np.float32)
    acc = np.float32(0)
    for k in range(40):
        acc = np.float32(acc + np.float32(af[1, k] * bf[0, k]))
        if k + 1 == 24:
            p = np.float32(af[1, 17] * bf[0, 17])
            acc = np.float32(np.float32(acc - p) + np.float32(bits_f32(f32_bits(float(p)) ^ (1 << 30))))
    C2, *_ = orc.gemm(orc.BF16, A, Bt, site(orc.KIND_TERM, 1, 0, 17, 1 << 30), 0, kstep=8)
    assert f32_bits(float(C2[1, 0])) == f32_bits(float(acc))


def brute_flags(Cm):
    M, N = Cm.shape
    bm = np.zeros((M, (N + 31) // 32), dtype=np.uint32)
    n = 0
    for i in range(M):
        for j in range(N):
            if abs(float(Cm[i, j])) >= 131072.0 or np.isnan(Cm[i, j]):
                bm[i, j // 32] |= np.uint32(1 << (j % 32)); n += 1
    return bm, n


def test_flag_bitmap_and_counts_bruteforce():
    """Flag = |value| >= 131072 (Table III threshold) or NaN; bit j%32 of word i*ceil(N/32)+j/32; count = popcount."""
    M, N, K = 9, 70, 8
    rng = np.random.default_rng(8)
    a = rng.standard_normal((M, K)).astype(np.float32)
    b = rng.standard_normal((N, K)).astype(np.float32)
    a[rng.integers(0, M, 5), rng.integers(0, K, 5)] *= 1e6      # some legitimately huge values
    A, Bt = synth.round_to_storage(a, orc.BF16), synth.round_to_storage(b, orc.BF16)
    sites = np.concatenate([site(orc.KIND_OUT, 8, 69, 0, 1 << 30), site(orc.KIND_OUT, 0, 33, 0, 1 << 29),
                            site(orc.KIND_OUT, 4, 31, 0, 1 << 30), site(orc.KIND_OUT, 99, 0, 0, 1)])
    raw, hdr0, *_ = orc.gemm(orc.BF16, A, Bt, sites, 0)
    assert hdr0[3] == 3 and hdr0[4] == 1 and hdr0[0] & 1          # the out-of-range site is skipped and reported
    Cd, hdr, log, bm = orc.gemm(orc.BF16, A, Bt, sites, orc.T_BOUND)
    want_bm, want_n = brute_flags(raw)
    assert np.array_equal(Cd.view(np.uint32), raw.view(np.uint32))    # detect-only leaves values alone
    assert np.array_equal(bm, want_bm) and hdr[1] == want_n and hdr[2] == 0 and want_n >= 3
    assert sum(bin(int(w)).count("1") for w in bm.reshape(-1)) == hdr[1]
    Cc, hdrc, logc, bmc = orc.gemm(orc.BF16, A, Bt, sites, orc.T_BOUND | orc.CORRECT)
    assert np.array_equal(bmc, want_bm) and hdrc[2] == want_n
    for i in range(M):
        for j in range(N):
            assert f32_bits(float(Cc[i, j])) == orc.boundcheck_correct(f32_bits(float(raw[i, j])))
    assert not brute_flags(Cc)[0].any()


def brute_record_stats(vals, clean, lins, detect_mode):
    n_det, h, first, maxdev, changed = 0, 0, 0xFFFFFFFF, 0.0, 0
    for v, c, lin in zip(vals, clean, lins):
        bits = f32_bits(float(v))
        det = orc.boundcheck_detect(bits) if (detect_mode & 3) == 1 else 0
        if det and detect_mode & orc.CORRECT:
            bits = orc.boundcheck_correct(bits)
        if det:
            n_det += 1; h = (h + (lin + 1) * HASH_MUL) & MASK64; first = min(first, lin)
        changed |= int(bits != f32_bits(float(c)))
        d = abs(np.float32(bits_f32(bits)) - np.float32(c))
        d = float("inf") if np.isnan(d) else float(d)
        maxdev = max(maxdev, d)
    return n_det, h, first, maxdev, changed


def record_from_full_recompute(Cf, bm, Cclean, lins, detect_mode):
    """What a trial's record must say, read off a full fault-injected GEMM with that one site: the flagged set is the
    GEMM's bitmap, the final values are the GEMM's output."""
    N = Cf.shape[1]
    n_det, h, first, maxdev, changed = 0, 0, 0xFFFFFFFF, 0.0, 0
    for lin in lins:
        i, j = divmod(lin, N)
        if (int(bm[i, j // 32]) >> (j % 32)) & 1:
            n_det += 1; h = (h + (lin + 1) * HASH_MUL) & MASK64; first = min(first, lin)
        fin, cl = Cf[i, j], Cclean[i, j]
        changed |= int(f32_bits(float(fin)) != f32_bits(float(cl)))
        with np.errstate(all="ignore"):
            d = abs(np.float32(fin) - np.float32(cl))
        maxdev = max(maxdev, float("inf") if np.isnan(d) else float(d))
    status = changed | (2 if n_det else 0) | (4 if n_det and (detect_mode & orc.CORRECT) and (detect_mode & 3) == 1 else 0)
    return n_det, h, first, maxdev, status


@pytest.mark.parametrize("name,mix,mode", [
    ("c1", "out", None), ("c2", "operand", None), ("c4", "acc2", None), ("c5", "mixed", None), ("c2", "term", None),
    ("c2", "term", orc.T_BOUND), ("c2", "term", orc.T_RMAX | orc.CORRECT), ("c2", "term", orc.T_RFLIP | orc.CORRECT),
    ("c5", "mixed", orc.T_NONE), ("c2", "term_op", orc.TERM_IN_FORMAT), ("c1", "term_op", orc.T_BOUND | orc.CORRECT | orc.TERM_IN_FORMAT),
    ("c4", "term_op", orc.T_RMAX | orc.CORRECT | orc.TERM_IN_FORMAT)])
def test_incremental_trials_equal_full_recompute(name, mix, mode):
    """Every trial record equals what a full fault-injected GEMM with that single site gives: the full recompute is
    the definition. ("c2", "term") runs TERM trials under BoundCheck + correction, where a product-level correction
    is followed by the output check on the corrected sum."""
    M, N, K = 24, 40, 96
    w = synth.make_workload(name, M, N, K, trials=40, mix=mix)
    dt = w.dtype
    mode = w.detect_mode if mode is None else mode
    if mix == "term":
        # single-bit flips of small products rarely reach the thresholds: put some masks on the exponent's top bits
        w.sites["xor_mask"][::3] = 1 << 30
        w.sites["xor_mask"][1::6] = 3 << 29
    if mix == "term_op":
        top = 18 if dt == orc.TF32 else 15
        w.sites["xor_mask"][::3] = 1 << (top - 1)
    Cclean, *_ = orc.gemm(dt, w.A, w.Bt)
    rec = orc.campaign(dt, w.A, w.Bt, Cclean, w.sites, mode)
    seen_status = set()
    for t in range(len(w.sites)):
        s = w.sites[t:t + 1]
        Cf, hdr, log, bm = orc.gemm(dt, w.A, w.Bt, s, mode)
        kind = int(s["kind"][0]); i, j = int(s["row"][0]), int(s["col"][0])
        if kind == orc.KIND_A:
            lins = [i * N + jj for jj in range(N)]
        elif kind == orc.KIND_B:
            lins = [ii * N + j for ii in range(M)]
        else:
            lins = [i * N + j]
        r = rec[t]
        # (1) the record read off the full recompute's output and bitmap
        n_det, h, first, maxdev, status = record_from_full_recompute(Cf, bm, Cclean, lins, mode)
        assert r["kind"] == kind and r["n_affected"] == len(lins)
        assert r["n_detected"] == n_det == hdr[1]
        assert int(r["idx_hash"]) == h and r["first_detected"] == first
        assert r["status"] == status, (t, r["status"], status)
        assert float(r["max_abs_dev"]) == maxdev or (np.isinf(maxdev) and np.isinf(r["max_abs_dev"]))
        assert r["before_bits"] == log["before_bits"][0] and r["after_bits"] == log["after_bits"][0]
        if kind in (orc.KIND_OUT, orc.KIND_ACC, orc.KIND_TERM):
            assert r["final_bits"] == f32_bits(float(Cf[i, j])) and r["primary_index"] == i * N + j
        else:
            assert r["final_bits"] == log["final_bits"][0] == log["after_bits"][0]
            assert r["primary_index"] == (i if kind == orc.KIND_A else j) * K + int(s["k"][0])
        seen_status.add(int(r["status"]))
        # (2) where the unchecked faulty value can be had (no product-level check in the way): the output check
        # restated on it, element by element
        if kind != orc.KIND_TERM or (mode & 3) == 0:
            Craw, *_ = orc.gemm(dt, w.A, w.Bt, s, mode & ~3)
            b_det, b_h, b_first, b_maxdev, b_changed = brute_record_stats(
                [Craw.reshape(-1)[l] for l in lins], [Cclean.reshape(-1)[l] for l in lins], lins, mode)
            assert (b_det, b_h, b_first, b_changed) == (n_det, h, first, status & 1)
            assert b_maxdev == maxdev or (np.isinf(maxdev) and np.isinf(b_maxdev))
        # untouched elements keep their clean value
        mask = np.ones(M * N, dtype=bool); mask[lins] = False
        assert np.array_equal(Cf.reshape(-1)[mask].view(np.uint32), Cclean.reshape(-1)[mask].view(np.uint32))
    if mix == "term" and (mode & 3):
        # the cases this pin is here for did occur: a trial that ends unflagged and changed, and (under BoundCheck
        # without correction of the product... or with it) both flagged and unflagged trials
        assert 1 in seen_status or 0 in seen_status
    if mix == "term" and mode == (orc.T_BOUND | orc.CORRECT):
        # product flagged and corrected, sum below the threshold afterwards: status "changed" only
        logs = [orc.gemm(dt, w.A, w.Bt, w.sites[t:t + 1], mode)[2][0] for t in range(len(w.sites))]
        assert any(l["status"] & 4 for l in logs) and any(not (l["status"] & 4) for l in logs)


def test_term_trial_product_correction_then_output_check():
    """A TERM trial under BoundCheck + correction, by hand: the product's exponent is corrected first (three bits
    cleared), the corrected product enters the sum by Eq. 1-2, and only then the output check looks at the sum."""
    K = 8
    a = np.zeros((1, K), dtype=np.float32); b = np.zeros((1, K), dtype=np.float32)
    a[0, :] = 1.0; b[0, :] = [1, 2, 3, 4, 5, 6, 7, 8]
    A, Bt = synth.round_to_storage(a, orc.BF16), synth.round_to_storage(b, orc.BF16)
    Cclean, *_ = orc.gemm(orc.BF16, A, Bt)
    assert Cclean[0, 0] == 36.0
    # term k=3 (product 4.0 = 0x40800000): flipping bit 29 gives exponent 0xC1 -> 2^66: flagged; the correction clears
    # exponent bits 6..4: 0xC1 -> 0x81, i.e. 4.0 again: the sum returns to 36 exactly
    s = site(orc.KIND_TERM, 0, 0, 3, 1 << 29)
    r = orc.campaign(orc.BF16, A, Bt, Cclean, s, orc.T_BOUND | orc.CORRECT, kstep=4)[0]
    assert r["before_bits"] == 0x40800000 and r["after_bits"] == 0x60800000
    assert bits_f32(int(r["final_bits"])) == 36.0 and r["status"] == 0 and r["n_detected"] == 0 and r["max_abs_dev"] == 0.0
    # detection only: the huge product stays, the sum is 2^66 (32 is lost in it), the output check flags it
    r = orc.campaign(orc.BF16, A, Bt, Cclean, s, orc.T_BOUND, kstep=4)[0]
    want = np.float32(np.float32(np.float32(10.0 - 4.0) + np.float32(2.0 ** 66)) + np.float32(26.0))
    assert bits_f32(int(r["final_bits"])) == float(want) and r["status"] == 3 and r["n_detected"] == 1
    assert r["first_detected"] == 0 and int(r["idx_hash"]) == HASH_MUL
    # correction on, but a flip the product check cannot see (bit 27: 4.0 -> 4 * 2^16 = 262144 has exponent 0x91...):
    # exponent 0x81 ^ 0x10 = 0x91 is flagged too; use bit 26 instead: 0x81 ^ 0x08 = 0x89 -> 4 * 2^8 = 1024, not flagged
    s = site(orc.KIND_TERM, 0, 0, 3, 1 << 26)
    r = orc.campaign(orc.BF16, A, Bt, Cclean, s, orc.T_BOUND | orc.CORRECT, kstep=4)[0]
    assert bits_f32(int(r["final_bits"])) == 36.0 - 4.0 + 1024.0 and r["status"] == 1 and r["max_abs_dev"] == 1020.0


@pytest.mark.parametrize("dtype", [orc.FP16, orc.BF16, orc.TF32])
def test_sampled_outputs_with_operand_sites_equal_the_full_recompute(dtype):
    """orc.sample with an A / B site table: bit-equal to the same elements of orc.gemm with those sites, including two
    sites that compose on one operand word and sites that miss the sampled rows and columns."""
    M, N, K = 9, 11, 50
    rng = np.random.default_rng(41)
    A = synth.round_to_storage(rng.standard_normal((M, K)).astype(np.float32), dtype)
    Bt = synth.round_to_storage(rng.standard_normal((N, K)).astype(np.float32), dtype)
    top = 18 if dtype == orc.TF32 else 15
    sites = np.concatenate([
        site(orc.KIND_A, row=2, k=7, mask=1 << (top - 1)),       # exponent MSB of A[2,7]
        site(orc.KIND_B, col=5, k=49, mask=1 << top),            # sign of B[49,5]
        site(orc.KIND_A, row=2, k=7, mask=0b101),                # composes with the first on the same word
        site(orc.KIND_B, col=0, k=0, mask=1 << 3),
        site(orc.KIND_A, row=8, k=49, mask=3 << 4),
    ])
    Cf, hdr, log, _ = orc.gemm(dtype, A, Bt, sites)
    C0, *_ = orc.gemm(dtype, A, Bt)
    assert hdr[3] == 5 and log["before_bits"][2] == log["after_bits"][0]
    si, sj = np.meshgrid(np.arange(M, dtype=np.uint32), np.arange(N, dtype=np.uint32), indexing="ij")
    sc, sap = orc.sample(dtype, A, Bt, si.reshape(-1), sj.reshape(-1), sites)
    assert np.array_equal(sc.view(np.uint32).reshape(M, N), Cf.view(np.uint32))
    # the sites did something, and only where they should
    moved = Cf.view(np.uint32) != C0.view(np.uint32)
    assert moved[2].all() and moved[:, 5].sum() >= M - 1 and moved[8].any() and moved[:, 0].any()
    quiet = np.ones((M, N), dtype=bool); quiet[[2, 8], :] = False; quiet[:, [0, 5]] = False
    assert not moved[quiet].any()
    # the magnitude sum uses the operands actually multiplied
    A2, B2 = A.copy(), Bt.copy()
    for t in sites:
        if t["kind"] == orc.KIND_A:
            A2[t["row"], t["k"]] = orc.flip_operand(dtype, int(A2[t["row"], t["k"]]), int(t["xor_mask"]))
        else:
            B2[t["col"], t["k"]] = orc.flip_operand(dtype, int(B2[t["col"], t["k"]]), int(t["xor_mask"]))
    assert np.allclose(sap.reshape(M, N), orc.absprod(dtype, A2, B2), rtol=1e-12)


@pytest.mark.parametrize("name", ["c1", "c2", "c3a", "c3b", "c4", "c5"])
def test_clean_workloads_raise_no_flags(name):
    """The workloads' clean outputs are far below the BoundCheck threshold: a fault-free run flags nothing."""
    w = synth.make_workload(name, 32, 48, min(synth.CONFIGS[name]["K"], 512), trials=1)
    Cm, hdr, _, bm = orc.gemm(w.dtype, w.A, w.Bt, None, orc.T_BOUND | orc.CORRECT)
    assert hdr[1] == 0 and not bm.any() and np.all(np.abs(Cm) < 131072.0)


def test_site_generators_follow_the_recipes():
    for name, cfg in synth.CONFIGS.items():
        M, N, K = 64, 96, 256
        s = synth.make_sites(cfg["mix"], cfg["dtype"], M, N, K, 2000, 1)
        kt = synth.kstep(cfg["dtype"])
        assert np.all(s["row"] < M) and np.all(s["col"] < N)
        acc = s["kind"] == synth.KIND_ACC
        assert np.all(s["k"][acc] % kt == 0) and np.all(s["k"][acc] >= kt) and np.all(s["k"][acc] <= K)
        op = (s["kind"] == synth.KIND_A) | (s["kind"] == synth.KIND_B)
        width = 19 if cfg["dtype"] == synth.DTYPE_TF32 else 16
        assert np.all(s["xor_mask"][op] < (1 << width)) and np.all(s["k"][op] < K)
        pop = np.array([bin(int(m)).count("1") for m in s["xor_mask"]])
        assert np.all(pop == (2 if cfg["mix"] == "acc2" else 1))
        if cfg["mix"] == "mixed":
            assert op.sum() > 500 and acc.sum() > 500 and (s["kind"] == synth.KIND_OUT).sum() > 500
    a, bt = synth.make_operands("c5", 64, 8, 32)
    assert (a.view(np.float16) >= 0).all() and (a == 0).mean() > 0.3          # ReLU: about half zeros
    a, _ = synth.make_operands("c4", 64, 8, 32)
    assert a.dtype == np.uint32 and not (a & 0x1FFF).any()


def test_summary_bruteforce_and_bin_edges():
    """Deviation summary: counts and exponent bins against a Python loop; bin e covers [2^(e-127), 2^(e-126))."""
    import math
    w = synth.make_workload("c5", 48, 40, 128, trials=300)
    Cc, *_ = orc.gemm(w.dtype, w.A, w.Bt)
    sites = w.sites.copy()
    sites["row"][7] = 10 ** 6                                   # one invalid site
    rec = orc.campaign(w.dtype, w.A, w.Bt, Cc, sites, w.detect_mode)
    out = orc.summary(rec)
    want = np.zeros(272, dtype=np.uint32)
    want[0] = len(rec)
    for r in rec:
        if r["status"] & 0x100:
            want[1] += 1; continue
        zero = not (r["status"] & 1)
        want[2] += zero; want[3] += bool(r["status"] & 2); want[4] += bool(r["status"] & 4)
        want[6 + r["kind"]] += 1; want[11 + r["kind"]] += zero
        d = float(r["max_abs_dev"])
        if math.isinf(d) or math.isnan(d):
            want[5] += 1; want[16 + 255] += 1
        elif d > 0:
            e = math.floor(math.log2(d)) + 127 if d >= 2.0 ** -126 else 0
            want[16 + e] += 1
    assert np.array_equal(out, want)
    assert want[1] == 1 and want[2] > 0 and want[16:].sum() > 100
    assert out[6:11].sum() == out[0] - out[1] and out[2] == out[11:16].sum()
    # hand-made records pin the bin edges
    r = np.zeros(6, dtype=orc.RECORD)
    r["status"] = 1
    r["max_abs_dev"] = [1.0, 1.9999999, 2.0, 2.0 ** -126, 2.0 ** -127, np.inf]
    h = orc.summary(r)[16:]
    assert h[127] == 2 and h[128] == 1 and h[1] == 1 and h[0] == 1 and h[255] == 1 and h.sum() == 6


# ---------------------------------------------------------------- D = A x B + C (Section II-B)

@pytest.mark.parametrize("dtype", [orc.FP16, orc.BF16, orc.TF32])
def test_addend_exact_integers_and_zero_operand(dtype):
    """Small integers: D = A x B + C exactly (a sign slip or a dropped addend shows); A = 0 gives D = C word for word."""
    M, N, K = 5, 7, 11
    a, b, A, Bt = int_operands(dtype, M, N, K, 21)
    rng = np.random.default_rng(22)
    cin = rng.integers(-100, 101, size=(M, N)).astype(np.float32)
    D, hdr, _, bm = orc.gemm(dtype, A, Bt, addend=cin)
    assert np.array_equal(D.astype(np.int64), a.astype(np.int64) @ b.astype(np.int64).T + cin.astype(np.int64))
    assert hdr[1] == 0 and not bm.any()
    cin = rng.standard_normal((M, N)).astype(np.float32)
    D, *_ = orc.gemm(dtype, np.zeros_like(A), Bt, addend=cin)
    assert np.array_equal(D.view(np.uint32), cin.view(np.uint32))


@pytest.mark.parametrize("dtype", [orc.FP16, orc.BF16, orc.TF32])
def test_addend_continues_an_accumulation(dtype):
    """A GEMM cut in two along k, the second half taking the first half's output as its addend, is the uncut
    GEMM bit for bit (one running sum in k order), and differs from summing the two halves separately."""
    M, N, K, K1 = 6, 9, 96, 40
    rng = np.random.default_rng(23)
    A = synth.round_to_storage(rng.standard_normal((M, K)).astype(np.float32), dtype)
    Bt = synth.round_to_storage(rng.standard_normal((N, K)).astype(np.float32), dtype)
    whole, *_ = orc.gemm(dtype, A, Bt)
    first, *_ = orc.gemm(dtype, np.ascontiguousarray(A[:, :K1]), np.ascontiguousarray(Bt[:, :K1]))
    second, *_ = orc.gemm(dtype, np.ascontiguousarray(A[:, K1:]), np.ascontiguousarray(Bt[:, K1:]), addend=first)
    assert np.array_equal(second.view(np.uint32), whole.view(np.uint32))
    alone, *_ = orc.gemm(dtype, np.ascontiguousarray(A[:, K1:]), np.ascontiguousarray(Bt[:, K1:]))
    assert not np.array_equal((first + alone).view(np.uint32), whole.view(np.uint32))


def test_addend_scalar_loop_and_sites():
    """Per-element Python loop in float32 starting from c_ij; an ACC site meets addend + partial sum, a TERM
    site's write-back and an OUT site act on sums that include the addend."""
    dtype, M, N, K = orc.BF16, 4, 5, 130
    rng = np.random.default_rng(24)
    A = synth.round_to_storage(rng.standard_normal((M, K)).astype(np.float32), dtype)
    Bt = synth.round_to_storage(rng.standard_normal((N, K)).astype(np.float32), dtype)
    cin = (rng.standard_normal((M, N)) * 3).astype(np.float32)
    af = (A.astype(np.uint32) << 16).view(np.float32)
    bf = (Bt.astype(np.uint32) << 16).view(np.float32)

    def chain(i, j, upto):
        acc = np.float32(cin[i, j])
        for k in range(upto):
            acc = np.float32(acc + np.float32(af[i, k] * bf[j, k]))
        return acc

    D, *_ = orc.gemm(dtype, A, Bt, addend=cin)
    for i in range(M):
        for j in range(N):
            assert f32_bits(D[i, j]) == f32_bits(chain(i, j, K))
    # sampled evaluation with a starting value per sample: the same chains, and |addend| joins the magnitude sum
    si = np.array([0, 3, 2], dtype=np.uint32); sj = np.array([4, 0, 2], dtype=np.uint32)
    sc, sap = orc.sample(dtype, A, Bt, si, sj, start=cin[si, sj])
    assert [f32_bits(v) for v in sc] == [f32_bits(chain(int(i), int(j), K)) for i, j in zip(si, sj)]
    ap = np.abs(af).astype(np.float64) @ np.abs(bf).astype(np.float64).T
    assert np.allclose(sap, ap[si, sj] + np.abs(cin[si, sj]).astype(np.float64), rtol=1e-12)
    # ACC site at boundary 64 of element (1, 2): the word flipped is addend + 64 products
    sites = np.concatenate([site(orc.KIND_ACC, 1, 2, 64, 1 << 20), site(orc.KIND_OUT, 3, 4, 0, 1 << 31),
                            site(orc.KIND_TERM, 2, 0, 70, 1 << 22)])
    D2, hdr, log, _ = orc.gemm(dtype, A, Bt, sites, addend=cin)
    assert log[0]["before_bits"] == f32_bits(chain(1, 2, 64)) and log[0]["after_bits"] == log[0]["before_bits"] ^ (1 << 20)
    acc = np.float32(bits_f32(int(log[0]["after_bits"])))
    for k in range(64, K):
        acc = np.float32(acc + np.float32(af[1, k] * bf[2, k]))
    assert f32_bits(D2[1, 2]) == f32_bits(acc)
    assert f32_bits(D2[3, 4]) == f32_bits(D[3, 4]) ^ (1 << 31)
    # TERM site on term 70: written back at boundary 128 into addend + 128 products (Eq. 1-2)
    p = np.float32(af[2, 70] * bf[0, 70])
    pe = np.float32(bits_f32(f32_bits(p) ^ (1 << 22)))
    acc = np.float32(np.float32(chain(2, 0, 128) - p) + pe)
    for k in range(128, K):
        acc = np.float32(acc + np.float32(af[2, k] * bf[0, k]))
    assert f32_bits(D2[2, 0]) == f32_bits(acc)
    untouched = np.ones((M, N), dtype=bool)
    untouched[1, 2] = untouched[3, 4] = untouched[2, 0] = False
    assert np.array_equal(D2[untouched].view(np.uint32), D[untouched].view(np.uint32)) and hdr[3] == 3


# ---------------------------------------------------------------- operand trials in the write-back form (Eq. 1-2)

@pytest.mark.parametrize("dtype", [orc.FP16, orc.BF16, orc.TF32])
def test_operand_writeback_is_exact_on_integers(dtype):
    """With small integers nothing rounds: Eq. 1-2 on the finished sum gives the recomputed row / column exactly,
    c' - c = (x' - x) * y, and the two forms of an operand trial give identical records. A swapped sign in Eq. 1,
    a wrong factor y (row/column mix-up) or the clean operand used twice all fail here."""
    M, N, K = 6, 7, 9
    a, b, A, Bt = int_operands(dtype, M, N, K, 31, lo=1, hi=5)
    Cclean, *_ = orc.gemm(dtype, A, Bt)
    sign = 18 if dtype == orc.TF32 else 15
    exp_lsb = {orc.FP16: 10, orc.BF16: 7, orc.TF32: 10}[dtype]
    sites = np.concatenate([site(orc.KIND_A, row=2, k=5, mask=1 << sign), site(orc.KIND_A, row=5, k=0, mask=1 << exp_lsb),
                            site(orc.KIND_B, col=3, k=8, mask=1 << sign), site(orc.KIND_B, col=6, k=2, mask=1 << exp_lsb)])
    for s in sites:
        isA = s["kind"] == orc.KIND_A
        v0 = orc.operand_trial_values(dtype, A, Bt, Cclean, s, form=0)
        v1 = orc.operand_trial_values(dtype, A, Bt, Cclean, s, form=1)
        assert np.array_equal(v0.view(np.uint32), v1.view(np.uint32)) and len(v1) == (N if isA else M)
        x = a[s["row"], s["k"]] if isA else b[s["col"], s["k"]]
        word = int(A[s["row"], s["k"]]) if isA else int(Bt[s["col"], s["k"]])
        xf = orc.widen(dtype, orc.flip_operand(dtype, word, int(s["xor_mask"])))
        y = b[:, s["k"]] if isA else a[:, s["k"]]
        c = Cclean[s["row"], :] if isA else Cclean[:, s["col"]]
        assert np.array_equal(v1.astype(np.float64) - c.astype(np.float64), (xf - float(x)) * y.astype(np.float64))
        Cf, *_ = orc.gemm(dtype, A, Bt, s.reshape(1))
        assert np.array_equal(v1, Cf[s["row"], :] if isA else Cf[:, s["col"]])
    for mode in (orc.T_NONE, orc.T_BOUND | orc.CORRECT):
        r0 = orc.campaign(dtype, A, Bt, Cclean, sites, mode, operand_form=0)
        r1 = orc.campaign(dtype, A, Bt, Cclean, sites, mode, operand_form=1)
        assert np.array_equal(r0.view(np.uint8), r1.view(np.uint8))
        assert (r1["status"] & 1).all() and (r1["n_affected"] == [N, N, M, M]).all()


@pytest.mark.parametrize("dtype", [orc.FP16, orc.BF16, orc.TF32])
def test_operand_writeback_on_rounded_data(dtype):
    """Away from exact data the write-back form is the finished sum with two more roundings: within
    2^-23 (|c| + |x y| + |x' y|) of (c - x y + x' y) taken exactly, and the order is Eq. 1 then Eq. 2."""
    from fractions import Fraction
    M, N, K = 7, 6, 40
    rng = np.random.default_rng(32)
    A = synth.round_to_storage(rng.standard_normal((M, K)).astype(np.float32), dtype)
    Bt = synth.round_to_storage(rng.standard_normal((N, K)).astype(np.float32), dtype)
    Cclean, *_ = orc.gemm(dtype, A, Bt)
    width = 19 if dtype == orc.TF32 else 16
    order_matters = 0
    for t in range(24):
        isA = t % 2 == 0
        s = site(orc.KIND_A if isA else orc.KIND_B, row=int(rng.integers(0, M)), col=int(rng.integers(0, N)),
                 k=int(rng.integers(0, K)), mask=1 << int(rng.integers(0, width - 2)))[0]
        word = int(A[s["row"], s["k"]]) if isA else int(Bt[s["col"], s["k"]])
        x = Fraction(orc.widen(dtype, word)); xf = Fraction(orc.widen(dtype, orc.flip_operand(dtype, word, int(s["xor_mask"]))))
        v1 = orc.operand_trial_values(dtype, A, Bt, Cclean, s, form=1)
        v0 = orc.operand_trial_values(dtype, A, Bt, Cclean, s, form=0)
        ap = orc.absprod(dtype, A, Bt)
        for o in range(len(v1)):
            y = Fraction(orc.widen(dtype, int(Bt[o, s["k"]]) if isA else int(A[o, s["k"]])))
            c = Cclean[s["row"], o] if isA else Cclean[o, s["col"]]
            exact = Fraction(float(c)) - x * y + xf * y                # products of two operands are exact in FP32
            bound = Fraction(2) ** -23 * (abs(Fraction(float(c))) + abs(x * y) + abs(xf * y))
            assert abs(Fraction(float(v1[o])) - exact) <= bound
            # Eq. 1 then Eq. 2, each rounded once (a float32 difference or sum of two float32 numbers of similar size
            # is exact in double, so one conversion to float32 is the single rounding)
            rep = np.float32(float(Fraction(float(c)) - x * y))
            want = np.float32(float(Fraction(float(rep)) + xf * y))
            assert f32_bits(float(v1[o])) == f32_bits(float(want))
            other = np.float32(float(Fraction(float(np.float32(float(Fraction(float(c)) + xf * y)))) - x * y))
            order_matters += int(f32_bits(float(other)) != f32_bits(float(want)))
            # and the recompute is the same number up to the accumulated rounding of both chains
            i_, j_ = (s["row"], o) if isA else (o, s["col"])
            assert abs(float(v0[o]) - float(v1[o])) <= 2 * K * 2.0 ** -24 * (ap[i_, j_] + float(abs(xf * y)))
    assert order_matters > 0        # the data does tell the two orders apart


# ---------------------------------------------------------------- the product held in the operand format (alternative reading)

def test_round_to_operand_format():
    """TF32: ties to even on the 13 dropped bits, carries into the exponent, against the generators' rounding; FP16 and
    BF16 are the 16-bit output rounding (pinned in test_oracle_output16.py)."""
    for w, want in [(0x3F801000, 0x3F800000), (0x3F803000, 0x3F804000), (0x3F801001, 0x3F802000), (0x3F800FFF, 0x3F800000),
                    (0x3FFFF000, 0x40000000), (0x7F7FF000, 0x7F800000), (0x7F800000, 0x7F800000), (0x80001000, 0x80000000),
                    (0x00003000, 0x00004000)]:
        assert orc.round_to_operand(orc.TF32, w) == want, hex(w)
    assert orc.round_to_operand(orc.TF32, 0x7F800001) & 0x007FE000                     # NaN stays NaN
    rng = np.random.default_rng(81)
    w = rng.integers(0, 1 << 32, 100000, dtype=np.uint64).astype(np.uint32)
    w = w[((w >> 23) & 0xFF) != 0xFF]
    got = np.array([orc.round_to_operand(orc.TF32, int(x)) for x in w], dtype=np.uint32)
    assert np.array_equal(got, synth.round_to_storage(w.view(np.float32), orc.TF32))
    assert orc.round_to_operand(orc.FP16, f32_bits(1.0 + 2.0 ** -11)) == 0x3C00 and orc.round_to_operand(orc.BF16, 0x3F818000) == 0x3F82


def test_term_in_operand_format_paper_example_and_closed_forms():
    """Section V-B's example: a product that is zero, held in FP16, with its first mantissa bit flipped, is
    0.00003052 (the value the paper prints) and changes the sum; the same flip of a BF16 zero is far too small to
    survive the accumulation. Then closed forms on exact data."""
    K = 8
    a = np.array([[1, 2, 0, 3, 1, 1, 2, 1]], dtype=np.float32); b = np.array([[2, 1, 5, 1, 1, 3, 1, 2]], dtype=np.float32)
    import os
    rows = [l.split() for l in open(os.path.join(os.path.dirname(__file__), "golden", "fp16_subnormal_example.txt"))
            if l.strip() and l[0] != "#"]
    fp16_row = [r for r in rows if r[0] == "FP16"][0]
    assert int(fp16_row[1], 2) == 1 << 9                   # the pattern the paper prints: first mantissa bit only
    golden = float(fp16_row[2])                            # 0.00003052 as printed
    for dtype, first_mantissa_bit, survives in ((orc.FP16, 9, True), (orc.BF16, 6, False)):
        A, Bt = synth.round_to_storage(a, dtype), synth.round_to_storage(b, dtype)
        C0, *_ = orc.gemm(dtype, A, Bt)
        assert C0[0, 0] == 15.0
        s = site(orc.KIND_TERM, 0, 0, 2, 1 << first_mantissa_bit)                       # term 2 is 0 * 5 = 0
        r = orc.campaign(dtype, A, Bt, C0, s, orc.TERM_IN_FORMAT, kstep=4)[0]
        assert r["before_bits"] == 0 and r["after_bits"] == 1 << first_mantissa_bit
        flipped = orc.widen(dtype, 1 << first_mantissa_bit)
        if dtype == orc.FP16:
            assert abs(flipped - golden) < 5e-9 and flipped == 2.0 ** -15               # 0000001000000000 = 0.00003052
        else:
            assert flipped == 2.0 ** -127
        if survives:
            assert bits_f32(int(r["final_bits"])) == float(np.float32(np.float32(7.0 - 0.0 + 2.0 ** -15) + np.float32(8.0)))
            assert r["status"] & 1 and r["max_abs_dev"] > 0
        else:
            assert bits_f32(int(r["final_bits"])) == 15.0 and r["status"] == 0 and r["max_abs_dev"] == 0.0
        # under the FP32-product reading the same mask is a low mantissa bit of an FP32 zero: nothing survives
        r32 = orc.campaign(dtype, A, Bt, C0, s, 0, kstep=4)[0]
        assert r32["status"] == 0
    # closed forms, exact data: sign flip of the narrow product subtracts it twice; exponent LSB doubles or halves it
    for dtype in (orc.FP16, orc.BF16, orc.TF32):
        A, Bt = synth.round_to_storage(a, dtype), synth.round_to_storage(b, dtype)
        C0, *_ = orc.gemm(dtype, A, Bt)
        sign = 18 if dtype == orc.TF32 else 15
        exp_lsb = {orc.FP16: 10, orc.BF16: 7, orc.TF32: 10}[dtype]
        r = orc.campaign(dtype, A, Bt, C0, site(orc.KIND_TERM, 0, 0, 3, 1 << sign), orc.TERM_IN_FORMAT, kstep=4)[0]
        assert bits_f32(int(r["final_bits"])) == 15.0 - 2 * 3.0
        r = orc.campaign(dtype, A, Bt, C0, site(orc.KIND_TERM, 0, 0, 3, 1 << exp_lsb), orc.TERM_IN_FORMAT, kstep=4)[0]
        p_new = orc.widen(dtype, orc.flip_operand(dtype, orc.round_to_operand(dtype, f32_bits(3.0)), 1 << exp_lsb))
        assert p_new in (1.5, 6.0) and bits_f32(int(r["final_bits"])) == 15.0 - 3.0 + p_new
        # the product-level check sees the widened faulty product: top exponent bit of the format's word
        top = sign - 1
        # term 4 is 1 * 1 = 1.0: with the top exponent bit of the format's word set it is infinite in every format;
        # RangeCheck-max detects it (exponent 255 above the bound 127 + 127 - 126 = 128) and puts the bound in: 2.0
        mode = orc.T_RMAX | orc.CORRECT | orc.TERM_IN_FORMAT
        r = orc.campaign(dtype, A, Bt, C0, site(orc.KIND_TERM, 0, 0, 4, 1 << top), mode, kstep=4)[0]
        Cf, _, log, _ = orc.gemm(dtype, A, Bt, site(orc.KIND_TERM, 0, 0, 4, 1 << top), mode, kstep=4)
        assert r["final_bits"] == f32_bits(float(Cf[0, 0])) and log["status"][0] & 4
        assert np.isinf(orc.widen(dtype, int(log["after_bits"][0]))) and log["final_bits"][0] == f32_bits(2.0)
        assert float(Cf[0, 0]) == 15.0 - 1.0 + 2.0
    # mask 0 away from exact data: the narrow product is subtracted and added back, at most two roundings of the sum
    rng = np.random.default_rng(82)
    A = synth.round_to_storage(rng.standard_normal((1, 40)).astype(np.float32), orc.BF16)
    Bt = synth.round_to_storage(rng.standard_normal((1, 40)).astype(np.float32), orc.BF16)
    C0, *_ = orc.gemm(orc.BF16, A, Bt)
    r = orc.campaign(orc.BF16, A, Bt, C0, site(orc.KIND_TERM, 0, 0, 17, 0), orc.TERM_IN_FORMAT, kstep=8)[0]
    ap = orc.absprod(orc.BF16, A, Bt)[0, 0]
    assert abs(bits_f32(int(r["final_bits"])) - float(C0[0, 0])) <= 2 * 2.0 ** -23 * ap
