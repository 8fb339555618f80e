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


@pytest.mark.parametrize("name,mix", [("c1", "out"), ("c2", "operand"), ("c4", "acc2"), ("c5", "mixed"), ("c2", "term")])
def test_incremental_trials_equal_full_recompute(name, mix):
    """Every trial record equals what a full fault-injected GEMM with that single site gives."""
    cfg = synth.CONFIGS[name]
    M, N, K = 24, 40, 96
    w = synth.make_workload(name, M, N, K, trials=40, mix=mix)
    dt, mode = w.dtype, w.detect_mode
    Cclean, *_ = orc.gemm(dt, w.A, w.Bt)
    rec = orc.campaign(dt, w.A, w.Bt, Cclean, w.sites, mode)
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
        # raw faulty values: rerun without the check
        Craw, _, lograw, _ = orc.gemm(dt, w.A, w.Bt, s, mode & ~3 if kind != orc.KIND_TERM else mode)
        if kind == orc.KIND_TERM and (mode & 3) == 1:
            # the product-level check is part of the trial; the output check is applied by brute_record_stats
            Craw = Cf.copy()
            if mode & orc.CORRECT:
                pytest.skip("corrected outputs hide the raw value; covered by the other mixes")
        n_det, h, first, maxdev, changed = brute_record_stats(
            [Craw.reshape(-1)[l] for l in lins], [Cclean.reshape(-1)[l] for l in lins], lins, mode)
        r = rec[t]
        assert r["kind"] == kind and r["n_affected"] == len(lins)
        assert r["n_detected"] == n_det == hdr[1]
        assert int(r["idx_hash"]) == h and r["first_detected"] == first
        assert (r["status"] & 1) == changed
        assert float(r["max_abs_dev"]) == maxdev or (np.isinf(maxdev) and np.isinf(r["max_abs_dev"]))
        assert r["before_bits"] == log["before_bits"][0] and r["after_bits"] == log["after_bits"][0]
        if kind in (orc.KIND_OUT, orc.KIND_ACC, orc.KIND_TERM):
            assert r["final_bits"] == f32_bits(float(Cf[i, j])) and r["primary_index"] == i * N + j
        # untouched elements keep their clean value
        mask = np.ones(M * N, dtype=bool); mask[lins] = False
        assert np.array_equal(Cf.reshape(-1)[mask].view(np.uint32), Cclean.reshape(-1)[mask].view(np.uint32))


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
