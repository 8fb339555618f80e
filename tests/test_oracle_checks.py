"""Pins for BoundCheck, RangeCheck-max and RangeCheck-flip (Section VI-A, VI-C, Table III)."""
import struct

import numpy as np

import oracle as orc


def f32_bits(x):
    return struct.unpack("<I", struct.pack("<f", x))[0]


def bits_f32(u):
    return struct.unpack("<f", struct.pack("<I", u & 0xFFFFFFFF))[0]


def test_boundcheck_threshold_rows_of_table3():
    """Table III rows: 10001000 (512..1020) passes, 10010000 (131072) and above are flagged."""
    for v in (2.0, 3.98438, 4.0, 63.75, 512.0, 1020.0, 65536.0, 131071.99):
        assert orc.boundcheck_detect(f32_bits(v)) == 0
    for v in (131072.0, 261120.0, 8.58993e9, 3.68935e19, 7.34987e19, 3.0e38, float("inf")):
        assert orc.boundcheck_detect(f32_bits(v)) == 1
        assert orc.boundcheck_detect(f32_bits(-v)) == 1
    # small magnitudes (MSB of the exponent clear) are never flagged, whatever the other bits
    for v in (0.0, 1e-30, 0.5, 1.0, 1.9999999):
        assert orc.boundcheck_detect(f32_bits(v)) == 0


def test_boundcheck_exhaustive_against_hardware_form():
    """Section VI-C: three inversions of the exponent MSB and an AND, i.e. eee_new = eee & ~MSB,
    must equal "detect, then clear the eee bits" on all 256 exponents."""
    for E in range(256):
        for sign in (0, 1):
            for mant in (0, 0x7FFFFF, 0x2AAAAA):
                bits = (sign << 31) | (E << 23) | mant
                msb = (E >> 7) & 1
                eee = (E >> 4) & 7
                eee_new = eee & (0 if msb else 7)           # eee AND (NOT msb) per bit
                hw = (sign << 31) | ((msb << 7 | eee_new << 4 | (E & 0xF)) << 23) | mant
                assert orc.boundcheck_correct(bits) == hw
                assert orc.boundcheck_detect(bits) == int(msb == 1 and eee != 0)
                # template 1eeexxxx -> 1000xxxx; corrected values land in [2, 32*2) * ... < 131072
                if orc.boundcheck_detect(bits):
                    c = orc.boundcheck_correct(bits)
                    assert (c >> 23) & 0xFF == 0x80 | (E & 0xF)
                    assert 2.0 <= abs(bits_f32(c)) < 131072.0
                    assert orc.boundcheck_detect(c) == 0


def test_rangecheck_never_flags_a_clean_product():
    """m1*m2 < 4  =>  e_m <= e1+e2+1: exhaustive over all exponent pairs with extreme mantissas,
    products formed by real FP32 multiplication (numpy), subnormals and zeros included."""
    mants = np.array([0, 1, 0x400000, 0x7FFFFF], dtype=np.uint32)
    E = np.arange(255, dtype=np.uint32)                       # finite operands
    a = (E[:, None] << 23 | mants[None, :]).reshape(-1)       # 1020 operand words
    af = a.view(np.float32)
    with np.errstate(over="ignore", under="ignore"):
        p = (af[:, None] * af[None, :]).astype(np.float32)
    pb = p.view(np.uint32)
    bound = np.clip((a[:, None] >> 23).astype(np.int64) + (a[None, :] >> 23).astype(np.int64) - 126, 0, 255)
    Em = (pb >> 23) & 0xFF
    assert np.all(Em <= bound)
    # and the oracle's own functions agree on a strided subset
    for i in range(0, len(a), 37):
        for j in range(0, len(a), 41):
            b = orc.rangecheck_bound(int(a[i]), int(a[j]))
            assert b == bound[i, j]
            assert orc.rangecheck_detect(int(pb[i, j]), b) == 0
    # tightness: 1.5 * 1.5 = 2.25 reaches e1+e2+1
    assert (f32_bits(1.5 * 1.5) >> 23) & 0xFF == orc.rangecheck_bound(f32_bits(1.5), f32_bits(1.5))


def test_rangecheck_max_is_min_of_exponents():
    """Section VI-C: an 8-bit add and a compare choosing the smaller exponent."""
    for E in range(256):
        for bound in range(256):
            bits = (1 << 31) | (E << 23) | 0x123456
            got = orc.rangecheck_max(bits, bound)
            assert (got >> 23) & 0xFF == min(E, bound)
            assert got & 0x807FFFFF == bits & 0x807FFFFF
            assert orc.rangecheck_detect(bits, bound) == int(E > bound)


def test_rangecheck_flip_worked_example_and_properties():
    # bound 130, faulty exponent 194 = 11000010: clear bit 1 -> 192, clear bit 6 -> 128 <= 130, stop
    bits = (194 << 23) | 0x555555
    got = orc.rangecheck_flip(bits, 130)
    assert (got >> 23) & 0xFF == 128
    assert got & 0x807FFFFF == bits & 0x807FFFFF
    # bound 200, exponent 201 = 11001001: clearing bit 0 is enough
    assert (orc.rangecheck_flip(201 << 23, 200) >> 23) & 0xFF == 200
    for E in range(256):
        for bound in range(0, 256, 3):
            out = (orc.rangecheck_flip(E << 23, bound) >> 23) & 0xFF
            if E <= bound:
                assert out == E
            else:
                assert out <= bound and (out & ~E) == 0           # only 1s were cleared
                # minimality: the bit cleared last was needed, so restoring it exceeds the bound
                cleared = E & ~out
                top = 1 << (cleared.bit_length() - 1)
                assert (out | top) > bound
                # bits above the last cleared one are untouched, all set bits below it are cleared
                assert out >> top.bit_length() == E >> top.bit_length()


def test_term_site_uses_the_selected_technique():
    """A TERM site's faulty product goes through the chosen check before Eq. 1-2 (Section VI-B)."""
    # K = 1: C = a*b. a = 1.5, b = 1.5 -> p = 2.25 (E = 128); flip exponent bit 5 -> E = 160
    A = np.array([[0x3FC0]], dtype=np.uint16)
    Bt = np.array([[0x3FC0]], dtype=np.uint16)
    s = np.zeros(1, dtype=orc.SITE)
    s["kind"] = orc.KIND_TERM; s["xor_mask"] = 1 << 28
    p = f32_bits(2.25)
    for mode, want in [
        (orc.T_NONE, p ^ (1 << 28)),
        (orc.T_BOUND, p ^ (1 << 28)),                                   # detect only: value unchanged
        (orc.T_BOUND | orc.CORRECT, p),                                 # eee cleared -> E = 128 again
        (orc.T_RMAX | orc.CORRECT, p),                                  # bound = 127+127-126 = 128
        (orc.T_RFLIP | orc.CORRECT, p),                                 # 10100000 -> clear bit 5 -> 128
        (orc.T_RMAX, p ^ (1 << 28)),
    ]:
        Cm, hdr, log, bm = orc.gemm(orc.BF16, A, Bt, s, mode)
        assert log["before_bits"][0] == p and log["after_bits"][0] == p ^ (1 << 28)
        assert log["final_bits"][0] == want, mode
        # (0 - p) + p' with exact arithmetic here: C equals the checked product (0 + p - p = 0, + p')
        assert f32_bits(float(Cm[0, 0])) == (orc.boundcheck_correct(want) if mode == (orc.T_BOUND | orc.CORRECT) else want)


def test_output_range_bound_has_no_false_positive_and_is_tight():
    """Extension of the product bound to a dot product: E(C_ij) <= EA_i + EB_j - 126 + ceil(log2 K).
    Never exceeded by a clean GEMM (adversarial: every operand at the top of its binade), reached exactly for
    K a power of two, and it flags what raises an exponent beyond it."""
    import synth
    rng = np.random.default_rng(61)
    mode = orc.T_RMAX | orc.OUTPUT_RANGE
    for K in (1, 2, 3, 4, 5, 8, 33, 64, 100, 128):
        # adversarial: all |a| = |b| = largest BF16 below 2.0, same signs: the sum is as large as it can get
        a = np.full((3, K), 1.9921875, dtype=np.float32); b = np.full((4, K), 1.9921875, dtype=np.float32)
        A, Bt = synth.round_to_storage(a, orc.BF16), synth.round_to_storage(b, orc.BF16)
        Cm, hdr, _, bm = orc.gemm(orc.BF16, A, Bt, None, mode)
        assert hdr[1] == 0 and not bm.any(), K
        EA, EB = orc.operand_exponents(orc.BF16, A), orc.operand_exponents(orc.BF16, Bt)
        assert (EA == 127).all() and (EB == 127).all()
        bound = orc.output_range_bound(127, 127, K)
        L = int(np.ceil(np.log2(K))) if K > 1 else 0
        assert bound == 128 + L
        E = (Cm.view(np.uint32) >> 23) & 0xFF
        assert (E <= bound).all()
        if K & (K - 1) == 0:
            assert (E == bound).all()                       # tight: K * 1.99^2 sits in the top binade allowed
        # random data, mixed magnitudes per row: still no flag
        a = (rng.standard_normal((6, K)) * np.exp2(rng.integers(-20, 20, (6, 1)))).astype(np.float32)
        b = (rng.standard_normal((5, K)) * np.exp2(rng.integers(-20, 20, (5, 1)))).astype(np.float32)
        for dt in (orc.FP16, orc.BF16, orc.TF32):
            aa = np.clip(a, -6e4, 6e4) if dt == orc.FP16 else a
            bb = np.clip(b, -6e4, 6e4) if dt == orc.FP16 else b
            A, Bt = synth.round_to_storage(aa, dt), synth.round_to_storage(bb, dt)
            _, hdr, _, bm = orc.gemm(dt, A, Bt, None, mode)
            assert hdr[1] == 0, (K, dt)
    # exponent maxima: zero rows give 0, Inf gives 255, the largest |value| decides otherwise
    X = synth.round_to_storage(np.array([[0, 0, 0], [0.5, -3.0, 1.0], [np.inf, 1, 1], [1e-3, 0, 0]], dtype=np.float32), orc.BF16)
    assert list(orc.operand_exponents(orc.BF16, X)) == [0, 128, 255, 117]
    # detection and the two corrections on an output site, and on an operand fault that the clean maxima expose
    a = rng.standard_normal((4, 16)).astype(np.float32); b = rng.standard_normal((5, 16)).astype(np.float32)
    A, Bt = synth.round_to_storage(a, orc.BF16), synth.round_to_storage(b, orc.BF16)
    s = np.zeros(2, dtype=orc.SITE)
    s["kind"] = [orc.KIND_OUT, orc.KIND_A]; s["row"] = [1, 3]; s["col"] = [2, 0]; s["k"] = [0, 5]
    C0, *_ = orc.gemm(orc.BF16, A, Bt)
    c_bits = int(C0[1, 2].view(np.uint32))
    up = 1 << 30 if not c_bits & (1 << 30) else 1 << 29          # a flip that raises the exponent by 64 or more
    assert not c_bits & up
    s["xor_mask"] = [up, 1 << 14]
    Cd, hdr, log, bm = orc.gemm(orc.BF16, A, Bt, s, orc.T_RMAX | orc.OUTPUT_RANGE)
    assert bm[1, 0] & (1 << 2) and hdr[1] >= 2 and hdr[2] == 0
    assert bin(int(bm[3, 0])).count("1") >= 4                       # the faulty operand lights up most of its row
    EA, EB = orc.operand_exponents(orc.BF16, A), orc.operand_exponents(orc.BF16, Bt)
    for tech in (orc.T_RMAX, orc.T_RFLIP):
        Cc, hdrc, _, bmc = orc.gemm(orc.BF16, A, Bt, s, tech | orc.CORRECT | orc.OUTPUT_RANGE)
        assert np.array_equal(bmc, bm) and hdrc[2] == hdrc[1]
        for i in range(4):
            for j in range(5):
                bound = orc.output_range_bound(EA[i], EB[j], 16)
                Ec = (int(Cc[i, j].view(np.uint32)) >> 23) & 0xFF
                assert Ec <= bound
                if not (bm[i, 0] >> j) & 1:
                    assert Cc[i, j].view(np.uint32) == Cd[i, j].view(np.uint32)
                else:
                    want = (orc.rangecheck_max if tech == orc.T_RMAX else orc.rangecheck_flip)(int(Cd[i, j].view(np.uint32)), bound)
                    assert int(Cc[i, j].view(np.uint32)) == want
    # without the flag the RangeCheck techniques leave outputs alone (they act on TERM products only)
    _, hdrn, _, bmn = orc.gemm(orc.BF16, A, Bt, s, orc.T_RMAX | orc.CORRECT)
    assert hdrn[1] == 0 and not bmn.any()
