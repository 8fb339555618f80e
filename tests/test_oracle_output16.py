"""Pins for the oracle's 16-bit output rounding (CPU only): library conversions, every tie, both ends of the range."""
import numpy as np
import pytest
import torch

import oracle as orc
import synth


def f32(u):
    return np.array(u, dtype=np.uint32).view(np.float32)


def round_all(fmt, words):
    return np.array([orc.round_output(fmt, int(w)) for w in words], dtype=np.uint32)


def test_fp16_values_round_to_themselves():
    """Every FP16 value, widened exactly by numpy, comes back as the same 16 bits (NaNs come back as NaNs)."""
    h = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    wide = h.view(np.float16).astype(np.float32).view(np.uint32)
    got = round_all(orc.OUT_FP16, wide)
    nan = np.isnan(h.view(np.float16))
    assert np.array_equal(got[~nan], h[~nan].astype(np.uint32))
    assert np.isnan(got[nan].astype(np.uint16).view(np.float16)).all()


def test_fp16_every_tie_goes_to_the_even_neighbour():
    """The midpoint of two neighbouring FP16 values (exact in FP32) rounds to the one with an even last bit; one FP32
    step to either side rounds to the nearer neighbour. Subnormals, the normal/subnormal seam and the step to infinity
    are all among the 31744 pairs."""
    h = np.arange(0, 0x7C00, dtype=np.uint32)                      # h and h+1: neighbours (0x7C00 = infinity)
    lo = h.astype(np.uint16).view(np.float16).astype(np.float64)
    hi = np.where(h + 1 < 0x7C00, (h + 1).astype(np.uint16).view(np.float16).astype(np.float64), 65536.0)
    mid = ((lo + hi) / 2).astype(np.float32)
    assert np.array_equal(mid.astype(np.float64), (lo + hi) / 2)    # the midpoints are FP32 numbers
    even = np.where(h % 2 == 0, h, h + 1)
    mw = mid.view(np.uint32)
    assert np.array_equal(round_all(orc.OUT_FP16, mw), even)
    assert np.array_equal(round_all(orc.OUT_FP16, mw + 1), h + 1)
    assert np.array_equal(round_all(orc.OUT_FP16, mw - 1), h)
    assert np.array_equal(round_all(orc.OUT_FP16, mw | 0x80000000), even | 0x8000)      # the sign rides along


def test_fp16_hand_listed_cases():
    cases = [
        (65504.0, 0x7BFF), (65519.996, 0x7BFF), (65520.0, 0x7C00), (1e9, 0x7C00), (-70000.0, 0xFC00),
        (2.0 ** -24, 0x0001), (2.0 ** -25, 0x0000), (2.0 ** -25 * 1.0000002, 0x0001), (1.5 * 2.0 ** -24, 0x0002),
        (2.0 ** -14, 0x0400), (2.0 ** -14 - 2.0 ** -25, 0x0400), (2.0 ** -14 - 2.0 ** -24, 0x03FF),
        (1.0, 0x3C00), (1.0 + 2.0 ** -11, 0x3C00), (1.0 + 3 * 2.0 ** -11, 0x3C02), (-0.0, 0x8000), (0.0, 0x0000),
        (np.inf, 0x7C00), (-np.inf, 0xFC00), (1e-30, 0x0000), (-1e-30, 0x8000),
    ]
    for v, want in cases:
        w = int(np.float32(v).view(np.uint32))
        assert orc.round_output(orc.OUT_FP16, w) == want, (v, hex(orc.round_output(orc.OUT_FP16, w)), hex(want))
    assert (orc.round_output(orc.OUT_FP16, 0x7FC00001) & 0x7FFF) > 0x7C00           # NaN stays NaN
    assert (orc.round_output(orc.OUT_BF16, 0xFF800001) & 0x7FFF) > 0x7F80


def test_fp16_against_numpy_on_random_words():
    rng = np.random.default_rng(61)
    w = rng.integers(0, 1 << 32, 300000, dtype=np.uint64).astype(np.uint32)
    # half of them near FP16's range, where the interesting cases live
    w[::2] = (w[::2] & np.uint32(0x807FFFFF)) | (rng.integers(127 - 27, 127 + 17, len(w[::2])).astype(np.uint32) << 23)
    v = w.view(np.float32)
    with np.errstate(over="ignore"):
        want = v.astype(np.float16).view(np.uint16).astype(np.uint32)
    got = round_all(orc.OUT_FP16, w)
    nan = np.isnan(v)
    assert np.array_equal(got[~nan], want[~nan])
    assert np.isnan(got[nan].astype(np.uint16).view(np.float16)).all()


def test_bf16_ties_ends_and_library_conversion():
    cases = [(0x3F800000, 0x3F80), (0x3F808000, 0x3F80), (0x3F808001, 0x3F81), (0x3F818000, 0x3F82), (0x3F817FFF, 0x3F81),
             (0x7F7FFFFF, 0x7F80), (0x7F7F7FFF, 0x7F7F), (0x7F7F8000, 0x7F80), (0x00008000, 0x0000), (0x00018000, 0x0002),
             (0x80008001, 0x8001), (0x7F800000, 0x7F80), (0xFF800000, 0xFF80), (0x007F8000, 0x0080)]
    for w, want in cases:
        assert orc.round_output(orc.OUT_BF16, w) == want, (hex(w), hex(orc.round_output(orc.OUT_BF16, w)))
    # every tie between neighbouring BF16 values of one binade and of the subnormals
    top = np.concatenate([np.arange(0x3F80, 0x4000), np.arange(0x0000, 0x0100)]).astype(np.uint32)
    mid = (top << 16) | 0x8000
    assert np.array_equal(round_all(orc.OUT_BF16, mid), np.where(top % 2 == 0, top, top + 1))
    rng = np.random.default_rng(62)
    w = rng.integers(0, 1 << 32, 300000, dtype=np.uint64).astype(np.uint32)
    v = torch.from_numpy(w.view(np.float32).copy())
    want = v.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16).astype(np.uint32)
    got = round_all(orc.OUT_BF16, w)
    nan = np.isnan(w.view(np.float32))
    assert np.array_equal(got[~nan], want[~nan])
    assert (got[nan] & 0x7FFF > 0x7F80).all()
    # a third formulation: the input generators' rounding
    assert np.array_equal(got[~nan], synth.round_to_storage(w.view(np.float32), orc.BF16).astype(np.uint32)[~nan])


@pytest.mark.parametrize("fmt", [orc.OUT_FP16, orc.OUT_BF16])
def test_gemm_with_16_bit_output_rounds_the_checked_fp32_result(fmt):
    """Sites, check, flags and counts are those of the FP32 GEMM; the stored element is its FP32 result rounded once.
    A value that overflows FP16 but stays under the BoundCheck threshold becomes infinity without a flag."""
    M, N, K = 5, 40, 16
    rng = np.random.default_rng(63)
    a = rng.standard_normal((M, K)).astype(np.float32); b = rng.standard_normal((N, K)).astype(np.float32)
    a[1, :] = 0; a[1, 0] = 280.0; b[7, 0] = 250.0          # C[1,7] = 70000: above FP16's range, below 131072
    a[3, :] = 0; a[3, 2] = 512.0; b[9, 2] = 256.0          # C[3,9] = 131072: flagged
    A, Bt = synth.round_to_storage(a, orc.BF16), synth.round_to_storage(b, orc.BF16)
    s = np.zeros(2, dtype=orc.SITE)
    s["kind"] = [orc.KIND_OUT, orc.KIND_ACC]; s["row"] = [0, 4]; s["col"] = [33, 2]; s["k"] = [0, 16]; s["xor_mask"] = [1 << 30, 1 << 22]
    for mode in (orc.T_BOUND, orc.T_BOUND | orc.CORRECT, orc.T_NONE):
        C32, hdr32, log32, bm32 = orc.gemm(orc.BF16, A, Bt, s, mode)
        D16, hdr, log, bm = orc.gemm_out16(orc.BF16, A, Bt, fmt, s, mode)
        assert np.array_equal(hdr, hdr32) and np.array_equal(bm, bm32) and np.array_equal(log.view(np.uint32), log32.view(np.uint32))
        want = np.array([[orc.round_output(fmt, int(x)) for x in row] for row in C32.view(np.uint32)], dtype=np.uint16)
        assert np.array_equal(D16, want)
        if mode & 3:
            assert (bm[1, 0] >> 7) & 1 == 0 and (bm[3, 0] >> 9) & 1 == 1
        if fmt == orc.OUT_FP16:
            assert D16[1, 7] == 0x7C00
            assert D16[3, 9] == (0x7C00 if not (mode & orc.CORRECT) else orc.round_output(fmt, orc.boundcheck_correct(0x48000000)))
    # with an addend the sum starts from it (Section II-B) and is rounded once at the end
    cin = rng.standard_normal((M, N)).astype(np.float32)
    C32, *_ = orc.gemm(orc.BF16, A, Bt, None, 0, addend=cin)
    D16, *_ = orc.gemm_out16(orc.BF16, A, Bt, fmt, None, 0, addend=cin)
    assert np.array_equal(D16, np.array([[orc.round_output(fmt, int(x)) for x in row] for row in C32.view(np.uint32)], dtype=np.uint16))
