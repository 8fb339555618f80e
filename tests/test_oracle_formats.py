"""Pins for the oracle's format handling and bit-flip semantics (CPU only)."""
import os
import struct

import numpy as np
import pytest
import torch

import oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def f32_bits(x):
    return struct.unpack("<I", struct.pack("<f", x))[0]


def bits_f32(u):
    return struct.unpack("<f", struct.pack("<I", u & 0xFFFFFFFF))[0]


def test_table3_bf16_values():
    """Table III: every printed value is reproduced from (exponent, mantissa) to the printed digits."""
    rows = [l.split() for l in open(os.path.join(GOLDEN, "table3_bf16_bounds.txt")) if l.strip() and l[0] != "#"]
    assert len(rows) == 16
    for e, m, printed in rows:
        storage = (int(e, 2) << 7) | int(m, 2)
        v = orc.widen(orc.BF16, storage)
        assert float("%.6g" % v) == pytest.approx(float(printed), rel=1e-9), (e, m, v, printed)
        # the same pattern sits in the top 16 bits of an FP32 product word
        assert orc.widen_bits(orc.BF16, storage) == storage << 16


def test_fp16_and_bf16_subnormal_examples():
    """Section V-B: FP16 0000001000000000 prints as 0.00003052; the BF16 twin is 2^-127."""
    rows = [l.split() for l in open(os.path.join(GOLDEN, "fp16_subnormal_example.txt")) if l.strip() and l[0] != "#"]
    fp16 = [r for r in rows if r[0] == "FP16"][0]
    v = orc.widen(orc.FP16, int(fp16[1], 2))
    assert "%.8f" % v == fp16[2]
    assert v == 2.0 ** -15
    bf16 = [r for r in rows if r[0] == "BF16"][0]
    assert orc.widen(orc.BF16, int(bf16[1], 2)) == 2.0 ** -127
    # subnormal scales named in the text: 2^-14 (FP16) and 2^-126 (BF16/TF32), smallest steps
    assert orc.widen(orc.FP16, 1) == 2.0 ** -14 * 2.0 ** -10
    assert orc.widen(orc.BF16, 1) == 2.0 ** -126 * 2.0 ** -7
    assert orc.widen(orc.TF32, 1 << 13) == 2.0 ** -126 * 2.0 ** -10


def test_fp16_widen_exhaustive_against_numpy():
    """All 65536 FP16 patterns agree with numpy's half -> float conversion (an independent routine)."""
    pats = np.arange(65536, dtype=np.uint16)
    ref = pats.view(np.float16).astype(np.float32).view(np.uint32)
    for p in range(65536):
        got = orc.widen_bits(orc.FP16, p)
        r = int(ref[p])
        if (r & 0x7F800000) == 0x7F800000 and (r & 0x7FFFFF):
            # NaN: payload conventions may differ by the quiet bit only
            assert (got & 0x7F800000) == 0x7F800000 and (got & 0x7FFFFF)
        else:
            assert got == r, hex(p)


def test_bf16_widen_exhaustive_against_torch():
    pats = torch.arange(65536, dtype=torch.int32).to(torch.int16)
    ref = pats.view(torch.bfloat16).to(torch.float32).view(torch.int32).numpy().astype(np.uint32)
    for p in range(0, 65536, 1):
        r = int(ref[p])
        if (r & 0x7F800000) == 0x7F800000 and (r & 0x7FFFFF):
            continue
        assert orc.widen_bits(orc.BF16, p) == r


def test_tf32_widen_ignores_low_13_bits():
    for u in (0x3F800000, 0x3F801FFF, 0xC0490FDB, 0x00001FFF, 0x7F7FFFFF):
        assert orc.widen_bits(orc.TF32, u) == (u & 0xFFFFE000)


def test_operand_flip_bit_numbering():
    # 16-bit formats: mask bit b is storage bit b; bits above 15 are ignored
    assert orc.flip_operand(orc.BF16, 0x3F80, 1 << 15) == 0xBF80
    assert orc.flip_operand(orc.FP16, 0x3C00, 0x10001) == 0x3C01
    # TF32: mask bit b (0..18) is FP32 bit b + 13; bit 18 is the sign
    assert orc.flip_operand(orc.TF32, 0x3F800000, 1 << 18) == 0xBF800000
    assert orc.flip_operand(orc.TF32, 0x3F800000, 1) == 0x3F802000
    assert orc.flip_operand(orc.TF32, 0x3F800000, 1 << 19) == 0x3F800000


@pytest.mark.parametrize("dtype,one,sign_bit,exp_lsb,exp_bits,bias", [
    (orc.FP16, 0x3C00, 15, 10, 5, 15),
    (orc.BF16, 0x3F80, 15, 7, 8, 127),
    (orc.TF32, 0x3F800000, 18, 10, 8, 127),
])
def test_operand_flip_closed_forms(dtype, one, sign_bit, exp_lsb, exp_bits, bias):
    """Sign flip negates; flipping exponent bit b of 1.0 scales by 2^(+-2^b); a mantissa flip adds 2^(m - mant_bits)."""
    assert orc.widen(dtype, orc.flip_operand(dtype, one, 1 << sign_bit)) == -1.0
    E = bias  # exponent field of 1.0
    for b in range(exp_bits):
        v = orc.widen(dtype, orc.flip_operand(dtype, one, 1 << (exp_lsb + b)))
        newE = E ^ (1 << b)
        if newE == (1 << exp_bits) - 1:
            assert v == float("inf")
        elif newE == 0:
            assert v == 0.0       # mantissa of 1.0 is zero: the subnormal with fraction 0
        else:
            assert v == 2.0 ** ((1 << b) if newE > E else -(1 << b))
    for m in range(exp_lsb):
        v = orc.widen(dtype, orc.flip_operand(dtype, one, 1 << m))
        assert v == 1.0 + 2.0 ** (m - exp_lsb)
    # flipping twice restores the word
    w = orc.flip_operand(dtype, one, 0x55)
    assert orc.flip_operand(dtype, w, 0x55) == one


def test_round_to_storage_is_rne_and_roundtrips():
    """The generator's rounding: exhaustive round trip of every 16-bit pattern, hand-listed ties, torch cross-check."""
    from synth import round_to_storage, DTYPE_BF16, DTYPE_FP16, DTYPE_TF32
    pats = np.arange(65536, dtype=np.uint32)
    wide = np.array([orc.widen_bits(orc.BF16, int(p)) for p in pats], dtype=np.uint32)
    finite = (wide & 0x7F800000) != 0x7F800000
    back = round_to_storage(wide.view(np.float32), DTYPE_BF16)
    assert np.array_equal(back[finite], pats[finite].astype(np.uint16))
    wide = np.array([orc.widen_bits(orc.FP16, int(p)) for p in pats], dtype=np.uint32)
    finite = (wide & 0x7F800000) != 0x7F800000
    back = round_to_storage(wide.view(np.float32), DTYPE_FP16)
    keep = finite & (pats != 0x8000)
    assert np.array_equal(back[keep], pats[keep].astype(np.uint16))
    # ties: 1 + 2^-8 is halfway between BF16 1.0 and 1+2^-7 -> even (1.0); 1 + 3*2^-8 -> 1 + 2^-6
    t = np.array([1 + 2.0 ** -8, 1 + 3 * 2.0 ** -8, 1 + 2.0 ** -8 + 2.0 ** -20], dtype=np.float32)
    assert list(round_to_storage(t, DTYPE_BF16)) == [0x3F80, 0x3F82, 0x3F81]
    # TF32 ties: 1 + 2^-11 halfway between 1 and 1 + 2^-10 -> even
    t = np.array([1 + 2.0 ** -11, 1 + 3 * 2.0 ** -11, 1 + 2.0 ** -11 + 2.0 ** -22], dtype=np.float32)
    assert list(round_to_storage(t, DTYPE_TF32)) == [0x3F800000, 0x3F804000, 0x3F802000]
    # torch's bfloat16 cast rounds the same way
    x = np.random.default_rng(0).standard_normal(100000).astype(np.float32)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(round_to_storage(x, DTYPE_BF16), ref)


def test_f32_flip_closed_forms_on_output_sites():
    """OUT sites on a 1x1 GEMM: sign flip negates, exponent bit b scales by 2^(+-2^b), mantissa bit m adds 2^(e-23+m)."""
    # A = [3.0], B = [0.5]  ->  C = 1.5 (E = 127, mantissa 0x400000)
    A = np.array([[0x4040]], dtype=np.uint16)      # bf16 3.0
    Bt = np.array([[0x3F00]], dtype=np.uint16)     # bf16 0.5
    def run(mask):
        s = np.zeros(1, dtype=orc.SITE)
        s["kind"] = orc.KIND_OUT; s["xor_mask"] = mask
        Cm, _, log, _ = orc.gemm(orc.BF16, A, Bt, s, 0)
        assert log["before_bits"][0] == f32_bits(1.5) and log["after_bits"][0] == f32_bits(1.5) ^ mask
        return float(Cm[0, 0])
    assert run(0) == 1.5
    assert run(1 << 31) == -1.5
    for b in range(8):
        v = run(1 << (23 + b))
        if b == 7:
            assert np.isnan(v)          # E = 255 with non-zero mantissa
        elif (127 >> b) & 1:
            assert v == 1.5 * 2.0 ** -(1 << b)
        else:
            assert v == 1.5 * 2.0 ** (1 << b)
    for m in range(23):
        v = run(1 << m)
        delta = 2.0 ** (0 - 23 + m)
        assert v == (1.5 - delta if m == 22 else 1.5 + delta)
