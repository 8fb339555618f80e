"""GPU parity of mpgemmfi_gemm_out16 (FP32 result rounded once to FP16 / BF16) against the oracle.

Rules. Sites, flags, counts and the site log are decided on the FP32 values: they are compared exactly as for
mpgemmfi_gemm (parity.check_gemm_against_oracle does that on the FP32 entry point; here the 16-bit run must give
the very same flags buffer as the FP32 run on the device). The 16-bit values:
  * against the oracle's: two FP32 results within the tolerance of each other may round to neighbouring 16-bit
    values, so |d_gpu - d_oracle| <= tol_ij + one unit in the last place of the format at that magnitude;
  * the rounding step itself, in the precision in which the device took it: the oracle's rounding applied to the
    FP32 words of the device's own FP32 run (same kernel, same accumulation) gives the device's 16-bit words
    bit for bit (NaN payloads aside).
"""
import numpy as np
import pytest
import torch

import oracle as orc
import paper_2311_05782_b200 as mpg
import synth
from parity import TOL, close, faulted_operands, to_dev

pytestmark = pytest.mark.gpu

FMTS = [(mpg.OUT_FP16, orc.OUT_FP16, torch.float16, np.float16), (mpg.OUT_BF16, orc.OUT_BF16, torch.bfloat16, None)]


@pytest.fixture(params=["single", "pair"])
def tile_policy(request):
    assert mpg.mpgemmfi_set_tile_policy(mpg.TILES_PAIR if request.param == "pair" else mpg.TILES_SINGLE) == 0
    yield request.param
    mpg.mpgemmfi_set_tile_policy(mpg.TILES_AUTO)


def widen16(bits, gfmt):
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    if gfmt == mpg.OUT_FP16:
        return bits.view(np.float16).astype(np.float64)
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def ulp16(x, gfmt):
    """One unit in the last place of the 16-bit format at magnitude |x| (the subnormal spacing below the normal range)."""
    mant, emin = (10, -14) if gfmt == mpg.OUT_FP16 else (7, -126)
    with np.errstate(divide="ignore", invalid="ignore"):
        e = np.floor(np.log2(np.abs(x)))
    e = np.where(np.isfinite(e), np.maximum(e, emin), emin)
    return np.exp2(e - mant)


def as_u16(t):
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


def rand_operands(dtype, M, N, K, seed, scale=1.0):
    rng = np.random.default_rng(seed)
    a = (rng.standard_normal((M, K)) * scale).astype(np.float32)
    b = (rng.standard_normal((N, K)) * scale).astype(np.float32)
    return synth.round_to_storage(a, dtype), synth.round_to_storage(b, dtype)


def check_out16(dtype, A, Bt, sites, mode, gfmt, ofmt, addend=None):
    M, K = A.shape
    N = Bt.shape[0]
    n = 0 if sites is None else len(sites)
    a, b = to_dev(A, dtype), to_dev(Bt, dtype)
    cin = None if addend is None else torch.from_numpy(addend).cuda()
    D16, f16 = mpg.gemm(dtype, a, b, sites, mode, addend=cin, out_format=gfmt)
    C32, f32 = mpg.gemm(dtype, a, b, sites, mode, addend=cin)
    torch.cuda.synchronize()
    fg16, fg32 = f16.cpu().numpy().view(np.uint32), f32.cpu().numpy().view(np.uint32)
    assert not (fg16[0] & mpg.STATUS_WAIT_LIMIT)
    # header (but for the word that says how the last round was scheduled), site log and bitmap: those of the FP32 run
    same = fg16 == fg32
    same[5] = True
    assert same.all(), f"flags buffer differs from the FP32 run at words {np.nonzero(~same)[0][:8]}"
    got = as_u16(D16)
    c32 = C32.cpu().numpy()
    # (1) the rounding step, on the device's own FP32 words
    want_bits = np.array([orc.round_output(ofmt, int(x)) for x in c32.view(np.uint32).reshape(-1)], dtype=np.uint16).reshape(M, N)
    nan = np.isnan(c32)
    assert np.array_equal(got[~nan], want_bits[~nan]), "rounding of the device's FP32 result is not round-to-nearest-even"
    assert np.isnan(widen16(got[nan], gfmt)).all()
    # (2) against the oracle's 16-bit result
    Do, hdr_o, log_o, bm_o = orc.gemm_out16(dtype, A, Bt, ofmt, sites, mode, addend=addend)
    A2, B2 = faulted_operands(dtype, A, Bt, [] if sites is None else sites)
    tol = TOL * orc.absprod(dtype, A2, B2)
    if addend is not None:
        tol = tol + TOL * np.abs(addend).astype(np.float64)
    touched = np.zeros((M, N), dtype=bool)
    if sites is not None:
        for s in sites:
            if int(s["kind"]) in (orc.KIND_ACC, orc.KIND_OUT, orc.KIND_TERM) and s["row"] < M and s["col"] < N:
                touched[s["row"], s["col"]] = True       # a flipped bit scales the tolerance: covered by the FP32 parity tests
    g, o = widen16(got, gfmt), widen16(Do, gfmt)
    ok = close(g, o, tol + ulp16(o, gfmt)) | touched
    # an FP32 value at the edge of the format's range may go to infinity on one side only
    top = 65504.0 if gfmt == mpg.OUT_FP16 else 3.3895313892515355e38
    ok |= (np.isinf(g) | np.isinf(o)) & (np.abs(np.where(np.isinf(g), o, g)) >= top - tol - ulp16(top, gfmt))
    assert ok.all(), f"{(~ok).sum()} elements out of tolerance, first at {np.argwhere(~ok)[:5].tolist()}"
    if not touched.any():
        assert np.array_equal(fg16[16 + 4 * n:].reshape(M, -1), bm_o) and fg16[1] == hdr_o[1]
    return got


@pytest.mark.parametrize("gfmt,ofmt,tdt,ndt", FMTS)
@pytest.mark.parametrize("dtype", [orc.FP16, orc.BF16, orc.TF32])
@pytest.mark.parametrize("shape", [(128, 64, 64), (300, 200, 136), (1000, 520, 72), (257, 132, 8 * 33), (64, 1040, 512)])
def test_clean_gemm_with_16_bit_output(dtype, shape, gfmt, ofmt, tdt, ndt, tile_policy):
    """Ragged shapes, several tiles, N a multiple of 8 (bulk stores) or not (2-byte stores: 132 = 4 * 33)."""
    M, N, K = shape
    A, Bt = rand_operands(dtype, M, N, K, 31)
    check_out16(dtype, A, Bt, None, orc.T_BOUND | orc.CORRECT, gfmt, ofmt)


@pytest.mark.parametrize("gfmt,ofmt,tdt,ndt", FMTS)
def test_exact_integers_and_library_view(gfmt, ofmt, tdt, ndt, tile_policy):
    """Small integers survive the rounding; the result read as a torch tensor of the format is the integer product."""
    M, N, K = 256, 320, 128
    rng = np.random.default_rng(32)
    a = rng.integers(-3, 4, size=(M, K)).astype(np.float32)
    b = rng.integers(-3, 4, size=(N, K)).astype(np.float32)
    A, Bt = synth.round_to_storage(a, orc.BF16), synth.round_to_storage(b, orc.BF16)
    D, flags = mpg.gemm(orc.BF16, to_dev(A, orc.BF16), to_dev(Bt, orc.BF16), None, orc.T_BOUND, out_format=gfmt)
    torch.cuda.synchronize()
    assert D.dtype == tdt
    ref = a.astype(np.int64) @ b.astype(np.int64).T            # |values| < 256: exact in both formats
    assert np.abs(ref).max() < 256
    assert np.array_equal(D.float().cpu().numpy().astype(np.int64), ref)


@pytest.mark.parametrize("gfmt,ofmt,tdt,ndt", FMTS)
@pytest.mark.parametrize("dtype", [orc.FP16, orc.BF16, orc.TF32])
def test_sites_checks_and_range_ends(dtype, gfmt, ofmt, tdt, ndt, tile_policy):
    """All five site kinds with detection + correction; values that overflow FP16 without reaching the BoundCheck
    threshold become infinities without a flag; flagged values are corrected before they are rounded."""
    kt = synth.kstep(dtype)
    M, N, K = 300, 264, 3 * kt
    A, Bt = rand_operands(dtype, M, N, K, 33)
    # row 7 of A and row 9 of Bt made large: C[7, 9] = 280 * 250 = 70000 (beyond FP16, below 131072)
    big = np.zeros((1, K), dtype=np.float32)
    big[0, 0] = 280.0
    A[7] = synth.round_to_storage(big, dtype)[0]
    big[0, 0] = 250.0
    Bt[9] = synth.round_to_storage(big, dtype)[0]
    width = 19 if dtype == orc.TF32 else 16
    s = np.zeros(6, dtype=orc.SITE)
    s["kind"] = [orc.KIND_A, orc.KIND_B, orc.KIND_ACC, orc.KIND_OUT, orc.KIND_TERM, orc.KIND_OUT]
    s["row"] = [17, 0, 250, 299, 40, 3]
    s["col"] = [0, 200, 100, 263, 40, 64]
    s["k"] = [5, kt + 3, 2 * kt, 0, kt + 1, 0]
    s["xor_mask"] = [1 << (width - 2), 1 << (width - 2), 1 << 30, 1 << 30, 1 << 30, 1 << 23]
    for mode in (orc.T_BOUND | orc.CORRECT, orc.T_BOUND, orc.T_NONE):
        got = check_out16(dtype, A, Bt, s, mode, gfmt, ofmt)
        if gfmt == mpg.OUT_FP16:
            assert got[7, 9] == 0x7C00                       # 70000 -> +inf, and no flag was raised for it
    # with an addend
    rng = np.random.default_rng(34)
    cin = (rng.standard_normal((M, N)) * 2).astype(np.float32)
    check_out16(dtype, A, Bt, s, orc.T_BOUND | orc.CORRECT, gfmt, ofmt, addend=cin)


def test_argument_checks():
    A, Bt = rand_operands(orc.BF16, 128, 128, 64, 35)
    a, b = to_dev(A, orc.BF16), to_dev(Bt, orc.BF16)
    d = torch.empty((128, 128), dtype=torch.bfloat16, device="cuda")
    c = torch.zeros((128, 128), dtype=torch.float32, device="cuda")
    st = torch.cuda.current_stream().cuda_stream
    args = (orc.BF16, 128, 128, 64, a.data_ptr(), b.data_ptr())
    assert mpg.mpgemmfi_gemm_out16(*args, None, mpg.OUT_FP32, d.data_ptr(), None, 0, 0, None, st) == -2
    assert mpg.mpgemmfi_gemm_out16(*args, None, 7, d.data_ptr(), None, 0, 0, None, st) == -2
    assert mpg.mpgemmfi_gemm_out16(*args, None, mpg.OUT_BF16, None, None, 0, 0, None, st) == -1
    assert mpg.mpgemmfi_gemm_out16(*args, None, mpg.OUT_BF16, d.data_ptr() + 1, None, 0, 0, None, st) == -3
    assert mpg.mpgemmfi_gemm_out16(*args, c.data_ptr(), mpg.OUT_BF16, c.data_ptr(), None, 0, 0, None, st) == -1   # overlap
    assert mpg.mpgemmfi_gemm_out16(*args, None, mpg.OUT_BF16, d.data_ptr(), None, 0, 1, None, st) == -1           # check without flags
    assert mpg.mpgemmfi_gemm_out16(*args, c.data_ptr(), mpg.OUT_BF16, d.data_ptr(), None, 0, 0, None, st) == 0
    torch.cuda.synchronize()
    assert np.isfinite(d.float().cpu().numpy()).all()


@pytest.mark.parametrize("name", ["c3a", "c5"])
def test_full_size_16_bit_output(name):
    """The benchmark's FP16 configs with an FP16 result, default launch policy, every element: the rounding step bit for
    bit on the device's own FP32 result, the flags buffer equal to the FP32 run's, and sampled outputs against the oracle."""
    w = synth.make_workload(name, trials=16)
    M, N, K = w.M, w.N, w.K
    a, b = to_dev(w.A, w.dtype), to_dev(w.Bt, w.dtype)
    sites = w.sites[:16]
    D16, f16 = mpg.gemm(w.dtype, a, b, sites, w.detect_mode, out_format=mpg.OUT_FP16)
    C32, f32 = mpg.gemm(w.dtype, a, b, sites, w.detect_mode)
    torch.cuda.synchronize()
    fg16, fg32 = f16.cpu().numpy().view(np.uint32), f32.cpu().numpy().view(np.uint32)
    same = fg16 == fg32
    same[5] = True
    assert same.all() and not (fg16[0] & mpg.STATUS_WAIT_LIMIT)
    # library conversion of the device's FP32 result (round to nearest even) against the device's 16-bit result
    want = C32.to(torch.float16)
    eq = (want.view(torch.int16) == D16.view(torch.int16)) | (torch.isnan(want) & torch.isnan(D16))
    assert bool(eq.all()), f"{int((~eq).sum())} elements differ from the library's rounding of the FP32 result"
    rng = np.random.default_rng(36)
    si = np.concatenate([rng.integers(0, M, 2000), [0, M - 1, 0, M - 1, 127, 128]]).astype(np.uint32)
    sj = np.concatenate([rng.integers(0, N, 2000), [0, N - 1, N - 1, 0, N - 1, 0]]).astype(np.uint32)
    ref, ap = orc.sample(w.dtype, w.A, w.Bt, si, sj)
    want16 = np.array([orc.round_output(orc.OUT_FP16, int(x)) for x in ref.view(np.uint32)], dtype=np.uint16)
    got16 = as_u16(D16[torch.from_numpy(si.astype(np.int64)).cuda(), torch.from_numpy(sj.astype(np.int64)).cuda()])
    hit = np.zeros(len(si), dtype=bool)                # samples that a site reaches are covered by the FP32 parity tests
    for t in sites:
        kind = int(t["kind"])
        if kind == orc.KIND_A:
            hit |= si == t["row"]
        elif kind == orc.KIND_B:
            hit |= sj == t["col"]
        else:
            hit |= (si == t["row"]) & (sj == t["col"])
    g, o = widen16(got16, mpg.OUT_FP16), widen16(want16, mpg.OUT_FP16)
    assert (close(g, o, TOL * ap + ulp16(o, mpg.OUT_FP16)) | hit).all()
