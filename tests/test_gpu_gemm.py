"""GPU parity: mpgemmfi_gemm through the C ABI against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle as orc
import paper_2311_05782_b200 as mpg
import synth
from parity import (check_gemm_against_oracle, run_gpu_gemm, to_dev, close, TOL)

pytestmark = pytest.mark.gpu

DTYPES = [orc.FP16, orc.BF16, orc.TF32]


@pytest.fixture(params=["single", "pair"], autouse=True)
def tile_policy(request):
    """Every test of this file runs under both tilings of the kernel: whole tiles per CTA, and CTA pairs
    (the fuzz test picks its own tiling; it still runs once per parameter, on different seeds' worth of luck)."""
    assert mpg.mpgemmfi_set_tile_policy(mpg.TILES_PAIR if request.param == "pair" else mpg.TILES_SINGLE) == 0
    yield request.param
    mpg.mpgemmfi_set_tile_policy(mpg.TILES_AUTO)


def site(kind, row=0, col=0, k=0, mask=0):
    s = np.zeros(1, dtype=orc.SITE)
    s["kind"], s["row"], s["col"], s["k"], s["xor_mask"] = kind, row, col, k, mask
    return s


def rand_operands(dtype, M, N, K, seed, scale=1.0):
    rng = np.random.default_rng(seed)
    a = (rng.standard_normal((M, K)) * scale).astype(np.float32)
    b = (rng.standard_normal((N, K)) * scale).astype(np.float32)
    return synth.round_to_storage(a, dtype), synth.round_to_storage(b, dtype)


@pytest.mark.parametrize("dtype", DTYPES)
def test_exact_integer_gemm_single_tile(dtype):
    """Small integers: the tensor-core result must be exactly the integer product (layout, swizzle, descriptors)."""
    M, N, K = 128, 256, 128
    rng = np.random.default_rng(11)
    a = rng.integers(-4, 5, size=(M, K)).astype(np.float32)
    b = rng.integers(-4, 5, size=(N, K)).astype(np.float32)
    A, Bt = synth.round_to_storage(a, dtype), synth.round_to_storage(b, dtype)
    Cg, hdr, log, bm = run_gpu_gemm(dtype, A, Bt, None, orc.T_BOUND)
    ref = a.astype(np.int64) @ b.astype(np.int64).T
    assert np.array_equal(Cg.astype(np.int64), ref)
    assert hdr[0] == 0 and hdr[1] == 0 and not bm.any()


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("shape", [(128, 64, 64), (300, 200, 136), (1000, 520, 72), (257, 129, 8 * 33), (64, 1040, 512)])
def test_clean_gemm_with_ragged_tiles(dtype, shape):
    M, N, K = shape
    A, Bt = rand_operands(dtype, M, N, K, 12)
    check_gemm_against_oracle(dtype, A, Bt, None, orc.T_BOUND | orc.CORRECT)


def test_plain_gemm_without_flags_buffer():
    A, Bt = rand_operands(orc.BF16, 256, 256, 256, 13)
    Cg = torch.empty((256, 256), dtype=torch.float32, device="cuda")
    a, b = to_dev(A, orc.BF16), to_dev(Bt, orc.BF16)
    rc = mpg.mpgemmfi_gemm(orc.BF16, 256, 256, 256, a.data_ptr(), b.data_ptr(),
                           Cg.data_ptr(), None, 0, 0, None, torch.cuda.current_stream().cuda_stream)
    assert rc == 0
    torch.cuda.synchronize()
    Co, *_ = orc.gemm(orc.BF16, A, Bt)
    assert close(Cg.cpu().numpy(), Co, TOL * orc.absprod(orc.BF16, A, Bt)).all()


def test_argument_errors_are_reported_not_launched():
    A, Bt = rand_operands(orc.BF16, 128, 128, 64, 14)
    a, b = to_dev(A, orc.BF16), to_dev(Bt, orc.BF16)
    c = torch.empty((128, 128), dtype=torch.float32, device="cuda")
    st = torch.cuda.current_stream().cuda_stream
    f = torch.empty(mpg.mpgemmfi_flags_bytes(128, 128, 0) // 4, dtype=torch.int32, device="cuda")
    assert mpg.mpgemmfi_gemm(7, 128, 128, 64, a.data_ptr(), b.data_ptr(), c.data_ptr(), None, 0, 0, f.data_ptr(), st) == -2
    assert mpg.mpgemmfi_gemm(1, 0, 128, 64, a.data_ptr(), b.data_ptr(), c.data_ptr(), None, 0, 0, f.data_ptr(), st) == -1
    assert mpg.mpgemmfi_gemm(1, 128, 128, 64, a.data_ptr() + 2, b.data_ptr(), c.data_ptr(), None, 0, 0, f.data_ptr(), st) == -3
    assert mpg.mpgemmfi_gemm(1, 128, 128, 60, a.data_ptr(), b.data_ptr(), c.data_ptr(), None, 0, 0, f.data_ptr(), st) == -3
    assert mpg.mpgemmfi_gemm(1, 128, 128, 64, a.data_ptr(), b.data_ptr(), c.data_ptr(), None, 1, 0, f.data_ptr(), st) == -1
    assert mpg.mpgemmfi_gemm(1, 128, 128, 64, a.data_ptr(), b.data_ptr(), c.data_ptr(), None, 0, 1, None, st) == -1
    torch.cuda.synchronize()


@pytest.mark.parametrize("dtype", DTYPES)
def test_every_bit_of_one_output_element(dtype):
    M, N, K = 256, 256, 128
    A, Bt = rand_operands(dtype, M, N, K, 15)
    sites = np.concatenate([site(orc.KIND_OUT, 200 + (b % 3), 7 * b + 1, 0, 1 << b) for b in range(32)])
    check_gemm_against_oracle(dtype, A, Bt, sites, orc.T_BOUND)
    check_gemm_against_oracle(dtype, A, Bt, sites, orc.T_BOUND | orc.CORRECT)
    check_gemm_against_oracle(dtype, A, Bt, sites, orc.T_NONE)


@pytest.mark.parametrize("dtype", DTYPES)
def test_operand_sites_corners_and_every_bit(dtype):
    M, N, K = 384, 512, 192
    A, Bt = rand_operands(dtype, M, N, K, 16, scale=0.25)
    width = 19 if dtype == orc.TF32 else 16
    parts = []
    for b in range(width):
        parts.append(site(orc.KIND_A, (37 * b) % M, 0, (11 * b) % K, 1 << b))
        parts.append(site(orc.KIND_B, 0, (53 * b) % N, (13 * b + 5) % K, 1 << b))
    parts += [site(orc.KIND_A, 0, 0, 0, 1 << (width - 2)), site(orc.KIND_A, M - 1, 0, K - 1, 1 << (width - 2)),
              site(orc.KIND_B, 0, 0, 0, 1 << (width - 2)), site(orc.KIND_B, 0, N - 1, K - 1, 1 << (width - 2)),
              site(orc.KIND_A, 5, 0, 70, 0x3), site(orc.KIND_A, 5, 0, 70, 0x3)]      # the last two cancel
    sites = np.concatenate(parts)
    check_gemm_against_oracle(dtype, A, Bt, sites, orc.T_BOUND | orc.CORRECT, max_fragile=0)
    check_gemm_against_oracle(dtype, A, Bt, sites, orc.T_BOUND)


@pytest.mark.parametrize("dtype", DTYPES)
def test_accumulator_sites_at_every_boundary(dtype):
    kt = synth.kstep(dtype)
    M, N, K = 256, 320, 5 * kt + kt // 2          # ragged last k-step: the boundary k = K is allowed
    A, Bt = rand_operands(dtype, M, N, K, 17)
    parts = []
    for b in range(1, 6):
        parts.append(site(orc.KIND_ACC, (61 * b) % M, (97 * b) % N, b * kt, 1 << (20 + b)))
    parts.append(site(orc.KIND_ACC, 255, 319, K, 1 << 30))
    parts.append(site(orc.KIND_ACC, 0, 0, kt, 3 << 29))
    parts.append(site(orc.KIND_ACC, 130, 300, 2 * kt, 1 << 31))
    parts.append(site(orc.KIND_ACC, 130, 300, 4 * kt, 1 << 22))      # same element, two boundaries
    parts.append(site(orc.KIND_ACC, 3, 3, kt + 1, 1 << 30))           # not on a boundary: skipped on the GPU
    sites = np.concatenate(parts)
    # the oracle accepts any k; give it only what the GPU interface admits, then check the skip separately
    Cg, hdr, log, bm = run_gpu_gemm(dtype, A, Bt, sites, orc.T_BOUND)
    assert hdr[4] == 1 and hdr[0] & mpg.STATUS_SITE_SKIPPED and log["status"][-1] == 2
    check_gemm_against_oracle(dtype, A, Bt, sites[:-1], orc.T_BOUND, max_fragile=1)
    check_gemm_against_oracle(dtype, A, Bt, sites[:-1], orc.T_BOUND | orc.CORRECT, max_fragile=1)


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("tech", [orc.T_NONE, orc.T_BOUND, orc.T_RMAX, orc.T_RFLIP])
def test_term_sites_with_each_technique(dtype, tech):
    kt = synth.kstep(dtype)
    M, N, K = 128, 192, 3 * kt
    A, Bt = rand_operands(dtype, M, N, K, 18)
    rng = np.random.default_rng(19)
    parts = []
    for n in range(24):
        nb = (1, 2, 4)[n % 3]
        start = int(rng.integers(0, 33 - nb))
        parts.append(site(orc.KIND_TERM, int(rng.integers(0, M)), int(rng.integers(0, N)), int(rng.integers(0, K)),
                          ((1 << nb) - 1) << start))
    parts.append(site(orc.KIND_TERM, 127, 191, K - 1, 1 << 30))
    parts.append(site(orc.KIND_TERM, 0, 0, 0, 1 << 30))
    sites = np.concatenate(parts)
    for corr in (0, orc.CORRECT):
        check_gemm_against_oracle(dtype, A, Bt, sites, tech | corr, max_fragile=0)


def test_term_site_sees_a_faulty_operand():
    kt = 64
    A, Bt = rand_operands(orc.BF16, 128, 128, 2 * kt, 20)
    sites = np.concatenate([site(orc.KIND_A, 9, 0, 70, 1 << 14), site(orc.KIND_TERM, 9, 17, 70, 1 << 3),
                            site(orc.KIND_B, 0, 40, 5, 1 << 15), site(orc.KIND_TERM, 77, 40, 5, 1 << 29)])
    check_gemm_against_oracle(orc.BF16, A, Bt, sites, orc.T_RMAX | orc.CORRECT)
    check_gemm_against_oracle(orc.BF16, A, Bt, sites, orc.T_BOUND | orc.CORRECT)


def test_boundcheck_over_all_256_exponents():
    """Outputs on every FP32 exponent: products 2^(i-64) * 2^(j-32) * (1 + j/64), and all 256 exponents via OUT sites."""
    M, N, K = 128, 64, 64
    a = np.zeros((M, K), dtype=np.float32)
    b = np.zeros((N, K), dtype=np.float32)
    a[:, 0] = np.ldexp(1.0, np.arange(M) - 64)
    b[:, 0] = np.ldexp(1.0 + np.arange(N) / 64.0, np.arange(N) - 32)
    A, Bt = synth.round_to_storage(a, orc.BF16), synth.round_to_storage(b, orc.BF16)
    Cg, hdr, log, bm = run_gpu_gemm(orc.BF16, A, Bt, None, orc.T_BOUND)
    assert hdr[1] == (np.abs(Cg) >= 131072.0).sum() > 500
    check_gemm_against_oracle(orc.BF16, A, Bt, None, orc.T_BOUND)
    check_gemm_against_oracle(orc.BF16, A, Bt, None, orc.T_BOUND | orc.CORRECT)
    z = np.zeros((128, 64), dtype=np.uint16)
    zb = np.zeros((64, 64), dtype=np.uint16)
    sites = np.concatenate([site(orc.KIND_OUT, e % 128, e // 4, 0, (e << 23) | (0x155555 if e % 2 else 0))
                            for e in range(256)])
    check_gemm_against_oracle(orc.BF16, z, zb, sites, orc.T_BOUND)
    check_gemm_against_oracle(orc.BF16, z, zb, sites, orc.T_BOUND | orc.CORRECT)


def test_many_sites_on_one_element_and_determinism():
    A, Bt = rand_operands(orc.FP16, 128, 128, 128, 21)
    sites = np.concatenate([site(orc.KIND_OUT, 5, 6, 0, 1 << 30), site(orc.KIND_OUT, 5, 6, 0, 1 << 29),
                            site(orc.KIND_ACC, 5, 6, 64, 1 << 31), site(orc.KIND_TERM, 5, 6, 100, 1 << 25),
                            site(orc.KIND_OUT, 5, 6, 0, 1 << 30)])
    check_gemm_against_oracle(orc.FP16, A, Bt, sites, orc.T_BOUND | orc.CORRECT, max_fragile=1)
    r1 = run_gpu_gemm(orc.FP16, A, Bt, sites, orc.T_BOUND)
    r2 = run_gpu_gemm(orc.FP16, A, Bt, sites, orc.T_BOUND)
    for x, y in zip(r1, r2):
        assert np.array_equal(np.asarray(x).view(np.uint8), np.asarray(y).view(np.uint8))


def test_injection_disabled_equals_empty_table_bitwise():
    A, Bt = rand_operands(orc.BF16, 512, 512, 512, 22)
    c0, *_ = run_gpu_gemm(orc.BF16, A, Bt, None, orc.T_NONE)
    c1, hdr, log, bm = run_gpu_gemm(orc.BF16, A, Bt, site(orc.KIND_OUT, 9999, 0, 0, 1), orc.T_BOUND)
    assert np.array_equal(c0.view(np.uint32), c1.view(np.uint32)) and hdr[4] == 1 and hdr[3] == 0


@pytest.mark.parametrize("name,shape,trials", [
    ("c1", (256, 256, 256), 64),
    ("c2", (512, 768, 512), 96),
    ("c3a", (640, 512, 256), 128),
    ("c3b", (640, 256, 512), 128),
    ("c4", (384, 512, 256), 96),
    ("c5", (2048, 64, 576), 128),
])
def test_config_tables_in_one_gemm(name, shape, trials):
    """The configs' site mixes at reduced sizes, all sites of the table applied in one call."""
    M, N, K = shape
    w = synth.make_workload(name, M, N, K, trials=trials)
    check_gemm_against_oracle(w.dtype, w.A, w.Bt, w.sites, w.detect_mode, max_fragile=1)


@pytest.mark.parametrize("dtype", DTYPES)
def test_host_table_in_the_launch_parameters_equals_the_device_table(dtype):
    """A table of up to INLINE_FAULTS entries in host memory travels in the launch parameters; the same table in
    device memory gives the same C and the same flags buffer bit for bit, on every entry point. The host-table
    results are also checked against the oracle (every other test that passes a short numpy table goes that way)."""
    kt = synth.kstep(dtype)
    M, N, K = 520, 392, 5 * kt
    A, Bt = rand_operands(dtype, M, N, K, 23)
    hi = 31 if dtype == orc.TF32 else 15
    full = np.concatenate([
        site(orc.KIND_A, 300, 0, 2 * kt + 1, 1 << (hi - 1)), site(orc.KIND_B, 0, 391, 7, 1 << (hi - 2)),
        site(orc.KIND_ACC, 519, 3, 3 * kt, 1 << 30), site(orc.KIND_TERM, 128, 256, 4 * kt + 3, 1 << 29),
        site(orc.KIND_OUT, 0, 0, 0, 1 << 30), site(orc.KIND_OUT, 9999, 0, 0, 1),      # the last one is out of range
        site(orc.KIND_OUT, 257, 131, 0, 1 << 27), site(orc.KIND_A, 300, 0, 2 * kt + 1, 1 << (hi - 3))])
    assert len(full) == mpg.INLINE_FAULTS
    a, b = to_dev(A, dtype), to_dev(Bt, dtype)
    cin = torch.from_numpy(np.random.default_rng(24).standard_normal((M, N)).astype(np.float32)).cuda()
    for n in (1, 5, 8):
        sites = full[:n]
        for mode in (orc.T_BOUND | orc.CORRECT, orc.T_RMAX):
            check_gemm_against_oracle(dtype, A, Bt, sites, mode, max_fragile=1)
            for kw in ({}, {"addend": cin}, {"out_format": mpg.OUT_BF16}):
                c_h, f_h = mpg.gemm(dtype, a, b, sites, mode, inline_sites=True, **kw)
                c_d, f_d = mpg.gemm(dtype, a, b, sites, mode, inline_sites=False, **kw)
                torch.cuda.synchronize()
                fh, fd = f_h.cpu().numpy(), f_d.cpu().numpy()
                assert np.array_equal(fh, fd), (n, mode, kw.keys(), np.nonzero(fh != fd)[0][:8])
                assert torch.equal(c_h.view(torch.int32 if c_h.dtype == torch.float32 else torch.int16),
                                   c_d.view(torch.int32 if c_d.dtype == torch.float32 else torch.int16))
                if n >= 6:
                    assert fh.view(np.uint32)[4] == 1          # the out-of-range entry was skipped, not applied
    # a host table beyond the limit is refused before anything is launched
    long = np.ascontiguousarray(np.concatenate([full, full[:1]]))
    c = torch.empty((M, N), dtype=torch.float32, device="cuda")
    f = torch.empty(mpg.mpgemmfi_flags_bytes(M, N, len(long)) // 4, dtype=torch.int32, device="cuda")
    host = np.zeros(len(long) * 8 + 4, dtype=np.int32)
    off = (-host.ctypes.data % 16) // 4
    host[off:off + len(long) * 8] = long.view(np.int32).reshape(-1)
    rc = mpg.mpgemmfi_gemm(dtype, M, N, K, a.data_ptr(), b.data_ptr(), c.data_ptr(), host.ctypes.data + 4 * off, len(long),
                           orc.T_BOUND, f.data_ptr(), torch.cuda.current_stream().cuda_stream)
    assert rc == -1
    torch.cuda.synchronize()


@pytest.mark.parametrize("name,shape,mix,trials", [
    ("c5", (384, 192, 256), "mixed", 700),
    ("c2", (520, 392, 320), "operand", 600),
    ("c5", (384, 192, 256), "term_op", 300),
    ("c4", (300, 264, 160), "acc", 500),
])
def test_long_tables_on_few_tiles(name, shape, mix, trials):
    """Hundreds of sites on a handful of tiles: every CTA's list is longer than its shared-memory cache and holds
    operand, accumulator / term and output sites side by side (the list is kept by class, each class in table
    order); many sites share rows, columns and k-steps. Everything against the oracle: values, flags, header, log."""
    M, N, K = shape
    w = synth.make_workload(name, M, N, K, trials=trials, mix=mix)
    extra = synth.make_workload(name, M, N, K, trials=trials // 3, mix="out").sites
    sites = np.concatenate([w.sites, extra]) if mix != "mixed" else w.sites
    check_gemm_against_oracle(w.dtype, w.A, w.Bt, sites, w.detect_mode, max_fragile=3)


def test_maximum_site_count():
    w = synth.make_workload("c5", 1024, 64, 192, trials=mpg.MAX_FAULTS, mix="out")
    check_gemm_against_oracle(w.dtype, w.A, w.Bt, w.sites, w.detect_mode, max_fragile=2)
    a, b = to_dev(w.A, w.dtype), to_dev(w.Bt, w.dtype)
    with pytest.raises(mpg.MpgemmfiError):
        mpg.gemm(w.dtype, a, b, np.zeros(mpg.MAX_FAULTS + 1, dtype=orc.SITE), 0)


def test_tf32_low_mantissa_bits_are_ignored(tile_policy):
    """FP32 words whose low 13 bits are not zero: the tensor core must see only the top 19 bits (the oracle masks them)."""
    rng = np.random.default_rng(23)
    M, N, K = 256, 256, 96
    a = rng.standard_normal((M, K)).astype(np.float32).view(np.uint32)
    b = rng.standard_normal((N, K)).astype(np.float32).view(np.uint32)
    assert (a & 0x1FFF).any()
    Cg, *_ = run_gpu_gemm(orc.TF32, a, b, None, orc.T_NONE)
    Co, *_ = orc.gemm(orc.TF32, a, b)                       # widens with the low 13 bits dropped
    ok = close(Cg, Co, TOL * orc.absprod(orc.TF32, a, b))
    # a tensor core that rounded instead of truncating would be off by up to 2^-11 relative per operand: still inside
    # the 1e-3 tolerance, so also demand the tight bound that only truncation meets
    tight = np.abs(Cg - Co) <= 2e-6 * orc.absprod(orc.TF32, a, b)
    assert ok.all() and tight.mean() > 0.999


@pytest.mark.parametrize("dtype", DTYPES)
def test_degenerate_shapes_and_special_values(dtype, tile_policy):
    """One row, one column, the shortest legal K; zeros, subnormals, huge values, Inf and NaN among the operands."""
    kmin = 4 if dtype == orc.TF32 else 8                      # K * element size must be a multiple of 16 bytes
    for (M, N, K) in [(1, 1, kmin), (1, 37, kmin), (129, 1, 3 * kmin), (5, 7, 72)]:
        A, Bt = rand_operands(dtype, M, N, K, 40 + M + N)
        check_gemm_against_oracle(dtype, A, Bt, site(orc.KIND_OUT, M - 1, N - 1, 0, 1 << 30), orc.T_BOUND | orc.CORRECT)
    M, N, K = 130, 70, 80
    rng = np.random.default_rng(41)
    a = rng.standard_normal((M, K)).astype(np.float32)
    b = rng.standard_normal((N, K)).astype(np.float32)
    a[rng.random((M, K)) < 0.3] = 0.0                         # sparse rows, as after a ReLU
    a[3, 5] = np.inf; a[7, 9] = -np.inf; a[11, 2] = np.nan
    a[20, :] = 0.0                                            # a whole zero row: exact zeros out
    a[30, 1] = 3e4 if dtype == orc.FP16 else 1e30             # products far above the BoundCheck threshold
    b[4, 5] = 1e-7 if dtype == orc.FP16 else 1e-39            # FP16 / FP32 subnormal after rounding
    b[6, :] = 0.0
    b[8, 9] = np.inf                                          # meets -inf * ... and 0 * inf -> NaN
    A, Bt = synth.round_to_storage(a, dtype), synth.round_to_storage(b, dtype)
    for mode in (orc.T_BOUND, orc.T_BOUND | orc.CORRECT, orc.T_NONE):
        Cg, hdr, log, bm = run_gpu_gemm(dtype, A, Bt, None, mode)
        Co, hdr_o, _, bm_o = orc.gemm(dtype, A, Bt, None, mode)
        tol = TOL * orc.absprod(dtype, A, Bt)                 # infinite or NaN where a special value takes part
        assert close(Cg, Co, tol).all()
        special = ~np.isfinite(tol)
        assert np.array_equal(np.isnan(Cg[special]) | np.isinf(Cg[special]) | (mode == (orc.T_BOUND | orc.CORRECT)),
                              np.isnan(Co[special]) | np.isinf(Co[special]) | (mode == (orc.T_BOUND | orc.CORRECT)))
        d = np.argwhere(bm != bm_o)
        info = [(int(i), int(w), hex(int(bm[i, w])), hex(int(bm_o[i, w])), Cg[i, 32 * w:32 * w + 32][:12].tolist(), Co[i, 32 * w:32 * w + 32][:12].tolist()) for i, w in d[:3]]
        assert np.array_equal(bm, bm_o) and hdr[1] == hdr_o[1], info      # NaN, Inf and huge values are flagged alike
        assert (Cg[20][np.isfinite(tol[20])] == 0).all() and (Cg[:, 6][np.isfinite(tol[:, 6])] == 0).all()


@pytest.mark.parametrize("dtype", DTYPES)
def test_output_level_range_check(dtype, tile_policy):
    """RangeCheck extended to output elements (exponent maxima of the clean operands): clean runs flag nothing,
    operand / output / accumulator faults that push an exponent over the bound are flagged and corrected as the oracle says."""
    kt = synth.kstep(dtype)
    M, N, K = 300, 330, 4 * kt + 8
    rng = np.random.default_rng(71)
    a = (rng.standard_normal((M, K)) * np.exp2(rng.integers(-6, 6, (M, 1)))).astype(np.float32)
    b = (rng.standard_normal((N, K)) * np.exp2(rng.integers(-6, 6, (N, 1)))).astype(np.float32)
    A, Bt = synth.round_to_storage(a, dtype), synth.round_to_storage(b, dtype)
    # exponent maxima kernel against the oracle
    ea = torch.empty(M, dtype=torch.int32, device="cuda"); eb = torch.empty(N, dtype=torch.int32, device="cuda")
    da, db = to_dev(A, dtype), to_dev(Bt, dtype)
    st = torch.cuda.current_stream().cuda_stream
    assert mpg.mpgemmfi_operand_exponents(dtype, M, K, da.data_ptr(), ea.data_ptr(), st) == 0
    assert mpg.mpgemmfi_operand_exponents(dtype, N, K, db.data_ptr(), eb.data_ptr(), st) == 0
    torch.cuda.synchronize()
    assert np.array_equal(ea.cpu().numpy().view(np.uint32), orc.operand_exponents(dtype, A))
    assert np.array_equal(eb.cpu().numpy().view(np.uint32), orc.operand_exponents(dtype, Bt))
    width = 19 if dtype == orc.TF32 else 16
    sites = np.concatenate([
        site(orc.KIND_A, 17, 0, 5, 1 << (width - 2)), site(orc.KIND_B, 0, 200, kt + 3, 1 << (width - 2)),
        site(orc.KIND_OUT, 299, 329, 0, 1 << 30), site(orc.KIND_OUT, 150, 31, 0, 1 << 29), site(orc.KIND_OUT, 3, 64, 0, 1 << 23),
        site(orc.KIND_ACC, 250, 100, 2 * kt, 1 << 30), site(orc.KIND_TERM, 40, 40, 3 * kt + 1, 1 << 30),
    ])
    for mode in (orc.T_RMAX | orc.OUTPUT_RANGE, orc.T_RMAX | orc.CORRECT | orc.OUTPUT_RANGE, orc.T_RFLIP | orc.CORRECT | orc.OUTPUT_RANGE):
        Cg, hdr, log, bm = run_gpu_gemm(dtype, A, Bt, None, mode)
        assert hdr[0] == 0 and hdr[1] == 0 and not bm.any()           # no false positive on a clean product
        Cg, hdr, log, bm = run_gpu_gemm(dtype, A, Bt, sites, mode)
        Co, hdr_o, log_o, bm_o = orc.gemm(dtype, A, Bt, sites, mode)
        assert hdr[0] == 0 and hdr[3] == len(sites)
        from parity import faulted_operands
        A2, B2 = faulted_operands(dtype, A, Bt, sites)
        tol = TOL * orc.absprod(dtype, A2, B2)
        # flags: exact, except where an element sits within tolerance of the binade edge that its bound happens to be:
        # the side that left it unflagged still holds the unchecked value, which must lie just below 2^(bound - 126)
        EA0, EB0 = orc.operand_exponents(dtype, A), orc.operand_exponents(dtype, Bt)
        diff = bm ^ bm_o
        n_edge = 0
        for (i, w) in np.argwhere(diff):
            for j in range(32 * w, min(N, 32 * w + 32)):
                if (int(diff[i, w]) >> (j % 32)) & 1:
                    raw = float(Co[i, j]) if (int(bm[i, w]) >> (j % 32)) & 1 else float(Cg[i, j])
                    edge = 2.0 ** (orc.output_range_bound(int(EA0[i]), int(EB0[j]), K) - 126)
                    assert 0.0 <= edge - abs(raw) <= tol[i, j], (i, j, raw, edge)
                    n_edge += 1
        assert hdr[1] > N // 2                                          # the faulty A element shows in most of its row
        assert abs(int(hdr[1]) - int(hdr_o[1])) <= n_edge
        touched = np.zeros((M, N), dtype=bool)
        for s_ in sites:
            if s_["kind"] in (orc.KIND_OUT, orc.KIND_ACC, orc.KIND_TERM):
                touched[s_["row"], s_["col"]] = True
        unflagged = np.zeros((M, N), dtype=bool)
        for i in range(M):
            for w in range(bm.shape[1]):
                both = ~(bm[i, w] | bm_o[i, w])
                for j in range(32 * w, min(N, 32 * w + 32)):
                    unflagged[i, j] = (both >> (j % 32)) & 1
        assert (close(Cg, Co, tol) | touched | ~unflagged).all()
        if mode & orc.CORRECT:
            # every stored exponent respects its bound
            EA, EB = orc.operand_exponents(dtype, A), orc.operand_exponents(dtype, Bt)
            L = int(np.ceil(np.log2(K)))
            bound = np.clip(EA[:, None].astype(np.int64) + EB[None, :].astype(np.int64) - 126 + L, 0, 255)
            assert (((Cg.view(np.uint32) >> 23) & 0xFF).astype(np.int64) <= bound).all()
    # the plain entry point refuses the flag; the ranged one refuses it with BoundCheck or without maxima
    c = torch.empty((M, N), dtype=torch.float32, device="cuda")
    f = torch.empty(mpg.mpgemmfi_flags_bytes(M, N, 0) // 4, dtype=torch.int32, device="cuda")
    args = (dtype, M, N, K, da.data_ptr(), db.data_ptr(), c.data_ptr(), None, 0)
    assert mpg.mpgemmfi_gemm(*args, orc.T_RMAX | orc.OUTPUT_RANGE, f.data_ptr(), st) == -1
    assert mpg.mpgemmfi_gemm_ranged(*args, orc.T_BOUND | orc.OUTPUT_RANGE, f.data_ptr(), ea.data_ptr(), eb.data_ptr(), st) == -1
    assert mpg.mpgemmfi_gemm_ranged(*args, orc.T_RMAX | orc.OUTPUT_RANGE, f.data_ptr(), None, eb.data_ptr(), st) == -1
    assert mpg.mpgemmfi_gemm_ranged(*args, orc.T_RMAX, f.data_ptr(), None, None, st) == 0
    torch.cuda.synchronize()


@pytest.mark.parametrize("seed", range(24))
def test_random_shapes_tables_and_modes(seed):
    """Differential fuzz against the oracle: random shape, format, tiling, check mode and site table (all kinds,
    repeated elements, a few invalid entries)."""
    rng = np.random.default_rng(1000 + seed)
    dtype = int(rng.integers(0, 3))
    kt = synth.kstep(dtype)
    unit = 4 if dtype == orc.TF32 else 8
    M = int(rng.integers(1, 700)); N = int(rng.integers(1, 700)); K = unit * int(rng.integers(1, 60))
    policy = [mpg.TILES_AUTO, mpg.TILES_SINGLE, mpg.TILES_PAIR][seed % 3]
    mode = int(rng.choice([orc.T_NONE, orc.T_BOUND, orc.T_BOUND | orc.CORRECT, orc.T_RMAX | orc.CORRECT, orc.T_RFLIP | orc.CORRECT]))
    A, Bt = rand_operands(dtype, M, N, K, 2000 + seed, scale=float(rng.choice([0.01, 1.0, 30.0])))
    n = int(rng.integers(0, 40))
    s = np.zeros(n, dtype=orc.SITE)
    s["kind"] = rng.integers(0, 5, n)
    s["row"] = rng.integers(0, M, n); s["col"] = rng.integers(0, N, n)
    nb = (K + kt - 1) // kt
    k_acc = np.minimum(rng.integers(1, nb + 1, n) * kt, K)
    s["k"] = np.where(s["kind"] == orc.KIND_ACC, k_acc, rng.integers(0, K, n))
    width = np.where(s["kind"] <= orc.KIND_B, 19 if dtype == orc.TF32 else 16, 32)
    nbits = rng.choice([1, 2, 4], n)
    s["xor_mask"] = [(((1 << int(b)) - 1) << int(rng.integers(0, int(w) - int(b) + 1))) for b, w in zip(nbits, width)]
    if n >= 4:                                             # repeats on one element, and entries the device must skip
        s[1] = s[0]; s["row"][2] = M + 5; s["kind"][3] = 7
    mpg.mpgemmfi_set_tile_policy(policy)
    try:
        check_gemm_against_oracle(dtype, A, Bt, s, mode, max_fragile=2)
    finally:
        mpg.mpgemmfi_set_tile_policy(mpg.TILES_AUTO)
