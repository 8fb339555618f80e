"""GPU parity of mpgemmfi_gemm_addend (D = A x B + C_in, Section II-B) against the CPU oracle.

The addend is where every running sum starts, so besides the values themselves the tests look at what the
accumulator / term / output sites meet, at both tilings, at the split schedule (a cut tile's first part takes
the addend, the later parts the sums left in D), at addends that allow no 16-byte reads, and at D written
over C_in.
"""
import numpy as np
import pytest
import torch

import oracle as orc
import paper_2311_05782_b200 as mpg
import synth
from parity import check_gemm_against_oracle, run_gpu_gemm, to_dev

pytestmark = pytest.mark.gpu

DTYPES = [orc.FP16, orc.BF16, orc.TF32]


@pytest.fixture
def policies():
    yield
    mpg.mpgemmfi_set_tile_policy(mpg.TILES_AUTO)
    mpg.mpgemmfi_set_split_policy(mpg.SPLIT_AUTO)


def rand_operands(dtype, M, N, K, seed):
    rng = np.random.default_rng(seed)
    a = rng.standard_normal((M, K)).astype(np.float32)
    b = rng.standard_normal((N, K)).astype(np.float32)
    return synth.round_to_storage(a, dtype), synth.round_to_storage(b, dtype)


def rand_addend(M, N, seed, scale=4.0):
    return (np.random.default_rng(seed).standard_normal((M, N)) * scale).astype(np.float32)


def site_table(dtype, M, N, K, n, seed):
    """All five kinds, uniformly placed, single-bit masks; accumulator sites on k-step boundaries."""
    rng = np.random.default_rng(seed)
    kt = synth.kstep(dtype)
    s = np.zeros(n, dtype=orc.SITE)
    s["kind"] = rng.integers(0, 5, n)
    s["row"] = rng.integers(0, M, n); s["col"] = rng.integers(0, N, n)
    nb = (K + kt - 1) // kt
    k_acc = np.minimum(rng.integers(1, nb + 1, n) * kt, K)
    s["k"] = np.where(s["kind"] == orc.KIND_ACC, k_acc, rng.integers(0, K, n))
    width = np.where(s["kind"] <= orc.KIND_B, 19 if dtype == orc.TF32 else 16, 32)
    s["xor_mask"] = [1 << int(rng.integers(0, int(w))) for w in width]
    return s


@pytest.mark.parametrize("tiles", [mpg.TILES_SINGLE, mpg.TILES_PAIR])
@pytest.mark.parametrize("dtype", DTYPES)
def test_exact_integers_with_addend(dtype, tiles, policies):
    """Small integers: D is the integer product plus the addend exactly, on several tiles with ragged edges."""
    assert mpg.mpgemmfi_set_tile_policy(tiles) == 0
    M, N, K = 520, 776, 200
    rng = np.random.default_rng(31)
    a = rng.integers(-4, 5, size=(M, K)).astype(np.float32)
    b = rng.integers(-4, 5, size=(N, K)).astype(np.float32)
    cin = rng.integers(-1000, 1001, size=(M, N)).astype(np.float32)
    A, Bt = synth.round_to_storage(a, dtype), synth.round_to_storage(b, dtype)
    D, hdr, _, bm = run_gpu_gemm(dtype, A, Bt, None, orc.T_BOUND, addend=cin)
    assert np.array_equal(D.astype(np.int64), a.astype(np.int64) @ b.astype(np.int64).T + cin.astype(np.int64))
    assert hdr[0] == 0 and hdr[1] == 0 and not bm.any()


@pytest.mark.parametrize("tiles", [mpg.TILES_SINGLE, mpg.TILES_PAIR])
@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("shape", [(300, 200, 136), (1000, 520, 72), (257, 131, 8 * 33), (64, 1040, 512)])
def test_addend_with_sites_against_oracle(dtype, shape, tiles, policies):
    """Values, site logs and flags with an addend; (257, 131, ...) has rows that allow no 16-byte reads."""
    assert mpg.mpgemmfi_set_tile_policy(tiles) == 0
    M, N, K = shape
    A, Bt = rand_operands(dtype, M, N, K, 32)
    cin = rand_addend(M, N, 33)
    sites = site_table(dtype, M, N, K, 200, 34)
    check_gemm_against_oracle(dtype, A, Bt, sites, orc.T_BOUND | orc.CORRECT, max_fragile=2, addend=cin)


@pytest.mark.parametrize("dtype", DTYPES)
def test_addend_large_enough_to_be_flagged(dtype):
    """An addend beyond BoundCheck's threshold carries through to D and is flagged (and corrected) there."""
    M, N, K = 256, 320, 128
    A, Bt = rand_operands(dtype, M, N, K, 35)
    cin = rand_addend(M, N, 36)
    cin[5, 7] = 3.0e6
    cin[200, 319] = -1.0e9
    for mode in (orc.T_BOUND, orc.T_BOUND | orc.CORRECT):
        D, hdr, _, bm = run_gpu_gemm(dtype, A, Bt, None, mode, addend=cin)
        assert hdr[1] == 2 and (bm[5, 0] >> 7) & 1 and (bm[200, 9] >> 31) & 1
        check_gemm_against_oracle(dtype, A, Bt, None, mode, addend=cin)


def test_in_place_equals_out_of_place(policies):
    """D written over C_in gives the same words as D written elsewhere, under both tilings and with a cut last round."""
    dtype, M, N, K = orc.BF16, 2304, 2300, 520
    A, Bt = rand_operands(dtype, M, N, K, 37)
    cin = rand_addend(M, N, 38)
    sites = site_table(dtype, M, N, K, 300, 39)
    for tiles in (mpg.TILES_SINGLE, mpg.TILES_PAIR):
        for split in (mpg.SPLIT_OFF, mpg.SPLIT_ON):
            assert mpg.mpgemmfi_set_tile_policy(tiles) == 0 and mpg.mpgemmfi_set_split_policy(split) == 0
            out = run_gpu_gemm(dtype, A, Bt, sites, orc.T_BOUND, addend=cin)
            inp = run_gpu_gemm(dtype, A, Bt, sites, orc.T_BOUND, addend=cin.copy(), in_place=True)
            assert not (out[1][0] & mpg.STATUS_WAIT_LIMIT) and not (inp[1][0] & mpg.STATUS_WAIT_LIMIT)
            assert np.array_equal(out[0].view(np.uint32), inp[0].view(np.uint32))
            assert np.array_equal(out[3], inp[3])
            for f in out[2].dtype.names:
                assert np.array_equal(out[2][f], inp[2][f]), f


# (tile policy, dtype, M, N, K): a few tiles left over for the last round, which the split schedule cuts along K
SPLIT_CASES = [
    (mpg.TILES_PAIR, orc.BF16, 2304, 2300, 520),
    (mpg.TILES_PAIR, orc.TF32, 3584, 3072, 264),
    (mpg.TILES_SINGLE, orc.FP16, 1500, 3328, 512),
]


@pytest.mark.parametrize("case", SPLIT_CASES)
def test_addend_under_the_split_schedule(case, policies):
    """Cut tiles (first part from the addend, later parts from the sums left in D) equal whole tiles word for word,
    and both agree with the oracle."""
    tiles, dtype, M, N, K = case
    A, Bt = rand_operands(dtype, M, N, K, 40)
    cin = rand_addend(M, N, 41)
    sites = site_table(dtype, M, N, K, 400, 42)
    assert mpg.mpgemmfi_set_tile_policy(tiles) == 0
    out = {}
    for name, pol in (("whole", mpg.SPLIT_OFF), ("split", mpg.SPLIT_ON)):
        assert mpg.mpgemmfi_set_split_policy(pol) == 0
        out[name] = run_gpu_gemm(dtype, A, Bt, sites, orc.T_BOUND | orc.CORRECT, addend=cin)
    Cw, hw, lw, bw = out["whole"]
    Cs, hs, ls, bs = out["split"]
    assert hw[5] == 0 and hs[5] >= 2, "the split schedule did not engage on this device"
    assert not (hs[0] & mpg.STATUS_WAIT_LIMIT) and hs[0] == hw[0]
    assert np.array_equal(Cw.view(np.uint32), Cs.view(np.uint32)) and np.array_equal(bw, bs)
    for f in lw.dtype.names:
        assert np.array_equal(lw[f], ls[f]), f
    check_gemm_against_oracle(dtype, A, Bt, sites, orc.T_BOUND | orc.CORRECT, max_fragile=2, addend=cin)


def test_addend_continues_an_accumulation_on_the_device():
    """The second half of a GEMM cut along k at a k-step boundary, with the first half's output as its addend,
    gives the uncut GEMM's words: the tensor core carries on from the accumulators it is handed."""
    dtype, M, N, K, K1 = orc.FP16, 640, 768, 1024, 384
    A, Bt = rand_operands(dtype, M, N, K, 43)
    whole, *_ = run_gpu_gemm(dtype, A, Bt, None, orc.T_NONE)
    first, *_ = run_gpu_gemm(dtype, np.ascontiguousarray(A[:, :K1]), np.ascontiguousarray(Bt[:, :K1]), None, orc.T_NONE)
    second, *_ = run_gpu_gemm(dtype, np.ascontiguousarray(A[:, K1:]), np.ascontiguousarray(Bt[:, K1:]), None, orc.T_NONE,
                              addend=first)
    assert np.array_equal(second.view(np.uint32), whole.view(np.uint32))


def test_addend_argument_errors():
    A, Bt = rand_operands(orc.BF16, 128, 128, 64, 44)
    a, b = to_dev(A, orc.BF16), to_dev(Bt, orc.BF16)
    buf = torch.zeros(2 * 128 * 128, dtype=torch.float32, device="cuda")
    st = torch.cuda.current_stream().cuda_stream
    f = torch.empty(mpg.mpgemmfi_flags_bytes(128, 128, 0) // 4, dtype=torch.int32, device="cuda")
    base = buf.data_ptr()
    call = lambda cin, d: mpg.mpgemmfi_gemm_addend(1, 128, 128, 64, a.data_ptr(), b.data_ptr(), cin, d, None, 0, 0, f.data_ptr(), st)
    assert call(None, base) == -1                       # no addend
    assert call(base + 2, base + 4 * 128 * 128) == -3   # misaligned addend
    assert call(base + 64, base) == -1                  # partial overlap
    assert call(base, base) == 0 and call(base, base + 4 * 128 * 128) == 0
    torch.cuda.synchronize()


@pytest.mark.parametrize("seed", range(16))
def test_random_shapes_tables_and_modes_with_addend(seed, policies):
    """Differential fuzz against the oracle: random shape, format, tiling, schedule, check mode, multi-bit site table
    (repeats on one element, entries the device must skip), addend scale, in place or not."""
    rng = np.random.default_rng(5000 + seed)
    dtype = int(rng.integers(0, 3))
    kt = synth.kstep(dtype)
    unit = 4 if dtype == orc.TF32 else 8
    M = int(rng.integers(1, 900)); N = int(rng.integers(1, 900)); K = unit * int(rng.integers(1, 60))
    mode = int(rng.choice([orc.T_NONE, orc.T_BOUND, orc.T_BOUND | orc.CORRECT, orc.T_RMAX | orc.CORRECT, orc.T_RFLIP | orc.CORRECT]))
    A, Bt = rand_operands(dtype, M, N, K, 6000 + seed)
    cin = rand_addend(M, N, 7000 + seed, scale=float(rng.choice([0.0, 1.0, 100.0, 1.0e4])))   # (never near BoundCheck's threshold)
    n = int(rng.integers(0, 40))
    s = site_table(dtype, M, N, K, n, 8000 + seed)
    width = np.where(s["kind"] <= orc.KIND_B, 19 if dtype == orc.TF32 else 16, 32)
    nbits = rng.choice([1, 2, 4], n)
    s["xor_mask"] = [(((1 << int(b)) - 1) << int(rng.integers(0, int(w) - int(b) + 1))) for b, w in zip(nbits, width)]
    if n >= 4:
        s[1] = s[0]; s["row"][2] = M + 5; s["kind"][3] = 7
    assert mpg.mpgemmfi_set_tile_policy([mpg.TILES_AUTO, mpg.TILES_SINGLE, mpg.TILES_PAIR][seed % 3]) == 0
    assert mpg.mpgemmfi_set_split_policy([mpg.SPLIT_AUTO, mpg.SPLIT_ON][seed % 2]) == 0
    check_gemm_against_oracle(dtype, A, Bt, s, mode, max_fragile=2, addend=cin, in_place=bool(seed & 4))
