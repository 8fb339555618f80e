"""GPU tests of the split schedule of the last round of tiles (mpgemmfi_set_split_policy).

A cut tile must come out bit for bit as the whole tile does (same accumulation order, sites on the same
running sums), so the first test compares the two schedules with each other on C, the site log and the
flags; the second compares the split schedule with the oracle like any other GEMM.
"""
import numpy as np
import pytest
import torch

import oracle as orc
import paper_2311_05782_b200 as mpg
import synth
from parity import check_gemm_against_oracle, run_gpu_gemm, to_dev

pytestmark = pytest.mark.gpu


def rand_operands(dtype, M, N, K, seed):
    rng = np.random.default_rng(seed)
    a = rng.standard_normal((M, K)).astype(np.float32)
    b = rng.standard_normal((N, K)).astype(np.float32)
    return synth.round_to_storage(a, dtype), synth.round_to_storage(b, dtype)


def site_table(dtype, M, N, K, n, seed):
    """All five kinds, uniformly placed; accumulator sites on every boundary, so that some fall inside the first
    run of a cut tile, some on the cut and some after it."""
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


# (tile policy, dtype, M, N, K): more tiles than tile walkers, few tiles left over for the last round
#   pair tiles are 256 x 256 on 74 CTA pairs, single tiles 128 x 256 on 148 CTAs (a B200)
CASES = [
    (mpg.TILES_PAIR, orc.BF16, 2304, 2300, 520),      # 81 tiles: 7 left over, two runs each, ragged N and K
    (mpg.TILES_PAIR, orc.FP16, 3328, 2048, 512),      # 104 tiles: 30 left over, two runs
    (mpg.TILES_PAIR, orc.TF32, 3584, 3072, 264),      # 168 tiles: 20 left over after two rounds, three runs
    (mpg.TILES_SINGLE, orc.FP16, 1500, 3328, 512),    # 156 tiles of 128 x 256: 8 left over, ragged M
]


@pytest.fixture
def policies():
    yield
    mpg.mpgemmfi_set_tile_policy(mpg.TILES_AUTO)
    mpg.mpgemmfi_set_split_policy(mpg.SPLIT_AUTO)


@pytest.mark.parametrize("case", CASES)
@pytest.mark.parametrize("mode", [orc.T_NONE, orc.T_BOUND | orc.CORRECT, orc.T_RFLIP | orc.CORRECT])
def test_split_schedule_is_bit_identical(case, mode, policies):
    tiles, dtype, M, N, K = case
    A, Bt = rand_operands(dtype, M, N, K, 77)
    sites = site_table(dtype, M, N, K, 600, 78)
    assert mpg.mpgemmfi_set_tile_policy(tiles) == 0
    out = {}
    for name, pol in (("whole", mpg.SPLIT_OFF), ("split", mpg.SPLIT_ON)):
        assert mpg.mpgemmfi_set_split_policy(pol) == 0
        out[name] = run_gpu_gemm(dtype, A, Bt, sites, mode)
    Cw, hw, lw, bw = out["whole"]
    Cs, hs, ls, bs = out["split"]
    assert hw[5] == 0 and hs[5] >= 2, "the split schedule did not engage on this device"
    assert hs[0] == hw[0] and not (hs[0] & mpg.STATUS_WAIT_LIMIT)
    same = Cw.view(np.uint32) == Cs.view(np.uint32)
    assert same.all(), f"{(~same).sum()} elements differ, first at {np.argwhere(~same)[:5].tolist()}"
    assert np.array_equal(hw[1:5], hs[1:5])
    for f in lw.dtype.names:
        assert np.array_equal(lw[f], ls[f]), f
    assert np.array_equal(bw, bs)


def test_split_schedule_without_flags_buffer(policies):
    """The plain product (no sites, no check, no flags buffer) under both schedules, twice under the split one."""
    dtype, M, N, K = orc.BF16, 2304, 2304, 1024
    A, Bt = rand_operands(dtype, M, N, K, 5)
    a, b = to_dev(A, dtype), to_dev(Bt, dtype)
    st = torch.cuda.current_stream().cuda_stream
    mpg.mpgemmfi_set_tile_policy(mpg.TILES_PAIR)
    res = []
    for pol in (mpg.SPLIT_OFF, mpg.SPLIT_ON, mpg.SPLIT_ON):
        mpg.mpgemmfi_set_split_policy(pol)
        c = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
        assert mpg.mpgemmfi_gemm(dtype, M, N, K, a.data_ptr(), b.data_ptr(), c.data_ptr(), None, 0, 0, None, st) == 0
        torch.cuda.synchronize()
        res.append(c.cpu().numpy().view(np.uint32))
    assert np.array_equal(res[0], res[1]) and np.array_equal(res[0], res[2])


@pytest.mark.parametrize("case", CASES[:2] + CASES[3:])
def test_split_schedule_against_oracle(case, policies):
    tiles, dtype, M, N, K = case
    A, Bt = rand_operands(dtype, M, N, K, 91)
    sites = site_table(dtype, M, N, K, 300, 92)
    mpg.mpgemmfi_set_tile_policy(tiles)
    mpg.mpgemmfi_set_split_policy(mpg.SPLIT_ON)
    check_gemm_against_oracle(dtype, A, Bt, sites, orc.T_BOUND | orc.CORRECT, max_fragile=2)


def test_split_policy_argument():
    assert mpg.mpgemmfi_set_split_policy(3) == -1
    assert mpg.mpgemmfi_set_split_policy(mpg.SPLIT_AUTO) == 0


def test_two_streams_at_once(policies):
    """Two split-schedule GEMMs with flags buffers in flight on two streams (each launch has its own hand-over slot
    and tag): every result equals the one of the same GEMM run alone."""
    dtype = orc.BF16
    shapes = [(2304, 2304, 1024), (3328, 2048, 512)]
    mpg.mpgemmfi_set_tile_policy(mpg.TILES_PAIR)
    mpg.mpgemmfi_set_split_policy(mpg.SPLIT_ON)
    ops, alone = [], []
    for i, (M, N, K) in enumerate(shapes):
        A, Bt = rand_operands(dtype, M, N, K, 40 + i)
        sites = site_table(dtype, M, N, K, 64, 50 + i)
        a, b = to_dev(A, dtype), to_dev(Bt, dtype)
        sd = torch.from_numpy(sites.view(np.int32).reshape(-1, 8)).cuda()
        ops.append((M, N, K, a, b, sd))
        Cg, flags = mpg.gemm(dtype, a, b, sites, orc.T_BOUND | orc.CORRECT)
        torch.cuda.synchronize()
        alone.append((Cg.cpu().numpy().view(np.uint32), flags.cpu().numpy()))
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    outs = []
    for (M, N, K, a, b, sd) in ops:
        c = torch.empty((M, N), dtype=torch.float32, device="cuda")
        f = torch.empty(mpg.mpgemmfi_flags_bytes(M, N, 64) // 4, dtype=torch.int32, device="cuda")
        outs.append((c, f))
    torch.cuda.synchronize()
    for rep in range(6):
        for k, (M, N, K, a, b, sd) in enumerate(ops):
            c, f = outs[k]
            rc = mpg.mpgemmfi_gemm(dtype, M, N, K, a.data_ptr(), b.data_ptr(), c.data_ptr(), sd.data_ptr(), 64,
                                   orc.T_BOUND | orc.CORRECT, f.data_ptr(), streams[k].cuda_stream)
            assert rc == 0
    torch.cuda.synchronize()
    for k in range(2):
        c, f = outs[k]
        fg = f.cpu().numpy()
        assert not (int(fg[0]) & mpg.STATUS_WAIT_LIMIT)
        assert np.array_equal(c.cpu().numpy().view(np.uint32), alone[k][0])
        assert np.array_equal(fg, alone[k][1])


@pytest.mark.parametrize("seed", range(8))
def test_random_shapes_under_split_schedule(seed, policies):
    """Differential fuzz against the oracle with the split schedule forced on: random shape (enough tiles for a
    left-over round under either tiling), format, check mode and site table (all kinds, a repeat, invalid entries)."""
    rng = np.random.default_rng(7000 + seed)
    dtype = int(rng.integers(0, 3))
    kt = synth.kstep(dtype)
    unit = 4 if dtype == orc.TF32 else 8
    M = int(rng.integers(2100, 3700)); N = int(rng.integers(2100, 3700)); K = unit * int(rng.integers(40, 80))
    N -= N % 4                                    # the split schedule needs 16-byte rows of C
    mode = int(rng.choice([orc.T_NONE, orc.T_BOUND, orc.T_BOUND | orc.CORRECT, orc.T_RMAX | orc.CORRECT, orc.T_RFLIP | orc.CORRECT]))
    A, Bt = rand_operands(dtype, M, N, K, 7100 + seed)
    s = site_table(dtype, M, N, K, 48, 7200 + seed)
    s[1] = s[0]; s["row"][2] = M + 5; s["kind"][3] = 7
    mpg.mpgemmfi_set_tile_policy([mpg.TILES_PAIR, mpg.TILES_SINGLE][seed % 2])
    mpg.mpgemmfi_set_split_policy(mpg.SPLIT_ON)
    check_gemm_against_oracle(dtype, A, Bt, s, mode, max_fragile=2)


def test_more_launches_in_flight_than_slots(policies):
    """24 split-schedule GEMMs with flags buffers queued on 4 streams before any has finished: more than the 16
    hand-over slots. A launch that gets a slot for the second time waits (in stream order, on the device) for the
    launch that held it before, so every result equals the one of the same GEMM run alone."""
    dtype = orc.BF16
    M, N, K = 2304, 2304, 2048
    mpg.mpgemmfi_set_tile_policy(mpg.TILES_PAIR)
    mpg.mpgemmfi_set_split_policy(mpg.SPLIT_ON)
    A, Bt = rand_operands(dtype, M, N, K, 60)
    sites = site_table(dtype, M, N, K, 32, 61)
    a, b = to_dev(A, dtype), to_dev(Bt, dtype)
    sd = torch.from_numpy(sites.view(np.int32).reshape(-1, 8)).cuda()
    Cg, flags = mpg.gemm(dtype, a, b, sites, orc.T_BOUND | orc.CORRECT)
    torch.cuda.synchronize()
    want_c, want_f = Cg.cpu().numpy().view(np.uint32), flags.cpu().numpy()
    assert want_f.view(np.uint32)[5] >= 2                 # the last round is cut: the hand-over words are in use
    n_launch = 24
    streams = [torch.cuda.Stream() for _ in range(4)]
    outs = [(torch.empty((M, N), dtype=torch.float32, device="cuda"),
             torch.empty(mpg.mpgemmfi_flags_bytes(M, N, 32) // 4, dtype=torch.int32, device="cuda")) for _ in range(n_launch)]
    torch.cuda.synchronize()
    for i, (c, f) in enumerate(outs):
        rc = mpg.mpgemmfi_gemm(dtype, M, N, K, a.data_ptr(), b.data_ptr(), c.data_ptr(), sd.data_ptr(), 32,
                               orc.T_BOUND | orc.CORRECT, f.data_ptr(), streams[i % 4].cuda_stream)
        assert rc == 0
    torch.cuda.synchronize()
    for i, (c, f) in enumerate(outs):
        fg = f.cpu().numpy()
        assert not (int(fg[0]) & mpg.STATUS_WAIT_LIMIT), i
        assert np.array_equal(fg, want_f), i
        assert np.array_equal(c.cpu().numpy().view(np.uint32), want_c), i


def test_a_wait_that_runs_out_ends_the_launch_with_a_status(policies):
    """The give-up path of the bounded waits, made to run without any fault: with the test hook on, the CTAs that
    continue a cut tile wait for a hand-over tag that nobody writes; with the limit set to a few milliseconds the wait
    runs out, every warp of the CTA (pair) leaves its loop, tensor memory is released, the kernel returns, and the
    header says WAIT_LIMIT. The device stays usable: the same GEMM queued next, with the hook off, gives bit for bit
    what it gave before."""
    dtype = orc.BF16
    M, N, K = 2560, 2560, 1024                            # 100 tiles of 256 x 256 on 74 pairs: 26 left over, cut in two
    mpg.mpgemmfi_set_tile_policy(mpg.TILES_PAIR)
    mpg.mpgemmfi_set_split_policy(mpg.SPLIT_ON)
    A, Bt = rand_operands(dtype, M, N, K, 70)
    sites = site_table(dtype, M, N, K, 16, 71)
    a, b = to_dev(A, dtype), to_dev(Bt, dtype)
    C0, f0 = mpg.gemm(dtype, a, b, sites, orc.T_BOUND)
    torch.cuda.synchronize()
    want_c, want_f = C0.cpu().numpy().view(np.uint32), f0.cpu().numpy().view(np.uint32)
    assert want_f[5] >= 2 and not (want_f[0] & mpg.STATUS_WAIT_LIMIT)
    try:
        assert mpg.mpgemmfi_set_wait_limit_ms(3) == 0
        assert mpg.mpgemmfi_debug_break_handover(1) == 0
        t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
        t0.record()
        C1, f1 = mpg.gemm(dtype, a, b, sites, orc.T_BOUND)
        t1.record()
        torch.cuda.synchronize()
    finally:
        mpg.mpgemmfi_debug_break_handover(0)
        mpg.mpgemmfi_set_wait_limit_ms(4000)
    got = f1.cpu().numpy().view(np.uint32)
    assert got[0] & mpg.STATUS_WAIT_LIMIT, "the launch did not report that a wait ran out"
    assert t0.elapsed_time(t1) < 3000.0                  # it gave up after milliseconds (plus the drain), not seconds
    # the whole tiles of that launch did not depend on the hand-over and are as before
    assert np.array_equal(C1.cpu().numpy().view(np.uint32)[:256, :256], want_c[:256, :256])
    # the next ordinary launch: everything as in the first one
    C2, f2 = mpg.gemm(dtype, a, b, sites, orc.T_BOUND)
    torch.cuda.synchronize()
    assert np.array_equal(f2.cpu().numpy().view(np.uint32), want_f)
    assert np.array_equal(C2.cpu().numpy().view(np.uint32), want_c)
