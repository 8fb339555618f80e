"""CPU-only checks of the C-ABI library: it loads, exports every declared symbol, and its host helpers work."""
import ctypes
import os
import re

import numpy as np

import paper_2311_05782_b200 as mpg

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "mpgemmfi.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mpgemmfi_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_2311_05782_b200.build import build
    lib = ctypes.CDLL(build())
    names = declared_symbols()
    assert "mpgemmfi_gemm" in names and "mpgemmfi_campaign" in names
    for n in names:
        assert hasattr(lib, n), f"{n} declared in the header but not exported"
    assert sorted(mpg.exported_symbols()) == [n for n in names if n in mpg.exported_symbols()]
    for n in names:
        assert n in mpg.exported_symbols(), f"{n} has no Python binding"


def test_host_helpers():
    assert mpg.mpgemmfi_version() >= 100
    assert [mpg.mpgemmfi_kstep(d) for d in (0, 1, 2, 3)] == [64, 64, 32, 0]
    assert mpg.mpgemmfi_flags_bitmap_offset(5) == 16 + 20
    assert mpg.mpgemmfi_flags_bytes(10, 33, 5) == 4 * (36 + 10 * 2)
    assert mpg.mpgemmfi_campaign_workspace_bytes(0, 8, 8, 8, 1000) % 256 == 0
    assert mpg.mpgemmfi_campaign_workspace_bytes(0, 8, 8, 8, 1000) >= 12000
    assert "align" in mpg.mpgemmfi_strerror(-3)
    # tuning knobs: argument checks need no device
    assert mpg.mpgemmfi_set_tile_policy(7) == -1 and mpg.mpgemmfi_set_tile_policy(mpg.TILES_AUTO) == 0
    assert mpg.mpgemmfi_set_split_policy(-1) == -1 and mpg.mpgemmfi_set_split_policy(mpg.SPLIT_AUTO) == 0
    assert mpg.mpgemmfi_set_wait_limit_ms(0) == -1 and mpg.mpgemmfi_set_wait_limit_ms(60001) == -1
    assert mpg.mpgemmfi_set_wait_limit_ms(4000) == 0
    # struct sizes the ABI promises
    assert mpg.SITE_DTYPE.itemsize == 32 and mpg.SITE_LOG_DTYPE.itemsize == 16 and mpg.RECORD_DTYPE.itemsize == 48


def test_validate_sites_rules():
    s = np.zeros(6, dtype=mpg.SITE_DTYPE)
    s["kind"] = [mpg.SITE_A, mpg.SITE_B, mpg.SITE_ACC, mpg.SITE_OUT, mpg.SITE_TERM, mpg.SITE_ACC]
    s["row"] = [3, 0, 3, 3, 3, 3]; s["col"] = [0, 4, 4, 4, 4, 4]; s["k"] = [99, 99, 64, 0, 99, 100]
    assert mpg.mpgemmfi_validate_sites(s, mpg.BF16, 8, 8, 100) == (0, -1)       # k = K is a legal ACC boundary
    s["k"][2] = 65
    assert mpg.mpgemmfi_validate_sites(s, mpg.BF16, 8, 8, 100) == (-4, 2)        # not on a k-step boundary
    s["k"][2] = 32
    assert mpg.mpgemmfi_validate_sites(s, mpg.TF32, 8, 8, 100) == (0, -1)        # TF32 k-step is 32
    s["row"][3] = 8
    assert mpg.mpgemmfi_validate_sites(s, mpg.TF32, 8, 8, 100) == (-4, 3)
    assert mpg.mpgemmfi_validate_sites(s, 5, 8, 8, 100)[0] == -2


def test_launch_slots_and_tags():
    """Slots are handed out in turn, 16 of them; a launch's tag is its counter value in 29 bits and never 0 (0 is what
    a never-used hand-over word holds), also where the counter wraps."""
    seen = [mpg.mpgemmfi_debug_launch_slot(n) for n in range(1, 40)]
    assert [s for s, _ in seen] == [n % 16 for n in range(1, 40)]
    assert [t for _, t in seen] == list(range(1, 40))
    for n in (0x20000000, 0x40000000, 0xE0000000, 0):
        slot, tag = mpg.mpgemmfi_debug_launch_slot(n)
        assert tag == 1 and slot == 0
    slot, tag = mpg.mpgemmfi_debug_launch_slot(0x3FFFFFFF)
    assert tag == 0x1FFFFFFF and slot == 15
    # two launches that share a slot never share a tag unless 2^29 launches lie between them
    assert mpg.mpgemmfi_debug_launch_slot(5)[1] != mpg.mpgemmfi_debug_launch_slot(21)[1]
    assert mpg.mpgemmfi_debug_launch_slot(5)[0] == mpg.mpgemmfi_debug_launch_slot(21)[0]


def test_tile_schedule_covers_every_k_step_once_and_orders_the_parts():
    """The schedule the kernel's tile walkers follow, enumerated on the host for many shapes and all three policies:
    every k-step of every tile is computed exactly once; a cut tile's parts are consecutive runs of k-steps, the first
    starting fresh and leaving its sums, the last loading and finishing; and the walker of part g has a LOWER index than
    the walker of part g + 1 and runs its part no later in its own order than the next walker runs the following one --
    the order of dispatch the hand-over's bounded wait relies on."""
    rng = np.random.default_rng(5)
    shapes = [(256, 64, 74), (81, 9, 74), (104, 8, 74), (168, 9, 74), (156, 8, 148), (1024, 16, 74), (100, 16, 74), (75, 64, 74),
              (73, 64, 74), (148, 3, 74), (6272, 9, 148)]
    shapes += [(int(rng.integers(1, 700)), int(rng.integers(1, 200)), int(rng.choice([74, 148, 132, 66]))) for _ in range(60)]
    engaged = 0
    for num_tiles, num_kt, walkers in shapes:
        for policy in (mpg.SPLIT_AUTO, mpg.SPLIT_OFF, mpg.SPLIT_ON):
            seg = mpg.mpgemmfi_debug_segments(num_tiles, num_kt, walkers, policy)
            cover = np.zeros((num_tiles, num_kt), dtype=np.int32)
            for w, i, t, k0, k1, part, load, save in seg:
                assert t < num_tiles and k0 < k1 <= num_kt
                cover[t, k0:k1] += 1
                assert bool(load) == (k0 > 0) and bool(save) == (k1 < num_kt)
            assert (cover == 1).all(), (num_tiles, num_kt, walkers, policy)
            # per walker: indices 0, 1, 2, ... without gaps
            for w in np.unique(seg[:, 0]):
                idx = seg[seg[:, 0] == w][:, 1]
                assert list(idx) == list(range(len(idx)))
            cut = seg[(seg[:, 6] == 1) | (seg[:, 7] == 1)]
            if policy == mpg.SPLIT_OFF:
                assert len(cut) == 0
            if len(cut):
                engaged += 1
                for t in np.unique(cut[:, 2]):
                    parts = cut[cut[:, 2] == t]
                    parts = parts[np.argsort(parts[:, 5])]
                    assert list(parts[:, 5]) == list(range(len(parts))) and 2 <= len(parts) <= 4
                    assert parts[0, 3] == 0 and parts[-1, 4] == num_kt and (parts[1:, 3] == parts[:-1, 4]).all()
                    assert (parts[:, 4] - parts[:, 3] >= 4).all()                  # no part shorter than four k-steps
                    assert (parts[1:, 0] > parts[:-1, 0]).all()                     # producer has the lower walker index
                    assert (parts[1:, 1] >= parts[:-1, 1]).all()                    # ... and runs its part no later
                # a walker that hands a part on never waits for anybody before it: its part's predecessors are lower walkers
                # that run theirs first
                first = cut[cut[:, 5] == 0]
                assert (first[:, 1] == 0).all()
    assert engaged >= 10                          # the cut schedule did engage on a fair number of the shapes
    # the benchmark's c2 (256 tiles of 64 k-steps on 74 pairs): 34 left-over tiles cut in two under AUTO
    seg = mpg.mpgemmfi_debug_segments(256, 64, 74, mpg.SPLIT_AUTO)
    assert ((seg[:, 7] == 1).sum(), (seg[:, 6] == 1).sum()) == (34, 34)
    # c3a (1024 tiles of 16 k-steps): too short to pay, left whole
    seg = mpg.mpgemmfi_debug_segments(1024, 16, 74, mpg.SPLIT_AUTO)
    assert not seg[:, 6].any() and not seg[:, 7].any()
    assert mpg.load_library().mpgemmfi_debug_segments(0, 1, 1, 0, None, 0) == -1
