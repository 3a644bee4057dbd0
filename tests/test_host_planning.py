"""Host-side planning logic of the library (segments, packed rows, pipeline stages), compiled as plain C++ and checked
on the CPU for the invariants the kernels and the pipelined calls rely on.  No GPU, no oracle: pure host arithmetic."""
import ctypes
import os
import subprocess

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
WARPS = 148 * 32


@pytest.fixture(scope="module")
def plan(tmp_path_factory):
    so = tmp_path_factory.mktemp("host_logic") / "libplan.so"
    subprocess.check_call(["g++", "-O1", "-std=c++17", "-Wall", "-Wextra", "-Werror", "-shared", "-fPIC", "-o", str(so),
                           os.path.join(ROOT, "tests", "host_logic", "plan_check.cpp")])
    lib = ctypes.CDLL(str(so))
    Z, U = ctypes.c_size_t, ctypes.c_uint32
    lib.plan_launch.argtypes = [ctypes.c_int, Z, U, U, U, U, ctypes.c_int, Z, Z, U, ctypes.c_void_p]
    lib.plan_stages.argtypes = [Z, Z, Z, Z, ctypes.c_void_p]
    lib.plan_stages.restype = Z
    return lib


def launch(lib, cb, sample_bytes, n_chunks, kind=0, row_slots=0, pack_max=4096, run=0, group=0, sms=148, geometry=False, fold=0):
    out = np.zeros(11, np.uint64)
    lib.plan_launch(sms, cb, row_slots, pack_max, run, group, kind, sample_bytes, n_chunks, fold, out.ctypes.data)
    return [int(x) for x in (out if geometry else out[:6])]


CHUNKS = [16, 32, 48, 64, 112, 256, 496, 512, 528, 992, 1008, 1024, 4096, 16384, 65536, 1 << 20, 4 << 20, 1 << 30]
COUNTS = [1, 2, 3, 17, 100, 591, 592, 593, 4735, 4736, 4737, 65536, 1 << 20, (1 << 24) + 1, (1 << 28) + 7]


@pytest.mark.parametrize("kind", [0, 1, 2])
def test_launch_plans_are_consistent(plan, kind):
    for cb in CHUNKS:
        blocks = cb // 16
        rows = (blocks + 2 + 31) // 32
        for n_chunks in COUNTS:
            if cb * n_chunks > 1 << 42:
                continue
            grid, wu, n_slots, run, group, p_items, rows_full, rows_last, rows_sample, total, fold = launch(
                plan, cb, cb * n_chunks, n_chunks, kind, geometry=True)
            # folded tails: only the fused passes, only chunks that end in a row of one or two counters, only where a
            # warp's range holds a chunk start or more
            foldable = kind == 0 and blocks >= 31 and (blocks + 2) % 32 in (1, 2)
            assert fold in ((0, 1) if foldable else (0,))
            if foldable:
                plain_slots = launch(plan, cb, cb * n_chunks, n_chunks, kind, fold=1)[2]
                assert fold == (1 if n_chunks >= plain_slots or (plain_slots >= 148 * 24 and 2 * n_chunks >= plain_slots) else 0)
            # row kernels: the slots cover the row space without an empty range, on at most one CTA per SM
            assert rows_full == rows - fold and rows_last == rows - fold and rows_sample == (rows - fold) * n_chunks == total
            assert 1 <= n_slots <= min(total, WARPS) and 1 <= grid <= 148 and 1 <= wu <= 32
            assert (grid - 1) * wu < n_slots <= grid * wu, "every CTA of the grid holds at least one slot"
            assert n_slots * total < 1 << 63, "slot boundaries are computed in 64 bits"
            # packed rows: whole chunks per item, no empty item, everything within 32 bits
            lanes = group
            if run:
                counters = blocks + 1
                assert 1 <= run <= counters and blocks <= 4096
                assert lanes == -(-counters // run)
                assert 1 <= p_items <= min(n_chunks, WARPS)
                assert n_chunks * lanes < (1 << 32) - 64
            else:
                assert lanes == 0 and p_items == 0
            # a few long chains stay with the row kernels
            if blocks > 31 and n_chunks * 16 < WARPS:
                assert run == 0


def test_packed_rows_can_be_switched_off_and_forced(plan):
    for cb in (16, 256, 1024, 4096):
        for n_chunks in (1, 1000, 1 << 20):
            assert launch(plan, cb, cb * n_chunks, n_chunks, pack_max=0)[3:] == [0, 0, 0]
            for run in (1, 2, 5, 300):
                got = launch(plan, cb, cb * n_chunks, n_chunks, run=run)
                assert got[3] == min(run, cb // 16 + 1) or got[3] == 0          # 0: no admissible item size
                forced = launch(plan, cb, cb * n_chunks, n_chunks, run=run, group=7)
                if forced[3]:
                    assert forced[5] == -(-n_chunks // 7)                 # items of about seven chunks
    assert launch(plan, 65552, 65552 * 100000, 100000)[3] == 0                 # 4097 blocks: above the packed limit
    assert launch(plan, 65536, 65536 * 100000, 100000, run=5)[3] == 5          # 4096 blocks: still admissible


def test_small_chunks_in_large_numbers_take_the_packed_rows(plan):
    """The planner's raison d'etre: where the row layout would idle most lanes, the packed one is chosen."""
    for cb in (16, 32, 64, 256, 1024):
        for n_chunks in (1 << 16, 1 << 20, 1 << 24):
            run = launch(plan, cb, cb * n_chunks, n_chunks)[3]
            assert run >= 1, (cb, n_chunks)
    for cb in (65536, 1 << 20, 4 << 20):                                        # the benchmark's sizes stay with the rows
        for n_chunks in (1, 64, 4096):
            assert launch(plan, cb, cb * n_chunks, n_chunks)[3] == 0
    # in between, the fixed cost of a launch decides (the row kernels end with every warp's closing product and a
    # hand-over between CTAs): measured on B200, 1 to 4 MiB of 1 or 2 KiB chunks are faster packed, 16 KiB chunks in rows
    for n in (1 << 20, 2 << 20, 4 << 20):
        assert launch(plan, 1024, n, n // 1024)[3] >= 1
        assert launch(plan, 16384, n, n // 16384)[3] == 0
    assert launch(plan, 2048, 4 << 20, 2048)[3] >= 1


def test_folded_tails_follow_the_option_and_the_shape(plan):
    """A chunk whose last row would hold one or two counters has one row less when its tail is folded; by itself the
    planner folds where there are at least as many chunks as warps at work; the option switches that off or forces it; a sample's
    short last chunk is judged by its own length."""
    for cb, rows in ((512, 2), (16384, 33), (65536, 129), (496, 2), (1 << 20, 2049)):
        for n_chunks in (100, 16384, 1 << 20):
            auto, never, always = (launch(plan, cb, cb * n_chunks, n_chunks, geometry=True, fold=f, pack_max=0) for f in (0, 1, 2))
            assert never[6] == rows and never[10] == 0
            assert always[6] == rows - 1 and always[10] == 1
            assert auto[6:] == (always[6:] if n_chunks >= never[2] or (never[2] >= 148 * 24 and 2 * n_chunks >= never[2]) else never[6:])
    assert launch(plan, 16384, 256 << 20, 16384, geometry=True)[10] == 1        # the benchmark's 256 MiB of 16 KiB chunks: folded
    assert launch(plan, 16384, 64 << 20, 4096, geometry=True)[10] == 1          # 64 MiB: 1.7 chunks per warp
    assert launch(plan, 16384, 16 << 20, 1024, geometry=True)[10] == 0          # 16 MiB of them: a chunk spans two warps
    assert launch(plan, 4 << 20, 256 << 20, 64, geometry=True)[10] == 0         # the headline shape: never
    for cb in (48, 480, 528, 16400):                       # no tail of one or two counters: nothing to fold, whatever the option says
        assert launch(plan, cb, cb * 100, 100, geometry=True, fold=2)[10] == 0
    # samples of 3 chunks of 1 KiB and a last one of 496 bytes (31 blocks: folds) / of 400 bytes (25 blocks: does not)
    got = launch(plan, 1024, 3 * 1024 + 496, 4 * 50, geometry=True, pack_max=0, fold=2)
    assert got[10] == 1 and got[6] == 2 and got[7] == 1 and got[8] == 7 and got[9] == 7 * 50
    got = launch(plan, 1024, 3 * 1024 + 400, 4 * 50, geometry=True, pack_max=0, fold=2)
    assert got[10] == 1 and got[6] == 2 and got[7] == 1
    got = launch(plan, 1040, 3 * 1040 + 496, 4 * 50, geometry=True, pack_max=0, fold=2)      # only the last chunk folds
    assert got[10] == 1 and got[6] == 3 and got[7] == 1
    for kind in (1, 2):                                    # the other passes never fold
        assert launch(plan, 16384, 16384 * 100, 100, kind=kind, geometry=True, fold=2)[10] == 0


def test_row_geometry_of_random_sample_shapes(plan):
    """Whatever the folding: a sample's last chunk never has more rows than a full one (the kernel locates a row by
    dividing by the rows of a full chunk), the rows add up, and no warp's range is empty."""
    rng = np.random.default_rng(9)
    for _ in range(3000):
        cb = 16 * int(rng.integers(1, 5000))
        cps = int(rng.integers(1, 6))
        last = 16 * int(rng.integers(1, cb // 16 + 1)) - int(rng.integers(0, 16))
        sample = (cps - 1) * cb + last
        n_samples = int(rng.choice([1, 2, 7, 300, 100000]))
        for fold in (0, 1, 2):
            grid, wu, n_slots, _, _, _, rows_full, rows_last, rows_sample, total, folded = launch(
                plan, cb, sample, cps * n_samples, geometry=True, fold=fold, pack_max=0)
            assert 1 <= rows_last <= rows_full
            assert rows_sample == (cps - 1) * rows_full + rows_last and total == rows_sample * n_samples
            assert 1 <= n_slots <= total and (grid - 1) * wu < n_slots <= grid * wu
            blocks_full, blocks_last = -(-min(cb, sample) // 16), -(-last // 16)
            for blocks, rows in ((blocks_full, rows_full), (blocks_last, rows_last)):
                plain = (blocks + 2 + 31) // 32
                folds = folded and blocks >= 31 and (blocks + 2) % 32 in (1, 2)
                assert rows == plain - (1 if folds else 0)
                assert 32 * rows >= blocks + 2 - (2 if folds else 0) > 32 * (rows - 1)      # the rows cover every counter that is theirs
            if fold == 1:
                assert not folded


def test_sample_batches_plan_on_the_sample_geometry(plan):
    # samples shorter than a chunk: the chunk that exists is the sample
    got = launch(plan, 4096, 400, 262144, geometry=True)
    assert got[3] >= 1 and got[6] == got[7] == 1 and got[9] == 262144
    # samples of several chunks: three full ones and a 16-byte one
    got = launch(plan, 1024, 3 * 1024 + 16, 4 * 50000, geometry=True, fold=1)
    assert got[6] == 3 and got[7] == 1 and got[8] == 10 and got[9] == 10 * 50000
    got = launch(plan, 1024, 3 * 1024 + 16, 4 * 50000, geometry=True)              # the 1 KiB chunks' tails folded
    assert got[10] == 1 and got[6] == 2 and got[7] == 1 and got[8] == 7 and got[9] == 7 * 50000


def test_row_slots_follow_the_size_of_the_launch(plan):
    """Small launches use few warps per SM (every warp pays a closing product), large ones more, always a whole
    number per quarter of an SM from four warps on; a forced slot count is honoured up to the number of rows and of warps."""
    used = [launch(plan, 4 << 20, n, -(-n // (4 << 20)))[1] for n in (1 << 16, 1 << 20, 4 << 20, 16 << 20, 64 << 20, 256 << 20)]
    assert used == sorted(used) and used[0] <= 2 and used[1] <= 8 and 16 <= used[-1] <= 32
    assert all(u % 4 == 0 for u in used if u >= 4)
    for want in (1, 2, 147, 148, 149, 1000, 4736, 10 ** 6):
        grid, wu, n_slots = launch(plan, 65536, 1 << 24, 256, row_slots=want)[:3]
        assert n_slots == min(want, WARPS) and (grid - 1) * wu < n_slots <= grid * wu
    assert launch(plan, 16, 16 * 5, 5, row_slots=4736)[2] == 5          # one row per chunk: never more slots than rows


def stages(lib, cb, length, unit=None, stage_bytes=0):
    out = np.zeros(96, np.uint64)
    n = lib.plan_stages(cb, stage_bytes, length, unit or cb, out.ctypes.data)
    return [int(x) for x in out[:n]]


def test_pipeline_stages_cover_the_buffer_in_whole_units(plan):
    rng = np.random.default_rng(3)
    cases = [(65536, 1), (65536, 65536), (65536, 77_070_336), (4 << 20, 256 << 20), (4 << 20, 670_000_000), (1 << 30, 5 << 30),
             (16, 4 << 20), (1 << 20, (1 << 20) * 1000 + 5)]
    cases += [(int(16 * rng.integers(1, 1 << 16)), int(rng.integers(1, 1 << 32))) for _ in range(300)]
    for cb, length in cases:
        whole = -(-length // cb) * cb                       # the pipelined calls plan on whole units and clip the last stage
        st = stages(plan, cb, whole)
        assert 1 <= len(st) <= 96 and sum(st) == whole, (cb, length)
        assert all(s % cb == 0 and s > 0 for s in st)
        if len(st) < 96:
            assert all(a >= b for a, b in zip(st, st[1:-1])), "stages shrink (the last may absorb a sliver)"
            if len(st) > 1:
                assert min(st) >= min(2 << 20, whole) // 2 or cb >= (2 << 20)


def test_pipeline_stage_override_and_sample_units(plan):
    st = stages(plan, 4096, 1 << 24, stage_bytes=300000)
    assert all(s == -(-300000 // 4096) * 4096 for s in st[:-1]) and sum(st) == 1 << 24
    st = stages(plan, 256, 301056 * 64, unit=301056)        # a batch of 64 samples: stages of whole samples
    assert sum(st) == 301056 * 64 and all(s % 301056 == 0 for s in st)
    st = stages(plan, 65536, 1 << 40, stage_bytes=65536)    # more pieces than stages: the last stage takes the rest
    assert len(st) == 96 and sum(st) == 1 << 40
