"""The CUDA library's per-lane device code, compiled as plain C++ and run lane by lane on the host, against the
oracle (tests/device_on_host/emulate.cpp explains what is and is not emulated).  This is test infrastructure:
it lets the CPU-only run check the kernels' arithmetic; the GPU tests check the real thing."""
import ctypes
import os
import subprocess

import numpy as np
import pytest

import oracle

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
DEC, ENC, CTR, VERIFY, PADGEN, PADDEC = range(6)


@pytest.fixture(scope="module")
def emu(tmp_path_factory):
    so = tmp_path_factory.mktemp("device_on_host") / "libemulate.so"
    subprocess.check_call(["g++", "-O2", "-std=c++17", "-shared", "-fPIC", "-o", str(so),
                           os.path.join(ROOT, "tests", "device_on_host", "emulate.cpp")])
    lib = ctypes.CDLL(str(so))
    V, Z, U = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_uint32
    lib.emu_pass.argtypes = [ctypes.c_int, V, V, Z, V, Z, V, V, V, V, V, V, U, U, U, U, Z, V, U]
    lib.emu_pass.restype = ctypes.c_int
    for name in ("emu_gf128_mul_device", "emu_gf128_mul_keysetup"):
        getattr(lib, name).argtypes = [ctypes.c_char_p] * 3
    lib.emu_keysetup.argtypes = [ctypes.c_char_p, V, V]
    lib.emu_packed.argtypes = [ctypes.c_int, V, V, Z, V, Z, V, V, V, V, U, U, U, U, Z, V]
    lib.emu_packed.restype = ctypes.c_int
    return lib


def run(lib, mode, key, iv, cb, data, n, pad=None, mask=None, tags=None, seg=8, first=0, aad=0, sample_bytes=0, ivs=None, sms=3, fold=0):
    """fold = the tail-folding option (0 automatic, 1 never, 2 wherever a chunk allows); seg = rows per warp (0: the planner's own choice) on an emulated GPU of `sms` SMs: few SMs, so that chunks are
    shared between warps of one CTA and between CTAs even in small cases."""
    K = (n + cb - 1) // cb if not sample_bytes else (n // sample_bytes) * ((sample_bytes + cb - 1) // cb)
    k = np.frombuffer(key, np.uint8).copy()
    v = np.frombuffer(iv, np.uint8).copy()
    src = np.ascontiguousarray(data, np.uint8) if data is not None else np.zeros(n, np.uint8)
    out = np.full(n + 64, 0xA5, np.uint8)
    tin = np.ascontiguousarray(tags, np.uint8) if tags is not None else np.zeros((K, 16), np.uint8)
    tout = np.zeros((K, 16), np.uint8)
    ok = np.full(K, 7, np.uint32)
    pad_a = np.ascontiguousarray(pad, np.uint8) if pad is not None else np.zeros(n, np.uint8)
    mask_a = np.ascontiguousarray(mask, np.uint8) if mask is not None else np.zeros((K, 16), np.uint8)
    if mode == VERIFY:
        out[:n] = src                                   # the pass does not store; keep the guard check meaningful
    rc = lib.emu_pass(mode, k.ctypes.data, v.ctypes.data, cb, src.ctypes.data, n, out.ctypes.data, pad_a.ctypes.data,
                      mask_a.ctypes.data, tin.ctypes.data, tout.ctypes.data, ok.ctypes.data, seg, sms, first, aad, sample_bytes,
                      ivs.ctypes.data if ivs is not None else None, fold)
    assert rc == 0, f"emulation reports inconsistency {rc}"
    assert (out[n:] == 0xA5).all()
    return out[:n], tout, ok, mask_a


def test_key_setup_matches_oracle(emu):
    rng = np.random.default_rng(1)
    for _ in range(8):
        key = rng.bytes(32)
        rk = np.zeros(240, np.uint8)
        h = np.zeros(16, np.uint8)
        emu.emu_keysetup(key, rk.ctypes.data, h.ctypes.data)
        assert rk.tobytes() == oracle.aes256_key_expand(key)
        assert h.tobytes() == oracle.hash_subkey(key)


def test_both_gf128_products_match_oracle(emu):
    rng = np.random.default_rng(2)
    cases = [(rng.bytes(16), rng.bytes(16)) for _ in range(2000)] + [(bytes([0xFF] * 16),) * 2]
    for i in range(0, 128, 3):
        for j in (0, 1, 31, 32, 33, 63, 64, 65, 96, 127):
            x, y = bytearray(16), bytearray(16)
            x[i // 8] |= 1 << (7 - i % 8)
            y[j // 8] |= 1 << (7 - j % 8)
            cases.append((bytes(x), bytes(y)))
    for a, b in cases:
        ref = oracle.gf128_mul(a, b)
        for fn in (emu.emu_gf128_mul_device, emu.emu_gf128_mul_keysetup):
            o = ctypes.create_string_buffer(16)
            fn(a, b, o)
            assert o.raw == ref


SHAPES = [(1, 16, 8), (16, 16, 8), (15, 64, 2), (17, 64, 4), (33, 32, 8), (480, 480, 8), (512, 512, 1), (513, 1024, 8),
          (1000, 256, 2), (4096, 1024, 8), (5000, 2048, 4), (70000, 16384, 8), (70001, 65536, 16), (200000, 65536, 24),
          (100, 65536, 8), (300000, 100000 // 16 * 16, 3), (300000, 100000 // 16 * 16, 0), (150000, 496, 1), (150000, 1008, 5),
          (99999, 16, 7), (400000, 4096, 13)]


@pytest.mark.parametrize("n,cb,seg", SHAPES)
@pytest.mark.parametrize("aad", [0, 16])
def test_fused_and_split_passes_match_oracle(emu, n, cb, seg, aad):
    rng = np.random.default_rng(n + cb + aad)
    key, iv = rng.bytes(32), rng.bytes(8) + bytes([0xFF, 0xFF, 0xFF, 0xFE])
    p = np.frombuffer(rng.bytes(n), np.uint8)
    if aad:
        c_ref, t_ref = oracle.mc_encrypt_framed(key, iv, cb, aad, p, 4)
    else:
        c_ref, t_ref = oracle.mc_encrypt(key, iv, cb, p, 4)
    K = t_ref.shape[0]
    c, t, _, _ = run(emu, ENC, key, iv, cb, p, n, seg=seg, aad=aad)
    assert np.array_equal(c, c_ref) and np.array_equal(t, t_ref)

    bad_c, bad_t = c_ref.copy(), t_ref.copy()
    bad_c[n // 2] ^= 0x10
    if K > 1:
        bad_t[K - 1, 3] ^= 4
    if aad:
        p_ref, ok_ref = oracle.mc_decrypt_framed(key, iv, cb, aad, bad_c, bad_t, 4)
    else:
        p_ref, ok_ref = oracle.mc_decrypt(key, iv, cb, bad_c, bad_t, 4)
    out, _, ok, _ = run(emu, DEC, key, iv, cb, bad_c, n, tags=bad_t, seg=seg, aad=aad)
    assert np.array_equal(out, p_ref) and np.array_equal(ok, ok_ref)

    out, _, _, _ = run(emu, CTR, key, iv, cb, bad_c, n, seg=seg, aad=aad)
    assert np.array_equal(out, p_ref)
    _, _, ok, _ = run(emu, VERIFY, key, iv, cb, bad_c, n, tags=bad_t, seg=seg, aad=aad)
    assert np.array_equal(ok, ok_ref)

    pad, _, _, mask = run(emu, PADGEN, key, iv, cb, None, n, seg=seg, aad=aad)
    assert np.array_equal(pad, oracle.mc_encrypt(key, iv, cb, np.zeros(n, np.uint8), 4)[0])
    out, _, ok, _ = run(emu, PADDEC, key, iv, cb, bad_c, n, pad=pad, mask=mask, tags=bad_t, seg=seg, aad=aad)
    assert np.array_equal(out, p_ref) and np.array_equal(ok, ok_ref)


FOLD_SHAPES = [  # n, chunk bytes, rows per warp (0: planner), emulated SMs
    (512 * 40, 512, 8, 3),                  # 32 blocks: two counters behind the last row; 40 chunks, several passes of ten per warp
    (512 * 40 - 5, 512, 1, 3),              # the folded block is the buffer's partial last block
    (496 * 25, 496, 3, 2),                  # 31 blocks: one counter behind the last row, one row per chunk
    (1008 * 9 + 16 * 31, 1008, 2, 3),       # 63 blocks; the short last chunk (31 blocks) folds too
    (1024 * 30 + 400, 1024, 5, 3),          # the short last chunk (25 blocks) does not fold
    (16384 * 12 - 1, 16384, 8, 3),          # 1024 blocks (the benchmark's small chunk), chunks shared between warps
    (16384 * 12, 16384, 40, 2),             # a warp holds whole chunks and pieces
    (65536 * 3 + 4096, 65536, 0, 3),        # planner's own slots
    (2 * 1048576 + 512, 1048576, 0, 4),     # 2049 rows: folded only when forced
]


@pytest.mark.parametrize("n,cb,seg,sms", FOLD_SHAPES)
@pytest.mark.parametrize("aad", [0, 7])
@pytest.mark.parametrize("fold", [0, 1, 2])
def test_folded_tails_match_oracle(emu, n, cb, seg, sms, aad, fold):
    """Chunks that end in a row of one or two counters: with the tail folded (the kernel's prework pass takes those
    counters and every tag mask, ten chunks at a time) and without, the same bytes, tags and verdicts as the oracle."""
    rng = np.random.default_rng(n + cb + aad)
    key, iv = rng.bytes(32), rng.bytes(8) + bytes([0xFF, 0xFF, 0xFF, 0xFD])
    p = np.frombuffer(rng.bytes(n), np.uint8)
    c_ref, t_ref = oracle.mc_encrypt_framed(key, iv, cb, aad, p, 4) if aad else oracle.mc_encrypt(key, iv, cb, p, 4)
    K = t_ref.shape[0]
    c, t, _, _ = run(emu, ENC, key, iv, cb, p, n, seg=seg, aad=aad, sms=sms, fold=fold)
    assert np.array_equal(c, c_ref) and np.array_equal(t, t_ref)
    bad_c, bad_t = c_ref.copy(), t_ref.copy()
    bad_c[min(n - 1, cb - 3)] ^= 0x40                    # inside the folded tail of chunk 0 (its last block)
    if K > 2:
        bad_t[K - 2, 15] ^= 1
    p_ref, ok_ref = (oracle.mc_decrypt_framed(key, iv, cb, aad, bad_c, bad_t, 4) if aad else
                     oracle.mc_decrypt(key, iv, cb, bad_c, bad_t, 4))
    assert ok_ref[0] == 0 and ok_ref.sum() == K - (2 if K > 2 else 1)
    out, _, ok, _ = run(emu, DEC, key, iv, cb, bad_c, n, tags=bad_t, seg=seg, aad=aad, sms=sms, fold=fold)
    assert np.array_equal(out, p_ref) and np.array_equal(ok, ok_ref)


def test_a_stage_that_starts_at_a_later_chunk(emu):
    """Pipelined calls launch a pass per stage: IV index and serial number continue from the stage's first chunk."""
    rng = np.random.default_rng(77)
    key, iv = rng.bytes(32), rng.bytes(12)
    cb, n, first, aad = 1024, 1024 * 7 + 100, 5, 3
    p = np.frombuffer(rng.bytes(cb * first + n), np.uint8)
    c_ref, t_ref = oracle.mc_encrypt_framed(key, iv, cb, aad, p, 4)
    c, t, _, _ = run(emu, ENC, key, iv, cb, p[cb * first:], n, seg=8, first=first, aad=aad)
    assert np.array_equal(c, c_ref[cb * first:]) and np.array_equal(t, t_ref[first:])


@pytest.mark.parametrize("sample_bytes,cb,n_samples,aad,seg", [(64, 16, 3, 0, 8), (1024, 1024, 5, 0, 2), (1040, 1024, 4, 16, 8),
                                                              (3 * 4096 + 160, 4096, 6, 4, 4), (301056, 65536, 2, 16, 8),
                                                              (2 * 1024 + 496, 1024, 23, 5, 3), (1040 + 512, 1040, 9, 0, 1)])
@pytest.mark.parametrize("fold", [1, 2])
def test_batch_of_samples_each_under_its_own_iv(emu, sample_bytes, cb, n_samples, aad, seg, fold):
    """Paper Section 4.2: every sample is its own multi-chain message; a batch is many of them in one launch."""
    rng = np.random.default_rng(sample_bytes + n_samples)
    key = rng.bytes(32)
    ivs = np.frombuffer(rng.bytes(12 * n_samples), np.uint8).copy()
    n = sample_bytes * n_samples
    p = np.frombuffer(rng.bytes(n), np.uint8)
    cs, ts = [], []
    for s in range(n_samples):
        part = p[s * sample_bytes:(s + 1) * sample_bytes]
        iv = ivs[12 * s:12 * s + 12].tobytes()
        c1, t1 = oracle.mc_encrypt_framed(key, iv, cb, aad, part, 2) if aad else oracle.mc_encrypt(key, iv, cb, part, 2)
        cs.append(c1)
        ts.append(t1)
    c_ref, t_ref = np.concatenate(cs), np.concatenate(ts)
    c, t, _, _ = run(emu, ENC, key, bytes(12), cb, p, n, seg=seg, aad=aad, sample_bytes=sample_bytes, ivs=ivs, fold=fold)
    assert np.array_equal(c, c_ref) and np.array_equal(t, t_ref)
    bad_t = t_ref.copy()
    bad_t[len(bad_t) // 2, 0] ^= 1
    out, _, ok, _ = run(emu, DEC, key, bytes(12), cb, c_ref, n, tags=bad_t, seg=seg, aad=aad, sample_bytes=sample_bytes, ivs=ivs, fold=fold)
    exp = np.ones(len(bad_t), np.uint32)
    exp[len(bad_t) // 2] = 0
    assert np.array_equal(out, p) and np.array_equal(ok, exp)


def run_packed(lib, mode, key, iv, cb, data, n, tags=None, group=1, run_len=1, first=0, aad=0, sample_bytes=0, ivs=None):
    K = (n + cb - 1) // cb if not sample_bytes else (n // sample_bytes) * ((sample_bytes + cb - 1) // cb)
    k = np.frombuffer(key, np.uint8).copy()
    v = np.frombuffer(iv, np.uint8).copy()
    src = np.ascontiguousarray(data, np.uint8)
    out = np.full(n + 64, 0xA5, np.uint8)
    tin = np.ascontiguousarray(tags, np.uint8) if tags is not None else np.zeros((K, 16), np.uint8)
    tout = np.zeros((K, 16), np.uint8)
    ok = np.full(K, 7, np.uint32)
    rc = lib.emu_packed(mode, k.ctypes.data, v.ctypes.data, cb, src.ctypes.data, n, out.ctypes.data, tin.ctypes.data,
                        tout.ctypes.data, ok.ctypes.data, group, run_len, first, aad, sample_bytes,
                        ivs.ctypes.data if ivs is not None else None)
    assert rc == 0 and (out[n:] == 0xA5).all()
    return out[:n], tout, ok


def run_packed_verify(lib, key, iv, cb, cipher, n, tags, group, run_len, aad):
    """Verify-only pass: `out` is never written, so hand it the ciphertext's own buffer with guard bytes behind it."""
    K = (n + cb - 1) // cb
    buf = np.full(n + 64, 0xA5, np.uint8)
    buf[:n] = cipher
    k = np.frombuffer(key, np.uint8).copy()
    v = np.frombuffer(iv, np.uint8).copy()
    tin = np.ascontiguousarray(tags, np.uint8)
    tout = np.zeros((K, 16), np.uint8)
    ok = np.full(K, 7, np.uint32)
    rc = lib.emu_packed(VERIFY, k.ctypes.data, v.ctypes.data, cb, buf.ctypes.data, n, buf.ctypes.data, tin.ctypes.data,
                        tout.ctypes.data, ok.ctypes.data, group, run_len, 0, aad, 0, None)
    assert rc == 0 and (buf[n:] == 0xA5).all() and np.array_equal(buf[:n], cipher)
    return buf[:n], tout, ok


PACKED_SHAPES = [(1, 16, 1), (16, 16, 1), (16 * 100, 16, 7), (16 * 100 + 5, 16, 300), (32 * 37 + 17, 32, 5), (48 * 50, 48, 4),
                 (112 * 9 + 1, 112, 2), (240 * 33, 240, 3), (496 * 5 + 495, 496, 2), (512 * 6 + 16, 512, 1), (528 * 4, 528, 3),
                 (1024 * 5 + 1000, 1024, 2), (2048 * 3 + 31, 2048, 1), (700, 4096, 1),
                 (4096 * 3 + 100, 4096, 2), (65536 + 17, 16384, 1)]        # runs that cross a 256-counter group


@pytest.mark.parametrize("n,cb,group", PACKED_SHAPES)
@pytest.mark.parametrize("aad,run_len", [(0, 1), (5, 1), (0, 2), (5, 4), (0, 8), (0, 3), (5, 32), (0, 300)])
def test_packed_rows_match_oracle(emu, n, cb, group, aad, run_len):
    """Small chunks, several to a row: ciphertext, tags, plaintext and verdicts (with tampering) equal the oracle's."""
    rng = np.random.default_rng(n * 31 + cb + aad)
    key, iv = rng.bytes(32), rng.bytes(8) + bytes([0xFF, 0xFF, 0xFF, 0xFD])          # the chunk index wraps the IV's counter
    p = np.frombuffer(rng.bytes(n), np.uint8)
    enc = (lambda q: oracle.mc_encrypt_framed(key, iv, cb, aad, q, 4)) if aad else (lambda q: oracle.mc_encrypt(key, iv, cb, q, 4))
    c_ref, t_ref = enc(p)
    K = t_ref.shape[0]
    c, t, _ = run_packed(emu, ENC, key, iv, cb, p, n, group=group, run_len=run_len, aad=aad)
    assert np.array_equal(c, c_ref) and np.array_equal(t, t_ref)
    bad_c, bad_t = c_ref.copy(), t_ref.copy()
    bad_c[n // 2] ^= 0x10
    if K > 1:
        bad_t[K - 1, 3] ^= 4
    if K > 4:
        bad_t[1, 15] ^= 0x80
    if aad:
        p_ref, ok_ref = oracle.mc_decrypt_framed(key, iv, cb, aad, bad_c, bad_t, 4)
    else:
        p_ref, ok_ref = oracle.mc_decrypt(key, iv, cb, bad_c, bad_t, 4)
    assert 0 < int(ok_ref.sum()) < K or K <= 2
    out, _, ok = run_packed(emu, DEC, key, iv, cb, bad_c, n, tags=bad_t, group=group, run_len=run_len, aad=aad)
    assert np.array_equal(out, p_ref) and np.array_equal(ok, ok_ref)
    out, _, _ = run_packed(emu, CTR, key, iv, cb, bad_c, n, group=group, run_len=run_len, aad=aad)
    assert np.array_equal(out, p_ref)
    keep = bad_c.copy()
    _, _, ok = run_packed_verify(emu, key, iv, cb, keep, n, bad_t, group, run_len, aad)
    assert np.array_equal(ok, ok_ref)


@pytest.mark.parametrize("cb,n_chunks,run_len,aad", [(16, 70, 2, 0), (16, 70, 9, 3), (48, 33, 4, 0), (112, 40, 8, 5), (1024, 5, 65, 0)])
def test_packed_rows_on_a_stage_that_starts_at_a_later_chunk(emu, cb, n_chunks, run_len, aad):
    """One lane per chunk, launched from chunk 1 and from chunk 2 of a buffer (pipelined calls do that): the IV index
    and the serial number continue, and both closing variants of the whole-chunk layout are exercised (the emulation
    picks the general product for odd starts)."""
    rng = np.random.default_rng(cb + n_chunks)
    key, iv = rng.bytes(32), rng.bytes(12)
    for first in (1, 2):
        n = cb * n_chunks - 5
        p = np.frombuffer(rng.bytes(cb * first + n), np.uint8)
        c_ref, t_ref = (oracle.mc_encrypt_framed(key, iv, cb, aad, p, 4) if aad else oracle.mc_encrypt(key, iv, cb, p, 4))
        c, t, _ = run_packed(emu, ENC, key, iv, cb, p[cb * first:], n, group=3, run_len=run_len, first=first, aad=aad)
        assert np.array_equal(c, c_ref[cb * first:]) and np.array_equal(t, t_ref[first:])
        bad_t = t_ref[first:].copy()
        bad_t[n_chunks // 2, 5] ^= 1
        out, _, ok = run_packed(emu, DEC, key, iv, cb, c_ref[cb * first:], n, tags=bad_t, group=3, run_len=run_len, first=first, aad=aad)
        expect = np.ones(n_chunks, np.uint32)
        expect[n_chunks // 2] = 0
        assert np.array_equal(out, p[cb * first:]) and np.array_equal(ok, expect)


@pytest.mark.parametrize("run_len", [1, 4, 7])
@pytest.mark.parametrize("sample_bytes,cb,n_samples,aad,group", [(16, 16, 40, 0, 3), (48, 16, 9, 0, 4), (400, 400, 11, 0, 2),
                                                                (400, 112, 7, 16, 5), (1040, 1024, 4, 16, 1), (208, 64, 6, 3, 100)])
def test_packed_rows_over_a_batch_of_samples(emu, sample_bytes, cb, n_samples, aad, group, run_len):
    rng = np.random.default_rng(sample_bytes * 7 + n_samples)
    key = rng.bytes(32)
    ivs = np.frombuffer(rng.bytes(12 * n_samples), np.uint8).copy()
    n = sample_bytes * n_samples
    p = np.frombuffer(rng.bytes(n), np.uint8)
    c_ref, t_ref = [], []
    for s_ in range(n_samples):
        q = p[s_ * sample_bytes:(s_ + 1) * sample_bytes]
        iv_s = ivs[12 * s_:12 * s_ + 12].tobytes()
        c_s, t_s = (oracle.mc_encrypt_framed(key, iv_s, cb, aad, q, 2) if aad else oracle.mc_encrypt(key, iv_s, cb, q, 2))
        c_ref.append(c_s)
        t_ref.append(t_s)
    c_ref, t_ref = np.concatenate(c_ref), np.concatenate(t_ref)
    c, t, _ = run_packed(emu, ENC, key, bytes(12), cb, p, n, group=group, run_len=run_len, aad=aad, sample_bytes=sample_bytes, ivs=ivs)
    assert np.array_equal(c, c_ref) and np.array_equal(t, t_ref)
    bad_t = t_ref.copy()
    bad_t[len(bad_t) // 2, 0] ^= 1
    out, _, ok = run_packed(emu, DEC, key, bytes(12), cb, c_ref, n, tags=bad_t, group=group, run_len=run_len, aad=aad, sample_bytes=sample_bytes, ivs=ivs)
    expect = np.ones(len(bad_t), np.uint32)
    expect[len(bad_t) // 2] = 0
    assert np.array_equal(out, p) and np.array_equal(ok, expect)


def test_index_arithmetic_under_address_and_ub_sanitizers(tmp_path):
    """The per-lane code again, as a stand-alone program built with -fsanitize=address,undefined over heap buffers of
    exactly the sizes the C ABI asks for: 400+ shapes x 6 pass modes must run clean, and the same program given an
    output buffer one byte short must be stopped by the sanitizer."""
    exe = tmp_path / "emulate_sanitized"
    src = os.path.join(ROOT, "tests", "device_on_host", "emulate.cpp")
    subprocess.check_call(["g++", "-O1", "-g", "-std=c++17", "-fsanitize=address,undefined", "-fno-sanitize-recover=all",
                           "-DEMU_SANITIZER_MAIN", "-o", str(exe), src])
    ok = subprocess.run([str(exe)], capture_output=True, text=True, timeout=600)
    assert ok.returncode == 0, ok.stderr[-2000:]
    assert "status 0" in ok.stdout
    short = subprocess.run([str(exe), "short-output"], capture_output=True, text=True, timeout=600)
    assert short.returncode != 0 and "AddressSanitizer" in short.stderr
