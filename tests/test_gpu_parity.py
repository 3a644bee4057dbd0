"""GPU parity: the CUDA path, called through the C ABI, must be BIT-EXACT against the CPU oracle
(ciphertext / plaintext bytes, per-chunk tags, accept / reject flags) on the same seeded inputs."""
import numpy as np
import pytest

import oracle
from paper_2410_15240_b200 import synth

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")
if not torch.cuda.is_available():
    pytest.skip("no CUDA device", allow_module_level=True)

from gpu_harness import Gpu  # noqa: E402

NT = oracle.host_threads()


def check_both_directions(key, iv, cb, plain, in_place=False):
    """encrypt on GPU == oracle encrypt; decrypt of the oracle's output on GPU == original, all accepted."""
    c_ref, t_ref = oracle.mc_encrypt(key, iv, cb, plain, NT)
    with Gpu(key, cb) as g:
        c, t = g.encrypt(iv, plain, in_place=in_place)
        assert np.array_equal(c, c_ref), "ciphertext differs from the oracle"
        assert np.array_equal(t, t_ref), "tags differ from the oracle"
        p, ok = g.decrypt(iv, c_ref, t_ref, in_place=in_place)
        assert np.array_equal(p, plain), "plaintext differs"
        assert ok.dtype == np.uint32 and (ok == 1).all() and ok.size == oracle.num_chunks(plain.size, cb)


@pytest.mark.parametrize("cb", [16, 32, 48, 512, 1024, 16384])
def test_tiny_and_ragged_sizes(cb):
    key, iv = synth.key_and_iv(0)
    sizes = {1, 15, 16, 17, 31, 32, 33, 511, 512, 513, cb - 1, cb, cb + 1, 2 * cb, 2 * cb + 1, 3 * cb - 1, 3 * cb + 17}
    for n in sorted(s for s in sizes if s > 0):
        check_both_directions(key, iv, cb, synth.random_bytes(n, 0, salt=n + cb))


def test_empty_buffer_is_a_no_op():
    key, iv = synth.key_and_iv(0)
    with Gpu(key, 1024) as g:
        p, ok = g.decrypt(iv, np.zeros(0, np.uint8), np.zeros(0, np.uint8))
        assert p.size == 0 and ok.size == 0
        c, t = g.encrypt(iv, np.zeros(0, np.uint8))
        assert c.size == 0 and t.size == 0


@pytest.mark.parametrize("n,cb", [(70001, 16384), (200000, 65536), (1 << 20, 65536), (3 * (1 << 20) + 4321, 1 << 20),
                                  ((1 << 22) + 16, 1 << 22), (5 * (1 << 20) + 1, 48 * 1024)])
@pytest.mark.parametrize("in_place", [False, True])
def test_multi_segment_chunks(n, cb, in_place):
    key, iv = synth.key_and_iv(1)
    check_both_directions(key, iv, cb, synth.random_bytes(n, 1, salt=n), in_place=in_place)


def test_iv_index_wraps_in_last_four_bytes():
    key, _ = synth.key_and_iv(0)
    iv = bytes(range(8)) + bytes([0xFF, 0xFF, 0xFF, 0xFD])
    check_both_directions(key, iv, 256, synth.random_bytes(256 * 7 + 5, 0, salt=77))


def test_config0_one_mib_sixteen_chains_with_two_tampered():
    """1 MiB, 64 KiB chunks -> 16 chains; one ciphertext bit of chunk 5 and one tag bit of chunk 11 flipped."""
    key, iv = synth.key_and_iv(0)
    cb, n = 64 * 1024, 1 << 20
    plain = synth.random_bytes(n, 0)
    c, t = oracle.mc_encrypt(key, iv, cb, plain, NT)
    rng = np.random.Generator(np.random.PCG64(synth.BASE_SEED + 2))
    plan = [(5, "cipher", int(rng.integers(0, cb * 8))), (11, "tag", int(rng.integers(0, 128)))]
    synth.apply_tamper(c, t, cb, plan)
    p_ref, ok_ref = oracle.mc_decrypt(key, iv, cb, c, t, NT)
    assert [int(k) for k in np.flatnonzero(ok_ref == 0)] == [5, 11]
    with Gpu(key, cb) as g:
        p, ok = g.decrypt(iv, c, t)
    assert np.array_equal(ok, ok_ref)
    assert np.array_equal(p, p_ref)                      # even the rejected chunks decrypt identically
    for k in range(16):
        if k != 5:
            assert np.array_equal(p[k * cb:(k + 1) * cb], plain[k * cb:(k + 1) * cb])


def test_every_tampered_position_class_is_rejected():
    """First/last byte of a chunk, first/last chunk, the partial last block, every tag byte."""
    key, iv = synth.key_and_iv(0)
    cb, n = 4096, 4096 * 5 + 7
    plain = synth.random_bytes(n, 0, salt=5)
    c, t = oracle.mc_encrypt(key, iv, cb, plain, NT)
    with Gpu(key, cb) as g:
        for pos in [0, 15, 16, 4095, 4096, 2 * 4096 + 511, 5 * 4096 - 1, 5 * 4096, n - 1]:
            bad = c.copy()
            bad[pos] ^= 0x80
            _, ok = g.decrypt(iv, bad, t)
            exp = np.ones(6, np.uint32); exp[pos // cb] = 0
            assert np.array_equal(ok, exp), pos
        for k in (0, 3, 5):
            for byte in range(16):
                bad = t.copy()
                bad[k, byte] ^= 1 << (byte % 8)
                p, ok = g.decrypt(iv, c, bad)
                exp = np.ones(6, np.uint32); exp[k] = 0
                assert np.array_equal(ok, exp) and np.array_equal(p, plain)


def test_reordered_chunks_are_rejected():
    """Paper Section 4.4, reorder attacks: chunks moved together with their tags must fail."""
    key, iv = synth.key_and_iv(0)
    cb, n = 8192, 8192 * 12
    plain = synth.random_bytes(n, 0, salt=6)
    c, t = oracle.mc_encrypt(key, iv, cb, plain, NT)
    sc, stg = c.copy(), t.copy()
    sc[2 * cb:3 * cb], sc[9 * cb:10 * cb] = c[9 * cb:10 * cb], c[2 * cb:3 * cb]
    stg[2], stg[9] = t[9], t[2]
    _, ok_ref = oracle.mc_decrypt(key, iv, cb, sc, stg, NT)
    with Gpu(key, cb) as g:
        _, ok = g.decrypt(iv, sc, stg)
    assert np.array_equal(ok, ok_ref) and [int(k) for k in np.flatnonzero(ok == 0)] == [2, 9]


def test_wrong_key_or_iv_rejects_everything():
    key, iv = synth.key_and_iv(0)
    key2, iv2 = synth.key_and_iv(1)
    cb, n = 1024, 10 * 1024
    c, t = oracle.mc_encrypt(key, iv, cb, synth.random_bytes(n, 0, salt=8), NT)
    with Gpu(key2, cb) as g:
        assert (g.decrypt(iv, c, t)[1] == 0).all()
    with Gpu(key, cb) as g:
        assert (g.decrypt(iv2, c, t)[1] == 0).all()
        assert (g.decrypt(iv, c, t)[1] == 1).all()


def test_context_reuse_many_calls_and_growing_chunk_counts():
    """The per-chunk scratch must come back clean after every call, also when it has to grow."""
    key, iv = synth.key_and_iv(0)
    cb = 1024
    with Gpu(key, cb) as g:
        for n in [cb * 3, cb * 2000 + 5, cb * 7, cb * 5000, 100]:
            plain = synth.random_bytes(n, 0, salt=n)
            c_ref, t_ref = oracle.mc_encrypt(key, iv, cb, plain, NT)
            for _ in range(2):
                c, t = g.encrypt(iv, plain)
                assert np.array_equal(c, c_ref) and np.array_equal(t, t_ref)
                p, ok = g.decrypt(iv, c_ref, t_ref)
                assert np.array_equal(p, plain) and (ok == 1).all()


def test_non_default_stream():
    key, iv = synth.key_and_iv(0)
    cb, n = 65536, 65536 * 9 + 3
    plain = synth.random_bytes(n, 0, salt=10)
    c_ref, t_ref = oracle.mc_encrypt(key, iv, cb, plain, NT)
    st = torch.cuda.Stream()
    with Gpu(key, cb) as g:
        with torch.cuda.stream(st):
            p, ok = g.decrypt(iv, c_ref, t_ref, stream=st)
    assert np.array_equal(p, plain) and (ok == 1).all()


@pytest.mark.parametrize("K", [1, 4, 16, 64, 256, 1024])
def test_config1_chain_count_sweep_64mib(K):
    """64 MiB, K = 1 .. 1024 chains (chunk 64 MiB .. 64 KiB): both directions against the oracle."""
    key, iv = synth.key_and_iv(1)
    n = 64 << 20
    cb = n // K
    plain = synth.random_bytes(n, 1)
    check_both_directions(key, iv, cb, plain)
