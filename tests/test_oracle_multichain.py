"""Pins for the oracle's multi-chaining layer (paper Section 4.2) under the per-chunk IV reading."""
import numpy as np
import pytest

import oracle
from paper_2410_15240_b200 import synth


def test_chunk_iv_rule():
    base = bytes(range(12))
    assert oracle.chunk_iv(base, 0) == base
    assert oracle.chunk_iv(base, 1) == bytes(range(11)) + bytes([0x0C])
    assert oracle.chunk_iv(base, 0x1F5) == bytes(range(8)) + (0x08090A0B + 0x1F5).to_bytes(4, "big")
    wrap = bytes(range(8)) + bytes([0xFF] * 4)
    assert oracle.chunk_iv(wrap, 1) == bytes(range(8)) + bytes(4)        # first 8 bytes untouched
    assert oracle.chunk_iv(wrap, 3) == bytes(range(8)) + bytes([0, 0, 0, 2])


def test_num_chunks():
    assert oracle.num_chunks(0, 64) == 0
    assert oracle.num_chunks(1, 64) == 1
    assert oracle.num_chunks(64, 64) == 1
    assert oracle.num_chunks(65, 64) == 2
    assert oracle.num_chunks(1 << 20, 1 << 16) == 16


@pytest.mark.parametrize("n", [0, 1, 15, 16, 17, 31, 32, 33, 1000, 4096])
def test_single_chain_equals_plain_gcm(n):
    rng = np.random.default_rng(31 + n)
    key, iv, p = rng.bytes(32), rng.bytes(12), rng.bytes(n)
    c, tags = oracle.mc_encrypt(key, iv, max(16, (n + 15) // 16 * 16), p)
    ref_c, ref_t = oracle.gcm_encrypt(key, iv, b"", p)
    assert c.tobytes() == ref_c
    if n:
        assert tags.shape == (1, 16) and tags.tobytes() == ref_t
    else:
        assert tags.shape == (0, 16)


@pytest.mark.parametrize("length,cb", [(64, 32), (40, 32), (1000, 96), (4096, 1024), (4097, 1024), (5000, 16)])
def test_each_chunk_is_a_standalone_openssl_gcm_call(length, cb):
    """Chunk k == AES-256-GCM(key, IV_k, no AAD) of that slice, by an independent library."""
    from cryptography.hazmat.primitives.ciphers.aead import AESGCM
    rng = np.random.default_rng(length * 7 + cb)
    key, base, p = rng.bytes(32), rng.bytes(8) + bytes([0xFF, 0xFF, 0xFF, 0xFE]), rng.bytes(length)
    c, tags = oracle.mc_encrypt(key, base, cb, p, n_threads=3)
    K = (length + cb - 1) // cb
    assert tags.shape == (K, 16)
    for k in range(K):
        ctr = (int.from_bytes(base[8:], "big") + k) % (1 << 32)
        iv_k = base[:8] + ctr.to_bytes(4, "big")
        ref = AESGCM(key).encrypt(iv_k, p[k * cb:(k + 1) * cb], None)
        assert c[k * cb:(k + 1) * cb].tobytes() + tags[k].tobytes() == ref


def test_worked_example_structure(golden):
    """key 00..1f, iv_base 00..0b, P[i] = i, len 64, cb 32: chunk 1 is GCM under IV ..0a0c of P[32:].  The stored
    values (tests/golden/multichain_worked_example.txt) are what SP 800-38D gives under the per-chunk IV rule; they
    are compared with the oracle and, chunk by chunk, with OpenSSL."""
    from cryptography.hazmat.primitives.ciphers.aead import AESGCM
    g = golden("multichain_worked_example.txt")
    key, base = bytes(range(32)), bytes(range(12))
    p = bytes(range(64))
    c, tags = oracle.mc_encrypt(key, base, 32, p)
    assert g["iv0"] == base and g["iv1"] == bytes(range(11)) + bytes([0x0C])
    assert c[:32].tobytes() == g["c0"] and tags[0].tobytes() == g["t0"]
    assert c[32:].tobytes() == g["c1"] and tags[1].tobytes() == g["t1"]
    assert AESGCM(key).encrypt(g["iv0"], p[:32], None) == g["c0"] + g["t0"]
    assert AESGCM(key).encrypt(g["iv1"], p[32:], None) == g["c1"] + g["t1"]
    assert AESGCM(key).encrypt(g["iv1"], p[32:40], None) == g["tail8_c"] + g["tail8_t"]
    c40g, t40g = oracle.mc_encrypt(key, base, 32, p[:40])
    assert c40g[32:].tobytes() == g["tail8_c"] and t40g[1].tobytes() == g["tail8_t"]
    h0 = oracle.hash_subkey(bytes(32))
    assert oracle.gf128_mul(h0, h0) == g["h_zero_key_squared"]
    c1, t1 = oracle.gcm_encrypt(key, bytes(range(11)) + bytes([0x0C]), b"", p[32:])
    assert c[32:].tobytes() == c1 and tags[1].tobytes() == t1
    # the short-tail variant shares its first chunk and the prefix of chunk 1's keystream
    c40, tags40 = oracle.mc_encrypt(key, base, 32, p[:40])
    assert c40.tobytes() == c[:40].tobytes()
    assert tags40[0].tobytes() == tags[0].tobytes() and tags40[1].tobytes() != tags[1].tobytes()


@pytest.mark.parametrize("n", [0, 1, 15, 16, 17, 31, 32, 33, 1023, 1024, 1025, 70000])
def test_round_trip_and_thread_independence(n):
    key, base = synth.key_and_iv(0)
    p = synth.random_bytes(n, 0, salt=n)
    c1, t1 = oracle.mc_encrypt(key, base, 1024, p, n_threads=1)
    c8, t8 = oracle.mc_encrypt(key, base, 1024, p, n_threads=8)
    assert np.array_equal(c1, c8) and np.array_equal(t1, t8)
    back, ok = oracle.mc_decrypt(key, base, 1024, c1, t1, n_threads=4)
    assert np.array_equal(back, p) and ok.all() and ok.size == (n + 1023) // 1024


def test_tamper_and_reorder_detection():
    key, base = synth.key_and_iv(0)
    cb, n = 1024, 16 * 1024 + 100
    p = synth.random_bytes(n, 0, salt=99)
    c, tags = oracle.mc_encrypt(key, base, cb, p, n_threads=4)
    plan = [(5, "cipher", 777), (11, "tag", 101), (16, "cipher", 3)]
    bad_c, bad_t = c.copy(), tags.copy()
    synth.apply_tamper(bad_c, bad_t, cb, plan)
    back, ok = oracle.mc_decrypt(key, base, cb, bad_c, bad_t, n_threads=4)
    assert [int(k) for k in np.flatnonzero(ok == 0)] == [5, 11, 16]
    for k in range(17):
        if k not in (5, 16):                       # tag-only tamper leaves the plaintext intact
            assert np.array_equal(back[k * cb:(k + 1) * cb], p[k * cb:(k + 1) * cb])
    # swap chunks 2 and 9 together with their tags: both are decrypted under the wrong IV
    sw_c, sw_t = c.copy(), tags.copy()
    sw_c[2 * cb:3 * cb], sw_c[9 * cb:10 * cb] = c[9 * cb:10 * cb], c[2 * cb:3 * cb]
    sw_t[2], sw_t[9] = tags[9], tags[2]
    _, ok = oracle.mc_decrypt(key, base, cb, sw_c, sw_t, n_threads=4)
    assert [int(k) for k in np.flatnonzero(ok == 0)] == [2, 9]


def test_cost_accounting_of_n_chains():
    """n chains cost n - 1 extra tags (16 bytes each); at 64 KiB chunks that is 0.024 % of the bytes."""
    for length, cb in [(1 << 20, 1 << 16), (77_070_336, 4 << 20)]:
        K = oracle.num_chunks(length, cb)
        assert 16 * K / length < 0.01
    assert abs(16 * 16 / (1 << 20) - 0.000244) < 1e-6


@pytest.mark.parametrize("length,cb,n", [(64, 32, 16), (1000, 96, 4), (4097, 1024, 3), (5000, 16, 256), (40, 32, 1)])
def test_framed_chunks_are_openssl_gcm_calls_with_a_serial_byte_as_aad(length, cb, n):
    """Paper Sections 4.2 / 4.4: chunk k authenticates the byte (k mod n) as AAD; independent check by OpenSSL."""
    from cryptography.hazmat.primitives.ciphers.aead import AESGCM
    rng = np.random.default_rng(length + cb + n)
    key, base, p = rng.bytes(32), rng.bytes(12), rng.bytes(length)
    c, tags = oracle.mc_encrypt_framed(key, base, cb, n, p, n_threads=3)
    K = (length + cb - 1) // cb
    for k in range(K):
        ref = AESGCM(key).encrypt(oracle.chunk_iv(base, k), p[k * cb:(k + 1) * cb], bytes([k % n]))
        assert c[k * cb:(k + 1) * cb].tobytes() + tags[k].tobytes() == ref
    back, ok = oracle.mc_decrypt_framed(key, base, cb, n, c, tags, n_threads=2)
    assert ok.all() and back.tobytes() == p
    # the ciphertext does not depend on the framing, every tag does
    c0, t0 = oracle.mc_encrypt(key, base, cb, p)
    assert np.array_equal(c0, c) and all(not np.array_equal(t0[k], tags[k]) for k in range(K))
    # a verifier without the framing (or with another sample size) rejects every chunk
    assert not oracle.mc_decrypt(key, base, cb, c, tags)[1].any()
    if 1 < n < 256 and K > 1:
        _, ok2 = oracle.mc_decrypt_framed(key, base, cb, n + 1, c, tags)
        assert [bool(x) for x in ok2] == [(k % n) == (k % (n + 1)) for k in range(K)]
