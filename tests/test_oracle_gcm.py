"""Pins for the oracle's AES-256-GCM: the GCM specification's test cases 13-16 and OpenSSL."""
import numpy as np
import pytest

import oracle


@pytest.mark.parametrize("tc", ["tc13", "tc14", "tc15", "tc16"])
def test_gcm_spec_cases(golden, tc):
    g = golden("gcm_aes256_testcases.txt")
    key, iv, aad, p = g[f"{tc}_key"], g[f"{tc}_iv"], g[f"{tc}_aad"], g[f"{tc}_p"]
    assert oracle.hash_subkey(key) == g[f"{tc}_h"]
    c, t = oracle.gcm_encrypt(key, iv, aad, p)
    assert c == g[f"{tc}_c"]
    assert t == g[f"{tc}_t"]
    back, ok = oracle.gcm_decrypt(key, iv, aad, c, t)
    assert ok and back == p


def test_gcm_decrypt_rejects_any_single_bit_flip(golden):
    g = golden("gcm_aes256_testcases.txt")
    key, iv, aad, c, t = g["tc16_key"], g["tc16_iv"], g["tc16_aad"], g["tc16_c"], g["tc16_t"]
    for bit in range(0, len(c) * 8, 13):
        bad = bytearray(c)
        bad[bit // 8] ^= 1 << (bit % 8)
        assert not oracle.gcm_decrypt(key, iv, aad, bytes(bad), t)[1]
    for bit in range(128):
        bad = bytearray(t)
        bad[bit // 8] ^= 1 << (bit % 8)
        p, ok = oracle.gcm_decrypt(key, iv, aad, c, bytes(bad))
        assert not ok and p == g["tc16_p"]       # plaintext is released whatever the verdict
    bad_aad = bytearray(aad)
    bad_aad[0] ^= 1
    assert not oracle.gcm_decrypt(key, iv, bytes(bad_aad), c, t)[1]


def test_gcm_against_openssl_random_lengths():
    from cryptography.hazmat.primitives.ciphers.aead import AESGCM
    rng = np.random.default_rng(21)
    for n in [0, 1, 15, 16, 17, 31, 32, 33, 255, 256, 257, 1000, 4096, 65537]:
        for aad_len in (0, 1, 16, 29):
            key, iv = rng.bytes(32), rng.bytes(12)
            aad, p = rng.bytes(aad_len), rng.bytes(n)
            c, t = oracle.gcm_encrypt(key, iv, aad, p)
            assert AESGCM(key).encrypt(iv, p, aad if aad else None) == c + t


def test_counter_wraps_inside_last_four_bytes_only():
    """inc32: IV || ffffffff would wrap; reachable here through J0 = IV||1 only after 2^32 blocks,
    so check the keystream position instead: block j uses counter 2 + j."""
    rng = np.random.default_rng(22)
    key, iv = rng.bytes(32), rng.bytes(12)
    p = bytes(16 * 300)
    c, _ = oracle.gcm_encrypt(key, iv, b"", p)
    for j in (0, 1, 254, 255, 256, 299):
        ctr_block = iv + (2 + j).to_bytes(4, "big")
        assert c[16 * j:16 * j + 16] == oracle.aes256_encrypt_block(key, ctr_block)
