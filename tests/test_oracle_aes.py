"""Pins for the oracle's AES-256 (FIPS-197): computed S-box, key schedule, block cipher."""
import numpy as np

import oracle


def test_sbox_spot_values_and_permutation(golden):
    g = golden("fips197_aes256.txt")
    s = oracle.sbox()
    assert s[0x00] == g["sbox_00"][0]
    assert s[0x01] == g["sbox_01"][0]
    assert s[0x53] == g["sbox_53"][0]
    assert s[0xFF] == g["sbox_ff"][0]
    assert sorted(s) == list(range(256))          # a permutation of the bytes
    x = 0
    for v in s:
        x ^= v
    assert x == 0 and sum(s) == 32640
    assert all(s[i] != i and s[i] != (i ^ 0xFF) for i in range(256))   # no fixed / opposite points


def test_key_schedule_appendix_a3(golden):
    g = golden("fips197_aes256.txt")
    w = oracle.aes256_key_expand(g["a3_key"])
    assert len(w) == 240
    assert w[:32] == g["a3_key"]
    assert w[4 * 8: 4 * 9] == g["a3_w8"]
    assert w[4 * 59: 4 * 60] == g["a3_w59"]


def test_cipher_appendix_c3(golden):
    g = golden("fips197_aes256.txt")
    w = oracle.aes256_key_expand(g["c3_key"])
    assert w[32:48] == g["c3_round2_key"]
    assert w[224:240] == g["c3_round14_key"]
    assert oracle.aes256_encrypt_block(g["c3_key"], g["c3_plaintext"]) == g["c3_ciphertext"]


def test_block_cipher_against_openssl_ecb():
    """Independent implementation: OpenSSL AES-256-ECB on random keys and blocks."""
    from cryptography.hazmat.primitives.ciphers import Cipher, algorithms, modes
    rng = np.random.default_rng(7)
    for _ in range(64):
        key, blk = rng.bytes(32), rng.bytes(16)
        enc = Cipher(algorithms.AES(key), modes.ECB()).encryptor()
        assert oracle.aes256_encrypt_block(key, blk) == enc.update(blk) + enc.finalize()


def test_hash_subkey_is_encryption_of_zero(golden):
    g = golden("gcm_aes256_testcases.txt")
    assert oracle.hash_subkey(g["tc13_key"]) == g["tc13_h"]
    assert oracle.hash_subkey(g["tc15_key"]) == g["tc15_h"]
