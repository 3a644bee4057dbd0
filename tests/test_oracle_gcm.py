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


def test_ghash_is_linear_over_equal_shapes():
    """GHASH_H(A, C) xor GHASH_H(A', C') xor GHASH_H(A xor A', C xor C') = GHASH_H(0, 0) for equal lengths:
    the map is affine, the length block being the constant part."""
    rng = np.random.default_rng(41)
    h = rng.bytes(16)
    for la, lc in [(0, 16), (0, 100), (13, 77), (32, 4096)]:
        a1, a2, c1, c2 = rng.bytes(la), rng.bytes(la), rng.bytes(lc), rng.bytes(lc)
        ax = bytes(x ^ y for x, y in zip(a1, a2))
        cx = bytes(x ^ y for x, y in zip(c1, c2))
        g = [oracle.ghash(h, a1, c1), oracle.ghash(h, a2, c2), oracle.ghash(h, ax, cx), oracle.ghash(h, bytes(la), bytes(lc))]
        acc = bytes(16)
        for t in g:
            acc = bytes(x ^ y for x, y in zip(acc, t))
        assert acc == bytes(16)


def test_ctr_keystream_is_data_independent_and_xor_symmetric():
    rng = np.random.default_rng(42)
    key, iv = rng.bytes(32), rng.bytes(12)
    for n in (1, 16, 33, 1000):
        p1, p2 = rng.bytes(n), rng.bytes(n)
        c1, _ = oracle.gcm_encrypt(key, iv, b"", p1)
        c2, _ = oracle.gcm_encrypt(key, iv, b"", p2)
        assert bytes(a ^ b for a, b in zip(c1, c2)) == bytes(a ^ b for a, b in zip(p1, p2))
        ks, _ = oracle.gcm_encrypt(key, iv, b"", bytes(n))
        assert bytes(a ^ b for a, b in zip(ks, p1)) == c1
        # one flipped ciphertext bit flips exactly that plaintext bit (and the verdict)
        bad = bytearray(c1)
        bad[n // 2] ^= 0x20
        _, t1 = oracle.gcm_encrypt(key, iv, b"", p1)
        back, ok = oracle.gcm_decrypt(key, iv, b"", bytes(bad), t1)
        assert not ok
        diff = [i for i in range(n) if back[i] != p1[i]]
        assert diff == [n // 2] and back[n // 2] ^ p1[n // 2] == 0x20


def test_tag_of_empty_message_is_len_block_times_h_xor_mask():
    """No data, no AAD: GHASH is 0 * H = 0 (the length block is all zero), so the tag is E_K(J0) itself."""
    rng = np.random.default_rng(43)
    key, iv = rng.bytes(32), rng.bytes(12)
    _, t = oracle.gcm_encrypt(key, iv, b"", b"")
    assert t == oracle.aes256_encrypt_block(key, iv + bytes([0, 0, 0, 1]))
    # one block of zeros as AAD only: tag = (LEN * H) xor E_K(J0) with LEN = BE64(128) || BE64(0)
    _, t = oracle.gcm_encrypt(key, iv, bytes(16), b"")
    h = oracle.hash_subkey(key)
    lenblk = (128).to_bytes(8, "big") + bytes(8)
    expect = bytes(a ^ b for a, b in zip(oracle.gf128_mul(lenblk, h), oracle.aes256_encrypt_block(key, iv + bytes([0, 0, 0, 1]))))
    assert t == expect
