"""Pins for the oracle's GF(2^128) product (SP 800-38D Algorithm 1) and GHASH.

The brute force below is written independently in Python integers: a block is mapped to a
polynomial with bit 0 (the MSB of byte 0) as the coefficient of x^0, the two polynomials are
multiplied by the schoolbook method and the product is reduced by long division by
x^128 + x^7 + x^2 + x + 1.
"""
import numpy as np

import oracle

P128 = (1 << 128) | (1 << 7) | (1 << 2) | (1 << 1) | 1
ONE = bytes([0x80]) + bytes(15)
X1 = bytes([0x40]) + bytes(15)


def to_poly(b: bytes) -> int:
    """bit i of the block (MSB-first inside each byte) -> coefficient of x^i."""
    v = 0
    for i in range(128):
        if (b[i // 8] >> (7 - i % 8)) & 1:
            v |= 1 << i
    return v


def from_poly(v: int) -> bytes:
    out = bytearray(16)
    for i in range(128):
        if (v >> i) & 1:
            out[i // 8] |= 1 << (7 - i % 8)
    return bytes(out)


def brute_mul(a: bytes, b: bytes) -> bytes:
    pa, pb = to_poly(a), to_poly(b)
    prod = 0
    for i in range(128):
        if (pa >> i) & 1:
            prod ^= pb << i
    for d in range(prod.bit_length() - 1, 127, -1):
        if (prod >> d) & 1:
            prod ^= P128 << (d - 128)
    return from_poly(prod)


def xor(a, b):
    return bytes(x ^ y for x, y in zip(a, b))


def test_identity_zero_and_times_x(golden):
    h = golden("gcm_aes256_testcases.txt")["tc13_h"]
    assert oracle.gf128_mul(h, ONE) == h and oracle.gf128_mul(ONE, h) == h
    assert oracle.gf128_mul(h, bytes(16)) == bytes(16)
    # H * x: H ends in a 1 bit, so the result is (H >> 1) with R = e1 00..00 folded in.
    shifted = (int.from_bytes(h, "big") >> 1).to_bytes(16, "big")
    expect = bytes([shifted[0] ^ 0xE1]) + shifted[1:]
    assert h[15] & 1 == 1
    assert oracle.gf128_mul(h, X1) == expect
    assert expect.hex() == "8f4ae03c512044c4d6a4510a49421043"
    # x^127 * x = x^128 = x^7 + x^2 + x + 1  ->  bits 0,1,2,7 -> byte 0 = 0xe1
    x127 = bytes(15) + bytes([0x01])
    assert oracle.gf128_mul(x127, X1) == bytes([0xE1]) + bytes(15)


def test_against_schoolbook_brute_force():
    rng = np.random.default_rng(11)
    pairs = [(rng.bytes(16), rng.bytes(16)) for _ in range(10000)]
    singles = [from_poly(1 << i) for i in range(128)]
    for i in range(0, 128, 7):
        for j in range(0, 128, 5):
            pairs.append((singles[i], singles[j]))
    pairs += [(singles[127], singles[127]), (singles[0], singles[127]), (bytes([0xFF] * 16), bytes([0xFF] * 16))]
    for a, b in pairs:
        assert oracle.gf128_mul(a, b) == brute_mul(a, b)


def test_field_axioms():
    rng = np.random.default_rng(12)
    for _ in range(200):
        a, b, c = rng.bytes(16), rng.bytes(16), rng.bytes(16)
        assert oracle.gf128_mul(a, b) == oracle.gf128_mul(b, a)
        assert oracle.gf128_mul(a, xor(b, c)) == xor(oracle.gf128_mul(a, b), oracle.gf128_mul(a, c))
        assert oracle.gf128_mul(oracle.gf128_mul(a, b), c) == oracle.gf128_mul(a, oracle.gf128_mul(b, c))


def test_pow_matches_repeated_brute_force():
    rng = np.random.default_rng(13)
    h = rng.bytes(16)
    acc = ONE
    for e in range(0, 40):
        assert oracle.gf128_pow(h, e) == acc
        acc = brute_mul(acc, h)


def test_ghash_chain_equals_power_sum():
    """Horner chain == closed form sum X_i * H^(m-i+1), for ragged and whole inputs."""
    rng = np.random.default_rng(14)
    h = rng.bytes(16)
    for m in [1, 2, 3, 17, 64, 300]:
        blocks = rng.bytes(16 * m)
        # ghash() appends the length block; rebuild the same block list for the closed form
        lens = (0).to_bytes(8, "big") + (8 * 16 * m).to_bytes(8, "big")
        assert oracle.ghash(h, b"", blocks) == oracle.ghash_pow(h, blocks + lens)
    # brute-force power sum on a tiny case, independent of the oracle's multiply
    blocks = rng.bytes(16 * 5)
    lens = (0).to_bytes(8, "big") + (8 * 80).to_bytes(8, "big")
    allb = blocks + lens
    acc = bytes(16)
    for i in range(6):
        p = ONE
        for _ in range(6 - i):
            p = brute_mul(p, h)
        acc = xor(acc, brute_mul(allb[16 * i:16 * i + 16], p))
    assert oracle.ghash(h, b"", blocks) == acc


def test_ghash_padding_and_aad_layout():
    """A ragged tail is zero-padded; AAD and ciphertext are padded separately; lengths are in bits."""
    rng = np.random.default_rng(15)
    h = rng.bytes(16)
    aad, c = rng.bytes(20), rng.bytes(37)
    blocks = aad + bytes(12) + c + bytes(11) + (160).to_bytes(8, "big") + (296).to_bytes(8, "big")
    assert oracle.ghash(h, aad, c) == oracle.ghash_pow(h, blocks)
