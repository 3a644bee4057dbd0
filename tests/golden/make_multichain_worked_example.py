"""Writes tests/golden/multichain_worked_example.txt: the two-chunk worked example of the per-chunk IV rule.

The values are fixed by SP 800-38D once the rule IV_k = iv_base[0..7] || BE32(BE32(iv_base[8..11]) + k) is adopted
(the paper, Section 4.2, gives every chain a nonce of its own but no derivation).  This script calls only the CPU
oracle; tests/test_oracle_multichain.py compares the stored values with the oracle AND, live, with OpenSSL.

    python tests/golden/make_multichain_worked_example.py
"""
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)
import oracle  # noqa: E402

key, base = bytes(range(32)), bytes(range(12))
p = bytes(range(64))
c, t = oracle.mc_encrypt(key, base, 32, p)
c40, t40 = oracle.mc_encrypt(key, base, 32, p[:40])
h0 = oracle.hash_subkey(bytes(32))
lines = [
    "# Two-chunk worked example of the multi-chain layer: key 00..1f, iv_base 00..0b, P[i] = i, chunk_bytes 32.",
    "# Chunk k is AES-256-GCM (SP 800-38D, no AAD, 128-bit tag) of its 32-byte slice under",
    "# IV_k = iv_base[0..7] || BE32(BE32(iv_base[8..11]) + k); `tail8_*` is chunk 1 when the buffer is 40 bytes long.",
    "# h_zero_key_squared: H * H in GF(2^128) for the all-zero AES-256 key (H = dc95c078...).",
    "# Written by tests/golden/make_multichain_worked_example.py (CPU oracle only); the test also checks OpenSSL live.",
    "",
    f"iv0 = {base.hex()}",
    f"c0  = {c[:32].tobytes().hex()}",
    f"t0  = {t[0].tobytes().hex()}",
    f"iv1 = {(base[:8] + (int.from_bytes(base[8:], 'big') + 1).to_bytes(4, 'big')).hex()}",
    f"c1  = {c[32:].tobytes().hex()}",
    f"t1  = {t[1].tobytes().hex()}",
    f"tail8_c = {c40[32:].tobytes().hex()}",
    f"tail8_t = {t40[1].tobytes().hex()}",
    f"h_zero_key_squared = {oracle.gf128_mul(h0, h0).hex()}",
    "",
]
with open(os.path.join(ROOT, "tests", "golden", "multichain_worked_example.txt"), "w") as f:
    f.write("\n".join(lines))
print("\n".join(lines))
