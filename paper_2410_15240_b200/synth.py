"""Seeded synthetic inputs shared by the tests, the smoke check and the benchmark.

This module holds NONE of the method's arithmetic (no AES, no GF(2^128), no IV derivation): it only
produces keys, IV bases, payload bytes and tamper plans from fixed seeds, so that the CUDA path and
the CPU oracle can be fed the same bytes.  numpy only.

The payloads stand in for the paper's ML transfers (Section 5.1: ImageNet batches for ResNet50,
ogbn-products sub-graphs for GraphSAGE, MovieLens-1M for the two-tower model), none of which is
needed for a cipher whose cost and correctness do not depend on the data: uniform random bytes, an
fp16 image batch 256x3x224x224 ~ N(0,1) and a bf16 parameter buffer ~ N(0,0.02).
"""
from __future__ import annotations

import math
import numpy as np

BASE_SEED = 241015240

MIB = 1 << 20
KIB = 1 << 10


def _rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(int(seed)))


def key_and_iv(config: int):
    """32-byte AES-256 key and 12-byte IV base for config index `config`."""
    raw = _rng(BASE_SEED + 10 * config).bytes(44)
    return raw[:32], raw[32:44]


def fresh_iv(config: int, n: int = 1) -> bytes:
    """Another 12-byte IV base for the same config (n-th re-encryption)."""
    return _rng(BASE_SEED + 10 * config + 5 + 1000 * n).bytes(12)


def random_bytes(n: int, config: int = 0, salt: int = 0) -> np.ndarray:
    """n uniform random bytes (uint8 array)."""
    rng = _rng(BASE_SEED + 10 * config + 1 + 100003 * salt)
    out = np.empty(n, np.uint8)
    step = 1 << 26
    for off in range(0, n, step):
        m = min(step, n - off)
        out[off:off + m] = np.frombuffer(rng.bytes(m), np.uint8)
    return out


def fp16_image_batch(batch: int = 256, config: int = 2) -> np.ndarray:
    """fp16 tensor batch x 3 x 224 x 224 with values ~ N(0,1), returned as its raw bytes."""
    rng = _rng(BASE_SEED + 10 * config + 1)
    n = batch * 3 * 224 * 224
    out = np.empty(n, np.float16)
    step = 1 << 24
    for off in range(0, n, step):
        m = min(step, n - off)
        out[off:off + m] = rng.standard_normal(m, dtype=np.float32).astype(np.float16)
    return out.view(np.uint8)


def bf16_params(n_elems: int = 335_000_000, config: int = 3, std: float = 0.02) -> np.ndarray:
    """bf16 buffer of n_elems values ~ N(0, std), returned as its raw bytes (2 per element).

    bf16 is the upper half of the fp32 pattern, rounded to nearest even."""
    rng = _rng(BASE_SEED + 10 * config + 1)
    out = np.empty(n_elems, np.uint16)
    step = 1 << 24
    for off in range(0, n_elems, step):
        m = min(step, n_elems - off)
        f = (rng.standard_normal(m, dtype=np.float32) * np.float32(std)).view(np.uint32)
        rounded = f + np.uint32(0x7FFF) + ((f >> np.uint32(16)) & np.uint32(1))
        out[off:off + m] = (rounded >> np.uint32(16)).astype(np.uint16)
    return out.view(np.uint8)


def chunk_lengths(length: int, chunk_bytes: int):
    """Byte length of every chunk of a buffer (only the last may be short)."""
    k = 0 if length == 0 else (length + chunk_bytes - 1) // chunk_bytes
    return [min(chunk_bytes, length - i * chunk_bytes) for i in range(k)]


def tamper_plan(length: int, chunk_bytes: int, config: int, fraction: float = 0.01, salt: int = 0):
    """Which chunks to corrupt and how: list of (chunk, 'cipher'|'tag', bit index in that field).

    ceil(fraction*K) chunks if K >= 2, none if K < 2; chunks by a seeded shuffle; per chunk a seeded
    coin picks ciphertext or tag and a seeded bit index inside len_k*8 (ciphertext) or 128 (tag)."""
    lens = chunk_lengths(length, chunk_bytes)
    K = len(lens)
    if K < 2:
        return []
    n_t = max(1, math.ceil(fraction * K))
    rng = _rng(BASE_SEED + 10 * config + 2 + 7919 * salt)
    chosen = sorted(int(x) for x in rng.permutation(K)[:n_t])
    plan = []
    for k in chosen:
        if rng.integers(0, 2) == 0:
            plan.append((k, "cipher", int(rng.integers(0, lens[k] * 8))))
        else:
            plan.append((k, "tag", int(rng.integers(0, 128))))
    return plan


def apply_tamper(cipher: np.ndarray, tags: np.ndarray, chunk_bytes: int, plan) -> None:
    """Flip the planned bits in place.  `tags` is uint8[K,16] or flat uint8[16K]."""
    flat_tags = tags.reshape(-1)
    for k, where, bit in plan:
        if where == "cipher":
            cipher[k * chunk_bytes + bit // 8] ^= np.uint8(1 << (bit % 8))
        else:
            flat_tags[16 * k + bit // 8] ^= np.uint8(1 << (bit % 8))
