"""CPU oracle for the Fastrack hot path -- TEST INFRASTRUCTURE ONLY.

Thin ctypes wrapper over ``fastrack_oracle.c`` (plain C, FIPS-197 + SP 800-38D written out
byte by byte; see that file's header for what each function follows).  Only the tests, the
smoke check and the benchmark's cpu_baseline / reference arm may import this package; the
product (``paper_2410_15240_b200``) never does, and this package never imports the product.

Buffers are ``bytes`` / ``bytearray`` / C-contiguous uint8 numpy arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fastrack_oracle.c")
_LIB = os.path.join(_HERE, "libfastrack_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc -O2 (no intrinsics, no vector flags).  Returns the .so path."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fvisibility=hidden", "-pthread",
             "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is not None:
        return _lib
    lib = ctypes.CDLL(build())
    u8p, sz, u64, i32 = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_uint64, ctypes.c_int
    sig = {
        "fo_sbox": (None, [u8p]),
        "fo_aes256_key_expand": (None, [u8p, u8p]),
        "fo_aes256_encrypt_block": (None, [u8p, u8p, u8p]),
        "fo_gf128_mul": (None, [u8p, u8p, u8p]),
        "fo_gf128_pow": (None, [u8p, u64, u8p]),
        "fo_ghash": (None, [u8p, u8p, sz, u8p, sz, u8p]),
        "fo_ghash_pow": (None, [u8p, u8p, sz, u8p]),
        "fo_gcm_encrypt": (None, [u8p, u8p, u8p, sz, u8p, sz, u8p, u8p]),
        "fo_gcm_decrypt": (i32, [u8p, u8p, u8p, sz, u8p, sz, u8p, u8p]),
        "fo_chunk_iv": (None, [u8p, u64, u8p]),
        "fo_num_chunks": (sz, [sz, sz]),
        "fo_mc_encrypt": (None, [u8p, u8p, sz, u8p, sz, u8p, u8p, i32]),
        "fo_mc_decrypt": (None, [u8p, u8p, sz, u8p, sz, u8p, u8p, u8p, i32]),
        "fo_mc_encrypt_framed": (None, [u8p, u8p, sz, ctypes.c_uint, u8p, sz, u8p, u8p, i32]),
        "fo_mc_decrypt_framed": (None, [u8p, u8p, sz, ctypes.c_uint, u8p, sz, u8p, u8p, u8p, i32]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype = res
        fn.argtypes = args
    _lib = lib
    return lib


def _arr(buf, n=None) -> np.ndarray:
    """View the input as a contiguous uint8 array (copying only if it has to)."""
    if isinstance(buf, np.ndarray):
        a = np.ascontiguousarray(buf).view(np.uint8).reshape(-1)
    else:
        a = np.frombuffer(bytes(buf), dtype=np.uint8)
    if n is not None and a.size != n:
        raise ValueError(f"expected {n} bytes, got {a.size}")
    return a


def _ptr(a: np.ndarray):
    return a.ctypes.data if a.size else None


def host_threads() -> int:
    return os.cpu_count() or 1


def sbox() -> bytes:
    out = np.zeros(256, np.uint8)
    _load().fo_sbox(_ptr(out))
    return out.tobytes()


def aes256_key_expand(key) -> bytes:
    k = _arr(key, 32)
    w = np.zeros(240, np.uint8)
    _load().fo_aes256_key_expand(_ptr(k), _ptr(w))
    return w.tobytes()


def aes256_encrypt_block(key, block) -> bytes:
    w = _arr(aes256_key_expand(key))
    b = _arr(block, 16)
    out = np.zeros(16, np.uint8)
    _load().fo_aes256_encrypt_block(_ptr(w), _ptr(b), _ptr(out))
    return out.tobytes()


def hash_subkey(key) -> bytes:
    """H = E_K(0^128)."""
    return aes256_encrypt_block(key, bytes(16))


def gf128_mul(x, y) -> bytes:
    a, b = _arr(x, 16), _arr(y, 16)
    out = np.zeros(16, np.uint8)
    _load().fo_gf128_mul(_ptr(a), _ptr(b), _ptr(out))
    return out.tobytes()


def gf128_pow(h, e: int) -> bytes:
    a = _arr(h, 16)
    out = np.zeros(16, np.uint8)
    _load().fo_gf128_pow(_ptr(a), int(e), _ptr(out))
    return out.tobytes()


def ghash(h, aad, c) -> bytes:
    hh, a, cc = _arr(h, 16), _arr(aad), _arr(c)
    out = np.zeros(16, np.uint8)
    _load().fo_ghash(_ptr(hh), _ptr(a), a.size, _ptr(cc), cc.size, _ptr(out))
    return out.tobytes()


def ghash_pow(h, blocks) -> bytes:
    hh, b = _arr(h, 16), _arr(blocks)
    if b.size % 16:
        raise ValueError("whole blocks only")
    out = np.zeros(16, np.uint8)
    _load().fo_ghash_pow(_ptr(hh), _ptr(b), b.size // 16, _ptr(out))
    return out.tobytes()


def gcm_encrypt(key, iv, aad, p):
    """-> (ciphertext bytes, 16-byte tag)."""
    k, v, a, pp = _arr(key, 32), _arr(iv, 12), _arr(aad), _arr(p)
    c = np.zeros(pp.size, np.uint8)
    tag = np.zeros(16, np.uint8)
    _load().fo_gcm_encrypt(_ptr(k), _ptr(v), _ptr(a), a.size, _ptr(pp), pp.size, _ptr(c), _ptr(tag))
    return c.tobytes(), tag.tobytes()


def gcm_decrypt(key, iv, aad, c, tag):
    """-> (plaintext bytes, ok bool).  Plaintext is returned whatever the verdict."""
    k, v, a, cc, t = _arr(key, 32), _arr(iv, 12), _arr(aad), _arr(c), _arr(tag, 16)
    p = np.zeros(cc.size, np.uint8)
    ok = _load().fo_gcm_decrypt(_ptr(k), _ptr(v), _ptr(a), a.size, _ptr(cc), cc.size, _ptr(t), _ptr(p))
    return p.tobytes(), bool(ok)


def chunk_iv(iv_base, k: int) -> bytes:
    b = _arr(iv_base, 12)
    out = np.zeros(12, np.uint8)
    _load().fo_chunk_iv(_ptr(b), int(k), _ptr(out))
    return out.tobytes()


def num_chunks(length: int, chunk_bytes: int) -> int:
    return int(_load().fo_num_chunks(int(length), int(chunk_bytes)))


def mc_encrypt(key, iv_base, chunk_bytes: int, p, n_threads: int = 1):
    """Multi-chain encrypt: -> (cipher uint8[len], tags uint8[K,16])."""
    k, v, pp = _arr(key, 32), _arr(iv_base, 12), _arr(p)
    K = num_chunks(pp.size, chunk_bytes)
    c = np.zeros(pp.size, np.uint8)
    tags = np.zeros((K, 16), np.uint8)
    _load().fo_mc_encrypt(_ptr(k), _ptr(v), int(chunk_bytes), _ptr(pp), pp.size, _ptr(c), _ptr(tags),
                          int(n_threads))
    return c, tags


def mc_decrypt(key, iv_base, chunk_bytes: int, c, tags, n_threads: int = 1):
    """Multi-chain decrypt+verify: -> (plain uint8[len], ok uint32[K])."""
    k, v, cc = _arr(key, 32), _arr(iv_base, 12), _arr(c)
    K = num_chunks(cc.size, chunk_bytes)
    t = _arr(tags, 16 * K)
    p = np.zeros(cc.size, np.uint8)
    ok = np.zeros(K, np.uint32)
    _load().fo_mc_decrypt(_ptr(k), _ptr(v), int(chunk_bytes), _ptr(cc), cc.size, _ptr(t), _ptr(p),
                          _ptr(ok), int(n_threads))
    return p, ok


def mc_encrypt_framed(key, iv_base, chunk_bytes: int, chains_per_sample: int, p, n_threads: int = 1):
    """Multi-chain encrypt with the paper's one-byte serial-number AAD per chunk (k mod chains_per_sample)."""
    k, v, pp = _arr(key, 32), _arr(iv_base, 12), _arr(p)
    K = num_chunks(pp.size, chunk_bytes)
    c = np.zeros(pp.size, np.uint8)
    tags = np.zeros((K, 16), np.uint8)
    _load().fo_mc_encrypt_framed(_ptr(k), _ptr(v), int(chunk_bytes), int(chains_per_sample), _ptr(pp), pp.size,
                                 _ptr(c), _ptr(tags), int(n_threads))
    return c, tags


def mc_decrypt_framed(key, iv_base, chunk_bytes: int, chains_per_sample: int, c, tags, n_threads: int = 1):
    k, v, cc = _arr(key, 32), _arr(iv_base, 12), _arr(c)
    K = num_chunks(cc.size, chunk_bytes)
    t = _arr(tags, 16 * K)
    p = np.zeros(cc.size, np.uint8)
    ok = np.zeros(K, np.uint32)
    _load().fo_mc_decrypt_framed(_ptr(k), _ptr(v), int(chunk_bytes), int(chains_per_sample), _ptr(cc), cc.size,
                                 _ptr(t), _ptr(p), _ptr(ok), int(n_threads))
    return p, ok
