"""Helpers for the GPU tests: run the C-ABI entry points on numpy buffers with guard bands.

torch is used for device memory, pinned memory and streams only."""
from __future__ import annotations

import numpy as np
import torch

from paper_2410_15240_b200 import fastrack

PAD = 4096
CANARY = 0xA5


def _guarded(n: int) -> torch.Tensor:
    """Device buffer of n payload bytes with a 4 KiB 0xA5 guard band before and after it."""
    return torch.full((n + 2 * PAD,), CANARY, dtype=torch.uint8, device="cuda")


def _payload(t: torch.Tensor, n: int) -> torch.Tensor:
    return t[PAD:PAD + n]


def _check_guards(t: torch.Tensor, n: int, what: str) -> None:
    assert bool((t[:PAD] == CANARY).all()) and bool((t[PAD + n:] == CANARY).all()), f"{what}: guard band overwritten"


def to_dev(a: np.ndarray) -> torch.Tensor:
    a = np.ascontiguousarray(a).reshape(-1).view(np.uint8)
    g = _guarded(a.size)
    if a.size:
        _payload(g, a.size).copy_(torch.from_numpy(a))
    return g


class Gpu:
    """One library context plus numpy-in / numpy-out wrappers around the three data-path calls."""

    def __init__(self, key: bytes, chunk_bytes: int, options=None):
        self.ctx = fastrack.Context(key, chunk_bytes, options)
        self.cb = chunk_bytes

    def close(self):
        self.ctx.close()

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def decrypt(self, iv: bytes, cipher: np.ndarray, tags: np.ndarray, in_place: bool = False, stream=None):
        n = int(cipher.size)
        K = self.ctx.num_chunks(n)
        d_c = to_dev(cipher)
        d_t = to_dev(tags)
        d_p = d_c if in_place else _guarded(n)
        d_ok = torch.full((K + 2 * PAD // 4,), 0x5A5A5A5A, dtype=torch.int32, device="cuda")
        st = stream if stream is not None else torch.cuda.current_stream()
        self.ctx.decrypt_verify(iv, _payload(d_c, n).data_ptr(), n, _payload(d_t, 16 * K).data_ptr(),
                                _payload(d_p, n).data_ptr(), d_ok[PAD // 4:].data_ptr(), st.cuda_stream)
        st.synchronize()
        _check_guards(d_c, n, "cipher"); _check_guards(d_p, n, "plain"); _check_guards(d_t, 16 * K, "tags")
        okh = d_ok.cpu().numpy().view(np.uint32)
        assert (okh[:PAD // 4] == 0x5A5A5A5A).all() and (okh[PAD // 4 + K:] == 0x5A5A5A5A).all(), "ok: guard overwritten"
        if not in_place and n:
            assert bool((_payload(d_c, n).cpu() == torch.from_numpy(np.ascontiguousarray(cipher).reshape(-1))).all()), \
                "input ciphertext was modified"
        return _payload(d_p, n).cpu().numpy(), okh[PAD // 4:PAD // 4 + K].copy()

    def encrypt(self, iv: bytes, plain: np.ndarray, in_place: bool = False):
        n = int(plain.size)
        K = self.ctx.num_chunks(n)
        d_p = to_dev(plain)
        d_c = d_p if in_place else _guarded(n)
        d_t = _guarded(16 * K)
        st = torch.cuda.current_stream()
        self.ctx.encrypt_tag(iv, _payload(d_p, n).data_ptr(), n, _payload(d_c, n).data_ptr(),
                             _payload(d_t, 16 * K).data_ptr(), st.cuda_stream)
        st.synchronize()
        _check_guards(d_c, n, "cipher"); _check_guards(d_p, n, "plain"); _check_guards(d_t, 16 * K, "tags")
        return _payload(d_c, n).cpu().numpy(), _payload(d_t, 16 * K).cpu().numpy().reshape(K, 16)

    def pipelined(self, iv: bytes, cipher: np.ndarray, tags: np.ndarray, n_streams: int, pinned_tags: bool = False):
        n = int(cipher.size)
        K = self.ctx.num_chunks(n)
        h_c = torch.from_numpy(np.ascontiguousarray(cipher).reshape(-1)).pin_memory()
        h_t = torch.from_numpy(np.ascontiguousarray(tags).reshape(-1).copy())
        if pinned_tags:
            h_t = h_t.pin_memory()
        d_p = _guarded(n)
        d_ok = torch.full((K + 2 * PAD // 4,), 0x5A5A5A5A, dtype=torch.int32, device="cuda")
        torch.cuda.synchronize()
        self.ctx.pipelined_h2d(iv, h_c.data_ptr(), n, h_t.data_ptr(), _payload(d_p, n).data_ptr(),
                               d_ok[PAD // 4:].data_ptr(), n_streams)
        # the call is blocking: results must be complete without any further synchronisation
        _check_guards(d_p, n, "plain")
        okh = d_ok.cpu().numpy().view(np.uint32)
        assert (okh[:PAD // 4] == 0x5A5A5A5A).all() and (okh[PAD // 4 + K:] == 0x5A5A5A5A).all(), "ok: guard overwritten"
        return _payload(d_p, n).cpu().numpy(), okh[PAD // 4:PAD // 4 + K].copy()
