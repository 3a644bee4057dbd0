"""ctypes binding of the C-ABI CUDA library (see include/fastrack.h for the contract).

Argument marshalling only: every step of the path runs in the library's kernels.  Device and
pinned-host buffers are passed as integer addresses (``tensor.data_ptr()``), streams as the integer
``cudaStream_t`` (``torch.cuda.current_stream().cuda_stream``); ``key`` and ``iv_base`` are bytes.
Importing this module raises if ``libfastrack.so`` has not been built -- there is no fallback.
"""
from __future__ import annotations

import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libfastrack.so")

OK = 0
ERR_ARG, ERR_CHUNK, ERR_NOT_PINNED, ERR_CUDA, ERR_NOMEM, ERR_TOO_MANY, ERR_LIMIT = -1, -2, -3, -4, -5, -6, -7
NOALLOC_MAX_CHUNKS = 16384
MAX_CHUNK_BYTES = 1 << 30

# fastrack_ctx_set_option: test and tuning controls (the library reads no environment variable)
OPT_ROW_SLOTS, OPT_GENERIC_SMEM, OPT_NO_OVERLAP_LAUNCH, OPT_STAGE_BYTES = 1, 2, 3, 4
OPT_DIRECT_SMALL, OPT_PACK_MAX_BLOCKS, OPT_PACK_RUN, OPT_PACK_GROUP, OPT_FOLD_TAIL = 5, 6, 7, 8, 9

EXPORTS = ("fastrack_ctx_create", "fastrack_ctx_destroy", "fastrack_num_chunks", "fastrack_ctx_reserve", "fastrack_ctx_set_option",
           "fastrack_last_cuda_error", "fastrack_decrypt_verify", "fastrack_encrypt_tag",
           "fastrack_pipelined_h2d", "fastrack_launch_count", "fastrack_decrypt_verify_noalloc",
           "fastrack_ctr_crypt", "fastrack_verify", "fastrack_keystream", "fastrack_xor_verify",
           "fastrack_pipelined_h2d_ahead", "fastrack_ctx_set_framing", "fastrack_verify_sequential", "fastrack_pipelined_d2h", "fastrack_ctx_set_trace", "fastrack_ctx_get_trace",
           "fastrack_decrypt_verify_samples", "fastrack_encrypt_tag_samples", "fastrack_pipelined_h2d_samples",
           "fastrack_pipelined_d2h_samples")

if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2410_15240_b200.build` "
                      "(there is no CPU fallback)")

_lib = ctypes.CDLL(LIB_PATH)
_vp, _sz, _int = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int
_lib.fastrack_ctx_create.restype = _int
_lib.fastrack_ctx_create.argtypes = [ctypes.c_char_p, _sz, ctypes.POINTER(_vp)]
_lib.fastrack_ctx_destroy.restype = None
_lib.fastrack_ctx_destroy.argtypes = [_vp]
_lib.fastrack_num_chunks.restype = _sz
_lib.fastrack_num_chunks.argtypes = [_vp, _sz]
_lib.fastrack_ctx_reserve.restype = _int
_lib.fastrack_ctx_reserve.argtypes = [_vp, _sz]
_lib.fastrack_ctx_set_option.restype = _int
_lib.fastrack_ctx_set_option.argtypes = [_vp, _int, ctypes.c_uint64]
_lib.fastrack_ctx_set_framing.restype = _int
_lib.fastrack_ctx_set_framing.argtypes = [_vp, ctypes.c_uint]
class StageTrace(ctypes.Structure):
    _fields_ = [("offset", ctypes.c_size_t), ("bytes", ctypes.c_size_t), ("stream", ctypes.c_int),
                ("copy_start_ms", ctypes.c_float), ("copy_end_ms", ctypes.c_float), ("kernel_end_ms", ctypes.c_float)]


_lib.fastrack_ctx_set_trace.restype = _int
_lib.fastrack_ctx_set_trace.argtypes = [_vp, _int]
_lib.fastrack_ctx_get_trace.restype = _sz
_lib.fastrack_ctx_get_trace.argtypes = [_vp, ctypes.POINTER(StageTrace), _sz]
_lib.fastrack_last_cuda_error.restype = _int
_lib.fastrack_last_cuda_error.argtypes = [_vp]
_lib.fastrack_launch_count.restype = ctypes.c_uint64
_lib.fastrack_launch_count.argtypes = [_vp]
_lib.fastrack_decrypt_verify.restype = _int
_lib.fastrack_decrypt_verify.argtypes = [_vp, ctypes.c_char_p, _vp, _sz, _vp, _vp, _vp, _vp]
_lib.fastrack_decrypt_verify_noalloc.restype = _int
_lib.fastrack_decrypt_verify_noalloc.argtypes = [_vp, ctypes.c_char_p, _vp, _sz, _vp, _vp, _vp, _vp]
_lib.fastrack_encrypt_tag.restype = _int
_lib.fastrack_encrypt_tag.argtypes = [_vp, ctypes.c_char_p, _vp, _sz, _vp, _vp, _vp]
_lib.fastrack_decrypt_verify_samples.restype = _int
_lib.fastrack_decrypt_verify_samples.argtypes = [_vp, _vp, _sz, _sz, _vp, _vp, _vp, _vp, _vp]
_lib.fastrack_encrypt_tag_samples.restype = _int
_lib.fastrack_encrypt_tag_samples.argtypes = [_vp, _vp, _sz, _sz, _vp, _vp, _vp, _vp]
_lib.fastrack_pipelined_h2d_samples.restype = _int
_lib.fastrack_pipelined_h2d_samples.argtypes = [_vp, _vp, _sz, _sz, _vp, _vp, _vp, _vp, _int]
_lib.fastrack_ctr_crypt.restype = _int
_lib.fastrack_ctr_crypt.argtypes = [_vp, ctypes.c_char_p, _vp, _sz, _vp, _vp]
_lib.fastrack_verify.restype = _int
_lib.fastrack_verify.argtypes = [_vp, ctypes.c_char_p, _vp, _sz, _vp, _vp, _vp]
_lib.fastrack_verify_sequential.restype = _int
_lib.fastrack_verify_sequential.argtypes = [_vp, ctypes.c_char_p, _vp, _sz, _vp, _vp, _vp]
_lib.fastrack_keystream.restype = _int
_lib.fastrack_keystream.argtypes = [_vp, ctypes.c_char_p, _sz, _vp, _vp, _vp]
_lib.fastrack_xor_verify.restype = _int
_lib.fastrack_xor_verify.argtypes = [_vp, ctypes.c_char_p, _vp, _sz, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.fastrack_pipelined_h2d_ahead.restype = _int
_lib.fastrack_pipelined_h2d_ahead.argtypes = [_vp, ctypes.c_char_p, _vp, _sz, _vp, _vp, _vp, _vp, _int]
_lib.fastrack_pipelined_d2h.restype = _int
_lib.fastrack_pipelined_d2h.argtypes = [_vp, ctypes.c_char_p, _vp, _sz, _vp, _vp, _vp, _int]
_lib.fastrack_pipelined_d2h_samples.restype = _int
_lib.fastrack_pipelined_d2h_samples.argtypes = [_vp, _vp, _sz, _sz, _vp, _vp, _vp, _vp, _int]
_lib.fastrack_pipelined_h2d.restype = _int
_lib.fastrack_pipelined_h2d.argtypes = [_vp, ctypes.c_char_p, _vp, _sz, _vp, _vp, _vp, _int]


class FastrackError(RuntimeError):
    def __init__(self, code: int, cuda_error: int = 0):
        self.code, self.cuda_error = code, cuda_error
        super().__init__(f"fastrack error {code}" + (f" (CUDA error {cuda_error})" if cuda_error else ""))


def fastrack_ctx_create(key: bytes, chunk_bytes: int):
    """-> (return code, context handle or None)."""
    handle = _vp()
    key_arg = bytes(key) if key is not None else None
    rc = _lib.fastrack_ctx_create(key_arg, chunk_bytes, ctypes.byref(handle))
    return rc, (handle.value if rc == OK else None)


def fastrack_ctx_destroy(ctx) -> None:
    _lib.fastrack_ctx_destroy(ctx)


def fastrack_num_chunks(ctx, length: int) -> int:
    return int(_lib.fastrack_num_chunks(ctx, length))


def fastrack_ctx_reserve(ctx, max_len: int) -> int:
    return _lib.fastrack_ctx_reserve(ctx, max_len)


def fastrack_ctx_set_option(ctx, option: int, value: int) -> int:
    return _lib.fastrack_ctx_set_option(ctx, option, value)


def fastrack_ctx_set_framing(ctx, chains_per_sample: int) -> int:
    return _lib.fastrack_ctx_set_framing(ctx, chains_per_sample)


def fastrack_ctx_set_trace(ctx, enable: int) -> int:
    return _lib.fastrack_ctx_set_trace(ctx, int(enable))


def fastrack_ctx_get_trace(ctx):
    """-> list of dicts, one per stage of the most recent pipelined host->device call."""
    n = int(_lib.fastrack_ctx_get_trace(ctx, None, 0))
    if n == 0:
        return []
    buf = (StageTrace * n)()
    n = int(_lib.fastrack_ctx_get_trace(ctx, buf, n))
    return [{f: getattr(buf[i], f) for f, _ in StageTrace._fields_} for i in range(n)]


def fastrack_last_cuda_error(ctx) -> int:
    return _lib.fastrack_last_cuda_error(ctx)


def fastrack_launch_count(ctx) -> int:
    return int(_lib.fastrack_launch_count(ctx))


def fastrack_decrypt_verify(ctx, iv_base: bytes, d_cipher: int, length: int, d_tags: int, d_plain: int,
                            d_ok: int, stream: int = 0) -> int:
    return _lib.fastrack_decrypt_verify(ctx, iv_base, d_cipher, length, d_tags, d_plain, d_ok, stream)


def fastrack_decrypt_verify_noalloc(ctx, iv_base: bytes, d_cipher: int, length: int, d_tags: int, d_plain: int,
                                    d_ok: int, stream: int = 0) -> int:
    """fastrack_decrypt_verify for callers that must not allocate: fixed scratch inside the library,
    at most NOALLOC_MAX_CHUNKS chunks per call, one call in flight per device at a time."""
    return _lib.fastrack_decrypt_verify_noalloc(ctx, iv_base, d_cipher, length, d_tags, d_plain, d_ok, stream)


def fastrack_encrypt_tag(ctx, iv_base: bytes, d_plain: int, length: int, d_cipher: int, d_tags: int,
                         stream: int = 0) -> int:
    return _lib.fastrack_encrypt_tag(ctx, iv_base, d_plain, length, d_cipher, d_tags, stream)


def fastrack_pipelined_h2d(ctx, iv_base: bytes, h_cipher_pinned: int, length: int, h_tags: int, d_plain: int,
                           d_ok: int, n_streams: int) -> int:
    return _lib.fastrack_pipelined_h2d(ctx, iv_base, h_cipher_pinned, length, h_tags, d_plain, d_ok, n_streams)


def fastrack_decrypt_verify_samples(ctx, d_iv_bases: int, sample_bytes: int, n_samples: int, d_cipher: int, d_tags: int,
                                    d_plain: int, d_ok: int, stream: int = 0) -> int:
    return _lib.fastrack_decrypt_verify_samples(ctx, d_iv_bases, sample_bytes, n_samples, d_cipher, d_tags, d_plain, d_ok,
                                                stream)


def fastrack_encrypt_tag_samples(ctx, d_iv_bases: int, sample_bytes: int, n_samples: int, d_plain: int, d_cipher: int,
                                 d_tags: int, stream: int = 0) -> int:
    return _lib.fastrack_encrypt_tag_samples(ctx, d_iv_bases, sample_bytes, n_samples, d_plain, d_cipher, d_tags, stream)


def fastrack_pipelined_h2d_samples(ctx, h_iv_bases: int, sample_bytes: int, n_samples: int, h_cipher_pinned: int,
                                   h_tags: int, d_plain: int, d_ok: int, n_streams: int) -> int:
    return _lib.fastrack_pipelined_h2d_samples(ctx, h_iv_bases, sample_bytes, n_samples, h_cipher_pinned, h_tags, d_plain,
                                               d_ok, n_streams)


def fastrack_ctr_crypt(ctx, iv_base: bytes, d_in: int, length: int, d_out: int, stream: int = 0) -> int:
    return _lib.fastrack_ctr_crypt(ctx, iv_base, d_in, length, d_out, stream)


def fastrack_verify(ctx, iv_base: bytes, d_cipher: int, length: int, d_tags: int, d_ok: int, stream: int = 0) -> int:
    return _lib.fastrack_verify(ctx, iv_base, d_cipher, length, d_tags, d_ok, stream)


def fastrack_verify_sequential(ctx, iv_base: bytes, d_cipher: int, length: int, d_tags: int, d_ok: int,
                               stream: int = 0) -> int:
    return _lib.fastrack_verify_sequential(ctx, iv_base, d_cipher, length, d_tags, d_ok, stream)


def fastrack_keystream(ctx, iv_base: bytes, length: int, d_pad: int, d_mask: int, stream: int = 0) -> int:
    return _lib.fastrack_keystream(ctx, iv_base, length, d_pad, d_mask, stream)


def fastrack_xor_verify(ctx, iv_base: bytes, d_cipher: int, length: int, d_pad: int, d_mask: int, d_tags: int,
                        d_plain: int, d_ok: int, stream: int = 0) -> int:
    return _lib.fastrack_xor_verify(ctx, iv_base, d_cipher, length, d_pad, d_mask, d_tags, d_plain, d_ok, stream)


def fastrack_pipelined_h2d_ahead(ctx, iv_base: bytes, h_cipher_pinned: int, length: int, h_tags: int, d_pad: int,
                                 d_plain: int, d_ok: int, n_streams: int) -> int:
    return _lib.fastrack_pipelined_h2d_ahead(ctx, iv_base, h_cipher_pinned, length, h_tags, d_pad, d_plain, d_ok,
                                             n_streams)


def fastrack_pipelined_d2h_samples(ctx, h_iv_bases: int, sample_bytes: int, n_samples: int, d_plain: int, d_cipher: int,
                                   h_cipher_pinned: int, h_tags: int, n_streams: int) -> int:
    return _lib.fastrack_pipelined_d2h_samples(ctx, h_iv_bases, sample_bytes, n_samples, d_plain, d_cipher, h_cipher_pinned,
                                               h_tags, n_streams)


def fastrack_pipelined_d2h(ctx, iv_base: bytes, d_plain: int, length: int, d_cipher: int, h_cipher_pinned: int,
                           h_tags: int, n_streams: int) -> int:
    return _lib.fastrack_pipelined_d2h(ctx, iv_base, d_plain, length, d_cipher, h_cipher_pinned, h_tags, n_streams)


class Context:
    """RAII wrapper: ``with Context(key, chunk_bytes) as ctx: ctx.decrypt_verify(...)``; raises FastrackError."""

    def __init__(self, key: bytes, chunk_bytes: int, options=None):
        """options: {OPT_*: value} passed to fastrack_ctx_set_option right after creation (tests, tuning)."""
        rc, handle = fastrack_ctx_create(key, chunk_bytes)
        if rc != OK:
            raise FastrackError(rc)
        self.handle = handle
        self.chunk_bytes = chunk_bytes
        for option, value in (options or {}).items():
            self.set_option(option, value)

    def set_option(self, option: int, value: int) -> None:
        self._check(fastrack_ctx_set_option(self.handle, option, value))

    def _check(self, rc: int) -> None:
        if rc != OK:
            raise FastrackError(rc, fastrack_last_cuda_error(self.handle))

    def num_chunks(self, length: int) -> int:
        return fastrack_num_chunks(self.handle, length)

    def set_framing(self, chains_per_sample: int) -> None:
        self._check(fastrack_ctx_set_framing(self.handle, chains_per_sample))

    def set_trace(self, enable: bool) -> None:
        self._check(fastrack_ctx_set_trace(self.handle, int(enable)))

    def get_trace(self):
        return fastrack_ctx_get_trace(self.handle)

    def reserve(self, max_len: int) -> None:
        self._check(fastrack_ctx_reserve(self.handle, max_len))

    def decrypt_verify(self, iv_base, d_cipher, length, d_tags, d_plain, d_ok, stream=0) -> None:
        self._check(fastrack_decrypt_verify(self.handle, iv_base, d_cipher, length, d_tags, d_plain, d_ok, stream))

    def decrypt_verify_noalloc(self, iv_base, d_cipher, length, d_tags, d_plain, d_ok, stream=0) -> None:
        self._check(fastrack_decrypt_verify_noalloc(self.handle, iv_base, d_cipher, length, d_tags, d_plain, d_ok,
                                                    stream))

    def encrypt_tag(self, iv_base, d_plain, length, d_cipher, d_tags, stream=0) -> None:
        self._check(fastrack_encrypt_tag(self.handle, iv_base, d_plain, length, d_cipher, d_tags, stream))

    def pipelined_h2d(self, iv_base, h_cipher_pinned, length, h_tags, d_plain, d_ok, n_streams=4) -> None:
        self._check(fastrack_pipelined_h2d(self.handle, iv_base, h_cipher_pinned, length, h_tags, d_plain, d_ok,
                                           n_streams))

    def decrypt_verify_samples(self, d_iv_bases, sample_bytes, n_samples, d_cipher, d_tags, d_plain, d_ok, stream=0) -> None:
        self._check(fastrack_decrypt_verify_samples(self.handle, d_iv_bases, sample_bytes, n_samples, d_cipher, d_tags,
                                                    d_plain, d_ok, stream))

    def encrypt_tag_samples(self, d_iv_bases, sample_bytes, n_samples, d_plain, d_cipher, d_tags, stream=0) -> None:
        self._check(fastrack_encrypt_tag_samples(self.handle, d_iv_bases, sample_bytes, n_samples, d_plain, d_cipher,
                                                 d_tags, stream))

    def pipelined_h2d_samples(self, h_iv_bases, sample_bytes, n_samples, h_cipher_pinned, h_tags, d_plain, d_ok,
                              n_streams=4) -> None:
        self._check(fastrack_pipelined_h2d_samples(self.handle, h_iv_bases, sample_bytes, n_samples, h_cipher_pinned, h_tags,
                                                   d_plain, d_ok, n_streams))

    def ctr_crypt(self, iv_base, d_in, length, d_out, stream=0) -> None:
        self._check(fastrack_ctr_crypt(self.handle, iv_base, d_in, length, d_out, stream))

    def verify(self, iv_base, d_cipher, length, d_tags, d_ok, stream=0) -> None:
        self._check(fastrack_verify(self.handle, iv_base, d_cipher, length, d_tags, d_ok, stream))

    def verify_sequential(self, iv_base, d_cipher, length, d_tags, d_ok, stream=0) -> None:
        self._check(fastrack_verify_sequential(self.handle, iv_base, d_cipher, length, d_tags, d_ok, stream))

    def keystream(self, iv_base, length, d_pad, d_mask, stream=0) -> None:
        self._check(fastrack_keystream(self.handle, iv_base, length, d_pad, d_mask, stream))

    def xor_verify(self, iv_base, d_cipher, length, d_pad, d_mask, d_tags, d_plain, d_ok, stream=0) -> None:
        self._check(fastrack_xor_verify(self.handle, iv_base, d_cipher, length, d_pad, d_mask, d_tags, d_plain, d_ok,
                                        stream))

    def pipelined_h2d_ahead(self, iv_base, h_cipher_pinned, length, h_tags, d_pad, d_plain, d_ok, n_streams=4) -> None:
        self._check(fastrack_pipelined_h2d_ahead(self.handle, iv_base, h_cipher_pinned, length, h_tags, d_pad, d_plain,
                                                 d_ok, n_streams))

    def pipelined_d2h(self, iv_base, d_plain, length, d_cipher, h_cipher_pinned, h_tags, n_streams=4) -> None:
        self._check(fastrack_pipelined_d2h(self.handle, iv_base, d_plain, length, d_cipher, h_cipher_pinned, h_tags,
                                           n_streams))

    def pipelined_d2h_samples(self, h_iv_bases, sample_bytes, n_samples, d_plain, d_cipher, h_cipher_pinned, h_tags,
                              n_streams=4) -> None:
        self._check(fastrack_pipelined_d2h_samples(self.handle, h_iv_bases, sample_bytes, n_samples, d_plain, d_cipher,
                                                   h_cipher_pinned, h_tags, n_streams))

    @property
    def launches(self) -> int:
        return fastrack_launch_count(self.handle)

    def close(self) -> None:
        if self.handle is not None:
            fastrack_ctx_destroy(self.handle)
            self.handle = None

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
