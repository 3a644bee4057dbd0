"""CPU-side checks of the C-ABI library: it loads, exports what include/fastrack.h declares, and
refuses bad arguments before touching CUDA.  No compute call is made here."""
import ctypes
import os
import re

from paper_2410_15240_b200 import fastrack

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "fastrack.h")).read()
    return sorted(set(re.findall(r"FASTRACK_API\s+[\w\s\*]+?\b(fastrack_\w+)\s*\(", text)))


def test_header_and_binding_agree():
    names = declared_functions()
    assert len(names) >= 23
    assert sorted(fastrack.EXPORTS) == names


def test_every_declared_symbol_is_exported():
    lib = ctypes.CDLL(fastrack.LIB_PATH)
    for name in declared_functions():
        assert hasattr(lib, name), name


def test_error_codes_match_header():
    text = open(os.path.join(ROOT, "include", "fastrack.h")).read()
    codes = dict(re.findall(r"#define\s+(FASTRACK_(?:OK|ERR_\w+))\s+(-?\d+)", text))
    assert int(codes["FASTRACK_OK"]) == fastrack.OK
    assert int(codes["FASTRACK_ERR_ARG"]) == fastrack.ERR_ARG
    assert int(codes["FASTRACK_ERR_CHUNK"]) == fastrack.ERR_CHUNK
    assert int(codes["FASTRACK_ERR_NOT_PINNED"]) == fastrack.ERR_NOT_PINNED
    assert int(codes["FASTRACK_ERR_CUDA"]) == fastrack.ERR_CUDA
    assert int(codes["FASTRACK_ERR_NOMEM"]) == fastrack.ERR_NOMEM
    assert int(codes["FASTRACK_ERR_TOO_MANY"]) == fastrack.ERR_TOO_MANY
    assert int(codes["FASTRACK_ERR_LIMIT"]) == fastrack.ERR_LIMIT
    assert int(re.search(r"#define\s+FASTRACK_NOALLOC_MAX_CHUNKS\s+(\d+)", text).group(1)) == fastrack.NOALLOC_MAX_CHUNKS


def test_argument_checks_that_need_no_device():
    assert fastrack.fastrack_ctx_create(None, 65536) == (fastrack.ERR_ARG, None)
    for bad in (0, 8, 17, 65536 + 1, (1 << 30) + 16):
        assert fastrack.fastrack_ctx_create(bytes(32), bad) == (fastrack.ERR_CHUNK, None)
    assert fastrack.fastrack_num_chunks(None, 100) == 0
    assert fastrack.fastrack_last_cuda_error(None) == 0
    assert fastrack.fastrack_launch_count(None) == 0
    assert fastrack.fastrack_ctx_reserve(None, 1) == fastrack.ERR_ARG
    assert fastrack.fastrack_ctx_set_framing(None, 16) == fastrack.ERR_ARG
    assert fastrack.fastrack_ctx_set_option(None, fastrack.OPT_PACK_RUN, 3) == fastrack.ERR_ARG
    assert fastrack.fastrack_ctx_set_trace(None, 1) == fastrack.ERR_ARG
    assert fastrack.fastrack_ctx_get_trace(None) == []
    assert fastrack.fastrack_decrypt_verify(None, bytes(12), 0, 16, 0, 0, 0, 0) == fastrack.ERR_ARG
    assert fastrack.fastrack_encrypt_tag(None, bytes(12), 0, 16, 0, 0, 0) == fastrack.ERR_ARG
    assert fastrack.fastrack_decrypt_verify_noalloc(None, bytes(12), 0, 16, 0, 0, 0, 0) == fastrack.ERR_ARG
    assert fastrack.fastrack_decrypt_verify_samples(None, 0, 16, 1, 0, 0, 0, 0, 0) == fastrack.ERR_ARG
    assert fastrack.fastrack_encrypt_tag_samples(None, 0, 16, 1, 0, 0, 0, 0) == fastrack.ERR_ARG
    assert fastrack.fastrack_pipelined_h2d_samples(None, 0, 16, 1, 0, 0, 0, 0, 2) == fastrack.ERR_ARG
    assert fastrack.fastrack_ctr_crypt(None, bytes(12), 0, 16, 0, 0) == fastrack.ERR_ARG
    assert fastrack.fastrack_verify(None, bytes(12), 0, 16, 0, 0, 0) == fastrack.ERR_ARG
    assert fastrack.fastrack_keystream(None, bytes(12), 16, 0, 0, 0) == fastrack.ERR_ARG
    assert fastrack.fastrack_verify_sequential(None, bytes(12), 0, 16, 0, 0, 0) == fastrack.ERR_ARG
    assert fastrack.fastrack_xor_verify(None, bytes(12), 0, 16, 0, 0, 0, 0, 0, 0) == fastrack.ERR_ARG
    assert fastrack.fastrack_pipelined_h2d_ahead(None, bytes(12), 0, 16, 0, 0, 0, 0, 2) == fastrack.ERR_ARG
    assert fastrack.fastrack_pipelined_h2d(None, bytes(12), 0, 16, 0, 0, 0, 2) == fastrack.ERR_ARG
    assert fastrack.fastrack_pipelined_d2h(None, bytes(12), 0, 16, 0, 0, 0, 2) == fastrack.ERR_ARG
    fastrack.fastrack_ctx_destroy(None)          # allowed


def test_no_cpu_fallback_without_a_device():
    """Without a CUDA device context creation fails with a CUDA error; it never computes on the host."""
    import torch
    if torch.cuda.is_available():
        return
    rc, handle = fastrack.fastrack_ctx_create(bytes(32), 65536)
    assert rc == fastrack.ERR_CUDA and handle is None
