"""GPU-side API and error-path checks of the C ABI."""
import numpy as np
import pytest

import oracle
from paper_2410_15240_b200 import fastrack, synth

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")
if not torch.cuda.is_available():
    pytest.skip("no CUDA device", allow_module_level=True)


def test_context_lifecycle_and_chunk_count():
    rc, ctx = fastrack.fastrack_ctx_create(bytes(32), 65536)
    assert rc == fastrack.OK and ctx
    assert fastrack.fastrack_num_chunks(ctx, 0) == 0
    assert fastrack.fastrack_num_chunks(ctx, 1) == 1
    assert fastrack.fastrack_num_chunks(ctx, 65536) == 1
    assert fastrack.fastrack_num_chunks(ctx, 65537) == 2
    assert fastrack.fastrack_ctx_reserve(ctx, 1 << 30) == fastrack.OK
    assert fastrack.fastrack_last_cuda_error(ctx) == 0
    assert fastrack.fastrack_launch_count(ctx) == 0
    fastrack.fastrack_ctx_destroy(ctx)


def test_argument_errors():
    rc, ctx = fastrack.fastrack_ctx_create(bytes(32), 1024)
    assert rc == fastrack.OK
    buf = torch.zeros(8192, dtype=torch.uint8, device="cuda")
    tags = torch.zeros(16 * 8, dtype=torch.uint8, device="cuda")
    ok = torch.zeros(8, dtype=torch.int32, device="cuda")
    b, t, o = buf.data_ptr(), tags.data_ptr(), ok.data_ptr()
    iv = bytes(12)
    D, E = fastrack.fastrack_decrypt_verify, fastrack.fastrack_encrypt_tag
    assert D(ctx, iv, b, 0, t, b, o, 0) == fastrack.OK                       # len 0: nothing to do
    assert D(ctx, None, b, 1024, t, b, o, 0) == fastrack.ERR_ARG
    assert D(ctx, iv, 0, 1024, t, b, o, 0) == fastrack.ERR_ARG
    assert D(ctx, iv, b, 1024, 0, b, o, 0) == fastrack.ERR_ARG
    assert D(ctx, iv, b, 1024, t, 0, o, 0) == fastrack.ERR_ARG
    assert D(ctx, iv, b, 1024, t, b, 0, 0) == fastrack.ERR_ARG
    assert D(ctx, iv, b + 8, 1024, t, b + 4096, o, 0) == fastrack.ERR_ARG    # misaligned input
    assert D(ctx, iv, b, 1024, t, b + 4096 + 4, o, 0) == fastrack.ERR_ARG    # misaligned output
    assert D(ctx, iv, b, 1024, t + 8, b + 4096, o, 0) == fastrack.ERR_ARG    # misaligned tags
    assert D(ctx, iv, b, 2048, t, b + 1024, o, 0) == fastrack.ERR_ARG        # partial overlap
    assert D(ctx, iv, b + 1024, 2048, t, b, o, 0) == fastrack.ERR_ARG
    assert E(ctx, iv, b, 2048, b + 16, t, 0) == fastrack.ERR_ARG
    assert E(ctx, iv, b, 2048, b, 0, 0) == fastrack.ERR_ARG
    assert D(ctx, iv, b, 2048, t, b + 2048, o, 0) == fastrack.OK             # adjacent, no overlap
    assert D(ctx, iv, b, 2048, t, b, o, 0) == fastrack.OK                    # exact alias = in place
    torch.cuda.synchronize()
    # pipelined: pageable source is refused, stream count is bounded
    pageable = np.zeros(4096, np.uint8)
    h_tags = np.zeros(64, np.uint8)
    P = fastrack.fastrack_pipelined_h2d
    assert P(ctx, iv, pageable.ctypes.data, 4096, h_tags.ctypes.data, b, o, 2) == fastrack.ERR_NOT_PINNED
    pinned = torch.zeros(4096, dtype=torch.uint8).pin_memory()
    assert P(ctx, iv, pinned.data_ptr(), 4096, h_tags.ctypes.data, b, o, 0) == fastrack.ERR_ARG
    assert P(ctx, iv, pinned.data_ptr(), 4096, h_tags.ctypes.data, b, o, 9) == fastrack.ERR_ARG
    assert P(ctx, iv, pinned.data_ptr(), 0, h_tags.ctypes.data, b, o, 2) == fastrack.OK
    assert P(ctx, iv, pinned.data_ptr(), 4096, h_tags.ctypes.data, b, o, 2) == fastrack.OK
    assert fastrack.fastrack_launch_count(ctx) >= 3
    fastrack.fastrack_ctx_destroy(ctx)


def test_calls_are_asynchronous_and_ordered_on_the_stream():
    """encrypt then decrypt queued back to back on one stream without host synchronisation in between."""
    key, iv = synth.key_and_iv(0)
    cb, n = 65536, 4 << 20
    plain = synth.random_bytes(n, 0, salt=21)
    K = n // cb
    with fastrack.Context(key, cb) as ctx:
        d_p = torch.from_numpy(plain).cuda()
        d_c = torch.empty_like(d_p)
        d_back = torch.empty_like(d_p)
        d_t = torch.empty(16 * K, dtype=torch.uint8, device="cuda")
        d_ok = torch.zeros(K, dtype=torch.int32, device="cuda")
        st = torch.cuda.Stream()
        with torch.cuda.stream(st):
            ctx.encrypt_tag(iv, d_p.data_ptr(), n, d_c.data_ptr(), d_t.data_ptr(), st.cuda_stream)
            ctx.decrypt_verify(iv, d_c.data_ptr(), n, d_t.data_ptr(), d_back.data_ptr(), d_ok.data_ptr(), st.cuda_stream)
        st.synchronize()
        assert ctx.launches == 2
        assert bool((d_back == d_p).all()) and bool((d_ok == 1).all())
        c_ref, t_ref = oracle.mc_encrypt(key, iv, cb, plain, oracle.host_threads())
        assert np.array_equal(d_c.cpu().numpy(), c_ref) and np.array_equal(d_t.cpu().numpy().reshape(K, 16), t_ref)


def test_long_dependent_chain_without_host_synchronisation():
    """100 x (encrypt A->B, decrypt B->A, verify-only, in place) queued on one stream with no host sync, on two
    contexts with different keys taking turns: every kernel's table build may overlap its predecessor's tail,
    the data dependencies must still hold."""
    key1, iv = synth.key_and_iv(0)
    key2, _ = synth.key_and_iv(1)
    cb, n = 65536, (2 << 20) + 4096 + 16
    K = (n + cb - 1) // cb
    plain = synth.random_bytes(n, 0, salt=31)
    with fastrack.Context(key1, cb) as c1, fastrack.Context(key2, cb) as c2:
        st = torch.cuda.Stream()
        a = torch.from_numpy(plain).cuda()
        b = torch.empty_like(a)
        tags = torch.empty(16 * K, dtype=torch.uint8, device="cuda")
        oks = torch.zeros(100, K, dtype=torch.int32, device="cuda")
        oks2 = torch.zeros(100, K, dtype=torch.int32, device="cuda")
        torch.cuda.synchronize()
        with torch.cuda.stream(st):
            for i in range(100):
                ctx = c1 if i % 2 == 0 else c2
                ctx.encrypt_tag(iv, a.data_ptr(), n, b.data_ptr(), tags.data_ptr(), st.cuda_stream)
                ctx.verify(iv, b.data_ptr(), n, tags.data_ptr(), oks2[i].data_ptr(), st.cuda_stream)
                a.zero_()                                                   # a torch kernel in between
                ctx.decrypt_verify(iv, b.data_ptr(), n, tags.data_ptr(), a.data_ptr(), oks[i].data_ptr(), st.cuda_stream)
        st.synchronize()
        assert bool((oks == 1).all()) and bool((oks2 == 1).all())
        assert np.array_equal(a.cpu().numpy(), plain)
        c_ref, _ = oracle.mc_encrypt(key2, iv, cb, plain, oracle.host_threads())       # the last round used key 2
        assert np.array_equal(b.cpu().numpy(), c_ref)


def test_contexts_on_concurrent_streams_do_not_interfere():
    """Four contexts (own keys, chunk sizes in both kernel families), each on its own stream, 30 rounds of
    encrypt -> decrypt queued without host synchronisation so that their kernels overlap on the device; every
    context's result must equal the oracle's for its key."""
    shapes = [(65536, (3 << 20) + 100), (1 << 20, (5 << 20) + 16), (256, (1 << 20) + 7), (4096, 2 << 20)]
    iv = synth.key_and_iv(0)[1]
    ctxs, streams, bufs = [], [], []
    try:
        for i, (cb, n) in enumerate(shapes):
            key = synth.key_and_iv(20 + i)[0]
            ctx = fastrack.Context(key, cb)
            K = ctx.num_chunks(n)
            ctx.reserve(n)
            plain = synth.random_bytes(n, 20 + i, salt=41)
            ctxs.append((ctx, key, cb, n, K, plain))
            streams.append(torch.cuda.Stream())
            bufs.append((torch.from_numpy(plain).cuda(), torch.empty(n, dtype=torch.uint8, device="cuda"),
                         torch.empty(n, dtype=torch.uint8, device="cuda"), torch.empty(16 * K, dtype=torch.uint8, device="cuda"),
                         torch.zeros(30, K, dtype=torch.int32, device="cuda")))
        torch.cuda.synchronize()
        for r in range(30):
            for (ctx, key, cb, n, K, plain), st, (d_p, d_c, d_o, d_t, d_ok) in zip(ctxs, streams, bufs):
                ctx.encrypt_tag(iv, d_p.data_ptr(), n, d_c.data_ptr(), d_t.data_ptr(), st.cuda_stream)
                ctx.decrypt_verify(iv, d_c.data_ptr(), n, d_t.data_ptr(), d_o.data_ptr(), d_ok[r].data_ptr(), st.cuda_stream)
        torch.cuda.synchronize()
        for (ctx, key, cb, n, K, plain), (d_p, d_c, d_o, d_t, d_ok) in zip(ctxs, bufs):
            c_ref, t_ref = oracle.mc_encrypt(key, iv, cb, plain, oracle.host_threads())
            assert bool((d_ok == 1).all())
            assert np.array_equal(d_o.cpu().numpy(), plain)
            assert np.array_equal(d_c.cpu().numpy(), c_ref) and np.array_equal(d_t.cpu().numpy().reshape(K, 16), t_ref)
    finally:
        for c in ctxs:
            c[0].close()


def test_option_interface():
    """Unknown options are refused; known ones are accepted at any time and never change results (the layout tests
    cover the latter; here: a call after a change of layout on a live context is still exact)."""
    key, iv = synth.key_and_iv(3)
    cb, n = 4096, 4096 * 37 + 5
    plain = synth.random_bytes(n, 3, salt=1)
    c_ref, t_ref = oracle.mc_encrypt(key, iv, cb, plain, oracle.host_threads())
    K = t_ref.shape[0]
    with fastrack.Context(key, cb) as ctx:
        assert fastrack.fastrack_ctx_set_option(ctx.handle, 0, 1) == fastrack.ERR_ARG
        assert fastrack.fastrack_ctx_set_option(ctx.handle, 99, 1) == fastrack.ERR_ARG
        assert fastrack.fastrack_ctx_set_option(ctx.handle, fastrack.OPT_FOLD_TAIL, 3) == fastrack.ERR_ARG      # 0, 1 or 2
        d_p = torch.from_numpy(plain).cuda()
        d_c = torch.empty_like(d_p)
        d_t = torch.empty(16 * K, dtype=torch.uint8, device="cuda")
        for options in ({}, {fastrack.OPT_PACK_MAX_BLOCKS: 0}, {fastrack.OPT_ROW_SLOTS: 5}, {fastrack.OPT_FOLD_TAIL: 2}, {fastrack.OPT_FOLD_TAIL: 1}, {fastrack.OPT_PACK_MAX_BLOCKS: 4096, fastrack.OPT_PACK_RUN: 7},
                        {fastrack.OPT_PACK_RUN: 0, fastrack.OPT_ROW_SLOTS: 0, fastrack.OPT_GENERIC_SMEM: 1, fastrack.OPT_NO_OVERLAP_LAUNCH: 1}):
            for option, value in options.items():
                ctx.set_option(option, value)
            d_c.zero_(); d_t.zero_()
            ctx.encrypt_tag(iv, d_p.data_ptr(), n, d_c.data_ptr(), d_t.data_ptr(), 0)
            torch.cuda.synchronize()
            assert np.array_equal(d_c.cpu().numpy(), c_ref) and np.array_equal(d_t.cpu().numpy().reshape(K, 16), t_ref)


@pytest.mark.skipif(torch.cuda.device_count() < 2, reason="needs a second GPU to be the wrong current device")
def test_calls_on_the_wrong_current_device_are_refused():
    key, iv = synth.key_and_iv(3)
    torch.cuda.set_device(0)
    with fastrack.Context(key, 4096) as ctx:
        buf = torch.zeros(8192, dtype=torch.uint8, device="cuda:0")
        tags = torch.zeros(32, dtype=torch.uint8, device="cuda:0")
        ok = torch.full((2,), 7, dtype=torch.int32, device="cuda:0")
        torch.cuda.set_device(1)
        try:
            rc = fastrack.fastrack_decrypt_verify(ctx.handle, iv, buf.data_ptr(), 8192, tags.data_ptr(), buf.data_ptr(), ok.data_ptr(), 0)
            assert rc == fastrack.ERR_ARG
            assert fastrack.fastrack_ctr_crypt(ctx.handle, iv, buf.data_ptr(), 8192, buf.data_ptr(), 0) == fastrack.ERR_ARG
        finally:
            torch.cuda.set_device(0)
        torch.cuda.synchronize()
        assert bool((ok == 7).all())
