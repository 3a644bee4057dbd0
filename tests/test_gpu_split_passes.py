"""GPU parity of the split passes (paper Section 4.3): decrypt-only + verify-only (eager evaluation) and
keystream-ahead + XOR/verify (parallel AES evaluation), each against the CPU oracle."""
import numpy as np
import pytest

import oracle
from paper_2410_15240_b200 import fastrack, synth

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")
if not torch.cuda.is_available():
    pytest.skip("no CUDA device", allow_module_level=True)

NT = oracle.host_threads()
CASES = [(1, 16), (17, 64), (1000, 256), (4096, 4096), (70001, 16384), ((1 << 20) + 33, 65536),
         (3 * (1 << 20) + 4321, 1 << 20), ((9 << 20) + 12345, 4 << 20)]


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a).reshape(-1)).cuda()


@pytest.mark.parametrize("n,cb", CASES)
def test_ctr_crypt_then_verify_equals_oracle(n, cb):
    key, iv = synth.key_and_iv(1)
    plain = synth.random_bytes(n, 1, salt=n)
    c, t = oracle.mc_encrypt(key, iv, cb, plain, NT)
    plan = synth.tamper_plan(n, cb, 1, fraction=0.2, salt=n)
    synth.apply_tamper(c, t, cb, plan)
    p_ref, ok_ref = oracle.mc_decrypt(key, iv, cb, c, t, NT)
    K = ok_ref.size
    with fastrack.Context(key, cb) as ctx:
        st = torch.cuda.current_stream().cuda_stream
        d_c, d_t = dev(c), dev(t)
        d_p = torch.empty_like(d_c)
        d_ok = torch.full((K,), 7, dtype=torch.int32, device="cuda")
        ctx.ctr_crypt(iv, d_c.data_ptr(), n, d_p.data_ptr(), st)                 # plaintext first ...
        torch.cuda.synchronize()
        assert np.array_equal(d_p.cpu().numpy(), p_ref)
        assert bool((d_ok == 7).all())                                            # ... no verdict yet
        ctx.verify(iv, d_c.data_ptr(), n, d_t.data_ptr(), d_ok.data_ptr(), st)    # ... verdict later
        torch.cuda.synchronize()
        assert np.array_equal(d_ok.cpu().numpy().view(np.uint32), ok_ref)
        assert np.array_equal(d_c.cpu().numpy(), c)                               # verify leaves the ciphertext alone
        # ctr_crypt is its own inverse, also in place
        ctx.ctr_crypt(iv, d_p.data_ptr(), n, d_p.data_ptr(), st)
        torch.cuda.synchronize()
        assert np.array_equal(d_p.cpu().numpy(), c)


def test_deferred_verify_overlaps_next_buffer_on_another_stream():
    """verify of buffer A on a side stream while buffer B is decrypted+verified on the main stream."""
    key, iv = synth.key_and_iv(1)
    iv_b = synth.fresh_iv(1)
    cb, n = 65536, 8 << 20
    pa, pb = synth.random_bytes(n, 1, salt=1), synth.random_bytes(n, 1, salt=2)
    ca, ta = oracle.mc_encrypt(key, iv, cb, pa, NT)
    cbuf, tb = oracle.mc_encrypt(key, iv_b, cb, pb, NT)
    synth.apply_tamper(ca, ta, cb, [(3, "cipher", 5), (100, "tag", 9)])
    synth.apply_tamper(cbuf, tb, cb, [(7, "tag", 1)])
    K = n // cb
    with fastrack.Context(key, cb) as ctx:
        ctx.reserve(n)
        side, main = torch.cuda.Stream(), torch.cuda.Stream()
        d_ca, d_ta, d_cb, d_tb = dev(ca), dev(ta), dev(cbuf), dev(tb)
        d_pb = torch.empty_like(d_cb)
        ok_a = torch.full((K,), 7, dtype=torch.int32, device="cuda")
        ok_b = torch.full((K,), 7, dtype=torch.int32, device="cuda")
        torch.cuda.synchronize()
        for _ in range(3):
            ctx.verify(iv, d_ca.data_ptr(), n, d_ta.data_ptr(), ok_a.data_ptr(), side.cuda_stream)
            ctx.decrypt_verify(iv_b, d_cb.data_ptr(), n, d_tb.data_ptr(), d_pb.data_ptr(), ok_b.data_ptr(), main.cuda_stream)
        torch.cuda.synchronize()
        exp_a = np.ones(K, np.uint32); exp_a[[3, 100]] = 0
        exp_b = np.ones(K, np.uint32); exp_b[7] = 0
        assert np.array_equal(ok_a.cpu().numpy().view(np.uint32), exp_a)
        assert np.array_equal(ok_b.cpu().numpy().view(np.uint32), exp_b)
        assert np.array_equal(d_pb.cpu().numpy(), pb)


@pytest.mark.parametrize("n,cb", CASES)
def test_keystream_ahead_then_xor_verify_equals_oracle(n, cb):
    key, iv = synth.key_and_iv(2)
    plain = synth.random_bytes(n, 2, salt=n)
    c, t = oracle.mc_encrypt(key, iv, cb, plain, NT)
    plan = synth.tamper_plan(n, cb, 2, fraction=0.2, salt=n)
    synth.apply_tamper(c, t, cb, plan)
    p_ref, ok_ref = oracle.mc_decrypt(key, iv, cb, c, t, NT)
    K = ok_ref.size
    # the pad is the encryption of zeros; the mask of chunk k is E_K(IV_k || 1)
    pad_ref, _ = oracle.mc_encrypt(key, iv, cb, np.zeros(n, np.uint8), NT)
    mask_ref = np.stack([np.frombuffer(oracle.aes256_encrypt_block(key, oracle.chunk_iv(iv, k) + bytes([0, 0, 0, 1])), np.uint8)
                         for k in range(K)])
    with fastrack.Context(key, cb) as ctx:
        st = torch.cuda.current_stream().cuda_stream
        d_pad = torch.full((n,), 0xEE, dtype=torch.uint8, device="cuda")
        d_mask = torch.zeros(16 * K, dtype=torch.uint8, device="cuda")
        ctx.keystream(iv, n, d_pad.data_ptr(), d_mask.data_ptr(), st)
        torch.cuda.synchronize()
        assert np.array_equal(d_pad.cpu().numpy(), pad_ref)
        assert np.array_equal(d_mask.cpu().numpy().reshape(K, 16), mask_ref)
        d_c, d_t = dev(c), dev(t)
        d_ok = torch.full((K,), 7, dtype=torch.int32, device="cuda")
        ctx.xor_verify(iv, d_c.data_ptr(), n, d_pad.data_ptr(), d_mask.data_ptr(), d_t.data_ptr(), d_c.data_ptr(),
                       d_ok.data_ptr(), st)                                      # in place
        torch.cuda.synchronize()
        assert np.array_equal(d_ok.cpu().numpy().view(np.uint32), ok_ref)
        assert np.array_equal(d_c.cpu().numpy(), p_ref)


@pytest.mark.parametrize("n,cb,n_streams", [(100, 1024, 1), ((1 << 20) + 17, 65536, 2), ((9 << 20) + 12345, 256 * 1024, 3),
                                             (77_070_336, 4 << 20, 4)])
def test_pipelined_keystream_ahead_matches_oracle(n, cb, n_streams):
    key, iv = synth.key_and_iv(2)
    plain = synth.fp16_image_batch() if n == 77_070_336 else synth.random_bytes(n, 2, salt=n + 1)
    c, t = oracle.mc_encrypt(key, iv, cb, plain, NT)
    plan = synth.tamper_plan(n, cb, 2, fraction=0.1, salt=n + 1)
    synth.apply_tamper(c, t, cb, plan)
    p_ref, ok_ref = oracle.mc_decrypt(key, iv, cb, c, t, NT)
    K = ok_ref.size
    with fastrack.Context(key, cb) as ctx:
        h_c = torch.from_numpy(c).pin_memory()
        h_t = torch.from_numpy(t.reshape(-1).copy())
        d_pad = torch.empty(n, dtype=torch.uint8, device="cuda")
        d_p = torch.empty(n, dtype=torch.uint8, device="cuda")
        d_ok = torch.full((K,), 7, dtype=torch.int32, device="cuda")
        torch.cuda.synchronize()
        for _ in range(2):
            ctx.pipelined_h2d_ahead(iv, h_c.data_ptr(), n, h_t.data_ptr(), d_pad.data_ptr(), d_p.data_ptr(),
                                    d_ok.data_ptr(), n_streams)
            assert np.array_equal(d_ok.cpu().numpy().view(np.uint32), ok_ref)
            assert np.array_equal(d_p.cpu().numpy(), p_ref)


def test_split_pass_argument_errors():
    rc, ctx = fastrack.fastrack_ctx_create(bytes(32), 1024)
    assert rc == fastrack.OK
    buf = torch.zeros(8192, dtype=torch.uint8, device="cuda")
    small = torch.zeros(256, dtype=torch.uint8, device="cuda")
    ok = torch.zeros(8, dtype=torch.int32, device="cuda")
    b, t, o, iv = buf.data_ptr(), small.data_ptr(), ok.data_ptr(), bytes(12)
    assert fastrack.fastrack_ctr_crypt(ctx, iv, b, 0, b, 0) == fastrack.OK
    assert fastrack.fastrack_ctr_crypt(ctx, iv, 0, 16, b, 0) == fastrack.ERR_ARG
    assert fastrack.fastrack_ctr_crypt(ctx, iv, b, 2048, b + 16, 0) == fastrack.ERR_ARG
    assert fastrack.fastrack_verify(ctx, iv, b, 1024, 0, o, 0) == fastrack.ERR_ARG
    assert fastrack.fastrack_verify(ctx, iv, b + 4, 1024, t, o, 0) == fastrack.ERR_ARG
    assert fastrack.fastrack_keystream(ctx, iv, 1024, 0, t, 0) == fastrack.ERR_ARG
    assert fastrack.fastrack_keystream(ctx, iv, 1024, b, 0, 0) == fastrack.ERR_ARG
    assert fastrack.fastrack_xor_verify(ctx, iv, b, 1024, b, t, t + 128, b, o, 0) == fastrack.ERR_ARG      # pad == plain
    assert fastrack.fastrack_xor_verify(ctx, iv, b, 1024, b + 4096, t, t + 128, b, o, 0) == fastrack.OK
    pinned = torch.zeros(4096, dtype=torch.uint8).pin_memory()
    h_tags = np.zeros(64, np.uint8)
    A = fastrack.fastrack_pipelined_h2d_ahead
    assert A(ctx, iv, pinned.data_ptr(), 4096, h_tags.ctypes.data, 0, b, o, 2) == fastrack.ERR_ARG
    assert A(ctx, iv, pinned.data_ptr(), 4096, h_tags.ctypes.data, b, b, o, 2) == fastrack.ERR_ARG
    assert A(ctx, iv, pinned.data_ptr(), 4096, h_tags.ctypes.data, b + 4096, b, o, 2) == fastrack.OK
    torch.cuda.synchronize()
    fastrack.fastrack_ctx_destroy(ctx)


@pytest.mark.parametrize("n,cb,chains", [(1, 16, 0), (1000, 64, 0), (70001, 4096, 0), ((1 << 20) + 5, 65536, 0),
                                         (200 * 1024 + 9, 1024, 0), (70001, 4096, 16), (33 * 160 + 3, 160, 3)])
def test_sequential_chain_comparator_gives_the_same_verdicts(n, cb, chains):
    """The one-thread-per-chain kernel (the paper's starting point) must agree with the oracle as well."""
    key, iv = synth.key_and_iv(1)
    plain = synth.random_bytes(n, 1, salt=n + 7)
    if chains:
        c, t = oracle.mc_encrypt_framed(key, iv, cb, chains, plain, NT)
    else:
        c, t = oracle.mc_encrypt(key, iv, cb, plain, NT)
    plan = synth.tamper_plan(n, cb, 1, fraction=0.2, salt=n + 7)
    synth.apply_tamper(c, t, cb, plan)
    if chains:
        _, ok_ref = oracle.mc_decrypt_framed(key, iv, cb, chains, c, t, NT)
    else:
        _, ok_ref = oracle.mc_decrypt(key, iv, cb, c, t, NT)
    K = ok_ref.size
    with fastrack.Context(key, cb) as ctx:
        ctx.set_framing(chains)
        d_c, d_t = dev(c), dev(t)
        d_ok = torch.full((K,), 7, dtype=torch.int32, device="cuda")
        ctx.verify_sequential(iv, d_c.data_ptr(), n, d_t.data_ptr(), d_ok.data_ptr(), torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        assert np.array_equal(d_ok.cpu().numpy().view(np.uint32), ok_ref)
        assert np.array_equal(d_c.cpu().numpy(), c)


def test_counter_mode_only_as_first_call_on_a_context():
    """The pass without authentication as the very first call on a fresh context, with thousands of chunks that are
    cut between warps (row kernels forced): it needs nothing that an earlier call would have set up."""
    key, iv = synth.key_and_iv(6)
    cb, n = 4096, 4096 * 3000 + 77
    plain = synth.random_bytes(n, 6, salt=5)
    c_ref, _ = oracle.mc_encrypt(key, iv, cb, plain, oracle.host_threads())
    with fastrack.Context(key, cb, {fastrack.OPT_PACK_MAX_BLOCKS: 0}) as ctx:
        d_p = torch.from_numpy(plain).cuda()
        d_c = torch.empty_like(d_p)
        ctx.ctr_crypt(iv, d_p.data_ptr(), n, d_c.data_ptr(), 0)          # first call on the context
        torch.cuda.synchronize()
        assert np.array_equal(d_c.cpu().numpy(), c_ref)
