"""GPU parity of the paper-faithful framing (Sections 4.2 / 4.4): every chunk authenticates a one-byte serial
number (its index inside the sample) as AAD.  Checked against the CPU oracle's framed functions."""
import numpy as np
import pytest

import oracle
from paper_2410_15240_b200 import fastrack, synth

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")
if not torch.cuda.is_available():
    pytest.skip("no CUDA device", allow_module_level=True)

NT = oracle.host_threads()


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a).reshape(-1)).cuda()


@pytest.mark.parametrize("n,cb,chains", [(1, 16, 1), (16, 16, 16), (31 * 16, 16, 16), (1000, 64, 3), (70001, 4096, 16),
                                         ((1 << 20) + 5, 65536, 16), (16 * 36864 * 4, 36864, 16), (600 * 1024, 1024, 256),
                                         ((6 << 20) + 77, 1 << 20, 8)])
def test_framed_encrypt_and_decrypt_match_oracle(n, cb, chains):
    key, iv = synth.key_and_iv(3)
    plain = synth.random_bytes(n, 3, salt=n + chains)
    c_ref, t_ref = oracle.mc_encrypt_framed(key, iv, cb, chains, plain, NT)
    K = t_ref.shape[0]
    with fastrack.Context(key, cb) as ctx:
        ctx.set_framing(chains)
        st = torch.cuda.current_stream().cuda_stream
        d_p = dev(plain)
        d_c = torch.empty_like(d_p)
        d_t = torch.empty(16 * K, dtype=torch.uint8, device="cuda")
        ctx.encrypt_tag(iv, d_p.data_ptr(), n, d_c.data_ptr(), d_t.data_ptr(), st)
        torch.cuda.synchronize()
        assert np.array_equal(d_c.cpu().numpy(), c_ref)
        assert np.array_equal(d_t.cpu().numpy().reshape(K, 16), t_ref)

        bad_c, bad_t = c_ref.copy(), t_ref.copy()
        plan = synth.tamper_plan(n, cb, 3, fraction=0.15, salt=n)
        synth.apply_tamper(bad_c, bad_t, cb, plan)
        p_ref, ok_ref = oracle.mc_decrypt_framed(key, iv, cb, chains, bad_c, bad_t, NT)
        d_bc, d_bt = dev(bad_c), dev(bad_t)
        d_o = torch.empty_like(d_bc)
        d_ok = torch.full((K,), 7, dtype=torch.int32, device="cuda")
        ctx.decrypt_verify(iv, d_bc.data_ptr(), n, d_bt.data_ptr(), d_o.data_ptr(), d_ok.data_ptr(), st)
        torch.cuda.synchronize()
        assert np.array_equal(d_ok.cpu().numpy().view(np.uint32), ok_ref)
        assert np.array_equal(d_o.cpu().numpy(), p_ref)

        # the split passes and the fixed-scratch entry point follow the same framing
        d_ok.fill_(7)
        ctx.verify(iv, d_bc.data_ptr(), n, d_bt.data_ptr(), d_ok.data_ptr(), st)
        torch.cuda.synchronize()
        assert np.array_equal(d_ok.cpu().numpy().view(np.uint32), ok_ref)
        if K <= fastrack.NOALLOC_MAX_CHUNKS:
            d_ok.fill_(7)
            ctx.decrypt_verify_noalloc(iv, d_bc.data_ptr(), n, d_bt.data_ptr(), d_o.data_ptr(), d_ok.data_ptr(), st)
            torch.cuda.synchronize()
            assert np.array_equal(d_ok.cpu().numpy().view(np.uint32), ok_ref)

        # a receiver with another framing rejects every chunk; switching back accepts again
        ctx.set_framing(0)
        d_ok.fill_(7)
        ctx.decrypt_verify(iv, dev(c_ref).data_ptr(), n, dev(t_ref).data_ptr(), d_o.data_ptr(), d_ok.data_ptr(), st)
        torch.cuda.synchronize()
        assert bool((d_ok == 0).all())


def test_framed_reordering_inside_a_sample_is_rejected():
    """Section 4.4: chunks X_i, X_j of one sample swapped together with their tags."""
    key, iv = synth.key_and_iv(3)
    cb, chains, n = 8192, 16, 8192 * 32
    plain = synth.random_bytes(n, 3, salt=1)
    c, t = oracle.mc_encrypt_framed(key, iv, cb, chains, plain, NT)
    sc, stg = c.copy(), t.copy()
    sc[4 * cb:5 * cb], sc[9 * cb:10 * cb] = c[9 * cb:10 * cb], c[4 * cb:5 * cb]
    stg[4], stg[9] = t[9], t[4]
    _, ok_ref = oracle.mc_decrypt_framed(key, iv, cb, chains, sc, stg, NT)
    with fastrack.Context(key, cb) as ctx:
        ctx.set_framing(chains)
        d_c, d_t = dev(sc), dev(stg)
        d_ok = torch.zeros(32, dtype=torch.int32, device="cuda")
        ctx.decrypt_verify(iv, d_c.data_ptr(), n, d_t.data_ptr(), d_c.data_ptr(), d_ok.data_ptr(), 0)
        torch.cuda.synchronize()
    ok = d_ok.cpu().numpy().view(np.uint32)
    assert np.array_equal(ok, ok_ref) and [int(k) for k in np.flatnonzero(ok == 0)] == [4, 9]


@pytest.mark.parametrize("ahead", [False, True])
def test_framed_pipelined_h2d(ahead):
    """Stages start at chunk indices that are not multiples of the sample size: the serial number must follow."""
    key, iv = synth.key_and_iv(3)
    cb, chains, n = 192 * 1024, 5, (11 << 20) + 12345
    plain = synth.random_bytes(n, 3, salt=2)
    c, t = oracle.mc_encrypt_framed(key, iv, cb, chains, plain, NT)
    plan = synth.tamper_plan(n, cb, 3, fraction=0.1, salt=2)
    synth.apply_tamper(c, t, cb, plan)
    p_ref, ok_ref = oracle.mc_decrypt_framed(key, iv, cb, chains, c, t, NT)
    K = ok_ref.size
    with fastrack.Context(key, cb) as ctx:
        ctx.set_framing(chains)
        h_c, h_t = torch.from_numpy(c).pin_memory(), torch.from_numpy(t.reshape(-1).copy())
        d_p = torch.empty(n, dtype=torch.uint8, device="cuda")
        d_pad = torch.empty(n, dtype=torch.uint8, device="cuda")
        d_ok = torch.full((K,), 7, dtype=torch.int32, device="cuda")
        torch.cuda.synchronize()
        if ahead:
            ctx.pipelined_h2d_ahead(iv, h_c.data_ptr(), n, h_t.data_ptr(), d_pad.data_ptr(), d_p.data_ptr(), d_ok.data_ptr(), 3)
        else:
            ctx.pipelined_h2d(iv, h_c.data_ptr(), n, h_t.data_ptr(), d_p.data_ptr(), d_ok.data_ptr(), 3)
        assert np.array_equal(d_ok.cpu().numpy().view(np.uint32), ok_ref)
        assert np.array_equal(d_p.cpu().numpy(), p_ref)


def test_framing_argument_range():
    rc, ctx = fastrack.fastrack_ctx_create(bytes(32), 1024)
    assert rc == fastrack.OK
    assert fastrack.fastrack_ctx_set_framing(ctx, 257) == fastrack.ERR_ARG
    assert fastrack.fastrack_ctx_set_framing(ctx, 256) == fastrack.OK
    assert fastrack.fastrack_ctx_set_framing(ctx, 0) == fastrack.OK
    fastrack.fastrack_ctx_destroy(ctx)


@pytest.mark.parametrize("sample_bytes,cb,n_samples,chains", [(16, 16, 1, 0), (64, 16, 3, 0), (1040, 1024, 5, 16),
                                                               (301056, 301056 // 16 // 16 * 16, 64, 16),     # ResNet-style batch
                                                               (301056, 65536, 64, 0), (1 << 20, 1 << 16, 9, 16)])
def test_batch_of_samples_each_under_its_own_iv(sample_bytes, cb, n_samples, chains):
    """Paper Section 4.2: every input sample is split into n chunks with n tags, and the user encrypted every
    sample on its own.  One launch over the batch must equal one oracle multi-chain call per sample."""
    key, _ = synth.key_and_iv(3)
    rng = np.random.Generator(np.random.PCG64(sample_bytes + n_samples))
    ivs = np.frombuffer(rng.bytes(12 * n_samples), np.uint8).copy()
    n = sample_bytes * n_samples
    plain = synth.random_bytes(n, 3, salt=n_samples)
    cs, ts = [], []
    for s in range(n_samples):
        part, iv = plain[s * sample_bytes:(s + 1) * sample_bytes], ivs[12 * s:12 * s + 12].tobytes()
        c1, t1 = (oracle.mc_encrypt_framed(key, iv, cb, chains, part, NT) if chains else oracle.mc_encrypt(key, iv, cb, part, NT))
        cs.append(c1)
        ts.append(t1)
    c_ref, t_ref = np.concatenate(cs), np.concatenate(ts)
    K = t_ref.shape[0]
    with fastrack.Context(key, cb) as ctx:
        ctx.set_framing(chains)
        st = torch.cuda.current_stream().cuda_stream
        # the IV bases need no alignment: odd sample counts get them at an odd address (byte loads), the others at an
        # aligned one (word loads)
        iv_store = torch.zeros(12 * n_samples + 4, dtype=torch.uint8, device="cuda")
        d_iv = iv_store[n_samples % 2:n_samples % 2 + 12 * n_samples]
        d_iv.copy_(torch.from_numpy(ivs))
        assert d_iv.data_ptr() % 4 == n_samples % 2
        d_p = dev(plain)
        d_c = torch.empty_like(d_p)
        d_t = torch.empty(16 * K, dtype=torch.uint8, device="cuda")
        ctx.encrypt_tag_samples(d_iv.data_ptr(), sample_bytes, n_samples, d_p.data_ptr(), d_c.data_ptr(), d_t.data_ptr(), st)
        torch.cuda.synchronize()
        assert np.array_equal(d_c.cpu().numpy(), c_ref)
        assert np.array_equal(d_t.cpu().numpy().reshape(K, 16), t_ref)

        bad_c, bad_t = c_ref.copy(), t_ref.copy()
        hits = sorted({0, K // 2, K - 1})
        for i, k in enumerate(hits):
            if i % 2:
                bad_t[k, 5] ^= 0x40
            else:
                sample, kk = divmod(k, K // n_samples)
                bad_c[sample * sample_bytes + kk * cb] ^= 1
        d_bc, d_bt = dev(bad_c), dev(bad_t)
        d_ok = torch.full((K,), 7, dtype=torch.int32, device="cuda")
        ctx.decrypt_verify_samples(d_iv.data_ptr(), sample_bytes, n_samples, d_bc.data_ptr(), d_bt.data_ptr(), d_bc.data_ptr(),
                                   d_ok.data_ptr(), st)                                       # in place
        torch.cuda.synchronize()
        ok = d_ok.cpu().numpy().view(np.uint32)
        assert [int(k) for k in np.flatnonzero(ok == 0)] == hits
        out = d_bc.cpu().numpy()
        diff = np.flatnonzero(out != plain)
        assert diff.size == len([1 for i in range(len(hits)) if i % 2 == 0])                   # one flipped bit per ciphertext hit
        # the oracle agrees sample by sample
        for s in (0, n_samples - 1):
            iv = ivs[12 * s:12 * s + 12].tobytes()
            lo, cps = s * sample_bytes, K // n_samples
            args = (key, iv, cb) + ((chains,) if chains else ()) + (bad_c[lo:lo + sample_bytes], bad_t[s * cps:(s + 1) * cps], NT)
            p_s, ok_s = (oracle.mc_decrypt_framed(*args) if chains else oracle.mc_decrypt(*args))
            assert np.array_equal(ok_s, ok[s * cps:(s + 1) * cps]) and np.array_equal(p_s, out[lo:lo + sample_bytes])


def test_sample_batch_argument_errors():
    rc, ctx = fastrack.fastrack_ctx_create(bytes(32), 1024)
    assert rc == fastrack.OK
    buf = torch.zeros(8192, dtype=torch.uint8, device="cuda")
    ivs = torch.zeros(96, dtype=torch.uint8, device="cuda")
    tags = torch.zeros(256, dtype=torch.uint8, device="cuda")
    ok = torch.zeros(16, dtype=torch.int32, device="cuda")
    b, i, t, o = buf.data_ptr(), ivs.data_ptr(), tags.data_ptr(), ok.data_ptr()
    D = fastrack.fastrack_decrypt_verify_samples
    assert D(ctx, i, 1024, 0, b, t, b, o, 0) == fastrack.OK                 # empty batch
    assert D(ctx, 0, 1024, 2, b, t, b, o, 0) == fastrack.ERR_ARG            # no IVs
    assert D(ctx, i, 1000, 2, b, t, b, o, 0) == fastrack.ERR_ARG            # sample size not a multiple of 16
    assert D(ctx, i, 0, 2, b, t, b, o, 0) == fastrack.ERR_ARG
    assert D(ctx, i, 1024, 2, b, t, b + 16, o, 0) == fastrack.ERR_ARG       # partial overlap
    assert D(ctx, i, 1536, 2, b, t, b + 4096, o, 0) == fastrack.OK          # 2 samples x 2 chunks (1024 + 512)
    torch.cuda.synchronize()
    fastrack.fastrack_ctx_destroy(ctx)


@pytest.mark.parametrize("sample_bytes,cb,n_samples,chains,n_streams", [(1040, 1024, 5, 16, 1), (301056, 18816, 64, 16, 3),
                                                                        (1 << 20, 1 << 16, 9, 0, 2)])
def test_pipelined_h2d_of_a_batch_of_samples(sample_bytes, cb, n_samples, chains, n_streams):
    """The inference input path of the paper: an encrypted batch of samples arrives in pinned host memory."""
    key, _ = synth.key_and_iv(3)
    rng = np.random.Generator(np.random.PCG64(sample_bytes + n_samples + 1))
    ivs = np.frombuffer(rng.bytes(12 * n_samples), np.uint8).copy()
    n = sample_bytes * n_samples
    plain = synth.random_bytes(n, 3, salt=n_samples + 100)
    cs, ts = [], []
    for s in range(n_samples):
        part, iv = plain[s * sample_bytes:(s + 1) * sample_bytes], ivs[12 * s:12 * s + 12].tobytes()
        c1, t1 = (oracle.mc_encrypt_framed(key, iv, cb, chains, part, NT) if chains else oracle.mc_encrypt(key, iv, cb, part, NT))
        cs.append(c1)
        ts.append(t1)
    c, t = np.concatenate(cs), np.concatenate(ts)
    K = t.shape[0]
    t[K // 3, 2] ^= 8
    c[n - 1] ^= 0x80
    with fastrack.Context(key, cb) as ctx:
        ctx.set_framing(chains)
        h_c = torch.from_numpy(c).pin_memory()
        h_t = torch.from_numpy(t.reshape(-1).copy())
        d_p = torch.empty(n, dtype=torch.uint8, device="cuda")
        d_ok = torch.full((K,), 7, dtype=torch.int32, device="cuda")
        torch.cuda.synchronize()
        for _ in range(2):
            ctx.pipelined_h2d_samples(ivs.ctypes.data, sample_bytes, n_samples, h_c.data_ptr(), h_t.data_ptr(), d_p.data_ptr(),
                                      d_ok.data_ptr(), n_streams)
            ok = d_ok.cpu().numpy().view(np.uint32)
            assert [int(k) for k in np.flatnonzero(ok == 0)] == sorted({K // 3, K - 1})
            out = d_p.cpu().numpy()
            assert np.flatnonzero(out != plain).tolist() == [n - 1]


@pytest.mark.parametrize("sample_bytes,cb,n_samples,chains,n_streams,in_place",
                         [(1040, 1024, 5, 16, 1, False), (301056, 18816, 64, 16, 3, False), (1 << 20, 1 << 16, 9, 0, 2, True),
                          (400, 400, 30000, 0, 4, False), (4096, 256, 3000, 16, 2, True)])
def test_pipelined_d2h_of_a_batch_of_samples(sample_bytes, cb, n_samples, chains, n_streams, in_place):
    """The outbound mirror: a batch of results leaves the GPU, every sample encrypted and tagged under its own IV base,
    the device-to-host copies overlapped with the kernels.  Ciphertext and tags must equal the oracle's per sample."""
    key, _ = synth.key_and_iv(3)
    rng = np.random.Generator(np.random.PCG64(sample_bytes + n_samples + 2))
    ivs = np.frombuffer(rng.bytes(12 * n_samples), np.uint8).copy()
    n = sample_bytes * n_samples
    plain = synth.random_bytes(n, 3, salt=n_samples + 200)
    cs, ts = [], []
    for s in range(n_samples):
        part, iv = plain[s * sample_bytes:(s + 1) * sample_bytes], ivs[12 * s:12 * s + 12].tobytes()
        c1, t1 = (oracle.mc_encrypt_framed(key, iv, cb, chains, part, 1) if chains else oracle.mc_encrypt(key, iv, cb, part, 1))
        cs.append(c1)
        ts.append(t1)
    c_ref, t_ref = np.concatenate(cs), np.concatenate(ts)
    K = t_ref.shape[0]
    with fastrack.Context(key, cb) as ctx:
        ctx.set_framing(chains)
        h_c = torch.full((n + 64,), 0xA5, dtype=torch.uint8).pin_memory()
        h_t = np.full(16 * K + 64, 0xA5, np.uint8)
        for rep in range(2):
            d_p = torch.from_numpy(plain).cuda()
            d_c = d_p if in_place else torch.empty_like(d_p)
            torch.cuda.synchronize()
            ctx.pipelined_d2h_samples(ivs.ctypes.data, sample_bytes, n_samples, d_p.data_ptr(), d_c.data_ptr(),
                                      h_c[32:].data_ptr(), h_t[32:].ctypes.data, n_streams)
            # blocking call: the host buffers are complete now
            assert np.array_equal(h_c[32:32 + n].numpy(), c_ref), f"rep {rep}"
            assert np.array_equal(h_t[32:32 + 16 * K].reshape(K, 16), t_ref), f"rep {rep}"
            assert bool((h_c[:32] == 0xA5).all()) and bool((h_c[32 + n:] == 0xA5).all())
            assert (h_t[:32] == 0xA5).all() and (h_t[32 + 16 * K:] == 0xA5).all()
            if not in_place:
                assert np.array_equal(d_p.cpu().numpy(), plain)
            h_c[32:32 + n] = 0
            h_t[32:32 + 16 * K] = 0
    rc, raw = fastrack.fastrack_ctx_create(key, cb)
    assert rc == fastrack.OK
    buf = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    pinned = torch.zeros(4096, dtype=torch.uint8).pin_memory()
    tags = np.zeros(4096, np.uint8)
    D = fastrack.fastrack_pipelined_d2h_samples
    assert D(raw, None, 1024, 2, buf.data_ptr(), buf.data_ptr(), pinned.data_ptr(), tags.ctypes.data, 2) == fastrack.ERR_ARG
    assert D(raw, ivs.ctypes.data, 1000, 2, buf.data_ptr(), buf.data_ptr(), pinned.data_ptr(), tags.ctypes.data, 2) == fastrack.ERR_ARG
    assert D(raw, ivs.ctypes.data, 1024, 2, buf.data_ptr(), buf.data_ptr(), tags.ctypes.data, tags.ctypes.data, 2) == fastrack.ERR_NOT_PINNED
    assert D(raw, ivs.ctypes.data, 1024, 0, buf.data_ptr(), buf.data_ptr(), pinned.data_ptr(), tags.ctypes.data, 2) == fastrack.OK
    fastrack.fastrack_ctx_destroy(raw)
