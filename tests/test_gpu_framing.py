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
