"""GPU parity of the packed-row kernels: launches with many chunks that are not large give every LANE a short run of
one chunk's counters instead of giving a warp 32 consecutive blocks (paper Section 4.2 leaves the chunk size open;
batches of small samples -- table rows, node features -- make chunks of tens of bytes).  Every case runs with the
row kernels only, with the planner's own choice, and with several forced packings, and all must equal the oracle:
the two kernel families share no reduction code, so each also checks the other."""
import numpy as np
import pytest

import oracle
from gpu_harness import Gpu
from paper_2410_15240_b200 import fastrack, synth

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")
if not torch.cuda.is_available():
    pytest.skip("no CUDA device", allow_module_level=True)

NT = oracle.host_threads()


FAMILIES = {      # kernel layouts forced through fastrack_ctx_set_option
    "general": {fastrack.OPT_PACK_MAX_BLOCKS: 0},                                  # row kernels only
    "general-every-warp": {fastrack.OPT_PACK_MAX_BLOCKS: 0, fastrack.OPT_ROW_SLOTS: 148 * 32},   # ... rows spread as thinly as they go
    "general-37-warps": {fastrack.OPT_PACK_MAX_BLOCKS: 0, fastrack.OPT_ROW_SLOTS: 37},   # ... chunks shared between warps and CTAs
    "general-folded": {fastrack.OPT_PACK_MAX_BLOCKS: 0, fastrack.OPT_FOLD_TAIL: 2},  # ... a chunk's last row of one or two blocks folded away wherever there is one
    "general-folded-37-warps": {fastrack.OPT_PACK_MAX_BLOCKS: 0, fastrack.OPT_FOLD_TAIL: 2, fastrack.OPT_ROW_SLOTS: 37},
    "general-unfolded": {fastrack.OPT_PACK_MAX_BLOCKS: 0, fastrack.OPT_FOLD_TAIL: 1},  # ... and nowhere
    "auto": {},                                                                   # the planner decides
    "run1": {fastrack.OPT_PACK_RUN: 1},                                           # packed rows, one counter per lane
    "run5": {fastrack.OPT_PACK_RUN: 5},                                           # packed rows, five counters per lane
    "run3-group7": {fastrack.OPT_PACK_RUN: 3, fastrack.OPT_PACK_GROUP: 7},        # odd item size: rows that straddle chunks
    "run300": {fastrack.OPT_PACK_RUN: 300},                                       # one lane per chunk, crossing 256-counter groups
}


@pytest.fixture(params=list(FAMILIES))
def family(request):
    return FAMILIES[request.param]


SHAPES = [(1, 16), (15, 16), (16, 16), (17, 16), (16 * 31, 16), (16 * 32 + 3, 16), (16 * 5000 + 9, 16), (32 * 777 + 31, 32),
          (48 * 1000, 48), (112 * 300 + 1, 112), (240 * 129, 240), (496 * 64 + 495, 496), (512 * 301 + 16, 512),
          (528 * 100, 528), (1024 * 97 + 1000, 1024), (700, 1024), (1024, 1024), (1025, 1024), (4096 * 40 + 77, 4096),
          (8192 * 9 + 8191, 8192), (65536 * 3 + 100, 65536)]


@pytest.mark.parametrize("n,cb", SHAPES)
def test_small_chunks_match_oracle(family, n, cb):
    key, iv = synth.key_and_iv(4)
    plain = synth.random_bytes(n, 4, salt=n + cb)
    c_ref, t_ref = oracle.mc_encrypt(key, iv, cb, plain, NT)
    bad_c, bad_t = c_ref.copy(), t_ref.copy()
    synth.apply_tamper(bad_c, bad_t, cb, synth.tamper_plan(n, cb, 4, fraction=0.2, salt=n))
    p_ref, ok_ref = oracle.mc_decrypt(key, iv, cb, bad_c, bad_t, NT)
    with Gpu(key, cb, family) as g:
        c, t = g.encrypt(iv, plain)
        assert np.array_equal(c, c_ref) and np.array_equal(t, t_ref)
        c, t = g.encrypt(iv, plain, in_place=True)
        assert np.array_equal(c, c_ref) and np.array_equal(t, t_ref)
        for in_place in (False, True):
            p, ok = g.decrypt(iv, bad_c, bad_t, in_place=in_place)
            assert np.array_equal(ok, ok_ref)
            keep = np.repeat(ok_ref == 1, cb)[:n]
            assert np.array_equal(p[keep], p_ref[keep]) and np.array_equal(p, p_ref)
        p, ok = g.pipelined(iv, bad_c, bad_t, 3)
        assert np.array_equal(ok, ok_ref) and np.array_equal(p, p_ref)
        # the two halves of the fused pass (eager evaluation: plaintext first, verdicts later)
        K = t_ref.shape[0]
        d_c = torch.from_numpy(bad_c).cuda()
        d_t = torch.from_numpy(bad_t.reshape(-1).copy()).cuda()
        d_o = torch.full((n + 32,), 0xA5, dtype=torch.uint8, device="cuda")
        d_ok = torch.full((K + 8,), 0x5A5A5A5A, dtype=torch.int32, device="cuda")
        g.ctx.ctr_crypt(iv, d_c.data_ptr(), n, d_o[16:].data_ptr(), 0)
        g.ctx.verify(iv, d_c.data_ptr(), n, d_t.data_ptr(), d_ok[4:].data_ptr(), 0)
        torch.cuda.synchronize()
        assert np.array_equal(d_o[16:16 + n].cpu().numpy(), p_ref)
        assert bool((d_o[:16] == 0xA5).all()) and bool((d_o[16 + n:] == 0xA5).all())
        okh = d_ok.cpu().numpy().view(np.uint32)
        assert np.array_equal(okh[4:4 + K], ok_ref) and (okh[:4] == 0x5A5A5A5A).all() and (okh[4 + K:] == 0x5A5A5A5A).all()
        assert np.array_equal(d_c.cpu().numpy(), bad_c)                       # verify-only leaves the ciphertext alone


def test_two_million_sixteen_byte_chunks(family):
    key, iv = synth.key_and_iv(4)
    cb, n = 16, 32 << 20
    plain = synth.random_bytes(n, 4, salt=99)
    c_ref, t_ref = oracle.mc_encrypt(key, iv, cb, plain, NT)
    K = t_ref.shape[0]
    bad_t = t_ref.copy()
    rej = np.unique(np.random.default_rng(5).integers(0, K, 1000))
    bad_t[rej, 7] ^= 0x20
    expect = np.ones(K, np.uint32)
    expect[rej] = 0
    with fastrack.Context(key, cb, family) as ctx:
        d_p = torch.from_numpy(plain).cuda()
        d_c = torch.empty_like(d_p)
        d_t = torch.empty(16 * K, dtype=torch.uint8, device="cuda")
        ctx.encrypt_tag(iv, d_p.data_ptr(), n, d_c.data_ptr(), d_t.data_ptr(), 0)
        torch.cuda.synchronize()
        assert np.array_equal(d_c.cpu().numpy(), c_ref) and np.array_equal(d_t.cpu().numpy().reshape(K, 16), t_ref)
        d_t.copy_(torch.from_numpy(bad_t.reshape(-1)))
        d_ok = torch.full((K,), 7, dtype=torch.int32, device="cuda")
        ctx.decrypt_verify(iv, d_c.data_ptr(), n, d_t.data_ptr(), d_c.data_ptr(), d_ok.data_ptr(), 0)      # in place
        torch.cuda.synchronize()
        assert np.array_equal(d_ok.cpu().numpy().view(np.uint32), expect)
        assert np.array_equal(d_c.cpu().numpy(), plain)


@pytest.mark.parametrize("sample_bytes,cb,n_samples,chains", [(16, 16, 5000, 0), (48, 16, 700, 0), (400, 400, 3000, 0),
                                                              (400, 112, 500, 4), (208, 64, 999, 4), (1040, 1024, 300, 16),
                                                              (4096, 256, 64, 16)])
def test_batches_of_small_samples(family, sample_bytes, cb, n_samples, chains):
    """Per-sample IVs (and the serial-number AAD) with samples of a few blocks: one launch for the whole batch."""
    key, _ = synth.key_and_iv(5)
    n = sample_bytes * n_samples
    plain = synth.random_bytes(n, 5, salt=sample_bytes + n_samples)
    ivs = [synth.fresh_iv(5, s + 1) for s in range(n_samples)]
    c_ref, t_ref = [], []
    for s in range(n_samples):
        q = plain[s * sample_bytes:(s + 1) * sample_bytes]
        c_s, t_s = (oracle.mc_encrypt_framed(key, ivs[s], cb, chains, q, 1) if chains else oracle.mc_encrypt(key, ivs[s], cb, q, 1))
        c_ref.append(c_s)
        t_ref.append(t_s)
    c_ref, t_ref = np.concatenate(c_ref), np.concatenate(t_ref)
    K = t_ref.shape[0]
    with fastrack.Context(key, cb, family) as ctx:
        if chains:
            ctx.set_framing(chains)
        d_iv = torch.from_numpy(np.frombuffer(b"".join(ivs), np.uint8).copy()).cuda()
        d_p = torch.from_numpy(plain).cuda()
        d_c = torch.empty_like(d_p)
        d_t = torch.empty(16 * K, dtype=torch.uint8, device="cuda")
        ctx.encrypt_tag_samples(d_iv.data_ptr(), sample_bytes, n_samples, d_p.data_ptr(), d_c.data_ptr(), d_t.data_ptr(), 0)
        torch.cuda.synchronize()
        assert np.array_equal(d_c.cpu().numpy(), c_ref) and np.array_equal(d_t.cpu().numpy().reshape(K, 16), t_ref)
        bad_c, bad_t = c_ref.copy(), t_ref.copy()
        bad_c[n // 3] ^= 1
        bad_t[K - 1, 0] ^= 0x80
        expect = np.ones(K, np.uint32)
        cps = K // n_samples
        s_hit, off = divmod(n // 3, sample_bytes)
        expect[s_hit * cps + off // cb] = 0
        expect[K - 1] = 0
        d_c.copy_(torch.from_numpy(bad_c))
        d_t.copy_(torch.from_numpy(bad_t.reshape(-1)))
        d_o = torch.empty_like(d_p)
        d_ok = torch.full((K,), 7, dtype=torch.int32, device="cuda")
        ctx.decrypt_verify_samples(d_iv.data_ptr(), sample_bytes, n_samples, d_c.data_ptr(), d_t.data_ptr(), d_o.data_ptr(),
                                   d_ok.data_ptr(), 0)
        torch.cuda.synchronize()
        assert np.array_equal(d_ok.cpu().numpy().view(np.uint32), expect)
        good = np.ones(n, bool)
        good[(n // 3) // 16 * 16:(n // 3) // 16 * 16 + 16] = False
        assert np.array_equal(d_o.cpu().numpy()[good], plain[good])
        # the pipelined form of the same batch
        h_c = torch.from_numpy(bad_c).pin_memory()
        d_ok.fill_(7)
        d_o.zero_()
        h_iv = np.frombuffer(b"".join(ivs), np.uint8).copy()
        h_t = np.ascontiguousarray(bad_t.reshape(-1))
        ctx.pipelined_h2d_samples(h_iv.ctypes.data, sample_bytes, n_samples, h_c.data_ptr(), h_t.ctypes.data, d_o.data_ptr(),
                                  d_ok.data_ptr(), 2)
        assert np.array_equal(d_ok.cpu().numpy().view(np.uint32), expect)
        assert np.array_equal(d_o.cpu().numpy()[good], plain[good])
