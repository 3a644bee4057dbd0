"""The entry point that allocates nothing: checked against the CPU oracle and against fastrack_decrypt_verify.

It serves callers that cannot call cudaMalloc once they are running (all device memory owned by another
allocator, or a serving loop that cannot afford an allocation's device-wide synchronisation): the records in
which CTAs combine their pieces of a chunk are a fixed array inside the library, shared by every call.  The file
name makes pytest collect it last, so a run that stops at the first failure has already run every other test."""
import numpy as np
import pytest

import oracle
from paper_2410_15240_b200 import fastrack, synth

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")
if not torch.cuda.is_available():
    pytest.skip("no CUDA device", allow_module_level=True)

NT = oracle.host_threads()


def _run(ctx, entry, iv, d_c, n, d_t, K):
    d_p = torch.full((n,), 0xEE, dtype=torch.uint8, device="cuda")
    d_ok = torch.full((K,), 7, dtype=torch.int32, device="cuda")
    st = torch.cuda.current_stream()
    entry(iv, d_c.data_ptr(), n, d_t.data_ptr(), d_p.data_ptr(), d_ok.data_ptr(), st.cuda_stream)
    st.synchronize()
    return d_p.cpu().numpy(), d_ok.cpu().numpy().view(np.uint32)


def test_noalloc_matches_oracle_and_allocating_entry_point_twice_in_a_row():
    key, iv = synth.key_and_iv(0)
    cb = 64 * 1024                                   # 129 rows per chunk: every chunk is shared by several warps
    cases = [((3 << 20) + 4099, [(2, "cipher", 999), (40, "tag", 5)]),      # 49 chunks, ragged tail
             ((1 << 20) + 16, [(0, "tag", 127), (16, "cipher", 3)])]         # 17 chunks, other reject set
    with fastrack.Context(key, cb) as ctx:
        for n, plan in cases:                        # two calls in a row on the shared array
            K = ctx.num_chunks(n)
            plain = synth.random_bytes(n, 0, salt=n)
            c, t = oracle.mc_encrypt(key, iv, cb, plain, NT)
            synth.apply_tamper(c, t, cb, plan)
            p_ref, ok_ref = oracle.mc_decrypt(key, iv, cb, c, t, NT)          # the oracle decides what is right
            assert sorted(k for k, _, _ in plan) == [int(k) for k in np.flatnonzero(ok_ref == 0)]
            d_c, d_t = torch.from_numpy(c).cuda(), torch.from_numpy(t.reshape(-1)).cuda()
            p_new, ok_new = _run(ctx, ctx.decrypt_verify_noalloc, iv, d_c, n, d_t, K)
            assert np.array_equal(ok_new, ok_ref)                            # bit-exact: integer work
            assert np.array_equal(p_new, p_ref)
            p_old, ok_old = _run(ctx, ctx.decrypt_verify, iv, d_c, n, d_t, K)
            assert np.array_equal(ok_new, ok_old) and np.array_equal(p_new, p_old)
            p_again, ok_again = _run(ctx, ctx.decrypt_verify_noalloc, iv, d_c, n, d_t, K)
            assert np.array_equal(ok_again, ok_ref) and np.array_equal(p_again, p_ref)


@pytest.mark.parametrize("row_slots", [0, 148 * 32, 1000])
def test_noalloc_at_its_chunk_limit_with_chunks_shared_between_warps(row_slots):
    """The most chunks a call may cover, 16 384 of 3 KiB (7 rows each), so that chunk boundaries fall inside the
    ranges of warps and of CTAs everywhere; first and last chunk tampered; compared with the oracle."""
    key, iv = synth.key_and_iv(1)
    cb = 3072
    K = fastrack.NOALLOC_MAX_CHUNKS
    n = cb * K - 5
    plain = synth.random_bytes(n, 1, salt=K)
    c, t = oracle.mc_encrypt(key, iv, cb, plain, NT)
    synth.apply_tamper(c, t, cb, [(0, "cipher", 7), (K - 1, "tag", 100), (K // 2, "cipher", 12345)])
    p_ref, ok_ref = oracle.mc_decrypt(key, iv, cb, c, t, NT)
    assert [int(k) for k in np.flatnonzero(ok_ref == 0)] == [0, K // 2, K - 1]
    with fastrack.Context(key, cb, {fastrack.OPT_ROW_SLOTS: row_slots}) as ctx:
        assert ctx.num_chunks(n) == K
        d_c, d_t = torch.from_numpy(c).cuda(), torch.from_numpy(t.reshape(-1)).cuda()
        for _ in range(2):
            p, ok = _run(ctx, ctx.decrypt_verify_noalloc, iv, d_c, n, d_t, K)
            assert np.array_equal(ok, ok_ref) and np.array_equal(p, p_ref)


def test_noalloc_rejects_more_chunks_than_its_limit():
    key, iv = synth.key_and_iv(0)
    with fastrack.Context(key, 16) as ctx:
        n = 16 * (fastrack.NOALLOC_MAX_CHUNKS + 1)
        buf = torch.zeros(n, dtype=torch.uint8, device="cuda")
        tags = torch.zeros(16 * (fastrack.NOALLOC_MAX_CHUNKS + 1), dtype=torch.uint8, device="cuda")
        ok = torch.full((fastrack.NOALLOC_MAX_CHUNKS + 1,), 7, dtype=torch.int32, device="cuda")
        rc = fastrack.fastrack_decrypt_verify_noalloc(ctx.handle, iv, buf.data_ptr(), n, tags.data_ptr(),
                                                      buf.data_ptr(), ok.data_ptr(), 0)
        assert rc == fastrack.ERR_LIMIT
        torch.cuda.synchronize()
        assert bool((ok == 7).all())                                         # nothing ran
        rc = fastrack.fastrack_decrypt_verify_noalloc(ctx.handle, iv, buf.data_ptr(), n - 16, tags.data_ptr(),
                                                      buf.data_ptr(), ok.data_ptr(), 0)
        assert rc == fastrack.OK                                             # exactly the maximum is accepted
        torch.cuda.synchronize()
