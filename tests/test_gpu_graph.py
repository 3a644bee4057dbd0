"""The asynchronous calls inside a captured CUDA graph.

A serving loop that handles the same batch shape over and over can capture the library's launches once and replay
them.  The per-sample calls read their IV bases from device memory, so every replay can run under fresh IVs (the
single-buffer calls take the IV by value, which a replay would repeat -- fine for a test, wrong for GCM in production).
Each replay is checked against the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2410_15240_b200 import synth

pytestmark = pytest.mark.gpu


def _fresh_ivs(n, rep):
    return [synth.fresh_iv(7, 100 * rep + s + 1) for s in range(n)]


@pytest.mark.parametrize("cb,sample_bytes,n_samples", [(64 << 10, 150528, 6),      # 3 chunks per sample, the last one 19 456 bytes
                                                       (256, 4096 + 48, 700)])      # many small chunks: the packed-row kernels
def test_sample_batch_round_trip_replayed_from_a_graph(cb, sample_bytes, n_samples):
    from paper_2410_15240_b200 import fastrack
    key, _ = synth.key_and_iv(7)
    n = sample_bytes * n_samples
    with fastrack.Context(key, cb) as ctx:
        cps = ctx.num_chunks(sample_bytes)
        K = cps * n_samples
        d_iv = torch.zeros(12 * n_samples, dtype=torch.uint8, device="cuda")
        d_p = torch.zeros(n, dtype=torch.uint8, device="cuda")
        d_c = torch.zeros(n, dtype=torch.uint8, device="cuda")
        d_t = torch.zeros(16 * K, dtype=torch.uint8, device="cuda")
        d_o = torch.zeros(n, dtype=torch.uint8, device="cuda")
        d_ok = torch.zeros(K, dtype=torch.int32, device="cuda")

        def both(stream):
            ctx.encrypt_tag_samples(d_iv.data_ptr(), sample_bytes, n_samples, d_p.data_ptr(), d_c.data_ptr(), d_t.data_ptr(), stream)
            ctx.decrypt_verify_samples(d_iv.data_ptr(), sample_bytes, n_samples, d_c.data_ptr(), d_t.data_ptr(), d_o.data_ptr(),
                                       d_ok.data_ptr(), stream)

        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            both(side.cuda_stream)                                # warm-up outside the capture
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        before = ctx.launches
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            both(torch.cuda.current_stream().cuda_stream)
        assert ctx.launches == before + 2                   # two launches were recorded, none ran yet

        for rep in range(3):
            ivs = _fresh_ivs(n_samples, rep)
            plain = synth.random_bytes(n, 7, salt=rep + 1)
            d_iv.copy_(torch.from_numpy(np.frombuffer(b"".join(ivs), dtype=np.uint8).copy()))
            d_p.copy_(torch.from_numpy(plain))
            d_ok.fill_(0x5A5A5A5A)
            d_o.zero_()
            graph.replay()
            torch.cuda.synchronize()
            got_c, got_t = d_c.cpu().numpy(), d_t.cpu().numpy().reshape(K, 16)
            for s in range(n_samples):
                c_ref, t_ref = oracle.mc_encrypt(key, ivs[s], cb, plain[s * sample_bytes:(s + 1) * sample_bytes])
                assert np.array_equal(got_c[s * sample_bytes:(s + 1) * sample_bytes], c_ref), f"replay {rep} sample {s}"
                assert np.array_equal(got_t[s * cps:(s + 1) * cps], t_ref), f"replay {rep} sample {s}"
            assert bool((d_ok == 1).all()) and np.array_equal(d_o.cpu().numpy(), plain), f"replay {rep}"
        assert ctx.launches == before + 2                   # replays do not pass through the library


def test_replayed_verification_sees_tampering_between_replays():
    from paper_2410_15240_b200 import fastrack
    key, iv = synth.key_and_iv(8)
    cb, n = 16 << 10, (1 << 20) + 4099
    plain = synth.random_bytes(n, 8, salt=1)
    c_ref, t_ref = oracle.mc_encrypt(key, iv, cb, plain, n_threads=oracle.host_threads())
    with fastrack.Context(key, cb) as ctx:
        K = ctx.num_chunks(n)
        d_c = torch.from_numpy(c_ref.copy()).cuda()
        d_t = torch.from_numpy(t_ref.reshape(-1).copy()).cuda()
        d_o = torch.zeros(n, dtype=torch.uint8, device="cuda")
        d_ok = torch.zeros(K, dtype=torch.int32, device="cuda")
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            ctx.decrypt_verify(iv, d_c.data_ptr(), n, d_t.data_ptr(), d_o.data_ptr(), d_ok.data_ptr(), side.cuda_stream)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            ctx.decrypt_verify(iv, d_c.data_ptr(), n, d_t.data_ptr(), d_o.data_ptr(), d_ok.data_ptr(),
                               torch.cuda.current_stream().cuda_stream)
        expect = np.ones(K, np.int32)
        for rep, (chunk, where) in enumerate([(None, None), (5, "cipher"), (K - 1, "tag"), (None, None)]):
            d_c.copy_(torch.from_numpy(c_ref))
            d_t.copy_(torch.from_numpy(t_ref.reshape(-1)))
            expect[:] = 1
            if where == "cipher":
                d_c[chunk * cb + 77] ^= 0x10
                expect[chunk] = 0
            elif where == "tag":
                d_t[16 * chunk + 3] ^= 0x01
                expect[chunk] = 0
            d_ok.fill_(0x5A5A5A5A)
            graph.replay()
            torch.cuda.synchronize()
            assert np.array_equal(d_ok.cpu().numpy(), expect), f"replay {rep}"
            if where != "cipher":
                assert np.array_equal(d_o.cpu().numpy(), plain), f"replay {rep}"
