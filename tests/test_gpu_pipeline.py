"""GPU parity of the pipelined H2D path (paper Section 4.3) against the CPU oracle."""
import numpy as np
import pytest

import oracle
from paper_2410_15240_b200 import synth

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")
if not torch.cuda.is_available():
    pytest.skip("no CUDA device", allow_module_level=True)

from gpu_harness import Gpu  # noqa: E402

NT = oracle.host_threads()


@pytest.mark.parametrize("n,cb", [(1, 16), (100, 1024), (1 << 20, 65536), ((1 << 20) + 17, 65536), (700001, 256), (2500000, 4096),
                                  (3 * (1 << 20) + 5, 1 << 20), (9 * (1 << 20) + 12345, 256 * 1024),
                                  ((5 << 20) - 16, 48 * 1024), (2 * (1 << 22) + 999, 1 << 22)])
@pytest.mark.parametrize("n_streams", [1, 3])
@pytest.mark.parametrize("direct", ["1", "0"])
def test_pipelined_matches_oracle_small(n, cb, n_streams, direct):
    """Single-stage transfers (up to about 3 MiB) are by default read from the page-locked host buffer by the kernel
    itself, pinned tags included; the option set to 0 keeps them on the copy engine.  Both must equal the oracle."""
    from paper_2410_15240_b200 import fastrack
    options = {fastrack.OPT_DIRECT_SMALL: int(direct)}
    key, iv = synth.key_and_iv(2)
    plain = synth.random_bytes(n, 2, salt=n)
    c, t = oracle.mc_encrypt(key, iv, cb, plain, NT)
    plan = synth.tamper_plan(n, cb, 2, fraction=0.1, salt=n)
    synth.apply_tamper(c, t, cb, plan)
    p_ref, ok_ref = oracle.mc_decrypt(key, iv, cb, c, t, NT)
    with Gpu(key, cb, options) as g:
        p, ok = g.pipelined(iv, c, t, n_streams)
        assert np.array_equal(ok, ok_ref)
        assert np.array_equal(p, p_ref)
        p2, ok2 = g.pipelined(iv, c, t, n_streams, pinned_tags=True)      # context reuse
        assert np.array_equal(ok2, ok_ref) and np.array_equal(p2, p_ref)
    assert sorted(k for k, _, _ in plan) == [int(k) for k in np.flatnonzero(ok_ref == 0)]


@pytest.mark.parametrize("cb", [256 * 1024, 1 << 20, 4 << 20, 8 << 20])
def test_config2_fp16_image_batch(cb):
    """fp16 256x3x224x224 ~ N(0,1) (77 070 336 B), oracle-encrypted, pipelined H2D + decrypt/verify: every chunk size
    of the configuration with 2, 3 and 4 streams (the oracle encrypts once per chunk size)."""
    key, iv = synth.key_and_iv(2)
    plain = synth.fp16_image_batch()
    assert plain.size == 77_070_336
    c, t = oracle.mc_encrypt(key, iv, cb, plain, NT)
    with Gpu(key, cb) as g:
        for n_streams in (2, 3, 4):
            p, ok = g.pipelined(iv, c, t, n_streams)
            assert (ok == 1).all() and ok.size == oracle.num_chunks(plain.size, cb)
            assert np.array_equal(p, plain)


@pytest.mark.parametrize("n,cb,n_streams,in_place", [(1, 16, 1, False), (100, 1024, 2, True), ((1 << 20) + 17, 65536, 2, False),
                                                      (700001, 256, 2, False), (2500000, 4096, 1, False), (2500000, 4096, 1, True),
                                                      ((9 << 20) + 12345, 256 * 1024, 3, True),
                                                      (2 * (1 << 22) + 999, 1 << 22, 4, False), (77_070_336, 4 << 20, 4, False)])
@pytest.mark.parametrize("direct,pinned_tags", [("1", False), ("1", True), ("0", False)])
def test_pipelined_d2h_encrypt_matches_oracle(n, cb, n_streams, in_place, direct, pinned_tags):
    """GPU encrypt+tag with overlapped device->host copies; the host side (oracle) verifies and decrypts.
    Single-stage transfers are by default written to the page-locked host buffers by the kernel itself (tags too when
    their buffer is page-locked); the option set to 0 keeps them on the copy engine."""
    from paper_2410_15240_b200 import fastrack
    key, iv = synth.key_and_iv(3)
    plain = synth.fp16_image_batch() if n == 77_070_336 else synth.random_bytes(n, 3, salt=n)
    c_ref, t_ref = oracle.mc_encrypt(key, iv, cb, plain, NT)
    K = t_ref.shape[0]
    with fastrack.Context(key, cb, {fastrack.OPT_DIRECT_SMALL: int(direct)}) as ctx:
        d_p = torch.from_numpy(plain).cuda()
        d_c = d_p if in_place else torch.empty_like(d_p)
        h_c = torch.full((n,), 0xEE, dtype=torch.uint8).pin_memory()
        h_t = torch.zeros(16 * K, dtype=torch.uint8)
        if pinned_tags:
            h_t = h_t.pin_memory()
        torch.cuda.synchronize()
        for _ in range(1 if in_place else 2):
            ctx.pipelined_d2h(iv, d_p.data_ptr(), n, d_c.data_ptr(), h_c.data_ptr(), h_t.data_ptr(), n_streams)
            assert np.array_equal(h_c.numpy(), c_ref)
            assert np.array_equal(h_t.numpy().reshape(K, 16), t_ref)
        if not in_place:
            assert np.array_equal(d_p.cpu().numpy(), plain)
    back, ok = oracle.mc_decrypt(key, iv, cb, h_c.numpy(), h_t.numpy(), NT)
    assert ok.all() and np.array_equal(back, plain)


def test_stage_trace_shows_copies_hiding_kernels():
    """Section 4.3: the copy of stage i+1 runs while the kernel of stage i does, so a stage's kernel ends before
    the next stage's copy does; only the last kernel sticks out."""
    from paper_2410_15240_b200 import fastrack
    key, iv = synth.key_and_iv(2)
    cb, n = 1 << 20, 64 << 20
    with fastrack.Context(key, cb) as ctx:
        K = ctx.num_chunks(n)
        d_p = torch.randint(0, 256, (n,), dtype=torch.uint8, device="cuda")
        d_c = torch.empty_like(d_p)
        d_t = torch.empty(16 * K, dtype=torch.uint8, device="cuda")
        ctx.encrypt_tag(iv, d_p.data_ptr(), n, d_c.data_ptr(), d_t.data_ptr(), 0)
        torch.cuda.synchronize()
        h_c, h_t = d_c.cpu().pin_memory(), d_t.cpu()
        d_o = torch.empty_like(d_p)
        d_ok = torch.zeros(K, dtype=torch.int32, device="cuda")
        assert ctx.get_trace() == []
        ctx.set_trace(True)
        for _ in range(2):
            ctx.pipelined_h2d(iv, h_c.data_ptr(), n, h_t.data_ptr(), d_o.data_ptr(), d_ok.data_ptr(), 2)
        tr = ctx.get_trace()
        assert bool((d_ok == 1).all()) and bool((d_o == d_p).all())
        ctx.set_trace(False)
        assert ctx.get_trace() == []
    assert len(tr) >= 4
    assert tr[0]["offset"] == 0 and sum(s["bytes"] for s in tr) == n
    for a, b in zip(tr, tr[1:]):
        assert b["offset"] == a["offset"] + a["bytes"] and b["bytes"] <= a["bytes"]          # shrinking stages
        assert a["copy_start_ms"] <= a["copy_end_ms"] <= a["kernel_end_ms"]
        assert b["copy_start_ms"] >= a["copy_start_ms"]
        assert a["kernel_end_ms"] <= b["copy_end_ms"] + 0.05, "a stage's kernel should finish under the next copy"
    total = tr[-1]["kernel_end_ms"]
    copies = sum(s["copy_end_ms"] - s["copy_start_ms"] for s in tr)
    assert total < 1.25 * copies                                                              # the kernels are hidden
