"""Seeded random shapes: every data-path entry point against the oracle on odd sizes, odd chunk sizes,
in place and out of place, with and without the serial-number framing, with seeded tampering."""
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


def _shapes(seed, count):
    rng = np.random.Generator(np.random.PCG64(seed))
    for _ in range(count):
        cb = 16 * int(rng.choice([1, 2, 3, 31, 32, 33, 64, 100, 255, 256, 257, 1000, 1024, 4096, 4099, 16384, 65536]))
        K = int(rng.choice([1, 1, 2, 3, 5, 17, 40]))
        tail = int(rng.integers(0, cb)) if rng.integers(0, 3) else 0
        n = max(1, (K - 1) * cb + (tail if tail else cb))
        if n > 6 << 20:
            n = (6 << 20) + int(rng.integers(0, 64))
        yield n, cb, int(rng.choice([0, 0, 1, 4, 16, 256])), bool(rng.integers(0, 2)), int(rng.integers(0, 1 << 30))


LAYOUTS = {"planner": {}, "rows-folded-tails": {fastrack.OPT_PACK_MAX_BLOCKS: 0, fastrack.OPT_FOLD_TAIL: 2}}


@pytest.mark.parametrize("layout", list(LAYOUTS))
@pytest.mark.parametrize("seed", [1, 2, 3, 4])
def test_random_shapes_all_entry_points(seed, layout):
    key, iv = synth.key_and_iv(seed)
    for n, cb, chains, in_place, salt in _shapes(seed, 30):
        plain = synth.random_bytes(n, seed, salt=salt)
        if chains:
            c, t = oracle.mc_encrypt_framed(key, iv, cb, chains, plain, NT)
        else:
            c, t = oracle.mc_encrypt(key, iv, cb, plain, NT)
        K = t.shape[0]
        what = f"n={n} cb={cb} chains={chains} in_place={in_place}"
        with fastrack.Context(key, cb, LAYOUTS[layout]) as ctx:
            ctx.set_framing(chains)
            st = torch.cuda.current_stream().cuda_stream
            # encrypt
            d_p = dev(plain)
            d_c = d_p if in_place else torch.empty_like(d_p)
            d_t = torch.empty(16 * K, dtype=torch.uint8, device="cuda")
            ctx.encrypt_tag(iv, d_p.data_ptr(), n, d_c.data_ptr(), d_t.data_ptr(), st)
            torch.cuda.synchronize()
            assert np.array_equal(d_c.cpu().numpy(), c), what
            assert np.array_equal(d_t.cpu().numpy().reshape(K, 16), t), what
            # tamper, then every decrypting / verifying entry point
            bad_c, bad_t = c.copy(), t.copy()
            synth.apply_tamper(bad_c, bad_t, cb, synth.tamper_plan(n, cb, seed, fraction=0.3, salt=salt))
            if chains:
                p_ref, ok_ref = oracle.mc_decrypt_framed(key, iv, cb, chains, bad_c, bad_t, NT)
            else:
                p_ref, ok_ref = oracle.mc_decrypt(key, iv, cb, bad_c, bad_t, NT)

            def fresh():
                return dev(bad_c), dev(bad_t), torch.full((K,), 7, dtype=torch.int32, device="cuda")

            def check(d_out, d_ok, name):
                torch.cuda.synchronize()
                assert np.array_equal(d_ok.cpu().numpy().view(np.uint32), ok_ref), f"{name}: {what}"
                if d_out is not None:
                    assert np.array_equal(d_out.cpu().numpy(), p_ref), f"{name}: {what}"

            d_bc, d_bt, d_ok = fresh()
            d_o = d_bc if in_place else torch.empty_like(d_bc)
            ctx.decrypt_verify(iv, d_bc.data_ptr(), n, d_bt.data_ptr(), d_o.data_ptr(), d_ok.data_ptr(), st)
            check(d_o, d_ok, "decrypt_verify")

            d_bc, d_bt, d_ok = fresh()
            d_o = torch.empty_like(d_bc)
            ctx.ctr_crypt(iv, d_bc.data_ptr(), n, d_o.data_ptr(), st)
            ctx.verify(iv, d_bc.data_ptr(), n, d_bt.data_ptr(), d_ok.data_ptr(), st)
            check(d_o, d_ok, "ctr_crypt+verify")

            d_ok.fill_(7)
            ctx.verify_sequential(iv, d_bc.data_ptr(), n, d_bt.data_ptr(), d_ok.data_ptr(), st)
            check(None, d_ok, "verify_sequential")

            d_bc, d_bt, d_ok = fresh()
            d_pad = torch.empty_like(d_bc)
            d_m = torch.empty(16 * K, dtype=torch.uint8, device="cuda")
            d_o = d_bc if in_place else torch.empty_like(d_bc)
            ctx.keystream(iv, n, d_pad.data_ptr(), d_m.data_ptr(), st)
            ctx.xor_verify(iv, d_bc.data_ptr(), n, d_pad.data_ptr(), d_m.data_ptr(), d_bt.data_ptr(), d_o.data_ptr(),
                           d_ok.data_ptr(), st)
            check(d_o, d_ok, "keystream+xor_verify")

            if K <= fastrack.NOALLOC_MAX_CHUNKS:
                d_bc, d_bt, d_ok = fresh()
                d_o = d_bc if in_place else torch.empty_like(d_bc)
                ctx.decrypt_verify_noalloc(iv, d_bc.data_ptr(), n, d_bt.data_ptr(), d_o.data_ptr(), d_ok.data_ptr(), st)
                check(d_o, d_ok, "decrypt_verify_noalloc")

            h_c, h_t = torch.from_numpy(bad_c).pin_memory(), torch.from_numpy(bad_t.reshape(-1).copy())
            d_o = torch.empty(n, dtype=torch.uint8, device="cuda")
            d_ok = torch.full((K,), 7, dtype=torch.int32, device="cuda")
            torch.cuda.synchronize()
            ctx.pipelined_h2d(iv, h_c.data_ptr(), n, h_t.data_ptr(), d_o.data_ptr(), d_ok.data_ptr(), 1 + seed % 3)
            check(d_o, d_ok, "pipelined_h2d")


def test_portable_shared_addressing_path():
    """The kernel puts table base addresses into load immediates when the shared window starts where it
    expects, and falls back to ordinary pointer arithmetic otherwise.  The option forces the fallback so that it
    is exercised on hardware where the fast form applies."""
    _every_pass_on([(1, 16, 0), (70001, 4096, 0), ((1 << 20) + 33, 65536, 16), ((5 << 20) + 7, 1 << 20, 0)],
                   {fastrack.OPT_GENERIC_SMEM: 1})


def test_portable_shared_addressing_path_folded_tails():
    """The same fallback in the row kernels' variant with folded tails."""
    _every_pass_on([(512 * 50 + 9, 512, 0), (16384 * 21 - 3, 16384, 4), ((1 << 20) + 33, 65536, 16)],
                   {fastrack.OPT_GENERIC_SMEM: 1, fastrack.OPT_PACK_MAX_BLOCKS: 0, fastrack.OPT_FOLD_TAIL: 2})


def test_portable_shared_addressing_path_packed_rows():
    """The same fallback in the packed-row kernels (forced here by fixing the run length)."""
    _every_pass_on([(1, 16, 0), (80009, 16, 0), (154128, 512, 4), (70001, 4096, 0), (300000, 16384, 16)],
                   {fastrack.OPT_GENERIC_SMEM: 1, fastrack.OPT_PACK_RUN: 3})


def _every_pass_on(cases, options):
    key, iv = synth.key_and_iv(7)
    for n, cb, chains in cases:
        plain = synth.random_bytes(n, 7, salt=n)
        c, t = (oracle.mc_encrypt_framed(key, iv, cb, chains, plain, NT) if chains else oracle.mc_encrypt(key, iv, cb, plain, NT))
        K = t.shape[0]
        bad_c, bad_t = c.copy(), t.copy()
        synth.apply_tamper(bad_c, bad_t, cb, synth.tamper_plan(n, cb, 7, fraction=0.3, salt=n))
        p_ref, ok_ref = (oracle.mc_decrypt_framed(key, iv, cb, chains, bad_c, bad_t, NT) if chains
                         else oracle.mc_decrypt(key, iv, cb, bad_c, bad_t, NT))
        with fastrack.Context(key, cb, options) as ctx:
            ctx.set_framing(chains)
            st = torch.cuda.current_stream().cuda_stream
            d_p = dev(plain)
            d_c = torch.empty_like(d_p)
            d_t = torch.empty(16 * K, dtype=torch.uint8, device="cuda")
            ctx.encrypt_tag(iv, d_p.data_ptr(), n, d_c.data_ptr(), d_t.data_ptr(), st)
            d_bc, d_bt = dev(bad_c), dev(bad_t)
            d_o = torch.empty_like(d_bc)
            d_ok = torch.full((K,), 7, dtype=torch.int32, device="cuda")
            d_ok2 = torch.full((K,), 7, dtype=torch.int32, device="cuda")
            ctx.decrypt_verify(iv, d_bc.data_ptr(), n, d_bt.data_ptr(), d_o.data_ptr(), d_ok.data_ptr(), st)
            ctx.verify(iv, d_bc.data_ptr(), n, d_bt.data_ptr(), d_ok2.data_ptr(), st)
            torch.cuda.synchronize()
            assert np.array_equal(d_c.cpu().numpy(), c) and np.array_equal(d_t.cpu().numpy().reshape(K, 16), t)
            assert np.array_equal(d_o.cpu().numpy(), p_ref)
            assert np.array_equal(d_ok.cpu().numpy().view(np.uint32), ok_ref)
            assert np.array_equal(d_ok2.cpu().numpy().view(np.uint32), ok_ref)


def test_one_context_many_mixed_calls_leave_scratch_clean():
    """200 calls of every kind, sizes going up and down, on ONE context: every call must still be exact,
    i.e. each pass leaves the per-chunk accumulators and counters (both banks) zeroed for the next one."""
    key, iv = synth.key_and_iv(9)
    cb = 8192
    rng = np.random.Generator(np.random.PCG64(9))
    sizes = [cb * int(k) + int(t) for k, t in zip(rng.integers(1, 300, 12), rng.integers(0, cb, 12))]
    cases = []
    for n in sizes:
        plain = synth.random_bytes(n, 9, salt=n)
        c, t = oracle.mc_encrypt(key, iv, cb, plain, NT)
        synth.apply_tamper(c, t, cb, synth.tamper_plan(n, cb, 9, fraction=0.05, salt=n))
        p_ref, ok_ref = oracle.mc_decrypt(key, iv, cb, c, t, NT)
        cases.append((n, dev(c), dev(t), p_ref, ok_ref, dev(plain)))
    with fastrack.Context(key, cb) as ctx:
        st = torch.cuda.current_stream().cuda_stream
        for it in range(200):
            n, d_c, d_t, p_ref, ok_ref, d_plain = cases[int(rng.integers(0, len(cases)))]
            K = ok_ref.size
            kind = int(rng.integers(0, 5))
            d_o = torch.empty(n, dtype=torch.uint8, device="cuda")
            d_ok = torch.full((K,), 7, dtype=torch.int32, device="cuda")
            if kind == 0:
                ctx.decrypt_verify(iv, d_c.data_ptr(), n, d_t.data_ptr(), d_o.data_ptr(), d_ok.data_ptr(), st)
            elif kind == 1:
                ctx.verify(iv, d_c.data_ptr(), n, d_t.data_ptr(), d_ok.data_ptr(), st)
                d_o = None
            elif kind == 2:
                ctx.decrypt_verify_noalloc(iv, d_c.data_ptr(), n, d_t.data_ptr(), d_o.data_ptr(), d_ok.data_ptr(), st)
            elif kind == 3:
                d_pad = torch.empty(n, dtype=torch.uint8, device="cuda")
                d_m = torch.empty(16 * K, dtype=torch.uint8, device="cuda")
                ctx.keystream(iv, n, d_pad.data_ptr(), d_m.data_ptr(), st)
                ctx.xor_verify(iv, d_c.data_ptr(), n, d_pad.data_ptr(), d_m.data_ptr(), d_t.data_ptr(), d_o.data_ptr(),
                               d_ok.data_ptr(), st)
            else:
                d_tt = torch.empty(16 * K, dtype=torch.uint8, device="cuda")
                ctx.encrypt_tag(iv, d_plain.data_ptr(), n, d_o.data_ptr(), d_tt.data_ptr(), st)   # tags unchecked here
                ctx.decrypt_verify(iv, d_o.data_ptr(), n, d_tt.data_ptr(), d_o.data_ptr(), d_ok.data_ptr(), st)
                torch.cuda.synchronize()
                assert bool((d_ok == 1).all()) and bool((d_o == d_plain).all()), f"iteration {it}"
                continue
            torch.cuda.synchronize()
            assert np.array_equal(d_ok.cpu().numpy().view(np.uint32), ok_ref), f"iteration {it} kind {kind}"
            if d_o is not None:
                assert np.array_equal(d_o.cpu().numpy(), p_ref), f"iteration {it} kind {kind}"
