"""GPU parity at the full sizes of the benchmark configurations 3 and 4.

Config 3 goes through the oracle in full.  Config 4 reaches 4 GiB, which the plain oracle cannot cover in
reasonable time: there the ciphertext and tags come from OpenSSL (python `cryptography`, an independent
library -- never from the CUDA path), the expected plaintext is the original buffer, the expected verdicts
follow from the tamper plan, and the oracle itself re-checks a sample of chunks (every tampered chunk up to
a byte budget, the first and the last chunk, seeded others) bit for bit."""
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest

import oracle
from paper_2410_15240_b200 import fastrack, synth

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")
if not torch.cuda.is_available():
    pytest.skip("no CUDA device", allow_module_level=True)

NT = oracle.host_threads()
KIB, MIB, GIB = 1 << 10, 1 << 20, 1 << 30


def test_config3_training_state_round_trip():
    """bf16 buffer of 335 M values ~ N(0, 0.02) (670 MB), 4 MiB chunks: GPU encrypt+tag -> D2H -> oracle
    verify+decrypt == original; oracle re-encrypt under a fresh IV -> H2D -> GPU decrypt+verify == original."""
    key, iv = synth.key_and_iv(3)
    cb = 4 * MIB
    plain = synth.bf16_params()
    n = plain.size
    assert n == 670_000_000
    K = (n + cb - 1) // cb
    assert K == 160 and n - 159 * cb == 3_105_664
    with fastrack.Context(key, cb) as ctx:
        st = torch.cuda.current_stream().cuda_stream
        d_p = torch.from_numpy(plain).cuda()
        d_c = torch.empty_like(d_p)
        d_t = torch.empty(16 * K, dtype=torch.uint8, device="cuda")
        ctx.encrypt_tag(iv, d_p.data_ptr(), n, d_c.data_ptr(), d_t.data_ptr(), st)
        torch.cuda.synchronize()
        c_gpu, t_gpu = d_c.cpu().numpy(), d_t.cpu().numpy().reshape(K, 16)
        back, ok = oracle.mc_decrypt(key, iv, cb, c_gpu, t_gpu, NT)
        assert ok.all() and np.array_equal(back, plain)

        iv2 = synth.fresh_iv(3)
        c2, t2 = oracle.mc_encrypt(key, iv2, cb, plain, NT)
        assert not np.array_equal(c2[:64], c_gpu[:64])
        d_c.copy_(torch.from_numpy(c2))
        d_t.copy_(torch.from_numpy(t2.reshape(-1)))
        d_ok = torch.zeros(K, dtype=torch.int32, device="cuda")
        ctx.decrypt_verify(iv2, d_c.data_ptr(), n, d_t.data_ptr(), d_c.data_ptr(), d_ok.data_ptr(), st)   # in place
        torch.cuda.synchronize()
        assert bool((d_ok == 1).all())
        assert bool((d_c == d_p).all())


_plain_cache = {}


def _plain(n):
    if n not in _plain_cache:
        _plain_cache.clear()
        _plain_cache[n] = synth.random_bytes(n, 4, salt=n)
    return _plain_cache[n]


def _iv_k(iv: bytes, k: int) -> bytes:
    return iv[:8] + ((int.from_bytes(iv[8:], "big") + k) % (1 << 32)).to_bytes(4, "big")


def _openssl_encrypt(key, iv, cb, plain):
    from cryptography.hazmat.primitives.ciphers.aead import AESGCM
    n = plain.size
    K = (n + cb - 1) // cb
    cipher = np.empty(n, np.uint8)
    tags = np.empty((K, 16), np.uint8)
    aead = AESGCM(key)
    view = memoryview(plain)

    def work(lo, hi):
        for k in range(lo, hi):
            out = aead.encrypt(_iv_k(iv, k), view[k * cb:min(n, (k + 1) * cb)], None)
            m = len(out) - 16
            cipher[k * cb:k * cb + m] = np.frombuffer(out, np.uint8, m)
            tags[k] = np.frombuffer(out, np.uint8, 16, m)

    step = max(1, (K + NT - 1) // NT)
    with ThreadPoolExecutor(NT) as ex:
        list(ex.map(lambda lo: work(lo, min(K, lo + step)), range(0, K, step)))
    return cipher, tags


SIZES = [4 ** e for e in range(6, 17)]                     # 4 KiB .. 4 GiB
CHUNKS = [16 * KIB, 64 * KIB, 256 * KIB, MIB, 4 * MIB, 16 * MIB]


def _cells():
    for n in SIZES:
        for cb in CHUNKS:
            yield pytest.param(n, cb, id=f"len{n}-cb{cb}")


@pytest.mark.parametrize("n,cb", list(_cells()))
def test_config4_size_sweep_with_one_percent_tampered(n, cb):
    key, iv = synth.key_and_iv(4)
    plain = _plain(n)
    K = (n + cb - 1) // cb
    if n <= 16 * MIB:
        cipher, tags = oracle.mc_encrypt(key, iv, cb, plain, NT)            # small cells: the oracle makes the input
    else:
        cipher, tags = _openssl_encrypt(key, iv, cb, plain)
    plan = synth.tamper_plan(n, cb, 4, 0.01, salt=n // cb + cb)
    synth.apply_tamper(cipher, tags, cb, plan)
    rejected = sorted(k for k, _, _ in plan)
    cipher_hit = {k for k, where, _ in plan if where == "cipher"}
    assert len(rejected) == (0 if K < 2 else -(-K // 100))

    with fastrack.Context(key, cb) as ctx:
        d_c = torch.from_numpy(cipher).cuda()
        d_t = torch.from_numpy(tags.reshape(-1)).cuda()
        d_p = torch.empty_like(d_c)
        d_ok = torch.full((K,), 7, dtype=torch.int32, device="cuda")
        ctx.decrypt_verify(iv, d_c.data_ptr(), n, d_t.data_ptr(), d_p.data_ptr(), d_ok.data_ptr(),
                           torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        ok = d_ok.cpu().numpy().view(np.uint32)
        p = d_p.cpu().numpy()
    del d_c, d_p

    # exact reject set
    assert [int(k) for k in np.flatnonzero(ok == 0)] == rejected
    assert set(np.unique(ok).tolist()) <= {0, 1}
    # bit-exact plaintext of every chunk whose ciphertext was not touched (accepted ones and tag-only rejects)
    mism = np.flatnonzero(p != plain)
    assert set((mism // cb).tolist()) <= cipher_hit
    for k in cipher_hit:                                   # a flipped ciphertext bit flips exactly that plaintext bit
        assert np.count_nonzero(p[k * cb:(k + 1) * cb] != plain[k * cb:(k + 1) * cb]) == 1

    # the oracle on a sample: tampered chunks first, then first / last / seeded others, within a byte budget
    budget = 48 * MIB if cb >= 4 * MIB else 24 * MIB
    rng = np.random.Generator(np.random.PCG64(synth.BASE_SEED + n % 1000003 + cb))
    order = rejected + [0, K - 1] + [int(x) for x in rng.integers(0, K, 64)]
    sample, used = [], 0
    for k in dict.fromkeys(order):
        m = min(cb, n - k * cb)
        if used + m > budget and sample:
            break
        sample.append(k)
        used += m

    def check(k):
        lo, hi = k * cb, min(n, (k + 1) * cb)
        pk, okk = oracle.gcm_decrypt(key, _iv_k(iv, k), b"", cipher[lo:hi], tags[k])
        return k, bool(okk) == bool(ok[k]) and np.array_equal(np.frombuffer(pk, np.uint8), p[lo:hi])

    with ThreadPoolExecutor(NT) as ex:
        for k, good in ex.map(check, sample):
            assert good, f"chunk {k} differs from the oracle"


def _sampled_oracle_blocks(key, iv, cb, cipher, plain, offsets):
    """Ciphertext blocks at the given byte offsets, recomputed one by one with the oracle's AES (counter mode)."""
    for off in offsets:
        k, j = off // cb, (off % cb) // 16
        ks = oracle.aes256_encrypt_block(key, _iv_k(iv, k) + (2 + j).to_bytes(4, "big"))
        blk = bytes(a ^ b for a, b in zip(plain[off:off + 16].tobytes(), ks))
        assert cipher[off:off + 16].tobytes() == blk[:len(cipher[off:off + 16])], off


def test_largest_chunk_one_gib_single_chain():
    """chunk_bytes = FASTRACK_MAX_CHUNK_BYTES: one 1 GiB chain (67 108 864 blocks, power table of 1 GiB).
    The oracle cannot walk a 1 GiB chain in reasonable time, so the tag expectation comes from OpenSSL and the
    oracle re-computes sampled ciphertext blocks (first, last, around 2^32 bits, seeded others)."""
    from cryptography.hazmat.primitives.ciphers.aead import AESGCM
    key, iv = synth.key_and_iv(4)
    n = cb = fastrack.MAX_CHUNK_BYTES
    plain = synth.random_bytes(n, 4, salt=99)
    ref = AESGCM(key).encrypt(iv, memoryview(plain), None)
    c_ref = np.frombuffer(ref, np.uint8, n)
    t_ref = np.frombuffer(ref, np.uint8, 16, n)
    rng = np.random.Generator(np.random.PCG64(7))
    offs = [0, 16, n - 16, (1 << 29) - 16, 1 << 29] + [int(x) * 16 for x in rng.integers(0, n // 16, 32)]
    _sampled_oracle_blocks(key, iv, cb, c_ref, plain, offs)
    with fastrack.Context(key, cb) as ctx:
        st = torch.cuda.current_stream().cuda_stream
        d_p = torch.from_numpy(plain).cuda()
        d_c = torch.empty_like(d_p)
        d_t = torch.empty(16, dtype=torch.uint8, device="cuda")
        ctx.encrypt_tag(iv, d_p.data_ptr(), n, d_c.data_ptr(), d_t.data_ptr(), st)
        torch.cuda.synchronize()
        assert np.array_equal(d_c.cpu().numpy(), c_ref)
        assert np.array_equal(d_t.cpu().numpy(), t_ref)
        d_ok = torch.full((1,), 7, dtype=torch.int32, device="cuda")
        ctx.decrypt_verify(iv, d_c.data_ptr(), n, d_t.data_ptr(), d_c.data_ptr(), d_ok.data_ptr(), st)
        torch.cuda.synchronize()
        assert int(d_ok.item()) == 1 and bool((d_c == d_p).all())
        d_c[n // 3] ^= 1                                                    # now holds plaintext: any bit flips the verdict
        ctx.verify(iv, d_c.data_ptr(), n, d_t.data_ptr(), d_ok.data_ptr(), st)
        torch.cuda.synchronize()
        assert int(d_ok.item()) == 0


def test_buffer_beyond_four_gib_uses_64_bit_offsets():
    """4 GiB + 16 MiB + 5 bytes in 16 MiB chunks (K = 258, last chunk 5 bytes): byte offsets above 2^32."""
    key, iv = synth.key_and_iv(4)
    cb = 16 * MIB
    n = 4 * GIB + cb + 5
    plain = synth.random_bytes(n, 4, salt=n)
    cipher, tags = _openssl_encrypt(key, iv, cb, plain)
    K = tags.shape[0]
    assert K == 258
    plan = [(0, "cipher", 3), (255, "tag", 9), (256, "cipher", 12345), (257, "cipher", 39)]
    synth.apply_tamper(cipher, tags, cb, plan)
    rng = np.random.Generator(np.random.PCG64(11))
    with fastrack.Context(key, cb) as ctx:
        d_c = torch.from_numpy(cipher).cuda()
        d_t = torch.from_numpy(tags.reshape(-1)).cuda()
        d_ok = torch.full((K,), 7, dtype=torch.int32, device="cuda")
        ctx.decrypt_verify(iv, d_c.data_ptr(), n, d_t.data_ptr(), d_c.data_ptr(), d_ok.data_ptr(),
                           torch.cuda.current_stream().cuda_stream)          # in place
        torch.cuda.synchronize()
        ok = d_ok.cpu().numpy().view(np.uint32)
        p = d_c.cpu().numpy()
    assert [int(k) for k in np.flatnonzero(ok == 0)] == [0, 255, 256, 257]
    mism = np.flatnonzero(p != plain)
    assert set((mism // cb).tolist()) == {0, 256, 257} and mism.size == 3
    # the oracle on the chunks that straddle and follow the 2^32-byte boundary, and on the 5-byte tail
    for k in (255, 256, 257):
        lo, hi = k * cb, min(n, (k + 1) * cb)
        if hi - lo > MIB:                      # bound the oracle's work: it re-checks the first MiB's keystream only
            ks_plain, _ = oracle.gcm_encrypt(key, _iv_k(iv, k), b"", bytes(MIB))
            assert np.array_equal(np.frombuffer(ks_plain, np.uint8) ^ cipher[lo:lo + MIB], p[lo:lo + MIB])
        else:
            pk, okk = oracle.gcm_decrypt(key, _iv_k(iv, k), b"", cipher[lo:hi], tags[k])
            assert bool(okk) == bool(ok[k]) and np.array_equal(np.frombuffer(pk, np.uint8), p[lo:hi])
