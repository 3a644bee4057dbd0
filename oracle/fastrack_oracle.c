/*
 * fastrack_oracle.c -- plain, slow, obviously-correct CPU oracle.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the reference the CUDA path is checked against.  It is not part of the product:
 * only the tests, the smoke check and the benchmark's cpu_baseline / reference arm may build or
 * call it, and it shares no code, table or constant with the CUDA library.
 *
 * What it computes (paper Section 2.3 "AES-GCM": the AES block cipher in counter mode plus the
 * GMAC tag over GF(2^128); Section 4.2 "Multi-chaining authentication": one input is split into
 * chunks, each chunk carries its own nonce block and its own 128-bit tag).  The paper summarises
 * AES-GCM and defers to the standards it cites, so every step below is the definition from
 * FIPS-197 (AES) and NIST SP 800-38D (GCM) written out byte by byte and bit by bit:
 *
 *   - the S-box is COMPUTED from its definition (GF(2^8) inverse, then the affine map), never typed;
 *   - the cipher is byte-wise SubBytes / ShiftRows / MixColumns / AddRoundKey, no T-tables;
 *   - the GF(2^128) product is the bit-serial Algorithm 1 of SP 800-38D, no tables;
 *   - GHASH is the sequential chain Y_i = (Y_{i-1} xor X_i) * H (the chain the paper's
 *     Section 2.3 describes and Section 4.2 shortens);
 *   - the tag is GHASH xor E_K(J0) (Section 4.2 "one more AES block for the nonce" per chain).
 *
 * Readings of points the paper leaves open (all listed in the design notes):
 *   - per-chunk IV: 96-bit, IV_k = iv_base[0..7] || BE32(BE32(iv_base[8..11]) + k mod 2^32);
 *   - AAD is empty on the multi-chain path (chunk order is bound by the IV); the single-call
 *     GCM functions still take AAD so that the standards' worked examples can be run;
 *   - a partial last block is zero-padded for GHASH only; tags are 128 bits, never truncated.
 *
 * Parity pins (tests/test_oracle_*.py): FIPS-197 Appendix A.3 / C.3, the GCM specification's
 * AES-256 test cases 13-16, GF(2^128) algebraic identities and a schoolbook brute force,
 * K = 1 equals plain GCM, chunk k equals a stand-alone GCM call, decrypt(encrypt(x)) = x.
 */
#include <stdint.h>
#include <stddef.h>
#include <string.h>
#include <stdlib.h>
#include <pthread.h>

#define FO_API __attribute__((visibility("default")))

/* ------------------------------------------------------------------ AES-256, FIPS-197 ---- */

static uint8_t g_sbox[256];
static int g_sbox_ready = 0;

/* GF(2^8) product modulo x^8 + x^4 + x^3 + x + 1 (FIPS-197 Section 4.2), shift-and-add. */
static uint8_t gf256_mul(uint8_t a, uint8_t b)
{
    uint8_t p = 0;
    for (int i = 0; i < 8; i++) {
        if (b & 1) p ^= a;
        uint8_t hi = a & 0x80;
        a = (uint8_t)(a << 1);
        if (hi) a ^= 0x1b;
        b >>= 1;
    }
    return p;
}

/* FIPS-197 Section 5.1.1: multiplicative inverse (0 -> 0) by exhaustive search, then the
 * affine map b'_i = b_i ^ b_{i+4} ^ b_{i+5} ^ b_{i+6} ^ b_{i+7} ^ c_i, c = 0x63. */
static void sbox_init(void)
{
    if (g_sbox_ready) return;
    for (int x = 0; x < 256; x++) {
        uint8_t inv = 0;
        if (x != 0) {
            for (int y = 1; y < 256; y++) {
                if (gf256_mul((uint8_t)x, (uint8_t)y) == 1) { inv = (uint8_t)y; break; }
            }
        }
        uint8_t out = 0;
        for (int i = 0; i < 8; i++) {
            int bit = ((inv >> i) & 1) ^ ((inv >> ((i + 4) & 7)) & 1) ^ ((inv >> ((i + 5) & 7)) & 1)
                    ^ ((inv >> ((i + 6) & 7)) & 1) ^ ((inv >> ((i + 7) & 7)) & 1) ^ ((0x63 >> i) & 1);
            out |= (uint8_t)(bit << i);
        }
        g_sbox[x] = out;
    }
    g_sbox_ready = 1;
}

FO_API void fo_sbox(uint8_t out[256])
{
    sbox_init();
    memcpy(out, g_sbox, 256);
}

/* FIPS-197 Section 5.2, Nk = 8, Nr = 14: 60 words, stored as 240 bytes (word i = bytes 4i..4i+3). */
FO_API void fo_aes256_key_expand(const uint8_t key[32], uint8_t w[240])
{
    sbox_init();
    memcpy(w, key, 32);
    uint8_t rcon = 0x01;
    for (int i = 8; i < 60; i++) {
        uint8_t t[4];
        memcpy(t, w + 4 * (i - 1), 4);
        if (i % 8 == 0) {
            /* RotWord then SubWord then xor Rcon */
            uint8_t r0 = t[0];
            t[0] = g_sbox[t[1]] ^ rcon;
            t[1] = g_sbox[t[2]];
            t[2] = g_sbox[t[3]];
            t[3] = g_sbox[r0];
            rcon = gf256_mul(rcon, 2);
        } else if (i % 8 == 4) {
            for (int j = 0; j < 4; j++) t[j] = g_sbox[t[j]];
        }
        for (int j = 0; j < 4; j++) w[4 * i + j] = w[4 * (i - 8) + j] ^ t[j];
    }
}

/* FIPS-197 Section 5.1.  State s[r][c] = in[r + 4c]. */
FO_API void fo_aes256_encrypt_block(const uint8_t w[240], const uint8_t in[16], uint8_t out[16])
{
    uint8_t s[4][4];
    for (int c = 0; c < 4; c++)
        for (int r = 0; r < 4; r++) s[r][c] = in[r + 4 * c] ^ w[4 * c + r];
    for (int round = 1; round <= 14; round++) {
        /* SubBytes */
        for (int r = 0; r < 4; r++)
            for (int c = 0; c < 4; c++) s[r][c] = g_sbox[s[r][c]];
        /* ShiftRows: row r rotates left by r */
        for (int r = 1; r < 4; r++) {
            uint8_t row[4];
            for (int c = 0; c < 4; c++) row[c] = s[r][(c + r) & 3];
            for (int c = 0; c < 4; c++) s[r][c] = row[c];
        }
        /* MixColumns (not in the last round) */
        if (round != 14) {
            for (int c = 0; c < 4; c++) {
                uint8_t a0 = s[0][c], a1 = s[1][c], a2 = s[2][c], a3 = s[3][c];
                s[0][c] = gf256_mul(a0, 2) ^ gf256_mul(a1, 3) ^ a2 ^ a3;
                s[1][c] = a0 ^ gf256_mul(a1, 2) ^ gf256_mul(a2, 3) ^ a3;
                s[2][c] = a0 ^ a1 ^ gf256_mul(a2, 2) ^ gf256_mul(a3, 3);
                s[3][c] = gf256_mul(a0, 3) ^ a1 ^ a2 ^ gf256_mul(a3, 2);
            }
        }
        /* AddRoundKey */
        for (int c = 0; c < 4; c++)
            for (int r = 0; r < 4; r++) s[r][c] ^= w[16 * round + 4 * c + r];
    }
    for (int c = 0; c < 4; c++)
        for (int r = 0; r < 4; r++) out[r + 4 * c] = s[r][c];
}

/* ------------------------------------------------------- GF(2^128), SP 800-38D Sec. 6.3 ---- */

/* Algorithm 1: Z = X * Y.  Bit i of a block is bit (7 - i%8) of byte i/8 (bit 0 = MSB of byte 0). */
FO_API void fo_gf128_mul(const uint8_t x[16], const uint8_t y[16], uint8_t z_out[16])
{
    uint8_t z[16] = {0};
    uint8_t v[16];
    memcpy(v, y, 16);
    for (int i = 0; i < 128; i++) {
        int xi = (x[i / 8] >> (7 - (i % 8))) & 1;
        if (xi)
            for (int j = 0; j < 16; j++) z[j] ^= v[j];
        int lsb = v[15] & 1;                 /* bit 127 */
        for (int j = 15; j > 0; j--) v[j] = (uint8_t)((v[j] >> 1) | ((v[j - 1] & 1) << 7));
        v[0] >>= 1;
        if (lsb) v[0] ^= 0xe1;               /* R = 11100001 || 0^120 */
    }
    memcpy(z_out, z, 16);
}

/* H^e by repeated multiplication; H^0 is the field's one, 0x80 00..00. */
FO_API void fo_gf128_pow(const uint8_t h[16], uint64_t e, uint8_t out[16])
{
    uint8_t acc[16] = {0};
    acc[0] = 0x80;
    for (uint64_t i = 0; i < e; i++) fo_gf128_mul(acc, h, acc);
    memcpy(out, acc, 16);
}

/* One GHASH step over a byte string zero-padded to whole blocks: Y = (Y ^ X_i) * H. */
static void ghash_absorb(const uint8_t h[16], uint8_t y[16], const uint8_t* data, size_t len)
{
    size_t off = 0;
    while (off < len) {
        uint8_t blk[16] = {0};
        size_t n = len - off < 16 ? len - off : 16;
        memcpy(blk, data + off, n);
        for (int j = 0; j < 16; j++) y[j] ^= blk[j];
        fo_gf128_mul(y, h, y);
        off += n;
    }
}

static void put_be64(uint8_t* p, uint64_t v)
{
    for (int i = 0; i < 8; i++) p[i] = (uint8_t)(v >> (56 - 8 * i));
}

/* SP 800-38D Sec. 6.4 applied as in Sec. 7.1 step 5: pad(A) || pad(C) || [len(A)]_64 || [len(C)]_64. */
FO_API void fo_ghash(const uint8_t h[16], const uint8_t* aad, size_t aad_len,
                     const uint8_t* c, size_t c_len, uint8_t out[16])
{
    uint8_t y[16] = {0};
    ghash_absorb(h, y, aad, aad_len);
    ghash_absorb(h, y, c, c_len);
    uint8_t lens[16];
    put_be64(lens, (uint64_t)aad_len * 8);
    put_be64(lens + 8, (uint64_t)c_len * 8);
    ghash_absorb(h, y, lens, 16);
    memcpy(out, y, 16);
}

/* Closed form of the chain, used only to cross-check the chain itself and power tables:
 * sum over blocks X_1..X_m of X_i * H^(m - i + 1), each power built by repeated multiplication. */
FO_API void fo_ghash_pow(const uint8_t h[16], const uint8_t* blocks, size_t m, uint8_t out[16])
{
    uint8_t acc[16] = {0};
    for (size_t i = 1; i <= m; i++) {
        uint8_t p[16], t[16];
        fo_gf128_pow(h, (uint64_t)(m - i + 1), p);
        fo_gf128_mul(blocks + 16 * (i - 1), p, t);
        for (int j = 0; j < 16; j++) acc[j] ^= t[j];
    }
    memcpy(out, acc, 16);
}

/* ----------------------------------------------------------------- GCM, SP 800-38D Sec. 7 ---- */

/* inc32: add 1 to the last four bytes as a big-endian integer mod 2^32. */
static void inc32(uint8_t cb[16])
{
    for (int i = 15; i >= 12; i--) {
        cb[i]++;
        if (cb[i] != 0) break;
    }
}

/* GCTR with ICB = inc32(J0); the last block uses only the bytes it needs. */
static void gctr(const uint8_t w[240], const uint8_t j0[16], const uint8_t* in, size_t len, uint8_t* out)
{
    uint8_t cb[16], ks[16];
    memcpy(cb, j0, 16);
    size_t off = 0;
    while (off < len) {
        inc32(cb);
        fo_aes256_encrypt_block(w, cb, ks);
        size_t n = len - off < 16 ? len - off : 16;
        for (size_t j = 0; j < n; j++) out[off + j] = in[off + j] ^ ks[j];
        off += n;
    }
}

static void gcm_tag(const uint8_t w[240], const uint8_t j0[16], const uint8_t* aad, size_t aad_len,
                    const uint8_t* c, size_t len, uint8_t tag[16])
{
    uint8_t zero[16] = {0}, h[16], s[16], ekj0[16];
    fo_aes256_encrypt_block(w, zero, h);
    fo_ghash(h, aad, aad_len, c, len, s);
    fo_aes256_encrypt_block(w, j0, ekj0);
    for (int j = 0; j < 16; j++) tag[j] = s[j] ^ ekj0[j];
}

/* Algorithm 4 with a 96-bit IV: J0 = IV || 0^31 || 1. */
FO_API void fo_gcm_encrypt(const uint8_t key[32], const uint8_t iv[12],
                           const uint8_t* aad, size_t aad_len,
                           const uint8_t* p, size_t len, uint8_t* c, uint8_t tag[16])
{
    uint8_t w[240], j0[16];
    fo_aes256_key_expand(key, w);
    memcpy(j0, iv, 12);
    j0[12] = 0; j0[13] = 0; j0[14] = 0; j0[15] = 1;
    gctr(w, j0, p, len, c);
    gcm_tag(w, j0, aad, aad_len, c, len, tag);
}

/* Algorithm 5.  The plaintext is written whatever the verdict (the paper's eager evaluation,
 * Section 4.3, releases it before the verdict); returns 1 if all 128 tag bits match, else 0. */
FO_API int fo_gcm_decrypt(const uint8_t key[32], const uint8_t iv[12],
                          const uint8_t* aad, size_t aad_len,
                          const uint8_t* c, size_t len, const uint8_t tag[16], uint8_t* p)
{
    uint8_t w[240], j0[16], t[16];
    fo_aes256_key_expand(key, w);
    memcpy(j0, iv, 12);
    j0[12] = 0; j0[13] = 0; j0[14] = 0; j0[15] = 1;
    gcm_tag(w, j0, aad, aad_len, c, len, t);
    gctr(w, j0, c, len, p);
    uint8_t diff = 0;
    for (int j = 0; j < 16; j++) diff |= (uint8_t)(t[j] ^ tag[j]);
    return diff == 0;
}

/* ------------------------------------------------ multi-chaining (paper Section 4.2) ---- */

/* IV of chunk k: first 8 bytes of iv_base, then BE32(BE32(iv_base[8..11]) + k mod 2^32). */
FO_API void fo_chunk_iv(const uint8_t iv_base[12], uint64_t k, uint8_t iv[12])
{
    memcpy(iv, iv_base, 8);
    uint32_t ctr = ((uint32_t)iv_base[8] << 24) | ((uint32_t)iv_base[9] << 16)
                 | ((uint32_t)iv_base[10] << 8) | (uint32_t)iv_base[11];
    ctr += (uint32_t)k;
    iv[8] = (uint8_t)(ctr >> 24); iv[9] = (uint8_t)(ctr >> 16);
    iv[10] = (uint8_t)(ctr >> 8); iv[11] = (uint8_t)ctr;
}

FO_API size_t fo_num_chunks(size_t len, size_t chunk_bytes)
{
    if (len == 0 || chunk_bytes == 0) return 0;
    return (len + chunk_bytes - 1) / chunk_bytes;
}

typedef struct {
    const uint8_t* key;
    const uint8_t* iv_base;
    size_t chunk_bytes, len, k_first, k_step, k_count_total;
    const uint8_t* in;
    uint8_t* out;
    uint8_t* tags_out;          /* encrypt */
    const uint8_t* tags_in;     /* decrypt */
    uint32_t* ok;               /* decrypt */
    int encrypt;
    unsigned chains_per_sample; /* 0: no AAD; n > 0: chunk k carries the one-byte AAD (k mod n) */
} mc_job;

static void* mc_worker(void* arg)
{
    mc_job* j = (mc_job*)arg;
    for (size_t k = j->k_first; k < j->k_count_total; k += j->k_step) {
        size_t off = k * j->chunk_bytes;
        size_t n = j->len - off < j->chunk_bytes ? j->len - off : j->chunk_bytes;
        uint8_t iv[12];
        fo_chunk_iv(j->iv_base, k, iv);
        /* paper Section 4.2 / 4.4: one byte of AAD per chunk holds its serial number inside the sample */
        uint8_t serial = j->chains_per_sample ? (uint8_t)(k % j->chains_per_sample) : 0;
        const uint8_t* aad = j->chains_per_sample ? &serial : NULL;
        size_t aad_len = j->chains_per_sample ? 1 : 0;
        if (j->encrypt)
            fo_gcm_encrypt(j->key, iv, aad, aad_len, j->in + off, n, j->out + off, j->tags_out + 16 * k);
        else
            j->ok[k] = (uint32_t)fo_gcm_decrypt(j->key, iv, aad, aad_len, j->in + off, n,
                                                j->tags_in + 16 * k, j->out + off);
    }
    return NULL;
}

/* Chunks are independent GCM calls; worker t takes chunks t, t + n_threads, ... */
static void mc_run(mc_job proto, int n_threads)
{
    size_t K = fo_num_chunks(proto.len, proto.chunk_bytes);
    proto.k_count_total = K;
    if (K == 0) return;
    if (n_threads < 1) n_threads = 1;
    if ((size_t)n_threads > K) n_threads = (int)K;
    sbox_init();                 /* before any thread reads it */
    if (n_threads == 1) {
        proto.k_first = 0; proto.k_step = 1;
        mc_worker(&proto);
        return;
    }
    pthread_t* th = (pthread_t*)malloc(sizeof(pthread_t) * (size_t)n_threads);
    mc_job* jobs = (mc_job*)malloc(sizeof(mc_job) * (size_t)n_threads);
    for (int t = 0; t < n_threads; t++) {
        jobs[t] = proto;
        jobs[t].k_first = (size_t)t;
        jobs[t].k_step = (size_t)n_threads;
        pthread_create(&th[t], NULL, mc_worker, &jobs[t]);
    }
    for (int t = 0; t < n_threads; t++) pthread_join(th[t], NULL);
    free(th); free(jobs);
}

/* Encrypt + one tag per chunk.  c[len], tags[16*K]. */
FO_API void fo_mc_encrypt(const uint8_t key[32], const uint8_t iv_base[12], size_t chunk_bytes,
                          const uint8_t* p, size_t len, uint8_t* c, uint8_t* tags, int n_threads)
{
    mc_job j; memset(&j, 0, sizeof j);
    j.key = key; j.iv_base = iv_base; j.chunk_bytes = chunk_bytes; j.len = len;
    j.in = p; j.out = c; j.tags_out = tags; j.encrypt = 1;
    mc_run(j, n_threads);
}

/* Decrypt + verify each chunk.  p[len], ok[K] = 1 accept / 0 reject. */
FO_API void fo_mc_decrypt(const uint8_t key[32], const uint8_t iv_base[12], size_t chunk_bytes,
                          const uint8_t* c, size_t len, const uint8_t* tags,
                          uint8_t* p, uint32_t* ok, int n_threads)
{
    mc_job j; memset(&j, 0, sizeof j);
    j.key = key; j.iv_base = iv_base; j.chunk_bytes = chunk_bytes; j.len = len;
    j.in = c; j.out = p; j.tags_in = tags; j.ok = ok; j.encrypt = 0;
    mc_run(j, n_threads);
}

/* Paper-faithful framing (Sections 4.2 and 4.4): every sample is cut into chains_per_sample chunks and each
 * chunk authenticates, as its one byte of AAD, its serial number inside the sample (k mod chains_per_sample).
 * Everything else is as in fo_mc_encrypt / fo_mc_decrypt; chains_per_sample in 1..256. */
FO_API void fo_mc_encrypt_framed(const uint8_t key[32], const uint8_t iv_base[12], size_t chunk_bytes,
                                 unsigned chains_per_sample, const uint8_t* p, size_t len, uint8_t* c,
                                 uint8_t* tags, int n_threads)
{
    mc_job j; memset(&j, 0, sizeof j);
    j.key = key; j.iv_base = iv_base; j.chunk_bytes = chunk_bytes; j.len = len;
    j.in = p; j.out = c; j.tags_out = tags; j.encrypt = 1; j.chains_per_sample = chains_per_sample;
    mc_run(j, n_threads);
}

FO_API void fo_mc_decrypt_framed(const uint8_t key[32], const uint8_t iv_base[12], size_t chunk_bytes,
                                 unsigned chains_per_sample, const uint8_t* c, size_t len, const uint8_t* tags,
                                 uint8_t* p, uint32_t* ok, int n_threads)
{
    mc_job j; memset(&j, 0, sizeof j);
    j.key = key; j.iv_base = iv_base; j.chunk_bytes = chunk_bytes; j.len = len;
    j.in = c; j.out = p; j.tags_in = tags; j.ok = ok; j.encrypt = 0; j.chains_per_sample = chains_per_sample;
    mc_run(j, n_threads);
}
