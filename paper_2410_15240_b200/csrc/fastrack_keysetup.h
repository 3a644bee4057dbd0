// fastrack_keysetup.h -- host-side key derivation, run once per context: the AES S-box and round
// table, the AES-256 key schedule, one block encryption (for the hash subkey H = E_K(0^128), paper
// Section 2.3) and a GF(2^128) product used to build the byte tables of H^32.  Plain C++; none of
// this touches payload data.
#pragma once
#include <stdint.h>
#include <string.h>

namespace fr_host {

struct Gf128 { uint64_t hi, lo; };   // hi = bytes 0..7 big-endian (bit 0 of the block = bit 63 of hi)

inline Gf128 gf_load(const uint8_t b[16])
{
    Gf128 r = {0, 0};
    for (int i = 0; i < 8; i++) { r.hi = (r.hi << 8) | b[i]; r.lo = (r.lo << 8) | b[8 + i]; }
    return r;
}

inline void gf_store(Gf128 v, uint8_t b[16])
{
    for (int i = 0; i < 8; i++) { b[i] = (uint8_t)(v.hi >> (56 - 8 * i)); b[8 + i] = (uint8_t)(v.lo >> (56 - 8 * i)); }
}

// Product in GF(2^128) with GCM's bit order: walk the bits of a from x^0 up while b is multiplied by x.
inline Gf128 gf_mul(Gf128 a, Gf128 b)
{
    Gf128 z = {0, 0};
    for (int i = 0; i < 128; i++) {
        uint64_t bit = (i < 64) ? (a.hi >> (63 - i)) & 1 : (a.lo >> (127 - i)) & 1;
        if (bit) { z.hi ^= b.hi; z.lo ^= b.lo; }
        uint64_t carry = b.lo & 1;
        b.lo = (b.lo >> 1) | (b.hi << 63);
        b.hi >>= 1;
        if (carry) b.hi ^= 0xE100000000000000ull;
    }
    return z;
}

inline uint8_t xtime(uint8_t a) { return (uint8_t)((a << 1) ^ ((a >> 7) * 0x1b)); }

// S-box from the discrete logarithm to base 3 in GF(2^8): inverse(a) = 3^(255 - log a), then the affine map.
inline void make_sbox(uint8_t sbox[256])
{
    uint8_t exp3[256], log3[256];
    uint8_t v = 1;
    for (int i = 0; i < 255; i++) { exp3[i] = v; log3[v] = (uint8_t)i; v = (uint8_t)(v ^ xtime(v)); }
    exp3[255] = exp3[0];
    for (int a = 0; a < 256; a++) {
        uint8_t inv = (a == 0) ? 0 : exp3[(255 - log3[a]) % 255];
        uint8_t r = inv;
        r ^= (uint8_t)((inv << 1) | (inv >> 7));
        r ^= (uint8_t)((inv << 2) | (inv >> 6));
        r ^= (uint8_t)((inv << 3) | (inv >> 5));
        r ^= (uint8_t)((inv << 4) | (inv >> 4));
        sbox[a] = (uint8_t)(r ^ 0x63);
    }
}

// Key schedule as 60 little-endian words.
inline void expand_key(const uint8_t key[32], const uint8_t sbox[256], uint32_t rk[60])
{
    for (int i = 0; i < 8; i++)
        rk[i] = (uint32_t)key[4 * i] | ((uint32_t)key[4 * i + 1] << 8) | ((uint32_t)key[4 * i + 2] << 16) | ((uint32_t)key[4 * i + 3] << 24);
    uint8_t rcon = 1;
    for (int i = 8; i < 60; i++) {
        uint32_t t = rk[i - 1];
        if ((i & 7) == 0) {
            t = (t >> 8) | (t << 24);    // RotWord on little-endian bytes
            t = (uint32_t)sbox[t & 0xff] | ((uint32_t)sbox[(t >> 8) & 0xff] << 8) | ((uint32_t)sbox[(t >> 16) & 0xff] << 16) | ((uint32_t)sbox[t >> 24] << 24);
            t ^= rcon;
            rcon = xtime(rcon);
        } else if ((i & 7) == 4) {
            t = (uint32_t)sbox[t & 0xff] | ((uint32_t)sbox[(t >> 8) & 0xff] << 8) | ((uint32_t)sbox[(t >> 16) & 0xff] << 16) | ((uint32_t)sbox[t >> 24] << 24);
        }
        rk[i] = rk[i - 8] ^ t;
    }
}

// One block through the cipher with the round table Te0 (used once per context, for H).
inline void encrypt_block_host(const uint32_t rk[60], const uint32_t te0[256], const uint8_t sbox[256], const uint8_t in[16], uint8_t out[16])
{
    auto rotl = [](uint32_t x, int n) { return (x << n) | (x >> (32 - n)); };
    uint32_t s[4], t[4];
    for (int c = 0; c < 4; c++)
        s[c] = ((uint32_t)in[4 * c] | ((uint32_t)in[4 * c + 1] << 8) | ((uint32_t)in[4 * c + 2] << 16) | ((uint32_t)in[4 * c + 3] << 24)) ^ rk[c];
    for (int r = 1; r < 14; r++) {
        for (int c = 0; c < 4; c++)
            t[c] = te0[s[c] & 0xff] ^ rotl(te0[(s[(c + 1) & 3] >> 8) & 0xff], 8) ^ rotl(te0[(s[(c + 2) & 3] >> 16) & 0xff], 16) ^
                   rotl(te0[s[(c + 3) & 3] >> 24], 24) ^ rk[4 * r + c];
        memcpy(s, t, sizeof s);
    }
    for (int c = 0; c < 4; c++) {
        t[c] = ((uint32_t)sbox[s[c] & 0xff] | ((uint32_t)sbox[(s[(c + 1) & 3] >> 8) & 0xff] << 8) |
                ((uint32_t)sbox[(s[(c + 2) & 3] >> 16) & 0xff] << 16) | ((uint32_t)sbox[s[(c + 3) & 3] >> 24] << 24)) ^ rk[56 + c];
        out[4 * c] = (uint8_t)t[c]; out[4 * c + 1] = (uint8_t)(t[c] >> 8); out[4 * c + 2] = (uint8_t)(t[c] >> 16); out[4 * c + 3] = (uint8_t)(t[c] >> 24);
    }
}

}  // namespace fr_host

