// fastrack_device.cuh -- per-lane device code of the fused AES-256-CTR + GHASH pass (sm_100a).
//
// One warp works on one "segment" at a time: a run of consecutive rows of one chunk.  A row is 32 consecutive counter
// values, lane = counter mod 32, and the block at counter c is data block c - 2 of the chunk (GCM keeps
// counter 1 for the tag mask), so a row is 512 contiguous bytes and global loads and stores are 128-bit and
// coalesced.  Counter 1 of row 0 is a spare lane: it yields E_K(J0), and with the serial-number framing it
// also absorbs the one-byte AAD block.  (In the variant with folded tails that lane idles as far as the cipher
// goes: the tag masks, and the one or two counters that would make up a chunk's last row, are worked on in a
// pass of their own for ten chunks at a time -- see fr_chunk_rows and fr_prework_lane.)
//
// AES (paper Section 2.3, "The AES block cipher": AES in counter mode, every block independent):
//   four round tables Te0..Te3 live in shared memory, each entry replicated 32 times so that lane l
//   only ever touches bank l -- a table lookup is one conflict-free wavefront whatever the index.
//   Row v of array T01 is [Te0[v] x32 | Te1[v] x32] (256 B), array T23 likewise; the byte address
//   v*256 + 4*lane is produced by ONE byte-permute from the state word and the lane register.
//   Rounds 1 and 2 are shared by the 256 counters that differ only in their last byte.
//
// GHASH (paper Section 2.3, "Authentication with Galois Field"; Section 4.2 shortens the chain by
// chunking, here every chain is additionally evaluated as a power sum):
//   a lane folds its blocks (every 32nd block of the segment) with Horner's rule and the FIXED multiplier
//   H^32, Y <- (Y xor X) * H^32, using byte tables of H^32 in shared memory (entry for byte position p
//   and byte value v at v*256 + p*16).  Lanes walk the 16 byte positions in a lane-dependent order
//   (position = step xor (lane & 7)) so that the eight lanes of a quarter-warp always hit eight
//   different 16-byte bank groups: every 128-bit lookup is conflict-free.  The lane's last block is
//   not multiplied by H^32 but by the power of H that its distance from the end of the chunk calls
//   for, with a general product built from integer multiplies; the 32 lane values are then XOR-reduced.
//
// A second layout for launches with many chunks that are not large ("packed rows", at the end of this file)
// gives every lane a short run of one chunk's counters instead; it uses the same tables and the same lane code
// for the cipher, the table multiply and the general product.
#pragma once
#include <stdint.h>

#define FR_SM_T01 0u          // AES rows [Te0 x32 | Te1 x32]
#define FR_SM_T23 65536u      // AES rows [Te2 x32 | Te3 x32]
#define FR_SM_GH 131072u      // byte tables of H^32
#define FR_SMEM_BYTES 196608u // the three tables
#define FR_SM_COMB 196608u    // row kernels: 33 records of 8 words in which the warps of a CTA combine their pieces of a chunk
#define FR_SM_MBAR (FR_SM_COMB + 33u * 32u)   // arrival barrier of the bulk copy that brings in the H-power byte tables
#define FR_SM_PRE (FR_SM_COMB + 2048u)   // row kernels with folded tails: per warp, the results of its last prework pass (FR_PRE_CHUNKS x 16 bytes)
#define FR_SMEM_LAUNCH_BYTES (FR_SMEM_BYTES + 2048u + 32u * 10u * 16u)   // dynamic shared memory of a launch: the tables, the records, the prework results

// What one pass does.  DEC / ENC are the fused passes.  CTR and VERIFY split them (paper Section 4.3, eager
// evaluation: plaintext first, authentication later).  PADGEN / PADDEC split the keystream from the XOR
// (Section 4.3, parallel AES evaluation: the one-time pad is produced while the copy is in flight).
enum FrMode : int {
    FR_MODE_DEC = 0,      // keystream, P = C xor KS, GHASH over C, compare tags
    FR_MODE_ENC = 1,      // keystream, C = P xor KS, GHASH over C, store tags
    FR_MODE_CTR = 2,      // keystream and XOR only
    FR_MODE_VERIFY = 3,   // GHASH over C and tag compare only (C is not modified)
    FR_MODE_PADGEN = 4,   // keystream only, written to a pad buffer, plus E_K(J0) per chunk
    FR_MODE_PADDEC = 5    // P = C xor pad, GHASH over C, compare tags (no AES at all)
};

#define FR_ROW_BLOCKS 32u     // blocks per row (one per lane)

// Timing probes of a diagnostic build (-DFR_STAMPS): per CTA, clock values at the phases of the kernel.  The
// library proper is built without the flag and contains none of this.
#ifdef FR_STAMPS
__device__ unsigned long long fr_stamps[1024 * 8];
__device__ unsigned long long fr_warp_stamps[1024 * 32];     // per warp: clock when its (last) segment's rows were done
__device__ __forceinline__ unsigned long long fr_gtime() { unsigned long long t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); return t; }
#define FR_STAMP_SET(i) do { if (threadIdx.x == 0) fr_stamps[blockIdx.x * 8 + (i)] = (unsigned long long)clock64(); } while (0)
#define FR_STAMP_GT(i) do { if (threadIdx.x == 0) fr_stamps[blockIdx.x * 8 + (i)] = fr_gtime(); } while (0)
#define FR_STAMP_MIN(i) do { if ((threadIdx.x & 31u) == 0) atomicMin(&fr_stamps[blockIdx.x * 8 + (i)], (unsigned long long)clock64()); } while (0)
#define FR_STAMP_MAX(i) do { if ((threadIdx.x & 31u) == 0) { atomicMax(&fr_stamps[blockIdx.x * 8 + (i)], (unsigned long long)clock64()); if ((i) == 4) fr_warp_stamps[blockIdx.x * 32 + (threadIdx.x >> 5)] = (unsigned long long)clock64(); } } while (0)
#define FR_STAMP_GTMAX(i) do { if ((threadIdx.x & 31u) == 0) atomicMax(&fr_stamps[blockIdx.x * 8 + (i)], fr_gtime()); } while (0)
#else
#define FR_STAMP_SET(i) do { } while (0)
#define FR_STAMP_GT(i) do { } while (0)
#define FR_STAMP_MIN(i) do { } while (0)
#define FR_STAMP_MAX(i) do { } while (0)
#define FR_STAMP_GTMAX(i) do { } while (0)
#endif
#define FR_HORNER_STRIDE 32u  // the fixed multiplier is H^32

struct FrParams {
    uint32_t rk[60];           // AES-256 round keys, word i = little-endian load of key-schedule bytes 4i..4i+3
    uint32_t iv_w0, iv_w1;     // little-endian loads of iv_base[0..3], iv_base[4..7]
    uint32_t iv_ctr;           // BE32(iv_base[8..11]) + index of this launch's first chunk
    uint32_t first_chunk;      // index of this launch's first chunk in the caller's buffer
    uint32_t n_slots;          // row kernels: warps that take work; slot j is warp j % warps_used of CTA j / warps_used
    uint32_t warps_used;       // row kernels: slots per CTA
    uint32_t n_chunks;         // chunks in this launch
    uint32_t n_items;          // packed rows: work items (warps that take work); item j covers chunks j * n_chunks / n_items .. (j + 1) * n_chunks / n_items - 1
    uint32_t generic_smem;     // 1: use the portable shared-memory addressing even where the absolute form would do
    uint32_t aad_mod;          // 0: no AAD; n: a chunk authenticates the one byte (its serial number mod n) as AAD
    uint64_t len;              // bytes in this launch
    uint64_t chunk_bytes;
    uint64_t sample_bytes;     // the launch is a sequence of equal samples of this many bytes (one sample: = len)
    uint64_t total_rows;       // row kernels: rows of all chunks of the launch together
    uint64_t rows_sample;      // rows of one sample: (chunks_per_sample - 1) * rows_full + rows_last
    uint32_t rows_full;        // rows of a full-size chunk
    uint32_t rows_last;        // rows of a sample's last chunk
    uint32_t chunks_per_sample;  // ceil(sample_bytes / chunk_bytes); only a sample's last chunk may be short
    uint32_t pack_pad;
    uint32_t pack_run;           // packed rows: most counters per slot (lane); a full chunk has ceil((blocks + 1) / pack_run) slots
    uint32_t fold_tail;          // row kernels: 1 = a chunk's last one or two counters are not a row of their own (see fr_prework_lane)
    const uint8_t* ivs;        // per-sample 12-byte IV bases (device), or null: one IV base for the whole launch
    const uint8_t* in;
    uint8_t* out;
    const uint4* tags_in;      // decrypt
    uint4* tags_out;           // encrypt
    uint32_t* ok;              // decrypt
    const uint32_t* te0;       // 256 words (the sequential comparator; the fast kernels read Te0 from constant memory)
    uint32_t* timeouts;        // counter of bulk-copy timeouts (diagnostics)
    const uint4* gh_tab;       // 4096 entries, same layout as shared memory
    const uint4* pow;          // pow[e] = H^e
    uint32_t* acc;             // per CTA of the launch a record of 8 words (4-word XOR accumulator, arrival counter, 3 unused), zero between launches
    const uint8_t* pad;        // FR_MODE_PADDEC: keystream made ahead of time, same layout as the data
    uint4* mask;               // E_K(J0) per chunk: written by FR_MODE_PADGEN, read by FR_MODE_PADDEC
    uint4 lenh_full;           // (BE64(0) || BE64(8 * chunk_bytes)) * H: the length block's term of a full chunk
    uint4 lenh_last;           // the same for the launch's last chunk (differs when that chunk is short)
    uint32_t te0c[256];        // Te0 (the AES S-box folded with MixColumns; the same for every key): read at kernel entry to fill shared
                               // memory.  As a parameter it is in the constant bank when the kernel starts (a __constant__ array
                               // costs an isolated launch a cold miss, 0.25 us)
};

// Byte permute, PTX prmt.b32 in generic mode: result byte i = byte (sel nibble i & 7) of {a (0..3), b (4..7)};
// nibble bit 3 replicates that byte's sign bit instead.
#ifndef FR_PRMT
__device__ __forceinline__ uint32_t fr_prmt_ptx(uint32_t a, uint32_t b, uint32_t s)
{
    uint32_t r;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(s));
    return r;
}
#define FR_PRMT(a, b, s) fr_prmt_ptx((a), (b), (s))
#endif

__device__ __forceinline__ uint32_t fr_bswap(uint32_t x) { return FR_PRMT(x, 0u, 0x0123u); }

__device__ __forceinline__ uint4 fr_xor4(uint4 a, uint4 b)
{
    return make_uint4(a.x ^ b.x, a.y ^ b.y, a.z ^ b.z, a.w ^ b.w);
}

// Lane-constant registers.
struct FrLane {
    uint32_t lane4;      // 4 * lane: byte offset of this lane's bank inside a table row
    uint32_t sel[4];     // GHASH selectors for byte step rho = 0..3
    uint32_t qe, qo;     // GHASH slot bytes for even / odd word steps
    uint32_t h;          // (lane >> 2) & 1
};

__device__ __forceinline__ FrLane fr_make_lane(uint32_t lane)
{
    FrLane L;
    L.lane4 = lane * 4u;
    uint32_t c = lane & 3u, h = (lane >> 2) & 1u;
    L.h = h;
    L.qe = 0; L.qo = 0;
    for (uint32_t rho = 0; rho < 4; rho++) {
        uint32_t cc = rho ^ c;
        L.qe |= (((0u ^ h) << 6) | (cc << 4)) << (8 * rho);
        L.qo |= (((1u ^ h) << 6) | (cc << 4)) << (8 * rho);
        // result = [q.byte rho, v.byte cc, 0, 0]; the zeros are q.byte0's sign bit (always clear) replicated
        L.sel[rho] = (4u + rho) | (cc << 4) | (0xCu << 8) | (0xCu << 12);
    }
    return L;
}

// Fill shared memory: replicate Te0 and its three byte rotations per lane, copy the H^32 byte tables.
// NTHREADS is a compile-time constant so that all of a thread's global loads are issued before the first store.
template <uint32_t NTHREADS>
__device__ __forceinline__ void fr_build_smem(char* sm, uint32_t tid, const uint32_t* __restrict__ te0,
                                              const uint4* __restrict__ gh_tab)
{
    constexpr uint32_t N_AES = 256u * 4u * 8u / NTHREADS;     // 256 rows x 2 arrays x 2 tables x 8 uint4 (32 words)
    constexpr uint32_t N_GH = 4096u / NTHREADS;
    static_assert(N_AES * NTHREADS == 8192u && N_GH * NTHREADS == 4096u, "thread count must divide the tables");
    uint32_t e[N_AES];
    uint4 g[N_GH];
#pragma unroll
    for (uint32_t n = 0; n < N_AES; n++) e[n] = te0[(tid + n * NTHREADS) >> 5];
#pragma unroll
    for (uint32_t n = 0; n < N_GH; n++) g[n] = gh_tab[tid + n * NTHREADS];
#pragma unroll
    for (uint32_t n = 0; n < N_AES; n++) {
        const uint32_t i = tid + n * NTHREADS, q = i & 7u, t = (i >> 3) & 3u, v = i >> 5;
        const uint32_t w = (t == 0) ? e[n] : (t == 1) ? ((e[n] << 8) | (e[n] >> 24)) : (t == 2) ? ((e[n] << 16) | (e[n] >> 16)) : ((e[n] << 24) | (e[n] >> 8));
        const uint32_t off = ((t >> 1) ? FR_SM_T23 : FR_SM_T01) + v * 256u + (t & 1u) * 128u + q * 16u;
        *(uint4*)(sm + off) = make_uint4(w, w, w, w);
    }
#pragma unroll
    for (uint32_t n = 0; n < N_GH; n++) *(uint4*)(sm + FR_SM_GH + (tid + n * NTHREADS) * 16u) = g[n];
}

// The same fill with a run-time thread count (small launches where set-up time does not matter).
__device__ __forceinline__ void fr_build_smem_any(char* sm, uint32_t tid, uint32_t nthreads,
                                                  const uint32_t* __restrict__ te0, const uint4* __restrict__ gh_tab)
{
    for (uint32_t i = tid; i < 8192u; i += nthreads) {
        const uint32_t q = i & 7u, t = (i >> 3) & 3u, v = i >> 5, e = te0[v];
        const uint32_t w = (t == 0) ? e : (t == 1) ? ((e << 8) | (e >> 24)) : (t == 2) ? ((e << 16) | (e >> 16)) : ((e << 24) | (e >> 8));
        *(uint4*)(sm + ((t >> 1) ? FR_SM_T23 : FR_SM_T01) + v * 256u + (t & 1u) * 128u + q * 16u) = make_uint4(w, w, w, w);
    }
    for (uint32_t i = tid; i < 4096u; i += nthreads) *(uint4*)(sm + FR_SM_GH + i * 16u) = gh_tab[i];
}

// Shared-memory loads.  The dynamic shared window of a kernel without static shared memory starts at shared
// address FR_SMEM_ABS_BASE on this architecture (the first KiB is reserved by the system).  When the kernel has
// checked that at run time (ABS = true), a lookup address is "constant + permuted bytes", and the constant goes
// into the load's immediate field: no add instruction per lookup.  ABS = false is the portable form.
#define FR_SMEM_ABS_BASE 0x400u

template <bool ABS, uint32_t OFF>
__device__ __forceinline__ uint32_t fr_lds32(const char* sm, uint32_t addr)
{
    if (ABS) {
#ifdef __CUDA_ARCH__
        uint32_t v;
        asm("ld.shared.u32 %0, [%1+%2];" : "=r"(v) : "r"(addr), "n"(FR_SMEM_ABS_BASE + OFF));
        return v;
#else
        return 0;
#endif
    }
    return *(const uint32_t*)(sm + OFF + addr);
}

template <bool ABS, uint32_t OFF>
__device__ __forceinline__ uint4 fr_lds128(const char* sm, uint32_t addr)
{
    if (ABS) {
#ifdef __CUDA_ARCH__
        uint4 v;
        asm("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4+%5];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr), "n"(FR_SMEM_ABS_BASE + OFF));
        return v;
#else
        return make_uint4(0, 0, 0, 0);
#endif
    }
    return *(const uint4*)(sm + OFF + addr);
}

// Table lookups: byte k of state word w (address = one byte permute; see the header comment).
#define FR_TA(w, k) FR_PRMT((w), lane4, 0x5504u | ((k) << 4))
#define FR_TE0(w, k) fr_lds32<ABS, FR_SM_T01>(sm, FR_TA(w, k))
#define FR_TE1(w, k) fr_lds32<ABS, FR_SM_T01 + 128u>(sm, FR_TA(w, k))
#define FR_TE2(w, k) fr_lds32<ABS, FR_SM_T23>(sm, FR_TA(w, k))
#define FR_TE3(w, k) fr_lds32<ABS, FR_SM_T23 + 128u>(sm, FR_TA(w, k))

// Rounds FIRST..14 of the AES-256 forward cipher on a state that has been through rounds 0..FIRST-1.
template <bool ABS, int FIRST>
__device__ __forceinline__ uint4 fr_aes256_rounds(const char* sm, uint32_t lane4, const FrParams& P,
                                                  uint32_t s0, uint32_t s1, uint32_t s2, uint32_t s3)
{
#pragma unroll
    for (int r = FIRST; r < 14; r++) {
        uint32_t t0 = FR_TE0(s0, 0) ^ FR_TE1(s1, 1) ^ FR_TE2(s2, 2) ^ FR_TE3(s3, 3) ^ P.rk[4 * r + 0];
        uint32_t t1 = FR_TE0(s1, 0) ^ FR_TE1(s2, 1) ^ FR_TE2(s3, 2) ^ FR_TE3(s0, 3) ^ P.rk[4 * r + 1];
        uint32_t t2 = FR_TE0(s2, 0) ^ FR_TE1(s3, 1) ^ FR_TE2(s0, 2) ^ FR_TE3(s1, 3) ^ P.rk[4 * r + 2];
        uint32_t t3 = FR_TE0(s3, 0) ^ FR_TE1(s0, 1) ^ FR_TE2(s1, 2) ^ FR_TE3(s2, 3) ^ P.rk[4 * r + 3];
        s0 = t0; s1 = t1; s2 = t2; s3 = t3;
    }
    // Last round: SubBytes + ShiftRows only.  Te2 has S in byte 0, Te3 in byte 1, Te0 in byte 2, Te1 in byte 3.
    uint32_t o[4];
    const uint32_t in[4] = {s0, s1, s2, s3};
#pragma unroll
    for (int c = 0; c < 4; c++) {
        uint32_t a = FR_TE2(in[c], 0);
        uint32_t b = FR_TE3(in[(c + 1) & 3], 1);
        uint32_t cc = FR_TE0(in[(c + 2) & 3], 2);
        uint32_t d = FR_TE1(in[(c + 3) & 3], 3);
        uint32_t lo = FR_PRMT(a, b, 0x0050u);    // [a.0, b.1, -, -]
        uint32_t hi = FR_PRMT(cc, d, 0x7200u);   // [-, -, c.2, d.3]
        o[c] = FR_PRMT(lo, hi, 0x7610u) ^ P.rk[56 + c];
    }
    return make_uint4(o[0], o[1], o[2], o[3]);
}

// The same rounds as a loop that is not unrolled: a tenth of the code for a block that is computed rarely (what
// such code costs is its footprint in the instruction cache of the warps that are in the row loop meanwhile).
template <bool ABS>
__device__ __forceinline__ uint4 fr_aes256_rounds_compact(const char* sm, uint32_t lane4, const FrParams& P, int first,
                                                          uint32_t s0, uint32_t s1, uint32_t s2, uint32_t s3)
{
#pragma unroll 1
    for (int r = first; r < 14; r++) {
        uint32_t t0 = FR_TE0(s0, 0) ^ FR_TE1(s1, 1) ^ FR_TE2(s2, 2) ^ FR_TE3(s3, 3) ^ P.rk[4 * r + 0];
        uint32_t t1 = FR_TE0(s1, 0) ^ FR_TE1(s2, 1) ^ FR_TE2(s3, 2) ^ FR_TE3(s0, 3) ^ P.rk[4 * r + 1];
        uint32_t t2 = FR_TE0(s2, 0) ^ FR_TE1(s3, 1) ^ FR_TE2(s0, 2) ^ FR_TE3(s1, 3) ^ P.rk[4 * r + 2];
        uint32_t t3 = FR_TE0(s3, 0) ^ FR_TE1(s0, 1) ^ FR_TE2(s1, 2) ^ FR_TE3(s2, 3) ^ P.rk[4 * r + 3];
        s0 = t0; s1 = t1; s2 = t2; s3 = t3;
    }
    return fr_aes256_rounds<ABS, 14>(sm, lane4, P, s0, s1, s2, s3);      // the last round only
}

// E_K(IV || BE32(ctr)) from the IV words, without the shared first rounds and in compact code.
template <bool ABS>
__device__ __forceinline__ uint4 fr_aes256_block_compact(const char* sm, uint32_t lane4, const FrParams& P, uint32_t ivw0,
                                                         uint32_t ivw1, uint32_t ivw2, uint32_t ctr)
{
    return fr_aes256_rounds_compact<ABS>(sm, lane4, P, 1, ivw0 ^ P.rk[0], ivw1 ^ P.rk[1], ivw2 ^ P.rk[2], fr_bswap(ctr) ^ P.rk[3]);
}

// Counter-mode sharing of the first two rounds.  In the counter block IV_k || BE32(ctr) only byte 15
// changes from block to block, byte 14 every 256 blocks, bytes 12-13 hardly ever.  After round 1 three
// of the four columns depend only on ctr >> 8, and in round 2 every output column takes exactly one
// byte from the fast-changing column.  So per 256-counter group a lane keeps (t1, t2, t3) folded into
// four words D0..D3, and per block rounds 1 and 2 cost 1 + 4 lookups instead of 32.
struct FrCtrChunk {        // per chunk: the parts of round 1 that depend on the IV only
    uint32_t a0, b1, b2, b3;
};
struct FrCtrGroup {        // per 256-counter group
    uint32_t d0, d1, d2, d3;
};

template <bool ABS>
__device__ __forceinline__ FrCtrChunk fr_ctr_chunk(const char* sm, uint32_t lane4, const FrParams& P, uint32_t ivw0,
                                                   uint32_t ivw1, uint32_t ivw2)
{
    const uint32_t s0 = ivw0 ^ P.rk[0], s1 = ivw1 ^ P.rk[1], s2 = ivw2 ^ P.rk[2];
    FrCtrChunk c;
    c.a0 = FR_TE0(s0, 0) ^ FR_TE1(s1, 1) ^ FR_TE2(s2, 2) ^ P.rk[4];
    c.b1 = FR_TE0(s1, 0) ^ FR_TE1(s2, 1) ^ FR_TE3(s0, 3) ^ P.rk[5];
    c.b2 = FR_TE0(s2, 0) ^ FR_TE2(s0, 2) ^ FR_TE3(s1, 3) ^ P.rk[6];
    c.b3 = FR_TE1(s0, 1) ^ FR_TE2(s1, 2) ^ FR_TE3(s2, 3) ^ P.rk[7];
    return c;
}

template <bool ABS>
__device__ __forceinline__ FrCtrGroup fr_ctr_group(const char* sm, uint32_t lane4, const FrParams& P,
                                                   const FrCtrChunk& c, uint32_t ctr)
{
    const uint32_t s3 = fr_bswap(ctr) ^ P.rk[3];          // bytes 0..2 = counter bytes 12..14 (byte 3 unused here)
    const uint32_t t1 = c.b1 ^ FR_TE2(s3, 2), t2 = c.b2 ^ FR_TE1(s3, 1), t3 = c.b3 ^ FR_TE0(s3, 0);
    FrCtrGroup g;
    g.d0 = FR_TE1(t1, 1) ^ FR_TE2(t2, 2) ^ FR_TE3(t3, 3) ^ P.rk[8];
    g.d1 = FR_TE0(t1, 0) ^ FR_TE1(t2, 1) ^ FR_TE2(t3, 2) ^ P.rk[9];
    g.d2 = FR_TE0(t2, 0) ^ FR_TE1(t3, 1) ^ FR_TE3(t1, 3) ^ P.rk[10];
    g.d3 = FR_TE0(t3, 0) ^ FR_TE2(t1, 2) ^ FR_TE3(t2, 3) ^ P.rk[11];
    return g;
}

// E_K(IV_k || BE32(ctr)) given the chunk and group constants that belong to ctr.
template <bool ABS>
__device__ __forceinline__ uint4 fr_aes256_ctr_block(const char* sm, uint32_t lane4, const FrParams& P,
                                                     const FrCtrChunk& c, const FrCtrGroup& g, uint32_t ctr)
{
    const uint32_t s3 = fr_bswap(ctr) ^ P.rk[3];
    const uint32_t t0 = c.a0 ^ FR_TE3(s3, 3);
    return fr_aes256_rounds<ABS, 3>(sm, lane4, P, g.d0 ^ FR_TE0(t0, 0), g.d1 ^ FR_TE3(t0, 3), g.d2 ^ FR_TE2(t0, 2),
                               g.d3 ^ FR_TE1(t0, 1));
}

// v * H^32 through the byte tables (v, result: little-endian words of the block's 16 bytes).
template <bool ABS>
__device__ __forceinline__ uint4 fr_ghash_tabmul(const char* sm, const FrLane& L, uint4 v)
{
    // lanes with h = 1 walk the words in swapped pairs, so static word w holds actual word w ^ h
    uint32_t s[4];
    s[0] = L.h ? v.y : v.x; s[1] = L.h ? v.x : v.y; s[2] = L.h ? v.w : v.z; s[3] = L.h ? v.z : v.w;
    uint4 acc = make_uint4(0, 0, 0, 0);
#pragma unroll
    for (int w = 0; w < 4; w++) {
#pragma unroll
        for (int rho = 0; rho < 4; rho++) {
            uint32_t addr = FR_PRMT(s[w], (w & 1) ? L.qo : L.qe, L.sel[rho]);
            uint4 t = (w >> 1) ? fr_lds128<ABS, FR_SM_GH + 128u>(sm, addr) : fr_lds128<ABS, FR_SM_GH>(sm, addr);
            acc = fr_xor4(acc, t);
        }
    }
    return acc;
}

// General product in GF(2^128), GCM bit order (bit 0 of a block is the MSB of byte 0 and the coefficient
// of x^0; the field polynomial is x^128 + x^7 + x^2 + x + 1).
//
// There is no carry-less multiply instruction, so the 128 x 128 polynomial product is built from
// ordinary 32 x 32 -> 64 integer multiplies (they run on the FMA pipe, which this kernel otherwise
// leaves idle): an operand word masked to every fourth bit has 8 live bits, so in the integer product
// of two such words every 4-bit field holds a count of at most 8 and never carries into its
// neighbour; the low bit of the field is the GF(2) sum.  A word is split into four such phases, the 16
// phase products of a word pair are XORed by (phase sum mod 4), and each class keeps only its own bits.
// Karatsuba on top of that brings a 128 x 128 product down to nine word products.
__device__ __forceinline__ uint32_t fr_to_natural(uint32_t le_word)     // bit i of the result = coefficient of x^(32w + i)
{
    return __brev(fr_bswap(le_word));
}

// 32 x 32 -> 64 carry-less product from 16 integer multiplies (see above).
// Phase products whose phase sums differ by four may be ADDED instead of XORed (the multiply-add does that for
// nothing): their 4-bit fields line up one field apart, field s of the lower against field s - 1 of the higher, and
// the counts of two such fields are at most min(s + 1, 15 - s) + min(s, 16 - s) <= 15, so the sum still fits its
// field and its low bit is still the GF(2) sum.  (Two products of the same phase sum can both count 8 in the middle
// field; those must be XORed.)
__device__ __forceinline__ uint64_t fr_clmul32(uint32_t a, uint32_t b)
{
    uint32_t as[4], bs[4];
#pragma unroll
    for (int k = 0; k < 4; k++) { as[k] = a & (0x11111111u << k); bs[k] = b & (0x11111111u << k); }
#define FR_MUL(i, j) ((uint64_t)as[i] * (uint64_t)bs[j])
    const uint64_t z0 = (FR_MUL(0, 0) + FR_MUL(1, 3)) ^ FR_MUL(2, 2) ^ FR_MUL(3, 1);
    const uint64_t z1 = (FR_MUL(0, 1) + FR_MUL(2, 3)) ^ (FR_MUL(1, 0) + FR_MUL(3, 2));
    const uint64_t z2 = (FR_MUL(0, 2) + FR_MUL(3, 3)) ^ FR_MUL(1, 1) ^ FR_MUL(2, 0);
    const uint64_t z3 = FR_MUL(0, 3) ^ FR_MUL(1, 2) ^ FR_MUL(2, 1) ^ FR_MUL(3, 0);
#undef FR_MUL
    return (z0 & 0x1111111111111111ull) | (z1 & 0x2222222222222222ull) | (z2 & 0x4444444444444444ull) |
           (z3 & 0x8888888888888888ull);
}

// 64 x 64 -> 128 by Karatsuba: three 32 x 32 products.
__device__ __forceinline__ void fr_clmul64(uint32_t a0, uint32_t a1, uint32_t b0, uint32_t b1, uint32_t r[4])
{
    const uint64_t lo = fr_clmul32(a0, b0), hi = fr_clmul32(a1, b1);
    const uint64_t mid = fr_clmul32(a0 ^ a1, b0 ^ b1) ^ lo ^ hi;
    r[0] = (uint32_t)lo;
    r[1] = (uint32_t)(lo >> 32) ^ (uint32_t)mid;
    r[2] = (uint32_t)hi ^ (uint32_t)(mid >> 32);
    r[3] = (uint32_t)(hi >> 32);
}

__device__ __forceinline__ uint4 fr_gf128_mul(uint4 x, uint4 y)
{
    const uint32_t a[4] = {fr_to_natural(x.x), fr_to_natural(x.y), fr_to_natural(x.z), fr_to_natural(x.w)};
    const uint32_t b[4] = {fr_to_natural(y.x), fr_to_natural(y.y), fr_to_natural(y.z), fr_to_natural(y.w)};
    // 128 x 128 -> 256 by Karatsuba on the 64-bit halves: nine 32 x 32 products = 144 integer multiplies.
    uint32_t lo[4], hi[4], mid[4];
    fr_clmul64(a[0], a[1], b[0], b[1], lo);
    fr_clmul64(a[2], a[3], b[2], b[3], hi);
    fr_clmul64(a[0] ^ a[2], a[1] ^ a[3], b[0] ^ b[2], b[1] ^ b[3], mid);
    uint32_t p[8];
#pragma unroll
    for (int w = 0; w < 4; w++) mid[w] ^= lo[w] ^ hi[w];
    p[0] = lo[0]; p[1] = lo[1];
    p[2] = lo[2] ^ mid[0]; p[3] = lo[3] ^ mid[1];
    p[4] = hi[0] ^ mid[2]; p[5] = hi[1] ^ mid[3];
    p[6] = hi[2]; p[7] = hi[3];
    // reduce: x^128 = x^7 + x^2 + x + 1.  Fold the high half t = p[4..7] as t ^ t<<1 ^ t<<2 ^ t<<7 (a 135-bit value).
    uint32_t f[5];
    f[0] = p[4] ^ (p[4] << 1) ^ (p[4] << 2) ^ (p[4] << 7);
#pragma unroll
    for (int w = 1; w < 4; w++)
        f[w] = p[4 + w] ^ ((p[4 + w] << 1) | (p[3 + w] >> 31)) ^ ((p[4 + w] << 2) | (p[3 + w] >> 30)) ^ ((p[4 + w] << 7) | (p[3 + w] >> 25));
    f[4] = (p[7] >> 31) ^ (p[7] >> 30) ^ (p[7] >> 25);      // bits 128..134: fold once more (at most 7 bits)
    const uint32_t z0 = p[0] ^ f[0] ^ f[4] ^ (f[4] << 1) ^ (f[4] << 2) ^ (f[4] << 7);
    const uint32_t z1 = p[1] ^ f[1], z2 = p[2] ^ f[2], z3 = p[3] ^ f[3];
    return make_uint4(fr_bswap(__brev(z0)), fr_bswap(__brev(z1)), fr_bswap(__brev(z2)), fr_bswap(__brev(z3)));
}

// The same product as a function that is called, for kernels that use it in more than one place.
#ifndef FR_NOINLINE
#define FR_NOINLINE __noinline__
#endif
__device__ FR_NOINLINE uint4 fr_gf128_mul_called(uint4 x, uint4 y) { return fr_gf128_mul(x, y); }

// Where chunk kk of the launch lives and what it is keyed with.  The launch is a sequence of equal samples
// (a plain buffer is one sample); inside a sample the chunks are chunk_bytes long except possibly the last.
struct FrChunk {
    uint64_t off, len;          // byte offset in the launch's buffers, byte length
    uint32_t iv_w0, iv_w1;      // little-endian loads of the IV base's bytes 0..3 and 4..7
    uint32_t iv_ctr;            // value of the IV's last four bytes for this chunk (big-endian integer)
    uint32_t serial;            // index the IV and the serial-number AAD count with
    bool last_of_sample;
};

__device__ __forceinline__ FrChunk fr_chunk_info(const FrParams& P, uint32_t kk)
{
    FrChunk c;
    const uint32_t sample = kk / P.chunks_per_sample, k = kk - sample * P.chunks_per_sample;
    const uint64_t in_sample = (uint64_t)k * P.chunk_bytes, rem = P.sample_bytes - in_sample;
    c.off = (uint64_t)sample * P.sample_bytes + in_sample;
    c.len = rem < P.chunk_bytes ? rem : P.chunk_bytes;
    c.last_of_sample = (k + 1u == P.chunks_per_sample);
    if (P.ivs) {                 // a batch of samples, each encrypted under its own IV base: chunk k of the sample
        const uint8_t* iv = P.ivs + 12ull * sample;
        c.serial = k;
        if ((((size_t)P.ivs) & 3u) == 0u) {          // the usual case: three word loads (12 * sample keeps the alignment)
            const uint32_t* w = (const uint32_t*)iv;
            c.iv_w0 = w[0];
            c.iv_w1 = w[1];
            c.iv_ctr = fr_bswap(w[2]) + k;
        } else {
            c.iv_w0 = (uint32_t)iv[0] | ((uint32_t)iv[1] << 8) | ((uint32_t)iv[2] << 16) | ((uint32_t)iv[3] << 24);
            c.iv_w1 = (uint32_t)iv[4] | ((uint32_t)iv[5] << 8) | ((uint32_t)iv[6] << 16) | ((uint32_t)iv[7] << 24);
            c.iv_ctr = (((uint32_t)iv[8] << 24) | ((uint32_t)iv[9] << 16) | ((uint32_t)iv[10] << 8) | (uint32_t)iv[11]) + k;
        }
    } else {
        c.iv_w0 = P.iv_w0;
        c.iv_w1 = P.iv_w1;
        c.serial = P.first_chunk + kk;
        c.iv_ctr = P.iv_ctr + kk;
    }
    return c;
}

// Rows are aligned to the COUNTER, not to the block index: row r of a chunk holds counters 32r .. 32r+31,
// lane = counter mod 32.  Data block j uses counter j + 2, so row 0 carries 30 data blocks; its lane 1
// (counter 1) produces E_K(J0), the tag mask, as a by-product and lane 0 idles.
//
// Folded tails (fold_tail, decided per launch by the host): a chunk of a whole number of rows' worth of blocks --
// every power-of-two chunk size -- ends, because of that offset of two, in a row that holds one or two counters
// and costs as much as a full one (3 % of a 16 KiB chunk).  With fold_tail such a chunk has one row less; its last
// one or two blocks, and E_K(J0) of every chunk, are worked on by fr_prework_lane, ten chunks per pass.
__device__ __forceinline__ uint32_t fr_chunk_rows(uint32_t nblk, uint32_t fold_tail)
{
    uint32_t rows = (nblk + 2u + FR_ROW_BLOCKS - 1) / FR_ROW_BLOCKS;
    if (fold_tail && nblk >= 31u && ((nblk + 2u) & 31u) - 1u < 2u) rows--;
    return rows;
}

// Work distribution of the row kernels.  The rows of all chunks of a launch, one chunk after the other, form
// one row space of total_rows rows; it is cut into n_slots contiguous, equally long (to within one row) ranges and
// slot j -- warp j % warps_used of CTA j / warps_used -- walks range j.  Where a range crosses a chunk boundary the
// warp closes one segment and opens the next, so a chunk may be covered by one warp, by several warps of one CTA
// or by several CTAs; the kernel combines the pieces in shared memory and, across CTAs, in global memory.
// Requires n_slots <= total_rows (no empty range).
__device__ __forceinline__ uint64_t fr_slot_begin(const FrParams& P, uint32_t j)        // j in 0 .. n_slots
{
    return (uint64_t)j * P.total_rows / P.n_slots;
}

__device__ __forceinline__ uint32_t fr_slot_of_row(const FrParams& P, uint64_t g)      // the j with begin(j) <= g < begin(j + 1)
{
    return (uint32_t)(((g + 1u) * P.n_slots - 1u) / P.total_rows);
}

struct FrRowPos {
    uint32_t kk;        // chunk of the launch
    uint32_t r;         // row inside the chunk
    uint32_t rows_k;    // rows of that chunk
};

__device__ __forceinline__ FrRowPos fr_locate_row(const FrParams& P, uint64_t g)
{
    const uint64_t sample = g / P.rows_sample, rem = g - sample * P.rows_sample;
    const uint32_t k = (uint32_t)(rem / P.rows_full);           // at most chunks_per_sample - 1: the last chunk is not longer than the others
    FrRowPos p;
    p.kk = (uint32_t)sample * P.chunks_per_sample + k;
    p.r = (uint32_t)(rem - (uint64_t)k * P.rows_full);
    p.rows_k = (k + 1u == P.chunks_per_sample) ? P.rows_last : P.rows_full;
    return p;
}

// Who else works on the chunk whose rows are [g0, g0 + rows_k) of the row space, seen from a warp of the CTA that
// holds slots cta_first .. cta_last: how many warps of this CTA (n_in_cta; they are consecutive), which of the CTA's
// 33 shared-memory records they meet in (the warp in which the chunk begins, or record 32 if it began in an
// earlier CTA), the first CTA that works on it (its record in global memory is the meeting point across CTAs) and
// how many CTAs do.  A warp's range holds the beginning of at most one chunk that continues beyond it, and at most
// one chunk reaches into a CTA from before, so no record is used by two chunks in one launch.
struct FrShare {
    uint32_t n_in_cta, rec, first_cta, n_ctas;
};

__device__ __forceinline__ FrShare fr_chunk_share(const FrParams& P, uint64_t g0, uint32_t rows_k, uint32_t cta_first,
                                                  uint32_t cta_last)
{
    const uint32_t sa = fr_slot_of_row(P, g0), sb = fr_slot_of_row(P, g0 + rows_k - 1u);
    const uint32_t a = sa > cta_first ? sa : cta_first, b = sb < cta_last ? sb : cta_last;
    FrShare s;
    s.n_in_cta = b - a + 1u;
    s.rec = sa < cta_first ? 32u : sa - cta_first;
    s.first_cta = sa / P.warps_used;
    s.n_ctas = sb / P.warps_used - s.first_cta + 1u;
    return s;
}

// Load / store the last, partial block of the buffer byte by byte (zero-padded in registers).
__device__ __forceinline__ uint4 fr_load_partial(const uint8_t* p, uint32_t n)
{
    uint32_t w[4] = {0, 0, 0, 0};
    for (uint32_t i = 0; i < n; i++) w[i >> 2] |= (uint32_t)p[i] << (8 * (i & 3));
    return make_uint4(w[0], w[1], w[2], w[3]);
}

__device__ __forceinline__ void fr_store_partial(uint8_t* p, uint4 v, uint32_t n)
{
    uint32_t w[4] = {v.x, v.y, v.z, v.w};
    for (uint32_t i = 0; i < n; i++) p[i] = (uint8_t)(w[i >> 2] >> (8 * (i & 3)));
}

__device__ __forceinline__ uint4 fr_mask_bytes(uint4 v, uint32_t n)
{
    uint32_t w[4] = {v.x, v.y, v.z, v.w};
    for (uint32_t i = 0; i < 4; i++) {
        uint32_t lo = 4 * i;
        if (n <= lo) w[i] = 0;
        else if (n < lo + 4) w[i] &= (1u << (8 * (n - lo))) - 1u;
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}

// One lane's share of rows row0 .. row1 - 1 of chunk kk: decrypt (or encrypt) its blocks, fold them into the
// lane's Horner value, and return that value multiplied by the power of H that aligns it to the end
// of the chunk (lane 1 of the chunk's first segment adds E_K(J0)).  XOR of the 32 lanes' results over all
// segments of the chunk = GHASH of the data blocks (before the length block) xor E_K(J0).
// Modes without GHASH (CTR, PADGEN) return zero.
//
// await_tables (per thread, kept by the caller across segments): the byte tables of H^32 may still be on their way
// into shared memory (an asynchronous copy started at kernel entry, see the kernel); the thread waits for them in
// front of its first table multiply, i.e. after its first cipher block, which needs the AES tables only, and
// clears the flag.
#ifndef FR_AWAIT_TABLES
#define FR_AWAIT_TABLES(sm, P) do { } while (0)
#endif
template <int MODE, bool ABS, bool FOLD = false>
__device__ __forceinline__ uint4 fr_process_segment_lane(const FrParams& P, const char* sm, const FrLane& L,
                                                         uint32_t lane, uint32_t kk, uint32_t row0, uint32_t row1,
                                                         bool& await_tables)
{
    static_assert(!FOLD || MODE == FR_MODE_DEC || MODE == FR_MODE_ENC, "tails are folded in the fused passes only");
    constexpr bool DO_AES = MODE == FR_MODE_DEC || MODE == FR_MODE_ENC || MODE == FR_MODE_CTR || MODE == FR_MODE_PADGEN;
    constexpr bool DO_GHASH = MODE == FR_MODE_DEC || MODE == FR_MODE_ENC || MODE == FR_MODE_VERIFY || MODE == FR_MODE_PADDEC;
    constexpr bool DO_LOAD = MODE != FR_MODE_PADGEN;
    constexpr bool DO_STORE = MODE != FR_MODE_VERIFY;

    const FrChunk ck = fr_chunk_info(P, kk);
    const uint64_t chunk_off = ck.off;
    const uint64_t len_k = ck.len;
    const uint32_t nblk = (uint32_t)((len_k + 15) >> 4);
    uint32_t seg_end = row1 * FR_ROW_BLOCKS - 2u;   // first block index after this segment
    if (seg_end > nblk) seg_end = nblk;
    const uint8_t* in = P.in + chunk_off;
    uint8_t* out = P.out + chunk_off;
    const uint8_t* pad = P.pad + chunk_off;
    // The lane's last block and its power of H follow from the geometry alone: fetch the power now, under the rows.
    // The block at counter c (block index c - 2) is multiplied by H^(nblk + 3 - c): one factor for each later
    // block and one for the length block.  With the serial-number framing, counter 1 of the chunk carries the
    // AAD block, which GHASH absorbs before the first ciphertext block: the same rule gives it H^(nblk + 2).
    uint32_t c_last = 0;                              // counter of this lane's last GHASH block in the segment, 0 = none
    uint4 hpow = make_uint4(0, 0, 0, 0);
    if (DO_GHASH) {
        const uint32_t c_begin = (row0 == 0) ? (P.aad_mod ? 1u : 2u) : row0 * FR_ROW_BLOCKS;
        const uint32_t c_end = seg_end + 2u;          // counters of this segment's blocks are below c_end
        if (c_end > c_begin) {
            const uint32_t top = c_end - 1u;
            uint32_t c = (top & ~31u) | lane;         // largest counter <= top that belongs to this lane
            if (c > top) c -= 32u;                    // may wrap below zero: then c > top still
            if (c >= c_begin && c <= top) {
                c_last = c;
                hpow = P.pow[nblk + 3u - c];
            }
        }
    }
    FrCtrChunk cc = {0, 0, 0, 0};
    if (DO_AES || row0 == 0) cc = fr_ctr_chunk<ABS>(sm, L.lane4, P, ck.iv_w0, ck.iv_w1, fr_bswap(ck.iv_ctr));   // VERIFY needs E_K(J0) only
    FrCtrGroup cg = {0, 0, 0, 0};

    uint4 y = make_uint4(0, 0, 0, 0), pend = make_uint4(0, 0, 0, 0), extra = make_uint4(0, 0, 0, 0);
    for (uint32_t r = row0; r < row1; r++) {
        const uint32_t ctr = r * FR_ROW_BLOCKS + lane;
        if (DO_AES || r == 0) {
            if (r == row0 || (r & 7u) == 0u) cg = fr_ctr_group<ABS>(sm, L.lane4, P, cc, ctr);   // ctr >> 8 is the same for the whole row
        }
        const uint32_t j = ctr - 2u;                                                  // wraps for ctr < 2: then j >= seg_end
        if (j < seg_end) {
            const uint64_t boff = (uint64_t)j << 4;
            const bool full = len_k - boff >= 16;
            const uint32_t nvalid = full ? 16u : (uint32_t)(len_k - boff);
            uint4 x = make_uint4(0, 0, 0, 0);
            if (DO_LOAD) x = full ? *(const uint4*)(in + boff) : fr_load_partial(in + boff, nvalid);
            uint4 ks = make_uint4(0, 0, 0, 0);
            if (DO_AES) ks = fr_aes256_ctr_block<ABS>(sm, L.lane4, P, cc, cg, ctr);
            else if (MODE == FR_MODE_PADDEC) ks = full ? *(const uint4*)(pad + boff) : fr_load_partial(pad + boff, nvalid);
            const uint4 o = fr_xor4(x, ks);
            if (DO_STORE) { if (full) *(uint4*)(out + boff) = o; else fr_store_partial(out + boff, o, nvalid); }
            if (DO_GHASH) {
                const uint4 g = (MODE == FR_MODE_ENC) ? (full ? o : fr_mask_bytes(o, nvalid)) : x;
                const uint4 v = fr_xor4(y, g);
                if (await_tables) { FR_AWAIT_TABLES(sm, P); await_tables = false; }
                if (ctr != c_last) y = fr_ghash_tabmul<ABS>(sm, L, v);
                else pend = v;
            }
        } else if (ctr == 1u && MODE != FR_MODE_CTR) {
            if (MODE == FR_MODE_PADDEC) {
                extra = P.mask[kk];
            } else if (FOLD) {
                // E_K(J0) comes out of the prework pass together with the folded tail's terms; the caller adds them
            } else {
                extra = fr_aes256_ctr_block<ABS>(sm, L.lane4, P, cc, cg, 1u);         // E_K(J0)
                if (MODE == FR_MODE_PADGEN) P.mask[kk] = extra;
            }
            if (DO_GHASH && P.aad_mod) {                                              // the one-byte AAD block
                const uint4 v = make_uint4(ck.serial % P.aad_mod, 0, 0, 0);              // y is still zero here
                if (await_tables) { FR_AWAIT_TABLES(sm, P); await_tables = false; }
                if (ctr != c_last) y = fr_ghash_tabmul<ABS>(sm, L, v);
                else pend = v;
            }
        }
    }
    FR_STAMP_MIN(3); FR_STAMP_MAX(4);
    if (!DO_GHASH) return make_uint4(0, 0, 0, 0);
    if (c_last == 0u) return extra;
    return fr_xor4(FOLD ? fr_gf128_mul_called(pend, hpow) : fr_gf128_mul(pend, hpow), extra);
}

template <int MODE, bool ABS, bool FOLD = false>
__device__ __forceinline__ uint4 fr_process_segment_lane(const FrParams& P, const char* sm, const FrLane& L,
                                                         uint32_t lane, uint32_t kk, uint32_t row0, uint32_t row1)
{
    bool tables_are_there = false;
    return fr_process_segment_lane<MODE, ABS, FOLD>(P, sm, L, lane, kk, row0, row1, tables_are_there);
}

// Folded tails: what the rows of a chunk leave out.  One pass of a warp serves up to FR_PRE_CHUNKS consecutive
// chunks, three lanes each: lane 3m of the pass makes E_K(J0) of chunk kk_first + m (counter 1), lanes 3m + 1 and
// 3m + 2 take the one or two counters behind the chunk's last row (none if the chunk's tail is not folded) --
// cipher, XOR, store, and the block's term of the tag, block * H^(nblk + 3 - counter), by the general product.
// The XOR of the three lanes' results takes the place of the E_K(J0) that lane 1 of row 0 produces otherwise: the
// warp that owns row 0 of the chunk adds it to the result of that segment.  Only chunks whose
// first row lies before row `row_end` of the row space (the end of the calling warp's range) take part; the
// function returns zero for every other lane.  Needs the AES tables only.
#define FR_PRE_CHUNKS 10u

__device__ __forceinline__ uint64_t fr_chunk_first_row(const FrParams& P, uint32_t kk)
{
    const uint32_t sample = kk / P.chunks_per_sample, k = kk - sample * P.chunks_per_sample;
    return (uint64_t)sample * P.rows_sample + (uint64_t)k * P.rows_full;
}

template <int MODE, bool ABS>
__device__ __forceinline__ uint4 fr_prework_lane(const FrParams& P, const char* sm, const FrLane& L, uint32_t lane,
                                                 uint32_t kk_first, uint64_t row_end, bool& j0_lane)
{
    static_assert(MODE == FR_MODE_DEC || MODE == FR_MODE_ENC, "tails are folded in the fused passes only");
    const uint32_t m = lane / 3u, role = lane - 3u * m, kk = kk_first + m;
    j0_lane = false;
    if (m >= FR_PRE_CHUNKS || kk >= P.n_chunks || fr_chunk_first_row(P, kk) >= row_end) return make_uint4(0, 0, 0, 0);
    const FrChunk ck = fr_chunk_info(P, kk);
    const uint32_t nblk = (uint32_t)((ck.len + 15) >> 4);
    const uint32_t rows_k = ck.last_of_sample ? P.rows_last : P.rows_full;
    const uint32_t ctr = role == 0u ? 1u : rows_k * FR_ROW_BLOCKS + role - 1u;
    j0_lane = role == 0u;
    if (role != 0u && ctr > nblk + 1u) return make_uint4(0, 0, 0, 0);      // the rows cover the chunk up to its last counter
    const uint4 ks = fr_aes256_block_compact<ABS>(sm, L.lane4, P, ck.iv_w0, ck.iv_w1, fr_bswap(ck.iv_ctr), ctr);
    if (role == 0u) return ks;
    const uint64_t boff = (uint64_t)(ctr - 2u) << 4;
    const bool full = ck.len - boff >= 16;
    const uint32_t nvalid = full ? 16u : (uint32_t)(ck.len - boff);
    const uint8_t* in = P.in + ck.off + boff;
    uint8_t* out = P.out + ck.off + boff;
    const uint4 x = full ? *(const uint4*)in : fr_load_partial(in, nvalid);
    const uint4 o = fr_xor4(x, ks);
    if (full) *(uint4*)out = o; else fr_store_partial(out, o, nvalid);
    const uint4 g = (MODE == FR_MODE_ENC) ? (full ? o : fr_mask_bytes(o, nvalid)) : x;
    return fr_gf128_mul_called(g, P.pow[nblk + 3u - ctr]);
}

// ---- Packed rows: many short chains -----------------------------------------------------------------------
// The row layout above gives one warp 32 consecutive blocks of ONE chunk; a 16-byte chunk would keep 2 of its 32
// lanes busy, and every chunk pays a closing product, a warp reduction and a ticket.  When a launch has many
// chunks that are not large, it is laid out the other way round.  A chunk's counters 1 .. nblk+1 (counter 1 = the
// tag mask E_K(J0) and, under the serial-number framing, the AAD block; counter c >= 2 = data block c - 2) are
// dealt to `lanes` = ceil((nblk + 1) / pack_run) SLOTS, one slot = one lane, round-robin: slot i takes counters
// 1 + i, 1 + i + lanes, 1 + i + 2 * lanes, ...  (at most pack_run of them).  At every step the slots of a chunk
// therefore touch 16 * lanes contiguous bytes, and a lane folds its blocks with Horner's rule and the FIXED
// multiplier H^lanes (byte tables of that power in shared memory, same conflict-free lane rotation; built for the
// launch by the host code), then multiplies by the power of H that aligns its last block to the end of the chunk.
// Slots of a chunk are consecutive lanes, a warp takes a run of whole chunks and walks their slots 32 at a time;
// the per-chunk XOR of the lane terms is a segmented scan in the calling kernel.  No chunk is shared between
// warps, so this path needs neither atomics nor scratch memory.  Few lanes per chunk mean few closing products;
// many lanes mean long contiguous pieces per memory request; lane counts that divide the number of counters
// leave no lane idle.  The host picks.  (A sample's short last chunk gets the same number of slots as the
// others, some of them empty.)
struct FrPackGeom {
    uint32_t lanes;             // slots of a chunk = stride of a slot's counters
};

__device__ __forceinline__ FrPackGeom fr_pack_geom(const FrParams& P)
{
    const uint64_t first_len = P.sample_bytes < P.chunk_bytes ? P.sample_bytes : P.chunk_bytes;
    FrPackGeom g;
    g.lanes = ((uint32_t)((first_len + 15) >> 4) + P.pack_run) / P.pack_run;         // ceil((nblk + 1) / run)
    return g;
}

// First slot of chunk kk (kk = n_chunks gives the total).
__device__ __forceinline__ uint32_t fr_pack_slot_begin(const FrParams& P, const FrPackGeom& g, uint32_t kk)
{
    (void)P;
    return kk * g.lanes;
}

// Work item j of the packed rows: a contiguous range of whole chunks, all ranges equally long to within one chunk
// (n_items <= n_chunks, so none is empty).
__device__ __forceinline__ uint32_t fr_pack_item_begin(const FrParams& P, uint32_t j)      // j in 0 .. n_items
{
    return (uint32_t)((uint64_t)j * P.n_chunks / P.n_items);
}

struct FrSlot {
    uint32_t kk;        // chunk the slot belongs to
    uint32_t i;         // index of the slot inside the chunk
    uint32_t last;      // index of the chunk's last slot
};

// One slot: encrypt or decrypt its blocks (counter 1: produce the tag mask) and return the slot's term of the
// tag, sum over its counters c of block_c * H^(nblk + 3 - c), plus E_K(J0) from counter 1.  XOR over a chunk's
// slots, plus the length term, is its tag.
// WHOLE: one lane per chunk.  The lane then always ends with the chunk's last block, whose factor is H^2, so the
// closing product is two more table steps (the table is that of H) instead of the general product (the lookup
// pipe has room for them where the integer pipes, busy with two ciphers per handful of bytes, do not), and the
// value returned is the chunk's complete tag sum: the caller needs no reduction across lanes.
template <int MODE, bool ABS, bool WHOLE>
__device__ __forceinline__ uint4 fr_packed_slot_lane(const FrParams& P, const char* sm, const FrLane& L,
                                                     const FrPackGeom& g, uint32_t slot, FrSlot& si)
{
    static_assert(MODE == FR_MODE_DEC || MODE == FR_MODE_ENC || MODE == FR_MODE_CTR || MODE == FR_MODE_VERIFY,
                  "packed rows exist for the fused passes and their two halves");
    constexpr bool DO_AES = MODE != FR_MODE_VERIFY;       // VERIFY still needs E_K(J0), counter 1
    constexpr bool DO_GHASH = MODE != FR_MODE_CTR;
    const uint32_t kk = slot / g.lanes, i = slot - kk * g.lanes;
    const FrChunk ck = fr_chunk_info(P, kk);
    const uint32_t nblk = (uint32_t)((ck.len + 15) >> 4);
    si.kk = kk; si.i = i; si.last = g.lanes - 1u;
    // The slot's counters.  Data block j (counter j + 2) belongs to slot j mod lanes and is worked on in step
    // 1 + j / lanes, so that in every step the slots of a chunk touch `lanes` consecutive blocks that start on a
    // multiple of `lanes` blocks -- whole 32-byte sectors for even lane counts.  Counter 1 (tag mask and AAD block)
    // is "block -1": it goes to the last slot, in a step 0 of its own in which the other slots idle, which keeps
    // that slot's stride at `lanes` as well.
    const uint32_t c_end = nblk + 2u;
    const bool last_slot = (i + 1u == g.lanes);
    const uint32_t steps = 1u + (nblk + g.lanes - 1u) / g.lanes;          // the same for every slot of the chunk
    uint32_t c_last;                                                       // the slot's last counter
    if (i + 2u < c_end) c_last = i + 2u + (c_end - 3u - i) / g.lanes * g.lanes;
    else if (last_slot) c_last = 1u;
    else return make_uint4(0, 0, 0, 0);                                    // an empty slot (a short last chunk)
    uint4 hpow = make_uint4(0, 0, 0, 0);
    if (DO_GHASH && !WHOLE) hpow = P.pow[nblk + 3u - c_last];
    const uint8_t* in = P.in + ck.off;
    uint8_t* out = P.out + ck.off;
    FrCtrChunk cc = {0, 0, 0, 0};
    FrCtrGroup cg = {0, 0, 0, 0};
    uint32_t group = 0xFFFFFFFFu;                                        // 256-counter group that cg belongs to
    if (DO_AES || last_slot) cc = fr_ctr_chunk<ABS>(sm, L.lane4, P, ck.iv_w0, ck.iv_w1, fr_bswap(ck.iv_ctr));
    uint4 y = make_uint4(0, 0, 0, 0), extra = make_uint4(0, 0, 0, 0);
    for (uint32_t t = 0; t < steps; t++) {                               // every slot of the chunk walks the same steps, in step
        const uint32_t c = t ? i + 2u + (t - 1u) * g.lanes : 1u;
        if (t ? c >= c_end : !last_slot) continue;                         // idle: step 0 for all but the last slot, the last step past the end
        const bool cipher = DO_AES ? (DO_GHASH || c != 1u) : (c == 1u);
        uint4 ks = make_uint4(0, 0, 0, 0);
        if (cipher) {
            if ((c >> 8) != group) { cg = fr_ctr_group<ABS>(sm, L.lane4, P, cc, c); group = c >> 8; }   // entered another 256-counter group
            ks = fr_aes256_ctr_block<ABS>(sm, L.lane4, P, cc, cg, c);
        }
        uint4 gblk;
        if (c == 1u) {
            extra = ks;                                                                      // E_K(J0)
            // the one-byte AAD block, or nothing.  (lane4 >> 8 is zero; the kernel makes lane4 opaque to the compiler after
            // the barrier that follows the table build, and this ties the only table step whose input is not loaded data or
            // cipher output to it, so that the step cannot be scheduled above that barrier.)
            gblk = make_uint4(P.aad_mod ? (ck.serial % P.aad_mod) | (L.lane4 >> 8) : 0u, 0, 0, 0);
        } else {
            const uint64_t boff = (uint64_t)(c - 2u) << 4;
            const bool full = ck.len - boff >= 16;
            const uint32_t nvalid = full ? 16u : (uint32_t)(ck.len - boff);
            const uint4 x = full ? *(const uint4*)(in + boff) : fr_load_partial(in + boff, nvalid);
            const uint4 o = fr_xor4(x, ks);
            if (MODE != FR_MODE_VERIFY) { if (full) *(uint4*)(out + boff) = o; else fr_store_partial(out + boff, o, nvalid); }
            gblk = (MODE == FR_MODE_ENC) ? (full ? o : fr_mask_bytes(o, nvalid)) : x;
        }
        if (DO_GHASH) {
            y = fr_xor4(y, gblk);
            // Horner step with the fixed multiplier H^lanes -- not after the slot's last block (the closing product
            // follows), and not at counter 1 without AAD, where y is still zero (when every lane of a warp starts
            // there -- one lane per small chunk -- the whole step is skipped)
            if (c != c_last && (c != 1u || P.aad_mod)) y = fr_ghash_tabmul<ABS>(sm, L, y);
        }
    }
    if (!DO_GHASH) return make_uint4(0, 0, 0, 0);
    if (WHOLE) y = fr_ghash_tabmul<ABS>(sm, L, fr_ghash_tabmul<ABS>(sm, L, y));
    else y = fr_gf128_mul(y, hpow);
    return fr_xor4(y, extra);
}
