// emulate.cpp -- TEST INFRASTRUCTURE ONLY: the per-lane device functions of the CUDA library
// (paper_2410_15240_b200/csrc/fastrack_device.cuh) compiled as plain C++ and driven lane by lane on the host,
// so that the CPU-only test run can compare the kernels' arithmetic (table layouts, lane rotations, counter
// sharing, Horner exponents, ragged tails, framing, every pass mode) with the oracle before anything reaches
// a GPU.  It stands in for the few lines of kernel code that are not in that header: shared memory is a host
// array, the warp XOR tree and the per-chunk accumulator are plain loops.  It is built by
// tests/test_device_code_on_host.py into a temporary directory, is never shipped, and nothing in the product
// can reach it (the product has no CPU data path).
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <map>
#include <set>
#include <utility>
#include <vector>

// ---- what the device header needs from CUDA, as plain C++ ----
#define __device__
#define __forceinline__ inline
#define FR_NOINLINE inline
struct uint4 { uint32_t x, y, z, w; };
static inline uint4 make_uint4(uint32_t a, uint32_t b, uint32_t c, uint32_t d) { return uint4{a, b, c, d}; }

// PTX prmt.b32, generic mode: nibble bits 0-2 pick a byte of {a, b}, bit 3 replicates that byte's sign bit.
static inline uint32_t host_prmt(uint32_t a, uint32_t b, uint32_t s)
{
    uint8_t src[8];
    for (int i = 0; i < 4; i++) { src[i] = (uint8_t)(a >> (8 * i)); src[4 + i] = (uint8_t)(b >> (8 * i)); }
    uint32_t r = 0;
    for (int i = 0; i < 4; i++) {
        const uint32_t n = (s >> (4 * i)) & 0xf;
        uint8_t v = src[n & 7];
        if (n & 8) v = (v & 0x80) ? 0xff : 0x00;
        r |= (uint32_t)v << (8 * i);
    }
    return r;
}
#define FR_PRMT(a, b, s) host_prmt((a), (b), (s))

static inline uint32_t __brev(uint32_t x)
{
    uint32_t r = 0;
    for (int i = 0; i < 32; i++) r |= ((x >> i) & 1u) << (31 - i);
    return r;
}

#include "../../paper_2410_15240_b200/csrc/fastrack_device.cuh"
#include "../../paper_2410_15240_b200/csrc/fastrack_keysetup.h"
#include "../../paper_2410_15240_b200/csrc/fastrack_plan.h"
using namespace fr_host;

namespace {

struct Setup {
    FrParams P;
    uint32_t te0[256];
    uint8_t h[16];
    std::vector<uint8_t> gh_tab;     // byte tables of H^32
    std::vector<uint4> pow;          // powers of H
    std::vector<char> sm;            // the "shared memory" image
};

// The same derivation fastrack_ctx_create performs (host part) plus the power table and the shared-memory fill.
void setup(Setup& S, const uint8_t key[32], size_t cb, uint32_t power = 32)   // byte tables of H^power: H^32 for the rows, H^lanes for the packed rows
{
    memset(&S.P, 0, sizeof S.P);
    uint8_t sbox[256];
    make_sbox(sbox);
    for (int v = 0; v < 256; v++) {
        const uint8_t s1 = sbox[v], s2 = xtime(s1), s3 = (uint8_t)(s2 ^ s1);
        S.te0[v] = (uint32_t)s2 | ((uint32_t)s1 << 8) | ((uint32_t)s1 << 16) | ((uint32_t)s3 << 24);
    }
    expand_key(key, sbox, S.P.rk);
    const uint8_t zero[16] = {0};
    encrypt_block_host(S.P.rk, S.te0, sbox, zero, S.h);
    const Gf128 H = gf_load(S.h);
    Gf128 G = H;
    for (uint32_t i = 1; i < power; i++) G = gf_mul(G, H);
    S.gh_tab.assign(65536, 0);
    for (int p = 0; p < 16; p++) {
        Gf128 basis[8];
        for (int b = 0; b < 8; b++) {
            uint8_t blk[16] = {0};
            blk[p] = (uint8_t)(1u << b);
            basis[b] = gf_mul(gf_load(blk), G);
        }
        for (int v = 0; v < 256; v++) {
            Gf128 acc = {0, 0};
            for (int b = 0; b < 8; b++)
                if (v & (1 << b)) { acc.hi ^= basis[b].hi; acc.lo ^= basis[b].lo; }
            gf_store(acc, &S.gh_tab[(size_t)v * 256 + (size_t)p * 16]);
        }
    }
    const size_t npow = cb / 16 + 66;
    S.pow.assign(npow, uint4{0, 0, 0, 0});
    uint8_t seed[32] = {0};
    seed[0] = 0x80;
    memcpy(seed + 16, S.h, 16);
    memcpy(S.pow.data(), seed, 32);
    for (size_t half = 1; half + 1 < npow; half *= 2)                       // fr_pow_double_kernel, pass by pass
        for (size_t i = half + 1; i <= std::min(2 * half, npow - 1); i++) S.pow[i] = fr_gf128_mul(S.pow[i - half], S.pow[half]);
    S.sm.assign(FR_SMEM_BYTES, 0);
    for (uint32_t tid = 0; tid < 1024; tid++) fr_build_smem<1024>(S.sm.data(), tid, S.te0, (const uint4*)S.gh_tab.data());
    S.P.te0 = S.te0;
    S.P.gh_tab = (const uint4*)S.gh_tab.data();
    S.P.pow = S.pow.data();
}

uint4 length_term(const Setup& S, uint64_t bytes, uint32_t aad_mod)
{
    uint8_t blk[16] = {0}, o[16];
    const uint64_t bits = bytes * 8;
    if (aad_mod) blk[7] = 8;
    for (int i = 0; i < 8; i++) blk[8 + i] = (uint8_t)(bits >> (56 - 8 * i));
    gf_store(gf_mul(gf_load(blk), gf_load(S.h)), o);
    uint4 r;
    memcpy(&r, o, 16);
    return r;
}

// The row kernels' work distribution, slot by slot as fr_crypt_body walks it (the slots stand for warps), with
// the XOR of the pieces of a chunk done in a plain array instead of the shared-memory and global records.  What the
// kernel derives from fr_chunk_share -- how many warps of the CTA and how many CTAs meet on a chunk, and in which
// record -- is checked here against what the walk really does.  Returns 0, or a code that says which check failed.
template <int MODE, bool FOLD = false>
int run_pass(Setup& S, std::vector<uint4>& acc)
{
    const FrParams& P = S.P;
    struct Piece { uint32_t slot; uint64_t g0; uint32_t rows_k; };
    std::map<uint32_t, std::vector<Piece>> partial;          // chunk -> pieces of it that are not the whole chunk
    std::vector<uint32_t> pieces_of(P.n_chunks, 0);
    std::vector<uint64_t> rows_done(P.n_chunks, 0);
    if (P.n_slots == 0 || P.n_slots > P.total_rows) return 10;
    for (uint32_t slot = 0; slot < P.n_slots; slot++) {
        uint64_t g = fr_slot_begin(P, slot);
        const uint64_t end = fr_slot_begin(P, slot + 1u);
        if (end <= g) return 11;                                                     // no empty range
        if (fr_slot_of_row(P, g) != slot || fr_slot_of_row(P, end - 1) != slot) return 12;
        uint4 pre_results[FR_PRE_CHUNKS];                                            // folded tails, as fr_crypt_body keeps them
        uint32_t pre_first = 0, pre_count = 0;
        while (g < end) {
            const FrRowPos pos = fr_locate_row(P, g);
            if (pos.kk >= P.n_chunks || pos.r >= pos.rows_k) return 13;
            uint32_t take = pos.rows_k - pos.r;
            if (take > end - g) take = (uint32_t)(end - g);
            bool add_pre = false;
            if constexpr (FOLD) {
                if (pos.r == 0u) {
                    if (pos.kk - pre_first >= pre_count) {
                        uint4 t[34];
                        bool j0_lane[32];
                        for (uint32_t lane = 0; lane < 32; lane++)
                            t[lane] = fr_prework_lane<MODE, false>(P, S.sm.data(), fr_make_lane(lane), lane, pos.kk, end, j0_lane[lane]);
                        t[32] = t[33] = uint4{0, 0, 0, 0};
                        pre_count = 0;
                        for (uint32_t lane = 0; lane < 32; lane++) {
                            if (!j0_lane[lane]) continue;
                            if (lane % 3u != 0u || lane / 3u != pre_count) return 21;        // the chunks of a pass are consecutive, three lanes each
                            pre_results[pre_count++] = fr_xor4(t[lane], fr_xor4(t[lane + 1], t[lane + 2]));
                        }
                        pre_first = pos.kk;
                        if (pre_count == 0) return 22;                                       // the chunk that asked is always served
                    }
                    add_pre = true;
                }
            }
            for (uint32_t lane = 0; lane < 32; lane++) {                             // the warp, one lane after the other
                const FrLane L = fr_make_lane(lane);
                acc[pos.kk] = fr_xor4(acc[pos.kk], fr_process_segment_lane<MODE, false, FOLD>(P, S.sm.data(), L, lane, pos.kk, pos.r, pos.r + take));
            }
            if (add_pre) acc[pos.kk] = fr_xor4(acc[pos.kk], pre_results[pos.kk - pre_first]);
            pieces_of[pos.kk]++;
            rows_done[pos.kk] += take;
            if (take != pos.rows_k) partial[pos.kk].push_back(Piece{slot, g - pos.r, pos.rows_k});
            g += take;
        }
    }
    if (fr_slot_begin(P, P.n_slots) != P.total_rows) return 14;
    for (uint32_t kk = 0; kk < P.n_chunks; kk++)
        if (rows_done[kk] == 0 || (pieces_of[kk] > 1) != (partial.count(kk) != 0)) return 15;
    std::set<std::pair<uint32_t, uint32_t>> shared_recs;     // (CTA, record) pairs in use
    std::set<uint32_t> global_recs;
    for (const auto& kv : partial) {
        const std::vector<Piece>& v = kv.second;
        std::map<uint32_t, uint32_t> per_cta;
        for (const Piece& pc : v) per_cta[pc.slot / P.warps_used]++;
        for (const Piece& pc : v) {
            const uint32_t cta = pc.slot / P.warps_used, cta_first = cta * P.warps_used;
            uint32_t cta_last = cta_first + P.warps_used - 1u;
            if (cta_last >= P.n_slots) cta_last = P.n_slots - 1u;
            const FrShare sh = fr_chunk_share(P, pc.g0, pc.rows_k, cta_first, cta_last);
            if (sh.n_in_cta != per_cta[cta]) return 16;
            if (sh.n_ctas != per_cta.size() || sh.first_cta != per_cta.begin()->first) return 17;
            if (sh.rec > 32u || (sh.rec < 32u && sh.rec >= P.warps_used)) return 18;
        }
        for (const auto& c : per_cta) {
            const uint32_t cta_first = c.first * P.warps_used;
            uint32_t cta_last = cta_first + P.warps_used - 1u;
            if (cta_last >= P.n_slots) cta_last = P.n_slots - 1u;
            const FrShare sh = fr_chunk_share(P, v[0].g0, v[0].rows_k, cta_first, cta_last);
            if (c.second > 1 && !shared_recs.insert({c.first, sh.rec}).second) return 19;      // one chunk per shared record
        }
        if (per_cta.size() > 1 && !global_recs.insert(per_cta.begin()->first).second) return 20;   // one chunk per global record
    }
    return 0;
}

}  // namespace

// One pass of mode `mode` (FrMode) over a buffer, laid out by the library's own planner (fr_plan_rows) for a GPU of
// `num_sms` SMs; rows_per_slot > 0 asks for that many rows per warp instead of the planner's choice (any value >= 1).
extern "C" int emu_pass(int mode, const uint8_t* key, const uint8_t* iv_base, size_t cb, const uint8_t* in, size_t len,
                        uint8_t* out, const uint8_t* pad, uint8_t* mask, const uint8_t* tags_in, uint8_t* tags_out,
                        uint32_t* ok, uint32_t rows_per_slot, uint32_t num_sms, uint32_t first_chunk, uint32_t aad_mod,
                        size_t sample_bytes, const uint8_t* ivs, uint32_t fold_mode)
{
    Setup S;
    setup(S, key, cb);
    FrParams& P = S.P;
    auto be32 = [](const uint8_t* p) { return ((uint32_t)p[0] << 24) | ((uint32_t)p[1] << 16) | ((uint32_t)p[2] << 8) | p[3]; };
    auto le32 = [](const uint8_t* p) { return ((uint32_t)p[3] << 24) | ((uint32_t)p[2] << 16) | ((uint32_t)p[1] << 8) | p[0]; };
    P.iv_w0 = le32(iv_base);
    P.iv_w1 = le32(iv_base + 4);
    P.iv_ctr = be32(iv_base + 8) + first_chunk;
    P.first_chunk = first_chunk;
    P.aad_mod = aad_mod;
    P.len = len;
    P.chunk_bytes = cb;
    if (sample_bytes == 0) sample_bytes = len;                                   // a plain buffer is one sample
    const size_t cps = (sample_bytes + cb - 1) / cb;
    const size_t n_chunks = (len / sample_bytes) * cps;
    const size_t first_len = std::min(sample_bytes, cb);
    P.sample_bytes = sample_bytes;
    P.chunks_per_sample = (uint32_t)cps;
    P.ivs = ivs;
    P.n_chunks = (uint32_t)n_chunks;
    FrPlanConfig cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.num_sms = (int)(num_sms ? num_sms : 148);
    cfg.chunk_bytes = cb;
    cfg.fold_tail_mode = fold_mode;                                              // as FASTRACK_OPT_FOLD_TAIL
    const bool may_fold = mode == FR_MODE_DEC || mode == FR_MODE_ENC;
    FrRowPlan rows = fr_plan_rows(cfg, sample_bytes, n_chunks, may_fold);
    if (rows_per_slot) {
        cfg.row_slots_override = (uint32_t)((rows.total_rows + rows_per_slot - 1) / rows_per_slot);
        rows = fr_plan_rows(cfg, sample_bytes, n_chunks, may_fold);
    }
    P.fold_tail = rows.fold_tail;
    P.n_slots = rows.n_slots;
    P.warps_used = rows.warps_used;
    P.rows_full = rows.rows_full;
    P.rows_last = rows.rows_last;
    P.rows_sample = rows.rows_sample;
    P.total_rows = rows.total_rows;
    if ((uint64_t)rows.grid * rows.warps_used < rows.n_slots || rows.warps_used > 32 || rows.grid > (uint32_t)cfg.num_sms) return -2;
    P.lenh_full = length_term(S, first_len, aad_mod);
    P.lenh_last = length_term(S, sample_bytes - (cps - 1) * cb, aad_mod);
    P.in = in;
    P.out = out;
    P.pad = pad;
    P.mask = (uint4*)mask;
    std::vector<uint4> acc(n_chunks, uint4{0, 0, 0, 0});
    int rc;
    switch (mode) {
        case FR_MODE_DEC: rc = P.fold_tail ? run_pass<FR_MODE_DEC, true>(S, acc) : run_pass<FR_MODE_DEC>(S, acc); break;
        case FR_MODE_ENC: rc = P.fold_tail ? run_pass<FR_MODE_ENC, true>(S, acc) : run_pass<FR_MODE_ENC>(S, acc); break;
        case FR_MODE_CTR: return run_pass<FR_MODE_CTR>(S, acc);
        case FR_MODE_VERIFY: rc = run_pass<FR_MODE_VERIFY>(S, acc); break;
        case FR_MODE_PADGEN: return run_pass<FR_MODE_PADGEN>(S, acc);
        case FR_MODE_PADDEC: rc = run_pass<FR_MODE_PADDEC>(S, acc); break;
        default: return -1;
    }
    if (rc) return rc;
    for (uint32_t kk = 0; kk < n_chunks; kk++) {                            // the finishing warp's part
        const uint4 tag = fr_xor4(acc[kk], ((kk + 1) % P.chunks_per_sample == 0) ? P.lenh_last : P.lenh_full);
        if (mode == FR_MODE_ENC) memcpy(tags_out + 16 * kk, &tag, 16);
        else ok[kk] = memcmp(&tag, tags_in + 16 * kk, 16) == 0;
    }
    return 0;
}

// The packed-row kernels (small chunks): the lane function from the header, and the kernel body's segmented scan,
// carry and finishing step written out over an array of 32 lane values, shuffle by shuffle.
template <int MODE, bool WHOLE>
static void run_packed(Setup& S, const uint8_t* tags_in, uint8_t* tags_out, uint32_t* ok)
{
    FrParams& P = S.P;
    const FrPackGeom g = fr_pack_geom(P);
    for (uint32_t item = 0; item < P.n_items; item++) {
        const uint32_t kk0 = fr_pack_item_begin(P, item), kk1 = fr_pack_item_begin(P, item + 1u);
        if (kk1 <= kk0 || kk1 > P.n_chunks) abort();                       // no empty item, nothing past the end
        const uint32_t slot_end = fr_pack_slot_begin(P, g, kk1);
        uint4 carry = {0, 0, 0, 0};
        for (uint32_t base = fr_pack_slot_begin(P, g, kk0); base < slot_end; base += 32u) {
            uint4 z[32];
            FrSlot si[32];
            bool valid[32];
            for (uint32_t lane = 0; lane < 32; lane++) {
                const FrLane L = fr_make_lane(lane);
                valid[lane] = base + lane < slot_end;
                si[lane] = FrSlot{0u, lane, 0xFFFFFFFFu};
                z[lane] = uint4{0, 0, 0, 0};
                if (valid[lane]) z[lane] = fr_packed_slot_lane<MODE, false, WHOLE>(P, S.sm.data(), L, g, base + lane, si[lane]);
            }
            if (MODE == FR_MODE_CTR) continue;
            if (!WHOLE) {                                   // one lane per chunk: nothing to reduce
            if (si[0].i != 0u) z[0] = fr_xor4(z[0], carry);
            for (uint32_t d = 1; d < 32; d <<= 1) {
                uint4 up[32];
                for (uint32_t lane = 0; lane < 32; lane++) up[lane] = z[lane >= d ? lane - d : lane];   // shfl_up
                for (uint32_t lane = 0; lane < 32; lane++) {
                    const uint32_t first = lane >= si[lane].i ? lane - si[lane].i : 0u;
                    if (lane >= first + d) z[lane] = fr_xor4(z[lane], up[lane]);
                }
            }
            carry = z[31];
            }
            for (uint32_t lane = 0; lane < 32; lane++) {
                if (!(valid[lane] && si[lane].i == si[lane].last)) continue;
                const uint32_t kk = si[lane].kk;
                const uint4 tag = fr_xor4(z[lane], ((kk + 1u) % P.chunks_per_sample == 0u) ? P.lenh_last : P.lenh_full);
                if (MODE == FR_MODE_ENC) memcpy(tags_out + 16 * (size_t)kk, &tag, 16);
                else ok[kk] = memcmp(&tag, tags_in + 16 * (size_t)kk, 16) == 0;
            }
        }
    }
}

// One packed-row pass (mode 0 = decrypt + verify, 1 = encrypt + tag, 2 = counter mode only, 3 = verify only): at most pack_run counters per slot, about pack_chunks chunks per work item.
extern "C" int emu_packed(int mode, const uint8_t* key, const uint8_t* iv_base, size_t cb, const uint8_t* in, size_t len,
                          uint8_t* out, const uint8_t* tags_in, uint8_t* tags_out, uint32_t* ok, uint32_t pack_chunks,
                          uint32_t pack_run, uint32_t first_chunk, uint32_t aad_mod, size_t sample_bytes, const uint8_t* ivs)
{
    if (sample_bytes == 0) sample_bytes = len;
    const uint32_t run_ = pack_run ? pack_run : 1;
    const uint32_t lanes = (uint32_t)(((std::min(sample_bytes, cb) + 15) / 16 + run_) / run_);      // slots per chunk, as fr_pack_geom has it
    Setup S;
    setup(S, key, cb, lanes);
    FrParams& P = S.P;
    auto be32 = [](const uint8_t* p) { return ((uint32_t)p[0] << 24) | ((uint32_t)p[1] << 16) | ((uint32_t)p[2] << 8) | p[3]; };
    auto le32 = [](const uint8_t* p) { return ((uint32_t)p[3] << 24) | ((uint32_t)p[2] << 16) | ((uint32_t)p[1] << 8) | p[0]; };
    P.iv_w0 = le32(iv_base);
    P.iv_w1 = le32(iv_base + 4);
    P.iv_ctr = be32(iv_base + 8) + first_chunk;
    P.first_chunk = first_chunk;
    P.aad_mod = aad_mod;
    P.len = len;
    P.chunk_bytes = cb;
    if (sample_bytes == 0) sample_bytes = len;
    const size_t cps = (sample_bytes + cb - 1) / cb;
    const size_t n_chunks = (len / sample_bytes) * cps;
    P.sample_bytes = sample_bytes;
    P.chunks_per_sample = (uint32_t)cps;
    P.ivs = ivs;
    P.n_chunks = (uint32_t)n_chunks;
    P.pack_run = pack_run ? pack_run : 1;
    P.n_items = (uint32_t)((n_chunks + (pack_chunks ? pack_chunks : 1) - 1) / (pack_chunks ? pack_chunks : 1));   // items of about pack_chunks chunks
    P.lenh_full = length_term(S, std::min(sample_bytes, cb), aad_mod);
    P.lenh_last = length_term(S, sample_bytes - (cps - 1) * cb, aad_mod);
    P.in = in;
    P.out = out;
    // the one-lane-per-chunk variant wherever it applies (launch_pass uses it for a subset of these shapes), except
    // when first_chunk is odd, so that the general closing product is exercised on whole-chunk runs too
    const bool whole = P.pack_run > (std::min(sample_bytes, cb) + 15) / 16 && !(first_chunk & 1u);
    if (mode == FR_MODE_DEC) whole ? run_packed<FR_MODE_DEC, true>(S, tags_in, tags_out, ok) : run_packed<FR_MODE_DEC, false>(S, tags_in, tags_out, ok);
    else if (mode == FR_MODE_ENC) whole ? run_packed<FR_MODE_ENC, true>(S, tags_in, tags_out, ok) : run_packed<FR_MODE_ENC, false>(S, tags_in, tags_out, ok);
    else if (mode == FR_MODE_CTR) whole ? run_packed<FR_MODE_CTR, true>(S, tags_in, tags_out, ok) : run_packed<FR_MODE_CTR, false>(S, tags_in, tags_out, ok);
    else if (mode == FR_MODE_VERIFY) whole ? run_packed<FR_MODE_VERIFY, true>(S, tags_in, tags_out, ok) : run_packed<FR_MODE_VERIFY, false>(S, tags_in, tags_out, ok);
    else return -1;
    return 0;
}

extern "C" void emu_gf128_mul_device(const uint8_t* a, const uint8_t* b, uint8_t* o)
{
    uint4 x, y;
    memcpy(&x, a, 16);
    memcpy(&y, b, 16);
    const uint4 z = fr_gf128_mul(x, y);
    memcpy(o, &z, 16);
}

extern "C" void emu_gf128_mul_keysetup(const uint8_t* a, const uint8_t* b, uint8_t* o)
{
    gf_store(gf_mul(gf_load(a), gf_load(b)), o);
}

// Round keys (240 bytes, as the little-endian words the kernel receives) and H from the host-side key set-up.
extern "C" void emu_keysetup(const uint8_t* key, uint8_t* round_keys, uint8_t* h)
{
    Setup S;
    setup(S, key, 16);
    memcpy(round_keys, S.P.rk, 240);
    memcpy(h, S.h, 16);
}

#ifdef EMU_SANITIZER_MAIN
// Stand-alone driver for a build with -fsanitize=address,undefined (the GPU-side memory checker is not available
// to this project, so the index arithmetic of the per-lane code is checked here instead): every buffer is a heap
// block of exactly the size the C ABI asks the caller for, so a lane that reads or writes one byte outside the
// payload, the tag / verdict / mask arrays, the power table or the shared-memory image stops the program.
// Results are not compared here -- the Python tests do that -- only memory safety and the return code.
#include <stdio.h>

static uint32_t lcg(uint32_t& s) { return s = s * 1664525u + 1013904223u; }

static size_t g_short_out = 0;      // self-test: allocate the output this many bytes short, which must be caught

static int run_case(size_t cb, size_t len, uint32_t seg, uint32_t first, uint32_t aad, size_t sample_bytes)
{
    const size_t sb = sample_bytes ? sample_bytes : len;
    const size_t n_samples = len / sb, cps = (sb + cb - 1) / cb, K = n_samples * cps;
    uint32_t s = (uint32_t)(cb * 31 + len * 7 + seg + first + aad);
    uint8_t key[32], iv[12];
    for (auto& b : key) b = (uint8_t)(lcg(s) >> 24);
    for (auto& b : iv) b = (uint8_t)(lcg(s) >> 24);
    int bad = 0;
    for (int mode = 0; mode < 6; mode++) {
        uint8_t* in = new uint8_t[len];
        uint8_t* out = new uint8_t[len - g_short_out];
        uint8_t* pad = new uint8_t[len];
        uint8_t* mask = new uint8_t[16 * K];
        uint8_t* tin = new uint8_t[16 * K];
        uint8_t* tout = new uint8_t[16 * K];
        uint32_t* ok = new uint32_t[K];
        uint8_t* ivs = sample_bytes ? new uint8_t[12 * n_samples] : nullptr;
        for (size_t i = 0; i < len; i++) { in[i] = (uint8_t)(lcg(s) >> 24); pad[i] = (uint8_t)(lcg(s) >> 16); }
        for (size_t i = 0; i < 16 * K; i++) { mask[i] = (uint8_t)(lcg(s) >> 24); tin[i] = (uint8_t)(lcg(s) >> 24); tout[i] = 0; }
        for (size_t i = 0; i < K; i++) ok[i] = 9;
        if (ivs) for (size_t i = 0; i < 12 * n_samples; i++) ivs[i] = (uint8_t)(lcg(s) >> 24);
        bad |= emu_pass(mode, key, iv, cb, in, len, out, pad, mask, tin, tout, ok, seg, 2 + seg % 3, first, aad, sample_bytes, ivs, 2);   // tails folded wherever a chunk has one
        bad |= emu_pass(mode, key, iv, cb, in, len, out, pad, mask, tin, tout, ok, seg, 2 + seg % 3, first, aad, sample_bytes, ivs, 1);   // and never
        bad |= emu_pass(mode, key, iv, cb, in, len, out, pad, mask, tin, tout, ok, 0, 148, first, aad, sample_bytes, ivs, 0);
        if (mode <= FR_MODE_VERIFY)                     // the packed-row form of the same pass, seg doubling as group size and run length
            for (uint32_t run : {1u, seg + 1u, 40u})
                bad |= emu_packed(mode, key, iv, cb, in, len, out, tin, tout, ok, seg * 3 - 2, run, first, aad, sample_bytes, ivs);
        delete[] in; delete[] out; delete[] pad; delete[] mask; delete[] tin; delete[] tout; delete[] ok; delete[] ivs;
    }
    return bad;
}

int main(int argc, char** argv)
{
    if (argc > 1 && !strcmp(argv[1], "short-output")) {     // must die inside the sanitizer: proves the check has teeth
        g_short_out = 1;
        return run_case(512, 1041, 2, 0, 0, 0);
    }
    int bad = 0, cases = 0;
    const size_t cbs[] = {16, 32, 496, 512, 528, 1024, 4112};
    for (size_t cb : cbs) {
        const size_t lens[] = {1, 15, 16, 17, 31, 33, cb - 1, cb, cb + 1, 2 * cb, 3 * cb + 5, 7 * cb + cb / 2 + 3};
        for (size_t len : lens) {
            if (len == 0 || len > 40000) continue;
            for (uint32_t seg : {1u, 2u, 8u}) {
                bad |= run_case(cb, len, seg, 0, 0, 0);
                cases++;
            }
            bad |= run_case(cb, len, 4, 0xfffffffeu, 3, 0);                 // wrapping chunk index, framing on
            cases++;
        }
        for (size_t sb : {(size_t)16, (size_t)48, cb, cb + 16, 3 * cb - 16}) {  // batches of samples
            if (sb * 5 > 40000) continue;
            bad |= run_case(cb, sb * 5, 2, 0, 0, sb);
            bad |= run_case(cb, sb * 5, 8, 0, 16, sb);
            cases += 2;
        }
    }
    printf("%d cases, status %d\n", cases, bad);
    return bad ? 1 : 0;
}
#endif
