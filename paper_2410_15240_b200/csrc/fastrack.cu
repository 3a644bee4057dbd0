// fastrack.cu -- kernels, context and C ABI of the B200 (sm_100a) Fastrack channel library.
// The entry points are documented in include/fastrack.h; the per-lane device code is in
// fastrack_device.cuh.  There is no CPU data path here: host code only derives key material
// (round keys, H, the byte tables of H^32) once per context and launches kernels.
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <new>

#include "../../include/fastrack.h"
// Waits (whole warp) until the bulk copy of the H-power byte tables has landed in shared memory; defined below.
__device__ __forceinline__ void fr_await_tables(const char* sm, const uint4* gh_tab, uint32_t* timeouts);
#define FR_AWAIT_TABLES(sm, P) fr_await_tables((sm), (P).gh_tab, (P).timeouts)
#include "fastrack_device.cuh"
#include "fastrack_keysetup.h"
#include "fastrack_plan.h"

using namespace fr_host;

// ------------------------------------------------------------------------------------ kernels ----

// (Te0 reaches the kernels as a parameter, FrParams::te0c.  Tried instead: the 256 words as immediates in the code of
// the warp that stores them -- slower, 2.0 against 1.4 us for the fill, because then every warp runs code of its own
// and the instruction fetch becomes the cost; a __constant__ array -- a cold miss per isolated launch.)

// Fills shared memory at the start of a kernel, up to but not including the barrier that publishes it.
//   AES rows: every thread replicates eight entries of Te0 (and its byte rotations) across the 32 banks; the
//     entries come from the kernel parameters (constant bank) with a warp-uniform index.
//   H-power byte tables (64 KiB, per context): two bulk asynchronous copies, global -> shared, issued by thread 0
//     before anything else and signalled on an mbarrier.  Nobody waits for them here: every lane starts with a
//     cipher block, which needs the AES rows only, and waits in front of its first table multiply
//     (fr_await_tables), by which time the 64 KiB have long arrived.
//     (Passes that do not authenticate have no use for them and start no copy: a CTA must not exit with a copy
//     into its shared memory still in flight, and only the table multiply waits for it.)
template <uint32_t NTHREADS, bool WITH_H_TABLES>
__device__ __forceinline__ void fr_fill_smem(char* sm, const uint4* __restrict__ gh_tab, const FrParams& P)
{
    const uint32_t tid = threadIdx.x;
    if (WITH_H_TABLES && tid == 0) {
        const uint32_t mbar = (uint32_t)__cvta_generic_to_shared(sm + FR_SM_MBAR);
        const uint32_t dst = (uint32_t)__cvta_generic_to_shared(sm + FR_SM_GH);
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(mbar) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(mbar), "r"(65536u) : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(dst), "l"(gh_tab), "r"(32768u), "r"(mbar) : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(dst + 32768u), "l"((const char*)gh_tab + 32768), "r"(32768u), "r"(mbar) : "memory");
    }
    constexpr uint32_t N_AES = 256u * 4u * 8u / NTHREADS;     // 256 rows x 2 arrays x 2 tables x 8 uint4 (32 words)
    static_assert(N_AES * NTHREADS == 8192u, "thread count must divide the tables");
#pragma unroll
    for (uint32_t n = 0; n < N_AES; n++) {
        const uint32_t i = tid + n * NTHREADS, q = i & 7u, t = (i >> 3) & 3u, v = i >> 5;
        const uint32_t e = P.te0c[v];
        const uint32_t w = __funnelshift_l(e, e, 8u * t);                 // Te1..Te3 are Te0 rotated left by 1..3 bytes
        const uint32_t off = ((t >> 1) ? FR_SM_T23 : FR_SM_T01) + v * 256u + (t & 1u) * 128u + q * 16u;
        *(uint4*)(sm + off) = make_uint4(w, w, w, w);
    }
    if (tid < 33u * 8u) ((uint32_t*)(sm + FR_SM_COMB))[tid] = 0u;        // the combine records start at zero
}

// Every thread calls this once, in front of its first table multiply: it polls the copy's mbarrier a bounded
// number of times (each attempt gives up by itself after a while; in practice the first one succeeds, the copy
// having had a whole cipher block's time to land).  Should the copy never arrive, the thread counts the event in
// *timeouts and goes on: the tags it computes from an incomplete table do not match, so every chunk it touches
// is rejected (or, when encrypting, will be rejected by the receiver) -- wrong towards refusal, never acceptance.
__device__ __forceinline__ void fr_await_tables(const char* sm, const uint4* gh_tab, uint32_t* timeouts)
{
    (void)gh_tab;
    const uint32_t mbar = (uint32_t)__cvta_generic_to_shared(sm + FR_SM_MBAR);
    uint32_t done = 0;
    for (uint32_t attempt = 0; attempt < 4096u && !done; attempt++)
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], 0;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(done) : "r"(mbar) : "memory");
    if (!done) atomicAdd(timeouts, 1u);
}

template <int MODE, bool ABS, bool FOLD>
__device__ __forceinline__ void fr_crypt_body(const FrParams& P, char* sm, FrLane L)
{
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    if (warp >= P.warps_used) return;
    const uint32_t cta_first = blockIdx.x * P.warps_used, slot = cta_first + warp;
    if (slot >= P.n_slots) return;
    uint32_t cta_last = cta_first + P.warps_used - 1u;
    if (cta_last >= P.n_slots) cta_last = P.n_slots - 1u;
    uint32_t* const comb = (uint32_t*)(sm + FR_SM_COMB);

    uint64_t g = fr_slot_begin(P, slot);
    const uint64_t end = fr_slot_begin(P, slot + 1u);
    bool await_tables = true;                            // the H tables may still be on their way into shared memory (per thread)
    uint4* const pre_results = (uint4*)(sm + FR_SM_PRE) + warp * FR_PRE_CHUNKS;
    uint32_t pre_first = 0, pre_count = 0;               // FOLD: the chunks whose prework results the warp holds
    while (g < end) {                                    // one segment per chunk that the warp's range touches
        const FrRowPos pos = fr_locate_row(P, g);
        uint32_t take = pos.rows_k - pos.r;
        if (take > end - g) take = (uint32_t)(end - g);
        if constexpr (FOLD) {
            // Folded tails: the warp in whose range a chunk begins also makes that chunk's tag mask and works on the
            // one or two blocks behind its last row, for up to ten chunks of its range in one pass (see fr_prework_lane).
            if (pos.r == 0u && pos.kk - pre_first >= pre_count) {
                bool j0_lane;
                uint4 t = fr_prework_lane<MODE, ABS>(P, sm, L, lane, pos.kk, end, j0_lane);
                t.x ^= __shfl_down_sync(0xFFFFFFFFu, t.x, 1) ^ __shfl_down_sync(0xFFFFFFFFu, t.x, 2);
                t.y ^= __shfl_down_sync(0xFFFFFFFFu, t.y, 1) ^ __shfl_down_sync(0xFFFFFFFFu, t.y, 2);
                t.z ^= __shfl_down_sync(0xFFFFFFFFu, t.z, 1) ^ __shfl_down_sync(0xFFFFFFFFu, t.z, 2);
                t.w ^= __shfl_down_sync(0xFFFFFFFFu, t.w, 1) ^ __shfl_down_sync(0xFFFFFFFFu, t.w, 2);
                if (j0_lane) pre_results[lane / 3u] = t;
                pre_first = pos.kk;
                pre_count = __popc(__ballot_sync(0xFFFFFFFFu, j0_lane));
                __syncwarp();
            }
        }
        uint4 z = fr_process_segment_lane<MODE, ABS, FOLD>(P, sm, L, lane, pos.kk, pos.r, pos.r + take, await_tables);
        if constexpr (FOLD) {
            if (pos.r == 0u && lane == 1u) z = fr_xor4(z, pre_results[pos.kk - pre_first]);
        }
        const uint64_t g0 = g - pos.r;                   // the chunk's first row in the row space
        g += take;
        if (MODE != FR_MODE_CTR && MODE != FR_MODE_PADGEN) {                // the other passes authenticate
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            z.x ^= __shfl_xor_sync(0xFFFFFFFFu, z.x, off);
            z.y ^= __shfl_xor_sync(0xFFFFFFFFu, z.y, off);
            z.z ^= __shfl_xor_sync(0xFFFFFFFFu, z.z, off);
            z.w ^= __shfl_xor_sync(0xFFFFFFFFu, z.w, off);
        }
        // A chunk covered by several warps: each XORs its part into a record and takes a ticket; whoever takes the
        // last ticket carries the sum on (XOR commutes, so the result does not depend on the order of arrival).
        // First among the warps of this CTA, in shared memory; then among CTAs, in the global record of the first
        // CTA that works on the chunk.  Records are left zeroed.  No warp ever waits for another.
        bool finisher = true;
        if (take != pos.rows_k) {
            const FrShare sh = fr_chunk_share(P, g0, pos.rows_k, cta_first, cta_last);
            if (sh.n_in_cta > 1u) {
                uint32_t* rec = comb + 8u * sh.rec;
                uint32_t ticket = 0;
                if (lane == 0) {
                    atomicXor(rec + 0, z.x); atomicXor(rec + 1, z.y); atomicXor(rec + 2, z.z); atomicXor(rec + 3, z.w);
                    __threadfence_block();
                    ticket = atomicAdd(rec + 4, 1u);
                }
                ticket = __shfl_sync(0xFFFFFFFFu, ticket, 0);
                finisher = (ticket == sh.n_in_cta - 1u);
                if (finisher && lane == 0) {
                    __threadfence_block();
                    z.x = atomicExch(rec + 0, 0u); z.y = atomicExch(rec + 1, 0u);
                    z.z = atomicExch(rec + 2, 0u); z.w = atomicExch(rec + 3, 0u);
                }
            }
            if (finisher && sh.n_ctas > 1u) {
                uint32_t* rec = P.acc + 8u * sh.first_cta;
                uint32_t ticket = 0;
                if (lane == 0) {
                    atomicXor(rec + 0, z.x); atomicXor(rec + 1, z.y); atomicXor(rec + 2, z.z); atomicXor(rec + 3, z.w);
                    // The ticket is one read-modify-write that both publishes the four XORs above (release) and makes
                    // the earlier arrivals' XORs visible to the reads below (acquire); the tickets of a record form
                    // one chain of read-modify-writes, so the last one synchronises with all.  (A fence on either
                    // side of a relaxed ticket does the same and costs 0.4 us more per launch.)
                    asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;" : "=r"(ticket) : "l"(rec + 4) : "memory");
                }
                ticket = __shfl_sync(0xFFFFFFFFu, ticket, 0);
                finisher = (ticket == sh.n_ctas - 1u);
                if (finisher && lane == 0) {              // read the sum and leave the record zeroed
                    z.x = atomicExch(rec + 0, 0u); z.y = atomicExch(rec + 1, 0u);
                    z.z = atomicExch(rec + 2, 0u); z.w = atomicExch(rec + 3, 0u);
                    atomicExch(rec + 4, 0u);
                }
            }
        }
        if (finisher && lane == 0) {
            const uint4 lenh = ((pos.kk + 1u) % P.chunks_per_sample == 0u) ? P.lenh_last : P.lenh_full;
            const uint4 tag = fr_xor4(z, lenh);           // z already holds GHASH of the data xor E_K(J0)
            if (MODE == FR_MODE_ENC) {
                P.tags_out[pos.kk] = tag;
            } else {
                const uint4 t = P.tags_in[pos.kk];
                const uint32_t diff = (tag.x ^ t.x) | (tag.y ^ t.y) | (tag.z ^ t.z) | (tag.w ^ t.w);
                P.ok[pos.kk] = diff == 0u ? 1u : 0u;
            }
        }
        }
    }
}

// Fused pass: keystream, XOR, per-segment GHASH partial, per-chunk tag.  Every warp that takes work walks one
// contiguous range of the launch's rows (see fr_slot_begin in the device header).
template <int MODE, bool FOLD = false>
__global__ void __launch_bounds__(FR_THREADS, 1) fr_crypt_kernel(const __grid_constant__ FrParams P)
{
    extern __shared__ __align__(256) char sm[];
    FR_STAMP_GT(0); FR_STAMP_SET(7);
    fr_fill_smem<FR_THREADS, MODE != FR_MODE_CTR && MODE != FR_MODE_PADGEN>(sm, P.gh_tab, P);
    FR_STAMP_SET(1);
    // Programmatic dependent launch: the table build above touches only per-context constants, so it may run
    // while the previous kernel in the stream is still finishing; everything below waits until that kernel has
    // completed and its writes are visible (a no-op when the launch carries no such dependency).  Kernels queued
    // behind this one may be scheduled as soon as SMs free up; they wait at the same point.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;");
    __syncthreads();
    FR_STAMP_SET(2);
    // Lane constants are made to depend on a value the compiler cannot see through and that is produced
    // after the barrier, so that no table load can be scheduled above the barrier.
    uint32_t after_barrier;
    asm volatile("mov.u32 %0, 0;" : "=r"(after_barrier)::"memory");
    FrLane L = fr_make_lane(threadIdx.x & 31u);
    L.lane4 |= after_barrier;
    L.qe |= after_barrier;
    L.qo |= after_barrier;
    if ((uint32_t)__cvta_generic_to_shared(sm) == FR_SMEM_ABS_BASE && !P.generic_smem) fr_crypt_body<MODE, true, FOLD>(P, sm, L);
    else fr_crypt_body<MODE, false, FOLD>(P, sm, L);
    FR_STAMP_MAX(5); FR_STAMP_GTMAX(6);
}

// Packed rows (many short chains, see the device header): a warp takes a contiguous range of whole chunks and walks
// their slots 32 at a time; the per-chunk XOR of the lane terms is a segmented inclusive scan over the row (a lane adds
// the lane d below it only if that lane belongs to the same chunk), a chunk that continues into the next row hands
// its running sum to that row's lane 0, and the lane holding a chunk's last slot finishes the tag.  No chunk is
// shared between warps.  The shared-memory GHASH tables hold H here, not H^32.
template <int MODE, bool ABS, bool WHOLE>
__device__ __forceinline__ void fr_packed_body(const FrParams& P, const char* sm, FrLane L)
{
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    const uint32_t total_warps = gridDim.x * (blockDim.x >> 5);
    const FrPackGeom g = fr_pack_geom(P);

    for (uint32_t item = warp * gridDim.x + blockIdx.x; item < P.n_items; item += total_warps) {
        const uint32_t kk0 = fr_pack_item_begin(P, item), kk1 = fr_pack_item_begin(P, item + 1u);
        const uint32_t slot_end = fr_pack_slot_begin(P, g, kk1);
        uint4 carry = make_uint4(0, 0, 0, 0);
        for (uint32_t base = fr_pack_slot_begin(P, g, kk0); base < slot_end; base += 32u) {
            const uint32_t slot = base + lane;
            const bool valid = slot < slot_end;               // only the item's last row has idle lanes, at its top
            FrSlot si = {0u, lane, 0xFFFFFFFFu};
            uint4 z = make_uint4(0, 0, 0, 0);
            if (valid) z = fr_packed_slot_lane<MODE, ABS, WHOLE>(P, sm, L, g, slot, si);
            if (MODE == FR_MODE_CTR) continue;                   // nothing to authenticate
            if (!WHOLE) {                                        // (one lane per chunk: z is the chunk's sum already)
            if (lane == 0u && si.i != 0u) z = fr_xor4(z, carry);
            const uint32_t first = lane >= si.i ? lane - si.i : 0u;      // lowest lane of this row in the same chunk
#pragma unroll
            for (uint32_t d = 1; d < 32u; d <<= 1) {
                const uint32_t tx = __shfl_up_sync(0xFFFFFFFFu, z.x, d), ty = __shfl_up_sync(0xFFFFFFFFu, z.y, d);
                const uint32_t tz = __shfl_up_sync(0xFFFFFFFFu, z.z, d), tw = __shfl_up_sync(0xFFFFFFFFu, z.w, d);
                if (lane >= first + d) { z.x ^= tx; z.y ^= ty; z.z ^= tz; z.w ^= tw; }
            }
            carry.x = __shfl_sync(0xFFFFFFFFu, z.x, 31); carry.y = __shfl_sync(0xFFFFFFFFu, z.y, 31);
            carry.z = __shfl_sync(0xFFFFFFFFu, z.z, 31); carry.w = __shfl_sync(0xFFFFFFFFu, z.w, 31);
            }
            if (valid && si.i == si.last) {
                const uint4 lenh = ((si.kk + 1u) % P.chunks_per_sample == 0u) ? P.lenh_last : P.lenh_full;
                const uint4 tag = fr_xor4(z, lenh);
                if (MODE == FR_MODE_ENC) {
                    P.tags_out[si.kk] = tag;
                } else {
                    const uint4 t = P.tags_in[si.kk];
                    const uint32_t diff = (tag.x ^ t.x) | (tag.y ^ t.y) | (tag.z ^ t.z) | (tag.w ^ t.w);
                    P.ok[si.kk] = diff == 0u ? 1u : 0u;
                }
            }
        }
    }
}

template <int MODE, bool WHOLE>
__global__ void __launch_bounds__(FR_THREADS, 1) fr_packed_kernel(const __grid_constant__ FrParams P)
{
    extern __shared__ __align__(256) char sm[];
    fr_fill_smem<FR_THREADS, MODE != FR_MODE_CTR>(sm, P.gh_tab, P);
    asm volatile("griddepcontrol.wait;" ::: "memory");           // as in fr_crypt_kernel
    asm volatile("griddepcontrol.launch_dependents;");
    __syncthreads();
    if (MODE != FR_MODE_CTR) fr_await_tables(sm, P.gh_tab, P.timeouts);      // (a packed row may start with a table step: wait here)
    uint32_t after_barrier;
    asm volatile("mov.u32 %0, 0;" : "=r"(after_barrier)::"memory");
    FrLane L = fr_make_lane(threadIdx.x & 31u);
    L.lane4 |= after_barrier;          // no table load above the barrier, as in fr_crypt_kernel: every lookup address here
                                       // derives from lane4, from loaded data, or (the AAD block) is tied to lane4 by the lane code
    if ((uint32_t)__cvta_generic_to_shared(sm) == FR_SMEM_ABS_BASE && !P.generic_smem) fr_packed_body<MODE, true, WHOLE>(P, sm, L);
    else fr_packed_body<MODE, false, WHOLE>(P, sm, L);
}

// pow[i] = pow[i - half] * pow[half] for i in (half, min(2*half, n - 1)]: one doubling pass of the table
// of powers (pow[half] itself was the last entry of the previous pass; pow[0] = 1 and pow[1] = H are given).
__global__ void fr_pow_double_kernel(uint4* pow, uint32_t half, uint32_t n)
{
    const uint32_t i = half + 1u + blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t last = (2u * half < n - 1u) ? 2u * half : n - 1u;
    if (i <= last) pow[i] = fr_gf128_mul(pow[i - half], pow[half]);
}

// Byte tables of H^e, in the layout of the shared-memory image (entry for byte position p and byte value v at
// uint4 index v * 16 + p), from the table of powers: one block per byte position; eight threads multiply the unit
// bytes 1 << b at that position by H^e, then thread v XORs the products its bits select.  The packed-row kernels
// need the tables of H^lanes, which depends on the launch geometry; this runs only when that changes.
__global__ void __launch_bounds__(256) fr_byte_tables_kernel(const uint4* __restrict__ pow, uint32_t e, uint4* __restrict__ out)
{
    __shared__ uint4 basis[8];
    const uint32_t p = blockIdx.x, v = threadIdx.x;
    if (v < 8u) {
        uint32_t w[4] = {0, 0, 0, 0};
        w[p >> 2] = (1u << v) << (8u * (p & 3u));
        basis[v] = fr_gf128_mul(make_uint4(w[0], w[1], w[2], w[3]), pow[e]);
    }
    __syncthreads();
    uint4 acc = make_uint4(0, 0, 0, 0);
#pragma unroll
    for (uint32_t b = 0; b < 8u; b++)
        if (v & (1u << b)) acc = fr_xor4(acc, basis[b]);
    out[v * 16u + p] = acc;
}

// Comparator, not the fast path: the authentication kernel in the shape the paper starts from (Section 4.2:
// the m block multiplications of a chain are evaluated one after the other; parallel only across chains).
// One THREAD walks one chunk's whole chain, Y <- (Y xor X_i) * H, with the byte tables of H itself in shared
// memory, then the length block, then E_K(J0) and the tag compare.  Time grows with the chain length, so it
// falls as 1/K when a buffer is cut into K chunks -- the effect the paper's multi-chaining exploits.
__global__ void __launch_bounds__(32, 1) fr_verify_sequential_kernel(const __grid_constant__ FrParams P)
{
    extern __shared__ __align__(256) char sm[];
    fr_build_smem_any(sm, threadIdx.x, blockDim.x, P.te0, P.gh_tab);      // gh_tab holds the tables of H^1 here
    __syncthreads();
    const uint32_t lane = threadIdx.x;
    const FrLane L = fr_make_lane(lane);
    const uint32_t kk = blockIdx.x * 32u + lane;
    if (kk >= P.n_chunks) return;
    const FrChunk ck = fr_chunk_info(P, kk);
    const uint64_t len_k = ck.len;
    const uint32_t nblk = (uint32_t)((len_k + 15) >> 4);
    const uint8_t* in = P.in + ck.off;
    uint4 y = make_uint4(0, 0, 0, 0);
    if (P.aad_mod) y = fr_ghash_tabmul<false>(sm, L, make_uint4(ck.serial % P.aad_mod, 0, 0, 0));
    uint32_t j = 0;
    for (; j + 8 <= nblk && ((uint64_t)(j + 8) << 4) <= len_k; j += 8) {      // eight loads in flight per thread
        uint4 x[8];
#pragma unroll
        for (int u = 0; u < 8; u++) x[u] = *(const uint4*)(in + ((uint64_t)(j + u) << 4));
#pragma unroll
        for (int u = 0; u < 8; u++) y = fr_ghash_tabmul<false>(sm, L, fr_xor4(y, x[u]));
    }
    for (; j < nblk; j++) {
        const uint64_t boff = (uint64_t)j << 4;
        const bool full = len_k - boff >= 16;
        const uint4 x = full ? *(const uint4*)(in + boff) : fr_load_partial(in + boff, (uint32_t)(len_k - boff));
        y = fr_ghash_tabmul<false>(sm, L, fr_xor4(y, x));
    }
    const uint64_t bits = len_k << 3;
    const uint4 lenblk = make_uint4(0, P.aad_mod ? fr_bswap(8u) : 0u, fr_bswap((uint32_t)(bits >> 32)), fr_bswap((uint32_t)bits));
    y = fr_ghash_tabmul<false>(sm, L, fr_xor4(y, lenblk));
    const FrCtrChunk cc = fr_ctr_chunk<false>(sm, L.lane4, P, ck.iv_w0, ck.iv_w1, fr_bswap(ck.iv_ctr));
    const FrCtrGroup cg = fr_ctr_group<false>(sm, L.lane4, P, cc, 1u);
    const uint4 tag = fr_xor4(y, fr_aes256_ctr_block<false>(sm, L.lane4, P, cc, cg, 1u));
    const uint4 t = P.tags_in[kk];
    P.ok[kk] = ((tag.x ^ t.x) | (tag.y ^ t.y) | (tag.z ^ t.z) | (tag.w ^ t.w)) == 0u ? 1u : 0u;
}

#ifdef FR_STAMPS
// Diagnostic build only: reset the probes (rows-done minimum to all ones, the rest to zero) / copy them out.
extern "C" __attribute__((visibility("default"))) int fastrack_stamps_reset(void)
{
    static unsigned long long init[1024 * 8];
    for (int b = 0; b < 1024; b++)
        for (int i = 0; i < 8; i++) init[b * 8 + i] = (i == 3) ? ~0ull : 0ull;
    return (int)cudaMemcpyToSymbol(fr_stamps, init, sizeof init);
}
extern "C" __attribute__((visibility("default"))) int fastrack_stamps_read(unsigned long long* out)
{
    return (int)cudaMemcpyFromSymbol(out, fr_stamps, sizeof(unsigned long long) * 1024 * 8);
}
extern "C" __attribute__((visibility("default"))) int fastrack_warp_stamps_read(unsigned long long* out)
{
    return (int)cudaMemcpyFromSymbol(out, fr_warp_stamps, sizeof(unsigned long long) * 1024 * 32);
}
#endif

// ------------------------------------------------------------------------------------ context ----

struct fastrack_ctx {
    int device;
    int num_sms;
    size_t chunk_bytes;
    FrPlanConfig plan;            // what the host-side planners need (fastrack_plan.h); num_sms and chunk_bytes repeated
    uint32_t rk[60];
    uint8_t h[16];
    uint32_t* d_te0;
    uint32_t te0_host[256];    // Te0, copied into every launch's parameters
    uint4* d_gh_tab;           // byte tables of H^32
    uint4* d_gh1_tab;          // byte tables of H (packed rows with one lane per chunk, sequential-chain comparator)
    uint4* d_pack_tab[2];      // byte tables of H^lanes for the packed rows, per scratch bank (see launch_pass)
    uint32_t pack_tab_lanes[2];   // which power each currently holds (0: none)
    uint4* d_pow;
    size_t pow_entries;
    uint32_t* d_timeouts;      // one word: how often a kernel's bulk copy of the H tables did not arrive in time (see fr_fill_smem)
    uint32_t* d_scratch;       // combine records of the row kernels: 2 banks x FR_SCRATCH_WINDOWS windows x num_sms records of 8 words
    uint4* d_tags_stage;       // pipelined calls: device copy of the tags, then (second half) the E_K(J0) masks
    size_t tags_stage_chunks;
    cudaStream_t streams[8];
    cudaEvent_t tags_ready, pad_ready;
    int trace_on;                               // stage-level event trace of pipelined calls
    cudaEvent_t trace_ev[3 * FR_MAX_STAGES];    // per stage: before the copy, after the copy, after the kernel
    fastrack_stage_trace trace[FR_MAX_STAGES];
    size_t trace_count;
    int last_cuda_error;
    uint64_t launches;
    uint32_t aad_mod;             // 0 = no AAD, else chains per sample of the serial-number framing
    uint32_t generic_smem;        // FASTRACK_OPT_GENERIC_SMEM: exercise the portable addressing path (tests)
    uint32_t no_overlap_launch;   // FASTRACK_OPT_NO_OVERLAP_LAUNCH: plain stream-ordered launches (experiments)
    uint32_t direct_small_h2d;    // single-stage pipelined transfers read / write the host buffer from the kernel (FASTRACK_OPT_DIRECT_SMALL)
    struct { size_t sample_bytes, n_chunks; FrPackPlan plan; bool valid; } pack_memo[3];   // fr_plan_packed's last answer per kind of pass (callers repeat shapes)
};

#define FR_CUDA(ctx, call)                                              \
    do {                                                                \
        cudaError_t e_ = (call);                                        \
        if (e_ != cudaSuccess) {                                        \
            (ctx)->last_cuda_error = (int)e_;                           \
            (void)cudaGetLastError();                                   \
            return FASTRACK_ERR_CUDA;                                   \
        }                                                               \
    } while (0)

// Zeroing that the compiler may not drop (key-derived data about to be freed).
static void secure_zero(void* p, size_t n)
{
    volatile uint8_t* q = (volatile uint8_t*)p;
    for (size_t i = 0; i < n; i++) q[i] = 0;
}

// The row kernels combine the pieces of a chunk that several CTAs worked on in one 32-byte record per CTA of the
// launch (see fr_crypt_body).  Launches that may be in flight at the same time use different windows of
// num_sms records: window 0 serves the caller's stream, window 1 + i the library's internal stream i (stages of
// the pipelined calls), and fastrack_verify has a bank of its own.  The size does not depend on the data.
#define FR_SCRATCH_WINDOWS 9
static size_t scratch_words(const fastrack_ctx* ctx) { return (size_t)2 * FR_SCRATCH_WINDOWS * (size_t)ctx->num_sms * 8; }

// Every entry point that launches work or touches device memory runs on the context's device only.
static int check_device(fastrack_ctx* ctx)
{
    int dev = -1;
    FR_CUDA(ctx, cudaGetDevice(&dev));
    return dev == ctx->device ? FASTRACK_OK : FASTRACK_ERR_ARG;
}

extern "C" int fastrack_ctx_create(const uint8_t key[32], size_t chunk_bytes, fastrack_ctx** out)
{
    if (out) *out = nullptr;
    if (!key || !out) return FASTRACK_ERR_ARG;
    if (chunk_bytes == 0 || (chunk_bytes & 15) || chunk_bytes > FASTRACK_MAX_CHUNK_BYTES) return FASTRACK_ERR_CHUNK;
    fastrack_ctx* ctx = new (std::nothrow) fastrack_ctx();
    if (!ctx) return FASTRACK_ERR_NOMEM;
    memset(ctx, 0, sizeof *ctx);
    ctx->chunk_bytes = chunk_bytes;
    auto fail = [&](int code) { fastrack_ctx_destroy(ctx); return code; };

    cudaError_t e = cudaGetDevice(&ctx->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&ctx->num_sms, cudaDevAttrMultiProcessorCount, ctx->device);
    if (e != cudaSuccess) { (void)cudaGetLastError(); return fail(FASTRACK_ERR_CUDA); }
    ctx->plan.num_sms = ctx->num_sms;
    ctx->plan.chunk_bytes = chunk_bytes;
    ctx->direct_small_h2d = 1;
    ctx->plan.pack_max_blocks = FR_PACK_MAX_BLOCKS;

    // key material on the host: S-box, Te0, round keys, H, byte tables of H^32
    uint8_t sbox[256];
    uint32_t te0[256];
    make_sbox(sbox);
    for (int v = 0; v < 256; v++) {
        uint8_t s1 = sbox[v], s2 = xtime(s1), s3 = (uint8_t)(s2 ^ s1);
        te0[v] = (uint32_t)s2 | ((uint32_t)s1 << 8) | ((uint32_t)s1 << 16) | ((uint32_t)s3 << 24);
    }
    expand_key(key, sbox, ctx->rk);
    uint8_t zero[16] = {0};
    encrypt_block_host(ctx->rk, te0, sbox, zero, ctx->h);
    memcpy(ctx->te0_host, te0, sizeof te0);

    Gf128 H = gf_load(ctx->h), G = H;
    for (int i = 0; i < 5; i++) G = gf_mul(G, G);           // H^32
    uint8_t* tab = (uint8_t*)malloc(2 * 65536);             // tables of H^32, then of H
    if (!tab) return fail(FASTRACK_ERR_NOMEM);
    for (int which = 0; which < 2; which++) {
        const Gf128 mult = which == 0 ? G : H;
        for (int p = 0; p < 16; p++) {
            Gf128 basis[8];
            for (int b = 0; b < 8; b++) {
                uint8_t blk[16] = {0};
                blk[p] = (uint8_t)(1u << b);
                basis[b] = gf_mul(gf_load(blk), mult);
            }
            for (int v = 0; v < 256; v++) {
                Gf128 acc = {0, 0};
                for (int b = 0; b < 8; b++)
                    if (v & (1 << b)) { acc.hi ^= basis[b].hi; acc.lo ^= basis[b].lo; }
                gf_store(acc, tab + (size_t)which * 65536 + (size_t)v * 256 + (size_t)p * 16);
            }
        }
    }

    ctx->pow_entries = chunk_bytes / 16 + 64 + 2;
    do {
        if ((e = cudaMalloc(&ctx->d_te0, sizeof te0)) != cudaSuccess) break;
        if ((e = cudaMalloc(&ctx->d_gh_tab, 65536)) != cudaSuccess) break;
        if ((e = cudaMalloc(&ctx->d_gh1_tab, 65536)) != cudaSuccess) break;
        if ((e = cudaMalloc(&ctx->d_pack_tab[0], 65536)) != cudaSuccess) break;
        if ((e = cudaMalloc(&ctx->d_pack_tab[1], 65536)) != cudaSuccess) break;
        if ((e = cudaMalloc(&ctx->d_pow, ctx->pow_entries * 16)) != cudaSuccess) break;
        if ((e = cudaMalloc(&ctx->d_scratch, scratch_words(ctx) * sizeof(uint32_t))) != cudaSuccess) break;
        if ((e = cudaMemset(ctx->d_scratch, 0, scratch_words(ctx) * sizeof(uint32_t))) != cudaSuccess) break;
        if ((e = cudaMemcpy(ctx->d_te0, te0, sizeof te0, cudaMemcpyHostToDevice)) != cudaSuccess) break;
        if ((e = cudaMalloc(&ctx->d_timeouts, 256)) != cudaSuccess) break;
        if ((e = cudaMemset(ctx->d_timeouts, 0, 256)) != cudaSuccess) break;
        if ((e = cudaMemcpy(ctx->d_gh_tab, tab, 65536, cudaMemcpyHostToDevice)) != cudaSuccess) break;
        if ((e = cudaMemcpy(ctx->d_gh1_tab, tab + 65536, 65536, cudaMemcpyHostToDevice)) != cudaSuccess) break;
        uint8_t seed[32] = {0};
        seed[0] = 0x80;                                     // H^0 = the field's one
        memcpy(seed + 16, ctx->h, 16);                      // H^1
        if ((e = cudaMemcpy(ctx->d_pow, seed, 32, cudaMemcpyHostToDevice)) != cudaSuccess) break;
        for (size_t half = 1; half + 1 < ctx->pow_entries; half *= 2) {
            size_t last = 2 * half < ctx->pow_entries - 1 ? 2 * half : ctx->pow_entries - 1;
            size_t todo = last - half;
            fr_pow_double_kernel<<<(unsigned)((todo + 255) / 256), 256>>>(ctx->d_pow, (uint32_t)half, (uint32_t)ctx->pow_entries);
        }
        if ((e = cudaGetLastError()) != cudaSuccess) break;
        if ((e = cudaFuncSetAttribute(fr_crypt_kernel<FR_MODE_DEC>, cudaFuncAttributeMaxDynamicSharedMemorySize, FR_SMEM_LAUNCH_BYTES)) != cudaSuccess) break;
        if ((e = cudaFuncSetAttribute(fr_crypt_kernel<FR_MODE_ENC>, cudaFuncAttributeMaxDynamicSharedMemorySize, FR_SMEM_LAUNCH_BYTES)) != cudaSuccess) break;
        if ((e = cudaFuncSetAttribute(fr_crypt_kernel<FR_MODE_DEC, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, FR_SMEM_LAUNCH_BYTES)) != cudaSuccess) break;
        if ((e = cudaFuncSetAttribute(fr_crypt_kernel<FR_MODE_ENC, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, FR_SMEM_LAUNCH_BYTES)) != cudaSuccess) break;
        if ((e = cudaFuncSetAttribute(fr_crypt_kernel<FR_MODE_CTR>, cudaFuncAttributeMaxDynamicSharedMemorySize, FR_SMEM_LAUNCH_BYTES)) != cudaSuccess) break;
        if ((e = cudaFuncSetAttribute(fr_crypt_kernel<FR_MODE_VERIFY>, cudaFuncAttributeMaxDynamicSharedMemorySize, FR_SMEM_LAUNCH_BYTES)) != cudaSuccess) break;
        if ((e = cudaFuncSetAttribute(fr_crypt_kernel<FR_MODE_PADGEN>, cudaFuncAttributeMaxDynamicSharedMemorySize, FR_SMEM_LAUNCH_BYTES)) != cudaSuccess) break;
        if ((e = cudaFuncSetAttribute(fr_crypt_kernel<FR_MODE_PADDEC>, cudaFuncAttributeMaxDynamicSharedMemorySize, FR_SMEM_LAUNCH_BYTES)) != cudaSuccess) break;
        if ((e = cudaFuncSetAttribute(fr_verify_sequential_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, FR_SMEM_BYTES)) != cudaSuccess) break;
        if ((e = cudaFuncSetAttribute(fr_packed_kernel<FR_MODE_DEC, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, FR_SMEM_LAUNCH_BYTES)) != cudaSuccess) break;
        if ((e = cudaFuncSetAttribute(fr_packed_kernel<FR_MODE_DEC, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, FR_SMEM_LAUNCH_BYTES)) != cudaSuccess) break;
        if ((e = cudaFuncSetAttribute(fr_packed_kernel<FR_MODE_ENC, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, FR_SMEM_LAUNCH_BYTES)) != cudaSuccess) break;
        if ((e = cudaFuncSetAttribute(fr_packed_kernel<FR_MODE_ENC, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, FR_SMEM_LAUNCH_BYTES)) != cudaSuccess) break;
        if ((e = cudaFuncSetAttribute(fr_packed_kernel<FR_MODE_CTR, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, FR_SMEM_LAUNCH_BYTES)) != cudaSuccess) break;
        if ((e = cudaFuncSetAttribute(fr_packed_kernel<FR_MODE_CTR, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, FR_SMEM_LAUNCH_BYTES)) != cudaSuccess) break;
        if ((e = cudaFuncSetAttribute(fr_packed_kernel<FR_MODE_VERIFY, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, FR_SMEM_LAUNCH_BYTES)) != cudaSuccess) break;
        if ((e = cudaFuncSetAttribute(fr_packed_kernel<FR_MODE_VERIFY, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, FR_SMEM_LAUNCH_BYTES)) != cudaSuccess) break;
        for (int i = 0; i < 8 && e == cudaSuccess; i++) e = cudaStreamCreateWithFlags(&ctx->streams[i], cudaStreamNonBlocking);
        if (e != cudaSuccess) break;
        if ((e = cudaEventCreateWithFlags(&ctx->tags_ready, cudaEventDisableTiming)) != cudaSuccess) break;
        if ((e = cudaEventCreateWithFlags(&ctx->pad_ready, cudaEventDisableTiming)) != cudaSuccess) break;
        e = cudaDeviceSynchronize();
    } while (0);
    secure_zero(tab, 2 * 65536);
    free(tab);
    if (e != cudaSuccess) {
        ctx->last_cuda_error = (int)e;
        (void)cudaGetLastError();
        return fail(e == cudaErrorMemoryAllocation ? FASTRACK_ERR_NOMEM : FASTRACK_ERR_CUDA);
    }
    *out = ctx;
    return FASTRACK_OK;
}

extern "C" void fastrack_ctx_destroy(fastrack_ctx* ctx)
{
    if (!ctx) return;
    cudaDeviceSynchronize();
    if (ctx->d_gh_tab) { cudaMemset(ctx->d_gh_tab, 0, 65536); }
    if (ctx->d_gh1_tab) { cudaMemset(ctx->d_gh1_tab, 0, 65536); }
    for (int i = 0; i < 2; i++)
        if (ctx->d_pack_tab[i]) { cudaMemset(ctx->d_pack_tab[i], 0, 65536); }
    if (ctx->d_pow) { cudaMemset(ctx->d_pow, 0, ctx->pow_entries * 16); }
    if (ctx->d_tags_stage) { cudaMemset(ctx->d_tags_stage, 0, ctx->tags_stage_chunks * 32); }   // its second half held tag masks E_K(J0)
    cudaDeviceSynchronize();
    cudaFree(ctx->d_te0);
    cudaFree(ctx->d_gh_tab);
    cudaFree(ctx->d_gh1_tab);
    cudaFree(ctx->d_pack_tab[0]);
    cudaFree(ctx->d_pack_tab[1]);
    cudaFree(ctx->d_pow);
    cudaFree(ctx->d_scratch);
    cudaFree(ctx->d_timeouts);
    cudaFree(ctx->d_tags_stage);
    for (int i = 0; i < 8; i++)
        if (ctx->streams[i]) cudaStreamDestroy(ctx->streams[i]);
    if (ctx->tags_ready) cudaEventDestroy(ctx->tags_ready);
    if (ctx->pad_ready) cudaEventDestroy(ctx->pad_ready);
    for (int i = 0; i < 3 * FR_MAX_STAGES; i++)
        if (ctx->trace_ev[i]) cudaEventDestroy(ctx->trace_ev[i]);
    (void)cudaGetLastError();
    secure_zero(ctx, sizeof *ctx);
    delete ctx;
}

extern "C" size_t fastrack_num_chunks(const fastrack_ctx* ctx, size_t len)
{
    if (!ctx || len == 0) return 0;
    return (len + ctx->chunk_bytes - 1) / ctx->chunk_bytes;
}

extern "C" int fastrack_ctx_reserve(fastrack_ctx* ctx, size_t max_len)
{
    (void)max_len;                       // the scratch is a fixed set of records per context: nothing to grow
    return ctx ? FASTRACK_OK : FASTRACK_ERR_ARG;
}

extern "C" int fastrack_ctx_set_option(fastrack_ctx* ctx, int option, uint64_t value)
{
    if (!ctx) return FASTRACK_ERR_ARG;
    for (auto& memo : ctx->pack_memo) memo.valid = false;         // the planners' answers depend on these
    switch (option) {
        case FASTRACK_OPT_ROW_SLOTS:         ctx->plan.row_slots_override = (uint32_t)(value > 0xFFFFFFFFull ? 0xFFFFFFFFull : value); break;
        case FASTRACK_OPT_GENERIC_SMEM:      ctx->generic_smem = value != 0; break;
        case FASTRACK_OPT_NO_OVERLAP_LAUNCH: ctx->no_overlap_launch = value != 0; break;
        case FASTRACK_OPT_STAGE_BYTES:       ctx->plan.stage_bytes_override = (size_t)value; break;
        case FASTRACK_OPT_DIRECT_SMALL:      ctx->direct_small_h2d = value != 0; break;
        case FASTRACK_OPT_PACK_MAX_BLOCKS:   ctx->plan.pack_max_blocks = (uint32_t)(value > FR_PACK_MAX_BLOCKS ? FR_PACK_MAX_BLOCKS : value); break;
        case FASTRACK_OPT_PACK_RUN:          ctx->plan.pack_run_override = (uint32_t)(value > 0xFFFFFFFFull ? 0xFFFFFFFFull : value); break;
        case FASTRACK_OPT_PACK_GROUP:        ctx->plan.pack_group_override = (uint32_t)(value > 0xFFFFFFFFull ? 0xFFFFFFFFull : value); break;
        case FASTRACK_OPT_FOLD_TAIL:         if (value > 2) return FASTRACK_ERR_ARG; ctx->plan.fold_tail_mode = (uint32_t)value; break;
        default: return FASTRACK_ERR_ARG;
    }
    return FASTRACK_OK;
}

extern "C" int fastrack_ctx_set_framing(fastrack_ctx* ctx, unsigned chains_per_sample)
{
    if (!ctx || chains_per_sample > 256) return FASTRACK_ERR_ARG;
    ctx->aad_mod = chains_per_sample;
    return FASTRACK_OK;
}

extern "C" int fastrack_ctx_set_trace(fastrack_ctx* ctx, int enable)
{
    if (!ctx) return FASTRACK_ERR_ARG;
    if (enable && !ctx->trace_ev[0]) {
        for (int i = 0; i < 3 * FR_MAX_STAGES; i++) FR_CUDA(ctx, cudaEventCreate(&ctx->trace_ev[i]));
    }
    ctx->trace_on = enable ? 1 : 0;
    ctx->trace_count = 0;
    return FASTRACK_OK;
}

extern "C" size_t fastrack_ctx_get_trace(const fastrack_ctx* ctx, fastrack_stage_trace* out, size_t cap)
{
    if (!ctx) return 0;
    if (out)
        for (size_t i = 0; i < ctx->trace_count && i < cap; i++) out[i] = ctx->trace[i];
    return ctx->trace_count;
}

extern "C" int fastrack_last_cuda_error(const fastrack_ctx* ctx) { return ctx ? ctx->last_cuda_error : 0; }

extern "C" uint64_t fastrack_launch_count(const fastrack_ctx* ctx) { return ctx ? ctx->launches : 0; }

// ------------------------------------------------------------------------------------ launches ----

static uint32_t load_be32(const uint8_t* p) { return ((uint32_t)p[0] << 24) | ((uint32_t)p[1] << 16) | ((uint32_t)p[2] << 8) | p[3]; }
static uint32_t load_le32(const uint8_t* p) { return ((uint32_t)p[3] << 24) | ((uint32_t)p[2] << 16) | ((uint32_t)p[1] << 8) | p[0]; }


// (BE64(8 * aad bytes) || BE64(8 * bytes)) * H: the length block's term of a chunk of `bytes` bytes.
static uint4 length_term(const fastrack_ctx* ctx, uint64_t bytes)
{
    uint8_t blk[16] = {0}, out[16];
    const uint64_t bits = bytes * 8;
    if (ctx->aad_mod) blk[7] = 8;                    // BE64(bit length of the AAD): one byte
    for (int i = 0; i < 8; i++) blk[8 + i] = (uint8_t)(bits >> (56 - 8 * i));
    gf_store(gf_mul(gf_load(blk), gf_load(ctx->h)), out);
    uint4 r;
    memcpy(&r, out, 16);
    return r;
}

// Fills the geometry of a launch into P: the row kernels' plan (fastrack_plan.h) and the per-sample layout.
static FrRowPlan plan_rows(const fastrack_ctx* ctx, int mode, size_t sample_bytes, size_t n_chunks, FrParams& P)
{
    const FrRowPlan rows = fr_plan_rows(ctx->plan, sample_bytes, n_chunks, mode == FR_MODE_DEC || mode == FR_MODE_ENC);
    P.fold_tail = rows.fold_tail;
    P.n_slots = rows.n_slots;
    P.warps_used = rows.warps_used;
    P.rows_full = rows.rows_full;
    P.rows_last = rows.rows_last;
    P.rows_sample = rows.rows_sample;
    P.total_rows = rows.total_rows;
    const size_t first_len = sample_bytes < ctx->chunk_bytes ? sample_bytes : ctx->chunk_bytes;
    const size_t cps = (sample_bytes + ctx->chunk_bytes - 1) / ctx->chunk_bytes;
    const size_t last_len = sample_bytes - (cps - 1) * ctx->chunk_bytes;     // a sample's last chunk may be short
    P.sample_bytes = sample_bytes;
    P.chunks_per_sample = (uint32_t)cps;
    P.lenh_full = length_term(ctx, first_len);
    P.lenh_last = length_term(ctx, last_len);
    return rows;
}

// Row kernels (false) or packed-row kernels (true; P is switched over to them)?
// fr_plan_packed decides; its last answer per kind of pass is kept, since callers repeat shapes.
static bool plan_packed(fastrack_ctx* ctx, int mode, size_t sample_bytes, size_t n_chunks, const FrRowPlan& rows, FrParams& P)
{
    const int kind = mode == FR_MODE_CTR ? FR_PASS_CTR : mode == FR_MODE_VERIFY ? FR_PASS_VERIFY : FR_PASS_FUSED;
    auto& memo = ctx->pack_memo[kind];
    if (!(memo.valid && memo.sample_bytes == sample_bytes && memo.n_chunks == n_chunks)) {
        memo.plan = fr_plan_packed(ctx->plan, kind, sample_bytes, n_chunks, rows);
        memo.sample_bytes = sample_bytes;
        memo.n_chunks = n_chunks;
        memo.valid = true;
    }
    if (!memo.plan.run) return false;
    P.pack_run = memo.plan.run;
    P.n_items = memo.plan.n_items;
    return true;
}

// Buffers of one pass (which ones are used depends on the mode, see FrMode).
struct PassBuffers {
    const void* in = nullptr;
    void* out = nullptr;
    const void* pad = nullptr;
    void* mask = nullptr;
    const void* tags_in = nullptr;
    void* tags_out = nullptr;
    uint32_t* ok = nullptr;
    int bank = 0;              // which bank of combine records the pass uses (1: fastrack_verify)
    int window = 0;            // which window of that bank: 0 = the caller's stream, 1 + i = internal stream i
    uint32_t* acc_override = nullptr;   // combine records outside the context's own (fastrack_decrypt_verify_noalloc)
    bool plain_launch = false;          // launch without the programmatic-dependency attribute
    bool rows_only = false;             // never the packed-row kernels
    const void* ivs = nullptr; // batch of samples: per-sample IV bases on the device (then iv_base is unused)
    size_t sample_bytes = 0;   // batch of samples: bytes per sample (0: the launch is one plain buffer)
};

// Launch one pass over `len` bytes that start at chunk index `first_chunk` of the caller's buffer.
static int launch_pass(fastrack_ctx* ctx, int mode, const uint8_t iv_base[12], size_t first_chunk, size_t len,
                       const PassBuffers& b, cudaStream_t stream)
{
    FrParams P;
    memset(&P, 0, sizeof P);
    memcpy(P.rk, ctx->rk, sizeof P.rk);
    memcpy(P.te0c, ctx->te0_host, sizeof P.te0c);
    if (iv_base) {
        P.iv_w0 = load_le32(iv_base);
        P.iv_w1 = load_le32(iv_base + 4);
        P.iv_ctr = load_be32(iv_base + 8) + (uint32_t)first_chunk;
    }
    P.ivs = (const uint8_t*)b.ivs;
    P.first_chunk = (uint32_t)first_chunk;
    P.aad_mod = ctx->aad_mod;
    P.generic_smem = ctx->generic_smem;
    P.len = len;
    P.chunk_bytes = ctx->chunk_bytes;
    const size_t sample_bytes = b.sample_bytes ? b.sample_bytes : len;
    const size_t cps = (sample_bytes + ctx->chunk_bytes - 1) / ctx->chunk_bytes;
    const size_t n_chunks = (len / sample_bytes) * cps;            // len is a whole number of samples
    P.n_chunks = (uint32_t)n_chunks;

    const FrRowPlan rows = plan_rows(ctx, mode, sample_bytes, n_chunks, P);
    // Many short chains: one run of counters per lane (see fr_packed_body) when that is predicted to be faster.
    const bool packed = !b.rows_only && (mode == FR_MODE_DEC || mode == FR_MODE_ENC || mode == FR_MODE_CTR || mode == FR_MODE_VERIFY) &&
                        plan_packed(ctx, mode, sample_bytes, n_chunks, rows, P);

    P.in = (const uint8_t*)b.in;
    P.out = (uint8_t*)b.out;
    P.pad = (const uint8_t*)b.pad;
    P.mask = (uint4*)b.mask;
    P.tags_in = (const uint4*)b.tags_in;
    P.tags_out = (uint4*)b.tags_out;
    P.ok = b.ok;
    P.te0 = ctx->d_te0;
    P.timeouts = ctx->d_timeouts;
    P.gh_tab = ctx->d_gh_tab;
    const size_t full_blocks = ((sample_bytes < ctx->chunk_bytes ? sample_bytes : ctx->chunk_bytes) + 15) / 16;
    bool tables_rebuilt = false;
    if (packed) {
        // The packed rows fold with the fixed multiplier H^lanes (lanes = slots per chunk).  H and H^32 exist per
        // context; any other power gets its byte tables built on the stream, in front of the kernel that needs
        // them, and is kept until a launch asks for another one.  (Per scratch bank, so that a fastrack_verify on
        // another stream does not pull the tables from under the pass it overlaps.)
        const uint32_t lanes = (uint32_t)((full_blocks + P.pack_run) / P.pack_run);
        if (lanes == 1u) {
            P.gh_tab = ctx->d_gh1_tab;
        } else if (lanes != FR_HORNER_STRIDE) {
            if (ctx->pack_tab_lanes[b.bank] != lanes) {
                ctx->pack_tab_lanes[b.bank] = 0;
                fr_byte_tables_kernel<<<16, 256, 0, stream>>>(ctx->d_pow, lanes, ctx->d_pack_tab[b.bank]);
                ctx->launches++;
                FR_CUDA(ctx, cudaGetLastError());
                // a pipelined call issues its stages on several streams: the others must not run ahead of this
                if (b.window != 0) FR_CUDA(ctx, cudaStreamSynchronize(stream));
                ctx->pack_tab_lanes[b.bank] = lanes;
                tables_rebuilt = true;
            }
            P.gh_tab = ctx->d_pack_tab[b.bank];
        }
    }
    // One lane per chunk (run >= blocks + 1) has a kernel variant of its own that closes with two table steps and needs
    // no reduction across lanes.  It wins while the integer pipes are the busier ones (up to 3 blocks per chunk) or the
    // launch is short enough for the reduction's latency to show; beyond that the general product is the better closing.
    const bool whole = packed && P.pack_run > full_blocks &&
                       (full_blocks <= 3 || n_chunks <= 2 * (size_t)ctx->num_sms * FR_THREADS);
    P.pow = ctx->d_pow;
    P.acc = b.acc_override ? b.acc_override
                           : ctx->d_scratch + ((size_t)b.bank * FR_SCRATCH_WINDOWS + (size_t)b.window) * (size_t)ctx->num_sms * 8;

    unsigned grid = rows.grid;
    if (packed) {
        grid = (unsigned)ctx->num_sms;
        if (P.n_items < grid) grid = P.n_items;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(FR_THREADS);
    cfg.dynamicSmemBytes = FR_SMEM_LAUNCH_BYTES;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    if (!ctx->no_overlap_launch && !b.plain_launch && !tables_rebuilt) {     // (the kernel reads its tables before it waits for its predecessor)
        // let this kernel's table build overlap the tail of the previous kernel in the stream (see the kernel)
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
    }
    cudaError_t le;
    switch (mode) {
        case FR_MODE_DEC:    le = packed ? (whole ? cudaLaunchKernelEx(&cfg, fr_packed_kernel<FR_MODE_DEC, true>, P)
                                                  : cudaLaunchKernelEx(&cfg, fr_packed_kernel<FR_MODE_DEC, false>, P))
                                         : P.fold_tail ? cudaLaunchKernelEx(&cfg, fr_crypt_kernel<FR_MODE_DEC, true>, P)
                                                       : cudaLaunchKernelEx(&cfg, fr_crypt_kernel<FR_MODE_DEC>, P); break;
        case FR_MODE_ENC:    le = packed ? (whole ? cudaLaunchKernelEx(&cfg, fr_packed_kernel<FR_MODE_ENC, true>, P)
                                                  : cudaLaunchKernelEx(&cfg, fr_packed_kernel<FR_MODE_ENC, false>, P))
                                         : P.fold_tail ? cudaLaunchKernelEx(&cfg, fr_crypt_kernel<FR_MODE_ENC, true>, P)
                                                       : cudaLaunchKernelEx(&cfg, fr_crypt_kernel<FR_MODE_ENC>, P); break;
        case FR_MODE_CTR:    le = packed ? (whole ? cudaLaunchKernelEx(&cfg, fr_packed_kernel<FR_MODE_CTR, true>, P)
                                                  : cudaLaunchKernelEx(&cfg, fr_packed_kernel<FR_MODE_CTR, false>, P))
                                         : cudaLaunchKernelEx(&cfg, fr_crypt_kernel<FR_MODE_CTR>, P); break;
        case FR_MODE_VERIFY: le = packed ? (whole ? cudaLaunchKernelEx(&cfg, fr_packed_kernel<FR_MODE_VERIFY, true>, P)
                                                  : cudaLaunchKernelEx(&cfg, fr_packed_kernel<FR_MODE_VERIFY, false>, P))
                                         : cudaLaunchKernelEx(&cfg, fr_crypt_kernel<FR_MODE_VERIFY>, P); break;
        case FR_MODE_PADGEN: le = cudaLaunchKernelEx(&cfg, fr_crypt_kernel<FR_MODE_PADGEN>, P); break;
        case FR_MODE_PADDEC: le = cudaLaunchKernelEx(&cfg, fr_crypt_kernel<FR_MODE_PADDEC>, P); break;
        default: return FASTRACK_ERR_ARG;
    }
    if (le != cudaSuccess) { ctx->last_cuda_error = (int)le; (void)cudaGetLastError(); return FASTRACK_ERR_CUDA; }
    ctx->launches++;
    FR_CUDA(ctx, cudaGetLastError());
    return FASTRACK_OK;
}

static bool misaligned(const void* p, size_t a) { return ((uintptr_t)p & (a - 1)) != 0; }

static bool bad_overlap(const void* a, const void* b, size_t len)
{
    if (a == b) return false;
    uintptr_t x = (uintptr_t)a, y = (uintptr_t)b;
    return x < y + len && y < x + len;
}

extern "C" int fastrack_decrypt_verify(fastrack_ctx* ctx, const uint8_t iv_base[12], const void* d_cipher, size_t len,
                                       const void* d_tags, void* d_plain, uint32_t* d_ok, void* stream)
{
    if (!ctx || !iv_base) return FASTRACK_ERR_ARG;
    if (len == 0) return FASTRACK_OK;
    if (!d_cipher || !d_tags || !d_plain || !d_ok) return FASTRACK_ERR_ARG;
    if (misaligned(d_cipher, 16) || misaligned(d_plain, 16) || misaligned(d_tags, 16) || misaligned(d_ok, 4)) return FASTRACK_ERR_ARG;
    if (bad_overlap(d_cipher, d_plain, len)) return FASTRACK_ERR_ARG;
    const size_t K = fastrack_num_chunks(ctx, len);
    if (K > 0xFFFFFFFFull) return FASTRACK_ERR_TOO_MANY;
    int rc = check_device(ctx);
    if (rc != FASTRACK_OK) return rc;
    PassBuffers b;
    b.in = d_cipher; b.out = d_plain; b.tags_in = d_tags; b.ok = d_ok;
    return launch_pass(ctx, FR_MODE_DEC, iv_base, 0, len, b, (cudaStream_t)stream);
}

extern "C" int fastrack_encrypt_tag(fastrack_ctx* ctx, const uint8_t iv_base[12], const void* d_plain, size_t len,
                                    void* d_cipher, void* d_tags, void* stream)
{
    if (!ctx || !iv_base) return FASTRACK_ERR_ARG;
    if (len == 0) return FASTRACK_OK;
    if (!d_plain || !d_cipher || !d_tags) return FASTRACK_ERR_ARG;
    if (misaligned(d_cipher, 16) || misaligned(d_plain, 16) || misaligned(d_tags, 16)) return FASTRACK_ERR_ARG;
    if (bad_overlap(d_cipher, d_plain, len)) return FASTRACK_ERR_ARG;
    const size_t K = fastrack_num_chunks(ctx, len);
    if (K > 0xFFFFFFFFull) return FASTRACK_ERR_TOO_MANY;
    int rc = check_device(ctx);
    if (rc != FASTRACK_OK) return rc;
    PassBuffers b;
    b.in = d_plain; b.out = d_cipher; b.tags_out = d_tags;
    return launch_pass(ctx, FR_MODE_ENC, iv_base, 0, len, b, (cudaStream_t)stream);
}

// Stage = the unit that is copied and processed in place: whole chunks.  In a pipelined transfer only two
// things are not hidden behind a copy: a few microseconds per copy boundary and ONE kernel (the last stage's
// on the way in, the first stage's on the way out).  So the stages shrink geometrically: three quarters of
// the buffer, then three quarters of the rest, ... down to about 2 MiB (never less than one chunk) -- few copies,
// and a short exposed kernel.  A stage's kernel is 6-9 times faster than a copy of the same size, so it still
// finishes under the next stage's copy, which is a quarter as large.  Returns the stage sizes in descending order (host->device order).
static size_t plan_stages(const fastrack_ctx* ctx, size_t len, size_t unit, size_t out[FR_MAX_STAGES])
{
    return fr_plan_stages(ctx->plan, len, unit, out);
}

// Common body of the two pipelined entry points.  d_pad == nullptr: fused decrypt+verify per stage.
// d_pad != nullptr: the keystream for the whole buffer is produced first, on a stream of its own, while the
// first copy is in flight; the stages then only XOR and authenticate.
static int pipelined_impl(fastrack_ctx* ctx, const uint8_t iv_base[12], const void* h_cipher_pinned, size_t len,
                          const void* h_tags, void* d_pad, void* d_plain, uint32_t* d_ok, int n_streams,
                          const void* h_iv_bases = nullptr, size_t sample_bytes = 0)
{
    if (!ctx || (!iv_base && !h_iv_bases)) return FASTRACK_ERR_ARG;
    if (n_streams < 1 || n_streams > 8) return FASTRACK_ERR_ARG;
    if (len == 0) return FASTRACK_OK;
    if (!h_cipher_pinned || !h_tags || !d_plain || !d_ok) return FASTRACK_ERR_ARG;
    if (misaligned(d_plain, 16) || misaligned(d_ok, 4)) return FASTRACK_ERR_ARG;
    if (d_pad && (misaligned(d_pad, 16) || d_pad == d_plain || bad_overlap(d_pad, d_plain, len))) return FASTRACK_ERR_ARG;
    cudaPointerAttributes attr;
    cudaError_t e = cudaPointerGetAttributes(&attr, h_cipher_pinned);
    if (e != cudaSuccess) { (void)cudaGetLastError(); return FASTRACK_ERR_NOT_PINNED; }
    if (attr.type != cudaMemoryTypeHost) return FASTRACK_ERR_NOT_PINNED;
    const size_t cps = sample_bytes ? (sample_bytes + ctx->chunk_bytes - 1) / ctx->chunk_bytes : 0;
    const size_t n_samples = sample_bytes ? len / sample_bytes : 0;
    const size_t K = sample_bytes ? cps * n_samples : fastrack_num_chunks(ctx, len);
    if (K > 0xFFFFFFFFull) return FASTRACK_ERR_TOO_MANY;
    int rc = check_device(ctx);
    if (rc != FASTRACK_OK) return rc;
    const size_t need_slots = K + (12 * n_samples + 15) / 16;      // tags, then (batch of samples) the IV bases
    if (need_slots > ctx->tags_stage_chunks) {
        size_t cap = ctx->tags_stage_chunks ? ctx->tags_stage_chunks : 1024;
        while (cap < need_slots) cap *= 2;
        FR_CUDA(ctx, cudaDeviceSynchronize());
        if (ctx->d_tags_stage) cudaMemset(ctx->d_tags_stage, 0, ctx->tags_stage_chunks * 32);    // tag masks may be in there
        cudaFree(ctx->d_tags_stage);
        ctx->d_tags_stage = nullptr;
        ctx->tags_stage_chunks = 0;
        e = cudaMalloc(&ctx->d_tags_stage, cap * 32);       // tags (+ IV bases), then the E_K(J0) masks of the keystream-ahead variant
        if (e != cudaSuccess) { ctx->last_cuda_error = (int)e; (void)cudaGetLastError(); return FASTRACK_ERR_NOMEM; }
        ctx->tags_stage_chunks = cap;
    }
    uint4* d_mask = ctx->d_tags_stage + ctx->tags_stage_chunks;

    // Tags: one small copy on a stream of its own.  It (and, if asked for, the keystream kernel) is issued right
    // after the first payload copy has been queued, so that nothing delays that copy; every working stream waits
    // for both before its first kernel.
    cudaStream_t tag_stream = ctx->streams[7], pad_stream = ctx->streams[6];
    bool waited[8] = {false, false, false, false, false, false, false, false};   // per working stream: events already awaited

    size_t stage_bytes[FR_MAX_STAGES];
    const size_t cb = ctx->chunk_bytes;
    const size_t n_stages = plan_stages(ctx, len, sample_bytes ? sample_bytes : cb, stage_bytes);
    uint8_t* d_ivs = (uint8_t*)(ctx->d_tags_stage + K);            // batch of samples: device copy of the IV bases

    // A transfer of a single stage has nothing to overlap: copy, then kernel, each with its own start-up latency.
    // There the kernel reads the ciphertext straight from the page-locked host buffer instead (every block is read
    // exactly once, 512 contiguous bytes per warp request), so the transfer IS the kernel: no copy engine set-up,
    // no copy-to-kernel dependency.  Larger transfers keep the copy engine, which leaves the SMs free.
    // (Measured: a gain of 3-10 us up to 1 MiB whatever the chunk size; from there to the 3 MiB a single stage can
    // have, only while a lane's reads stay wide -- small chunks in the packed layout read 16 bytes at a stride, which
    // the link serves poorly.)
    if (n_stages == 1 && !d_pad && ctx->direct_small_h2d && attr.devicePointer && !misaligned(attr.devicePointer, 16) &&
        (len <= ((size_t)1 << 20) || cb >= 4096)) {
        cudaStream_t st = ctx->streams[0];
        const uint4* tags_src = ctx->d_tags_stage;
        cudaPointerAttributes ta;
        if (cudaPointerGetAttributes(&ta, h_tags) == cudaSuccess && ta.type == cudaMemoryTypeHost && ta.devicePointer &&
            !misaligned(ta.devicePointer, 16)) {
            tags_src = (const uint4*)ta.devicePointer;             // page-locked tags are read in place too
        } else {
            (void)cudaGetLastError();
            FR_CUDA(ctx, cudaMemcpyAsync(ctx->d_tags_stage, h_tags, K * 16, cudaMemcpyHostToDevice, st));
        }
        if (sample_bytes) FR_CUDA(ctx, cudaMemcpyAsync(d_ivs, h_iv_bases, 12 * n_samples, cudaMemcpyHostToDevice, st));
        const bool tracing = ctx->trace_on;
        if (tracing) { cudaEventRecord(ctx->trace_ev[0], st); cudaEventRecord(ctx->trace_ev[1], st); }
        PassBuffers b;
        b.window = 1;
        b.in = attr.devicePointer; b.out = d_plain; b.tags_in = tags_src; b.ok = d_ok;
        if (sample_bytes) { b.ivs = d_ivs; b.sample_bytes = sample_bytes; }
        rc = launch_pass(ctx, FR_MODE_DEC, iv_base, 0, len, b, st);
        if (tracing) cudaEventRecord(ctx->trace_ev[2], st);
        cudaError_t se = cudaStreamSynchronize(st);
        if (rc != FASTRACK_OK) return rc;
        FR_CUDA(ctx, se);
        if (tracing) {
            ctx->trace_count = 1;
            ctx->trace[0].offset = 0; ctx->trace[0].bytes = len; ctx->trace[0].stream = 0;
            cudaEventElapsedTime(&ctx->trace[0].copy_start_ms, ctx->trace_ev[0], ctx->trace_ev[0]);
            cudaEventElapsedTime(&ctx->trace[0].copy_end_ms, ctx->trace_ev[0], ctx->trace_ev[1]);
            cudaEventElapsedTime(&ctx->trace[0].kernel_end_ms, ctx->trace_ev[0], ctx->trace_ev[2]);
            (void)cudaGetLastError();
        }
        return FASTRACK_OK;
    }

    size_t off = 0;
    for (size_t stage = 0; stage < n_stages; stage++) {
        const size_t n = stage_bytes[stage];
        const size_t k0 = sample_bytes ? (off / sample_bytes) * cps : off / cb;
        cudaStream_t st = ctx->streams[stage % (size_t)n_streams];
        uint8_t* dst = (uint8_t*)d_plain + off;
        rc = FASTRACK_OK;
        const bool tracing = ctx->trace_on && stage < FR_MAX_STAGES;
        if (tracing) cudaEventRecord(ctx->trace_ev[3 * stage], st);
        e = cudaMemcpyAsync(dst, (const uint8_t*)h_cipher_pinned + off, n, cudaMemcpyHostToDevice, st);
        if (e != cudaSuccess) { ctx->last_cuda_error = (int)e; (void)cudaGetLastError(); rc = FASTRACK_ERR_CUDA; }
        if (tracing) cudaEventRecord(ctx->trace_ev[3 * stage + 1], st);
        if (rc == FASTRACK_OK && stage == 0) {
            e = cudaMemcpyAsync(ctx->d_tags_stage, h_tags, K * 16, cudaMemcpyHostToDevice, tag_stream);
            if (e == cudaSuccess && sample_bytes)
                e = cudaMemcpyAsync(d_ivs, h_iv_bases, 12 * n_samples, cudaMemcpyHostToDevice, tag_stream);
            if (e == cudaSuccess) e = cudaEventRecord(ctx->tags_ready, tag_stream);
            if (e != cudaSuccess) { ctx->last_cuda_error = (int)e; (void)cudaGetLastError(); rc = FASTRACK_ERR_CUDA; }
            if (rc == FASTRACK_OK && d_pad) {
                PassBuffers pb;            // (no authentication in this pass: it uses no combine records)
                pb.out = d_pad; pb.mask = d_mask;
                rc = launch_pass(ctx, FR_MODE_PADGEN, iv_base, 0, len, pb, pad_stream);
                if (rc == FASTRACK_OK && (e = cudaEventRecord(ctx->pad_ready, pad_stream)) != cudaSuccess) {
                    ctx->last_cuda_error = (int)e; (void)cudaGetLastError(); rc = FASTRACK_ERR_CUDA;
                }
            }
        }
        const size_t si = stage % (size_t)n_streams;
        if (rc == FASTRACK_OK && !waited[si]) {
            // the stream's first kernel (not its first copy) waits for the tags and, if used, the keystream
            waited[si] = true;
            if (st != tag_stream) e = cudaStreamWaitEvent(st, ctx->tags_ready, 0);
            if (e == cudaSuccess && d_pad && st != pad_stream) e = cudaStreamWaitEvent(st, ctx->pad_ready, 0);
            if (e != cudaSuccess) { ctx->last_cuda_error = (int)e; (void)cudaGetLastError(); rc = FASTRACK_ERR_CUDA; }
        }
        if (rc == FASTRACK_OK) {
            PassBuffers b;
            b.window = 1 + (int)si;
            b.in = dst; b.out = dst; b.tags_in = ctx->d_tags_stage + k0; b.ok = d_ok + k0;
            if (sample_bytes) { b.ivs = d_ivs + 12 * (off / sample_bytes); b.sample_bytes = sample_bytes; }
            if (d_pad) { b.pad = (const uint8_t*)d_pad + off; b.mask = d_mask + k0; }
            rc = launch_pass(ctx, d_pad ? FR_MODE_PADDEC : FR_MODE_DEC, iv_base, k0, n, b, st);
        }
        if (tracing) {
            cudaEventRecord(ctx->trace_ev[3 * stage + 2], st);
            ctx->trace[stage].offset = off;
            ctx->trace[stage].bytes = n;
            ctx->trace[stage].stream = (int)(stage % (size_t)n_streams);
        }
        if (rc != FASTRACK_OK) {
            for (int i = 0; i < 8; i++) cudaStreamSynchronize(ctx->streams[i]);
            (void)cudaGetLastError();
            return rc;
        }
        off += n;
    }
    FR_CUDA(ctx, cudaStreamSynchronize(tag_stream));
    if (d_pad) FR_CUDA(ctx, cudaStreamSynchronize(pad_stream));
    for (int i = 0; i < n_streams; i++) FR_CUDA(ctx, cudaStreamSynchronize(ctx->streams[i]));
    if (d_pad) FR_CUDA(ctx, cudaMemsetAsync(d_mask, 0, 16 * K, tag_stream));   // the tag masks E_K(J0) are as sensitive as H: do not leave them behind
    if (d_pad) FR_CUDA(ctx, cudaStreamSynchronize(tag_stream));
    if (ctx->trace_on) {
        ctx->trace_count = n_stages < FR_MAX_STAGES ? n_stages : FR_MAX_STAGES;
        for (size_t i = 0; i < ctx->trace_count; i++) {
            cudaEventElapsedTime(&ctx->trace[i].copy_start_ms, ctx->trace_ev[0], ctx->trace_ev[3 * i]);
            cudaEventElapsedTime(&ctx->trace[i].copy_end_ms, ctx->trace_ev[0], ctx->trace_ev[3 * i + 1]);
            cudaEventElapsedTime(&ctx->trace[i].kernel_end_ms, ctx->trace_ev[0], ctx->trace_ev[3 * i + 2]);
        }
        (void)cudaGetLastError();
    }
    return FASTRACK_OK;
}

extern "C" int fastrack_pipelined_h2d(fastrack_ctx* ctx, const uint8_t iv_base[12], const void* h_cipher_pinned, size_t len,
                                      const void* h_tags, void* d_plain, uint32_t* d_ok, int n_streams)
{
    return pipelined_impl(ctx, iv_base, h_cipher_pinned, len, h_tags, nullptr, d_plain, d_ok, n_streams);
}

extern "C" int fastrack_pipelined_h2d_samples(fastrack_ctx* ctx, const void* h_iv_bases, size_t sample_bytes, size_t n_samples,
                                              const void* h_cipher_pinned, const void* h_tags, void* d_plain, uint32_t* d_ok,
                                              int n_streams)
{
    if (!ctx || !h_iv_bases) return FASTRACK_ERR_ARG;
    if (sample_bytes == 0 || (sample_bytes & 15)) return FASTRACK_ERR_ARG;
    if (n_samples > ((size_t)1 << 40) / sample_bytes) return FASTRACK_ERR_TOO_MANY;
    return pipelined_impl(ctx, nullptr, h_cipher_pinned, sample_bytes * n_samples, h_tags, nullptr, d_plain, d_ok, n_streams,
                          h_iv_bases, sample_bytes);
}

extern "C" int fastrack_pipelined_h2d_ahead(fastrack_ctx* ctx, const uint8_t iv_base[12], const void* h_cipher_pinned,
                                            size_t len, const void* h_tags, void* d_pad, void* d_plain, uint32_t* d_ok,
                                            int n_streams)
{
    if (!d_pad) return FASTRACK_ERR_ARG;
    return pipelined_impl(ctx, iv_base, h_cipher_pinned, len, h_tags, d_pad, d_plain, d_ok, n_streams);
}

static int pipelined_d2h_impl(fastrack_ctx* ctx, const uint8_t iv_base[12], const void* d_plain, size_t len, void* d_cipher,
                              void* h_cipher_pinned, void* h_tags, int n_streams, const void* h_iv_bases = nullptr,
                              size_t sample_bytes = 0)
{
    if (!ctx || (!iv_base && !h_iv_bases)) return FASTRACK_ERR_ARG;
    if (n_streams < 1 || n_streams > 8) return FASTRACK_ERR_ARG;
    if (len == 0) return FASTRACK_OK;
    if (!d_plain || !d_cipher || !h_cipher_pinned || !h_tags) return FASTRACK_ERR_ARG;
    if (misaligned(d_plain, 16) || misaligned(d_cipher, 16) || bad_overlap(d_plain, d_cipher, len)) return FASTRACK_ERR_ARG;
    cudaPointerAttributes attr;
    cudaError_t e = cudaPointerGetAttributes(&attr, h_cipher_pinned);
    if (e != cudaSuccess) { (void)cudaGetLastError(); return FASTRACK_ERR_NOT_PINNED; }
    if (attr.type != cudaMemoryTypeHost) return FASTRACK_ERR_NOT_PINNED;
    const size_t cb = ctx->chunk_bytes;
    const size_t cps = sample_bytes ? (sample_bytes + cb - 1) / cb : 0;
    const size_t n_samples = sample_bytes ? len / sample_bytes : 0;
    const size_t K = sample_bytes ? cps * n_samples : fastrack_num_chunks(ctx, len);
    if (K > 0xFFFFFFFFull) return FASTRACK_ERR_TOO_MANY;
    int rc = check_device(ctx);
    if (rc != FASTRACK_OK) return rc;
    const size_t need_slots = K + (12 * n_samples + 15) / 16;      // tags, then (batch of samples) the IV bases
    if (need_slots > ctx->tags_stage_chunks) {
        size_t cap = ctx->tags_stage_chunks ? ctx->tags_stage_chunks : 1024;
        while (cap < need_slots) cap *= 2;
        FR_CUDA(ctx, cudaDeviceSynchronize());
        if (ctx->d_tags_stage) cudaMemset(ctx->d_tags_stage, 0, ctx->tags_stage_chunks * 32);    // tag masks may be in there
        cudaFree(ctx->d_tags_stage);
        ctx->d_tags_stage = nullptr;
        ctx->tags_stage_chunks = 0;
        e = cudaMalloc(&ctx->d_tags_stage, cap * 32);
        if (e != cudaSuccess) { ctx->last_cuda_error = (int)e; (void)cudaGetLastError(); return FASTRACK_ERR_NOMEM; }
        ctx->tags_stage_chunks = cap;
    }
    uint8_t* d_ivs = (uint8_t*)(ctx->d_tags_stage + K);
    cudaStream_t iv_stream = ctx->streams[7];
    if (sample_bytes) {                          // the IV bases go in first: one small copy, every working stream waits for it
        e = cudaMemcpyAsync(d_ivs, h_iv_bases, 12 * n_samples, cudaMemcpyHostToDevice, iv_stream);
        if (e == cudaSuccess) e = cudaEventRecord(ctx->tags_ready, iv_stream);
        if (e != cudaSuccess) { ctx->last_cuda_error = (int)e; (void)cudaGetLastError(); return FASTRACK_ERR_CUDA; }
    }
    // On the way out the FIRST stage's kernel is the exposed one: smallest stage first.  The plan is made on
    // whole chunks (K * chunk_bytes), or whole samples, and walked backwards, so every stage starts on a chunk
    // (sample) boundary and the short last chunk, if any, stays at the end of the last (largest) stage.
    size_t stage_bytes[FR_MAX_STAGES];
    const size_t unit = sample_bytes ? sample_bytes : cb;
    const size_t n_stages = plan_stages(ctx, sample_bytes ? len : K * cb, unit, stage_bytes);
    // A transfer of a single stage: the kernel writes ciphertext (and tags, if their buffer is page-locked too) straight
    // into the host buffers instead of into d_cipher followed by two copies -- the mirror of the small host-to-device case.
    // Not when encrypting in place: the caller then expects d_plain to hold the ciphertext afterwards.
    if (n_stages == 1 && ctx->direct_small_h2d && d_cipher != d_plain && attr.devicePointer && !misaligned(attr.devicePointer, 16) &&
        (len <= ((size_t)1 << 20) || cb >= 4096)) {
        cudaStream_t st = ctx->streams[0];
        if (sample_bytes) FR_CUDA(ctx, cudaStreamWaitEvent(st, ctx->tags_ready, 0));          // the IV bases
        cudaPointerAttributes ta;
        void* tags_dst = nullptr;
        if (cudaPointerGetAttributes(&ta, h_tags) == cudaSuccess && ta.type == cudaMemoryTypeHost && ta.devicePointer &&
            !misaligned(ta.devicePointer, 16)) tags_dst = ta.devicePointer;
        (void)cudaGetLastError();
        PassBuffers b;
        b.window = 1;
        b.in = d_plain; b.out = attr.devicePointer; b.tags_out = tags_dst ? tags_dst : (void*)ctx->d_tags_stage;
        if (sample_bytes) { b.ivs = d_ivs; b.sample_bytes = sample_bytes; }
        rc = launch_pass(ctx, FR_MODE_ENC, iv_base, 0, len, b, st);
        if (rc == FASTRACK_OK && !tags_dst) {
            e = cudaMemcpyAsync(h_tags, ctx->d_tags_stage, 16 * K, cudaMemcpyDeviceToHost, st);
            if (e != cudaSuccess) { ctx->last_cuda_error = (int)e; (void)cudaGetLastError(); rc = FASTRACK_ERR_CUDA; }
        }
        cudaError_t se = cudaStreamSynchronize(st);
        if (sample_bytes) cudaStreamSynchronize(iv_stream);
        if (rc != FASTRACK_OK) return rc;
        FR_CUDA(ctx, se);
        return FASTRACK_OK;
    }
    // Tags bound for page-locked memory leave with their stage.  A device-to-host copy into pageable memory blocks
    // the host until it is done, which would keep the next stage's kernel from being queued under the current
    // copy; such tags stay on the device until every stage is queued and leave in one copy at the end.
    bool tags_pinned = false;
    {
        cudaPointerAttributes ta;
        if (cudaPointerGetAttributes(&ta, h_tags) == cudaSuccess && ta.type == cudaMemoryTypeHost) tags_pinned = true;
        (void)cudaGetLastError();
    }
    bool waited[8] = {false, false, false, false, false, false, false, false};
    size_t off = 0;
    for (size_t i = 0; i < n_stages; i++) {
        size_t n = stage_bytes[n_stages - 1 - i];
        if (n > len - off) n = len - off;
        const size_t k0 = sample_bytes ? (off / sample_bytes) * cps : off / cb;
        const size_t k_here = sample_bytes ? (n / sample_bytes) * cps : (n + cb - 1) / cb;
        const size_t si = i % (size_t)n_streams;
        cudaStream_t st = ctx->streams[si];
        rc = FASTRACK_OK;
        if (sample_bytes && !waited[si]) {
            waited[si] = true;
            if (st != iv_stream && (e = cudaStreamWaitEvent(st, ctx->tags_ready, 0)) != cudaSuccess) {
                ctx->last_cuda_error = (int)e; (void)cudaGetLastError(); rc = FASTRACK_ERR_CUDA;
            }
        }
        PassBuffers b;
        b.window = 1 + (int)si;
        b.in = (const uint8_t*)d_plain + off; b.out = (uint8_t*)d_cipher + off; b.tags_out = ctx->d_tags_stage + k0;
        if (sample_bytes) { b.ivs = d_ivs + 12 * (off / sample_bytes); b.sample_bytes = sample_bytes; }
        if (rc == FASTRACK_OK) rc = launch_pass(ctx, FR_MODE_ENC, iv_base, k0, n, b, st);
        if (rc == FASTRACK_OK) {
            e = cudaMemcpyAsync((uint8_t*)h_cipher_pinned + off, (const uint8_t*)d_cipher + off, n, cudaMemcpyDeviceToHost, st);
            if (e == cudaSuccess && tags_pinned) e = cudaMemcpyAsync((uint8_t*)h_tags + 16 * k0, ctx->d_tags_stage + k0, 16 * k_here,
                                                                     cudaMemcpyDeviceToHost, st);
            if (e != cudaSuccess) { ctx->last_cuda_error = (int)e; (void)cudaGetLastError(); rc = FASTRACK_ERR_CUDA; }
        }
        if (rc != FASTRACK_OK) {
            for (int s2 = 0; s2 < 8; s2++) cudaStreamSynchronize(ctx->streams[s2]);
            (void)cudaGetLastError();
            return rc;
        }
        off += n;
    }
    if (sample_bytes) FR_CUDA(ctx, cudaStreamSynchronize(iv_stream));
    for (int i = 0; i < n_streams; i++) FR_CUDA(ctx, cudaStreamSynchronize(ctx->streams[i]));
    if (!tags_pinned) FR_CUDA(ctx, cudaMemcpy(h_tags, ctx->d_tags_stage, 16 * K, cudaMemcpyDeviceToHost));
    return FASTRACK_OK;
}

extern "C" int fastrack_pipelined_d2h(fastrack_ctx* ctx, const uint8_t iv_base[12], const void* d_plain, size_t len,
                                      void* d_cipher, void* h_cipher_pinned, void* h_tags, int n_streams)
{
    if (!iv_base) return FASTRACK_ERR_ARG;
    return pipelined_d2h_impl(ctx, iv_base, d_plain, len, d_cipher, h_cipher_pinned, h_tags, n_streams);
}

extern "C" int fastrack_pipelined_d2h_samples(fastrack_ctx* ctx, const void* h_iv_bases, size_t sample_bytes, size_t n_samples,
                                              const void* d_plain, void* d_cipher, void* h_cipher_pinned, void* h_tags,
                                              int n_streams)
{
    if (!ctx || !h_iv_bases) return FASTRACK_ERR_ARG;
    if (sample_bytes == 0 || (sample_bytes & 15)) return FASTRACK_ERR_ARG;
    if (n_samples > ((size_t)1 << 40) / sample_bytes) return FASTRACK_ERR_TOO_MANY;
    return pipelined_d2h_impl(ctx, nullptr, d_plain, sample_bytes * n_samples, d_cipher, h_cipher_pinned, h_tags, n_streams,
                              h_iv_bases, sample_bytes);
}

// Argument checks shared by the two batch-of-samples entry points.
static int check_samples(fastrack_ctx* ctx, const void* d_iv_bases, size_t sample_bytes, size_t n_samples, size_t* K_out)
{
    if (!ctx || !d_iv_bases) return FASTRACK_ERR_ARG;
    if (sample_bytes == 0 || (sample_bytes & 15)) return FASTRACK_ERR_ARG;       // samples must stay 16-byte aligned
    if (n_samples > ((size_t)1 << 40) / sample_bytes) return FASTRACK_ERR_TOO_MANY;
    const size_t cps = (sample_bytes + ctx->chunk_bytes - 1) / ctx->chunk_bytes;
    if (cps * n_samples > 0xFFFFFFFFull) return FASTRACK_ERR_TOO_MANY;
    *K_out = cps * n_samples;
    return FASTRACK_OK;
}

extern "C" int fastrack_decrypt_verify_samples(fastrack_ctx* ctx, const void* d_iv_bases, size_t sample_bytes,
                                               size_t n_samples, const void* d_cipher, const void* d_tags, void* d_plain,
                                               uint32_t* d_ok, void* stream)
{
    size_t K = 0;
    int rc = check_samples(ctx, d_iv_bases, sample_bytes, n_samples, &K);
    if (rc != FASTRACK_OK) return rc;
    if (n_samples == 0) return FASTRACK_OK;
    const size_t len = sample_bytes * n_samples;
    if (!d_cipher || !d_tags || !d_plain || !d_ok) return FASTRACK_ERR_ARG;
    if (misaligned(d_cipher, 16) || misaligned(d_plain, 16) || misaligned(d_tags, 16) || misaligned(d_ok, 4)) return FASTRACK_ERR_ARG;
    if (bad_overlap(d_cipher, d_plain, len)) return FASTRACK_ERR_ARG;
    rc = check_device(ctx);
    if (rc != FASTRACK_OK) return rc;
    PassBuffers b;
    b.in = d_cipher; b.out = d_plain; b.tags_in = d_tags; b.ok = d_ok; b.ivs = d_iv_bases; b.sample_bytes = sample_bytes;
    return launch_pass(ctx, FR_MODE_DEC, nullptr, 0, len, b, (cudaStream_t)stream);
}

extern "C" int fastrack_encrypt_tag_samples(fastrack_ctx* ctx, const void* d_iv_bases, size_t sample_bytes, size_t n_samples,
                                            const void* d_plain, void* d_cipher, void* d_tags, void* stream)
{
    size_t K = 0;
    int rc = check_samples(ctx, d_iv_bases, sample_bytes, n_samples, &K);
    if (rc != FASTRACK_OK) return rc;
    if (n_samples == 0) return FASTRACK_OK;
    const size_t len = sample_bytes * n_samples;
    if (!d_plain || !d_cipher || !d_tags) return FASTRACK_ERR_ARG;
    if (misaligned(d_cipher, 16) || misaligned(d_plain, 16) || misaligned(d_tags, 16)) return FASTRACK_ERR_ARG;
    if (bad_overlap(d_cipher, d_plain, len)) return FASTRACK_ERR_ARG;
    rc = check_device(ctx);
    if (rc != FASTRACK_OK) return rc;
    PassBuffers b;
    b.in = d_plain; b.out = d_cipher; b.tags_out = d_tags; b.ivs = d_iv_bases; b.sample_bytes = sample_bytes;
    return launch_pass(ctx, FR_MODE_ENC, nullptr, 0, len, b, (cudaStream_t)stream);
}

extern "C" int fastrack_ctr_crypt(fastrack_ctx* ctx, const uint8_t iv_base[12], const void* d_in, size_t len, void* d_out,
                                  void* stream)
{
    if (!ctx || !iv_base) return FASTRACK_ERR_ARG;
    if (len == 0) return FASTRACK_OK;
    if (!d_in || !d_out) return FASTRACK_ERR_ARG;
    if (misaligned(d_in, 16) || misaligned(d_out, 16) || bad_overlap(d_in, d_out, len)) return FASTRACK_ERR_ARG;
    if (fastrack_num_chunks(ctx, len) > 0xFFFFFFFFull) return FASTRACK_ERR_TOO_MANY;
    int rc = check_device(ctx);
    if (rc != FASTRACK_OK) return rc;
    PassBuffers b;
    b.in = d_in; b.out = d_out;
    return launch_pass(ctx, FR_MODE_CTR, iv_base, 0, len, b, (cudaStream_t)stream);
}

extern "C" int fastrack_verify(fastrack_ctx* ctx, const uint8_t iv_base[12], const void* d_cipher, size_t len,
                               const void* d_tags, uint32_t* d_ok, void* stream)
{
    if (!ctx || !iv_base) return FASTRACK_ERR_ARG;
    if (len == 0) return FASTRACK_OK;
    if (!d_cipher || !d_tags || !d_ok) return FASTRACK_ERR_ARG;
    if (misaligned(d_cipher, 16) || misaligned(d_tags, 16) || misaligned(d_ok, 4)) return FASTRACK_ERR_ARG;
    const size_t K = fastrack_num_chunks(ctx, len);
    if (K > 0xFFFFFFFFull) return FASTRACK_ERR_TOO_MANY;
    int rc = check_device(ctx);
    if (rc != FASTRACK_OK) return rc;
    PassBuffers b;
    b.in = d_cipher; b.out = const_cast<void*>(d_cipher); b.tags_in = d_tags; b.ok = d_ok; b.bank = 1;
    return launch_pass(ctx, FR_MODE_VERIFY, iv_base, 0, len, b, (cudaStream_t)stream);
}

extern "C" int fastrack_verify_sequential(fastrack_ctx* ctx, const uint8_t iv_base[12], const void* d_cipher, size_t len,
                                          const void* d_tags, uint32_t* d_ok, void* stream)
{
    if (!ctx || !iv_base) return FASTRACK_ERR_ARG;
    if (len == 0) return FASTRACK_OK;
    if (!d_cipher || !d_tags || !d_ok) return FASTRACK_ERR_ARG;
    if (misaligned(d_cipher, 16) || misaligned(d_tags, 16) || misaligned(d_ok, 4)) return FASTRACK_ERR_ARG;
    const size_t K = fastrack_num_chunks(ctx, len);
    if (K > 0xFFFFFFFFull) return FASTRACK_ERR_TOO_MANY;
    int rc = check_device(ctx);
    if (rc != FASTRACK_OK) return rc;
    FrParams P;
    memset(&P, 0, sizeof P);
    memcpy(P.rk, ctx->rk, sizeof P.rk);
    memcpy(P.te0c, ctx->te0_host, sizeof P.te0c);
    P.iv_w0 = load_le32(iv_base);
    P.iv_w1 = load_le32(iv_base + 4);
    P.iv_ctr = load_be32(iv_base + 8);
    P.aad_mod = ctx->aad_mod;
    P.len = len;
    P.chunk_bytes = ctx->chunk_bytes;
    P.n_chunks = (uint32_t)K;
    P.sample_bytes = len;
    P.chunks_per_sample = (uint32_t)K;
    P.in = (const uint8_t*)d_cipher;
    P.tags_in = (const uint4*)d_tags;
    P.ok = d_ok;
    P.te0 = ctx->d_te0;
    P.gh_tab = ctx->d_gh1_tab;
    fr_verify_sequential_kernel<<<(unsigned)((K + 31) / 32), 32, FR_SMEM_BYTES, (cudaStream_t)stream>>>(P);
    ctx->launches++;
    FR_CUDA(ctx, cudaGetLastError());
    return FASTRACK_OK;
}

extern "C" int fastrack_keystream(fastrack_ctx* ctx, const uint8_t iv_base[12], size_t len, void* d_pad, void* d_mask,
                                  void* stream)
{
    if (!ctx || !iv_base) return FASTRACK_ERR_ARG;
    if (len == 0) return FASTRACK_OK;
    if (!d_pad || !d_mask) return FASTRACK_ERR_ARG;
    if (misaligned(d_pad, 16) || misaligned(d_mask, 16)) return FASTRACK_ERR_ARG;
    if (fastrack_num_chunks(ctx, len) > 0xFFFFFFFFull) return FASTRACK_ERR_TOO_MANY;
    int rc = check_device(ctx);
    if (rc != FASTRACK_OK) return rc;
    PassBuffers b;
    b.out = d_pad; b.mask = d_mask;
    return launch_pass(ctx, FR_MODE_PADGEN, iv_base, 0, len, b, (cudaStream_t)stream);
}

extern "C" int fastrack_xor_verify(fastrack_ctx* ctx, const uint8_t iv_base[12], const void* d_cipher, size_t len,
                                   const void* d_pad, const void* d_mask, const void* d_tags, void* d_plain,
                                   uint32_t* d_ok, void* stream)
{
    if (!ctx || !iv_base) return FASTRACK_ERR_ARG;
    if (len == 0) return FASTRACK_OK;
    if (!d_cipher || !d_pad || !d_mask || !d_tags || !d_plain || !d_ok) return FASTRACK_ERR_ARG;
    if (misaligned(d_cipher, 16) || misaligned(d_plain, 16) || misaligned(d_pad, 16) || misaligned(d_mask, 16) ||
        misaligned(d_tags, 16) || misaligned(d_ok, 4)) return FASTRACK_ERR_ARG;
    if (bad_overlap(d_cipher, d_plain, len) || d_pad == d_plain || bad_overlap(d_pad, d_plain, len)) return FASTRACK_ERR_ARG;
    const size_t K = fastrack_num_chunks(ctx, len);
    if (K > 0xFFFFFFFFull) return FASTRACK_ERR_TOO_MANY;
    int rc = check_device(ctx);
    if (rc != FASTRACK_OK) return rc;
    PassBuffers b;
    b.in = d_cipher; b.out = d_plain; b.pad = d_pad; b.mask = const_cast<void*>(d_mask); b.tags_in = d_tags; b.ok = d_ok;
    return launch_pass(ctx, FR_MODE_PADDEC, iv_base, 0, len, b, (cudaStream_t)stream);
}

// ------------------------------------------------------------- entry point that allocates nothing ----
//
// Combine records for fastrack_decrypt_verify_noalloc: one 32-byte record per CTA of a launch (a launch has one
// CTA per SM), FR_NOALLOC_MAX_CTAS of them.  The array is part of the library image, so every GPU that loads the
// library holds these 32 KiB until the process exits, and every call on a device shares them.
#define FR_NOALLOC_MAX_CTAS 1024
static __device__ __align__(256) uint32_t fr_static_scratch[8 * FR_NOALLOC_MAX_CTAS];

// In host code the array's name above is only a handle for the runtime, not a device address; the real
// address differs per device and is looked up once per device with that device current.
#define FR_MAX_DEVICES 64
static uint32_t* fr_static_scratch_addr[FR_MAX_DEVICES];

extern "C" int fastrack_decrypt_verify_noalloc(fastrack_ctx* ctx, const uint8_t iv_base[12], const void* d_cipher,
                                               size_t len, const void* d_tags, void* d_plain, uint32_t* d_ok,
                                               void* stream)
{
    if (!ctx || !iv_base) return FASTRACK_ERR_ARG;
    if (len == 0) return FASTRACK_OK;
    if (!d_cipher || !d_tags || !d_plain || !d_ok) return FASTRACK_ERR_ARG;
    if (misaligned(d_cipher, 16) || misaligned(d_plain, 16) || misaligned(d_tags, 16) || misaligned(d_ok, 4)) return FASTRACK_ERR_ARG;
    if (bad_overlap(d_cipher, d_plain, len)) return FASTRACK_ERR_ARG;
    const size_t K = fastrack_num_chunks(ctx, len);
    if (K > FASTRACK_NOALLOC_MAX_CHUNKS || ctx->num_sms > FR_NOALLOC_MAX_CTAS) return FASTRACK_ERR_LIMIT;

    int rc = check_device(ctx);
    if (rc != FASTRACK_OK) return rc;
    const int dev = ctx->device;
    if (dev < 0 || dev >= FR_MAX_DEVICES) return FASTRACK_ERR_ARG;
    if (!fr_static_scratch_addr[dev]) {                 // first call on this device: resolve the symbol
        uint32_t* ptr = nullptr;
        FR_CUDA(ctx, cudaGetSymbolAddress((void**)&ptr, fr_static_scratch));
        if (!ptr) return FASTRACK_ERR_CUDA;
        fr_static_scratch_addr[dev] = ptr;
    }
    uint32_t* acc = fr_static_scratch_addr[dev];
    cudaStream_t st = (cudaStream_t)stream;
    // the array keeps whatever the previous call (possibly a failed one) left: zero what this call may use, one
    // 32-byte record per CTA of the launch
    FR_CUDA(ctx, cudaMemsetAsync(acc, 0, (size_t)ctx->num_sms * 8 * sizeof(uint32_t), st));
    // same launch as the allocating entry point, combine records aside
    PassBuffers b;
    b.in = d_cipher; b.out = d_plain; b.tags_in = d_tags; b.ok = d_ok;
    b.acc_override = acc;
    b.plain_launch = true;
    b.rows_only = true;
    return launch_pass(ctx, FR_MODE_DEC, iv_base, 0, len, b, st);
}
