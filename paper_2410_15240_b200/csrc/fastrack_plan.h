// fastrack_plan.h -- host-side planning of a launch and of a pipelined transfer: plain C++ without CUDA, so that
// the CPU-only tests can include it and check its invariants (tests/host_logic).  Three decisions are made here:
//   fr_plan_rows:     how the row kernels spread the rows of a launch over warps;
//   fr_plan_packed:   whether a launch takes the packed-row kernels instead, and with which run length and
//                     work-item size;
//   fr_plan_stages:   how a pipelined host<->device transfer is cut into stages.
// All costs are estimates in SM clocks with constants fitted to measurements on B200.
#pragma once
#include <stddef.h>
#include <stdint.h>

#ifndef FR_THREADS
#define FR_THREADS 1024
#endif
#define FR_WARPS (FR_THREADS / 32)
#define FR_MAX_STAGES 96          // most stages a pipelined call is cut into
#define FR_PLAN_ROW_BLOCKS 32     // blocks per row of the row kernels (one per lane)
#define FR_PACK_MAX_BLOCKS 4096   // chunks of more blocks than this never take the packed-row kernels
#define FR_PACK_MAX_ITEM_SLOTS 1024   // most runs (lanes' worth of work) in one packed work item

struct FrPlanConfig {
    int num_sms;
    size_t chunk_bytes;
    uint32_t row_slots_override;    // 0 = automatic; else the row kernels spread a launch over this many warps (tests, tuning)
    uint32_t pack_max_blocks;       // chunks of at most this many blocks may take the packed-row kernels (0 = never)
    uint32_t pack_run_override;     // 0 = automatic; else packed rows with this run length wherever they apply (tests)
    uint32_t pack_group_override;   // 0 = automatic; else this many chunks per packed work item (tests)
    size_t stage_bytes_override;    // 0 = automatic; else the stage size of pipelined transfers (experiments)
};

// How the row kernels spread a launch over warps: the rows of all chunks, one chunk after the other, are cut into
// n_slots contiguous ranges of equal length (to within a row); slot j is warp j % warps_used of CTA j / warps_used.
struct FrRowPlan {
    uint32_t grid;              // CTAs
    uint32_t warps_used;        // slots per CTA (the other warps of a CTA only help to fill shared memory)
    uint32_t n_slots;           // <= grid * warps_used and <= total_rows
    uint32_t rows_full;         // rows of a full-size chunk
    uint32_t rows_last;         // rows of a sample's last chunk
    uint64_t rows_sample;       // rows of a sample
    uint64_t total_rows;
};

struct FrPackPlan {
    uint32_t run;               // counters per lane; 0 = use the row kernels
    uint32_t group;             // whole chunks per work item
    uint32_t n_items;           // ceil(n_chunks / group)
};

enum FrPassKind : int { FR_PASS_FUSED = 0, FR_PASS_CTR = 1, FR_PASS_VERIFY = 2 };

// Rows of a chunk of `bytes` bytes: rows are aligned to the counter and block j sits at counter j + 2.
static inline uint32_t fr_rows_of(size_t bytes)
{
    return (uint32_t)(((bytes + 15) / 16 + 2 + FR_PLAN_ROW_BLOCKS - 1) / FR_PLAN_ROW_BLOCKS);
}

// Row-kernel geometry of a launch over n_chunks chunks of samples of `sample_bytes` bytes (a plain buffer is one
// sample).  Every warp that takes work pays one closing GF(2^128) product per chunk it touches, at least one; a
// warp's rows run one after the other.  So a launch of T rows on S SMs wants about sqrt(T / S) warps per SM: more
// warps shorten the row sequence of each, fewer warps mean fewer closings -- up to the 32 a CTA has, from about
// 64 MiB on.  (Fitted on B200: best rows per warp 3 / 4 / 6 / 9 / 13 at 1 / 2 / 4 / 8 / 16 MiB.)
static inline FrRowPlan fr_plan_rows(const FrPlanConfig& cfg, size_t sample_bytes, size_t n_chunks)
{
    FrRowPlan p;
    const size_t cps = (sample_bytes + cfg.chunk_bytes - 1) / cfg.chunk_bytes;
    const size_t first_len = sample_bytes < cfg.chunk_bytes ? sample_bytes : cfg.chunk_bytes;
    p.rows_full = fr_rows_of(first_len);
    p.rows_last = fr_rows_of(sample_bytes - (cps - 1) * cfg.chunk_bytes);
    p.rows_sample = (uint64_t)(cps - 1) * p.rows_full + p.rows_last;
    p.total_rows = (uint64_t)(n_chunks / cps) * p.rows_sample;
    const uint64_t sms = (uint64_t)cfg.num_sms, cap = sms * FR_WARPS;
    uint64_t slots;
    if (cfg.row_slots_override) {
        slots = cfg.row_slots_override;
    } else {
        const uint64_t per_sm = p.total_rows / sms;
        uint64_t wu = per_sm < 4 ? 1 : per_sm < 8 ? 2 : per_sm < 12 ? 4 : per_sm < 20 ? 8 : per_sm < 50 ? 12 : per_sm < 600 ? 16 : 24;
        if (wu > FR_WARPS) wu = FR_WARPS;
        slots = sms * wu;
    }
    if (slots > cap) slots = cap;
    if (slots > p.total_rows) slots = p.total_rows;
    if (slots < 1) slots = 1;
    p.n_slots = (uint32_t)slots;
    p.warps_used = (uint32_t)((slots + sms - 1) / sms);
    p.grid = (uint32_t)((slots + p.warps_used - 1) / p.warps_used);
    return p;
}

// Cost constants of the two layouts for one kind of pass, in SM clocks.
struct FrPackCosts {
    size_t row_clocks, seg_clocks, row_step_latency;      // row kernels: per row, per segment; latency of a row for a lone warp
    size_t fixed, step_latency;                           // packed rows: per row of 32 runs; latency per counter for a lone warp
    size_t step[14];                                      // packed rows: clocks per counter of a run, by run length (0 unused)
    size_t step_long;                                     // ... for longer runs
};

// Decides between the row kernels (`rows` is their plan) and the packed-row kernels, and in the latter case picks
// the run length and the work-item size.  Both are judged by the same kind of estimate: the shared-memory work of
// the busiest SM or the latency of the busiest warp, whichever is larger (plus a quarter of the other: between the
// two regimes both show).  For the fused passes a row kernel costs about 285 clocks per row plus 400 per segment;
// a packed row costs about 280 plus, per counter of its run, 258 clocks for runs up to 3 counters and more beyond (a
// lane's 16-byte loads and stores are 16 * run bytes apart, so longer runs touch more cache lines per request; runs
// whose byte stride is a power of two do worst: the lanes' pieces fall on the same few cache banks).  The two
// halves of the fused pass have constants of their own.
static inline FrPackPlan fr_plan_packed(const FrPlanConfig& cfg, int kind, size_t sample_bytes, size_t n_chunks,
                                        const FrRowPlan& rows)
{
    static const FrPackCosts costs[3] = {
        // fused passes: cipher + Horner step per counter, one general product per run
        {285, 400, 1000, 280, 2250, {0, 258, 257, 256, 289, 264, 281, 330, 396, 302, 304, 304, 327, 305}, 335},
        // counter mode only: no product, no reduction
        {218, 100, 900, 30, 2000, {0, 227, 227, 227, 245, 227, 240, 270, 330, 250, 252, 252, 270, 255}, 260},
        // verify only: no cipher (but counter 1), so the closing product weighs more and longer runs pay
        {85, 400, 300, 465, 700, {0, 65, 65, 65, 80, 65, 75, 85, 120, 86, 88, 88, 100, 90}, 95},
    };
    const FrPackPlan rows_kernels = {0, 0, 0};
    if (!cfg.pack_max_blocks || n_chunks == 0) return rows_kernels;
    const FrPackCosts& C = costs[kind];
    const size_t first_len = sample_bytes < cfg.chunk_bytes ? sample_bytes : cfg.chunk_bytes;
    const size_t counters = (first_len + 15) / 16 + 1;
    if (counters - 1 > cfg.pack_max_blocks) return rows_kernels;
    const size_t sms = (size_t)cfg.num_sms, warps = sms * FR_WARPS;
    if (!cfg.pack_run_override && counters > 32 && n_chunks * 8 < warps) return rows_kernels;   // a few long chains: rows, no search needed

    // row kernels: every slot closes one segment per chunk it touches
    const size_t pieces = (size_t)rows.n_slots + n_chunks;
    const size_t rows_per_slot = (size_t)((rows.total_rows + rows.n_slots - 1) / rows.n_slots);
    const size_t segs_per_slot = (pieces + rows.n_slots - 1) / rows.n_slots;
    const size_t row_thr = (size_t)((rows.total_rows + sms - 1) / sms) * C.row_clocks + (pieces + sms - 1) / sms * C.seg_clocks;
    const size_t row_lat = rows_per_slot * C.row_step_latency + segs_per_slot * 4000;
    const size_t row_cost = row_thr > row_lat ? row_thr : row_lat;

    size_t best_run = 0, best_group = 1, best_cost = ~(size_t)0;
    const size_t cand[] = {1, 2, 3, 4, 5, 6, 9, 10, 11, 13, counters <= 64 ? counters : 5};
    for (size_t run : cand) {
        if (cfg.pack_run_override) run = cfg.pack_run_override;
        if (run > counters) run = counters;
        const size_t slots = (counters + run - 1) / run;
        // slots and chunks are counted in 32 bits; a row may overshoot by 31, an item's first chunk index by its size
        if (n_chunks * slots >= ((size_t)1 << 32) - 2 * FR_PACK_MAX_ITEM_SLOTS) continue;
        const size_t per_row = C.fixed + run * (run < 14 ? C.step[run] : C.step_long);
        const size_t row_latency = 2500 + run * C.step_latency;       // one warp alone on its SM partition
        // a work item is `group` whole chunks.  Its last row is only partly filled, and an instruction costs the same
        // with idle lanes; on the other hand a launch with fewer items than warps leaves warps idle.  Try a range of
        // item sizes and count the rows each really takes.
        const size_t sizes[] = {1, 2, 3, 4, 5, 6, 8, 10, 12, 16, 24, 32, 48, 64, 96, 128, 256, 512,
                                32 / slots, 64 / slots, 128 / slots, 256 / slots, 512 / slots};
        for (size_t group : sizes) {
            if (cfg.pack_group_override) group = cfg.pack_group_override;
            if (group < 1 || group * slots > FR_PACK_MAX_ITEM_SLOTS) continue;
            if (group > n_chunks) group = n_chunks;
            const size_t rows_per_item = (group * slots + 31) / 32;
            const size_t items = (n_chunks + group - 1) / group;
            const size_t thr = (items * rows_per_item + sms - 1) / sms * per_row;
            const size_t lat = (items + warps - 1) / warps * rows_per_item * row_latency;
            const size_t cost = thr > lat ? thr + lat / 4 : lat + thr / 4;
            if (cost < best_cost) { best_cost = cost; best_run = run; best_group = group; }
        }
    }
    if (!best_run) return rows_kernels;
    if (!cfg.pack_run_override && best_cost >= row_cost) return rows_kernels;
    FrPackPlan p;
    p.run = (uint32_t)best_run;
    p.group = (uint32_t)best_group;
    p.n_items = (uint32_t)((n_chunks + best_group - 1) / best_group);
    return p;
}

// Stages of a pipelined transfer of `len` bytes in whole multiples of `unit` (a chunk, or a sample in a batch of
// samples): three quarters of what is left each time, never less than about 2 MiB, no sliver at the end.  Host to
// device the list is walked as it is (the last, smallest stage's kernel is the exposed one); device to host
// backwards.  Returns the number of stages (at most FR_MAX_STAGES).
static inline size_t fr_plan_stages(const FrPlanConfig& cfg, size_t len, size_t unit, size_t out[FR_MAX_STAGES])
{
    const size_t cb = unit;
    const size_t floor_bytes = (size_t)2 << 20;
    const size_t min_stage = cb >= floor_bytes ? cb : (floor_bytes + cb - 1) / cb * cb;
    size_t off = 0, count = 0;
    while (off < len) {
        const size_t remaining = len - off;
        size_t n;
        if (cfg.stage_bytes_override) {
            n = (cfg.stage_bytes_override + cb - 1) / cb * cb;
        } else {
            n = (remaining / 4 * 3) / cb * cb;
            if (n < min_stage) n = min_stage;
            if (remaining < n + min_stage / 2) n = remaining;      // do not leave a sliver behind
        }
        if (n > remaining || count == FR_MAX_STAGES - 1) n = remaining;
        out[count++] = n;
        off += n;
    }
    return count;
}
