// fastrack_plan.h -- host-side planning of a launch and of a pipelined transfer: plain C++ without CUDA, so that
// the CPU-only tests can include it and check its invariants (tests/host_logic).  Three decisions are made here:
//   fr_plan_segments: how the row kernels cut chunks into segments (one warp per segment);
//   fr_plan_packed:   whether a launch takes the packed-row kernels instead, and with which run length and
//                     work-item size;
//   fr_plan_stages:   how a pipelined host<->device transfer is cut into stages.
// All costs are estimates in SM clocks with constants fitted to measurements on B200.
#pragma once
#include <stddef.h>
#include <stdint.h>

#define FR_THREADS 1024
#define FR_WARPS (FR_THREADS / 32)
#define FR_MAX_STAGES 96          // most stages a pipelined call is cut into
#define FR_PLAN_ROW_BLOCKS 32     // blocks per row of the row kernels (one per lane)
#define FR_PACK_MAX_BLOCKS 4096   // chunks of more blocks than this never take the packed-row kernels
#define FR_PACK_MAX_ITEM_SLOTS 1024   // most runs (lanes' worth of work) in one packed work item

struct FrPlanConfig {
    int num_sms;
    size_t chunk_bytes;
    uint32_t seg_rows_override;     // 0 = automatic (FASTRACK_SEG_ROWS, for experiments)
    uint32_t pack_max_blocks;       // chunks of at most this many blocks may take the packed-row kernels (FASTRACK_PACK_MAX_BLOCKS; 0 = never)
    uint32_t pack_run_override;     // 0 = automatic; else packed rows with this run length wherever they apply (FASTRACK_PACK_RUN, tests)
    uint32_t pack_group_override;   // 0 = automatic; else this many chunks per packed work item (FASTRACK_PACK_GROUP, tests)
    size_t stage_bytes_override;    // 0 = automatic (FASTRACK_STAGE_BYTES, for experiments)
};

struct FrSegPlan {
    uint32_t seg_rows;          // rows per segment
    uint32_t segs_per_chunk;    // segments of a full-size chunk
    uint32_t n_items;           // segs_per_chunk * n_chunks
};

struct FrPackPlan {
    uint32_t run;               // counters per lane; 0 = use the row kernels
    uint32_t group;             // whole chunks per work item
    uint32_t n_items;           // ceil(n_chunks / group)
};

enum FrPassKind : int { FR_PASS_FUSED = 0, FR_PASS_CTR = 1, FR_PASS_VERIFY = 2 };

// Segment geometry of a launch over n_chunks chunks of samples of `sample_bytes` bytes (a plain buffer is one
// sample): rows are aligned to the counter (block j sits at counter j + 2), segments longer than four rows are
// whole multiples of 8 rows so that they start on a 256-counter group.
static inline FrSegPlan fr_plan_segments(const FrPlanConfig& cfg, size_t sample_bytes, size_t n_chunks)
{
    const size_t first_len = sample_bytes < cfg.chunk_bytes ? sample_bytes : cfg.chunk_bytes;
    const size_t rows_ref = ((first_len + 15) / 16 + 2 + FR_PLAN_ROW_BLOCKS - 1) / FR_PLAN_ROW_BLOCKS;
    const size_t warps = (size_t)cfg.num_sms * FR_WARPS;
    // Segments are dealt round-robin to the resident warps.  Two things bound a launch: the latency of the
    // busiest warp (about 1000 cycles per row when few warps run, plus about 4000 per segment for the closing
    // GF(2^128) product, the atomics and the tag), and the shared-memory work of the busiest SM (about 270
    // wavefront-cycles per row plus about 300 per segment).  Try short segments (2 or 4 rows, for small buffers)
    // and 1..8 segments per warp in whole 8-row groups, and keep the split with the smaller bound.
    size_t seg_rows = 8, spc = (rows_ref + 7) / 8;
    if (cfg.seg_rows_override) {
        seg_rows = cfg.seg_rows_override;
        spc = (rows_ref + seg_rows - 1) / seg_rows;
    } else {
        size_t best_cost = ~(size_t)0;
        for (int cand = 0; cand < 10; cand++) {
            size_t rows;
            if (cand < 2) {
                rows = cand == 0 ? 2 : 4;
            } else {
                size_t want = (size_t)(cand - 1) * warps / n_chunks;
                if (want < 1) want = 1;
                rows = ((rows_ref + want - 1) / want + 7) / 8 * 8;
                if (rows > 1024) rows = 1024;
            }
            const size_t per_chunk = (rows_ref + rows - 1) / rows;
            const size_t items = per_chunk * n_chunks;
            const size_t waves = (items + warps - 1) / warps;
            const size_t per_sm = (items + (size_t)cfg.num_sms - 1) / (size_t)cfg.num_sms;
            const size_t latency = waves * (rows * 1000 + 4000);
            const size_t throughput = per_sm * (rows * 270 + 300);
            const size_t cost = latency > throughput ? latency : throughput;
            if (cost < best_cost) { best_cost = cost; seg_rows = rows; spc = per_chunk; }
        }
    }
    while (spc * n_chunks >= ((size_t)1 << 31)) { seg_rows *= 2; spc = (rows_ref + seg_rows - 1) / seg_rows; }
    FrSegPlan p;
    p.seg_rows = (uint32_t)seg_rows;
    p.segs_per_chunk = (uint32_t)spc;
    p.n_items = (uint32_t)(spc * n_chunks);
    return p;
}

// Cost constants of the two layouts for one kind of pass, in SM clocks.
struct FrPackCosts {
    size_t row_clocks, seg_clocks, row_step_latency;      // row kernels: per row, per segment; latency of a row for a lone warp
    size_t fixed, step_latency;                           // packed rows: per row of 32 runs; latency per counter for a lone warp
    size_t step[14];                                      // packed rows: clocks per counter of a run, by run length (0 unused)
    size_t step_long;                                     // ... for longer runs
};

// Decides between the row kernels (`seg` is their plan) and the packed-row kernels, and in the latter case picks
// the run length and the work-item size.  Both are judged by the same kind of estimate: the shared-memory work of
// the busiest SM or the latency of the busiest warp, whichever is larger (plus a quarter of the other: between the
// two regimes both show).  For the fused passes a row kernel costs about 285 clocks per row plus 400 per segment;
// a packed row costs about 280 plus, per counter of its run, 258 clocks for runs up to 3 counters and more beyond (a
// lane's 16-byte loads and stores are 16 * run bytes apart, so longer runs touch more cache lines per request; runs
// whose byte stride is a power of two do worst: the lanes' pieces fall on the same few cache banks).  The two
// halves of the fused pass have constants of their own.
static inline FrPackPlan fr_plan_packed(const FrPlanConfig& cfg, int kind, size_t sample_bytes, size_t n_chunks,
                                        const FrSegPlan& seg)
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

    const size_t rows_ref = (counters + 1 + FR_PLAN_ROW_BLOCKS - 1) / FR_PLAN_ROW_BLOCKS;
    const size_t waves = ((size_t)seg.n_items + warps - 1) / warps;
    const size_t row_thr = (n_chunks * rows_ref + sms - 1) / sms * C.row_clocks + ((size_t)seg.n_items + sms - 1) / sms * C.seg_clocks;
    const size_t row_lat = waves * ((size_t)seg.seg_rows * C.row_step_latency + 4000);
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
