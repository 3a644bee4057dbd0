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

struct FrPlanConfig {
    int num_sms;
    size_t chunk_bytes;
    uint32_t row_slots_override;    // 0 = automatic; else the row kernels spread a launch over this many warps (tests, tuning)
    uint32_t pack_max_blocks;       // chunks of at most this many blocks may take the packed-row kernels (0 = never)
    uint32_t pack_run_override;     // 0 = automatic; else packed rows with this run length wherever they apply (tests)
    uint32_t pack_group_override;   // 0 = automatic; else this many chunks per packed work item (tests)
    size_t stage_bytes_override;    // 0 = automatic; else the stage size of pipelined transfers (experiments)
    uint32_t fold_tail_mode;        // row kernels, fused passes: 0 = fold the tails of chunks where it pays, 1 = never, 2 = wherever a chunk has one (tests)
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
    uint32_t fold_tail;         // 1: the row counts above are those of folded tails (see fr_rows_of)
};

struct FrPackPlan {
    uint32_t run;               // most counters per lane; 0 = use the row kernels.  A chunk has ceil(counters / run) lanes
    uint32_t n_items;           // warps that take work; item j covers chunks j * n_chunks / n_items .. (j + 1) * n_chunks / n_items - 1
};

enum FrPassKind : int { FR_PASS_FUSED = 0, FR_PASS_CTR = 1, FR_PASS_VERIFY = 2 };

// Rows of a chunk of `bytes` bytes: rows are aligned to the counter and block j sits at counter j + 2, so a chunk of
// a whole number of rows' worth of blocks (or one block less) ends in a row of two counters (or one).  With `fold`
// that row does not exist: the kernel works on those counters in a pass that it makes anyway for the tag masks of
// up to ten chunks at a time (fr_prework_lane in the device header).
static inline bool fr_tail_folds(size_t bytes)
{
    const size_t blocks = (bytes + 15) / 16, in_last_row = (blocks + 2) % FR_PLAN_ROW_BLOCKS;
    return blocks >= 31 && (in_last_row == 1 || in_last_row == 2);
}

static inline uint32_t fr_rows_of(size_t bytes, bool fold)
{
    const uint32_t rows = (uint32_t)(((bytes + 15) / 16 + 2 + FR_PLAN_ROW_BLOCKS - 1) / FR_PLAN_ROW_BLOCKS);
    return fold && fr_tail_folds(bytes) ? rows - 1 : rows;
}

// Row-kernel geometry of a launch over n_chunks chunks of samples of `sample_bytes` bytes (a plain buffer is one
// sample).  Every warp that takes work pays one closing GF(2^128) product per chunk it touches, at least one; a
// warp's rows run one after the other.  (Fitted on B200; see the comment at the choice below.)
// may_fold: the pass is one that can fold tails (decrypt + verify, encrypt + tag); whether it does is decided here.
static inline FrRowPlan fr_plan_rows(const FrPlanConfig& cfg, size_t sample_bytes, size_t n_chunks, bool may_fold = false)
{
    FrRowPlan p;
    const size_t cps = (sample_bytes + cfg.chunk_bytes - 1) / cfg.chunk_bytes;
    const size_t first_len = sample_bytes < cfg.chunk_bytes ? sample_bytes : cfg.chunk_bytes;
    const size_t last_len = sample_bytes - (cps - 1) * cfg.chunk_bytes;
    const uint64_t sms = (uint64_t)cfg.num_sms, cap = sms * FR_WARPS;
    auto geometry = [&](bool fold) {
        p.fold_tail = fold ? 1u : 0u;
        p.rows_full = fr_rows_of(first_len, fold);
        p.rows_last = fr_rows_of(last_len, fold);
        p.rows_sample = (uint64_t)(cps - 1) * p.rows_full + p.rows_last;
        p.total_rows = (uint64_t)(n_chunks / cps) * p.rows_sample;
    };
    auto slots_for = [&](uint64_t total_rows) {
        uint64_t slots;
        if (cfg.row_slots_override) {
            slots = cfg.row_slots_override;
        } else {
            // Small launches are bound by the latency of a warp's row sequence (a row takes a lone warp about as long as it
            // takes sixteen warps to do one each), so they want at most two rows per warp; from four warps per SM on only
            // whole numbers of warps per quarter of an SM (each quarter has its own scheduler).  Large launches are bound by
            // the lookup pipe, which sixteen warps saturate; beyond that, more warps hide a little more latency.
            const uint64_t per_sm = (total_rows + sms - 1) / sms;
            uint64_t wu = per_sm < 600 ? 16 : 24;
            if (per_sm <= 32) {
                wu = (per_sm + 1) / 2;
                if (wu > 4) wu = (wu + 3) / 4 * 4;
            }
            if (wu > FR_WARPS) wu = FR_WARPS;
            slots = sms * wu;
        }
        if (slots > cap) slots = cap;
        if (slots > total_rows) slots = total_rows;
        if (slots < 1) slots = 1;
        return slots;
    };
    geometry(false);
    // Folding pays where a warp's range holds a chunk start or several, so that the extra pass serves them all: measured
    // at 4.6 chunks per warp 4 % with 16 KiB chunks, 8 % with 8 KiB, 15 % with 4 KiB (more than the row saved, since
    // row 0 of a chunk then no longer runs the cipher a second time for the tag mask), still 1 to 2 % at one chunk per
    // warp.  Below that most warps would make a pass for a single chunk: a gain of under 1 % down to half a chunk per
    // warp where 24 warps per SM hide the pass, a loss of 1 to 3 % with 16.
    const uint64_t plain_slots = slots_for(p.total_rows);
    if (may_fold && cfg.fold_tail_mode != 1 && (fr_tail_folds(first_len) || fr_tail_folds(last_len)) &&
        (cfg.fold_tail_mode == 2 || n_chunks >= plain_slots || (plain_slots >= sms * 24 && 2 * n_chunks >= plain_slots)))
        geometry(true);
    const uint64_t slots = slots_for(p.total_rows);
    p.n_slots = (uint32_t)slots;
    p.warps_used = (uint32_t)((slots + sms - 1) / sms);
    p.grid = (uint32_t)((slots + p.warps_used - 1) / p.warps_used);
    return p;
}

// Cost constants of the two layouts for one kind of pass, in SM clocks.
struct FrPackCosts {
    size_t row_clocks, seg_clocks, row_step_latency;      // row kernels: per row, per segment; latency of a row for a lone warp
    size_t close, step, step_latency;                     // packed rows, per row of 32 lanes: the closing; one counter step; its latency for a lone warp
    size_t row_fixed, pack_fixed;                         // per launch, beyond what scales with the work: rows (closing products of all
                                                          // warps at once, the hand-over between CTAs), packed rows
    size_t seg_folded;                                    // row kernels with folded tails, per segment (row 0 no longer runs the cipher
                                                          // a second time for the tag mask; that comes from the prework passes)
};

// Decides between the row kernels (`rows` is their plan) and the packed-row kernels, and in the latter case picks
// how many lanes share a chunk and how many warps take work.  Both layouts are judged by the same kind of
// estimate: the shared-memory work of the busiest SM or the latency of the busiest warp, whichever is larger
// (plus a quarter of the other: between the two regimes both show).
// Packed rows: a chunk of B blocks on L lanes takes S = 1 + ceil(B / L) steps (one for counter 1, in which only
// one lane of the chunk works); a warp that holds n chunks walks ceil(n * L / 32) rows of S steps each plus one
// closing per row.  Few lanes per chunk mean long runs and few closings, but coarse rows (a warp's last row is
// partly empty) and short contiguous pieces per memory request (16 * L bytes: an odd number of blocks does not
// fill whole 32-byte sectors, which costs extra cycles on the memory pipe that bounds the kernel); lane counts
// that do not divide B leave lanes idle in the last step.  All of that is counted below; the constants are fitted
// to measurements on B200.
static inline FrPackPlan fr_plan_packed(const FrPlanConfig& cfg, int kind, size_t sample_bytes, size_t n_chunks,
                                        const FrRowPlan& rows)
{
    static const FrPackCosts costs[3] = {
        {279, 400, 1000, 300, 279, 2250, 10800, 4900, 260},     // fused passes: cipher + Horner step per counter, one general product per lane
        {218, 100, 900, 30, 227, 2000, 0, 0, 0},              // counter mode only: no product, no reduction
        {85, 400, 300, 465, 65, 700, 0, 0, 0},                // verify only: no cipher (but counter 1), so the closing weighs more
    };
    const FrPackPlan rows_kernels = {0, 0};
    if (!cfg.pack_max_blocks || n_chunks == 0) return rows_kernels;
    const FrPackCosts& C = costs[kind];
    const size_t first_len = sample_bytes < cfg.chunk_bytes ? sample_bytes : cfg.chunk_bytes;
    const size_t counters = (first_len + 15) / 16 + 1;
    if (counters - 1 > cfg.pack_max_blocks) return rows_kernels;
    const size_t sms = (size_t)cfg.num_sms, warps = sms * FR_WARPS;
    if (!cfg.pack_run_override && counters > 32 && n_chunks * 16 < warps) return rows_kernels;  // a few long chains: rows, no search needed

    // row kernels: every slot closes one segment per chunk it touches
    const size_t pieces = (size_t)rows.n_slots + n_chunks;
    const size_t rows_per_slot = (size_t)((rows.total_rows + rows.n_slots - 1) / rows.n_slots);
    const size_t segs_per_slot = (pieces + rows.n_slots - 1) / rows.n_slots;
    // (folded tails: one more pass of a cipher block and a product per ten chunk starts, at least one per warp that sees a start)
    size_t pre_passes = rows.fold_tail ? n_chunks / 10 + rows.n_slots : 0;
    if (pre_passes > n_chunks) pre_passes = n_chunks;
    const size_t row_thr = (size_t)((rows.total_rows + sms - 1) / sms) * C.row_clocks +
                           (pieces + sms - 1) / sms * (rows.fold_tail ? C.seg_folded : C.seg_clocks) +
                           (pre_passes + sms - 1) / sms * (C.step + C.close);
    const size_t row_lat = rows_per_slot * C.row_step_latency + segs_per_slot * 4000;
    const size_t row_cost = (row_thr > row_lat ? row_thr : row_lat) + C.row_fixed;

    size_t best_run = 0, best_items = 1, best_cost = ~(size_t)0;
    const size_t max_lanes = counters < 64 ? counters : 64;
    for (size_t lanes = 1; lanes <= max_lanes + 1; lanes++) {
        size_t run = lanes <= max_lanes ? (counters + lanes - 1) / lanes : 1;     // (last round: one counter per lane)
        if (cfg.pack_run_override) run = cfg.pack_run_override < counters ? cfg.pack_run_override : counters;
        const size_t l = (counters + run - 1) / run;                               // the lane count this run length gives
        if (!cfg.pack_run_override && lanes <= max_lanes && l != lanes) continue;  // not reachable as ceil(counters / run)
        const size_t steps = 1 + (counters - 1 + l - 1) / l;
        // slots and chunks are counted in 32 bits; a row may overshoot by 31 slots
        if (n_chunks * l >= ((size_t)1 << 32) - 64) continue;
        // memory pipe: a chunk's lanes touch 16 * l contiguous bytes per step, starting on a multiple of that; per row of
        // 32 lanes that is 32 / l such pieces against the 16 sectors of a dense request
        const size_t row_sectors2 = (64 * ((l + 1) / 2) + l - 1) / l;                              // twice the sectors per row
        const size_t extra = row_sectors2 > 32 ? (row_sectors2 - 32) * 5 / 4 : 0;                  // about 2.5 clocks per extra sector, load and store
        const size_t per_row = C.close + steps * (C.step + extra);
        const size_t row_latency = 2500 + steps * C.step_latency;       // one warp alone on its SM partition
        // a work item is one warp's contiguous range of whole chunks, and every warp takes one (fewer warps with longer
        // ranges would fill their last rows better, but measured slower)
        for (size_t div = 1; div <= 1; div *= 2) {
            size_t items = warps / div;
            if (cfg.pack_group_override) items = (n_chunks + cfg.pack_group_override - 1) / cfg.pack_group_override;
            if (items > n_chunks) items = n_chunks;
            if (items < 1) items = 1;
            const size_t most = (n_chunks + items - 1) / items;                    // chunks of the longest item
            const size_t rows_most = (most * l + 31) / 32;
            const size_t per_sm = (items + sms - 1) / sms;                          // warps of the busiest SM
            const size_t thr = per_sm * rows_most * per_row;
            const size_t lat = rows_most * row_latency;
            const size_t cost = (thr > lat ? thr + lat / 4 : lat + thr / 4) + C.pack_fixed;
            if (cost < best_cost) { best_cost = cost; best_run = run; best_items = items; }
        }
        if (cfg.pack_run_override) break;
    }
    if (!best_run) return rows_kernels;
    if (!cfg.pack_run_override && best_cost >= row_cost) return rows_kernels;
    FrPackPlan p;
    p.run = (uint32_t)best_run;
    p.n_items = (uint32_t)best_items;
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
