// plan_check.cpp -- TEST INFRASTRUCTURE: the library's host-side planners (paper_2410_15240_b200/csrc/fastrack_plan.h,
// plain C++) behind a C interface, so that the CPU-only tests can check their invariants over many shapes.
#include "../../paper_2410_15240_b200/csrc/fastrack_plan.h"

extern "C" {

static FrPlanConfig make(int num_sms, size_t chunk_bytes, uint32_t row_slots, uint32_t pack_max, uint32_t run, uint32_t group,
                         size_t stage_bytes, uint32_t fold_mode = 0)
{
    FrPlanConfig c;
    c.fold_tail_mode = fold_mode;
    c.num_sms = num_sms; c.chunk_bytes = chunk_bytes; c.row_slots_override = row_slots; c.pack_max_blocks = pack_max;
    c.pack_run_override = run; c.pack_group_override = group; c.stage_bytes_override = stage_bytes;
    return c;
}

// out[0..2] = grid, warps_used, n_slots of the row kernels; out[3..5] = run, lanes per chunk, n_items of the packed rows;
// out[6..9] = rows_full, rows_last, rows_sample, total_rows; out[10] = 1 if the tails are folded.
// kind 0 (the fused passes) may fold tails; fold_mode is the option's value (0 automatic, 1 never, 2 wherever possible).
void plan_launch(int num_sms, size_t chunk_bytes, uint32_t row_slots, uint32_t pack_max, uint32_t run, uint32_t group, int kind,
                 size_t sample_bytes, size_t n_chunks, uint32_t fold_mode, uint64_t out[11])
{
    const FrPlanConfig c = make(num_sms, chunk_bytes, row_slots, pack_max, run, group, 0, fold_mode);
    const FrRowPlan r = fr_plan_rows(c, sample_bytes, n_chunks, kind == 0);
    const FrPackPlan p = fr_plan_packed(c, kind, sample_bytes, n_chunks, r);
    out[0] = r.grid; out[1] = r.warps_used; out[2] = r.n_slots;
    const size_t first_len = sample_bytes < chunk_bytes ? sample_bytes : chunk_bytes;
    out[3] = p.run; out[4] = p.run ? ((first_len + 15) / 16 + p.run) / p.run : 0; out[5] = p.n_items;
    out[6] = r.rows_full; out[7] = r.rows_last; out[8] = r.rows_sample; out[9] = r.total_rows; out[10] = r.fold_tail;
}

size_t plan_stages(size_t chunk_bytes, size_t stage_bytes, size_t len, size_t unit, size_t* out)
{
    const FrPlanConfig c = make(148, chunk_bytes, 0, FR_PACK_MAX_BLOCKS, 0, 0, stage_bytes);
    return fr_plan_stages(c, len, unit, out);
}

int plan_max_stages(void) { return FR_MAX_STAGES; }

}
