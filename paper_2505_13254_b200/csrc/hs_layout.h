// Host-side geometry shared by the launchers: limits, workspace regions, row chunking.
#pragma once

#include <stddef.h>
#include <stdint.h>

#include "../../include/heterospec.h"

#define HS_MAX_BATCH 4096
#define HS_MAX_ROWS 16384

// Workspace head: self-resetting arrival counters (ints), zeroed once at hs_create.
#define HS_COUNTER_BYTES (256 * 1024)
#define HS_CNT_QUANT_ROW 0        // [HS_MAX_ROWS]  chunks of a draft row that have finished
#define HS_CNT_PRUNE_FLAG 16384   // [HS_MAX_BATCH] fused tree stage + pruning: kept count + 1 of a sequence, once known
#define HS_CNT_ACC_ROW 20480      // [2*HS_MAX_ROWS] chunks of a target / draft row
#define HS_CNT_ACC_SEQ 53248      // [HS_MAX_BATCH] merged target rows of a sequence
#define HS_CNT_ERROR 61440        // [1] sticky device error word (bounded wait expired)
#define HS_CNT_PRUNE_DONE 61504   // [1] fused tree stage + pruning: CTAs that have read the counts ahead of theirs

// Vocabulary pass: a CTA of HS_ROW_THREADS threads keeps HS_ROW_VPT 16-byte vectors per thread in
// registers, so one CTA covers at most 256*8*8 = 16384 bf16 or 8192 f32 logits of a row.
#define HS_ROW_THREADS 256
#define HS_ROW_VPT 8

static inline int hs_vec_elems(hs_dtype dt) { return dt == HS_BF16 ? 8 : 4; }
static inline int hs_row_chunks(int32_t vocab, hs_dtype dt) {
    int cap = HS_ROW_THREADS * HS_ROW_VPT * hs_vec_elems(dt);
    return (vocab + cap - 1) / cap;
}

// per (row, chunk) partial of the quantify pass: {max, sum e, sum e*x, pad} + HS_MAX_TOPK keys
#define HS_ROW_PARTIAL_BYTES (16 + HS_MAX_TOPK * 8)
// per (row, chunk) partial of the accept pass: {argmax key (8 bytes), max, sum e}
#define HS_ACC_PARTIAL_BYTES 16

