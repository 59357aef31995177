// Weight-streaming matrix-vector kernel for small row counts (CUDA cores).
//
// Used where the projection is bound by HBM bandwidth: every weight row is read exactly
// once, by a bulk copy into a deep shared-memory ring, and multiplied with up to four
// activation rows that sit in shared memory.  The logits are never written out (unless the caller asks for the
// debug dump); each CTA folds them into a running (max, sum of exp, best-8) state per
// (activation row, slot), and the last CTA to finish merges all partial states into the
// per-slot log-sum-exp and top-k (draft head) or the arg-max (LM head).
#pragma once

#include "common.cuh"

namespace ctcsd {

struct GemvParams {
    const void* x;            // [x_row_count,H]
    const int* x_rows;        // [M] or null: activation row m is x[x_rows[m]] (null: x[m])
    int x_row_count;          // rows of x (bound for x_rows)
    const void* W;            // [slots, rows_per_slot, H]
    const int* row_seq;       // [M] or null
    const float* blank_bias;  // [B] or null; added to the last row of every slot
    int m0;                   // first activation row of this pass
    int mcount;               // activation rows in this pass (<= MROWS)
    int H;
    int slots;
    int rows_per_slot;
    int grid;                 // CTAs launched (also the stride of the partial array)
    DraftPartial* part;       // [MROWS][grid][2]
    int* part_slot;           // [grid][2] slot id of each partial (-1 = unused)
    unsigned* counter;        // ticket counter, zero on entry, zero again on exit
    int mode;                 // 0: top-k + lse outputs, 1: arg-max output, 2: the products themselves (to logits_dbg)
    int k;
    int* out_topk_id;         // mode 0: [M,slots,k]
    float* out_topk_lp;       // mode 0: [M,slots,k]
    float* out_lse;           // mode 0: [M,slots]
    int* out_argmax;          // mode 1: [M]
    float* logits_dbg;        // null or [M,slots,rows_per_slot]
    int* status;              // device status word
    SampleNoise sn;           // mode 1: noise added to the scaled logit before the arg-max (null: none)
    const void* pf_ptr;       // optional: range the CTAs ask L2 to fetch once their own stream is issued
    unsigned long long pf_bytes;
};

int launch_gemv_stream(Handle* h, cudaStream_t stream, int dtype, int M, GemvParams p);

}  // namespace ctcsd
