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

// What the kernel does to the activation rows while it loads them into shared memory (every CTA
// repeats it on its own copy: a few rows, hidden behind the first weight copies already in flight).
struct ActOp {
    int op;               // 0: x as it is; 1: RMSNorm(x) * gain; 2: RMSNorm(x + add) * gain; 3: SiLU(gate) * up
    float eps;            // ops 1, 2
    const float* gain;    // ops 1, 2: [H]
    const float* add;     // op 2: [M,H] float32, added to activation row m before the norm
    float* sum_out;       // op 2: [M,H] float32 or null: x + add, written by the first CTA
    const float* gu;      // op 3: [M,2H] float32, gate then up (x is not read)
    const int* n_new;     // op 1: row m = b * R + j is all zero when j >= n_new[b] (null: every row is live)
    int R;
};

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
    int mode;                 // 0: top-k + lse outputs, 1: arg-max output, 2: the products themselves (to logits_dbg and/or plain_out_t)
    int k;
    int* out_topk_id;         // mode 0: [M,slots,k]
    float* out_topk_lp;       // mode 0: [M,slots,k]
    float* out_lse;           // mode 0: [M,slots]
    int* out_argmax;          // mode 1: [M]
    float* logits_dbg;        // null or [M,slots,rows_per_slot]
    ActOp act;                // applied to the activation rows as they are loaded
    const float* plain_add;   // mode 2: null or [M,slots*rows_per_slot] float32 added to the products
    void* plain_out_t;        // mode 2: null or [M,slots*rows_per_slot] in the activation type: the (summed) products
    int* status;              // device status word
    SampleNoise sn;           // mode 1: noise added to the scaled logit before the arg-max (null: none)
    const void* pf_ptr;       // optional: range the CTAs ask L2 to fetch once their own stream is issued
    unsigned long long pf_bytes;
};

int launch_gemv_stream(Handle* h, cudaStream_t stream, int dtype, int M, GemvParams p);

}  // namespace ctcsd
