// Tensor-core (tcgen05 / TMEM) LM head with fused row arg-max.
#pragma once

#include "common.cuh"
#include "accept.cuh"

namespace ctcsd {

// True when the handle's shape and dtype are served by the tensor-core kernel.
bool lm_head_tc_supported(const Handle* h);

// y = hn . Wl^T on the 5th-generation tensor cores with the row arg-max folded into the
// epilogue; the CTA that finishes last decodes the arg-max and runs the greedy acceptance walk
// `acc` over it.  Returns CTCSD_ERR_UNSUPPORTED when the shape is not covered.
int launch_lm_head_tc(Handle* h, cudaStream_t stream, int M, const void* hn, const void* Wl,
                      int* out_argmax, float* out_logits_dbg, const AcceptParams& acc, const SampleNoise& sn);

// Draft head on the tensor cores for more than 8 activation rows: the same weight-stream kernel
// with a per-row online (max, sum of exp, best-8) epilogue per vocabulary tile and a merge
// kernel over the tiles of every slot.
bool draft_head_tc_supported(const Handle* h, int M);
int draft_tc_tile_rows(int classes);
// Each vocabulary tile of the tensor-core draft head leaves this many partial states per row
// (its epilogue warps split the tile's columns).
constexpr int kDraftColSplit = 4;
int launch_draft_head_tc(Handle* h, cudaStream_t stream, int M, const void* x, const void* Wd, const int* row_seq,
                         const float* blank_bias, int* out_topk_id, float* out_topk_lp, float* out_lse,
                         float* out_logits_dbg);

}  // namespace ctcsd
