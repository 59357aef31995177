// ctcsd_draft_logits: draft-head projection, per-slot log-softmax and per-slot top-k.
#include "gemv_stream.cuh"
#include "lm_head_tc.cuh"

using namespace ctcsd;

namespace {

int draft_logits_impl(ctcsd_handle* hh, void* stream, int M, const void* x, int x_row_count, const int* x_rows,
                      const void* Wd, const int* row_seq, const float* blank_bias,
                      int* out_topk_id, float* out_topk_lp, float* out_lse, float* out_logits_dbg) {
    if (!hh || !x || !Wd || !out_topk_id || !out_topk_lp || !out_lse) return CTCSD_ERR_INVALID_ARG;
    Handle* h = &hh->h;
    const ctcsd_config& c = h->cfg;
    if (M < 1 || M > c.max_draft_rows) return CTCSD_ERR_INVALID_ARG;
    if (x_rows && x_row_count < 1) return CTCSD_ERR_INVALID_ARG;
    if (!row_seq && blank_bias && M > c.B) return CTCSD_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(Wd)) & 15) return CTCSD_ERR_INVALID_ARG;

    // more than 8 rows: the tensor-core weight stream reads the weights once for up to 128 rows
    // (it reads x as a dense tile, so a row map takes the weight-streaming passes below instead)
    if (!x_rows && draft_head_tc_supported(h, M)) {
        int rc = launch_draft_head_tc(h, static_cast<cudaStream_t>(stream), M, x, Wd, row_seq, blank_bias,
                                      out_topk_id, out_topk_lp, out_lse, out_logits_dbg);
        if (rc != CTCSD_ERR_UNSUPPORTED) return rc;
    }
    GemvParams p = {};
    p.x = x;
    p.x_rows = x_rows;
    p.x_row_count = x_rows ? x_row_count : M;
    p.W = Wd;
    p.row_seq = row_seq;
    p.blank_bias = blank_bias;
    p.m0 = 0;
    p.mcount = 0;
    p.H = c.H;
    p.slots = c.T;
    p.rows_per_slot = c.V + 1;
    p.grid = 0;
    p.part = nullptr;
    p.part_slot = nullptr;
    p.counter = nullptr;
    p.mode = 0;
    p.k = c.k;
    p.out_topk_id = out_topk_id;
    p.out_topk_lp = out_topk_lp;
    p.out_lse = out_lse;
    p.out_argmax = nullptr;
    p.logits_dbg = out_logits_dbg;
    p.sn.noise = nullptr; p.sn.depth = nullptr; p.sn.max_nodes = 1; p.sn.rows_per_seq = 1; p.sn.inv_temp = 1.f;
    p.pf_ptr = h->l2_hint_ptr;
    p.pf_bytes = h->l2_hint_bytes;
    return launch_gemv_stream(h, static_cast<cudaStream_t>(stream), c.dtype, M, p);
}

}  // namespace

extern "C" int ctcsd_draft_logits(ctcsd_handle* hh, void* stream, int M, const void* x, const void* Wd,
                                  const int* row_seq, const float* blank_bias,
                                  int* out_topk_id, float* out_topk_lp, float* out_lse, float* out_logits_dbg) {
    return draft_logits_impl(hh, stream, M, x, M, nullptr, Wd, row_seq, blank_bias,
                             out_topk_id, out_topk_lp, out_lse, out_logits_dbg);
}

extern "C" int ctcsd_draft_logits_rows(ctcsd_handle* hh, void* stream, int M, const void* x, int x_row_count,
                                       const int* x_rows, const void* Wd, const int* row_seq, const float* blank_bias,
                                       int* out_topk_id, float* out_topk_lp, float* out_lse, float* out_logits_dbg) {
    if (!x_rows) return CTCSD_ERR_INVALID_ARG;
    return draft_logits_impl(hh, stream, M, x, x_row_count, x_rows, Wd, row_seq, blank_bias,
                             out_topk_id, out_topk_lp, out_lse, out_logits_dbg);
}
