// ctcsd_verify_accept: LM head with row arg-max at every tree node, then the greedy walk
// down the token tree.
#include "gemv_stream.cuh"
#include "lm_head_tc.cuh"
#include "accept.cuh"

namespace ctcsd {
namespace {

// One warp per sequence (used when the arg-max comes from the CUDA-core path).
__global__ void __launch_bounds__(32) greedy_accept_kernel(AcceptParams p) {
    __shared__ int scratch[kAcceptScratchInts];
    accept_warp(p, blockIdx.x, threadIdx.x, scratch);
}

}  // namespace
}  // namespace ctcsd

using namespace ctcsd;

static int verify_accept_common(ctcsd_handle* hh, void* stream, const void* hn, const void* Wl,
                                const int* node_tok, const int* parent, const int* kept, const int* nka,
                                const int* n_nodes, int* out_argmax, int* out_acc_len, int* out_acc_nodes,
                                int* out_acc_tok, int* out_next_tok, float* out_logits_dbg,
                                const float* noise = nullptr, const int* depth = nullptr, float inv_temp = 1.f) {
    Handle* h = &hh->h;
    const ctcsd_config& c = h->cfg;
    if ((reinterpret_cast<uintptr_t>(hn) | reinterpret_cast<uintptr_t>(Wl)) & 15) return CTCSD_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int M = c.B * c.max_nodes;

    AcceptParams a;
    a.node_tok = node_tok; a.parent = parent; a.n_nodes = n_nodes; a.argmax = out_argmax;
    a.B = c.B; a.T = c.T; a.max_nodes = c.max_nodes;
    a.acc_len = out_acc_len; a.acc_nodes = out_acc_nodes; a.acc_tok = out_acc_tok; a.next_tok = out_next_tok;
    a.kept = kept; a.nka = nka;
    a.status = status_ptr(h);
    SampleNoise sn;
    sn.noise = noise; sn.depth = depth; sn.max_nodes = c.max_nodes; sn.rows_per_seq = c.T + 1; sn.inv_temp = inv_temp;

    // tensor-core path: the acceptance walk runs in the tail of the LM-head kernel
    if (lm_head_tc_supported(h)) {
        int rc = launch_lm_head_tc(h, s, M, hn, Wl, out_argmax, out_logits_dbg, a, sn);
        if (rc != CTCSD_ERR_UNSUPPORTED) return rc;
    }
    GemvParams g = {};
    g.x = hn; g.x_rows = nullptr; g.x_row_count = M; g.W = Wl; g.row_seq = nullptr; g.blank_bias = nullptr;
    g.m0 = 0; g.mcount = 0; g.H = c.H; g.slots = 1; g.rows_per_slot = c.V; g.grid = 0;
    g.part = nullptr; g.part_slot = nullptr; g.counter = nullptr;
    g.mode = 1; g.k = 1;
    g.out_topk_id = nullptr; g.out_topk_lp = nullptr; g.out_lse = nullptr;
    g.out_argmax = out_argmax;
    g.logits_dbg = out_logits_dbg;
    g.sn = sn;
    g.pf_ptr = nullptr; g.pf_bytes = 0;
    int rc = launch_gemv_stream(h, s, c.dtype, M, g);
    if (rc != CTCSD_OK) return rc;
    greedy_accept_kernel<<<c.B, 32, 0, s>>>(a);
    CTCSD_LAUNCH_CHECK(h);
    return CTCSD_OK;
}

extern "C" int ctcsd_verify_accept(ctcsd_handle* hh, void* stream, const void* hn, const void* Wl,
                                   const int* node_tok, const int* parent, const int* n_nodes,
                                   int* out_argmax, int* out_acc_len, int* out_acc_nodes, int* out_acc_tok,
                                   int* out_next_tok, float* out_logits_dbg) {
    if (!hh || !hn || !Wl || !node_tok || !parent || !n_nodes || !out_argmax || !out_acc_len || !out_acc_nodes ||
        !out_acc_tok || !out_next_tok)
        return CTCSD_ERR_INVALID_ARG;
    return verify_accept_common(hh, stream, hn, Wl, node_tok, parent, nullptr, nullptr, n_nodes, out_argmax,
                                out_acc_len, out_acc_nodes, out_acc_tok, out_next_tok, out_logits_dbg);
}

extern "C" int ctcsd_verify_accept_raw(ctcsd_handle* hh, void* stream, const void* hn, const void* Wl,
                                       const int* node_tok, const int* kept, const int* nka, const int* n_nodes,
                                       int* out_argmax, int* out_acc_len, int* out_acc_nodes, int* out_acc_tok,
                                       int* out_next_tok, float* out_logits_dbg) {
    if (!hh || !hn || !Wl || !node_tok || !kept || !nka || !n_nodes || !out_argmax || !out_acc_len || !out_acc_nodes ||
        !out_acc_tok || !out_next_tok)
        return CTCSD_ERR_INVALID_ARG;
    return verify_accept_common(hh, stream, hn, Wl, node_tok, nullptr, kept, nka, n_nodes, out_argmax,
                                out_acc_len, out_acc_nodes, out_acc_tok, out_next_tok, out_logits_dbg);
}

extern "C" int ctcsd_verify_accept_sampled(ctcsd_handle* hh, void* stream, const void* hn, const void* Wl,
                                           const int* node_tok, const int* parent, const int* depth, const int* n_nodes,
                                           const float* noise, float temperature,
                                           int* out_token, int* out_acc_len, int* out_acc_nodes, int* out_acc_tok,
                                           int* out_next_tok, float* out_logits_dbg) {
    if (!hh || !hn || !Wl || !node_tok || !parent || !depth || !n_nodes || !noise || !out_token || !out_acc_len ||
        !out_acc_nodes || !out_acc_tok || !out_next_tok)
        return CTCSD_ERR_INVALID_ARG;
    if (!(temperature > 0.f)) return CTCSD_ERR_INVALID_ARG;
    return verify_accept_common(hh, stream, hn, Wl, node_tok, parent, nullptr, nullptr, n_nodes, out_token,
                                out_acc_len, out_acc_nodes, out_acc_tok, out_next_tok, out_logits_dbg,
                                noise, depth, 1.0f / temperature);
}
