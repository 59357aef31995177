// ctcsd_verify_accept: LM head with row arg-max at every tree node, then the greedy walk
// down the token tree.
#include "gemv_stream.cuh"
#include "lm_head_tc.cuh"

namespace ctcsd {
namespace {

struct AcceptParams {
    const int* node_tok; const int* parent; const int* n_nodes; const int* argmax;
    int T, max_nodes;
    int* acc_len; int* acc_nodes; int* acc_tok; int* next_tok;
};

// One warp per sequence: starting at the root, move to the child whose token equals the
// base model's greedy token at the current node; stop when no child matches.
__global__ void __launch_bounds__(32) greedy_accept_kernel(AcceptParams p) {
    const int b = blockIdx.x, lane = threadIdx.x;
    const int n_max = p.max_nodes;
    int n = p.n_nodes[b];
    n = n < 1 ? 1 : (n > n_max ? n_max : n);
    const int* tok = p.node_tok + (size_t)b * n_max;
    const int* par = p.parent + (size_t)b * n_max;
    const int* am = p.argmax + (size_t)b * n_max;
    int cur = 0, len = 0;
    while (len < p.T) {
        const int want = am[cur];
        int found = -1;
        for (int base = 0; base < n && found < 0; base += 32) {
            int c = base + lane;
            bool hit = c >= 1 && c < n && par[c] == cur && tok[c] == want;
            unsigned bal = __ballot_sync(0xffffffffu, hit);
            if (bal) found = base + __ffs(bal) - 1;
        }
        if (found < 0) break;
        if (lane == 0) {
            p.acc_nodes[(size_t)b * p.T + len] = found;
            p.acc_tok[(size_t)b * p.T + len] = want;
        }
        cur = found;
        ++len;
    }
    for (int l = len + lane; l < p.T; l += 32) {
        p.acc_nodes[(size_t)b * p.T + l] = -1;
        p.acc_tok[(size_t)b * p.T + l] = -1;
    }
    if (lane == 0) {
        p.acc_len[b] = len;
        p.next_tok[b] = am[cur];
    }
}

}  // namespace
}  // namespace ctcsd

using namespace ctcsd;

extern "C" int ctcsd_verify_accept(ctcsd_handle* hh, void* stream, const void* hn, const void* Wl,
                                   const int* node_tok, const int* parent, const int* n_nodes,
                                   int* out_argmax, int* out_acc_len, int* out_acc_nodes, int* out_acc_tok,
                                   int* out_next_tok, float* out_logits_dbg) {
    if (!hh || !hn || !Wl || !node_tok || !parent || !n_nodes || !out_argmax || !out_acc_len || !out_acc_nodes ||
        !out_acc_tok || !out_next_tok)
        return CTCSD_ERR_INVALID_ARG;
    Handle* h = &hh->h;
    const ctcsd_config& c = h->cfg;
    if ((reinterpret_cast<uintptr_t>(hn) | reinterpret_cast<uintptr_t>(Wl)) & 15) return CTCSD_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int M = c.B * c.max_nodes;

    int rc = CTCSD_ERR_UNSUPPORTED;
    if (lm_head_tc_supported(h)) rc = launch_lm_head_tc(h, s, M, hn, Wl, out_argmax, out_logits_dbg);
    if (rc == CTCSD_ERR_UNSUPPORTED) {
        GemvParams g;
        g.x = hn; g.W = Wl; g.row_seq = nullptr; g.blank_bias = nullptr;
        g.m0 = 0; g.mcount = 0; g.H = c.H; g.slots = 1; g.rows_per_slot = c.V; g.grid = 0;
        g.part = nullptr; g.part_slot = nullptr; g.counter = nullptr;
        g.mode = 1; g.k = 1;
        g.out_topk_id = nullptr; g.out_topk_lp = nullptr; g.out_lse = nullptr;
        g.out_argmax = out_argmax;
        g.logits_dbg = out_logits_dbg;
        rc = launch_gemv_stream(h, s, c.dtype, M, g);
    }
    if (rc != CTCSD_OK) return rc;

    AcceptParams a;
    a.node_tok = node_tok; a.parent = parent; a.n_nodes = n_nodes; a.argmax = out_argmax;
    a.T = c.T; a.max_nodes = c.max_nodes;
    a.acc_len = out_acc_len; a.acc_nodes = out_acc_nodes; a.acc_tok = out_acc_tok; a.next_tok = out_next_tok;
    greedy_accept_kernel<<<c.B, 32, 0, s>>>(a);
    CTCSD_LAUNCH_CHECK(h);
    return CTCSD_OK;
}
