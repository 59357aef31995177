// Greedy acceptance walk over the token tree (paper Sec. 2.2 / Sec. 3.3: a drafted token is
// kept only where it equals the base model's greedy choice; the longest such path wins).
#pragma once

#include "common.cuh"

namespace ctcsd {

struct AcceptParams {
    const int* node_tok; const int* parent; const int* n_nodes; const int* argmax;
    int B, T, max_nodes;
    int* acc_len; int* acc_nodes; int* acc_tok; int* next_tok;
};

#ifdef __CUDACC__
// Executed by one full warp for sequence b: starting at the root, move to the child whose
// token equals the arg-max at the current node; stop when no child matches.
__device__ __forceinline__ void greedy_accept_warp(const AcceptParams& p, int b, int lane) {
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
#endif

}  // namespace ctcsd
