// Greedy acceptance walk over the token tree (paper Sec. 2.2 / Sec. 3.3: a drafted token is
// kept only where it equals the base model's greedy choice; the longest such path wins).
#pragma once

#include "common.cuh"

namespace ctcsd {

struct AcceptParams {
    const int* node_tok; const int* parent; const int* n_nodes; const int* argmax;
    int B, T, max_nodes;
    int* acc_len; int* acc_nodes; int* acc_tok; int* next_tok;
    // raw-tree layout (the paper's own): nodes removed by the CTC transform stay in the tree;
    // kept[b,i] != 0 marks the survivors, nka[b,i] is the nearest kept proper ancestor.  Null for
    // the packed tree.
    const int* kept; const int* nka;
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

// Acceptance on the raw tree, executed by one full warp for sequence b (at most 256 nodes).  A
// kept node d follows kept node p when nka[d] == p; best[p] = longest chain p -> d1 -> d2 ... in
// which every node's token equals the arg-max at its predecessor; among equally long
// continuations the lowest node id wins.  Lane l holds nodes l, l+32, ..., l+224.
__device__ __forceinline__ void raw_accept_warp(const AcceptParams& p, int b, int lane) {
    const int n_max = p.max_nodes;
    int n = p.n_nodes[b];
    n = n < 1 ? 1 : (n > n_max ? n_max : n);
    const int* am = p.argmax + (size_t)b * n_max;
    constexpr int kQ = 8;                              // nodes per lane
    int tok[kQ], kp[kQ], na[kQ], best[kQ], succ[kQ];
#pragma unroll
    for (int q = 0; q < kQ; ++q) {
        const int d = lane + 32 * q;
        const bool in = d < n;
        tok[q] = in ? p.node_tok[(size_t)b * n_max + d] : -1;
        kp[q] = in ? p.kept[(size_t)b * n_max + d] : 0;
        na[q] = in ? p.nka[(size_t)b * n_max + d] : -2;
        best[q] = 0;
        succ[q] = -1;
    }
    for (int pn = n - 1; pn >= 0; --pn) {
        const int owner = pn & 31, oq = pn >> 5;
        int pk = 0;
#pragma unroll
        for (int q = 0; q < kQ; ++q) pk = (q == oq) ? kp[q] : pk;
        pk = __shfl_sync(0xffffffffu, pk, owner);
        if (!pk) continue;                                      // uniform
        const int want = am[pn];
        // this lane's best follower: longer chain first, then lower id
        int val = 0, who = 0x7fffffff;
#pragma unroll
        for (int q = 0; q < kQ; ++q) {
            const int d = lane + 32 * q;
            if (d > pn && kp[q] && na[q] == pn && tok[q] == want) {
                const int v = 1 + best[q];
                if (v > val || (v == val && d < who)) { val = v; who = d; }
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const int v2 = __shfl_xor_sync(0xffffffffu, val, o);
            const int w2 = __shfl_xor_sync(0xffffffffu, who, o);
            if (v2 > val || (v2 == val && w2 < who)) { val = v2; who = w2; }
        }
        if (lane == owner) {
#pragma unroll
            for (int q = 0; q < kQ; ++q)
                if (q == oq) { best[q] = val; succ[q] = val > 0 ? who : -1; }
        }
    }
    int cur = 0, len = 0;
    while (len < p.T) {
        int sc = -1;
#pragma unroll
        for (int q = 0; q < kQ; ++q) sc = (q == (cur >> 5)) ? succ[q] : sc;
        sc = __shfl_sync(0xffffffffu, sc, cur & 31);
        if (sc < 0) break;
        cur = sc;
        int tk = -1;
#pragma unroll
        for (int q = 0; q < kQ; ++q) tk = (q == (cur >> 5)) ? tok[q] : tk;
        tk = __shfl_sync(0xffffffffu, tk, cur & 31);
        if (lane == 0) {
            p.acc_nodes[(size_t)b * p.T + len] = cur;
            p.acc_tok[(size_t)b * p.T + len] = tk;
        }
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

// Dispatch on the layout.
__device__ __forceinline__ void accept_warp(const AcceptParams& p, int b, int lane) {
    if (p.kept != nullptr) raw_accept_warp(p, b, lane);
    else greedy_accept_warp(p, b, lane);
}
#endif

}  // namespace ctcsd
