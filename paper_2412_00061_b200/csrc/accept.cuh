// Greedy acceptance over the token tree (paper Sec. 2.2 / Sec. 3.3: a drafted token is kept
// only where it equals the base model's greedy choice; the longest such path wins).
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
    int* status;             // device status word
};

#ifdef __CUDACC__
constexpr int kAcceptScratchInts = 3 * CTCSD_MAX_NODES;     // shared-memory ints one warp needs

// Acceptance for sequence b, executed by one full warp; `scratch` is kAcceptScratchInts ints of
// shared memory owned by this warp.
//
// Node d follows node a(d): its parent in the packed tree, its nearest kept ancestor in the raw
// tree (removed nodes follow nobody).  d agrees when its token equals the arg-max at a(d).  The
// accepted path is the longest chain root -> d1 -> d2 ... of agreeing nodes; among equally long
// continuations the lowest node id wins at every level.  (In the packed tree siblings carry
// distinct tokens, so at most one child agrees and this is the plain greedy walk.)
//
// Three passes, each over all nodes at once (lane l holds nodes l, l+32, ...), so the cost does
// not grow with the tree: (1) level[d] = length of the agreeing chain that reaches d, found
// level by level; (2) from the deepest level up, every reached node offers 1 + its own best
// continuation to the node it follows (a shared-memory maximum over (length, lowest id));
// (3) the walk from the root along the recorded best followers.
__device__ __forceinline__ void accept_warp(const AcceptParams& p, int b, int lane, int* scratch) {
    constexpr int kQ = CTCSD_MAX_NODES / 32;                // nodes per lane
    const int n_max = p.max_nodes;
    int n = p.n_nodes[b];
    n = n < 1 ? 1 : (n > n_max ? n_max : n);
    int* s_am = scratch;                                    // arg-max at each node
    int* s_level = scratch + CTCSD_MAX_NODES;               // -1: not reached
    unsigned* s_best = reinterpret_cast<unsigned*>(scratch + 2 * CTCSD_MAX_NODES);   // (length << 16) | (0xffff - follower)
    const bool raw = p.kept != nullptr;
    const int* follows = (raw ? p.nka : p.parent) + (size_t)b * n_max;

    int tok[kQ], fo[kQ], level[kQ];
#pragma unroll
    for (int q = 0; q < kQ; ++q) {
        const int d = lane + 32 * q;
        const bool in = d >= 1 && d < n;
        tok[q] = in ? p.node_tok[(size_t)b * n_max + d] : -1;
        int f = in ? follows[d] : -1;
        if (raw && in && p.kept[(size_t)b * n_max + d] == 0) f = -1;
        fo[q] = (f >= 0 && f < n) ? f : -1;
        level[q] = -1;
        if (d < CTCSD_MAX_NODES) {
            s_am[d] = d < n ? p.argmax[(size_t)b * n_max + d] : -1;
            s_level[d] = d == 0 ? 0 : -1;
            s_best[d] = 0u;
        }
    }
    __syncwarp();
    bool agrees[kQ];
#pragma unroll
    for (int q = 0; q < kQ; ++q) agrees[q] = fo[q] >= 0 && tok[q] == s_am[fo[q]];

    // (1) levels
    int deepest = 0;
    for (int r = 1; r <= p.T; ++r) {
        bool any = false;
#pragma unroll
        for (int q = 0; q < kQ; ++q) {
            if (agrees[q] && level[q] < 0 && s_level[fo[q]] == r - 1) { level[q] = r; any = true; }
        }
        __syncwarp();
#pragma unroll
        for (int q = 0; q < kQ; ++q)
            if (level[q] == r) s_level[lane + 32 * q] = r;
        __syncwarp();
        if (!__any_sync(0xffffffffu, any)) break;
        deepest = r;
    }
    // (2) best continuation, deepest level first
    for (int r = deepest; r >= 1; --r) {
#pragma unroll
        for (int q = 0; q < kQ; ++q) {
            if (level[q] == r) {
                const int d = lane + 32 * q;
                const unsigned len = 1u + (s_best[d] >> 16);
                atomicMax(&s_best[fo[q]], (len << 16) | (0xffffu - (unsigned)d));
            }
        }
        __syncwarp();
    }
    // (3) the walk
    int cur = 0, len = 0;
    while (len < p.T) {
        const unsigned e = s_best[cur];
        if ((e >> 16) == 0u) break;
        const int nxt = (int)(0xffffu - (e & 0xffffu));
        if (lane == 0 && CTCSD_IN_BOUNDS(p.status, 20, nxt, n_max)) {
            p.acc_nodes[(size_t)b * p.T + len] = nxt;
            p.acc_tok[(size_t)b * p.T + len] = s_am[cur];      // an agreeing node's token is the arg-max before it
        }
        cur = nxt;
        ++len;
    }
    for (int l = len + lane; l < p.T; l += 32) {
        p.acc_nodes[(size_t)b * p.T + l] = -1;
        p.acc_tok[(size_t)b * p.T + l] = -1;
    }
    if (lane == 0) {
        p.acc_len[b] = len;
        p.next_tok[b] = s_am[cur];
    }
    __syncwarp();
}
#endif

}  // namespace ctcsd
