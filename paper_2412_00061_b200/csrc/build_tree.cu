// ctcsd_build_tree: ranked candidates -> prefix trie with ancestor bit-masks.
//
// One CTA per sequence, one thread per (candidate c, prefix length l).  A prefix creates a
// node iff no better-ranked candidate starts with the same l tokens; node ids are the
// 1-based positions of the creating prefixes in (c, l) order, which is the order of first
// appearance, so the node budget is applied by dropping ids >= max_nodes.
#include "common.cuh"

namespace ctcsd {
namespace {

constexpr int kThreads = 512;   // >= CTCSD_MAX_TOPN * CTCSD_MAX_T

struct TreeParams {
    const int* base_tok; const int* kv_len;
    const int* cand_tok; const int* cand_len; const int* n_cand;
    int T, topN, max_nodes;
    int* node_tok; int* parent; int* depth; int* pos;
    unsigned long long* mask; int* retrieve; int* n_nodes;
};

__global__ void __launch_bounds__(kThreads) build_tree_kernel(TreeParams p) {
    __shared__ int s_tok[CTCSD_MAX_TOPN * CTCSD_MAX_T];
    __shared__ int s_len[CTCSD_MAX_TOPN];
    __shared__ int s_node[CTCSD_MAX_TOPN * CTCSD_MAX_T];     // node id of each (c,l), -1 if none
    __shared__ int s_newid[CTCSD_MAX_TOPN * CTCSD_MAX_T];    // id given to a creating prefix
    __shared__ int s_parent[CTCSD_MAX_NODES];
    __shared__ int s_warp_total[kThreads / 32];
    __shared__ int s_total;

    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int T = p.T, N = p.topN, n_max = p.max_nodes;
    int nc = p.n_cand[b];
    nc = nc < 0 ? 0 : (nc > N ? N : nc);
    const int* ctok = p.cand_tok + (size_t)b * N * T;
    if (tid < N * T) s_tok[tid] = ctok[tid];
    if (tid < N) {
        int l = tid < nc ? p.cand_len[(size_t)b * N + tid] : 0;
        s_len[tid] = l < 0 ? 0 : (l > T ? T : l);
    }
    __syncthreads();

    // does this thread's prefix exist, and is it the first candidate to contain it?
    const int c = tid / T, l = tid - c * T + 1;          // prefix = first l tokens of candidate c
    const bool live = tid < N * T && c < nc && l <= s_len[c];
    int owner = c;
    if (live) {
        for (int c2 = 0; c2 < c; ++c2) {
            if (s_len[c2] < l) continue;
            bool same = true;
            for (int q = 0; q < l; ++q) same = same && (s_tok[c2 * T + q] == s_tok[c * T + q]);
            if (same) { owner = c2; break; }
        }
    }
    const bool creates = live && owner == c;
    unsigned bal = __ballot_sync(0xffffffffu, creates);
    if (lane == 0) s_warp_total[warp] = __popc(bal);
    __syncthreads();
    int before = __popc(bal & ((1u << lane) - 1u));
    for (int w = 0; w < warp; ++w) before += s_warp_total[w];
    if (tid == 0) {
        int tot = 0;
        for (int w = 0; w < kThreads / 32; ++w) tot += s_warp_total[w];
        s_total = tot;
    }
    if (tid < N * T) s_newid[tid] = creates ? 1 + before : -1;
    __syncthreads();
    int node = -1;
    if (live) {
        int id = s_newid[owner * T + (l - 1)];
        node = id < n_max ? id : -1;
    }
    if (tid < N * T) s_node[tid] = node;
    __syncthreads();

    const int n = (1 + s_total) < n_max ? (1 + s_total) : n_max;
    int* o_tok = p.node_tok + (size_t)b * n_max;
    int* o_par = p.parent + (size_t)b * n_max;
    int* o_dep = p.depth + (size_t)b * n_max;
    int* o_pos = p.pos + (size_t)b * n_max;
    const int L = p.kv_len[b];
    if (tid < N * T) p.retrieve[(size_t)b * N * T + tid] = node;
    if (creates && node >= 0) {
        int par = (l == 1) ? 0 : s_node[c * T + (l - 2)];
        o_tok[node] = s_tok[c * T + (l - 1)];
        o_par[node] = par;
        o_dep[node] = l;
        o_pos[node] = L + l;
        s_parent[node] = par;
    }
    if (tid == 0) {
        o_tok[0] = p.base_tok[b]; o_par[0] = -1; o_dep[0] = 0; o_pos[0] = L;
        s_parent[0] = -1;
        p.n_nodes[b] = n;
    }
    if (tid >= n && tid < n_max) { o_tok[tid] = -1; o_par[tid] = -1; o_dep[tid] = 0; o_pos[tid] = 0; }
    __syncthreads();

    const int W = (n_max + 63) / 64;
    if (tid < n_max) {
        unsigned long long m0 = 0ull, m1 = 0ull;
        if (tid < n) {
            int j = tid;
            for (int hop = 0; hop <= CTCSD_MAX_T && j >= 0; ++hop) {
                if (j < 64) m0 |= 1ull << j; else m1 |= 1ull << (j - 64);
                j = s_parent[j];
            }
        }
        unsigned long long* row = p.mask + ((size_t)b * n_max + tid) * W;
        row[0] = m0;
        if (W > 1) row[1] = m1;
    }
}

}  // namespace
}  // namespace ctcsd

using namespace ctcsd;

extern "C" int ctcsd_build_tree(ctcsd_handle* hh, void* stream, const int* base_tok, const int* kv_len,
                                const int* cand_tok, const int* cand_len, const int* n_cand,
                                int* out_node_tok, int* out_parent, int* out_depth, int* out_pos,
                                unsigned long long* out_mask, int* out_retrieve, int* out_n_nodes) {
    if (!hh || !base_tok || !kv_len || !cand_tok || !cand_len || !n_cand || !out_node_tok || !out_parent ||
        !out_depth || !out_pos || !out_mask || !out_retrieve || !out_n_nodes)
        return CTCSD_ERR_INVALID_ARG;
    Handle* h = &hh->h;
    const ctcsd_config& c = h->cfg;
    TreeParams p;
    p.base_tok = base_tok; p.kv_len = kv_len;
    p.cand_tok = cand_tok; p.cand_len = cand_len; p.n_cand = n_cand;
    p.T = c.T; p.topN = c.topN; p.max_nodes = c.max_nodes;
    p.node_tok = out_node_tok; p.parent = out_parent; p.depth = out_depth; p.pos = out_pos;
    p.mask = out_mask; p.retrieve = out_retrieve; p.n_nodes = out_n_nodes;
    build_tree_kernel<<<c.B, kThreads, 0, static_cast<cudaStream_t>(stream)>>>(p);
    CTCSD_LAUNCH_CHECK(h);
    return CTCSD_OK;
}
