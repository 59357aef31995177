// ctcsd_build_tree: ranked candidates -> prefix trie with ancestor bit-masks.
//
// One warp per sequence; lane c (and c + 32 when more than 32 candidates are kept) owns
// candidate c and keeps its tokens in registers.  The trie is grown level by level: the
// prefix of length l of candidate c is identified by (owner of its length l-1 prefix, token
// l), and its owner - the best-ranked candidate with the same prefix - is found with one
// warp match instruction.  A prefix creates a node iff its owner is the candidate itself;
// since a candidate's new prefixes are always its longest ones, node ids follow from an
// exclusive scan of the per-candidate counts, which reproduces the order of first
// appearance (candidates by rank, each left to right).  Ids >= max_nodes are dropped.
#include "common.cuh"

namespace ctcsd {
namespace {

constexpr int kT = CTCSD_MAX_T;

struct TreeParams {
    const int* base_tok; const int* kv_len;
    const int* cand_tok; const int* cand_len; const int* n_cand;
    int T, topN, max_nodes;
    int* node_tok; int* parent; int* depth; int* pos;
    unsigned long long* mask; int* retrieve; int* n_nodes;
    // raw layout (Sec. 3.3): candidates are full-length slot paths (cand_len null), the blank is
    // a symbol like any other in the trie, and kept/nka/mask/pos describe the CTC transform
    int* kept; int* nka; int blank;
    int* status;
};

__device__ __forceinline__ int warp_excl_scan(int v, int lane, int& total) {
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
    }
    total = __shfl_sync(0xffffffffu, inc, 31);
    return inc - v;
}

// Ancestor set of one node: bit j of word j/64.
struct NodeSet {
    unsigned long long w[4];
    __device__ __forceinline__ void clear() { w[0] = w[1] = w[2] = w[3] = 0ull; }
    __device__ __forceinline__ void add(int j) {
        const unsigned long long bit = 1ull << (j & 63);
        const int q = j >> 6;
        w[0] |= q == 0 ? bit : 0ull;
        w[1] |= q == 1 ? bit : 0ull;
        w[2] |= q == 2 ? bit : 0ull;
        w[3] |= q == 3 ? bit : 0ull;
    }
    __device__ __forceinline__ void store(unsigned long long* dst, int W) const {
        dst[0] = w[0];
        if (W > 1) dst[1] = w[1];
        if (W > 2) dst[2] = w[2];
        if (W > 3) dst[3] = w[3];
    }
};
static_assert(CTCSD_MAX_NODES <= 256, "NodeSet holds four 64-bit words");

__global__ void __launch_bounds__(32) build_tree_kernel(TreeParams p) {
    const int b = blockIdx.x, lane = threadIdx.x;
    const int T = p.T, N = p.topN, n_max = p.max_nodes;
    pdl_wait();                      // the candidates come from the preceding kernel
    pdl_trigger();
    // every input is requested at once (the candidate arrays are full-sized whatever n_cand and the
    // lengths say), so the kernel pays one memory latency, not three dependent ones
    int nc = p.n_cand[b];
    const int L = p.kv_len[b];
    int raw_len[2], raw_tok[2][kT];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int c = lane + 32 * h;
        raw_len[h] = (c < N && p.cand_len) ? p.cand_len[(size_t)b * N + c] : T;
#pragma unroll
        for (int q = 0; q < kT; ++q) raw_tok[h][q] = (c < N && q < T) ? p.cand_tok[((size_t)b * N + c) * T + q] : -1;
    }
    nc = nc < 0 ? 0 : (nc > N ? N : nc);
    const int halves = nc > 32 ? 2 : 1;
    const int W = (n_max + 63) / 64;

    int tok[2][kT], len[2], shared_lv[2], base[2];
    int own[2][kT];                      // owner candidate of each prefix (valid for l < len)
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int c = lane + 32 * h;
        int l = 0;
        if (c < nc) { l = raw_len[h]; l = l < 0 ? 0 : (l > T ? T : l); }
        len[h] = l;
#pragma unroll
        for (int q = 0; q < kT; ++q) tok[h][q] = (q < l) ? raw_tok[h][q] : -1;
    }

    // ---- owners, level by level ----
    int prev[2] = {0, 0};                // owner of the previous level's prefix (all start at the root)
#pragma unroll
    for (int l = 0; l < kT; ++l) {
        if (l < T) {
            unsigned long long key[2];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const bool active = len[h] > l;
                // inactive lanes get a key nobody else has
                key[h] = active ? (((unsigned long long)(unsigned)prev[h] << 32) | (unsigned)tok[h][l])
                                : (0xffffffff00000000ull | (unsigned)(lane + 32 * h));
            }
            unsigned m0 = __match_any_sync(0xffffffffu, key[0]);
            own[0][l] = __ffs(m0) - 1;
            own[1][l] = -1;
            if (halves == 2) {
                unsigned m1 = __match_any_sync(0xffffffffu, key[1]);
                int o = 32 + __ffs(m1) - 1;
                for (int j = 31; j >= 0; --j) {              // a match among candidates 0..31 ranks first
                    unsigned long long kj = __shfl_sync(0xffffffffu, key[0], j);
                    if (kj == key[1]) o = j;
                }
                own[1][l] = o;
            }
            prev[0] = own[0][l];
            prev[1] = own[1][l];
        }
    }

    // ---- node ids: a candidate's shared prefixes come first, its own (new) ones after ----
    int total[2] = {0, 0};
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        int sh = 0;
#pragma unroll
        for (int l = 0; l < kT; ++l) sh += (l < len[h] && own[h][l] != lane + 32 * h) ? 1 : 0;
        shared_lv[h] = sh;
        base[h] = warp_excl_scan(len[h] - sh, lane, total[h]);
    }
    base[0] += 1;
    base[1] += 1 + total[0];
    const int n_all = 1 + total[0] + total[1];
    const int n = n_all < n_max ? n_all : n_max;

    int* o_tok = p.node_tok + (size_t)b * n_max;
    int* o_par = p.parent + (size_t)b * n_max;
    int* o_dep = p.depth + (size_t)b * n_max;
    int* o_pos = p.pos + (size_t)b * n_max;
    unsigned long long* o_mask = p.mask + (size_t)b * n_max * W;

#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int c = lane + 32 * h;
        NodeSet anc;
        anc.clear();
        anc.add(0);                                    // the root is everybody's ancestor
        int parent_node = 0;
#pragma unroll
        for (int l = 0; l < kT; ++l) {
            if (l < T) {
                // owner's numbering data (all lanes take part in the shuffles)
                const int o = (l < len[h]) ? own[h][l] : 0;
                const int ob0 = __shfl_sync(0xffffffffu, base[0], o & 31);
                const int ob1 = __shfl_sync(0xffffffffu, base[1], o & 31);
                const int os0 = __shfl_sync(0xffffffffu, shared_lv[0], o & 31);
                const int os1 = __shfl_sync(0xffffffffu, shared_lv[1], o & 31);
                int node = -1;
                if (l < len[h] && parent_node >= 0) {
                    const int ob = o >= 32 ? ob1 : ob0, os = o >= 32 ? os1 : os0;
                    node = ob + (l - os);
                    if (node >= n_max) node = -1;
                }
                if (c < N) p.retrieve[((size_t)b * N + c) * T + l] = node;
                if (node >= 0 && CTCSD_IN_BOUNDS(p.status, 10, node, n_max)) {
                    anc.add(node);
                    if (o == c) {                          // this candidate creates the node
                        o_tok[node] = tok[h][l];
                        o_par[node] = parent_node;
                        o_dep[node] = l + 1;
                        o_pos[node] = L + l + 1;
                        anc.store(o_mask + (size_t)node * W, W);
                    }
                }
                parent_node = node;
            }
        }
    }
    if (lane == 0) {
        o_tok[0] = p.base_tok[b]; o_par[0] = -1; o_dep[0] = 0; o_pos[0] = L;
        o_mask[0] = 1ull;
        for (int w = 1; w < W; ++w) o_mask[w] = 0ull;
        p.n_nodes[b] = n;
    }
    for (int i = n + lane; i < n_max; i += 32) {
        o_tok[i] = -1; o_par[i] = -1; o_dep[i] = 0; o_pos[i] = 0;
        for (int w = 0; w < W; ++w) o_mask[(size_t)i * W + w] = 0ull;
    }
    if (p.kept == nullptr) return;

    // ---- raw layout: which nodes survive the CTC transform, and what each node may attend to ----
    // A node is kept iff its symbol is not the blank and differs from its parent's symbol (the
    // root holds the base token and is not part of the alignment).  Removed nodes are masked out
    // of every row, their own included; positions count kept nodes only.
    __syncwarp();                                   // the warp's own writes above are now visible to it
    int* o_kept = p.kept + (size_t)b * n_max;
    int* o_nka = p.nka + (size_t)b * n_max;
    for (int i = lane; i < n_max; i += 32) {
        if (i >= n) { o_kept[i] = 0; o_nka[i] = -1; continue; }
        NodeSet vis;
        vis.clear();
        vis.add(0);
        int count = 0, near = -1, self_kept = 1;
        int j = i;
        for (int step = 0; step <= kT && j > 0; ++step) {
            const int par = o_par[j];
            const int sym = o_tok[j];
            const bool kj = sym != p.blank && (par == 0 || sym != o_tok[par]);
            if (j == i) self_kept = kj ? 1 : 0;
            if (kj) {
                vis.add(j);
                ++count;
                if (j != i && near < 0) near = j;
            }
            j = par;
        }
        if (i > 0 && near < 0) near = 0;
        o_kept[i] = self_kept;
        o_nka[i] = near;
        o_pos[i] = L + count;
        vis.store(o_mask + (size_t)i * W, W);
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
    p.status = status_ptr(h);
    p.node_tok = out_node_tok; p.parent = out_parent; p.depth = out_depth; p.pos = out_pos;
    p.mask = out_mask; p.retrieve = out_retrieve; p.n_nodes = out_n_nodes;
    p.kept = nullptr; p.nka = nullptr; p.blank = c.V;
    CTCSD_CUDA_CHECK(h, launch_pdl(build_tree_kernel, dim3(c.B), dim3(32), 0, static_cast<cudaStream_t>(stream), 1, p));
    CTCSD_LAUNCH_CHECK(h);
    return CTCSD_OK;
}

extern "C" int ctcsd_build_raw_tree(ctcsd_handle* hh, void* stream, const int* base_tok, const int* kv_len,
                                    const int* raw_tok, const int* n_raw,
                                    int* out_node_tok, int* out_parent, int* out_depth, int* out_pos,
                                    unsigned long long* out_mask, int* out_retrieve, int* out_n_nodes,
                                    int* out_kept, int* out_nka) {
    if (!hh || !base_tok || !kv_len || !raw_tok || !n_raw || !out_node_tok || !out_parent || !out_depth ||
        !out_pos || !out_mask || !out_retrieve || !out_n_nodes || !out_kept || !out_nka)
        return CTCSD_ERR_INVALID_ARG;
    Handle* h = &hh->h;
    const ctcsd_config& c = h->cfg;
    TreeParams p;
    p.base_tok = base_tok; p.kv_len = kv_len;
    p.cand_tok = raw_tok; p.cand_len = nullptr; p.n_cand = n_raw;
    p.T = c.T; p.topN = c.topN; p.max_nodes = c.max_nodes;
    p.status = status_ptr(h);
    p.node_tok = out_node_tok; p.parent = out_parent; p.depth = out_depth; p.pos = out_pos;
    p.mask = out_mask; p.retrieve = out_retrieve; p.n_nodes = out_n_nodes;
    p.kept = out_kept; p.nka = out_nka; p.blank = c.V;
    CTCSD_CUDA_CHECK(h, launch_pdl(build_tree_kernel, dim3(c.B), dim3(32), 0, static_cast<cudaStream_t>(stream), 1, p));
    CTCSD_LAUNCH_CHECK(h);
    return CTCSD_OK;
}
