/*
 * ctcsd - the per-step draft-and-verify pass of CTC-drafted speculative decoding,
 * as CUDA kernels for NVIDIA B200 (sm_100a) behind a plain C ABI.
 *
 * One decoding step (paper Sec. 3.3, "Inference"): the base model has produced a hidden
 * state and a greedy base token; a draft head turns the hidden state into one distribution
 * per draft slot over the vocabulary plus the CTC blank; the k best symbols per slot are
 * combined into slot paths; each path is collapsed by beta^{-1} (Sec. 2.3), duplicates are
 * merged and scored by the sum over their alignments (Eq. 1 / Eq. 5, with Eq. 6 for one
 * alignment); the N best candidates become a token tree (Sec. 2.2) that the base model
 * verifies in one pass (tree attention + LM head), and the longest candidate that agrees
 * with the base model's greedy choice is accepted (Sec. 2.2, Sec. 3.3).
 *
 * Conventions
 *  - Every function returns an int status: CTCSD_OK (0) or a negative CTCSD_ERR_* code.
 *    Nothing throws; arguments are validated on the host before any launch.
 *  - Unless a parameter is marked [host], every pointer is a DEVICE pointer owned by the
 *    caller; inputs are read-only, outputs are the parameters named out_*.  The library
 *    never allocates device memory: all scratch lives in the workspace given to
 *    ctcsd_create.  Buffers must not alias unless stated.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Calls
 *    enqueue work on it and return without synchronising.  Two calls on the same handle
 *    must not overlap on the device (they share the workspace).
 *  - Problems found by a kernel (for example a bounded wait that ran out) are recorded in a
 *    device status word that ctcsd_poll_status reads.
 *  - dtype: 0 = float32, 1 = bfloat16 for activations, weights, Q/K/V and the attention
 *    output; logits, log-probabilities and scores are always float32 on the device.
 *  - Tensors are dense, row-major, last index fastest, in the shapes given.
 */
#ifndef CTCSD_H_
#define CTCSD_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

#define CTCSD_OK                0
#define CTCSD_ERR_INVALID_ARG  -1   /* null pointer, bad shape, value out of the documented range */
#define CTCSD_ERR_UNSUPPORTED  -2   /* a legal request this build has no kernel for */
#define CTCSD_ERR_WORKSPACE    -3   /* workspace missing, misaligned or too small */
#define CTCSD_ERR_CUDA         -4   /* a CUDA runtime/driver call failed (see ctcsd_last_cuda_error) */
#define CTCSD_ERR_TIMEOUT      -5   /* a bounded device-side wait ran out */
#define CTCSD_ERR_INTERNAL     -6
#define CTCSD_ERR_TOO_LARGE    -7   /* the problem does not fit the built-in scratch of a no-allocation call */

#define CTCSD_DTYPE_F32   0
#define CTCSD_DTYPE_BF16  1

#define CTCSD_SCORE_SUM   0   /* candidate score = log sum over alignments (Eq. 1 / Eq. 5) */
#define CTCSD_SCORE_MAX   1   /* candidate score = best single alignment (enumeration only) */

#define CTCSD_MAX_T        8    /* draft slots */
#define CTCSD_MAX_K        8    /* symbols kept per slot */
#define CTCSD_MAX_NODES    256  /* tree nodes per sequence, root included */
#define CTCSD_MAX_TOPN     64   /* candidates kept */
#define CTCSD_MAX_PATHS    4096 /* k^T limit for exhaustive enumeration */
#define CTCSD_MAX_BEAM     128
#define CTCSD_STATIC_ATTN_SCRATCH_BYTES  (32u << 20)  /* built-in scratch of ctcsd_tree_attention_static */

/* Problem shape, fixed per handle.  Notation follows the paper: T draft slots, blank id = V. */
typedef struct ctcsd_config {
    int B;          /* sequences per step (>= 1) */
    int H;          /* hidden size, multiple of 8 */
    int V;          /* vocabulary size; the draft head has V+1 classes, blank = V */
    int T;          /* draft slots, 1..CTCSD_MAX_T */
    int k;          /* symbols kept per slot, 1..CTCSD_MAX_K, T*k <= 64 */
    int beam;       /* 0: enumerate all k^T slot paths (k^T <= CTCSD_MAX_PATHS);
                       >0: CTC prefix beam search of this width (<= CTCSD_MAX_BEAM) */
    int topN;       /* candidates kept, 1..CTCSD_MAX_TOPN */
    int max_nodes;  /* tree node budget per sequence including the root, 2..CTCSD_MAX_NODES */
    int Hq;         /* query heads */
    int Hkv;        /* key/value heads, divides Hq */
    int D;          /* head dimension: 64 or 128 */
    int dtype;      /* CTCSD_DTYPE_* */
    int score_mode; /* CTCSD_SCORE_* */
    int max_draft_rows; /* largest M passed to ctcsd_draft_logits; 0 means B */
} ctcsd_config;

typedef struct ctcsd_handle ctcsd_handle;

/* Bytes of device workspace a handle for `cfg` needs.  [host] cfg, [host] out_bytes. */
int ctcsd_workspace_bytes(const ctcsd_config* cfg, size_t* out_bytes);

/* Creates a handle on the current CUDA device.  `workspace` is device memory, 256-byte
 * aligned, at least ctcsd_workspace_bytes() large, owned by the caller and kept alive until
 * ctcsd_destroy; its first bytes are cleared here (synchronously).  [host] out_handle, cfg. */
int ctcsd_create(ctcsd_handle** out_handle, const ctcsd_config* cfg, void* workspace, size_t workspace_bytes);

/* Frees the host-side handle.  The workspace stays with the caller. */
int ctcsd_destroy(ctcsd_handle* h);

/* Synchronises `stream`, then reads and clears the device status word.  [host] out_status
 * receives CTCSD_OK or the first error a kernel recorded. */
int ctcsd_poll_status(ctcsd_handle* h, void* stream, int* out_status);

/* Self-test of the failure path: enqueues a kernel that waits, with the bounded wait all
 * streaming kernels use, on a barrier nothing ever signals.  The wait gives up after about a
 * millisecond and records CTCSD_ERR_TIMEOUT in the device status word (ctcsd_poll_status then
 * returns it and clears it); the context stays usable. */
int ctcsd_selftest_timeout(ctcsd_handle* h, void* stream);

/* Text for a status code; never NULL.  The string is static. */
const char* ctcsd_strerror(int status);

/* cudaError_t value of the most recent failing CUDA call made through handle `h` (0 if none). */
int ctcsd_last_cuda_error(const ctcsd_handle* h);

/* 1 when the library was built with -DCTCSD_DEBUG_BOUNDS (the kernels then check the index of
 * every store into a caller's array or an internal list, record CTCSD_ERR_INTERNAL with
 * 1000 + the site number in the device status word and skip the store), else 0. */
int ctcsd_debug_bounds_enabled(void);

/* Number of kernels this handle has launched since creation (for launch accounting). */
long long ctcsd_launch_count(const ctcsd_handle* h);

/*
 * Optional hint, off unless set.  Names a range of device memory, owned by the caller and never
 * written while the handle is in use, that ctcsd_draft_logits asks the L2 cache to fetch as soon
 * as its own weight stream has been requested (meant for data that a later call of the step
 * streams, while the small kernels in between leave HBM idle).  Measured on a B200 at the 7B
 * shape with the head of the LM-head weights: no gain up to 48 MB, a loss beyond (the requests
 * lengthen the draft head's tail and compete with the attention's reads), so the step does not
 * use it.  0 turns the hint off.  [host] call; `ptr` 16-byte aligned.
 */
int ctcsd_set_l2_prefetch(ctcsd_handle* h, const void* ptr, size_t bytes);

/*
 * Draft head, per-slot log-softmax and per-slot top-k (Sec. 3.2: one probability
 * distribution per place from the projected hidden state; Sec. 3.3: every place keeps its k most
 * probable symbols, best first, k fixed in advance).
 *   z[m,t,v]   = sum_h x[m,h] * Wd[t,v,h]  (+ blank_bias[row_seq[m]] when v == V)
 *   lse[m,t]   = log sum_v exp z[m,t,v]
 *   top-k      = the k largest z[m,t,:] over all V+1 classes, descending, ties to the lower id;
 *                out_topk_lp = z - lse.
 * M          rows of x, 1 <= M <= max_draft_rows.
 * x          [M,H] dtype.            Wd  [T,V+1,H] dtype (hidden axis contiguous).
 * row_seq    [M] int32 sequence index of each row, or NULL for the identity (needs M <= B).
 * blank_bias [B] float32, or NULL for no bias.
 * out_topk_id [M,T,k] int32;  out_topk_lp [M,T,k] float32;  out_lse [M,T] float32.
 * out_logits_dbg  NULL, or [M,T,V+1] float32 receiving every logit exactly as the kernel
 *                 computed it (for checking the selection against the kernel's own values).
 */
int ctcsd_draft_logits(ctcsd_handle* h, void* stream, int M, const void* x, const void* Wd,
                       const int* row_seq, const float* blank_bias,
                       int* out_topk_id, float* out_topk_lp, float* out_lse, float* out_logits_dbg);

/*
 * ctcsd_draft_logits with a row map: draft row m reads the hidden state x[x_rows[m]], everything
 * else as above.  This is how decoding steps chain without host work (Sec. 3.3: the draft module
 * takes the base model's hidden state at the current position): x is the previous step's
 * [B*max_nodes,H] array of tree-node hidden states and x_rows the out_sel_row that
 * ctcsd_commit_accepted produced, so the next step drafts from the last accepted node.
 * x [x_row_count,H] dtype;  x_rows [M] int32 (device), each in 0..x_row_count-1: an entry outside
 * that range records CTCSD_ERR_INVALID_ARG in the device status word and that row drafts from a
 * zero vector.  With more than 8 rows the weights are streamed once per 8 rows.
 */
int ctcsd_draft_logits_rows(ctcsd_handle* h, void* stream, int M, const void* x, int x_row_count,
                            const int* x_rows, const void* Wd, const int* row_seq, const float* blank_bias,
                            int* out_topk_id, float* out_topk_lp, float* out_lse, float* out_logits_dbg);

/*
 * Slot paths -> collapsed, deduplicated, scored candidates -> the topN best (Sec. 3.3: the
 * per-slot tokens are combined into sequences, of which the best-scoring are kept; Sec. 2.3 /
 * Sec. 3.1: beta^{-1} merges adjacent repeats, then removes blanks; Eq. 6: a path's
 * probability is the product over slots; Eq. 1 / Eq. 5: a candidate's probability is the sum
 * over the paths that collapse to it).
 * With beam == 0 all k^T paths are enumerated; with beam > 0 a CTC prefix beam search over
 * the same per-slot lists keeps the `beam` most probable prefixes after every slot.
 * Candidates are ordered by score descending, then shorter first, then token ids
 * lexicographically ascending; the empty candidate is never returned.  Scores are formed in
 * float64 from the float32 inputs and returned as float32.
 * M          rows in topk_id/topk_lp.    topk_id [M,T,k] int32;  topk_lp [M,T,k] float32.
 * sel_row    [B] int32: sequence b drafts from row sel_row[b]; NULL means row b.
 * out_cand_tok [B,topN,T] int32 (-1 padded);  out_cand_len [B,topN] int32 (0 when unused);
 * out_cand_score [B,topN] float32 (-inf when unused);  out_n_cand [B] int32.
 */
int ctcsd_topk_collapse(ctcsd_handle* h, void* stream, int M, const int* topk_id, const float* topk_lp,
                        const int* sel_row,
                        int* out_cand_tok, int* out_cand_len, float* out_cand_score, int* out_n_cand);

/*
 * Packs the ranked candidates into a token tree (Sec. 2.2: candidates are the root-to-leaf
 * paths of a tree verified under a tree attention mask; Sec. 3.3: the greedy base token
 * comes first).  Node 0 is the root holding base_tok[b]; further nodes are the distinct
 * candidate prefixes in order of first appearance (candidates by rank, each left to right);
 * prefixes that would get an id >= max_nodes are dropped.
 * base_tok [B] int32;  kv_len [B] int32 (cached tokens before the tree);
 * cand_tok [B,topN,T], cand_len [B,topN], n_cand [B] as produced by ctcsd_topk_collapse.
 * out_node_tok/out_parent/out_depth/out_pos [B,max_nodes] int32 (parent of the root = -1,
 *   pos = kv_len + depth; entries of unused nodes: token -1, parent -1, depth 0, pos 0);
 * out_mask [B,max_nodes,W] uint64 with W = ceil(max_nodes/64): bit j of row i is set iff
 *   node j is node i or one of its ancestors;
 * out_retrieve [B,topN,T] int32: node id of candidate c's prefix of length l+1, or -1;
 * out_n_nodes [B] int32.
 */
int ctcsd_build_tree(ctcsd_handle* h, void* stream, const int* base_tok, const int* kv_len,
                     const int* cand_tok, const int* cand_len, const int* n_cand,
                     int* out_node_tok, int* out_parent, int* out_depth, int* out_pos,
                     unsigned long long* out_mask, int* out_retrieve, int* out_n_nodes);

/*
 * Tree attention (Sec. 2.2 / Sec. 3.3: all candidates are verified in one pass of the base
 * model; a node attends to the cached prefix and to its own ancestors):
 *   O[b,i,h,:] = softmax_j( scale * q[b,i,h,:] . k[b,g,j,:] ) v[b,g,j,:],  g = h / (Hq/Hkv),
 *   j over cache rows 0..kv_len[b]-1 and rows kv_len[b]+j' for every node j' whose mask bit
 *   is set in row i.
 * Q [B,max_nodes,Hq,D] dtype;  K, V [B,Hkv,Lcap,D] dtype, the caller having written node j's
 * key/value at cache row kv_len[b]+j;  Lcap >= max_b(kv_len[b]) + max_nodes.
 * kv_len, n_nodes [B] int32;  mask as produced by ctcsd_build_tree.
 * out_O [B,max_nodes,Hq,D] dtype; rows i >= n_nodes[b] are written as zero.
 */
int ctcsd_tree_attention(ctcsd_handle* h, void* stream, const void* Q, const void* K, const void* V,
                         int Lcap, const int* kv_len, const int* n_nodes,
                         const unsigned long long* mask, float scale, void* out_O);

/*
 * LM head with row arg-max at every tree node, then greedy acceptance (Eq. 3-4 form:
 * argmax of the LM head's distribution; Sec. 2.2: a draft is accepted only where it matches
 * the base model's greedy output; Sec. 3.3: the longest such candidate is the step's output).
 *   y[m,v] = sum_h hn[m,h] * Wl[v,h];  am[m] = argmax_v y[m,v], ties to the lower id.
 *   Walk: cur = root; while some child c of cur has node_tok[c] == am[cur]: accept c.  Siblings
 *   carry distinct tokens in a tree from ctcsd_build_tree, so at most one child qualifies; in a
 *   hand-made tree with equal siblings the longest agreeing path is taken, lowest id on ties.
 * hn [B*max_nodes,H] dtype (row b*max_nodes+i is node i of sequence b; rows of unused nodes,
 *   i >= n_nodes[b], are never looked at: with bfloat16 and more than 128 tree rows the live
 *   rows are first packed densely into the workspace, so unused rows cost no arithmetic);
 *   Wl [V,H] dtype;  node_tok, parent [B,max_nodes], n_nodes [B].
 * out_argmax [B,max_nodes] int32 (entries of unused nodes: not meaningful, -1 where the rows
 *   were packed);  out_acc_len [B] int32 (accepted draft tokens, root and
 *   bonus token excluded);  out_acc_nodes, out_acc_tok [B,T] int32 (-1 padded);
 *   out_next_tok [B] int32 = am at the last accepted node (the bonus token);
 * out_logits_dbg  NULL or [B*max_nodes,V] float32 receiving every logit as computed (rows of
 *   unused nodes may be left untouched).
 */
int ctcsd_verify_accept(ctcsd_handle* h, void* stream, const void* hn, const void* Wl,
                        const int* node_tok, const int* parent, const int* n_nodes,
                        int* out_argmax, int* out_acc_len, int* out_acc_nodes, int* out_acc_tok,
                        int* out_next_tok, float* out_logits_dbg);

/*
 * Sampling acceptance (Sec. 2, second paragraph: a drafted token is accepted with probability
 * min(1, p/p') - the ratio is printed upside down there - and after a rejection a token is drawn
 * from norm(max(0, P - P')); Sec. 6 names sampling as the next step).  The tree's tokens are a
 * deterministic function of the draft head's output, so the proposal P' of a child that is tried
 * is the point mass on its token: it is accepted with probability P(child), and the rejected
 * token is removed from P.  Trying a node's children in turn under this rule amounts to one draw
 * from P that is accepted iff it is a child's token, which is what is computed:
 *   x[b,i] = argmax_v fma( y[b,i,v], 1/temperature, noise[b, depth[b,i], v] ),  ties to the lower id,
 * a draw from softmax(y/temperature) when `noise` holds independent standard Gumbel variates
 * (-log(-log(U))); then the walk of ctcsd_verify_accept with x in place of the arg-max.  Nodes of
 * equal depth lie on different paths and share a noise row; nodes along a path use different rows.
 * temperature -> 0 approaches greedy acceptance.  The fused multiply-add is rounded once, to float32.
 * depth [B,max_nodes] int32 as produced by ctcsd_build_tree;  noise [B,T+1,V] float32;
 * temperature > 0;  out_token [B,max_nodes] int32 = x;  out_next_tok = x at the last accepted node;
 * everything else as for ctcsd_verify_accept (out_logits_dbg receives the logits y, without noise).
 */
int ctcsd_verify_accept_sampled(ctcsd_handle* h, void* stream, const void* hn, const void* Wl,
                                const int* node_tok, const int* parent, const int* depth, const int* n_nodes,
                                const float* noise, float temperature,
                                int* out_token, int* out_acc_len, int* out_acc_nodes, int* out_acc_tok,
                                int* out_next_tok, float* out_logits_dbg);

/*
 * History update after acceptance (Sec. 3.3, last paragraph: the step's output joins the decoding
 * history): the accepted path becomes part of the cached prefix, so that the next step can
 * start without host work.  For sequence b with L = kv_len[b]: the root's key/value row (cache
 * row L) stays; for l = 0 .. acc_len[b]-1 the row of accepted node acc_nodes[b,l] (cache row
 * L + node) is moved to row L + 1 + l, for every kv head, in K and in V; rows are read as they
 * were before the call (a destination may be another accepted node's source).
 * K, V [B,Hkv,Lcap,D] dtype, updated IN PLACE;  kv_len, acc_len [B], acc_nodes [B,T] as
 * produced by ctcsd_verify_accept.
 * out_kv_len [B] int32 = kv_len + 1 + acc_len; it may be the same array as kv_len (the new
 *   length of a sequence is written only after every kv head of that sequence has read the old one);
 * out_sel_row [B] int32 or NULL = b*max_nodes + last accepted node (the root if none): the
 *   tree row whose hidden state the next step drafts from (see sel_row of ctcsd_topk_collapse).
 * A sequence whose path would leave the cache is left unchanged and CTCSD_ERR_INVALID_ARG is
 * recorded in the device status word.
 */
int ctcsd_commit_accepted(ctcsd_handle* h, void* stream, void* K, void* V, int Lcap,
                          const int* kv_len, const int* acc_len, const int* acc_nodes,
                          int* out_kv_len, int* out_sel_row);

/*
 * The paper's own verification layout (Sec. 3.3): instead of collapsing the slot paths before
 * the tree is built, the most probable RAW paths - blanks and repeats still in place - form the
 * token tree, and the CTC transform acts through the attention map: a position whose symbol the
 * transform removes is masked for every query row, so that the base model scores exactly the
 * collapsed sequences.  Three calls replace ctcsd_topk_collapse / ctcsd_build_tree /
 * ctcsd_verify_accept; ctcsd_draft_logits, ctcsd_tree_attention and ctcsd_commit_accepted are
 * used unchanged (the latter moves kept nodes only, since only those are ever accepted).
 *
 * ctcsd_select_raw_paths: the topN most probable of the k^T slot paths of each sequence.  Path
 *   score = sum over the slots of the per-slot log-probability (Eq. 6), accumulated in slot
 *   order in float64; equal scores are ordered by path index (slot 1 most significant, the
 *   per-slot rank as the digit).  Requires k^T <= CTCSD_MAX_PATHS (else CTCSD_ERR_UNSUPPORTED);
 *   the handle's beam setting plays no part.
 *   topk_id, topk_lp [M,T,k], sel_row [B] or NULL: as for ctcsd_topk_collapse.
 *   out_raw_tok [B,topN,T] int32 (the blank is id V; unused rows -1);
 *   out_raw_score [B,topN] float32 (unused -inf);  out_n_raw [B] int32 = min(topN, k^T).
 *
 * ctcsd_build_raw_tree: the prefix trie of the raw paths, numbered like ctcsd_build_tree (the
 *   blank is a symbol like any other; every path has T symbols), plus the transform:
 *   out_kept [B,max_nodes] int32: 1 iff the node survives - its symbol is not the blank and
 *     differs from its parent's symbol; the root (the base token, not part of the alignment)
 *     is kept and does not count as a preceding symbol;  0 for removed and unused nodes;
 *   out_nka [B,max_nodes] int32: nearest kept proper ancestor (-1 for the root and unused nodes);
 *   out_mask: bit j of row i set iff j is the root, a kept proper ancestor of i, or i itself
 *     when i is kept;  out_pos = kv_len + number of kept non-root nodes on the path root..i;
 *   the remaining outputs as for ctcsd_build_tree.  Nodes beyond max_nodes are dropped.
 *
 * ctcsd_verify_accept_raw: LM head and arg-max exactly as ctcsd_verify_accept, then acceptance
 *   over the kept nodes: kept node d follows kept node p when nka[d] == p; the accepted path is
 *   the longest chain root -> d1 -> d2 ... in which every node's token equals the arg-max at
 *   its predecessor; among equally long continuations the lowest node id wins (at every level).
 *   out_acc_nodes holds kept node ids.
 */
int ctcsd_select_raw_paths(ctcsd_handle* h, void* stream, int M, const int* topk_id, const float* topk_lp,
                           const int* sel_row, int* out_raw_tok, float* out_raw_score, int* out_n_raw);
int ctcsd_build_raw_tree(ctcsd_handle* h, void* stream, const int* base_tok, const int* kv_len,
                         const int* raw_tok, const int* n_raw,
                         int* out_node_tok, int* out_parent, int* out_depth, int* out_pos,
                         unsigned long long* out_mask, int* out_retrieve, int* out_n_nodes,
                         int* out_kept, int* out_nka);
int ctcsd_verify_accept_raw(ctcsd_handle* h, void* stream, const void* hn, const void* Wl,
                            const int* node_tok, const int* kept, const int* nka, const int* n_nodes,
                            int* out_argmax, int* out_acc_len, int* out_acc_nodes, int* out_acc_tok,
                            int* out_next_tok, float* out_logits_dbg);

/*
 * The paper's Attention Draft Module (Sec. 3.1: one transformer layer, built like the base model's, on
 * the base model's hidden states; Sec. 3.2: F_hat = DraftModule(F), whose projection gives one
 * distribution per place; Sec. 4.3: it takes 14.93 % of the paper's decoding time).  The paper gives
 * no further detail; the layer built here is a LLaMA-style decoder layer with the handle's head
 * shape (Hq, Hkv, D):
 *   a = RMSNorm(F; g1);  q,k,v = a Wqkv^T;  rotary embedding of q and k at the row's position;
 *   attention of the newest position over all positions so far (scale 1/sqrt(D));
 *   h1 = F + Wo attn;  m = RMSNorm(h1; g2);  F_hat = h1 + Wdn ( SiLU(Wg m) * (Wu m) ).
 * No final norm.  Per step the caller hands over the hidden states of the newest n_new[b] <= R
 * positions of every sequence (what the previous step accepted); keys and values are made for all
 * of them and appended to the layer's own cache, the rest of the layer runs for the newest one,
 * and its output F_hat [B,H] is what ctcsd_draft_logits projects to the T places.
 *
 * ctcsd_draft_layer: weights, all device pointers, the matrices in the handle's dtype with the
 *   input axis contiguous: Wqkv [(Hq+2Hkv)*D, H] (query rows, then key rows, then value rows),
 *   Wo [H, Hq*D], Wgu [2I, H] (gate rows, then up rows), Wdn [H, I]; g1, g2 [H] float32;
 *   I the MLP width (multiple of 8), eps the RMSNorm epsilon, rope_theta the rotary base (the
 *   rotation pairs element i with i + D/2, frequency rope_theta^(-2i/D)).
 * workspace: device memory of ctcsd_draft_module_workspace_bytes(cfg, R, I) bytes, 256-byte aligned,
 *   owned by the caller, used only during the call.
 * F_new [B,R,H] dtype;  n_new [B] int32 in 1..R;  kv_len [B] int32: positions already in the cache;
 * Kd, Vd [B,Hkv,Lcap,D] dtype, updated in place at rows kv_len[b] .. kv_len[b]+n_new[b]-1;
 * out_F [B,H] dtype;  out_kv_len [B] int32 = kv_len + n_new (must not be the array kv_len);
 * out_F_dbg NULL or [B,H] float32: F_hat before it is rounded to dtype.
 * A sequence with n_new outside 1..R or kv_len + n_new > Lcap records CTCSD_ERR_INVALID_ARG in the
 * device status word; its cache is left alone and its output row is not meaningful.
 */
typedef struct ctcsd_draft_layer {
    const float* g1;
    const void*  Wqkv;
    const void*  Wo;
    const float* g2;
    const void*  Wgu;
    const void*  Wdn;
    int   I;
    float eps;
    float rope_theta;
} ctcsd_draft_layer;

int ctcsd_draft_module_workspace_bytes(const ctcsd_config* cfg, int R, int I, size_t* out_bytes);
int ctcsd_draft_module(ctcsd_handle* h, void* stream, const ctcsd_draft_layer* layer,
                       void* workspace, size_t workspace_bytes,
                       int R, const void* F_new, const int* n_new, const int* kv_len,
                       void* Kd, void* Vd, int Lcap,
                       void* out_F, int* out_kv_len, float* out_F_dbg);

/*
 * Tree attention without a handle and without any allocation (the paper has no counterpart:
 * this is a packaging variant of ctcsd_tree_attention, same arithmetic, same kernels).
 *
 * Who it is for: code that is not allowed to obtain device memory when it runs - an operator
 * plugged into a runtime that owns the memory plan, a service whose allocator is frozen after
 * start-up, a latency-critical loop where cudaMalloc's implicit device synchronisation is not
 * acceptable.  Such callers cannot provide the workspace that ctcsd_create asks for.  Here the
 * scratch (the per-split partial results that the merge pass combines) lives in an array of
 * CTCSD_STATIC_ATTN_SCRATCH_BYTES (+256) bytes inside the library's device image, which
 * every device that loads the library keeps reserved until the process exits.  The call
 * itself uses no cudaMalloc/cudaFree and no allocating routine.
 *
 * Works on the current device, bfloat16 only.  Shapes and tensors as for
 * ctcsd_tree_attention, given explicitly instead of through a handle:
 *   Q, out_O [B,max_nodes,Hq,D];  K, V [B,Hkv,Lcap,D];  kv_len, n_nodes [B];
 *   mask [B,max_nodes,ceil(max_nodes/64)] uint64;  D is 64 or 128;  2 <= max_nodes <= 128.
 * out_status: NULL, or a device int[2] that the call clears and in which a kernel records
 *   CTCSD_ERR_INVALID_ARG (and the sequence index) if kv_len/n_nodes would read outside the cache;
 *   such a sequence is treated as empty (no key is read, its output rows are zero).  With
 *   out_status == NULL the record goes to a private block that no call reads back: the zero rows
 *   are then the only sign, so pass a status array unless the lengths are known to be valid.
 * Limits and caveats:
 *   - B*Hq*max_nodes*(D+2)*4 bytes must not exceed CTCSD_STATIC_ATTN_SCRATCH_BYTES, else
 *     CTCSD_ERR_TOO_LARGE is returned and nothing is launched; within the limit the number of
 *     KV splits is reduced until the partials fit.
 *   - The first call on each device looks up the array's device address; make that first call
 *     outside any stream capture.
 *   - All calls on a device share the one array: two calls that overlap on the GPU (different
 *     streams, or concurrent graphs) race on it.  Serialise them.
 */
int ctcsd_tree_attention_static(void* stream, int B, int max_nodes, int Hq, int Hkv, int D,
                                const void* Q, const void* K, const void* V, int Lcap,
                                const int* kv_len, const int* n_nodes,
                                const unsigned long long* mask, float scale, void* out_O,
                                int* out_status);

#ifdef __cplusplus
}
#endif
#endif /* CTCSD_H_ */
