"""CPU oracle for the CTC-drafted draft-and-verify step.  TEST INFRASTRUCTURE ONLY.

A plain, slow, fp64/int64 restatement of what one decoding step computes, written from
the paper's definitions so that it can be checked against them by eye.  It shares no
code with the CUDA path and must never be imported by it: only the tests, the smoke
check and the benchmark's CPU-baseline leg may call into this file.

Each function names the passage it follows.  Notation is the paper's: T draft slots
("places"), blank symbol (the paper's epsilon) with id V, alignment a = (a_1..a_T),
beta^{-1} the collapse map, Y the collapsed candidate.

Pins (see tests/test_oracle_pins.py): every function below is pinned by something other
than itself - hand-worked collapse cases, the total-mass closed form, the Graves forward
recursion (torch's ctc_loss and an independent alpha recursion), library matmul /
log-softmax / top-k / scaled-dot-product attention in fp64, brute-force tries and
acceptance definitions, the closed-form mean accepted length on a chain, and - for the
history update - the equality of ordinary attention over the updated prefix with tree
attention over the old cache, plus a hand-worked overlap case.  The finite-beam prefix
search is a heuristic the paper does not specify (Sec. 3.3 only says that the most valuable
combinations are kept): WHICH pruning rule is used is this build's reading; HOW it executes
is pinned - with a beam that never prunes to exact enumeration, with a pruning beam to an
alignment-level brute force of the survivor sets after every slot (masses split by the last
symbol), to hand-worked cases with the arithmetic written out (tests/golden/), ties at the
cut included.  The batch wrapper topk_collapse (row mapping, padding, decision margin) is
pinned against per-sequence enumeration and an independent sort.
"""
from __future__ import annotations

import itertools
import math
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

NEG_INF = float("-inf")


# --------------------------------------------------------------------------------------
# S1  draft head: per-slot logits (Sec. 3.2: the projected draft features give one
#     distribution per place; here the projection is a linear head over V+1 classes)
# --------------------------------------------------------------------------------------
def draft_logits(x: np.ndarray, Wd: np.ndarray, blank_bias: Optional[np.ndarray] = None,
                 row_seq: Optional[np.ndarray] = None) -> np.ndarray:
    """z[m,t,v] = sum_h x[m,h] * Wd[t,v,h]; the blank class v = V additionally gets
    blank_bias[row_seq[m]].  x [M,H], Wd [T,V+1,H] -> z [M,T,V+1] in fp64."""
    x64 = np.asarray(x, dtype=np.float64)
    M = x64.shape[0]
    T, V1, _ = Wd.shape
    z = np.empty((M, T, V1), dtype=np.float64)
    for t in range(T):
        z[:, t, :] = x64 @ np.asarray(Wd[t], dtype=np.float64).T
    if blank_bias is not None:
        for m in range(M):
            s = m if row_seq is None else int(row_seq[m])
            z[m, :, V1 - 1] += float(blank_bias[s])
    return z


# --------------------------------------------------------------------------------------
# S2  per-slot log-softmax (Sec. 3.2: P_hat = Softmax(...), one distribution per place)
# --------------------------------------------------------------------------------------
def log_softmax_slots(z: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """lse[m,t] = log sum_v exp z[m,t,v];  lp = z - lse."""
    z = np.asarray(z, dtype=np.float64)
    mx = z.max(axis=-1, keepdims=True)
    lse = mx + np.log(np.exp(z - mx).sum(axis=-1, keepdims=True))
    return lse[..., 0], z - lse


# --------------------------------------------------------------------------------------
# S3  per-slot top-k (Sec. 3.3: each place keeps its k most probable symbols, best first,
#     k fixed in advance); blank is eligible; ties go to the lower id
# --------------------------------------------------------------------------------------
def topk_slots(z: np.ndarray, k: int) -> Tuple[np.ndarray, np.ndarray]:
    """Returns (topk_id [M,T,k] int64, topk_lp [M,T,k] fp64) with lp = z - lse."""
    z = np.asarray(z, dtype=np.float64)
    lse, _ = log_softmax_slots(z)
    order = np.argsort(-z, axis=-1, kind="stable")[..., :k]   # stable: equal values keep id order
    vals = np.take_along_axis(z, order, axis=-1)
    return order.astype(np.int64), vals - lse[..., None]


# --------------------------------------------------------------------------------------
# S5  CTC collapse beta^{-1} (Sec. 2.3 and Sec. 3.1, CTC Transform Module: runs of one
#     repeated symbol shrink to a single symbol, then every blank is deleted)
# --------------------------------------------------------------------------------------
def ctc_collapse(a: Sequence[int], blank: int) -> Tuple[int, ...]:
    out: List[int] = []
    prev = None
    for s in a:
        s = int(s)
        if s != prev and s != blank:      # compared with the previous RAW symbol, blank included
            out.append(s)
        prev = s
    return tuple(out)


def _logaddexp(a: float, b: float) -> float:
    if a == NEG_INF:
        return b
    if b == NEG_INF:
        return a
    hi, lo = (a, b) if a >= b else (b, a)
    return hi + math.log1p(math.exp(lo - hi))


# --------------------------------------------------------------------------------------
# S4 + S6  enumerate every slot path, score it (Eq. 6: P(A) = prod_t p(a_t)), collapse it,
#          and give each distinct collapsed sequence the sum over its alignments
#          (Eq. 1 / Eq. 5: P(Y) = sum_{A in beta(Y)} P(A))
# --------------------------------------------------------------------------------------
def enumerate_candidates(topk_id: np.ndarray, topk_lp: np.ndarray, blank: int,
                         score_mode: int = 0) -> Dict[Tuple[int, ...], float]:
    """topk_id, topk_lp: [T,k] for one drafting row.  Returns {collapsed sequence: log score},
    the empty sequence included.  score_mode 0: log sum exp over alignments; 1: best alignment."""
    T, k = topk_id.shape
    groups: Dict[Tuple[int, ...], List[float]] = {}
    for a in itertools.product(range(k), repeat=T):
        s = 0.0
        for t in range(T):
            s += float(topk_lp[t, a[t]])
        y = ctc_collapse([int(topk_id[t, a[t]]) for t in range(T)], blank)
        groups.setdefault(y, []).append(s)
    out: Dict[Tuple[int, ...], float] = {}
    for y, ss in groups.items():
        m = max(ss)
        if score_mode == 1:
            out[y] = m
        else:
            out[y] = m + math.log(sum(math.exp(s - m) for s in ss))
    return out


def order_o1(item: Tuple[Tuple[int, ...], float]):
    """Total order on candidates: score descending, then shorter first, then token ids
    lexicographically ascending (the paper is silent on ties)."""
    y, score = item
    return (-score, len(y), y)


# --------------------------------------------------------------------------------------
# S7  keep the N best non-empty candidates (Sec. 3.3: only the most valuable of the
#     combined sequences go on to verification)
# --------------------------------------------------------------------------------------
def select_top_n(cands: Dict[Tuple[int, ...], float], N: int) -> List[Tuple[Tuple[int, ...], float]]:
    items = [(y, s) for y, s in cands.items() if len(y) > 0]
    items.sort(key=order_o1)
    return items[:N]


def selection_margin(cands: Dict[Tuple[int, ...], float], N: int) -> float:
    """Smallest score gap that the top-N selection relied on: between adjacent kept
    candidates and between the last kept and the first dropped one (inf if none)."""
    items = [(y, s) for y, s in cands.items() if len(y) > 0]
    items.sort(key=order_o1)
    gaps = [items[i][1] - items[i + 1][1] for i in range(min(N, len(items) - 1))]
    return min(gaps) if gaps else float("inf")


# --------------------------------------------------------------------------------------
# S4'  CTC prefix beam search restricted to each slot's top-k symbols.  The paper gives no
#      pruning rule; this is the textbook prefix search (probability mass of a prefix split
#      into alignments ending in blank / ending in its last token), pruned to `beam`
#      prefixes after every slot.
# --------------------------------------------------------------------------------------
def prefix_beam_candidates(topk_id: np.ndarray, topk_lp: np.ndarray, blank: int, beam: int,
                           stats: Optional[dict] = None) -> Dict[Tuple[int, ...], float]:
    """Returns {prefix: log(pb + pnb)} for the prefixes alive after the last slot."""
    T, k = topk_id.shape
    cur: Dict[Tuple[int, ...], Tuple[float, float]] = {(): (0.0, NEG_INF)}   # (log pb, log pnb)
    min_cut_gap = float("inf")
    beams: List[Dict[Tuple[int, ...], Tuple[float, float]]] = []             # the beam after every slot
    for t in range(T):
        nxt: Dict[Tuple[int, ...], List[float]] = {}

        def acc(prefix, which, val):
            if val == NEG_INF:                              # no alignment reaches it: not a prefix
                return
            e = nxt.setdefault(prefix, [NEG_INF, NEG_INF])
            e[which] = _logaddexp(e[which], val)

        for prefix, (pb, pnb) in cur.items():
            tot = _logaddexp(pb, pnb)
            for j in range(k):
                s = int(topk_id[t, j])
                p = float(topk_lp[t, j])
                if s == blank:
                    acc(prefix, 0, tot + p)                 # stays, now ends in blank
                elif len(prefix) > 0 and s == prefix[-1]:
                    acc(prefix, 1, pnb + p)                 # repeat merges into the same prefix
                    acc(prefix + (s,), 1, pb + p)           # a blank in between starts a new token
                else:
                    acc(prefix + (s,), 1, tot + p)
        ranked = sorted(((y, _logaddexp(e[0], e[1])) for y, e in nxt.items()),
                        key=lambda it: (-it[1], len(it[0]), it[0]))
        if len(ranked) > beam:
            min_cut_gap = min(min_cut_gap, ranked[beam - 1][1] - ranked[beam][1])
        cur = {y: (nxt[y][0], nxt[y][1]) for y, _ in ranked[:beam]}
        beams.append(dict(cur))
    if stats is not None:
        stats["min_cut_gap"] = min_cut_gap
        stats["beams"] = beams
    return {y: _logaddexp(pb, pnb) for y, (pb, pnb) in cur.items()}


def topk_collapse(topk_id: np.ndarray, topk_lp: np.ndarray, blank: int, T: int, N: int,
                  beam: int = 0, score_mode: int = 0, sel_row: Optional[np.ndarray] = None,
                  B: Optional[int] = None, stats: Optional[dict] = None):
    """S4-S7 for a batch.  topk_id/topk_lp: [M,T,k]; sequence b drafts from row sel_row[b]
    (default b).  Returns cand_tok [B,N,T] (pad -1), cand_len [B,N], cand_score [B,N]
    (pad -inf), n_cand [B]."""
    M = topk_id.shape[0]
    B = M if B is None else B
    cand_tok = np.full((B, N, T), -1, dtype=np.int64)
    cand_len = np.zeros((B, N), dtype=np.int64)
    cand_score = np.full((B, N), NEG_INF, dtype=np.float64)
    n_cand = np.zeros((B,), dtype=np.int64)
    margins = []
    for b in range(B):
        r = b if sel_row is None else int(sel_row[b])
        st: dict = {}
        if beam > 0:
            cands = prefix_beam_candidates(topk_id[r], topk_lp[r], blank, beam, st)
        else:
            cands = enumerate_candidates(topk_id[r], topk_lp[r], blank, score_mode)
        margins.append(min(selection_margin(cands, N), st.get("min_cut_gap", float("inf"))))
        kept = select_top_n(cands, N)
        n_cand[b] = len(kept)
        for c, (y, s) in enumerate(kept):
            cand_len[b, c] = len(y)
            cand_tok[b, c, :len(y)] = y
            cand_score[b, c] = s
    if stats is not None:
        stats["margin"] = margins
    return cand_tok, cand_len, cand_score, n_cand


# --------------------------------------------------------------------------------------
# S8  token tree (Sec. 2.2: candidates are root-to-leaf paths of a tree verified in one
#     pass under a tree attention mask; Sec. 3.3: the base token precedes the drafts)
# --------------------------------------------------------------------------------------
def build_tree(base_tok: np.ndarray, kv_len: np.ndarray, cand_tok: np.ndarray,
               cand_len: np.ndarray, n_cand: np.ndarray, n_max: int):
    """Prefix trie of the ranked candidates under a root that holds the base token.
    Nodes are numbered in order of first appearance while walking candidates by rank and
    each candidate left to right; a new node is made only while fewer than n_max exist.
    mask bit j of row i is set iff j is i or an ancestor of i."""
    B, N, T = cand_tok.shape
    W = (n_max + 63) // 64
    node_tok = np.full((B, n_max), -1, dtype=np.int64)
    parent = np.full((B, n_max), -1, dtype=np.int64)
    depth = np.zeros((B, n_max), dtype=np.int64)
    pos = np.zeros((B, n_max), dtype=np.int64)
    mask = np.zeros((B, n_max, W), dtype=np.uint64)
    retrieve = np.full((B, N, T), -1, dtype=np.int64)
    n_nodes = np.zeros((B,), dtype=np.int64)
    for b in range(B):
        node_of: Dict[Tuple[int, ...], int] = {(): 0}
        node_tok[b, 0] = int(base_tok[b])
        n = 1
        for c in range(int(n_cand[b])):
            for l in range(1, int(cand_len[b, c]) + 1):
                pre = tuple(int(v) for v in cand_tok[b, c, :l])
                if pre not in node_of:
                    if pre[:-1] not in node_of or n >= n_max:
                        break                                  # budget hit: rest of this candidate is dropped
                    node_of[pre] = n
                    node_tok[b, n] = pre[-1]
                    parent[b, n] = node_of[pre[:-1]]
                    depth[b, n] = l
                    n += 1
                retrieve[b, c, l - 1] = node_of[pre]
        n_nodes[b] = n
        for i in range(n):
            pos[b, i] = int(kv_len[b]) + depth[b, i]
            j = i
            while j >= 0:
                mask[b, i, j // 64] |= np.uint64(1) << np.uint64(j % 64)
                j = int(parent[b, j])
    return node_tok, parent, depth, pos, mask, retrieve, n_nodes


# --------------------------------------------------------------------------------------
# S9  tree attention: plain softmax(q k^T / sqrt(d)) v over the cached prefix (all
#     visible) and the tree nodes allowed by the ancestor mask (Sec. 2.2, Sec. 3.3)
# --------------------------------------------------------------------------------------
def tree_attention(Q: np.ndarray, K: np.ndarray, Vc: np.ndarray, kv_len: np.ndarray,
                   n_nodes: np.ndarray, mask: np.ndarray, scale: float) -> np.ndarray:
    """Q [B,n_max,Hq,D]; K,Vc [B,Hkv,Lcap,D] with node j's key/value at row kv_len[b]+j.
    Query head h reads kv head h // (Hq/Hkv).  Returns O [B,n_max,Hq,D] fp64 (dead rows 0)."""
    B, n_max, Hq, D = Q.shape
    Hkv = K.shape[1]
    grp = Hq // Hkv
    O = np.zeros((B, n_max, Hq, D), dtype=np.float64)
    for b in range(B):
        L, n = int(kv_len[b]), int(n_nodes[b])
        for h in range(Hq):
            Kh = np.asarray(K[b, h // grp, :L + n], dtype=np.float64)
            Vh = np.asarray(Vc[b, h // grp, :L + n], dtype=np.float64)
            for i in range(n):
                q = np.asarray(Q[b, i, h], dtype=np.float64)
                s = (Kh @ q) * scale
                vis = np.ones(L + n, dtype=bool)
                for j in range(n):
                    bit = (int(mask[b, i, j // 64]) >> (j % 64)) & 1
                    vis[L + j] = bool(bit)
                s = np.where(vis, s, NEG_INF)
                p = np.exp(s - s.max())
                p /= p.sum()
                O[b, i, h] = p @ Vh
    return O


# --------------------------------------------------------------------------------------
# S10  LM head and greedy token at every tree node (Eq. 3-4 form: argmax Softmax(LmHead(F)))
# --------------------------------------------------------------------------------------
def lm_head_argmax(hn: np.ndarray, Wl: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """y[m,v] = sum_h hn[m,h] Wl[v,h]; am[m] = argmax_v y[m,v] (lowest id on ties)."""
    y = np.asarray(hn, dtype=np.float64) @ np.asarray(Wl, dtype=np.float64).T
    return y, np.argmax(y, axis=1).astype(np.int64)


def argmax_rows(y: np.ndarray) -> np.ndarray:
    return np.argmax(np.asarray(y, dtype=np.float64), axis=1).astype(np.int64)


# --------------------------------------------------------------------------------------
# S11  greedy acceptance (Sec. 2.2: only sequences matching the target model's greedy
#      output are accepted; Sec. 3.3: the longest such sequence is the step's output)
# --------------------------------------------------------------------------------------
def greedy_accept(node_tok: np.ndarray, parent: np.ndarray, n_nodes: np.ndarray,
                  am: np.ndarray, T: int):
    """am [B,n_max]: base model's greedy token after each node.  Walk down from the root:
    move to the child whose token equals am[current]; stop when no child matches.
    Returns acc_len [B], acc_nodes [B,T] (pad -1), acc_tok [B,T] (pad -1), next_tok [B]."""
    B = node_tok.shape[0]
    acc_len = np.zeros((B,), dtype=np.int64)
    acc_nodes = np.full((B, T), -1, dtype=np.int64)
    acc_tok = np.full((B, T), -1, dtype=np.int64)
    next_tok = np.zeros((B,), dtype=np.int64)
    for b in range(B):
        cur = 0
        while True:
            want = int(am[b, cur])
            nxt = -1
            for c in range(int(n_nodes[b])):
                if int(parent[b, c]) == cur and int(node_tok[b, c]) == want:
                    nxt = c
                    break
            if nxt < 0 or acc_len[b] >= T:
                break
            acc_nodes[b, acc_len[b]] = nxt
            acc_tok[b, acc_len[b]] = want
            acc_len[b] += 1
            cur = nxt
        next_tok[b] = int(am[b, cur])
    return acc_len, acc_nodes, acc_tok, next_tok


# --------------------------------------------------------------------------------------
# S12  history update after acceptance (Sec. 3.3, last paragraph: the step's output is
#      appended to the decoding history): the accepted path becomes part of the cached prefix
# --------------------------------------------------------------------------------------
def commit_accepted(K: np.ndarray, Vc: np.ndarray, kv_len: np.ndarray, acc_len: np.ndarray,
                    acc_nodes: np.ndarray, max_nodes: int):
    """K, Vc [B,Hkv,Lcap,D] with tree node j of sequence b at cache row kv_len[b]+j.  The root
    (row kv_len[b]) stays; the l-th accepted node's key/value row moves to row kv_len[b]+1+l,
    read from the cache as it was before the call.  Returns (K', V', kv_len' = kv_len+1+acc_len,
    sel_row [B] = b*max_nodes + last accepted node (the root if nothing was accepted): the tree
    row whose hidden state the next step drafts from)."""
    K2, V2 = np.array(K, copy=True), np.array(Vc, copy=True)
    B = K.shape[0]
    new_len = np.zeros((B,), dtype=np.int64)
    sel_row = np.zeros((B,), dtype=np.int64)
    for b in range(B):
        L = int(kv_len[b])
        last = 0
        for l in range(int(acc_len[b])):
            node = int(acc_nodes[b, l])
            K2[b, :, L + 1 + l, :] = K[b, :, L + node, :]
            V2[b, :, L + 1 + l, :] = Vc[b, :, L + node, :]
            last = node
        new_len[b] = L + 1 + int(acc_len[b])
        sel_row[b] = b * max_nodes + last
    return K2, V2, new_len, sel_row


# --------------------------------------------------------------------------------------
# The paper's own verification layout (Sec. 3.1 "CTC Transform Module", Sec. 3.3): the raw,
# fixed-length slot paths stay in the token tree; the tokens that the CTC transform removes
# (blanks, and repeats of the previous slot's symbol) are masked out of the attention map
# instead of being dropped from the tree.
# --------------------------------------------------------------------------------------
def select_raw_paths(topk_id: np.ndarray, topk_lp: np.ndarray, N: int):
    """The N most probable slot paths of one sequence (Sec. 3.3: the raw candidates are the most
    valuable combinations of the per-place symbols): path probability = product over the
    slots (Eq. 6); equal scores go to the path that is first when the per-slot ranks are read as
    a number (slot 1 most significant).  topk_id/topk_lp [T,k] -> (raw_tok [n,T], score [n])."""
    T, k = topk_id.shape
    paths = []
    for idx, a in enumerate(itertools.product(range(k), repeat=T)):
        s = 0.0
        for t in range(T):
            s += float(topk_lp[t, a[t]])
        paths.append((-s, idx, a))
    paths.sort(key=lambda e: (e[0], e[1]))
    keep = paths[:N]
    raw = np.array([[int(topk_id[t, a[t]]) for t in range(T)] for _, _, a in keep], dtype=np.int64).reshape(len(keep), T)
    score = np.array([-ns for ns, _, _ in keep], dtype=np.float64)
    return raw, score


def build_raw_tree(base_tok: np.ndarray, kv_len: np.ndarray, raw_tok: np.ndarray, n_raw: np.ndarray,
                   blank: int, n_max: int):
    """Token tree over the raw paths raw_tok [B,N,T] (symbols include the blank).  The trie is
    the one build_tree makes; on top of it:
      kept[i]   - node i survives the CTC transform: its symbol is not the blank and differs from
                  its parent's symbol (the root, which holds the base token, is not part of the
                  alignment: a first-slot symbol is kept iff it is not the blank; the root is kept);
      mask[i]   - bit j set iff j is the root or a kept ancestor of i, or j == i and i is kept
                  (the removed tokens' positions are masked in the attention map);
      pos[i]    - kv_len + number of kept non-root nodes on the path root..i;
      nka[i]    - nearest kept proper ancestor of i (-1 for the root)."""
    B, N, T = raw_tok.shape
    raw_len = np.full((B, N), T, dtype=np.int64)
    node_tok, parent, depth, _, anc, retrieve, n_nodes = build_tree(base_tok, kv_len, raw_tok, raw_len, n_raw, n_max)
    W = (n_max + 63) // 64
    kept = np.zeros((B, n_max), dtype=np.int64)
    nka = np.full((B, n_max), -1, dtype=np.int64)
    pos = np.zeros((B, n_max), dtype=np.int64)
    mask = np.zeros((B, n_max, W), dtype=np.uint64)
    for b in range(B):
        for i in range(int(n_nodes[b])):
            if i == 0:
                kept[b, 0] = 1
            else:
                par = int(parent[b, i])
                s = int(node_tok[b, i])
                prev = None if par == 0 else int(node_tok[b, par])
                kept[b, i] = 1 if (s != blank and s != prev) else 0
            path = []
            j = i
            while j >= 0:
                path.append(j)
                j = int(parent[b, j])
            count = 0
            for j in path:
                if j == 0 or kept[b, j]:
                    mask[b, i, j // 64] |= np.uint64(1) << np.uint64(j % 64)
                    if j != 0:
                        count += 1
            pos[b, i] = int(kv_len[b]) + count
            for j in path[1:]:
                if j == 0 or kept[b, j]:
                    nka[b, i] = j
                    break
    return node_tok, parent, depth, pos, mask, retrieve, n_nodes, kept, nka


def raw_accept(node_tok: np.ndarray, kept: np.ndarray, nka: np.ndarray, n_nodes: np.ndarray,
               am: np.ndarray, T: int):
    """Greedy acceptance on the raw tree (Sec. 3.3: of the candidates that pass verification the
    longest one is the output).  am[b,i] is the base model's greedy token after kept node i.  A kept node d
    follows kept node p when p is d's nearest kept ancestor (removed nodes in between are
    transparent).  best[p] = longest chain p -> d1 -> d2 ... with node_tok[d] == am[previous];
    among equally long continuations the lowest node id wins.
    Returns acc_len [B], acc_nodes [B,T] (kept node ids, pad -1), acc_tok [B,T], next_tok [B]."""
    B = node_tok.shape[0]
    acc_len = np.zeros((B,), dtype=np.int64)
    acc_nodes = np.full((B, T), -1, dtype=np.int64)
    acc_tok = np.full((B, T), -1, dtype=np.int64)
    next_tok = np.zeros((B,), dtype=np.int64)
    for b in range(B):
        n = int(n_nodes[b])
        best = [0] * n
        succ = [-1] * n
        for p in range(n - 1, -1, -1):                # children have larger ids than their ancestors
            if not kept[b, p]:
                continue
            for d in range(p + 1, n):
                if kept[b, d] and int(nka[b, d]) == p and int(node_tok[b, d]) == int(am[b, p]):
                    if 1 + best[d] > best[p]:
                        best[p] = 1 + best[d]
                        succ[p] = d
        cur = 0
        while succ[cur] >= 0 and acc_len[b] < T:
            cur = succ[cur]
            acc_nodes[b, acc_len[b]] = cur
            acc_tok[b, acc_len[b]] = int(node_tok[b, cur])
            acc_len[b] += 1
        next_tok[b] = int(am[b, cur])
    return acc_len, acc_nodes, acc_tok, next_tok


# --------------------------------------------------------------------------------------
# Several decoding steps in a row (Sec. 3.3 describes one step and ends with the history
# update; Eq. 11 counts tokens per step over such a loop).  A plain loop over the functions
# above, nothing else: step s drafts from the base model's hidden state at the last accepted
# node of step s-1, its root is the bonus token of step s-1, and it runs on the cache that
# commit_accepted left.
# --------------------------------------------------------------------------------------
def decode_chain(n_steps: int, x0: np.ndarray, base_tok0: np.ndarray, kv_len0: np.ndarray,
                 Wd: np.ndarray, blank_bias: Optional[np.ndarray], Wl: np.ndarray,
                 K: np.ndarray, Vc: np.ndarray, q_of_step, kv_of_step, hidden_of_step,
                 T: int, k: int, N: int, n_max: int, beam: int = 0, score_mode: int = 0,
                 scale: Optional[float] = None):
    """x0 [B,H]: hidden states the first step drafts from; base_tok0, kv_len0 [B].
    K, Vc [B,Hkv,Lcap,D]: the cache (copied, not modified).  The base model's per-step outputs
    are supplied by the caller:
      q_of_step(s)            -> Q [B,n_max,Hq,D], the tree nodes' queries;
      kv_of_step(s)           -> (Kt, Vt) [B,Hkv,n_max,D], the tree nodes' keys/values, which are
                                 written to cache rows kv_len[b]+j for every j < n_max;
      hidden_of_step(s, tree) -> hn [B*n_max,H], the tree nodes' final hidden states (tree is the
                                 tuple build_tree returned, so the caller can plant agreement).
    Returns (records, K, Vc, kv_len): one dict per step with every intermediate result."""
    B = x0.shape[0]
    V = Wl.shape[0]
    K, Vc = np.array(K, copy=True), np.array(Vc, copy=True)
    kv_len = np.asarray(kv_len0, dtype=np.int64).copy()
    base_tok = np.asarray(base_tok0, dtype=np.int64).copy()
    x = np.asarray(x0)
    records = []
    for s in range(n_steps):
        z = draft_logits(x, Wd, blank_bias)
        ids, lps = topk_slots(z, k)
        st: dict = {}
        ctok, clen, cscore, ncand = topk_collapse(ids, lps, V, T, N, beam, score_mode, stats=st)
        tree = build_tree(base_tok, kv_len, ctok, clen, ncand, n_max)
        node_tok, parent, depth, pos, mask, retrieve, n_nodes = tree
        Kt, Vt = kv_of_step(s)
        for b in range(B):
            L = int(kv_len[b])
            K[b, :, L:L + n_max, :] = Kt[b]
            Vc[b, :, L:L + n_max, :] = Vt[b]
        Q = q_of_step(s)
        D = Q.shape[-1]
        O = tree_attention(Q, K, Vc, kv_len, n_nodes, mask, (1.0 / math.sqrt(D)) if scale is None else scale)
        hn = hidden_of_step(s, tree)
        y, am = lm_head_argmax(hn, Wl)
        am = am.reshape(B, n_max)
        acc_len, acc_nodes, acc_tok, next_tok = greedy_accept(node_tok, parent, n_nodes, am, T)
        rec = dict(x=x, base_tok=base_tok.copy(), kv_len=kv_len.copy(), z=z, topk_id=ids, topk_lp=lps,
                   cand_tok=ctok, cand_len=clen, cand_score=cscore, n_cand=ncand, margin=st["margin"],
                   node_tok=node_tok, parent=parent, depth=depth, pos=pos, mask=mask, retrieve=retrieve,
                   n_nodes=n_nodes, O=O, hn=hn, argmax=am, acc_len=acc_len, acc_nodes=acc_nodes,
                   acc_tok=acc_tok, next_tok=next_tok)
        K, Vc, kv_len, sel_row = commit_accepted(K, Vc, kv_len, acc_len, acc_nodes, n_max)
        rec["new_kv_len"], rec["sel_row"] = kv_len.copy(), sel_row
        records.append(rec)
        x = hn[sel_row]                       # the next step drafts from the last accepted node's hidden state
        base_tok = next_tok.copy()            # and its root is this step's bonus token
    return records, K, Vc, kv_len


# --------------------------------------------------------------------------------------
# Sampling acceptance (Sec. 2, second paragraph: a drafted token is accepted with probability
# min(1, p/p') - the paper typesets the ratio upside down - and on rejection a token is drawn
# from norm(max(0, P - P')); Sec. 6 names sampling as future work).
#
# Reading.  The tree's tokens are a deterministic function of the draft head's output (the k
# best symbols per place, the N best candidates), so the proposal P' for a child that is tried
# is the point mass on that child's token: p' = 1, the child is accepted with probability
# P(child), and after a rejection P - P' clipped at zero and renormalised is P without that
# token.  Trying the children of a node one after the other under this rule emits child c
# with probability P(c) and any other token x with probability P(x): exactly one draw from
# P, accepted iff it is a child.  That is what is computed here, with the draw made by the
# Gumbel-max rule so that it is a deterministic function of noise the caller passes in:
#     x[b,i] = argmax_v ( y[b,i,v] / temperature + noise[b, depth(i), v] ),   noise ~ Gumbel(0,1)
# (nodes of equal depth lie on different paths, at most one of them is reached, so they may
# share their noise; nodes along one path use independent noise).  The acceptance walk is
# the greedy one with x in place of the arg-max.  temperature -> 0 gives greedy acceptance.
# --------------------------------------------------------------------------------------
def sample_tokens(y: np.ndarray, depth: np.ndarray, n_nodes: np.ndarray, noise: np.ndarray,
                  inv_temperature: float, fp32: bool = False) -> np.ndarray:
    """y [B,n_max,V] logits, depth [B,n_max], noise [B,T+1,V] -> x [B,n_max] int64 (dead nodes 0).
    fp32=True forms y * inv_temperature + noise as one fused multiply-add rounded to float32
    (the precision in which the CUDA path takes this decision), else in float64."""
    B, n_max, V = y.shape
    x = np.zeros((B, n_max), dtype=np.int64)
    it = np.float64(np.float32(inv_temperature)) if fp32 else np.float64(inv_temperature)
    for b in range(B):
        for i in range(int(n_nodes[b])):
            z = np.asarray(y[b, i], dtype=np.float64) * it + np.asarray(noise[b, int(depth[b, i])], dtype=np.float64)
            if fp32:
                z = z.astype(np.float32)
            x[b, i] = int(np.argmax(z))              # first maximum: lowest id on ties
    return x


def sample_accept(node_tok: np.ndarray, parent: np.ndarray, n_nodes: np.ndarray, depth: np.ndarray,
                  y: np.ndarray, noise: np.ndarray, inv_temperature: float, T: int, fp32: bool = False):
    """Returns (x, acc_len, acc_nodes, acc_tok, next_tok): the base model's sampled token after
    every node and the accepted path (next_tok is the sampled token at the last accepted node)."""
    x = sample_tokens(y, depth, n_nodes, noise, inv_temperature, fp32)
    return (x,) + tuple(greedy_accept(node_tok, parent, n_nodes, x, T))


# --------------------------------------------------------------------------------------
# The paper's Attention Draft Module (Sec. 3.1: one transformer layer, built like the base
# model's layers, on the base model's hidden states; Sec. 3.2: F_hat = DraftModule(F), then the
# projection to one distribution per place).  The paper gives no further detail.  Reading taken:
# a LLaMA-style decoder layer with the base model's head shape (pre-norm residual blocks: RMSNorm,
# rotary self-attention over the hidden states of all positions so far, RMSNorm, SwiGLU MLP), no
# final norm; the layer's output at the newest position is the state that draft_logits projects
# to the T places.  Keys and values of earlier positions are cached, as in the base model.
# --------------------------------------------------------------------------------------
def rms_norm(x: np.ndarray, gamma: np.ndarray, eps: float) -> np.ndarray:
    """y = x / sqrt(mean(x^2) + eps) * gamma over the last axis."""
    x = np.asarray(x, dtype=np.float64)
    return x / np.sqrt((x * x).mean(axis=-1, keepdims=True) + eps) * np.asarray(gamma, dtype=np.float64)


def rope_rotate(v: np.ndarray, pos: int, theta: float) -> np.ndarray:
    """Rotary position embedding of one head vector v [D] at position pos, half-split pairing
    (element i is paired with i + D/2, frequency theta^(-2i/D)), the LLaMA convention."""
    v = np.asarray(v, dtype=np.float64)
    D = v.shape[-1]
    half = D // 2
    out = np.empty_like(v)
    for i in range(half):
        ang = pos * theta ** (-2.0 * i / D)
        c, s = math.cos(ang), math.sin(ang)
        out[i] = v[i] * c - v[i + half] * s
        out[i + half] = v[i + half] * c + v[i] * s
    return out


def draft_module(F_new: np.ndarray, n_new: np.ndarray, kv_len: np.ndarray, Kd: np.ndarray, Vd: np.ndarray,
                 w: dict, Hq: int, Hkv: int, D: int, eps: float = 1e-5, theta: float = 10000.0, store=None):
    """One step of the draft layer.  F_new [B,R,H]: the base model's hidden states of the newest
    n_new[b] <= R positions of each sequence (positions kv_len[b] .. kv_len[b]+n_new[b]-1; the
    layer's cache Kd, Vd [B,Hkv,Lcap,D] already holds positions < kv_len[b]).  w: g1 [H], Wqkv
    [(Hq+2Hkv)D, H] (query rows first, then key rows, then value rows), Wo [H, Hq*D], g2 [H],
    Wgu [2I, H] (gate rows, then up rows), Wdn [H, I].
    store: None, or a function that rounds an array to the storage type of the activations (e.g.
    to bfloat16).  A mixed-precision implementation keeps the four activation vectors that feed a
    projection - the normalised input, the attention output, the normalised h1, the SwiGLU product -
    in that type, as it keeps the cached keys and values; with `store` the same four vectors (and
    the cached rows) are rounded here too, everything else stays float64.
    Returns (F_hat [B,H]: the layer's output at each sequence's newest position, Kd', Vd' with the
    new positions' keys/values appended, kv_len' = kv_len + n_new)."""
    st = (lambda a: a) if store is None else (lambda a: np.asarray(store(np.asarray(a, dtype=np.float32)), dtype=np.float64))
    F_new = np.asarray(F_new, dtype=np.float64)
    B, R, H = F_new.shape
    Kd, Vd = np.array(Kd, dtype=np.float64, copy=True), np.array(Vd, dtype=np.float64, copy=True)
    Wqkv, Wo = np.asarray(w["Wqkv"], dtype=np.float64), np.asarray(w["Wo"], dtype=np.float64)
    Wgu, Wdn = np.asarray(w["Wgu"], dtype=np.float64), np.asarray(w["Wdn"], dtype=np.float64)
    I = Wdn.shape[1]
    grp = Hq // Hkv
    F_hat = np.zeros((B, H), dtype=np.float64)
    new_len = np.zeros((B,), dtype=np.int64)
    for b in range(B):
        L, r = int(kv_len[b]), int(n_new[b])
        q_last = None
        for j in range(r):
            a = st(rms_norm(F_new[b, j], w["g1"], eps))
            qkv = Wqkv @ a
            q = qkv[:Hq * D].reshape(Hq, D)
            k = qkv[Hq * D:(Hq + Hkv) * D].reshape(Hkv, D)
            v = qkv[(Hq + Hkv) * D:].reshape(Hkv, D)
            for g in range(Hkv):
                Kd[b, g, L + j] = st(rope_rotate(k[g], L + j, theta))
                Vd[b, g, L + j] = st(v[g])
            q_last = st(np.stack([rope_rotate(q[h], L + j, theta) for h in range(Hq)]))
        n_keys = L + r
        attn = np.zeros((Hq, D))
        for h in range(Hq):                          # the newest position attends to every position so far
            s = (Kd[b, h // grp, :n_keys] @ q_last[h]) / math.sqrt(D)
            p = np.exp(s - s.max())
            p /= p.sum()
            attn[h] = p @ Vd[b, h // grp, :n_keys]
        h1 = F_new[b, r - 1] + Wo @ st(attn).reshape(-1)
        m = st(rms_norm(h1, w["g2"], eps))
        gu = Wgu @ m
        gate, up = gu[:I], gu[I:]
        act = st(gate / (1.0 + np.exp(-gate)) * up)   # SiLU(gate) * up
        F_hat[b] = h1 + Wdn @ act
        new_len[b] = n_keys
    return F_hat, Kd, Vd, new_len
