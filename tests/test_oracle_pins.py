"""Pins for the CPU oracle: each part is checked against something the paper or the
mathematics fixes (hand-worked cases, closed forms, library routines, a different
algorithm for the same quantity), never against a retyping of its own formula."""
import itertools
import math
import os

import numpy as np
import pytest
import torch

from oracle import ctcsd_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
BLANK = 99


def _rand_topk(rng, T, k, V, blank_rate=0.5, repeat_rate=0.5):
    """Random per-slot top-k lists over tokens 0..V-1 plus blank id V, built so that blanks
    and repeats across neighbouring slots are common."""
    ids = np.zeros((T, k), dtype=np.int64)
    lps = np.zeros((T, k), dtype=np.float64)
    for t in range(T):
        pool = list(range(V + 1))
        rng.shuffle(pool)
        row = []
        if rng.random() < blank_rate:
            row.append(V)
        if t > 0 and rng.random() < repeat_rate:
            for s in ids[t - 1]:
                if s not in row and len(row) < k and rng.random() < 0.7:
                    row.append(int(s))
        for s in pool:
            if len(row) >= k:
                break
            if s not in row:
                row.append(s)
        rng.shuffle(row)
        p = rng.dirichlet(np.ones(k + 1))[:k]           # leaves some mass outside the top-k
        order = np.argsort(-p)
        ids[t] = np.asarray(row)[order]
        lps[t] = np.log(p[order])
    return ids, lps


# ------------------------------------------------------------------ S5 collapse
def test_collapse_golden_cases():
    sym = {"_": BLANK}
    n = 0
    with open(os.path.join(GOLDEN, "ctc_collapse_cases.txt")) as f:
        for line in f:
            line = line.rstrip("\n")
            if not line.strip() or line.startswith("#"):
                continue
            lhs, rhs = line.split("->")
            a = [sym.setdefault(s, len(sym)) for s in lhs.split()]
            want = tuple(sym[s] for s in rhs.split())
            assert orc.ctc_collapse(a, BLANK) == want, line
            n += 1
    assert n >= 8


def test_collapse_properties():
    rng = np.random.default_rng(0)
    for _ in range(300):
        T = int(rng.integers(1, 9))
        a = rng.integers(0, 4, size=T).tolist()
        a = [BLANK if s == 3 else s for s in a]
        y = orc.ctc_collapse(a, BLANK)
        assert len(y) <= T and BLANK not in y
        # a blank-free, repeat-free alignment is its own image
        if BLANK not in a and all(a[i] != a[i + 1] for i in range(T - 1)):
            assert y == tuple(a)
        # two-step form: run-length merge first, blank removal second
        merged = [s for i, s in enumerate(a) if i == 0 or s != a[i - 1]]
        assert y == tuple(s for s in merged if s != BLANK)


# ------------------------------------------------------------------ S4/S6 scores
def _alpha_score(lp_t, y, blank, semiring="sum"):
    """Graves et al. forward recursion over the blank-interleaved label sequence
    (the dynamic programme the paper points to for Eq. 5).  lp_t[t][symbol] -> log prob
    (missing symbols have probability 0).  semiring 'max' gives the best alignment."""
    add = (lambda a, b: max(a, b)) if semiring == "max" else (lambda a, b: np.logaddexp(a, b))
    ext = [blank]
    for s in y:
        ext += [s, blank]
    S, T = len(ext), len(lp_t)
    get = lambda t, s: lp_t[t].get(s, -np.inf)
    alpha = np.full((T, S), -np.inf)
    alpha[0, 0] = get(0, blank)
    if S > 1:
        alpha[0, 1] = get(0, ext[1])
    for t in range(1, T):
        for s in range(S):
            v = alpha[t - 1, s]
            if s >= 1:
                v = add(v, alpha[t - 1, s - 1])
            if s >= 2 and ext[s] != blank and ext[s] != ext[s - 2]:
                v = add(v, alpha[t - 1, s - 2])
            alpha[t, s] = v + get(t, ext[s])
    out = alpha[T - 1, S - 1]
    if S > 1:
        out = add(out, alpha[T - 1, S - 2])
    return float(out)


@pytest.mark.parametrize("T,k,V", [(4, 3, 6), (5, 4, 9), (3, 2, 3), (6, 3, 5)])
def test_sum_score_is_graves_forward_and_ctc_loss(T, k, V):
    rng = np.random.default_rng(T * 100 + k)
    deduped = False
    for trial in range(4):
        ids, lps = _rand_topk(rng, T, k, V)
        cands = orc.enumerate_candidates(ids, lps, blank=V)
        lp_t = [{int(ids[t, j]): float(lps[t, j]) for j in range(k)} for t in range(T)]
        dense = torch.full((T, 1, V + 1), -float("inf"), dtype=torch.float64)
        for t in range(T):
            for j in range(k):
                dense[t, 0, ids[t, j]] = lps[t, j]
        deduped = deduped or len(cands) < k ** T
        for y, score in cands.items():
            assert score == pytest.approx(_alpha_score(lp_t, y, V), abs=1e-10)
            if len(y) > 0:
                loss = torch.nn.functional.ctc_loss(
                    dense, torch.tensor([list(y)]), torch.tensor([T]), torch.tensor([len(y)]),
                    blank=V, reduction="sum")
                assert score == pytest.approx(-float(loss), abs=1e-9)
        # sequences that were NOT produced have no alignment inside the top-k lists
        toks = sorted({int(s) for s in ids.reshape(-1) if s != V})
        for y in itertools.product(toks, repeat=2):
            if y not in cands:
                assert _alpha_score(lp_t, y, V) == -np.inf
    assert deduped                                        # several alignments really merged


def test_max_score_is_best_alignment():
    rng = np.random.default_rng(7)
    for trial in range(5):
        ids, lps = _rand_topk(rng, 5, 3, 6)
        mx = orc.enumerate_candidates(ids, lps, blank=6, score_mode=1)
        sm = orc.enumerate_candidates(ids, lps, blank=6, score_mode=0)
        lp_t = [{int(ids[t, j]): float(lps[t, j]) for j in range(3)} for t in range(5)]
        assert mx.keys() == sm.keys()
        for y in mx:
            assert mx[y] == pytest.approx(_alpha_score(lp_t, y, 6, "max"), abs=1e-10)
            assert mx[y] <= sm[y] + 1e-12


def test_total_mass_closed_form():
    # sum over all collapsed sequences of exp(score) = prod_t sum_j exp(lp[t,j])   (Eq. 1 + Eq. 6)
    rng = np.random.default_rng(3)
    for T, k, V in [(4, 3, 1000), (5, 4, 50), (2, 5, 7)]:
        ids, lps = _rand_topk(rng, T, k, V)
        cands = orc.enumerate_candidates(ids, lps, blank=V)
        total = sum(math.exp(s) for s in cands.values())
        want = float(np.prod(np.exp(lps).sum(axis=1)))
        assert total == pytest.approx(want, rel=1e-12)
    # k = V+1 on a toy vocabulary: the lists hold whole distributions, total mass is 1
    V, T = 3, 4
    z = rng.normal(size=(1, T, V + 1))
    ids, lps = orc.topk_slots(z, V + 1)
    cands = orc.enumerate_candidates(ids[0], lps[0], blank=V)
    assert sum(math.exp(s) for s in cands.values()) == pytest.approx(1.0, abs=1e-12)


def test_top_n_order_and_empty_dropped():
    cands = {(): -0.1, (5,): -1.0, (4,): -1.0, (4, 1): -1.0, (3, 9): -0.5, (7,): -3.0}
    kept = orc.select_top_n(cands, 4)
    # score desc; ties: shorter first, then lexicographic tokens; empty sequence never kept
    assert kept == [((3, 9), -0.5), ((4,), -1.0), ((5,), -1.0), ((4, 1), -1.0)]
    assert orc.selection_margin(cands, 4) == 0.0
    assert orc.selection_margin({(1,): -1.0, (2,): -1.5, (3,): -4.0}, 2) == pytest.approx(0.5)


# ------------------------------------------------------------------ S4' prefix beam
@pytest.mark.parametrize("T,k,V", [(4, 3, 6), (6, 4, 8)])
def test_prefix_beam_without_pruning_equals_enumeration(T, k, V):
    rng = np.random.default_rng(11 + T)
    for trial in range(3):
        ids, lps = _rand_topk(rng, T, k, V)
        exact = orc.enumerate_candidates(ids, lps, blank=V)
        beam = orc.prefix_beam_candidates(ids, lps, blank=V, beam=10 ** 6)
        assert beam.keys() == exact.keys()
        for y in exact:
            assert beam[y] == pytest.approx(exact[y], abs=1e-12)


def test_prefix_beam_pruned_bounds():
    rng = np.random.default_rng(5)
    for trial in range(5):
        ids, lps = _rand_topk(rng, 6, 4, 8)
        exact = orc.enumerate_candidates(ids, lps, blank=8)
        st = {}
        beam = orc.prefix_beam_candidates(ids, lps, blank=8, beam=8, stats=st)
        assert len(beam) <= 8 and st["min_cut_gap"] >= 0.0
        for y, s in beam.items():
            assert y in exact and s <= exact[y] + 1e-12
        # the best exact candidate's mass is concentrated enough to survive a beam of 8
        best = max((y for y in exact), key=lambda y: exact[y])
        assert best in beam


def _beam_trajectory_brute_force(ids, lps, blank, beam):
    """The pruned search restated over whole alignments, with no per-prefix recursion: an alignment
    of the first t slots counts at slot t iff the collapse of each of its shorter heads survived
    the cut at that slot (only survivors are ever extended).  Its probability is the product over
    the slots (Eq. 6); a prefix's mass is the sum over its alignments (Eq. 1 / Eq. 5), split by
    whether the alignment's last symbol is the blank.  Returns the survivor sets S_1..S_T as
    {prefix: (pb, pnb)} in the probability domain."""
    T, k = ids.shape
    alive = [{()}]
    out = []
    for t in range(1, T + 1):
        mass = {}
        for a in itertools.product(range(k), repeat=t):
            syms = [int(ids[s, a[s]]) for s in range(t)]
            if any(orc.ctc_collapse(syms[:s], blank) not in alive[s] for s in range(t)):
                continue
            p = math.exp(sum(float(lps[s, a[s]]) for s in range(t)))
            e = mass.setdefault(orc.ctc_collapse(syms, blank), [0.0, 0.0])
            e[0 if syms[-1] == blank else 1] += p
        ranked = sorted(mass, key=lambda y: (-(mass[y][0] + mass[y][1]), len(y), y))[:beam]
        alive.append(set(ranked))
        out.append({y: tuple(mass[y]) for y in ranked})
    return out


@pytest.mark.parametrize("T,k,V", [(5, 3, 4), (4, 3, 6), (5, 2, 3), (3, 3, 2)])
@pytest.mark.parametrize("beam", [1, 2, 3, 5])
def test_pruned_prefix_beam_follows_the_alignment_level_definition(T, k, V, beam):
    rng = np.random.default_rng(1000 * T + 10 * k + beam)
    pruned_somewhere = False
    for trial in range(6):
        ids, lps = _rand_topk(rng, T, k, V, blank_rate=0.8, repeat_rate=0.8)
        st = {}
        final = orc.prefix_beam_candidates(ids, lps, blank=V, beam=beam, stats=st)
        want = _beam_trajectory_brute_force(ids, lps, V, beam)
        assert len(st["beams"]) == T
        for t in range(T):
            got = st["beams"][t]
            assert set(got) == set(want[t]), (t, got, want[t])
            for y, (pb, pnb) in got.items():
                assert math.exp(pb) == pytest.approx(want[t][y][0], rel=1e-12, abs=1e-15)
                assert math.exp(pnb) == pytest.approx(want[t][y][1], rel=1e-12, abs=1e-15)
        assert set(final) == set(want[-1])
        for y, s in final.items():
            assert math.exp(s) == pytest.approx(sum(want[-1][y]), rel=1e-12)
        exact = orc.enumerate_candidates(ids, lps, blank=V)
        pruned_somewhere = pruned_somewhere or any(
            math.exp(final[y]) < math.exp(exact[y]) * (1 - 1e-9) for y in final) or len(final) < len(exact)
    assert pruned_somewhere


def test_pruned_prefix_beam_hand_worked_cases():
    cases, cur = [], None
    with open(os.path.join(GOLDEN, "prefix_beam_pruned_cases.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            w = line.split()
            if w[0] == "case":
                cur = dict(name=w[1], beam=int(w[3]), slots=[], after={})
                cases.append(cur)
            elif w[0] == "slot":
                cur["slots"].append([(s.split("=")[0], float(s.split("=")[1])) for s in w[1:]])
            elif w[0] == "after":
                t = int(w[1])
                entries = line.split(":", 1)[1].split(";")
                cur["after"][t] = [e.strip().split("|") for e in entries]
    assert len(cases) >= 4
    for c in cases:
        sym = {"_": BLANK}
        T, k = len(c["slots"]), len(c["slots"][0])
        ids = np.zeros((T, k), dtype=np.int64)
        lps = np.zeros((T, k))
        for t, row in enumerate(c["slots"]):
            for j, (s, p) in enumerate(row):
                ids[t, j] = sym.setdefault(s, len(sym))
                lps[t, j] = math.log(p)
        st = {}
        orc.prefix_beam_candidates(ids, lps, blank=BLANK, beam=c["beam"], stats=st)
        for t in range(1, T + 1):
            want = {}
            for pre, pb, pnb in c["after"][t]:
                y = () if pre.strip() == "-" else tuple(sym[s] for s in pre.split())
                want[y] = (float(pb), float(pnb))
            got = st["beams"][t - 1]
            assert set(got) == set(want), (c["name"], t)
            for y in want:
                assert math.exp(got[y][0]) == pytest.approx(want[y][0], abs=1e-12), (c["name"], t, y)
                assert math.exp(got[y][1]) == pytest.approx(want[y][1], abs=1e-12), (c["name"], t, y)


@pytest.mark.parametrize("beam", [0, 3])
def test_batch_wrapper_maps_rows_pads_and_reports_its_margin(beam):
    """topk_collapse: sequence b drafts from row sel_row[b] (B < M, rows permuted), unused entries
    are padded (-1 / 0 / -inf), and the margin it reports is the smallest gap its decisions relied
    on - recomputed here from scratch with a plain sort of (score, length, tokens)."""
    rng = np.random.default_rng(77 + beam)
    M, B, T, k, V, N = 5, 3, 4, 3, 5, 6
    ids = np.zeros((M, T, k), dtype=np.int64)
    lps = np.zeros((M, T, k))
    for m in range(M):
        ids[m], lps[m] = _rand_topk(rng, T, k, V, blank_rate=0.8, repeat_rate=0.8)
    sel_row = np.array([4, 0, 2])
    st = {}
    tok, ln, sc, nc = orc.topk_collapse(ids, lps, blank=V, T=T, N=N, beam=beam, sel_row=sel_row, B=B, stats=st)
    assert tok.shape == (B, N, T) and ln.shape == (B, N) and sc.shape == (B, N) and nc.shape == (B,)
    few = False
    for b in range(B):
        r = int(sel_row[b])
        if beam == 0:
            cands = orc.enumerate_candidates(ids[r], lps[r], blank=V)            # pinned above
            cut_gap = float("inf")
        else:
            traj = _beam_trajectory_brute_force(ids[r], lps[r], V, beam)        # independent of the oracle
            cands = {y: math.log(pb + pnb) for y, (pb, pnb) in traj[-1].items()}
            cut_gap = float("inf")
            # the gap at every cut: beam-th against (beam+1)-th total mass among that slot's extensions
            alive = [{()}]
            for t in range(1, T + 1):
                mass = {}
                for a in itertools.product(range(k), repeat=t):
                    syms = [int(ids[r, s, a[s]]) for s in range(t)]
                    if any(orc.ctc_collapse(syms[:s], V) not in alive[s] for s in range(t)):
                        continue
                    y = orc.ctc_collapse(syms, V)
                    mass[y] = mass.get(y, 0.0) + math.exp(sum(float(lps[r, s, a[s]]) for s in range(t)))
                order = sorted(mass, key=lambda y: (-mass[y], len(y), y))
                if len(order) > beam:
                    cut_gap = min(cut_gap, math.log(mass[order[beam - 1]]) - math.log(mass[order[beam]]))
                alive.append(set(order[:beam]))
        rows = sorted(((-s, len(y), y) for y, s in cands.items() if len(y) > 0))
        n = min(N, len(rows))
        few = few or n < N
        assert nc[b] == n
        for c in range(n):
            y = rows[c][2]
            assert ln[b, c] == len(y)
            assert tuple(tok[b, c, :len(y)]) == y and np.all(tok[b, c, len(y):] == -1)
            assert sc[b, c] == pytest.approx(-rows[c][0], abs=1e-12)
        assert np.all(tok[b, n:] == -1) and np.all(ln[b, n:] == 0) and np.all(np.isneginf(sc[b, n:]))
        gaps = [rows[i + 1][0] - rows[i][0] for i in range(min(N, len(rows) - 1))]
        want_margin = min(gaps + [cut_gap])
        assert st["margin"][b] == pytest.approx(want_margin, abs=1e-9)
        assert st["margin"][b] >= 0.0
    if beam > 0:
        assert few                                   # a beam of 3 leaves fewer than N candidates: padding is exercised
    # default mapping: no sel_row, B = M
    tok2, ln2, sc2, nc2 = orc.topk_collapse(ids, lps, blank=V, T=T, N=N, beam=beam)
    assert tok2.shape[0] == M
    np.testing.assert_array_equal(tok2[4], tok[0])
    np.testing.assert_array_equal(tok2[0], tok[1])
    np.testing.assert_array_equal(tok2[2], tok[2])


def test_a_tie_shows_up_as_a_zero_margin():
    # two alignments with equal probability that collapse to different sequences of equal length
    ids = np.array([[1, 2]], dtype=np.int64)
    lps = np.log(np.array([[0.3, 0.3]]))
    st = {}
    orc.topk_collapse(ids[None], lps[None], blank=9, T=1, N=2, stats=st)
    assert st["margin"][0] == 0.0
    st = {}
    orc.topk_collapse(ids[None], lps[None], blank=9, T=1, N=1, beam=1, stats=st)
    assert st["margin"][0] == 0.0                    # the beam cut itself sits on the tie
    # the gap between the last kept and the first dropped candidate counts too
    ids = np.array([[1, 2, 3]], dtype=np.int64)
    lps = np.log(np.array([[0.5, 0.3, 0.29]]))
    st = {}
    orc.topk_collapse(ids[None], lps[None], blank=9, T=1, N=2, stats=st)
    assert st["margin"][0] == pytest.approx(math.log(0.3 / 0.29), abs=1e-12)
    st = {}
    orc.topk_collapse(ids[None], lps[None], blank=9, T=1, N=3, stats=st)      # nothing dropped: kept pairs only
    assert st["margin"][0] == pytest.approx(math.log(0.3 / 0.29), abs=1e-12)
    st = {}
    orc.topk_collapse(ids[None], lps[None], blank=9, T=1, N=1, stats=st)
    assert st["margin"][0] == pytest.approx(math.log(0.5 / 0.3), abs=1e-12)


# ------------------------------------------------------------------ S1-S3
def test_draft_logits_against_library_and_bias_placement():
    rng = np.random.default_rng(2)
    M, H, T, V = 3, 32, 4, 10
    x = rng.normal(size=(M, H)).astype(np.float32)
    Wd = rng.normal(size=(T, V + 1, H)).astype(np.float32)
    bias = np.array([0.5, -1.0], dtype=np.float32)
    row_seq = np.array([1, 0, 1])
    z = orc.draft_logits(x, Wd, bias, row_seq)
    ref = torch.einsum("mh,tvh->mtv", torch.tensor(x, dtype=torch.float64),
                       torch.tensor(Wd, dtype=torch.float64)).numpy()
    ref[:, :, V] += bias[row_seq][:, None]
    np.testing.assert_allclose(z, ref, rtol=0, atol=1e-12)
    # hand case: H = 1, x = 2 -> logits are twice the weights, blank gets +bias
    z1 = orc.draft_logits(np.array([[2.0]]), np.array([[[1.0], [3.0], [-1.0]]]), np.array([0.25]))
    np.testing.assert_array_equal(z1, [[[2.0, 6.0, -1.75]]])


def test_log_softmax_and_topk_against_library():
    rng = np.random.default_rng(4)
    z = rng.normal(size=(2, 3, 501)) * 3.0
    lse, lp = orc.log_softmax_slots(z)
    np.testing.assert_allclose(np.exp(lp).sum(-1), 1.0, atol=1e-12)
    np.testing.assert_allclose(lp, torch.log_softmax(torch.tensor(z), -1).numpy(), atol=1e-12)
    np.testing.assert_allclose(lse, torch.logsumexp(torch.tensor(z), -1).numpy(), atol=1e-12)
    ids, lps = orc.topk_slots(z, 5)
    tv, ti = torch.topk(torch.tensor(lp), 5, dim=-1)
    np.testing.assert_array_equal(ids, ti.numpy())
    np.testing.assert_allclose(lps, tv.numpy(), atol=1e-12)
    # ties go to the lower id, blank (last id) is eligible
    zt = np.array([[[1.0, 5.0, 5.0, 0.0, 5.0]]])
    ids, _ = orc.topk_slots(zt, 4)
    assert ids.tolist() == [[[1, 2, 4, 0]]]


# ------------------------------------------------------------------ S8 tree
def _pack(cands, N, T):
    tok = np.full((1, N, T), -1, dtype=np.int64)
    ln = np.zeros((1, N), dtype=np.int64)
    for c, y in enumerate(cands):
        tok[0, c, :len(y)] = y
        ln[0, c] = len(y)
    return tok, ln, np.array([len(cands)])


def test_tree_hand_example_and_truncation():
    tok, ln, nc = _pack([(5, 6), (5, 7), (8,)], 4, 3)
    node_tok, parent, depth, pos, mask, retrieve, n = orc.build_tree(
        np.array([1]), np.array([10]), tok, ln, nc, n_max=8)
    assert n[0] == 5
    assert node_tok[0, :5].tolist() == [1, 5, 6, 7, 8]
    assert parent[0, :5].tolist() == [-1, 0, 1, 1, 0]
    assert depth[0, :5].tolist() == [0, 1, 2, 2, 1]
    assert pos[0, :5].tolist() == [10, 11, 12, 12, 11]
    assert [int(m) for m in mask[0, :5, 0]] == [0b1, 0b11, 0b111, 0b1011, 0b10001]
    assert retrieve[0, :3].tolist() == [[1, 2, -1], [1, 3, -1], [4, -1, -1]]
    # node budget 4 (root included): ids >= 4 are dropped, earlier prefixes still resolve
    node_tok, parent, depth, pos, mask, retrieve, n = orc.build_tree(
        np.array([1]), np.array([10]), tok, ln, nc, n_max=4)
    assert n[0] == 4 and node_tok[0].tolist() == [1, 5, 6, 7]
    assert retrieve[0, :3].tolist() == [[1, 2, -1], [1, 3, -1], [-1, -1, -1]]


def test_tree_invariants_against_bruteforce_trie():
    rng = np.random.default_rng(9)
    for trial in range(46):
        N, T = int(rng.integers(1, 9)), int(rng.integers(1, 6))
        n_max = int(rng.integers(2, 70))
        alphabet = 3
        if trial >= 40:                                   # large trees: masks of three and four words
            N, T, n_max, alphabet = int(rng.integers(40, 65)), 8, int(rng.integers(130, 257)), 4
        seen, cands = set(), []
        for _ in range(N):
            y = tuple(rng.integers(0, alphabet, size=int(rng.integers(1, T + 1))).tolist())
            if y not in seen:
                seen.add(y)
                cands.append(y)
        tok, ln, nc = _pack(cands, N, T)
        node_tok, parent, depth, pos, mask, retrieve, n = orc.build_tree(
            np.array([42]), np.array([100]), tok, ln, nc, n_max=n_max)
        n = int(n[0])
        prefixes = []                                     # distinct prefixes in first-seen order
        for y in cands:
            for l in range(1, len(y) + 1):
                if y[:l] not in prefixes:
                    prefixes.append(y[:l])
        assert n == min(n_max, 1 + len(prefixes))
        path = {0: ()}
        for i in range(1, n):
            assert 0 <= parent[0, i] < i
            path[i] = path[int(parent[0, i])] + (int(node_tok[0, i]),)
            assert path[i] == prefixes[i - 1]
            assert depth[0, i] == len(path[i]) and pos[0, i] == 100 + len(path[i])
        for i in range(n):                                # mask == ancestor-or-self relation
            anc, j = set(), i
            while j >= 0:
                anc.add(j)
                j = int(parent[0, j])
            bits = {j for j in range(n_max) if (int(mask[0, i, j // 64]) >> (j % 64)) & 1}
            assert bits == anc and len(bits) == depth[0, i] + 1
        for i in range(1, n):                             # siblings carry distinct tokens
            sib = [int(node_tok[0, c]) for c in range(1, n) if parent[0, c] == parent[0, i]]
            assert len(sib) == len(set(sib))
        for c, y in enumerate(cands):                     # retrieve round-trips
            for l in range(len(y)):
                r = int(retrieve[0, c, l])
                want = prefixes.index(y[:l + 1]) + 1
                assert r == (want if want < n_max else -1)
            assert all(retrieve[0, c, len(y):] == -1)


# ------------------------------------------------------------------ S9 attention
def _sdpa_ref(Q, K, V, kv_len, n_nodes, mask, scale):
    B, n_max, Hq, D = Q.shape
    grp = Hq // K.shape[1]
    O = np.zeros((B, n_max, Hq, D))
    for b in range(B):
        L, n = int(kv_len[b]), int(n_nodes[b])
        allow = torch.ones((n, L + n), dtype=torch.bool)
        for i in range(n):
            for j in range(n):
                allow[i, L + j] = bool((int(mask[b, i, j // 64]) >> (j % 64)) & 1)
        q = torch.tensor(Q[b, :n], dtype=torch.float64).permute(1, 0, 2)          # [Hq,n,D]
        k = torch.tensor(K[b, :, :L + n], dtype=torch.float64).repeat_interleave(grp, 0)
        v = torch.tensor(V[b, :, :L + n], dtype=torch.float64).repeat_interleave(grp, 0)
        o = torch.nn.functional.scaled_dot_product_attention(q, k, v, attn_mask=allow, scale=scale)
        O[b, :n] = o.permute(1, 0, 2).numpy()
    return O


def _random_tree(rng, n, n_max):
    parent = np.full(n_max, -1, dtype=np.int64)
    for i in range(1, n):
        parent[i] = rng.integers(0, i)
    W = (n_max + 63) // 64
    mask = np.zeros((n_max, W), dtype=np.uint64)
    for i in range(n):
        j = i
        while j >= 0:
            mask[i, j // 64] |= np.uint64(1) << np.uint64(j % 64)
            j = int(parent[j])
    return parent, mask


def test_attention_against_sdpa_and_special_cases():
    rng = np.random.default_rng(6)
    B, n_max, Hq, Hkv, D, Lcap = 2, 70, 4, 2, 16, 120
    Q = rng.normal(size=(B, n_max, Hq, D))
    K = rng.normal(size=(B, Hkv, Lcap, D))
    V = rng.normal(size=(B, Hkv, Lcap, D))
    kv_len = np.array([37, 5])
    n_nodes = np.array([70, 9])
    mask = np.zeros((B, n_max, 2), dtype=np.uint64)
    for b in range(B):
        _, mask[b] = _random_tree(rng, int(n_nodes[b]), n_max)
    scale = 1.0 / math.sqrt(D)
    O = orc.tree_attention(Q, K, V, kv_len, n_nodes, mask, scale)
    np.testing.assert_allclose(O, _sdpa_ref(Q, K, V, kv_len, n_nodes, mask, scale), atol=1e-12)
    assert np.all(O[1, 9:] == 0)
    # a tree above 128 nodes: four mask words
    nb = 256
    Qb = rng.normal(size=(1, nb, Hq, D))
    Kb = rng.normal(size=(1, Hkv, 300, D))
    Vb = rng.normal(size=(1, Hkv, 300, D))
    mb = np.zeros((1, nb, 4), dtype=np.uint64)
    _, mb[0] = _random_tree(rng, 231, nb)
    Ob = orc.tree_attention(Qb, Kb, Vb, np.array([41]), np.array([231]), mb, scale)
    np.testing.assert_allclose(Ob, _sdpa_ref(Qb, Kb, Vb, np.array([41]), np.array([231]), mb, scale), atol=1e-12)
    # GQA == MHA with the kv heads repeated
    O2 = orc.tree_attention(Q, np.repeat(K, 2, axis=1), np.repeat(V, 2, axis=1), kv_len, n_nodes, mask, scale)
    np.testing.assert_allclose(O, O2, atol=1e-13)
    # chain tree == causal attention over prefix + chain; single node == plain decode attention
    n = 6
    chain = np.zeros((1, n_max, 2), dtype=np.uint64)
    for i in range(n):
        chain[0, i, 0] = np.uint64((1 << (i + 1)) - 1)
    Oc = orc.tree_attention(Q[:1], K[:1], V[:1], np.array([20]), np.array([n]), chain, scale)
    for i in range(n):
        k = torch.tensor(K[0, 0, :20 + i + 1])
        v = torch.tensor(V[0, 0, :20 + i + 1])
        p = torch.softmax(k @ torch.tensor(Q[0, i, 0]) * scale, 0)
        np.testing.assert_allclose(Oc[0, i, 0], (p @ v).numpy(), atol=1e-12)


# ------------------------------------------------------------------ S10 / S11
def test_lm_head_argmax_against_library_and_ties():
    rng = np.random.default_rng(8)
    hn = rng.normal(size=(5, 16)).astype(np.float32)
    Wl = rng.normal(size=(40, 16)).astype(np.float32)
    y, am = orc.lm_head_argmax(hn, Wl)
    ref = torch.tensor(hn, dtype=torch.float64) @ torch.tensor(Wl, dtype=torch.float64).T
    np.testing.assert_allclose(y, ref.numpy(), atol=1e-12)
    np.testing.assert_array_equal(am, ref.argmax(1).numpy())
    assert orc.argmax_rows(np.array([[1.0, 7.0, 7.0, 2.0]])).tolist() == [1]


def test_greedy_accept_against_candidate_definition():
    """Definition used as the pin: the accepted length is the longest candidate prefix whose
    every token equals the base model's greedy token at the node before it."""
    rng = np.random.default_rng(10)
    for trial in range(60):
        N, T = int(rng.integers(1, 7)), int(rng.integers(1, 6))
        cands = list({tuple(rng.integers(0, 3, size=int(rng.integers(1, T + 1))).tolist()) for _ in range(N)})
        tok, ln, nc = _pack(cands, len(cands), T)
        node_tok, parent, depth, pos, mask, retrieve, n = orc.build_tree(
            np.array([1]), np.array([0]), tok, ln, nc, n_max=64)
        am = rng.integers(0, 3, size=(1, 64))
        acc_len, acc_nodes, acc_tok, next_tok = orc.greedy_accept(node_tok, parent, n, am, T)
        best = 0
        for c, y in enumerate(cands):
            l, prev = 0, 0
            while l < len(y) and am[0, prev] == y[l]:
                prev = int(retrieve[0, c, l])
                l += 1
            best = max(best, l)
        assert acc_len[0] == best <= int(depth[0, :n[0]].max()) <= T
        cur = 0
        for l in range(best):                             # accepted nodes form a root path
            nd = int(acc_nodes[0, l])
            assert parent[0, nd] == cur and node_tok[0, nd] == acc_tok[0, l] == am[0, cur]
            cur = nd
        assert next_tok[0] == am[0, cur]
        assert all(acc_nodes[0, best:] == -1) and all(acc_tok[0, best:] == -1)


def test_greedy_accept_chain_extremes():
    tok, ln, nc = _pack([(3, 4, 5, 6)], 1, 4)
    node_tok, parent, depth, pos, mask, retrieve, n = orc.build_tree(
        np.array([2]), np.array([0]), tok, ln, nc, n_max=16)
    am = np.zeros((1, 16), dtype=np.int64)
    am[0, :5] = [3, 4, 5, 6, 9]                           # full agreement along the chain
    acc_len, acc_nodes, acc_tok, next_tok = orc.greedy_accept(node_tok, parent, n, am, 4)
    assert acc_len[0] == 4 and acc_tok[0].tolist() == [3, 4, 5, 6] and next_tok[0] == 9
    am[0, 0] = 7                                          # no agreement at the root
    acc_len, acc_nodes, acc_tok, next_tok = orc.greedy_accept(node_tok, parent, n, am, 4)
    assert acc_len[0] == 0 and next_tok[0] == 7


def test_mean_accepted_length_on_a_chain_matches_the_closed_form():
    """Sec. 3.3 accepts the longest agreeing candidate.  On a chain of depth T whose every node
    agrees with the base model independently with probability p, depth d is reached with
    probability p^d, so E[acc_len] = sum_{d=1..T} p^d.  The seeded generator of the node hidden
    states, the LM-head arg-max and the acceptance walk together must reproduce that mean."""
    from paper_2412_00061_b200 import synth
    T, p, n_seeds = 5, 0.6, 2400
    cfg = synth.CONFIGS["c1"].replace(name="chain", H=64, V=40, T=T, max_nodes=8, agree_p=p)
    Wl = synth.gen_lm_head(cfg, 123)
    tok, ln, nc = _pack([(3, 4, 5, 6, 7)], 1, T)
    node_tok, parent, depth, pos, mask, retrieve, n = orc.build_tree(
        np.array([2]), np.array([0]), tok, ln, nc, n_max=cfg.max_nodes)
    assert n[0] == T + 1
    total, hist = 0, np.zeros(T + 1, dtype=np.int64)
    for seed in range(n_seeds):
        hn, target = synth.gen_node_hidden(cfg, seed, Wl, node_tok, parent, n)
        _, am = orc.lm_head_argmax(hn, Wl)
        assert np.array_equal(am[:T + 1], target[0, :T + 1])           # the planted token wins the arg-max
        acc_len, acc_nodes, acc_tok, next_tok = orc.greedy_accept(node_tok, parent, n, am.reshape(1, -1), T)
        total += int(acc_len[0])
        hist[int(acc_len[0])] += 1
    want = sum(p ** d for d in range(1, T + 1))
    var = sum((2 * d - 1) * p ** d for d in range(1, T + 1)) - want ** 2      # E[L^2] = sum (2d-1) P(L >= d)
    assert abs(total / n_seeds - want) <= 4.0 * math.sqrt(var / n_seeds)
    # the whole distribution: P(L = d) = p^d (1 - p) below the leaf, p^T at the leaf
    for d in range(T + 1):
        q = p ** d * ((1 - p) if d < T else 1.0)
        assert abs(hist[d] / n_seeds - q) <= 4.0 * math.sqrt(q * (1 - q) / n_seeds) + 1e-3


# ------------------------------------------------------------------ S12 history update
def test_commit_accepted_makes_the_accepted_path_the_prefix():
    """After the update, ordinary attention of the last accepted node over the new prefix must
    equal tree attention of that node over the old cache (prefix + its ancestors): the same
    key/value rows in both, so the two (separately pinned) attention results agree to rounding."""
    rng = np.random.default_rng(5)
    B, Hkv, Hq, D, n_max, T = 3, 2, 4, 8, 16, 4
    for trial in range(6):
        kv_len = rng.integers(1, 9, size=B)
        Lcap = int(kv_len.max()) + n_max
        # random tree: parent[i] < i
        parent = np.full((B, n_max), -1, dtype=np.int64)
        n_nodes = rng.integers(2, n_max + 1, size=B)
        mask = np.zeros((B, n_max, 1), dtype=np.uint64)
        depth = np.zeros((B, n_max), dtype=np.int64)
        for b in range(B):
            mask[b, 0, 0] = np.uint64(1)
            for i in range(1, int(n_nodes[b])):
                par = int(rng.integers(max(0, i - 3), i))
                if depth[b, par] >= T:
                    par = 0
                parent[b, i] = par
                depth[b, i] = depth[b, par] + 1
                mask[b, i, 0] = mask[b, par, 0] | np.uint64(1 << i)
        # an accepted path: walk down from the root picking children at random
        acc_len = np.zeros(B, dtype=np.int64)
        acc_nodes = np.full((B, T), -1, dtype=np.int64)
        for b in range(B):
            cur = 0
            while acc_len[b] < T:
                kids = [c for c in range(int(n_nodes[b])) if parent[b, c] == cur]
                if not kids or rng.random() < 0.2:
                    break
                cur = int(rng.choice(kids))
                acc_nodes[b, acc_len[b]] = cur
                acc_len[b] += 1
        K = rng.standard_normal((B, Hkv, Lcap, D))
        V = rng.standard_normal((B, Hkv, Lcap, D))
        Q = rng.standard_normal((B, n_max, Hq, D))
        K2, V2, new_len, sel_row = orc.commit_accepted(K, V, kv_len, acc_len, acc_nodes, n_max)
        O_tree = orc.tree_attention(Q, K, V, kv_len, n_nodes, mask, 0.3)
        for b in range(B):
            last = int(acc_nodes[b, acc_len[b] - 1]) if acc_len[b] > 0 else 0
            assert sel_row[b] == b * n_max + last
            assert new_len[b] == kv_len[b] + 1 + acc_len[b]
            # the last accepted node as a one-node "tree" on top of the new prefix
            q1 = np.zeros((1, n_max, Hq, D))
            q1[0, 0] = Q[b, last]
            one = orc.tree_attention(q1, K2[b:b + 1], V2[b:b + 1], np.array([new_len[b] - 1]), np.array([1]),
                                     np.ones((1, n_max, 1), dtype=np.uint64), 0.3)
            np.testing.assert_allclose(one[0, 0], O_tree[b, last], rtol=1e-12, atol=1e-12)
            # nothing below the tree rows changes; a chain 1,2,..,k is already in place
            assert np.array_equal(K2[b, :, :kv_len[b] + 1], K[b, :, :kv_len[b] + 1])
            if list(acc_nodes[b, :acc_len[b]]) == list(range(1, int(acc_len[b]) + 1)):
                assert np.array_equal(K2[b], K[b]) and np.array_equal(V2[b], V[b])


def test_commit_accepted_reads_the_cache_as_it_was():
    # accepted nodes 2 then 3: row L+1 <- row L+2, row L+2 <- row L+3 (the old row L+2 must be read first)
    K = np.arange(2 * 1 * 8 * 1, dtype=np.float64).reshape(2, 1, 8, 1)
    V = -K
    K2, V2, new_len, sel = orc.commit_accepted(K, V, np.array([2, 1]), np.array([2, 0]),
                                               np.array([[2, 3], [-1, -1]]), 4)
    assert K2[0, 0, :, 0].tolist() == [0, 1, 2, 4, 5, 5, 6, 7]
    assert V2[0, 0, :, 0].tolist() == [0, -1, -2, -4, -5, -5, -6, -7]
    assert np.array_equal(K2[1], K[1]) and new_len.tolist() == [5, 2] and sel.tolist() == [3, 4]


# ------------------------------------------------------------------ sampling acceptance
def _sequential_rule_distribution(p, children):
    """Sec. 2's rule written out for a deterministic proposal, with exact probabilities: the
    children of a node are tried one after the other; a tried child is accepted with probability
    min(1, P(c) / P'(c)) where P' is the point mass on c; after a rejection P becomes
    norm(max(0, P - P')), i.e. P without c.  If every child is rejected a token is drawn from what
    is left.  Returns the probability of every token being the one emitted after this node."""
    p = np.asarray(p, dtype=np.float64).copy()
    out = np.zeros_like(p)
    reach = 1.0                                   # probability that the trials get this far
    for c in children:
        a = min(1.0, p[c] / 1.0)
        out[c] += reach * a
        reach *= 1.0 - a
        resid = np.maximum(0.0, p - np.eye(len(p))[c])
        p = resid / resid.sum()
    out += reach * p
    return out


def test_sequential_acceptance_with_point_mass_proposals_emits_the_target_distribution():
    rng = np.random.default_rng(21)
    for _ in range(20):
        V = int(rng.integers(3, 8))
        p = rng.dirichlet(np.ones(V))
        kids = list(rng.permutation(V)[:int(rng.integers(1, V))])
        np.testing.assert_allclose(_sequential_rule_distribution(p, kids), p, atol=1e-12)


def test_sample_tokens_draws_from_the_softmax_and_a_chain_accepts_with_the_product_rule():
    """The oracle's rule (one Gumbel-max draw per node, accepted iff it is a child) against the
    distribution the sequential rule emits (= the target distribution, test above): frequencies
    over many noise draws, and the accepted length on a chain against prod_d P_d(child_d)."""
    from paper_2412_00061_b200 import synth
    V, T, n = 5, 3, 4
    cfg = synth.CONFIGS["c1"].replace(name="samp", B=1, V=V, T=T, max_nodes=n)
    rng = np.random.default_rng(5)
    y = rng.normal(size=(1, n, V)) * 1.5
    inv_temp = 1.0 / 0.7
    tok, ln, nc = _pack([(2, 0, 3)], 1, T)
    node_tok, parent, depth, pos, mask, retrieve, nn = orc.build_tree(np.array([1]), np.array([0]), tok, ln, nc, n_max=n)
    probs = torch.softmax(torch.tensor(y[0]) * inv_temp, -1).numpy()          # [n,V] target distributions
    trials = 20000
    first = np.zeros(V)
    lens = np.zeros(T + 1)
    for s in range(trials):
        g = synth.gen_gumbel_noise(cfg, s)
        x, acc_len, acc_nodes, acc_tok, next_tok = orc.sample_accept(node_tok, parent, nn, depth, y, g, inv_temp, T)
        first[x[0, 0]] += 1
        lens[acc_len[0]] += 1
    want_first = probs[0]
    assert np.all(np.abs(first / trials - want_first) <= 4 * np.sqrt(want_first * (1 - want_first) / trials) + 1e-3)
    a = [probs[0, 2], probs[1, 0], probs[2, 3]]                                # P_d(child_d) along the chain
    want_len = [1 - a[0], a[0] * (1 - a[1]), a[0] * a[1] * (1 - a[2]), a[0] * a[1] * a[2]]
    for d in range(T + 1):
        q = want_len[d]
        assert abs(lens[d] / trials - q) <= 4 * math.sqrt(q * (1 - q) / trials) + 1e-3


def test_sampling_acceptance_special_cases():
    from paper_2412_00061_b200 import synth
    rng = np.random.default_rng(6)
    V, T, n = 9, 4, 16
    cfg = synth.CONFIGS["c1"].replace(name="samp2", B=2, V=V, T=T, max_nodes=n)
    cands = [(1, 2, 3), (1, 4), (5,)]
    tok, ln, nc = _pack(cands, 3, T)
    tok, ln, nc = np.repeat(tok, 2, 0), np.repeat(ln, 2, 0), np.repeat(nc, 2, 0)
    node_tok, parent, depth, pos, mask, retrieve, nn = orc.build_tree(np.array([0, 0]), np.array([0, 0]), tok, ln, nc, n_max=n)
    y = rng.normal(size=(2, n, V))
    g = synth.gen_gumbel_noise(cfg, 3)
    # temperature -> 0: the draw is the arg-max, acceptance is the greedy one
    cold = orc.sample_accept(node_tok, parent, nn, depth, y, g, 1e9, T)
    am = np.argmax(y, axis=-1)
    for got, want in zip(cold[1:], orc.greedy_accept(node_tok, parent, nn, am, T)):
        np.testing.assert_array_equal(got, want)
    # a target that puts all its mass on a child's token (P = P', the point mass): always accepted
    y2 = np.full((2, n, V), -50.0)
    for b in range(2):
        y2[b, 0, 1] = y2[b, 1, 2] = y2[b, 2, 3] = 50.0
    for s in range(10):
        out = orc.sample_accept(node_tok, parent, nn, depth, y2, synth.gen_gumbel_noise(cfg, s), 1.0, T)
        assert out[1].tolist() == [3, 3] and out[3][0].tolist() == [1, 2, 3, -1]
    # nodes of equal depth share their noise, nodes along a path do not; the float32 decision differs
    # from the float64 one only through rounding
    x64 = orc.sample_tokens(y, depth, nn, g, 1.3)
    x32 = orc.sample_tokens(y, depth, nn, g, 1.3, fp32=True)
    assert np.mean(x64 == x32) > 0.9
    i, j = 2, 4                                              # nodes (1,2) and (1,4): both depth 2
    assert depth[0, i] == depth[0, j] == 2
    same_logits = y.copy()
    same_logits[0, j] = same_logits[0, i]
    xs = orc.sample_tokens(same_logits, depth, nn, g, 1.3)
    assert xs[0, i] == xs[0, j]


# ------------------------------------------------------------------ the attention draft module
def _draft_module_case(rng, B=2, R=3, H=32, Hq=4, Hkv=2, D=8, I=48, Lcap=24, zero=False):
    sc = 0.0 if zero else 0.3
    w = dict(g1=rng.normal(size=H) * 0.2 + 1.0, g2=rng.normal(size=H) * 0.2 + 1.0,
             Wqkv=rng.normal(size=((Hq + 2 * Hkv) * D, H)) * 0.3, Wo=rng.normal(size=(H, Hq * D)) * sc,
             Wgu=rng.normal(size=(2 * I, H)) * 0.3, Wdn=rng.normal(size=(H, I)) * sc)
    F = rng.normal(size=(B, R, H))
    n_new = rng.integers(1, R + 1, size=B)
    kv_len = rng.integers(0, 9, size=B)
    Kd = rng.normal(size=(B, Hkv, Lcap, D))
    Vd = rng.normal(size=(B, Hkv, Lcap, D))
    return w, F, n_new, kv_len, Kd, Vd, (Hq, Hkv, D, I)


def _torch_layer_reference(F, n_new, kv_len, Kd, Vd, w, Hq, Hkv, D, eps, theta):
    """The same layer out of library pieces: F.rms_norm, rotary embedding as complex multiplication
    on (x_i, x_{i+D/2}) pairs, scaled_dot_product_attention, F.silu."""
    import torch.nn.functional as Fn
    t = lambda a: torch.tensor(np.asarray(a), dtype=torch.float64)
    B, R, H = F.shape
    I = w["Wdn"].shape[1]
    out = np.zeros((B, H))
    Kd, Vd = t(Kd).clone(), t(Vd).clone()

    def rope(x, pos):                                  # x [heads, D]
        half = D // 2
        freqs = theta ** (-2.0 * torch.arange(half, dtype=torch.float64) / D)
        rot = torch.polar(torch.ones(half, dtype=torch.float64), pos * freqs)
        z = torch.complex(x[:, :half], x[:, half:]) * rot
        return torch.cat([z.real, z.imag], dim=1)

    for b in range(B):
        L, r = int(kv_len[b]), int(n_new[b])
        for j in range(r):
            a = Fn.rms_norm(t(F[b, j]), (H,), t(w["g1"]), eps)
            qkv = t(w["Wqkv"]) @ a
            q = rope(qkv[:Hq * D].reshape(Hq, D), L + j)
            Kd[b, :, L + j] = rope(qkv[Hq * D:(Hq + Hkv) * D].reshape(Hkv, D), L + j)
            Vd[b, :, L + j] = qkv[(Hq + Hkv) * D:].reshape(Hkv, D)
        n = L + r
        k = Kd[b, :, :n].repeat_interleave(Hq // Hkv, 0)
        v = Vd[b, :, :n].repeat_interleave(Hq // Hkv, 0)
        o = Fn.scaled_dot_product_attention(q[:, None, :], k, v)[:, 0, :]
        h1 = t(F[b, r - 1]) + t(w["Wo"]) @ o.reshape(-1)
        m = Fn.rms_norm(h1, (H,), t(w["g2"]), eps)
        gu = t(w["Wgu"]) @ m
        out[b] = (h1 + t(w["Wdn"]) @ (Fn.silu(gu[:I]) * gu[I:])).numpy()
    return out, Kd.numpy(), Vd.numpy()


def test_draft_module_against_library_pieces():
    rng = np.random.default_rng(31)
    for trial in range(4):
        w, F, n_new, kv_len, Kd, Vd, (Hq, Hkv, D, I) = _draft_module_case(rng)
        got = orc.draft_module(F, n_new, kv_len, Kd, Vd, w, Hq, Hkv, D, eps=1e-5, theta=10000.0)
        want = _torch_layer_reference(F, n_new, kv_len, Kd, Vd, w, Hq, Hkv, D, 1e-5, 10000.0)
        np.testing.assert_allclose(got[0], want[0], atol=1e-11)
        np.testing.assert_allclose(got[1], want[1], atol=1e-12)
        np.testing.assert_allclose(got[2], want[2], atol=1e-12)
        np.testing.assert_array_equal(got[3], kv_len + n_new)
        for b in range(F.shape[0]):                    # nothing but the new rows of the cache changes
            L, r = int(kv_len[b]), int(n_new[b])
            assert np.array_equal(got[1][b, :, :L], Kd[b, :, :L]) and np.array_equal(got[1][b, :, L + r:], Kd[b, :, L + r:])


def test_draft_module_special_cases():
    rng = np.random.default_rng(32)
    # output projections at zero: both residual branches vanish, the layer is the identity on the
    # newest hidden state, so drafting from its output equals drafting from the hidden state itself
    w, F, n_new, kv_len, Kd, Vd, (Hq, Hkv, D, I) = _draft_module_case(rng, zero=True)
    F_hat, _, _, _ = orc.draft_module(F, n_new, kv_len, Kd, Vd, w, Hq, Hkv, D)
    last = np.stack([F[b, n_new[b] - 1] for b in range(F.shape[0])])
    np.testing.assert_allclose(F_hat, last, atol=1e-15)
    Wd = rng.normal(size=(3, 11, F.shape[2]))
    np.testing.assert_allclose(orc.draft_logits(F_hat, Wd), orc.draft_logits(last, Wd), atol=1e-12)
    # the attention inside the layer is the (separately pinned) tree attention of a one-node tree
    w, F, n_new, kv_len, Kd, Vd, (Hq, Hkv, D, I) = _draft_module_case(rng, B=1, R=2)
    w["Wdn"] = np.zeros_like(w["Wdn"])                 # MLP off: F_hat = h + Wo attn
    F_hat, K2, V2, L2 = orc.draft_module(F, n_new, kv_len, Kd, Vd, w, Hq, Hkv, D)
    r, L = int(n_new[0]), int(kv_len[0])
    a = orc.rms_norm(F[0, r - 1], w["g1"], 1e-5)
    q = (w["Wqkv"] @ a)[:Hq * D].reshape(Hq, D)
    Q = np.zeros((1, 4, Hq, D))
    Q[0, 0] = np.stack([orc.rope_rotate(q[h], L + r - 1, 10000.0) for h in range(Hq)])
    one = orc.tree_attention(Q, K2, V2, np.array([L + r - 1]), np.array([1]), np.ones((1, 4, 1), dtype=np.uint64),
                             1.0 / math.sqrt(D))
    np.testing.assert_allclose(F_hat[0], F[0, r - 1] + w["Wo"] @ one[0, 0].reshape(-1), atol=1e-12)
    # the optional storage rounding: the identity changes nothing, bfloat16 moves the output by a few 1e-3
    from paper_2412_00061_b200 import synth
    w, F, n_new, kv_len, Kd, Vd, (Hq, Hkv, D, I) = _draft_module_case(rng)
    plain = orc.draft_module(F, n_new, kv_len, Kd, Vd, w, Hq, Hkv, D)
    same = orc.draft_module(F, n_new, kv_len, Kd, Vd, w, Hq, Hkv, D, store=lambda a: a.astype(np.float64))
    np.testing.assert_allclose(same[0], plain[0], atol=1e-5)            # (float32 round trip of the stored vectors)
    rounded = orc.draft_module(F, n_new, kv_len, Kd, Vd, w, Hq, Hkv, D, store=synth.round_bf16)
    assert 0 < np.max(np.abs(rounded[0] - plain[0])) < 0.2
    np.testing.assert_array_equal(rounded[1][0, :, int(kv_len[0])], synth.round_bf16(rounded[1][0, :, int(kv_len[0])].astype(np.float32)))
    # rotary embedding: a rotation (norm kept), position 0 is the identity, relative-position property
    v, u = rng.normal(size=D), rng.normal(size=D)
    np.testing.assert_allclose(orc.rope_rotate(v, 0, 10000.0), v, atol=0)
    assert abs(np.linalg.norm(orc.rope_rotate(v, 17, 10000.0)) - np.linalg.norm(v)) < 1e-12
    d1 = orc.rope_rotate(v, 9, 10000.0) @ orc.rope_rotate(u, 4, 10000.0)
    d2 = orc.rope_rotate(v, 25, 10000.0) @ orc.rope_rotate(u, 20, 10000.0)
    assert abs(d1 - d2) < 1e-10


# ------------------------------------------------------------------ chained steps
def _chain_case(seed, n_steps, p=0.8):
    from paper_2412_00061_b200 import synth
    cfg = synth.CONFIGS["c1"].replace(name="chain", B=2, H=48, V=30, T=3, k=3, topN=6, max_nodes=12, Hq=2, Hkv=1,
                                      D=8, kv_lo=2, kv_hi=6, agree_p=p)
    big = synth.chain_cache_config(cfg, n_steps)
    x0, Wd, bb = synth.gen_draft(cfg, seed)
    base_tok, kv_len = synth.gen_base(cfg, seed)
    _, K, V = synth.gen_attention(big, seed)
    Wl = synth.gen_lm_head(cfg, seed)
    Qtab, Ktab, Vtab = synth.gen_chain_tables(cfg, seed, n_steps)
    hidden = lambda s, tree: synth.gen_node_hidden(cfg, synth.chain_step_seed(seed, s), Wl, tree[0], tree[1], tree[6])[0]
    out = orc.decode_chain(n_steps, x0, base_tok, kv_len, Wd, bb, Wl, K, V, lambda s: Qtab[s],
                           lambda s: (Ktab[s], Vtab[s]), hidden, cfg.T, cfg.k, cfg.topN, cfg.max_nodes)
    return cfg, (x0, base_tok, kv_len, K, V, Qtab, Ktab, Vtab), out


def test_chained_steps_leave_exactly_the_emitted_tokens_in_the_cache():
    """What a chain of steps must amount to, stated without the loop: the cache grows by each step's
    root and accepted nodes, in order, and nothing else moves; every step starts where the previous
    one stopped (root = previous bonus token, drafting state = hidden state of the last accepted
    node); and the tree attention an accepted node saw equals ordinary causal attention of its
    query over the final cache up to its own row (the rows before it are exactly its prefix)."""
    n_steps, accepted = 5, 0
    for seed in (0, 1, 2):
        cfg, (x0, base_tok, kv_len0, K0, V0, Qtab, Ktab, Vtab), (recs, K, V, kv_len) = _chain_case(seed, n_steps)
        n_max = cfg.max_nodes
        for b in range(cfg.B):
            L0 = int(kv_len0[b])
            rows_k, rows_v, queries = [], [], []
            for s, r in enumerate(recs):
                path = [0] + [int(v) for v in r["acc_nodes"][b, :r["acc_len"][b]]]
                accepted += len(path) - 1
                for node in path:
                    rows_k.append(Ktab[s][b, :, node])
                    rows_v.append(Vtab[s][b, :, node])
                    queries.append((s, node))
                assert r["kv_len"][b] == L0 + len(rows_k) - len(path)
                if s + 1 < n_steps:
                    assert recs[s + 1]["base_tok"][b] == r["next_tok"][b]
                    np.testing.assert_array_equal(recs[s + 1]["x"][b], r["hn"][b * n_max + path[-1]])
            assert kv_len[b] == L0 + len(rows_k) == L0 + sum(int(r["acc_len"][b]) + 1 for r in recs)
            np.testing.assert_array_equal(K[b, :, :L0], K0[b, :, :L0])
            np.testing.assert_array_equal(K[b, :, L0:L0 + len(rows_k)], np.stack(rows_k, axis=1))
            np.testing.assert_array_equal(V[b, :, L0:L0 + len(rows_v)], np.stack(rows_v, axis=1))
            for i, (s, node) in enumerate(queries):
                for h in range(cfg.Hq):
                    q = torch.tensor(Qtab[s][b, node, h], dtype=torch.float64)
                    kk = torch.tensor(K[b, 0, :L0 + i + 1], dtype=torch.float64)
                    vv = torch.tensor(V[b, 0, :L0 + i + 1], dtype=torch.float64)
                    pr = torch.softmax(kk @ q / math.sqrt(cfg.D), 0)
                    np.testing.assert_allclose(recs[s]["O"][b, node, h], (pr @ vv).numpy(), atol=1e-12)
    assert accepted >= 10                                  # the chains really accept draft tokens


def test_a_chain_of_one_step_is_the_single_step():
    cfg, (x0, base_tok, kv_len0, K0, V0, Qtab, Ktab, Vtab), (recs, K, V, kv_len) = _chain_case(3, 1)
    r = recs[0]
    from paper_2412_00061_b200 import synth
    x, Wd, bb = synth.gen_draft(cfg, 3)
    ids, lps = orc.topk_slots(orc.draft_logits(x, Wd, bb), cfg.k)
    np.testing.assert_array_equal(r["topk_id"], ids)
    ctok, clen, _, nc = orc.topk_collapse(ids, lps, cfg.V, cfg.T, cfg.topN)
    tree = orc.build_tree(base_tok, kv_len0, ctok, clen, nc, cfg.max_nodes)
    for name, want in zip(["node_tok", "parent", "depth", "pos", "mask", "retrieve", "n_nodes"], tree):
        np.testing.assert_array_equal(r[name], want)


# ------------------------------------------------------------------ the paper's raw-tree layout
def test_raw_paths_are_the_most_probable_alignments():
    rng = np.random.default_rng(11)
    ids, lps = _rand_topk(rng, 4, 3, 7)
    raw, score = orc.select_raw_paths(ids, lps, 10)
    # brute force with a different mechanism: score every alignment with numpy, stable argsort
    idx = np.array(list(itertools.product(range(3), repeat=4)))
    tot = lps[np.arange(4)[None, :], idx].sum(axis=1)
    order = np.argsort(-tot, kind="stable")[:10]
    np.testing.assert_array_equal(raw, ids[np.arange(4)[None, :], idx[order]])
    np.testing.assert_allclose(score, tot[order], rtol=0, atol=1e-12)
    assert np.all(np.diff(score) <= 1e-15)


def test_raw_tree_masks_exactly_the_tokens_the_ctc_transform_removes():
    """Along every root-to-node path of the raw tree, the kept nodes spell the CTC collapse of the
    raw prefix (the pinned collapse function), the attention mask holds the root plus those kept
    nodes, and the position counts them."""
    rng = np.random.default_rng(12)
    V = 5
    for trial in range(8):
        T, k, N = 5, 3, 12
        ids, lps = _rand_topk(rng, T, k, V, blank_rate=0.7, repeat_rate=0.8)
        raw, _ = orc.select_raw_paths(ids, lps, N)
        raw_tok = raw[None]
        out = orc.build_raw_tree(np.array([3]), np.array([10]), raw_tok, np.array([N]), V, 64)
        node_tok, parent, depth, pos, mask, retrieve, n_nodes, kept, nka = out
        n = int(n_nodes[0])
        for c in range(N):
            for l in range(1, T + 1):
                i = int(retrieve[0, c, l - 1])
                want = orc.ctc_collapse(raw[c, :l].tolist(), V)
                path = []
                j = i
                while j > 0:
                    path.append(j)
                    j = int(parent[0, j])
                path.reverse()
                got = tuple(int(node_tok[0, j]) for j in path if kept[0, j])
                assert got == want
                bits = {j for j in range(n) if (int(mask[0, i, 0]) >> j) & 1}
                assert bits == {0} | {j for j in path if kept[0, j]}
                assert pos[0, i] == 10 + len(want)
                kept_anc = [j for j in [0] + path[:-1] if j == 0 or kept[0, j]]
                assert nka[0, i] == kept_anc[-1]
        assert kept[0, 0] == 1 and nka[0, 0] == -1


def test_raw_accept_is_the_longest_collapsed_candidate_that_agrees():
    """Brute force over the raw paths: collapse each one, count how many of its tokens agree with
    the base model's greedy choice after the (collapsed) prefix, take the longest."""
    rng = np.random.default_rng(13)
    V = 4
    for trial in range(30):
        T, k, N = 5, 3, 14
        ids, lps = _rand_topk(rng, T, k, V, blank_rate=0.7, repeat_rate=0.8)
        raw, _ = orc.select_raw_paths(ids, lps, N)
        out = orc.build_raw_tree(np.array([1]), np.array([0]), raw[None], np.array([N]), V, 64)
        node_tok, parent, depth, pos, mask, retrieve, n_nodes, kept, nka = out
        n = int(n_nodes[0])
        # the base model's greedy token is a function of the collapsed prefix only
        table = {}
        def nxt(prefix):
            if prefix not in table:
                table[prefix] = int(rng.integers(0, V))
            return table[prefix]
        am = np.zeros((1, 64), dtype=np.int64)
        for i in range(n):
            path = []
            j = i
            while j > 0:
                path.append(j)
                j = int(parent[0, j])
            path.reverse()
            am[0, i] = nxt(tuple(int(node_tok[0, j]) for j in path if kept[0, j]))
        acc_len, acc_nodes, acc_tok, next_tok = orc.raw_accept(node_tok, kept, nka, n_nodes, am, T)
        best = ()
        for c in range(N):
            y = orc.ctc_collapse(raw[c].tolist(), V)
            l = 0
            while l < len(y) and y[l] == nxt(y[:l]):
                l += 1
            if l > len(best):
                best = y[:l]
        assert acc_len[0] == len(best)
        # greedy agreement determines the tokens uniquely: every agreeing prefix is the same sequence
        assert tuple(int(v) for v in acc_tok[0, :acc_len[0]]) == best
        assert next_tok[0] == nxt(best)
        assert all(kept[0, int(i)] for i in acc_nodes[0, :acc_len[0]])
