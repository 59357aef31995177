"""Seeded synthetic inputs for the draft-and-verify step.

This module only draws random numbers and shapes them; it performs none of the
method's arithmetic (no projections, soft-max, collapse, tree or attention code
lives here).  The CPU oracle's tests and the CUDA path's tests/benchmark both
take their inputs from here so that the two sides see identical values.

Every array is produced on the host with numpy's PCG64 generator, keyed by
``(seed, stream tag)`` so that one tensor's values do not depend on whether
another tensor was drawn first.  Floating-point tensors are returned as
``float32`` arrays whose values are exactly representable in the run dtype
(``bf16`` values are rounded to nearest-even on the upper 16 bits), which lets
the fp64 oracle and the bf16 kernels start from bit-identical operands.

The five named workloads mirror the shapes of LLaMA/Vicuna-family decoding steps
(hidden size, heads, 32000-token vocabulary plus one CTC blank); the paper's
datasets and trained weights are not available, so weights are N(0, 0.02^2) and
hidden states N(0, 1).
"""
from __future__ import annotations

import dataclasses
from dataclasses import dataclass
from typing import Dict, Optional, Tuple

import numpy as np

_TAGS = {"x": 1, "Wd": 2, "bias": 3, "base": 4, "kvlen": 5, "Q": 6, "K": 7, "V": 8,
         "Wl": 9, "hn_noise": 10, "agree": 11, "repeat": 12, "gumbel": 13,
         "dm_g1": 14, "dm_g2": 15, "dm_qkv": 16, "dm_o": 17, "dm_gu": 18, "dm_dn": 19, "dm_F": 20, "dm_K": 21,
         "dm_V": 22, "dm_n": 23, "dm_len": 24}


@dataclass(frozen=True)
class StepConfig:
    """Shape of one draft-and-verify step (names follow the paper's notation:
    T draft slots, k tokens kept per slot, blank id = V)."""
    name: str
    B: int            # sequences
    H: int            # hidden size
    V: int            # vocabulary size (blank id = V, so V + 1 draft classes)
    T: int            # draft slots
    k: int            # top-k per slot
    beam: int         # 0 = enumerate all k^T slot paths, >0 = CTC prefix beam width
    topN: int         # collapsed candidates kept
    max_nodes: int    # tree node budget per sequence, root included
    Hq: int
    Hkv: int
    D: int
    kv_lo: int        # cached tokens per sequence drawn uniformly in [kv_lo, kv_hi]
    kv_hi: int
    dtype: str        # "fp32" | "bf16"
    agree_p: float = 0.6
    blank_bias: Tuple[float, ...] = (1.0,)   # cycled over sequences (shuffled by the seed)
    score_mode: int = 0                      # 0 = sum over alignments, 1 = best alignment

    @property
    def Lcap(self) -> int:
        # cache capacity: longest prefix plus room for the tree rows, rounded up to 64
        return ((self.kv_hi + self.max_nodes + 63) // 64) * 64

    def replace(self, **kw) -> "StepConfig":
        return dataclasses.replace(self, **kw)


CONFIGS: Dict[str, StepConfig] = {
    # tiny CPU-seconds instance, fp32 throughout
    "c1": StepConfig("c1", B=1, H=256, V=1000, T=4, k=3, beam=0, topN=8, max_nodes=32,
                     Hq=4, Hkv=4, D=64, kv_lo=128, kv_hi=128, dtype="fp32", agree_p=0.6),
    # Vicuna-7B-shaped step (the headline workload)
    "c2": StepConfig("c2", B=1, H=4096, V=32000, T=5, k=4, beam=0, topN=16, max_nodes=64,
                     Hq=32, Hkv=32, D=128, kv_lo=1024, kv_hi=1024, dtype="bf16", agree_p=0.6),
    # 7B shape, batch 8, ragged KV lengths, prefix beam
    "c3": StepConfig("c3", B=8, H=4096, V=32000, T=6, k=4, beam=64, topN=16, max_nodes=64,
                     Hq=32, Hkv=32, D=128, kv_lo=512, kv_hi=2048, dtype="bf16", agree_p=0.6,
                     blank_bias=(0.0, 1.0, 2.0)),
    # Vicuna-13B-shaped step
    "c4": StepConfig("c4", B=4, H=5120, V=32000, T=8, k=5, beam=128, topN=32, max_nodes=128,
                     Hq=40, Hkv=40, D=128, kv_lo=4096, kv_hi=4096, dtype="bf16", agree_p=0.5),
    # GQA 70B-shaped stress step
    "c5": StepConfig("c5", B=32, H=8192, V=32000, T=6, k=4, beam=64, topN=16, max_nodes=64,
                     Hq=64, Hkv=8, D=128, kv_lo=1024, kv_hi=4096, dtype="bf16", agree_p=0.6),
    # the 7B shape with a large tree: 64 candidates of up to 6 tokens, 256 nodes
    "c6": StepConfig("c6", B=1, H=4096, V=32000, T=6, k=4, beam=0, topN=64, max_nodes=256,
                     Hq=32, Hkv=32, D=128, kv_lo=1024, kv_hi=1024, dtype="bf16", agree_p=0.6),
}


def _rng(seed: int, tag: str) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64([int(seed), _TAGS[tag]]))


def round_bf16(a: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bfloat16 (ties to even); result stays float32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32)
    out = np.empty_like(u)
    step = 1 << 24
    flat_in, flat_out = u.reshape(-1), out.reshape(-1)
    for s in range(0, flat_in.size, step):
        c = flat_in[s:s + step]
        flat_out[s:s + step] = (c + (((c >> 16) & 1) + 0x7FFF)) & 0xFFFF0000
    return out.view(np.float32)


def to_dtype(a: np.ndarray, dtype: str) -> np.ndarray:
    if dtype == "bf16":
        return round_bf16(a)
    if dtype == "fp32":
        return np.ascontiguousarray(a, dtype=np.float32)
    raise ValueError(dtype)


def _normal(seed: int, tag: str, shape, std: float, dtype: str) -> np.ndarray:
    g = _rng(seed, tag)
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.float32)
    step = 1 << 24
    for s in range(0, n, step):
        e = min(n, s + step)
        g.standard_normal(e - s, dtype=np.float32, out=out[s:e])
    if std != 1.0:
        out *= np.float32(std)
    return to_dtype(out.reshape(shape), dtype)


def gen_draft(cfg: StepConfig, seed: int = 0, M: Optional[int] = None,
              force_repeats: bool = False):
    """x [M,H] ~ N(0,1); Wd [T,V+1,H] ~ N(0,0.02^2) (hidden axis contiguous);
    blank_bias [B] float32.  ``force_repeats`` copies each slot's blank row onto a
    scaled mix of its neighbour so that repeats and blanks show up more often."""
    M = cfg.B if M is None else M
    x = _normal(seed, "x", (M, cfg.H), 1.0, cfg.dtype)
    Wd = _normal(seed, "Wd", (cfg.T, cfg.V + 1, cfg.H), 0.02, cfg.dtype)
    if force_repeats:
        # make slot t+1 favour the same tokens as slot t: copy a band of rows across slots
        g = _rng(seed, "repeat")
        rows = g.choice(cfg.V, size=min(64, cfg.V), replace=False)
        for t in range(1, cfg.T):
            Wd[t, rows, :] = Wd[0, rows, :]
    bb = np.asarray(cfg.blank_bias, dtype=np.float32)
    idx = np.arange(cfg.B) % len(bb)
    _rng(seed, "bias").shuffle(idx)
    blank_bias = bb[idx].astype(np.float32)
    return x, Wd, blank_bias


def gen_base(cfg: StepConfig, seed: int = 0):
    """base_tok [B] uniform in [0,V); kv_len [B] uniform integer in [kv_lo, kv_hi]."""
    base_tok = _rng(seed, "base").integers(0, cfg.V, size=cfg.B).astype(np.int32)
    kv_len = _rng(seed, "kvlen").integers(cfg.kv_lo, cfg.kv_hi + 1, size=cfg.B).astype(np.int32)
    return base_tok, kv_len


def gen_attention(cfg: StepConfig, seed: int = 0):
    """Q [B,max_nodes,Hq,D], K and V [B,Hkv,Lcap,D], all ~ N(0,1).  The caller treats
    cache rows kv_len[b] .. kv_len[b]+n_nodes[b]-1 as the tree nodes' keys/values."""
    Q = _normal(seed, "Q", (cfg.B, cfg.max_nodes, cfg.Hq, cfg.D), 1.0, cfg.dtype)
    K = _normal(seed, "K", (cfg.B, cfg.Hkv, cfg.Lcap, cfg.D), 1.0, cfg.dtype)
    V = _normal(seed, "V", (cfg.B, cfg.Hkv, cfg.Lcap, cfg.D), 1.0, cfg.dtype)
    return Q, K, V


def gen_lm_head(cfg: StepConfig, seed: int = 0) -> np.ndarray:
    """Wl [V,H] ~ N(0, 0.02^2)."""
    return _normal(seed, "Wl", (cfg.V, cfg.H), 0.02, cfg.dtype)


def gen_node_hidden(cfg: StepConfig, seed: int, Wl: np.ndarray, node_tok: np.ndarray,
                    parent: np.ndarray, n_nodes: np.ndarray, p: Optional[float] = None):
    """Hidden states hn [B*max_nodes, H] at the tree nodes such that the base model's
    greedy token after node i equals one of i's children with probability p.

    For each live node a target token is drawn: with probability p (and if the node has
    children) a uniformly chosen child's token, otherwise a uniform token that is not a
    child's token.  hn[i] = Wl[target] + 0.01 * N(0,1), which puts the target's logit
    tens of standard deviations above every other row's, so the arg-max does not depend
    on the accumulation precision.  Rows of dead nodes are zero.  Returns (hn, target)."""
    p = cfg.agree_p if p is None else p
    B, n_max = cfg.B, cfg.max_nodes
    g = _rng(seed, "agree")
    target = np.full((B, n_max), -1, dtype=np.int32)
    for b in range(B):
        n = int(n_nodes[b])
        for i in range(n):
            kids = [int(node_tok[b, c]) for c in range(n) if int(parent[b, c]) == i]
            u = g.random()
            pick = g.integers(0, 1 << 30)
            if kids and u < p:
                target[b, i] = kids[pick % len(kids)]
            else:
                t = pick % cfg.V
                while t in kids:
                    t = (t + 1) % cfg.V
                target[b, i] = t
    noise = _normal(seed, "hn_noise", (B * n_max, cfg.H), 0.01, "fp32")
    hn = np.zeros((B * n_max, cfg.H), dtype=np.float32)
    flat = target.reshape(-1)
    live = flat >= 0
    hn[live] = Wl[flat[live]] + noise[live]
    return to_dtype(hn, cfg.dtype), target


def chain_cache_config(cfg: StepConfig, n_steps: int) -> StepConfig:
    """The same shape with a cache large enough for n_steps chained steps: every step appends
    its root and at most T accepted tokens, and the last tree still needs max_nodes rows."""
    return cfg.replace(kv_hi=cfg.kv_hi + n_steps * (cfg.T + 1))


def gen_chain_tables(cfg: StepConfig, seed: int, n_steps: int):
    """Per-step stand-ins for what the base model produces at the tree nodes of each of n_steps
    chained steps: queries Qtab [S,B,max_nodes,Hq,D] and keys/values Ktab, Vtab
    [S,B,Hkv,max_nodes,D], all ~ N(0,1), drawn independently per step."""
    S = n_steps
    Qtab = np.stack([_normal(seed * 1009 + 1 + s, "Q", (cfg.B, cfg.max_nodes, cfg.Hq, cfg.D), 1.0, cfg.dtype)
                     for s in range(S)])
    Ktab = np.stack([_normal(seed * 1009 + 1 + s, "K", (cfg.B, cfg.Hkv, cfg.max_nodes, cfg.D), 1.0, cfg.dtype)
                     for s in range(S)])
    Vtab = np.stack([_normal(seed * 1009 + 1 + s, "V", (cfg.B, cfg.Hkv, cfg.max_nodes, cfg.D), 1.0, cfg.dtype)
                     for s in range(S)])
    return Qtab, Ktab, Vtab


def chain_step_seed(seed: int, step: int) -> int:
    """Seed of gen_node_hidden for step `step` of a chain."""
    return seed * 1009 + 1 + step


def gen_gumbel_noise(cfg: StepConfig, seed: int = 0) -> np.ndarray:
    """Standard Gumbel noise [B, T+1, V] float32 for sampling acceptance: -log(-log(U)) with U
    uniform on the open interval (0,1).  One row per (sequence, tree depth)."""
    g = _rng(seed, "gumbel")
    u = g.random((cfg.B, cfg.T + 1, cfg.V), dtype=np.float64)
    u = np.clip(u, 1e-300, 1.0 - 1e-16)
    return (-np.log(-np.log(u))).astype(np.float32)


def gen_draft_layer(cfg: StepConfig, seed: int, I: int, R: int, kv_lo: int, kv_hi: int):
    """Random-init weights and inputs of one step of the attention draft module (Sec. 3.1): norm
    gains ~ 1 + 0.1 N(0,1), projection weights ~ N(0, 0.02^2) like the other weights, hidden states
    of the R newest positions ~ N(0,1), n_new uniform in 1..R, the layer's own key/value cache
    ~ N(0,1) with kv_lo..kv_hi positions already in it.  Returns (weights dict, F_new [B,R,H],
    n_new [B], kv_len [B], Kd, Vd [B,Hkv,Lcap,D])."""
    H, Hq, Hkv, D = cfg.H, cfg.Hq, cfg.Hkv, cfg.D
    w = dict(g1=(1.0 + 0.1 * _rng(seed, "dm_g1").standard_normal(H)).astype(np.float32),
             g2=(1.0 + 0.1 * _rng(seed, "dm_g2").standard_normal(H)).astype(np.float32),
             Wqkv=_normal(seed, "dm_qkv", ((Hq + 2 * Hkv) * D, H), 0.02, cfg.dtype),
             Wo=_normal(seed, "dm_o", (H, Hq * D), 0.02, cfg.dtype),
             Wgu=_normal(seed, "dm_gu", (2 * I, H), 0.02, cfg.dtype),
             Wdn=_normal(seed, "dm_dn", (H, I), 0.02, cfg.dtype))
    F_new = _normal(seed, "dm_F", (cfg.B, R, H), 1.0, cfg.dtype)
    n_new = _rng(seed, "dm_n").integers(1, R + 1, size=cfg.B).astype(np.int32)
    kv_len = _rng(seed, "dm_len").integers(kv_lo, kv_hi + 1, size=cfg.B).astype(np.int32)
    Lcap = ((kv_hi + R + 63) // 64) * 64
    Kd = _normal(seed, "dm_K", (cfg.B, Hkv, Lcap, D), 1.0, cfg.dtype)
    Vd = _normal(seed, "dm_V", (cfg.B, Hkv, Lcap, D), 1.0, cfg.dtype)
    return w, F_new, n_new, kv_len, Kd, Vd
