"""ctypes binding of libctcsd.so: argument marshalling only.

Every step of the draft-and-verify pass runs inside the CUDA library; this module turns
torch tensors (used purely as device-memory owners) into raw pointers, checks shapes and
dtypes, and forwards to the C entry points of the same names.  There is no CPU fallback:
if the library cannot be loaded, or a call reports an error, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libctcsd.so")

DTYPE_F32, DTYPE_BF16 = 0, 1
SCORE_SUM, SCORE_MAX = 0, 1

EXPORTS = [
    "ctcsd_workspace_bytes", "ctcsd_create", "ctcsd_destroy", "ctcsd_poll_status", "ctcsd_strerror",
    "ctcsd_last_cuda_error", "ctcsd_launch_count", "ctcsd_debug_bounds_enabled", "ctcsd_set_l2_prefetch", "ctcsd_selftest_timeout",
    "ctcsd_draft_logits", "ctcsd_topk_collapse", "ctcsd_build_tree", "ctcsd_tree_attention",
    "ctcsd_verify_accept", "ctcsd_commit_accepted", "ctcsd_tree_attention_static", "ctcsd_draft_logits_rows",
    "ctcsd_verify_accept_sampled", "ctcsd_draft_module_workspace_bytes", "ctcsd_draft_module",
    "ctcsd_select_raw_paths", "ctcsd_build_raw_tree", "ctcsd_verify_accept_raw",
]


class CtcsdError(RuntimeError):
    pass


class CConfig(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in (
        "B", "H", "V", "T", "k", "beam", "topN", "max_nodes", "Hq", "Hkv", "D", "dtype", "score_mode",
        "max_draft_rows")]


class CDraftLayer(ctypes.Structure):
    _fields_ = [("g1", ctypes.c_void_p), ("Wqkv", ctypes.c_void_p), ("Wo", ctypes.c_void_p), ("g2", ctypes.c_void_p),
                ("Wgu", ctypes.c_void_p), ("Wdn", ctypes.c_void_p), ("I", ctypes.c_int), ("eps", ctypes.c_float),
                ("rope_theta", ctypes.c_float)]


_lib = None


def load_library(path: Optional[str] = None) -> ctypes.CDLL:
    """Loads libctcsd.so (built in-tree by paper_2412_00061_b200.build).  Raises if absent."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or LIB_PATH
    if not os.path.exists(p):
        raise CtcsdError("CUDA library %s is missing: run `python -m paper_2412_00061_b200.build`" % p)
    lib = ctypes.CDLL(p)
    vp, ci, cs = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
    lib.ctcsd_workspace_bytes.argtypes = [ctypes.POINTER(CConfig), ctypes.POINTER(cs)]
    lib.ctcsd_create.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(CConfig), vp, cs]
    lib.ctcsd_destroy.argtypes = [vp]
    lib.ctcsd_poll_status.argtypes = [vp, vp, ctypes.POINTER(ci)]
    lib.ctcsd_strerror.argtypes = [ci]
    lib.ctcsd_strerror.restype = ctypes.c_char_p
    lib.ctcsd_last_cuda_error.argtypes = [vp]
    lib.ctcsd_set_l2_prefetch.argtypes = [vp, vp, cs]
    lib.ctcsd_selftest_timeout.argtypes = [vp, vp]
    lib.ctcsd_debug_bounds_enabled.argtypes = []
    lib.ctcsd_launch_count.argtypes = [vp]
    lib.ctcsd_launch_count.restype = ctypes.c_longlong
    lib.ctcsd_draft_logits.argtypes = [vp, vp, ci] + [vp] * 8
    lib.ctcsd_draft_logits_rows.argtypes = [vp, vp, ci, vp, ci] + [vp] * 8
    lib.ctcsd_topk_collapse.argtypes = [vp, vp, ci] + [vp] * 7
    lib.ctcsd_build_tree.argtypes = [vp, vp] + [vp] * 12
    lib.ctcsd_tree_attention.argtypes = [vp, vp, vp, vp, vp, ci, vp, vp, vp, ctypes.c_float, vp]
    lib.ctcsd_verify_accept.argtypes = [vp, vp] + [vp] * 11
    lib.ctcsd_verify_accept_sampled.argtypes = [vp, vp] + [vp] * 7 + [ctypes.c_float] + [vp] * 6
    lib.ctcsd_draft_module_workspace_bytes.argtypes = [ctypes.POINTER(CConfig), ci, ci, ctypes.POINTER(cs)]
    lib.ctcsd_draft_module.argtypes = [vp, vp, ctypes.POINTER(CDraftLayer), vp, cs, ci, vp, vp, vp, vp, vp, ci, vp, vp, vp]
    lib.ctcsd_commit_accepted.argtypes = [vp, vp, vp, vp, ci, vp, vp, vp, vp, vp]
    lib.ctcsd_select_raw_paths.argtypes = [vp, vp, ci] + [vp] * 6
    lib.ctcsd_build_raw_tree.argtypes = [vp, vp] + [vp] * 13
    lib.ctcsd_verify_accept_raw.argtypes = [vp, vp] + [vp] * 12
    lib.ctcsd_tree_attention_static.argtypes = [vp, ci, ci, ci, ci, ci, vp, vp, vp, ci, vp, vp, vp,
                                                ctypes.c_float, vp, vp]
    for name in EXPORTS:
        if name not in ("ctcsd_strerror", "ctcsd_launch_count"):
            getattr(lib, name).restype = ci
    if path is None:
        _lib = lib
    return lib


def use_library(path: Optional[str]) -> ctypes.CDLL:
    """Makes `path` (for example the debug-bounds build) the library that new handles use; None goes
    back to the regular build."""
    global _lib
    _lib = None
    if path is None:
        return load_library()
    _lib = load_library(path)
    return _lib


def _ptr(t: Optional[torch.Tensor], dtype=None, numel: Optional[int] = None, name: str = "") -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise CtcsdError("%s must be a contiguous CUDA tensor" % name)
    if dtype is not None and t.dtype != dtype:
        raise CtcsdError("%s must have dtype %s, got %s" % (name, dtype, t.dtype))
    if numel is not None and t.numel() != numel:
        raise CtcsdError("%s must have %d elements, got %d" % (name, numel, t.numel()))
    return t.data_ptr()


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


class Handle:
    """Owns a ctcsd handle and its device workspace (a torch uint8 tensor)."""

    def __init__(self, B, H, V, T, k, beam, topN, max_nodes, Hq, Hkv, D, dtype, score_mode=SCORE_SUM,
                 max_draft_rows=0, device="cuda:0"):
        self.lib = load_library()
        if not torch.cuda.is_available():
            raise CtcsdError("ctcsd needs a CUDA device (B200); there is no CPU path")
        self.cfg = CConfig(B, H, V, T, k, beam, topN, max_nodes, Hq, Hkv, D, dtype, score_mode, max_draft_rows)
        self.device = torch.device(device)
        self.act_dtype = torch.bfloat16 if dtype == DTYPE_BF16 else torch.float32
        self.M_draft_max = max_draft_rows or B
        nbytes = ctypes.c_size_t(0)
        self._check(self.lib.ctcsd_workspace_bytes(ctypes.byref(self.cfg), ctypes.byref(nbytes)), "workspace_bytes")
        with torch.cuda.device(self.device):
            self.workspace = torch.empty(nbytes.value + 256, dtype=torch.uint8, device=self.device)
            base = self.workspace.data_ptr()
            self._ws_ptr = (base + 255) // 256 * 256
            h = ctypes.c_void_p()
            self._check(self.lib.ctcsd_create(ctypes.byref(h), ctypes.byref(self.cfg), self._ws_ptr, nbytes.value),
                        "create")
        self._h = h

    def _check(self, rc: int, what: str):
        if rc != 0:
            extra = ""
            if rc == -4 and getattr(self, "_h", None):
                extra = " (cudaError %d)" % self.lib.ctcsd_last_cuda_error(self._h)
            raise CtcsdError("ctcsd_%s failed: %s%s" % (what, self.lib.ctcsd_strerror(rc).decode(), extra))

    def close(self):
        if getattr(self, "_h", None):
            self.lib.ctcsd_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def launch_count(self) -> int:
        return int(self.lib.ctcsd_launch_count(self._h))

    def set_l2_prefetch(self, tensor: Optional[torch.Tensor], nbytes: int = 0):
        """Hint: after the draft head, prefetch the first `nbytes` of `tensor` (the LM-head weights)
        into L2; None or 0 turns it off."""
        if tensor is None or nbytes <= 0:
            self._check(self.lib.ctcsd_set_l2_prefetch(self._h, None, 0), "set_l2_prefetch")
            return
        nbytes = min(int(nbytes), tensor.numel() * tensor.element_size())
        self._check(self.lib.ctcsd_set_l2_prefetch(self._h, _ptr(tensor, name="prefetch"), nbytes), "set_l2_prefetch")

    def selftest_timeout(self, stream=None):
        self._check(self.lib.ctcsd_selftest_timeout(self._h, _stream_ptr(stream)), "selftest_timeout")

    def poll_status(self, stream=None) -> int:
        st = ctypes.c_int(0)
        self._check(self.lib.ctcsd_poll_status(self._h, _stream_ptr(stream), ctypes.byref(st)), "poll_status")
        return st.value

    # ---- the five calls of the hot path ------------------------------------------------
    def draft_logits(self, x, Wd, row_seq, blank_bias, out_topk_id, out_topk_lp, out_lse,
                     out_logits_dbg=None, stream=None):
        c = self.cfg
        M = x.shape[0]
        i32, f32 = torch.int32, torch.float32
        rc = self.lib.ctcsd_draft_logits(
            self._h, _stream_ptr(stream), M,
            _ptr(x, self.act_dtype, M * c.H, "x"), _ptr(Wd, self.act_dtype, c.T * (c.V + 1) * c.H, "Wd"),
            _ptr(row_seq, i32, M, "row_seq"), _ptr(blank_bias, f32, c.B, "blank_bias"),
            _ptr(out_topk_id, i32, M * c.T * c.k, "out_topk_id"), _ptr(out_topk_lp, f32, M * c.T * c.k, "out_topk_lp"),
            _ptr(out_lse, f32, M * c.T, "out_lse"),
            _ptr(out_logits_dbg, f32, M * c.T * (c.V + 1), "out_logits_dbg"))
        self._check(rc, "draft_logits")

    def draft_logits_rows(self, x, x_rows, Wd, row_seq, blank_bias, out_topk_id, out_topk_lp, out_lse,
                          out_logits_dbg=None, stream=None):
        """Draft row m reads x[x_rows[m]] (x_rows: int32 device tensor of M entries)."""
        c = self.cfg
        M = x_rows.shape[0]
        R = x.shape[0]
        i32, f32 = torch.int32, torch.float32
        rc = self.lib.ctcsd_draft_logits_rows(
            self._h, _stream_ptr(stream), M,
            _ptr(x, self.act_dtype, R * c.H, "x"), R, _ptr(x_rows, i32, M, "x_rows"),
            _ptr(Wd, self.act_dtype, c.T * (c.V + 1) * c.H, "Wd"),
            _ptr(row_seq, i32, M, "row_seq"), _ptr(blank_bias, f32, c.B, "blank_bias"),
            _ptr(out_topk_id, i32, M * c.T * c.k, "out_topk_id"), _ptr(out_topk_lp, f32, M * c.T * c.k, "out_topk_lp"),
            _ptr(out_lse, f32, M * c.T, "out_lse"),
            _ptr(out_logits_dbg, f32, M * c.T * (c.V + 1), "out_logits_dbg"))
        self._check(rc, "draft_logits_rows")

    def topk_collapse(self, topk_id, topk_lp, sel_row, out_cand_tok, out_cand_len, out_cand_score, out_n_cand,
                      stream=None):
        c = self.cfg
        M = topk_id.shape[0]
        i32, f32 = torch.int32, torch.float32
        rc = self.lib.ctcsd_topk_collapse(
            self._h, _stream_ptr(stream), M,
            _ptr(topk_id, i32, M * c.T * c.k, "topk_id"), _ptr(topk_lp, f32, M * c.T * c.k, "topk_lp"),
            _ptr(sel_row, i32, c.B, "sel_row"),
            _ptr(out_cand_tok, i32, c.B * c.topN * c.T, "out_cand_tok"), _ptr(out_cand_len, i32, c.B * c.topN, "out_cand_len"),
            _ptr(out_cand_score, f32, c.B * c.topN, "out_cand_score"), _ptr(out_n_cand, i32, c.B, "out_n_cand"))
        self._check(rc, "topk_collapse")

    def build_tree(self, base_tok, kv_len, cand_tok, cand_len, n_cand, out_node_tok, out_parent, out_depth,
                   out_pos, out_mask, out_retrieve, out_n_nodes, stream=None):
        c = self.cfg
        i32 = torch.int32
        W = (c.max_nodes + 63) // 64
        nn = c.B * c.max_nodes
        rc = self.lib.ctcsd_build_tree(
            self._h, _stream_ptr(stream),
            _ptr(base_tok, i32, c.B, "base_tok"), _ptr(kv_len, i32, c.B, "kv_len"),
            _ptr(cand_tok, i32, c.B * c.topN * c.T, "cand_tok"), _ptr(cand_len, i32, c.B * c.topN, "cand_len"),
            _ptr(n_cand, i32, c.B, "n_cand"),
            _ptr(out_node_tok, i32, nn, "out_node_tok"), _ptr(out_parent, i32, nn, "out_parent"),
            _ptr(out_depth, i32, nn, "out_depth"), _ptr(out_pos, i32, nn, "out_pos"),
            _ptr(out_mask, torch.int64, nn * W, "out_mask"),
            _ptr(out_retrieve, i32, c.B * c.topN * c.T, "out_retrieve"), _ptr(out_n_nodes, i32, c.B, "out_n_nodes"))
        self._check(rc, "build_tree")

    def tree_attention(self, Q, K, V, kv_len, n_nodes, mask, scale, out_O, stream=None):
        c = self.cfg
        i32 = torch.int32
        Lcap = K.shape[2]
        W = (c.max_nodes + 63) // 64
        rc = self.lib.ctcsd_tree_attention(
            self._h, _stream_ptr(stream),
            _ptr(Q, self.act_dtype, c.B * c.max_nodes * c.Hq * c.D, "Q"),
            _ptr(K, self.act_dtype, c.B * c.Hkv * Lcap * c.D, "K"), _ptr(V, self.act_dtype, c.B * c.Hkv * Lcap * c.D, "V"),
            Lcap, _ptr(kv_len, i32, c.B, "kv_len"), _ptr(n_nodes, i32, c.B, "n_nodes"),
            _ptr(mask, torch.int64, c.B * c.max_nodes * W, "mask"), float(scale),
            _ptr(out_O, self.act_dtype, c.B * c.max_nodes * c.Hq * c.D, "out_O"))
        self._check(rc, "tree_attention")

    def verify_accept(self, hn, Wl, node_tok, parent, n_nodes, out_argmax, out_acc_len, out_acc_nodes,
                      out_acc_tok, out_next_tok, out_logits_dbg=None, stream=None):
        c = self.cfg
        i32 = torch.int32
        nn = c.B * c.max_nodes
        rc = self.lib.ctcsd_verify_accept(
            self._h, _stream_ptr(stream),
            _ptr(hn, self.act_dtype, nn * c.H, "hn"), _ptr(Wl, self.act_dtype, c.V * c.H, "Wl"),
            _ptr(node_tok, i32, nn, "node_tok"), _ptr(parent, i32, nn, "parent"), _ptr(n_nodes, i32, c.B, "n_nodes"),
            _ptr(out_argmax, i32, nn, "out_argmax"), _ptr(out_acc_len, i32, c.B, "out_acc_len"),
            _ptr(out_acc_nodes, i32, c.B * c.T, "out_acc_nodes"), _ptr(out_acc_tok, i32, c.B * c.T, "out_acc_tok"),
            _ptr(out_next_tok, i32, c.B, "out_next_tok"),
            _ptr(out_logits_dbg, torch.float32, nn * c.V, "out_logits_dbg"))
        self._check(rc, "verify_accept")

    def verify_accept_sampled(self, hn, Wl, node_tok, parent, depth, n_nodes, noise, temperature, out_token,
                              out_acc_len, out_acc_nodes, out_acc_tok, out_next_tok, out_logits_dbg=None, stream=None):
        """Sampling acceptance: noise [B,T+1,V] float32 standard Gumbel variates, temperature > 0."""
        c = self.cfg
        i32 = torch.int32
        nn = c.B * c.max_nodes
        rc = self.lib.ctcsd_verify_accept_sampled(
            self._h, _stream_ptr(stream),
            _ptr(hn, self.act_dtype, nn * c.H, "hn"), _ptr(Wl, self.act_dtype, c.V * c.H, "Wl"),
            _ptr(node_tok, i32, nn, "node_tok"), _ptr(parent, i32, nn, "parent"), _ptr(depth, i32, nn, "depth"),
            _ptr(n_nodes, i32, c.B, "n_nodes"), _ptr(noise, torch.float32, c.B * (c.T + 1) * c.V, "noise"),
            float(temperature),
            _ptr(out_token, i32, nn, "out_token"), _ptr(out_acc_len, i32, c.B, "out_acc_len"),
            _ptr(out_acc_nodes, i32, c.B * c.T, "out_acc_nodes"), _ptr(out_acc_tok, i32, c.B * c.T, "out_acc_tok"),
            _ptr(out_next_tok, i32, c.B, "out_next_tok"),
            _ptr(out_logits_dbg, torch.float32, nn * c.V, "out_logits_dbg"))
        self._check(rc, "verify_accept_sampled")

    # ---- the paper's attention draft module (Sec. 3.1) ----
    def make_draft_layer(self, g1, Wqkv, Wo, g2, Wgu, Wdn, eps=1e-5, rope_theta=10000.0, R=None):
        """Bundles the layer's weights (device tensors) and allocates the call's workspace."""
        c = self.cfg
        I = Wdn.shape[1]
        f32 = torch.float32
        layer = CDraftLayer(_ptr(g1, f32, c.H, "g1"), _ptr(Wqkv, self.act_dtype, (c.Hq + 2 * c.Hkv) * c.D * c.H, "Wqkv"),
                            _ptr(Wo, self.act_dtype, c.H * c.Hq * c.D, "Wo"), _ptr(g2, f32, c.H, "g2"),
                            _ptr(Wgu, self.act_dtype, 2 * I * c.H, "Wgu"), _ptr(Wdn, self.act_dtype, c.H * I, "Wdn"),
                            I, float(eps), float(rope_theta))
        R = R or (c.T + 1)
        n = ctypes.c_size_t(0)
        self._check(self.lib.ctcsd_draft_module_workspace_bytes(ctypes.byref(self.cfg), R, I, ctypes.byref(n)),
                    "draft_module_workspace_bytes")
        ws = torch.empty(n.value + 256, dtype=torch.uint8, device=self.device)
        keep = (g1, Wqkv, Wo, g2, Wgu, Wdn)
        return dict(layer=layer, ws=ws, ws_ptr=(ws.data_ptr() + 255) // 256 * 256, ws_bytes=n.value, R=R, keep=keep)

    def draft_module(self, dl, F_new, n_new, kv_len, Kd, Vd, out_F, out_kv_len, out_F_dbg=None, stream=None):
        c = self.cfg
        i32 = torch.int32
        R = F_new.shape[1]
        Lcap = Kd.shape[2]
        rc = self.lib.ctcsd_draft_module(
            self._h, _stream_ptr(stream), ctypes.byref(dl["layer"]), dl["ws_ptr"], dl["ws_bytes"], R,
            _ptr(F_new, self.act_dtype, c.B * R * c.H, "F_new"), _ptr(n_new, i32, c.B, "n_new"),
            _ptr(kv_len, i32, c.B, "kv_len"),
            _ptr(Kd, self.act_dtype, c.B * c.Hkv * Lcap * c.D, "Kd"), _ptr(Vd, self.act_dtype, c.B * c.Hkv * Lcap * c.D, "Vd"),
            Lcap, _ptr(out_F, self.act_dtype, c.B * c.H, "out_F"), _ptr(out_kv_len, i32, c.B, "out_kv_len"),
            _ptr(out_F_dbg, torch.float32, c.B * c.H, "out_F_dbg"))
        self._check(rc, "draft_module")

    # ---- the paper's raw-tree layout (Sec. 3.3) ----
    def select_raw_paths(self, topk_id, topk_lp, sel_row, out_raw_tok, out_raw_score, out_n_raw, stream=None):
        c = self.cfg
        M = topk_id.shape[0]
        i32, f32 = torch.int32, torch.float32
        rc = self.lib.ctcsd_select_raw_paths(
            self._h, _stream_ptr(stream), M,
            _ptr(topk_id, i32, M * c.T * c.k, "topk_id"), _ptr(topk_lp, f32, M * c.T * c.k, "topk_lp"),
            _ptr(sel_row, i32, c.B, "sel_row"),
            _ptr(out_raw_tok, i32, c.B * c.topN * c.T, "out_raw_tok"),
            _ptr(out_raw_score, f32, c.B * c.topN, "out_raw_score"), _ptr(out_n_raw, i32, c.B, "out_n_raw"))
        self._check(rc, "select_raw_paths")

    def build_raw_tree(self, base_tok, kv_len, raw_tok, n_raw, out_node_tok, out_parent, out_depth, out_pos,
                       out_mask, out_retrieve, out_n_nodes, out_kept, out_nka, stream=None):
        c = self.cfg
        i32 = torch.int32
        W = (c.max_nodes + 63) // 64
        nn = c.B * c.max_nodes
        rc = self.lib.ctcsd_build_raw_tree(
            self._h, _stream_ptr(stream),
            _ptr(base_tok, i32, c.B, "base_tok"), _ptr(kv_len, i32, c.B, "kv_len"),
            _ptr(raw_tok, i32, c.B * c.topN * c.T, "raw_tok"), _ptr(n_raw, i32, c.B, "n_raw"),
            _ptr(out_node_tok, i32, nn, "out_node_tok"), _ptr(out_parent, i32, nn, "out_parent"),
            _ptr(out_depth, i32, nn, "out_depth"), _ptr(out_pos, i32, nn, "out_pos"),
            _ptr(out_mask, torch.int64, nn * W, "out_mask"),
            _ptr(out_retrieve, i32, c.B * c.topN * c.T, "out_retrieve"), _ptr(out_n_nodes, i32, c.B, "out_n_nodes"),
            _ptr(out_kept, i32, nn, "out_kept"), _ptr(out_nka, i32, nn, "out_nka"))
        self._check(rc, "build_raw_tree")

    def verify_accept_raw(self, hn, Wl, node_tok, kept, nka, n_nodes, out_argmax, out_acc_len, out_acc_nodes,
                          out_acc_tok, out_next_tok, out_logits_dbg=None, stream=None):
        c = self.cfg
        i32 = torch.int32
        nn = c.B * c.max_nodes
        rc = self.lib.ctcsd_verify_accept_raw(
            self._h, _stream_ptr(stream),
            _ptr(hn, self.act_dtype, nn * c.H, "hn"), _ptr(Wl, self.act_dtype, c.V * c.H, "Wl"),
            _ptr(node_tok, i32, nn, "node_tok"), _ptr(kept, i32, nn, "kept"), _ptr(nka, i32, nn, "nka"),
            _ptr(n_nodes, i32, c.B, "n_nodes"),
            _ptr(out_argmax, i32, nn, "out_argmax"), _ptr(out_acc_len, i32, c.B, "out_acc_len"),
            _ptr(out_acc_nodes, i32, c.B * c.T, "out_acc_nodes"), _ptr(out_acc_tok, i32, c.B * c.T, "out_acc_tok"),
            _ptr(out_next_tok, i32, c.B, "out_next_tok"),
            _ptr(out_logits_dbg, torch.float32, nn * c.V, "out_logits_dbg"))
        self._check(rc, "verify_accept_raw")

    def commit_accepted(self, K, V, kv_len, acc_len, acc_nodes, out_kv_len, out_sel_row=None, stream=None):
        c = self.cfg
        i32 = torch.int32
        Lcap = K.shape[2]
        rc = self.lib.ctcsd_commit_accepted(
            self._h, _stream_ptr(stream),
            _ptr(K, self.act_dtype, c.B * c.Hkv * Lcap * c.D, "K"), _ptr(V, self.act_dtype, c.B * c.Hkv * Lcap * c.D, "V"),
            Lcap, _ptr(kv_len, i32, c.B, "kv_len"), _ptr(acc_len, i32, c.B, "acc_len"),
            _ptr(acc_nodes, i32, c.B * c.T, "acc_nodes"), _ptr(out_kv_len, i32, c.B, "out_kv_len"),
            _ptr(out_sel_row, i32, c.B, "out_sel_row"))
        self._check(rc, "commit_accepted")


def tree_attention_static(Q, K, V, kv_len, n_nodes, mask, scale, out_O, out_status=None, stream=None):
    """ctcsd_tree_attention_static: tree attention for callers that may not allocate device
    memory (no handle, no workspace; the scratch is a fixed array inside the library).
    Q, out_O [B,max_nodes,Hq,D] bfloat16; K, V [B,Hkv,Lcap,D] bfloat16; kv_len, n_nodes [B] int32;
    mask [B,max_nodes,W] int64 bit-masks; out_status None or int32[2].  Raises CtcsdError on a
    non-zero status, e.g. when the shape exceeds the built-in scratch."""
    lib = load_library()
    B, n, Hq, D = Q.shape
    Hkv, Lcap = K.shape[1], K.shape[2]
    W = (n + 63) // 64
    bf, i32 = torch.bfloat16, torch.int32
    rc = lib.ctcsd_tree_attention_static(
        _stream_ptr(stream), B, n, Hq, Hkv, D,
        _ptr(Q, bf, B * n * Hq * D, "Q"), _ptr(K, bf, B * Hkv * Lcap * D, "K"), _ptr(V, bf, B * Hkv * Lcap * D, "V"),
        Lcap, _ptr(kv_len, i32, B, "kv_len"), _ptr(n_nodes, i32, B, "n_nodes"),
        _ptr(mask, torch.int64, B * n * W, "mask"), float(scale), _ptr(out_O, bf, B * n * Hq * D, "out_O"),
        _ptr(out_status, i32, 2, "out_status"))
    if rc != 0:
        raise CtcsdError("ctcsd_tree_attention_static failed: %s" % lib.ctcsd_strerror(rc).decode())
