"""ctypes binding of libgraft.so -- argument marshalling only; every step of the round runs in the
library's CUDA kernels.  Method names mirror the C entry points of include/graft.h.

Tensors are torch CUDA tensors (device memory) or, for ``build_trees_host``, pinned CPU tensors; the
binding passes raw pointers and the current torch stream.  There is no fallback: if the shared library is
missing or a call fails, a GraftError is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import torch

from . import build as _build

F32, BF16 = 0, 1
ST_BAD_LOGITS, ST_TAU_CLAMPED, ST_FRONTIER_EMPTY, ST_INTERNAL = 1, 2, 4, 8

ENTRY_POINTS = [
    "graft_create", "graft_destroy", "graft_nmax", "graft_mask_words", "graft_set_saba", "graft_set_tdes_tables",
    "graft_tdes_precompute", "graft_build_trees", "graft_vocab_pass", "graft_vocab_pass_static", "graft_tdes_edges",
    "graft_accept", "graft_tdes_loss", "graft_saba_fit", "graft_set_edge_rows", "graft_edge_rows", "graft_set_hist_window", "graft_vocab_pass_partial", "graft_vocab_merge",
    "graft_build_trees_host", "graft_launch_count", "graft_set_timing", "graft_read_timing", "graft_status_str",
    "graft_version",
]


VOCAB_PARTIAL_BYTES = 280  # sizeof(graft_vocab_partial)


class GraftError(RuntimeError):
    pass


class _Config(C.Structure):
    _fields_ = [("V", C.c_int32), ("L", C.c_int32), ("K", C.c_int32), ("m", C.c_int32), ("hidden_dim", C.c_int32),
                ("max_batch", C.c_int32), ("budget_min", C.c_int32), ("budget_max", C.c_int32),
                ("budget_step", C.c_int32), ("beta", C.c_float), ("root_edge", C.c_int32),
                ("logits_dtype", C.c_int), ("hidden_dtype", C.c_int)]


class _Saba(C.Structure):
    _fields_ = [("phi_conf", C.c_float), ("phi_degen", C.c_float), ("phi_hist", C.c_float), ("phi_bias", C.c_float),
                ("tau_min", C.c_float), ("cost_mode", C.c_int32), ("c0", C.c_float), ("c1", C.c_float),
                ("c2", C.c_float), ("n_pts", C.c_int32), ("pts_n", C.POINTER(C.c_float)),
                ("pts_t", C.POINTER(C.c_float))]


class _TreeOut(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in (
        "d_n_nodes", "d_budget", "d_token", "d_parent", "d_depth", "d_position", "d_path_score", "d_mask", "d_status",
        "d_topk_id", "d_topk_lp", "d_lse", "d_edge", "d_state")]


class _TdesTraces(C.Structure):
    _fields_ = [("n_groups", C.c_int32), ("d_g_parent", C.c_void_p), ("d_g_depth", C.c_void_p),
                ("d_g_child", C.c_void_p), ("d_g_logq", C.c_void_p), ("d_g_ztgt", C.c_void_p),
                ("n_pairs", C.c_int32), ("d_pairs", C.c_void_p), ("n_edges", C.c_int32), ("d_edges", C.c_void_p)]


class _TdesLossConfig(C.Structure):
    _fields_ = [("gamma", C.c_float), ("w1", C.c_float), ("lambda_kl", C.c_float), ("lambda_pair", C.c_float),
                ("lambda_bce", C.c_float)]


_lib = None


def library_path() -> str:
    return _build.LIB


def load_library():
    """Load libgraft.so (building it with nvcc first if it is missing or stale).  Raises if that fails."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.LIB
    if not os.path.exists(path) or _build.needs_build():
        try:
            _build.build()
        except Exception as e:  # no silent fallback
            raise GraftError(f"libgraft.so is missing and could not be built: {e}") from e
    lib = C.CDLL(path)
    vp = C.c_void_p
    lib.graft_create.argtypes = [C.POINTER(_Config), C.POINTER(vp)]
    lib.graft_destroy.argtypes = [vp]
    lib.graft_nmax.argtypes = [vp]
    lib.graft_nmax.restype = C.c_size_t
    lib.graft_mask_words.argtypes = [vp]
    lib.graft_mask_words.restype = C.c_size_t
    lib.graft_set_saba.argtypes = [vp, C.POINTER(_Saba)]
    lib.graft_set_tdes_tables.argtypes = [vp, vp, vp, vp, C.c_float, vp]
    lib.graft_set_edge_rows.argtypes = [vp, C.c_int32]
    lib.graft_set_hist_window.argtypes = [vp, C.c_int32, vp, vp, vp]
    lib.graft_vocab_pass_partial.argtypes = [vp, C.c_int32, vp, vp, vp]
    lib.graft_vocab_merge.argtypes = [vp, C.c_int32, C.c_int32, vp, vp, vp, vp, vp, vp, vp]
    lib.graft_edge_rows.argtypes = [vp]
    lib.graft_edge_rows.restype = C.c_int32
    lib.graft_tdes_precompute.argtypes = [vp, vp, C.c_int, C.c_int32, vp, vp, vp, vp]
    lib.graft_build_trees.argtypes = [vp, C.c_int32, vp, vp, vp, vp, vp, vp, C.POINTER(_TreeOut), vp]
    lib.graft_build_trees_host.argtypes = lib.graft_build_trees.argtypes
    lib.graft_vocab_pass.argtypes = [vp, C.c_int32, vp, vp, vp, vp, vp, vp]
    lib.graft_tdes_edges.argtypes = [vp, C.c_int32, vp, vp, vp, vp, vp]
    lib.graft_vocab_pass_static.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int, vp, vp, vp, vp, vp, vp]
    lib.graft_accept.argtypes = [vp, C.c_int32, C.POINTER(_TreeOut), vp, vp, vp, vp, vp]
    lib.graft_tdes_loss.argtypes = [vp, C.POINTER(_TdesTraces), C.POINTER(_TdesLossConfig), vp, vp, vp, vp, vp, vp, vp]
    lib.graft_saba_fit.argtypes = [vp, C.c_int64, vp, vp, vp, vp, vp, vp, vp]
    lib.graft_launch_count.argtypes = [vp]
    lib.graft_launch_count.restype = C.c_uint64
    lib.graft_set_timing.argtypes = [vp, C.c_int32]
    lib.graft_read_timing.argtypes = [vp, C.POINTER(C.c_int32), C.POINTER(C.c_float), C.POINTER(C.c_float),
                                      C.POINTER(C.c_float)]
    lib.graft_status_str.argtypes = [C.c_int]
    lib.graft_status_str.restype = C.c_char_p
    lib.graft_version.restype = C.c_char_p
    _lib = lib
    return lib


def _check(lib, rc, what):
    if rc != 0:
        raise GraftError(f"{what}: {lib.graft_status_str(rc).decode()} (status {rc})")


def _ptr(t, dtype=None, cuda=True):
    if t is None:
        return None
    if cuda and not t.is_cuda:
        raise GraftError("expected a CUDA tensor")
    if not cuda and t.is_cuda:
        raise GraftError("expected a CPU tensor")
    if not t.is_contiguous():
        raise GraftError("tensor must be contiguous")
    if dtype is not None and t.dtype != dtype:
        raise GraftError(f"expected dtype {dtype}, got {t.dtype}")
    return C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def vocab_pass_static(logits, K, topk_id, topk_lp, lse, row_status):
    """graft_vocab_pass_static: the vocab pass for callers that cannot let the library allocate (no context;
    the scratch is a static device array inside the library).  logits [batch, L, V] on the GPU."""
    lib = load_library()
    batch, L, V = logits.shape
    if logits.dtype not in (torch.bfloat16, torch.float32):
        raise GraftError(f"logits must be bfloat16 or float32, got {logits.dtype}")
    dt = BF16 if logits.dtype == torch.bfloat16 else F32
    # the library writes batch*L*K ids and log-probabilities and batch*L log-sum-exps and status words
    for name, t, need in (("topk_id", topk_id, batch * L * K), ("topk_lp", topk_lp, batch * L * K),
                          ("lse", lse, batch * L), ("row_status", row_status, batch * L)):
        if t is None or t.numel() < need:
            raise GraftError(f"{name} must hold at least {need} elements")
    _check(lib, lib.graft_vocab_pass_static(batch, L, V, K, dt, _ptr(logits), _ptr(topk_id, torch.int32),
                                            _ptr(topk_lp, torch.float32), _ptr(lse, torch.float32),
                                            _ptr(row_status, torch.int32), _stream()), "graft_vocab_pass_static")


@dataclass
class TreeOut:
    """Caller-owned output tensors of build_trees (see graft_tree_out in include/graft.h)."""
    n_nodes: torch.Tensor
    budget: torch.Tensor
    token: torch.Tensor
    parent: torch.Tensor
    depth: torch.Tensor
    position: torch.Tensor
    path_score: torch.Tensor
    mask: torch.Tensor
    status: torch.Tensor
    topk_id: torch.Tensor | None = None
    topk_lp: torch.Tensor | None = None
    lse: torch.Tensor | None = None
    edge: torch.Tensor | None = None
    state: torch.Tensor | None = None

    def _c(self, cuda=True):
        o = _TreeOut()
        i32, f32 = torch.int32, torch.float32
        o.d_n_nodes = _ptr(self.n_nodes, i32, cuda)
        o.d_budget = _ptr(self.budget, i32, cuda)
        o.d_token = _ptr(self.token, i32, cuda)
        o.d_parent = _ptr(self.parent, i32, cuda)
        o.d_depth = _ptr(self.depth, i32, cuda)
        o.d_position = _ptr(self.position, i32, cuda)
        o.d_path_score = _ptr(self.path_score, f32, cuda)
        o.d_mask = _ptr(self.mask, i32, cuda)  # uint32 bit patterns held in an int32 tensor
        o.d_status = _ptr(self.status, i32, cuda)
        o.d_topk_id = _ptr(self.topk_id, i32, cuda)
        o.d_topk_lp = _ptr(self.topk_lp, f32, cuda)
        o.d_lse = _ptr(self.lse, f32, cuda)
        o.d_edge = _ptr(self.edge, f32, cuda)
        o.d_state = _ptr(self.state, f32, cuda)
        return o

    def cpu(self) -> dict:
        out = {}
        for k, v in self.__dict__.items():
            if v is not None:
                out[k] = v.cpu().numpy()
        out["mask"] = out["mask"].view("uint32")
        return out


class Graft:
    """One library context (graft_create .. graft_destroy).  Use on one stream at a time."""

    def __init__(self, V, L, K, m, hidden_dim, max_batch, budget_min, budget_max, budget_step=16, beta=0.2,
                 root_edge=1, logits_dtype=BF16, hidden_dtype=BF16):
        self.lib = load_library()
        if not torch.cuda.is_available():
            raise GraftError("no CUDA device: the library has no CPU path")
        self.cfg = _Config(V, L, K, m, hidden_dim, max_batch, budget_min, budget_max, budget_step, beta, root_edge,
                           logits_dtype, hidden_dtype)
        self._ctx = C.c_void_p()
        _check(self.lib, self.lib.graft_create(C.byref(self.cfg), C.byref(self._ctx)), "graft_create")
        self.nmax = int(self.lib.graft_nmax(self._ctx))
        self.mask_words = int(self.lib.graft_mask_words(self._ctx))
        self._keep = []

    # ---- lifetime
    def destroy(self):
        if getattr(self, "_ctx", None) and self._ctx.value:
            self.lib.graft_destroy(self._ctx)
            self._ctx = C.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    # ---- parameters
    def set_saba(self, phi_conf, phi_degen, phi_hist, phi_bias=0.0, tau_min=1e-3, cost_mode=0, c0=0.0, c1=0.0, c2=0.0,
                 pts_n=(), pts_t=()):
        n = (C.c_float * len(pts_n))(*pts_n)
        t = (C.c_float * len(pts_t))(*pts_t)
        p = _Saba(phi_conf, phi_degen, phi_hist, phi_bias, tau_min, cost_mode, c0, c1, c2, len(pts_n),
                  C.cast(n, C.POINTER(C.c_float)), C.cast(t, C.POINTER(C.c_float)))
        _check(self.lib, self.lib.graft_set_saba(self._ctx, C.byref(p)), "graft_set_saba")

    # ---- vocabulary-parallel vocab pass
    def vocab_pass_partial(self, logits_shard, parts):
        """parts: uint8 [batch*L, VOCAB_PARTIAL_BYTES] on the device (this shard's pieces of every row)."""
        batch = logits_shard.shape[0]
        if parts.dtype != torch.uint8 or parts.numel() != batch * self.cfg.L * VOCAB_PARTIAL_BYTES:
            raise GraftError("parts must be uint8 [batch*L, VOCAB_PARTIAL_BYTES]")
        _check(self.lib, self.lib.graft_vocab_pass_partial(self._ctx, batch, _ptr(logits_shard), _ptr(parts), _stream()),
               "graft_vocab_pass_partial")

    def vocab_merge(self, parts_all, v_offsets, ids, lp, lse, row_status):
        """parts_all: uint8 [n_shards, batch*L, VOCAB_PARTIAL_BYTES]; v_offsets: first global id of each shard."""
        n_shards = parts_all.shape[0]
        batch = ids.shape[0]
        off = (C.c_int32 * n_shards)(*[int(v) for v in v_offsets])
        _check(self.lib, self.lib.graft_vocab_merge(self._ctx, batch, n_shards, _ptr(parts_all, torch.uint8), off,
                                                    _ptr(ids, torch.int32), _ptr(lp, torch.float32),
                                                    _ptr(lse, torch.float32), _ptr(row_status, torch.int32),
                                                    _stream()), "graft_vocab_merge")

    def set_hist_window(self, w, window=None, count=None, hist=None):
        """graft_accept keeps hist_t (Eq. 15) on the device: window [batch, w] int32, count [batch] int32,
        hist [batch] float32 (pass `hist` to the next build_trees).  w = 0 switches it off."""
        if w == 0:
            _check(self.lib, self.lib.graft_set_hist_window(self._ctx, 0, None, None, None), "graft_set_hist_window")
            self._hist_keep = None
            return
        _check(self.lib, self.lib.graft_set_hist_window(self._ctx, int(w), _ptr(window, torch.int32),
                                                        _ptr(count, torch.int32), _ptr(hist, torch.float32)),
               "graft_set_hist_window")
        self._hist_keep = (window, count, hist)  # borrowed by the library

    def set_edge_rows(self, rows):
        """Depths [0, rows) are scored ahead of the expansion, deeper ones on demand (graft_set_edge_rows)."""
        _check(self.lib, self.lib.graft_set_edge_rows(self._ctx, int(rows)), "graft_set_edge_rows")

    def edge_rows(self) -> int:
        return int(self.lib.graft_edge_rows(self._ctx))

    def set_tdes_tables(self, P, Ctab, u, s=1.0):
        f32 = torch.float32
        _check(self.lib, self.lib.graft_set_tdes_tables(self._ctx, _ptr(P, f32), _ptr(Ctab, f32), _ptr(u, f32),
                                                        C.c_float(s), _stream()), "graft_set_tdes_tables")
        self._keep = [P, Ctab]  # borrowed by the library

    def tdes_precompute(self, emb, W, bias, out):
        dt = BF16 if emb.dtype == torch.bfloat16 else F32
        E = emb.shape[1]
        _check(self.lib, self.lib.graft_tdes_precompute(self._ctx, _ptr(emb), dt, E, _ptr(W, torch.float32),
                                                        _ptr(bias, torch.float32), _ptr(out, torch.float32),
                                                        _stream()), "graft_tdes_precompute")

    # ---- outputs
    def alloc_out(self, batch, debug=False, device="cuda", pinned=False) -> TreeOut:
        kw = dict(device=device)
        if device == "cpu" and pinned:
            kw["pin_memory"] = True
        i32, f32 = torch.int32, torch.float32
        N, W, L, K = self.nmax, self.mask_words, self.cfg.L, self.cfg.K
        e = lambda shape, dt: torch.empty(shape, dtype=dt, **kw)  # noqa: E731
        o = TreeOut(e((batch,), i32), e((batch,), i32), e((batch, N), i32), e((batch, N), i32), e((batch, N), i32),
                    e((batch, N), i32), e((batch, N), f32), e((batch, N, W), i32), e((batch,), i32))
        if debug:
            o.topk_id, o.topk_lp = e((batch, L, K), i32), e((batch, L, K), f32)
            o.lse, o.edge, o.state = e((batch, L), f32), e((batch, L, K, K), f32), e((batch, 4), f32)
        return o

    # ---- the round
    def build_trees(self, logits, hidden, root_token, hist, prefix_len, fixed_budget, out: TreeOut):
        batch = logits.shape[0]
        i32 = torch.int32
        oc = out._c()
        _check(self.lib, self.lib.graft_build_trees(
            self._ctx, batch, _ptr(logits), _ptr(hidden), _ptr(root_token, i32), _ptr(hist, torch.float32),
            _ptr(prefix_len, i32), _ptr(fixed_budget, i32), C.byref(oc), _stream()), "graft_build_trees")
        return out

    def build_trees_host(self, logits, hidden, root_token, hist, prefix_len, fixed_budget, out: TreeOut):
        """All tensors on the CPU (pinned for asynchronous copies); returns after the results are in `out`."""
        batch = logits.shape[0]
        i32 = torch.int32
        oc = out._c(cuda=False)
        _check(self.lib, self.lib.graft_build_trees_host(
            self._ctx, batch, _ptr(logits, cuda=False), _ptr(hidden, cuda=False), _ptr(root_token, i32, False),
            _ptr(hist, torch.float32, False), _ptr(prefix_len, i32, False), _ptr(fixed_budget, i32, False),
            C.byref(oc), _stream()), "graft_build_trees_host")
        return out

    def vocab_pass(self, logits, topk_id, topk_lp, lse, row_status=None):
        batch = logits.shape[0]
        _check(self.lib, self.lib.graft_vocab_pass(self._ctx, batch, _ptr(logits), _ptr(topk_id, torch.int32),
                                                   _ptr(topk_lp, torch.float32), _ptr(lse, torch.float32),
                                                   _ptr(row_status, torch.int32), _stream()), "graft_vocab_pass")

    def tdes_edges(self, topk_id, topk_lp, root_token, edge):
        batch = topk_id.shape[0]
        _check(self.lib, self.lib.graft_tdes_edges(self._ctx, batch, _ptr(topk_id, torch.int32),
                                                   _ptr(topk_lp, torch.float32), _ptr(root_token, torch.int32),
                                                   _ptr(edge, torch.float32), _stream()), "graft_tdes_edges")

    def accept(self, trees: TreeOut, target_next, accept_len, accept_path, bonus_token):
        batch = target_next.shape[0]
        i32 = torch.int32
        oc = trees._c()
        _check(self.lib, self.lib.graft_accept(self._ctx, batch, C.byref(oc), _ptr(target_next, i32),
                                               _ptr(accept_len, i32), _ptr(accept_path, i32),
                                               _ptr(bonus_token, i32), _stream()), "graft_accept")

    def tdes_loss(self, groups, pairs, edges, gamma, w1, lambda_kl, lambda_pair, lambda_bce, loss, skipped=None,
                  gP=None, gC=None, gu=None, gs=None):
        """Training objective of the scorer and its gradients (Eq. 7-12) on device-resident traces.
        groups: dict(parent [G], depth [G], child [G, K], logq [G, K], ztgt [G, K]) or None; pairs [N, 6] int32 or
        None; edges [N, 4] int32 or None; loss: float64 [4] (overwritten); gP, gC [V, m], gu [L, m], gs [1] float32,
        added to (all or none)."""
        i32, f32 = torch.int32, torch.float32
        t = _TdesTraces()
        if groups is not None and groups["parent"].numel() > 0:
            t.n_groups = groups["parent"].numel()
            t.d_g_parent, t.d_g_depth = _ptr(groups["parent"], i32), _ptr(groups["depth"], i32)
            t.d_g_child, t.d_g_logq, t.d_g_ztgt = (_ptr(groups["child"], i32), _ptr(groups["logq"], f32),
                                                   _ptr(groups["ztgt"], f32))
        if pairs is not None and pairs.numel() > 0:
            t.n_pairs, t.d_pairs = pairs.shape[0], _ptr(pairs, i32)
        if edges is not None and edges.numel() > 0:
            t.n_edges, t.d_edges = edges.shape[0], _ptr(edges, i32)
        lc = _TdesLossConfig(gamma, w1, lambda_kl, lambda_pair, lambda_bce)
        _check(self.lib, self.lib.graft_tdes_loss(self._ctx, C.byref(t), C.byref(lc), _ptr(loss, torch.float64),
                                                  _ptr(skipped, i32), _ptr(gP, f32), _ptr(gC, f32), _ptr(gu, f32),
                                                  _ptr(gs, f32), _stream()), "graft_tdes_loss")

    def saba_fit(self, state, budget, gain, prefix_len, latency, out):
        """Least-squares fit of the gain and cost models (Eq. 16-17) to n logged rounds on the device.
        state [n, 3] float32, budget / prefix_len [n] int32, gain / latency [n] float32; out: float64 [10] =
        phi_conf, phi_degen, phi_hist, phi_bias, c0, c1, c2, rounds in the gain fit, rounds in the cost fit, status."""
        i32, f32 = torch.int32, torch.float32
        _check(self.lib, self.lib.graft_saba_fit(self._ctx, int(budget.numel()), _ptr(state, f32), _ptr(budget, i32),
                                                 _ptr(gain, f32), _ptr(prefix_len, i32), _ptr(latency, f32),
                                                 _ptr(out, torch.float64), _stream()), "graft_saba_fit")

    # ---- bookkeeping
    def launch_count(self) -> int:
        return int(self.lib.graft_launch_count(self._ctx))

    def set_timing(self, enable):
        """0 / False: stop; 1 / True: record and reset the call count; 2: record, keep counting."""
        _check(self.lib, self.lib.graft_set_timing(self._ctx, int(enable)), "graft_set_timing")

    def read_timing(self):
        n = C.c_int32()
        a, b, c = C.c_float(), C.c_float(), C.c_float()
        _check(self.lib, self.lib.graft_read_timing(self._ctx, C.byref(n), C.byref(a), C.byref(b), C.byref(c)),
               "graft_read_timing")
        return n.value, a.value, b.value, c.value
