"""Thin binding over ``libtra_b200.so`` (the C ABI of ``include/tra.h``).

Argument marshalling only: every step of the path runs in the library's CUDA kernels.
PyTorch supplies device memory and streams.  There is no CPU fallback: if the shared
library is missing or cannot be loaded, importing this module raises.
"""
from __future__ import annotations

import ctypes
import math
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# TRA_B200_LIB selects another build of the same library (the bounds-checking debug build)
LIB_PATH = os.environ.get("TRA_B200_LIB") or os.path.join(_HERE, "libtra_b200.so")

TRA_OK = 0
TRA_ERR_INVALID_ARG, TRA_ERR_UNSUPPORTED, TRA_ERR_CAPACITY, TRA_ERR_CUDA, TRA_ERR_TIMEOUT, TRA_ERR_BOUNDS = -1, -2, -3, -4, -5, -6
TRA_KEEP_DIAGONAL = 1
TRA_ORDER_RASTER = 2
TRA_ORDER_RASTER_QO = 4
TRA_RADII_EXTENDED = 0
TRA_RADII_LITERAL = 1
TRA_BUDGET_UNIFORM = 0
TRA_BUDGET_LOGNORMAL = 1

EXPORTS = [
    "tra_plan_create", "tra_plan_destroy", "tra_plan_num_tokens", "tra_plan_num_video_tokens", "tra_plan_num_blocks",
    "tra_plan_num_radii", "tra_plan_num_tile_pairs", "tra_plan_tables", "tra_plan_count_table", "tra_plan_status",
    "tra_status_string", "tra_selftest_wait_timeout", "tra_tile_major_gather", "tra_tile_major_scatter",
    "tra_entropy_attn", "tra_budget_radius", "tra_build_block_mask", "tra_sparse_attn",
    "tra_build_block_list_static",
    "tra_hot_path_host_workspace_bytes", "tra_hot_path_host",
]


class tra_config_t(ctypes.Structure):
    _fields_ = [
        ("T", ctypes.c_int), ("H", ctypes.c_int), ("W", ctypes.c_int),
        ("head_dim", ctypes.c_int), ("block", ctypes.c_int),
        ("tile_h", ctypes.c_int), ("tile_w", ctypes.c_int),
        ("tau", ctypes.c_double), ("gamma", ctypes.c_double),
        ("radii", ctypes.POINTER(ctypes.c_double)), ("n_radii", ctypes.c_int),
        ("radius_policy", ctypes.c_int), ("flags", ctypes.c_uint), ("budget_map", ctypes.c_int),
        ("n_text", ctypes.c_int),
    ]


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2608_02504_b200.build` "
            "(there is no CPU fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, f32 = ctypes.c_void_p, ctypes.c_int, ctypes.c_float
    lib.tra_plan_create.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(tra_config_t), vp]
    lib.tra_plan_destroy.argtypes = [vp]
    for name in ("tra_plan_num_tokens", "tra_plan_num_video_tokens", "tra_plan_num_blocks", "tra_plan_num_radii",
                 "tra_plan_num_tile_pairs"):
        getattr(lib, name).argtypes = [vp]
    lib.tra_plan_tables.argtypes = [vp, vp, vp, vp]
    lib.tra_plan_count_table.argtypes = [vp, vp]
    lib.tra_plan_status.argtypes = [vp, vp]
    lib.tra_status_string.argtypes = [i32]
    lib.tra_selftest_wait_timeout.argtypes = [vp, i32, vp]
    lib.tra_hot_path_host_workspace_bytes.argtypes = [vp, i32]
    lib.tra_hot_path_host_workspace_bytes.restype = ctypes.c_size_t
    lib.tra_hot_path_host.argtypes = [vp, vp, vp, vp, vp, vp, ctypes.c_size_t, i32, i32, i32, f32, vp]
    lib.tra_status_string.restype = ctypes.c_char_p
    lib.tra_tile_major_gather.argtypes = [vp, vp, vp, i32, i32, vp]
    lib.tra_tile_major_scatter.argtypes = [vp, vp, vp, i32, i32, vp]
    lib.tra_entropy_attn.argtypes = [vp, vp, vp, vp, vp, vp, vp, i32, i32, f32, vp]
    lib.tra_budget_radius.argtypes = [vp, vp, vp, vp, vp, i32, i32, vp]
    lib.tra_build_block_mask.argtypes = [vp, vp, vp, vp, vp, ctypes.c_int64, vp, vp, i32, i32, vp]
    lib.tra_sparse_attn.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, i32, i32, f32, vp]
    lib.tra_build_block_list_static.argtypes = [vp, vp, vp, vp, ctypes.c_int64, vp, vp, i32, i32, vp]
    return lib


_lib = _load()


class TraError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        super().__init__(f"{where}: {_lib.tra_status_string(code).decode()} ({code})")


def _check(code, where):
    if code != TRA_OK:
        raise TraError(code, where)


def _stream(stream=None):
    s = stream if stream is not None else torch.cuda.current_stream()
    return ctypes.c_void_p(s.cuda_stream)


def _dev(t, dtype, name):
    if t is None:
        return None
    if not (t.is_cuda and t.is_contiguous() and t.dtype == dtype):
        raise ValueError(f"{name}: expected a contiguous CUDA tensor of dtype {dtype}")
    return ctypes.c_void_p(t.data_ptr())


class Plan:
    """Owns a ``tra_plan_t`` (geometry, thresholds, count table, block boxes)."""

    def __init__(self, T, H, W, head_dim, block, tile_h, tile_w, tau=0.9, gamma=0.6, radii=None,
                 radius_policy=TRA_RADII_EXTENDED, flags=0, budget_map=TRA_BUDGET_UNIFORM, n_text=0,
                 stream=None):
        cfg = tra_config_t()
        cfg.T, cfg.H, cfg.W = T, H, W
        cfg.head_dim, cfg.block, cfg.tile_h, cfg.tile_w = head_dim, block, tile_h, tile_w
        cfg.tau, cfg.gamma = tau, gamma
        self._radii_keepalive = None
        if radii is not None:
            arr = (ctypes.c_double * len(radii))(*[float(r) for r in radii])
            self._radii_keepalive = arr
            cfg.radii = ctypes.cast(arr, ctypes.POINTER(ctypes.c_double))
            cfg.n_radii = len(radii)
        cfg.radius_policy, cfg.flags, cfg.budget_map = radius_policy, flags, budget_map
        cfg.n_text = n_text
        self.cfg = cfg
        self._h = ctypes.c_void_p()
        _check(_lib.tra_plan_create(ctypes.byref(self._h), ctypes.byref(cfg), _stream(stream)), "tra_plan_create")
        self.N = _lib.tra_plan_num_tokens(self._h)              # tokens per sequence (video + text)
        self.N_video = _lib.tra_plan_num_video_tokens(self._h)
        self.NB = _lib.tra_plan_num_blocks(self._h)
        self.n_radii = _lib.tra_plan_num_radii(self._h)
        self.T, self.H, self.W = T, H, W
        self.head_dim, self.block, self.flags = head_dim, block, flags

    @classmethod
    def from_config(cls, cfg: dict, **overrides):
        kw = dict(T=cfg["T"], H=cfg["H"], W=cfg["W"], head_dim=cfg["head_dim"], block=cfg["block"],
                  tile_h=cfg["tile_h"], tile_w=cfg["tile_w"], tau=cfg["tau"], gamma=cfg["gamma"])
        kw.update(overrides)
        return cls(**kw)

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            _lib.tra_plan_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- host copies of the plan tables -------------------------------------------------
    def tables(self):
        import numpy as np
        radii = np.empty(self.n_radii, np.float64)
        theta = np.empty((self.n_radii, self.T), np.int32)
        coord = np.empty((self.N_video, 3), np.int32)
        _check(_lib.tra_plan_tables(self._h, radii.ctypes.data, theta.ctypes.data, coord.ctypes.data),
               "tra_plan_tables")
        return radii, theta, coord

    def count_table(self):
        import numpy as np
        counts = np.empty((self.T, self.H, self.W, self.n_radii), np.uint32)
        _check(_lib.tra_plan_count_table(self._h, counts.ctypes.data), "tra_plan_count_table")
        return counts

    def status(self, stream=None):
        return _lib.tra_plan_status(self._h, _stream(stream))

    def selftest_wait_timeout(self, limit_ms=20):
        """Runs the bounded-wait self-test kernel; the plan status then reads TRA_ERR_TIMEOUT."""
        _check(_lib.tra_selftest_wait_timeout(self._h, limit_ms, _stream()), "tra_selftest_wait_timeout")

    def check_status(self, stream=None):
        _check(self.status(stream), "tra_plan_status")

    # -- layout ---------------------------------------------------------------------------
    def _permute(self, fn, src, name, out=None):
        if not (src.is_cuda and src.is_contiguous()):
            raise ValueError(f"{name}: expected a contiguous CUDA tensor")
        if src.dim() < 2 or src.shape[-2] != self.N:
            raise ValueError(f"{name}: expected [..., N, row]")
        row_bytes = src.shape[-1] * src.element_size()
        n_bh = src.numel() // (self.N * src.shape[-1])
        dst = torch.empty_like(src) if out is None else out
        if not (dst.is_cuda and dst.is_contiguous() and dst.shape == src.shape and dst.dtype == src.dtype):
            raise ValueError(f"{name}: `out` must be a contiguous CUDA tensor like the input")
        _check(fn(self._h, ctypes.c_void_p(src.data_ptr()), ctypes.c_void_p(dst.data_ptr()), n_bh,
                  row_bytes, _stream()), name)
        return dst

    def tile_major_gather(self, x_raster, out=None):
        """raster-order [..., N, row] -> tile-major order (a new tensor, or ``out``)."""
        return self._permute(_lib.tra_tile_major_gather, x_raster, "tra_tile_major_gather", out)

    def tile_major_scatter(self, x_tile_major, out=None):
        """tile-major order [..., N, row] -> raster order (a new tensor, or ``out``)."""
        return self._permute(_lib.tra_tile_major_scatter, x_tile_major, "tra_tile_major_scatter", out)

    # -- the four hot calls -------------------------------------------------------------
    def _bh(self, Q):
        if Q.dim() != 4 or Q.shape[2] != self.N or Q.shape[3] != self.head_dim:
            raise ValueError("expected Q/K/V of shape [B, heads, N, head_dim]")
        return Q.shape[0], Q.shape[1]

    def entropy_attn(self, Q, K, V, O=None, entropy=None, lse=None, want_entropy=True, want_lse=False,
                     sm_scale=None):
        """Dense attention + per-query entropy (tile-major inputs).  Returns (O, entropy, lse)."""
        B, heads = self._bh(Q)
        if O is None:
            O = torch.empty_like(Q)
        if entropy is None and want_entropy:
            entropy = torch.empty(B, heads, self.N, dtype=torch.float32, device=Q.device)
        if lse is None and want_lse:
            lse = torch.empty(B, heads, self.N, dtype=torch.float32, device=Q.device)
        scale = 1.0 / math.sqrt(self.head_dim) if sm_scale is None else sm_scale
        bf = torch.bfloat16
        _check(_lib.tra_entropy_attn(self._h, _dev(Q, bf, "Q"), _dev(K, bf, "K"), _dev(V, bf, "V"),
                                     _dev(O, bf, "O"), _dev(entropy, torch.float32, "entropy"),
                                     _dev(lse, torch.float32, "lse"), B, heads, scale, _stream()),
               "tra_entropy_attn")
        return O, entropy, lse

    def budget_radius(self, entropy, budget=None, radius=None, ridx=None, want_budget=True,
                      want_radius=True):
        """entropy [B, heads, N] fp32 -> (budget int32, radius fp32, ridx as int16 storage of uint16)."""
        B, heads = entropy.shape[0], entropy.shape[1]
        dev = entropy.device
        if budget is None and want_budget:
            budget = torch.empty(B, heads, self.N, dtype=torch.int32, device=dev)
        if radius is None and want_radius:
            radius = torch.empty(B, heads, self.N, dtype=torch.float32, device=dev)
        if ridx is None:
            ridx = torch.empty(B, heads, self.N, dtype=torch.int16, device=dev)
        _check(_lib.tra_budget_radius(self._h, _dev(entropy, torch.float32, "entropy"),
                                      _dev(budget, torch.int32, "budget"),
                                      _dev(radius, torch.float32, "radius"),
                                      _dev(ridx, torch.int16, "ridx"), B, heads, _stream()),
               "tra_budget_radius")
        return budget, radius, ridx

    @property
    def n_tile_pairs(self):
        """Thread blocks per (batch, head) of a block-sparse launch: pairs of query tiles (a tile holds two
        blocks of up to 64 tokens, or one larger block)."""
        return _lib.tra_plan_num_tile_pairs(self._h)

    def build_block_mask(self, ridx, block_mask=None, row_ptr=None, col_idx=None, nnz=None, tile_pairs=None,
                         want_tile_pairs=False):
        """ridx [B, heads, N] -> (block_mask uint8 [B, heads, NB, NB], row_ptr, col_idx, nnz); with
        ``want_tile_pairs`` (or a ``tile_pairs`` buffer) a fifth result: the int32 [B*heads, pairs, 2]
        table of query tiles that share a thread block in ``sparse_attn``."""
        B, heads = ridx.shape[0], ridx.shape[1]
        dev = ridx.device
        rows = B * heads * self.NB
        if block_mask is None:
            block_mask = torch.empty(B, heads, self.NB, self.NB, dtype=torch.uint8, device=dev)
        if row_ptr is None:
            row_ptr = torch.empty(rows + 1, dtype=torch.int32, device=dev)
        if col_idx is None:
            col_idx = torch.empty(rows * self.NB, dtype=torch.int32, device=dev)
        if nnz is None:
            nnz = torch.zeros(1, dtype=torch.int64, device=dev)
        if tile_pairs is None and want_tile_pairs:
            # (blocks of 32 tokens or fewer have no tile pairs: one entry, so that the library's refusal is seen)
            tile_pairs = torch.empty(B * heads, max(self.n_tile_pairs, 1), 2, dtype=torch.int32, device=dev)
        _check(_lib.tra_build_block_mask(self._h, _dev(ridx, torch.int16, "ridx"),
                                         _dev(block_mask, torch.uint8, "block_mask"),
                                         _dev(row_ptr, torch.int32, "row_ptr"),
                                         _dev(col_idx, torch.int32, "col_idx"), col_idx.numel(),
                                         _dev(nnz, torch.int64, "nnz"), _dev(tile_pairs, torch.int32, "tile_pairs"),
                                         B, heads, _stream()),
               "tra_build_block_mask")
        if tile_pairs is not None:
            return block_mask, row_ptr, col_idx, nnz, tile_pairs
        return block_mask, row_ptr, col_idx, nnz

    def build_block_list_static(self, ridx, row_ptr, col_idx, nnz=None, tile_pairs=None):
        """ridx [B, heads, N] -> the active-block list, written into the caller's ``row_ptr`` / ``col_idx``
        (and ``nnz`` / ``tile_pairs`` when given), through ``tra_build_block_list_static``: the variant of
        ``build_block_mask`` for callers that must not allocate.  The Boolean mask stays in a fixed
        16 MiB array inside the library, so every output must be passed in and nothing is created here;
        shapes whose mask is larger raise ``TraError`` (TRA_ERR_CAPACITY)."""
        B, heads = ridx.shape[0], ridx.shape[1]
        _check(_lib.tra_build_block_list_static(self._h, _dev(ridx, torch.int16, "ridx"),
                                                _dev(row_ptr, torch.int32, "row_ptr"),
                                                _dev(col_idx, torch.int32, "col_idx"), col_idx.numel(),
                                                _dev(nnz, torch.int64, "nnz"),
                                                _dev(tile_pairs, torch.int32, "tile_pairs"), B, heads, _stream()),
               "tra_build_block_list_static")

    def sparse_attn(self, Q, K, V, row_ptr, col_idx, O=None, lse=None, want_lse=False, sm_scale=None,
                    ridx=None, tile_pairs=None):
        """Block-sparse attention over the retained key blocks (tile-major inputs).  With ``ridx`` the
        token mask of Eq. 15 is applied inside the retained blocks as well; with ``ridx`` and
        ``row_ptr = col_idx = None`` the call evaluates Eq. 16 itself (token mask alone, no block list)."""
        B, heads = self._bh(Q)
        if O is None:
            O = torch.empty_like(Q)
        if lse is None and want_lse:
            lse = torch.empty(B, heads, self.N, dtype=torch.float32, device=Q.device)
        scale = 1.0 / math.sqrt(self.head_dim) if sm_scale is None else sm_scale
        bf = torch.bfloat16
        _check(_lib.tra_sparse_attn(self._h, _dev(Q, bf, "Q"), _dev(K, bf, "K"), _dev(V, bf, "V"),
                                    _dev(row_ptr, torch.int32, "row_ptr"),
                                    _dev(col_idx, torch.int32, "col_idx"), _dev(ridx, torch.int16, "ridx"),
                                    _dev(tile_pairs, torch.int32, "tile_pairs"), _dev(O, bf, "O"),
                                    _dev(lse, torch.float32, "lse"), B, heads, scale, _stream()),
               "tra_sparse_attn")
        return O, lse


class HostPipeline:
    """One pass of the hot path over tensors that live in pinned host memory (``tra_hot_path_host``).

    The library runs the pass in groups of heads (heads are independent problems): while the kernels
    of group g run, the inputs of group g + 1 travel to the device on a copy stream and the output of
    group g - 1 travels back on another, so the PCIe time hides behind the kernels.  This class only
    owns the device workspace the call needs.

    Inputs and outputs are bf16, raster token order, shape [1, heads, N, head_dim], pinned.
    """

    def __init__(self, plan: "Plan", heads: int, group: int = 8, device=None, sm_scale=None, first_group=None):
        """``first_group`` (default ``group``): heads in the first group; a small first group lets the
        kernels start while most of the input is still on its way."""
        if heads < 1 or group < 1 or (first_group is not None and first_group < 1):
            raise ValueError("heads, group and first_group must be positive")
        self.plan, self.heads, self.group = plan, heads, min(group, heads)
        self.first_group = self.group if first_group is None else min(first_group, self.group)
        self.dev = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
        self.scale = 1.0 / math.sqrt(plan.head_dim) if sm_scale is None else sm_scale
        self.workspace_bytes = int(_lib.tra_hot_path_host_workspace_bytes(plan._h, self.group))
        self.workspace = torch.empty(self.workspace_bytes + 256, dtype=torch.uint8, device=self.dev)
        self._ws_ptr = (self.workspace.data_ptr() + 255) & ~255
        # 3 gathers, dense, budget, vote + scan + fill + pairing, sparse, scatter; a raster-order plan has no
        # gathers and no scatter, one with only Q and O in raster order gathers K and V
        self.launches_per_group = 7 if plan.flags & TRA_ORDER_RASTER else (9 if plan.flags & TRA_ORDER_RASTER_QO else 11)
        self.n_groups = len(self.group_sizes(heads, self.group, self.first_group))

    @staticmethod
    def group_sizes(heads, group, first_group):
        """The head groups of one pass (mirrors the library): a small first group, doubling up to
        ``group``, and a small last group."""
        sizes, left, ramp = [], heads, first_group
        while left > 0:
            n = min(ramp, left)
            if left - n == 0 and n > first_group and sizes:
                n -= first_group
            sizes.append(n)
            left -= n
            ramp = min(2 * ramp, group)
        return sizes

    @staticmethod
    def _check_host(t, shape, name):
        if t.is_cuda or not t.is_pinned() or t.dtype != torch.bfloat16 or tuple(t.shape) != shape or \
                not t.is_contiguous():
            raise ValueError(f"{name}: expected a contiguous pinned bf16 host tensor of shape {shape}")

    def run(self, Qh, Kh, Vh, Oh):
        """Q, K, V (pinned host) -> O (pinned host).  Returns the number of kernels launched once every
        copy and kernel has been enqueued; synchronise the current stream before reading ``Oh``."""
        shape = (1, self.heads, self.plan.N, self.plan.head_dim)
        for t, name in ((Qh, "Q"), (Kh, "K"), (Vh, "V"), (Oh, "O")):
            self._check_host(t, shape, name)
        vp = ctypes.c_void_p
        _check(_lib.tra_hot_path_host(self.plan._h, vp(Qh.data_ptr()), vp(Kh.data_ptr()), vp(Vh.data_ptr()),
                                      vp(Oh.data_ptr()), vp(self._ws_ptr), self.workspace_bytes, self.heads,
                                      self.group, self.first_group, self.scale,
                                      _stream(torch.cuda.current_stream(self.dev))), "tra_hot_path_host")
        return self.n_groups * self.launches_per_group
