"""fp64 CPU oracle for the Token Radius Attention hot path (test infrastructure).

This package wraps ``tra_oracle.c`` (plain C, fp64) with ctypes and numpy.  It is
the independent definition the CUDA library is checked against; it is NOT part of
the product path and must only be used by the tests, the smoke check and the
benchmark's CPU-baseline leg.  It imports nothing from the CUDA package.

Every function cites the passage of the paper it follows; see ``tra_oracle.c``
for the arithmetic.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "tra_oracle.c")
_LIB = os.path.join(_HERE, "libtra_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile ``tra_oracle.c`` with gcc (OpenMP) next to its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-std=c11", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


def _ptr(a, ctype):
    return a.ctypes.data_as(ctypes.POINTER(ctype)) if a is not None else None


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.tra_oracle_grid_count_brute.restype = ctypes.c_int64
    return _lib


def num_threads() -> int:
    return int(lib().tra_oracle_num_threads())


def _c(a, dtype):
    return np.ascontiguousarray(a, dtype=dtype)


# --------------------------------------------------------------------------- #
# geometry
# --------------------------------------------------------------------------- #
def tile_major(T, H, W, tile_h, tile_w):
    """coord[p] = (t, y, x) of tile-major position p (Section 3.3)."""
    coord = np.empty((T * H * W, 3), np.int32)
    n = lib().tra_oracle_tile_major(T, H, W, tile_h, tile_w, _ptr(coord, ctypes.c_int32))
    assert n == T * H * W
    return coord


def default_radii(T, H, W, gamma, policy=0):
    """Candidate set R of Eq. 14 under the stated reading (see the C source)."""
    out = np.empty(4096, np.float64)
    n = lib().tra_oracle_default_radii(T, H, W, ctypes.c_double(gamma), policy,
                                       _ptr(out, ctypes.c_double), out.size)
    assert n > 0
    return out[:n].copy()


def theta_table(radii, T, H, W, gamma):
    """theta[k, delta] = min(floor(r_k^2 exp(-2 gamma delta)), diag^2) (Eq. 10, Eq. 15)."""
    radii = _c(radii, np.float64)
    th = np.empty((radii.size, T), np.int32)
    lib().tra_oracle_theta(_ptr(radii, ctypes.c_double), radii.size, T, H, W,
                           ctypes.c_double(gamma), _ptr(th, ctypes.c_int32))
    return th


def grid_count_brute(T, H, W, theta_row, f, y, x) -> int:
    """C_grid of Eq. 13 for one query and one candidate, by enumeration."""
    theta_row = _c(theta_row, np.int32)
    return int(lib().tra_oracle_grid_count_brute(T, H, W, _ptr(theta_row, ctypes.c_int32), int(f), int(y), int(x)))


def grid_count_table(T, H, W, theta):
    """C_grid for every (t, y, x, candidate): uint32 [T, H, W, n_radii]."""
    theta = _c(theta, np.int32)
    counts = np.empty((T, H, W, theta.shape[0]), np.uint32)
    lib().tra_oracle_grid_count_table(T, H, W, _ptr(theta, ctypes.c_int32), theta.shape[0],
                                      _ptr(counts, ctypes.c_uint32))
    return counts


# --------------------------------------------------------------------------- #
# entropy -> budget -> radius
# --------------------------------------------------------------------------- #
def budget(entropy_f32, tau, N):
    """K = ceil(tau exp(H)) clamped to [1, N] (Eq. 8); also the 'fragile' flags."""
    e = _c(entropy_f32, np.float32)
    out = np.empty(e.shape, np.int32)
    frag = np.empty(e.shape, np.uint8)
    lib().tra_oracle_budget(_ptr(e, ctypes.c_float), ctypes.c_int64(e.size), ctypes.c_double(tau),
                            N, _ptr(out, ctypes.c_int32), _ptr(frag, ctypes.c_uint8))
    return out, frag.astype(bool)


def budget_lognormal(entropy_f32, tau, N):
    """K = ceil(N * Phibar(sqrt(2 (log N - H)) - Phi^-1(tau))) clamped to [1, N] (Appendix,
    entropy-identified Lognormal mapping); also the 'fragile' flags."""
    from statistics import NormalDist
    z_tau = NormalDist().inv_cdf(tau) if tau < 1.0 else float("inf")
    e = _c(entropy_f32, np.float32)
    out = np.empty(e.shape, np.int32)
    frag = np.empty(e.shape, np.uint8)
    lib().tra_oracle_budget_lognormal(_ptr(e, ctypes.c_float), ctypes.c_int64(e.size),
                                      ctypes.c_double(z_tau), N, _ptr(out, ctypes.c_int32),
                                      _ptr(frag, ctypes.c_uint8))
    return out, frag.astype(bool)


def select_radius(budget_hn, coord, H, W, counts):
    """ridx[h, p] = index of the smallest candidate with C_grid >= K (Eq. 14)."""
    b = _c(budget_hn, np.int32)
    heads, N = b.shape
    coord = _c(coord, np.int32)
    counts = _c(counts, np.uint32)
    n_radii = counts.shape[-1]
    ridx = np.empty((heads, N), np.uint16)
    lib().tra_oracle_select_radius(_ptr(b, ctypes.c_int32), heads, N, _ptr(coord, ctypes.c_int32),
                                   H, W, _ptr(counts, ctypes.c_uint32), n_radii,
                                   _ptr(ridx, ctypes.c_uint16))
    return ridx


# --------------------------------------------------------------------------- #
# masks
# --------------------------------------------------------------------------- #
def token_mask_row(coord, T, theta, qi, ridx_q):
    """Row qi of the logical token mask M of Eq. 15 (bool [N])."""
    coord = _c(coord, np.int32)
    theta = _c(theta, np.int32)
    N = coord.shape[0]
    row = np.empty(N, np.uint8)
    lib().tra_oracle_token_mask_row(_ptr(coord, ctypes.c_int32), N, T, _ptr(theta, ctypes.c_int32),
                                    int(qi), int(ridx_q), _ptr(row, ctypes.c_uint8))
    return row.astype(bool)


def block_vote(coord, T, b, theta, ridx_head, u_list=None, keep_diagonal=False, n_text=0):
    """Algorithm 1 for one head: uint8 [len(u_list), NB], no bounding-box shortcut.
    n_text text tokens follow the video tokens; their blocks stay dense."""
    coord = _c(coord, np.int32)
    theta = _c(theta, np.int32)
    ridx_head = _c(ridx_head, np.uint16)
    N = coord.shape[0]
    NB = (N + n_text + b - 1) // b
    if u_list is None:
        u_list = np.arange(NB)
    u_list = _c(u_list, np.int32)
    out = np.empty((u_list.size, NB), np.uint8)
    lib().tra_oracle_block_vote(_ptr(coord, ctypes.c_int32), N, T, b, _ptr(theta, ctypes.c_int32),
                                _ptr(ridx_head, ctypes.c_uint16), _ptr(u_list, ctypes.c_int32),
                                u_list.size, int(bool(keep_diagonal)), int(n_text),
                                _ptr(out, ctypes.c_uint8))
    return out


def csr_from_block_mask(mask):
    """row_ptr / col_idx (ascending key block per row) of a [..., NB, NB] byte mask."""
    m = np.asarray(mask).astype(bool)
    flat = m.reshape(-1, m.shape[-1])
    row_ptr = np.zeros(flat.shape[0] + 1, np.int64)
    np.cumsum(flat.sum(axis=1), out=row_ptr[1:])
    col_idx = np.nonzero(flat)[1].astype(np.int32)
    return row_ptr, col_idx


def visible_rows(coord, T, b, theta, ridx_head, rows, block_rows, mode, n_text=0):
    """Visible key sets (bool [len(rows), N + n_text]) of the sparse pass; see the C source for modes."""
    coord = _c(coord, np.int32)
    theta = _c(theta, np.int32)
    ridx_head = _c(ridx_head, np.uint16)
    rows = _c(rows, np.int32)
    N = coord.shape[0]
    block_rows = _c(block_rows, np.uint8) if block_rows is not None else None
    vis = np.empty((rows.size, N + n_text), np.uint8)
    lib().tra_oracle_visible_rows(_ptr(coord, ctypes.c_int32), N, T, b,
                                  _ptr(theta, ctypes.c_int32), _ptr(ridx_head, ctypes.c_uint16),
                                  _ptr(rows, ctypes.c_int32), rows.size,
                                  _ptr(block_rows, ctypes.c_uint8), mode, int(n_text),
                                  _ptr(vis, ctypes.c_uint8))
    return vis


# --------------------------------------------------------------------------- #
# attention
# --------------------------------------------------------------------------- #
def attention_rows(Q, K, V, scale, rows, visible=None):
    """Eq. 1 (restricted to ``visible``) and Eq. 2 for the query positions ``rows``.

    Q, K, V: uint16 [N, d] bf16 bit patterns of one head.  Returns a dict with
    O [n, d], H_def, H_lse, lse (all fp64).
    """
    Q = _c(Q, np.uint16)
    K = _c(K, np.uint16)
    V = _c(V, np.uint16)
    rows = _c(rows, np.int32)
    N, d = K.shape
    n = rows.size
    vis = _c(visible, np.uint8) if visible is not None else None
    if vis is not None:
        assert vis.shape == (n, N)
    O = np.empty((n, d), np.float64)
    H_def = np.empty(n, np.float64)
    H_lse = np.empty(n, np.float64)
    lse = np.empty(n, np.float64)
    lib().tra_oracle_attention_rows(_ptr(Q, ctypes.c_uint16), _ptr(K, ctypes.c_uint16),
                                    _ptr(V, ctypes.c_uint16), N, d, ctypes.c_double(scale),
                                    _ptr(rows, ctypes.c_int32), n, _ptr(vis, ctypes.c_uint8),
                                    _ptr(O, ctypes.c_double), _ptr(H_def, ctypes.c_double),
                                    _ptr(H_lse, ctypes.c_double), _ptr(lse, ctypes.c_double))
    return {"O": O, "H_def": H_def, "H_lse": H_lse, "lse": lse}


def attention_rows_alg2(Q, K, V, scale, rows, tile):
    """Algorithm 2 (online softmax with the entropy accumulator) in fp64."""
    Q = _c(Q, np.uint16)
    K = _c(K, np.uint16)
    V = _c(V, np.uint16)
    rows = _c(rows, np.int32)
    N, d = K.shape
    O = np.empty((rows.size, d), np.float64)
    H = np.empty(rows.size, np.float64)
    lib().tra_oracle_attention_rows_alg2(_ptr(Q, ctypes.c_uint16), _ptr(K, ctypes.c_uint16),
                                         _ptr(V, ctypes.c_uint16), N, d, ctypes.c_double(scale),
                                         int(tile), _ptr(rows, ctypes.c_int32), rows.size,
                                         _ptr(O, ctypes.c_double), _ptr(H, ctypes.c_double))
    return {"O": O, "H": H}


# --------------------------------------------------------------------------- #
# one object that carries the plan-time tables of a configuration
# --------------------------------------------------------------------------- #
@dataclass
class Geometry:
    T: int
    H: int
    W: int
    tile_h: int
    tile_w: int
    block: int
    gamma: float
    tau: float
    radii: np.ndarray
    coord: np.ndarray      # [N, 3] (t, y, x) per tile-major position
    theta: np.ndarray      # [n_radii, T]
    counts: np.ndarray     # [T, H, W, n_radii]

    @property
    def N(self):
        return self.T * self.H * self.W

    @property
    def NB(self):
        return (self.N + self.block - 1) // self.block


def geometry(T, H, W, tile_h, tile_w, block, gamma, tau, radii=None, policy=0) -> Geometry:
    if radii is None:
        radii = default_radii(T, H, W, gamma, policy)
    coord = tile_major(T, H, W, tile_h, tile_w)
    theta = theta_table(radii, T, H, W, gamma)
    counts = grid_count_table(T, H, W, theta)
    return Geometry(T, H, W, tile_h, tile_w, block, gamma, tau, np.asarray(radii), coord, theta, counts)


def schedule(n_steps, warm_fraction=0.25):
    """Warm-up rule (Section 4.1 'Implementation details'): the first floor(fraction*n_steps)
    steps are dense; the entropy of the last of them is the one consumed."""
    n_warm = int(np.floor(warm_fraction * n_steps))
    return ["dense"] * n_warm + ["sparse"] * (n_steps - n_warm), n_warm
