"""Helpers shared by the GPU parity tests: seeded inputs, the oracle pipeline, tolerances."""
import math

import numpy as np
import torch

import oracle
from paper_2608_02504_b200 import workloads

# Tolerances of the parity bar: entropy within 1e-3 absolute (fp32 accumulation); attention output
# in bf16 with fp32 accumulation: |o - o_ref| <= max(1e-2, one bf16 ulp of o_ref) per element
# (half an ulp of a bf16 value in [4, 8) is already 1.6e-2) and relative L2 error <= 5e-3.
ENTROPY_ATOL = 1e-3
OUT_ATOL = 1e-2
OUT_REL_L2 = 5e-3


def small_config(T, H, W, heads, head_dim, block, tile_h, tile_w, gamma=0.6, tau=0.9, seed=77,
                 s_lo=0.3, s_hi=3.0):
    return dict(T=T, H=H, W=W, heads=heads, head_dim=head_dim, block=block, tile_h=tile_h, tile_w=tile_w,
                s_lo=s_lo, s_hi=s_hi, gamma=gamma, tau=tau, seed=seed)


def oracle_geometry(cfg, policy=0):
    return oracle.geometry(cfg["T"], cfg["H"], cfg["W"], cfg["tile_h"], cfg["tile_w"], cfg["block"],
                           cfg["gamma"], cfg["tau"], policy=policy)


def raster_of_pos(geo):
    c = geo.coord
    return (c[:, 0] * geo.H + c[:, 1]) * geo.W + c[:, 2]


def bf16_ulp(x):
    """Spacing of bf16 numbers at |x| (fp64 array)."""
    ax = np.maximum(np.abs(x), 2.0 ** -126)
    return 2.0 ** (np.floor(np.log2(ax)) - 7)


def check_output(o_gpu_bf16, o_ref):
    """o_gpu_bf16: torch bf16 [n, d] (any device); o_ref: fp64 [n, d].  Returns diagnostics."""
    got = o_gpu_bf16.detach().float().cpu().numpy().astype(np.float64)
    err = np.abs(got - o_ref)
    allowed = np.maximum(OUT_ATOL, bf16_ulp(o_ref))
    rel_l2 = float(np.linalg.norm(got - o_ref) / max(np.linalg.norm(o_ref), 1e-30))
    return {
        "max_abs": float(err.max()) if err.size else 0.0,
        "n_over_atol": int((err > OUT_ATOL).sum()),
        "n_fail": int((err > allowed).sum()),
        "rel_l2": rel_l2,
    }


def assert_output(o_gpu_bf16, o_ref, what=""):
    d = check_output(o_gpu_bf16, o_ref)
    assert d["n_fail"] == 0, f"{what}: {d}"
    assert d["rel_l2"] <= OUT_REL_L2, f"{what}: {d}"
    return d


def scale_of(cfg):
    return 1.0 / math.sqrt(cfg["head_dim"])


def to_tile_major_bits(x_raster_bf16, geo):
    """torch bf16 [1, heads, N, d] raster -> numpy uint16 [heads, N, d] in tile-major order."""
    bits = workloads.bf16_bits(x_raster_bf16)[0]
    return np.ascontiguousarray(bits[:, raster_of_pos(geo), :])
