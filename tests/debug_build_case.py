"""Runs the whole hot path on the small and ragged shapes and prints, as JSON, the plan status after
every case and a digest of every output.  tests/test_gpu_debug_build.py executes this file twice,
once per build of the library (TRA_B200_LIB selects the bounds-checking build), and compares."""
import hashlib
import json
import os
import sys

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from paper_2608_02504_b200 import api, workloads   # noqa: E402
from tests import common                           # noqa: E402


def digest(*tensors):
    h = hashlib.sha1()
    for t in tensors:
        h.update(t.detach().contiguous().cpu().view(torch.uint8).numpy().tobytes())
    return h.hexdigest()


def main():
    cases = [
        (workloads.CONFIGS["tiny"], 0),
        (common.small_config(3, 7, 10, heads=3, head_dim=64, block=64, tile_h=4, tile_w=4, seed=78), 0),
        (common.small_config(5, 9, 11, heads=2, head_dim=128, block=128, tile_h=4, tile_w=4, seed=79), 0),
        (common.small_config(3, 9, 14, heads=2, head_dim=128, block=64, tile_h=4, tile_w=8, seed=81), 0),
        (common.small_config(6, 16, 24, heads=2, head_dim=128, block=128, tile_h=8, tile_w=16, seed=80,
                             s_lo=0.2, s_hi=5.0), 100),
        (common.small_config(3, 7, 10, heads=3, head_dim=64, block=64, tile_h=4, tile_w=4, seed=78), 50),
        # blocks that are neither 64 nor 128 tokens (no token mask inside blocks for these)
        (common.small_config(3, 11, 23, heads=2, head_dim=128, block=90, tile_h=9, tile_w=10, seed=82), 0),
        (common.small_config(3, 10, 16, heads=2, head_dim=128, block=40, tile_h=5, tile_w=8, seed=83), 30),
    ]
    out = []
    for cfg, n_text in cases:
        plan = api.Plan.from_config(cfg, n_text=n_text)
        Qr, Kr, Vr = workloads.make_qkv(cfg, "cuda")
        if n_text:
            Qr, Kr, Vr = workloads.append_text(Qr, Kr, Vr, cfg, n_text)
        Q, K, V = (plan.tile_major_gather(x) for x in (Qr, Kr, Vr))
        O, H, lse = plan.entropy_attn(Q, K, V, want_lse=True)
        budget, radius, ridx = plan.budget_radius(H)
        mask, row_ptr, col_idx, nnz, pairs = plan.build_block_mask(ridx, want_tile_pairs=True)
        Os, lse_s = plan.sparse_attn(Q, K, V, row_ptr, col_idx, tile_pairs=pairs, want_lse=True)
        token_mask = cfg["block"] in (64, 128)
        Ot, _ = plan.sparse_attn(Q, K, V, row_ptr, col_idx, ridx=ridx if token_mask else None, tile_pairs=pairs)
        Oe, _ = plan.sparse_attn(Q, K, V, None, None, ridx=ridx) if token_mask else (Ot, None)
        back = plan.tile_major_scatter(Os)
        status = plan.status()
        # a list that overflows its buffer, and candidate indices past the table: both are clamped
        small = torch.zeros(5, dtype=torch.int32, device="cuda")
        _, rp2, _, _ = plan.build_block_mask(ridx, col_idx=small)
        Oc, _ = plan.sparse_attn(Q, K, V, rp2, small)
        status_overflow = plan.status()
        wild = torch.full_like(ridx, -1)
        mw, rpw, ciw, _ = plan.build_block_mask(wild)
        Ow, _ = plan.sparse_attn(Q, K, V, rpw, ciw, ridx=wild if token_mask else None)
        status_wild = plan.status()
        # a list whose offsets run backwards (no entry is read: every row comes out empty); only the
        # bounds-checking build notices
        bad = row_ptr.flip(0).contiguous()
        plan.sparse_attn(Q, K, V, bad, col_idx)
        status_bad_list = plan.status()
        out.append({"tokens": plan.N, "n_text": n_text, "status": status, "status_overflow": status_overflow,
                    "status_wild": status_wild, "status_bad_list": status_bad_list,
                    "digest": digest(O, H, lse, budget, radius, ridx, mask, row_ptr, col_idx[: int(nnz.item())], pairs,
                                     Os, lse_s, Ot, Oe, back, Oc, mw, Ow)})
        plan.close()
    print(json.dumps({"lib": os.path.basename(api.LIB_PATH), "cases": out}))


if __name__ == "__main__":
    main()
