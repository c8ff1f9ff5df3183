"""The allocation-free list builder gives the same active-block list as ``tra_build_block_mask``.

``tra_build_block_list_static`` serves callers that may not allocate device memory where the mask
is rebuilt (a plugin inside another framework's memory pool, a server whose device memory is all
handed out at start-up, a thread that must stay out of the allocator's lock): the Boolean mask,
which such a caller never reads, lives in a fixed 16 MiB array inside the library.  The test calls it
through the C ABI twice in a row, on different radii, because every call reuses that one array: the
second result must not depend on what the first call left there.  It also checks the size limit.

The file name makes pytest collect it after every other test file.
"""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2608_02504_b200 import workloads
from tests import common

pytestmark = pytest.mark.gpu

DEV = "cuda"

# ragged (N = 495, last block 111 tokens) and a shape with several frames of whole 8 x 16 tiles
CASES = [
    common.small_config(5, 9, 11, heads=2, head_dim=128, block=128, tile_h=4, tile_w=4, seed=79),
    common.small_config(6, 16, 24, heads=3, head_dim=128, block=128, tile_h=8, tile_w=16, seed=80, s_lo=0.2, s_hi=5.0),
    common.small_config(3, 9, 14, heads=2, head_dim=128, block=64, tile_h=4, tile_w=8, seed=81),
]


def _ridx(geo, heads, rng, sharp):
    """Candidate indices through the real entropy -> budget -> radius map (oracle side)."""
    hi = math.log(geo.N) * (0.5 if sharp else 1.0)
    H = rng.uniform(0.0, hi, (heads, geo.N)).astype(np.float32)
    bud, _ = oracle.budget(H, geo.tau, geo.N)
    return oracle.select_radius(bud, geo.coord, geo.H, geo.W, geo.counts)


@pytest.mark.parametrize("cfg", CASES, ids=["ragged128", "mid128", "d128b64"])
def test_static_list_equals_allocating_call_twice_in_a_row(cfg):
    from paper_2608_02504_b200 import api
    geo = common.oracle_geometry(cfg)
    plan = api.Plan.from_config(cfg)
    heads, NB = cfg["heads"], geo.NB
    rows = heads * NB
    rng = np.random.default_rng(2024)
    # the caller owns every output; the call under test creates nothing
    row_ptr = torch.empty(rows + 1, dtype=torch.int32, device=DEV)
    col_idx = torch.empty(rows * NB, dtype=torch.int32, device=DEV)
    nnz = torch.zeros(1, dtype=torch.int64, device=DEV)
    pairs = torch.empty(heads, plan.n_tile_pairs, 2, dtype=torch.int32, device=DEV)
    for call, sharp in enumerate((False, True)):
        ridx_np = _ridx(geo, heads, rng, sharp)
        ridx = torch.from_numpy(ridx_np.view(np.int16)).to(DEV)[None]
        mask_ref, rp_ref, ci_ref, nnz_ref, pairs_ref = plan.build_block_mask(ridx, want_tile_pairs=True)
        row_ptr.fill_(-1)
        col_idx.fill_(-1)
        pairs.fill_(-7)
        plan.build_block_list_static(ridx, row_ptr, col_idx, nnz=nnz, tile_pairs=pairs)
        plan.check_status()
        n = int(nnz_ref.item())
        assert int(nnz.item()) == n, f"call {call}"
        assert torch.equal(row_ptr, rp_ref), f"call {call}"
        assert torch.equal(col_idx[:n], ci_ref[:n]), f"call {call}"
        assert torch.equal(pairs, pairs_ref), f"call {call}"
        # and the list is the oracle's vote (integer work: bit-exact)
        for h in range(heads):
            ref = oracle.block_vote(geo.coord, geo.T, geo.block, geo.theta, ridx_np[h])
            rp = row_ptr.cpu().numpy()[h * NB: (h + 1) * NB + 1]
            ci = col_idx.cpu().numpy()
            for u in range(NB):
                assert np.array_equal(ci[rp[u]: rp[u + 1]], np.flatnonzero(ref[u])), (call, h, u)
    plan.close()


def test_static_list_rejects_masks_larger_than_its_array():
    from paper_2608_02504_b200 import api
    cfg = workloads.CONFIGS["tiny"]
    plan = api.Plan.from_config(cfg)
    NB = plan.NB
    heads = (16 << 20) // (NB * NB) + 1            # one head too many for the 16 MiB array
    ridx = torch.zeros(1, 1, plan.N, dtype=torch.int16, device=DEV)
    row_ptr = torch.zeros(8, dtype=torch.int32, device=DEV)
    col_idx = torch.zeros(8, dtype=torch.int32, device=DEV)
    # the size check comes before any launch, so the small buffers are never touched
    rc = api._lib.tra_build_block_list_static(plan._h, ridx.data_ptr(), row_ptr.data_ptr(), col_idx.data_ptr(), 8,
                                              None, None, 1, heads, None)
    assert rc == api.TRA_ERR_CAPACITY
    assert api._lib.tra_build_block_list_static(None, None, None, None, 0, None, None, 1, 1, None) \
        == api.TRA_ERR_INVALID_ARG
    plan.check_status()
    plan.close()
