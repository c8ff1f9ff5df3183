"""GPU parity: every stage of the CUDA path, called through the C ABI, against the fp64 oracle
on the same seeded inputs.  Integer stages are compared bit for bit; entropy and outputs within
the tolerances stated in tests/common.py."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2608_02504_b200 import workloads
from tests import common

pytestmark = pytest.mark.gpu

DEV = "cuda"


def api():
    from paper_2608_02504_b200 import api as _api
    return _api


CFG_TINY = workloads.CONFIGS["tiny"]
# ragged shapes: N = 210 with b = 64 (last block 18 tokens, last CTA half empty);
# N = 495 with b = 128 (last block 111 tokens, second CTA's second tile ragged)
CFG_RAGGED64 = common.small_config(3, 7, 10, heads=3, head_dim=64, block=64, tile_h=4, tile_w=4, seed=78)
CFG_RAGGED128 = common.small_config(5, 9, 11, heads=2, head_dim=128, block=128, tile_h=4, tile_w=4, seed=79)
CFG_MID128 = common.small_config(6, 16, 24, heads=2, head_dim=128, block=128, tile_h=8, tile_w=16, seed=80,
                                 s_lo=0.2, s_hi=5.0)
# head_dim 128 with 64-token blocks (two query blocks per 128-row tile), ragged: N = 378
CFG_D128_B64 = common.small_config(3, 9, 14, heads=2, head_dim=128, block=64, tile_h=4, tile_w=8, seed=81)
SMALL = [CFG_TINY, CFG_RAGGED64, CFG_RAGGED128, CFG_MID128, CFG_D128_B64]
IDS = ["tiny", "ragged64", "ragged128", "mid128", "d128b64"]


def make_plan(cfg, **kw):
    return api().Plan.from_config(cfg, **kw)


def tile_major_inputs(cfg, plan, heads=None):
    Qr, Kr, Vr = workloads.make_qkv(cfg, DEV, heads)
    return plan.tile_major_gather(Qr), plan.tile_major_gather(Kr), plan.tile_major_gather(Vr)


# ----------------------------------------------------------------------------- plan tables
@pytest.mark.parametrize("cfg", SMALL + [workloads.CONFIGS["wan1.3b-480p"]], ids=IDS + ["wan1.3b"])
@pytest.mark.parametrize("policy", [0, 1])
def test_plan_tables_bit_exact(cfg, policy):
    geo = common.oracle_geometry(cfg, policy)
    plan = make_plan(cfg, radius_policy=policy)
    radii, theta, coord = plan.tables()
    assert plan.N == geo.N and plan.NB == geo.NB
    assert np.array_equal(radii, geo.radii)
    assert np.array_equal(theta, geo.theta)
    assert np.array_equal(coord, geo.coord)
    assert np.array_equal(plan.count_table(), geo.counts)
    plan.close()


def test_plan_rejects_bad_arguments():
    a = api()
    for kw in (dict(head_dim=96), dict(block=8), dict(tau=0.0), dict(gamma=-1.0), dict(T=0),
               dict(flags=8),                         # an unknown flag
               dict(radii=[0.0, 1.0, 2.0]),          # last candidate does not reach full support
               dict(radii=[0.0, 2.0, 1.0, 1e9])):    # not ascending
        with pytest.raises(a.TraError):
            make_plan(CFG_TINY, **kw)
    p = make_plan(CFG_TINY, radii=[0.0, 1.0, 3.5, float("inf")])
    assert p.n_radii == 4
    p.close()


# ----------------------------------------------------------------------------- layout
@pytest.mark.parametrize("cfg", SMALL, ids=IDS)
def test_tile_major_gather_scatter(cfg):
    geo = common.oracle_geometry(cfg)
    plan = make_plan(cfg)
    x = torch.randn(2, 3, geo.N, 64, device=DEV).to(torch.bfloat16)
    g = plan.tile_major_gather(x)
    ref = x.cpu()[:, :, torch.from_numpy(common.raster_of_pos(geo)).long(), :]
    assert torch.equal(g.cpu(), ref)
    assert torch.equal(plan.tile_major_scatter(g), x)
    plan.close()


# ----------------------------------------------------------------------------- budget / radius
@pytest.mark.parametrize("cfg", SMALL + [workloads.CONFIGS["wan1.3b-480p"]], ids=IDS + ["wan1.3b"])
def test_budget_radius_bit_exact(cfg):
    geo = common.oracle_geometry(cfg)
    plan = make_plan(cfg)
    rng = np.random.default_rng(11)
    heads = 3
    H = rng.uniform(0.0, math.log(geo.N), (1, heads, geo.N)).astype(np.float32)
    H[0, 0, :7] = [0.0, math.log(geo.N), 1e-6, 30.0, -1.0, 3.0, math.log(geo.N) - 1e-3]
    bud_ref, fragile = oracle.budget(H[0], geo.tau, geo.N)
    ridx_ref = oracle.select_radius(bud_ref, geo.coord, geo.H, geo.W, geo.counts)
    budget, radius, ridx = plan.budget_radius(torch.from_numpy(H).to(DEV))
    ok = ~fragile
    assert fragile.sum() <= 2                      # elements a one-ulp exp() difference could move
    assert np.array_equal(budget.cpu().numpy()[0][ok], bud_ref[ok])
    got_ridx = ridx.cpu().numpy().view(np.uint16)[0]
    assert np.array_equal(got_ridx[ok], ridx_ref[ok])
    assert np.array_equal(radius.cpu().numpy()[0][ok], geo.radii[ridx_ref].astype(np.float32)[ok])
    plan.close()


@pytest.mark.parametrize("cfg", [CFG_TINY, workloads.CONFIGS["wan1.3b-480p"]], ids=["tiny", "wan1.3b"])
def test_budget_radius_lognormal_map_bit_exact(cfg):
    geo = common.oracle_geometry(cfg)
    plan = make_plan(cfg, budget_map=api().TRA_BUDGET_LOGNORMAL)
    rng = np.random.default_rng(21)
    H = rng.uniform(0.0, math.log(geo.N), (1, 2, geo.N)).astype(np.float32)
    H[0, 0, :4] = [0.0, math.log(geo.N), 30.0, 1e-3]
    bud_ref, fragile = oracle.budget_lognormal(H[0], geo.tau, geo.N)
    ridx_ref = oracle.select_radius(bud_ref, geo.coord, geo.H, geo.W, geo.counts)
    budget, radius, ridx = plan.budget_radius(torch.from_numpy(H).to(DEV))
    ok = ~fragile
    assert fragile.sum() <= 2
    assert np.array_equal(budget.cpu().numpy()[0][ok], bud_ref[ok])
    assert np.array_equal(ridx.cpu().numpy().view(np.uint16)[0][ok], ridx_ref[ok])
    plan.close()
    with pytest.raises(api().TraError):
        make_plan(cfg, budget_map=7)


# ----------------------------------------------------------------------------- block mask
def run_mask(plan, ridx_np):
    ridx = torch.from_numpy(ridx_np.view(np.int16)).to(DEV)[None]
    mask, row_ptr, col_idx, nnz = plan.build_block_mask(ridx)
    plan.check_status()
    return mask.cpu().numpy()[0], row_ptr.cpu().numpy(), col_idx.cpu().numpy(), int(nnz.item())


def random_ridx(geo, heads, rng, kind):
    n = geo.radii.size
    if kind == "uniform":
        return rng.integers(0, n, (heads, geo.N)).astype(np.uint16)
    if kind == "small":
        return rng.integers(0, max(2, n // 8), (heads, geo.N)).astype(np.uint16)
    if kind == "entropy":        # through the real map, like the pipeline does
        H = rng.uniform(0.0, math.log(geo.N), (heads, geo.N)).astype(np.float32)
        bud, _ = oracle.budget(H, geo.tau, geo.N)
        return oracle.select_radius(bud, geo.coord, geo.H, geo.W, geo.counts)
    if kind == "blocky":         # whole blocks sharp or diffuse: exercises empty rows and full rows
        per_block = rng.integers(0, n, (heads, geo.NB))
        r = np.repeat(per_block, geo.block, axis=1)[:, : geo.N]
        return r.astype(np.uint16)
    raise ValueError(kind)


@pytest.mark.parametrize("cfg", SMALL, ids=IDS)
@pytest.mark.parametrize("kind", ["uniform", "small", "entropy", "blocky"])
def test_block_mask_bit_exact(cfg, kind):
    geo = common.oracle_geometry(cfg)
    heads = 3
    ridx = random_ridx(geo, heads, np.random.default_rng(12), kind)
    for flags in (0, api().TRA_KEEP_DIAGONAL):
        plan = make_plan(cfg, flags=flags)
        mask, row_ptr, col_idx, nnz = run_mask(plan, ridx)
        ref = np.stack([oracle.block_vote(geo.coord, geo.T, geo.block, geo.theta, ridx[h],
                                          keep_diagonal=bool(flags)) for h in range(heads)])
        assert np.array_equal(mask, ref)
        rp, ci = oracle.csr_from_block_mask(ref)
        assert nnz == rp[-1]
        assert np.array_equal(row_ptr.astype(np.int64), rp)
        assert np.array_equal(col_idx[:nnz], ci)
        plan.close()


# The vote kernel has three layouts of its per-frame count field, chosen by the plan: sixteen cells of a row are
# one run of positions inside a block (W, tile width and block multiples of 16), four cells are (multiples of 4),
# or neither.  Full-size shapes use the first; these small grids cover all three, with blocks that straddle tiles
# and frames, a ragged last block, and text tokens.
VOTE_LAYOUT_CASES = [
    ("runs of 16, b=128", common.small_config(4, 12, 32, heads=2, head_dim=128, block=128, tile_h=8, tile_w=16, seed=91)),
    ("runs of 16, b=64", common.small_config(3, 8, 48, heads=2, head_dim=64, block=64, tile_h=4, tile_w=16, seed=92)),
    ("runs of 16, b=48", common.small_config(3, 10, 32, heads=2, head_dim=128, block=48, tile_h=8, tile_w=16, seed=93)),
    ("runs of 16, b=80, tile 2x32", common.small_config(5, 7, 32, heads=2, head_dim=128, block=80, tile_h=2, tile_w=32, seed=94)),
    ("runs of 4, b=64", common.small_config(4, 9, 24, heads=2, head_dim=64, block=64, tile_h=4, tile_w=8, seed=95)),
    ("runs of 4, b=36", common.small_config(3, 11, 20, heads=2, head_dim=128, block=36, tile_h=4, tile_w=4, seed=96)),
    ("runs of 4 only (b=40)", common.small_config(3, 6, 32, heads=2, head_dim=128, block=40, tile_h=2, tile_w=16, seed=97)),
    ("single cells (b=30)", common.small_config(3, 6, 32, heads=2, head_dim=128, block=30, tile_h=2, tile_w=16, seed=98)),
    ("single cells (W=10)", common.small_config(4, 9, 10, heads=2, head_dim=64, block=64, tile_h=4, tile_w=4, seed=99)),
]


@pytest.mark.parametrize("name,cfg", VOTE_LAYOUT_CASES, ids=[c[0] for c in VOTE_LAYOUT_CASES])
@pytest.mark.parametrize("n_text", [0, 45])
def test_block_vote_count_field_layouts(name, cfg, n_text):
    geo = common.oracle_geometry(cfg)
    heads = cfg["heads"]
    for kind, flags in (("entropy", 0), ("uniform", api().TRA_KEEP_DIAGONAL), ("small", 0), ("blocky", 0)):
        ridx = random_ridx(geo, heads, np.random.default_rng(31), kind)
        plan = make_plan(cfg, flags=flags, n_text=n_text)
        S = geo.N + n_text
        full = np.full((heads, S), geo.radii.size - 1, np.uint16)      # text positions: the last candidate
        full[:, : geo.N] = ridx
        mask, row_ptr, col_idx, nnz = run_mask(plan, full)
        ref = np.stack([oracle.block_vote(geo.coord, geo.T, geo.block, geo.theta, full[h], keep_diagonal=bool(flags),
                                          n_text=n_text) for h in range(heads)])
        assert np.array_equal(mask, ref), (name, kind)
        rp, ci = oracle.csr_from_block_mask(ref)
        assert nnz == rp[-1] and np.array_equal(row_ptr.astype(np.int64), rp) and np.array_equal(col_idx[:nnz], ci)
        plan.close()


def _random_geometries(n, seed):
    rng = np.random.default_rng(seed)
    out = []
    for i in range(n):
        block = int(rng.choice([64, 128]))
        th, tw = int(rng.choice([1, 2, 4, 8, 16])), int(rng.choice([4, 8, 16, 32]))
        out.append(common.small_config(int(rng.integers(1, 7)), int(rng.integers(3, 34)), int(rng.integers(3, 50)),
                                       heads=2, head_dim=int(rng.choice([64, 128])), block=block, tile_h=th, tile_w=tw,
                                       gamma=float(rng.choice([0.0, 0.0513, 0.6, 0.95, 2.0])),
                                       tau=float(rng.choice([0.3, 0.5, 0.9, 1.0])), seed=200 + i))
    return out


@pytest.mark.parametrize("cfg", _random_geometries(10, 5), ids=lambda c: f"{c['T']}x{c['H']}x{c['W']}-d{c['head_dim']}-b{c['block']}-"
                                                                         f"t{c['tile_h']}x{c['tile_w']}")
def test_random_geometries_integer_stages_and_token_mask(cfg):
    """Seeded random grids, tile shapes, decay rates and target masses: plan tables, budget, radius,
    block mask and active-block list bit for bit; sparse attention with the token mask against the
    oracle (its slices are row runs for some of these tile shapes and per-key tests for others)."""
    geo = common.oracle_geometry(cfg)
    plan = make_plan(cfg)
    radii, theta, coord = plan.tables()
    assert np.array_equal(radii, geo.radii) and np.array_equal(theta, geo.theta) and np.array_equal(coord, geo.coord)
    assert np.array_equal(plan.count_table(), geo.counts)
    rng = np.random.default_rng(cfg["seed"])
    heads = cfg["heads"]
    H = rng.uniform(0.0, math.log(max(geo.N, 2)), (1, heads, geo.N)).astype(np.float32)
    bud_ref, fragile = oracle.budget(H[0], geo.tau, geo.N)
    ridx_ref = oracle.select_radius(bud_ref, geo.coord, geo.H, geo.W, geo.counts)
    budget, radius, ridx = plan.budget_radius(torch.from_numpy(H).to(DEV))
    ok = ~fragile
    assert fragile.sum() <= 2
    assert np.array_equal(budget.cpu().numpy()[0][ok], bud_ref[ok])
    assert np.array_equal(ridx.cpu().numpy().view(np.uint16)[0][ok], ridx_ref[ok])
    # masks and lists from the oracle's candidate indices
    ridx_t = torch.from_numpy(ridx_ref.astype(np.uint16).view(np.int16)).to(DEV)[None]
    mask, row_ptr, col_idx, nnz = plan.build_block_mask(ridx_t)
    plan.check_status()
    ref = np.stack([oracle.block_vote(geo.coord, geo.T, geo.block, geo.theta, ridx_ref[h]) for h in range(heads)])
    assert np.array_equal(mask.cpu().numpy()[0], ref)
    rp, ci = oracle.csr_from_block_mask(ref)
    assert int(nnz.item()) == rp[-1]
    assert np.array_equal(row_ptr.cpu().numpy().astype(np.int64), rp)
    assert np.array_equal(col_idx.cpu().numpy()[: rp[-1]], ci)
    # dense attention + entropy, block-sparse attention, and the token mask inside the retained blocks
    Q, K, V = tile_major_inputs(cfg, plan)
    Od, Hd, _ = plan.entropy_attn(Q, K, V)
    Os, _ = plan.sparse_attn(Q, K, V, row_ptr, col_idx)
    O, _ = plan.sparse_attn(Q, K, V, row_ptr, col_idx, ridx=ridx_t)
    plan.check_status()
    Qb, Kb, Vb = (workloads.bf16_bits(x)[0] for x in (Q, K, V))
    rows = np.arange(geo.N)
    for h in range(heads):
        rd = oracle.attention_rows(Qb[h], Kb[h], Vb[h], common.scale_of(cfg), rows)
        common.assert_output(Od[0, h], rd["O"], f"dense head {h}")
        assert np.abs(Hd[0, h].cpu().numpy() - rd["H_def"]).max() <= common.ENTROPY_ATOL
        vis0 = oracle.visible_rows(geo.coord, geo.T, geo.block, geo.theta, ridx_ref[h], rows, ref[h][rows // geo.block], 0)
        rs = oracle.attention_rows(Qb[h], Kb[h], Vb[h], common.scale_of(cfg), rows, vis0)
        common.assert_output(Os[0, h], rs["O"], f"sparse head {h}")
        vis1 = oracle.visible_rows(geo.coord, geo.T, geo.block, geo.theta, ridx_ref[h], rows, ref[h][rows // geo.block], 1)
        r = oracle.attention_rows(Qb[h], Kb[h], Vb[h], common.scale_of(cfg), rows, vis1)
        common.assert_output(O[0, h], r["O"], f"token-mask head {h}")
    plan.close()


# Blocks of the paper's sizes (Appendix, hyper-parameter tables: 40, 48, 72, 90, 120 tokens; tiles used as
# blocks) and a few more, each with a tile shape that holds exactly one block or that blocks straddle.
PAPER_BLOCK_CASES = [
    (40, dict(T=3, H=10, W=16, tile_h=5, tile_w=8)),       # 5 x 8 tiles = blocks, N = 480
    (48, dict(T=4, H=12, W=16, tile_h=6, tile_w=8)),       # N = 768
    (56, dict(T=3, H=9, W=14, tile_h=4, tile_w=8)),        # blocks straddle tiles, ragged last block (N = 378)
    (72, dict(T=3, H=16, W=18, tile_h=8, tile_w=9)),       # N = 864
    (90, dict(T=4, H=9, W=20, tile_h=9, tile_w=10)),       # the 9 x 10 tiles of a 45 x 80 frame, N = 720
    (90, dict(T=3, H=11, W=23, tile_h=9, tile_w=10)),      # clipped edge tiles, ragged last block (N = 759)
    (100, dict(T=3, H=10, W=20, tile_h=10, tile_w=10)),    # N = 600
    (120, dict(T=5, H=10, W=24, tile_h=10, tile_w=12)),    # N = 1200
    (33, dict(T=2, H=11, W=9, tile_h=4, tile_w=4)),        # the smallest block the attention calls take
    (90, dict(T=3, H=9, W=20, tile_h=9, tile_w=10, head_dim=64)),
    (40, dict(T=3, H=10, W=16, tile_h=5, tile_w=8, head_dim=64)),
    (112, dict(T=3, H=14, W=16, tile_h=7, tile_w=16, head_dim=64)),
]


@pytest.mark.parametrize("block,grid", PAPER_BLOCK_CASES, ids=[f"b{b}-{g['T']}x{g['H']}x{g['W']}-d{g.get('head_dim', 128)}" for b, g in PAPER_BLOCK_CASES])
def test_paper_block_sizes_whole_path(block, grid):
    """Dense attention + entropy, block vote, tile pairs and block-sparse attention with blocks that are neither
    64 nor 128 tokens: every row against the oracle, lists bit for bit."""
    cfg = common.small_config(grid["T"], grid["H"], grid["W"], heads=2, head_dim=grid.get("head_dim", 128), block=block,
                              tile_h=grid["tile_h"], tile_w=grid["tile_w"], seed=300 + block, s_lo=0.2, s_hi=5.0)
    geo = common.oracle_geometry(cfg)
    plan = make_plan(cfg)
    Q, K, V = tile_major_inputs(cfg, plan)
    O, H, lse = plan.entropy_attn(Q, K, V, want_lse=True)
    O2, _, _ = plan.entropy_attn(Q, K, V, want_entropy=False)
    plan.check_status()
    Qb, Kb, Vb = (workloads.bf16_bits(x)[0] for x in (Q, K, V))
    rows = np.arange(geo.N)
    dense = [oracle.attention_rows(Qb[h], Kb[h], Vb[h], common.scale_of(cfg), rows) for h in range(cfg["heads"])]
    for h in range(cfg["heads"]):
        common.assert_output(O[0, h], dense[h]["O"], f"dense head {h}")
        common.assert_output(O2[0, h], dense[h]["O"], f"dense (no entropy) head {h}")
        assert np.abs(H[0, h].cpu().numpy().astype(np.float64) - dense[h]["H_def"]).max() <= common.ENTROPY_ATOL
        assert np.abs(lse[0, h].cpu().numpy().astype(np.float64) - dense[h]["lse"]).max() <= 1e-3
    # the pipeline's own radii, then two synthetic kinds (whole blocks sharp or diffuse: empty and full rows)
    _, _, ridx_t = plan.budget_radius(H)
    kinds = [("pipeline", ridx_t.cpu().numpy().view(np.uint16)[0])]
    kinds += [(k, random_ridx(geo, cfg["heads"], np.random.default_rng(41), k)) for k in ("blocky", "small")]
    for kind, ridx in kinds:
        ridx_t = torch.from_numpy(np.ascontiguousarray(ridx).view(np.int16)).to(DEV)[None]
        mask, row_ptr, col_idx, nnz, pairs = plan.build_block_mask(ridx_t, want_tile_pairs=True)
        Os, lse_s = plan.sparse_attn(Q, K, V, row_ptr, col_idx, want_lse=True)
        Op, _ = plan.sparse_attn(Q, K, V, row_ptr, col_idx, tile_pairs=pairs)
        plan.check_status()
        assert torch.equal(Os, Op), kind                              # the pairing only moves time
        per_tile = 2 if block <= 64 else 1
        NT = (geo.NB + per_tile - 1) // per_tile
        for h in range(cfg["heads"]):
            used = pairs[h].flatten().cpu().numpy()
            assert sorted(used[used >= 0].tolist()) == list(range(NT)), kind      # a perfect matching of the tiles
            ref_mask = oracle.block_vote(geo.coord, geo.T, geo.block, geo.theta, ridx[h])
            assert np.array_equal(mask.cpu().numpy()[0, h], ref_mask), kind
            vis = oracle.visible_rows(geo.coord, geo.T, geo.block, geo.theta, ridx[h], rows, ref_mask[rows // block], 0)
            ref = oracle.attention_rows(Qb[h], Kb[h], Vb[h], common.scale_of(cfg), rows, vis)
            common.assert_output(Os[0, h], ref["O"], f"sparse ({kind}) head {h}")
            empty = ~vis.any(axis=1)
            assert np.all(Os[0, h].float().cpu().numpy()[empty] == 0)
            got_lse = lse_s[0, h].cpu().numpy().astype(np.float64)
            assert np.all(np.isneginf(got_lse[empty]))
            if (~empty).any():
                assert np.abs(got_lse[~empty] - ref["lse"][~empty]).max() <= 1e-3
    # every block retained: the sparse launch gives the dense launch's bits
    full = torch.ones(1, cfg["heads"], geo.NB, geo.NB, dtype=torch.uint8)
    rp, ci = oracle.csr_from_block_mask(full.numpy()[0])
    Of, _ = plan.sparse_attn(Q, K, V, torch.from_numpy(rp.astype(np.int32)).to(DEV), torch.from_numpy(ci).to(DEV))
    assert torch.equal(Of, O2)
    # the token mask inside blocks needs whole 16-key slices: refused, nothing runs
    with pytest.raises(api().TraError) as err:
        plan.sparse_attn(Q, K, V, row_ptr, col_idx, ridx=ridx_t)
    assert err.value.code == api().TRA_ERR_UNSUPPORTED
    plan.check_status()
    plan.close()


def test_small_blocks_have_a_mask_but_no_attention_launch():
    """Blocks of 32 tokens or fewer: the block mask is built (bit for bit against the oracle), the attention calls
    and the tile-pair table are refused before anything runs, and the mask buffers stay untouched."""
    block = 24
    cfg = common.small_config(4, 12, 20, heads=2, head_dim=128, block=block, tile_h=4, tile_w=8, seed=85)
    geo = common.oracle_geometry(cfg)
    ridx = random_ridx(geo, cfg["heads"], np.random.default_rng(21), "entropy")
    plan = make_plan(cfg)
    mask, row_ptr, col_idx, nnz = run_mask(plan, ridx)
    ref = np.stack([oracle.block_vote(geo.coord, geo.T, geo.block, geo.theta, ridx[h]) for h in range(cfg["heads"])])
    assert np.array_equal(mask, ref)
    rp, ci = oracle.csr_from_block_mask(ref)
    assert nnz == rp[-1] and np.array_equal(row_ptr.astype(np.int64), rp) and np.array_equal(col_idx[:nnz], ci)
    ridx_t = torch.from_numpy(ridx.view(np.int16)).to(DEV)[None]
    sentinel = torch.full((1, cfg["heads"], geo.NB, geo.NB), 7, dtype=torch.uint8, device=DEV)
    with pytest.raises(api().TraError) as err:
        plan.build_block_mask(ridx_t, block_mask=sentinel, want_tile_pairs=True)
    assert err.value.code == api().TRA_ERR_UNSUPPORTED
    Q, K, V = tile_major_inputs(cfg, plan)
    with pytest.raises(api().TraError) as err:
        plan.entropy_attn(Q, K, V)
    assert err.value.code == api().TRA_ERR_UNSUPPORTED
    torch.cuda.synchronize()
    assert bool((sentinel == 7).all())
    plan.check_status()
    plan.close()


def test_block_mask_capacity_error_is_reported():
    cfg = CFG_TINY
    geo = common.oracle_geometry(cfg)
    plan = make_plan(cfg)
    full = np.full((1, geo.N), geo.radii.size - 1, np.uint16)
    ridx = torch.from_numpy(full.view(np.int16)).to(DEV)[None]
    small = torch.full((3 + 64,), -7, dtype=torch.int32, device=DEV)      # 3 entries of capacity, then a guard zone
    _, row_ptr, _, nnz = plan.build_block_mask(ridx, col_idx=small[:3])
    # an asynchronous caller chains the attention call before it reads the status: the list offsets
    # are clamped to the capacity, so the kernel stays inside col_idx
    Q, K, V = tile_major_inputs(cfg, plan, heads=[0])
    O, _ = plan.sparse_attn(Q, K, V, row_ptr, small[:3])
    assert plan.status() == -3          # TRA_ERR_CAPACITY
    assert plan.status() == 0           # cleared by the read
    rp = row_ptr.cpu().numpy()
    assert rp[0] == 0 and np.all(np.diff(rp) >= 0) and rp.max() == 3
    assert int(nnz.item()) == geo.NB * geo.NB            # the true count is still reported
    assert torch.all(small[3:] == -7)                   # nothing was written past the capacity
    assert torch.isfinite(O.float()).all()
    # candidate indices past the table are read as its last entry (full support), not out of bounds
    wild = torch.full((1, 1, geo.N), -1, dtype=torch.int16, device=DEV)     # 65535 as uint16
    m_wild, rp_w, ci_w, _ = plan.build_block_mask(wild)
    m_full, _, _, _ = plan.build_block_mask(ridx)
    assert torch.equal(m_wild, m_full)
    Ow, _ = plan.sparse_attn(Q, K, V, rp_w, ci_w, ridx=wild)
    Of, _ = plan.sparse_attn(Q, K, V, rp_w, ci_w, ridx=ridx)
    plan.check_status()
    assert torch.equal(Ow, Of)
    plan.close()


def test_block_mask_sampled_rows_wan13b():
    # full-size integer stage at the 32,760-token shape: GPU over all rows, oracle on sampled rows
    cfg = workloads.CONFIGS["wan1.3b-480p"]
    geo = common.oracle_geometry(cfg)
    plan = make_plan(cfg)
    rng = np.random.default_rng(13)
    heads = 2
    ridx = random_ridx(geo, heads, rng, "entropy")
    mask, row_ptr, col_idx, nnz = run_mask(plan, ridx)
    u_list = np.unique(np.concatenate([[0, 1, geo.NB - 2, geo.NB - 1], rng.integers(0, geo.NB, 12)]))
    for h in range(heads):
        ref = oracle.block_vote(geo.coord, geo.T, geo.block, geo.theta, ridx[h], u_list=u_list)
        assert np.array_equal(mask[h][u_list], ref)
    rp, ci = oracle.csr_from_block_mask(mask)      # CSR must be the ascending list of the mask itself
    assert np.array_equal(row_ptr.astype(np.int64), rp) and np.array_equal(col_idx[:nnz], ci)
    assert 0.005 < mask.mean() < 0.98
    plan.close()


# ----------------------------------------------------------------------------- dense attention + entropy
def oracle_dense_rows(cfg, geo, Qb, Kb, Vb, h, rows):
    return oracle.attention_rows(Qb[h], Kb[h], Vb[h], common.scale_of(cfg), rows)


@pytest.mark.parametrize("cfg", SMALL, ids=IDS)
def test_entropy_attn_all_rows(cfg):
    geo = common.oracle_geometry(cfg)
    plan = make_plan(cfg)
    Q, K, V = tile_major_inputs(cfg, plan)
    O, H, lse = plan.entropy_attn(Q, K, V, want_lse=True)
    O2, _, _ = plan.entropy_attn(Q, K, V, want_entropy=False)       # plain dense: same output
    plan.check_status()
    Qb, Kb, Vb = (workloads.bf16_bits(x)[0] for x in (Q, K, V))
    rows = np.arange(geo.N)
    for h in range(cfg["heads"]):
        ref = oracle_dense_rows(cfg, geo, Qb, Kb, Vb, h, rows)
        common.assert_output(O[0, h], ref["O"], f"dense head {h}")
        common.assert_output(O2[0, h], ref["O"], f"dense(no entropy) head {h}")
        dH = np.abs(H[0, h].cpu().numpy().astype(np.float64) - ref["H_def"])
        assert dH.max() <= common.ENTROPY_ATOL, dH.max()
        dl = np.abs(lse[0, h].cpu().numpy().astype(np.float64) - ref["lse"])
        assert dl.max() <= 1e-3, dl.max()
    plan.close()


def test_entropy_attn_uniform_and_one_hot_rows():
    # Q = 0 -> uniform attention: H = log N, O = mean of V.  A huge query -> near one-hot: H ~ 0.
    cfg = CFG_RAGGED128
    geo = common.oracle_geometry(cfg)
    plan = make_plan(cfg)
    Q, K, V = tile_major_inputs(cfg, plan)
    Q[:, 0] = 0
    Q[:, 1] = K[:, 1] * 40
    O, H, _ = plan.entropy_attn(Q, K, V)
    plan.check_status()
    assert torch.allclose(H[0, 0], torch.full_like(H[0, 0], math.log(geo.N)), atol=1e-4)
    assert torch.allclose(O[0, 0].float(), V[0, 0].float().mean(0, keepdim=True).expand(geo.N, -1), atol=1e-2)
    Qb, Kb, Vb = (workloads.bf16_bits(x)[0] for x in (Q, K, V))
    ref = oracle.attention_rows(Qb[1], Kb[1], Vb[1], common.scale_of(cfg), np.arange(geo.N))
    assert np.abs(H[0, 1].cpu().numpy() - ref["H_def"]).max() <= common.ENTROPY_ATOL
    common.assert_output(O[0, 1], ref["O"], "one-hot head")
    plan.close()


# ----------------------------------------------------------------------------- sparse attention
def sparse_case(cfg, ridx_kind, flags=0, seed=14):
    geo = common.oracle_geometry(cfg)
    plan = make_plan(cfg, flags=flags)
    Q, K, V = tile_major_inputs(cfg, plan)
    ridx = random_ridx(geo, cfg["heads"], np.random.default_rng(seed), ridx_kind)
    ridx_t = torch.from_numpy(ridx.view(np.int16)).to(DEV)[None]
    mask, row_ptr, col_idx, nnz = plan.build_block_mask(ridx_t)
    O, lse = plan.sparse_attn(Q, K, V, row_ptr, col_idx, want_lse=True)
    plan.check_status()
    return geo, plan, (Q, K, V), ridx, mask.cpu().numpy()[0], O, lse


@pytest.mark.parametrize("cfg", SMALL, ids=IDS)
@pytest.mark.parametrize("kind", ["entropy", "blocky", "small"])
def test_sparse_attn_all_rows(cfg, kind):
    geo, plan, (Q, K, V), ridx, mask, O, lse = sparse_case(cfg, kind)
    Qb, Kb, Vb = (workloads.bf16_bits(x)[0] for x in (Q, K, V))
    rows = np.arange(geo.N)
    n_empty = 0
    for h in range(cfg["heads"]):
        ref_mask = oracle.block_vote(geo.coord, geo.T, geo.block, geo.theta, ridx[h])
        assert np.array_equal(mask[h], ref_mask)
        vis = oracle.visible_rows(geo.coord, geo.T, geo.block, geo.theta, ridx[h], rows,
                                  ref_mask[rows // geo.block], 0)
        ref = oracle.attention_rows(Qb[h], Kb[h], Vb[h], common.scale_of(cfg), rows, vis)
        common.assert_output(O[0, h], ref["O"], f"sparse head {h}")
        empty = ~vis.any(axis=1)
        n_empty += int(empty.sum())
        got = O[0, h].float().cpu().numpy()
        assert np.all(got[empty] == 0)                               # empty block row -> zeros
        got_lse = lse[0, h].cpu().numpy().astype(np.float64)
        assert np.all(np.isneginf(got_lse[empty]))
        if (~empty).any():
            assert np.abs(got_lse[~empty] - ref["lse"][~empty]).max() <= 1e-3
    if kind == "small":
        assert n_empty > 0                                           # the degenerate case is exercised
    plan.close()


CFG_FRAMES128 = common.small_config(5, 32, 48, heads=2, head_dim=128, block=128, tile_h=8, tile_w=16, seed=84,
                                    s_lo=0.2, s_hi=5.0)      # 12 query tiles per frame


@pytest.mark.parametrize("cfg,n_text,gamma", [(CFG_TINY, 0, None), (CFG_RAGGED64, 50, None), (CFG_D128_B64, 0, None),
                                              (CFG_MID128, 0, None), (CFG_FRAMES128, 0, None),
                                              (CFG_FRAMES128, 100, 0.05)],
                         ids=["tiny", "ragged64+text", "d128_b64", "mid128", "frames128", "frames128+text-slow-decay"])
def test_tile_pair_table(cfg, n_text, gamma):
    """The tile-pair table of the block-mask call: every 128-row query tile appears exactly once, and
    the sparse launch gives the same bits with it as with consecutive tiles (plain and with the token
    mask).  The last two shapes have more tiles per frame than the pairing window, so tiles one frame
    ahead are candidates too."""
    if gamma is not None:
        cfg = dict(cfg, gamma=gamma)
    geo = common.oracle_geometry(cfg)
    plan = make_plan(cfg, n_text=n_text)
    S = geo.N + n_text
    heads = cfg["heads"]
    Qr, Kr, Vr = workloads.make_qkv(cfg, DEV)
    if n_text:
        Qr, Kr, Vr = workloads.append_text(Qr, Kr, Vr, cfg, n_text)
    Q, K, V = (plan.tile_major_gather(x) for x in (Qr, Kr, Vr))
    _, H, _ = plan.entropy_attn(Q, K, V)
    _, _, ridx = plan.budget_radius(H)
    mask, row_ptr, col_idx, nnz, pairs = plan.build_block_mask(ridx, want_tile_pairs=True)
    plan.check_status()
    n_tiles = (S + 127) // 128 if 128 % geo.block == 0 else (S + geo.block - 1) // geo.block
    p = pairs.reshape(heads, -1, 2).cpu().numpy()
    assert p.shape[1] == (n_tiles + 1) // 2
    for h in range(heads):
        assert np.array_equal(np.sort(p[h][p[h] >= 0]), np.arange(n_tiles))
        assert (p[h][:, 0] >= 0).all()                               # only the second slot may be empty
    O1, lse1 = plan.sparse_attn(Q, K, V, row_ptr, col_idx, tile_pairs=pairs, want_lse=True)
    O2, lse2 = plan.sparse_attn(Q, K, V, row_ptr, col_idx, want_lse=True)
    assert torch.equal(O1, O2) and torch.equal(lse1, lse2)
    T1, _ = plan.sparse_attn(Q, K, V, row_ptr, col_idx, ridx=ridx, tile_pairs=pairs)
    T2, _ = plan.sparse_attn(Q, K, V, row_ptr, col_idx, ridx=ridx)
    plan.check_status()
    assert torch.equal(T1, T2)
    plan.close()


@pytest.mark.parametrize("cfg,n_text", [(CFG_TINY, 0), (CFG_RAGGED64, 0), (CFG_RAGGED128, 0), (CFG_MID128, 0),
                                        (CFG_RAGGED64, 50), (CFG_RAGGED128, 200)],
                         ids=["tiny", "ragged64", "ragged128", "mid128", "ragged64+text", "ragged128+text"])
@pytest.mark.parametrize("kind", ["entropy", "small", "uniform"])
def test_sparse_attn_with_token_mask(cfg, n_text, kind):
    """ridx passed to the sparse call: block list AND the token mask of Eq. 15 (oracle mode 1)."""
    geo = common.oracle_geometry(cfg)
    plan = make_plan(cfg, n_text=n_text)
    S, b = geo.N + n_text, geo.block
    NB = (S + b - 1) // b
    Qr, Kr, Vr = workloads.make_qkv(cfg, DEV)
    if n_text:
        Qr, Kr, Vr = workloads.append_text(Qr, Kr, Vr, cfg, n_text)
    Q, K, V = (plan.tile_major_gather(x) for x in (Qr, Kr, Vr))
    rv = random_ridx(geo, cfg["heads"], np.random.default_rng(31), kind)
    ridx = np.full((cfg["heads"], S), geo.radii.size - 1, np.uint16)
    ridx[:, : geo.N] = rv
    ridx_t = torch.from_numpy(ridx.view(np.int16)).to(DEV)[None]
    mask, row_ptr, col_idx, nnz = plan.build_block_mask(ridx_t)
    O, lse = plan.sparse_attn(Q, K, V, row_ptr, col_idx, ridx=ridx_t, want_lse=True)
    plan.check_status()
    Qb, Kb, Vb = (workloads.bf16_bits(x)[0] for x in (Q, K, V))
    rows = np.arange(S)
    n_empty = n_masked = 0
    for h in range(cfg["heads"]):
        ref_mask = oracle.block_vote(geo.coord, geo.T, b, geo.theta, ridx[h], u_list=np.arange(NB), n_text=n_text)
        assert np.array_equal(mask[0, h].cpu().numpy(), ref_mask)
        vis0 = oracle.visible_rows(geo.coord, geo.T, b, geo.theta, ridx[h], rows, ref_mask[rows // b], 0, n_text=n_text)
        vis1 = oracle.visible_rows(geo.coord, geo.T, b, geo.theta, ridx[h], rows, ref_mask[rows // b], 1, n_text=n_text)
        n_masked += int(vis0.sum() - vis1.sum())
        ref = oracle.attention_rows(Qb[h], Kb[h], Vb[h], common.scale_of(cfg), rows, vis1)
        common.assert_output(O[0, h], ref["O"], f"token-mask head {h}")
        empty = ~vis1.astype(bool).any(axis=1)
        n_empty += int(empty.sum())
        assert np.all(O[0, h].float().cpu().numpy()[empty] == 0)
        assert np.all(np.isneginf(lse[0, h].cpu().numpy()[empty]))
    if kind == "uniform":
        assert n_masked > 0                   # the token mask removed pairs the block list kept
    plan.close()


@pytest.mark.parametrize("cfg,n_text", [(CFG_TINY, 0), (CFG_RAGGED64, 0), (CFG_RAGGED128, 0), (CFG_MID128, 0),
                                        (CFG_RAGGED64, 50), (CFG_MID128, 100)],
                         ids=["tiny", "ragged64", "ragged128", "mid128", "ragged64+text", "mid128+text"])
@pytest.mark.parametrize("kind", ["entropy", "small", "uniform"])
def test_sparse_attn_token_level_without_block_list(cfg, n_text, kind):
    """ridx and no block list: Eq. 16 itself (oracle mode 2) — every query over exactly the keys inside
    its disk; the kernel derives the reachable key blocks from the plan's boxes."""
    geo = common.oracle_geometry(cfg)
    plan = make_plan(cfg, n_text=n_text)
    S, b = geo.N + n_text, geo.block
    Qr, Kr, Vr = workloads.make_qkv(cfg, DEV)
    if n_text:
        Qr, Kr, Vr = workloads.append_text(Qr, Kr, Vr, cfg, n_text)
    Q, K, V = (plan.tile_major_gather(x) for x in (Qr, Kr, Vr))
    rv = random_ridx(geo, cfg["heads"], np.random.default_rng(41), kind)
    ridx = np.full((cfg["heads"], S), geo.radii.size - 1, np.uint16)
    ridx[:, : geo.N] = rv
    ridx_t = torch.from_numpy(ridx.view(np.int16)).to(DEV)[None]
    O, lse = plan.sparse_attn(Q, K, V, None, None, ridx=ridx_t, want_lse=True)
    plan.check_status()
    Qb, Kb, Vb = (workloads.bf16_bits(x)[0] for x in (Q, K, V))
    rows = np.arange(S)
    for h in range(cfg["heads"]):
        vis2 = oracle.visible_rows(geo.coord, geo.T, b, geo.theta, ridx[h], rows, None, 2, n_text=n_text)
        assert vis2.any(axis=1).all()              # a query always sees itself
        ref = oracle.attention_rows(Qb[h], Kb[h], Vb[h], common.scale_of(cfg), rows, vis2)
        common.assert_output(O[0, h], ref["O"], f"token-level head {h}")
        assert np.abs(lse[0, h].cpu().numpy().astype(np.float64) - ref["lse"]).max() <= 1e-3
    with pytest.raises(api().TraError):
        plan.sparse_attn(Q, K, V, None, None)       # neither a block list nor radii
    plan.close()


def test_sparse_attn_full_mask_equals_dense():
    # every block retained: the sparse call reproduces dense attention (full-support radius)
    cfg = CFG_RAGGED128
    geo = common.oracle_geometry(cfg)
    plan = make_plan(cfg)
    Q, K, V = tile_major_inputs(cfg, plan)
    full = np.full((cfg["heads"], geo.N), geo.radii.size - 1, np.uint16)
    mask, row_ptr, col_idx, nnz = plan.build_block_mask(torch.from_numpy(full.view(np.int16)).to(DEV)[None])
    assert int(nnz.item()) == cfg["heads"] * geo.NB * geo.NB
    Os, _ = plan.sparse_attn(Q, K, V, row_ptr, col_idx)
    Od, _, _ = plan.entropy_attn(Q, K, V, want_entropy=False)
    plan.check_status()
    assert torch.equal(Os, Od)
    plan.close()


# ----------------------------------------------------------------------------- the chained pipeline
@pytest.mark.parametrize("cfg", [CFG_TINY, CFG_MID128], ids=["tiny", "mid128"])
def test_pipeline_chained_on_gpu(cfg):
    """entropy_attn -> budget_radius -> build_block_mask -> sparse_attn with the GPU's own
    intermediate results; the oracle is fed the GPU's fp32 entropies for the integer stages."""
    geo = common.oracle_geometry(cfg)
    plan = make_plan(cfg)
    Q, K, V = tile_major_inputs(cfg, plan)
    _, H, _ = plan.entropy_attn(Q, K, V)
    budget, radius, ridx = plan.budget_radius(H)
    mask, row_ptr, col_idx, nnz = plan.build_block_mask(ridx)
    O, _ = plan.sparse_attn(Q, K, V, row_ptr, col_idx)
    plan.check_status()
    Hn = H.cpu().numpy()[0]
    bud_ref, fragile = oracle.budget(Hn, geo.tau, geo.N)
    assert not fragile.any()
    ridx_ref = oracle.select_radius(bud_ref, geo.coord, geo.H, geo.W, geo.counts)
    assert np.array_equal(budget.cpu().numpy()[0], bud_ref)
    assert np.array_equal(ridx.cpu().numpy().view(np.uint16)[0], ridx_ref)
    Qb, Kb, Vb = (workloads.bf16_bits(x)[0] for x in (Q, K, V))
    rows = np.arange(geo.N)
    density = []
    for h in range(cfg["heads"]):
        ref_mask = oracle.block_vote(geo.coord, geo.T, geo.block, geo.theta, ridx_ref[h])
        assert np.array_equal(mask.cpu().numpy()[0, h], ref_mask)
        density.append(ref_mask.mean())
        vis = oracle.visible_rows(geo.coord, geo.T, geo.block, geo.theta, ridx_ref[h], rows,
                                  ref_mask[rows // geo.block], 0)
        ref = oracle.attention_rows(Qb[h], Kb[h], Vb[h], common.scale_of(cfg), rows, vis)
        common.assert_output(O[0, h], ref["O"], f"pipeline head {h}")
        # the entropy the GPU produced is the oracle's, within tolerance
        dense = oracle.attention_rows(Qb[h], Kb[h], Vb[h], common.scale_of(cfg), rows)
        assert np.abs(Hn[h] - dense["H_def"]).max() <= common.ENTROPY_ATOL
    assert 0.0 < np.mean(density) <= 1.0
    plan.close()


# ----------------------------------------------------------------------------- full-size sampled parity
def sampled_rows(geo, rng, n_random):
    b = geo.block
    fixed = [0, b - 1, b, 2 * b - 1, 2 * b, geo.N - 1, (geo.NB - 1) * b, (geo.NB - 1) * b - 1,
             geo.N // 2, geo.N // 2 + 1]
    return np.unique(np.concatenate([fixed, rng.integers(0, geo.N, n_random)])).astype(np.int32)


@pytest.mark.parametrize("name,heads_checked,n_random",
                         [("wan1.3b-480p", (0, 3, 7, 11), 100), ("wan14b-720p", (0, 13, 26, 39), 100),
                          ("hunyuan-720p", (0, 7, 15, 23), 60)])
def test_full_size_sampled_rows(name, heads_checked, n_random):
    """At the three full-size shapes, all heads resident, in the launch configuration the benchmark times:
    sampled (head, row) pairs of dense attention + entropy, the integer stages of their block
    rows, sparse attention, and sparse attention with the token mask inside the blocks.  Rows cover the first / last blocks and the ragged tail."""
    cfg = workloads.CONFIGS[name]
    geo = common.oracle_geometry(cfg)
    plan = make_plan(cfg)
    Q, K, V = tile_major_inputs(cfg, plan)
    O, H, _ = plan.entropy_attn(Q, K, V)
    budget, radius, ridx = plan.budget_radius(H)
    mask, row_ptr, col_idx, nnz = plan.build_block_mask(ridx)
    Os, _ = plan.sparse_attn(Q, K, V, row_ptr, col_idx)
    Ot, _ = plan.sparse_attn(Q, K, V, row_ptr, col_idx, ridx=ridx)      # token mask inside the blocks
    Oe, _ = plan.sparse_attn(Q, K, V, None, None, ridx=ridx)            # Eq. 16 itself, no block list
    plan.check_status()
    rng = np.random.default_rng(15)
    for h in heads_checked:
        rows = sampled_rows(geo, rng, n_random)
        rows_t = torch.from_numpy(rows).long().to(DEV)
        Qb, Kb, Vb = (workloads.bf16_bits(x[0, h]) for x in (Q, K, V))
        ref = oracle.attention_rows(Qb, Kb, Vb, common.scale_of(cfg), rows)
        common.assert_output(O[0, h][rows_t], ref["O"], f"dense {name} h{h}")
        Hn = H[0, h].cpu().numpy()
        dH = np.abs(Hn[rows] - ref["H_def"])
        assert dH.max() <= common.ENTROPY_ATOL, dH.max()
        # integer stages of this head, fed with the GPU's fp32 entropies: bit-exact
        bud_ref, fragile = oracle.budget(Hn[None], geo.tau, geo.N)
        assert fragile.sum() <= 1
        ridx_ref = oracle.select_radius(bud_ref, geo.coord, geo.H, geo.W, geo.counts)[0]
        ok = ~fragile[0]
        assert np.array_equal(budget[0, h].cpu().numpy()[ok], bud_ref[0][ok])
        ridx_np = ridx[0, h].cpu().numpy().view(np.uint16)
        assert np.array_equal(ridx_np[ok], ridx_ref[ok])
        u_list = np.unique(rows // geo.block)
        ref_mask = oracle.block_vote(geo.coord, geo.T, geo.block, geo.theta, ridx_np, u_list=u_list)
        assert np.array_equal(mask[0, h].cpu().numpy()[u_list], ref_mask)
        block_rows = ref_mask[np.searchsorted(u_list, rows // geo.block)]
        vis = oracle.visible_rows(geo.coord, geo.T, geo.block, geo.theta, ridx_np, rows, block_rows, 0)
        refs = oracle.attention_rows(Qb, Kb, Vb, common.scale_of(cfg), rows, vis)
        common.assert_output(Os[0, h][rows_t], refs["O"], f"sparse {name} h{h}")
        vis1 = oracle.visible_rows(geo.coord, geo.T, geo.block, geo.theta, ridx_np, rows, block_rows, 1)
        assert vis1.sum() < vis.sum()
        reft = oracle.attention_rows(Qb, Kb, Vb, common.scale_of(cfg), rows, vis1)
        common.assert_output(Ot[0, h][rows_t], reft["O"], f"token mask {name} h{h}")
        vis2 = oracle.visible_rows(geo.coord, geo.T, geo.block, geo.theta, ridx_np, rows, None, 2)
        refe = oracle.attention_rows(Qb, Kb, Vb, common.scale_of(cfg), rows, vis2)
        common.assert_output(Oe[0, h][rows_t], refe["O"], f"token level {name} h{h}")
    # CSR of every head is the ascending list of the mask the same call wrote
    m = mask[0].reshape(-1, geo.NB).bool()
    counts = m.sum(dim=1)
    assert torch.equal(row_ptr[1:].long() - row_ptr[:-1].long(), counts)
    assert int(nnz.item()) == int(counts.sum().item())
    cols = torch.nonzero(m)[:, 1].int()
    assert torch.equal(col_idx[: cols.numel()], cols)
    density = float(counts.sum().item()) / (cfg["heads"] * geo.NB * geo.NB)
    assert 0.02 < density < 0.9, density
    plan.close()


# ----------------------------------------------------------------------------- joint text-video attention
TEXT_CASES = [(CFG_TINY, 40), (CFG_RAGGED64, 50), (CFG_RAGGED128, 200), (CFG_MID128, 100)]


@pytest.mark.parametrize("cfg,n_text", TEXT_CASES, ids=["tiny+40", "ragged64+50", "ragged128+200", "mid128+100"])
def test_text_tokens_pipeline(cfg, n_text):
    """Section 3.2 (last paragraph) / Algorithm 1 with S = N + n_text: text tokens stay in place in
    the tile-major order, get the full-support candidate, their blocks are dense, video blocks vote
    over video tokens only, and both attentions run over the whole sequence."""
    geo = common.oracle_geometry(cfg)
    plan = make_plan(cfg, n_text=n_text)
    S, b = geo.N + n_text, geo.block
    NB = (S + b - 1) // b
    assert plan.N == S and plan.N_video == geo.N and plan.NB == NB
    Qr, Kr, Vr = workloads.append_text(*workloads.make_qkv(cfg, DEV), cfg, n_text)
    Q, K, V = (plan.tile_major_gather(x) for x in (Qr, Kr, Vr))
    perm = np.concatenate([common.raster_of_pos(geo), np.arange(geo.N, S)])
    assert torch.equal(Q.cpu(), Qr.cpu()[:, :, torch.from_numpy(perm).long(), :])
    assert torch.equal(plan.tile_major_scatter(Q), Qr)

    O, H, _ = plan.entropy_attn(Q, K, V)
    budget, radius, ridx = plan.budget_radius(H)
    mask, row_ptr, col_idx, nnz = plan.build_block_mask(ridx)
    Os, _ = plan.sparse_attn(Q, K, V, row_ptr, col_idx)
    plan.check_status()

    Hn = H.cpu().numpy()[0]
    ridx_np = ridx.cpu().numpy().view(np.uint16)[0]
    assert np.all(ridx_np[:, geo.N:] == geo.radii.size - 1)
    assert np.all(budget.cpu().numpy()[0][:, geo.N:] == S)
    assert np.all(np.isinf(radius.cpu().numpy()[0][:, geo.N:]))
    bud_ref, fragile = oracle.budget(Hn[:, : geo.N], geo.tau, geo.N)
    assert not fragile.any()
    ridx_ref = oracle.select_radius(bud_ref, geo.coord, geo.H, geo.W, geo.counts)
    assert np.array_equal(ridx_np[:, : geo.N], ridx_ref)
    Qb, Kb, Vb = (workloads.bf16_bits(x)[0] for x in (Q, K, V))
    rows = np.arange(S)
    for h in range(cfg["heads"]):
        dense = oracle.attention_rows(Qb[h], Kb[h], Vb[h], common.scale_of(cfg), rows)
        common.assert_output(O[0, h], dense["O"], f"dense+text head {h}")
        assert np.abs(Hn[h] - dense["H_def"]).max() <= common.ENTROPY_ATOL
        ref_mask = oracle.block_vote(geo.coord, geo.T, b, geo.theta, ridx_np[h], u_list=np.arange(NB),
                                     n_text=n_text)
        assert np.array_equal(mask[0, h].cpu().numpy(), ref_mask)
        vis = oracle.visible_rows(geo.coord, geo.T, b, geo.theta, ridx_np[h], rows, ref_mask[rows // b], 0,
                                  n_text=n_text)
        ref = oracle.attention_rows(Qb[h], Kb[h], Vb[h], common.scale_of(cfg), rows, vis)
        common.assert_output(Os[0, h], ref["O"], f"sparse+text head {h}")
    rp, ci = oracle.csr_from_block_mask(mask[0].cpu().numpy())
    assert np.array_equal(row_ptr.cpu().numpy().astype(np.int64), rp)
    assert np.array_equal(col_idx.cpu().numpy()[: int(nnz.item())], ci)
    plan.close()


# ----------------------------------------------------------------------------- reuse across steps
def test_mask_reuse_across_denoising_steps():
    """Warm-up reuse (Section 3.3): radii and mask of the last dense step serve every later step;
    the sparse call never writes them, and with drifted Q/K it still equals the oracle under the
    frozen mask."""
    cfg = CFG_MID128
    geo = common.oracle_geometry(cfg)
    plan = make_plan(cfg)
    Q, K, V = tile_major_inputs(cfg, plan)
    q_state, k_state = Q.float(), K.float()
    _, H, _ = plan.entropy_attn(Q, K, V)
    _, _, ridx = plan.budget_radius(H)
    mask, row_ptr, col_idx, nnz = plan.build_block_mask(ridx)
    frozen = [t.clone() for t in (ridx, mask, row_ptr, col_idx)]
    ridx_np = ridx.cpu().numpy().view(np.uint16)[0]
    rows = np.arange(geo.N)
    for step in range(3):
        workloads.drift_(q_state, step, 5)
        workloads.drift_(k_state, step, 6)
        Q.copy_(q_state)
        K.copy_(k_state)
        O, _ = plan.sparse_attn(Q, K, V, row_ptr, col_idx)
        plan.check_status()
        for t, f in zip((ridx, mask, row_ptr, col_idx), frozen):
            assert torch.equal(t, f)
        Qb, Kb, Vb = (workloads.bf16_bits(x)[0] for x in (Q, K, V))
        for h in range(cfg["heads"]):
            mh = frozen[1][0, h].cpu().numpy()
            vis = oracle.visible_rows(geo.coord, geo.T, geo.block, geo.theta, ridx_np[h], rows,
                                      mh[rows // geo.block], 0)
            ref = oracle.attention_rows(Qb[h], Kb[h], Vb[h], common.scale_of(cfg), rows, vis)
            common.assert_output(O[0, h], ref["O"], f"step {step} head {h}")
    plan.close()


def test_bounded_wait_reports_timeout_and_context_survives():
    """A device-side wait that can never be satisfied gives up after its limit, records
    TRA_ERR_TIMEOUT in the plan status and the kernel returns; later calls work normally."""
    cfg = CFG_TINY
    plan = make_plan(cfg)
    assert plan.status() == 0
    plan.selftest_wait_timeout(limit_ms=20)
    assert plan.status() == -5          # TRA_ERR_TIMEOUT
    assert plan.status() == 0           # cleared by the read
    Q, K, V = tile_major_inputs(cfg, plan)
    O, H, _ = plan.entropy_attn(Q, K, V)
    plan.check_status()
    assert torch.isfinite(H).all() and torch.isfinite(O.float()).all()
    plan.close()


def test_batch_and_side_stream():
    """B = 2 equals two B = 1 calls, and calls enqueued on a non-default stream give the same bits."""
    cfg = CFG_MID128
    plan = make_plan(cfg)
    Q1, K1, V1 = tile_major_inputs(cfg, plan)
    cfg2 = dict(cfg, seed=cfg["seed"] + 1)
    Q2, K2, V2 = tile_major_inputs(cfg2, plan)
    Q, K, V = (torch.cat([a, b], dim=0).contiguous() for a, b in ((Q1, Q2), (K1, K2), (V1, V2)))
    O, H, _ = plan.entropy_attn(Q, K, V)
    _, _, ridx = plan.budget_radius(H)
    mask, row_ptr, col_idx, nnz, pairs = plan.build_block_mask(ridx, want_tile_pairs=True)
    Os, _ = plan.sparse_attn(Q, K, V, row_ptr, col_idx, tile_pairs=pairs)      # the table is per (batch, head)
    Ot, _ = plan.sparse_attn(Q, K, V, row_ptr, col_idx, ridx=ridx, tile_pairs=pairs)
    plan.check_status()
    assert torch.equal(Os, plan.sparse_attn(Q, K, V, row_ptr, col_idx)[0])
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    for b, (q, k, v) in enumerate(((Q1, K1, V1), (Q2, K2, V2))):
        with torch.cuda.stream(side):
            o, h, _ = plan.entropy_attn(q, k, v)
            _, _, r = plan.budget_radius(h)
            m, rp, ci, nz = plan.build_block_mask(r)
            os_, _ = plan.sparse_attn(q, k, v, rp, ci)
            ot_, _ = plan.sparse_attn(q, k, v, rp, ci, ridx=r)
        side.synchronize()
        assert torch.equal(o[0], O[b]) and torch.equal(h[0], H[b])
        assert torch.equal(r[0], ridx[b]) and torch.equal(m[0], mask[b])
        assert torch.equal(os_[0], Os[b]) and torch.equal(ot_[0], Ot[b])
    plan.check_status()
    plan.close()


@pytest.mark.parametrize("cfg", [dict(CFG_MID128, heads=5),
                                 common.small_config(4, 9, 20, heads=5, head_dim=128, block=90, tile_h=9, tile_w=10,
                                                     seed=87, s_lo=0.2, s_hi=5.0)], ids=["mid128", "b90"])
def test_host_pipeline_matches_device_path(cfg):
    """The head-group pipeline over pinned host tensors (copies overlapped with kernels) returns the
    bits of the one-shot device path, with a ragged last group and with one group."""
    plan = make_plan(cfg)
    Qr, Kr, Vr = workloads.make_qkv(cfg, "cuda")
    Q, K, V = (plan.tile_major_gather(x) for x in (Qr, Kr, Vr))
    _, H, _ = plan.entropy_attn(Q, K, V)
    _, _, ridx = plan.budget_radius(H)
    _, row_ptr, col_idx, _ = plan.build_block_mask(ridx)
    Os, _ = plan.sparse_attn(Q, K, V, row_ptr, col_idx)
    expect = plan.tile_major_scatter(Os).cpu()
    host = [t.cpu().pin_memory() for t in (Qr, Kr, Vr)]
    for group, first in ((2, None), (8, None), (3, 1)):
        pipe = api().HostPipeline(plan, cfg["heads"], group=group, first_group=first)
        out = torch.zeros(expect.shape, dtype=torch.bfloat16).pin_memory()
        for _ in range(2):                      # the second run reuses every buffer
            launches = pipe.run(host[0], host[1], host[2], out)
            torch.cuda.synchronize()
            assert torch.equal(out, expect)
        sizes = api().HostPipeline.group_sizes(cfg["heads"], pipe.group, pipe.first_group)
        assert sum(sizes) == cfg["heads"] and max(sizes) <= pipe.group and sizes[0] <= pipe.first_group
        assert launches == 11 * len(sizes)
    with pytest.raises(ValueError):
        pipe.run(Qr, host[1], host[2], out)     # a device tensor where a pinned host tensor belongs
    # the C entry point refuses a workspace that is too small or misaligned, before any work
    import ctypes
    lib, vp = api()._lib, ctypes.c_void_p
    args = [vp(t.data_ptr()) for t in host] + [vp(out.data_ptr())]
    need = pipe.workspace_bytes
    assert lib.tra_hot_path_host(plan._h, *args, vp(pipe._ws_ptr), need - 1, cfg["heads"], pipe.group, 1, 1.0,
                                 None) == -3
    assert lib.tra_hot_path_host(plan._h, *args, vp(pipe._ws_ptr + 16), need, cfg["heads"], pipe.group, 1, 1.0,
                                 None) == -1
    assert lib.tra_hot_path_host(plan._h, *args, vp(pipe._ws_ptr), need, 0, pipe.group, 1, 1.0, None) == -1
    plan.check_status()
    plan.close()


# Grids whose 16-position runs are 16 consecutive raster rows (W and the tile width multiples of 16).
RASTER_CASES = [
    ("b128", common.small_config(4, 12, 32, heads=2, head_dim=128, block=128, tile_h=8, tile_w=16, seed=101, s_lo=0.2,
                                 s_hi=5.0), 0),
    ("b128 clipped tiles + text", common.small_config(3, 11, 48, heads=2, head_dim=128, block=128, tile_h=8, tile_w=16,
                                                      seed=102), 70),
    ("b64 d64", common.small_config(3, 8, 48, heads=2, head_dim=64, block=64, tile_h=4, tile_w=16, seed=103), 0),
    ("b96", common.small_config(3, 12, 32, heads=2, head_dim=128, block=96, tile_h=6, tile_w=16, seed=104), 0),
    ("b48 + text", common.small_config(4, 9, 16, heads=2, head_dim=128, block=48, tile_h=3, tile_w=16, seed=105), 20),
]


@pytest.mark.parametrize("name,cfg,n_text", RASTER_CASES, ids=[c[0] for c in RASTER_CASES])
def test_raster_order_plan_equals_gather_attend_scatter(name, cfg, n_text):
    """A plan with TRA_ORDER_RASTER reads Q, K, V in raster order through 16-row TMA boxes and writes O in raster
    order: every launch gives the bits of gather -> the same launch on tile-major tensors -> scatter, and the
    per-token outputs (entropy, lse), which stay tile-major, are identical."""
    plan_t = make_plan(cfg, n_text=n_text)
    plan_r = make_plan(cfg, n_text=n_text, flags=api().TRA_ORDER_RASTER)
    Qr, Kr, Vr = workloads.make_qkv(cfg, DEV)
    if n_text:
        Qr, Kr, Vr = workloads.append_text(Qr, Kr, Vr, cfg, n_text)
    Qr, Kr, Vr = (x.contiguous() for x in (Qr, Kr, Vr))
    Q, K, V = (plan_t.tile_major_gather(x) for x in (Qr, Kr, Vr))
    token_mask = cfg["block"] in (64, 128)
    # dense + entropy, plain dense
    O_t, H_t, lse_t = plan_t.entropy_attn(Q, K, V, want_lse=True)
    O_r, H_r, lse_r = plan_r.entropy_attn(Qr, Kr, Vr, want_lse=True)
    assert torch.equal(O_r, plan_t.tile_major_scatter(O_t)) and torch.equal(H_r, H_t) and torch.equal(lse_r, lse_t)
    P_t, _, _ = plan_t.entropy_attn(Q, K, V, want_entropy=False)
    P_r, _, _ = plan_r.entropy_attn(Qr, Kr, Vr, want_entropy=False)
    assert torch.equal(P_r, plan_t.tile_major_scatter(P_t))
    # the integer stages do not depend on the order of Q, K, V
    _, _, ridx = plan_t.budget_radius(H_t)
    _, _, ridx_r = plan_r.budget_radius(H_r)
    assert torch.equal(ridx, ridx_r)
    mask, row_ptr, col_idx, nnz, pairs = plan_t.build_block_mask(ridx, want_tile_pairs=True)
    mask_r, row_ptr_r, col_idx_r, nnz_r, pairs_r = plan_r.build_block_mask(ridx, want_tile_pairs=True)
    assert torch.equal(mask, mask_r) and torch.equal(row_ptr, row_ptr_r) and torch.equal(pairs, pairs_r)
    # block-sparse, with and without tile pairs, with lse; token mask inside blocks; Eq. 16 without a list
    S_t, sl_t = plan_t.sparse_attn(Q, K, V, row_ptr, col_idx, tile_pairs=pairs, want_lse=True)
    S_r, sl_r = plan_r.sparse_attn(Qr, Kr, Vr, row_ptr, col_idx, tile_pairs=pairs, want_lse=True)
    assert torch.equal(S_r, plan_t.tile_major_scatter(S_t)) and torch.equal(sl_r, sl_t)
    S2_r, _ = plan_r.sparse_attn(Qr, Kr, Vr, row_ptr, col_idx)
    assert torch.equal(S2_r, S_r)
    if token_mask:
        for rp, ci in ((row_ptr, col_idx), (None, None)):
            M_t, _ = plan_t.sparse_attn(Q, K, V, rp, ci, ridx=ridx)
            M_r, _ = plan_r.sparse_attn(Qr, Kr, Vr, rp, ci, ridx=ridx)
            assert torch.equal(M_r, plan_t.tile_major_scatter(M_t))
    # only Q and O in raster order (TRA_ORDER_RASTER_QO): K and V tile-major
    plan_q = make_plan(cfg, n_text=n_text, flags=api().TRA_ORDER_RASTER_QO)
    O_q, H_q, lse_q = plan_q.entropy_attn(Qr, K, V, want_lse=True)
    assert torch.equal(O_q, O_r) and torch.equal(H_q, H_t) and torch.equal(lse_q, lse_t)
    S_q, sl_q = plan_q.sparse_attn(Qr, K, V, row_ptr, col_idx, tile_pairs=pairs, want_lse=True)
    assert torch.equal(S_q, S_r) and torch.equal(sl_q, sl_t)
    if token_mask:
        M_q, _ = plan_q.sparse_attn(Qr, K, V, row_ptr, col_idx, ridx=ridx)
        assert torch.equal(M_q, plan_t.tile_major_scatter(plan_t.sparse_attn(Q, K, V, row_ptr, col_idx, ridx=ridx)[0]))
    # the host pipelines of such plans: no gather and no scatter (7 kernels per group), or two gathers (9)
    host = [t.cpu().pin_memory() for t in (Qr, Kr, Vr)]
    for p_, n_launch in ((plan_r, 7), (plan_q, 9)):
        out = torch.zeros(S_r.shape, dtype=torch.bfloat16).pin_memory()
        pipe = api().HostPipeline(p_, cfg["heads"], group=1)
        assert pipe.run(host[0], host[1], host[2], out) == n_launch * cfg["heads"]
        torch.cuda.synchronize()
        assert torch.equal(out, S_r.cpu())
    for p_ in (plan_t, plan_r, plan_q):
        p_.check_status()
        p_.close()


def test_raster_order_needs_runs_of_sixteen():
    """W, the tile width and the block size must be multiples of 16 for a raster-order plan."""
    for kw in (dict(W=24, tile_w=8, block=128), dict(W=32, tile_w=16, block=72), dict(W=40, tile_w=16, block=128)):
        cfg = common.small_config(3, 8, kw["W"], heads=1, head_dim=128, block=kw["block"], tile_h=4, tile_w=kw["tile_w"])
        with pytest.raises(api().TraError) as err:
            make_plan(cfg, flags=api().TRA_ORDER_RASTER)
        assert err.value.code == api().TRA_ERR_UNSUPPORTED
        make_plan(cfg).close()


def test_largest_supported_sequence():
    """NB = 2048 key blocks (262,144 tokens) is the largest sequence the attention calls take; one
    more block is refused.  One head, sampled rows against the oracle."""
    cfg = common.small_config(32, 64, 128, heads=1, head_dim=128, block=128, tile_h=8, tile_w=16, seed=91,
                              s_lo=0.2, s_hi=5.0)
    geo = common.oracle_geometry(cfg)
    assert geo.NB == 2048
    plan = make_plan(cfg)
    Q, K, V = tile_major_inputs(cfg, plan)
    O, H, _ = plan.entropy_attn(Q, K, V)
    _, _, ridx = plan.budget_radius(H)
    mask, row_ptr, col_idx, nnz = plan.build_block_mask(ridx)
    Os, _ = plan.sparse_attn(Q, K, V, row_ptr, col_idx)
    plan.check_status()
    rng = np.random.default_rng(17)
    rows = np.unique(np.concatenate([[0, geo.N - 1, geo.N // 2], rng.integers(0, geo.N, 9)])).astype(np.int32)
    rows_t = torch.from_numpy(rows).long().to(DEV)
    Qb, Kb, Vb = (workloads.bf16_bits(x[0, 0]) for x in (Q, K, V))
    ref = oracle.attention_rows(Qb, Kb, Vb, common.scale_of(cfg), rows)
    common.assert_output(O[0, 0][rows_t], ref["O"], "dense at 262,144 tokens")
    Hn = H[0, 0].cpu().numpy()
    assert np.abs(Hn[rows] - ref["H_def"]).max() <= common.ENTROPY_ATOL
    bud_ref, fragile = oracle.budget(Hn[None], geo.tau, geo.N)
    ridx_ref = oracle.select_radius(bud_ref, geo.coord, geo.H, geo.W, geo.counts)[0]
    ridx_np = ridx[0, 0].cpu().numpy().view(np.uint16)
    assert np.array_equal(ridx_np[~fragile[0]], ridx_ref[~fragile[0]]) and fragile.sum() <= 1
    u_list = np.unique(rows // geo.block)
    ref_mask = oracle.block_vote(geo.coord, geo.T, geo.block, geo.theta, ridx_np, u_list=u_list)
    assert np.array_equal(mask[0, 0].cpu().numpy()[u_list], ref_mask)
    vis = oracle.visible_rows(geo.coord, geo.T, geo.block, geo.theta, ridx_np, rows,
                              ref_mask[np.searchsorted(u_list, rows // geo.block)], 0)
    refs = oracle.attention_rows(Qb, Kb, Vb, common.scale_of(cfg), rows, vis)
    common.assert_output(Os[0, 0][rows_t], refs["O"], "sparse at 262,144 tokens")
    plan.close()
    # one block more: the attention calls refuse, the integer stages still run
    big = make_plan(cfg, n_text=1)
    assert big.NB == 2049
    z = torch.zeros(1, 1, big.N, 128, dtype=torch.bfloat16, device=DEV)
    with pytest.raises(api().TraError) as e:
        big.entropy_attn(z, z, z)
    assert e.value.code == -2          # TRA_ERR_UNSUPPORTED
    big.close()


def test_attention_rejects_bad_arguments():
    a = api()
    plan = make_plan(CFG_TINY)
    Q = torch.zeros(1, 2, plan.N, 64, dtype=torch.bfloat16, device=DEV)
    with pytest.raises(ValueError):
        plan.entropy_attn(Q[:, :, :-1].contiguous(), Q, Q)          # wrong token count
    with pytest.raises(ValueError):
        plan.entropy_attn(Q.float(), Q, Q)                           # wrong dtype
    with pytest.raises(a.TraError):
        plan.entropy_attn(Q, Q, Q, sm_scale=0.0)                      # non-positive scale
    base = torch.zeros(Q.numel() + 8, dtype=torch.bfloat16, device=DEV)
    misaligned = base[8:].view(Q.shape)                              # 16-byte, not 128-byte aligned
    with pytest.raises(a.TraError):
        plan.entropy_attn(misaligned, Q, Q)
    plan.close()
