"""Pins for the fp64 oracle: values the paper and the mathematics fix, closed forms,
textbook/library special cases and brute force on tiny inputs.  None of these tests
touches the CUDA path."""
import math
import os

import numpy as np
import pytest
import scipy.special
import scipy.stats

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bf16(x):
    """Round fp32/fp64 array to bf16 (round-to-nearest-even) and return the uint16 bits."""
    a = np.asarray(x, np.float32).view(np.uint32).astype(np.uint64)
    r = ((a + 0x7FFF + ((a >> 16) & 1)) >> 16).astype(np.uint16)
    return r


def widen(bits):
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def rand_qkv(rng, N, d, qscale=1.0):
    Q = bf16(rng.standard_normal((N, d)) * qscale)
    K = bf16(rng.standard_normal((N, d)))
    V = bf16(rng.standard_normal((N, d)))
    return Q, K, V


# ----------------------------------------------------------------------------- entropy
def test_entropy_uniform_is_log_n():
    # Eq. 2: 0 <= H <= log N, with equality for the uniform row (all scores equal).
    N, d = 300, 8
    rng = np.random.default_rng(0)
    Q = np.zeros((N, d), np.uint16)
    _, K, V = rand_qkv(rng, N, d)
    r = oracle.attention_rows(Q, K, V, 1.0, np.arange(5))
    assert np.allclose(r["H_def"], math.log(N), atol=1e-12)
    assert np.allclose(r["H_lse"], math.log(N), atol=1e-12)
    assert np.allclose(r["O"], widen(V).mean(axis=0)[None, :], atol=1e-12)
    a2 = oracle.attention_rows_alg2(Q, K, V, 1.0, np.arange(5), tile=64)
    assert np.allclose(a2["H"], math.log(N), atol=1e-12)


def test_entropy_one_hot_is_zero():
    # one key 80 above the rest: H = 80 (N-1) e^-80 to first order, i.e. 0.
    N, d = 64, 4
    Q = bf16(np.tile([8.0, 0, 0, 0], (N, 1)))
    Kf = np.zeros((N, d))
    Kf[7, 0] = 10.0
    K = bf16(Kf)
    V = bf16(np.random.default_rng(1).standard_normal((N, d)))
    r = oracle.attention_rows(Q, K, V, 1.0, np.array([0, 3]))
    expected = 80.0 * (N - 1) * math.exp(-80.0)
    assert np.all(np.abs(r["H_def"]) < 1e-27) and np.all(np.abs(r["H_def"] - expected) < 1e-30)
    assert np.all(np.abs(r["H_lse"]) < 1e-12)     # this form cancels 80 - 80 in fp64
    assert np.allclose(r["O"], widen(V)[7][None, :], atol=1e-30)


def test_entropy_two_level_closed_form():
    # n1 keys at score a, the other N - n1 at 0: Z = n1 e^a + N - n1, H = ln Z - n1 a e^a / Z.
    N, d, n1, a = 200, 4, 13, 3.0
    Q = bf16(np.tile([1.0, 0, 0, 0], (2, 1)))
    Kf = np.zeros((N, d))
    Kf[:n1, 0] = a
    K = bf16(Kf)
    V = bf16(np.ones((N, d)))
    r = oracle.attention_rows(Q, K, V, 1.0, np.array([0, 1]))
    Z = n1 * math.exp(a) + N - n1
    H = math.log(Z) - n1 * a * math.exp(a) / Z
    assert np.allclose(r["H_def"], H, atol=1e-12)
    assert np.allclose(r["H_lse"], H, atol=1e-12)
    assert np.allclose(r["lse"], math.log(Z), atol=1e-12)


@pytest.mark.parametrize("tile", [1, 7, 64, 1000])
def test_entropy_three_forms_agree_and_match_scipy(tile):
    # Eq. 2, its rewrite (Appendix, fused entropy) and Algorithm 2 are the same number;
    # scipy's softmax/entropy/logsumexp are the library routines they reduce to.
    N, d = 333, 16
    rng = np.random.default_rng(2)
    Q, K, V = rand_qkv(rng, N, d, qscale=3.0)
    rows = np.array([0, 1, 100, 332])
    scale = 1.0 / math.sqrt(d)
    r = oracle.attention_rows(Q, K, V, scale, rows)
    a2 = oracle.attention_rows_alg2(Q, K, V, scale, rows, tile)
    S = (widen(Q)[rows] @ widen(K).T) * scale
    P = scipy.special.softmax(S, axis=1)
    assert np.allclose(r["O"], P @ widen(V), atol=1e-12)
    assert np.allclose(a2["O"], P @ widen(V), atol=1e-12)
    H = scipy.stats.entropy(P, axis=1)
    assert np.allclose(r["H_def"], H, atol=1e-10)
    assert np.allclose(r["H_lse"], H, atol=1e-10)
    assert np.allclose(a2["H"], H, atol=1e-10)
    assert np.allclose(r["lse"], scipy.special.logsumexp(S, axis=1), atol=1e-12)
    assert np.all(r["H_def"] >= 0) and np.all(r["H_def"] <= math.log(N) + 1e-12)


def test_attention_transposed_operand_would_fail():
    # a query/key swap or a V indexed by query must not pass: asymmetric hand-made case.
    Q = bf16([[1.0, 0.0], [0.0, 2.0]])
    K = bf16([[3.0, 0.0], [0.0, 1.0]])
    V = bf16([[1.0, 0.0], [0.0, 1.0]])
    r = oracle.attention_rows(Q, K, V, 1.0, np.array([0, 1]))
    p0 = math.exp(3.0) / (math.exp(3.0) + 1.0)          # row 0: scores (3, 0)
    p1 = 1.0 / (1.0 + math.exp(2.0))                    # row 1: scores (0, 2)
    assert np.allclose(r["O"], [[p0, 1 - p0], [p1, 1 - p1]], atol=1e-14)


# ----------------------------------------------------------------------------- budget
def test_budget_closed_forms_and_monotone():
    N, tau = 32760, 0.9
    H = np.array([0.0, math.log(N), 1.0, 5.0], np.float32)
    b, frag = oracle.budget(H, tau, N)
    assert b[0] == 1                                           # H = 0 -> ceil(tau) = 1
    assert b[1] == math.ceil(tau * math.exp(float(H[1])))      # H = ln N -> ceil(tau N) up to fp32 of ln N
    assert abs(int(b[1]) - math.ceil(tau * N)) <= 2
    hs = np.linspace(0, math.log(N), 5000).astype(np.float32)
    bs, _ = oracle.budget(hs, tau, N)
    assert np.all(np.diff(bs) >= 0)                            # monotone in entropy (Section 3.1)
    e = np.exp(hs.astype(np.float64))
    inner = bs < N
    assert np.all((bs[inner] - 1) / tau < e[inner] + 1e-9) and np.all(e[inner] <= bs[inner] / tau + 1e-9)
    big, _ = oracle.budget(np.array([30.0], np.float32), tau, N)
    assert big[0] == N                                         # clamp
    _, fr = oracle.budget(np.array([0.0], np.float32), 1.0, N)  # tau e^0 = 1 exactly: fragile
    assert fr[0]


def test_budget_lognormal_closed_forms():
    # Appendix, entropy-identified Lognormal mapping: sigma = sqrt(2 (ln N - H)),
    # B = Phibar(sigma - Phi^-1(tau)); scipy's norm.sf / norm.ppf are the library routines.
    import scipy.stats
    N, tau = 75600, 0.9
    H = np.array([math.log(N), 0.0, 5.0, 9.0, 10.5, 11.0], np.float32)
    b, _ = oracle.budget_lognormal(H, tau, N)
    # sigma = 0 at H = ln N: B = Phibar(-z_tau) = tau (the uniform map's value there)
    # (fp32 ln N is a hair below ln N and dB/dsigma is steep at 0, hence the small slack)
    assert abs(int(b[0]) - math.ceil(tau * N)) <= 20
    assert 1 <= b[1] < 100                                     # a sharp row keeps a handful of keys
    sig = np.sqrt(2 * np.maximum(0.0, math.log(N) - H.astype(np.float64)))
    ref = np.ceil(N * scipy.stats.norm.sf(sig - scipy.stats.norm.ppf(tau)))
    assert np.array_equal(b, np.clip(ref, 1, N).astype(np.int32))
    # the defining property: the largest B*N of N lognormal weights hold mass tau
    for s_, B in zip(sig[2:5], (N * scipy.stats.norm.sf(sig - scipy.stats.norm.ppf(tau)))[2:5] / N):
        assert abs(scipy.stats.norm.sf(scipy.stats.norm.ppf(1 - B) - s_) - tau) < 1e-9
    hs = np.linspace(0, math.log(N), 3000).astype(np.float32)
    bs, _ = oracle.budget_lognormal(hs, tau, N)
    assert np.all(np.diff(bs) >= 0)                            # monotone in entropy
    # Table of the appendix: the lognormal map over-estimates relative to the uniform one at
    # mid entropies (mean error +0.0164 vs -0.0415) -- its budgets are the larger ones there
    bu, _ = oracle.budget(hs, tau, N)
    mid = (hs > 0.5 * math.log(N)) & (hs < 0.95 * math.log(N))
    assert np.all(bs[mid] >= bu[mid])


# ----------------------------------------------------------------------------- grid count
def gauss_circle():
    with open(os.path.join(GOLDEN, "gauss_circle.txt")) as f:
        line = [l for l in f if not l.startswith("#")][0]
    return [int(v) for v in line.split()]


def test_grid_count_gauss_circle_gamma0():
    # gamma = 0, interior query of a frame larger than the disk: every frame holds the
    # Gauss-circle number of lattice points, so C_grid(r) = T * G(r).
    G = gauss_circle()
    T, H, W = 3, 41, 41
    radii = np.arange(0, 21, dtype=np.float64)
    th = oracle.theta_table(radii, T, H, W, 0.0)
    assert np.array_equal(th[:, 0], (radii ** 2).astype(np.int32))
    for r in range(21):
        assert oracle.grid_count_brute(T, H, W, th[r], 1, 20, 20) == T * G[r]
    counts = oracle.grid_count_table(T, H, W, th)
    assert np.array_equal(counts[1, 20, 20], T * np.array(G))


def test_grid_count_float_sqrt_form_and_table():
    # Eq. 13 in the paper's literal floating form (sqrt distance vs r*exp(-gamma*delta)),
    # evaluated by numpy over all keys, against the oracle's integer form; non-integer
    # thresholds keep the comparison away from ties.
    T, H, W, gamma = 5, 9, 11, 0.6
    radii = oracle.default_radii(T, H, W, gamma)
    th = oracle.theta_table(radii, T, H, W, gamma)
    counts = oracle.grid_count_table(T, H, W, th)
    tt, yy, xx = np.meshgrid(np.arange(T), np.arange(H), np.arange(W), indexing="ij")
    rng = np.random.default_rng(3)
    for _ in range(40):
        f, y, x = rng.integers(T), rng.integers(H), rng.integers(W)
        k = rng.integers(radii.size)
        ds = np.sqrt((yy - y) ** 2 + (xx - x) ** 2)
        rho = radii[k] * np.exp(-gamma * np.abs(tt - f))
        near_tie = np.abs(ds - rho) < 1e-9
        near_tie &= ~((np.abs(tt - f) == 0) & (ds <= rho))    # delta=0 integer radii: exact ties are 'inside'
        assert not near_tie.any()
        ref = int((ds <= rho).sum())
        assert oracle.grid_count_brute(T, H, W, th[k], f, y, x) == ref
        assert counts[f, y, x, k] == ref
    # whole table against the enumeration, every entry
    for f in range(T):
        for y in range(H):
            for x in range(W):
                for k in range(0, radii.size, 3):
                    assert counts[f, y, x, k] == oracle.grid_count_brute(T, H, W, th[k], f, y, x)


@pytest.mark.parametrize("T,H,W", [(21, 45, 80), (33, 45, 80)])
@pytest.mark.parametrize("gamma", [0.6, 0.95, 0.0513])
def test_grid_count_float_sqrt_form_on_the_full_size_grids(T, H, W, gamma):
    # Eq. 13 in its literal floating form (Euclidean distance against r exp(-gamma delta)), evaluated
    # by numpy over every key of the real latent grids, for a centre and a corner query, against the
    # oracle's integer-threshold enumeration.  Candidates whose decayed radius comes within 1e-9 of a
    # lattice distance are skipped (the two forms may round a tie differently); few are.  A key at the
    # query's own (y, x) is inside for every radius >= 0 in both forms.
    radii = oracle.default_radii(T, H, W, gamma)
    th = oracle.theta_table(radii, T, H, W, gamma)
    tt, yy, xx = np.meshgrid(np.arange(T), np.arange(H), np.arange(W), indexing="ij")
    diag = math.hypot(H - 1, W - 1)
    checked = 0
    for f, y, x in ((T // 2, H // 2, W // 2), (0, 0, 0), (T - 1, H - 1, 0)):
        ds = np.sqrt((yy - y) ** 2 + (xx - x) ** 2)
        dt = np.abs(tt - f)
        for k in list(range(0, radii.size, 7)) + [radii.size - 1]:
            rho = np.minimum(radii[k] * np.exp(-gamma * dt), diag)      # the frame diagonal is full support
            near_tie = (np.abs(ds - rho) < 1e-9) & ~((dt == 0) & (ds <= rho)) & (rho < diag) & (ds > 0)
            if near_tie.any():
                continue
            assert oracle.grid_count_brute(T, H, W, th[k], f, y, x) == int((ds <= rho).sum()), (f, y, x, k)
            checked += 1
    assert checked >= 30
    # r = 0 keeps the query's own cell in every frame; the last candidate is full support
    assert oracle.grid_count_brute(T, H, W, th[0], T // 2, H // 2, W // 2) == T
    assert oracle.grid_count_brute(T, H, W, th[-1], 0, 0, 0) == T * H * W


def test_grid_count_limits_monotone_and_continuous_estimate():
    T, H, W, gamma = 21, 45, 80, 0.6
    radii = oracle.default_radii(T, H, W, gamma)
    th = oracle.theta_table(radii, T, H, W, gamma)
    N = T * H * W
    f, y, x = 10, 22, 40
    c = np.array([oracle.grid_count_brute(T, H, W, th[k], f, y, x) for k in range(radii.size)])
    assert c[0] == T                       # r = 0 keeps the same (y, x) in every frame (<= is inclusive)
    assert c[-1] == N                      # last candidate is the full-support radius
    assert np.all(np.diff(c) >= 0)
    # Eq. 11: C_cont(r) = sum_t pi r^2 phi^2; close to the lattice count for an interior query
    for r in (10, 20):
        cont = sum(math.pi * r * r * math.exp(-2 * gamma * abs(t - f)) for t in range(T))
        assert abs(c[r] - cont) / cont < 0.05
    # corner queries see fewer keys than interior ones at the same radius (boundary awareness)
    assert oracle.grid_count_brute(T, H, W, th[30], 0, 0, 0) < c[30]
    # literal policy: the infinite radius is the full support as well
    lit = oracle.default_radii(T, H, W, gamma, policy=1)
    thl = oracle.theta_table(lit, T, H, W, gamma)
    assert np.isinf(lit[-1]) and oracle.grid_count_brute(T, H, W, thl[-1], 0, 0, 0) == N
    assert np.array_equal(thl[:-1], th[: lit.size - 1])


def test_theta_monotone_in_radius_and_delta():
    T, H, W, gamma = 33, 45, 80, 0.95
    radii = oracle.default_radii(T, H, W, gamma)
    th = oracle.theta_table(radii, T, H, W, gamma)
    assert np.all(np.diff(radii) > 0)
    assert np.all(np.diff(th, axis=0) >= 0) and np.all(np.diff(th, axis=1) <= 0)
    assert th.max() == (H - 1) ** 2 + (W - 1) ** 2 and np.all(th[-1] == th.max())


def test_full_support_radius_covers_frames_with_an_integer_diagonal():
    """The last candidate of the extended set is the full-support radius: at every frame distance its threshold is
    the squared frame diagonal, also when the diagonal is an integer (3-4-5, 5-12-13, 8-15-17 grids), where the
    rounded product D^2 e^{2 gamma (T-1)} e^{-2 gamma (T-1)} can come out a hair below D^2.  On other grids the
    extended candidates are D e^{gamma m} to the last bit."""
    for H, W in ((4, 5), (13, 6), (9, 16), (16, 9), (21, 21)):
        for T in (2, 4, 21, 33):
            for gamma in (0.0513, 0.3, 0.6, 0.95, 2.0):
                radii = oracle.default_radii(T, H, W, gamma)
                th = oracle.theta_table(radii, T, H, W, gamma)
                diag2 = (H - 1) ** 2 + (W - 1) ** 2
                assert np.all(np.diff(radii) > 0)
                assert np.all(th[-1] == diag2), (H, W, T, gamma)
                assert oracle.grid_count_brute(T, H, W, th[-1], 0, 0, 0) == T * H * W
                D = math.ceil(math.sqrt(diag2))
                want = D * math.exp(gamma * (T - 1))
                assert radii[-1] == want or 0 < radii[-1] - want <= 4 * np.spacing(want)
    T, H, W, gamma = 21, 45, 80, 0.6
    radii = oracle.default_radii(T, H, W, gamma)
    D = math.ceil(math.sqrt(44 ** 2 + 79 ** 2))
    assert np.array_equal(radii[D + 1:], [D * math.exp(gamma * m) for m in range(1, T)])


# ----------------------------------------------------------------------------- radius
def test_radius_selection_minimal_and_sufficient():
    g = oracle.geometry(4, 8, 8, 4, 4, 64, 0.6, 0.9)
    rng = np.random.default_rng(4)
    heads = 3
    H = rng.uniform(0, math.log(g.N), (heads, g.N)).astype(np.float32)
    K, _ = oracle.budget(H, g.tau, g.N)
    ridx = oracle.select_radius(K, g.coord, g.H, g.W, g.counts)
    for h in range(heads):
        for p in range(g.N):
            t, y, x = g.coord[p]
            k = ridx[h, p]
            assert g.counts[t, y, x, k] >= K[h, p]                 # spec: support meets the budget
            assert k == 0 or g.counts[t, y, x, k - 1] < K[h, p]    # and is the smallest such (Eq. 14)
            # row sum of the token mask equals C_grid(r_i)
            if p % 37 == 0:
                assert oracle.token_mask_row(g.coord, g.T, g.theta, p, k).sum() == g.counts[t, y, x, k]
    small = np.full((1, g.N), g.T, np.int32)
    assert np.all(oracle.select_radius(small, g.coord, g.H, g.W, g.counts) == 0)   # K <= T -> r = 0
    full = np.full((1, g.N), g.N, np.int32)
    r_full = oracle.select_radius(full, g.coord, g.H, g.W, g.counts)
    for p in range(g.N):
        t, y, x = g.coord[p]
        assert g.counts[t, y, x, r_full[0, p]] == g.N


def test_radius_tracks_analytic_initialisation():
    # Eq. 12: r~ = sqrt(K / (pi sum_t phi^2)); for an interior query the selected lattice
    # radius stays within one cell plus a few percent of it.
    T, H, W, gamma = 9, 45, 80, 0.6
    g = oracle.geometry(T, H, W, 8, 16, 128, gamma, 0.9)
    p = int(np.nonzero((g.coord == [4, 22, 40]).all(axis=1))[0][0])
    for K in (50, 200, 800, 2000):
        bud = np.ones((1, g.N), np.int32)
        bud[0, p] = K
        k = oracle.select_radius(bud, g.coord, H, W, g.counts)[0, p]
        denom = math.pi * sum(math.exp(-2 * gamma * abs(t - 4)) for t in range(T))
        r_tilde = math.sqrt(K / denom)
        assert abs(g.radii[k] - r_tilde) <= 1.0 + 0.1 * r_tilde


# ----------------------------------------------------------------------------- tile-major order
def test_tile_major_is_a_permutation_with_contiguous_tiles():
    T, H, W, th, tw = 2, 10, 7, 4, 3
    coord = oracle.tile_major(T, H, W, th, tw)
    raster = (coord[:, 0] * H + coord[:, 1]) * W + coord[:, 2]
    assert np.array_equal(np.sort(raster), np.arange(T * H * W))
    # walking the order, the (frame, tile-row, tile-col) key never decreases and each
    # tile's tokens are consecutive and row-major inside the tile
    key = (coord[:, 0] * 100 + coord[:, 1] // th) * 100 + coord[:, 2] // tw
    assert np.all(np.diff(key) >= 0)
    for kv in np.unique(key):
        idx = np.nonzero(key == kv)[0]
        assert np.array_equal(idx, np.arange(idx[0], idx[0] + idx.size))
        inner = coord[idx, 1] * W + coord[idx, 2]
        assert np.all(np.diff(inner) > 0)
    # exact tiling: tile k of frame 0 holds positions [k*th*tw, (k+1)*th*tw)
    c2 = oracle.tile_major(1, 8, 8, 4, 4)
    assert np.array_equal(c2[16:32, 1:], [[y, x] for y in range(4) for x in range(4, 8)])


# ----------------------------------------------------------------------------- token mask
def numpy_token_mask(g, ridx_head):
    """Eq. 15 in floating form for every (query, key) pair of one head."""
    c = g.coord.astype(np.float64)
    ds = np.sqrt((c[:, None, 1] - c[None, :, 1]) ** 2 + (c[:, None, 2] - c[None, :, 2]) ** 2)
    dt = np.abs(c[:, None, 0] - c[None, :, 0])
    rho = g.radii[ridx_head][:, None] * np.exp(-g.gamma * dt)
    return ds <= rho + 1e-12 * (dt == 0)      # delta = 0: integer radius, exact tie counts as inside


def test_token_mask_matches_float_form_and_is_nested():
    g = oracle.geometry(4, 8, 8, 4, 4, 64, 0.6, 0.9)
    rng = np.random.default_rng(5)
    ridx = rng.integers(0, g.radii.size, g.N).astype(np.uint16)
    M = numpy_token_mask(g, ridx)
    for p in range(0, g.N, 5):
        assert np.array_equal(oracle.token_mask_row(g.coord, g.T, g.theta, p, ridx[p]), M[p])
    for p in (0, 77, 255):
        prev = np.zeros(g.N, bool)
        for k in range(g.radii.size):
            row = oracle.token_mask_row(g.coord, g.T, g.theta, p, k)
            assert np.all(row[prev])          # nested disks (Section 3.2)
            assert row[p]                     # M_ii = 1
            prev = row
        assert prev.all()                     # full-support radius sees every key


# ----------------------------------------------------------------------------- block vote
def numpy_block_vote(M, b):
    N = M.shape[0]
    NB = (N + b - 1) // b
    out = np.zeros((NB, NB), np.uint8)
    for u in range(NB):
        for v in range(NB):
            c = M[u * b:(u + 1) * b, v * b:(v + 1) * b].sum(axis=0)
            nonempty, high = int((c > 0).sum()), int((c > b / 3).sum())
            out[u, v] = nonempty > 0 and 10 * high > 6 * nonempty
    return out


@pytest.mark.parametrize("shape", [(4, 8, 8, 4, 4, 64), (3, 7, 10, 4, 4, 32), (2, 5, 9, 2, 3, 48)])
def test_block_vote_matches_numpy_brute_force(shape):
    T, H, W, th, tw, b = shape
    g = oracle.geometry(T, H, W, th, tw, b, 0.6, 0.9)
    rng = np.random.default_rng(6)
    ridx = rng.integers(0, g.radii.size * 2 // 3, g.N).astype(np.uint16)
    ref = numpy_block_vote(numpy_token_mask(g, ridx), b)
    got = oracle.block_vote(g.coord, T, b, g.theta, ridx)
    assert np.array_equal(got, ref)
    assert 0 < ref.mean() < 1
    kd = oracle.block_vote(g.coord, T, b, g.theta, ridx, keep_diagonal=True)
    assert np.array_equal(kd, np.maximum(ref, np.eye(g.NB, dtype=np.uint8)))
    full = np.full(g.N, g.radii.size - 1, np.uint16)
    assert oracle.block_vote(g.coord, T, b, g.theta, full).all()      # all-ones token mask keeps everything


def test_block_vote_threshold_is_strict():
    # one frame, one row of 10 tokens, blocks of 5 (Algorithm 1 with b = 5: high means c > 5/3).
    T, H, W, b = 1, 1, 10, 5
    coord = oracle.tile_major(T, H, W, 1, 5)
    radii = np.arange(0, 12, dtype=np.float64)
    th = oracle.theta_table(radii, T, H, W, 0.0)

    def vote(r):
        return oracle.block_vote(coord, T, b, th, np.array(r + [0] * 5, np.uint16))[0, 1]

    # query x=4 (r=5) reaches keys 5..9 once; query x=3 (r=4) reaches 5,6,7: c = 2,2,2,1,1
    assert vote([0, 0, 0, 4, 5]) == 0        # |C|=5, |C_hi|=3: 30 > 30 is false -> dropped
    assert vote([0, 0, 0, 5, 5]) == 1        # c = 2,2,2,2,1: |C_hi|=4 -> kept
    assert vote([0, 0, 0, 0, 0]) == 0        # nothing reaches block 1: |C| = 0
    # b = 6: c = 2 is exactly b/3, not high; c = 3 is
    T, H, W, b = 1, 1, 12, 6
    coord = oracle.tile_major(T, H, W, 1, 6)
    th = oracle.theta_table(np.arange(0, 14, dtype=np.float64), T, H, W, 0.0)
    two = np.array([0, 0, 0, 0, 6, 6] + [0] * 6, np.uint16)      # x=4 reaches ..10, x=5 reaches ..11
    assert oracle.block_vote(coord, T, b, th, two)[0, 1] == 0   # c = 2,2,2,2,2,1 -> no high column
    three = np.array([0, 0, 0, 8, 7, 6] + [0] * 6, np.uint16)    # all three reach ..11: c = 3 everywhere
    assert oracle.block_vote(coord, T, b, th, three)[0, 1] == 1


def test_csr_is_ascending():
    m = np.array([[[1, 0, 1], [0, 0, 0], [1, 1, 1]]], np.uint8)
    rp, ci = oracle.csr_from_block_mask(m)
    assert rp.tolist() == [0, 2, 2, 5] and ci.tolist() == [0, 2, 0, 1, 2]


# ----------------------------------------------------------------------------- sparse attention
def test_sparse_attention_modes_against_bias_matrix():
    # Eq. 16: softmax(QK^T/sqrt(d) + B(M)) V with B = 0 / -inf, written with numpy/scipy.
    g = oracle.geometry(4, 8, 8, 4, 4, 64, 0.6, 0.9)
    d = 16
    rng = np.random.default_rng(7)
    Q, K, V = rand_qkv(rng, g.N, d, qscale=2.0)
    ridx = rng.integers(0, 6, g.N).astype(np.uint16)
    scale = 1 / math.sqrt(d)
    rows = np.arange(g.N)
    M = numpy_token_mask(g, ridx)
    blk = oracle.block_vote(g.coord, g.T, g.block, g.theta, ridx)
    S = (widen(Q) @ widen(K).T) * scale
    for mode in (0, 1, 2):
        block_rows = blk[rows // g.block]
        vis = oracle.visible_rows(g.coord, g.T, g.block, g.theta, ridx, rows, block_rows, mode)
        blk_tok = np.repeat(np.repeat(blk, g.block, 0), g.block, 1).astype(bool)
        ref_vis = {0: blk_tok, 1: blk_tok & M, 2: M}[mode]
        assert np.array_equal(vis.astype(bool), ref_vis)
        out = oracle.attention_rows(Q, K, V, scale, rows, vis)
        bias = np.where(ref_vis, 0.0, -np.inf)
        nonempty = ref_vis.any(axis=1)
        P = scipy.special.softmax(S[nonempty] + bias[nonempty], axis=1)
        assert np.allclose(out["O"][nonempty], P @ widen(V), atol=1e-12)
        assert np.all(out["O"][~nonempty] == 0)                       # empty row -> zero output
    # full radius: mode 2 reproduces dense attention (spec invariant)
    full = np.full(g.N, g.radii.size - 1, np.uint16)
    vis = oracle.visible_rows(g.coord, g.T, g.block, g.theta, full, rows, None, 2)
    assert vis.all()
    dense = oracle.attention_rows(Q, K, V, scale, rows)
    assert np.allclose(oracle.attention_rows(Q, K, V, scale, rows, vis)["O"], dense["O"], atol=0)
    # one retained block: softmax over that block alone
    one = np.zeros((g.N, g.NB), np.uint8)
    one[:, 2] = 1
    vis = oracle.visible_rows(g.coord, g.T, g.block, g.theta, ridx, rows, one, 0)
    sl = slice(2 * g.block, 3 * g.block)
    P = scipy.special.softmax(S[:, sl], axis=1)
    assert np.allclose(oracle.attention_rows(Q, K, V, scale, rows, vis)["O"], P @ widen(V)[sl], atol=1e-12)
    # nothing retained
    none = np.zeros((4, g.NB), np.uint8)
    vis = oracle.visible_rows(g.coord, g.T, g.block, g.theta, ridx, np.arange(4), none, 0)
    r = oracle.attention_rows(Q, K, V, scale, np.arange(4), vis)
    assert np.all(r["O"] == 0) and np.all(np.isneginf(r["lse"]))


def test_ragged_last_block_rows_and_columns_do_not_exist():
    # N = 3*7*10 = 210, b = 32: last block has 18 valid tokens; votes count valid columns only.
    g = oracle.geometry(3, 7, 10, 4, 4, 32, 0.6, 0.9)
    assert g.NB == 7 and g.N - 6 * 32 == 18
    full = np.full(g.N, g.radii.size - 1, np.uint16)
    assert oracle.block_vote(g.coord, g.T, 32, g.theta, full).all()
    # only 10 valid queries with a disk in the last block: c <= 10 < 32/3 -> never high
    ridx = np.zeros(g.N, np.uint16)
    out = oracle.block_vote(g.coord, g.T, 32, g.theta, ridx, u_list=[6])
    assert out.shape == (1, 7)
    M = numpy_token_mask(g, ridx)
    assert np.array_equal(out[0], numpy_block_vote(M, 32)[6])


def test_text_tokens_keep_their_blocks_dense():
    # Section 3.2 (last paragraph) and Algorithm 1: blocks with u >= B_v or v >= B_v are kept, B_v
    # counting the blocks made of video tokens only; the token mask covers the video-key submatrix.
    g = oracle.geometry(3, 7, 10, 4, 4, 32, 0.6, 0.9)          # N = 210: B_v = 6, block 6 holds both kinds
    n_text, b = 50, 32
    S = g.N + n_text
    NB = (S + b - 1) // b
    assert NB == 9
    rng = np.random.default_rng(8)
    ridx = rng.integers(0, 8, S).astype(np.uint16)
    with_text = oracle.block_vote(g.coord, g.T, b, g.theta, ridx, u_list=np.arange(NB), n_text=n_text)
    video_only = oracle.block_vote(g.coord, g.T, b, g.theta, ridx[: g.N])
    assert with_text.shape == (NB, NB)
    assert np.array_equal(with_text[:6, :6], video_only[:6, :6])   # pure video blocks: the video-only vote
    assert with_text[6:, :].all() and with_text[:, 6:].all()   # rows and columns that hold a text token are dense
    assert not video_only[:, 6].all()                          # the vote alone would have dropped that block somewhere
    assert 0 < video_only.mean() < 1
    rows = np.array([0, 100, 209, 210, 259])
    M = numpy_token_mask(g, ridx[: g.N])
    for mode in (0, 1, 2):
        vis = oracle.visible_rows(g.coord, g.T, b, g.theta, ridx, rows, with_text[rows // b], mode,
                                  n_text=n_text).astype(bool)
        assert vis.shape == (rows.size, S)
        blk = np.repeat(with_text[rows // b], b, axis=1)[:, :S].astype(bool)
        tok = np.ones((rows.size, S), bool)
        tok[:3, : g.N] = M[rows[:3]]                            # video queries: disks on video keys only
        ref = {0: blk, 1: blk & tok, 2: tok}[mode]
        assert np.array_equal(vis, ref)
        assert vis[3:].all()                                     # text queries see every key
        assert vis[:, g.N:].all()                                # every text key is visible to every query


# ----------------------------------------------------------------------------- schedule
def test_schedule_warmup_rule():
    with open(os.path.join(GOLDEN, "paper_schedule.txt")) as f:
        n_steps, n_warm = [int(v) for v in [l for l in f if not l.startswith("#")][0].split()]
    kinds, nw = oracle.schedule(n_steps)
    assert nw == n_warm and kinds.count("dense") == n_warm
    kinds, nw = oracle.schedule(50)
    assert nw == 12 and kinds[:12] == ["dense"] * 12 and kinds[12:] == ["sparse"] * 38
