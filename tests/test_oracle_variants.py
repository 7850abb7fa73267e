"""Pins of the oracle's walk/pair variants and of its Adam update (CPU only).

Window shrinking, sub-sampling of frequent nodes and the start-node shuffle each draw their
own random words, so each is pinned by what its definition fixes: value ranges and
distributions, exact special cases, invariants that a slip (off-by-one window, inverted
comparison, a round function that is not undone) breaks.  Adam is pinned against torch's
optimizers.
"""
import numpy as np
import pytest
import torch
from scipy import stats

from oracle import gs_oracle as O
from paper_2407_15452_b200 import workloads as WL

CHI2_P = 1e-4


def np_graph(g):
    return g.offsets.cpu().numpy().astype(np.int64), g.cols.cpu().numpy()


def chi2_uniform_ok(counts):
    counts = np.asarray(counts, dtype=np.float64)
    exp = counts.sum() / len(counts)
    stat = ((counts - exp) ** 2 / exp).sum()
    return stat < stats.chi2.ppf(1 - CHI2_P, len(counts) - 1)


def tiny_setup(n=300, L=30, n_walks=600, seed=5):
    g = WL.chung_lu_graph(n, 8, 2.3, seed=21)
    off, col = np_graph(g)
    thr, alias = O.build_alias((off[1:] - off[:-1]).astype(np.float64), 0.75)
    walks, _ = O.uniform_walks(off, col, None, n_walks, 40, L, seed)
    return off, col, thr, alias, walks


# ---------------------------------------------------------------- window shrinking
@pytest.mark.parametrize("w", [1, 3, 5, 8])
def test_shrunk_windows_are_symmetric_uniform_on_1_to_w_and_keep_the_negatives(w):
    off, col, thr, alias, walks = tiny_setup()
    n_walks, L = walks.shape
    K, S = 3, 2 * w
    c0, o0, n0, p0 = O.expand_lists(walks, 40, w, K, thr, alias, 9)
    c1, o1, n1, p1 = O.expand_lists(walks, 40, w, K, thr, alias, 9, shrink=True)
    full = c0.reshape(n_walks, L, S) >= 0
    kept = c1.reshape(n_walks, L, S) >= 0
    assert not (kept & ~full).any()                       # nothing new appears
    # a kept pair is the pair of the full window, negatives included
    m = c1 >= 0
    assert np.array_equal(c1[m], c0[m]) and np.array_equal(o1[m], o0[m])
    assert np.array_equal(n1[m], n0[m]) and (n1[~m] == -1).all()
    assert p1 == int(m.sum()) and (p1 < p0 or w == 1)
    # distance of slot sigma from the center: w - sigma for sigma < w, sigma - w + 1 otherwise
    dist = np.array([w - s if s < w else s - w + 1 for s in range(S)])
    counts = np.zeros(w + 1, dtype=np.int64)
    for a in range(n_walks):
        for i in range(L):
            if not full[a, i].any():
                continue
            present = full[a, i]
            # the window the position used: every available slot within it is kept, none beyond
            ks = kept[a, i]
            if not ks.any():
                # only possible when the available slots are all farther than the drawn window
                assert dist[present].min() > 1
                continue
            b = dist[ks].max()
            assert 1 <= b <= w
            assert np.array_equal(ks, present & (dist <= b))       # symmetric, contiguous
            # with the full window available the drawn width is exactly b
            if present.all():
                counts[b] += 1
    assert counts[0] == 0
    if w > 1:
        assert counts[1:].min() > 50 and chi2_uniform_ok(counts[1:])   # uniform on 1..w


def test_shrunk_window_mean_pair_count_is_w_plus_one():
    # interior positions of full walks: 2 * E[w_i] = w + 1 pairs on average
    w, L = 6, 40
    walks = np.tile(np.arange(L, dtype=np.int32), (4000, 1))
    thr, alias = O.build_alias(np.ones(L), 0.75)
    c, _, _, _ = O.expand_lists(walks, 0, w, 1, thr, alias, 2, shrink=True)
    per_pos = (c.reshape(4000, L, 2 * w) >= 0).sum(axis=2)[:, w:L - w]
    mean = per_pos.mean()
    sd = np.sqrt(4 * (w * w - 1) / 12.0 / per_pos.size)            # 2 * uniform{1..w}
    assert abs(mean - (w + 1)) < 5 * sd


# ---------------------------------------------------------------- sub-sampling
def test_keep_thresholds_exact_special_cases():
    # relative frequencies 1/2, 1/4, 1/8, 1/8 and t = 1/32: sqrt(t/f) = 1/4, sqrt(1/8), 1/2, 1/2
    wgt = np.array([4.0, 2.0, 1.0, 1.0])
    thr = O.keep_thresholds(wgt, 1.0 / 32)
    assert thr[0] == 2 ** 30 and thr[2] == 2 ** 31 and thr[3] == 2 ** 31
    assert abs(int(thr[1]) - 2 ** 32 / np.sqrt(8.0)) <= 1
    # f <= t: always kept
    assert (O.keep_thresholds(wgt, 0.5) == 0xFFFFFFFF).all()
    # zero weight never occurs in a walk; it is marked "always"
    assert O.keep_thresholds(np.array([0.0, 1.0]), 0.1)[0] == 0xFFFFFFFF
    with pytest.raises(ValueError):
        O.keep_thresholds(np.zeros(3), 0.1)


def test_subsampled_walks_are_ordered_subsequences_with_the_stated_retention():
    off, col, thr_a, alias, walks = tiny_setup(n=200, L=40, n_walks=3000)
    n = len(off) - 1
    deg = (off[1:] - off[:-1]).astype(np.float64)
    t = 1.0 / (4 * n)                                            # most nodes are above t
    keep_thr = O.keep_thresholds(deg, t)
    out, kept = O.subsample_walks(walks, 40, keep_thr, 13)
    assert kept == int((out >= 0).sum())
    seen = np.zeros(n)
    stay = np.zeros(n)
    for W, Z in zip(walks, out):
        z = Z[Z >= 0]
        assert (Z[len(z):] == -1).all()                           # -1 only as a suffix
        # z is a subsequence of W: greedy match
        k = 0
        for v in W[W >= 0]:
            if k < len(z) and z[k] == v:
                k += 1
        assert k == len(z)
        np.add.at(seen, W[W >= 0], 1)
        np.add.at(stay, z, 1)
    f = deg / deg.sum()
    p_keep = np.minimum(1.0, np.sqrt(t / np.maximum(f, 1e-300)))
    for v in np.argsort(-seen)[:40]:                              # the most visited nodes
        sd = np.sqrt(seen[v] * p_keep[v] * (1 - p_keep[v])) + 1e-9
        assert abs(stay[v] - seen[v] * p_keep[v]) < 5 * sd + 1, (v, stay[v], seen[v], p_keep[v])
    # with every threshold at "always" the walks come back unchanged
    same, kept_all = O.subsample_walks(walks, 40, np.full(n, 0xFFFFFFFF, dtype=np.uint32), 13)
    assert np.array_equal(same, walks) and kept_all == int((walks >= 0).sum())
    # a threshold of zero drops every occurrence of that node
    z = np.full(n, 0xFFFFFFFF, dtype=np.uint32)
    hub = int(np.argmax(seen))
    z[hub] = 0
    dropped, _ = O.subsample_walks(walks, 40, z, 13)
    assert not (dropped == hub).any()
    assert (dropped >= 0).sum() == (walks >= 0).sum() - seen[hub]


def test_subsampling_decisions_depend_on_walk_id_and_position_only():
    off, col, thr_a, alias, walks = tiny_setup(n=200, L=20, n_walks=64)
    keep_thr = O.keep_thresholds((off[1:] - off[:-1]).astype(np.float64), 1e-3)
    whole, _ = O.subsample_walks(walks, 40, keep_thr, 13)
    part, _ = O.subsample_walks(walks[10:30], 50, keep_thr, 13)
    assert np.array_equal(whole[10:30], part)
    other, _ = O.subsample_walks(walks, 41, keep_thr, 13)
    assert not np.array_equal(whole, other)


# ---------------------------------------------------------------- start-node shuffle
@pytest.mark.parametrize("n", [1, 2, 3, 4, 5, 16, 17, 1000, 1024, 1025, 65537])
def test_shuffle_is_a_bijection_of_the_node_range(n):
    for epoch in (0, 1, 7):
        st = O.shuffled_starts(n, 99, epoch, 0, n)
        assert np.array_equal(np.sort(st), np.arange(n, dtype=np.int32))


def test_shuffle_stays_injective_at_the_largest_node_count():
    n = 2**31 - 1
    st = O.shuffled_starts(n, 5, 1, 0, 200_000).astype(np.int64)
    assert st.min() >= 0 and st.max() < n and len(np.unique(st)) == len(st)
    # images are spread over the whole range
    assert chi2_uniform_ok(np.bincount(st * 16 // n, minlength=16))


def test_shuffle_depends_on_seed_and_epoch_and_wraps_over_walk_ids():
    n = 5000
    a = O.shuffled_starts(n, 1, 0, 0, n)
    assert not np.array_equal(a, O.shuffled_starts(n, 1, 1, 0, n))
    assert not np.array_equal(a, O.shuffled_starts(n, 2, 0, 0, n))
    assert (a != np.arange(n)).mean() > 0.99                    # about one fixed point expected
    # walk id a starts at shuffle(a mod n): the second repetition repeats the first
    b = O.shuffled_starts(n, 1, 0, n - 10, 30)
    assert np.array_equal(b[:10], a[-10:]) and np.array_equal(b[10:], a[:20])
    assert O.shuffle_node(17, n, 1, 0) == a[17]


def test_shuffle_images_are_uniform_over_epochs():
    n = 12
    counts = np.zeros((n, n))
    for epoch in range(6000):
        st = O.shuffled_starts(n, 3, epoch, 0, n)
        counts[np.arange(n), st] += 1
    for v in range(n):
        assert chi2_uniform_ok(counts[v])                        # image of node v
        assert chi2_uniform_ok(counts[:, v])                     # preimage of node v


# ---------------------------------------------------------------- Adam
def test_adam_rows_match_library_adam_dense_and_sparse():
    rng = np.random.default_rng(0)
    n, d, lr, b1, b2, eps = 7, 5, 0.01, 0.9, 0.999, 1e-8
    x0 = rng.normal(size=(n, d))
    # dense: every row touched in every step = torch.optim.Adam
    x, m, v = x0.copy(), np.zeros((n, d)), np.zeros((n, d))
    p = torch.tensor(x0, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.Adam([p], lr=lr, betas=(b1, b2), eps=eps)
    for step in range(1, 6):
        g = rng.normal(size=(n, d))
        O.adam_rows(x, m, v, g, np.arange(n), lr, b1, b2, eps, step)
        p.grad = torch.tensor(g)
        opt.step()
    assert np.abs(x - p.detach().numpy()).max() < 1e-12
    # sparse: only some rows per step = torch.optim.SparseAdam (moments of the other rows rest,
    # one step counter for all rows).  That routine adds eps before the bias correction of the
    # second moment, Algorithm 1 after it (pinned by the dense case above); with a vanishing
    # eps the two agree, which isolates the row selection.
    eps = 1e-300
    x, m, v = x0.copy(), np.zeros((n, d)), np.zeros((n, d))
    p = torch.nn.Parameter(torch.tensor(x0, dtype=torch.float64))
    opt = torch.optim.SparseAdam([p], lr=lr, betas=(b1, b2), eps=eps)
    for step in range(1, 8):
        rows = np.sort(rng.choice(n, size=3, replace=False))
        g = np.zeros((n, d))
        g[rows] = rng.normal(size=(3, d))
        O.adam_rows(x, m, v, g, rows, lr, b1, b2, eps, step)
        p.grad = torch.sparse_coo_tensor(torch.tensor(rows[None, :]), torch.tensor(g[rows]), (n, d))
        opt.step()
    assert np.abs(x - p.detach().numpy()).max() < 1e-12
    # first step of Adam moves every touched value by lr * sign(g) (up to eps)
    x, m, v = np.zeros((2, 3)), np.zeros((2, 3)), np.zeros((2, 3))
    g = np.array([[1.0, -2.0, 0.5], [3.0, 3.0, 3.0]])
    O.adam_rows(x, m, v, g, np.array([0]), lr, b1, b2, 1e-8, 1)
    assert np.allclose(x[0], -lr * np.sign(g[0]), atol=1e-9) and (x[1] == 0).all()


def test_touched_rows_and_adam_step_on_lists():
    off, col, thr, alias, walks = tiny_setup(n=120, L=12, n_walks=40)
    n = len(off) - 1
    c, o, ng, pairs = O.expand_lists(walks, 40, 3, 4, thr, alias, 9)
    rows_in, rows_out = O.touched_rows(c, o, ng)
    ok = c >= 0
    assert set(rows_in) == set(c[ok])
    want_out = set(o[ok])
    for e in np.nonzero(ok)[0]:
        want_out |= {x for x in ng[e] if x >= 0 and x != o[e]}
    assert set(rows_out) == want_out
    rng = np.random.default_rng(1)
    U, V = rng.normal(size=(n, 8)) * 0.1, rng.normal(size=(n, 8)) * 0.1
    U0, V0 = U.copy(), V.copy()
    MU, VU, MV, VV = (np.zeros_like(U) for _ in range(4))
    loss, cnt = O.sgns_adam_step_from_lists(U, V, MU, VU, MV, VV, c, o, ng, 0.01, 0.9, 0.999, 1e-8, 1)
    assert cnt == pairs and loss > 0
    untouched_in = np.setdiff1d(np.arange(n), rows_in)
    assert np.array_equal(U[untouched_in], U0[untouched_in]) and (MU[untouched_in] == 0).all()
    GU, GV, _, _ = O.sgns_grad_from_lists(U0, V0, c, o, ng)
    moved = np.abs(GV) > 1e-6                                     # step 1: lr * sign(g)
    assert np.allclose((V - V0)[moved], -0.01 * np.sign(GV[moved]), atol=1e-6)


# ---------------------------------------------------------------- stochastic rounding to 16 bits
def neighbours_f16(x32):
    """(lo, hi) of |x32| among the binary16 values, lo towards zero, by numpy's own conversion and
    nextafter; hi is inf above the largest finite value."""
    ax = np.abs(x32.astype(np.float64))
    a = np.abs(x32).astype(np.float16)                       # to nearest
    lo = np.where(a.astype(np.float64) <= ax, a, np.nextafter(a, np.float16(0)))
    hi = np.nextafter(lo, np.float16(np.inf))
    return lo.astype(np.float64), hi.astype(np.float64)


def neighbours_bf16(x32):
    """(lo, hi) of |x32| among the bfloat16 values: the upper 16 bits of the fp32 pattern."""
    bits = np.abs(x32).view(np.uint32)
    lo = (bits & np.uint32(0xFFFF0000)).view(np.float32).astype(np.float64)
    hi = ((bits & np.uint32(0xFFFF0000)) + np.uint32(0x10000)).view(np.float32).astype(np.float64)
    return lo, hi


def sample_values(rng, n, fmt):
    mags = rng.uniform(-30, 12, n) if fmt == 0 else rng.uniform(-120, 100, n)   # includes binary16 subnormals
    return (rng.choice([-1.0, 1.0], n) * rng.uniform(1, 2, n) * 2.0 ** mags).astype(np.float32)


@pytest.mark.parametrize("fmt", [0, 1])
def test_stochastic_rounding_picks_a_neighbour_with_the_right_threshold(fmt):
    rng = np.random.default_rng(3 + fmt)
    x = sample_values(rng, 20000, fmt)
    lo, hi = (neighbours_f16 if fmt == 0 else neighbours_bf16)(x)
    finite = np.isfinite(hi)
    ax = np.abs(x.astype(np.float64))
    frac = np.where(finite & (hi > lo), (ax - lo) / np.where(finite & (hi > lo), hi - lo, 1.0), 0.0)
    thr = np.floor(frac * 65536.0).astype(np.int64)
    assert ((frac >= 0) & (frac < 1)).all() and (thr[frac > 0] >= 0).all()
    sign = np.sign(x.astype(np.float64))
    for u in (np.zeros_like(thr), np.maximum(thr - 1, 0), thr, np.full_like(thr, 65535), rng.integers(0, 65536, len(thr))):
        got = O.round_sr(x.astype(np.float64), fmt, u.astype(np.uint32))
        want = sign * np.where((u < thr) & finite, hi, lo)
        assert np.array_equal(got, want)
    # representable values never move, whatever the dither
    rep = lo[lo > 0] * sign[lo > 0]
    for u in (0, 1, 40000, 65535):
        assert np.array_equal(O.round_sr(rep.copy(), fmt, np.full(len(rep), u, dtype=np.uint32)), rep)


@pytest.mark.parametrize("fmt", [0, 1])
def test_stochastic_rounding_is_unbiased_and_saturates(fmt):
    # over all 65536 dithers the mean is lo + (hi - lo) * thr / 2^16: within one 2^-16 of the spacing of x
    rng = np.random.default_rng(8)
    u_all = np.arange(65536, dtype=np.uint32)
    for x in sample_values(rng, 12, fmt):
        lo, hi = (neighbours_f16 if fmt == 0 else neighbours_bf16)(np.array([x], dtype=np.float32))
        got = O.round_sr(np.full(65536, float(x)), fmt, u_all)
        assert set(np.unique(np.abs(got))) <= {lo[0], hi[0]}
        assert abs(got.mean() - float(x)) <= (hi[0] - lo[0]) / 65536.0 + 1e-300
        ups = int((np.abs(got) == hi[0]).sum()) if hi[0] > lo[0] else 0
        assert ups == int(np.floor((abs(float(x)) - lo[0]) / (hi[0] - lo[0]) * 65536.0))
    # an exact tie goes up for exactly half of the dithers
    tie = 1.0 + (2.0 ** -11 if fmt == 0 else 2.0 ** -8)
    got = O.round_sr(np.full(65536, tie), fmt, u_all)
    assert int((got > 1.0).sum()) == 32768 and np.array_equal(got > 1.0, u_all < 32768)
    # beyond the largest finite value, and a step up from it: the largest finite value, never inf
    top = 65504.0 if fmt == 0 else float(np.array([0x7F7F0000], dtype=np.uint32).view(np.float32)[0])
    edge = np.array([top, -top, top * (1 + 2.0 ** -13), 1e39, -1e39, np.inf])
    for u in (0, 65535):
        got = O.round_sr(edge.copy(), fmt, np.full(len(edge), u, dtype=np.uint32))
        assert np.array_equal(got, [top, -top, top, top, -top, top])
    # symmetric in the sign
    x = sample_values(rng, 500, fmt).astype(np.float64)
    u = rng.integers(0, 65536, len(x)).astype(np.uint32)
    assert np.array_equal(O.round_sr(x.copy(), fmt, u), -O.round_sr(-x, fmt, u))


def test_dithers_of_a_row_write_are_keyed_well_spread_and_distinct():
    rng = np.random.default_rng(1)
    counts = np.zeros(64)
    for _ in range(400):
        r = rng.integers(0, 2 ** 32, 4, dtype=np.uint64).astype(np.uint32)
        salt = int(rng.integers(0, 2 ** 17))
        d = O.dither16(r, salt, 256)
        assert np.array_equal(d, O.dither16(r, salt, 256)) and d.max() < 65536      # a function of its key
        assert not np.array_equal(d, O.dither16(r, salt + 1, 256))                  # the salt matters
        r2 = r.copy()
        r2[2] ^= 1
        assert not np.array_equal(d, O.dither16(r2, salt, 256))                     # so does every word
        # columns 2k and 2k+1 are the halves of one mixed word, and the mixed words of a row are
        # pairwise distinct (the mix is a bijection and the columns feed it distinct inputs
        # unless two of the four words happen to collide, which random words do not)
        words = (d[0::2].astype(np.uint64) << np.uint64(16)) | d[1::2].astype(np.uint64)
        assert len(np.unique(words)) == len(words)
        counts += np.bincount(d >> 10, minlength=64)
    assert chi2_uniform_ok(counts)


def sync_event(seed, row, table, base):
    return O.philox4x32_10([row & 0xFFFFFFFF, table, base & 0xFFFFFFFF, (8 << 24) | ((base >> 32) & 0xFFFFFF)],
                           [seed & 0xFFFFFFFF, seed >> 32])


@pytest.mark.parametrize("fmt", [0, 1])
def test_synchronous_step_with_stochastic_write_back(fmt):
    # the step is the full-precision step followed by ONE stochastic rounding of every written value,
    # keyed by (row, table, first walk id of the step): re-assembled here from the Philox block,
    # the dithers and the rounding of single values
    off, col, thr, alias, walks = tiny_setup(n_walks=40, L=12)
    n, d, seed, base = len(off) - 1, 32, 77, (5 << 32) + 40
    c, o, ng, _ = O.expand_lists(walks, base, 3, 2, thr, alias, seed)
    rng = np.random.default_rng(2)
    rnd = O.round_f16 if fmt == 0 else O.round_bf16
    U0 = rnd(rng.uniform(-0.3, 0.3, (n, d)))
    V0 = rnd(rng.uniform(-0.3, 0.3, (n, d)))
    Ue, Ve = U0.copy(), V0.copy()
    O.sgns_det_from_lists(Ue, Ve, c, o, ng, 0.05)                        # exact step
    U, V = U0.copy(), V0.copy()
    O.sgns_det_sr_from_lists(U, V, c, o, ng, 0.05, fmt, seed, base)
    for X, Xe, X0, table in ((U, Ue, U0, 0), (V, Ve, V0, 1)):
        touched = np.nonzero((Xe != X0).any(axis=1))[0]
        assert len(touched) > 50
        assert np.array_equal(np.delete(X, touched, axis=0), np.delete(X0, touched, axis=0))   # others keep their bits
        for row in touched[:40]:
            u = O.dither16(sync_event(seed, int(row), table, base), 0, d)
            assert np.array_equal(X[row], O.round_sr(Xe[row].copy(), fmt, u))
    # another step (another first walk id) or another seed rounds differently; the same key repeats
    U2, V2 = U0.copy(), V0.copy()
    O.sgns_det_sr_from_lists(U2, V2, c, o, ng, 0.05, fmt, seed, base)
    assert np.array_equal(U, U2) and np.array_equal(V, V2)
    U3, V3 = U0.copy(), V0.copy()
    O.sgns_det_sr_from_lists(U3, V3, c, o, ng, 0.05, fmt, seed + 1, base)
    assert not np.array_equal(V, V3)
    # unbiased where to-nearest is not: mean over seeds against the exact value
    rows = np.nonzero((Ve != V0).any(axis=1))[0][:8]
    acc = np.zeros((len(rows), d))
    n_seeds = 300
    for s in range(n_seeds):
        Us, Vs = U0.copy(), V0.copy()
        O.sgns_det_sr_from_lists(Us, Vs, c, o, ng, 0.05, fmt, 1000 + s, base)
        acc += Vs[rows]
    spacing = np.abs(Ve[rows]) * 2.0 ** (-10 if fmt == 0 else -7)         # at most one unit in the last place
    assert (np.abs(acc / n_seeds - Ve[rows]) <= 4 * 0.5 * spacing / np.sqrt(n_seeds) + 1e-9).all()


@pytest.mark.parametrize("fmt", [0, 1])
def test_sequential_mode_with_stochastic_write_back_keys_every_write(fmt):
    # one walk, no negatives: the first pair of position 0 writes the context row and, after the
    # position's last pair, the center row - with the block (walk id, position, tag 9), salt 1 + index
    # in the position's target list for the target and 0x10000 for the center
    n, d, L, w, seed, base = 50, 16, 4, 1, 9, 1234
    walk = np.array([[3, 7, 11, 15]], dtype=np.int32)
    thr, alias = O.build_alias(np.ones(n), 1.0)
    c, o, ng, _ = O.expand_lists(walk, base, w, 0, thr, alias, seed)
    rng = np.random.default_rng(4)
    rnd = O.round_f16 if fmt == 0 else O.round_bf16
    U0, V0 = rnd(rng.uniform(-0.4, 0.4, (n, d))), rnd(rng.uniform(-0.4, 0.4, (n, d)))
    U, V = U0.copy(), V0.copy()
    O.sgns_seq_sr_from_lists(U, V, c, o, ng, 2 * w, 0.1, fmt, seed, base, L)
    # position 0 has one pair: (3, 7) in slot 1 (the later context); K = 0, so its list index is 1
    ev = O.philox4x32_10([base & 0xFFFFFFFF, base >> 32, 0, 9 << 24], [seed, 0])
    f = float(U0[3] @ V0[7])
    g = 1.0 / (1.0 + np.exp(-f)) - 1.0
    want_v = O.round_sr(V0[7] - 0.1 * g * U0[3], fmt, O.dither16(ev, 1 + 1, d))
    want_u = O.round_sr(U0[3] - 0.1 * g * V0[7], fmt, O.dither16(ev, 0x10000, d))
    assert np.array_equal(U[3], want_u)
    # row 7 is written again by position 2 (center 11): undo nothing, compare after position 0 only
    Ua, Va = U0.copy(), V0.copy()
    O.sgns_seq_sr_from_lists(Ua, Va, c[:2], o[:2], ng[:2], 2 * w, 0.1, fmt, seed, base, L)
    assert np.array_equal(Va[7], want_v) and np.array_equal(Ua[3], want_u)
    # with dithers that never round up the result is truncation; the mode differs from to-nearest
    Ub, Vb = U0.copy(), V0.copy()
    (O.sgns_seq_f16_from_lists if fmt == 0 else O.sgns_seq_bf16_from_lists)(Ub, Vb, c, o, ng, 2 * w, 0.1)
    assert not np.array_equal(V, Vb)
    assert np.abs(V - Vb).max() <= np.abs(Vb).max() * 2.0 ** (-9 if fmt == 0 else -6)


# ---- increments rounded to the format and added in the format (Section 3.2: the trainer sends
# increments, the storage adds them), sequential order
def _round_to_bits(x, bits):
    """Nearest-even rounding of float64 values to `bits` significant bits (normal range), written
    with frexp / rint / ldexp: independent of the oracle's C code."""
    m, e = np.frexp(np.asarray(x, dtype=np.float64))
    return np.ldexp(np.rint(m * 2.0 ** bits), e - bits)


@pytest.mark.parametrize("fmt", [0, 1])
def test_increment_and_add_rounds_twice_where_the_plain_write_back_rounds_once(fmt):
    # One pair, dimension 1, no negative: context value 1.0, center value 2^-10.  The learning rate
    # is chosen so that the context's increment is a hair above HALF a unit of 1.0 in the format:
    # written back in one rounding, 1 + inc goes up to the next value; sent as an increment, inc is
    # first rounded to exactly half a unit, the sum is a tie, and ties go to the even neighbour 1.0.
    import math
    bits = 11 if fmt == 0 else 8                      # significant bits of the format
    half_unit = 2.0 ** -bits                          # half the spacing just above 1.0
    u, v = 2.0 ** -10, 1.0
    g = 1.0 / (1.0 + math.exp(-u * v)) - 1.0          # context: sigmoid(f) - 1
    lr = half_unit * (1.0 + 2.0 ** -19) / (-g * u)
    assert abs(-lr * g * u / half_unit - 1.0 - 2.0 ** -19) < 1e-12
    c = np.array([0], dtype=np.int32)
    o = np.array([1], dtype=np.int32)
    ng = np.array([[-1]], dtype=np.int32)
    seq16 = O.sgns_seq_f16_from_lists if fmt == 0 else O.sgns_seq_bf16_from_lists

    def tables():
        return np.array([[u], [0.0]]), np.array([[0.0], [v]])
    U1, V1 = tables()
    seq16(U1, V1, c, o, ng, 1, lr)
    assert V1[1, 0] == 1.0 + 2.0 * half_unit          # one rounding: up
    U2, V2 = tables()
    loss, cnt = O.sgns_seq_add16_from_lists(U2, V2, c, o, ng, 1, lr, fmt)
    assert cnt == 1 and abs(loss - math.log1p(math.exp(-u * v))) < 1e-15
    assert V2[1, 0] == 1.0                            # two roundings: the tie goes to even
    # the center row: its increment -lr * g * v = inc / u is representable after rounding, and so is the sum here
    inc_u = _round_to_bits(-lr * g * v, bits)
    assert U2[0, 0] == _round_to_bits(u + inc_u, bits)


@pytest.mark.parametrize("fmt", [0, 1])
def test_increment_and_add_is_the_full_precision_step_rounded_as_increment_then_as_sum(fmt):
    # One position whose targets are all different rows: every row is written once, so the clause
    # must equal  round(old + round(new_full - old))  with new_full from the full-precision sequential
    # step and the rounding done here with frexp / rint (binary16 also with numpy's conversion).
    bits = 11 if fmt == 0 else 8
    rng = np.random.default_rng(17 + fmt)
    n, d, S, K = 64, 24, 6, 3
    ids = rng.permutation(n)
    c = np.full(S, ids[0], dtype=np.int32)
    o = ids[1:1 + S].astype(np.int32)
    ng = ids[1 + S:1 + S + S * K].reshape(S, K).astype(np.int32)
    c[4], o[4], ng[4] = -1, -1, -1                     # a slot without a pair
    ng[2, 1] = -1                                      # an absent negative
    U0 = _round_to_bits(rng.uniform(-0.5, 0.5, (n, d)), bits)
    V0 = _round_to_bits(rng.uniform(-0.5, 0.5, (n, d)), bits)
    lr = 0.05
    Uf, Vf = U0.copy(), V0.copy()
    loss_f, cnt_f = O.sgns_seq_from_lists(Uf, Vf, c, o, ng, S, lr)
    U, V = U0.copy(), V0.copy()
    loss, cnt = O.sgns_seq_add16_from_lists(U, V, c, o, ng, S, lr, fmt)
    assert cnt == cnt_f == S - 1 and abs(loss - loss_f) < 1e-12
    want_U = _round_to_bits(U0 + _round_to_bits(Uf - U0, bits), bits)
    want_V = _round_to_bits(V0 + _round_to_bits(Vf - V0, bits), bits)
    # new_full - old carries fp64 rounding of about 1e-17, far from deciding a rounding here
    assert np.array_equal(U, want_U) and np.array_equal(V, want_V)
    touched = np.concatenate([[ids[0]], o[o >= 0], ng[ng >= 0]])
    assert (V != V0).any(axis=1).sum() == len(touched) - 1 and (U != U0).any(axis=1).sum() == 1
    if fmt == 0:                                       # numpy has binary16: round with its conversion as well
        h = lambda x: x.astype(np.float16).astype(np.float64)
        assert np.array_equal(V, h(V0 + h(Vf - V0))) and np.array_equal(U, h(U0 + h(Uf - U0)))
    # and it is not the single rounding: some values differ from the plain 16-bit write-back
    U1, V1 = U0.copy(), V0.copy()
    (O.sgns_seq_f16_from_lists if fmt == 0 else O.sgns_seq_bf16_from_lists)(U1, V1, c, o, ng, S, lr)
    assert np.abs(V1 - V).max() <= 2.0 ** (1 - bits) and (V1 != V).any()


def test_increment_and_add_drops_increments_below_half_a_unit_of_the_stored_value():
    # The same tiny increment sent 200 times (one position with 200 slots that name the same context,
    # so the center row stays as it is meanwhile): each is below half a unit of the stored value, so
    # a table that adds in its own format never moves, while the increments add up to more than a unit.
    c = np.zeros(200, dtype=np.int32)
    o = np.ones(200, dtype=np.int32)
    ng = np.full((200, 1), -1, dtype=np.int32)
    U = np.array([[2.0 ** -12], [0.0]])
    V = np.array([[0.0], [1.0]])
    lr = 0.05                                          # increment about 0.05 * 0.5 * 2^-12 = 6e-6; half a unit of 1.0 is 4.9e-4
    O.sgns_seq_add16_from_lists(U, V, c, o, ng, 200, lr, 0)
    assert V[1, 0] == 1.0
    Uf, Vf = np.array([[2.0 ** -12], [0.0]]), np.array([[0.0], [1.0]])
    O.sgns_seq_from_lists(Uf, Vf, c, o, ng, 200, lr)
    assert Vf[1, 0] - 1.0 > 1e-3
