"""Pins of the CPU oracle against what the literature and the mathematics fix.

None of these tests touches the CUDA library.  Each one is chosen so that a
plausible slip in the oracle (dropped term, wrong sign, off-by-one index,
transposed operand) makes it fail.
"""
from pathlib import Path

import numpy as np
import pytest
import torch
from scipy import stats

from oracle import gs_oracle as O
from paper_2407_15452_b200 import workloads as WL

GOLDEN = Path(__file__).parent / "golden"
CHI2_P = 1e-4          # fixed seeds, so a pass is reproducible; this is the alarm level


def pairs_per_full_walk(L, w):
    """Number of (center, context) pairs of a walk without dead ends, by direct counting: position
    i pairs with every other position within w of it."""
    return sum(min(L - 1, i + w) - max(0, i - w) for i in range(L))


def np_graph(g):
    return g.offsets.cpu().numpy().astype(np.int64), g.cols.cpu().numpy()


def adjacency_sets(off, col):
    return [set(col[off[v]:off[v + 1]].tolist()) for v in range(len(off) - 1)]


def chi2_ok(counts, probs):
    counts = np.asarray(counts, dtype=np.float64)
    probs = np.asarray(probs, dtype=np.float64)
    keep = probs > 0
    assert counts[~keep].sum() == 0
    exp = probs[keep] * counts.sum()
    stat = ((counts[keep] - exp) ** 2 / exp).sum()
    return stat < stats.chi2.ppf(1 - CHI2_P, keep.sum() - 1), stat


# ---------------------------------------------------------------- Philox
def test_philox_known_answers():
    rows = [l.split() for l in (GOLDEN / "philox4x32_10_kat.txt").read_text().splitlines()
            if l.strip() and not l.startswith("#")]
    assert len(rows) == 3
    for r in rows:
        w = [int(x, 16) for x in r]
        out = O.philox4x32_10(w[0:4], w[4:6])
        assert [int(x) for x in out] == w[6:10]


# ---------------------------------------------------------------- uniform walks
def test_uniform_walks_follow_edges_and_pad_after_dead_ends():
    g = WL.rmat_graph(2000, 6000, seed=7)          # directed: has dead ends
    off, col = np_graph(g)
    adj = adjacency_sets(off, col)
    deg = off[1:] - off[:-1]
    assert (deg == 0).any() and (deg > 0).any()
    walks, steps = O.uniform_walks(off, col, None, 4000, 0, 12, seed=3)
    n_steps = 0
    saw_dead = False
    for i, W in enumerate(walks):
        assert W[0] == i % 2000
        alive = True
        for t in range(11):
            if alive and deg[W[t]] > 0:
                assert W[t + 1] in adj[W[t]]
                n_steps += 1
            else:
                alive = False
                saw_dead = True
                assert W[t + 1] == -1
    assert saw_dead and n_steps == steps


def test_uniform_walk_one_step_transition_matrix():
    g = WL.ring_with_chords(6)
    off, col = np_graph(g)
    adj = adjacency_sets(off, col)
    n_walks = 120_000
    starts = (np.arange(n_walks) % 6).astype(np.int32)
    walks, _ = O.uniform_walks(off, col, starts, n_walks, 10, 2, seed=11)
    for v in range(6):
        nxt = walks[walks[:, 0] == v, 1]
        probs = np.array([1.0 / len(adj[v]) if u in adj[v] else 0.0 for u in range(6)])
        ok, stat = chi2_ok(np.bincount(nxt, minlength=6), probs)
        assert ok, (v, stat)


def test_uniform_walk_keeps_degree_proportional_distribution():
    # On a connected, non-bipartite, undirected graph deg(v)/sum(deg) is stationary:
    # walks started from it must show it at every later position.
    g = WL.ring_with_chords(12)
    off, col = np_graph(g)
    deg = (off[1:] - off[:-1]).astype(np.float64)
    pi = deg / deg.sum()
    rng = np.random.default_rng(5)
    n_walks = 200_000
    starts = rng.choice(12, size=n_walks, p=pi).astype(np.int32)
    walks, _ = O.uniform_walks(off, col, starts, n_walks, 0, 8, seed=2)
    for t in range(1, 8):
        ok, stat = chi2_ok(np.bincount(walks[:, t], minlength=12), pi)
        assert ok, (t, stat)


def test_uniform_long_walks_from_every_node_approach_stationary_mass():
    g = WL.ring_with_chords(12)
    off, col = np_graph(g)
    deg = (off[1:] - off[:-1]).astype(np.float64)
    walks, _ = O.uniform_walks(off, col, None, 12 * 5000, 0, 40, seed=9)
    ok, stat = chi2_ok(np.bincount(walks[:, 39], minlength=12), deg / deg.sum())
    assert ok, stat


def test_walks_depend_on_walk_id_not_on_batching():
    g = WL.chung_lu_graph(500, 6, 2.5, seed=1)
    off, col = np_graph(g)
    full, _ = O.uniform_walks(off, col, None, 900, 0, 9, seed=4)
    part, _ = O.uniform_walks(off, col, None, 300, 450, 9, seed=4)
    assert np.array_equal(full[450:750], part)
    other, _ = O.uniform_walks(off, col, None, 900, 0, 9, seed=5)
    assert not np.array_equal(full, other)


# ---------------------------------------------------------------- node2vec
def six_node_graph():
    # prev=0, cur=1: adj(1) = {0: back, 2: neighbour of 0, 3 and 4: far}
    edges = [(0, 1), (1, 2), (0, 2), (1, 3), (1, 4), (3, 5), (4, 5)]
    s = torch.tensor([e[0] for e in edges] + [e[1] for e in edges], dtype=torch.int64)
    d = torch.tensor([e[1] for e in edges] + [e[0] for e in edges], dtype=torch.int64)
    return WL._csr_from_directed(s, d, 6, False)


def closed_form_node2vec(adj, prev, cur, p, q):
    wts = {}
    for x in adj[cur]:
        wts[x] = 1.0 / p if x == prev else (1.0 if x in adj[prev] else 1.0 / q)
    z = sum(wts.values())
    return {x: a / z for x, a in wts.items()}


@pytest.mark.parametrize("p,q", [(0.5, 2.0), (4.0, 0.25), (1.0, 1.0)])
def test_node2vec_transition_probabilities_match_closed_form(p, q):
    g = six_node_graph()
    off, col = np_graph(g)
    adj = adjacency_sets(off, col)
    n_walks = 240_000
    walks, steps, caps = O.node2vec_walks(off, col, None, n_walks, 0, 4, seed=21, p=p, q=q)
    assert caps == 0 and steps == n_walks * 3
    if (p, q) == (0.5, 2.0):
        cf = closed_form_node2vec(adj, 0, 1, p, q)
        assert np.allclose([cf[0], cf[2], cf[3], cf[4]], [0.5, 0.25, 0.125, 0.125])
    checked = 0
    for t in (1, 2):
        for prev in range(6):
            for cur in adj[prev]:
                sel = (walks[:, t - 1] == prev) & (walks[:, t] == cur)
                if sel.sum() < 2000:
                    continue
                cf = closed_form_node2vec(adj, prev, cur, p, q)
                probs = np.array([cf.get(x, 0.0) for x in range(6)])
                ok, stat = chi2_ok(np.bincount(walks[sel, t + 1], minlength=6), probs)
                assert ok, (prev, cur, stat)
                checked += 1
    assert checked >= 10


def test_node2vec_thresholds():
    assert O.node2vec_thresholds(0.5, 2.0).tolist() == [2 ** 32, 2 ** 31, 2 ** 30]
    assert O.node2vec_thresholds(1.0, 1.0).tolist() == [2 ** 32] * 3
    assert O.node2vec_thresholds(4.0, 0.25).tolist() == [2 ** 28, 2 ** 30, 2 ** 32]


def test_node2vec_first_step_is_uniform_and_walks_follow_edges():
    g = WL.chung_lu_graph(300, 6, 2.5, seed=3)
    off, col = np_graph(g)
    adj = adjacency_sets(off, col)
    walks, _, _ = O.node2vec_walks(off, col, None, 3000, 0, 10, seed=8, p=0.5, q=2.0)
    for W in walks:
        for t in range(9):
            if W[t + 1] >= 0:
                assert W[t + 1] in adj[W[t]]
            else:
                assert W[t] == -1 or len(adj[W[t]]) == 0


def test_node2vec_rejection_cap_keeps_last_proposal():
    g = six_node_graph()
    off, col = np_graph(g)
    # q huge: far candidates are almost never accepted; one round only -> cap hits happen,
    # and the walk still moves along an edge.
    walks, steps, caps = O.node2vec_walks(off, col, None, 6000, 0, 5, seed=1, p=1e9, q=1e9,
                                          max_rounds=1)
    adj = adjacency_sets(off, col)
    assert caps > 0 and steps == 6000 * 4
    for W in walks[:500]:
        for t in range(4):
            assert W[t + 1] in adj[W[t]]


# ---------------------------------------------------------------- pairs
def brute_pairs(W, w):
    out = []
    for i in range(len(W)):
        for j in range(len(W)):
            if i != j and abs(i - j) <= w and W[i] >= 0 and W[j] >= 0:
                out.append((i, j, int(W[i]), int(W[j])))
    return out


@pytest.mark.parametrize("L,w", [(10, 5), (40, 10), (5, 3), (7, 9), (3, 1)])
def test_pair_expansion_count_identity_and_brute_force(L, w):
    rng = np.random.default_rng(L * 100 + w)
    walks = rng.integers(0, 50, size=(6, L)).astype(np.int32)
    walks[4, L // 2:] = -1                               # a walk that died early
    walks[5, 1:] = -1
    thr = np.full(50, 0xFFFFFFFF, dtype=np.uint32)
    alias = np.arange(50, dtype=np.int32)
    c, o, ng, n_pairs = O.expand_lists(walks, 0, w, 2, thr, alias, seed=0)
    c = c.reshape(6, L, 2 * w)
    o = o.reshape(6, L, 2 * w)
    if L > w:
        assert pairs_per_full_walk(L, w) == 2 * (w * L - w * (w + 1) // 2)
    total = 0
    for a in range(6):
        got = []
        for i in range(L):
            for sg in range(2 * w):
                if c[a, i, sg] >= 0:
                    j = i - w + sg + (1 if sg >= w else 0)
                    got.append((i, j, int(c[a, i, sg]), int(o[a, i, sg])))
                else:
                    assert o[a, i, sg] == -1
        want = brute_pairs(walks[a], w)
        assert sorted(got) == sorted(want)
        assert got == sorted(got)                        # canonical order: i, then j
        # symmetry: (x, y) at (i, j) <=> (y, x) at (j, i)
        assert {(i, j, x, y) for (i, j, x, y) in got} == {(j, i, y, x) for (i, j, x, y) in got}
        if a < 4:
            assert len(got) == pairs_per_full_walk(L, w)
        total += len(got)
    assert total == n_pairs
    assert (ng.reshape(6, L, 2 * w, 2)[c < 0] == -1).all()


def test_forward_only_pairs_are_the_later_half_and_line_edges():
    rng = np.random.default_rng(3)
    walks = rng.integers(0, 50, size=(5, 9)).astype(np.int32)
    walks[4, 5:] = -1
    thr = np.full(50, 0xFFFFFFFF, dtype=np.uint32)
    alias = np.arange(50, dtype=np.int32)
    w = 3
    c, o, ng, n_all = O.expand_lists(walks, 0, w, 2, thr, alias, 1)
    cf, of, ngf, n_fwd = O.expand_lists(walks, 0, w, 2, thr, alias, 1, forward_only=True)
    for a in range(5):
        want = [(i, j, x, y) for (i, j, x, y) in brute_pairs(walks[a], w) if j > i]
        got = []
        for i in range(9):
            for sg in range(2 * w):
                e = (a * 9 + i) * 2 * w + sg
                if cf[e] >= 0:
                    j = i - w + sg + (1 if sg >= w else 0)
                    got.append((i, j, int(cf[e]), int(of[e])))
                    assert np.array_equal(ngf[e], ng[e])      # same draws as in the two-sided list
        assert got == want
    assert 2 * n_fwd == n_all                                  # pairs are symmetric: half are forward
    # LINE: walks of two nodes, window 1 -> exactly one pair (source, neighbour) per source
    edges = rng.integers(0, 50, size=(40, 2)).astype(np.int32)
    cl, ol, _, n_line = O.expand_lists(edges, 0, 1, 3, thr, alias, 1, forward_only=True)
    assert n_line == 40
    sel = cl >= 0
    assert np.array_equal(cl[sel], edges[:, 0]) and np.array_equal(ol[sel], edges[:, 1])


# ---------------------------------------------------------------- alias table, negatives
def implied_mass(thr, alias):
    n = len(thr)
    keep = thr.astype(np.float64) / 2.0 ** 32
    keep[(thr == 0xFFFFFFFF) & (alias == np.arange(n))] = 1.0
    mass = keep.copy()
    np.add.at(mass, alias, 1.0 - keep)
    return mass / n


@pytest.mark.parametrize("power", [0.75, 1.0, 0.0])
def test_alias_table_mass_identity(power):
    rng = np.random.default_rng(17)
    wgt = rng.pareto(1.2, size=5000) + 0.01
    wgt[rng.integers(0, 5000, 300)] = 0.0
    thr, alias = O.build_alias(wgt, power)
    target = np.where(wgt > 0, np.power(np.where(wgt > 0, wgt, 1.0), power), 0.0)
    target /= target.sum()
    assert np.abs(implied_mass(thr, alias) - target).max() < 2.0 ** -30
    assert (alias >= 0).all() and (alias < 5000).all()
    if power == 0.0:
        pos = wgt > 0
        assert np.allclose(implied_mass(thr, alias)[pos], 1.0 / pos.sum(), atol=2.0 ** -30)


def test_alias_rejects_all_zero_weights():
    with pytest.raises(ValueError):
        O.build_alias(np.zeros(8), 0.75)


def test_negative_draws_follow_unigram_power_distribution():
    wgt = np.array([1, 2, 3, 4, 0, 6, 7, 8, 50, 100], dtype=np.float64)
    thr, alias = O.build_alias(wgt, 0.75)
    L, w, K = 10, 5, 5
    walks = np.tile(np.arange(10, dtype=np.int32), (3000, 1))
    c, o, ng, n_pairs = O.expand_lists(walks, 1000, w, K, thr, alias, seed=33)
    draws = ng[c >= 0].ravel()
    assert len(draws) == n_pairs * K and n_pairs == 3000 * pairs_per_full_walk(L, w)
    probs = wgt ** 0.75
    probs /= probs.sum()
    ok, stat = chi2_ok(np.bincount(draws, minlength=10), probs)
    assert ok, stat
    assert (draws != 4).all()                            # zero weight: never drawn
    # draws of different slots / walks are distinct streams
    first = np.flatnonzero(c >= 0)[:2]
    assert not np.array_equal(ng[first[0]], ng[first[1]])
    per_walk = ng.reshape(3000, -1)
    assert not np.array_equal(per_walk[0], per_walk[1])
    # the K draws of one pair are distinct streams too (each column has the same law)
    valid = ng[c >= 0]
    for k in range(K):
        ok, stat = chi2_ok(np.bincount(valid[:, k], minlength=10), probs)
        assert ok, (k, stat)
    assert np.mean(valid[:, 0] == valid[:, 1]) < 0.5


# ---------------------------------------------------------------- SGNS step
def small_problem(seed, n=30, d=8, K=3, L=6, w=2, n_walks=5, zero_V=False):
    rng = np.random.default_rng(seed)
    U = rng.normal(0, 0.5, size=(n, d))
    V = np.zeros((n, d)) if zero_V else rng.normal(0, 0.5, size=(n, d))
    walks = rng.integers(0, n, size=(n_walks, L)).astype(np.int32)
    walks[-1, 3:] = -1
    thr, alias = O.build_alias(rng.random(n) + 0.1, 0.75)
    c, o, ng, n_pairs = O.expand_lists(walks, 7, w, K, thr, alias, seed=seed)
    # force some masked negatives (negative == context)
    idx = np.flatnonzero(c >= 0)[::5]
    ng[idx, 0] = o[idx]
    return U, V, c, o, ng, n_pairs


def torch_loss(U, V, c, o, ng):
    """Textbook form: binary cross-entropy with logits, label 1 for the context and 0 for
    each unmasked negative, summed (library routine, independent of the oracle's code)."""
    Ut = torch.tensor(U, requires_grad=True)
    Vt = torch.tensor(V, requires_grad=True)
    sel = np.flatnonzero(c >= 0)
    cc = torch.tensor(c[sel].astype(np.int64))
    oo = torch.tensor(o[sel].astype(np.int64))
    nn_ = torch.tensor(ng[sel].astype(np.int64))
    pos = (Ut[cc] * Vt[oo]).sum(-1)
    neg = (Ut[cc][:, None, :] * Vt[nn_]).sum(-1)
    bce = torch.nn.functional.binary_cross_entropy_with_logits
    lp = bce(pos, torch.ones_like(pos), reduction="sum")
    ln = bce(neg, torch.zeros_like(neg), reduction="none")
    ln = (ln * (nn_ != oo[:, None])).sum()
    return Ut, Vt, lp + ln


def test_sgns_loss_and_gradients_match_library_cross_entropy():
    U, V, c, o, ng, n_pairs = small_problem(1)
    Ut, Vt, loss = torch_loss(U, V, c, o, ng)
    loss.backward()
    assert abs(O.sgns_loss_from_lists(U, V, c, o, ng) - loss.item()) < 1e-10 * abs(loss.item())
    U1, V1 = U.copy(), V.copy()
    lr = 0.05
    ls, pc = O.sgns_det_from_lists(U1, V1, c, o, ng, lr)
    assert pc == n_pairs and abs(ls - loss.item()) < 1e-10 * abs(ls)
    assert np.allclose((U - U1) / lr, Ut.grad.numpy(), atol=1e-11)
    assert np.allclose((V - V1) / lr, Vt.grad.numpy(), atol=1e-11)


def test_sgns_gradients_match_central_finite_differences():
    U, V, c, o, ng, _ = small_problem(2)
    lr = 1.0
    U1, V1 = U.copy(), V.copy()
    O.sgns_det_from_lists(U1, V1, c, o, ng, lr)
    GU, GV = U - U1, V - V1
    rng = np.random.default_rng(0)
    h = 1e-6
    for tab, G, which in ((U, GU, 0), (V, GV, 1)):
        for _ in range(40):
            r, j = rng.integers(0, tab.shape[0]), rng.integers(0, tab.shape[1])
            plus, minus = tab.copy(), tab.copy()
            plus[r, j] += h
            minus[r, j] -= h
            a = (plus, V) if which == 0 else (U, plus)
            b = (minus, V) if which == 0 else (U, minus)
            fd = (O.sgns_loss_from_lists(*a, c, o, ng) - O.sgns_loss_from_lists(*b, c, o, ng)) / (2 * h)
            assert abs(fd - G[r, j]) < 1e-6 * max(1.0, abs(fd)), (which, r, j, fd, G[r, j])
    assert np.abs(GU).max() > 1e-3 and np.abs(GV).max() > 1e-3


def test_first_step_from_zero_output_vectors_has_closed_form():
    # With V = 0 every sigmoid is 1/2: U stays, V[r] = lr/2 (sum over contexts - sum over
    # unmasked negatives of the center vectors), and each term of the loss is ln 2.
    U, V, c, o, ng, n_pairs = small_problem(3, zero_V=True)
    lr = 0.025
    U1, V1 = U.copy(), V.copy()
    ls, pc = O.sgns_det_from_lists(U1, V1, c, o, ng, lr)
    sel = c >= 0
    unmasked = (ng[sel] != o[sel][:, None])
    assert abs(ls - (pc + unmasked.sum()) * np.log(2.0)) < 1e-9
    assert np.array_equal(U1, U)
    want = np.zeros_like(V)
    np.add.at(want, o[sel], 0.5 * lr * U[c[sel]])
    for k in range(ng.shape[1]):
        m = unmasked[:, k]
        np.subtract.at(want, ng[sel][m, k], 0.5 * lr * U[c[sel][m]])
    assert np.allclose(V1, want, atol=1e-14)
    assert (~unmasked).sum() > 0


def test_synchronous_step_does_not_depend_on_pair_order():
    U, V, c, o, ng, _ = small_problem(4, n_walks=12)
    Ua, Va, Ub, Vb = U.copy(), V.copy(), U.copy(), V.copy()
    la, _ = O.sgns_det_from_lists(Ua, Va, c, o, ng, 0.1)
    order = np.random.default_rng(1).permutation(len(c))
    lb, _ = O.sgns_det_from_lists(Ub, Vb, c, o, ng, 0.1, order=order)
    assert np.abs(Ua - Ub).max() < 1e-12 and np.abs(Va - Vb).max() < 1e-12
    assert abs(la - lb) < 1e-10


def test_sequential_mode_equals_synchronous_when_rows_are_touched_once():
    rng = np.random.default_rng(6)
    U, V = rng.normal(size=(10, 4)), rng.normal(size=(10, 4))
    c = np.array([1, -1], dtype=np.int32)
    o = np.array([2, -1], dtype=np.int32)
    ng = np.array([[3, 4, 2], [-1, -1, -1]], dtype=np.int32)     # third one is masked
    Ua, Va, Ub, Vb = U.copy(), V.copy(), U.copy(), V.copy()
    la, pa = O.sgns_det_from_lists(Ua, Va, c, o, ng, 0.3)
    lb, pb = O.sgns_seq_from_lists(Ub, Vb, c, o, ng, 2, 0.3)
    assert pa == pb == 1 and abs(la - lb) < 1e-14
    assert np.allclose(Ua, Ub, atol=1e-15) and np.allclose(Va, Vb, atol=1e-15)
    assert not np.array_equal(Va[3], V[3]) and np.array_equal(Va[5], V[5])


def test_sequential_mode_sees_earlier_updates():
    rng = np.random.default_rng(7)
    U, V = rng.normal(size=(6, 4)), rng.normal(size=(6, 4))
    # two positions, same context row: the second must use the row the first one wrote
    c = np.array([1, 0], dtype=np.int32)
    o = np.array([2, 2], dtype=np.int32)
    ng = np.full((2, 1), -1, dtype=np.int32)
    Ub, Vb = U.copy(), V.copy()
    O.sgns_seq_from_lists(Ub, Vb, c, o, ng, 1, 0.5)
    sig = lambda x: 1 / (1 + np.exp(-x))
    v1 = V[2] - 0.5 * (sig(U[1] @ V[2]) - 1) * U[1]
    v2 = v1 - 0.5 * (sig(U[0] @ v1) - 1) * U[0]
    assert np.allclose(Vb[2], v2, atol=1e-14)


# ---------------------------------------------------------------- momentum
def test_gradient_function_agrees_with_the_synchronous_step():
    U, V, c, o, ng, n_pairs = small_problem(8)
    GU, GV, loss, cnt = O.sgns_grad_from_lists(U, V, c, o, ng)
    U1, V1 = U.copy(), V.copy()
    l1, c1 = O.sgns_det_from_lists(U1, V1, c, o, ng, 0.5)
    assert cnt == c1 == n_pairs and abs(loss - l1) < 1e-12 * abs(l1)
    assert np.allclose((U - U1) / 0.5, GU, atol=1e-13) and np.allclose((V - V1) / 0.5, GV, atol=1e-13)


def test_momentum_update_matches_library_sgd_and_closed_forms():
    rng = np.random.default_rng(9)
    x0 = rng.normal(size=(7, 5))
    grads = [rng.normal(size=(7, 5)) * (rng.random((7, 1)) < 0.5) for _ in range(6)]   # sparse rows
    lr, mu = 0.05, 0.9
    # library routine: torch.optim.SGD(momentum) is buf <- mu buf + g ; p <- p - lr buf
    p = torch.tensor(x0.copy(), requires_grad=True)
    opt = torch.optim.SGD([p], lr=lr, momentum=mu)
    x, m = x0.copy(), np.zeros_like(x0)
    for g in grads:
        p.grad = torch.tensor(g)
        opt.step()
        O.momentum_update(x, m, np.ascontiguousarray(g), lr, mu)
        assert np.allclose(x, p.detach().numpy(), atol=1e-14)
    # mu = 0 is plain SGD
    x, m = x0.copy(), np.zeros_like(x0)
    O.momentum_update(x, m, grads[0], lr, 0.0)
    assert np.allclose(x, x0 - lr * grads[0], atol=1e-15)
    # one impulse, then k iterations without gradient: geometric series
    x, m = x0.copy(), np.zeros_like(x0)
    O.momentum_update(x, m, grads[1], lr, mu)
    zero = np.zeros_like(x0)
    for _ in range(4):
        O.momentum_update(x, m, zero, lr, mu)
    assert np.allclose(x, x0 - lr * grads[1] * (1 - mu ** 5) / (1 - mu), atol=1e-13)
    assert np.allclose(m, grads[1] * mu ** 4, atol=1e-14)


def test_momentum_step_with_zero_momentum_is_the_synchronous_step():
    U, V, c, o, ng, _ = small_problem(10)
    Ua, Va, Ub, Vb = U.copy(), V.copy(), U.copy(), V.copy()
    la, ca = O.sgns_det_from_lists(Ua, Va, c, o, ng, 0.1)
    lb, cb = O.sgns_momentum_step_from_lists(Ub, Vb, np.zeros_like(U), np.zeros_like(V), c, o, ng, 0.1, 0.0)
    assert ca == cb and abs(la - lb) < 1e-12
    assert np.allclose(Ua, Ub, atol=1e-14) and np.allclose(Va, Vb, atol=1e-14)


# ---------------------------------------------------------------- half-precision storage
def test_binary16_rounding_matches_library_conversion_and_ties_to_even():
    rng = np.random.default_rng(11)
    x = np.concatenate([rng.normal(size=5000), rng.normal(size=5000) * 1e-3, [0.0, 65504.0, -65504.0]])
    # exact ties: midpoints between neighbouring binary16 values
    h = np.float16(0.3).astype(np.float64)
    nxt = np.nextafter(np.float16(0.3), np.float16(1.0)).astype(np.float64)
    x = np.concatenate([x, [(h + nxt) / 2, 1.0 + 2.0 ** -11, 1.0 + 3 * 2.0 ** -11]])
    got = O.round_f16(x.copy())
    assert np.array_equal(got, x.astype(np.float16).astype(np.float64))     # numpy: IEEE RN-even
    assert got[-2] == 1.0 and got[-1] == 1.0 + 2.0 ** -9                      # ties go to even


def test_bfloat16_rounding_matches_library_conversion_and_ties_to_even():
    rng = np.random.default_rng(13)
    # fp32-representable inputs, so that the library's float -> bfloat16 conversion is ONE rounding
    x = np.concatenate([rng.normal(size=5000), rng.normal(size=5000) * 1e-3, rng.normal(size=2000) * 1e30,
                        rng.normal(size=2000) * 1e-39, [0.0, -0.0, 3.3895313892515355e38, 1e-45]])
    x = x.astype(np.float32).astype(np.float64)
    got = O.round_bf16(x.copy())
    want = torch.from_numpy(x.astype(np.float32)).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(got, want)
    # ties: 1 + 2^-8 lies midway between 1 and 1 + 2^-7 and goes to the even neighbour; 1 + 3*2^-8
    # lies midway between 1 + 2^-7 and 1 + 2^-6 and goes up to the even one
    t = O.round_bf16(np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -40]))
    assert t[0] == 1.0 and t[1] == 1.0 + 2.0 ** -6 and t[2] == 1.0 + 2.0 ** -7
    # a value that a detour over fp32 would round twice: just above a bfloat16 midpoint by less than
    # half an fp32 ulp
    v = 1.0 + 2.0 ** -8 + 2.0 ** -30
    assert O.round_bf16(np.array([v]))[0] == 1.0 + 2.0 ** -7
    assert np.float64(np.float32(v)) == 1.0 + 2.0 ** -8            # fp32 first would land on the tie
    assert np.isinf(O.round_bf16(np.array([3.4e38]))[0])


def test_bfloat16_sequential_step_reduces_to_full_precision_plus_rounding():
    rng = np.random.default_rng(14)
    U = O.round_bf16(rng.normal(size=(8, 4)))
    V = O.round_bf16(rng.normal(size=(8, 4)))
    c = np.array([1], dtype=np.int32)
    o = np.array([2], dtype=np.int32)
    ng = np.array([[3, 4]], dtype=np.int32)
    Ua, Va, Ub, Vb = U.copy(), V.copy(), U.copy(), V.copy()
    O.sgns_seq_from_lists(Ua, Va, c, o, ng, 1, 0.3)
    O.sgns_seq_bf16_from_lists(Ub, Vb, c, o, ng, 1, 0.3)
    assert np.array_equal(Ub, O.round_bf16(Ua)) and np.array_equal(Vb, O.round_bf16(Va))
    assert not np.array_equal(Vb, V)


def test_half_precision_sequential_step_reduces_to_full_precision_plus_rounding():
    # one pair, rows touched once: the f16 result is the rounded full-precision result
    rng = np.random.default_rng(12)
    U = O.round_f16(rng.normal(size=(8, 4)))
    V = O.round_f16(rng.normal(size=(8, 4)))
    c = np.array([1], dtype=np.int32)
    o = np.array([2], dtype=np.int32)
    ng = np.array([[3, 4]], dtype=np.int32)
    Ua, Va, Ub, Vb = U.copy(), V.copy(), U.copy(), V.copy()
    O.sgns_seq_from_lists(Ua, Va, c, o, ng, 1, 0.3)
    O.sgns_seq_f16_from_lists(Ub, Vb, c, o, ng, 1, 0.3)
    assert np.array_equal(Ub, O.round_f16(Ua)) and np.array_equal(Vb, O.round_f16(Va))
    assert not np.array_equal(Vb, V)


# ---------------------------------------------------------------- initialisation
def test_initial_rows_are_uniform_and_exact_in_single_precision():
    rows = np.arange(0, 4000, dtype=np.int64) * 12345
    d = 64
    U = O.init_rows(rows, d, seed=0)
    assert U.min() >= -0.5 / d and U.max() < 0.5 / d
    assert np.array_equal(U.astype(np.float32).astype(np.float64), U)
    ok, stat = chi2_ok(np.histogram(U.ravel(), bins=32, range=(-0.5 / d, 0.5 / d))[0],
                       np.full(32, 1 / 32))
    assert ok, stat
    assert abs(np.corrcoef(U[:, :-1].ravel(), U[:, 1:].ravel())[0, 1]) < 0.01
    again = O.init_rows(rows[100:110], d, seed=0)
    assert np.array_equal(again, U[100:110])
    assert not np.array_equal(O.init_rows(rows[:4], d, seed=1), U[:4])


# ---------------------------------------------------------------- epoch
def test_epoch_on_tiny_workload_starts_at_ln2_scale_and_decreases():
    wl = WL.WORKLOADS["tiny_deepwalk"]
    g = wl.make_graph(scale=0.2)
    off, col = np_graph(g)
    n = g.n_nodes
    thr, alias = O.build_alias((off[1:] - off[:-1]).astype(np.float64), 0.75)
    U = O.init_rows(np.arange(n), wl.dim, seed=0)
    V = np.zeros_like(U)
    kw = dict(walks_per_node=1, L=wl.walk_len, w=wl.window, K=wl.n_neg, lr0=wl.lr0,
              schedule="linear", batch_walks=500, seed=0)
    first = O.sgns_epoch(off, col, thr, alias, U.copy(), V.copy(), num_batches=1, **kw)
    per_pair = first["loss_sum"] / first["pairs"]
    assert (1 + wl.n_neg - 0.05) * np.log(2) < per_pair <= (1 + wl.n_neg) * np.log(2) + 1e-12
    # resuming at a batch boundary reproduces the uninterrupted run
    Ua, Va = U.copy(), V.copy()
    full = O.sgns_epoch(off, col, thr, alias, Ua, Va, **kw)
    Ub, Vb = U.copy(), V.copy()
    h1 = O.sgns_epoch(off, col, thr, alias, Ub, Vb, first_batch=0, num_batches=2, **kw)
    h2 = O.sgns_epoch(off, col, thr, alias, Ub, Vb, first_batch=2, **kw)
    assert np.array_equal(Ua, Ub) and np.array_equal(Va, Vb)
    assert abs(full["loss_sum"] - h1["loss_sum"] - h2["loss_sum"]) < 1e-9
    assert full["pairs"] == h1["pairs"] + h2["pairs"]
    # a second epoch over the same walks has lower loss
    again = O.sgns_epoch(off, col, thr, alias, Ua, Va, **kw)
    assert again["loss_sum"] < full["loss_sum"]
