"""GPU parity: the CUDA library (through the C ABI) against the CPU oracle on the same
seeded inputs.  Integer outputs (walks, pairs, negative draws, counts) must be bit-exact;
embeddings after one synchronous step within 1e-4 absolute of the fp64 oracle; epoch loss
within 1e-3 relative."""
import numpy as np
import pytest
import torch

from oracle import gs_oracle as O
from paper_2407_15452_b200 import binding as B
from paper_2407_15452_b200 import workloads as WL
from tests.helpers import alias_to_device, compact_problem, degree_alias, np_graph

pytestmark = pytest.mark.gpu

EMB_TOL = 1e-4        # max |delta| after one synchronous step (fp32 kernels vs fp64 oracle)
LOSS_RTOL = 1e-3      # mean epoch loss
DEV = "cuda"


@pytest.fixture(scope="module")
def tiny():
    wl = WL.WORKLOADS["tiny_deepwalk"]
    g = wl.make_graph()
    off, col = np_graph(g)
    thr, alias = degree_alias(off)
    return wl, g, off, col, thr, alias


def load(g, offsets64=False, flags=B.GS_VALIDATE | B.GS_REQUIRE_SORTED):
    off = g.offsets.to(torch.int64 if offsets64 else torch.int32).to(DEV)
    return B.gs_graph_load_csr(off, g.cols.to(DEV), flags)


# ---------------------------------------------------------------- graph loading
def test_graph_validation_reports_errors(tiny):
    _, g, off, col, _, _ = tiny
    G = load(g)
    info = G.info()
    assert info["n_nodes"] == g.n_nodes and info["n_edges"] == g.n_edges
    assert info["max_degree"] == int((off[1:] - off[:-1]).max()) and info["rows_sorted"]
    # unsorted row
    bad = g.cols.clone()
    v = int(np.flatnonzero((off[1:] - off[:-1]) >= 2)[5])
    a = int(off[v])
    bad[a], bad[a + 1] = g.cols[a + 1].item(), g.cols[a].item()
    with pytest.raises(B.GsError) as e:
        B.gs_graph_load_csr(g.offsets.to(DEV), bad.to(DEV), B.GS_VALIDATE | B.GS_REQUIRE_SORTED)
    assert e.value.status == -3 and f"row {v} " in str(e.value)
    B.gs_graph_load_csr(g.offsets.to(DEV), bad.to(DEV), B.GS_VALIDATE).close()   # fine unsorted
    # column out of range
    bad = g.cols.clone()
    bad[a] = g.n_nodes
    with pytest.raises(B.GsError) as e:
        B.gs_graph_load_csr(g.offsets.to(DEV), bad.to(DEV), B.GS_VALIDATE)
    assert e.value.status == -2 and f"row {v} " in str(e.value)
    # decreasing offsets, wrong end
    boff = g.offsets.clone()
    boff[v + 1] = boff[v] - 1
    with pytest.raises(B.GsError) as e:
        B.gs_graph_load_csr(boff.to(DEV), g.cols.to(DEV), B.GS_VALIDATE)
    assert e.value.status == -2
    boff = g.offsets.clone()
    boff[-1] -= 1
    with pytest.raises(B.GsError) as e:
        B.gs_graph_load_csr(boff.to(DEV), g.cols.to(DEV), B.GS_VALIDATE)
    assert e.value.status == -2
    # node2vec refuses a graph whose rows were not verified
    G2 = load(g, flags=B.GS_VALIDATE)
    with pytest.raises(B.GsError) as e:
        B.gs_node2vec_walks(G2, None, 4, 0, 5, 0, 0.5, 2.0)
    assert e.value.status == -3


# ---------------------------------------------------------------- walks
@pytest.mark.parametrize("offsets64", [False, True])
def test_uniform_walks_bit_exact(tiny, offsets64):
    wl, g, off, col, _, _ = tiny
    G = load(g, offsets64)
    n = g.n_nodes
    steps = torch.zeros(1, dtype=torch.int64, device=DEV)
    # ragged count (not a multiple of the block size), ids continue past one repetition
    got = B.gs_random_walks(G, None, 2 * n + 77, 123, wl.walk_len, 0, steps=steps)
    want, st = O.uniform_walks(off, col, None, 2 * n + 77, 123, wl.walk_len, 0)
    assert np.array_equal(got.cpu().numpy(), want)
    assert int(steps.item()) == st
    # explicit start nodes, another seed, long walks
    rng = np.random.default_rng(1)
    starts = rng.integers(0, n, size=3001).astype(np.int32)
    got = B.gs_random_walks(G, torch.from_numpy(starts).to(DEV), 3001, 5_000_000_000, 80,
                            0xDEADBEEFCAFEF00D)
    want, _ = O.uniform_walks(off, col, starts, 3001, 5_000_000_000, 80, 0xDEADBEEFCAFEF00D)
    assert np.array_equal(got.cpu().numpy(), want)


@pytest.mark.parametrize("offsets64", [False, True])
def test_uniform_walks_over_the_walk_index_are_the_same_walks(tiny, offsets64):
    wl, g, off, col, _, _ = tiny
    G = load(g, offsets64, flags=B.GS_BUILD_WALK_INDEX)
    steps = torch.zeros(1, dtype=torch.int64, device=DEV)
    got = B.gs_random_walks(G, None, 20011, 999, 40, 17, steps=steps)
    want, st = O.uniform_walks(off, col, None, 20011, 999, 40, 17)
    assert np.array_equal(got.cpu().numpy(), want) and int(steps.item()) == st
    # odd walk length: falls back to the scalar path, same result
    got = B.gs_random_walks(G, None, 777, 5, 13, 17)
    want, _ = O.uniform_walks(off, col, None, 777, 5, 13, 17)
    assert np.array_equal(got.cpu().numpy(), want)
    G.close()
    # directed graph with dead ends
    g2 = WL.rmat_graph(3000, 9000, seed=5)
    off2, col2 = np_graph(g2)
    G2 = load(g2, offsets64, flags=B.GS_BUILD_WALK_INDEX)
    starts = np.random.default_rng(3).integers(0, 3000, 5000).astype(np.int32)
    got = B.gs_random_walks(G2, torch.from_numpy(starts).to(DEV), 5000, 0, 24, 9)
    want, _ = O.uniform_walks(off2, col2, starts, 5000, 0, 24, 9)
    assert (want == -1).any() and np.array_equal(got.cpu().numpy(), want)


def test_uniform_walks_dead_ends_and_degenerate_sizes():
    g = WL.rmat_graph(3000, 9000, seed=5)           # directed: dead ends
    off, col = np_graph(g)
    G = load(g, offsets64=True, flags=B.GS_VALIDATE)
    got = B.gs_random_walks(G, None, 6000, 0, 20, 9)
    want, _ = O.uniform_walks(off, col, None, 6000, 0, 20, 9)
    assert (want == -1).any() and np.array_equal(got.cpu().numpy(), want)
    assert B.gs_random_walks(G, None, 0, 0, 20, 9).shape == (0, 20)
    got = B.gs_random_walks(G, None, 10, 0, 1, 9)                      # length 1: just the start
    assert np.array_equal(got.cpu().numpy()[:, 0], np.arange(10))


@pytest.mark.parametrize("p,q,max_rounds", [(0.5, 2.0, 1024), (4.0, 0.25, 1024), (1.0, 1.0, 1024),
                                             (0.5, 2.0, 3), (100.0, 100.0, 1), (0.5, 2.0, 37)])
def test_node2vec_walks_bit_exact_for_every_group_width(tiny, p, q, max_rounds):
    _, g, off, col, _, _ = tiny
    # with the walk index when the cap is the default, without it otherwise: both paths covered
    G = load(g, flags=B.GS_VALIDATE | B.GS_REQUIRE_SORTED | (B.GS_BUILD_WALK_INDEX if max_rounds == 1024 else 0))
    n_walks, L = 5003, 24
    want, st, caps = O.node2vec_walks(off, col, None, n_walks, 77, L, 5, p, q, max_rounds)
    try:
        for lanes in (0, 1, 2, 4, 8, 32):
            B.gs_tune_node2vec_group(lanes)
            steps = torch.zeros(1, dtype=torch.int64, device=DEV)
            hits = torch.zeros(1, dtype=torch.int64, device=DEV)
            got = B.gs_node2vec_walks(G, None, n_walks, 77, L, 5, p, q, max_rounds, steps=steps,
                                      cap_hits=hits)
            assert np.array_equal(got.cpu().numpy(), want), lanes
            assert int(steps.item()) == st and int(hits.item()) == caps, lanes
    finally:
        B.gs_tune_node2vec_group(0)
    if max_rounds <= 3:
        assert caps > 0


def test_node2vec_on_directed_graph_with_dead_ends_and_int64_offsets():
    g = WL.rmat_graph(3000, 12000, seed=6)
    off, col = np_graph(g)
    G = load(g, offsets64=True)
    rng = np.random.default_rng(2)
    starts = rng.integers(0, 3000, size=4000).astype(np.int32)
    want, _, _ = O.node2vec_walks(off, col, starts, 4000, 0, 30, 11, 0.25, 4.0)
    got = B.gs_node2vec_walks(G, torch.from_numpy(starts).to(DEV), 4000, 0, 30, 11, 0.25, 4.0)
    assert np.array_equal(got.cpu().numpy(), want)
    # one walk per thread, over the walk index and without it, walk length a multiple of 4
    want, _, _ = O.node2vec_walks(off, col, starts, 4000, 9, 32, 12, 0.25, 4.0)
    for flags in (3, 7, 3 | B.GS_BUILD_EDGE_SET, 7 | B.GS_BUILD_EDGE_SET):      # edge set: hashed membership test
        for o64 in (True, False):
            G2 = load(g, offsets64=o64, flags=flags)
            for lanes in (0, 1):                       # flattened loop, nested loops
                B.gs_tune_node2vec_group(lanes)
                got = B.gs_node2vec_walks(G2, torch.from_numpy(starts).to(DEV), 4000, 9, 32, 12, 0.25, 4.0)
                assert np.array_equal(got.cpu().numpy(), want), (flags, o64, lanes)
                for L in (4, 12, 36):                  # 8m + 4 entries: the tail store of the flat kernel
                    w2, _, _ = O.node2vec_walks(off, col, starts[:500], 500, 3, L, 12, 0.25, 4.0)
                    g2 = B.gs_node2vec_walks(G2, torch.from_numpy(starts[:500].copy()).to(DEV), 500, 3, L, 12,
                                             0.25, 4.0)
                    assert np.array_equal(g2.cpu().numpy(), w2), (flags, o64, lanes, L)
    B.gs_tune_node2vec_group(0)


@pytest.mark.parametrize("p,q", [(0.5, 2.0), (4.0, 0.25), (2.0, 0.5)])
def test_node2vec_with_the_edge_set_is_bit_exact_on_the_power_law_graph(tiny, p, q):
    # hubs with thousands of neighbours and many triangles: every class of candidate occurs
    _, g, off, col, _, _ = tiny
    G = load(g, flags=B.GS_REQUIRE_SORTED | B.GS_BUILD_WALK_INDEX | B.GS_BUILD_EDGE_SET)
    want, st, caps = O.node2vec_walks(off, col, None, 20000, 5, 40, 21, p, q)
    for lanes in (0, 1):
        B.gs_tune_node2vec_group(lanes)
        steps = torch.zeros(1, dtype=torch.int64, device=DEV)
        got = B.gs_node2vec_walks(G, None, 20000, 5, 40, 21, p, q, steps=steps)
        assert np.array_equal(got.cpu().numpy(), want) and int(steps.item()) == st
    B.gs_tune_node2vec_group(0)


# ---------------------------------------------------------------- initialisation
@pytest.mark.parametrize("dim", [32, 64, 128, 256])
def test_initial_tables_equal_oracle_exactly(dim):
    n = 5000
    w_in = torch.empty((n, dim), dtype=torch.float32, device=DEV)
    w_out = torch.full((n, dim), 7.0, dtype=torch.float32, device=DEV)
    B.gs_init_embeddings(w_in, w_out, seed=42)
    want = O.init_rows(np.arange(n), dim, 42)
    assert np.array_equal(w_in.cpu().numpy().astype(np.float64), want)
    assert not w_out.any()


# ---------------------------------------------------------------- SGNS step
def run_step(w_in, w_out, walks, base, w, K, alias_dev, lr, seed, mode, dump=True):
    n_walks, L = walks.shape
    loss = torch.zeros(1, dtype=torch.float64, device=DEV)
    cnt = torch.zeros(1, dtype=torch.int64, device=DEV)
    pd = nd = None
    if dump:
        pd = torch.full((n_walks, L, 2 * w, 2), -7, dtype=torch.int32, device=DEV)
        nd = torch.full((n_walks, L, 2 * w, max(K, 1)), -7, dtype=torch.int32, device=DEV)[..., :K].contiguous()
    B.gs_sgns_step(w_in, w_out, walks, base, w, K, alias_dev, lr, seed, mode, loss, cnt, pd, nd)
    torch.cuda.synchronize()
    return loss.item(), cnt.item(), pd, nd


def oracle_step(U0, V0, walks, base, w, K, thr, alias, lr, seed):
    c, o, ng, n_pairs = O.expand_lists(walks, base, w, K, thr, alias, seed)
    U, V = U0.astype(np.float64), V0.astype(np.float64)
    loss, cnt = O.sgns_det_from_lists(U, V, c, o, ng, lr)
    return U, V, loss, cnt, c, o, ng


def random_tables(n, dim, seed, scale=0.3):
    gen = torch.Generator().manual_seed(seed)
    w_in = (torch.rand((n, dim), generator=gen) - 0.5) * scale
    w_out = (torch.rand((n, dim), generator=gen) - 0.5) * scale
    return w_in, w_out


@pytest.mark.parametrize("dim,L,w,K", [(64, 10, 5, 5), (128, 40, 10, 5), (32, 7, 3, 4),
                                        (256, 12, 2, 1), (128, 6, 8, 10), (64, 9, 4, 0)])
def test_deterministic_step_matches_oracle(tiny, dim, L, w, K):
    _, g, off, col, thr, alias = tiny
    n = g.n_nodes
    n_walks = 301                                      # several blocks and a ragged tail
    walks, _ = O.uniform_walks(off, col, None, n_walks, 50, L, 3)
    walks[5, L // 2:] = -1                             # a walk that stopped early
    walks[6, :] = -1
    w_in0, w_out0 = random_tables(n, dim, 1)
    U, V, loss_o, cnt_o, c, o, ng = oracle_step(w_in0.numpy(), w_out0.numpy(), walks, 50, w, K,
                                                thr, alias, 0.025, 3)
    a_dev = alias_to_device(thr, alias)
    w_in, w_out = w_in0.to(DEV), w_out0.to(DEV)
    loss, cnt, pd, nd = run_step(w_in, w_out, torch.from_numpy(walks).to(DEV), 50, w, K, a_dev,
                                 0.025, 3, B.GS_DETERMINISTIC)
    # integer work: pairs and negative draws bit-exact
    pd = pd.cpu().numpy().reshape(-1, 2)
    assert np.array_equal(pd[:, 0], c) and np.array_equal(pd[:, 1], o)
    if K > 0:
        assert np.array_equal(nd.cpu().numpy().reshape(-1, K), ng)
    assert cnt == cnt_o
    assert abs(loss - loss_o) <= 2e-6 * abs(loss_o)
    assert np.abs(w_in.cpu().numpy() - U).max() <= EMB_TOL
    assert np.abs(w_out.cpu().numpy() - V).max() <= EMB_TOL
    # and the step really moved the tables by much more than the tolerance
    assert np.abs(V - w_out0.numpy()).max() > 20 * EMB_TOL
    # bitwise reproducible
    w_in2, w_out2 = w_in0.to(DEV), w_out0.to(DEV)
    loss2, _, _, _ = run_step(w_in2, w_out2, torch.from_numpy(walks).to(DEV), 50, w, K, a_dev,
                              0.025, 3, B.GS_DETERMINISTIC, dump=False)
    assert torch.equal(w_in, w_in2) and torch.equal(w_out, w_out2) and loss == loss2


@pytest.mark.parametrize("L,w,K,dim", [(2, 1, 5, 128), (9, 3, 2, 64)])
def test_forward_only_pairs_line_shape(tiny, L, w, K, dim):
    # LINE: walks of two nodes, window 1, forward pairs only -> one (source, neighbour) pair per walk
    _, g, off, col, thr, alias = tiny
    n = g.n_nodes
    walks, _ = O.uniform_walks(off, col, None, 1500, 0, L, 4)
    c, o, ng, n_pairs = O.expand_lists(walks, 0, w, K, thr, alias, 4, forward_only=True)
    if L == 2:
        assert n_pairs == int((walks[:, 1] >= 0).sum())
    w_in0, w_out0 = random_tables(n, dim, 7)
    U, V = w_in0.numpy().astype(np.float64), w_out0.numpy().astype(np.float64)
    loss_o, cnt_o = O.sgns_det_from_lists(U, V, c, o, ng, 0.025)
    a_dev = alias_to_device(thr, alias)
    wd = torch.from_numpy(walks).to(DEV)
    for mode in (B.GS_DETERMINISTIC, B.GS_HOGWILD):
        w_in, w_out = w_in0.to(DEV), w_out0.to(DEV)
        loss, cnt, pd, nd = run_step(w_in, w_out, wd, 0, w, K, a_dev, 0.025, 4,
                                     mode | B.GS_PAIRS_FORWARD_ONLY)
        pd = pd.cpu().numpy().reshape(-1, 2)
        assert np.array_equal(pd[:, 0], c) and np.array_equal(pd[:, 1], o)
        assert np.array_equal(nd.cpu().numpy().reshape(-1, K), ng)
        assert cnt == cnt_o == n_pairs
        if mode == B.GS_DETERMINISTIC:
            assert abs(loss - loss_o) <= 2e-6 * abs(loss_o)
            assert np.abs(w_in.cpu().numpy() - U).max() <= EMB_TOL
            assert np.abs(w_out.cpu().numpy() - V).max() <= EMB_TOL


@pytest.mark.parametrize("dim,L,w,K,n_walks", [(128, 1024, 32, 7, 3),     # longest walk, 512 targets per position
                                                 (64, 40, 7, 32, 9),        # most negatives
                                                 (32, 5, 32, 0, 70),        # window wider than the walk, no negatives
                                                 (256, 1, 1, 3, 50)])       # walks of one node: no pairs at all
def test_limits_of_the_supported_shapes(tiny, dim, L, w, K, n_walks):
    _, g, off, col, thr, alias = tiny
    n = g.n_nodes
    walks, _ = O.uniform_walks(off, col, None, n_walks, 0, L, 6)
    c, o, ng, n_pairs = O.expand_lists(walks, 0, w, K, thr, alias, 6)
    w_in0, w_out0 = random_tables(n, dim, 11, scale=0.2)
    U, V = w_in0.numpy().astype(np.float64), w_out0.numpy().astype(np.float64)
    loss_o, cnt_o = O.sgns_det_from_lists(U, V, c, o, ng, 0.01)
    a_dev = alias_to_device(thr, alias)
    wd = torch.from_numpy(walks).to(DEV)
    for mode in (B.GS_DETERMINISTIC, B.GS_HOGWILD, B.GS_HOGWILD_RED):
        w_in, w_out = w_in0.to(DEV), w_out0.to(DEV)
        loss, cnt, pd, nd = run_step(w_in, w_out, wd, 0, w, K, a_dev, 0.01, 6, mode)
        pd = pd.cpu().numpy().reshape(-1, 2)
        assert np.array_equal(pd[:, 0], c) and np.array_equal(pd[:, 1], o)
        if K > 0:
            assert np.array_equal(nd.cpu().numpy().reshape(-1, K), ng)
        assert cnt == cnt_o == n_pairs
        if mode == B.GS_DETERMINISTIC:
            assert abs(loss - loss_o) <= 2e-6 * max(abs(loss_o), 1e-30)
            assert np.abs(w_in.cpu().numpy() - U).max() <= EMB_TOL
            assert np.abs(w_out.cpu().numpy() - V).max() <= EMB_TOL
        else:
            assert torch.isfinite(w_in).all() and torch.isfinite(w_out).all()
    if L == 1:
        assert n_pairs == 0
    # one past each limit is refused
    for bad in (dict(window=33), dict(n_neg=33), dict(window=32, n_neg=8)):
        kw = dict(window=2, n_neg=2)
        kw.update(bad)
        with pytest.raises(B.GsError) as e:
            B.gs_sgns_step(w_in, w_out, wd, 0, kw["window"], kw["n_neg"], a_dev, 0.01, 6, B.GS_HOGWILD)
        assert e.value.status == -6


@pytest.mark.parametrize("dim", [32, 64, 128, 256])
def test_deterministic_step_where_most_output_rows_receive_one_contribution(dim):
    # 300,000 rows and a batch of 40 short walks: the tables have far more rows than the batch has
    # list entries, the regime of large graphs, in which the step adds the increment of a row that
    # receives a single contribution straight from the coefficient pass.  The power-law graph makes
    # both kinds of rows occur (hubs collect several contributions).  Oracle on the touched rows.
    wl = WL.WORKLOADS["deepwalk_medium"]
    g = wl.make_graph(scale=0.3)
    n = g.n_nodes
    off, col = np_graph(g)
    thr, alias = degree_alias(off)
    L, w, K, n_walks, base, seed, lr = 10, 3, 4, 40, 12345, 6, 0.05
    walks, _ = O.uniform_walks(off, col, None, n_walks, base, L, seed)
    walks[3, L // 2:] = -1
    c, o, ng, n_pairs = O.expand_lists(walks, base, w, K, thr, alias, seed)
    ids, cc, oo, nn = compact_problem(c, o, ng)
    assert n >= 3 * n_walks * L * 32                   # rows per (padded) list entry: the shortcut is on
    pair_ok = cc >= 0
    hits = np.bincount(oo[pair_ok], minlength=len(ids))
    negs = nn[pair_ok]
    hits += np.bincount(negs[(negs >= 0) & (negs != oo[pair_ok][:, None])], minlength=len(ids))
    assert (hits == 1).sum() > 100 and (hits > 1).sum() > 20 and hits.max() >= 4
    w_in0, w_out0 = random_tables(n, dim, 11)
    U = w_in0[torch.from_numpy(ids)].numpy().astype(np.float64)
    V = w_out0[torch.from_numpy(ids)].numpy().astype(np.float64)
    V0 = V.copy()
    loss_o, cnt_o = O.sgns_det_from_lists(U, V, cc, oo, nn, lr)
    a_dev = alias_to_device(thr, alias)
    w_in, w_out = w_in0.to(DEV), w_out0.to(DEV)
    loss, cnt, pd, nd = run_step(w_in, w_out, torch.from_numpy(walks).to(DEV), base, w, K, a_dev, lr, seed,
                                 B.GS_DETERMINISTIC)
    pd = pd.cpu().numpy().reshape(-1, 2)
    assert np.array_equal(pd[:, 0], c) and np.array_equal(pd[:, 1], o)
    assert np.array_equal(nd.cpu().numpy().reshape(-1, K), ng)
    assert cnt == cnt_o == n_pairs and abs(loss - loss_o) <= 2e-6 * abs(loss_o)
    ids_dev = torch.from_numpy(ids).to(DEV)
    assert np.abs(w_in[ids_dev].cpu().numpy() - U).max() <= EMB_TOL
    got_out = w_out[ids_dev].cpu().numpy()
    assert np.abs(got_out - V).max() <= EMB_TOL
    # every output row that the lists name moved, whether it was hit once or several times, by much
    # more than the tolerance; every row outside the batch kept its bits
    moved = np.abs(V - V0).max(axis=1)
    assert (moved[hits == 1] > 20 * EMB_TOL).all() and (moved[hits > 1] > 20 * EMB_TOL).all()
    assert np.array_equal(np.abs(got_out - V0).max(axis=1) > 0, hits > 0)
    outside = torch.ones(n, dtype=torch.bool)
    outside[torch.from_numpy(ids)] = False
    assert torch.equal(w_in.cpu()[outside], w_in0[outside]) and torch.equal(w_out.cpu()[outside], w_out0[outside])
    # bitwise reproducible, and the allocation-free entry point gives the same bits
    for step in (B.gs_sgns_step, B.gs_sgns_step_static):
        w_in2, w_out2 = w_in0.to(DEV), w_out0.to(DEV)
        if step is B.gs_sgns_step:
            step(w_in2, w_out2, torch.from_numpy(walks).to(DEV), base, w, K, a_dev, lr, seed, B.GS_DETERMINISTIC)
        else:
            step(w_in2, w_out2, torch.from_numpy(walks).to(DEV), base, w, K, a_dev, lr, seed)
        torch.cuda.synchronize()
        assert torch.equal(w_in, w_in2) and torch.equal(w_out, w_out2)


def test_deterministic_step_hub_rows_with_thousands_of_contributions():
    # a star: every walk alternates hub / leaf, so one output row collects most contributions
    n = 400
    leaves = torch.arange(1, n, dtype=torch.int64)
    hub = torch.zeros(n - 1, dtype=torch.int64)
    g = WL._csr_from_directed(torch.cat([hub, leaves]), torch.cat([leaves, hub]), n, False)
    off, col = np_graph(g)
    thr, alias = degree_alias(off)
    walks, _ = O.uniform_walks(off, col, None, 512, 0, 40, 8)
    w_in0, w_out0 = random_tables(n, 128, 2, scale=0.1)
    U, V, loss_o, cnt_o, *_ = oracle_step(w_in0.numpy(), w_out0.numpy(), walks, 0, 5, 5, thr,
                                          alias, 0.001, 8)
    w_in, w_out = w_in0.to(DEV), w_out0.to(DEV)
    loss, cnt, _, _ = run_step(w_in, w_out, torch.from_numpy(walks).to(DEV), 0, 5, 5,
                               alias_to_device(thr, alias), 0.001, 8, B.GS_DETERMINISTIC, dump=False)
    assert cnt == cnt_o and abs(loss - loss_o) <= 2e-6 * abs(loss_o)
    assert np.abs(w_in.cpu().numpy() - U).max() <= EMB_TOL
    assert np.abs(w_out.cpu().numpy() - V).max() <= EMB_TOL


@pytest.mark.parametrize("mode", [B.GS_HOGWILD, B.GS_HOGWILD_RED])
def test_lock_free_modes_draw_the_same_pairs_and_negatives(tiny, mode):
    _, g, off, col, thr, alias = tiny
    L, w, K, dim = 10, 5, 5, 64
    walks, _ = O.uniform_walks(off, col, None, 700, 0, L, 3)
    walks[9, 4:] = -1
    c, o, ng, n_pairs = O.expand_lists(walks, 0, w, K, thr, alias, 3)
    w_in = torch.empty((g.n_nodes, dim), dtype=torch.float32, device=DEV)
    w_out = torch.empty_like(w_in)
    B.gs_init_embeddings(w_in, w_out, 0)
    loss, cnt, pd, nd = run_step(w_in, w_out, torch.from_numpy(walks).to(DEV), 0, w, K,
                                 alias_to_device(thr, alias), 0.025, 3, mode)
    pd = pd.cpu().numpy().reshape(-1, 2)
    assert np.array_equal(pd[:, 0], c) and np.array_equal(pd[:, 1], o)
    assert np.array_equal(nd.cpu().numpy().reshape(-1, K), ng)
    assert cnt == n_pairs
    assert torch.isfinite(w_in).all() and torch.isfinite(w_out).all()
    # from zero output vectors the first terms are ln 2 each; later ones are already smaller
    unmasked = (ng[c >= 0] != o[c >= 0][:, None]).sum()
    assert 0.9 * (cnt + unmasked) * np.log(2) < loss <= (cnt + unmasked) * np.log(2) * (1 + 1e-6)


@pytest.mark.parametrize("dim", [32, 64, 128, 256])
def test_lock_free_single_walk_equals_sequential_oracle(dim):
    # One walk = one warp running its positions in order: no races between warps.  Rows that
    # repeat inside one chunk of targets are the only difference to strictly sequential SGD,
    # so use a walk and negatives without repeats.
    n, L, w, K = 4000, 12, 2, 3
    rng = np.random.default_rng(4)
    walk = rng.permutation(n)[:L].astype(np.int32)[None, :]
    thr, alias = O.build_alias(np.ones(n), 1.0)
    c, o, ng, _ = O.expand_lists(walk, 0, w, K, thr, alias, 12)
    w_in0, w_out0 = random_tables(n, dim, 5)
    U, V = w_in0.numpy().astype(np.float64), w_out0.numpy().astype(np.float64)
    loss_o, cnt_o = O.sgns_seq_from_lists(U, V, c, o, ng, 2 * w, 0.05)
    # rows that occur more than once among the targets of ONE position (a negative drawn twice, or
    # equal to another slot's context): the kernel loads a chunk of targets before it stores any, so
    # such a row - and the center row of that position - may differ from strictly sequential SGD
    S = 2 * w
    repeated, their_centers = set(), set()
    for p0 in range(0, len(c), S):
        targets = []
        for e in range(p0, p0 + S):
            if c[e] >= 0:
                targets.append(int(o[e]))
                targets += [int(t) for t in ng[e] if t >= 0 and t != o[e]]
        dup = {t for t in targets if targets.count(t) > 1}
        if dup:
            repeated |= dup
            their_centers.add(int(c[p0:p0 + S].max()))
    for mode in (B.GS_HOGWILD, B.GS_HOGWILD_RED):
        w_in, w_out = w_in0.to(DEV), w_out0.to(DEV)
        loss, cnt, _, _ = run_step(w_in, w_out, torch.from_numpy(walk).to(DEV), 0, w, K,
                                   alias_to_device(thr, alias), 0.05, 12, mode, dump=False)
        assert cnt == cnt_o and abs(loss - loss_o) < 1e-5 * abs(loss_o)
        diff_in = np.abs(w_in.cpu().numpy() - U).max(axis=1)
        diff_out = np.abs(w_out.cpu().numpy() - V).max(axis=1)
        assert set(np.nonzero(diff_out > 1e-5)[0].tolist()) <= repeated, (repeated, np.nonzero(diff_out > 1e-5))
        assert set(np.nonzero(diff_in > 1e-5)[0].tolist()) <= their_centers
        assert len(repeated) <= 4                      # the case stays almost free of repeats
        assert np.abs(V - w_out0.numpy()).max() > 1e-3


@pytest.mark.parametrize("dim,L,w", [(128, 40, 5), (64, 20, 5), (256, 24, 3), (32, 16, 2), (128, 2, 1)])
def test_lock_free_many_walks_without_shared_rows_equal_sequential_oracle(dim, L, w):
    # Hundreds of walks run concurrently (ticket counter, several row groups per warp, every launch
    # shape of the kernel), but no two walks share a row and no walk visits a node twice: walk k
    # runs along its own stretch of distinct nodes, and K = 0 leaves no negative draws.  Without
    # shared rows nothing can race, so the concurrent result must equal strictly sequential SGD.
    n_walks, span = 700, 64
    n = n_walks * span
    rng = np.random.default_rng(dim + L)
    walks = np.empty((n_walks, L), dtype=np.int32)
    for k in range(n_walks):
        walks[k] = k * span + rng.permutation(span)[:L]
    walks[5, L // 2:] = -1                                # a walk that ended early
    thr, alias = O.build_alias(np.ones(n), 1.0)
    c, o, ng, n_pairs = O.expand_lists(walks, 9, w, 0, thr, alias, 3)
    w_in0, w_out0 = random_tables(n, dim, 8)
    U, V = w_in0.numpy().astype(np.float64), w_out0.numpy().astype(np.float64)
    loss_o, cnt_o = O.sgns_seq_from_lists(U, V, c, o, ng, 2 * w, 0.05)
    assert cnt_o == n_pairs > 0
    for mode in (B.GS_HOGWILD, B.GS_HOGWILD_RED):
        w_in, w_out = w_in0.to(DEV), w_out0.to(DEV)
        loss, cnt, _, _ = run_step(w_in, w_out, torch.from_numpy(walks).to(DEV), 9, w, 0, None, 0.05, 3,
                                   mode, dump=False)
        assert cnt == cnt_o and abs(loss - loss_o) < 2e-6 * abs(loss_o)
        assert np.abs(w_in.cpu().numpy() - U).max() <= 1e-5
        assert np.abs(w_out.cpu().numpy() - V).max() <= 1e-5
    assert np.abs(V - w_out0.numpy()).max() > 1e-3


def test_sgns_step_edge_cases(tiny):
    _, g, off, col, thr, alias = tiny
    a_dev = alias_to_device(thr, alias)
    w_in0, w_out0 = random_tables(g.n_nodes, 64, 3)
    for mode in (B.GS_DETERMINISTIC, B.GS_HOGWILD):
        w_in, w_out = w_in0.to(DEV), w_out0.to(DEV)
        # no walks at all
        loss, cnt, _, _ = run_step(w_in, w_out, torch.empty((0, 10), dtype=torch.int32, device=DEV),
                                   0, 5, 5, a_dev, 0.1, 0, mode, dump=False)
        assert loss == 0.0 and cnt == 0
        # walks made only of dead entries / single nodes: no pairs, tables untouched
        walks = torch.full((33, 10), -1, dtype=torch.int32, device=DEV)
        walks[:, 0] = torch.arange(33, dtype=torch.int32)
        loss, cnt, pd, nd = run_step(w_in, w_out, walks, 0, 5, 5, a_dev, 0.1, 0, mode)
        assert loss == 0.0 and cnt == 0 and (pd == -1).all() and (nd == -1).all()
        assert torch.equal(w_in.cpu(), w_in0) and torch.equal(w_out.cpu(), w_out0)
    with pytest.raises(B.GsError) as e:
        B.gs_sgns_step(w_in, w_out, walks, 0, 33, 5, a_dev, 0.1, 0, 0)
    assert e.value.status == -6


# ---------------------------------------------------------------- epoch
def test_epoch_tiny_deepwalk_deterministic_matches_oracle(tiny):
    wl, g, off, col, thr, alias = tiny
    n = g.n_nodes
    U = O.init_rows(np.arange(n), wl.dim, 0)
    V = np.zeros_like(U)
    want = O.sgns_epoch(off, col, thr, alias, U, V, walks_per_node=1, L=wl.walk_len, w=wl.window,
                        K=wl.n_neg, lr0=wl.lr0, schedule="linear", batch_walks=512, seed=0)
    G = load(g)
    w_in = torch.empty((n, wl.dim), dtype=torch.float32, device=DEV)
    w_out = torch.empty_like(w_in)
    B.gs_init_embeddings(w_in, w_out, 0)
    res = B.gs_sgns_epoch(G, alias_to_device(thr, alias), w_in, w_out, walks_per_node=1,
                          walk_len=wl.walk_len, window=wl.window, n_neg=wl.n_neg, lr0=wl.lr0,
                          batch_walks=512, seed=0, mode=B.GS_DETERMINISTIC,
                          lr_schedule=B.GS_LR_LINEAR)
    assert res.pairs == want["pairs"] and res.steps == want["steps"]
    assert res.masked_negs == want["masked_negs"] > 0
    assert res.batches == (n + 511) // 512
    assert abs(res.loss_sum / res.pairs - want["loss_sum"] / want["pairs"]) <= LOSS_RTOL * want["loss_sum"] / want["pairs"]
    assert np.abs(w_in.cpu().numpy() - U).max() <= EMB_TOL
    assert np.abs(w_out.cpu().numpy() - V).max() <= EMB_TOL
    # resume: two halves equal one run, bit for bit
    w_in2 = torch.empty_like(w_in)
    w_out2 = torch.empty_like(w_in)
    B.gs_init_embeddings(w_in2, w_out2, 0)
    kw = dict(walks_per_node=1, walk_len=wl.walk_len, window=wl.window, n_neg=wl.n_neg,
              lr0=wl.lr0, batch_walks=512, seed=0, mode=B.GS_DETERMINISTIC,
              lr_schedule=B.GS_LR_LINEAR)
    r1 = B.gs_sgns_epoch(G, alias_to_device(thr, alias), w_in2, w_out2, first_batch=0, num_batches=7, **kw)
    r2 = B.gs_sgns_epoch(G, alias_to_device(thr, alias), w_in2, w_out2, first_batch=7, **kw)
    assert torch.equal(w_in, w_in2) and torch.equal(w_out, w_out2)
    assert r1.pairs + r2.pairs == res.pairs


def test_lock_free_loss_not_worse_than_synchronous_on_medium_workload():
    # The synchronous mode computes every gradient of a 512-walk batch from the batch-start
    # tables; the lock-free modes see earlier updates and so reach a LOWER loss.  The criterion
    # "lock-free holds the loss within 1 % of the deterministic mode" is therefore checked as:
    # racing must not cost more than 1 % against the synchronous mode.
    wl = WL.WORKLOADS["deepwalk_medium"]
    g = wl.make_graph(device=DEV)
    G = B.gs_graph_load_csr(g.offsets, g.cols, B.GS_VALIDATE | B.GS_REQUIRE_SORTED)
    deg = g.degrees().cpu().numpy().astype(np.float64)
    a_dev = torch.from_numpy(B.gs_build_alias(deg, 0.75).view(np.int64)).to(DEV)
    losses = {}
    for mode, bw in ((B.GS_DETERMINISTIC, 512), (B.GS_HOGWILD, 16384), (B.GS_HOGWILD_RED, 16384)):
        w_in = torch.empty((g.n_nodes, wl.dim), dtype=torch.float32, device=DEV)
        w_out = torch.empty_like(w_in)
        B.gs_init_embeddings(w_in, w_out, 1)
        kw = dict(walks_per_node=wl.walks_per_node, walk_len=wl.walk_len, window=wl.window,
                  n_neg=wl.n_neg, lr0=wl.lr0, batch_walks=bw, seed=1, mode=mode)
        n_b = 131072 // bw
        B.gs_sgns_epoch(G, a_dev, w_in, w_out, first_batch=0, num_batches=n_b, **kw)
        res = B.gs_sgns_epoch(G, a_dev, w_in, w_out, first_batch=n_b, num_batches=n_b, **kw)
        losses[mode] = res.loss_sum / res.pairs
    det = losses[B.GS_DETERMINISTIC]
    assert det < 0.9 * (1 + wl.n_neg) * np.log(2), losses     # training did reduce the loss
    for mode in (B.GS_HOGWILD, B.GS_HOGWILD_RED):
        assert losses[mode] <= 1.01 * det, losses
    # the two lock-free variants agree with each other within 1 % at this graph size
    assert abs(losses[B.GS_HOGWILD] - losses[B.GS_HOGWILD_RED]) <= 0.01 * losses[B.GS_HOGWILD_RED], losses


@pytest.mark.parametrize("mode", [B.GS_HOGWILD_RED, B.GS_HOGWILD])
def test_lock_free_loss_within_one_percent_of_race_free_schedule(tiny, mode):
    # Race-free reference of the lock-free schedule: the oracle's sequential mode (walks one
    # after another, fp64).  With increments sent as reductions, concurrency on the GPU may only
    # move the epoch's mean loss by 1 % (measured: +0.15 %).  Plain stores on THIS graph are another
    # matter, and the test says so with the measured bound: 10^4 nodes, 512 walks at a time, and
    # the hub rows are targets of most of them, so two warps that update a hub row at the same
    # moment keep one of the two increments.  The epoch then ends 12 % above the race-free run
    # (4.05 against 3.61); it still learns (below the untrained 4.159), and on graphs of a
    # million nodes the same mode stays within 1 % (next test).
    wl, g, off, col, thr, alias = tiny
    n = g.n_nodes
    U = O.init_rows(np.arange(n), wl.dim, 0)
    V = np.zeros_like(U)
    want = O.sgns_epoch(off, col, thr, alias, U, V, walks_per_node=2, L=wl.walk_len, w=wl.window,
                        K=wl.n_neg, lr0=wl.lr0, schedule="constant", batch_walks=512, seed=0,
                        mode="seq")
    ref = want["loss_sum"] / want["pairs"]
    G = load(g)
    w_in = torch.empty((n, wl.dim), dtype=torch.float32, device=DEV)
    w_out = torch.empty_like(w_in)
    B.gs_init_embeddings(w_in, w_out, 0)
    res = B.gs_sgns_epoch(G, alias_to_device(thr, alias), w_in, w_out, walks_per_node=2,
                          walk_len=wl.walk_len, window=wl.window, n_neg=wl.n_neg, lr0=wl.lr0,
                          batch_walks=512, seed=0, mode=mode)
    assert res.pairs == want["pairs"]
    got = res.loss_sum / res.pairs
    assert ref < 0.97 * (1 + wl.n_neg) * np.log(2)
    if mode == B.GS_HOGWILD_RED:
        assert abs(got - ref) <= 0.01 * ref, (got, ref)
    else:
        assert ref < got <= 1.15 * ref, (got, ref)              # lost increments cost, never help
        assert got < 0.985 * (1 + wl.n_neg) * np.log(2), got    # and the run still learns


def test_lock_free_modes_against_their_race_free_schedule_on_the_medium_workload():
    # The criterion "the lock-free mode holds the loss within 1 % of the deterministic mode", looked
    # at two-sided and at a matched schedule on the 1M-node workload - and found NOT to hold while
    # the loss falls fast.  The matched schedule of a lock-free run is the strictly sequential one
    # (walks one after another, every pair seeing all earlier updates): the oracle's sequential
    # mode in fp64 is deterministic and free of races.  (A synchronous batch is not that schedule,
    # whatever its size: it takes every gradient of a walk from the same batch-start rows.
    # Measured here, second half of 2 x 131,072 walks: synchronous batches of 512, 16 and 1 walks
    # end at 2.866, 2.838 and 2.838, the lock-free variants at 2.572 (plain stores) and 2.550
    # (reductions): ten per cent lower because of the schedule, not of the races.)
    # What separates a lock-free GPU run from the sequential one is the number of walks in flight:
    # each of them computes its gradients from rows that the others are changing.  The learning
    # rate here is four times the workload's, so that 2 x 16,384 walks - one minute of oracle -
    # leave the start (3.50, then 2.21, from 4.16); that also makes stale gradients cost more.
    # Measured gap to the sequential run, first / second half:
    #   launches of   128 walks: reductions +0.7 % / +3.2 %, plain stores +1.3 % / +4.0 %
    #   launches of 16384 walks: reductions +5.2 % / +18 %,  plain stores +8.7 % / +20 %
    # (about 3000 walks run at once in a large launch).  The gap is a property of running
    # thousands of walks at once; lost increments (plain stores against reductions) add one to
    # four points.  Where the loss has flattened the variants agree within 1 % (previous test).
    # The bounds asserted below are these measurements with head room, not the criterion.
    wl = WL.WORKLOADS["deepwalk_medium"]
    g = wl.make_graph(device=DEV)
    n, seed, half, lr = g.n_nodes, wl.graph_seed, 16384, 4 * wl.lr0
    off = g.offsets.cpu().numpy().astype(np.int64)
    col = g.cols.cpu().numpy()
    thr, alias = O.build_alias((off[1:] - off[:-1]).astype(np.float64), 0.75)
    U = O.init_rows(np.arange(n), wl.dim, seed)
    V = np.zeros_like(U)
    okw = dict(walks_per_node=wl.walks_per_node, L=wl.walk_len, w=wl.window, K=wl.n_neg, lr0=lr,
               schedule="constant", batch_walks=half, seed=seed, mode="seq")
    want = [O.sgns_epoch(off, col, thr, alias, U, V, first_batch=b, num_batches=1, **okw) for b in (0, 1)]
    ref = [r["loss_sum"] / r["pairs"] for r in want]
    untrained = (1 + wl.n_neg) * np.log(2)
    assert ref[1] < 0.6 * untrained and ref[0] < 0.9 * untrained, ref      # the run has left the start
    G = B.gs_graph_load_csr(g.offsets, g.cols, B.GS_VALIDATE | B.GS_REQUIRE_SORTED | B.GS_BUILD_WALK_INDEX)
    a_dev = alias_to_device(thr, alias)
    gap = {}
    for mode in (B.GS_HOGWILD_RED, B.GS_HOGWILD):
        for bw in (128, half):
            w_in = torch.empty((n, wl.dim), dtype=torch.float32, device=DEV)
            w_out = torch.empty_like(w_in)
            B.gs_init_embeddings(w_in, w_out, seed)
            kw = dict(walks_per_node=wl.walks_per_node, walk_len=wl.walk_len, window=wl.window,
                      n_neg=wl.n_neg, lr0=lr, batch_walks=bw, seed=seed, mode=mode)
            nb = half // bw
            for b in (0, 1):
                res = B.gs_sgns_epoch(G, a_dev, w_in, w_out, first_batch=b * nb, num_batches=nb, **kw)
                assert res.pairs == want[b]["pairs"]
                gap[mode, bw, b] = (res.loss_sum / res.pairs - ref[b]) / ref[b]
    print({k: round(v, 4) for k, v in gap.items()})
    for mode in (B.GS_HOGWILD_RED, B.GS_HOGWILD):
        for b in (0, 1):
            assert -0.01 <= gap[mode, 128, b] <= 0.06, gap           # few walks in flight: close
            assert gap[mode, 128, b] <= gap[mode, half, b] <= 0.25, gap   # thousands in flight: further
    for bw in (128, half):
        for b in (0, 1):                                             # lost increments never help
            assert gap[B.GS_HOGWILD, bw, b] >= gap[B.GS_HOGWILD_RED, bw, b] - 0.01, gap
    G.close()
    B.gs_release_workspace()


def test_lock_free_modes_track_the_sequential_run_at_the_workload_rate():
    # The same comparison at the workload's own learning rate and in the launch shape the benchmark
    # times (16,384 walks per launch, thousands in flight), over 2 x 131,072 walks: the sequential
    # oracle's losses per stretch of 16,384 walks are stored (tests/golden, seven minutes of
    # oracle), the GPU runs are compared with them stretch by stretch.  Measured: reductions end
    # +0.9 % (first half) and +1.2 % (second half) above the sequential run, plain stores +3.7 % and
    # +2.1 %.  Two-sided bounds with head room; the 1 % of the criterion is NOT met by either
    # variant in this stretch of training, and the assertion says by how much.
    from pathlib import Path
    rows = [l.split() for l in (Path(__file__).parent / "golden" / "sequential_losses_medium.txt")
            .read_text().splitlines() if l and not l.startswith("#")]
    ref = np.array([float(r[1]) for r in rows])
    ref_pairs = [int(r[2]) for r in rows]
    wl = WL.WORKLOADS["deepwalk_medium"]
    g = wl.make_graph()                                  # on the CPU, as the stored run did
    n, seed, stretch = g.n_nodes, 1, 16384
    deg = g.degrees().numpy().astype(np.float64)
    thr, alias = O.build_alias(deg, 0.75)
    G = B.gs_graph_load_csr(g.offsets.to(DEV), g.cols.to(DEV),
                            B.GS_VALIDATE | B.GS_REQUIRE_SORTED | B.GS_BUILD_WALK_INDEX)
    a_dev = alias_to_device(thr, alias)
    bounds = {B.GS_HOGWILD_RED: (0.015, 0.02), B.GS_HOGWILD: (0.05, 0.03)}
    for mode in (B.GS_HOGWILD_RED, B.GS_HOGWILD):
        w_in = torch.empty((n, wl.dim), dtype=torch.float32, device=DEV)
        w_out = torch.empty_like(w_in)
        B.gs_init_embeddings(w_in, w_out, seed)
        got = []
        for b in range(len(ref)):
            res = B.gs_sgns_epoch(G, a_dev, w_in, w_out, walks_per_node=wl.walks_per_node,
                                  walk_len=wl.walk_len, window=wl.window, n_neg=wl.n_neg, lr0=wl.lr0,
                                  batch_walks=stretch, seed=seed, mode=mode, first_batch=b, num_batches=1)
            assert res.pairs == ref_pairs[b], (b, res.pairs, ref_pairs[b])     # the same walks
            got.append(res.loss_sum / res.pairs)
        got = np.array(got)
        h = len(ref) // 2
        gaps = [(got[:h].mean() - ref[:h].mean()) / ref[:h].mean(), (got[h:].mean() - ref[h:].mean()) / ref[h:].mean()]
        print(f"mode {mode}: gap to the sequential run {gaps[0]:+.4f} / {gaps[1]:+.4f}; last stretch {got[-1]:.4f} vs {ref[-1]:.4f}")
        for gap, hi in zip(gaps, bounds[mode]):
            assert -0.01 <= gap <= hi, (mode, gaps)
    G.close()
    B.gs_release_workspace()


def test_epoch_node2vec_runs_and_counts_match_oracle(tiny):
    wl, g, off, col, thr, alias = tiny
    n = g.n_nodes
    U = O.init_rows(np.arange(n), 64, 1)
    V = np.zeros_like(U)
    want = O.sgns_epoch(off, col, thr, alias, U, V, walks_per_node=1, L=12, w=3, K=3, lr0=0.025,
                        schedule="constant", batch_walks=1000, seed=1, kind="node2vec", p=0.5,
                        q=2.0, num_batches=4)
    G = load(g)
    w_in = torch.empty((n, 64), dtype=torch.float32, device=DEV)
    w_out = torch.empty_like(w_in)
    B.gs_init_embeddings(w_in, w_out, 1)
    res = B.gs_sgns_epoch(G, alias_to_device(thr, alias), w_in, w_out, walks_per_node=1,
                          walk_len=12, window=3, n_neg=3, lr0=0.025, batch_walks=1000, seed=1,
                          mode=B.GS_DETERMINISTIC, walk_kind=B.GS_WALK_NODE2VEC, p=0.5, q=2.0,
                          num_batches=4)
    assert res.pairs == want["pairs"] and res.steps == want["steps"] and res.batches == 4
    assert res.masked_negs == want["masked_negs"]
    assert abs(res.loss_sum - want["loss_sum"]) <= LOSS_RTOL * want["loss_sum"]
    assert np.abs(w_out.cpu().numpy() - V).max() <= EMB_TOL
    # the integer statistics do not depend on the update mode
    res2 = B.gs_sgns_epoch(G, alias_to_device(thr, alias), w_in, w_out, walks_per_node=1,
                           walk_len=12, window=3, n_neg=3, lr0=0.025, batch_walks=1000, seed=1,
                           mode=B.GS_HOGWILD, walk_kind=B.GS_WALK_NODE2VEC, p=0.5, q=2.0,
                           num_batches=4)
    assert (res2.pairs, res2.steps, res2.masked_negs) == (res.pairs, res.steps, res.masked_negs)


# ---------------------------------------------------------------- ids outside the graph
def test_out_of_range_ids_count_as_absent_instead_of_faulting(tiny):
    # The library never dereferences an id it has not range-checked: a start node, a walk entry or
    # an alias-table cell outside [0, n_nodes) is treated like -1.
    wl, g, off, col, thr, alias = tiny
    n = g.n_nodes
    starts = np.array([3, -5, n, 2**31 - 1, 7, n + 1000, 0, n - 1] * 40, dtype=np.int32)
    ok = (starts >= 0) & (starts < n)
    want, _ = O.uniform_walks(off, col, np.where(ok, starts, 0).astype(np.int32), len(starts), 9, 16, 2)
    want[~ok] = -1
    sd = torch.from_numpy(starts).to(DEV)
    B.gs_refused_ids(clear=True)
    for flags in (B.GS_VALIDATE | B.GS_REQUIRE_SORTED, B.GS_BUILD_WALK_INDEX | B.GS_REQUIRE_SORTED):
        G = load(g, flags=flags)
        assert np.array_equal(B.gs_random_walks(G, sd, len(starts), 9, 16, 2).cpu().numpy(), want)
        # every start outside the graph was counted, once (the counter is sticky until cleared)
        assert B.gs_refused_ids() == int((~ok).sum())
        assert B.gs_refused_ids(clear=True) == int((~ok).sum()) and B.gs_refused_ids() == 0
        assert np.array_equal(B.gs_random_walks(G, sd, len(starts), 9, 13, 2).cpu().numpy()[~ok],
                              np.full((int((~ok).sum()), 13), -1))
        assert B.gs_refused_ids(clear=True) == int((~ok).sum())
        want2, _, _ = O.node2vec_walks(off, col, np.where(ok, starts, 0).astype(np.int32), len(starts), 9, 16,
                                       2, 0.5, 2.0)
        want2[~ok] = -1
        for lanes in (0, 1, 4, 32):
            B.gs_tune_node2vec_group(lanes)
            got = B.gs_node2vec_walks(G, sd, len(starts), 9, 16, 2, 0.5, 2.0)
            assert np.array_equal(got.cpu().numpy(), want2)
            assert B.gs_refused_ids(clear=True) == int((~ok).sum())
        B.gs_tune_node2vec_group(0)
    # walk entries outside the tables behave like -1 in the update
    walks, _ = O.uniform_walks(off, col, None, 200, 0, 12, 5)
    dirty = walks.copy()
    rng = np.random.default_rng(0)
    hit = rng.random(walks.shape) < 0.1
    dirty[hit] = rng.choice([n, n + 7, 2**31 - 1, -9], size=int(hit.sum()))
    clean = np.where(hit, -1, walks).astype(np.int32)
    a_dev = alias_to_device(thr, alias)
    w_in0, w_out0 = random_tables(n, 64, 4)
    # what the kernels must refuse: a bad entry as a center (once per position) and as a context
    # of every live center within the window (-9 included: only -1 means "no entry")
    w_ = 3
    n_refused = 0
    for wk_row, hit_row in zip(dirty, hit):
        for i in range(len(wk_row)):
            if hit_row[i]:
                n_refused += 1
            elif wk_row[i] >= 0:
                n_refused += int(hit_row[max(0, i - w_):i + w_ + 1].sum())
    res = []
    B.gs_refused_ids(clear=True)
    for wk in (clean, dirty):
        w_in, w_out = w_in0.to(DEV), w_out0.to(DEV)
        loss, cnt, pd, nd = run_step(w_in, w_out, torch.from_numpy(wk).to(DEV), 0, 3, 4, a_dev, 0.025, 5,
                                     B.GS_DETERMINISTIC)
        res.append((loss, cnt, pd, nd, w_in, w_out))
        assert B.gs_refused_ids(clear=True) == (n_refused if wk is dirty else 0)
    assert res[0][0] == res[1][0] and res[0][1] == res[1][1] > 0
    for x, y in zip(res[0][2:], res[1][2:]):
        assert torch.equal(x, y)
    w_in, w_out = w_in0.to(DEV), w_out0.to(DEV)
    loss, cnt, _, _ = run_step(w_in, w_out, torch.from_numpy(dirty).to(DEV), 0, 3, 4, a_dev, 0.025, 5,
                               B.GS_HOGWILD, dump=False)
    assert cnt == res[0][1] and np.isfinite(loss) and torch.isfinite(w_out).all()
    assert B.gs_refused_ids(clear=True) == n_refused        # the lock-free kernel counts the same ids
    # an alias table whose cells point outside the graph yields no such negative
    bad_alias = alias.copy()
    bad_alias[::3] = n + 5
    w_in, w_out = w_in0.to(DEV), w_out0.to(DEV)
    loss, cnt, pd, nd = run_step(w_in, w_out, torch.from_numpy(clean).to(DEV), 0, 3, 4,
                                 alias_to_device(thr, bad_alias), 0.025, 5, B.GS_DETERMINISTIC)
    ndn = nd.cpu().numpy()
    assert ndn.max() < n and cnt == res[0][1] and torch.isfinite(w_out).all()
    # every draw that landed on a bad cell is reported: those are the -1 entries of pairs that
    # exist (a masked negative keeps its id in the dump)
    pdn = pd.cpu().numpy().reshape(-1, 2)
    lost = int((ndn.reshape(-1, 4)[pdn[:, 0] >= 0] < 0).sum())
    assert lost > 0 and B.gs_refused_ids(clear=True) == lost
