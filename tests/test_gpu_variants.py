"""GPU parity of the corpus variants (window shrinking, frequent-node sub-sampling, keyed start
shuffle) and of the Adam step against the CPU oracle: integer results bit-exact, tables within
1e-4 of the fp64 oracle."""
import numpy as np
import pytest
import torch

from oracle import gs_oracle as O
from paper_2407_15452_b200 import binding as B
from paper_2407_15452_b200 import workloads as WL
from tests.helpers import alias_to_device, degree_alias, np_graph

pytestmark = pytest.mark.gpu
DEV = "cuda"
EMB_TOL = 1e-4


@pytest.fixture(scope="module")
def tiny():
    wl = WL.WORKLOADS["tiny_deepwalk"]
    g = wl.make_graph()
    off, col = np_graph(g)
    thr, alias = degree_alias(off)
    return wl, g, off, col, thr, alias


def thr_to_device(keep_thr):
    return torch.from_numpy(keep_thr.view(np.int32)).to(DEV)


def random_tables(n, dim, seed, scale=0.3):
    gen = torch.Generator().manual_seed(seed)
    return ((torch.rand((n, dim), generator=gen) - 0.5) * scale,
            (torch.rand((n, dim), generator=gen) - 0.5) * scale)


# ---------------------------------------------------------------- window shrinking
@pytest.mark.parametrize("dim,L,w,K,mode", [(128, 40, 10, 5, B.GS_DETERMINISTIC), (64, 11, 4, 3, B.GS_DETERMINISTIC),
                                             (128, 20, 5, 5, B.GS_HOGWILD), (32, 9, 1, 2, B.GS_HOGWILD_RED)])
def test_window_shrinking_pairs_bit_exact_and_step_matches(tiny, dim, L, w, K, mode):
    _, g, off, col, thr, alias = tiny
    n, n_walks, base, seed = g.n_nodes, 333, 77, 12
    walks, _ = O.uniform_walks(off, col, None, n_walks, base, L, seed)
    walks[3, L // 3:] = -1
    c, o, ng, n_pairs = O.expand_lists(walks, base, w, K, thr, alias, seed, shrink=True)
    full_pairs = O.expand_lists(walks, base, w, K, thr, alias, seed)[3]
    assert n_pairs < full_pairs or w == 1
    w_in0, w_out0 = random_tables(n, dim, 2)
    w_in, w_out = w_in0.to(DEV), w_out0.to(DEV)
    loss = torch.zeros(1, dtype=torch.float64, device=DEV)
    cnt = torch.zeros(1, dtype=torch.int64, device=DEV)
    pd = torch.full((n_walks, L, 2 * w, 2), -7, dtype=torch.int32, device=DEV)
    nd = torch.full((n_walks, L, 2 * w, K), -7, dtype=torch.int32, device=DEV)
    B.gs_sgns_step(w_in, w_out, torch.from_numpy(walks).to(DEV), base, w, K, alias_to_device(thr, alias),
                   0.025, seed, mode | B.GS_WINDOW_SHRINK, loss, cnt, pd, nd)
    torch.cuda.synchronize()
    pdn = pd.cpu().numpy().reshape(-1, 2)
    assert np.array_equal(pdn[:, 0], c) and np.array_equal(pdn[:, 1], o)
    assert np.array_equal(nd.cpu().numpy().reshape(-1, K), ng)
    assert cnt.item() == n_pairs
    if mode == B.GS_DETERMINISTIC:
        U, V = w_in0.numpy().astype(np.float64), w_out0.numpy().astype(np.float64)
        loss_o, _ = O.sgns_det_from_lists(U, V, c, o, ng, 0.025)
        assert abs(loss.item() - loss_o) <= 2e-6 * abs(loss_o)
        assert np.abs(w_in.cpu().numpy() - U).max() <= EMB_TOL
        assert np.abs(w_out.cpu().numpy() - V).max() <= EMB_TOL


# ---------------------------------------------------------------- sub-sampling
@pytest.mark.parametrize("L,n_walks", [(40, 2501), (1, 100), (33, 64), (1024, 9), (80, 0)])
def test_subsampled_walks_bit_exact(tiny, L, n_walks):
    _, g, off, col, _, _ = tiny
    deg = (off[1:] - off[:-1]).astype(np.float64)
    keep_thr = B.gs_build_keep_thresholds(deg, 2e-5)
    assert np.array_equal(keep_thr, O.keep_thresholds(deg, 2e-5))
    walks, _ = O.uniform_walks(off, col, None, n_walks, 10**10, L, 8)
    if n_walks > 7:
        walks[7, L // 2:] = -1
    want, kept_o = O.subsample_walks(walks, 10**10, keep_thr, 8)
    if n_walks > 50:
        assert 0 < kept_o < (walks >= 0).sum()                    # the thresholds bite
    wd = torch.from_numpy(walks).to(DEV).reshape(n_walks, L)
    kept = torch.zeros(1, dtype=torch.int64, device=DEV)
    got = B.gs_subsample_walks(wd, 10**10, thr_to_device(keep_thr), 8, kept=kept)
    assert np.array_equal(got.cpu().numpy(), want) and kept.item() == kept_o
    # in place
    B.gs_subsample_walks(wd, 10**10, thr_to_device(keep_thr), 8, out=wd)
    assert np.array_equal(wd.cpu().numpy(), want)


# ---------------------------------------------------------------- start shuffle
@pytest.mark.parametrize("n", [1, 2, 5, 1000, 1024, 1025, 65537, 3_000_001])
def test_shuffled_starts_bit_exact_and_bijective(n):
    for epoch, seed in ((0, 1), (9, 2**63 + 5)):
        got = B.gs_shuffled_starts(n, seed, epoch, 0, n, DEV)
        assert torch.equal(torch.sort(got).values, torch.arange(n, dtype=torch.int32, device=DEV))
        cnt = min(n, 5000)
        first = max(n - 17, 0)
        part = B.gs_shuffled_starts(n, seed, epoch, first, cnt, DEV).cpu().numpy()
        assert np.array_equal(part, O.shuffled_starts(n, seed, epoch, first, cnt))
    assert B.gs_shuffled_starts(n, 1, 0, 5, 0, DEV).numel() == 0


def test_shuffled_starts_at_the_largest_node_count():
    # 2^31 - 1 nodes: 32-bit halves in the network, ids beyond 2^31 as walk ids; sampled ranges only
    n = 2**31 - 1
    for first in (0, n - 500, 5 * n + 12345):
        got = B.gs_shuffled_starts(n, 77, 3, first, 4096, DEV).cpu().numpy()
        assert np.array_equal(got, O.shuffled_starts(n, 77, 3, first, 4096))
        assert got.min() >= 0 and len(np.unique(got)) == 4096


# ---------------------------------------------------------------- epoch with every variant on
def test_epoch_with_shuffle_subsampling_and_shrinking_matches_oracle(tiny):
    wl, g, off, col, thr, alias = tiny
    n = g.n_nodes
    deg = (off[1:] - off[:-1]).astype(np.float64)
    keep_thr = O.keep_thresholds(deg, 1e-4)
    U = O.init_rows(np.arange(n), wl.dim, 3)
    V = np.zeros_like(U)
    want = O.sgns_epoch(off, col, thr, alias, U, V, walks_per_node=1, L=wl.walk_len, w=wl.window,
                        K=wl.n_neg, lr0=wl.lr0, schedule="linear", batch_walks=512, seed=3,
                        shrink=True, keep_thr=keep_thr, shuffle_epoch=4)
    plain = O.sgns_epoch(off, col, thr, alias, O.init_rows(np.arange(n), wl.dim, 3), np.zeros_like(U),
                         walks_per_node=1, L=wl.walk_len, w=wl.window, K=wl.n_neg, lr0=wl.lr0,
                         schedule="linear", batch_walks=512, seed=3)
    assert want["pairs"] < plain["pairs"]
    G = B.gs_graph_load_csr(g.offsets.to(DEV), g.cols.to(DEV), B.GS_VALIDATE | B.GS_REQUIRE_SORTED)
    w_in = torch.empty((n, wl.dim), dtype=torch.float32, device=DEV)
    w_out = torch.empty_like(w_in)
    B.gs_init_embeddings(w_in, w_out, 3)
    res = B.gs_sgns_epoch(G, alias_to_device(thr, alias), w_in, w_out, walks_per_node=1,
                          walk_len=wl.walk_len, window=wl.window, n_neg=wl.n_neg, lr0=wl.lr0,
                          batch_walks=512, seed=3, mode=B.GS_DETERMINISTIC | B.GS_WINDOW_SHRINK,
                          lr_schedule=B.GS_LR_LINEAR, keep_thr=thr_to_device(keep_thr), shuffle_epoch=4)
    assert res.pairs == want["pairs"] and res.steps == want["steps"]
    assert res.masked_negs == want["masked_negs"]
    mean_o = want["loss_sum"] / want["pairs"]
    assert abs(res.loss_sum / res.pairs - mean_o) <= 1e-3 * mean_o
    assert np.abs(w_in.cpu().numpy() - U).max() <= EMB_TOL
    assert np.abs(w_out.cpu().numpy() - V).max() <= EMB_TOL


# ---------------------------------------------------------------- Adam
@pytest.mark.parametrize("dim,pair_mode", [(128, 0), (64, B.GS_WINDOW_SHRINK), (32, B.GS_PAIRS_FORWARD_ONLY),
                                           (256, 0)])
def test_adam_steps_match_oracle(dim, pair_mode):
    wl = WL.WORKLOADS["tiny_deepwalk"]
    g = wl.make_graph(scale=0.3)                       # 3000 nodes: rows are hit in some steps only
    off, col = np_graph(g)
    thr, alias = degree_alias(off)
    n = g.n_nodes
    L, w, K, seed = 12, 3, 4, 5
    lr, b1, b2, eps = 0.002, 0.9, 0.999, 1e-8
    rng = np.random.default_rng(0)
    U0 = ((rng.random((n, dim)) - 0.5) * 0.4).astype(np.float32).astype(np.float64)
    V0 = ((rng.random((n, dim)) - 0.5) * 0.4).astype(np.float32).astype(np.float64)
    batches = []
    for it in range(6):
        base = 100 + 150 * it
        walks, _ = O.uniform_walks(off, col, None, 150, base, L, seed)
        batches.append((walks, base))
    U, V = U0.copy(), V0.copy()
    MU, VU, MV, VV = (np.zeros_like(U) for _ in range(4))
    want_losses, pairs = [], 0
    # Adam's step is lr * m / sqrt(v): where a touched value's gradient is within rounding of zero
    # the SIGN of the step is decided by that rounding (fp32 on the GPU, fp64 in the oracle), and
    # the two sides may move by up to about lr each, in opposite directions.  Such values are
    # recorded here and bounded separately.
    near_zero_U, near_zero_V = np.zeros(U.shape, bool), np.zeros(V.shape, bool)
    for it, (walks, base) in enumerate(batches):
        c, o, ng, _ = O.expand_lists(walks, base, w, K, thr, alias, seed,
                                     forward_only=bool(pair_mode & B.GS_PAIRS_FORWARD_ONLY),
                                     shrink=bool(pair_mode & B.GS_WINDOW_SHRINK))
        GU, GV, _, _ = O.sgns_grad_from_lists(U, V, c, o, ng)
        rows_in, rows_out = O.touched_rows(c, o, ng)
        near_zero_U[rows_in] |= np.abs(GU[rows_in]) < 1e-6
        near_zero_V[rows_out] |= np.abs(GV[rows_out]) < 1e-6
        ls, pc = O.sgns_adam_step_from_lists(U, V, MU, VU, MV, VV, c, o, ng, lr, b1, b2, eps, it + 1)
        want_losses.append(ls)
        pairs += pc

    def run():
        w_in = torch.from_numpy(U0.astype(np.float32)).to(DEV)
        w_out = torch.from_numpy(V0.astype(np.float32)).to(DEV)
        m_in, v_in, m_out, v_out = (torch.zeros_like(w_in) for _ in range(4))
        a_dev = alias_to_device(thr, alias)
        loss = torch.zeros(1, dtype=torch.float64, device=DEV)
        cnt = torch.zeros(1, dtype=torch.int64, device=DEV)
        losses = []
        for it, (walks, base) in enumerate(batches):
            loss.zero_()
            B.gs_sgns_step_adam(w_in, w_out, m_in, v_in, m_out, v_out, torch.from_numpy(walks).to(DEV),
                                base, w, K, a_dev, lr, b1, b2, eps, it + 1, seed, pair_mode, loss, cnt)
            losses.append(loss.item())
        torch.cuda.synchronize()
        return w_in, w_out, m_in, v_in, m_out, v_out, losses, cnt.item()

    w_in, w_out, m_in, v_in, m_out, v_out, losses, cnt = run()
    assert cnt == pairs
    for a, b in zip(losses, want_losses):
        assert abs(a - b) <= 2e-5 * abs(b)
    for got, ref, near_zero in ((w_in, U, near_zero_U), (w_out, V, near_zero_V)):
        delta = np.abs(got.cpu().numpy() - ref)
        assert delta[~near_zero].max() <= EMB_TOL
        assert near_zero.mean() < 1e-3 and delta.max() <= 4 * lr * len(batches)
    for got, ref in ((m_in, MU), (v_in, VU), (m_out, MV), (v_out, VV)):
        # moments are fp32 on the GPU and inherit the 1e-4 table differences through later gradients
        assert np.abs(got.cpu().numpy() - ref).max() <= 1e-4 * np.abs(ref).max()
    # the run moved touched rows by about lr per step and left the other rows alone
    moved = np.abs(V - V0).max(axis=1)
    assert moved.max() > 3 * lr and (moved == 0).any()
    untouched = moved == 0
    assert np.array_equal(w_out.cpu().numpy()[untouched], V0[untouched].astype(np.float32))
    again = run()
    for a, b in zip(again[:6], (w_in, w_out, m_in, v_in, m_out, v_out)):
        assert torch.equal(a, b)                       # bitwise reproducible


def test_subsampling_drops_entries_outside_the_threshold_table(tiny):
    _, g, off, col, _, _ = tiny
    n = g.n_nodes
    keep_thr = np.full(n, 0xFFFFFFFF, dtype=np.uint32)
    walks, _ = O.uniform_walks(off, col, None, 300, 0, 20, 1)
    dirty = walks.copy()
    hit = np.random.default_rng(2).random(walks.shape) < 0.15
    dirty[hit] = n + 3
    want, _ = O.subsample_walks(np.where(hit, -1, walks).astype(np.int32), 0, keep_thr, 1)
    got = B.gs_subsample_walks(torch.from_numpy(dirty).to(DEV), 0, thr_to_device(keep_thr), 1)
    assert np.array_equal(got.cpu().numpy(), want)


# ---------------------------------------------------------------- optimizers inside the epoch driver
def test_epoch_with_momentum_matches_the_dense_oracle(tiny):
    wl, g, off, col, thr, alias = tiny
    n, dim, mu, lr = g.n_nodes, wl.dim, 0.9, 0.0025
    U = O.init_rows(np.arange(n), dim, 0)
    V = np.zeros_like(U)
    state = {"MU": np.zeros_like(U), "MV": np.zeros_like(U)}
    nb = 8                                               # eight batches of 512 walks, then two halves
    want = O.sgns_epoch(off, col, thr, alias, U, V, walks_per_node=1, L=wl.walk_len, w=wl.window,
                        K=wl.n_neg, lr0=lr, schedule="constant", batch_walks=512, seed=0, num_batches=nb,
                        optimizer="momentum", state=state, momentum=mu)
    G = B.gs_graph_load_csr(g.offsets.to(DEV), g.cols.to(DEV), B.GS_VALIDATE | B.GS_REQUIRE_SORTED)
    w_in = torch.empty((n, dim), dtype=torch.float32, device=DEV)
    w_out = torch.empty_like(w_in)
    B.gs_init_embeddings(w_in, w_out, 0)
    m_in, m_out = torch.zeros_like(w_in), torch.zeros_like(w_in)
    last_in = torch.zeros(n, dtype=torch.int32, device=DEV)
    last_out = torch.zeros_like(last_in)
    kw = dict(walks_per_node=1, walk_len=wl.walk_len, window=wl.window, n_neg=wl.n_neg, lr0=lr,
              batch_walks=512, seed=0, mode=B.GS_DETERMINISTIC, optimizer=B.GS_OPT_MOMENTUM, momentum=mu,
              m_in=m_in, m_out=m_out, last_in=last_in, last_out=last_out)
    a_dev = alias_to_device(thr, alias)
    r1 = B.gs_sgns_epoch(G, a_dev, w_in, w_out, first_batch=0, num_batches=3, **kw)
    r2 = B.gs_sgns_epoch(G, a_dev, w_in, w_out, first_batch=3, num_batches=nb - 3, **kw)
    B.gs_momentum_flush(w_in, m_in, last_in, lr, mu, nb)
    B.gs_momentum_flush(w_out, m_out, last_out, lr, mu, nb)
    torch.cuda.synchronize()
    assert r1.pairs + r2.pairs == want["pairs"] and r1.batches + r2.batches == nb
    assert abs(r1.loss_sum + r2.loss_sum - want["loss_sum"]) <= 1e-3 * want["loss_sum"]
    for got, ref in ((w_in, U), (w_out, V), (m_in, state["MU"]), (m_out, state["MV"])):
        assert np.abs(got.cpu().numpy() - ref).max() <= EMB_TOL
    assert np.abs(state["MV"]).max() > 50 * EMB_TOL
    with pytest.raises(B.GsError):                        # momentum needs a constant learning rate
        B.gs_sgns_epoch(G, a_dev, w_in, w_out, num_batches=1, lr_schedule=B.GS_LR_LINEAR, **kw)
    with pytest.raises(B.GsError):                        # and the synchronous mode
        B.gs_sgns_epoch(G, a_dev, w_in, w_out, num_batches=1, **{**kw, "mode": B.GS_HOGWILD})


def test_epoch_with_adam_matches_the_oracle(tiny):
    wl, g, off, col, thr, alias = tiny
    n, dim, lr = g.n_nodes, wl.dim, 0.001
    rng = np.random.default_rng(3)
    U0 = ((rng.random((n, dim)) - 0.5) * 0.4).astype(np.float32).astype(np.float64)
    V0 = ((rng.random((n, dim)) - 0.5) * 0.4).astype(np.float32).astype(np.float64)
    U, V = U0.copy(), V0.copy()
    MU, VU, MV, VV = (np.zeros_like(U) for _ in range(4))
    nb, base_it = 5, 7
    near_zero_U, near_zero_V = np.zeros(U.shape, bool), np.zeros(V.shape, bool)
    pairs, loss_o = 0, 0.0
    for b in range(nb):                                   # the oracle's epoch, batch by batch, so that the
        walks, _ = O.uniform_walks(off, col, None, 512, b * 512, wl.walk_len, 0)   # sign-sensitive values are known
        c, o, ng, _ = O.expand_lists(walks, b * 512, wl.window, wl.n_neg, thr, alias, 0, shrink=True)
        GU, GV, _, _ = O.sgns_grad_from_lists(U, V, c, o, ng)
        rows_in, rows_out = O.touched_rows(c, o, ng)
        near_zero_U[rows_in] |= np.abs(GU[rows_in]) < 1e-6
        near_zero_V[rows_out] |= np.abs(GV[rows_out]) < 1e-6
        ls, pc = O.sgns_adam_step_from_lists(U, V, MU, VU, MV, VV, c, o, ng, lr, 0.9, 0.999, 1e-8,
                                             base_it + b + 1)
        pairs += pc
        loss_o += ls
    G = B.gs_graph_load_csr(g.offsets.to(DEV), g.cols.to(DEV), B.GS_VALIDATE | B.GS_REQUIRE_SORTED)
    w_in = torch.from_numpy(U0.astype(np.float32)).to(DEV)
    w_out = torch.from_numpy(V0.astype(np.float32)).to(DEV)
    m_in, v_in, m_out, v_out = (torch.zeros_like(w_in) for _ in range(4))
    res = B.gs_sgns_epoch(G, alias_to_device(thr, alias), w_in, w_out, walks_per_node=1,
                          walk_len=wl.walk_len, window=wl.window, n_neg=wl.n_neg, lr0=lr, batch_walks=512,
                          seed=0, mode=B.GS_DETERMINISTIC | B.GS_WINDOW_SHRINK, num_batches=nb,
                          optimizer=B.GS_OPT_ADAM, momentum=0.9, beta2=0.999, eps=1e-8,
                          iteration_base=base_it, m_in=m_in, m_out=m_out, v_in=v_in, v_out=v_out)
    assert res.pairs == pairs and abs(res.loss_sum - loss_o) <= 1e-3 * loss_o
    for got, ref, near_zero in ((w_in, U, near_zero_U), (w_out, V, near_zero_V)):
        delta = np.abs(got.cpu().numpy() - ref)
        assert delta[~near_zero].max() <= EMB_TOL and delta.max() <= 4 * lr * nb
    for got, ref in ((m_in, MU), (v_in, VU), (m_out, MV), (v_out, VV)):
        assert np.abs(got.cpu().numpy() - ref).max() <= 1e-4 * np.abs(ref).max()
