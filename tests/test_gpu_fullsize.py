"""GPU parity at the full sizes of the named workloads, in the launch shape bench.py times
(one mini-batch of up to 2^20 walks from the middle of the epoch).

The oracle cannot run a whole batch at these sizes in seconds, so: walks are compared on
sampled ranges of walk ids computed one range at a time; counters are checked against
properties that hold at any size; the synchronous SGNS step is compared on 512 walks with the
oracle working on the touched rows only (ids renumbered one-to-one, row values read from the
device before the step as input data)."""
import numpy as np
import pytest
import torch

from oracle import gs_oracle as O
from paper_2407_15452_b200 import binding as B
from paper_2407_15452_b200 import workloads as WL
from tests.helpers import compact_problem, unpack_alias

pytestmark = pytest.mark.gpu
DEV = "cuda"
EMB_TOL = 1e-4


def count_pairs(walks, w):
    """Pairs formed by a batch of walks (pure counting on the device)."""
    ok = walks >= 0
    total = 0
    for k in range(1, w + 1):
        if k < walks.shape[1]:
            total += 2 * int((ok[:, k:] & ok[:, :-k]).sum())
    return total


def check_synchronous_step(wl, w_in, w_out, sub, sub_base, a_dev, thr, alias, seed):
    """One synchronous step of the 512 walks `sub` at full table size against the oracle working
    on the touched rows only.  The touched rows first get seeded values large enough that the
    step moves every one of them by far more than the tolerance, so a row that the apply pass
    skipped, wrote twice or wrote at a wrong address could not pass; all rows outside the batch
    inside three windows of a million rows (start, middle and end of the tables) must keep
    their bits."""
    n = w_in.shape[0]
    sub_h = sub.cpu().numpy()
    c, o, ng, n_pairs = O.expand_lists(sub_h, sub_base, wl.window, wl.n_neg, thr, alias, seed)
    ids, cc, oo, nn = compact_problem(c, o, ng)
    ids_dev = torch.from_numpy(ids).to(DEV)
    gen = torch.Generator().manual_seed(1234 + int(sub_base % 1000))
    u0 = (torch.rand((len(ids), wl.dim), generator=gen) - 0.5) * 0.6       # input rows: up to 0.3
    v0 = (torch.rand((len(ids), wl.dim), generator=gen) - 0.5) * 0.15      # output rows: up to 0.075
    w_in[ids_dev] = u0.to(DEV)
    w_out[ids_dev] = v0.to(DEV)
    U, V = u0.numpy().astype(np.float64), v0.numpy().astype(np.float64)
    U0, V0 = U.copy(), V.copy()
    win = min(1 << 20, n)
    windows = sorted({0, max(0, n // 2 - win // 2), n - win})
    keep = []
    for lo in windows:
        outside = torch.ones(win, dtype=torch.bool, device=DEV)
        inside = ids_dev[(ids_dev >= lo) & (ids_dev < lo + win)] - lo
        outside[inside] = False
        keep.append((lo, outside, w_in[lo:lo + win].clone(), w_out[lo:lo + win].clone()))
    loss_o, cnt_o = O.sgns_det_from_lists(U, V, cc, oo, nn, wl.lr0)
    loss = torch.zeros(1, dtype=torch.float64, device=DEV)
    cnt = torch.zeros(1, dtype=torch.int64, device=DEV)
    pd = torch.empty((512, wl.walk_len, 2 * wl.window, 2), dtype=torch.int32, device=DEV)
    nd = torch.empty((512, wl.walk_len, 2 * wl.window, wl.n_neg), dtype=torch.int32, device=DEV)
    B.gs_sgns_step(w_in, w_out, sub, sub_base, wl.window, wl.n_neg, a_dev, wl.lr0, seed,
                   B.GS_DETERMINISTIC, loss, cnt, pd, nd)
    torch.cuda.synchronize()
    pd = pd.cpu().numpy().reshape(-1, 2)
    assert np.array_equal(pd[:, 0], c) and np.array_equal(pd[:, 1], o)
    assert np.array_equal(nd.cpu().numpy().reshape(-1, wl.n_neg), ng)
    assert int(cnt.item()) == cnt_o == n_pairs > 0
    assert abs(loss.item() - loss_o) <= 2e-6 * abs(loss_o)
    err_in = np.abs(w_in[ids_dev].cpu().numpy() - U).max()
    err_out = np.abs(w_out[ids_dev].cpu().numpy() - V).max()
    assert err_in <= EMB_TOL and err_out <= EMB_TOL, (err_in, err_out)

    # what the step moved, row by row (oracle values): every center row, and every output row
    # that received exactly one contribution, moved by at least 20 x the tolerance.  An output
    # row can move less only where contributions of opposite sign met (a node that is context
    # in one slot and negative in another slot of the same center): those rows are counted.
    is_center = np.zeros(len(ids), dtype=bool)
    is_center[cc[cc >= 0]] = True
    pair_ok = cc >= 0
    hits = np.bincount(oo[pair_ok], minlength=len(ids))
    negs = nn[pair_ok]
    negs = negs[(negs >= 0) & (negs != oo[pair_ok][:, None])]
    hits += np.bincount(negs, minlength=len(ids))
    moved_in = np.abs(U - U0).max(axis=1)
    moved_out = np.abs(V - V0).max(axis=1)
    min_in = moved_in[is_center].min()
    min_single = moved_out[hits == 1].min()
    small = int(((hits > 0) & (moved_out < 20 * EMB_TOL)).sum())
    print(f"{wl.name} base {sub_base}: {len(ids)} rows touched, ids {ids.min()}..{ids.max()}; smallest move "
          f"of a center row {min_in:.2e}, of an output row hit once {min_single:.2e}; "
          f"{small} of {int((hits > 0).sum())} output rows moved less than 20 x tol; "
          f"errors {err_in:.1e} / {err_out:.1e}")
    assert min_in >= 20 * EMB_TOL and min_single >= 20 * EMB_TOL
    assert small <= 1e-3 * (hits > 0).sum()
    assert np.array_equal(moved_in > 0, is_center) and np.array_equal(moved_out > 0, hits > 0)
    for lo, outside, before_in, before_out in keep:
        assert torch.equal(w_in[lo:lo + win][outside], before_in[outside]), lo
        assert torch.equal(w_out[lo:lo + win][outside], before_out[outside]), lo


@pytest.mark.parametrize("name", ["deepwalk_medium", "node2vec_4m", "deepwalk_large", "rmat_billion"])
def test_fullsize_workload(name):
    wl = WL.WORKLOADS[name]
    torch.cuda.empty_cache()
    g = wl.make_graph(device=DEV)
    n = g.n_nodes
    assert n == wl.n_nodes
    # the graph handle bench.py uses: walk index, and the hashed edge set for node2vec
    flags = B.GS_VALIDATE | B.GS_REQUIRE_SORTED | B.GS_BUILD_WALK_INDEX
    if wl.walk_kind != "uniform":
        flags |= B.GS_BUILD_EDGE_SET
    G = B.gs_graph_load_csr(g.offsets, g.cols, flags)
    deg = g.degrees()
    assert G.info()["max_degree"] == int(deg.max())
    off = g.offsets.cpu().numpy().astype(np.int64)
    col = g.cols.cpu().numpy()
    seed = wl.graph_seed

    # ---- alias table: product builder == oracle builder, bit for bit, at full size
    degf = deg.cpu().numpy().astype(np.float64)
    table = B.gs_build_alias(degf, 0.75)
    thr, alias = O.build_alias(degf, 0.75)
    t2, a2 = unpack_alias(table)
    assert np.array_equal(t2, thr) and np.array_equal(a2, alias)
    del t2, a2, degf
    a_dev = torch.from_numpy(table.view(np.int64)).to(DEV)

    # ---- walks of one bench-sized batch from the middle of the epoch
    total = n * wl.walks_per_node
    bw = min(1 << 20, total)
    base = ((total // bw) // 2) * bw
    steps = torch.zeros(1, dtype=torch.int64, device=DEV)
    caps = torch.zeros(1, dtype=torch.int64, device=DEV)
    if wl.walk_kind == "uniform":
        walks = B.gs_random_walks(G, None, bw, base, wl.walk_len, seed, steps=steps)
    else:
        walks = B.gs_node2vec_walks(G, None, bw, base, wl.walk_len, seed, wl.p, wl.q,
                                    steps=steps, cap_hits=caps)
    torch.cuda.synchronize()
    assert int(steps.item()) == int((walks[:, 1:] >= 0).sum())
    assert int(caps.item()) == 0
    assert torch.equal(walks[:, 0].to(torch.int64),
                       (torch.arange(base, base + bw, device=DEV) % n))
    for lo in (0, bw // 2 - 333, bw - 1024):
        if wl.walk_kind == "uniform":
            want, _ = O.uniform_walks(off, col, None, 1024, base + lo, wl.walk_len, seed)
        else:
            want, _, _ = O.node2vec_walks(off, col, None, 1024, base + lo, wl.walk_len, seed, wl.p, wl.q)
        assert np.array_equal(walks[lo:lo + 1024].cpu().numpy(), want), lo

    # ---- corpus variants at full size: shuffled start order is a bijection of all nodes and
    # matches the oracle on sampled ranges; sub-sampled walks match the oracle on sampled ranges
    starts_all = B.gs_shuffled_starts(n, seed, 3, 0, n, DEV)
    assert int(torch.bincount(starts_all.to(torch.int64), minlength=n).max()) == 1
    for lo in (0, n // 2 - 77, n - 4096):
        assert np.array_equal(starts_all[lo:lo + 4096].cpu().numpy(), O.shuffled_starts(n, seed, 3, lo, 4096))
    del starts_all
    degf = deg.cpu().numpy().astype(np.float64)
    keep_thr = B.gs_build_keep_thresholds(degf, 1e-6)
    assert np.array_equal(keep_thr, O.keep_thresholds(degf, 1e-6))
    del degf
    kept = torch.zeros(1, dtype=torch.int64, device=DEV)
    thinned = B.gs_subsample_walks(walks, base, torch.from_numpy(keep_thr.view(np.int32)).to(DEV), seed, kept=kept)
    assert int(kept.item()) == int((thinned >= 0).sum()) < int((walks >= 0).sum())
    for lo in (0, bw // 2 - 333, bw - 1024):
        want, _ = O.subsample_walks(walks[lo:lo + 1024].cpu().numpy(), base + lo, keep_thr, seed)
        assert np.array_equal(thinned[lo:lo + 1024].cpu().numpy(), want), lo
    del thinned, keep_thr

    # ---- tables; one lock-free step on the whole batch (makes the output rows non-zero)
    w_in = torch.empty((n, wl.dim), dtype=torch.float32, device=DEV)
    w_out = torch.empty_like(w_in)
    B.gs_init_embeddings(w_in, w_out, seed)
    probe = torch.from_numpy(np.random.default_rng(0).integers(0, n, 64)).to(DEV)
    assert np.array_equal(w_in[probe].cpu().numpy().astype(np.float64),
                          O.init_rows(probe.cpu().numpy(), wl.dim, seed))
    loss = torch.zeros(1, dtype=torch.float64, device=DEV)
    cnt = torch.zeros(1, dtype=torch.int64, device=DEV)
    B.gs_sgns_step(w_in, w_out, walks, base, wl.window, wl.n_neg, a_dev, wl.lr0, seed,
                   B.GS_HOGWILD, loss, cnt)
    torch.cuda.synchronize()
    assert int(cnt.item()) == count_pairs(walks, wl.window)
    per_pair = loss.item() / cnt.item()
    assert 0.3 < per_pair <= (1 + wl.n_neg) * np.log(2) * (1 + 1e-6)

    # ---- synchronous step on 512 walks against the oracle on the touched rows: once in the middle
    # of the epoch and once on the epoch's last 512 walk ids, whose start nodes are the last rows
    # of the tables
    check_synchronous_step(wl, w_in, w_out, walks[4096:4096 + 512].contiguous(), base + 4096, a_dev,
                           thr, alias, seed)
    last = total - 512
    if wl.walk_kind == "uniform":
        tail = B.gs_random_walks(G, None, 512, last, wl.walk_len, seed)
        want, _ = O.uniform_walks(off, col, None, 512, last, wl.walk_len, seed)
    else:
        tail = B.gs_node2vec_walks(G, None, 512, last, wl.walk_len, seed, wl.p, wl.q)
        want, _, _ = O.node2vec_walks(off, col, None, 512, last, wl.walk_len, seed, wl.p, wl.q)
    assert np.array_equal(tail.cpu().numpy(), want)
    assert int(tail[-1, 0]) == n - 1
    check_synchronous_step(wl, w_in, w_out, tail, last, a_dev, thr, alias, seed)

    G.close()
    del w_in, w_out, walks, g, a_dev
    B.gs_release_workspace()
    torch.cuda.empty_cache()


@pytest.mark.parametrize("name,nb,lr_mult,tol", [("node2vec_4m", 8, 1, 1e-6), ("deepwalk_large", 8, 1, 1e-6),
                                                 ("rmat_billion", 16, 1, 1e-6),
                                                 ("deepwalk_medium", 48, 2, 1e-4)])
def test_truncated_epoch_on_touched_rows_matches_the_oracle(name, nb, lr_mult, tol):
    # The first nb 512-walk batches of the epoch through the epoch driver at full size (walks generated
    # by the driver, the table-independent part of batch b+1 overlapping the update of batch b),
    # against the oracle run batch by batch on the rows these batches touch (fp64; the rows'
    # start values come from the oracle's own table initialisation): walk steps, pairs and masked
    # negatives equal, mean loss within 1e-3, every touched value within 1e-6 (the rows are still
    # small this early in training, so the bar is a hundredth of the usual one).
    # The 1M-node workload runs 48 batches at twice its learning rate, in two calls (40 + 8), so
    # that the rows grow (values up to about 1) and the mean loss of the last eight batches has left
    # its start value (1 + K) ln 2 = 4.159; there the bar is the usual 1e-4.
    wl = WL.WORKLOADS[name]
    lr = wl.lr0 * lr_mult
    torch.cuda.empty_cache()
    g = wl.make_graph(device=DEV)
    n, seed, bw = g.n_nodes, wl.graph_seed, 512
    off = g.offsets.cpu().numpy().astype(np.int64)
    col = g.cols.cpu().numpy()
    thr, alias = O.build_alias((off[1:] - off[:-1]).astype(np.float64), 0.75)
    # ---- oracle side: walks and lists of every batch, then the union of the rows they touch
    batches, steps_o = [], 0
    for b in range(nb):
        if wl.walk_kind == "uniform":
            walks, st = O.uniform_walks(off, col, None, bw, b * bw, wl.walk_len, seed)
        else:
            walks, st, _ = O.node2vec_walks(off, col, None, bw, b * bw, wl.walk_len, seed, wl.p, wl.q)
        steps_o += st
        batches.append(O.expand_lists(walks, b * bw, wl.window, wl.n_neg, thr, alias, seed)[:3])
    union = np.unique(np.concatenate([np.concatenate([c, o, ng.ravel()]) for c, o, ng in batches]))
    union = union[union >= 0]
    U = O.init_rows(union, wl.dim, seed)
    V = np.zeros_like(U)
    loss_o, pairs_o, masked_o = 0.0, 0, 0
    tail_from = nb - 8 if lr_mult > 1 else nb                     # batches of the second call
    loss_tail, pairs_tail = 0.0, 0
    for b, (c, o, ng) in enumerate(batches):
        ids, cc, oo, nn = compact_problem(c, o, ng)              # this batch's rows, renumbered
        at = np.searchsorted(union, ids)
        Ub, Vb = np.ascontiguousarray(U[at]), np.ascontiguousarray(V[at])
        ls, pc = O.sgns_det_from_lists(Ub, Vb, cc, oo, nn, lr)
        U[at], V[at] = Ub, Vb
        loss_o += ls
        pairs_o += pc
        if b >= tail_from:
            loss_tail += ls
            pairs_tail += pc
        masked_o += int(((ng == o[:, None]) & (c >= 0)[:, None]).sum())
    # ---- the library
    flags = B.GS_VALIDATE | B.GS_REQUIRE_SORTED | B.GS_BUILD_WALK_INDEX
    if wl.walk_kind != "uniform":
        flags |= B.GS_BUILD_EDGE_SET
    G = B.gs_graph_load_csr(g.offsets, g.cols, flags)
    w_in = torch.empty((n, wl.dim), dtype=torch.float32, device=DEV)
    w_out = torch.empty_like(w_in)
    B.gs_init_embeddings(w_in, w_out, seed)
    table = (alias.astype(np.uint64) << np.uint64(32)) | thr.astype(np.uint64)
    kind = B.GS_WALK_UNIFORM if wl.walk_kind == "uniform" else B.GS_WALK_NODE2VEC
    a_dev = torch.from_numpy(table.view(np.int64)).to(DEV)
    kw = dict(walks_per_node=wl.walks_per_node, walk_len=wl.walk_len, window=wl.window, n_neg=wl.n_neg,
              lr0=lr, batch_walks=bw, seed=seed, mode=B.GS_DETERMINISTIC, walk_kind=kind, p=wl.p, q=wl.q)
    res = B.gs_sgns_epoch(G, a_dev, w_in, w_out, num_batches=tail_from, **kw)
    if tail_from < nb:                                            # the rest in a second call
        more = B.gs_sgns_epoch(G, a_dev, w_in, w_out, first_batch=tail_from, num_batches=nb - tail_from, **kw)
        assert (more.pairs, more.batches) == (pairs_tail, nb - tail_from)
        assert abs(more.loss_sum - loss_tail) <= 1e-3 * loss_tail
        assert more.loss_sum / more.pairs < 0.97 * (1 + wl.n_neg) * np.log(2.0)   # the loss has left its start value
        for f in ("pairs", "steps", "masked_negs", "batches", "refused_ids", "loss_sum"):
            setattr(res, f, getattr(res, f) + getattr(more, f))
    assert (res.pairs, res.steps, res.masked_negs, res.batches, res.refused_ids) == (pairs_o, steps_o, masked_o, nb, 0)
    assert abs(res.loss_sum - loss_o) <= 1e-3 * loss_o
    rel = abs(res.loss_sum - loss_o) / loss_o
    rows = torch.from_numpy(union).to(DEV)
    err_in = np.abs(w_in[rows].cpu().numpy() - U).max()
    err_out = np.abs(w_out[rows].cpu().numpy() - V).max()
    print(f"{name}: {nb} batches, {len(union)} rows touched, loss {res.loss_sum / res.pairs:.5f} (rel. diff {rel:.1e}), "
          f"largest output value {np.abs(V).max():.2e}, errors {err_in:.1e} / {err_out:.1e}")
    assert err_in <= tol and err_out <= tol, (err_in, err_out)
    assert np.abs(V).max() > 1e3 * tol                            # the batches did move the rows
    G.close()
    del w_in, w_out, g
    B.gs_release_workspace()
    torch.cuda.empty_cache()


def test_truncated_epoch_of_the_medium_workload_matches_the_oracle():
    # The first eight 512-walk batches of the 1M-node workload through the epoch driver against the
    # oracle's epoch on dense fp64 tables (2 x 1 GB on the host): pair, step and masked counts equal,
    # mean loss within 1e-3, every table value within 1e-4.
    wl = WL.WORKLOADS["deepwalk_medium"]
    torch.cuda.empty_cache()
    g = wl.make_graph(device=DEV)
    n, nb, seed = g.n_nodes, 8, wl.graph_seed
    off = g.offsets.cpu().numpy().astype(np.int64)
    col = g.cols.cpu().numpy()
    thr, alias = O.build_alias((off[1:] - off[:-1]).astype(np.float64), 0.75)
    U = O.init_rows(np.arange(n), wl.dim, seed)
    V = np.zeros_like(U)
    want = O.sgns_epoch(off, col, thr, alias, U, V, walks_per_node=wl.walks_per_node, L=wl.walk_len,
                        w=wl.window, K=wl.n_neg, lr0=wl.lr0, schedule="constant", batch_walks=512,
                        seed=seed, num_batches=nb)
    G = B.gs_graph_load_csr(g.offsets, g.cols, B.GS_VALIDATE | B.GS_REQUIRE_SORTED | B.GS_BUILD_WALK_INDEX)
    w_in = torch.empty((n, wl.dim), dtype=torch.float32, device=DEV)
    w_out = torch.empty_like(w_in)
    B.gs_init_embeddings(w_in, w_out, seed)
    table = (alias.astype(np.uint64) << np.uint64(32)) | thr.astype(np.uint64)
    res = B.gs_sgns_epoch(G, torch.from_numpy(table.view(np.int64)).to(DEV), w_in, w_out,
                          walks_per_node=wl.walks_per_node, walk_len=wl.walk_len, window=wl.window,
                          n_neg=wl.n_neg, lr0=wl.lr0, batch_walks=512, seed=seed, mode=B.GS_DETERMINISTIC,
                          num_batches=nb)
    assert (res.pairs, res.steps, res.masked_negs, res.batches) == (want["pairs"], want["steps"],
                                                                   want["masked_negs"], nb)
    assert abs(res.loss_sum - want["loss_sum"]) <= 1e-3 * want["loss_sum"]
    # early in training the rows are small (start values within 0.5/128, eight batches move the
    # output rows by up to 5e-3), so the 1e-4 bar says little here: ask for 1e-6, a thousandth of
    # what the rows moved
    err_in = np.abs(w_in.cpu().numpy() - U).max()
    err_out = np.abs(w_out.cpu().numpy() - V).max()
    assert err_in <= 1e-6 and err_out <= 1e-6, (err_in, err_out)
    assert np.abs(V).max() > 1e-3
    G.close()
    B.gs_release_workspace()


@pytest.mark.parametrize("fmt", ["f16", "bf16"])
def test_16bit_tables_at_the_largest_table_size(fmt):
    # Tables of the 50M-node workload stored in a 16-bit format: 12.8 GB each, so the byte offset of
    # a row passes 2^32 after a third of the table.  Start values checked on sampled rows across the
    # whole table; a synchronous step of the epoch's last 512 walks (their start nodes are the last
    # rows) against the oracle on the touched rows, seeded so that the step moves them: every value
    # within one unit of the format and all but a few per cent bit-equal, rows outside the batch in
    # three windows of a million rows keep their bits; then the whole batch through the lock-free
    # kernel: pair count and a loss in the expected range.
    wl = WL.WORKLOADS["deepwalk_large"]
    torch.cuda.empty_cache()
    tdt = torch.float16 if fmt == "f16" else torch.bfloat16
    init = B.gs_init_embeddings_f16 if fmt == "f16" else B.gs_init_embeddings_bf16
    step = B.gs_sgns_step_f16 if fmt == "f16" else B.gs_sgns_step_bf16
    rnd = O.round_f16 if fmt == "f16" else O.round_bf16
    det = O.sgns_det_f16_from_lists if fmt == "f16" else O.sgns_det_bf16_from_lists
    frac_bits = 10 if fmt == "f16" else 7

    def unit(x):                                    # spacing of the format at |x| (normal range)
        return 2.0 ** (np.floor(np.log2(np.maximum(np.abs(x), 2.0 ** -14))) - frac_bits)

    g = wl.make_graph(device=DEV)
    n, seed = g.n_nodes, wl.graph_seed
    off = g.offsets.cpu().numpy().astype(np.int64)
    col = g.cols.cpu().numpy()
    thr, alias = O.build_alias((off[1:] - off[:-1]).astype(np.float64), 0.75)
    table = (alias.astype(np.uint64) << np.uint64(32)) | thr.astype(np.uint64)
    a_dev = torch.from_numpy(table.view(np.int64)).to(DEV)
    G = B.gs_graph_load_csr(g.offsets, g.cols, B.GS_VALIDATE | B.GS_REQUIRE_SORTED | B.GS_BUILD_WALK_INDEX)
    w_in = torch.empty((n, wl.dim), dtype=tdt, device=DEV)
    w_out = torch.empty_like(w_in)
    assert w_in.numel() * 2 > 1 << 33
    init(w_in, w_out, seed)
    probe = np.concatenate([np.random.default_rng(1).integers(0, n, 61), [0, n // 3 + 1, n - 1]])
    got = w_in[torch.from_numpy(probe).to(DEV)].float().cpu().numpy().astype(np.float64)
    assert np.array_equal(got, rnd(O.init_rows(probe, wl.dim, seed)))

    total = n * wl.walks_per_node
    last = total - 512
    tail = B.gs_random_walks(G, None, 512, last, wl.walk_len, seed)
    tail_h = tail.cpu().numpy()
    want, _ = O.uniform_walks(off, col, None, 512, last, wl.walk_len, seed)
    assert np.array_equal(tail_h, want) and int(tail_h[-1, 0]) == n - 1
    c, o, ng, n_pairs = O.expand_lists(tail_h, last, wl.window, wl.n_neg, thr, alias, seed)
    ids, cc, oo, nn = compact_problem(c, o, ng)
    assert ids.max() == n - 1 and (ids > n // 3).any()
    ids_dev = torch.from_numpy(ids).to(DEV)
    gen = torch.Generator().manual_seed(99)
    u0 = ((torch.rand((len(ids), wl.dim), generator=gen) - 0.5) * 0.6).to(tdt)
    v0 = ((torch.rand((len(ids), wl.dim), generator=gen) - 0.5) * 0.15).to(tdt)
    w_in[ids_dev] = u0.to(DEV)
    w_out[ids_dev] = v0.to(DEV)
    U, V = u0.float().numpy().astype(np.float64), v0.float().numpy().astype(np.float64)
    U0, V0 = U.copy(), V.copy()
    win = 1 << 20
    keep = []
    for lo in (0, n // 2 - win // 2, n - win):
        outside = torch.ones(win, dtype=torch.bool, device=DEV)
        outside[ids_dev[(ids_dev >= lo) & (ids_dev < lo + win)] - lo] = False
        keep.append((lo, outside, w_in[lo:lo + win].clone(), w_out[lo:lo + win].clone()))
    lr = 4 * wl.lr0                                  # so that most written values change in 16 bits
    loss_o, cnt_o = det(U, V, cc, oo, nn, lr)
    loss = torch.zeros(1, dtype=torch.float64, device=DEV)
    cnt = torch.zeros(1, dtype=torch.int64, device=DEV)
    step(w_in, w_out, tail, last, wl.window, wl.n_neg, a_dev, lr, seed, B.GS_DETERMINISTIC, loss, cnt)
    torch.cuda.synchronize()
    assert int(cnt.item()) == cnt_o == n_pairs > 0
    assert abs(loss.item() - loss_o) <= 2e-6 * abs(loss_o)
    for name, tab, want_rows, before in (("in", w_in, U, U0), ("out", w_out, V, V0)):
        got = tab[ids_dev].float().cpu().numpy().astype(np.float64)
        diff = np.abs(got - want_rows)
        assert (diff <= unit(want_rows) * 1.0001 + 1e-6).all(), (name, float((diff / unit(want_rows)).max()))
        assert np.mean(diff > 0) <= 0.02, (name, float(np.mean(diff > 0)))
        touched = (want_rows != before).any(axis=1)
        assert np.mean((got != before)[touched]) > 0.5, name      # the step is not lost in the rounding
    for lo, outside, before_in, before_out in keep:
        assert torch.equal(w_in[lo:lo + win][outside], before_in[outside]), lo
        assert torch.equal(w_out[lo:lo + win][outside], before_out[outside]), lo
    del keep

    bw = 1 << 20
    base = ((total // bw) // 2) * bw
    walks = B.gs_random_walks(G, None, bw, base, wl.walk_len, seed)
    loss.zero_()
    cnt.zero_()
    step(w_in, w_out, walks, base, wl.window, wl.n_neg, a_dev, wl.lr0, seed, B.GS_HOGWILD, loss, cnt)
    torch.cuda.synchronize()
    assert int(cnt.item()) == count_pairs(walks, wl.window)
    assert 0.3 < loss.item() / cnt.item() <= (1 + wl.n_neg) * np.log(2) * (1 + 1e-3)
    assert bool(torch.isfinite(w_out[ids_dev].float()).all())
    G.close()
    del w_in, w_out, walks, g, a_dev
    B.gs_release_workspace()
    torch.cuda.empty_cache()
