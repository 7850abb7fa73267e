"""GPU parity with tables stored as bfloat16 (fp32 arithmetic, round-to-nearest-even write-back).

The oracle computes in fp64 and rounds a written value once to bfloat16 (8 significant bits); the
kernels compute in fp32 (fp64 accumulators in the synchronous apply pass) and round that.  The
two can land on different sides of a rounding boundary, so the bar is: no element differs by
more than one bfloat16 ulp at its magnitude and all but a small fraction are bit-equal."""
import numpy as np
import pytest
import torch

from oracle import gs_oracle as O
from paper_2407_15452_b200 import binding as B
from paper_2407_15452_b200 import workloads as WL
from tests.helpers import alias_to_device, degree_alias, np_graph

pytestmark = pytest.mark.gpu
DEV = "cuda"


def ulp_bf16(x):
    """Spacing of bfloat16 at |x| (normal range)."""
    a = np.maximum(np.abs(x), 2.0 ** -120)
    return 2.0 ** (np.floor(np.log2(a)) - 7)


def to_f64(t):
    return t.cpu().to(torch.float64).numpy()


def bf16_tables(n, dim, seed, scale=0.5):
    gen = torch.Generator().manual_seed(seed)
    a = ((torch.rand((n, dim), generator=gen) - 0.5) * scale).to(torch.bfloat16)
    b = ((torch.rand((n, dim), generator=gen) - 0.5) * scale).to(torch.bfloat16)
    return a, b


@pytest.fixture(scope="module")
def tiny():
    wl = WL.WORKLOADS["tiny_deepwalk"]
    g = wl.make_graph()
    off, col = np_graph(g)
    thr, alias = degree_alias(off)
    return g, off, col, thr, alias


@pytest.mark.parametrize("dim", [64, 128, 256])
def test_initial_tables_are_the_rounded_start_values(dim):
    n = 3000
    w_in = torch.empty((n, dim), dtype=torch.bfloat16, device=DEV)
    w_out = torch.ones((n, dim), dtype=torch.bfloat16, device=DEV)
    B.gs_init_embeddings_bf16(w_in, w_out, 9)
    want = O.round_bf16(O.init_rows(np.arange(n), dim, 9))
    assert np.array_equal(to_f64(w_in), want)
    assert not w_out.any()


@pytest.mark.parametrize("dim,L,w,K", [(128, 20, 5, 5), (64, 10, 3, 10), (256, 8, 2, 3)])
def test_deterministic_step_on_bfloat16_tables(tiny, dim, L, w, K):
    g, off, col, thr, alias = tiny
    n = g.n_nodes
    walks, _ = O.uniform_walks(off, col, None, 400, 10, L, 2)
    walks[7, L // 2:] = -1
    c, o, ng, n_pairs = O.expand_lists(walks, 10, w, K, thr, alias, 2)
    h_in, h_out = bf16_tables(n, dim, 1)
    U, V = to_f64(h_in), to_f64(h_out)
    U0, V0 = U.copy(), V.copy()
    lr = 0.2                                            # 8 significant bits: small steps vanish
    loss_o, cnt_o = O.sgns_det_bf16_from_lists(U, V, c, o, ng, lr)
    a_dev = alias_to_device(thr, alias)
    wd = torch.from_numpy(walks).to(DEV)
    w_in, w_out = h_in.to(DEV), h_out.to(DEV)
    loss = torch.zeros(1, dtype=torch.float64, device=DEV)
    cnt = torch.zeros(1, dtype=torch.int64, device=DEV)
    pd = torch.empty((400, L, 2 * w, 2), dtype=torch.int32, device=DEV)
    nd = torch.empty((400, L, 2 * w, K), dtype=torch.int32, device=DEV)
    B.gs_sgns_step_bf16(w_in, w_out, wd, 10, w, K, a_dev, lr, 2, B.GS_DETERMINISTIC, loss, cnt, pd, nd)
    torch.cuda.synchronize()
    pd = pd.cpu().numpy().reshape(-1, 2)
    assert np.array_equal(pd[:, 0], c) and np.array_equal(pd[:, 1], o)
    assert np.array_equal(nd.cpu().numpy().reshape(-1, K), ng)
    assert cnt.item() == cnt_o == n_pairs
    assert abs(loss.item() - loss_o) <= 2e-6 * abs(loss_o)
    # one ulp at the value's magnitude, plus the absolute fp32 noise of the unrounded value (where old
    # value and step cancel, the result is tiny and its own ulp is far below that noise)
    for got, want in ((to_f64(w_in), U), (to_f64(w_out), V)):
        diff = np.abs(got - want)
        assert (diff <= ulp_bf16(want) * 1.0001 + 1e-6).all(), float((diff / (ulp_bf16(want) + 1e-6)).max())
        assert np.mean(diff > 0) <= 0.01
    assert np.mean(V != V0) > 0.02 and np.mean(U != U0) > 0.02      # the step is not lost in the rounding
    w_in2, w_out2 = h_in.to(DEV), h_out.to(DEV)
    B.gs_sgns_step_bf16(w_in2, w_out2, wd, 10, w, K, a_dev, lr, 2, B.GS_DETERMINISTIC)
    torch.cuda.synchronize()
    assert torch.equal(w_in, w_in2) and torch.equal(w_out, w_out2)   # bitwise reproducible


@pytest.mark.parametrize("dim,L,w", [(128, 40, 5), (64, 20, 5), (256, 24, 3)])
def test_lock_free_many_walks_without_shared_rows_on_bfloat16_tables(dim, L, w):
    # no two walks share a row, no walk repeats a node, no negatives: nothing can race
    n_walks, span = 500, 64
    n = n_walks * span
    rng = np.random.default_rng(dim)
    walks = np.empty((n_walks, L), dtype=np.int32)
    for k in range(n_walks):
        walks[k] = k * span + rng.permutation(span)[:L]
    thr, alias = O.build_alias(np.ones(n), 1.0)
    c, o, ng, n_pairs = O.expand_lists(walks, 0, w, 0, thr, alias, 3)
    h_in, h_out = bf16_tables(n, dim, 6, scale=0.6)
    U, V = to_f64(h_in), to_f64(h_out)
    U0, V0 = U.copy(), V.copy()
    loss_o, cnt_o = O.sgns_seq_bf16_from_lists(U, V, c, o, ng, 2 * w, 0.2)
    w_in, w_out = h_in.to(DEV), h_out.to(DEV)
    loss = torch.zeros(1, dtype=torch.float64, device=DEV)
    cnt = torch.zeros(1, dtype=torch.int64, device=DEV)
    B.gs_sgns_step_bf16(w_in, w_out, torch.from_numpy(walks).to(DEV), 0, w, 0, None, 0.2, 3,
                        B.GS_HOGWILD, loss, cnt)
    torch.cuda.synchronize()
    assert cnt.item() == cnt_o == n_pairs and abs(loss.item() - loss_o) < 2e-3 * abs(loss_o)
    for got, want, start in ((to_f64(w_in), U, U0), (to_f64(w_out), V, V0)):
        scale = np.maximum(np.maximum(np.abs(want), np.abs(start)), 2e-2)
        assert (np.abs(got - want) <= 4 * ulp_bf16(scale)).all()
        assert np.mean(got == want) > 0.9
    assert np.mean(to_f64(w_out) != V0) > 0.3


def test_synchronous_epoch_on_bfloat16_tables_matches_the_rounded_oracle(tiny):
    g, off, col, thr, alias = tiny
    n, dim = g.n_nodes, 64
    U = O.round_bf16(O.init_rows(np.arange(n), dim, 2))
    V = np.zeros_like(U)
    U0 = U.copy()
    want = O.sgns_epoch(off, col, thr, alias, U, V, walks_per_node=1, L=10, w=5, K=5, lr0=0.1,
                        schedule="linear", batch_walks=512, seed=2, mode="det_bf16")
    G = B.gs_graph_load_csr(g.offsets.to(DEV), g.cols.to(DEV), B.GS_VALIDATE)
    w_in = torch.empty((n, dim), dtype=torch.bfloat16, device=DEV)
    w_out = torch.empty_like(w_in)
    B.gs_init_embeddings_bf16(w_in, w_out, 2)
    res = B.gs_sgns_epoch(G, alias_to_device(thr, alias), w_in, w_out, walks_per_node=1, walk_len=10,
                          window=5, n_neg=5, lr0=0.1, batch_walks=512, seed=2, mode=B.GS_DETERMINISTIC,
                          lr_schedule=B.GS_LR_LINEAR)
    assert res.pairs == want["pairs"] and res.steps == want["steps"]
    assert abs(res.loss_sum - want["loss_sum"]) <= 1e-3 * want["loss_sum"]
    for got, ref in ((w_in, U), (w_out, V)):
        got = to_f64(got)
        # A row is rewritten once per batch that touches it (hub rows in all 20 batches), and a
        # one-ulp difference of one write is a 0.4-0.8 % change of that value that feeds every later
        # gradient.  So: nearly all values bit-equal, and no value off by more than a few ulps of the
        # table's largest magnitude.
        assert np.mean(got == ref) > 0.95, float(np.mean(got == ref))
        assert np.abs(got - ref).max() <= 4 * ulp_bf16(np.abs(ref).max()), float(np.abs(got - ref).max())
    assert np.abs(V).max() > 0.01


def test_bfloat16_tables_reject_what_they_do_not_support(tiny):
    g, off, col, thr, alias = tiny
    a_dev = alias_to_device(thr, alias)
    walks = torch.zeros((4, 8), dtype=torch.int32, device=DEV)
    w32 = torch.zeros((g.n_nodes, 32), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(B.GsError) as e:
        B.gs_sgns_step_bf16(w32, w32.clone(), walks, 0, 2, 2, a_dev, 0.1, 0, B.GS_HOGWILD)
    assert e.value.status == -6
    w = torch.zeros((g.n_nodes, 64), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(B.GsError) as e:                    # the reduction unit rounds to nearest only
        B.gs_sgns_step_bf16(w, w.clone(), walks, 0, 2, 2, a_dev, 0.1, 0, B.GS_HOGWILD_RED | B.GS_ROUND_STOCHASTIC)
    assert e.value.status == -6
