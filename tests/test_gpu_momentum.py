"""GPU parity of the momentum step (lazy per-row updates) against the oracle's dense definition:
every row of both tables gets m <- mu m (+ grad), w <- w - lr m in every iteration."""
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


def run_gpu(g_tensors, thr, alias, U0, V0, batches, L, w, K, lr, mu, seed, flush_at):
    n, dim = U0.shape
    w_in = torch.from_numpy(U0.astype(np.float32)).to(DEV)
    w_out = torch.from_numpy(V0.astype(np.float32)).to(DEV)
    m_in, m_out = torch.zeros_like(w_in), torch.zeros_like(w_out)
    last_in = torch.zeros(n, dtype=torch.int32, device=DEV)
    last_out = torch.zeros_like(last_in)
    a_dev = alias_to_device(thr, alias)
    loss = torch.zeros(1, dtype=torch.float64, device=DEV)
    cnt = torch.zeros(1, dtype=torch.int64, device=DEV)
    losses = []
    for it, (walks, base) in enumerate(batches):
        loss.zero_()
        B.gs_sgns_step_momentum(w_in, w_out, m_in, m_out, last_in, last_out,
                                torch.from_numpy(walks).to(DEV), base, w, K, a_dev, lr, mu, it, seed,
                                loss, cnt)
        losses.append(loss.item())
    B.gs_momentum_flush(w_in, m_in, last_in, lr, mu, flush_at)
    B.gs_momentum_flush(w_out, m_out, last_out, lr, mu, flush_at)
    torch.cuda.synchronize()
    return w_in, w_out, m_in, m_out, last_in, last_out, losses, cnt.item()


@pytest.mark.parametrize("dim,mu", [(128, 0.9), (64, 0.5), (32, 0.0)])
def test_momentum_steps_match_dense_oracle(dim, mu):
    wl = WL.WORKLOADS["tiny_deepwalk"]
    g = wl.make_graph(scale=0.3)                       # 3000 nodes: rows are hit in some iterations only
    off, col = np_graph(g)
    thr, alias = degree_alias(off)
    n = g.n_nodes
    L, w, K, lr, seed = 12, 3, 4, 0.02, 5
    rng = np.random.default_rng(0)
    U0 = (rng.random((n, dim)) - 0.5) * 0.4
    V0 = (rng.random((n, dim)) - 0.5) * 0.4
    U0, V0 = U0.astype(np.float32).astype(np.float64), V0.astype(np.float32).astype(np.float64)
    batches = []
    for it in range(7):
        base = 100 + 150 * it
        walks, _ = O.uniform_walks(off, col, None, 150, base, L, seed)
        batches.append((walks, base))
    # oracle: dense definition
    U, V = U0.copy(), V0.copy()
    MU, MV = np.zeros_like(U), np.zeros_like(V)
    want_losses, pairs = [], 0
    for walks, base in batches:
        c, o, ng, _ = O.expand_lists(walks, base, w, K, thr, alias, seed)
        ls, pc = O.sgns_momentum_step_from_lists(U, V, MU, MV, c, o, ng, lr, mu)
        want_losses.append(ls)
        pairs += pc
    # two more iterations without any batch (the flush below must account for them)
    zero = np.zeros_like(U)
    for _ in range(2):
        O.momentum_update(U, MU, zero, lr, mu)
        O.momentum_update(V, MV, zero, lr, mu)
    w_in, w_out, m_in, m_out, last_in, last_out, losses, cnt = run_gpu(
        None, thr, alias, U0, V0, batches, L, w, K, lr, mu, seed, flush_at=len(batches) + 2)
    assert cnt == pairs
    for a, b in zip(losses, want_losses):
        assert abs(a - b) <= 2e-5 * abs(b)
    assert np.abs(w_in.cpu().numpy() - U).max() <= EMB_TOL
    assert np.abs(w_out.cpu().numpy() - V).max() <= EMB_TOL
    assert np.abs(m_in.cpu().numpy() - MU).max() <= EMB_TOL
    assert np.abs(m_out.cpu().numpy() - MV).max() <= EMB_TOL
    assert (last_in == len(batches) + 2).all() and (last_out == len(batches) + 2).all()
    # the run moved the tables by far more than the tolerance, and momentum mattered
    assert np.abs(V - V0).max() > 50 * EMB_TOL
    if mu > 0:
        assert np.abs(MV).max() > 50 * EMB_TOL
    # bitwise reproducible
    again = run_gpu(None, thr, alias, U0, V0, batches, L, w, K, lr, mu, seed, flush_at=len(batches) + 2)
    assert torch.equal(again[0], w_in) and torch.equal(again[1], w_out)
    assert torch.equal(again[2], m_in) and torch.equal(again[3], m_out)


def test_zero_momentum_equals_plain_synchronous_step():
    g = WL.chung_lu_graph(5000, 8, 2.4, seed=2)
    off, col = np_graph(g)
    thr, alias = degree_alias(off)
    n, dim, L, w, K = g.n_nodes, 128, 20, 5, 5
    walks, _ = O.uniform_walks(off, col, None, 256, 0, L, 1)
    gen = torch.Generator().manual_seed(3)
    w_in0 = ((torch.rand((n, dim), generator=gen) - 0.5) * 0.3)
    w_out0 = ((torch.rand((n, dim), generator=gen) - 0.5) * 0.3)
    a_dev = alias_to_device(thr, alias)
    wd = torch.from_numpy(walks).to(DEV)
    a_in, a_out = w_in0.to(DEV), w_out0.to(DEV)
    B.gs_sgns_step(a_in, a_out, wd, 0, w, K, a_dev, 0.025, 1, B.GS_DETERMINISTIC)
    b_in, b_out = w_in0.to(DEV), w_out0.to(DEV)
    m_in, m_out = torch.zeros_like(b_in), torch.zeros_like(b_out)
    l_in = torch.zeros(n, dtype=torch.int32, device=DEV)
    l_out = torch.zeros_like(l_in)
    B.gs_sgns_step_momentum(b_in, b_out, m_in, m_out, l_in, l_out, wd, 0, w, K, a_dev, 0.025, 0.0, 0, 1)
    torch.cuda.synchronize()
    assert (a_in - b_in).abs().max().item() <= 1e-7 and (a_out - b_out).abs().max().item() <= 1e-7
    with pytest.raises(B.GsError):
        B.gs_sgns_step_momentum(b_in, b_out, m_in, m_out, l_in, l_out, wd, 0, w, K, a_dev, 0.025, 1.0, 1, 1)
