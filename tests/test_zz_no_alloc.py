"""The allocation-free SGNS step (gs_sgns_step_static) against the regular deterministic step.

Some callers of this library cannot allocate device memory while they run (their memory
budget is fully handed out, or an allocation's implicit device-wide wait is not acceptable in
their loop, or their framework owns the allocator).  For them the library offers a variant
whose scratch is a fixed array inside the library.  It runs the same code as
gs_sgns_step(GS_DETERMINISTIC) on that array, so tables, loss and pair count must equal that
step's bit for bit - checked here on two calls in a row (the second one smaller, so it runs
over the first one's leftovers) - and must agree with the CPU oracle within the tolerance of
the other synchronous-step tests.  Free device memory must not move across a call, also after
the library's own scratch cache has been released, and the size limit must be reported as an
error, not hit as a fault.

Collected last on purpose: a failure here cannot hide the result of any other test."""
import numpy as np
import pytest
import torch

from oracle import gs_oracle as O
from paper_2407_15452_b200 import binding as B
from paper_2407_15452_b200 import workloads as WL
from tests.helpers import unpack_alias

pytestmark = pytest.mark.gpu
DEV = "cuda"
EMB_TOL = 1e-4


def test_static_scratch_step_matches_regular_step_twice_in_a_row():
    g = WL.chung_lu_graph(30000, 12, 2.3, seed=21)
    G = B.gs_graph_load_csr(g.offsets.to(DEV), g.cols.to(DEV), B.GS_VALIDATE)
    deg = g.degrees().numpy().astype(np.float64)
    table = B.gs_build_alias(deg, 0.75)
    thr, alias_h = unpack_alias(table)
    alias = torch.from_numpy(table.view(np.int64)).to(DEV)
    dim, L, w, K, seed = 128, 40, 5, 5, 3
    w_in_a = torch.empty((g.n_nodes, dim), dtype=torch.float32, device=DEV)
    w_out_a = torch.empty_like(w_in_a)
    B.gs_init_embeddings(w_in_a, w_out_a, seed)
    w_in_a.mul_(40.0)                                   # values of order 0.1: one step moves rows
    w_out_a.copy_(w_in_a.roll(1, 0))                    # by much more than the tolerance
    w_in_b, w_out_b = w_in_a.clone(), w_out_a.clone()
    U = w_in_a.cpu().numpy().astype(np.float64)         # the oracle's tables
    V = w_out_a.cpu().numpy().astype(np.float64)
    start_out = V.copy()
    for n_walks, base in ((300, 0), (77, 300)):         # second call: smaller, over stale scratch
        walks = B.gs_random_walks(G, None, n_walks, base, L, seed)
        la = torch.zeros(1, dtype=torch.float64, device=DEV)
        ca = torch.zeros(1, dtype=torch.int64, device=DEV)
        lb, cb = torch.zeros_like(la), torch.zeros_like(ca)
        B.gs_sgns_step(w_in_a, w_out_a, walks, base, w, K, alias, 0.025, seed, B.GS_DETERMINISTIC, la, ca)
        B.gs_sgns_step_static(w_in_b, w_out_b, walks, base, w, K, alias, 0.025, seed, lb, cb)
        torch.cuda.synchronize()
        # the same code on other scratch: the same bits
        assert ca.item() == cb.item() > 0
        assert la.item() == lb.item()
        assert torch.equal(w_in_a, w_in_b) and torch.equal(w_out_a, w_out_b)
        # and the CPU oracle's synchronous step on the same walks
        c, o, ng, n_pairs = O.expand_lists(walks.cpu().numpy(), base, w, K, thr, alias_h, seed)
        loss_o, cnt_o = O.sgns_det_from_lists(U, V, c, o, ng, 0.025)
        assert cb.item() == cnt_o == n_pairs
        assert abs(lb.item() - loss_o) <= 2e-6 * abs(loss_o)
        assert np.abs(w_in_b.cpu().numpy() - U).max() <= EMB_TOL
        assert np.abs(w_out_b.cpu().numpy() - V).max() <= EMB_TOL
    assert np.abs(V - start_out).max() > 20 * EMB_TOL   # the steps moved rows far beyond the tolerance


def test_static_scratch_step_leaves_free_device_memory_unchanged():
    # After one set-up call (which loads the library's device code and looks up the array), a call
    # must not change the amount of free device memory - not even when the library's growing
    # scratch cache, which the regular step would refill, has just been released.
    g = WL.chung_lu_graph(5000, 10, 2.3, seed=5)
    G = B.gs_graph_load_csr(g.offsets.to(DEV), g.cols.to(DEV), B.GS_VALIDATE)
    alias = torch.from_numpy(B.gs_build_alias(g.degrees().numpy().astype(np.float64), 0.75)
                             .view(np.int64)).to(DEV)
    dim, L, w, K, seed = 64, 20, 5, 5, 9
    w_in = torch.empty((g.n_nodes, dim), dtype=torch.float32, device=DEV)
    w_out = torch.empty_like(w_in)
    B.gs_init_embeddings(w_in, w_out, seed)
    walks = B.gs_random_walks(G, None, 200, 0, L, seed)
    loss = torch.zeros(1, dtype=torch.float64, device=DEV)
    cnt = torch.zeros(1, dtype=torch.int64, device=DEV)
    B.gs_sgns_step_static(w_in, w_out, walks, 0, w, K, alias, 0.025, seed, loss, cnt)   # set-up call
    torch.cuda.synchronize()
    B.gs_release_workspace()                            # the growing cache is empty now
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    for _ in range(3):
        B.gs_sgns_step_static(w_in, w_out, walks, 0, w, K, alias, 0.025, seed, loss, cnt)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before
    assert cnt.item() > 0 and torch.isfinite(w_out).all()


def test_static_scratch_step_rejects_batches_beyond_its_fixed_array():
    n, dim = 1000, 128
    w_in = torch.zeros((n, dim), dtype=torch.float32, device=DEV)
    w_out = torch.zeros_like(w_in)
    walks = torch.zeros((4096, 40), dtype=torch.int32, device=DEV)
    alias = torch.zeros(n, dtype=torch.int64, device=DEV)
    with pytest.raises(B.GsError) as e:
        B.gs_sgns_step_static(w_in, w_out, walks, 0, 5, 5, alias, 0.025, 0)
    assert e.value.status == -6 and "bytes of scratch" in str(e.value)
    assert not w_in.any() and not w_out.any()
