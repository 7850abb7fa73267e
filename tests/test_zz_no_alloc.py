"""The allocation-free SGNS step (gs_sgns_step_static) against the regular deterministic step.

Some callers of this library cannot allocate device memory while they run (their memory
budget is fully handed out, or an allocation's implicit device-wide wait is not acceptable in
their loop, or their framework owns the allocator).  For them the library offers a variant
whose scratch is a fixed array inside the library.  It launches the same kernels in the same
order, so its tables must equal those of gs_sgns_step(GS_DETERMINISTIC) - checked here on two
calls in a row (the second one smaller, so it runs over the first one's leftovers), and the
size limit must be reported as an error, not hit as a fault.

Collected last on purpose: a failure here cannot hide the result of any other test."""
import numpy as np
import pytest
import torch

from paper_2407_15452_b200 import binding as B
from paper_2407_15452_b200 import workloads as WL

pytestmark = pytest.mark.gpu
DEV = "cuda"
EMB_TOL = 1e-4


def test_static_scratch_step_matches_regular_step_twice_in_a_row():
    g = WL.chung_lu_graph(30000, 12, 2.3, seed=21)
    G = B.gs_graph_load_csr(g.offsets.to(DEV), g.cols.to(DEV), B.GS_VALIDATE)
    deg = g.degrees().numpy().astype(np.float64)
    alias = torch.from_numpy(B.gs_build_alias(deg, 0.75).view(np.int64)).to(DEV)
    dim, L, w, K, seed = 128, 40, 5, 5, 3
    w_in_a = torch.empty((g.n_nodes, dim), dtype=torch.float32, device=DEV)
    w_out_a = torch.empty_like(w_in_a)
    B.gs_init_embeddings(w_in_a, w_out_a, seed)
    w_out_a.copy_(w_in_a.roll(1, 0))                    # non-zero output vectors
    w_in_b, w_out_b = w_in_a.clone(), w_out_a.clone()
    start_in = w_in_a.clone()
    for n_walks, base in ((300, 0), (77, 300)):         # second call: smaller, over stale scratch
        walks = B.gs_random_walks(G, None, n_walks, base, L, seed)
        la = torch.zeros(1, dtype=torch.float64, device=DEV)
        ca = torch.zeros(1, dtype=torch.int64, device=DEV)
        lb, cb = torch.zeros_like(la), torch.zeros_like(ca)
        B.gs_sgns_step(w_in_a, w_out_a, walks, base, w, K, alias, 0.025, seed, B.GS_DETERMINISTIC, la, ca)
        B.gs_sgns_step_static(w_in_b, w_out_b, walks, base, w, K, alias, 0.025, seed, lb, cb)
        torch.cuda.synchronize()
        assert ca.item() == cb.item() > 0
        assert abs(la.item() - lb.item()) <= 2e-6 * abs(la.item())
        assert (w_in_a - w_in_b).abs().max().item() <= EMB_TOL
        assert (w_out_a - w_out_b).abs().max().item() <= EMB_TOL
    assert (w_in_a - start_in).abs().max().item() > 10 * EMB_TOL      # the steps did something


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
