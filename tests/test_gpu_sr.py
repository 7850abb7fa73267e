"""GPU parity of the stochastic write-back for 16-bit tables (GS_ROUND_STOCHASTIC).

The oracle computes the update in fp64, rounds it once to fp32 and decides the stochastic rounding
on that value; the kernels compute in fp32 and decide on their value with the same keyed dithers.
Where the two fp32 values differ in their last bit the threshold moves by 2^-13 (binary16) or 2^-16
(bfloat16) of the dither range, so a decision differs for about one value in 10^4: the bar is "no
element further than one unit in the last place of the format, all but a small fraction bit-equal"."""
import numpy as np
import pytest
import torch

from oracle import gs_oracle as O
from paper_2407_15452_b200 import binding as B
from paper_2407_15452_b200 import workloads as WL
from tests.helpers import alias_to_device, degree_alias, np_graph

pytestmark = pytest.mark.gpu
DEV = "cuda"
FMT = {torch.float16: 0, torch.bfloat16: 1}
STEP = {torch.float16: B.gs_sgns_step_f16, torch.bfloat16: B.gs_sgns_step_bf16}


def ulp(x, dt):
    """Spacing of the 16-bit format at |x| (normal range)."""
    bits, tiny = (10, 2.0 ** -14) if dt == torch.float16 else (7, 2.0 ** -126)
    return 2.0 ** (np.floor(np.log2(np.maximum(np.abs(x), tiny))) - bits)


def tables16(n, dim, seed, dt, scale=0.5):
    gen = torch.Generator().manual_seed(seed)
    a = ((torch.rand((n, dim), generator=gen) - 0.5) * scale).to(dt)
    b = ((torch.rand((n, dim), generator=gen) - 0.5) * scale).to(dt)
    return a, b


def f64(t):
    return t.to(torch.float32).cpu().numpy().astype(np.float64)


@pytest.fixture(scope="module")
def tiny():
    wl = WL.WORKLOADS["tiny_deepwalk"]
    g = wl.make_graph()
    off, col = np_graph(g)
    thr, alias = degree_alias(off)
    return g, off, col, thr, alias


@pytest.mark.parametrize("dt", [torch.float16, torch.bfloat16])
@pytest.mark.parametrize("dim,L,w,K", [(128, 20, 5, 5), (64, 10, 3, 10), (256, 8, 2, 3)])
def test_synchronous_step_with_stochastic_write_back(tiny, dt, dim, L, w, K):
    g, off, col, thr, alias = tiny
    n = g.n_nodes
    base, seed, lr = (3 << 32) + 10, 2, 0.05           # a first walk id beyond 32 bits: both key words matter
    walks, _ = O.uniform_walks(off, col, None, 400, base, L, seed)
    c, o, ng, n_pairs = O.expand_lists(walks, base, w, K, thr, alias, seed)
    h_in, h_out = tables16(n, dim, 1, dt)
    U, V = f64(h_in), f64(h_out)
    U0, V0 = U.copy(), V.copy()
    loss_o, cnt_o = O.sgns_det_sr_from_lists(U, V, c, o, ng, lr, FMT[dt], seed, base)
    a_dev = alias_to_device(thr, alias)
    wd = torch.from_numpy(walks).to(DEV)
    mode = B.GS_DETERMINISTIC | B.GS_ROUND_STOCHASTIC
    w_in, w_out = h_in.to(DEV), h_out.to(DEV)
    loss = torch.zeros(1, dtype=torch.float64, device=DEV)
    cnt = torch.zeros(1, dtype=torch.int64, device=DEV)
    STEP[dt](w_in, w_out, wd, base, w, K, a_dev, lr, seed, mode, loss, cnt)
    torch.cuda.synchronize()
    assert cnt.item() == cnt_o == n_pairs and abs(loss.item() - loss_o) <= 2e-6 * abs(loss_o)
    for got, want, start in ((f64(w_in), U, U0), (f64(w_out), V, V0)):
        # one unit of the format at the value's magnitude, plus the 1e-6 that fp32 arithmetic on
        # values of order 0.1 can be off by (where old value and step cancel, the result is tiny
        # and its own unit is far below that noise)
        diff = np.abs(got - want)
        assert (diff <= ulp(want, dt) * 1.0001 + 1e-6).all(), float((diff / (ulp(want, dt) + 1e-6)).max())
        assert np.mean(diff > 0) <= 2e-3, float(np.mean(diff > 0))
        untouched = (want == start).all(axis=1)
        assert np.array_equal(got[untouched], start[untouched])
        assert np.mean(want != start) > 0.02
    # it IS another rounding than to-nearest: many stored values differ from the to-nearest step's
    w_in_n, w_out_n = h_in.to(DEV), h_out.to(DEV)
    STEP[dt](w_in_n, w_out_n, wd, base, w, K, a_dev, lr, seed, B.GS_DETERMINISTIC)
    assert (w_out_n != w_out).float().mean().item() > 0.005
    # reproducible bit for bit with the same keys; another seed rounds differently
    w_in2, w_out2 = h_in.to(DEV), h_out.to(DEV)
    STEP[dt](w_in2, w_out2, wd, base, w, K, a_dev, lr, seed, mode)
    assert torch.equal(w_in, w_in2) and torch.equal(w_out, w_out2)


@pytest.mark.parametrize("dt", [torch.float16, torch.bfloat16])
@pytest.mark.parametrize("dim,L,w", [(128, 40, 5), (64, 20, 5), (256, 24, 3)])
def test_lock_free_walks_without_shared_rows_with_stochastic_write_back(dt, dim, L, w):
    # No two walks share a row, no walk visits a node twice, no negatives: nothing can race, so the
    # concurrent run must follow the sequential oracle write by write - same dithers, keyed by walk
    # id, position and target index.  A row is written up to 2w times; where one decision differs
    # (fp32 against fp64 arithmetic) the row stays a unit apart, so a few units are allowed on a
    # small fraction of the values.
    n_walks, span = 500, 64
    n = n_walks * span
    rng = np.random.default_rng(dim)
    walks = np.empty((n_walks, L), dtype=np.int32)
    for k in range(n_walks):
        walks[k] = k * span + rng.permutation(span)[:L]
    walks[3, L // 2:] = -1
    base, seed = 77, 3
    thr, alias = O.build_alias(np.ones(n), 1.0)
    c, o, ng, n_pairs = O.expand_lists(walks, base, w, 0, thr, alias, seed)
    h_in, h_out = tables16(n, dim, 6, dt, scale=0.6)
    U, V = f64(h_in), f64(h_out)
    V0 = V.copy()
    loss_o, cnt_o = O.sgns_seq_sr_from_lists(U, V, c, o, ng, 2 * w, 0.05, FMT[dt], seed, base, L)
    w_in, w_out = h_in.to(DEV), h_out.to(DEV)
    loss = torch.zeros(1, dtype=torch.float64, device=DEV)
    cnt = torch.zeros(1, dtype=torch.int64, device=DEV)
    STEP[dt](w_in, w_out, torch.from_numpy(walks).to(DEV), base, w, 0, None, 0.05, seed,
             B.GS_HOGWILD | B.GS_ROUND_STOCHASTIC, loss, cnt)
    torch.cuda.synchronize()
    assert cnt.item() == cnt_o == n_pairs and abs(loss.item() - loss_o) < 1e-4 * abs(loss_o)
    for got, want, start in ((f64(w_in), U, f64(h_in)), (f64(w_out), V, f64(h_out))):
        # measured: 2e-5 .. 5e-5 of the written values differ, nearly all by one unit of the format
        # at the magnitude the value had while it was written.  A first differing decision in a
        # walk changes its later gradients a little, so a handful of values (6 of 4e6) end up to
        # four units apart: the bound is on the fraction, with a loose cap on the distance
        diff = np.abs(got - want)
        scale = np.maximum(np.maximum(np.abs(want), np.abs(start)), 1e-3)
        assert (diff <= 8 * ulp(scale, dt)).all(), float((diff / ulp(scale, dt)).max())
        assert np.mean(diff > 0) <= 2e-4, float(np.mean(diff > 0))
        assert np.mean(diff > ulp(scale, dt) * 1.0001) <= 2e-5
    assert np.mean(V != V0) > 0.05
    # and it is not the to-nearest result
    Un, Vn = f64(h_in), f64(h_out)
    (O.sgns_seq_f16_from_lists if dt == torch.float16 else O.sgns_seq_bf16_from_lists)(Un, Vn, c, o, ng, 2 * w, 0.05)
    assert np.mean(f64(w_out) != Vn) > 0.01


def test_stochastic_write_back_needs_16_bit_tables_and_keeps_small_increments_alive(tiny):
    g, off, col, thr, alias = tiny
    n = g.n_nodes
    a_dev = alias_to_device(thr, alias)
    walks = torch.from_numpy(O.uniform_walks(off, col, None, 64, 0, 10, 1)[0]).to(DEV)
    w32 = torch.zeros((n, 64), dtype=torch.float32, device=DEV)
    with pytest.raises(B.GsError) as e:
        B.gs_sgns_step(w32, w32.clone(), walks, 0, 3, 2, a_dev, 0.025, 1, B.GS_HOGWILD | B.GS_ROUND_STOCHASTIC)
    assert e.value.status == -6
    # bfloat16 tables whose values are so large that one increment is below half a unit in the last
    # place: to-nearest loses every increment, stochastic rounding moves the expected fraction of them
    wl = WL.WORKLOADS["tiny_deepwalk"]
    G = B.gs_graph_load_csr(g.offsets.to(DEV), g.cols.to(DEV), B.GS_VALIDATE | B.GS_REQUIRE_SORTED)
    moved = {}
    for name, flag in (("nearest", 0), ("stochastic", B.GS_ROUND_STOCHASTIC)):
        w_in = torch.full((n, 64), 4.0, dtype=torch.bfloat16, device=DEV)        # spacing 2^-5 at 4.0
        w_out = torch.full((n, 64), 4.0, dtype=torch.bfloat16, device=DEV)
        res = B.gs_sgns_epoch(G, a_dev, w_in, w_out, walks_per_node=1, walk_len=10, window=5, n_neg=5,
                              lr0=1e-6, batch_walks=512, seed=0, mode=B.GS_HOGWILD | flag)
        assert res.pairs > 0
        moved[name] = (w_out != 4.0).float().mean().item()
    assert moved["nearest"] == 0.0 and moved["stochastic"] > 1e-4, moved


@pytest.mark.parametrize("dt", [torch.float16, torch.bfloat16])
def test_synchronous_epoch_with_stochastic_write_back_matches_the_oracle(tiny, dt):
    # 20 batches through the epoch driver (part A of batch b+1 beside the update of batch b): the keys
    # of the dithers are the batch's first walk id and the row, so they do not depend on how the
    # epoch is cut into calls
    g, off, col, thr, alias = tiny
    n, dim = g.n_nodes, 64
    U = O.init_rows(np.arange(n), dim, 2)
    (O.round_f16 if dt == torch.float16 else O.round_bf16)(U)
    V = np.zeros_like(U)
    U0 = U.copy()
    want = O.sgns_epoch(off, col, thr, alias, U, V, walks_per_node=1, L=10, w=5, K=5, lr0=0.025,
                        schedule="linear", batch_walks=512, seed=2,
                        mode="det_sr_f16" if dt == torch.float16 else "det_sr_bf16")
    G = B.gs_graph_load_csr(g.offsets.to(DEV), g.cols.to(DEV), B.GS_VALIDATE)
    w_in = torch.empty((n, dim), dtype=dt, device=DEV)
    w_out = torch.empty_like(w_in)
    (B.gs_init_embeddings_f16 if dt == torch.float16 else B.gs_init_embeddings_bf16)(w_in, w_out, 2)
    assert np.array_equal(f64(w_in), U0)
    kw = dict(walks_per_node=1, walk_len=10, window=5, n_neg=5, lr0=0.025, batch_walks=512, seed=2,
              mode=B.GS_DETERMINISTIC | B.GS_ROUND_STOCHASTIC, lr_schedule=B.GS_LR_LINEAR)
    r1 = B.gs_sgns_epoch(G, alias_to_device(thr, alias), w_in, w_out, first_batch=0, num_batches=9, **kw)
    r2 = B.gs_sgns_epoch(G, alias_to_device(thr, alias), w_in, w_out, first_batch=9, **kw)
    assert r1.pairs + r2.pairs == want["pairs"] and r1.steps + r2.steps == want["steps"]
    assert abs(r1.loss_sum + r2.loss_sum - want["loss_sum"]) <= 1e-3 * want["loss_sum"]
    for got, ref, start in ((f64(w_in), U, U0), (f64(w_out), V, np.zeros_like(V))):
        scale = np.maximum(np.maximum(np.abs(ref), np.abs(start)), 1e-3)
        assert (np.abs(got - ref) <= 4 * ulp(scale, dt)).all()
        assert np.mean(got == ref) > 0.97, float(np.mean(got == ref))
    assert np.abs(V).max() > 0.01
