"""ctypes front end of the CPU oracle (gs_oracle.c).

TEST INFRASTRUCTURE ONLY.  Nothing on the product path may import this module;
it exists so that tests, the smoke check and the benchmark's CPU-baseline leg
can call the plain C restatement of the walk + SGNS path.  It shares no code
with the CUDA library and takes every input (CSR arrays, alias table, walks,
tables) as plain numpy data.

Array conventions: CSR offsets are passed as int64 (int32 offsets are widened
here), columns / walks / lists as int32, tables as C-contiguous float64.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "gs_oracle.c"
_LIB = _HERE / "libgs_oracle.so"
_lib = None


def build(force: bool = False) -> Path:
    """Compile gs_oracle.c with gcc (-O2, no fast-math) if the library is stale."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".{os.getpid()}.tmp")
        subprocess.run(
            ["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-ffp-contract=off",
             "-o", str(tmp), str(_SRC), "-lm"],
            check=True,
        )
        os.replace(tmp, _LIB)
    return _LIB


def _p(a, ct):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ct))


def lib():
    global _lib
    if _lib is None:
        build()
        L = ctypes.CDLL(str(_LIB))
        L.gso_uniform_walks.restype = ctypes.c_int64
        L.gso_node2vec_walks.restype = ctypes.c_int64
        L.gso_expand_lists.restype = ctypes.c_int64
        L.gso_sgns_loss_from_lists.restype = ctypes.c_double
        L.gso_subsample_walks.restype = ctypes.c_int64
        L.gso_shuffle_node.restype = ctypes.c_int64
        _lib = L
    return _lib


def _i64(a):
    return np.ascontiguousarray(a, dtype=np.int64)


def _i32(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.int32)


def philox4x32_10(ctr, key):
    """Philox4x32-10 block for a 4-word counter and 2-word key (SC'11)."""
    c = np.ascontiguousarray(ctr, dtype=np.uint32)
    k = np.ascontiguousarray(key, dtype=np.uint32)
    out = np.zeros(4, dtype=np.uint32)
    lib().gso_philox4x32_10(_p(c, ctypes.c_uint32), _p(k, ctypes.c_uint32),
                            _p(out, ctypes.c_uint32))
    return out


def uniform_walks(off, col, starts, n_walks, walk_id_base, L, seed):
    """DeepWalk walks (Section 2.2).  Returns (walks[n_walks, L], steps)."""
    off = _i64(off)
    col = _i32(col)
    starts = _i32(starts)
    walks = np.empty((n_walks, L), dtype=np.int32)
    steps = lib().gso_uniform_walks(
        ctypes.c_int64(len(off) - 1), _p(off, ctypes.c_int64), _p(col, ctypes.c_int32),
        _p(starts, ctypes.c_int32), ctypes.c_int64(n_walks), ctypes.c_int64(walk_id_base),
        ctypes.c_int32(L), ctypes.c_uint64(seed), _p(walks, ctypes.c_int32))
    return walks, int(steps)


def node2vec_thresholds(p, q):
    T = np.zeros(3, dtype=np.uint64)
    lib().gso_node2vec_thresholds(ctypes.c_double(p), ctypes.c_double(q),
                                  _p(T, ctypes.c_uint64))
    return T


def node2vec_walks(off, col, starts, n_walks, walk_id_base, L, seed, p, q, max_rounds=1024):
    """node2vec walks (Section 2.2).  Returns (walks, steps, cap_hits)."""
    off = _i64(off)
    col = _i32(col)
    starts = _i32(starts)
    walks = np.empty((n_walks, L), dtype=np.int32)
    caps = ctypes.c_int64(0)
    steps = lib().gso_node2vec_walks(
        ctypes.c_int64(len(off) - 1), _p(off, ctypes.c_int64), _p(col, ctypes.c_int32),
        _p(starts, ctypes.c_int32), ctypes.c_int64(n_walks), ctypes.c_int64(walk_id_base),
        ctypes.c_int32(L), ctypes.c_uint64(seed), ctypes.c_double(p), ctypes.c_double(q),
        ctypes.c_int32(max_rounds), _p(walks, ctypes.c_int32), ctypes.byref(caps))
    return walks, int(steps), int(caps.value)


def expand_lists(walks, walk_id_base, w, K, thr, alias, seed, forward_only=False, shrink=False):
    """Window pairs and negative draws, slot layout [(walk, i, sigma)].

    Returns (centers[n_slots], contexts[n_slots], negs[n_slots, K], n_pairs).
    """
    walks = _i32(walks)
    n_walks, L = walks.shape
    thr = np.ascontiguousarray(thr, dtype=np.uint32)
    alias = _i32(alias)
    n_slots = n_walks * L * 2 * w
    centers = np.empty(n_slots, dtype=np.int32)
    contexts = np.empty(n_slots, dtype=np.int32)
    negs = np.empty((n_slots, K), dtype=np.int32)
    n_pairs = lib().gso_expand_lists(
        _p(walks, ctypes.c_int32), ctypes.c_int64(n_walks), ctypes.c_int64(walk_id_base),
        ctypes.c_int32(L), ctypes.c_int32(w), ctypes.c_int32(K),
        _p(thr, ctypes.c_uint32), _p(alias, ctypes.c_int32), ctypes.c_int64(len(thr)),
        ctypes.c_uint64(seed), ctypes.c_int32(1 if forward_only else 0),
        ctypes.c_int32(1 if shrink else 0),
        _p(centers, ctypes.c_int32), _p(contexts, ctypes.c_int32), _p(negs, ctypes.c_int32))
    return centers, contexts, negs, int(n_pairs)


def build_alias(weights, power=0.75):
    """Alias table for p(v) ~ weight(v)**power.  Returns (thr uint32, alias int32)."""
    wgt = np.ascontiguousarray(weights, dtype=np.float64)
    n = len(wgt)
    thr = np.empty(n, dtype=np.uint32)
    alias = np.empty(n, dtype=np.int32)
    rc = lib().gso_build_alias(_p(wgt, ctypes.c_double), ctypes.c_int64(n),
                               ctypes.c_double(power), _p(thr, ctypes.c_uint32),
                               _p(alias, ctypes.c_int32))
    if rc != 0:
        raise ValueError("alias table needs at least one positive weight")
    return thr, alias


def init_rows(rows, d, seed):
    """Initial input vectors of the given node ids (uniform in [-0.5/d, 0.5/d))."""
    rows = _i64(rows)
    U = np.empty((len(rows), d), dtype=np.float64)
    lib().gso_init_rows(_p(rows, ctypes.c_int64), ctypes.c_int64(len(rows)),
                        ctypes.c_int32(d), ctypes.c_uint64(seed), _p(U, ctypes.c_double))
    return U


def sgns_loss_from_lists(U, V, centers, contexts, negs):
    d = U.shape[1]
    negs = _i32(negs)
    K = negs.shape[1]
    return float(lib().gso_sgns_loss_from_lists(
        _p(U, ctypes.c_double), _p(V, ctypes.c_double), ctypes.c_int32(d),
        ctypes.c_int64(len(centers)), ctypes.c_int32(K),
        _p(_i32(centers), ctypes.c_int32), _p(_i32(contexts), ctypes.c_int32),
        _p(negs, ctypes.c_int32)))


def sgns_det_from_lists(U, V, centers, contexts, negs, lr, order=None):
    """Synchronous mini-batch step in place on float64 tables U, V.

    Returns (loss_sum, pair_count); the loss is taken at the entry tables.
    """
    assert U.dtype == np.float64 and V.dtype == np.float64
    assert U.flags.c_contiguous and V.flags.c_contiguous and U.shape == V.shape
    n_rows, d = U.shape
    centers, contexts, negs = _i32(centers), _i32(contexts), _i32(negs)
    K = negs.shape[1]
    order = None if order is None else _i64(order)
    loss = ctypes.c_double(0.0)
    cnt = ctypes.c_int64(0)
    rc = lib().gso_sgns_det_from_lists(
        _p(U, ctypes.c_double), _p(V, ctypes.c_double), ctypes.c_int64(n_rows),
        ctypes.c_int32(d), ctypes.c_int64(len(centers)), ctypes.c_int32(K),
        _p(centers, ctypes.c_int32), _p(contexts, ctypes.c_int32), _p(negs, ctypes.c_int32),
        _p(order, ctypes.c_int64), ctypes.c_double(lr), ctypes.byref(loss), ctypes.byref(cnt))
    if rc != 0:
        raise MemoryError("oracle gradient buffers")
    return float(loss.value), int(cnt.value)


def sgns_grad_from_lists(U, V, centers, contexts, negs):
    """Summed mini-batch gradients at fixed tables.  Returns (GU, GV, loss_sum, pair_count)."""
    n_rows, d = U.shape
    centers, contexts, negs = _i32(centers), _i32(contexts), _i32(negs)
    K = negs.shape[1]
    GU, GV = np.empty_like(U), np.empty_like(V)
    loss = ctypes.c_double(0.0)
    cnt = ctypes.c_int64(0)
    lib().gso_sgns_grad_from_lists(
        _p(U, ctypes.c_double), _p(V, ctypes.c_double), ctypes.c_int64(n_rows), ctypes.c_int32(d),
        ctypes.c_int64(len(centers)), ctypes.c_int32(K), _p(centers, ctypes.c_int32),
        _p(contexts, ctypes.c_int32), _p(negs, ctypes.c_int32), _p(GU, ctypes.c_double),
        _p(GV, ctypes.c_double), ctypes.byref(loss), ctypes.byref(cnt))
    return GU, GV, float(loss.value), int(cnt.value)


def momentum_update(x, m, g, lr, mu):
    """In place: m <- mu m; m += g; x <- x - lr m, over whole tables (Section 3.2)."""
    assert x.flags.c_contiguous and m.flags.c_contiguous and g.flags.c_contiguous
    lib().gso_momentum_update(_p(x, ctypes.c_double), _p(m, ctypes.c_double), _p(g, ctypes.c_double),
                              ctypes.c_int64(x.size), ctypes.c_double(lr), ctypes.c_double(mu))


def sgns_momentum_step_from_lists(U, V, MU, MV, centers, contexts, negs, lr, mu):
    """Synchronous mini-batch step with momentum on dense float64 tables, in place."""
    GU, GV, loss, cnt = sgns_grad_from_lists(U, V, centers, contexts, negs)
    momentum_update(U, MU, GU, lr, mu)
    momentum_update(V, MV, GV, lr, mu)
    return loss, cnt


def sgns_seq_from_lists(U, V, centers, contexts, negs, S, lr):
    """Sequential per-pair SGD in place (race-free limit of the lock-free mode)."""
    assert U.dtype == np.float64 and V.dtype == np.float64
    d = U.shape[1]
    centers, contexts, negs = _i32(centers), _i32(contexts), _i32(negs)
    K = negs.shape[1]
    loss = ctypes.c_double(0.0)
    cnt = ctypes.c_int64(0)
    rc = lib().gso_sgns_seq_from_lists(
        _p(U, ctypes.c_double), _p(V, ctypes.c_double), ctypes.c_int32(d),
        ctypes.c_int64(len(centers)), ctypes.c_int32(S), ctypes.c_int32(K),
        _p(centers, ctypes.c_int32), _p(contexts, ctypes.c_int32), _p(negs, ctypes.c_int32),
        ctypes.c_double(lr), ctypes.byref(loss), ctypes.byref(cnt))
    if rc != 0:
        raise MemoryError("oracle accumulator")
    return float(loss.value), int(cnt.value)


def round_f16(x):
    """In place: every value to the nearest IEEE binary16 (ties to even)."""
    assert x.dtype == np.float64 and x.flags.c_contiguous
    lib().gso_round_f16(_p(x, ctypes.c_double), ctypes.c_int64(x.size))
    return x


def round_bf16(x):
    """In place: every value to the nearest bfloat16 (8 significant bits, ties to even)."""
    assert x.dtype == np.float64 and x.flags.c_contiguous
    lib().gso_round_bf16(_p(x, ctypes.c_double), ctypes.c_int64(x.size))
    return x


def sgns_det_bf16_from_lists(U, V, centers, contexts, negs, lr):
    """Synchronous step on bfloat16-valued tables: full-precision step, written rows rounded."""
    out = sgns_det_from_lists(U, V, centers, contexts, negs, lr)
    round_bf16(U)
    round_bf16(V)
    return out


def sgns_seq_bf16_from_lists(U, V, centers, contexts, negs, S, lr):
    """Sequential per-pair SGD on bfloat16-valued tables, in place."""
    d = U.shape[1]
    centers, contexts, negs = _i32(centers), _i32(contexts), _i32(negs)
    K = negs.shape[1]
    loss = ctypes.c_double(0.0)
    cnt = ctypes.c_int64(0)
    rc = lib().gso_sgns_seq_bf16_from_lists(
        _p(U, ctypes.c_double), _p(V, ctypes.c_double), ctypes.c_int32(d),
        ctypes.c_int64(len(centers)), ctypes.c_int32(S), ctypes.c_int32(K),
        _p(centers, ctypes.c_int32), _p(contexts, ctypes.c_int32), _p(negs, ctypes.c_int32),
        ctypes.c_double(lr), ctypes.byref(loss), ctypes.byref(cnt))
    if rc != 0:
        raise MemoryError("oracle accumulator")
    return float(loss.value), int(cnt.value)


def sgns_det_f16_from_lists(U, V, centers, contexts, negs, lr):
    """Synchronous step on binary16-valued tables: full-precision step, written rows rounded
    (rows that are not written hold binary16 values already, so rounding them changes nothing)."""
    out = sgns_det_from_lists(U, V, centers, contexts, negs, lr)
    round_f16(U)
    round_f16(V)
    return out


def sgns_seq_f16_from_lists(U, V, centers, contexts, negs, S, lr):
    """Sequential per-pair SGD on binary16-valued tables, in place."""
    d = U.shape[1]
    centers, contexts, negs = _i32(centers), _i32(contexts), _i32(negs)
    K = negs.shape[1]
    loss = ctypes.c_double(0.0)
    cnt = ctypes.c_int64(0)
    rc = lib().gso_sgns_seq_f16_from_lists(
        _p(U, ctypes.c_double), _p(V, ctypes.c_double), ctypes.c_int32(d),
        ctypes.c_int64(len(centers)), ctypes.c_int32(S), ctypes.c_int32(K),
        _p(centers, ctypes.c_int32), _p(contexts, ctypes.c_int32), _p(negs, ctypes.c_int32),
        ctypes.c_double(lr), ctypes.byref(loss), ctypes.byref(cnt))
    if rc != 0:
        raise MemoryError("oracle accumulator")
    return float(loss.value), int(cnt.value)


def sgns_seq_add16_from_lists(U, V, centers, contexts, negs, S, lr, fmt):
    """Sequential per-pair SGD on 16-bit-valued tables where every change is an increment rounded
    to the format and added in the format (fmt 0: binary16, 1: bfloat16), in place."""
    d = U.shape[1]
    centers, contexts, negs = _i32(centers), _i32(contexts), _i32(negs)
    K = negs.shape[1]
    loss = ctypes.c_double(0.0)
    cnt = ctypes.c_int64(0)
    rc = lib().gso_sgns_seq_add16_from_lists(
        _p(U, ctypes.c_double), _p(V, ctypes.c_double), ctypes.c_int32(d),
        ctypes.c_int64(len(centers)), ctypes.c_int32(S), ctypes.c_int32(K),
        _p(centers, ctypes.c_int32), _p(contexts, ctypes.c_int32), _p(negs, ctypes.c_int32),
        ctypes.c_double(lr), ctypes.c_int32(fmt), ctypes.byref(loss), ctypes.byref(cnt))
    if rc != 0:
        raise MemoryError("oracle accumulator")
    return float(loss.value), int(cnt.value)


def round_sr(x, fmt, u16):
    """In place: every value rounded stochastically to binary16 (fmt 0) or bfloat16 (fmt 1) with the
    given 16-bit dithers (one per value)."""
    assert x.dtype == np.float64 and x.flags.c_contiguous
    u = np.ascontiguousarray(u16, dtype=np.uint32)
    assert u.size == x.size
    lib().gso_round_sr(_p(x, ctypes.c_double), ctypes.c_int64(x.size), ctypes.c_int32(fmt), _p(u, ctypes.c_uint32))
    return x


def dither16(words, salt, d):
    """The 16-bit dithers of the d columns of a row-write event with Philox block `words`."""
    r = np.ascontiguousarray(words, dtype=np.uint32)
    out = np.empty(d, dtype=np.uint32)
    lib().gso_dither16(_p(r, ctypes.c_uint32), ctypes.c_uint32(salt), ctypes.c_int32(d), _p(out, ctypes.c_uint32))
    return out


def round_sr_rows(X, fmt, seed, table, walk_id_base):
    """In place: table X (0 input, 1 output) as the synchronous step with stochastic write-back
    leaves it: every value rounded with the dither of its (row, column) for that step."""
    assert X.dtype == np.float64 and X.flags.c_contiguous
    lib().gso_round_sr_rows(_p(X, ctypes.c_double), ctypes.c_int64(X.shape[0]), ctypes.c_int32(X.shape[1]),
                            ctypes.c_int32(fmt), ctypes.c_uint64(seed), ctypes.c_uint32(table),
                            ctypes.c_int64(walk_id_base))
    return X


def sgns_det_sr_from_lists(U, V, centers, contexts, negs, lr, fmt, seed, walk_id_base):
    """Synchronous step on 16-bit-valued tables with stochastic write-back: full-precision step,
    then every written value rounded stochastically (rows that are not written hold representable
    values, which never move)."""
    out = sgns_det_from_lists(U, V, centers, contexts, negs, lr)
    round_sr_rows(U, fmt, seed, 0, walk_id_base)
    round_sr_rows(V, fmt, seed, 1, walk_id_base)
    return out


def sgns_seq_sr_from_lists(U, V, centers, contexts, negs, S, lr, fmt, seed, walk_id_base, L):
    """Sequential per-pair SGD on 16-bit-valued tables with stochastic write-back, in place."""
    d = U.shape[1]
    centers, contexts, negs = _i32(centers), _i32(contexts), _i32(negs)
    K = negs.shape[1]
    loss = ctypes.c_double(0.0)
    cnt = ctypes.c_int64(0)
    rc = lib().gso_sgns_seq_sr_from_lists(
        _p(U, ctypes.c_double), _p(V, ctypes.c_double), ctypes.c_int32(d),
        ctypes.c_int64(len(centers)), ctypes.c_int32(S), ctypes.c_int32(K),
        _p(centers, ctypes.c_int32), _p(contexts, ctypes.c_int32), _p(negs, ctypes.c_int32),
        ctypes.c_double(lr), ctypes.c_int32(fmt), ctypes.c_uint64(seed), ctypes.c_int64(walk_id_base),
        ctypes.c_int32(L), ctypes.byref(loss), ctypes.byref(cnt))
    if rc != 0:
        raise MemoryError("oracle accumulator")
    return float(loss.value), int(cnt.value)


def keep_thresholds(weights, t):
    """Sub-sampling thresholds: keep(v) = min(1, sqrt(t / f(v))) as uint32 (0xFFFFFFFF = always)."""
    wgt = np.ascontiguousarray(weights, dtype=np.float64)
    thr = np.empty(len(wgt), dtype=np.uint32)
    rc = lib().gso_keep_thresholds(_p(wgt, ctypes.c_double), ctypes.c_int64(len(wgt)),
                                   ctypes.c_double(t), _p(thr, ctypes.c_uint32))
    if rc != 0:
        raise ValueError("sub-sampling needs at least one positive weight")
    return thr


def subsample_walks(walks, walk_id_base, keep_thr, seed):
    """Drops walk entries by the keep thresholds and compacts each walk.  Returns (walks, kept)."""
    walks = _i32(walks)
    n_walks, L = walks.shape
    keep_thr = np.ascontiguousarray(keep_thr, dtype=np.uint32)
    out = np.empty_like(walks)
    kept = lib().gso_subsample_walks(_p(walks, ctypes.c_int32), ctypes.c_int64(n_walks),
                                     ctypes.c_int64(walk_id_base), ctypes.c_int32(L),
                                     _p(keep_thr, ctypes.c_uint32), ctypes.c_uint64(seed),
                                     _p(out, ctypes.c_int32))
    return out, int(kept)


def shuffle_node(v, n, seed, epoch):
    return int(lib().gso_shuffle_node(ctypes.c_int64(v), ctypes.c_int64(n), ctypes.c_uint64(seed),
                                      ctypes.c_uint32(epoch)))


def shuffled_starts(n, seed, epoch, walk_id_first, count):
    """Start nodes of walk ids [first, first + count): the keyed bijection of (id mod n)."""
    out = np.empty(count, dtype=np.int32)
    lib().gso_shuffled_starts(ctypes.c_int64(n), ctypes.c_uint64(seed), ctypes.c_uint32(epoch),
                              ctypes.c_int64(walk_id_first), ctypes.c_int64(count),
                              _p(out, ctypes.c_int32))
    return out


def adam_rows(x, m, v, g, rows, lr, b1, b2, eps, step):
    """In place Adam update of the given distinct rows of table x with moments m, v."""
    for a in (x, m, v, g):
        assert a.dtype == np.float64 and a.flags.c_contiguous
    rows = _i64(rows)
    lib().gso_adam_rows(_p(x, ctypes.c_double), _p(m, ctypes.c_double), _p(v, ctypes.c_double),
                        _p(g, ctypes.c_double), ctypes.c_int32(x.shape[1]), _p(rows, ctypes.c_int64),
                        ctypes.c_int64(len(rows)), ctypes.c_double(lr), ctypes.c_double(b1),
                        ctypes.c_double(b2), ctypes.c_double(eps), ctypes.c_int64(step))


def touched_rows(centers, contexts, negs):
    """Distinct rows a mini-batch reads and writes: (rows of the input table, rows of the output
    table).  A masked negative (equal to its pair's context) is not a touched row by itself."""
    centers, contexts, negs = _i32(centers), _i32(contexts), _i32(negs)
    ok = centers >= 0
    rows_in = np.unique(centers[ok])
    ng = negs[ok]
    unmasked = ng[(ng >= 0) & (ng != contexts[ok][:, None])]
    rows_out = np.unique(np.concatenate([contexts[ok], unmasked]))
    return rows_in.astype(np.int64), rows_out.astype(np.int64)


def sgns_adam_step_from_lists(U, V, MU, VU, MV, VV, centers, contexts, negs, lr, b1, b2, eps, step):
    """Synchronous mini-batch step with Adam on the batch's rows, dense float64 tables, in place.
    (MU, VU) and (MV, VV) are the first and second moments of U and V."""
    GU, GV, loss, cnt = sgns_grad_from_lists(U, V, centers, contexts, negs)
    rows_in, rows_out = touched_rows(centers, contexts, negs)
    adam_rows(U, MU, VU, GU, rows_in, lr, b1, b2, eps, step)
    adam_rows(V, MV, VV, GV, rows_out, lr, b1, b2, eps, step)
    return loss, cnt


def lr_at(schedule, lr0, b, num_batches):
    """Learning rate of mini-batch b: 'constant', or 'linear' decay floored at 1e-4 lr0."""
    if schedule == "constant":
        return lr0
    if schedule == "linear":
        return lr0 * max(1.0 - b / num_batches, 1e-4)
    raise ValueError(schedule)


def sgns_epoch(off, col, thr, alias, U, V, *, walks_per_node, L, w, K, lr0, schedule,
               batch_walks, seed, mode="det", kind="uniform", p=1.0, q=1.0,
               first_batch=0, num_batches=None, shrink=False, keep_thr=None, shuffle_epoch=None,
               optimizer="sgd", state=None, momentum=0.9, beta2=0.999, eps=1e-8, iteration_base=0):
    """One pass over walk ids rep*N + v in order, batch by batch (dense tables).

    Each batch: generate its walks, expand pairs and negatives, apply one step.
    shuffle_epoch (int or None): walk id a starts at the keyed bijection of a mod N for that
    epoch instead of at a mod N.  keep_thr (uint32[N] or None): frequent-node sub-sampling of
    the generated walks before the windows are formed.  shrink: per-position window draw.
    optimizer: "sgd"; "momentum" (dense update of both tables per batch, Section 3.2; state =
    dict(MU, MV) of zero-initialised tables); "adam" (rows of the batch only; state = dict(MU, VU,
    MV, VV); step = iteration_base + batch index + 1).  Both need mode "det".
    Returns dict(loss_sum, pairs, steps).  Tables are updated in place.
    """
    n_nodes = len(off) - 1
    total = n_nodes * walks_per_node
    nb_total = (total + batch_walks - 1) // batch_walks
    if num_batches is None:
        num_batches = nb_total - first_batch
    loss_sum, pairs, steps, masked = 0.0, 0, 0, 0
    for b in range(first_batch, first_batch + num_batches):
        base = b * batch_walks
        n = min(batch_walks, total - base)
        starts = None if shuffle_epoch is None else shuffled_starts(n_nodes, seed, shuffle_epoch, base, n)
        if kind == "uniform":
            walks, st = uniform_walks(off, col, starts, n, base, L, seed)
        else:
            walks, st, _ = node2vec_walks(off, col, starts, n, base, L, seed, p, q)
        if keep_thr is not None:
            walks, _ = subsample_walks(walks, base, keep_thr, seed)
        c, o, ng, _ = expand_lists(walks, base, w, K, thr, alias, seed, shrink=shrink)
        lr = lr_at(schedule, lr0, b, nb_total)
        if optimizer == "momentum":
            ls, pc = sgns_momentum_step_from_lists(U, V, state["MU"], state["MV"], c, o, ng, lr, momentum)
        elif optimizer == "adam":
            ls, pc = sgns_adam_step_from_lists(U, V, state["MU"], state["VU"], state["MV"], state["VV"],
                                               c, o, ng, lr, momentum, beta2, eps, iteration_base + b + 1)
        elif mode == "det":
            ls, pc = sgns_det_from_lists(U, V, c, o, ng, lr)
        elif mode == "det_f16":                        # binary16-valued tables, written rows rounded
            ls, pc = sgns_det_f16_from_lists(U, V, c, o, ng, lr)
        elif mode == "det_bf16":
            ls, pc = sgns_det_bf16_from_lists(U, V, c, o, ng, lr)
        elif mode in ("det_sr_f16", "det_sr_bf16"):    # 16-bit tables, stochastic write-back
            ls, pc = sgns_det_sr_from_lists(U, V, c, o, ng, lr, 0 if mode == "det_sr_f16" else 1, seed, base)
        elif mode in ("seq_sr_f16", "seq_sr_bf16"):
            ls, pc = sgns_seq_sr_from_lists(U, V, c, o, ng, 2 * w, lr, 0 if mode == "seq_sr_f16" else 1,
                                            seed, base, L)
        else:
            ls, pc = sgns_seq_from_lists(U, V, c, o, ng, 2 * w, lr)
        loss_sum += ls
        pairs += pc
        steps += st
        masked += int(((ng == o[:, None]) & (c >= 0)[:, None]).sum())   # negatives equal to their context
    return {"loss_sum": loss_sum, "pairs": pairs, "steps": steps, "masked_negs": masked}
