"""Thin ctypes binding of the C ABI in include/gs.h.

Argument marshalling only: every function takes torch tensors (device memory)
or numpy arrays (host memory), checks dtype/device/contiguity, passes raw
pointers and the current CUDA stream to the library, and raises GsError on a
non-zero status.  Nothing here computes anything; if the shared library has
not been built the first call raises.
"""
from __future__ import annotations

import ctypes
from dataclasses import dataclass
from pathlib import Path

import numpy as np
import torch

_LIB_PATH = Path(__file__).resolve().parent / "libgs_b200.so"
_lib = None

GS_VALIDATE, GS_REQUIRE_SORTED, GS_BUILD_WALK_INDEX, GS_BUILD_EDGE_SET = 1, 2, 4, 8
GS_DETERMINISTIC, GS_HOGWILD, GS_HOGWILD_RED = 0, 1, 2
GS_PAIRS_FORWARD_ONLY = 0x100
GS_WINDOW_SHRINK = 0x200
GS_ROUND_STOCHASTIC = 0x400
GS_WALK_UNIFORM, GS_WALK_NODE2VEC = 0, 1
GS_LR_CONSTANT, GS_LR_LINEAR = 0, 1
GS_TABLE_F32, GS_TABLE_F16, GS_TABLE_BF16 = 0, 1, 2
GS_OPT_SGD, GS_OPT_MOMENTUM, GS_OPT_ADAM = 0, 1, 2

EXPORTS = [
    "gs_last_error", "gs_graph_load_csr", "gs_graph_free", "gs_graph_info", "gs_build_alias",
    "gs_init_embeddings", "gs_random_walks", "gs_node2vec_walks", "gs_sgns_step",
    "gs_sgns_epoch", "gs_release_workspace", "gs_tune_node2vec_group", "gs_sgns_step_static", "gs_sgns_step_momentum", "gs_momentum_flush",
    "gs_init_embeddings_f16", "gs_sgns_step_f16", "gs_sgns_step_adam", "gs_build_keep_thresholds",
    "gs_subsample_walks", "gs_shuffled_starts", "gs_refused_ids",
    "gs_init_embeddings_bf16", "gs_sgns_step_bf16",
]


class GsError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"gs status {status}: {message}")
        self.status = status


class SgnsConfig(ctypes.Structure):
    _fields_ = [
        ("dim", ctypes.c_int32), ("walks_per_node", ctypes.c_int32), ("walk_len", ctypes.c_int32),
        ("window", ctypes.c_int32), ("n_neg", ctypes.c_int32), ("walk_kind", ctypes.c_int32),
        ("lr_schedule", ctypes.c_int32), ("mode", ctypes.c_int32), ("max_rounds", ctypes.c_int32),
        ("table_dtype", ctypes.c_int32), ("p", ctypes.c_double), ("q", ctypes.c_double),
        ("lr0", ctypes.c_double), ("batch_walks", ctypes.c_int64), ("first_batch", ctypes.c_int64),
        ("num_batches", ctypes.c_int64), ("seed", ctypes.c_uint64),
        ("d_keep_thr", ctypes.c_void_p), ("shuffle_starts", ctypes.c_int32), ("epoch", ctypes.c_uint32),
        ("optimizer", ctypes.c_int32), ("momentum", ctypes.c_float), ("beta2", ctypes.c_float),
        ("eps", ctypes.c_float), ("iteration_base", ctypes.c_int64),
        ("d_m_in", ctypes.c_void_p), ("d_m_out", ctypes.c_void_p), ("d_v_in", ctypes.c_void_p),
        ("d_v_out", ctypes.c_void_p), ("d_last_in", ctypes.c_void_p), ("d_last_out", ctypes.c_void_p),
    ]


class EpochStats(ctypes.Structure):
    _fields_ = [
        ("loss_sum", ctypes.c_double), ("pairs", ctypes.c_int64), ("steps", ctypes.c_int64),
        ("cap_hits", ctypes.c_int64), ("batches", ctypes.c_int64), ("masked_negs", ctypes.c_int64),
        ("ms_walk", ctypes.c_float),
        ("ms_sgns", ctypes.c_float), ("ms_total", ctypes.c_float), ("ms_prepare", ctypes.c_float),
        ("refused_ids", ctypes.c_int64),
    ]


def library_path() -> Path:
    return _LIB_PATH


def lib():
    """Loads libgs_b200.so; fails loudly if it is missing (there is no fallback path)."""
    global _lib
    if _lib is None:
        if not _LIB_PATH.exists():
            raise FileNotFoundError(
                f"{_LIB_PATH} not built; run `python -m paper_2407_15452_b200.build`")
        L = ctypes.CDLL(str(_LIB_PATH))
        L.gs_last_error.restype = ctypes.c_char_p
        L.gs_graph_free.restype = None
        for name in EXPORTS:
            if name not in ("gs_last_error", "gs_graph_free"):
                getattr(L, name).restype = ctypes.c_int32
        _lib = L
    return _lib


def _check(status: int):
    if status != 0:
        raise GsError(status, lib().gs_last_error().decode())


def _stream() -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _dev(t, dtype, name, allow_none=False) -> ctypes.c_void_p:
    if t is None:
        if allow_none:
            return ctypes.c_void_p(0)
        raise TypeError(f"{name} is required")
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise TypeError(f"{name} must be a contiguous CUDA tensor of {dtype}")
    return ctypes.c_void_p(t.data_ptr())


class Graph:
    """Owns a gs_graph handle and keeps the CSR tensors alive."""

    def __init__(self, offsets: torch.Tensor, cols: torch.Tensor, flags: int = GS_VALIDATE):
        if offsets.dtype not in (torch.int32, torch.int64):
            raise TypeError("offsets must be int32 or int64")
        self.offsets, self.cols = offsets, cols
        self.n_nodes = offsets.numel() - 1
        self.n_edges = cols.numel()
        self._h = ctypes.c_void_p(0)
        _check(lib().gs_graph_load_csr(
            ctypes.c_int64(self.n_nodes), ctypes.c_int64(self.n_edges),
            _dev(offsets, offsets.dtype, "offsets"), ctypes.c_int32(offsets.dtype == torch.int64),
            _dev(cols, torch.int32, "cols", allow_none=self.n_edges == 0),
            ctypes.c_uint32(flags), _stream(), ctypes.byref(self._h)))

    def info(self):
        n, e, m, s = ctypes.c_int64(), ctypes.c_int64(), ctypes.c_int64(), ctypes.c_int32()
        _check(lib().gs_graph_info(self._h, ctypes.byref(n), ctypes.byref(e), ctypes.byref(m),
                                   ctypes.byref(s)))
        return {"n_nodes": n.value, "n_edges": e.value, "max_degree": m.value,
                "rows_sorted": bool(s.value)}

    def close(self):
        if self._h:
            lib().gs_graph_free(self._h)
            self._h = ctypes.c_void_p(0)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def gs_graph_load_csr(offsets, cols, flags=GS_VALIDATE) -> Graph:
    return Graph(offsets, cols, flags)


def gs_build_alias(weights: np.ndarray, power: float = 0.75) -> np.ndarray:
    """Host call.  Returns the packed table (uint64: thr low, alias high)."""
    w = np.ascontiguousarray(weights, dtype=np.float64)
    out = np.empty(len(w), dtype=np.uint64)
    _check(lib().gs_build_alias(w.ctypes.data_as(ctypes.c_void_p), ctypes.c_int64(len(w)),
                                ctypes.c_double(power), out.ctypes.data_as(ctypes.c_void_p)))
    return out


def gs_init_embeddings(w_in, w_out, seed: int):
    ref = w_in if w_in is not None else w_out
    n, d = ref.shape
    _check(lib().gs_init_embeddings(_dev(w_in, torch.float32, "w_in", True),
                                    _dev(w_out, torch.float32, "w_out", True),
                                    ctypes.c_int64(n), ctypes.c_int32(d), ctypes.c_uint64(seed),
                                    _stream()))


def gs_random_walks(graph: Graph, starts, n_walks: int, walk_id_base: int, walk_len: int,
                    seed: int, out=None, steps=None):
    """Returns walks[n_walks, walk_len] (int32, CUDA).  steps: optional uint64/int64[1] counter."""
    if out is None:
        out = torch.empty((n_walks, walk_len), dtype=torch.int32, device=graph.cols.device)
    _check(lib().gs_random_walks(
        graph._h, _dev(starts, torch.int32, "starts", True), ctypes.c_int64(n_walks),
        ctypes.c_int64(walk_id_base), ctypes.c_int32(walk_len), ctypes.c_uint64(seed),
        _dev(out, torch.int32, "out"), _dev(steps, torch.int64, "steps", True), _stream()))
    return out


def gs_node2vec_walks(graph: Graph, starts, n_walks: int, walk_id_base: int, walk_len: int,
                      seed: int, p: float, q: float, max_rounds: int = 1024, out=None,
                      steps=None, cap_hits=None):
    if out is None:
        out = torch.empty((n_walks, walk_len), dtype=torch.int32, device=graph.cols.device)
    _check(lib().gs_node2vec_walks(
        graph._h, _dev(starts, torch.int32, "starts", True), ctypes.c_int64(n_walks),
        ctypes.c_int64(walk_id_base), ctypes.c_int32(walk_len), ctypes.c_uint64(seed),
        ctypes.c_double(p), ctypes.c_double(q), ctypes.c_int32(max_rounds),
        _dev(out, torch.int32, "out"), _dev(steps, torch.int64, "steps", True),
        _dev(cap_hits, torch.int64, "cap_hits", True), _stream()))
    return out


def gs_sgns_step(w_in, w_out, walks, walk_id_base: int, window: int, n_neg: int, alias,
                 lr: float, seed: int, mode: int, loss_sum=None, pair_count=None,
                 pairs_dump=None, negs_dump=None):
    """One SGNS update over walks[n_walks, walk_len]; loss_sum (float64[1]) and pair_count
    (int64[1]) are accumulated into; dumps are optional int32 tensors (see gs.h)."""
    n_nodes, dim = w_in.shape
    n_walks, walk_len = walks.shape
    _check(lib().gs_sgns_step(
        _dev(w_in, torch.float32, "w_in"), _dev(w_out, torch.float32, "w_out"),
        ctypes.c_int64(n_nodes), ctypes.c_int32(dim), _dev(walks, torch.int32, "walks", n_walks == 0),
        ctypes.c_int64(n_walks), ctypes.c_int64(walk_id_base), ctypes.c_int32(walk_len),
        ctypes.c_int32(window), ctypes.c_int32(n_neg), _dev(alias, torch.int64, "alias", n_neg == 0),
        ctypes.c_float(lr), ctypes.c_uint64(seed), ctypes.c_int32(mode),
        _dev(loss_sum, torch.float64, "loss_sum", True), _dev(pair_count, torch.int64, "pair_count", True),
        _dev(pairs_dump, torch.int32, "pairs_dump", True), _dev(negs_dump, torch.int32, "negs_dump", True),
        _stream()))


def gs_init_embeddings_f16(w_in, w_out, seed: int):
    """Start values of gs_init_embeddings rounded to half; tables are torch.float16."""
    ref = w_in if w_in is not None else w_out
    n, d = ref.shape
    _check(lib().gs_init_embeddings_f16(_dev(w_in, torch.float16, "w_in", True),
                                        _dev(w_out, torch.float16, "w_out", True),
                                        ctypes.c_int64(n), ctypes.c_int32(d), ctypes.c_uint64(seed),
                                        _stream()))


def gs_sgns_step_f16(w_in, w_out, walks, walk_id_base: int, window: int, n_neg: int, alias,
                     lr: float, seed: int, mode: int, loss_sum=None, pair_count=None,
                     pairs_dump=None, negs_dump=None):
    """gs_sgns_step on torch.float16 tables (fp32 arithmetic, round-to-nearest write-back)."""
    n_nodes, dim = w_in.shape
    n_walks, walk_len = walks.shape
    _check(lib().gs_sgns_step_f16(
        _dev(w_in, torch.float16, "w_in"), _dev(w_out, torch.float16, "w_out"),
        ctypes.c_int64(n_nodes), ctypes.c_int32(dim), _dev(walks, torch.int32, "walks", n_walks == 0),
        ctypes.c_int64(n_walks), ctypes.c_int64(walk_id_base), ctypes.c_int32(walk_len),
        ctypes.c_int32(window), ctypes.c_int32(n_neg), _dev(alias, torch.int64, "alias", n_neg == 0),
        ctypes.c_float(lr), ctypes.c_uint64(seed), ctypes.c_int32(mode),
        _dev(loss_sum, torch.float64, "loss_sum", True), _dev(pair_count, torch.int64, "pair_count", True),
        _dev(pairs_dump, torch.int32, "pairs_dump", True), _dev(negs_dump, torch.int32, "negs_dump", True),
        _stream()))


def gs_init_embeddings_bf16(w_in, w_out, seed: int):
    """Start values of gs_init_embeddings rounded to bfloat16; tables are torch.bfloat16."""
    ref = w_in if w_in is not None else w_out
    n, d = ref.shape
    _check(lib().gs_init_embeddings_bf16(_dev(w_in, torch.bfloat16, "w_in", True),
                                        _dev(w_out, torch.bfloat16, "w_out", True),
                                        ctypes.c_int64(n), ctypes.c_int32(d), ctypes.c_uint64(seed),
                                        _stream()))


def gs_sgns_step_bf16(w_in, w_out, walks, walk_id_base: int, window: int, n_neg: int, alias,
                     lr: float, seed: int, mode: int, loss_sum=None, pair_count=None,
                     pairs_dump=None, negs_dump=None):
    """gs_sgns_step on torch.bfloat16 tables (fp32 arithmetic, round-to-nearest write-back)."""
    n_nodes, dim = w_in.shape
    n_walks, walk_len = walks.shape
    _check(lib().gs_sgns_step_bf16(
        _dev(w_in, torch.bfloat16, "w_in"), _dev(w_out, torch.bfloat16, "w_out"),
        ctypes.c_int64(n_nodes), ctypes.c_int32(dim), _dev(walks, torch.int32, "walks", n_walks == 0),
        ctypes.c_int64(n_walks), ctypes.c_int64(walk_id_base), ctypes.c_int32(walk_len),
        ctypes.c_int32(window), ctypes.c_int32(n_neg), _dev(alias, torch.int64, "alias", n_neg == 0),
        ctypes.c_float(lr), ctypes.c_uint64(seed), ctypes.c_int32(mode),
        _dev(loss_sum, torch.float64, "loss_sum", True), _dev(pair_count, torch.int64, "pair_count", True),
        _dev(pairs_dump, torch.int32, "pairs_dump", True), _dev(negs_dump, torch.int32, "negs_dump", True),
        _stream()))


def gs_sgns_step_static(w_in, w_out, walks, walk_id_base: int, window: int, n_neg: int, alias,
                        lr: float, seed: int, loss_sum=None, pair_count=None):
    """Deterministic SGNS step that allocates nothing on the device (fixed 32 MiB scratch inside
    the library).  For callers that may not call cudaMalloc; small batches only - see gs.h."""
    n_nodes, dim = w_in.shape
    n_walks, walk_len = walks.shape
    _check(lib().gs_sgns_step_static(
        _dev(w_in, torch.float32, "w_in"), _dev(w_out, torch.float32, "w_out"),
        ctypes.c_int64(n_nodes), ctypes.c_int32(dim), _dev(walks, torch.int32, "walks", n_walks == 0),
        ctypes.c_int64(n_walks), ctypes.c_int64(walk_id_base), ctypes.c_int32(walk_len),
        ctypes.c_int32(window), ctypes.c_int32(n_neg), _dev(alias, torch.int64, "alias", n_neg == 0),
        ctypes.c_float(lr), ctypes.c_uint64(seed),
        _dev(loss_sum, torch.float64, "loss_sum", True), _dev(pair_count, torch.int64, "pair_count", True),
        _stream()))


def gs_sgns_step_momentum(w_in, w_out, m_in, m_out, last_in, last_out, walks, walk_id_base: int,
                          window: int, n_neg: int, alias, lr: float, momentum: float, iteration: int,
                          seed: int, loss_sum=None, pair_count=None):
    """Synchronous step with SGD momentum, rows updated lazily (see gs.h)."""
    n_nodes, dim = w_in.shape
    n_walks, walk_len = walks.shape
    _check(lib().gs_sgns_step_momentum(
        _dev(w_in, torch.float32, "w_in"), _dev(w_out, torch.float32, "w_out"),
        _dev(m_in, torch.float32, "m_in"), _dev(m_out, torch.float32, "m_out"),
        _dev(last_in, torch.int32, "last_in"), _dev(last_out, torch.int32, "last_out"),
        ctypes.c_int64(n_nodes), ctypes.c_int32(dim), _dev(walks, torch.int32, "walks", n_walks == 0),
        ctypes.c_int64(n_walks), ctypes.c_int64(walk_id_base), ctypes.c_int32(walk_len),
        ctypes.c_int32(window), ctypes.c_int32(n_neg), _dev(alias, torch.int64, "alias", n_neg == 0),
        ctypes.c_float(lr), ctypes.c_float(momentum), ctypes.c_int32(iteration), ctypes.c_uint64(seed),
        _dev(loss_sum, torch.float64, "loss_sum", True), _dev(pair_count, torch.int64, "pair_count", True),
        _stream()))


def gs_momentum_flush(w, m, last, lr: float, momentum: float, iteration: int):
    n_rows, dim = w.shape
    _check(lib().gs_momentum_flush(
        _dev(w, torch.float32, "w"), _dev(m, torch.float32, "m"), _dev(last, torch.int32, "last"),
        ctypes.c_int64(n_rows), ctypes.c_int32(dim), ctypes.c_float(lr), ctypes.c_float(momentum),
        ctypes.c_int32(iteration), _stream()))


def gs_sgns_step_adam(w_in, w_out, m_in, v_in, m_out, v_out, walks, walk_id_base: int, window: int,
                      n_neg: int, alias, lr: float, beta1: float, beta2: float, eps: float, step: int,
                      seed: int, pair_mode: int = 0, loss_sum=None, pair_count=None):
    """Synchronous step with Adam on the rows of the batch (see gs.h); step counts from 1."""
    n_nodes, dim = w_in.shape
    n_walks, walk_len = walks.shape
    _check(lib().gs_sgns_step_adam(
        _dev(w_in, torch.float32, "w_in"), _dev(w_out, torch.float32, "w_out"),
        _dev(m_in, torch.float32, "m_in"), _dev(v_in, torch.float32, "v_in"),
        _dev(m_out, torch.float32, "m_out"), _dev(v_out, torch.float32, "v_out"),
        ctypes.c_int64(n_nodes), ctypes.c_int32(dim), _dev(walks, torch.int32, "walks", n_walks == 0),
        ctypes.c_int64(n_walks), ctypes.c_int64(walk_id_base), ctypes.c_int32(walk_len),
        ctypes.c_int32(window), ctypes.c_int32(n_neg), _dev(alias, torch.int64, "alias", n_neg == 0),
        ctypes.c_float(lr), ctypes.c_float(beta1), ctypes.c_float(beta2), ctypes.c_float(eps),
        ctypes.c_int64(step), ctypes.c_uint64(seed), ctypes.c_int32(pair_mode),
        _dev(loss_sum, torch.float64, "loss_sum", True), _dev(pair_count, torch.int64, "pair_count", True),
        _stream()))


def gs_build_keep_thresholds(weights: np.ndarray, t: float) -> np.ndarray:
    """Host call.  Sub-sampling thresholds (uint32, 0xFFFFFFFF = always kept)."""
    w = np.ascontiguousarray(weights, dtype=np.float64)
    out = np.empty(len(w), dtype=np.uint32)
    _check(lib().gs_build_keep_thresholds(w.ctypes.data_as(ctypes.c_void_p), ctypes.c_int64(len(w)),
                                          ctypes.c_double(t), out.ctypes.data_as(ctypes.c_void_p)))
    return out


def gs_subsample_walks(walks, walk_id_base: int, keep_thr, seed: int, out=None, kept=None):
    """Drops walk entries by the thresholds (int32 CUDA tensor holding the uint32 bit patterns)
    and compacts each walk; out may be walks itself."""
    n_walks, walk_len = walks.shape
    if out is None:
        out = torch.empty_like(walks)
    _check(lib().gs_subsample_walks(
        _dev(walks, torch.int32, "walks", n_walks == 0), ctypes.c_int64(n_walks),
        ctypes.c_int64(walk_id_base), ctypes.c_int32(walk_len),
        _dev(keep_thr, torch.int32, "keep_thr", n_walks == 0),
        ctypes.c_int64(keep_thr.numel() if keep_thr is not None else 1), ctypes.c_uint64(seed),
        _dev(out, torch.int32, "out", n_walks == 0), _dev(kept, torch.int64, "kept", True), _stream()))
    return out


def gs_shuffled_starts(n_nodes: int, seed: int, epoch: int, walk_id_first: int, count: int, device,
                       out=None):
    """Start nodes of walk ids [first, first + count) under the keyed bijection of the epoch."""
    if out is None:
        out = torch.empty(count, dtype=torch.int32, device=device)
    _check(lib().gs_shuffled_starts(ctypes.c_int64(n_nodes), ctypes.c_uint64(seed),
                                    ctypes.c_uint32(epoch), ctypes.c_int64(walk_id_first),
                                    ctypes.c_int64(count), _dev(out, torch.int32, "out", count == 0),
                                    _stream()))
    return out


@dataclass
class EpochResult:
    loss_sum: float
    pairs: int
    steps: int
    cap_hits: int
    batches: int
    masked_negs: int
    ms_walk: float
    ms_sgns: float
    ms_total: float
    ms_prepare: float = 0.0
    refused_ids: int = 0


def gs_sgns_epoch(graph: Graph, alias, w_in, w_out, *, walks_per_node, walk_len, window, n_neg,
                  lr0, batch_walks, seed, mode, walk_kind=GS_WALK_UNIFORM,
                  lr_schedule=GS_LR_CONSTANT, p=1.0, q=1.0, max_rounds=1024, first_batch=0,
                  num_batches=0, keep_thr=None, shuffle_epoch=None, optimizer=GS_OPT_SGD, momentum=0.0,
                  beta2=0.999, eps=1e-8, iteration_base=0, m_in=None, m_out=None, v_in=None, v_out=None,
                  last_in=None, last_out=None) -> EpochResult:
    if w_in.dtype not in (torch.float32, torch.float16, torch.bfloat16) or w_out.dtype != w_in.dtype:
        raise TypeError("tables must both be float32, both float16 or both bfloat16")
    tdt = w_in.dtype
    cfg = SgnsConfig(dim=w_in.shape[1], walks_per_node=walks_per_node, walk_len=walk_len,
                     window=window, n_neg=n_neg, walk_kind=walk_kind, lr_schedule=lr_schedule,
                     mode=mode, max_rounds=max_rounds,
                     table_dtype={torch.float16: GS_TABLE_F16, torch.bfloat16: GS_TABLE_BF16}.get(tdt, GS_TABLE_F32),
                     p=p, q=q, lr0=lr0,
                     batch_walks=batch_walks, first_batch=first_batch, num_batches=num_batches,
                     seed=seed, d_keep_thr=_dev(keep_thr, torch.int32, "keep_thr", True).value,
                     shuffle_starts=0 if shuffle_epoch is None else 1,
                     epoch=0 if shuffle_epoch is None else shuffle_epoch,
                     optimizer=optimizer, momentum=momentum, beta2=beta2, eps=eps,
                     iteration_base=iteration_base,
                     d_m_in=_dev(m_in, torch.float32, "m_in", True).value,
                     d_m_out=_dev(m_out, torch.float32, "m_out", True).value,
                     d_v_in=_dev(v_in, torch.float32, "v_in", True).value,
                     d_v_out=_dev(v_out, torch.float32, "v_out", True).value,
                     d_last_in=_dev(last_in, torch.int32, "last_in", True).value,
                     d_last_out=_dev(last_out, torch.int32, "last_out", True).value)
    st = EpochStats()
    _check(lib().gs_sgns_epoch(graph._h, _dev(alias, torch.int64, "alias", n_neg == 0),
                               _dev(w_in, tdt, "w_in"), _dev(w_out, tdt, "w_out"),
                               ctypes.byref(cfg), ctypes.byref(st), _stream()))
    return EpochResult(st.loss_sum, st.pairs, st.steps, st.cap_hits, st.batches, st.masked_negs, st.ms_walk,
                       st.ms_sgns, st.ms_total, st.ms_prepare, st.refused_ids)


def gs_refused_ids(clear: bool = False) -> int:
    """Ids refused by the kernels of the current device so far (waits for the current stream)."""
    out = ctypes.c_uint64(0)
    _check(lib().gs_refused_ids(ctypes.byref(out), ctypes.c_int32(1 if clear else 0), _stream()))
    return out.value


def gs_release_workspace():
    _check(lib().gs_release_workspace())


def gs_tune_node2vec_group(lanes: int):
    _check(lib().gs_tune_node2vec_group(ctypes.c_int32(lanes)))
