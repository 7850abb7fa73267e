"""Shared glue of the tests: data conversion between the oracle (numpy) and the library
(torch CUDA tensors).  No arithmetic of the method lives here."""
import numpy as np
import torch

from oracle import gs_oracle as O


def np_graph(g):
    return g.offsets.cpu().numpy().astype(np.int64), g.cols.cpu().numpy()


def pack_alias(thr, alias):
    """(thr uint32, alias int32) -> packed uint64 entries: thr low, alias high."""
    return (alias.astype(np.uint64) << np.uint64(32)) | thr.astype(np.uint64)


def unpack_alias(table):
    t = np.asarray(table, dtype=np.uint64)
    return (t & np.uint64(0xFFFFFFFF)).astype(np.uint32), (t >> np.uint64(32)).astype(np.int32)


def alias_to_device(thr, alias, device="cuda"):
    return torch.from_numpy(pack_alias(thr, alias).view(np.int64)).to(device)


def degree_alias(off):
    deg = (off[1:] - off[:-1]).astype(np.float64)
    return O.build_alias(deg, 0.75)


def compact_problem(centers, contexts, negs):
    """Renumber the node ids that occur in the lists to 0..m-1 (a one-to-one map), so that the
    oracle can work on the touched rows only.  Returns (ids, c, o, ng) with -1 kept."""
    allv = np.concatenate([centers, contexts, negs.ravel()])
    ids = np.unique(allv[allv >= 0])
    def remap(a):
        out = np.full(a.shape, -1, dtype=np.int32)
        m = a >= 0
        out[m] = np.searchsorted(ids, a[m]).astype(np.int32)
        return out
    return ids, remap(centers), remap(contexts), remap(negs)
