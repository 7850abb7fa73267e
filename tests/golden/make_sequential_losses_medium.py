"""Writes tests/golden/sequential_losses_medium.txt: the mean training loss of strictly sequential
SGNS (the oracle's sequential mode, fp64) over the first 16 stretches of 16,384 walks of the 1M-node
DeepWalk workload, at the workload's own learning rate.

    python tests/golden/make_sequential_losses_medium.py          (about seven minutes on one core)

Calls only the oracle and the seeded input generators.  The graph is generated on the CPU; the
test that reads the file generates it the same way.  Sequential SGD is the race-free execution of
the lock-free schedule (Section 3.2 "Synchronization" of the paper: trainers write increments
without waiting for each other), so these values are what a lock-free run is compared with.
"""
import sys
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parents[2]
sys.path.insert(0, str(ROOT))

from oracle import gs_oracle as O                                  # noqa: E402
from paper_2407_15452_b200 import workloads as WL                 # noqa: E402

STRETCH, N_STRETCHES, SEED = 16384, 16, 1


def main():
    wl = WL.WORKLOADS["deepwalk_medium"]
    g = wl.make_graph()
    n = g.n_nodes
    off = g.offsets.numpy().astype(np.int64)
    col = g.cols.numpy()
    thr, alias = O.build_alias((off[1:] - off[:-1]).astype(np.float64), 0.75)
    U = O.init_rows(np.arange(n), wl.dim, SEED)
    V = np.zeros_like(U)
    lines = ["# Mean SGNS loss per pair of the oracle's sequential mode (fp64) over consecutive stretches of",
             f"# {STRETCH} walks of workload deepwalk_medium (graph seed {wl.graph_seed}, CPU-generated; walk and table",
             f"# seed {SEED}; lr {wl.lr0} constant).  Written by tests/golden/make_sequential_losses_medium.py.",
             "# stretch  mean_loss  pairs"]
    for b in range(N_STRETCHES):
        r = O.sgns_epoch(off, col, thr, alias, U, V, walks_per_node=wl.walks_per_node, L=wl.walk_len,
                         w=wl.window, K=wl.n_neg, lr0=wl.lr0, schedule="constant", batch_walks=STRETCH,
                         seed=SEED, mode="seq", first_batch=b, num_batches=1)
        lines.append(f"{b} {r['loss_sum'] / r['pairs']!r} {r['pairs']}")
        print(lines[-1], flush=True)
    (Path(__file__).parent / "sequential_losses_medium.txt").write_text("\n".join(lines) + "\n")


if __name__ == "__main__":
    main()
