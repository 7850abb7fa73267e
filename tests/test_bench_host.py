"""Host logic of bench.py that needs no GPU: byte accounting, the recorded ncu traffic and its pin
to the kernel's source, the per-config legs."""
import hashlib
import importlib.util
import sys
from pathlib import Path

ROOT = Path(__file__).resolve().parent.parent


def load_bench():
    spec = importlib.util.spec_from_file_location("bench_module", ROOT / "bench.py")
    mod = importlib.util.module_from_spec(spec)
    sys.modules["bench_module"] = mod
    spec.loader.exec_module(mod)
    return mod


def test_algorithmic_bytes_match_the_stated_accounting():
    b = load_bench()
    # per pair (1 + K) rows read and written + K alias entries; per center position one row read and
    # written + its walk entry: d = 128, K = 5 gives 6184 B per pair and 1028 B per position
    assert b.algorithmic_bytes(1, 0, 128, 5) == 6 * 2 * 4 * 128 + 8 * 5 == 6184
    assert b.algorithmic_bytes(0, 1, 128, 5) == 2 * 4 * 128 + 4 == 1028
    assert b.algorithmic_bytes(10, 3, 64, 10, elem=2) == 10 * (11 * 2 * 2 * 64 + 80) + 3 * (2 * 2 * 64 + 4)
    # a transition over the walk index reads one 16-byte record and stores one entry; DRAM moves 64 bytes for it
    assert b.walk_bytes(7, True, indexed=True) == 7 * 20 and b.walk_granule_bytes(7, indexed=True) == 7 * 68
    assert b.walk_bytes(7, True) == 7 * 24 and b.walk_bytes(7, False) == 7 * 16


def test_recorded_traffic_is_pinned_to_the_kernel_part_of_the_source(tmp_path, monkeypatch):
    b = load_bench()
    got, note = b.recorded_traffic("sgns_hogwild_kernel", "deepwalk_large")
    src = (ROOT / "paper_2407_15452_b200" / "csrc" / "gs_sgns.cu").read_text()
    marker = "// ---------------------------------------------------------------- synchronous mode"
    assert marker in src
    text = (ROOT / "profiles" / "sgns_hogwild_kernel__deepwalk_large.md").read_text()
    pinned = hashlib.sha256(src[:src.index(marker)].encode()).hexdigest() in text
    # the figure is served exactly when the part of the file before the marker is the one captured
    assert (got is not None) == pinned
    if got is not None:
        assert 3000 < got < 7000 and "5M-node" in note
    # a changed kernel drops the figure: same summary, source with one more character
    fake = tmp_path / "repo"
    (fake / "profiles").mkdir(parents=True)
    (fake / "paper_2407_15452_b200" / "csrc").mkdir(parents=True)
    (fake / "profiles" / "sgns_hogwild_kernel__deepwalk_large.md").write_text(text)
    (fake / "paper_2407_15452_b200" / "csrc" / "gs_sgns.cu").write_text("// x\n" + src)
    monkeypatch.setattr(b, "ROOT", fake)
    assert b.recorded_traffic("sgns_hogwild_kernel", "deepwalk_large") == (None, None)
    assert b.recorded_traffic("no_such_kernel", "deepwalk_large") == (None, None)


def test_per_config_legs_name_known_workloads_and_cover_the_other_configurations():
    b = load_bench()
    sys.path.insert(0, str(ROOT))
    from paper_2407_15452_b200.workloads import WORKLOADS
    names = [leg[0] for leg in b.PER_CONFIG_LEGS]
    assert set(names) <= set(WORKLOADS)
    assert {"tiny_deepwalk", "deepwalk_medium", "node2vec_4m", "rmat_billion"} <= set(names)
    assert ("deepwalk_medium", "deterministic") in [(l[0], l[1]) for l in b.PER_CONFIG_LEGS]
    assert all(l[3] >= 3 for l in b.PER_CONFIG_LEGS)                 # at least three warm-up steps each
    # launches of a synchronous batch: walks, targets, 3 per radix pass, coefficients, apply, last launch
    assert b.sync_step_launches(1_000_000) == 1 + 1 + 9 + 1 + 2 and b.sync_step_launches(50_000_000) == 1 + 1 + 12 + 1 + 2
