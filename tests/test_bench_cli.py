"""Host-side checks of bench.py that need no GPU: `--gpus N` without a torchrun environment starts N ranks itself
(one process per GPU, rendezvous on 127.0.0.1), and the traffic table only answers for unchanged kernel sources."""
import importlib
import json
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _bench():
    if ROOT not in sys.path:
        sys.path.insert(0, ROOT)
    return importlib.import_module("bench")


def test_gpus_flag_spawns_one_rank_per_gpu(monkeypatch):
    bench = _bench()
    seen = {}

    def fake_call(cmd, env=None):
        seen["cmd"], seen["env"] = cmd, env
        return 0

    monkeypatch.setattr(bench.subprocess, "call", fake_call)
    monkeypatch.delenv("WORLD_SIZE", raising=False)
    monkeypatch.delenv("NCCL_DEBUG", raising=False)
    monkeypatch.setattr(sys, "argv", ["bench.py", "--gpus", "4", "--steps", "2", "--warmup", "3"])
    assert bench.main() == 0
    cmd = seen["cmd"]
    assert cmd[1:3] == ["-m", "torch.distributed.run"] and "--nproc-per-node=4" in cmd and "--nnodes=1" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert 0 < int(cmd[cmd.index("--master-port") + 1]) < 65536
    assert os.path.basename(cmd[cmd.index("--master-port") + 2]) == "bench.py"
    assert cmd[-6:] == ["--gpus", "4", "--steps", "2", "--warmup", "3"]
    assert seen["env"]["NCCL_DEBUG"] == "INFO" and "NCCL_DEBUG_FILE" in seen["env"]      # the communicator log stays on


def test_under_torchrun_nothing_is_spawned(monkeypatch):
    bench = _bench()
    called = []
    monkeypatch.setattr(bench.subprocess, "call", lambda *a, **k: called.append(a) or 0)
    monkeypatch.setattr(bench, "run_ours", lambda args: 7)
    monkeypatch.setenv("WORLD_SIZE", "4")
    monkeypatch.setattr(sys, "argv", ["bench.py", "--gpus", "4"])
    assert bench.main() == 7 and not called


def test_traffic_table_rows_go_stale_with_the_source(tmp_path, monkeypatch):
    bench = _bench()
    with open(bench.TRAFFIC_TABLE) as f:
        table = json.load(f)
    assert {"cwac_stats_kernel", "qlinear_cwac_kernel@cfg4"} <= set(table)
    for row in table.values():
        assert os.path.exists(os.path.join(ROOT, row["profile"].split(" ")[0]))
        assert all(os.path.exists(os.path.join(bench.CSRC, f)) for f in row["source_files"])
    key = "cwac_stats_kernel"
    fake = dict(table)
    fake[key] = dict(table[key], source_sha=bench.source_hash(table[key]["source_files"]))
    p = tmp_path / "t.json"
    p.write_text(json.dumps(fake))
    monkeypatch.setattr(bench, "TRAFFIC_TABLE", str(p))
    ratio, prov = bench.traffic_ratio(key)
    assert ratio == table[key]["dram_bytes_per_algorithmic_byte"] and prov.startswith("profiles/")
    fake[key]["source_sha"] = "0" * 16
    p.write_text(json.dumps(fake))
    ratio, why = bench.traffic_ratio(key)
    assert ratio is None and "changed" in why
    assert bench.traffic_ratio("no such kernel")[0] is None
