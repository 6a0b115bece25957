"""Host logic of the bench: byte accounting, and the replicas-only multi-GPU aggregation run as two
gloo ranks on CPU (the job's time is the slowest rank's; no data-path collective exists)."""
import json
import os
import subprocess
import sys
import textwrap
from pathlib import Path

import numpy as np

import oracle
from paper_2608_09291_b200 import workloads

ROOT = Path(__file__).resolve().parent.parent
sys.path.insert(0, str(ROOT))
import bench  # noqa: E402


def test_algorithmic_bytes_closed_form():
    from paper_2608_09291_b200 import binding as b
    W = workloads.make_weight(256, 2048, 0.5, seed=7)
    h = b.us_encode(W, fmt=(16, 1024, 2, 1), flags=b.US_ENCODE_HOST_ONLY)
    st = b.us_get_stats(h)
    b.us_destroy(h)
    ref = oracle.encode(W, 16, 1024, 2, 1)["stats"]
    got = bench.algorithmic_bytes(st, 8, True)
    want = ref["bytes_payload"] + 256 * 2048 // 16 + 4 * (ref["n_lt"] + 1) + 8 * 1024 + 8 * 256 * 2 + 2 * (256 + 8)
    assert got == want
    # expectation for a Bernoulli mask, per dense element: 0.5 (1 - s^2) + 1/16 + 4/(16*1024)
    per_elem = (ref["bytes_payload"] + ref["bytes_bitmap"] + ref["bytes_offsets"]) / (256 * 2048)
    assert abs(per_elem - (0.5 * 0.75 + 1 / 16 + 1 / 4096)) < 3e-3


def test_max_over_ranks_two_gloo_ranks(tmp_path):
    script = tmp_path / "rank.py"
    src = textwrap.dedent(f"""
        import os, sys, json
        sys.path.insert(0, {str(ROOT)!r})
        import torch.distributed as dist
        import bench
        dist.init_process_group("gloo")
        r = dist.get_rank()
        t = bench.max_over_ranks(1.0 + r, dist, "cpu")
        dist.barrier()
        open(os.path.join({str("OUTDIR")!r}, f"rank{{r}}.json"), "w").write(json.dumps({{"rank": r, "t": t}}))
        dist.destroy_process_group()
    """)
    script.write_text(src.replace("OUTDIR", str(tmp_path)))
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29531")
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
                          "--master-addr", "127.0.0.1", "--master-port", "29531", str(script)],
                         capture_output=True, text=True, env=env, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    recs = [json.loads((tmp_path / f"rank{r}.json").read_text()) for r in (0, 1)]
    assert sorted(r["rank"] for r in recs) == [0, 1]
    assert all(r["t"] == 2.0 for r in recs)        # both ranks see the slowest rank's time


def test_reference_arm_prints_contract_line():
    out = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0"],
                         capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    d = json.loads(out.stdout.strip().splitlines()[-1])
    assert d["impl"] == "reference" and d["metric"] == bench.METRIC and d["unit"] == bench.UNIT
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["value"] > 0


def test_gpus_flag_starts_replicas_or_refuses(monkeypatch):
    """--gpus N outside a torchrun environment re-launches the script as N replica processes; inside
    one, a world size that contradicts the flag is an error (the flag never lies about n_gpus)."""
    cmd = bench.torchrun_command(["--gpus", "4", "--steps", "2"], 4, port=29999)
    assert cmd[1:4] == ["-m", "torch.distributed.run", "--nnodes=1"]
    assert cmd[cmd.index("--nproc-per-node") + 1] == "4" and cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert cmd[-4:] == ["--gpus", "4", "--steps", "2"] and cmd[-5].endswith("bench.py")
    called = {}
    monkeypatch.delenv("WORLD_SIZE", raising=False)
    monkeypatch.setattr(bench.os, "execvp", lambda exe, argv: called.setdefault("argv", argv) and (_ for _ in ()).throw(SystemExit(0)))
    try:
        bench.main(["--gpus", "2", "--steps", "1"])
    except SystemExit:
        pass
    assert called["argv"][called["argv"].index("--nproc-per-node") + 1] == "2"
    monkeypatch.setenv("WORLD_SIZE", "2")
    try:
        bench.main(["--gpus", "4"])
        raise AssertionError("a contradicting world size must be refused")
    except SystemExit as e:
        assert "WORLD_SIZE=2" in str(e)
