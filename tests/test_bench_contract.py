"""bench.py's reference arm (the oracle on host cores) prints one JSON line with the contract's keys."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_prints_one_contract_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0",
                          "--workload", "rep_n15_s2_d100k"], capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert out.returncode == 0, out.stderr
    lines = [ln for ln in out.stdout.splitlines() if ln.strip()]
    assert len(lines) == 1
    rec = json.loads(lines[0])
    for key in ("impl", "metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "cpu_baseline", "e2e"):
        assert key in rec, key
    assert rec["impl"] == "reference" and rec["value"] > 0 and rec["vs_baseline"] is None
    assert rec["cpu_baseline"]["kind"] == "oracle" and rec["cpu_baseline"]["cores"] >= 1
    assert rec["e2e"]["h2d_bytes_per_step"] == 0 and rec["config"]["workload"] == "rep_n15_s2_d100k"


def test_non_zero_ranks_of_the_reference_arm_do_no_work():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0"],
                         capture_output=True, text=True, timeout=120, cwd=ROOT, env=env)
    assert out.returncode == 0 and out.stdout.strip() == ""


def test_sweep_table_renders_one_row_per_point(tmp_path):
    point = {"code": "cyc", "n": 15, "s": 2, "d": 1_000_000, "encode_ms": 0.05, "decode_ms": 0.08, "coded_GBps_produced": 2400.0,
             "coded_GBps_consumed": 1500.0, "encode_hbm_GBps": 3600.0, "encode_frac": 0.55, "decode_hbm_GBps": 3000.0,
             "decode_frac": 0.46, "checks": {"0": {"err": 2e-7}, "s": {"err": 3e-7}, ">s": {"err": 5.0}},
             "flags_ok_upto_s": True, "beyond_s_fails": True}
    path = tmp_path / "sweep.jsonl"
    path.write_text(json.dumps(point) + "\n" + json.dumps(dict(point, n=45, flags_ok_upto_s=False)) + "\n" + json.dumps({"mode": "sweep"}) + "\n")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--sweep-table", str(path)], capture_output=True, text=True,
                         timeout=120, cwd=ROOT)
    assert out.returncode == 0, out.stderr
    rows = [ln for ln in out.stdout.splitlines() if ln.startswith("| cyc")]
    assert len(rows) == 2 and "| 15 | 2 | 1.0 M | 0.050 | 3600 (0.55) | 0.080 | 3000 (0.46) | 2400 / 1500 |" in rows[0]
    assert rows[0].rstrip().endswith("| yes | yes |") and "| NO | yes |" in rows[1]


def test_gpus_n_started_by_hand_launches_n_ranks_under_torchrun():
    """`python bench.py --gpus 4` without torchrun's environment re-executes itself as 4 ranks (dry run: the plan only)."""
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "4", "--steps", "3", "--warmup", "3", "--dry-run"],
                         capture_output=True, text=True, timeout=120, cwd=ROOT, env=env)
    assert out.returncode == 0, out.stderr
    plan = json.loads(out.stdout.strip())
    cmd = plan["launch"]
    assert plan["ranks"] == 4 and cmd[1:3] == ["-m", "torch.distributed.run"]
    assert "--nproc-per-node=4" in cmd and "--standalone" in cmd and "--dry-run" not in cmd
    assert cmd[cmd.index("--local-addr") + 1] == "127.0.0.1" and plan["env"]["MASTER_ADDR"] == "127.0.0.1"
    tail = cmd[cmd.index(os.path.join(ROOT, "bench.py")) + 1:]
    assert tail == ["--gpus", "4", "--steps", "3", "--warmup", "3"]
    # one GPU, and the reference arm at any N, start no process group
    for extra in (["--gpus", "1"], ["--gpus", "4", "--impl", "reference"]):
        out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--dry-run"] + extra, capture_output=True, text=True,
                             timeout=120, cwd=ROOT, env=env)
        plan = json.loads(out.stdout.strip())
        assert plan["ranks"] == 1 and "torch.distributed.run" not in plan["launch"] and plan["env"] == {}
