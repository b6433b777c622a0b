"""The multi-GPU mode is "replicas only": N independent contexts, no collective on the data path.
What N > 1 adds is host logic -- per-rank seeds, the barrier, the max-over-ranks of the device
time, the whole-job aggregate -- covered here with two gloo ranks on the CPU."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _torchrun(script_args, tmp_path, extra_env=None):
    env = dict(os.environ, **(extra_env or {}))
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port())] + script_args
    return subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)


def test_two_replicas_draw_their_own_inputs_and_share_the_slowest_time(tmp_path):
    out = tmp_path / "rank0.json"
    r = _torchrun([os.path.join(ROOT, "tests", "_rank_worker.py")], tmp_path, {"VVS_RANK_TEST_OUT": str(out)})
    assert r.returncode == 0, r.stderr[-2000:]
    res = json.loads(out.read_text())
    assert res["world"] == 2
    assert res["fills"][0] != res["fills"][1]                 # different seeds, different cache fills
    assert res["ms_total"] == 11.0 and res["ms_e2e"] == 20.0  # element-wise maximum over the ranks
    assert abs(res["value"] - 2 * res["drafts"] * 4 / 11e-3) < 1e-6
    # regions of 4 steps, each timed as the slower rank's 70 + i, until 500 ms are covered: 71 + ... + 77 = 518
    assert res["regions"] == [71.0 + i for i in range(7)] and res["region_calls"] == [4] * 7


def test_reference_arm_runs_on_rank_0_only(tmp_path):
    """Under torchrun the oracle arm is timed by rank 0 alone; the other rank leaves at once."""
    r = _torchrun([os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                   "--workload", "1"], tmp_path)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["cpu_baseline"]["kind"] == "oracle" and d["value"] > 0
