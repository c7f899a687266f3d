"""bench.py's own rank launcher, on CPU: ``--gpus 2`` outside a torch.distributed launch must start two ranks
(gloo here, a host stand-in for the step), take the maximum over ranks and let rank 0 print one line with
``n_gpus: 2``; inside a launch (WORLD_SIZE set) it must not start ranks again."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def run_bench(*argv, env=None):
    e = dict(os.environ)
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT"):
        e.pop(k, None)
    e.update(env or {})
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *argv], capture_output=True, text=True, env=e, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, r.stdout[-2000:]          # rank 0 alone prints
    return json.loads(lines[0])


def test_gpus_2_starts_two_ranks():
    line = run_bench("--stub-step", "--gpus", "2", "--steps", "2")
    assert line["n_gpus"] == 2 and line["stub"] is True and line["scaling"] == "weak"
    assert line["config"]["parallelism"].startswith("dp2")
    one = run_bench("--stub-step", "--gpus", "1", "--steps", "2")
    assert one["n_gpus"] == 1
    # whole-job value: both ranks' requests over the slowest rank's time
    assert abs(line["value"] - 2 * line["config"]["requests_per_gpu"] / (line["ms_per_step"] * 1e-3)) <= 1e-6 * line["value"]


def test_inside_a_launch_no_second_launch():
    # WORLD_SIZE = 1 stands for "already launched": --gpus 4 must then run as the single rank it is
    line = run_bench("--stub-step", "--gpus", "4", "--steps", "2", env={"WORLD_SIZE": "1", "RANK": "0", "LOCAL_RANK": "0"})
    assert line["n_gpus"] == 1
