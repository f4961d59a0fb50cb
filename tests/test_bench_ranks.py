"""Host logic of the N > 1 benchmark path: the path does not shard, so N GPUs run N independent
replicas; the only cross-rank step is the max over ranks of the timed region.  Runs on CPU
with the gloo backend, world size 2."""
import json
import os
import socket
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys
sys.path.insert(0, {root!r})
import torch.distributed as dist
import bench
rank = int(os.environ["RANK"])
dist.init_process_group("gloo", init_method="tcp://127.0.0.1:{port}", rank=rank, world_size=2)
mine = 1.5 if rank == 0 else 2.25          # rank 1 is the slow one
got = bench.max_over_ranks(mine, dist, None)
alone = bench.max_over_ranks(mine, None, None)
dist.barrier()
dist.destroy_process_group()
print("RESULT", rank, got, alone)
"""


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


@pytest.mark.timeout(300)
def test_timed_region_is_the_max_over_ranks_gloo_world_size_2():
    code = WORKER.format(root=ROOT, port=_free_port())
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1")
        procs.append(subprocess.Popen([sys.executable, "-c", code], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=280) for p in procs]
    for p, (out, err) in zip(procs, outs):
        assert p.returncode == 0, err[-2000:]
    for rank, (out, _) in enumerate(outs):
        tag, r, got, alone = [ln for ln in out.splitlines() if ln.startswith("RESULT")][0].split()
        assert int(r) == rank
        assert float(got) == 2.25                       # every rank sees the slowest rank's time
        assert float(alone) == (1.5 if rank == 0 else 2.25)


def test_reference_arm_prints_on_rank_0_only():
    # under a multi-rank launch the other ranks leave without work and without output
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"],
                       env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_reference_arm_line_has_the_contract_keys():
    env = dict(os.environ, RANK="0", WORLD_SIZE="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                        "--warmup", "0", "--workload", "medium", "--scale", "0.02"],
                       env=env, capture_output=True, text=True, timeout=280)
    assert r.returncode == 0, r.stderr[-2000:]
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["metric"] == "aggregated_edges_per_s" and line["unit"] == "edges/s"
    assert line["higher_is_better"] is True and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] == 1
    assert line["e2e"] == {"value": line["value"], "unit": "edges/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}


def test_clock_samples_are_windowed_to_the_timed_region():
    """The clock sampler starts before the warm-up (nvidia-smi is slow to deliver its first sample);
    only samples that arrived during the timed region may enter the record, and throttle reasons
    seen outside it must not be charged to it."""
    sys.path.insert(0, ROOT)
    import bench

    class _Done:
        def terminate(self):
            pass

        def wait(self, timeout=None):
            return 0

    s = bench.ClockSampler(0)
    s.proc = _Done()
    s.t_begin, s.t_end = 100.0, 101.0
    s.lines = [
        (99.0, "1200, 1965, 300.0, Not Active, Active, Not Active, Not Active"),     # warm-up: thermal flag
        (100.2, "1800, 1965, 900.0, Not Active, Not Active, Not Active, Active"),
        (100.6, "1900, 1965, 950.0, Not Active, Not Active, Not Active, Active"),
        (101.05, "1850, 1965, 940.0, Not Active, Not Active, Not Active, Not Active"),  # one period late: kept
        (102.0, "600, 1965, 100.0, Active, Not Active, Not Active, Not Active"),      # after: hardware flag
    ]
    rec = s.stop()
    assert rec["samples"] == 3 and rec["sm_mhz"] == 1850.0 and rec["sm_max_mhz"] == 1965.0
    assert rec["reasons"] == ["sw_power_cap"] and rec["power_w_max"] == 950.0
    # without a window every sample counts
    s2 = bench.ClockSampler(0)
    s2.proc = _Done()
    s2.lines = list(s.lines)
    assert s2.stop()["samples"] == 5
