"""`bench.py --gpus 2` started as one process, on CPU: the launcher starts two ranks (gloo), each runs a stand-in
job that has no kernels, the timing is reduced as the max over ranks, and rank 0 prints one line whose n_gpus is the
number of ranks that really ran."""
import json
import time

import bench
from paper_2507_00715_b200 import replicas, workloads as wl


class StandInJob:
    """What the rank logic needs from a job, with a sleep where the kernels would be; rank 1 is the slow replica."""
    launches_per_step = 7

    def __init__(self, w, device, rank):
        self.w, self.rank, self.steps = w, rank, 0

    def step(self, record=False):
        time.sleep(0.004 * (self.rank + 1))
        self.steps += 1

    def segment_times(self):
        return {}

    def device_status(self):
        return 0

    def kv_entries(self, generated):
        return 1


def test_gpus_flag_without_a_launcher_starts_the_ranks_itself(capfd, monkeypatch):
    for var in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT"):
        monkeypatch.delenv(var, raising=False)
    bench.main(["--gpus", "2", "--steps", "3", "--warmup", "3", "--config", "tiny"], backend="gloo",
               job_factory=StandInJob)
    lines = [json.loads(l) for l in capfd.readouterr().out.splitlines() if l.startswith("{")]
    assert len(lines) == 1, "exactly one rank prints"
    line = lines[0]
    w = wl.CONFIGS["tiny"]
    tokens = int(wl.seqlens(w).sum()) + w.batch * w.beams * w.decode_steps
    assert line["n_gpus"] == 2 and line["steps"] == 3 and line["scaling"] == "weak"
    assert line["ms_per_step"] >= 8.0                      # the slow rank's 8 ms per step, not rank 0's 4 ms
    assert abs(line["value"] - replicas.job_throughput(tokens, 2, line["ms_per_step"] * 1e-3)) < 1e-6 * line["value"]
    assert line["gpu_launches"] == 7 * 3


def test_one_gpu_runs_in_process(capfd, monkeypatch):
    for var in ("RANK", "LOCAL_RANK", "WORLD_SIZE"):
        monkeypatch.delenv(var, raising=False)
    bench.main(["--gpus", "1", "--steps", "2", "--config", "tiny"], backend="gloo", job_factory=StandInJob)
    line = json.loads([l for l in capfd.readouterr().out.splitlines() if l.startswith("{")][0])
    assert line["n_gpus"] == 1 and line["ms_per_step"] >= 4.0


def test_decode_steps_override_gives_the_prefill_only_point():
    args = bench.parse_args(["--decode-steps", "0"])
    w = bench.pick_workload(args)
    assert w.decode_steps == 0 and w.name == "7b"
    a = bench.algorithmic(w)
    # compaction moves the K and V register rows (read + write) and the index list
    assert a["compact"]["bytes"] == 2 * 2 * 64 * 32 * 8 * 128 * 2 + 64 * 32 * 4
    assert a["register"]["bytes"] == 64 * 32 * 128 * 2 * (2 * 32 + 2 * 8)
