"""One rank of a stand-in job for the benchmark's launcher test (CPU, gloo): joins the process group
from the environment bench.spawn_ranks gives it, pretends that its timed region took a rank-dependent
time, reduces that with the maximum over ranks as the benchmark does, and lets rank 0 print the
benchmark's one line through bench.build_line. No kernels, no oracle: only the plumbing is exercised."""
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import bench  # noqa: E402
from paper_2509_11628_b200 import dist as D  # noqa: E402

STEP_BYTES = 3.0e9          # per rank and step
BASE_MS, PER_RANK_MS = 10.0, 5.0


def main() -> int:
    info = D.init("gloo")
    assert info.world == int(os.environ["WORLD_SIZE"]) and info.rank == int(os.environ["RANK"])
    assert os.environ["MASTER_ADDR"] == "127.0.0.1" and int(os.environ["LOCAL_RANK"]) == info.rank
    D.barrier()
    mine_ms = BASE_MS + PER_RANK_MS * info.rank
    slowest = D.max_over_ranks(mine_ms)
    D.barrier()
    print("rank %d: this line must not reach the job's stdout unless it is rank 0's" % info.rank, file=sys.stderr)
    if info.is_main:
        k = {"ms": slowest, "gbs": 1.0, "algorithmic_bytes": 1}
        print(bench.build_line(
            value=bench.job_value(STEP_BYTES, info.world, slowest), ms_per_step=slowest, n_gpus=info.world, steps=4, warmup=3,
            config={"workload": "stub"}, roofline=None, cpu_baseline=None, e2e=None, gpu_launches=0, clocks=None,
            kernels={"update": k, "forecast": k, "verify": k, "select": k}, forecast_verify_gbs=1.0,
            speculative_steps_per_s=1.0), flush=True)
    else:
        print("a non-zero rank's stdout is dropped by the launcher", flush=True)
    D.shutdown()
    return 0


if __name__ == "__main__":
    sys.exit(main())
