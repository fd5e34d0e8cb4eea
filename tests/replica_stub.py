"""A stand-in for one benchmark rank, run by tests/test_replicas_gloo.py through
replicas.launch: joins the gloo group, "times" a stub step (no GPU), reduces like bench.py
does and lets rank 0 print the line."""
import json
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from paper_2511_04063_b200 import inputs as gen      # noqa: E402
from paper_2511_04063_b200 import replicas           # noqa: E402


def main():
    out_dir = sys.argv[1]
    rank, local_rank, world = replicas.init_process_group("gloo")
    w = replicas.workload_for_rank(gen.scaled(gen.WORKLOADS["c2_7b"], d=64, n_tokens=128, n_outlier_channels=2), rank)
    steps = 20
    ms_local = 10.0 + 5.0 * rank                      # the stub step: rank 1 is the slow one
    replicas.barrier()
    line = replicas.headline("calibration steps/sec", "steps/s", steps, world, ms_local)
    line["seed"] = w.seed
    with open(os.path.join(out_dir, "rank%d.json" % rank), "w") as f:
        json.dump({"rank": rank, "local_rank": local_rank, "world": world, "line": line}, f)
    if rank == 0:
        print(json.dumps(line), flush=True)
    replicas.shutdown()


if __name__ == "__main__":
    main()
