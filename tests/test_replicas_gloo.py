"""The N > 1 path of the benchmark on CPU: two gloo ranks, each with its own seeded problem,
timings reduced with a max over ranks, whole-job rate = units of all ranks / slowest time."""
import os

import numpy as np
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2511_04063_b200 import inputs as gen
from paper_2511_04063_b200 import replicas


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = replicas.workload_for_rank(gen.scaled(gen.WORKLOADS["c2_7b"], d=64, n_tokens=128, n_outlier_channels=2), rank)
        X = gen.gen_activations(w)
        local_ms = [10.0 + 5.0 * rank, 3.0 - rank]            # rank 1 is slower on the first, faster on the second
        got = replicas.max_over_ranks(local_ms)
        np.save(os.path.join(out_dir, "x%d.npy" % rank), X)
        np.save(os.path.join(out_dir, "t%d.npy" % rank), np.array(got))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_get_distinct_problems_and_max_reduced_times(tmp_path):
    world, port = 2, 29500 + (os.getpid() % 2000)
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    x0, x1 = np.load(tmp_path / "x0.npy"), np.load(tmp_path / "x1.npy")
    assert x0.shape == x1.shape and not np.array_equal(x0, x1)      # independent rotation sites
    for r in range(world):
        assert np.allclose(np.load(tmp_path / ("t%d.npy" % r)), [15.0, 3.0])
    assert replicas.whole_job_rate(20, world, 15.0) == 2 * 20 / 0.015


def test_single_process_is_identity():
    assert replicas.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    w = gen.WORKLOADS["c1_tiny"]
    assert replicas.workload_for_rank(w, 0) == w and replicas.workload_for_rank(w, 3).seed == w.seed + 3


def test_launch_starts_every_rank_and_rank0_prints_the_reduced_line(tmp_path):
    """What `bench.py --gpus 2` does without an external launcher: replicas.launch starts the ranks
    (RANK / LOCAL_RANK / WORLD_SIZE / MASTER_* in their environment), each joins the group, and the
    line rank 0 prints carries n_gpus = 2 and the rate over the slowest rank's time."""
    import json
    import sys
    stub = os.path.join(os.path.dirname(os.path.abspath(__file__)), "replica_stub.py")
    codes, text = replicas.launch(2, [stub, str(tmp_path)], timeout=300, capture_rank0=True)
    assert codes == [0, 0]
    line = json.loads(text.strip().splitlines()[-1])
    assert line["n_gpus"] == 2 and line["scaling"] == "weak"
    assert abs(line["value"] - 2 * 20 / 0.015) < 1e-6 and abs(line["ms_per_step"] - 0.75) < 1e-12
    seen = [json.load(open(tmp_path / ("rank%d.json" % r))) for r in range(2)]
    assert [s["rank"] for s in seen] == [0, 1] and [s["local_rank"] for s in seen] == [0, 1]
    assert all(s["world"] == 2 for s in seen)
    assert seen[0]["line"]["value"] == seen[1]["line"]["value"]      # the reduction reached both ranks
    assert seen[0]["line"]["seed"] != seen[1]["line"]["seed"]        # independent rotation sites


def test_launch_reports_a_failing_rank(tmp_path):
    codes, _ = replicas.launch(2, ["-c", "import os, sys; sys.exit(3 if os.environ['RANK'] == '1' else 0)"], timeout=60)
    assert codes == [0, 3]
    assert not replicas.launched_externally() or "WORLD_SIZE" in os.environ
