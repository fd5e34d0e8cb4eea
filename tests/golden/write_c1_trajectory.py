"""Writes tests/golden/c1_tiny_trajectory.json from the float64 oracle alone:
the loss of each of the 20 steps of the tiny workload (d=256, N=2048, lr 1e-2,
seed 0; Algorithm 1 with the Whip loss of Eq. 4) and summary statistics of the
final rotation.  Run from the repository root:  python tests/golden/write_c1_trajectory.py
"""
import json
import os
import sys

import numpy as np

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__)))))
import oracle as orc  # noqa: E402
from paper_2511_04063_b200 import inputs as gen  # noqa: E402

w = gen.WORKLOADS["c1_tiny"]
X = gen.gen_activations(w)[0]
Z0 = gen.gen_latent_init(w)[0]
losses, Z, R = orc.calib_run(X, Z0, w.lr, w.steps)
out = {
    "source": "oracle.calib_run on workload c1_tiny (Algorithm 1; Eq. 4; Algorithm 2)",
    "losses": [float(v) for v in losses],
    "R_final_trace": float(np.trace(R)),
    "R_final_abs_sum": float(np.abs(R).sum()),
    "Z_final_fro": float(np.linalg.norm(Z)),
}
path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "c1_tiny_trajectory.json")
with open(path, "w") as f:
    json.dump(out, f, indent=1)
print("wrote", path, losses[0], losses[-1])
