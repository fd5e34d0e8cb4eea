"""Float64 CPU oracle for one rotational-distribution-calibration step.

TEST INFRASTRUCTURE ONLY.  Nothing in the product package imports this; only
the test-suite, the smoke check and the CPU-baseline leg of the benchmark do.
It shares no code with the CUDA path.
"""
from .calib_oracle import (  # noqa: F401
    whip_per_token, whip_loss, whip_grad_wrt_output, householder_qr_alg2,
    qr_pos, qr_pos_lapack, rotate, grad_wrt_rotation, qr_backward, sgd_step, momentum_step, adam_step,
    calib_step, calib_run, widen_input,
)
from .token_sampling import philox4x32_10, permute_index, gather_tokens  # noqa: F401,E402
from .eval_metrics import outlier_count, quantize_per_token_asymmetric, quantization_mse  # noqa: F401,E402
from .cayley_oracle import cayley_sgd_step, cayley_calib_step, cayley_calib_run  # noqa: F401,E402
from . import objectives  # noqa: F401,E402
from . import epochs  # noqa: F401,E402
