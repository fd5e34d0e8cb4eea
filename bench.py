#!/usr/bin/env python
"""Benchmark of the calibration hot path (one step = qr(Z) -> X R -> Whip ->
backward -> SGD) on synthetic LLM-shaped activations.

  python bench.py --gpus N --steps K --warmup W [--workload c2_7b] [--impl reference]

Prints ONE JSON line (rank 0).  `value` is calibration steps/s with inputs resident in
HBM; `e2e` is the same metric through the C ABI with host buffers (a fresh activation
batch copied host->device and the loss read back every step); `roofline` is the
forward X R + Whip tensor-core kernel against the measured bf16 peak; `cpu_baseline`
is the float64 oracle timed on this machine's host cores on a bounded sample.
With N > 1 every rank calibrates an independent rotation (replicas, no collective
on the data path): weak scaling.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "calibration steps/sec"
UNIT = "steps/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# DRAM traffic (bytes read + written) of one launch of the roofline kernel, from an ncu capture of
# that kernel on the named workload; None where no capture of the current kernel exists.
NCU_TRAFFIC_BYTES = {"c2_7b": 307.4e6}
NCU_TRAFFIC_BYTES_HEADS = {"c3_heads": 138.9e6}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        p["_source"] = "measured"
        return p
    p = dict(FALLBACK_PEAKS)
    p["_source"] = "fallback"
    return p


class ClockSampler:
    """SM clock and throttle reasons during the timed region: an NVML polling thread (2 ms period, so that a
    timed region of a few tens of milliseconds still holds several samples) beside the nvidia-smi query loop
    (whose first sample can come later than a short region lasts).  Reads only; nothing is set."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, gpu_index: int, uuid: str = None):
        self.gpu = gpu_index
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        self.nvml = None
        self.handle = None
        self.rows = []          # (sm MHz, reason bit mask) from NVML
        self.stop_flag = threading.Event()
        self.thread = None
        self.sm_max = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.handle = None
            if uuid:
                try:
                    self.handle = pynvml.nvmlDeviceGetHandleByUUID(uuid if uuid.startswith("GPU-") else "GPU-" + uuid)
                except Exception:
                    self.handle = None
            if self.handle is None:
                self.handle = pynvml.nvmlDeviceGetHandleByIndex(gpu_index)
            self.sm_max = float(pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM))
            self.nvml = pynvml
        except Exception:
            self.nvml = None

    def _poll(self):
        nv = self.nvml
        while not self.stop_flag.is_set():
            try:
                sm = nv.nvmlDeviceGetClockInfo(self.handle, nv.NVML_CLOCK_SM)
                mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.handle)
                self.rows.append((float(sm), int(mask)))
            except Exception:
                pass
            time.sleep(0.002)

    def start(self):
        if self.nvml is not None:
            self.thread = threading.Thread(target=self._poll, daemon=True)
            self.thread.start()
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.Q,
                                       "--format=csv,noheader,nounits", "-lms", "10"],
                                      stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": self.sm_max, "reasons": [], "samples": 0}
        sm, reasons = [], set()
        if self.thread is not None:
            self.stop_flag.set()
            self.thread.join(timeout=2)
            nv = self.nvml
            bits = {"hw_slowdown": nv.nvmlClocksThrottleReasonHwSlowdown,
                    "hw_thermal_slowdown": nv.nvmlClocksThrottleReasonHwThermalSlowdown,
                    "sw_thermal_slowdown": nv.nvmlClocksThrottleReasonSwThermalSlowdown,
                    "sw_power_cap": nv.nvmlClocksThrottleReasonSwPowerCap}
            for clock, mask in self.rows:
                sm.append(clock)
                for nme, bit in bits.items():
                    if mask & bit:
                        reasons.add(nme)
        if self.p is not None:
            self.p.terminate()
            try:
                self.p.wait(timeout=5)
            except Exception:
                self.p.kill()
            self.f.flush()
            rows = [l.strip().split(", ") for l in open(self.f.name) if l.strip()]
            for r in rows:
                if len(r) < 9:
                    continue
                try:
                    sm.append(float(r[1]))
                    out["sm_max_mhz"] = float(r[2])
                except ValueError:
                    continue
                for k, nme in enumerate(self.NAMES):
                    if r[5 + k].strip().lower().startswith("active"):
                        reasons.add(nme)
        try:
            os.unlink(self.f.name)
        except OSError:
            pass
        if sm:
            out["sm_mhz"] = float(np.median(sm))
        out["reasons"] = sorted(reasons)
        out["samples"] = len(sm)
        return out


def oracle_thread_count() -> int:
    try:
        from threadpoolctl import threadpool_info
        return max([i.get("num_threads", 1) for i in threadpool_info()] + [1])
    except Exception:
        return os.cpu_count() or 1


class OracleRun:
    """The float64 oracle (oracle.calib_step, as it stands) on a workload's own inputs, one problem.

    The QR of a step is the oracle's literal Algorithm 2 loop up to d = 512 and its library-QR form
    (oracle.qr_pos_lapack: the same unique factors, which the oracle's tests pin the loop to) beyond, where
    the loop's d dependent rank-one updates would take minutes per step.  A workload whose step costs more
    than `max_flops` float64 flops is sampled: a prefix of the token rows, the rate scaled by the ratio of the
    step's flop counts and the line marked as extrapolated."""

    def __init__(self, w, max_flops: float = 4e12):
        import oracle as orc
        from paper_2511_04063_b200 import inputs as gen
        self.orc, self.w = orc, w
        d, n = w.d, w.n_tokens
        cost = lambda nt: 4.0 * nt * d * d + 10.0 * d ** 3
        self.n_used = n
        while cost(self.n_used) > max_flops and self.n_used > 2048:
            self.n_used //= 2
        self.extrapolated = self.n_used != n
        self.scale = cost(self.n_used) / cost(n)          # full-size steps per sampled step
        wx = gen.scaled(w, batch=1)                       # one problem; a batch is `batch` such steps
        X = gen.activations_as_f32(wx, gen.gen_activations(wx))[0]
        self.X = X[:self.n_used].astype(np.float64)
        self.Z = gen.gen_latent_init(wx)[0].astype(np.float64)
        self.qr = orc.qr_pos if d <= 512 else orc.qr_pos_lapack
        self.cores = oracle_thread_count()

    def step(self):
        self.Z = self.orc.calib_step(self.X, self.Z, self.w.lr, qr=self.qr)["Z_new"]

    def time_steps(self, n_steps: int) -> float:
        """Seconds per full-size step of the whole batch, from n_steps oracle steps."""
        t0 = time.perf_counter()
        for _ in range(n_steps):
            self.step()
        dt = (time.perf_counter() - t0) / n_steps
        return dt * self.w.batch / self.scale

    def sample(self, n_steps: int) -> str:
        s = "oracle.calib_step(qr=%s) x%d at d=%d, N=%d" % (self.qr.__name__, n_steps, self.w.d, self.n_used)
        if self.w.batch > 1:
            s += ", one of the %d problems (time x%d)" % (self.w.batch, self.w.batch)
        if self.extrapolated:
            s += "; a prefix of the %d token rows, time scaled by the step's flop count (x%.2f)" % (
                self.w.n_tokens, 1.0 / self.scale)
        return s


def run_reference(args, w):
    """The reference arm: the oracle on the host cores, W untimed and K timed steps on the arm's workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    run = OracleRun(w)
    K, W = max(1, args.steps), max(0, args.warmup)
    if W:
        run.time_steps(W)
    sec = run.time_steps(K)
    v = 1.0 / sec
    line = {"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * sec, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "d": w.d, "n_tokens": w.n_tokens, "batch": w.batch, "lr": w.lr},
            "cpu_baseline": {"value": v, "unit": UNIT, "cores": run.cores, "kind": "oracle", "sample": run.sample(K),
                             "extrapolated": run.extrapolated},
            "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="c2_7b")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--qr", default="incremental", choices=["incremental", "householder"],
                    help="QR-Orth forward on the tensor-core path (see dq_calib_set_qr_method); the other one is "
                         "timed as well and reported beside the headline")
    args = ap.parse_args()

    from paper_2511_04063_b200 import inputs as gen
    w = gen.WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, w)
        return

    from paper_2511_04063_b200 import replicas
    if args.gpus > 1 and not replicas.launched_externally():
        # no launcher gave this process a rank: start one process per GPU on this node and let rank 0 print
        codes, _ = replicas.launch(args.gpus, [os.path.abspath(__file__)] + sys.argv[1:])
        raise SystemExit(max(abs(c) for c in codes))

    import torch
    import paper_2511_04063_b200 as dq

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the calibration path has no CPU implementation")
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    rank, local_rank, world = replicas.init_process_group("nccl")

    def barrier():
        replicas.barrier()
        torch.cuda.synchronize()

    # ---------------------------------------------------------------- inputs
    # every rank gets its own seeded problem (an independent rotation site)
    wr = replicas.workload_for_rank(w, rank)
    X_host = gen.gen_activations(wr)
    Z0_host = gen.gen_latent_init(wr)
    as_torch = (lambda a: torch.from_numpy(a)) if wr.x_dtype == "fp32" else \
        (lambda a: torch.from_numpy(a.view(np.int16)).view(torch.bfloat16))
    X_pinned = as_torch(X_host).pin_memory()
    Xd = X_pinned.cuda(non_blocking=True)
    Zd = torch.from_numpy(Z0_host).cuda()
    path = dq.DQ_PATH_FP32 if wr.path == "fp32" else dq.DQ_PATH_BF16_TC
    h = dq.dq_calib_init(Xd, Zd, lr=wr.lr, path=path)
    QR_ENUM = {"incremental": dq.DQ_QR_ITERATIVE, "householder": dq.DQ_QR_HOUSEHOLDER}
    other_qr = "householder" if args.qr == "incremental" else "incremental"
    dq.dq_calib_set_qr_method(h, QR_ENUM[args.qr], 0)
    K, W = args.steps, max(args.warmup, 3)
    loss_dev = torch.empty((max(K, W), wr.batch), dtype=torch.float32, device="cuda")

    # ---------------------------------------------------------------- device-resident timing
    dq.dq_calib_step(h, W, loss_dev)
    st = dq.dq_calib_status(h)
    assert st == dq.DQ_OK, dq.status_string(st)
    sampler = ClockSampler(local_rank, str(getattr(torch.cuda.get_device_properties(local_rank), "uuid", "") or ""))
    launches0 = dq.dq_calib_launch_count(h)
    barrier()
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    dq.dq_calib_step(h, K, loss_dev)
    e1.record()
    barrier()
    clocks = sampler.stop()
    ms = e0.elapsed_time(e1)
    launches = dq.dq_calib_launch_count(h) - launches0
    st = dq.dq_calib_status(h)
    assert st == dq.DQ_OK, dq.status_string(st)
    losses = loss_dev[:K].float().cpu().numpy()

    # ---------------------------------------------------------------- per-phase times (events inside the library)
    dq.dq_calib_set_timing(h, True)
    n_phase_steps = min(K, 5)
    flops0 = dq.dq_calib_mma_flops(h)
    dq.dq_calib_step(h, n_phase_steps, loss_dev)
    mma_flops_per_step = (dq.dq_calib_mma_flops(h) - flops0) / n_phase_steps
    phases = dq.dq_calib_get_timings(h)
    dq.dq_calib_set_timing(h, False)

    # ---------------------------------------------------------------- one QR-Orth product alone
    prod_ms = None
    if path == dq.DQ_PATH_BF16_TC and wr.d != 128:
        prod_ms = {3: dq.dq_calib_time_product(h, 3, 10), 1: dq.dq_calib_time_product(h, 1, 10)}

    # ---------------------------------------------------------------- same workload, the other QR-Orth forward
    alt = None
    if path == dq.DQ_PATH_BF16_TC and wr.d != 128:
        dq.dq_calib_set_qr_method(h, QR_ENUM[other_qr], 0)
        dq.dq_calib_step(h, W, loss_dev)
        barrier()
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a0.record()
        dq.dq_calib_step(h, K, loss_dev)
        a1.record()
        barrier()
        ms_alt = a0.elapsed_time(a1)
        dq.dq_calib_set_timing(h, True)
        dq.dq_calib_step(h, n_phase_steps, loss_dev)
        phases_alt = dq.dq_calib_get_timings(h)
        dq.dq_calib_set_timing(h, False)
        st = dq.dq_calib_status(h)
        assert st == dq.DQ_OK, dq.status_string(st)
        alt = {"ms_per_step": ms_alt / K, "phases_ms": phases_alt}
        dq.dq_calib_set_qr_method(h, QR_ENUM[args.qr], 0)

    # ---------------------------------------------------------------- same contractions, Cayley SGD (Algorithm 3)
    cay = None
    if path == dq.DQ_PATH_BF16_TC and wr.d != 128:
        dq.dq_calib_set_orth_method(h, dq.DQ_ORTH_CAYLEY, 0.9)
        dq.dq_calib_step(h, W, loss_dev)
        barrier()
        c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        c0.record()
        dq.dq_calib_step(h, K, loss_dev)
        c1.record()
        barrier()
        ms_cay = c0.elapsed_time(c1)
        dq.dq_calib_set_timing(h, True)
        dq.dq_calib_step(h, n_phase_steps, loss_dev)
        phases_cay = dq.dq_calib_get_timings(h)
        dq.dq_calib_set_timing(h, False)
        st = dq.dq_calib_status(h)
        assert st == dq.DQ_OK, dq.status_string(st)
        cay = {"ms_per_step": ms_cay / K, "update_ms": phases_cay["qr_backward"]}
        dq.dq_calib_set_orth_method(h, dq.DQ_ORTH_QR)

    # ---------------------------------------------------------------- Y = X R materialised (dq_rotate_apply)
    rot = None
    if path == dq.DQ_PATH_BF16_TC and wr.batch == 1:
        Rdev = torch.empty((wr.d, wr.d), dtype=torch.float32, device="cuda")
        dq.dq_calib_get_rotation(h, Rdev)
        Y = torch.empty((wr.n_tokens, wr.d), dtype=torch.bfloat16, device="cuda")
        for _ in range(3):
            dq.dq_rotate_apply(Xd[0], Rdev, Y)
        r0, r1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        r0.record()
        for _ in range(10):
            dq.dq_rotate_apply(Xd[0], Rdev, Y)
        r1.record()
        torch.cuda.synchronize()
        rot = r0.elapsed_time(r1) / 10
        del Y

    # ---------------------------------------------------------------- end to end (host buffers)
    loss_host = torch.empty((1, wr.batch), dtype=torch.float32).pin_memory()
    Ke = min(K, 10)
    barrier()
    t0e, t1e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    # Every step's batch travels host -> device inside the timed region.  The copy of batch i + 1 (into one of
    # two staging buffers, on a copy stream) overlaps the step on batch i; a device-to-device copy then moves the
    # staged batch into the buffer the handle borrows.  The loss of every step is read back before the next one.
    main = torch.cuda.current_stream()
    copy_stream = torch.cuda.Stream()
    stage = [torch.empty_like(Xd), torch.empty_like(Xd)]
    ready = [torch.cuda.Event(), torch.cuda.Event()]
    freed = [torch.cuda.Event(), torch.cuda.Event()]
    used = [False, False]

    def start_copy(slot):
        if used[slot]:
            copy_stream.wait_event(freed[slot])
        with torch.cuda.stream(copy_stream):
            stage[slot].copy_(X_pinned, non_blocking=True)
            ready[slot].record(copy_stream)
        used[slot] = True

    t0e.record()
    copy_stream.wait_event(t0e)
    start_copy(0)
    for i in range(Ke):
        cur = i % 2
        if i + 1 < Ke:
            start_copy((i + 1) % 2)
        main.wait_event(ready[cur])
        Xd.copy_(stage[cur], non_blocking=True)
        freed[cur].record(main)
        dq.dq_calib_refresh_inputs(h)
        dq.dq_calib_step(h, 1, loss_dev)
        loss_host.copy_(loss_dev[:1], non_blocking=True)  # the step's result, device -> host
        main.synchronize()
    t1e.record()
    barrier()
    ms_e2e = t0e.elapsed_time(t1e)
    h2d = X_pinned.numel() * X_pinned.element_size()
    d2h = loss_host.numel() * 4

    # ---------------------------------------------------------------- reduce over ranks
    ms, ms_e2e = replicas.max_over_ranks([ms, ms_e2e], device="cuda")
    value = replicas.whole_job_rate(K, world, ms)
    e2e_value = replicas.whole_job_rate(Ke, world, ms_e2e)

    if rank == 0:
        peaks = load_peaks()
        d, N, B = wr.d, wr.n_tokens, wr.batch
        fwd_flops = 2.0 * N * d * d * B
        t_fwd = phases["rotate_whip"] * 1e-3
        t_bwd = phases["grad_rotation"] * 1e-3
        achieved = fwd_flops / t_fwd / 1e12 if t_fwd > 0 else 0.0
        # the phase timer brackets each phase of single steps with events and synchronises after every step, i.e.
        # it times the kernel alone: the burst peak is the denominator (the sustained one is reported beside it;
        # `clocks` describes the long timed region of `value`, where the power cap may be active)
        capped = False
        peak = peaks["bf16_tflops"]
        gemm_tflops = 2 * fwd_flops / (t_fwd + t_bwd) / 1e12 if (t_fwd + t_bwd) > 0 else 0.0
        total_phase = sum(phases.values())
        roofline = {"bound": "tensor", "kernel": ("tc_gemm2_kernel<WHIP>" if d % 256 == 0 else "tc_gemm_kernel<256,1,WHIP>") + " (O^T = R^T X^T, Eq. 4 epilogue)"
                    if path == dq.DQ_PATH_BF16_TC else "gemm_ffma_kernel<WHIP>",
                    "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                    "peak_source": "%s (%s bf16 matmul peak)" % (peaks["_source"], "sustained" if capped else "burst"),
                    "frac_of_sustained_peak": achieved / peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]),
                    "frac_of_nominal_2250": achieved / 2250.0,
                    "traffic": NCU_TRAFFIC_BYTES.get(wr.name),
                    "algorithmic_flops_per_launch": fwd_flops}
        if path == dq.DQ_PATH_BF16_TC and d == 128 and t_fwd > 0:
            # per-head rotations: both contractions and the Eq. 4 epilogue are one kernel that reads the activations
            # once and keeps everything else on chip: 128 flop per byte, below the ridge of this GPU: HBM roofline
            hb = 2.0 * N * d * B
            roofline = {"bound": "hbm", "kernel": "heads_whip_kernel (O = X R_h, Eq. 4, Gq_h = X^T dL/dO fused)",
                        "achieved": hb / t_fwd / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                        "frac": hb / t_fwd / 1e9 / peaks["hbm_gbs"],
                        "peak_source": "%s (copy bandwidth)" % peaks["_source"],
                        "traffic": NCU_TRAFFIC_BYTES_HEADS.get(wr.name),
                        "algorithmic_bytes_per_launch": hb}
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
                "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": "bf16" if path == dq.DQ_PATH_BF16_TC else "f32", "data": "synthetic",
                "config": {"workload": wr.name, "d": d, "n_tokens": N, "batch": B, "lr": wr.lr,
                           "parallelism": "replicas x%d" % world, "qr": args.qr,
                           "l2": "inputs (%.0f MiB X + G) exceed the 126 MB L2" % (2 * h2d / 2 ** 20)},
                "clocks": {"sm_mhz": clocks["sm_mhz"], "sm_max_mhz": clocks["sm_max_mhz"],
                           "reasons": clocks["reasons"], "samples": clocks["samples"]},
                "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                        "steps": Ke},
                "gpu_launches": int(launches),
                "roofline": roofline,
                "phases_ms": phases,
                "gemm_tflops": gemm_tflops,
                "gemm_frac_of_measured_burst": gemm_tflops / peaks["bf16_tflops"],
                "gemm_frac_of_nominal_2250": gemm_tflops / 2250.0,
                "qr_orth_share": (phases["qr_forward"] + phases["qr_backward"]) / total_phase if total_phase else None,
                "loss_first_last": [float(losses[0].mean()), float(losses[-1].mean())]}
        # the optimiser update is the HBM-bound kernel of the path: 12 bytes per latent entry (SGD: read Z and
        # dL/dZ, write Z) plus 4 on the tensor-core path (the split-bf16 copy of the new latent for the next QR)
        upd_bytes = (16.0 if path == dq.DQ_PATH_BF16_TC else 12.0) * d * d * B
        if phases["update"] > 0 and d != 128:      # for d = 128 the update is fused into the backward kernel
            gbs = upd_bytes / (phases["update"] * 1e-3) / 1e9
            line["update_hbm"] = {"kernel": "sgd_kernel", "bytes_per_launch": upd_bytes, "achieved_gbs": gbs,
                                  "peak_gbs": peaks["hbm_gbs"], "frac": gbs / peaks["hbm_gbs"],
                                  "note": "event-timed phase (includes launch latency; meaningful for d >= 2048)"}
        if alt is not None:
            # same metric with the other dq_calib_set_qr_method: blocked Householder at every step (no
            # assumption on the step size) against the incremental factorisation (triangular tensor-core GEMMs)
            ta = sum(alt["phases_ms"].values())
            line["qr_" + other_qr] = {"value": world * 1e3 / alt["ms_per_step"], "unit": UNIT,
                                    "ms_per_step": alt["ms_per_step"], "phases_ms": alt["phases_ms"],
                                    "qr_orth_share": (alt["phases_ms"]["qr_forward"] + alt["phases_ms"]["qr_backward"]) / ta}
        if path == dq.DQ_PATH_BF16_TC and d != 128:
            # issued bf16 MMA flops (counted by the library at launch: three products per split-bf16 term, k clipped
            # to the non-zero blocks of triangular operands) over the event-timed phases that issue them
            qr_flops = mma_flops_per_step - 2 * fwd_flops
            t_qr = (phases["qr_forward"] + phases["qr_backward"]) * 1e-3
            t_all = t_qr + (phases["rotate_whip"] + phases["grad_rotation"]) * 1e-3
            line["mma_issued"] = {"flops_per_step": mma_flops_per_step,
                                  "step_tflops": mma_flops_per_step / t_all / 1e12,
                                  "qr_orth_flops_per_step": qr_flops,
                                  "qr_orth_tflops": qr_flops / t_qr / 1e12 if t_qr > 0 else None,
                                  "qr_orth_frac_of_measured_burst": qr_flops / t_qr / 1e12 / peaks["bf16_tflops"],
                                  "note": "QR-Orth phases also hold their HBM-bound element-wise kernels"}
        if prod_ms is not None:
            # The kernel family QR-Orth spends its time in, timed alone: one dense d^3 product on split-bf16
            # operands (three bf16 MMAs per product term: 6 d^3 issued MMA flops for 2 d^3 algorithmic ones) and on
            # plain bf16 operands, against the measured burst bf16 peak; and the share of the step's event-timed
            # phases that each family of kernels takes.
            issued3, issued1 = 6.0 * d ** 3 * B, 2.0 * d ** 3 * B
            line["roofline_qr_orth"] = {
                "bound": "tensor", "kernel": "tc_gemm2_kernel<3,GEN> / <1,GEN> (d x d products of QR-Orth)",
                "achieved": issued3 / (prod_ms[3] * 1e-3) / 1e12, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                "frac": issued3 / (prod_ms[3] * 1e-3) / 1e12 / peaks["bf16_tflops"],
                "peak_source": "%s (burst bf16 matmul peak)" % peaks["_source"],
                "ms_per_launch": prod_ms[3], "issued_flops_per_launch": issued3,
                "algorithmic_flops_per_launch": 2.0 * d ** 3 * B,
                "algorithmic_tflops": 2.0 * d ** 3 * B / (prod_ms[3] * 1e-3) / 1e12,
                "plain_bf16": {"ms_per_launch": prod_ms[1], "achieved": issued1 / (prod_ms[1] * 1e-3) / 1e12,
                               "frac": issued1 / (prod_ms[1] * 1e-3) / 1e12 / peaks["bf16_tflops"]},
                "traffic": None}
            line["phase_share"] = {k: v / total_phase for k, v in phases.items()} if total_phase else None
        if rot is not None:
            # includes the fp32 -> bf16 transpose of R (d^2 entries) in front of the contraction
            line["rotate_apply"] = {"ms": rot, "tflops": 2.0 * N * d * d / (rot * 1e-3) / 1e12,
                                    "hbm_bytes": 4.0 * N * d + 6.0 * d * d}
        if cay is not None:
            # Table 4's comparison on this GPU: the same loss and dL/dR, rotation updated by Cayley SGD with
            # momentum (six d x d split-bf16 products, 12 d^3 flops, three bf16 MMAs per product)
            line["cayley_sgd"] = {"value": world * 1e3 / cay["ms_per_step"], "unit": UNIT,
                                  "ms_per_step": cay["ms_per_step"], "update_ms": cay["update_ms"],
                                  "update_mma_tflops": 3 * 12.0 * d ** 3 * B / (cay["update_ms"] * 1e-3) / 1e12
                                  if cay["update_ms"] > 0 else None}
        if not args.no_cpu_baseline and world == 1:
            run = OracleRun(w, max_flops=2.5e12)          # a bounded leg: about 10-30 s of host time
            n_cpu = 3
            sec = run.time_steps(n_cpu)
            line["cpu_baseline"] = {"value": 1.0 / sec, "unit": UNIT, "cores": run.cores, "kind": "oracle",
                                    "sample": run.sample(n_cpu), "extrapolated": run.extrapolated}
        print(json.dumps(line), flush=True)
    dq.dq_calib_destroy(h)
    replicas.shutdown()


if __name__ == "__main__":
    main()
