#!/usr/bin/env python
"""Benchmark of the SASQ hot path on B200.

One step = one pass of the whole hot path over one batch of synthetic input with
the shapes of one LLaMA-2-7B decoder layer at T = 2048 bf16 tokens:
  phase A (training mode)  fused fake-quant forward + STE backward with the
                           scale-gradient reduction of the seven linear inputs,
                           one multi-tensor call -> seven scale gradients;
  phase B (inference mode) static W8A8 linear of the same seven linears with the
                           fixed factors, int8 per-channel weights, bf16 output.
`value` is phase A's HBM GB/s (8 algorithmic bytes per element over phase A's
device time); `w8a8_linear.value` is phase B's INT8 TOPS (2*T*N*K over phase B's
device time).  Both phases are timed with CUDA events on the launching stream
inside the same K steps.

Launch:  python bench.py --gpus N --steps K --warmup W            (N = 1)
         python -m torch.distributed.run --nproc-per-node N ... bench.py --gpus N ...   (N > 1: one replica of
         the workload per rank, no data-path collective; value is the sum over ranks over the slowest rank's time)
         python bench.py --impl reference ...   times the CPU oracle on bounded samples of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import sasq_workloads as W  # noqa: E402

METRIC = "SASQ quantizer fwd+bwd HBM GB/s; static W8A8 linear INT8 TOPS (% of peak)"
WORKLOAD = "llama2_7b_decoder_layer_7_linear_inputs_T2048_bf16"
T_TOKENS = 2048
BITS = 8
CONFIG_ID = 2
L2_BYTES = 126 * 1024 * 1024
INT8_OVER_BF16_NOMINAL = 2.0          # dense INT8 peak is twice the dense bf16 peak (4.5 vs 2.25 P-op/s nominal)
# DRAM bytes (read + write) per launch from the ncu captures summarised under profiles/ (T = 2048 workload only;
# set to None whenever the kernel changes after its capture)
NCU_TRAFFIC_FAKEQUANT = 532.0e6        # profiles/fakequant_kernel_llama7b_layer_T2048.md
NCU_TRAFFIC_GEMM = 671.0e6              # DRAM bytes of the step's one GEMM launch (profiles/w8a8_gemm_pair_kernel_T2048.md)
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return d, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def quantizer_bytes():
    """Algorithmic bytes of phase A: read x, g; write y, dx: 4 x 2 bytes per element."""
    return 8 * sum(T_TOKENS * K for _, K, _ in W.LLAMA2_7B_LINEARS)


def linear_ops():
    """Integer operations of phase B: 2 * T * N * K per linear."""
    return 2 * sum(T_TOKENS * K * N for _, K, N in W.LLAMA2_7B_LINEARS)


# ---------------------------------------------------------------------------
# clocks during the timed region (NVML, read-only)
# ---------------------------------------------------------------------------
class ClockSampler:
    PERIOD_S = 0.005

    REASONS = {
        0x0000000000000004: "sw_power_cap",
        0x0000000000000008: "hw_slowdown",
        0x0000000000000020: "sw_thermal_slowdown",
        0x0000000000000040: "hw_thermal_slowdown",
        0x0000000000000080: "hw_power_brake_slowdown",
    }

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._nv = None

    def _run(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(self.PERIOD_S)

    def start(self):
        if self._nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
        return {"sm_mhz": (statistics.median(self.samples) if self.samples else None), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def physical_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


# ---------------------------------------------------------------------------
# the workload on the device
# ---------------------------------------------------------------------------
class Layer:
    def __init__(self, P, device, rank: int, linear_calls: str = "layer"):
        self.P = P
        dt = torch.bfloat16
        self.x, self.g, self.y, self.dx, self.w_int, self.w_scale, self.out = [], [], [], [], [], [], []
        scales = torch.empty(7, dtype=torch.float32, device=device)
        cal_ws = torch.empty(P.sasq_absmax_scale_workspace(0), dtype=torch.uint8, device=device)
        for i, (_, K, N) in enumerate(W.LLAMA2_7B_LINEARS):
            seed = W.seed_of(CONFIG_ID, i) + 100_000 * rank
            x = W.activations(T_TOKENS, K, dt, seed, W.NORMAL_OUTLIERS, device=device)
            self.x.append(x)
            self.g.append(W.upstream_grad(T_TOKENS, K, dt, seed, device=device))
            self.y.append(torch.empty_like(x))
            self.dx.append(torch.empty_like(x))
            # initial factor: Eq. 1 on a 64-token calibration slice (library kernel, set-up only)
            P.sasq_absmax_scale(x[:W.CALIBRATION_TOKENS], scales[i:i + 1], cal_ws, BITS)
            w = W.weights_fp32(N, K, seed + 50, device=device)
            w_int = torch.empty((N, K), dtype=torch.int8, device=device)
            w_scale = torch.empty(N, dtype=torch.float32, device=device)
            P.sasq_quantize_weight(w, w_int, w_scale, 8)
            del w
            self.w_int.append(w_int)
            self.w_scale.append(w_scale)
            self.out.append(torch.empty((T_TOKENS, N), dtype=dt, device=device))
        self.scales = scales
        self.grads = torch.zeros(7, dtype=torch.float32, device=device)
        self.q_ws = torch.empty(P.sasq_fakequant_multi_workspace(7), dtype=torch.uint8, device=device)
        self.shapes = [(T_TOKENS, N, K) for _, K, N in W.LLAMA2_7B_LINEARS]
        self.l_ws = torch.empty(P.sasq_static_w8a8_linear_multi_workspace(self.shapes), dtype=torch.uint8,
                                device=device)
        self.linears = [(self.x[i], self.w_int[i], self.w_scale[i], self.scales[i:i + 1], self.out[i])
                        for i in range(7)]
        # descriptor tables marshalled once: the step submits the same buffers every time
        self.calls = [(P.LinearProblems([self.linears[i] for i in call]),
                       P.sasq_static_w8a8_linear_multi_launches([self.shapes[i] for i in call]))
                      for call in LINEAR_CALLS[linear_calls]]
        self.descs = P.QuantTensors([(self.x[i], self.g[i], self.y[i], self.dx[i], i) for i in range(7)])
        torch.cuda.synchronize()
        assert P.sasq_device_status() == 0

    # kernels launched per step: one fused quantizer launch (the reduction's second stage runs in its last block),
    # then the linears (activation quantizer inside the GEMM kernel): the seven problems of the step are independent
    # and resident, so by default they are submitted in one call, which runs them in one launch while their int8
    # codes fit L2; the other groupings are there for comparison
    def phase_a(self):
        self.P.sasq_fakequant_fwd_bwd_multi(self.descs, self.scales, self.grads, self.q_ws, BITS)
        return 1

    def phase_b(self):
        n = 0
        for problems, launches in self.calls:
            self.P.sasq_static_w8a8_linear_multi(problems, self.l_ws, bits=BITS)
            n += launches
        return n


# how phase B submits the seven linears: all in one call; the groups a decoder layer's data flow allows
# (q/k/v, o, gate/up, down); or one call per linear
LINEAR_CALLS = {"layer": [[0, 1, 2, 3, 4, 5, 6]], "dependent": [[0, 1, 2], [3], [4, 5], [6]],
                "each": [[i] for i in range(7)]}


def max_over_ranks(values, dist, device):
    """Element-wise maximum of per-rank timings (the slowest rank decides); identity without a process group."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.tolist()]


def throughput(world: int, units_per_rank: float, steps: int, ms: float) -> float:
    """Whole-job rate: the units all ranks processed over the slowest rank's time (weak scaling, replicas)."""
    return world * units_per_rank * steps / (ms * 1e-3)


def run_ours(args):
    import paper_2512_14481_b200 as P          # raises if the CUDA library has not been built: no fallback

    P.load_library()
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (sm_100a); there is no CPU path")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)

    layer = Layer(P, device, rank, args.linear_calls)
    stream = torch.cuda.current_stream()

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        layer.phase_a()
        layer.phase_b()
    barrier()

    K = args.steps
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(K)]
    sampler = ClockSampler(physical_gpu_index(local_rank))
    launches = 0
    sampler.start()
    barrier()
    t_wall = time.perf_counter()
    for k in range(K):
        ev[k][0].record(stream)
        launches += layer.phase_a()
        ev[k][1].record(stream)
        launches += layer.phase_b()
        ev[k][2].record(stream)
    barrier()
    t_wall = time.perf_counter() - t_wall
    clocks = sampler.stop()
    assert P.sasq_device_status() == 0

    ms_a = sum(ev[k][0].elapsed_time(ev[k][1]) for k in range(K))
    ms_b = sum(ev[k][1].elapsed_time(ev[k][2]) for k in range(K))
    ms_total = ev[0][0].elapsed_time(ev[K - 1][2])
    ms_a, ms_b, ms_total = max_over_ranks([ms_a, ms_b, ms_total], dist, device)

    # ---------------- phase B in the other ways of submitting the seven linears (context, outside the timed region) ----
    groupings = {}
    if world == 1:
        for name in LINEAR_CALLS:
            calls = [P.LinearProblems([layer.linears[i] for i in call]) for call in LINEAR_CALLS[name]]
            for _ in range(3):
                for problems in calls:
                    P.sasq_static_w8a8_linear_multi(problems, layer.l_ws, bits=BITS)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            reps = max(3, min(K, 20))
            torch.cuda.synchronize()
            e0.record(stream)
            for _ in range(reps):
                for problems in calls:
                    P.sasq_static_w8a8_linear_multi(problems, layer.l_ws, bits=BITS)
            e1.record(stream)
            torch.cuda.synchronize()
            groupings[name] = round(linear_ops() * reps / (e0.elapsed_time(e1) * 1e-3) / 1e12, 2)

    # ---------------- end to end through the public API with HOST buffers ----------------
    e2e = measure_e2e(P, layer, device, dist, steps=max(2, min(K, 5)))

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return
    peaks, peak_kind = measured_peaks()
    qbytes, lops = quantizer_bytes(), linear_ops()
    gbs = throughput(world, qbytes, K, ms_a) / 1e9
    tops = throughput(world, lops, K, ms_b) / 1e12
    int8_peak = peaks["bf16_tflops_sustained"] * INT8_OVER_BF16_NOMINAL
    ach_q = qbytes * K / (ms_a * 1e-3) / 1e9            # per GPU
    ach_l = lops * K / (ms_b * 1e-3) / 1e12
    line = {
        "metric": METRIC, "value": round(gbs, 2), "unit": "GB/s", "n_gpus": world, "steps": K,
        "warmup": max(args.warmup, 3), "ms_per_step": round(ms_total / K, 5), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16 storage, fp32 quantizer arithmetic, int8 x int8 -> int32 GEMM",
        "data": "synthetic",
        "config": {"workload": WORKLOAD, "tokens": T_TOKENS, "bits": BITS, "tensors": 7,
                   "phases": "A: fused fake-quant fwd+bwd + scale-gradient reduction; B: 7 static W8A8 linears",
                   "linear_calls": args.linear_calls,
                   "l2": f"inputs larger than L2 ({qbytes / 1e6:.0f} MB streamed in phase A, "
                         f"{(202.4e6 + 2 * qbytes / 8) / 1e6:.0f} MB of weights+activations in phase B)",
                   "parallelism": "replicas" if world > 1 else "single"},
        "ms_phase_a": round(ms_a / K, 5), "ms_phase_b": round(ms_b / K, 5),
        "w8a8_linear": {"value": round(tops, 2), "unit": "TOPS", "ops_per_step": lops,
                        "frac_of_nominal_int8_4500": round(tops / world / 4500.0, 4),
                        # phase B alone, back to back, for each way of submitting the seven linears
                        "tops_by_linear_calls": groupings},
        "roofline": {"kernel": "w8a8_gemm_pair_kernel (tcgen05 int8, CTA pairs, activation quantizer inside)",
                     "bound": "tensor", "achieved": round(ach_l, 2),
                     "peak": round(int8_peak, 1), "unit": "TOP/s", "frac": round(ach_l / int8_peak, 4),
                     "traffic": (NCU_TRAFFIC_GEMM if T_TOKENS == 2048 and args.linear_calls == "layer" else None),
                     "traffic_note": "DRAM bytes of the launch that runs the step's seven linears",
                     "peak_source": f"{peak_kind} sustained bf16 cuBLAS x 2 (nominal int8:bf16 ratio)"},
        "roofline_quantizer": {"kernel": "fakequant_kernel (fused fwd+bwd)", "bound": "hbm", "achieved": round(ach_q, 1),
                               "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": round(ach_q / peaks["hbm_gbs"], 4),
                               "frac_of_nominal_8000": round(ach_q / 8000.0, 4),
                               "traffic": (NCU_TRAFFIC_FAKEQUANT if T_TOKENS == 2048 else None),
                               "peak_source": f"{peak_kind} copy bandwidth"},
        "e2e": e2e, "gpu_launches": launches, "clocks": clocks, "wall_s": round(t_wall, 3),
    }
    line["cpu_baseline"] = cpu_baseline()
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def measure_e2e(P, layer, device, dist, steps: int):
    """Same step, but each step copies x and g of all seven tensors from pinned host memory, and reads the seven
    scale gradients and the layer's last output (down_proj) back to the host."""
    hx = [t.cpu().pin_memory() for t in layer.x]
    hg = [t.cpu().pin_memory() for t in layer.g]
    h_grads = torch.empty(7, dtype=torch.float32).pin_memory()
    h_out = torch.empty(layer.out[6].shape, dtype=layer.out[6].dtype).pin_memory()
    h2d = sum(t.numel() * t.element_size() for t in hx + hg)
    d2h = h_grads.numel() * 4 + h_out.numel() * h_out.element_size()
    stream = torch.cuda.current_stream()

    def step():
        for i in range(7):
            layer.x[i].copy_(hx[i], non_blocking=True)
            layer.g[i].copy_(hg[i], non_blocking=True)
        layer.phase_a()
        layer.phase_b()
        h_grads.copy_(layer.grads, non_blocking=True)
        h_out.copy_(layer.out[6], non_blocking=True)

    step()
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(steps):
        step()
    e1.record(stream)
    torch.cuda.synchronize()
    world = 1 if dist is None else dist.get_world_size()
    ms = max_over_ranks([e0.elapsed_time(e1)], dist, device)[0] / steps
    return {"value": round(world * quantizer_bytes() / (ms * 1e-3) / 1e9, 2), "unit": "GB/s",
            "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": round(ms, 4), "steps": steps,
            "w8a8_tops": round(world * linear_ops() / (ms * 1e-3) / 1e12, 3)}


# ---------------------------------------------------------------------------
# CPU oracle legs
# ---------------------------------------------------------------------------
def _oracle_sample(gemm_rows: int):
    """Times the oracle, as it stands, on a bounded sample of the step: the quantizer forward and backward on
    all seven full tensors, and the integer GEMM + dequant on `gemm_rows` rows of each of the seven linears."""
    import numpy as np
    import oracle

    t_q = 0.0
    t_l = 0.0
    ops = 0
    for i, (_, K, N) in enumerate(W.LLAMA2_7B_LINEARS):
        seed = W.seed_of(CONFIG_ID, i)
        xb, tag = oracle.bits_of(W.activations(T_TOKENS, K, torch.bfloat16, seed))
        gb, _ = oracle.bits_of(W.upstream_grad(T_TOKENS, K, torch.bfloat16, seed))
        s = float(oracle.absmax_scale(xb[:W.CALIBRATION_TOKENS], tag, BITS))
        t0 = time.perf_counter()
        oracle.fakequant_fwd(xb, tag, s, BITS, want_codes=False)
        oracle.fakequant_bwd(xb, gb, tag, s, BITS)
        t_q += time.perf_counter() - t0
        rng = np.random.default_rng(seed)
        w_int = rng.integers(-127, 128, size=(N, K), dtype=np.int64).astype(np.int8)
        w_scale = np.full(N, 1e-3, np.float32)
        t0 = time.perf_counter()
        oracle.w8a8_linear(xb, tag, w_int, w_scale, s, BITS, row_begin=0, row_end=gemm_rows)
        t_l += time.perf_counter() - t0
        ops += 2 * gemm_rows * K * N
    return t_q, t_l, ops


def cpu_baseline(budget_seconds: float = 25.0):
    import oracle
    # the whole step if the oracle can do it within the budget on this host, otherwise as many GEMM rows as fit
    # (sized from a 64-row probe); the quantizer part always runs on the full tensors
    _, t_probe, _ = _oracle_sample(min(64, T_TOKENS))
    gemm_rows = T_TOKENS if t_probe * max(1.0, T_TOKENS / 64) <= budget_seconds else \
        int(max(64, 64 * budget_seconds / max(t_probe, 1e-3)))
    if gemm_rows >= 8:
        gemm_rows -= gemm_rows % 8
    t_q, t_l, ops = _oracle_sample(gemm_rows)
    # the oracle runs forward and backward as two passes: 4 + 6 algorithmic bytes per element;
    # the reported GB/s uses the step's 8 bytes per element so that it is the same metric
    return {"value": round(quantizer_bytes() / t_q / 1e9, 3), "unit": "GB/s", "cores": oracle.num_threads(),
            "kind": "oracle",
            "sample": f"quantizer fwd+bwd on all 7 full tensors (T={T_TOKENS}); int GEMM+dequant on the first "
                      f"{gemm_rows} rows of each of the 7 linears",
            "w8a8_tops": round(ops / t_l / 1e12, 5), "seconds": round(t_q + t_l, 2)}


def run_reference(args):
    """Reference arm: the CPU oracle, as it stands, on the machine's host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    K = max(1, args.steps)
    rows = min(32, T_TOKENS)
    for _ in range(min(args.warmup, 1)):
        _oracle_sample(rows)
    t_q = t_l = 0.0
    ops = 0
    t_all = time.perf_counter()
    done = 0
    for _ in range(K):
        a, b, c = _oracle_sample(rows)
        t_q += a
        t_l += b
        ops += c
        done += 1
        if time.perf_counter() - t_all > 150:      # keep the whole run within a few minutes
            break
    gbs = quantizer_bytes() * done / t_q / 1e9
    sample = (f"per step: quantizer fwd+bwd on all 7 full tensors (T={T_TOKENS}); int GEMM+dequant on the first {rows} "
              f"rows of each of the 7 linears; {done} of {K} requested steps timed")
    line = {
        "impl": "reference", "metric": METRIC, "value": round(gbs, 3), "unit": "GB/s",
        "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": done, "warmup": min(args.warmup, 1),
        "ms_per_step": round((t_q + t_l) / done * 1e3, 3), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "fp32 quantizer arithmetic with double accumulation; int32 GEMM", "data": "synthetic",
        "config": {"workload": WORKLOAD, "tokens": T_TOKENS, "bits": BITS, "tensors": 7},
        "w8a8_linear": {"value": round(ops / t_l / 1e12, 5), "unit": "TOPS"},
        "cpu_baseline": {"value": round(gbs, 3), "unit": "GB/s", "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": round(gbs, 3), "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--linear-calls", choices=["layer", "dependent", "each"], default="layer",
                    help="phase B submits the seven linears in one call, in the groups a decoder layer's data flow "
                         "allows (q/k/v | o | gate/up | down), or one call per linear")
    ap.add_argument("--tokens", type=int, default=2048,
                    help="tokens per step (default 2048, the headline workload; other values time the same layer at "
                         "decode or longer-prefill sizes and are named as such in config.workload)")
    args = ap.parse_args()
    global T_TOKENS, WORKLOAD
    if args.tokens != T_TOKENS:
        if args.tokens < 1:
            ap.error("--tokens must be positive")
        T_TOKENS = args.tokens
        WORKLOAD = f"llama2_7b_decoder_layer_7_linear_inputs_T{T_TOKENS}_bf16"
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
