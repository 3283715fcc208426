#!/usr/bin/env python
"""Benchmark of the SASQ hot path on B200.

Default workload: the full 32-layer LLaMA-2-7B-shaped stack of 224 quantizers (7 per layer) over 8 x 2048 = 16 384
bf16 tokens.  One step = one pass of the whole hot path over that batch:
  phase A (training mode)  one scale-only training step: for every layer, the fused fake-quant forward + STE
                           backward with the scale-gradient reduction of its seven linear inputs (one multi-tensor
                           launch per layer -> 224 scale gradients);
  phase B (inference mode) static W8A8 prefill of all 224 linears with the fixed factors, frozen int8 per-channel
                           weights, bf16 output, submitted layer by layer in the groups a decoder layer's data flow
                           allows (q/k/v | o | gate/up | down).
The activation buffers are reused layer by layer; every layer has its own weights and factors.
`value` is phase A's HBM GB/s (8 algorithmic bytes per element over phase A's device time); `w8a8_linear.value` is
phase B's INT8 TOPS (2*T*N*K over phase B's device time).  Both phases are timed with CUDA events on the launching
stream inside the same K steps.  After the timed region the same run measures, for context: the forward-only and
backward-only quantizer, one layer at the other token counts (decode through prefill, each way of submitting the
seven linears), and two same-box yard-sticks for the tensor peak (a library INT8 GEMM and the issue rate of the
GEMM's own tensor-core instruction).

Launch:  python bench.py --gpus N --steps K --warmup W            (N = 1)
         python -m torch.distributed.run --nproc-per-node N ... bench.py --gpus N ...   (N > 1: one replica of
         the workload per rank, no data-path collective; value is the sum over ranks over the slowest rank's time)
         python bench.py --impl reference ...   times the CPU oracle on bounded samples of the same workload.
         python bench.py --layers 1 --tokens 2048 --no-extras ...   one layer at another token count (profiles).
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
BITS = 8
CONFIG_ID = 5
L2_BYTES = 126 * 1024 * 1024
INT8_OVER_BF16_NOMINAL = 2.0          # dense INT8 peak is twice the dense bf16 peak (4.5 vs 2.25 P-op/s nominal)
NOMINAL_INT8_TOPS = 4500.0
NOMINAL_HBM_GBS = 8000.0
BURST_REGION_S = 0.05                 # a timed region shorter than this is compared with the burst tensor peak,
SUSTAINED_REGION_S = 1.0              # one longer than this with the sustained one; in between, with the burst one
CPU_SAMPLE_TOKENS = 2048              # the oracle legs run on the first tokens of layer 0
# DRAM bytes (read + write) per launch, from ncu captures of these kernels (dram__bytes_read.sum + dram__bytes_write.sum);
# None whenever the kernel has changed since its capture.  Keyed by (kernel, tokens): traffic grows with the tokens.
NCU_TRAFFIC = {
    ("fakequant", 2048): 531.6e6,
    ("gemm_layer", 2048): 672.0e6,         # the seven linears of a layer in one launch (522 MB algorithmic)
    ("fakequant", 16384): 4617.0e6,
    ("gemm_q_proj", 16384): 351.0e6,       # one q_proj launch, 16384 x 4096 x 4096 (285 MB algorithmic)
}
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}

# how phase B submits the seven linears of a layer: all in one call; the groups a decoder layer's data flow allows
# (q/k/v, o, gate/up, down); or one call per linear
LINEAR_CALLS = {"layer": [[0, 1, 2, 3, 4, 5, 6]], "dependent": [[0, 1, 2], [3], [4, 5], [6]],
                "each": [[i] for i in range(7)]}
LINEARS = W.LLAMA2_7B_LINEARS
CONFIG3_TOKENS = (1, 16, 128, 2048, 8192)


def workload_name(layers: int, tokens: int) -> str:
    return (f"llama2_7b_{layers}_layers_x7_quantizers_T{tokens}_bf16_scale_only_step_then_static_w8a8_prefill"
            if layers > 1 else f"llama2_7b_decoder_layer_7_linear_inputs_T{tokens}_bf16")


def config_of(args) -> dict:
    """The `config` object, the same for both arms."""
    T, L = args.tokens, args.layers
    world = int(os.environ.get("WORLD_SIZE", "1"))
    return {"workload": workload_name(L, T), "layers": L, "tokens": T,
            "bits": BITS, "quantizers": 7 * L,
            "phases": "A: fused fake-quant fwd+bwd + scale-gradient reduction, one launch per layer; "
                      "B: static W8A8 linears of every layer",
            "linear_calls": args.linear_calls,
            "l2": f"inputs larger than L2: {quantizer_bytes(T) / 1e6:.0f} MB streamed per layer in phase A, "
                  f"{(weight_bytes() + 2 * quantizer_elements(T)) / 1e6:.0f} MB of weights+activations per "
                  f"layer in phase B, {L} layers with their own weights",
            "parallelism": "replicas" if world > 1 else "single"}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return d, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def quantizer_elements(tokens: int) -> int:
    return sum(tokens * K for _, K, _ in LINEARS)


def quantizer_bytes(tokens: int, layers: int = 1) -> int:
    """Algorithmic bytes of phase A: read x, g; write y, dx: 4 x 2 bytes per element."""
    return 8 * quantizer_elements(tokens) * layers


def linear_ops(tokens: int, layers: int = 1) -> int:
    """Integer operations of phase B: 2 * T * N * K per linear."""
    return 2 * sum(tokens * K * N for _, K, N in LINEARS) * layers


def weight_bytes() -> int:
    return sum(K * N for _, K, N in LINEARS)


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
                "sm_mhz_min": (min(self.samples) if self.samples else None),
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
class Stack:
    """`layers` decoder layers' worth of quantizers and frozen linears over `tokens` tokens.  The activation,
    gradient and output buffers are shared by the layers; weights, factors and gradient slots are per layer."""

    def __init__(self, P, device, rank: int, layers: int, tokens: int, training: bool = True):
        self.P, self.layers, self.tokens = P, layers, tokens
        self.stream = torch.cuda.current_stream().cuda_stream      # raw handle: the cheapest thing to pass per call
        dt = torch.bfloat16
        self.x, self.g, self.y, self.dx, self.out = [], [], [], [], []
        self.w_int = [[None] * 7 for _ in range(layers)]
        self.w_scale = [[None] * 7 for _ in range(layers)]
        self.scales = torch.empty((layers, 7), dtype=torch.float32, device=device)
        self.grads = torch.zeros((layers, 7), dtype=torch.float32, device=device)
        cal_ws = torch.empty(P.sasq_absmax_scale_workspace(0), dtype=torch.uint8, device=device)
        for i, (_, K, N) in enumerate(LINEARS):
            seed = W.seed_of(CONFIG_ID, i) + 100_000 * rank
            x = W.activations(tokens, K, dt, seed, W.NORMAL_OUTLIERS, device=device)
            self.x.append(x)
            if training:
                self.g.append(W.upstream_grad(tokens, K, dt, seed, device=device))
                self.y.append(torch.empty_like(x))
                self.dx.append(torch.empty_like(x))
            # initial factor: Eq. 1 on a 64-token calibration slice (library kernel, set-up only)
            P.sasq_absmax_scale(x[:W.CALIBRATION_TOKENS], self.scales[0, i:i + 1], cal_ws, BITS)
            self.out.append(torch.empty((tokens, N), dtype=dt, device=device))
        self.scales[1:] = self.scales[0]
        for layer in range(layers):
            for i, (_, K, N) in enumerate(LINEARS):
                w = W.weights_fp32(N, K, W.seed_of(CONFIG_ID, 1000 + layer * 7 + i) + 100_000 * rank, device=device)
                w_int = torch.empty((N, K), dtype=torch.int8, device=device)
                w_scale = torch.empty(N, dtype=torch.float32, device=device)
                P.sasq_quantize_weight(w, w_int, w_scale, 8)
                del w
                self.w_int[layer][i], self.w_scale[layer][i] = w_int, w_scale
        self.training = training
        if training:
            self.q_ws = torch.empty(P.sasq_fakequant_multi_workspace(7), dtype=torch.uint8, device=device)
            self.descs = P.QuantTensors([(self.x[i], self.g[i], self.y[i], self.dx[i], i) for i in range(7)])
        shapes = [(tokens, N, K) for _, K, N in LINEARS]
        self.l_ws = torch.empty(P.sasq_static_w8a8_linear_multi_workspace(shapes), dtype=torch.uint8, device=device)
        torch.cuda.synchronize()
        assert P.sasq_device_status() == 0

    def problems(self, layer: int, call, tokens: int | None = None):
        """The descriptor table of one call: the linears `call` of `layer` on the first `tokens` rows."""
        T = self.tokens if tokens is None else tokens
        return self.P.LinearProblems([(self.x[i][:T], self.w_int[layer][i], self.w_scale[layer][i],
                                       self.scales[layer, i:i + 1], self.out[i][:T]) for i in call])

    def prepare(self, linear_calls: str):
        """Descriptor tables marshalled once: the step submits the same buffers every time."""
        shapes = [(self.tokens, N, K) for _, K, N in LINEARS]
        self.calls = [[(self.problems(layer, call),
                        self.P.sasq_static_w8a8_linear_multi_launches([shapes[i] for i in call]))
                       for call in LINEAR_CALLS[linear_calls]] for layer in range(self.layers)]

    # kernels launched per step: one fused quantizer launch per layer (the reduction's second stage runs in its
    # last block), then the linears (activation quantizer inside the GEMM kernel)
    def phase_a_layer(self, layer: int):
        self.P.sasq_fakequant_fwd_bwd_multi(self.descs, self.scales[layer], self.grads[layer], self.q_ws, BITS,
                                            stream=self.stream)
        return 1

    def phase_b_layer(self, layer: int):
        n = 0
        for problems, launches in self.calls[layer]:
            self.P.sasq_static_w8a8_linear_multi(problems, self.l_ws, bits=BITS, stream=self.stream)
            n += launches
        return n

    def phase_a(self):
        return sum(self.phase_a_layer(layer) for layer in range(self.layers)) if self.training else 0

    def phase_b(self):
        return sum(self.phase_b_layer(layer) for layer in range(self.layers))


def max_over_ranks(values, dist, device):
    """Element-wise maximum of per-rank timings (the slowest rank decides); identity without a process group."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.tolist()]


def throughput(world: int, units_per_rank: float, steps: int, ms: float) -> float:
    """Whole-job rate: the units all ranks processed over the slowest rank's time (weak scaling, replicas)."""
    return world * units_per_rank * steps / (ms * 1e-3)


def tensor_peak_for(region_s: float, peaks: dict, peak_kind: str):
    """bf16 library peak x the nominal int8 : bf16 ratio; the burst figure for a short timed region, the sustained
    one for a region of a second or more."""
    if region_s >= SUSTAINED_REGION_S:
        return peaks["bf16_tflops_sustained"] * INT8_OVER_BF16_NOMINAL, f"{peak_kind} sustained bf16 x 2"
    return peaks["bf16_tflops"] * INT8_OVER_BF16_NOMINAL, f"{peak_kind} burst bf16 x 2"


def timed_reps(fn, min_seconds: float, min_reps: int = 5, max_reps: int = 2000, back_to_back: int = 0):
    """Runs fn() repeatedly between pairs of CUDA events until `min_seconds` of device time and `min_reps` samples
    have accumulated; returns milliseconds per call.  A sample is `back_to_back` calls submitted one after the other
    between one pair of events (0: as many as make a sample about a millisecond long, at most 50), so that short
    kernels are timed the way they run in a step, each behind the one before, not each behind an idle device."""
    stream = torch.cuda.current_stream()
    for _ in range(3):
        fn()
    torch.cuda.synchronize()
    inner = back_to_back
    if inner <= 0:
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        fn()
        b.record(stream)
        torch.cuda.synchronize()
        inner = int(max(1, min(50, round(1.0 / max(a.elapsed_time(b), 1e-3)))))
    out = []
    total = 0.0
    while (total < min_seconds * 1e3 or len(out) < min_reps) and len(out) < max_reps:
        batch = max(min_reps, min(50, max_reps - len(out)))
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(batch)]
        for a, b in ev:
            a.record(stream)
            for _ in range(inner):
                fn()
            b.record(stream)
        torch.cuda.synchronize()
        ms = [a.elapsed_time(b) for a, b in ev]
        out += [m / inner for m in ms]
        total += sum(ms)
    return out


def med_min(ms_list):
    return statistics.median(ms_list), min(ms_list)


# ---------------------------------------------------------------------------
# context measurements, outside the timed region (rank 0 of a single-GPU run)
# ---------------------------------------------------------------------------
def quantizer_modes(P, stack, tokens: int, seconds: float):
    """The quantizer on the seven tensors of a layer at `tokens` rows, one launch: forward only (4 B/element),
    backward only (6), fused (8)."""
    xs = [t[:tokens] for t in stack.x]
    gs = [t[:tokens] for t in stack.g]
    ys = [t[:tokens] for t in stack.y]
    dxs = [t[:tokens] for t in stack.dx]
    n = quantizer_elements(tokens)
    tables = {
        "fwd": (P.QuantTensors([(xs[i], None, ys[i], None, i) for i in range(7)]), 4),
        "bwd": (P.QuantTensors([(xs[i], gs[i], None, dxs[i], i) for i in range(7)]), 6),
        "fused": (P.QuantTensors([(xs[i], gs[i], ys[i], dxs[i], i) for i in range(7)]), 8),
    }
    out = {}
    for name, (tab, bpe) in tables.items():
        ms = timed_reps(lambda: P.sasq_fakequant_fwd_bwd_multi(tab, stack.scales[0], stack.grads[0], stack.q_ws, BITS),
                        seconds)
        med, mn = med_min(ms)
        out[name] = {"bytes_per_element": bpe, "us_median": round(med * 1e3, 2), "us_min": round(mn * 1e3, 2),
                     "gbs_median": round(bpe * n / (med * 1e-3) / 1e9, 1), "gbs_best": round(bpe * n / (mn * 1e-3) / 1e9, 1),
                     "reps": len(ms)}
    return out


def linears_by_calls(P, stack, tokens: int, seconds: float, modes=("each", "dependent", "layer"), graph: bool = False):
    """The seven static linears of a layer at `tokens` rows, back to back, for each way of submitting them; the
    layers' weights take turns so that no repetition finds its weights in L2.  graph: the calls of up to eight
    layers are captured once into a CUDA graph and the graph is replayed, which takes the host's per-call cost
    (about 5 us, of the order of a decode-sized kernel) out of the measurement; times are per layer."""
    ops = linear_ops(tokens)
    out = {}
    for name in modes:
        tables = [[stack.problems(layer, call, tokens) for call in LINEAR_CALLS[name]]
                  for layer in range(stack.layers)]
        turn = [0]

        def run():
            for problems in tables[turn[0] % len(tables)]:
                P.sasq_static_w8a8_linear_multi(problems, stack.l_ws, bits=BITS, stream=stack.stream)
            turn[0] += 1

        per = 1
        if graph:
            per = min(8, len(tables))
            for _ in range(per):
                run()                           # one-time set-up of every shape happens outside the capture
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            handle = stack.stream
            with torch.cuda.stream(side):
                stack.stream = side.cuda_stream
                turn[0] = 0
                with torch.cuda.graph(g, stream=side):
                    for _ in range(per):
                        run()
            stack.stream = handle
            torch.cuda.current_stream().wait_stream(side)
            torch.cuda.synchronize()
            ms = [m / per for m in timed_reps(g.replay, seconds)]
        else:
            ms = timed_reps(run, seconds)
        med, mn = med_min(ms)
        out[name] = {"us_median": round(med * 1e3, 2), "us_min": round(mn * 1e3, 2),
                     "tops_median": round(ops / (med * 1e-3) / 1e12, 2), "tops_best": round(ops / (mn * 1e-3) / 1e12, 2),
                     "weight_gbs_median": round(weight_bytes() / (med * 1e-3) / 1e9, 1), "reps": len(ms)}
    return out


def dynamic_per_token(P, stack, tokens: int, seconds: float):
    """Sec. 4.4, generation phase: the seven linears of a layer with dynamic per-token factors at `tokens` rows, one
    call per linear, submitted directly and replayed from a CUDA graph (times per layer)."""
    ws = torch.empty(max(P.sasq_dynamic_w8a8_linear_workspace(tokens, N, K) for _, K, N in LINEARS), dtype=torch.uint8,
                     device=stack.x[0].device)
    turn = [0]
    handle = [stack.stream]

    def run():
        layer = turn[0] % stack.layers
        for i in range(7):
            P.sasq_dynamic_w8a8_linear(stack.x[i][:tokens], stack.w_int[layer][i], stack.w_scale[layer][i],
                                       stack.out[i][:tokens], workspace=ws, stream=handle[0])
        turn[0] += 1

    out = {}
    ms = timed_reps(run, seconds)
    out["direct"] = {"us_median": round(statistics.median(ms) * 1e3, 2), "us_min": round(min(ms) * 1e3, 2)}
    per = min(8, stack.layers)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        handle[0] = side.cuda_stream
        turn[0] = 0
        with torch.cuda.graph(g, stream=side):
            for _ in range(per):
                run()
    handle[0] = stack.stream
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    ms = [m / per for m in timed_reps(g.replay, seconds)]
    out["graph_replay"] = {"us_median": round(statistics.median(ms) * 1e3, 2), "us_min": round(min(ms) * 1e3, 2)}
    return out


def yardsticks(P, device):
    """Same-box figures for the tensor peak: a library INT8 GEMM (yard-stick only, never the product path) and the
    issue rate of the GEMM's own tensor-core instruction, each as a burst and over about a second."""
    out = {}
    try:
        n = 8192
        a = torch.randint(-127, 128, (n, n), dtype=torch.int8, device=device)
        b = torch.randint(-127, 128, (n, n), dtype=torch.int8, device=device).t()     # column-major second operand
        ms = timed_reps(lambda: torch._int_mm(a, b), 0.0, min_reps=10, max_reps=10)
        burst = 2 * n ** 3 / (min(ms) * 1e-3) / 1e12
        ms = timed_reps(lambda: torch._int_mm(a, b), 1.0)
        out["library_int8_gemm_8192"] = {"tops_burst": round(burst, 1),
                                         "tops_sustained": round(2 * n ** 3 * len(ms) / (sum(ms) * 1e-3) / 1e12, 1),
                                         "what": "torch._int_mm 8192^3, int8 x int8 -> int32"}
        del a, b
    except Exception as e:  # the yard-stick is optional
        out["library_int8_gemm_8192"] = {"unavailable": f"{type(e).__name__}: {e}"[:160]}
    ops_b, mac_b = P.sasq_debug_int8_issue_rate(32 * 1024, 256)             # about 5 ms
    ops_s, mac_s = P.sasq_debug_int8_issue_rate(32 * 1024 * 192, 256)       # about a second
    out["int8_issue_rate_256x256x32"] = {"tops_burst": round(ops_b / 1e12, 1), "tops_sustained": round(ops_s / 1e12, 1),
                                         "mac_per_clk_per_sm": round(mac_b, 1),
                                         "what": "back-to-back tcgen05.mma.cta_group::2.kind::i8 from shared memory, "
                                                 "no loads, no epilogue"}
    return out


# ---------------------------------------------------------------------------
# our arm
# ---------------------------------------------------------------------------
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

    # the bench submits everything on one stream: launches need not be co-operative grids
    P.sasq_set_gang_launch(False)
    L, T = args.layers, args.tokens
    do_a, do_b = "a" in args.phases, "b" in args.phases
    stack = Stack(P, device, rank, L, T, training=do_a)
    stack.prepare(args.linear_calls)
    stream = torch.cuda.current_stream()

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def phase_a():
        return stack.phase_a() if do_a else 0

    def phase_b():
        return stack.phase_b() if do_b else 0

    warmup = max(args.warmup, 3)
    for _ in range(warmup):
        phase_a()
        phase_b()
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
        launches += phase_a()
        ev[k][1].record(stream)
        launches += phase_b()
        ev[k][2].record(stream)
    barrier()
    t_wall = time.perf_counter() - t_wall
    clocks = sampler.stop()
    assert P.sasq_device_status() == 0

    a_steps = [ev[k][0].elapsed_time(ev[k][1]) for k in range(K)]
    b_steps = [ev[k][1].elapsed_time(ev[k][2]) for k in range(K)]
    ms_a, ms_b = sum(a_steps), sum(b_steps)
    ms_total = ev[0][0].elapsed_time(ev[K - 1][2])
    ms_a, ms_b, ms_total = max_over_ranks([ms_a, ms_b, ms_total], dist, device)

    # a short timed region says little about a power-capped part: more steps of the same kind, outside the K timed
    # ones, until a second of device time has been seen; median and minimum per phase over all of them
    extra_a, extra_b = list(a_steps), list(b_steps)
    if world == 1 and not args.no_extras:
        while sum(extra_a) + sum(extra_b) < 1000.0 and len(extra_a) < 4000:
            e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
            e[0].record(stream); phase_a(); e[1].record(stream); phase_b(); e[2].record(stream)
            torch.cuda.synchronize()
            extra_a.append(e[0].elapsed_time(e[1]))
            extra_b.append(e[1].elapsed_time(e[2]))

    context = {}
    if world == 1 and not args.no_extras and do_a and do_b:
        context["quantizer_modes"] = quantizer_modes(P, stack, T, 0.3)
        cfg3 = {}
        for t3 in CONFIG3_TOKENS:
            if t3 <= T:
                cfg3[f"T{t3}"] = linears_by_calls(P, stack, t3, 0.3 if t3 >= 2048 else 0.15)
                if t3 <= 128:       # decode sizes: also with the host's per-call cost taken out
                    cfg3[f"T{t3}_graph_replay"] = linears_by_calls(P, stack, t3, 0.15, graph=True)
        context["config3_one_layer_by_tokens"] = cfg3
        context["dynamic_per_token_T1"] = dynamic_per_token(P, stack, 1, 0.15)
        if T >= 2048:
            context["config2_quantizer_T2048"] = quantizer_modes(P, stack, 2048, 0.3)["fused"]
            P.sasq_set_gang_launch(True)          # what callers that overlap linears on several streams switch on
            context["T2048_cooperative_launch"] = linears_by_calls(P, stack, 2048, 0.2, modes=("each", "dependent"))
            P.sasq_set_gang_launch(False)
        context["yardsticks"] = yardsticks(P, device)
        assert P.sasq_device_status() == 0

    # ---------------- end to end through the public API with HOST buffers ----------------
    e2e = measure_e2e(P, stack, device, dist, steps=2 if L > 4 else 5) if (do_a and do_b) else None

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return
    peaks, peak_kind = measured_peaks()
    qbytes, lops = quantizer_bytes(T, L), linear_ops(T, L)
    gbs = throughput(world, qbytes, K, ms_a) / 1e9 if do_a else None
    tops = throughput(world, lops, K, ms_b) / 1e12 if do_b else None
    region_s = ms_total * 1e-3
    int8_peak, int8_peak_src = tensor_peak_for(region_s, peaks, peak_kind)
    ach_q = qbytes * K / (ms_a * 1e-3) / 1e9 if do_a else None            # per GPU
    ach_l = lops * K / (ms_b * 1e-3) / 1e12 if do_b else None
    ys = context.get("yardsticks", {})
    issue = ys.get("int8_issue_rate_256x256x32", {})
    issue_peak = issue.get("tops_sustained" if region_s >= SUSTAINED_REGION_S else "tops_burst")
    # the denominator is a bf16 library GEMM scaled by the nominal ratio; the int8 instruction draws less power per
    # operation, so under the power cap the tensor cores themselves can retire more than that: when the same-box
    # issue-rate measurement is the higher of the two it is the bound, and the line says so
    peak, peak_src = int8_peak, int8_peak_src
    if issue_peak is not None and issue_peak > peak:
        peak, peak_src = issue_peak, ("same-run int8 tensor-core issue rate (" +
                                      ("sustained" if region_s >= SUSTAINED_REGION_S else "burst") + ")")
    line = {
        "metric": METRIC, "value": round(gbs, 2) if do_a else None, "unit": "GB/s", "n_gpus": world, "steps": K,
        "warmup": warmup, "ms_per_step": round(ms_total / K, 5), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16 storage, fp32 quantizer arithmetic, int8 x int8 -> int32 GEMM", "data": "synthetic",
        "config": config_of(args),
        "launch_mode": "single stream, plain launches (sasq_set_gang_launch(0))",
        "ms_phase_a": round(ms_a / K, 5), "ms_phase_b": round(ms_b / K, 5),
        "phase_stats": {"steps_seen": len(extra_a),
                        "a_ms_median": round(statistics.median(extra_a), 5), "a_ms_min": round(min(extra_a), 5),
                        "b_ms_median": round(statistics.median(extra_b), 5), "b_ms_min": round(min(extra_b), 5)},
        "gpu_launches": launches, "clocks": clocks, "wall_s": round(t_wall, 3),
    }
    if do_b:
        line["w8a8_linear"] = {"value": round(tops, 2), "unit": "TOPS", "ops_per_step": lops,
                               "frac_of_nominal_int8_4500": round(tops / world / NOMINAL_INT8_TOPS, 4),
                               "linear_calls": args.linear_calls}
        line["roofline"] = {
            "kernel": "w8a8_gemm_pair_kernel (tcgen05 int8, CTA pairs, activation quantizer inside)",
            "bound": "tensor", "achieved": round(ach_l, 2), "peak": round(peak, 1), "unit": "TOP/s",
            "frac": round(ach_l / peak, 4), "peak_source": peak_src,
            "timed_region_s": round(region_s, 4),
            "traffic": NCU_TRAFFIC.get(("gemm_q_proj" if T == 16384 else "gemm_layer", T)),
            "traffic_note": ("DRAM bytes of one q_proj launch (T x 4096 x 4096)" if T == 16384 else
                             "DRAM bytes of the launch that runs a layer's seven linears"),
            "alternative_peaks": {
                "bf16_library_x2": {"peak": round(int8_peak, 1), "frac": round(ach_l / int8_peak, 4),
                                    "source": int8_peak_src},
                "nominal_int8": {"peak": NOMINAL_INT8_TOPS, "frac": round(ach_l / NOMINAL_INT8_TOPS, 4)},
                "int8_issue_rate": ({"peak": issue_peak, "frac": round(ach_l / issue_peak, 4)} if issue_peak else None),
                "library_int8_gemm": ys.get("library_int8_gemm_8192"),
            }}
    if do_a:
        line["roofline_quantizer"] = {
            "kernel": "fakequant_kernel (fused fwd+bwd)", "bound": "hbm", "achieved": round(ach_q, 1),
            "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": round(ach_q / peaks["hbm_gbs"], 4),
            "frac_of_nominal_8000": round(ach_q / NOMINAL_HBM_GBS, 4),
            "traffic": NCU_TRAFFIC.get(("fakequant", T)), "peak_source": f"{peak_kind} copy bandwidth"}
    line.update(context)
    line["e2e"] = e2e
    if do_a and do_b:
        line["cpu_baseline"] = cpu_baseline()
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def measure_e2e(P, stack, device, dist, steps: int):
    """The same step through the public API with HOST inputs: for every layer the step copies that layer's x and g
    (seven tensors each) from pinned host memory into the shared device buffers, runs the layer's quantizer launch
    and its linears, and at the end reads the 7 x layers scale gradients and the last layer's down_proj output back
    to the host.  One layer's worth of pinned host memory serves every layer (the bytes copied are what counts)."""
    hx = [t.cpu().pin_memory() for t in stack.x]
    hg = [t.cpu().pin_memory() for t in stack.g]
    h_grads = torch.empty(stack.grads.shape, dtype=torch.float32).pin_memory()
    h_out = torch.empty(stack.out[6].shape, dtype=stack.out[6].dtype).pin_memory()
    h2d = sum(t.numel() * t.element_size() for t in hx + hg) * stack.layers
    d2h = h_grads.numel() * 4 + h_out.numel() * h_out.element_size()
    stream = torch.cuda.current_stream()

    def step():
        for layer in range(stack.layers):
            for i in range(7):
                stack.x[i].copy_(hx[i], non_blocking=True)
                stack.g[i].copy_(hg[i], non_blocking=True)
            stack.phase_a_layer(layer)
            stack.phase_b_layer(layer)
        h_grads.copy_(stack.grads, non_blocking=True)
        h_out.copy_(stack.out[6], non_blocking=True)

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
    return {"value": round(world * quantizer_bytes(stack.tokens, stack.layers) / (ms * 1e-3) / 1e9, 2), "unit": "GB/s",
            "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": round(ms, 4), "steps": steps,
            "w8a8_tops": round(world * linear_ops(stack.tokens, stack.layers) / (ms * 1e-3) / 1e12, 3)}


# ---------------------------------------------------------------------------
# CPU oracle legs
# ---------------------------------------------------------------------------
def _oracle_sample(gemm_rows: int):
    """Times the oracle, as it stands, on a bounded sample of the step: the quantizer forward and backward on the
    first CPU_SAMPLE_TOKENS tokens of the seven tensors of layer 0, and the integer GEMM + dequant on `gemm_rows`
    rows of each of that layer's seven linears."""
    import numpy as np
    import oracle

    t_q = 0.0
    t_l = 0.0
    ops = 0
    for i, (_, K, N) in enumerate(LINEARS):
        seed = W.seed_of(CONFIG_ID, i)
        xb, tag = oracle.bits_of(W.activations(CPU_SAMPLE_TOKENS, K, torch.bfloat16, seed))
        gb, _ = oracle.bits_of(W.upstream_grad(CPU_SAMPLE_TOKENS, K, torch.bfloat16, seed))
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


def cpu_baseline(budget_seconds: float = 20.0):
    import oracle
    # as many GEMM rows as fit the budget (sized from a 32-row probe); the quantizer part runs on all sampled tokens
    _, t_probe, _ = _oracle_sample(32)
    gemm_rows = int(min(CPU_SAMPLE_TOKENS, max(32, 32 * budget_seconds / max(t_probe, 1e-3))))
    gemm_rows -= gemm_rows % 8
    t_q, t_l, ops = _oracle_sample(gemm_rows)
    # the oracle runs forward and backward as two passes: 4 + 6 algorithmic bytes per element;
    # the reported GB/s uses the step's 8 bytes per element so that it is the same metric
    return {"value": round(quantizer_bytes(CPU_SAMPLE_TOKENS) / t_q / 1e9, 3), "unit": "GB/s",
            "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"layer 0, first {CPU_SAMPLE_TOKENS} tokens: quantizer fwd+bwd on the 7 tensors; int GEMM+dequant "
                      f"on the first {gemm_rows} rows of each of the 7 linears",
            "w8a8_tops": round(ops / t_l / 1e12, 5), "seconds": round(t_q + t_l, 2)}


def run_reference(args):
    """Reference arm: the CPU oracle, as it stands, on the machine's host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    K = max(1, args.steps)
    rows = 32
    warm = 0
    t_warm = time.perf_counter()
    for _ in range(max(0, args.warmup)):
        if time.perf_counter() - t_warm > 30:      # the oracle has no caches to warm: a bounded courtesy
            break
        _oracle_sample(rows)
        warm += 1
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
        if time.perf_counter() - t_all > 120:      # keep the whole run within a few minutes
            break
    gbs = quantizer_bytes(CPU_SAMPLE_TOKENS) * done / t_q / 1e9
    sample = (f"per step: layer 0, first {CPU_SAMPLE_TOKENS} of {args.tokens} tokens: quantizer fwd+bwd on the 7 "
              f"tensors; int GEMM+dequant on the first {rows} rows of each of the 7 linears; {done} of {K} requested "
              f"steps timed")
    line = {
        "impl": "reference", "metric": METRIC, "value": round(gbs, 3), "unit": "GB/s",
        "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": done, "warmup": warm,
        "ms_per_step": round((t_q + t_l) / done * 1e3, 3), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "fp32 quantizer arithmetic with double accumulation; int32 GEMM", "data": "synthetic",
        "config": config_of(args),
        "w8a8_linear": {"value": round(ops / t_l / 1e12, 5), "unit": "TOPS"},
        "cpu_baseline": {"value": round(gbs, 3), "unit": "GB/s", "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": round(gbs, 3), "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--linear-calls", choices=["layer", "dependent", "each"], default="dependent",
                    help="phase B submits the seven linears of a layer in the groups a decoder layer's data flow "
                         "allows (q/k/v | o | gate/up | down; the default), in one call, or one call per linear")
    ap.add_argument("--tokens", type=int, default=16384,
                    help="tokens per step (default 8 x 2048, the full calibration batch)")
    ap.add_argument("--layers", type=int, default=32, help="decoder layers (default 32, the full stack)")
    ap.add_argument("--phases", choices=["ab", "a", "b"], default="ab", help="run only one phase (profiling)")
    ap.add_argument("--no-extras", action="store_true",
                    help="skip the context measurements after the timed region (profiling)")
    args = ap.parse_args()
    if args.tokens < 1 or args.layers < 1:
        ap.error("--tokens and --layers must be positive")
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
