#!/usr/bin/env python
"""Benchmark of the FP8 linear hot path (amax -> bias -> cast -> FP8 matmuls
with unscale, forward + backward) on synthetic tensors shaped like the
paper's layers.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

One "step" is one pass of the whole path over one batch: every tensor of the
workload's decoder block is quantised (weights, activations and, for
training workloads, output gradients: amax, Eq. 3 bias, cast), then every
linear runs its forward, input-gradient and weight-gradient matmul.  Prints ONE
JSON line on rank 0.  With N > 1 (torchrun) every rank runs the same single-GPU
path on its own tensors (replicas; the method has no exchange step).

`--impl reference` times the CPU oracle, as it stands, on the host cores.

Single-kernel legs (one line of text per shape, no JSON):

    python bench.py --leg gemm  --shapes 8192x8192x16384 8192x22016x4096   # MxNxK forward matmuls and fused epilogues
    python bench.py --leg cast  --shapes 8192x4096 8192x22016              # amax, cast, amax+cast of bf16 [rows x cols]
    python bench.py --leg stack --shapes 24x1024x4096                      # layers x d x tokens: the SGD stack
    python bench.py --leg mlp   --shapes 8192x4096x11008                   # tokens x d x ffn: a gated MLP, unfused vs fused
    python bench.py --leg group --workload c2_gpt                          # fp8_cast_group over a workload's tensors, each mode
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch

from paper_2309_17224_b200 import inputs as I

METRIC = "fp8_linear_fwd_bwd_tflops"
UNIT = "TFLOP/s"
DEFAULT_WORKLOAD = "c3_llama7b"
ORACLE_SAMPLE_TOKENS = 256          # floor of the sample; see oracle_sample_tokens
EVENT_EVERY = 8   # per-kernel CUDA-event pairs are recorded on every eighth timed step
ORACLE_SAMPLE_LAYER = 1  # the square attention-output projection
NOMINAL_FP8_TFLOPS = 4500.0         # dense FP8, the vendor's figure for the part
FP8_FLOP_PER_CLK_PER_SM = 16384.0   # 8192 multiply-adds per clock per SM: nominal peak / (148 SMs x 1.856 GHz)
# dram__bytes_read.sum + dram__bytes_write.sum per matmul launch, from one ncu capture of the workload's steps
# (profiles/launch_list_c3_llama7b.md); keyed by (workload, tokens, one launch per step or one per matmul)
GEMM_DRAM_BYTES_PER_LAUNCH = {("c3_llama7b", 8192, "per-call"): 331.3e6, ("c3_llama7b", 8192, "group"): 4722.9e6}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# ----------------------------------------------------------------------------
# clocks
# ----------------------------------------------------------------------------

class ClockSampler:
    """SM clock and throttle reasons sampled DURING the timed region: NVML polled every 10 ms from a thread
    (read-only queries), or `nvidia-smi -lms 100` when the NVML binding is missing."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, device_index: int):
        self.proc = None
        self.path = None
        self.thread = None
        self.sm, self.mx, self.reasons = [], [], set()
        try:
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
        except Exception:
            return
        try:
            import pynvml as N
            N.nvmlInit()
            try:
                h = N.nvmlDeviceGetHandleByUUID(uuid)
            except TypeError:
                h = N.nvmlDeviceGetHandleByUUID(uuid.encode())
            self.mx.append(float(N.nvmlDeviceGetMaxClockInfo(h, N.NVML_CLOCK_SM)))
            bits = {"hw_slowdown": N.nvmlClocksThrottleReasonHwSlowdown,
                    "hw_thermal_slowdown": N.nvmlClocksThrottleReasonHwThermalSlowdown,
                    "sw_thermal_slowdown": N.nvmlClocksThrottleReasonSwThermalSlowdown,
                    "sw_power_cap": N.nvmlClocksThrottleReasonSwPowerCap}
            self._stop = threading.Event()

            def poll():
                while not self._stop.is_set():
                    try:
                        self.sm.append(float(N.nvmlDeviceGetClockInfo(h, N.NVML_CLOCK_SM)))
                        r = N.nvmlDeviceGetCurrentClocksThrottleReasons(h)
                        for name, bit in bits.items():
                            if r & bit:
                                self.reasons.add(name)
                    except Exception:
                        pass
                    self._stop.wait(0.01)

            self.thread = threading.Thread(target=poll, daemon=True)
            self.thread.start()
            return
        except Exception:
            self.thread = None
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", uuid, f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.thread is not None:
            self._stop.set()
            self.thread.join(timeout=2)
            if self.sm:
                out.update(sm_mhz=statistics.median(self.sm), sm_max_mhz=max(self.mx), reasons=sorted(self.reasons),
                           samples=len(self.sm), source="nvml, 10 ms")
            return out
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        try:
            with open(self.path) as fh:
                for line in fh:
                    parts = [x.strip() for x in line.split(",")]
                    if len(parts) < 7:
                        continue
                    try:
                        sm.append(float(parts[0]))
                        mx.append(float(parts[1]))
                    except ValueError:
                        continue
                    for n, v in zip(self.NAMES, parts[3:7]):
                        if v.lower().startswith("active"):
                            reasons.add(n)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm),
                       source="nvidia-smi, 100 ms")
        return out


# ----------------------------------------------------------------------------
# our arm
# ----------------------------------------------------------------------------

class LayerState:
    """Device buffers of one linear: bf16 inputs, FP8 copies, device scalars, bf16 outputs."""

    def __init__(self, wl, li, device, seed, backward, tokens=0, transposed=False):
        l = wl.layers[li]
        T, K, N = tokens or wl.tokens, l.K, l.N
        self.T, self.K, self.N, self.name = T, K, N, l.name
        t = I.layer_tensors(wl, li, device=device, seed=seed, tokens=T)
        self.x, self.w = t["x"], t["w"]
        self.g = t.get("g")
        u8 = dict(dtype=torch.uint8, device=device)
        self.x8, self.w8 = torch.empty((T, K), **u8), torch.empty((N, K), **u8)
        self.y = torch.empty((T, N), dtype=torch.bfloat16, device=device)
        self.scal_f = torch.zeros(4, dtype=torch.float32, device=device)
        self.scal_i = torch.zeros(4, dtype=torch.int32, device=device)
        self.backward = backward
        self.transposed = transposed
        if backward:
            self.x8t = self.w8t = self.g8t = None
            if transposed:
                self.x8t, self.w8t = torch.empty((K, T), **u8), torch.empty((K, N), **u8)
                self.g8t = torch.empty((N, T), **u8)
            self.g8 = torch.empty((T, N), **u8)
            self.dx = torch.empty((T, K), dtype=torch.bfloat16, device=device)
            self.dw = torch.empty((N, K), dtype=torch.bfloat16, device=device)
        else:
            self.x8t = self.w8t = self.g8 = self.g8t = self.dx = self.dw = None

    def gemm_flops(self):
        return 2.0 * self.T * self.K * self.N * (3 if self.backward else 1)

    def gemm_bytes(self):
        """FP8 operands + bf16 output of this layer's matmuls."""
        T, K, N = self.T, self.K, self.N
        fwd = T * K + N * K + 2 * T * N
        if not self.backward:
            return fwd
        return fwd + (T * N + N * K + 2 * T * K) + (T * N + T * K + 2 * N * K)

    def cast_elements(self):
        if not self.backward:
            return self.T * self.K          # weights were quantised once, at load
        return self.T * self.K + self.N * self.K + self.T * self.N

    def quant_items(self):
        """(format, tensor, amax word, bias word, FP8 bytes) of every tensor this layer quantises per step."""
        E4, E5 = 0, 1
        af, bi = self.scal_f, self.scal_i
        items = [(E4, self.x, af[1:2], bi[1:2], self.x8)]
        if self.backward:   # training: the weights are re-quantised every step; inference: once at load
            items = [(E4, self.w, af[0:1], bi[0:1], self.w8)] + items + [(E5, self.g, af[2:3], bi[2:3], self.g8)]
        return items


class Timers:
    """CUDA-event pairs around groups of launches, on the launching stream."""

    def __init__(self):
        self.pairs = {"gemm": [], "amax_cast": []}
        self.layers = {}   # layer name -> event pairs around the layer's matmuls

    def span(self, key):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        self.pairs[key].append((a, b))
        return a, b

    def layer_span(self, name):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        self.layers.setdefault(name, []).append((a, b))
        return a, b

    def layer_ms(self):
        return {k: sum(a.elapsed_time(b) for a, b in v) / len(v) for k, v in self.layers.items()}

    def total_ms(self, key):
        return sum(a.elapsed_time(b) for a, b in self.pairs[key])

    def count(self, key):
        return len(self.pairs[key])


def _timed(timers, key, fn):
    if timers is None:
        fn()
    else:
        a, b = timers.span(key)
        a.record()
        fn()
        b.record()


def run_matmuls(ctx, L, timers=None):
    bi = L.scal_i
    # forward-only workloads run on weights quantised once at load: the inference call may read them early
    fwd = ctx.linear_fwd if L.backward else ctx.linear_infer
    _timed(timers, "gemm", lambda: fwd(L.x8, bi[1:2], L.w8, bi[0:1], L.y))
    if L.backward:
        if L.transposed:   # contraction over contiguous bytes, from the transposed copies
            _timed(timers, "gemm", lambda: ctx.linear_dgrad(L.g8, bi[2:3], None, L.w8t, bi[0:1], L.dx))
            _timed(timers, "gemm", lambda: ctx.linear_wgrad(None, L.g8t, bi[2:3], None, L.x8t, bi[1:2], L.dw, L.T))
        else:              # the tensor core reads the forward layouts directly
            _timed(timers, "gemm", lambda: ctx.linear_dgrad(L.g8, bi[2:3], L.w8, None, bi[0:1], L.dx))
            _timed(timers, "gemm", lambda: ctx.linear_wgrad(L.g8, None, bi[2:3], L.x8, None, bi[1:2], L.dw, L.T))


def fused_decode(L):
    """Forward-only layer on at most 128 rows: one launch quantises the activation and multiplies."""
    return (not L.backward) and L.T <= 128 and not L.transposed and not NO_FUSED_DECODE


def run_layer(ctx, L, timers=None, predict=False):
    """One layer of one step with every tensor quantised by its own call (two launches per tensor; one pass with
    predict=True when the bias left by the previous step still holds)."""
    af, bi = L.scal_f, L.scal_i
    E4, E5 = 0, 1
    if fused_decode(L):
        # inference on a few rows: the activation is quantised by the matmul's own launch (fp8_linear_infer_cast)
        _timed(timers, "gemm", lambda: ctx.linear_infer_cast(L.x, af[1:2], bi[1:2], L.x8, L.w8, bi[0:1], L.y))
        return
    if predict and not L.transposed:
        quant = lambda fmt, x, j, y, yt: ctx.cast_predicted(fmt, x, af[j:j + 1], bi[j:j + 1], y)
    else:
        quant = lambda fmt, x, j, y, yt: (ctx.cast_e4 if fmt == E4 else ctx.cast_e5)(
            x, None, d_amax_out=af[j:j + 1], d_bias_out=bi[j:j + 1], y=y, y_t=yt)
    if L.backward:
        _timed(timers, "amax_cast", lambda: quant(E4, L.w, 0, L.w8, L.w8t))
    _timed(timers, "amax_cast", lambda: quant(E4, L.x, 1, L.x8, L.x8t))
    if L.backward:
        _timed(timers, "amax_cast", lambda: quant(E5, L.g, 2, L.g8, L.g8t))
    run_matmuls(ctx, L, timers)


NO_FUSED_DECODE = False   # --no-fused-decode: decode layers as fp8_cast_e4 + fp8_linear_infer (two launches)

QUANT_MODES = ("group-predicted", "group", "per-tensor", "per-tensor-predicted")


class Step:
    """One step of a workload under one quantisation mode.

    group-predicted       every tensor of the step in one fp8_cast_group call, FP8_GROUP_PREDICTED: one pass per
                          tensor when the bias its previous step left still holds, the tensor cast again otherwise
                          (results identical to the just-in-time path either way)
    group                 the same call, FP8_GROUP_AMAX_CAST: an amax pass and a cast pass over the whole group
    per-tensor            fp8_cast_e4 / _e5 per tensor (two launches each), layer by layer
    per-tensor-predicted  fp8_cast_predicted per tensor
    Decode-size batches (at most 128 tokens) always take the per-tensor path: their activations fit the
    single-launch register-resident kernel, which chains into the matmul behind it."""

    def __init__(self, ctx, fp8lin, layers, mode, tokens, matmuls="group"):
        """matmuls: "group" = all matmuls of the step in one fp8_linear_group call (the layers of a step are
        independent here: every operand is quantised before the first matmul), "per-call" = one call each."""
        self.ctx, self.layers = ctx, layers
        grouped = mode.startswith("group") and tokens > 128 and not any(L.transposed for L in layers)
        self.mode = mode if grouped or not mode.startswith("group") else "per-tensor"
        self.items = None
        self.mm_items = None
        if grouped:
            self.items = fp8lin.group_items([it for L in layers for it in L.quant_items()])
            self.group_mode = fp8lin.GROUP_PREDICTED if mode == "group-predicted" else fp8lin.GROUP_AMAX_CAST
            if matmuls == "group":
                mm = []
                for L in layers:
                    bi = L.scal_i
                    mm.append((fp8lin.MATMUL_FWD, L.x8, bi[1:2], L.w8, bi[0:1], L.y))
                    if L.backward:
                        mm.append((fp8lin.MATMUL_DGRAD, L.g8, bi[2:3], L.w8, bi[0:1], L.dx))
                        mm.append((fp8lin.MATMUL_WGRAD, L.g8, bi[2:3], L.x8, bi[1:2], L.dw))
                self.mm_items = fp8lin.matmul_items(mm)
        self.matmuls = "group" if self.mm_items is not None else "per-call"

    def launches_per_step(self):
        """Kernel launches the library enqueues per step, counted by the library itself (fp8_launch_count)."""
        import paper_2309_17224_b200.fp8lin as lib
        n0 = lib.launch_count()
        self.run()
        return lib.launch_count() - n0

    def run(self, timers=None):
        ctx = self.ctx
        if self.items is not None:
            _timed(timers, "amax_cast", lambda: ctx.cast_group(self.items, mode=self.group_mode))
            if self.mm_items is not None:
                _timed(timers, "gemm", lambda: ctx.linear_group(self.mm_items))
                return
            for L in self.layers:
                if timers is not None:
                    la, lb = timers.layer_span(L.name)
                    la.record()
                run_matmuls(ctx, L, timers)
                if timers is not None:
                    lb.record()
        else:
            for L in self.layers:
                run_layer(ctx, L, timers, predict=self.mode == "per-tensor-predicted")


def dist_setup(n_gpus, backend="nccl"):
    """One process per GPU (torchrun sets RANK / WORLD_SIZE / LOCAL_RANK).  The ranks are independent replicas:
    the process group serves the barrier and the max-over-ranks of the measured time only.  `backend="gloo"`
    is the CPU form used by the tests."""
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    cuda = backend == "nccl"
    if world > 1:
        import torch.distributed as dist
        if cuda:
            torch.cuda.set_device(local)
            dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        else:
            dist.init_process_group(backend)
        return rank, world, local, dist
    if cuda:
        torch.cuda.set_device(0)
    return 0, 1, 0, None


def barrier_sync(dist, cuda=True):
    if cuda:
        torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    if cuda:
        torch.cuda.synchronize()


def whole_job_value(world, step_flops, ms_per_step):
    """Aggregate TFLOP/s of `world` replicas that each did `step_flops` per step in the slowest rank's time."""
    return world * step_flops / (ms_per_step * 1e-3) / 1e12


def max_over_ranks(value, dist, device):
    if dist is None:
        return value
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def timed_loop(fn, steps, dist, device):
    """ms per call of fn over `steps` calls: CUDA events on the launching stream, barrier + synchronize on both
    sides, max over ranks."""
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier_sync(dist)
    a.record()
    for _ in range(steps):
        fn()
    b.record()
    barrier_sync(dist)
    return max_over_ranks(a.elapsed_time(b), dist, device) / steps


def quantisation_kernel_bandwidths(ctx, fp8lin, layers, peak_gbs, reps=3):
    """The quantisation kernels timed one launch at a time (CUDA events on the launching stream), each against its
    own algorithmic bytes, with the inputs out of L2 (the tensors of a step total far more than L2 and every launch
    walks all of them, or the launches cycle through them).

    grouped: the amax pass, the cast pass and the one-pass (amax + cast) kernel of fp8_cast_group over all tensors
    of the step; per tensor: fp8_amax and fp8_cast_* on one tensor per launch; library_copy: torch's
    device-to-device copy of the same tensors (2 B read + 2 B written per element), the rate a plain copy reaches
    at these sizes."""
    tensors = [it for L in layers for it in L.quant_items()]
    dev = tensors[0][1].device
    amax = torch.zeros(1, dtype=torch.float32, device=dev)
    bias = torch.zeros(1, dtype=torch.int32, device=dev)
    items = fp8lin.group_items(tensors)
    elems = sum(t[1].numel() for t in tensors)
    out = {"how": f"one launch at a time, {reps} passes after one untimed, inputs out of L2; grouped kernels walk the step's "
                  f"{len(tensors)} tensors ({elems / 1e6:.0f} M elements) per launch"}

    def timed_once(fn):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda._sleep(100000)  # ~50 us of spinning ahead of the pair: the host enqueues the event, the launch
        a.record()                 # and the event while the stream is busy, so the interval holds the kernel and
        fn()                       # not the host's launch latency
        b.record()
        return a, b

    grouped = (("group_amax", 2, lambda: ctx.cast_group(items, mode=fp8lin.GROUP_AMAX_ONLY)),
               ("group_cast", 3, lambda: ctx.cast_group(items, mode=fp8lin.GROUP_CAST_ONLY)),
               ("group_amax_cast_one_pass", 3, lambda: ctx.cast_group(items, mode=fp8lin.GROUP_PREDICTED)))
    for key, bpe, fn in grouped:
        spans = [timed_once(fn) for _ in range(reps + 1)][1:]
        torch.cuda.synchronize()
        ms = [a.elapsed_time(b) for a, b in spans]
        gbs = elems * bpe / (sum(ms) / len(ms) * 1e-3) / 1e9
        out[key] = {"gbs": gbs, "frac": gbs / peak_gbs, "ms": sum(ms) / len(ms), "bytes_per_element": bpe}
    out["group_amax_cast_one_pass"]["note"] = ("both launches of the call (the second finds nothing to redo: every "
                                               "guess holds on repeated tensors)")

    scratch = torch.empty(max(t[1].numel() for t in tensors), dtype=tensors[0][1].dtype, device=dev)

    def launch(key, fmt, x, y):
        if key == "amax":
            ctx.amax(x, amax)
        elif key == "cast":
            (ctx.cast_e5 if fmt else ctx.cast_e4)(x, bias, y=y)
        else:
            scratch[:x.numel()].copy_(x.reshape(-1))

    for key, bpe in (("amax", 2), ("cast", 3), ("library_copy", 4)):   # one kind at a time: a tensor was last touched a whole round ago
        spans = []
        for rep in range(reps + 1):
            for fmt, x, _, _, y in tensors:
                a, b = timed_once(lambda: launch(key, fmt, x, y))
                if rep > 0:                # the first pass loads the kernels
                    spans.append((x.numel(), a, b))
        torch.cuda.synchronize()
        rates = [n * bpe / (a.elapsed_time(b) * 1e-3) / 1e9 for n, a, b in spans]
        total_b = sum(n * bpe for n, _, _ in spans)
        total_s = sum(a.elapsed_time(b) for _, a, b in spans) * 1e-3
        out["per_tensor_" + key if key != "library_copy" else key] = {
            "gbs": total_b / total_s / 1e9, "frac": total_b / total_s / 1e9 / peak_gbs, "slowest_tensor_gbs": min(rates),
            "bytes_per_element": bpe}
    return out


# ----------------------------------------------------------------------------
# the CPU oracle as a timed baseline
# ----------------------------------------------------------------------------

def oracle_sample_tokens(wl, seconds):
    """Token count at which one oracle pass over the sample layer takes about `seconds` on this host: a 32-token
    pass is timed first (the quantisation of the weight tensor is a fixed cost, the matmuls grow with the tokens)."""
    probe = min(32, wl.tokens)
    oracle_sample_run(wl, I.BASE_SEED, probe)   # the oracle's one-time table set-up stays out of the estimate
    dt_small = oracle_sample_run(wl, I.BASE_SEED, probe)[0]
    dt_big = oracle_sample_run(wl, I.BASE_SEED, min(2 * probe, wl.tokens))[0]
    per_token = max((dt_big - dt_small) / probe, 1e-6)
    fixed = max(dt_small - per_token * probe, 0.0)
    T = int(max(seconds - fixed, 0.0) / per_token) // 16 * 16
    return max(16, min(T, 1024, wl.tokens))


ORACLE_SPLIT = {}   # the last oracle_sample_run's time, split into quantisation (3 B per element) and matmuls


def oracle_sample_run(wl, seed, tokens=ORACLE_SAMPLE_TOKENS):
    """One bounded sample of the workload on the CPU oracle: the whole path
    (amax, bias, cast of X, W, dY; the three matmuls) for one layer at a
    reduced token count.  Returns (seconds, flops, description, threads, layer, tokens)."""
    import oracle as O
    li = min(ORACLE_SAMPLE_LAYER, len(wl.layers) - 1)
    l = wl.layers[li]
    T = min(tokens, wl.tokens)
    t = I.layer_tensors(wl, li, device="cpu", seed=seed, tokens=T)
    xb, wb = I.bits(t["x"]), I.bits(t["w"])
    gb = I.bits(t["g"]) if wl.backward else None
    t0 = time.perf_counter()
    _, bx, x8 = O.quantise(xb, O.E4)
    _, bw, w8 = O.quantise(wb, O.E4)
    elements = xb.size + wb.size
    if wl.backward:
        _, bg, g8 = O.quantise(gb, O.E5)
        elements += gb.size
    t1 = time.perf_counter()
    O.linear_fwd(x8, bx + 1, w8, bw + 1)
    flops = 2.0 * T * l.K * l.N
    if wl.backward:
        O.linear_dgrad(g8, bg, w8, bw + 1)
        O.linear_wgrad(g8, bg, x8, bx + 1)
        flops *= 3
    dt = time.perf_counter() - t0
    ORACLE_SPLIT.update(quantise_seconds=t1 - t0, quantise_elements=int(elements), matmul_seconds=dt - (t1 - t0),
                        amax_cast_gbs=3.0 * elements / (t1 - t0) / 1e9, matmul_tflops=flops / (dt - (t1 - t0)) / 1e12)
    what = (f"layer '{l.name}' ({l.K}->{l.N}) of {wl.name} at {T} of {wl.tokens} tokens: amax+bias+cast of X, W"
            f"{', dY' if wl.backward else ''} and {'3 matmuls' if wl.backward else '1 matmul'}, {flops / 1e9:.1f} GFLOP")
    return dt, flops, what, O.num_threads(), l, T


def reference_arm(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    import oracle as O
    O.build()
    # exactly W warm-up and K timed steps; the sample shrinks so that the whole run stays near two minutes
    steps, warmup = max(1, args.steps), max(0, args.warmup)
    tokens = oracle_sample_tokens(wl, min(15.0, 120.0 / (steps + warmup)))
    for _ in range(warmup):
        oracle_sample_run(wl, I.BASE_SEED, tokens)
    times, flops, what, cores, layer, T = [], 0.0, "", 1, None, tokens
    for _ in range(steps):
        dt, flops, what, cores, layer, T = oracle_sample_run(wl, I.BASE_SEED, tokens)
        times.append(dt)
    ms = 1e3 * sum(times) / len(times)
    value = flops / (ms * 1e-3) / 1e12
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
        "warmup": warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        # what each step of THIS arm computes: a bounded sample of the workload, not the whole of it
        "config": {"workload": f"{wl.name}: sample of one layer at reduced tokens", "of_workload": wl.name,
                   "tokens": T, "of_tokens": wl.tokens, "layers": [f"{layer.name}:{layer.K}->{layer.N}"],
                   "of_layers": [f"{l.name}:{l.K}->{l.N}" for l in wl.layers],
                   "passes": "fwd+bwd" if wl.backward else "fwd"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": what, **ORACLE_SPLIT},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


# ----------------------------------------------------------------------------
# single-kernel legs
# ----------------------------------------------------------------------------

def _time_each(fn, iters, pre=None):
    fn()   # first launch of a kernel pays its one-time load
    torch.cuda.synchronize()
    total = 0.0
    for _ in range(iters):
        if pre:
            pre()
        s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s.record()
        fn()
        e.record()
        torch.cuda.synchronize()
        total += s.elapsed_time(e)
    return total / iters


def _time_burst(fn, iters, warm=3):
    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    s.record()
    for _ in range(iters):
        fn()
    e.record()
    torch.cuda.synchronize()
    return s.elapsed_time(e) / iters


def leg_gemm(ctx, fp8lin, shapes, iters=20, fused=True):
    """MxNxK forward matmuls on random FP8 bytes (no NaN codes), then the fused epilogues on the same operands."""
    for M, N, K in shapes:
        a = torch.randint(0, 0x78, (M, K), dtype=torch.uint8, device="cuda")
        b = torch.randint(0, 0x78, (N, K), dtype=torch.uint8, device="cuda")
        bias = torch.zeros(1, dtype=torch.int32, device="cuda")
        y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
        ms = _time_burst(lambda: ctx.linear_fwd(a, bias, b, bias, y), iters)
        line = f"gemm M={M} N={N} K={K}: {2.0 * M * N * K / ms / 1e9:8.1f} TFLOP/s  {ms * 1e3:8.1f} us"
        if M > 128 and N % 8 == 0:
            t = _time_burst(lambda: ctx.selftest_mma_ceiling(y, bias, K), iters)
            line += f" | operand loads off {2.0 * M * N * K / t / 1e9:7.1f} TF {t * 1e3:7.1f} us"
        if fused and N % 16 == 0 and K % 16 == 0:
            # GELU + amax; GELU + amax + FP8 bytes; GELU' of a stored pre-activation + amax + FP8 bytes (an
            # input-gradient matmul, so its output is [M, K])
            z = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
            z8 = torch.empty((M, N), dtype=torch.uint8, device="cuda")
            amax = torch.zeros(1, dtype=torch.float32, device="cuda")
            g8 = torch.empty((M, K), dtype=torch.uint8, device="cuda")
            pre = torch.randn((M, K), device="cuda").to(torch.bfloat16)
            dy = torch.randint(0, 0x78, (M, N), dtype=torch.uint8, device="cuda")
            runs = (("gelu", lambda: ctx.linear_fwd_act(a, bias, b, bias, y, z, d_amax_act=amax)),
                    ("gelu->fp8", lambda: ctx.linear_fwd_q(a, bias, b, bias, z8, bias, y_pre=y, d_amax_z=amax,
                                                           act=fp8lin.ACT_GELU)),
                    ("gelu->fp8 (bytes only)", lambda: ctx.linear_fwd_q(a, bias, b, bias, z8, bias, act=fp8lin.ACT_GELU)),
                    ("->fp8 (bytes only)", lambda: ctx.linear_fwd_q(a, bias, b, bias, z8, bias)),
                    ("dgrad gelu'->fp8", lambda: ctx.linear_dgrad_q(dy, bias, b, None, bias, g8, bias, y_pre=pre,
                                                                     d_amax_g=amax, act=fp8lin.ACT_GELU)))
            if N % 64 == 0 and K % 32 == 0:
                zs = torch.empty((M, N // 2), dtype=torch.uint8, device="cuda")
                gs = torch.empty((M, 2 * K), dtype=torch.uint8, device="cuda")
                pre2 = torch.randn((M, 2 * K), device="cuda").to(torch.bfloat16)
                runs += (("swiglu->fp8", lambda: ctx.linear_fwd_q(a, bias, b, bias, zs, bias, y_pre=y, d_amax_z=amax,
                                                                  act=fp8lin.ACT_SWIGLU)),
                         ("dgrad swiglu'->fp8", lambda: ctx.linear_dgrad_q(dy, bias, b, None, bias, gs, bias, y_pre=pre2,
                                                                           d_amax_g=amax, act=fp8lin.ACT_SWIGLU)))
            for name, fn in runs:
                t = _time_burst(fn, iters)
                line += f" | {name} {2.0 * M * N * K / t / 1e9:7.1f} TF {t * 1e3:7.1f} us"
        print(line, flush=True)


def leg_cast(ctx, fp8lin, shapes, iters=10):
    """amax, cast, cast + transposed copy and amax+bias+cast of bf16 [rows x cols]; 512 MB written between timings."""
    flush = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")
    for rows, cols in shapes:
        x = torch.randn(rows, cols, device="cuda").to(torch.bfloat16)
        n = rows * cols
        amax = torch.zeros(1, dtype=torch.float32, device="cuda")
        bias = torch.zeros(1, dtype=torch.int32, device="cuda")
        y = torch.empty((rows, cols), dtype=torch.uint8, device="cuda")
        yt = torch.empty((cols, rows), dtype=torch.uint8, device="cuda")
        ctx.amax(x, amax)
        ctx.scaling_bias(amax, fp8lin.E4, fp8lin.CONV_PAPER, 0, bias)
        fl = flush.zero_
        t_amax = _time_each(lambda: ctx.amax(x, amax), iters, fl)
        t_flat = _time_each(lambda: ctx.cast_e4(x, bias, y=y), iters, fl)
        t_both = _time_each(lambda: ctx.cast_e4(x, bias, y=y, y_t=yt), iters, fl)
        t_fused = _time_each(lambda: ctx.cast_e4(x, None, d_amax_out=amax, d_bias_out=bias, y=y), iters, fl)
        t_pred = _time_each(lambda: ctx.cast_predicted(fp8lin.E4, x, amax, bias, y), iters, fl)
        print(f"cast {rows}x{cols} ({2 * n / 1e6:.0f} MB): amax {t_amax * 1e3:6.1f} us ({2 * n / t_amax / 1e9:5.2f} TB/s)"
              f" | cast {t_flat * 1e3:6.1f} us ({3 * n / t_flat / 1e9:5.2f} TB/s)"
              f" | cast+transposed copy {t_both * 1e3:6.1f} us ({4 * n / t_both / 1e9:5.2f} TB/s)"
              f" | amax+bias+cast {t_fused * 1e3:6.1f} us ({3 * n / t_fused / 1e9:5.2f} TB/s on 3 B/element)"
              f" | one pass, guess held {t_pred * 1e3:6.1f} us ({3 * n / t_pred / 1e9:5.2f} TB/s)", flush=True)


def leg_stack(ctx, fp8lin, shapes, steps=40, warmup=8, only=None, graph=True, quiet=False):
    """ms per SGD step of the stack of FP8 linears (torch glue included): every tensor scaled just in time with
    separate activation kernels; activation and amax fused into the matmul epilogues; amax-history scaling with
    the FP8 bytes written by the epilogues."""
    from paper_2309_17224_b200 import stack as S
    say = (lambda *a, **k: None) if quiet else print
    results = []
    for layers, d, tokens in shapes:
        kw = dict(layers=layers, d=d, tokens=tokens)
        variants = (("just in time", lambda: S.Fp8Stack(ctx, **kw)),
                    ("fused epilogues", lambda: S.Fp8Stack(ctx, fused_activation=True, **kw)),
                    ("amax history", lambda: S.Fp8StackHistory(ctx, margin=1, **kw)))
        for name, make in variants:
            if only and only not in name:
                continue
            st = make()
            for i in range(warmup):
                st.step(i)
            torch.cuda.synchronize()
            s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            s.record()
            for i in range(warmup, warmup + steps):
                r = st.step(i)
            e.record()
            torch.cuda.synchronize()
            ms = s.elapsed_time(e) / steps
            rec = {"layers": layers, "d": d, "tokens": tokens, "variant": name, "ms_per_step": ms,
                   "tflops": st.flops_per_step() / ms / 1e9, "loss": float(r["loss"].item())}
            if graph:
                # the same step replayed from a CUDA graph: device time without the host's launch overhead
                g = torch.cuda.CUDAGraph()
                side = torch.cuda.Stream()
                side.wait_stream(torch.cuda.current_stream())
                with torch.cuda.stream(side):
                    st.step(warmup + steps)
                    with torch.cuda.graph(g, stream=side):
                        st.step(warmup + steps)
                torch.cuda.current_stream().wait_stream(side)
                g.replay()
                torch.cuda.synchronize()
                s.record()
                for _ in range(steps):
                    g.replay()
                e.record()
                torch.cuda.synchronize()
                rec["graph_ms_per_step"] = s.elapsed_time(e) / steps
                rec["graph_tflops"] = st.flops_per_step() / rec["graph_ms_per_step"] / 1e9
                del g
            say(f"stack {layers}x{d}x{tokens} {name:16s}: {ms:7.3f} ms/step  {rec['tflops']:7.1f} TFLOP/s"
                + (f" | from a CUDA graph {rec['graph_ms_per_step']:7.3f} ms/step  {rec['graph_tflops']:7.1f} TFLOP/s"
                   if graph else "") + f" | loss {rec['loss']:.5f}", flush=True)
            results.append(rec)
            del st
    return results


def leg_mlp(ctx, fp8lin, shapes, iters=20, quiet=False):
    """A gated MLP (x -> SiLU(x Wg^T) * (x Wu^T) -> . Wd^T), every linear in FP8: (a) each linear quantises its
    input just in time and the gated unit is separate torch kernels; (b) the gate_up matmul's epilogue computes the
    gated unit and writes the down projection's FP8 input under a bias carried over from the previous call
    (amax-history scaling).  Weights are quantised once, outside the timed region, in both variants."""
    results = []
    say = (lambda *a, **k: None) if quiet else print
    for T, d, F in shapes:
        dev = dict(device="cuda")
        x = torch.randn(T, d, **dev).to(torch.bfloat16)
        wg, wu = (torch.randn(F, d, **dev) * 0.02).to(torch.bfloat16), (torch.randn(F, d, **dev) * 0.02).to(torch.bfloat16)
        wd = (torch.randn(d, F, **dev) * 0.02).to(torch.bfloat16)
        w_gu = torch.cat((wg, wu), 0).contiguous()           # unfused: gate rows then up rows
        w_il = I.interleave32(wg, wu).contiguous()           # fused: blocks of 32 gate rows, 32 up rows
        sc_f = torch.zeros(8, dtype=torch.float32, **dev)
        sc_i = torch.zeros(8, dtype=torch.int32, **dev)
        u8 = dict(dtype=torch.uint8, **dev)
        w_gu8, w_il8, wd8 = torch.empty((2 * F, d), **u8), torch.empty((2 * F, d), **u8), torch.empty((d, F), **u8)
        ctx.ptq_weights(w_gu, fp8lin.CONV_PAPER, w_gu8, None, sc_i[0:1], sc_f[0:1])
        ctx.ptq_weights(w_il, fp8lin.CONV_PAPER, w_il8, None, sc_i[1:2], sc_f[1:2])
        ctx.ptq_weights(wd, fp8lin.CONV_PAPER, wd8, None, sc_i[2:3], sc_f[2:3])
        x8, z8 = torch.empty((T, d), **u8), torch.empty((T, F), **u8)
        h = torch.empty((T, 2 * F), dtype=torch.bfloat16, **dev)
        out = torch.empty((T, d), dtype=torch.bfloat16, **dev)

        def unfused():
            ctx.cast_e4(x, None, d_amax_out=sc_f[3:4], d_bias_out=sc_i[3:4], y=x8)
            ctx.linear_fwd(x8, sc_i[3:4], w_gu8, sc_i[0:1], h)
            z = (torch.nn.functional.silu(h[:, :F].float()) * h[:, F:].float()).to(torch.bfloat16)
            ctx.cast_e4(z, None, d_amax_out=sc_f[4:5], d_bias_out=sc_i[4:5], y=z8)
            ctx.linear_fwd(z8, sc_i[4:5], wd8, sc_i[2:3], out)

        def fused():
            ctx.cast_e4(x, None, d_amax_out=sc_f[3:4], d_bias_out=sc_i[3:4], y=x8)
            ctx.linear_fwd_q(x8, sc_i[3:4], w_il8, sc_i[1:2], z8, sc_i[5:6], d_amax_z=sc_f[5:6], act=fp8lin.ACT_SWIGLU)
            ctx.linear_fwd(z8, sc_i[5:6], wd8, sc_i[2:3], out)
            ctx.scaling_bias(sc_f[5:6], fp8lin.E4, fp8lin.CONV_PAPER, 1, sc_i[5:6])   # next call's bias, margin 1

        unfused()
        sc_i[5:6].copy_(sc_i[4:5] - 1)                       # history for the first fused call
        res = {name: _time_burst(fn, iters) for name, fn in (("unfused", unfused), ("SwiGLU epilogue", fused))}
        flops = 2.0 * T * d * 3 * F
        say(f"mlp T={T} d={d} ffn={F} forward: " + " | ".join(f"{k} {v:7.3f} ms {flops / v / 1e9:7.1f} TFLOP/s" for k, v in res.items()),
            flush=True)
        results.append({"tokens": T, "d": d, "ffn": F, "pass": "fwd", "unfused_ms": res["unfused"],
                        "fused_ms": res["SwiGLU epilogue"], "fused_tflops": flops / res["SwiGLU epilogue"] / 1e9})
        if T < 256:
            continue
        # ---- forward + backward of the same block (training step without the optimiser) ----
        dy = (torch.randn(T, d, **dev) * 1e-3).to(torch.bfloat16)
        dy8, g8 = torch.empty((T, d), **u8), torch.empty((T, 2 * F), **u8)
        dz = torch.empty((T, F), dtype=torch.bfloat16, **dev)
        dx = torch.empty((T, d), dtype=torch.bfloat16, **dev)
        dw_gu = torch.empty((2 * F, d), dtype=torch.bfloat16, **dev)
        dw_d = torch.empty((d, F), dtype=torch.bfloat16, **dev)
        h_il = torch.empty((T, 2 * F), dtype=torch.bfloat16, **dev)

        def unfused_step():
            unfused()
            ctx.cast_e5(dy, None, d_amax_out=sc_f[6:7], d_bias_out=sc_i[6:7], y=dy8)
            ctx.linear_dgrad(dy8, sc_i[6:7], wd8, None, sc_i[2:3], dz)
            ctx.linear_wgrad(dy8, None, sc_i[6:7], z8, None, sc_i[4:5], dw_d, T)
            a, u_ = h[:, :F].float(), h[:, F:].float()
            sg = torch.sigmoid(a)
            g = torch.cat(((dz.float() * u_ * (sg + a * sg * (1 - sg))), (dz.float() * a * sg)), 1).to(torch.bfloat16)
            ctx.cast_e5(g, None, d_amax_out=sc_f[7:8], d_bias_out=sc_i[7:8], y=g8)
            ctx.linear_dgrad(g8, sc_i[7:8], w_gu8, None, sc_i[0:1], dx)
            ctx.linear_wgrad(g8, None, sc_i[7:8], x8, None, sc_i[3:4], dw_gu, T)

        gb = torch.zeros(2, dtype=torch.int32, **dev)      # history bias of the gate/up gradient, and its next value
        ga = torch.zeros(1, dtype=torch.float32, **dev)

        def fused_step():
            ctx.cast_e4(x, None, d_amax_out=sc_f[3:4], d_bias_out=sc_i[3:4], y=x8)
            ctx.linear_fwd_q(x8, sc_i[3:4], w_il8, sc_i[1:2], z8, sc_i[5:6], y_pre=h_il, d_amax_z=sc_f[5:6],
                             act=fp8lin.ACT_SWIGLU)
            ctx.linear_fwd(z8, sc_i[5:6], wd8, sc_i[2:3], out)
            ctx.cast_e5(dy, None, d_amax_out=sc_f[6:7], d_bias_out=sc_i[6:7], y=dy8)
            ctx.linear_dgrad_q(dy8, sc_i[6:7], wd8, None, sc_i[2:3], g8, gb[0:1], y_pre=h_il, d_amax_g=ga,
                               act=fp8lin.ACT_SWIGLU)
            ctx.linear_wgrad(dy8, None, sc_i[6:7], z8, None, sc_i[5:6], dw_d, T)
            ctx.linear_dgrad(g8, gb[0:1], w_il8, None, sc_i[1:2], dx)
            ctx.linear_wgrad(g8, None, gb[0:1], x8, None, sc_i[3:4], dw_gu, T)
            ctx.scaling_bias(sc_f[5:6], fp8lin.E4, fp8lin.CONV_PAPER, 1, sc_i[5:6])
            ctx.scaling_bias(ga, fp8lin.E5, fp8lin.CONV_PAPER, 1, gb[0:1])

        unfused_step()
        gb[0:1].copy_(sc_i[7:8] - 1)
        res = {name: _time_burst(fn, iters) for name, fn in (("unfused", unfused_step), ("SwiGLU epilogues", fused_step))}
        flops *= 3
        say(f"mlp T={T} d={d} ffn={F} forward + backward: "
            + " | ".join(f"{k} {v:7.3f} ms {flops / v / 1e9:7.1f} TFLOP/s" for k, v in res.items()), flush=True)
        results.append({"tokens": T, "d": d, "ffn": F, "pass": "fwd+bwd", "unfused_ms": res["unfused"],
                        "fused_ms": res["SwiGLU epilogues"], "fused_tflops": flops / res["SwiGLU epilogues"] / 1e9})
    return results


def leg_group(ctx, fp8lin, wl, reps=3):
    """fp8_cast_group over every tensor a step of the workload quantises, one launch pair at a time: the amax pass,
    the cast pass, the one-pass mode (every guess holds) and the two-pass mode."""
    layers = [LayerState(wl, li, "cuda", I.BASE_SEED, wl.backward) for li in range(len(wl.layers))]
    tensors = [it for L in layers for it in L.quant_items()]
    items = fp8lin.group_items(tensors)
    elems = sum(t[1].numel() for t in tensors)
    ctx.cast_group(items)
    line = f"group {wl.name}: {len(tensors)} tensors, {elems / 1e6:.0f} M elements:"
    for name, bpe, mode in (("amax pass", 2, fp8lin.GROUP_AMAX_ONLY), ("cast pass", 3, fp8lin.GROUP_CAST_ONLY),
                            ("one pass", 3, fp8lin.GROUP_PREDICTED), ("two passes", 5, fp8lin.GROUP_AMAX_CAST)):
        ms = []
        for r in range(reps + 1):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda._sleep(200000)
            a.record()
            ctx.cast_group(items, mode=mode)
            b.record()
            torch.cuda.synchronize()
            if r:
                ms.append(a.elapsed_time(b))
        t = sum(ms) / len(ms)
        line += f" | {name} {t * 1e3:6.1f} us {elems * bpe / t / 1e6:6.0f} GB/s on {bpe} B/element"
    print(line, flush=True)


def run_leg(args):
    from paper_2309_17224_b200 import build as B
    B.build()
    from paper_2309_17224_b200 import fp8lin
    shapes = [tuple(int(v) for v in a.split("x")) for a in args.shapes]
    if not shapes and args.leg != "group":
        print(__doc__)
        return 2
    torch.cuda.set_device(0)
    ctx = fp8lin.Context(0)
    if args.leg == "group":
        leg_group(ctx, fp8lin, I.WORKLOADS[args.workload])
    elif args.leg == "gemm":
        leg_gemm(ctx, fp8lin, shapes, fused=not args.plain_only)
    elif args.leg == "cast":
        leg_cast(ctx, fp8lin, shapes)
    elif args.leg == "mlp":
        leg_mlp(ctx, fp8lin, shapes)
    else:
        leg_stack(ctx, fp8lin, shapes, steps=args.steps, warmup=max(2, args.warmup), only=args.only, graph=not args.no_graph_leg)
    flags = ctx.device_flags()
    if flags & fp8lin.FLAG_TIMEOUT:
        print("a device-side wait expired", file=sys.stderr)
        return 3
    return 0


# ----------------------------------------------------------------------------
# the step benchmark
# ----------------------------------------------------------------------------

def workload_summary(ctx, fp8lin, wl_name, tokens, device, seed, peaks, steps=20):
    """One short line for a workload other than the headline's: eager step time and the same step replayed from a
    CUDA graph, default quantisation mode; decode-size batches add the weight-streaming rate of the whole block."""
    wl = I.WORKLOADS[wl_name]
    T = tokens or wl.tokens
    layers = [LayerState(wl, li, device, seed, wl.backward, T) for li in range(len(wl.layers))]
    if not wl.backward:
        for L in layers:
            ctx.ptq_weights(L.w, fp8lin.CONV_PAPER, L.w8, None, L.scal_i[0:1], L.scal_f[0:1])
            L.w = None   # the 16-bit weights are needed at load only
        torch.cuda.empty_cache()
    st = Step(ctx, fp8lin, layers, "group-predicted", T)
    for _ in range(3):
        st.run()
    eager = timed_loop(st.run, steps, None, device)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        st.run()
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        st.run()
    for _ in range(3):
        graph.replay()
    graphed = timed_loop(graph.replay, steps, None, device)
    flops = sum(L.gemm_flops() for L in layers)
    rec = {"workload": wl_name, "tokens": T, "passes": "fwd+bwd" if wl.backward else "fwd", "quantisation": st.mode,
           "ms_per_step": eager, "tflops": flops / eager / 1e9, "graph_ms_per_step": graphed,
           "graph_tflops": flops / graphed / 1e9, "launches_per_step": st.launches_per_step()}
    if T <= 128:
        wbytes = float(sum(L.N * L.K for L in layers))
        rec["weight_stream_gbs_whole_block"] = wbytes / (graphed * 1e-3) / 1e9
        rec["frac_of_hbm_peak"] = rec["weight_stream_gbs_whole_block"] / peaks["hbm_gbs"]
    del graph, st, layers
    torch.cuda.empty_cache()
    return rec


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(I.WORKLOADS))
    ap.add_argument("--tokens", type=int, default=0, help="override the workload's token count (c4: 1, 16, 64, 2048)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--quant", default="group-predicted", choices=QUANT_MODES,
                    help="how the step quantises its tensors (see class Step)")
    ap.add_argument("--matmuls", default="group", choices=("group", "per-call"),
                    help="all matmuls of a step in one fp8_linear_group call, or one call each")
    ap.add_argument("--transposed-copies", action="store_true",
                    help="also write transposed FP8 copies and contract the backward matmuls over contiguous bytes "
                         "(per-tensor quantisation)")
    ap.add_argument("--no-fused-decode", action="store_true",
                    help="forward-only layers on at most 128 rows as fp8_cast_e4 + fp8_linear_infer instead of fp8_linear_infer_cast")
    ap.add_argument("--no-graph-leg", action="store_true", help="skip the extra timed loop that replays a CUDA graph")
    ap.add_argument("--no-extra-legs", action="store_true",
                    help="skip every leg beside the headline: other quantisation modes, moving gradients, sustained "
                         "run, tensor-pipe ceiling, fused MLP, other workloads")
    ap.add_argument("--no-ceiling-leg", action="store_true", help="skip the tensor-pipe ceiling measurement")
    ap.add_argument("--sustain-seconds", type=float, default=3.0)
    ap.add_argument("--e2e-steps", type=int, default=20)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--leg", default="step", choices=["step", "gemm", "cast", "stack", "mlp", "group"])
    ap.add_argument("--shapes", nargs="*", default=[])
    ap.add_argument("--only", default=None, help="--leg stack: run only the variant whose name contains this")
    ap.add_argument("--plain-only", action="store_true", help="--leg gemm: skip the fused epilogues")
    args = ap.parse_args()
    global NO_FUSED_DECODE
    NO_FUSED_DECODE = args.no_fused_decode
    wl = I.WORKLOADS[args.workload]
    if args.impl == "reference":
        return reference_arm(args, wl)

    if not torch.cuda.is_available():
        print("bench.py: no CUDA device; the FP8 path has no CPU fallback", file=sys.stderr)
        return 2
    if args.leg != "step":
        return run_leg(args)
    from paper_2309_17224_b200 import build as B
    B.build()
    from paper_2309_17224_b200 import fp8lin

    rank, world, local, dist = dist_setup(args.gpus)
    device = torch.device("cuda", local)
    warmup = max(3, args.warmup)
    ctx = fp8lin.Context(local)
    seed = I.BASE_SEED + 7919 * rank
    quant = "per-tensor" if args.transposed_copies else args.quant
    layers = [LayerState(wl, li, device, seed, wl.backward, args.tokens, args.transposed_copies)
              for li in range(len(wl.layers))]
    peaks = load_peaks()
    tokens = args.tokens or wl.tokens
    if not wl.backward:  # post-training quantisation, once, outside the timed region
        for L in layers:
            ctx.ptq_weights(L.w, fp8lin.CONV_PAPER, L.w8, None, L.scal_i[0:1], L.scal_f[0:1])
    step = Step(ctx, fp8lin, layers, quant, tokens, args.matmuls)
    step_matmuls = step.matmuls

    ctx.prediction_stats(clear=True)
    for _ in range(warmup):
        step.run()
    barrier_sync(dist)
    if ctx.device_flags(clear=True) & fp8lin.FLAG_TIMEOUT:
        print("bench.py: a device-side wait expired during warm-up", file=sys.stderr)
        return 3
    ctx.prediction_stats(clear=True)

    # ---- timed region: K steps, device time, max over ranks ----
    sampler = ClockSampler(local) if rank == 0 else None
    timers = Timers()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier_sync(dist)
    launches_before = fp8lin.launch_count()
    start.record()
    for i in range(args.steps):
        # per-kernel event pairs on every eighth step only: they serialise the launches they bracket
        step.run(timers if i % EVENT_EVERY == 0 else None)
    stop.record()
    launches_timed = fp8lin.launch_count() - launches_before   # the library's own count of what it enqueued
    barrier_sync(dist)
    clocks = sampler.stop() if sampler else None
    total_ms = max_over_ranks(start.elapsed_time(stop), dist, device)
    flags = ctx.device_flags(clear=True)
    if flags & fp8lin.FLAG_TIMEOUT:
        print("bench.py: a device-side wait expired during the timed region", file=sys.stderr)
        return 3
    guesses = ctx.prediction_stats(clear=True)

    ms_per_step = total_ms / args.steps
    step_flops = sum(L.gemm_flops() for L in layers)
    value = whole_job_value(world, step_flops, ms_per_step)

    sampled_steps = (args.steps + EVENT_EVERY - 1) // EVENT_EVERY     # steps that carried per-kernel events
    gemm_ms = timers.total_ms("gemm")
    gemm_launches = timers.count("gemm")
    gemm_tflops = sampled_steps * step_flops / (gemm_ms * 1e-3) / 1e12
    cast_ms = timers.total_ms("amax_cast")
    cast_elems = sampled_steps * sum(L.cast_elements() for L in layers)
    bytes_per_elem = 4 if (wl.backward and args.transposed_copies) else 3  # read once, write one byte per layout
    # the denominator that matches the run: the burst figure when the SM clock held its maximum over the timed
    # region (a short run, not yet power-capped), the sustained one otherwise
    held_max = bool(clocks and clocks.get("sm_mhz") and clocks["sm_mhz"] >= 0.95 * clocks["sm_max_mhz"])
    peak_kind = "burst" if held_max else "sustained"
    fp8_peak = 2.0 * (peaks["bf16_tflops"] if held_max else peaks["bf16_tflops_sustained"])
    decode = tokens <= 128   # one tile row: the matmuls stream the weights, the bound is HBM
    weight_bytes = float(sum(l.K * l.N for l in wl.layers))
    sm_count = torch.cuda.get_device_properties(local).multi_processor_count
    if decode:
        # fp8_linear_infer_cast quantises an activation of at most 64 KB inside the matmul launch, larger ones by a cast launch
        in_launch = fused_decode(layers[0]) and all(L.T * L.K * 2 <= (64 << 10) for L in layers)
        roofline = {"bound": "hbm", "kernel": "decode_kernel (activation quantised in the same launch)" if in_launch
                    else "decode_kernel (+ splitk_finalize_kernel where the contraction is split through the workspace; the "
                         "activation's cast is a launch of its own)",
                    "achieved": sampled_steps * weight_bytes / (gemm_ms * 1e-3) / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "peak_source": f"{peaks['source']} copy bandwidth", "launches": gemm_launches,
                    "avg_launch_ms": gemm_ms / max(1, gemm_launches),
                    "algorithmic_bytes_per_launch": weight_bytes / max(1, gemm_launches / sampled_steps),
                    "timed_on": f"every {EVENT_EVERY}th step of the timed region ({sampled_steps} steps)", "traffic": None}
    else:
        roofline = {"bound": "tensor",
                    "kernel": "gemm_pair_group_kernel (all matmuls of the step in one launch)" if step.matmuls == "group"
                    else "gemm_pair_kernel", "achieved": gemm_tflops, "peak": fp8_peak,
                    "unit": "TFLOP/s",
                    "peak_source": f"2 x {peaks['source']} {peak_kind} bf16 cuBLAS "
                                   f"({peaks['bf16_tflops' if held_max else 'bf16_tflops_sustained']} TFLOP/s); "
                                   f"median SM clock {clocks['sm_mhz'] if clocks else None} MHz over the timed region",
                    "launches": gemm_launches, "avg_launch_ms": gemm_ms / max(1, gemm_launches),
                    "algorithmic_bytes_per_launch": sum(L.gemm_bytes() for L in layers) / max(1, gemm_launches / sampled_steps),
                    "timed_on": f"every {EVENT_EVERY}th step of the timed region ({sampled_steps} steps)",
                    "traffic": GEMM_DRAM_BYTES_PER_LAUNCH.get((wl.name, tokens, step.matmuls))}
    roofline["frac"] = roofline["achieved"] / roofline["peak"]
    if not decode:
        # the same achieved rate against the two other denominators in use: the vendor's dense-FP8 figure (what the
        # 70 % target of the benchmark spec refers to) and that figure's per-clock rate at the clock sampled here
        roofline["frac_of_nominal_4500"] = gemm_tflops / NOMINAL_FP8_TFLOPS
        if clocks and clocks.get("sm_mhz"):
            at_clock = sm_count * FP8_FLOP_PER_CLK_PER_SM * clocks["sm_mhz"] * 1e6 / 1e12
            roofline["nominal_rate_at_sampled_clock"] = at_clock
            roofline["frac_of_nominal_rate_at_sampled_clock"] = gemm_tflops / at_clock
        roofline["targets"] = ("task statement: matmuls >= 0.70 of dense-FP8 tensor peak (frac_of_nominal_4500), amax and "
                               "cast >= 0.80 of HBM peak (amax_cast.per_kernel.*.frac); frac is against 2 x the cuBLAS "
                               "bf16 rate measured on this pool")

    # ---- what the matmul kernel reaches when moving operands costs nothing ----
    ceiling = None
    if not args.no_ceiling_leg and not decode and rank == 0:
        try:
            big = max(layers, key=lambda L: L.T * L.N * L.K)
            zero = torch.zeros(1, dtype=torch.int32, device=device)
            c_sampler = ClockSampler(local)
            shapes = {"long_k": (8192, 8192, 16384), "largest_layer_fwd": (big.T, big.N, big.K)}
            ceiling = {"how": "fp8_selftest_mma_ceiling: gemm_pair_kernel with its operand loads off (barriers, MMAs, "
                              "epilogue and stores as usual), 10 launches back to back right after the timed region, beside "
                              "the same shape with loads; when the power cap already holds the clock down the two meet: "
                              "the limit is then the power of the tensor pipe, not the operand feed"}
            for name, (M, N, K) in shapes.items():
                out = torch.empty((M, N), dtype=torch.bfloat16, device=device)
                a8 = torch.randint(0, 0x78, (M, K), dtype=torch.uint8, device=device)
                b8 = torch.randint(0, 0x78, (N, K), dtype=torch.uint8, device=device)
                t_off = _time_burst(lambda: ctx.selftest_mma_ceiling(out, zero, K), 10, warm=2)
                t_on = _time_burst(lambda: ctx.linear_fwd(a8, zero, b8, zero, out), 10, warm=2)
                ceiling[name] = {"shape_mnk": [M, N, K], "loads_off_tflops": 2.0 * M * N * K / t_off / 1e9,
                                 "with_loads_tflops": 2.0 * M * N * K / t_on / 1e9}
                try:   # context only: the vendor library's FP8 matmul on the same operands, same moment, same clock
                    one = torch.ones((), dtype=torch.float32, device=device)
                    af, bf = a8.view(torch.float8_e4m3fn), b8.view(torch.float8_e4m3fn).t()
                    t_lib = _time_burst(lambda: torch._scaled_mm(af, bf, scale_a=one, scale_b=one, out_dtype=torch.bfloat16),
                                        10, warm=2)
                    ceiling[name]["library_fp8_matmul_tflops"] = 2.0 * M * N * K / t_lib / 1e9
                except Exception:
                    pass
                del out, a8, b8
            ceiling["clocks"] = c_sampler.stop()
            roofline["ceiling"] = ceiling
        except Exception as exc:
            roofline["ceiling"] = {"error": str(exc)[:200]}
            torch.cuda.synchronize()

    extra = not args.no_extra_legs
    # ---- the quantisation kernels, each against its own algorithmic bytes (outside the timed region) ----
    per_kernel = quantisation_kernel_bandwidths(ctx, fp8lin, layers, peaks["hbm_gbs"])

    # ---- the same step under the other quantisation modes (same per-kernel event schedule as the headline) ----
    other_modes = {}
    layer_ms = timers.layer_ms()   # empty when the step's matmuls are one call; then taken from the per-call leg
    if extra and not decode and not args.transposed_copies:
        def time_variant(st):
            for _ in range(3):
                st.run()
            ctx.prediction_stats(clear=True)
            m_steps = min(args.steps, 100)
            tm = Timers()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            barrier_sync(dist)
            a.record()
            for i in range(m_steps):
                st.run(tm if i % EVENT_EVERY == 0 else None)
            b.record()
            barrier_sync(dist)
            m_ms = max_over_ranks(a.elapsed_time(b), dist, device) / m_steps
            m_sampled = (m_steps + EVENT_EVERY - 1) // EVENT_EVERY
            out = {"value": whole_job_value(world, step_flops, m_ms), "unit": UNIT, "ms_per_step": m_ms,
                   "steps": m_steps, "amax_cast_ms_per_step": tm.total_ms("amax_cast") / m_sampled,
                   "gemm_ms_per_step": tm.total_ms("gemm") / m_sampled, "matmuls": st.matmuls,
                   "launches_per_step": st.launches_per_step()}
            if "predicted" in st.mode:
                out["guesses_held_missed"] = list(ctx.prediction_stats(clear=True))
            return out, tm

        if step.matmuls == "group":   # the headline's quantisation with one call per matmul: what the one launch buys
            other_modes["per-call matmuls"], tm_calls = time_variant(Step(ctx, fp8lin, layers, step.mode, tokens, "per-call"))
            layer_ms = tm_calls.layer_ms()
        for mode in QUANT_MODES:
            if mode == step.mode:
                continue
            other_modes[mode], _ = time_variant(Step(ctx, fp8lin, layers, mode, tokens, args.matmuls))

    # ---- gradients whose magnitude moves every step: what a wrong guess costs ----
    moving = None
    if extra and wl.backward and step.items is not None and step.mode == "group-predicted":
        g_keep = [L.g.clone() for L in layers]
        ctx.prediction_stats(clear=True)
        m_steps = min(args.steps, 40)
        tm = Timers()

        def moving_step(i, timers=None):
            for L, g0 in zip(layers, g_keep):      # dY <- seeded dY x 2^(i mod 3): exact, and the E5 bias moves by one or two
                torch.mul(g0, float(2 ** (i % 3)), out=L.g)
            step.run(timers)

        for i in range(3):
            moving_step(i)
        ctx.prediction_stats(clear=True)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier_sync(dist)
        a.record()
        for i in range(m_steps):
            moving_step(i + 3, tm if i % EVENT_EVERY == 0 else None)
        b.record()
        barrier_sync(dist)
        mv_ms = max_over_ranks(a.elapsed_time(b), dist, device) / m_steps
        held, missed = ctx.prediction_stats(clear=True)
        m_sampled = (m_steps + EVENT_EVERY - 1) // EVENT_EVERY
        moving = {"ms_per_step": mv_ms, "steps": m_steps, "guesses_held": held, "guesses_missed": missed,
                  "amax_cast_ms_per_step": tm.total_ms("amax_cast") / m_sampled,
                  "note": "every step each layer's dY is the seeded tensor times 2^(step mod 3), rewritten by a torch "
                          "kernel inside the loop (its time is in ms_per_step, not in amax_cast_ms_per_step): the four "
                          "gradient guesses miss every step and those tensors are cast twice; results stay identical "
                          "to the just-in-time path"}
        for L, g0 in zip(layers, g_keep):
            L.g.copy_(g0)
        del g_keep
        step.run()   # leave the bias words at the repeated tensors' values again

    # ---- the same step captured once in a CUDA graph and replayed (launch gaps removed) ----
    graphed = None
    if not args.no_graph_leg:
        try:
            g_steps = min(args.steps, 100)
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):          # warm-up on the capture stream, as torch requires
                step.run()
            torch.cuda.current_stream().wait_stream(side)
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                step.run()
            for _ in range(3):
                graph.replay()
            g_ms = timed_loop(graph.replay, g_steps, dist, device)
            graphed = {"value": whole_job_value(world, step_flops, g_ms), "unit": UNIT, "ms_per_step": g_ms,
                       "steps": g_steps, "launches_per_graph": step.launches_per_step()}
            del graph
        except Exception as exc:  # capture is an extra leg; the headline never depends on it
            graphed = {"error": str(exc)[:200]}
            torch.cuda.synchronize()

    # ---- the same loop for seconds: the clock settles under the power cap ----
    sustained = None
    if extra and args.sustain_seconds > 0:
        n = max(args.steps, int(args.sustain_seconds * 1e3 / ms_per_step) + 1)
        s_sampler = ClockSampler(local) if rank == 0 else None
        s_timers, s_i = Timers(), [0]

        def s_run():   # per-kernel event pairs on every 32nd step, in the second half of the run (clock settled)
            s_i[0] += 1
            step.run(s_timers if (s_i[0] % 32 == 0 and s_i[0] > n // 2) else None)

        s_ms = timed_loop(s_run, n, dist, device)
        s_clocks = s_sampler.stop() if s_sampler else None
        sustained = {"value": whole_job_value(world, step_flops, s_ms), "unit": UNIT, "ms_per_step": s_ms, "steps": n,
                     "seconds": s_ms * n * 1e-3, "clocks": s_clocks}
        if s_timers.count("gemm") > 0:
            s_steps = s_timers.count("amax_cast") if s_timers.count("amax_cast") > 0 else s_timers.count("gemm")
            s_gemm_ms = s_timers.total_ms("gemm") / s_steps
            sustained["gemm_ms_per_step"] = s_gemm_ms
            sustained["gemm_tflops"] = step_flops / (s_gemm_ms * 1e-3) / 1e12
            sustained["gemm_frac_of_2x_sustained_bf16"] = sustained["gemm_tflops"] / (2.0 * peaks["bf16_tflops_sustained"])
            if s_timers.count("amax_cast") > 0:
                sustained["amax_cast_ms_per_step"] = s_timers.total_ms("amax_cast") / s_steps
        if s_clocks and s_clocks.get("sm_mhz"):
            sustained["ms_times_sm_ghz"] = s_ms * s_clocks["sm_mhz"] * 1e-3
            sustained["frac_of_2x_sustained_bf16"] = sustained["value"] / world / (2.0 * peaks["bf16_tflops_sustained"])
            sustained["note"] = ("whole step (quantisation included) against 2 x the sustained cuBLAS bf16 rate, and the matmul "
                                 "launches alone (events on every 32nd step of the second half) against the same; "
                                 "ms_times_sm_ghz compares runs at different clocks")

    # ---- the gated MLP of the same model as one chained block, unfused against the fused epilogues ----
    fused_mlp = None
    if extra and wl.name == "c3_llama7b":
        gate_up = next(l for l in wl.layers if l.name == "gate_up")
        r = leg_mlp(ctx, fp8lin, [(tokens, gate_up.K, gate_up.N // 2)], iters=10, quiet=True)[-1]
        fused_mlp = {"block": f"x[{tokens},{gate_up.K}] -> SiLU(x Wg^T) * (x Wu^T) -> . Wd^T, forward + backward, all six matmuls "
                              "in FP8, every quantisation included",
                     "unfused_ms": r["unfused_ms"], "fused_ms": r["fused_ms"], "fused_tflops": r["fused_tflops"],
                     "how": "unfused: just-in-time amax + cast per tensor, gated unit and its backward as torch kernels; fused: "
                            "fp8_linear_fwd_q / fp8_linear_dgrad_q with the SwiGLU epilogues, amax-history biases (margin 1)"}

    # ---- end to end through the public API with host buffers ----
    e2e = None
    if args.e2e_steps > 0:
        host_in, host_out = [], []
        for L in layers:
            ins = [L.x] + ([L.w, L.g] if wl.backward else [])
            outs = [L.y] + ([L.dx, L.dw] if wl.backward else [])
            host_in.append([torch.empty(t.shape, dtype=t.dtype, pin_memory=True).copy_(t) for t in ins])
            host_out.append([torch.empty(t.shape, dtype=t.dtype, pin_memory=True) for t in outs])
        h2d = sum(t.numel() * t.element_size() for ts in host_in for t in ts)
        d2h = sum(t.numel() * t.element_size() for ts in host_out for t in ts)

        # three streams: host->device copies, compute, device->host copies; per layer the copy of its inputs,
        # its kernels and the copy of its results are ordered by events, so the copies of one layer overlap the
        # kernels of another (what a user of the API would do with pinned buffers)
        s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
        s_comp = torch.cuda.current_stream()
        ev_comp = [None] * len(layers)   # kernels of layer i done (its inputs may be overwritten, its outputs read)
        ev_out = [None] * len(layers)    # results of layer i copied out (its outputs may be overwritten)

        def e2e_step():
            for i, (L, hin, hout) in enumerate(zip(layers, host_in, host_out)):
                ins = [L.x] + ([L.w, L.g] if wl.backward else [])
                outs = [L.y] + ([L.dx, L.dw] if wl.backward else [])
                with torch.cuda.stream(s_in):
                    if ev_comp[i] is not None:
                        s_in.wait_event(ev_comp[i])
                    for d, h in zip(ins, hin):
                        d.copy_(h, non_blocking=True)
                    ev_in = torch.cuda.Event()
                    ev_in.record(s_in)
                s_comp.wait_event(ev_in)
                if ev_out[i] is not None:
                    s_comp.wait_event(ev_out[i])
                run_layer(ctx, L, predict=True)
                ev_comp[i] = torch.cuda.Event()
                ev_comp[i].record(s_comp)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(ev_comp[i])
                    for h, d in zip(hout, outs):
                        h.copy_(d, non_blocking=True)
                    ev_out[i] = torch.cuda.Event()
                    ev_out[i].record(s_out)

        e2e_step()
        barrier_sync(dist)
        t0 = time.perf_counter()
        for _ in range(args.e2e_steps):
            e2e_step()
        barrier_sync(dist)
        e2e_ms = max_over_ranks(1e3 * (time.perf_counter() - t0) / args.e2e_steps, dist, device)
        # the host link by itself, both directions at once, on the same pinned buffers: the floor for these bytes
        torch.cuda.synchronize()
        pairs = [(d, h) for L, hin in zip(layers, host_in) for d, h in zip([L.x] + ([L.w, L.g] if wl.backward else []), hin)]
        backs = [(h, d) for L, hout in zip(layers, host_out)
                 for h, d in zip(hout, [L.y] + ([L.dx, L.dw] if wl.backward else []))]
        t0 = time.perf_counter()
        with torch.cuda.stream(s_in):
            for d, h in pairs:
                d.copy_(h, non_blocking=True)
        with torch.cuda.stream(s_out):
            for h, d in backs:
                h.copy_(d, non_blocking=True)
        torch.cuda.synchronize()
        link_ms = 1e3 * (time.perf_counter() - t0)
        e2e = {"value": world * step_flops / (e2e_ms * 1e-3) / 1e12, "unit": UNIT, "ms_per_step": e2e_ms,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "copies_alone_ms": link_ms,
               "how": "pinned host buffers; copies in, kernels and copies out on three streams, ordered per layer (each "
                      "layer quantises its own tensors as they arrive: fp8_cast_predicted per tensor); copies_alone_ms = "
                      "the same copies, both directions at once, with no kernels"}
        del host_in, host_out

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return 0

    # ---- the other configurations, one short line each (their tensors replace the headline's on the device) ----
    others = None
    if extra and world == 1 and wl.name == DEFAULT_WORKLOAD and not args.tokens:
        del step, layers
        torch.cuda.empty_cache()
        others = []
        for name, tk in (("c1_single", 0), ("c2_gpt", 0), ("c4_llama70b_ptq", 2048), ("c4_llama70b_ptq", 64),
                         ("c4_llama70b_ptq", 16), ("c4_llama70b_ptq", 1)):
            try:
                others.append(workload_summary(ctx, fp8lin, name, tk, device, seed, peaks))
            except Exception as exc:
                others.append({"workload": name, "tokens": tk, "error": str(exc)[:200]})
                torch.cuda.synchronize()

    cpu_baseline = None
    if world == 1 and not args.no_cpu_baseline:
        import oracle as O
        O.build()
        dt, fl, what, cores, _, _ = oracle_sample_run(wl, I.BASE_SEED, oracle_sample_tokens(wl, 12.0))
        cpu_baseline = {"value": fl / dt / 1e12, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": what,
                        "seconds": dt, **ORACLE_SPLIT}

    quant_note = {
        "group-predicted": "FP8-AMAX for W, X, dY every step, all tensors of the step in one fp8_cast_group call; each tensor "
                           "is cast in the pass that takes its amax, with the bias its previous step left, and cast again "
                           "if Eq. 3 gives another bias (bit-identical to the two-pass path)",
        "group": "FP8-AMAX for W, X, dY every step, all tensors of the step in one fp8_cast_group call (amax pass, cast pass)",
        "per-tensor": "FP8-AMAX recomputed every step, one fp8_cast_e4 / _e5 call per tensor",
        "per-tensor-predicted": "FP8-AMAX recomputed every step, one fp8_cast_predicted call per tensor"}[
            "per-tensor" if decode and quant.startswith("group") else quant]
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "fp8_e4m3/e5m2 operands, f32 accumulate, bf16 out", "data": "synthetic",
        "config": {"workload": wl.name, "tokens": tokens,
                   "layers": [f"{l.name}:{l.K}->{l.N}" for l in wl.layers],
                   "passes": "fwd+bwd" if wl.backward else "fwd (weights quantised once at load)",
                   "scaling_bias": quant_note if wl.backward else "FP8-AMAX for X every step; " + quant_note,
                   "quantisation_mode": "per-tensor" if decode and quant.startswith("group") else quant,
                   "matmuls": "all matmuls of the step in one fp8_linear_group call (one persistent launch; the layers of "
                              "a step are independent here)" if step_matmuls == "group" else "one call per matmul",

                   "l2": "inputs larger than L2 (each layer's tensors exceed 126 MB); no flush between steps",
                   "fp8_layouts": "row-major + transposed copy" if args.transposed_copies else "row-major only",
                   "parallelism": "replicas" if world > 1 else "single"},
        "clocks": clocks,
        "e2e": e2e,
        "gpu_launches": launches_timed,
        "roofline": roofline,
        "amax_cast": {"effective_gbs": cast_elems * bytes_per_elem / (cast_ms * 1e-3) / 1e9 if cast_ms > 0 else None,
                      "bytes_per_element": bytes_per_elem, "ms_per_step": cast_ms / sampled_steps,
                      "hbm_peak_gbs": peaks["hbm_gbs"],
                      "frac": cast_elems * bytes_per_elem / (cast_ms * 1e-3) / 1e9 / peaks["hbm_gbs"] if cast_ms > 0 else None,
                      "guesses_held_missed": list(guesses),
                      "note": "amax + bias + cast of every tensor of a step as timed inside the step (events on every "
                              "eighth step), against the 3 B/element a single pass must move; per_kernel holds each "
                              "kernel alone against its own bytes; other_modes and moving_gradients the same step under "
                              "the other quantisation paths and with biases that move",
                      "per_kernel": per_kernel},
        "layer_matmul_ms": {k: round(v, 4) for k, v in layer_ms.items()},
        "other_modes": other_modes,
        "moving_gradients": moving,
        "with_cuda_graph": graphed,
        "sustained": sustained,
        "fused_mlp": fused_mlp,
        "other_workloads": others,
        "gemm_ms_per_step": gemm_ms / sampled_steps,
        "weight_stream_gbs": (None if wl.backward else
                              weight_bytes * sampled_steps / (gemm_ms * 1e-3) / 1e9),
        "device_flags": flags,
        "cpu_baseline": cpu_baseline,
    }
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
