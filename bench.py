#!/usr/bin/env python
"""Benchmark of the core-sparse FFN path: tokens/s of the whole request (selection +
compaction + batch-1 decode through all layers) on synthetic, model-shaped data.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--impl reference]

One "step" is one request: per layer, core-neuron selection on the resident pre-fill
activations and compaction of the selected weights, then `decode_steps` batch-1 tokens, each
one launch through all compacted layers.  Rank 0 prints ONE JSON line.

--impl reference times the CPU oracle, as it stands, on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "core-sparse decode tokens/s at batch 1; achieved HBM GB/s vs B200 peak"
UNIT = "tokens/s"
FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum of one decode_stack_kernel launch at the bench
# workload, from an ncu capture of a 4-layer launch of the same shapes scaled by the layer count
# (every layer streams its own weights).  None whenever the kernel has changed since the capture.
NCU_TRAFFIC_BYTES_PER_LAUNCH = {"opt6.7b": 219.17e6 / 4 * 32}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", default="opt6.7b")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-dense", action="store_true", help="skip the dense (alpha = beta = 1) comparison")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-configs", action="store_true",
                    help="skip the per-configuration block (decode, dense, selection and compaction timings of the "
                         "other workload shapes, measured after the timed region)")
    ap.add_argument("--no-graph", action="store_true", help="issue every call from the host instead of replaying CUDA graphs")
    ap.add_argument("--decode-only", type=int, default=0, metavar="LAYERS",
                    help="profiling target: only decode launches through the first LAYERS layers of the config "
                         "on random compacted weights (small enough for an ncu capture); prints a short JSON line")
    ap.add_argument("--prefill-only", type=int, default=0, metavar="LAYERS",
                    help="profiling target: tensor-core activations, selection and compaction of the first LAYERS "
                         "layers of the config, nothing else (small enough for an ncu capture); prints a short JSON line")
    ap.add_argument("--tokens", type=int, default=2, help="decode launches per step in --decode-only mode")
    ap.add_argument("--batch", type=int, default=1, help="sequences per decode step in --decode-only mode (1..8)")
    ap.add_argument("--stamps", action="store_true",
                    help="with --decode-only: run the phase-timing build of the library (-DCOREINFER_STAMPS) and add "
                         "the per-phase table of the last launch (median over CTAs and layers, microseconds)")
    ap.add_argument("--sequences", type=int, default=None,
                    help="also time the compacted stack for this many sequences sharing the core sets (2..8; "
                         "default: 8 for the gated Llama-shaped workload, which is specified at 1 and 8, else off)")
    return ap.parse_args()


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ------------------------------------------------------------------ clocks ---
class ClockSampler(threading.Thread):
    """Samples SM clock and clock-event reasons of one GPU through NVML while the timed region runs."""
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown",
               0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown"}

    def __init__(self, torch_device_index: int, period_s: float = 0.05):
        super().__init__(daemon=True)
        self.period = period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        self.handle = None
        try:
            import pynvml
            import torch
            self.nv = pynvml
            pynvml.nvmlInit()
            try:
                uuid = "GPU-" + str(torch.cuda.get_device_properties(torch_device_index).uuid)
                self.handle = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                self.handle = pynvml.nvmlDeviceGetHandleByIndex(torch_device_index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.handle = None

    def run(self):
        if self.handle is None:
            return
        while not self._stop_evt.is_set():
            try:
                self.samples.append(int(self.nv.nvmlDeviceGetClockInfo(self.handle, self.nv.NVML_CLOCK_SM)))
                try:
                    mask = int(self.nv.nvmlDeviceGetCurrentClocksEventReasons(self.handle))
                except Exception:
                    mask = int(self.nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.handle))
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop_evt.wait(self.period)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2.0)
        s = sorted(self.samples)
        return {"sm_mhz": (s[len(s) // 2] if s else None), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(s)}


# ------------------------------------------------------------- CPU baseline ---
def host_activations(cfg, X, w_up, w_gate):
    """Input of the CPU baseline's selection: the layer's pre-fill activations [T, d_ff] fp32, made
    with torch's CPU matmul (input generation, neither the oracle nor the CUDA path)."""
    import torch
    u = X.float() @ w_up.float().t()
    if cfg.gated:
        return (torch.relu(X.float() @ w_gate.float().t()) * u).numpy()
    return torch.relu(u).numpy()


def reduce_max(value: float, device=None) -> float:
    """Max over ranks of a host scalar (identity without a process group)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tokens_per_s(world: int, steps: int, tokens_per_step: int, max_ms: float) -> float:
    """Every rank serves its own requests (no data-path collective): units of all ranks / slowest rank's time."""
    return world * steps * tokens_per_step / (max_ms * 1e-3)


def oracle_sample(cfg, n_layers=2, n_tokens=4, seed_layer=0):
    """Times the oracle on a bounded sample of the workload: selection + compaction of `n_layers`
    layers (full T, d_ff) and `n_tokens` decode tokens through those layers (with the glue),
    then scales to the whole request: L layers, cfg.decode_steps tokens.  Returns tokens/s."""
    import numpy as np
    import torch
    import oracle
    from paper_2410_18311_b200 import workloads as wl

    f32 = lambda t: None if t is None else t.float().numpy()
    kind = oracle.RELU_GATED if cfg.gated else oracle.RELU
    X = wl.prompt_hidden(cfg, device="cpu")
    t_select = t_compact = t_decode = 0.0
    layers = []
    for l in range(n_layers):
        w_up, w_gate, w_down = wl.layer_weights(cfg, seed_layer + l, device="cpu")
        H = host_activations(cfg, X, w_up, w_gate)                                    # untimed input
        t0 = time.perf_counter()
        S, _ = oracle.select(H, cfg.alpha, cfg.beta)
        t1 = time.perf_counter()
        raw = lambda t: None if t is None else (t.view(torch.int16).numpy() if t.dtype == torch.bfloat16 else t.numpy())
        up_c, gate_c, down_c, _ = oracle.compact(raw(w_up), raw(w_gate), raw(w_down), None, S)
        t2 = time.perf_counter()
        t_select += t1 - t0
        t_compact += t2 - t1
        back = lambda a: None if a is None else (torch.from_numpy(a.view(np.int16)).view(torch.bfloat16).float().numpy()
                                                if cfg.dtype == "bf16" else a)
        layers.append((back(up_c), back(gate_c), back(down_c)))
    for tok in range(n_tokens):
        x = f32(wl.decode_input(cfg, tok, device="cpu"))
        t0 = time.perf_counter()
        for (up_c, gate_c, down_c) in layers:
            y = oracle.ffn(x, kind, up_c, gate_c, down_c)
            x = torch.from_numpy(oracle.glue(x, y)).to(cfg.torch_dtype).float().numpy()[None, :]
        t_decode += time.perf_counter() - t0
    per_layer_prefill = (t_select + t_compact) / n_layers
    per_token = t_decode / n_tokens / n_layers * cfg.L
    request_s = per_layer_prefill * cfg.L + per_token * cfg.decode_steps
    return {
        "value": cfg.decode_steps / request_s, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
        "sample": "%d of %d layers (selection T=%d + compaction) and %d decode tokens through them, scaled "
                  "linearly to %d layers x %d tokens" % (n_layers, cfg.L, cfg.T, n_tokens, cfg.L, cfg.decode_steps),
        "select_ms_per_layer": 1e3 * t_select / n_layers, "compact_ms_per_layer": 1e3 * t_compact / n_layers,
        "decode_ms_per_token": 1e3 * per_token, "sample_seconds": t_select + t_compact + t_decode,
    }


def config_dict(cfg, K):
    """The workload description both arms print."""
    nbytes = cfg.L * cfg.n_mat * K * cfg.d_model * cfg.esize + cfg.L * 2 * cfg.d_model * 4
    return {"workload": cfg.name, "L": cfg.L, "d_model": cfg.d_model, "d_ff": cfg.d_ff, "T": cfg.T,
            "alpha": cfg.alpha, "beta": cfg.beta, "K": K, "decode_steps": cfg.decode_steps, "batch": 1,
            "gated": cfg.gated, "step": "selection + compaction of all layers, then decode_steps tokens",
            "l2": "inputs larger than L2 (%.2f GB of compacted weights per token)" % (nbytes / 1e9),
            "parallelism": "independent requests per GPU, no collective"}


def run_reference(args, cfg):
    """--impl reference: the oracle on host cores; each step is one bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import count as oracle_count
    for _ in range(min(args.warmup, 1)):
        oracle_sample(cfg, n_layers=1, n_tokens=1)
    vals, t0 = [], time.perf_counter()
    last = None
    for _ in range(args.steps):
        last = oracle_sample(cfg, n_layers=1, n_tokens=2)
        vals.append(last["value"])
    wall = time.perf_counter() - t0
    v = sum(vals) / len(vals)
    line = {
        "impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * cfg.decode_steps / v, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
        "config": config_dict(cfg, oracle_count(cfg.beta, cfg.d_ff)),
        "cpu_baseline": {"value": v, "unit": UNIT, "cores": last["cores"], "kind": "oracle", "sample": last["sample"]},
        "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0, "wall_s": wall,
    }
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------- GPU arm ----
def prefill_inputs(ci, wl, cfg, device):
    """Synthetic request state resident in HBM: dense weights of every layer and the fp32
    pre-fill activations A[l] = [T, d_ff] (dense FFN chained through the layers with the same
    residual + RMS glue the decode stack uses)."""
    import torch
    kind = ci.FFN_RELU_GATED if cfg.gated else ci.FFN_RELU
    weights, acts = [], []
    X = wl.prompt_hidden(cfg, device=device)
    for l in range(cfg.L):
        if cfg.planted:
            w = wl.layer_weights(cfg, l, device=device)
            A, _ = wl.planted_activations(cfg, l, cfg.T, device=device)
        else:
            w = wl.layer_weights(cfg, l, device=device)
            A = torch.empty((cfg.T, cfg.d_ff), device=device)
            Y = torch.empty((cfg.T, cfg.d_model), device=device)
            ci.coreinfer_ffn_dense_ref(X, kind, w[0], w[1], w[2], None, None, A, Y)
            V = X.float() + Y
            X = (V / V.pow(2).mean(dim=1, keepdim=True).sqrt()).to(cfg.torch_dtype)
        weights.append(w)
        acts.append(A)
    torch.cuda.synchronize()
    return weights, acts


def run_ours(args, cfg):
    import torch
    import torch.distributed as dist
    import paper_2410_18311_b200 as ci
    from paper_2410_18311_b200 import _build, workloads as wl

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        _build.build()
    if world > 1:
        dist.barrier()
    ci.binding.load()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    weights, acts = prefill_inputs(ci, wl, cfg, dev)
    stack = ci.pipeline.CoreSparseStack(cfg, device=dev)
    steps_tok = cfg.decode_steps
    xs = torch.cat([wl.decode_input(cfg, s, device=dev) for s in range(steps_tok)], dim=0)   # [steps, d]
    ys = torch.empty((steps_tok, cfg.d_model), device=dev)
    stream = torch.cuda.current_stream()

    def request(ev=None):
        if ev: ev[0].record(stream)
        stack.prefill(acts, weights, stream)
        if ev: ev[1].record(stream)
        for s in range(steps_tok):
            stack.decode(xs[s:s + 1], ys[s:s + 1], stream=stream)
        if ev: ev[2].record(stream)

    request()
    barrier()
    stack.check()
    # The request's calls are captured once into two CUDA graphs (pre-fill stage, decode stage) and
    # replayed: the same kernels with the same arguments, without the per-call host work between them.
    graphs = None
    if not args.no_graph:
        try:
            cap = torch.cuda.Stream(device=dev)
            cap.wait_stream(stream)
            g_pre, g_dec = torch.cuda.CUDAGraph(), torch.cuda.CUDAGraph()
            with torch.cuda.graph(g_pre, stream=cap, capture_error_mode="relaxed"):
                stack.prefill(acts, weights, torch.cuda.current_stream())
            with torch.cuda.graph(g_dec, stream=cap, capture_error_mode="relaxed"):
                cs = torch.cuda.current_stream()
                for s in range(steps_tok):
                    stack.decode(xs[s:s + 1], ys[s:s + 1], stream=cs)
            stream.wait_stream(cap)
            graphs = (g_pre, g_dec)
        except Exception as exc:                      # capture not possible here: plain calls
            print("bench: CUDA graph capture failed (%s); using plain calls" % str(exc).splitlines()[0], file=sys.stderr)
            torch.cuda.synchronize()
            graphs = None
    if graphs is not None:
        def request(ev=None):
            if ev: ev[0].record(stream)
            graphs[0].replay()
            if ev: ev[1].record(stream)
            graphs[1].replay()
            if ev: ev[2].record(stream)

    for _ in range(max(args.warmup, 3)):
        request()
    barrier()
    stack.check()

    sampler = ClockSampler(local)
    sampler.start()
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    barrier()
    t_wall0 = time.perf_counter()
    for i in range(args.steps):
        request(evs[i])
    barrier()
    wall = time.perf_counter() - t_wall0
    clocks = sampler.stop()
    stack.check()
    total_ms = evs[0][0].elapsed_time(evs[-1][2])
    prefill_ms = sum(e[0].elapsed_time(e[1]) for e in evs) / args.steps
    decode_ms = sum(e[1].elapsed_time(e[2]) for e in evs) / args.steps

    total_ms_max = reduce_max(total_ms, dev)
    value = whole_job_tokens_per_s(world, args.steps, steps_tok, total_ms_max)

    # ---- per-stage latencies (outside the timed region) ----
    def time_call(fn, reps=5):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        fn(); torch.cuda.synchronize()
        a.record(stream)
        for _ in range(reps): fn()
        b.record(stream); torch.cuda.synchronize()
        return a.elapsed_time(b) / reps
    sel_ms = time_call(lambda: [stack.select_layer(l, acts[l], None, stream) for l in range(cfg.L)]) / cfg.L
    cmp_ms = time_call(lambda: [stack.compact_layer(l, *weights[l], stream=stream) for l in range(cfg.L)]) / cfg.L

    # ---- end to end through the public API with host buffers ----
    e2e = None
    if not args.no_e2e:
        acts_h = [torch.empty(a.shape, dtype=a.dtype, pin_memory=True).copy_(a) for a in acts]
        xs_h = torch.empty(xs.shape, dtype=xs.dtype, pin_memory=True).copy_(xs)
        ys_h = torch.empty(ys.shape, dtype=ys.dtype, pin_memory=True)
        x_d = torch.empty((1, cfg.d_model), dtype=xs.dtype, device=dev)
        y_d = torch.empty((1, cfg.d_model), device=dev)
        acts_d = [torch.empty_like(a) for a in acts]

        # one token = copy of x from pinned memory, one decode launch, copy of y back: captured once
        x_pin = torch.empty((1, cfg.d_model), dtype=xs.dtype, pin_memory=True)
        y_pin = torch.empty((1, cfg.d_model), dtype=torch.float32, pin_memory=True)
        g_tok = None
        if graphs is not None:
            try:
                cap = torch.cuda.Stream(device=dev)
                cap.wait_stream(stream)
                g_tok = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g_tok, stream=cap, capture_error_mode="relaxed"):
                    x_d.copy_(x_pin, non_blocking=True)
                    stack.decode(x_d, y_d, stream=torch.cuda.current_stream())
                    y_pin.copy_(y_d, non_blocking=True)
                stream.wait_stream(cap)
            except Exception:
                torch.cuda.synchronize()
                g_tok = None
        copy_stream = torch.cuda.Stream(device=dev)
        copied = [torch.cuda.Event() for _ in range(cfg.L)]
        # host-side views for the per-token host-to-host copies (numpy has no bf16: same bytes as int16 / int32)
        raw = torch.int16 if cfg.esize == 2 else torch.int32
        xs_np, x_pin_np = xs_h.view(raw).numpy(), x_pin.view(raw).numpy()
        ys_np, y_pin_np = ys_h.numpy(), y_pin.numpy()

        def request_e2e():
            # activations arrive layer by layer on a copy stream; each layer is selected and
            # compacted as soon as its activations are on the device
            copy_stream.wait_stream(stream)
            with torch.cuda.stream(copy_stream):
                for l in range(cfg.L):
                    acts_d[l].copy_(acts_h[l], non_blocking=True)
                    copied[l].record(copy_stream)
            for l in range(cfg.L):
                stream.wait_event(copied[l])
                stack.select_layer(l, acts_d[l], None, stream)
                stack.compact_layer(l, *weights[l], stream=stream)
            for s in range(steps_tok):
                if g_tok is not None:
                    x_pin_np[0] = xs_np[s]                # host to host, 8 KB
                    g_tok.replay()                        # x to the device, one decode launch, y back
                    stream.synchronize()                  # the token's result is on the host before the next one starts
                    ys_np[s] = y_pin_np[0]
                else:
                    x_d.copy_(xs_h[s:s + 1], non_blocking=True)
                    stack.decode(x_d, y_d, stream=stream)
                    ys_h[s:s + 1].copy_(y_d, non_blocking=True)
                    stream.synchronize()
        request_e2e()
        barrier()
        n_e2e = max(1, min(args.steps, 5))
        t0 = time.perf_counter()
        for _ in range(n_e2e):
            request_e2e()
        barrier()
        dt = time.perf_counter() - t0
        dt_max = reduce_max(dt, dev)
        h2d = sum(a.numel() * 4 for a in acts) + steps_tok * cfg.d_model * cfg.esize
        e2e = {"value": whole_job_tokens_per_s(world, n_e2e, steps_tok, dt_max * 1e3), "unit": UNIT,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": steps_tok * cfg.d_model * 4,
               "requests_timed": n_e2e}
        del acts_h, acts_d

    # ---- the same kernel run dense (alpha = beta = 1), a few tokens ----
    dense = None
    if not args.no_dense and rank == 0:
        try:
            dcfg = cfg
            dstack = ci.pipeline.CoreSparseStack(dcfg, device=dev, alpha=1.0, beta=1.0)
            all_idx = torch.arange(cfg.d_ff, dtype=torch.int32, device=dev)
            for l in range(cfg.L):
                dstack.core_idx[l].copy_(all_idx)
                dstack.compact_layer(l, *weights[l], stream=stream)
            ntok = 8
            ms = time_call(lambda: [dstack.decode(xs[s:s + 1], ys[s:s + 1], stream=stream) for s in range(ntok)], reps=2)
            dstack.check()
            dbytes = dstack.compacted_bytes_per_token()
            dense = {"tok_s": ntok / (ms * 1e-3), "gbs": dbytes * ntok / (ms * 1e-3) / 1e9, "bytes_per_token": dbytes,
                     "tokens_timed": 2 * ntok}
            del dstack
        except torch.OutOfMemoryError:
            dense = {"skipped": "not enough free HBM for a second, dense copy of the stack"}

    # ---- the same compacted stack for several sequences that share the core sets ----
    batched = None
    n_seq = args.sequences if args.sequences is not None else (8 if cfg.gated else 0)
    if n_seq > 1 and rank == 0:
        nb, nstep = n_seq, 16
        xb = wl.decode_input(cfg, 0, device=dev, batch=nb)
        yb = torch.empty((nb, cfg.d_model), device=dev)
        wsb = torch.empty(ci.coreinfer_ffn_decode_stack_workspace_bytes(cfg.L, nb, cfg.d_model, stack.K),
                          dtype=torch.uint8, device=dev)
        ms = time_call(lambda: [ci.coreinfer_ffn_decode_stack(stack.layers, xb, stack.kind, yb, None, None, wsb, stream)
                                for _ in range(nstep)], reps=2) / nstep
        ci.coreinfer_workspace_status(wsb)
        batched = {"batch": nb, "ms_per_step": ms, "sequence_tok_s": nb / (ms * 1e-3),
                   "gbs": stack.compacted_bytes_per_token() / (ms * 1e-3) / 1e9, "steps_timed": 2 * nstep}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_src = measured_peak()
    bytes_tok = stack.compacted_bytes_per_token() + cfg.L * 2 * cfg.d_model * 4
    launch_s = decode_ms * 1e-3 / steps_tok
    achieved = bytes_tok / launch_s / 1e9
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": total_ms_max / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
        "config": config_dict(cfg, stack.K),
        "launch_mode": "two CUDA graphs per request (pre-fill stage, decode stage)" if graphs is not None
                       else "one host call per kernel group",
        "decode": {"tok_s": steps_tok / (decode_ms * 1e-3), "ms_per_token": decode_ms / steps_tok,
                   "gbs": achieved, "frac_of_8TBs": achieved / 8000.0},
        "select_ms_per_layer": sel_ms, "compact_ms_per_layer": cmp_ms, "prefill_ms_per_request": prefill_ms,
        "dense": dense, "batched": batched,
        "roofline": {"bound": "hbm", "kernel": "decode_stack_kernel", "achieved": achieved, "peak": peak,
                     "unit": "GB/s", "frac": achieved / peak, "peak_source": "of " + peak_src,
                     "bytes_per_launch": bytes_tok, "launch_us": launch_s * 1e6,
                     "traffic": NCU_TRAFFIC_BYTES_PER_LAUNCH.get(cfg.name)},
        "e2e": e2e,
        "gpu_launches": args.steps * (cfg.L * (stack.SELECT_KERNELS_PER_LAYER + stack.COMPACT_KERNELS_PER_LAYER)
                                      + steps_tok * stack.DECODE_KERNELS_PER_TOKEN),
        "clocks": clocks, "wall_s": wall,
        "context": "paper (TITAN Xp, end to end, other workload): 10.33x over HuggingFace, 2.72x over PowerInfer",
    }
    if not args.no_configs and world == 1:
        del weights, acts, stack
        torch.cuda.empty_cache()
        pre = prefill_stage_times(ci, wl, cfg, cfg.T, cfg.beta)
        pre["select_floor_us_at_measured_peak"] = pre["activation_bytes"] / peak / 1e3
        line["prefill_stage_one_layer"] = pre
        line["configs"] = other_configs(ci, wl, peak, cfg.name)
        line["extensions"] = extension_times(ci, wl, peak)
    if not args.no_cpu_baseline and world == 1:
        line["cpu_baseline"] = oracle_sample(cfg, n_layers=4, n_tokens=min(cfg.decode_steps, 256))
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


# ------------------------------------------------- the other configurations ---
def _time_ms(fn, stream, reps):
    import torch
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    fn(); torch.cuda.synchronize()
    a.record(stream)
    for _ in range(reps): fn()
    b.record(stream); torch.cuda.synchronize()
    return a.elapsed_time(b) / reps


def decode_stack_rate(ci, wl, cfg, K, layers, batch, peak, tokens=16, reps=3):
    """Decode launches alone through `layers` layers of random compacted [K, d] weights of cfg's shape
    (the decode stage does not care how the rows were chosen); rates are per full stack of cfg.L layers,
    scaled from the cut by the layer count when layers < cfg.L."""
    import torch
    cut = cfg.with_(L=layers)
    w = [wl.compacted_weights_random(cut, l, K, device="cuda") for l in range(layers)]
    arr = ci.binding.make_layers([(u, g, dn, None, None) for (u, g, dn) in w])
    kind = ci.FFN_RELU_GATED if cfg.gated else ci.FFN_RELU
    xs = [wl.decode_input(cfg, s, device="cuda", batch=batch) for s in range(tokens)]
    y = torch.empty((batch, cfg.d_model), device="cuda")
    ws = torch.empty(ci.coreinfer_ffn_decode_stack_workspace_bytes(layers, batch, cfg.d_model, K), dtype=torch.uint8,
                     device="cuda")
    stream = torch.cuda.current_stream()
    ms = _time_ms(lambda: [ci.coreinfer_ffn_decode_stack(arr, xs[t], kind, y, None, None, ws, stream) for t in range(tokens)],
                  stream, reps) / tokens
    ci.coreinfer_workspace_status(ws)
    nbytes = layers * cfg.n_mat * K * cfg.d_model * cfg.esize
    gbs = nbytes / (ms * 1e-3) / 1e9
    full_ms = ms * cfg.L / layers
    out = {"K": K, "batch": batch, "layers_timed": layers, "us_per_layer": 1e3 * ms / layers, "gbs": gbs,
           "frac_of_measured": gbs / peak, "frac_of_8TBs": gbs / 8000.0,
           "steps_per_s_full_stack": 1e3 / full_ms, "sequence_tok_s_full_stack": batch * 1e3 / full_ms,
           "launches_timed": tokens * reps}
    del w, arr
    return out


def prefill_stage_times(ci, wl, cfg, T, beta, layer=0):
    """Selection and compaction of ONE full-size layer of cfg: microseconds per layer."""
    import torch
    kind = ci.FFN_RELU_GATED if cfg.gated else ci.FFN_RELU
    w_up, w_gate, w_down = wl.layer_weights(cfg, layer, device="cuda")
    act_us = None
    stream = torch.cuda.current_stream()
    if cfg.planted:
        A, _ = wl.planted_activations(cfg, layer, T, device="cuda")
    else:
        X = wl.prompt_hidden(cfg, device="cuda", T=T)
        A = torch.empty((T, cfg.d_ff), device="cuda")
        if cfg.dtype == "bf16":      # the activations as the tensor-core pre-fill produces them
            tws = torch.empty(ci.coreinfer_prefill_activations_workspace_bytes(), dtype=torch.uint8, device="cuda")
            act_us = 1e3 * _time_ms(lambda: ci.coreinfer_prefill_activations(X, kind, w_up, w_gate, None, A, tws, stream),
                                    stream, 10)
            ci.coreinfer_workspace_status(tws)
        else:
            ci.coreinfer_ffn_dense_ref(X, kind, w_up, w_gate, w_down, None, None, A, None)
    K = ci.coreinfer_count(beta, cfg.d_ff)
    S = torch.empty(K, dtype=torch.int32, device="cuda")
    ws = torch.empty(ci.coreinfer_select_workspace_bytes(T, cfg.d_ff), dtype=torch.uint8, device="cuda")
    sel = _time_ms(lambda: ci.coreinfer_select_core(A, cfg.alpha, beta, S, None, ws, stream), stream, 10)
    new = lambda: torch.empty((K, cfg.d_model), dtype=cfg.torch_dtype, device="cuda")
    up_c, down_c, gate_c = new(), new(), (new() if cfg.gated else None)
    cmp_ = _time_ms(lambda: ci.coreinfer_compact(w_up, w_gate, w_down, None, S, K, up_c, gate_c, down_c, None, stream),
                    stream, 5)
    return {"T": T, "K": K, "activations_tensor_core_us": act_us,
            "activations_tflops": (None if act_us is None else
                                   2.0 * T * cfg.d_model * cfg.d_ff * (2 if cfg.gated else 1) / act_us / 1e6),
            "select_us": 1e3 * sel, "select_floor_us_at_measured_peak": None,
            "activation_bytes": 4 * T * cfg.d_ff, "compact_us": 1e3 * cmp_}


def extension_times(ci, wl, peak):
    """The calls beyond the timed path, at the headline shapes: the SiLU-gated / fp16 decode stack
    (Llama-2-7B shape), and the set calls (top fraction by count, similarity, nearest centroid,
    in-place update of 5 % of a deployed OPT-6.7B-shaped layer)."""
    import numpy as np
    import torch
    out = {}
    cfg = wl.CONFIGS["relu-llama2-7b"]
    K = ci.coreinfer_count(cfg.beta, cfg.d_ff)
    w = [tuple(t if t is None else t.to(torch.float16) for t in wl.compacted_weights_random(cfg, l, K, device="cuda"))
         for l in range(cfg.L)]
    arr = ci.binding.make_layers([(u, g, dn, None, None) for (u, g, dn) in w])
    xs = [wl.decode_input(cfg, s, device="cuda").to(torch.float16) for s in range(16)]
    y = torch.empty((1, cfg.d_model), device="cuda")
    ws = torch.empty(ci.coreinfer_ffn_decode_stack_workspace_bytes(cfg.L, 1, cfg.d_model, K), dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()
    ms = _time_ms(lambda: [ci.coreinfer_ffn_decode_stack(arr, xs[t], ci.FFN_SILU_GATED, y, None, None, ws, stream)
                           for t in range(16)], stream, 3) / 16
    ci.coreinfer_workspace_status(ws)
    nbytes = cfg.L * 3 * K * cfg.d_model * 2
    out["silu_gated_fp16_decode_llama_shape"] = {"us_per_layer": 1e3 * ms / cfg.L, "tok_s": 1e3 / ms,
                                                 "gbs": nbytes / ms / 1e6, "frac_of_measured": nbytes / ms / 1e6 / peak}
    del w, arr
    torch.cuda.empty_cache()
    c2 = wl.CONFIGS["opt6.7b"]
    N, K2 = c2.d_ff, ci.coreinfer_count(c2.beta, c2.d_ff)
    g = torch.Generator(device="cuda").manual_seed(1)
    counts = torch.randint(0, c2.T + 1, (N,), generator=g, device="cuda", dtype=torch.int32)
    S = torch.empty(K2, dtype=torch.int32, device="cuda")
    out["top_by_count_us"] = 1e3 * _time_ms(lambda: ci.coreinfer_top_by_count(counts, c2.T, c2.beta, S, stream), stream, 20)
    rng = np.random.default_rng(0)
    S0 = np.sort(rng.choice(N, size=K2, replace=False)).astype(np.int32)
    keep = rng.choice(S0, size=K2 - K2 // 20, replace=False)
    S1 = np.sort(np.concatenate([keep, rng.choice(np.setdiff1d(np.arange(N), S0), size=K2 - len(keep), replace=False)])).astype(np.int32)
    a, b = torch.from_numpy(S0).cuda(), torch.from_numpy(S1).cuda()
    pair = torch.empty(2, dtype=torch.int32, device="cuda")
    out["core_similarity_us"] = 1e3 * _time_ms(lambda: ci.coreinfer_core_similarity(a, b, pair, stream), stream, 20)
    C = torch.randn((16, c2.d_model), generator=g, device="cuda")
    v = torch.randn((c2.d_model,), generator=g, device="cuda")
    cws = torch.empty(ci.coreinfer_nearest_centroid_workspace_bytes(16), dtype=torch.uint8, device="cuda")
    gi = torch.empty(1, dtype=torch.int32, device="cuda")
    out["nearest_centroid_16_groups_us"] = 1e3 * _time_ms(lambda: ci.coreinfer_nearest_centroid(C, v, gi, cws, stream), stream, 20)
    w_up, _, w_down = wl.layer_weights(c2, 0, device="cuda")
    # activations kept in bf16: tensor-core pre-fill writing bf16, selection reading it
    X = wl.prompt_hidden(c2, device="cuda")
    A16 = torch.empty((c2.T, N), dtype=torch.bfloat16, device="cuda")
    tws = torch.empty(ci.coreinfer_prefill_activations_workspace_bytes(), dtype=torch.uint8, device="cuda")
    sws = torch.empty(ci.coreinfer_select_workspace_bytes(c2.T, N), dtype=torch.uint8, device="cuda")
    out["activations_bf16_out_us"] = 1e3 * _time_ms(
        lambda: ci.coreinfer_prefill_activations(X, ci.FFN_RELU, w_up, None, None, A16, tws, stream), stream, 10)
    out["select_on_bf16_us"] = 1e3 * _time_ms(
        lambda: ci.coreinfer_select_core(A16, c2.alpha, c2.beta, S, None, sws, stream), stream, 10)
    ci.coreinfer_workspace_status(tws)
    ci.coreinfer_workspace_status(sws)
    new = lambda: torch.empty((K2, c2.d_model), dtype=c2.torch_dtype, device="cuda")
    up_c, down_c = new(), new()
    ci.coreinfer_compact(w_up, None, w_down, None, a, K2, up_c, None, down_c, None, stream)
    uws = torch.empty(ci.coreinfer_update_core_set_workspace_bytes(N, K2), dtype=torch.uint8, device="cuda")
    nch = torch.empty(1, dtype=torch.int32, device="cuda")
    slot = a.clone()
    sets = [b, a]

    def flip(i=[0]):          # alternate between the two sets: every call rewrites 5 % of the rows
        ci.coreinfer_update_core_set(w_up, None, w_down, None, slot, sets[i[0] & 1], up_c, None, down_c, None, nch, uws, stream)
        i[0] += 1
    out["update_core_set_5pct_us"] = 1e3 * _time_ms(flip, stream, 10)
    out["update_core_set_rows_changed"] = int(nch.item())
    return out


def other_configs(ci, wl, peak, headline):
    """Decode rates (sparse and dense), selection and compaction times of every workload
    configuration other than the headline one; CUDA events, outside the timed region."""
    import torch
    out = {}
    for name in ("opt125m-1layer", "opt13b", "relu-llama2-7b", "opt66b"):
        if name == headline:
            continue
        cfg = wl.CONFIGS[name]
        block = {"dtype": cfg.dtype, "L": cfg.L, "d_model": cfg.d_model, "d_ff": cfg.d_ff, "gated": cfg.gated}
        # the OPT-66B-shaped stack is timed on a cut (its 64 compacted layers hold 17 GB, its dense ones 87 GB)
        layers = 16 if name == "opt66b" else cfg.L
        betas = wl.OPT13B_BETAS if name == "opt13b" else (cfg.beta,)
        block["decode"] = {}
        for beta in betas:
            K = ci.coreinfer_count(beta, cfg.d_ff)
            tokens = 16 if K * cfg.d_model * layers < 4e9 else 4
            block["decode"]["beta=%g" % beta] = decode_stack_rate(ci, wl, cfg, K, layers, 1, peak, tokens=tokens)
            torch.cuda.empty_cache()
        if 1.0 not in betas:
            dl = min(layers, 16)
            block["dense"] = decode_stack_rate(ci, wl, cfg, cfg.d_ff, dl, 1, peak, tokens=4, reps=2)
            torch.cuda.empty_cache()
        if name == "relu-llama2-7b":
            K = ci.coreinfer_count(cfg.beta, cfg.d_ff)
            block["decode"]["beta=%g, 8 sequences" % cfg.beta] = decode_stack_rate(ci, wl, cfg, K, layers, 8, peak)
        Ts = wl.OPT66B_TS if name == "opt66b" else (cfg.T,)
        block["prefill"] = []
        for T in Ts:
            r = prefill_stage_times(ci, wl, cfg, T, cfg.beta)
            r["select_floor_us_at_measured_peak"] = r["activation_bytes"] / peak / 1e3
            block["prefill"].append(r)
            torch.cuda.empty_cache()
        out[name] = block
    return out


def run_decode_only(args, cfg):
    """A few launches of the decode kernel alone, on a stack cut to --decode-only layers: the target
    of the full-counter ncu capture (a whole 32-layer launch is too long to replay 40 times)."""
    import torch
    import paper_2410_18311_b200 as ci
    from paper_2410_18311_b200 import _build, workloads as wl
    _build.build()
    if args.stamps:
        ci.binding.use_library(_build.build(stamps=True))
    cfg = cfg.with_(L=args.decode_only)
    K = ci.coreinfer_count(cfg.beta, cfg.d_ff)
    layers = [wl.compacted_weights_random(cfg, l, K, device="cuda") for l in range(cfg.L)]
    arr = ci.binding.make_layers([(u, g, dn, None, None) for (u, g, dn) in layers])
    kind = ci.FFN_RELU_GATED if cfg.gated else ci.FFN_RELU
    B = args.batch
    xs = torch.stack([wl.decode_input(cfg, s, device="cuda", batch=B) for s in range(args.tokens)], dim=0)
    ys = torch.empty((args.tokens, B, cfg.d_model), device="cuda")
    ws = torch.empty(ci.coreinfer_ffn_decode_stack_workspace_bytes(cfg.L, B, cfg.d_model, K), dtype=torch.uint8,
                     device="cuda")

    def step():
        for t in range(args.tokens):
            ci.coreinfer_ffn_decode_stack(arr, xs[t], kind, ys[t], None, None, ws)
    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    ci.coreinfer_workspace_status(ws)
    us = e0.elapsed_time(e1) * 1e3 / (args.steps * args.tokens)
    nbytes = cfg.L * cfg.n_mat * K * cfg.d_model * cfg.esize
    line = {"mode": "decode-only", "workload": cfg.name, "layers": cfg.L, "K": K, "batch": B,
            "us_per_launch": us, "us_per_layer": us / cfg.L, "bytes_per_launch": nbytes,
            "gbs": nbytes / us / 1e3, "sequence_tokens_per_s": B * 1e6 / us}
    if args.stamps:
        line["phases_us"] = phase_table(ci, lambda: ci.coreinfer_ffn_decode_stack(arr, xs[0], kind, ys[0], None, None, ws),
                                        cfg.L, B)
    print(json.dumps(line), flush=True)


PHASES_B1 = [("up rows", 0, 1), ("h formed", 1, 2), ("down rows", 2, 3), ("partial assembled", 3, 4),
             ("bulk reduction", 4, 5), ("release arrival", 5, 6), ("wait for all CTAs", 6, 7),
             ("read-back", 7, 8), ("next input", 8, 9)]
PHASES_BATCHED = [("up units", 0, 1), ("down units", 1, 3), ("flush of the partial", 3, 4),
                  ("grid barrier", 4, 7), ("read-back of the sums", 7, 8), ("next input", 8, 9)]


def phase_table(ci, launch, L, batch):
    """One more launch with cycle stamps recorded (phase-timing build): per phase the median and
    the mean over all CTAs and the layers 1 .. L-2, in microseconds at the SM clock sampled meanwhile."""
    import torch
    n_sm = torch.cuda.get_device_properties(0).multi_processor_count
    stamps = torch.zeros((n_sm, L, ci.binding.STAMP_SLOTS), dtype=torch.int64, device="cuda")
    ci.coreinfer_debug_stamps(stamps)
    sampler = ClockSampler(0, period_s=0.01)
    sampler.start()
    for _ in range(20):
        launch()
    torch.cuda.synchronize()
    mhz = sampler.stop()["sm_mhz"] or 1965
    ci.coreinfer_debug_stamps(None)
    st = stamps.cpu().double()
    inner = st[:, 1:L - 1] if L > 2 else st
    out = {"sm_mhz": mhz}
    for name, a, b in (PHASES_B1 if batch == 1 else PHASES_BATCHED):
        dt = (inner[:, :, b] - inner[:, :, a]).flatten() / mhz
        out[name] = {"median": round(float(dt.median()), 3), "mean": round(float(dt.mean()), 3)}
    if L > 2:
        lay = (st[:, 2:, 0] - st[:, 1:-1, 0]).flatten() / mhz
        out["layer"] = {"median": round(float(lay.median()), 3), "mean": round(float(lay.mean()), 3)}
    return out


def run_prefill_only(args, cfg):
    """The pre-fill stage alone on a few layers: activations (tensor cores; synthesised for the planted
    configuration), selection, compaction.  The target of ncu captures of those kernels."""
    import torch
    import paper_2410_18311_b200 as ci
    from paper_2410_18311_b200 import _build, workloads as wl
    _build.build()
    L = args.prefill_only
    kind = ci.FFN_RELU_GATED if cfg.gated else ci.FFN_RELU
    K = ci.coreinfer_count(cfg.beta, cfg.d_ff)
    X = wl.prompt_hidden(cfg, device="cuda")
    weights = [wl.layer_weights(cfg, l, device="cuda") for l in range(L)]
    A = torch.empty((cfg.T, cfg.d_ff), device="cuda")
    S = torch.empty(K, dtype=torch.int32, device="cuda")
    tws = torch.empty(ci.coreinfer_prefill_activations_workspace_bytes(), dtype=torch.uint8, device="cuda")
    sws = torch.empty(ci.coreinfer_select_workspace_bytes(cfg.T, cfg.d_ff), dtype=torch.uint8, device="cuda")
    new = lambda: torch.empty((K, cfg.d_model), dtype=cfg.torch_dtype, device="cuda")
    up_c, down_c, gate_c = new(), new(), (new() if cfg.gated else None)
    planted = [wl.planted_activations(cfg, l, cfg.T, device="cuda")[0] for l in range(L)] if cfg.planted else None
    stream = torch.cuda.current_stream()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
    t = [0.0, 0.0, 0.0]

    def step(timed):
        for l in range(L):
            w_up, w_gate, w_down = weights[l]
            ev[0].record(stream)
            if cfg.planted:
                act = planted[l]
            else:
                ci.coreinfer_prefill_activations(X, kind, w_up, w_gate, None, A, tws, stream)
                act = A
            ev[1].record(stream)
            ci.coreinfer_select_core(act, cfg.alpha, cfg.beta, S, None, sws, stream)
            ev[2].record(stream)
            ci.coreinfer_compact(w_up, w_gate, w_down, None, S, K, up_c, gate_c, down_c, None, stream)
            ev[3].record(stream)
            if timed:
                torch.cuda.synchronize()
                for i in range(3):
                    t[i] += ev[i].elapsed_time(ev[i + 1])
    for _ in range(args.warmup):
        step(False)
    torch.cuda.synchronize()
    for _ in range(args.steps):
        step(True)
    ci.coreinfer_workspace_status(sws)
    n = args.steps * L
    print(json.dumps({"mode": "prefill-only", "workload": cfg.name, "layers": L, "T": cfg.T, "K": K,
                      "activations_us_per_layer": None if cfg.planted else 1e3 * t[0] / n,
                      "select_us_per_layer": 1e3 * t[1] / n, "compact_us_per_layer": 1e3 * t[2] / n}), flush=True)


def main():
    args = parse_args()
    from paper_2410_18311_b200 import workloads as wl
    cfg = wl.CONFIGS[args.config]
    if args.prefill_only > 0:
        return run_prefill_only(args, cfg)
    if args.decode_only > 0:
        return run_decode_only(args, cfg)
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
