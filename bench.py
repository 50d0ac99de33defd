#!/usr/bin/env python
"""Roofline benchmark of the ResQ mixed-precision linear layer on B200.

A step is one pass of the whole hot path over one batch: the seven linear layers of one
Llama-3-8B-shaped decoder block at T = 4096 prefill tokens (q|k|v and gate|up served as one
N-concatenated layer each; the down_proj input goes through the online bf16 projection), i.e. per
layer: [projection GEMM] -> per-token split quantization -> mixed INT8/INT4 GEMM with the fp32 scale
epilogue.  Prints ONE JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

`--impl reference` times the CPU oracle on a bounded row sample of the same workload instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

# The headline workload (--model 8b) and the two other block shapes of the benchmark configurations
# (--model 1b / 70b: same legs, for the per-configuration table; not the headline line).
# name -> (workload, prefill tokens, [(layer, K, n_out, online projection)])
MODELS = {
    "1b": ("llama3.2-1b-decoder-block-linears-prefill-T2048", 2048,
           [("qkv", 2048, 3072, False), ("o", 2048, 2048, False), ("gate_up", 2048, 16384, False), ("down", 8192, 2048, True)]),
    "8b": ("llama3-8b-decoder-block-linears-prefill-T4096", 4096,
           [("qkv", 4096, 6144, False), ("o", 4096, 4096, False), ("gate_up", 4096, 28672, False), ("down", 14336, 4096, True)]),
    "70b": ("llama3-70b-decoder-block-linears-prefill-T8192", 8192,
            [("qkv", 8192, 10240, False), ("o", 8192, 8192, False), ("gate_up", 8192, 57344, False), ("down", 28672, 8192, True)]),
}
MODEL = "8b"
WORKLOAD, T_PREFILL, LAYERS = MODELS[MODEL]


def select_model(name: str):
    global MODEL, WORKLOAD, T_PREFILL, LAYERS
    MODEL = name
    WORKLOAD, T_PREFILL, LAYERS = MODELS[name]

ORACLE_SAMPLE_ROWS = 1024      # cpu_baseline leg of our arm: one pass, about 10-20 s of CPU work
REFERENCE_STEP_ROWS = 64       # --impl reference: rows per step, so that K steps end within minutes
NOMINAL = {"int8_tops": 4500.0, "bf16_tflops": 2250.0, "hbm_gbs": 8000.0}  # 8 TB/s: the figure the decode target names
# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu capture summarised under profiles/
# (same kernel source, same shapes: T = 4096, K = 14336).
NCU_TRAFFIC_BYTES = {"project_gemm": 2.2e9}
METRIC, UNIT = "prefill tokens/s through one decoder block's ResQ linear layers", "tokens/s"


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_burst": d["bf16_tflops"], "bf16_sustained": d["bf16_tflops_sustained"],
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_burst": 1590.0, "bf16_sustained": 1400.0, "source": "fallback"}


def measure_int8_peak(torch, dev):
    """Same-box dense INT8 tensor-core rate: a library s8 x s8 -> s32 GEMM (torch._int_mm, cuBLASLt) at 8192^3, best of
    10 launches (burst) and back to back for about 2 s (sustained), like the driver-written bf16 peaks.  Context for
    the mixed GEMM's fraction only; nothing on the timed path calls it."""
    n = 8192
    a = torch.randint(-127, 128, (n, n), dtype=torch.int8, device=dev)
    b = torch.randint(-127, 128, (n, n), dtype=torch.int8, device=dev)
    ops = 2.0 * n ** 3
    try:
        for _ in range(3):
            torch._int_mm(a, b)
        torch.cuda.synchronize()
        best = float("inf")
        for _ in range(10):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            torch._int_mm(a, b)
            e1.record()
            e1.synchronize()
            best = min(best, e0.elapsed_time(e1))
        reps = max(10, int(2000.0 / best))
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            torch._int_mm(a, b)
        e1.record()
        e1.synchronize()
        sustained = e0.elapsed_time(e1) / reps
    except Exception as e:  # the library GEMM is context only: its absence must not fail the benchmark
        return {"unavailable": repr(e)[:200]}
    return {"burst": round(ops / (best * 1e-3) / 1e12, 1), "sustained": round(ops / (sustained * 1e-3) / 1e12, 1),
            "how": f"torch._int_mm {n}^3: best of 10, and {reps} back to back"}


# --------------------------------------------------------------------------------------- ranks
def max_over_ranks(ms: float, device) -> float:
    """The slowest rank's time: replicas run independently, the job is as fast as its slowest replica."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms)
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_value(tokens_per_rank: int, world: int, ms_per_step: float) -> float:
    """Whole-job throughput: every rank processes `tokens_per_rank` tokens per step (weak scaling)."""
    return world * tokens_per_rank / (ms_per_step * 1e-3)


# --------------------------------------------------------------------------------------- clocks
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_id: str):
        self.gpu_id, self.proc = gpu_id, None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", self.gpu_id, f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            time.sleep(0.3)  # let the first samples start
        except OSError:
            self.proc = None

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        out, _ = self.proc.communicate(timeout=10)
        sm, mx, pw, reasons = [], [], [], set()
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1])); pw.append(float(f[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(pw) if pw else None, "samples": len(sm), "reasons": sorted(reasons)}


# --------------------------------------------------------------------------------------- workload
class Layer:
    pass


def build_layers(device, rows=None, with_weights=True, only=None):
    """Seeded synthetic inputs of the workload on `device` (activations, projected weights, P)."""
    import synth
    rows = T_PREFILL if rows is None else rows
    layers = []
    for li, (name, K, N, online) in enumerate(LAYERS):
        if only and name not in only:
            continue
        L = Layer()
        L.name, L.K, L.N, L.r, L.online = name, K, N, K // 8, online
        L.X = synth.t_activations(rows, K, device, "t4", seed=synth.SEED_ACT + 10 * li)
        L.W_proj = synth.t_projected_weights_direct(N, K, device, seed=synth.SEED_W + 10 * li) if with_weights else None
        L.P = synth.t_kron_orthogonal_bf16(K, device) if online else None
        layers.append(L)
    return layers


def oracle_sample_step(layers_host):
    """One pass of the oracle over the sampled rows of every layer; returns the LayerResults."""
    import oracle
    out = []
    for L in layers_host:
        out.append(oracle.linear(L["X_bits"], L["P_bits"], L["pw"]))
    return out


def to_bits(t):
    import torch
    return t.contiguous().view(torch.int16).cpu().numpy().view("uint16")


def host_sample(layers, rows):
    """Copies the first `rows` rows of each layer's input and the full projected weights to the host
    and quantizes the weights with the oracle (untimed set-up of the CPU baseline)."""
    import oracle
    hs = []
    for L in layers:
        hs.append({"name": L.name, "X_bits": to_bits(L.X[:rows]), "P_bits": to_bits(L.P) if L.online else None,
                   "pw": oracle.pack_weights(L.W_proj.cpu().numpy(), L.r)})
    return hs


# --------------------------------------------------------------------------------------- decode leg
DECODE_T = (1, 4, 16)
HOST_LEAD_CYCLES = 60_000_000  # ~30 ms of device idling, enough for the host to enqueue a whole timed batch
DECODE_COPIES = 3  # distinct copies of the packed weights, cycled per step: one block's 123 MB would sit in the 126 MB L2


def decode_leg_with_clocks(gpu_id, *a):
    """decode_leg with the SM clock sampled over the leg (the timed chains last under a millisecond each, far below
    the sampling period, so the record covers the leg as a whole): adds `clocks` and, per T, the chain's time x the
    median clock in SM cycles, which is what to compare between boxes that settle at different clocks."""
    sampler = ClockSampler(gpu_id)
    sampler.start()
    out = decode_leg(*a)
    out["clocks"] = sampler.stop()
    mhz = out["clocks"].get("sm_mhz")
    if mhz:
        for k, v in out.items():
            if isinstance(v, dict) and "mixed_gemv_us" in v:
                v["mixed_gemv_sm_kcycles"] = round(v["mixed_gemv_us"] * mhz / 1e3, 1)
    return out


def decode_leg(resq, torch, dev, peaks, layers, steps):
    """Few-token variant of the same block: packed INT8 + nibble-packed INT4 weights with fp16 scales,
    streamed once per step.  Reports the weight-stream rate of the mixed GEMV kernels against the HBM
    peak, the P stream of the online projection separately, and the latency of the block's linears."""
    stream = torch.cuda.current_stream()

    def ev():
        e = torch.cuda.Event(enable_timing=True)
        e.record(stream)
        return e

    resq.resq_set_option(resq.OPT_DECODE_EARLY_WEIGHTS, 1)  # weights are packed once, long before any step
    sets, weight_bytes = [], 0
    for L in layers:
        desc = resq.layer_desc(L.K, L.N, L.r, resq.SCALE_FP16)
        base = resq.resq_pack_weights(desc, L.W_proj, with_w4_i8=False)
        copies = [base] + [resq.Weights(desc, base.w8.clone(), base.w4.clone(), base.s_w8.clone(), base.s_w4.clone())
                           for _ in range(DECODE_COPIES - 1)]
        sets.append((L, desc, copies))
        weight_bytes += L.N * (L.r + (L.K - L.r) // 2) + 2 * 2 * L.N
    p_bytes = sum(2 * L.K * L.K for L in layers if L.online)
    # The paper's own form of the layer that needs an online basis (Section 4.3): Hadamard U_D + uniform INT4 weights.
    had_sets = {}
    for L in layers:
        if L.online:
            d0 = resq.layer_desc(L.K, L.N, 0, resq.SCALE_FP16)
            b0 = resq.resq_pack_weights(d0, L.W_proj, with_w4_i8=False)
            had_sets[L.name] = (d0, [b0] + [resq.Weights(d0, b0.w8.clone() if b0.w8 is not None else None, b0.w4.clone(),
                                                         b0.s_w8.clone(), b0.s_w4.clone())
                                            for _ in range(DECODE_COPIES - 1)])
    out = {"workload": WORKLOAD.split("-prefill")[0] + "-decode", "weight_bytes_per_step": weight_bytes,
           "p_bytes_per_step": p_bytes, "weight_copies_cycled": DECODE_COPIES, "steps": steps}
    for T in DECODE_T:
        bufs = []
        for L, desc, _ in sets:
            K4 = L.K - L.r
            bufs.append(dict(X=L.X[:T].contiguous(), x8=torch.empty((T, L.r), dtype=torch.int8, device=dev),
                             x4=torch.empty((T, K4 // 2), dtype=torch.uint8, device=dev),
                             sx8=torch.empty(T, dtype=torch.float32, device=dev),
                             sx4=torch.empty(T, dtype=torch.float32, device=dev),
                             Y=torch.empty((T, L.N), dtype=torch.bfloat16, device=dev),
                             ws=resq.alloc_workspace(desc, T, L.online, False, device=dev)))

        def step(i, events=None):
            for (L, desc, copies), b in zip(sets, bufs):
                e0 = ev() if events is not None else None
                resq.resq_project_quantize(b["X"], L.P, L.r, b["x8"], b["x4"], b["sx8"], b["sx4"], None,
                                           b["ws"] if L.online else None)
                e1 = ev() if events is not None else None
                resq.resq_mixed_gemm(copies[i % DECODE_COPIES], b["x8"], b["x4"], b["sx8"], b["sx4"], b["Y"], b["ws"])
                if events is not None:
                    events.append((L, e0, e1, ev()))

        for i in range(3):
            step(i)
        torch.cuda.synchronize()
        events = []
        torch.cuda._sleep(HOST_LEAD_CYCLES)  # the host queues the whole batch while the device idles on this
        t0 = ev()
        for i in range(steps):
            step(i, events)
        t1 = ev()
        torch.cuda.synchronize()
        gemv_iso = sum(e1.elapsed_time(e2) for _, _, e1, e2 in events) / steps
        quant = sum(e0.elapsed_time(e1) for L, e0, e1, _ in events if not L.online) / steps
        proj = sum(e0.elapsed_time(e1) for L, e0, e1, _ in events if L.online) / steps
        # The mixed GEMV kernels of the block back to back on the codes of the last step, no events
        # between them: one launch's average duration in the stream = span / launches.
        torch.cuda._sleep(HOST_LEAD_CYCLES)
        c0 = ev()
        for i in range(steps):
            for (L, desc, copies), b in zip(sets, bufs):
                resq.resq_mixed_gemm(copies[i % DECODE_COPIES], b["x8"], b["x4"], b["sx8"], b["sx4"], b["Y"], b["ws"])
        c1 = ev()
        # The whole block (quantize + GEMV per layer, online projection for down), no events inside.
        torch.cuda._sleep(HOST_LEAD_CYCLES)
        t0 = ev()
        for i in range(steps):
            step(i)
        t1 = ev()
        torch.cuda.synchronize()
        # The block through resq_linear, the call a user makes: row quantizer + streaming kernel per layer without P;
        # down_proj runs projection, slice reduction, row quantizer and the streaming kernel.
        def linear_chain(i):
            for (L, desc, copies), b in zip(sets, bufs):
                resq.resq_linear(copies[i % DECODE_COPIES], b["X"], L.P if L.online else None, b["Y"], b["ws"])

        for i in range(3):
            linear_chain(i)
        torch.cuda.synchronize()
        torch.cuda._sleep(HOST_LEAD_CYCLES)
        l0 = ev()
        for i in range(steps):
            linear_chain(i)
        l1 = ev()
        torch.cuda.synchronize()
        total_linear = l0.elapsed_time(l1) / steps
        # The same calls recorded once into a CUDA graph (one graph = DECODE_COPIES steps, so that the weight copies
        # still cycle) and replayed: the library allocates nothing and never synchronises, so its calls can be captured.
        total_graph = None
        try:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                for i in range(DECODE_COPIES):
                    linear_chain(i)
            reps = max(1, steps // DECODE_COPIES)
            for _ in range(2):
                g.replay()
            torch.cuda.synchronize()
            torch.cuda._sleep(HOST_LEAD_CYCLES)
            g0 = ev()
            for _ in range(reps):
                g.replay()
            g1 = ev()
            torch.cuda.synchronize()
            total_graph = g0.elapsed_time(g1) / (reps * DECODE_COPIES)
        except RuntimeError as e:
            print(f"[bench] graph capture of the few-token block failed: {e}", file=sys.stderr)
            torch.cuda.synchronize()
        # The same block with the Hadamard form of the online layer(s).
        hb = {}
        for (L, desc, _), b in zip(sets, bufs):
            if L.online:
                d0 = had_sets[L.name][0]
                hb[L.name] = dict(x4=torch.empty((T, L.K // 2), dtype=torch.uint8, device=dev),
                                  s8=torch.empty(T, dtype=torch.float32, device=dev),
                                  s4=torch.empty(T, dtype=torch.float32, device=dev),
                                  ws=resq.alloc_workspace(d0, T, False, False, device=dev))

        def hadamard_chain(i):
            for (L, desc, copies), b in zip(sets, bufs):
                if L.online:
                    h = hb[L.name]
                    resq.resq_hadamard_quantize(b["X"], 0, None, h["x4"], h["s8"], h["s4"], None)
                    resq.resq_mixed_gemm(had_sets[L.name][1][i % DECODE_COPIES], None, h["x4"], h["s8"], h["s4"], b["Y"], h["ws"])
                else:
                    resq.resq_linear(copies[i % DECODE_COPIES], b["X"], None, b["Y"], b["ws"])

        total_hadamard = None
        try:
            for i in range(3):
                hadamard_chain(i)
            torch.cuda.synchronize()
            torch.cuda._sleep(HOST_LEAD_CYCLES)
            h0 = ev()
            for i in range(steps):
                hadamard_chain(i)
            h1 = ev()
            torch.cuda.synchronize()
            total_hadamard = h0.elapsed_time(h1) / steps
        except resq.ResqError:   # a width the Hadamard kernel or the streaming kernel's staging does not take
            torch.cuda.synchronize()
        # The same GEMV chain with asymmetric activation codes (unsigned codes, zero-points, weight row sums).
        ab = []
        for (L, desc, copies), b in zip(sets, bufs):
            K4 = L.K - L.r
            z = lambda *shape, dt=torch.float32: torch.empty(shape, dtype=dt, device=dev)
            a = dict(u8=z(T, L.r, dt=torch.uint8), u4=z(T, K4 // 2, dt=torch.uint8), sx8=z(T), sx4=z(T), zx8=z(T),
                     zx4=z(T), wsp=resq.alloc_workspace_asym(desc, T, False, False, device=dev))
            a["ws8"], a["ws4"] = resq.resq_weight_row_sums(copies[0])
            Xc = b["X"] if not L.online else L.X[:T, :L.K].contiguous()   # codes of raw rows: same cost, no projection
            resq.resq_project_quantize_asym(Xc, None, L.r, a["u8"], a["u4"], a["sx8"], a["sx4"], a["zx8"], a["zx4"])
            ab.append(a)

        def asym_chain(i):
            for (L, desc, copies), b, a in zip(sets, bufs, ab):
                resq.resq_mixed_gemm_asym(copies[i % DECODE_COPIES], a["ws8"], a["ws4"], a["u8"], a["u4"], a["sx8"],
                                          a["sx4"], a["zx8"], a["zx4"], b["Y"], a["wsp"])

        for i in range(3):
            asym_chain(i)
        torch.cuda.synchronize()
        torch.cuda._sleep(HOST_LEAD_CYCLES)
        a0 = ev()
        for i in range(steps):
            asym_chain(i)
        a1 = ev()
        torch.cuda.synchronize()
        gemv_asym = a0.elapsed_time(a1) / steps
        gemv = c0.elapsed_time(c1) / steps
        total = t0.elapsed_time(t1) / steps
        gbs = weight_bytes / (gemv * 1e-3) / 1e9
        out[f"T{T}"] = {"mixed_gemv_us": round(gemv * 1e3, 2), "mixed_gemv_sum_of_isolated_us": round(gemv_iso * 1e3, 2),
                        "weight_stream_gbs": round(gbs, 1),
                        "frac_of_hbm_peak": round(gbs / peaks["hbm_gbs"], 4),
                        "frac_of_nominal_8000": round(gbs / NOMINAL["hbm_gbs"], 4),
                        "asymmetric_mixed_gemv_us": round(gemv_asym * 1e3, 2),
                        "asymmetric_weight_stream_gbs": round(weight_bytes / (gemv_asym * 1e-3) / 1e9, 1),
                        "folded_quantize_us": round(quant * 1e3, 2),
                        "online_projection_us": round(proj * 1e3, 2),
                        "online_projection_p_stream_gbs": round(p_bytes / (proj * 1e-3) / 1e9, 1) if proj > 0 else None,
                        "block_split_calls_us": round(total * 1e3, 2),
                        "block_linears_us": round(total_linear * 1e3, 2),
                        "tokens_per_s": round(T / (total_linear * 1e-3), 1),
                        "block_linears_cuda_graph_us": round(total_graph * 1e3, 2) if total_graph else None,
                        "block_linears_hadamard_down_us": round(total_hadamard * 1e3, 2) if total_hadamard else None,
                        "tokens_per_s_hadamard_down": round(T / (total_hadamard * 1e-3), 1) if total_hadamard else None}
    resq.resq_set_option(resq.OPT_DECODE_EARLY_WEIGHTS, 0)
    st = resq.resq_device_status()
    if st != resq.OK:
        raise SystemExit(f"device status {st}: {resq.status_string(st)}")
    return out


# --------------------------------------------------------------------------------------- asymmetric leg
def asym_leg(resq, torch, dev, layers, T, steps):
    """One pass of the block with asymmetric per-token activation codes (unsigned codes + zero-points,
    u8 x s8 products, rank-one zero-point terms in the epilogue); the weights are those of the main leg."""
    stream = torch.cuda.current_stream()

    def ev():
        e = torch.cuda.Event(enable_timing=True)
        e.record(stream)
        return e

    bufs = []
    for L in layers:
        K4 = L.K - L.r
        z = lambda *shape, dt=torch.float32: torch.empty(shape, dtype=dt, device=dev)
        bufs.append(dict(ws8=None, Y=torch.empty_like(L.Y), u8=z(T, L.r, dt=torch.uint8), u4e=z(T, K4, dt=torch.uint8), sx8=z(T), sx4=z(T),
                         zx8=z(T), zx4=z(T), wsp=resq.alloc_workspace_asym(L.desc, T, L.online, True, device=dev)))
        bufs[-1]["ws8"], bufs[-1]["ws4"] = resq.resq_weight_row_sums(L.W)

    def step(events=None):
        for L, b in zip(layers, bufs):
            e0 = ev() if events is not None else None
            resq.resq_project_quantize_asym(L.X, L.P, L.r, b["u8"], None, b["sx8"], b["sx4"], b["zx8"], b["zx4"], b["u4e"],
                                            b["wsp"] if L.online else None)
            e1 = ev() if events is not None else None
            resq.resq_mixed_gemm_asym(L.W, b["ws8"], b["ws4"], b["u8"], None, b["sx8"], b["sx4"], b["zx8"], b["zx4"], b["Y"],
                                      b["wsp"], u4_u8=b["u4e"])
            if events is not None:
                events.append((L, e0, e1, ev()))

    for _ in range(3):
        step()
    torch.cuda.synchronize()
    events = []
    t0 = ev()
    for _ in range(steps):
        step(events)
    t1 = ev()
    torch.cuda.synchronize()
    ms = t0.elapsed_time(t1) / steps
    per_layer, ops, g_ms = {}, 0.0, 0.0
    for L in layers:
        q = statistics.mean(e0.elapsed_time(e1) for l, e0, e1, _ in events if l is L)
        g = statistics.mean(e1.elapsed_time(e2) for l, _, e1, e2 in events if l is L)
        per_layer[L.name] = {"quantize_ms": round(q, 4), "mixed_gemm_ms": round(g, 4),
                             "mixed_gemm_tops": round(2.0 * T * L.K * L.N / (g * 1e-3) / 1e12, 1)}
        ops += 2.0 * T * L.K * L.N
        g_ms += g
    st = resq.resq_device_status()
    if st != resq.OK:
        raise SystemExit(f"device status {st}: {resq.status_string(st)}")
    return {"workload": WORKLOAD + "-asymmetric-activations", "steps": steps, "ms_per_step": round(ms, 4),
            "tokens_per_s": round(T / (ms * 1e-3), 1), "mixed_gemm_tops": round(ops / (g_ms * 1e-3) / 1e12, 1),
            "per_layer": per_layer}


# --------------------------------------------------------------------------------------- Hadamard leg
def hadamard_leg(resq, torch, dev, L, T, steps, peaks):
    """down_proj as the paper runs it (Section 4.3): Hadamard transform fused with uniform INT4 quantization of
    the input, uniform INT4 weights (r = 0), instead of the dense bf16 projection with a mixed 8/4 split."""
    stream = torch.cuda.current_stream()

    def ev():
        e = torch.cuda.Event(enable_timing=True)
        e.record(stream)
        return e

    desc = resq.layer_desc(L.K, L.N, 0)
    W = resq.resq_pack_weights(desc, L.W_proj, with_w4_i8=True)   # stands in for (H^T W / sqrt(K))^T: same distribution
    x4e = torch.empty((T, L.K), dtype=torch.int8, device=dev)
    s8 = torch.empty(T, dtype=torch.float32, device=dev)
    s4 = torch.empty(T, dtype=torch.float32, device=dev)
    ws = resq.alloc_workspace(desc, T, False, True, device=dev)
    Y = torch.empty_like(L.Y)  # the main leg's outputs stay untouched for the parity spot check

    def step(events=None):
        e0 = ev() if events is not None else None
        resq.resq_hadamard_quantize(L.X, 0, None, None, s8, s4, x4e)
        e1 = ev() if events is not None else None
        resq.resq_mixed_gemm(W, None, None, s8, s4, Y, ws, x4_i8=x4e)
        if events is not None:
            events.append((e0, e1, ev()))

    for _ in range(3):
        step()
    torch.cuda.synchronize()
    events = []
    for _ in range(steps):
        step(events)
    torch.cuda.synchronize()
    q = statistics.mean(a.elapsed_time(b) for a, b, _ in events)
    g = statistics.mean(b.elapsed_time(c) for _, b, c in events)
    st = resq.resq_device_status()
    if st != resq.OK:
        raise SystemExit(f"device status {st}: {resq.status_string(st)}")
    # The same layer for a generation step (T = 1, 4, 16): transform + quantize, then the streaming kernel on packed
    # INT4 weights; five weight copies (> L2 together) are cycled so that every weight byte comes from DRAM.
    copies = [resq.resq_pack_weights(desc, L.W_proj, with_w4_i8=False) for _ in range(5)]
    few = {}
    for Tf in DECODE_T:
        Xf = L.X[:Tf].contiguous()
        x4 = torch.empty((Tf, L.K // 2), dtype=torch.uint8, device=dev)
        f8 = torch.empty(Tf, dtype=torch.float32, device=dev)
        f4 = torch.empty(Tf, dtype=torch.float32, device=dev)
        Yf = torch.empty((Tf, L.N), dtype=torch.bfloat16, device=dev)
        wsf = resq.alloc_workspace(desc, Tf, False, False, device=dev)

        def few_step(i, events=None):
            e0 = ev() if events is not None else None
            resq.resq_hadamard_quantize(Xf, 0, None, x4, f8, f4, None)
            e1 = ev() if events is not None else None
            resq.resq_mixed_gemm(copies[i % len(copies)], None, x4, f8, f4, Yf, wsf)
            if events is not None:
                events.append((e0, e1, ev()))

        try:
            for i in range(3):
                few_step(i)
        except resq.ResqError as e:   # e.g. 16 rows of 28672 uniform INT4 codes do not fit the streaming kernel's staging
            few[f"T{Tf}"] = {"unsupported": str(e)}
            continue
        torch.cuda.synchronize()
        fev = []
        for i in range(steps):
            few_step(i, fev)
        torch.cuda.synchronize()
        torch.cuda._sleep(HOST_LEAD_CYCLES)
        c0 = ev()
        for i in range(steps):
            few_step(i)
        c1 = ev()
        torch.cuda.synchronize()
        few[f"T{Tf}"] = {"hadamard_quantize_us": round(statistics.mean(a.elapsed_time(b) for a, b, _ in fev) * 1e3, 2),
                         "int4_gemv_us": round(statistics.mean(b.elapsed_time(c) for _, b, c in fev) * 1e3, 2),
                         "layer_us": round(c0.elapsed_time(c1) / steps * 1e3, 2)}
    st = resq.resq_device_status()
    if st != resq.OK:
        raise SystemExit(f"device status {st}: {resq.status_string(st)}")
    bytes_q = T * (2.0 * L.K + L.K + 8)   # read bf16, write one code per byte + scales
    return {"workload": f"down_proj {L.K}->{L.N}, T={T}: Hadamard U_D + uniform INT4 (r = 0)", "steps": steps,
            "few_tokens": few,
            "hadamard_quantize_ms": round(q, 4), "hadamard_quantize_gbs": round(bytes_q / (q * 1e-3) / 1e9, 1),
            "hadamard_quantize_frac_of_hbm_peak": round(bytes_q / (q * 1e-3) / 1e9 / peaks["hbm_gbs"], 4),
            "int4_gemm_ms": round(g, 4), "int4_gemm_tops": round(2.0 * T * L.K * L.N / (g * 1e-3) / 1e12, 1),
            "layer_ms": round(q + g, 4)}


# --------------------------------------------------------------------------------------- attention-block leg
KV_HQ, KV_HKV, KV_D = 32, 8, 128   # Llama-3-8B attention geometry


def kv_leg(resq, torch, dev, peaks, steps, n_seqs=16, seq_len=8192, prefill_T=4096):
    """The attention-block path (Section 4.3, Eq. 8; Section 5.1): 8-bit U_C projection of query and key, the
    per-head 8/4-bit KV cache, and single-query attention over it for `n_seqs` sequences of `seq_len` cached
    positions.  Two cache copies (each larger than L2) are cycled so that every timed byte comes from DRAM."""
    import numpy as np
    import synth
    from paper_2412_14363_b200 import kv
    stream = torch.cuda.current_stream()

    def ev():
        e = torch.cuda.Event(enable_timing=True)
        e.record(stream)
        return e

    def timed(fn, n):
        for i in range(3):
            fn(i)
        torch.cuda.synchronize()
        t0 = ev()
        for i in range(n):
            fn(i)
        t1 = ev()
        torch.cuda.synchronize()
        return t0.elapsed_time(t1) / n

    W_C = torch.from_numpy(np.ascontiguousarray(synth.haar_orthogonal(KV_D).T.astype(np.float32))).to(dev)
    wq, s_u = kv.resq_uc_quantize(W_C)
    caches = [kv.KvCache(n_seqs, KV_HKV, seq_len, device=dev) for _ in range(2)]
    pos = torch.arange(seq_len, dtype=torch.int32, device=dev)
    for b in range(n_seqs):   # fill through the library's own append (checked against the oracle in the tests)
        k = synth.t_head_vectors(seq_len, KV_HKV, KV_D, dev, stream=1000 + b, lead=1.0, scale=1.5)
        v = synth.t_head_vectors(seq_len, KV_HKV, KV_D, dev, stream=2000 + b, lead=4.0, shift=0.2)
        ids = torch.full((seq_len,), b, dtype=torch.int32, device=dev)
        for c in caches:
            kv.resq_kv_append(c, k, v, ids, pos, wq, s_u)
    q = synth.t_head_vectors(n_seqs, KV_HQ, KV_D, dev, stream=3000, lead=1.0, scale=1.5)
    q16 = torch.empty((n_seqs, KV_HQ, KV_D), dtype=torch.float16, device=dev)
    out = torch.empty((n_seqs, KV_HQ, KV_D), dtype=torch.float32, device=dev)
    lens = torch.full((n_seqs,), seq_len, dtype=torch.int32, device=dev)
    ws = kv.attention_workspace(caches[0], KV_HQ)
    kv.resq_query_project(q, wq, s_u, q16)
    attn_ms = timed(lambda i: kv.resq_attention_decode(caches[i % 2], q16, lens, out, ws), steps)
    cache_bytes = caches[0].nbytes
    # one generation step's cache update and query projection (launch-latency sized)
    k1 = synth.t_head_vectors(n_seqs, KV_HKV, KV_D, dev, stream=3001, lead=1.0)
    v1 = synth.t_head_vectors(n_seqs, KV_HKV, KV_D, dev, stream=3002)
    ids1 = torch.arange(n_seqs, dtype=torch.int32, device=dev)
    pos1 = torch.full((n_seqs,), seq_len - 1, dtype=torch.int32, device=dev)
    app1_ms = timed(lambda i: kv.resq_kv_append(caches[i % 2], k1, v1, ids1, pos1, wq, s_u), steps)
    qp1_ms = timed(lambda i: kv.resq_query_project(q, wq, s_u, q16), steps)
    fused1_ms = timed(lambda i: kv.resq_qkv_project_append(caches[i % 2], q, q16, k1, v1, ids1, pos1, wq, s_u), steps)
    # prefill-sized update: prefill_T tokens of one sequence
    T = min(prefill_T, seq_len)
    kp = synth.t_head_vectors(T, KV_HKV, KV_D, dev, stream=3003, lead=1.0)
    vp = synth.t_head_vectors(T, KV_HKV, KV_D, dev, stream=3004)
    qp = synth.t_head_vectors(T, KV_HQ, KV_D, dev, stream=3005, lead=1.0)
    qp16 = torch.empty((T, KV_HQ, KV_D), dtype=torch.float16, device=dev)
    idsp = torch.zeros(T, dtype=torch.int32, device=dev)
    appp_ms = timed(lambda i: kv.resq_kv_append(caches[i % 2], kp, vp, idsp, pos[:T], wq, s_u), steps)
    qpp_ms = timed(lambda i: kv.resq_query_project(qp, wq, s_u, qp16), steps)
    # many-query (causal prefill) attention of the last Tp tokens of one full sequence: every row streams its own prefix
    Tp = min(1024, seq_len)
    qa16 = torch.empty((Tp, KV_HQ, KV_D), dtype=torch.float16, device=dev)
    kv.resq_query_project(qp[:Tp], wq, s_u, qa16)
    oa = torch.empty((Tp, KV_HQ, KV_D), dtype=torch.float32, device=dev)
    qs = torch.zeros(Tp, dtype=torch.int32, device=dev)
    ql = torch.arange(seq_len - Tp + 1, seq_len + 1, dtype=torch.int32, device=dev)
    wsq = torch.empty(int(resq.lib.resq_attention_queries_workspace_bytes(Tp, KV_HQ, KV_HKV, KV_D)), dtype=torch.uint8, device=dev)
    mq_ms = timed(lambda i: kv.resq_attention_queries(caches[i % 2], qa16, qs, ql, oa, wsq), max(3, steps // 4))
    mq_blocks = int(((ql + 31) // 32).sum().item()) * KV_HKV
    # the same rows tile-wise on the tensor cores, then the causal attention of the whole sequence
    pf_ms = timed(lambda i: kv.resq_attention_prefill(caches[i % 2], qa16, 0, seq_len - Tp, oa), max(3, steps // 4))
    pf_flops = 4.0 * KV_D * KV_HQ * float(ql.sum().item())
    Tf = min(seq_len, 8192)
    qf16 = torch.empty((Tf, KV_HQ, KV_D), dtype=torch.float16, device=dev)
    for t0 in range(0, Tf, T):
        kv.resq_query_project(qp[:min(T, Tf - t0)], wq, s_u, qf16[t0:t0 + min(T, Tf - t0)])
    of = torch.empty((Tf, KV_HQ, KV_D), dtype=torch.float32, device=dev)
    full_ms = timed(lambda i: kv.resq_attention_prefill(caches[i % 2], qf16, 0, 0, of), max(3, steps // 4))
    full_flops = 4.0 * KV_D * KV_HQ * (Tf * (Tf + 1) / 2)
    app_bytes = T * KV_HKV * (2 * 2 * KV_D + 2 * 88)
    qp_bytes = T * KV_HQ * (2 * KV_D + 2 * KV_D)
    st = resq.resq_device_status()
    if st != resq.OK:
        raise SystemExit(f"device status {st}: {resq.status_string(st)}")
    gbs = cache_bytes / (attn_ms * 1e-3) / 1e9
    return {"workload": f"llama3-8b attention, {KV_HQ} query / {KV_HKV} KV heads x {KV_D}: {n_seqs} sequences x {seq_len} cached positions",
            "steps": steps, "cache_bytes": cache_bytes, "bytes_per_head_vector": 88, "vs_bf16_cache": round(256 / 88, 2),
            "attention_decode_us": round(attn_ms * 1e3, 2), "attention_cache_stream_gbs": round(gbs, 1),
            "attention_frac_of_hbm_peak": round(gbs / peaks["hbm_gbs"], 4),
            "decode_step_kv_append_us": round(app1_ms * 1e3, 2), "decode_step_query_project_us": round(qp1_ms * 1e3, 2),
            "decode_step_fused_project_append_us": round(fused1_ms * 1e3, 2),
            "prefill_tokens": T, "prefill_kv_append_us": round(appp_ms * 1e3, 2),
            "prefill_kv_append_gbs": round(app_bytes / (appp_ms * 1e-3) / 1e9, 1),
            "prefill_query_project_us": round(qpp_ms * 1e3, 2),
            "prefill_query_project_gbs": round(qp_bytes / (qpp_ms * 1e-3) / 1e9, 1),
            "many_query_attention": {"queries": Tp, "prefix_positions": f"{seq_len - Tp + 1}..{seq_len}",
                                     "us": round(mq_ms * 1e3, 1),
                                     "cache_block_reads_gbs": round(mq_blocks * 5632 / (mq_ms * 1e-3) / 1e9, 1),
                                     "note": "each query row streams its own prefix (L2-resident): batched single-query passes"},
            "prefill_attention": {"kernel": "attention_prefill_kernel (tcgen05 kind::f16, 128 rows x 64 positions per step)",
                                  "chunk": {"queries": Tp, "prefix_positions": f"{seq_len - Tp + 1}..{seq_len}",
                                            "us": round(pf_ms * 1e3, 1), "tflops": round(pf_flops / (pf_ms * 1e-3) / 1e12, 1),
                                            "vs_many_query_call": round(mq_ms / pf_ms, 2)},
                                  "whole_sequence": {"tokens": Tf, "us": round(full_ms * 1e3, 1),
                                                     "tflops": round(full_flops / (full_ms * 1e-3) / 1e12, 1)},
                                  "flops": "4 d_head per (query head, attended position): both products, causal part only"}}


# --------------------------------------------------------------------------------------- projection GEMM study
def project_study(resq, torch, dev, peaks, T, launches=60):
    """The online projection GEMM of the block's down_proj alone, `launches` times back to back, with the SM clock
    sampled alongside: time per launch, TFLOP/s, and SM cycles per K block of one CTA pair (time x median MHz over
    the K blocks a pair executes), so that runs at different clocks or widths can be compared."""
    import synth
    name, K, N, _ = [l for l in LAYERS if l[3]][0]
    X = synth.t_activations(T, K, dev, "t4", seed=synth.SEED_ACT)
    P = synth.t_kron_orthogonal_bf16(K, dev)
    C = torch.empty((min(T, 4096), K), dtype=torch.float32, device=dev)
    ws = torch.empty(resq.resq_project_workspace_bytes(), dtype=torch.uint8, device=dev)
    rows = C.shape[0]
    Xp = X[:rows].contiguous()
    for _ in range(3):
        resq.resq_project(Xp, P, C, ws)
    torch.cuda.synchronize()
    gpu_id = str(getattr(torch.cuda.get_device_properties(dev), "uuid", 0))
    if not gpu_id.startswith("GPU-") and "-" in gpu_id:
        gpu_id = "GPU-" + gpu_id
    sampler = ClockSampler(gpu_id)
    sampler.start()
    evs = []
    for _ in range(launches):
        a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
        a.record()
        resq.resq_project(Xp, P, C, ws)
        b.record()
        evs.append((a, b))
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = sorted(a.elapsed_time(b) for a, b in evs)
    med = ms[len(ms) // 2]
    tiles = ((rows + 255) // 256) * ((K + 255) // 256)
    kblocks_per_pair = tiles / 74.0 * (K / 64.0)   # 64 bf16 elements (128 bytes) per K block
    mhz = clocks.get("sm_mhz") or 0.0
    st = resq.resq_device_status()
    if st != resq.OK:
        raise SystemExit(f"device status {st}: {resq.status_string(st)}")
    return {"layer": f"{name} {K}x{K} P, {rows} token rows", "launches": launches, "ms_median": round(med, 4),
            "ms_min": round(ms[0], 4), "ms_max": round(ms[-1], 4),
            "tflops_median": round(2.0 * rows * K * K / (med * 1e-3) / 1e12, 1),
            "frac_of_bf16_burst": round(2.0 * rows * K * K / (med * 1e-3) / 1e12 / peaks["bf16_burst"], 4),
            "frac_of_bf16_sustained": round(2.0 * rows * K * K / (med * 1e-3) / 1e12 / peaks["bf16_sustained"], 4),
            "sm_mhz_median": mhz, "clocks": clocks,
            "sm_cycles_per_k_block": round(med * 1e-3 * mhz * 1e6 / kblocks_per_pair, 1) if mhz else None,
            "nominal_cycles_per_k_block": round(256 * 256 * 64 * 2 / (2 * NOMINAL["bf16_tflops"] * 1e12 / 148 / 1.965e9), 1),   # 256 x 256 x 64 multiply-adds per pair
            "tiles": tiles, "rounds_of_74_pairs": round(tiles / 74.0, 2)}


# --------------------------------------------------------------------------------------- our arm
def run_ours(args):
    import numpy as np
    import torch
    import torch.distributed as dist

    import paper_2412_14363_b200 as resq

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    peaks = load_peaks()
    T = T_PREFILL

    if args.project_study:  # profiling runs: the projection GEMM alone with the clock alongside
        print(json.dumps({"project_gemm_study": project_study(resq, torch, dev, peaks, T)}))
        return
    only = [x for x in args.layers.split(",") if x]
    layers = build_layers(dev, only=only)
    for L in layers:
        L.desc = resq.layer_desc(L.K, L.N, L.r)
        L.W = resq.resq_pack_weights(L.desc, L.W_proj, with_w4_i8=True)
        K4 = L.K - L.r
        L.x8 = torch.empty((T, L.r), dtype=torch.int8, device=dev)
        L.x4e = torch.empty((T, K4), dtype=torch.int8, device=dev)
        L.sx8 = torch.empty(T, dtype=torch.float32, device=dev)
        L.sx4 = torch.empty(T, dtype=torch.float32, device=dev)
        L.Y = torch.empty((T, L.N), dtype=torch.bfloat16, device=dev)
        L.ws = resq.alloc_workspace(L.desc, T, L.online, True, device=dev)
    torch.cuda.synchronize()
    stream = torch.cuda.current_stream()

    def ev():
        e = torch.cuda.Event(enable_timing=True)
        e.record(stream)
        return e

    # One step; with `events` an event is recorded after every C-ABI call so that each kernel's time
    # is measured live on the launching stream.
    # Kernels of this library per step are counted by the library itself (resq_launch_count): 4 split-quantize,
    # 1 projection GEMM (+ its slice reduction when the last round of tiles is cut along K), 4 mixed GEMM.

    def step(events=None):
        for L in layers:
            e0 = ev() if events is not None else None
            resq.resq_project_quantize(L.X, L.P, L.r, L.x8, None, L.sx8, L.sx4, L.x4e, L.ws if L.online else None)
            e1 = ev() if events is not None else None
            resq.resq_mixed_gemm(L.W, L.x8, None, L.sx8, L.sx4, L.Y, L.ws, x4_i8=L.x4e)
            if events is not None:
                events.append((L.name, e0, e1, ev()))

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    gpu_id = str(getattr(torch.cuda.get_device_properties(dev), "uuid", local_rank))
    if not gpu_id.startswith("GPU-") and "-" in gpu_id:
        gpu_id = "GPU-" + gpu_id

    if args.kv_only:  # profiling runs: the attention-block leg alone
        print(json.dumps({"kv_cache_path": kv_leg(resq, torch, dev, peaks, max(5, min(args.steps, 20)), args.kv_seqs,
                                                  args.kv_len)}))
        return
    if args.decode_only:  # profiling runs: the few-token leg alone
        print(json.dumps({"decode": decode_leg_with_clocks(gpu_id, resq, torch, dev, peaks, layers, max(5, min(args.steps, 20)))}))
        return

    for _ in range(max(args.warmup, 3)):
        step()
    st = resq.resq_device_status()
    if st != resq.OK:
        raise SystemExit(f"device status {st}: {resq.status_string(st)}")

    sampler = ClockSampler(gpu_id)
    sampler.start()
    events = []
    barrier()
    launches0 = resq.resq_launch_count()
    t_start = ev()
    for _ in range(args.steps):
        step(events)
    t_end = ev()
    gpu_launches = resq.resq_launch_count() - launches0
    barrier()
    clocks = sampler.stop()
    ms_total = t_start.elapsed_time(t_end)
    ms_total = max_over_ranks(ms_total, dev)
    ms_per_step = ms_total / args.steps
    value = job_value(T, world, ms_per_step)

    # ---- per-kernel times (this rank), averaged over the timed steps
    kq = {L.name: [] for L in layers}
    kg = {L.name: [] for L in layers}
    for name, e0, e1, e2 in events:
        kq[name].append(e0.elapsed_time(e1))
        kg[name].append(e1.elapsed_time(e2))
    per_layer = {}
    gemm_ops = gemm_ms = 0.0
    quant_bytes = quant_ms = 0.0
    for L in layers:
        q_ms, g_ms = statistics.mean(kq[L.name]), statistics.mean(kg[L.name])
        ops = 2.0 * T * L.K * L.N
        per_layer[L.name] = {"K": L.K, "N": L.N, "quantize_ms": round(q_ms, 4), "mixed_gemm_ms": round(g_ms, 4),
                             "mixed_gemm_tops": round(ops / (g_ms * 1e-3) / 1e12, 1)}
        gemm_ops += ops
        gemm_ms += g_ms
        if not L.online:
            # per token: read 2K bytes of bf16, write r + (K - r) codes + 8 bytes of scales
            quant_bytes += T * (2.0 * L.K + L.K + 8)
            quant_ms += q_ms
    online = [L for L in layers if L.online]
    proj_ms = sum(per_layer[L.name]["quantize_ms"] for L in online)  # projection GEMM + its split-quantize pass
    proj_flops = sum(2.0 * T * L.K * L.K for L in online)
    timed_seconds = ms_total * 1e-3
    bf16_peak = peaks["bf16_sustained"] if timed_seconds > 1.0 else peaks["bf16_burst"]
    peak_kind = ("sustained" if timed_seconds > 1.0 else "burst") + " of " + peaks["source"]
    # INT8 denominators: the measured bf16 peak x the nominal INT8/bf16 ratio (4500/2250), a library INT8 GEMM
    # measured on this machine in this run (rank 0), and the nominal figure.
    int8_peak = 2.0 * bf16_peak
    int8_measured = measure_int8_peak(torch, dev) if rank == 0 and not args.no_int8_peak else None
    gemm_tops = gemm_ops / (gemm_ms * 1e-3) / 1e12
    kernels = {
        "mixed_gemm": {"bound": "tensor", "dtype": "int8", "achieved": round(gemm_tops, 1),
                       "peak": round(int8_peak, 1), "unit": "TOP/s", "ms_per_step": round(gemm_ms, 4),
                       "frac_of_nominal_4500": round(gemm_tops / NOMINAL["int8_tops"], 4)},
    }
    int8_fracs = {"vs_measured_bf16_x2": round(gemm_tops / int8_peak, 4),
                  "vs_nominal_4500": round(gemm_tops / NOMINAL["int8_tops"], 4)}
    if int8_measured and "burst" in int8_measured:
        int8_fracs["vs_measured_int8_gemm_burst"] = round(gemm_tops / int8_measured["burst"], 4)
        int8_fracs["vs_measured_int8_gemm_sustained"] = round(gemm_tops / int8_measured["sustained"], 4)
    if online:
        kernels["project_gemm+quantize"] = {"bound": "tensor", "dtype": "bf16",
                                            "achieved": round(proj_flops / (proj_ms * 1e-3) / 1e12, 1),
                                            "peak": round(bf16_peak, 1), "unit": "TFLOP/s", "ms_per_step": round(proj_ms, 4)}
    if quant_ms > 0:
        kernels["split_quantize"] = {"bound": "hbm", "dtype": "f32",
                                     "achieved": round(quant_bytes / (quant_ms * 1e-3) / 1e9, 1),
                                     "peak": peaks["hbm_gbs"], "unit": "GB/s", "ms_per_step": round(quant_ms, 4)}
    # The projection GEMM alone (its own C-ABI call), so that the dominant kernel has its own launch time.
    for L in online:
        Cpanel = torch.empty((T, L.K), dtype=torch.float32, device=dev)
        Cscratch = torch.empty(resq.resq_project_workspace_bytes(), dtype=torch.uint8, device=dev)
        for _ in range(3):
            resq.resq_project(L.X, L.P, Cpanel, Cscratch)
        pe = []
        for _ in range(max(5, min(args.steps, 10))):
            a = ev()
            resq.resq_project(L.X, L.P, Cpanel, Cscratch)
            pe.append((a, ev()))
        torch.cuda.synchronize()
        g_ms = statistics.mean(a.elapsed_time(b) for a, b in pe)
        del Cpanel
        kernels["project_gemm"] = {"bound": "tensor", "dtype": "bf16",
                                   "achieved": round(2.0 * T * L.K * L.K / (g_ms * 1e-3) / 1e12, 1),
                                   "peak": round(bf16_peak, 1), "unit": "TFLOP/s", "ms_per_step": round(g_ms, 4),
                                   "traffic": NCU_TRAFFIC_BYTES.get("project_gemm") if MODEL == "8b" else None}
    for k in kernels.values():
        k["frac"] = round(k["achieved"] / k["peak"], 4)
    # Dominant kernel: the single launch with the most time per step (the combined figure of the online
    # layer stays in the table but is two launches).
    dom_name = max((k for k in kernels if k != "project_gemm+quantize"), key=lambda k: kernels[k]["ms_per_step"])
    dom = kernels[dom_name]
    roofline = {"kernel": dom_name, "bound": dom["bound"], "achieved": dom["achieved"], "peak": dom["peak"],
                "unit": dom["unit"], "frac": dom["frac"], "traffic": dom.get("traffic"), "peak_kind": peak_kind,
                "kernels": kernels}

    # ---- end to end through the public whole-layer call with host buffers
    e2e = None
    if not args.no_e2e:
        hx = [torch.empty(L.X.shape, dtype=torch.bfloat16).pin_memory() for L in layers]
        hy = [torch.empty(L.Y.shape, dtype=torch.bfloat16).pin_memory() for L in layers]
        for h, L in zip(hx, layers):
            h.copy_(L.X)
        dx = [torch.empty_like(L.X) for L in layers]
        h2d = sum(h.numel() * 2 for h in hx)
        d2h = sum(h.numel() * 2 for h in hy)

        # Copies run on their own streams (PCIe is full duplex) so that the upload of the next layer's
        # input and the download of the previous layer's output overlap the kernels of this one; every
        # step still uploads all of its inputs and downloads all of its outputs inside the timed region.
        up, down = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
        in_ready = [torch.cuda.Event() for _ in layers]    # upload of layer i's input done
        in_free = [torch.cuda.Event() for _ in layers]     # kernels that read dx[i] done
        out_ready = [torch.cuda.Event() for _ in layers]   # kernels that wrote Y[i] done
        out_free = [torch.cuda.Event() for _ in layers]    # download of Y[i] done
        for e in in_free + out_free:
            e.record(stream)

        def e2e_step():
            for i, L in enumerate(layers):
                with torch.cuda.stream(up):
                    up.wait_event(in_free[i])
                    dx[i].copy_(hx[i], non_blocking=True)
                    in_ready[i].record(up)
                stream.wait_event(in_ready[i])
                stream.wait_event(out_free[i])
                resq.resq_linear(L.W, dx[i], L.P, L.Y, L.ws)
                in_free[i].record(stream)
                out_ready[i].record(stream)
                with torch.cuda.stream(down):
                    down.wait_event(out_ready[i])
                    hy[i].copy_(L.Y, non_blocking=True)
                    out_free[i].record(down)
            stream.wait_stream(down)  # the step ends when its last result is on the host

        for _ in range(3):
            e2e_step()
        barrier()
        e_steps = max(3, min(args.steps, 10))
        s0 = ev()
        for _ in range(e_steps):
            e2e_step()
        s1 = ev()
        barrier()
        e_ms = s0.elapsed_time(s1)
        e_ms = max_over_ranks(e_ms, dev)
        e2e = {"value": round(job_value(T, world, e_ms / e_steps), 1), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "ms_per_step": round(e_ms / e_steps, 4), "steps": e_steps}
    st = resq.resq_device_status()
    if st != resq.OK:
        raise SystemExit(f"device status {st}: {resq.status_string(st)}")

    # ---- the same prefill block with asymmetric per-token activations (the paper's experimental setting)
    asym = None
    if not args.no_asym and not only:
        asym = asym_leg(resq, torch, dev, layers, T, max(5, min(args.steps, 10)))

    # ---- the paper's own down_proj path: Hadamard U_D + uniform INT4 (r = 0)
    had = None
    if not args.no_asym and online:
        had = hadamard_leg(resq, torch, dev, online[0], T, max(5, min(args.steps, 10)), peaks)

    # ---- decode variant of the same block (this rank only; reported by rank 0)
    decode = None
    if not args.no_decode and not only:
        decode = decode_leg_with_clocks(gpu_id, resq, torch, dev, peaks, layers, max(5, min(args.steps, 20)))
        k = decode["T1"]
        kernels["mixed_gemm_decode_T1"] = {"bound": "hbm", "dtype": "int8", "achieved": k["weight_stream_gbs"],
                                           "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                           "ms_per_step": round(k["mixed_gemv_us"] * 1e-3, 5),
                                           "frac": k["frac_of_hbm_peak"]}

    # ---- the attention-block path: U_C projection, mixed-precision KV cache, single-query attention
    kvp = None
    if not args.no_kv and not only and MODEL == "8b":
        kvp = kv_leg(resq, torch, dev, peaks, max(5, min(args.steps, 20)), args.kv_seqs, args.kv_len)
        kernels["attention_decode"] = {"bound": "hbm", "dtype": "f16", "achieved": kvp["attention_cache_stream_gbs"],
                                       "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                       "ms_per_step": round(kvp["attention_decode_us"] * 1e-3, 5),
                                       "frac": kvp["attention_frac_of_hbm_peak"]}

    # ---- CPU baseline: the oracle on a row sample, rank 0 at N = 1 only; also a parity spot check
    cpu_baseline, parity = None, None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        S = min(ORACLE_SAMPLE_ROWS if MODEL != "70b" else 128, T)   # the 28672-wide fp64 projection is 4x the work per row
        hs = host_sample(layers, S)
        t0 = time.perf_counter()
        res = oracle_sample_step(hs)
        dt = time.perf_counter() - t0
        cpu_baseline = {"value": round(S / dt, 2), "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                        "sample": f"first {S} of {T} token rows through all four fused layers "
                                  f"(incl. the fp64 online projection), {dt:.1f} s"}
        # GPU outputs of the last step against the oracle on the sampled rows (folded layers: exact path)
        worst = 0.0
        for L, h, r_ in zip(layers, hs, res):
            if L.online:
                continue
            y = L.Y[:S].float().cpu().numpy()
            mag = (np.abs(r_.acc8.astype(np.float64) * r_.s_x8[:, None] * h["pw"].s8[None, :])
                   + np.abs(r_.acc4.astype(np.float64) * r_.s_x4[:, None] * h["pw"].s4[None, :]))
            # bf16 output: half an ulp of bf16 (2^-9 relative) on top of the fp32 tolerance
            worst = max(worst, float((np.abs(y - r_.y32) / (np.abs(r_.y32) * 2.0 ** -8 + 1e-5 * mag + 1e-30)).max()))
        parity = {"sampled_rows": S, "folded_layers_within_tolerance": bool(worst <= 1.0)}

    if rank == 0:
        line = {
            "metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": round(ms_per_step, 4), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
            "config": {"workload": WORKLOAD, "tokens_per_step_per_gpu": T,
                       "layers": {n: [k, o] for n, k, o, _ in LAYERS}, "r": "K/8",
                       "l2": "working set per step (weights 0.2 GB + P 0.41 GB + activations) exceeds the 126 MB L2",
                       "parallelism": f"replicas x{world}, no collective"},
            "mixed_gemm_tops": kernels["mixed_gemm"]["achieved"],
            "mixed_gemm_frac_of_int8_peak": int8_fracs, "int8_peak_measured": int8_measured,
            "per_layer": per_layer,
            "roofline": roofline, "decode": decode, "asymmetric": asym, "hadamard_down_proj": had, "kv_cache_path": kvp, "e2e": e2e, "cpu_baseline": cpu_baseline, "parity_spot_check": parity,
            "gpu_launches": gpu_launches, "clocks": clocks,
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


# --------------------------------------------------------------------------------------- reference arm
def run_reference(args):
    """The CPU oracle, as it stands, on a bounded sample of the same workload (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    if "LOCAL_RANK" in os.environ and os.environ.get("OMP_NUM_THREADS") == "1":
        # A multi-rank launcher pins every rank to one OpenMP thread; here rank 0 alone works and the other
        # ranks have exited, so the oracle gets the host cores it would have in a single-process run.
        del os.environ["OMP_NUM_THREADS"]
    import torch

    import oracle
    dev = torch.device("cuda", 0) if torch.cuda.is_available() else torch.device("cpu")
    S = REFERENCE_STEP_ROWS
    layers = build_layers(dev, rows=S)
    hs = host_sample(layers, S)
    del layers
    W = max(args.warmup, 1)
    for _ in range(W):
        oracle_sample_step(hs)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_sample_step(hs)
    dt = (time.perf_counter() - t0) / args.steps
    v = round(S / dt, 2)
    sample = f"first {S} of {T_PREFILL} token rows through all four fused layers per step"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
        "steps": args.steps, "warmup": W, "ms_per_step": round(dt * 1e3, 3), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        "config": {"workload": WORKLOAD, "sample": sample},
        "cpu_baseline": {"value": v, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def spawn_ranks(n: int, argv) -> int:
    """Re-runs this script as n ranks of one node (torch.distributed.run, rendezvous on 127.0.0.1, a free port)."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.abspath(__file__), *argv]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the oracle timing (profiling runs)")
    ap.add_argument("--no-int8-peak", action="store_true", help="skip the library INT8 GEMM timing (profiling runs)")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end leg (profiling runs)")
    ap.add_argument("--no-asym", action="store_true", help="skip the asymmetric-activation leg (profiling runs)")
    ap.add_argument("--no-decode", action="store_true", help="skip the few-token leg (profiling runs)")
    ap.add_argument("--decode-only", action="store_true", help="run only the few-token leg (profiling runs)")
    ap.add_argument("--no-kv", action="store_true", help="skip the attention-block leg (profiling runs)")
    ap.add_argument("--project-study", action="store_true", help="time the projection GEMM alone with SM clocks (profiling runs)")
    ap.add_argument("--tokens", type=int, default=0, help="override the prefill token count (profiling runs)")
    ap.add_argument("--kv-only", action="store_true", help="run only the attention-block leg (profiling runs)")
    ap.add_argument("--kv-seqs", type=int, default=16, help="sequences in the attention-block leg")
    ap.add_argument("--kv-len", type=int, default=8192, help="cached positions per sequence in the attention-block leg")
    ap.add_argument("--model", default="8b", choices=sorted(MODELS), help="block shape: 8b is the headline workload")
    ap.add_argument("--layers", default="", help="comma-separated subset of qkv,o,gate_up,down (profiling runs)")
    args = ap.parse_args()
    select_model(args.model)
    if args.tokens > 0:
        global T_PREFILL
        T_PREFILL = args.tokens
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # Plain `python bench.py --gpus N`: start the N ranks here, one process per GPU, the way a launcher would.
        sys.exit(spawn_ranks(args.gpus, sys.argv[1:]))
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
