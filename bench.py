#!/usr/bin/env python
"""Benchmark of the MUXQ linear hot path on B200.

A "step" is one pass of the whole hot path -- outlier detection, redistribute + quantize, INT8
tensor-core GEMM with the Aux correction and dequantization -- over the four GPT-2-large-shaped
linears (1280->3840, 1280->1280, 1280->5120, 5120->1280) at M = 16384 tokens, per-tensor INT8, on
seeded synthetic activations with 8 outlier channels (the largest single-GPU prefill workload of the
benchmark list).  The GPT-2-small set at M = 8192 is measured the same way and reported beside it,
and so are the decode shapes (M = 1, 4, 16) as a stream of layers.  Weights are quantized once
before timing.

    python bench.py --gpus 1 --steps K --warmup W          # the CUDA library (one JSON line)
    python bench.py --impl reference ...                    # the CPU oracle on a bounded sample

Metric: effective INT8 TOPS = sum over layers of 2*M*N*K / time (Aux ops are not credited).
Multi-GPU: the path does not shard (one GPU per problem); N ranks run N independent replicas.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import muxq_synth as synth  # noqa: E402

METRIC = "muxq_linear_effective_int8_tops_prefill"
UNIT = "TOPS"
HEADLINE_CONFIG = 3
NOMINAL_INT8_TOPS = 4500.0

WORKLOAD_TEXT = {
    1: "configs[1]: GPT-2-small linear set (768->2304, 768->768, 768->3072, 3072->768), M={M} tokens, "
       "6 outlier channels x40-80, per-tensor INT8, fp16 in/out",
    3: "configs[3] prefill: GPT-2-large linear set (1280->3840, 1280->1280, 1280->5120, 5120->1280), M={M} tokens, "
       "8 outlier channels x60, per-tensor INT8, fp16 in/out",
}

# DRAM traffic per launch from ncu captures (dram__bytes_read.sum + dram__bytes_write.sum, see profiles/): reported
# only while the kernel's sources still hash to what was captured, null otherwise.
CSRC = os.path.join(ROOT, "paper_2604_04701_b200", "csrc")
TRAFFIC = {
    # kernel key: (source files, sha16 of their concatenation at capture time, {workload: bytes per launch}, note)
    "k_gemm_i8_pair": (["k3p_gemm_pair.cu", "gemm_common.cuh", "ptx.cuh"], "cf2bd61da2081cdb",
                       {"cfg3": {"16384x1280->1280": 26.6e6, "16384x1280->5120": 138.1e6}},
                       "profiles/k_gemm_i8_pair_configs3.md"),
    "k_prep": (["k12_prep.cu", "quant.cuh"], "376646cd649c08db",
               {"cfg3": {"16384x1280": 46.9e6, "16384x5120": 328.9e6}}, "profiles/k_prep_configs3.md"),
    "k_decode_stream": (["k4s_decode_stream.cu", "quant.cuh", "ptx.cuh"], "ecf2c0babe5cc1a0",
                        {"chain": 712.4e6}, "profiles/k_decode_stream_chain144.md"),
}


def _src_sha16(files):
    h = hashlib.sha256()
    for f in files:
        with open(os.path.join(CSRC, f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def traffic_for(kernel, shape):
    ent = TRAFFIC.get(kernel)
    if not ent:
        return None
    files, sha, table, _ = ent
    if _src_sha16(files) != sha:
        return None  # the kernel has changed since the counters were taken
    return table.get(shape)


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": d["hbm_gbs"], "bf16_burst": d["bf16_tflops"],
                "bf16_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_burst": 1590.0, "bf16_sustained": 1400.0, "source": "fallback"}


def int8_peak_for(peaks, clocks):
    """Dense INT8 rate = 2 x the bf16 rate (8192 against 4096 MAC per clock and SM).  The burst figure applies when
    the timed region ran at the maximum SM clock, the sustained one when the clock had dropped under the power cap."""
    sm, mx_ = clocks.get("sm_mhz"), clocks.get("sm_max_mhz")
    burst = sm is None or mx_ is None or sm >= 0.97 * mx_
    kind = "burst" if burst else "sustained"
    return 2.0 * peaks["bf16_" + kind], f"2 x bf16_tflops{'' if burst else '_sustained'} ({kind}) of {peaks['source']}"


def workload(cfg_id=HEADLINE_CONFIG, M=None):
    specs = synth.config_layers(cfg_id, M=M)
    ops = sum(2.0 * s.M * s.N * s.K for s in specs)
    return specs, ops


def config_dict(cfg_id, specs, extra=None):
    x_mb = sum(2.0 * s.M * s.K for s in specs) / 1e6
    y_mb = sum(2.0 * s.M * s.N for s in specs) / 1e6
    q_mb = sum(1.0 * s.M * s.K for s in specs) / 1e6
    d = {"workload": WORKLOAD_TEXT[cfg_id].format(M=specs[0].M),
         "layers_per_step": len(specs), "granularity": "per-tensor",
         "l2": f"no explicit flush: one step streams ~{x_mb + y_mb + q_mb:.0f} MB (X {x_mb:.0f} MB, codes {q_mb:.0f} MB, "
               f"Y {y_mb:.0f} MB) > 126 MB L2"}
    if extra:
        d.update(extra)
    return d


# --------------------------------------------------------------------------- clocks
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid):
        self.uuid = uuid
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "25",
                 "-i", self.uuid], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, pw = [], [], []
        reasons = set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in out.strip().splitlines():
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1])); pw.append(float(parts[2]))
            except ValueError:
                continue
            for nm, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "power_w_max": max(pw),
                "samples": len(sm), "reasons": sorted(reasons)}


# --------------------------------------------------------------------------- CPU oracle leg
def oracle_sample(specs, rows_per_layer):
    """Times the oracle (as it stands) on the first `rows_per_layer` token rows of every layer."""
    import oracle
    oracle.build()
    prepared = []
    for s in specs:
        x, _ = synth.make_x(s.seed, s.tensor_id, rows_per_layer, s.K, s.n_outliers, s.mult_lo, s.mult_hi,
                            s.bulk, s.bulk_scale)
        wq, sw = oracle.quantize_weight(s.w())
        prepared.append((x, wq, sw, s))
    t0 = time.perf_counter()
    for x, wq, sw, s in prepared:
        oracle.linear(x, wq, sw, want_codes=False)
    dt = time.perf_counter() - t0
    ops = sum(2.0 * rows_per_layer * s.N * s.K for s in specs)
    return ops / dt / 1e12, dt, oracle.num_threads()


REFERENCE_ROWS = 1024


def run_reference(args, rank):
    if rank != 0:
        return
    specs, _ = workload()
    rows = REFERENCE_ROWS
    vals = []
    oracle_sample(specs, rows)  # one untimed pass
    t_all = 0.0
    steps = max(1, min(args.steps, 5))
    for _ in range(steps):
        v, dt, cores = oracle_sample(specs, rows)
        vals.append(v); t_all += dt
    value = statistics.mean(vals)
    sample = f"first {rows} of {specs[0].M} token rows of each of the 4 layers per step, {steps} steps"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": steps, "warmup": 1, "ms_per_step": 1e3 * t_all / steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
            "config": config_dict(HEADLINE_CONFIG, specs),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# --------------------------------------------------------------------------- CUDA arm
def max_over_ranks(ms: float, world: int, device) -> float:
    """The slowest rank's time: what a replica run is charged (all-reduce MAX over the process group)."""
    if world <= 1:
        return ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tops(world: int, ops_per_step: float, ms_per_step: float) -> float:
    """Replicas only: every rank does the same work, the job's rate is the sum over ranks at the slowest rank's time."""
    return world * ops_per_step / (ms_per_step * 1e-3) / 1e12


def prep_bytes(s, aux_written=32):
    """Algorithmic bytes of the preparation kernel for one layer: X read once (fp16), Body_q written, the Aux columns
    the GEMM reads (codes up to the next multiple of 32) and the W_aux gather."""
    return s.M * (2.0 * s.K + s.K + aux_written) + s.N * aux_written


def layer_bytes(s):
    """Algorithmic HBM bytes of the whole layer: X fp16 read once, W_q, Y fp16 written once."""
    return 2.0 * s.M * s.K + s.N * s.K + 2.0 * s.M * s.N


class Timer:
    def __init__(self, torch):
        self.torch = torch

    def replays(self, graph, n):
        t = self.torch
        e0, e1 = t.cuda.Event(enable_timing=True), t.cuda.Event(enable_timing=True)
        t.cuda.synchronize()
        e0.record()
        for _ in range(n):
            graph.replay()
        e1.record()
        t.cuda.synchronize()
        return e0.elapsed_time(e1) / n  # ms per replay


def build_layers(mx, torch, dev, specs, p, out_kind):
    layers = []
    for s in specs:
        x, _ = s.x()
        w = s.w()
        xd = torch.from_numpy(x).to(dev)
        w_q, s_w = mx.muxq_quantize(torch.from_numpy(w).to(dev), p, True,
                                    mx.Workspace(mx.muxq_small_workspace_bytes(s.N), dev))
        ws = mx.Workspace(mx.muxq_host_workspace_bytes(s.M, s.K, s.N, p, out_kind), dev)
        y = torch.empty(s.M, s.N, dtype=torch.float16, device=dev)
        layers.append({"spec": s, "x": xd, "w_q": w_q, "s_w": s_w, "ws": ws, "y": y, "x_host": x})
    torch.cuda.synchronize()
    return layers


def check_status(mx, layers):
    for L in layers:
        st = mx.muxq_read_status(L["ws"])
        if st != 0:
            raise RuntimeError(f"device status {st} ({mx.muxq_status_string(st)}) on {L['spec'].name}")


def capture(torch, side, fn):
    with torch.cuda.stream(side):
        fn()
        side.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            fn()
    torch.cuda.synchronize()
    return g


def measure_prefill(mx, torch, dist, dev, world, cfg_id, steps, warmup, headline):
    """Times one workload: the whole step (graph replay), the kernels inside it (event-record nodes), the GEMM
    launches on their own; for the headline workload also the end-to-end leg and the sampled clocks."""
    specs, ops_per_step = workload(cfg_id)
    p = mx.MuxqParams(max_outliers=32)
    layers = build_layers(mx, torch, dev, specs, p, mx.MUXQ_OUT_F16)
    side = torch.cuda.Stream(device=dev)
    timer = Timer(torch)

    def step():
        for L in layers:
            mx.muxq_linear(L["x"], L["w_q"], L["s_w"], p, L["ws"], mx.MUXQ_OUT_F16, out=L["y"])

    def barrier():
        if world > 1:
            dist.barrier()

    # One step = 4 layers x (fused prepare kernel, GEMM kernel): the host cannot enqueue 10-50 us kernels fast
    # enough, so the step is captured once into a CUDA graph (the entry points only enqueue work) and replayed;
    # the graph holds exactly the launches muxq_linear makes.
    g_step = capture(torch, side, step)
    check_status(mx, layers)
    for _ in range(max(warmup, 3)):
        g_step.replay()
    torch.cuda.synchronize()
    check_status(mx, layers)

    clocks = None
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier(); torch.cuda.synchronize()
    sampler = None
    if headline:
        uuid = str(torch.cuda.get_device_properties(dev).uuid)
        sampler = ClockSampler(uuid if uuid.startswith("GPU-") else "GPU-" + uuid)
        sampler.start()
    e0.record()
    for _ in range(steps):
        g_step.replay()
    e1.record()
    torch.cuda.synchronize(); barrier()
    if sampler:
        clocks = sampler.stop()
    check_status(mx, layers)
    ms = max_over_ranks(e0.elapsed_time(e1), world, dev)
    ms_per_step = ms / steps
    value = whole_job_tops(world, ops_per_step, ms_per_step)

    # ---- per-kernel durations: the same step captured with event-record nodes at the kernel
    # boundaries (same stream, same buffers), replayed and read back one replay at a time
    ksteps = min(steps, 100)
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in layers]
    for per_layer in evs:
        for e in per_layer:
            e.record()  # creates the CUDA handle
    torch.cuda.synchronize()
    with torch.cuda.stream(side):
        g_ev = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g_ev, stream=side):
            for li, L in enumerate(layers):
                mx.muxq_linear_events(L["x"], L["w_q"], L["s_w"], p, L["ws"], evs[li], mx.MUXQ_OUT_F16, out=L["y"])
    torch.cuda.synchronize()
    acc_us = [[0.0, 0.0, 0.0] for _ in layers]  # entry -> kernel 1 (empty for these shapes), prepare, gemm
    for i in range(ksteps + 3):
        g_ev.replay()
        torch.cuda.synchronize()
        if i < 3:
            continue
        for li in range(len(layers)):
            for j in range(3):
                acc_us[li][j] += evs[li][j].elapsed_time(evs[li][j + 1]) * 1e3 / ksteps
    kern_us = {"event_node": [a[0] for a in acc_us], "prepare": [a[1] for a in acc_us], "gemm": [a[2] for a in acc_us]}
    total_us = sum(sum(v) for v in kern_us.values())
    del g_ev

    # ---- the dominant kernel on its own: a graph of only the four GEMM launches, fed from the
    # intermediates the last step left in each layer's workspace (Body_q, Aux_q, W_aux, r, s_X)
    def ws_tensor(L, off, nbytes, dtype, shape):
        return L["ws"].buf[off: off + nbytes].view(dtype).view(*shape)

    gemm_calls = []
    for L in layers:
        sp = L["spec"]
        v = mx.muxq_workspace_view(sp.M, sp.K, sp.N, p)
        gemm_calls.append((
            ws_tensor(L, v.body_q, sp.M * v.ld_body_q, torch.int8, (sp.M, v.ld_body_q)),
            ws_tensor(L, v.aux_q, sp.M * v.aux_cols, torch.int8, (sp.M, v.aux_cols)),
            L["w_q"], ws_tensor(L, v.w_aux, sp.N * v.aux_cols, torch.int8, (sp.N, v.aux_cols)),
            ws_tensor(L, v.n_outliers, 4, torch.int32, (1,)), ws_tensor(L, v.s_x, 4, torch.float32, (1,)),
            L["s_w"], L["ws"], L["y"]))

    def gemm_step():
        for (bq, aq, wq, wa, nout, sx, sw, wsx, y) in gemm_calls:
            mx.muxq_gemm(bq, aq, wq, wa, nout, p, sx, sw, mx.MUXQ_OUT_F16, wsx, out=y)

    g_gemm = capture(torch, side, gemm_step)
    for _ in range(3):
        g_gemm.replay()
    gemm_us_per_step = timer.replays(g_gemm, ksteps) * 1e3
    check_status(mx, layers)
    del g_gemm

    out = {"cfg": cfg_id, "specs": specs, "ops_per_step": ops_per_step, "ms_per_step": ms_per_step, "value": value,
           "clocks": clocks, "kern_us": kern_us, "total_us": total_us, "gemm_us_per_step": gemm_us_per_step,
           "p": p, "e2e": None, "per_vector": None}

    # ---- end to end: host buffers, copies inside the timed region
    if headline:
        esteps = max(3, min(steps, 10))
        hosts = []
        for L in layers:
            xh = torch.from_numpy(L["x_host"]).pin_memory()
            yh = torch.empty(L["spec"].M, L["spec"].N, dtype=torch.float16).pin_memory()
            hosts.append((xh, yh))
        # Consecutive layers alternate between two streams, so one layer's device-to-host copy of Y overlaps the
        # next layer's host-to-device copy of X (PCIe is full duplex); each layer has its own buffers.
        h_streams = [torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)]

        def step_host():
            for i, (L, (xh, yh)) in enumerate(zip(layers, hosts)):
                with torch.cuda.stream(h_streams[i & 1]):
                    mx.muxq_linear_host(xh, L["w_q"], L["s_w"], p, L["ws"], yh, mx.MUXQ_OUT_F16)

        for _ in range(2):
            step_host()
        torch.cuda.synchronize(); barrier()
        h0, h1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        h0.record()
        for hs in h_streams:
            hs.wait_stream(torch.cuda.current_stream())
        for _ in range(esteps):
            step_host()
        for hs in h_streams:
            torch.cuda.current_stream().wait_stream(hs)
        h1.record()
        torch.cuda.synchronize(); barrier()
        check_status(mx, layers)
        ems = max_over_ranks(h0.elapsed_time(h1), world, dev)
        out["e2e"] = {"value": whole_job_tops(world, ops_per_step, ems / esteps), "unit": UNIT,
                      "h2d_bytes_per_step": int(sum(xh.numel() * 2 for xh, _ in hosts)),
                      "d2h_bytes_per_step": int(sum(yh.numel() * 2 for _, yh in hosts)), "steps": esteps,
                      "ms_per_step": ems / esteps}
        del hosts

    # ---- the per-vector variant of the same workload (per-token X scales, per-channel W scales)
    if world == 1:
        pv = mx.MuxqParams(max_outliers=32, gran=mx.MUXQ_PER_VECTOR)
        pv_layers = []
        for L in layers:
            sp = L["spec"]
            w_q, s_w = mx.muxq_quantize(torch.from_numpy(sp.w()).to(dev), pv, True,
                                        mx.Workspace(mx.muxq_small_workspace_bytes(sp.N), dev))
            pv_layers.append((L["x"], w_q, s_w, L["ws"], L["y"]))

        def pv_step():
            for (xd, w_q, s_w, wsx, y) in pv_layers:
                mx.muxq_linear(xd, w_q, s_w, pv, wsx, mx.MUXQ_OUT_F16, out=y)

        g_pv = capture(torch, side, pv_step)
        check_status(mx, layers)
        for _ in range(3):
            g_pv.replay()
        pv_ms = timer.replays(g_pv, ksteps)
        check_status(mx, layers)
        out["per_vector"] = {"granularity": "per-token X, per-channel W", "ms_per_step": pv_ms,
                             "value": ops_per_step / (pv_ms * 1e-3) / 1e12, "unit": UNIT}
        del g_pv, pv_layers
    del g_step, layers
    torch.cuda.empty_cache()
    return out


def int8_probe(mx, torch, dev):
    """The repo's own issue-bound tcgen05.mma kind::i8 loop (operands resident in shared memory, no loads): the INT8
    rate the tensor pipes attain at the clocks of this moment.  Timed with CUDA events around the launch."""
    ws = mx.Workspace(256, dev)
    ctas = torch.cuda.get_device_properties(dev).multi_processor_count
    iters = 16384
    mx.muxq_int8_mma_peak(256, 1024, ctas, ws)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    cyc = mx.muxq_int8_mma_peak(256, iters, ctas, ws)
    e1.record()
    torch.cuda.synchronize()
    if mx.muxq_read_status(ws) != 0:
        return None
    ops = 2.0 * 128 * 256 * 32 * iters * ctas
    ms = e0.elapsed_time(e1)
    return {"tops": ops / (ms * 1e-3) / 1e12, "cycles_per_mma_m128n256k32": float(cyc.double().mean().item()) / iters,
            "ctas": ctas, "iters": iters, "how": "CUDA events around one launch of the issue-bound MMA loop"}


def prefill_report(res, peaks, int8_peak, peak_source, probe):
    """roofline blocks of one measured workload"""
    specs, ops = res["specs"], res["ops_per_step"]
    kern_us = res["kern_us"]
    node = statistics.mean(kern_us["event_node"])  # a segment with no work in it: two records back to back
    achieved = ops / (res["gemm_us_per_step"] * 1e-6) / 1e12
    gemm = {"kernel": "k_gemm_i8_pair (tcgen05 kind::i8 cta_group::2, fused Aux + dequant epilogue)",
            "bound": "tensor", "achieved": achieved, "peak": int8_peak, "unit": "TOPS",
            "frac": achieved / int8_peak, "peak_source": peak_source,
            "int8_probe_tops": probe["tops"] if probe else None,
            "frac_vs_probe": achieved / probe["tops"] if probe else None,
            "frac_vs_nominal_4500": achieved / NOMINAL_INT8_TOPS,
            "traffic": traffic_for("k_gemm_i8_pair", f"cfg{res['cfg']}"),
            "algorithmic_bytes_per_step": sum(s.M * s.K + s.N * s.K + 2.0 * s.M * s.N for s in specs),
            "launches_per_step": len(specs), "us_per_step": res["gemm_us_per_step"],
            "how": "CUDA events around replays of a graph holding only the step's four GEMM launches",
            "per_layer_in_step": [{"layer": s.name, "M": s.M, "K": s.K, "N": s.N,
                                   "event_node_us": kern_us["event_node"][i], "prepare_us": kern_us["prepare"][i],
                                   "gemm_us": kern_us["gemm"][i]} for i, s in enumerate(specs)],
            "share_of_step": {k: sum(v) / res["total_us"] for k, v in kern_us.items()},
            "share_note": "from event-record nodes inside the step graph; each segment carries node overhead, and "
                          "event_node is a segment with no work in it (two records back to back)"}
    pbytes = sum(prep_bytes(s) for s in specs)
    pus = sum(max(u - node, 0.1) for u in kern_us["prepare"])
    prep = {"kernel": "k_prep (fused detect + redistribute + quantize, cooperative, one CTA per SM)", "bound": "hbm",
            "achieved": pbytes / pus / 1e3, "peak": peaks["hbm_gbs"], "unit": "GB/s",
            "frac": pbytes / pus / 1e3 / peaks["hbm_gbs"], "peak_source": f"hbm_gbs of {peaks['source']}",
            "traffic": traffic_for("k_prep", f"cfg{res['cfg']}"), "algorithmic_bytes_per_step": pbytes,
            "us_per_step": pus,
            "how": "event-record segments around the kernel inside the step graph, minus the empty segment's overhead; "
                   "bytes = M(2K + K + 32) + 32N per layer"}
    t_roof_us = 0.0
    for s in specs:
        t_c = 2.0 * s.M * s.N * s.K / (int8_peak * 1e12) * 1e6
        t_m = layer_bytes(s) / (peaks["hbm_gbs"] * 1e9) * 1e6
        t_roof_us += max(t_c, t_m)
    step = {"t_roof_us": t_roof_us, "frac": t_roof_us / (res["ms_per_step"] * 1e3),
            "peaks": {"int8_tops": int8_peak, "hbm_gbs": peaks["hbm_gbs"], "source": peak_source},
            "how": "per layer the slower of the INT8 tensor time and the HBM time of X + W_q + Y, summed"}
    return gemm, prep, step


def measure_decode(mx, torch, dev, peaks, p):
    """Decode shapes (M <= 16): the 36 x 4 GPT-2-large linears as one stream of layers with distinct weights
    (708 MB of W_q, far more than the L2 holds), replayed from a graph; GB/s = W_q bytes / time."""
    side = torch.cuda.Stream(device=dev)
    timer = Timer(torch)
    d = 1280
    dshapes = [(d, 3 * d), (d, d), (d, 4 * d), (4 * d, d)]
    gen = torch.Generator(device=dev)
    gen.manual_seed(4)
    dlayers = []
    for _ in range(36):
        for (K, N) in dshapes:
            dlayers.append((K, N, torch.randint(-127, 128, (N, K), dtype=torch.int8, device=dev, generator=gen)))
    wbytes = sum(K * N for K, N, _ in dlayers)
    sw1 = torch.full((1,), 0.02 / 127.0, device=dev)
    decode = {"workload": "configs[3]/[4] decode: 36 x (1280->3840, 1280->1280, 1280->5120, 5120->1280), "
                          "8 outlier channels x60, per-tensor INT8; us_per_layer etc.: one fused launch per layer (graph replay), "
                          "one_launch: the whole list in one muxq_chain_run",
              "w_bytes": wbytes, "layers": len(dlayers), "hbm_peak_gbs": peaks["hbm_gbs"]}
    for Md in (1, 4, 16):
        dx = {K: torch.from_numpy(synth.make_x(3, 100 + K, Md, K, 8, 60.0, 60.0)[0]).to(dev) for K in (d, 4 * d)}
        dy = {N: torch.empty(Md, N, dtype=torch.float16, device=dev) for N in (d, 3 * d, 4 * d)}
        dws = {K: mx.Workspace(mx.muxq_workspace_bytes(Md, K, 4 * d, p), dev) for K in (d, 4 * d)}

        def chain():
            for (K, N, wq) in dlayers:
                mx.muxq_linear(dx[K], wq, sw1, p, dws[K], mx.MUXQ_OUT_F16, out=dy[N])

        g_dec = capture(torch, side, chain)
        for _ in range(3):
            g_dec.replay()
        us = timer.replays(g_dec, 10) * 1e3
        # the same 144 layers as ONE persistent launch (muxq_chain_run): the weight stream runs on across layers
        lst = mx.Chain([(dx[K], wq, sw1, dy[N], 0) for (K, N, wq) in dlayers], p, mx.MUXQ_OUT_F16)
        for _ in range(3):
            lst.run()
        l0, l1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        l0.record()
        for _ in range(10):
            lst.run()
        l1.record()
        torch.cuda.synchronize()
        if lst.read_status() != 0:
            raise RuntimeError("device status raised on the decode list launch")
        list_us = l0.elapsed_time(l1) * 1e3 / 10
        del lst
        for K in dws:
            if mx.muxq_read_status(dws[K]) != 0:
                raise RuntimeError("device status raised on the decode chain")
        gbs = wbytes / us / 1e3
        decode[f"M{Md}"] = {"us_per_layer": us / len(dlayers), "gb_per_s": gbs, "frac_of_measured_hbm": gbs / peaks["hbm_gbs"],
                            "one_launch": {"us_per_layer": list_us / len(dlayers), "gb_per_s": wbytes / list_us / 1e3,
                                           "frac_of_measured_hbm": wbytes / list_us / 1e3 / peaks["hbm_gbs"]}}
        del g_dec
        # one call on its own (nothing before it in the stream to overlap with, weights cold): the call is captured
        # with event-record nodes at its boundaries and replayed 15 times, each after a write of 256 MB that
        # pushes the weights out of L2; median device time between the records (includes their node overhead)
        flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
        iso = {}
        for li, (K, N, wq) in enumerate(dlayers[:4]):
            ievs = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
            for e in ievs:
                e.record()
            torch.cuda.synchronize()
            with torch.cuda.stream(side):
                g_one = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g_one, stream=side):
                    mx.muxq_linear_events(dx[K], wq, sw1, p, dws[K], ievs, mx.MUXQ_OUT_F16, out=dy[N])
            torch.cuda.synchronize()
            ts = []
            for _ in range(15):
                flush.fill_(li)
                torch.cuda.synchronize()
                g_one.replay()
                torch.cuda.synchronize()
                ts.append(ievs[0].elapsed_time(ievs[3]) * 1e3)
            iso[f"{K}->{N}"] = statistics.median(ts)
            del g_one
        decode[f"M{Md}"]["isolated_call_us"] = iso
        del flush
    del dlayers
    torch.cuda.empty_cache()
    # a list of four large layers (1280 -> 50304 each, 258 MB of W_q) in one launch: the streaming rate of the
    # kernel when per-layer work is negligible; one run per measurement, median of 7
    big = [torch.randint(-127, 128, (50304, d), dtype=torch.int8, device=dev, generator=gen) for _ in range(4)]
    large = {}
    for Md in (1, 16):
        xb = torch.from_numpy(synth.make_x(3, 7, Md, d, 8, 60.0, 60.0)[0]).to(dev)
        yb = [torch.empty(Md, 50304, dtype=torch.float16, device=dev) for _ in big]
        lst = mx.Chain([(xb, wq, sw1, y, 0) for wq, y in zip(big, yb)], p, mx.MUXQ_OUT_F16)
        lst.run()
        ts = []
        for _ in range(7):
            b0, b1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            b0.record(); lst.run(); b1.record()
            torch.cuda.synchronize()
            ts.append(b0.elapsed_time(b1) * 1e3)
        us = statistics.median(ts)
        nbytes = 4 * 50304 * d
        large[f"M{Md}"] = {"us": us, "gb_per_s": nbytes / us / 1e3, "frac_of_measured_hbm": nbytes / us / 1e3 / peaks["hbm_gbs"]}
        del lst
    decode["large_call"] = {"workload": "4 x (1280 -> 50304) in one muxq_chain_run, 258 MB of W_q (> L2), host launch "
                                        "latency inside the timed region", **large}
    del big
    torch.cuda.empty_cache()
    best = max(max(decode[f"M{m}"]["gb_per_s"], decode[f"M{m}"]["one_launch"]["gb_per_s"]) for m in (1, 4, 16))
    m1 = decode["M1"]["one_launch"]
    roof = {"kernel": "k_decode_stream (144 layers in one persistent launch, W_q streamed once)", "bound": "hbm",
            "achieved": m1["gb_per_s"], "peak": peaks["hbm_gbs"], "unit": "GB/s",
            "frac": m1["frac_of_measured_hbm"], "peak_source": f"hbm_gbs of {peaks['source']}",
            "traffic": traffic_for("k_decode_stream", "chain"), "algorithmic_bytes_per_chain": wbytes,
            "best_over_M_gb_per_s": best,
            "per_layer_launches_gb_per_s": decode["M1"]["gb_per_s"],
            "how": "W_q bytes of the 144-layer list / CUDA-event time of muxq_chain_run, M = 1"}
    return decode, roof


def run_muxq(args, rank, world):
    import torch
    import torch.distributed as dist

    import paper_2604_04701_b200 as mx

    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    mx.lib()  # fails loudly if the CUDA library is missing
    peaks = load_peaks()

    if args.decode_only:  # profiling aid: only the decode section, printed as its own JSON line
        decode, decode_roof = measure_decode(mx, torch, dev, peaks, mx.MuxqParams(max_outliers=32))
        print(json.dumps({"decode": decode, "roofline_decode": decode_roof}))
        return
    head = measure_prefill(mx, torch, dist, dev, world, HEADLINE_CONFIG, args.steps, args.warmup, headline=True)
    clocks = head["clocks"]
    int8_peak, peak_source = int8_peak_for(peaks, clocks)
    probe = int8_probe(mx, torch, dev) if world == 1 else None
    gemm_roof, prep_roof, step_roof = prefill_report(head, peaks, int8_peak, peak_source, probe)

    extra = {}
    if world == 1 and not args.no_small:
        small = measure_prefill(mx, torch, dist, dev, world, 1, max(args.steps, 50), args.warmup, headline=False)
        s_gemm, s_prep, s_step = prefill_report(small, peaks, int8_peak, peak_source, probe)
        extra["configs1"] = {"config": config_dict(1, small["specs"]), "value": small["value"], "unit": UNIT,
                             "ms_per_step": small["ms_per_step"],
                             "us_per_layer": small["ms_per_step"] * 1e3 / len(small["specs"]),
                             "pct_of_nominal_int8_peak_4500": 100.0 * small["value"] / NOMINAL_INT8_TOPS,
                             "roofline": s_gemm, "roofline_prep": s_prep, "step_roofline": s_step,
                             "per_vector": small["per_vector"]}

    decode = decode_roof = None
    if world == 1 and not args.no_decode:
        decode, decode_roof = measure_decode(mx, torch, dev, peaks, head["p"])

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        rows = 4096
        v, dt, cores = oracle_sample(head["specs"], rows)
        cpu_baseline = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "seconds": dt,
                        "sample": f"first {rows} of {head['specs'][0].M} token rows of each of the 4 layers, one pass"}

    if rank == 0:
        specs = head["specs"]
        line = {"metric": METRIC, "value": head["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": max(args.warmup, 3), "ms_per_step": head["ms_per_step"], "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
                "config": config_dict(HEADLINE_CONFIG, specs,
                                      {"parallelism": "replicas only" if world > 1 else "single GPU"}),
                "us_per_layer": head["ms_per_step"] * 1e3 / len(specs),
                "pct_of_nominal_int8_peak_4500": 100.0 * head["value"] / world / NOMINAL_INT8_TOPS,
                "clocks": clocks, "e2e": head["e2e"], "gpu_launches": args.steps * len(specs) * 2,
                "roofline": gemm_roof, "roofline_prep": prep_roof, "roofline_decode": decode_roof,
                "step_roofline": step_roof, "int8_probe": probe, "per_vector": head["per_vector"],
                "extra": extra, "decode": decode, "cpu_baseline": cpu_baseline}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="muxq", choices=["muxq", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-decode", action="store_true")
    ap.add_argument("--no-small", action="store_true", help="skip the GPT-2-small workload reported under extra")
    ap.add_argument("--decode-only", action="store_true", help="run only the decode measurements (for profiling)")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        run_reference(args, rank)
    else:
        run_muxq(args, rank, world)


if __name__ == "__main__":
    main()
