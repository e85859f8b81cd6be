#!/usr/bin/env python
"""Benchmark of the streaming-scan hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Workload (config.workload = cfg3_128k_4layers_kq): a 128K-token context streamed in chunks of 8192
tokens through 4 target layers; per chunk and layer the key projections (1024 -> 16384, k = 32) and the
query projections (4096 -> 32768, k = 64) are SAE-encoded with fused Top-k, their postings are built and
appended to the host-resident index. One STEP = one chunk through all of that, plus one batched
retrieval (256 queries x 64 tokens encoded with the key SAE at k = 64, co-activation scoring of 2045
overlapping 64-token spans against a 32K-token device-staged index, 0.5/0.5 fusion with a lexical score
vector, top-16), so that every stage of the path runs in every step. metric = scanned context tokens/s.

Prints ONE JSON line (rank 0). `--impl reference` times the CPU oracle (oracle/) on a bounded sample of
the same workload on the host cores instead. `--workload cfg5 | cfg2` runs the other scan configurations (scan only).
With `--gpus N` and no launcher around it the script starts its own N ranks (one process per GPU).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from workloads import configs as C, generators as G  # noqa: E402

METRIC = "scanned tokens/s (SAE Top-k encode + postings) at 128K ctx"
# Measured DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum, ncu) of one grouped encode launch of the benchmark
# step (see profiles/); None when the encode kernel has changed since the counters were taken.
ENCODE_DRAM_BYTES = {("cfg3", "encode_query"): 0.89e9}    # (workload, timer name) -> bytes per launch
UNIT = "tokens/s"


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"source": "measured", "hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"])}
    return {"source": "fallback", "hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU while the timed region runs: NVML from a thread every few
    milliseconds (nvidia-smi's own source, without its start-up time), or an nvidia-smi loop if NVML cannot be loaded.
    Read-only queries."""
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
    Q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device: torch.device):
        self.device = device
        self.samples = []          # (wall time, sm MHz, max MHz, set of active reasons)
        self.thread = None
        self.proc = None
        self.stop_flag = threading.Event()
        self.source = None

    def start(self):
        try:
            import pynvml as N
            N.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(self.device).uuid)
            try:
                h = N.nvmlDeviceGetHandleByUUID(("GPU-" + uuid).encode())
            except Exception:
                h = N.nvmlDeviceGetHandleByIndex(self.device.index or 0)
            mx = N.nvmlDeviceGetMaxClockInfo(h, N.NVML_CLOCK_SM)
            bits = {"hw_slowdown": N.nvmlClocksThrottleReasonHwSlowdown, "hw_thermal_slowdown": N.nvmlClocksThrottleReasonHwThermalSlowdown,
                    "sw_thermal_slowdown": N.nvmlClocksThrottleReasonSwThermalSlowdown, "sw_power_cap": N.nvmlClocksThrottleReasonSwPowerCap}

            def loop():
                while not self.stop_flag.is_set():
                    try:
                        sm = N.nvmlDeviceGetClockInfo(h, N.NVML_CLOCK_SM)
                        r = N.nvmlDeviceGetCurrentClocksThrottleReasons(h)
                        self.samples.append((time.time(), float(sm), float(mx), {n for n, b in bits.items() if r & b}))
                    except Exception:
                        pass
                    time.sleep(0.004)
            self.thread = threading.Thread(target=loop, daemon=True)
            self.thread.start()
            self.source = "nvml"
            return
        except Exception:
            pass
        try:
            idx = self.device.index or 0
            if "CUDA_VISIBLE_DEVICES" in os.environ:
                idx = int(os.environ["CUDA_VISIBLE_DEVICES"].split(",")[idx])
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "20", "-i", str(idx)], stdout=subprocess.PIPE, text=True)

            def read():
                for line in self.proc.stdout:
                    f = [v.strip() for v in line.split(",")][1:]
                    try:
                        self.samples.append((time.time(), float(f[0]), float(f[1]),
                                             {n for n, v in zip(self.NAMES, f[3:7]) if v.lower().startswith("active")}))
                    except (ValueError, IndexError):
                        continue
            self.thread = threading.Thread(target=read, daemon=True)
            self.thread.start()
            self.source = "nvidia-smi"
        except Exception:
            self.proc = None

    def stop(self, t_begin=None, t_end=None):
        self.stop_flag.set()
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()
        if self.source is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "samples": 0, "reasons": ["no clock source"]}
        sel = [x for x in self.samples if t_begin is None or t_begin <= x[0] <= t_end]
        reasons = set()
        for x in sel:
            reasons |= x[3]
        return {"sm_mhz": statistics.median(x[1] for x in sel) if sel else None, "sm_max_mhz": max((x[2] for x in sel), default=None),
                "samples": len(sel), "reasons": sorted(reasons), "source": self.source}


WORKLOADS = {"cfg3": (C.CFG3, C.CFG4), "cfg5": (C.CFG5, None), "cfg2": (C.CFG2, None), "cfg1": (C.CFG1, None)}


def workload_config(cfg, rcfg, L_idx, ns):
    """The `config` object of the JSON line (same for both arms)."""
    out = {"workload": cfg.name, "context_tokens": cfg.L, "chunk": cfg.chunk, "layers": cfg.n_layers,
           "key_sae": [cfg.key.d_in, cfg.key.d_sae, cfg.key.k],
           "query_sae": [cfg.query.d_in, cfg.query.d_sae, cfg.query.k] if cfg.query else None,
           "l2_policy": "inputs larger than L2: every step reads a different activation chunk and all layers' encoder weights",
           "parallelism": "independent context replicas per GPU, no collectives"}
    if rcfg is not None:
        out["retrieval_per_step"] = {"queries": rcfg.Q, "query_tokens": rcfg.nq, "k": rcfg.kq, "index_tokens": L_idx,
                                     "spans": ns, "width": rcfg.width, "stride": rcfg.stride, "top": rcfg.s}
    return out


def max_over_ranks(seconds_or_ms: float, world: int, device=None) -> float:
    """The slowest rank's time (every rank returns it). The path has no exchange step, so this reduction of one
    timing scalar is the only collective of a multi-GPU run."""
    if world <= 1:
        return float(seconds_or_ms)
    t = torch.tensor([seconds_or_ms], dtype=torch.float64, device=device if device is not None else "cpu")
    torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank_step: int, steps: int, world: int, slowest_seconds: float) -> float:
    """Units all ranks processed divided by the slowest rank's time (weak scaling: every rank does the same work)."""
    return units_per_rank_step * steps * world / slowest_seconds


def pick_tensor_peak(peaks: dict, region_seconds: float):
    """The measured bf16 rate that applies to a kernel timed inside a region of that length: the burst rate for a
    region that ends before the power cap has pulled the clocks down (about two seconds), else the sustained one."""
    if region_seconds < 2.0:
        return peaks["bf16_tflops"], f"{peaks['source']} burst bf16 matmul (timed region {region_seconds:.2f} s < 2 s)"
    return peaks["bf16_tflops_sustained"], f"{peaks['source']} sustained bf16 matmul (timed region {region_seconds:.2f} s)"


def mean_ms(pairs):
    v = [a.elapsed_time(b) for a, b in pairs]
    return sum(v) / len(v) if v else None


# ------------------------------------------------------------------------------------------ our arm

def run_ours(args, rank, world, local_rank):
    import paper_2601_17702_b200 as S
    from paper_2601_17702_b200.scan import SaeSlot, ScanPipeline, stage_index_on_device

    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    cfg, rcfg = WORKLOADS[args.workload]
    peaks = load_peaks()
    sampler = ClockSampler(dev)
    if rank == 0:
        sampler.start()
    inp = C.ScanInputs(cfg, device=dev)
    nl, chunk = cfg.n_layers, cfg.chunk

    key_saes = [S.Sae(*inp.sae("key", l)) for l in range(nl)]
    slots = [SaeSlot("key", key_saes, cfg.key.k, chunk)]
    if cfg.query:
        slots.append(SaeSlot("query", [S.Sae(*inp.sae("query", l)) for l in range(nl)], cfg.query.k, chunk))
    pipe = ScanPipeline(slots, grouped=args.group, overlap=args.overlap)
    e2e_steps = max(2, min(args.steps, 32))      # the first step's upload cannot overlap anything: enough steps to carry it
    total_steps = 2 * args.steps + args.warmup + e2e_steps + 4
    pipe.reserve_index((total_steps + 2) * chunk)

    n_distinct = min(cfg.n_chunks, args.steps + args.warmup)
    xs = [{s.name: [inp.x(s.name, l, c * chunk, chunk) for l in range(nl)] for s in slots} for c in range(n_distinct)]

    # retrieval side: a 32K-token key index of layer 0 staged on the device, and the query batch
    launches = [0]
    timers = {}
    retrieval = None
    L_idx = ns = None
    if rcfg is not None:
        rpipe = ScanPipeline([SaeSlot("key", [key_saes[0]], cfg.key.k, chunk)])
        for c in range(rcfg.scan.L // chunk):
            rpipe.scan_chunk(c * chunk, {"key": [xs[c % n_distinct]["key"][0]]})
        rpipe.finish()
        csr = stage_index_on_device(rpipe.slots[0].index, dev)
        L_idx = rcfg.scan.L
        ns = C.n_spans(L_idx, rcfg.width, rcfg.stride)
        xqry = inp.retrieval_queries(0, rcfg.Q, rcfg.nq)
        q_ids = torch.empty((rcfg.Q * rcfg.nq, rcfg.kq), dtype=torch.int32, device=dev)
        q_vals = torch.empty((rcfg.Q * rcfg.nq, rcfg.kq), dtype=torch.float32, device=dev)
        q_ws = S.new_workspace(key_saes[0].encode_workspace_bytes(rcfg.Q * rcfg.nq, rcfg.kq), dev)
        s_ws = S.new_workspace(S.s3_score_workspace_bytes(rcfg.Q, rcfg.nq, rcfg.kq, 1, ns, rcfg.s), dev)
        bm25 = G.gamma21(rcfg.bm25_seed, rcfg.Q, ns).to(dev)
        top_idx = torch.empty((rcfg.Q, rcfg.s), dtype=torch.int32, device=dev)
        top_score = torch.empty((rcfg.Q, rcfg.s), dtype=torch.float32, device=dev)
        top_idx_h = torch.empty((rcfg.Q, rcfg.s), dtype=torch.int32).pin_memory()

        def retrieval(xqry_in, timed=False):
            S.s3_sae_encode_topk(key_saes[0], xqry_in, rcfg.kq, q_ids, q_vals, q_ws)
            if timed:
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
            S.s3_coactivation_score_topspans(csr, cfg.key.d_sae, L_idx, q_ids.view(1, rcfg.Q, rcfg.nq, rcfg.kq),
                                             q_vals.view(1, rcfg.Q, rcfg.nq, rcfg.kq), rcfg.width, rcfg.stride, rcfg.s,
                                             rcfg.alpha, rcfg.beta, s_ws, bm25, top_idx=top_idx, top_score=top_score)
            if timed:
                e1.record()
                timers.setdefault("score", []).append((e0, e1))
            launches[0] += 2 + S.SCORE_LAUNCHES

        # algorithmic bytes of the scoring call: every (query, unique feature) pair gathers its list once
        retrieval(xqry)
        lens = (csr[0][0][1:] - csr[0][0][:-1])
        gathered = 0
        for q in range(rcfg.Q):
            f = q_ids.view(rcfg.Q, -1)[q].long()
            gathered += int(lens[torch.unique(f[f >= 0])].sum().item())
        score_bytes = gathered * 4 + rcfg.Q * ns * 4 + rcfg.Q * rcfg.s * 8

    def step(i, x_c, timed=False, xqry_in=None, append=True):
        pipe.timers = timers if timed else None
        pipe.scan_chunk(i * chunk, x_c, append=append)
        if retrieval is not None:
            retrieval(xqry if xqry_in is None else xqry_in, timed)

    def barrier():
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing (inputs already in HBM)
    for i in range(args.warmup):
        step(i, xs[i % n_distinct])
    barrier()
    torch.cuda.reset_peak_memory_stats()
    mem_after_warm = torch.cuda.memory_allocated()
    free_after_warm = torch.cuda.mem_get_info()[0]
    l0 = pipe.launches + launches[0]
    wall0 = time.time()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for j in range(args.steps):
        i = args.warmup + j
        step(i, xs[i % n_distinct], timed=True)
    t1.record()
    host_enqueue_s = time.time() - wall0            # the host is done queueing here; the device is still working
    barrier()
    wall1 = time.time()
    ms = t0.elapsed_time(t1)
    clocks = sampler.stop(wall0, wall1) if rank == 0 else None
    gpu_launches = pipe.launches + launches[0] - l0
    peak_mem = torch.cuda.max_memory_allocated()
    free_after_run = torch.cuda.mem_get_info()[0]
    kernel_ms = {name: mean_ms(p) for name, p in timers.items()}
    n_timed = {name: len(p) for name, p in timers.items()}
    pipe.timers = None
    pipe.finish()
    if retrieval is not None:
        assert S.s3_workspace_status(q_ws) == 0 and S.s3_workspace_status(s_ws) == 0

    ms = max_over_ranks(ms, world, dev)
    value = whole_job_rate(chunk, args.steps, world, ms * 1e-3)

    # ---- the same steps without the hand-over to the host index: what the appends cost on top of the device work
    base = args.warmup + args.steps
    barrier()
    t0.record()
    for j in range(args.steps):
        step(base + j, xs[(base + j) % n_distinct], append=False)
    t1.record()
    barrier()
    ms_noappend = t0.elapsed_time(t1)
    d2h_index = sum(nl * (chunk * s.k * 4 + (s.d_sae + 1) * 4) for s in slots)
    pinned = torch.empty(d2h_index, dtype=torch.uint8).pin_memory()
    devbuf = torch.empty(d2h_index, dtype=torch.uint8, device=dev)
    pinned.copy_(devbuf, non_blocking=True)
    torch.cuda.synchronize()
    t0.record()
    for _ in range(4):
        pinned.copy_(devbuf, non_blocking=True)
    t1.record()
    torch.cuda.synchronize()
    d2h_alone_ms = t0.elapsed_time(t1) / 4
    del pinned, devbuf
    exposed_ms = max(0.0, (ms - ms_noappend) / args.steps)

    # ---- end to end: the step's inputs come from pinned host memory, its result goes back to the host
    n_host = min(4, n_distinct)
    x_h = [{n: [t.cpu().pin_memory() for t in ts] for n, ts in xs[c].items()} for c in range(n_host)]
    # two sets of device input buffers: while a step computes on one, the next step's inputs are copied into the
    # other on a copy stream (events order buffer reuse), so the PCIe transfer hides behind the encodes
    x_d = [{n: [torch.empty_like(t) for t in ts] for n, ts in xs[0].items()} for _ in range(2)]
    h2d = sum(t.numel() * t.element_size() for ts in x_h[0].values() for t in ts)
    d2h = 0
    if retrieval is not None:
        xqry_d = [torch.empty_like(xqry) for _ in range(2)]
        xqry_h = xqry.cpu().pin_memory()
        h2d += xqry.numel() * xqry.element_size()
        d2h = top_idx_h.numel() * 4
    else:
        stats_h = torch.empty(8, dtype=torch.int32).pin_memory()     # the scan's per-step result: the last list offsets
        d2h = stats_h.numel() * 4
    copy_stream = torch.cuda.Stream(device=dev)
    ready = [torch.cuda.Event() for _ in range(2)]      # inputs of the buffer set have arrived
    consumed = [torch.cuda.Event() for _ in range(2)]   # the step that read the buffer set has finished

    def e2e_upload(i):
        b, c = i % 2, i % n_host
        with torch.cuda.stream(copy_stream):
            copy_stream.wait_event(consumed[b])
            for n, ts in x_h[c].items():
                for l, t in enumerate(ts):
                    x_d[b][n][l].copy_(t, non_blocking=True)
            if retrieval is not None:
                xqry_d[b].copy_(xqry_h, non_blocking=True)
            ready[b].record(copy_stream)

    def e2e_step(i, last):
        b = i % 2
        if not last:
            e2e_upload(i + 1)                           # next step's inputs travel while this step computes
        torch.cuda.current_stream().wait_event(ready[b])
        step(i, x_d[b], xqry_in=xqry_d[b] if retrieval is not None else None)
        consumed[b].record()
        if retrieval is not None:
            top_idx_h.copy_(top_idx, non_blocking=True)
        else:
            stats_h.copy_(slots[0].row_ptr[0][-8:], non_blocking=True)

    base = args.warmup + 2 * args.steps
    for b in range(2):
        consumed[b].record()
    e2e_upload(base)
    e2e_step(base, last=True)                           # untimed warm-up of the end-to-end path
    barrier()
    w0 = time.perf_counter()
    e2e_upload(base + 1)                                # the first timed step's upload is inside the timed region
    for j in range(e2e_steps):
        e2e_step(base + 1 + j, last=(j == e2e_steps - 1))
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - w0
    pipe.finish()
    e2e_s = max_over_ranks(e2e_s, world, dev)
    e2e_value = whole_job_rate(chunk, e2e_steps, world, e2e_s)

    if rank != 0:
        return None
    # dominant kernel: the encode launch kind that carries the most FLOPs of a step (a grouped launch over layers and SAE
    # streams, a grouped launch over one stream's layers, or single launches)
    shapes = {s.name: (cfg.key if s.name == "key" else cfg.query) for s in slots}
    best = None
    for name in kernel_ms:
        if not name.startswith("encode"):
            continue
        per_step = n_timed[name] / args.steps
        if name == "encode_group":
            fl_step = sum(nl * 2.0 * chunk * sh.d_in * sh.d_sae for sh in shapes.values())
            desc = f"grouped launch over the {nl} layers of {' + '.join(shapes)} SAEs"
        elif name.startswith("encode_group_"):
            sh = shapes[name[len("encode_group_"):]]
            fl_step = nl * 2.0 * chunk * sh.d_in * sh.d_sae
            desc = f"grouped launch over the {nl} layers' {name[len('encode_group_'):]} SAEs {sh.d_in}->{sh.d_sae}, k={sh.k}"
        else:
            sh = shapes[name[len("encode_"):]]
            fl_step = nl * 2.0 * chunk * sh.d_in * sh.d_sae
            desc = f"{name[len('encode_'):]} SAE {sh.d_in}->{sh.d_sae}, k={sh.k}, one launch per layer"
        if best is None or fl_step > best[0]:
            best = (fl_step, name, per_step, desc)
    fl_step, enc_name, per_step, desc = best
    flops = fl_step / per_step
    enc_avg_ms = kernel_ms[enc_name]
    enc_desc = f"encode_tc_kernel, {desc} (T={chunk}; {per_step:g} launch(es) per step; duration includes the Top-k merge kernel)"
    tflops = flops / (enc_avg_ms * 1e-3) / 1e12
    peak, peak_source = pick_tensor_peak(peaks, ms * 1e-3)
    bound = "tensor"
    if cfg.dtype == torch.float32:
        # fp32 inputs run on the FFMA kernel: 128 FMA lanes per SM and clock, at the clock sampled during the run
        sm_count = torch.cuda.get_device_properties(dev).multi_processor_count
        mhz = (clocks or {}).get("sm_mhz") or 1965.0
        bound, peak = "alu", sm_count * 128 * 2 * mhz * 1e6 / 1e12
        peak_source = f"{sm_count} SMs x 128 fp32 FMA lanes x 2 FLOP x {mhz:.0f} MHz (sampled)"
        enc_desc = enc_desc.replace("encode_tc_kernel", "encode_simt_kernel")
    post_bytes = sum(nl * (chunk * s.k * 8 + (s.d_sae + 1) * 4) for s in slots)
    post_gbs = post_bytes / (kernel_ms["postings"] * 1e-3) / 1e9
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32" if cfg.dtype == torch.float32 else "bf16", "data": "synthetic",
        "config": workload_config(cfg, rcfg, L_idx, ns),
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "steps": e2e_steps, "note": "every step's activations are copied from pinned host memory (double-buffered on a copy stream, overlapping the previous step's kernels) and the step's result is read back, all inside the timed region (the first step's upload included, which nothing overlaps); postings also travel device->host (index append) in both numbers"},
        "gpu_launches": gpu_launches,
        "clocks": clocks,
        "roofline": {"bound": bound, "kernel": enc_desc,
                     "achieved": tflops, "peak": peak, "unit": "TFLOP/s", "frac": tflops / peak, "peak_source": peak_source,
                     "frac_of_measured_burst": tflops / peaks["bf16_tflops"], "frac_of_measured_sustained": tflops / peaks["bf16_tflops_sustained"],
                     "frac_of_nominal_2250": tflops / 2250.0, "launch_ms": enc_avg_ms, "launches_timed": n_timed[enc_name], "flop_per_launch": flops,
                     # dram__bytes_read.sum + dram__bytes_write.sum of one full-size launch of this kernel (ncu, one pass);
                     # null when the kernel has changed since the counters were taken or the workload has no capture
                     "traffic": ENCODE_DRAM_BYTES.get((args.workload, enc_name)), "traffic_unit": "bytes per launch"},
        "roofline_postings": {"bound": "hbm", "kernel": "postings_partition_kernel + postings_bucket_kernel (all chunk-layers of a step in one batch)",
                              "achieved": post_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": post_gbs / peaks["hbm_gbs"],
                              "frac_of_nominal_8000": post_gbs / 8000.0, "peak_source": f"{peaks['source']} copy bandwidth",
                              "bytes_per_launch": post_bytes, "launch_ms": kernel_ms["postings"], "launches_timed": n_timed["postings"],
                              "traffic": None},
        "append_overlap": {"ms_per_step": ms / args.steps, "ms_per_step_without_append": ms_noappend / args.steps,
                           "index_d2h_bytes_per_step": d2h_index, "d2h_alone_ms": d2h_alone_ms, "exposed_ms_per_step": exposed_ms,
                           "hidden_frac": 1.0 - min(1.0, exposed_ms / d2h_alone_ms)},
        "host": {"syncs_in_chunk_loop": pipe.host_syncs, "enqueue_ms_per_step": host_enqueue_s * 1e3 / args.steps,
                 "note": "the host queued all timed steps in enqueue_ms_per_step each, ahead of the device (ms_per_step): nothing in the loop waits for the GPU"},
        "kernel_ms_in_step": kernel_ms,
        "device_mem": {"allocated_after_warmup_mib": mem_after_warm / 2**20, "peak_in_timed_region_mib": peak_mem / 2**20,
                       "cudaMemGetInfo_free_delta_bytes": free_after_warm - free_after_run},
    }
    if retrieval is not None:
        sc_gbs = score_bytes / (kernel_ms["score"] * 1e-3) / 1e9
        out["roofline_scoring"] = {"bound": "hbm", "kernel": "span scoring + fusion + top-s (index L2-resident: gathered bytes, not DRAM bytes)",
                                   "achieved": sc_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": sc_gbs / peaks["hbm_gbs"],
                                   "frac_of_nominal_8000": sc_gbs / 8000.0, "peak_source": f"{peaks['source']} copy bandwidth",
                                   "bytes_per_launch": score_bytes, "gathered_postings": gathered, "launch_ms": kernel_ms["score"],
                                   "launches_timed": n_timed["score"], "traffic": None}
    return out


# ------------------------------------------------------------------------------------------ oracle arm

def oracle_step(n_tok, seed_row, cfg, inp_cpu, weights):
    """One bounded sample of the workload through the CPU oracle: n_tok tokens through every layer's key
    (and query) SAE (encode, Top-k, postings), then one query scored against the sample's own postings."""
    import numpy as np
    import oracle as O
    ids_key = []
    for l in range(cfg.n_layers):
        for which, shp in (("key", cfg.key), ("query", cfg.query)):
            if shp is None:
                continue
            W, b_enc, b_dec = weights[(which, l)]
            x = inp_cpu.x(which, l, seed_row, n_tok).float().numpy()
            ids, vals = O.encode_topk(x, W, b_enc, b_dec, shp.k)
            O.postings(ids, shp.d_sae, seed_row)
            if which == "key":
                ids_key.append(ids)
    w = min(64, n_tok)
    q = ids_key[0][: min(n_tok, 4)]
    co = O.score_spans(ids_key[0][None], q[None, None], np.ones(q.shape, np.float32)[None, None], cfg.key.d_sae, w, max(1, w // 4), 0)
    O.fuse_select(co, None, 1.0, 0.0, 1)


def run_reference(args, cpu_only_sample=None):
    import oracle as O
    cfg, rcfg = WORKLOADS[args.workload]
    inp = C.ScanInputs(cfg, device="cpu")
    weights = {}
    for l in range(cfg.n_layers):
        for which in ("key", "query") if cfg.query else ("key",):
            W, b_enc, b_dec = inp.sae(which, l)
            weights[(which, l)] = (W.float().numpy(), b_enc.numpy(), b_dec.numpy())
    n_tok = cpu_only_sample or 16
    steps, warm = (1, 0) if cpu_only_sample else (args.steps, min(args.warmup, 1))
    for i in range(warm):
        oracle_step(n_tok, i * n_tok, cfg, inp, weights)
    t0 = time.perf_counter()
    for i in range(steps):
        oracle_step(n_tok, (warm + i) * n_tok, cfg, inp, weights)
    dt = time.perf_counter() - t0
    value = steps * n_tok / dt
    cores = O.num_threads()
    sample = (f"{n_tok} context tokens per step through all {cfg.n_layers} layers' SAEs (encode, Top-k, postings) "
              f"plus one query scored on the sample; {steps} steps")
    if cpu_only_sample:
        return {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample, "seconds": dt}
    L_idx = rcfg.scan.L if rcfg else None
    ns = C.n_spans(L_idx, rcfg.width, rcfg.stride) if rcfg else None
    return {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps, "warmup": warm,
            "ms_per_step": dt / steps * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic", "impl": "reference",
            "config": workload_config(cfg, rcfg, L_idx, ns),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}


# ------------------------------------------------------------------------------------------ single-kernel cases

def run_case(args):
    """Runs ONE kernel of the path a few times on a small, L2-exceeding case and prints its event-timed
    duration: the command line that the ncu captures under profiles/ were taken with."""
    import paper_2601_17702_b200 as S
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    cfg = C.CFG3
    inp = C.ScanInputs(cfg, device=dev)
    reps = args.steps
    out = {"case": args.case, "reps": reps}
    if args.case in ("encode_key", "encode_query", "encode_retrieval"):
        which = "query" if args.case == "encode_query" else "key"
        shp = cfg.query if which == "query" else cfg.key
        k = C.CFG4.kq if args.case == "encode_retrieval" else shp.k
        T = args.tokens or (C.CFG4.Q * C.CFG4.nq if args.case == "encode_retrieval" else cfg.chunk)
        sae = S.Sae(*inp.sae(which, 0))
        sae.set_schedule(args.slices, args.max_ctas)
        xs = [inp.x(which, 0, c * T, T) for c in range(2)]
        ids = torch.empty((T, k), dtype=torch.int32, device=dev)
        vals = torch.empty((T, k), dtype=torch.float32, device=dev)
        ws = S.new_workspace(sae.encode_workspace_bytes(T, k), dev)
        run = lambda i: S.s3_sae_encode_topk(sae, xs[i % 2], k, ids, vals, ws)
        out.update(T=T, d_in=shp.d_in, d_sae=shp.d_sae, k=k, flop=2.0 * T * shp.d_in * shp.d_sae)
    elif args.case == "postings":
        n_items, T, k, D = args.items, cfg.chunk, cfg.query.k, cfg.query.d_sae
        g = torch.Generator(device=dev).manual_seed(1)
        idss = [torch.rand((T, D), device=dev, generator=g).topk(k, dim=1).indices.to(torch.int32) for _ in range(n_items)]
        rps = [torch.zeros(D + 1, dtype=torch.int32, device=dev) for _ in range(n_items)]
        pss = [torch.zeros(T * k, dtype=torch.int32, device=dev) for _ in range(n_items)]
        items = [S.make_postings_item(idss[i], D, 0, rps[i], pss[i]) for i in range(n_items)]
        ws = S.new_workspace(min(n_items, 32) * S.s3_postings_workspace_bytes(T, k, D), dev)

        def run(i):
            for j in range(0, n_items, 32):
                S.s3_postings_build_batched(items[j:j + 32], ws)
        out.update(items=n_items, T=T, k=k, d_sae=D, bytes=n_items * (T * k * 8 + (D + 1) * 4))
    elif args.case == "score":
        # retrieval scoring alone: a random index of L tokens (k ids per token out of D features) as one
        # merged CSR, Q queries of nq tokens with kq ids each; bytes = gathered postings + lexical scores + outputs
        r = C.CFG4
        nQ = args.queries or r.Q
        L = args.tokens or r.scan.L
        k, D = (r.scan.key.k, r.scan.key.d_sae) if not args.tokens else (16, 8192)
        stride = r.stride if not args.tokens else 64
        g = torch.Generator(device=dev).manual_seed(1)
        ids = torch.cat([torch.rand((min(65536, L - t0), D), device=dev, generator=g).topk(k, dim=1).indices.to(torch.int32)
                         for t0 in range(0, L, 65536)])
        rp32 = torch.zeros(D + 1, dtype=torch.int32, device=dev)
        pos = torch.zeros(L * k, dtype=torch.int32, device=dev)
        step_t = 131072
        ws = S.new_workspace(S.s3_postings_workspace_bytes(step_t, k, D), dev)
        ix = S.Index(1, D, 64 << 20)
        for t0 in range(0, L, step_t):
            n = min(step_t, L - t0)
            ix.stream_wait()
            S.s3_postings_build(ids[t0:t0 + n], D, t0, rp32, pos, ws)
            ix.append(0, rp32, pos, n, k, t0)
        rp, ps, _ = ix.export_csr(0)
        csr = [(rp.to(dev), ps.to(dev))]
        ix.close()
        q_ids = torch.rand((nQ * r.nq, D), device=dev, generator=g).topk(r.kq, dim=1).indices.to(torch.int32).view(1, nQ, r.nq, r.kq)
        q_vals = torch.ones(q_ids.shape, dtype=torch.float32, device=dev)
        ns = C.n_spans(L, r.width, stride)
        bm25 = G.gamma21(r.bm25_seed, nQ, ns).to(dev)
        top_idx = torch.empty((nQ, r.s), dtype=torch.int32, device=dev)
        top_score = torch.empty((nQ, r.s), dtype=torch.float32, device=dev)
        lens = (csr[0][0][1:] - csr[0][0][:-1])
        gathered = 0
        for q in range(nQ):
            gathered += int(lens[torch.unique(q_ids[0, q].flatten().long())].sum().item())
        sws = S.new_workspace(S.s3_score_workspace_bytes(nQ, r.nq, r.kq, 1, ns, r.s), dev)
        run = lambda i: S.s3_coactivation_score_topspans(csr, D, L, q_ids, q_vals, r.width, stride, r.s, r.alpha, r.beta, sws,
                                                         bm25, top_idx=top_idx, top_score=top_score)
        if args.compact:
            # the same index in block-delta form: build timed once, then the scorer decodes blocks in its gather
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            cws = S.new_workspace(S.s3_compact_workspace_bytes(csr[0][1].numel(), D), dev)
            S.s3_compact_build(csr[0][0], csr[0][1], D, 0, cws)
            e0.record()
            comp = S.s3_compact_build(csr[0][0], csr[0][1], D, 0, cws)
            e1.record()
            torch.cuda.synchronize()
            ref_idx, ref_score = run(0)
            ref_idx, ref_score = ref_idx.clone(), ref_score.clone()
            run = lambda i: S.s3_coactivation_score_topspans_compact([comp], D, L, q_ids, q_vals, r.width, stride, r.s, r.alpha,
                                                                     r.beta, sws, bm25, top_idx=top_idx, top_score=top_score)
            run(0)
            torch.cuda.synchronize()
            out.update(compact_bytes=comp.nbytes(), compact_build_ms=e0.elapsed_time(e1),
                       same_result=bool(torch.equal(ref_idx, top_idx) and torch.equal(ref_score, top_score)))
        out.update(L=L, d_sae=D, k=k, Q=nQ, nq=r.nq, kq=r.kq, spans=ns, stride=stride, gathered_postings=gathered,
                   index_bytes=int(ps.numel()) * 4, bytes=gathered * 4 + nQ * ns * 4 + nQ * r.s * 8)
    elif args.case == "heads":
        # per-head SAE as in Sec. 3.3 (x in R^d_head, one feature-ID space): the key SAE's dictionary width and k with
        # d_head = 128 inputs, 8 KV heads per token, then head aggregation back to k features per token
        H, d_head, D, k = 8, 128, cfg.key.d_sae, args.k or cfg.key.k
        T = args.tokens or cfg.chunk
        g = torch.Generator(device=dev).manual_seed(1)
        W = (torch.randn((d_head, D), device=dev, generator=g) / d_head ** 0.5).to(torch.bfloat16)
        sae = S.Sae(W, torch.zeros(D, device=dev), torch.zeros(d_head, device=dev))
        xs = [torch.randn((T * H, d_head), device=dev, generator=g).to(torch.bfloat16) for _ in range(2)]
        ids = torch.empty((T * H, k), dtype=torch.int32, device=dev)
        vals = torch.empty((T * H, k), dtype=torch.float32, device=dev)
        ws = S.new_workspace(sae.encode_workspace_bytes(T * H, k), dev)

        def run(i):
            S.s3_sae_encode_topk(sae, xs[i % 2], k, ids, vals, ws)
            if not args.no_union:
                S.s3_head_aggregate_topk(ids.view(T, H, k), vals.view(T, H, k), D, k)
        out.update(T=T, H=H, d_head=d_head, d_sae=D, k=k, flop=2.0 * T * H * d_head * D)
    elif args.case == "project_encode":
        # the key projection of a Llama-3.1-8B layer (d_model 4096 -> 8 KV heads of 128) and the per-head SAE (128 -> 16384) of one
        # chunk: fused (the projected tile stays on the SM) or, with --no-union, as the chain projection -> bf16 K -> encode
        d_model, H, D, k = 4096, 8, cfg.key.d_sae, args.k or cfg.key.k
        T = args.tokens or cfg.chunk
        g = torch.Generator(device=dev).manual_seed(1)
        Wp = (torch.randn((d_model, H * 128), device=dev, generator=g) / d_model ** 0.5).to(torch.bfloat16)
        proj = S.Sae(Wp, torch.zeros(H * 128, device=dev), torch.zeros(d_model, device=dev))
        W = (torch.randn((128, D), device=dev, generator=g) / 128 ** 0.5).to(torch.bfloat16)
        sae = S.Sae(W, torch.zeros(D, device=dev), torch.zeros(128, device=dev))
        hs = [torch.randn((T, d_model), device=dev, generator=g).to(torch.bfloat16) for _ in range(2)]
        ids = torch.empty((T, H, k), dtype=torch.int32, device=dev)
        vals = torch.empty((T, H, k), dtype=torch.float32, device=dev)
        xbuf = torch.empty((T, H * 128), dtype=torch.bfloat16, device=dev)
        pws = S.new_workspace(64, dev)
        ws = S.new_workspace(max(S.s3_sae_project_encode_workspace_bytes(sae, T, H, k), sae.encode_workspace_bytes(T * H, k)), dev)

        def run(i):
            if args.no_union:
                S.s3_sae_preact(proj, hs[i % 2], torch.bfloat16, xbuf, pws)
                S.s3_sae_encode_topk(sae, xbuf.view(T * H, 128), k, ids.view(T * H, k), vals.view(T * H, k), ws)
            else:
                S.s3_sae_project_encode_topk(proj, sae, hs[i % 2], H, k, ids, vals, ws)
        out.update(T=T, d_model=d_model, H=H, d_sae=D, k=k, fused=not args.no_union, flop=2.0 * T * d_model * H * 128 + 2.0 * T * H * 128 * D)
    elif args.case == "project":
        # the upstream projections of a Llama-3.1-8B layer on one chunk (d_model 4096 -> keys 1024, queries 4096) through the
        # dense-epilogue form of the encode GEMM, bf16 in and out
        d_model = 4096
        d_out = args.k or 1024
        T = args.tokens or cfg.chunk
        g = torch.Generator(device=dev).manual_seed(1)
        Wp = (torch.randn((d_model, d_out), device=dev, generator=g) / d_model ** 0.5).to(torch.bfloat16)
        proj = S.Sae(Wp, torch.zeros(d_out, device=dev), torch.zeros(d_model, device=dev))
        hs = [torch.randn((T, d_model), device=dev, generator=g).to(torch.bfloat16) for _ in range(2)]
        outp = torch.empty((T, d_out), dtype=torch.bfloat16, device=dev)
        pws = S.new_workspace(64, dev)
        run = lambda i: S.s3_sae_preact(proj, hs[i % 2], torch.bfloat16, outp, pws)
        out.update(T=T, d_model=d_model, d_out=d_out, flop=2.0 * T * d_model * d_out)
    elif args.case == "train":
        # one fp32 training step of the paper's SAE shape (appendix: batches of 4096 tokens, expansion 128 over d_head = 128,
        # k = 128, Adam at 1e-3): encode + Top-k, backward through the code, Adam on the four parameter tensors
        T, d_in, D, k = args.tokens or 4096, 128, 16384, args.k or 128
        g = torch.Generator(device=dev).manual_seed(1)
        W_enc = torch.randn((d_in, D), device=dev, generator=g) / d_in ** 0.5
        params = [W_enc, torch.zeros(D, device=dev), W_enc.t().contiguous(), torch.zeros(d_in, device=dev)]
        moments = [(torch.zeros_like(p), torch.zeros_like(p)) for p in params]
        xs = [torch.randn((T, d_in), device=dev, generator=g) for _ in range(2)]
        ids = torch.empty((T, k), dtype=torch.int32, device=dev)
        vals = torch.empty((T, k), dtype=torch.float32, device=dev)
        bws = S.new_workspace(S.s3_sae_backward_workspace_bytes(T), dev)
        state = {"step": 0}
        if args.fp32_forward:
            sae = S.Sae(params[0], params[1], params[3])      # fp32: the handle reads the parameters in place
            ws = S.new_workspace(sae.encode_workspace_bytes(T, k), dev)
        else:
            W16 = torch.empty((d_in, D), dtype=torch.bfloat16, device=dev)
            x16 = torch.empty((T, d_in), dtype=torch.bfloat16, device=dev)
            ws = None

        def run(i):
            nonlocal ws
            state["step"] += 1
            x = xs[i % 2]
            if args.fp32_forward:
                S.s3_sae_encode_topk(sae, x, k, ids, vals, ws)
                code = vals
            else:
                # the tensor cores select the active set from bf16 copies; the gradient below is taken in fp32
                S.s3_cast_f32_to_bf16(params[0], W16)
                S.s3_cast_f32_to_bf16(x, x16)
                sae16 = S.Sae(W16, params[1], params[3])
                if ws is None:
                    ws = S.new_workspace(sae16.encode_workspace_bytes(T, k), dev)
                S.s3_sae_encode_topk(sae16, x16, k, ids, vals, ws)
                code = None
            _, gWe, gbe, gWd, gbd = S.s3_sae_backward(params[0], params[2], params[3], x, ids, code, bws, b_enc=params[1])
            for p, (m, v), gr in zip(params, moments, (gWe, gbe, gWd, gbd)):
                S.s3_adam_update(p, m, v, gr, 1e-3, 0.9, 0.999, 1e-8, state["step"])
            if not args.fp32_forward:
                sae16.close()                                 # its buffers return to torch's allocator in stream order
        out.update(T=T, d_in=d_in, d_sae=D, k=k, forward="fp32" if args.fp32_forward else "bf16", flop=2.0 * T * d_in * D, adam_bytes=(2 * d_in * D + D + d_in) * 28)
    elif args.case == "decode":
        # SAE decode alone on the key SAE's shape: x_hat = z_hat W_dec + b_dec and the squared reconstruction error.
        # bytes = the k gathered dictionary rows per token (mostly L2 hits: the dictionary is 32 MB) + x read + x_hat written
        shp = cfg.key
        T, k = args.tokens or cfg.chunk, shp.k
        g = torch.Generator(device=dev).manual_seed(1)
        W_dec = (torch.randn((shp.d_sae, shp.d_in), device=dev, generator=g) / shp.d_in ** 0.5).to(torch.bfloat16)
        b_dec = torch.zeros(shp.d_in, device=dev)
        xs = [torch.randn((T, shp.d_in), device=dev, generator=g).to(torch.bfloat16) for _ in range(2)]
        idss = [torch.cat([torch.rand((2048, shp.d_sae), device=dev, generator=g).topk(k, dim=1).indices.to(torch.int32)
                           for _ in range(0, T, 2048)])[:T].contiguous() for _ in range(2)]
        vals = torch.rand((T, k), device=dev, generator=g)
        run = lambda i: S.s3_sae_decode(W_dec, b_dec, idss[i % 2], vals, xs[i % 2])
        out.update(T=T, d_in=shp.d_in, d_sae=shp.d_sae, k=k, bytes=T * k * shp.d_in * 2 + T * shp.d_in * (2 + 4),
                   hbm_bytes=shp.d_sae * shp.d_in * 2 + T * shp.d_in * (2 + 4))
    elif args.case == "density":
        # the paper's Phase 2 tail alone: per-position relevance (Eq. 6), box-smoothed density (48 taps), greedy NMS
        # with 40 centres, then the index-set union of Eq. 7 (256-token windows, 64 lexical hits, 64 lead / tail);
        # same random index and queries as the score case
        r = C.CFG4
        L = args.tokens or r.scan.L
        k, D = (r.scan.key.k, r.scan.key.d_sae) if not args.tokens else (16, 8192)
        g = torch.Generator(device=dev).manual_seed(1)
        ids = torch.cat([torch.rand((min(65536, L - t0), D), device=dev, generator=g).topk(k, dim=1).indices.to(torch.int32)
                         for t0 in range(0, L, 65536)])
        rp32 = torch.zeros(D + 1, dtype=torch.int32, device=dev)
        pos = torch.zeros(L * k, dtype=torch.int32, device=dev)
        ws = S.new_workspace(S.s3_postings_workspace_bytes(L, k, D), dev)
        S.s3_postings_build(ids, D, 0, rp32, pos, ws)
        layers = [(rp32.to(torch.int64), pos)]
        q_ids = torch.rand((r.Q * r.nq, D), device=dev, generator=g).topk(r.kq, dim=1).indices.to(torch.int32).view(1, r.Q, r.nq, r.kq)
        q_vals = torch.rand(q_ids.shape, dtype=torch.float32, device=dev, generator=g)
        lexical = torch.randint(0, L, (r.Q, 64), device=dev, generator=g, dtype=torch.int32)
        dws = S.new_workspace(S.s3_density_workspace_bytes(r.Q, L, 1, D, r.nq, r.kq), dev)
        fws = S.new_workspace(S.s3_fuse_workspace_bytes(r.Q, L), dev)
        cap = 40 * 256 + 64 + 128
        lens = (rp32[1:] - rp32[:-1])
        gathered = 0
        for q in range(r.Q):
            gathered += int(lens[torch.unique(q_ids[0, q].flatten().long())].sum().item())

        def run(i):
            c, _ = S.s3_position_density_topcenters(layers, D, L, q_ids, q_vals, 48, 24, 40, dws)
            if not args.no_union:
                S.s3_fuse_index_sets(c, 256, lexical, 64, 64, L, cap, fws)
        out.update(L=L, d_sae=D, k=k, Q=r.Q, nq=r.nq, kq=r.kq, conv_kernel=48, nms_radius=24, n_centers=40,
                   gathered_postings=gathered, bytes=gathered * 4 + r.Q * L * 16)
    else:
        raise SystemExit(f"unknown case {args.case}")
    for i in range(2):
        run(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(reps):
        run(i)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / reps
    out["ms"] = ms
    if "flop" in out:
        out["tflops"] = out["flop"] / ms / 1e9
    if "bytes" in out:
        out["gbs"] = out["bytes"] / ms / 1e6
    print(json.dumps(out), flush=True)


def spawn_ranks(args) -> int:
    """`python bench.py --gpus N` without a launcher around it: N child processes of this script, one per GPU, with the
    rendezvous variables a launcher would set (127.0.0.1). Rank 0's JSON line is the output; returns the worst exit code."""
    import socket
    with socket.socket() as sck:
        sck.bind(("127.0.0.1", 0))
        port = sck.getsockname()[1]
    procs = []
    for r in range(args.gpus):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(args.gpus), LOCAL_WORLD_SIZE=str(args.gpus),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__)] + sys.argv[1:], env=env))
    return max(abs(p.wait()) for p in procs)


def run_stub(args, rank, world):
    """The launch, barrier and max-over-ranks plumbing of a multi-rank run with a sleep in place of the GPU step
    (backend gloo, no GPU): what the CPU tests drive."""
    def step():
        time.sleep(0.002 * (rank + 1))
    for _ in range(args.warmup):
        step()
    torch.distributed.barrier()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = time.perf_counter() - t0
    torch.distributed.barrier()
    slowest = max_over_ranks(dt, world)
    if rank != 0:
        return None
    return {"metric": METRIC, "value": whole_job_rate(1, args.steps, world, slowest), "unit": "stub steps/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": slowest / args.steps * 1e3, "impl": "stub"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--case", default=None, help="run one kernel alone: encode_key | encode_query | encode_retrieval | postings | score | density | decode | heads | train | project (--k = output width) | project_encode (--no-union: unfused chain)")
    ap.add_argument("--workload", default="cfg3", choices=sorted(WORKLOADS), help="cfg3 = the 128K-token 4-layer key+query scan the metric is quoted on (default); cfg5 = the 1M-token 8-layer Zipf scan; cfg2 = the 32K-token one-layer scan; cfg1 = the tiny fp32 scan")
    ap.add_argument("--tokens", type=int, default=0)
    ap.add_argument("--slices", type=int, default=0)
    ap.add_argument("--max-ctas", type=int, default=0)
    ap.add_argument("--items", type=int, default=8)
    ap.add_argument("--k", type=int, default=0, help="heads case: Top-k per head and per token (default: the key SAE's)")
    ap.add_argument("--queries", type=int, default=0, help="score case: number of queries (default: the retrieval workload's 256)")
    ap.add_argument("--fp32-forward", action="store_true", help="train case: fp32 FFMA forward pass instead of the bf16 one")
    ap.add_argument("--compact", action="store_true", help="score case: read the block-delta compact index")
    ap.add_argument("--no-union", action="store_true", help="density case: leave out the index-set union; heads case: leave out the aggregation")
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=96)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference", "stub"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--overlap", action="store_true", help="run the grouped launch of narrow encoders on a second stream beside the wide encoders' launches (on the SMs those leave free) instead of after them")
    ap.add_argument("--group", default="auto", help="how a chunk's encodes are launched: all | slot | none | <stream name> | auto")
    ap.add_argument("--cpu-sample-tokens", type=int, default=2048, help="context tokens the CPU oracle is timed on for cpu_baseline")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and not args.case:
        sys.exit(spawn_ranks(args))               # no launcher around us: start the ranks ourselves
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.case:
        if rank == 0:
            run_case(args)
        return
    if args.impl == "reference":
        if rank == 0:
            print(json.dumps(run_reference(args)), flush=True)
        return
    if args.impl == "stub":
        torch.distributed.init_process_group("gloo")
        out = run_stub(args, rank, world)
        if rank == 0:
            print(json.dumps(out), flush=True)
        torch.distributed.destroy_process_group()
        return
    if world > 1:
        torch.distributed.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    out = run_ours(args, rank, world, local_rank)
    if rank == 0:
        if world == 1 and not args.no_cpu_baseline:
            out["cpu_baseline"] = run_reference(args, cpu_only_sample=args.cpu_sample_tokens)
        print(json.dumps(out), flush=True)
    if world > 1:
        torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
