#!/usr/bin/env python
"""Benchmark of the per-axis 1-bit delta hot path on B200.

A step is one pass of the whole path over a Llama-7B-shaped decoder block (q/k/v/o 4096x4096,
gate/up 11008x4096, down 4096x11008), all through the C ABI:

    pack      : pd_pack_delta on the 7 linears (mask + both scale vectors)
    decode    : pd_linear, M in {1, 4, 16} x {row, col} x 7 linears          <- headline metric
    prefill   : pd_linear, M in {256, 2048, 8192} x {row, col} x 7 linears
    multi     : pd_linear_multivariant, 16 variants, M = 64 and M = 64 + 4*512
    merge     : pd_merge on the 7 linears, row and col

`value` is the decode section: algorithmic bytes (2 B weight + 1/8 B mask per element, plus x, y
and v) divided by its device time, GB/s.  Every other section is reported under "sections" with
its own unit.  One process per GPU; with N > 1 the ranks are independent replicas (the path has
no exchange step), timed with a barrier on both sides and the max over ranks.

--impl reference times the CPU oracle (the stand-in for a reference implementation, which the
paper does not have) on a bounded sample of the same decode workload.
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

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

BLOCK = [("q", 4096, 4096), ("k", 4096, 4096), ("v", 4096, 4096), ("o", 4096, 4096),
         ("gate", 11008, 4096), ("up", 11008, 4096), ("down", 4096, 11008)]
DECODE_M = (1, 4, 16)
PREFILL_M = (256, 2048, 8192)
N_VARIANTS = 16
MULTI_M = (64, 64 + 4 * 512)
ROW, COL = 0, 1
# ncu dram__bytes_read.sum + dram__bytes_write.sum over algorithmic bytes, 4096 x 11008 captures in profiles/
# (merge: reads only -- half of its writes are still dirty in L2 when the kernel ends)
NCU_DRAM_RATIO = {"decode": 96.19 / 95.81, "pack": (180.52 + 4.82) / (180.36 + 5.67), "merge": 1.0}
METRIC = "fused delta-linear decode HBM GB/s (7B block sweep, M in {1,4,16}, row+col axes)"


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "tflops_burst": p["bf16_tflops"],
                "tflops_sustained": p["bf16_tflops_sustained"], "source": "measured"}
    return {"hbm_gbs": 6650.0, "tflops_burst": 1590.0, "tflops_sustained": 1400.0, "source": "fallback"}


def linear_bytes(m, d_out, d_in, axis):
    e = d_out * d_in
    return 2 * e + e // 8 + 2 * m * (d_in + d_out) + 2 * (d_out if axis == ROW else d_in)


def pack_bytes(d_out, d_in):
    e = d_out * d_in
    return 4 * e + e // 8 + 2 * (d_out + d_in)


def merge_bytes(d_out, d_in, axis):
    e = d_out * d_in
    return 4 * e + e // 8 + 2 * (d_out if axis == ROW else d_in)


def multi_bytes(m, d_out, d_in):
    e = d_out * d_in
    return 2 * e + N_VARIANTS * (e // 8) + 2 * m * (d_in + d_out) + 2 * N_VARIANTS * d_out


class ClockSampler:
    """Samples nvidia-smi SM clocks and throttle reasons while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([t.strip() for t in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx = float(r[1])
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, r[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


# --------------------------------------------------------------------------- reference arm (CPU oracle)
def oracle_sample(steps, warmup):
    """Times the oracle's fused linear on a bounded sample of the decode workload: the q (4096x4096)
    and gate (11008x4096) linears at M in {1, 4, 16}, row and col axis, on the host cores."""
    from oracle import pd_oracle as orc
    from paper_2512_19720_b200 import synth
    cases, nbytes = [], 0
    for d_out, d_in in ((4096, 4096), (11008, 4096)):
        w_b = synth.gen_base(d_out, d_in, 0)
        w_f = synth.gen_finetuned(w_b, 1000)
        mask, v_row, v_col = orc.pack(w_f, w_b)
        for m in DECODE_M:
            x = synth.gen_x(m, d_in, 2000 + m)
            cases.append((x, w_b, mask, v_row, v_col))
            nbytes += linear_bytes(m, d_out, d_in, ROW) + linear_bytes(m, d_out, d_in, COL)
    times = []
    for i in range(warmup + steps):
        t0 = time.perf_counter()
        for x, w_b, mask, v_row, v_col in cases:
            orc.linear(x, w_b, mask, v_row, ROW)
            orc.linear(x, w_b, mask, v_col, COL)
        if i >= warmup:
            times.append(time.perf_counter() - t0)
    dt = sum(times) / len(times)
    return {"value": nbytes / dt / 1e9, "unit": "GB/s", "cores": orc.threads(), "kind": "oracle",
            "sample": f"oracle linear on the q (4096x4096) and gate (11008x4096) linears, M in {{1,4,16}}, row+col: "
                      f"{len(times)} timed passes of {dt:.2f} s after {warmup} warm-up",
            "ms_per_step": dt * 1e3}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cb = oracle_sample(max(1, min(args.steps, 5)), 1)
    line = {"impl": "reference", "metric": METRIC, "value": cb["value"], "unit": "GB/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": cb["ms_per_step"], "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": "llama7b_block_decode (bounded sample: q and gate linears, M in {1,4,16}, row+col)"},
            "cpu_baseline": {k: cb[k] for k in ("value", "unit", "cores", "kind", "sample")},
            "e2e": {"value": cb["value"], "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def max_over_ranks(values, world, device):
    """Element-wise maximum of a list of floats over all ranks (every rank gets the result): the time of a
    multi-GPU step is the slowest rank's.  Uses the default process group (nccl on GPUs, gloo in the CPU tests)."""
    import torch
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


# --------------------------------------------------------------------------- our arm
def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2512_19720_b200 import api, synth_torch

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    # ---- resident state (untimed): base, fine-tune, 16 variants' deltas, activations
    layers = []
    for li, (name, d_out, d_in) in enumerate(BLOCK):
        w_b = synth_torch.gen_base(d_out, d_in, 10 + li, dev)
        w_f = synth_torch.gen_finetuned(w_b, 100 + li)
        mask, v_row, v_col = api.pd_pack_delta(w_f, w_b)
        stride = max(d_out, d_in)
        masks = torch.empty((N_VARIANTS, d_out, d_in // 32), dtype=torch.int32, device=dev)
        vs = torch.zeros((N_VARIANTS, stride), dtype=torch.float16, device=dev)
        for g in range(N_VARIANTS):
            wf_g = synth_torch.gen_finetuned(w_b, 1000 + 16 * li + g)
            _, vr, _ = api.pd_pack_delta(wf_g, w_b, want_col=False, mask=masks[g])
            vs[g, :d_out] = vr
            del wf_g
        layers.append(dict(name=name, d_out=d_out, d_in=d_in, w_b=w_b, w_f=w_f, mask=mask, v=(v_row, v_col),
                           masks=masks, vs=vs, w_hat=torch.empty_like(w_b)))
    max_m = max(PREFILL_M + MULTI_M)
    x_all = {d_in: synth_torch.gen_x(max_m, d_in, 2000 + d_in, dev) for d_in in (4096, 11008)}
    y_all = {d_out: torch.empty((max_m, d_out), dtype=torch.float16, device=dev) for d_out in (4096, 11008)}
    ids = {m: synth_torch.gen_ids(m, N_VARIANTS, 3000 + m, dev) for m in MULTI_M}
    axes = [ROW] * N_VARIANTS
    torch.cuda.synchronize()

    sections = ["pack", "decode", "prefill", "multi_decode", "multi_prefill", "merge"]

    def run_pack():
        for L in layers:
            api.pd_pack_delta(L["w_f"], L["w_b"], mask=L["mask"], v_row=L["v"][0], v_col=L["v"][1])

    def run_linear(ms):
        for m in ms:
            for axis in (ROW, COL):
                for L in layers:
                    api.pd_linear(x_all[L["d_in"]][:m], L["w_b"], L["mask"], L["v"][axis], axis, y=y_all[L["d_out"]][:m])

    def run_multi(m):
        if True:
            for L in layers:
                api.pd_linear_multivariant(x_all[L["d_in"]][:m], ids[m], L["w_b"], L["masks"], L["vs"], axes,
                                           y=y_all[L["d_out"]][:m])

    def run_merge():
        for axis in (ROW, COL):
            for L in layers:
                api.pd_merge(L["w_b"], L["mask"], L["v"][axis], axis, w_hat=L["w_hat"])

    bodies = {"pack": run_pack, "decode": lambda: run_linear(DECODE_M), "prefill": lambda: run_linear(PREFILL_M),
              "multi_decode": lambda: run_multi(MULTI_M[0]), "multi_prefill": lambda: run_multi(MULTI_M[1]),
              "merge": run_merge}

    # Every section is captured once into a CUDA graph (the calls only enqueue kernels on the current
    # stream) and replayed: a decode kernel lasts ~10 us, less than the host needs to issue it.
    side = torch.cuda.Stream(device=dev)
    graphs, launches_per = {}, {}
    for name in sections:
        bodies[name]()  # eager once: sizes every cached workspace before capture
    torch.cuda.synchronize()
    for name in sections:
        g = torch.cuda.CUDAGraph()
        n0 = api.launch_count()
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                bodies[name]()
        launches_per[name] = api.launch_count() - n0
        graphs[name] = g
    torch.cuda.synchronize()

    def step(events=None):
        for i, name in enumerate(sections):
            if events is not None:
                events[i].record()
            graphs[name].replay()
        if events is not None:
            events[len(sections)].record()

    work = {
        "pack": sum(pack_bytes(L["d_out"], L["d_in"]) for L in layers),
        "decode": sum(linear_bytes(m, L["d_out"], L["d_in"], ax) for m in DECODE_M for ax in (ROW, COL) for L in layers),
        "prefill": sum(2 * m * L["d_out"] * L["d_in"] for m in PREFILL_M for _ in (ROW, COL) for L in layers),
        "multi_decode": sum(multi_bytes(MULTI_M[0], L["d_out"], L["d_in"]) for L in layers),
        "multi_prefill": sum(2 * MULTI_M[1] * L["d_out"] * L["d_in"] for L in layers),
        "merge": sum(merge_bytes(L["d_out"], L["d_in"], ax) for ax in (ROW, COL) for L in layers),
    }
    calls_per = {"pack": 7, "decode": 42, "prefill": 42, "multi_decode": 7, "multi_prefill": 7, "merge": 14}

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    barrier()
    if api.pd_device_status() != 0:
        raise RuntimeError("device status latched an error during warm-up")

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    events = [[torch.cuda.Event(enable_timing=True) for _ in range(len(sections) + 1)] for _ in range(args.steps)]
    barrier()
    for k in range(args.steps):
        step(events[k])
    barrier()
    launches = args.steps * sum(launches_per.values())  # kernels inside the replayed graphs
    clocks = sampler.stop() if rank == 0 else None
    if api.pd_device_status() != 0:
        raise RuntimeError("device status latched an error during the timed region")

    sec_ms = {s: sum(events[k][i].elapsed_time(events[k][i + 1]) for k in range(args.steps)) / args.steps
              for i, s in enumerate(sections)}
    total_ms = events[0][0].elapsed_time(events[-1][len(sections)]) / args.steps

    # ---- end to end for the headline metric: host x -> device, pd_linear, y -> host, every call
    host_x = {d_in: x_all[d_in][:16].cpu().pin_memory() for d_in in x_all}
    host_y = {d_out: torch.empty((16, d_out), dtype=torch.float16).pin_memory() for d_out in y_all}
    dx = {d_in: torch.empty((16, d_in), dtype=torch.float16, device=dev) for d_in in x_all}

    def e2e_step():
        for m in DECODE_M:
            for axis in (ROW, COL):
                for L in layers:
                    api.pd_linear_host(host_x[L["d_in"]][:m], dx[L["d_in"]], L["w_b"], L["mask"], L["v"][axis], axis,
                                       y_all[L["d_out"]], host_y[L["d_out"]][:m])
    h2d = sum(2 * m * L["d_in"] for m in DECODE_M for _ in (ROW, COL) for L in layers)
    d2h = sum(2 * m * L["d_out"] for m in DECODE_M for _ in (ROW, COL) for L in layers)
    for _ in range(max(3, args.warmup)):
        e2e_step()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        e2e_step()
    e1.record()
    barrier()
    e2e_ms = e0.elapsed_time(e1) / args.steps

    # ---- max over ranks
    stats = max_over_ranks([total_ms, e2e_ms] + [sec_ms[s] for s in sections], world, dev)
    total_ms, e2e_ms = stats[0], stats[1]
    sec_ms = dict(zip(sections, stats[2:]))

    if rank == 0:
        pk = peaks()
        gbs = {s: work[s] * world / (sec_ms[s] * 1e-3) / 1e9 for s in ("pack", "decode", "multi_decode", "merge")}
        tfl = work["prefill"] * world / (sec_ms["prefill"] * 1e-3) / 1e12
        tfl_mv = work["multi_prefill"] * world / (sec_ms["multi_prefill"] * 1e-3) / 1e12

        def hbm(section, kernel):
            per_gpu = gbs[section] / world
            return {"kernel": kernel, "bound": "hbm", "achieved": round(per_gpu, 1), "peak": pk["hbm_gbs"],
                    "unit": "GB/s", "frac": round(per_gpu / pk["hbm_gbs"], 4), "frac_of": pk["source"],
                    "frac_of_nominal_8TBs": round(per_gpu / 8000.0, 4),
                    # DRAM bytes per call = algorithmic bytes x (ncu dram bytes / algorithmic bytes) of the captured
                    # case under profiles/ (traffic grows in proportion to the elements streamed)
                    "traffic": (round(work[section] / calls_per[section] * NCU_DRAM_RATIO[section])
                                if section in NCU_DRAM_RATIO else None),
                    "algorithmic_bytes_per_call": work[section] // calls_per[section],
                    "avg_call_ms": round(sec_ms[section] / calls_per[section], 5),
                    "share_of_step": round(sec_ms[section] / sum(sec_ms.values()), 4)}
        def tensor(section, tf_total, kernel):
            per_gpu = tf_total / world
            return {"kernel": kernel, "bound": "tensor", "achieved": round(per_gpu, 1), "peak": pk["tflops_sustained"],
                    "unit": "TFLOP/s", "frac": round(per_gpu / pk["tflops_sustained"], 4),
                    "frac_of": pk["source"] + " sustained (fp16 and bf16 share one tensor peak)",
                    "frac_of_burst": round(per_gpu / pk["tflops_burst"], 4),
                    "frac_of_nominal_2250": round(per_gpu / 2250.0, 4), "traffic": None,
                    "algorithmic_flops_per_call": work[section] // calls_per[section],
                    "avg_call_ms": round(sec_ms[section] / calls_per[section], 5),
                    "share_of_step": round(sec_ms[section] / sum(sec_ms.values()), 4)}
        gemm_roof = tensor("prefill", tfl, "gemm_pair_kernel (tcgen05 prefill on CTA pairs)")
        cpu = oracle_sample(4, 1) if (world == 1 and not args.no_cpu_baseline) else None
        all_roofs = {"decode": hbm("decode", "gemv_stream_kernel (decode)"), "pack": hbm("pack", "pack_kernel"),
                     "merge": hbm("merge", "merge_kernel"), "multivariant_decode": hbm("multi_decode", "gemm_kernel (grouped, M=64 over 16 variants)"),
                     "multivariant_prefill": tensor("multi_prefill", tfl_mv, "gemm_kernel (grouped, M=2112 over 16 variants)"),
                     "prefill": gemm_roof}
        dominant = max(all_roofs, key=lambda k: all_roofs[k]["share_of_step"])  # the kernel the step spends most time in
        line = {
            "metric": METRIC, "value": round(gbs["decode"], 1), "unit": "GB/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": round(total_ms, 4), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f16", "data": "synthetic",
            "config": {"workload": "llama7b_block: pack + decode M{1,4,16} + prefill M{256,2048,8192} + "
                                   "multivariant V16 M{64,2112} + merge, row and col axes",
                       "l2": "every sweep streams >= 430 MB of weights, larger than the 126 MB L2",
                       "replicas": "independent per GPU, no collective"},
            "sections": {
                "pack_GBps": round(gbs["pack"], 1), "decode_GBps": round(gbs["decode"], 1),
                "prefill_TFLOPps": round(tfl, 1), "multivariant_decode_GBps": round(gbs["multi_decode"], 1),
                "multivariant_prefill_TFLOPps": round(tfl_mv, 1),
                "merge_GBps": round(gbs["merge"], 1), "ms": {s: round(sec_ms[s], 4) for s in sections}},
            "roofline": dict(all_roofs[dominant], section=dominant),
            "rooflines": all_roofs,
            "e2e": {"value": round(work["decode"] * world / (e2e_ms * 1e-3) / 1e9, 1), "unit": "GB/s",
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": round(e2e_ms, 4),
                    "what": "decode section through pd_linear_host: x from pinned host memory, y back to pinned host memory, every call"},
            "gpu_launches": launches, "clocks": clocks,
        }
        if cpu is not None:
            line["cpu_baseline"] = {k: (round(cpu[k], 3) if k == "value" else cpu[k])
                                    for k in ("value", "unit", "cores", "kind", "sample")}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_only(args):
    """One kernel family on one layer shape: a few calls over rotated weight copies (more than L2 in total),
    timed with CUDA events.  Small enough to sit under a profiler."""
    import torch
    from paper_2512_19720_b200 import api, synth_torch
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    d_out, d_in = (int(t) for t in args.shape.split("x"))
    axis = ROW if args.axis == "row" else COL
    copies = max(2, int(300e6 // (2 * d_out * d_in)) + 1)
    layers = []
    for c in range(copies):
        w_b = synth_torch.gen_base(d_out, d_in, 10 + c, dev)
        w_f = synth_torch.gen_finetuned(w_b, 100 + c)
        mask, v_row, v_col = api.pd_pack_delta(w_f, w_b)
        layers.append((w_b, w_f, mask, (v_row, v_col), torch.empty_like(w_b)))
    x = synth_torch.gen_x(args.m, d_in, 5, dev)
    y = torch.empty((args.m, d_out), dtype=torch.float16, device=dev)

    def call(i):
        w_b, w_f, mask, v, out = layers[i % copies]
        if args.only == "linear":
            api.pd_linear(x, w_b, mask, v[axis], axis, y=y)
        elif args.only == "pack":
            api.pd_pack_delta(w_f, w_b, mask=mask, v_row=v[0], v_col=v[1])
        else:
            api.pd_merge(w_b, mask, v[axis], axis, w_hat=out)

    call(0)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(args.calls):
        call(i + 1)
    e1.record()
    torch.cuda.synchronize()
    if api.pd_device_status() != 0:
        raise RuntimeError("device status latched an error")
    print(json.dumps({"only": args.only, "shape": [d_out, d_in], "m": args.m, "axis": args.axis, "calls": args.calls,
                      "ms_per_call_incl_launch": round(e0.elapsed_time(e1) / args.calls, 5)}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--only", choices=["linear", "pack", "merge"], help="run one kernel family on one layer (for profiling)")
    ap.add_argument("--shape", default="4096x4096")
    ap.add_argument("--m", type=int, default=16)
    ap.add_argument("--axis", default="row", choices=["row", "col"])
    ap.add_argument("--calls", type=int, default=4)
    args = ap.parse_args()
    if args.only:
        run_only(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
