#!/usr/bin/env python
"""Benchmark of the per-axis 1-bit delta hot path on B200.

A step is one pass of the whole path, all through the C ABI, inputs resident in HBM:

  Llama-7B-shaped decoder block (q/k/v/o 4096x4096, gate/up 11008x4096, down 4096x11008)
    pack           pd_pack_delta on the 7 linears (mask + both scale vectors)
    decode_m*      pd_linear, M in {1, 4, 16} x {row, col} x 7 linears             <- headline metric
    *_par*         decode, pack, merge and prefill M = 256 with the sweep's calls dealt to four streams (the linears of a
                   sweep are independent: their kernels may overlap)
    prefill_m*     pd_linear, M in {256, 2048, 8192} x {row, col} x 7 linears
    multi_*        pd_linear_multivariant, 16 variants over one base: 64 decode rows; 64 + 4 x 512 rows with an id
                   per row; the same with one id per 512-row sequence; both batch sizes with mixed axes
    merge          pd_merge on the 7 linears, row and col
    bf16_*         pack, decode (M in {1, 4, 16}), prefill (M = 2048) and merge with bfloat16 weights and activations
    fit_*          one training step of the scales per linear (pd_fit_loss_grad + pd_fit_adamw_step) on 2048 calibration
                   tokens, row axis and col axis
  single 1024 x 1024 layer
    c1_*           pd_linear at M = 1 and 16 over 128 rotated copies (weights from HBM) and on one copy (L2-resident)
  Llama-70B-shaped block, 80 layers streamed through one set of per-layer buffers
    c5_*           pd_pack_delta -> pd_merge -> dense GEMV on the merged weights and fused GEMV, M = 1

`value` is the decode sections together: algorithmic bytes (2 B weight + 1/8 B mask per element, plus x, y and v)
divided by their device time, GB/s.  Every section is reported under "sections" / "rooflines" with its own unit.
One process per GPU; with N > 1 the ranks are independent replicas (the path has no exchange step), timed with a
barrier on both sides and the max over ranks.  `--gpus N` without a torchrun environment starts the N ranks itself.

--impl reference times the CPU oracle (the stand-in for a reference implementation, which the paper does not
have) on a bounded sample of the same decode workload.
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

BLOCK = [("q", 4096, 4096), ("k", 4096, 4096), ("v", 4096, 4096), ("o", 4096, 4096),
         ("gate", 11008, 4096), ("up", 11008, 4096), ("down", 4096, 11008)]
BLOCK_70B = [("q", 8192, 8192), ("k", 1024, 8192), ("v", 1024, 8192), ("o", 8192, 8192),
             ("gate", 28672, 8192), ("up", 28672, 8192), ("down", 8192, 28672)]
N_LAYERS_70B = 80
DECODE_M = (1, 4, 16)
PREFILL_M = (256, 2048, 8192)
N_VARIANTS = 16
MULTI_M = (64, 64 + 4 * 512)
FIT_M = 2048  # calibration tokens per training step of the scale fit
C1_COPIES = 128
ROW, COL = 0, 1
# ncu dram bytes / algorithmic bytes of the captures summarised in profiles/ (4096x11008 for the streaming kernels,
# 4096x4096 with 64 tokens over 16 variants for the multi-variant decode; their traffic grows in proportion to the
# elements streamed).  Pack and multi-variant decode: read + write.  Decode GEMV and merge: the read ratio -- the GEMV
# writes 8 KB, what ncu counts as its writes is earlier data leaving the L2, and half of merge's writes are still dirty
# in L2 when the kernel ends.  None = the kernel has changed since its counters were taken.
NCU_DRAM_RATIO = {"decode": 1.004, "pack": 1.0, "merge": 1.0, "multi_decode": 0.987}
METRIC = "fused delta-linear decode HBM GB/s (7B block sweep, M in {1,4,16}, row+col axes)"


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "tflops_burst": p["bf16_tflops"],
                "tflops_sustained": p["bf16_tflops_sustained"], "source": "measured"}
    return {"hbm_gbs": 6650.0, "tflops_burst": 1590.0, "tflops_sustained": 1400.0, "source": "fallback"}


def linear_bytes(m, d_out, d_in, axis, delta=True):
    e = d_out * d_in
    return 2 * e + (e // 8 + 2 * (d_out if axis == ROW else d_in) if delta else 0) + 2 * m * (d_in + d_out)


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


# --------------------------------------------------------------------------- CPU oracle legs
def _timed(fn, passes, warmup=1):
    for _ in range(warmup):
        fn()
    t0 = time.perf_counter()
    for _ in range(passes):
        fn()
    return (time.perf_counter() - t0) / passes


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
            "ms_per_step": dt * 1e3, "timed_passes": len(times)}


def oracle_other_ops():
    """The oracle's other operations, each timed once after one warm-up call on the host cores: pack and merge on
    every 7B shape, the fused linear at M = 256 on a sample of 8 token rows (4096x4096 and 11008x4096), and the
    multi-variant linear at M = 64 over 16 variants (4096x4096).  Same algorithmic bytes / flops as the GPU rows."""
    from oracle import pd_oracle as orc
    from paper_2512_19720_b200 import synth
    out = {}
    for d_out, d_in in ((4096, 4096), (11008, 4096), (4096, 11008)):
        tag = f"{d_out}x{d_in}"
        w_b = synth.gen_base(d_out, d_in, 0)
        w_f = synth.gen_finetuned(w_b, 1000)
        mask, v_row, v_col = orc.pack(w_f, w_b)
        out[f"pack_{tag}_GBps"] = round(pack_bytes(d_out, d_in) / _timed(lambda: orc.pack(w_f, w_b), 1) / 1e9, 3)
        out[f"merge_row_{tag}_GBps"] = round(merge_bytes(d_out, d_in, ROW) / _timed(lambda: orc.merge(w_b, mask, v_row, ROW), 1) / 1e9, 3)
        out[f"merge_col_{tag}_GBps"] = round(merge_bytes(d_out, d_in, COL) / _timed(lambda: orc.merge(w_b, mask, v_col, COL), 1) / 1e9, 3)
        if d_in == 4096:
            x = synth.gen_x(256, d_in, 2256)
            rows = synth.sample_rows(256, n_random=2)[:8]
            xs = x[rows].copy()
            dt = _timed(lambda: orc.linear(xs, w_b, mask, v_row, ROW), 1)
            out[f"linear_m256_{tag}_GFLOPps (8 sampled token rows)"] = round(2.0 * len(rows) * d_out * d_in / dt / 1e9, 2)
        if d_out == d_in:
            import numpy as np
            masks = np.empty((N_VARIANTS, d_out, d_in // 32), dtype=np.uint32)
            vs = np.zeros((N_VARIANTS, d_out), dtype=np.float16)
            for g in range(N_VARIANTS):
                masks[g], vs[g], _ = orc.pack(synth.gen_finetuned(w_b, 1001 + g), w_b, want_col=False)
            x = synth.gen_x(64, d_in, 2064)
            ids = synth.gen_ids(64, N_VARIANTS, 3064)
            axes = np.zeros(N_VARIANTS, dtype=np.uint8)
            dt = _timed(lambda: orc.linear_multivariant(x, ids, w_b, masks, vs, axes), 1)
            out[f"multivariant_m64_v16_{tag}_GBps"] = round(multi_bytes(64, d_out, d_in) / dt / 1e9, 3)
    # one loss + gradient evaluation of the scale fit on 4 calibration tokens (4096x4096), both axes
    from oracle import pd_oracle_fit as orc_fit
    w_b = synth.gen_base(4096, 4096, 0)
    w_f = synth.gen_finetuned(w_b, 1000)
    mask, v_row, v_col = orc.pack(w_f, w_b)
    x = synth.gen_x(4, 4096, 2004)
    y = synth.gen_teacher_outputs(x, w_f)
    for axis, v, mult in ((ROW, v_row, 2), (COL, v_col, 3)):
        dt = _timed(lambda: orc_fit.loss_grad(x, y, w_b, mask, v.astype("float64"), axis), 1)
        out[f"fit_{'row' if axis == ROW else 'col'}_4096x4096_GFLOPps (4 tokens)"] = round(mult * 2.0 * 4 * 4096 * 4096 / dt / 1e9, 3)
    out["cores"] = orc.threads()
    return out


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    steps = max(1, min(args.steps, 5))  # every pass is ~2 s of CPU work: a bounded number of them
    cb = oracle_sample(steps, 1)
    line = {"impl": "reference", "metric": METRIC, "value": cb["value"], "unit": "GB/s", "n_gpus": args.gpus,
            "steps": cb["timed_passes"], "warmup": 1, "ms_per_step": cb["ms_per_step"], "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": "llama7b_block_decode (bounded sample: q and gate linears, M in {1,4,16}, row+col)",
                       "requested_steps": args.steps, "requested_warmup": args.warmup},
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


def replica_command(n, argv):
    """Command line that starts n replica ranks of this script on this node (one per GPU), as the multi-GPU launch
    contract does: torch.distributed.run, rendezvous on 127.0.0.1 and a free port."""
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1",
            "--master-port", str(port), os.path.abspath(__file__)] + list(argv)


def spawn_replicas(n, argv):
    """`bench.py --gpus N` outside a torchrun environment: start the N ranks and pass rank 0's line through."""
    r = subprocess.run(replica_command(n, argv), stdout=subprocess.PIPE, text=True)
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    if lines:
        print(lines[-1])
    return r.returncode


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
        vs = torch.zeros((N_VARIANTS, stride), dtype=torch.float16, device=dev)       # all row axis
        vs_mixed = torch.zeros((N_VARIANTS, stride), dtype=torch.float16, device=dev)  # odd variants col axis
        for g in range(N_VARIANTS):
            wf_g = synth_torch.gen_finetuned(w_b, 1000 + 16 * li + g)
            _, vr, vc = api.pd_pack_delta(wf_g, w_b, mask=masks[g])
            vs[g, :d_out] = vr
            if g % 2:
                vs_mixed[g, :d_in] = vc
            else:
                vs_mixed[g, :d_out] = vr
            del wf_g
        layers.append(dict(name=name, d_out=d_out, d_in=d_in, w_b=w_b, w_f=w_f, mask=mask, v=(v_row, v_col),
                           masks=masks, vs=vs, vs_mixed=vs_mixed, w_hat=torch.empty_like(w_b)))
    max_m = max(PREFILL_M + MULTI_M)
    x_all = {d_in: synth_torch.gen_x(max_m, d_in, 2000 + d_in, dev) for d_in in (4096, 11008)}
    y_all = {d_out: torch.empty((max_m, d_out), dtype=torch.float16, device=dev) for d_out in (4096, 11008)}
    ids = {m: synth_torch.gen_ids(m, N_VARIANTS, 3000 + m, dev) for m in MULTI_M}
    seq_ids = torch.cat([synth_torch.gen_ids(64, N_VARIANTS, 3500, dev),
                         synth_torch.gen_ids(4, N_VARIANTS, 3501, dev).repeat_interleave(512)]).contiguous()
    axes_row = [ROW] * N_VARIANTS
    axes_mixed = [g % 2 for g in range(N_VARIANTS)]

    # config 1: 128 copies of a 1024 x 1024 layer (268 MB of weights + masks: more than the L2)
    c1 = []
    for c in range(C1_COPIES):
        w_b = synth_torch.gen_base(1024, 1024, 500 + c, dev)
        mask, v_row, _ = api.pd_pack_delta(synth_torch.gen_finetuned(w_b, 700 + c), w_b, want_col=False)
        c1.append((w_b, mask, v_row))
    c1_x = synth_torch.gen_x(16, 1024, 2999, dev)
    c1_y = torch.empty((16, 1024), dtype=torch.float16, device=dev)

    # config 5: one 70B-shaped layer's buffers, reused for all 80 layers
    big = []
    if not args.no_config5:
        for li, (name, d_out, d_in) in enumerate(BLOCK_70B):
            w_b = synth_torch.gen_base(d_out, d_in, 300 + li, dev)
            w_f = synth_torch.gen_finetuned(w_b, 400 + li)
            big.append(dict(name=name, d_out=d_out, d_in=d_in, w_b=w_b, w_f=w_f, w_hat=torch.empty_like(w_b),
                            mask=torch.empty((d_out, d_in // 32), dtype=torch.int32, device=dev),
                            v_row=torch.empty(d_out, dtype=torch.float16, device=dev),
                            v_col=torch.empty(d_in, dtype=torch.float16, device=dev)))
        big_x = synth_torch.gen_x(1, 28672, 2070, dev)
        big_y = torch.empty((1, 28672), dtype=torch.float16, device=dev)
    # BF16 variants: the same block with base, fine-tune and activations in bfloat16
    bf_layers = []
    for li, (name, d_out, d_in) in enumerate(BLOCK):
        w_b = synth_torch.gen_base(d_out, d_in, 10 + li, dev).bfloat16()
        w_f = synth_torch.gen_finetuned(w_b, 100 + li)
        mask, v_row, v_col = api.pd_pack_delta(w_f, w_b)
        bf_layers.append(dict(name=name, d_out=d_out, d_in=d_in, w_b=w_b, w_f=w_f, mask=mask, v=(v_row, v_col),
                              w_hat=torch.empty_like(w_b)))
    # scale fitting: teacher outputs of the fine-tuned layers for 2048 calibration tokens, fp32 scales and optimiser state
    fit = []
    for L in layers:
        xs = x_all[L["d_in"]][:FIT_M]
        st = {}
        for axis, v0 in ((ROW, L["v"][0]), (COL, L["v"][1])):
            v = v0.float().contiguous()
            st[axis] = dict(v=v, m1=torch.zeros_like(v), m2=torch.zeros_like(v), g=torch.zeros_like(v))
        fit.append(dict(L=L, y=(xs @ L["w_f"].T).contiguous(), mask_t=api.pd_transpose_mask(L["mask"], L["d_out"], L["d_in"]),
                        st=st, loss=torch.zeros(1, device=dev)))
    fit_opt = api.adamw(lr=1e-4)
    bf_x = {d_in: x_all[d_in][:2048].bfloat16() for d_in in x_all}
    bf_y = {d_out: torch.empty((2048, d_out), dtype=torch.bfloat16, device=dev) for d_out in y_all}
    torch.cuda.synchronize()

    # ---- sections: name -> (body, algorithmic work, unit, calls, kernel label)
    def run_pack():
        for L in layers:
            api.pd_pack_delta(L["w_f"], L["w_b"], mask=L["mask"], v_row=L["v"][0], v_col=L["v"][1])

    def run_linear(m, resident):
        for axis in (ROW, COL):
            for L in layers:
                api.pd_linear(x_all[L["d_in"]][:m], L["w_b"], L["mask"], L["v"][axis], axis, y=y_all[L["d_out"]][:m],
                              weights_resident=resident)

    PAR = 4  # parallel branches of the decode_par_* sections
    par_streams = [torch.cuda.Stream(device=dev) for _ in range(PAR)]
    par_y = [{d_out: torch.empty((16, d_out), dtype=torch.float16, device=dev) for d_out in (4096, 11008)} for _ in range(PAR)]

    def run_linear_par(m):
        # the same 14 calls as decode_m*, dealt to PAR streams: the linears of a sweep do not depend on one another (in a
        # decoder block q, k, v share an input, and so do gate and up), so their kernels may overlap on the GPU
        cur = torch.cuda.current_stream()
        for ps in par_streams:
            ps.wait_stream(cur)
        i = 0
        for axis in (ROW, COL):
            for L in layers:
                b = i % PAR
                i += 1
                with torch.cuda.stream(par_streams[b]):
                    api.pd_linear(x_all[L["d_in"]][:m], L["w_b"], L["mask"], L["v"][axis], axis, y=par_y[b][L["d_out"]][:m],
                                  weights_resident=True)
        for ps in par_streams:
            cur.wait_stream(ps)

    def on_branches(calls):
        """Deals the calls (callables taking the branch index) to the PAR streams and joins them."""
        cur = torch.cuda.current_stream()
        for ps in par_streams:
            ps.wait_stream(cur)
        for i, call in enumerate(calls):
            with torch.cuda.stream(par_streams[i % PAR]):
                call(i % PAR)
        for ps in par_streams:
            cur.wait_stream(ps)

    # pack and the split-K prefill use scratch memory: one workspace per branch (the pack's starts zeroed and is left zeroed)
    par_pack_ws = [torch.zeros(max(api.workspace_bytes(api.OP_PACK, 0, 0, L["d_out"], L["d_in"]) for L in layers), dtype=torch.uint8,
                               device=dev) for _ in range(PAR)]
    par_lin_ws = [torch.zeros(max(api.workspace_bytes(api.OP_LINEAR, 256, 0, L["d_out"], L["d_in"]) for L in layers), dtype=torch.uint8,
                              device=dev) for _ in range(PAR)]
    par_y256 = [{d_out: torch.empty((256, d_out), dtype=torch.float16, device=dev) for d_out in (4096, 11008)} for _ in range(PAR)]

    def run_pack_par():
        on_branches([lambda b, L=L: api.pd_pack_delta(L["w_f"], L["w_b"], mask=L["mask"], v_row=L["v"][0], v_col=L["v"][1],
                                                      workspace=par_pack_ws[b]) for L in layers])

    def run_merge_par():
        # both axes write the layer's one w_hat buffer: one axis per layer here, so that no two branches share an output
        on_branches([lambda b, L=L, axis=axis: api.pd_merge(L["w_b"], L["mask"], L["v"][axis], axis, w_hat=L["w_hat"])
                     for axis, L in zip([ROW, COL] * len(layers), layers)])

    def run_prefill256_par():
        on_branches([lambda b, L=L, axis=axis: api.pd_linear(x_all[L["d_in"]][:256], L["w_b"], L["mask"], L["v"][axis], axis,
                                                             y=par_y256[b][L["d_out"]], workspace=par_lin_ws[b])
                     for axis in (ROW, COL) for L in layers])

    def run_multi(m, id_t, key, axes):
        for L in layers:
            api.pd_linear_multivariant(x_all[L["d_in"]][:m], id_t, L["w_b"], L["masks"], L[key], axes, y=y_all[L["d_out"]][:m])

    def run_merge():
        for axis in (ROW, COL):
            for L in layers:
                api.pd_merge(L["w_b"], L["mask"], L["v"][axis], axis, w_hat=L["w_hat"])

    def bf_pack():
        for L in bf_layers:
            api.pd_pack_delta(L["w_f"], L["w_b"], mask=L["mask"], v_row=L["v"][0], v_col=L["v"][1])

    def bf_linear(ms, resident):
        for m in ms:
            for axis in (ROW, COL):
                for L in bf_layers:
                    api.pd_linear(bf_x[L["d_in"]][:m], L["w_b"], L["mask"], L["v"][axis], axis, y=bf_y[L["d_out"]][:m],
                                  weights_resident=resident)

    def bf_merge():
        for axis in (ROW, COL):
            for L in bf_layers:
                api.pd_merge(L["w_b"], L["mask"], L["v"][axis], axis, w_hat=L["w_hat"])

    def run_fit(axis):
        # one training step per layer: loss, gradient and AdamW update (step 1 of the bias correction every time, so
        # that replays do the same arithmetic; the updates still move v)
        for F in fit:
            L, st = F["L"], F["st"][axis]
            api.pd_fit_loss_grad(x_all[L["d_in"]][:FIT_M], F["y"], L["w_b"], L["mask"], st["v"], axis, mask_t=F["mask_t"],
                                 loss=F["loss"], grad=st["g"])
            api.pd_fit_adamw_step(st["v"], st["m1"], st["m2"], st["g"], 1, fit_opt)

    def run_c1(m, rotated):
        for c in range(C1_COPIES):
            w_b, mask, v_row = c1[c if rotated else 0]
            api.pd_linear(c1_x[:m], w_b, mask, v_row, ROW, y=c1_y[:m], weights_resident=True)

    def c5_pack():
        for L in big:
            api.pd_pack_delta(L["w_f"], L["w_b"], mask=L["mask"], v_row=L["v_row"], v_col=L["v_col"])

    def c5_merge():
        for L in big:
            api.pd_merge(L["w_b"], L["mask"], L["v_row"], ROW, w_hat=L["w_hat"])

    def c5_dense():
        for L in big:
            api.pd_linear(big_x[:, :L["d_in"]], L["w_hat"], None, None, ROW, y=big_y[:, :L["d_out"]])

    def c5_fused():
        for L in big:
            api.pd_linear(big_x[:, :L["d_in"]], L["w_b"], L["mask"], L["v_row"], ROW, y=big_y[:, :L["d_out"]])

    flops = lambda m: sum(2 * m * L["d_out"] * L["d_in"] for L in layers)
    S = {}  # name -> dict(body, work, unit, calls, kernel, reps)

    def add(name, body, work, unit, calls, kernel, reps=1, bound=None):
        S[name] = dict(body=body, work=work, unit=unit, calls=calls, kernel=kernel, reps=reps,
                       bound=bound or ("hbm" if unit == "GB/s" else "tensor"))

    add("pack", run_pack, sum(pack_bytes(L["d_out"], L["d_in"]) for L in layers), "GB/s", 7, "pack_kernel")
    for m in DECODE_M:
        add(f"decode_m{m}", lambda m=m: run_linear(m, True),
            sum(linear_bytes(m, L["d_out"], L["d_in"], ax) for ax in (ROW, COL) for L in layers), "GB/s", 14,
            "gemv_stream_kernel")
    for m in DECODE_M:
        add(f"decode_par_m{m}", lambda m=m: run_linear_par(m), S[f"decode_m{m}"]["work"], "GB/s", 14,
            "gemv_stream_kernel, four streams")
    add("pack_par", run_pack_par, S["pack"]["work"], "GB/s", 7, "pack_kernel, four streams")
    add("merge_par", run_merge_par, sum(merge_bytes(L["d_out"], L["d_in"], ax) for ax, L in zip([ROW, COL] * len(layers), layers)), "GB/s", 7,
        "merge_kernel, four streams")
    add("prefill_par_m256", run_prefill256_par, 2 * flops(256), "TFLOP/s", 14, "gemm_pair_kernel (split-K), four streams",
        bound="max(hbm, tensor)")
    for m in PREFILL_M:
        add(f"prefill_m{m}", lambda m=m: run_linear(m, False), 2 * flops(m), "TFLOP/s", 14, "gemm_pair_kernel (tcgen05, CTA pairs)",
            bound="tensor" if m > 256 else "max(hbm, tensor)")
    add("multi_decode", lambda: run_multi(MULTI_M[0], ids[MULTI_M[0]], "vs", axes_row),
        sum(multi_bytes(MULTI_M[0], L["d_out"], L["d_in"]) for L in layers), "GB/s", 7, "mv_decode_kernel (+ mv_prepare_kernel)")
    add("multi_prefill", lambda: run_multi(MULTI_M[1], ids[MULTI_M[1]], "vs", axes_row), flops(MULTI_M[1]), "TFLOP/s", 7,
        "gemm_pair_kernel<grouped> (+ group_rows, gather_rows)")
    add("multi_prefill_seq", lambda: run_multi(MULTI_M[1], seq_ids, "vs", axes_row), flops(MULTI_M[1]), "TFLOP/s", 7,
        "gemm_pair_kernel<grouped> (+ group_rows, gather_rows)")
    add("multi_decode_mixed", lambda: run_multi(MULTI_M[0], ids[MULTI_M[0]], "vs_mixed", axes_mixed),
        sum(multi_bytes(MULTI_M[0], L["d_out"], L["d_in"]) for L in layers), "GB/s", 7, "mv_decode_kernel<col axis present>")
    add("multi_prefill_mixed", lambda: run_multi(MULTI_M[1], ids[MULTI_M[1]], "vs_mixed", axes_mixed), flops(MULTI_M[1]),
        "TFLOP/s", 7, "gemm_pair_kernel<grouped>")
    add("merge", run_merge, sum(merge_bytes(L["d_out"], L["d_in"], ax) for ax in (ROW, COL) for L in layers), "GB/s", 14,
        "merge_kernel")
    add("bf16_pack", bf_pack, S["pack"]["work"], "GB/s", 7, "pack_kernel<bf16>")
    add("bf16_decode", lambda: bf_linear(DECODE_M, True), sum(S[f"decode_m{m}"]["work"] for m in DECODE_M), "GB/s", 42,
        "gemv_stream_kernel<bf16>")
    add("bf16_prefill_m2048", lambda: bf_linear((2048,), False), 2 * flops(2048), "TFLOP/s", 14, "gemm_pair_kernel<bf16>")
    add("bf16_merge", bf_merge, S["merge"]["work"], "GB/s", 14, "merge_kernel<bf16>")
    add("fit_row_m2048", lambda: run_fit(ROW), 2 * flops(FIT_M), "TFLOP/s", 7, "fit_gemm_kernel<row> (two tcgen05 accumulators)")
    add("fit_col_m2048", lambda: run_fit(COL), 3 * flops(FIT_M), "TFLOP/s", 7, "fit_gemm_kernel<col forward>, <col backward>")
    for m in (1, 16):
        for rotated in (True, False):
            add(f"c1_m{m}_{'rotated' if rotated else 'resident'}", lambda m=m, r=rotated: run_c1(m, r),
                C1_COPIES * linear_bytes(m, 1024, 1024, ROW), "GB/s", C1_COPIES, "gemv_stream_kernel",
                bound="hbm" if rotated else "l2-resident (latency)")
    if big:
        e70 = sum(L["d_out"] * L["d_in"] for L in big)
        add("c5_pack", c5_pack, sum(pack_bytes(L["d_out"], L["d_in"]) for L in big), "GB/s", 7, "pack_kernel", reps=N_LAYERS_70B)
        add("c5_merge", c5_merge, sum(merge_bytes(L["d_out"], L["d_in"], ROW) for L in big), "GB/s", 7, "merge_kernel", reps=N_LAYERS_70B)
        add("c5_gemv_dense", c5_dense, sum(linear_bytes(1, L["d_out"], L["d_in"], ROW, delta=False) for L in big), "GB/s", 7,
            "gemv_stream_kernel (mask = NULL)", reps=N_LAYERS_70B)
        add("c5_gemv_fused", c5_fused, sum(linear_bytes(1, L["d_out"], L["d_in"], ROW) for L in big), "GB/s", 7,
            "gemv_stream_kernel", reps=N_LAYERS_70B)
        assert e70 == 855638016
    sections = list(S)

    # Every section is captured once into a CUDA graph (the calls only enqueue kernels on the current
    # stream) and replayed: a decode kernel lasts ~10 us, less than the host needs to issue it.
    side = torch.cuda.Stream(device=dev)
    for name in sections:
        S[name]["body"]()  # eager once: sizes every cached workspace before capture
    torch.cuda.synchronize()
    for name in sections:
        g = torch.cuda.CUDAGraph()
        n0 = api.launch_count()
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                S[name]["body"]()
        S[name]["launches"] = (api.launch_count() - n0) * S[name]["reps"]
        S[name]["graph"] = g
    torch.cuda.synchronize()

    c5_names = [n for n in sections if n.startswith("c5_")]
    plain = [n for n in sections if not n.startswith("c5_")]

    def timed(ev, name, fn):
        if ev is None:
            fn()
            return
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        ev[name].append((e0, e1))

    def step_block(ev=None):
        """The 7B-block, BF16 and 1024x1024 sections of one step.  ev: dict name -> list of (start, end) events."""
        for name in plain:
            timed(ev, name, S[name]["graph"].replay)

    def step_model(ev=None):
        """The 70B-shaped part of one step, layer by layer: pack -> merge -> dense GEMV, fused GEMV."""
        for _ in range(N_LAYERS_70B if c5_names else 0):
            for name in c5_names:
                timed(ev, name, S[name]["graph"].replay)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(args.warmup):
        step_block()
    for _ in range(args.warmup):
        step_model()
    barrier()
    if api.pd_device_status() != 0:
        raise RuntimeError("device status latched an error during warm-up")

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    evs = [{n: [] for n in sections} for _ in range(args.steps)]
    t_first, t_last = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t_first.record()
    # The K steps run as K block parts followed by K model parts: the 80-layer part keeps HBM saturated for
    # ~0.15 s per step and would otherwise set the power state the short decode kernels are measured in.
    for k in range(args.steps):
        step_block(evs[k])
    for k in range(args.steps):
        step_model(evs[k])
    t_last.record()
    barrier()
    launches = args.steps * sum(S[n]["launches"] for n in sections)  # kernels inside the replayed graphs
    clocks = sampler.stop() if rank == 0 else None
    if api.pd_device_status() != 0:
        raise RuntimeError("device status latched an error during the timed region")

    sec_ms = {n: sum(a.elapsed_time(b) for k in range(args.steps) for a, b in evs[k][n]) / args.steps for n in sections}
    total_ms = t_first.elapsed_time(t_last) / args.steps

    # ---- end to end for the headline metric: host x -> device, pd_linear, y -> host, every call
    host_x = {d_in: x_all[d_in][:16].cpu().pin_memory() for d_in in x_all}
    host_y = {d_out: torch.empty((16, d_out), dtype=torch.float16).pin_memory() for d_out in y_all}
    dx = {d_in: torch.empty((16, d_in), dtype=torch.float16, device=dev) for d_in in x_all}

    def e2e_step():
        for m in DECODE_M:
            for axis in (ROW, COL):
                for L in layers:
                    api.pd_linear_host(host_x[L["d_in"]][:m], dx[L["d_in"]], L["w_b"], L["mask"], L["v"][axis], axis,
                                       y_all[L["d_out"]], host_y[L["d_out"]][:m], weights_resident=True)
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
    e2e_eager_ms = e0.elapsed_time(e1) / args.steps  # one host call per linear: the host's ~35 us per call is what this measures
    # the same calls captured once into a CUDA graph (copy nodes from and to pinned host memory around every kernel) and
    # replayed: what a serving loop does with a fixed decode step
    # -- the calls of a step are independent, so the graph has E2E_BRANCHES parallel branches with their own staging and
    # output buffers: one call's copies overlap the other branches' kernels (a copy over PCIe costs ~10 us whatever its size)
    E2E_BRANCHES = 4
    br_streams = [torch.cuda.Stream(device=dev) for _ in range(E2E_BRANCHES)]
    br_dx = [{d_in: torch.empty((16, d_in), dtype=torch.float16, device=dev) for d_in in x_all} for _ in range(E2E_BRANCHES)]
    br_y = [{d_out: torch.empty((16, d_out), dtype=torch.float16, device=dev) for d_out in y_all} for _ in range(E2E_BRANCHES)]
    br_host_y = [{d_out: torch.empty((16, d_out), dtype=torch.float16).pin_memory() for d_out in y_all} for _ in range(E2E_BRANCHES)]

    def e2e_step_branches():
        cur = torch.cuda.current_stream()
        for bs in br_streams:
            bs.wait_stream(cur)
        i = 0
        for m in DECODE_M:
            for axis in (ROW, COL):
                for L in layers:
                    b = i % E2E_BRANCHES
                    i += 1
                    with torch.cuda.stream(br_streams[b]):
                        api.pd_linear_host(host_x[L["d_in"]][:m], br_dx[b][L["d_in"]], L["w_b"], L["mask"], L["v"][axis], axis,
                                           br_y[b][L["d_out"]], br_host_y[b][L["d_out"]][:m], weights_resident=True)
        for bs in br_streams:
            cur.wait_stream(bs)

    with torch.cuda.stream(side):
        e2e_step_branches()  # eager once
    torch.cuda.synchronize()
    e2e_graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(e2e_graph, stream=side):
            e2e_step_branches()
    for _ in range(3):
        e2e_graph.replay()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        e2e_graph.replay()
    e1.record()
    barrier()
    e2e_ms = e0.elapsed_time(e1) / args.steps
    # the last replay's outputs reached the host buffers and equal the one-by-one run's (same inputs, same kernels)
    last = len(DECODE_M) * 2 * len(layers) - 1
    assert torch.equal(br_host_y[last % E2E_BRANCHES][layers[-1]["d_out"]][:DECODE_M[-1]], host_y[layers[-1]["d_out"]][:DECODE_M[-1]])

    # ---- cold start (pd_load_merged): the delta artifacts of N_LOAD_LAYERS blocks in pinned host memory are copied
    # module by module while the previous module is merged into the resident base; beside it, the same bytes of
    # dense fp16 weights copied from pinned host memory (what loading a full fine-tuned checkpoint moves)
    N_LOAD_LAYERS = 2
    load_mods = []
    for _ in range(N_LOAD_LAYERS):
        for L in layers:
            load_mods.append((L["w_b"], L["w_hat"], api.make_artifact(L["mask"], L["v"][ROW]), ROW))
    art_bytes = sum(api.artifact_bytes(L["d_out"], L["d_in"], ROW) for L in layers) * N_LOAD_LAYERS
    staging = torch.zeros(2 * ((max(api.artifact_bytes(L["d_out"], L["d_in"], ROW) for L in layers) + 255) // 256 * 256),
                          dtype=torch.uint8, device=dev)
    copy_stream = torch.cuda.Stream(device=dev)
    dense_host = [torch.empty(L["w_b"].shape, dtype=torch.float16).pin_memory() for L in layers]
    dense_bytes = sum(t.numel() * 2 for t in dense_host) * N_LOAD_LAYERS

    def load_delta():
        api.pd_load_merged(load_mods, staging, copy_stream)

    def load_dense():
        for _ in range(N_LOAD_LAYERS):
            for L, h in zip(layers, dense_host):
                L["w_hat"].copy_(h, non_blocking=True)

    load_ms = {}
    for name, fn in (("delta_on_resident_base", load_delta), ("dense_checkpoint", load_dense)):
        fn()
        barrier()
        l0, l1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        l0.record()
        for _ in range(3):
            fn()
        l1.record()
        barrier()
        load_ms[name] = l0.elapsed_time(l1) / 3

    # ---- max over ranks
    stats = max_over_ranks([total_ms, e2e_ms] + [sec_ms[s] for s in sections], world, dev)
    total_ms, e2e_ms = stats[0], stats[1]
    sec_ms = dict(zip(sections, stats[2:]))

    if rank == 0:
        pk = peaks()
        step_ms = sum(sec_ms.values())

        def roof(name):
            s = S[name]
            per_gpu = s["work"] * s["reps"] / (sec_ms[name] * 1e-3) / (1e9 if s["unit"] == "GB/s" else 1e12)
            calls = s["calls"] * s["reps"]
            r = {"kernel": s["kernel"], "bound": s["bound"], "achieved": round(per_gpu, 1), "unit": s["unit"],
                 "avg_call_ms": round(sec_ms[name] / calls, 5), "share_of_step": round(sec_ms[name] / step_ms, 4)}
            if s["unit"] == "GB/s":
                base = name.split("_m")[0] if name.startswith("decode") else name.replace("c5_", "")
                ratio = NCU_DRAM_RATIO.get(base)
                r.update({"peak": pk["hbm_gbs"], "frac": round(per_gpu / pk["hbm_gbs"], 4), "frac_of": pk["source"],
                          "frac_of_nominal_8TBs": round(per_gpu / 8000.0, 4),
                          "algorithmic_bytes_per_call": s["work"] // s["calls"],
                          # DRAM bytes per call = algorithmic bytes x the ncu ratio of the captured case under profiles/
                          "traffic": round(s["work"] / s["calls"] * ratio) if ratio else None})
            else:
                # a tensor-bound section stands against the burst peak when it is short (timed alone for a few ms),
                # the sustained peak is printed beside it; fp16 and bf16 share one tensor peak
                r.update({"peak": pk["tflops_burst"], "frac": round(per_gpu / pk["tflops_burst"], 4),
                          "frac_of": pk["source"] + " burst (fp16 and bf16 share one tensor peak)",
                          "frac_of_sustained": round(per_gpu / pk["tflops_sustained"], 4),
                          "frac_of_nominal_2250": round(per_gpu / 2250.0, 4), "traffic": None,
                          "algorithmic_flops_per_call": s["work"] // s["calls"]})
                if name == "prefill_m256":  # co-limited by HBM: the bound is the slower of the two rooflines
                    t_hbm = sum(linear_bytes(256, L["d_out"], L["d_in"], ax) for ax in (ROW, COL) for L in layers) / (pk["hbm_gbs"] * 1e9)
                    t_mma = s["work"] / (pk["tflops_burst"] * 1e12)
                    r["frac_of_max_hbm_tensor"] = round(max(t_hbm, t_mma) / (sec_ms[name] * 1e-3), 4)
            return r

        all_roofs = {n: roof(n) for n in sections}
        dec_names = [f"decode_m{m}" for m in DECODE_M]
        dec_ms = sum(sec_ms[n] for n in dec_names)
        dec_work = sum(S[n]["work"] for n in dec_names)
        dec_gbs = dec_work * world / (dec_ms * 1e-3) / 1e9
        all_roofs["decode"] = {"kernel": "gemv_stream_kernel", "bound": "hbm", "achieved": round(dec_gbs / world, 1),
                               "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": round(dec_gbs / world / pk["hbm_gbs"], 4),
                               "frac_of": pk["source"], "frac_of_nominal_8TBs": round(dec_gbs / world / 8000.0, 4),
                               "algorithmic_bytes_per_call": dec_work // 42, "avg_call_ms": round(dec_ms / 42, 5),
                               "traffic": round(dec_work / 42 * NCU_DRAM_RATIO["decode"]) if NCU_DRAM_RATIO["decode"] else None,
                               "share_of_step": round(dec_ms / step_ms, 4), "what": "decode_m1 + decode_m4 + decode_m16"}
        pre_names = [f"prefill_m{m}" for m in PREFILL_M]
        pre_tf = sum(S[n]["work"] for n in pre_names) / (sum(sec_ms[n] for n in pre_names) * 1e-3) / 1e12
        dominant = max(sections, key=lambda n: sec_ms[n])  # the section the step spends most time in

        # per-shape table of the 7B kernels (separate short runs, CUDA events inside graphs over rotated copies)
        cpu = oracle_sample(2, 1) if (world == 1 and not args.no_cpu_baseline) else None
        cpu_other = oracle_other_ops() if (world == 1 and not args.no_cpu_baseline) else None
        line = {
            "metric": METRIC, "value": round(dec_gbs, 1), "unit": "GB/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": round(total_ms, 4), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f16", "data": "synthetic",
            "config": {"workload": "llama7b_block: pack + decode M{1,4,16} + prefill M{256,2048,8192} + "
                                   "multivariant V16 M{64,2112} + merge, row and col axes",
                       "also_in_step": "config 1 (1024x1024 layer, 128 rotated copies and L2-resident), multivariant per-sequence ids and "
                                       "mixed axes, config 5 (70B block x 80 layers: pack -> merge -> dense and fused GEMV at M=1)"
                                       if big else "config 1, multivariant per-sequence ids and mixed axes (config 5 skipped)",
                       "order": "the timed region runs the block sections of all K steps, then the 70B-shaped sections of all K steps",
                       "l2": "every sweep streams >= 268 MB of weights, larger than the 126 MB L2, except the sections named *_resident",
                       "replicas": "independent per GPU, no collective"},
            "sections": {
                "pack_GBps": all_roofs["pack"]["achieved"], "decode_GBps": round(dec_gbs, 1),
                "prefill_TFLOPps": round(pre_tf, 1), "multivariant_decode_GBps": all_roofs["multi_decode"]["achieved"],
                "multivariant_prefill_TFLOPps": all_roofs["multi_prefill"]["achieved"],
                "merge_GBps": all_roofs["merge"]["achieved"], "ms": {s: round(sec_ms[s], 4) for s in sections}},
            "roofline": dict(all_roofs[dominant], section=dominant),
            "rooflines": all_roofs,
            "e2e": {"value": round(dec_work * world / (e2e_ms * 1e-3) / 1e9, 1), "unit": "GB/s",
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": round(e2e_ms, 4),
                    "eager_value": round(dec_work * world / (e2e_eager_ms * 1e-3) / 1e9, 1), "eager_ms_per_step": round(e2e_eager_ms, 4),
                    "what": "decode sections through pd_linear_host: x from pinned host memory, y back to pinned host memory, every "
                            "call; `value` replays the step's calls from a CUDA graph of four parallel branches (copies included; the calls "
                            "are independent), `eager_value` issues them one by one on one stream"},
            "cold_start": {"what": f"{N_LOAD_LAYERS} 7B blocks ({len(load_mods)} modules): pd_load_merged from pinned host artifacts "
                                   "(H2D of module i+1 overlaps the merge of module i) against an H2D copy of the dense fp16 weights",
                           "delta_ms": round(load_ms["delta_on_resident_base"], 3), "delta_artifact_bytes": art_bytes,
                           "delta_artifact_GBps": round(art_bytes / load_ms["delta_on_resident_base"] / 1e6, 1),
                           "dense_ms": round(load_ms["dense_checkpoint"], 3), "dense_bytes": dense_bytes,
                           "speedup": round(load_ms["dense_checkpoint"] / load_ms["delta_on_resident_base"], 2)},
            "gpu_launches": launches, "clocks": clocks,
        }
        if cpu is not None:
            line["cpu_baseline"] = {k: (round(cpu[k], 3) if k == "value" else cpu[k])
                                    for k in ("value", "unit", "cores", "kind", "sample")}
            line["cpu_baseline"]["other_ops"] = cpu_other
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
    per_copy = (4 if args.only == "multi" else 2) * d_out * d_in
    copies = max(2, int(300e6 // per_copy) + 1)
    layers = []
    for c in range(copies):
        w_b = synth_torch.gen_base(d_out, d_in, 10 + c, dev)
        w_f = synth_torch.gen_finetuned(w_b, 100 + c)
        mask, v_row, v_col = api.pd_pack_delta(w_f, w_b)
        L = [w_b, w_f, mask, (v_row, v_col), torch.empty_like(w_b)]
        if args.only == "multi":
            masks = torch.empty((N_VARIANTS, d_out, d_in // 32), dtype=torch.int32, device=dev)
            vs = torch.zeros((N_VARIANTS, max(d_out, d_in)), dtype=torch.float16, device=dev)
            for g in range(N_VARIANTS):
                _, vr, vc = api.pd_pack_delta(synth_torch.gen_finetuned(w_b, 1000 + 16 * c + g), w_b, mask=masks[g])
                if axis == ROW:
                    vs[g, :d_out] = vr
                else:
                    vs[g, :d_in] = vc
            L += [masks, vs]
        layers.append(L)
    x = synth_torch.gen_x(args.m, d_in, 5, dev)
    y = torch.empty((args.m, d_out), dtype=torch.float16, device=dev)
    ids = synth_torch.gen_ids(args.m, N_VARIANTS, 3000 + args.m, dev)
    if args.only == "fit":
        y_fit = [(x @ L[1].T).contiguous() for L in layers]
        mask_t = [api.pd_transpose_mask(L[2], d_out, d_in) for L in layers]
        v32 = [L[3][axis].float().contiguous() for L in layers]
        fit_loss, fit_grad = torch.zeros(1, device=dev), torch.zeros_like(v32[0])

    def call(i):
        L = layers[i % copies]
        w_b, w_f, mask, v, out = L[:5]
        if args.only == "fit":
            c = i % copies
            api.pd_fit_loss_grad(x, y_fit[c], w_b, mask, v32[c], axis, mask_t=mask_t[c], loss=fit_loss, grad=fit_grad)
        elif args.only == "linear":
            api.pd_linear(x, w_b, mask, v[axis], axis, y=y, weights_resident=True)
        elif args.only == "pack":
            api.pd_pack_delta(w_f, w_b, mask=mask, v_row=v[0], v_col=v[1])
        elif args.only == "multi":
            api.pd_linear_multivariant(x, ids, w_b, L[5], L[6], [axis] * N_VARIANTS, y=y)
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
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-config5", action="store_true", help="leave the 70B-shaped sections out (they need ~6 GB and ~0.2 s per step)")
    ap.add_argument("--only", choices=["linear", "pack", "merge", "multi", "fit"], help="run one kernel family on one layer (for profiling)")
    ap.add_argument("--shape", default="4096x4096")
    ap.add_argument("--m", type=int, default=16)
    ap.add_argument("--axis", default="row", choices=["row", "col"])
    ap.add_argument("--calls", type=int, default=4)
    args = ap.parse_args()
    if args.only:
        run_only(args)
    elif args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_replicas(args.gpus, sys.argv[1:]))
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
