#!/usr/bin/env python
"""Benchmark of the nested int8 -> int4 -> int2 weight path on one node.

A step is one pass of the whole path over the Gemma-2-2B-shaped MLP stack
(26 layers x {gate, up: 9216x2304, down: 2304x9216}, bf16 weights N(0, 0.02)):

  quantize (Eq. 1)                      bf16 W -> uint8 codes, alpha, z
  slice_pack r=4 (Eq. 6)                codes -> packed int4 plane
  slice_pack r=2 + extra precision      codes -> packed int2 plane + Eq. 8 overflow lists
  decode GEMV  r=4  B=1, B=8            packed plane, bf16 x -> fp32 y
  decode GEMV  r=2  B=1, B=8
  decode GEMV  r=2  extra precision, B=1

The dense multi-precision forward (Eq. 7) has no place in a decode-shaped workload (1 or 8 activations per layer);
it is measured on its own configuration, the Mistral-7B-shaped co-training forward (W 14336x4096, 4096 tokens,
r = 8, 4, 2 in one call), and reported in the same JSON line under `gemm_multi_cfg4` with its tensor roofline.

Every matrix of the stack has its own buffers, so each stage streams far more
than the L2 holds.  `value` is the algorithmic HBM bytes of the step divided by
the device time of the step (inputs resident in HBM); `e2e` runs the same step
from host buffers with the copies inside the timed region.  `stages` gives the
per-stage figures (GB/s against the measured copy bandwidth, TFLOP/s for the
dense forward); `roofline` describes the stage that takes the largest share.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--layers L]
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time
from concurrent.futures import ThreadPoolExecutor

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2502_06786_b200 import synth  # noqa: E402

METRIC = "sliced int{8,4,2} GEMV HBM GB/s (% of peak); multi-precision GEMM TFLOP/s"
# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) per launch from the ncu captures summarised under
# profiles/, for kernels that have not changed since; a stage that is missing here reports traffic = null.
NCU_TRAFFIC = {"quantize": 42780000}
NCU_TRAFFIC_NOTE = {"quantize": "ncu, one 9216x2304 launch: 42.50 MB read (= the algorithmic 42.47 MB) + 0.29 MB written; "
                                "the 21.2 MB of codes were still in the L2 when the launch ended, so the write-back "
                                "shows up in later launches"}
CONFIG_ID = 2
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1590.0


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_tflops=float(d["bf16_tflops"]),
                    bf16_tflops_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=FALLBACK_HBM_GBS, bf16_tflops=FALLBACK_BF16_TFLOPS, bf16_tflops_sustained=1400.0,
                source="fallback")


# ----------------------------------------------------------------------------
# algorithmic bytes per call (what the kernels must move at minimum)
# ----------------------------------------------------------------------------

def bytes_quantize(N, K):
    return 3 * N * K + 8 * N


def bytes_slice_pack(N, K, r, nnz=None):
    b = N * K + N * K * r // 8
    if nnz is not None:
        b += 4 * (N + 1) + 2 * nnz + 8
    return b


def bytes_gemv(N, K, r, B, nnz=None):
    b = N * K * r // 8 + 8 * N + 2 * B * K + 4 * B * N
    if nnz is not None:
        b += 4 * (N + 1) + 2 * nnz
    return b


def host_stack(rank: int, layers: int):
    """Seeded host tensors of the stack: weights (bf16 bits) and activations for B = 8 (B = 1 is row 0)."""
    shapes = synth.stack_shapes(CONFIG_ID, layers)
    workers = max(1, min(16, len(os.sched_getaffinity(0))))

    def make(item):
        idx, layer, name, N, K = item
        W = synth.normal_bf16((N, K), 0.02, synth.seed_for(CONFIG_ID, idx) + 100000 * rank)
        x = synth.normal_bf16((8, K), 1.0, synth.seed_for(CONFIG_ID, 500 + idx) + 100000 * rank)
        return W, x

    with ThreadPoolExecutor(workers) as ex:
        data = list(ex.map(make, shapes))
    return shapes, [d[0] for d in data], [d[1] for d in data]


# ----------------------------------------------------------------------------
# clocks
# ----------------------------------------------------------------------------

class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if not self.proc:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=[], samples=0)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for l in self.lines:
            f = [t.strip() for t in l.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for nm, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return dict(sm_mhz=float(np.median(sm)) if sm else None, sm_max_mhz=float(max(mx)) if mx else None,
                    reasons=sorted(reasons), samples=len(sm))


# ----------------------------------------------------------------------------
# the CUDA arm
# ----------------------------------------------------------------------------

class DeviceStack:
    """Device buffers of one stack and the stage-major call plan of a step."""

    def __init__(self, shapes, W_host, x_host, mq, torch):
        self.mq, self.torch = mq, torch
        self.shapes = shapes
        dev = "cuda"
        u8, f32 = torch.uint8, torch.float32
        self.W = [torch.empty((N, K), dtype=torch.bfloat16, device=dev) for (_, _, _, N, K) in shapes]
        self.x8 = [torch.empty((8, K), dtype=torch.bfloat16, device=dev) for (_, _, _, N, K) in shapes]
        self.q = [torch.empty((N, K), dtype=u8, device=dev) for (_, _, _, N, K) in shapes]
        self.alpha = [torch.empty(N, dtype=f32, device=dev) for (_, _, _, N, K) in shapes]
        self.zero = [torch.empty(N, dtype=f32, device=dev) for (_, _, _, N, K) in shapes]
        self.p4 = [torch.empty((N, K // 2), dtype=u8, device=dev) for (_, _, _, N, K) in shapes]
        self.p2 = [torch.empty((N, K // 4), dtype=u8, device=dev) for (_, _, _, N, K) in shapes]
        self.cap = [max(1024, N * K // 16) for (_, _, _, N, K) in shapes]
        self.rp = [torch.empty(N + 1, dtype=torch.int32, device=dev) for (_, _, _, N, K) in shapes]
        self.col = [torch.empty(c, dtype=torch.uint16, device=dev) for c in self.cap]
        self.cnt = [torch.zeros(1, dtype=torch.int64, device=dev) for _ in shapes]
        self.y = {nm: [torch.empty((B, N), dtype=f32, device=dev) for (_, _, _, N, K) in shapes]
                  for nm, B in (("g4b1", 1), ("g4b8", 8), ("g2b1", 1), ("g2b8", 8), ("g2ep", 1))}
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.has_gemm = self._probe_gemm()
        self.W_pinned = self.x_pinned = None
        self.upload(W_host, x_host)

    def _probe_gemm(self):
        mq, torch = self.mq, self.torch
        try:
            q = torch.zeros((128, 128), dtype=torch.uint8, device="cuda")
            X = torch.zeros((128, 128), dtype=torch.bfloat16, device="cuda")
            a = torch.ones(128, dtype=torch.float32, device="cuda")
            mq.gemm_multi(mq.SRC_CODES8, q, 128, X, alpha=a, zero=a)
            torch.cuda.synchronize()
            return True
        except mq.MatqError as e:
            if e.status == mq.ERR_UNSUPPORTED:
                return False
            raise

    def upload(self, W_host, x_host):
        torch = self.torch
        for i, (W, x) in enumerate(zip(W_host, x_host)):
            self.W[i].view(torch.uint16).copy_(torch.from_numpy(W))
            self.x8[i].view(torch.uint16).copy_(torch.from_numpy(x))
        torch.cuda.synchronize()

    # stage-major plan: name -> (callable over the whole stack, kernels launched, algorithmic bytes, flops)
    def stages(self):
        mq = self.mq
        S = self.shapes
        n = len(S)

        def quant():
            for i in range(n):
                mq.quantize(self.W[i], q=self.q[i], alpha=self.alpha[i], zero=self.zero[i], dev_status=self.status)

        def sp4():
            for i in range(n):
                mq.slice_pack(self.q[i], 4, packed=self.p4[i])

        def sp2():
            for i in range(n):
                mq.slice_pack(self.q[i], 2, extra_precision=True, packed=self.p2[i], ovf_row_ptr=self.rp[i],
                              ovf_col=self.col[i], ovf_capacity=self.cap[i], ovf_count=self.cnt[i], dev_status=self.status)

        def gemv(nm, r, B, ep=False):
            planes = self.p4 if r == 4 else self.p2

            def run():
                for i in range(n):
                    K = S[i][4]
                    mq.gemv(planes[i], K, r, self.alpha[i], self.zero[i], self.x8[i][:B], y=self.y[nm][i],
                            ovf_row_ptr=self.rp[i] if ep else None, ovf_col=self.col[i] if ep else None,
                            flags=mq.GEMV_AUTO | mq.GEMV_PDL)
            return run

        nnz = getattr(self, "nnz", [0] * n)
        plan = [
            ("quantize", quant, n, sum(bytes_quantize(N, K) for (_, _, _, N, K) in S), 0),
            ("slice_pack_r4", sp4, n, sum(bytes_slice_pack(N, K, 4) for (_, _, _, N, K) in S), 0),
            ("slice_pack_r2_ep", sp2, 3 * n, sum(bytes_slice_pack(N, K, 2, z) for (_, _, _, N, K), z in zip(S, nnz)), 0),
            ("gemv_r4_b1", gemv("g4b1", 4, 1), n, sum(bytes_gemv(N, K, 4, 1) for (_, _, _, N, K) in S), 0),
            ("gemv_r4_b8", gemv("g4b8", 4, 8), n, sum(bytes_gemv(N, K, 4, 8) for (_, _, _, N, K) in S), 0),
            ("gemv_r2_b1", gemv("g2b1", 2, 1), n, sum(bytes_gemv(N, K, 2, 1) for (_, _, _, N, K) in S), 0),
            ("gemv_r2_b8", gemv("g2b8", 2, 8), n, sum(bytes_gemv(N, K, 2, 8) for (_, _, _, N, K) in S), 0),
            ("gemv_r2_ep_b1", gemv("g2ep", 2, 1, True), n,
             sum(bytes_gemv(N, K, 2, 1, z) for (_, _, _, N, K), z in zip(S, nnz)), 0),
        ]
        return plan


def run_cuda(args, rank, world, local_rank):
    import torch
    import torch.distributed as dist

    from paper_2502_06786_b200 import binding as mq

    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    peaks = measured_peaks()
    shapes, W_host, x_host = host_stack(rank, args.layers)
    st = DeviceStack(shapes, W_host, x_host, mq, torch)

    # one eager pass: warms the kernels up and gives the overflow counts the byte model needs
    for _, fn, _, _, _ in st.stages():
        fn()
    torch.cuda.synchronize()
    assert int(st.status.item()) == 0, f"device status {int(st.status.item())}"
    st.nnz = [int(c.item()) for c in st.cnt]
    plan = st.stages()

    # one CUDA graph per stage: launch overhead of ~800 small kernels would otherwise dominate
    graphs = []
    side = torch.cuda.Stream()
    for name, fn, launches, nbytes, flops in plan:
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            fn()
            torch.cuda.synchronize()
            with torch.cuda.graph(g, stream=side):
                fn()
        graphs.append(g)
    torch.cuda.synchronize()

    def step(events=None):
        for j, g in enumerate(graphs):
            if events is not None:
                events[j].record()
            g.replay()
        if events is not None:
            events[len(graphs)].record()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.3)
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(len(graphs) + 1)] for _ in range(args.steps)]
    barrier()
    for k in range(args.steps):
        step(ev[k])
    barrier()
    clocks = sampler.stop()
    total_ms = ev[0][0].elapsed_time(ev[-1][-1])
    stage_ms = [sum(ev[k][j].elapsed_time(ev[k][j + 1]) for k in range(args.steps)) / args.steps
                for j in range(len(graphs))]
    ms_per_step = total_ms / args.steps
    if world > 1:
        t = torch.tensor([ms_per_step], device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms_per_step = float(t.item())
    step_bytes = sum(p[3] for p in plan)
    value = world * step_bytes / (ms_per_step * 1e-3) / 1e9

    stages = {}
    for (name, fn, launches, nbytes, flops), ms in zip(plan, stage_ms):
        d = dict(ms=round(ms, 4), share=round(ms / sum(stage_ms), 4), GBps=round(nbytes / (ms * 1e-3) / 1e9, 1),
                 frac_hbm=round(nbytes / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"], 4), bytes=nbytes)
        if flops:
            d["TFLOPs"] = round(flops / (ms * 1e-3) / 1e12, 2)
            d["frac_tensor"] = round(flops / (ms * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"], 4)
        stages[name] = d

    # roofline of the stage with the largest share of the step
    dom = max(range(len(plan)), key=lambda j: stage_ms[j])
    name, _, launches, nbytes, flops = plan[dom]
    if flops and name.startswith("gemm"):
        ach = flops / (stage_ms[dom] * 1e-3) / 1e12
        roofline = dict(kernel=name, bound="tensor", achieved=round(ach, 2), peak=peaks["bf16_tflops_sustained"],
                        unit="TFLOP/s", frac=round(ach / peaks["bf16_tflops_sustained"], 4), traffic=None,
                        peak_source=peaks["source"] + " (sustained)")
    else:
        ach = nbytes / (stage_ms[dom] * 1e-3) / 1e9
        roofline = dict(kernel=name, bound="hbm", achieved=round(ach, 1), peak=peaks["hbm_gbs"], unit="GB/s",
                        frac=round(ach / peaks["hbm_gbs"], 4), traffic=NCU_TRAFFIC.get(name), peak_source=peaks["source"],
                        avg_launch_us=round(stage_ms[dom] * 1e3 / len(shapes), 3),
                        bytes_per_launch=nbytes // len(shapes))
        if name in NCU_TRAFFIC_NOTE:
            roofline["traffic_note"] = NCU_TRAFFIC_NOTE[name]

    gpu_launches = sum((p[2] if p[2] is not None else 2 * len(shapes)) for p in plan)

    # ------------------------------------------------------------------ end to end from host buffers
    e2e = e2e_leg(st, plan, W_host, x_host, args, torch, world, dist if world > 1 else None)

    cfg4 = None
    extras = {}
    if st.has_gemm and world == 1 and not args.no_cfg4:
        for t in (st.W, st.q, st.p4, st.p2):       # free the stack's large buffers first
            t.clear()
        torch.cuda.empty_cache()
        cfg4 = gemm_cfg4(mq, torch, peaks)
        torch.cuda.empty_cache()
        extras = {"gemv_cfg3": gemv_cfg3(mq, torch, peaks), "gemm_multi_cfg5_prefill": gemm_cfg5_prefill(mq, torch, peaks)}
        torch.cuda.empty_cache()
        extras["quantize_clip_cfg5"] = quantize_clip_cfg5(mq, torch, peaks)
        torch.cuda.empty_cache()
        extras["gemv_cfg2_mixnmatch"] = gemv_cfg2_mixnmatch(mq, torch, peaks)

    out = None
    if rank == 0:
        out = {
            "metric": METRIC, "value": round(value, 1), "unit": "GB/s", "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": round(ms_per_step, 4), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "u8 codes / fp32 accumulate", "data": "synthetic",
            "config": {"workload": f"configs[1] Gemma-2-2B-shaped MLP decode stack, {args.layers} layers x (gate,up 9216x2304; down 2304x9216), "
                                   "bf16 N(0,0.02) weights, x bf16 N(0,1)",
                       "step": "quantize -> slice_pack r=4 -> slice_pack r=2 + extra-precision lists -> gemv r=4 B=1,8 -> gemv r=2 B=1,8 -> gemv r=2 E.P. B=1"
                               + "; dense multi-precision forward measured separately (gemm_multi_cfg4)",
                       "value_definition": "algorithmic HBM bytes of the step / device time; one CUDA graph per stage",
                       "l2": "inputs larger than L2: every matrix has its own buffers, each stage streams >= 0.4 GB",
                       "parallelism": "one independent stack per GPU (rows are independent; no collective)" if world > 1 else "single GPU",
                       "overflow_fraction_r2": round(sum(st.nnz) / sum(N * K for (_, _, _, N, K) in shapes), 6)},
            "clocks": clocks, "e2e": e2e, "gpu_launches": gpu_launches, "stages": stages, "roofline": roofline,
        }
        if cfg4 is not None:
            out["gemm_multi_cfg4"] = cfg4
        out.update(extras)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    return out, st


def gemm_cfg4(mq, torch, peaks, reps=5):
    """configs[3]: Mistral-7B-shaped co-training forward, one fused call: quantize + slice r = 8, 4, 2 + three GEMMs."""
    N, K, M = 14336, 4096, 4096
    W = torch.from_numpy(synth.normal_bf16((N, K), 0.02, synth.seed_for(4, 0))).cuda().view(torch.bfloat16)
    X = torch.from_numpy(synth.normal_bf16((M, K), 1.0, synth.seed_for(4, 500))).cuda().view(torch.bfloat16)
    Ys = [torch.empty((M, N), dtype=torch.float32, device="cuda") for _ in range(3)]
    a = torch.empty(N, dtype=torch.float32, device="cuda"); z = torch.empty_like(a)
    ws = torch.empty(mq.gemm_multi_workspace_bytes(mq.SRC_BF16, M, N, K, 3), dtype=torch.uint8, device="cuda")
    for _ in range(2):
        mq.gemm_multi(mq.SRC_BF16, W, K, X, alpha=a, zero=z, Ys=Ys, workspace=ws)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        mq.gemm_multi(mq.SRC_BF16, W, K, X, alpha=a, zero=z, Ys=Ys, workspace=ws)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / reps
    flops = 3 * 2.0 * M * N * K
    tf = flops / (ms * 1e-3) / 1e12
    # the same pass as Eq. 7's objective: the three outputs are compared with a target in the epilogue and never stored
    Yt = Ys[0]                                      # any fp32 [M, N] serves as the target for timing
    del Ys[1:]
    wl = torch.empty(mq.gemm_multi_loss_workspace_bytes(mq.SRC_BF16, M, N, K, 3), dtype=torch.uint8, device="cuda")
    loss = torch.empty(4, dtype=torch.float64, device="cuda")
    for _ in range(2):
        mq.gemm_multi_loss(mq.SRC_BF16, W, K, X, Yt, (1.0, 1.0, 1.0), alpha=a, zero=z, loss=loss, workspace=wl)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(reps):
        mq.gemm_multi_loss(mq.SRC_BF16, W, K, X, Yt, (1.0, 1.0, 1.0), alpha=a, zero=z, loss=loss, workspace=wl)
    e1.record()
    torch.cuda.synchronize()
    ms_loss = e0.elapsed_time(e1) / reps
    tf_loss = flops / (ms_loss * 1e-3) / 1e12
    return {"workload": "configs[3] W 14336x4096 bf16, X 4096x4096 bf16, r = 8, 4, 2, fp32 outputs, one matq_gemm_multi(MATQ_SRC_BF16) call",
            "loss_variant": {"call": "matq_gemm_multi_loss: lambda-weighted squared error against a target instead of the outputs",
                             "ms": round(ms_loss, 3), "TFLOPs": round(tf_loss, 1),
                             "frac_tensor_sustained": round(tf_loss / peaks["bf16_tflops_sustained"], 4)},
            "ms": round(ms, 3), "TFLOPs": round(tf, 1), "frac_tensor_sustained": round(tf / peaks["bf16_tflops_sustained"], 4),
            "frac_tensor_burst": round(tf / peaks["bf16_tflops"], 4), "flops": flops,
            "roofline": {"kernel": "gemm_multi (quantize + expand + rowsum + tcgen05 GEMM)", "bound": "tensor", "achieved": round(tf, 1),
                         "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s", "frac": round(tf / peaks["bf16_tflops_sustained"], 4),
                         "traffic": None, "peak_source": peaks["source"] + " (sustained)"}}


def gemv_cfg3(mq, torch, peaks, layers=6, reps=10):
    """configs[2] shapes: Gemma-2-9B decoder layers (q, k, v, o, gate, up, down), B = 1, r = 4 and r = 2.  The planes are
    random bytes (the kernels' speed does not depend on the field values); every matrix has its own buffers."""
    per_layer = [(n, k) for (_, n, k) in synth.gemma2_9b_decoder_layer()]
    # q, k, v share their input and so do gate, up: stacked along N they are one matrix each (rows are quantised
    # independently, so stacking changes no result); 4 launches per layer instead of 7
    d, ff = per_layer[0][1], per_layer[4][0]
    fused_layer = [(per_layer[0][0] + per_layer[1][0] + per_layer[2][0], d), per_layer[3], (2 * ff, d), per_layer[6]]
    out = {"workload": f"configs[2] Gemma-2-9B decoder layer shapes x {layers} layers, r = 8, 4, 2 at B = 1 and r = 4, 2 at B = 4, 16, "
                       "one CUDA graph per case, PDL; "
                       "'_fused' = q,k,v and gate,up stacked into one matrix each (4 launches per layer)"}
    for r, fused, B in ((8, False, 1), (4, False, 1), (2, False, 1), (8, True, 1), (4, True, 1), (2, True, 1),
                        (4, False, 4), (2, False, 4), (4, False, 16), (2, False, 16)):
        shapes = [s for _ in range(layers) for s in (fused_layer if fused else per_layer)]
        planes = [torch.randint(0, 256, (n, k * r // 8), dtype=torch.uint8, device="cuda") for n, k in shapes]
        xs = [torch.randn(B, k, device="cuda").to(torch.bfloat16) for n, k in shapes]
        ys = [torch.empty(B, n, device="cuda") for n, k in shapes]
        al = [torch.ones(n, device="cuda") for n, k in shapes]

        def run():
            for i, (n, k) in enumerate(shapes):
                mq.gemv(planes[i], k, r, al[i], al[i], xs[i], y=ys[i], flags=mq.GEMV_AUTO | mq.GEMV_PDL)
        side = torch.cuda.Stream()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            run()
            torch.cuda.synchronize()
            with torch.cuda.graph(g, stream=side):
                run()
        torch.cuda.synchronize()
        for _ in range(3):
            g.replay()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            g.replay()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / reps
        nbytes = sum(bytes_gemv(n, k, r, B) for n, k in shapes)
        out[f"r{r}_b{B}" + ("_fused" if fused else "")] = {"ms": round(ms, 4), "GBps": round(nbytes / ms / 1e6, 1),
                           "frac_hbm": round(nbytes / ms / 1e6 / peaks["hbm_gbs"], 4), "launches": len(shapes)}
        del planes, xs, ys, al, g
        torch.cuda.empty_cache()
    return out


def quantize_clip_cfg5(mq, torch, peaks, layers=2, reps=10):
    """Eq. 3 on configs[4]'s weights: Gemma-2-9B MLP shapes, Student-t(3) weights, clipping scales gamma = beta = 0.5
    on every channel (learning them is outside the library), then the extra-precision int2 slice of those codes:
    the fraction of codes in the extra bucket comes from the weights and the clamp, not from injected codes."""
    shapes = [(n, k) for _ in range(layers) for (_, n, k) in synth.gemma2_9b_mlp_layer()]
    Ws = [torch.from_numpy(synth.weight_bf16(5, i, n, k)).cuda().view(torch.bfloat16) for i, (n, k) in enumerate(shapes)]
    outs = [(torch.empty((n, k), dtype=torch.uint8, device="cuda"), torch.empty(n, device="cuda"), torch.empty(n, device="cuda"))
            for n, k in shapes]
    gs = [torch.full((n,), 0.5, device="cuda") for n, k in shapes]

    def run():
        for W, (q, a, z), g in zip(Ws, outs, gs):
            mq.quantize(W, q=q, alpha=a, zero=z, gamma=g, beta=g)
    side = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        run()
        torch.cuda.synchronize()
        with torch.cuda.graph(g, stream=side):
            run()
    torch.cuda.synchronize()
    for _ in range(3):
        g.replay()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        g.replay()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / reps
    nbytes = sum(bytes_quantize(n, k) + 8 * n for n, k in shapes)
    n0, k0 = shapes[0]
    sp = mq.slice_pack(outs[0][0], 2, extra_precision=True, ovf_capacity=n0 * k0)
    return {"workload": f"Eq. 3 on configs[4] weights: {layers} Gemma-2-9B MLP layers, Student-t(3), gamma = beta = 0.5, matq_quantize_clip",
            "ms": round(ms, 4), "GBps": round(nbytes / ms / 1e6, 1), "frac_hbm": round(nbytes / ms / 1e6 / peaks["hbm_gbs"], 4),
            "launches": len(shapes), "overflow_fraction_r2": round(int(sp["ovf_count"].item()) / (n0 * k0), 4)}


def gemv_cfg2_mixnmatch(mq, torch, peaks, reps=10):
    """Layer-wise Mix'n'Match on configs[1]: the 26-layer Gemma-2-2B MLP stack served with the Pyramid assignment
    (int2 at both ends, int8 in the centre, int4 in between; 8 + 10 + 8 layers = 4.62 effective bits), B = 1, every
    matrix of a layer at that layer's precision, one CUDA graph, PDL.  Planes are random bytes."""
    from paper_2502_06786_b200 import mixnmatch
    rs = mixnmatch.assign(8, 10, 8, "pyramid")
    mats = [(n, k, rs[l]) for l in range(len(rs)) for (_, n, k) in synth.gemma2_2b_mlp_layer()]
    planes = [torch.randint(0, 256, (n, k * r // 8), dtype=torch.uint8, device="cuda") for n, k, r in mats]
    xs = [torch.randn(1, k, device="cuda").to(torch.bfloat16) for n, k, r in mats]
    ys = [torch.empty(1, n, device="cuda") for n, k, r in mats]
    al = [torch.ones(n, device="cuda") for n, k, r in mats]

    def run():
        for i, (n, k, r) in enumerate(mats):
            mq.gemv(planes[i], k, r, al[i], al[i], xs[i], y=ys[i], flags=mq.GEMV_AUTO | mq.GEMV_PDL)
    side = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        run()
        torch.cuda.synchronize()
        with torch.cuda.graph(g, stream=side):
            run()
    torch.cuda.synchronize()
    for _ in range(3):
        g.replay()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        g.replay()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / reps
    nbytes = sum(bytes_gemv(n, k, r, 1) for n, k, r in mats)
    return {"workload": "configs[1] stack, Pyramid Mix'n'Match: 4 int2 + 5 int4 + 8 int8 + 5 int4 + 4 int2 layers, B = 1, PDL",
            "effective_bits": round(mixnmatch.effective_bits(rs), 3), "ms": round(ms, 4), "GBps": round(nbytes / ms / 1e6, 1),
            "frac_hbm": round(nbytes / ms / 1e6 / peaks["hbm_gbs"], 4), "launches": len(mats)}


def gemm_cfg5_prefill(mq, torch, peaks, reps=3):
    """configs[4] prefill: extra-precision int2 plane (+ overflow lists, 5 % of the codes in the extra bucket) of a
    Gemma-2-9B gate matrix (14336 x 3584), M = 2048 tokens, matq_gemm_multi(MATQ_SRC_PACKED)."""
    N, K, M = 14336, 3584, 2048
    q = torch.from_numpy(synth.skewed_codes((N, K), 0.05, 224, synth.seed_for(5, 0))).cuda()
    sp = mq.slice_pack(q, 2, extra_precision=True, ovf_capacity=N * K // 8)
    X = torch.from_numpy(synth.normal_bf16((M, K), 1.0, synth.seed_for(5, 500))).cuda().view(torch.bfloat16)
    a = torch.full((N,), 1e-3, dtype=torch.float32, device="cuda"); z = torch.full((N,), 128.0, dtype=torch.float32, device="cuda")
    Y = [torch.empty((M, N), dtype=torch.float32, device="cuda")]
    ws = torch.empty(mq.gemm_multi_workspace_bytes(mq.SRC_PACKED, M, N, K, 1), dtype=torch.uint8, device="cuda")

    def run():
        mq.gemm_multi(mq.SRC_PACKED, sp["packed"], K, X, rs=(2,), alpha=a, zero=z, extra_precision=True,
                      ovf_row_ptr=sp["ovf_row_ptr"], ovf_col=sp["ovf_col"], Ys=Y, workspace=ws)
    run(); run()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        run()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / reps
    tf = 2.0 * M * N * K / (ms * 1e-3) / 1e12
    return {"workload": "configs[4] prefill: E.P. int2 plane + overflow lists, 14336x3584, M = 2048, one matq_gemm_multi(MATQ_SRC_PACKED) call",
            "ms": round(ms, 3), "TFLOPs": round(tf, 1), "frac_tensor_sustained": round(tf / peaks["bf16_tflops_sustained"], 4),
            "overflow_fraction": round(int(sp["ovf_count"].item()) / (N * K), 4)}


def e2e_leg(st, plan, W_host, x_host, args, torch, world, dist):
    """The same step from HOST buffers: weights and activations are copied from pinned memory, every y is read back."""
    n = len(st.shapes)
    Wp = [torch.from_numpy(w).pin_memory() for w in W_host]
    xp = [torch.from_numpy(x).pin_memory() for x in x_host]
    yp = {nm: [torch.empty(t.shape, dtype=t.dtype).pin_memory() for t in ts] for nm, ts in st.y.items()}
    h2d = sum(w.numel() * 2 for w in Wp) + sum(x.numel() * 2 for x in xp)
    d2h = sum(t.numel() * 4 for ts in yp.values() for t in ts)

    def step():
        for i in range(n):
            st.W[i].view(torch.uint16).copy_(Wp[i], non_blocking=True)
            st.x8[i].view(torch.uint16).copy_(xp[i], non_blocking=True)
        for _, fn, _, _, _ in plan:
            fn()
        for nm, ts in st.y.items():
            for i in range(n):
                yp[nm][i].copy_(ts[i], non_blocking=True)

    steps = max(1, min(args.steps, 3))
    step()
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    if dist is not None:
        t = torch.tensor([ms], device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())
    step_bytes = sum(p[3] for p in plan)
    return {"value": round(world * step_bytes / (ms * 1e-3) / 1e9, 1), "unit": "GB/s", "ms_per_step": round(ms, 3),
            "steps": steps, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h}


# ----------------------------------------------------------------------------
# the oracle arm (CPU baseline and --impl reference)
# ----------------------------------------------------------------------------

def oracle_step(shapes, W_host, x_host, ref):
    """The same stages, executed by the CPU oracle as it stands.  Returns (seconds, algorithmic bytes)."""
    nbytes = 0
    t0 = time.perf_counter()
    for (idx, layer, name, N, K), W, x in zip(shapes, W_host, x_host):
        st, q, a, z = ref.quantize(W)
        sp4 = ref.slice_pack(q, 4, want_unpacked=False)
        sp2 = ref.slice_pack(q, 2, extra_precision=True, want_unpacked=False)
        nnz = sp2["ovf_count"]
        x1 = np.ascontiguousarray(x[:1])
        ref.gemv(sp4["packed"], K, 4, a, z, x1)
        ref.gemv(sp4["packed"], K, 4, a, z, x)
        ref.gemv(sp2["packed"], K, 2, a, z, x1)
        ref.gemv(sp2["packed"], K, 2, a, z, x)
        ref.gemv(sp2["packed"], K, 2, a, z, x1, sp2["ovf_row_ptr"], sp2["ovf_col"])
        nbytes += (bytes_quantize(N, K) + bytes_slice_pack(N, K, 4) + bytes_slice_pack(N, K, 2, nnz) +
                   bytes_gemv(N, K, 4, 1) + bytes_gemv(N, K, 4, 8) + bytes_gemv(N, K, 2, 1) + bytes_gemv(N, K, 2, 8) +
                   bytes_gemv(N, K, 2, 1, nnz))
    return time.perf_counter() - t0, nbytes


def cpu_baseline(shapes, W_host, x_host, sample_layers):
    from oracle import ref
    ref.build()
    per_layer = len(synth.WORKLOADS[CONFIG_ID]["layer"])
    k = sample_layers * per_layer
    secs, nbytes = oracle_step(shapes[:k], W_host[:k], x_host[:k], ref)
    return {"value": round(nbytes / secs / 1e9, 3), "unit": "GB/s", "cores": ref.num_threads(), "kind": "oracle",
            "sample": f"first {sample_layers} of {synth.WORKLOADS[CONFIG_ID]['layers']} layers of the same stack, same stages "
                      f"(no dense forward), {secs:.1f} s of CPU work",
            "seconds": round(secs, 2)}


def run_reference(args, rank):
    if rank != 0:
        return None
    from oracle import ref
    ref.build()
    sample_layers = min(args.layers, 2)
    shapes, W_host, x_host = host_stack(0, sample_layers)
    for _ in range(min(args.warmup, 1)):
        oracle_step(shapes[:3], W_host[:3], x_host[:3], ref)
    steps = max(1, min(args.steps, 5))
    tot_s = tot_b = 0.0
    for _ in range(steps):
        s, b = oracle_step(shapes, W_host, x_host, ref)
        tot_s += s
        tot_b += b
    v = round(tot_b / tot_s / 1e9, 3)
    sample = f"each step = first {sample_layers} layers of the stack, same stages without the dense forward"
    return {"impl": "reference", "metric": METRIC, "value": v, "unit": "GB/s", "n_gpus": args.gpus, "steps": steps,
            "warmup": min(args.warmup, 1), "ms_per_step": round(tot_s / steps * 1e3, 2), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": "configs[1] Gemma-2-2B-shaped MLP decode stack (bounded sample)", "sample": sample},
            "cpu_baseline": {"value": v, "unit": "GB/s", "cores": ref.num_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": v, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--layers", type=int, default=synth.WORKLOADS[CONFIG_ID]["layers"])
    ap.add_argument("--cpu-sample-layers", type=int, default=6)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-cfg4", action="store_true", help="skip the extra Mistral-7B-shaped gemm_multi measurement")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        out = run_reference(args, rank)
        if out is not None:
            print(json.dumps(out), flush=True)
        return

    out, st = run_cuda(args, rank, world, local_rank)
    if rank == 0:
        if world == 1 and not args.no_cpu_baseline:
            k = min(args.cpu_sample_layers, args.layers)
            shapes, W_host, x_host = host_stack(0, k)
            out["cpu_baseline"] = cpu_baseline(shapes, W_host, x_host, k)
        print(json.dumps(out), flush=True)


if __name__ == "__main__":
    main()
