#!/usr/bin/env python
"""Benchmark of the nested int8 -> int4 -> int2 weight path on one node.

A step is one pass of the whole path over the Gemma-2-2B-shaped MLP stack
(26 layers x {gate, up: 9216x2304, down: 2304x9216}, bf16 weights N(0, 0.02)):

  quantize (Eq. 1)                      bf16 W -> uint8 codes, alpha, z            one launch per matrix
  slice_pack r=4 (Eq. 6)                codes -> packed int4 plane                 one launch per matrix
  slice_pack r=2 + extra precision      codes -> packed int2 plane + Eq. 8 lists   one launch per matrix
  decode GEMV  r=4, r=2        B=1      packed planes, bf16 x -> fp32 y            matq_gemv_grouped, the whole stack per call
  decode GEMV  r=2 + Eq. 8     B=1      the same with the overflow lists           matq_gemv_grouped
  decode GEMV  r=4, r=2        B=8      bf16 tensor kernel                         one launch per matrix

The metric is the decode GEMV's HBM throughput, so `value` is the algorithmic bytes of the two B = 1 GEMV stages
(r = 4 and r = 2) over their device time, and `roofline` describes that kernel; the other stages and the blended
figure of the whole step are in `stages` / `step_GBps`.  `roofline.gemv_frac_hbm` lists every GEMV measurement of
the run as a fraction of the measured copy bandwidth: this stack at three launch granularities, the Gemma-2-9B
decoder stack (configs[2], 42 layers, r = 8, 4, 2 at B = 1, 4, 16) and the extra-precision int2 MLP stack
(configs[4], Student-t weights, and the 5 % overflow regime of trained codes).

The dense multi-precision forward (Eq. 7) has no place in a decode-shaped workload; it is measured on its own
configuration, the Mistral-7B-shaped co-training forward, and reported under `gemm_multi_cfg4` with its roofline.

Every matrix of a stack has its own buffers, so each stage streams far more than the L2 holds.  Before anything is
timed, the first matrix of the stack goes through every stage once and is compared with the CPU oracle; a mismatch
aborts the run.

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
# profiles/; a kernel that has changed since its capture reports traffic = null.
NCU = {
    # matq_gemv_grouped on 12 matrices of this stack (profiles/gemv_stream_*.md): DRAM bytes / algorithmic bytes
    "gemv_stream_ratio_r4": 1.022,
    "gemv_stream_ratio_r2": 0.992,
    "quantize": 42780000,
}
CONFIG_ID = 2
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1590.0
TOL_INT8, TOL_TENSOR = 1e-4, 1e-2


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
# timing helpers
# ----------------------------------------------------------------------------

def capture(torch, fn):
    """One CUDA graph of `fn` (run once eagerly first).  The inputs were produced on the default stream: wait for them."""
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        fn()
        torch.cuda.synchronize()
        with torch.cuda.graph(g, stream=side):
            fn()
    torch.cuda.synchronize()
    return g


def time_graph(torch, g, reps=10, warm=3):
    for _ in range(warm):
        g.replay()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        g.replay()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / reps


def gemv_entry(ms, nbytes, peaks, launches):
    return {"ms": round(ms, 4), "GBps": round(nbytes / ms / 1e6, 1), "frac_hbm": round(nbytes / ms / 1e6 / peaks["hbm_gbs"], 4),
            "launches": launches}


def chunks(seq, n):
    return [seq[i:i + n] for i in range(0, len(seq), n)]


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
        self.W_pinned = self.x_pinned = None
        self.upload(W_host, x_host)
        self._groups = {}

    def upload(self, W_host, x_host):
        torch = self.torch
        for i, (W, x) in enumerate(zip(W_host, x_host)):
            self.W[i].view(torch.uint16).copy_(torch.from_numpy(W))
            self.x8[i].view(torch.uint16).copy_(torch.from_numpy(x))
        torch.cuda.synchronize()

    def problems(self, nm, r, ep, idx, batch=False):
        """matq_gemv_grouped descriptors of the matrices `idx`: the first activation vector, or all eight (`batch`)."""
        key = (nm, r, ep, tuple(idx), batch)
        if key not in self._groups:
            planes = self.p4 if r == 4 else self.p2
            self._groups[key] = self.mq.gemv_group([
                dict(packed=planes[i], K=self.shapes[i][4], r=r, alpha=self.alpha[i], zero=self.zero[i],
                     x=self.x8[i] if batch else self.x8[i][0], y=self.y[nm][i] if batch else self.y[nm][i][0],
                     ovf_row_ptr=self.rp[i] if ep else None, ovf_col=self.col[i] if ep else None) for i in idx])
        return self._groups[key]

    def gemv_b1(self, nm, r, ep, group):
        """B = 1 GEMV over the stack: `group` matrices per matq_gemv_grouped call (0 = one matq_gemv per matrix)."""
        mq, n, S = self.mq, len(self.shapes), self.shapes
        if group == 0:
            planes = self.p4 if r == 4 else self.p2

            def run():
                for i in range(n):
                    mq.gemv(planes[i], S[i][4], r, self.alpha[i], self.zero[i], self.x8[i][:1], y=self.y[nm][i],
                            ovf_row_ptr=self.rp[i] if ep else None, ovf_col=self.col[i] if ep else None,
                            flags=mq.GEMV_AUTO | mq.GEMV_PDL)
            return run, n
        groups = [self.problems(nm, r, ep, idx) for idx in chunks(list(range(n)), group)]

        def run():
            for g in groups:
                mq.gemv_grouped(g, flags=mq.GEMV_PDL, dev_status=self.status)
        return run, sum((len(g) + 127) // 128 for g in groups)

    def gemv_b8_per_matrix(self, nm, r):
        """B = 8 with one matq_gemv (the bf16 tensor kernel) per matrix: the comparison for the whole-stack call."""
        mq, n, S = self.mq, len(self.shapes), self.shapes
        planes = self.p4 if r == 4 else self.p2

        def run():
            for i in range(n):
                mq.gemv(planes[i], S[i][4], r, self.alpha[i], self.zero[i], self.x8[i], y=self.y[nm][i], flags=mq.GEMV_AUTO | mq.GEMV_PDL)
        return run, n

    # stage-major plan: (name, callable over the whole stack, kernels launched, algorithmic bytes)
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

        def sp42():
            for i in range(n):
                mq.slice_pack_nested(self.q[i], extra_precision=True, packed4=self.p4[i], packed2=self.p2[i], ovf_row_ptr=self.rp[i],
                                     ovf_col=self.col[i], ovf_capacity=self.cap[i], ovf_count=self.cnt[i], dev_status=self.status)
        self.slice_alone = {"slice_pack_r4_alone": (sp4, n, sum(bytes_slice_pack(N, K, 4) for (_, _, _, N, K) in S)),
                            "slice_pack_r2_ep_alone": (sp2, 2 * n, sum(bytes_slice_pack(N, K, 2, z) for (_, _, _, N, K), z in
                                                                       zip(S, getattr(self, "nnz", [0] * n))))}

        def gemv_b8(nm, r):
            """B = 8 over the whole stack in one matq_gemv_grouped call."""
            g = self.problems(nm, r, False, list(range(n)), batch=True)

            def run():
                mq.gemv_grouped(g, flags=mq.GEMV_PDL, dev_status=self.status)
            return run, mq.gemv_grouped_launches(g)

        nnz = getattr(self, "nnz", [0] * n)
        g4, l4 = self.gemv_b1("g4b1", 4, False, n)
        g2, l2 = self.gemv_b1("g2b1", 2, False, n)
        gep, lep = self.gemv_b1("g2ep", 2, True, n)
        return [
            ("quantize", quant, n, sum(bytes_quantize(N, K) for (_, _, _, N, K) in S)),
            # the int4 and the int2 plane (+ lists) from one read of the codes: the codes count once
            ("slice_pack_r4_r2_ep", sp42, 2 * n, sum(bytes_slice_pack(N, K, 4) + bytes_slice_pack(N, K, 2, z) - N * K
                                                     for (_, _, _, N, K), z in zip(S, nnz))),
            # the decode stages come last, the B = 1 ones after the B = 8 ones: a stage that directly follows slice_pack
            # also pays the write-back of the planes that stage left dirty in the L2, which no decode loop ever sees
            ("gemv_r4_b8", *gemv_b8("g4b8", 4), sum(bytes_gemv(N, K, 4, 8) for (_, _, _, N, K) in S)),
            ("gemv_r2_b8", *gemv_b8("g2b8", 2), sum(bytes_gemv(N, K, 2, 8) for (_, _, _, N, K) in S)),
            ("gemv_r4_b1", g4, l4, sum(bytes_gemv(N, K, 4, 1) for (_, _, _, N, K) in S)),
            ("gemv_r2_b1", g2, l2, sum(bytes_gemv(N, K, 2, 1) for (_, _, _, N, K) in S)),
            ("gemv_r2_ep_b1", gep, lep, sum(bytes_gemv(N, K, 2, 1, z) for (_, _, _, N, K), z in zip(S, nnz))),
        ]


def parity_check(st, W0, x0):
    """The first matrix of the stack through every stage, compared with the CPU oracle (outside any timed region)."""
    from oracle import ref
    torch = st.torch

    def host(t):
        torch.cuda.synchronize()
        return t.cpu().numpy()

    def close(y, y_ref, tol, what):
        err = float(np.abs(y - y_ref).max())
        rms = float(np.sqrt(np.mean(np.square(y_ref))))
        if not err <= tol * rms:
            raise SystemExit(f"parity check failed before timing: {what}: max|dy| {err:.3e} > {tol} * rms {rms:.3e}")

    N, K = st.shapes[0][3], st.shapes[0][4]
    rst, q_ref, a_ref, z_ref = ref.quantize(W0)
    if not (np.array_equal(host(st.q[0]), q_ref) and np.array_equal(host(st.alpha[0]), a_ref) and np.array_equal(host(st.zero[0]), z_ref)):
        raise SystemExit("parity check failed before timing: quantize differs from the oracle")
    sp4 = ref.slice_pack(q_ref, 4, want_unpacked=False)
    sp2 = ref.slice_pack(q_ref, 2, extra_precision=True, want_unpacked=False)
    if not (np.array_equal(host(st.p4[0]), sp4["packed"]) and np.array_equal(host(st.p2[0]), sp2["packed"])):
        raise SystemExit("parity check failed before timing: packed planes differ from the oracle")
    cnt = int(host(st.cnt[0])[0])
    if not (cnt == sp2["ovf_count"] and np.array_equal(host(st.rp[0]), sp2["ovf_row_ptr"]) and np.array_equal(host(st.col[0])[:cnt], sp2["ovf_col"])):
        raise SystemExit("parity check failed before timing: extra-precision lists differ from the oracle")
    x1 = np.ascontiguousarray(x0[:1])
    for nm, packed, r, x, rp, col, tol in (("g4b1", sp4["packed"], 4, x1, None, None, TOL_INT8), ("g2b1", sp2["packed"], 2, x1, None, None, TOL_INT8),
                                           ("g2ep", sp2["packed"], 2, x1, sp2["ovf_row_ptr"], sp2["ovf_col"], TOL_INT8),
                                           ("g4b8", sp4["packed"], 4, x0, None, None, TOL_TENSOR), ("g2b8", sp2["packed"], 2, x0, None, None, TOL_TENSOR)):
        _, y_ref = ref.gemv(packed, K, r, a_ref, z_ref, x, rp, col)
        close(host(st.y[nm][0]).astype(np.float64), y_ref, tol, f"gemv {nm}")
    return "first matrix of the stack: codes, alpha, z, planes and lists bit-exact; y within 1e-4 (B = 1) / 1e-2 (B = 8) of rms(y)"


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
    n = len(shapes)

    # one eager pass: warms the kernels up and gives the overflow counts the byte model needs
    for _, fn, _, _ in st.stages():
        fn()
    torch.cuda.synchronize()
    assert int(st.status.item()) == 0, f"device status {int(st.status.item())}"
    st.nnz = [int(c.item()) for c in st.cnt]
    parity = parity_check(st, W_host[0], x_host[0])
    plan = st.stages()

    # One CUDA graph per stage of many launches: the launch overhead of ~500 small kernels would otherwise dominate.
    # A stage that is one or two launches (the whole-stack decode calls) is launched directly: the host is
    # milliseconds ahead of the GPU by then, and a graph launch would put its own start-up, a tenth of such a
    # stage, between the stage's two events.
    graphs = [capture(torch, fn) if launches > 2 else None for _, fn, launches, _ in plan]

    def step(events=None):
        for j, g in enumerate(graphs):
            if events is not None:
                events[j].record()
            if g is None:
                plan[j][1]()
            else:
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
    assert int(st.status.item()) == 0, f"device status {int(st.status.item())} after the timed region"
    total_ms = ev[0][0].elapsed_time(ev[-1][-1])
    stage_ms = [sum(ev[k][j].elapsed_time(ev[k][j + 1]) for k in range(args.steps)) / args.steps
                for j in range(len(graphs))]
    del graphs
    ms_per_step = total_ms / args.steps
    names = [p[0] for p in plan]
    i4, i2 = names.index("gemv_r4_b1"), names.index("gemv_r2_b1")
    gemv_ms = stage_ms[i4] + stage_ms[i2]
    if world > 1:
        t = torch.tensor([ms_per_step, gemv_ms], device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms_per_step, gemv_ms = float(t[0].item()), float(t[1].item())
    step_bytes = sum(p[3] for p in plan)
    gemv_bytes = plan[i4][3] + plan[i2][3]
    value = world * gemv_bytes / (gemv_ms * 1e-3) / 1e9

    stages = {}
    for (name, fn, launches, nbytes), ms in zip(plan, stage_ms):
        stages[name] = dict(ms=round(ms, 4), share=round(ms / sum(stage_ms), 4), GBps=round(nbytes / (ms * 1e-3) / 1e9, 1),
                            frac_hbm=round(nbytes / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"], 4), bytes=nbytes, launches=launches)

    # the same B = 1 GEMV stages at the two finer launch granularities (not part of the step)
    per_layer = len(synth.WORKLOADS[CONFIG_ID]["layer"])
    gemv_frac = {}
    for nm, r, ep, key in (("g4b1", 4, False, "gemv_r4_b1"), ("g2b1", 2, False, "gemv_r2_b1"), ("g2ep", 2, True, "gemv_r2_ep_b1")):
        nbytes = plan[names.index(key)][3]
        gemv_frac[f"cfg2_{key[5:]}_whole_stack_call"] = stages[key]["frac_hbm"]
        for gran, label in ((per_layer, "call_per_layer"), (0, "launch_per_matrix")):
            fn, launches = st.gemv_b1(nm, r, ep, gran)
            ms = time_graph(torch, capture(torch, fn))
            stages[f"{key}_{label}"] = dict(gemv_entry(ms, nbytes, peaks, launches), in_step=False)
            gemv_frac[f"cfg2_{key[5:]}_{label}"] = stages[f"{key}_{label}"]["frac_hbm"]
    for key, (fn, launches, nbytes) in st.slice_alone.items():          # the two planes by separate calls, for comparison
        ms = time_graph(torch, capture(torch, fn))
        stages[key] = dict(gemv_entry(ms, nbytes, peaks, launches), in_step=False)
    for nm, r, key in (("g4b8", 4, "gemv_r4_b8"), ("g2b8", 2, "gemv_r2_b8")):
        gemv_frac[f"cfg2_{key[5:]}_whole_stack_call"] = stages[key]["frac_hbm"]
        fn, launches = st.gemv_b8_per_matrix(nm, r)
        ms = time_graph(torch, capture(torch, fn))
        stages[f"{key}_launch_per_matrix"] = dict(gemv_entry(ms, plan[names.index(key)][3], peaks, launches), in_step=False)
        gemv_frac[f"cfg2_{key[5:]}_launch_per_matrix"] = stages[f"{key}_launch_per_matrix"]["frac_hbm"]

    gpu_launches = sum(p[2] for p in plan)

    # ------------------------------------------------------------------ end to end from host buffers
    e2e = e2e_leg(st, plan, W_host, x_host, args, torch, world, dist if world > 1 else None)

    extras = {}
    if world == 1 and not args.quick:
        for t in (st.W, st.q, st.p4, st.p2, st.col):       # free the stack's large buffers first
            t.clear()
        st._groups.clear()
        torch.cuda.empty_cache()
        extras["gemm_multi_cfg4"] = gemm_cfg4(mq, torch, peaks)
        torch.cuda.empty_cache()
        extras["gemv_cfg3"] = gemv_cfg3(mq, torch, peaks, gemv_frac)
        torch.cuda.empty_cache()
        extras["cfg5_extra_precision"] = cfg5_extra_precision(mq, torch, peaks, gemv_frac)
        torch.cuda.empty_cache()
        extras["gemm_multi_cfg5_prefill"] = gemm_cfg5_prefill(mq, torch, peaks)
        torch.cuda.empty_cache()
        extras["quantize_clip_cfg5"] = quantize_clip_cfg5(mq, torch, peaks)
        torch.cuda.empty_cache()
        extras["gemv_cfg2_mixnmatch"] = gemv_cfg2_mixnmatch(mq, torch, peaks, gemv_frac)
        extras["cfg1_linear_1024"] = cfg1_linear(mq, torch, peaks)

    out = None
    if rank == 0:
        ach = gemv_bytes / (gemv_ms * 1e-3) / 1e9
        r4x, r2x = NCU["gemv_stream_ratio_r4"], NCU["gemv_stream_ratio_r2"]
        n_l = plan[i4][2] + plan[i2][2]
        traffic = None if r4x is None or r2x is None else int((plan[i4][3] * r4x + plan[i2][3] * r2x) / n_l)
        roofline = dict(kernel="gemv_stream (matq_gemv_grouped: persistent integer-MMA GEMV, B = 1), r = 4 and r = 2 stages of the step",
                        bound="hbm", achieved=round(ach, 1), peak=peaks["hbm_gbs"], unit="GB/s", frac=round(ach / peaks["hbm_gbs"], 4),
                        traffic=traffic, peak_source=peaks["source"],
                        traffic_note="DRAM bytes per launch (mean of the r = 4 and r = 2 whole-stack launches, like bytes_per_launch), scaled by "
                                     "planes read from the ncu captures of 12-matrix calls (profiles/gemv_stream_cfg2_12_matrices.md)",
                        avg_launch_us=round(gemv_ms * 1e3 / (plan[i4][2] + plan[i2][2]), 2),
                        bytes_per_launch=gemv_bytes // (plan[i4][2] + plan[i2][2]), gemv_frac_hbm=gemv_frac)
        out = {
            "metric": METRIC, "value": round(value, 1), "unit": "GB/s", "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": round(ms_per_step, 4), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None,
            "dtype": "u8 fields x block-scaled 30-bit integer activations, s32 sums (B = 1); bf16 x bf16 -> fp32 (B = 8, dense forward)",
            "data": "synthetic",
            "config": {"workload": f"configs[1] Gemma-2-2B-shaped MLP decode stack, {args.layers} layers x (gate,up 9216x2304; down 2304x9216), "
                                   "bf16 N(0,0.02) weights, x bf16 N(0,1)",
                       "step": "quantize -> slice_pack r=4 and r=2 + extra-precision lists in one pass (matq_slice_pack_nested) -> gemv r=4, r=2 at B=8 -> gemv r=4, r=2, r=2 E.P. at B=1 "
                               "(all decode stages: matq_gemv_grouped, whole stack per call)"
                               "; dense multi-precision forward measured separately (gemm_multi_cfg4)",
                       "value_definition": "decode GEMV at B = 1: algorithmic HBM bytes of the gemv_r4_b1 and gemv_r2_b1 stages / their device time "
                                           f"({round(gemv_ms, 4)} ms of the step); step_GBps is the same ratio over all stages",
                       "l2": "inputs larger than L2: every matrix has its own buffers, each stage streams >= 0.4 GB",
                       "parallelism": "one independent stack per GPU (rows are independent; no collective)" if world > 1 else "single GPU",
                       "overflow_fraction_r2": round(sum(st.nnz) / sum(N * K for (_, _, _, N, K) in shapes), 6),
                       "parity_before_timing": parity},
            "clocks": clocks, "e2e": e2e, "gpu_launches": gpu_launches, "roofline": roofline,
            "step_GBps": round(world * step_bytes / (ms_per_step * 1e-3) / 1e9, 1), "stages": stages,
        }
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
    q = torch.empty((N, K), dtype=torch.uint8, device="cuda")
    ws = torch.empty(mq.gemm_multi_workspace_bytes(mq.SRC_BF16, M, N, K, 3), dtype=torch.uint8, device="cuda")

    def timed(fn):
        fn(); fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps

    ms = timed(lambda: mq.gemm_multi(mq.SRC_BF16, W, K, X, alpha=a, zero=z, Ys=Ys, workspace=ws))
    # where the call's time goes: Eq. 1 alone, and the call from ready-made codes (field planes + row sums + GEMM)
    ms_quant = timed(lambda: mq.quantize(W, q=q, alpha=a, zero=z))
    ms_codes = timed(lambda: mq.gemm_multi(mq.SRC_CODES8, q, K, X, alpha=a, zero=z, Ys=Ys, workspace=ws))
    flops = 3 * 2.0 * M * N * K
    tf = flops / (ms * 1e-3) / 1e12
    # the same pass as Eq. 7's objective: the three outputs are compared with a target in the epilogue and never stored
    Yt = Ys[0]                                      # any fp32 [M, N] serves as the target for timing
    del Ys[1:]
    wl = torch.empty(mq.gemm_multi_loss_workspace_bytes(mq.SRC_BF16, M, N, K, 3), dtype=torch.uint8, device="cuda")
    loss = torch.empty(4, dtype=torch.float64, device="cuda")
    ms_loss = timed(lambda: mq.gemm_multi_loss(mq.SRC_BF16, W, K, X, Yt, (1.0, 1.0, 1.0), alpha=a, zero=z, loss=loss, workspace=wl))
    tf_loss = flops / (ms_loss * 1e-3) / 1e12
    # DRAM traffic of the GEMM kernel, scaled from the ncu capture at M = 1024 (profiles/gemm_multi_kernel_m1024_14336x4096.md):
    # the three bf16 planes are read once whatever M is (394 MB - 8.4 MB of X at M = 1024), X and the outputs grow with M
    traffic = int((394e6 - 8.4e6) + 8.4e6 * M / 1024 + 176e6 * M / 1024)
    return {"workload": "configs[3] W 14336x4096 bf16, X 4096x4096 bf16, r = 8, 4, 2, fp32 outputs, one matq_gemm_multi(MATQ_SRC_BF16) call",
            "loss_variant": {"call": "matq_gemm_multi_loss: lambda-weighted squared error against a target instead of the outputs",
                             "ms": round(ms_loss, 3), "TFLOPs": round(tf_loss, 1),
                             "frac_tensor_sustained": round(tf_loss / peaks["bf16_tflops_sustained"], 4)},
            "ms": round(ms, 3), "TFLOPs": round(tf, 1), "frac_tensor_sustained": round(tf / peaks["bf16_tflops_sustained"], 4),
            "frac_tensor_burst": round(tf / peaks["bf16_tflops"], 4), "flops": flops,
            "split_ms": {"matq_quantize alone (Eq. 1)": round(ms_quant, 3),
                         "call from uint8 codes (field planes + row sums + tcgen05 GEMM)": round(ms_codes, 3),
                         "kernel shares of the call": "profiles/gemm_multi_kernel_m1024_14336x4096.md"},
            "roofline": {"kernel": "gemm_multi (quantize + expand + rowsum + tcgen05 GEMM)", "bound": "tensor", "achieved": round(tf, 1),
                         "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s", "frac": round(tf / peaks["bf16_tflops_sustained"], 4),
                         "traffic": traffic, "traffic_note": "GEMM kernel only, scaled from the ncu capture at M = 1024 (planes constant, X and Y in proportion to M)",
                         "peak_source": peaks["source"] + " (sustained)"}}


def _gemv_cases(mq, torch, shapes, planes, r, xs, ys, al, Bs, per_layer, peaks, out, gemv_frac, prefix, rps=None, cols=None, nnz=None):
    """GEMV over a stack of planes: B = 1 at three launch granularities, other batches one launch per matrix."""
    n = len(shapes)
    for B in Bs:
        nbytes = sum(bytes_gemv(N, K, r, B, None if nnz is None else nnz[i]) for i, (N, K) in enumerate(shapes))
        ep = rps is not None

        def per_matrix():
            for i, (N, K) in enumerate(shapes):
                mq.gemv(planes[i], K, r, al[i], al[i], xs[i][:B], y=ys[i][:B], ovf_row_ptr=rps[i] if ep else None,
                        ovf_col=cols[i] if ep else None, flags=mq.GEMV_AUTO | mq.GEMV_PDL)
        ms = time_graph(torch, capture(torch, per_matrix), reps=5)
        out[f"r{r}_b{B}_launch_per_matrix"] = gemv_entry(ms, nbytes, peaks, n)
        gemv_frac[f"{prefix}_r{r}_b{B}_launch_per_matrix"] = out[f"r{r}_b{B}_launch_per_matrix"]["frac_hbm"]
        if B != 1:
            if ep:
                continue
            # batches: the whole stack in one matq_gemv_grouped call (the batched persistent kernel)
            g = mq.gemv_group([dict(packed=planes[i], K=K, r=r, alpha=al[i], zero=al[i], x=xs[i][:B], y=ys[i][:B])
                               for i, (N, K) in enumerate(shapes)])
            ms = time_graph(torch, capture(torch, lambda: mq.gemv_grouped(g, flags=mq.GEMV_PDL)), reps=5)
            out[f"r{r}_b{B}_whole_stack_call"] = gemv_entry(ms, nbytes, peaks, mq.gemv_grouped_launches(g))
            gemv_frac[f"{prefix}_r{r}_b{B}_whole_stack_call"] = out[f"r{r}_b{B}_whole_stack_call"]["frac_hbm"]
            continue
        probs = [dict(packed=planes[i], K=K, r=r, alpha=al[i], zero=al[i], x=xs[i][0], y=ys[i][0],
                      ovf_row_ptr=rps[i] if ep else None, ovf_col=cols[i] if ep else None) for i, (N, K) in enumerate(shapes)]
        for gran, label in ((per_layer, "call_per_layer"), (n, "whole_stack_call")):
            groups = [mq.gemv_group(c) for c in chunks(probs, gran)]

            def grouped():
                for g in groups:
                    mq.gemv_grouped(g, flags=mq.GEMV_PDL)
            ms = time_graph(torch, capture(torch, grouped), reps=5)
            launches = sum((len(g) + 127) // 128 for g in groups)
            out[f"r{r}_b1_{label}"] = gemv_entry(ms, nbytes, peaks, launches)
            gemv_frac[f"{prefix}_r{r}_b1_{label}"] = out[f"r{r}_b1_{label}"]["frac_hbm"]


def gemv_cfg3(mq, torch, peaks, gemv_frac):
    """configs[2]: the Gemma-2-9B decoder stack, all 42 layers (q, k, v, o, gate, up, down: 8.32 G weights), r = 8, 4, 2 at
    B = 1, 4, 16.  The planes are random bytes (the kernels' speed does not depend on the field values); every matrix has
    its own buffers."""
    layers = synth.WORKLOADS[3]["layers"]
    per_layer = [(n, k) for (_, n, k) in synth.gemma2_9b_decoder_layer()]
    shapes = [s for _ in range(layers) for s in per_layer]
    out = {"workload": f"configs[2] Gemma-2-9B decoder stack, {layers} layers x (q, k, v, o, gate, up, down), r = 8, 4, 2 at B = 1, 4, 16; "
                       "B = 1: one launch per matrix (PDL chain), one matq_gemv_grouped call per layer, one for the whole stack; "
                       "B = 4, 16: one launch per matrix (bf16 tensor kernel) and one matq_gemv_grouped call for the whole stack (batched "
                       "integer kernel); one CUDA graph per case"}
    xs = [torch.randn(16, k, device="cuda").to(torch.bfloat16) for n, k in shapes]
    ys = [torch.empty(16, n, device="cuda") for n, k in shapes]
    al = [torch.ones(n, device="cuda") for n, k in shapes]
    for r in (8, 4, 2):
        planes = [torch.randint(0, 256, (n, k * r // 8), dtype=torch.uint8, device="cuda") for n, k in shapes]
        _gemv_cases(mq, torch, shapes, planes, r, xs, ys, al, (1, 4, 16), len(per_layer), peaks, out, gemv_frac, "cfg3")
        del planes
        torch.cuda.empty_cache()
    return out


def cfg5_extra_precision(mq, torch, peaks, gemv_frac):
    """configs[4]: extra-precision int2 on the Gemma-2-9B MLP stack (42 layers x gate, up 14336x3584, down 3584x14336).
    (a) Student-t(3) weights scaled to std 0.02, generated on the GPU from a seeded torch generator (t = z0 / sqrt(chi2_3 / 3);
    the host generator of the tests would need minutes for 6.5 G weights), quantised with Eq. 1, sliced with Eq. 8: the
    overflow fraction is what plain min-max gives on heavy-tailed rows.  (b) '5b': codes drawn with P(q >= 224) = 0.05,
    the share of the extra bucket that the paper reports for trained int2 models (Table 7's 2.05 bits)."""
    layers = synth.WORKLOADS[5]["layers"]
    per_layer = [(n, k) for (_, n, k) in synth.gemma2_9b_mlp_layer()]
    shapes = [s for _ in range(layers) for s in per_layer]
    n = len(shapes)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(synth.seed_for(5, 0))
    out = {"workload": f"configs[4] Gemma-2-9B MLP stack, {layers} layers, extra-precision int2 (Eq. 8), B = 1"}
    xs = [torch.randn(1, k, device="cuda", generator=gen).to(torch.bfloat16) for N, k in shapes]
    ys = [torch.empty(1, N, device="cuda") for N, k in shapes]
    for variant in ("student_t", "5b"):
        codes, alphas, zeros = [], [], []
        for (N, K) in shapes:
            if variant == "student_t":
                z0 = torch.randn(N, K, device="cuda", generator=gen)
                chi = torch.randn(N, K, device="cuda", generator=gen).square_()
                chi += torch.randn(N, K, device="cuda", generator=gen).square_()
                chi += torch.randn(N, K, device="cuda", generator=gen).square_()
                W = (z0 * torch.rsqrt(chi / 3.0) * (0.02 / 3.0 ** 0.5)).to(torch.bfloat16)
                del z0, chi
                q, a, z = mq.quantize(W)
                del W
            else:
                top = torch.rand(N, K, device="cuda", generator=gen) < 0.05
                q = torch.where(top, torch.randint(224, 256, (N, K), device="cuda", generator=gen, dtype=torch.uint8),
                                torch.randint(0, 224, (N, K), device="cuda", generator=gen, dtype=torch.uint8))
                del top
                a = torch.full((N,), 1e-3, device="cuda"); z = torch.full((N,), 128.0, device="cuda")
            codes.append(q); alphas.append(a); zeros.append(z)
        caps = [N * K // 8 for N, K in shapes]
        planes = [torch.empty((N, K // 4), dtype=torch.uint8, device="cuda") for N, K in shapes]
        rps = [torch.empty(N + 1, dtype=torch.int32, device="cuda") for N, K in shapes]
        cols = [torch.empty(c, dtype=torch.uint16, device="cuda") for c in caps]
        cnts = [torch.zeros(1, dtype=torch.int64, device="cuda") for _ in shapes]
        status = torch.zeros(n, dtype=torch.int32, device="cuda")

        def sp():
            for i in range(n):
                mq.slice_pack(codes[i], 2, extra_precision=True, packed=planes[i], ovf_row_ptr=rps[i], ovf_col=cols[i],
                              ovf_capacity=caps[i], ovf_count=cnts[i], dev_status=status[i:i + 1])
        ms = time_graph(torch, capture(torch, sp), reps=3, warm=1)
        nnz = [int(c.item()) for c in cnts]
        bad = [(i, int(v), nnz[i], caps[i]) for i, v in enumerate(status.tolist()) if v]
        assert not bad, f"slice_pack (matrix, status, count, capacity): {bad[:8]}"
        sp_bytes = sum(bytes_slice_pack(N, K, 2, z) for (N, K), z in zip(shapes, nnz))
        sub = {"overflow_fraction": round(sum(nnz) / sum(N * K for N, K in shapes), 6),
               "avg_bits_paper": round(2 + sum(nnz) / sum(N * K for N, K in shapes), 4),
               "slice_pack_r2_ep": gemv_entry(ms, sp_bytes, peaks, 2 * n)}
        del codes
        torch.cuda.empty_cache()
        _gemv_cases(mq, torch, shapes, planes, 2, xs, ys, alphas, (1,), len(per_layer), peaks, sub, gemv_frac, f"cfg5_{variant}_ep",
                    rps=rps, cols=cols, nnz=nnz)
        out[variant] = sub
        del planes, rps, cols
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
    ms = time_graph(torch, capture(torch, run), reps=reps)
    nbytes = sum(bytes_quantize(n, k) + 8 * n for n, k in shapes)
    n0, k0 = shapes[0]
    sp = mq.slice_pack(outs[0][0], 2, extra_precision=True, ovf_capacity=n0 * k0)
    return {"workload": f"Eq. 3 on configs[4] weights: {layers} Gemma-2-9B MLP layers, Student-t(3), gamma = beta = 0.5, matq_quantize_clip",
            "ms": round(ms, 4), "GBps": round(nbytes / ms / 1e6, 1), "frac_hbm": round(nbytes / ms / 1e6 / peaks["hbm_gbs"], 4),
            "launches": len(shapes), "overflow_fraction_r2": round(int(sp["ovf_count"].item()) / (n0 * k0), 4)}


def gemv_cfg2_mixnmatch(mq, torch, peaks, gemv_frac, reps=10):
    """Layer-wise Mix'n'Match on configs[1]: the 26-layer Gemma-2-2B MLP stack served with the Pyramid assignment
    (int2 at both ends, int8 in the centre, int4 in between; 8 + 10 + 8 layers = 4.62 effective bits), B = 1, every
    matrix of a layer at that layer's precision.  Planes are random bytes."""
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
    group = mq.gemv_group([dict(packed=planes[i], K=k, r=r, alpha=al[i], zero=al[i], x=xs[i][0], y=ys[i][0]) for i, (n, k, r) in enumerate(mats)])
    nbytes = sum(bytes_gemv(n, k, r, 1) for n, k, r in mats)
    ms = time_graph(torch, capture(torch, run), reps=reps)
    ms_g = time_graph(torch, capture(torch, lambda: mq.gemv_grouped(group, flags=mq.GEMV_PDL)), reps=reps)
    gemv_frac["cfg2_mixnmatch_pyramid_b1_whole_stack_call"] = round(nbytes / ms_g / 1e6 / peaks["hbm_gbs"], 4)
    gemv_frac["cfg2_mixnmatch_pyramid_b1_launch_per_matrix"] = round(nbytes / ms / 1e6 / peaks["hbm_gbs"], 4)
    return {"workload": "configs[1] stack, Pyramid Mix'n'Match: 4 int2 + 5 int4 + 8 int8 + 5 int4 + 4 int2 layers, B = 1",
            "effective_bits": round(mixnmatch.effective_bits(rs), 3),
            "launch_per_matrix": gemv_entry(ms, nbytes, peaks, len(mats)), "whole_stack_call": gemv_entry(ms_g, nbytes, peaks, 1)}


def cfg1_linear(mq, torch, peaks, reps=20):
    """configs[0]: one 1024 x 1024 linear layer (1-2 MB per tensor: L2-resident and launch-bound, a parity configuration;
    reported for completeness and excluded from any bandwidth bar).  One CUDA graph of 24 calls per case, time per call."""
    N = K = 1024
    W = torch.from_numpy(synth.normal_bf16((N, K), 0.02, synth.seed_for(1, 0))).cuda().view(torch.bfloat16)
    x = torch.from_numpy(synth.normal_bf16((1, K), 1.0, synth.seed_for(1, 500))).cuda().view(torch.bfloat16)
    q, a, z = mq.quantize(W)
    out = {"workload": "configs[0] single linear 1024x1024, B = 1; microseconds per call inside a graph of 24 calls"}

    def per_call(fn, nbytes):
        def run():
            for _ in range(24):
                fn()
        us = time_graph(torch, capture(torch, run), reps=reps) * 1e3 / 24
        return {"us": round(us, 2), "GBps": round(nbytes / us / 1e3, 1)}
    out["quantize"] = per_call(lambda: mq.quantize(W, q=q, alpha=a, zero=z), bytes_quantize(N, K))
    y = torch.empty(1, N, device="cuda")
    for r in (8, 4, 2):
        p = torch.empty((N, K * r // 8), dtype=torch.uint8, device="cuda")
        out[f"slice_pack_r{r}"] = per_call(lambda: mq.slice_pack(q, r, packed=p), bytes_slice_pack(N, K, r))
        out[f"gemv_r{r}"] = per_call(lambda: mq.gemv(p, K, r, a, z, x, y=y, flags=mq.GEMV_AUTO | mq.GEMV_PDL), bytes_gemv(N, K, r, 1))
    return out


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
    """The same step from HOST buffers: weights and activations are copied from pinned memory, every y is read back.
    The value is the algorithmic bytes of all stages over the time of the whole end-to-end step."""
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
        for _, fn, _, _ in plan:
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
            "steps": steps, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
            "definition": "algorithmic bytes of ALL stages of the step / time of the step run through the public calls from pinned host "
                          "buffers (weights and activations copied in, every y copied out); PCIe-bound"}


# ----------------------------------------------------------------------------
# the oracle arm (CPU baseline and --impl reference)
# ----------------------------------------------------------------------------

def oracle_step(shapes, W_host, x_host, ref):
    """The same stages, executed by the CPU oracle as it stands.  Returns (seconds, algorithmic bytes, GEMV B = 1 seconds, bytes)."""
    nbytes = 0
    g_s = g_b = 0.0
    t0 = time.perf_counter()
    for (idx, layer, name, N, K), W, x in zip(shapes, W_host, x_host):
        st, q, a, z = ref.quantize(W)
        sp4 = ref.slice_pack(q, 4, want_unpacked=False)
        sp2 = ref.slice_pack(q, 2, extra_precision=True, want_unpacked=False)
        nnz = sp2["ovf_count"]
        x1 = np.ascontiguousarray(x[:1])
        t1 = time.perf_counter()
        ref.gemv(sp4["packed"], K, 4, a, z, x1)
        ref.gemv(sp2["packed"], K, 2, a, z, x1)
        g_s += time.perf_counter() - t1
        g_b += bytes_gemv(N, K, 4, 1) + bytes_gemv(N, K, 2, 1)
        ref.gemv(sp2["packed"], K, 2, a, z, x1, sp2["ovf_row_ptr"], sp2["ovf_col"])
        ref.gemv(sp4["packed"], K, 4, a, z, x)
        ref.gemv(sp2["packed"], K, 2, a, z, x)
        nbytes += (bytes_quantize(N, K) + bytes_slice_pack(N, K, 4) + bytes_slice_pack(N, K, 2, nnz) +
                   bytes_gemv(N, K, 4, 1) + bytes_gemv(N, K, 4, 8) + bytes_gemv(N, K, 2, 1) + bytes_gemv(N, K, 2, 8) +
                   bytes_gemv(N, K, 2, 1, nnz))
    return time.perf_counter() - t0, nbytes, g_s, g_b


def oracle_dense_block(ref, which):
    """The oracle's dense forward on an M = 128 block of the benchmark shape: measured seconds and the linear extrapolation."""
    if which == "cfg4":
        N, K, M_full, rs, flops_full = 14336, 4096, 4096, (8, 4, 2), 3 * 2.0 * 4096 * 14336 * 4096
        W = synth.normal_bf16((N, K), 0.02, synth.seed_for(4, 0))
        X = synth.normal_bf16((128, K), 1.0, synth.seed_for(4, 500))
        t0 = time.perf_counter()
        ref.gemm_multi(ref.SRC_BF16, W, K, X, rs=rs)
    else:
        N, K, M_full, flops_full = 14336, 3584, 2048, 2.0 * 2048 * 14336 * 3584
        q = synth.skewed_codes((N, K), 0.05, 224, synth.seed_for(5, 0))
        sp = ref.slice_pack(q, 2, extra_precision=True, want_unpacked=False)
        X = synth.normal_bf16((128, K), 1.0, synth.seed_for(5, 500))
        a = np.full(N, 1e-3, np.float32); z = np.full(N, 128.0, np.float32)
        t0 = time.perf_counter()
        ref.gemm_multi(ref.SRC_PACKED, sp["packed"], K, X, rs=(2,), alpha=a, zero=z, extra_precision=True,
                       ovf_row_ptr=sp["ovf_row_ptr"], ovf_col=sp["ovf_col"])
    secs = time.perf_counter() - t0
    full = secs * M_full / 128
    return {"measured": f"M = 128 rows of {M_full}", "seconds_measured": round(secs, 2), "seconds_extrapolated_full_M": round(full, 1),
            "TFLOPs_extrapolated": round(flops_full / full / 1e12, 5), "label": "linear extrapolation in M, not a measurement of the full shape"}


def cpu_baseline(shapes, W_host, x_host, sample_layers, dense=True):
    from oracle import ref
    ref.build()
    per_layer = len(synth.WORKLOADS[CONFIG_ID]["layer"])
    k = sample_layers * per_layer
    secs, nbytes, g_s, g_b = oracle_step(shapes[:k], W_host[:k], x_host[:k], ref)
    out = {"value": round(g_b / g_s / 1e9, 3), "unit": "GB/s", "cores": ref.num_threads(), "kind": "oracle",
           "sample": f"first {sample_layers} of {synth.WORKLOADS[CONFIG_ID]['layers']} layers of the same stack, same stages; value = the two B = 1 GEMV "
                     f"stages (r = 4, r = 2), like the GPU line's; {secs:.1f} s of CPU work for the whole sampled step",
           "step_GBps": round(nbytes / secs / 1e9, 3), "seconds": round(secs, 2),
           "threads": "quantize, slice, gemv and the dense forward run OpenMP over rows on all cores; pack / unpack of a plane are single-threaded"}
    if dense:
        out["dense_forward_cfg4"] = oracle_dense_block(ref, "cfg4")
        out["dense_prefill_cfg5"] = oracle_dense_block(ref, "cfg5")
    return out


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
    tot_s = tot_b = g_s = g_b = 0.0
    for _ in range(steps):
        s, b, gs, gb = oracle_step(shapes, W_host, x_host, ref)
        tot_s += s; tot_b += b; g_s += gs; g_b += gb
    v = round(g_b / g_s / 1e9, 3)
    sample = (f"each step = first {sample_layers} layers of the stack, same stages without the dense forward; value = the two B = 1 GEMV "
              "stages (r = 4, r = 2) of the step, as in the GPU line")
    return {"impl": "reference", "metric": METRIC, "value": v, "unit": "GB/s", "n_gpus": args.gpus, "steps": steps,
            "warmup": min(args.warmup, 1), "ms_per_step": round(tot_s / steps * 1e3, 2), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": "configs[1] Gemma-2-2B-shaped MLP decode stack (bounded sample)", "sample": sample},
            "step_GBps": round(tot_b / tot_s / 1e9, 3),
            "cpu_baseline": {"value": v, "unit": "GB/s", "cores": ref.num_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": v, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}


# ----------------------------------------------------------------------------
# launching
# ----------------------------------------------------------------------------

def rank_environments(n: int, port: int):
    """Environment of each of the n ranks that `--gpus n` starts when no launcher has set WORLD_SIZE."""
    return [dict(RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n), LOCAL_WORLD_SIZE=str(n), MASTER_ADDR="127.0.0.1",
                 MASTER_PORT=str(port)) for r in range(n)]


def spawn_ranks(args) -> int:
    """`python bench.py --gpus N` without a launcher: start one process per GPU (rank r on GPU r), NCCL's log left on."""
    port = 29500 + os.getpid() % 2000
    procs = []
    for env in rank_environments(args.gpus, port):
        e = dict(os.environ); e.update(env)
        e.setdefault("NCCL_DEBUG", "WARN")
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__)] + sys.argv[1:], env=e))
    rc = 0
    for p in procs:
        rc = rc or p.wait()
    return rc


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--layers", type=int, default=synth.WORKLOADS[CONFIG_ID]["layers"])
    ap.add_argument("--cpu-sample-layers", type=int, default=6)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--quick", action="store_true", help="the step and its stages only: skip configs[0], [2], [3], [4] and Mix'n'Match")
    ap.add_argument("--print-rank-env", action="store_true", help="print this process's rank variables and exit (launch test)")
    args = ap.parse_args()
    if "WORLD_SIZE" not in os.environ and args.gpus > 1 and args.impl == "cuda":
        sys.exit(spawn_ranks(args))
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.print_rank_env:
        print(json.dumps({k: os.environ.get(k) for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}), flush=True)
        return

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
            out["cpu_baseline"] = cpu_baseline(shapes, W_host, x_host, k, dense=not args.quick)
        print(json.dumps(out), flush=True)


if __name__ == "__main__":
    main()
