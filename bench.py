#!/usr/bin/env python
"""Benchmark of the Quaff quantized linear layer hot path (forward + backward) on B200.

A step is one pass of the whole path - momentum scale update, outlier weight-row re-quantization,
activation scaling + quantization, INT8 forward GEMM with fused dequantization and LoRA, and the
backward (grad-input through the dequantized INT8 weight, LoRA gradients) - over one batch of
synthetic tokens through every linear layer of the workload.  Default workload: the LLaMA-2-7B-shaped decoder
block (8192 tokens; q/k/v/o 4096->4096, gate/up 4096->11008, down 11008->4096; 0.5 % outlier channels; LoRA r=64),
the largest configuration that is timed on one GPU.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]
    python bench.py --workload sweep          # the shape sweep: one JSON line with a table of 324 points

Prints ONE JSON line (rank 0).  The timed region (`--steps` steps between two CUDA events) is repeated `--repeats`
times; `ms_per_step` is the median over the repeats.  `--impl reference` times the CPU oracle on a bounded token sample.
"""
import argparse
import dataclasses
import hashlib
import json
import os
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2505_14742_b200 import synth  # noqa: E402

METRIC = "qlinear fwd+bwd tokens/s"
UNIT = "tokens/s"
REPLICAS = 3  # rotating buffer sets, so that every step starts from cold HBM data


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with one `nvidia-smi -lms` process while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index, period_ms=20):
        self.index = index
        self.period_ms = period_ms
        self.rows = []
        self.proc = None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", str(self.period_ms)],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            time.sleep(0.25)          # let the sampler start before the timed region
        except Exception:
            self.proc = None
        return self

    def __exit__(self, *a):
        if self.proc is None:
            return
        time.sleep(0.05)
        self.proc.terminate()          # the exact process started above
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        for line in out.strip().splitlines():
            self.rows.append([c.strip() for c in line.split(",")])

    def summary(self):
        sm, mx, power, reasons = [], [], [], set()
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1])); power.append(float(r[2]))
            except Exception:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        # samples taken while the GPU was working: the upper half by power draw
        busy = [c for c, p in zip(sm, power) if power and p >= 0.5 * (min(power) + max(power))] or sm
        return {"sm_mhz": float(np.median(busy)) if busy else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm), "power_w_max": max(power) if power else None}


def layer_ops(M, sp, nOp):
    """Algorithmic work of one layer-step: INT8 ops of the forward GEMMs (Eq. 9: main and outlier contraction), bf16
    flops of the LoRA up-projection, bf16 flops of the grad-input GEMM (through the weight, the outlier rows, G A^T)."""
    fwd_int8 = 2.0 * M * sp.N * (sp.K + nOp)
    fwd_lora = 2.0 * M * sp.N * sp.r
    bwd_bf16 = 2.0 * M * sp.N * sp.K + 2.0 * M * sp.N * nOp + 2.0 * M * sp.K * sp.r
    return fwd_int8, fwd_lora, bwd_bf16


def kernel_source_hash():
    """Hash of the CUDA sources: DRAM traffic figures taken with ncu are only valid for the sources they were taken on."""
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2505_14742_b200", "csrc")
    for name in sorted(os.listdir(csrc)):
        if name.endswith((".cu", ".cuh")):
            h.update(open(os.path.join(csrc, name), "rb").read())
    return h.hexdigest()[:16]


def ncu_traffic_table():
    """profiles/dram_traffic.txt: lines `kind M K N nO r bytes_per_launch source_hash` copied from ncu captures
    (dram__bytes_read.sum + dram__bytes_write.sum).  Entries taken on other sources than the present ones are dropped."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.txt")
    table = {}
    if not os.path.exists(path):
        return table
    now = kernel_source_hash()
    for line in open(path):
        f = line.split()
        if len(f) != 8 or line.startswith("#"):
            continue
        if f[7] == now:
            table[(f[0],) + tuple(int(v) for v in f[1:6])] = float(f[6])
    return table


# --------------------------------------------------------------------------------------- CPU oracle legs
def oracle_sample_step(wl, sample_tokens, lins, state):
    """One fwd+bwd of the oracle over `sample_tokens` tokens through every layer; returns seconds."""
    import oracle
    t0 = time.perf_counter()
    for li, lin in enumerate(lins):
        sp = lin.spec
        st = state[li]
        X, dY = st["X"], st["dY"]
        nOp = synth.pad_to(sp.nO, 32)
        scale = wl.lora_alpha / sp.r
        st["s"], _, _ = oracle.momentum_update(X, lin.O_idx, st["wmax"], wl.gamma, st["s"])
        wq, dw = oracle.requant_weight_rows(st["W_O"], st["s"], nOp)
        Xq, xqo, dx = oracle.quant_act(X, lin.O_idx, st["s"], nOp)
        Y, T, _, _ = oracle.qlinear_fwd(Xq, xqo, dx, st["Wq"], st["dW"], wq, dw, X, lin.A, lin.B, scale)
        oracle.qlinear_bwd(dY, st["Wq"], st["dW"], wq, dw, lin.O_idx, st["s"], X, T, lin.A, lin.B, scale)
    return time.perf_counter() - t0


def oracle_setup(wl, sample_tokens):
    import oracle
    oracle.build()
    lins = [synth.layer_inputs(wl, li, b_std=0.02) for li in range(len(wl.layers))]
    state = []
    small = dataclasses.replace(wl, M=sample_tokens)      # the same workload with a batch of `sample_tokens` tokens
    for li, lin in enumerate(lins):
        Wq, dW, W_O, wmax = oracle.prepare_weight(lin.W, lin.O_idx)
        X, dY = synth.step_inputs(small, li, 0, lin)
        state.append({"Wq": Wq, "dW": dW, "W_O": W_O, "wmax": wmax, "s": np.ones(lin.spec.nO, np.float32), "X": X, "dY": dY})
    return lins, state


def cpu_baseline(wl, sample_tokens=16, reps=1):
    import oracle
    lins, state = oracle_setup(wl, sample_tokens)
    best = min(oracle_sample_step(wl, sample_tokens, lins, state) for _ in range(reps))
    return {"value": sample_tokens / best, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"{sample_tokens} of {wl.M} tokens through all {len(wl.layers)} layers, fwd+bwd; best of {reps} runs, {best:.2f} s each"}


def run_reference(args, wl):
    """--impl reference: the CPU oracle, as it stands, on the host cores (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import oracle
    sample = args.sample_tokens
    lins, state = oracle_setup(wl, sample)
    for _ in range(args.warmup):
        oracle_sample_step(wl, sample, lins, state)
    times = [oracle_sample_step(wl, sample, lins, state) for _ in range(args.steps)]
    ms = 1e3 * float(np.mean(times))
    value = sample / (ms / 1e3)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "int8 forward (int64 accumulate), f64 backward", "data": "synthetic",
            "config": {"workload": wl.name, "tokens": wl.M, "sample_tokens_per_step": sample,
                       "layers": [f"{l.name} {l.K}->{l.N}" for l in wl.layers]},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                             "sample": f"{sample} of {wl.M} tokens per step through all layers, fwd+bwd"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------------------- GPU arm
def run_gpu(args, wl):
    import torch
    import torch.distributed as dist
    from paper_2505_14742_b200 import binding as Q, build, dist as qdist
    from paper_2505_14742_b200.layer import QuaffLinear

    rank, world, local = qdist.rank_world()
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        build.build_library()
    if world > 1:
        dist.barrier()
    Q.lib()  # raises when the CUDA library is missing: there is no fallback path

    def to_bf16(bits):
        return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)

    # Each rank owns its own batch of tokens (weak scaling, no data-path collective): rank-specific seed offset.
    M = wl.M
    nl = len(wl.layers)
    lins = [synth.layer_inputs(wl, li, b_std=0.02) for li in range(nl)]
    sets = []  # REPLICAS x layers
    host_in = []
    for rep in range(REPLICAS):
        layers, xs, dys, hx, hdy = [], [], [], [], []
        for li, lin in enumerate(lins):
            sp = lin.spec
            layer = QuaffLinear(to_bf16(lin.W), torch.from_numpy(lin.O_idx).cuda(), to_bf16(lin.A), to_bf16(lin.B),
                                wl.lora_alpha / sp.r, wl.gamma, M, int8_grad=args.int8_grad, lean_bwd=args.lean_bwd)
            X, dY = synth.step_inputs(wl, li, qdist.batch_index(rep, rank), lin)
            layers.append(layer)
            xs.append(to_bf16(X)); dys.append(to_bf16(dY))
            hx.append(torch.from_numpy(X.view(np.int16)).pin_memory()); hdy.append(torch.from_numpy(dY.view(np.int16)).pin_memory())
        sets.append((layers, xs, dys))
        host_in.append((hx, hdy))
    torch.cuda.synchronize()

    from paper_2505_14742_b200.layer import StepGraph

    def step(i, timing=None):
        layers, xs, dys = sets[i % REPLICAS]
        for li in range(nl):
            if timing is not None:
                ev = timing[i % REPLICAS][li]
                Q.quaff_debug_time_gemm(0, ev[0], ev[1])
                Q.quaff_debug_time_gemm(1, ev[2], ev[3])
            layers[li].forward(xs[li])
            layers[li].backward(dys[li])

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    for i in range(args.warmup):
        step(i)
    sync_all()

    # One pair of CUDA events around each tensor-core GEMM of each buffer set (torch creates the event lazily
    # at its first record(): materialise every handle now).  In graph mode they are recorded by the graph.
    timing = [[[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(nl)] for _ in range(REPLICAS)]
    for per_set in timing:
        for evs in per_set:
            for e in evs:
                e.record()
    # ---- the step as a CUDA graph per buffer set (default), or enqueued launch by launch (--eager)
    # Two versions of the step: the plain one is what the timed region runs; the instrumented one carries a CUDA
    # event pair around each tensor-core GEMM (as event-record nodes of the graph).  Those nodes turn the programmatic
    # dependencies around the GEMMs into full ones and cost the step some 50 us, so the GEMM durations for the
    # roofline come from a second pass over the same steps, directly after the timed region.
    launches0 = Q.quaff_debug_launch_count()
    if args.eager:
        step(0)
        run_step = lambda i: step(i)
        run_step_timed = lambda i: step(i, timing)
    else:
        graphs = [StepGraph(lambda rep=rep: step(rep)) for rep in range(REPLICAS)]
        run_step = lambda i: graphs[i % REPLICAS].replay()
    launches_per_step = (Q.quaff_debug_launch_count() - launches0) // (1 if args.eager else REPLICAS)
    if not args.eager:
        graphs_timed = [StepGraph(lambda rep=rep: step(rep, timing)) for rep in range(REPLICAS)]
        run_step_timed = lambda i: graphs_timed[i % REPLICAS].replay()
    for i in range(REPLICAS):
        run_step(i)
    sync_all()
    for layers, _, _ in sets:
        for l in layers:
            assert int(l.status[0].item()) == 0, "device-side wait timed out"

    # ---- device-resident timed region: `steps` steps between two events, repeated; the median repeat counts
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    region_ms = []
    with ClockSampler(local, period_ms=10) as clocks:
        for rep in range(args.repeats):
            sync_all()
            e0.record()
            for i in range(args.steps):
                run_step(i)
            e1.record()
            sync_all()
            region_ms.append(qdist.max_over_ranks(e0.elapsed_time(e1), "cuda"))
    launches = launches_per_step * args.steps
    ms_per_step = float(np.median(region_ms)) / args.steps
    # ---- the same steps once more with the event pairs: GEMM durations of the latest step on each buffer set
    inst_steps = max(REPLICAS, min(args.steps, 200))
    sync_all()
    e0.record()
    for i in range(inst_steps):
        run_step_timed(i)
    e1.record()
    sync_all()
    inst_ms_per_step = e0.elapsed_time(e1) / inst_steps
    gemm_ms = [[float(np.mean([timing[rep][li][a].elapsed_time(timing[rep][li][a + 1]) for rep in range(REPLICAS)]))
                for a in (0, 2)] for li in range(nl)]

    # ---- end to end: host buffers in, host buffers out, copies inside the timed region
    h_out = []
    for li, lin in enumerate(lins):
        sp = lin.spec
        h_out.append((torch.empty((M, sp.N), dtype=torch.bfloat16).pin_memory(), torch.empty((M, sp.K), dtype=torch.bfloat16).pin_memory()))
    h2d = sum(M * (sp.K + sp.N) * 2 for sp in wl.layers)
    d2h = sum(M * (sp.N + sp.K) * 2 for sp in wl.layers)

    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()     # upload and download beside the compute stream

    def step_e2e(i):
        """Host buffers in, host buffers out: the uploads of layer l+1 and the downloads of layer l-1 run
        (on their own streams, both copy engines) while layer l computes; everything is joined at the end."""
        layers, xs, dys = sets[i % REPLICAS]
        hx, hdy = host_in[i % REPLICAS]
        main = torch.cuda.current_stream()
        s_in.wait_stream(main)
        s_out.wait_stream(main)
        for li in range(nl):
            with torch.cuda.stream(s_in):
                xs[li].view(torch.int16).copy_(hx[li], non_blocking=True)
                dys[li].view(torch.int16).copy_(hdy[li], non_blocking=True)
                uploaded = torch.cuda.Event()
                uploaded.record(s_in)
            main.wait_event(uploaded)
            Y = layers[li].forward(xs[li])
            dX, _, _ = layers[li].backward(dys[li])
            computed = torch.cuda.Event()
            computed.record(main)
            with torch.cuda.stream(s_out):
                s_out.wait_event(computed)
                h_out[li][0].copy_(Y, non_blocking=True)
                h_out[li][1].copy_(dX, non_blocking=True)
        main.wait_stream(s_in)
        main.wait_stream(s_out)

    e2e_steps = max(3, min(args.steps, 60))
    for i in range(2):
        step_e2e(i)
    sync_all()
    if args.eager:
        run_e2e = step_e2e
    else:
        e2e_graphs = [StepGraph(lambda rep=rep: step_e2e(rep)) for rep in range(REPLICAS)]
        run_e2e = lambda i: e2e_graphs[i % REPLICAS].replay()
        for i in range(REPLICAS):
            run_e2e(i)
    sync_all()
    # the buffer sets are independent, so consecutive steps go to one stream per set: the uploads of the next
    # step run while this one computes and the previous one downloads (a pipelined loader)
    pipes = [torch.cuda.Stream() for _ in range(REPLICAS)]
    main = torch.cuda.current_stream()
    e0.record()
    for ps in pipes:
        ps.wait_stream(main)
    for i in range(e2e_steps):
        with torch.cuda.stream(pipes[i % REPLICAS]):
            run_e2e(i)
    for ps in pipes:
        main.wait_stream(ps)
    e1.record()
    sync_all()
    e2e_ms = qdist.max_over_ranks(e0.elapsed_time(e1), "cuda") / e2e_steps

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- per-kernel figures and the roofline of the dominant kernel
    peaks = load_peaks()
    # The HBM-bound kernels of every layer, each alone on the layer's own buffers: one launch between two events, L2
    # flushed before it (the launch latency is inside the figure, which is what bounds the small shapes).
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    hbm_kernels = []
    layers0, xs0, _ = sets[0]

    def alone_ms(fn):
        ts = []
        for i in range(13):
            flush.sum()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(); fn(); b.record()
            torch.cuda.synchronize()
            if i >= 3:
                ts.append(a.elapsed_time(b))
        return float(np.median(ts))

    one = torch.zeros(1, device="cuda")
    launch_floor_ms = alone_ms(lambda: one.zero_())      # the same bracket around a one-element fill: what no kernel can go below
    for li, sp in enumerate(wl.layers):
        l = layers0[li]
        nOp = synth.pad_to(sp.nO, 32)
        cases = [("quant_act", lambda l=l, li=li: Q.quaff_quant_act(xs0[li], l.O_idx, l.s_O, l.Xq, l.xq_O, l.dx),
                  M * sp.K * 3 + M * nOp + 4 * M)]
        if sp.nO:
            cases.append(("momentum", lambda l=l, li=li: Q.quaff_momentum_update(xs0[li], l.O_idx, l.wmax_O, l.gamma, l.s_O, l.ws, l.colmax_O, l.beta_O),
                          32 * M * sp.nO))
            cases.append(("requant_rows", lambda l=l: Q.quaff_requant_weight_rows(l.W_O, l.s_O, l.wq_O, l.dw_O),
                          2 * sp.nO * sp.N + nOp * sp.N + 4 * sp.N))
        for kname, fn, nbytes in cases:
            kms = alone_ms(fn)
            gbs = nbytes / (kms * 1e-3) / 1e9
            entry = {"layer": sp.name, "kernel": kname, "ms": kms, "algorithmic_bytes": nbytes, "gbs": gbs,
                     "frac_of_hbm_peak": gbs / peaks["hbm_gbs"]}
            if kname == "quant_act" and REPLICAS * nbytes > 2 * 126e6:
                # the same kernel back to back over the buffer sets (together larger than L2): the launch latency of a launch
                # overlaps the launch before it, as it does inside a step
                def b2b(li=li):
                    for layers_r, xs_r, _ in sets:
                        lr = layers_r[li]
                        Q.quaff_quant_act(xs_r[li], lr.O_idx, lr.s_O, lr.Xq, lr.xq_O, lr.dx)
                ts = []
                for i in range(8):
                    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    a.record()
                    for _ in range(4):
                        b2b()
                    b.record()
                    torch.cuda.synchronize()
                    if i >= 2:
                        ts.append(a.elapsed_time(b) / (4 * REPLICAS))
                bms = float(np.median(ts))
                entry["back_to_back"] = {"ms": bms, "gbs": nbytes / (bms * 1e-3) / 1e9, "frac_of_hbm_peak": nbytes / (bms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                         "launches_per_event_pair": 4 * REPLICAS}
            hbm_kernels.append(entry)
    ncu_traffic = ncu_traffic_table()
    timed_total_ms = float(np.sum(region_ms))
    sustained = timed_total_ms > 1000.0       # a region longer than a second runs under the power cap
    bf16_peak = peaks["bf16_tflops_sustained"] if sustained else peaks["bf16_tflops"]
    peak_note = f"{peaks['source']} cuBLAS bf16 {'sustained' if sustained else 'burst'}"
    per_layer = []
    dominant = None
    # the grad-input GEMM runs in bf16 (the paper quantizes no gradient); with --int8-grad it is the INT8 variant's kernel
    bwd_peak = bf16_peak * (2.0 if args.int8_grad else 1.0)
    bwd_unit = "TOP/s" if args.int8_grad else "TFLOP/s"
    for li, sp in enumerate(wl.layers):
        nOp = synth.pad_to(sp.nO, 32)
        f_ms, b_ms = gemm_ms[li]
        fwd_int8, fwd_lora, bwd_bf16 = layer_ops(M, sp, nOp)
        f_tops, b_tflops = (fwd_int8 + fwd_lora) / (f_ms * 1e-3) / 1e12, bwd_bf16 / (b_ms * 1e-3) / 1e12
        entry = {"layer": sp.name, "K": sp.K, "N": sp.N, "nO": sp.nO, "r": sp.r,
                 "fwd_gemm_ms": f_ms, "fwd_int8_tops": fwd_int8 / (f_ms * 1e-3) / 1e12,
                 "fwd_pct_of_int8_nominal_4500": 100.0 * fwd_int8 / (f_ms * 1e-3) / 4.5e15,
                 "fwd_roofline": {"bound": "tensor", "achieved": f_tops, "peak": 2.0 * bf16_peak, "unit": "TOP/s", "frac": f_tops / (2.0 * bf16_peak),
                                  "traffic": ncu_traffic.get(("fwd_int8_gemm", M, sp.K, sp.N, sp.nO, sp.r))},
                 "bwd_gemm_ms": b_ms, "bwd_bf16_tflops": b_tflops,
                 "bwd_pct_of_bf16_nominal_2250": 100.0 * b_tflops / 2.25e3,
                 "bwd_pct_of_int8_nominal_4500": 100.0 * b_tflops / 4.5e3,
                 "bwd_roofline": {"bound": "tensor", "achieved": b_tflops, "peak": bwd_peak, "unit": bwd_unit, "frac": b_tflops / bwd_peak,
                                  "traffic": ncu_traffic.get(("bwd_bf16_gemm", M, sp.K, sp.N, sp.nO, sp.r))}}
        per_layer.append(entry)
        for kind, ms, work in (("fwd_int8_gemm", f_ms, fwd_int8 + fwd_lora), ("bwd_bf16_gemm", b_ms, bwd_bf16)):
            if dominant is None or ms > dominant[2]:
                dominant = (sp.name, kind, ms, work, ncu_traffic.get((kind, M, sp.K, sp.N, sp.nO, sp.r)))
    name, kind, ms, work, traffic = dominant
    achieved = work / (ms * 1e-3) / 1e12
    int8_kernel = kind == "fwd_int8_gemm" or args.int8_grad
    peak = bf16_peak * (2.0 if int8_kernel else 1.0)
    kname = ("forward INT8 GEMM (Eq. 9 + LoRA)" if kind == "fwd_int8_gemm" else
             "INT8 grad-input GEMM (variant, not the paper's method)" if args.int8_grad else "umma_gemm_kernel<EPI_BWD> grad-input GEMM")
    roofline = {"bound": "tensor", "kernel": f"{kname} ({name})",
                "achieved": achieved, "peak": peak, "unit": "TOP/s" if int8_kernel else "TFLOP/s",
                "frac": achieved / peak, "traffic": traffic,
                "peak_source": peak_note + (" x2 (nominal int8:bf16 ratio)" if int8_kernel else "")
                               + f"; the timed region ran {timed_total_ms:.0f} ms",
                "avg_launch_ms": ms,
                "timing": f"CUDA event pair around the kernel in an instrumented pass over the same steps ({inst_steps} steps, "
                          f"{inst_ms_per_step:.4f} ms per step with the event nodes in the graph)"}
    if kind == "bwd_bf16_gemm" and not args.int8_grad:
        # Inside the step the grad-input GEMM shares the SMs: the split-K GEMMs of dA and dB are scheduled into the SMs
        # its last wave leaves idle, which shortens the step and lengthens the GEMM.  The same kernel alone (a backward
        # call for dX only on the same layer's buffers, L2 flushed before it) is reported beside it.
        li = [sp.name for sp in wl.layers].index(name)
        l = layers0[li]
        dY0 = sets[0][2][li]
        def gemm_alone():
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(); b.record()
            Q.quaff_debug_time_gemm(1, a, b)
            Q.quaff_qlinear_bwd(dY0, l.Wq, l.dW, l.wq_O, l.dw_O, l.O_idx, l.s_O, l._X, l.T, l.A, l.B, l.lora_scale, l.dX, None, None,
                                False, l.ws, l.status)
            torch.cuda.synchronize()
            return a.elapsed_time(b)
        ts = []
        for i in range(13):
            flush.sum()
            t_ms = gemm_alone()
            if i >= 3:
                ts.append(t_ms)
        alone_ms_ = float(np.median(ts))
        roofline["alone"] = {"avg_launch_ms": alone_ms_, "achieved": work / (alone_ms_ * 1e-3) / 1e12,
                             "frac": work / (alone_ms_ * 1e-3) / 1e12 / peaks["bf16_tflops"],
                             "note": "the same kernel without the LoRA-gradient GEMMs beside it (backward for dX only, L2 flushed), "
                                     "against the burst peak"}

    # the oracle on the host cores: a single-GPU run only (with more ranks every GPU of the job would be held meanwhile)
    cpu = cpu_baseline(wl, min(wl.M, 8 * args.sample_tokens), reps=2) if (world == 1 and not args.no_cpu_baseline) else None
    line = {"metric": METRIC, "value": qdist.whole_job_rate(M, world, ms_per_step), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "repeats": {"n": args.repeats, "ms_per_step_min": float(np.min(region_ms)) / args.steps,
                        "ms_per_step_max": float(np.max(region_ms)) / args.steps, "ms_per_step_median": ms_per_step},
            "vs_baseline": None, "dtype": "int8 forward (int32 accumulate), " + ("int8 grad-input (variant)" if args.int8_grad else "bf16 backward (f32 accumulate)"),
            "data": "synthetic",
            "config": {"workload": wl.name, "tokens_per_gpu": M,
                       "backward": "INT8 grad-input variant (NOT the paper's method; reported separately)" if args.int8_grad
                                   else ("bf16 grad-input, INT8 codes expanded inside the GEMM (no copy of the weight)" if args.lean_bwd
                                         else "bf16 grad-input through a transient bf16 copy of the INT8 weight (the paper quantizes no gradient)"),
                       "layers": [f"{l.name} {l.K}->{l.N} nO={l.nO} r={l.r}" for l in wl.layers], "gamma": wl.gamma,
                       "l2": f"rotating {REPLICAS} full buffer sets (weights, activations, outputs); one set alone exceeds the 126 MB L2",
                       "launch": "eager" if args.eager else "one CUDA graph replay per step"},
            "clocks": clocks.summary(),
            "e2e": {"value": qdist.whole_job_rate(M, world, e2e_ms), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "ms_per_step": e2e_ms, "steps": e2e_steps},
            "gpu_launches": int(launches),
            "roofline": roofline, "layers": per_layer, "hbm_kernels": {"timing": "each kernel alone on the layer's buffers, one launch between two events, L2 flushed before it; "
                                      "launch_floor_ms is the same bracket around a one-element fill",
                            "launch_floor_ms": launch_floor_ms, "hbm_peak_gbs": peaks["hbm_gbs"], "kernels": hbm_kernels},
            "cpu_baseline": cpu}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_micro(args):
    """--micro NAME: one HBM-bound kernel alone on rows of a given shape, L2 flushed (read-only sweep of a
    512 MB buffer) before every launch, CUDA events around each launch; prints its own JSON line.  Used for
    the per-kernel rooflines and as the small command of the ncu captures."""
    import torch
    from paper_2505_14742_b200 import binding as Q, build
    build.build_library()
    Q.lib()
    torch.cuda.set_device(0)
    M, K, N, nO = args.micro_shape
    nOp = synth.pad_to(nO, 32)
    g = torch.Generator(device="cuda").manual_seed(1234)
    X = torch.randn((M, K), device="cuda", generator=g).to(torch.bfloat16)
    O = torch.sort(torch.randperm(K, device="cuda", generator=g)[:nO])[0].to(torch.int32)
    X[:, O.long()] *= 50.0
    s = 1.0 + 10.0 * torch.rand(nO, device="cuda", generator=g)
    flush = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")
    if args.micro in ("fwd", "bwd", "bwd8"):
        # one layer's forward (or backward) call on random codes; the tensor-core GEMM inside it is timed by the
        # library's event pair (quaff_debug_time_gemm), everything else of the call runs untimed around it
        r = args.micro_rank
        i8 = lambda *shape: torch.randint(-127, 128, shape, dtype=torch.int8, device="cuda", generator=g)
        Xq, Wq, xqo, wqo = i8(M, K), i8(N, K), i8(M, nOp), i8(N, nOp)
        dxv, dWv, dwOv = (torch.rand(n, device="cuda", generator=g) * 1e-2 for n in (M, N, N))
        A = (0.02 * torch.randn((K, r), device="cuda", generator=g)).to(torch.bfloat16)
        B = (0.02 * torch.randn((r, N), device="cuda", generator=g)).to(torch.bfloat16)
        T = torch.empty((M, r), dtype=torch.bfloat16, device="cuda")
        Y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
        dY = (0.01 * torch.randn((M, N), device="cuda", generator=g)).to(torch.bfloat16)
        dX = torch.empty((M, K), dtype=torch.bfloat16, device="cuda")
        dA = torch.zeros((K, r), device="cuda"); dB = torch.zeros((r, N), device="cuda")
        st = torch.zeros(4, dtype=torch.int32, device="cuda")
        ws = torch.empty(max(Q.workspace_bytes(Q.QUAFF_WS_FWD, M, K, N, nOp, r),
                             Q.workspace_bytes(Q.QUAFF_WS_BWD_INT8 if args.micro == "bwd8" else
                                               (Q.QUAFF_WS_BWD_LEAN if args.lean_bwd else Q.QUAFF_WS_BWD), M, K, N, nOp, r)),
                         dtype=torch.uint8, device="cuda")
        Q.quaff_qlinear_fwd(Xq, xqo, dxv, Wq, dWv, wqo, dwOv, X, A, B, 1.0, T, Y, ws, None, None, st)
        which = 0 if args.micro == "fwd" else 1
        times = []
        for i in range(args.warmup + args.steps):
            flush.sum()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); e1.record()
            Q.quaff_debug_time_gemm(which, e0, e1)
            if which == 0:
                Q.quaff_qlinear_fwd(Xq, xqo, dxv, Wq, dWv, wqo, dwOv, X, A, B, 1.0, T, Y, ws, None, None, st)
            elif args.micro == "bwd8":   # the INT8 grad-input variant (not the paper's method): its INT8 GEMM is the timed kernel
                Q.quaff_qlinear_bwd_int8(dY, Wq, dWv, wqo, dwOv, O, s, X, T, A, B, 1.0, dX, None, None, False, ws, st)
            else:
                # (dX only: with dA / dB the library schedules their split-K GEMMs into the SMs the grad-input GEMM leaves idle)
                Q.quaff_qlinear_bwd(dY, Wq, dWv, wqo, dwOv, O, s, X, T, A, B, 1.0, dX, None, None, False, ws, st)
            torch.cuda.synchronize()
            if i >= args.warmup:
                times.append(e0.elapsed_time(e1))
        assert int(st[0].item()) == 0, "device-side wait timed out"
        ms = float(np.median(times))
        peaks = load_peaks()
        work = 2.0 * M * N * (K + nOp + r) if which == 0 else 2.0 * M * N * (K + nOp) + 2.0 * M * K * r
        int8 = which == 0 or args.micro == "bwd8"
        peak = peaks["bf16_tflops"] * (2.0 if int8 else 1.0)
        print(json.dumps({"micro": args.micro, "shape": {"M": M, "K": K, "N": N, "nO": nO, "r": r}, "ms_per_launch": ms, "launches": len(times),
                          "roofline": {"bound": "tensor", "achieved": work / (ms * 1e-3) / 1e12, "peak": peak,
                                       "unit": "TOP/s" if int8 else "TFLOP/s", "frac": work / (ms * 1e-3) / 1e12 / peak,
                                       "peak_source": f"{peaks['source']} cuBLAS bf16 burst" + (" x2 (nominal int8:bf16 ratio)" if int8 else "")}}),
              flush=True)
        return
    # R rotating buffer sets, together at least 2.5 times the 126 MB L2, so that back-to-back launches read HBM
    nbytes_qa = M * K * 3 + M * nOp + 4 * M
    R = max(2, int(np.ceil(2.5 * 126e6 / max(nbytes_qa, 1))))
    fns = []
    if args.micro == "quant_act":
        for i in range(R):
            Xi = X if i == 0 else X.clone()
            Xq = torch.empty((M, K), dtype=torch.int8, device="cuda")
            xqo = torch.empty((M, nOp), dtype=torch.int8, device="cuda")
            dx = torch.empty(M, device="cuda")
            fns.append(lambda Xi=Xi, Xq=Xq, xqo=xqo, dx=dx: Q.quaff_quant_act(Xi, O, s, Xq, xqo, dx))
        nbytes = nbytes_qa
    elif args.micro == "quant_grad":
        dWv = torch.rand(K, device="cuda", generator=g) * 1e-3 + 1e-5
        for i in range(R):
            Xi = X if i == 0 else X.clone()
            Zq = torch.empty((M, K), dtype=torch.int8, device="cuda")
            dz = torch.empty(M, device="cuda")
            fns.append(lambda Xi=Xi, Zq=Zq, dz=dz: Q.quaff_quant_grad(Xi, dWv, Zq, dz))
        nbytes = M * K * 3 + 4 * M + 4 * K
    elif args.micro == "outlier_count":
        xi = torch.zeros(K, dtype=torch.int32, device="cuda")
        ws = torch.empty(Q.workspace_bytes(Q.QUAFF_WS_CALIBRATE, M, K, 0, 0, 0), dtype=torch.uint8, device="cuda")
        fns.append(lambda: Q.quaff_outlier_count(X, 100, xi, ws))
        nbytes = 2 * M * K              # one pass over the sample
    elif args.micro == "lora_down":
        r = 64
        A = (0.02 * torch.randn((K, r), device="cuda", generator=g)).to(torch.bfloat16)
        T = torch.empty((M, r), dtype=torch.bfloat16, device="cuda")
        st = torch.zeros(4, dtype=torch.int32, device="cuda")
        ws = torch.empty(Q.workspace_bytes(Q.QUAFF_WS_FWD, M, K, N, nOp, r), dtype=torch.uint8, device="cuda")
        fns.append(lambda: Q.quaff_lora_down(X, A, T, ws, st))
        nbytes = 2 * M * K + 2 * K * r + 2 * M * r
    elif args.micro == "momentum":
        wmax = 0.05 + 0.05 * torch.rand(nO, device="cuda", generator=g)
        ws = torch.empty(Q.workspace_bytes(Q.QUAFF_WS_MOMENTUM, M, K, N, nOp, 0), dtype=torch.uint8, device="cuda")
        fns.append(lambda: Q.quaff_momentum_update(X, O, wmax, 0.2, s, ws))
        nbytes = 32 * M * nO            # one 32-byte sector per gathered element
    else:
        W_O = (0.02 * torch.randn((nO, N), device="cuda", generator=g)).to(torch.bfloat16)
        wq = torch.empty((N, nOp), dtype=torch.int8, device="cuda")
        dw = torch.empty(N, device="cuda")
        fns.append(lambda: Q.quaff_requant_weight_rows(W_O, s, wq, dw))
        nbytes = 2 * nO * N + nOp * N + 4 * N
    fn = fns[0]
    times = []
    for i in range(args.warmup + args.steps):
        flush.sum()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); fn(); e1.record()
        torch.cuda.synchronize()
        if i >= args.warmup:
            times.append(e0.elapsed_time(e1))
    ms = float(np.median(times))
    peaks = load_peaks()
    gbs = nbytes / (ms * 1e-3) / 1e9
    line = {"micro": args.micro, "shape": {"M": M, "K": K, "N": N, "nO": nO}, "ms_per_launch": ms, "launches": len(times),
            "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": gbs / peaks["hbm_gbs"], "algorithmic_bytes": nbytes,
                         "peak_source": f"{peaks['source']} copy bandwidth",
                         "timing": "one launch between two CUDA events, L2 flushed before it: the figure contains the launch latency "
                                   "(about 6 us on this machine; the event clock ticks every 2 us)"}}
    if len(fns) > 1:
        # the same kernel back to back over R buffer sets (every launch reads and writes memory that has left L2): the launch
        # latency of a launch overlaps the one before, as it does inside a step
        rounds = 6
        bt = []
        for i in range(args.warmup + args.steps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(rounds):
                for f in fns:
                    f()
            e1.record()
            torch.cuda.synchronize()
            if i >= args.warmup:
                bt.append(e0.elapsed_time(e1) / (rounds * len(fns)))
        bms = float(np.median(bt))
        bg = nbytes / (bms * 1e-3) / 1e9
        line["back_to_back"] = {"ms_per_launch": bms, "achieved": bg, "frac": bg / peaks["hbm_gbs"], "buffer_sets": len(fns),
                                "launches_per_event_pair": rounds * len(fns),
                                "timing": f"{rounds * len(fns)} launches between two events over {len(fns)} rotating buffer sets "
                                          f"({len(fns) * nbytes / 1e6:.0f} MB, more than the L2 holds)"}
    print(json.dumps(line), flush=True)


def run_sweep(args):
    """--workload sweep: one quantized linear layer, forward + backward, over the shape sweep - tokens M in {512, 2048,
    8192, 32768}, K and N in {2048, 4096, 8192}, LoRA rank in {8, 32, 64}, outlier fraction in {0.5 %, 1 %, 5 %} of K -
    324 points, 1 warm-up + 20 timed steps each (one CUDA graph replay per step, CUDA events around the 20).  Inputs
    are drawn on the device (N(0,1) activations with nO seeded channels at 20-100x, N(0, 0.02) weight and LoRA factors):
    this mode only times; parity at sweep points is the tests' business.  One JSON line with the table."""
    import torch
    from paper_2505_14742_b200 import binding as Q, build
    from paper_2505_14742_b200.layer import QuaffLinear, StepGraph
    build.build_library()
    Q.lib()
    torch.cuda.set_device(0)
    peaks = load_peaks()
    g = torch.Generator(device="cuda").manual_seed(synth.BASE_SEED + 4)
    Ms = (512, 2048, 8192, 32768) if not args.sweep_quick else (512, 8192)
    KN = (2048, 4096, 8192) if not args.sweep_quick else (2048, 8192)
    ranks, fracs, steps = (8, 32, 64), (0.005, 0.01, 0.05), 20
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    points = []
    launches = 0
    with ClockSampler(0, period_ms=50) as clocks:
        for K in KN:
            for N in KN:
                W = (0.02 * torch.randn((N, K), device="cuda", generator=g)).to(torch.bfloat16)
                for frac in fracs:
                    nO = max(1, int(round(frac * K)))
                    nOp = synth.pad_to(nO, 32)
                    O = torch.sort(torch.randperm(K, device="cuda", generator=g)[:nO])[0].to(torch.int32)
                    mag = 20.0 + 80.0 * torch.rand(nO, device="cuda", generator=g)
                    for r in ranks:
                        A = (0.02 * torch.randn((K, r), device="cuda", generator=g)).to(torch.bfloat16)
                        B = (0.02 * torch.randn((r, N), device="cuda", generator=g)).to(torch.bfloat16)
                        for M in Ms:
                            layer = QuaffLinear(W, O, A, B, 1.0, 0.2, M)
                            X = torch.randn((M, K), device="cuda", generator=g)
                            X[:, O.long()] *= mag
                            X = X.to(torch.bfloat16)
                            dY = (0.01 * torch.randn((M, N), device="cuda", generator=g)).to(torch.bfloat16)

                            def body():
                                layer.forward(X)
                                layer.backward(dY)

                            n0 = Q.quaff_debug_launch_count()
                            body()                                        # warm-up step (also sets function attributes)
                            per_step = Q.quaff_debug_launch_count() - n0
                            torch.cuda.synchronize()
                            graph = StepGraph(body)
                            flush.zero_()                                 # the first timed step starts from cold HBM data
                            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                            e0.record()
                            for _ in range(steps):
                                graph.replay()
                            e1.record()
                            torch.cuda.synchronize()
                            assert int(layer.status[0].item()) == 0, "device-side wait timed out"
                            ms = e0.elapsed_time(e1) / steps
                            launches += per_step * steps
                            fwd = 2.0 * M * N * (K + nOp + r)
                            bwd = 2.0 * M * N * (K + nOp) + 2.0 * M * K * r
                            # against a step whose forward ran at the INT8 rate and whose grad-input ran at the bf16 rate
                            t_roof = (fwd / (2.0 * peaks["bf16_tflops"]) + bwd / peaks["bf16_tflops"]) / 1e12 * 1e3
                            points.append({"M": M, "K": K, "N": N, "r": r, "frac": frac, "nO": nO, "ms_per_step": round(ms, 5),
                                           "tokens_per_s": round(M / (ms * 1e-3), 1), "tera_ops_per_s": round((fwd + bwd) / (ms * 1e-3) / 1e12, 1),
                                           "frac_of_gemm_roofline": round(t_roof / ms, 4)})
                            del graph, layer, X, dY
    fr = [p["frac_of_gemm_roofline"] for p in points]
    line = {"workload": "sweep", "metric": METRIC, "unit": UNIT, "n_gpus": 1, "points": len(points), "steps_per_point": steps,
            "warmup_per_point": 1, "data": "synthetic (drawn on the device)", "gpu_launches": int(launches), "clocks": clocks.summary(),
            "roofline_of_a_point": "time of the forward's INT8 ops at 2x the measured bf16 burst peak plus the grad-input's bf16 flops at that "
                                   "peak, over the measured step (everything else of the step - quantization, LoRA GEMMs - counts as overhead)",
            "frac_of_gemm_roofline": {"min": min(fr), "median": float(np.median(fr)), "max": max(fr)},
            "columns": ["M", "K", "N", "r", "frac", "nO", "ms_per_step", "tokens_per_s", "tera_ops_per_s", "frac_of_gemm_roofline"],
            "table": [[p[c] for c in ("M", "K", "N", "r", "frac", "nO", "ms_per_step", "tokens_per_s", "tera_ops_per_s", "frac_of_gemm_roofline")]
                      for p in points]}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--micro", default=None, choices=["quant_act", "quant_grad", "momentum", "requant", "outlier_count", "lora_down", "fwd", "bwd", "bwd8"],
                    help="time one HBM-bound kernel alone instead of the step")
    ap.add_argument("--micro-shape", type=lambda v: tuple(int(x) for x in v.split(",")), default=(8192, 11008, 4096, 55),
                    help="M,K,N,nO of --micro (default: the LLaMA-2-7B down_proj rows)")
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--micro-rank", type=int, default=64, help="LoRA rank of --micro fwd / bwd")
    ap.add_argument("--workload", default="llama7b_block", choices=sorted(synth.WORKLOADS) + ["sweep"])
    ap.add_argument("--int8-grad", action="store_true",
                    help="run the backward through quaff_qlinear_bwd_int8, the INT8 grad-input variant (not the paper's method)")
    ap.add_argument("--lean-bwd", action="store_true",
                    help="give the backward a workspace without room for a bf16 copy of the weight: the codes are expanded inside the GEMM")
    ap.add_argument("--sweep-quick", action="store_true", help="--workload sweep on a 2 x 2 x 2 corner of the (M, K, N) grid only")
    ap.add_argument("--repeats", type=int, default=30, help="how often the timed region of --steps steps is repeated (median reported)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--sample-tokens", type=int, default=128, help="tokens per step of the CPU oracle (reference arm); the cpu_baseline leg uses 8x this")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--eager", action="store_true", help="enqueue every launch from Python instead of replaying a CUDA graph of the step")
    ap.add_argument("--fwd-tile", type=int, default=0, choices=[0, 128, 192, 256],
                    help="force the forward kernel's output-column tile (0: the library's cost model decides)")
    args = ap.parse_args()
    if args.workload == "sweep":
        return run_sweep(args)
    wl = synth.WORKLOADS[args.workload]
    if args.fwd_tile and args.impl != "reference":
        from paper_2505_14742_b200 import binding, build
        build.build_library()
        binding.quaff_debug_force_fwd_tile(args.fwd_tile)
    if args.micro:
        if args.steps == 20:
            args.steps = 30
        return run_micro(args)
    if args.impl == "reference":
        run_reference(args, wl)
    else:
        run_gpu(args, wl)


if __name__ == "__main__":
    main()
