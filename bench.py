#!/usr/bin/env python
"""Benchmark: training samples/s of the partitioned training step on B200.

A step is one pass of the whole path over one synthetic batch: forward through every stage,
backward through every stage, SGD on every stage (ftp_train_step), on the partition chosen by
ftp_choose_partition from ftp_profile_layers times.  Prints ONE JSON line (rank 0).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload cfg2|cfg1]

N > 1 (under torchrun): the path has no sharding and no collective, so every rank runs an
independent replica of the same workload ("replicas only"); value is the aggregate.
"""
import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

FP32_ALU_PEAK_TFLOPS = 2 * 128 * 148 * 1.965e9 / 1e12      # FMA lanes x SMs x max SM clock (nominal unit counts)
FALLBACK_HBM_GBS = 6650.0


def workload(name, batch=None):
    import synth
    if name == "cfg1":
        ls, cfg = synth.har_cnn()
        return dict(index=0, name="config 1: HAR 1D-CNN 32x9x128 fp32, 2 stages split after layer 2", layers=ls, cfg=cfg,
                    caps=None, points=[0, 2, 5])
    if name in ("cfg3", "cfg5"):
        b = batch or 64
        ls, cfg = synth.mobilenetv2(b, 224, 1000, 1, False)
        cfg["max_stages"] = 5
        if name == "cfg3":
            return dict(index=2, name=f"config 3: MobileNetV2 224x224x3 batch {b} bf16, 4 stages under capacity ratios 1:2:5:10",
                        layers=ls, cfg=cfg, caps=[1.0, 2.0, 5.0, 10.0], points=None)
        return dict(index=4, name=f"config 5: MobileNetV2 224x224x3 batch {b} bf16, 5 stages, capacities U[1,10] redrawn and partition "
                    "re-chosen every 50 iterations, chain + global snapshots every 20", layers=ls, cfg=cfg, caps=[1.0] * 5, points=None,
                    dynamic=dict(repartition=50, snapshot=20))
    if name == "cfg4":
        b = batch or 256
        ls, cfg = synth.vgg16(b, 32, 10, 1)
        return dict(index=3, name=f"config 4: VGG-16-style 32x32x3 batch {b} bf16, 3 stages from the partition optimiser", layers=ls,
                    cfg=cfg, caps=[1.0, 1.0, 1.0], points=None)
    if name == "cl8":
        ls, cfg = synth.continual_mbv2(batch or 8)
        return dict(index=5, name=f"continuous-learning shape (Sec. IV-F): MobileNetV2 28x28x1 batch {batch or 8} fp32, lr 0.00625, 3 stages at equal capacity",
                    layers=ls, cfg=cfg, caps=[1.0, 1.0, 1.0], points=None)
    ls, cfg = synth.mobilenetv2(batch or 128, 32, 10, 0, True)
    return dict(index=1, name=f"config 2: MobileNetV2 32x32x3 batch {batch or 128} fp32, 3 stages at equal capacity", layers=ls,
                cfg=cfg, caps=[1.0, 1.0, 1.0], points=None)


FALLBACK_BF16_TFLOPS = 1400.0            # sustained figure of the fallback measurement


def step_work(layers, cfg):
    """Whole-step algorithmic work from the layer list at the configured batch.  Per contraction / depthwise op with I
    input and O output elements: model A = every tensor pass of separate conv / BN forward / BN backward / data-gradient /
    weight-gradient kernels counted once, (3 I + 11 O) elements; model B = batch-norm statistics from the producer and
    both batch-norm apply passes folded into their neighbours, (3 I + 5 O) elements.  Flops: forward plus twice that for
    the backward pass.  Returns (bytes A, bytes B, dense flop, depthwise flop)."""
    import synth
    K = synth.KIND
    s = 2 if cfg["precision"] == 1 else 4
    n, h, w, c = cfg["batch"], cfg["in_h"], cfg["in_w"], cfg["in_c"]
    a = b = dense = dw = 0
    for l in layers:
        if l.kind in (K["CONV1D"], K["CONV2D"], K["FC"], K["DWCONV3x3"]):
            kh, kw, ph, pw = (1, l.k, 0, l.pad) if l.kind == K["CONV1D"] else ((1, 1, 0, 0) if l.kind == K["FC"] else (l.k, l.k, l.pad, l.pad))
            ho, wo = (h + 2 * ph - kh) // l.stride + 1, (w + 2 * pw - kw) // l.stride + 1
            i_el, o_el = n * h * w * c, n * ho * wo * l.cout
            a += (3 * i_el + 11 * o_el) * s
            b += (3 * i_el + 5 * o_el) * s
            if l.kind == K["DWCONV3x3"]:
                dw += 3 * 18 * o_el
            else:
                dense += 3 * 2 * n * ho * wo * kh * kw * c * l.cout
            h, w, c = ho, wo, l.cout
        elif l.kind == K["MAXPOOL2"]:
            h, w = h // 2, w // 2
        elif l.kind == K["GAP"]:
            h = w = 1
    return a, b, dense, dw


# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) of all launches of a kernel class in one step of the default
# workload, from one ncu pass.  An entry is valid only for the kernel source it was taken on (sha256 of the file) and is
# added only together with a retaken pass; without a valid entry `traffic` is null.
NCU_TRAFFIC = {
    ("cfg2", "tc_gemm_tf32x3_wgrad"): {"bytes_per_step": 895.0e6, "source": "paper_2110_02781_b200/csrc/gemm_tc32.cu",
                                       "sha256": "a07b2bde7b907b32341c3cecfad488f58cd67ed974cb3d8042982182b4b67c16"},
}


def ncu_traffic(wl_key, kernel, default_batch):
    e = NCU_TRAFFIC.get((wl_key, kernel))
    if not e or not default_batch:
        return None
    import hashlib
    try:
        with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), e["source"]), "rb") as f:
            if hashlib.sha256(f.read()).hexdigest() != e["sha256"]:
                return None
    except OSError:
        return None
    return e["bytes_per_step"]


def peaks():
    """(HBM GB/s, bf16 tensor TFLOP/s sustained, source).  The sustained tensor figure applies: kernels are timed inside a long step."""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), float(d.get("bf16_tflops_sustained", d.get("bf16_tflops", FALLBACK_BF16_TFLOPS))), "measured"
    return FALLBACK_HBM_GBS, FALLBACK_BF16_TFLOPS, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.rows, self.proc, self.index = [], None, index

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"], stdout=subprocess.PIPE, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except OSError:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def __exit__(self, *a):
        if self.proc:
            time.sleep(0.15)
            self.proc.terminate()
            self.t.join(timeout=2)

    def summary(self):
        sm = [float(r[0]) for r in self.rows if len(r) >= 7 and r[0].replace(".", "").isdigit()]
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for k, n in enumerate(names) if any(len(r) >= 7 and r[3 + k].lower().startswith("active") for r in self.rows)]
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": float(self.rows[0][1]), "reasons": reasons,
                "samples": len(sm)}


def run_reference(args, wl):
    """The oracle as it stands, on the host cores, on a bounded sample of the workload."""
    import numpy as np
    import oracle
    import synth
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        cores = os.cpu_count() or 1
    ls, cfg = wl["layers"], dict(wl["cfg"])
    sample_batch = min(cfg["batch"], {0: cfg["batch"], 1: 16, 2: 2, 3: 8, 4: 2, 5: cfg["batch"]}[wl["index"]])
    cfg["batch"] = sample_batch
    om = oracle.OracleModel(ls, cfg, synth.init_params(wl["index"], ls), synth.init_state(ls))
    L = om.L
    pts = wl["points"] or [0, L // 3, 2 * L // 3, L]
    x, y = synth.make_batch(wl["index"], cfg)
    times = []
    for it in range(args.warmup_ref + args.steps):
        t = time.perf_counter()
        om.step(pts, x, y)
        if it >= args.warmup_ref:
            times.append(time.perf_counter() - t)
    tot = sum(times)
    value = sample_batch * len(times) / tot
    sample = (f"{len(times)} steps of the same network at batch {sample_batch} (of {wl['cfg']['batch']}), float64 numpy"
              + (", bf16 storage mode" if cfg["precision"] == 1 else ""))
    return {"impl": "reference", "metric": "training samples/sec per partitioned step", "value": value, "unit": "samples/s",
            "n_gpus": args.gpus, "steps": len(times), "warmup": args.warmup_ref, "ms_per_step": 1e3 * tot / len(times),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": wl["name"], "stages": len(pts) - 1, "sample_batch": sample_batch},
            "cpu_baseline": {"value": value, "unit": "samples/s", "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "samples/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}


def run_dynamic(m, F, wl, layer_times, xd, yd, xh, yh, lr, steps, on_host, fail=None, out_bytes=None):
    """Config 5: train `steps` iterations; after every `repartition`-th the stage capacities are redrawn from U[1,10] and the
    partition re-chosen (Eq. 4 on the profiled layer times); after every `snapshot`-th each stage's weights are copied to
    the next stage's replica buffer (last stage -> central) and every stage's to the central pinned-host buffer.
    fail = (iteration, stage): after that iteration the stage is declared lost (a host-side event; Sec. III-F), the
    survivors take over at the partition Eq. 4 gives for their capacities, the lost units reload from the replicas of
    the last replication tick, and the stage rejoins at the next repartition.
    Returns (total ms, per-iteration ms list, log of partitions)."""
    import numpy as np
    import torch
    import synth
    dyn = wl["dynamic"]
    n_st = len(wl["caps"])
    rng = synth.rng_stream(wl["index"], "capacity")
    L = m.L
    sizes = [m.ftp_unit_param_span(u)[1] + m.ftp_unit_state_span(u)[1] for u in range(L)]
    total = sum(sizes)
    replicas = [torch.empty(total, dtype=torch.float32, device="cuda") for _ in range(n_st)]      # chain targets (device)
    central = torch.empty(2 * total, dtype=torch.float32).pin_memory()                             # chain tail + global copy (host)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    log = []
    last_caps = list(wl["caps"])
    factors = rng.uniform(1.0, 10.0, n_st).tolist()              # slowdown factors of the simulated devices in the current window
    closed_loop = not on_host
    window = []
    # Eq. 4-5 with the links this machine has: a boundary activation and its gradient cross a device-to-device copy
    # (measured here, Sec. III-B); without the unit sizes the term is left out
    link = None
    if out_bytes is not None:
        d2d, d2h = m.ftp_measure_bandwidth(central, min(64 << 20, central.numel() * 4), 5)
        link = dict(out_bytes=[float(b) for b in out_bytes], d2d_GBps=round(d2d / 1e9, 1), d2h_GBps=round(d2h / 1e9, 1), bw=d2d)
        log.append(dict(measured_link_bandwidth_GBps=dict(device_to_device=link["d2d_GBps"], device_to_pinned_host=link["d2h_GBps"])))
    choose = lambda caps: F.ftp_choose_partition(layer_times, caps, link["out_bytes"] if link else None,
                                                 [link["bw"]] * (len(caps) - 1) if link and len(caps) > 1 else None)
    if closed_loop:
        m.ftp_stage_timing_enable(True)
    replicated_at = None                 # partition under which the replicas were last written
    torch.cuda.synchronize()
    ev[0].record()
    for it in range(steps):
        if on_host:
            m.ftp_train_step(xh, yh, lr, inputs_on_host=True, want_loss=True)
        else:
            m.ftp_train_step(xd, yd, lr, inputs_on_host=False, want_loss=False)
        if (it + 1) % dyn["snapshot"] == 0:
            pts = m.ftp_get_partition()
            off = 0
            for s in range(len(pts) - 1):
                n = sum(sizes[pts[s]:pts[s + 1]])
                if s + 1 < len(pts) - 1:
                    m.ftp_snapshot_weights(s, replicas[s + 1][:n])                     # chain: to the next stage
                else:
                    m.ftp_snapshot_weights(s, central[total + off:total + off + n])    # chain: last stage to the central node
                m.ftp_snapshot_weights(s, central[off:off + n])                        # global: every stage to the central node
                off += n
            replicated_at = tuple(pts)
        if fail and it + 1 == fail[0] and fail[1] < len(m.ftp_get_partition()) - 1:
            pts = m.ftp_get_partition()
            caps = [c for s, c in enumerate(last_caps[:len(pts) - 1]) if s != fail[1]]
            new_pts, bott = choose(caps)
            t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
            t0.record()
            nxt = fail[1] + 1
            chain = replicas[nxt][:sum(sizes[pts[fail[1]]:pts[fail[1] + 1]])] if nxt < len(pts) - 1 else \
                central[total + sum(sizes[:pts[fail[1]]]):total + sum(sizes[:pts[fail[1] + 1]])]
            counts = m.ftp_recover({fail[1]: chain if replicated_at == tuple(pts) else None}, new_pts, central[:total] if replicated_at else None)
            t1.record()
            torch.cuda.synchronize()
            log.append(dict(after_iteration=it + 1, failed_stage=fail[1], points=new_pts, from_stage_replica_central=list(counts),
                            recovery_ms=round(t0.elapsed_time(t1), 4), virtual_bottleneck_ms=round(bott * 1e3, 4)))
        if closed_loop and (it + 1) % 10 == 0:                  # a worker reports its batch time now and then (Sec. III-B)
            window.append(m.ftp_stage_times())
        if (it + 1) % dyn["repartition"] == 0:
            n_now = len(m.ftp_get_partition()) - 1
            reports = [w for w in window if len(w) == n_now]
            if closed_loop and reports:
                # Eq. 1-3 on what the workers reported over the window: reported time = device time of the stage x the
                # slowdown factor its simulated device had; the central node's own layer times are the profile x its
                # factor, so C_0 = 1 and C_i comes out near f_i / f_0.  A stage that rejoins has reported nothing yet.
                mean = [sum(w[s] for w in reports) / len(reports) for s in range(n_now)]
                central_times = [t * factors[0] for t in layer_times]
                caps = F.ftp_estimate_capacity(central_times, m.ftp_get_partition(), [mean[s] * factors[s] for s in range(n_now)])
                caps += [factors[s] / factors[0] for s in range(n_now, n_st)]
            else:
                caps = list(factors)
            window = []
            pts, bott = choose(caps)
            moved = m.ftp_set_partition(pts)
            log.append(dict(after_iteration=it + 1, capacities=[round(c, 3) for c in caps], factors=[round(f, 3) for f in factors], points=pts,
                            moved_units=moved, virtual_bottleneck_ms=round(bott * 1e3, 4)))
            last_caps = list(caps)
            factors = rng.uniform(1.0, 10.0, n_st).tolist()      # the simulated devices change speed for the next window
        ev[it + 1].record()
    torch.cuda.synchronize()
    if closed_loop:
        m.ftp_stage_timing_enable(False)
    per_it = [ev[i].elapsed_time(ev[i + 1]) for i in range(steps)]
    return ev[0].elapsed_time(ev[steps]), per_it, log


def measure(args, wl_key, reps, steps, warmup, local_rank, replicas, batch=None, points=None, graph=1, fail=None, lean=False):
    """Builds one workload, times `reps` blocks of `steps` steps on the device (median block), then the end-to-end
    leg (host inputs copied in, loss read back, every step) and a per-launch event trace.  Returns the fields of a
    bench line for that workload."""
    import torch
    import synth
    import paper_2110_02781_b200 as F
    wl = workload(wl_key, batch)
    ls, cfg = wl["layers"], wl["cfg"]
    m = F.Model(ls, cfg, f"cuda:{local_rank}")
    m.load_params(synth.init_params(wl["index"], ls), synth.init_state(ls))
    x, y = synth.make_batch(wl["index"], cfg)
    bf16 = cfg["precision"] == 1
    xt = torch.from_numpy(x).to(torch.bfloat16) if bf16 else torch.from_numpy(x)
    xd, yd = xt.cuda(), torch.from_numpy(y).cuda()
    xh, yh = xt.pin_memory(), torch.from_numpy(y).pin_memory()
    lr = cfg["lr"]

    # partition: profile -> capacities -> optimiser (or the split the workload fixes)
    fwd_s = bwd_s = unit_bytes = None
    if points:
        wl["points"] = list(points)
    else:
        fwd_s, bwd_s, unit_bytes = m.ftp_profile_layers(10, xd, yd)
    if wl["points"] is None:
        pts, _ = F.ftp_choose_partition((fwd_s + bwd_s).tolist(), wl["caps"])
    else:
        pts = wl["points"]
    m.ftp_set_partition(pts)

    def barrier():
        replicas.barrier()
        torch.cuda.synchronize()

    def timed(fn, n):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record()
        for _ in range(n):
            fn()
        e1.record()
        barrier()
        return replicas.max_over_ranks(e0.elapsed_time(e1))

    step_eager = lambda: m.ftp_train_step(xd, yd, lr, inputs_on_host=False, want_loss=False)
    step_dev = step_eager
    dynamic = wl.get("dynamic")
    if dynamic:
        graph = 0                        # the partition changes during the run: launches are issued eagerly
    if graph:
        # the launches of one step captured once on a side stream and replayed: same kernels, no per-launch CPU cost
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for _ in range(2):
                step_eager()
        torch.cuda.current_stream().wait_stream(side)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            step_eager()
        step_dev = g.replay
    # end to end: the same step through the public call with pinned host inputs and the loss read back on the host every step
    step_e2e = lambda: m.ftp_train_step(xh, yh, lr, inputs_on_host=True, want_loss=True)
    e2e_launch = "eager"
    if graph:
        # ... captured once as well: the copies of the inputs and of the loss are nodes of the graph; a replay, a
        # synchronisation and the read of the pinned loss make one step
        try:
            loss_pin = torch.zeros(1, dtype=torch.float32).pin_memory()
            side2 = torch.cuda.Stream()
            side2.wait_stream(torch.cuda.current_stream())
            g2 = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g2, stream=side2):
                m.ftp_train_step(xh, yh, lr, inputs_on_host=True, loss_pinned=loss_pin)

            def step_e2e():
                g2.replay()
                torch.cuda.current_stream().synchronize()
                return float(loss_pin[0])
            e2e_launch = "cuda graph replay of ftp_train_step with host inputs"
        except Exception as e:                                   # keep the eager call
            sys.stderr.write(f"end-to-end graph capture failed ({e}); timing eager calls\n")
            step_e2e = lambda: m.ftp_train_step(xh, yh, lr, inputs_on_host=True, want_loss=True)
            torch.cuda.synchronize()
            try:                                                 # the first call after a broken capture reports (and clears) its error
                step_eager()
            except Exception:
                pass
            torch.cuda.synchronize()
    for _ in range(warmup):
        step_dev()
    dyn_info = None
    blocks = []
    with ClockSampler(local_rank) as clk:
        if dynamic:
            lt = (fwd_s + bwd_s).tolist()
            barrier()
            ms, per_it, plog = run_dynamic(m, F, wl, lt, xd, yd, xh, yh, lr, steps, False, fail, unit_bytes)
            barrier()
            blocks = [replicas.max_over_ranks(ms)]
            tick = lambda i, p: (i + 1) % p == 0
            plain = [t for i, t in enumerate(per_it) if not tick(i, dynamic["snapshot"]) and not tick(i, dynamic["repartition"])]
            snap = [t for i, t in enumerate(per_it) if tick(i, dynamic["snapshot"]) and not tick(i, dynamic["repartition"])]
            rep = [t for i, t in enumerate(per_it) if tick(i, dynamic["repartition"])]
            med = lambda v: round(statistics.median(v), 4) if v else None
            dyn_info = dict(ms_plain_iteration=med(plain), ms_snapshot_iteration=med(snap), ms_repartition_iteration=med(rep),
                            repartitions=plog[:12], snapshot_bytes_per_tick=int(3 * 4 * sum(m.ftp_unit_param_span(u)[1] + m.ftp_unit_state_span(u)[1] for u in range(m.L))))
        else:
            blocks = [timed(step_dev, steps) for _ in range(reps)]
    ms = statistics.median(blocks)
    c0 = m.ftp_launch_count()
    step_eager()                        # a replay re-issues the captured launches without passing through the counter
    per_step = m.ftp_launch_count() - c0
    out = {"workload": wl["name"], "index": wl["index"], "points": [int(p) for p in pts], "batch": cfg["batch"], "bf16": bf16, "steps": steps,
           "ms_per_step": ms / steps, "value": replicas.job_throughput(cfg["batch"] * steps, ms),
           "blocks_ms_per_step": {"median": ms / steps, "min": min(blocks) / steps, "max": max(blocks) / steps, "blocks": len(blocks)},
           "clocks": clk.summary(), "launches_per_step": int(per_step), "gpu_launches": int(per_step * steps * len(blocks)),
           "graph": bool(graph), "caps": wl["caps"], "dynamic": dyn_info}
    if lean:
        m.close()
        return out
    for _ in range(3):
        step_e2e()
    e2e_steps = steps
    if dynamic:
        e2e_steps = max(dynamic["repartition"] * 2, steps // 5)
        m.ftp_set_partition(pts)
        barrier()
        ms_e2e, _, _ = run_dynamic(m, F, wl, (fwd_s + bwd_s).tolist(), xd, yd, xh, yh, lr, e2e_steps, True)
        barrier()
        ms_e2e = replicas.max_over_ranks(ms_e2e)
        m.ftp_set_partition(pts)
    else:
        ms_e2e = timed(step_e2e, steps)
    out["e2e"] = {"value": replicas.job_throughput(cfg["batch"] * e2e_steps, ms_e2e), "unit": "samples/s",
                  "h2d_bytes_per_step": int(xh.numel() * xh.element_size() + yh.numel() * 4), "d2h_bytes_per_step": 4,
                  "ms_per_step": ms_e2e / e2e_steps, "steps": e2e_steps, "launch": "eager" if dynamic else e2e_launch}

    # per-kernel roofline: three more steps with every launch bracketed by events.  Eager launches are issued more
    # slowly than the GPU runs them, and an event pair around a launch the GPU has to wait for would time the host
    # (tensor-map encoding, the launch call), not the kernel: so untraced steps are queued first, enough of them that
    # the host stays ahead of the device for the whole of the traced steps.
    torch.cuda.synchronize()
    lead = max(8, int(math.ceil(60.0 / max(ms / steps, 1e-3))))
    for _ in range(min(lead, 400)):
        step_eager()
    m.ftp_trace_enable(True)
    for _ in range(3):
        step_eager()
    recs = m.ftp_trace_read()
    m.ftp_trace_enable(False)
    by = {}
    for r in recs:
        k = by.setdefault(r["kernel"], dict(ms=0.0, bytes=0.0, flops=0.0, n=0))
        k["ms"] += r["ms"]; k["bytes"] += r["bytes"]; k["flops"] += r["flops"]; k["n"] += 1
    total_ms = sum(k["ms"] for k in by.values())
    hbm_peak, tensor_peak, peak_src = peaks()
    table = {}
    for name, k in sorted(by.items(), key=lambda kv: -kv[1]["ms"]):
        gbs = k["bytes"] / (k["ms"] * 1e-3) / 1e9 if k["ms"] > 0 else 0.0
        tf = k["flops"] / (k["ms"] * 1e-3) / 1e12 if k["ms"] > 0 else 0.0
        # bf16 products: the measured bf16 matmul rate.  Split-tf32 products (three tf32 MMAs per float product): that rate x the
        # nominal tf32 / bf16 ratio (1.1 / 2.25 PFLOP/s dense), a third of it per float product.  Everything else: the fp32 FMA rate.
        math_peak = tensor_peak if name.startswith("tc_gemm_bf16") else (tensor_peak * (1.1 / 2.25) / 3.0 if name.startswith("tc_gemm_tf32x3") else FP32_ALU_PEAK_TFLOPS)
        table[name] = dict(share=round(k["ms"] / total_ms, 4), launches_per_step=k["n"] // 3, ms_per_step=round(k["ms"] / 3, 4),
                           gbs=round(gbs, 1), tflops=round(tf, 2), frac_hbm=round(gbs / hbm_peak, 3),
                           frac_math=round(tf / math_peak, 3))
    dom = next(iter(table))
    d = table[dom]
    math_bound = d["frac_math"] > d["frac_hbm"]
    tensor = dom.startswith("tc_gemm_")
    tpeak = tensor_peak if dom.startswith("tc_gemm_bf16") else tensor_peak * (1.1 / 2.25) / 3.0
    roofline = {"kernel": dom, "bound": ("tensor" if tensor else "alu") if math_bound else "hbm",
                "achieved": d["tflops"] if math_bound else d["gbs"],
                "peak": (round(tpeak, 1) if tensor else round(FP32_ALU_PEAK_TFLOPS, 1)) if math_bound else hbm_peak,
                "unit": "TFLOP/s" if math_bound else "GB/s",
                "frac": d["frac_math"] if math_bound else d["frac_hbm"],
                "peak_source": ((f"{peak_src} bf16 matmul, sustained" + ("" if dom.startswith("tc_gemm_bf16") else " x 1.1/2.25 (tf32) / 3 products")
                                 if tensor else "derived: 2 x 128 lanes x 148 SMs x 1.965 GHz") if math_bound else f"{peak_src} HBM copy"),
                "traffic": ncu_traffic(wl_key, dom, batch is None), "share_of_step": d["share"],
                "note": "achieved = algorithmic bytes (or flops) of all launches of the kernel in a step / their CUDA-event time",
                "kernels": table}
    wa, wb, dense, dwf = step_work(ls, cfg)
    step_s = ms / steps * 1e-3
    tfs = (dense + dwf) / step_s / 1e12
    roofline["step"] = {"algorithmic_GB_separate_passes": round(wa / 1e9, 3), "algorithmic_GB_fused_bn": round(wb / 1e9, 3),
                        "frac_hbm_separate_passes": round(wa / step_s / 1e9 / hbm_peak, 3), "frac_hbm_fused_bn": round(wb / step_s / 1e9 / hbm_peak, 3),
                        "TFLOP/s": round(tfs, 2), "frac_tensor": round(dense / step_s / 1e12 / tensor_peak, 3) if bf16 else None,
                        "note": "whole step: algorithmic bytes of all kernels / device time of a step, against the count with separate "
                                "batch-norm passes ((3I+11O) per convolution) and against the count with them folded into their neighbours ((3I+5O))"}
    out["roofline"] = roofline
    m.close()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None, help="timed steps per block (default 50; 500 for cfg5)")
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--reps", type=int, default=5, help="timed blocks of --steps steps; the median block is reported")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2", choices=["cfg1", "cfg2", "cfg3", "cfg4", "cfg5", "cl8"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-configs", action="store_true", help="skip the short entries for the other workloads")
    ap.add_argument("--batch", type=int, default=None, help="smaller batch of the same network (profiling captures only)")
    ap.add_argument("--points", default=None, help="comma-separated partition points; skips the profile-and-optimise step")
    ap.add_argument("--graph", type=int, default=1, help="1: time CUDA-graph replays of the step (default); 0: eager launches")
    ap.add_argument("--fail", default=None, help="cfg5 only, ITERATION:STAGE: that stage is lost after that iteration and recovered from the replicas")
    ap.add_argument("--lean", action="store_true", help="timed region only: no end-to-end leg, no kernel trace (profiling captures)")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.steps is None:
        args.steps = 500 if args.workload == "cfg5" else 50

    if args.impl == "reference":
        if rank != 0:
            return 0
        args.warmup_ref = min(args.warmup, 1)
        args.steps = min(args.steps, 3)
        print(json.dumps(run_reference(args, workload(args.workload, args.batch))), flush=True)
        return 0

    import torch
    assert args.warmup >= 3, "at least 3 warm-up steps"
    torch.cuda.set_device(local_rank)
    from paper_2110_02781_b200.replicas import Replicas
    reps = Replicas("nccl", torch.device("cuda", local_rank))

    points = [int(v) for v in args.points.split(",")] if args.points else None
    fail = tuple(int(v) for v in args.fail.split(":")) if args.fail else None
    r = measure(args, args.workload, args.reps, args.steps, args.warmup, local_rank, reps, args.batch, points, args.graph, fail, args.lean)
    if args.lean:
        if rank == 0:
            print(json.dumps({"lean": True, "ms_per_step": r["ms_per_step"], "blocks_ms_per_step": r["blocks_ms_per_step"],
                              "gpu_launches": r["gpu_launches"]}), flush=True)
        reps.close()
        return 0
    bf16 = r["bf16"]
    out = {"metric": "training samples/sec per partitioned step", "value": r["value"], "unit": "samples/s", "n_gpus": world,
           "steps": args.steps, "warmup": args.warmup, "ms_per_step": r["ms_per_step"], "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if bf16 else "f32 (tf32x3 contractions)", "data": "synthetic",
           "config": {"workload": r["workload"], "points": r["points"], "stages": len(r["points"]) - 1, "batch": r["batch"],
                      "parallelism": "replicas only" if world > 1 else "1 GPU, all stages resident",
                      "cache": "a step streams far more activation bytes than the 126 MB L2 holds",
                      "capacities": r["caps"], "launch": "cuda graph replay of ftp_train_step" if r["graph"] else "eager",
                      "timed": f"{r['blocks_ms_per_step']['blocks']} blocks of {args.steps} steps, median block reported",
                      "blocks_ms_per_step": r["blocks_ms_per_step"], "launches_per_step": r["launches_per_step"]},
           "clocks": r["clocks"], "gpu_launches": r["gpu_launches"], "e2e": r["e2e"], "roofline": r["roofline"]}
    if r["dynamic"]:
        out["config"]["dynamic"] = r["dynamic"]
    if world == 1 and not args.no_configs:
        # the other workloads, briefly: value, end-to-end value, the dominant kernel's fraction and the clocks seen, each
        others = {}
        for key in ("cfg1", "cfg2", "cfg3", "cfg4", "cfg5", "cl8"):
            if key == args.workload:
                continue
            q = measure(args, key, 3, 100 if key == "cfg5" else 20, 3, local_rank, reps)
            rf = q["roofline"]
            others[key] = {"workload": q["workload"], "value": round(q["value"], 1), "unit": "samples/s", "ms_per_step": round(q["ms_per_step"], 4),
                           "blocks_ms_per_step": q["blocks_ms_per_step"], "points": q["points"], "launches_per_step": q["launches_per_step"],
                           "e2e": {k: q["e2e"][k] for k in ("value", "h2d_bytes_per_step", "d2h_bytes_per_step", "ms_per_step")},
                           "dtype": "bf16" if q["bf16"] else "f32 (tf32x3 contractions)",
                           "dominant_kernel": {k: rf[k] for k in ("kernel", "bound", "achieved", "peak", "unit", "frac", "share_of_step")},
                           "step": rf["step"], "clocks": q["clocks"]}
            if q["dynamic"]:
                others[key]["dynamic"] = {k: q["dynamic"][k] for k in ("ms_plain_iteration", "ms_snapshot_iteration", "ms_repartition_iteration")}
        out["configs"] = others
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        a2 = argparse.Namespace(**vars(args))
        a2.warmup_ref, a2.steps = 0, 2
        out["cpu_baseline"] = run_reference(a2, workload(args.workload, args.batch))["cpu_baseline"]
    if rank == 0:
        print(json.dumps(out), flush=True)
    reps.close()
    return 0


if __name__ == "__main__":
    sys.exit(main())
