#!/usr/bin/env python
"""Benchmark of the coded training step (one process per GPU, replicas only).

    python bench.py --gpus N --steps K --warmup W [--impl reference] [--workload c3]

A step is one pass of the whole hot path -- additional encoding of the vectors, feedforward
products with detection / location / decoding, loss, fused backpropagation products + coded
rank-B update with its checks -- over one batch of synthetic input.  The default workload is
the 8192 x 8192 fp32 layer on an 8x8 data grid with one parity block-row and block-column,
batch 1, soft errors injected into block outputs with probability 1e-3 per node and phase.

One JSON line is printed by rank 0.  ``value`` is coded-SGD iterations per second per layer
summed over all ranks with inputs resident in HBM; ``e2e`` is the same through the public API
with inputs copied from pinned host memory and the loss and reports read back every step.
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler(threading.Thread):
    """Samples SM clocks and throttle reasons while the timed region runs: through NVML when the Python
    binding is there, otherwise from a read-only ``nvidia-smi --query-gpu`` loop.  Nothing is ever set."""

    NAMES = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, index, period=0.01):
        super().__init__(daemon=True)
        self.index = index
        self.period = period
        self.sm = []
        self.reason_bits = 0
        self.sm_max = None
        self.source = None
        self.stop_flag = threading.Event()
        # the library is opened here, before the timed region: a region of twenty steps lasts 2.5 ms, and a sampler
        # that first has to load NVML inside it comes back with no sample at all
        self.nv = self.handle = None
        try:
            import pynvml as nv
            nv.nvmlInit()
            self.handle = nv.nvmlDeviceGetHandleByIndex(index)
            self.sm_max = float(nv.nvmlDeviceGetMaxClockInfo(self.handle, nv.NVML_CLOCK_SM))
            nv.nvmlDeviceGetClockInfo(self.handle, nv.NVML_CLOCK_SM)      # first calls are the slow ones
            nv.nvmlDeviceGetCurrentClocksEventReasons(self.handle)
            self.nv = nv
        except Exception:
            self.nv = None

    def _run_nvml(self):
        nv, h = self.nv, self.handle
        if nv is None:
            raise RuntimeError("no NVML binding")
        self.source = "nvml"
        n = 0
        while not self.stop_flag.is_set():
            self.sm.append(float(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM)))
            self.reason_bits |= int(nv.nvmlDeviceGetCurrentClocksEventReasons(h))
            n += 1
            # every half millisecond at first (short regions get a few samples), then at the set period
            self.stop_flag.wait(0.0005 if n < 40 else self.period)

    def _run_smi(self):
        uuid = None
        try:
            import torch
            uuid = "GPU-" + str(torch.cuda.get_device_properties(self.index).uuid)
        except Exception:
            pass
        cmd = ["nvidia-smi", "--query-gpu=clocks.sm,clocks.max.sm,clocks_event_reasons.active",
               "--format=csv,noheader,nounits", "-lms", "100", "-i", uuid or str(self.index)]
        proc = subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        self.source = "nvidia-smi"
        try:
            while not self.stop_flag.is_set():
                row = proc.stdout.readline()
                if not row:
                    break
                f = [x.strip() for x in row.split(",")]
                try:
                    self.sm.append(float(f[0]))
                    self.sm_max = float(f[1])
                    self.reason_bits |= int(f[2], 16)
                except (ValueError, IndexError):
                    continue
        finally:
            proc.terminate()

    def run(self):
        try:
            self._run_nvml()
        except Exception:
            try:
                self._run_smi()
            except Exception as exc:
                self.error = str(exc)

    def summary(self):
        if not self.sm:
            return {"sm_mhz": None, "sm_max_mhz": self.sm_max, "reasons": ["no samples"]}
        reasons = [n for bit, n in self.NAMES.items() if self.reason_bits & bit]
        sm = sorted(self.sm)
        return {"sm_mhz": sm[len(sm) // 2], "sm_min_mhz": sm[0], "sm_max_mhz": self.sm_max, "reasons": reasons,
                "samples": len(sm), "source": self.source}


def max_over_ranks(seconds, world, device="cuda"):
    """The slowest rank's time: replicas run independently, the job is as slow as its slowest one."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([seconds], device=device, dtype=torch.float64)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(world, steps, layers, seconds_max):
    """Layer-iterations per second summed over all replicas."""
    return world * steps * layers / seconds_max


def _ncu_traffic(workload):
    """DRAM bytes per launch of the workload's dominant kernel (dram__bytes_read.sum + dram__bytes_write.sum of one
    ncu capture), from the table kept in profiles/dram_traffic.md; None where no capture exists."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.md")
    try:
        for row in open(path):
            f = [x.strip() for x in row.strip().strip("|").split("|")]
            if len(f) >= 3 and f[0] == workload:
                return float(f[2])
    except (OSError, ValueError):
        pass
    return None


def _workload_bytes(sp, esz):
    """Algorithmic bytes of one layer-iteration: the forward pass reads the (m+r_row) x n active
    blocks, the backward+update pass reads and writes every stored block once."""
    b_r, b_c = -(-sp.n_out // sp.m), -(-sp.n_in // sp.n)
    blk = b_r * b_c * esz
    fwd = (sp.m + sp.r_row) * sp.n * blk
    stored = (sp.m * sp.n + sp.r_row * sp.n + sp.r_col * sp.m) * blk
    return fwd, 2 * stored


def run_reference(args, cfg, rank, world):
    """Times the CPU oracle, as it stands, on this host's cores."""
    if rank != 0:
        return
    from oracle import oracle as orc
    from paper_1903_01042_b200 import workloads as wl
    cores = os.cpu_count() or 1
    orc.set_threads(cores)
    layers = []
    for l, sp in enumerate(cfg.layers):
        W = wl.weights(sp.n_out, sp.n_in, seed=cfg.seed, layer=l, bf16=cfg.bf16)
        Pr, Pc = (wl.layer_codes(sp, cfg.seed, l) if sp.gaussian_code else (None, None))
        layers.append(orc.Layer(W, sp.m, sp.n, sp.r_row, sp.r_col, P_row=Pr, P_col=Pc, store_bf16=cfg.bf16,
                                check_rows=sp.check_rows, check_cols=sp.check_cols,
                                tau_rel=3e-2 if cfg.bf16 else 1e-3))
    act = {"identity": 0, "relu": 1}[cfg.activation]
    loss = {"mse": 0, "softmax_ce": 1}[cfg.loss]
    net = orc.Net(layers, activation=act, loss=loss)
    mode = {"bernoulli": 1, "exactly_one": 2, "none": 0}[cfg.fault_mode]
    faults = [orc.make_fault(seed=cfg.seed, layer=l, mode=mode, p=cfg.p, sigma=cfg.sigma) for l in range(len(layers))]
    inputs = [wl.layer_inputs(cfg, it) for it in range(args.warmup + args.steps)]
    for it in range(args.warmup):
        net.step(inputs[it][0], inputs[it][1], cfg.lr, faults, it)
    t0 = time.perf_counter()
    for it in range(args.warmup, args.warmup + args.steps):
        net.step(inputs[it][0], inputs[it][1], cfg.lr, faults, it)
    dt = time.perf_counter() - t0
    per_layer = args.steps * len(layers) / dt
    sample = "%d full-size iterations of %s" % (args.steps, cfg.name)
    line = {
        "impl": "reference", "metric": "coded_sgd_iterations_per_s_per_layer", "value": per_layer,
        "unit": "layer-iterations/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * dt / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": _config_dict(cfg, args),
        "cpu_baseline": {"value": per_layer, "unit": "layer-iterations/s", "cores": orc.get_threads(),
                         "kind": "oracle", "sample": sample},
        "e2e": {"value": per_layer, "unit": "layer-iterations/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def _config_dict(cfg, args):
    sp = cfg.layers[0]
    return {"workload": "%s: %d layer(s) %dx%d %s, %dx%d data grid + %d parity row(s) + %d parity column(s), batch %d, "
                        "soft-error probability %g per node and phase, sigma %g, lr %g"
                        % (cfg.name, len(cfg.layers), sp.n_out, sp.n_in, "bf16" if cfg.bf16 else "fp32", sp.m, sp.n,
                           sp.r_row, sp.r_col, cfg.batch, cfg.p, cfg.sigma, cfg.lr),
            "layers": len(cfg.layers), "batch": cfg.batch, "parallelism": "replicas only",
            "l2": "coded weights (%.0f MB per layer) exceed the 126 MB L2, so every pass streams from HBM"
                  % (sum(_workload_bytes(s, 2 if cfg.bf16 else 4)[1] for s in cfg.layers) / 2 / len(cfg.layers) / 1e6)}


_WEIGHTS = {}   # host copies of the synthetic weights, so that the comparison legs do not draw them again


def build_net(cn, wl, torch, cfg, locate_mode=None, coded=True):
    layers = []
    for l, sp in enumerate(cfg.layers):
        key = (cfg.name, l, sp.n_out, sp.n_in, cfg.seed, cfg.bf16)
        if key not in _WEIGHTS:
            _WEIGHTS[key] = wl.weights(sp.n_out, sp.n_in, seed=cfg.seed, layer=l, bf16=cfg.bf16)
        W = _WEIGHTS[key]
        Wd = torch.tensor(W, device="cuda").to(torch.bfloat16 if cfg.bf16 else torch.float32)
        rr, rc = (sp.r_row, sp.r_col) if coded else (0, 0)
        Pr, Pc = (wl.layer_codes(sp, cfg.seed, l) if (sp.gaussian_code and coded) else (None, None))
        lm = locate_mode if locate_mode is not None else cn.LOCATE_NODECHECK
        # batches >= 64 multiply on tensor-core tiles: bfloat16 blocks as bf16, fp32 blocks as tf32
        math = cn.MATH_FFMA if cfg.batch < 64 else (cn.MATH_BF16 if cfg.bf16 else cn.MATH_TF32)
        layers.append(cn.encode_layer(Wd, sp.m, sp.n, rr, rc, P_row=Pr, P_col=Pc, batch_max=cfg.batch, math=math,
                                      locate_mode=lm, check_rows=sp.check_rows, check_cols=sp.check_cols))
        del Wd
    act = {"identity": 0, "relu": 1}[cfg.activation]
    loss = {"mse": 0, "softmax_ce": 1}[cfg.loss]
    return layers, cn.net_create(layers, activation=act, loss=loss)


def timed_steps(cn, torch, net, layers, cfg, wl, steps, warmup, inject, e2e=False, sampler=None, lookahead=True,
                graphs=False):
    """Returns (seconds for `steps` steps, kernel launches in the timed region)."""
    L = len(layers)
    pool = 8
    cn.net_set_lookahead(net, bool(lookahead))
    total = warmup + steps
    its = torch.arange(total, dtype=torch.int32, device="cuda")
    mode = {"bernoulli": 1, "exactly_one": 2, "none": 0}[cfg.fault_mode] if inject else 0
    reps = cn.new_reports(2 * L)
    loss_dev = torch.zeros(1, device="cuda")
    host = [wl.layer_inputs(cfg, k) for k in range(pool)]
    if e2e:
        # one upload and one download per step: [next input | this step's target] go up as one pinned buffer
        # into the staging buffer of the step's parity, [reports | loss] come down as one.  Step `it` reads
        # its input from the staging buffer of the other parity, where the previous step put it.
        hx = [torch.tensor(h[0]) for h in host]
        ht = [torch.tensor(h[1]) for h in host]
        xb, tb = hx[0].numel() * hx[0].element_size(), ht[0].numel() * ht[0].element_size()
        hs = [torch.cat([hx[(k + 1) % pool].reshape(-1).view(torch.uint8), ht[k].reshape(-1).view(torch.uint8)]).pin_memory()
              for k in range(pool)]
        stage = [torch.empty(xb + tb, dtype=torch.uint8, device="cuda") for _ in range(2)]
        sx = [st_[:xb].view(hx[0].dtype).view(hx[0].shape) for st_ in stage]
        stt = [st_[xb:].view(ht[0].dtype).view(ht[0].shape) for st_ in stage]
        sx[1].copy_(hx[0])                                   # the input of step 0
        rb = reps.numel()
        out_dev = torch.zeros(rb + 16, dtype=torch.uint8, device="cuda")
        reps, loss_dev = out_dev[:rb], out_dev[rb:rb + 4].view(torch.float32)
        # two host buffers for the results and one event per buffer: the host waits for step it - 1's results
        # (and reads them) after it has queued step it, so the device never waits for the host's launches
        houts = [torch.empty(rb + 16, dtype=torch.uint8).pin_memory() for _ in range(2)]
        hout = houts[0]
        done = [torch.cuda.Event() for _ in range(2)]
        seen = {"loss": 0.0}
        # (recorded steps: a ring of four staging buffers, see below; the last warm-up step announces its first one)
        stage3 = [torch.empty(xb + tb, dtype=torch.uint8, device="cuda") for _ in range(4)]
        sx3 = [st_[:xb].view(hx[0].dtype).view(hx[0].shape) for st_ in stage3]
        st3 = [st_[xb:].view(ht[0].dtype).view(ht[0].shape) for st_ in stage3]
        sx3[3].copy_(hx[warmup % pool])                      # the input of the first recorded step

        def results_down(it):
            houts[it % 2].copy_(out_dev, non_blocking=True)
            done[it % 2].record()
            if it > 0:
                done[(it - 1) % 2].synchronize()
                seen["loss"] = float(houts[(it - 1) % 2][rb:rb + 4].view(torch.float32)[0])   # the caller's read
    else:
        dxs = [torch.tensor(h[0], device="cuda") for h in host]
        dts = [torch.tensor(h[1], device="cuda") for h in host]

    def one(it):
        faults = [cn.make_fault(seed=cfg.seed, layer=l, mode=mode, p=cfg.p, sigma=cfg.sigma, iteration_dev=its[it:])
                  for l in range(L)]
        if e2e:
            # this step's target and the NEXT step's input go up now (the input of this step went up
            # during the previous one), so that the update sweep can already use the next input
            stage[it % 2].copy_(hs[it % pool], non_blocking=True)
            if lookahead:
                cn.net_set_next_input(net, sx3[3] if (graphs and it == warmup - 1) else sx[it % 2])
            cn.step(net, sx[(it + 1) % 2], stt[it % 2], cfg.lr, faults=faults, reps_dev=reps, loss_dev=loss_dev)
            results_down(it)
        else:
            if lookahead:
                cn.net_set_next_input(net, dxs[(it + 1) % pool])
            cn.step(net, dxs[it % pool], dts[it % pool], cfg.lr, faults=faults, reps_dev=reps, loss_dev=loss_dev)

    for it in range(warmup):
        one(it)
    torch.cuda.synchronize()
    replay = None
    if graphs:
        # Recorded steps.  The K timed steps are cut into consecutive segments of 40 (and the rest), each one graph:
        # between two graph launches the device idles for 8-15 us, which a long recording makes rare.  40 is a
        # multiple of the input pool and of the staging ring, so one 40-step recording serves every whole segment.
        # (A short run is not slower because it is short: the start of the timed region costs 12-13 us once.  What
        # differs between windows of 10-20 steps is how many injected faults fall into them: the plan is fixed by
        # seed and iteration, a step with a detected codeword takes 10-13 us longer, and iterations 5-24 of
        # configuration 3 hold six of them where the long-run average is three.)
        it_ctr = torch.full((1,), warmup, dtype=torch.int32, device="cuda")
        faults = [cn.make_fault(seed=cfg.seed, layer=l, mode=mode, p=cfg.p, sigma=cfg.sigma, iteration_dev=it_ctr)
                  for l in range(L)]
        segs, left = [], steps
        while left > 0:
            segs.append(min(40, left)); left -= segs[-1]
        starts = [sum(segs[:q]) for q in range(len(segs))]
        group = max(segs)
    if graphs and e2e:
        # End to end with the steps in graphs of the caller's own: the steps of a segment are captured together WITH
        # their copies, uploads and downloads on streams of their own.  Step k (counted from the first timed step)
        # reads its input from staging buffer (k - 1) % 4 (it went up for step k - 1) and its target and the next
        # input from buffer k % 4, which may go up as soon as step k - 3, its last reader, has ended; every step has
        # its own result slot, copied down behind it.  The host reads a replay's losses from pinned memory after it
        # has queued the next replay.  The network advances the fault plans' iteration counter itself.
        cn.net_set_iteration_counter(net, it_ctr)
        slot = rb + 16
        outs_dev = torch.zeros(group * slot, dtype=torch.uint8, device="cuda")
        outs_host = [torch.empty(group * slot, dtype=torch.uint8).pin_memory() for _ in range(2)]
        main, up, down = torch.cuda.current_stream(), torch.cuda.Stream(), torch.cuda.Stream()
        torch.cuda.synchronize()

        def record(dst_host, base, n_rec):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=main):
                step_done = []
                up.wait_stream(main)
                down.wait_stream(main)
                for k in range(n_rec):
                    src, ring = (warmup + base + k) % pool, (base + k) % 4
                    if k >= 3:
                        up.wait_event(step_done[k - 3])
                    with torch.cuda.stream(up):
                        stage3[ring].copy_(hs[src], non_blocking=True)       # [x of the next step | target of this one]
                    main.wait_stream(up)
                    o = outs_dev[k * slot:(k + 1) * slot]
                    if lookahead:
                        cn.net_set_next_input(net, sx3[ring])
                    cn.step(net, sx3[(ring - 1) % 4], st3[ring], cfg.lr, faults=faults, reps_dev=o[:rb],
                            loss_dev=o[rb:rb + 4].view(torch.float32))
                    ev = torch.cuda.Event()
                    ev.record(main)
                    step_done.append(ev)
                    down.wait_event(ev)
                    with torch.cuda.stream(down):
                        dst_host[k * slot:(k + 1) * slot].copy_(o, non_blocking=True)
                main.wait_stream(up)
                main.wait_stream(down)
            return g
        before = cn.launch_count()
        # recorded in the order of the replays (each recording continues the look-ahead state of the one before);
        # replay q writes host buffer q % 2
        recorded, seg_graph = {}, []
        for q, (base, size) in enumerate(zip(starts, segs)):
            key = (base % 8, size, q % 2)
            if key not in recorded:
                recorded[key] = record(outs_host[q % 2], base, size)
            seg_graph.append(recorded[key])
        net.launches_per_recorded_step = (cn.launch_count() - before) // max(1, sum(k[1] for k in recorded))
        done = [torch.cuda.Event() for _ in range(2)]
        seen = {"loss": 0.0}
        hout = outs_host[0][:slot]
        seg_at = {st_: q for q, st_ in enumerate(starts)}

        def read_losses(q):
            for w in range(segs[q]):                         # the caller's read of every step's loss
                seen["loss"] = float(outs_host[q % 2][w * slot + rb:w * slot + rb + 4].view(torch.float32)[0])

        def replay(it):
            q = seg_at.get(it - warmup)
            if q is None:
                return
            seg_graph[q].replay()
            done[q % 2].record()
            if q > 0:
                done[(q - 1) % 2].synchronize()
                read_losses(q - 1)
        torch.cuda.synchronize()
    if graphs and not e2e:
        # the iteration counter is a single device word that every recorded step advances
        before = cn.launch_count()
        recorded, seg_graph = {}, []
        for base, size in zip(starts, segs):
            key = (base % pool, size)
            if key not in recorded:
                order = [(warmup + base + k) % pool for k in range(size + 1)]
                recorded[key] = cn.net_capture_steps(net, [dxs[k] for k in order[:size]], [dts[k] for k in order[:size]],
                                                     cfg.lr, faults=faults, reps_dev=reps, loss_dev=loss_dev,
                                                     X_next_dev=dxs[order[size]] if lookahead else None)
            seg_graph.append(recorded[key])
        net.launches_per_recorded_step = (cn.launch_count() - before) // max(1, sum(k[1] for k in recorded))
        seg_at = {st_: q for q, st_ in enumerate(starts)}

        def replay(it):
            q = seg_at.get(it - warmup)
            if q is not None:
                cn.net_replay(net, seg_graph[q])
        torch.cuda.synchronize()
    if sampler is not None:
        sampler.start()
    torch.cuda.synchronize()
    launches0 = cn.launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for it in range(warmup, total):
        if replay is not None:
            replay(it)
        else:
            one(it)
    ev1.record()
    torch.cuda.synchronize()
    if e2e and graphs and segs:
        read_losses(len(segs) - 1)                           # the last replay's losses, read like the others
    if sampler is not None:
        sampler.stop_flag.set()
    secs = ev0.elapsed_time(ev1) / 1e3
    bytes_in = int(hs[0].numel()) if e2e else 0
    bytes_out = int(hout.numel()) if e2e else 0
    launched = cn.launch_count() - launches0
    cn.net_set_iteration_counter(net, None)
    if replay is not None:
        launched = steps * getattr(net, "launches_per_recorded_step", 0)
    return secs, launched, bytes_in, bytes_out


def _stats(vals):
    v = sorted(vals)
    return {"ms": v[len(v) // 2], "ms_min": v[0], "ms_max": v[-1], "repeats": len(v)}


def overhead_legs(cn, wl, torch, cfg, la, steps, repeats):
    """Detect / decode overhead = (T_coded - T_coded,checks-off) / T_uncoded and the cost of the redundant blocks
    alone, T_checks-off / T_uncoded - 1.  Each leg is timed like the headline value: recorded steps replayed
    `steps` times, `repeats` times over; the median counts, the spread is printed.  The checks-off and uncoded
    legs launch no check kernel at all (their sums come from one plain reduction kernel)."""
    legs = {}
    for name, kw in (("coded", {}), ("checks_off", {"locate_mode": cn.LOCATE_OFF}),
                     ("uncoded", {"coded": False, "locate_mode": cn.LOCATE_OFF})):
        ls, nt = build_net(cn, wl, torch, cfg, **kw)
        times, launches = [], 0
        for _ in range(repeats):
            sec, launches, _, _ = timed_steps(cn, torch, nt, ls, cfg, wl, steps, 3, name == "coded", lookahead=la, graphs=True)
            times.append(1e3 * sec / steps)
        legs[name] = _stats(times)
        legs[name]["launches_per_step"] = launches / steps
        nt.free()
        for lay in ls:
            lay.free()
    c, o, u = legs["coded"]["ms"], legs["checks_off"]["ms"], legs["uncoded"]["ms"]
    worst = (legs["coded"]["ms_max"] - legs["checks_off"]["ms_min"]) / legs["uncoded"]["ms_min"]
    best = (legs["coded"]["ms_min"] - legs["checks_off"]["ms_max"]) / legs["uncoded"]["ms_max"]
    return {"ms_coded": c, "ms_checks_off": o, "ms_uncoded": u, "legs": legs, "steps_per_leg": steps,
            "detect_decode_overhead_pct": 100.0 * (c - o) / u,
            "detect_decode_overhead_pct_range": [100.0 * best, 100.0 * worst],
            "redundancy_cost_pct": 100.0 * (o / u - 1.0),
            "method": "recorded steps, median of %d runs of %d steps per leg" % (repeats, steps)}


def p_sweep(cn, wl, torch, cfg, la, steps, count_steps):
    """Throughput and decision counts at each soft-error probability the configuration names."""
    import dataclasses
    rows = []
    for p in cfg.p_sweep:
        cfgp = dataclasses.replace(cfg, p=p)
        ls, nt = build_net(cn, wl, torch, cfgp)
        L = len(ls)
        sec, _, _, _ = timed_steps(cn, torch, nt, ls, cfgp, wl, steps, 3, p > 0, lookahead=la, graphs=True)
        # decisions: a short run that reads every report
        mode = {"bernoulli": 1, "exactly_one": 2, "none": 0}[cfgp.fault_mode] if p > 0 else 0
        its = torch.arange(100000, 100000 + count_steps, dtype=torch.int32, device="cuda")
        reps = cn.new_reports(2 * L)
        loss_dev = torch.zeros(1, device="cuda")
        xs = [wl.layer_inputs(cfgp, k) for k in range(4)]
        dx = [(torch.tensor(a, device="cuda"), torch.tensor(b, device="cuda")) for a, b in xs]
        det = corr = fb = hit_phases = 0
        for it in range(count_steps):
            faults = [cn.make_fault(seed=cfgp.seed, layer=l, mode=mode, p=p, sigma=cfgp.sigma, iteration_dev=its[it:]) for l in range(L)]
            cn.step(nt, dx[it % 4][0], dx[it % 4][1], cfgp.lr, faults=faults, reps_dev=reps, loss_dev=loss_dev)
            for r in cn.read_reports(reps):
                det += r.n_detected_cw
                fb += r.n_fallback_cw
                corr += r.n_detected_cw - r.n_fallback_cw
                hit_phases += 1 if any(r.injected_mask) else 0
        codewords = count_steps * sum(sp.m + sp.n for sp in cfgp.layers)
        rows.append({"p": p, "ms_per_step": 1e3 * sec / steps, "layer_iterations_per_s": steps * L / sec,
                     "phases_with_a_hit_pct": 100.0 * hit_phases / (count_steps * 2 * L),
                     "detected_codewords": det, "corrected_codewords": corr, "fallback_codewords": fb,
                     "fallback_rate_per_codeword": fb / codewords, "counted_steps": count_steps})
        nt.free()
        for lay in ls:
            lay.free()
    return rows


def workload_bytes_per_step(cfg, la):
    """Algorithmic bytes of one step: the forward pass reads the (m + r_row) x n active blocks of each layer, the
    backward + update pass reads and writes every stored block once; with layer 1's next products taken in the
    update sweep its forward read drops out."""
    esz = 2 if cfg.bf16 else 4
    b = sum(sum(_workload_bytes(sp, esz)) for sp in cfg.layers)
    if la:
        b -= _workload_bytes(cfg.layers[0], esz)[0]
    return b


def workload_flops_per_step(cfg):
    return sum(2.0 * cfg.batch * (-(-s.n_out // s.m)) * (-(-s.n_in // s.n)) *
               ((s.m + s.r_row) * s.n + s.m * (s.n + s.r_col) + s.m * s.n + s.r_row * s.n + s.r_col * s.m)
               for s in cfg.layers)


def short_workload_leg(cn, wl, torch, name, steps, peak):
    """A bounded run of another configuration beside the headline one: iterations/s, step bytes / time, tensor
    TFLOP/s, detect / decode overhead."""
    cfg = wl.config(name)
    L = len(cfg.layers)
    la = cfg.batch <= 8
    ls, nt = build_net(cn, wl, torch, cfg)
    sec, launches, _, _ = timed_steps(cn, torch, nt, ls, cfg, wl, steps, 5, True, lookahead=la, graphs=True)
    nt.free()
    for lay in ls:
        lay.free()
    byts = workload_bytes_per_step(cfg, la)
    out = {"workload": name, "steps": steps, "ms_per_step": 1e3 * sec / steps, "layer_iterations_per_s": steps * L / sec,
           "launches_per_step": launches / steps, "bytes_per_step": byts,
           "step_GBs": byts * steps / sec / 1e9, "step_frac_of_hbm_peak": byts * steps / sec / 1e9 / peak}
    if cfg.batch >= 64:
        out["tflops"] = workload_flops_per_step(cfg) * steps / sec / 1e12
    out["overhead"] = overhead_legs(cn, wl, torch, cfg, la, steps, 1)
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c3")
    ap.add_argument("--scale", type=int, default=1, help="divide layer widths (for quick checks only)")
    ap.add_argument("--no-extras", action="store_true", help="skip overhead, CPU-baseline and e2e legs")
    ap.add_argument("--no-others", action="store_true", help="skip the short legs of the batched configurations")
    ap.add_argument("--no-graphs", action="store_true", help="launch every step kernel by kernel instead of replaying recorded steps")
    ap.add_argument("--no-lookahead", action="store_true",
                    help="do not take layer 1's next feedforward products in the update sweep (3-pass)")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3

    from paper_1903_01042_b200 import workloads as wl
    cfg = wl.config(args.workload, scale=args.scale)
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        if args.steps > 20:
            args.steps = 20                      # bounded sample: the oracle is deliberately slow
        run_reference(args, cfg, rank, world)
        return

    import torch
    import torch.distributed as dist
    from paper_1903_01042_b200 import codenet as cn
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    cn.lib()
    torch.cuda.set_stream(torch.cuda.Stream())   # a created stream: the default stream cannot record graphs
    L = len(cfg.layers)
    esz = 2 if cfg.bf16 else 4
    layers, net = build_net(cn, wl, torch, cfg)
    sampler = ClockSampler(local_rank) if rank == 0 else None

    # ---- main timed region: inputs resident in HBM ----
    barrier()
    la = not args.no_lookahead and cfg.batch <= 8
    secs, launches, _, _ = timed_steps(cn, torch, net, layers, cfg, wl, args.steps, args.warmup, True, sampler=sampler,
                                       lookahead=la, graphs=not args.no_graphs)
    barrier()
    secs_max = max_over_ranks(secs, world)
    value = whole_job_value(world, args.steps, L, secs_max)

    # ---- per-kernel timing of the dominant kernel, same workload, CUDA events on its stream ----
    cn.profile_enable(True)
    timed_steps(cn, torch, net, layers, cfg, wl, args.steps, 3, True, lookahead=la)
    bu_ms, bu_n = cn.profile_read(cn.KERNEL_BACKWARD_UPDATE)
    fw_ms, fw_n = cn.profile_read(cn.KERNEL_FORWARD)
    bw_ms, bw_n = cn.profile_read(cn.KERNEL_BACKWARD)
    up_ms, up_n = cn.profile_read(cn.KERNEL_UPDATE)
    cn.profile_enable(False)
    dominant = "backward_update_kernel" if cfg.batch <= 8 else "tc_backward_update_kernel"
    if not bu_n and up_n:
        # batches > 8: products and update are separate kernels; the update (read + write of every
        # stored block) is the dominant one
        bu_ms, bu_n, dominant = up_ms, up_n, "tc_update_kernel"
    peak, peak_kind = _peaks()
    fwd_b = sum(_workload_bytes(s, esz)[0] for s in cfg.layers) / L
    bu_b = sum(_workload_bytes(s, esz)[1] for s in cfg.layers) / L
    roofline = None
    if bu_n:
        ach = bu_b / (bu_ms / bu_n * 1e-3) / 1e9
        roofline = {"bound": "hbm", "kernel": dominant, "achieved": ach, "peak": peak,
                    "peak_kind": peak_kind + " copy bandwidth", "unit": "GB/s", "frac": ach / peak,
                    "traffic": _ncu_traffic(cfg.name) if args.scale == 1 else None, "bytes_per_launch": bu_b, "ms_per_launch": bu_ms / bu_n}
        if fw_n:
            fa = fwd_b / (fw_ms / fw_n * 1e-3) / 1e9
            roofline["forward_kernel"] = {"achieved": fa, "frac": fa / peak, "bytes_per_launch": fwd_b,
                                          "ms_per_launch": fw_ms / fw_n}
        bw_b = sum((s.m * (s.n + s.r_col)) * (-(-s.n_out // s.m)) * (-(-s.n_in // s.n)) * esz for s in cfg.layers)
        if bw_n:
            # backward products alone read the m x (n + r_col) active blocks
            ba = (bw_b / L) / (bw_ms / bw_n * 1e-3) / 1e9
            roofline["backward_kernel"] = {"achieved": ba, "frac": ba / peak, "bytes_per_launch": bw_b / L,
                                           "ms_per_launch": bw_ms / bw_n}
        two_pass = la and fw_n * 2 < bu_n
        # algorithmic bytes of the step (layers that take the products and the update as two kernels move more
        # than that: their extra backward read is reported beside it, not counted as useful traffic)
        step_bytes = workload_bytes_per_step(cfg, two_pass)
        if bw_n:
            roofline["extra_bytes_of_unfused_layers"] = bw_b
        roofline["passes"] = "2-pass (next feedforward products of layer 1 fused into the update sweep)" \
            if two_pass else "3-pass"
        roofline["step"] = {"bytes_per_step": step_bytes, "achieved": step_bytes * args.steps / secs / 1e9,
                            "frac": step_bytes * args.steps / secs / 1e9 / peak,
                            "frac_of_8TBs": step_bytes * args.steps / secs / 1e9 / 8000.0}

    line = {
        "metric": "coded_sgd_iterations_per_s_per_layer", "value": value, "unit": "layer-iterations/s",
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * secs_max / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16 storage, f32 accumulate" if cfg.bf16 else ("f32 storage, tf32 multiply, f32 accumulate" if cfg.batch >= 64 else "f32"),
        "data": "synthetic",
        "config": _config_dict(cfg, args), "gpu_launches": launches, "roofline": roofline,
    }

    if cfg.name == "paper":
        # context only: the paper's run includes checkpoints, roll-backs and its network; another machine
        line["paper_context"] = {"iterations_per_s": 2000.0 / 2322.0, "network_iterations_per_s_here": value / L,
                                 "note": "Table 1: 2000 iterations of the same 784-10^4-10^4-10 network in 2322 s on 38 "
                                         "Amazon EC2 m3.medium nodes, checkpoints every 200 iterations included"}
    if cfg.batch >= 64:
        flops = workload_flops_per_step(cfg)
        line["tensor"] = {"flops_per_step": flops, "achieved_tflops": flops * args.steps / secs / 1e12,
                          "note": "algorithmic flops of the three products; the small bf16 operands are staged as "
                                  "hi + lo pairs, so the tensor pipe executes up to twice the product flops"}
    if not args.no_extras:
        # ---- end to end through the public API: pinned host inputs in, loss and reports out ----
        barrier()
        e_secs, _, bi, bo = timed_steps(cn, torch, net, layers, cfg, wl, args.steps, 3, True, e2e=True, lookahead=la,
                                        graphs=not args.no_graphs)
        barrier()
        line["e2e"] = {"value": whole_job_value(world, args.steps, L, max_over_ranks(e_secs, world)),
                       "unit": "layer-iterations/s",
                       "h2d_bytes_per_step": bi, "d2h_bytes_per_step": bo,
                       "note": "every step: one pinned upload of [next input | target], the step, one download of "
                               "[reports | loss]; up to forty steps and their copies are captured in one graph of the "
                               "caller's (uploads and downloads on streams of their own), the host reads a replay's "
                               "losses from pinned memory after it has queued the next replay"
                               if not args.no_graphs else
                               "every step: one pinned upload of [next input | target], the step, one download of "
                               "[reports | loss]; the host reads step k - 1's loss after it has queued step k"}
    if rank == 0 and not args.no_extras:
        # ---- regeneration of a stored block from the code of its block-column: one launch per block, walking
        # the data grid so that every launch reads blocks the previous ones did not leave in L2 ----
        lay0, sp0 = layers[0], cfg.layers[0]
        if sp0.r_row > 0:
            esz = 2 if cfg.bf16 else 4
            blk_bytes = (-(-sp0.n_out // sp0.m)) * (-(-sp0.n_in // sp0.n)) * esz
            cn.profile_enable(True)
            n_reg = 0
            for rep_i in range(2):
                for j in range(sp0.n):
                    cn.regenerate_block(lay0, (j + rep_i) % sp0.m, j, 0)
                    n_reg += 1
            torch.cuda.synchronize()
            ms, cnt = cn.profile_read(cn.KERNEL_REGENERATE)
            cn.profile_enable(False)
            if cnt:
                byts = blk_bytes * (sp0.m + 1)          # m source blocks read, one block written
                ga = byts / (ms / cnt * 1e-3) / 1e9
                line["regenerate"] = {"us_per_block": 1e3 * ms / cnt, "bytes_per_launch": byts, "achieved": ga,
                                      "unit": "GB/s", "frac": ga / peak, "launches": int(cnt),
                                      "note": "block (i, j) rebuilt from the other blocks of block-column j; "
                                              "the blocks are intact here, so the weights do not change beyond rounding"}
        # ---- checkpoint / roll-back: the copy kernels timed with CUDA events, and the paper's expected-time
        # model (Theorem 2) evaluated with the times measured here ----
        try:
            from paper_1903_01042_b200 import rollback_model as rbm
            for lay in layers:
                cn.checkpoint_save(lay)             # the first save allocates
            torch.cuda.synchronize()
            evs = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
            evs[0].record()
            for lay in layers:
                cn.checkpoint_save(lay)
            evs[1].record()
            for lay in layers:
                cn.checkpoint_restore(lay)
            evs[2].record()
            torch.cuda.synchronize()
            t_cpt, t_res = evs[0].elapsed_time(evs[1]) * 1e-3, evs[1].elapsed_time(evs[2]) * 1e-3
            stored = 0
            for sp_ in cfg.layers:
                b_r, b_c = -(-sp_.n_out // sp_.m), -(-sp_.n_in // sp_.n)
                nodes_ = (sp_.m + sp_.r_row) * (sp_.n + sp_.r_col) - sp_.r_row * sp_.r_col
                stored += nodes_ * b_r * b_c * (2 if cfg.bf16 else 4)
            tau_f = secs / args.steps
            n_nodes = max((sp_.m + sp_.r_row) * (sp_.n + sp_.r_col) - sp_.r_row * sp_.r_col for sp_ in cfg.layers)
            p_node = cfg.p if cfg.p > 0 else 1e-3
            p0_, p1_ = rbm.node_probabilities(p_node, n_nodes, L, t=1)
            tau_b = t_res + tau_f                   # a roll-back: the restore, then the iteration again
            i_cn, t_cn = rbm.best_period(1.0, p0_, p1_, tau_f, tau_b, t_cpt)
            i_rep, t_rep = rbm.best_period(1.0, p0_, 0.0, tau_f, tau_b, t_cpt)
            line["rollback"] = {"checkpoint_us": 1e6 * t_cpt, "restore_us": 1e6 * t_res, "stored_bytes": stored,
                                "copy_GBs": 2 * stored / t_cpt / 1e9,
                                "model": {"p_node": p_node, "p0": p0_, "p1": p1_, "tau_f_us": 1e6 * tau_f,
                                          "tau_b_us": 1e6 * tau_b, "tau_cpt_us": 1e6 * t_cpt,
                                          "best_period_codenet": i_cn, "best_period_detect_only": i_rep,
                                          "expected_us_per_iteration_codenet": 1e6 * t_cn,
                                          "expected_us_per_iteration_detect_only": 1e6 * t_rep,
                                          "ratio": t_rep / t_cn},
                                "note": "device-to-device checkpoint of the coded blocks and inner checksums; the model "
                                        "is the paper's Theorem 2 with the times measured here (tau_b = restore + one "
                                        "iteration; single-error patterns count as correctable)"}
        except Exception as exc:                    # an extra: never fail the bench line
            line["rollback"] = {"error": str(exc)[:200]}
        # ---- detect/decode overhead: coded with checks vs coded without checks vs uncoded ----
        for lay in layers:
            lay.free()
        ksteps = max(200, min(1000, args.steps))
        line["overhead"] = overhead_legs(cn, wl, torch, cfg, la, ksteps, 3)
        # ---- the error-rate sweep the configuration names, with the fallback rate at each rate ----
        if cfg.p_sweep:
            try:
                line["p_sweep"] = p_sweep(cn, wl, torch, cfg, la, max(100, min(300, args.steps)), 100 if cfg.batch <= 8 else 30)
            except Exception as exc:
                line["p_sweep"] = {"error": str(exc)[:200]}
        # ---- the batched configurations beside the headline one (bounded legs) ----
        if cfg.name == "c3" and args.scale == 1 and not args.no_others:
            others = {}
            for name in ("c4", "c5"):
                try:
                    others[name] = short_workload_leg(cn, wl, torch, name, 100, peak)
                except Exception as exc:
                    others[name] = {"error": str(exc)[:200]}
                _WEIGHTS.clear()
            line["other_workloads"] = others
        # ---- CPU baseline: the oracle as it stands, bounded sample, this host's cores ----
        from oracle import oracle as orc
        cores = os.cpu_count() or 1
        orc.set_threads(cores)
        sp = cfg.layers[0]
        W = wl.weights(sp.n_out, sp.n_in, seed=cfg.seed, bf16=cfg.bf16)
        Pr, Pc = (wl.layer_codes(sp, cfg.seed, 0) if sp.gaussian_code else (None, None))
        ol = orc.Layer(W, sp.m, sp.n, sp.r_row, sp.r_col, P_row=Pr, P_col=Pc, store_bf16=cfg.bf16,
                       check_rows=sp.check_rows, check_cols=sp.check_cols, tau_rel=3e-2 if cfg.bf16 else 1e-3)
        onet = orc.Net([ol])
        fo = [orc.make_fault(seed=cfg.seed, layer=0, mode=1, p=cfg.p, sigma=cfg.sigma)]
        n_cpu = 6
        xin = wl.gaussian_inputs(cfg.batch, sp.n_in, cfg.seed, 0)
        tin = wl.gaussian_targets(cfg.batch, sp.n_out, cfg.seed, 0)
        onet.step(xin, tin, cfg.lr, fo, 0)
        t0 = time.perf_counter()
        for it in range(1, 1 + n_cpu):
            onet.step(xin, tin, cfg.lr, fo, it)
        dt = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": n_cpu / dt, "unit": "layer-iterations/s", "cores": orc.get_threads(),
                                "kind": "oracle", "sample": "%d iterations of layer 1 of %s at full size" % (n_cpu, cfg.name)}
        if cfg.batch <= 8:      # the same oracle on one thread (two iterations; the batched layers take minutes there)
            orc.set_threads(1)
            t0 = time.perf_counter()
            for it in range(1 + n_cpu, 3 + n_cpu):
                onet.step(xin, tin, cfg.lr, fo, it)
            line["cpu_baseline"]["single_thread_value"] = 2 / (time.perf_counter() - t0)
            orc.set_threads(cores)
    if rank == 0:
        line["clocks"] = sampler.summary()
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
