#!/usr/bin/env python
"""Benchmark of the GPTQ layer solver on synthetic OPT/BLOOM-shaped layer sets.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c0..c4] [--impl reference]

One step = the whole hot path (Hessian accumulation, dampening + Cholesky-inverse factor,
blocked quantization for every grid of the workload) over every layer of the workload, inputs
resident in HBM.  Prints ONE JSON line (rank 0).  With N > 1 (torchrun) every rank solves its own
copy of the layer set (weak scaling, layers are independent units; no data-path collective).

--impl reference times the fp64 CPU oracle (as it stands) on a bounded sample of the same workload.
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

# The overlapped schedule keeps about fifteen streams busy (one chain per layer, one more per extra grid, the library's
# own side streams).  With the default of 8 hardware queues several of them share a queue and wait for each other's
# kernels; the setting is read when the CUDA context is created, so it has to be in the environment before torch starts.
os.environ.setdefault("CUDA_DEVICE_MAX_CONNECTIONS", "32")

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "gptq_weights_quantized_per_second"
UNIT = "weights/s"
DEFAULT_WORKLOAD = "c3"


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm_gbs=d["hbm_gbs"], bf16_burst=d["bf16_tflops"], bf16_sustained=d["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_burst=1590.0, bf16_sustained=1400.0, source="fallback")


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if not self.proc:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        top = sorted(sm)[len(sm) // 2:] if sm else []     # samples under load: upper half
        return dict(sm_mhz=statistics.median(top) if top else None, sm_max_mhz=max(mx) if mx else None,
                    samples=len(sm), reasons=sorted(reasons))


# ----------------------------------------------------------------------------- reference arm (CPU oracle)
def _oracle_threads():
    from threadpoolctl import threadpool_info
    return max([p.get("num_threads", 1) for p in threadpool_info()] + [1])


def _sample_inputs(L, c_s, t_s, r_s):
    """Leading c_s channels x t_s tokens of the layer's activations and r_s x c_s of its weights (seeded generator;
    the device filler, bit-identical to the host generator, is used when a GPU is present because it is ~1000x faster)."""
    import numpy as np
    try:
        import torch
        if torch.cuda.is_available():
            from paper_2210_17323_b200.synth import device as D
            X = D.fill_x(L, 0, t_s)[:, :c_s].contiguous()
            W = D.fill_w(L)[:r_s, :c_s].contiguous() if L.R * L.C <= (1 << 28) else None
            Xb = X.view(torch.int16).cpu().numpy().view(np.uint16)
            Wn = W.cpu().numpy() if W is not None else L.w(rows=np.arange(r_s))[:, :c_s]
            return Xb, Wn
    except ImportError:
        pass
    return L.x_bits(0, t_s, cols=np.arange(c_s), scales=L.scales()), L.w(rows=np.arange(r_s))[:, :c_s]


class OracleSample:
    """The oracle, as it stands, on a bounded sample of the workload: per distinct layer shape the leading
    c_s-channel sub-problem (t_s tokens, r_s rows) is solved for real and timed; the whole layer set's time is then
    extrapolated by stage work (Hessian ~ C^2 m, factor ~ C^3, quantize ~ R C^2).  Inputs are generated once."""

    def __init__(self, wl, c_s=4096, t_s=8192, r_s=128):
        self.wl, self.c_s, self.t_s, self.r_s = wl, c_s, t_s, r_s
        self.shapes = {}
        for L in wl.layers:
            key = (L.R, L.C, L.n_tokens)
            if key not in self.shapes:
                cs, ts, rs = min(L.C, c_s), min(L.n_tokens, t_s), min(L.R, r_s)
                self.shapes[key] = (L, cs, ts, rs) + _sample_inputs(L, cs, ts, rs)

    def stage_model(self, L, cs, ts, rs, t_h, t_u, t_q):
        return t_h * (L.C / cs) ** 2 * (L.n_tokens / ts) + t_u * (L.C / cs) ** 3 + t_q * (L.R / rs) * (L.C / cs) ** 2

    def run(self):
        """One pass over the sample.  Returns (seconds measured, seconds extrapolated to the layer set, notes, per-shape times)."""
        import numpy as np
        from oracle import gptq_oracle as O
        wl = self.wl
        measured, per_shape, notes = 0.0, {}, []
        for key, (L, cs, ts, rs, Xb, W) in self.shapes.items():
            t0 = time.perf_counter(); H = O.hessian_accumulate(np.zeros((cs, cs)), Xb); t_h = time.perf_counter() - t0
            t0 = time.perf_counter(); U = O.cholesky_inverse_upper(O.dampen(H, wl.damp)[0]); t_u = time.perf_counter() - t0
            t_q = 0.0
            for g in wl.grids:
                t0 = time.perf_counter()
                O.quantize_layer(W, U, g.bits, g.group_size if g.group_size <= cs else 0, g.sym, wl.block)
                t_q += time.perf_counter() - t0
            measured += t_h + t_u + t_q
            per_shape[key] = (t_h, t_u, t_q)
            notes.append(f"{L.kind}[{L.R}x{L.C}]: H on {ts} tok x {cs} ch {t_h:.2f}s, factor {cs}^2 {t_u:.2f}s, "
                         f"quantize {rs} rows x {cs} cols {t_q:.2f}s")
        total_est = sum(self.stage_model(*self.shapes[(L.R, L.C, L.n_tokens)][:4], *per_shape[(L.R, L.C, L.n_tokens)])
                        for L in wl.layers)
        return measured, total_est, notes, per_shape

    def sample_text(self, notes):
        return ("per distinct layer shape the leading sub-problem is solved and timed, then extrapolated by stage work "
                "(C^2 m, C^3, R C^2); " + "; ".join(notes))


def whole_layer_check(wl, sample, per_shape):
    """One UN-extrapolated oracle run of a whole mid-size layer (4096 x 4096, all 262144 tokens, every grid of the
    workload), next to what the sampling model predicts for it from the sample's own stage times."""
    import numpy as np
    from oracle import gptq_oracle as O
    from paper_2210_17323_b200.synth import workloads as WL
    L = WL.Layer(wl.config_id, 0, "q", 4096, 4096, wl.layers[0].n_tokens)
    try:
        import torch
        from paper_2210_17323_b200.synth import device as D
        if not torch.cuda.is_available():
            return None                      # the host generator would need minutes for 10^9 activations
        Xb = D.fill_x(L).view(torch.int16).cpu().numpy().view(np.uint16)
        W = D.fill_w(L).cpu().numpy()
    except ImportError:
        return None
    t0 = time.perf_counter(); H = O.hessian_accumulate(np.zeros((L.C, L.C)), Xb, chunk=16384); t_h = time.perf_counter() - t0
    t0 = time.perf_counter(); U = O.cholesky_inverse_upper(O.dampen(H, wl.damp)[0]); t_u = time.perf_counter() - t0
    t0 = time.perf_counter()
    for g in wl.grids:
        O.quantize_layer(W, U, g.bits, g.group_size, g.sym, wl.block)
    t_q = time.perf_counter() - t0
    # model prediction from the sampled shape with the closest C
    key = min(per_shape, key=lambda k: abs(k[1] - L.C))
    Ls, cs, ts, rs = sample.shapes[key][:4]
    model = sample.stage_model(L, cs, ts, rs, *per_shape[key])
    return dict(layer=f"{L.R}x{L.C}, {L.n_tokens} tokens, {len(wl.grids)} grid(s)", measured_s=t_h + t_u + t_q,
                stages_s=dict(hessian=t_h, factor=t_u, quantize=t_q), model_s=model,
                weights_per_s=L.R * L.C * len(wl.grids) / (t_h + t_u + t_q))


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    t_all = time.perf_counter()
    n_runs = max(1, args.steps) + max(0, args.warmup)
    # size the per-step sample so that the whole run stays within a few minutes
    c_s = 4096 if n_runs <= 8 else (3072 if n_runs <= 16 else 2048)
    sample = OracleSample(wl, c_s=c_s)
    for _ in range(args.warmup):
        sample.run()
    runs = [sample.run() for _ in range(max(1, args.steps))]
    measured = statistics.median(r[0] for r in runs)
    est = statistics.median(r[1] for r in runs)
    notes, per_shape = runs[-1][2], runs[-1][3]
    weights = wl.weights * len(wl.grids)
    v = weights / est
    cores = _oracle_threads()
    check = None if args.no_whole_layer_check else whole_layer_check(wl, sample, per_shape)
    line = dict(metric=METRIC, value=v, unit=UNIT, impl="reference", n_gpus=args.gpus, steps=args.steps,
                warmup=args.warmup, ms_per_step=measured * 1e3, higher_is_better=True, scaling="weak",
                vs_baseline=None, dtype="f64", data="synthetic",
                config=dict(workload=wl.name, layers=len(wl.layers),
                            note="each step solves a bounded sample of the workload for real (ms_per_step is that measured "
                                 "time); value is the whole layer set's weights / its time extrapolated from the sample",
                            extrapolated_s_per_workload_step=est),
                cpu_baseline=dict(value=v, unit=UNIT, cores=cores, kind="oracle", sample=sample.sample_text(notes)),
                e2e=dict(value=v, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0),
                whole_layer_check=check, wall_s=time.perf_counter() - t_all)
    print(json.dumps(line))
    return 0


# ----------------------------------------------------------------------------- our arm
def run_gpu(args, wl):
    import torch
    import torch.distributed as dist
    from paper_2210_17323_b200 import binding as B, multi
    from paper_2210_17323_b200.synth import device as D, workloads as WL

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    # each rank solves its own copy of the layer set (block index = rank -> its own seeds)
    layers = multi.rank_layers(wl.layers, rank)
    if args.no_overlap:
        args.schedule = "sequential"
    overlap = args.schedule != "sequential"
    state = []
    ws_bytes = 256
    for L in layers:
        st = dict(L=L, X=D.fill_x(L, device=dev), W=D.fill_w(L, device=dev),
                  H=torch.empty((L.C, L.C), dtype=torch.float32, device=dev),
                  U=torch.empty((L.C, L.C), dtype=torch.float32, device=dev),
                  info=torch.zeros(2, dtype=torch.int32, device=dev))
        st["ws_bytes"] = max(256, B.gptq_hessian_workspace_bytes(L.C, L.n_tokens), B.gptq_prepare_hinv_workspace_bytes(L.C),
                             *[B.gptq_quantize_workspace_bytes(L.R, L.C, g.bits, g.group_size, wl.block) for g in wl.grids])
        ws_bytes = max(ws_bytes, st["ws_bytes"])
        state.append(st)
    # Layers are independent problems.  Overlapped schedule (default): the Hessians run back to back on one
    # stream, most expensive layer first; each layer's stages 2 and 3 follow on that layer's own stream as soon
    # as its Hessian is done, so the latency-bound kernel chains of different layers fill the SMs together and
    # run beside the next Hessians.  Every layer then needs its own workspace.  Sequential schedule
    # (--no-overlap): one stream, one shared workspace, layer after layer.
    shared_ws = None
    if overlap:
        for st in state:
            st["ws"] = torch.empty(st["ws_bytes"], dtype=torch.uint8, device=dev)
    else:
        shared_ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
        for st in state:
            st["ws"] = shared_ws
    order = sorted(range(len(state)), key=lambda i: -(state[i]["L"].C ** 2) * (state[i]["L"].n_tokens + state[i]["L"].C))
    main = torch.cuda.Stream(device=dev)
    chain_streams = [torch.cuda.Stream(device=dev) if overlap else main for _ in state]
    # A layer's grids are independent once its factor exists: in the overlapped schedule every grid after the first gets
    # a stream and a stage-3 workspace of its own, so one grid's column chains run beside the other's lazy-update GEMMs.
    side_grids = overlap and not args.grids_in_turn and len(wl.grids) > 1
    for st in state:
        st["ws_g"] = [st["ws"]] * len(wl.grids)
        st["grid_streams"] = []
        if side_grids:
            L = st["L"]
            st["ws_g"] = [st["ws"]] + [torch.empty(max(256, B.gptq_quantize_workspace_bytes(L.R, L.C, g.bits, g.group_size, wl.block)),
                                                   dtype=torch.uint8, device=dev) for g in wl.grids[1:]]
            st["grid_streams"] = [torch.cuda.Stream(device=dev) for _ in wl.grids[1:]]
    torch.cuda.synchronize()

    stage_events = []                             # (layer idx, events) of the timed steps
    factor = _factor_form(args, wl)
    for st in state:                              # per layer: the factor form where it pays (more than one block of 1024 columns)
        st["factor"] = factor and B.factor_form_pays(st["L"].R, st["L"].C, len(wl.grids))

    graphs = []                                   # per layer: CUDA graphs of the three stages (launch-bound inner loops)

    def stage_fns(st):
        return ([("H", lambda: (st["H"].zero_(), B.gptq_hessian_accumulate(st["H"], st["X"], ws=st["ws"]))),
                 ("U", lambda: B.gptq_prepare_hinv(st["H"], wl.damp, U=st["U"], ws=st["ws"], dev_info=st["info"],
                                                   factor=factor and st["factor"]))] +
                [(f"Q{gi}", (lambda gi=gi, g=g: st["out"].__setitem__(gi, B.gptq_quantize_layer(
                    st["W"], st["U"], g.bits, g.group_size, g.sym, wl.block, ws=st["ws_g"][gi], factor=factor and st["factor"]))))
                 for gi, g in enumerate(wl.grids)])

    def run_stage(li, name, fn):
        if graphs:
            graphs[li][name].replay()
        else:
            fn()

    def step(record):
        done = []
        layer_order = order if overlap else range(len(state))
        evs = {li: ([torch.cuda.Event(enable_timing=True) for _ in range(4 + len(wl.grids))] if record else None)
               for li in layer_order}
        h_done = {}

        def hessian(li):
            ev = evs[li]
            with torch.cuda.stream(main):
                if record: ev[0].record(main)
                run_stage(li, *stage_fns(state[li])[0])
                if record:
                    ev[1].record(main); h_done[li] = ev[1]
                else:
                    h_done[li] = torch.cuda.Event(); h_done[li].record(main)

        def chain(li, after):
            ev, cs, fns = evs[li], chain_streams[li], stage_fns(state[li])
            with torch.cuda.stream(cs):
                cs.wait_event(after)
                if record: ev[2].record(cs)
                run_stage(li, *fns[1])
                fac_done = ev[3] if record else torch.cuda.Event()
                fac_done.record(cs)
                joins = []
                for gi, gs in enumerate(state[li]["grid_streams"], start=1):      # the other grids beside the first one
                    with torch.cuda.stream(gs):
                        gs.wait_event(fac_done)
                        run_stage(li, *fns[2 + gi])
                        joins.append(torch.cuda.Event()); joins[-1].record(gs)
                for gi in range(len(wl.grids)):
                    if gi == 0 or not state[li]["grid_streams"]:
                        run_stage(li, *fns[2 + gi])
                for e in joins:
                    cs.wait_event(e)
                end = ev[4 + len(wl.grids) - 1] if record else torch.cuda.Event()
                end.record(cs)
            done.append(end)
            if record:
                stage_events.append((li, ev))

        if args.schedule == "hessians-first":
            for li in layer_order:
                hessian(li)
            last = h_done[list(layer_order)[-1]]
            for li in layer_order:
                chain(li, last)
        elif args.schedule == "small-first":
            # cheap layers first: their Hessians back to back, their chains side by side; the most expensive layer's Hessian
            # starts when those chains have drained (a persistent Hessian launch would starve them), and its own chain
            # then has the GPU to itself
            asc = list(layer_order)[::-1]
            for li in asc[:-1]:
                hessian(li)
                chain(li, h_done[li])
            for e in done:
                main.wait_event(e)
            hessian(asc[-1])
            chain(asc[-1], h_done[asc[-1]])
        elif args.schedule == "big-last":
            # cheap layers first, each chain launched behind its Hessian; the most expensive layer's Hessian follows at once
            # (the other chains get few SMs while it runs) and its chain, the longest, then shares the GPU with what is left
            # of the others instead of running alone at the end
            for li in list(layer_order)[::-1]:
                hessian(li)
                chain(li, h_done[li])
        else:
            for li in layer_order:
                hessian(li)
                chain(li, h_done[li])
        for e in done:                            # the step ends when every layer's chain has ended
            main.wait_event(e)

    def capture_graphs():
        """Every stage of every layer becomes one CUDA graph (same kernels, same order, same buffers): the
        ~2400 small launches of a step are then issued by the GPU front end instead of the host."""
        for li, st in enumerate(state):
            gs = {}
            for name, fn in stage_fns(st):
                cg = torch.cuda.CUDAGraph()
                with torch.cuda.graph(cg):
                    fn()
                gs[name] = cg
            graphs.append(gs)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for st in state:
        st["out"] = {}
    launches_before = B.gptq_launch_count()
    step(False)                                   # first pass eager (sets kernel attributes, checks the path)
    barrier()
    launches_per_step = B.gptq_launch_count() - launches_before
    if not args.no_graphs:
        capture_graphs()
    for _ in range(args.warmup):
        step(False)
    barrier()
    for st in state:
        assert st["info"].tolist()[0] == 0, "prepare_hinv reported an error"
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    barrier()
    t0.record(main)
    for _ in range(args.steps):
        step(True)
    t1.record(main)
    barrier()
    launches = launches_per_step * args.steps     # kernels of this library in the timed region (replayed from graphs or host-issued)
    clocks = sampler.stop() if rank == 0 else None
    ms = t0.elapsed_time(t1)
    ms = multi.max_over_ranks(ms, dev)
    ms_per_step = ms / args.steps
    n_grids = len(wl.grids)
    weights_step = wl.weights * n_grids * world
    value = weights_step / (ms_per_step * 1e-3)

    # per-stage device times (rank 0), averaged over the timed steps
    per = {}
    for li, ev in stage_events:
        L = state[li]["L"]
        d = per.setdefault(li, dict(layer=L.name, hessian_ms=0.0, hinv_ms=0.0, quantize_ms=0.0))
        d["hessian_ms"] += ev[0].elapsed_time(ev[1]) / args.steps
        d["hinv_ms"] += ev[2].elapsed_time(ev[3]) / args.steps
        d["quantize_ms"] += ev[3].elapsed_time(ev[3 + n_grids]) / args.steps
    # when each layer's stages began and ended in the last timed step, in ms after the step's first launch
    timeline = []
    last_step = stage_events[-len(state):] if stage_events else []
    if last_step:
        t0 = last_step[0][1][0]
        for li, ev in last_step:
            timeline.append(dict(layer=state[li]["L"].name,
                                 hessian=[round(t0.elapsed_time(ev[0]), 1), round(t0.elapsed_time(ev[1]), 1)],
                                 factor=[round(t0.elapsed_time(ev[2]), 1), round(t0.elapsed_time(ev[3]), 1)],
                                 quantize_end=round(t0.elapsed_time(ev[3 + n_grids]), 1)))
    peaks = _peaks()
    tot = {k: sum(d[k] for d in per.values()) for k in ("hessian_ms", "hinv_ms", "quantize_ms")}
    # roofline of the dominant kernel.  Hessian: algorithmic flops C (C + 1) m per launch (symmetric half).
    hess_flops = sum(L.C * (L.C + 1) * L.n_tokens for L in layers)
    upd_flops = sum(2 * L.R * (L.C * L.C - L.C * wl.block) / 2 * n_grids for L in layers)   # lazy updates, R (C^2 - C B)
    uses_factor = {st["L"].name: st["factor"] for st in state}
    if factor:      # + per outer block of 1024 columns the product with the block's own U (triangular: half of R 1024^2 MACs)
        upd_flops += sum(L.R * 1024 * max(0, L.C - 1024) * n_grids for L in layers if uses_factor[L.name])
    # the stage sums overlap one another in the overlapped schedule, so the dominant kernel is chosen against the step
    if tot["hessian_ms"] >= tot["quantize_ms"] or tot["hessian_ms"] >= 0.3 * ms_per_step:
        ach = hess_flops / (tot["hessian_ms"] * 1e-3) / 1e12
        # DRAM traffic per launch: dram__bytes_read + dram__bytes_write of this kernel, captured at 4096, 12288, 16384 and
        # 49152 channels x 65536 tokens, is 1.39 - 1.45e-3 bytes per token and channel^2 at every size (18 % of the operand
        # fill of the CTA pairs comes from DRAM): it grows with the flops, not with the algorithmic bytes, so the full-size
        # launches' figure is that rate x C^2 x tokens
        kTrafficPerTokenChannel2 = 1.41e-3
        algo_bytes = sum(L.n_tokens * L.C * 2 + L.C * L.C * 4 for L in layers) / len(layers)
        est_traffic = sum(max(kTrafficPerTokenChannel2 * L.C * L.C * L.n_tokens, L.n_tokens * L.C * 2 + L.C * L.C * 4)
                          for L in layers) / len(layers)
        roof = dict(kernel="hessian_accumulate", bound="tensor", achieved=ach, peak=peaks["bf16_sustained"],
                    unit="TFLOP/s", frac=ach / peaks["bf16_sustained"], traffic=est_traffic,
                    traffic_note=f"bytes per launch, mean over layers = {est_traffic / algo_bytes:.1f} x algorithmic bytes (X once + H "
                                 "once); 1.41e-3 bytes per token and channel^2, from ncu captures of 4096- to 49152-channel "
                                 "launches of 65536 tokens (1.39 - 1.45e-3 at every size)",
                    peak_source=f"bf16 sustained, {peaks['source']}")
    else:
        ach = 3 * upd_flops / (tot["quantize_ms"] * 1e-3) / 1e12
        pk = peaks["bf16_sustained"]
        roof = dict(kernel="quantize_layer (lazy update contraction, fp16 pairs: executed flops = 3 x useful)", bound="tensor",
                    achieved=ach, peak=pk, unit="TFLOP/s", frac=ach / pk, traffic=None,
                    peak_source=f"bf16 sustained (kind::f16 runs at the bf16 rate), {peaks['source']}")

    # every stage against the roofline that bounds it (CUDA events around the stage's launches; in the overlapped
    # schedules the stages of different layers run side by side, so these are in-context rates)
    f16_peak = peaks["bf16_sustained"]           # kind::f16 instructions run at the bf16 rate
    fac_flops = sum((1.0 if uses_factor[L.name] else 2.0) * L.C ** 3 / 3.0 for L in layers)
    hess_ach = hess_flops / (tot["hessian_ms"] * 1e-3) / 1e12
    fac_ach = fac_flops / (tot["hinv_ms"] * 1e-3) / 1e12
    upd_ach = upd_flops / (tot["quantize_ms"] * 1e-3) / 1e12
    stage_rooflines = [
        dict(stage="hessian_accumulate", bound="tensor", dtype="bf16", achieved=hess_ach, peak=peaks["bf16_sustained"],
             unit="TFLOP/s", frac=hess_ach / peaks["bf16_sustained"], flops="algorithmic C (C + 1) m"),
        dict(stage="prepare_hinv", bound="tensor", dtype="fp16 pairs, 3 products per term", achieved=fac_ach, executed=3 * fac_ach,
             peak=f16_peak, unit="TFLOP/s", frac=3 * fac_ach / f16_peak, useful_frac=fac_ach / f16_peak,
             flops=("useful C^3 / 3 for the layers in the factor form (the backwards factorisation alone), 2 C^3 / 3 for the others"
                    if factor else "useful 2 C^3 / 3") +
                   "; executed = 3 x (hi*hi + hi*lo + lo*hi); the serial 128 x 128 diagonal-block chain and the "
                   "CUDA-core work inside an outer panel are inside this time"),
        dict(stage="quantize_layer", bound="tensor", dtype="fp16 pairs, 3 products per term", achieved=upd_ach, executed=3 * upd_ach,
             peak=f16_peak, unit="TFLOP/s", frac=3 * upd_ach / f16_peak, useful_frac=upd_ach / f16_peak,
             flops="useful R (C^2 - C B) per grid (lazy updates)" + (" + R C 1024 (the blocks' own U, factor form)" if factor else "") +
                   "; the column chains, packing and grids are inside this time"),
    ]
    for r in stage_rooflines:
        r["peak_source"] = f"bf16 sustained, {peaks['source']}"

    line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps, warmup=args.warmup,
                ms_per_step=ms_per_step, higher_is_better=True, scaling="weak", vs_baseline=None,
                dtype="bf16 x bf16 -> f32 (Hessian); f32 factor (fp16-pair contractions, f64 diagonal blocks); f64 working weights + f32 update sums (quantize)",
                data="synthetic",
                config=dict(workload=wl.name, layers=[l.name for l in wl.layers],
                            grids=[dict(bits=g.bits, group_size=g.group_size, sym=g.sym) for g in wl.grids],
                            block=wl.block, damp=wl.damp, calib_tokens=wl.layers[0].n_tokens,
                            form=("factor: gptq_prepare_factor + gptq_quantize_layer_factor (E = (W - Q) U~; "
                                  "the factor's inverse is never formed); inverse form for: " +
                                  (", ".join(n for n, f in uses_factor.items() if not f) or "no layer")) if factor
                                 else "inverse: gptq_prepare_hinv + gptq_quantize_layer (U = Cholesky(H^-1)^T)",
                            cache="inputs larger than L2 (X >= 0.4 GB per layer); no flush needed",
                            launch="CUDA graphs, one per stage per layer" if graphs else "host-issued launches",
                            schedule={"pipelined": "pipelined: Hessians back to back on one stream, each layer's stages 2-3 on its own "
                                                   "stream as soon as its Hessian is done; stage_ms are in-context times that overlap",
                                      "hessians-first": "hessians-first: all Hessians on one stream, then every layer's stages 2-3 side by "
                                                        "side on its own stream; stage 2-3 times overlap one another",
                                      "small-first": "small-first: the cheaper layers' Hessians back to back with their stages 2-3 side by side on "
                                                     "their own streams; the most expensive layer's Hessian starts when those have drained and "
                                                     "its stages 2-3 then run alone; stage 2-3 times of the cheaper layers overlap one another",
                                      "big-last": "big-last: Hessians back to back, cheapest layer first, each layer's stages 2-3 on its own "
                                                  "stream behind its Hessian; the most expensive layer's stages 2-3 run last, beside what is "
                                                  "left of the others",
                                      "sequential": "sequential: one stream, layer after layer"}[args.schedule],
                            parallelism=f"layer-set replica per GPU x{world}"),
                sec_per_layer=ms_per_step * 1e-3 / len(layers),
                stage_ms=tot, per_layer=list(per.values()), timeline=timeline,
                roofline=roof, stage_rooflines=stage_rooflines, gpu_launches=int(launches), clocks=clocks)

    if rank == 0 and world == 1 and not args.no_e2e:
        shared_ws = None                          # the host-buffer call brings its own device workspace
        line["e2e"] = run_e2e(args, wl, state, value)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        smp = OracleSample(wl)
        measured, est, notes, _ = smp.run()
        line["cpu_baseline"] = dict(value=wl.weights * n_grids / est, unit=UNIT, cores=_oracle_threads(), kind="oracle",
                                    sample=smp.sample_text(notes), sample_seconds=measured)
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


def run_gpu_strong(args, wl):
    """Strong scaling of the SAME layer set over the ranks (paper_2210_17323_b200/multi.py): every layer's calibration tokens
    are sharded over the ranks, each rank accumulates its partial Hessian, ONE NCCL all-reduce of H per layer (a plain sum of
    local buffers) gives every rank the full matrix, the factor is computed on every rank, and each rank quantizes its
    stripe of rows.  Sequential schedule, host-issued launches.  value = the layer set's weights / the slowest rank's time."""
    import torch
    import torch.distributed as dist
    from paper_2210_17323_b200 import binding as B, multi
    from paper_2210_17323_b200.synth import device as D

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    state, ws_bytes = [], 256
    for L in wl.layers:
        tr = multi.token_shard(L.n_tokens, world, rank)
        rows = multi.shard_units(L.R, world, rank)
        Wfull = D.fill_w(L, device=dev)
        st = dict(L=L, X=D.fill_x(L, tr.start, tr.stop, device=dev), W=Wfull[rows.start:rows.stop].contiguous(), rows=rows,
                  H=torch.empty((L.C, L.C), dtype=torch.float32, device=dev),
                  U=torch.empty((L.C, L.C), dtype=torch.float32, device=dev),
                  info=torch.zeros(2, dtype=torch.int32, device=dev), out={})
        del Wfull
        ws_bytes = max(ws_bytes, B.gptq_hessian_workspace_bytes(L.C, len(tr)), B.gptq_prepare_hinv_workspace_bytes(L.C),
                       *[B.gptq_quantize_workspace_bytes(max(1, len(rows)), L.C, g.bits, g.group_size, wl.block) for g in wl.grids])
        state.append(st)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
    comm_bytes = sum(st["L"].C ** 2 * 4 for st in state)

    def step():
        for st in state:
            multi.solve_layer_sharded(
                st["L"].n_tokens, st["L"].R, world, rank,
                hessian_of_tokens=lambda tr, st=st: (st["H"].zero_(), B.gptq_hessian_accumulate(st["H"], st["X"], ws=ws))[1],
                factor_of=lambda H, st=st: B.gptq_prepare_hinv(H, wl.damp, U=st["U"], ws=ws, dev_info=st["info"])[0],
                quantize_rows=lambda rr, U, st=st: [st["out"].__setitem__(gi, B.gptq_quantize_layer(
                    st["W"], U, g.bits, g.group_size, g.sym, wl.block, ws=ws)) for gi, g in enumerate(wl.grids)] if len(rr) else None)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    launches0 = B.gptq_launch_count()
    step(); barrier()
    launches_per_step = B.gptq_launch_count() - launches0
    for _ in range(args.warmup):
        step()
    barrier()
    for st in state:
        assert st["info"].tolist()[0] == 0, "prepare_hinv reported an error"
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    barrier()
    t0.record()
    for _ in range(args.steps):
        step()
    t1.record()
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    ms_per_step = multi.max_over_ranks(t0.elapsed_time(t1), dev) / args.steps
    n_grids = len(wl.grids)
    line = dict(metric=METRIC, value=wl.weights * n_grids / (ms_per_step * 1e-3), unit=UNIT, n_gpus=world, steps=args.steps,
                warmup=args.warmup, ms_per_step=ms_per_step, higher_is_better=True, scaling="strong", vs_baseline=None,
                dtype="bf16 x bf16 -> f32 (Hessian); f32 factor (fp16-pair contractions, f64 diagonal blocks); f64 working weights + f32 update sums (quantize)",
                data="synthetic",
                config=dict(workload=wl.name, layers=[l.name for l in wl.layers],
                            grids=[dict(bits=g.bits, group_size=g.group_size, sym=g.sym) for g in wl.grids],
                            block=wl.block, damp=wl.damp, calib_tokens=wl.layers[0].n_tokens,
                            cache="inputs larger than L2; no flush needed", launch="host-issued launches",
                            parallelism=f"tokens of every Hessian and rows of every layer sharded x{world}; one all-reduce of H per "
                                        f"layer ({comm_bytes} bytes per step), factor replicated"),
                sec_per_layer=ms_per_step * 1e-3 / len(wl.layers), gpu_launches=int(launches_per_step * args.steps), clocks=clocks)
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


def run_block_sweep(args, wl):
    """Stage 3 across block sizes and forms (config 4 asks for this sweep to profile the lazy update): one layer, one
    Hessian and factor, then gptq_quantize_layer timed for B in {32, 64, 128, 256} x {row-stripe, per-inner-block} x grids."""
    import torch
    from paper_2210_17323_b200 import binding as B
    from paper_2210_17323_b200.synth import device as D

    torch.cuda.set_device(0)
    L = wl.layers[0] if not args.layer else wl.layers[0]
    X = D.fill_x(L)
    H = torch.zeros((L.C, L.C), dtype=torch.float32, device="cuda")
    B.gptq_hessian_accumulate(H, X)
    del X
    U, info = B.gptq_prepare_hinv(H, wl.damp)
    W = D.fill_w(L)
    torch.cuda.synchronize()
    assert info.tolist()[0] == 0
    peaks = _peaks()
    rows = []
    for g in wl.grids:
        base = None
        for blk in (32, 64, 128, 256):
            if g.group_size > 0 and (g.group_size % blk and blk % g.group_size):
                continue
            for variant in (1, 0):
                B.gptq_set_stage3_variant(variant)
                ws = torch.empty(B.gptq_quantize_workspace_bytes(L.R, L.C, g.bits, g.group_size, blk), dtype=torch.uint8, device="cuda")
                out = None
                ts = []
                for it in range(max(2, args.warmup) + max(3, args.steps)):
                    e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
                    e0.record()
                    out = B.gptq_quantize_layer(W, U, g.bits, g.group_size, g.sym, blk, ws=ws)
                    e1.record(); torch.cuda.synchronize()
                    if it >= max(2, args.warmup):
                        ts.append(e0.elapsed_time(e1))
                ms = statistics.median(ts)
                if base is None:
                    base = out["qweight"].clone()
                same = float((out["qweight"] == base).float().mean().item())
                useful = L.R * (L.C * L.C - L.C * blk) / (ms * 1e-3) / 1e12
                rows.append(dict(bits=g.bits, group_size=g.group_size, block=blk,
                                 form="row-stripe" if variant == 1 else "per-inner-block", ms=ms,
                                 useful_tflops=useful, executed_tflops=3 * useful,
                                 frac_of_bf16_sustained=3 * useful / peaks["bf16_sustained"],
                                 packed_words_identical_to_first=same, loss=out["loss"].item()))
    B.gptq_set_stage3_variant(1)
    line = dict(metric="gptq_stage3_ms_by_block_size", unit="ms", value=min(r["ms"] for r in rows), n_gpus=1, higher_is_better=False,
                data="synthetic", dtype="f64 working weights; fp16-pair (3 products) f32 update sums",
                config=dict(workload=wl.name, layer=L.name, note="executed flops = 3 x useful R (C^2 - C B); peak = bf16 sustained "
                            f"({peaks['source']}): the update contractions are kind::f16 tensor-core instructions"),
                sweep=rows)
    print(json.dumps(line))
    return 0


def _factor_form(args, wl):
    """True if the run uses the factor form: asked for, in the row-stripe form of stage 3, and the workload's block and
    group sizes give outer blocks of 1024 columns."""
    if getattr(args, "form", "factor") != "factor" or getattr(args, "stage3_variant", 1) != 1:
        return False
    block = getattr(args, "block", None) or wl.block
    for g in wl.grids:
        unit = max(g.group_size if g.group_size > 0 else 0, block)
        if 1024 % unit != 0:
            return False
    return True


def run_e2e(args, wl, state, device_value):
    """Same metric end to end from HOST buffers through the package's host-input solver: every step, every layer's X and
    W cross from pinned host memory to the device (copies overlapped with the Hessian accumulation and with the other
    layers' stages), every grid is solved, and codes, scales, zeros and losses are copied back to pinned host memory."""
    import torch

    from paper_2210_17323_b200 import pipeline
    grids = [(g.bits, g.group_size, g.sym) for g in wl.grids]
    layers = [(st["W"].cpu().pin_memory(), st["X"].cpu().pin_memory()) for st in state]
    shapes = [(st["L"].R, st["L"].C, st["L"].n_tokens) for st in state]
    for st in state:                       # the device copies of the device-timed leg are not needed any more
        st["X"] = st["W"] = st["H"] = st["U"] = st["ws"] = None
    state.clear()
    torch.cuda.empty_cache()
    solver = pipeline.HostLayerSolver(shapes, grids, block=wl.block, damp=wl.damp, factor=_factor_form(args, wl))
    torch.cuda.synchronize()
    steps = max(1, min(args.steps, 5))      # each step moves every layer's activations across PCIe again (seconds)
    solver.solve(layers)                    # warm-up (kernel attributes, allocator)
    solver.solve(layers)
    t0 = time.perf_counter()
    for _ in range(steps):
        solver.solve(layers)                # returns with the results on the host: wall clock is the e2e time
    dt = (time.perf_counter() - t0) / steps
    return dict(value=wl.weights * len(wl.grids) / dt, unit=UNIT, h2d_bytes_per_step=int(solver.h2d_bytes()),
                d2h_bytes_per_step=int(solver.d2h_bytes()), ms_per_step=dt * 1e3, steps=steps,
                api="pipeline.HostLayerSolver.solve (pinned host buffers; one copy stream, the most expensive layer's activations "
                    "first, in token chunks of up to 4 GiB; Hessians accumulated chunk by chunk as the chunks land; every layer's stages "
                    f"2-3 on its own stream, replayed from a CUDA graph after the first solve, all {len(grids)} grid(s) from one Hessian "
                    "and factor and side by side; results copied back to pinned memory)")


def run_inference(args, wl):
    """Bandwidth of the inference-side kernels (packed-matrix x fp16-vector, whole-matrix dequantization) and of the
    round-to-nearest entry point on the workload's largest layer, quantized with that entry point (the kernels' speed does
    not depend on the codes)."""
    import torch
    from paper_2210_17323_b200 import binding as B
    from paper_2210_17323_b200.synth import device as D

    torch.cuda.set_device(0)
    L = max(wl.layers, key=lambda l: l.R * l.C)
    W = D.fill_w(L)
    peaks = _peaks()
    rows = []
    L2_BYTES = 126 << 20
    for g in wl.grids:
        q = B.gptq_rtn_layer(W, g.bits, g.group_size, g.sym)
        x = torch.randn(L.C, device="cuda").to(torch.float16)
        y = torch.empty(L.R, dtype=torch.float32, device="cuda")
        out = torch.empty((L.R, L.C), dtype=torch.float16, device="cuda")
        # Copies of the packed matrix that together exceed three L2 sizes, used in rotation: every launch reads codes
        # that have left the cache, and the launches run back to back, so the figure is the kernel's own time (plus
        # the gap between two launches) without the host's call overhead that a single timed launch would include.
        n_rot = max(2, -(-3 * L2_BYTES // (q["qweight"].numel() * 4)))
        qws = [q["qweight"]] + [q["qweight"].clone() for _ in range(n_rot - 1)]
        res = {}
        Ws = [W] + [W.clone() for _ in range(max(1, -(-3 * L2_BYTES // (W.numel() * 2))) - 1)]   # rotated like the codes
        for name, fn, nbytes in (
                ("rtn", lambda i: B.gptq_rtn_layer(Ws[i % len(Ws)], g.bits, g.group_size, g.sym),
                 W.numel() * 2 + q["qweight"].numel() * 4 + q["scales"].numel() * 8),
                ("matvec", lambda i: B.gptq_matvec(qws[i % n_rot], q["scales"], q["zeros"], x, L.C, g.bits, g.group_size, out=y),
                 q["qweight"].numel() * 4 + q["scales"].numel() * 8 + L.C * 2 + L.R * 4),
                ("dequantize", lambda i: B.gptq_dequantize(qws[i % n_rot], q["scales"], q["zeros"], L.C, g.bits, g.group_size, out=out),
                 q["qweight"].numel() * 4 + q["scales"].numel() * 8 + L.R * L.C * 2)):
            for i in range(max(3, args.warmup) * n_rot):
                fn(i)
            ts = []
            n = 8 * n_rot
            for _ in range(max(5, args.steps)):
                torch.cuda.synchronize()
                e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
                e0.record()
                for i in range(n):
                    fn(i)
                e1.record(); torch.cuda.synchronize()
                ts.append(e0.elapsed_time(e1) / n)
            ms = statistics.median(ts)
            res[name] = dict(ms=ms, gbs=nbytes / ms / 1e6, frac_of_hbm=nbytes / ms / 1e6 / peaks["hbm_gbs"], bytes=nbytes)
        rows.append(dict(bits=g.bits, group_size=g.group_size, **res))
        del qws, Ws
    line = dict(metric="gptq_inference_kernel_bandwidth", unit="GB/s", value=rows[0]["matvec"]["gbs"], n_gpus=1,
                higher_is_better=True, data="synthetic", dtype="packed codes -> f32 accumulate",
                config=dict(workload=wl.name, layer=L.name,
                            cache="packed matrix held in copies that together exceed 3 x L2, read in rotation, launches back to back"),
                roofline=dict(kernel="gptq_matvec", bound="hbm", achieved=rows[0]["matvec"]["gbs"], peak=peaks["hbm_gbs"],
                              unit="GB/s", frac=rows[0]["matvec"]["frac_of_hbm"], traffic=None,
                              peak_source=f"STREAM-style copy, {peaks['source']}"),
                kernels=rows)
    print(json.dumps(line))
    return 0


def run_block(args, wl):
    """Transformer-block pipeline on one GPU (paper_2210_17323_b200/pipeline.py): q, k and v read the same input, so they
    share ONE Hessian and ONE factor U; o, fc1 and fc2 have their own.  One grid (--grid) per run, as a real
    quantization run has.  Prints the block time and the solver-only time of a whole model of such blocks."""
    import torch
    from paper_2210_17323_b200 import binding as B, pipeline as P
    from paper_2210_17323_b200.synth import device as D

    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    g = wl.grids[min(args.grid, len(wl.grids) - 1)]
    groups = P.group_by_shared_input(wl.layers, lambda L: D.fill_x(L, device=dev), lambda L: D.fill_w(L, device=dev))
    solver = P.BlockSolver(groups, g.bits, g.group_size, g.sym, wl.block, wl.damp, factor=_factor_form(args, wl))
    main = solver.main
    torch.cuda.synchronize()
    graphs = {}

    def run(key, fn):
        if key in graphs:
            graphs[key].replay()
        else:
            fn()

    launches0 = B.gptq_launch_count()
    solver.enqueue(run)
    torch.cuda.synchronize()
    launches_per_step = B.gptq_launch_count() - launches0
    if not args.no_graphs:
        for key, fn in solver.stage_calls():
            cg = torch.cuda.CUDAGraph()
            with torch.cuda.graph(cg):
                fn()
            graphs[key] = cg
    for _ in range(args.warmup):
        solver.enqueue(run)
    torch.cuda.synchronize()
    solver.check()
    sampler = ClockSampler(0)
    sampler.start()
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    t0.record(main)
    for _ in range(args.steps):
        solver.enqueue(run)
    t1.record(main)
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = t0.elapsed_time(t1) / args.steps
    blocks_here = len({L.block_idx for L in wl.layers})
    model_blocks = {1: 12, 2: 32, 3: 96, 4: 70}.get(wl.config_id)     # OPT-125M, OPT-6.7B, OPT-175B, BLOOM-176B
    sec_per_block = ms * 1e-3 / blocks_here
    line = dict(metric=METRIC, value=wl.weights / (ms * 1e-3), unit=UNIT, n_gpus=1, steps=args.steps, warmup=args.warmup,
                ms_per_step=ms, higher_is_better=True, scaling="weak", vs_baseline=None, data="synthetic",
                dtype="bf16 x bf16 -> f32 (Hessian); f32 factor (fp16-pair contractions, f64 diagonal blocks); f64 working weights + f32 update sums (quantize)",
                config=dict(workload=wl.name, mode="block pipeline: q, k, v share one Hessian and one factor",
                            grid=dict(bits=g.bits, group_size=g.group_size, sym=g.sym), block=wl.block, damp=wl.damp,
                            input_groups=[[m["m"].name for m in st["members"]] for st in solver.state],
                            hessians_per_block=len(solver.state) // blocks_here,
                            launch="CUDA graphs, one per stage" if graphs else "host-issued launches"),
                sec_per_block=sec_per_block,
                model_estimate=(dict(blocks=model_blocks, solver_seconds=model_blocks * sec_per_block,
                                     note="solver only (this library's three stages) for a model of that many such blocks; the "
                                          "paper's ~4 GPU-hours for OPT-175B on one A100 cover its whole pipeline and are "
                                          "context, not a comparison") if model_blocks else None),
                gpu_launches=int(launches_per_step * args.steps), clocks=clocks)
    print(json.dumps(line))
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--no-graphs", action="store_true", help="issue every kernel launch from the host instead of replaying CUDA graphs")
    ap.add_argument("--schedule", default="pipelined", choices=["pipelined", "hessians-first", "small-first", "big-last", "sequential"],
                    help="pipelined: Hessians back to back on one stream, each layer's stages 2-3 on its own stream as soon as "
                         "its Hessian is done; hessians-first: all Hessians, then all layers' stages 2-3 side by side; "
                         "sequential: one stream, layer after layer")
    ap.add_argument("--no-overlap", action="store_true", help="same as --schedule sequential")
    ap.add_argument("--grids-in-turn", action="store_true",
                    help="overlapped schedules: run a layer's grids one after the other on the layer's stream (default: every "
                         "grid after the first on a stream and workspace of its own, beside the first)")
    ap.add_argument("--scaling", default="weak", choices=["weak", "strong"],
                    help="weak (default): every rank solves its own copy of the layer set; strong: the same layer set, tokens of "
                         "every Hessian and rows of every layer sharded over the ranks with one all-reduce of H per layer")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-whole-layer-check", action="store_true",
                    help="--impl reference: skip the one un-extrapolated whole-layer oracle run")
    ap.add_argument("--mode", default="solver", choices=["solver", "inference", "block"],
                    help="solver: the layer-solver step (default, the headline metric); inference: bandwidth of the "
                         "packed matvec / dequantize kernels; block: Transformer-block pipeline in which q, k, v share "
                         "one Hessian and one factor")
    ap.add_argument("--grid", type=int, default=0, help="--mode block: index of the workload's grid to run")
    ap.add_argument("--block", type=int, default=None, help="block size B of Algorithm 1 (default: the workload's, 128)")
    ap.add_argument("--form", default="factor", choices=["factor", "inverse"],
                    help="factor (default): stage 2 stops after the backwards factorisation and stage 3 feeds the plain residuals "
                         "back through the factor (gptq_prepare_factor / gptq_quantize_layer_factor: same results, the factor's "
                         "inverse is never formed); inverse: U = Cholesky(H^-1)^T as Algorithm 1 writes it "
                         "(gptq_prepare_hinv / gptq_quantize_layer)")
    ap.add_argument("--stage3-variant", type=int, default=1, choices=[0, 1],
                    help="form of the loops inside an outer block: 1 row-stripe kernel (default), 0 one in-block kernel plus one "
                         "small contraction per inner block")
    ap.add_argument("--block-sweep", action="store_true",
                    help="--mode sweep helper: time stage 3 of the workload's largest-Hessian layer for B in {32, 64, 128, 256} "
                         "and both forms, on one Hessian and factor")
    ap.add_argument("--layer", default=None, metavar="RxCxTOKENS",
                    help="profile one layer of this shape (grid, block and damp of --workload) instead of the "
                         "whole layer set -- a small case of the same kernels for profiler captures")
    args = ap.parse_args()
    from paper_2210_17323_b200.synth import workloads as WL
    wl = WL.workload(int(args.workload.lstrip("c")))
    if args.layer:
        R, C, T = (int(v) for v in args.layer.lower().split("x"))
        wl = WL.Workload(wl.config_id, f"{wl.name}-single-{R}x{C}x{T}", (WL.Layer(wl.config_id, 0, "q", R, C, T),),
                         wl.grids, wl.block, wl.damp)
    if args.block:
        import dataclasses
        wl = dataclasses.replace(wl, block=args.block)
    if args.impl == "reference":
        return run_reference(args, wl)
    if args.block_sweep:
        return run_block_sweep(args, wl)
    if args.stage3_variant != 1:
        from paper_2210_17323_b200 import binding as _B
        _B.gptq_set_stage3_variant(args.stage3_variant)
    if args.mode == "inference":
        return run_inference(args, wl)
    if args.mode == "block":
        return run_block(args, wl)
    if args.scaling == "strong":
        return run_gpu_strong(args, wl)
    return run_gpu(args, wl)


if __name__ == "__main__":
    sys.exit(main())
