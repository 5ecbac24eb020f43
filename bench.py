#!/usr/bin/env python
"""Benchmark of the PipeMare hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload cfg4|cfg5|cfg3|cfg1]

A step is one pipeline tick in steady state: every stage runs one forward with the weights it holds, one
backward against the discrepancy-corrected weights for the microbatch that entered it tau_i updates ago, and
the fused PipeMare update; one microbatch leaves the pipeline per tick.  The default workload is the largest
one built: the 6-layer Transformer encoder (config 4; 25 stages; a sample is one sequence of 128 tokens, 32 per
tick), which exercises every kind of stage.  The 32-stage bf16 MLP (config 3; a sample is one row, 128 per
tick) and the 4-stage fp32 MLP (config 1) are measured in the same run and reported under `other_workloads`.

`roofline` describes the kernel class with the largest share of the step, timed live with CUDA events on
the launch stream; `roofline_update` is the fused PipeMare update against the HBM peak (the second half of the
metric), also live inside the step; `update_sweep` times that kernel alone over a parameter-count sweep.

With N > 1 (launched by torch.distributed.run) every rank runs an independent replica of the same pipeline on
its own GPU: the path is not sharded in this build, no collective is on the data path, `value` is the sum
over ranks divided by the slowest rank's time.

`--impl reference` times the CPU oracle, as it stands, on the host cores.
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

METRIC = "async-pipeline train samples/s on 1 B200; PipeMare update GB/s vs HBM peak"
UNIT = "samples/s"
BYTES_PER_PARAM = {"sgdm": 30, "adam": 38}     # fp32 g,w,m,delta read + w,m,delta write + bf16 copy (+ s r/w)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), "measured"
    return 6650.0, 1400.0, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc, self.first = index, [], None, 0

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def wait_first(self, timeout=3.0):
        t0 = time.time()
        while self.proc is not None and not self.rows and time.time() - t0 < timeout:
            time.sleep(0.02)

    def mark(self):
        """Samples taken before this point (start-up, pipeline fill) are not reported."""
        self.first = max(len(self.rows) - 1, 0)

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows[self.first:]:
            if len(r) < 6:
                continue
            try:
                sm.append(float(r[0]))
                mx = float(r[1])
            except ValueError:
                continue
            for name, v in zip(names, r[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


def dist_setup(n_gpus):
    import torch
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        backend = "nccl" if torch.cuda.is_available() else "gloo"
        if not dist.is_initialized():
            dist.init_process_group(backend=backend)
    return world, rank, local


def reduce_over_ranks(elapsed_ms, units, world, device=None):
    """Slowest rank's time and the total number of units processed by all ranks."""
    if world == 1:
        return elapsed_ms, units
    import torch
    import torch.distributed as dist
    t = torch.tensor([elapsed_ms], dtype=torch.float64, device=device)
    u = torch.tensor([float(units)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def barrier(world):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


# ---- the CUDA arm ---------------------------------------------------------------------------------

WORKLOADS = {
    "cfg1": "cfg1: 4-stage MLP, 1 Linear(256,256)+ReLU per stage, fp32 (SIMT GEMMs), microbatch 32, SGD momentum 0.9, "
            "T1 (K=32) + T2 (D=0.5), tau=(7,5,3,1)",
    "cfg3": "cfg3: 32-stage MLP, 2x Linear(1024,1024)+GELU per stage, bf16 GEMMs, fp32 master weights, microbatch 128, "
            "SGD momentum 0.9, T1 (K=125) + T2 (D=0.5), tau_i=2(32-i)+1",
    "cfg5": "cfg5 cut to 7 + 7 layers: Transformer encoder-decoder, d_model 1024, 16 heads, FFN 4096, 16 sequences x 256 "
            "tokens per microbatch, vocabulary 32000 (Zipf ids), bf16 GEMMs, fp32 master weights, one stage per weight GEMM "
            "(78 stages), Adam(0.9, 0.98), T1 (K=1000) + T2 (D=0.1), tau_i=2(78-i)+1; 166 GB on the device; the full "
            "12 + 12 layers (133 stages) need more than 450 GB of activation rings",
    "cfg4": "cfg4: Transformer encoder, 6 layers, d_model 512, 8 heads, FFN 2048, 32 sequences x 128 tokens per "
            "microbatch, vocabulary 8192, bf16 GEMMs, fp32 master weights, one stage per weight GEMM (25 stages), "
            "Adam(0.9, 0.98), T1 (K=100) + T2 (D=0.1), tau_i=2(25-i)+1",
}


def build_workload(args):
    """Workload description, initial parameters, samples per step and parameter count."""
    import pm_inputs as I
    if args.workload == "cfg4":
        wl = I.cfg4()
        if args.stages:      # profiler captures only: fewer layers of the same shape, not a bench result
            wl = I.encoder_workload(wl.name + f"_{args.stages}layers", args.stages, 512, 8, 2048, 128, 32, 8192, compute="bf16",
                                    optimizer="adam", alpha=wl.alpha, beta1=0.9, beta2=0.98, eps=1e-8, K=wl.K, D=wl.D,
                                    steps=wl.steps, seed=wl.seed)
        params0 = I.init_encoder_params(wl)
        n_params = sum(int(a.size) for st in params0 for a in st)
        return wl, params0, wl.microbatch // wl.seq_len, n_params
    if args.workload == "cfg5":
        wl = I.cfg5_cut(args.stages, args.stages) if args.stages else I.cfg5_cut()
        params0 = I.init_encoder_params(wl)
        n_params = sum(int(a.size) for st in params0 for a in st)
        return wl, params0, wl.microbatch // wl.seq_len, n_params
    if args.workload == "cfg1":
        wl = I.cfg1()
        params0 = I.init_stage_params(wl)
        return wl, params0, wl.microbatch, sum(sp.n_in * sp.n_out + sp.n_out for st in wl.stages for sp in st)
    wl = I.cfg3()
    if args.stages:          # profiler captures only: fewer stages of the same shape, not a bench result
        wl = I.mlp_workload(wl.name + f"_first{args.stages}", args.stages, 1024, 2, "gelu", wl.microbatch, compute="bf16",
                            optimizer=wl.optimizer, alpha=wl.alpha, beta1=wl.beta1, K=wl.K, D=wl.D, steps=wl.steps,
                            seed=wl.seed)
    params0 = I.init_stage_params(wl)
    n_params = sum(sp.n_in * sp.n_out + sp.n_out for st in wl.stages for sp in st)
    return wl, params0, wl.microbatch, n_params


def make_batches(wl, n, device):
    import torch
    import pm_inputs as I
    if wl.kind == "encoder":
        import numpy as np
        host = []
        encdec = any(sp.pre == "embed_dec" for sp in wl.stage_specs)
        for t in range(n):
            if encdec:                                         # two token streams: [source | decoder input]
                src, dec_in, tg = I.seq2seq_batch(wl, t)
                ids = np.concatenate([src, dec_in])
            else:
                ids, tg = I.token_batch(wl, t)
            host.append((torch.from_numpy(ids.astype(np.int32)).pin_memory(), torch.from_numpy(tg.astype(np.int32)).pin_memory()))
        return host, [(x.to(device), y.to(device)) for x, y in host]
    teacher = I.teacher_params(wl)
    xs, ys = [], []
    for t in range(n):
        x, y = I.batch(wl, t, teacher)
        xs.append(torch.from_numpy(x))
        ys.append(torch.from_numpy(y))
    in_dtype = torch.bfloat16 if wl.compute == "bf16" else torch.float32
    host = [(x.to(in_dtype).pin_memory(), y.pin_memory()) for x, y in zip(xs, ys)]
    dev = [(x.to(device), y.to(device)) for x, y in host]
    return host, dev


def cpu_baseline(wl, n_steps, samples_per_step):
    """The oracle, as it stands, on this machine's host cores."""
    import pm_inputs as I
    if wl.kind == "encoder":
        from oracle.transformer import run_workload
        params0 = I.init_encoder_params(wl)
        encdec = any(sp.pre == "embed_dec" for sp in wl.stage_specs)
        batches = [I.seq2seq_batch(wl, t) if encdec else I.token_batch(wl, t) for t in range(n_steps)]
    else:
        from oracle.mlp import run_workload
        params0 = I.init_stage_params(wl)
        teacher = I.teacher_params(wl)
        batches = [I.batch(wl, t, teacher) for t in range(n_steps)]
    t0 = time.perf_counter()
    run_workload(wl, params0, lambda t: batches[t], n_steps=n_steps)
    dt = time.perf_counter() - t0
    return {"value": samples_per_step * n_steps / dt, "unit": UNIT, "cores": os.cpu_count(), "kind": "oracle",
            "sample": f"{n_steps} microbatch steps of the {wl.name} workload (forward, backward, update of all "
                      f"{wl.n_stages} stages), {dt:.1f} s"}


def update_sweep(device, peak_gbs, quick=False):
    """Stand-alone fused update over a parameter-count sweep; cold L2 by rotating arena sets."""
    import torch
    import paper_1910_05124_b200 as pm
    import pm_inputs as I
    out = []
    sizes = [1_000_000, 10_000_000, 100_000_000] + ([] if quick else [1_000_000_000])
    for opt in ("sgdm", "adam"):
        for n in sizes:
            for P in (8, 64, 512):
                base, rem = divmod(n, P)
                counts = [base + (1 if i < rem else 0) for i in range(P)]
                offsets, cur = [], 0
                for c in counts:
                    offsets.append(cur)
                    cur += -(-c // 64) * 64
                total = cur
                tau_f, tau_b = I.pipemare_delays(P)
                bpp = BYTES_PER_PARAM[opt]
                sets = max(1, min(16, -(-400_000_000 // (bpp * n))))      # > 2x L2 touched between reuses
                arenas = []
                g = torch.Generator(device=device)
                g.manual_seed(1910 + P)
                for _ in range(sets):
                    w = torch.randn(total, device=device, generator=g)
                    gr = torch.randn(total, device=device, generator=g) * 1e-3
                    m = torch.randn(total, device=device, generator=g) * 1e-3
                    dl = torch.randn(total, device=device, generator=g) * 1e-4
                    s = (torch.randn(total, device=device, generator=g) * 1e-3) ** 2 if opt == "adam" else None
                    lp = torch.empty(total, dtype=torch.bfloat16, device=device)
                    arenas.append((w, m, s, dl, gr, lp))
                fu = pm.FlatUpdate(offsets, counts, tau_f, tau_b, optimizer=opt, alpha=0.01 if opt == "sgdm" else 5e-4,
                                   K=64, D=0.5, device=device)
                iters = 20
                for i in range(3):
                    fu.pm_update_flat(*arenas[i % sets], 32)
                torch.cuda.synchronize()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for i in range(iters):
                    fu.pm_update_flat(*arenas[i % sets], 32)
                e1.record()
                torch.cuda.synchronize()
                ms = e0.elapsed_time(e1) / iters
                gbs = bpp * n / (ms * 1e-3) / 1e9
                out.append({"n_params": n, "P": P, "optimizer": opt, "ms": round(ms, 5), "GB/s": round(gbs, 1),
                            "frac_of_measured_peak": round(gbs / peak_gbs, 4), "arena_sets": sets})
                del arenas, fu
                torch.cuda.empty_cache()
    return out


def run_update_only(args):
    """A few launches of the stand-alone fused update on one arena set (for profiler captures)."""
    import torch
    import paper_1910_05124_b200 as pm
    import pm_inputs as I
    device = torch.device("cuda:0")
    n, P = args.update_only, 64
    base, rem = divmod(n, P)
    counts = [base + (1 if i < rem else 0) for i in range(P)]
    offsets, cur = [], 0
    for c in counts:
        offsets.append(cur)
        cur += -(-c // 64) * 64
    tau_f, tau_b = I.pipemare_delays(P)
    g = torch.Generator(device=device)
    g.manual_seed(1910)
    w = torch.randn(cur, device=device, generator=g)
    gr = torch.randn(cur, device=device, generator=g) * 1e-3
    m = torch.randn(cur, device=device, generator=g) * 1e-3
    dl = torch.randn(cur, device=device, generator=g) * 1e-4
    lp = torch.empty(cur, dtype=torch.bfloat16, device=device)
    fu = pm.FlatUpdate(offsets, counts, tau_f, tau_b, optimizer="sgdm", alpha=0.01, K=64, D=0.5, device=device)
    for _ in range(3):
        fu.pm_update_flat(w, m, None, dl, gr, lp, 32)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(max(args.steps, 1)):
        fu.pm_update_flat(w, m, None, dl, gr, lp, 32)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / max(args.steps, 1)
    print(json.dumps({"update_only": {"n_params": n, "P": P, "ms": ms, "GB/s": 30 * n / (ms * 1e-3) / 1e9}}), flush=True)


def gemm_flops(wl):
    """Algorithmic FLOPs of one tick per GEMM class: 2*T*in*out per Linear; the first Linear of a network fed raw
    inputs has no input gradient."""
    T = wl.microbatch
    if wl.kind == "encoder":
        lin = [(sp.n_in, sp.n_out) for sp in wl.stage_specs]
        first_needs_dgrad = True            # the embedding needs the gradient of its output
    else:
        lin = [(sp.n_in, sp.n_out) for st in wl.stages for sp in st]
        first_needs_dgrad = False
    full = sum(2.0 * T * a * b for a, b in lin)
    dgrad = full if first_needs_dgrad else full - 2.0 * T * lin[0][0] * lin[0][1]
    return {"gemm_fwd": full, "wgrad": full, "dgrad": dgrad}


def gemm_bytes(wl):
    """Algorithmic HBM bytes of one tick per GEMM class on the bf16 path: every operand read once, every result
    written once (bf16 activations, fp32 weights / discrepancy / gradient, fp32 logits under cross-entropy)."""
    T = wl.microbatch
    if wl.kind == "encoder":
        lin = [(sp.n_in, sp.n_out, sp.act) for sp in wl.stage_specs]
        gaps = [f - b for f, b in zip(wl.tau_fwd, wl.tau_bkwd)]
        logits_f32 = True
    else:
        lin = [(sp.n_in, sp.n_out, sp.act) for st in wl.stages for sp in st]
        gaps = [f - b for st, f, b in zip(wl.stages, wl.tau_fwd, wl.tau_bkwd) for _ in st]
        logits_f32 = False
    fwd = wgrad = dgrad = 0.0
    for j, ((a, b, act), gap) in enumerate(zip(lin, gaps)):
        last = j == len(lin) - 1
        # z stash and activation y; a ReLU that is not the very last Linear stashes only y
        out_b = 4 if (last and logits_f32) else 2 * (2 if (act == "gelu" or (act == "relu" and last)) else 1)
        fwd += 2.0 * T * a + 2.0 * a * b + out_b * T * b
        wgrad += 2.0 * T * a + 2.0 * T * b + 4.0 * a * b
        if j > 0 or wl.kind == "encoder":
            dgrad += 2.0 * T * b + (8.0 if (wl.t2 and gap > 0) else 4.0) * a * b + 2.0 * T * a
    return {"gemm_fwd": fwd, "wgrad": wgrad, "dgrad": dgrad}


# DRAM traffic per launch from ncu captures summarised under profiles/ (bytes); scaled to the benchmark workload by
# the stated unit counts because the full-size workloads hold more device memory than a multi-pass capture may.
NCU_TRAFFIC = {
    # GEMM kernels: measured DRAM bytes / algorithmic bytes on the 2-layer cut of cfg4
    # (profiles/gemm_and_attention_kernels_cfg4_2layer_cut.md); every operand crosses HBM once, so traffic grows
    # with the algorithmic bytes of the launch
    "gemm_fwd_ratio": (84.2 + 149.1) / (83.9 + 209.7),
    "wgrad_ratio": (211.1 + 24.9) / (205.5 + 42.0),
    "dgrad_ratio": (231.8 + 29.2) / (226.5 + 33.6),
    # fused update: 2.941 GB at 100 M parameters, momentum SGD (profiles/update_kernel_100M_params.md); pure streaming,
    # so it is scaled by the algorithmic bytes of the launch (30 B/param there; 38 B/param with Adam's second moment)
    "update_bytes_per_param": 29.41,
}


def measure(args, workload, world, rank, local, device, sampler=None, with_e2e=True):
    """Runs one workload: K timed steps with inputs resident in HBM, K profiled steps (per-class CUDA events), and
    K end-to-end steps from pinned host buffers.  Returns a dict of results (rank 0 consumes it)."""
    import torch
    import paper_1910_05124_b200 as pm
    a2 = argparse.Namespace(**vars(args))
    a2.workload = workload
    wl, params0, samples_per_step, n_params = build_workload(a2)
    P = wl.n_stages
    pipe = pm.Pipeline(wl, params0, device=str(device))
    host_b, dev_b = make_batches(wl, 4, device)
    warm = max(args.warmup, 3)
    fill = 2 * P - 1
    for s in range(fill + warm):
        pipe.pm_step(*dev_b[s % len(dev_b)])
    torch.cuda.synchronize(device)

    # ---- timed region 1: K steps, inputs resident in HBM
    if sampler is not None:
        sampler.wait_first()
        sampler.mark()
    launches0 = pipe.pm_launch_count()
    barrier(world)
    torch.cuda.synchronize(device)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for s in range(args.steps):
        pipe.pm_step(*dev_b[s % len(dev_b)])
    e1.record()
    torch.cuda.synchronize(device)
    barrier(world)
    elapsed_ms = e0.elapsed_time(e1)
    launches = pipe.pm_launch_count() - launches0
    t_ms, units = reduce_over_ranks(elapsed_ms, samples_per_step * args.steps, world, device)

    # ---- timed region 2: the same K steps with CUDA events around every launch (on the launch stream)
    pipe.pm_profile_enable(True)
    for s in range(args.steps):
        pipe.pm_step(*dev_b[s % len(dev_b)])
    prof = pipe.pm_profile_read()
    pipe.pm_profile_enable(False)
    clocks = sampler.stop() if sampler is not None else None
    per_tick = {k: v[0] / args.steps for k, v in prof.items() if v[1] > 0}
    total_prof = sum(per_tick.values())

    res = {"wl": wl, "P": P, "fill": fill, "samples_per_step": samples_per_step, "n_params": n_params,
           "t_ms": t_ms, "units": units, "launches": launches, "clocks": clocks, "per_tick_ms": per_tick,
           "ring_bytes": pipe.ring_bytes, "state_bytes": pipe.state_bytes, "prof": prof, "total_prof": total_prof}

    # ---- timed region 3: end to end through the C ABI with host buffers
    if with_e2e:
        xin = torch.empty_like(dev_b[0][0])
        yin = torch.empty_like(dev_b[0][1])
        barrier(world)
        torch.cuda.synchronize(device)
        loss_sink = 0.0
        t0 = time.perf_counter()
        for s in range(args.steps):
            hx, hy = host_b[s % len(host_b)]
            xin.copy_(hx, non_blocking=True)
            yin.copy_(hy, non_blocking=True)
            pipe.pm_step(xin, yin)
            # loss of the microbatch whose backward started this tick: device -> host, synchronises
            mb_done = fill + warm + 2 * args.steps + s - P
            loss_sink += float(pipe.pm_get_losses(mb_done, 1)[0])
        torch.cuda.synchronize(device)
        e2e_ms = (time.perf_counter() - t0) * 1e3
        barrier(world)
        e2e_t, e2e_units = reduce_over_ranks(e2e_ms, samples_per_step * args.steps, world, device)
        res.update(e2e_t=e2e_t, e2e_units=e2e_units, h2d=sum(x.numel() * x.element_size() for x in host_b[0]),
                   last_loss=loss_sink / args.steps)
    pipe.close()
    del pipe
    torch.cuda.empty_cache()
    return res


def rooflines(res, hbm_peak, tf_peak, peak_kind, steps):
    """Roofline objects: the dominant kernel class of the step, and the fused update against HBM."""
    wl, per_tick = res["wl"], res["per_tick_ms"]
    step_ms = res["t_ms"] / steps
    upd_ms = per_tick.get("update", 0.0)
    alg_bytes = BYTES_PER_PARAM[wl.optimizer] * res["n_params"]
    upd_gbs = alg_bytes / (upd_ms * 1e-3) / 1e9 if upd_ms > 0 else 0.0
    update = {"kernel": "update_kernel (fused PipeMare update)", "bound": "hbm", "achieved": round(upd_gbs, 1),
              "peak": hbm_peak, "unit": "GB/s", "frac": round(upd_gbs / hbm_peak, 4), "of": peak_kind,
              "traffic": int(NCU_TRAFFIC["update_bytes_per_param"] * alg_bytes / 30.0),
              "algorithmic_bytes_per_launch": alg_bytes, "avg_launch_ms": round(upd_ms, 5),
              "frac_of_nominal_8TBs": round(upd_gbs / 8000.0, 4), "share_of_step": round(upd_ms / res["total_prof"], 4)}
    dominant = max(per_tick, key=per_tick.get)
    if dominant == "update":
        return update, update
    flops = gemm_flops(wl)
    if dominant in flops and wl.compute == "f32":
        # fp32 path: plain FFMA on the CUDA cores; peak derived from unit counts and clocks:
        # 148 SMs x 128 lanes x 2 flop x 1.965 GHz = 74.4 TFLOP/s
        tfs = flops[dominant] / (per_tick[dominant] * 1e-3) / 1e12
        dom = {"kernel": "simt_gemm_kernel (" + dominant + ")", "bound": "alu", "achieved": round(tfs, 3), "peak": 74.4,
               "unit": "TFLOP/s", "frac": round(tfs / 74.4, 5), "of": "derived (148 SMs x 128 FFMA lanes x 1.965 GHz)",
               "traffic": None, "avg_ms_per_step": round(per_tick[dominant], 5),
               "share_of_step": round(per_tick[dominant] / res["total_prof"], 4),
               "note": "46 MFLOP per step: launch-latency bound, not arithmetic bound"}
        return dom, update
    if dominant in flops:
        launches = res["prof"][dominant][1] / steps
        tfs = flops[dominant] / (per_tick[dominant] * 1e-3) / 1e12
        names = {"gemm_fwd": "umma_pair_gemm_kernel<0> / umma_gemm_kernel<0> (forward GEMMs)",
                 "wgrad": "umma_pair_gemm_kernel<2> / umma_gemm_kernel<2> (wgrad GEMMs)",
                 "dgrad": "umma_dgrad_pair_kernel / umma_dgrad_kernel (dgrad GEMMs, weights corrected while loading)"}
        dom = {"kernel": names[dominant], "bound": "tensor", "achieved": round(tfs, 1), "peak": tf_peak, "unit": "TFLOP/s",
               "frac": round(tfs / tf_peak, 4), "of": peak_kind + " (sustained bf16 matmul)",
               "traffic": int(NCU_TRAFFIC[dominant + "_ratio"] * gemm_bytes(wl)[dominant] / launches),
               "traffic_note": "DRAM bytes per launch, scaled from the ncu capture of the 2-layer cut by algorithmic bytes",
               "algorithmic_bytes_per_step": gemm_bytes(wl)[dominant],
               "algorithmic_flops_per_step": flops[dominant], "launches_per_step": launches,
               "avg_ms_per_step": round(per_tick[dominant], 5), "frac_of_nominal_2250TFs": round(tfs / 2250.0, 4),
               "share_of_step": round(per_tick[dominant] / res["total_prof"], 4)}
        return dom, update
    dom = {"kernel": dominant, "bound": "alu", "achieved": None, "peak": None, "unit": None, "frac": None, "traffic": None,
           "avg_ms_per_step": round(per_tick[dominant], 5), "share_of_step": round(per_tick[dominant] / res["total_prof"], 4)}
    return dom, update


def run_cuda(args):
    import torch
    world, rank, local = dist_setup(args.gpus)
    device = torch.device(f"cuda:{local}")
    torch.cuda.set_device(device)
    hbm_peak, tf_peak, peak_kind = measured_peaks()
    sampler = ClockSampler(local) if rank == 0 else None
    if sampler is not None:
        sampler.start()
    res = measure(args, args.workload, world, rank, local, device, sampler)
    others = []
    if world == 1 and not args.no_other and not args.stages:
        for name in ("cfg5", "cfg4", "cfg3", "cfg1"):
            if name != args.workload:
                try:
                    others.append((name, measure(args, name, world, rank, local, device, None, with_e2e=False)))
                except RuntimeError as exc:                  # e.g. cfg5's 166 GB on a device that has less free
                    import torch
                    torch.cuda.empty_cache()
                    others.append((name, {"error": str(exc).splitlines()[0][:200]}))
    if rank != 0:
        return
    wl, P = res["wl"], res["P"]
    value = res["units"] / (res["t_ms"] * 1e-3)
    dom, upd = rooflines(res, hbm_peak, tf_peak, peak_kind, args.steps)
    flops = gemm_flops(wl)
    gemm_ms = sum(res["per_tick_ms"].get(k, 0.0) for k in flops)
    line = {
        "metric": METRIC, "value": round(value, 2), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": round(res["t_ms"] / args.steps, 5), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32" if wl.compute == "f32" else "bf16", "data": "synthetic",
        "config": {"workload": WORKLOADS[args.workload] + (f" [cut to {args.stages} for profiling]" if args.stages else ""),
                   "parallelism": "replicas only" if world > 1 else f"single GPU, {P} emulated pipeline stages",
                   "samples_per_step": res["samples_per_step"], "pipeline_fill_ticks": res["fill"],
                   "cache": "per-step working set (state + rings, see state_bytes) far exceeds the 126 MB L2: no flush needed",
                   "ring_bytes": res["ring_bytes"], "state_bytes": res["state_bytes"], "params": res["n_params"]},
        "clocks": res["clocks"],
        "e2e": {"value": round(res["e2e_units"] / (res["e2e_t"] * 1e-3), 2), "unit": UNIT, "h2d_bytes_per_step": res["h2d"],
                "d2h_bytes_per_step": 4, "ms_per_step": round(res["e2e_t"] / args.steps, 5), "last_loss": res["last_loss"]},
        "gpu_launches": res["launches"],
        "roofline": dom,
        "roofline_update": upd,
        "gemm_all": {"TFLOP/s": round(sum(flops.values()) / (gemm_ms * 1e-3) / 1e12, 1) if gemm_ms > 0 else None,
                     "frac_of_measured_sustained": round(sum(flops.values()) / (gemm_ms * 1e-3) / 1e12 / tf_peak, 4) if gemm_ms > 0 else None,
                     "ms_per_step": round(gemm_ms, 5)},
        "kernel_ms_per_step": {k: round(v, 5) for k, v in sorted(res["per_tick_ms"].items(), key=lambda kv: -kv[1])},
    }
    line["other_workloads"] = []
    for name, other in others:
        if "error" in other:
            line["other_workloads"].append({"workload": WORKLOADS[name], "error": other["error"]})
            continue
        od, ou = rooflines(other, hbm_peak, tf_peak, peak_kind, args.steps)
        line["other_workloads"].append({
            "workload": WORKLOADS[name], "value": round(other["units"] / (other["t_ms"] * 1e-3), 2), "unit": UNIT,
            "ms_per_step": round(other["t_ms"] / args.steps, 5), "roofline": od, "roofline_update": ou,
            "kernel_ms_per_step": {k: round(v, 5) for k, v in sorted(other["per_tick_ms"].items(), key=lambda kv: -kv[1])}})
    if world == 1:
        if not args.no_cpu:
            line["cpu_baseline"] = cpu_baseline(wl, 2 if args.workload == "cfg3" else 1, res["samples_per_step"]) \
                if args.workload != "cfg5" else None         # one full-width cfg5 step takes minutes on the host: see --impl reference
        if not args.no_sweep:
            line["update_sweep"] = update_sweep(device, hbm_peak)
    print(json.dumps(line), flush=True)


# ---- the reference arm: the CPU oracle -------------------------------------------------------------

def run_reference(args):
    """Times the oracle on the host cores on a bounded sample of the same workload, sized after a pilot step so
    that the whole run stays within a few minutes.  cfg3: each step sends one microbatch through the first n of
    the 32 (identical) stages.  cfg4: each step sends b of the 32 sequences through l of the 6 layers plus the
    embedding and vocabulary stages.  Throughput is scaled to the full workload by the sampled fraction of its
    matrix-product FLOPs."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import pm_inputs as I
    budget_s = 150.0
    total_steps = args.steps + args.warmup
    marks = {}

    def on_step(t, w):
        if t == args.warmup - 1:
            marks["t0"] = time.perf_counter()

    if args.workload == "cfg3":
        from oracle.mlp import run_workload
        full = I.cfg3()

        def sub(n_stages):
            return I.mlp_workload(full.name, n_stages, 1024, 2, "gelu", full.microbatch, compute="bf16",
                                  optimizer=full.optimizer, alpha=full.alpha, beta1=full.beta1, K=full.K, D=full.D,
                                  steps=total_steps, seed=full.seed)
        wl1 = sub(1)
        p1, t1 = I.init_stage_params(wl1), I.teacher_params(wl1)
        b1 = I.batch(wl1, 0, t1)
        t0 = time.perf_counter()
        run_workload(wl1, p1, lambda t: b1, n_steps=2)
        per_stage_step = (time.perf_counter() - t0) / 2
        n_stages = int(max(1, min(full.n_stages, budget_s / (total_steps * per_stage_step))))
        wl = sub(n_stages)
        params0, teacher = I.init_stage_params(wl), I.teacher_params(wl)
        batches = [I.batch(wl, t, teacher) for t in range(min(total_steps, 4))]
        scale = n_stages / full.n_stages
        samples_per_step = full.microbatch
        sample = (f"each step: one microbatch of 128 through {n_stages} of the {full.n_stages} stages "
                  f"(forward, backward, update); samples/s scaled by {n_stages}/{full.n_stages}")
    elif args.workload == "cfg5":
        from oracle.transformer import run_workload
        full = I.cfg5_cut()

        def sub(layers, seqs):
            wl_ = I.cfg5_cut(layers, layers, batch=seqs)
            wl_.steps = total_steps
            return wl_

        def mm_flops(layers, seqs):
            enc = 1024 * (3072 + 1024 + 4096 + 4096)
            dec = 1024 * (3072 + 1024 + 1024 + 2048 + 1024 + 4096 + 4096)
            return 6.0 * seqs * 256 * (layers * (enc + dec) + 1024 * 32000)
        wl1 = sub(1, 1)
        p1 = I.init_encoder_params(wl1)
        b1 = I.seq2seq_batch(wl1, 0)
        t0 = time.perf_counter()
        run_workload(wl1, p1, lambda t: b1, n_steps=1)
        per_flop = (time.perf_counter() - t0) / mm_flops(1, 1)
        layers, seqs = 7, 16
        while layers > 1 and total_steps * per_flop * mm_flops(layers, seqs) > budget_s:
            layers -= 1
        while seqs > 1 and total_steps * per_flop * mm_flops(layers, seqs) > budget_s:
            seqs //= 2
        wl = sub(layers, seqs)
        params0 = I.init_encoder_params(wl)
        batches = [I.seq2seq_batch(wl, t) for t in range(min(total_steps, 4))]
        scale = mm_flops(layers, seqs) / mm_flops(7, 16)
        samples_per_step = 16
        sample = (f"each step: {seqs} of the 16 sequences through {layers} + {layers} of the 7 + 7 layers plus embedding and "
                  f"vocabulary stages (forward, backward, update); samples/s scaled by the sampled fraction "
                  f"{scale:.5f} of the workload's matrix-product FLOPs")
    else:
        from oracle.transformer import run_workload
        full = I.cfg4()

        def sub(layers, seqs):
            return I.encoder_workload(full.name, layers, 512, 8, 2048, 128, seqs, 8192, compute="bf16", optimizer="adam",
                                      alpha=full.alpha, beta1=0.9, beta2=0.98, eps=1e-8, K=full.K, D=full.D,
                                      steps=total_steps, seed=full.seed)

        def mm_flops(layers, seqs):
            per_layer = 512 * (1536 + 512 + 2048 + 2048)
            return 6.0 * seqs * 128 * (layers * per_layer + 512 * 8192)
        wl1 = sub(1, 4)
        p1 = I.init_encoder_params(wl1)
        b1 = I.token_batch(wl1, 0)
        t0 = time.perf_counter()
        run_workload(wl1, p1, lambda t: b1, n_steps=1)
        pilot = time.perf_counter() - t0
        per_flop = pilot / mm_flops(1, 4)
        layers, seqs = 6, 32
        while layers > 1 and total_steps * per_flop * mm_flops(layers, seqs) > budget_s:
            layers -= 1
        while seqs > 1 and total_steps * per_flop * mm_flops(layers, seqs) > budget_s:
            seqs //= 2
        wl = sub(layers, seqs)
        params0 = I.init_encoder_params(wl)
        batches = [I.token_batch(wl, t) for t in range(min(total_steps, 4))]
        scale = mm_flops(layers, seqs) / mm_flops(6, 32)
        samples_per_step = 32
        sample = (f"each step: {seqs} of the 32 sequences through {layers} of the 6 layers plus embedding and "
                  f"vocabulary stages (forward, backward, update); samples/s scaled by the sampled fraction "
                  f"{scale:.4f} of the workload's matrix-product FLOPs")
    if args.warmup == 0:
        marks["t0"] = time.perf_counter()
    run_workload(wl, params0, lambda t: batches[t % len(batches)], n_steps=total_steps, on_step=on_step)
    dt = time.perf_counter() - marks["t0"]
    value = samples_per_step * args.steps / dt * scale
    line = {"impl": "reference", "metric": METRIC, "value": round(value, 4), "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(dt / args.steps * 1e3 / scale, 3),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOADS[args.workload] + " (CPU oracle, bf16-rounded operands, float64 accumulation)"},
            "cpu_baseline": {"value": round(value, 4), "unit": UNIT, "cores": os.cpu_count(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": round(value, 4), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--no-sweep", action="store_true", help="skip the stand-alone update sweep")
    ap.add_argument("--workload", default="cfg4", choices=sorted(WORKLOADS))
    ap.add_argument("--no-other", action="store_true", help="skip the short run of the other built workload")
    ap.add_argument("--stages", type=int, default=0, help="profiling runs: same workload cut to this many stages")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle baseline leg (profiling runs)")
    ap.add_argument("--update-only", type=int, default=0, metavar="N_PARAMS",
                    help="run only the stand-alone fused update on N_PARAMS parameters (profiling runs)")
    args = ap.parse_args()
    if args.update_only:
        run_update_only(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
