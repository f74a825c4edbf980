#!/usr/bin/env python
"""Benchmark of the compressed linear-operator hot path (forward + backward + reconstruct).

One step = one pass of the whole path over one batch: for each of the workload's linears,
acx_linear_fwd (Y, XS), acx_linear_bwd (dX, A) and acx_reconstruct (dW).  Prints ONE JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload llama3b_layer] [--r 128]
    python bench.py --impl reference ...      # the CPU oracle, timed on the host cores

With N > 1 (launched by torch.distributed.run) every rank runs the same step on its own batch of
tokens (the path has no exchange step: weak scaling, no data-path collective); the time is the
maximum over ranks and the value the tokens of all ranks divided by it.
"""
from __future__ import annotations

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

import numpy as np  # noqa: E402

from paper_2605_01255_b200 import inputs as I  # noqa: E402

METRIC = "co-compressed linear fwd+bwd tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


# ------------------------------------------------------------------ algorithmic work per linear
# bytes per element of the weight matrix that the last op of a linear moves, by --update
UPDATE_BYTES = {"reconstruct": 4, "adamw": 26, "lowrank": 8}


def work(m, d_in, d_out, r_fwd, e=2, r=None, update="reconstruct"):
    """Algorithmic flops and bytes of each op of one linear (e = bytes per I/O element).  r_fwd is the rank of the
    factor this linear's forward stores (0 if another linear on the same input stores it), r the rank of the backward."""
    r = r_fwd if r is None else r
    return {
        "fwd": (2.0 * m * d_in * (d_out + r_fwd), e * (m * d_in + d_out * d_in + m * d_out + m * r_fwd)),
        "dx": (2.0 * m * d_out * d_in, e * (m * d_out + d_out * d_in + m * d_in)),
        "factor": (2.0 * m * d_out * r, e * (m * d_out + m * r) + 4 * d_out * r),
        "reconstruct": (2.0 * d_out * r * d_in, 4 * d_out * r + UPDATE_BYTES[update] * d_out * d_in),
    }


# DRAM traffic and tensor-pipe activity of the forward kernel from ncu captures (dram__bytes_read.sum, dram__bytes_write.sum,
# sm__pipe_tensor_cycles_active.avg.pct_of_peak_sustained_elapsed; one launch per distinct (variant, shape) of the default
# workload, 16384 tokens, r = 128; summaries under profiles/fwd_*).  "plain" is the forward of a linear whose input's factor
# another linear stores.  Reported only for a workload whose every forward launch was captured, and dropped (null) when
# the kernel sources differ from the captured ones.
NCU_FWD_CAPTURE = {
    "tokens": 16384, "r": 128, "sources_sha": "3dd6b7de493b5609",
    # (variant, d_in, d_out): (bytes read, bytes written, tensor pipe % of elapsed cycles)
    "launches": {
        ('in-kernel', 3072, 3072): (122764032, 73668352, 68.9),
        ('in-kernel', 3072, 8192): (597660160, 251255808, 80.7),
        ('in-kernel', 8192, 3072): (585623040, 96458240, 76.3),
        ('workspace', 3072, 3072): (121392384, 80954112, 84.0),
        ('workspace', 3072, 8192): (461384960, 258895616, 91.8),
        ('workspace', 8192, 3072): (1068425728, 99412224, 87.6),
        ('plain', 3072, 3072): (119585280, 76793856, 88.2),
        ('plain', 3072, 8192): (398878464, 252640768, 94.2),
    },
}
FWD_KERNEL_SOURCES = ("acx_gemm_sm100.cuh", "acx_sketch.cuh", "acx_umma.cuh")


def fwd_kernel_sources_sha():
    import hashlib
    h = hashlib.sha256()
    try:
        for f in FWD_KERNEL_SOURCES:
            with open(os.path.join(ROOT, "paper_2605_01255_b200", "csrc", f), "rb") as fh:
                h.update(fh.read())
    except OSError:
        return None
    return h.hexdigest()[:16]


def fwd_ncu_figures(tokens, r, launches, sketch):
    """(average DRAM bytes per forward launch, flop-weighted tensor-pipe %) of one step's forward launches from the ncu
    captures, or (None, None).  `launches` = [(d_in, d_out, stores_factor)] of the step."""
    if (tokens, r) != (NCU_FWD_CAPTURE["tokens"], NCU_FWD_CAPTURE["r"]) or fwd_kernel_sources_sha() != NCU_FWD_CAPTURE["sources_sha"]:
        return None, None
    total, pipe, flops = 0.0, 0.0, 0.0
    for d_in, d_out, stores in launches:
        c = NCU_FWD_CAPTURE["launches"].get((sketch if stores else "plain", d_in, d_out))
        if c is None:
            return None, None
        f = float(d_in) * d_out
        total, pipe, flops = total + c[0] + c[1], pipe + c[2] * f, flops + f
    return round(total / len(launches)), round(pipe / flops, 1)


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {k: float(p[k]) for k in FALLBACK_PEAKS if k in p} | {"source": "measured"}
    return dict(FALLBACK_PEAKS) | {"source": "fallback"}


def activation_bytes(wl):
    slots = {}
    for lin in wl.linears:
        slots[lin.slot] = lin.d_in
    e = 2 if wl.dtype == "bf16" else 4
    full = sum(wl.tokens * d * e for d in slots.values()) * wl.layers
    kept = len(slots) * wl.tokens * wl.r * e * wl.layers
    return full, kept


# ------------------------------------------------------------------ clocks sampler
class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append(line.strip())

    def mark(self):
        """Number of samples read so far: brackets the timed region."""
        return len(self.rows)

    def stop_reading(self):
        if not self.proc:
            return []
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        return self.rows

    def summary(self, first=0, last=None):
        """Median SM clock, power and the throttle reasons seen in the samples [first, last)."""
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for row in self.rows[first:last]:
            f = [x.strip() for x in row.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1])); pw.append(float(f[2]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(pw) if pw else None, "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------ the CUDA arm
OPS = ("fwd", "dx", "factor", "reconstruct")


def fma_peak_tflops(sm_max_mhz=1965.0, sms=148, lanes=128):
    """Peak of the fp32 path (config 1), which runs on the FMA pipes: SMs x 128 fp32 lanes x 2 flop x the maximum SM
    clock.  At 148 SMs and 1965 MHz that is 74.4 TFLOP/s."""
    return sms * lanes * 2 * sm_max_mhz * 1e6 / 1e12


def op_roofline(flops, nbytes, ms, peaks, dtype, applicable):
    """Roofline record of one op: flops and bytes are its algorithmic work in the `ms` it took.  The tensor bound is
    given against both measured GEMM peaks (burst: a kernel timed alone or in a sub-second region; sustained: inside a
    seconds-long region under the power cap); `frac` uses the one named by `applicable`."""
    sec = ms * 1e-3
    if sec <= 0:
        return None
    hbm = peaks["hbm_gbs"]
    if dtype == "bf16":
        pk = {"burst": peaks["bf16_tflops"], "sustained": peaks["bf16_tflops_sustained"]}
        compute_bound = "tensor"
    else:
        pk = {"burst": fma_peak_tflops(), "sustained": fma_peak_tflops()}
        compute_bound = "alu"
    t_hbm = nbytes / (hbm * 1e9)
    t_cmp = flops / (pk[applicable] * 1e12)
    if t_cmp >= t_hbm:
        ach = flops / sec / 1e12
        return {"bound": compute_bound, "achieved": round(ach, 2), "unit": "TFLOP/s", "peak": pk[applicable],
                "peak_kind": applicable, "frac": round(ach / pk[applicable], 4), "frac_of_burst_peak": round(ach / pk["burst"], 4),
                "frac_of_sustained_peak": round(ach / pk["sustained"], 4)}
    ach = nbytes / sec / 1e9
    return {"bound": "hbm", "achieved": round(ach, 1), "unit": "GB/s", "peak": hbm, "peak_kind": "copy", "frac": round(ach / hbm, 4)}


def run_acx(args):
    import torch
    import torch.distributed as dist

    from paper_2605_01255_b200 import binding as B
    from paper_2605_01255_b200 import replicas as R
    from paper_2605_01255_b200 import sharded as SH

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the acx arm has no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    B.lib()  # fail loudly if the library is missing
    if args.debug_gemm_mode:
        B.acx_debug_force_gemm_mode(args.debug_gemm_mode)

    wl = I.workload(args.workload, args.r)
    if args.layers:
        wl = I.Workload(wl.name, wl.tokens, wl.linears, wl.r, wl.dtype, wl.recipe, args.layers)
    m, r, dtype = wl.tokens, wl.r, wl.dtype
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    esz = 2 if dtype == "bf16" else 4
    dev = torch.device("cuda", local)
    sharded = args.parallelism == "sharded"

    # ---- seeded synthetic inputs (host, pinned) and device buffers; every rank draws its own batch of tokens
    def pin(a):
        if dtype == "bf16":
            t = torch.from_numpy(I.f32_to_bf16_bits(a).view(np.int16)).view(torch.bfloat16)
        else:
            t = torch.from_numpy(a)
        return t.pin_memory()

    slots = sorted({lin.slot for lin in wl.linears})
    hX = {s: pin(I.make_x(wl, rank, next(l for l in wl.linears if l.slot == s))) for s in slots}
    hG = [pin(I.make_g(wl, rank, k)) for k in range(len(wl.linears))]
    dXin = {s: hX[s].to(dev) for s in slots}
    dG = [g.to(dev) for g in hG]
    dW = [pin(I.make_w(wl, 0, k)).to(dev) for k in range(len(wl.linears))]
    # A stack of `layers` decoder layers keeps one XS per (layer, distinct input) and one A per (layer, linear);
    # X, G, W are drawn once and serve every layer (the stored factors still differ: each layer has its own sketch seed).
    layers = wl.layers
    XS_store = {(l, s): torch.empty(m, r, dtype=tdt, device=dev) for l in range(layers) for s in slots}
    lins = []
    for k, lin in enumerate(wl.linears):
        desc = B.make_desc(m, lin.d_in, lin.d_out, r, I.sketch_seed(args.seed, 0, lin.slot), dtype)
        descs = [B.make_desc(m, lin.d_in, lin.d_out, r, I.sketch_seed(args.seed, l, lin.slot), dtype) for l in range(layers)]
        lins.append(dict(
            k=k, lin=lin, desc=desc, descs=descs, stores_xs=all(o.slot != lin.slot for o in wl.linears[:k]), X=dXin[lin.slot], W=dW[k], G=dG[k],
            Y=torch.empty(m, lin.d_out, dtype=tdt, device=dev), XS=[XS_store[(l, lin.slot)] for l in range(layers)],
            dX=torch.empty(m, lin.d_in, dtype=tdt, device=dev),
            A=[torch.empty(lin.d_out, r, dtype=torch.float32, device=dev) for _ in range(layers)],
            dWfull=torch.empty(lin.d_out, lin.d_in, dtype=torch.float32, device=dev),
            ws_f=B.alloc_workspace(desc, B.ACX_OP_FWD, dev),
            ws_b=B.alloc_workspace(desc, B.ACX_OP_BWD, dev),
            ws_r=B.alloc_workspace(desc, B.ACX_OP_RECONSTRUCT, dev),
            work=work(m, lin.d_in, lin.d_out, r if all(o.slot != lin.slot for o in wl.linears[:k]) else 0, esz, r, args.update)))
    if args.update != "reconstruct":
        if dtype != "bf16":
            raise SystemExit("bench.py: --update adamw/lowrank needs a bf16 workload")
        for L in lins:  # fp32 master weights and optimizer states; the step counter advances with every call
            lin = L["lin"]
            L["Wm"] = L["W"].float()
            L["W_lp"] = torch.empty_like(L["W"])
            if args.update == "adamw":
                L["m"], L["v"] = torch.zeros_like(L["Wm"]), torch.zeros_like(L["Wm"])
            else:
                L["mA"] = [torch.zeros(lin.d_out, r, device=dev) for _ in range(layers)]
                L["vA"] = [torch.zeros(lin.d_out, r, device=dev) for _ in range(layers)]
    opt_step = [0]
    resident = sum(t.numel() * t.element_size() for L in lins for t in (L["Y"], L["dX"], L["dWfull"], L["W"], L["G"], *L["A"]))
    resident += sum(t.numel() * t.element_size() for t in dXin.values()) + sum(t.numel() * t.element_size() for t in XS_store.values())

    # Where per-op times are taken (CUDA events around every call), acx_linear_bwd is called twice per linear (input
    # gradient, then gradient factor: each output may be left out of a call) so that the events can tell its two
    # kernels apart; the headline steps carry no events inside and make the one full call a user makes.
    event_pool = []  # timing events are created before a timed region: creating one costs more host time than a launch
    mode = {"sketch": args.sketch}   # which forward variant `call` runs: "workspace" or "in-kernel"

    def call(op, L, l, events):
        if events is not None:
            e0 = event_pool.pop(); e0.record()
        if op == "fwd":   # the factor of an input shared by several linears is stored by the first of them
            B.acx_linear_fwd(L["descs"][l], L["X"], L["W"], L["Y"], L["XS"][l] if L["stores_xs"] else None,
                             L["ws_f"] if mode["sketch"] == "workspace" else None)
        elif op == "bwd":   # one call, both outputs: what a user makes (the factor's grid follows dX's without waiting for it)
            B.acx_linear_bwd(L["descs"][l], L["G"], L["W"], L["XS"][l], L["dX"], L["A"][l], L["ws_b"])
        elif op == "dx":
            B.acx_linear_bwd(L["descs"][l], L["G"], L["W"], L["XS"][l], L["dX"], None, L["ws_b"])
        elif op == "factor":
            B.acx_linear_bwd(L["descs"][l], L["G"], L["W"], L["XS"][l], None, L["A"][l], L["ws_b"])
        elif args.update == "adamw":     # optimizer strategy (i) fused: the gradient is never written
            opt_step[0] += 1
            B.acx_reconstruct_adamw(L["descs"][l], L["A"][l], L["Wm"], L["m"], L["v"], L["W_lp"], step=opt_step[0], lr=1e-5,
                                    weight_decay=0.01, ws=L["ws_r"])
        elif args.update == "lowrank":   # optimizer strategy (ii): moments kept for the factor
            opt_step[0] += 1
            B.acx_lowrank_adamw(L["descs"][l], L["A"][l], L["mA"][l], L["vA"][l], L["Wm"], step=opt_step[0], lr=1e-5,
                                weight_decay=0.01, ws=L["ws_r"])
        else:
            B.acx_reconstruct(L["descs"][l], L["A"][l], L["dWfull"], 0.0, L["ws_r"])
        if events is not None:
            e1 = event_pool.pop(); e1.record()
            events.append((op, L["k"], e0, e1))

    # token-sharded data parallelism: the factors of a layer travel as one bucket, summed over the ranks by one
    # all-reduce on a side stream while the backward of the layer below runs; the reconstruction follows the sum
    comm = {"events": None, "stream": torch.cuda.Stream(device=dev) if sharded else None,
            "bucket": torch.empty(sum(L["lin"].d_out * r for L in lins), dtype=torch.float32, device=dev) if sharded else None}

    def on_reduce(l, what):
        if comm["events"] is not None:
            ev = event_pool.pop()
            ev.record()           # on the current (side) stream
            comm["events"].append((l, what, ev))

    def step(events=None, before_layer=None):
        """Forward through every layer (only XS survives), then backward from the last layer with reconstruction."""
        if sharded:
            def fwd_layer(l):
                for L in lins:
                    call("fwd", L, l, events)

            def bwd_layer(l):
                for L in lins:
                    if events is None:
                        call("bwd", L, l, None)
                    else:
                        call("dx", L, l, events)
                        call("factor", L, l, events)

            def rec_layer(l):
                for L in lins:
                    call("reconstruct", L, l, events)

            SH.ShardedStep(layers, fwd_layer, bwd_layer, lambda l: [L["A"][l] for L in lins], rec_layer,
                           bucket=comm["bucket"], comm_stream=comm["stream"], on_reduce=on_reduce).run()
            return
        for l in range(layers):
            if before_layer:
                before_layer("fwd", l)
            for L in lins:
                call("fwd", L, l, events)
        for l in reversed(range(layers)):
            if before_layer:
                before_layer("bwd", l)
            for L in lins:
                if events is None:
                    call("bwd", L, l, None)
                else:
                    call("dx", L, l, events)
                    call("factor", L, l, events)
                call("reconstruct", L, l, events)

    def barrier():
        R.barrier(dev)

    def max_over_ranks(x):
        return R.max_over_ranks(x, dev)

    def check_status(where):
        st = B.acx_last_device_status()
        if st != B.ACX_OK:
            raise SystemExit("bench.py: device status %s: %s" % (where, B.status_string(st)))

    events_per_step = 2 * len(OPS) * len(lins) * layers + (2 * layers if sharded else 0)

    def timed_region(n_steps, sampler=None, with_events=True):
        """n_steps steps bracketed by barrier + synchronize, with CUDA events around the region and, with_events, around
        every call.  Returns (ms of the region: max over ranks, per-call event list per step, clocks seen, all-reduce
        event list)."""
        if with_events:
            event_pool.extend(torch.cuda.Event(enable_timing=True) for _ in range(events_per_step * n_steps))
        per_step = []
        comm["events"] = [] if (sharded and with_events) else None
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        mark0 = sampler.mark() if sampler else 0
        t0.record()
        for _ in range(n_steps):
            ev = [] if with_events else None
            step(ev)
            per_step.append(ev or [])
        t1.record()
        barrier()
        mark1 = sampler.mark() if sampler else 0
        ms = max_over_ranks(t0.elapsed_time(t1))
        comm_events, comm["events"] = comm["events"], None
        return ms, per_step, (mark0, mark1), comm_events

    def op_medians(per_step):
        """{(op, k): median over the steps of that call's ms}."""
        acc = {}
        for ev in per_step:
            for op, k, e0, e1 in ev:
                acc.setdefault((op, k), []).append(e0.elapsed_time(e1))
        return {key: float(np.median(v)) for key, v in acc.items()}

    def ops_summary(med, applicable, peaks):
        """Per-op time of one step (sum over the linears and layers of the per-call medians) and its roofline."""
        out_ms, out_rf = {}, {}
        for op in OPS:
            ms_op = layers * sum(v for (o, k), v in med.items() if o == op)   # every layer makes the same calls
            fl = layers * sum(lins[k]["work"][op][0] for (o, k) in med if o == op)
            by = layers * sum(lins[k]["work"][op][1] for (o, k) in med if o == op)
            out_ms[op] = round(ms_op, 4)
            rf = op_roofline(fl, by, ms_op, peaks, dtype, applicable)
            if rf is not None:
                rf["ms_per_step"] = round(ms_op, 4)
            out_rf[op] = rf
        return out_ms, out_rf

    peaks = load_peaks()
    sampler = ClockSampler(local)   # started early: nvidia-smi needs a moment before its first sample
    sampler.start()
    # ---- warm-up: W steps, then keep stepping until the GPU has been under load for --preheat-seconds, so that the
    # timed steps run at the clock the power cap settles at and the result does not depend on how many steps are timed
    for _ in range(args.warmup):
        step()
    barrier()
    check_status("after warm-up")
    t_pre = time.perf_counter()
    pre_steps = 0
    while time.perf_counter() - t_pre < args.preheat_seconds:
        for _ in range(max(1, 8 // layers)):
            step()
            pre_steps += 1
        torch.cuda.synchronize()
    step_est_ms = (time.perf_counter() - t_pre) * 1e3 / max(pre_steps, 1) if pre_steps else None
    if world > 1:   # every rank leaves the pre-heat together
        barrier()

    # ---- timed region: exactly --steps steps, device-resident inputs
    launches0 = B.acx_kernel_launches()
    ms, _, marks, _ = timed_region(args.steps, sampler, with_events=False)
    launches = B.acx_kernel_launches() - launches0
    check_status("after the timed region")
    step_ms = ms / args.steps
    region_s = ms * 1e-3
    # ---- the same steps again with CUDA events around every call (and acx_linear_bwd split in two): per-op times
    ms_ev, per_step, _, comm_events = timed_region(args.steps, sampler)
    check_status("after the per-op region")
    # which measured GEMM peak the timed steps are compared with: the sustained one if the GPU had been under load for
    # seconds when they ran (pre-heat + region), else the burst one
    applicable = "sustained" if (args.preheat_seconds + region_s) >= 2.0 else "burst"
    med = op_medians(per_step)
    ops_ms, ops_rf = ops_summary(med, applicable, peaks)
    per_linear = {op: {lins[k]["lin"].name: round(v, 4) for (o, k), v in sorted(med.items(), key=lambda kv: kv[0][1]) if o == op}
                  for op in OPS}
    step_times = [sum(e0.elapsed_time(e1) for _, _, e0, e1 in ev) for ev in per_step]

    # ---- a second, seconds-long region (the clock sampler sees it at its 50 ms period) for the sustained figures
    sustained = None
    if args.sustain_seconds > 0:
        n_sus = int(min(max(3, np.ceil(args.sustain_seconds * 1e3 / step_ms)), 4000))
        ms_s, per_step_s, marks_s, _ = timed_region(n_sus, sampler)
        check_status("after the sustained region")
        med_s = op_medians(per_step_s)
        ops_ms_s, ops_rf_s = ops_summary(med_s, "sustained", peaks)
        ms_p, _, _, _ = timed_region(n_sus, sampler, with_events=False)   # and once more the way the headline is timed
        sustained = {"steps": n_sus, "seconds": round(ms_s * 1e-3, 3), "ms_per_step_with_op_events": round(ms_s / n_sus, 4),
                     "ms_per_step": round(ms_p / n_sus, 4), "value": round(world * m / (ms_p / n_sus * 1e-3), 1),
                     "ops_ms_per_step": ops_ms_s, "ops_roofline": ops_rf_s, "marks": marks_s}

    # ---- the other forward variant, same step: S^T written once per call into a workspace ("workspace") or every
    # thread block generating its slices of S inside the GEMM, nothing of S in memory ("in-kernel")
    other = None
    if dtype == "bf16" and args.variant_seconds > 0:
        other_mode = "in-kernel" if args.sketch == "workspace" else "workspace"
        mode["sketch"] = other_mode
        for _ in range(2):
            step()
        n_o = int(min(max(3, np.ceil(args.variant_seconds * 1e3 / step_ms)), 2000))
        ms_o, per_step_o, marks_o, _ = timed_region(n_o, sampler)
        check_status("after the variant region")
        mode["sketch"] = args.sketch
        med_o = op_medians(per_step_o)
        ops_ms_o, ops_rf_o = ops_summary(med_o, "sustained", peaks)
        other = {"sketch": other_mode, "steps": n_o, "seconds": round(ms_o * 1e-3, 3), "ms_per_step": round(ms_o / n_o, 4),
                 "value": round(world * m / (ms_o / n_o * 1e-3), 1), "fwd_ms_per_step": ops_ms_o["fwd"], "fwd_roofline": ops_rf_o["fwd"],
                 "marks": marks_o}

    # ---- every op timed alone: its calls for all linears (layer 0) back to back, nothing else in between and no event
    # inside, repeated; the GPU is not held at the power cap by the GEMMs then, so the short memory-bound kernels run at
    # the clock they would have on their own (tensor-bound ops are compared with the burst peak here)
    ops_alone = None
    if args.alone_reps > 0 and not sharded:
        ops_alone = {}
        for op in OPS:
            for L in lins:
                call(op, L, 0, None)
            barrier()
            a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a0.record()
            for _ in range(args.alone_reps):
                for L in lins:
                    call(op, L, 0, None)
            a1.record()
            barrier()
            ms_a = max_over_ranks(a0.elapsed_time(a1)) / args.alone_reps
            fl = sum(L["work"][op][0] for L in lins)
            by = sum(L["work"][op][1] for L in lins)
            rf = op_roofline(fl, by, ms_a, peaks, dtype, "burst")
            ops_alone[op] = {"ms_per_layer": round(ms_a, 4), "roofline": rf}
        check_status("after the per-op loops")

    time.sleep(0.06)                       # let the last samples arrive
    sampler.stop_reading()
    clocks = sampler.summary(max(0, marks[0]), max(marks[1], marks[0] + 1))
    for rec in (sustained, other):
        if rec is not None:
            mk = rec.pop("marks")
            rec["clocks"] = sampler.summary(max(0, mk[0]), max(mk[1], mk[0] + 1))

    # ---- headline roofline record: the op with the largest share of the step
    dominant = max(OPS, key=lambda o: ops_ms[o])
    n_dom = sum(1 for (o, k) in med if o == dominant) * layers   # launches of that op per step
    roofline = dict(ops_rf[dominant] or {})
    roofline["kernel"] = dominant
    roofline["traffic"] = roofline["ncu_tensor_pipe_pct"] = None
    if dominant == "fwd" and dtype == "bf16":
        roofline["traffic"], roofline["ncu_tensor_pipe_pct"] = fwd_ncu_figures(
            m, r, [(L["lin"].d_in, L["lin"].d_out, L["stores_xs"]) for L in lins] * layers, args.sketch)
    roofline.update({"peak_source": peaks["source"], "launch_ms_avg": round(ops_ms[dominant] / max(n_dom, 1), 4),
                     "launches_per_step": n_dom,
                     "peak_note": "frac is against the %s bf16 GEMM peak: the timed steps ran after %.1f s of pre-heat under load "
                                  "(region %.2f s); both fractions are given" % (applicable, args.preheat_seconds, region_s)
                     if dtype == "bf16" else "fp32 path on the FMA pipes: peak = 148 SMs x 128 lanes x 2 flop x 1965 MHz"})
    if sustained is not None and sustained["clocks"].get("sm_mhz") and dtype == "bf16":
        # clock-normalised: each tensor-bound op's rate against what the tensor pipes can do at the SM clock sampled
        # during the region: SMs x 8192 flop per clock (dense bf16; 148 SMs x 8192 x 1.86 GHz is the nominal 2.25 PFLOP/s)
        c = sustained["clocks"]
        sms = torch.cuda.get_device_properties(dev).multi_processor_count
        per_clock_peak = sms * 8192 * c["sm_mhz"] * 1e6 / 1e12
        sustained["clock_normalised"] = {
            "sm_mhz_median": c["sm_mhz"], "tensor_peak_at_that_clock_tflops": round(per_clock_peak, 1),
            "frac": {op: round(rf["achieved"] / per_clock_peak, 4) for op, rf in sustained["ops_roofline"].items()
                     if rf and rf["bound"] == "tensor"},
            "ms_x_mhz": {op: round(v * c["sm_mhz"], 1) for op, v in sustained["ops_ms_per_step"].items()}}
    # whole-step roofline: sum over ops of max(flops/compute peak, bytes/hbm)
    cmp_peak = (peaks["bf16_tflops_sustained" if applicable == "sustained" else "bf16_tflops"] if dtype == "bf16" else fma_peak_tflops())
    bound_s = 0.0
    total_flops = 0.0
    for L in lins:
        for key in OPS:
            f, b = L["work"][key]
            bound_s += layers * max(f / (cmp_peak * 1e12), b / (peaks["hbm_gbs"] * 1e9))
            total_flops += layers * f

    comm_rec = None
    if sharded:
        begins = {}
        ar_ms = []
        for l, what, ev in comm_events:
            if what == "begin":
                begins[l] = ev
            else:
                ar_ms.append(begins[l].elapsed_time(ev))
        comm_rec = {"collective": "all_reduce(SUM) of the layer's gradient factors, one fp32 bucket per layer, NCCL, side stream",
                    "bucket_bytes_per_layer": int(comm["bucket"].numel() * 4), "all_reduces_per_step": layers,
                    "all_reduce_ms_median": round(float(np.median(ar_ms)), 4) if ar_ms else None,
                    "dense_gradient_bytes_per_layer": int(sum(L["lin"].d_out * L["lin"].d_in * 4 for L in lins))}

    # ---- end to end: every layer's inputs start in pinned host memory, its results are read back, every step
    hOut = [dict(Y=torch.empty_like(L["Y"], device="cpu").pin_memory(), XS=torch.empty_like(L["XS"][0], device="cpu").pin_memory(),
                 dX=torch.empty_like(L["dX"], device="cpu").pin_memory(), A=torch.empty_like(L["A"][0], device="cpu").pin_memory())
            for L in lins]
    h2d = layers * (sum(t.numel() * t.element_size() for t in hX.values()) + sum(t.numel() * t.element_size() for t in hG))
    d2h = layers * sum(t.numel() * t.element_size() for o in hOut for t in o.values())

    # Copies run on two extra streams so that host->device, device->host (PCIe is full duplex) and the kernels
    # overlap inside a step; events order every buffer's writer before its readers and the reverse.
    s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    # A single layer alternates between two sets of device output buffers, so that the kernels of a step need not wait
    # for the previous step's device->host reads (the PCIe link, not the GPU, bounds this loop: it should never idle).
    out_sets = [lins]
    if layers == 1:
        xs_alt = {key: torch.empty_like(t) for key, t in XS_store.items()}   # linears on one input share its factor here too
        out_sets.append([dict(L, Y=torch.empty_like(L["Y"]), XS=[xs_alt[(l, L["lin"].slot)] for l in range(layers)],
                              dX=torch.empty_like(L["dX"]), A=[torch.empty_like(a) for a in L["A"]]) for L in lins])
    e2e_state = {"out_done": [None] * len(out_sets), "n": 0}

    def fence(src, dst):
        """Everything queued on src so far happens before what is queued on dst from now on."""
        ev = torch.cuda.Event()
        ev.record(src)
        dst.wait_event(ev)
        return ev

    def e2e_step():
        main = torch.cuda.current_stream()
        which = e2e_state["n"] % len(out_sets)
        e2e_state["n"] += 1
        lins = out_sets[which]
        if e2e_state["out_done"][which] is not None:
            main.wait_event(e2e_state["out_done"][which])  # the reads of this buffer set's Y, XS, dX, A are over
        g_ready = None
        for l in range(layers):
            fence(main, s_in)                            # earlier kernels that read the input buffers
            with torch.cuda.stream(s_in):
                for s_ in slots:
                    dXin[s_].copy_(hX[s_], non_blocking=True)
            fence(s_in, main)
            if layers == 1:                              # G is not reused inside the step: fetch it behind X
                with torch.cuda.stream(s_in):
                    g_ready = []
                    for k, g in enumerate(hG):
                        dG[k].copy_(g, non_blocking=True)
                        ev = torch.cuda.Event(); ev.record(s_in); g_ready.append(ev)
            if l > 0:
                fence(s_out, main)                       # Y buffers of the previous layer are still being read
            for L, o in zip(lins, hOut):
                call("fwd", L, l, None)
                fence(main, s_out)
                with torch.cuda.stream(s_out):
                    o["Y"].copy_(L["Y"], non_blocking=True)
                    o["XS"].copy_(L["XS"][l], non_blocking=True)
        for l in reversed(range(layers)):
            if g_ready is None or layers > 1:
                fence(main, s_in)                        # the bwd of the layer after this one read dG
                with torch.cuda.stream(s_in):
                    g_ready = []
                    for k, g in enumerate(hG):
                        dG[k].copy_(g, non_blocking=True)
                        ev = torch.cuda.Event(); ev.record(s_in); g_ready.append(ev)
                fence(s_out, main)                       # dX buffers of the layer after this one are still being read
            for k, (L, o) in enumerate(zip(lins, hOut)):
                main.wait_event(g_ready[k])
                call("bwd", L, l, None)
                if not sharded:
                    call("reconstruct", L, l, None)
                fence(main, s_out)
                with torch.cuda.stream(s_out):
                    o["dX"].copy_(L["dX"], non_blocking=True)
                    if not sharded:
                        o["A"].copy_(L["A"][l], non_blocking=True)
            if sharded:   # the factors are summed over the ranks before anybody uses them
                SH.allreduce_factors([L["A"][l] for L in lins], bucket=comm["bucket"])
                for L, o in zip(lins, hOut):
                    call("reconstruct", L, l, None)
                fence(main, s_out)
                with torch.cuda.stream(s_out):
                    for L, o in zip(lins, hOut):
                        o["A"].copy_(L["A"][l], non_blocking=True)
        ev = torch.cuda.Event(); ev.record(s_out)
        e2e_state["out_done"][which] = ev

    def e2e_drain():
        """The event recorded next on the main stream waits for both copy streams."""
        main = torch.cuda.current_stream()
        fence(s_in, main)
        fence(s_out, main)

    e2e_steps = max(1, min(args.steps, args.e2e_steps if layers == 1 else 1))
    e2e_step()
    e2e_drain()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(e2e_steps):
        e2e_step()
    e2e_drain()
    e1.record()
    barrier()
    e2e_ms = max_over_ranks(e0.elapsed_time(e1)) / e2e_steps

    full, kept = activation_bytes(wl)
    step_desc = {"reconstruct": "reconstruct", "adamw": "reconstruct fused with AdamW (no dW written)",
                 "lowrank": "low-rank AdamW (moments kept for the factor)"}[args.update]
    out = {
        "metric": METRIC, "value": round(world * m / (step_ms * 1e-3), 1), "unit": "tokens/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(step_ms, 4), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": dtype, "data": "synthetic",
        "config": {"workload": wl.name, "tokens_per_gpu": m, "rank": r, "layers": layers, "recipe": wl.recipe,
                   "linears": [[l.name, l.d_in, l.d_out] for l in wl.linears],
                   "step": "fwd of every linear of every layer (XS kept), then bwd + %s from the last layer back" % step_desc,
                   "l2": "inputs larger than L2 (%.1f GB resident per GPU, each call streams different buffers)" % (resident / 1e9),
                   "sketch": args.sketch + (": S^T written once per call into the call's workspace (r x d_in bf16) and read back by the GEMM"
                                            if args.sketch == "workspace" else ": S generated inside the GEMM, never in global memory"),
                   "parallelism": ("token-sharded, one all-reduce of the factors per layer" if sharded else "replicas") if world > 1 or sharded else "single",
                   "debug_gemm_mode": args.debug_gemm_mode, "preheat_s": args.preheat_seconds, "preheat_steps": pre_steps,
                   "timing": "value and ms_per_step: CUDA events around the --steps steps, nothing recorded inside them, acx_linear_bwd called "
                             "once per linear for both outputs; per-op times: the same steps repeated with events around every call and "
                             "acx_linear_bwd split into its two outputs, medians over the steps of each call, summed over the linears"},
        "tflops": round(total_flops / (step_ms * 1e-3) / 1e12, 2),
        "step_roofline_frac": round(bound_s * 1e3 / step_ms, 4),
        "step_roofline_peak": applicable if dtype == "bf16" else "fma",
        "step_ms_median_of_op_sums": round(float(np.median(step_times)), 4),
        "ms_per_step_with_op_events": round(ms_ev / args.steps, 4),
        "ops_ms_per_step": ops_ms,
        "ops_roofline": ops_rf,
        "ops_ms_per_linear": per_linear,
        "roofline": roofline,
        "sustained": sustained,
        "other_sketch_variant": other,
        "ops_alone": ops_alone,
        "e2e": {"value": round(world * m / (e2e_ms * 1e-3), 1), "unit": "tokens/s", "ms_per_step": round(e2e_ms, 3),
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps,
                "note": "every step X and G are copied from pinned host memory and Y, XS, dX, A read back, on copy streams that "
                        "overlap the kernels and, with two sets of device output buffers, the next step; W resident; dW stays on the device"},
        "gpu_launches": int(launches),
        "clocks": clocks,
        "activation_bytes": {"uncompressed_X": full, "stored_XS": kept, "saved_MB": round((full - kept) / 1e6, 1),
                             "stored_XS_allocated": sum(t.numel() * t.element_size() for t in XS_store.values())},
    }
    if comm_rec is not None:
        out["comm"] = comm_rec
    if args.memory_report:
        out["peak_memory"] = memory_report(torch, step, XS_store, dXin, layers, slots)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = oracle_timing(wl, args.cpu_tokens, repeats=1)
    if rank == 0:
        print(json.dumps(out), flush=True)
    if world > 1:
        dist.destroy_process_group()


def memory_report(torch, step, XS_store, dXin, layers, slots):
    """Peak device memory (torch.cuda.max_memory_allocated, the paper's own measure) of one step that keeps XS,
    against the same step when the layer inputs X themselves are kept for the backward pass."""
    torch.cuda.synchronize()
    base = torch.cuda.memory_allocated()
    torch.cuda.reset_peak_memory_stats()
    step()
    torch.cuda.synchronize()
    peak_c = torch.cuda.max_memory_allocated()
    kept_xs = sum(t.numel() * t.element_size() for t in XS_store.values())
    torch.cuda.reset_peak_memory_stats()
    x_store = {}

    def keep_x(phase, l):
        if phase == "fwd":
            for s_ in slots:
                x_store[(l, s_)] = dXin[s_].clone()   # what autograd would save for the weight gradient

    step(None, keep_x)
    torch.cuda.synchronize()
    peak_u = torch.cuda.max_memory_allocated()
    kept_x = sum(t.numel() * t.element_size() for t in x_store.values())
    x_store.clear()
    return {"method": "torch.cuda.max_memory_allocated over one step", "resident_before_bytes": base,
            "peak_keeping_XS_bytes": peak_c, "peak_keeping_X_too_bytes": peak_u, "kept_XS_bytes": kept_xs, "kept_X_bytes": kept_x,
            "activation_saving_bytes": kept_x - kept_xs}


# ------------------------------------------------------------------ the oracle leg (CPU)
def oracle_step(wl, tokens, layer=0, seed=0):
    """One pass of the whole path in the fp64 oracle on the first `tokens` tokens.  Returns seconds."""
    from oracle import linear as ol
    from oracle import sketch as osk

    data = []
    for k, lin in enumerate(wl.linears):
        data.append((lin, I.make_x(wl, layer, lin, tokens), I.make_w(wl, layer, k), I.make_g(wl, layer, k, tokens)))
    t0 = time.perf_counter()
    for lin, X, W, G in data:
        S = osk.sketch_for_dtype(I.sketch_seed(seed, layer, lin.slot), lin.d_in, wl.r, wl.dtype)
        Y, U = ol.linear_fwd(X, W, S)
        dX, A = ol.linear_bwd(G, W, U)
        ol.reconstruct(A, S)
    return time.perf_counter() - t0


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads") for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else os.cpu_count()
    except Exception:
        return os.cpu_count()


def oracle_timing(wl, tokens, repeats=1):
    tokens = min(tokens, wl.tokens)
    secs = min(oracle_step(wl, tokens) for _ in range(repeats))
    return {"value": round(tokens / (secs * wl.layers), 1), "unit": "tokens/s", "cores": blas_threads(), "kind": "oracle",
            "seconds": round(secs, 3),
            "sample": "first %d of %d tokens, all %d linears of one layer%s, fwd+bwd+reconstruct incl. sketch generation, numpy float64" %
                      (tokens, wl.tokens, len(wl.linears), " (time x %d layers)" % wl.layers if wl.layers > 1 else "")}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = I.workload(args.workload, args.r)
    if args.layers:
        wl = I.Workload(wl.name, wl.tokens, wl.linears, wl.r, wl.dtype, wl.recipe, args.layers)
    tokens = min(args.ref_tokens, wl.tokens)
    for _ in range(args.warmup):
        oracle_step(wl, tokens)
    t = [oracle_step(wl, tokens) for _ in range(args.steps)]
    sec = sum(t) / len(t) * wl.layers   # one layer is timed; a stack costs that many times it
    val = round(tokens / sec, 1)
    out = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": "tokens/s", "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(sec * 1e3, 3), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "tokens_per_gpu": wl.tokens, "rank": wl.r,
                   "step": "fwd + bwd + reconstruct of every linear on a %d-token sample" % tokens},
        "cpu_baseline": {"value": val, "unit": "tokens/s", "cores": blas_threads(), "kind": "oracle",
                         "sample": "%d of %d tokens per step, all %d linears, numpy float64 oracle on the host cores" %
                                   (tokens, wl.tokens, len(wl.linears))},
        "e2e": {"value": val, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(out), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--preheat-seconds", type=float, default=3.0,
                    help="after the warm-up steps keep stepping (untimed) this long, so that the timed steps run at the clock the "
                         "power cap settles at; 0 times a cold GPU")
    ap.add_argument("--sustain-seconds", type=float, default=3.0,
                    help="length of the second timed region whose per-op figures go into 'sustained' (0 = skip)")
    ap.add_argument("--variant-seconds", type=float, default=1.5,
                    help="length of the region that times the same step with the other forward variant (0 = skip)")
    ap.add_argument("--debug-gemm-mode", type=int, default=0,
                    help="test/debug: force the tile shape of the forward and dX (acx_debug_force_gemm_mode; 0 = the cost models)")
    ap.add_argument("--alone-reps", type=int, default=20,
                    help="repetitions of the loops that time every op on its own, back to back ('ops_alone'; 0 = skip)")
    ap.add_argument("--parallelism", default="replicas", choices=["replicas", "sharded"],
                    help="N > 1: independent replicas (default), or token-sharded data parallelism: every rank runs the step on "
                         "its own tokens and the gradient factors of each layer are summed by one all-reduce before reconstruction")
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="acx", choices=["acx", "reference"])
    ap.add_argument("--workload", default="llama3b_layer", choices=I.WORKLOADS)
    ap.add_argument("--layers", type=int, default=None, help="override the number of layers of a stack workload")
    ap.add_argument("--memory-report", action="store_true", help="add measured peak memory with and without keeping X")
    ap.add_argument("--r", type=int, default=None)
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--e2e-steps", type=int, default=10)
    ap.add_argument("--cpu-tokens", type=int, default=16384, help="tokens of the oracle sample in cpu_baseline (10-20 s of CPU work)")
    ap.add_argument("--ref-tokens", type=int, default=256, help="tokens per step of the --impl reference arm")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sketch", default="in-kernel", choices=["workspace", "in-kernel"],
                    help="forward: no workspace at all, every thread block regenerates its slices of S inside the GEMM and nothing of S "
                         "reaches global memory (default: the method as stated), or S^T written once per call into the call's "
                         "workspace and read back by the GEMM (same bits, a few per cent faster; reported as other_sketch_variant)")
    ap.add_argument("--update", default="reconstruct", choices=sorted(UPDATE_BYTES),
                    help="last op of every linear: rebuild dW (default, the metric's step), or apply the optimizer step directly: "
                         "adamw = reconstruct fused with AdamW, lowrank = Adam moments kept for the gradient factor")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "acx":
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_acx(args)


if __name__ == "__main__":
    main()
