#!/usr/bin/env python
"""Benchmark of the AdaDim layer-quantization path on B200.

One step = one pass of the whole path over one layer: calibration Hessian over all tokens,
RTN in both grouping dimensions, score + select, damped Cholesky-inverse factor, GPTQ in both
dimensions, score + select.  Default workload (the one the metric is quoted on): the LLaMA-7B
q_proj-shaped layer (W 4096 x 4096 fp16, X 262144 x 4096 bf16), 3-bit, group 128, seeded
synthetic tensors.  `--workload down_proj | block | mlp70b` times the other benchmark
configurations (one step = every layer and variant of that configuration once); they report the
same keys per layer and for the whole set, without the host-buffer leg.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

Prints one JSON line.  With N > 1 (under torchrun) every rank quantizes its own replica of the
layer; there is no data-path collective.  `--impl reference` times the CPU oracle on a bounded
sample of the same workload.
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

METRIC = "AdaDim layer quant weights/s (RTN & GPTQ, 3b g128); % of HBM/tensor roofline"
BITS, GROUP = 3, 128
DTYPE = "bf16 (Hessian and scorer: bf16 tensor cores, fp32 accumulation); f32 (quantizer); f64 (factor, GPTQ)"
WORKLOAD = ("llama7b_q_proj W[4096,4096] fp16, X[262144,4096] bf16, 3-bit g128, "
            "Hessian + RTN both dims + score + factor + GPTQ both dims + score")


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def stage_rooflines(stage_ms, out, inp, ntok, bits, group, peaks, mhz, clocks):
    """What bounds each stage of one layer's pass, from the stage's CUDA-event time.
    Tensor-core stages are given against both measured bf16 figures: the burst one applies when the
    SM clock stayed at its maximum with no power cap during the timed region, the sustained one
    when sw_power_cap was active; `frac` follows whichever applies."""
    tile = 256
    weights = out * inp
    capped = bool(clocks and "sw_power_cap" in (clocks.get("reasons") or []))
    r = {}

    def tensor(name, flops):
        ach = flops / (stage_ms[name] * 1e-3) / 1e12
        r[name] = {"bound": "tensor", "achieved": ach, "unit": "TFLOP/s",
                   "peak": peaks["bf16_tflops_sustained"] if capped else peaks["bf16_tflops"],
                   "peak_source": peaks["source"] + (" (sustained bf16: power cap active)" if capped
                                                      else " (burst bf16: full clock, no cap)"),
                   "frac_of_burst": ach / peaks["bf16_tflops"], "frac_of_sustained": ach / peaks["bf16_tflops_sustained"]}
        r[name]["frac"] = r[name]["frac_of_sustained"] if capped else r[name]["frac_of_burst"]

    if "hessian" in stage_ms:
        tensor("hessian", ntok * inp * (inp + tile))          # lower-triangle tiles of the symmetric product
    for name in ("score_rtn", "score_gptq"):
        if name in stage_ms:
            tensor(name, 2 * out * inp * (inp + tile))        # D^T D on lower-triangle tiles, both dims
    if "rtn" in stage_ms:
        ach = weights * (2 + 2 * (bits / 8 + 4 / group)) / (stage_ms["rtn"] * 1e-3) / 1e9
        r["rtn"] = {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "peak_source": peaks["source"], "frac": ach / peaks["hbm_gbs"]}
    if "factor" in stage_ms:
        ach = 2 * inp ** 3 / 3 / (stage_ms["factor"] * 1e-3) / 1e12       # Cholesky + triangular inverse
        pk = 148 * 64 * 2 * mhz * 1e6 / 1e12
        r["factor"] = {"bound": "alu", "achieved": ach, "peak": pk, "unit": "TFLOP/s", "frac": ach / pk,
                       "note": "fp64 FMA: 148 SMs x 64 FMA/clk x 2 at the sampled SM clock"}
    if "gptq" in stage_ms:
        blocks = inp // 128
        r["gptq"] = {"bound": "latency", "ms": stage_ms["gptq"], "column_blocks": blocks,
                     "us_per_column_block": stage_ms["gptq"] * 1e3 / blocks,
                     "cycles_per_column": stage_ms["gptq"] * 1e-3 * mhz * 1e6 / inp,
                     "note": "a chain of `column_blocks` block kernels, each 128 dependent column steps; the "
                             "tensor-core trailing updates run beside it on a second stream"}
    return r


def measured_traffic(name):
    """DRAM bytes of one launch of the dominant kernel from the ncu capture kept beside its
    profile summary; null once the kernel's sources differ from the ones the capture was taken with."""
    import hashlib
    path = os.path.join(ROOT, "profiles", name + ".traffic.json")
    if not os.path.exists(path):
        return {"traffic": None, "traffic_note": "no capture on file"}
    d = json.load(open(path))
    h = hashlib.sha256()
    for f in d["sources"]:
        h.update(open(os.path.join(ROOT, f), "rb").read())
    if h.hexdigest() != d["sources_sha256"]:
        return {"traffic": None, "traffic_note": "kernel sources changed since the capture"}
    return {"traffic": d["dram_bytes_read"] + d["dram_bytes_write"], "traffic_unit": d["unit"],
            "traffic_algorithmic": d["algorithmic_bytes"], "traffic_note": d["note"]}


# --------------------------------------------------------------------------- clocks sampler
class ClockSampler:
    def __init__(self, gpu_index: int):
        self.gpu, self.rows, self.proc, self.thread = gpu_index, [], None, None

    def start(self):
        q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ts, line in self.rows:
            if ts < t0 or ts > t1 + 0.1:
                continue
            f = [x.strip() for x in line.split(",")]
            try:
                sm.append(float(f[0]))
                mx = float(f[1])
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, f[2:]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


# --------------------------------------------------------------------------- launch count
def _inverse_launches(n: int, dones) -> int:
    """Launches of the factor's inverse: the seeds and the two merge steps of every pair, issued after
    each group of panels as soon as the columns they need are final (mirrors the host-side schedule;
    `dones` are the column counts after each group)."""
    levels = []
    s = 64
    while s < n:
        levels.append({"s": s, "npairs": (n - s + 2 * s - 1) // (2 * s), "slots": max(1, 256 // (2 * s)), "m1": 0, "m2": 0, "rows2": 0})
        s *= 2
    count, seeded = 0, 0
    for done in dones:
        if done // 64 > seeded:
            count, seeded = count + 1, done // 64
        for lv in levels:
            s = lv["s"]
            while True:
                if s > 256:
                    if lv["m2"] < lv["m1"]:
                        b0 = lv["m2"] * 2 * s + s
                        sB = min(s, n - b0)
                        avail = (min(done, b0 + sB) - b0) // 64
                        half = s // 128
                        if avail * 64 < sB:
                            avail = avail // half * half
                        if avail > lv["rows2"]:
                            count, lv["rows2"] = count + 1, avail
                        if lv["rows2"] * 64 >= sB:
                            lv["m2"], lv["rows2"] = lv["m2"] + 1, 0
                else:
                    q2 = lv["m2"]
                    while q2 < lv["m1"] and min((q2 + 1) * 2 * s, n) <= done:
                        q2 += 1
                    if q2 > lv["m2"]:
                        count, lv["m2"] = count + 1, q2
                if lv["m2"] < lv["m1"]:
                    break
                q1 = lv["m1"]
                while q1 < lv["npairs"] and q1 - lv["m1"] < lv["slots"] and q1 * 2 * s + s <= done:
                    q1 += 1
                if q1 == lv["m1"]:
                    break
                count, lv["m1"] = count + 1, q1
    return count


def launches_hessian_factor(inp: int) -> int:
    """Kernels launched by one Hessian accumulation plus one factor (mirrors the host-side launch logic)."""
    nb = inp // 64
    factor = 2 + 1                                       # damping, build; diagonal block 0 (the later ones are factored inside the update kernels)
    dones = []
    for g0 in range(0, nb, 4):
        g1 = min(g0 + 4, nb)
        for k in range(g0, g1):
            below, inner = nb - k - 1, g1 - k - 1
            factor += (1 if below > 0 else 0) + (1 if below > 0 and inner > 0 else 0)   # panel, in-group update
        factor += (1 if g1 * 64 < inp else 0) + (1 if g1 * 64 + 256 < inp else 0)   # rank-256 update: next group's columns, rest
        dones.append(min(g1 * 64, inp))
    factor += _inverse_launches(inp, dones)
    factor += 1                                          # emit
    hessian = 2 if inp > 256 else 1
    return hessian + factor


def launches_layer(inp: int, score_gptq: bool = True) -> int:
    """Kernels launched for one layer: RTN, scoring, GPTQ (with a precomputed factor), scoring."""
    blocks = inp // 128
    gptq = 1 + 1 + blocks + (blocks - 1) + max(blocks - 2, 0) + 1   # init, U slicing, block kernels, next-block and rest trailing kernels, loss
    rtn = 1
    score = 1 + 1 + 1                                  # difference kernel, Gram product, finalize
    return rtn + score + gptq + (score if score_gptq else 0)


def launches_per_step(out: int, inp: int) -> int:
    return launches_hessian_factor(inp) + launches_layer(inp)


# --------------------------------------------------------------------------- rank aggregation
def max_over_ranks(ms: float, world: int, device) -> float:
    """Largest of the ranks' device-timed durations (every rank gets the same number back)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(world: int, units_per_rank: int, ms_per_step: float) -> float:
    """Units per second over all replicas: each rank quantizes its own layer (weak scaling)."""
    return world * units_per_rank / (ms_per_step * 1e-3)


# --------------------------------------------------------------------------- our arm
def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2309_15531_b200 import binding as B
    from paper_2309_15531_b200 import inputs as I

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    wl = I.workload_qproj()
    wspec, xspec = wl["layers"]["q_proj"]
    out, inp, ntok = wspec.out, wspec.inp, xspec.n_tokens
    W = I.make_weight(wspec, dev)
    X = I.make_calib(xspec, dev)
    H = torch.zeros(inp, inp, device=dev)
    st = torch.zeros(1, dtype=torch.int32, device=dev)
    ws_g = torch.empty(B.workspace_bytes(B.WS_GPTQ, out, inp), dtype=torch.uint8, device=dev)
    ws_s = torch.empty(B.workspace_bytes(B.WS_SCORE, out, inp), dtype=torch.uint8, device=dev)
    ws_f = torch.empty(B.workspace_bytes(B.WS_FACTOR, 0, inp), dtype=torch.uint8, device=dev)
    r_oc, r_ic = B.QTensor(out, inp, BITS, GROUP, B.DIM_OC, dev), B.QTensor(out, inp, BITS, GROUP, B.DIM_IC, dev)
    g_oc, g_ic = B.QTensor(out, inp, BITS, GROUP, B.DIM_OC, dev), B.QTensor(out, inp, BITS, GROUP, B.DIM_IC, dev)
    err_r = torch.zeros(2, dtype=torch.float64, device=dev)
    err_g = torch.zeros(2, dtype=torch.float64, device=dev)
    ch_r = torch.zeros(1, dtype=torch.int32, device=dev)
    ch_g = torch.zeros(1, dtype=torch.int32, device=dev)
    loss = torch.zeros(2, dtype=torch.float64, device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)       # > 126 MB L2

    stages = ["hessian", "rtn", "score_rtn", "factor", "gptq", "score_gptq"]

    def one_step(Wd, Xd, ev=None):
        def mark(i):
            if ev is not None:
                ev[i].record()
        mark(0)
        H.zero_()
        B.hessian_accumulate(Xd, H, st)
        mark(1)
        B.quantize_rtn(Wd, BITS, GROUP, B.DIM_BOTH, r_oc, r_ic)
        mark(2)
        B.score_select(Wd, H, BITS, GROUP, r_oc, r_ic, err_r, ch_r, st, ws_s)
        mark(3)
        U = B.cholesky_inverse_factor(H, 0.01, st, ws_f)
        mark(4)
        B.quantize_gptq(Wd, H, BITS, GROUP, B.DIM_BOTH, 0.01, U, g_oc, g_ic, loss, st, ws_g)
        mark(5)
        B.score_select(Wd, H, BITS, GROUP, g_oc, g_ic, err_g, ch_g, st, ws_s)
        mark(6)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        one_step(W, X)
    barrier()
    assert int(st.item()) == 0, f"device status {int(st.item())}"

    # ---- device-resident timing ------------------------------------------------------------
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(7)] for _ in range(args.steps)]
    barrier()
    t_wall0 = time.time()
    for k in range(args.steps):
        flush.fill_(k & 0xFF)                      # evict W / H / outputs from L2 between steps
        one_step(W, X, evs[k])
    barrier()
    t_wall1 = time.time()
    clocks = sampler.stop(t_wall0, t_wall1) if rank == 0 else None
    step_ms = [evs[k][0].elapsed_time(evs[k][6]) for k in range(args.steps)]
    stage_ms = {s: sum(evs[k][i].elapsed_time(evs[k][i + 1]) for k in range(args.steps)) / args.steps
                for i, s in enumerate(stages)}
    total_ms = sum(step_ms)
    total_ms = max_over_ranks(total_ms, world, dev)
    ms_per_step = total_ms / args.steps
    weights = out * inp
    value = whole_job_value(world, weights, ms_per_step)

    resident_err = torch.cat([err_r, err_g]).cpu()

    # ---- end to end: host buffers in, results out --------------------------------------------
    # Every step copies its own W and X from pinned host memory and reads every result back.  The
    # calibration tokens go through the public chunked interface (H += 2 X_c^T X_c per chunk): chunks
    # are copied on a second stream into a small ring of device buffers while earlier chunks are
    # accumulated, and the ring lets the copies of the next step start during this step's
    # factorization and GPTQ, as a layer-after-layer run would.
    e2e = None
    if not args.no_e2e:
        Wh = W.cpu().pin_memory()
        Xh = X.cpu().pin_memory()
        outs = [r_oc, r_ic, g_oc, g_ic]
        host_out = [(torch.empty_like(q.codes, device="cpu").pin_memory(),
                     torch.empty_like(q.scales, device="cpu").pin_memory(),
                     torch.empty_like(q.zeros, device="cpu").pin_memory()) for q in outs]
        host_err = torch.empty(4, dtype=torch.float64).pin_memory()
        host_ch = torch.empty(2, dtype=torch.int32).pin_memory()
        n_chunks, n_buf = 8, 3
        rows = ntok // n_chunks
        assert rows * n_chunks == ntok
        xbuf = [torch.empty(rows, inp, dtype=X.dtype, device=dev) for _ in range(n_buf)]
        wbuf = [torch.empty_like(W) for _ in range(2)]
        copied = [torch.cuda.Event() for _ in range(n_buf)]
        consumed = [torch.cuda.Event() for _ in range(n_buf)]
        w_copied = [torch.cuda.Event() for _ in range(2)]
        w_consumed = [torch.cuda.Event() for _ in range(2)]
        copy_stream = torch.cuda.Stream()
        main_stream = torch.cuda.current_stream()
        counter = {"step": 0}

        def e2e_step():
            s = counter["step"]
            counter["step"] += 1
            wb = s & 1
            with torch.cuda.stream(copy_stream):
                if s >= 2:
                    copy_stream.wait_event(w_consumed[wb])
                wbuf[wb].copy_(Wh, non_blocking=True)
                w_copied[wb].record(copy_stream)
            H.zero_()
            for c in range(n_chunks):
                g = s * n_chunks + c
                b = g % n_buf
                with torch.cuda.stream(copy_stream):
                    if g >= n_buf:
                        copy_stream.wait_event(consumed[b])
                    xbuf[b].copy_(Xh[c * rows:(c + 1) * rows], non_blocking=True)
                    copied[b].record(copy_stream)
                main_stream.wait_event(copied[b])
                B.hessian_accumulate(xbuf[b], H, st)
                consumed[b].record(main_stream)
            main_stream.wait_event(w_copied[wb])
            Wd = wbuf[wb]
            B.quantize_rtn(Wd, BITS, GROUP, B.DIM_BOTH, r_oc, r_ic)
            B.score_select(Wd, H, BITS, GROUP, r_oc, r_ic, err_r, ch_r, st, ws_s)
            U = B.cholesky_inverse_factor(H, 0.01, st, ws_f)
            B.quantize_gptq(Wd, H, BITS, GROUP, B.DIM_BOTH, 0.01, U, g_oc, g_ic, loss, st, ws_g)
            B.score_select(Wd, H, BITS, GROUP, g_oc, g_ic, err_g, ch_g, st, ws_s)
            w_consumed[wb].record(main_stream)
            for q, (c_, s_, z_) in zip(outs, host_out):
                c_.copy_(q.codes, non_blocking=True)
                s_.copy_(q.scales, non_blocking=True)
                z_.copy_(q.zeros, non_blocking=True)
            host_err[:2].copy_(err_r, non_blocking=True)
            host_err[2:].copy_(err_g, non_blocking=True)
            host_ch[:1].copy_(ch_r, non_blocking=True)
            host_ch[1:].copy_(ch_g, non_blocking=True)

        e2e_step()
        barrier()
        assert int(st.item()) == 0, f"device status {int(st.item())}"
        counter["step"] = 0                                   # no events pending: start the ring afresh
        n_e2e = max(1, min(args.steps, 5))
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        copy_stream.wait_event(e0)                            # no copy of a timed step starts before the clock does
        for _ in range(n_e2e):
            e2e_step()
        main_stream.wait_stream(copy_stream)
        e1.record()
        barrier()
        e2e_ms = max_over_ranks(e0.elapsed_time(e1) / n_e2e, world, dev)
        h2d = Wh.numel() * Wh.element_size() + Xh.numel() * Xh.element_size()
        d2h = sum(t.numel() * t.element_size() for trip in host_out for t in trip) + 4 * 8 + 2 * 4
        e2e = {"value": whole_job_value(world, weights, e2e_ms), "unit": "weights/s", "ms_per_step": e2e_ms,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": n_e2e,
               "how": f"X in {n_chunks} chunks through a ring of {n_buf} device buffers on a copy stream, "
                      "Hessian accumulated chunk by chunk; results read back every step"}
        # the chunked path must reproduce the device-resident run (chunks end on drain boundaries)
        e2e["matches_resident_run"] = bool(torch.allclose(host_err, resident_err, rtol=1e-9, atol=0.0))

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- rooflines -------------------------------------------------------------------------------
    peaks = _peaks()
    mhz = (clocks or {}).get("sm_mhz") or 1965.0
    roof_all = stage_rooflines(stage_ms, out, inp, ntok, BITS, GROUP, peaks, mhz, clocks)
    # The dominant kernel is the Hessian's tensor-core kernel (the factor and GPTQ stages are longer
    # but are sequences of short launches).  Its time is the hessian stage's CUDA-event time (zeroing
    # H + the tensor-core kernel + the 24 us mirror copy).
    roofline = dict(roof_all["hessian"])
    roofline["kernel"] = "tc_kernel<Hessian>"
    roofline.update(measured_traffic("tc_kernel_hessian_llama7b_q_proj"))

    cpu = None if args.no_cpu_baseline else cpu_baseline()

    line = {
        "metric": METRIC, "value": value, "unit": "weights/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": DTYPE, "data": "synthetic",
        "config": {"workload": WORKLOAD,
                   "l2": "flushed between steps by writing a 256 MiB buffer; X (2.1 GB) exceeds L2",
                   "replicas": world},
        "stages_ms": stage_ms,
        "stage_weights_per_s": {s: weights / (t * 1e-3) for s, t in stage_ms.items()},
        "rooflines": roof_all, "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "clocks": clocks,
        "gpu_launches": launches_per_step(out, inp) * args.steps,
        "chosen": {"rtn": B.DIM_NAMES[int(ch_r.item())], "gptq": B.DIM_NAMES[int(ch_g.item())]},
        "errors": {"rtn": err_r.tolist(), "gptq": err_g.tolist()},
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


# --------------------------------------------------------------------------- the other configurations
def config_jobs(name):
    """(workload dict, list of (layer name, [(bits, group, mode)])) for a benchmark configuration.
    mode "both": RTN in both dimensions + score, GPTQ in both dimensions + score + select.
    mode "ada":  the paper's flow: RTN in both dimensions + score + select, GPTQ in the chosen one."""
    from paper_2309_15531_b200 import inputs as I
    if name == "down_proj":
        wl = I.workload_downproj()
        return wl, [("down_proj", [(b, g, "both") for b, g in wl["variants"]])]
    if name == "block":
        wl = I.workload_block()
        return wl, [(n, [(3, 128, "ada")]) for n in wl["layers"]]
    if name == "mlp70b":
        wl = I.workload_mlp70b()
        return wl, [(n, [(4, 128, "both")]) for n in wl["layers"]]
    raise ValueError(name)


def run_config(args):
    """One step = every Hessian, factor, layer and variant of the configuration once.  Layers that
    share an input width share one activation tensor, one Hessian and one factor."""
    import torch
    from paper_2309_15531_b200 import binding as B
    from paper_2309_15531_b200 import inputs as I

    if int(os.environ.get("RANK", "0")) != 0:
        return                                            # one replica is enough for these lines
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    wl, jobs = config_jobs(args.workload)
    xspecs = {}
    for lname, _ in jobs:
        xs = wl["layers"][lname][1]
        xspecs.setdefault(xs, []).append(lname)
    Ws = {n: I.make_weight(wl["layers"][n][0], dev) for n, _ in jobs}
    Xs = {xs: I.make_calib(xs, dev) for xs in xspecs}
    Hs = {xs: torch.zeros(xs.inp, xs.inp, device=dev) for xs in xspecs}
    Us = {xs: torch.empty(xs.inp, xs.inp, dtype=torch.float64, device=dev) for xs in xspecs}
    st = torch.zeros(1, dtype=torch.int32, device=dev)
    max_g = max(B.workspace_bytes(B.WS_GPTQ, w.out, w.inp) for w, _ in wl["layers"].values())
    max_s = max(B.workspace_bytes(B.WS_SCORE, w.out, w.inp) for w, _ in wl["layers"].values())
    max_f = max(B.workspace_bytes(B.WS_FACTOR, 0, xs.inp) for xs in xspecs)
    ws_g = torch.empty(max_g, dtype=torch.uint8, device=dev)
    ws_s = torch.empty(max_s, dtype=torch.uint8, device=dev)
    ws_f = torch.empty(max_f, dtype=torch.uint8, device=dev)
    q = {}
    for lname, variants in jobs:
        w = wl["layers"][lname][0]
        for bits, group, _ in variants:
            q[(lname, bits, group)] = [B.QTensor(w.out, w.inp, bits, group, d, dev)
                                       for d in (B.DIM_OC, B.DIM_IC, B.DIM_OC, B.DIM_IC)]
    err_r = torch.zeros(2, dtype=torch.float64, device=dev)
    err_g = torch.zeros(2, dtype=torch.float64, device=dev)
    ch_r = torch.zeros(1, dtype=torch.int32, device=dev)
    ch_g = torch.zeros(1, dtype=torch.int32, device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    chosen = {}

    def one_step(rec):
        def timed(key, fn):
            if rec is None:
                fn()
                return
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); fn(); e1.record()
            rec.append((key, e0, e1))
        for xs in xspecs:
            def hess(xs=xs):
                Hs[xs].zero_()
                B.hessian_accumulate(Xs[xs], Hs[xs], st)
            timed(("hessian", xs.inp), hess)
            timed(("factor", xs.inp), lambda xs=xs: lib_factor(B, Hs[xs], Us[xs], st, ws_f))
        for lname, variants in jobs:
            W = Ws[lname]
            xs = wl["layers"][lname][1]
            H, U = Hs[xs], Us[xs]
            for bits, group, mode in variants:
                r_oc, r_ic, g_oc, g_ic = q[(lname, bits, group)]
                timed(("rtn", lname, bits, group), lambda: B.quantize_rtn(W, bits, group, B.DIM_BOTH, r_oc, r_ic))
                timed(("score_rtn", lname, bits, group),
                      lambda: B.score_select(W, H, bits, group, r_oc, r_ic, err_r, ch_r, st, ws_s))
                if mode == "both":
                    timed(("gptq", lname, bits, group),
                          lambda: B.quantize_gptq(W, H, bits, group, B.DIM_BOTH, 0.01, U, g_oc, g_ic, None, st, ws_g))
                    timed(("score_gptq", lname, bits, group),
                          lambda: B.score_select(W, H, bits, group, g_oc, g_ic, err_g, ch_g, st, ws_s))
                    chosen[(lname, bits, group)] = ch_g.clone()
                else:
                    dim = int(ch_r.item())               # the one read-back per layer: it decides what runs next
                    chosen[(lname, bits, group)] = dim
                    timed(("gptq", lname, bits, group),
                          lambda: B.quantize_gptq(W, H, bits, group, dim, 0.01, U,
                                                  g_oc if dim == B.DIM_OC else None,
                                                  g_ic if dim == B.DIM_IC else None, None, st, ws_g))

    for _ in range(max(args.warmup, 1)):
        one_step(None)
    torch.cuda.synchronize()
    assert int(st.item()) == 0, f"device status {int(st.item())}"
    sampler = ClockSampler(0)
    sampler.start()
    recs, whole = [], []
    t0 = time.time()
    for k in range(args.steps):
        flush.fill_(k & 0xFF)
        rec = []
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); one_step(rec); e1.record()
        recs.append(rec); whole.append((e0, e1))
    torch.cuda.synchronize()
    clocks = sampler.stop(t0, time.time())
    assert int(st.item()) == 0, f"device status {int(st.item())}"
    ms_per_step = sum(a.elapsed_time(b) for a, b in whole) / args.steps
    ms = {}
    for rec in recs:
        for key, a, b in rec:
            ms[key] = ms.get(key, 0.0) + a.elapsed_time(b) / args.steps

    peaks = _peaks()
    mhz = (clocks or {}).get("sm_mhz") or 1965.0
    ntok = next(iter(xspecs)).n_tokens
    weights_total = sum(w.out * w.inp for w, _ in wl["layers"].values())
    hess_ms = sum(v for k, v in ms.items() if k[0] == "hessian")
    layers = {}
    for lname, variants in jobs:
        w = wl["layers"][lname][0]
        for bits, group, mode in variants:
            stage = {k[0]: v for k, v in ms.items() if k[1:] == (lname, bits, group)}
            roof = stage_rooflines(stage, w.out, w.inp, ntok, bits, group, peaks, mhz, clocks)
            t_layer = sum(stage.values())
            c = chosen[(lname, bits, group)]
            layers[f"{lname} {bits}b g{group}"] = {
                "shape": [w.out, w.inp], "flow": mode, "stages_ms": stage, "ms": t_layer,
                "weights_per_s": w.out * w.inp / (t_layer * 1e-3),
                "chosen": B.DIM_NAMES[int(c.item()) if hasattr(c, "item") else c], "rooflines": roof}
    shared = {}
    for xs in xspecs:
        stage = {"hessian": ms[("hessian", xs.inp)], "factor": ms[("factor", xs.inp)]}
        shared[f"in={xs.inp} ({', '.join(xspecs[xs])})"] = {
            "stages_ms": stage, "rooflines": stage_rooflines(stage, 0, xs.inp, xs.n_tokens, 0, 1, peaks, mhz, clocks)}
    n_var = sum(len(v) for _, v in jobs)
    block_flow = None
    if args.workload == "block":
        # the same block through flows.block_gptq_ada: layers that share an input run GPTQ stacked in one
        # batched call, the dimension is read on the device, the factor runs beside RTN and scoring
        from paper_2309_15531_b200 import flows
        flow_layers = [(n, Ws[n], Xs[wl["layers"][n][1]]) for n, _ in jobs]
        for _ in range(2):
            res = flows.block_gptq_ada(flow_layers, 3, 128, status=st)
        torch.cuda.synchronize()
        t_flow = []
        for k in range(args.steps):
            flush.fill_(k & 0xFF)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            res = flows.block_gptq_ada(flow_layers, 3, 128, status=st)
            e1.record()
            torch.cuda.synchronize()
            t_flow.append(e0.elapsed_time(e1))
        assert int(st.item()) == 0, f"device status {int(st.item())}"
        flow_ms = sum(t_flow) / len(t_flow)
        same = all(int(res[n][0].item()) == (chosen[(n, 3, 128)]) for n, _ in jobs)
        block_flow = {"ms_per_block": flow_ms, "ms_per_block_without_hessians": flow_ms - hess_ms,
                      "weights_per_s": weights_total / (flow_ms * 1e-3),
                      "weights_per_s_without_hessians": weights_total / ((flow_ms - hess_ms) * 1e-3),
                      "same_choices_as_layer_by_layer": bool(same),
                      "how": "flows.block_gptq_ada: layers that share an input share H and U and run GPTQ stacked in batched "
                             "calls of at most 148 slabs (q,k,v,o together; gate, up, down one call each); the factor runs "
                             "beside RTN and scoring; no host read-back between RTN selection and GPTQ"}
    # the dominant kernel of these configurations too is the Hessian's tensor-core kernel
    big = max(xspecs, key=lambda xs: xs.inp)
    roofline = dict(shared[f"in={big.inp} ({', '.join(xspecs[big])})"]["rooflines"]["hessian"])
    roofline["kernel"] = f"tc_kernel<Hessian>, in={big.inp}"
    roofline["traffic"] = None
    line = {
        "metric": METRIC, "value": weights_total / (ms_per_step * 1e-3), "unit": "weights/s", "n_gpus": 1,
        "steps": args.steps, "warmup": max(args.warmup, 1), "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": DTYPE, "data": "synthetic",
        "config": {"workload": f"{wl['name']}: {len(jobs)} layer(s), {n_var} layer-variant(s), {ntok} calibration tokens; "
                               "one Hessian and one factor per distinct input width",
                   "l2": "flushed between steps by writing a 256 MiB buffer; every X exceeds L2", "replicas": 1},
        "ms_per_step_without_hessians": ms_per_step - hess_ms,
        "weights_per_s_without_hessians": weights_total / ((ms_per_step - hess_ms) * 1e-3),
        "layers": layers, "shared": shared, "block_flow": block_flow, "roofline": roofline, "cpu_baseline": None,
        "e2e": None, "e2e_note": "the host-buffer leg is measured on the default workload only",
        "clocks": clocks,
        "gpu_launches": args.steps * (sum(launches_hessian_factor(xs.inp) for xs in xspecs) +
                                      sum(launches_layer(wl["layers"][n][0].inp, m == "both")
                                          for n, v in jobs for _, _, m in v)),
    }
    print(json.dumps(line))


# A100-80GB latencies the paper prints for its own per-IC kernel on this workload (Appendix D, Table 10), ms
PAPER_GEMV_MS = {(4, 128): 0.50477, (4, 256): 0.32926, (4, 512): 0.24570, (4, 2048): 0.20425,
                 (3, 128): 0.47336, (3, 256): 0.29957, (3, 512): 0.21457, (3, 2048): 0.16735}


def run_gemv(args):
    """The matrix-vector product of Appendix D: weight 4m x m with m = 12288, per-IC groups of 128 ... 2048,
    INT3 / INT4, fp16 vector in and out.  One step = one product; codes and parameters are seeded random
    (the product's cost does not depend on their values)."""
    import torch
    from paper_2309_15531_b200 import binding as B

    if int(os.environ.get("RANK", "0")) != 0:
        return
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    m = 12288
    out, inp = 4 * m, m
    peaks = _peaks()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    g = torch.Generator(device=dev).manual_seed(230915531)
    x = torch.randn(inp, device=dev, generator=g).half()
    y = torch.empty(out, dtype=torch.float16, device=dev)
    sampler = ClockSampler(0)
    sampler.start()
    t0 = time.time()
    rows = {}
    for bits in (4, 3):
        codes = torch.randint(-2 ** 31, 2 ** 31 - 1, (out, inp * bits // 32), device=dev, generator=g,
                              dtype=torch.int64).int()
        for group in (128, 256, 512, 2048):
            scales = (torch.rand(out // group, inp, device=dev, generator=g) * 0.01 + 0.001).half()
            zeros = torch.randint(0, 2 ** bits, (out // group, inp), device=dev, generator=g).half()
            ws = torch.empty(B.workspace_bytes(B.WS_GEMV, out, inp, bits, group), dtype=torch.uint8, device=dev)
            for _ in range(max(args.warmup, 3)):
                B.dequant_gemv(codes, scales, zeros, bits, group, x, y, ws)
            ts = []
            for k in range(args.steps):
                flush.fill_(k & 0xFF)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(); B.dequant_gemv(codes, scales, zeros, bits, group, x, y, ws); e1.record()
                torch.cuda.synchronize()
                ts.append(e0.elapsed_time(e1))
            ms = sum(ts) / len(ts)
            nbytes = out * inp * bits / 8 + (out // group) * inp * 4 + inp * 2 + out * 2
            ach = nbytes / (ms * 1e-3) / 1e9
            rows[f"int{bits} g{group}"] = {"ms": ms, "weights_per_s": out * inp / (ms * 1e-3),
                                           "roofline": {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                                        "frac": ach / peaks["hbm_gbs"], "algorithmic_bytes": nbytes},
                                           "paper_a100_ms": PAPER_GEMV_MS[(bits, group)],
                                           "paper_a100_ms_over_ours": PAPER_GEMV_MS[(bits, group)] / ms}
    clocks = sampler.stop(t0, time.time())
    head = rows["int3 g128"]
    line = {"metric": "per-IC dequant GEMV latency (4m x m, m = 12288; Appendix D Table 10)", "value": head["ms"], "unit": "ms",
            "n_gpus": 1, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": head["ms"],
            "higher_is_better": False, "scaling": "weak", "vs_baseline": head["ms"] / PAPER_GEMV_MS[(3, 128)],
            "vs_baseline_note": "the paper's number is its own kernel on an A100-80GB: context, not a target",
            "dtype": "s8 (integer matrix instruction on unpacked codes against a 21-bit fixed-point image of scale * x), fp16 in and out",
            "data": "synthetic", "config": {"workload": "OPT-175B first FFN layer shape W[49152,12288], INT3 g128 (headline); "
                                                        "all of Table 10's group sizes and both precisions in `cases`",
                                            "l2": "flushed between steps by writing a 256 MiB buffer", "replicas": 1},
            "cases": rows, "roofline": dict(head["roofline"], kernel="gemv_product_kernel<3> (+ gemv_prepare_kernel)", traffic=None),
            "cpu_baseline": None, "e2e": None, "clocks": clocks, "gpu_launches": 2 * 8 * args.steps}
    print(json.dumps(line))


def lib_factor(B, H, U, st, ws_f):
    """adadim_cholesky_inverse_factor into a preallocated U."""
    rc = B.lib().adadim_cholesky_inverse_factor(H.data_ptr(), H.shape[0], 0.01, U.data_ptr(), st.data_ptr(),
                                                ws_f.data_ptr(), ws_f.numel(), B._stream())
    B._check(rc, "adadim_cholesky_inverse_factor")


# --------------------------------------------------------------------------- CPU oracle arm
def cpu_baseline():
    """Times the oracle, as it stands, on a bounded sample of the same workload and scales each
    stage to the full layer.  Returns the cpu_baseline object."""
    import numpy as np
    import torch
    from oracle import adadim_oracle as O
    from paper_2309_15531_b200 import inputs as I

    wl = I.workload_qproj(n_tokens=1024)
    wspec, xspec = wl["layers"]["q_proj"]
    out, inp, full_tokens = wspec.out, wspec.inp, 128 * 2048
    W = I.make_weight(wspec, "cpu").float().numpy()
    X = I.make_calib(xspec, "cpu").float().numpy()
    slab = 128
    t = {}
    t0 = time.time(); H = O.hessian(X); t["hessian"] = (time.time() - t0) * (full_tokens / xspec.n_tokens)
    t0 = time.time()
    r = {d: O.quantize_rtn(W, BITS, GROUP, d) for d in ("oc", "ic")}
    t["rtn"] = time.time() - t0
    t0 = time.time()
    for d in ("oc", "ic"):
        O.recon_error_trace(W[:512], r[d]["Q"][:512], H)
    t["score"] = (time.time() - t0) * (out / 512) * 2           # scored twice per step (RTN and GPTQ outputs)
    t0 = time.time(); Hd, dead = O.damped_hessian(H, 0.01); U = O.cholesky_inverse_factor(Hd); t["factor"] = time.time() - t0
    t0 = time.time()
    for d in ("oc", "ic"):
        O.quantize_gptq(W[:slab], H, BITS, GROUP, d, 0.01, U=U, dead=dead)
    t["gptq"] = (time.time() - t0) * (out / slab)
    total = sum(t.values())
    cores = len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else os.cpu_count()
    return {"value": out * inp / total, "unit": "weights/s", "cores": min(cores, torch.get_num_threads() or cores),
            "kind": "oracle",
            "sample": "Hessian on 1024 of 262144 tokens, RTN on the full W, scorer on 512 of 4096 rows, "
                      "factor in full, GPTQ on one 128-row slab of 32; each stage scaled linearly to the full layer",
            "stage_seconds_scaled": t}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    vals = []
    for _ in range(max(1, min(args.warmup, 1))):
        cpu_baseline()
    t_all = 0.0
    last = None
    n = max(1, min(args.steps, 3))
    for _ in range(n):
        last = cpu_baseline()
        vals.append(last["value"])
    value = sum(vals) / len(vals)
    last["value"] = value
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": "weights/s", "n_gpus": args.gpus,
            "steps": n, "warmup": 1, "ms_per_step": 4096 * 4096 / value * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD, "l2": "not applicable: CPU oracle on a bounded sample scaled to the full layer",
                       "replicas": 1},
            "cpu_baseline": last,
            "e2e": {"value": value, "unit": "weights/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="q_proj", choices=["q_proj", "down_proj", "block", "mlp70b", "gemv"])
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the oracle timing (profiling runs)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.workload == "gemv":
        run_gemv(args)
    elif args.workload != "q_proj":
        run_config(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
