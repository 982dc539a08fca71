#!/usr/bin/env python
"""Benchmark of the SAGE selection hot path on B200.

A "step" is one pass of the whole path over one synthetic workload: pass 1 (Frequent-Directions sketch
of all N rows, including the freeze), pass 2 (projection, normalisation, consensus, agreement scores)
and the top-k selection. Metric: gradient rows per second through the whole path (N / step time),
summed over ranks; with more than one GPU every rank runs an independent replica of the workload.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workloads c1,c2,c3,c4,c5] [--headline c5]
                    [--impl ours|reference]

One invocation runs every listed workload and prints ONE JSON line (rank 0). The top-level fields are those of
the headline workload (default: c5, the largest one that fits one GPU), timed over exactly K steps after W
warm-up steps; the other workloads follow under "workloads" with the same fields, each timed over
10 steps (c1-c3) or min(K, 5) steps (c4) so that the whole run stays within minutes: c1..c4 with the paper's sequential sketch, the same four
with the merged form of pass 1 (16 sketches, "cN_merged16"), and c2 / c3 given as the factors of their rows
("cN_factored"). `--impl reference` times the fp64 CPU oracle on
the host cores instead, on a bounded sample of the headline workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

# The merged form of pass 1 runs one stream per sketch; CUDA gives every stream a hardware queue of its own only up to this
# number (default 8). It is read when CUDA is initialised, so it has to be set before torch touches the device.
os.environ.setdefault("CUDA_DEVICE_MAX_CONNECTIONS", "32")

import torch  # noqa: E402

METRIC = "gradient rows/s (FD sketch + agreement scoring + top-k, whole path)"
UNIT = "rows/s"
FP32_ALU_PEAK_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12     # SMs x FMA lanes x 2 flop x max SM clock
ALL = ("c1", "c2", "c3", "c4", "c5")
# DRAM bytes per launch of the dominant streaming kernels from one ncu capture each (profiles/): the capture ran on a
# scaled-down D and the traffic grows in proportion to D, so the figure is stored per buffer column.
# (Gram and rebuild: launches of cycles that read their 65 new rows in place, as 7 of 8 cycles of c5 do.)
NCU_TRAFFIC_PER_COLUMN = {("c5", "rebuild"): (431.471e6 + 246.243e6) / 1117396, ("c5", "gram"): (433.734e6 + 3.507e6) / 1117396,
                          ("c5", "project"): (1294.674e6 + 3.727e6) / 1117396}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def shrink_schedule(N: int, ell: int):
    """Row counts of every factorisation of one pass 1: full buffers (m rows) and the final one."""
    m, keep = 2 * ell, ell - 1
    fill, full = 0, 0
    left = N
    while left > 0:
        take = min(left, m - fill)
        fill += take
        left -= take
        if fill == m:
            full += 1
            fill = keep
    return full, fill


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples taken while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None

    def start(self):
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100",
                                       "-i", str(self.gpu)], stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self):
        if self.p is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, reasons, power = [], [], set(), []
        for line in self.f.read().splitlines():
            c = [x.strip() for x in line.split(",")]
            if len(c) < 9:
                continue
            try:
                sm.append(float(c[1]))
                mx.append(float(c[2]))
                power.append(float(c[3]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), c[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        os.unlink(self.f.name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


# Rows of each workload the oracle is timed on: chosen so that one run costs roughly 10 to 40 s of host time.
CPU_SAMPLE_ROWS = {"c1": 4096, "c2": 20000, "c3": 2000, "c4": 768, "c5": 100}


def sample_rows_for(w, n):
    """The first n rows of a workload as a CPU tensor (streamed workloads are generated on the device and copied)."""
    from paper_2510_02470_b200 import workloads as wl
    if w.on_device:
        stream = wl.DeviceStream(wl.scaled(w, N=n), 0, "cuda" if torch.cuda.is_available() else "cpu")
        return torch.cat([stream.chunk(j) for j in range((n + w.chunk_rows - 1) // w.chunk_rows)])[:n].cpu()
    return wl.host_rows(w, 0, n)


def cpu_oracle_sample(w, sample_rows, rows=None):
    """The oracle, as it stands, on the first `sample_rows` rows of the workload, on the host cores."""
    import oracle
    if rows is None:
        rows = sample_rows_for(w, sample_rows)
    oracle.lib()
    route = 0 if w.D <= 20000 else 1
    t0 = time.perf_counter()
    out = oracle.run(rows, w.D, w.ell, w.keep_rates[0], route=route)
    dt = time.perf_counter() - t0
    cores = int(os.environ.get("OMP_NUM_THREADS", os.cpu_count() or 1))
    return {"value": sample_rows / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"first {sample_rows} rows of {w.name} through sketch+freeze+score+select, {dt:.1f} s, "
                      f"{out['stats']['shrinks']} shrinks, SVD route {'rows (Hestenes)' if route == 0 else 'Gram'}",
            "seconds": dt}


# Rough cost model of the oracle (host seconds) used only to size the reference arm's sample: flops of the Gram route per
# shrink and per scored row at a nominal 8 GFLOP/s for its naive fp64 loops on the host cores.
def oracle_seconds_estimate(w, n):
    full, r_final = shrink_schedule(n, w.ell)
    m = 2 * w.ell
    if w.D <= 20000:
        flop = (full + 1) * 8 * 6.0 * m * m * w.D          # Hestenes: about 8 sweeps of 6 m^2 D
    else:
        flop = full * (m * m + 2.0 * w.ell * m) * w.D + (r_final * r_final + 2.0 * w.ell * r_final) * w.D
    flop += 2.0 * n * w.ell * w.D
    return flop / 8e9


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    # a bounded sample: the whole run (warm-up + timed steps) should end within a few minutes
    budget = 200.0 / max(1, args.steps + args.warmup)
    sample = min(CPU_SAMPLE_ROWS[w.name], w.N)
    while sample > 16 and oracle_seconds_estimate(w, sample) > budget:
        sample = max(16, int(sample * 0.8))
    rows = sample_rows_for(w, sample)
    times = []
    base = None
    for i in range(args.warmup + args.steps):
        base = cpu_oracle_sample(w, sample, rows)
        if i >= args.warmup:
            times.append(base["seconds"])
    dt = sum(times) / len(times)
    v = sample / dt
    line = {"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "N": w.N, "D": w.D, "ell": w.ell, "rows_dtype": str(w.dtype).replace("torch.", ""),
                       "sample_rows_per_step": sample},
            "cpu_baseline": {"value": v, "unit": UNIT, "cores": base["cores"], "kind": "oracle", "sample": base["sample"]},
            "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}, "gpu_launches": 0}
    print(json.dumps(line))


def run_workload(w, args, steps, warmup, ctx, want_e2e, want_cpu, sketches, factored=False):
    """Times `steps` steps of one workload after `warmup` warm-up steps; returns the fields of its JSON entry."""
    import paper_2510_02470_b200 as sage
    from paper_2510_02470_b200 import replicas
    from paper_2510_02470_b200 import workloads as wl
    dev, local, world, rank = ctx["dev"], ctx["local"], ctx["world"], ctx["rank"]
    N, D, ell = w.N, w.D, w.ell
    e = w.elem_bytes
    # ---- inputs ------------------------------------------------------------------------------------
    t_gen0 = time.perf_counter()
    host_rows = None
    stream = None
    rows = None
    chunk_buf = None
    qf = hf = None
    C_out = F_out = 0
    if factored:             # last-layer workloads given as the factors of their rows (no N x D matrix anywhere)
        C_out = {"c2": 10, "c3": 100}[w.name]
        F_out = (D - C_out) // C_out
        q_host, h_host = wl.host_factors(w, args.seed, N)
        qf, hf = q_host.to(dev), h_host.to(dev)
    elif w.on_device:
        stream = wl.DeviceStream(w, args.seed, dev)
        chunk_buf = torch.zeros((w.chunk_rows, w.ld), dtype=w.dtype, device=dev)
    else:
        host_rows = wl.host_rows(w, args.seed).pin_memory()
        rows = host_rows.to(dev, non_blocking=True)
    torch.cuda.synchronize()
    t_gen = time.perf_counter() - t_gen0

    fd = sage.SageFD(D, ell, w.dtype, local)
    if sketches > 1:
        fd.set_option(6, sketches)
    scores = torch.empty((N,), dtype=torch.float32, device=dev)
    # one selection at the largest keep-rate: the output is ordered (score descending, index ascending), so the
    # selection for every smaller keep-rate is a prefix of it
    top_rate = max(w.keep_rates)
    idx_buf = torch.empty((sage.sage_select_count(N, top_rate),), dtype=torch.int64, device=dev)
    ev = lambda: torch.cuda.Event(enable_timing=True)

    def one_step(phase_events=None):
        """sketch all rows -> freeze -> score all rows -> select; results stay on the device."""
        marks = [ev() for _ in range(4)] if phase_events is not None else None
        fd.reset()
        if marks: marks[0].record()
        if factored:
            fd.update_outer(qf, hf, C_out, F_out)
        elif stream is None:
            fd.update(rows)
        else:
            for j in range(w.num_chunks):
                g0, g1 = ev(), ev()
                g0.record()
                c = stream.chunk(j, chunk_buf)
                g1.record()
                fd.update(c)
                if sketches > 1:
                    fd.join()        # the next chunk is generated only after this one's work: generator time can be subtracted
                if phase_events is not None:
                    phase_events.setdefault("gen1", []).append((g0, g1))
        fd.finalize(allow=(6, 7))
        if marks: marks[1].record()
        if factored:
            fd.score_outer(qf, hf, C_out, F_out, scores)
        elif stream is None:
            fd.score(rows, scores)
        else:
            fd.score_begin(N)
            for j in range(w.num_chunks):
                g0, g1 = ev(), ev()
                g0.record()
                c = stream.chunk(j, chunk_buf)
                g1.record()
                fd.score_chunk(c, j * w.chunk_rows)
                if phase_events is not None:
                    phase_events.setdefault("gen2", []).append((g0, g1))
            fd.score_end(scores)
        if marks: marks[2].record()
        sage.sage_select(scores, top_rate, idx_buf)
        if marks:
            marks[3].record()
            phase_events["marks"] = marks

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
            torch.cuda.synchronize()

    # ---- warm-up (the last warm-up step is profiled per kernel class to find the dominant kernel) ----
    for i in range(warmup):
        if i == warmup - 1:
            fd.set_option(3, 0x1FF)
            fd.profile()
        one_step()
    torch.cuda.synchronize()
    prof_all = fd.profile()
    dominant = max(prof_all, key=lambda k: prof_all[k]["ms"])
    dom_bit = sage.KERNEL_CLASSES.index(dominant)
    fd.set_option(3, 1 << dom_bit)          # during the timed region only the dominant kernel is bracketed by events

    # ---- timed region -----------------------------------------------------------------------------------
    sampler = ClockSampler(local)
    phase = [dict() for _ in range(steps)]
    launches0 = sage.sage_launch_count()
    barrier()
    sampler.start()
    t0, t1 = ev(), ev()
    t0.record()
    for s in range(steps):
        one_step(phase[s])
    t1.record()
    barrier()
    clocks = sampler.stop()
    launches = sage.sage_launch_count() - launches0
    total_ms = t0.elapsed_time(t1)
    gen1_ms = sum(a.elapsed_time(b) for p in phase for (a, b) in p.get("gen1", [])) / steps
    gen2_ms = sum(a.elapsed_time(b) for p in phase for (a, b) in p.get("gen2", [])) / steps
    gen_total_ms = (gen1_ms + gen2_ms) * steps
    step_ms = (total_ms - gen_total_ms) / steps          # generator time (streamed workloads) excluded
    prof_dom = fd.profile()[dominant]
    p1 = statistics.mean(p["marks"][0].elapsed_time(p["marks"][1]) for p in phase) - gen1_ms   # generator time excluded
    p2 = statistics.mean(p["marks"][1].elapsed_time(p["marks"][2]) for p in phase) - gen2_ms
    p3 = statistics.mean(p["marks"][2].elapsed_time(p["marks"][3]) for p in phase)
    gen_per_step = gen_total_ms / steps
    stats = fd.stats()

    step_ms = replicas.max_over_ranks(step_ms, dev)            # replicas only: the job is as slow as its slowest rank
    value = replicas.whole_job_rows_per_s(N, world, step_ms)

    # ---- roofline of the dominant kernel -------------------------------------------------------------------
    peaks = measured_peaks()
    full, r_final = shrink_schedule(N, ell)
    m, keep = 2 * ell, ell - 1
    keep_final = (ell - 1) if r_final > ell else min(r_final, ell)
    # rows that whole shrink cycles read in place (never appended; bf16, 2 bytes instead of the buffer's 4): counted by the
    # library since the reset at the start of the last step
    in_place = stats.get("rows_in_place", 0)
    per_step_bytes = {
        "append": (N - in_place) * D * (e + 4),
        "gram": (full * m + r_final) * D * 4 - in_place * D * (4 - e),
        "rebuild": (full * (m + keep) + (r_final + max(keep_final, ell))) * D * 4 - in_place * D * (4 - e),
        "project": N * D * e,
        "normalise": N * ell * 8,
        "score": N * ell * 4 + N * 4,
    }
    eig_flops = 9.0 * (full * m ** 3 + r_final ** 3)
    dom_ms_per_step = prof_dom["ms"] / steps
    dom_launches_per_step = prof_dom["launches"] / steps
    if dominant == "eig_shrink":
        achieved = eig_flops / (dom_ms_per_step * 1e-3) / 1e12
        roof = {"kernel": "k_eig_shrink_fast" if 2 * ell <= 64 else "k_eig_shrink_dsm", "bound": "alu", "achieved": achieved,
                "peak": FP32_ALU_PEAK_TFLOPS, "unit": "TFLOP/s", "frac": achieved / FP32_ALU_PEAK_TFLOPS, "traffic": None,
                "peak_source": "derived: 148 SMs x 128 fp32 FMA lanes x 2 flop x 1.965 GHz",
                "algorithmic": "9*n^3 flop per n x n symmetric eigen-solve (textbook count)",
                "frac_of_the_sms_it_runs_on": achieved / (FP32_ALU_PEAK_TFLOPS * (1 if 2 * ell <= 64 else 8) / 148.0)}
    else:
        gbs = per_step_bytes.get(dominant, 0) / (dom_ms_per_step * 1e-3) / 1e9
        kname = {"gram": "k_tc_gemm_nt_x3 (Gram)", "rebuild": "k_tc_rebuild", "append": "k_append",
                 "project": "k_tc_gemm_nt (projection)"}.get(dominant, dominant)
        traffic = NCU_TRAFFIC_PER_COLUMN.get((w.name, dominant))
        roof = {"kernel": kname, "bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": gbs / peaks["hbm_gbs"], "traffic": traffic * D if traffic else None,
                "peak_source": f"{peaks['source']} STREAM-style copy",
                "algorithmic_bytes_per_launch": per_step_bytes.get(dominant, 0) / max(dom_launches_per_step, 1)}
    if sketches > 1:
        roof["note"] = (f"{sketches} sketches run their kernels side by side: the per-kernel times are sums over launches that overlap "
                        "in time, so achieved / share_of_step describe one launch's pace, not the device's")
    roof["avg_launch_ms"] = dom_ms_per_step / max(dom_launches_per_step, 1)
    roof["launches_per_step"] = dom_launches_per_step
    roof["share_of_step"] = dom_ms_per_step / step_ms
    kernels = {}
    for name, v in prof_all.items():
        if v["launches"] == 0:
            continue
        entry = {"ms_per_step": v["ms"], "launches_per_step": v["launches"]}
        if name in per_step_bytes and v["ms"] > 0:
            entry["GBps"] = per_step_bytes[name] / (v["ms"] * 1e-3) / 1e9
            entry["frac_of_hbm"] = entry["GBps"] / peaks["hbm_gbs"]
        kernels[name] = entry
    roof_pass2_s = max(N * D * e / (peaks["hbm_gbs"] * 1e9), 2.0 * N * ell * D / (peaks["bf16_tflops_sustained"] * 1e12))
    # pass-1 roofline: the bytes of the method with every row appended to an fp32 buffer (append read + write, Gram read,
    # rebuild read + write); cycles that read their rows in place move fewer, so the fraction compares TIME with that model
    p1_bytes = N * D * (e + 4) + (full * m + r_final) * D * 4 + (full * (m + keep) + (r_final + max(keep_final, ell))) * D * 4
    roof_pass1_s = p1_bytes / (peaks["hbm_gbs"] * 1e9)
    stream_ms = sum(prof_all[k]["ms"] for k in ("append", "gram", "gram_reduce", "rebuild"))

    # ---- class-balanced variant on the scores of the last step (reported beside the step, not part of it) ----
    cb_info = None
    try:
        C_cls = {"c1": 16, "c2": 10, "c3": 100, "c4": 64, "c5": 10}[w.name]
        gcb = torch.Generator(device=dev)
        gcb.manual_seed(1234)
        labels = torch.randint(0, C_cls, (N,), generator=gcb, device=dev, dtype=torch.int32)
        cb_scores = torch.empty((N,), dtype=torch.float32, device=dev)
        c0, c1 = ev(), ev()
        fd.score_classes(labels, C_cls, cb_scores)
        sage.sage_select_classes(cb_scores, labels, C_cls, w.keep_rates[0])
        torch.cuda.synchronize()
        c0.record()
        for _ in range(3):
            fd.score_classes(labels, C_cls, cb_scores)
            sage.sage_select_classes(cb_scores, labels, C_cls, w.keep_rates[0])
        c1.record()
        torch.cuda.synchronize()
        cb_info = {"classes": C_cls, "labels": "uniform random (synthetic)", "ms_score_and_select": c0.elapsed_time(c1) / 3}
    except Exception as exc:       # the variant needs a finished scoring pass on the handle
        cb_info = {"error": str(exc)}

    fd.close()
    del rows, chunk_buf, stream, scores, idx_buf, qf, hf
    torch.cuda.empty_cache()

    # ---- end to end through the host-pointer entry point ------------------------------------------------
    e2e = None
    if want_e2e and not factored:
        note = None
        if host_rows is None:
            # streamed workloads do not fit host memory as N x D: a prefix of the same rows, copied to pinned host memory
            n_e2e = min(N, max(4 * ell, int(24e9 // (w.ld * e))))
            host_rows = sample_rows_for(w, n_e2e).pin_memory()
            torch.cuda.empty_cache()
            note = f"first {n_e2e} rows of the workload (the N x D matrix does not fit host memory); cost per row does not depend on N"
        n_rows = host_rows.shape[0]
        reps = max(1, min(steps, 3))
        sage.sage_select_from_host(host_rows, D, ell, w.keep_rates[0], 0, local)      # warm-up
        torch.cuda.synchronize()
        t_e = time.perf_counter()
        for _ in range(reps):
            sc, ix = sage.sage_select_from_host(host_rows, D, ell, w.keep_rates[0], 0, local)
        torch.cuda.synchronize()
        dt = (time.perf_counter() - t_e) / reps
        dt = replicas.max_over_ranks(dt, dev)
        e2e = {"value": replicas.whole_job_rows_per_s(n_rows, world, dt * 1e3), "unit": UNIT,
               "h2d_bytes_per_step": 2 * n_rows * w.ld * e, "d2h_bytes_per_step": n_rows * 4 + int(ix.numel()) * 8,
               "ms_per_step": dt * 1e3, "rows": n_rows,
               "call": "sage_select_from_host (pinned host rows, both passes streamed over PCIe, one keep_rate; the handle, "
                       "its buffers and streams are created and destroyed inside the call)"}
        if note:
            e2e["sample"] = note
    del host_rows

    cpu = None
    if want_cpu and rank == 0 and world == 1:
        b = cpu_oracle_sample(w, min(CPU_SAMPLE_ROWS[w.name], N))
        cpu = {k: b[k] for k in ("value", "unit", "cores", "kind", "sample")}

    return {
        "value": value, "unit": UNIT, "steps": steps, "warmup": warmup, "ms_per_step": step_ms,
        "config": {"workload": w.name, "N": N, "D": D, "ell": ell, "rows_dtype": str(w.dtype).replace("torch.", ""),
                   "ld": w.ld, "keep_rates": list(w.keep_rates), "sketches": sketches,
                   "input": "factors of the rows (softmax - onehot, features)" if factored else "rows", "multi_gpu": "replicas only",
                   "l2": "inputs larger than L2" if N * D * e > 200e6 else "inputs fit in L2 (no flush: stated, c1 only)",
                   "generator_ms_per_step_excluded": gen_per_step, "input_generation_s": t_gen},
        "passes": {"pass1_ms": p1, "pass2_ms": p2, "select_ms": p3,
                   "pass1_rows_per_s": N / (p1 * 1e-3) if p1 > 0 else None, "pass2_rows_per_s": N / (p2 * 1e-3) if p2 > 0 else None,
                   "pass1_frac_of_hbm_roofline": roof_pass1_s / (p1 * 1e-3) if p1 > 0 else None,
                   "pass2_frac_of_roofline": roof_pass2_s / (p2 * 1e-3) if p2 > 0 else None,
                   "pass1_stream_kernels_ms": stream_ms, "pass1_eig_ms": prof_all["eig_shrink"]["ms"],
                   "pass1_stream_frac_of_hbm_roofline": (roof_pass1_s * 1e3) / max(1e-9, stream_ms),
                   "note": "generator time of streamed workloads is excluded from the pass times; *_stream_* figures are "
                           "CUDA-event sums over the streaming kernels of the profiled warm-up step (eigen-solves apart)"},
        "roofline": roof, "kernels_profiled_step": kernels, "class_balanced": cb_info,
        "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": int(launches), "clocks": clocks,
        "fd_stats": {k: stats[k] for k in ("shrinks", "max_sweeps", "last_rank", "device_flags")},
    }


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workloads", default=",".join(ALL), help="comma-separated subset of c1..c5 to run")
    ap.add_argument("--workload", default=None, help="run this one workload only (it is then the headline)")
    ap.add_argument("--headline", default="c5", help="workload whose fields go to the top level of the JSON line")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--rows", type=int, default=0, help="use only the first ROWS rows of each workload (debugging)")
    ap.add_argument("--dim", type=int, default=0, help="override the row dimension D (small cases for profiler captures)")
    ap.add_argument("--sketches", type=int, default=1, help="number of sub-sketches of pass 1 (1 = the sequential sketch)")
    ap.add_argument("--no-variants", action="store_true", help="skip the merged-sketch and factored-input runs")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--seed", type=int, default=0)
    args = ap.parse_args()

    from paper_2510_02470_b200 import workloads as wl
    names = [args.workload] if args.workload else [n for n in args.workloads.split(",") if n]
    for n in names:
        if n not in ALL:
            raise SystemExit(f"unknown workload {n}")
    headline = args.headline if args.headline in names else names[-1]

    def shaped(name):
        w = wl.WORKLOADS[name]
        if args.rows:
            w = wl.scaled(w, N=min(args.rows, w.N))
        if args.dim:
            w = wl.scaled(w, D=args.dim)
        return w

    if args.impl == "reference":
        run_reference(args, shaped(headline))
        return
    args.warmup = max(args.warmup, 3)

    import paper_2510_02470_b200 as sage
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    sage.lib()
    ctx = {"dev": dev, "local": local, "world": world, "rank": rank}

    # Every workload with the paper's sequential sketch; beside it (unless --no-variants) the merged form of pass 1 with 16
    # sketches on the workloads whose pass 1 is a chain of eigen-solves, and the last-layer workloads given as factors.
    # The headline comes last and is the only one timed over exactly --steps steps.
    runs = [(n, n, args.sketches, False) for n in names if n != headline]
    if not args.no_variants and args.sketches == 1 and not args.rows and not args.dim:
        runs += [(f"{n}_merged16", n, 16, False) for n in names if n in ("c1", "c2", "c3", "c4") and n != headline]
        runs += [(f"{n}_factored", n, 1, True) for n in names if n in ("c2", "c3") and n != headline]
    runs.append((headline, headline, args.sketches, False))
    results = {}
    for key, n, P, fact in runs:
        w = shaped(n)
        is_head = key == headline
        # the headline is timed over exactly --steps steps; beside it the short workloads (c1-c3: a step is 6-460 ms) get
        # ten timed steps, the long one (c4) at most five, unless fewer were asked for
        steps = args.steps if is_head else (min(args.steps, 5) if (n in ("c4", "c5") or args.steps < 3) else 10)
        warm = args.warmup if is_head else 3
        results[key] = run_workload(w, args, steps, warm, ctx, want_e2e=not args.no_e2e and not fact and P == args.sketches and (is_head or not w.on_device),
                                    want_cpu=not args.no_cpu_baseline and is_head, sketches=P, factored=fact)

    if rank == 0:
        head = results[headline]
        line = {"metric": METRIC, "value": head["value"], "unit": UNIT, "n_gpus": world, "steps": head["steps"],
                "warmup": head["warmup"], "ms_per_step": head["ms_per_step"], "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "f32", "data": "synthetic"}
        for k in ("config", "passes", "roofline", "kernels_profiled_step", "class_balanced", "cpu_baseline", "e2e",
                  "gpu_launches", "clocks", "fd_stats"):
            line[k] = head[k]
        line["workloads"] = {n: r for n, r in results.items() if n != headline}
        print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
