#!/usr/bin/env python
"""Benchmark of the CIAR hot path: tokens/s quantified + verified on synthetic LlamaGen-384-like
logits (16 images x 24x24 tokens, V = 16384, bf16, draft window 16).

One "step" is one pass of the whole path over the batch: ciar_quantify on every row, then
ciar_verify (Algorithm 1's anchored windows) with the flags and softmax statistics quantify
produced.  `value` times K steps with the inputs resident in HBM; `e2e` times the same calls
with the step's inputs copied from pinned host memory and the results copied back inside the
timed region.  `--impl reference` times the CPU oracle on a bounded sample of the same workload.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]
Multi-GPU: launched by torchrun, one rank per GPU; every rank processes its own batch (weak
scaling), no data-path collective; time = max over ranks.
"""
import argparse
import json
import os
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2603_25463_b200 import dist as ciar_dist, synth

METRIC = "tokens/s quantified+verified"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
CLOCK_QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
               "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
               "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """nvidia-smi polled in the background while the timed region runs (read-only)."""

    def __init__(self, device_index: int):
        self.proc = None
        self.why = None
        self.path = "/tmp/ciar_clocks_%d_%d.csv" % (os.getpid(), device_index)
        try:
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            sel = uuid if uuid.startswith("GPU-") else "GPU-" + uuid
        except Exception:
            sel = str(device_index)
        self.cmd = ["nvidia-smi", "-i", sel, "--query-gpu=" + CLOCK_QUERY, "--format=csv,noheader,nounits", "-lms", "50"]

    def start(self):
        try:
            self.out = open(self.path, "w")
            self.err = open(self.path + ".err", "w")
            self.proc = subprocess.Popen(self.cmd, stdout=self.out, stderr=self.err)
        except Exception as e:
            self.proc = None
            self.why = "nvidia-smi could not be started: %r" % (e,)

    def stop(self):
        res = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            res["note"] = self.why
            return res
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.out.close()
        self.err.close()
        sm, mx, reasons = [], [], set()
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1])); mx.append(float(f[2]))
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.remove(self.path)
        except Exception:
            pass
        if sm:
            res.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), reasons=sorted(reasons), samples=len(sm))
        else:
            try:
                res["note"] = "no samples: " + open(self.path + ".err").read().strip()[:200]
            except Exception:
                res["note"] = "no samples"
        try:
            os.remove(self.path + ".err")
        except Exception:
            pass
        return res


def dist_setup(n_gpus):
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    else:
        torch.cuda.set_device(0)
    return rank, world, local


def barrier(world):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    torch.cuda.synchronize()


def max_over_ranks(x: float, world: int) -> float:
    return ciar_dist.max_over_ranks(x, world, torch.device("cuda") if world > 1 else None)


class Step:
    """The hot path on one resident batch: quantify -> verify through the C ABI binding."""

    def __init__(self, ciar, wl, inp, per_code=False):
        self.ciar, self.wl = ciar, wl
        dev = inp.draft.device
        self.draft, self.target = inp.draft, inp.target
        self.tokens, self.ua, self.ur = inp.tokens, inp.u_accept, inp.u_resample
        if per_code:  # one raw radius per code, as the interval head emits it (Softplus applied on the device)
            self.params = ciar.IntervalParams(radius_mode=ciar.RADIUS_PER_CODE, radius=inp.radius_code, radius_is_raw=True,
                                              tau=wl.tau)
        else:
            self.params = ciar.IntervalParams(radius_mode=ciar.RADIUS_PER_ROW, radius=inp.radius_row, tau=wl.tau)
        rows = inp.draft.shape[0]
        self.rows = rows
        self.qout = ciar.QuantifyOut.allocate(rows, dev)
        self.vout = ciar.VerifyOut.allocate(rows, wl.window, dev)
        self.ws = ciar.alloc_workspace(rows, wl.window, dev)

    def quantify(self):
        self.ciar.quantify(self.draft, self.params, self.qout, self.wl.valid_begin, self.wl.n_valid)

    def verify(self):
        self.ciar.verify(self.draft, self.target, self.tokens, self.qout.flag, self.qout.row_max, self.qout.sum_exp,
                         self.ua, self.ur, self.wl.window, self.ciar.VERIFY_ANCHORED, self.vout, self.ws,
                         self.wl.valid_begin, self.wl.n_valid)

    def __call__(self):
        self.quantify()
        self.verify()

    def traffic_model(self):
        """Rows the method has to touch in this batch: (sent rows, resampled rows, flagged fraction)."""
        f = self.vout.first_flag.cpu().numpy().astype(np.int64)
        a = self.vout.accepted_len.cpu().numpy().astype(np.int64)
        w = self.wl.window
        sent = int((w - f).sum())
        resampled = int((a < w).sum())
        flagged = float(self.qout.flag.float().mean().item())
        return sent, resampled, flagged


def timed_steps(ciar, step, K, warm, world, dev, roll_s=0.8):
    """`warm` untimed steps, then K timed steps with CUDA events around every kernel of every step.  nvidia-smi samples the
    clocks from before the first untimed step to after the last: the timed region is bracketed by about `roll_s` seconds
    of the same steps on either side, so that the samples are taken under this very load even when K steps take a few
    milliseconds.  Returns (total ms max over ranks, mean quantify ms, mean verify ms, clocks, launches in the timed region)."""
    sampler = ClockSampler(dev.index or 0)
    sampler.start()
    t0 = time.perf_counter()
    for _ in range(warm):
        step()
    torch.cuda.synchronize()
    s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    s.record(); step(); e.record(); torch.cuda.synchronize()
    est_ms = max(1e-3, s.elapsed_time(e))
    roll = int(min(20000, max(0, roll_s * 1e3 / est_ms)))

    def untimed(n):
        for i in range(n):
            step()
            if i % 256 == 255:
                torch.cuda.synchronize()  # keeps the launch queue short
        torch.cuda.synchronize()
    untimed(roll)
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(K)]
    launches0 = ciar.launch_count()
    barrier(world)
    t_start = torch.cuda.Event(enable_timing=True); t_end = torch.cuda.Event(enable_timing=True)
    t_start.record()
    for k in range(K):
        ev[k][0].record()
        step.quantify()
        ev[k][1].record()
        step.verify()
        ev[k][2].record()
    t_end.record()
    barrier(world)
    launches = ciar.launch_count() - launches0
    untimed(roll)
    clocks = sampler.stop()
    clocks["sampled_s"] = round(time.perf_counter() - t0, 2)
    total_ms = max_over_ranks(t_start.elapsed_time(t_end), world)
    q_ms = float(np.mean([ev[k][0].elapsed_time(ev[k][1]) for k in range(K)]))
    v_ms = float(np.mean([ev[k][1].elapsed_time(ev[k][2]) for k in range(K)]))
    clocks["time_x_mhz"] = None if clocks["sm_mhz"] is None else {"quantify": q_ms * clocks["sm_mhz"], "verify": v_ms * clocks["sm_mhz"]}
    return total_ms, q_ms, v_ms, clocks, launches


def config_of(name, wl, rows, radius):
    """The workload as both arms name it."""
    return {"workload": name, "rows_per_gpu": rows, "vocab": wl.vocab, "valid_codes": wl.n_valid, "logits": wl.dtype,
            "window": wl.window, "verify_mode": "anchored", "radius": radius, "tau": wl.tau,
            "l2": "inputs (%.0f MB) larger than L2; no flush" % (2 * rows * wl.n_valid * wl.elem_bytes / 1e6)}


def kernel_names(wl, per_code):
    wide = wl.n_valid > 16384  # rows that do not fit a stage take the chunked kernels
    q = "quantify_percode_kernel" if per_code else ("quantify_wide_kernel" if wide else "quantify_stream_kernel")
    return q, ("verify_plan+accept_wide+window" if wide else "verify_plan+accept+window")


def workload_report(wl, rows, per_code, q_ms, v_ms, ms_per_step, sent, resampled, peak):
    """Algorithmic bytes of one step and what they make of the measured times."""
    row_bytes = wl.n_valid * wl.elem_bytes
    q_bytes = rows * row_bytes * (2 if per_code else 1) + rows * 48  # a per-code radius row is as wide as its logit row
    v_bytes = sent * row_bytes + resampled * 2 * row_bytes + rows * 16 + (rows // wl.window) * 16
    q_name, v_name = kernel_names(wl, per_code)
    q_gbs, v_gbs = q_bytes / (q_ms * 1e-3) / 1e9, v_bytes / (v_ms * 1e-3) / 1e9
    return {q_name: {"ms": q_ms, "algorithmic_bytes": int(q_bytes), "GB/s": q_gbs, "frac": q_gbs / peak},
            v_name: {"ms": v_ms, "algorithmic_bytes": int(v_bytes), "GB/s": v_gbs, "frac": v_gbs / peak},
            "step_GB/s": (q_bytes + v_bytes) / (ms_per_step * 1e-3) / 1e9}


def side_workload(ciar, name, steps, dev, peak):
    """One of the other large-batch workloads, measured like the main one (device-resident, CUDA events, clocks sampled)."""
    wl = synth.WORKLOADS[name]
    inp = synth.make_inputs(wl, device=dev)
    step = Step(ciar, wl, inp, False)
    total_ms, q_ms, v_ms, clocks, _ = timed_steps(ciar, step, steps, 3, 1, dev, roll_s=0.6)
    sent, resampled, flagged = step.traffic_model()
    rep = workload_report(wl, step.rows, False, q_ms, v_ms, total_ms / steps, sent, resampled, peak)
    rep.update({"rows": step.rows, "valid_codes": wl.n_valid, "logits": wl.dtype, "window": wl.window, "steps": steps,
                "ms_per_step": total_ms / steps, "tokens/s": step.rows * steps / (total_ms * 1e-3),
                "cloud_flag_fraction": flagged, "sent_fraction": sent / step.rows,
                "clocks": {k: clocks[k] for k in ("sm_mhz", "sm_max_mhz", "reasons", "samples")},
                "l2": "inputs (%.0f MB) larger than L2; no flush" % (2 * step.rows * wl.n_valid * wl.elem_bytes / 1e6)})
    del step, inp
    torch.cuda.empty_cache()
    return rep


def run_ours(args):
    from paper_2603_25463_b200 import ciar
    rank, world, local = dist_setup(args.gpus)
    dev = torch.device("cuda", local if world > 1 else 0)
    wl = synth.WORKLOADS[args.workload]
    if args.images:
        wl = wl.scaled(images=args.images)  # a smaller batch of the same recipe (profiler captures)
    wl = ciar_dist.rank_workload(wl, rank)  # every rank draws its own batch (weak scaling)
    per_code = args.radius == "per_code"
    inp = synth.make_inputs(wl, device=dev, per_code_radius=per_code)
    step = Step(ciar, wl, inp, per_code)
    rows = step.rows
    row_bytes = wl.n_valid * wl.elem_bytes

    warm = max(3, args.warmup)
    total_ms, q_ms, v_ms, clocks, launches = timed_steps(ciar, step, args.steps, warm, world, dev)
    K = args.steps
    sent, resampled, flagged = step.traffic_model()
    ms_per_step = total_ms / K
    value = world * rows * K / (total_ms * 1e-3)

    # ---- end to end: inputs start in pinned host memory, results end in host memory
    e2e = None
    if not args.no_e2e:
        hd, ht = inp.draft.cpu().pin_memory(), inp.target.cpu().pin_memory()
        htok, hua, hur, hrad = (x.cpu().pin_memory() for x in (inp.tokens, inp.u_accept, inp.u_resample,
                                                               inp.radius_code if per_code else inp.radius_row))
        res_dev = [step.qout.flag, step.qout.score, step.vout.accept, step.vout.accepted_len, step.vout.resampled_token,
                   step.vout.first_flag]
        res_host = [torch.empty(t.shape, dtype=t.dtype).pin_memory() for t in res_dev]
        ins = [(step.draft, hd), (step.target, ht), (step.tokens, htok), (step.ua, hua), (step.ur, hur),
               (step.params.radius, hrad)]
        h2d = sum(h.numel() * h.element_size() for _, h in ins)
        d2h = sum(h.numel() * h.element_size() for h in res_host)

        def e2e_step():
            for d, h in ins:
                d.copy_(h, non_blocking=True)
            step()
            for d, h in zip(res_dev, res_host):
                h.copy_(d, non_blocking=True)
        Ke = max(3, min(K, args.e2e_steps))
        for _ in range(3):
            e2e_step()
        barrier(world)
        s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s.record()
        for _ in range(Ke):
            e2e_step()
        e.record()
        barrier(world)
        e_ms = max_over_ranks(s.elapsed_time(e), world)
        e2e = {"value": world * rows * Ke / (e_ms * 1e-3), "unit": "tokens/s", "h2d_bytes_per_step": int(h2d),
               "d2h_bytes_per_step": int(d2h), "steps": Ke, "ms_per_step": e_ms / Ke}

    if rank != 0:
        return
    peak, peak_kind = measured_peak()
    kernels = workload_report(wl, rows, per_code, q_ms, v_ms, ms_per_step, sent, resampled, peak)
    q_name, v_name = kernel_names(wl, per_code)
    dominant = q_name if q_ms >= v_ms else v_name
    dom_gbs = kernels[dominant]["GB/s"]
    traffic = None if args.images else load_traffic(dominant, args.workload)  # the captures are of full batches
    roofline = {"bound": "hbm", "kernel": dominant, "achieved": dom_gbs, "peak": peak, "unit": "GB/s",
                "frac": dom_gbs / peak, "peak_kind": "of " + peak_kind, "traffic": traffic,
                "frac_of_nominal_8TBs": dom_gbs / NOMINAL_HBM_GBS,
                "kernels": {q_name: kernels[q_name], v_name: kernels[v_name]}, "step_GB/s": kernels["step_GB/s"]}
    # the other large-batch workloads, each with its own kernel times, bytes and fractions (single GPU, default run)
    per_workload = None
    if world == 1 and args.side_workloads and not args.images and args.workload == "llamagen384" and not per_code:
        del step, inp
        torch.cuda.empty_cache()
        per_workload = {}
        for name, steps in (("anole", 200), ("largevocab", 5)):
            try:
                per_workload[name] = side_workload(ciar, name, steps, dev, peak)
            except torch.cuda.OutOfMemoryError as e:
                per_workload[name] = {"skipped": "not enough free device memory: %s" % str(e)[:80]}
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        cpu = cpu_oracle_baseline(synth.WORKLOADS[args.workload], sample_rows=args.cpu_rows)
    line = {
        "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": K, "warmup": max(3, args.warmup),
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": config_of(args.workload, wl, rows, args.radius),
        "clocks": clocks,
        "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline, "cpu_baseline": cpu,
        "cloud_flag_fraction": flagged, "sent_fraction": sent / rows, "resampled_windows": resampled,
        "per_workload": per_workload,
    }
    print(json.dumps(line))


# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) from the ncu captures summarised under
# profiles/, keyed by (kernel, workload).  An entry is dropped (-> null) when its kernel changes after the capture.
NCU_TRAFFIC = {
    # captured on 2304 of the 9216 rows and scaled by the rows: profiles/quantify_percode_kernel_llamagen384.md
    ("quantify_percode_kernel", "llamagen384"): 4 * (151.1e6 + 4.7e6),
    ("quantify_stream_kernel", "llamagen384"): 302.1e6 + 4.4e6,  # profiles/quantify_stream_kernel_llamagen384.md
    # captured on 2048 of the 65536 rows and scaled by the rows (every row is handled alone): profiles/quantify_wide_kernel_largevocab.md
    ("quantify_wide_kernel", "largevocab"): 32 * (1078.5e6 + 15.1e6),
}


def load_traffic(kernel, workload):
    return NCU_TRAFFIC.get((kernel, workload))


def cpu_oracle_baseline(wl, sample_rows, threads=0):
    """The CPU oracle, as it stands, timed on a bounded sample of the same workload (whole images)."""
    import oracle
    inp = synth.make_inputs(wl, device="cpu", row_limit=sample_rows)
    rows = inp.draft.shape[0]
    prm = oracle.IntervalParams(radius_mode=oracle.RADIUS_PER_ROW, radius=inp.radius_row, tau=wl.tau)
    oracle.quantify(inp.draft[:wl.window], prm, wl.valid_begin, wl.n_valid)  # load the library
    t0 = time.perf_counter()
    q = oracle.quantify(inp.draft, prm, wl.valid_begin, wl.n_valid, threads=threads)
    oracle.verify(inp.draft, inp.target, inp.tokens, q.flag, inp.u_accept, inp.u_resample, wl.window,
                  oracle.VERIFY_ANCHORED, wl.valid_begin, wl.n_valid, threads=threads)
    dt = time.perf_counter() - t0
    cores = threads or oracle.max_threads()
    return {"value": rows / dt, "unit": "tokens/s", "cores": cores, "kind": "oracle",
            "sample": "first %d rows of %s (quantify + verify), %.2f s wall" % (rows, wl.name, dt)}


def run_decode(args):
    """Serving decode loop (--workload decode): `requests` concurrent requests, each generating
    seq_len tokens in draft windows; one step = ciar_decode_step for every unfinished request.
    Reports the whole loop's tokens/s and the per-step device latency (CUDA events around each step)."""
    from paper_2603_25463_b200 import ciar
    rank, world, local = dist_setup(args.gpus)
    dev = torch.device("cuda", local if world > 1 else 0)
    wl = ciar_dist.rank_workload(synth.WORKLOADS["decode"], rank)
    if args.decode_requests:
        wl = wl.scaled(images=args.decode_requests)
    per_code = args.radius == "per_code"
    inp = synth.make_inputs(wl, device=dev, per_code_radius=per_code)
    req, seq = wl.images, wl.tokens_per_image
    if per_code:  # a pool of raw per-code radii indexed like the logit pools
        params = ciar.IntervalParams(radius_mode=ciar.RADIUS_PER_CODE, radius=inp.radius_code, radius_is_raw=True, tau=wl.tau)
    else:
        params = ciar.IntervalParams(radius_mode=ciar.RADIUS_PER_ROW, radius=inp.radius_row, tau=wl.tau)
    state = ciar.DecodeState.allocate(req, seq, dev)
    ws = ciar.alloc_workspace(req * wl.window, wl.window, dev)

    def one_step():
        ciar.decode_step(state, inp.draft, inp.target, inp.tokens, inp.u_accept, inp.u_resample, params, wl.window,
                         ciar.VERIFY_ANCHORED, ws, wl.valid_begin, wl.n_valid)

    graph = None
    launches_per_step = None

    def loop(record):
        ciar.decode_init(state, 0)
        events = []
        steps = 0
        while True:
            if record:
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
            if graph is not None:
                graph.replay()  # the step's launches, recorded once (every argument lives on the device)
            else:
                one_step()
            if record:
                e1.record()
                events.append((e0, e1))
            steps += 1
            if steps % 16 == 0 and int(state.counters[7].item()) >= req:  # every request has finished
                break
            if steps > 4 * seq:
                raise RuntimeError("decode loop did not finish")
        return steps, events

    loop(False)  # warm-up: one whole generation
    torch.cuda.synchronize()
    if args.decode_graph:
        # ciar_decode_step allocates nothing and never synchronises, so a caller may record it in a CUDA graph
        n0 = ciar.launch_count()
        side = torch.cuda.Stream(device=dev)
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            one_step()
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        launches_per_step = ciar.launch_count() - n0
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            one_step()
        loop(False)  # warm-up of the replays
        torch.cuda.synchronize()
    sampler = ClockSampler(dev.index or 0)
    sampler.start()
    # whole untimed generations on either side of the timed one, so that the clock samples are taken under this load
    w0 = time.perf_counter()
    loop(False)
    torch.cuda.synchronize()
    n_roll = int(min(200, max(1, 0.8 / max(1e-3, time.perf_counter() - w0))))
    for _ in range(n_roll):
        loop(False)
    torch.cuda.synchronize()
    launches0 = ciar.launch_count()
    barrier(world)
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    steps, events = loop(True)
    t1.record()
    barrier(world)
    launches_timed = ciar.launch_count() - launches0
    for _ in range(n_roll):
        loop(False)
    torch.cuda.synchronize()
    clocks = sampler.stop()
    launches = launches_timed
    if graph is not None:
        launches = steps * launches_per_step  # replays do not pass through the library's counter
    total_ms = max_over_ranks(t0.elapsed_time(t1), world)
    cnt = state.counters.cpu().numpy()
    # steps after the last request finished do no work but are inside the timed region: count only useful ones
    lat = np.array([a.elapsed_time(b) for a, b in events]) * 1e3
    useful = int(np.ceil(cnt[0] / req)) if req else 0
    if rank != 0:
        return
    print(json.dumps({
        "metric": METRIC, "value": world * req * seq / (total_ms * 1e-3), "unit": "tokens/s", "n_gpus": world,
        "steps": steps, "warmup": 1, "ms_per_step": total_ms / steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": "decode", "requests_per_gpu": req, "seq_len": seq, "vocab": wl.vocab, "logits": wl.dtype,
                   "window": wl.window, "verify_mode": "anchored", "radius": args.radius, "tau": wl.tau,
                   "launch": "cuda graph replay" if graph is not None else "direct",
                   "l2": "pools of %.1f GB, rows touched once" % ((3 if per_code else 2) * req * seq * wl.vocab * wl.elem_bytes / 1e9)},
        "clocks": clocks,
        "gpu_launches": int(launches),
        "step_latency_us": {"p50": float(np.percentile(lat, 50)), "p99": float(np.percentile(lat, 99)),
                            "max": float(lat.max()), "timed_with": "CUDA events around every ciar_decode_step"},
        "decode": {"windows": int(cnt[0]), "cloud_call_windows": int(cnt[1]), "rows_sent": int(cnt[2]),
                   "rows_flagged": int(cnt[3]), "draft_tokens_kept": int(cnt[4]), "resampled": int(cnt[5]),
                   "rows_quantified": int(cnt[6]), "useful_steps": useful},
    }))


def run_reference(args):
    """The base contract's reference arm: here the CPU oracle on host cores (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import oracle
    wl = synth.WORKLOADS[args.workload]
    steps = max(1, min(args.steps, 20))
    warm = max(3, min(args.warmup, 5))
    inp = synth.make_inputs(wl, device="cpu", row_limit=args.cpu_rows)
    rows = inp.draft.shape[0]
    prm = oracle.IntervalParams(radius_mode=oracle.RADIUS_PER_ROW, radius=inp.radius_row, tau=wl.tau)

    def one():
        q = oracle.quantify(inp.draft, prm, wl.valid_begin, wl.n_valid)
        oracle.verify(inp.draft, inp.target, inp.tokens, q.flag, inp.u_accept, inp.u_resample, wl.window,
                      oracle.VERIFY_ANCHORED, wl.valid_begin, wl.n_valid)
    for _ in range(warm):
        one()
    t0 = time.perf_counter()
    for _ in range(steps):
        one()
    dt = time.perf_counter() - t0
    value = rows * steps / dt
    cores = oracle.max_threads()
    sample = "each step = first %d rows of %s through the CPU oracle (quantify + verify)" % (rows, wl.name)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": args.gpus, "steps": steps,
        "warmup": warm, "ms_per_step": dt / steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_of(args.workload, wl, rows, "per_row"),
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llamagen384", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--e2e-steps", type=int, default=20)
    ap.add_argument("--cpu-rows", type=int, default=9216, help="rows of the CPU oracle's bounded sample")
    ap.add_argument("--decode-requests", type=int, default=0, help="decode workload: concurrent requests (default 256)")
    ap.add_argument("--images", type=int, default=0,
                    help="images of the workload (default: the workload's own); a smaller batch for profiler captures")
    ap.add_argument("--decode-graph", action=argparse.BooleanOptionalAction, default=True,
                    help="decode workload: replay each step from a CUDA graph (default) or launch it directly")
    ap.add_argument("--radius", default="per_row", choices=["per_row", "per_code"],
                    help="interval radius: one per row (default) or one raw value per code, a tensor as large as the logits")
    ap.add_argument("--side-workloads", action=argparse.BooleanOptionalAction, default=True,
                    help="default run on one GPU: also measure the anole and largevocab workloads (per_workload block)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the CIAR path has no CPU fallback "
                         "(use --impl reference for the CPU oracle)")
    if args.workload == "decode":
        run_decode(args)
    else:
        run_ours(args)
    if int(os.environ.get("WORLD_SIZE", "1")) > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
