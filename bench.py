#!/usr/bin/env python
"""Benchmark of batched plan evaluation: one step = one pe_eval_batch over a resident batch.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

Prints ONE JSON line (rank 0).  `value` is operator-evaluations per second (candidates x
operators / time) over all GPUs, with `plans_per_s` beside it; `roofline` rates the evaluation
kernel against the HBM copy peak on the bytes the method must move; `e2e` is the same metric
through the host-buffer entry point, copies included; `cpu_baseline` is the CPU oracle on a
bounded sample of the same workload.
"""
import argparse
import hashlib
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2503_09357_b200 import workloads as wl  # noqa: E402

WORKLOADS = {
    "tiny_pipeline": lambda: wl.make_config(1),
    "bidirectional_pipeline": lambda: wl.make_config(2),
    "moe_branchy": lambda: wl.make_config(3),
    "multimodal_mimo": lambda: wl.make_config(4),
}
for _V, _D in wl.SWEEP_POINTS:
    WORKLOADS[f"random_layered_V{_V}_D{_D}"] = (lambda V=_V, D=_D: wl.make_config(5, V=V, D=D))
DEFAULT_WORKLOAD = "random_layered_V16384_D64"   # the largest configuration: sweep point V=16384, D=64, K=65536

FALLBACK_HBM_GBS = 6650.0
# the kernel each variant runs for graphs that have a compact encoding (all benchmark workloads do)
KERNEL_OF_VARIANT = {"shared": "pe_eval_lane_kernel<STATE_SMEM=true>", "global": "pe_eval_lane_kernel<STATE_SMEM=false>",
                     "warp": "pe_eval_warp2_kernel", "team": "pe_eval_team_kernel"}

# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) per operator-evaluation of the evaluation kernel
# from an ncu capture, keyed by kernel variant, valid only while the sources that kernel is built from hash to
# the value recorded with it.  Reported as null when those sources have changed since the capture.
KERNEL_SOURCES = {
    "team": ("pe_kernel_team.cuh", "pe_team.cu", "pe_team_launch.h", "pe_transpose.cuh"),
    "warp": ("pe_kernel_warp2.cuh", "pe_warp2_launch.h", "pe_device.cuh", "pe_kernel_lane.cuh"),
    "global": ("pe_kernel_lane.cuh", "pe_lane_launch.h", "pe_device.cuh"),
    "shared": ("pe_kernel_lane.cuh", "pe_lane_launch.h", "pe_device.cuh"),
}
NCU_TRAFFIC = {
    # variant: (hash of its sources at capture time, DRAM bytes per operator-evaluation, captured workload)
    "team": ("698c9fc757a7e542", 10.13, "random_layered_V16384_D64 at K = 3552 (one chunk), scaled by operator-evaluations; "
                        "the staging transpositions around the kernel move another 22 B per operator-evaluation"),
}


def kernel_source_hash(variant):
    """Hash of the sources the kernel of `variant` is built from."""
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2503_09357_b200", "csrc")
    for name in KERNEL_SOURCES.get(variant, ()):
        with open(os.path.join(csrc, name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def compulsory_bytes(V, D, K, order_bytes, want_times=True):
    """Bytes the method must move per launch: machine id + order entry (+ start + finish) per
    operator-evaluation, makespan + status + busy[D] + peak[D] per candidate."""
    per_op = 1 + order_bytes + (8 if want_times else 0)
    return K * V * per_op + K * (8 + 8 * D)


class ClockSampler:
    """nvidia-smi clock/throttle samples every 100 ms; `stop(t0, t1)` keeps those taken inside the
    wall-clock window of the timed region (or the nearest ones when the region is shorter than a period)."""
    QUERY = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.proc = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(gpu_index)], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
        except OSError:
            pass

    def stop(self, t0, t1):
        import datetime
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            text, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            text, _ = self.proc.communicate()
        rows = []
        for line in text.splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                ts = datetime.datetime.strptime(f[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                rows.append((ts, float(f[1]), float(f[2]), float(f[3]), [v.lower().startswith("active") for v in f[5:9]]))
            except ValueError:
                continue
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        inside = [r for r in rows if t0 <= r[0] <= t1]
        if not inside:                                    # region shorter than a sampling period: nearest sample
            inside = [min(rows, key=lambda r: abs(r[0] - 0.5 * (t0 + t1)))]
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        reasons = sorted({n for r in inside for n, on in zip(names, r[4]) if on})
        return {"sm_mhz": statistics.median(r[1] for r in inside), "sm_max_mhz": max(r[2] for r in inside),
                "power_w_max": max(r[3] for r in inside), "samples": len(inside), "reasons": reasons}


def time_oracle(w, assign, order, target_s, threads):
    """Oracle (as it stands) on a bounded sample of the workload's candidates: the first n, with n
    grown until one run takes about target_s of wall time (or the whole batch is used)."""
    from oracle import pe_oracle as orc
    V, K = order.shape
    n = min(K, max(threads * 4, 64))
    while True:
        a = np.ascontiguousarray(assign[:, :n]); o = np.ascontiguousarray(order[:, :n])
        t0 = time.perf_counter()
        ref = orc.evaluate(w, a, o, threads=threads)
        dt = max(time.perf_counter() - t0, 1e-6)
        if n >= K or dt >= 0.4 * target_s:
            return n, dt, ref
        n = int(min(K, max(2 * n, n * min(16.0, 0.8 * target_s / dt))))


def compare_with_oracle(gpu, ref, n):
    """Element-by-element comparison of the timed run's outputs (first n candidates) with the oracle's:
    every array of every valid candidate, the two validity bits of the others."""
    invalid_bits = 3
    gst = gpu["status"][:n].view(np.uint32)
    rst = ref["status"]
    bad = (rst & invalid_bits) != 0
    mism = int(np.count_nonzero((gst & invalid_bits) != (rst & invalid_bits)))
    ok = ~bad
    mism += int(np.count_nonzero(gst[ok] != rst[ok]))
    arrays = 1
    for key in ("makespan", "busy", "peak_mem", "start", "finish"):
        if key not in gpu or ref.get(key) is None:
            continue
        a = gpu[key][..., :n]
        mism += int(np.count_nonzero(a[..., ok] != ref[key][..., ok]))
        arrays += 1
    return {"candidates": int(n), "arrays": arrays, "mismatches": mism, "against": "oracle, element by element"}


def run_reference(args):
    """--impl reference: the CPU oracle on the host cores, each step a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = WORKLOADS[args.workload]()
    V, D = w.num_ops, w.num_devices
    threads = os.cpu_count() or 1
    budget_s = 90.0                                          # whole run, warm-up included
    per_step = budget_s / (args.steps + args.warmup)
    K_gen = int(min(w.num_candidates, 8192))
    assign, order = wl.make_candidates(w, K=K_gen)
    n, dt, _ = time_oracle(w, assign, order, min(per_step, 10.0) * 0.8, threads)   # sizes the per-step sample
    if n > K_gen:
        n = K_gen
    from oracle import pe_oracle as orc
    a = np.ascontiguousarray(assign[:, :n]); o = np.ascontiguousarray(order[:, :n])
    for _ in range(args.warmup):
        orc.evaluate(w, a, o, threads=threads)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        orc.evaluate(w, a, o, threads=threads)
    dt = time.perf_counter() - t0
    value = n * V * args.steps / dt
    line = {
        "impl": "reference", "metric": "op_evals_per_s", "value": value, "unit": "op-evals/s",
        "plans_per_s": value / V, "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "int32", "data": "synthetic",
        "config": {"workload": args.workload, "V": V, "E": w.num_edges, "D": D, "L": w.num_link_classes,
                   "K_per_gpu": w.num_candidates, "outputs": "full", "order_bytes": 2 if V <= 65536 else 4,
                   "sample": f"the oracle evaluates {n} of the {w.num_candidates} candidates per step"},
        "cpu_baseline": {"value": value, "unit": "op-evals/s", "cores": threads, "kind": "oracle",
                         "sample": f"{n} of {w.num_candidates} candidates per step, {args.steps} steps"},
        "e2e": {"value": value, "unit": "op-evals/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def time_decode(pe, name, dev, local_rank, stream, op_budget, steps=5):
    """pe_decode_priority on uniformly random priority lists of one workload (made on the device: argsort of
    random numbers per candidate), K * V about `op_budget`; mean of `steps` timed calls after two warm-ups."""
    import torch
    ow = WORKLOADS[name]()
    oV = ow.num_ops
    oK = int(min(ow.num_candidates, max(1024, op_budget // oV)))
    og = pe.Graph(ow, device=local_rank)
    gen = torch.Generator(device=dev); gen.manual_seed(oV)
    plist = torch.argsort(torch.rand((oV, oK), device=dev, generator=gen), dim=0).to(torch.int16).contiguous()
    for _ in range(2):
        og.decode_priority(plist)
    torch.cuda.synchronize(dev)
    times = []
    for _ in range(steps):
        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
        e0.record(stream); dorder, dstatus = og.decode_priority(plist); e1.record(stream)
        torch.cuda.synchronize(dev)
        times.append(e0.elapsed_time(e1))
    ms = statistics.mean(times)
    assert int(dstatus.abs().max()) == 0
    dalg = oK * oV * 4 + oK * 4                    # list in, order out, status
    rec = {"workload": name, "V": oV, "K": oK, "kernel_variant": pe.VARIANT_NAMES[pe.pe_decode_variant(og.handle, oK, 0)],
           "ms": ms, "op_decodes_per_s": oK * oV / (ms * 1e-3), "gbs": dalg / (ms * 1e-3) / 1e9}
    og.close()
    return rec


def time_exclusive(pe, name, dev, local_rank, stream, op_budget, want_times, steps=5):
    """pe_eval_batch with PE_COMM_EXCLUSIVE (one transfer per channel at a time) on the first K candidates of a
    workload, K * V about `op_budget`; same compulsory bytes as the plain evaluation."""
    import torch
    ow = WORKLOADS[name]()
    oV, oD = ow.num_ops, ow.num_devices
    oK = int(min(ow.num_candidates, max(1024, op_budget // oV)))
    oa, oo = wl.make_candidates(ow, K=oK)
    og = pe.Graph(ow, device=local_rank)
    flags = pe.PE_COMM_EXCLUSIVE
    da = torch.from_numpy(oa).to(dev); do = torch.from_numpy(oo.view(np.int16)).to(dev)
    oout = og.alloc_outputs(oK, want_times)
    ows = og.alloc_workspace(oK, flags)
    for _ in range(2):
        og.eval_batch(da, do, flags=flags, out=oout, workspace=ows)
    torch.cuda.synchronize(dev)
    times = []
    for _ in range(steps):
        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
        e0.record(stream); og.eval_batch(da, do, flags=flags, out=oout, workspace=ows); e1.record(stream)
        torch.cuda.synchronize(dev)
        times.append(e0.elapsed_time(e1))
    ms = statistics.mean(times)
    rec = {"workload": name, "V": oV, "D": oD, "K": oK, "kernel_variant": og.variant(oK, flags), "ms": ms,
           "op_evals_per_s": oK * oV / (ms * 1e-3), "gbs": compulsory_bytes(oV, oD, oK, 2, want_times) / (ms * 1e-3) / 1e9}
    og.close()
    return rec


def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2503_09357_b200 import binding as pe
    from paper_2503_09357_b200.sharding import max_over_ranks, weak_scaling_first

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()

    w = WORKLOADS[args.workload]()
    V, D, K = w.num_ops, w.num_devices, (args.candidates or w.num_candidates)
    want_times = args.outputs == "full"
    flags = {"auto": pe.PE_VARIANT_AUTO, "global": pe.PE_VARIANT_GLOBAL, "shared": pe.PE_VARIANT_SHARED,
             "warp": pe.PE_VARIANT_WARP, "team": pe.PE_VARIANT_TEAM}[args.variant]
    obytes = 2 if V <= 65536 else 4
    odt = torch.int16 if obytes == 2 else torch.int32

    # inputs in pinned host memory (weak scaling: every rank draws its own K candidates)
    t_gen = time.perf_counter()
    h_assign = torch.empty((V, K), dtype=torch.uint8).pin_memory()
    h_order = torch.empty((V, K), dtype=odt).pin_memory()
    wl.make_candidates(w, K=K, first=weak_scaling_first(K, rank), out_assign=h_assign.numpy(),
                       out_order=h_order.numpy().view(np.uint16 if obytes == 2 else np.uint32))
    t_gen = time.perf_counter() - t_gen

    g = pe.Graph(w, device=local_rank)
    variant = g.variant(K, flags)
    d_assign = h_assign.to(dev, non_blocking=True)
    d_order = h_order.to(dev, non_blocking=True)
    d_out = g.alloc_outputs(K, want_times)
    ws, ws_bytes = g.alloc_workspace(K, flags)
    outs = pe.make_outputs(**{k: v.data_ptr() for k, v in d_out.items()})
    stream = torch.cuda.current_stream(dev)

    def step():
        rc = pe.pe_eval_batch(g.handle, K, d_assign.data_ptr(), d_order.data_ptr(), obytes, flags, outs,
                              ws.data_ptr(), ws_bytes, stream.cuda_stream)
        if rc != pe.PE_OK:
            raise pe.PeError(rc, "pe_eval_batch")

    sampler = ClockSampler(local_rank) if rank == 0 else None
    torch.cuda.synchronize(dev)
    t_w = time.perf_counter()
    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize(dev)
    t_w = (time.perf_counter() - t_w) / args.warmup
    if args.steps <= 0:                                     # default: about two seconds of timed work
        args.steps = int(min(2000, max(10, 2.0 / max(t_w, 1e-5))))
        if world > 1:
            st = torch.tensor([args.steps], dtype=torch.int64, device=dev)
            dist.all_reduce(st, op=dist.ReduceOp.MAX)
            args.steps = int(st.item())

    # ---- timed region: device resident, CUDA events on the launching stream ----
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    launches0 = pe.pe_kernel_launches()
    barrier(); torch.cuda.synchronize(dev)
    t_first = torch.cuda.Event(enable_timing=True); t_last = torch.cuda.Event(enable_timing=True)
    wall0 = time.time()
    t_first.record(stream)
    for a, b in ev:
        a.record(stream); step(); b.record(stream)
    t_last.record(stream)
    torch.cuda.synchronize(dev)
    wall1 = time.time()
    barrier()
    launches = pe.pe_kernel_launches() - launches0
    clocks = sampler.stop(wall0, wall1) if sampler else None
    total_ms = t_first.elapsed_time(t_last)
    kernel_ms = [a.elapsed_time(b) for a, b in ev]
    if pe.pe_graph_poll_error(g.handle, stream.cuda_stream) != pe.PE_OK:
        raise SystemExit("device-side error word set during the timed region")
    total_ms = max_over_ranks(total_ms, dev)
    ms_per_step = total_ms / args.steps
    # outputs of the last timed step, kept for the comparison with the oracle below
    timed_out = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        timed_out = {k: v.cpu().numpy() for k, v in d_out.items()}
    value = world * K * V / (ms_per_step * 1e-3)

    # ---- end to end: host buffers through pe_eval_batch_host, copies inside the timed region ----
    h_out = {k: torch.empty(v.shape, dtype=v.dtype).pin_memory() for k, v in d_out.items()}
    houts = pe.make_outputs(**{k: v.data_ptr() for k, v in h_out.items()})

    def e2e_step():
        rc = pe.pe_eval_batch_host(g.handle, K, h_assign.data_ptr(), h_order.data_ptr(), obytes, flags, houts,
                                   d_assign.data_ptr(), d_order.data_ptr(), outs, ws.data_ptr(), ws_bytes,
                                   stream.cuda_stream)
        if rc != pe.PE_OK:
            raise pe.PeError(rc, "pe_eval_batch_host")

    e2e_steps = max(1, min(args.steps, args.e2e_steps))
    e2e_step()
    barrier(); torch.cuda.synchronize(dev)
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        e2e_step()
    torch.cuda.synchronize(dev)
    e2e_s = time.perf_counter() - t0
    e2e_value = world * K * V * e2e_steps / max_over_ranks(e2e_s, dev)
    h2d = V * K * (1 + obytes)
    d2h = sum(v.numel() * v.element_size() for v in d_out.values())
    # the same call when a search loop only wants the summary outputs back (makespan, busy, peak, status)
    e2e_summary = None
    if want_times:
        souts = pe.make_outputs(**{k: v.data_ptr() for k, v in h_out.items() if k not in ("start", "finish")})

        def e2e_summary_step():
            rc = pe.pe_eval_batch_host(g.handle, K, h_assign.data_ptr(), h_order.data_ptr(), obytes, flags, souts,
                                       d_assign.data_ptr(), d_order.data_ptr(), outs, ws.data_ptr(), ws_bytes,
                                       stream.cuda_stream)
            if rc != pe.PE_OK:
                raise pe.PeError(rc, "pe_eval_batch_host")

        e2e_summary_step()
        barrier(); torch.cuda.synchronize(dev)
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            e2e_summary_step()
        torch.cuda.synchronize(dev)
        es = time.perf_counter() - t0
        e2e_summary = {"value": world * K * V * e2e_steps / max_over_ranks(es, dev), "unit": "op-evals/s",
                       "outputs": "summary", "h2d_bytes_per_step": h2d,
                       "d2h_bytes_per_step": sum(v.numel() * v.element_size() for k, v in d_out.items()
                                                 if k not in ("start", "finish")), "steps": e2e_steps}

    others = None
    decode = []
    exclusive = []
    if rank == 0 and world == 1 and args.all_workloads:
        # free the headline's buffers, then time every other configuration (device-resident, fewer steps)
        del d_assign, d_order, d_out, ws, h_out, houts, outs
        torch.cuda.empty_cache()
        others = []
        for name in sorted(WORKLOADS):
            if name == args.workload:
                continue
            ow = WORKLOADS[name]()
            oK = ow.num_candidates
            oa, oo = wl.make_candidates(ow, K=oK)
            og = pe.Graph(ow, device=local_rank)
            da = torch.from_numpy(oa).to(dev); do = torch.from_numpy(oo.view(np.int16)).to(dev)
            oout = og.alloc_outputs(oK, want_times)
            ows = og.alloc_workspace(oK, flags)
            for _ in range(3):
                og.eval_batch(da, do, flags=flags, out=oout, workspace=ows)
            torch.cuda.synchronize(dev)
            times = []
            for _ in range(5):
                e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
                e0.record(stream); og.eval_batch(da, do, flags=flags, out=oout, workspace=ows); e1.record(stream)
                torch.cuda.synchronize(dev)
                times.append(e0.elapsed_time(e1))
            ms = statistics.mean(times)
            oalg = compulsory_bytes(ow.num_ops, ow.num_devices, oK, 2, want_times)
            others.append({"workload": name, "V": ow.num_ops, "D": ow.num_devices, "K": oK,
                           "kernel_variant": og.variant(oK, flags), "ms": ms,
                           "op_evals_per_s": oK * ow.num_ops / (ms * 1e-3),
                           "gbs": oalg / (ms * 1e-3) / 1e9})
            og.close()
            del da, do, oout, ows
            torch.cuda.empty_cache()
        # the step in front of the path: priority-list decoding, K * V = 2^28 per workload
        for name in sorted(WORKLOADS):
            if name.endswith("_D64") or name == "tiny_pipeline":
                continue                                  # decoding does not depend on the machines
            decode.append(time_decode(pe, name, dev, local_rank, stream, 1 << 28))
        # the model variant with exclusive channels (Eqs. 14-15), K * V = 2^26 per workload
        for name in ("bidirectional_pipeline", "multimodal_mimo", "random_layered_V256_D8", "random_layered_V4096_D64"):
            exclusive.append(time_exclusive(pe, name, dev, local_rank, stream, 1 << 26, want_times))

    if rank == 0:
        peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
        if os.path.exists(peaks_path):
            peak, peak_src = float(json.load(open(peaks_path))["hbm_gbs"]), "measured"
        else:
            peak, peak_src = FALLBACK_HBM_GBS, "fallback"
        kms = statistics.mean(kernel_ms)
        alg = compulsory_bytes(V, D, K, obytes, want_times)
        achieved = alg / (kms * 1e-3) / 1e9
        traffic = None
        rec = NCU_TRAFFIC.get(variant)
        if rec and rec[0] == kernel_source_hash(variant):
            traffic = rec[1] * K * V
        cpu = None
        parity = None
        if world == 1 and not args.no_cpu_baseline:
            threads = os.cpu_count() or 1
            n, dt, ref = time_oracle(w, h_assign.numpy(), h_order.numpy().view(np.uint16 if obytes == 2 else np.uint32),
                                     args.cpu_seconds, threads)
            cpu = {"value": n * V / dt, "unit": "op-evals/s", "cores": threads, "kind": "oracle",
                   "sample": f"first {n} of {K} candidates, all outputs, {dt:.1f} s"}
            parity = compare_with_oracle(timed_out, ref, n)
        line = {
            "metric": "op_evals_per_s", "value": value, "unit": "op-evals/s", "plans_per_s": value / V,
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int32", "data": "synthetic",
            "config": {"workload": args.workload, "V": V, "E": w.num_edges, "D": D, "L": w.num_link_classes,
                       "K_per_gpu": K, "outputs": args.outputs, "order_bytes": obytes, "kernel_variant": variant,
                       "l2": "inputs and outputs larger than L2" if alg > 252e6 else "working set below 2x L2: not flushed",
                       "candidate_generation_s": round(t_gen, 1)},
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "traffic": traffic, "peak_source": f"of {peak_src}", "kernel": KERNEL_OF_VARIANT[variant],
                         "kernel_ms": kms, "algorithmic_bytes_per_launch": alg},
            "e2e": {"value": e2e_value, "unit": "op-evals/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "steps": e2e_steps},
            "e2e_summary_outputs": e2e_summary,
            "gpu_launches": launches, "clocks": clocks, "cpu_baseline": cpu, "parity": parity,
        }
        if others is not None:
            for o in others:
                o["frac"] = o["gbs"] / peak
            line["other_workloads"] = others
            for o in decode:
                o["frac"] = o["gbs"] / peak
            line["decode"] = decode
            for o in exclusive:
                o["frac"] = o["gbs"] / peak
            line["exclusive_channels"] = exclusive
        print(json.dumps(line), flush=True)
        if parity is not None and parity["mismatches"] != 0:
            raise SystemExit(f"the timed run's outputs differ from the oracle: {parity}")
    g.close()
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=0, help="timed steps (default: enough for about 2 s)")
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", choices=sorted(WORKLOADS), default=DEFAULT_WORKLOAD)
    ap.add_argument("--outputs", choices=["full", "summary"], default="full")
    ap.add_argument("--variant", choices=["auto", "global", "shared", "warp", "team"], default="auto",
                    help="force a kernel variant (default: the library chooses)")
    ap.add_argument("--candidates", type=int, default=0, help="override K per GPU (default: the configuration's K)")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--headline-only", dest="all_workloads", action="store_false",
                    help="skip the device-resident timing of every other configuration (other_workloads); "
                         "it runs by default on 1 GPU and adds about a minute")
    ap.add_argument("--all-workloads", dest="all_workloads", action="store_true", help=argparse.SUPPRESS)
    ap.add_argument("--decode-only", action="store_true",
                    help="time pe_decode_priority alone on --workload (K * V = 2^26) and print its record")
    ap.set_defaults(all_workloads=True)
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.decode_only:
        import torch
        from paper_2503_09357_b200 import binding as pe
        torch.cuda.set_device(0)
        print(json.dumps(time_decode(pe, args.workload, torch.device("cuda", 0), 0, torch.cuda.current_stream(), 1 << 26)),
              flush=True)
        return
    if args.impl == "reference":
        args.steps = args.steps if args.steps > 0 else 5
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
