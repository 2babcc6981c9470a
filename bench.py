#!/usr/bin/env python
"""Benchmark of the DVP hot path: pruned log-prob forward+backward tokens/s.

A step is one pass of the whole hot path over one synthetic batch: one
``dvp_forward`` call that reads the training and inference logits and writes
the gradient (Def. 5.1, Def. 5.2, Prop. 5.4) for every token of the batch.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--rho R]
  python bench.py --impl reference ...     # the fp64 CPU checker on host cores

With N > 1 every rank (one per GPU) processes its own batch of the same shape:
rows are independent, so there is no data-path collective, only the barrier and
the max-over-ranks of the device time.  Started without a launcher, ``--gpus N``
starts the N ranks itself through ``torch.distributed.run`` on 127.0.0.1.
Rank 0 prints one JSON line.  At N = 1 the default run appends, after the
headline workload has freed its batch, one sub-object per other configuration
(``c1_bf16_fwd``, ``c3_f32_heavy``, ``c4_fused_lmhead``), each timed the same way.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "pruned_logprob_fwd_bwd_tokens_per_s"
UNIT = "tokens/s"
FALLBACK_HBM_GBS = 6650.0

# DRAM bytes per launch of the row kernel (dram__bytes_read.sum + dram__bytes_write.sum
# from one ncu capture of `bench.py --rows T ...`), keyed by (workload, rho); valid only for
# the kernel sources whose digest is recorded with it, scaled by rows to the full batch.
NCU_TRAFFIC = {
    ("c2_bf16_fwdbwd", 1e-4): {"digest": "47f036696d37ae2e", "T": 2048, "bytes": 1.663986e9 + 0.608635e9},
    ("c2_bf16_fwdbwd", 1e-3): {"digest": "47f036696d37ae2e", "T": 2048, "bytes": 1.354420e9 + 0.603881e9},
    ("c3_f32_heavy", 1e-4): {"digest": "47f036696d37ae2e", "T": 1024, "bytes": 2.148133e9 + 1.068105e9},
}


def _kernel_digest(names=("dvp_common.cuh", "dvp_rows_impl.cuh")) -> str:
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2512_23087_b200", "csrc")
    for name in names:
        h.update(open(os.path.join(csrc, name), "rb").read())
    return h.hexdigest()[:16]


# DRAM bytes of the contractions of the fused step (dram__bytes_read.sum + dram__bytes_write.sum of the six
# gemm_tn_pair_kernel launches of `bench.py --workload c4_fused_lmhead --rows 8192`, H = 4096, V = 151,936,
# panels of 4096 rows): the first panel's three and a later panel's three (whose d_w contraction also reads
# the d_w it adds to).  Valid for the sources whose digest is recorded; a step of P panels is taken as the
# first panel's launches plus P - 1 times the later panel's.
NCU_TRAFFIC_FUSED = {"digest": "607894dc2e40aeae", "H": 4096, "V": 151936, "panel": 4096,
                     "first": (4.016951e9 + 2.557340e9) + (13.478416e9 + 0.144871e9) + (4.635654e9 + 2.545532e9),
                     "later": (3.567931e9 + 2.542042e9) + (13.443569e9 + 0.145225e9) + (7.493283e9 + 2.471862e9)}
FUSED_SOURCES = ("dvp_gemm.cuh", "dvp_fused.cu", "dvp_panel.cuh")


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            return float(json.load(open(path))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while a region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.file = None

    def start(self):
        try:
            self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=self.file, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.file.flush()
        self.file.seek(0)
        sm, smax, reasons, power = [], [], set(), []
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in self.file.read().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 8:
                continue
            try:
                sm.append(float(parts[0]))
                smax.append(float(parts[1]))
                power.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(names, parts[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        self.file.close()
        os.unlink(self.file.name)
        if sm:
            sm.sort()
            out.update(sm_mhz=sm[len(sm) // 2], sm_max_mhz=max(smax), reasons=sorted(reasons),
                       samples=len(sm), power_w_max=max(power))
        return out


def _dist_setup():
    import torch
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    else:
        torch.cuda.set_device(0)
    return rank, world, local


def _oracle_sample(host, rho, threads, want_grad):
    """Time the fp64 checker on ``host`` (a dict of host arrays)."""
    import oracle
    t0 = time.perf_counter()
    res = oracle.dvp_rows(host["train"], host["ids"], rho, dtype=host["dtype"], infer=host["infer"],
                          upstream=host["upstream"] if want_grad else None, want_grad=want_grad,
                          threads=threads)
    return time.perf_counter() - t0, res.threads


def _host_rows(batch, r0, r1):
    import numpy as np
    import torch
    import oracle

    def st(x):
        x = x[r0:r1].cpu()
        return x.numpy() if x.dtype == torch.float32 else x.view(torch.int16).numpy().view(np.uint16)
    code = {torch.float32: oracle.F32, torch.bfloat16: oracle.BF16, torch.float16: oracle.F16}
    return {"train": st(batch.train), "infer": st(batch.infer), "ids": batch.ids[r0:r1].cpu().numpy(),
            "upstream": batch.upstream[r0:r1].cpu().numpy().astype("f8"),
            "dtype": code[batch.train.dtype]}


def cpu_baseline(batch, rho, backward):
    """The checker as it stands, all host cores, on the first rows of the batch."""
    cores = os.cpu_count() or 1
    slab = 256
    total_t, rows, used = 0.0, 0, 1
    for i in range(16):
        r0 = i * slab
        if r0 + slab > batch.train.shape[0]:
            break
        dt, used = _oracle_sample(_host_rows(batch, r0, r0 + slab), rho, cores, backward)
        total_t += dt
        rows += slab
        if total_t * used > 20.0:
            break
    # the same checker on one thread, on fewer rows
    one_rows = min(64, batch.train.shape[0])
    one_t, _ = _oracle_sample(_host_rows(batch, 0, one_rows), rho, 1, backward)
    return {"value": rows / total_t, "unit": UNIT, "cores": used, "kind": "oracle",
            "sample": f"first {rows} rows of the batch (V={batch.train.shape[1]}), fp64, {used} threads, "
                      f"rows split statically, {total_t:.2f} s wall",
            "one_thread": {"value": one_rows / one_t, "unit": UNIT, "cores": 1,
                           "sample": f"first {one_rows} rows, {one_t:.2f} s wall"}}


def run_reference(args):
    """--impl reference: the fp64 CPU checker, timed on host cores."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    from paper_2512_23087_b200 import inputs
    w = inputs.WORKLOADS[args.workload]
    rho = args.rho if args.rho is not None else w.rhos[0]
    rows_per_step = 128
    batch = inputs.make_rows(w, seed=0, device="cpu", T=rows_per_step * 2, chunk_rows=64)
    cores = os.cpu_count() or 1
    host = [_host_rows(batch, i * rows_per_step, (i + 1) * rows_per_step) for i in range(2)]
    for i in range(args.warmup):
        _oracle_sample(host[i % 2], rho, cores, w.backward)
    t, used = 0.0, 1
    for i in range(args.steps):
        dt, used = _oracle_sample(host[i % 2], rho, cores, w.backward)
        t += dt
    value = rows_per_step * args.steps / t
    sample = (f"{rows_per_step} rows per step of {w.name} (V={w.V}, {w.dtype}), fp64 CPU checker, "
              f"{used} threads")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": w.name, "T_per_step": rows_per_step, "V": w.V, "rho": rho,
                   "logits_dtype": w.dtype, "note": "bounded sample of the workload per step"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": used, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def run_ours(args):
    import torch
    from paper_2512_23087_b200 import binding, inputs

    rank, world, local = _dist_setup()
    dev = torch.device("cuda", local)
    w = inputs.WORKLOADS[args.workload]
    rho = args.rho if args.rho is not None else w.rhos[0]
    T = args.rows if args.rows else w.T
    elem = 2 if w.dtype in ("bf16", "f16") else 4
    grad_dtype = inputs.torch_dtype(w.grad_dtype or w.dtype)
    grad_elem = torch.empty(0, dtype=grad_dtype).element_size()
    batch = inputs.make_rows(w, seed=rank, device=dev, T=T)
    V = batch.train.shape[1]
    stream = torch.cuda.current_stream()

    def step(out=None):
        return binding.dvp_forward(batch.train, batch.ids, rho, infer_logits=batch.infer,
                                   upstream=batch.upstream if w.backward else None,
                                   grad_dtype=grad_dtype, stream=stream, launch_hint=args.launch_hint,
                                   out=out)

    warmup = max(args.warmup, 3)
    res = step()
    for _ in range(warmup - 1):
        step(res)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            torch.distributed.barrier()
            torch.cuda.synchronize()

    sampler = ClockSampler(local)
    barrier()
    sampler.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record(stream)
    # an event after the first steps as well: a long run of this kernel reaches the board's power limit and its
    # clock drops, a short one does not (the copy that measured `peak` was a short one)
    n_first = min(20, args.steps)
    ev_first = torch.cuda.Event(enable_timing=True)
    for i in range(args.steps):
        step(res)
        if i + 1 == n_first:
            ev_first.record(stream)
    ev1.record(stream)
    barrier()
    ms = ev0.elapsed_time(ev1)
    ms_first = ev0.elapsed_time(ev_first) / n_first
    clocks = sampler.stop()
    launches = args.steps          # one kernel per dvp_forward call

    # the workload's other threshold, timed the same way and reported beside the headline
    other = None
    if args.rho is None and len(w.rhos) > 1:
        rho2 = w.rhos[1]
        res2 = None
        for _ in range(3):
            res2 = binding.dvp_forward(batch.train, batch.ids, rho2, infer_logits=batch.infer,
                                       upstream=batch.upstream if w.backward else None,
                                       grad_dtype=grad_dtype, stream=stream, out=res2)
        barrier()
        ev2, ev3 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev2.record(stream)
        for _ in range(args.steps):
            binding.dvp_forward(batch.train, batch.ids, rho2, infer_logits=batch.infer,
                                upstream=batch.upstream if w.backward else None,
                                grad_dtype=grad_dtype, stream=stream, out=res2)
        ev3.record(stream)
        barrier()
        other = {"rho": rho2, "ms_per_step": ev2.elapsed_time(ev3) / args.steps}
        launches += args.steps

    # ---- end to end: host buffers in, per-token results out, copies inside the timed region
    slab = min(T, 2048)
    n_slabs = (T + slab - 1) // slab
    pool = 2
    h_train = [torch.empty(slab, V, dtype=batch.train.dtype).pin_memory() for _ in range(pool)]
    h_infer = [torch.empty(slab, V, dtype=batch.train.dtype).pin_memory() for _ in range(pool)]
    for i in range(pool):
        r0 = i * slab if (i + 1) * slab <= T else 0
        h_train[i].copy_(batch.train[r0:r0 + slab])
        h_infer[i].copy_(batch.infer[r0:r0 + slab])
    h_ids = batch.ids.cpu().pin_memory()
    h_up = batch.upstream.cpu().pin_memory()
    h_out = torch.empty(3, T, dtype=torch.float32).pin_memory()
    h_flags = torch.empty(T, dtype=torch.uint8).pin_memory()
    d_train = [torch.empty(slab, V, dtype=batch.train.dtype, device=dev) for _ in range(2)]
    d_infer = [torch.empty(slab, V, dtype=batch.train.dtype, device=dev) for _ in range(2)]
    d_grad = [torch.empty(slab, V, dtype=grad_dtype, device=dev) for _ in range(2)]
    copy_stream = torch.cuda.Stream(device=dev)
    e2e_steps = max(1, min(args.steps, args.e2e_steps))

    def e2e_step():
        d_ids = h_ids.to(dev, non_blocking=True)
        d_up = h_up.to(dev, non_blocking=True)
        ready = [torch.cuda.Event(), torch.cuda.Event()]
        done = [None, None]
        for s in range(n_slabs):
            b = s % 2
            rows = min(slab, T - s * slab)
            with torch.cuda.stream(copy_stream):
                if done[b] is not None:
                    copy_stream.wait_event(done[b])
                d_train[b][:rows].copy_(h_train[s % pool][:rows], non_blocking=True)
                d_infer[b][:rows].copy_(h_infer[s % pool][:rows], non_blocking=True)
                ready[b].record(copy_stream)
            stream.wait_event(ready[b])
            sl = slice(s * slab, s * slab + rows)
            r = binding.dvp_forward(d_train[b][:rows], d_ids[sl], rho, infer_logits=d_infer[b][:rows],
                                    upstream=d_up[sl] if w.backward else None,
                                    grad_train=d_grad[b][:rows] if w.backward else None,
                                    stream=stream, launch_hint=args.launch_hint)
            h_out[0, sl].copy_(r.train.logp_mp, non_blocking=True)
            h_out[1, sl].copy_(r.infer.logp_mp, non_blocking=True)
            h_out[2, sl].copy_(r.log_ratio, non_blocking=True)
            h_flags[sl].copy_(r.flags, non_blocking=True)
            done[b] = torch.cuda.Event()
            done[b].record(stream)

    e2e_step()
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        e2e_step()
    barrier()
    e2e_s = time.perf_counter() - t0
    h2d = 2 * T * V * elem + T * 8 + T * 4
    d2h = 3 * T * 4 + T

    if world > 1:
        t = torch.tensor([ms, e2e_s, ms_first], device=dev, dtype=torch.float64)
        torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
        ms, e2e_s, ms_first = t.tolist()
    tokens = T * world
    value = tokens * args.steps / (ms * 1e-3)
    peak, peak_kind = _peaks()
    alg_bytes = (2 * elem + (grad_elem if w.backward else 0)) * T * V
    achieved = alg_bytes / (ms * 1e-3 / args.steps) / 1e9
    traffic = None
    rec = NCU_TRAFFIC.get((w.name, rho))
    if rec and rec["digest"] == _kernel_digest():
        traffic = rec["bytes"] * (T / rec["T"])      # rows are independent: traffic grows with T

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": warmup, "ms_per_step": ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": w.name, "T_per_gpu": T, "V": V, "logits_dtype": w.dtype,
                   "grad_dtype": str(grad_dtype).replace("torch.", ""), "rho": rho,
                   "backward": w.backward,
                   "parallelism": f"rows sharded over {world} GPU(s), no collective",
                   "l2": "inputs larger than L2, no flush" if alg_bytes > (1 << 30) else "inputs fit L2",
                   "launch_hint": args.launch_hint},
        "clocks": clocks,
        "e2e": {"value": tokens * e2e_steps / e2e_s, "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "steps": e2e_steps,
                "note": f"pinned host slabs of {slab} rows, copies overlapped with kernels on a second "
                        f"stream, per-token results copied back, gradient stays on the device"},
        "gpu_launches": launches,
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "traffic": traffic, "peak_kind": f"of {peak_kind}",
                     "kernel": "dvp_row_kernel", "bytes_per_launch": alg_bytes,
                     "frac_of_nominal_8TBs": achieved / 8000.0,
                     # DRAM bytes actually moved per second against the same peak: how busy HBM is,
                     # revisits included (None without a traffic record for these kernel sources)
                     "dram_busy_frac": (traffic / (ms * 1e-3 / args.steps) / 1e9 / peak) if traffic else None,
                     # the first steps of the same timed region, before the power limit lowers the clock
                     "first_steps": {"steps": n_first, "ms_per_step": ms_first,
                                     "achieved": alg_bytes / (ms_first * 1e-3) / 1e9,
                                     "frac": alg_bytes / (ms_first * 1e-3) / 1e9 / peak}},
    }
    if other is not None:
        if world > 1:
            t2 = torch.tensor([other["ms_per_step"]], device=dev, dtype=torch.float64)
            torch.distributed.all_reduce(t2, op=torch.distributed.ReduceOp.MAX)
            other["ms_per_step"] = t2.item()
        sec2 = other["ms_per_step"] * 1e-3
        other.update(value=tokens / sec2, unit=UNIT, achieved_gbs=alg_bytes / sec2 / 1e9,
                     frac=alg_bytes / sec2 / 1e9 / peak)
        line["other_threshold"] = other
    if rank == 0:
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(batch, rho, w.backward)
        if world == 1 and args.workload == "c2_bf16_fwdbwd" and not args.rows and not args.no_extras:
            # the other configurations, one after the other, each with the device to itself
            del batch, res, h_train, h_infer, d_train, d_infer, d_grad
            if other is not None:
                del res2
            torch.cuda.empty_cache()
            steps = max(3, min(args.steps, 10))
            for name in ("c1_bf16_fwd", "c3_f32_heavy"):
                line[name] = rows_extra(name, steps, dev, peak, peak_kind, args.no_cpu_baseline)
                torch.cuda.empty_cache()
            fargs = argparse.Namespace(**vars(args))
            fargs.workload, fargs.rho, fargs.steps, fargs.e2e_steps = "c4_fused_lmhead", None, steps, 1
            fline = fused_measure(fargs, 0, 1, dev)
            line["c4_fused_lmhead"] = {k: fline[k] for k in ("ms_per_step", "value", "unit", "config", "clocks", "e2e",
                                                             "roofline", "parity_sample", "cpu_baseline",
                                                             "gpu_launches") if k in fline}
            line["gpu_launches"] += sum(line[n].get("gpu_launches", 0)
                                        for n in ("c1_bf16_fwd", "c3_f32_heavy", "c4_fused_lmhead"))
        print(json.dumps(line))
    if world > 1:
        torch.distributed.destroy_process_group()


def rows_extra(name, steps, dev, peak, peak_kind, no_cpu_baseline):
    """One row configuration beside the headline: ms per step, tokens/s, algorithmic GB/s and
    its fraction of the peak, per threshold, with its own clock samples."""
    import torch
    from paper_2512_23087_b200 import binding, inputs
    w = inputs.WORKLOADS[name]
    batch = inputs.make_rows(w, seed=0, device=dev, T=w.T)
    T, V = batch.train.shape
    elem = batch.train.element_size()
    grad_dtype = inputs.torch_dtype(w.grad_dtype or w.dtype)
    alg_bytes = (2 * elem + (torch.empty(0, dtype=grad_dtype).element_size() if w.backward else 0)) * T * V
    stream = torch.cuda.current_stream()
    out = {"config": {"workload": name, "T": T, "V": V, "logits_dtype": w.dtype, "backward": w.backward,
                      "l2": "inputs larger than L2, no flush"}, "bytes_per_launch": alg_bytes, "thresholds": []}
    sampler = ClockSampler(dev.index or 0)
    sampler.start()
    launches = 0
    res = None
    for rho in w.rhos:
        for _ in range(3):
            res = binding.dvp_forward(batch.train, batch.ids, rho, infer_logits=batch.infer,
                                      upstream=batch.upstream if w.backward else None, grad_dtype=grad_dtype,
                                      stream=stream, out=res)
        torch.cuda.synchronize()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record(stream)
        for _ in range(steps):
            binding.dvp_forward(batch.train, batch.ids, rho, infer_logits=batch.infer,
                                upstream=batch.upstream if w.backward else None, grad_dtype=grad_dtype,
                                stream=stream, out=res)
        ev1.record(stream)
        torch.cuda.synchronize()
        sec = ev0.elapsed_time(ev1) * 1e-3 / steps
        launches += steps
        out["thresholds"].append({"rho": rho, "ms_per_step": sec * 1e3, "value": T / sec, "unit": UNIT,
                                  "achieved_gbs": alg_bytes / sec / 1e9, "frac": alg_bytes / sec / 1e9 / peak,
                                  "peak_kind": f"of {peak_kind}", "frac_of_nominal_8TBs": alg_bytes / sec / 1e9 / 8000.0})
    out["clocks"] = sampler.stop()
    out["steps"] = steps
    out["gpu_launches"] = launches
    if not no_cpu_baseline:
        cores = os.cpu_count() or 1
        rows = 256
        dt, used = _oracle_sample(_host_rows(batch, 0, rows), w.rhos[0], cores, w.backward)
        one_t, _ = _oracle_sample(_host_rows(batch, 0, 32), w.rhos[0], 1, w.backward)
        out["cpu_baseline"] = {"value": rows / dt, "unit": UNIT, "cores": used, "kind": "oracle",
                               "sample": f"first {rows} rows, fp64, {used} threads, {dt:.2f} s wall",
                               "one_thread": {"value": 32 / one_t, "unit": UNIT, "cores": 1,
                                              "sample": f"first 32 rows, {one_t:.2f} s wall"}}
    return out


def run_fused(args):
    """Secondary line: the fused LM-head entry point (tensor-core bound)."""
    import torch
    rank, world, local = _dist_setup()
    line = fused_measure(args, rank, world, torch.device("cuda", local))
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        torch.distributed.destroy_process_group()


def fused_measure(args, rank, world, dev):
    import numpy as np
    import torch
    from paper_2512_23087_b200 import binding, inputs

    local = dev.index or 0
    w = inputs.WORKLOADS[args.workload]
    rho = args.rho if args.rho is not None else w.rhos[0]
    T = args.rows if args.rows else w.T
    batch = inputs.make_fused(w, seed=rank, device=dev, T=T)
    H, V = w.H, w.V
    stream = torch.cuda.current_stream()
    state = {"ws": None, "dw": torch.empty(V, H, dtype=torch.float32, device=dev)}

    def step(hidden=batch.hidden, wv=batch.w_vocab, infer=batch.infer, ids=batch.ids, up=batch.upstream):
        r = binding.dvp_fused_lmhead_forward_backward(hidden, wv, ids, rho, up, infer_logits=infer,
                                                      d_w=state["dw"], panel_rows=args.panel_rows,
                                                      workspace=state["ws"], stream=stream)
        state["ws"] = r.workspace
        return r

    warmup = max(args.warmup, 3)
    for _ in range(warmup):
        res = step()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            torch.distributed.barrier()
            torch.cuda.synchronize()

    sampler = ClockSampler(local)
    barrier()
    sampler.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record(stream)
    for _ in range(args.steps):
        res = step()
    ev1.record(stream)
    barrier()
    ms = ev0.elapsed_time(ev1)
    clocks = sampler.stop()
    status = int(res.workspace[:4].view(torch.int32).item())
    n_panels = (T + (args.panel_rows or min(4096, (T + 127) // 128 * 128)) - 1) // (args.panel_rows or min(4096, (T + 127) // 128 * 128))
    launches = args.steps * (3 + 5 * n_panels + 2)
    safe_total = float(res.train.count.double().sum().item())

    # end to end: operands from pinned host memory, per-token results back
    h_hidden, h_w = batch.hidden.cpu().pin_memory(), batch.w_vocab.cpu().pin_memory()
    h_ids, h_up = batch.ids.cpu().pin_memory(), batch.upstream.cpu().pin_memory()
    slab = min(T, 2048)
    h_infer = batch.infer[:slab].cpu().pin_memory()
    d_infer = torch.empty_like(batch.infer)
    h_out = torch.empty(3, T, dtype=torch.float32).pin_memory()
    e2e_steps = max(1, min(args.steps, args.e2e_steps))

    def e2e_step():
        hd, wd = h_hidden.to(dev, non_blocking=True), h_w.to(dev, non_blocking=True)
        idd, upd = h_ids.to(dev, non_blocking=True), h_up.to(dev, non_blocking=True)
        for r0 in range(0, T, slab):
            rows = min(slab, T - r0)
            d_infer[r0:r0 + rows].copy_(h_infer[:rows], non_blocking=True)
        r = step(hd, wd, d_infer, idd, upd)
        h_out[0].copy_(r.train.logp_mp, non_blocking=True)
        h_out[1].copy_(r.infer.logp_mp, non_blocking=True)
        h_out[2].copy_(r.log_ratio, non_blocking=True)

    e2e_step()
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        e2e_step()
    barrier()
    e2e_s = time.perf_counter() - t0
    h2d = T * H * 2 + V * H * 2 + T * V * 2 + T * 12
    d2h = 3 * T * 4

    if world > 1:
        t = torch.tensor([ms, e2e_s], device=dev, dtype=torch.float64)
        torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
        ms, e2e_s = t.tolist()
    tokens = T * world
    sec = ms * 1e-3 / args.steps
    flops = 2.0 * T * V * H + 4.0 * H * safe_total       # logits, then dH and dW over the safe entries
    peak, burst, kind = 1400.0, 1590.0, "fallback"
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            pk = json.load(open(path))
            peak, burst, kind = float(pk["bf16_tflops_sustained"]), float(pk["bf16_tflops"]), "measured (sustained)"
        except Exception:
            pass
    achieved = flops / sec / 1e12
    # DRAM bytes per launch of the contraction kernel, averaged over the step's launches
    traffic = None
    rec = NCU_TRAFFIC_FUSED
    panel = args.panel_rows or min(4096, (T + 127) // 128 * 128)
    if (rec["digest"] == _kernel_digest(FUSED_SOURCES) and (H, V, panel) == (rec["H"], rec["V"], rec["panel"])
            and T % panel == 0):
        n_p = T // panel
        traffic = (rec["first"] + (n_p - 1) * rec["later"]) / (3 * n_p)
    line = {
        "metric": "fused_lmhead_" + METRIC, "value": tokens / sec, "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": warmup, "ms_per_step": ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "T_per_gpu": T, "H": H, "V": V, "rho": rho,
                   "panel_rows": args.panel_rows or "default", "mean_safe_set": safe_total / T,
                   "l2": "operands larger than L2, no flush", "status_word": status},
        "clocks": clocks,
        "e2e": {"value": tokens * e2e_steps / e2e_s, "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "steps": e2e_steps,
                "note": "hidden, W, infer logits, ids, upstream from pinned host memory each step; "
                        "per-token results copied back; d_hidden and d_w stay on the device"},
        "gpu_launches": launches,
        "roofline": {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                     "frac": achieved / peak, "traffic": traffic, "peak_kind": f"of {kind}",
                     "kernel": "gemm_tn_pair_kernel (three contractions per panel; traffic = DRAM bytes per launch, "
                               "mean over the step's launches)",
                     "flops_per_step": flops, "frac_of_burst": achieved / burst,
                     "frac_of_nominal_2250": achieved / 2250.0},
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        n = 16
        bits = lambda x: x.detach().cpu().view(torch.int16).numpy().view(np.uint16)
        t0 = time.perf_counter()
        want = oracle.dvp_fused_lmhead(bits(batch.hidden[:n]), bits(batch.w_vocab), bits(batch.infer[:n]),
                                       batch.ids[:n].cpu().numpy(), rho, batch.upstream[:n].cpu().numpy().astype("f8"))
        dt = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": n / dt, "unit": UNIT, "cores": os.cpu_count(), "kind": "oracle",
                                "sample": f"first {n} rows, full V and H, fp64 (numpy matmul threads + "
                                          f"row oracle), {dt:.1f} s wall"}
        # the timed result's first rows against what the checker just computed: tokens whose
        # safe-set size agrees (no logit flipped within rounding distance of the threshold)
        # must match in log-probability (1e-4) and in their d_hidden row (1e-3 relative L2)
        same = res.train.count[:n].cpu().numpy() == want.rows.train.count
        lp = res.train.logp_mp[:n].cpu().double().numpy()
        fin = np.isfinite(want.rows.train.logp_mp) & np.isfinite(lp) & same
        lp_err = float(np.abs(lp - want.rows.train.logp_mp)[fin].max()) if fin.any() else 0.0
        dh = res.d_hidden[:n].cpu().double().numpy()
        num = np.linalg.norm(dh - want.d_hidden, axis=1)[same]
        den = np.linalg.norm(want.d_hidden, axis=1)[same]
        dh_err = float((num / np.maximum(den, 1e-6 * max(den.max(), 1e-300))).max()) if same.any() else 0.0
        line["parity_sample"] = {"rows": n, "rows_with_the_same_safe_set_size": int(same.sum()),
                                 "logp_mp_max_err": lp_err, "d_hidden_worst_row_rel_l2": dh_err,
                                 "status_word": status}
        if status != 0 or lp_err > 1e-4 or dh_err > 1e-3 or not same.any():
            print(json.dumps(line))
            raise SystemExit("fused LM-head result disagrees with the fp64 checker on its first rows")
    return line


def spawn_ranks(n: int) -> int:
    """`bench.py --gpus N` without a launcher: start N ranks of this same command line, one per
    GPU, through torch.distributed.run on the loopback address."""
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "WARN")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__), *sys.argv[1:]]
    return subprocess.call(cmd, env=env)


def dry_run_ranks(args):
    """The multi-rank plumbing without a GPU: rendezvous over gloo, shard the rows, take the
    maximum of a per-rank number the way the timed paths do, rank 0 prints one line."""
    import torch
    import torch.distributed as dist
    from paper_2512_23087_b200 import inputs
    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("gloo")
    w = inputs.WORKLOADS[args.workload]
    r0, r1 = inputs.shard_rows(w.T * world, rank, world)     # weak scaling: every rank its own w.T rows
    t = torch.tensor([float(rank + 1), float(r1 - r0)], dtype=torch.float64)
    if world > 1:
        dist.barrier()
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    if rank == 0:
        print(json.dumps({"dry_run": True, "n_gpus": world, "max_over_ranks": t[0].item(),
                          "rows_per_rank": int(t[1].item()), "scaling": "weak"}))
    if world > 1:
        dist.destroy_process_group()


def run_row_classes(args):
    """Where the time of a row workload goes: batches made of copies of ONE row each, the rows taken at
    percentiles of the number of 32-byte granules that hold a safe token (every copy has its own memory),
    timed like the headline.  One JSON line; a diagnostic, not the benchmark."""
    import math
    import torch
    from paper_2512_23087_b200 import binding, inputs
    w = inputs.WORKLOADS[args.workload]
    rho = args.rho if args.rho is not None else w.rhos[0]
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(dev)
    pool, T, V = 2048, args.rows or 8192, w.V
    b = inputs.make_rows(w, seed=0, device=dev, T=pool)
    elem = b.train.element_size()
    per_granule = 32 // elem
    z = b.train.float()
    tau = z.max(dim=1).values + math.log(rho)
    hot = (z.view(pool, -1, per_granule).max(dim=2).values >= tau[:, None]).sum(dim=1)
    safe = (z >= tau[:, None]).sum(dim=1)
    del z
    order = torch.argsort(hot)
    grad_dtype = torch.float32 if w.dtype == "f32" else b.train.dtype
    out = []
    for pct in (1, 25, 50, 75, 90, 95, 99, 100):
        i = int(order[min(pool - 1, pool * pct // 100)])
        train = b.train[i:i + 1].expand(T, V).contiguous()
        infer = b.infer[i:i + 1].expand(T, V).contiguous()
        ids = b.ids[i:i + 1].expand(T).contiguous()
        up = b.upstream[i:i + 1].expand(T).contiguous() if w.backward else None
        res = None
        for _ in range(max(3, args.warmup)):
            res = binding.dvp_forward(train, ids, rho, infer_logits=infer, upstream=up, grad_dtype=grad_dtype,
                                      launch_hint=args.launch_hint, out=res)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.steps):
            binding.dvp_forward(train, ids, rho, infer_logits=infer, upstream=up, grad_dtype=grad_dtype,
                                launch_hint=args.launch_hint, out=res)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / args.steps
        alg = (2 * elem + (res.grad_train.element_size() if w.backward else 0)) * T * V
        out.append({"percentile": pct, "hot_granules": int(hot[i]), "safe_tokens": int(safe[i]),
                    "ms_per_step": ms, "achieved_gbs": alg / ms / 1e6})
        del train, infer, res
    peak, kind = _peaks()
    for o in out:
        o["frac"] = o["achieved_gbs"] / peak
    print(json.dumps({"row_classes": out, "workload": w.name, "rho": rho, "T": T, "V": V, "granules_per_row":
                      (V + per_granule - 1) // per_granule, "steps": args.steps, "peak": peak,
                      "peak_kind": f"of {kind}"}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    # 40 steps of the headline kernel are a quarter of a second: a dozen clock samples, and short of the run length
    # (about 100 steps) at which the board's power limit starts to lower the SM clock
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c2_bf16_fwdbwd")
    ap.add_argument("--rho", type=float, default=None)
    ap.add_argument("--rows", type=int, default=0, help="override T (rows per GPU)")
    ap.add_argument("--launch-hint", type=int, default=0)
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--panel-rows", type=int, default=0, help="fused workload: tokens per panel")
    ap.add_argument("--no-extras", action="store_true", help="headline workload only")
    ap.add_argument("--row-classes", action="store_true",
                    help="time batches of copies of one row each, by percentile of revisited granules (a diagnostic)")
    ap.add_argument("--dry-run-ranks", action="store_true",
                    help="ranks only rendezvous (gloo, no GPU) and reduce a number: checks the launch path")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        raise SystemExit(spawn_ranks(args.gpus))
    if args.dry_run_ranks:
        return dry_run_ranks(args)
    if args.row_classes:
        return run_row_classes(args)
    if args.workload == "c4_fused_lmhead":
        if args.impl == "reference":
            if int(os.environ.get("RANK", "0")) == 0:
                print(json.dumps({"impl": "reference", "unavailable":
                                  "the reference arm is defined for the row workloads only"}))
        else:
            run_fused(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
