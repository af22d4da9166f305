#!/usr/bin/env python
"""Benchmark of the EMU reshard: GB/s (bytes read + written) and ms per model-stage transition.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

A step is one pass of the whole hot path (table walk: claim, copy / cast, finish) over one workload, by
default the 8B Split TP1PP1 -> TP4PP2 the metric is quoted on; at N = 1 the default run then measures the other
configurations one after the other in the same process and appends them as `workloads` to the one JSON line.  Inputs are seeded synthetic N(0, 0.02)
weights, resident in HBM before the timed region; the working set (>= 32 GB) is far larger than L2, so no
flush is needed between iterations.  With N > 1 (torchrun) every rank runs an independent replica of the
workload on its own GPU (the path has no exchange step: replicas only), and the value is the sum over
ranks divided by the slowest rank's time.

`--impl reference` times the CPU oracle (the only "reference implementation" there is: the paper ships no
code) on a bounded sample of the same workload, on the host cores.
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

METRIC = "reshard_throughput"
UNIT = "GB/s"
DEFAULT_WORKLOAD = "8b_tp1pp1_to_tp4pp2"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
# DRAM traffic of one nereus_walk launch, from the ncu captures summarised under profiles/ (2-layer 8B stand-ins,
# 2.8 and 4.2 GB on the device): dram__bytes_read.sum equals the algorithmic bytes read (to 0.1%; tables that carry
# per-tile records read those as well, 48 B per tile), and dram__bytes_write.sum falls short of the algorithmic
# bytes written by what is still in L2 when the kernel ends: a constant, not a fraction (51.8 MB for the bit copy,
# 39.2 MB for the cast, the same on the 4-layer stand-ins).  A full launch is scaled accordingly.
NCU_WRITES_LEFT_IN_L2 = {"copy": 51.8e6, "cast": 39.2e6}


def scaled_traffic(rd, wr):
    left = NCU_WRITES_LEFT_IN_L2["cast" if rd > wr else "copy"]
    return rd + wr - min(left, wr)


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--e2e-steps", type=int, default=6)
    ap.add_argument("--cpu-layers", type=int, default=12,
                    help="layers in the CPU-oracle sample, next to embedding and head (about 1 s each on one core)")
    ap.add_argument("--others", default="all", choices=["all", "configs", "none"],
                    help="workloads measured after the headline in the same run (N = 1 only): the other BASELINE "
                         "configs, or those and the k-unit / optimizer-state / layout / DAG workloads, or none")
    ap.add_argument("--other-steps", type=int, default=10)
    ap.add_argument("--small-steps", type=int, default=2000,
                    help="timed iterations of a workload smaller than L2 (long enough for the clock sampler)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--tile-bytes", type=int, default=0)
    ap.add_argument("--ctas-per-sm", type=int, default=0)
    ap.add_argument("--threads", type=int, default=0)
    ap.add_argument("--variant", type=int, default=0)
    return ap.parse_args()


# ------------------------------------------------------------------------------------------------ peaks

def measured_hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ------------------------------------------------------------------------------------------------ clocks

class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_id: str):
        self.gpu_id = gpu_id
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(prefix="nereus_clocks_", suffix=".csv")
            os.close(fd)
            self.out = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.gpu_id}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=self.out, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()          # the exact process this object started
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.out.close()
        sm, mx, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        with open(self.path) as f:
            for line in f:
                p = [x.strip() for x in line.split(",")]
                if len(p) < 8:
                    continue
                try:
                    sm.append(float(p[0])); mx.append(float(p[1])); power.append(float(p[2]))
                except ValueError:
                    continue
                for name, v in zip(names, p[4:8]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
        try:
            os.unlink(self.path)
        except OSError:
            pass
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm), "power_w_max": max(power)}


# ------------------------------------------------------------------------------------------------ workload

class DoesNotFit(RuntimeError):
    pass


def workload_device_bytes(name) -> int:
    """Device memory the workload's shard buffers take (host work only: layouts and compiled tables)."""
    from paper_2609_34645_b200 import binding as B
    from paper_2609_34645_b200 import inputs as I

    wl = I.WORKLOADS[name]
    if wl.dag:
        dag, descs = _plan_dag(wl)
        t = dag.lower(descs)
        ns, nd = t.num_buffers()
        return sum(t.buffer_bytes(False, i) for i in range(ns)) + sum(t.buffer_bytes(True, j) for j in range(nd))
    tot = 0
    for st in wl.stages:
        sh = st.shape
        d = B.ModelDesc(sh.layers, sh.hidden, sh.heads, sh.kv_heads, sh.ffn, sh.vocab, B.DTYPES[st.src[2]], st.value_head)
        for plan, k in ((st.src, 1), (st.dst, st.replicas)):
            tot += k * sum(d.shard_sizes(B.Plan(plan[0], plan[1], B.DTYPES[plan[2]], I.layout_of(plan))))
            tot += st.n_opt * sum(d.shard_sizes(B.Plan(plan[0], plan[1], B.FP32, I.layout_of(plan))))
    return tot                                  # a round trip lands in the sources: nothing more


def build_workload(name, device, tune, check_fit=False):
    """Compiles the workload's transition(s) and allocates seeded sources and sentinel destinations.
    check_fit: raise DoesNotFit instead of allocating when cudaMemGetInfo says the buffers do not fit."""
    import torch
    from paper_2609_34645_b200 import binding as B
    from paper_2609_34645_b200 import inputs as I

    wl = I.WORKLOADS[name]
    if check_fit:
        torch.cuda.empty_cache()
        need, (free, _) = workload_device_bytes(name), torch.cuda.mem_get_info(device)
        if need * 1.01 + (1 << 30) > free:
            raise DoesNotFit(f"needs {need / 1e9:.1f} GB of device memory, {free / 1e9:.1f} GB free")
    parts, descs, srcs, dsts, keep = [], [], [], [], []
    if wl.dag:
        return build_dag_workload(wl, device, tune)
    for st in wl.stages:
        sh = st.shape
        d = B.ModelDesc(sh.layers, sh.hidden, sh.heads, sh.kv_heads, sh.ffn, sh.vocab, B.DTYPES[st.src[2]],
                        st.value_head)
        pa = B.Plan(st.src[0], st.src[1], B.DTYPES[st.src[2]], I.layout_of(st.src))
        pb = B.Plan(st.dst[0], st.dst[1], B.DTYPES[st.dst[2]], I.layout_of(st.dst))
        if st.replicas > 1:
            t = d.compile_replicated(pa, pb, st.replicas)
        elif st.n_opt:
            t = d.compile_state(pa, pb, st.n_opt)
        else:
            t = d.compile(pa, pb)

        def tied_sources(plan, dtype, seed):
            s = I.make_shards(d.shard_sizes(plan), dtype, seed, device)
            es = I.element_size(dtype)
            groups = []
            for tid in range(d.num_tensors()):
                g = []
                for k in range(d.num_shards(plan)):
                    off, rows, cols, rep = d.tensor_slice(plan, k, tid)
                    if rep and rows:
                        g.append((k, off, rows * cols * es))
                if len(g) > 1:
                    groups.append(g)
            I.tie_replicas(s, groups)
            return s

        srcs += tied_sources(pa, st.src[2], st.seed)
        for k in range(st.n_opt):                      # optimizer tensors: fp32, same (tp, pp)
            srcs += tied_sources(B.Plan(pa.tp, pa.pp, B.FP32, pa.layout), "fp32", st.seed * 101 + k)
        n_dst = t.num_buffers()[1]
        dsts += I.sentinel_shards([t.buffer_bytes(True, j) for j in range(n_dst)], device)
        parts.append(t)
        descs.append((d, pa, pb))
        keep.append(d)
    if wl.round_trip:
        assert len(parts) == 1
        d, pa, pb = descs[0]
        back = d.compile(pb, pa)
        parts.append(back)
        t = B.Transition.fuse(parts, chained=True)
        dsts = dsts + srcs                      # the way back lands in the original source buffers
    elif len(parts) > 1:
        t = B.Transition.fuse(parts, chained=False)
    else:
        t = parts[0]
    if any(tune.values()):
        t.tune(**tune)
    t.prepare()
    return wl, t, srcs, dsts, (parts, keep, descs)


def _plan_dag(wl):
    from paper_2609_34645_b200 import binding as B

    dag, descs = B.Dag(), []
    for st, (kind, current, target) in zip(wl.stages, wl.dag):
        sh = st.shape
        d = B.ModelDesc(sh.layers, sh.hidden, sh.heads, sh.kv_heads, sh.ffn, sh.vocab, B.DTYPES[st.src[2]],
                        st.value_head)
        descs.append(d)
        state = sum(d.shard_sizes(B.Plan(1, 1)))
        m = dag.add_stage(kind, state)
        for is_target, coll in ((False, current), (True, target)):
            for tp, pp, first in coll:
                dag.add_unit(m, is_target, tp, pp, list(range(first, first + tp * pp)))
    dag.plan(0)
    return dag, descs


def build_dag_workload(wl, device, tune):
    """A plan change planned as a DAG of EMU primitives and lowered to one task table."""
    from paper_2609_34645_b200 import binding as B
    from paper_2609_34645_b200 import inputs as I

    dag, descs = _plan_dag(wl)
    t = dag.lower(descs)
    units, prims = dag.units(), dag.prims()
    created = {u for p in prims for u in p["dst"]}
    srcs = []
    for u, (m, tp, pp, gpus) in enumerate(units):
        if u in created:
            continue
        d, st = descs[m], wl.stages[m]
        plan = B.Plan(tp, pp)
        s = I.make_shards(d.shard_sizes(plan), st.src[2], st.seed + 31 * u, device)
        es = I.element_size(st.src[2])
        groups = []
        for tid in range(d.num_tensors()):
            g = [(k, off, rows * cols * es) for k in range(tp * pp)
                 for off, rows, cols, rep in [d.tensor_slice(plan, k, tid)] if rep and rows]
            if len(g) > 1:
                groups.append(g)
        I.tie_replicas(s, groups)
        srcs += s
    n_dst = t.num_buffers()[1]
    dsts = I.sentinel_shards([t.buffer_bytes(True, j) for j in range(n_dst)], device)
    if any(tune.values()):
        t.tune(**tune)
    t.prepare()
    return wl, t, srcs, dsts, ([t], descs + [dag], [(descs[0], None, None)])


# ------------------------------------------------------------------------------------------------ CPU oracle leg

def oracle_sample(workload_name, layers, device_srcs=None, with_ends=False, workers=1):
    """Times the oracle, as it stands, on the logical tensors of the first `layers` layers of the workload's
    first stage (gather -> cast -> slice per logical tensor), with_ends also on the embedding, the final norm
    and the head.  workers = 1: one tensor after the other on one core, the oracle as defined.  workers > 1: the
    same single-threaded routine over disjoint tensors on a pool of host threads (ctypes releases the
    interpreter lock), wall-clock over the whole pool.  Returns (GB/s on algorithmic bytes, seconds, what)."""
    import numpy as np
    from concurrent.futures import ThreadPoolExecutor
    from oracle import oracle as O
    from paper_2609_34645_b200 import inputs as I

    st = I.WORKLOADS[workload_name].stages[0]
    sh = st.shape
    odt = {"bf16": O.BF16, "fp32": O.FP32}
    m = O.Model(sh.layers, sh.hidden, sh.heads, sh.kv_heads, sh.ffn, sh.vocab, odt[st.src[2]], st.value_head)
    pa = O.Plan(st.src[0], st.src[1], 0, I.layout_of(st.src))
    pb = O.Plan(st.dst[0], st.dst[1], odt[st.dst[2]], I.layout_of(st.dst))
    layers = max(1, min(layers, sh.layers))
    ses, des = I.element_size(st.src[2]), I.element_size(st.dst[2])
    ids = list(range(1, 1 + 9 * layers))
    if with_ends:
        ids = [0] + ids + [9 * sh.layers + 1, 9 * sh.layers + 2]
    jobs, total_bytes = [], 0
    for tid in ids:
        src_parts, dst_parts = [], []
        for s in range(O.num_shards(m, pa)):
            p = O.locate(m, pa, s, tid)
            if not p.held:
                src_parts.append(None)
                continue
            n = p.nr * p.nc * ses
            if device_srcs is not None:
                src_parts.append(device_srcs[s][p.offset:p.offset + n].cpu().numpy())
            else:
                src_parts.append(I.normal_bytes(n, st.src[2], st.seed * 7919 + tid).numpy())
        # replicated tensors must agree across ranks
        held = [x for x in src_parts if x is not None]
        rows, cols = O.logical_shape(m, tid)
        if len(held) > 1 and held[0].size == rows * cols * ses:
            for x in held[1:]:
                x[:] = held[0]
        for d in range(O.num_shards(m, pb)):
            p = O.locate(m, pb, d, tid)
            dst_parts.append(np.empty(p.nr * p.nc * des, np.uint8) if p.held else None)
            if p.held:
                total_bytes += p.nr * p.nc * (ses + des)
        jobs.append((tid, src_parts, dst_parts))
    t0 = time.perf_counter()
    if workers <= 1:
        for tid, sp, dp in jobs:
            O.reshard_tensor_parts(m, pa, pb, tid, sp, dp)
    else:
        jobs.sort(key=lambda j: -sum(x.size for x in j[2] if x is not None))
        with ThreadPoolExecutor(max_workers=workers) as pool:
            list(pool.map(lambda j: O.reshard_tensor_parts(m, pa, pb, j[0], j[1], j[2]), jobs))
    total_s = time.perf_counter() - t0
    ends = "embedding, final norm, head and " if with_ends else ""
    what = f"oracle on {len(ids)} logical tensors ({ends}layers 0..{layers - 1}) of stage '{st.name}': " \
           f"{total_bytes / 1e9:.2f} GB read+written of the workload's {_algorithmic_gb(workload_name):.2f} GB"
    return total_bytes / total_s / 1e9, total_s, what


def _algorithmic_gb(workload_name):
    from paper_2609_34645_b200 import binding as B
    from paper_2609_34645_b200 import inputs as I
    st = I.WORKLOADS[workload_name].stages[0]
    sh = st.shape
    d = B.ModelDesc(sh.layers, sh.hidden, sh.heads, sh.kv_heads, sh.ffn, sh.vocab, B.DTYPES[st.src[2]], st.value_head)
    t = d.compile(B.Plan(st.src[0], st.src[1], B.DTYPES[st.src[2]], I.layout_of(st.src)),
                  B.Plan(st.dst[0], st.dst[1], B.DTYPES[st.dst[2]], I.layout_of(st.dst)))
    return sum(t.bytes()) / 1e9


def host_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def run_reference(args):
    """The reference arm: the CPU oracle on a bounded sample, timed on the host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import oracle as O
    O.build()
    vals, secs, what = [], [], ""
    for k in range(args.warmup + args.steps):
        v, s, what = oracle_sample(args.workload, 1)
        if k >= args.warmup:
            vals.append(v); secs.append(s)
    value = sum(vals) / len(vals)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * sum(secs) / len(secs),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic", "config": {"workload": args.workload, "sample": what},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": what},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------ ours

def aggregate_over_ranks(total_ms, steps, bytes_per_step, world, device):
    """Replicas only: every rank moved `bytes_per_step` per step; the job's time is the slowest rank's.
    Returns (ms per step, GB/s summed over ranks)."""
    import torch
    import torch.distributed as dist

    tm = torch.tensor([total_ms], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(tm, op=dist.ReduceOp.MAX)
    ms_per_step = float(tm.item()) / steps
    return ms_per_step, world * bytes_per_step / 1e9 / (ms_per_step / 1e3)


def run_ours(args):
    import torch
    import torch.distributed as dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    assert torch.cuda.is_available(), "bench.py needs a CUDA device; the reshard has no CPU fallback"
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)

    from paper_2609_34645_b200 import binding as B

    tune = dict(tile_bytes=args.tile_bytes, ctas_per_sm=args.ctas_per_sm, threads=args.threads,
                variant=args.variant)
    wl, t, srcs, dsts, keep = build_workload(args.workload, device, tune)
    rd, wr = t.bytes()
    stream = torch.cuda.current_stream()
    sp = B.Transition.pointer_array([b.data_ptr() for b in srcs])
    dp = B.Transition.pointer_array([b.data_ptr() for b in dsts])

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        t.run(sp, dp, stream.cuda_stream)
    torch.cuda.synchronize()
    assert t.status() == B.DEV_OK

    props = torch.cuda.get_device_properties(device)
    gpu_id = f"GPU-{props.uuid}" if hasattr(props, "uuid") else str(local)
    sampler = ClockSampler(gpu_id)
    if rank == 0:
        sampler.start()
    launches0 = t.launches()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    barrier()
    for a, b in ev:
        a.record(stream)
        t.run(sp, dp, stream.cuda_stream)
        b.record(stream)
    barrier()
    per_step = [a.elapsed_time(b) for a, b in ev]                   # ms, one launch each
    total_ms = ev[0][0].elapsed_time(ev[-1][1])
    launches = t.launches() - launches0
    clocks = sampler.stop() if rank == 0 else None
    assert t.status() == B.DEV_OK

    ms_per_step, value = aggregate_over_ranks(total_ms, args.steps, rd + wr, world, device)

    # end to end: host buffers in, host buffers out, copies inside the timed region
    e2e = None
    if not args.no_e2e:
        e2e = run_e2e(args, t, srcs, dsts, sp, dp, stream, rd + wr, world, device)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_hbm_peak()
    kernel_ms = statistics.mean(per_step)
    achieved = (rd + wr) / 1e9 / (kernel_ms / 1e3)
    n_trans = len(wl.stages) * (2 if wl.round_trip else 1)
    if wl.dag:
        n_trans = t.num_tiles()[1]                 # dependency levels of the lowered DAG
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None,
        "dtype": "bf16" if all(s.src[2] == "bf16" for s in wl.stages) else "fp32->bf16",
        "data": "synthetic",
        "config": {"workload": wl.name, "transitions_per_step": n_trans,
                   "ms_per_transition": ms_per_step / n_trans,
                   "bytes_read": rd, "bytes_written": wr, "l2": "inputs larger than L2, no flush",
                   "multi_gpu": "replicas only", "tiles": t.num_tiles()[0], "levels": t.num_tiles()[1]},
        "frac_of_nominal_8TBps": achieved / NOMINAL_HBM_GBS,
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": scaled_traffic(rd, wr),
                     "traffic_note": "ncu captures on 2-layer stand-ins: reads = algorithmic bytes, writes = "
                                     "algorithmic bytes minus the ~50 MB still in L2 at kernel end",
                     "peak_kind": f"of {peak_kind}", "kernel": t.launch_info()["kernel"], "launch": t.launch_info(),
                     "kernel_ms": kernel_ms, "kernel_ms_min": min(per_step)},
        "clocks": clocks, "gpu_launches": launches,
    }
    if e2e is not None:
        line["e2e"] = e2e
    per_stage = time_stages_alone(wl, keep, srcs, dsts, stream)
    if per_stage:
        line["config"]["ms_per_stage_alone"] = per_stage
    if world == 1:
        try:
            line["config"]["balance"] = block_balance(t, sp, dp, stream)
        except Exception as e:      # a diagnostic, never a dependency of the number
            line["config"]["balance"] = {"error": repr(e)}
    if not args.no_cpu_baseline and world == 1:
        try:
            from oracle import oracle as O
            O.build()
            v, s, what = oracle_sample(args.workload, args.cpu_layers, srcs, with_ends=True)
            line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": what,
                                    "seconds": s}
            cores = host_cores()
            v, s, what = oracle_sample(args.workload, args.cpu_layers, srcs, with_ends=True, workers=cores)
            line["cpu_baseline_all_cores"] = {
                "value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "seconds": s,
                "sample": what + f"; the same single-threaded routine over disjoint tensors on {cores} host threads"}
        except Exception as e:      # the baseline is a report, never a dependency of the GPU number
            line["cpu_baseline"] = {"value": None, "unit": UNIT, "cores": 1, "kind": "oracle",
                                    "sample": f"failed: {e!r}"}
    if world == 1 and args.others != "none" and args.workload == DEFAULT_WORKLOAD:
        del srcs, dsts, sp, dp, t, keep, wl
        try:                        # the headline above never depends on what follows
            line["workloads"] = measure_others(args, device, gpu_id, peak, peak_kind)
        except Exception as e:
            line["workloads"] = [{"error": repr(e)}]
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


OTHER_CONFIGS = ["tiny_tp2pp1_to_tp1pp1", "8b_tp4pp2_to_tp1pp1", "8b_fp32_tp2pp2_to_bf16_tp4pp1", "ppo5_8b",
                 "32b_tp2pp4_to_tp8pp1_and_back"]
OTHER_NEXT = ["8b_extend_tp4pp2_x2", "8b_fp32_tp2pp2_to_bf16_tp4pp1_x2", "8b_state_adam_tp2pp2_to_tp4pp1",
              "8b_grouped_fp32_tp2pp2_to_blocked_bf16_tp4pp1", "8b_tp4pp1_to_tp16pp1", "8b_dag_tp4pp8_to_tp8pp2"]
L2_BYTES = 126 << 20


def measure_others(args, device, gpu_id, peak, peak_kind):
    """The other configurations, one after the other in this process, each on freshly allocated buffers: kernel
    time per launch by CUDA events on the launching stream, clocks sampled during each timed region.  Workloads
    smaller than L2 get L2 flushed between iterations (256 MiB written, then 256 MiB read, so that no dirty
    lines are left to be written back during the timed launch); a workload that does not fit is skipped with
    the reason."""
    import gc
    import torch
    from paper_2609_34645_b200 import binding as B

    out = []
    tune = dict(tile_bytes=0, ctas_per_sm=0, threads=0, variant=0)
    stream = torch.cuda.current_stream()
    for name in OTHER_CONFIGS + (OTHER_NEXT if args.others == "all" else []):
        gc.collect()
        torch.cuda.empty_cache()
        t0 = time.perf_counter()
        try:
            wl, t, srcs, dsts, keep = build_workload(name, device, tune, check_fit=True)
        except DoesNotFit as e:
            out.append({"workload": name, "skipped": str(e)})
            continue
        except Exception as e:      # e.g. an allocation that fails although the pre-flight passed
            out.append({"workload": name, "skipped": f"could not be set up: {e!r}"})
            gc.collect()
            torch.cuda.empty_cache()
            continue
        rd, wr = t.bytes()
        sp = B.Transition.pointer_array([b.data_ptr() for b in srcs])
        dp = B.Transition.pointer_array([b.data_ptr() for b in dsts])
        small = rd + wr < 4 * L2_BYTES
        steps = max(3, args.small_steps if small else args.other_steps)
        flush = (torch.empty(256 << 20, dtype=torch.uint8, device=device),
                 torch.ones(32 << 20, dtype=torch.int64, device=device)) if small else None
        for _ in range(3):
            t.run(sp, dp, stream.cuda_stream)
        torch.cuda.synchronize()
        build_s = time.perf_counter() - t0
        sampler = ClockSampler(gpu_id)
        sampler.start()
        timed = min(steps, 200)                                     # event pairs kept for the per-launch time
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(timed)]
        torch.cuda.synchronize()
        launches0 = t.launches()
        for k in range(steps):
            if flush:
                flush[0].fill_(k & 127)
                flush[1].sum()
            if k < timed:
                ev[k][0].record(stream)
            t.run(sp, dp, stream.cuda_stream)
            if k < timed:
                ev[k][1].record(stream)
        torch.cuda.synchronize()
        clocks = sampler.stop()
        per = [a.elapsed_time(b) for a, b in ev]
        kernel_ms = statistics.mean(per)
        n_trans = t.num_tiles()[1] if wl.dag else len(wl.stages) * (2 if wl.round_trip else 1)
        achieved = (rd + wr) / 1e9 / (kernel_ms / 1e3)
        ok = t.status() == B.DEV_OK
        out.append({
            "workload": name, "ms_per_step": kernel_ms, "ms_min": min(per), "value": achieved, "unit": UNIT,
            "ms_per_transition": kernel_ms / n_trans, "transitions_per_step": n_trans,
            "frac_of_nominal_8TBps": achieved / NOMINAL_HBM_GBS,
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "frac": achieved / peak,
                         "peak_kind": f"of {peak_kind}"},
            "kernel": t.launch_info()["kernel"], "launch": t.launch_info(), "tiles": t.num_tiles()[0],
            "levels": t.num_tiles()[1], "bytes_read": rd, "bytes_written": wr, "steps": steps,
            "gpu_launches": t.launches() - launches0, "device_status_ok": ok,
            "l2": "flushed between iterations: 256 MiB written, then 256 MiB read" if small
                  else "inputs larger than L2, no flush",
            "clocks": clocks, "build_s": round(build_s, 1)})
        alone = time_stages_alone(wl, keep, srcs, dsts, stream)
        if alone:
            out[-1]["ms_per_stage_alone"] = alone        # every model-stage's transition launched on its own
        try:
            out[-1]["balance"] = block_balance(t, sp, dp, stream)
        except Exception as e:
            out[-1]["balance"] = {"error": repr(e)}
        del srcs, dsts, sp, dp, t, keep, wl, flush
    return out


def block_balance(t, sp, dp, stream):
    """One traced run (outside every timed region): how evenly the blocks of the launch were loaded and how far
    apart they finished, from the GPU's global timer."""
    import torch

    t.trace(True)
    t.prepare()
    for _ in range(2):
        t.run(sp, dp, stream.cuda_stream)
    torch.cuda.synchronize()
    rec = [r for r in t.trace_read() if r[3]]
    t.trace(False)
    t.prepare()
    if not rec:
        return None
    begin, ends = min(r[1] for r in rec), [r[2] for r in rec]
    return {"blocks": len(rec), "tiles_min": min(r[3] for r in rec), "tiles_max": max(r[3] for r in rec),
            "start_spread_us": (max(r[1] for r in rec) - begin) / 1e3,
            "first_block_done_us": (min(ends) - begin) / 1e3, "last_block_done_us": (max(ends) - begin) / 1e3,
            "finish_spread_us": (max(ends) - min(ends)) / 1e3}


def host_memory_budget() -> int:
    """Bytes of host memory this process may safely take: MemAvailable, capped by the cgroup limit."""
    avail = 0
    try:
        with open("/proc/meminfo") as f:
            for line in f:
                if line.startswith("MemAvailable:"):
                    avail = int(line.split()[1]) * 1024
    except OSError:
        pass
    for path, cur in (("/sys/fs/cgroup/memory.max", "/sys/fs/cgroup/memory.current"),
                      ("/sys/fs/cgroup/memory/memory.limit_in_bytes", "/sys/fs/cgroup/memory/memory.usage_in_bytes")):
        try:
            lim = open(path).read().strip()
            if lim != "max":
                used = int(open(cur).read().strip())
                avail = min(avail, max(0, int(lim) - used)) if avail else max(0, int(lim) - used)
        except (OSError, ValueError):
            pass
    return avail


def time_stages_alone(wl, keep, srcs, dsts, stream, runs=5):
    """Multi-stage tables only: every model-stage's transition launched on its own (outside the timed region
    of the metric), ms per launch by CUDA events."""
    import torch

    parts = keep[0]
    if wl.dag or wl.round_trip or len(parts) < 2:
        return None
    out, si, di = {}, 0, 0
    for st, part in zip(wl.stages, parts):
        ns, nd = part.num_buffers()
        sp = [b.data_ptr() for b in srcs[si:si + ns]]
        dp = [b.data_ptr() for b in dsts[di:di + nd]]
        si, di = si + ns, di + nd
        for _ in range(2):
            part.run(sp, dp, stream.cuda_stream)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(runs):
            part.run(sp, dp, stream.cuda_stream)
        b.record(stream)
        stream.synchronize()
        out[st.name] = a.elapsed_time(b) / runs
    return out


def run_e2e(args, t, srcs, dsts, sp, dp, stream, algo_bytes, world, device):
    """Same metric through the C ABI with HOST buffers: every step copies the source shards from pinned host
    memory to the device, runs the transition, and reads the destination shards back to pinned host memory.
    When the device has room for a second set of shard buffers the steps are pipelined over three streams (the
    copy-in of step i+1 and the copy-out of step i-1 run beside the kernel of step i, PCIe being full duplex);
    every step still moves all of its inputs and outputs inside the timed region.  Else one stream, one step
    after the other."""
    import torch
    import torch.distributed as dist
    from paper_2609_34645_b200 import binding as B

    need = sum(b.numel() for b in srcs) + sum(b.numel() for b in dsts)
    budget = host_memory_budget() // max(1, world)      # every rank of the node pins its own copy
    if need > 0.5 * budget:
        return {"value": None, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0,
                "note": f"skipped: {need / 1e9:.1f} GB of pinned host memory needed, {budget / 1e9:.1f} GB available"}
    try:
        h_src = [torch.empty(b.numel(), dtype=torch.uint8, pin_memory=True) for b in srcs]
        h_dst = [torch.empty(b.numel(), dtype=torch.uint8, pin_memory=True) for b in dsts]
    except Exception as e:
        return {"value": None, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0,
                "note": f"pinned host allocation failed: {e!r}"}
    for h, b in zip(h_src, srcs):
        h.copy_(b)
    h2d = sum(b.numel() for b in srcs)
    d2h = sum(b.numel() for b in dsts)
    steps = max(1, args.e2e_steps)

    # a second set of device buffers, if it fits: distinct destination memory only (a round trip lands in its
    # sources, which then are part of both lists)
    sets = [(srcs, dsts, sp, dp)]
    free, _ = torch.cuda.mem_get_info(device)
    aliased = {b.data_ptr() for b in srcs} & {b.data_ptr() for b in dsts}
    if not aliased and need * 1.02 + (2 << 30) < free:
        try:
            srcs2 = [torch.empty_like(b) for b in srcs]
            dsts2 = [torch.empty_like(b) for b in dsts]
            sets.append((srcs2, dsts2, B.Transition.pointer_array([b.data_ptr() for b in srcs2]),
                         B.Transition.pointer_array([b.data_ptr() for b in dsts2])))
        except Exception:           # no room after all: one set, one step after the other
            srcs2 = dsts2 = None
            torch.cuda.empty_cache()
    n = len(sets)
    s_in, s_out = (torch.cuda.Stream(device), torch.cuda.Stream(device)) if n == 2 else (stream, stream)
    ev_in = [torch.cuda.Event() for _ in range(n)]
    ev_k = [torch.cuda.Event() for _ in range(n)]
    ev_out = [torch.cuda.Event() for _ in range(n)]

    def step(i):
        k = i % n
        S, D, spk, dpk = sets[k]
        with torch.cuda.stream(s_in):
            if i >= n:
                s_in.wait_event(ev_k[k])                 # the kernel that last read this set's sources is done
            for h, b in zip(h_src, S):
                b.copy_(h, non_blocking=True)
            ev_in[k].record(s_in)
        stream.wait_event(ev_in[k])
        if i >= n:
            stream.wait_event(ev_out[k])                 # ... and the copy-out that last read its destinations
        t.run(spk, dpk, stream.cuda_stream)
        ev_k[k].record(stream)
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev_k[k])
            for h, b in zip(h_dst, D):
                h.copy_(b, non_blocking=True)
            ev_out[k].record(s_out)

    for i in range(n):
        step(i)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    a.record(stream)
    s_in.wait_event(a)
    for i in range(steps):
        step(n + i)                                       # i >= n: every wait above is armed
    s_out.wait_stream(stream)
    b.record(s_out)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    ok = all(torch.equal(x, y) for x, y in zip(sets[0][1], sets[-1][1]))     # both sets hold the same result
    ms = torch.tensor([a.elapsed_time(b) / steps], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(ms, op=dist.ReduceOp.MAX)
    ms = float(ms.item())
    return {"value": world * algo_bytes / 1e9 / (ms / 1e3), "unit": UNIT, "h2d_bytes_per_step": h2d,
            "d2h_bytes_per_step": d2h, "ms_per_step": ms, "steps": steps,
            "pipelined": n == 2, "device_buffer_sets": n, "results_equal": ok}


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
