#!/usr/bin/env python
"""Benchmark of the GaLore-Adam optimizer step (parameters updated per second).

A "step" is one pass of the whole path (projection, Adam on R with the
configured state format, back-projection, weight write) over every matrix of
the workload's layer set, on synthetic gradients already resident in HBM.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

N > 1 (under torch.distributed.run) runs N independent replicas of the same
workload, one per GPU: the path has no exchange step, so nothing is sharded
and no collective is on the data path; only the timing is reduced over ranks.
`--impl reference` times the CPU oracle on the host cores on a bounded sample.
Prints ONE JSON line on rank 0.
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

METRIC = "galore_adam_step_params_per_sec"
UNIT = "params/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# fp32 FMA peak of the part: 148 SMs x 128 lanes x 2 flop x 1.965 GHz (unit counts and max clock)
FP32_FMA_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        p["source"] = "measured"
        return p
    p = dict(FALLBACK_PEAKS)
    p["source"] = "fallback"
    return p


def elem_bytes(dt):
    return 2 if dt == "bf16" else 4


def algorithmic_cost(w, m, n):
    """Bytes the method must move and flops it must do for one matrix and one step."""
    r = w.rank
    left = m <= n
    d, big = (m, n) if left else (n, m)
    nel = r * big
    state = state_bytes_per_step(w, nel, r, big)
    by = m * n * elem_bytes(w.g_dtype) + 2 * m * n * elem_bytes(w.w_dtype) + state + d * r * elem_bytes(p_dtype_of(w))
    return by, 4 * m * n * r


NOMINAL_HBM_GBS = 8000.0          # data-sheet HBM3e bandwidth
NOMINAL_BF16_TFLOPS = 2250.0       # data-sheet dense bf16 tensor rate


def state_bytes_per_step(w, nel, r, big):
    """Optimizer statistics read and written once per step: two fp32 moments, two 8-bit moments with their
    absmax values, or Adafactor's fp32 first moment with one value per row and per column of R."""
    if w.state_fmt == "f32":
        return 4 * nel * 4
    if w.state_fmt == "adafactor":
        return 2 * nel * 4 + 2 * (r + big) * 4
    return 4 * nel + 4 * 4 * ((nel + w.q_block - 1) // w.q_block)


def p_dtype_of(w):
    return "bf16" if w.g_dtype == "bf16" else "f32"


# DRAM traffic of the step's kernels from ncu captures of the kernels as they are now (dram__bytes_read.sum +
# dram__bytes_write.sum of one launch over a group of attention-shaped matrices, summarised under profiles/
# with the command that made them), as a multiple of the algorithmic bytes of that launch (kernel_costs
# below).  Traffic grows in proportion to the matrices a launch covers, so a full-size launch is taken to
# move the same multiple of its own algorithmic bytes.  Absent: not captured since the kernel last changed.
KERNEL_DRAM_OVER_ALGORITHMIC = {
    # (rank, state format): {kernel: measured / algorithmic}
    # (the fp32 R the projection writes and the Adam kernel reads, 134.2 MB here, is traffic the method does not need)
    (1024, "q8"): {"projection": 607.6 / 335.5, "adam": 405.3 / 201.3, "back_projection": 830.0 / 671.1},
    (512, "f32"): {"projection_with_adam": 560.9 / 469.8, "back_projection": 438.1 / 335.5},
}


def kernel_costs(w, shapes):
    """Algorithmic flops and bytes of each kernel of the step, summed over the layer set.

    projection (with Adam in its epilogue when fused): reads G and P, reads and writes the moments, writes N.
    back-projection: reads P and N, reads and writes W.  N (r x max(m, n) bf16 or fp32) is an intermediate
    the method itself does not need; it is counted here because these are per-kernel roofs."""
    proj = {"flops": 0, "bytes": 0}
    back = {"flops": 0, "bytes": 0}
    adam = {"flops": 0, "bytes": 0}
    n_b = 2 if w.g_dtype == "bf16" else 4
    for (m, n) in shapes:
        r = w.rank
        d, big = (m, n) if m <= n else (n, m)
        nel = r * big
        state = state_bytes_per_step(w, nel, r, big)
        p_bytes = d * r * elem_bytes(p_dtype_of(w))
        proj["flops"] += 2 * m * n * r
        proj["bytes"] += m * n * elem_bytes(w.g_dtype) + p_bytes
        adam["bytes"] += state + nel * n_b
        back["flops"] += 2 * m * n * r
        back["bytes"] += 2 * m * n * elem_bytes(w.w_dtype) + p_bytes + nel * n_b
    return proj, adam, back


def max_over_ranks(value: float, dist, device) -> float:
    """The slowest rank's time: every multi-GPU number is a maximum over ranks."""
    if dist is None:
        return float(value)
    import torch
    t = torch.tensor([value], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.out = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=self.out, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        res = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return res
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.out.close()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        with open(self.path) as f:
            for line in f:
                parts = [p.strip() for p in line.split(",")]
                if len(parts) < 8:
                    continue
                try:
                    sm.append(float(parts[0]))
                    mx.append(float(parts[1]))
                except ValueError:
                    continue
                for name, val in zip(names, parts[4:8]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
        os.unlink(self.path)
        if sm:
            res.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return res


def _blas_threads():
    try:
        from threadpoolctl import threadpool_info
        return max([p.get("num_threads", 1) for p in threadpool_info()] or [os.cpu_count() or 1])
    except Exception:
        return os.cpu_count() or 1


def cpu_oracle_sample(w, steps=1, extras=False):
    """Times the oracle, as it stands (numpy on the host's BLAS, fp64), on one matrix of each distinct shape.

    extras: also one step on the smallest shape with the BLAS pool limited to one thread, and one projector
    refresh (the oracle's SVD through the library routine it uses at sizes its Jacobi code cannot reach in
    test time) on the smallest shape.  Returns (params/s, cores, seconds, extras dict)."""
    import numpy as np
    from oracle import galore_oracle as go
    from paper_2403_03507_b200 import workloads as wl
    cores = _blas_threads()
    total_params, total_time = 0, 0.0
    rng = np.random.default_rng(0)
    smallest = None
    for (m, n, _count) in w.shapes:
        side = "left" if m <= n else "right"
        orc = go.GaLoreOracle(m, n, w.rank, w.alpha, w.refresh_gap, w.beta1, w.beta2, w.eps, w_store=w.w_dtype,
                              state="f32" if w.state_fmt == "adafactor" else w.state_fmt, q_block=w.q_block,
                              inner="adafactor" if w.state_fmt == "adafactor" else "adam")
        d = m if side == "left" else n
        P, _ = np.linalg.qr(rng.standard_normal((d, w.rank)))       # any orthonormal projector: timing only
        orc.set_projector(P)
        G = wl.round_to(rng.standard_normal((m, n)) * 0.05, w.g_dtype)
        W = wl.round_to(rng.standard_normal((m, n)) * 0.02, w.w_dtype)
        t0 = time.perf_counter()
        for _ in range(steps):
            W = orc.step(W, G, w.lr, auto_refresh=False)
        total_time += time.perf_counter() - t0
        total_params += m * n * steps
        if smallest is None or m * n < smallest[0] * smallest[1]:
            smallest = (m, n, orc, G, W, side)
    extra = {}
    if extras and smallest is not None:
        m, n, orc, G, W, side = smallest
        try:
            from threadpoolctl import threadpool_limits
            with threadpool_limits(limits=1):
                t0 = time.perf_counter()
                orc.step(W, G, w.lr, auto_refresh=False)
                t1 = time.perf_counter() - t0
            extra["one_thread"] = {"value": m * n / t1, "unit": UNIT, "shape": [m, n], "seconds": t1}
        except Exception as e:                                  # threadpoolctl missing: say so rather than guess
            extra["one_thread"] = {"unavailable": repr(e)}
        t0 = time.perf_counter()
        go.top_r_projector(G, w.rank, side, method="lapack")
        extra["refresh"] = {"seconds": time.perf_counter() - t0, "shape": [m, n], "rank": w.rank, "cores": cores,
                            "method": "library SVD as one step (the Jacobi code is the pinned definition at small sizes)"}
    return total_params / total_time, cores, total_time, extra


def run_reference(args, w):
    value, cores, _ = None, None, None
    times = []
    for i in range(args.warmup + args.steps):
        v, cores, t, _ = cpu_oracle_sample(w, 1)
        if i >= args.warmup:
            times.append((v, t))
    value = sum(v for v, _ in times) / len(times)
    ms = 1e3 * sum(t for _, t in times) / len(times)
    sample = f"1 oracle step on one matrix of each distinct shape ({len(w.shapes)} of {w.matrices} matrices), given projector"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic", "config": {"workload": w.name, "rank": w.rank, "state_fmt": w.state_fmt},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "backend": "numpy on the host BLAS, fp64",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="llama_7b_q8")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--mode", default="batch", choices=["batch", "layer", "arrive"],
                    help="batch: galore_step_batch over the layer set (grouped launches); layer: galore_step per layer; "
                         "arrive: galore_step per layer as its gradient arrives from a producer stream into a ring of "
                         "--ring gradient buffers per shape (per-layer weight updates, Sec. 'Reducing memory footprint "
                         "of gradients': the full set of gradients never exists)")
    ap.add_argument("--ring", type=int, default=2, help="gradient buffers per distinct shape in --mode arrive")
    ap.add_argument("--projector", default="refresh", choices=["refresh", "random"],
                    help="refresh: one real refresh per distinct shape (timed, reported); random: a random orthonormal "
                         "projector (step timing does not depend on P's values; for short profiling runs)")
    ap.add_argument("--weight-decay", type=float, default=0.0,
                    help="GaLore-AdamW: decoupled weight decay folded into the weight update (0 = plain Adam)")
    ap.add_argument("--adam-place", default="auto", choices=["auto", "projection", "own"],
                    help="where Adam on R runs when K is not sliced: in the projection kernel's epilogue or in its own kernel")
    ap.add_argument("--refresh-slots", type=int, default=8,
                    help="layers of one shape refreshed together by galore_refresh_batch (workspace copies; 1 = one by one)")
    ap.add_argument("--layers", type=int, default=0,
                    help="keep only this many transformer layers of the workload's layer set (0 = all): a small case "
                         "of the same kernels for profiler captures")
    ap.add_argument("--rank", type=int, default=0, help="override the workload's rank (rank sweep on one shape)")
    ap.add_argument("--state-fmt", default="", choices=["", "f32", "q8", "adafactor"], help="override the workload's state format")
    ap.add_argument("--refresh-warm", type=int, default=0,
                    help="power steps of a refresh started from the stored projector (0: every refresh starts cold); "
                         "with N > 0 the whole set is also refreshed a second time from slightly moved gradients")
    ap.add_argument("--refresh-only", action="store_true",
                    help="run the projector refresh of each distinct shape and print its timings; no step is timed "
                         "(for profiling the refresh on its own)")
    ap.add_argument("--extra-workloads", default="llama_1b_q8,llama_1b_f32,llama_1b_adafactor,llama_130m,sweep",
                    help="comma-separated workloads also timed, device-resident only, reported under other_workloads "
                         "(only with the default workload; empty string to skip).  'sweep' = the rank sweep on one "
                         "4096 x 11008 matrix: six ranks x both state formats, one matrix per step, with the refresh "
                         "and the throughput with the refresh spread over T = 50, 200, 1000 steps")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else max(args.warmup, 0)

    from paper_2403_03507_b200 import workloads as wl
    w = wl.WORKLOADS[args.workload]
    if args.rank or args.state_fmt:
        import dataclasses
        w = dataclasses.replace(w, rank=args.rank or w.rank, state_fmt=args.state_fmt or w.state_fmt)
    if args.layers > 0 and len(w.shapes) == 3:
        import dataclasses
        (a, b, c4), (d, e, c2), (f, g, c1) = w.shapes
        keep = min(args.layers, c1)
        w = dataclasses.replace(w, shapes=((a, b, 4 * keep), (d, e, 2 * keep), (f, g, keep)))
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        if rank == 0:
            run_reference(args, w)
        return 0

    import torch
    from paper_2403_03507_b200 import binding as gb
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the step has no CPU path")
    gb.lib()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    res = time_workload(w, args, dev, dist, world, rank, full=True)
    if rank == 0:
        extras = []
        names = [x for x in args.extra_workloads.split(",") if x] if args.workload == "llama_7b_q8" and world == 1 and not args.refresh_only else []
        import dataclasses
        for name in names:
            if name == "sweep":
                args.amortise_gaps = wl.SWEEP_GAPS
                for r in wl.SWEEP_RANKS:
                    for fmt in ("q8", "f32"):
                        ws = dataclasses.replace(wl.WORKLOADS["sweep_4096x11008"], rank=r, state_fmt=fmt)
                        extras.append(time_workload(ws, args, dev, None, 1, 0, full=False, mode="layer"))
                args.amortise_gaps = ()
            else:
                extras.append(time_workload(wl.WORKLOADS[name], args, dev, None, 1, 0, full=False))
        if extras:
            res["other_workloads"] = extras
        print(json.dumps(res), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    return 0


def time_workload(w, args, dev, dist, world, rank, full, mode=None):
    mode = mode or args.mode
    import torch
    from paper_2403_03507_b200 import binding as gb
    from paper_2403_03507_b200 import workloads as wl

    tdt = {"f32": torch.float32, "bf16": torch.bfloat16}
    peaks = load_peaks()
    stream = torch.cuda.current_stream()

    def padded(m, n, dtype):
        ld = (n + 15) // 16 * 16       # 32-byte bf16 rows: TMA-addressable, and whole-sector vector accesses
        buf = torch.empty(m, ld, dtype=dtype, device=dev)
        return buf[:, :n]

    # ---- build the layer set -------------------------------------------------------------------
    layers, Ws, Gs, shapes_of = [], [], [], []
    refresh_info = []
    max_ws = 0
    cfgs = {}
    for (m, n, count) in w.shapes:
        cfg = gb.make_config(m, n, w.rank, alpha=w.alpha, refresh_gap=w.refresh_gap, beta1=w.beta1, beta2=w.beta2,
                             eps=w.eps, w_dtype=w.w_dtype, g_dtype=w.g_dtype, state_fmt=w.state_fmt,
                             q_block=w.q_block, auto_refresh=False, seed=w.seed, weight_decay=args.weight_decay,
                             refresh_warm_iters=args.refresh_warm,
                             adam_place={"auto": gb.ADAM_AUTO, "projection": gb.ADAM_IN_PROJECTION, "own": gb.ADAM_OWN_KERNEL}[args.adam_place])
        cfgs[(m, n)] = cfg
        max_ws = max(max_ws, gb.galore_query_bytes(cfg)[1])
    workspace = torch.empty(max_ws, dtype=torch.uint8, device=dev)      # shared: layers step one after another
    bytes_alg, flops_alg = 0, 0
    for si, (m, n, count) in enumerate(w.shapes):
        pool = []
        for j in range(2):                                             # two gradients per distinct shape, cycled
            g = wl.make_gradient_torch(m, n, wl.sub_seed(w.seed, si, j) & 0x7FFFFFFF, w.spectrum_p, w.noise, dev,
                                       tdt[w.g_dtype])
            gp = padded(m, n, tdt[w.g_dtype])
            gp.copy_(g)
            pool.append(gp)
            del g
        first = None
        for c in range(count):
            layer = gb.Layer(cfgs[(m, n)], device=dev, workspace=workspace)
            if first is None and args.projector == "random":
                d = m if m <= n else n
                first = torch.linalg.qr(torch.randn(d, w.rank, device=dev))[0].contiguous()
                layer.set_projector(first)
            elif first is None:
                t0 = torch.cuda.Event(enable_timing=True)
                t1 = torch.cuda.Event(enable_timing=True)
                for rep in range(1 if args.refresh_only else 2):         # the second run is the warm one
                    t0.record()
                    st, info = layer.galore_refresh_projector(pool[0])
                    t1.record()
                    torch.cuda.synchronize()
                refresh_info.append({"shape": [m, n], "count": count, "ms": t0.elapsed_time(t1), "status": st,
                                     **info.as_dict()})
                first = layer.get_projector()
                if args.refresh_only:
                    break
            elif args.projector == "random":
                layer.set_projector(first)                              # timing does not depend on P's values
            Wt = padded(m, n, tdt[w.w_dtype])
            Wt.copy_(torch.randn(m, n, device=dev) * 0.02)
            layers.append(layer)
            Ws.append(Wt)
            Gs.append(pool[c % 2])
            shapes_of.append((m, n))
            by, fl = algorithmic_cost(w, m, n)
            bytes_alg += by
            flops_alg += fl
    torch.cuda.synchronize()
    if args.refresh_only:
        return {"refresh": refresh_info, "config": {"workload": w.name, "rank": w.rank}}

    # ---- the refresh of the whole layer set, as it happens every `refresh_gap` steps ------------------
    refresh_set = None
    if args.projector == "refresh":
        import time
        # room for eight layers of one shape at a time: the library then refreshes them as a group
        need = max(gb.galore_refresh_query_bytes(l) for l in layers)
        slots = max(1, min(8, int(args.refresh_slots)))
        space = torch.empty(slots * need, dtype=torch.uint8, device=dev)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        st, infos = gb.galore_refresh_batch(layers, Gs, stream=stream, workspace=space)
        torch.cuda.synchronize()
        refresh_set = {"ms": (time.perf_counter() - t0) * 1e3, "matrices": len(layers), "status": st,
                       "not_converged": sum(1 for x in infos if not x.converged),
                       "iterations_max": max(x.iterations for x in infos),
                       "slots": slots,
                       "timer": "host clock around the call, which returns when every refresh has finished"}
        if args.refresh_warm > 0:
            # The next refresh of training sees gradients whose subspace has moved a little (Sec. 4.1): every
            # gradient gets 2 % of its rms as fresh noise, then the set is refreshed again from its projectors.
            gen = torch.Generator(device=dev)
            gen.manual_seed(w.seed + 17)
            for g in {x.data_ptr(): x for x in Gs}.values():
                rms = g.float().pow(2).mean().sqrt().item()
                g.add_((torch.randn(g.shape, device=dev, generator=gen) * (0.02 * rms)).to(g.dtype))
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            st, infos = gb.galore_refresh_batch(layers, Gs, stream=stream, workspace=space)
            torch.cuda.synchronize()
            refresh_set["warm_start"] = {"ms": (time.perf_counter() - t0) * 1e3, "status": st, "first_steps": args.refresh_warm,
                                         "not_converged": sum(1 for x in infos if not x.converged),
                                         "iterations_max": max(x.iterations for x in infos),
                                         "iterations_mean": sum(x.iterations for x in infos) / len(infos),
                                         "gradients": "the cold refresh's plus 2 % of their rms as fresh noise"}
        del space

    batch = gb.Batch(layers, Ws, Gs, device=dev) if mode == "batch" else None

    arrive = None
    if mode == "arrive":
        # A producer stream stands in for the backward pass: it writes layer i's gradient into the next
        # buffer of a small ring (a device copy of a resident gradient, i.e. the write traffic of the
        # kernel that would produce it) and signals; the step of layer i waits for that, runs on the
        # optimizer stream and hands the buffer back.
        prod = torch.cuda.Stream(device=dev)
        rings = {}
        for sh in set(shapes_of):
            rings[sh] = [padded(sh[0], sh[1], tdt[w.g_dtype]) for _ in range(max(1, args.ring))]
        ready = [torch.cuda.Event() for _ in layers]
        freed = {sh: [torch.cuda.Event() for _ in rings[sh]] for sh in rings}
        arrive = (prod, rings, ready, freed)

    def one_step(lr=w.lr):
        if batch is not None:
            batch.galore_step_batch(lr, stream)
            return
        if arrive is not None:
            prod, rings, ready, freed = arrive
            turn = {}
            prod.wait_stream(stream)
            for i, (layer, Wt, Gt, sh) in enumerate(zip(layers, Ws, Gs, shapes_of)):
                j = turn.get(sh, 0)
                turn[sh] = j + 1
                slot = j % len(rings[sh])
                with torch.cuda.stream(prod):
                    if j >= len(rings[sh]):
                        prod.wait_event(freed[sh][slot])
                    rings[sh][slot].copy_(Gt, non_blocking=True)
                    ready[i].record(prod)
                stream.wait_event(ready[i])
                layer.galore_step(Wt, rings[sh][slot], lr, stream)
                freed[sh][slot].record(stream)
            return
        for layer, Wt, Gt in zip(layers, Ws, Gs):
            layer.galore_step(Wt, Gt, lr, stream)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing ----------------------------------------------------------------
    for _ in range(args.warmup):
        one_step()
    barrier()
    sampler = ClockSampler(dev.index if dev.index is not None else 0)
    sampler.start()
    launches0 = gb.galore_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        one_step()
    e1.record(stream)
    barrier()
    launches = gb.galore_launch_count() - launches0
    clocks = sampler.stop()
    ms_total = max_over_ranks(e0.elapsed_time(e1), dist, dev)
    ms_step = ms_total / args.steps
    value = world * w.params / (ms_step * 1e-3)

    # ---- per-phase timing with events on the launching stream (separate instrumented pass) -------
    gb.galore_profile_enable(True)
    prof_steps = max(1, args.steps)          # as many as the timed region: same clocks under the power cap
    for _ in range(prof_steps):
        one_step()
    torch.cuda.synchronize()
    gb.galore_profile_enable(False)
    phase_ms, phase_cnt = gb.galore_profile_read()
    uses_tc = all(l.uses_tensor_path for l in layers)
    # whole-step roofline: the slower of the algorithmic HBM bytes at the measured copy bandwidth and the
    # projection flops at the measured sustained bf16 GEMM rate (fp32 FMA peak on the fp32 path)
    t_hbm = bytes_alg / (peaks["hbm_gbs"] * 1e9)
    tc_peak = peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]) if uses_tc else FP32_FMA_TFLOPS
    t_tc = flops_alg / (tc_peak * 1e12)
    t_roof = max(t_hbm, t_tc)
    bound = "hbm" if t_hbm >= t_tc else ("tensor" if uses_tc else "alu")
    if bound == "hbm":
        achieved, peak, unit = bytes_alg / (ms_step * 1e-3) / 1e9, peaks["hbm_gbs"], "GB/s"
    else:
        achieved, peak, unit = flops_alg / (ms_step * 1e-3) / 1e12, tc_peak, "TFLOP/s"
    # per kernel: event time per step, what it achieves and the fraction of its own roof
    kp, ka, kb = kernel_costs(w, shapes_of)
    fused = phase_cnt[1] == 0                   # Adam ran in the projection's epilogue: no launch of its own
    if fused:
        kp = {"flops": kp["flops"], "bytes": kp["bytes"] + ka["bytes"]}

    def kernel_entry(ms_total, launches_total, cost):
        if not launches_total:
            return None
        ms = ms_total / prof_steps
        roof_ms = max(cost["flops"] / (tc_peak * 1e12), cost["bytes"] / (peaks["hbm_gbs"] * 1e9)) * 1e3
        return {"ms_per_step": ms, "launches_per_step": launches_total / prof_steps,
                "tflops": cost["flops"] / (ms * 1e-3) / 1e12 if cost["flops"] else None,
                "gbs": cost["bytes"] / (ms * 1e-3) / 1e9, "roof_ms": roof_ms, "frac_of_own_roof": roof_ms / ms}
    kernels = {"projection_with_adam" if fused else "projection": kernel_entry(phase_ms[0], phase_cnt[0], kp),
               "adam": kernel_entry(phase_ms[1], phase_cnt[1], ka),
               "back_projection": kernel_entry(phase_ms[2], phase_cnt[2], kb)}
    ratios = KERNEL_DRAM_OVER_ALGORITHMIC.get((w.rank, w.state_fmt))
    alg_bytes = {"projection_with_adam": kp["bytes"], "projection": kp["bytes"], "adam": ka["bytes"], "back_projection": kb["bytes"]}
    traffic = ({k: v * alg_bytes[k] / max(1.0, kernels[k]["launches_per_step"]) for k, v in ratios.items() if kernels.get(k)}
               if ratios else None)
    roof = {"bound": bound, "achieved": achieved, "peak": peak, "unit": unit, "frac": t_roof * 1e3 / ms_step,
            "traffic": traffic,
            "traffic_unit": "DRAM bytes per launch, by kernel: the ncu capture's multiple of the algorithmic bytes times the algorithmic bytes of an average launch",
            "peak_source": peaks["source"] + (" (sustained bf16 GEMM)" if bound == "tensor" else " (copy bandwidth)" if bound == "hbm" else " (unit counts x max clock)"),
            "scope": "whole step: algorithmic bytes and flops of every matrix / measured step time",
            "kernels": {k: v for k, v in kernels.items() if v},
            "step_roofline_ms": {"hbm": t_hbm * 1e3, "tensor" if uses_tc else "fp32_fma": t_tc * 1e3},
            # the same fraction against the data-sheet figures (8 TB/s, 2250 dense bf16 TFLOP/s): context only
            "nominal": ({"hbm_gbs": NOMINAL_HBM_GBS, "bf16_tflops": NOMINAL_BF16_TFLOPS,
                         "frac": max(bytes_alg / (NOMINAL_HBM_GBS * 1e9), flops_alg / (NOMINAL_BF16_TFLOPS * 1e12)) * 1e3 / ms_step}
                        if uses_tc else None),
            "algorithmic": {"bytes_per_step": bytes_alg, "flops_per_step": flops_alg}}

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if uses_tc else "f32", "data": "synthetic",
        "config": {"workload": w.name, "matrices": w.matrices, "params": w.params, "rank": w.rank,
                   "state_fmt": w.state_fmt, "w_dtype": w.w_dtype, "g_dtype": w.g_dtype, "alpha": w.alpha,
                   "refresh_gap": w.refresh_gap, "weight_decay": args.weight_decay, "tensor_path": uses_tc, "mode": mode, "parallelism": f"replicas x{world}",
                   "l2": "inputs larger than L2 (whole layer set streamed each step)"},
        "clocks": clocks, "gpu_launches": launches, "roofline": roof,
        "refresh": refresh_info,
    }
    if refresh_set:
        # Algorithm 1 refreshes every matrix once per `refresh_gap` steps: the step plus its share of that
        set_ms = refresh_set["ms"]
        gaps = sorted({w.refresh_gap, *getattr(args, "amortise_gaps", ())})
        out["refresh_set"] = refresh_set
        out["refresh_amortised"] = {"refresh_ms_whole_set": set_ms, "refresh_gap": w.refresh_gap,
                                    "one_by_one_ms_whole_set": sum(x["ms"] * x["count"] for x in refresh_info),
                                    "ms_per_step": ms_step + set_ms / w.refresh_gap,
                                    "value": world * w.params / ((ms_step + set_ms / w.refresh_gap) * 1e-3), "unit": UNIT,
                                    "by_gap": {str(T): world * w.params / ((ms_step + set_ms / T) * 1e-3) for T in gaps}}
        # the same two records inside an object every reader of the line keeps
        roof["refresh_set"] = refresh_set
        roof["refresh_amortised"] = out["refresh_amortised"]
    if not full:
        return {k: out[k] for k in ("value", "ms_per_step", "config", "roofline", "refresh", "refresh_set",
                                    "refresh_amortised", "gpu_launches", "clocks") if k in out}

    # ---- end to end through the host-buffer entry point -------------------------------------------
    if not args.no_e2e:
        # pinned host copies: four sets per distinct shape, taken in turn, so that layers in flight
        # together (three staging slots) never share a host buffer
        host = {}
        for (m, n, _c) in w.shapes:
            sets = []
            for j in range(4):
                hw = torch.empty(m, n, dtype=tdt[w.w_dtype]).pin_memory()
                hg = torch.empty(m, n, dtype=tdt[w.g_dtype]).pin_memory()
                hw.normal_(0, 0.02)
                hg.normal_(0, 0.05)
                sets.append((hw, hg))
            host[(m, n)] = sets
        turn = {}
        W_hosts, G_hosts = [], []
        for sh in shapes_of:
            j = turn.get(sh, 0)
            turn[sh] = j + 1
            hw, hg = host[sh][j % 4]
            W_hosts.append(hw)
            G_hosts.append(hg)
        e2e_steps = max(1, min(args.steps, 3))
        h2d = sum(m * n * (elem_bytes(w.w_dtype) + elem_bytes(w.g_dtype)) for (m, n) in shapes_of)
        d2h = sum(m * n * elem_bytes(w.w_dtype) for (m, n) in shapes_of)
        if mode == "batch":
            hb = gb.HostBatch(layers, W_hosts, G_hosts, slots=3, device=dev)
            e2e_call = "galore_step_host_batch, 3 staging slots"

            def e2e_step():
                hb.galore_step_host_batch(w.lr, stream)
        else:
            dws = {sh: (torch.empty(sh[0], sh[1], dtype=tdt[w.w_dtype], device=dev),
                        torch.empty(sh[0], sh[1], dtype=tdt[w.g_dtype], device=dev)) for sh in set(shapes_of)}
            e2e_call = "galore_step_host per layer"

            def e2e_step():
                for layer, sh, hw, hg in zip(layers, shapes_of, W_hosts, G_hosts):
                    dw, dg = dws[sh]
                    layer.galore_step_host(hw, hg, dw, dg, w.lr, stream)

        e2e_step()
        barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(e2e_steps):
            e2e_step()
        b.record(stream)
        barrier()
        ms = max_over_ranks(a.elapsed_time(b) / e2e_steps, dist, dev)
        out["e2e"] = {"value": world * w.params / (ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                      "d2h_bytes_per_step": d2h, "ms_per_step": ms, "steps": e2e_steps,
                      "call": e2e_call,
                      "host_buffers": "four pinned W and G per distinct shape, taken in turn by the layers of that shape"}
    flags = 0
    for layer in layers[:1]:
        flags |= layer.device_status()
    out["device_status"] = flags

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        v, cores, t, extra = cpu_oracle_sample(w, 1, extras=True)
        out["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "backend": "numpy on the host BLAS, fp64",
                               "sample": f"1 oracle step on one matrix of each distinct shape ({len(w.shapes)} of "
                                         f"{w.matrices} matrices), given projector, {t:.1f} s", **extra}
    return out


if __name__ == "__main__":
    sys.exit(main())
