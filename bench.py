#!/usr/bin/env python
"""Benchmark of the AdaPM optimizer step (one step = one adapm_step over every block of a parameter set).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload gpt2_1p5b] [--v-mode blockmean]
  python bench.py --impl reference ...      # times the fp64 CPU oracle instead (a deliberately slow baseline)

Prints ONE JSON line (rank 0).  `value` = optimizer steps per second with every input resident in HBM,
timed with CUDA events over exactly K steps; `e2e` = the same with the step's gradients copied from pinned
host memory and the updated parameters copied back inside the timed region.  With N > 1 the N ranks run
independent replicas of the same set (the step has no cross-GPU exchange); value = all ranks' steps / max time.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

METRIC = "adapm_optimizer_steps_per_sec"
UNIT = "steps/s"
SM_COUNT, FMA_LANES = 148, 128


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                "sm_max_mhz": float(d.get("sm_max_mhz", 1965.0)), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "sm_max_mhz": 1965.0,
            "source": "fallback"}


TRAFFIC_FILE = os.path.join(ROOT, "profiles", "dram_traffic_per_launch.md")
KERNEL_SOURCES = ("tc_engine.cuh", "tc_apply.cuh", "tc_common.cuh", "lowrank_tc.cu", "stream_kernels.cu")


def kernel_source_digest() -> str:
    """Short hash of the kernel sources: a traffic figure is only quoted while the kernels are the ones captured."""
    import hashlib
    h = hashlib.sha256()
    for f in KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_2510_09103_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:12]


def recorded_traffic(kind: str, workload: str, v_mode: str):
    """DRAM bytes per launch (ncu dram__bytes_read.sum + dram__bytes_write.sum) from the table under profiles/:
    rows `| kernel | workload | v_mode | bytes per launch | capture | scale | kernel sources |`.  Returns
    (bytes, note) or (None, why): a row taken from other kernel sources than the present ones does not count."""
    if not os.path.exists(TRAFFIC_FILE):
        return None, "no capture recorded"
    digest = kernel_source_digest()
    stale = False
    for line in open(TRAFFIC_FILE):
        cells = [c.strip() for c in line.strip().strip("|").split("|")]
        if len(cells) < 7 or cells[0] != kind or cells[1] != workload or cells[2] != v_mode:
            continue
        if cells[6] != digest:
            stale = True
            continue
        return float(cells[3]), f"{cells[4]}, scaled x{cells[5]}, kernel sources {cells[6]}"
    return None, "kernels changed since the last capture" if stale else "no capture recorded"


# ------------------------------------------------------------------------------------------------ oracle arm

def _oracle_hparams(w):
    from oracle import adapm_oracle as O
    return O.HParams(lr=w.lr, beta1=w.beta1, beta2=w.beta2, eps=w.eps)


class OracleSet:
    """Every block of a parameter set in the oracle.  Blocks of equal shape share one W and one g array (the
    oracle's time does not depend on the values); every block has its own optimizer state."""

    def __init__(self, w, blocks, only=None):
        from oracle import adapm_oracle as O
        import workloads as WL
        self.O, self.w = O, w
        self.hp = _oracle_hparams(w)
        self.ids = list(range(len(blocks))) if only is None else list(only)
        rng = np.random.default_rng(0)
        self.arrays, self.items = {}, []
        for i in self.ids:
            b = blocks[i]
            key = (b.rows, b.cols)
            if key not in self.arrays:
                W = rng.standard_normal((b.rows, b.cols)) * 0.02
                g, _ = WL.to_grad_dtype((rng.standard_normal((b.rows, b.cols), dtype=np.float32) * np.float32(1e-3)),
                                        w.grad_dtype)
                self.arrays[key] = (W, g.astype(np.float64))
            ob = O.Block(b.rows, b.cols, b.mom_mode, b.rank, b.v_mode, b.v_group_rows, b.lr_scale, b.weight_decay)
            L0 = None
            if b.mom_mode == O.MOM_LOWRANK:
                L0 = np.linalg.qr(rng.standard_normal((b.rows, b.rank)))[0]      # orthonormal columns, cheaply
            self.items.append((key, ob, O.new_state(ob, L0)))
        self.t = 0
        self.elems = sum(b.rows * b.cols for b in (blocks[i] for i in self.ids))

    def step(self) -> float:
        """One oracle step over the blocks; returns seconds."""
        self.t += 1
        t0 = time.perf_counter()
        for key, ob, st in self.items:
            W, g = self.arrays[key]
            self.O.block_step(W, g, st, ob, self.hp, self.t)
        return time.perf_counter() - t0


def oracle_layer_sample(w, blocks, budget_s: float = 25.0):
    """The bounded CPU sample of the default run: the blocks of the first transformer layer (all of them, full size)
    and the small leading tensors, stepped once with every BLAS thread and once with one thread; the set's time
    is that of the layer times the layer count plus the embeddings' share by element count.
    Returns (estimated seconds per full step all threads, the same for one thread or None, description)."""
    from threadpoolctl import threadpool_limits
    names = [t.name for t in w.tensors]
    layer_tags = sorted({n.split(".")[0] + "." + n.split(".")[1] if n.startswith("layers.") else n.split(".")[0]
                         for n in names if n.startswith(("h", "layers.")) and "." in n})
    first = layer_tags[0] if layer_tags else None
    n_layers = max(len(layer_tags), 1)
    # tensor index -> block indices (a fused QKV tensor is three blocks)
    t2b, k = [], 0
    for t in w.tensors:
        nb = 3 if t.role == 4 else 1
        t2b.append(list(range(k, k + nb))); k += nb
    in_layer = [i for ti, t in enumerate(w.tensors) if first and t.name.startswith(first + ".") for i in t2b[ti]]
    outside = [i for ti, t in enumerate(w.tensors) if not t.name.startswith(("h", "layers.")) or "." not in t.name
               for i in t2b[ti]]
    small_out = [i for i in outside if blocks[i].rows * blocks[i].cols <= 8_000_000]
    big_out = [i for i in outside if i not in small_out]
    sample = OracleSet(w, blocks, in_layer + small_out)
    layer_elems = sum(blocks[i].rows * blocks[i].cols for i in in_layer)
    small_elems = sum(blocks[i].rows * blocks[i].cols for i in small_out)
    big_elems = sum(blocks[i].rows * blocks[i].cols for i in big_out)
    t_all = sample.step()
    # blocks without low-rank factors cost per element what the sampled ones of that kind cost: use the sample's
    # elementwise share, measured on the small outside tensors when there are any
    per_elem = None
    if small_out:
        so = OracleSet(w, blocks, small_out)
        per_elem = so.step() / max(small_elems, 1)
    def scale(t_sample):
        t_small = (per_elem or 0.0) * small_elems
        t_layer = max(t_sample - t_small, 0.0)
        return t_layer * n_layers + t_small + (per_elem or t_sample / max(sample.elems, 1)) * big_elems
    est_all = scale(t_all)
    est_one = None
    if t_all * 12 < budget_s:
        with threadpool_limits(limits=1):
            t_one = sample.step()
        est_one = scale(t_one)
    desc = (f"every block of the first of {n_layers} layers at full size plus the small leading tensors "
            f"({sample.elems} of {sum(b.rows * b.cols for b in blocks)} elements), one oracle step; layer time x "
            f"{n_layers}, embeddings by element count")
    return est_all, est_one, desc


def _blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        return max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        return 1


def run_reference(args) -> None:
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import workloads as WL
    from oracle import planner_oracle as P
    w = WL.get_workload(args.workload)
    blocks = P.plan(w.tensors, w.weight_decay, w.rank_pct, args.v_mode == "blockmean")
    # Full oracle steps over every block of the set, timed one by one.  A step of the 1.5B-shaped set takes the
    # better part of a minute on 16 cores, so the run stops asking for more once `budget_s` is spent: `steps` is
    # the number of steps that were timed, `steps_requested` what the command line asked for.  The oracle has
    # nothing to warm up beyond its first call, which is timed like the rest and reported.
    budget_s = float(os.environ.get("ADAPM_REFERENCE_BUDGET_S", "150"))
    t_setup = time.perf_counter()
    oset = OracleSet(w, blocks)
    setup_s = time.perf_counter() - t_setup
    times = []
    while len(times) < max(args.steps, 1):
        times.append(oset.step())
        if sum(times) + times[-1] > budget_s:
            break
    sec = float(np.mean(times))
    val = 1.0 / sec
    cores = _blas_threads()
    desc = (f"{len(times)} full oracle step(s) over all {len(blocks)} blocks ({oset.elems} elements), numpy fp64, "
            f"BLAS on {cores} threads, blocks one after another; {setup_s:.0f} s of untimed setup")
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": len(times),
        "steps_requested": args.steps, "warmup": 0, "ms_per_step": sec * 1e3, "step_seconds": times,
        "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "params": w.numel, "v_mode": args.v_mode, "grad_dtype": w.grad_dtype},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "cores_os": os.cpu_count(), "kind": "oracle",
                         "sample": desc},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------ GPU arm

def whole_job_value(ms_local: float, steps: int, dist=None, device=None):
    """(slowest rank's milliseconds, steps per second of the whole job).

    The ranks run independent replicas of the same parameter set (the optimizer step has no exchange
    between GPUs), so the job's throughput is all ranks' steps over the slowest rank's time.
    `dist` is an initialised torch.distributed module or None for a single process.
    """
    world = 1
    ms = float(ms_local)
    if dist is not None:
        import torch
        world = dist.get_world_size()
        t = torch.tensor([ms], dtype=torch.float64, device=device if device is not None else "cpu")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())
    return ms, world * steps / (ms * 1e-3)


class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid: str):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", uuid, f"--query-gpu={self.FIELDS}",
                                       "--format=csv,noheader,nounits", "-lms", "100"], stdout=self.f,
                                      stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self) -> dict:
        if self.p is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush()
        rows = [l.strip().split(", ") for l in open(self.f.name) if l.strip()]
        os.unlink(self.f.name)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except Exception:
                continue
            for n, v in zip(names, r[4:8]):
                if v.strip().lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "reasons": sorted(reasons),
                "samples": len(sm)}


def kernel_algorithmic_work(kind: str, blocks, gsz: int, k_eff: int):
    """(bound, amount, unit) of one launch of `kind`: bytes for HBM-bound kernels, flops for the others."""
    import paper_2510_09103_b200 as A
    nb = lambda b: b.rows * b.cols
    groups = lambda b: nb(b) if b.v_mode == A.V_ELEMENT else (1 if b.v_group_rows == 0 else b.rows // b.v_group_rows)
    lowr = [b for b in blocks if b.mom_mode == A.MOM_LOWRANK]
    if kind == "stream_update":
        tot = 0
        for b in blocks:
            if b.mom_mode == A.MOM_LOWRANK:
                continue
            tot += nb(b) * (gsz + 8 + (8 if b.mom_mode == A.MOM_FULL else 0)) + groups(b) * 8
        return "hbm", tot, "bytes"
    if kind in ("apply_simt", "tc_apply"):
        # g + W in, W out, plus the factors once; flops of the rank-2r product reported separately
        tot = sum(nb(b) * (gsz + 8) + groups(b) * (8 if b.v_mode == A.V_ELEMENT else 4)
                  + 2 * 4 * b.rank * (b.rows + b.cols) for b in lowr)
        return "hbm", tot, "bytes"
    if kind == "gemm_simt":
        # averaged over the 4 GEMM launches of one refit pass: (4 m n r + 8 r^2 (m + n)) / 4
        fl = sum(4.0 * nb(b) * b.rank + 8.0 * b.rank * b.rank * (b.rows + b.cols) for b in lowr) / 4.0
        return "alu", fl, "flops"
    if kind == "tc_panel":
        # One refit pass is a contraction: g R^T and L^T g, 4 m n r flops per block (the doubling by the hi/lo
        # operand split and the small r x r products are the kernel's own and not counted).
        fl = sum(4.0 * nb(b) * b.rank for b in lowr)
        return "tensor", fl, "flops"
    if kind == "tc_panel_hbm":
        # The same launch seen from memory, the method's bytes only: g once, the fp32 factors read and written
        # (the split-bf16 copies are the kernel's own traffic and show up in `traffic`, not here).
        tot = sum(nb(b) * gsz + 8 * b.rank * (b.rows + b.cols) for b in lowr)
        return "hbm", tot, "bytes"
    if kind == "tc_gram":
        fl = sum(4.0 * b.rank * b.rank * (b.rows + b.cols) for b in lowr)
        return "tensor", fl, "flops"
    if kind == "tc_convert":
        tot = sum(b.rank * (b.rows + b.cols) * (4 + 4) for b in lowr)
        return "hbm", tot, "bytes"
    if kind in ("reduce_partial",):
        return "hbm", sum(nb(b) * gsz for b in lowr), "bytes"
    if kind == "reduce_rows":
        return "hbm", sum(b.rows * 4 + groups(b) * 8 for b in lowr), "bytes"
    return "hbm", 0, "bytes"


def run_gpu(args) -> None:
    import torch
    import workloads as WL
    import paper_2510_09103_b200 as A

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the optimizer step has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    w = WL.get_workload(args.workload)
    blockmean = args.v_mode == "blockmean"
    blocks, total = A.adapm_plan_default(w.tensors, w.rank_pct, w.rank_override,
                                         A.V_BLOCKMEAN if blockmean else A.V_ELEMENT, w.weight_decay)
    gd = A.GRAD_BF16 if w.grad_dtype == "bf16" else A.GRAD_F32
    gsz = 2 if w.grad_dtype == "bf16" else 4
    path = {"auto": A.PATH_AUTO, "simt": A.PATH_SIMT, "tensor": A.PATH_TENSOR}[args.path]
    flags = ((A.FLAG_NO_PANEL_TEAMS if args.teams == "off" else 0) | (A.FLAG_FORCE_PANEL_TEAMS if args.teams == "force" else 0)
             | (A.FLAG_NO_SUMSQ_FOLD if args.no_fold else 0))
    hp = A.hparams(lr=w.lr, beta1=w.beta1, beta2=w.beta2, eps=w.eps, grad_dtype=gd, lowrank_path=path, flags=flags,
                   tune_panels=args.panels, tune_stage_k=args.stage_k, max_grad_norm=args.max_grad_norm,
                   refresh_period=args.refresh_period, inner_precond=1 if args.precond else 0)
    ctx = A.adapm_create(blocks, hp)

    # synthetic inputs: parameters N(0, 0.02^2) drawn on the device; gradients tiled from a seeded host pool
    gen = torch.Generator(device=dev); gen.manual_seed(1)
    params = torch.empty(total, dtype=torch.float32, device=dev).normal_(0.0, 0.02, generator=gen)
    pool = WL.GradPool(w, pool_elems=1 << 24)
    raw = pool.raw.view(np.int16) if w.grad_dtype == "bf16" else pool.raw
    tdt = torch.int16 if w.grad_dtype == "bf16" else torch.float32
    pool_t = torch.from_numpy(raw)
    # sets beyond 2e9 parameters: no end-to-end leg (48+ GB of pinned host memory) and the gradients are tiled on
    # the device
    if total > 2_000_000_000:
        args.no_e2e = True
    grads = torch.empty(total, dtype=torch.bfloat16 if w.grad_dtype == "bf16" else torch.float32, device=dev)
    grads_host = None
    if args.no_e2e:
        pool_d = pool_t.to(dev)
        gv = grads.view(tdt)
        for i in range(0, total, pool_d.numel()):
            n = min(pool_d.numel(), total - i)
            gv[i:i + n].copy_(pool_d[:n])
        del pool_d
    else:
        grads_host = torch.empty(total, dtype=tdt, pin_memory=True)
        reps = -(-total // pool_t.numel())
        grads_host.copy_(pool_t.repeat(reps)[:total])
        grads.view(tdt).copy_(grads_host)
    shadow = None
    if args.shadow:
        shadow = torch.zeros(total, dtype=torch.bfloat16, device=dev)
        ctx.adapm_set_shadow_params(shadow)
    state = torch.zeros(ctx.adapm_state_bytes() // 4, dtype=torch.float32, device=dev)
    work = torch.zeros(max(ctx.adapm_workspace_bytes() // 4, 64), dtype=torch.float32, device=dev)
    ctx.adapm_set_workspace(work)
    ctx.adapm_state_init(state)
    torch.cuda.synchronize()

    t = 0

    def do_steps(n):
        nonlocal t
        for _ in range(n):
            t += 1
            ctx.adapm_step(params, grads, state, t)

    # ---- device-resident timing ----
    do_steps(args.warmup)
    uuid = str(torch.cuda.get_device_properties(dev).uuid)
    uuid = uuid if uuid.startswith("GPU-") else "GPU-" + uuid
    sampler = ClockSampler(uuid) if rank == 0 else None
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    launches_timed = 0
    for _ in range(args.steps):
        do_steps(1)
        launches_timed += ctx.adapm_launch_count()
    e1.record()
    barrier()
    ms_total, value = whole_job_value(e0.elapsed_time(e1), args.steps, dist, dev)
    clocks = sampler.stop() if sampler else None
    status = ctx.adapm_get_status()
    if status != 0:
        raise SystemExit(f"device status word {status}: a bounded wait expired; numbers are invalid")
    ms_step = ms_total / args.steps

    # ---- per-kernel durations (separate profiled pass; CUDA events on the launching stream) ----
    per_kind = {}
    ctx.adapm_set_profiling(True)
    for _ in range(args.steps):
        do_steps(1)
        for kind, ms in ctx.adapm_get_launch_times():
            d = per_kind.setdefault(kind, [0, 0.0])
            d[0] += 1; d[1] += ms
    ctx.adapm_set_profiling(False)
    tot_ms = sum(v[1] for v in per_kind.values()) or 1.0
    kernels = {k: {"launches_per_step": v[0] / args.steps, "ms_per_step": v[1] / args.steps, "share": v[1] / tot_ms}
               for k, v in per_kind.items()}

    # ---- end to end: host gradients in, updated parameters out, inside the timed region ----
    e2e = None
    if not args.no_e2e:
        # As a training loop would drive the library: the gradients of step i + 1 go up (a second device buffer, a
        # copy stream) while step i runs and its parameters come down (another copy stream); PCIe is full duplex.
        # Every step's gradients still come from pinned host memory and every step's parameters still land there,
        # all inside the timed region.
        params_host = torch.empty(total, dtype=torch.float32, pin_memory=True)
        gbuf = [grads, torch.empty_like(grads)]
        up, down, cur = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.current_stream()
        ev_up = [torch.cuda.Event(), torch.cuda.Event()]
        ev_step = [torch.cuda.Event(), torch.cuda.Event()]
        ev_down = torch.cuda.Event()

        def e2e_step(i):
            nonlocal t
            b = i & 1
            with torch.cuda.stream(up):
                up.wait_event(ev_step[b])            # the step that last read this buffer is done with it
                gbuf[b].view(tdt).copy_(grads_host, non_blocking=True)
                ev_up[b].record(up)
            cur.wait_event(ev_up[b])
            cur.wait_event(ev_down)                  # the previous parameters are on the host before they change
            t += 1
            ctx.adapm_step(params, gbuf[b], state, t)
            ev_step[b].record(cur)
            with torch.cuda.stream(down):
                down.wait_event(ev_step[b])
                params_host.copy_(params, non_blocking=True)
                ev_down.record(down)

        for i in range(2):
            e2e_step(i)
        cur.wait_event(ev_down)
        barrier()
        e0.record()
        for i in range(args.steps):
            e2e_step(i)
        cur.wait_event(ev_down)
        e1.record()
        barrier()
        ms_e2e, value_e2e = whole_job_value(e0.elapsed_time(e1), args.steps, dist, dev)
        e2e = {"value": value_e2e, "unit": UNIT, "h2d_bytes_per_step": total * gsz,
               "d2h_bytes_per_step": total * 4, "ms_per_step": ms_e2e / args.steps,
               "overlap": "upload of the next step's gradients runs beside this step and the download of its parameters"}

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peaks = _peaks()
    k_eff = 4
    step_bytes = ctx.adapm_step_bytes()
    dom = max(kernels, key=lambda k: kernels[k]["share"]) if kernels else "stream_update"

    def roofline_of(kind, work=None):
        if kind not in kernels or kernels[kind]["launches_per_step"] == 0:
            return None
        bound, amount, _ = kernel_algorithmic_work(work or kind, blocks, gsz, k_eff)
        sec = kernels[kind]["ms_per_step"] / kernels[kind]["launches_per_step"] * 1e-3
        if bound == "hbm":
            ach, peak, unit = amount / sec / 1e9, peaks["hbm_gbs"], "GB/s"
        elif bound == "tensor":
            ach, peak, unit = amount / sec / 1e12, peaks["bf16_tflops_sustained"], "TFLOP/s"
        else:
            ach, peak, unit = amount / sec / 1e12, SM_COUNT * FMA_LANES * 2 * peaks["sm_max_mhz"] * 1e6 / 1e12, "TFLOP/s"
        traffic, note = recorded_traffic(kind, w.name, args.v_mode)
        return {"kernel": kind, "bound": bound, "achieved": ach, "peak": peak, "unit": unit, "frac": ach / peak,
                "traffic": traffic, "traffic_source": note, "peak_source": peaks["source"],
                "per_launch_ms": sec * 1e3, "algorithmic_per_launch": amount}

    cpu_all, cpu_one, cpu_desc = (float("nan"), None, "skipped (--no-cpu)") if args.no_cpu else oracle_layer_sample(w, blocks)
    sb = ctx.adapm_state_breakdown()
    state_bytes = sum(sb.values())
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": w.name, "params": w.numel, "blocks": len(blocks), "v_mode": args.v_mode,
                   "max_grad_norm": args.max_grad_norm, "refresh_period": args.refresh_period, "bf16_shadow": args.shadow,
                   "inner_precond": bool(args.precond),
                   "grad_dtype": w.grad_dtype, "state_dtype": "f32", "lowrank_path": args.path,
                   "lowrank_kernels": "tensor" if any(k.startswith("tc_") for k in kernels) else "simt",
                   "parallelism": f"replicas x{world}" if world > 1 else "single GPU",
                   "l2": "inputs larger than L2 (no flush between steps)"},
        "params_per_s": value * w.numel,
        "step_bytes": step_bytes, "step_gbs": step_bytes / (ms_step * 1e-3) / 1e9,
        "step_hbm_frac_of_measured": step_bytes / (ms_step * 1e-3) / 1e9 / peaks["hbm_gbs"],
        "step_hbm_frac_of_8tbs": step_bytes / (ms_step * 1e-3) / 1e9 / 8000.0,
        "step_contraction_tflops": ctx.adapm_step_flops() / (ms_step * 1e-3) / 1e12,
        "state_bytes": state_bytes, "state_breakdown": sb, "adamw_state_bytes": 8 * w.numel,
        "state_saving_vs_adamw": 1.0 - state_bytes / (8.0 * w.numel),
        "gpu_launches": launches_timed,
        "launches_per_step": ctx.adapm_launch_count(),
        "kernels": kernels,
        "roofline": roofline_of(dom),
        "roofline_stream_update": roofline_of("stream_update"),
        "roofline_tc_apply": roofline_of("tc_apply"),
        "roofline_tc_panel_hbm": roofline_of("tc_panel", "tc_panel_hbm"),
        "clocks": clocks,
        "e2e": e2e,
        "cpu_baseline": {"value": 1.0 / cpu_all, "unit": UNIT, "cores": _blas_threads(), "cores_os": os.cpu_count(),
                         "kind": "oracle", "sample": cpu_desc, "est_s_per_step": cpu_all,
                         "one_thread_est_s_per_step": cpu_one},
    }
    print(json.dumps(line))
    ctx.adapm_destroy()
    if dist is not None:
        dist.destroy_process_group()


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="gpt2_1p5b")
    ap.add_argument("--v-mode", default="blockmean", choices=["blockmean", "element"])
    ap.add_argument("--path", default="auto", choices=["auto", "simt", "tensor"])
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle sample (kernel sweeps)")
    ap.add_argument("--panels", type=int, default=0, help="tensor path: panels per refit item (0 = automatic)")
    ap.add_argument("--stage-k", type=int, default=0, help="tensor path: K per stage, 64 or 128 (0 = automatic)")
    ap.add_argument("--teams", default="auto", choices=["auto", "off", "force"], help="panel team schedule")
    ap.add_argument("--no-fold", action="store_true", help="row sums of g^2 from a pass of their own")
    ap.add_argument("--max-grad-norm", type=float, default=0.0, help="global gradient-norm clipping threshold (0 = off)")
    ap.add_argument("--precond", action="store_true",
                    help="preconditioned refit passes (a variant that is not in the paper)")
    ap.add_argument("--refresh-period", type=int, default=0, help="T: refit both factors every T steps (0/1 = every step)")
    ap.add_argument("--shadow", action="store_true", help="also write the bf16 copy of the parameters")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
