#!/usr/bin/env python
"""Benchmark of the EntropyInfer sparse prefill path on B200.

One "step" = one attention layer of the whole hot path (ei_plan: pool, observe, budget, select;
then ei_sparse_prefill) on a seeded synthetic workload already resident in HBM.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

Prints ONE JSON line (rank 0).  With --gpus N > 1 (launched by torchrun) every rank runs an
independent replica of the layer on its own GPU ("replicas only": the path has no exchange step).
--impl reference times the CPU oracle on the host cores instead (bounded sample per step).
"""
import argparse
import json
import math
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import synth  # noqa: E402

METRIC = "128k-token sparse prefill attention ms/layer; tensor-pipe % of B200 peak"
UNIT = "ms/layer"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
NOMINAL_BF16_TFLOPS = 2250.0
NOMINAL_HBM_GBS = 8000.0
NCU_COUNTERS = os.path.join(ROOT, "profiles", "ncu_counters_attention.txt")
KERNEL_SOURCES = {"sparse_attention_quad_kernel": "ei_attention_quad.cu", "sparse_attention_quad_persistent_kernel": "ei_attention_quad.cu",
                  "sparse_attention_quad1_kernel": "ei_attention_quad.cu", "sparse_attention_split_kernel": "ei_attention.cu",
                  "sparse_attention_persistent_kernel": "ei_attention.cu", "sparse_attention_pair_kernel": "ei_attention.cu",
                  "sparse_attention_kernel": "ei_attention.cu", "sparse_attention_tri_kernel": "ei_attention_tri.cu"}


def git_blob_hash(path: str) -> str:
    """What `git hash-object` prints for the file (sha1 of "blob <size>\\0" + contents); no git needed."""
    import hashlib
    with open(path, "rb") as f:
        data = f.read()
    return hashlib.sha1(b"blob %d\0" % len(data) + data).hexdigest()


def ncu_counters(workload: str, fraction: float, kernel: str, no_skip: bool):
    """Counters of one ncu capture of this command, from the tracked table profiles/ncu_counters_attention.txt
    (one row per capture: workload, fraction, kernel, shortcut on/off, the kernel source's git blob hash at
    capture time, tensor-pipe-active %, DRAM bytes per launch).  A row whose hash is not the current source's is
    reported as stale and its numbers are withheld."""
    none = {"tensor_pipe_active_pct_ncu": None, "traffic": None, "stale": None}
    src = KERNEL_SOURCES.get(kernel)
    if src is None or not os.path.exists(NCU_COUNTERS):
        return none
    cur = git_blob_hash(os.path.join(ROOT, "paper_2606_09508_b200", "csrc", src))
    with open(NCU_COUNTERS) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if not line:
                continue
            wname, frac, kname, mode, h, tp, dram = line.split()
            if wname == workload and abs(float(frac) - fraction) < 1e-9 and kname == kernel and mode == ("no_skip" if no_skip else "skip"):
                if h != cur:
                    return {"tensor_pipe_active_pct_ncu": None, "traffic": None, "stale": True}
                return {"tensor_pipe_active_pct_ncu": None if tp == "-" else float(tp),
                        "traffic": None if dram == "-" else float(dram), "stale": False}
    return none


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


# ----------------------------------------------------------------------------------------------
# work accounting (host arithmetic on the plan's lists; no method arithmetic)
# ----------------------------------------------------------------------------------------------
def executed_tiles(wl, k_counts: np.ndarray) -> int:
    """128 x L_B tiles the attention kernel issues: every non-diagonal selected block for each of
    the L_S/128 row tiles, plus the diagonal blocks not entirely above the row tile."""
    tps = wl.L_S // 128
    diag = 0
    for qt in range(tps):
        last_row = qt * 128 + 127           # within the segment
        diag += min(wl.r, last_row // wl.L_B + 1)
    nondiag = (k_counts.astype(np.int64) - wl.r).sum() * tps
    return int(nondiag + diag * k_counts.size)


def tile_flops(wl) -> float:
    return 4.0 * 128 * wl.L_B * wl.d     # QK^T and PV, 2 flop per multiply-add


def max_over_ranks(value: float, dist=None, device=None) -> float:
    """Step time of the job = the slowest rank's (replicas run independently, so only timing is reduced)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_value(ms_per_step: float, world: int) -> float:
    """ms per layer over all layers the job processed: N replicas finish N layers per step."""
    return ms_per_step / world


# ----------------------------------------------------------------------------------------------
# clocks sampler
# ----------------------------------------------------------------------------------------------
class ClockSampler:
    """Polls SM clock, power and clock-event reasons through NVML (read-only) in a thread while the timed
    region runs; falls back to one `nvidia-smi` query if NVML is not importable."""
    REASONS = {"hw_slowdown": 0x8, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20, "sw_power_cap": 0x4}

    def __init__(self, gpu_index: int, period_s: float = 0.004):
        self.gpu, self.period = gpu_index, period_s
        self.rows, self._stop, self.t, self.h, self.nv = [], threading.Event(), None, None, None

    def start(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            idx = self.gpu
            vis = os.environ.get("CUDA_VISIBLE_DEVICES")
            if vis:
                try:
                    idx = int(vis.split(",")[self.gpu])
                except Exception:
                    idx = self.gpu
            self.h = pynvml.nvmlDeviceGetHandleByIndex(idx)
            self.nv = pynvml
            self.max_sm = float(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.t = threading.Thread(target=self._poll, daemon=True)
            self.t.start()
        except Exception:
            self.nv = None

    def _poll(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                sm = nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)
                pw = nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0
                try:
                    rs = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    rs = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                self.rows.append((time.time(), float(sm), pw, int(rs)))
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self, t0=None, t1=None):
        self._stop.set()
        if self.t is not None:
            self.t.join(timeout=1.0)
        if self.nv is None:
            return self._smi_once()
        rows = [r for r in self.rows if (t0 is None or r[0] >= t0) and (t1 is None or r[0] <= t1)] or self.rows
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": getattr(self, "max_sm", None), "reasons": ["no samples"]}
        reasons = sorted(n for n, bit in self.REASONS.items() if any(r[3] & bit for r in rows))
        return {"sm_mhz": float(np.median([r[1] for r in rows])), "sm_min_mhz": float(min(r[1] for r in rows)),
                "sm_max_mhz": self.max_sm, "power_w": float(np.median([r[2] for r in rows])), "samples": len(rows),
                "reasons": reasons, "source": "nvml"}

    def _smi_once(self):
        q = "clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active"
        try:
            o = subprocess.run(["nvidia-smi", f"--query-gpu={q}", "--format=csv,noheader,nounits", "-i", str(self.gpu)],
                               capture_output=True, text=True, timeout=10).stdout.strip().split(",")
            return {"sm_mhz": float(o[0]), "sm_max_mhz": float(o[1]), "power_w": float(o[2]), "samples": 1,
                    "reasons": [o[3].strip()], "source": "nvidia-smi after the run"}
        except Exception:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}


# ----------------------------------------------------------------------------------------------
# CPU oracle leg (cpu_baseline and --impl reference)
# ----------------------------------------------------------------------------------------------
def sample_cells(wl, rigid: np.ndarray, n_cells: int, seed: int):
    """Stratified (head class x segment position) sample of (h, i) cells."""
    rng = np.random.default_rng(seed)
    heads_r = np.flatnonzero(rigid)
    heads_d = np.flatnonzero(~rigid.astype(bool))
    cells = []
    segs = np.linspace(0, wl.C_S - 1, num=max(2, n_cells // 2)).round().astype(int)
    for idx, i in enumerate(segs):
        for group in (heads_r, heads_d):
            if len(group):
                cells.append((int(group[rng.integers(len(group))]), int(i)))
    return cells[:n_cells]


def oracle_step(wl, q, k, v, n_cells: int, seed: int = 0):
    """Times the oracle: stages O1-O6 in full, O7 on a cell sample, extrapolated by key blocks."""
    import oracle
    t0 = time.perf_counter()
    op = oracle.plan(q, k, wl.L_S, wl.L_B, fraction=wl.fraction)
    t_plan = time.perf_counter() - t0
    cells = sample_cells(wl, op.rigid, n_cells, seed)
    t0 = time.perf_counter()
    oracle.sparse_attention(q, k, v, wl.L_S, wl.L_B, op.offsets, op.idx, cells=cells)
    t_attn_sample = time.perf_counter() - t0
    sampled_blocks = sum(int(op.k[h, i]) for h, i in cells)
    total_blocks = int(op.k.sum())
    t_attn_full = t_attn_sample * total_blocks / max(1, sampled_blocks)
    return dict(t_plan=t_plan, t_attn_sample=t_attn_sample, t_attn_full=t_attn_full, cells=len(cells),
                sampled_blocks=sampled_blocks, total_blocks=total_blocks, cores=oracle.num_threads())


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    q, k, v, st = synth.generate(wl)
    times, last = [], None
    for s in range(args.warmup + args.steps):
        last = oracle_step(wl, q, k, v, args.ref_cells, seed=s)
        if s >= args.warmup:
            times.append(last["t_plan"] + last["t_attn_full"])
    ms = 1e3 * float(np.mean(times))
    sample = (f"O1-O6 in full; O7 on {last['cells']} of {wl.H * wl.C_S} (head, segment) cells "
              f"({last['sampled_blocks']} of {last['total_blocks']} key blocks), scaled by key blocks (extrapolated)")
    line = {
        "impl": "reference", "metric": METRIC, "value": ms, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": False,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(wl),
        "cpu_baseline": {"value": ms, "unit": UNIT, "cores": last["cores"], "kind": "oracle", "sample": sample},
        "e2e": {"value": ms, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def workload_config(wl, group_shared=False):
    return {"workload": wl.name, "n_q_heads": wl.H, "n_kv_heads": wl.Hkv, "head_dim": wl.d, "seq_len": wl.N,
            "segment_len": wl.L_S, "block_len": wl.L_B, "budget_fraction": wl.fraction,
            "rigid_fraction": wl.rigid_fraction, "batch": 1, "seed": wl.seed,
            "lists": "per KV group" if group_shared else "per query head",
            "l2": "inputs larger than L2 (Q alone exceeds 126 MB); no explicit flush",
            "parallelism": "replicas only"}


# ----------------------------------------------------------------------------------------------
# GPU leg
# ----------------------------------------------------------------------------------------------
def run_ours(args, wl):
    import torch

    import paper_2606_09508_b200 as ei

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    peaks = load_peaks()
    q, k, v, st = synth.generate(wl)

    def dev(b):
        return torch.from_numpy(b.view(np.int16)).cuda().view(torch.bfloat16)

    qd, kd, vd = dev(q), dev(k), dev(v)
    out = torch.empty((wl.H, wl.N, wl.d), dtype=torch.bfloat16, device="cuda")
    params = ei.params_default(wl.H, wl.Hkv, wl.d, wl.N, wl.L_S, wl.L_B, wl.fraction)
    if args.group_shared:
        params.flags |= ei.FLAG_GROUP_SHARED
    params.flags |= attention_flags(ei, args.attention)
    if args.no_skip:
        params.flags |= ei.FLAG_ATTN_NO_SKIP
    plan = ei.Plan(params)
    stream = torch.cuda.current_stream()

    def step():
        plan.plan(qd, kd, vd)
        plan.sparse_prefill(qd, kd, vd, out)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    if plan.status() != 0:
        raise RuntimeError("device-side wait timed out during warm-up")

    # ---- timed region: K whole steps -----------------------------------------------------------------
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    barrier()
    launches0 = plan.launches()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_wall0 = time.time()
    ev0.record(stream)
    for _ in range(args.steps):
        step()
    ev1.record(stream)
    barrier()
    t_wall1 = time.time()
    launches = plan.launches() - launches0
    elapsed_ms = max_over_ranks(ev0.elapsed_time(ev1), dist, "cuda")
    clocks = sampler.stop(t_wall0, t_wall1) if rank == 0 else None
    if plan.status() != 0:
        raise RuntimeError("device-side wait timed out during the timed region")
    ms_per_step = elapsed_ms / args.steps

    # ---- per-call and per-kernel timing over K more steps (events on the launching stream) ----------------
    # ei_plan and ei_sparse_prefill as whole calls, then the four planning kernels one by one (ei_stage_*).
    pe = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    for s_ in range(args.steps):
        pe[s_][0].record(stream)
        plan.plan(qd, kd, vd)
        pe[s_][1].record(stream)
        plan.sparse_prefill(qd, kd, vd, out)
        pe[s_][2].record(stream)
    torch.cuda.synchronize()
    plan_call_ms = float(np.mean([pe[s_][0].elapsed_time(pe[s_][1]) for s_ in range(args.steps)]))
    attn_ms = float(np.mean([pe[s_][1].elapsed_time(pe[s_][2]) for s_ in range(args.steps)]))
    names = ["pool", "observe", "budget", "select"]
    calls = [lambda: plan.stage_pool(qd, kd), plan.stage_observe, plan.stage_budget, plan.stage_select]
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(len(names) + 1)] for _ in range(args.steps)]
    for s_ in range(args.steps):
        evs[s_][0].record(stream)
        for j, c in enumerate(calls):
            c()
            evs[s_][j + 1].record(stream)
    torch.cuda.synchronize()
    kernel_ms = {n: float(np.mean([evs[s_][j].elapsed_time(evs[s_][j + 1]) for s_ in range(args.steps)]))
                 for j, n in enumerate(names)}
    kernel_ms["attention"] = attn_ms

    res = plan.results()
    k_per_head = np.repeat(res["k"], wl.H // wl.Hkv, axis=0) if args.group_shared else res["k"]
    tiles = executed_tiles(wl, k_per_head)
    flops = tiles * tile_flops(wl)
    att_tflops = flops / (kernel_ms["attention"] * 1e-3) / 1e12

    # ---- the same attention launch with every probability evaluated (EI_FLAG_ATTN_NO_SKIP): what the shortcut for
    # negligible half rows is worth on this input (it depends on how peaked the heads are) ------------------------
    every_p = None
    if not args.no_skip and world == 1:
        params2 = ei.params_default(wl.H, wl.Hkv, wl.d, wl.N, wl.L_S, wl.L_B, wl.fraction)
        params2.flags = params.flags | ei.FLAG_ATTN_NO_SKIP
        plan2 = ei.Plan(params2)
        plan2.plan(qd, kd, vd)
        out2 = torch.empty_like(out)
        for _ in range(3):
            plan2.sparse_prefill(qd, kd, vd, out2)
        ne = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
        ne[0].record(stream)
        for s_ in range(args.steps):
            plan2.sparse_prefill(qd, kd, vd, out2)
            ne[s_ + 1].record(stream)
        torch.cuda.synchronize()
        if plan2.status() != 0:
            raise RuntimeError("device-side wait timed out")
        ns_ms = float(np.mean([ne[s_].elapsed_time(ne[s_ + 1]) for s_ in range(args.steps)]))
        every_p = {"attention_ms": ns_ms, "tflops": flops / (ns_ms * 1e-3) / 1e12,
                   "what": "EI_FLAG_ATTN_NO_SKIP: no shortcut for rows below 2^-24 of the row maximum"}
        del plan2, out2
    # ---- the same kernel at full budget (every causal block selected): one launch, for the sparse / dense ratio ----
    dense = None
    if world == 1 and not args.no_dense:
        pd = ei.params_default(wl.H, wl.Hkv, wl.d, wl.N, wl.L_S, wl.L_B, 1.0)
        pd.flags = params.flags
        pland = ei.Plan(pd)
        pland.plan(qd, kd, vd)
        outd = torch.empty_like(out)
        pland.sparse_prefill(qd, kd, vd, outd)        # warm-up launch
        d0, d1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        d0.record(stream)
        pland.sparse_prefill(qd, kd, vd, outd)
        d1.record(stream)
        torch.cuda.synchronize()
        if pland.status() != 0:
            raise RuntimeError("device-side wait timed out")
        dres = pland.results()
        dk = np.repeat(dres["k"], wl.H // wl.Hkv, axis=0) if args.group_shared else dres["k"]
        dense_ms = d0.elapsed_time(d1)
        dense = {"attention_ms": dense_ms, "executed_tflop": executed_tiles(wl, dk) * tile_flops(wl) / 1e12,
                 "tflops": executed_tiles(wl, dk) * tile_flops(wl) / (dense_ms * 1e-3) / 1e12,
                 "speedup_of_sparse": dense_ms / kernel_ms["attention"], "launches_timed": 1,
                 "what": "the same stage-4 kernel with every causal block selected (budget 100 %)"}
        del pland, outd
    # The tensor roofline's denominator follows the length of the timed region: cuBLAS bf16 as a burst when the
    # K timed steps take under a second (the clock has not yet come down under the power cap), the seconds-long
    # sustained figure otherwise.
    timed_s = ms_per_step * args.steps * 1e-3
    peak_key = "bf16_tflops" if timed_s < 1.0 else "bf16_tflops_sustained"
    tensor_peak = peaks[peak_key]
    qk_bytes = (wl.H + wl.Hkv) * wl.N * wl.d * 2
    pool_bytes = qk_bytes + 2 * (wl.H * wl.C_S + wl.Hkv * wl.C_B) * wl.d * 2
    plan_ms = plan_call_ms
    staged_plan_ms = sum(kernel_ms[n] for n in names)

    # ---- end to end through the host-buffer entry point --------------------------------------------------
    e2e = None
    if world == 1 and not args.no_e2e:
        hq = torch.from_numpy(q.view(np.int16)).pin_memory()
        hk = torch.from_numpy(k.view(np.int16)).pin_memory()
        hv = torch.from_numpy(v.view(np.int16)).pin_memory()
        ho = torch.empty((wl.H, wl.N, wl.d), dtype=torch.int16).pin_memory()
        plan.prefill_host(hq, hk, hv, ho)     # allocates staging, warm-up
        e2e_steps = max(1, min(args.steps, 5))
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(e2e_steps):
            plan.prefill_host(hq, hk, hv, ho)
        e1.record(stream)
        torch.cuda.synchronize()
        e2e_ms = e0.elapsed_time(e1) / e2e_steps
        same = bool(torch.equal(ho.view(-1), out.view(torch.int16).cpu().view(-1)))
        e2e = {"value": e2e_ms, "unit": UNIT, "h2d_bytes_per_step": int(q.nbytes + k.nbytes + v.nbytes),
               "d2h_bytes_per_step": int(ho.numel() * 2), "steps": e2e_steps, "matches_device_path": same}

    # ---- CPU oracle beside it (rank 0, N = 1 only) ----------------------------------------------------------
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu:
        o = oracle_step(wl, q, k, v, args.ref_cells)
        cpu = {"value": 1e3 * (o["t_plan"] + o["t_attn_full"]), "unit": UNIT, "cores": o["cores"], "kind": "oracle",
               "sample": (f"O1-O6 in full ({o['t_plan']:.2f} s); O7 on {o['cells']} of {wl.H * wl.C_S} cells "
                          f"({o['sampled_blocks']} of {o['total_blocks']} key blocks, {o['t_attn_sample']:.2f} s), "
                          "scaled by key blocks (extrapolated)")}

    # ---- follow-on path (optional): latent KV-cache compression of Alg. 4 on the same K/V -----------------
    compress = None
    if args.with_compress and world == 1:
        n_w, b_d = 64, 1024
        cp = ei.compress_params(wl.H, wl.Hkv, wl.d, wl.N, n_w, b_d)
        ws = torch.empty(ei.latent_compress_workspace_bytes(cp) // 4, dtype=torch.float32, device="cuda")
        cidx = torch.empty((wl.Hkv, b_d), dtype=torch.int32, device="cuda")
        cko = torch.empty((wl.Hkv, b_d, wl.d), dtype=torch.bfloat16, device="cuda")
        cvo = torch.empty_like(cko)
        qwin = qd[:, -n_w:, :].contiguous()
        for _ in range(3):
            ei.latent_compress(cp, qwin, kd, vd, ws, cidx, cko, cvo)
        ce = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
        ce[0].record(stream)
        for s_ in range(args.steps):
            ei.latent_compress(cp, qwin, kd, vd, ws, cidx, cko, cvo)
            ce[s_ + 1].record(stream)
        torch.cuda.synchronize()
        cms = float(np.mean([ce[s_].elapsed_time(ce[s_ + 1]) for s_ in range(args.steps)]))
        cbytes = wl.Hkv * wl.N * wl.d * 2 + 4 * wl.Hkv * b_d * wl.d * 2
        compress = {"ms": cms, "window": n_w, "budget": b_d, "kv_len": wl.N, "algorithmic_bytes": int(cbytes),
                    "roofline": {"bound": "hbm", "achieved": cbytes / (cms * 1e-3) / 1e9, "peak": peaks["hbm_gbs"],
                                 "unit": "GB/s", "frac": cbytes / (cms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                 "what": "K read once + kept K,V rows read and written / whole ei_latent_compress call"}}

    # ---- producer-side pooling (optional): the rotary embedding of Q and K with Alg. 1's pooling folded in ---------
    producer = None
    if args.with_producer and world == 1:
        cos, sin = synth.rope_tables(wl.N, wl.d)
        cd, sd = torch.from_numpy(cos).cuda(), torch.from_numpy(sin).cuda()
        q_rot, k_rot = torch.empty_like(qd), torch.empty_like(kd)
        pp = ei.params_default(wl.H, wl.Hkv, wl.d, wl.N, wl.L_S, wl.L_B, wl.fraction)
        pp.flags = ei.FLAG_GROUP_SHARED if args.group_shared else 0
        pplan = ei.Plan(pp)

        def timed(fn):
            for _ in range(3):
                fn()
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
            ev[0].record(stream)
            for s_ in range(args.steps):
                fn()
                ev[s_ + 1].record(stream)
            torch.cuda.synchronize()
            return float(np.mean([ev[s_].elapsed_time(ev[s_ + 1]) for s_ in range(args.steps)]))
        t_rope = timed(lambda: pplan.rope_pool(qd, kd, cd, sd, q_rot, k_rot, pool=False))
        t_rope_pool = timed(lambda: pplan.rope_pool(qd, kd, cd, sd, q_rot, k_rot))
        t_pooled = timed(lambda: pplan.plan_pooled())
        t_plan = timed(lambda: pplan.plan(q_rot, k_rot))
        if pplan.status() != 0:
            raise RuntimeError("device-side wait timed out")
        rbytes = 2 * (q.nbytes + k.nbytes)
        producer = {"rope_ms": t_rope, "rope_pool_ms": t_rope_pool, "plan_pooled_ms": t_pooled, "plan_ms": t_plan,
                    "separate_ms": t_rope + t_plan, "fused_ms": t_rope_pool + t_pooled,
                    "algorithmic_bytes": int(rbytes),
                    "roofline": {"bound": "hbm", "achieved": rbytes / (t_rope_pool * 1e-3) / 1e9, "peak": peaks["hbm_gbs"],
                                 "unit": "GB/s", "frac": rbytes / (t_rope_pool * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                 "what": "Q and K read and written once / ei_rope_pool"}}

    # ---- the same step captured once in a CUDA graph and replayed (launch overhead matters on short sequences) ----
    graph_info = None
    if args.graph and world == 1:
        side = torch.cuda.Stream()
        side.wait_stream(stream)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            plan.plan(qd, kd, vd, stream=side)
            plan.sparse_prefill(qd, kd, vd, out, stream=side)
        for _ in range(3):
            g.replay()
        torch.cuda.synchronize()
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record(stream)
        for _ in range(args.steps):
            g.replay()
        g1.record(stream)
        torch.cuda.synchronize()
        graph_info = {"ms_per_step": g0.elapsed_time(g1) / args.steps, "eager_ms_per_step": ms_per_step}

    # ---- group-shared planning: deviation from the dense result, next to the per-head plan's ------------------
    group_cmp = None
    if args.group_shared and world == 1:
        def run_with(flags, fraction):
            pp = ei.params_default(wl.H, wl.Hkv, wl.d, wl.N, wl.L_S, wl.L_B, fraction)
            pp.flags = flags
            pl_ = ei.Plan(pp)
            o_ = torch.empty_like(out)
            pl_.plan(qd, kd, vd)
            pl_.sparse_prefill(qd, kd, vd, o_)
            torch.cuda.synchronize()
            return o_
        dense_o = run_with(0, 1.0).float()
        dev_group = float((out.float() - dense_o).abs().mean())
        dev_head = float((run_with(0, wl.fraction).float() - dense_o).abs().mean())
        group_cmp = {"mean_abs_dev_from_dense_group_shared": dev_group, "mean_abs_dev_from_dense_per_head": dev_head,
                     "mean_abs_dense": float(dense_o.abs().mean())}
        del dense_o

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    kname = attention_kernel_name(wl, args, plan.total_blocks())
    counters = ncu_counters(wl.name, wl.fraction, kname, args.no_skip)
    counters_all = ncu_counters(wl.name, wl.fraction, kname, True)
    if every_p is not None:
        every_p["frac_of_burst"] = every_p["tflops"] / peaks["bf16_tflops"]
        every_p["tensor_pipe_active_pct_ncu"] = counters_all["tensor_pipe_active_pct_ncu"]
        every_p["counters_stale"] = counters_all["stale"]

    line = {
        "metric": METRIC, "value": job_value(ms_per_step, world), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": workload_config(wl, args.group_shared),
        "tokens_per_s": wl.N * world / (ms_per_step * 1e-3),
        "kernel_ms": kernel_ms, "plan_ms": plan_ms, "staged_plan_ms": staged_plan_ms,
        "executed_tiles": tiles, "executed_tflop": flops / 1e12,
        "roofline": {"bound": "tensor", "achieved": att_tflops, "peak": tensor_peak, "unit": "TFLOP/s",
                     "frac": att_tflops / tensor_peak, "traffic": counters["traffic"],
                     "kernel": kname,
                     "algorithmic_bytes": int(2 * wl.H * wl.N * wl.d * 2 + 2 * wl.Hkv * wl.N * wl.d * 2),
                     "tensor_pipe_active_pct_ncu": counters["tensor_pipe_active_pct_ncu"], "stale": counters["stale"],
                     "peak_kind": f"cuBLAS bf16 {'burst' if peak_key == 'bf16_tflops' else 'sustained'} ({peaks['source']}): "
                                  f"the {args.steps} timed steps took {timed_s:.2f} s",
                     "frac_of_burst": att_tflops / peaks["bf16_tflops"],
                     "frac_of_sustained": att_tflops / peaks["bf16_tflops_sustained"],
                     "frac_of_nominal_2250": att_tflops / NOMINAL_BF16_TFLOPS},
        "dense": dense, "dense_speedup": None if dense is None else dense["speedup_of_sparse"],
        "roofline_plan": {"bound": "hbm", "achieved": qk_bytes / (plan_ms * 1e-3) / 1e9, "peak": peaks["hbm_gbs"],
                          "unit": "GB/s", "frac": qk_bytes / (plan_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                          "frac_of_nominal_8000": qk_bytes / (plan_ms * 1e-3) / 1e9 / NOMINAL_HBM_GBS,
                          "what": "Q+K bytes / whole ei_plan call (K pooling, fused Q pooling + observation, budget, select)", "peak_kind": f"copy, {peaks['source']}",
                          "pool_kernel_gbs": pool_bytes / (kernel_ms["pool"] * 1e-3) / 1e9},
        "cuda_graph": graph_info, "group_shared": group_cmp, "every_probability_evaluated": every_p, "latent_compress": compress, "producer_pooling": producer, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": int(launches), "clocks": clocks,
        "plan_stats": {"rigid_heads": int(res["stats"][1]), "total_blocks": int(res["stats"][0]),
                       "min_k": int(res["stats"][4]), "max_k": int(res["stats"][5])},
    }
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


# ----------------------------------------------------------------------------------------------
# Parameter sweeps (speed only; the paper sweeps segment / block size and budgets for quality, Fig. 5-6, and
# reports end-to-end latency against input length, Section 5.3).  One JSON line per point.
# ----------------------------------------------------------------------------------------------
# ----------------------------------------------------------------------------------------------
# One layer's heads sharded over the ranks by KV group (--shard kv): strong scaling of ONE layer
# ----------------------------------------------------------------------------------------------
def shard_heads(H: int, Hkv: int, rank: int, world: int):
    """Rank p of `world` holds the KV heads [p*Hkv/world, (p+1)*Hkv/world) and the query heads that read them."""
    if Hkv % world != 0:
        raise ValueError(f"{Hkv} KV heads do not split over {world} ranks")
    g_per, G = Hkv // world, H // Hkv
    g0 = rank * g_per
    return g0 * G, (g0 + g_per) * G, g0, g0 + g_per


def total_blocks_all(wl) -> int:
    """T of the whole layer, as ei_plan_create works it out for a plan over all heads."""
    SC = sum(min(wl.r * (i + 1), wl.C_B) for i in range(wl.C_S))
    return int(math.floor(wl.fraction * float(wl.H) * float(SC) + 0.5))


def run_shard_kv(args, wl):
    """The layer of the workload with its heads sharded over the ranks by KV group.  Everything of the method is
    per head except TOTAL mode's common total: every rank works out the multipliers of its heads, the int32
    tables are all-gathered (NCCL, the one collective of the path), and every rank apportions the layer's total
    over the gathered table and keeps its own rows.  Each rank then selects and attends for its heads alone."""
    import torch

    import paper_2606_09508_b200 as ei

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    peaks = load_peaks()
    h0, h1, g0, g1 = shard_heads(wl.H, wl.Hkv, rank, world)
    q, k, v, st = synth.generate(wl)          # every rank draws the layer (seeded), keeps its heads

    def dev(b):
        return torch.from_numpy(np.ascontiguousarray(b).view(np.int16)).cuda().view(torch.bfloat16)

    qd, kd, vd = dev(q[h0:h1]), dev(k[g0:g1]), dev(v[g0:g1])
    Hl, Hkvl = h1 - h0, g1 - g0
    out = torch.empty((Hl, wl.N, wl.d), dtype=torch.bfloat16, device="cuda")
    params = ei.params_default(Hl, Hkvl, wl.d, wl.N, wl.L_S, wl.L_B, wl.fraction)
    params.flags |= ei.FLAG_HEAD_SHARD | attention_flags(ei, args.attention)
    if args.no_skip:
        params.flags |= ei.FLAG_ATTN_NO_SKIP
    plan = ei.Plan(params)
    stream = torch.cuda.current_stream()
    T_all = total_blocks_all(wl)
    m_all = torch.zeros((wl.H, wl.C_S), dtype=torch.int32, device="cuda")
    m_loc = torch.zeros((Hl, wl.C_S), dtype=torch.int32, device="cuda")

    def plan_step():
        plan.observe(qd, kd)
        if world > 1:
            plan.stage_multipliers(out=m_loc)
            dist.all_gather_into_tensor(m_all.view(-1), m_loc.view(-1))
        else:
            plan.stage_multipliers(out=m_all)
        plan.stage_apportion(m_all, wl.H, h0, T_all)
        plan.stage_select()

    def step():
        plan_step()
        plan.sparse_prefill(qd, kd, vd, out)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    if plan.status() != 0:
        raise RuntimeError("device-side wait timed out during warm-up")
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    barrier()
    launches0 = plan.launches()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_wall0 = time.time()
    ev0.record(stream)
    for _ in range(args.steps):
        step()
    ev1.record(stream)
    barrier()
    t_wall1 = time.time()
    launches = plan.launches() - launches0
    elapsed_ms = max_over_ranks(ev0.elapsed_time(ev1), dist, "cuda")
    clocks = sampler.stop(t_wall0, t_wall1) if rank == 0 else None
    if plan.status() != 0:
        raise RuntimeError("device-side wait timed out during the timed region")
    ms_per_step = elapsed_ms / args.steps

    # per-call timing on this rank (max over ranks): the planning sequence with its all-gather, the attention launch
    pe = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    for s_ in range(args.steps):
        pe[s_][0].record(stream)
        plan_step()
        pe[s_][1].record(stream)
        plan.sparse_prefill(qd, kd, vd, out)
        pe[s_][2].record(stream)
    torch.cuda.synchronize()
    plan_ms = max_over_ranks(float(np.mean([pe[s_][0].elapsed_time(pe[s_][1]) for s_ in range(args.steps)])), dist, "cuda")
    attn_ms = max_over_ranks(float(np.mean([pe[s_][1].elapsed_time(pe[s_][2]) for s_ in range(args.steps)])), dist, "cuda")
    res = plan.results()
    tiles_local = executed_tiles(synth.generator.with_(wl, H=Hl, Hkv=Hkvl), res["k"])
    tiles_t = torch.tensor([float(tiles_local)], dtype=torch.float64, device="cuda")
    if dist is not None:
        dist.all_reduce(tiles_t)
    flops = float(tiles_t.item()) * tile_flops(wl)

    # the shards against one plan over all heads (rank 0, which has drawn the whole layer): same rows, bit for bit
    matches = None
    if rank == 0 and not args.no_dense:
        pf = ei.params_default(wl.H, wl.Hkv, wl.d, wl.N, wl.L_S, wl.L_B, wl.fraction)
        pf.flags = params.flags & ~ei.FLAG_HEAD_SHARD
        full = ei.Plan(pf)
        qf, kf = dev(q), dev(k)
        full.plan(qf, kf)
        rf = full.results()
        cells = Hl * wl.C_S
        lo = int(rf["offsets"][h0 * wl.C_S])
        matches = bool(np.array_equal(rf["k"][h0:h1], res["k"]) and
                       np.array_equal(rf["offsets"][h0 * wl.C_S:h0 * wl.C_S + cells + 1] - lo, res["offsets"]) and
                       np.array_equal(rf["idx"][lo:lo + int(res["offsets"][-1])], res["idx"][:int(res["offsets"][-1])]))
        del full, qf, kf

    # end to end: this rank's heads from pinned host buffers, result back to the host, every step
    e2e = None
    if not args.no_e2e:
        hq, hk, hv = (torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).pin_memory()
                      for a in (q[h0:h1], k[g0:g1], v[g0:g1]))
        hout = torch.empty((Hl, wl.N, wl.d), dtype=torch.int16).pin_memory()
        qi, ki, vi = (torch.empty_like(t_, device="cuda") for t_ in (hq, hk, hv))

        def e2e_step():
            qi.copy_(hq, non_blocking=True)
            ki.copy_(hk, non_blocking=True)
            vi.copy_(hv, non_blocking=True)
            qb, kb, vb = (t_.view(torch.bfloat16) for t_ in (qi, ki, vi))
            plan.observe(qb, kb)
            if world > 1:
                plan.stage_multipliers(out=m_loc)
                dist.all_gather_into_tensor(m_all.view(-1), m_loc.view(-1))
            else:
                plan.stage_multipliers(out=m_all)
            plan.stage_apportion(m_all, wl.H, h0, T_all)
            plan.stage_select()
            plan.sparse_prefill(qb, kb, vb, out)
            hout.copy_(out.view(torch.int16), non_blocking=True)
        e2e_step()
        barrier()
        n_e = max(2, min(args.steps, 5))
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(n_e):
            e2e_step()
        e1.record(stream)
        barrier()
        e_ms = max_over_ranks(e0.elapsed_time(e1), dist, "cuda") / n_e
        e2e = {"value": e_ms, "unit": "ms/layer", "h2d_bytes_per_step": int((hq.numel() + hk.numel() + hv.numel()) * 2),
               "d2h_bytes_per_step": int(hout.numel() * 2), "steps": n_e,
               "what": "per rank: its heads' Q, K, V up from pinned host memory, sharded planning, attention, output down"}

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return
    timed_s = ms_per_step * args.steps * 1e-3
    peak_key = "bf16_tflops" if timed_s < 1.0 else "bf16_tflops_sustained"
    att_tflops = flops / (attn_ms * 1e-3) / 1e12
    kern = attention_kernel_name(wl, args, 0)
    ctr = {"tensor_pipe_active_pct_ncu": None, "traffic": None, "stale": None}   # no capture of the sharded launch
    cfg = workload_config(wl)
    cfg["parallelism"] = f"one layer, heads sharded by KV group over {world} GPU(s): {Hkvl} KV heads + {Hl} query heads per rank"
    cfg["exchange"] = "one all-gather of the int32 multiplier table (H x C_S) per step (NCCL)" if world > 1 else "none (one rank)"
    line = {"metric": "128k-token sparse prefill attention ms/layer; tensor-pipe % of B200 peak", "value": ms_per_step,
            "unit": "ms/layer", "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": ms_per_step, "higher_is_better": False, "scaling": "strong", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic", "config": cfg,
            "kernel_ms": {"plan_with_exchange": plan_ms, "attention": attn_ms},
            "executed_tflop": flops / 1e12,
            "roofline": {"bound": "tensor", "achieved": att_tflops, "peak": peaks[peak_key] * world, "unit": "TFLOP/s",
                         "frac": att_tflops / (peaks[peak_key] * world), "traffic": ctr["traffic"],
                         "kernel": kern, "tensor_pipe_active_pct_ncu": ctr["tensor_pipe_active_pct_ncu"], "stale": ctr["stale"],
                         "peak_kind": f"{world} x cuBLAS bf16 " + ("burst" if peak_key == "bf16_tflops" else "sustained") + " (measured)",
                         "what": "all ranks' executed tiles / the slowest rank's attention launch"},
            "shards_match_unsharded_plan": matches, "cpu_baseline": None, "e2e": e2e, "gpu_launches": int(launches),
            "clocks": clocks}
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()



ATTENTION_CHOICES = {"default": "sparse_attention_quad_kernel", "per_cta": "sparse_attention_quad_kernel",
                     "quad_persistent": "sparse_attention_quad_persistent_kernel",
                     "quad_single_tile": "sparse_attention_quad1_kernel", "split": "sparse_attention_split_kernel",
                     "persistent": "sparse_attention_persistent_kernel", "tri": "sparse_attention_tri_kernel"}


def attention_flags(ei, choice: str) -> int:
    return {"default": 0, "per_cta": ei.FLAG_ATTN_PER_CTA, "quad_persistent": ei.FLAG_ATTN_QUAD | ei.FLAG_ATTN_PERSISTENT,
            "quad_single_tile": ei.FLAG_ATTN_QUAD | ei.FLAG_ATTN_SINGLE_TILE, "split": ei.FLAG_ATTN_SPLIT,
            "persistent": ei.FLAG_ATTN_PERSISTENT, "tri": ei.FLAG_ATTN_TRI}[choice]


def attention_kernel_name(wl, args, total_blocks) -> str:
    """Which stage-4 kernel ei_sparse_prefill launches for this workload."""
    if not (wl.d == 128 and wl.L_B == 128 and wl.L_S % 256 == 0):
        return "sparse_attention_pair_kernel" if wl.L_S % 256 == 0 else "sparse_attention_kernel"
    return ATTENTION_CHOICES[args.attention]


def run_chunk_sweep(args, ei, torch, wl):
    """Chunked prefill of the benchmark workload: the same 128k sequence in 1, 2, 4 and 8 chunks, one plan
    re-targeted chunk by chunk (ei_plan_set_lengths), every chunk planned and attended against all keys so far with
    the pooled K representatives of earlier chunks kept; BASE mode at B_h = 2048 tokens."""
    q, k, v, _ = synth.generate(wl)
    qd, kd, vd = (torch.from_numpy(b.view(np.int16)).cuda().view(torch.bfloat16) for b in (q, k, v))
    stream = torch.cuda.current_stream()
    p = ei.params_default(wl.H, wl.Hkv, wl.d, wl.N, wl.L_S, wl.L_B, 0.0)
    p.base_budget_tokens = 2048.0
    plan = ei.Plan(p)                                  # one plan for the full length, re-targeted per chunk
    out = torch.empty((wl.H, wl.N, wl.d), dtype=torch.bfloat16, device="cuda")
    for n_chunks in (1, 2, 4, 8):
        clen = wl.N // n_chunks

        def step():
            for c in range(n_chunks):
                lo, hi = c * clen, (c + 1) * clen
                plan.set_lengths(hi, clen, k_blocks_valid=lo // wl.L_B)   # earlier blocks keep their representatives
                plan.plan(qd[:, lo:hi], kd, vd)
                plan.sparse_prefill(qd[:, lo:hi], kd, vd, out[:, lo:hi])
        for _ in range(max(args.warmup, 3)):
            step()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(args.steps):
            step()
        e1.record(stream)
        torch.cuda.synchronize()
        if plan.status() != 0:
            raise RuntimeError("device-side wait timed out")
        print(json.dumps({"sweep": "chunks", "config": workload_config(wl), "budget": "B_h = 2048 tokens (BASE)",
                          "chunks": n_chunks, "chunk_len": clen, "ms_per_sequence": e0.elapsed_time(e1) / args.steps,
                          "steps": args.steps}), flush=True)


def run_varlen(args):
    """A packed batch of many short sequences (64 x 2048 tokens, Llama-3-8B heads, L_S 256 / L_B 128, half of each
    sequence's causal blocks): ei_prefill_varlen in one set of five launches against one ei_plan +
    ei_sparse_prefill per sequence (what a batch cost before; still what group-shared lists and the other kernels do)."""
    import torch

    import paper_2606_09508_b200 as ei
    Hq, Hkv, d, L_S, L_B, n_seq, n_tok, f = 32, 8, 128, 256, 128, 64, 2048, 0.5
    total = n_seq * n_tok
    q, k, v = synth.generate_plain(Hq, Hkv, total, d, seed=4242)

    def dev(b):
        return torch.from_numpy(b.view(np.int16)).cuda().view(torch.bfloat16)
    qd, kd, vd = dev(q), dev(k), dev(v)
    out_a, out_b = torch.zeros_like(qd), torch.zeros_like(qd)
    cu = np.arange(n_seq + 1, dtype=np.int32) * n_tok
    pa = ei.params_default(Hq, Hkv, d, total, L_S, L_B, f)         # room for all sequences' tables side by side
    plan_a = ei.Plan(pa)
    pb = ei.params_default(Hq, Hkv, d, n_tok, L_S, L_B, f)           # one sequence at a time
    pb.q_stride_head = pb.k_stride_head = pb.v_stride_head = pb.o_stride_head = total * d
    plan_b = ei.Plan(pb)
    stream = torch.cuda.current_stream()

    def packed():
        plan_a.prefill_varlen(qd, kd, vd, out_a, cu)

    def loop():
        for b in range(n_seq):
            lo, hi = b * n_tok, (b + 1) * n_tok
            plan_b.plan(qd[:, lo:hi], kd[:, lo:hi])
            plan_b.sparse_prefill(qd[:, lo:hi], kd[:, lo:hi], vd[:, lo:hi], out_b[:, lo:hi])
    res = {}
    for name, fn, pl in (("one_set_of_launches", packed, plan_a), ("per_sequence_loop", loop, plan_b)):
        for _ in range(max(args.warmup, 3)):
            fn()
        torch.cuda.synchronize()
        l0 = pl.launches()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(args.steps):
            fn()
        e1.record(stream)
        torch.cuda.synchronize()
        if pl.status() != 0:
            raise RuntimeError("device-side wait timed out")
        res[name] = {"ms_per_batch": e0.elapsed_time(e1) / args.steps, "launches_per_batch": (pl.launches() - l0) // args.steps}
    same = bool(torch.equal(out_a.view(torch.int16), out_b.view(torch.int16)))
    print(json.dumps({"sweep": "varlen", "batch": f"{n_seq} x {n_tok} tokens", "heads": [Hq, Hkv], "head_dim": d,
                      "segment_len": L_S, "block_len": L_B, "budget_fraction": f, **res,
                      "speedup": res["per_sequence_loop"]["ms_per_batch"] / res["one_set_of_launches"]["ms_per_batch"],
                      "outputs_identical": same}))


def run_sweep(args):
    import torch

    import paper_2606_09508_b200 as ei

    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
    base = synth.WORKLOADS["llama3_8b_128k"]
    with_ = synth.generator.with_
    points = []
    if args.sweep == "chunks":
        return run_chunk_sweep(args, ei, torch, base)
    if args.sweep == "length":
        # BASE mode at the paper's B_h = 2048 tokens, Llama-3-8B attention shape, 4K ... 140K tokens
        for n in (4096, 8192, 16384, 32768, 65536, 98304, 131072, 143360):
            points.append((with_(base, name=f"llama3_8b_{n}", N=n), "base"))
    else:
        for l_s in (128, 256, 512):
            for l_b in (64, 128):
                points.append((with_(base, name=f"llama3_8b_128k_LS{l_s}_LB{l_b}", L_S=l_s, L_B=l_b), "total"))
    stream = torch.cuda.current_stream()
    for wl, mode in points:
        q, k, v, _ = synth.generate(wl)
        qd, kd, vd = (torch.from_numpy(b.view(np.int16)).cuda().view(torch.bfloat16) for b in (q, k, v))
        out = torch.empty((wl.H, wl.N, wl.d), dtype=torch.bfloat16, device="cuda")

        def timed(params):
            plan = ei.Plan(params)
            for _ in range(max(args.warmup, 3)):
                plan.plan(qd, kd, vd)
                plan.sparse_prefill(qd, kd, vd, out)
            torch.cuda.synchronize()
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
            t_plan = t_att = 0.0
            for _ in range(args.steps):
                ev[0].record(stream)
                plan.plan(qd, kd, vd)
                ev[1].record(stream)
                plan.sparse_prefill(qd, kd, vd, out)
                ev[2].record(stream)
                torch.cuda.synchronize()
                t_plan += ev[0].elapsed_time(ev[1])
                t_att += ev[1].elapsed_time(ev[2])
            if plan.status() != 0:
                raise RuntimeError("device-side wait timed out")
            res = plan.results()
            tiles = executed_tiles(wl, res["k"])
            return t_plan / args.steps, t_att / args.steps, tiles, int(res["stats"][1])

        p = ei.params_default(wl.H, wl.Hkv, wl.d, wl.N, wl.L_S, wl.L_B, wl.fraction)
        if mode == "base":
            p.budget_mode = ei.binding.BUDGET_BASE_TOKENS
            p.base_budget_tokens = 2048.0
        p.flags |= attention_flags(ei, args.attention)
        plan_ms, att_ms, tiles, rigid = timed(p)
        dense = ei.params_default(wl.H, wl.Hkv, wl.d, wl.N, wl.L_S, wl.L_B, 1.0)
        _, dense_att_ms, dense_tiles, _ = timed(dense)
        print(json.dumps({
            "sweep": args.sweep, "config": workload_config(wl), "budget": "B_h = 2048 tokens (BASE)" if mode == "base"
            else f"{wl.fraction:g} of causal blocks (TOTAL)", "plan_ms": plan_ms, "attention_ms": att_ms,
            "step_ms": plan_ms + att_ms, "dense_attention_ms": dense_att_ms,
            "speedup_vs_dense_attention": dense_att_ms / (plan_ms + att_ms), "executed_tiles": tiles,
            "density": tiles / dense_tiles, "attention_tflops": tiles * tile_flops(wl) / (att_ms * 1e-3) / 1e12,
            "rigid_heads": rigid, "steps": args.steps}), flush=True)
        del qd, kd, vd, out
        torch.cuda.empty_cache()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama3_8b_128k", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--fraction", type=float, default=None, help="override the budget fraction")
    ap.add_argument("--ref-cells", type=int, default=24, help="cells the CPU oracle attends over per step")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-dense", action="store_true", help="skip the one launch at full budget (dense_speedup)")
    ap.add_argument("--with-producer", action="store_true",
                    help="also time the rotary producer with and without the pooling folded in (ei_rope_pool, ei_plan_pooled)")
    ap.add_argument("--with-compress", action="store_true", help="also time the Alg. 4 KV-cache compression")
    ap.add_argument("--attention", default="default", choices=sorted(ATTENTION_CHOICES),
                    help="persistent: the persistent form of the two-threads-per-row attention kernel; tri: the three-buffer kernel")
    ap.add_argument("--no-skip", action="store_true",
                    help="evaluate every probability (EI_FLAG_ATTN_NO_SKIP): no shortcut for negligible half rows")
    ap.add_argument("--graph", action="store_true", help="also time the step replayed from a CUDA graph")
    ap.add_argument("--group-shared", action="store_true",
                    help="plan once per KV group (EI_FLAG_GROUP_SHARED) instead of once per query head")
    ap.add_argument("--shard", default=None, choices=["kv"],
                    help="kv: ONE layer with its heads sharded over the --gpus ranks by KV group (strong scaling; one "
                         "all-gather of the multiplier table per step) instead of one replica of the layer per rank")
    ap.add_argument("--sweep", default=None, choices=["length", "blocks", "chunks", "varlen"],
                    help="speed sweeps on the Llama-3-8B shape instead of the benchmark line: input length at the "
                         "paper's B_h = 2048 tokens, or segment x block size at 128k")
    args = ap.parse_args()
    if args.sweep == "varlen":
        run_varlen(args)
        return
    if args.sweep:
        run_sweep(args)
        return
    wl = synth.WORKLOADS[args.workload]
    if args.fraction is not None:
        wl = synth.generator.with_(wl, fraction=args.fraction)
    if args.impl == "reference":
        run_reference(args, wl)
    elif args.shard == "kv":
        run_shard_kv(args, wl)
    else:
        run_ours(args, wl)


if __name__ == "__main__":
    main()
