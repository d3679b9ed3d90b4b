#!/usr/bin/env python
"""Benchmark: context tokens/s of one full-model LAVa prefill eviction on B200.

A "step" is one pass of the whole hot path (score all layers -> layer budgets -> layer-wide
top-k -> gather/compact) over one batch of synthetic input.  Default workload: Llama-3-8B shaped,
one 32K-token sequence, w=32, max-pool 7, 2048 rows per KV head on average, dynamic budgets.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

Prints ONE JSON line (rank 0).  With --impl reference the CPU oracle is timed instead.
Multi-GPU: the path does not shard (one sequence batch per GPU, no collective): N independent
replicas, weak scaling, max-over-ranks timing.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "context tokens/s per full-model prefill eviction"
UNIT = "tokens/s"
FALLBACK_HBM_GBS = 6650.0


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="llama8b_32k")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--cpu-layers", type=int, default=64,
                    help="upper bound on the layers the CPU oracle is timed on (cpu_baseline)")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--path", default="evict", choices=["evict", "cascade", "decode"],
                    help="evict: the one-shot hot path (the headline line); cascade: Algorithm 2 one "
                         "layer per call; decode: attention of one new token over the packed cache")
    ap.add_argument("--layers", type=int, default=0,
                    help="run only the first N layers of the workload (small cases for profiling; "
                         "the budget shrinks in proportion and the line says so)")
    return ap.parse_args()


# ----------------------------------------------------------------------------- helpers
def measured_hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (6.65 TB/s, MEASURED_PEAKS.json absent)"


def committed_traffic(workload):
    """DRAM bytes per launch of the dominant kernel from the committed ncu capture, or None."""
    path = os.path.join(ROOT, "profiles", "traffic.json")
    try:
        with open(path) as f:
            return json.load(f).get(workload)
    except Exception:
        return None


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self._nv = None

    def _loop(self):
        nv = self._nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4),
        }
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
                mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h)
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(0.002)

    def start(self):
        if self._nv is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
        return {
            "sm_mhz": statistics.median(self.samples) if self.samples else None,
            "sm_max_mhz": self.max_mhz,
            "reasons": sorted(self.reasons),
            "samples": len(self.samples),
        }


def visible_gpu_index(local_rank):
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


def roofline_bytes(cfg):
    """Algorithmic HBM bytes of one full-model eviction: K and V read once plus the packed
    cache written (2 * H_kv * n * d * e per layer + 2 * B * d * e)."""
    es = 2 if cfg.dtype == "bf16" else 4
    kv = 2 * cfg.n_kv_heads * cfg.total_tokens * cfg.head_dim * es * cfg.n_layers
    out = 2 * sum(cfg.total_budget(b) for b in range(cfg.batch)) * cfg.head_dim * es
    return kv, out


# ----------------------------------------------------------------------------- oracle legs
def _oracle_layer(cfg, tensors):
    """score + entropy + select + compact of one layer with the CPU oracle, as it stands (budgets
    are uniform per layer here: a bounded sample has too few layers to share the total)."""
    import torch
    from lava_workloads import to_numpy64
    from oracle import lava_oracle as O
    hkv, w = cfg.n_kv_heads, cfg.window
    tok0 = 0
    for b, n in enumerate(cfg.seq_lens):
        q = to_numpy64(tensors["q_win"][b])
        k = to_numpy64(tensors["k"][:, tok0: tok0 + n])
        v = to_numpy64(tensors["v"][:, tok0: tok0 + n])
        s = O.lava_scores(q, k, v, w, cfg.pool_kind, cfg.pool_kernel)
        O.layer_entropy(s, n)
        keep, _ = O.select_topk(s, cfg.budget_per_head * hkv, w)
        bits = torch.int16 if cfg.dtype == "bf16" else torch.int32
        O.compact_kv(tensors["k"][:, tok0: tok0 + n].view(bits).numpy(),
                     tensors["v"][:, tok0: tok0 + n].view(bits).numpy(), keep, w)
        tok0 += n


_POOL_STATE = {}


def _pool_init(barrier, workload):
    """Worker start-up: one BLAS thread per worker (the workers are the parallelism), imports done
    and the workload known before anything is timed."""
    from threadpoolctl import threadpool_limits
    import torch
    from lava_workloads import get_config
    torch.set_num_threads(1)
    _POOL_STATE["limits"] = threadpool_limits(limits=1)
    _POOL_STATE["barrier"] = barrier
    _POOL_STATE["cfg"] = get_config(workload)


def _pool_work(layers):
    """Generates this worker's layers (untimed), meets the other workers, then times the oracle."""
    from lava_workloads import generate_layer
    cfg = _POOL_STATE["cfg"]
    tensors = [generate_layer(cfg, l, "cpu") for l in layers]
    _POOL_STATE["barrier"].wait()
    t0 = time.time()
    for t in tensors:
        _oracle_layer(cfg, t)
    return t0, time.time()


class OraclePool:
    """The oracle over distinct layers of the workload, one layer stream per host core."""

    def __init__(self, workload, workers):
        import multiprocessing as mp
        ctx = mp.get_context("spawn")
        self.workers = workers
        self.barrier = ctx.Barrier(workers)
        self.pool = ctx.Pool(workers, initializer=_pool_init, initargs=(self.barrier, workload))

    def run(self, layers_per_worker, n_layers):
        """Wall seconds (first start to last end) for workers * layers_per_worker layers."""
        jobs = [[(w * layers_per_worker + i) % n_layers for i in range(layers_per_worker)]
                for w in range(self.workers)]
        spans = self.pool.map(_pool_work, jobs, chunksize=1)
        return max(e for _, e in spans) - min(s for s, _ in spans)

    def close(self):
        self.pool.close()
        self.pool.join()


def host_cores():
    return len(os.sched_getaffinity(0))


def oracle_single_core(cfg, n_layers=1):
    """Seconds of the oracle for `n_layers` layers in this process with one BLAS thread."""
    from threadpoolctl import threadpool_limits
    from lava_workloads import generate_layer
    tensors = [generate_layer(cfg, l, "cpu") for l in range(n_layers)]
    with threadpool_limits(limits=1):
        t0 = time.perf_counter()
        for t in tensors:
            _oracle_layer(cfg, t)
        return time.perf_counter() - t0


def run_reference(args, rank):
    """The reference arm of this tier: the fp64 CPU oracle, as it stands, on the host cores.
    One step = the oracle over a bounded sample of the workload's layers, one layer stream per
    core; `ms_per_step` is the measured time of that sample and `model_ms_extrapolated` scales it
    linearly to all layers (the layers are independent problems of equal size)."""
    if rank != 0:
        return
    from lava_workloads import get_config
    cfg = get_config(args.workload)
    workers = max(1, min(host_cores(), cfg.n_layers))
    per_worker = 1
    sample_layers = workers * per_worker
    pool = OraclePool(cfg.name, workers)
    try:
        for _ in range(args.warmup):
            pool.run(per_worker, cfg.n_layers)
        times = [pool.run(per_worker, cfg.n_layers) for _ in range(args.steps)]
    finally:
        pool.close()
    t_step = sum(times) / len(times)
    t_model = t_step * cfg.n_layers / sample_layers
    value = cfg.total_tokens / t_model
    sample = ("%d of %d layers per step (one per core, %d cores), scaled linearly to the model"
              % (sample_layers, cfg.n_layers, workers))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": t_step * 1e3,
        "model_ms_extrapolated": t_model * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": {"workload": cfg.name, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": workers, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------- further paths
def run_next_path(args, cfg, plan, q, k, v, stream, steps, warmup, local_rank, rank, world):
    """The layer-by-layer cascade (Algorithm 2) or the decode-time consumer of the packed cache,
    timed like the headline path (CUDA events, clocks sampled, one JSON line)."""
    import torch
    import paper_2509_09754_b200 as lava
    from paper_2509_09754_b200 import replicas

    L, d = cfg.n_layers, cfg.head_dim
    es = 2 if cfg.dtype == "bf16" else 4
    rows = int(plan.total_budget.sum().item())
    peak, peak_src = measured_hbm_peak()
    kv_bytes, out_bytes = roofline_bytes(cfg)
    if args.path == "cascade":
        cas = lava.Cascade(plan.desc, L, rows, kv_dtype=q.dtype, device=q.device)

        def step():
            cas.begin(plan.total_budget, stream)
            for l in range(L):
                cas.step(q[l], k[l], v[l], stream=stream)
        metric, unit, units = "context tokens/s per layer-by-layer eviction (Algorithm 2)", UNIT, cfg.total_tokens
        alg_bytes = kv_bytes + out_bytes
        note = ("K + V read once + the final packed cache; every step also re-evicts all lower "
                "layers (rows moved once per step), which this figure does not credit")
        workspace = cas.workspace
    else:
        dev = q.device
        gen = torch.Generator(device="cpu").manual_seed(3)
        q_new = torch.randn((L, cfg.batch, cfg.n_q_heads, d), generator=gen).to(q.dtype).to(dev)
        out = torch.empty((L, cfg.batch, cfg.n_q_heads, d), dtype=torch.float32, device=dev)
        ws = torch.empty(max(256, lava.lava_decode_workspace_bytes(plan.desc, L)), dtype=torch.uint8,
                         device=dev)

        def step():
            lava.lava_decode_attention_layers(plan.desc, L, q_new, plan.k_out, plan.v_out,
                                              plan.head_offsets, plan.layer_row_offset, out, ws, stream)
        metric, unit, units = "cached KV rows/s read by one decode step over all layers", "rows/s", rows
        alg_bytes = rows * 2 * d * es
        note = "one K row and one V row per retained (KV head, position), read once for the whole query group"
        workspace = plan.workspace
    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    sampler = ClockSampler(visible_gpu_index(local_rank))
    launches0 = lava.lava_launch_count()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    sampler.start()
    ev[0].record(stream)
    for i in range(steps):
        step()
        ev[i + 1].record(stream)
    torch.cuda.synchronize()
    clocks = sampler.stop()
    status = lava.lava_poll_status(workspace)
    if status != 0:
        raise SystemExit("device status word %d" % status)
    per_step = sorted(ev[i].elapsed_time(ev[i + 1]) for i in range(steps))
    ms = replicas.slowest_rank_ms(ev[0].elapsed_time(ev[steps])) / steps
    gbs = alg_bytes / (ms * 1e-3) / 1e9
    if rank == 0:
        print(json.dumps({
            "metric": metric, "value": replicas.whole_job_units(units) / (ms * 1e-3), "unit": unit,
            "n_gpus": world, "steps": steps, "warmup": warmup, "ms_per_step": ms,
            "ms_per_step_median": statistics.median(per_step), "ms_per_step_min": per_step[0],
            "ms_per_step_max": per_step[-1], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
            "config": {"workload": cfg.name, "path": args.path, "n_layers": L,
                       "seq_lens": list(cfg.seq_lens), "packed_rows": rows,
                       "l2": "the packed cache and the inputs exceed the 126 MB L2; no flush"
                             if alg_bytes > 126e6 else "working set below L2: not an HBM number"},
            "roofline": {"bound": "hbm", "achieved": gbs, "peak": peak, "unit": "GB/s",
                         "frac": gbs / peak, "traffic": None, "peak_source": peak_src,
                         "algorithmic_bytes": alg_bytes, "note": note},
            "e2e": None, "cpu_baseline": None,
            "gpu_launches": lava.lava_launch_count() - launches0, "clocks": clocks}), flush=True)


# ----------------------------------------------------------------------------- CUDA arm
def main():
    args = parse_args()
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        run_reference(args, rank)
        return

    import torch
    import torch.distributed as dist
    import paper_2509_09754_b200 as lava
    from paper_2509_09754_b200 import replicas
    from lava_workloads import generate_layer, get_config

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (the hot path has no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)
    lava.load_library()

    cfg = get_config(args.workload)
    if args.layers > 0:
        cfg = cfg.scaled(n_layers=min(args.layers, cfg.n_layers))
    steps, warmup = max(1, args.steps), max(3, args.warmup)
    tdt = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
    L, hkv, hq, d, w, T = (cfg.n_layers, cfg.n_kv_heads, cfg.n_q_heads, cfg.head_dim, cfg.window,
                           cfg.total_tokens)
    q = torch.empty((L, cfg.batch, hq, w, d), dtype=tdt, device=dev)
    k = torch.empty((L, hkv, T, d), dtype=tdt, device=dev)
    v = torch.empty((L, hkv, T, d), dtype=tdt, device=dev)
    cu = None
    for l in range(L):
        t = generate_layer(cfg, l, dev)
        q[l], k[l], v[l] = t["q_win"], t["k"], t["v"]
        cu = t["cu_seqlens"]
        del t
    desc = lava.LayerDesc.for_tensors(q[0], k[0], v[0], w, cfg.pool_kind, cfg.pool_kernel,
                                      cu_seqlens=cu if cfg.batch > 1 else None,
                                      max_seqlen=max(cfg.seq_lens))
    budgets = [cfg.total_budget(b) for b in range(cfg.batch)]
    plan = lava.EvictionPlan.create(desc, L, budgets, cfg.seq_lens, device=dev, kv_dtype=tdt)
    mode = lava.LAVA_BUDGET_DYNAMIC if cfg.dynamic_layers else lava.LAVA_BUDGET_UNIFORM
    stream = torch.cuda.current_stream()

    def step(events=None):
        dsc, nl = plan.desc, plan.n_layers
        if events is not None:
            events[0].record(stream)
        lava.lava_score_layers(dsc, nl, q, k, v, q.stride(0), k.stride(0), v.stride(0), None,
                               plan.scores, plan.vbar, plan.entropy, plan.workspace, stream)
        if events is not None:
            events[1].record(stream)
        lava.lava_layer_budgets(nl, dsc.batch, plan.entropy, plan.total_budget, plan.floor,
                                plan.cap, mode, plan.layer_budget, plan.layer_row_offset,
                                plan.workspace, stream)
        if events is not None:
            events[2].record(stream)
        lava.lava_select_topk_layers(dsc, nl, plan.scores, plan.layer_budget, plan.keep_idx,
                                     plan.head_offsets, plan.workspace, stream)
        if events is not None:
            events[3].record(stream)
        lava.lava_compact_kv_layers(dsc, nl, k, v, k.stride(0), v.stride(0), plan.keep_idx,
                                    plan.head_offsets, plan.layer_row_offset, plan.k_out,
                                    plan.v_out, stream)
        if events is not None:
            events[4].record(stream)

    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    status = lava.lava_poll_status(plan.workspace)
    if status != 0:
        raise SystemExit("device status word %d after warm-up" % status)

    if args.path != "evict":
        run_next_path(args, cfg, plan, q, k, v, stream, steps, warmup, local_rank, rank, world)
        return

    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(steps)]
    sampler = ClockSampler(visible_gpu_index(local_rank))
    launches0 = lava.lava_launch_count()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    sampler.start()
    t_start = torch.cuda.Event(enable_timing=True)
    t_end = torch.cuda.Event(enable_timing=True)
    t_start.record(stream)
    for i in range(steps):
        step(ev[i])
    t_end.record(stream)
    torch.cuda.synchronize()
    clocks = sampler.stop()
    if world > 1:
        dist.barrier()
    launches = lava.lava_launch_count() - launches0
    total_ms = replicas.slowest_rank_ms(t_start.elapsed_time(t_end))
    ms_per_step = total_ms / steps
    phase_ms = [sum(ev[i][j].elapsed_time(ev[i][j + 1]) for i in range(steps)) / steps
                for j in range(4)]
    per_step = sorted(ev[i][0].elapsed_time(ev[i][4]) for i in range(steps))
    value = replicas.whole_job_units(cfg.total_tokens) / (ms_per_step * 1e-3)

    kv_bytes, out_bytes = roofline_bytes(cfg)
    peak, peak_src = measured_hbm_peak()
    score_gbs = kv_bytes / (phase_ms[0] * 1e-3) / 1e9
    whole_gbs = (kv_bytes + out_bytes) / (ms_per_step * 1e-3) / 1e9
    roofline = {
        "bound": "hbm", "kernel": "lava_score_layers", "achieved": score_gbs, "peak": peak,
        "unit": "GB/s", "frac": score_gbs / peak, "traffic": committed_traffic(cfg.name),
        "peak_source": peak_src, "algorithmic_bytes_per_launch": kv_bytes,
        "whole_path": {"achieved": whole_gbs, "frac": whole_gbs / peak,
                       "frac_of_8TBs_nominal": whole_gbs / 8000.0,
                       "algorithmic_bytes": kv_bytes + out_bytes},
        "phase_ms": {"score": phase_ms[0], "budgets": phase_ms[1], "select": phase_ms[2],
                     "compact": phase_ms[3]},
    }

    # ---- end to end through the host-buffer entry point (pinned host inputs) --------------
    e2e = None
    if not args.no_e2e:
        rows = sum(budgets)
        hq_, hk_, hv_ = (torch.empty(x.shape, dtype=x.dtype, pin_memory=True) for x in (q, k, v))
        hq_.copy_(q), hk_.copy_(k), hv_.copy_(v)
        out_budget = torch.empty((L, cfg.batch), dtype=torch.int64, pin_memory=True)
        out_hoff = torch.empty((L, cfg.batch, hkv + 1), dtype=torch.int32, pin_memory=True)
        out_k = torch.empty((rows, d), dtype=tdt, pin_memory=True)
        out_v = torch.empty((rows, d), dtype=tdt, pin_memory=True)
        seq_lens = torch.tensor(cfg.seq_lens, dtype=torch.int32)
        tb = torch.tensor(budgets, dtype=torch.int64)
        arena = torch.empty(lava.lava_host_arena_bytes(desc, L, rows), dtype=torch.uint8,
                            device=dev)
        h2d = sum(x.numel() * x.element_size() for x in (hq_, hk_, hv_))
        d2h = sum(x.numel() * x.element_size() for x in (out_budget, out_hoff, out_k, out_v))

        def e2e_step():
            lava.lava_evict_model_host(desc, L, hq_, hk_, hv_, seq_lens, tb, mode, out_budget,
                                       out_hoff, out_k, out_v, arena, stream)
        e2e_step()
        torch.cuda.synchronize()
        assert torch.equal(out_budget, plan.layer_budget.cpu()), "host path disagrees"
        n_e2e = max(1, args.e2e_steps)
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(n_e2e):
            e2e_step()
        e1.record(stream)
        torch.cuda.synchronize()
        e2e_ms = e0.elapsed_time(e1) / n_e2e
        if world > 1:
            tt = torch.tensor([e2e_ms], dtype=torch.float64, device=dev)
            dist.all_reduce(tt, op=dist.ReduceOp.MAX)
            e2e_ms = float(tt.item())
        e2e = {"value": world * cfg.total_tokens / (e2e_ms * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms,
               "steps": n_e2e, "api": "lava_evict_model_host (pinned host buffers)"}
        del arena, hq_, hk_, hv_

    # ---- the oracle on this machine's host cores (rank 0, N == 1 only) -------------------------
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        workers = max(1, min(host_cores(), cfg.n_layers))
        per_worker = max(1, min(args.cpu_layers // workers, 4))
        pool = OraclePool(cfg.name, workers)
        try:
            pool.run(1, cfg.n_layers)                       # imports and first-touch, untimed
            secs = pool.run(per_worker, cfg.n_layers)
        finally:
            pool.close()
        nl = workers * per_worker
        t_model = secs * cfg.n_layers / nl
        one = oracle_single_core(cfg, 1)
        cpu_baseline = {"value": cfg.total_tokens / t_model, "unit": UNIT, "cores": workers,
                        "kind": "oracle", "seconds_measured": secs,
                        "sample": "%d layers of %s (score+entropy+select+compact), %d at a time on "
                                  "%d cores with one BLAS thread each, scaled linearly to %d layers"
                                  % (nl, cfg.name, workers, workers, cfg.n_layers),
                        "single_core": {"value": cfg.total_tokens / (one * cfg.n_layers),
                                        "unit": UNIT, "seconds_measured": one,
                                        "sample": "1 layer in-process, one BLAS thread"}}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps,
            "warmup": warmup, "ms_per_step": ms_per_step,
            "ms_per_step_median": statistics.median(per_step), "ms_per_step_min": per_step[0],
            "ms_per_step_max": per_step[-1], "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
            "config": {"workload": cfg.name, "n_layers": L, "n_q_heads": hq, "n_kv_heads": hkv,
                       "head_dim": d, "seq_lens": list(cfg.seq_lens), "window": w,
                       "pool": ["none", "max", "avg"][cfg.pool_kind] + str(cfg.pool_kernel),
                       "total_budget": budgets, "budget_mode": "dynamic" if mode == 0 else "uniform",
                       "parallelism": "replicas only (%d)" % world,
                       "l2": "inputs (%.2f GB of K,V per step) exceed the 126 MB L2; no flush"
                             % (kv_bytes / 1e9)},
            "roofline": roofline, "e2e": e2e, "cpu_baseline": cpu_baseline,
            "gpu_launches": int(launches), "clocks": clocks,
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
