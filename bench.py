#!/usr/bin/env python
"""Benchmark of the DAF prefill-attention path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--impl ours|reference]

Without --config the run covers the context range the metric is quoted on: the 32k
configuration (c3, the largest single-GPU one) is the headline (`value`, `config`,
`roofline`, `e2e`, `cpu_baseline`), and the 6k and 16k configurations (c1, c2) are
measured the same way in the same process and reported under `by_config`.

One step = one pass of the whole path (select + gather + hybrid-cache update,
important-token attention, question-document attention with the fusion done by
the epilogues) over every layer of the workload, each layer with its own seeded
synthetic tensors already resident in HBM.  Prints ONE JSON line.

metric: microseconds per layer (lower is better); the same run also reports the
algorithmic TFLOP/s, the roofline of the dominant kernel, the full-recompute
comparison, an end-to-end figure through the host-buffer entry point, and the
CPU oracle timed on this machine's cores.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2607_21599_b200 import workloads as W  # noqa: E402

METRIC = "daf_prefill_attention_us_per_layer"
UNIT = "us/layer"

Q_IN_PLACE_MIN_K = 16384    # from this many important tokens on, the layer is called without a packed-Q buffer
# DRAM bytes per launch of the dominant kernel (the joint attention launch), dram__bytes_read.sum +
# dram__bytes_write.sum of the committed ncu capture of that workload; no entry where none was captured.
NCU_TRAFFIC_BYTES = {"c1": 21746944, "c2": 93970176, "c3": 148794368}
DEFAULT_PRIMARY, DEFAULT_OTHERS = "c3", ("c1", "c2")


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"bf16_tflops": float(d["bf16_tflops"]), "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", 0)),
                "hbm_gbs": float(d["hbm_gbs"]), "source": "measured"}
    return {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read only) while the timed region runs."""

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._nv = None

    def _run(self):
        nv = self._nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
        }
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                try:
                    mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
                except Exception:
                    mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
                for n, bit in names.items():
                    if mask & bit:
                        self.reasons.add(n)
            except Exception:
                pass
            time.sleep(0.002)

    def __enter__(self):
        if self._nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        return {"sm_mhz": int(statistics.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def _dist_env():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))


def replica_layers(rank: int, w: W.Workload):
    """Layer seeds of rank `rank`: every rank owns its own replica of the workload (weak scaling, no exchange)."""
    return [rank * w.layers + i for i in range(w.layers)]


def max_over_ranks(dist, value: float, device) -> float:
    """A duration is reported as the maximum over ranks (single process: the value itself)."""
    if dist is None:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def _config_dict(w: W.Workload, n_gpus: int):
    return {"workload": f"{w.name}: {w.layers} layers, Hq={w.n_q_heads} Hkv={w.n_kv_heads} D={w.head_dim}, "
                        f"L_d={w.L_d} ({w.n_docs} docs of {w.doc_len}), L_q={w.L_q}, r={w.r} (k={w.k}), "
                        f"{w.selection} importance scores",
            "layers": w.layers, "L_d": w.L_d, "L_q": w.L_q, "r": w.r, "k": w.k,
            "n_q_heads": w.n_q_heads, "n_kv_heads": w.n_kv_heads, "head_dim": w.head_dim,
            "parallelism": f"replicas x{n_gpus} (no data-path collective)",
            "l2_policy": "inputs larger than L2: every layer has its own tensors, a step touches far more than 126 MB"}


# ----------------------------------------------------------------------------- the CPU oracle, timed
ORACLE_PAIR_BUDGET = 6.0e7     # (row, key, head) triples per timed oracle call: about a second on 16 cores


def _host_arrays(L):
    f = lambda t: t.float().cpu().numpy()  # noqa: E731
    return {n: (None if t is None else (f(t) if t.dtype == torch.bfloat16 else t.cpu().numpy())) for n, t in L.items()}


def oracle_layer_seconds(oracle, A, w: W.Workload):
    """Times the oracle, as it stands, on one layer.  Small layers run whole (oracle.daf_layer).  Layers
    whose attention would take much longer than a second run selection, gather and cache update in full and
    the two attention stages on every s-th query row; the attention time is scaled by the share of the
    visible (row, key) pairs that the sampled rows cover.  Returns (seconds for the whole layer, description)."""
    pairs = W.attention_pairs(w)
    triples = (pairs["important"] + pairs["question"]) * w.n_q_heads
    if triples <= ORACLE_PAIR_BUDGET:
        t0 = time.perf_counter()
        oracle.daf_layer(A["q_fresh"], A["k_fresh"], A["v_fresh"], A["k_cached"], A["v_cached"], w.L_d, w.L_q,
                         w.softmax_scale, scores=A["scores"], idx=A["idx_in"], r=w.r)
        return time.perf_counter() - t0, "whole layer"
    import numpy as np
    stride = int(math.ceil(triples / ORACLE_PAIR_BUDGET))
    t0 = time.perf_counter()
    k = oracle.num_important(w.L_d, w.r)
    idx = oracle.select(A["scores"], k) if A["scores"] is not None else A["idx_in"]
    q_pack, k_pack, v_pack = (oracle.gather_rows(A[n], idx) for n in ("q_fresh", "k_fresh", "v_fresh"))
    kv_k = oracle.hybrid_kv(A["k_cached"], A["k_fresh"], idx, w.L_d, w.L_q)
    kv_v = oracle.hybrid_kv(A["v_cached"], A["v_fresh"], idx, w.L_d, w.L_q)
    t_move = time.perf_counter() - t0
    rows_i = np.arange(stride // 2, k, stride, dtype=np.int32)
    rows_q = np.arange(min(stride // 2, w.L_q - 1), w.L_q, stride, dtype=np.int32)
    t0 = time.perf_counter()
    oracle.important_attn(q_pack, k_pack, v_pack, w.softmax_scale, rows=rows_i)
    oracle.qd_attn(A["q_fresh"][w.L_d:], kv_k, kv_v, w.L_d, w.softmax_scale, rows=rows_q)
    t_attn = time.perf_counter() - t0
    covered = int((rows_i.astype(np.int64) + 1).sum()) + int((rows_q.astype(np.int64) + 1 + w.L_d).sum())
    share = covered / float(pairs["important"] + pairs["question"])
    return t_move + t_attn / share, (f"selection, gather and cache update in full; attention on every {stride}th query row "
                                    f"({share:.3%} of the visible pairs), attention time scaled by that share (extrapolated)")


# ----------------------------------------------------------------------------- reference arm (the CPU oracle)
def run_reference(args, w: W.Workload):
    rank, _, world = _dist_env()
    if rank != 0:
        return
    import oracle
    cores = oracle.num_threads()
    n_layers = min(w.layers, max(1, min(args.steps + args.warmup, 4)))
    arrs = [_host_arrays(W.make_layer(w, i)) for i in range(n_layers)]
    how = ""
    for i in range(args.warmup):
        oracle_layer_seconds(oracle, arrs[i % n_layers], w)
    total = 0.0
    for i in range(args.steps):
        dt, how = oracle_layer_seconds(oracle, arrs[(args.warmup + i) % n_layers], w)
        total += dt
    us_per_layer = total / args.steps * 1e6
    sample = f"each step = one layer of {w.name} through the fp64 CPU oracle ({cores} OpenMP threads): {how}"
    line = {"impl": "reference", "metric": METRIC, "value": us_per_layer, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": total / args.steps * 1e3,
            "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": _config_dict(w, args.gpus),
            "cpu_baseline": {"value": us_per_layer, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": us_per_layer, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ----------------------------------------------------------------------------- our arm
class LayerBuffers:
    """Device tensors of one layer plus the outputs the library writes."""

    def __init__(self, w: W.Workload, layer: int, api, dev):
        L = W.make_layer(w, layer, dev)
        self.L = L
        N, Hq, Hkv = w.N, w.n_q_heads, w.n_kv_heads
        k = api.daf_num_important(w.L_d, w.r)
        self.k = k
        bf = torch.bfloat16
        self.kv_k = torch.empty(N, Hkv, 128, dtype=bf, device=dev)
        self.kv_v = torch.empty(N, Hkv, 128, dtype=bf, device=dev)
        self.kv_k[: w.L_d] = L["k_cached"]
        self.kv_v[: w.L_d] = L["v_cached"]
        self.kv_k[w.L_d:] = 0
        self.kv_v[w.L_d:] = 0
        self.idx_out = torch.zeros(max(k, 1), dtype=torch.int32, device=dev)
        self.q_pack = torch.empty(max(k, 1), Hq, 128, dtype=bf, device=dev)
        self.k_pack = torch.empty(max(k, 1), Hkv, 128, dtype=bf, device=dev)
        self.v_pack = torch.empty(max(k, 1), Hkv, 128, dtype=bf, device=dev)
        self.hidden = torch.empty(k + w.L_q, Hq, 128, dtype=bf, device=dev)
        self.idx_sel = torch.zeros(max(k, 1), dtype=torch.int32, device=dev)     # positions from the hoisted selection
        self.n_sig = 0 if L["scores"] is None else L["scores"].shape[0]


class Env:
    """What every measured configuration shares: the device, the rank plumbing, the library, the peaks."""

    def __init__(self, args):
        self.args = args
        self.rank, self.local_rank, self.world = _dist_env()
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device: the DAF library has no CPU fallback")
        torch.cuda.set_device(self.local_rank)
        self.dev = torch.device("cuda", self.local_rank)
        self.dist = None
        if self.world > 1:
            import torch.distributed as dist_mod
            self.dist = dist_mod
            self.dist.init_process_group("nccl", device_id=self.dev)
        from paper_2607_21599_b200 import api, build
        if self.rank == 0 or self.world == 1:
            build.build()
        if self.dist is not None:
            self.dist.barrier()
        api.lib()
        self.api = api
        self.peaks = _peaks()
        self.use_graph = not args.no_graph

    def barrier(self):
        torch.cuda.synchronize()
        if self.dist is not None:
            self.dist.barrier()
            torch.cuda.synchronize()


def measure_config(env: Env, w: W.Workload, primary: bool):
    """All measurements of one workload.  Returns the fields of the JSON line that belong to it."""
    args, api, dev, dist, rank, world, peaks = env.args, env.api, env.dev, env.dist, env.rank, env.world, env.peaks
    use_graph, barrier = env.use_graph, env.barrier
    p = api.make_params(w.L_d, w.L_q, w.r, w.n_q_heads, w.n_kv_heads)
    ws = api.alloc_workspace(p, dev)
    # every rank owns its own replica of the workload (distinct seeds per rank): weak scaling, no exchange
    bufs = [LayerBuffers(w, layer, api, dev) for layer in replica_layers(rank, w)]
    torch.cuda.synchronize()
    Hq = w.n_q_heads
    row_bytes = Hq * 256

    # All launches below go to torch's current stream (the capture stream while a graph is recorded).
    # With both stages present the layer needs no packed copy of the Q rows: step 2 can read them in place.
    # That saves most of the gather traffic but costs each work item a scattered fetch of its Q rows; measured
    # on B200 the layer time changes by -2 % (k = 41780), +-1 % (k = 6554) and +10 % (k = 922), so only very
    # long condensed sequences are run that way.
    both = w.k > 0 and w.L_q > 0
    q_in_place = both and w.k >= Q_IN_PLACE_MIN_K
    # Likewise the K/V rows of step 2 (--kv-in-place; slower, for comparison): the attention kernel fetches them
    # through the positions and the kernel in front of it only updates the hybrid cache.
    kv_in_place = both and args.kv_in_place

    def layer_call(b: LayerBuffers):
        L = b.L
        api.check(api.daf_layer(p, L["scores"], b.n_sig, L["idx_in"], L["q_fresh"], L["k_fresh"], L["v_fresh"], b.kv_k,
                                b.kv_v, b.idx_out, None if q_in_place else b.q_pack, None if kv_in_place else b.k_pack,
                                None if kv_in_place else b.v_pack, b.hidden, None, ws),
                  "daf_layer")

    def st_select(b, pack_q=False):
        L = b.L
        api.check(api.daf_select(p, L["scores"], b.n_sig, L["idx_in"], L["q_fresh"], L["k_fresh"], L["v_fresh"],
                                 b.kv_k, b.kv_v, b.idx_out, b.q_pack if (pack_q or not q_in_place) else None, b.k_pack, b.v_pack,
                                 ws), "daf_select")

    def st_imp(b):
        api.check(api.daf_important_attn(p, b.k, b.q_pack, b.k_pack, b.v_pack, b.hidden, row_bytes, None, None, ws),
                  "daf_important_attn")

    def st_qd(b):
        api.check(api.daf_qd_attn(p, b.L["q_fresh"][w.L_d:], b.kv_k, b.kv_v, b.hidden, row_bytes, None, None, ws,
                                  out_offset_bytes=b.k * row_bytes), "daf_qd_attn")

    def st_both_launches(which):
        def run(b):
            api.check(api.daf_imp_qd_attn_launches(p, None if q_in_place else b.q_pack, b.L["q_fresh"], b.k_pack, b.v_pack,
                                                   b.L["q_fresh"][w.L_d:], b.kv_k, b.kv_v, b.idx_out, b.hidden, ws, which),
                      "daf_imp_qd_attn_launches")
        return run

    n_full = min(len(bufs), 4)
    pf = api.make_params(w.N, 0, 1.0, w.n_q_heads, w.n_kv_heads)
    wsf = api.alloc_workspace(pf, dev)
    full_out = torch.empty(w.N, Hq, 128, dtype=torch.bfloat16, device=dev)

    def st_full(b):
        api.check(api.daf_full_causal_attn(pf, w.N, b.L["q_fresh"], b.L["k_fresh"], b.L["v_fresh"], full_out, None,
                                           wsf), "daf_full_causal_attn")

    def over(fn, items):
        def run():
            for b in items:
                fn(b)
        return run

    def capture(run):
        """Records `run` (one pass over the layers) into a CUDA graph: a replay issues the same kernels
        with the same arguments without host-side launch cost between them."""
        launches_before = api.daf_launch_count()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            run()
        return g, api.daf_launch_count() - launches_before

    def time_replays(g, reps):
        stream = torch.cuda.current_stream()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(reps):
            g.replay()
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps  # ms per replay

    # The selection of a layer depends only on that layer's scores (in the method they come from the signal layers,
    # long before the layer is reached), so the step schedules the selections of all layers on a second stream:
    # they run beside the attention of earlier layers, and each layer proper (gather, cache update, both attention
    # stages, fusion) starts from the positions its selection left.  Every kernel of the path still runs, and
    # is timed, once per layer per step.  --no-overlap keeps everything on one stream.
    overlap = (not args.no_overlap) and w.k > 0 and bufs[0].L["scores"] is not None
    side = torch.cuda.Stream(device=dev) if overlap else None

    def step_overlapped():
        main = torch.cuda.current_stream()
        side.wait_stream(main)
        events = []
        for b in bufs:
            api.check(api.daf_select_topk(p, b.L["scores"], b.n_sig, b.idx_sel, ws, stream=side), "daf_select_topk")
            e = torch.cuda.Event()
            e.record(side)
            events.append(e)
        for b, e in zip(bufs, events):
            main.wait_event(e)
            L = b.L
            api.check(api.daf_layer(p, None, 0, b.idx_sel, L["q_fresh"], L["k_fresh"], L["v_fresh"], b.kv_k, b.kv_v, b.idx_out,
                                    None if q_in_place else b.q_pack, None if kv_in_place else b.k_pack,
                                    None if kv_in_place else b.v_pack, b.hidden, None, ws, stream=main),
                      "daf_layer")
        main.wait_stream(side)

    step = step_overlapped if overlap else over(layer_call, bufs)
    for _ in range(max(args.warmup, 3)):     # eager warm-up: also sets function attributes before capture
        step()
    barrier()
    api.check(api.daf_poll_status(ws), "warm-up (device status)")

    launches_per_step = 0
    if use_graph:
        g_step, launches_per_step = capture(step)
        g_step.replay()
        barrier()

    stream = torch.cuda.current_stream()
    launches0 = api.daf_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(env.local_rank) as clocks:
        barrier()
        e0.record(stream)
        marks = []                      # one event after every step (on the same stream: they cost nothing measurable)
        for _ in range(args.steps):
            if use_graph:
                g_step.replay()
            else:
                step()
            m = torch.cuda.Event(enable_timing=True)
            m.record(stream)
            marks.append(m)
        e1.record(stream)
        barrier()
    ms_total = e0.elapsed_time(e1)
    step_ms = [a.elapsed_time(b) for a, b in zip([e0] + marks[:-1], marks)]
    launches = launches_per_step * args.steps if use_graph else api.daf_launch_count() - launches0
    api.check(api.daf_poll_status(ws), "timed region (device status)")
    ms_total = max_over_ranks(dist, ms_total, dev)
    ms_per_step = ms_total / args.steps
    us_per_layer = ms_per_step * 1e3 / (w.layers * world)

    flops = W.attention_flops(w)
    daf_flops = flops["important"] + flops["question"]
    tflops = daf_flops * w.layers * world / (ms_per_step * 1e-3) / 1e12

    # ---- per-stage timings: each stage's launches over all layers, replayed back to back (us per layer)
    def time_stage(fn, items, reps=5):
        run = over(fn, items)
        run()
        torch.cuda.synchronize()
        if use_graph:
            g, _ = capture(run)
            g.replay()
            torch.cuda.synchronize()
            return time_replays(g, reps) * 1e3 / len(items)
        stream2 = torch.cuda.current_stream()
        a, z = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream2)
        for _ in range(reps):
            run()
        z.record(stream2)
        torch.cuda.synchronize()
        return a.elapsed_time(z) / reps * 1e3 / len(items)

    dev_scores = torch.empty(w.L_d, dtype=torch.float32, device=dev)

    def st_dev(b):
        api.check(api.daf_deviation_scores(p, b.L["k_fresh"], b.L["v_fresh"], b.L["k_cached"], b.L["v_cached"],
                                           dev_scores), "daf_deviation_scores")

    # the signal of three layers aggregated in one pass (what daf_select_from_kv runs ahead of the top-k): timed
    # alone through that entry point with r = 0 and no question rows, so that nothing else is launched
    n_sig_layers = min(3, len(bufs))
    p_sig = api.make_params(w.L_d, 0, 0.0, w.n_q_heads, w.n_kv_heads)
    ws_sig = api.alloc_workspace(p_sig, dev)

    def st_dev_sum(b):
        i = bufs.index(b)
        grp = [bufs[(i + j) % len(bufs)].L for j in range(n_sig_layers)]
        api.check(api.daf_select_from_kv(p_sig, [g["k_fresh"] for g in grp], [g["v_fresh"] for g in grp],
                                         [g["k_cached"] for g in grp], [g["v_cached"] for g in grp], None, None, None, None,
                                         None, None, None, None, None, dev_scores, ws_sig), "daf_select_from_kv (signal only)")

    us_layer_one_stream = time_stage(layer_call, bufs)     # the whole layer from scores on one stream, for comparison
    for b in bufs:                       # the stand-alone important-token stage below reads packed Q rows
        st_select(b, pack_q=True)
    us_dev = time_stage(st_dev, bufs)
    us_dev_sum = time_stage(st_dev_sum, bufs)
    us_select = time_stage(st_select, bufs)
    us_imp = time_stage(st_imp, bufs) if w.k > 0 else 0.0
    us_qd = time_stage(st_qd, bufs) if w.L_q > 0 else 0.0
    # the two attention stages the way the layer runs them: one launch over both stages' work items and one merge
    # launch; each launch is also timed alone (the attention launch writes the partial rows the merge launch reads)
    if both:
        with ClockSampler(env.local_rank) as clocks_attn:
            us_kernel = time_stage(st_both_launches(1), bufs)
        us_merge = time_stage(st_both_launches(2), bufs)
        us_both = time_stage(st_both_launches(3), bufs)
    else:
        clocks_attn = clocks
        us_kernel, us_merge, us_both = us_imp + us_qd, 0.0, us_imp + us_qd
    # full recompute on the same kernel (comparison path), bounded number of layers
    with ClockSampler(env.local_rank) as clocks_full:
        us_full = time_stage(st_full, bufs[:n_full], reps=3)
    # selective recomputation over the FULL context on the same kernel (the r L_d^2 + L_d L_q scheme of the
    # paper's complexity analysis): the compact rows attend every earlier key of the hybrid cache
    blend = None
    if primary or args.config is not None:
        blend_pairs = 0
        for b in bufs[:n_full]:
            pos = torch.cat([b.idx_out[: b.k], torch.arange(w.L_d, w.N, dtype=torch.int32, device=dev)])
            b.row_pos = pos.contiguous()
            b.q_rows = b.L["q_fresh"][pos.long()].contiguous()
            blend_pairs += int((pos.long() + 1).sum().item())
        blend_out = torch.empty(w.k + w.L_q, Hq, 128, dtype=torch.bfloat16, device=dev)

        def st_blend(b):
            api.check(api.daf_blend_attn(p, w.k + w.L_q, b.q_rows, b.kv_k, b.kv_v, b.row_pos, blend_out, row_bytes, None,
                                         ws), "daf_blend_attn")

        us_blend = time_stage(st_blend, bufs[:n_full], reps=3)
        blend_flops = 4.0 * w.head_dim * Hq * blend_pairs / n_full
        blend = {"us_per_layer": us_blend, "tflops": blend_flops / (us_blend * 1e-6) / 1e12,
                 "flop_ratio_vs_daf": blend_flops / daf_flops,
                 "time_ratio_vs_daf_attention": us_blend / max(us_both, 1e-9),
                 "note": "comparison only: important + question rows attend the whole hybrid cache"}
    # the same layers from an offline cache stored in fp8 (one byte per element, one scale per KV head): the cache
    # is expanded into one reused bf16 buffer pair per layer, then the layer runs as above
    fp8 = None
    if hasattr(torch, "float8_e4m3fn"):
        n_f8 = min(len(bufs), 8)
        kv8_k, kv8_v = bufs[0].kv_k, bufs[0].kv_v                       # the reused hybrid-cache buffers
        ones = torch.ones(w.n_kv_heads, dtype=torch.float32, device=dev)
        for b in bufs[:n_f8]:
            b.k8 = b.L["k_cached"].float().to(torch.float8_e4m3fn).view(torch.uint8)
            b.v8 = b.L["v_cached"].float().to(torch.float8_e4m3fn).view(torch.uint8)

        def st_layer_fp8(b):
            L = b.L
            api.check(api.daf_layer_fp8(p, L["scores"], b.n_sig, L["idx_in"], L["q_fresh"], L["k_fresh"], L["v_fresh"], b.k8, b.v8,
                                        ones, ones, kv8_k, kv8_v, b.idx_out, None if q_in_place else b.q_pack, b.k_pack, b.v_pack,
                                        b.hidden, None, ws), "daf_layer_fp8")

        def st_layer_bf16(b):
            layer_call(b)

        us_f8 = time_stage(st_layer_fp8, bufs[:n_f8])
        us_b16 = time_stage(st_layer_bf16, bufs[:n_f8])

        # The offline cache is known long before its layer is reached, so its expansion can run ahead: layer i + 1's
        # cache is expanded on a second stream into the other of TWO bf16 buffer pairs while layer i runs from the first.
        pairs_kv = [(kv8_k, kv8_v), (torch.empty_like(kv8_k), torch.empty_like(kv8_v))]
        side8 = torch.cuda.Stream(device=dev)

        def run_fp8_ahead():
            main = torch.cuda.current_stream()
            side8.wait_stream(main)
            layer_done = [None, None]            # last layer that read each buffer pair
            for i, b in enumerate(bufs[:n_f8]):
                kk, vv = pairs_kv[i & 1]
                if layer_done[i & 1] is not None:
                    side8.wait_event(layer_done[i & 1])
                api.check(api.daf_expand_fp8_cache(p, b.k8, b.v8, ones, ones, kk, vv, stream=side8), "daf_expand_fp8_cache")
                ready = torch.cuda.Event()
                ready.record(side8)
                main.wait_event(ready)
                L = b.L
                api.check(api.daf_layer(p, L["scores"], b.n_sig, L["idx_in"], L["q_fresh"], L["k_fresh"], L["v_fresh"], kk, vv,
                                        b.idx_out, None if q_in_place else b.q_pack, b.k_pack, b.v_pack, b.hidden, None, ws,
                                        stream=main), "daf_layer")
                done = torch.cuda.Event()
                done.record(main)
                layer_done[i & 1] = done
            main.wait_stream(side8)

        run_fp8_ahead()
        torch.cuda.synchronize()
        if use_graph:
            g8, _ = capture(run_fp8_ahead)
            g8.replay()
            torch.cuda.synchronize()
            us_f8_ahead = time_replays(g8, 5) * 1e3 / n_f8
        else:
            us_f8_ahead = None
        cache_bytes = 2 * w.L_d * w.n_kv_heads * 128
        fp8 = {"us_per_layer": us_f8, "bf16_us_per_layer_same_layers": us_b16, "layers_timed": n_f8,
               "us_per_layer_expanded_ahead": us_f8_ahead,
               "offline_cache_bytes_per_layer": cache_bytes, "bf16_offline_cache_bytes_per_layer": 2 * cache_bytes,
               "expansion_bytes_per_layer": 3 * cache_bytes,
               "note": "offline document cache kept in e4m3 + one scale per KV head; expanded per layer into one reused "
                       "bf16 buffer pair, the selection kernel running beside the expansion (us_per_layer); or expanded "
                       "one layer ahead on a second stream into the other of two buffer pairs (us_per_layer_expanded_ahead)"}
        del pairs_kv
        for b in bufs[:n_f8]:                 # the first layer's cache buffers were used as the shared pair
            del b.k8, b.v8
        bufs[0].kv_k[: w.L_d] = bufs[0].L["k_cached"]
        bufs[0].kv_v[: w.L_d] = bufs[0].L["v_cached"]
    api.check(api.daf_poll_status(wsf), "full recompute (device status)")
    api.check(api.daf_poll_status(ws), "stage timing (device status)")

    imp_tflops = flops["important"] / (us_imp * 1e-6) / 1e12 if us_imp else 0.0
    qd_tflops = flops["question"] / (us_qd * 1e-6) / 1e12 if us_qd else 0.0
    full_tflops = flops["full"] / (us_full * 1e-6) / 1e12
    packed_heads = 2 * w.n_kv_heads + (0 if q_in_place else w.n_q_heads)     # heads of a packed row
    gather_bytes = 2 * w.k * packed_heads * 256 + (w.k + 2 * w.L_q) * 2 * w.n_kv_heads * 256
    dev_bytes = 4 * w.L_d * w.n_kv_heads * 256 + 4 * w.L_d

    kernel_tflops = daf_flops / (us_kernel * 1e-6) / 1e12 if us_kernel else 0.0
    both_tflops = daf_flops / (us_both * 1e-6) / 1e12 if us_both else 0.0
    pairs = W.attention_pairs(w)
    roofline = {
        "kernel": "attn_fwd_kernel, the launch a layer makes: important-token and question work items in one grid",
        "bound": "tensor",
        "flops_per_launch": daf_flops,
        "flops_formula": f"4*D*Hq*pairs = 4*128*{Hq}*({pairs['important']} + {pairs['question']})",
        "kernel_us": us_kernel, "merge_us": us_merge, "kernel_plus_merge_us": us_both,
        "achieved": kernel_tflops,
        "peak": peaks["bf16_tflops"],
        "unit": "TFLOP/s",
        "frac": kernel_tflops / peaks["bf16_tflops"],
        "frac_with_merge": both_tflops / peaks["bf16_tflops"],
        "frac_of_sustained_peak": (kernel_tflops / peaks["bf16_tflops_sustained"]) if peaks.get("bf16_tflops_sustained") else None,
        "peak_source": f"{peaks['source']} bf16 burst (kernel timed alone, all layers back to back)",
        "traffic": NCU_TRAFFIC_BYTES.get(w.name),
        "clocks": clocks_attn.summary(),
    }

    # ---- end to end through the host-buffer entry point (pinned host tensors, copies inside the timed region)
    e2e = None
    if primary and (rank == 0 or world > 1):
        per_layer_in = (w.N * (w.n_q_heads + 2 * w.n_kv_heads) + 2 * w.L_d * w.n_kv_heads) * 256 + \
                       (w.L_d * 4 * max(bufs[0].n_sig, 1))
        n_e2e = max(1, min(w.layers, int(2e9 // per_layer_in)))
        # two arenas and two streams: the copies in of layer i + 1 run beside the kernels and the copies out of layer i
        arenas = [torch.zeros(api.daf_layer_host_arena_bytes(p), dtype=torch.uint8, device=dev) for _ in range(2)]
        lanes = [torch.cuda.Stream(device=dev) for _ in range(2)]
        host = []
        for b in bufs[:n_e2e]:
            h = {n: (None if t is None else t.cpu().pin_memory()) for n, t in b.L.items()}
            h["kv_k"] = torch.zeros(w.N, w.n_kv_heads, 128, dtype=torch.bfloat16).pin_memory()
            h["kv_v"] = torch.zeros(w.N, w.n_kv_heads, 128, dtype=torch.bfloat16).pin_memory()
            h["kv_k"][: w.L_d] = h["k_cached"]
            h["kv_v"][: w.L_d] = h["v_cached"]
            h["hidden"] = torch.empty(b.k + w.L_q, Hq, 128, dtype=torch.bfloat16).pin_memory()
            h["n_sig"] = b.n_sig
            host.append(h)

        def e2e_step():
            pending = None
            for i, h in enumerate(host):
                lane = i & 1
                api.check(api.daf_layer_host_begin(p, h["scores"], h["n_sig"], h["idx_in"], h["q_fresh"], h["k_fresh"],
                                                   h["v_fresh"], h["kv_k"], h["kv_v"], 0, h["hidden"], None, arenas[lane],
                                                   stream=lanes[lane]), "daf_layer_host_begin")
                if pending is not None:
                    api.check(api.daf_layer_host_end(p, arenas[pending], stream=lanes[pending]), "daf_layer_host_end")
                pending = lane
            api.check(api.daf_layer_host_end(p, arenas[pending], stream=lanes[pending]), "daf_layer_host_end")

        e2e_steps = max(1, min(args.steps, 5))
        e2e_step()
        barrier()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            e2e_step()
        torch.cuda.synchronize()
        dt = time.perf_counter() - t0
        dt = max_over_ranks(dist, dt, dev)
        # what crosses the link per layer: the scores, the document rows of the offline cache, the question's Q rows
        # (copies) and the fresh Q/K/V rows of the important tokens and K/V rows of the question, which the gather /
        # cache-update kernel reads straight from the pinned host tensors; the rest of the fresh tensors stays on the host
        kv_row = 2 * w.n_kv_heads * 256
        crossing = (w.L_d * 4 * max(bufs[0].n_sig, 1) + w.L_d * kv_row + w.L_q * row_bytes +
                    w.k * (row_bytes + kv_row) + w.L_q * kv_row)
        e2e = {"value": dt / e2e_steps / (n_e2e * world) * 1e6, "unit": UNIT,
               "h2d_bytes_per_step": int(crossing * n_e2e), "d2h_bytes_per_step": int((w.k + w.L_q) * row_bytes * n_e2e),
               "host_input_bytes_per_step": int(per_layer_in * n_e2e),
               "layers_per_step": n_e2e, "steps": e2e_steps,
               "api": "daf_layer_host_begin / daf_layer_host_end on two arenas and two streams (pinned host tensors in, "
                      "hidden rows out; every layer's result is waited for inside the timed region); of the fresh "
                      "tensors only the rows of the important tokens and of the question cross the link "
                      "(h2d_bytes_per_step), read in place by the gather kernel; host_input_bytes_per_step is the size "
                      "of all host input tensors"}
        del arenas, host

    # ---- CPU oracle on this machine's cores, bounded sample (rank 0, N = 1 only)
    cpu_baseline = None
    if primary and rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        t_cpu, n_cpu, how = 0.0, 0, ""
        while t_cpu < 10.0 and n_cpu < min(w.layers, 8):
            dt, how = oracle_layer_seconds(oracle, _host_arrays(bufs[n_cpu].L), w)
            t_cpu += dt
            n_cpu += 1
        cpu_baseline = {"value": t_cpu / n_cpu * 1e6, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                        "sample": f"first {n_cpu} of {w.layers} layers of {w.name}, fp64 oracle: {how}"}

    speedup = us_full / us_per_layer / world if world == 1 else None
    flop_ratio = flops["full"] / daf_flops
    res = {
        "value": us_per_layer, "unit": UNIT, "ms_per_step": ms_per_step, "config": _config_dict(w, world),
        "ms_per_step_median": float(statistics.median(step_ms)), "ms_per_step_min": float(min(step_ms)),
        "tflops": tflops, "frac_of_bf16_peak": tflops / (peaks["bf16_tflops"] * world),
        "roofline": roofline,
        "schedule": ("selection of every layer on a second stream (daf_select_topk), layers from idx_in on the main one"
                     if overlap else "one stream"),
        "us_per_layer_one_stream": us_layer_one_stream,
        "stages_us": {"select_gather_update": us_select, "imp_qd_attn": us_both, "imp_qd_attn_kernel_only": us_kernel,
                      "merge_only": us_merge, "important_attn_alone": us_imp, "question_attn_alone": us_qd},
        "stages": {
            "important_attn": {"bound": "tensor", "tflops": imp_tflops, "frac": imp_tflops / peaks["bf16_tflops"]},
            "question_attn": {"bound": "tensor", "tflops": qd_tflops, "frac": qd_tflops / peaks["bf16_tflops"],
                              "kv_gbs": 2 * w.N * w.n_kv_heads * 256 / (us_qd * 1e-6) / 1e9 if us_qd else None},
            "deviation_scores": {"bound": "hbm", "us": us_dev, "gbs": dev_bytes / (us_dev * 1e-6) / 1e9,
                                 "frac": dev_bytes / (us_dev * 1e-6) / 1e9 / peaks["hbm_gbs"],
                                 "note": "one signal layer; not part of the per-layer step"},
            "deviation_sum": {"bound": "hbm", "us": us_dev_sum, "signal_layers": n_sig_layers,
                              "gbs": (n_sig_layers * (dev_bytes - 4 * w.L_d) + 4 * w.L_d) / (us_dev_sum * 1e-6) / 1e9,
                              "frac": (n_sig_layers * (dev_bytes - 4 * w.L_d) + 4 * w.L_d) / (us_dev_sum * 1e-6) / 1e9 / peaks["hbm_gbs"],
                              "note": "signal of several layers aggregated in one pass (first kernel of daf_select_from_kv)"},
            "select_gather_update": {"bound": "hbm", "gbs": gather_bytes / (us_select * 1e-6) / 1e9,
                                     "frac": gather_bytes / (us_select * 1e-6) / 1e9 / peaks["hbm_gbs"],
                                     "note": "includes the latency-bound top-k kernel"},
        },
        "full_recompute": {"us_per_layer": us_full, "tflops": full_tflops, "frac": full_tflops / peaks["bf16_tflops"],
                           "speedup_daf_vs_full": speedup, "flop_ratio": flop_ratio,
                           "speedup_over_flop_ratio": (speedup / flop_ratio) if speedup else None,
                           "layers_timed": n_full, "clocks": clocks_full.summary()},
        "clocks": clocks.summary(),
        "gpu_launches": int(launches),
    }
    if "sw_power_cap" in res["clocks"]["reasons"] or "sw_power_cap" in roofline["clocks"]["reasons"]:
        res["clocks_note"] = "sw_power_cap was active during the timed region (1 kW part under dense tensor work); number kept"
    if fp8 is not None:
        res["fp8_offline_cache"] = fp8
    if blend is not None:
        res["full_context_variant"] = blend
    if e2e is not None:
        res["e2e"] = e2e
    if cpu_baseline is not None:
        res["cpu_baseline"] = cpu_baseline
    del bufs, ws, wsf, full_out
    torch.cuda.empty_cache()
    return res


def run_ours(args, primary_w: W.Workload, others):
    env = Env(args)
    by_config = {}
    for w in others:
        by_config[w.name] = measure_config(env, w, primary=False)
    res = measure_config(env, primary_w, primary=True)
    if env.rank == 0:
        line = {
            "metric": METRIC, "value": res.pop("value"), "unit": res.pop("unit"), "n_gpus": env.world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": res.pop("ms_per_step"), "higher_is_better": False,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": res.pop("config"),
        }
        line.update(res)
        line["launch_mode"] = "cuda_graph_replay" if env.use_graph else "eager"
        line["peaks"] = env.peaks
        line.setdefault("e2e", None)
        line.setdefault("cpu_baseline", None)
        if by_config:
            line["by_config"] = by_config
        print(json.dumps(line))
    if env.dist is not None:
        env.dist.barrier()
        env.dist.destroy_process_group()


def _lookup(name, num_important):
    if name in W.CONFIGS:
        return W.CONFIGS[name]
    if name in W.EXTRA_CONFIGS:
        return W.EXTRA_CONFIGS[name]
    pts = {x.name: x for x in W.sweep_points(num_important)}
    if name not in pts:
        raise SystemExit(f"unknown config {name}; choose from {list(W.CONFIGS) + list(W.EXTRA_CONFIGS) + list(pts)}")
    return pts[name]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--config", default=None,
                    help="one workload only: c0..c3, a sweep point name (c4_L<L_d>_r<r>) or x136k; "
                         f"default: {DEFAULT_PRIMARY} as the headline with {', '.join(DEFAULT_OTHERS)} under by_config")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="launch eagerly instead of replaying a CUDA graph")
    ap.add_argument("--no-overlap", action="store_true", help="keep the selection kernels on the layer's own stream")
    ap.add_argument("--kv-in-place", action="store_true",
                    help="step 2 reads its K/V rows in place (no packed copies are written); slower, for comparison")
    ap.add_argument("--layers", type=int, default=0, help="use only the first LAYERS layers (profiling captures)")
    args = ap.parse_args()
    import dataclasses
    cut = (lambda w: dataclasses.replace(w, layers=min(args.layers, w.layers))) if args.layers > 0 else (lambda w: w)
    if args.impl == "reference":
        import oracle
        count = oracle.num_important
    else:
        from paper_2607_21599_b200 import api, build
        build.build()
        count = api.daf_num_important
    primary = cut(_lookup(args.config or DEFAULT_PRIMARY, count))
    others = [] if args.config else [cut(_lookup(n, count)) for n in DEFAULT_OTHERS]
    if args.impl == "reference":
        run_reference(args, primary)
    else:
        run_ours(args, primary, others)


if __name__ == "__main__":
    main()
