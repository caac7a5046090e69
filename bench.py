#!/usr/bin/env python
"""Benchmark of the MEDA compression pass.

One "step" = the whole pass (phase A of every layer, the budget barrier, phase B of every layer)
over one synthetic prompt.  The metric is KV tokens compressed per second per layer-pass:
    value = n_gpus * n_layers * n_tokens / step_time        [token*layers / s]
With --gpus N > 1 (launched by torchrun) every rank compresses its own prompt (independent
problems, no data-path collective): weak scaling.

`--impl reference` times the CPU oracle (the only reference this paper has) on a bounded sample.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "kv_tokens_compressed_per_s_per_layer_pass"
UNIT = "token*layers/s"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="long_video_128k")
    ap.add_argument("--layers", type=int, default=0, help="keep only the first N layers (profiling captures); 0 = all")
    ap.add_argument("--streams", type=int, default=8, help="streams (and contexts) the layers alternate between")
    ap.add_argument("--eager", action="store_true", help="time eager launches instead of a CUDA-graph replay of the pass")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end leg")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-decode", action="store_true", help="skip the decoding-step context measurement")
    ap.add_argument("--no-prompt-scores", action="store_true",
                    help="skip the context measurement of Eq. 8 taken over every prompt row (one layer)")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--shard", default="prompts", choices=["prompts", "layers"],
                    help="with --gpus N > 1: every rank its own prompt (weak scaling, no collective; the default), or ONE "
                         "prompt with its layers dealt round-robin to the ranks and one all-reduce of the L entropies "
                         "between the phases (strong scaling)")
    ap.add_argument("--oracle-sampled", action="store_true",
                    help="time the oracle on the bounded sample even where the whole pass would be small enough")
    ap.add_argument("--oracle-whole-pass", action="store_true",
                    help="time the oracle on the whole pass, un-sampled, whatever its size (minutes for the large workloads)")
    return ap.parse_args()


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=p["hbm_gbs"], bf16_tflops=p["bf16_tflops"], bf16_sustained=p.get("bf16_tflops_sustained", p["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_sustained=1400.0, source="fallback")


# ------------------------------------------------------------------------------------------------
# CPU oracle leg (cpu_baseline and --impl reference)
# ------------------------------------------------------------------------------------------------

WHOLE_PASS_MAX_SIMILARITIES = 2.5e9     # below this many similarity entries the oracle runs the whole pass, un-sampled


def uniform_budgets(wl):
    """Budget rows (S, M, N) when no device run is at hand: every layer gets rho * n."""
    s = max(wl.min_budget, int(round(wl.rho * wl.n_tokens)))
    return [(s, (s * 3) // 4, s - (s * 3) // 4)] * wl.n_layers


def similarity_entries(wl, budgets):
    """(n - S_l) * S_l summed over layers and KV heads: the size of the oracle's dominant step."""
    return float(sum((wl.n_tokens - s) * s for s, _, _ in budgets)) * wl.n_kv_heads


def oracle_whole_pass_seconds(wl):
    """The oracle's whole pass (compress_pass: every layer, every head, nothing sampled), timed as it stands."""
    import torch
    from oracle import meda_oracle as O
    from paper_2502_17599_b200 import workloads as W
    layers = [tuple(t.to(torch.float64).numpy() for t in W.make_layer(wl, l, "cpu")) for l in range(wl.n_layers)]
    mod = wl.modality().numpy()
    t0 = time.perf_counter()
    O.compress_pass(layers, mod, wl.global_budget, wl.min_budget, wl.dtype)
    return time.perf_counter() - t0, "whole pass, every layer and head, un-sampled"


def oracle_sample_seconds(wl, budgets=None, whole_pass=False, sampled=False):
    """Times the oracle, as it stands, on a bounded sample of the workload and scales it to the whole pass.

    `budgets`: the (S, M, N) rows of the measured run (read back from the device), so that the sample has a
    budget the pass really has; without them (reference arm, no device) a uniform rho * n is assumed and said so.
    The sample is one layer (the one whose (n - S) S is closest to the mean over layers, i.e. a typical share of
    the dominant similarity step), KV head 0 with its query heads: scores + entropy of that head group, selection
    of that head at the layer's (M, N), and merging of every `stride`-th less-important row.  Scaling: phase A and
    selection x (KV heads x layers); the merge by the ratio of similarity entries, whole pass / sampled.
    Returns (seconds for the whole pass, description, extrapolated flag)."""
    import numpy as np
    import torch
    from oracle import meda_oracle as O
    from paper_2502_17599_b200 import workloads as W

    real = budgets is not None
    rows = [tuple(int(x) for x in b) for b in budgets] if real else uniform_budgets(wl)
    n = wl.n_tokens
    if whole_pass or (not sampled and similarity_entries(wl, rows) <= WHOLE_PASS_MAX_SIMILARITIES and wl.n_layers * n <= 1.2e6):
        sec, desc = oracle_whole_pass_seconds(wl)
        return sec, desc, False
    work = [(n - s) * s for s, _, _ in rows]
    mean_work = sum(work) / len(work)
    layer = min(range(len(rows)), key=lambda l: abs(work[l] - mean_work))
    s, m, n_imp = rows[layer]
    g = wl.n_q_heads // wl.n_kv_heads
    sub = wl.with_(n_layers=layer + 1)
    q, k, v = W.make_layer(sub, layer, "cpu")
    qh = q[:g].to(torch.float64).numpy()
    kh = k[:1].to(torch.float64).numpy()
    vh = v[:1].to(torch.float64).numpy()
    mod = wl.modality().numpy()
    # bound the merge sample to about 4e8 similarity entries (a few seconds of fp64 matmul and normalisation)
    stride = max(1, int(np.ceil((n - s) * s / 4e8)))
    t0 = time.perf_counter()
    a_s = O.window_scores(qh, kh)
    O.cross_modal_entropy(qh, kh, mod)
    conserved, less = O.select_topk(a_s[0], mod, m, n_imp)
    t1 = time.perf_counter()
    sampled = less[::stride]
    km, vm, counts, target = O.merge_kv(kh[0], vh[0], conserved, sampled)
    O.round_to_dtype(km, wl.dtype), O.round_to_dtype(vm, wl.dtype)
    t2 = time.perf_counter()
    per_head_layer = t1 - t0
    merge_scale = similarity_entries(wl, rows) / max(float(sampled.size) * s, 1.0)
    total = per_head_layer * wl.n_kv_heads * wl.n_layers + (t2 - t1) * merge_scale
    desc = (f"layer {layer}, KV head 0 of {wl.n_kv_heads} ({g} query heads), "
            f"{'budget row of the measured run' if real else 'uniform budget rho*n (no device run at hand)'} "
            f"(S, M, N) = ({s}, {m}, {n_imp}); phase A + selection timed once and x{wl.n_kv_heads * wl.n_layers} "
            f"(heads x layers); merge timed on every {stride}-th less-important row ({sampled.size} x {s} similarities) "
            f"and scaled x{merge_scale:.1f} to the pass's {similarity_entries(wl, rows):.3g} similarities")
    return total, desc, True


def oracle_throughput(wl, seconds):
    # `seconds` is the (measured or extrapolated) time of the whole pass
    return wl.n_layers * wl.n_tokens / seconds


def cpu_threads():
    try:
        from threadpoolctl import threadpool_info
        n = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
        return int(n)
    except Exception:
        return os.cpu_count() or 1


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2502_17599_b200 import workloads as W
    wl = W.WORKLOADS[args.workload]
    if args.layers > 0:
        wl = wl.with_(name=f"{wl.name}_first{args.layers}layers", n_layers=min(args.layers, wl.n_layers))
    import numpy  # noqa: F401  (loads BLAS before the thread count is read)
    times = []
    desc, extrapolated = "", False
    for i in range(args.warmup + args.steps):
        dt, desc, extrapolated = oracle_sample_seconds(wl, whole_pass=args.oracle_whole_pass, sampled=args.oracle_sampled)
        if i >= args.warmup:
            times.append(dt)
    sec = sum(times) / len(times)
    val = oracle_throughput(wl, sec)
    out = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "shape": wl.description, "sample": desc},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle", "sample": desc,
                         "extrapolated": extrapolated},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(out), flush=True)


# ------------------------------------------------------------------------------------------------
# Clock sampling during the timed region
# ------------------------------------------------------------------------------------------------

class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.rows = []
        self.proc = None
        self.index = device_index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            p = [x.strip() for x in r.split(",")]
            if len(p) < 7:
                continue
            try:
                sm.append(float(p[0]))
                smax.append(float(p[1]))
            except ValueError:
                continue
            for name, val in zip(names, p[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ------------------------------------------------------------------------------------------------
# Our arm
# ------------------------------------------------------------------------------------------------

def algorithmic_work(wl, budgets):
    """Algorithmic bytes / flops per layer-pass of each kernel class: stats reads the key cache once,
    the sweep reads it once and writes the scores, the similarity contraction is 2 (n - S) S d flops per
    head, the segmented average reads every key and value row once and writes the S merged rows."""
    e = wl.element_size
    n, d, hkv, hq, w = wl.n_tokens, wl.head_dim, wl.n_kv_heads, wl.n_q_heads, wl.window
    kbytes = hkv * n * d * e
    from paper_2502_17599_b200.binding import NEAREST_SMALL_MAX_S
    # bf16 / head_dim 128: layers that keep few slots take the streaming arg-max kernel (class nearest_small)
    split = wl.dtype == "bf16" and d == 128
    out = {"stats_bytes": [], "sweep_bytes": [], "nearest_flops": [], "nearest_small_flops": [], "reduce_bytes": [],
           "group_bytes": [], "select_bytes": []}
    sort_passes = 1 if n <= 512 else (2 if n <= 512 * 512 else 3)        # 9-bit digits until every slot < n is ordered
    for s in budgets:
        s = int(s)
        out["stats_bytes"].append(kbytes)
        out["sweep_bytes"].append(kbytes + 4 * hkv * n)
        small = split and s <= NEAREST_SMALL_MAX_S
        out["nearest_small_flops" if small else "nearest_flops"].append(2.0 * (n - s) * s * d * hkv if s < n else 0.0)
        out["reduce_bytes"].append(2 * hkv * n * d * e + 2 * hkv * s * d * e + 4 * hkv * s)
        # grouping: all n rows are sorted by slot; a pass reads the (slot, row) pairs twice (histogram, scatter)
        # and writes them once, and only the passes over digits that slots < S reach are executed
        executed = min(sort_passes, 1 if s <= 512 else (2 if s <= 512 * 512 else 3))
        out["group_bytes"].append(executed * (8 + 4 + 8) * hkv * n)
        out["select_bytes"].append(4 * hkv * n + 4 * hkv * n)
    return out


# DRAM traffic of one launch of each hot kernel on the long_video_128k shapes: dram__bytes_read.sum +
# dram__bytes_write.sum from the ncu captures whose summaries are kept under profiles/ (taken on the 2-layer cut
# of the same prompt: per launch every one of these kernels moves the same bytes whatever the layer, the key
# cache once or the key and value caches once).  A figure is reported only for that workload and only while the
# kernel's sources still hash to what was captured; otherwise null.
CSRC = "paper_2502_17599_b200/csrc/"
KERNEL_TRAFFIC = {
    # class: (bytes per launch, source files, sha256[:16] of their concatenation)
    "nearest": (138.9e6, (CSRC + "nearest_sm100.cuh", CSRC + "sm100_primitives.cuh"), "802a52cd62a33938"),
    "stats": (136.4e6, (CSRC + "window_stats_sm100.cuh", CSRC + "attn_sm100.cuh", CSRC + "sm100_primitives.cuh"), "a9878e61f71590db"),
    "sweep": (137.0e6, (CSRC + "window_sweep_sm100.cuh", CSRC + "window_stats_sm100.cuh", CSRC + "attn_sm100.cuh",
                        CSRC + "sm100_primitives.cuh"), "9054a40c91ee40f0"),
    "reduce": (288.9e6, (CSRC + "group_reduce.cuh",), "ddedc37dfed0b21f"),
}
NOMINAL_HBM_GBS = 8000.0     # the nominal figure the target is worded against; the measured copy peak is the denominator of `frac`


def sources_sha(files):
    import hashlib
    h = hashlib.sha256()
    for f in files:
        h.update(open(os.path.join(ROOT, f), "rb").read())
    return h.hexdigest()[:16]


def kernel_traffic(klass, workload_name):
    nbytes, files, sha = KERNEL_TRAFFIC.get(klass, (None, (), None))
    if nbytes is None or sha is None or not workload_name.startswith("long_video_128k"):
        return None
    return nbytes if sources_sha(files) == sha else None


def rank_workload(name, rank, layers=0):
    """The prompt rank `rank` compresses: the named workload with its own seed (independent prompts, so
    N ranks do N times the work: weak scaling, no data-path collective)."""
    from paper_2502_17599_b200 import workloads as W
    wl = W.WORKLOADS[name]
    wl = wl.with_(seed=wl.seed + 1000 * rank)
    if layers > 0:
        wl = wl.with_(name=f"{wl.name}_first{layers}layers", n_layers=min(layers, wl.n_layers))
    return wl


def max_over_ranks(ms, world, device):
    """The slowest rank's time: the only value exchanged between ranks."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t[0])


def whole_job_throughput(wl, world, ms_step):
    """token*layers per second over all ranks."""
    return world * wl.n_layers * wl.n_tokens / (ms_step * 1e-3)


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2502_17599_b200 import build
    from paper_2502_17599_b200 import workloads as W
    from paper_2502_17599_b200.pipeline import CompressionPass

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    if rank == 0:
        build.build()
    if world > 1:
        dist.barrier()

    by_layer = args.shard == "layers" and world > 1
    wl = rank_workload(args.workload, 0 if by_layer else rank, args.layers)
    L = wl.n_layers
    shard = (rank, world) if by_layer else None
    from paper_2502_17599_b200.pipeline import owned_layers
    mine = set(owned_layers(L, rank, world)) if by_layer else set(range(L))
    qs, ks, vs = [], [], []
    for l in range(L):
        q, k, v = W.make_layer(wl, l, "cuda") if l in mine else (None, None, None)
        qs.append(q); ks.append(k); vs.append(v)
    if by_layer:      # the legs below walk every layer of the prompt on one GPU
        args.eager = args.no_e2e = args.no_decode = args.no_prompt_scores = True
    input_bytes = sum(t.numel() * t.element_size() for ts in (qs, ks, vs) for t in ts if t is not None)
    cp = CompressionPass(wl, n_streams=args.streams)
    stream = torch.cuda.current_stream()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    # The timed region replays the whole pass as one CUDA graph (unless --eager): a step is then a
    # single launch on the host.  Kernel-level times come from a second region of the same K steps
    # run eagerly with every launch bracketed by events, whose overhead must not be in the headline.
    kernels_per_pass = cp.capture(qs, ks, vs) if not args.eager else None
    step = cp.replay if not args.eager else (lambda: cp.run(qs, ks, vs, layer_shard=shard))
    for _ in range(args.warmup):
        step()
    cp.check()
    budgets = cp.budgets.cpu().numpy()[:, 0]

    launches0 = cp.launch_count()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    barrier()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record(stream)
    for _ in range(args.steps):
        step()
    ev1.record(stream)
    barrier()
    ms_total = ev0.elapsed_time(ev1)
    launches = kernels_per_pass * args.steps if not args.eager else cp.launch_count() - launches0
    cp.check()

    cp.ctx.profile_enable(True)
    barrier()
    for _ in range(args.steps):
        cp.run(qs, ks, vs, single_stream=True, layer_shard=shard)      # one stream: a launch's events bracket that launch alone
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    dropped = cp.ctx.profile_dropped()
    prof = cp.ctx.profile_read()
    cp.ctx.profile_enable(False)
    cp.check()
    if dropped:
        raise RuntimeError(f"{dropped} launches of the per-kernel timing region went untimed (event pool full): "
                           "per-class times would not cover --steps steps; use fewer steps")
    ms_step = max_over_ranks(ms_total, world, "cuda") / args.steps
    value = whole_job_throughput(wl, 1 if by_layer else world, ms_step)      # one prompt in all when sharded by layer

    # context: one decoding step's attention (Eq. 3) over all layers, compressed caches against full ones
    decode = None
    if not args.no_decode and wl.head_dim in (64, 128) and (wl.n_q_heads // wl.n_kv_heads) in (1, 2, 3, 4, 7, 8):
        q_new = [q_[:, -1, :].contiguous() for q_ in qs]
        out = torch.zeros((wl.n_q_heads, wl.head_dim), dtype=torch.float32, device="cuda")

        def decode_ms(compressed):
            def one():
                for l in range(L):
                    if compressed:
                        cp.ctx.decode_attention(l, q_new[l], cp.k_out[l], cp.v_out[l], out, budgets=cp.budgets)
                    else:
                        cp.ctx.decode_attention(l, q_new[l], ks[l], vs[l], out, n_rows=wl.n_tokens)
            one()
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                one()
            for _ in range(3):
                graph.replay()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for _ in range(10):
                graph.replay()
            b.record(stream)
            torch.cuda.synchronize()
            return a.elapsed_time(b) / 10

        ms_c, ms_f = decode_ms(True), decode_ms(False)
        e = wl.element_size
        bytes_c = 2 * wl.n_kv_heads * wl.head_dim * e * float(budgets.sum())
        bytes_f = 2 * wl.n_kv_heads * wl.head_dim * e * float(L * wl.n_tokens)
        decode = {"what": "attention of one new token over every layer's cache (Eq. 3), one CUDA-graph replay per token",
                  "ms_per_token_compressed": ms_c, "ms_per_token_full": ms_f, "speedup": ms_f / ms_c,
                  "cache_bytes_compressed": bytes_c, "cache_bytes_full": bytes_f,
                  "GB/s_compressed": bytes_c / ms_c / 1e6, "GB/s_full": bytes_f / ms_f / 1e6}
        cp.check()

    # context: Eq. 8 as printed (every prompt row a query, no observation window), one layer
    prompt_ctx = None
    if not args.no_prompt_scores:
        q_all = W.make_prompt_queries(wl, 0, "cuda")
        scratch = torch.empty(max(cp.ctx.prompt_scores_scratch_bytes(), 16), dtype=torch.uint8, device="cuda")
        sc_all = torch.zeros((wl.n_kv_heads, wl.n_tokens), dtype=torch.float32, device="cuda")
        cp.ctx.prompt_scores(q_all, ks[0], sc_all, scratch)                  # warm-up
        cp.check()
        cp.ctx.profile_read()
        cp.ctx.profile_enable(True)
        reps = 2
        for _ in range(reps):
            cp.ctx.prompt_scores(q_all, ks[0], sc_all, scratch)
        cp.check()
        pr = {k_: v_[0] / reps for k_, v_ in cp.ctx.profile_read().items() if v_[1]}
        cp.ctx.profile_enable(False)
        logits = wl.n_q_heads * wl.n_tokens * (wl.n_tokens + 1) / 2
        ms_layer = sum(pr.values())
        sfu = 148 * 16 * ((clocks or {}).get("sm_max_mhz") or 1965.0) * 1e6
        prompt_ctx = {"what": "scores of Eq. 8 with every prompt row as a query (column sums of the causal attention), "
                              "one layer: normalisers pass, column-sum pass and two small kernels",
                      "ms_per_layer": ms_layer, "ms_normalisers": pr.get("stats"), "ms_column_sums": pr.get("sweep"),
                      "logits_per_pass": logits, "TFLOP/s": 2 * 2 * logits * wl.head_dim / (ms_layer * 1e-3) / 1e12,
                      "exp2/s": 2 * logits / (ms_layer * 1e-3), "frac_of_sfu_peak": 2 * logits / (ms_layer * 1e-3) / sfu,
                      "window_scores_ms_per_layer": (per_layer_window_ms(prof, L))}
        del q_all, scratch, sc_all

    # end-to-end leg: pinned host inputs -> device -> pass -> compacted caches back to the host
    e2e = None
    if not args.no_e2e:
        q_h = [t_.cpu().pin_memory() for t_ in qs]
        k_h = [t_.cpu().pin_memory() for t_ in ks]
        v_h = [t_.cpu().pin_memory() for t_ in vs]
        staging = {"q": qs, "k": ks, "v": vs}
        out_host = cp.alloc_host_outputs()
        h2d, d2h = cp.run_from_host(q_h, k_h, v_h, staging, out_host)      # warm-up
        barrier()
        t0 = time.perf_counter()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(args.e2e_steps):
            h2d, d2h = cp.run_from_host(q_h, k_h, v_h, staging, out_host)
        e1.record(stream)
        barrier()
        wall = (time.perf_counter() - t0) * 1e3
        ms_e2e = max(e0.elapsed_time(e1), wall) / args.e2e_steps
        ms_e2e = max_over_ranks(ms_e2e, world, "cuda")
        e2e = {"value": whole_job_throughput(wl, world, ms_e2e), "unit": UNIT,
               "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "ms_per_step": ms_e2e}
        del q_h, k_h, v_h, out_host

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    pk = peaks()
    own = sorted(mine)
    L_local = len(own)
    work = algorithmic_work(wl, budgets[own])          # rank 0's kernel times cover its own layers
    per_class = {name: {"ms_per_step": ms / args.steps, "launches_per_step": cnt / args.steps}
                 for name, (ms, cnt) in prof.items() if cnt}
    total_prof = sum(v["ms_per_step"] for v in per_class.values()) or 1.0
    for v in per_class.values():
        v["share"] = v["ms_per_step"] / total_prof
    dominant = max(per_class, key=lambda k_: per_class[k_]["ms_per_step"])
    # roofline of the dominant kernel
    if dominant == "nearest":
        flops = sum(work["nearest_flops"])
        achieved = flops / (per_class["nearest"]["ms_per_step"] * 1e-3) / 1e12
        roof = {"kernel": "nearest (merge similarity + arg-max)", "bound": "tensor", "achieved": achieved,
                "peak": pk["bf16_sustained"], "unit": "TFLOP/s", "frac": achieved / pk["bf16_sustained"],
                "traffic": kernel_traffic("nearest", wl.name), "traffic_unit": "bytes per launch (ncu, 2-layer capture of the same config)",
                "peak_source": pk["source"] + " (sustained cuBLAS bf16)", "flops_per_step": flops,
                # launches that had work: the kernel is enqueued for every layer and returns at once where the
                # layer's budget sends it to the streaming kernel (the budget never leaves the device)
                "working_launches_per_step": len(work["nearest_flops"]),
                "flops_per_launch": flops / max(len(work["nearest_flops"]), 1),
                "us_per_launch": 1e3 * per_class["nearest"]["ms_per_step"] / max(len(work["nearest_flops"]), 1)}
    else:
        key = {"stats": "stats_bytes", "sweep": "sweep_bytes", "reduce": "reduce_bytes", "group": "group_bytes",
               "select": "select_bytes"}.get(dominant)
        nbytes = sum(work[key]) if key else 0.0
        achieved = nbytes / (per_class[dominant]["ms_per_step"] * 1e-3) / 1e9 if key else 0.0
        roof = {"kernel": dominant, "bound": "hbm", "achieved": achieved, "peak": pk["hbm_gbs"], "unit": "GB/s",
                "frac": achieved / pk["hbm_gbs"], "traffic": kernel_traffic(dominant, wl.name),
                "peak_source": pk["source"] + " (copy)", "bytes_per_step": nbytes}
    # secondary fractions, for the record
    extra = {}
    for name, key in (("stats", "stats_bytes"), ("sweep", "sweep_bytes"), ("reduce", "reduce_bytes")):
        if name in per_class:
            gbs = sum(work[key]) / (per_class[name]["ms_per_step"] * 1e-3) / 1e9
            class_launches = max(per_class[name]["launches_per_step"], 1.0)
            extra[name] = {"GB/s": gbs, "frac_of_copy_peak": gbs / pk["hbm_gbs"], "frac_of_nominal_8TBs": gbs / NOMINAL_HBM_GBS,
                           "algorithmic_bytes_per_layer": sum(work[key]) / L_local,
                           "us_per_layer": 1e3 * per_class[name]["ms_per_step"] / L_local,
                           "launches_per_layer": class_launches / L_local,
                           "traffic": kernel_traffic(name, wl.name),
                           "traffic_unit": "dram bytes per layer's main launch (ncu, 2-layer capture of the same config)"}
    # the two phase-A sweeps evaluate one exp2 per logit on the special-function units: 16 per clock per SM
    exps = float(L_local) * wl.n_q_heads * wl.window * wl.n_tokens
    sfu_peak = 148 * 16 * (clocks["sm_max_mhz"] or 1965.0) * 1e6 if clocks else None
    for name in ("stats", "sweep"):
        if name in per_class and sfu_peak:
            rate = exps / (per_class[name]["ms_per_step"] * 1e-3)
            extra[name].update({"exp2/s": rate, "frac_of_sfu_peak": rate / sfu_peak})
    if "nearest" in per_class:
        tf = sum(work["nearest_flops"]) / (per_class["nearest"]["ms_per_step"] * 1e-3) / 1e12
        extra["nearest"] = {"TFLOP/s": tf, "frac_of_sustained_bf16": tf / pk["bf16_sustained"]}
    if "nearest_small" in per_class:
        ms_both = per_class["nearest_small"]["ms_per_step"] + per_class.get("nearest", {"ms_per_step": 0.0})["ms_per_step"]
        tf = (sum(work["nearest_flops"]) + sum(work["nearest_small_flops"])) / (ms_both * 1e-3) / 1e12
        extra["nearest_both_kernels"] = {"TFLOP/s": tf, "frac_of_sustained_bf16": tf / pk["bf16_sustained"],
                                         "layers_streaming_kernel": len(work["nearest_small_flops"])}

    cpu = None
    if not args.no_cpu_baseline:
        sec, desc, extrapolated = oracle_sample_seconds(wl, cp.budgets.cpu().numpy(), whole_pass=args.oracle_whole_pass,
                                                           sampled=args.oracle_sampled)
        cpu = {"value": oracle_throughput(wl, sec), "unit": UNIT, "cores": cpu_threads(), "kind": "oracle",
               "sample": desc, "pass_seconds": sec, "extrapolated": extrapolated}

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "strong" if by_layer else "weak", "vs_baseline": None,
        "dtype": "bf16" if wl.dtype == "bf16" else "f32", "data": "synthetic",
        "config": {"workload": wl.name, "shape": wl.description, "global_budget": wl.global_budget,
                   "input_bytes": input_bytes, "l2": "inputs larger than L2 (no flush needed)" if input_bytes > 256e6 else "inputs fit L2",
                   "parallelism": (f"one prompt, layers round-robin over {world} ranks, one all-reduce of {L} entropies"
                                   if by_layer else f"independent prompts x{world}"),
                   "launch": ("eager launches" if args.eager else f"one CUDA-graph replay per step ({kernels_per_pass} kernels)")
                             + f", layers alternate between {len(cp.contexts)} streams"},
        "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches),
        "roofline": roof, "kernels": per_class, "kernel_rooflines": extra, "cpu_baseline": cpu,
        "budgets_min_max": [int(budgets.min()), int(budgets.max())], "decode_context": decode,
        "prompt_scores_context": prompt_ctx,
    }
    print(json.dumps(out), flush=True)
    if world > 1:
        dist.destroy_process_group()


def per_layer_window_ms(prof, n_layers):
    """Device time per layer of the observation-window phase A in the profiled steps (for comparison)."""
    ms = sum(prof[c][0] for c in ("stats", "stats_combine", "sweep", "entropy_final") if c in prof and prof[c][1])
    cnt = prof["sweep"][1] if "sweep" in prof and prof["sweep"][1] else 0
    return ms / cnt if cnt else None


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
