#!/usr/bin/env python
"""Benchmark of the GVote compression pass: cached tokens compressed per second on B200.

A step is one pass of the whole hot path (fit, sample, project, vote, compact) over every layer
of the workload, one `gvote_compress` call per layer.  The default workload is the Llama-3-8B
shaped 32K-context pass (32 layers, N = 32768, S = 32, p = 0.95) on seeded synthetic inputs.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2] [--impl reference]

Prints one JSON line.  With --impl reference the CPU oracle is timed instead (rank 0 only).
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
from concurrent.futures import ThreadPoolExecutor

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "GVote KV tokens compressed/sec (all layers of the workload, 1 B200 per rank)"
UNIT = "tokens/s"
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1590.0


# ----------------------------------------------------------------------------- helpers
def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            d = json.load(open(path))
            return float(d["hbm_gbs"]), float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, FALLBACK_BF16_TFLOPS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    NAMES = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.perf_counter(), line.strip()))

    def stop(self, t0=None, t1=None):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for ts, line in self.lines:
            if t0 is not None and not (t0 <= ts <= t1):
                continue
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(self.NAMES, parts[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def gen_layers(cfg, layers, workers):
    from paper_2509_03136_b200 import synth
    with ThreadPoolExecutor(max_workers=workers) as ex:
        return list(ex.map(lambda l: synth.make_layer(cfg, l), layers))


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [i.get("num_threads", 1) for i in threadpool_info() if i.get("user_api") == "blas"]
        if n:
            return int(max(n))
    except Exception:
        pass
    return len(os.sched_getaffinity(0))


def time_oracle_layer(cfg, li, layer_id):
    from oracle import gvote_oracle as o
    t0 = time.perf_counter()
    res, Kc, Vc = o.compress_layer(li.h, li.W_q, li.b_q, li.K, li.V, li.cu_seqlens, n_q_heads=cfg.n_q_heads,
                                   d_k=cfg.d_k, theta=cfg.rope_theta, S=cfg.S, p_nuc=float(np.float32(cfg.p_nuc)),
                                   n_f=cfg.n_f, n_s=cfg.n_s, seed=cfg.seed, layer_id=layer_id)
    return time.perf_counter() - t0, res


def algorithmic_bytes(cfg, kept_frac):
    """Compulsory bytes per layer of each stage (no recompute, no materialised logits)."""
    T = cfg.total_tokens
    kv = T * cfg.n_kv_heads * cfg.d_k * 2
    return {
        "fit": (T - cfg.batch * cfg.n_s) * cfg.d_h * 4,
        "wq": cfg.d_h * cfg.n_q_heads * cfg.d_k * 2,
        "k": kv,
        "compact": 4.0 * kept_frac * kv,
    }


def flops(cfg):
    rows = cfg.batch * (cfg.S + 1)
    proj = 2.0 * rows * cfg.d_h * cfg.n_q_heads * cfg.d_k
    score = 2.0 * (cfg.S + 1) * cfg.n_q_heads * cfg.total_tokens * cfg.d_k
    return proj, score


STAGE_OF = {
    "fit_partial_kernel": "fit", "fit_finalize_kernel": "fit", "sample_kernel": "sample",
    "prep_kernel": "sample", "real_topp_kernel": "vote", "score_sample_kernel": "vote", "bracket_kernel": "vote",
    "score_sweep_kernel": "vote", "resolve_kernel": "vote", "commit_kernel": "vote",
    "xstage_kernel": "project", "rope_table_kernel": "project", "project_simt_kernel": "project",
    "project_umma_kernel": "project", "project_finish_kernel": "project",
    "score_simt_kernel": "vote", "score_umma_kernel": "vote", "topp_rows_kernel": "vote",
    "topk_rows_kernel": "vote", "softmax_dump_kernel": "vote", "budget_kernel": "vote",
    "mask_scan_kernel": "compact", "compact_kernel": "compact",
}


# ----------------------------------------------------------------------------- reference arm
def run_reference(args, cfg, rank, world):
    if rank != 0:
        return
    from paper_2509_03136_b200 import synth
    cores = blas_threads()
    times = []
    for s in range(args.warmup + args.steps):
        layer = s % cfg.n_layers
        li = synth.make_layer(cfg, layer)
        t, _ = time_oracle_layer(cfg, li, layer)
        if s >= args.warmup:
            times.append(t)
    per_layer = sum(times) / len(times)
    value = cfg.total_tokens / (per_layer * cfg.n_layers)
    sample = (f"a step times ONE layer of the workload's {cfg.n_layers} ({cfg.total_tokens} tokens; layers 0, 1, ... in "
              f"turn): the fp64 NumPy oracle as it stands (matmul, sort and cumsum are NumPy's, on {cores} BLAS threads); "
              f"value = tokens / (mean layer time x {cfg.n_layers} layers), ms_per_step = the measured layer time")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": per_layer * 1e3,
        "ms_per_full_pass_extrapolated": per_layer * cfg.n_layers * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(cfg, args),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def workload_config(cfg, args):
    return {"workload": f"{cfg.name}: {cfg.n_layers} layers, hidden {cfg.d_h}, {cfg.n_q_heads}/{cfg.n_kv_heads} heads, "
                        f"d_k {cfg.d_k}, requests {cfg.batch}, tokens {cfg.total_tokens}, S {cfg.S}, p {cfg.p_nuc}",
            "n_f": cfg.n_f, "n_s": cfg.n_s, "sel_mode": "topk_c0", "h_dtype": "f32", "kv_dtype": "bf16",
            "l2": "inputs larger than L2 (every layer has its own tensors; K/V restored from pristine copies "
                  "between steps, outside the timed intervals)",
            "streams": max(1, args.streams),
            "timing": "sum of per-step CUDA-event intervals on the launch stream"}


# ----------------------------------------------------------------------------- S and p sweeps
def select_once(gv, torch, cfg, li, d, S, p_nuc, mu, var, h_last, reps=5):
    """gvote_sample + gvote_project + gvote_vote + gvote_overlap for one (S, p) on one layer's device tensors.
    Returns (mask, budget [batch, Hkv], overlap [batch, Hq], milliseconds of the select step)."""
    from dataclasses import replace
    c = replace(cfg, S=S, p_nuc=p_nuc)
    p = gv.params_from_config(c)
    geom = (c.batch, c.total_tokens, max(c.seq_lens))
    ws = gv.alloc_workspace(p, *geom)
    Ht = torch.empty(c.batch, S, c.d_h, device="cuda")
    Q = torch.empty(c.batch, c.n_kv_heads, c.G * (S + 1), c.d_k, dtype=torch.bfloat16, device="cuda")
    mask = torch.empty(c.n_kv_heads, gv.mask_row_words(c.total_tokens, c.batch), dtype=torch.int32, device="cuda")
    budget = torch.empty(c.batch, c.n_kv_heads, dtype=torch.int32, device="cuda")
    b_step = torch.empty(c.batch, c.n_q_heads, dtype=torch.int32, device="cuda")
    ov = torch.empty(c.batch, c.n_q_heads, device="cuda")
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ms = 0.0
    for i in range(reps + 2):
        torch.cuda.synchronize()
        e0.record()
        gv.gvote_sample(p, mu, var, c.batch, Ht)
        gv.gvote_project(p, Ht, h_last, d["W_q"], d["b_q"], d["cu"], c.batch, Q, ws)
        gv.gvote_vote(p, Q, d["K"], d["cu"], geom, mask, budget, b_step, ws)
        e1.record()
        torch.cuda.synchronize()
        if i >= 2:
            ms += e0.elapsed_time(e1)
    gv.gvote_overlap(p, Q, d["K"], mask, d["cu"], geom, ov, ws)
    assert gv.gvote_poll_status(ws) == 0
    return mask.cpu().numpy(), budget.cpu().numpy(), ov.cpu().numpy(), ms / reps


def run_sweep(args, cfg):
    """Section 4.4's ablations on synthetic data: the budget the vote arrives at, the share of the current
    query's attention the kept keys hold (Section 3.3's yardstick) and the time of the select step, over
    S at p = 0.95 and over p at S = 32.  One JSON line per setting."""
    import torch
    from paper_2509_03136_b200 import build as gbuild, gvote as gv, synth
    gbuild.build()
    gv.load()
    torch.cuda.set_device(0)
    li = synth.make_layer(cfg, 0)
    d = {"W_q": gv.bf16_from_bits(li.W_q), "b_q": None, "K": gv.bf16_from_bits(li.K),
         "cu": torch.from_numpy(li.cu_seqlens).cuda()}
    h = torch.from_numpy(li.h).cuda()
    p0 = gv.params_from_config(cfg)
    geom = (cfg.batch, cfg.total_tokens, max(cfg.seq_lens))
    ws = gv.alloc_workspace(p0, *geom)
    mu = torch.empty(cfg.batch, cfg.d_h, device="cuda"); var = torch.empty_like(mu)
    gv.gvote_fit(p0, h, d["cu"], geom, mu, var, ws)
    cu = li.cu_seqlens
    h_last = torch.stack([h[int(cu[r + 1]) - 1] for r in range(cfg.batch)]).contiguous()
    rows = [("S", S, 0.95) for S in (1, 2, 4, 8, 16, 32, 64)] + [("p", 32, pn) for pn in (0.8, 0.9, 0.95, 0.98, 0.99)]
    prev_mask = None
    for axis, S, pn in rows:
        mask, budget, ov, ms = select_once(gv, torch, cfg, li, d, S, pn, mu, var, h_last)
        nested = None
        if axis == "S" and prev_mask is not None:
            nested = bool(np.all((prev_mask & ~mask) == 0))          # the smaller S's keep set lies inside this one
        prev_mask = mask if axis == "S" else None
        print(json.dumps({"sweep": axis, "workload": cfg.name, "S": S, "p_nuc": pn,
                          "kept_fraction": float(budget.sum() / (cfg.n_kv_heads * cfg.total_tokens)),
                          "budget_per_head": budget.reshape(-1).tolist(),
                          "attention_on_kept_keys_mean": float(ov.mean()), "attention_on_kept_keys_min": float(ov.min()),
                          "select_ms": ms, "contains_previous_S": nested}))


# ----------------------------------------------------------------------------- native arm
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--workload", default="c2")
    ap.add_argument("--layers", type=int, default=0, help="override the layer count (debugging)")
    ap.add_argument("--streams", type=int, default=6,
                    help="CUDA streams the layers of a step are spread over (each with its own workspace)")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-upstream-row", action="store_true")
    ap.add_argument("--no-recompress-row", action="store_true")
    ap.add_argument("--no-graph-row", action="store_true", help="skip the one-stream pass replayed as a CUDA graph")
    ap.add_argument("--sweep", action="store_true",
                    help="instead of the benchmark: budget, attention kept and select time over S and over p "
                         "(one layer of --workload, default c1)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)

    from paper_2509_03136_b200 import shard, synth
    # --gpus N without a launcher: start the N ranks here (one process per GPU, each with its own requests)
    cmd = shard.self_launch_command(os.path.abspath(__file__), sys.argv[1:], args.gpus, os.environ)
    if cmd is not None:
        sys.exit(subprocess.call(cmd))
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    over = {"n_layers": args.layers} if args.layers > 0 else {}
    base_cfg = synth.make_config(args.workload, **over)

    if args.impl == "reference":
        run_reference(args, base_cfg, rank, world)
        return
    if args.sweep:
        if rank == 0:
            run_sweep(args, base_cfg if "--workload" in sys.argv else synth.make_config("c1"))
        return

    import torch
    from paper_2509_03136_b200 import build as gbuild
    if rank == 0:
        gbuild.build()
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        dist.barrier()
    else:
        dist = None
        torch.cuda.set_device(local)
    from paper_2509_03136_b200 import gvote as gv
    gv.load()
    if args.warmup < 3:
        args.warmup = 3

    # weak scaling: every rank compresses its own requests (same shapes, its own seed)
    from paper_2509_03136_b200 import shard
    cfg = shard.rank_workload(base_cfg, rank)
    L = cfg.n_layers
    geom = (cfg.batch, cfg.total_tokens, max(cfg.seq_lens))
    workers = max(1, min(len(os.sched_getaffinity(0)) // max(world, 1), 16))
    t_gen = time.perf_counter()
    layers = gen_layers(cfg, range(L), workers)
    t_gen = time.perf_counter() - t_gen

    dev = torch.device("cuda", local)
    p_layer = [gv.params_from_config(cfg, layer_id=l) for l in range(L)]
    n_streams = max(1, min(args.streams, L))
    ws_s = [gv.alloc_workspace(p_layer[0], *geom) for _ in range(n_streams)]
    ws = ws_s[0]
    side = [torch.cuda.Stream(device=dev) for _ in range(n_streams - 1)]
    cu = torch.from_numpy(layers[0].cu_seqlens).to(dev)
    d_h = [torch.from_numpy(li.h).to(dev) for li in layers]
    d_W = [gv.bf16_from_bits(li.W_q, dev) for li in layers]
    d_K0 = [gv.bf16_from_bits(li.K, dev) for li in layers]
    d_V0 = [gv.bf16_from_bits(li.V, dev) for li in layers]
    d_K = [t.clone() for t in d_K0]
    d_V = [t.clone() for t in d_V0]
    words = gv.mask_row_words(cfg.total_tokens, cfg.batch)
    d_mask = [torch.empty(cfg.n_kv_heads, words, dtype=torch.int32, device=dev) for _ in range(L)]
    d_budget = [torch.empty(cfg.batch, cfg.n_kv_heads, dtype=torch.int32, device=dev) for _ in range(L)]
    d_bstep = [torch.empty(cfg.batch, cfg.n_q_heads, dtype=torch.int32, device=dev) for _ in range(L)]

    def restore():
        for l in range(L):
            d_K[l].copy_(d_K0[l]); d_V[l].copy_(d_V0[l])

    def one_pass(spread=True):
        # layers are independent (Section 3.2): layer l goes to stream l mod n_streams, so the short,
        # latency-bound kernels of one layer run under the streaming kernels of another
        main = torch.cuda.current_stream()
        side_now = side if spread else []
        ns = len(side_now) + 1
        if side_now:
            fork = torch.cuda.Event()
            fork.record(main)
            for st in side_now:
                st.wait_event(fork)
        for l in range(L):
            k = l % ns
            with torch.cuda.stream(main if k == 0 else side_now[k - 1]):
                gv.gvote_compress(p_layer[l], d_h[l], d_W[l], None, d_K[l], d_V[l], cu, geom, d_mask[l], d_budget[l],
                                  d_bstep[l], ws_s[k])
        for st in side_now:
            join = torch.cuda.Event()
            join.record(st)
            main.wait_event(join)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def timed_steps(n, spread=True):
        total_ms = 0.0
        for _ in range(n):
            restore()
            barrier()
            ev0.record()
            one_pass(spread)
            ev1.record()
            torch.cuda.synchronize()
            total_ms += ev0.elapsed_time(ev1)
        return total_ms

    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(1.0)
    tw0 = time.perf_counter()
    timed_steps(args.warmup)
    n0 = gv.gvote_launch_count()
    tc0 = time.perf_counter()
    total_ms = timed_steps(args.steps)
    tc1 = time.perf_counter()
    launches = gv.gvote_launch_count() - n0
    for w in ws_s:
        assert gv.gvote_poll_status(w) == 0, "a device-side wait timed out"
    # (request, KV head) pairs that had to be selected again by the exact route (warm-up and timed steps)
    exact_heads = sum(gv.gvote_exact_heads(w) for w in ws_s)
    total_ms = shard.max_over_ranks(total_ms, dist, dev)
    ms_per_step = total_ms / args.steps
    value = shard.job_throughput(cfg.total_tokens, world, ms_per_step * 1e-3)

    # ---- per-kernel timing: the same steps again with an event pair around every launch
    # (on one stream, so that every event pair brackets one kernel running alone)
    gv.gvote_profile_enable(True)
    serial_ms = timed_steps(args.steps, spread=False) / args.steps
    prof = gv.gvote_profile_report()
    gv.gvote_profile_enable(False)
    # clock samples cover the warm-up, the timed steps and their event-instrumented repeat (same work)
    clocks = sampler.stop(tw0, time.perf_counter())
    clocks["window"] = "warm-up + timed steps + instrumented repeat"
    budgets = torch.stack(d_budget).cpu().numpy()                       # [L, batch, Hkv]
    kept_frac = float(budgets.sum() / (L * cfg.n_kv_heads * cfg.total_tokens))
    hbm_gbs, bf16_tf, peak_kind = load_peaks()
    ab = algorithmic_bytes(cfg, kept_frac)
    f_proj, f_score = flops(cfg)
    per_kernel = {k: {"launches": n, "avg_us": ms / n * 1e3, "share": 0.0} for k, (n, ms) in prof.items()}
    tot_prof = sum(ms for _, ms in prof.values()) or 1.0
    for k, (n, ms) in prof.items():
        per_kernel[k]["share"] = ms / tot_prof
    stage_us = {}
    for k, (n, ms) in prof.items():
        st = STAGE_OF.get(k, "other")
        stage_us[st] = stage_us.get(st, 0.0) + ms * 1e3 / (args.steps * L)
    dom = max(prof.items(), key=lambda kv: kv[1][1])[0]
    dom_bytes = {"fit": ab["fit"], "project": ab["wq"], "vote": ab["k"], "compact": ab["compact"],
                 "sample": 0}.get(STAGE_OF.get(dom, "other"), 0)
    dom_avg_s = prof[dom][1] / prof[dom][0] * 1e-3
    achieved = dom_bytes / dom_avg_s / 1e9 if dom_avg_s > 0 else 0.0
    traffic = None
    tpath = os.path.join(ROOT, "profiles", f"{dom}_{cfg.name}_dram_bytes.txt")
    if os.path.exists(tpath):
        try:
            traffic = float(open(tpath).read().split()[0])
        except Exception:
            traffic = None
    roofline = {"bound": "hbm", "scope": "dominant kernel", "kernel": dom, "achieved": achieved, "peak": hbm_gbs, "unit": "GB/s",
                "frac": achieved / hbm_gbs, "traffic": traffic, "peak_kind": f"of {peak_kind}",
                "algorithmic_bytes_per_launch": dom_bytes, "avg_launch_us": dom_avg_s * 1e6,
                "timed_with": "CUDA event pairs around every launch on the launch stream, same steps repeated"}
    lit_t = max((f_proj + f_score) / (bf16_tf * 1e12), (ab["k"] + ab["compact"]) / (hbm_gbs * 1e9))
    full_t = max((f_proj + f_score) / (bf16_tf * 1e12),
                 (ab["fit"] + ab["wq"] + ab["k"] + ab["compact"]) / (hbm_gbs * 1e9))
    layer_s = ms_per_step * 1e-3 / L
    sel_s = (stage_us.get("project", 0) + stage_us.get("vote", 0) + stage_us.get("compact", 0)) * 1e-6
    # the uninstrumented pass on ONE stream (what an engine that compresses layer by layer sees)
    one_ms = 0.0
    for _ in range(args.steps):
        restore()
        barrier()
        ev0.record()
        one_pass(spread=False)
        ev1.record()
        torch.cuda.synchronize()
        one_ms += ev0.elapsed_time(ev1)
    one_ms = shard.max_over_ranks(one_ms, dist, dev) / args.steps
    one_stream_row = {"value": shard.job_throughput(cfg.total_tokens, world, one_ms * 1e-3), "unit": UNIT,
                      "ms_per_step": one_ms, "per_layer_us": one_ms * 1e3 / L,
                      "full_bytes_frac": full_t / (one_ms * 1e-3 / L), "literal_frac": lit_t / (one_ms * 1e-3 / L),
                      "note": "extra row: the same pass with every layer on one stream, no per-kernel events; not the headline"}
    # the same one-stream pass recorded once as a CUDA graph and replayed: what an engine that compresses layer
    # by layer gets when it captures the calls instead of enqueueing twelve launches per layer from the host
    if not args.no_graph_row:
        graph = torch.cuda.CUDAGraph()
        restore()
        torch.cuda.synchronize()
        with torch.cuda.graph(graph, capture_error_mode="thread_local"):
            one_pass(spread=False)
        torch.cuda.synchronize()
        g_ms = 0.0
        for i in range(2 + args.steps):                  # two untimed replays first
            restore()
            barrier()
            ev0.record()
            graph.replay()
            ev1.record()
            torch.cuda.synchronize()
            if i >= 2:
                g_ms += ev0.elapsed_time(ev1)
        g_ms = shard.max_over_ranks(g_ms, dist, dev) / args.steps
        del graph
        assert gv.gvote_poll_status(ws) == 0, "a device-side wait timed out"
        one_stream_row["as_cuda_graph"] = {
            "value": shard.job_throughput(cfg.total_tokens, world, g_ms * 1e-3), "unit": UNIT, "ms_per_step": g_ms,
            "per_layer_us": g_ms * 1e3 / L, "full_bytes_frac": full_t / (g_ms * 1e-3 / L),
            "note": "the one-stream pass captured once (torch.cuda.graph around the same gvote_compress calls) and replayed"}
    roofline["pass"] = {
        "note": "whole pass against its own roofline: the slower of the bf16 flops at the tensor peak and the bytes at "
                "the HBM peak; 'literal' counts the K read and the K/V compaction bytes only, 'full_bytes' also the "
                "hidden states the fit must read and W_q",
        "literal_frac": lit_t / layer_s, "full_bytes_frac": full_t / layer_s, "target_frac": 0.6,
        "target_met_literal": bool(lit_t / layer_s >= 0.6), "target_met_full_bytes": bool(full_t / layer_s >= 0.6),
        "fit_read_over_literal_roofline": (ab["fit"] / (hbm_gbs * 1e9)) / lit_t}
    pass_roofline = {
        "kept_fraction": kept_frac, "per_layer_us": layer_s * 1e6, "stage_us_per_layer": stage_us,
        "token_layers_per_s": value * L,
        "per_layer_us_one_stream_instrumented": serial_ms * 1e3 / L,
        "full_bytes_roofline_us": full_t * 1e6, "full_bytes_frac": full_t / layer_s,
        "literal_roofline_us": lit_t * 1e6, "literal_frac_whole_pass": lit_t / layer_s,
        "literal_frac_select_compact_only": (lit_t / sel_s) if sel_s > 0 else None,
        "peaks": {"hbm_gbs": hbm_gbs, "bf16_tflops": bf16_tf, "kind": peak_kind},
    }

    # ---- extra row (labelled, not the headline): the same pass when the engine has fitted the Gaussian
    # upstream, during prefill (gvote_fit_update / gvote_fit_finish), so the pass starts at the sampling
    upstream = None
    if not args.no_upstream_row:
        d_mu = [torch.empty(cfg.batch, cfg.d_h, device=dev) for _ in range(L)]
        d_var = [torch.empty(cfg.batch, cfg.d_h, device=dev) for _ in range(L)]
        cu_h = layers[0].cu_seqlens
        d_hl = [torch.stack([d_h[l][int(cu_h[r + 1]) - 1] for r in range(cfg.batch)]).contiguous() for l in range(L)]
        for l in range(L):
            gv.gvote_fit(p_layer[l], d_h[l], cu, geom, d_mu[l], d_var[l], ws)
        torch.cuda.synchronize()
        if STAGE_OF.get(dom) == "fit":
            # the dominant kernel once more without an event pair around every launch: the fits of all
            # layers back to back on one stream between two events (the tiny merge kernel rides along)
            ev0.record()
            for l in range(L):
                gv.gvote_fit(p_layer[l], d_h[l], cu, geom, d_mu[l], d_var[l], ws)
            ev1.record()
            torch.cuda.synchronize()
            b2b_us = ev0.elapsed_time(ev1) * 1e3 / L
            roofline["back_to_back"] = {"avg_launch_us": b2b_us, "achieved": dom_bytes / (b2b_us * 1e-6) / 1e9,
                                        "frac": dom_bytes / (b2b_us * 1e-6) / 1e9 / hbm_gbs,
                                        "note": "gvote_fit of every layer back to back on one stream, one event "
                                                "pair around all of them (includes the merge kernel)"}

        def one_pass_moments():
            main = torch.cuda.current_stream()
            if side:
                fork = torch.cuda.Event()
                fork.record(main)
                for st in side:
                    st.wait_event(fork)
            for l in range(L):
                k = l % n_streams
                with torch.cuda.stream(main if k == 0 else side[k - 1]):
                    gv.gvote_compress_moments(p_layer[l], d_mu[l], d_var[l], d_hl[l], d_W[l], None, d_K[l], d_V[l], cu,
                                              geom, d_mask[l], d_budget[l], d_bstep[l], ws_s[k])
            for st in side:
                join = torch.cuda.Event()
                join.record(st)
                main.wait_event(join)

        up_ms = 0.0
        for s_ in range(3 + args.steps):
            restore()
            barrier()
            ev0.record()
            one_pass_moments()
            ev1.record()
            torch.cuda.synchronize()
            if s_ >= 3:
                up_ms += ev0.elapsed_time(ev1)
        up_ms = shard.max_over_ranks(up_ms, dist, dev) / args.steps
        upstream = {"value": shard.job_throughput(cfg.total_tokens, world, up_ms * 1e-3), "unit": UNIT,
                    "ms_per_step": up_ms,
                    "note": "extra row: gvote_compress_moments, i.e. Algorithm 1 from the sampling step on, with mu and var "
                            "fitted beforehand (the engine accumulates them during prefill); not the headline"}

    # ---- extra row (labelled, not the headline): the pass applied again to the cache it has just pruned,
    # after 256 more tokens per head (gvote_recompress: per-head key counts, positions from tokens seen)
    recompress = None
    if not args.no_upstream_row and not args.no_recompress_row:
        restore()
        one_pass()
        torch.cuda.synchronize()
        grown = 256
        lens = torch.from_numpy(np.diff(layers[0].cu_seqlens).astype(np.int32)).to(dev)
        d_len = [torch.minimum(d_budget[l] + grown, lens[:, None]).contiguous() for l in range(L)]
        d_seen = lens + grown
        d_K1 = [t.clone() for t in d_K]
        d_V1 = [t.clone() for t in d_V]
        r_budget = [torch.empty_like(b) for b in d_budget]
        r_mask = [torch.empty_like(m_) for m_ in d_mask]
        r_bstep = [torch.empty_like(b) for b in d_bstep]
        rows_mean = float(torch.stack(d_len).float().mean().item())

        def one_pass_again():
            main = torch.cuda.current_stream()
            if side:
                fork = torch.cuda.Event()
                fork.record(main)
                for st in side:
                    st.wait_event(fork)
            for l in range(L):
                k = l % n_streams
                with torch.cuda.stream(main if k == 0 else side[k - 1]):
                    gv.gvote_recompress(p_layer[l], d_mu[l], d_var[l], d_hl[l], d_W[l], None, d_K[l], d_V[l], cu, d_len[l],
                                        d_seen, None, geom, r_mask[l], r_budget[l], r_bstep[l], ws_s[k])
            for st in side:
                join = torch.cuda.Event()
                join.record(st)
                main.wait_event(join)

        re_ms = 0.0
        for s_ in range(3 + args.steps):
            for l in range(L):
                d_K[l].copy_(d_K1[l]); d_V[l].copy_(d_V1[l])
            barrier()
            ev0.record()
            one_pass_again()
            ev1.record()
            barrier()
            if s_ >= 3:
                re_ms += ev0.elapsed_time(ev1)
        re_ms = shard.max_over_ranks(re_ms, dist, dev) / args.steps
        kept_again = float(torch.stack(r_budget).float().mean().item())
        recompress = {"value": shard.job_throughput(cfg.total_tokens, world, re_ms * 1e-3), "unit": UNIT,
                      "ms_per_step": re_ms, "rows_per_head_before": rows_mean, "rows_per_head_after": kept_again,
                      "note": "extra row: gvote_recompress on the cache the first pass left, 256 rows later "
                              "(mu and var given, as in upstream_fit_row); tokens = tokens of history; not the headline"}
        del d_K1, d_V1

    # ---- extra row (labelled, not the headline): the same pass over hidden states held in bf16, as an
    # engine that runs the model in bf16 has them (half the bytes of the fit)
    bf16_row = None
    if not args.no_upstream_row:
        d_hb = [t.bfloat16() for t in d_h]
        p_b = [gv.params_from_config(cfg, layer_id=l, h_dtype=gv.DTYPE_BF16) for l in range(L)]

        def one_pass_bf16():
            main = torch.cuda.current_stream()
            if side:
                fork = torch.cuda.Event()
                fork.record(main)
                for st in side:
                    st.wait_event(fork)
            for l in range(L):
                k = l % n_streams
                with torch.cuda.stream(main if k == 0 else side[k - 1]):
                    gv.gvote_compress(p_b[l], d_hb[l], d_W[l], None, d_K[l], d_V[l], cu, geom, d_mask[l], d_budget[l],
                                      d_bstep[l], ws_s[k])
            for st in side:
                join = torch.cuda.Event()
                join.record(st)
                main.wait_event(join)

        b_ms = 0.0
        for s_ in range(3 + args.steps):
            restore()
            barrier()
            ev0.record()
            one_pass_bf16()
            ev1.record()
            barrier()
            if s_ >= 3:
                b_ms += ev0.elapsed_time(ev1)
        b_ms = shard.max_over_ranks(b_ms, dist, dev) / args.steps
        bf16_row = {"value": shard.job_throughput(cfg.total_tokens, world, b_ms * 1e-3), "unit": UNIT,
                    "ms_per_step": b_ms,
                    "note": "extra row: gvote_compress with h_dtype = bf16 (the workload's hidden states rounded to "
                            "bf16); not the headline, which reads them as fp32"}
        del d_hb
        # leave the headline's results in the output buffers for the checks below
        restore()
        one_pass()
        torch.cuda.synchronize()

    # ---- end to end through the host-memory entry point
    e2e = None
    if not args.no_e2e:
        hK0 = [gv.bf16_from_bits(li.K, "cpu") for li in layers]
        hV0 = [gv.bf16_from_bits(li.V, "cpu") for li in layers]
        hh = [torch.from_numpy(li.h).pin_memory() for li in layers]
        hW = [gv.bf16_from_bits(li.W_q, "cpu", pin=True) for li in layers]
        hK = [t.clone().pin_memory() for t in hK0]
        hV = [t.clone().pin_memory() for t in hV0]
        hcu = torch.from_numpy(layers[0].cu_seqlens)
        hmask = [torch.empty(cfg.n_kv_heads, words, dtype=torch.int32).pin_memory() for _ in range(L)]
        hbud = [torch.empty(cfg.batch, cfg.n_kv_heads, dtype=torch.int32).pin_memory() for _ in range(L)]
        hbs = [torch.empty(cfg.batch, cfg.n_q_heads, dtype=torch.int32).pin_memory() for _ in range(L)]
        e2e_total = 0.0
        n_e2e = max(1, args.e2e_steps)
        for s in range(1 + n_e2e):
            for l in range(L):
                hK[l].copy_(hK0[l]); hV[l].copy_(hV0[l])
            barrier()
            t0 = time.perf_counter()
            for l in range(L):
                gv.gvote_compress_host(p_layer[l], hh[l], hW[l], None, hK[l], hV[l], hcu, hmask[l], hbud[l], hbs[l])
            dt = time.perf_counter() - t0
            if s >= 1:
                e2e_total += dt
        e2e_total = shard.max_over_ranks(e2e_total, dist, dev)
        gv.gvote_host_arena_release()
        h2d = sum(a.numel() * a.element_size() for l in range(L) for a in (hh[l], hW[l], hK[l], hV[l])) + L * hcu.numel() * 4
        d2h = sum(a.numel() * a.element_size() for l in range(L) for a in (hK[l], hV[l], hmask[l], hbud[l], hbs[l]))
        e2e = {"value": world * cfg.total_tokens / (e2e_total / n_e2e), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "steps": n_e2e, "ms_per_step": e2e_total / n_e2e * 1e3}
        same = all(np.array_equal(hbud[l].numpy(), d_budget[l].cpu().numpy()) for l in range(L))
        e2e["budgets_match_device_run"] = bool(same)

    # ---- the oracle on the host cores, on a bounded sample (rank 0, one GPU only)
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        # whole layers, until about ten seconds of oracle time have gone by (three layers of the 32K workload)
        t_or, n_or, ok = 0.0, 0, True
        tol = np.maximum(2, 0.005 * np.asarray(cfg.seq_lens)[:, None])
        while n_or < L and (n_or == 0 or t_or < 10.0):
            t_l, res = time_oracle_layer(cfg, layers[n_or], n_or)
            ob = np.stack([r.budget for r in res])
            ok = ok and bool(np.all(np.abs(ob - d_budget[n_or].cpu().numpy()) <= tol))
            t_or += t_l
            n_or += 1
        cpu_baseline = {"value": cfg.total_tokens * n_or / (t_or * L), "unit": UNIT, "cores": blas_threads(),
                        "kind": "oracle", "sample": f"layers 0..{n_or - 1} of {L} ({cfg.total_tokens} tokens each) took {t_or:.1f} s "
                        f"in the fp64 NumPy oracle as it stands (matmul, sort, cumsum are NumPy's; BLAS threads = cores); "
                        f"value = tokens / (the mean layer time x {L} layers)", "budgets_within_tolerance": ok}

    if rank == 0:
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": workload_config(cfg, args),
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "exact_route_heads": int(exact_heads),
            "roofline": roofline,
            "cpu_baseline": cpu_baseline, "pass_roofline": pass_roofline, "one_stream_row": one_stream_row,
            "upstream_fit_row": upstream, "recompress_row": recompress, "bf16_h_row": bf16_row, "kernels": per_kernel,
            "setup_s": {"generate": t_gen},
        }
        print(json.dumps(out))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
