#!/usr/bin/env python
"""Benchmark of the FastOCR decode-step attention hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

One "step" is one post-warm-up decode step of Algorithm 1 over all layers of the workload: focal
layers run dense attention with fused scoring plus top-k, every other layer runs pruned attention
over text + the current fixation set, the set of the deepest focal layer is carried to the next
step. The default workload is the roofline-sweep point the target is stated on (7B-shaped heads,
batch 64, N = 8192 image tokens, 256 text tokens, tau = 0.05) with 28 distinct layer caches
(31 GB, far beyond L2) scheduled with rho = 0.1 as in the 7B-shaped decode configuration.

Prints ONE JSON line (rank 0). Roofline figures use algorithmic bytes: the K and V rows the
method must read (2 x H_kv x 128 x 2 bytes per attended token) plus the index list.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import tempfile
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from workloads import fixation_track, get_config, make_kv, make_queries, make_page_table, scatter_to_pages  # noqa: E402

NOMINAL_HBM_GBS = 8000.0


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-slices", type=int, default=4, help="layer slices per end-to-end step (copies of one overlap the arithmetic of the next)")
    ap.add_argument("--workload", default="cfg4", choices=["cfg0", "cfg1", "cfg2", "cfg3", "cfg4"])
    ap.add_argument("--N", type=int, default=8192, help="image tokens (cfg4 only)")
    ap.add_argument("--batch", type=int, default=64, help="sequences (cfg4 only)")
    ap.add_argument("--tau", type=float, default=None)
    ap.add_argument("--layers", type=int, default=None, help="override the number of layer caches")
    ap.add_argument("--distinct-steps", type=int, default=16, help="length of the replayed fixation track")
    ap.add_argument("--focal", default=None, help="comma-separated focal layers (skips Focal Layer Selection)")
    ap.add_argument("--graph", default="auto", choices=["auto", "on", "off"],
                    help="replay each decode step from a CUDA graph (auto: on for the single-sequence workloads)")
    ap.add_argument("--sweep", action="store_true", help="roofline sweep over N and tau (7B-shaped layer, batch 64); prints one JSON line")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--cpu-seconds", type=float, default=15.0, help="target CPU time of the oracle sample")
    ap.add_argument("--per-seq-focal", action="store_true", help="one focal layer set per sequence (profiled per sample) instead of one for the batch")
    ap.add_argument("--union-sets", action="store_true", help="the union-of-selections variant of the step")
    ap.add_argument("--sustained-seconds", type=float, default=0.6,
                    help="when the K timed steps take less than this, a second region of at least this length is timed too")
    return ap.parse_args()


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def workload_config(args):
    if args.workload == "cfg4":
        cfg = get_config("cfg4", N=args.N, batch=args.batch, layers=args.layers or 28)
        cfg.name = f"cfg4[N={args.N},B={args.batch}]x{cfg.layers}layers"
    else:
        cfg = get_config(args.workload)
        if args.layers:
            cfg.layers = args.layers
    if args.tau is not None:
        cfg.tau = args.tau
    return cfg


class Workload:
    """Device-resident synthetic decode state: per-layer caches, a cyclic track of `n_distinct`
    decode steps (queries + sequence lengths), kept counts."""

    def __init__(self, cfg, n_distinct, device, rank=0, seq_slice=None, device_api=True):
        from workloads import kept_count_hint
        fo = None
        if device_api:
            import paper_2605_17447_b200 as fo
        self.cfg, self.dev, self.nd = cfg, device, n_distinct
        B_all = cfg.batch
        lo, hi = seq_slice or (0, B_all)
        self.seqs = list(range(lo, hi))
        B = self.B = hi - lo
        self.seq_offset = rank * B_all + lo            # distinct data per rank (weak scaling)
        self.H, self.Hkv, self.L = cfg.num_q_heads, cfg.num_kv_heads, cfg.layers
        self.vis_start = [cfg.vis_start[b] for b in self.seqs]
        self.vis_len = [cfg.vis_len[b] for b in self.seqs]
        self.S0 = [cfg.seq_len(0)[b] for b in self.seqs]
        self.text0 = [s - n for s, n in zip(self.S0, self.vis_len)]
        self.k = [(fo.kept_count if fo else kept_count_hint)(n, cfg.tau) for n in self.vis_len]
        self.S_stride = max(self.S0) + n_distinct
        self.max_kept = max(k + t for k, t in zip(self.k, self.text0)) + n_distinct
        self.sm_scale = 1.0 / math.sqrt(cfg.head_dim)
        i32 = lambda x: torch.tensor(x, dtype=torch.int32, device=device)
        self.vis_start_d, self.vis_len_d, self.k_d = i32(self.vis_start), i32(self.vis_len), i32(self.k)
        # step s of the track attends S0 + s + 1 tokens (the current token included)
        self.seq_len_table = torch.stack([i32([s0 + s + 1 for s0 in self.S0]) for s in range(n_distinct)])
        self.seq_len_d = self.seq_len_table[0].clone()
        gh = torch.tensor([cfg.grid_h[b] for b in self.seqs], device=device)
        gw = torch.tensor([cfg.grid_w[b] for b in self.seqs], device=device)
        tracks = np.stack([fixation_track(cfg.seed, self.seq_offset + i, n_distinct, cfg.grid_h[b], cfg.grid_w[b], cfg.advance)
                           for i, b in enumerate(self.seqs)])                                 # [B][nd][2]
        self.views, self.K, self.V = [], [], []
        self.q_all = torch.empty(n_distinct, self.L, B, self.H, cfg.head_dim, dtype=torch.bfloat16, device=device)
        self.block_table = None
        if cfg.page_size:
            table, self.num_pages = make_page_table(cfg.seed + rank, [self.S_stride] * B, cfg.page_size)
            self.block_table = table.to(device)
        # all layers' caches in one allocation per tensor ([L] leading), so that a decode step's new rows go
        # into every layer's cache with one scatter per tensor; layer l's cache is the view [l]
        self.K_all = self.V_all = None
        for l in range(self.L):
            K, V = make_kv(cfg.seed, l, B, self.S_stride, self.Hkv, cfg.head_dim, device, seq_offset=self.seq_offset)
            for s in range(n_distinct):
                centres = torch.tensor(tracks[:, s, :], device=device)
                self.q_all[s, l] = make_queries(cfg.seed, l, s, lambda b, pos: K[b, pos], self.vis_start_d.long(), centres,
                                                gh, gw, self.H, seq_offset=self.seq_offset)
            if cfg.page_size:
                K = scatter_to_pages(K, [self.S_stride] * B, self.block_table.cpu(), self.num_pages, cfg.page_size)
                V = scatter_to_pages(V, [self.S_stride] * B, self.block_table.cpu(), self.num_pages, cfg.page_size)
            if self.K_all is None:
                self.K_all = torch.empty((self.L,) + tuple(K.shape), dtype=K.dtype, device=device)
                self.V_all = torch.empty_like(self.K_all)
            self.K_all[l].copy_(K)
            self.V_all[l].copy_(V)
            K, V = self.K_all[l], self.V_all[l]
            self.K.append(K)
            self.V.append(V)
            if fo:
                self.views.append(fo.KVView(K, V, self.seq_len_d, self.vis_start_d, self.vis_len_d, self.H, self.S_stride,
                                            self.sm_scale, block_table=self.block_table))
        self.fo = fo
        if fo:
            self.ctx = fo.Context(B, self.H, self.Hkv, self.S_stride, max(self.vis_len))
            self.fix = torch.zeros(B, max(max(self.k), 1), dtype=torch.int32, device=device)

    def flat_row(self, s):
        """Row index (into the cache viewed as [rows][Hkv][d]) of the token appended at track step s."""
        pos = torch.tensor([s0 + s for s0 in self.S0], device=self.dev)
        b = torch.arange(self.B, device=self.dev)
        if self.cfg.page_size:
            ps = self.cfg.page_size
            return self.block_table[b, pos // ps].long() * ps + pos % ps
        return b * self.S_stride + pos

    # ---- byte model: rows of K and V the method must read, bf16 ----
    def row_bytes(self):
        return self.Hkv * self.cfg.head_dim * 2

    def dense_bytes(self, s):
        return 2 * self.row_bytes() * sum(s0 + s + 1 for s0 in self.S0)

    def sparse_bytes(self, s):
        return 2 * self.row_bytes() * sum(k + t + s + 1 for k, t in zip(self.k, self.text0)) + 4 * sum(self.k)

    def set_step(self, s):
        self.seq_len_d.copy_(self.seq_len_table[s % self.nd])

    def logical_rows(self, l, b, S):
        """K, V rows [S][Hkv][d] of local sequence b, layer l, as CPU tensors (for the oracle)."""
        if self.cfg.page_size:
            ps = self.cfg.page_size
            pages = self.block_table[b, :(S + ps - 1) // ps].long()
            K = self.K[l][pages].reshape(-1, self.Hkv, self.cfg.head_dim)[:S]
            V = self.V[l][pages].reshape(-1, self.Hkv, self.cfg.head_dim)[:S]
        else:
            K, V = self.K[l][b, :S], self.V[l][b, :S]
        return K.cpu().contiguous(), V.cpu().contiguous()


def choose_focal_layers(w: Workload, per_sequence=False):
    """Focal Layer Selection (Section 3.1.1; Algorithm 1's profiling block): w warm-up steps through
    fastocr_warmup_step (every layer dense, Eq. 1's ratio per layer and sequence from the same pass),
    then rank + greedy gap on the means. Untimed set-up. One set for the batch (from the batch mean of
    the ratios: the synthetic layers differ only by noise) or, with per_sequence, one per sequence."""
    cfg, fo = w.cfg, w.fo
    steps = max(1, min(cfg.warmup, w.nd))
    out = torch.empty(w.L, w.B, w.H, cfg.head_dim, dtype=torch.bfloat16, device=w.dev)
    r = torch.zeros(w.L, w.B, dtype=torch.float32, device=w.dev)
    ratio = np.zeros((steps, w.L, w.B))
    for s in range(steps):
        w.set_step(s)
        fo.fastocr_warmup_step(w.ctx, w.views, w.q_all[s], out, r)
        ratio[s] = r.cpu().numpy()
    mean = ratio.mean(axis=0)                                       # [L][B]
    if per_sequence:
        sets = [fo.focal_layers(mean[:, b], cfg.rho, cfg.gap) for b in range(w.B)]
        return sets, mean
    return fo.focal_layers(mean.mean(axis=1), cfg.rho, cfg.gap), mean


class ClockSampler:
    """nvidia-smi sampling in the background (every 20 ms, each sample with its wall-clock time), started
    before the warm-up and read out per measured region afterwards."""
    Q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.rows = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--id={index}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                       "-lms", "20"], stdout=self.f, stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None

    def stop(self):
        if self.p is None or self.rows is not None:
            return
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        import datetime
        self.rows = []
        for r in open(self.f.name):
            c = r.strip().split(", ")
            try:
                t = datetime.datetime.strptime(c[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                self.rows.append((t, float(c[1]), float(c[2]), float(c[3]), [v.strip().lower().startswith("active") for v in c[5:9]]))
            except (ValueError, IndexError):
                continue
        os.unlink(self.f.name)

    def window(self, t0, t1, pad=0.06):
        """Summary of the samples taken in [t0 - pad, t1 + pad] (wall-clock seconds)."""
        if self.p is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.stop()
        rows = [r for r in self.rows if t0 - pad <= r[0] <= t1 + pad]
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        reasons = set()
        for r in rows:
            for name, on in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[4]):
                if on:
                    reasons.add(name)
        return {"sm_mhz": float(np.median([r[1] for r in rows])), "sm_max_mhz": max(r[2] for r in rows), "reasons": sorted(reasons),
                "samples": len(rows), "power_w_max": max(r[3] for r in rows)}


def timed(fn, steps, dist_barrier, wall=None):
    """ms for `steps` calls, CUDA events on the current stream between a barrier + synchronize on both
    sides; wall (a list) receives the region's wall-clock start and end."""
    dist_barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.time()
    e0.record()
    for t in range(steps):
        fn(t)
    e1.record()
    torch.cuda.synchronize()
    t1 = time.time()
    dist_barrier()
    if wall is not None:
        wall[:] = [t0, t1]
    return e0.elapsed_time(e1)


def oracle_step_sample(w: Workload, focal, seq_ids, s, carried=None):
    """The oracle's Algorithm-1 step for some sequences of track step s. Returns seconds of oracle
    compute (input copies excluded) and the traces. The set carried in from step s - 1 is the oracle's
    own (its scoring of the previous step's deepest focal layer) unless `carried` gives one per sequence."""
    import oracle
    cfg = w.cfg
    total, traces = 0.0, []
    deepest = max(focal) if focal else 0
    for b in seq_ids:
        S = w.S0[b] + s + 1
        layers = []
        for l in range(w.L):
            K, V = w.logical_rows(l, b, S)
            layers.append((w.q_all[s % w.nd, l, b].cpu(), K, V))
        # last step's fixation set, from the oracle's own scoring of the previous step
        if carried is not None:
            f_last = carried[b]
        else:
            sp = (s - 1) % w.nd
            Kp, _ = w.logical_rows(deepest, b, w.S0[b] + sp + 1)
            sc, _ = oracle.scores(w.q_all[sp, deepest, b].cpu(), Kp, w.sm_scale, w.vis_start[b], w.vis_len[b])
            f_last = oracle.topk(sc, w.k[b])
        t0 = time.perf_counter()
        tr = oracle.decode_step(layers, focal, f_last, w.vis_start[b], w.vis_len[b], cfg.tau, w.sm_scale)
        total += time.perf_counter() - t0
        traces.append(tr)
    return total, traces


def run_reference(args):
    """Reference arm: the CPU oracle, as it stands, on a bounded sample of the same workload.
    Each timed step is one sequence's Algorithm-1 step over a subset of the layers, sized so that
    the whole run ends within a few minutes; the value is scaled to the full batch and depth."""
    import oracle
    cfg = workload_config(args)
    dev = "cuda" if torch.cuda.is_available() else "cpu"      # holds inputs only; the oracle runs on host cores
    budget = 120.0 / max(1, args.steps + args.warmup)         # seconds of oracle time per step
    threads = max(1, min(oracle.num_threads(), cfg.num_q_heads))
    S = cfg.seq_len(0)[0]
    per_layer = 4e-9 * cfg.num_q_heads * cfg.head_dim * S * (3 * cfg.rho + 0.15) / threads   # rough
    n_layers = cfg.layers
    while n_layers > 4 and per_layer * n_layers > budget:
        n_layers = max(4, n_layers // 2)
    sub = workload_config(args)
    sub.layers = n_layers
    w = Workload(sub, 2, dev, seq_slice=(0, 1), device_api=False)
    ratios = []
    for l in range(n_layers):                                  # one warm-up step of Eq. 1 per layer
        K, _ = w.logical_rows(l, 0, w.S0[0] + 1)
        ratios.append(oracle.scores(w.q_all[0, l, 0].cpu(), K, w.sm_scale, w.vis_start[0], w.vis_len[0])[1])
    focal = oracle.profile_focal_layers([ratios], max(cfg.rho, 1.0 / n_layers), cfg.gap)
    for _ in range(args.warmup):
        oracle_step_sample(w, focal, [0], 1)
    t = 0.0
    for _ in range(args.steps):
        dt, _ = oracle_step_sample(w, focal, [0], 1)
        t += dt
    per_step_full = t / max(1, args.steps) * cfg.batch * (cfg.layers / n_layers) * 1e6
    sample = (f"1 of {cfg.batch} sequences, {n_layers} of {cfg.layers} layers ({len(focal)} focal), "
              f"scaled to the full batch and depth")
    line = {"impl": "reference", "metric": "fastocr decode-attention step time", "value": per_step_full, "unit": "us/step",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": per_step_full / 1e3,
            "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": cfg.name, "tau": cfg.tau, "rho": cfg.rho},
            "cpu_baseline": {"value": per_step_full, "unit": "us/step", "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": per_step_full, "unit": "us/step", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def run_sweep(args):
    """Roofline sweep (7B-shaped layer, batch 64, N x tau grid): per point, the pruned layer and the dense layer
    timed back to back over 8 distinct layer caches (so every launch reads cold data), plus
    scoring + selection, as us per layer and GB/s of algorithmic bytes."""
    import paper_2605_17447_b200 as fo
    peak, peak_kind = measured_peaks()
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    points = []
    reps = 20
    for N in (1024, 4096, 8192, 16384, 32768):
        for tau in (0.02, 0.05, 0.10, 0.20, 1.0):
            cfg = get_config("cfg4", N=N, batch=args.batch, layers=8, tau=tau)
            if tau == 0.02:                       # one data set per N; tau only changes k
                w = Workload(cfg, 2, dev)
            else:
                w.cfg.tau = tau
                w.k = [fo.kept_count(n, tau) for n in w.vis_len]
                w.k_d.copy_(torch.tensor(w.k, dtype=torch.int32))
                w.fix = torch.zeros(w.B, max(w.k), dtype=torch.int32, device=dev)
            w.max_kept = max(k + t for k, t in zip(w.k, w.text0)) + w.nd
            out = torch.empty(w.L, w.B, w.H, cfg.head_dim, dtype=torch.bfloat16, device=dev)
            q = w.q_all[0]
            w.set_step(0)
            # a real selection for this tau: one focal pass on layer 0
            sel = fo.StepPlan(w.ctx, w.views[:1], [True], w.k_d, w.fix, max(w.vis_len))
            sel.run(q[:1], out[:1], False)
            chain = fo.StepPlan(w.ctx, w.views, [False] * w.L, w.k_d, w.fix, max(w.vis_len), w.max_kept)
            def sparse_chain(t):
                chain.run(q, out, True)
            def dense_chain(t):
                for l in range(w.L):
                    fo.fastocr_dense_decode_attn(w.ctx, w.views[l], q[l], out[l])
            scores = torch.zeros(w.B, max(w.vis_len), dtype=torch.float32, device=dev)
            def select_only(t):
                fo.fastocr_focal_scores(w.ctx, w.views[t % w.L], q[t % w.L], scores)
                fo.fastocr_select_topk(w.ctx, scores, w.vis_len_d, w.k_d, w.fix, max(w.vis_len))
            res = {}
            for name, fn, per in (("sparse", sparse_chain, w.L), ("dense", dense_chain, w.L), ("scores_topk", select_only, 1)):
                for t in range(3):
                    fn(t)
                res[name] = timed(fn, reps, lambda: None) / reps / per * 1e3
            sel.run(q[:1], out[:1], False)        # leave a valid selection behind
            sb, db = w.sparse_bytes(0), w.dense_bytes(0)
            points.append({"N": N, "tau": tau, "k": w.k[0], "sparse_us": res["sparse"], "dense_us": res["dense"],
                           "scores_topk_us": res["scores_topk"], "sparse_gbs": sb / res["sparse"] / 1e3,
                           "dense_gbs": db / res["dense"] / 1e3, "sparse_frac_of_8tbs": sb / res["sparse"] / 1e3 / NOMINAL_HBM_GBS,
                           "sparse_frac_of_measured": sb / res["sparse"] / 1e3 / peak, "dense_frac_of_measured": db / res["dense"] / 1e3 / peak,
                           "layer_speedup": res["dense"] / res["sparse"]})
        del w
        torch.cuda.empty_cache()
    print(json.dumps({"sweep": "cfg4", "batch": args.batch, "layers_cycled": 8, "peak_gbs": peak, "peak_kind": peak_kind, "points": points}))


def main():
    args = parse_args()
    if args.sweep:
        run_sweep(args)
        return
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        if rank == 0:
            run_reference(args)
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist_mod.init_process_group("nccl", device_id=dev)
        dist = dist_mod
    barrier = (lambda: dist.barrier()) if dist else (lambda: None)

    import paper_2605_17447_b200 as fo
    cfg = workload_config(args)
    peak, peak_kind = measured_peaks()
    # sequences are independent: every rank holds its own full batch (weak scaling), no data-path collective
    w = Workload(cfg, args.distinct_steps, dev, rank=rank)
    clocks = ClockSampler(local)                  # runs from here to the end of the measured regions
    focal_sets = None                             # per-sequence focal layer sets, when asked for
    if args.focal is not None:
        focal = sorted(int(x) for x in args.focal.split(",") if x != "")
    elif args.per_seq_focal:
        focal_sets, _ = choose_focal_layers(w, per_sequence=True)
        focal = sorted(set(l for c in focal_sets for l in c))
    else:
        focal, _ = choose_focal_layers(w)
    is_focal = [l in focal for l in range(w.L)]
    if focal_sets is not None:
        is_focal = [[l in focal_sets[b] for b in range(w.B)] for l in range(w.L)]
    out = torch.empty(w.L, w.B, w.H, cfg.head_dim, dtype=torch.bfloat16, device=dev)
    n_union = max(1, len(focal)) if args.union_sets else 1
    if args.union_sets:
        w.max_kept = max(n_union * k + t for k, t in zip(w.k, w.text0)) + w.nd
    plan = fo.StepPlan(w.ctx, w.views, is_focal, w.k_d, w.fix, max(w.vis_len), w.max_kept, union_sets=args.union_sets)
    state = {"have": False}

    def fastocr_step(t):
        w.set_step(t)
        state["have"] = plan.run(w.q_all[t % w.nd], out, state["have"])

    def dense_step(t):
        w.set_step(t)
        for l in range(w.L):
            fo.fastocr_dense_decode_attn(w.ctx, w.views[l], w.q_all[t % w.nd, l], out[l])

    for t in range(max(3, args.warmup)):
        fastocr_step(t)
    # Small batches are bound by the host's launch rate: capture one CUDA graph per distinct step of
    # the track (same kernels, same order, same arguments) and replay those in the timed region.
    use_graph = args.graph == "on" or (args.graph == "auto" and w.B * w.Hkv < 64)
    eager_step = fastocr_step
    launches_per_step = None
    if use_graph:
        torch.cuda.synchronize()
        graphs = []
        l0 = fo.launch_count()
        side = torch.cuda.Stream()
        with torch.cuda.stream(side):
            for s_ in range(w.nd):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=side):
                    w.set_step(s_)
                    plan.run(w.q_all[s_], out, True)
                graphs.append(g)
        torch.cuda.synchronize()
        launches_per_step = (fo.launch_count() - l0) // w.nd

        def fastocr_step(t):                      # noqa: F811
            graphs[t % w.nd].replay()
        for t in range(3):
            fastocr_step(t)
    launches0 = fo.launch_count()
    wall = [0.0, 0.0]
    ms = timed(fastocr_step, args.steps, barrier, wall)
    launches = fo.launch_count() - launches0 if launches_per_step is None else launches_per_step * args.steps
    # A short timed region is a burst figure (the board has not reached its power limit yet): time a
    # second, longer region too and report both.
    sustained = None
    if ms / 1e3 < args.sustained_seconds:
        n_sus = int(math.ceil(args.sustained_seconds * 1.1 / max(ms / 1e3 / args.steps, 1e-6)))
        wall_sus = [0.0, 0.0]
        ms_sus = timed(fastocr_step, n_sus, barrier, wall_sus)
        if dist:
            tt = torch.tensor([ms_sus], device=dev, dtype=torch.float64)
            dist.all_reduce(tt, op=dist.ReduceOp.MAX)
            ms_sus = float(tt[0])
        sustained = {"us_per_step": ms_sus / n_sus * 1e3, "steps": n_sus, "seconds": ms_sus / 1e3, "wall": wall_sus}
    fastocr_step = eager_step                     # the profiling and end-to-end passes launch directly
    dense_steps = max(3, min(args.steps, 20))
    for t in range(3):
        dense_step(t)
    ms_dense = timed(dense_step, dense_steps, barrier) / dense_steps
    clocks.stop()
    clock_info = clocks.window(wall[0], wall[1])
    if sustained is not None:
        sustained["clocks"] = clocks.window(*sustained.pop("wall"))
        if clock_info.get("sm_mhz") is None:      # the timed region fell between two samples: the longer region's record stands in
            clock_info = dict(sustained["clocks"], note="samples of the sustained region (the timed region was shorter than the sampling period)")

    # per-kernel average durations over the same steps, from CUDA events the library records on the
    # launching stream: "in_situ" times each maximal run of same-kernel launches as one interval (the
    # launches overlap exactly as in the timed region), "isolated" brackets every launch on its own
    prof_steps = min(args.steps, 50)
    profs = {}
    for mode, coalesce in (("in_situ", True), ("isolated", False)):
        w.ctx.profile_begin(prof_steps * (w.L * 2 + 8), coalesce_runs=coalesce)
        for t in range(prof_steps):
            fastocr_step(t)
        profs[mode] = w.ctx.profile_end()
    prof = profs["in_situ"]

    if dist:
        tt = torch.tensor([ms, ms_dense], device=dev, dtype=torch.float64)
        dist.all_reduce(tt, op=dist.ReduceOp.MAX)
        ms, ms_dense = float(tt[0]), float(tt[1])
    us_step = ms / args.steps * 1e3

    n_focal = len(focal)
    mean_s = (w.nd - 1) / 2.0
    sparse_b = w.sparse_bytes(mean_s)
    dense_b = w.dense_bytes(mean_s)
    step_bytes = n_focal * dense_b + (w.L - n_focal) * sparse_b
    kern = {}
    for name, bytes_per in (("attn_sparse", sparse_b), ("attn_dense", dense_b)):
        tot, n = prof[name]
        if n:
            us = tot / n * 1e3
            iso_tot, iso_n = profs["isolated"][name]
            kern[name] = {"us_per_launch": us, "us_per_launch_isolated": iso_tot / max(iso_n, 1) * 1e3,
                          "launches_per_step": n / prof_steps, "algorithmic_bytes": bytes_per,
                          "gbs": bytes_per / us / 1e3, "frac_of_measured": bytes_per / us / 1e3 / peak,
                          "frac_of_8tbs": bytes_per / us / 1e3 / NOMINAL_HBM_GBS}
    for name in ("scores_finalize", "select_topk"):
        tot, n = prof[name]
        if n:
            kern[name] = {"us_per_launch": tot / n * 1e3, "launches_per_step": n / prof_steps}
    total_prof = sum(v[0] for v in prof.values()) or 1.0
    for name in kern:
        kern[name]["share_of_step"] = prof[name][0] / total_prof
    share = {name: prof[name][0] for name in prof if prof[name][1]}
    dominant = max(("attn_sparse", "attn_dense"), key=lambda n: share.get(n, 0.0))
    traffic = None
    tpath = os.path.join(ROOT, "profiles", "ncu_traffic.json")
    if os.path.exists(tpath):
        traffic = json.load(open(tpath)).get(dominant, {}).get("traffic_bytes_per_launch")
    roofline = {"bound": "hbm", "kernel": dominant, "achieved": kern[dominant]["gbs"], "peak": peak, "unit": "GB/s",
                "frac": kern[dominant]["frac_of_measured"], "peak_kind": f"of {peak_kind}", "traffic": traffic,
                "frac_of_8tbs": kern[dominant]["frac_of_8tbs"],
                "timing": "CUDA events on the launching stream around each run of consecutive launches of this kernel, / launches"}

    # ---- end to end: per step, pinned-host queries + the new token's K/V rows in, outputs back ----
    e2e = None
    if not args.no_e2e:
        q_host = w.q_all.cpu().pin_memory()                                         # [nd][L][B][H][d]
        rows = [w.flat_row(s) for s in range(w.nd)]                                 # step s appends position S0+s
        flatK = w.K_all.view(w.L, -1, w.Hkv, cfg.head_dim)                          # [L][rows][Hkv][d]
        flatV = w.V_all.view(w.L, -1, w.Hkv, cfg.head_dim)
        newkv_host = torch.stack([torch.stack([flatK[:, rows[s]], flatV[:, rows[s]]], dim=1)
                                  for s in range(w.nd)]).cpu().pin_memory()         # [nd][L][2][B][Hkv][d]
        out_host = torch.empty(out.shape, dtype=out.dtype).pin_memory()
        q_dev = torch.empty_like(w.q_all[0])
        newkv_dev = torch.empty(newkv_host.shape[1:], dtype=newkv_host.dtype, device=dev)

        # The step runs as a few slices of consecutive layers (one library call each), so that the
        # copies overlap the arithmetic: slice i's inputs arrive while slice i - 1 computes, its
        # outputs leave while slice i + 1 computes. Steps themselves stay serial (autoregressive).
        n_sl = args.e2e_slices if (w.L >= 8 and w.B * w.Hkv >= 64) else 1   # small batches are bound by the host's calls: one slice
        cuts = [round(i * w.L / n_sl) for i in range(n_sl + 1)]
        slices = list(zip(cuts[:-1], cuts[1:]))
        plans = [fo.StepPlan(w.ctx, w.views[a:b], is_focal[a:b], w.k_d, w.fix, max(w.vis_len), w.max_kept) for a, b in slices]
        s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
        ev_in = [torch.cuda.Event() for _ in slices]
        ev_out = [torch.cuda.Event() for _ in slices]

        def e2e_step(t):
            s = t % w.nd
            cur = torch.cuda.current_stream()
            w.set_step(t)
            if n_sl == 1:                               # everything in stream order
                q_dev.copy_(q_host[s], non_blocking=True)
                newkv_dev.copy_(newkv_host[s], non_blocking=True)
                flatK.index_copy_(1, rows[s], newkv_dev[:, 0])
                flatV.index_copy_(1, rows[s], newkv_dev[:, 1])
                state["have"] = plans[0].run(q_dev, out, state["have"])
                out_host.copy_(out, non_blocking=True)
                return
            s_in.wait_stream(cur)                       # the previous step has consumed the staging buffers
            with torch.cuda.stream(s_in):
                for i, (a, b) in enumerate(slices):
                    q_dev[a:b].copy_(q_host[s, a:b], non_blocking=True)
                    newkv_dev[a:b].copy_(newkv_host[s, a:b], non_blocking=True)
                    ev_in[i].record(s_in)
            for i, (a, b) in enumerate(slices):
                cur.wait_event(ev_in[i])
                flatK[a:b].index_copy_(1, rows[s], newkv_dev[a:b, 0])      # append the current token's K/V rows to the
                flatV[a:b].index_copy_(1, rows[s], newkv_dev[a:b, 1])      # caches of the slice's layers
                state["have"] = plans[i].run(q_dev[a:b], out[a:b], state["have"])
                ev_out[i].record(cur)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(ev_out[i])
                    out_host[a:b].copy_(out[a:b], non_blocking=True)
            cur.wait_stream(s_out)                      # the step ends when its last output is on the host

        for t in range(3):
            e2e_step(t)
        e2e_steps = min(args.steps, 50)
        ms_e2e = timed(e2e_step, e2e_steps, barrier) / e2e_steps
        torch.cuda.synchronize()
        if not torch.equal(out_host, out.cpu()):        # every slice's copy-out was ordered after its arithmetic
            raise RuntimeError("end-to-end step: the host copy of the outputs differs from the device's")
        if dist:
            tt = torch.tensor([ms_e2e], device=dev, dtype=torch.float64)
            dist.all_reduce(tt, op=dist.ReduceOp.MAX)
            ms_e2e = float(tt[0])
        e2e = {"value": ms_e2e * 1e3, "unit": "us/step",
               "h2d_bytes_per_step": int(q_host[0].numel() * 2 + newkv_host[0].numel() * 2),
               "d2h_bytes_per_step": int(out_host.numel() * out_host.element_size()),
               "note": "per step: pinned-host queries and the new token's K/V rows in (appended to every layer's cache), "
                       "all layer outputs back to pinned host memory; the KV cache itself is resident by definition; "
                       + f"the step is issued as {n_sl} slice(s) of layers so that the copies overlap the arithmetic"}

    cpu_base, parity = None, None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        # The oracle's Algorithm-1 step on a sample of the sequences: timed as the CPU baseline, and its
        # traces checked against what the timed configuration (same plan, same chained launches, bf16
        # outputs) produces for the same track steps.
        import oracle
        focal_of = (lambda b: focal_sets[b]) if focal_sets is not None else (lambda b: focal)
        w.set_step(0)
        plan.run(w.q_all[0], out, False)                          # step 0: no carried set yet (fallback at layer 0)
        carried_gpu = w.fix.cpu().clone()
        w.set_step(1)
        plan.run(w.q_all[1], out, True)                           # step 1 starts from step 0's set
        torch.cuda.synchronize()
        out_gpu, fix_gpu = out.float().cpu(), w.fix.cpu()
        state["have"] = True

        def oracle_sample(seq_ids):
            total, traces = 0.0, {}
            for b in seq_ids:
                layers = []
                for l in range(w.L):
                    K, V = w.logical_rows(l, b, w.S0[b] + 2)
                    layers.append((w.q_all[1, l, b].cpu(), K, V))
                t0 = time.perf_counter()
                traces[b] = oracle.decode_step(layers, focal_of(b), carried_gpu[b, :w.k[b]], w.vis_start[b], w.vis_len[b], cfg.tau,
                                               w.sm_scale, union_sets=args.union_sets)
                total += time.perf_counter() - t0
            return total, traces

        dt1, _ = oracle_sample([0])
        n_s = int(max(1, min(w.B, args.cpu_seconds / max(dt1, 1e-3))))
        dt, traces = oracle_sample(list(range(n_s)))
        cpu_base = {"value": dt / n_s * w.B * 1e6, "unit": "us/step", "cores": oracle.num_threads(), "kind": "oracle",
                    "sample": f"{n_s} of {w.B} sequences, all {w.L} layers, one step ({dt:.2f} s of oracle time), scaled to the batch"}
        exact = near = 0
        max_abs, sum_abs, n_el = 0.0, 0.0, 0
        for b, tr in traces.items():
            # the set carried out of step 0 against the oracle's own selection at that step's deepest focal layer
            fb = focal_of(b)
            deepest = max(fb) if fb else 0
            Kp, _ = w.logical_rows(deepest, b, w.S0[b] + 1)
            sc0, _ = oracle.scores(w.q_all[0, deepest, b].cpu(), Kp, w.sm_scale, w.vis_start[b], w.vis_len[b])
            pairs = [(carried_gpu[b, :w.k[b]].tolist(), oracle.topk(sc0, w.k[b]).tolist(), sc0)]
            if tr.f_last is not None and fb:                      # and the set carried out of step 1
                K1, _ = w.logical_rows(deepest, b, w.S0[b] + 2)
                sc1, _ = oracle.scores(w.q_all[1, deepest, b].cpu(), K1, w.sm_scale, w.vis_start[b], w.vis_len[b])
                pairs.append((fix_gpu[b, :w.k[b]].tolist(), tr.f_last.tolist(), sc1))
            same = all(g == r for g, r, _ in pairs)
            tie = True
            for g, r, sc in pairs:
                if g != r and w.k[b] > 0:
                    kth = float(torch.sort(sc, descending=True).values[w.k[b] - 1])
                    tie = tie and all(abs(float(sc[i]) - kth) <= 1e-5 * abs(kth) for i in set(g) ^ set(r))
            exact += same
            near += (not same) and tie
            for l in range(w.L):
                err = (out_gpu[l, b] - tr.outputs[l]).abs()
                max_abs = max(max_abs, float(err.max()))
                sum_abs += float(err.sum())
                n_el += err.numel()
        parity = {"sequences": len(traces), "layers": w.L, "steps_compared": "track steps 0 (carried set) and 1 (outputs, carried set)",
                  "selection_exact": exact, "near_tie_only": near, "selection_mismatch": len(traces) - exact - near,
                  "max_abs": max_abs, "mean_abs": sum_abs / max(n_el, 1), "tolerance": {"max_abs": 1e-2, "mean_abs": 1e-3},
                  "out_dtype": "bf16", "oracle": "fp32"}
        parity["ok"] = bool(parity["selection_mismatch"] == 0 and max_abs <= 1e-2 and parity["mean_abs"] <= 1e-3)

    hidden = w.H * cfg.head_dim
    mean_S = float(np.mean(w.S0)) + (w.nd + 1) / 2.0
    mean_kept = float(np.mean([n_union * k + t for k, t in zip(w.k, w.text0)])) + (w.nd + 1) / 2.0
    flops = {"vanilla": fo.attn_flops(w.B, w.L, hidden, mean_S) / 1e9,
             "fastocr": fo.attn_flops_pruned(w.B, w.L, hidden, mean_S, len(focal) if focal_sets is None else
                                             float(np.mean([len(c) for c in focal_sets])), mean_kept) / 1e9,
             "formula": "Appendix B, b*l*(8h^2 + 4hs) with h = heads x 128; pruned layers attend kept image tokens + text"}

    if rank == 0:
        line = {
            "metric": "fastocr decode-attention step time", "value": us_step, "unit": "us/step", "n_gpus": world,
            "steps": args.steps, "warmup": max(3, args.warmup), "ms_per_step": us_step / 1e3, "higher_is_better": False,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": cfg.name, "layers": w.L, "focal_layers": focal, "arithmetic": "bf16 K/V/Q and outputs, fp32 accumulation",
                       "focal_sets": "per sequence" if focal_sets is not None else "one for the batch", "union_sets": bool(args.union_sets), "batch_per_gpu": w.B, "global_batch": w.B * world,
                       "num_q_heads": w.H, "num_kv_heads": w.Hkv, "head_dim": cfg.head_dim, "vis_tokens": [min(w.vis_len), max(w.vis_len)],
                       "text_tokens": [min(w.text0), max(w.text0)], "tau": cfg.tau, "rho": cfg.rho, "gap": cfg.gap, "kept": [min(w.k), max(w.k)],
                       "kv_dtype": "bf16", "paged": bool(cfg.page_size), "cuda_graph": bool(use_graph), "cache_bytes": int(sum(k.numel() * 4 for k in w.K)),
                       "l2": "inputs larger than L2: every layer has its own cache and the step cycles through all of them",
                       "parallelism": f"dp{world} (sequences sharded, no collective)"},
            "dense_us_per_step": ms_dense * 1e3, "speedup_vs_dense": ms_dense * 1e3 / us_step,
            "step_algorithmic_bytes": step_bytes, "step_gbs": step_bytes / us_step / 1e3,
            "step_frac_of_8tbs": step_bytes / us_step / 1e3 / NOMINAL_HBM_GBS, "step_frac_of_measured": step_bytes / us_step / 1e3 / peak,
            "dense_step_gbs": w.L * dense_b / (ms_dense * 1e3) / 1e3,
            "flops_G": flops, "step_mb": step_bytes / 1e6,
            "kernels": kern, "roofline": roofline, "cpu_baseline": cpu_base, "parity": parity, "e2e": e2e, "gpu_launches": int(launches),
            "sustained": sustained, "clocks": clock_info,
        }
        print(json.dumps(line))
        if parity is not None and not parity["ok"]:
            raise SystemExit("bench: the timed configuration's outputs or selections are outside the stated tolerance")
    if dist:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
