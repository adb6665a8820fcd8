#!/usr/bin/env python
"""Benchmark of the LIME ranking-inference hot path on B200.

One "step" = one batch through the online path: ragged offsets -> history gather -> n XOR layers (link states)
-> candidate scoring.  The offline candidate->link precompute is timed separately (the paper caches it).
Prints ONE JSON line (rank 0).  `--impl reference` times the fp64 CPU oracle on a bounded sample instead.

    python bench.py --gpus 1 --steps 20 --warmup 5
    python -m torch.distributed.run --nnodes=1 --nproc-per-node N ... bench.py --gpus N --steps K --warmup W
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

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2510_18239_b200 import synth  # noqa: E402

METRIC = "candidate_scores_per_sec"
UNIT = "candidates/s"
ROTATE = 4                      # input sets rotated between steps so that no step is served from L2
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
FP32_ALU_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12      # 148 SMs x 128 FP32 lanes x FMA x max SM clock


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return {k: float(d[k]) for k in FALLBACK_PEAKS if k in d} | {"source": "measured"}
    return dict(FALLBACK_PEAKS, source="fallback")


# ----------------------------------------------------------------------------- algorithmic work per kernel and step
def kernel_models(wl: synth.Workload, total_tokens: int, cand_heads: int = 1):
    """name -> dict(bytes=, flops=) : algorithmic work of ALL launches of that kernel in one step.  Bytes are what
    the stage must move through HBM (inputs read once, outputs written once, scratch excluded); flops what it must
    compute (2 per multiply-add).  A kernel with both is bounded by whichever floor (bytes / HBM peak, flops /
    tensor peak) is longer."""
    es = 4 if wl.dtype == synth.F32 else 2
    d, ell, H, n, f = wl.d, wl.ell, wl.H, wl.n_layers, wl.dff
    BC, BL, N, HL = wl.B * wl.C, wl.B * wl.ell, total_tokens, wl.H * wl.ell
    hist_proj = sum((3 if j < n - 1 else 2) for j in range(n)) * 2.0 * N * d * d
    link_proj = (ell + (n - 1) * BL) * 3 * 2.0 * d * d
    glu = 4.0 * d * f * (BL * n + N * (n - 1))
    down = 2.0 * d * f * (BL * n + N * (n - 1))
    return {
        # cand_heads = H: one weight row per (candidate, head), i.e. H * ell weights per candidate
        "k_score": dict(bytes=BC * (es * ell * cand_heads + es * d + 4.0)),
        # by id from the corpus caches: the same rows, fetched one by one, + the 4-byte id
        "k_score_gather_tc": dict(bytes=BC * (es * ell * cand_heads + es * d + 8.0)),
        "k_gather": dict(bytes=N * (4.0 + 2 * es * d)),
        "k_precompute": dict(bytes=BC * es * (d + ell * cand_heads)),
        # fused tensor-core layer kernels: history rows read once per direction, written once by the update
        "k_link_attn_tc": dict(bytes=n * N * d * es, flops=n * 4.0 * HL * d * N, pipe="tensor"),
        "k_hist_update_tc": dict(bytes=(n - 1) * 2.0 * N * d * es, flops=(n - 1) * 2.0 * N * (HL * d + 2 * HL * f + f * d),
                                 pipe="tensor"),
        "k_hist_update2_tc": dict(bytes=(n - 1) * 2.0 * N * d * es, flops=(n - 1) * 2.0 * N * (HL * d + 2 * HL * f + f * d),
                                  pipe="tensor"),
        # d = 256 kernels: folded scores against the stored rows, values mixed head by head, GatedMLP weights as they stand
        "k_link_attn_d256_tc": dict(bytes=n * N * d * es, flops=n * 4.0 * HL * d * N, pipe="tensor"),
        "k_hist_update_d256_tc": dict(bytes=(n - 1) * 2.0 * N * d * es,
                                      flops=(n - 1) * 2.0 * N * (HL * d + ell * d + 2 * d * f + f * d), pipe="tensor"),
        # link-side GEMMs (rows = users x links): PREP (layers 2..n: folded queries / keys and values or gate / up operands)
        # and the GatedMLP on the attention rows with W_V folded in
        "k_gemm_tc_prep": dict(flops=2.0 * BL * d * (max(n - 2, 0) * (2 * H * d + (d if d == 256 else 2 * H * f)) + (H * d if n > 1 else 0)),
                               pipe="tensor"),
        "k_link_mlp_tc": dict(flops=n * 2.0 * BL * (H * d * 2 * f + f * d), pipe="tensor"),
        # CUDA-core path (fp32 storage and shapes the tensor-core kernels do not serve)
        "k_linear_simt_ln": dict(flops=hist_proj + link_proj, pipe="alu"),
        "k_linear_simt_glu": dict(flops=glu, pipe="alu"),
        "k_linear_simt": dict(flops=down, pipe="alu"),
        "k_attn_link": dict(flops=4.0 * ell * d * N * n, pipe="alu"),
        "k_attn_hist": dict(flops=4.0 * ell * d * N * (n - 1), pipe="alu"),
    }


NOMINAL_HBM_GBS = 8000.0        # B200 HBM3e, vendor figure (7.7 TB/s on HGX boards); context beside the measured copy peak
NOMINAL_BF16_TFLOPS = 2250.0    # dense bf16, vendor figure


def roofline_entry(mdl, ms, pk):
    """Achieved rate of `ms` milliseconds of kernel time against the roofline that bounds it."""
    t = ms * 1e-3
    floors = {}
    if "bytes" in mdl:
        floors["hbm"] = mdl["bytes"] / (pk["hbm_gbs"] * 1e9)
    if "flops" in mdl:
        peak = FP32_ALU_TFLOPS if mdl.get("pipe") == "alu" else pk["bf16_tflops_sustained"]
        floors["alu" if mdl.get("pipe") == "alu" else "tensor"] = mdl["flops"] / (peak * 1e12)
    bound = max(floors, key=floors.get)
    if bound == "hbm":
        ach = mdl["bytes"] / t / 1e9
        return dict(bound="hbm", achieved=ach, peak=pk["hbm_gbs"], unit="GB/s", frac=ach / pk["hbm_gbs"],
                    frac_of_nominal=ach / NOMINAL_HBM_GBS)
    peak = FP32_ALU_TFLOPS if bound == "alu" else pk["bf16_tflops_sustained"]
    ach = mdl["flops"] / t / 1e12
    r = dict(bound=bound, achieved=ach, peak=peak, unit="TFLOP/s", frac=ach / peak)
    if bound == "tensor":
        r["frac_of_nominal"] = ach / NOMINAL_BF16_TFLOPS
    return r


def model_for(name, models):
    best = None
    for k in models:
        if name.startswith(k) and (best is None or len(k) > len(best)):
            best = k
    return models.get(best) if best else None


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    """nvidia-smi sampled every 50 ms; start() early (it takes a second to come up), then mark() the timed region (or ask
    for any window(t0, t1) of wall-clock time while it runs)."""

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []
        self.t0 = self.t1 = None

    def mark(self, begin: bool):
        if begin:
            self.t0 = time.time()
        else:
            self.t1 = time.time()

    def window(self, t0: float, t1: float):
        """Clock record of the samples taken between two wall-clock instants."""
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"], "samples": 0}
        return self._stats([ln for (ts, ln) in list(self.lines) if t0 - 0.02 <= ts <= t1 + 0.06])

    def start(self):
        q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={q}", "--format=csv,noheader,nounits",
                                          "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for ln in self.proc.stdout:
            self.lines.append((time.time(), ln.strip()))

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        inside = [ln for (ts, ln) in self.lines if self.t0 is None or (self.t0 - 0.05 <= ts <= (self.t1 or ts) + 0.1)]
        if not inside:
            inside = [ln for (_, ln) in self.lines[-3:]]
        return self._stats(inside)

    @staticmethod
    def _stats(inside):
        sm, mx, reasons = [], [], set()
        for ln in inside:
            p = [x.strip() for x in ln.split(",")]
            if len(p) < 7:
                continue
            try:
                sm.append(float(p[0])); mx.append(float(p[1]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), p[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ----------------------------------------------------------------------------- CPU oracle legs
HEAD_SEED = 11


def head_layers(wl, n1):
    """The interaction network used with --head: one hidden layer of n1 units (App. C lists [96] for the industrial model)."""
    return synth.ffn_weights(HEAD_SEED, "head", (2 * wl.d, n1, 1), wl.dtype)


def oracle_sample(wl, inp, users, budget_s=None, phi="softmax", cand_heads=False, head=0):
    """Time the fp64 oracle (as it stands) on `users` of the batch: gather + encode + precompute + score."""
    from oracle import lime_oracle as O
    from tests import lime_helpers as Hh
    cfg, layers = Hh.oracle_config(wl, phi=O.SILU if phi == "silu" else O.SOFTMAX), Hh.oracle_layers(inp, wl)
    links64 = synth.storage_to_f64(inp["links"], wl.dtype)
    off = O.lengths_to_offsets(inp["lengths"])

    tab = Hh.LazyTable64(inp["table"], wl.dtype)   # widens only the rows the sample touches (the table is GBs)
    head64 = [(synth.storage_to_f64(W, wl.dtype), b.astype(np.float64)) for W, b in head_layers(wl, head)] if head else None
    done, t0 = 0, time.perf_counter()
    for b in users:
        Hh.oracle_user(inp, wl, b, off, tab, links64, layers, cfg, cand_heads=cand_heads, head=head64)
        done += 1
        if budget_s is not None and time.perf_counter() - t0 > budget_s:
            break
    return done, time.perf_counter() - t0


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        return max([i.get("num_threads", 1) for i in threadpool_info()] or [1])
    except Exception:
        return os.cpu_count() or 1


def run_reference(args, wl):
    """--impl reference: the oracle, timed on host cores; each step is a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    inp = synth.make_inputs(wl, seed=0)
    _, t_user = oracle_sample(wl, inp, range(1), phi=args.phi, cand_heads=args.cand_heads, head=args.head)          # calibrates the per-step sample; also the first warm-up
    users_per_step = 2 if (wl.B >= 2 and 2 * t_user * args.steps < 120.0) else 1
    for _ in range(max(0, args.warmup - 1)):
        oracle_sample(wl, inp, range(1), phi=args.phi, cand_heads=args.cand_heads, head=args.head)
    times = []
    for s in range(args.steps):
        users = [(s * users_per_step + u) % wl.B for u in range(users_per_step)]
        _, dt = oracle_sample(wl, inp, users, phi=args.phi, cand_heads=args.cand_heads, head=args.head)
        times.append(dt)
    total = sum(times)
    value = users_per_step * wl.C * args.steps / total
    sample = f"{users_per_step} users x {wl.C} candidates per step (gather+encode+precompute+score), fp64 numpy"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": workload_config(wl),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}, "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def workload_config(wl):
    return {"workload": wl.name, "B": wl.B, "N": wl.n_max if not wl.ragged else [wl.n_min, wl.n_max], "d": wl.d, "H": wl.H,
            "ell": wl.ell, "n_layers": wl.n_layers, "C": wl.C, "V": wl.V, "zipf_s": wl.zipf_s,
            "l2": f"{ROTATE} rotating input sets per step slot (candidate streams total > 126 MB L2)"}


def launch_mode(args):
    return "host launches" if args.no_graph else f"one CUDA graph per input set ({ROTATE}), replayed"


# ----------------------------------------------------------------------------- the CUDA arm
# DRAM traffic per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the kernels captured with ncu, keyed by
# kernel and workload, with the hash of the kernel's source at capture time: once the source changes the figure
# is stale and the bench reports null.
NCU_TRAFFIC = {
    # dense scorer: 169.9 MB read + 4.0-4.5 MB written per launch
    ("k_score_tc", "bf16_baseline", 256, 2048): {"bytes": 174.2e6, "source": "k_score_tc.cu", "sha": "823248ada31d3d04"},
    # XOR-layer kernels: 33.7 MB (layer 1) and 42.2 MB (layer 2) read + written; average per launch
    ("k_link_attn_tc", "bf16_baseline", 256, 2048): {"bytes": 37.9e6, "source": "k_link_attn_tc.cu", "sha": "81680b45282491ef"},
    ("k_hist_update_tc", "bf16_baseline", 256, 2048): {"bytes": 34.6e6, "source": "k_hist_update_tc.cu", "sha": "a47ccfb7ddd4247f"},
    # scorer by id over packed corpus records: 174.5 MB read + 4.1 MB written per launch
    ("k_score_gather_tc", "bf16_baseline", 256, 2048): {"bytes": 178.6e6, "source": "k_score_gather_tc.cu", "sha": "580e539a2d79f57c"},
    # scorer through the interaction network (--head 96): 169.4 MB read + 4.4 MB written per launch
    ("k_score_head_tc", "bf16_baseline", 256, 2048): {"bytes": 173.8e6, "source": "k_score_head_tc.cu", "sha": "614556b96c1342b2"},
    # d = 256 kernels: captured on 128 users of the same model and length mix (327,693 tokens) and scaled by the tokens of
    # a launch (persistent kernels, identical tiles: traffic grows in proportion): bytes per token, average of the layers
    ("k_link_attn_d256_tc", "production_ragged", 1024, 8192): {"bytes_per_token": 560.0, "source": "k_link_attn_t64_tc.cu", "sha": "b26d676843314aed"},
    ("k_hist_update_d256_tc", "production_ragged", 1024, 8192): {"bytes_per_token": 893.0, "source": "k_hist_update_d256_tc.cu", "sha": "b84060b13975253c"},
}


def source_hash(rel):
    import hashlib
    with open(os.path.join(ROOT, "paper_2510_18239_b200", "csrc", rel), "rb") as f:
        return hashlib.sha256(f.read()).hexdigest()[:16]


def ncu_traffic(kernel, wl, args=None, tokens=None):
    rec = NCU_TRAFFIC.get((kernel, wl.name, wl.B, wl.C))
    if not rec or (args is not None and (args.cand_heads or args.phi != "softmax")):
        return None          # the captures were taken in the default mode
    try:
        if source_hash(rec["source"]) != rec["sha"]:
            return None
    except OSError:
        return None
    if "bytes_per_token" in rec:
        return rec["bytes_per_token"] * tokens if tokens else None
    return rec["bytes"]


def run_ours(args, wl, sampler=None, with_sweeps=False):
    import torch
    import torch.distributed as dist
    from paper_2510_18239_b200 import binding as Bd, shard

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.device("cuda", local)

    # inputs: one model (table, links, weights) per rank; ROTATE request sets; users are sharded across ranks with
    # a fixed per-GPU batch (weak scaling, no collective on the data path)
    inp = synth.make_inputs(wl, seed=rank)
    dt = Bd.LIME_F32 if wl.dtype == synth.F32 else Bd.LIME_BF16
    lime = Bd.Lime(wl.d, wl.H, wl.ell, wl.n_layers, dtype=dt, d_ff=wl.d_ff,
                   phi=Bd.LIME_PHI_SILU if args.phi == "silu" else Bd.LIME_PHI_SOFTMAX,
                   cand_heads=wl.H if args.cand_heads else 0)
    table = Bd.to_device(inp["table"], wl.dtype, dev)
    links = Bd.to_device(inp["links"], wl.dtype, dev)
    wts = {k: Bd.to_device(inp[k], wl.dtype, dev) for k in ("Wq", "Wk", "Wv", "Wg", "Wu", "Wo")}
    lime.set_weights(links, [{k: wts[k][j] for k in wts} for j in range(wl.n_layers)])
    head_dev = None
    if args.head:
        head_dev = [(Bd.to_device(W, wl.dtype, dev), torch.from_numpy(b).to(dev)) for W, b in head_layers(wl, args.head)]
        lime.set_head(head_dev)
        head_ws = torch.empty(Bd.lime_head_workspace_bytes(lime.ctx, wl.B), dtype=torch.uint8, device=dev)

    def score(ls_, W_, T_, ids_, out_, corpus=None):
        # the per-candidate stage: the dot product <O_c, T_c>, or (--head) the interaction network on [O_c | T_c]
        if args.head:
            Bd.lime_score_candidates_head(lime.ctx, ls_, wl.B, W_, T_, None, wl.C, wl.B * wl.C, ids_, out_, head_ws, corpus)
        else:
            Bd.lime_score_candidates(lime.ctx, ls_, wl.B, W_, T_, None, wl.C, wl.B * wl.C, ids_, out_, corpus)

    sets, host_sets = [], []
    pre_ms = []
    for r in range(ROTATE):
        lengths = synth.history_lengths(rank * 100 + r, wl.B, wl.n_min, wl.n_max)
        total = int(lengths.sum())
        hist_ids = synth.zipf_ids(rank * 100 + r, "hist_ids", total, wl.V, wl.zipf_s) if wl.zipf_s else inp["hist_ids"]
        cand_ids = synth.uniform_ids(rank * 100 + r, "cand_ids", wl.B * wl.C, wl.V) if wl.zipf_s else inp["cand_ids"]
        s = dict(lengths=torch.from_numpy(lengths).to(dev), hist_ids=torch.from_numpy(hist_ids).to(dev),
                 cand_ids=torch.from_numpy(cand_ids).to(dev), total=total)
        s["T"] = lime.gather_history(table, s["cand_ids"])
        s["W"] = lime.precompute_candidate_links(s["T"])
        sets.append(s)
        host_sets.append(dict(lengths=torch.from_numpy(lengths).pin_memory(), hist_ids=torch.from_numpy(hist_ids).pin_memory(),
                              cand_ids=torch.from_numpy(cand_ids).pin_memory(), total=total))
    # offline stage, timed on its own: one launch per input set, back to back, sets rotated (inputs > L2 in all)
    wscratch = torch.empty_like(sets[0]["W"])
    for s in sets:
        Bd.lime_precompute_candidate_links(lime.ctx, s["T"], wscratch)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    pre_reps = 5 * ROTATE
    e0.record()
    for i in range(pre_reps):
        Bd.lime_precompute_candidate_links(lime.ctx, sets[i % ROTATE]["T"], wscratch)
    e1.record()
    torch.cuda.synchronize()
    pre_ms = e0.elapsed_time(e1) / pre_reps
    max_total = max(s["total"] for s in sets)
    off = torch.empty(wl.B + 1, dtype=torch.int32, device=dev)
    hist = torch.empty((max_total, wl.d), dtype=lime.tdtype, device=dev)
    ls = torch.empty((wl.B, lime.ell_c, wl.d), dtype=lime.tdtype, device=dev)
    logits = torch.empty(wl.B * wl.C, dtype=torch.float32, device=dev)
    ws = lime.workspace(wl.B, max_total)
    ctx = lime.ctx

    def step(i):
        s = sets[i % ROTATE]
        h = hist[: s["total"]]
        Bd.lime_lengths_to_offsets(ctx, s["lengths"], off)
        # the lookup applies the first layer's LayerNorm on the way (every layer reads the history through it only)
        Bd.lime_gather_history_normalized(ctx, table, s["hist_ids"], h)
        Bd.lime_encode_user_normalized(ctx, h, off, wl.B, None, ls, ws)
        score(ls, s["W"], s["T"], None, logits)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    own_sampler = sampler is None
    if own_sampler:
        sampler = ClockSampler(local)
        if rank == 0:
            sampler.start()
    for i in range(max(args.warmup, ROTATE)):
        step(i)
    barrier()

    # One CUDA graph per rotating input set: the step's launches are recorded once and replayed, so the timed region
    # holds the library's kernels back to back instead of the host's launch calls.
    def capture(fn):
        graphs = []
        for r in range(ROTATE):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                fn(r)
            graphs.append(g)
        return graphs

    direct_step = step
    if not args.no_graph:
        step_graphs = capture(direct_step)

        def step(i):                                   # noqa: F811
            step_graphs[i % ROTATE].replay()

        for i in range(ROTATE):
            step(i)
        barrier()

    # ---- timed region: exactly `steps` steps, device-timed, nothing but the library's launches in between
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    barrier()
    t_wall0 = time.time()
    ev[0].record()
    for i in range(args.steps):
        step(i)
        ev[i + 1].record()
    torch.cuda.synchronize()
    t_wall1 = time.time()
    barrier()
    clocks = sampler.window(t_wall0, t_wall1) if rank == 0 else None
    total_ms = ev[0].elapsed_time(ev[-1])
    step_ms = sorted(ev[i].elapsed_time(ev[i + 1]) for i in range(args.steps))
    # every rank serves its own batch of B users (users are independent: no collective on the data path); the job's
    # throughput is all ranks' candidates over the slowest rank's device time
    total_ms = shard.max_over_ranks(total_ms, dev)
    value = shard.sum_over_ranks(wl.B * wl.C * args.steps, dev) / (total_ms * 1e-3)

    # ---- the same steps again with every launch of the library bracketed by CUDA events on its stream: per-kernel
    #      launch durations and the launch count of one step (the brackets add gaps, so this pass is not `value`)
    prof_steps = min(args.steps, 100)
    cap = 64 * prof_steps + 64
    Bd.lime_profile_start(cap)
    for i in range(prof_steps):
        direct_step(i)
    torch.cuda.synchronize()
    records, launches = Bd.lime_profile_stop(cap)
    launches_per_step = launches / prof_steps

    # ---- the scoring kernel alone, back to back over the rotating input sets (burst figure: no event brackets
    #      or neighbouring kernels inside the interval)
    score_reps = max(20, min(200, args.steps))
    for i in range(ROTATE):
        s = sets[i]
        score(ls, s["W"], s["T"], None, logits)
    torch.cuda.synchronize()
    e0.record()
    for i in range(score_reps):
        s = sets[i % ROTATE]
        score(ls, s["W"], s["T"], None, logits)
    e1.record()
    torch.cuda.synchronize()
    score_alone_ms = e0.elapsed_time(e1) / score_reps

    # ---- end to end through the C ABI from host buffers: request = (lengths, history ids, candidate ids) in pinned
    #      host memory; the corpus-level caches (table, phi(T L^t) for every item) are resident, as in the paper's
    #      serving flow; logits come back to pinned host memory
    #      Three streams pipeline consecutive requests - copies in | kernels | logits out - over two request slots, as
    #      a server would; every step's copies are inside the timed region.
    w_corpus = lime.precompute_candidate_links(table)
    # one record per item: [embedding row | cached weight row], so that scoring by id touches one place per candidate
    packed = lime.pack_corpus_cache(table, w_corpus)
    # a context whose row width is ell_c: the row lookup applied to the cached weights
    lime_w = Bd.Lime(lime.ell_c, (lime.ell_c + 127) // 128, 1, 1, dtype=dt)
    Tg = Wg = None
    if args.head:
        Tg = torch.empty((wl.B * wl.C, wl.d), dtype=lime.tdtype, device=dev)
        Wg = torch.empty((wl.B * wl.C, lime.ell_c), dtype=lime.tdtype, device=dev)
    SLOTS = 2
    d_len = [torch.empty(wl.B, dtype=torch.int32, device=dev) for _ in range(SLOTS)]
    d_hid = [torch.empty(max_total, dtype=torch.int32, device=dev) for _ in range(SLOTS)]
    d_cid = [torch.empty(wl.B * wl.C, dtype=torch.int32, device=dev) for _ in range(SLOTS)]
    d_logits = [torch.empty(wl.B * wl.C, dtype=torch.float32, device=dev) for _ in range(SLOTS)]
    h_logits = [torch.empty(wl.B * wl.C, dtype=torch.float32).pin_memory() for _ in range(SLOTS)]
    assert ROTATE % SLOTS == 0

    def e2e_copy_in(i):
        hs, k = host_sets[i % ROTATE], i % SLOTS
        n = hs["total"]
        d_len[k].copy_(hs["lengths"], non_blocking=True)
        d_hid[k][:n].copy_(hs["hist_ids"], non_blocking=True)
        d_cid[k].copy_(hs["cand_ids"], non_blocking=True)
        return 4 * (wl.B + n + wl.B * wl.C)

    def e2e_compute(i):
        k, n = i % SLOTS, host_sets[i % ROTATE]["total"]
        h = hist[:n]
        Bd.lime_lengths_to_offsets(ctx, d_len[k], off)
        Bd.lime_gather_history_normalized(ctx, table, d_hid[k][:n], h)
        Bd.lime_encode_user_normalized(ctx, h, off, wl.B, None, ls, ws)
        # candidates are scored straight from the corpus caches by id (no gather of their rows)
        if args.head:
            # the tensor-core interaction-network scorer takes dense streams: the candidates' rows are looked up first
            Bd.lime_gather_history(ctx, table, d_cid[k], Tg)
            Bd.lime_gather_history(lime_w.ctx, w_corpus, d_cid[k], Wg)
            score(ls, Wg, Tg, None, d_logits[k])
        else:
            Bd.lime_score_candidates_packed(ctx, ls, wl.B, packed, d_cid[k], None, wl.C, wl.B * wl.C, d_logits[k])

    def e2e_copy_out(i):
        k = i % SLOTS
        h_logits[k].copy_(d_logits[k], non_blocking=True)
        return 4 * wl.B * wl.C

    s_in, s_cmp, s_out = torch.cuda.Stream(dev), torch.cuda.Stream(dev), torch.cuda.Stream(dev)
    ev_in = [torch.cuda.Event() for _ in range(SLOTS)]
    ev_cmp = [torch.cuda.Event() for _ in range(SLOTS)]
    ev_out = [torch.cuda.Event() for _ in range(SLOTS)]
    e2e_graphs = None

    def e2e_step(i):
        k = i % SLOTS
        with torch.cuda.stream(s_in):
            s_in.wait_event(ev_cmp[k])                 # the kernels of request i - SLOTS have read this slot's ids
            a = e2e_copy_in(i)
            ev_in[k].record(s_in)
        with torch.cuda.stream(s_cmp):
            s_cmp.wait_event(ev_in[k])
            s_cmp.wait_event(ev_out[k])                # this slot's previous logits have left the device
            if e2e_graphs is None:
                e2e_compute(i)
            else:
                e2e_graphs[i % ROTATE].replay()
            ev_cmp[k].record(s_cmp)
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev_cmp[k])
            b = e2e_copy_out(i)
            ev_out[k].record(s_out)
        return a, b

    for i in range(2 * ROTATE):
        e2e_step(i)
    barrier()
    if not args.no_graph:
        graphs = []
        for r in range(ROTATE):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=s_cmp):
                e2e_compute(r)
            graphs.append(g)
        e2e_graphs = graphs
        for i in range(ROTATE):
            e2e_step(i)
        barrier()
    # the by-id scorer alone, back to back (random rows of the 256 MB+ table: no reuse between launches)
    torch.cuda.synchronize()
    eg0, eg1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    eg0.record()
    for i in range(50 if not args.head else 0):
        Bd.lime_score_candidates_packed(ctx, ls, wl.B, packed, d_cid[i % SLOTS], None, wl.C, wl.B * wl.C, d_logits[i % SLOTS])
    eg1.record()
    torch.cuda.synchronize()
    score_by_id_ms = eg0.elapsed_time(eg1) / 50
    eg0.record()
    for i in range(50 if not args.head else 0):
        score(ls, w_corpus, table, d_cid[i % SLOTS], d_logits[i % SLOTS])
    eg1.record()
    torch.cuda.synchronize()
    score_by_id_two_arrays_ms = eg0.elapsed_time(eg1) / 50
    h2d = d2h = 0
    e0.record(s_in)
    t_issue = time.perf_counter()
    for i in range(args.steps):
        a, b = e2e_step(i)
        h2d += a
        d2h += b
    e1.record(s_out)
    t_issue = time.perf_counter() - t_issue       # host time to issue the steps (the device may lag behind or wait for it)
    torch.cuda.synchronize()
    barrier()
    e2e_ms = e0.elapsed_time(e1)
    e2e_ms = shard.max_over_ranks(e2e_ms, dev)
    e2e_value = shard.sum_over_ranks(wl.B * wl.C * args.steps, dev) / (e2e_ms * 1e-3)
    extras = None
    if rank == 0 and world == 1 and not args.no_extras:
        extras = measure_extras(args, wl, lime, dict(table=table, sets=sets, hist=hist, off=off, ls=ls, ws=ws, logits=logits,
                                                     w_corpus=w_corpus, d_cid=d_cid, lime_w=lime_w), dev)
    Bd.lime_device_status(ctx)          # raises if any bounded in-kernel wait gave up during the run

    if rank == 0:
        pk = peaks()
        avg_tokens = int(sum(s["total"] for s in sets) / ROTATE)
        models = kernel_models(wl, avg_tokens, wl.H if args.cand_heads else 1)
        agg = {}
        for name, ms in records:
            a = agg.setdefault(name, [0, 0.0])
            a[0] += 1
            a[1] += ms
        ksum = sum(v[1] for v in agg.values()) or 1.0
        kernels = []
        for name, (cnt, ms) in sorted(agg.items(), key=lambda kv: -kv[1][1]):
            per_step_ms = ms / prof_steps
            entry = {"kernel": name, "launches_per_step": cnt / prof_steps, "ms_per_step": per_step_ms, "share": ms / ksum}
            mdl = model_for(name, models)
            if mdl and per_step_ms > 0:
                entry.update(roofline_entry(mdl, per_step_ms, pk))
            kernels.append(entry)

        def roof(k, ms=None, how="CUDA events around each launch inside the step"):
            mdl = model_for(k["kernel"], models)
            r = dict(kernel=k["kernel"], **roofline_entry(mdl, ms if ms is not None else k["ms_per_step"], pk))
            r["traffic"] = ncu_traffic(k["kernel"], wl, args, avg_tokens)
            r["peak_source"] = ("derived: 148 SM x 128 lanes x 2 x 1.965 GHz" if r["bound"] == "alu" else
                                f"{pk['source']} ({'copy bandwidth' if r['bound'] == 'hbm' else 'sustained bf16 GEMM'})")
            r["timing"] = how
            r["share_of_step"] = k["share"]
            return r

        dom = next((k for k in kernels if "bound" in k), None)
        roofline = roof(dom) if dom else None
        score = next((k for k in kernels if k["kernel"].startswith("k_score")), None)
        scoring = None
        if score:
            scoring = roof(score, score_alone_ms, f"{score_reps} back-to-back launches over {ROTATE} rotating input sets, CUDA events")
            scoring["ms_alone"] = score_alone_ms
            scoring["ms_in_step"] = score["ms_per_step"]
            scoring["frac_in_step"] = score.get("frac")
            if roofline and roofline["kernel"] == score["kernel"]:
                roofline = scoring

        cpu = None
        if world == 1 and not args.no_cpu_baseline:
            n_done, dt_s = oracle_sample(wl, inp, range(wl.B), budget_s=args.cpu_budget, phi=args.phi, cand_heads=args.cand_heads, head=args.head)
            cpu = {"value": n_done * wl.C / dt_s, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                   "sample": f"first {n_done} users x {wl.C} candidates of the same workload, {dt_s:.1f} s "
                             "(gather+encode+precompute+score, fp64 numpy)"}
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
                "ms_per_step": total_ms / args.steps, "p50_batch_latency_ms": step_ms[len(step_ms) // 2],
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if wl.dtype == synth.BF16 else "f32",
                "data": "synthetic", "config": dict(workload_config(wl), launch=launch_mode(args), phi=args.phi, cand_heads=bool(args.cand_heads)), "clocks": clocks,
                "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d // args.steps, "d2h_bytes_per_step": d2h // args.steps,
                        "ms_per_step": e2e_ms / args.steps, "host_issue_ms_per_step": 1e3 * t_issue / args.steps,
                        "score_by_id_alone_ms": score_by_id_ms, "score_by_id_two_arrays_ms": score_by_id_two_arrays_ms,
                        "score_by_id_roofline": dict(kernel="k_score_gather_tc", **roofline_entry(models["k_score_gather_tc"], score_by_id_ms, pk),
                                                     traffic=ncu_traffic("k_score_gather_tc", wl, args),
                                                     note="random rows of packed corpus records [embedding | weights] (score_by_id_two_arrays_ms: "
                                                          "the same from two separate caches); the copy peak is for contiguous streams"),
                        "how": "pinned host ids -> H2D | offsets, history gather, encode, scoring by candidate id from the resident "
                               "packed corpus records | logits D2H; three streams, two request slots"},
                "gpu_launches": int(round(launches_per_step * args.steps)), "roofline": roofline, "scoring_roofline": scoring,
                "kernels": kernels[:14],
                "precompute": {"ms": pre_ms, "candidates": wl.B * wl.C, "candidates_per_s": wl.B * wl.C / (pre_ms * 1e-3),
                               **roofline_entry(models["k_precompute"], pre_ms, pk)},
                "cpu_baseline": cpu, "peaks": pk}
        line["config"]["head"] = args.head or None
        if extras:
            if extras.get("head"):
                hm = dict(bytes=models["k_score"]["bytes"])
                extras["head"].update(roofline_entry(hm, extras["head"]["ms_alone"], pk))
            line["extras"] = extras
        if with_sweeps and world == 1:
            # free this workload's buffers before the sweep points allocate theirs
            del sets, host_sets, table, hist, ws, w_corpus, packed, wscratch, d_hid, d_cid, d_logits, h_logits, extras
            if not args.no_graph:
                del step_graphs, graphs, e2e_graphs
            torch.cuda.empty_cache()
            line["sweeps"] = run_sweeps(args, sampler, pk)
        print(json.dumps(line), flush=True)
    if own_sampler and rank == 0:
        sampler.stop()
    if world > 1:
        dist.destroy_process_group()


# ----------------------------------------------------------------------------- the stages around the core path
def measure_extras(args, wl, lime, bufs, dev):
    """Three short measurements on the bench workload, each with CUDA events on the launching stream:
    head      the per-candidate stage through a one-hidden-layer interaction network (Sec. 3.3; 96 units, App. C) alone;
    link_ctx  Eq. 2 (L^C = MLP(L (+) E^C), 32 context features, one hidden layer of d units) and the encode that takes
              per-user link rows, next to the encode on the shared links;
    overlap   the user side running beside a stand-in for candidate retrieval on a second stream (Sec. 3.3: the user-side
              computation runs in parallel with retrieval): fetching the candidates' cached weight rows and embedding
              rows by id into dense streams; alone, alone, and together."""
    import torch
    from paper_2510_18239_b200 import binding as Bd
    ctx, table, sets = lime.ctx, bufs["table"], bufs["sets"]
    ls, off, ws, logits, hist = bufs["ls"], bufs["off"], bufs["ws"], bufs["logits"], bufs["hist"]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def timed(fn, reps, warm=3):
        for i in range(warm):
            fn(i)
        torch.cuda.synchronize()
        e0.record()
        for i in range(reps):
            fn(i)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps

    out = {}
    # ---- interaction network
    n1 = args.head or 96
    hd = [(Bd.to_device(W, wl.dtype, dev), torch.from_numpy(b).to(dev)) for W, b in head_layers(wl, n1)]
    lime.set_head(hd)
    hws = torch.empty(Bd.lime_head_workspace_bytes(ctx, wl.B), dtype=torch.uint8, device=dev)

    def head_score(i):
        s = sets[i % ROTATE]
        Bd.lime_score_candidates_head(ctx, ls, wl.B, s["W"], s["T"], None, wl.C, wl.B * wl.C, None, logits, hws)

    Bd.lime_profile_start(16)
    head_score(0)
    torch.cuda.synchronize()
    rec, _ = Bd.lime_profile_stop(16)
    out["head"] = {"hidden": [n1], "ms_alone": timed(head_score, 40), "kernels": [k for k, _ in rec],
                   "note": "k_head_lsw (per-user link states x W_0[:d]) + the scorer; bytes per candidate as the dot-product scorer"}
    # ---- Eq. 2 and the encode on per-user link rows
    d_c = 32
    mlp = [(Bd.to_device(W, wl.dtype, dev), torch.from_numpy(b).to(dev)) for W, b in
           synth.ffn_weights(HEAD_SEED, "ctx", (wl.d + d_c, wl.d, wl.d), wl.dtype)]
    lime.set_context_mlp(d_c, mlp)
    ec = Bd.to_device(synth.normal_storage(HEAD_SEED, "ec", (wl.B, d_c), 1.0, wl.dtype), wl.dtype, dev)
    lc = torch.empty((wl.B, wl.ell, wl.d), dtype=torch.float32, device=dev)
    s0 = sets[0]
    h0 = hist[: s0["total"]]
    Bd.lime_lengths_to_offsets(ctx, s0["lengths"], off)
    Bd.lime_gather_history_normalized(ctx, table, s0["hist_ids"], h0)
    t_ctx = timed(lambda i: Bd.lime_contextualize_links(ctx, ec, wl.B, lc), 40)
    t_enc_shared = timed(lambda i: Bd.lime_encode_user_normalized(ctx, h0, off, wl.B, None, ls, ws), 40)
    t_enc_ctx = timed(lambda i: Bd.lime_encode_user_normalized(ctx, h0, off, wl.B, lc, ls, ws), 40)
    out["link_ctx"] = {"d_c": d_c, "hidden": [wl.d], "contextualize_ms": t_ctx, "encode_shared_links_ms": t_enc_shared,
                       "encode_per_user_links_ms": t_enc_ctx}
    # ---- encode beside the retrieval stand-in
    cid = bufs["d_cid"][0]
    Tg = torch.empty((wl.B * wl.C, wl.d), dtype=lime.tdtype, device=dev)
    Wg = torch.empty((wl.B * wl.C, lime.ell_c), dtype=lime.tdtype, device=dev)
    w_corpus = bufs["w_corpus"]
    lime_w = bufs["lime_w"]                     # a context of row width ell_c: the row lookup applied to the cached weights

    def fetch(i):
        Bd.lime_gather_history(ctx, table, cid, Tg)
        Bd.lime_gather_history(lime_w.ctx, w_corpus, cid, Wg)

    def encode(i):
        Bd.lime_encode_user_normalized(ctx, h0, off, wl.B, None, ls, ws)

    t_fetch, t_enc = timed(fetch, 20), timed(encode, 20)
    side = torch.cuda.Stream(dev)
    fork, join = torch.cuda.Event(), torch.cuda.Event()

    def both(i):
        fork.record()
        side.wait_event(fork)
        with torch.cuda.stream(side):
            fetch(i)
            join.record(side)
        encode(i)
        torch.cuda.current_stream().wait_event(join)

    t_both = timed(both, 20)
    out["overlap"] = {"encode_ms": t_enc, "retrieval_standin_ms": t_fetch, "together_ms": t_both,
                      "hidden_fraction": max(0.0, (t_enc + t_fetch - t_both) / max(min(t_enc, t_fetch), 1e-9)),
                      "standin": "lookup of the candidates' cached weight rows and embedding rows by id into dense streams, on a second stream"}
    return out


# ----------------------------------------------------------------------------- the metric's curves, point by point
# Latency vs number of candidates and vs history length (App. F, tables a and b) and the production-shaped batch: a few
# points of each, every one timed long enough for the clock sampler to see it.
SWEEP_POINTS = (
    ("candidate_sweep", dict(C=16)), ("candidate_sweep", dict(C=2048)), ("candidate_sweep", dict(C=32768)),
    ("long_history", dict(n_min=1024, n_max=1024)), ("long_history", dict(n_min=32768, n_max=32768)),
    ("production_ragged", dict()),
)
L2_FLUSH_BYTES = 256 << 20


def measure_point(wl, model, sampler, pk, args, min_seconds=0.35, max_steps=4000):
    """One workload point: p50 / p10 / p90 latency of the step (offsets -> lookup + LayerNorm -> encode -> score), each step
    timed by its own pair of CUDA events after an L2 flush (a 256 MB device buffer is overwritten in between; points
    whose candidate streams exceed 512 MB are not flushed), steps repeated until at least `min_seconds` of device time.
    The precompute for this point's candidates is timed separately, as the paper caches it."""
    import torch
    from paper_2510_18239_b200 import binding as Bd
    lime, table, dev = model["lime"], model["table"], model["dev"]
    ctx = lime.ctx
    seed = 7
    lengths = synth.history_lengths(seed, wl.B, wl.n_min, wl.n_max)
    total = int(lengths.sum())
    d_len = torch.from_numpy(lengths).to(dev)
    d_hid = torch.from_numpy(synth.zipf_ids(seed, "hist_ids", total, wl.V, wl.zipf_s)).to(dev)
    d_cid = torch.from_numpy(synth.uniform_ids(seed, "cand_ids", wl.B * wl.C, wl.V)).to(dev)
    T = lime.gather_history(table, d_cid)
    W = lime.precompute_candidate_links(T)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    stream_bytes = wl.B * wl.C * 2.0 * (wl.d + wl.ell)
    do_flush = stream_bytes < 2 * L2_FLUSH_BYTES
    pre = []
    for _ in range(5):
        flush.zero_()
        e0.record()
        Bd.lime_precompute_candidate_links(ctx, T, W)
        e1.record()
        torch.cuda.synchronize()
        pre.append(e0.elapsed_time(e1))
    off = torch.empty(wl.B + 1, dtype=torch.int32, device=dev)
    hist = torch.empty((total, wl.d), dtype=lime.tdtype, device=dev)
    ls = torch.empty((wl.B, lime.ell_c, wl.d), dtype=lime.tdtype, device=dev)
    logits = torch.empty(wl.B * wl.C, dtype=torch.float32, device=dev)
    ws = lime.workspace(wl.B, total)

    def direct_step():
        Bd.lime_lengths_to_offsets(ctx, d_len, off)
        Bd.lime_gather_history_normalized(ctx, table, d_hid, hist)
        Bd.lime_encode_user_normalized(ctx, hist, off, wl.B, None, ls, ws)
        Bd.lime_score_candidates(ctx, ls, wl.B, W, T, None, wl.C, wl.B * wl.C, None, logits)

    for _ in range(3):
        direct_step()
    torch.cuda.synchronize()
    step = direct_step
    if not args.no_graph:
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            direct_step()
        step = g.replay
        step()
        torch.cuda.synchronize()
    # per-kernel durations of one step (event brackets around every launch: read the shares)
    Bd.lime_profile_start(256)
    for _ in range(3):
        if do_flush:
            flush.zero_()
        direct_step()
    torch.cuda.synchronize()
    records, launches = Bd.lime_profile_stop(256)
    kms = {}
    for name, ms in records:
        kms[name] = kms.get(name, 0.0) + ms / 3
    # the timed steps
    times, busy = [], 0.0
    t_wall0 = time.time()
    while (busy < min_seconds * 1e3 or len(times) < 10) and len(times) < max_steps:
        batch = []
        for _ in range(10):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            if do_flush:
                flush.zero_()
            a.record()
            step()
            b.record()
            batch.append((a, b))
        torch.cuda.synchronize()
        for a, b in batch:
            times.append(a.elapsed_time(b))
        busy = sum(times) * (1.0 + (0.05 / max(statistics.median(times), 1e-3) if do_flush else 0.0))   # ~50 us per flush
    t_wall1 = time.time()
    Bd.lime_device_status(ctx)
    times.sort()
    p50 = times[len(times) // 2]
    clocks = sampler.window(t_wall0, t_wall1)
    score_ms = sum(v for k, v in kms.items() if k.startswith("k_score"))
    models = kernel_models(wl, total, 1)
    out = {"workload": wl.name, "B": wl.B, "N": wl.n_max if not wl.ragged else [wl.n_min, wl.n_max], "tokens": total, "C": wl.C,
           "d": wl.d, "H": wl.H, "ell": wl.ell, "n_layers": wl.n_layers,
           "p50_ms": p50, "p10_ms": times[len(times) // 10], "p90_ms": times[(len(times) * 9) // 10], "steps": len(times),
           "timed_s": (t_wall1 - t_wall0), "candidates_per_s": wl.B * wl.C / (p50 * 1e-3),
           "l2": "flushed before every step (256 MB overwritten)" if do_flush else "candidate streams exceed L2 many times over",
           "launches_per_step": launches / 3, "precompute_ms": sorted(pre)[len(pre) // 2],
           "clocks": clocks, "p50_ms_x_sm_mhz": (p50 * clocks["sm_mhz"]) if clocks.get("sm_mhz") else None,
           "score_ms": score_ms,
           "score_roofline": (dict(roofline_entry(models["k_score"], score_ms, pk), timing="CUDA events around the launch inside the step")
                              if score_ms > 0 else None),
           "kernels_ms": {k: round(v, 5) for k, v in sorted(kms.items(), key=lambda kv: -kv[1])[:8]}}
    enc = {k: v for k, v in kms.items() if not k.startswith(("k_score", "k_gather", "k_offsets"))}
    out["encode_ms"] = sum(enc.values())
    dom = max(enc, key=enc.get) if enc else None
    mdl = model_for(dom, models) if dom else None
    if mdl:
        out["encode_dominant"] = dict(kernel=dom, ms=enc[dom], **roofline_entry(mdl, enc[dom], pk))
    del T, W, hist, ws, flush, logits
    torch.cuda.empty_cache()
    return out


def run_sweeps(args, sampler, pk):
    import torch
    from paper_2510_18239_b200 import binding as Bd
    dev = torch.device("cuda", torch.cuda.current_device())
    named = synth.named_workloads()
    points, model, model_name = [], None, None
    for name, kw in SWEEP_POINTS:
        if args.sweep_only and name not in args.sweep_only.split(","):
            continue
        base = named[name]
        wl = base.replace(**kw) if kw else base
        if model_name != name:
            model = None
            torch.cuda.empty_cache()
            # the model of the named workload: table, links and layer weights (requests are drawn per point)
            inp = synth.make_inputs(base.replace(B=1, C=1, n_min=1, n_max=1), seed=0)
            lime = Bd.Lime(base.d, base.H, base.ell, base.n_layers, dtype=Bd.LIME_BF16, d_ff=base.d_ff)
            table = Bd.to_device(inp["table"], base.dtype, dev)
            links = Bd.to_device(inp["links"], base.dtype, dev)
            wts = {k: Bd.to_device(inp[k], base.dtype, dev) for k in ("Wq", "Wk", "Wv", "Wg", "Wu", "Wo")}
            lime.set_weights(links, [{k: wts[k][j] for k in wts} for j in range(base.n_layers)])
            model, model_name = dict(lime=lime, table=table, dev=dev, keep=(links, wts)), name
            del inp
        points.append(measure_point(wl, model, sampler, pk, args))
    # "flat in C": all growth with C is the candidate stream at >= 70 % of the copy peak on top of the C-independent encode
    cs = [q for q in points if q["workload"] == "candidate_sweep"]
    if cs:
        t_small = min(cs, key=lambda q: q["C"])["p50_ms"]
        for q in cs:
            stream = q["B"] * q["C"] * (2.0 * (q["d"] + q["ell"]) + 4.0)
            bound = t_small + stream / (0.7 * pk["hbm_gbs"] * 1e9) * 1e3
            q["flat_in_C"] = {"p50_ms": q["p50_ms"], "bound_ms": bound, "holds": q["p50_ms"] <= bound,
                              "rule": "t(C) <= t(smallest C) + stream bytes(C) / (0.7 x copy peak)"}
    return {"points": points,
            "paper": "LIME-XOR 2.07 -> 2.15 ms over C = 16..32768 and 2.08 -> 2.12 ms over N = 1024..16384 (App. F, hardware unstated)"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="bf16_baseline")
    ap.add_argument("--C", type=int, default=0, help="override candidates per user (candidate sweep)")
    ap.add_argument("--N", type=int, default=0, help="override history length (history sweep)")
    ap.add_argument("--B", type=int, default=0)
    ap.add_argument("--cpu-budget", type=float, default=12.0, help="seconds of oracle work for cpu_baseline")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sweep", default="", choices=["", "C", "N"], help="one line per point of the candidate / history sweep")
    ap.add_argument("--phi", default="softmax", choices=["softmax", "silu"],
                    help="attention activation of the XOR layers: online softmax (default) or SiLU(s) / n (Algorithms 1-2)")
    ap.add_argument("--cand-heads", action="store_true",
                    help="candidate side head by head (Eq. 1 applied to Eq. 4): H * ell cached weights per candidate")
    ap.add_argument("--head", type=int, default=0,
                    help="score through an interaction network with one hidden layer of this many units (Sec. 3.3; 0 = dot product)")
    ap.add_argument("--no-extras", action="store_true", help="leave out the `extras` object (head, link_ctx, overlap)")
    ap.add_argument("--no-graph", action="store_true", help="launch every step from the host instead of replaying CUDA graphs")
    ap.add_argument("--no-sweeps", action="store_true",
                    help="leave out the `sweeps` object (points of the candidate sweep, the history sweep and production_ragged)")
    ap.add_argument("--sweep-only", default="", help="comma-separated workload names whose sweep points to keep")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    wl = synth.named_workloads()[args.workload]
    if args.C:
        wl = wl.replace(C=args.C)
    if args.N:
        wl = wl.replace(n_min=args.N, n_max=args.N)
    if args.B:
        wl = wl.replace(B=args.B)
    if args.impl == "reference":
        run_reference(args, wl)
    elif args.sweep == "C":
        # latency vs number of candidates (App. F, table a): one JSON line per C, model and batch of `candidate_sweep`
        base = synth.named_workloads()["candidate_sweep"]
        for C in synth.CANDIDATE_SWEEP_C:
            run_ours(args, base.replace(C=C, B=args.B or base.B))
    elif args.sweep == "N":
        # latency vs history length (App. F, table b): one JSON line per N, model and batch of `long_history`
        base = synth.named_workloads()["long_history"]
        for N in synth.LONG_HISTORY_N:
            run_ours(args, base.replace(n_min=N, n_max=N, B=args.B or base.B))
    else:
        # the default run carries the metric's curves in its one line; explicit workloads and multi-GPU runs do not
        plain_default = args.workload == "bf16_baseline" and not (args.C or args.N or args.B) and args.phi == "softmax" and not args.cand_heads and not args.head
        run_ours(args, wl, with_sweeps=plain_default and not args.no_sweeps and int(os.environ.get("WORLD_SIZE", "1")) == 1)


if __name__ == "__main__":
    main()
