#!/usr/bin/env python
"""Benchmark of the LANTERN relaxed-verification step (metric: verified draft positions per second).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload batch_chain|stress|...] [--impl reference]

A step is one `verify` call over one batch of synthetic input: every drafted position of every
sequence is tested (guidance combine, softmax of target and drafter, A_{k,delta} aggregation,
relaxed accept test, residual resampling, walk, bonus draw).  The default workload is the
V = 16384, k = 1000, delta = 0.4 chain configuration with its 32 images x 256 positions
flattened into one call of 8192 sequences x 7 drafts (6.4 GB of bf16 logits, far larger than
L2, so consecutive steps cannot be served from cache).  The neighbour table is built once
before the timed region, as in the method, and its build time is reported separately.

With N > 1 (under torch.distributed.run) every rank verifies its own batch of the same
shape: the path has no exchange step, so this is weak scaling with no collective on the
data path; the ranks only meet at the timing barriers.

`--impl reference` times the CPU oracle (oracle/, as it stands, one thread) on a bounded
sample of the same workload and prints the same JSON line with "impl": "reference".
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "relaxed_verify_positions_per_s"
UNIT = "positions/s"

# the paper's guidance/neighbourhood settings per workload; B is the flattened call size
WORKLOADS = {
    "batch_chain": dict(config="batch_chain", B=32 * 256, note="32 images x 256 positions, chain of 7 drafts"),
    "stress": dict(config="stress", B=128, note="128 sequences x 60-node depth-6 trees"),
    "px512_tree": dict(config="px512_tree", B=8 * 64, note="8 images x 64 positions, 60-node trees"),
    "single_image": dict(config="single_image", B=256, note="1 image x 256 positions, 60-node trees"),
    "tiny": dict(config="tiny", B=64, note="64 steps of the tiny chain configuration"),
}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            return float(json.load(open(path))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


def algorithmic_bytes(cfg: dict, B: int, parents, greedy: bool = False) -> int:
    """Bytes the method must move per call: for each context with at least one child, two target
    rows and one drafter row (one target row without guidance; no drafter row in greedy
    decoding), plus one neighbour row of 4k bytes per drafted node.  Bonus rows, tokens, uniforms
    and outputs (< 0.1 %) are left out."""
    import lantern_inputs as li
    esize = 2 if cfg["dtype"] == li.BF16 else 4
    rows = (2 if cfg["has_uncond"] else 1) + (0 if greedy else 1)
    N, V, k = cfg["N"], cfg["V"], cfg["k"]
    if parents is None:
        n_ctx = B * N
    else:
        par = parents.cpu().numpy()
        n_ctx = sum(len(set(par[b].tolist())) for b in range(B))
    return n_ctx * rows * V * esize + B * N * 4 * k


# DRAM traffic of the fused kernel from one ncu capture (dram__bytes_read.sum + dram__bytes_write.sum)
# of a 512-sequence call of the chain workload, as a ratio to that call's algorithmic bytes; traffic
# grows in proportion to the contexts processed, so a full launch is scaled by its algorithmic bytes.
# Tied to the kernel revision the capture was taken on: any other revision reports null.
NCU_TRAFFIC = {"kernel_revision": 15, "workload": "batch_chain", "traffic_over_algorithmic": 377546752 / 366657536}


def ncu_traffic(workload, cfg, alg_bytes):
    import paper_2410_03355_b200 as lt
    if NCU_TRAFFIC["traffic_over_algorithmic"] is None or workload != NCU_TRAFFIC["workload"]:
        return None
    if lt.kernel_revision() != NCU_TRAFFIC["kernel_revision"]:
        return None
    return int(alg_bytes * NCU_TRAFFIC["traffic_over_algorithmic"])


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for nm, val in zip(names, f[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def oracle_sample_rate(host_inp, table_host, delta, budget_s=15.0, greedy=False, divergence=0, top_k=0):
    """Oracle throughput (drafted positions verified per second) on as many leading sequences of
    `host_inp` as fit in about `budget_s` seconds; returns (rate, n_sequences, seconds)."""
    import dataclasses

    import oracle
    done, t_used, pos = 0, 0.0, 0
    chunk = 8
    while done < host_inp.B and t_used < budget_s:
        n = min(chunk, host_inp.B - done)
        sl = slice(done, done + n)
        part = dataclasses.replace(
            host_inp, target_logits=np.ascontiguousarray(host_inp.target_logits[:, sl]),
            draft_logits=np.ascontiguousarray(host_inp.draft_logits[sl]),
            draft_tokens=np.ascontiguousarray(host_inp.draft_tokens[sl]),
            tree_parents=None if host_inp.tree_parents is None else np.ascontiguousarray(host_inp.tree_parents[sl]),
            uniforms=np.ascontiguousarray(host_inp.uniforms[sl]), B=n)
        t0 = time.perf_counter()
        if greedy:
            oracle.verify_greedy(part.target_logits, part.dtype, part.cfg_scale, part.has_uncond, part.draft_tokens,
                                 part.tree_parents, table_host, delta, divergence, top_k)
        else:
            oracle.verify_inputs(part, table_host, delta, divergence, top_k)
        t_used += time.perf_counter() - t0
        done += n
        pos += n * host_inp.N
        chunk = min(chunk * 2, 256)
    return pos / t_used, done, t_used


def max_over_ranks(values, dist=None, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (every rank gets the result).  The
    verification path has no exchange step: this reduction of the measured times is the only
    collective of a multi-rank run."""
    if dist is None:
        return [float(v) for v in values]
    import torch
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def rank_seed(base_seed: int, rank: int) -> int:
    """Every rank verifies its own, differently seeded batch of the same shape (weak scaling)."""
    return int(base_seed) + 17 * int(rank)


def aggregate_rate(world: int, sequences_per_rank: int, drafts: int, ms_per_step: float) -> float:
    """Whole-job positions per second: all ranks' positions over the slowest rank's step time."""
    return world * sequences_per_rank * drafts / (ms_per_step * 1e-3)


def run_reference(args, rank, world):
    """The reference arm: the CPU oracle as it stands, timed on host cores on a bounded sample."""
    if rank != 0:
        return
    import lantern_inputs as li
    import oracle
    w = WORKLOADS[args.workload]
    cfg = li.CONFIGS[w["config"]]
    # bounded sample: a few sequences per step so that the run ends within minutes
    nseq = {"batch_chain": 64, "stress": 4, "px512_tree": 4, "single_image": 4, "tiny": 64}[args.workload]
    cb = li.config_codebook(w["config"])
    steps_t = []
    div = oracle.DIV_JSD if args.divergence == "jsd" else oracle.DIV_TVD
    table_cache = {}   # the table is an input of the step: only the rows the sample's drafts touch are built

    def table_for(inp):
        need = np.unique(inp.draft_tokens)
        miss = np.array([t for t in need if t not in table_cache], dtype=np.int32)
        if miss.size:
            idx, _ = oracle.build_neighbors(cb, cfg["k"], rows=miss, metric=args.metric)
            for r, t in enumerate(miss):
                table_cache[int(t)] = idx[r]
        tab = np.zeros((cfg["V"], cfg["k"]), np.int32)
        tab[:, 0] = np.arange(cfg["V"])
        for t in need:
            tab[t] = table_cache[int(t)]
        return tab

    for step in range(args.warmup + args.steps):
        inp = li.config_verify_inputs(w["config"], step=step, B=nseq)
        tab = table_for(inp)
        t1 = time.perf_counter()
        if args.greedy:
            oracle.verify_greedy(inp.target_logits, inp.dtype, inp.cfg_scale, inp.has_uncond, inp.draft_tokens,
                                 inp.tree_parents, tab, cfg["delta"], div, args.top_k)
        else:
            oracle.verify_inputs(inp, tab, cfg["delta"], div, args.top_k)
        dt = time.perf_counter() - t1
        if step >= args.warmup:
            steps_t.append(dt)
    total = sum(steps_t)
    value = nseq * cfg["N"] * len(steps_t) / total
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / len(steps_t),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "V": cfg["V"], "k": cfg["k"], "delta": cfg["delta"], "N": cfg["N"],
                   "T": 0.0 if args.greedy else cfg["T"], "divergence": args.divergence, "metric": args.metric,
                   "top_k": args.top_k, "sequences_per_step": nseq},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle",
                         "sample": f"{nseq} sequences x {cfg['N']} drafts per step of the {args.workload} workload "
                                   f"(bounded sample; neighbour rows built by the oracle outside the timed region)"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def run_aggregate(args):
    """Side benchmark (not the headline metric): lantern_aggregate_all on `--aggregate-rows` root-context rows
    of the workload.  Every row re-reads the whole neighbour table (V * k * 4 bytes), which lives in L2."""
    import torch

    import lantern_inputs as li
    import lantern_inputs.device as lid
    import oracle
    import paper_2410_03355_b200 as lt
    torch.cuda.set_device(0)
    w = WORKLOADS[args.workload]
    cfg = li.CONFIGS[w["config"]]
    V, k, delta = cfg["V"], cfg["k"], cfg["delta"]
    rows = args.aggregate_rows
    cb = torch.from_numpy(li.config_codebook(w["config"])).cuda()
    table, _ = lt.build_neighbors(cb, k, with_dist=False, metric=args.metric)
    d = lid.config_verify_inputs_device(w["config"], B=rows, seed=li.BASE_SEED)
    logits = d["target_logits"][:, :, 0].contiguous()            # [C, rows, V]: the root contexts
    for _ in range(max(args.warmup, 3)):
        lt.aggregate_all(logits, d["cfg_scale"], d["T"], table, delta, with_m=False)
    torch.cuda.synchronize()
    a, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    steps = min(args.steps, 20)
    a.record()
    for _ in range(steps):
        agg, _, status = lt.aggregate_all(logits, d["cfg_scale"], d["T"], table, delta, with_m=False)
    b_.record()
    torch.cuda.synchronize()
    ms = a.elapsed_time(b_) / steps
    t0 = time.perf_counter()
    host = logits[:, :1].cpu()
    hl = host.view(torch.int16).numpy().view(np.uint16) if cfg["dtype"] == li.BF16 else host.numpy()
    oracle.aggregate_all(hl[0], hl[1] if cfg["has_uncond"] else None, cfg["dtype"], d["cfg_scale"], d["T"],
                         table.cpu().numpy(), delta)
    cpu_s = time.perf_counter() - t0
    table_bytes = rows * V * k * 4
    print(json.dumps({
        "metric": "all_token_aggregation_rows_per_s", "value": rows / (ms * 1e-3), "unit": "rows/s", "n_gpus": 1,
        "steps": steps, "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True, "data": "synthetic",
        "dtype": "f32", "config": {"workload": args.workload, "rows": rows, "V": V, "k": k, "delta": delta,
                                   "note": "side benchmark of the V x k gather-sum; not used by verification"},
        "roofline": {"bound": "l2", "kernel": "lantern_aggregate_kernel", "achieved": table_bytes / (ms * 1e-3) / 1e9,
                     "peak": None, "unit": "GB/s", "frac": None, "traffic": None,
                     "note": "achieved = neighbour-table bytes read per second (from L2); no measured L2 peak on file",
                     "gathers_per_s": rows * V * k / (ms * 1e-3)},
        "cpu_baseline": {"value": 1.0 / cpu_s, "unit": "rows/s", "cores": 1, "kind": "oracle", "sample": "1 row"},
        "gpu_launches": steps, "outputs": {"rows_with_status_bits": int((status != 0).sum().item()),
                                           "mean_aggregated_mass": float(agg.mean().item() * V)},
    }), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="batch_chain", choices=sorted(WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--batch", type=int, default=0, help="override the number of sequences per call")
    ap.add_argument("--rho", type=float, default=0.0, help="correlation of conditional and unconditional rows")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--divergence", default="tvd", choices=["tvd", "jsd"],
                    help="what delta bounds (Section 5.3.2); the JSD run uses the workload's delta as it is")
    ap.add_argument("--metric", default="l2", choices=["l2", "cosine"], help="latent proximity of the table")
    ap.add_argument("--top-k", type=int, default=0, dest="top_k",
                    help="top-k logit filter of the generation settings (Appendix B.2); 0 = off")
    ap.add_argument("--aggregate-rows", type=int, default=0, dest="aggregate_rows",
                    help="run the all-token aggregation side benchmark on this many rows instead of verification")
    ap.add_argument("--greedy", action="store_true",
                    help="run the workload at T = 0 (greedy decoding: no drafter rows, no random numbers)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        run_reference(args, rank, world)
        return
    if args.aggregate_rows > 0:
        if rank == 0:
            run_aggregate(args)
        return

    import torch

    import lantern_inputs as li
    import lantern_inputs.device as lid
    import paper_2410_03355_b200 as lt

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    lt.load_library()

    w = WORKLOADS[args.workload]
    cfg = li.CONFIGS[w["config"]]
    B = args.batch or w["B"]
    N, V, k, delta = cfg["N"], cfg["V"], cfg["k"], cfg["delta"]

    # ---- one-time neighbour table (timed separately) ----
    cb = torch.from_numpy(li.config_codebook(w["config"])).cuda()
    bws = torch.empty(max(lt.load_library().lantern_build_workspace_bytes_metric(V, cfg["D"], k, lt.METRICS[args.metric]), 256),
                      dtype=torch.uint8, device="cuda")
    lt.build_neighbors(cb, k, with_dist=False, workspace=bws, metric=args.metric)      # warm-up
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    table, _ = lt.build_neighbors(cb, k, with_dist=False, workspace=bws, metric=args.metric)
    e1.record()
    torch.cuda.synchronize()
    build_ms = e0.elapsed_time(e1)
    del bws

    # ---- inputs resident in HBM ----
    d = lid.config_verify_inputs_device(w["config"], B=B, seed=rank_seed(li.BASE_SEED, rank), rho=args.rho)
    torch.cuda.synchronize()
    alg_bytes = algorithmic_bytes(cfg, B, d["tree_parents"], args.greedy)
    T = 0.0 if args.greedy else d["T"]
    ws = torch.empty(lt.verify_workspace_bytes(B, N, V, k, cfg["dtype"], args.top_k), dtype=torch.uint8, device="cuda")
    i32 = dict(dtype=torch.int32, device="cuda")
    out = lt.VerifyOutputs(accept_len=torch.empty(B, **i32), next_token=torch.empty(B, **i32),
                           accept_path=torch.empty((B, N), **i32), status=torch.empty(B, **i32),
                           node_qa=None, node_px=None, node_m=None)
    stream = torch.cuda.current_stream()

    def step():
        lt.verify(d["target_logits"], None if args.greedy else d["draft_logits"], d["cfg_scale"], T, d["draft_tokens"],
                  d["tree_parents"], table, delta, None if args.greedy else d["uniforms"], out=out, workspace=ws,
                  stream=stream, divergence=args.divergence, top_k=args.top_k)

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()

    # per-step events around the fused kernel (dominant kernel of the roofline)
    kev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    for a, b_ in kev:       # torch creates the CUDA event on first record
        a.record()
        b_.record()
    torch.cuda.synchronize()

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    t_start, t_stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_start.record()
    for a, b_ in kev:
        lt.profile_events(a, b_)
        step()
    t_stop.record()
    torch.cuda.synchronize()
    lt.profile_events(None, None)
    if dist is not None:
        dist.barrier()
    clocks = sampler.stop() if rank == 0 else None
    ms_total = t_start.elapsed_time(t_stop)
    fused_ms = float(np.mean([a.elapsed_time(b_) for a, b_ in kev]))
    ms_total, fused_ms = max_over_ranks([ms_total, fused_ms], dist, "cuda")
    ms_per_step = ms_total / args.steps
    value = aggregate_rate(world, B, N, ms_per_step)

    status_bad = int((out.status != 0).sum().item())
    accept_mean = float(out.accept_len.float().mean().item())

    # ---- end to end: host buffers in, host results out, through the public API ----
    e2e = None
    if not args.no_e2e:
        host = {}
        names = ("target_logits", "draft_tokens", "tree_parents") if args.greedy else \
                ("target_logits", "draft_logits", "draft_tokens", "tree_parents", "uniforms")
        for name in names:
            t = d[name]
            host[name] = None if t is None else torch.empty(t.shape, dtype=t.dtype, pin_memory=True).copy_(t)
        h_len = torch.empty(B, dtype=torch.int32, pin_memory=True)
        h_tok = torch.empty(B, dtype=torch.int32, pin_memory=True)
        h2d = sum(t.numel() * t.element_size() for t in host.values() if t is not None)
        d2h = 2 * B * 4

        def e2e_step():
            for name, t in host.items():
                if t is not None:
                    d[name].copy_(t, non_blocking=True)
            step()
            h_len.copy_(out.accept_len, non_blocking=True)
            h_tok.copy_(out.next_token, non_blocking=True)

        e2e_step()
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        a, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(args.e2e_steps):
            e2e_step()
        b_.record()
        torch.cuda.synchronize()
        ms_e2e = a.elapsed_time(b_) / args.e2e_steps
        ms_e2e = max_over_ranks([ms_e2e], dist, "cuda")[0]
        e2e = {"value": aggregate_rate(world, B, N, ms_e2e), "unit": UNIT, "h2d_bytes_per_step": int(h2d),
               "d2h_bytes_per_step": int(d2h), "ms_per_step": ms_e2e, "steps": args.e2e_steps}
        del host

    # ---- CPU baseline: the oracle on a bounded sample of the same inputs (rank 0, N = 1) ----
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        n_s = min(B, 8192 if cfg["N"] <= 8 else 256)
        host_inp = lid.to_host(d, rows=np.arange(n_s))
        rate, n_done, secs = oracle_sample_rate(host_inp, table.cpu().numpy(), delta, greedy=args.greedy,
                                                divergence=1 if args.divergence == "jsd" else 0, top_k=args.top_k)
        cpu = {"value": rate, "unit": UNIT, "cores": 1, "kind": "oracle",
               "sample": f"first {n_done} sequences ({n_done * N} drafted positions) of this call, {secs:.1f} s"}

    if rank == 0:
        peak, peak_kind = load_peaks()
        achieved = alg_bytes / (fused_ms * 1e-3) / 1e9
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": args.workload, "note": w["note"], "sequences_per_call": B, "drafts_per_sequence": N,
                       "V": V, "k": k, "delta": delta, "cfg_scale": cfg["cfg_scale"], "T": T, "divergence": args.divergence, "metric": args.metric,
                       "top_k": args.top_k,
                       "logits": "bf16" if cfg["dtype"] == li.BF16 else "f32", "rho": args.rho,
                       "l2_policy": "inputs larger than L2 (%.2f GB of logits per call)" %
                                    ((d["target_logits"].numel() + (0 if args.greedy else d["draft_logits"].numel())) *
                                     d["target_logits"].element_size() / 1e9),
                       "parallelism": "replicas" if world > 1 else "single"},
            "roofline": {"bound": "hbm", "kernel": "lantern_greedy_context_kernel" if args.greedy else "lantern_context_kernel",
                         "achieved": achieved, "peak": peak,
                         "peak_kind": f"of {peak_kind}", "unit": "GB/s", "frac": achieved / peak,
                         "traffic": None if (args.greedy or args.divergence != "tvd" or 0 < args.top_k < V) else
                                    ncu_traffic(args.workload, cfg, alg_bytes),
                         "algorithmic_bytes_per_launch": int(alg_bytes), "kernel_ms": fused_ms},
            "cpu_baseline": cpu, "e2e": e2e,
            "gpu_launches": (4 + (0 if not 0 < args.top_k < V else (1 if args.greedy else 2))) * args.steps, "clocks": clocks,
            "neighbor_build": {"ms": build_ms, "V": V, "D": cfg["D"], "k": k,
                               "pairs_per_s": V * V / (build_ms * 1e-3)},
            "outputs": {"mean_accept_len": accept_mean, "sequences_with_status_bits": status_bad},
        }
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
