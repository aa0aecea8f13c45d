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


def context_bytes(cfg: dict, greedy: bool = False) -> int:
    """Logit bytes of one evaluated context: two target rows and one drafter row (one target row without
    guidance; no drafter row in greedy decoding)."""
    import lantern_inputs as li
    esize = 2 if cfg["dtype"] == li.BF16 else 4
    rows = (2 if cfg["has_uncond"] else 1) + (0 if greedy else 1)
    return rows * cfg["V"] * esize


def work_bytes(cfg: dict, contexts: int, nodes: int, greedy: bool = False) -> int:
    """Bytes that `contexts` evaluated contexts and `nodes` tested drafts must move: the contexts' logit rows
    plus one neighbour row of 4k bytes per tested node.  Bonus rows, tokens, uniforms and outputs (< 0.1 %)
    are left out."""
    return contexts * context_bytes(cfg, greedy) + nodes * 4 * cfg["k"]


def method_work(parents, accept_len, accept_path, N: int):
    """(contexts, nodes) that Algorithm 1's loop itself evaluates and tests on the accepted paths: it goes on
    from an accepted node only and stops at the first context whose children are all rejected.  For a tree
    the children of a context are tried in node order up to and including the accepted one."""
    al = accept_len.cpu().numpy().astype(np.int64)
    if parents is None:
        n = np.minimum(al + 1, N)            # the context after the last accepted draft is tested unless the chain ended
        return int(n.sum()), int(n.sum())
    par = parents.cpu().numpy()
    path = accept_path.cpu().numpy()
    contexts = nodes = 0
    for b in range(par.shape[0]):
        kids = {}
        for i, p_ in enumerate(par[b].tolist()):
            kids.setdefault(p_ + 1, []).append(i)
        cur = 0
        for j in range(int(al[b])):
            node = int(path[b, j])
            contexts += 1
            nodes += kids[cur].index(node) + 1
            cur = node + 1
        if cur in kids:                      # every child of the last context was rejected
            contexts += 1
            nodes += len(kids[cur])
    return contexts, nodes


# DRAM traffic of the fused kernel from one ncu capture (dram__bytes_read.sum + dram__bytes_write.sum) of a
# 1024-sequence call of the chain workload, as a ratio to the bytes of the 5348 contexts and nodes that call evaluated;
# traffic grows in proportion to the contexts evaluated, so a full launch is scaled by its evaluated bytes.
# Tied to the kernel revision the capture was taken on: any other revision reports null.
NCU_TRAFFIC = {"kernel_revision": 18, "workload": "batch_chain", "traffic_over_algorithmic": 564017408 / 548656352}


def ncu_traffic(workload, alg_bytes):
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


def oracle_table_rows(cb, k, tokens, metric="l2"):
    """[V, k] host table whose rows for the given drafted tokens are built by the oracle (the other rows are
    never read by a verification of those sequences and hold -1 beyond the token itself)."""
    import oracle
    V = cb.shape[0]
    need = np.unique(np.asarray(tokens).ravel())
    need = need[(need >= 0) & (need < V)].astype(np.int32)
    tab = np.full((V, k), -1, np.int32)
    tab[:, 0] = np.arange(V)
    if need.size:
        tab[need] = oracle.build_neighbors(cb, k, rows=need, metric=metric)[0]
    return tab, need


def _oracle_worker(config, step, nseq, barrier, queue):
    """One process of the all-cores oracle run: its own seeded sample of the workload, its own neighbour rows,
    then -- together with the others -- the timed verification."""
    import lantern_inputs as li
    import oracle
    cfg = li.CONFIGS[config]
    inp = li.config_verify_inputs(config, step=step, B=nseq)
    tab, _ = oracle_table_rows(li.config_codebook(config), cfg["k"], inp.draft_tokens)
    barrier.wait()
    t0 = time.perf_counter()
    oracle.verify_inputs(inp, tab, cfg["delta"])
    queue.put((nseq * cfg["N"], time.perf_counter() - t0))


def oracle_all_cores(config: str, nseq: int = 48, max_procs: int = 32):
    """The oracle as it stands (single-threaded code) run by one process per host core on disjoint seeded
    samples of the workload at the same time: positions per second over the slowest process.  Processes are
    started with `spawn`: a process forked after the first GPU call would hang."""
    import multiprocessing as mp
    ctx = mp.get_context("spawn")
    n = max(1, min(os.cpu_count() or 1, max_procs))
    barrier, queue = ctx.Barrier(n), ctx.Queue()
    procs = [ctx.Process(target=_oracle_worker, args=(config, 1000 + i, nseq, barrier, queue)) for i in range(n)]
    for p_ in procs:
        p_.start()
    got = [queue.get(timeout=600) for _ in procs]
    for p_ in procs:
        p_.join()
    return sum(g[0] for g in got) / max(g[1] for g in got), n


class Run:
    """One workload resident in HBM: inputs, table, outputs, workspace, and the timed call."""

    def __init__(self, args, workload, B=None, rank=0, seed=None):
        import torch

        import lantern_inputs as li
        import lantern_inputs.device as lid
        import paper_2410_03355_b200 as lt
        self.lt, self.torch, self.args = lt, torch, args
        self.workload = workload
        w = WORKLOADS[workload]
        self.cfg = cfg = li.CONFIGS[w["config"]]
        self.B = B or w["B"]
        self.N, self.V, self.k, self.delta = cfg["N"], cfg["V"], cfg["k"], cfg["delta"]
        self.greedy = args.greedy
        # ---- one-time neighbour table (timed separately) ----
        self.cb_host = li.config_codebook(w["config"])
        cb = torch.from_numpy(self.cb_host).cuda()
        bws = torch.empty(max(lt.load_library().lantern_build_workspace_bytes_metric(
            self.V, cfg["D"], self.k, lt.METRICS[args.metric]), 256), dtype=torch.uint8, device="cuda")
        lt.build_neighbors(cb, self.k, with_dist=False, workspace=bws, metric=args.metric)      # warm-up
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        self.table, _ = lt.build_neighbors(cb, self.k, with_dist=False, workspace=bws, metric=args.metric)
        e1.record()
        torch.cuda.synchronize()
        self.build_ms = e0.elapsed_time(e1)
        del bws
        # ---- inputs resident in HBM ----
        self.d = d = lid.config_verify_inputs_device(
            w["config"], B=self.B, seed=rank_seed(li.BASE_SEED, rank) if seed is None else seed, rho=args.rho)
        torch.cuda.synchronize()
        self.T = 0.0 if self.greedy else d["T"]
        self.ws = torch.empty(lt.verify_workspace_bytes(self.B, self.N, self.V, self.k, cfg["dtype"], args.top_k),
                              dtype=torch.uint8, device="cuda")
        i32 = dict(dtype=torch.int32, device="cuda")
        self.out = lt.VerifyOutputs(accept_len=torch.empty(self.B, **i32), next_token=torch.empty(self.B, **i32),
                                    accept_path=torch.empty((self.B, self.N), **i32), status=torch.empty(self.B, **i32),
                                    node_qa=None, node_px=None, node_m=None)
        self.stream = torch.cuda.current_stream()
        self.logit_gb = (d["target_logits"].numel() + (0 if self.greedy else d["draft_logits"].numel())) * \
            d["target_logits"].element_size() / 1e9

    def variant(self, args):
        """The same inputs and table under other settings (greedy decoding, logit filter, bound): own outputs and workspace."""
        import copy
        v = copy.copy(self)
        torch, lt = self.torch, self.lt
        v.args, v.greedy = args, args.greedy
        v.T = 0.0 if args.greedy else self.d["T"]
        v.ws = torch.empty(lt.verify_workspace_bytes(self.B, self.N, self.V, self.k, self.cfg["dtype"], args.top_k),
                           dtype=torch.uint8, device="cuda")
        v.out = lt.VerifyOutputs(*(None if t is None else torch.empty_like(t)
                                   for t in (getattr(self.out, f.name) for f in __import__("dataclasses").fields(self.out))))
        return v

    def step(self, out=None, trace=False):
        d, a = self.d, self.args
        return self.lt.verify(d["target_logits"], None if self.greedy else d["draft_logits"], d["cfg_scale"], self.T,
                              d["draft_tokens"], d["tree_parents"], self.table, self.delta,
                              None if self.greedy else d["uniforms"], out=None if trace else (out or self.out),
                              trace=trace, workspace=self.ws, stream=self.stream, divergence=a.divergence, top_k=a.top_k)

    def timed(self, steps, warmup, dist=None, flush=None):
        """`steps` calls between two events, with an event pair around every call's fused kernel.  `flush` (a
        buffer larger than L2) is rewritten between calls when the call's own inputs are smaller than L2."""
        torch, lt = self.torch, self.lt
        for _ in range(warmup):
            self.step()
        torch.cuda.synchronize()
        kev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for a, b_ in kev:       # torch creates the CUDA event on first record
            a.record()
            b_.record()
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        cev = []
        if flush is None:
            t0.record()
            for a, b_ in kev:
                lt.profile_events(a, b_)
                self.step()
            t1.record()
        else:                   # per-call events: the flush sits between calls, outside every timed interval
            for a, b_ in kev:
                flush.add_(1)
                c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                lt.profile_events(a, b_)
                c0.record()
                self.step()
                c1.record()
                cev.append((c0, c1))
        torch.cuda.synchronize()
        lt.profile_events(None, None)
        ms_total = t0.elapsed_time(t1) if flush is None else sum(c0.elapsed_time(c1) for c0, c1 in cev)
        fused_ms = float(np.mean([a.elapsed_time(b_) for a, b_ in kev]))
        return ms_total, fused_ms

    def accounting(self, fused_ms, peak):
        """Work and roofline figures of the last call."""
        counts = self.lt.verify_counts(self.ws)
        greedy = self.greedy
        n_ctx = counts["contexts"]
        ev_ctx = counts["evaluated"]
        ev_nodes = counts["nodes_tested"]
        m_ctx, m_nodes = method_work(self.d["tree_parents"], self.out.accept_len, self.out.accept_path, self.N)
        ev_bytes = work_bytes(self.cfg, ev_ctx, ev_nodes, greedy)
        m_bytes = work_bytes(self.cfg, m_ctx, m_nodes, greedy)
        all_bytes = work_bytes(self.cfg, n_ctx, self.B * self.N, greedy)
        sec = fused_ms * 1e-3
        return dict(contexts_with_children=n_ctx, contexts_evaluated=ev_ctx, contexts_skipped=counts["skipped"],
                    nodes_tested=ev_nodes, method_contexts=m_ctx, method_nodes=m_nodes,
                    evaluated_bytes=int(ev_bytes), method_bytes=int(m_bytes), all_context_bytes=int(all_bytes),
                    achieved=ev_bytes / sec / 1e9, frac=ev_bytes / sec / 1e9 / peak,
                    method_achieved=m_bytes / sec / 1e9, method_frac=m_bytes / sec / 1e9 / peak)

    def parity_sample(self, n_sample):
        """A traced call compared with the oracle on a seeded sample of its sequences (the oracle reads its own
        neighbour rows, which are first compared with the library's): counts of sequences with a decision
        inside the 1e-6 window and of mismatches outside it."""
        import lantern_inputs.device as lid
        sys.path.insert(0, os.path.join(ROOT, "tests"))
        import parity
        torch = self.torch
        out = self.step(trace=True)
        torch.cuda.synchronize()
        rows = np.sort(np.random.default_rng(5).choice(self.B, size=min(n_sample, self.B), replace=False))
        host = lid.to_host(self.d, rows=rows)
        tab, need = oracle_table_rows(self.cb_host, self.k, host.draft_tokens, self.args.metric)
        lib_rows = self.table[torch.from_numpy(need.astype(np.int64)).cuda()].cpu().numpy()
        idx = torch.as_tensor(rows, device="cuda")
        pick = lambda t: None if t is None else t[idx]
        sub = self.lt.VerifyOutputs(*(pick(getattr(out, f.name)) for f in __import__("dataclasses").fields(out)))
        div = 1 if self.args.divergence == "jsd" else 0
        res = parity.compare(host, tab, self.delta, sub, divergence=div, top_k=self.args.top_k)
        return dict(sequences=int(len(rows)), near=res["near"], mismatch_outside=res["mismatch_outside"],
                    status_equal=res["status_equal"], nodes_tested=res.get("nodes_tested"),
                    qa_rel_max=res.get("qa_rel_max"), px_rel_max=res.get("px_rel_max"),
                    table_rows_equal=bool(np.array_equal(lib_rows, tab[need])), table_rows_compared=int(need.size))


def config_line(args, name, peak, run=None, steps=20, sample=16, flush=None):
    """One entry of the `configs` block: the named configuration at its flattened call size."""
    own = run is None
    if own:
        run = Run(args, name)
    B, N = run.B, run.N
    small = run.logit_gb < 0.2            # inputs smaller than L2: flush between calls
    ms_total, fused_ms = run.timed(steps, 3, flush=flush if small else None)
    ms = ms_total / steps
    acc = run.accounting(fused_ms, peak)
    line = {"workload": name, "sequences_per_call": B, "drafts_per_sequence": N, "V": run.V, "k": run.k,
            "delta": run.delta, "positions_drafted_per_s": B * N / (ms * 1e-3),
            "positions_tested_per_s": acc["method_nodes"] / (ms * 1e-3), "ms_per_call": ms, "kernel_ms": fused_ms,
            "algorithmic_bytes": acc["evaluated_bytes"], "GB_per_s": acc["achieved"], "frac_of_hbm_peak": acc["frac"],
            "method_bytes": acc["method_bytes"], "method_frac_of_hbm_peak": acc["method_frac"],
            "contexts": {"with_children": acc["contexts_with_children"], "evaluated": acc["contexts_evaluated"],
                         "on_accepted_paths": acc["method_contexts"]},
            "mean_accept_len": float(run.out.accept_len.float().mean().item()),
            "l2_policy": "L2 flushed between calls" if small else "inputs larger than L2",
            "neighbor_build_ms": run.build_ms, "D": run.cfg["D"]}
    if not args.greedy and sample:
        line["parity"] = run.parity_sample(sample)
    if own:
        del run
        lit_B = li_config(name)["B"]
        if lit_B != B and name != "tiny":
            # the configuration's literal call (one verification step of its batch), plain stream launches
            import lantern_inputs as li
            lit = Run(args, name, B=lit_B, seed=li.BASE_SEED + 5)
            t_warm, f_warm = lit.timed(100, 5)
            t_cold, _ = lit.timed(30, 3, flush=flush)
            line["literal_call"] = {"sequences_per_call": lit_B, "us_per_call_back_to_back": 1e3 * t_warm / 100,
                                    "us_per_call_l2_flushed": 1e3 * t_cold / 30, "fused_kernel_us": 1e3 * f_warm,
                                    "mean_accept_len": float(lit.out.accept_len.float().mean().item())}
            del lit
    return line


def li_config(name):
    import lantern_inputs as li
    return li.CONFIGS[WORKLOADS[name]["config"]]


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
    ap.add_argument("--no-configs", action="store_true",
                    help="leave out the per-configuration block (five named configurations, sampled oracle comparison)")
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

    # the all-cores oracle run starts its processes before the first GPU call (rank 0 of a single-GPU run only)
    cpu_all = None
    plain = args.divergence == "tvd" and args.top_k == 0 and not args.greedy and args.metric == "l2"
    if rank == 0 and world == 1 and not args.no_cpu_baseline and plain:
        try:
            rate, procs = oracle_all_cores(WORKLOADS[args.workload]["config"],
                                           nseq=48 if args.workload in ("batch_chain", "tiny") else 4)
            cpu_all = {"value": rate, "unit": UNIT, "cores": procs, "kind": "oracle",
                       "sample": "one process per core, each its own seeded sample of the workload, timed together"}
        except Exception as e:      # the single-core figure below still stands
            cpu_all = {"value": None, "error": repr(e)}

    import torch

    import lantern_inputs as li
    import paper_2410_03355_b200 as lt

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    lt.load_library()
    peak, peak_kind = load_peaks()

    run = Run(args, args.workload, B=args.batch or None, rank=rank)
    cfg, B, N, V, k, delta = run.cfg, run.B, run.N, run.V, run.k, run.delta
    d, out = run.d, run.out
    T_used, logit_gb, build_ms = run.T, run.logit_gb, run.build_ms

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    ms_total, fused_ms = run.timed(args.steps, args.warmup, dist)
    if dist is not None:
        dist.barrier()
    clocks = sampler.stop() if rank == 0 else None
    ms_total, fused_ms = max_over_ranks([ms_total, fused_ms], dist, "cuda")
    ms_per_step = ms_total / args.steps
    value = aggregate_rate(world, B, N, ms_per_step)
    acc = run.accounting(fused_ms, peak)

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
            run.step()
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
        import lantern_inputs.device as lid
        # the oracle reads its own neighbour rows, built for the sampled sequences outside the timed part
        n_s = min(B, 2048 if cfg["N"] <= 8 else 32)
        host_inp = lid.to_host(d, rows=np.arange(n_s))
        tab, _ = oracle_table_rows(run.cb_host, k, host_inp.draft_tokens, args.metric)
        rate, n_done, secs = oracle_sample_rate(host_inp, tab, delta, greedy=args.greedy,
                                                divergence=1 if args.divergence == "jsd" else 0, top_k=args.top_k)
        cpu = {"value": rate, "unit": UNIT, "cores": 1, "kind": "oracle",
               "sample": f"first {n_done} sequences ({n_done * N} drafted positions) of this call, {secs:.1f} s; "
                         f"neighbour rows built by the oracle beforehand",
               "all_cores": cpu_all}

    # ---- the five named configurations, each with a sampled oracle comparison (rank 0, N = 1) ----
    configs = None
    if rank == 0 and world == 1 and not args.no_configs and plain and args.workload == "batch_chain" and not args.batch:
        flush = torch.zeros(192 << 20, dtype=torch.uint8, device="cuda")       # larger than the 126 MB L2
        configs = {}
        chain = config_line(args, "batch_chain", peak, run=run, steps=20, sample=64)
        # the configuration's literal call (32 sequences x 7 drafts), one call per step, plain stream launches
        lit = Run(args, "batch_chain", B=cfg["B"], seed=li.BASE_SEED + 5)
        lit_total, lit_fused = lit.timed(200, 5)
        lit_cold, _ = lit.timed(50, 3, flush=flush)
        chain["literal_call"] = {"sequences_per_call": lit.B, "us_per_call_back_to_back": 1e3 * lit_total / 200,
                                 "us_per_call_l2_flushed": 1e3 * lit_cold / 50, "fused_kernel_us": 1e3 * lit_fused,
                                 "stream_operations_per_call": lt.verify_launch_count(False, False),
                                 "note": "back to back the 23 MB of rows stay in L2; flushed they come from HBM"}
        del lit
        # the same call under the paper's other settings (same inputs, same table): greedy decoding (tau = 0), the
        # top-k 1000 logit filter of the generation settings, the JSD bound
        variants = {}
        for vname, kw in (("greedy", dict(greedy=True)), ("top_k_1000", dict(top_k=1000)), ("jsd", dict(divergence="jsd"))):
            va = argparse.Namespace(**{**vars(args), **kw})
            vr = run.variant(va)
            v_total, v_fused = vr.timed(20, 3)
            v_acc = vr.accounting(v_fused, peak)
            variants[vname] = {"ms_per_call": v_total / 20, "kernel_ms": v_fused,
                               "positions_drafted_per_s": B * N / (v_total / 20 * 1e-3),
                               "contexts_evaluated": v_acc["contexts_evaluated"], "GB_per_s": v_acc["achieved"],
                               "frac_of_hbm_peak": v_acc["frac"],
                               "mean_accept_len": float(vr.out.accept_len.float().mean().item())}
            del vr
        chain["variants"] = variants
        configs["batch_chain"] = chain
        del run, d, out
        torch.cuda.empty_cache()
        for name in ("tiny", "single_image", "px512_tree", "stress"):
            configs[name] = config_line(args, name, peak, steps=20, sample=16 if name != "tiny" else 64, flush=flush)
            torch.cuda.empty_cache()
        # throughput mode of the stress trees: 16 of its steps (128 sequences each) flattened into one call
        flat = Run(args, "stress", B=16 * WORKLOADS["stress"]["B"], seed=li.BASE_SEED + 7)
        f_total, f_fused = flat.timed(10, 3)
        f_acc = flat.accounting(f_fused, peak)
        configs["stress"]["flattened_16_steps"] = {
            "sequences_per_call": flat.B, "ms_per_call": f_total / 10, "kernel_ms": f_fused,
            "positions_drafted_per_s": flat.B * flat.N / (f_total / 10 * 1e-3), "contexts": {
                "with_children": f_acc["contexts_with_children"], "evaluated": f_acc["contexts_evaluated"],
                "on_accepted_paths": f_acc["method_contexts"]},
            "GB_per_s": f_acc["achieved"], "frac_of_hbm_peak": f_acc["frac"], "method_frac_of_hbm_peak": f_acc["method_frac"]}
        del flat
        torch.cuda.empty_cache()
        del flush

    if rank == 0:
        top_active = 0 < args.top_k < V
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": args.workload, "note": WORKLOADS[args.workload]["note"], "sequences_per_call": B,
                       "drafts_per_sequence": N,
                       "V": V, "k": k, "delta": delta, "cfg_scale": cfg["cfg_scale"], "T": T_used,
                       "divergence": args.divergence, "metric": args.metric, "top_k": args.top_k,
                       "logits": "bf16" if cfg["dtype"] == li.BF16 else "f32", "rho": args.rho,
                       "l2_policy": "inputs larger than L2 (%.2f GB of logits per call)" % logit_gb,
                       "parallelism": "replicas" if world > 1 else "single"},
            "positions": {"drafted_per_s": value, "tested_per_s": world * acc["method_nodes"] / (ms_per_step * 1e-3),
                          "note": "drafted = every drafted position of the call; tested = the positions Algorithm 1's "
                                  "loop tests before its first rejection"},
            "roofline": {"bound": "hbm", "kernel": "lantern_greedy_context_kernel" if args.greedy else "lantern_context_kernel",
                         "achieved": acc["achieved"], "peak": peak, "peak_kind": f"of {peak_kind}", "unit": "GB/s",
                         "frac": acc["frac"],
                         "traffic": None if (args.greedy or args.divergence != "tvd" or top_active) else
                                    ncu_traffic(args.workload, acc["evaluated_bytes"]),
                         "algorithmic_bytes_per_launch": acc["evaluated_bytes"], "kernel_ms": fused_ms,
                         "contexts_with_children": acc["contexts_with_children"],
                         "contexts_evaluated": acc["contexts_evaluated"], "nodes_tested": acc["nodes_tested"],
                         "method_contexts": acc["method_contexts"], "method_bytes_per_launch": acc["method_bytes"],
                         "method_achieved": acc["method_achieved"], "method_frac": acc["method_frac"],
                         "note": "algorithmic bytes = rows of the contexts the kernel evaluated + neighbour rows of the "
                                 "nodes it tested; method_* counts only what Algorithm 1's loop reaches"},
            "cpu_baseline": cpu, "e2e": e2e,
            "gpu_launches": (lt.verify_launch_count(args.greedy, top_active) - 1) * args.steps, "clocks": clocks,
            "neighbor_build": {"ms": build_ms, "V": V, "D": cfg["D"], "k": k, "pairs_per_s": V * V / (build_ms * 1e-3)},
            "outputs": {"mean_accept_len": accept_mean, "sequences_with_status_bits": status_bad},
            "configs": configs,
        }
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
