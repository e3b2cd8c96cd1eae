#!/usr/bin/env python
"""Benchmark of the VADUSA tree draft-and-verify step on B200.

One step = one speculative iteration (draft -> verify -> accept+commit) of the
VALL-E-like 12-layer, d-1024, 64-node-tree workload (batch 1, bf16, tolerance 3,
temperature 1.0), synthetic prefix and random-init weights.  Prints one JSON
line: generated speech tokens/s (whole job), ms per step (= verify-iteration
latency), a roofline object for the dominant kernel, the CPU oracle timed on a
bounded sample, and an end-to-end number through the host-buffer entry point.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

With N > 1 (under torchrun) every rank runs its own replica of the workload with
its own seed (sequences are independent; no collective on the data path).
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
sys.path.insert(0, ROOT)

WORKLOAD = "C2"


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return float(p["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.lines = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.gpu)], stdout=subprocess.PIPE, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def _setup_inputs(rank: int):
    import workloads as W
    wl = W.workload(WORKLOAD)
    weights = W.make_weights(wl.shape, wl.seed())
    tpl = W.static_template(wl.tree_nodes, wl.tree_caps)
    # every replica decodes its own sequence: item index = rank
    ph = W.phonemes(wl.phoneme_len[0], wl.shape.n_phonemes, wl.seed(rank))
    pr = W.markov_prompt(wl.prompt_len, wl.shape.vocab - 1, wl.seed(rank))
    prefix = np.concatenate([ph.astype(np.int32) + wl.shape.vocab, pr.astype(np.int32)])
    return wl, weights, tpl, ph, pr, prefix


# ------------------------------------------------------------------------------ oracle arm
def _oracle_run(wl, weights, tpl, ph, pr, steps: int, warmup: int, budget_s: float):
    """Times `steps` iterations of the oracle as it stands.  The defining mode
    (one pass per branch) is used when it fits the time budget, else the oracle's
    own cheaper modes with the same arithmetic."""
    import oracle as O
    model = O.Model.from_shape(wl.shape, weights)
    st = O.prefill_blocked(model, ph, pr, seq=0)
    sp = O.Sampling(tau=wl.tau, temperature=wl.temperature, top_p=wl.top_p, seed=wl.seed())
    t0 = time.perf_counter()
    O.vadusa_iteration(model, st, tpl, sp, mode="tree")
    t_tree = time.perf_counter() - t0
    total = steps + warmup
    branch_cost = t_tree * sum(len(tpl.node_path(l)) for l in tpl.leaves()) / 4.0     # rough: passes of one token each
    mode = "branch" if branch_cost * total < budget_s else ("memo" if branch_cost * total * 0.45 < budget_s else "tree")
    for _ in range(warmup):
        O.vadusa_iteration(model, st, tpl, sp, mode=mode)
    tokens = 0
    t0 = time.perf_counter()
    for _ in range(steps):
        tokens += O.vadusa_iteration(model, st, tpl, sp, mode=mode).accept_len
    dt = time.perf_counter() - t0
    what = {"branch": "one sequential causal pass per root-to-leaf branch (defining mode)",
            "memo": "one token pass per tree node after its ancestors' stored K/V (same arithmetic)",
            "tree": "one tree-masked pass over all nodes (same arithmetic)"}[mode]
    return tokens / dt, dt / steps * 1e3, f"{steps} iterations of {WORKLOAD} after its 325-token prefill; {what}", tokens


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl, weights, tpl, ph, pr, _ = _setup_inputs(0)
    cores = os.cpu_count() or 1
    val, ms, sample, _ = _oracle_run(wl, weights, tpl, ph, pr, args.steps, args.warmup, budget_s=200.0)
    line = {"impl": "reference", "metric": "generated speech tokens/s", "value": val, "unit": "tokens/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"{WORKLOAD}: 12L d1024 16H FFN4096 vocab1025, batch 1, 64-node tree, tau 3, T 1.0"},
            "cpu_baseline": {"value": val, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ------------------------------------------------------------------------------ our arm
def run_ours(args):
    import torch
    import torch.distributed as dist
    import workloads as W
    import paper_2410_21951_b200 as P

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    wl, weights, tpl, ph, pr, prefix = _setup_inputs(rank)
    K, Wm = args.steps, max(args.warmup, 3)
    max_depth = tpl.max_depth + 1
    # pages: prefix + all iterations at the longest acceptance + the tree behind the context
    gen_cap = wl.gen_tokens
    need = len(prefix) + (K + Wm + 64) * max_depth + wl.tree_nodes + gen_cap + 64
    need = min(need, wl.shape.max_pos - 1)
    table, total = W.shuffled_block_table([need], 64, wl.seed(77 + rank), spare_pages=2)
    g = P.Vadusa(wl.shape, weights, max_batch=1, max_tree_nodes=wl.tree_nodes, max_blocks_per_seq=table.shape[1],
                 kv_num_blocks=total, device=local)
    g.set_tree(tpl.parent, tpl.rank)
    sp = P.Sampling.make(tau=wl.tau, temperature=wl.temperature, top_p=wl.top_p, seed=wl.seed())
    bt = torch.from_numpy(table).to(g.dev)

    def fresh():
        g.begin(bt)
        g.prefill(prefix[None, :].copy(), [len(prefix)])

    def steps(n):
        for _ in range(n):
            g.draft(sp)
            g.verify_step()
            g.accept_and_commit(sp)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    # everything below is enqueued on the library's own stream (events are recorded there)
    torch.cuda.set_stream(g.stream)

    # ---- device-resident timing: K iterations, inputs (weights 321 MB + KV) larger than L2
    fresh()
    steps(Wm)
    len0 = int(g.lengths()[0])
    launches0 = g.kernel_launches()
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.3)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    steps(K)
    e1.record()
    barrier()
    ms = e0.elapsed_time(e1)
    clocks = sampler.stop()
    launches = g.kernel_launches() - launches0
    tokens = int(g.lengths()[0]) - len0
    g.check()

    # ---- per-kernel times of the same steps (events around every launch; separate pass)
    n_prof = min(K, 50)
    g.profile_begin()
    steps(n_prof)
    prof = g.profile_end()

    # ---- end to end through the host-buffer entry: prefix from host memory, tokens back to host
    h_out = np.zeros((1, gen_cap), dtype=np.int32)
    h_len = np.zeros(1, dtype=np.int32)
    h_prefix = torch.from_numpy(prefix[None, :].copy()).pin_memory().numpy()
    lens = np.array([len(prefix)], dtype=np.int32)
    g.generate_host(sp, bt, h_prefix, lens, 32, h_out[:, :32].copy(), h_len)          # warm
    barrier()
    t0 = time.perf_counter()
    st = g.generate_host(sp, bt, h_prefix, lens, gen_cap, h_out, h_len)
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    e2e_tokens = int(h_len[0])
    e2e_iters = max(int(st.iterations), 1)

    # ---- aggregate over ranks
    if world > 1:
        t = torch.tensor([ms, e2e_s], device=g.dev, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        c = torch.tensor([tokens, e2e_tokens, launches], device=g.dev, dtype=torch.float64)
        dist.all_reduce(c, op=dist.ReduceOp.SUM)
        ms, e2e_s = float(t[0]), float(t[1])
        tokens, e2e_tokens, launches = int(c[0]), int(c[1]), int(c[2])

    if rank == 0:
        peak, peak_kind = _peaks()
        sh = wl.shape
        es = 2
        d, f, vp = sh.d_model, sh.d_ffn, (sh.vocab + 127) // 128 * 128
        # algorithmic bytes of the weight-streaming matrix products of one iteration (weights only)
        gemm_bytes = {"gemm_qkv": 3 * d * d * es, "gemm_out": d * d * es, "gemm_ffn1": d * f * es,
                      "gemm_ffn2": d * f * es, "gemm_lm": vp * d * es}
        tot_ms = sum(v[1] for v in prof.values())
        gemm_ms = sum(prof[k][1] for k in gemm_bytes if k in prof)
        gemm_alg = sum(gemm_bytes[k] * prof[k][0] for k in gemm_bytes if k in prof)
        achieved = gemm_alg / (gemm_ms * 1e-3) / 1e9 if gemm_ms > 0 else 0.0
        shares = {k: round(v[1] / tot_ms, 4) for k, v in sorted(prof.items(), key=lambda kv: -kv[1][1])}
        cores = os.cpu_count() or 1
        cpu_val, _, cpu_sample, _ = _oracle_run(wl, weights, tpl, ph, pr, steps=2, warmup=0, budget_s=30.0)
        line = {
            "metric": "generated speech tokens/s", "value": tokens / (ms * 1e-3), "unit": "tokens/s",
            "n_gpus": world, "steps": K, "warmup": Wm, "ms_per_step": ms / K, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": f"{WORKLOAD}: 12L d1024 16H FFN4096 vocab1025 bf16, batch 1 per GPU, 64-node tree "
                                   f"(top-10/5/3/2), tau 3, T 1.0, 325-token prefix, random-init weights",
                       "step": "one draft+verify+accept/commit iteration", "mean_accepted_tokens": tokens / (K * world),
                       "l2": "inputs larger than L2 (321 MB of weights streamed per step)",
                       "verify_step_us": ms / K * 1e3},
            "roofline": {"bound": "hbm", "kernel": "projection GEMMs (qkv, out, ffn1, ffn2, lm head)",
                         "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "peak_source": f"{peak_kind} copy bandwidth", "traffic": None,
                         "kernel_time_shares": shares, "profiled_steps": n_prof,
                         "kernel_avg_us_with_event_overhead": {k: round(v[1] / v[0] * 1e3, 2) for k, v in prof.items()}},
            "cpu_baseline": {"value": cpu_val, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": cpu_sample},
            "e2e": {"value": e2e_tokens / e2e_s, "unit": "tokens/s",
                    "h2d_bytes_per_step": len(prefix) * 4 / e2e_iters, "d2h_bytes_per_step": (gen_cap + 1) * 4 / e2e_iters,
                    "what": f"vadusa_generate_host: prefix from pinned host memory, prefill, {gen_cap} tokens, tokens back to host"},
            "gpu_launches": launches, "clocks": clocks,
        }
        print(json.dumps(line))
    g.close()
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    args = ap.parse_args()
    if args.steps is None:
        args.steps = 20 if args.impl == "reference" else 400
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
