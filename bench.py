#!/usr/bin/env python
"""Benchmark of the Mixture-of-Attentions drafter hot path on B200.

One "step" of this benchmark is one drafting cycle over one batch of synthetic input: LSA on the newly
accepted tokens + self-attention prefix append + D drafter forwards with tree expansion + the final
top-m cut + the tree-attention mask. The headline metric is draft-tree steps per second (D drafter
forwards per cycle); drafted tokens per second (m kept nodes per cycle) rides along.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload c2|c4|c5|c1]

Prints ONE JSON line. With --impl reference it times the CPU oracle (a deliberately plain program) on a
bounded sample of the same workload instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

CFG_KEYS = ("d_model", "n_stack", "d_stack", "vocab", "head_dim", "lsa_hq", "lsa_hkv", "lsa_mlp", "sa_hq", "sa_hkv",
            "sa_mlp", "ca_hq", "ca_hkv", "ca_mlp", "tree_topk", "tree_depth", "tree_keep", "rms_eps", "rope_theta",
            "dtype", "n_tli", "tli_hq", "tli_hkv", "tli_mlp")


def algorithmic_bytes(p) -> dict:
    """Bytes one steady-state draft step must move: every weight once, every cache entry once per sequence."""
    e = 4 if p.dtype == "f32" else 2
    dh, E = p.head_dim, p.d_model
    sa_w = (p.sa_hq + 2 * p.sa_hkv) * dh * E + E * p.sa_hq * dh + 3 * E * p.sa_mlp
    ca_w = p.ca_hq * dh * E + E * p.ca_hq * dh + 3 * E * p.ca_mlp
    lm = p.vocab * E
    caches = p.batch * p.ctx * 2 * (p.sa_hkv + p.ca_hkv) * dh
    # Target Layer Inference: each LLM decoder layer's weights and its cache, once per forward
    tli = p.n_tli * ((p.tli_hq + 2 * p.tli_hkv) * dh * E + E * p.tli_hq * dh + 3 * E * p.tli_mlp
                     + p.batch * p.ctx * 2 * p.tli_hkv * dh)
    lsa_w = ((p.lsa_hq + 2 * p.lsa_hkv) * dh * p.d_stack + p.d_stack * p.lsa_hq * dh + 3 * p.d_stack * p.lsa_mlp
             + 2 * p.ca_hkv * dh * p.d_stack)
    lsa_in = p.batch * p.lsa_tokens * p.n_stack * p.d_stack
    return dict(step=(sa_w + ca_w + lm + caches + tli) * e, lm_head=lm * e, lsa=(lsa_w + lsa_in) * e)


def lm_head_traffic(name: str):
    """dram__bytes_read.sum + dram__bytes_write.sum of one LM-head launch from the tracked ncu summary
    profiles/lm_head_traffic.json (which names the commit the counters were taken on), or None when there is no
    entry for this workload."""
    path = os.path.join(ROOT, "profiles", "lm_head_traffic.json")
    try:
        with open(path) as f:
            e = json.load(f).get(name)
        return None if e is None else int(e["dram_bytes_read"]) + int(e["dram_bytes_write"])
    except (OSError, ValueError, KeyError):
        return None


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples taken while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc = index, None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms",
                                          "100", "-i", str(self.index)], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unsampled"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
            except ValueError:
                continue
            for nme, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(nme)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unsampled"]}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons), "samples": len(sm)}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def measured_tensor_peak():
    """Sustained dense bf16 rate (the kernel is timed inside a long step), else the fallback."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["bf16_tflops_sustained"]), "measured (sustained)"
    return 1413.4, "fallback"


# ---------------------------------------------------------------------------------------------------
# the CPU oracle, timed on a bounded sample (cpu_baseline leg and --impl reference)
# ---------------------------------------------------------------------------------------------------
class OracleSampler:
    """The CPU oracle set up once on a workload (weights drawn and widened to fp64: set-up, like loading a
    checkpoint), then timed on bounded samples: `lsa_tok` LSA tokens and `rows` drafter forward rows per sample,
    scaled to one drafting cycle."""

    def __init__(self, p):
        import numpy as np
        import torch
        from oracle import moa_oracle as O
        from paper_2410_03804_b200 import synth
        self.p, self.np, self.synth = p, np, synth
        self.cores = torch.get_num_threads()
        w = synth.make_weights(p)
        w.update(synth.make_tli_weights(p))
        cfg = {k: p.as_dict()[k] for k in CFG_KEYS}
        self.dr = O.Drafter(cfg, {k: v.float().numpy() for k, v in w.items()})
        for name in w:
            self.dr.w(name)
        self.ctx = min(p.ctx, 2048)
        one = synth.scaled(p, batch=1)
        caK, caV = synth.make_cache(one, "ca", self.ctx)
        saK, saV = synth.make_cache(one, "sa", self.ctx)
        self.caches = [t[0].float().numpy().astype(np.float64) for t in (caK, caV, saK, saV)]
        self.tli = [tuple(t[0].float().numpy().astype(np.float64) for t in synth.make_tli_cache(one, l, self.ctx))
                    for l in range(p.n_tli)]

    def sample(self, rows: int = None, lsa_tok: int = None):
        """Times the cycle's whole LSA token set of one sequence and the forwards of its first two tree levels (1 + B
        rows) unless told otherwise, and scales to a cycle. Returns (cycle_seconds_estimate, cores, description)."""
        p, synth = self.p, self.synth
        rows = 1 + p.tree_topk if rows is None else rows
        lsa_tok = p.lsa_tokens if lsa_tok is None else lsa_tok
        caK, caV, saK, saV = self.caches
        h = synth.make_h_stack(p, lsa_tok).float().numpy()
        t0 = time.perf_counter()
        self.dr.lsa_forward(h)
        t_lsa = (time.perf_counter() - t0) / lsa_tok
        toks = synth.make_root(synth.scaled(p, batch=rows)).tolist()
        t0 = time.perf_counter()
        for t in toks:
            self.dr.forward_row(t, self.ctx, saK, saV, caK, caV, p.tree_topk, self.tli)
        t_row = (time.perf_counter() - t0) / rows
        n_rows = p.batch * (1 + p.tree_topk * (p.tree_depth - 1))
        cycle = p.batch * p.lsa_tokens * t_lsa + n_rows * t_row
        what = (f"timed: {lsa_tok} LSA token(s) ({t_lsa:.2f} s each) + {rows} drafter forward rows ({t_row:.2f} s each) of {p.name}"
                f" with {self.ctx}-entry caches; extrapolated to one cycle = {p.batch * p.lsa_tokens} LSA tokens + {n_rows} rows;"
                f" weights widened to fp64 beforehand")
        return cycle, self.cores, what


def oracle_sample(p, rows: int = None, lsa_tok: int = None):
    return OracleSampler(p).sample(rows, lsa_tok)


def run_reference(args, p):
    sampler = OracleSampler(p)                       # set-up is not timed
    t_all = []
    for _ in range(args.warmup + args.steps):
        cycle, cores, what = sampler.sample()     # one bounded sample per step: the LSA token set + two tree levels
        t_all.append(cycle)
    t = statistics.mean(t_all[args.warmup:]) if len(t_all) > args.warmup else t_all[-1]
    D, m = p.tree_depth, p.tree_keep
    val = D / t
    line = {"impl": "reference", "metric": "draft_tree_steps_per_sec", "value": val, "unit": "steps/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": t * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(p),
            "cpu_baseline": {"value": val, "unit": "steps/s", "cores": cores, "kind": "oracle", "sample": what,
                             "extrapolated": True},
            "e2e": {"value": val, "unit": "steps/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "drafted_tokens_per_sec": p.batch * m / t}
    print(json.dumps(line))


def workload_config(p):
    return {"workload": f"{p.name}: Llama-3-shaped MoA drafter, one drafting cycle = LSA on {p.lsa_tokens} tokens/seq + "
                        f"SA append + {p.tree_depth} drafter forwards (tree top-{p.tree_topk}, keep {p.tree_keep}) + mask",
            "tli": p.n_tli, "batch": p.batch, "context": p.ctx, "d_model": p.d_model, "vocab": p.vocab, "n_stack": p.n_stack,
            "l2": "inputs larger than L2 (weights streamed per step exceed 126 MB)" if p.name != "c1" else "L2-resident"}


# ---------------------------------------------------------------------------------------------------
# replicas: the path does not shard, so N GPUs run N independent copies of the same cycle
# ---------------------------------------------------------------------------------------------------
def replica_aggregate(ms_local: float, units_per_rank: float, device=None):
    """Whole-job numbers from one rank's device time for its timed region: the slowest rank's time (max over
    ranks, as every rank must finish) and the units all ranks processed per second. No data-path collective:
    this all-reduce of one float is measurement only. Works on any initialised process group (NCCL or gloo)."""
    import torch
    import torch.distributed as dist
    world = dist.get_world_size() if dist.is_available() and dist.is_initialized() else 1
    ms = float(ms_local)
    if world > 1:
        t = torch.tensor([ms], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())
    return ms, world * units_per_rank / (ms * 1e-3)


# ---------------------------------------------------------------------------------------------------
# config 3: LSA prefill throughput (a dense contraction: reported against the tensor-core roofline)
# ---------------------------------------------------------------------------------------------------
def run_lsa_prefill(args, p, dev, rank, world):
    import torch
    from paper_2410_03804_b200 import moa, synth
    n_tok = p.lsa_tokens
    small = synth.scaled(p, vocab=256)           # the LSA pass touches neither the embedding nor the LM head
    w = {k: v.to(dev) for k, v in synth.make_weights(small).items()}
    cfg = {k: small.as_dict()[k] for k in CFG_KEYS}
    g = moa.MoA(cfg, w, 1, n_tok, lsa_chunk_tokens=256)
    h_host = synth.make_h_stack(p, n_tok).pin_memory()
    h_dev = h_host.to(dev)
    h_stage = torch.empty_like(h_dev)
    kv_host = torch.empty((n_tok, p.d_stack), dtype=h_dev.dtype).pin_memory()

    def step(h):
        g.moa_state_set_len("ca", [0])
        return g.moa_lsa_forward(h, [n_tok], want_kv=True)

    def step_e2e():
        h_stage.copy_(h_host, non_blocking=True)
        kv_host.copy_(step(h_stage), non_blocking=True)

    def timed(fn, k):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        for _ in range(k):
            fn()
        b.record()
        torch.cuda.synchronize()
        return replica_aggregate(a.elapsed_time(b), 1.0, dev)[0]

    for _ in range(args.warmup):
        step(h_dev)
    sampler = ClockSampler(dev.index or 0)
    sampler.start()
    n0 = g.moa_launch_count()
    g.moa_profile_begin()
    ms = timed(lambda: step(h_dev), args.steps) / args.steps
    launches = g.moa_launch_count() - n0
    ph = g.moa_profile_phases()
    g.moa_profile_end()
    ms_e2e = timed(step_e2e, args.steps) / args.steps
    # the server-side message codec on the same activations: 8-bit quantisation of the whole prompt's rows
    flat = h_dev.reshape(-1, p.d_stack)
    qout = (torch.empty(flat.shape, dtype=torch.int8, device=dev), torch.empty((flat.shape[0],), dtype=torch.float32, device=dev))
    moa.moa_quantize_rows(flat, out=qout)
    ms_q = timed(lambda: moa.moa_quantize_rows(flat, out=qout), args.steps) / args.steps
    deq = torch.empty_like(flat)
    moa.moa_dequantize_rows(qout[0], qout[1], out=deq)
    ms_dq = timed(lambda: moa.moa_dequantize_rows(qout[0], qout[1], out=deq), args.steps) / args.steps
    q_bytes = flat.numel() * 3 + flat.shape[0] * 4          # bf16 in, int8 out, one scale per row
    hbm = measured_peaks()[0]
    del deq
    clocks = sampler.stop()
    assert g.moa_state_status() == 0
    if args.phases:
        sys.stderr.write("[phases, last pass of 256 tokens] " + " ".join(f"{k}:{u:.1f}({w_:.1f})" for k, u, w_ in ph) + "\n")
    S, D_, F, dh = p.n_stack, p.d_stack, p.lsa_mlp, p.head_dim
    qkv = (p.lsa_hq + 2 * p.lsa_hkv) * dh
    flops = n_tok * S * 2.0 * (D_ * qkv + p.lsa_hq * dh * D_ + 3 * D_ * F) + n_tok * p.lsa_hq * 4.0 * S * S * dh
    peak, kind = measured_tensor_peak()
    tf = flops / (ms * 1e-3) / 1e12
    gemm_us = sum(u for k, u, _w in ph if k == "gemm")
    line = {"metric": "lsa_prefill_tokens_per_sec", "value": world * n_tok / (ms * 1e-3), "unit": "tokens/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": f"c3: LSA prefill, {n_tok} tokens x {S} stacked activations x {D_}, {p.lsa_hq} heads x {dh}, "
                                   f"MLP {F}; one step = moa_lsa_forward over all tokens in passes of 256",
                       "l2": "inputs larger than L2 (2.2 GB of activations, 436 MB of weights)"},
            "e2e": {"value": world * n_tok / (ms_e2e * 1e-3), "unit": "tokens/s",
                    "h2d_bytes_per_step": h_host.numel() * 2, "d2h_bytes_per_step": kv_host.numel() * 2},
            "gpu_launches": launches, "clocks": clocks,
            "roofline": {"bound": "tensor", "kernel": "phase_machine_kernel<256> (the whole fused LSA pass)",
                         "achieved": tf, "peak": peak, "unit": "TFLOP/s", "frac": tf / peak, "peak_kind": f"of {kind}",
                         "traffic": None, "algorithmic_flops_per_step": flops,
                         "gemm_phase_share_of_last_pass": gemm_us / max(sum(u for _, u, _w in ph), 1e-9)},
            "codec": {"what": f"moa_quantize_rows / moa_dequantize_rows over the prompt's {flat.shape[0]} x {flat.shape[1]} "
                              "bf16 activation rows (the server's first message), timed on their own",
                      "quantize_ms": ms_q, "quantize_gbs": q_bytes / ms_q / 1e6, "quantize_frac_of_measured_hbm": q_bytes / ms_q / 1e6 / hbm,
                      "dequantize_ms": ms_dq, "dequantize_gbs": q_bytes / ms_dq / 1e6,
                      "dequantize_frac_of_measured_hbm": q_bytes / ms_dq / 1e6 / hbm,
                      "algorithmic_bytes": q_bytes},
            "replicas": "replicas only: no data-path collective" if world > 1 else None}
    if rank == 0:
        print(json.dumps(line))


# ---------------------------------------------------------------------------------------------------
# the CUDA path
# ---------------------------------------------------------------------------------------------------
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours")
    ap.add_argument("--workload", default="c2")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="launch every cycle on the stream instead of replaying a CUDA graph")
    ap.add_argument("--tli", type=int, default=0,
                    help="Target Layer Inference: run the last N Llama-shaped decoder layers in every forward (default 0, "
                         "the headline configuration)")
    ap.add_argument("--phases", action="store_true", help="with --workload c3: print per-phase times of the last dense LSA pass to stderr")
    ap.add_argument("--timeline", action="store_true",
                    help="stage-by-stage timeline of one drafting cycle (library variant built with -DMOA_TRACE: every kernel "
                         "stamps the GPU timer when its predecessor completes); prints a table instead of the bench line")
    args = ap.parse_args()
    if args.timeline:
        os.environ["MOA_TRACE_BUILD"] = "1"
    args.warmup = max(args.warmup, 3) if args.impl != "reference" else args.warmup

    from paper_2410_03804_b200 import synth
    p = synth.PRESETS[args.workload]
    if args.tli > 0:          # the LLM's own layer shape: the drafter's SA head layout, MLP 3.5 x E
        p = synth.scaled(p, n_tli=args.tli, tli_hq=p.sa_hq, tli_hkv=p.sa_hkv, tli_mlp=p.d_model * 7 // 2)
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        if rank == 0:
            run_reference(args, p)
        return

    import torch
    import torch.distributed as dist
    from paper_2410_03804_b200 import moa

    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl")
    dev = torch.device("cuda", local)
    if args.workload == "c3":
        run_lsa_prefill(args, p, dev, rank, world)
        if world > 1:
            dist.destroy_process_group()
        return
    # Replicas only: the path does not shard (one sequence batch per GPU, no data-path collective).
    w = {k: v.to(dev) for k, v in synth.make_weights(p).items()}
    w.update({k: v.to(dev) for k, v in synth.make_tli_weights(p).items()})
    cfg = {k: p.as_dict()[k] for k in CFG_KEYS}
    max_ctx = p.ctx + 64
    g = moa.MoA(cfg, w, p.batch, max_ctx, lsa_chunk_tokens=p.batch * p.lsa_tokens)
    caK, caV = synth.make_cache(p, "ca")
    saK, saV = synth.make_cache(p, "sa")
    g.fill_cache("ca", caK.to(dev), caV.to(dev))
    g.fill_cache("sa", saK.to(dev), saV.to(dev))
    for l in range(p.n_tli):
        tk, tv = synth.make_tli_cache(p, l)
        g.fill_tli_cache(l, tk.to(dev), tv.to(dev))
    del caK, caV, saK, saV
    nb, A, D, B, m = p.batch, p.lsa_tokens, p.tree_depth, p.tree_topk, p.tree_keep
    h_host = synth.make_h_stack(p, nb * A).pin_memory()
    tok_host = synth.make_tokens(p, A).reshape(-1).contiguous().pin_memory()
    root_host = synth.make_root(p).pin_memory()
    h_dev, tok_dev, root_dev = h_host.to(dev), tok_host.to(dev), root_host.to(dev)
    h_stage, tok_stage, root_stage = torch.empty_like(h_dev), torch.empty_like(tok_dev), torch.empty_like(root_dev)
    W = m + 1
    ids_buf = torch.empty((nb * B, B), dtype=torch.int32, device=dev)
    lp_buf = torch.empty((nb * B, B), dtype=torch.float32, device=dev)
    outs = (torch.empty((nb, W), dtype=torch.int32, device=dev), torch.empty((nb, W), dtype=torch.int32, device=dev),
            torch.empty((nb, W), dtype=torch.int32, device=dev), torch.empty((nb, W), dtype=torch.float32, device=dev),
            torch.empty((nb,), dtype=torch.int32, device=dev))
    host_out = [torch.empty_like(t, device="cpu").pin_memory() for t in outs]
    mask_host = torch.empty((nb, W, W), dtype=torch.uint8).pin_memory()
    lens = [p.ctx] * nb

    split_ev = []      # when filled by the caller: (before forwards, after forwards) event pairs of each cycle

    def cycle(h, tok, root, mark=False):
        g.moa_state_set_len("ca", lens)
        g.moa_state_set_len("sa", lens)
        g.moa_lsa_forward(h, [A] * nb, want_kv=False)
        g.moa_sa_append(tok, [A] * nb)
        g.moa_tree_begin(root)
        res = None
        if mark:
            split_ev.append((torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)))
            split_ev[-1][0].record()
        for s in range(D):
            R = nb if s == 0 else nb * B
            ids, lp, _ = g.moa_draft_step(out=(ids_buf[:R], lp_buf[:R], None))
            res = g.moa_tree_expand(ids, lp, out=outs)
        if mark:
            split_ev[-1][1].record()
        return moa.moa_tree_attn_mask(res[1])

    def cycle_e2e():
        h_stage.copy_(h_host, non_blocking=True)
        tok_stage.copy_(tok_host, non_blocking=True)
        root_stage.copy_(root_host, non_blocking=True)
        mask = cycle(h_stage, tok_stage, root_stage)
        for hst, d in zip(host_out, outs):
            hst.copy_(d, non_blocking=True)
        mask_host.copy_(mask, non_blocking=True)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, k):
        start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        start.record()
        for _ in range(k):
            fn()
        stop.record()
        barrier()
        ms, _ = replica_aggregate(start.elapsed_time(stop), 1.0, dev)
        return ms

    for _ in range(args.warmup):
        cycle(h_dev, tok_dev, root_dev)
        cycle_e2e()
    torch.cuda.synchronize()
    assert g.moa_state_status() == 0

    if args.timeline:
        # one warm cycle traced kernel by kernel, stream launches; a stage's cost = next stamp - its own stamp
        for _ in range(3):
            cycle(h_dev, tok_dev, root_dev)
        torch.cuda.synchronize()
        g.moa_trace_begin()
        cycle(h_dev, tok_dev, root_dev)
        cycle(h_dev, tok_dev, root_dev)          # its first stamp closes the last stage of the traced cycle
        tr = g.moa_trace_end()
        n_cycle = len(tr) // 2
        rows = [(k, grid, (tr[i + 1][2] - t) * 1e-3) for i, (k, grid, t) in enumerate(tr[:n_cycle])]
        kinds = [r[0] for r in rows]          # a drafter forward opens with: row norm, q/k/v product, rotary, attention
        first = [i for i in range(len(rows) - 3) if kinds[i:i + 4] == ["row_norm", "gemm", "rope", "attention"]]
        print(f"# stage timeline of one {p.name} drafting cycle ({n_cycle} kernels, {sum(r[2] for r in rows):.1f} us)")
        print("| # | kernel | grid.x | us |\n|---|---|---|---|")
        for i, (k, grid, us) in enumerate(rows):
            mark = " (forward %d starts)" % first.index(i) if i in first else ""
            print(f"| {i} | {k}{mark} | {grid} | {us:.1f} |")
        if len(first) >= 3:
            a, b = first[2], first[3] if len(first) > 3 else n_cycle
            print(f"# forward 2 (steady state, {b - a} kernels): {sum(r[2] for r in rows[a:b]):.1f} us")
            by = {}
            for k, _, us in rows[a:b]:
                by[k] = by.get(k, 0.0) + us
            print("# by kind: " + ", ".join(f"{k} {v:.1f}" for k, v in sorted(by.items(), key=lambda kv: -kv[1])))
        return

    # The cycle's launches are recorded once into CUDA graphs (one with device-resident inputs, one with the
    # host<->device copies of the end-to-end path) and replayed: the library only enqueues work on the caller's
    # stream, so a caller can capture it like any other stream work.
    use_graph = not args.no_graph
    n0 = g.moa_launch_count()
    if use_graph:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            cycle(h_dev, tok_dev, root_dev)
            cycle_e2e()
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        n0 = g.moa_launch_count()
        graph_dev, graph_e2e = torch.cuda.CUDAGraph(), torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph_dev):
            cycle(h_dev, tok_dev, root_dev)
        launches_per_cycle = g.moa_launch_count() - n0
        with torch.cuda.graph(graph_e2e):
            cycle_e2e()
        run_dev, run_e2e = graph_dev.replay, graph_e2e.replay
    else:
        cycle(h_dev, tok_dev, root_dev)
        launches_per_cycle = g.moa_launch_count() - n0
        run_dev, run_e2e = (lambda: cycle(h_dev, tok_dev, root_dev)), cycle_e2e
    for _ in range(3):
        run_dev()
        run_e2e()
    torch.cuda.synchronize()

    sampler = ClockSampler(local)
    sampler.start()
    ms = timed(run_dev, args.steps)
    ms_e2e = timed(run_e2e, args.steps)
    # the same block replayed ten more times with an event pair around every cycle: spread of the per-cycle time
    n_dist = max(10 * args.steps, 200)
    dist_ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_dist)]
    torch.cuda.synchronize()
    for a, b in dist_ev:
        a.record()
        run_dev()
        b.record()
    torch.cuda.synchronize()
    cyc = sorted(a.elapsed_time(b) for a, b in dist_ev)
    # the dominant kernel (LM head), bracketed by CUDA events on the launching stream: same cycles, launched on
    # the stream (events cannot be read inside a graph), directly after the timed replays
    g.moa_profile_begin()
    ms_stream = timed(lambda: cycle(h_dev, tok_dev, root_dev), args.steps)
    lm_ms, lm_n = g.moa_profile_end()
    # the D forwards alone (draft step + expansion), stream launches, events around them inside each cycle
    timed(lambda: cycle(h_dev, tok_dev, root_dev, mark=True), args.steps)
    fwd_us = statistics.mean(a.elapsed_time(b) for a, b in split_ev) * 1e3 / D
    # verification bookkeeping (moa_verify_greedy) on the last cycle's kept tree with seeded synthetic LLM logits:
    # timed on its own, not part of the step
    gen = torch.Generator(device=dev)
    gen.manual_seed(synth.SEED_BASE + 77)
    vz = torch.randn((nb, W, p.vocab), generator=gen, device=dev, dtype=torch.float32).to(p.torch_dtype)
    vout = moa.moa_verify_greedy(outs[0], outs[1], vz, D + 1)
    torch.cuda.synchronize()
    vgraph = torch.cuda.CUDAGraph()               # `steps` calls recorded once: the calls are shorter than a Python call
    with torch.cuda.graph(vgraph):
        for _ in range(args.steps):
            moa.moa_verify_greedy(outs[0], outs[1], vz, D + 1, out=vout)
    vgraph.replay()
    ms_verify = timed(vgraph.replay, 1) / args.steps
    vbytes = vz.numel() * vz.element_size()
    del vz
    # the whole-sequence drafter pass (moa_drafter_prefill) over min(context, 2048) tokens of one sequence,
    # every cached LLM position visible: timed on its own, not part of the step
    n_pre = min(p.ctx, 2048)
    pre_tok = synth.make_tokens(synth.scaled(p, batch=1), n_pre, tensor_index=44).reshape(-1).contiguous().to(dev)
    pre_out = torch.empty((n_pre, p.d_model), dtype=p.torch_dtype, device=dev)

    def prefill():
        g.moa_state_set_len("sa", [0] * nb)
        g.moa_drafter_prefill(pre_tok, [n_pre] + [0] * (nb - 1), out=pre_out)

    prefill()
    ms_prefill = timed(prefill, 3) / 3
    g.moa_state_set_len("sa", lens)
    assert g.moa_state_status() == 0
    dh = p.head_dim
    pre_flops = n_pre * 2.0 * ((p.sa_hq + 2 * p.sa_hkv) * dh * p.d_model + p.sa_hq * dh * p.d_model + 3 * p.d_model * p.sa_mlp
                               + 2 * p.ca_hq * dh * p.d_model + 3 * p.d_model * p.ca_mlp) \
        + 4.0 * dh * (p.sa_hq * n_pre * (n_pre + 1) / 2 + p.ca_hq * n_pre * p.ctx)
    clocks = sampler.stop()
    launches = launches_per_cycle * args.steps
    assert g.moa_state_status() == 0

    t_cycle = ms / args.steps / 1e3
    t_e2e = ms_e2e / args.steps / 1e3
    ab = algorithmic_bytes(p)
    peak, peak_kind = measured_peaks()
    lm_avg_s = lm_ms / max(lm_n, 1) / 1e3
    achieved = ab["lm_head"] / lm_avg_s / 1e9 if lm_n else None
    h2d = h_host.numel() * h_host.element_size() + tok_host.numel() * 4 + root_host.numel() * 4
    d2h = sum(t.numel() * t.element_size() for t in host_out) + mask_host.numel()
    roofline = {"bound": "hbm", "kernel": "lm_head", "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": (achieved / peak) if achieved else None, "peak_kind": f"of {peak_kind}",
                "traffic": lm_head_traffic(p.name),
                "launches_timed": lm_n, "avg_launch_us": lm_avg_s * 1e6,
                "timed_over": "the same cycles launched on the stream right after the timed replays",
                "algorithmic_bytes_per_launch": ab["lm_head"]}
    if nb * B > 128 and lm_n:
        # More than 128 rows per forward: activations enter as two bf16 terms multiplied one after the other (4 R E V flop per
        # launch), and the launch is bound by the tensor cores, not by the weight stream. Mean over a cycle's D launches
        # (the first has nb rows, the others nb * B).
        flops = 4.0 * p.d_model * p.vocab * (nb + (D - 1) * nb * B) / D
        tpeak, tkind = measured_tensor_peak()
        tf = flops / lm_avg_s / 1e12
        roofline = {"bound": "tensor", "kernel": "lm_head", "achieved": tf, "peak": tpeak, "unit": "TFLOP/s", "frac": tf / tpeak,
                    "peak_kind": f"of {tkind}", "traffic": lm_head_traffic(p.name), "launches_timed": lm_n,
                    "avg_launch_us": lm_avg_s * 1e6, "timed_over": roofline["timed_over"],
                    "algorithmic_flops_per_launch": flops,
                    "hbm_view": {"achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                                 "algorithmic_bytes_per_launch": ab["lm_head"]}}
    line = {
        "metric": "draft_tree_steps_per_sec", "value": world * D / t_cycle, "unit": "steps/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": t_cycle * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": p.dtype, "data": "synthetic",
        "config": workload_config(p),
        "drafted_tokens_per_sec": world * nb * m / t_cycle,
        "e2e": {"value": world * D / t_e2e, "unit": "steps/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": launches,
        "launch_mode": "cuda graph replay of one recorded cycle" if use_graph else "stream launches",
        "ms_per_step_stream_launches": ms_stream / args.steps,
        "cycle_ms_distribution": {"n": n_dist, "median": cyc[n_dist // 2], "p10": cyc[n_dist // 10], "p90": cyc[(9 * n_dist) // 10],
                                  "what": "every cycle between its own event pair, same launch mode, right after the timed block"},
        "clocks": clocks,
        "roofline": roofline,
        "cycle_roofline": {"algorithmic_bytes_per_cycle": D * ab["step"] + ab["lsa"],
                           "achieved_gbs": (D * ab["step"] + ab["lsa"]) / t_cycle / 1e9,
                           "frac_of_measured": (D * ab["step"] + ab["lsa"]) / t_cycle / 1e9 / peak,
                           "frac_of_8tbs": (D * ab["step"] + ab["lsa"]) / t_cycle / 1e9 / 8000.0},
        "forward_roofline": {"what": "one drafter forward + tree expansion, mean over the cycle's forwards, stream launches",
                             "us": fwd_us, "algorithmic_bytes": ab["step"], "achieved_gbs": ab["step"] / fwd_us / 1e3,
                             "frac_of_measured": ab["step"] / fwd_us / 1e3 / peak,
                             "frac_of_8tbs": ab["step"] / fwd_us / 1e3 / 8000.0},
        "verify": {"what": f"moa_verify_greedy on [{nb}, {W}, {p.vocab}] {p.dtype} logits (arg-max + accepted-path walk), "
                           "back-to-back calls replayed from a CUDA graph, not part of the step",
                   "us": ms_verify * 1e3, "bytes": vbytes, "achieved_gbs": vbytes / ms_verify / 1e6,
                   "frac_of_measured": vbytes / ms_verify / 1e6 / peak,
                   "l2": "logits larger than L2" if vbytes > 126e6 else "logits fit in L2: not an HBM figure"},
        "prefill": {"what": f"moa_drafter_prefill over {n_pre} tokens of one sequence (causal SA, CA over {p.ctx} cached positions), "
                            "chunks of 256 rows, timed on its own",
                    "ms": ms_prefill, "tokens_per_sec": n_pre / ms_prefill * 1e3, "algorithmic_flops": pre_flops,
                    "tflops": pre_flops / ms_prefill / 1e9},
        "replicas": "replicas only: no data-path collective" if world > 1 else None,
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cyc, cores, what = oracle_sample(p)
        line["cpu_baseline"] = {"value": D / cyc, "unit": "steps/s", "cores": cores, "kind": "oracle", "sample": what,
                                "extrapolated": True}
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
