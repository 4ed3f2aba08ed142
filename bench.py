#!/usr/bin/env python
"""Benchmark of the verify step (64 layers of shared-prefix paged GQA attention + one
accept/resample pass) on the Qwen2.5-32B-shaped workload: N=16 branches, gamma=3, prefix 512,
4096 private tokens per branch, vocab 152064.  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config 32b|3b|tiny]

* value   = unique KV bytes + accept probability bytes of one step / device time of the step (GB/s),
            inputs resident in HBM; us_per_layer is reported beside it.
* e2e     = same bytes / time of tts_verify_step_host (pinned host q/out/probabilities copied inside
            the timed region; the KV cache is device-resident state).
* roofline= the attention main kernel: unique KV bytes of one layer / its CUDA-event duration,
            against the measured copy bandwidth of MEASURED_PEAKS.json.
* cpu_baseline = the CPU oracle timed on a bounded sample (whole layers + the accept pass).
With --gpus N > 1 (under torchrun) every rank runs an independent replica of the step (the path
has no exchange step); value sums the ranks' bytes over the slowest rank's time.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import time
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

import tts_inputs as ti  # noqa: E402

METRIC = "verify-step µs/layer and KV HBM GB/s vs peak at N branches × (γ+1) tokens"
FALLBACK_HBM_GBS = 6650.0


def measured_peaks():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        d = json.loads(p.read_text())
        return float(d["hbm_gbs"]), "measured"
    return FALLBACK_HBM_GBS, "fallback"


def accept_algorithmic_bytes(acc_len: np.ndarray, gamma: int, vocab: int) -> int:
    """Per branch: 2*gamma scalar gathers + one sweep of (p_k, q_k) after a rejection or of
    p_gamma after full acceptance."""
    rej = int((acc_len < gamma).sum())
    full = int((acc_len >= gamma).sum())
    return rej * 2 * vocab * 4 + full * vocab * 4 + len(acc_len) * gamma * 8


class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.idx = device_index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.idx)], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
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
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "reasons": sorted(reasons),
                "samples": len(sm)}


def oracle_sample(shape: ti.AttnShape, seed: int, budget_s: float = 12.0):
    """Times the CPU oracle on whole layers of the workload (as many passes over one generated
    layer as fit the budget, at most n_layers) plus one accept pass.
    Returns (bytes processed, seconds, description, cores)."""
    import oracle
    cores = oracle.n_cores()
    oracle.build()
    bytes_done, secs, layers = 0, 0.0, 0
    case = ti.make_attn_case(shape, seed)
    while layers < shape.n_layers:
        t0 = time.perf_counter()
        oracle.verify_attn(case.q, case.k_pages, case.v_pages, case.block_table, case.prefix_len,
                           case.branch_lens, shape.gamma)
        dt = time.perf_counter() - t0
        secs += dt; layers += 1; bytes_done += shape.unique_kv_bytes()
        if secs + dt > budget_s:
            break
    acc_case = ti.make_accept_case(shape.n_branches, shape.gamma, shape.vocab, shape.logit_sigma, seed + 2)
    t0 = time.perf_counter()
    acc, _, _ = oracle.accept(acc_case.p_target, acc_case.q_draft, acc_case.draft_tokens, acc_case.uniforms)
    secs += time.perf_counter() - t0
    bytes_done += accept_algorithmic_bytes(acc, shape.gamma, shape.vocab)
    return bytes_done, secs, f"{layers} of {shape.n_layers} layers of attention + 1 accept pass", cores


def run_reference(args, shape):
    """The CPU oracle as the reference arm: each step = one layer of attention + the accept pass."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    oracle.build()
    cores = oracle.n_cores()
    case = ti.make_attn_case(shape, 0x5EED + 2)
    acc_case = ti.make_accept_case(shape.n_branches, shape.gamma, shape.vocab, shape.logit_sigma, 0x5EED + 4)

    def step():
        oracle.verify_attn(case.q, case.k_pages, case.v_pages, case.block_table, case.prefix_len,
                           case.branch_lens, shape.gamma)
        a, _, _ = oracle.accept(acc_case.p_target, acc_case.q_draft, acc_case.draft_tokens, acc_case.uniforms)
        return a
    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        acc = step()
    dt = (time.perf_counter() - t0) / args.steps
    nbytes = shape.unique_kv_bytes() + accept_algorithmic_bytes(acc, shape.gamma, shape.vocab)
    gbs = nbytes / dt / 1e9
    sample = "1 layer of attention + 1 accept pass per step (of %d layers)" % shape.n_layers
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": gbs, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "us_per_layer": dt * 1e6,
        "config": {"workload": workload_name(shape), "sample": sample},
        "cpu_baseline": {"value": gbs, "unit": "GB/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": gbs, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }, ensure_ascii=False))


def workload_name(shape):
    return (f"{shape.name}-shaped: {shape.n_layers} layers, Hq={shape.n_q_heads}, Hkv={shape.n_kv_heads}, D=128, "
            f"prefix {shape.prefix_len} + {shape.n_branches} branches x {shape.private_len} private tokens, "
            f"gamma={shape.gamma}, page 16 (random permutation), vocab {shape.vocab}")


def aggregate_over_ranks(ms: float, e2e_ms: float, launches: int, world: int, device):
    """Replicas only: every rank runs the same step on its own data, so the job's time is the
    slowest rank's (MAX) and its launch count the sum; the bytes are summed by the caller as
    world x bytes of one replica.  Needs an initialised process group when world > 1."""
    if world <= 1:
        return ms, e2e_ms, launches
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms, e2e_ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    lt = torch.tensor([launches], device=device, dtype=torch.int64)
    dist.all_reduce(lt)
    return float(t[0]), float(t[1]), int(lt[0])


def run_ours(args, shape):
    import torch
    import torch.distributed as dist
    import paper_2505_19634_b200 as tts

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.device("cuda", local)

    L, N, g, V = shape.n_layers, shape.n_branches, shape.gamma, shape.vocab
    R = g + 1
    seed = 0x5EED + 2 + 7919 * rank
    bt_np, num_pages, max_blocks = ti.make_block_table(shape, seed)
    lens_np = shape.lens()
    gen = torch.Generator(device=dev); gen.manual_seed(seed)
    # K/V pools: one per layer, N(0,1) bf16 drawn on the device (Philox); q likewise
    k_pools = [torch.randn(num_pages, shape.n_kv_heads, 16, 128, device=dev, dtype=torch.bfloat16, generator=gen)
               for _ in range(L)]
    v_pools = [torch.randn(num_pages, shape.n_kv_heads, 16, 128, device=dev, dtype=torch.bfloat16, generator=gen)
               for _ in range(L)]
    q_all = torch.randn(L, N, R, shape.n_q_heads, 128, device=dev, dtype=torch.bfloat16, generator=gen)
    out_all = torch.empty_like(q_all)
    bt, lens = torch.from_numpy(bt_np).to(dev), torch.from_numpy(lens_np).to(dev)
    acc_case = ti.make_accept_case(N, g, V, shape.logit_sigma, seed + 2)
    p_t, q_d = torch.from_numpy(acc_case.p_target).to(dev), torch.from_numpy(acc_case.q_draft).to(dev)
    toks, unis = torch.from_numpy(acc_case.draft_tokens).to(dev), torch.from_numpy(acc_case.uniforms).to(dev)
    acc_len = torch.zeros(N, dtype=torch.int32, device=dev)
    nxt = torch.zeros(N, dtype=torch.int32, device=dev)

    stream = torch.cuda.Stream(device=dev)      # a side stream: graph capture needs one
    torch.cuda.set_stream(stream)
    ctx = tts.TtsContext(shape.n_q_heads, shape.n_kv_heads, N, R, max_blocks, num_pages, stream=stream)

    def step():
        for l in range(L):
            ctx.tts_verify_attn(q_all[l], k_pools[l], v_pools[l], bt, shape.prefix_len, lens, N, g,
                                tts.MASK_CAUSAL, out_all[l])
        ctx.tts_accept(p_t, q_d, toks, unis, N, g, V, acc_len, nxt)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    # The library's calls of one step (64 x attention + accept) are captured once into a CUDA graph and
    # the timed steps replay it: the same kernels on the same arguments, without the per-launch gaps.
    graph, run_step, launches_per_step = None, step, None
    if not args.no_graph:
        n0 = ctx.tts_launch_count()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            step()
        launches_per_step = ctx.tts_launch_count() - n0
        run_step = graph.replay
        for _ in range(3):
            run_step()
        barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    launches0 = ctx.tts_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record(stream)
    for _ in range(args.steps):
        run_step()
    e1.record(stream)
    barrier()
    ms = e0.elapsed_time(e1) / args.steps
    launches = launches_per_step * args.steps if graph is not None else ctx.tts_launch_count() - launches0
    status = ctx.tts_last_status()
    if status != 0:
        raise SystemExit(f"device status {status} after the timed region")

    # dominant kernel alone: the attention main kernel, event-timed per launch over K more steps
    ctx.tts_profile_enable(True)
    for _ in range(min(args.steps, 4096 // L)):
        step()
    main_us, merge_us, prof_calls = ctx.tts_profile_read()
    ctx.tts_profile_enable(False)
    clocks = sampler.stop() if rank == 0 else None

    acc_host = acc_len.cpu().numpy()
    step_bytes = shape.unique_kv_bytes() * L + accept_algorithmic_bytes(acc_host, g, V)

    # ---- end to end through the host entry point ----
    q_host = torch.empty(q_all.shape, dtype=torch.bfloat16, pin_memory=True); q_host.copy_(q_all)
    out_host = torch.empty(q_all.shape, dtype=torch.bfloat16, pin_memory=True)
    pin = lambda a: torch.from_numpy(a).pin_memory()
    h_bt, h_lens = pin(bt_np), pin(lens_np)
    h_p, h_q, h_t, h_u = pin(acc_case.p_target), pin(acc_case.q_draft), pin(acc_case.draft_tokens), pin(acc_case.uniforms)
    h_al = torch.zeros(N, dtype=torch.int32).pin_memory(); h_nt = torch.zeros(N, dtype=torch.int32).pin_memory()

    def step_host():
        ctx.tts_verify_step_host(L, q_host, k_pools, v_pools, h_bt, shape.prefix_len, h_lens, N, g, h_p, h_q, h_t,
                                 h_u, V, out_host, h_al, h_nt)
    e2e_steps = max(2, min(args.steps, 5))
    for _ in range(2):
        step_host()
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        step_host()
    torch.cuda.synchronize()
    e2e_ms = (time.perf_counter() - t0) / e2e_steps * 1e3
    h2d = (q_host.numel() * 2 + h_bt.numel() * 4 + h_lens.numel() * 4 + h_p.numel() * 4 + h_q.numel() * 4 +
           h_t.numel() * 4 + h_u.numel() * 4)
    d2h = out_host.numel() * 2 + 8 * N

    ms, e2e_ms, launches = aggregate_over_ranks(ms, e2e_ms, launches, world, dev)

    if rank == 0:
        peak, peak_kind = measured_peaks()
        total_bytes = step_bytes * world
        value = total_bytes / (ms * 1e-3) / 1e9
        layer_bytes = shape.unique_kv_bytes()
        # DRAM read + write bytes of one launch of the dominant kernel, from the ncu capture summarised in
        # profiles/attn_umma_t_kernel_32b_2layers.md (valid for the 32b workload and this kernel version only)
        traffic = 276.4e6 if shape.name == "32b" else None
        roof = {"bound": "hbm", "achieved": None, "peak": peak, "unit": "GB/s", "frac": None, "traffic": traffic,
                "peak_kind": f"of {peak_kind}", "kernel": "attn_umma_t_kernel (token-major tcgen05 attention, one layer per launch)"}
        if main_us:
            roof["achieved"] = layer_bytes / (main_us * 1e-6) / 1e9
            roof["frac"] = roof["achieved"] / peak
            roof["kernel_us"] = main_us
            roof["merge_kernel_us"] = merge_us
            roof["launches_timed"] = prof_calls
        cb_bytes, cb_s, cb_sample, cores = oracle_sample(shape, 0x5EED + 2)
        rec = {
            "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "us_per_layer": ms * 1e3 / L,
            "frac_of_hbm_peak": value / world / peak,
            "config": {"workload": workload_name(shape), "l2": "inputs larger than L2: %.2f GiB of KV per step, one K/V pool per layer (for a one-layer "
                             "config: that many independent copies of the layer)" % (layer_bytes * L / 2**30), "bytes_per_step": step_bytes,
                       "launch": "one CUDA graph replay per step" if graph is not None else "stream launches",
                       "attn_impl": "auto"},
            "clocks": clocks,
            "e2e": {"value": total_bytes / (e2e_ms * 1e-3) / 1e9, "unit": "GB/s", "ms_per_step": e2e_ms,
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
            "gpu_launches": launches,
            "roofline": roof,
            "cpu_baseline": {"value": cb_bytes / cb_s / 1e9, "unit": "GB/s", "cores": cores, "kind": "oracle",
                             "sample": cb_sample, "seconds": cb_s},
        }
        print(json.dumps(rec, ensure_ascii=False))
    ctx.close()
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="32b", choices=list(ti.CONFIGS))
    ap.add_argument("--no-graph", action="store_true", help="time plain stream launches instead of a CUDA graph replay")
    ap.add_argument("--layers", type=int, default=0,
                    help="run only this many layers of the config (small cases for profiler captures; "
                         "the workload name says so)")
    args = ap.parse_args()
    shape = ti.CONFIGS[args.config]
    if args.layers > 0:
        shape = ti.with_branches(shape, n_layers=args.layers)
    elif shape.n_layers == 1:
        # a one-layer config fits L2 (126 MB): time a rotation over enough independent copies of the
        # layer (own K/V/Q each) that the working set exceeds twice the L2
        shape = ti.with_branches(shape, n_layers=-(-2 * 132_000_000 // shape.unique_kv_bytes()))
    if args.impl == "reference":
        run_reference(args, shape)
    else:
        run_ours(args, shape)


if __name__ == "__main__":
    main()
