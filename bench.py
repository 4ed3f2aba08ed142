#!/usr/bin/env python
"""Benchmark of the verify step (64 layers of shared-prefix paged GQA attention + one
accept/resample pass) on the Qwen2.5-32B-shaped workload: N=16 branches, gamma=3, prefix 512,
4096 private tokens per branch, vocab 152064.  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                  [--config 32b|3b|tiny|tree|sweep|multireq]

* value   = unique KV bytes + accept probability bytes of one step / device time of the step (GB/s),
            inputs resident in HBM; us_per_layer is reported beside it.  A step is: one schedule
            (tts_attn_plan), one attention call per layer, one accept pass; the timed steps replay one
            CUDA graph of exactly those calls.
* e2e     = same bytes / time of tts_verify_step_host (pinned host q/out/probabilities copied inside
            the timed region; the KV cache is device-resident state).
* roofline= the attention main kernel: unique KV bytes of one layer / the time per layer of a graph of
            the attention calls alone (an upper bound for the kernel's duration, in the launch mode of the
            timed steps), against the measured copy bandwidth of MEASURED_PEAKS.json; for --config tree
            the flops against the measured bf16 GEMM rate.
* cpu_baseline = the CPU oracle timed on a bounded sample (whole layers + the accept pass).
--config sweep runs the branch / draft-length sweep (N x gamma x 3 seeds, ragged lengths), checks every
point against the oracle and prints a table before the JSON line.
With --gpus N > 1 (under torchrun) every rank runs an independent replica of the step (the path
has no exchange step); value sums the ranks' bytes over the slowest rank's time.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import subprocess
import sys
import time
from dataclasses import replace
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

import tts_inputs as ti  # noqa: E402

METRIC = "verify-step µs/layer and KV HBM GB/s vs peak at N branches × (γ+1) tokens"
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1400.0          # sustained
NOMINAL_HBM_GBS = 8000.0               # the nominal HBM3e figure the 70 % target is also quoted against
L2_BYTES = 132_000_000

TREE = ti.AttnShape("tree", n_q_heads=40, n_kv_heads=8, prefix_len=512, n_branches=8, gamma=59,
                    private_len=8192 - 512, vocab=152064, logit_sigma=3.0)
TREE_DEPTH = 6
# sources whose change invalidates the DRAM traffic figure kept beside the profile summaries
KERNEL_SOURCES = ["attn_umma_t.cu", "attn_plan.cuh", "umma_ptx.cuh", "tts_internal.cuh"]


def measured_peaks():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        d = json.loads(p.read_text())
        return float(d["hbm_gbs"]), float(d.get("bf16_tflops_sustained", FALLBACK_BF16_TFLOPS)), "measured"
    return FALLBACK_HBM_GBS, FALLBACK_BF16_TFLOPS, "fallback"


def kernel_source_hash() -> str:
    h = hashlib.sha256()
    for name in KERNEL_SOURCES:
        h.update((ROOT / "paper_2505_19634_b200" / "csrc" / name).read_bytes())
    return h.hexdigest()[:16]


def recorded_traffic(workload: str):
    """DRAM read + write bytes per launch of the dominant kernel from the last ncu capture, or None when
    the kernel's sources have changed since (the record carries their hash)."""
    p = ROOT / "profiles" / "attn_umma_t_kernel_traffic.json"
    if not p.exists():
        return None
    d = json.loads(p.read_text())
    if d.get("workload") != workload or d.get("kernel_source_hash") != kernel_source_hash():
        return None
    return float(d["dram_bytes_per_launch"])


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


def tree_parents_of(shape, seed):
    return ti.make_tree_parents(shape.n_branches, shape.rows_per_branch, TREE_DEPTH, seed) if shape.name == "tree" else None


def tree_flops(shape, parents) -> int:
    """4*D flops per (query row, visible key): every node sees the prefix, the committed private tokens,
    itself and its ancestors."""
    n = shape.rows_per_branch
    depth = np.zeros(parents.shape, np.int64)
    for i in range(n):
        depth[:, i] = np.where(parents[:, i] < 0, 1, depth[np.arange(parents.shape[0]), np.maximum(parents[:, i], 0)] + 1)
    visible = (shape.prefix_len + shape.lens().astype(np.int64)[:, None] - n) + depth      # [N][n]
    return int(4 * shape.head_dim * shape.n_q_heads * visible.sum())


def oracle_attn(case, shape, parents):
    import oracle
    if parents is None:
        return oracle.verify_attn(case.q, case.k_pages, case.v_pages, case.block_table, case.prefix_len,
                                  case.branch_lens, shape.gamma)
    return oracle.verify_attn(case.q, case.k_pages, case.v_pages, case.block_table, case.prefix_len,
                              case.branch_lens, shape.gamma, mask_kind=1, tree_parents=parents)


def oracle_sample(shape: ti.AttnShape, seed: int, budget_s: float = 12.0):
    """Times the CPU oracle on whole layers of the workload (as many passes over one generated
    layer as fit the budget, at most n_layers) plus one accept pass.
    Returns (bytes processed, seconds, description, cores)."""
    import oracle
    cores = oracle.n_cores()
    oracle.build()
    bytes_done, secs, layers = 0, 0.0, 0
    case = ti.make_attn_case(shape, seed)
    parents = tree_parents_of(shape, seed)
    while layers < shape.n_layers:
        t0 = time.perf_counter()
        oracle_attn(case, shape, parents)
        dt = time.perf_counter() - t0
        secs += dt; layers += 1; bytes_done += shape.unique_kv_bytes()
        if secs + dt > budget_s:
            break
    what = f"{layers} of {shape.n_layers} layers of attention"
    if parents is None:
        acc_case = ti.make_accept_case(shape.n_branches, shape.gamma, shape.vocab, shape.logit_sigma, seed + 2)
        t0 = time.perf_counter()
        acc, _, _ = oracle.accept(acc_case.p_target, acc_case.q_draft, acc_case.draft_tokens, acc_case.uniforms)
        secs += time.perf_counter() - t0
        bytes_done += accept_algorithmic_bytes(acc, shape.gamma, shape.vocab)
        what += " + 1 accept pass"
    return bytes_done, secs, what, cores


def run_reference(args, shape):
    """The CPU oracle as the reference arm: each step = one layer of attention + the accept pass."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    oracle.build()
    cores = oracle.n_cores()
    case = ti.make_attn_case(shape, 0x5EED + 2)
    parents = tree_parents_of(shape, 0x5EED + 2)
    acc_case = None if parents is not None else ti.make_accept_case(shape.n_branches, shape.gamma, shape.vocab,
                                                                    shape.logit_sigma, 0x5EED + 4)

    def step():
        oracle_attn(case, shape, parents)
        if acc_case is None:
            return None
        a, _, _ = oracle.accept(acc_case.p_target, acc_case.q_draft, acc_case.draft_tokens, acc_case.uniforms)
        return a
    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        acc = step()
    dt = (time.perf_counter() - t0) / args.steps
    nbytes = shape.unique_kv_bytes() + (accept_algorithmic_bytes(acc, shape.gamma, shape.vocab) if acc is not None else 0)
    gbs = nbytes / dt / 1e9
    sample = "1 layer of attention%s per step (of %d layers)" % ("" if acc is None else " + 1 accept pass", shape.n_layers)
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
    lens = (f"{shape.n_branches} branches x {shape.private_len} private tokens" if shape.branch_lens is None else
            f"{shape.n_branches} branches x ragged private tokens {min(shape.branch_lens)}..{max(shape.branch_lens)}")
    rows = f"{shape.rows_per_branch}-node draft trees (depth <= {TREE_DEPTH})" if shape.name == "tree" else f"gamma={shape.gamma}"
    return (f"{shape.name}-shaped: {shape.n_layers} layers, Hq={shape.n_q_heads}, Hkv={shape.n_kv_heads}, D=128, "
            f"prefix {shape.prefix_len} + {lens}, {rows}, page 16 (random permutation), vocab {shape.vocab}")


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


class DeviceStep:
    """The device-resident inputs of one workload and its step (plan + attention per layer [+ accept])."""

    def __init__(self, shape, seed, dev, stream, with_accept=True, first_layer_case=None, parents=None):
        import torch
        import paper_2505_19634_b200 as tts
        self.tts, self.torch, self.shape = tts, torch, shape
        L, N, V = shape.n_layers, shape.n_branches, shape.vocab
        self.R = shape.rows_per_branch
        bt_np, num_pages, max_blocks = ti.make_block_table(shape, seed)
        self.bt_np, self.lens_np = bt_np, shape.lens()
        gen = torch.Generator(device=dev); gen.manual_seed(seed)
        # K/V pools: one per layer, N(0,1) bf16 drawn on the device (Philox); q likewise.  Layer 0 may come from
        # a host-generated case (the one the oracle checks).
        pool = lambda: torch.randn(num_pages, shape.n_kv_heads, 16, 128, device=dev, dtype=torch.bfloat16, generator=gen)
        self.k_pools = [pool() for _ in range(L)]
        self.v_pools = [pool() for _ in range(L)]
        self.q_all = torch.randn(L, N, self.R, shape.n_q_heads, 128, device=dev, dtype=torch.bfloat16, generator=gen)
        if first_layer_case is not None:
            as_bf16 = lambda bits: torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(dev).view(torch.bfloat16)
            self.k_pools[0].copy_(as_bf16(first_layer_case.k_pages)); self.v_pools[0].copy_(as_bf16(first_layer_case.v_pages))
            self.q_all[0].copy_(as_bf16(first_layer_case.q))
        self.out_all = torch.empty_like(self.q_all)
        self.bt, self.lens = torch.from_numpy(bt_np).to(dev), torch.from_numpy(self.lens_np).to(dev)
        self.parents = None if parents is None else torch.from_numpy(np.ascontiguousarray(parents, dtype=np.int32)).to(dev)
        self.with_accept = with_accept and parents is None
        if self.with_accept:
            self.acc_case = ti.make_accept_case(N, shape.gamma, V, shape.logit_sigma, seed + 2)
            c = self.acc_case
            self.p_t, self.q_d = torch.from_numpy(c.p_target).to(dev), torch.from_numpy(c.q_draft).to(dev)
            self.toks, self.unis = torch.from_numpy(c.draft_tokens).to(dev), torch.from_numpy(c.uniforms).to(dev)
            self.acc_len = torch.zeros(N, dtype=torch.int32, device=dev)
            self.nxt = torch.zeros(N, dtype=torch.int32, device=dev)
        self.ctx = tts.TtsContext(shape.n_q_heads, shape.n_kv_heads, N, self.R, max_blocks, num_pages, stream=stream)
        self.stream = stream

    def plan(self):
        s = self.shape
        self.ctx.tts_attn_plan(self.bt, s.prefix_len, self.lens, s.n_branches, self.R)

    def step(self, accept=True, plan=True):
        s, c, tts = self.shape, self.ctx, self.tts
        if plan:
            self.plan()
        for l in range(s.n_layers):
            if self.parents is None:
                c.tts_verify_attn(self.q_all[l], self.k_pools[l], self.v_pools[l], self.bt, s.prefix_len, self.lens,
                                  s.n_branches, s.gamma, tts.MASK_CAUSAL, self.out_all[l])
            else:
                c.tts_verify_attn_tree(self.q_all[l], self.k_pools[l], self.v_pools[l], self.bt, s.prefix_len,
                                       self.lens, self.parents, s.n_branches, self.R, self.out_all[l])
        if self.with_accept and accept:
            c.tts_accept(self.p_t, self.q_d, self.toks, self.unis, s.n_branches, s.gamma, s.vocab, self.acc_len, self.nxt)

    def capture(self, accept=True, plan=True):
        torch = self.torch
        n0 = self.ctx.tts_launch_count()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=self.stream):
            self.step(accept, plan)
        return graph, self.ctx.tts_launch_count() - n0

    def kernel_times_stream(self):
        """(main us, merge us, launches timed) from CUDA events around the single stream launches of one step:
        each figure includes the gap of a stream launch, which a graph replay does not pay."""
        self.ctx.tts_profile_enable(True)
        self.step()
        main_us, merge_us, n = self.ctx.tts_profile_read()
        self.ctx.tts_profile_enable(False)
        return main_us, merge_us, n

    def out_layer0(self):
        return self.out_all[0].float().cpu().numpy().astype(np.float64)


def time_replays(torch, run, steps, stream, barrier):
    """K replays between two barriers; an event after every replay gives the per-step times."""
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    barrier()
    ev[0].record(stream)
    for i in range(steps):
        run()
        ev[i + 1].record(stream)
    barrier()
    per = np.array([ev[i].elapsed_time(ev[i + 1]) for i in range(steps)])
    return ev[0].elapsed_time(ev[steps]) / steps, per


def attn_errors(got, want):
    diff = np.abs(got - want)
    excess = float((diff - (1e-2 + 1e-2 * np.abs(want))).max())
    rms = float(np.sqrt((diff ** 2).mean()) / max(np.sqrt((want ** 2).mean()), 1e-30))
    return excess, rms


def run_ours(args, shape):
    import torch
    import torch.distributed as dist

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
    seed = 0x5EED + 2 + 7919 * rank
    parents = tree_parents_of(shape, seed)
    stream = torch.cuda.Stream(device=dev)      # a side stream: graph capture needs one
    torch.cuda.set_stream(stream)
    ds = DeviceStep(shape, seed, dev, stream, parents=parents)
    ctx = ds.ctx

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        ds.step()
    barrier()
    # The library's calls of one step are captured once into a CUDA graph and the timed steps replay it:
    # the same kernels on the same arguments, without the per-launch gaps.
    graph, run_step, launches_per_step = None, ds.step, None
    if not args.no_graph:
        graph, launches_per_step = ds.capture()
        run_step = graph.replay
        for _ in range(3):
            run_step()
        barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    launches0 = ctx.tts_launch_count()
    ms, per_step = time_replays(torch, run_step, args.steps, stream, barrier)
    launches = launches_per_step * args.steps if graph is not None else ctx.tts_launch_count() - launches0
    status = ctx.tts_last_status()
    if status != 0:
        raise SystemExit(f"device status {status} after the timed region")

    # The dominant kernel in the launch mode of the timed steps: a graph of the attention calls alone (schedule +
    # per layer the main kernel and its merge kernel), timed like the step.  Its time per layer bounds the main
    # kernel's duration from above (an event between two kernel nodes of a graph would add its own latency).
    if graph is not None:
        attn_graph, _ = ds.capture(accept=False)
        for _ in range(3):
            attn_graph.replay()
        attn_ms, _ = time_replays(torch, attn_graph.replay, args.steps, stream, barrier)
        del attn_graph
    else:
        attn_ms, _ = time_replays(torch, lambda: ds.step(accept=False), args.steps, stream, barrier)
    layer_us = attn_ms * 1e3 / L
    main_us, merge_us, prof_calls = ds.kernel_times_stream()
    clocks = sampler.stop() if rank == 0 else None

    acc_bytes = accept_algorithmic_bytes(ds.acc_len.cpu().numpy(), g, V) if ds.with_accept else 0
    step_bytes = shape.unique_kv_bytes() * L + acc_bytes

    # ---- end to end through the host entry point (chains only) ----
    e2e = None
    if ds.with_accept:
        q_host = torch.empty(ds.q_all.shape, dtype=torch.bfloat16, pin_memory=True); q_host.copy_(ds.q_all)
        out_host = torch.empty(ds.q_all.shape, dtype=torch.bfloat16, pin_memory=True)
        pin = lambda a: torch.from_numpy(a).pin_memory()
        c = ds.acc_case
        h_bt, h_lens = pin(ds.bt_np), pin(ds.lens_np)
        h_p, h_q, h_t, h_u = pin(c.p_target), pin(c.q_draft), pin(c.draft_tokens), pin(c.uniforms)
        h_al = torch.zeros(N, dtype=torch.int32).pin_memory(); h_nt = torch.zeros(N, dtype=torch.int32).pin_memory()

        def step_host():
            ctx.tts_verify_step_host(L, q_host, ds.k_pools, ds.v_pools, h_bt, shape.prefix_len, h_lens, N, g, h_p, h_q,
                                     h_t, h_u, V, out_host, h_al, h_nt)
        e2e_steps = max(2, min(args.steps, 5))
        for _ in range(2):
            step_host()
        barrier()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            step_host()
        torch.cuda.synchronize()
        e2e_ms = (time.perf_counter() - t0) / e2e_steps * 1e3
        # the two probability tensors are pinned: the accept kernel reads its share of them in place over the host
        # link (its algorithmic bytes), everything else is copied
        h2d_copied = q_host.numel() * 2 + h_bt.numel() * 4 + h_lens.numel() * 4 + h_t.numel() * 4 + h_u.numel() * 4
        h2d = h2d_copied + acc_bytes
        h2d_all = h2d_copied + (h_p.numel() + h_q.numel()) * 4
        d2h = out_host.numel() * 2 + 8 * N
        # the same step with the accept pass fed with bf16 logits (half the bytes of the two distribution tensors)
        e2e_logits = None
        if world == 1:
            import paper_2505_19634_b200 as tts
            lc = ti.make_accept_logits_case(N, g, V, shape.logit_sigma, seed + 3, bf16=True)
            h_tl, h_dl = pin(lc.target_logits.view(np.int16)), pin(lc.draft_logits.view(np.int16))
            h_lt, h_lu = pin(lc.draft_tokens), pin(lc.uniforms)

            def step_host_logits():
                ctx.tts_verify_step_host_logits(L, q_host, ds.k_pools, ds.v_pools, h_bt, shape.prefix_len, h_lens, N, g,
                                                h_tl, h_dl, tts.LOGITS_BF16, h_lt, h_lu, V, out_host, h_al, h_nt)
            for _ in range(2):
                step_host_logits()
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            for _ in range(e2e_steps):
                step_host_logits()
            torch.cuda.synchronize()
            lms = (time.perf_counter() - t0) / e2e_steps * 1e3
            e2e_logits = {"ms_per_step": lms, "value": step_bytes / (lms * 1e-3) / 1e9, "unit": "GB/s",
                          "h2d_bytes_per_step": h2d_copied + (h_tl.numel() + h_dl.numel()) * 2,
                          "d2h_bytes_per_step": d2h, "call": "tts_verify_step_host_logits, bf16 logits"}
    else:
        e2e_ms, h2d, d2h, e2e_logits, h_p, h_q = 0.0, 0, 0, None, None, None

    ms, e2e_ms, launches = aggregate_over_ranks(ms, e2e_ms, launches, world, dev)

    if rank == 0:
        peak, tf_peak, peak_kind = measured_peaks()
        total_bytes = step_bytes * world
        value = total_bytes / (ms * 1e-3) / 1e9
        layer_bytes = shape.unique_kv_bytes()
        is_tree = parents is not None
        kernel = ("attn_umma_kernel (row-major tcgen05 attention, one layer per launch)" if is_tree else
                  "attn_umma_t_kernel (token-major tcgen05 attention, one layer per launch)")
        if is_tree:
            flops = tree_flops(shape, parents)
        timing = ("duration = time per layer of a %s of the attention calls alone (main kernel + merge kernel), CUDA events "
                  "around %d replays: an upper bound for the main kernel, so achieved and frac are lower bounds"
                  % ("graph replay" if graph is not None else "stream-launched run", args.steps))
        if is_tree:
            flops = tree_flops(shape, parents)
            roof = {"bound": "tensor", "achieved": flops / (layer_us * 1e-6) / 1e12, "peak": tf_peak, "unit": "TFLOP/s",
                    "traffic": None, "peak_kind": f"of {peak_kind} (sustained bf16 GEMM)", "kernel": kernel,
                    "flops_per_launch": flops}
            roof["frac"] = roof["achieved"] / tf_peak
        else:
            roof = {"bound": "hbm", "achieved": layer_bytes / (layer_us * 1e-6) / 1e9, "peak": peak, "unit": "GB/s",
                    "traffic": recorded_traffic(shape.name) if not args.layers else None,
                    "peak_kind": f"of {peak_kind}", "kernel": kernel, "algorithmic_bytes_per_launch": layer_bytes}
            roof["frac"] = roof["achieved"] / peak
            roof["frac_of_nominal_peak"] = roof["achieved"] / NOMINAL_HBM_GBS
        roof.update({"kernel_us": layer_us, "kernel_timing": timing,
                     "stream_launch_events": {"main_kernel_us": main_us, "merge_kernel_us": merge_us, "launches": prof_calls,
                                              "note": "CUDA events around single stream launches; each includes the launch gap"}})
        cb_bytes, cb_s, cb_sample, cores = oracle_sample(shape, 0x5EED + 2)
        rec = {
            "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "ms_per_step_median": float(np.median(per_step)), "ms_per_step_min": float(per_step.min()),
            "us_per_layer": ms * 1e3 / L,
            "frac_of_measured_peak": value / world / peak, "measured_peak_gbs": peak,
            "frac_of_nominal_peak": value / world / NOMINAL_HBM_GBS, "nominal_peak_gbs": NOMINAL_HBM_GBS,
            "config": {"workload": workload_name(shape), "l2": "inputs larger than L2: %.2f GiB of KV per step, one K/V pool per layer (for a one-layer "
                             "config: that many independent copies of the layer)" % (layer_bytes * L / 2**30), "bytes_per_step": step_bytes,
                       "launch": "one CUDA graph replay per step" if graph is not None else "stream launches",
                       "step": "tts_attn_plan + %d x attention%s" % (L, " + tts_accept" if ds.with_accept else ""),
                       "attn_impl": "auto"},
            "clocks": clocks,
            "e2e": {"value": total_bytes / (e2e_ms * 1e-3) / 1e9 if e2e_ms else None, "unit": "GB/s", "ms_per_step": e2e_ms,
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "call": "tts_verify_step_host, fp32 probabilities in pinned host memory: copied are the queries and the small "
                            "arrays; of the %d bytes of probabilities the accept kernel reads its %d algorithmic bytes in place"
                            % ((h_p.numel() + h_q.numel()) * 4 if ds.with_accept else 0, acc_bytes)},
            "e2e_logits": e2e_logits,
            "gpu_launches": launches,
            "roofline": roof,
            "cpu_baseline": {"value": cb_bytes / cb_s / 1e9, "unit": "GB/s", "cores": cores, "kind": "oracle",
                             "sample": cb_sample, "seconds": cb_s},
        }
        print(json.dumps(rec, ensure_ascii=False))
    ctx.close()
    if world > 1:
        dist.destroy_process_group()


def run_sweep(args):
    """The branch / draft-length sweep on the 32B layer shape: every point timed L2-cold (a rotation over
    enough independent copies of the layer) and checked against the oracle (all rows of the first copy).
    The timed loop holds the attention calls only; the schedule (tts_attn_plan) is built once before it, as it
    is once per 64-layer step."""
    import torch
    import oracle
    if int(os.environ.get("RANK", "0")) != 0:
        return
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    stream = torch.cuda.Stream(device=dev)
    torch.cuda.set_stream(stream)
    peak, _, peak_kind = measured_peaks()
    oracle.build()
    rows, worst_excess, worst_rms = [], -1.0, 0.0
    print("| N | gamma | seed | private tokens | prefix | unique KV MB | layers rotated | us/layer | GB/s | frac of %s peak | max excess over band | rel RMS err |" % peak_kind)
    print("|---|---|---|---|---|---|---|---|---|---|---|---|")
    for n in ti.SWEEP_BRANCHES:
        for g in ti.SWEEP_GAMMAS:
            for seed in range(args.seeds):
                shp = ti.sweep_shape(n, g, 1000 * seed + 10 * n + g)
                copies = max(2, -(-2 * L2_BYTES // shp.unique_kv_bytes()))
                shp = replace(shp, n_layers=copies)
                case = ti.make_attn_case(shp, 77 + seed)
                ti.poison_unused_slots(case)
                ds = DeviceStep(shp, 77 + seed, dev, stream, with_accept=False, first_layer_case=case)
                for _ in range(3):
                    ds.step()
                torch.cuda.synchronize()
                excess, rms = attn_errors(ds.out_layer0(), oracle_attn(case, shp, None))
                ds.plan()                                   # once per step, not per layer: outside the timed loop
                graph, _ = ds.capture(accept=False, plan=False)
                for _ in range(3):
                    graph.replay()
                ms, _ = time_replays(torch, graph.replay, args.steps, stream, torch.cuda.synchronize)
                status = ds.ctx.tts_last_status()
                us = ms * 1e3 / copies
                gbs = shp.unique_kv_bytes() / us / 1e3
                worst_excess, worst_rms = max(worst_excess, excess), max(worst_rms, rms)
                rows.append(dict(N=n, gamma=g, seed=seed, us_per_layer=us, gbs=gbs, frac=gbs / peak, excess=excess, rms=rms,
                                 status=status))
                print(f"| {n} | {g} | {seed} | {int(shp.lens().sum())} | {shp.prefix_len} | {shp.unique_kv_bytes() / 1e6:.1f} | {copies} | "
                      f"{us:.2f} | {gbs:.0f} | {gbs / peak:.3f} | {excess:+.2e} | {rms:.2e} |", flush=True)
                del graph
                ds.ctx.close()
                del ds
                torch.cuda.empty_cache()
    ok = worst_excess <= 0 and worst_rms <= 5e-3 and all(r["status"] == 0 for r in rows)
    best = max(rows, key=lambda r: r["gbs"])
    print(json.dumps({"metric": METRIC, "value": best["gbs"], "unit": "GB/s", "n_gpus": 1, "steps": args.steps, "warmup": 3,
                      "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                      "config": {"workload": "sweep on the 32B layer shape: N in %s x gamma in %s x %d seeds, ragged private lengths "
                                 "1024..8192, prefix 256..1024, random page permutation; L2-cold rotation over copies of the layer; "
                                 "value = the best point" % (list(ti.SWEEP_BRANCHES), list(ti.SWEEP_GAMMAS), args.seeds)},
                      "parity": {"points": len(rows), "all_inside_band": ok, "worst_excess_over_band": worst_excess,
                                 "worst_rel_rms": worst_rms},
                      "points": rows}, ensure_ascii=False))
    if not ok:
        raise SystemExit("sweep: a point left the oracle's band")


def run_multireq(args):
    """Several questions per call on the 32B layer shape (the multi-request setting of the paper's appendix):
    #Req questions x B branches, every question with its own shared prompt; one tts_verify_attn_groups call per
    layer.  Every point is checked against the oracle (all rows of the first copy) and timed L2-cold."""
    import torch
    import oracle
    import paper_2505_19634_b200 as tts
    if int(os.environ.get("RANK", "0")) != 0:
        return
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    stream = torch.cuda.Stream(device=dev)
    torch.cuda.set_stream(stream)
    peak, tf_peak, peak_kind = measured_peaks()
    oracle.build()
    base = ti.CONFIGS["32b"]
    gamma, R = base.gamma, base.gamma + 1
    rows, ok = [], True
    print("| #Req | B | branches | unique KV MB | GFLOP | layers rotated | us/layer | GB/s | frac of %s HBM peak | TFLOP/s | max excess over band | rel RMS err |" % peak_kind)
    print("|---|---|---|---|---|---|---|---|---|---|---|---|")
    for n_req in (1, 4, 16):
        for B in (1, 4, 16):
            N = n_req * B
            case = ti.make_group_case(base.n_q_heads, base.n_kv_heads, gamma, [B] * n_req, [base.prefix_len] * n_req,
                                      [base.private_len] * N, seed=500 + 10 * n_req + B)
            kv_bytes = case.unique_kv_bytes()
            flops = 4 * 128 * R * base.n_q_heads * N * (base.prefix_len + base.private_len)
            copies = max(2, -(-2 * L2_BYTES // kv_bytes))
            as_bf16 = lambda bits: torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(dev).view(torch.bfloat16)
            gen = torch.Generator(device=dev); gen.manual_seed(n_req * 100 + B)
            pool = lambda: torch.randn(case.num_pages, base.n_kv_heads, 16, 128, device=dev, dtype=torch.bfloat16, generator=gen)
            k_pools = [as_bf16(case.k_pages)] + [pool() for _ in range(copies - 1)]
            v_pools = [as_bf16(case.v_pages)] + [pool() for _ in range(copies - 1)]
            q_all = torch.randn(copies, N, R, base.n_q_heads, 128, device=dev, dtype=torch.bfloat16, generator=gen)
            q_all[0].copy_(as_bf16(case.q))
            out_all = torch.empty_like(q_all)
            bt, bl = torch.from_numpy(case.block_table).to(dev), torch.from_numpy(case.branch_lens).to(dev)
            ctx = tts.TtsContext(base.n_q_heads, base.n_kv_heads, N, R, case.max_blocks, case.num_pages, stream=stream)

            def step(plan=True):
                if plan:
                    ctx.tts_attn_plan_groups(bt, case.group_sizes, case.group_prefix_lens, bl, N, R)
                for l in range(copies):
                    ctx.tts_verify_attn_groups(q_all[l], k_pools[l], v_pools[l], bt, case.group_sizes,
                                               case.group_prefix_lens, bl, N, gamma, out_all[l])
            for _ in range(3):
                step()
            torch.cuda.synchronize()
            want = oracle.verify_attn_groups(case.q, case.k_pages, case.v_pages, case.block_table, case.group_sizes,
                                             case.group_prefix_lens, case.branch_lens, gamma)
            excess, rms = attn_errors(out_all[0].float().cpu().numpy().astype(np.float64), want)
            ctx.tts_attn_plan_groups(bt, case.group_sizes, case.group_prefix_lens, bl, N, R)   # once per step: not timed
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                step(plan=False)
            for _ in range(3):
                graph.replay()
            ms, _ = time_replays(torch, graph.replay, args.steps, stream, torch.cuda.synchronize)
            status = ctx.tts_last_status()
            us = ms * 1e3 / copies
            gbs, tfs = kv_bytes / us / 1e3, flops / us / 1e6
            ok = ok and excess <= 0 and rms <= 5e-3 and status == 0
            rows.append(dict(n_req=n_req, B=B, us_per_layer=us, gbs=gbs, tflops=tfs, excess=excess, rms=rms, status=status))
            print(f"| {n_req} | {B} | {N} | {kv_bytes / 1e6:.1f} | {flops / 1e9:.2f} | {copies} | {us:.2f} | {gbs:.0f} | {gbs / peak:.3f} | "
                  f"{tfs:.1f} | {excess:+.2e} | {rms:.2e} |", flush=True)
            del graph, k_pools, v_pools, q_all, out_all
            ctx.close()
            torch.cuda.empty_cache()
    best = max(rows, key=lambda r: r["gbs"])
    print(json.dumps({"metric": METRIC, "value": best["gbs"], "unit": "GB/s", "n_gpus": 1, "steps": args.steps, "warmup": 3,
                      "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                      "config": {"workload": "several questions per call on the 32B layer shape: #Req in [1, 4, 16] x B in [1, 4, 16], "
                                 "prefix %d per question, %d private tokens per branch, gamma=%d; L2-cold rotation; value = the best point"
                                 % (base.prefix_len, base.private_len, gamma)},
                      "parity": {"points": len(rows), "all_inside_band": ok}, "points": rows}, ensure_ascii=False))
    if not ok:
        raise SystemExit("multireq: a point left the oracle's band")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="32b", choices=list(ti.CONFIGS) + ["tree", "sweep", "multireq"])
    ap.add_argument("--no-graph", action="store_true", help="time plain stream launches instead of a CUDA graph replay")
    ap.add_argument("--layers", type=int, default=0,
                    help="run only this many layers of the config (small cases for profiler captures; "
                         "the workload name says so)")
    ap.add_argument("--seeds", type=int, default=3, help="seeds per point of --config sweep")
    ap.add_argument("--kernel-hash", action="store_true", help="print the hash of the dominant kernel's sources and exit")
    args = ap.parse_args()
    if args.kernel_hash:
        print(kernel_source_hash())
        return
    if args.config == "sweep":
        if args.impl == "reference":
            raise SystemExit("the sweep has no reference arm (every point is checked against the oracle inside the run)")
        run_sweep(args)
        return
    if args.config == "multireq":
        if args.impl == "reference":
            raise SystemExit("the multi-request table has no reference arm (every point is checked against the oracle inside the run)")
        run_multireq(args)
        return
    shape = TREE if args.config == "tree" else ti.CONFIGS[args.config]
    if args.layers > 0:
        shape = replace(shape, n_layers=args.layers)
    elif shape.n_layers == 1:
        # a one-layer config fits L2 (126 MB) or nearly: time a rotation over enough independent copies of the
        # layer (own K/V/Q each) that the working set exceeds twice the L2
        shape = replace(shape, n_layers=max(2, -(-2 * L2_BYTES // shape.unique_kv_bytes())))
    if args.impl == "reference":
        run_reference(args, shape)
    else:
        run_ours(args, shape)


if __name__ == "__main__":
    main()
