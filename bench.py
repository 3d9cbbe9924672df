#!/usr/bin/env python
"""Benchmark of the fused LM-head log-probability + GRPO loss forward+backward path.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config k] [--impl reference]

One step = one pass of the whole hot path over one synthetic batch: GRPO advantages from the
rewards, mask scan / row compaction, forward statistics, per-token loss, dH and dW.  The default
workload is the 3B-class head (d=2048, V=151936, 8 prompts x 8 responses x up to 512 tokens).
Prints one JSON line (rank 0).  `--impl reference` times the float64 CPU oracle instead.
"""
import argparse
import hashlib
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "fused LM-head logprob+GRPO loss fwd+bwd tokens/s; % of bf16 tensor peak"
KIND_NAMES = ["gemm_kernel<EpiStats,square> (forward statistics)", "gemm_kernel<EpiGrad,square> (dlogits slab)",
              "gemm_kernel<EpiAcc,K,MN,wide> (dH)", "gemm_kernel<EpiAcc,MN,MN,wide> (dW)"]

# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of the tensor-core kernels from one ncu capture
# of a whole config-1 step (profiles/gemm_kernel_dram_config1.md; these three metrics take one pass), valid only
# for the sources of those kernels (main loop, epilogues, PTX wrappers) whose hash is recorded with it.  Bytes
# per AVERAGE launch of a step: kind 0 is the one forward launch, kinds 1-3 the mean over the five vocabulary
# slabs (four of 37888 columns and a last one of 384).
KERNEL_SOURCES = ("epilogues.cuh", "gemm_engine.cuh", "ptx.cuh")
NCU_TRAFFIC = {"sources_sha256": "cc9c6f00c5f33fcae3a65b4309e417718e75488ec6b70b158918234ae9c94a99", "config": 1,
               "bytes_per_avg_launch": {0: 1545302000, 1: 1553519400, 2: 1775721400, 3: 1739743800}}


def sources_hash():
    h = hashlib.sha256()
    cs = os.path.join(ROOT, "paper_2512_21450_b200", "csrc")
    for f in KERNEL_SOURCES:
        h.update(open(os.path.join(cs, f), "rb").read())
    return h.hexdigest()


NOMINAL_BF16_TFLOPS = 2250.0   # B200 dense bf16, vendor figure: context beside the measured peaks


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        j = json.load(open(p))
        return dict(burst=j["bf16_tflops"], sustained=j.get("bf16_tflops_sustained", j["bf16_tflops"]),
                    hbm=j["hbm_gbs"], source="measured", nominal=NOMINAL_BF16_TFLOPS)
    return dict(burst=1590.0, sustained=1400.0, hbm=6650.0, source="fallback", nominal=NOMINAL_BF16_TFLOPS)


def spawn_ranks(n_gpus):
    """`python bench.py --gpus N` started plainly: start N ranks of this same command line under
    torch.distributed.run (one process per GPU, NCCL over 127.0.0.1) and pass their exit code on."""
    import socket
    import torch
    have = torch.cuda.device_count()
    if have < n_gpus:
        print(f"bench.py: --gpus {n_gpus} asked for, but this machine shows {have} CUDA device(s); "
              f"nothing was run", file=sys.stderr)
        sys.exit(2)
    sock = socket.socket()
    sock.bind(("127.0.0.1", 0))
    port = sock.getsockname()[1]
    sock.close()
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n_gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    sys.exit(subprocess.run(cmd).returncode)


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs (read-only)."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.rows = []
        self.proc = None
        self.gpu = gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, reasons, power = [], None, set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            if len(r) < 7:
                continue
            try:
                sm.append(float(r[0]))
                smax = float(r[1])
            except ValueError:
                continue
            try:
                power.append(float(r[2]))
            except ValueError:
                pass
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        sm.sort()
        power.sort()
        return dict(sm_mhz=sm[len(sm) // 2] if sm else None, sm_max_mhz=smax, reasons=sorted(reasons),
                    samples=len(sm), power_w=power[len(power) // 2] if power else None)


def oracle_sample_time(w, n_rows, repeat=1):
    """Times the float64 oracle (as it stands) on the first n_rows valid rows of workload w."""
    import numpy as np
    import torch
    from oracle import grpo_oracle as O
    rows = torch.nonzero(w.mask, as_tuple=False)[:n_rows, 0]
    f64 = lambda t: t.double().cpu().numpy()  # noqa: E731
    H = f64(w.H[rows])
    W = f64(w.W)
    tok = w.tokens[rows].cpu().numpy()
    old = f64(w.old_logp[rows])
    ref = None if w.ref_logp is None else f64(w.ref_logp[rows])
    adv_seq = O.grpo_advantages(w.rewards.cpu().numpy(), w.G)
    adv = O.broadcast_to_tokens(adv_seq, w.seq_offsets.cpu().numpy(), w.T)[rows.cpu().numpy()]
    mask = np.ones(rows.numel(), dtype=np.uint8)
    best = None
    for _ in range(repeat):
        t0 = time.perf_counter()
        O.grpo_advantages(w.rewards.cpu().numpy(), w.G)
        O.policy_loss_fwd_bwd(H, W, tok, old, ref, adv, mask, w.eps_low, w.eps_high, w.beta, ent_coef=w.ent_coef)
        dt = time.perf_counter() - t0
        best = dt if best is None else min(best, dt)
    return rows.numel(), best


def workload_label(cfg_id, w):
    return (f"config {cfg_id}: {w.name} d={w.d} V={w.V} rows={w.T} valid_tokens={w.n_valid} "
            f"G={w.G} eps=({w.eps_low},{w.eps_high}) beta={w.beta} ent_coef={w.ent_coef}")


def run_reference(args):
    import torch
    from paper_2512_21450_b200.workloads import CONFIGS, make_workload
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    cfg = CONFIGS[args.config]
    # the inputs are the bench workload; only a bounded sample of its valid rows is timed per step
    small = dict(prompts=1, L_max=min(cfg["L_max"], 64)) if dev == "cpu" else {}
    w = make_workload(args.config, device=dev, **small)
    n_rows = args.reference_rows
    cores = len(os.sched_getaffinity(0))
    for _ in range(args.warmup):
        oracle_sample_time(w, min(n_rows, 32))
    t_total, n_tok = 0.0, 0
    for _ in range(args.steps):
        n, dt = oracle_sample_time(w, n_rows)
        t_total += dt
        n_tok += n
    value = n_tok / t_total
    sample = f"{n_tok // max(args.steps, 1)} valid rows per step of workload {w.name} (full d, V), float64 numpy"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t_total / max(args.steps, 1),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_label(args.config, w), "sample": sample},
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def run_library_comparison(args):
    """Context for the roofline numbers: the library's tensor-core kernels and torch.matmul (cuBLAS)
    on the same operand shapes, each looped for a few seconds so both sit at the board's power cap."""
    import torch
    from paper_2512_21450_b200 import Context
    from paper_2512_21450_b200.workloads import make_workload
    ctx = Context(0)
    w = make_workload(args.config)
    rows = torch.nonzero(w.mask)[:, 0]
    Hc = w.H[rows].contiguous()
    N = Hc.shape[0] // 256 * 256
    Hc = Hc[:N]
    slab = 18944
    G = torch.randn(N, slab, device="cuda").to(torch.bfloat16)
    Ws = w.W[:slab].contiguous()
    Vq = w.V // 4 // 256 * 256
    Wq = w.W[:Vq].contiguous()

    def sustained(fn, flops, secs=2.5):
        for _ in range(10):
            fn()
        torch.cuda.synchronize()
        smp = ClockSampler(0)
        smp.start()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0, n = time.time(), 0
        e0.record()
        while time.time() - t0 < secs:
            for _ in range(20):
                fn()
            n += 20
            torch.cuda.synchronize()
        e1.record()
        torch.cuda.synchronize()
        ck = smp.stop()
        ms = e0.elapsed_time(e1) / n
        return dict(ms=ms, tflops=flops / ms / 1e9, sm_mhz=ck["sm_mhz"])

    out_q = torch.empty(N, Vq, dtype=torch.bfloat16, device="cuda")
    C_h = torch.empty(N, w.d, dtype=torch.float32, device="cuda")
    C_w = torch.empty(slab, w.d, dtype=torch.float32, device="cuda")
    res = {
        "forward_shape": {"shape": [N, w.d, Vq], "library_matmul": sustained(lambda: torch.matmul(Hc, Wq.T, out=out_q), 2.0 * N * w.d * Vq),
                          "ours_fused_forward_full_vocab": sustained(lambda: ctx.rl_token_logprobs(w.H, w.W, w.tokens, w.mask),
                                                                     2.0 * w.n_valid * w.d * w.V)},
        "dH_shape": {"shape": [N, w.d, slab], "library_matmul": sustained(lambda: torch.matmul(G, Ws), 2.0 * N * w.d * slab),
                     "ours_gemm_engine": sustained(lambda: ctx.rl_selftest_gemm(G, Ws, N, w.d, slab, 0, 1, C=C_h), 2.0 * N * w.d * slab)},
        "dW_shape": {"shape": [slab, w.d, N], "library_matmul": sustained(lambda: torch.matmul(G.T, Hc), 2.0 * N * w.d * slab),
                     "ours_gemm_engine": sustained(lambda: ctx.rl_selftest_gemm(G, Hc, slab, w.d, N, 1, 1, C=C_w), 2.0 * N * w.d * slab)},
    }
    status, _ = ctx.last_device_status()
    assert status == 0
    print(json.dumps({"library_comparison": res, "note": "sustained loops of 2.5 s each, one kernel at a time"}))


def run_small_kernel_stress(args):
    """The HBM-bound helpers at a size where a bandwidth fraction means something: 2^26 token rows,
    2^20 GRPO groups of 8 responses.  Each kernel is timed alone with CUDA events (inputs far larger
    than L2), algorithmic bytes / time against the measured copy bandwidth."""
    import torch
    from paper_2512_21450_b200 import Context
    ctx = Context(0)
    peaks = measured_peaks()
    T, n_groups, G = 1 << 26, 1 << 20, 8
    n_seq = n_groups * G
    g = torch.Generator(device="cuda").manual_seed(SEED_STRESS)
    mask = (torch.rand(T, generator=g, device="cuda") < 0.55).to(torch.uint8)
    N = int(mask.sum().item())
    row_map = torch.empty(T, dtype=torch.int32, device="cuda")
    n_valid = torch.empty(1, dtype=torch.int32, device="cuda")
    rewards = (torch.rand(n_seq, generator=g, device="cuda") < 0.4).float()
    seq_offsets = torch.arange(0, T + 1, T // n_seq, dtype=torch.int32, device="cuda")
    stats = torch.randn(1, T, 4, generator=g, device="cuda")
    stats[..., 1] = stats[..., 1].abs() + 1.0          # S >= 1 as for real statistics

    def timed(fn, iters=10):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(iters):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / iters

    out = []

    def report(name, ms, nbytes, note):
        gbs = nbytes / (ms / 1e3) / 1e9
        out.append(dict(kernel=name, ms=ms, algorithmic_bytes=nbytes, gbs=gbs, frac_of_hbm_peak=gbs / peaks["hbm"],
                        bytes=note))

    ms = timed(lambda: ctx.rl_mask_scan(mask, row_map=row_map, n_valid=n_valid))
    report("mask scan (count, offsets, write)", ms, T + 4 * N, "mask read once + row map written (the kernels read the mask twice)")
    assert int(n_valid.item()) == N
    ms = timed(lambda: ctx.rl_grpo_advantages(rewards, G, seq_offsets=seq_offsets, T=T))
    report("GRPO advantages + broadcast", ms, 12 * n_seq + 4 * (n_seq + 1) + 4 * T,
           "rewards read, per-response advantages written and read back, offsets read, per-token advantages written "
           "(the call also clears the per-token array first; the binding allocates the outputs)")
    ms = timed(lambda: ctx.rl_merge_logit_stats(stats, mask))
    report("merge of softmax statistics -> logp, entropy, lse", ms, 16 * T + T + 12 * T,
           "16 B of statistics + 1 B of mask read, three fp32 outputs written per row (the binding allocates the outputs)")
    # token-level KL reward shaping: responses of 512 rows, k3 estimate, both outputs
    n_resp = T // 512
    off512 = torch.arange(0, T + 1, 512, dtype=torch.int32, device="cuda")
    value = torch.rand(n_resp, generator=g, device="cuda")
    lp = -torch.rand(T, generator=g, device="cuda")
    rf = lp + 0.1 * torch.randn(T, generator=g, device="cuda")
    ret = torch.empty(T, device="cuda")
    ms = timed(lambda: ctx.rl_kl_shaped_returns(value, lp, rf, mask, off512, T, 0.04, returns=ret, want_shaped=False))
    report("KL-shaped returns (k3, responses of 512 rows)", ms, 9 * T + 4 * T + 8 * n_resp,
           "two fp32 inputs + 1 B of mask read, returns written per row; offsets and per-response value read")
    # the same call on rollouts of a realistic length: 2^17 responses of 512 rows (2^14 groups of 8)
    n_resp8 = n_resp // G * G
    rewards512 = (torch.rand(n_resp8, generator=g, device="cuda") < 0.4).float()
    ms = timed(lambda: ctx.rl_grpo_advantages(rewards512, G, seq_offsets=off512[:n_resp8 + 1], T=T))
    report("GRPO advantages + broadcast, responses of 512 rows", ms, 12 * n_resp8 + 4 * (n_resp8 + 1) + 4 * T,
           "as above; the per-token array is nearly all of the traffic")
    # per-token loss on its own: ratio, clip, k3, entropy bonus, token mean; both derivatives written
    ent = torch.rand(T, generator=g, device="cuda") * 11.0
    adv_tok = torch.randn(T, generator=g, device="cuda")
    old = lp + 0.05 * torch.randn(T, generator=g, device="cuda")
    outs = dict(loss=torch.empty(1, device="cuda"), dlogp=torch.empty(T, device="cuda"),
                dentropy=torch.empty(T, device="cuda"), metrics=torch.empty(8, device="cuda"))
    ms = timed(lambda: ctx.rl_token_loss(lp, ent, old, rf, adv_tok, mask, 0.2, 0.28, 0.04, ent_coef=1e-3, out=outs))
    report("per-token loss (count, ratio / clip / k3 / entropy terms, reduction)", ms, (1 + 5 * 4 + 1 + 2 * 4) * T,
           "mask read by the count pass; five fp32 inputs + mask read and two fp32 derivatives written per row")
    ms = timed(lambda: ctx.rl_token_loss(lp, None, old, rf, adv_tok, mask, 0.2, 0.2, 0.04, want_grads=False,
                                         out=dict(loss=outs["loss"], metrics=outs["metrics"])))
    report("per-token loss, loss and metrics only (no entropy term)", ms, (1 + 4 * 4 + 1) * T,
           "mask read by the count pass; four fp32 inputs + mask read per row, nothing written per row")
    status, _ = ctx.last_device_status()
    assert status == 0
    print(json.dumps({"small_kernel_stress": {"rows": T, "valid_rows": N, "groups": n_groups, "group_size": G,
                                              "peak_gbs": peaks["hbm"], "peak_source": peaks["source"], "kernels": out}}))


SEED_STRESS = 251221450 + 99


def run_reduced_case(args):
    """A reduced copy of the bench workload for profiler captures: same d and distributions, 37888 vocabulary
    rows (W = 155 MB, larger than L2), two prompts (about 4.6 K valid rows), a few steps, nothing timed.
    The gradient slab is limited to 18944 columns here, so that one step launches the forward pass and, for each
    of two vocabulary slabs, the dlogits, dH and dW passes: seven tensor-core launches per step."""
    import torch
    from paper_2512_21450_b200 import Context
    from paper_2512_21450_b200.workloads import make_workload
    ctx = Context(0)
    ctx.set_slab_limits(0, 18944)
    w = make_workload(args.config, V=37888, prompts=2)
    dH = torch.empty(w.T, w.d, dtype=torch.bfloat16, device="cuda")
    dW = torch.empty(w.V, w.d, dtype=torch.float32, device="cuda")
    loss = torch.empty(1, dtype=torch.float32, device="cuda")
    for _ in range(args.steps):
        _, adv_tok = ctx.rl_grpo_advantages(w.rewards, w.G, seq_offsets=w.seq_offsets, T=w.T)
        ctx.rl_policy_loss_fwd_bwd(w.H, w.W, w.tokens, w.old_logp, w.ref_logp, adv_tok, w.mask, w.eps_low, w.eps_high,
                                   w.beta, ent_coef=w.ent_coef, dW=dW, dH=dH, loss=loss, want_aux=False)
    torch.cuda.synchronize()
    status, detail = ctx.last_device_status()
    assert status == 0, (status, detail)
    print(json.dumps({"reduced_case": workload_label(args.config, w), "steps": args.steps, "loss": loss.item(),
                      "launches": ctx.launch_count()}))


def run_cluster_probe(args):
    """Distributed-shared-memory data movement inside thread-block clusters (rl_selftest_cluster_exchange):
    what a cluster-fused gradient pass (mode 0) or operand forwarding between CTA pairs (mode 1) could move."""
    import torch
    from paper_2512_21450_b200 import Context
    ctx = Context(0)
    iters = 20000
    rows = []
    for cs in (2, 4, 8):
        ms, ncl = ctx.selftest_cluster_exchange(0, cs, iters)
        R = 128 // cs
        b_in, b_out = (cs - 1) * R * 128 * 4, (cs - 1) * R * 128 * 2
        rows.append(dict(mode="reduce-scatter fp32 + all-gather bf16 of a 128x128 tile", cluster=cs, clusters=ncl,
                         us_per_round=1e3 * ms / iters, bytes_in_per_cta=b_in, bytes_out_per_cta=b_out,
                         gb_per_s_per_cta=(b_in + b_out) / (ms / iters * 1e-3) / 1e9))
    for cs, px in ((2, 1), (4, 2), (8, 4)):
        for nbytes in (8192, 16384, 32768):
            ms, ncl = ctx.selftest_cluster_exchange(1, cs, iters, nbytes, px)
            rows.append(dict(mode="bulk copy to the partner CTA (rank ^ %d)" % px, cluster=cs, clusters=ncl, bytes=nbytes,
                             us_per_round=1e3 * ms / iters, gb_per_s_per_cta=nbytes / (ms / iters * 1e-3) / 1e9))
    status, detail = ctx.last_device_status()
    assert status == 0, (status, detail)
    print(json.dumps({"cluster_exchange": rows, "iters": iters,
                      "sm_clock_mhz_now": torch.cuda.clock_rate() if hasattr(torch.cuda, "clock_rate") else None}))


def measure_config(ctx, w, steps, warmup, dev, world=1, reducer=None, token_count=None, profile_steps=5):
    """Times `steps` steps of workload w (profiling off), then a short separate pass with the library's
    per-kernel event brackets on.  Returns a dict of raw timings; the caller turns them into the line."""
    import torch
    import torch.distributed as dist
    dH = torch.empty(w.T, w.d, dtype=torch.bfloat16, device=dev)
    dW = torch.empty(w.V, w.d, dtype=torch.float32, device=dev)
    loss = torch.empty(1, dtype=torch.float32, device=dev)
    ctx.ensure_workspace(w.T, w.d, w.V, host=True)
    if reducer is not None:
        reducer.dW = dW

    def step():
        _, adv_tok = ctx.rl_grpo_advantages(w.rewards, w.G, seq_offsets=w.seq_offsets, T=w.T)
        if reducer is not None:
            reducer.begin()
        ctx.rl_policy_loss_fwd_bwd(w.H, w.W, w.tokens, w.old_logp, w.ref_logp, adv_tok, w.mask, w.eps_low,
                                   w.eps_high, w.beta, ent_coef=w.ent_coef, token_count=token_count, dW=dW, dH=dH,
                                   loss=loss, want_aux=False)
        if reducer is not None:
            reducer.finish(loss)

    def fence():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(warmup):
        step()
    fence()
    status, detail = ctx.last_device_status()
    assert status == 0, f"device status {status} detail {detail:#x}"

    sampler = ClockSampler(dev.index)
    sampler.start()
    launches0 = ctx.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    fence()
    e0.record()
    for _ in range(steps):
        step()
    e1.record()
    fence()
    ms = e0.elapsed_time(e1)
    launches = ctx.launch_count() - launches0
    clocks = sampler.stop()
    status, detail = ctx.last_device_status()
    assert status == 0, f"device status {status} detail {detail:#x}"

    # per-kernel times: a separate pass directly behind the timed one (board still warm), events on
    ctx.set_profiling(True)
    for _ in range(profile_steps):
        step()
    kind_ms, kind_n = ctx.profile_read()
    ctx.set_profiling(False)
    fence()
    return dict(ms=ms, steps=steps, launches=launches, clocks=clocks, kind_ms=kind_ms, kind_n=kind_n,
                profile_steps=profile_steps, dH=dH, dW=dW, loss=loss, step=step, fence=fence)


def kernel_table(w, r, peaks):
    """Per tensor-core kernel kind: TFLOP/s from the profiling pass (2 d V flop per valid token and pass)."""
    flops_step = 2.0 * w.d * w.V * w.n_valid
    out = []
    for k in range(4):
        if r["kind_n"][k]:
            t_ms = r["kind_ms"][k] / r["profile_steps"]
            tf = flops_step / (t_ms / 1e3) / 1e12
            out.append(dict(kernel=KIND_NAMES[k], launches_per_step=r["kind_n"][k] // r["profile_steps"],
                            ms_per_step=t_ms, tflops=tf, frac_of_burst=tf / peaks["burst"],
                            frac_of_sustained=tf / peaks["sustained"]))
    return out


def summarise_config(cfg_id, w, r, peaks):
    """Short record of one configuration for the `other_configs` list of the line."""
    ms_step = r["ms"] / r["steps"]
    exec_tf = 8.0 * w.d * w.V * w.n_valid / (ms_step / 1e3) / 1e12
    return dict(workload=workload_label(cfg_id, w), steps=r["steps"], ms_per_step=ms_step,
                tokens_per_s=w.n_valid / (ms_step / 1e3), executed_tflops=exec_tf,
                executed_8dV_pct_of_burst=100 * exec_tf / peaks["burst"],
                executed_8dV_pct_of_sustained=100 * exec_tf / peaks["sustained"],
                useful_6dV_pct_of_nominal=75 * exec_tf / peaks["nominal"],
                kernels=[dict(kernel=k["kernel"], tflops=k["tflops"]) for k in kernel_table(w, r, peaks)],
                clocks=r["clocks"], gpu_launches=r["launches"])


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    # 100 steps of the default workload are 3.5 s: long enough for the board to settle at its power limit,
    # which is the regime a training job runs in (20 steps from a cool board come out about 3 % faster)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=1)
    ap.add_argument("--impl", default="ours")
    ap.add_argument("--reference-rows", type=int, default=256)
    ap.add_argument("--cpu-baseline-rows", type=int, default=512)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cluster-probe", action="store_true",
                    help="instead of the benchmark line, time data movement between the CTAs of a cluster")
    ap.add_argument("--reduced-case", action="store_true",
                    help="instead of the benchmark line, run --steps steps of a reduced workload (for profiler captures)")
    ap.add_argument("--no-other-configs", action="store_true",
                    help="skip the short runs of the other large workloads (configs 1-4 besides --config)")
    ap.add_argument("--other-steps", type=int, default=8)
    ap.add_argument("--dp-path-on-one-gpu", action="store_true",
                    help="run the data-parallel code path (global count, slab-wise all-reduce on a side stream, capped "
                         "grid) in a process group of one rank, to exercise it where only one GPU is at hand")
    ap.add_argument("--dp-free-sms", type=int, default=4,
                    help="with more than one GPU: SMs the persistent grids leave to the all-reduce kernels")
    ap.add_argument("--compare-library", action="store_true",
                    help="instead of the benchmark line, time the tensor-core kernels against torch.matmul")
    ap.add_argument("--stress-small", action="store_true",
                    help="instead of the benchmark line, time the HBM-bound helper kernels at 2^26 rows / 2^20 groups")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl != "reference" else args.warmup

    if args.impl == "reference":
        run_reference(args)
        return
    if args.compare_library:
        run_library_comparison(args)
        return
    if args.stress_small:
        run_small_kernel_stress(args)
        return
    if args.cluster_probe:
        run_cluster_probe(args)
        return
    if args.reduced_case:
        run_reduced_case(args)
        return


    world_env = os.environ.get("WORLD_SIZE")
    if world_env is None and args.gpus > 1:
        spawn_ranks(args.gpus)      # does not return

    import torch
    import torch.distributed as dist
    from paper_2512_21450_b200 import Context
    from paper_2512_21450_b200 import parallel as par
    from paper_2512_21450_b200.workloads import SEED_BASE, make_workload

    world = int(world_env or "1")
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dp_path = world > 1 or args.dp_path_on_one_gpu
    if dp_path:
        if world == 1:
            os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
            os.environ.setdefault("MASTER_PORT", "29533")
            os.environ.setdefault("RANK", "0")
            os.environ.setdefault("WORLD_SIZE", "1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.device("cuda", local)
    peaks = measured_peaks()

    # weak scaling: every rank owns a full batch of the configuration, with its own seed
    w = make_workload(args.config, device=dev, seed=SEED_BASE + args.config + 1000 * rank)
    ctx = Context(local)
    reducer, token_count = None, None
    if dp_path:
        # data parallel: the token mean is over all ranks' valid tokens (count summed on the device, never
        # read by the host) and dW is all-reduced slab by slab on a side stream while the backward pass of
        # the remaining slabs runs; a few SMs are left to the collective's kernels
        token_count = par.global_valid_count(w.mask)
        reducer = par.SlabGradientReducer(torch.empty(0, device=dev), single_rank_too=True)
        ctx.set_dw_slab_hook(reducer.on_slab)
        if args.dp_free_sms > 0:
            ctx.set_max_ctas(torch.cuda.get_device_properties(dev).multi_processor_count - args.dp_free_sms)

    r = measure_config(ctx, w, args.steps, args.warmup, dev, world, reducer, token_count,
                       profile_steps=max(1, min(args.steps, 20)))
    ms, dH, dW, loss = r["ms"], r["dH"], r["dW"], r["loss"]
    fence = r["fence"]
    device_loss = float(loss.item())

    t = torch.tensor([ms, float(w.n_valid)], dtype=torch.float64, device=dev)
    if world > 1:
        tmax = t.clone()
        dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
        tsum = t.clone()
        dist.all_reduce(tsum, op=dist.ReduceOp.SUM)
        ms, n_tok = float(tmax[0].item()), float(tsum[1].item())
    else:
        n_tok = float(w.n_valid)
    value = n_tok * args.steps / (ms / 1e3)

    # ---- end to end through the host-buffer entry point: per-step inputs start in pinned host memory
    pin = lambda x: None if x is None else x.cpu().pin_memory()  # noqa: E731
    hH, htok, hold, href, hmask = pin(w.H), pin(w.tokens), pin(w.old_logp), pin(w.ref_logp), pin(w.mask)
    hrew, hoff = pin(w.rewards), pin(w.seq_offsets)
    h2d = sum(x.numel() * x.element_size() for x in (hH, htok, hold, href, hmask, hrew, hoff) if x is not None)
    e2e_steps = max(3, min(args.steps, 30))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    # Two staging slots: the copies of step i+1 run on the library's copy stream while the kernels of step i
    # run; every step still copies its own inputs from pinned host memory and has its loss read back on the host.
    outs = [(dH, dW), (torch.empty_like(dH), torch.empty_like(dW))]
    ctx.set_dw_slab_hook(None)

    def e2e_submit(i):
        k = i % 2
        ctx.rl_policy_loss_fwd_bwd_host_submit(k, hH, w.W, htok, hold, href, None, hmask, w.eps_low, w.eps_high, w.beta,
                                               w.ent_coef, outs[k][0], outs[k][1], rewards_host=hrew, group_size=w.G,
                                               seq_offsets_host=hoff)

    def e2e_wait(i):
        k = i % 2
        out = ctx.rl_policy_loss_fwd_bwd_host_wait(k)
        if world > 1:
            # the host entry normalises by the local token count; the gradient exchange is the same
            par.allreduce_gradients(outs[k][1], loss)
        return out

    def e2e_run(n):
        e2e_submit(0)
        for i in range(1, n + 1):
            if i < n:
                e2e_submit(i)
            last = e2e_wait(i - 1)
        return last

    e2e_run(2)
    fence()
    e0.record()
    host_loss, _ = e2e_run(e2e_steps)
    e1.record()
    fence()
    e2e_ms = e0.elapsed_time(e1)
    if world > 1:
        tm = torch.tensor([e2e_ms], dtype=torch.float64, device=dev)
        dist.all_reduce(tm, op=dist.ReduceOp.MAX)
        e2e_ms = float(tm.item())
    e2e_val = n_tok * e2e_steps / (e2e_ms / 1e3)
    if world == 1:
        assert abs(host_loss - device_loss) <= 1e-5 * abs(device_loss) + 1e-7

    # ---- the other large workloads, a few steps each (one GPU only): the record carries all four
    other = []
    if world == 1 and not dp_path and not args.no_other_configs:
        del outs, hH
        for cfg_id in (1, 2, 3, 4):
            if cfg_id == args.config:
                continue
            r["dH"] = r["dW"] = r["step"] = dH = dW = None
            torch.cuda.empty_cache()
            w2 = make_workload(cfg_id, device=dev)
            r2 = measure_config(ctx, w2, args.other_steps, 3, dev, profile_steps=2)
            other.append(summarise_config(cfg_id, w2, r2, peaks))
            del r2, w2

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    kind_ms, kind_n, psteps = r["kind_ms"], r["kind_n"], r["profile_steps"]
    kinds = kernel_table(w, r, peaks)
    dom = max(range(4), key=lambda k: kind_ms[k])
    launches_dom = max(kind_n[dom] // psteps, 1)
    flops_launch = 2.0 * w.d * w.V * w.n_valid / launches_dom
    avg_launch_ms = kind_ms[dom] / max(kind_n[dom], 1)
    achieved = flops_launch / (avg_launch_ms / 1e3) / 1e12
    traffic = None
    if NCU_TRAFFIC["sources_sha256"] == sources_hash() and NCU_TRAFFIC["config"] == args.config:
        traffic = float(NCU_TRAFFIC["bytes_per_avg_launch"][dom])
    # which measured peak the kernel is held to: the burst figure when the timed region is short (the board
    # has not settled at its power limit yet), the sustained one for a region of seconds; both are printed
    timed_s = ms / 1e3
    peak_kind = "burst" if timed_s < 2.0 else "sustained"
    roofline = {
        "bound": "tensor", "kernel": KIND_NAMES[dom], "achieved": achieved, "peak": peaks[peak_kind],
        "unit": "TFLOP/s", "frac": achieved / peaks[peak_kind],
        "peak_source": f"of {peaks['source']} ({peak_kind}: timed region {timed_s:.2f} s)",
        "frac_of_burst": achieved / peaks["burst"], "frac_of_sustained": achieved / peaks["sustained"],
        "frac_of_nominal": achieved / peaks["nominal"],
        "traffic": traffic, "flops_per_launch": flops_launch, "avg_launch_ms": avg_launch_ms,
        "timing": f"CUDA events around every launch, separate pass of {psteps} steps directly behind the timed region",
        "kernels": kinds,
    }
    # HBM-bound helpers: algorithmic bytes per step against their event time
    N, Npad = w.n_valid, (w.n_valid + 127) // 128 * 128
    n_tiles = (w.V + 255) // 256
    m_units, workers = (N + 255) // 256, 74
    split = min(range(1, min(16, n_tiles) + 1),
                key=lambda sp: (-(-m_units * sp // workers) * -(-n_tiles // sp), sp))
    small_bytes = {
        4: ("mask scan (3 launches)", w.T + 4 * N),
        5: ("row gather", 2 * N * w.d + 2 * Npad * w.d + 12 * N),
        6: ("merge + per-token loss", N * (16 * split + 32)),
        7: ("dH scatter", 6 * N * w.d + 4 * N),
        8: ("GRPO advantages + broadcast", 12 * w.n_seq + 4 * w.T),
    }
    small = []
    for k, (name, nbytes) in small_bytes.items():
        if kind_n[k]:
            t_ms = kind_ms[k] / psteps
            small.append(dict(kernel=name, ms_per_step=t_ms, bytes_per_step=nbytes,
                              gbs=nbytes / (t_ms / 1e3) / 1e9, frac_of_hbm_peak=nbytes / (t_ms / 1e3) / 1e9 / peaks["hbm"]))
    exec_tflops = 8.0 * w.d * w.V * n_tok * args.steps / (ms / 1e3) / 1e12 / world
    clocks = r["clocks"]
    mhz = clocks.get("sm_mhz") or 0.0
    out = {
        "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": workload_label(args.config, w),
                   "l2": "inputs larger than L2 (W alone is %.0f MB; L2 126 MB)" % (w.V * w.d * 2 / 1e6),
                   "parallelism": (f"dp{world}: prompts sharded, dW all-reduced slab by slab under the backward pass"
                                   if dp_path else "single GPU"),
                   "masked_rows": "skipped (row compaction)",
                   "row_tiles": "%d valid rows = %d tiles of 256 rows%s" % (
                       N, (N + 255) // 256, " exactly (no ragged row tile at this seed)" if N % 256 == 0 else
                       " (last tile %d rows)" % (N % 256))},
        "pct_of_bf16_peak": {"executed_8dV_of_burst": 100 * exec_tflops / peaks["burst"],
                             "executed_8dV_of_sustained": 100 * exec_tflops / peaks["sustained"],
                             "executed_8dV_of_nominal": 100 * exec_tflops / peaks["nominal"],
                             "useful_6dV_of_burst": 75 * exec_tflops / peaks["burst"],
                             "useful_6dV_of_nominal": 75 * exec_tflops / peaks["nominal"],
                             "executed_tflops_per_gpu": exec_tflops, "peaks": peaks["source"],
                             "burst_tflops": peaks["burst"], "sustained_tflops": peaks["sustained"],
                             "nominal_tflops": peaks["nominal"],
                             "target": "60 % of the bf16 dense tensor peak on useful (6 d V) flops",
                             "ms_per_step_x_sm_ghz": ms / args.steps * mhz / 1e3},
        "clocks": clocks, "gpu_launches": r["launches"], "roofline": roofline,
        "small_kernels": {"bound": "hbm", "peak_gbs": peaks["hbm"], "kernels": small},
    }
    if other:
        out["other_configs"] = other
    if e2e_val is not None:
        out["e2e"] = {"value": e2e_val, "unit": "tokens/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": 64,
                      "steps": e2e_steps, "call": "rl_policy_loss_fwd_bwd_host_submit / _wait, two steps in flight (pinned host inputs, W resident)"}
    if world == 1 and not args.no_cpu_baseline:
        n, dt = oracle_sample_time(w, args.cpu_baseline_rows)
        out["cpu_baseline"] = {"value": n / dt, "unit": "tokens/s", "cores": len(os.sched_getaffinity(0)),
                               "kind": "oracle", "sample": f"first {n} valid rows of the same workload, full d and V, "
                                                           f"float64 numpy, one pass ({dt:.1f} s)"}
    print(json.dumps(out))
    if dp_path:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
