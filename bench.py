#!/usr/bin/env python
"""Benchmark of the decayed linear-attention hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One "step" is one pass of the whole training hot path -- la_fwd followed by
la_bwd (dQ, dK, dV) -- over one synthetic batch of the 7B-like long-context
workload (B=1, H=32, N=65536, d=e=128, bf16 in, fp32 accumulate, fp32 out).
The decode leg (batch 64, H=32, d=e=128, fp32 state, 256 recurrent steps after
a 4096-token prefill) is timed in the same run and reported under "decode".

Prints ONE JSON line.  `value` is fwd+bwd TFLOP/s counted with the block-method
flop count per token-head (intra-block MACs for i>=j only), inputs resident in
HBM.  `e2e` is the same metric through la_fwd_bwd_host with pinned host buffers
(copies inside the timed region).  `roofline` describes the dominant kernel (the
block walk), `step_roofline` the whole fwd+bwd step against
max(flops/tensor peak, bytes/HBM peak).  `--impl reference` times the CPU oracle
on a bounded sample of the same workload.

With N > 1 (torchrun) every rank runs its own copy of the workload (the path
shards over batch and heads with no exchange step): weak scaling, no collective
on the data path; timing is the max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "decayed linear-attn fwd+bwd TFLOP/s at 7B shape"
UNIT = "TFLOP/s"
WORKLOAD = "7b_long"


# ---- accounting (per token-head, d = e, block size C capped at 128) ----------------------------
def flops_per_token_head(d: int, C: int = 128) -> float:
    C = min(C, 128)
    fwd = 2 * C * d + 4 * d * d        # half score tile + half P.V tile, Q.KV, K^T V
    bwd = 5 * C * d + 10 * d * d
    return float(fwd + bwd)


def flop_conventions(d: int, C: int = 128) -> dict:
    """The three flop counts per token-head (d = e): the recurrence's lower bound F_min = 12 d^2, the block
    method with half tiles F_alg (the headline TFLOP/s uses it), and the full tiles the tensor cores are
    actually asked for with single-term operands, F_exec (hi/lo operand terms come on top of that)."""
    C = min(C, 128)
    return {"F_min": float(12 * d * d), "F_alg": flops_per_token_head(d, C),
            "F_exec": float((4 * C * d + 4 * d * d) + (10 * C * d + 10 * d * d))}


def bytes_per_token_head(d: int, out_bytes: int, what: str) -> float:
    fwd = 2 * 3 * d + out_bytes * d                 # read q,k,v ; write o
    bwd = 2 * 4 * d + out_bytes * 3 * d             # read q,k,v,dO ; write dq,dk,dv
    walk = 2 * 3 * d + out_bytes * d                # one walk launch: read a,b,c ; write out
    pair = 2 * 4 * d + out_bytes * 2 * d            # the dV and dK walks in one launch: read q,k,v,dO ; write dk,dv
    return float({"fwd": fwd, "bwd": bwd, "step": fwd + bwd, "walk": walk, "walk_pair": pair}[what])


# DRAM traffic of one walk launch per token-head, from the ncu capture summarised in
# profiles/tc_walk_full_kernel_small_case.md: 412.4 MB read per 524288 token-heads (the algorithmic
# 768 B plus 2.4 % for entry states and re-fetches).  The writes of that small launch (230 MB of the
# 268 MB of output; the rest was still in L2 when it ended) do not grow in proportion: at full size
# the 4.3 GB of output cannot stay in the 126 MB L2, so the output is counted in full (512 B).
WALK_DRAM_BYTES_PER_TOKEN_HEAD = 412.4e6 / 524288 + 512.0


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# ---- clocks sampling ----------------------------------------------------------------------------
class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu_index), "--query-gpu=" + self.QUERY,
                 "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
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
        except Exception:
            self.proc.kill()
        sm, smax, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                smax.append(float(f[2]))
                power.append(float(f[3]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


# ---- the CPU oracle leg -------------------------------------------------------------------------
def oracle_sample_run(heads: int, n_tokens: int, seed: int = 0):
    """Oracle fwd+bwd (token recurrence, fp64) on `heads` heads x n_tokens of the workload. Returns seconds."""
    import torch
    from oracle import la_oracle as orc
    from paper_2307_14995_b200 import inputs
    w = inputs.WORKLOADS[WORKLOAD]
    q, k, v, do = inputs.make_qkvdo(1, heads, n_tokens, w.d, w.e, dtype=w.in_dtype, seed=seed)
    lam = inputs.decay_rates(w.H, w.l_over_L)[:heads].double().numpy()
    t0 = time.perf_counter()
    orc.fwd_rec(q, k, v, lam)
    orc.bwd_rec(q, k, v, do, lam)
    return time.perf_counter() - t0


def cpu_baseline(target_seconds: float = 12.0):
    from oracle import la_oracle as orc
    from paper_2307_14995_b200 import inputs
    w = inputs.WORKLOADS[WORKLOAD]
    cores = orc.threads()
    heads = min(w.H, max(cores, 1))
    t_cal = oracle_sample_run(heads, 1024)
    n = int(min(w.N, max(1024, 1024 * target_seconds / max(t_cal, 1e-3))))
    n = max(1024, n // 1024 * 1024)
    t = oracle_sample_run(heads, n)
    th = heads * n
    # the recurrence the oracle runs executes 12 d e flops per token-head (4 forward, 8 backward)
    f_rec = 12.0 * w.d * w.e
    return {"value": th * f_rec / t / 1e12, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": "%d heads x %d tokens of the %s workload (fwd+bwd token recurrence, fp64), %.1f s"
                      % (heads, n, WORKLOAD, t),
            "flops_per_token_head": f_rec, "gflops": th * f_rec / t / 1e9, "token_heads_per_s": th / t}


def run_reference(args):
    """--impl reference: the oracle as it stands, on host cores, bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import la_oracle as orc
    from paper_2307_14995_b200 import inputs
    w = inputs.WORKLOADS[WORKLOAD]
    cores = orc.threads()
    heads = min(w.H, max(cores, 1))
    t_cal = oracle_sample_run(heads, 512)
    budget = 120.0 / max(1, args.steps + args.warmup)           # whole run within a few minutes
    n = int(min(w.N, max(512, 512 * min(budget, 20.0) / max(t_cal, 1e-3))))
    n = max(512, n // 512 * 512)
    for _ in range(args.warmup):
        oracle_sample_run(heads, n)
    times = [oracle_sample_run(heads, n) for _ in range(args.steps)]
    t = sum(times) / len(times)
    th = heads * n
    # same flop count per token-head as the GPU arm's line, so that the ratio of the two `value`s is the ratio of
    # token-heads per second; what the recurrence itself executes (12 d e) is given beside it
    value = th * flops_per_token_head(w.d) / t / 1e12
    sample = "%d heads x %d tokens of the %s workload per step (fwd+bwd token recurrence, fp64)" % (heads, n, WORKLOAD)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": t * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": "%s: B=1,H=%d,N=%d,d=e=%d (sample: %s)" % (WORKLOAD, w.H, w.N, w.d, sample)},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample,
                             "token_heads_per_s": th / t, "gflops_by_12de": th * 12.0 * w.d * w.e / t / 1e9},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ---- our arm ------------------------------------------------------------------------------------
def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2307_14995_b200 import binding as la, dist_utils, inputs

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    la.load()
    peaks = load_peaks()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(x: float) -> float:
        return dist_utils.max_over_ranks(x, device=dev)

    w = inputs.WORKLOADS[WORKLOAD]
    out_dtype = torch.float32
    data = inputs.device_randn_like_workload(WORKLOAD, dev, seed=rank)
    q, k, v, do, lam = data["q"], data["k"], data["v"], data["do"], data["lam"]
    if args.small:
        # profiling case: 16 heads x 32768 tokens (1.6 GB of inputs and outputs, far beyond L2; one wave of 144
        # thread blocks of 29 blocks each), same kernels
        import dataclasses
        w = dataclasses.replace(w, H=16, N=32768)
        q, k, v, do = (x[:, :16, :32768].contiguous() for x in (q, k, v, do))
        lam = lam[:16].contiguous()
    shape = la.make_shape(w.B, w.H, w.N, w.d, w.e, w.in_dtype, out_dtype, seg_len=args.seg_len, precision=args.precision)
    o = torch.empty((w.B, w.H, w.N, w.e), dtype=out_dtype, device=dev)
    dq, dk, dv = (torch.empty((w.B, w.H, w.N, w.d), dtype=out_dtype, device=dev) for _ in range(3))
    ws_f = la.alloc_workspace(la.LA_OP_FWD, shape, dev)
    ws_b = la.alloc_workspace(la.LA_OP_BWD, shape, dev)
    stream = torch.cuda.current_stream()

    def step():
        la.la_fwd(shape, q, k, v, lam, o, None, None, ws_f, stream)
        la.la_bwd(shape, q, k, v, do, lam, dq, dk, dv, None, None, None, ws_b, stream, fwd_workspace=ws_f)

    train_steps = 0 if args.only == "decode" else args.steps
    # clocks are sampled from before the warm-up until the last timed leg has finished
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    for _ in range(args.warmup if train_steps else 0):
        step()
    barrier()
    la.device_status()
    # ---- headline loop: profiling off, nothing but the launches between the two outer events; the
    # ---- events between steps only mark step boundaries for the median / min
    launches0 = la.launch_count()
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(train_steps + 1)]
    marks[0].record(stream)
    for i in range(train_steps):
        step()
        marks[i + 1].record(stream)
    barrier()
    launches = la.launch_count() - launches0
    la.device_status()  # a block whose bounded wait expired would have left its output unwritten: fail the run
    ms_step = max_over_ranks(marks[0].elapsed_time(marks[-1]) / max(train_steps, 1))
    per_step = sorted(marks[i].elapsed_time(marks[i + 1]) for i in range(train_steps))
    ms_median = max_over_ranks(per_step[len(per_step) // 2]) if per_step else None
    ms_min = max_over_ranks(per_step[0]) if per_step else None
    # ---- second, separate loop with per-launch event pairs: the per-kernel breakdown and the roofline of the
    # ---- dominant kernel come from here, never the headline number
    prof_steps = max(1, min(train_steps, 5))
    la.profile_enable(True)
    for _ in range(prof_steps if train_steps else 0):
        step()
    barrier()
    la.profile_enable(False)
    prof = la.profile_collect()
    la.device_status()

    th = w.token_heads
    F = flops_per_token_head(w.d)
    ms_step = max(ms_step, 1e-9)  # (--only decode times no training step)
    value = world * th * F / (ms_step * 1e-3) / 1e12
    ob = 4 if out_dtype == torch.float32 else 2
    step_bytes = th * bytes_per_token_head(w.d, ob, "step")
    t_roof = max(th * F / (peaks["bf16_tflops_sustained"] * 1e12), step_bytes / (peaks["hbm_gbs"] * 1e9))
    t_roof_datasheet = max(th * F / 2250e12, step_bytes / 8000e9)
    walk_ms, walk_n = prof["walk"]
    walk_bytes = th * bytes_per_token_head(w.d, ob, "walk")
    walk_avg_ms = walk_ms / max(walk_n, 1)
    achieved = walk_bytes / (walk_avg_ms * 1e-3) / 1e9 if walk_n else None
    pair_ms, pair_n = prof.get("walk_pair", (0.0, 0))
    pair_bytes = th * bytes_per_token_head(w.d, ob, "walk_pair")
    pair_avg_ms = pair_ms / max(pair_n, 1)
    pair_gbs = pair_bytes / (pair_avg_ms * 1e-3) / 1e9 if pair_n else None

    if args.only == "train":
        if rank == 0:
            print(json.dumps({"only": "train", "small": bool(args.small), "ms_per_step": ms_step,
                              "ms_per_step_median": ms_median, "ms_per_step_min": ms_min, "clocks": sampler.stop(),
                              "kernel_ms_per_step": {n: ms / prof_steps for n, (ms, _) in prof.items()},
                              "kernel_launches_per_step": {n: c / prof_steps for n, (_, c) in prof.items()},
                              "walk_gbs": achieved, "walk_pair_gbs": pair_gbs}), flush=True)
        return

    # forward and backward also timed on their own (same buffers, same rules), after the headline loop
    split_ms = {}
    for nm, fn in (("fwd", lambda: la.la_fwd(shape, q, k, v, lam, o, None, None, ws_f, stream)),
                   ("bwd", lambda: la.la_bwd(shape, q, k, v, do, lam, dq, dk, dv, None, None, None, ws_b, stream,
                                             fwd_workspace=ws_f))):
        fn()
        barrier()
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        nrep = max(1, min(train_steps, 10))
        s0.record(stream)
        for _ in range(nrep):
            fn()
        s1.record(stream)
        barrier()
        split_ms[nm] = max_over_ranks(s0.elapsed_time(s1) / nrep)

    # ---- the token mixer's output stage fused into the forward walk (y = SRMSNorm(o) (.) u), same shape ----
    gated = None
    if train_steps:
        gen_u = torch.Generator(dev)
        gen_u.manual_seed(77 + rank)
        ug = torch.randn((w.B, w.H, w.N, w.e), generator=gen_u, device=dev).to(torch.bfloat16)
        yg = torch.empty_like(o)
        dyg = torch.randn((w.B, w.H, w.N, w.e), generator=gen_u, device=dev).to(torch.bfloat16)
        dog = torch.empty((w.B, w.H, w.N, w.e), dtype=torch.bfloat16, device=dev)

        def time_loop(fn, n=10):
            fn()
            barrier()
            a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            l0 = la.launch_count()
            a0.record(stream)
            for _ in range(n):
                fn()
            a1.record(stream)
            barrier()
            la.device_status()
            return max_over_ranks(a0.elapsed_time(a1) / n), (la.launch_count() - l0) / n

        fused_ms, fused_l = time_loop(lambda: la.la_fwd_gated(shape, q, k, v, ug, lam, yg, None, None, None, None, ws_f, stream))
        train_ms, train_l = time_loop(lambda: la.la_fwd_gated(shape, q, k, v, ug, lam, yg, o, None, None, None, ws_f, stream))

        def unfused():
            la.la_fwd(shape, q, k, v, lam, o, None, None, ws_f, stream)
            la.la_gate_fwd(shape, o, ug, yg, None, stream)

        unfused_ms, unfused_l = time_loop(unfused)
        gbwd_ms, _ = time_loop(lambda: la.la_gate_bwd(shape, o, ug, dyg, dog, dv, stream))
        eb = 4 if out_dtype == torch.float32 else 2
        gated = {"what": "la_fwd_gated at the same shape: y = SRMSNorm(o) (.) u as the forward walk's epilogue (Eq. 3, Eq. 8)",
                 "fused_ms": fused_ms, "fused_launches": fused_l,
                 "fused_bytes_per_token_head": 2 * 4 * w.d + eb * w.d,      # read q,k,v,u ; write y (o never written)
                 "fused_also_writing_o_ms": train_ms,
                 "unfused_ms": unfused_ms, "unfused_launches": unfused_l,
                 "unfused_bytes_per_token_head": 2 * 4 * w.d + 3 * eb * w.d,  # + write o, read o back
                 "gate_bwd_ms": gbwd_ms,
                 "gate_bwd_gbs": th * (eb * w.d + 3 * 2 * w.d + eb * w.d) / (gbwd_ms * 1e-3) / 1e9}
        del ug, yg, dyg, dog

    # ---- LRPE-d (Eq. 1), the first layer's variant: feature doubling around two runs of the operator ----
    lrpe = None
    if train_steps and args.only == "all":
        theta = inputs.make_theta(w.H, w.d, seed=2).to(dev)
        dth = torch.empty((w.H, w.d), dtype=torch.float32, device=dev)
        wl_f = torch.empty(la.lrpe_workspace_bytes(la.LA_OP_FWD, shape), dtype=torch.uint8, device=dev)
        lf_ms, lf_l = time_loop(lambda: la.la_lrpe_fwd(shape, q, k, v, theta, lam, o, 0, None, None, wl_f, stream), n=5)
        wl_b = torch.empty(la.lrpe_workspace_bytes(la.LA_OP_BWD, shape), dtype=torch.uint8, device=dev)
        lb_ms, lb_l = time_loop(lambda: la.la_lrpe_bwd(shape, q, k, v, do, theta, lam, dq, dk, dv, dth, 0, None, None, None,
                                                       wl_b, stream), n=5)
        lrpe = {"what": "la_lrpe_fwd + la_lrpe_bwd at the same shape (rotation of Eq. 1 as position features, doubled "
                        "feature dimension = two runs of the operator plus element-wise kernels)",
                "fwd_ms": lf_ms, "bwd_ms": lb_ms, "fwd_launches": lf_l, "bwd_launches": lb_l,
                "ratio_to_plain_step": (lf_ms + lb_ms) / ms_step,
                "workspace_bytes": {"fwd": wl_f.numel(), "bwd": wl_b.numel()}}
        del wl_f, wl_b, theta, dth

    # ---- sequence parallelism: what one rank adds around its la_fwd / la_bwd when the shape is one chunk of a longer
    # sequence (the all-gather itself needs more than one GPU and is not timed here) ----
    seqpar_leg = None
    if train_steps and args.only == "all":
        st_loc = torch.empty((w.B, w.H, w.d, w.e), dtype=torch.float32, device=dev)
        st_all = torch.zeros((8, w.B, w.H, w.d, w.e), dtype=torch.float32, device=dev)
        ws_s = torch.empty(max(la.chunk_state_workspace_bytes(shape), 256), dtype=torch.uint8, device=dev)
        cs_f, _ = time_loop(lambda: la.la_chunk_state(shape, 0, k, v, lam, st_loc, ws_s, stream))
        cs_r, _ = time_loop(lambda: la.la_chunk_state(shape, 1, q, do, lam, st_loc, ws_s, stream))
        ch, _ = time_loop(lambda: la.la_chain_states(shape, 8 * w.N, w.N, 0, st_all, 8, 7, None, lam, st_loc, stream))
        seqpar_leg = {"what": "per-rank additions of the sequence-parallel protocol at this shape as one chunk of 8: "
                              "la_chunk_state (forward: k, v; reverse: q, dO), la_chain_states over 7 earlier chunks",
                      "chunk_state_fwd_ms": cs_f, "chunk_state_rev_ms": cs_r, "chain_ms": ch,
                      "gathered_bytes_per_rank_and_direction": st_loc.numel() * 4,
                      "added_fraction_of_step": (cs_f + cs_r + 2 * ch) / ms_step}
        del st_loc, st_all, ws_s

    # ---- packed batch of sequences of different lengths (prefill of a serving batch), forward only ----
    varlen_leg = None
    if train_steps and args.only == "all":
        gen_v = torch.Generator("cpu")
        gen_v.manual_seed(5)
        lens = [int(x) for x in torch.randint(64, 4097, (64,), generator=gen_v)]
        cu = [0]
        for n_ in lens:
            cu.append(cu[-1] + n_)
        Tt = cu[-1]
        vshape = la.make_shape(1, w.H, Tt, w.d, w.e, torch.bfloat16, out_dtype, layout=la.LA_LAYOUT_BNHD)
        gen_d = torch.Generator(dev)
        gen_d.manual_seed(6 + rank)
        vq = torch.nn.functional.silu(torch.randn((1, Tt, w.H, w.d), generator=gen_d, device=dev)).to(torch.bfloat16)
        vk = torch.nn.functional.silu(torch.randn((1, Tt, w.H, w.d), generator=gen_d, device=dev)).to(torch.bfloat16)
        vv = torch.randn((1, Tt, w.H, w.e), generator=gen_d, device=dev).to(torch.bfloat16)
        vo = torch.empty((1, Tt, w.H, w.e), dtype=out_dtype, device=dev)
        vkv = torch.empty((len(lens), w.H, w.d, w.e), dtype=torch.float32, device=dev)
        vws = torch.empty(max(la.varlen_workspace_bytes(la.LA_OP_FWD, vshape, cu), 256), dtype=torch.uint8, device=dev)
        pk_ms, pk_l = time_loop(lambda: la.la_fwd_varlen(vshape, vq, vk, vv, lam, vo, cu, None, vkv, vws, stream))

        def one_by_one():
            for i_ in range(len(lens)):
                a_, b_ = cu[i_], cu[i_ + 1]
                sh_ = la.make_shape(1, w.H, b_ - a_, w.d, w.e, torch.bfloat16, out_dtype, layout=la.LA_LAYOUT_BNHD)
                la.la_fwd(sh_, vq[:, a_:b_], vk[:, a_:b_], vv[:, a_:b_], lam, vo[:, a_:b_], None, vkv[i_:i_ + 1], vws, stream)

        sq_ms, sq_l = time_loop(one_by_one, n=3)
        eb = 4 if out_dtype == torch.float32 else 2
        vbytes = Tt * w.H * (3 * 2 * w.d + eb * w.e)
        varlen_leg = {"what": "la_fwd_varlen over 64 packed sequences of 64..4096 tokens (seeded lengths), %d tokens, H=%d, "
                              "d=e=%d: all sequences in one set of launches, against one la_fwd per sequence" % (Tt, w.H, w.d),
                      "packed_ms": pk_ms, "packed_launches": pk_l, "packed_gbs": vbytes / (pk_ms * 1e-3) / 1e9,
                      "frac_of_hbm_peak": vbytes / (pk_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                      "per_sequence_ms": sq_ms, "per_sequence_launches": sq_l, "tokens": Tt}
        del vq, vk, vv, vo, vkv, vws

    # ---- decode leg: prefill once, then timed recurrent steps on the fp32 state ----
    dw = inputs.WORKLOADS["decode"]
    gen = torch.Generator(dev)
    gen.manual_seed(1000 + rank)
    BHd = (dw.B, dw.H, dw.d)
    nsteps = args.decode_steps or dw.decode_steps
    qs = torch.nn.functional.silu(torch.randn((nsteps,) + BHd, generator=gen, device=dev)).to(torch.bfloat16)
    ks = torch.nn.functional.silu(torch.randn((nsteps,) + BHd, generator=gen, device=dev)).to(torch.bfloat16)
    vs = torch.randn((nsteps, dw.B, dw.H, dw.e), generator=gen, device=dev).to(torch.bfloat16)
    # the state the steps start from is the one the bf16 prefill over dw.N tokens leaves behind (la_fwd, kv_out)
    kv = torch.empty((dw.B, dw.H, dw.d, dw.e), dtype=torch.float32, device=dev)
    pshape = la.make_shape(dw.B, dw.H, dw.N, dw.d, dw.e, torch.bfloat16, torch.float32)
    pq = torch.nn.functional.silu(torch.randn((dw.B, dw.H, dw.N, dw.d), generator=gen, device=dev)).to(torch.bfloat16)
    pk = torch.nn.functional.silu(torch.randn((dw.B, dw.H, dw.N, dw.d), generator=gen, device=dev)).to(torch.bfloat16)
    pv = torch.randn((dw.B, dw.H, dw.N, dw.e), generator=gen, device=dev).to(torch.bfloat16)
    po = torch.empty((dw.B, dw.H, dw.N, dw.e), dtype=torch.float32, device=dev)
    dlam = inputs.decay_rates(dw.H, dw.l_over_L)
    la.la_fwd(pshape, pq, pk, pv, dlam, po, None, kv, la.alloc_workspace(la.LA_OP_FWD, pshape, dev), stream)
    barrier()
    la.device_status()
    del pq, pk, pv, po
    dshape = la.make_shape(dw.B, dw.H, 1, dw.d, dw.e, torch.bfloat16, torch.float32)
    od = torch.empty((nsteps, dw.B, dw.H, dw.e), dtype=torch.float32, device=dev)

    def decode_loop():
        for s in range(nsteps):
            la.la_decode_step(dshape, qs[s], ks[s], vs[s], dlam, kv, od[s], stream)

    decode_loop()  # warm-up pass (256 launches)
    barrier()
    d0, d1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    reps = 3
    d0.record(stream)
    for _ in range(reps):
        decode_loop()
    d1.record(stream)
    barrier()
    dec_ms = max_over_ranks(d0.elapsed_time(d1) / (reps * nsteps))
    dec_bytes = dw.B * dw.H * (2 * dw.d * dw.e * 4 + 2 * (2 * dw.d + dw.e) + 4 * dw.e)
    dec_gbs = dec_bytes / (dec_ms * 1e-3) / 1e9
    clocks = None
    if args.only == "decode":
        if rank == 0:
            print(json.dumps({"only": "decode", "us_per_step": dec_ms * 1e3, "achieved_gbs": dec_gbs}), flush=True)
        return

    # ---- end to end through the host-buffer entry point ----
    e2e = None
    try:
        arena = torch.empty(la.host_arena_bytes(shape), dtype=torch.uint8, device=dev)
        hq, hk, hv, hdo = (x.cpu().pin_memory() for x in (q, k, v, do))
        ho = torch.empty(o.shape, dtype=out_dtype).pin_memory()
        hdq, hdk, hdv = (torch.empty(dq.shape, dtype=out_dtype).pin_memory() for _ in range(3))
        e2e_steps = max(1, min(args.steps, 3))
        la.la_fwd_bwd_host(shape, hq, hk, hv, hdo, lam, ho, hdq, hdk, hdv, arena, stream)  # warm-up
        barrier()
        h0, h1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        h0.record(stream)
        for _ in range(e2e_steps):
            la.la_fwd_bwd_host(shape, hq, hk, hv, hdo, lam, ho, hdq, hdk, hdv, arena, stream)
        h1.record(stream)
        barrier()
        la.device_status()
        e2e_ms = max_over_ranks(h0.elapsed_time(h1) / e2e_steps)
        h2d = sum(x.numel() * x.element_size() for x in (hq, hk, hv, hdo))
        d2h = sum(x.numel() * x.element_size() for x in (ho, hdq, hdk, hdv))
        e2e = {"value": world * th * F / (e2e_ms * 1e-3) / 1e12, "unit": UNIT, "ms_per_step": e2e_ms,
               "steps": e2e_steps, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "api": "la_fwd_bwd_host (pinned host buffers)"}
    except Exception as ex:  # keep the device-resident numbers even if pinned memory is unavailable
        e2e = {"value": None, "unit": UNIT, "error": str(ex)[:200]}

    # ---- the two smaller model shapes (reported beside the headline, same step and timing rules) ----
    others = {}
    for name in ("pr1_ref", "385m", "1b"):
        ow = inputs.WORKLOADS[name]
        od_ = inputs.device_randn_like_workload(name, dev, seed=rank)
        oshape = la.make_shape(ow.B, ow.H, ow.N, ow.d, ow.e, ow.in_dtype, out_dtype)
        oo = torch.empty((ow.B, ow.H, ow.N, ow.e), dtype=out_dtype, device=dev)
        odq, odk, odv = (torch.empty((ow.B, ow.H, ow.N, ow.d), dtype=out_dtype, device=dev) for _ in range(3))
        owf = la.alloc_workspace(la.LA_OP_FWD, oshape, dev)
        owb = la.alloc_workspace(la.LA_OP_BWD, oshape, dev)
        # these shapes fit L2 (126 MB), so a buffer larger than L2 is rewritten between timed steps
        flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

        def ostep():
            la.la_fwd(oshape, od_["q"], od_["k"], od_["v"], od_["lam"], oo, None, None, owf, stream)
            la.la_bwd(oshape, od_["q"], od_["k"], od_["v"], od_["do"], od_["lam"], odq, odk, odv, None, None, None, owb,
                      stream, fwd_workspace=owf)

        for _ in range(max(3, args.warmup)):
            ostep()
        barrier()
        osteps = max(1, min(args.steps, 10))
        tot = 0.0
        for _ in range(osteps):
            flush.fill_(1)
            a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a0.record(stream)
            ostep()
            a1.record(stream)
            a1.synchronize()
            tot += a0.elapsed_time(a1)
        barrier()
        la.device_status()
        oms = max_over_ranks(tot / osteps)
        # per-launch breakdown from a separate profiled loop (L2 not flushed here: these are kernel times only)
        l0 = la.launch_count()
        la.profile_enable(True)
        for _ in range(3):
            ostep()
        barrier()
        la.profile_enable(False)
        oprof = la.profile_collect()
        olaunch = (la.launch_count() - l0) / 3
        oF = flops_per_token_head(ow.d)
        obytes = ow.token_heads * bytes_per_token_head(ow.d, ob, "step")
        if ow.in_dtype == torch.float32:
            obytes += ow.token_heads * 2 * 7 * ow.d  # q,k,v read twice and dO once, two bytes more each
        oroof = max(ow.token_heads * oF / (peaks["bf16_tflops_sustained"] * 1e12), obytes / (peaks["hbm_gbs"] * 1e9))
        others[name] = {"shape": "B=%d,H=%d,N=%d,d=e=%d" % (ow.B, ow.H, ow.N, ow.d), "ms_per_step": oms,
                        "tflops": world * ow.token_heads * oF / (oms * 1e-3) / 1e12,
                        "tokens_per_s": world * ow.B * ow.N / (oms * 1e-3),
                        "step_roofline_frac": oroof * 1e3 / oms, "l2": "flushed between timed steps",
                        "launches_per_step": olaunch,
                        "kernel_ms_per_step": {kn: ms / 3 for kn, (ms, _) in oprof.items()},
                        "kernel_launches_per_step": {kn: c / 3 for kn, (_, c) in oprof.items()},
                        "bound": ("latency (a few short launches over a shape that fits L2)"
                                  if ow.token_heads < 200000 else "hbm"),
                        "kernels": ("fp32 CUDA cores" if ow.in_dtype == torch.float32 else
                                    "tcgen05 (one thread block per head and segment)")}
        del od_, oo, odq, odk, odv, owf, owb, flush

    clocks = sampler.stop() if rank == 0 else None

    # ---- the same step held for about two seconds (last GPU leg, so that it heats nothing that is timed after it):
    # the headline loop above is a burst of a few tens of milliseconds from a GPU that was not under load just before;
    # held for longer, the step runs into the board's power limit and the SM clock settles below its maximum
    sustained = None
    if train_steps and world == 1:
        s_sampler = ClockSampler(local_rank)
        n_hold = max(20, int(2000.0 / ms_step))
        n_timed = n_hold // 2
        for _ in range(n_hold - n_timed):
            step()
        s_sampler.start()
        h0, h1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        h0.record(stream)
        for _ in range(n_timed):
            step()
        h1.record(stream)
        torch.cuda.synchronize()
        la.device_status()
        s_clocks = s_sampler.stop()
        s_ms = h0.elapsed_time(h1) / n_timed
        sustained = {"what": "the same fwd+bwd step after %d untimed steps, mean of the next %d (about a second each)"
                             % (n_hold - n_timed, n_timed),
                     "ms_per_step": s_ms, "value": th * F / (s_ms * 1e-3) / 1e12, "unit": "TFLOP/s",
                     "step_roofline_frac": t_roof * 1e3 / s_ms, "clocks": s_clocks}

    cpu = cpu_baseline() if (rank == 0 and world == 1 and not args.no_cpu_baseline) else None

    if rank == 0:
        seg = la.segment_length(shape)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "ms_per_step_median": ms_median, "ms_per_step_min": ms_min,
            "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "%s: B=%d,H=%d,N=%d,d=e=%d per GPU, bf16 in, fp32 accumulate, fp32 out; "
                                   "q,k=SiLU(N(0,1)), v,dO=N(0,1), lambda_h=exp(-(8h/H)(1-0.9))"
                                   % (WORKLOAD, w.B, w.H, w.N, w.d),
                       "segment_length": seg, "l2": "inputs (2.1 GB) and outputs (4.3 GB) exceed L2; no flush needed",
                       "parallelism": "replicas x%d (no collective on the path)" % world,
                       "flops_per_token_head": F, "flop_conventions": flop_conventions(w.d),
                       "tflops_by": {kn: world * th * fv / (ms_step * 1e-3) / 1e12
                                     for kn, fv in flop_conventions(w.d).items()},
                       "bytes_per_token_head": bytes_per_token_head(w.d, ob, "step"),
                       "timing": "headline loop: profiling off, CUDA events on the launching stream; "
                                 "kernel_ms_per_step and roofline come from a second, separately run profiled loop; the board reaches its 1000 W power limit after about 40 ms of this step (15-18 steps from idle) and lowers the SM clock, so a run with more timed steps than that mixes both regimes: ms_per_step_median and ms_per_step_min show the full-clock steps, `sustained` the settled state"},
            "tokens_per_s": world * w.B * w.N / (ms_step * 1e-3),
            "clocks": clocks, "e2e": e2e, "gpu_launches": launches, "other_workloads": others,
            "kernel_ms_per_step": {kname: ms / prof_steps for kname, (ms, _) in prof.items()},
            "kernel_launches_per_step": {kname: c / prof_steps for kname, (_, c) in prof.items()},
            "fwd_ms": split_ms.get("fwd"), "bwd_ms": split_ms.get("bwd"), "gated_forward": gated, "lrpe_d": lrpe, "sequence_parallel": seqpar_leg, "varlen_prefill": varlen_leg, "sustained": sustained,
            "roofline": {"scope": "ONE kernel, the dominant one; the whole-step figure the target is stated on is step_roofline",
                         "kernel": "full-width block walk (tc_walk_full_kernel), single-job launches (O and dQ)", "bound": "hbm",
                         "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": (achieved / peaks["hbm_gbs"]) if achieved else None,
                         "traffic": WALK_DRAM_BYTES_PER_TOKEN_HEAD * th,
                         "traffic_note": "ncu dram read bytes of a 524288-token-head launch scaled by token-heads + the full fp32 output",
                         "peak_source": peaks["source"],
                         "avg_launch_ms": walk_avg_ms, "launches": walk_n, "bytes_per_launch": walk_bytes,
                         "walk_pair": {"what": "the dV and dK walks of the backward pass in one launch",
                                       "avg_launch_ms": pair_avg_ms, "launches": pair_n, "bytes_per_launch": pair_bytes,
                                       "achieved": pair_gbs,
                                       "frac": (pair_gbs / peaks["hbm_gbs"]) if pair_gbs else None}},
            "step_roofline": {"scope": "whole fwd+bwd step against max(flops / tensor peak, algorithmic bytes / HBM peak)",
                              "t_roofline_ms": t_roof * 1e3, "frac": t_roof * 1e3 / ms_step,
                              "bytes": step_bytes, "flops": th * F, "peak_source": peaks["source"],
                              "datasheet": {"hbm_gbs": 8000.0, "bf16_tflops": 2250.0,
                                            "t_roofline_ms": t_roof_datasheet * 1e3,
                                            "frac": t_roof_datasheet * 1e3 / ms_step}},
            "decode": {"tok_per_s": world * dw.B / (dec_ms * 1e-3), "us_per_step": dec_ms * 1e3,
                       "workload": "batch %d, H=%d, d=e=%d, fp32 state left by a %d-token bf16 prefill (la_fwd), %d steps"
                                   % (dw.B, dw.H, dw.d, dw.N, nsteps),
                       "achieved_gbs": dec_gbs, "frac_of_hbm_peak": dec_gbs / peaks["hbm_gbs"],
                       "bytes_per_step": dec_bytes},
            "cpu_baseline": cpu,
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--only", default="all", choices=["all", "train", "decode"],
                    help="profiling aid: run only the fwd+bwd leg or only the decode leg (prints a short line)")
    ap.add_argument("--small", action="store_true",
                    help="profiling aid: 16 heads x 32768 tokens of the workload for the fwd+bwd leg")
    ap.add_argument("--decode-steps", type=int, default=0, help="profiling aid: recurrent steps per pass")
    ap.add_argument("--seg-len", type=int, default=0,
                    help="experiment: segment length in tokens (multiple of 128) instead of the library's choice")
    ap.add_argument("--precision", type=int, default=-1,
                    help="experiment: LA_SPLIT_* bits for the tensor-core kernels (-1 = library default, all on; "
                         "anything else does not meet the parity tolerance on every head)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
