#!/usr/bin/env python
"""Benchmark of the fused-attention hot path on B200.

One "step" = one pass of the hot path over the headline workload: D=128, H=16, 16384 total
tokens, non-causal AND causal, one launch set per sequence length of the sweep 1024..16384
(batch = 16384 / seqlen), forward + backward (`--pass fwd`: forward only), plus the causal
forward at seqlen 32768 (batch 1).  FLOPs are counted as 4*B*H*Sq*Sk*D per forward (halved when
causal) and 2.5x that per backward.

Prints ONE JSON line (see the keys below).  `--impl reference` times the float64 CPU oracle
on a bounded sample of the same workload instead.
"""

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

import numpy as np

SEQLENS = (1024, 2048, 4096, 8192, 16384)
LONG_SEQLEN = 32768          # forward, causal, batch 1 (the last member of the causal forward sweep)
TOKENS, HEADS, HEAD_DIM = 16384, 16, 128
PAPER_PEAK_TFLOPS = 2250.0
METRIC = "attention fwd/bwd TFLOPs/s (BF16, D=128, causal & non) and % of B200 BF16 peak"
# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the main kernel of each pass,
# each from the one ncu capture named beside it (a 16384-token member of the sweep; compulsory traffic
# depends on the token count only, K/V re-reads are served by L2).
NCU_TRAFFIC = {
    "fwd": {"bytes": 260.57e6 + 59.53e6,
            "capture": "profiles/ncu_fwd_pipe_kernel_S4096_B4_H16_D128.txt (one launch, B=4 S=4096 non-causal; "
                       "the causal launch of the same shape: 202.1e6 + 51.2e6)"},
    "bwd": {"bytes": 405.33e6 + 223.53e6,
            "capture": "profiles/ncu_bwd_fused_kernel_S4096_B4_H16_D128.txt (one launch, B=4 S=4096 non-causal)"},
}
ROOFLINE_KERNEL = {
    "fwd": "fwd_pipe_kernel (timed as fa_fwd: one launch; the shortest members run fwd_tile_kernel, see fa.h)",
    "bwd": "bwd_fused_kernel (timed as fa_bwd: preprocess + main + dQ conversion; the main kernel is 0.96 of it)",
}


def fwd_flops(B, H, Sq, Sk, D, causal):
    return 4.0 * B * H * Sq * Sk * D / (2.0 if causal else 1.0)


def max_over_ranks(ms, world, device):
    """Slowest rank's time: the job is as slow as its slowest replica (all-reduce MAX when world > 1)."""
    if world <= 1:
        return float(ms)
    import torch
    import torch.distributed as dist

    tt = torch.tensor([float(ms)], dtype=torch.float64, device=device)
    dist.all_reduce(tt, op=dist.ReduceOp.MAX)
    return float(tt.item())


def replicas_throughput(flops_per_rank_step, steps, ms_max, world):
    """Whole-job TFLOPs/s of `world` independent replicas (no collective on the data path)."""
    return world * flops_per_rank_step * steps / (ms_max * 1e-3) / 1e12


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return float(d["bf16_tflops"]), float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), "measured"
    return 1590.0, 1400.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.lines = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0, t1):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        rows = [l for (ts, l) in self.lines if t0 <= ts <= t1] or [l for (_, l) in self.lines]
        for l in rows:
            parts = [x.strip() for x in l.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0]))
                smax.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def workload_text(with_bwd, masks, seqlens, long_member, D=HEAD_DIM):
    mask_txt = {"both": "non-causal and causal", "causal": "causal", "noncausal": "non-causal"}[masks]
    long_txt = f", plus the causal forward at seqlen {LONG_SEQLEN} (batch 1)" if long_member else ""
    return (f"{'fwd+bwd' if with_bwd else 'fwd'} {mask_txt} D={D} H={HEADS * HEAD_DIM // D}, 16384 total tokens, seqlen sweep "
            f"{','.join(map(str, seqlens))} (batch = 16384/seqlen){long_txt}")


def oracle_sample(seconds_target=15.0, rounds_cap=64, with_bwd=True, masks=(False, True)):
    """Times the float64 oracle (as it stands) on a bounded sample of the step: whole (batch, head)
    slices of the S=4096 member, one forward (and one backward) per mask setting per round."""
    from oracle.attention import attn_bwd_head, attn_fwd_head
    from paper_2603_05451_b200 import inputs

    S, D = 4096, HEAD_DIM
    t = inputs.make_qkv(2000, 1, 1, 1, S, S, D, with_do=True)
    q, k, v, d_o = (t[n][1][0, :, 0, :] for n in ("q", "k", "v", "do"))
    scale = D ** -0.5
    t0 = time.perf_counter()
    n, flops = 0, 0.0
    while True:
        for causal in masks:
            attn_fwd_head(q, k, v, scale, causal)
            flops += fwd_flops(1, 1, S, S, D, causal)
            if with_bwd:
                attn_bwd_head(q, k, v, d_o, scale, causal)
                flops += 2.5 * fwd_flops(1, 1, S, S, D, causal)
        n += 1
        el = time.perf_counter() - t0
        if el >= seconds_target or n >= rounds_cap:
            break
    tflops = flops / el / 1e12
    try:
        import threadpoolctl
        cores = max([p.get("num_threads", 1) for p in threadpoolctl.threadpool_info()] + [1])
    except Exception:
        cores = os.cpu_count() or 1
    what = ("forward + backward" if with_bwd else "forward") + " of one (batch, head) slice of the S=4096 D=128 member, " + \
           " and ".join("causal" if c else "non-causal" for c in masks)
    return tflops, cores, f"{n} rounds of: {what}; {el:.1f} s", el, n


def run_reference(args, rank):
    if rank != 0:
        return
    masks = {"both": (False, True), "causal": (True,), "noncausal": (False,)}[args.masks]
    with_bwd = args.which == "fwdbwd"
    seqlens = [int(s) for s in args.seqlens.split(",")]
    vals, total_t = [], 0.0
    per_step = max(2.0, min(20.0, 150.0 / max(1, args.steps + args.warmup)))
    for i in range(args.warmup + args.steps):
        tf, cores, sample, el, n = oracle_sample(seconds_target=per_step, with_bwd=with_bwd, masks=masks)
        if i >= args.warmup:
            vals.append(tf)
            total_t += el
    value = float(np.mean(vals))
    line = {
        "impl": "reference", "metric": METRIC, "value": value,
        "unit": "TFLOPs/s", "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * total_t / max(1, args.steps), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_text(with_bwd, args.masks, seqlens, True in masks and not args.no_long),
                   "sample": "each step is a bounded sample of that workload: " + sample},
        "cpu_baseline": {"value": value, "unit": "TFLOPs/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "TFLOPs/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def throughput_table(launches, tokens=TOKENS):
    """Markdown table of burst throughput (CUDA-event mean of `launches` launches after 3 warm-ups) on
    the shapes of the paper's Section 5: `tokens` tokens in total (16384, or the paper's 32768; one
    sequence at seqlen 32768 either way), hidden size 2048, i.e. 16 heads of 128 or 32 heads of 64; FLOPs = 4 B H S^2 D forward (half that when causal),
    2.5 times that backward; fractions are of the 2250 TFLOPs/s dense BF16 peak."""
    import torch

    from paper_2603_05451_b200 import binding

    binding.lib()

    def timed(fn):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(launches):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / launches

    gen = torch.Generator(device="cuda").manual_seed(7)
    print("| D | H | seqlen | batch | causal | fwd TFLOPs/s | of 2250 | bwd TFLOPs/s | of 2250 |")
    print("|---|---|---|---|---|---|---|---|---|")
    for D, H in ((128, 16), (64, 32)):
        for causal in (False, True):
            for S in (1024, 2048, 4096, 8192, 16384, 32768):
                B = max(1, tokens // S)
                q, k, v, d_o = (torch.randn((B, S, H, D), generator=gen, device="cuda").to(torch.bfloat16)
                                for _ in range(4))
                o = torch.empty_like(q)
                lse = torch.empty((B, H, S), dtype=torch.float32, device="cuda")
                dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
                ws = torch.empty(binding.fa_bwd_workspace_bytes(B, H, H, S, S, D), dtype=torch.uint8, device="cuda")
                scale = D ** -0.5
                ms_f = timed(lambda: binding.fa_fwd(q, k, v, scale, causal, o=o, lse=lse))
                ms_b = timed(lambda: binding.fa_bwd(q, k, v, o, lse, d_o, scale, causal, dq=dq, dk=dk, dv=dv,
                                                    workspace=ws))
                assert binding.fa_last_device_status() == 0
                fl = fwd_flops(B, H, S, S, D, causal)
                tf, tb = fl / ms_f / 1e9, 2.5 * fl / ms_b / 1e9
                print(f"| {D} | {H} | {S} | {B} | {'yes' if causal else 'no'} | {tf:.0f} | {tf / PAPER_PEAK_TFLOPS:.1%} | "
                      f"{tb:.0f} | {tb / PAPER_PEAK_TFLOPS:.1%} |", flush=True)
                del q, k, v, d_o, o, lse, dq, dk, dv, ws


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--pass", dest="which", default="fwdbwd", choices=["fwd", "fwdbwd"])
    ap.add_argument("--masks", default="both", choices=["both", "causal", "noncausal"])
    ap.add_argument("--seqlens", default=",".join(str(s) for s in SEQLENS))
    ap.add_argument("--no-long", action="store_true", help="leave out the causal forward at seqlen 32768")
    ap.add_argument("--head-dim", type=int, default=HEAD_DIM, choices=[64, 128],
                    help="head dimension (hidden size 2048: 16 heads of 128, the headline; or 32 heads of 64, for profiles)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--table", action="store_true",
                    help="print forward / backward TFLOPs/s over head dim 64/128, seqlen 1k-32k, causal and not, and exit")
    ap.add_argument("--table-tokens", type=int, default=TOKENS, help="total tokens of the --table sweep (16384 or 32768)")
    args = ap.parse_args()
    args.warmup = max(3, args.warmup)

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        run_reference(args, rank)
        return
    if args.table:
        if rank == 0:
            throughput_table(max(3, min(args.steps, 10)), args.table_tokens)
        return

    import torch
    import torch.distributed as dist

    from paper_2603_05451_b200 import binding, inputs

    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    binding.lib()  # fail loudly if the CUDA library is missing

    seqlens = [int(s) for s in args.seqlens.split(",")]
    masks = {"both": (False, True), "causal": (True,), "noncausal": (False,)}[args.masks]
    D = args.head_dim
    H = HEADS * HEAD_DIM // D
    scale = D ** -0.5
    with_bwd = args.which == "fwdbwd"
    # The step's members: (seqlen, batch, causal, backward too?)
    members = [(S, TOKENS // S, c, with_bwd) for c in masks for S in seqlens]
    if True in masks and not args.no_long:
        members.append((LONG_SEQLEN, 1, True, False))
    max_tokens = max(S * B for S, B, _, _ in members)

    # Seeded synthetic inputs (i.i.d. N(0,1) rounded to bf16), generated on the host and staged in
    # pinned memory; one flat token buffer is viewed as [B, S, H, D] for every member of the step.
    names = ("q", "k", "v") + (("do",) if with_bwd else ())
    host = {}
    for n in names:
        bits, _ = inputs.make_tensor(3000 + rank, n, (max_tokens, H, D), values=False)
        host[n] = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).pin_memory()
    dev = {n: host[n].cuda(non_blocking=True) for n in names}
    o = torch.empty_like(dev["q"])
    lse = torch.empty(max_tokens * H, dtype=torch.float32, device="cuda")
    host_o = torch.empty_like(host["q"]).pin_memory()
    host_lse = torch.empty(max_tokens * H, dtype=torch.float32).pin_memory()
    ws_bytes = 0
    if with_bwd:
        dq, dk, dv = (torch.empty(TOKENS, H, D, dtype=torch.bfloat16, device="cuda") for _ in range(3))
        ws_bytes = max(binding.fa_bwd_workspace_bytes(TOKENS // S, H, H, S, S, D) for S in seqlens)
        ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
        host_g = [torch.empty(TOKENS, H, D, dtype=torch.bfloat16).pin_memory() for _ in range(3)]
    torch.cuda.synchronize()

    def view(t, S, B):
        return t[:B * S].view(B, S, H, D)

    def run_member(m, bufs, stream=None):
        S, B, causal, bwd = m
        i, oo, ll = bufs["in"], bufs["o"], bufs["lse"]
        binding.fa_fwd(view(i["q"], S, B), view(i["k"], S, B), view(i["v"], S, B), scale, causal,
                       o=view(oo, S, B), lse=ll[:B * H * S].view(B, H, S), stream=stream)
        if bwd:
            g = bufs["g"]
            binding.fa_bwd(view(i["q"], S, B), view(i["k"], S, B), view(i["v"], S, B), view(oo, S, B),
                           ll[:B * H * S].view(B, H, S), view(i["do"], S, B), scale, causal, dq=view(g[0], S, B),
                           dk=view(g[1], S, B), dv=view(g[2], S, B), workspace=bufs["ws"], stream=stream)
        return 1 + (binding.BWD_LAUNCHES if bwd else 0)

    main_bufs = {"in": dev, "o": o, "lse": lse}
    if with_bwd:
        main_bufs.update(g=[dq, dk, dv], ws=ws)

    def step(events=None):
        n = 0
        for m in members:
            if events is None:
                n += run_member(m, main_bufs)
                continue
            # per-pass timing: events around the forward launch and around the backward launches
            S, B, causal, bwd = m
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            n += run_member((S, B, causal, False), main_bufs)
            e1.record()
            events.append(("fwd", S, causal, e0, e1))
            if bwd:
                binding.fa_bwd(view(dev["q"], S, B), view(dev["k"], S, B), view(dev["v"], S, B), view(o, S, B),
                               lse[:B * H * S].view(B, H, S), view(dev["do"], S, B), scale, causal, dq=view(dq, S, B),
                               dk=view(dk, S, B), dv=view(dv, S, B), workspace=ws)
                e2 = torch.cuda.Event(enable_timing=True)
                e2.record()
                events.append(("bwd", S, causal, e1, e2))
                n += binding.BWD_LAUNCHES
        return n

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def member_flops(m, kind=None):
        S, B, causal, bwd = m
        f = fwd_flops(B, H, S, S, D, causal)
        if kind == "fwd":
            return f
        if kind == "bwd":
            return 2.5 * f
        return f * (3.5 if bwd else 1.0)

    flops_step = sum(member_flops(m) for m in members)

    for _ in range(args.warmup):
        step()
    barrier()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    barrier()
    events = []
    t_wall0 = time.time()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    launches = 0
    for _ in range(args.steps):
        launches += step(events)
    ev1.record()
    barrier()
    t_wall1 = time.time()
    ms_total = ev0.elapsed_time(ev1)
    clocks = sampler.stop(t_wall0, t_wall1) if rank == 0 else None
    if binding.fa_last_device_status() != 0:
        raise RuntimeError("a device-side wait timed out during the benchmark")
    ms_total = max_over_ranks(ms_total, world, "cuda")

    # End-to-end through the public API with HOST buffers: pinned host -> device copies of the
    # step's inputs and device -> host reads of its results are inside the timed region.
    e2e_steps = max(3, min(args.steps, 10))
    h2d = sum(len(names) * S * B * H * D * 2 for S, B, _, _ in members)
    d2h = sum(S * B * H * D * 2 + S * B * H * 4 + (3 * S * B * H * D * 2 if bwd else 0) for S, B, _, bwd in members)

    # Every member of the step is its own request: inputs in, kernels, results out.  As a caller
    # of the C ABI would, the three phases run on three streams with two sets of device buffers, so
    # the copy-in of request i+1 and the copy-out of request i-1 overlap the kernels of request i
    # (the library's entry points take the stream; nothing else about them changes).
    s_in, s_run, s_out = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
    sets = []
    for _ in range(2):
        b = {"in": {n: torch.empty_like(dev[n]) for n in names}, "o": torch.empty_like(o), "lse": torch.empty_like(lse)}
        if with_bwd:
            b["g"] = [torch.empty_like(dq) for _ in range(3)]
            b["ws"] = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
        b["in_ready"], b["run_done"], b["out_done"] = (torch.cuda.Event() for _ in range(3))
        sets.append(b)
    torch.cuda.synchronize()
    request = [0]

    def e2e_step():
        for m in members:
            S, B, causal, bwd = m
            n_tok = S * B
            b = sets[request[0] & 1]
            first_use = request[0] < 2
            request[0] += 1
            with torch.cuda.stream(s_in):
                if not first_use:
                    s_in.wait_event(b["run_done"])  # the kernels that read this input set have finished
                for n in names:
                    if n == "do" and not bwd:
                        continue
                    b["in"][n][:n_tok].copy_(host[n][:n_tok], non_blocking=True)
                b["in_ready"].record(s_in)
            with torch.cuda.stream(s_run):
                s_run.wait_event(b["in_ready"])
                if not first_use:
                    s_run.wait_event(b["out_done"])  # the previous results of this set have left the device
                run_member(m, b, stream=s_run)
                b["run_done"].record(s_run)
            with torch.cuda.stream(s_out):
                s_out.wait_event(b["run_done"])
                if bwd:
                    for g, hg in zip(b["g"], host_g):
                        hg[:n_tok].copy_(g[:n_tok], non_blocking=True)
                host_o[:n_tok].copy_(b["o"][:n_tok], non_blocking=True)
                host_lse[:n_tok * H].copy_(b["lse"][:n_tok * H], non_blocking=True)
                b["out_done"].record(s_out)

    e2e_step()
    barrier()
    ea, eb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for st in (s_in, s_run, s_out):
        st.wait_stream(torch.cuda.current_stream())
    ea.record(s_in)  # the first thing in the timed region is a copy-in
    for _ in range(e2e_steps):
        e2e_step()
    s_out.wait_stream(s_in)
    s_out.wait_stream(s_run)
    eb.record(s_out)  # the last thing is a copy-out
    barrier()
    e2e_ms = max_over_ranks(ea.elapsed_time(eb), world, "cuda")

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    value = replicas_throughput(flops_step, args.steps, ms_total, world)
    e2e_value = replicas_throughput(flops_step, e2e_steps, e2e_ms, world)

    # Roofline per pass: counted FLOPs of all its launches / their summed CUDA-event time.
    per = {}
    for kind, S, causal, a, b in events:
        per.setdefault((kind, S, causal), []).append(a.elapsed_time(b))
    burst, sustained, src = measured_peaks()
    # The kernels are timed inside a loop that keeps the GPU busy for seconds (power cap active), so the
    # sustained GEMM figure is the matching denominator; a run shorter than a second is a burst.
    long_run = ms_total > 1000.0
    peak = sustained if long_run else burst

    def roofline(kind):
        keys = [k for k in per if k[0] == kind]
        if not keys:
            return None
        ms = sum(sum(per[k]) for k in keys)
        fl = sum(len(per[k]) * fwd_flops(max(1, TOKENS // k[1]), H, k[1], k[1], D, k[2]) * (2.5 if kind == "bwd" else 1.0)
                 for k in keys)
        achieved = fl / (ms * 1e-3) / 1e12
        cap = NCU_TRAFFIC[kind]
        return {"bound": "tensor", "kernel": ROOFLINE_KERNEL[kind], "achieved": achieved, "peak": peak,
                "unit": "TFLOP/s", "frac": achieved / peak,
                "peak_source": f"bf16 GEMM {'sustained' if long_run else 'burst'}, {src}",
                "frac_of_burst_peak": achieved / burst, "frac_of_sustained_peak": achieved / sustained,
                "frac_of_2250": achieved / PAPER_PEAK_TFLOPS, "traffic": cap["bytes"], "traffic_capture": cap["capture"]}

    per_seqlen = {}
    for (kind, S, causal), v in sorted(per.items()):
        tf = fwd_flops(max(1, TOKENS // S), H, S, S, D, causal) * (2.5 if kind == "bwd" else 1.0) / (np.mean(v) * 1e-3) / 1e12
        per_seqlen[f"{kind}_{'causal' if causal else 'full'}_S{S}"] = {
            "ms": float(np.mean(v)), "tflops": tf, "frac_of_2250": tf / PAPER_PEAK_TFLOPS}

    cpu = None
    if not args.no_cpu_baseline:
        tf, cores, sample, _, _ = oracle_sample(with_bwd=with_bwd, masks=masks)
        cpu = {"value": tf, "unit": "TFLOPs/s", "cores": cores, "kind": "oracle", "sample": sample}

    line = {
        "metric": METRIC,
        "value": value, "unit": "TFLOPs/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_total / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {
            "workload": workload_text(with_bwd, args.masks, seqlens, members[-1][0] == LONG_SEQLEN, D),
            "inputs": "i.i.d. N(0,1) bf16, seeded; Q+K+V+O = 256 MiB per launch, larger than the 126 MB L2 (no flush)",
            "multi_gpu": "replicas only: every rank runs the same workload, no collective on the data path",
        },
        "frac_of_2250_peak": value / world / PAPER_PEAK_TFLOPS,
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": "TFLOPs/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": launches,
        "roofline": roofline("bwd" if with_bwd else "fwd"),
        "cpu_baseline": cpu,
        "per_seqlen": per_seqlen,
    }
    if with_bwd:
        line["roofline_fwd"] = roofline("fwd")
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
