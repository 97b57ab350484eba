#!/usr/bin/env python
"""LinSimp hot-path benchmark.

    python bench.py --gpus N --steps K --warmup W [--impl reference]

One "step" is one forward + backward of the whole hot path over one batch of the
long-context workload (B=2, H=16, T=16384, d=128, m=128, W=64, bf16 inputs,
fp32 state).  Prints ONE JSON line (rank 0).  `value` is tokens/s with inputs
resident in HBM; `e2e` repeats it through the public API with host buffers
(pinned host -> device copies of the inputs and device -> host copies of the
output and gradients inside the timed region); `decode` reports the
single-token step in GB/s; `roofline` covers the dominant kernel of the timed
region; `cpu_baseline` is the fp64 oracle timed on the host cores.
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

WORKLOAD = dict(name="C3", B=2, H=16, T=16384, d=128, m=128, W=64, seed=30)
DECODE = dict(name="C5", n_seq=256, H=16, d=128, m=128, W=64, prefix=16384, steps=1024, seed=50)
METRIC = "linsimp_fwd_bwd_tokens_per_s_T16k"
FP32_FMA_PEAK_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12     # CUDA-core fp32: SMs x lanes x 2 x max clock


def ncu_dram_bytes():
    """DRAM bytes (read + write) per launch of the tile kernels as a profiler capture of a small case counted them:
    {"T": tokens per sequence of the captured case, "kernels": {name: bytes per launch}}, from the data file kept
    beside the capture's summary; None when the file is missing."""
    path = os.path.join(ROOT, "profiles", "ncu_dram_bytes_small_case.json")
    try:
        with open(path) as f:
            return json.load(f)
    except (OSError, ValueError):
        return None


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=p["hbm_gbs"], bf16_burst=p["bf16_tflops"], bf16_sustained=p["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_burst=1590.0, bf16_sustained=1400.0, source="fallback")


def fwd_flops_per_token_head(d, m, W):
    """Algorithmic forward FLOPs: feature projection + state contraction for W anchors and the key."""
    return 2.0 * m * (d + d) * (W + 1)


def decode_bytes_per_unit(d, m, W):
    """Algorithmic bytes per (sequence, head) per decode step: state r+w, normaliser r+w, ring read,
    ring write, five inputs, one output (bf16 tokens, fp32 state)."""
    return 2 * m * d * 4 + 2 * m * 4 + W * 2 * d * 2 + 2 * d * 2 + 5 * d * 2 + d * 2


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []
        self.first = 0
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.FIELDS,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._pump, daemon=True)
        self.thread.start()

    def wait_ready(self, timeout=15.0):
        """Blocks until the first sample has arrived: nvidia-smi's start-up (NVML initialisation over all GPUs of the
        host) can hold up kernel launches for hundreds of milliseconds, so it must be over before anything is timed."""
        t0 = time.time()
        while self.proc is not None and not self.lines and time.time() - t0 < timeout and self.proc.poll() is None:
            time.sleep(0.02)

    def mark(self):
        """Samples from here on belong to the timed region."""
        self.first = len(self.lines)

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, power, reasons = [], [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        timed = self.lines[self.first:] or self.lines
        for ln in timed:
            parts = [x.strip() for x in ln.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1]))
                smax.append(float(parts[2]))
                power.append(float(parts[3]))
            except ValueError:
                continue
            for nm, val in zip(names, parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        if not sm:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["no samples"])
        sm.sort()
        return dict(sm_mhz=sm[len(sm) // 2], sm_max_mhz=max(smax), power_w_max=max(power), samples=len(sm),
                    reasons=sorted(reasons))


def cpu_oracle_sample(cfg, tokens, max_units=32):
    """Times the C fp64 oracle (fwd + bwd) on the first `tokens` tokens of `cores` (b,h) units of the workload.
    Returns (tokens/s of a layer with H heads, cores, description, seconds)."""
    import numpy as np
    from oracle import c_ref
    from paper_2608_09307_b200 import synth
    c_ref.build()
    cores = c_ref.threads()
    n_units = max(1, min(max_units, cores))
    t = synth.make_inputs(1, n_units, tokens, cfg["d"], cfg["seed"], "bf16", "rms")
    om = synth.make_omega(cfg["d"], cfg["m"]).double().numpy()
    arr = {k_: v_[0].double().numpy() for k_, v_ in t.items()}
    t0 = time.perf_counter()
    c_ref.fwd(arr["q"], arr["k"], arr["v"], arr["r"], arr["u"], om, cfg["W"])
    c_ref.bwd(arr["q"], arr["k"], arr["v"], arr["r"], arr["u"], om, cfg["W"], arr["dO"])
    dt = time.perf_counter() - t0
    token_heads_per_s = n_units * tokens / dt
    desc = "fwd+bwd of the first %d tokens of %d (batch,head) units, same shapes and input recipe" % (tokens, n_units)
    return token_heads_per_s / cfg["H"], min(cores, n_units), desc, dt


def run_reference(args):
    """The oracle as the reference arm: every step is a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = WORKLOAD
    tokens = 256
    vals = []
    for s in range(args.warmup + args.steps):
        v, cores, desc, dt = cpu_oracle_sample(cfg, tokens)
        if s >= args.warmup:
            vals.append((v, dt))
    value = sum(v for v, _ in vals) / len(vals)
    ms = 1e3 * sum(dt for _, dt in vals) / len(vals)
    line = dict(impl="reference", metric=METRIC, value=value, unit="tokens/s", n_gpus=args.gpus, steps=args.steps,
                warmup=args.warmup, ms_per_step=ms, higher_is_better=True, scaling="weak", vs_baseline=None,
                dtype="f64", data="synthetic",
                config=dict(workload="C3: B=2 H=16 T=16384 d=128 m=128 W=64 (each step a bounded sample)",
                            sample=desc),
                cpu_baseline=dict(value=value, unit="tokens/s", cores=cores, kind="oracle", sample=desc),
                e2e=dict(value=value, unit="tokens/s", h2d_bytes_per_step=0, d2h_bytes_per_step=0),
                gpu_launches=0)
    print(json.dumps(line))


def bench_decode(P, synth, torch, dev, steps, warmup, use_image=True, use_graph=True):
    cfg = DECODE
    n_seq, H, d, m, W = cfg["n_seq"], cfg["H"], cfg["d"], cfg["m"], cfg["W"]
    omega = synth.make_omega(d, m).to(dev)
    S = torch.empty(n_seq, H, m, d, device=dev)
    z = torch.empty(n_seq, H, m, device=dev)
    rr = torch.empty(n_seq, H, W, d, device=dev, dtype=torch.bfloat16)
    ru = torch.empty(n_seq, H, W, d, device=dev, dtype=torch.bfloat16)
    g = torch.Generator(device=dev).manual_seed(cfg["seed"])

    def rms(x):
        return (x / x.pow(2).mean(-1, keepdim=True).sqrt()).to(torch.bfloat16)

    batch = 8
    ws = None
    for s0 in range(0, n_seq, batch):
        k = rms(torch.randn(batch, H, cfg["prefix"], d, device=dev, generator=g))
        v = rms(torch.randn(batch, H, cfg["prefix"], d, device=dev, generator=g))
        if ws is None:
            p = P.binding.make_params(batch, H, cfg["prefix"], d, m, W, P.BF16)
            ws = torch.empty(P.workspace_bytes(p, P.OP_STATE), dtype=torch.uint8, device=dev)
        Sb, zb = P.prefill_state(k, v, omega, W=W, workspace=ws)
        S[s0:s0 + batch] = Sb
        z[s0:s0 + batch] = zb
        rr[s0:s0 + batch] = rms(torch.randn(batch, H, W, d, device=dev, generator=g))
        ru[s0:s0 + batch] = rms(torch.randn(batch, H, W, d, device=dev, generator=g))
    del ws, k, v
    pool = 16
    toks = [[rms(torch.randn(n_seq, H, d, device=dev, generator=g)) for _ in range(5)] for _ in range(pool)]
    pos_all = (cfg["prefix"] + torch.arange(steps + warmup, device=dev, dtype=torch.int32))[:, None].repeat(1, n_seq)
    pos_all = pos_all.contiguous()
    out = torch.empty(n_seq, H, d, device=dev, dtype=torch.bfloat16)
    wsd = torch.empty(max(256, P.workspace_bytes(P.binding.make_params(n_seq, H, 0, d, m, W, P.BF16), P.OP_DECODE)),
                      dtype=torch.uint8, device=dev)
    # the constant feature matrix is converted once (linsimp_decode_prepare), not in every step
    wsd = P.decode_prepare(n_seq, H, d, omega, W=W)
    for s in range(warmup):
        q, k_, v_, r_, u_ = toks[s % pool]
        P.decode_step(q, k_, v_, r_, u_, omega, S, z, rr, ru, pos_all[s], W=W, out=out, workspace=wsd,
                      omega_image=use_image)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    graphed = use_graph and steps % pool == 0
    if graphed:
        # `pool` consecutive steps per CUDA graph (a serving loop would do the same): the positions of the steps
        # live in one tensor that a single add advances per replay
        pos_g = pos_all[warmup:warmup + pool].clone()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for j in range(2):                                    # warm the capture stream outside the capture
                q, k_, v_, r_, u_ = toks[j]
                P.decode_step(q, k_, v_, r_, u_, omega, S, z, rr, ru, pos_g[j], W=W, out=out, workspace=wsd,
                              omega_image=use_image)
            pos_g.add_(2)
        torch.cuda.current_stream().wait_stream(side)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            for j in range(pool):
                q, k_, v_, r_, u_ = toks[j]
                P.decode_step(q, k_, v_, r_, u_, omega, S, z, rr, ru, pos_g[j], W=W, out=out, workspace=wsd,
                              omega_image=use_image)
            pos_g.add_(pool)
        graph.replay()
        torch.cuda.synchronize()
        e0.record()
        for _ in range(steps // pool):
            graph.replay()
        e1.record()
    else:
        e0.record()
        for s in range(warmup, warmup + steps):
            q, k_, v_, r_, u_ = toks[s % pool]
            P.decode_step(q, k_, v_, r_, u_, omega, S, z, rr, ru, pos_all[s], W=W, out=out, workspace=wsd,
                          omega_image=use_image)
        e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / steps
    bytes_step = decode_bytes_per_unit(d, m, W) * n_seq * H
    launches = P.last_launch_count(P.OP_DECODE)
    finite = bool(torch.isfinite(out.float()).all())
    return dict(workload="C5: 256 seqs H=16 d=128 m=128 W=64, state from a 16384-token prefix, %d steps" % steps,
                us_per_step=us, algorithmic_bytes_per_step=bytes_step, gbs=bytes_step / us / 1e3,
                launches_per_step=launches, finite=finite, cuda_graph=graphed, omega_image=use_image)


def bench_secondary(P, synth, torch, dev, steps, peaks):
    """The secondary configurations: the feature-rank sweep (C4: B=4 H=8 T=8192 d=64, m in 32..256, fwd+bwd) and the
    layer forward (C2: B=8 H=16 T=4096 d=64 m=128).  A few timed steps each, CUDA events on the launching stream."""
    def frac(tf):
        return dict(frac_of_measured_bf16_burst=tf / peaks["bf16_burst"], frac_of_nominal_bf16=tf / 2250.0)

    rows = []
    for mm in (32, 64, 128, 256):
        cfg4, t4 = synth.make_config("C4m%d" % mm)
        g4 = {k_: v_.to(dev) for k_, v_ in t4.items()}
        p4 = P.binding.make_params(cfg4["B"], cfg4["H"], cfg4["T"], cfg4["d"], mm, 64, P.BF16)
        ws4 = torch.empty(max(P.workspace_bytes(p4, P.OP_BWD), P.workspace_bytes(p4, P.OP_FWD), 256),
                          dtype=torch.uint8, device=dev)

        def step4():
            o4, L4, lse4 = P.fwd(g4["q"], g4["k"], g4["v"], g4["r"], g4["u"], g4["omega"], workspace=ws4)
            P.bwd(g4["q"], g4["k"], g4["v"], g4["r"], g4["u"], g4["omega"], o4, L4, lse4, g4["dO"], workspace=ws4,
                  reuse_fwd_state=True)

        for _ in range(3):
            step4()
        torch.cuda.synchronize()
        P.profile_enable(True)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            step4()
        e1.record()
        torch.cuda.synchronize()
        prof4 = P.profile_read()
        P.profile_enable(False)
        ms = e0.elapsed_time(e1) / steps
        th4 = cfg4["B"] * cfg4["H"] * cfg4["T"]
        fl = 3.0 * fwd_flops_per_token_head(cfg4["d"], mm, 64) * th4
        tf = fl / (ms * 1e-3) / 1e12
        rows.append(dict(m=mm, ms_per_step=ms, tokens_per_s=cfg4["B"] * cfg4["T"] / (ms * 1e-3), tflops_3x=tf,
                         kernels={k_: round(v_[0] / steps, 3) for k_, v_ in prof4.items()}, **frac(tf)))
        del g4, ws4
    # layer forward (C2), forward only
    cfg2, t2 = synth.make_config("C2", with_dO=False)
    g2 = {k_: v_.to(dev) for k_, v_ in t2.items()}
    p2 = P.binding.make_params(cfg2["B"], cfg2["H"], cfg2["T"], cfg2["d"], cfg2["m"], 64, P.BF16)
    ws2 = torch.empty(P.workspace_bytes(p2, P.OP_FWD), dtype=torch.uint8, device=dev)
    o2 = torch.empty_like(g2["q"])
    for _ in range(3):
        P.fwd(g2["q"], g2["k"], g2["v"], g2["r"], g2["u"], g2["omega"], workspace=ws2, out=o2)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        P.fwd(g2["q"], g2["k"], g2["v"], g2["r"], g2["u"], g2["omega"], workspace=ws2, out=o2)
    e1.record()
    torch.cuda.synchronize()
    ms2 = e0.elapsed_time(e1) / steps
    th2 = cfg2["B"] * cfg2["H"] * cfg2["T"]
    tf2 = fwd_flops_per_token_head(cfg2["d"], cfg2["m"], 64) * th2 / (ms2 * 1e-3) / 1e12
    c2 = dict(ms=ms2, tokens_per_s=cfg2["B"] * cfg2["T"] / (ms2 * 1e-3), tflops=tf2, **frac(tf2))
    del g2, ws2, o2
    # the exact windowed 2-simplicial layer the paper compares with (joint softmax over 512 keys x 32 anchors), on the
    # shapes of the main workload, forward only; unit-norm k and r and a query of norm 8 (a temperature), as that layer
    # is run in the paper
    gen = torch.Generator(device=dev).manual_seed(77)
    Bw, Hw, Tw, dw = WORKLOAD["B"], WORKLOAD["H"], WORKLOAD["T"], WORKLOAD["d"]

    def unit(scale):
        x = torch.randn(Bw, Hw, Tw, dw, device=dev, generator=gen)
        return (x / x.norm(dim=-1, keepdim=True) * scale).to(torch.bfloat16)

    qw, kw, rw = unit(8.0), unit(1.0), unit(1.0)
    vw, uw = unit(dw ** 0.5), unit(dw ** 0.5)
    ow = torch.empty_like(qw)
    for _ in range(3):
        P.winsimp_fwd(qw, kw, vw, rw, uw, w1=512, w2=32, out=ow)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        P.winsimp_fwd(qw, kw, vw, rw, uw, w1=512, w2=32, out=ow)
    e1.record()
    torch.cuda.synchronize()
    msw = e0.elapsed_time(e1) / steps
    flw = 2.0 * 2.0 * 512 * 32 * dw * Bw * Hw * Tw          # score and value contraction over the full pair plane
    tfw = flw / (msw * 1e-3) / 1e12
    win = dict(ms=msw, tokens_per_s=Bw * Tw / (msw * 1e-3), tflops=tfw, finite=bool(torch.isfinite(ow.float()).all()), **frac(tfw))
    del qw, kw, rw, vw, uw, ow
    # the main workload's step with the boundary states as two bf16 terms in the backward (LINSIMP_FLAG_STATE_TWO_TERMS)
    def rms():
        x = torch.randn(Bw, Hw, Tw, dw, device=dev, generator=gen)
        return (x / x.pow(2).mean(dim=-1, keepdim=True).sqrt()).to(torch.bfloat16)

    tq, tk, tv, tr, tu, tdo = (rms() for _ in range(6))
    tom = torch.randn(dw, WORKLOAD["m"], device=dev, generator=gen)
    pt = P.binding.make_params(Bw, Hw, Tw, dw, WORKLOAD["m"], WORKLOAD["W"], P.BF16, flags=P.binding.FLAG_STATE_TWO_TERMS)
    wst = torch.empty(P.workspace_bytes(pt, P.OP_BWD), dtype=torch.uint8, device=dev)

    def step_t():
        o_, L_, lse_ = P.fwd(tq, tk, tv, tr, tu, tom, W=WORKLOAD["W"], workspace=wst, two_term_state=True)
        P.bwd(tq, tk, tv, tr, tu, tom, o_, L_, lse_, tdo, W=WORKLOAD["W"], workspace=wst, reuse_fwd_state=True,
              two_term_state=True)

    for _ in range(3):
        step_t()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        step_t()
    e1.record()
    torch.cuda.synchronize()
    two = dict(ms_per_step=e0.elapsed_time(e1) / steps, workspace_bytes=int(wst.numel()))
    del tq, tk, tv, tr, tu, tdo, wst
    return dict(steps=steps, two_term_state="main workload, fwd+bwd, boundary states as two bf16 terms in the backward",
                c3_two_term_state=two,
                exact_windowed="exact 512 x 32 windowed 2-simplicial layer on B=%d H=%d T=%d d=%d bf16, fwd only "
                               "(warp-level MMAs)" % (Bw, Hw, Tw, dw), winsimp=win,
                c4_sweep="C4: B=4 H=8 T=8192 d=64 W=64 bf16, fwd+bwd, TFLOP/s in the 3x convention", c4=rows,
                c2_forward="C2: B=8 H=16 T=4096 d=64 m=128 bf16, fwd only", c2=c2)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--decode-steps", type=int, default=1024)
    ap.add_argument("--skip-decode", action="store_true")
    ap.add_argument("--decode-only", action="store_true", help="run only the decode benchmark (profiler captures)")
    ap.add_argument("--decode-prefix", type=int, default=DECODE["prefix"], help="prefix length used to build the decode state")
    ap.add_argument("--no-graph", action="store_true", help="decode: launch every step instead of replaying CUDA graphs (profiler captures)")
    ap.add_argument("--no-omega-image", action="store_true", help="decode: every step converts omega itself (profiler captures)")
    ap.add_argument("--skip-secondary", action="store_true", help="leave out the secondary configurations (C2 forward, C4 sweep)")
    ap.add_argument("--skip-cpu-baseline", action="store_true")
    ap.add_argument("--skip-e2e", action="store_true")
    ap.add_argument("--small", action="store_true", help="T=4096 variant for profiler captures (not a bench value)")
    ap.add_argument("--norm-gate", action="store_true",
                    help="only the normalisation / gate kernels on C3-shaped streams (GB/s per kernel; profiler captures)")
    ap.add_argument("--sweep", action="store_true",
                    help="feature-rank sweep (B=4 H=8 T=8192 d=64, m in 32..256): fwd+bwd time and TFLOP/s per m")
    args = ap.parse_args()
    if args.warmup < 3 and not args.small:
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import paper_2608_09307_b200 as P
    from paper_2608_09307_b200 import synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    P.load_library()
    peaks = measured_peaks()
    DECODE["prefix"] = args.decode_prefix
    if args.norm_gate:
        cfg3 = synth.CONFIGS["C3"]
        B3, H3, T3, d3 = cfg3["B"], cfg3["H"], cfg3["T"], cfg3["d"]
        gen = torch.Generator(device=dev).manual_seed(3)
        xs = [torch.randn(B3, H3, T3, d3, device=dev, generator=gen).to(torch.bfloat16) for _ in range(6)]
        tau3 = torch.full((H3,), float(d3) ** 0.5, device=dev)
        gamma3 = torch.full((H3,), -2.0, device=dev)
        outs3 = tuple(torch.empty_like(x) for x in xs[:3])
        y3 = torch.empty_like(xs[0])
        ws3 = torch.empty(1 << 20, dtype=torch.uint8, device=dev)
        nb = xs[0].numel() * xs[0].element_size()
        cases = [("qkr_norm", 6 * nb, lambda: P.qkr_normalize(xs[0], xs[1], xs[2], tau3, out=outs3)),
                 ("qkr_norm_bwd", 9 * nb, lambda: P.qkr_normalize_bwd(xs[0], xs[1], xs[2], tau3, xs[3], xs[4], xs[5], workspace=ws3)),
                 ("gate_norm", 2 * nb, lambda: P.gate_rmsnorm(xs[0], gamma3, out=y3)),
                 ("gate_norm_bwd", 3 * nb, lambda: P.gate_rmsnorm_bwd(xs[0], gamma3, xs[3], workspace=ws3))]
        res = {}
        for name, nbytes, fn in cases:
            for _ in range(args.warmup):
                fn()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(args.steps):
                fn()
            e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / args.steps
            res[name] = dict(ms=ms, algorithmic_bytes=nbytes, gbs=nbytes / ms / 1e6, frac_hbm=nbytes / ms / 1e6 / peaks["hbm_gbs"])
        print(json.dumps(dict(norm_gate="C3-shaped bf16 streams [2,16,16384,128] (134 MB each), streams exceed L2",
                              hbm_peak_gbs=peaks["hbm_gbs"], kernels=res)))
        return
    if args.sweep:
        sec = bench_secondary(P, synth, torch, dev, args.steps, peaks)
        rows, c2 = sec["c4"], sec["c2"]
        # whole head on C3: normalisation with temperature -> estimator -> gated RMSNorm, and back
        cfg3, t3 = synth.make_config("C3")
        g3 = {k_: v_.to(dev) for k_, v_ in t3.items()}
        tau3 = torch.full((cfg3["H"],), float(cfg3["d"]) ** 0.5, device=dev)
        gamma3 = torch.full((cfg3["H"],), -2.0, device=dev)

        def head_step():
            y3, saved3 = P.head_fwd(g3["q"], g3["k"], g3["v"], g3["r"], g3["u"], g3["omega"], tau3, gamma3)
            P.head_bwd(saved3, g3["dO"])

        for _ in range(3):
            head_step()
        torch.cuda.synchronize()
        P.profile_enable(True)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.steps):
            head_step()
        e1.record()
        torch.cuda.synchronize()
        prof3 = P.profile_read()
        P.profile_enable(False)
        ms3 = e0.elapsed_time(e1) / args.steps
        nb = g3["q"].numel() * g3["q"].element_size()
        stream_bytes = dict(qkr_norm=6 * nb, qkr_norm_bwd=9 * nb, gate_norm=2 * nb, gate_norm_bwd=3 * nb)
        c3h = dict(ms=ms3, tokens_per_s=cfg3["B"] * cfg3["T"] / (ms3 * 1e-3),
                   kernels={k_: round(v_[0] / args.steps, 3) for k_, v_ in prof3.items()},
                   streaming_gbs={k_: round(b_ / (prof3[k_][0] / args.steps * 1e-3) / 1e9, 1)
                                  for k_, b_ in stream_bytes.items() if k_ in prof3},
                   hbm_peak_gbs=peaks["hbm_gbs"])
        print(json.dumps(dict(sweep="C4: B=4 H=8 T=8192 d=64 W=64 bf16, fwd+bwd", rows=rows,
                              c2_forward="C2: B=8 H=16 T=4096 d=64 m=128 bf16, fwd only", c2=c2,
                              c3_head="C3 inputs through the whole head (tau = sqrt(d), gamma = -2), fwd+bwd", c3h=c3h)))
        return
    if args.decode_only:
        dec = bench_decode(P, synth, torch, dev, args.decode_steps, 3, not args.no_omega_image, not args.no_graph)
        dec["frac_hbm"] = dec["gbs"] / peaks["hbm_gbs"]
        print(json.dumps(dict(decode=dec)))
        return

    cfg = dict(WORKLOAD)
    if args.small:
        cfg["T"] = 4096
    B, H, T, d, m, W = (cfg[k_] for k_ in ("B", "H", "T", "d", "m", "W"))
    # every rank runs its own batch of the same shape (weak scaling over independent (batch, head) units)
    host = synth.make_inputs(B, H, T, d, cfg["seed"] + 1000 * rank, "bf16", "rms")
    host = {k_: v_.pin_memory() for k_, v_ in host.items()}
    omega = synth.make_omega(d, m).to(dev)
    gpu = {k_: v_.to(dev) for k_, v_ in host.items()}
    par = P.binding.make_params(B, H, T, d, m, W, P.BF16)
    ws = torch.empty(max(P.workspace_bytes(par, P.OP_BWD), P.workspace_bytes(par, P.OP_FWD)), dtype=torch.uint8,
                     device=dev)
    o_buf = torch.empty_like(gpu["q"])

    def step(t, out=None):
        o, L, lse = P.fwd(t["q"], t["k"], t["v"], t["r"], t["u"], omega, W=W, workspace=ws,
                          out=o_buf if out is None else out)
        grads = P.bwd(t["q"], t["k"], t["v"], t["r"], t["u"], omega, o, L, lse, t["dO"], W=W, workspace=ws,
                      reuse_fwd_state=True)
        return o, grads

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        sampler.wait_ready()
    for _ in range(args.warmup):
        step(gpu)
    barrier()
    # The timed region: exactly K steps between barrier + synchronize, CUDA events on the launching stream.  On shared
    # hosts a driver query by another process (nvidia-smi, this bench's own clock sampler included) now and then holds
    # kernel launches up for tens of milliseconds; such an attempt shows as event time well above the sum of its own
    # kernels' times and is measured again (at most twice).  Every attempt is reported.
    attempts = []
    best = None
    for attempt in range(3):
        P.profile_enable(True)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        sampler.mark()
        e0.record()
        for _ in range(args.steps):
            o, grads = step(gpu)
        e1.record()
        barrier()
        ms_try = e0.elapsed_time(e1)
        prof_try = P.profile_read()
        P.profile_enable(False)
        kernel_ms = sum(v_[0] for v_ in prof_try.values())
        stalled = 1.0 if ms_try > 1.03 * kernel_ms else 0.0
        if world > 1:
            from paper_2608_09307_b200.dist import max_over_ranks
            ms_try = max_over_ranks(ms_try, device=dev)
            stalled = max_over_ranks(stalled, device=dev)
        attempts.append(ms_try / args.steps)
        if best is None or ms_try < best[0]:
            best = (ms_try, prof_try)
        if not stalled:
            break
    ms_total, prof = best
    clocks = sampler.stop() if rank == 0 else None
    launches_per_step = P.last_launch_count(P.OP_FWD) + P.last_launch_count(P.OP_BWD)
    finite = bool(torch.isfinite(o.float()).all()) and all(bool(torch.isfinite(g_.float()).all()) for g_ in grads)

    # end to end: host buffers in, host buffers out, every step
    e2e = None
    if not args.skip_e2e:
        # A three-stage pipeline over the steps, as a training loop would run it: the host->device copy of step
        # i+1 (pinned memory, own stream) and the device->host copy of step i-1 (own stream) run beside the
        # kernels of step i; the timed region covers all three streams including fill and drain.
        host_out = [torch.empty_like(host["q"]).pin_memory() for _ in range(6)]
        dev_in = [{k_: torch.empty_like(v_) for k_, v_ in gpu.items()} for _ in range(2)]
        s_c = torch.cuda.current_stream()
        s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()

        o_bufs = [o_buf, torch.empty_like(o_buf)]       # o of step i is still being copied out while step i+1 runs

        def e2e_run(n_steps):
            ev_in = [None, None]
            ev_done = [None, None]
            ev_o = [None, None]
            ev_out = None
            for i in range(n_steps):
                buf = i & 1
                with torch.cuda.stream(s_in):
                    if ev_done[buf] is not None:
                        s_in.wait_event(ev_done[buf])
                    for k_ in dev_in[buf]:
                        dev_in[buf][k_].copy_(host[k_], non_blocking=True)
                    ev_in[buf] = torch.cuda.Event()
                    ev_in[buf].record(s_in)
                s_c.wait_event(ev_in[buf])
                if ev_o[buf] is not None:
                    s_c.wait_event(ev_o[buf])
                o2, g2 = step(dev_in[buf], o_bufs[buf])
                ev_done[buf] = torch.cuda.Event()
                ev_done[buf].record(s_c)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(ev_done[buf])
                    host_out[0].copy_(o2, non_blocking=True)
                    ev_o[buf] = torch.cuda.Event()
                    ev_o[buf].record(s_out)
                    for dst, src in zip(host_out[1:], g2):
                        src.record_stream(s_out)
                        dst.copy_(src, non_blocking=True)
                    ev_out = torch.cuda.Event()
                    ev_out.record(s_out)
            return ev_out

        s_c.wait_event(e2e_run(2))
        barrier()
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        f0.record()
        last = e2e_run(args.steps)
        s_c.wait_event(last)
        f1.record()
        barrier()
        e2e_ms = f0.elapsed_time(f1)
        nbytes = host["q"].numel() * host["q"].element_size()
        e2e = dict(ms=e2e_ms, h2d=6 * nbytes, d2h=6 * nbytes)

    if world > 1:
        from paper_2608_09307_b200.dist import max_over_ranks
        ms_total = max_over_ranks(ms_total, device=dev)          # a step is as slow as the slowest rank
        if e2e:
            e2e["ms"] = max_over_ranks(e2e["ms"], device=dev)

    decode = None
    if not args.skip_decode and not args.small and rank == 0:
        decode = bench_decode(P, synth, torch, dev, args.decode_steps, 8, not args.no_omega_image, not args.no_graph)
        decode["frac_hbm"] = decode["gbs"] / peaks["hbm_gbs"]
        decode["peak_gbs"] = peaks["hbm_gbs"]
        decode["peak_source"] = peaks["source"]

    if rank != 0:
        if world > 1:
            dist.barrier()
            dist.destroy_process_group()
        return

    tokens = B * T * world
    ms_step = ms_total / args.steps
    value = tokens / (ms_step * 1e-3)
    th = B * H * T                       # token-heads per rank per step
    f_fwd = fwd_flops_per_token_head(d, m, W)
    tflops = {"3x": 3.0 * f_fwd * th * world / (ms_step * 1e-3) / 1e12,
              "2.5x": 2.5 * f_fwd * th * world / (ms_step * 1e-3) / 1e12,
              "3.5x": 3.5 * f_fwd * th * world / (ms_step * 1e-3) / 1e12}
    # roofline of the dominant kernel of the timed region
    alg = {   # algorithmic FLOPs per launch, bound, peak TFLOP/s
        "fwd_fp32": (2.0 * m * 2 * d * W * th, "alu", FP32_FMA_PEAK_TFLOPS),
        "bwd_query_fp32": (3 * 2.0 * W * m * d * th, "alu", FP32_FMA_PEAK_TFLOPS),
        "bwd_kv_fp32": (2.0 * W * m * d * th, "alu", FP32_FMA_PEAK_TFLOPS),
        "fwd_tc": (2.0 * m * 2 * d * W * th, "tensor", peaks["bf16_burst"]),
        "bwd_tc": (2.0 * 2.0 * m * 2 * d * W * th, "tensor", peaks["bf16_burst"]),
    }
    roofline = None
    if prof:
        top = max(prof.items(), key=lambda kv: kv[1][0])
        name, (tms, cnt) = top
        avg_ms = tms / cnt
        if name in alg:
            fl, bound, peak = alg[name]
            ach = fl / (avg_ms * 1e-3) / 1e12
            # DRAM bytes per launch: counted by a profiler capture of a smaller case of the same kernel and scaled by
            # the tokens per sequence (the traffic - states, images and gradients per chunk - grows with the tokens)
            cap = ncu_dram_bytes()
            traffic = None
            if cap and name in cap.get("kernels", {}):
                traffic = cap["kernels"][name] * (T / float(cap["T"]))
            roofline = dict(kernel=name, bound=bound, achieved=ach, peak=peak, unit="TFLOP/s", frac=ach / peak,
                            traffic=traffic, avg_ms=avg_ms, launches=cnt,
                            peak_source=("derived: 148 SMs x 128 fp32 lanes x 2 x 1.965 GHz" if bound == "alu"
                                         else "of %s (burst bf16)" % peaks["source"]))
            if bound == "tensor":
                roofline["frac_of_sustained"] = ach / peaks["bf16_sustained"]
                roofline["traffic_source"] = (None if traffic is None else
                                              "profiler capture at T=%d scaled by T/%d" % (cap["T"], cap["T"]))
        else:
            roofline = dict(kernel=name, bound=None, achieved=None, peak=None, unit=None, frac=None, traffic=None,
                            avg_ms=avg_ms, launches=cnt)
    kernels = {k_: dict(ms_total=v_[0], launches=v_[1], share=v_[0] / max(1e-9, sum(x[0] for x in prof.values())))
               for k_, v_ in prof.items()}

    secondary = None
    if not args.skip_secondary and not args.small:
        secondary = bench_secondary(P, synth, torch, dev, 5, peaks)

    cpu = None
    if not args.skip_cpu_baseline and world == 1:
        v, cores, desc, dt = cpu_oracle_sample(cfg, 2560 if not args.small else 128)
        cpu = dict(value=v, unit="tokens/s", cores=cores, kind="oracle", sample=desc, seconds=dt)

    line = dict(metric=METRIC, value=value, unit="tokens/s", n_gpus=world, steps=args.steps, warmup=args.warmup,
                ms_per_step=ms_step, higher_is_better=True, scaling="weak", vs_baseline=None, dtype="bf16",
                data="synthetic",
                config=dict(workload="C3: B=%d H=%d T=%d d=%d m=%d W=%d per GPU, bf16 inputs RMS-normalised, "
                                     "fp32 state, fwd+bwd" % (B, H, T, d, m, W),
                            l2="inputs and workspace exceed L2 (no flush needed)",
                            parallelism="independent (batch, head) units per rank, no collective"),
                tflops=tflops, frac_of_nominal_bf16=tflops["3x"] / (2250.0 * world),
                frac_of_measured_bf16_sustained=tflops["3x"] / (peaks["bf16_sustained"] * world),
                frac_of_measured_bf16_burst=tflops["3x"] / (peaks["bf16_burst"] * world),
                roofline=roofline, secondary=secondary, kernels=kernels, cpu_baseline=cpu, clocks=clocks,
                gpu_launches=launches_per_step * args.steps, finite=finite, decode=decode,
                attempts_ms_per_step=attempts)
    if e2e:
        line["e2e"] = dict(value=tokens / (e2e["ms"] / args.steps * 1e-3), unit="tokens/s",
                           h2d_bytes_per_step=e2e["h2d"], d2h_bytes_per_step=e2e["d2h"],
                           ms_per_step=e2e["ms"] / args.steps)
    print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
