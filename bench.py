#!/usr/bin/env python
"""Benchmark of the ROSAQ hot path on B200.

Workload (N = 1): the seven linears of one LLaMA-7B-shaped decoder layer at M = 64 decode
tokens, INT4 g128 with K = 128 FP16 salient channels (seeded synthetic weights and
activations).  One step = one pass over the layer: three online rotations x.R (attention input and
MLP input: dense 4096 x 4096 fp16 R from a layer-wise PCA of synthetic calibration activations;
o_proj input: head-wise PCA, 32 blocks of 128 x 128 plus the global eigenvalue order, Eq. 6) and seven GEMM stages (q, k, v, o, gate, up, down; down_proj is not rotated, as in
the paper's appendix on weight splitting).  Steps alternate between two layers with distinct
weights (2 x 197 MB, larger than the 126 MB L2), replayed from CUDA graphs.

metric/value: algorithmic bytes of the step (packed codes + scales/zeros + FP16 salient rows +
activations in and out + the fp16 rotation matrices) divided by the device time, in GB/s.
`gemm_stage` reports the GEMM stage alone per shape (the quantity the 70 %-of-HBM target is
stated on) next to a cuBLAS FP16 GEMM of the same shape in the same harness.

`--impl reference` times the CPU oracle (oracle/) on a bounded sample of the same workload.
"""
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

METRIC = "rosaq_w4a16_decode_layer_hbm_gbs_m64"     # "w3" when run with --bits 3
UNIT = "GB/s"
M_TOKENS = 64
K_SALIENT = 128
NOMINAL_HBM_GBS = 8000.0
# dram__bytes_read.sum + dram__bytes_write.sum per launch, averaged over the 7 launches of an INT4 step
# (one ncu capture of this command with --steps 4 --warmup 3 --no-table --no-cpu-baseline; stale, and to be
# set to None, as soon as the kernel or the workload changes)
TRAFFIC_BYTES_PER_LAUNCH = 26941911


# ----------------------------------------------------------------------------- bytes / flops
def gemm_bytes(d_in, d_out, M, bits, k_salient=K_SALIENT):
    """Algorithmic bytes of one GEMM-stage call: codes + (scale, zero) + salient fp16 + x + y."""
    groups = d_in // 128
    gs = k_salient // 128
    return ((d_in - k_salient) * d_out * bits // 8 + (groups - gs) * d_out * 4 + k_salient * d_out * 2
            + M * d_in * 2 + M * d_out * 2)


def rotate_bytes(d, M, n_blocks=1):
    return d * (d // n_blocks) * 2 + 2 * M * d * 2


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        j = json.load(open(p))
        return dict(hbm_gbs=float(j["hbm_gbs"]), bf16_tflops=float(j["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, source="fallback")


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def __exit__(self, *a):
        if self.proc:
            time.sleep(0.15)
            self.proc.terminate()
            try:
                self.proc.wait(timeout=2)
            except Exception:
                pass

    def summary(self):
        sm = [float(r[0]) for r in self.rows if len(r) >= 6 and r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if len(r) >= 6 and r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = sorted({n for r in self.rows if len(r) >= 6 for n, v in zip(names, r[2:6]) if v == "Active"})
        return dict(sm_mhz=float(np.median(sm)) if sm else None, sm_max_mhz=max(mx) if mx else None,
                    reasons=reasons, samples=len(sm))


# ----------------------------------------------------------------------------- workload
def build_workload(ctx, bits, seed, n_layers, model):
    """Calibrate, rotate, quantize `n_layers` decoder layers of synthetic weights on the GPU."""
    import torch
    from paper_2506_13472_b200 import pca, synth
    d, f = model["d"], model["ffn"]
    layers = []
    for li in range(n_layers):
        rots, R32, perms = {}, {}, {}
        for inp in ("attn_in", "mlp_in"):                            # layer-wise PCA, dense R (Section 3.1)
            law = synth.ActivationLaw(d, 1.0, seed, f"L{li}/{inp}")
            X = torch.from_numpy(law.sample(2048, "calib", np.float16)).cuda()
            Cg = torch.zeros((d, d), dtype=torch.float32, device="cuda")
            ctx.calib_cov(X, Cg)
            R = pca.eigh_descending_device(Cg)                       # fp64 on the device, host-side step a2
            R32[inp] = R.to(torch.float32).contiguous()
            rots[inp] = ctx.rotation_create(R.to(torch.float16).contiguous())
        # o_proj input: head-wise PCA (Section 3.1.1, Eq. 6): one 128 x 128 rotation per head from
        # per-head activations, plus the global descending-eigenvalue column order
        H, hd = model["heads"], model["head_dim"]
        Xh = torch.from_numpy(head_law(model, seed).sample(4096, f"L{li}/calib", np.float16)).cuda()
        Cb = torch.zeros((H, hd, hd), dtype=torch.float32, device="cuda")
        ctx.calib_cov(Xh, Cb, n_blocks=H)
        Rb, perm, _ = pca.headwise_rotation(Cb.cpu().numpy())
        R32["o_in"] = torch.from_numpy(Rb.astype(np.float32)).cuda()
        perms["o_in"] = torch.from_numpy(perm).cuda()
        rots["o_in"] = ctx.rotation_create(torch.from_numpy(Rb.astype(np.float16)).cuda(), perms["o_in"])
        weights, fp16 = {}, {}
        for name, d_in, d_out, inp in synth.layer_shapes(model):
            W = torch.from_numpy(synth.weights(d_in, d_out, seed, f"L{li}/{name}", sigma=0.02,
                                               outlier_frac=0.01, outlier_scale=10.0)).cuda()
            weights[name] = ctx.quantize(W, R32.get(inp), perms.get(inp), bits=bits, k_salient=K_SALIENT)
            fp16[name] = W
        layers.append(dict(rots=rots, weights=weights, fp16=fp16))
        del R32
    xs = {}
    for inp, dd in (("attn_in", d), ("mlp_in", d), ("down_in", f)):
        law = synth.ActivationLaw(dd, 1.0, seed, f"x/{inp}")
        xs[inp] = law.sample(M_TOKENS, "x", np.float16)
    xs["o_in"] = head_law(model, seed).sample(M_TOKENS, "x", np.float16)
    return layers, xs


def head_law(model, seed):
    from paper_2506_13472_b200 import synth
    return synth.HeadwiseActivationLaw(model["heads"], model["head_dim"], seed, "o_in")


def layer_bytes(model, bits):
    from paper_2506_13472_b200 import synth
    b = sum(gemm_bytes(di, do, M_TOKENS, bits) for _, di, do, _ in synth.layer_shapes(model))
    return b + 2 * rotate_bytes(model["d"], M_TOKENS) + rotate_bytes(model["d"], M_TOKENS, model["heads"])


class LayerRunner:
    """Owns the device buffers of one layer pass and issues its library calls: three rotations and four
    GEMM-stage launches (q/k/v in one rosaq_linear_multi call, o, gate/up in one, down) = 7 kernels."""
    LAUNCHES = 7

    def __init__(self, ctx, layer, xs_dev, model):
        import torch
        self.ctx, self.L, self.x = ctx, layer, xs_dev
        d, f = model["d"], model["ffn"]
        mk = lambda n: torch.empty((M_TOKENS, n), dtype=torch.float16, device="cuda")
        self.xr = {k: mk(d) for k in ("attn_in", "o_in", "mlp_in")}
        self.y = {"q": mk(d), "k": mk(d), "v": mk(d), "o": mk(d), "gate": mk(f), "up": mk(f), "down": mk(d)}

    def run(self):
        c, L = self.ctx, self.L
        c.rotate(self.x["attn_in"], L["rots"]["attn_in"], out=self.xr["attn_in"])
        c.linear_multi(self.xr["attn_in"], [L["weights"][n] for n in ("q", "k", "v")], None,
                       outs=[self.y[n] for n in ("q", "k", "v")])
        c.rotate(self.x["o_in"], L["rots"]["o_in"], out=self.xr["o_in"])
        c.linear(self.xr["o_in"], L["weights"]["o"], None, out=self.y["o"])
        c.rotate(self.x["mlp_in"], L["rots"]["mlp_in"], out=self.xr["mlp_in"])
        c.linear_multi(self.xr["mlp_in"], [L["weights"][n] for n in ("gate", "up")], None,
                       outs=[self.y[n] for n in ("gate", "up")])
        c.linear(self.x["down_in"], L["weights"]["down"], None, out=self.y["down"])


def fp16_layer_graph(layers, xs_dev, model):
    """The same seven GEMMs per layer with the un-rotated fp16 weights through cuBLAS (torch.matmul): one
    CUDA graph that walks over all layers in turn (so the weights are as cold as on the quantized path);
    a replay is len(layers) steps.  The FP16 baseline of the layer replay."""
    import torch
    d, f = model["d"], model["ffn"]
    mk = lambda n: torch.empty((M_TOKENS, n), dtype=torch.float16, device="cuda")
    y = {"q": mk(d), "k": mk(d), "v": mk(d), "o": mk(d), "gate": mk(f), "up": mk(f), "down": mk(d)}
    inp = {"q": "attn_in", "k": "attn_in", "v": "attn_in", "o": "o_in", "gate": "mlp_in", "up": "mlp_in",
           "down": "down_in"}

    def run():
        for L in layers:
            for n in ("q", "k", "v", "o", "gate", "up", "down"):
                torch.matmul(xs_dev[inp[n]], L["fp16"][n], out=y[n])
    return capture(run)


def time_graphs(graphs, steps, warmup):
    """Replays the graphs round-robin; returns milliseconds for `steps` replays (CUDA events)."""
    import torch
    for i in range(warmup):
        graphs[i % len(graphs)].replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(steps):
        graphs[i % len(graphs)].replay()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1)


def capture(fn):
    import torch
    g = torch.cuda.CUDAGraph()
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        fn()                                    # warm-up outside capture (lazy allocations)
    torch.cuda.current_stream().wait_stream(s)
    torch.cuda.synchronize()
    with torch.cuda.graph(g):
        fn()
    return g


def gemm_stage_table(ctx, model, bits, peaks, reps=20):
    """Per shape: GEMM stage alone at M=64 over >= 2 x L2 of distinct weight copies, and cuBLAS FP16."""
    import torch
    from paper_2506_13472_b200 import synth
    d, f = model["d"], model["ffn"]
    out = []
    for d_in, d_out in ((d, d), (d, f), (f, d)):
        W = torch.from_numpy(synth.weights(d_in, d_out, 1, f"gs{d_in}x{d_out}", outlier_frac=0.01)).cuda()
        w0 = ctx.quantize(W, None, bits=bits, k_salient=K_SALIENT)
        e = w0.export()
        copies = max(2, int(np.ceil(2 * 126e6 / w0.device_bytes)))
        ws = [w0] + [ctx.weight_import(d_in, d_out, bits, 128, K_SALIENT, e["qw"], e["scales"], e["zeros"],
                                       e["salient"]) for _ in range(copies - 1)]
        x = torch.randn((M_TOKENS, d_in), device="cuda").to(torch.float16)
        y = torch.empty((M_TOKENS, d_out), dtype=torch.float16, device="cuda")
        g = capture(lambda: [ctx.linear(x, w, None, out=y) for w in ws])
        ms = sorted(time_graphs([g], 1, 1) for _ in range(reps))[reps // 2]
        us = ms * 1e3 / copies
        nb = gemm_bytes(d_in, d_out, M_TOKENS, bits)
        fcopies = max(2, int(np.ceil(2 * 126e6 / (d_in * d_out * 2))))
        Wf = [W] + [W.clone() for _ in range(fcopies - 1)]
        yf = torch.empty((M_TOKENS, d_out), dtype=torch.float16, device="cuda")
        gf = capture(lambda: [torch.matmul(x, w, out=yf) for w in Wf])
        msf = sorted(time_graphs([gf], 1, 1) for _ in range(reps))[reps // 2]
        usf = msf * 1e3 / fcopies
        gbs = nb / us / 1e3
        out.append(dict(shape=f"{d_in}x{d_out}", M=M_TOKENS, bits=bits, us=round(us, 3), gbs=round(gbs, 1),
                        frac_of_8tbs=round(gbs / NOMINAL_HBM_GBS, 4),
                        frac_of_measured=round(gbs / peaks["hbm_gbs"], 4),
                        tflops=round(2.0 * M_TOKENS * d_in * d_out / us / 1e6, 1),
                        cublas_fp16_us=round(usf, 3), speedup_vs_cublas_fp16=round(usf / us, 3)))
        for w in ws:
            w.free()
        del Wf, W
        torch.cuda.empty_cache()
    return out


def profile_shape(args):
    """One GEMM-stage shape over distinct random weight copies (>= 2 x L2), replayed from a CUDA graph:
    the small, self-contained case that ncu captures are taken on.  Prints one line."""
    import torch
    from paper_2506_13472_b200 import binding as rb
    d_in, d_out, M, bits = args.profile_shape
    ctx = rb.Context(0)
    g = torch.Generator(device="cuda").manual_seed(0)
    ks = d_in if bits == 16 else K_SALIENT            # bits 16: every group fp16 (the shape of a rotation operand)
    qbits = 4 if bits == 16 else bits
    nq = d_in - ks
    nw = nq // 8 if qbits == 4 else nq // 32 * 3
    qw = torch.randint(-2 ** 31, 2 ** 31 - 1, (nw, d_out), dtype=torch.int64, device="cuda", generator=g).to(torch.int32)
    sc = (torch.rand((nq // 128, d_out), device="cuda", generator=g) * 0.01 + 0.001).half()
    zr = torch.randint(0, 2 ** qbits, (nq // 128, d_out), device="cuda", generator=g).half()
    sal = (torch.randn((ks, d_out), device="cuda", generator=g) * 0.02).half()
    mk = lambda: ctx.weight_import(d_in, d_out, qbits, 128, ks, qw, sc, zr, sal)
    w0 = mk()
    copies = args.copies or max(2, int(np.ceil(2 * 126e6 / w0.device_bytes)))
    ws = [w0] + [mk() for _ in range(copies - 1)]
    x = torch.randn((M, d_in), device="cuda", generator=g).half()
    y = torch.empty((M, d_out), dtype=torch.float16, device="cuda")
    gph = capture(lambda: [ctx.linear(x, w, None, out=y) for w in ws])
    ts = sorted(time_graphs([gph], 1, 1) * 1e3 / copies for _ in range(args.steps))
    us = ts[len(ts) // 2]
    nb = gemm_bytes(d_in, d_out, M, qbits, ks)
    assert ctx.last_status() == 0
    line = {"shape": f"{d_in}x{d_out}", "M": M, "bits": bits, "copies": copies, "us": round(us, 3),
            "us_min": round(ts[0], 3), "gbs": round(nb / us / 1e3, 1),
            "frac_of_measured": round(nb / us / 1e3 / load_peaks()["hbm_gbs"], 4),
            "tflops": round(2.0 * M * d_in * d_out / us / 1e6, 1)}
    if args.with_cublas:                                   # an fp16 GEMM of the same shape, same replay harness
        for w in ws:
            w.free()
        fcopies = max(2, int(np.ceil(2 * 126e6 / (d_in * d_out * 2))))
        Wf = [(torch.randn((d_in, d_out), device="cuda", generator=g) * 0.02).half() for _ in range(fcopies)]
        gf = capture(lambda: [torch.matmul(x, w, out=y) for w in Wf])
        tf = sorted(time_graphs([gf], 1, 1) * 1e3 / fcopies for _ in range(args.steps))
        line["cublas_fp16_us"] = round(tf[len(tf) // 2], 3)
        line["speedup_vs_cublas_fp16"] = round(tf[len(tf) // 2] / us, 3)
    print(json.dumps(line))


def calib_cov_throughput(ctx, peaks, n_tokens=16384, d=5120, reps=5):
    """rosaq_calib_cov on one chunk of the 13B-shaped calibration stream (fp16 activations, fp32 C):
    device time per call and tensor throughput.  `tflops` counts the multiply-adds the kernel executes
    (the 256 x 256 tiles that touch the lower triangle); `tflops_full_square` credits the
    whole d x d result that those tiles produce by symmetry."""
    import torch
    X = torch.randn((n_tokens, d), device="cuda", dtype=torch.float16)
    Cm = torch.zeros((d, d), dtype=torch.float32, device="cuda")
    ctx.calib_cov(X, Cm)
    torch.cuda.synchronize()
    ts = []
    for _ in range(reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        ctx.calib_cov(X, Cm)
        e1.record()
        torch.cuda.synchronize()
        ts.append(e0.elapsed_time(e1))
    ms = sorted(ts)[len(ts) // 2]
    nb = (d + 255) // 256                              # 256 x 256 tiles that touch the lower triangle
    executed = 2.0 * n_tokens * 256 * 256 * (nb * (nb + 1) // 2)
    tf = executed / ms / 1e9
    return dict(tokens=n_tokens, d=d, ms=round(ms, 4), tflops=round(tf, 1),
                tflops_full_square=round(2.0 * n_tokens * d * d / ms / 1e9, 1),
                frac_of_bf16_peak=round(tf / peaks["bf16_tflops"], 4), peak_source=peaks["source"])


# ----------------------------------------------------------------------------- oracle legs
def oracle_sample(bits, seconds_hint=15.0):
    """Times the CPU oracle's forward (fp64, dequantise on the fly) on a column sample of the
    4096 x 4096, M = 64 linear of the workload.  Returns (GB/s on the sampled bytes, cores, text)."""
    from oracle import rosaq_oracle as orc
    from paper_2506_13472_b200 import synth
    d, n_cols = 4096, 1024
    W = synth.weights(d, n_cols, 1, "oracle-sample", outlier_frac=0.01)
    x = synth.ActivationLaw(d, 1.0, 1, "x/attn_in").sample(M_TOKENS, "x", np.float16)
    qd = orc.quantize(W.astype(np.float32), bits, 128, K_SALIENT)
    orc.forward(x[:, :], qd)                                   # page in
    t0 = time.perf_counter()
    reps = 0
    while True:
        orc.forward(x, qd)
        reps += 1
        dt = time.perf_counter() - t0
        if dt > seconds_hint or reps >= 5000:
            break
    nb = gemm_bytes(d, n_cols, M_TOKENS, bits) * reps
    return nb / dt / 1e9, orc.num_threads(), (f"oracle forward (fp64) on {n_cols} of 4096 output columns of the "
                                              f"4096x4096 M=64 INT{bits} linear, {reps} repetitions, {dt:.1f} s")


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    vals, t_steps = [], []
    for _ in range(args.warmup):
        oracle_sample(args.bits, seconds_hint=1.0)
    text, cores = "", 1
    for _ in range(args.steps):
        t0 = time.perf_counter()
        v, cores, text = oracle_sample(args.bits, seconds_hint=max(2.0, 60.0 / max(args.steps, 1)))
        t_steps.append(time.perf_counter() - t0)
        vals.append(v)
    v = float(np.mean(vals))
    print(json.dumps({
        "impl": "reference", "metric": METRIC.replace("w4", "w%d" % args.bits), "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(1e3 * float(np.mean(t_steps)), 3), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "7B decoder-layer linears, M=64, INT%d g128 K=128 (oracle on a column sample)" % args.bits},
        "cpu_baseline": {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": text},
        "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))


# ----------------------------------------------------------------------------- main arm
def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2506_13472_b200 import binding as rb
    from paper_2506_13472_b200 import synth
    from paper_2506_13472_b200.dist import max_over_ranks, init_from_env

    rank, world, local = init_from_env("nccl" if torch.cuda.is_available() else "gloo")
    torch.cuda.set_device(local)
    peaks = load_peaks()
    model = synth.LLAMA_7B
    ctx = rb.Context(local)
    layers, xs = build_workload(ctx, args.bits, seed=1 + rank, n_layers=2, model=model)
    xs_dev = {k: torch.from_numpy(v).cuda() for k, v in xs.items()}
    runners = [LayerRunner(ctx, L, xs_dev, model) for L in layers]
    graphs = [capture(r.run) for r in runners]
    step_bytes = layer_bytes(model, args.bits)

    # ---- device-resident timing: K graph replays, barrier + synchronize on both sides
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    with ClockSampler(local) as clocks:
        ms = time_graphs(graphs, args.steps, args.warmup)
    ms = max_over_ranks(ms)
    ms_per_step = ms / args.steps
    value = world * step_bytes / (ms_per_step * 1e-3) / 1e9

    # ---- end to end: pinned host activations in, results out, every step
    hx = {k: torch.from_numpy(v).pin_memory() for k, v in xs.items()}
    hy = {k: torch.empty(v.shape, dtype=torch.float16).pin_memory() for k, v in runners[0].y.items()}
    h2d = sum(v.numel() * 2 for v in hx.values())
    d2h = sum(v.numel() * 2 for v in hy.values())

    def e2e_step(i):
        r = runners[i % 2]
        for k in hx:
            xs_dev[k].copy_(hx[k], non_blocking=True)
        graphs[i % 2].replay()
        for k in hy:
            hy[k].copy_(r.y[k], non_blocking=True)

    for i in range(args.warmup):
        e2e_step(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(args.steps):
        e2e_step(i)
    e1.record()
    torch.cuda.synchronize()
    e2e_ms = max_over_ranks(e0.elapsed_time(e1)) / args.steps
    e2e_value = world * step_bytes / (e2e_ms * 1e-3) / 1e9
    assert ctx.last_status() == 0

    if rank != 0:
        return
    achieved = step_bytes / (ms_per_step * 1e-3) / 1e9
    line = {
        "metric": METRIC.replace("w4", "w%d" % args.bits), "value": round(value, 2), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(ms_per_step, 5), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f16", "data": "synthetic",
        "config": {"workload": "LLaMA-7B decoder-layer linears (q,k,v,o,gate,up,down) + 3 online rotations (dense "
                               "for q/k/v and gate/up inputs, head-wise 32 x 128 for o_proj input), "
                               "M=64, INT%d g128, K=128 FP16 salient, seed 1" % args.bits,
                   "bits": args.bits, "M": M_TOKENS, "bytes_per_step": step_bytes,
                   "cold_l2": "steps alternate between two layers of distinct weights (2 x %.0f MB > 126 MB L2)"
                              % (step_bytes / 1e6),
                   "replicas": "independent replica per GPU, no collective" if world > 1 else "single GPU"},
        "clocks": clocks.summary(),
        "gpu_launches": LayerRunner.LAUNCHES * args.steps,
        "e2e": {"value": round(e2e_value, 2), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": round(e2e_ms, 5)},
        "roofline": {"bound": "hbm", "achieved": round(achieved, 1), "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": round(achieved / peaks["hbm_gbs"], 4),
                     "traffic": TRAFFIC_BYTES_PER_LAUNCH if args.bits == 4 else None,
                     "peak_source": peaks["source"], "kernel": "linear_tc_kernel / linear_sk_kernel (all 7 launches of a step: 3 rotations, qkv, o, gate+up, down)",
                     "frac_of_8tbs": round(achieved / NOMINAL_HBM_GBS, 4)},
    }
    if not args.no_table:
        reps = max(args.steps // len(layers), 1)
        fms = time_graphs([fp16_layer_graph(layers, xs_dev, model)], reps, args.warmup) / (reps * len(layers))
        line["fp16_layer"] = {"what": "the 7 GEMMs of the layer with fp16 weights through cuBLAS, same graph replay",
                              "ms_per_step": round(fms, 5), "speedup_of_this_path": round(fms / ms_per_step, 3)}
        line["gemm_stage"] = gemm_stage_table(ctx, model, args.bits, peaks)
        line["calib_cov"] = calib_cov_throughput(ctx, peaks)
    if not args.no_cpu_baseline and world == 1:
        v, cores, text = oracle_sample(args.bits)
        line["cpu_baseline"] = {"value": round(v, 4), "unit": UNIT, "cores": cores, "kind": "oracle", "sample": text}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--bits", type=int, default=4, choices=[3, 4])
    ap.add_argument("--no-table", action="store_true", help="skip the per-shape GEMM-stage / cuBLAS table")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--profile-shape", type=int, nargs=4, metavar=("D_IN", "D_OUT", "M", "BITS"),
                    help="time the GEMM stage alone on one shape (random weights) and exit")
    ap.add_argument("--profile-cov", type=int, nargs=2, metavar=("TOKENS", "D"),
                    help="time rosaq_calib_cov alone on TOKENS x D fp16 activations and exit")
    ap.add_argument("--copies", type=int, default=0, help="--profile-shape: distinct weight copies (default: 2 x L2)")
    ap.add_argument("--with-cublas", action="store_true", help="--profile-shape: also time a cuBLAS FP16 GEMM of the shape")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.profile_shape:
        args.steps = min(args.steps, 30)
        return profile_shape(args)
    if args.profile_cov:
        from paper_2506_13472_b200 import binding as rb
        print(json.dumps(calib_cov_throughput(rb.Context(0), load_peaks(), *args.profile_cov)))
        return
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
