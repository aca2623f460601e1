#!/usr/bin/env python
"""Benchmark of the ROSAQ hot path on B200.

Workload (N = 1): the seven linears of a LLaMA-7B-shaped decoder layer at M = 64 decode tokens, INT4 g128
with K = 128 FP16 salient channels (seeded synthetic weights and activations), replayed over 32 layers of
distinct weights.  One step = one pass over one layer: three online rotations x.R (attention input and MLP
input: dense 4096 x 4096 fp16 R; o_proj input: head-wise, 32 blocks of 128 x 128 plus the global eigenvalue
order, Eq. 6) and seven GEMM stages (q, k, v, o, gate, up, down; down_proj is not rotated but quantized as
D W with a per-input-channel scale, as in the paper's appendix on weight splitting).  The ten operations of a
layer run as ONE persistent launch (rosaq_plan); the 32 plans are replayed in turn from a CUDA graph, so a
layer's 197 MB are never L2-resident when it runs.  Layers 0 and 1 go through the whole pipeline
(rosaq_calib_cov, eigensolve, rosaq_quantize); the other 30 get random packed codes and random fp16 rotation
operands of the same shapes (their values do not matter for the timing, their bytes are distinct).

metric/value: algorithmic bytes of the step (packed codes + scales/zeros + FP16 salient rows + activations in
and out + the fp16 rotation matrices) divided by the device time, in GB/s.  `gemm_stage` reports the GEMM
stage alone per shape next to a cuBLAS FP16 GEMM of the same shape in the same harness; `configs` carries the
INT3 and 13B-shape sweeps and the calibration stream.

`--impl reference` times the CPU oracle (oracle/) on a bounded sample of the same workload.
"""
import argparse
import hashlib
import json
import os
import re
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
N_LAYERS = 32
MIN_TIMED_SECONDS = 1.0
KERNEL_SOURCES = ("linear_plan.cu", "linear_common.cuh", "ptx.cuh")


def kernel_fingerprint():
    """First 16 hex digits of the SHA-256 of the sources of the timed kernel."""
    h = hashlib.sha256()
    for f in KERNEL_SOURCES:
        h.update(open(os.path.join(ROOT, "paper_2506_13472_b200", "csrc", f), "rb").read())
    return h.hexdigest()[:16]


def recorded_traffic():
    """DRAM bytes per launch of the layer plan from the tracked ncu summary, or None when that summary was
    taken on other kernel sources than the ones in the tree (the figure is then stale)."""
    p = os.path.join(ROOT, "profiles", "linear_plan_7b_layer_m64.md")
    if not os.path.exists(p):
        return None
    text = open(p).read()
    fp = re.search(r"kernel sources sha256/16:\s*([0-9a-f]{16})", text)
    tr = re.search(r"dram bytes per launch \(read \+ write\):\s*([0-9]+)", text)
    if not fp or not tr or fp.group(1) != kernel_fingerprint():
        return None
    return int(tr.group(1))


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
def check_rotation(Cg, R):
    """The conditions under which a library eigensolver's R is accepted (it stands in for the eigensolve
    between rosaq_calib_cov and rosaq_quantize): orthogonal, eigenpairs of C, eigenvalues descending."""
    import torch
    C64 = Cg.to(torch.float64)
    C64 = 0.5 * (C64 + C64.T)
    lam = torch.einsum("ij,ij->j", R, C64 @ R)
    nC = torch.linalg.norm(C64)
    eye = torch.eye(R.shape[0], dtype=torch.float64, device=R.device)
    ok = (float((R.T @ R - eye).abs().max()) <= 1e-9 and float((C64 @ R - R * lam[None, :]).abs().max()) <= 1e-7 * float(nC)
          and bool((lam[1:] - lam[:-1] <= 1e-7 * nC).all()))
    if not ok:
        raise RuntimeError("eigensolver output rejected: not orthogonal, not eigenpairs of C, or not descending")


def build_layer_full(ctx, bits, seed, li, model):
    """One decoder layer through the whole pipeline: calibrate, eigensolve, rotate + quantize."""
    import torch
    from paper_2506_13472_b200 import pca, synth
    d, f = model["d"], model["ffn"]
    rots, R32, perms = {}, {}, {}
    for inp in ("attn_in", "mlp_in"):                                # layer-wise PCA, dense R (Section 3.1)
        law = synth.ActivationLaw(d, 1.0, seed, f"L{li}/{inp}")
        X = torch.from_numpy(law.sample(2048, "calib", np.float16)).cuda()
        Cg = torch.zeros((d, d), dtype=torch.float32, device="cuda")
        ctx.calib_cov(X, Cg)
        R = pca.eigh_descending_device(Cg)                           # fp64 on the device, host-side step
        check_rotation(Cg, R)
        R32[inp] = R.to(torch.float32).contiguous()
        rots[inp] = ctx.rotation_create(R.to(torch.float16).contiguous())
    # o_proj input: head-wise PCA (Section 3.1.1, Eq. 6): one 128 x 128 rotation per head from per-head
    # activations, plus the global descending-eigenvalue column order
    H, hd = model["heads"], model["head_dim"]
    Xh = torch.from_numpy(head_law(model, seed).sample(4096, f"L{li}/calib", np.float16)).cuda()
    Cb = torch.zeros((H, hd, hd), dtype=torch.float32, device="cuda")
    ctx.calib_cov(Xh, Cb, n_blocks=H)
    Rb, perm, _ = pca.headwise_rotation(Cb.cpu().numpy())
    R32["o_in"] = torch.from_numpy(Rb.astype(np.float32)).cuda()
    perms["o_in"] = torch.from_numpy(perm).cuda()
    rots["o_in"] = ctx.rotation_create(torch.from_numpy(Rb.astype(np.float16)).cuda(), perms["o_in"])
    # down_proj: not rotated; D W with the fixed mean|x|^0.5 rule on synthetic calibration activations
    dlaw = synth.ActivationLaw(f, 1.0, seed, "x/down_in")
    dsc = torch.from_numpy(pca.channel_scale(dlaw.sample(512, f"L{li}/calib", np.float32))).cuda()
    weights, fp16 = {}, {}
    for name, d_in, d_out, inp in synth.layer_shapes(model):
        W = torch.from_numpy(synth.weights(d_in, d_out, seed, f"L{li}/{name}", sigma=0.02,
                                           outlier_frac=0.01, outlier_scale=10.0)).cuda()
        weights[name] = ctx.quantize(W, R32.get(inp), perms.get(inp), bits=bits, k_salient=K_SALIENT,
                                     in_scale=dsc if name == "down" else None)
        fp16[name] = W
    return dict(rots=rots, weights=weights, fp16=fp16, down_scale=dsc)


def random_weight(ctx, gen, d_in, d_out, bits):
    """A weight handle made of random packed codes, scales, zeros and salient rows (timing only)."""
    import torch
    nq = d_in - K_SALIENT
    nw = nq // 8 if bits == 4 else nq // 32 * 3
    qw = torch.randint(-2 ** 31, 2 ** 31 - 1, (nw, d_out), dtype=torch.int64, device="cuda", generator=gen).to(torch.int32)
    sc = (torch.rand((nq // 128, d_out), device="cuda", generator=gen) * 0.01 + 0.001).half()
    zr = torch.randint(0, 2 ** bits, (nq // 128, d_out), device="cuda", generator=gen).half()
    sal = (torch.randn((K_SALIENT, d_out), device="cuda", generator=gen) * 0.02).half()
    return ctx.weight_import(d_in, d_out, bits, 128, K_SALIENT, qw, sc, zr, sal)


def build_layer_random(ctx, bits, gen, model):
    """A layer of the same shapes with random operands: distinct bytes for the cold-cache replay."""
    import torch
    from paper_2506_13472_b200 import synth
    d, H, hd = model["d"], model["heads"], model["head_dim"]
    rnd = lambda *shape: (torch.randn(shape, device="cuda", generator=gen) / shape[-1] ** 0.5).half()
    rots = {"attn_in": ctx.rotation_create(rnd(d, d)), "mlp_in": ctx.rotation_create(rnd(d, d)),
            "o_in": ctx.rotation_create(rnd(H, hd, hd), torch.randperm(d, device="cuda", generator=gen).to(torch.int32))}
    weights = {name: random_weight(ctx, gen, d_in, d_out, bits) for name, d_in, d_out, _ in synth.layer_shapes(model)}
    return dict(rots=rots, weights=weights, fp16=None)


def build_workload(ctx, bits, seed, n_layers, model, n_full=2):
    """`n_layers` decoder layers (the first `n_full` through the whole pipeline) and the step's activations."""
    import torch
    from paper_2506_13472_b200 import synth
    d, f = model["d"], model["ffn"]
    gen = torch.Generator(device="cuda").manual_seed(1000 + seed)
    layers = [build_layer_full(ctx, bits, seed, li, model) if li < n_full else build_layer_random(ctx, bits, gen, model)
              for li in range(n_layers)]
    xs = {}
    for inp, dd in (("attn_in", d), ("mlp_in", d), ("down_in", f)):
        law = synth.ActivationLaw(dd, 1.0, seed, f"x/{inp}")
        xs[inp] = law.sample(M_TOKENS, "x", np.float16)
    xs["o_in"] = head_law(model, seed).sample(M_TOKENS, "x", np.float16)
    # what the caller feeds the scaled down_proj: x D^-1 (absorbed upstream in a real model)
    dsc = layers[0]["down_scale"].cpu().numpy()
    xs["down_in"] = (xs["down_in"].astype(np.float32) / dsc[None, :]).astype(np.float16)
    return layers, xs


def head_law(model, seed):
    from paper_2506_13472_b200 import synth
    return synth.HeadwiseActivationLaw(model["heads"], model["head_dim"], seed, "o_in")


def layer_bytes(model, bits):
    from paper_2506_13472_b200 import synth
    b = sum(gemm_bytes(di, do, M_TOKENS, bits) for _, di, do, _ in synth.layer_shapes(model))
    return b + 2 * rotate_bytes(model["d"], M_TOKENS) + rotate_bytes(model["d"], M_TOKENS, model["heads"])


class LayerRunner:
    """Owns the output buffers of one layer pass and its plans.  `run` is the timed step: the ten operations
    of the layer as one rosaq_plan launch.  `run_units` is the same work as four launches, one per group of
    operations that a real decoder layer could issue together (rotation + q/k/v, rotation + o, rotation +
    gate/up, down): reported next to the headline."""
    LAUNCHES = 1
    OUT = ("q", "k", "v", "o", "gate", "up", "down")

    def __init__(self, ctx, layer, x, y, xr):
        self.ctx, self.L, self.x, self.y, self.xr = ctx, layer, x, y, xr
        R, W = layer["rots"], layer["weights"]
        rot_ops = [(x["attn_in"], None, R["attn_in"], xr["attn_in"]), (x["mlp_in"], None, R["mlp_in"], xr["mlp_in"]),
                   (x["o_in"], None, R["o_in"], xr["o_in"])]
        self.plan = ctx.plan_create(M_TOKENS, rot_ops + [(x["down_in"], None, W["down"], y["down"])] +
                                    [(None, 0, W[n], y[n]) for n in ("q", "k", "v")] + [(None, 2, W["o"], y["o"])] +
                                    [(None, 1, W[n], y[n]) for n in ("gate", "up")])
        self.units = None

    def make_units(self):
        c, x, y, xr, R, W = self.ctx, self.x, self.y, self.xr, self.L["rots"], self.L["weights"]
        self.units = [
            c.plan_create(M_TOKENS, [(x["attn_in"], None, R["attn_in"], xr["attn_in"])] + [(None, 0, W[n], y[n]) for n in ("q", "k", "v")]),
            c.plan_create(M_TOKENS, [(x["o_in"], None, R["o_in"], xr["o_in"]), (None, 0, W["o"], y["o"])]),
            c.plan_create(M_TOKENS, [(x["mlp_in"], None, R["mlp_in"], xr["mlp_in"])] + [(None, 0, W[n], y[n]) for n in ("gate", "up")]),
            c.plan_create(M_TOKENS, [(x["down_in"], None, W["down"], y["down"])])]

    def run(self):
        self.plan.run()

    def run_units(self):
        for u in self.units:
            u.run()


def step_buffers(model, xs):
    """Device buffers shared by all layers of a replay: inputs x (one contiguous allocation, so that the
    end-to-end leg copies them in one transfer), rotated activations, outputs y (one allocation as well)."""
    import torch
    d, f = model["d"], model["ffn"]
    widths_in = (("attn_in", d), ("mlp_in", d), ("o_in", d), ("down_in", f))
    xin = torch.empty((M_TOKENS, sum(w for _, w in widths_in)), dtype=torch.float16, device="cuda")
    x, c0 = {}, 0
    for k, w in widths_in:
        x[k] = xin[:, c0:c0 + w]
        x[k].copy_(torch.from_numpy(xs[k]))
        c0 += w
    widths_out = (("q", d), ("k", d), ("v", d), ("o", d), ("gate", f), ("up", f), ("down", d))
    yout = torch.empty((M_TOKENS, sum(w for _, w in widths_out)), dtype=torch.float16, device="cuda")
    y, c0 = {}, 0
    for k, w in widths_out:
        y[k] = yout[:, c0:c0 + w]
        c0 += w
    xr = {k: torch.empty((M_TOKENS, d), dtype=torch.float16, device="cuda") for k in ("attn_in", "o_in", "mlp_in")}
    return xin, x, yout, y, xr


def fp16_layer_graph(layers, x, model):
    """The same seven GEMMs per layer with the un-rotated fp16 weights through cuBLAS (torch.matmul): one
    CUDA graph that walks over the given layers in turn (each layer's fp16 weights alone exceed the L2);
    a replay is len(layers) steps.  The FP16 baseline of the layer replay."""
    import torch
    d, f = model["d"], model["ffn"]
    mk = lambda n: torch.empty((M_TOKENS, n), dtype=torch.float16, device="cuda")
    y = {"q": mk(d), "k": mk(d), "v": mk(d), "o": mk(d), "gate": mk(f), "up": mk(f), "down": mk(d)}
    inp = {"q": "attn_in", "k": "attn_in", "v": "attn_in", "o": "o_in", "gate": "mlp_in", "up": "mlp_in",
           "down": "down_in"}
    xc = {k: v.contiguous() for k, v in x.items()}

    def run():
        for L in layers:
            for n in ("q", "k", "v", "o", "gate", "up", "down"):
                torch.matmul(xc[inp[n]], L["fp16"][n], out=y[n])
    return capture(run)


def time_replays(graph, steps_per_replay, min_seconds=MIN_TIMED_SECONDS, segments=5, warmup_replays=3):
    """Replays `graph` for at least `min_seconds` in `segments` segments timed with CUDA events on the current
    stream; returns (median ms per step, total steps timed, total ms)."""
    import torch
    for _ in range(warmup_replays):
        graph.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    graph.replay()
    e1.record()
    torch.cuda.synchronize()
    one = max(e0.elapsed_time(e1), 1e-3)
    reps = max(1, int(np.ceil(min_seconds * 1e3 / segments / one)))
    per_step, total = [], 0.0
    for _ in range(segments):
        e0.record()
        for _ in range(reps):
            graph.replay()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1)
        total += ms
        per_step.append(ms / (reps * steps_per_replay))
    return float(np.median(per_step)), segments * reps * steps_per_replay, total


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


def gemm_stage_table(ctx, model, bits, peaks, Ms=(M_TOKENS,), reps=12, with_cublas=True):
    """Per shape and token count: the GEMM stage alone (rosaq_linear on rotated input, one launch per call)
    over >= 2 x L2 of distinct weight copies replayed from a CUDA graph, next to a cuBLAS FP16 GEMM."""
    import torch
    d, f = model["d"], model["ffn"]
    gen = torch.Generator(device="cuda").manual_seed(7)
    out = []
    for d_in, d_out in ((d, d), (d, f), (f, d)):
        w0 = random_weight(ctx, gen, d_in, d_out, bits)
        copies = max(2, int(np.ceil(2 * 126e6 / w0.device_bytes)))
        ws = [w0] + [random_weight(ctx, gen, d_in, d_out, bits) for _ in range(copies - 1)]
        fcopies = max(2, int(np.ceil(2 * 126e6 / (d_in * d_out * 2))))
        Wf = [(torch.randn((d_in, d_out), device="cuda", generator=gen) * 0.02).half() for _ in range(fcopies)] if with_cublas else []
        for M in Ms:
            x = torch.randn((M, d_in), device="cuda", generator=gen).half()
            y = torch.empty((M, d_out), dtype=torch.float16, device="cuda")
            g = capture(lambda: [ctx.linear(x, w, None, out=y) for w in ws])
            us = sorted(time_graphs([g], 1, 1) for _ in range(reps))[reps // 2] * 1e3 / copies
            nb = gemm_bytes(d_in, d_out, M, bits)
            gbs = nb / us / 1e3
            row = dict(shape=f"{d_in}x{d_out}", M=M, bits=bits, us=round(us, 3), gbs=round(gbs, 1),
                       frac_of_8tbs=round(gbs / NOMINAL_HBM_GBS, 4), frac_of_measured=round(gbs / peaks["hbm_gbs"], 4),
                       tflops=round(2.0 * M * d_in * d_out / us / 1e6, 1))
            if with_cublas:
                gf = capture(lambda: [torch.matmul(x, w, out=y) for w in Wf])
                usf = sorted(time_graphs([gf], 1, 1) for _ in range(reps))[reps // 2] * 1e3 / fcopies
                row.update(cublas_fp16_us=round(usf, 3), speedup_vs_cublas_fp16=round(usf / us, 3))
            out.append(row)
            del g
        for w in ws:
            w.free()
        del Wf
        torch.cuda.empty_cache()
    return out


def calib_stream(ctx, peaks, d=5120, chunk=16384, chunks=16):
    """rosaq_calib_cov over a 13B-shaped calibration stream: `chunks` chunks of `chunk` fp16 tokens generated
    on the device and accumulated into one fp32 Gram matrix (the tokens are never resident at once)."""
    import torch
    gen = torch.Generator(device="cuda").manual_seed(4)
    Cm = torch.zeros((d, d), dtype=torch.float32, device="cuda")
    X = torch.randn((chunk, d), device="cuda", generator=gen).half()
    ctx.calib_cov(X, Cm)
    Cm.zero_()
    torch.cuda.synchronize()
    ms = 0.0
    for c in range(chunks):
        X = torch.randn((chunk, d), device="cuda", generator=gen).half()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        ctx.calib_cov(X, Cm)
        e1.record()
        torch.cuda.synchronize()
        ms += e0.elapsed_time(e1)
    nb = (d + 255) // 256
    executed = 2.0 * chunk * chunks * 256 * 256 * (nb * (nb + 1) // 2)
    tf = executed / ms / 1e9
    return dict(tokens=chunk * chunks, d=d, chunks=chunks, ms=round(ms, 3), tflops=round(tf, 1),
                frac_of_bf16_peak=round(tf / peaks["bf16_tflops"], 4), peak_source=peaks["source"])


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


def profile_layer(args):
    """The layer plan alone over a few layers of random operands (distinct bytes, more than the L2 together):
    the small, self-contained case that ncu captures of linear_plan_kernel are taken on.  Prints one line."""
    import torch
    from paper_2506_13472_b200 import binding as rb
    from paper_2506_13472_b200 import synth
    n_layers, bits = args.profile_layer
    model = synth.LLAMA_7B
    ctx = rb.Context(0)
    gen = torch.Generator(device="cuda").manual_seed(0)
    layers = [build_layer_random(ctx, bits, gen, model) for _ in range(n_layers)]
    xs = {k: np.zeros((M_TOKENS, w), np.float16) for k, w in (("attn_in", model["d"]), ("mlp_in", model["d"]),
                                                               ("o_in", model["d"]), ("down_in", model["ffn"]))}
    xin, x, yout, y, xr = step_buffers(model, xs)
    xin.copy_(torch.randn(xin.shape, device="cuda", generator=gen).half())
    runners = [LayerRunner(ctx, L, x, y, xr) for L in layers]
    for _ in range(2):
        for r in runners:
            r.run()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        for r in runners:
            r.run()
    e1.record()
    torch.cuda.synchronize()
    assert ctx.last_status() == 0
    us = e0.elapsed_time(e1) * 1e3 / (args.steps * n_layers)
    nb = layer_bytes(model, bits)
    print(json.dumps({"layers": n_layers, "bits": bits, "launches": (2 + args.steps) * n_layers, "us_per_launch_in_stream": round(us, 2),
                      "bytes_per_launch": nb, "kernel_sources_sha256_16": kernel_fingerprint()}))


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
_ORACLE_INPUTS = {}


def _oracle_sample_inputs(bits, d, n_cols):
    """Seeded inputs of the oracle sample, built once per process (quantized by the oracle itself)."""
    key = (bits, d, n_cols)
    if key not in _ORACLE_INPUTS:
        from oracle import rosaq_oracle as orc
        from paper_2506_13472_b200 import synth
        W = synth.weights(d, n_cols, 1, "oracle-sample", outlier_frac=0.01)
        x = synth.ActivationLaw(d, 1.0, 1, "x/attn_in").sample(M_TOKENS, "x", np.float16)
        qd = orc.quantize(W.astype(np.float32), bits, 128, K_SALIENT)
        orc.forward(x[:, :], qd)                               # page in
        _ORACLE_INPUTS[key] = (x, qd)
    return _ORACLE_INPUTS[key]


def oracle_sample(bits, seconds_hint=15.0):
    """Times the CPU oracle's forward (fp64, dequantise on the fly) on a column sample of the
    4096 x 4096, M = 64 linear of the workload.  Returns (GB/s on the sampled bytes, cores, text)."""
    from oracle import rosaq_oracle as orc
    d, n_cols = 4096, 1024
    x, qd = _oracle_sample_inputs(bits, d, n_cols)
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


def _omp_set_threads(n):
    """Sets the OpenMP thread count of this process (the oracle's loops are `omp parallel for`)."""
    import ctypes
    try:
        ctypes.CDLL("libgomp.so.1").omp_set_num_threads(int(n))
        return True
    except OSError:
        return False


def oracle_extra_timings(bits, seconds=2.0):
    """The other oracle steps of the path, each on a bounded sample: the forward on one thread, the Gram
    matrix (Eq. 4), and rotate + quantize (fp32 chain, RTN) on a column sample."""
    from oracle import rosaq_oracle as orc
    from paper_2506_13472_b200 import synth
    out = {}
    cores = orc.num_threads()

    def timed(fn, budget):
        fn()
        t0, reps = time.perf_counter(), 0
        while True:
            fn()
            reps += 1
            dt = time.perf_counter() - t0
            if dt > budget or reps >= 1000:
                return dt / reps
    d, n_cols = 4096, 256
    W = synth.weights(d, n_cols, 1, "oracle-sample", outlier_frac=0.01)
    x = synth.ActivationLaw(d, 1.0, 1, "x/attn_in").sample(M_TOKENS, "x", np.float16)
    qd = orc.quantize(W.astype(np.float32), bits, 128, K_SALIENT)
    if _omp_set_threads(1):
        t = timed(lambda: orc.forward(x, qd), seconds)
        out["forward_1_thread"] = dict(gbs=round(gemm_bytes(d, n_cols, M_TOKENS, bits) / t / 1e9, 4),
                                       sample=f"{n_cols} of 4096 columns of the 4096x4096 M=64 linear")
        _omp_set_threads(cores)
    X = synth.ActivationLaw(1024, 1.0, 1, "oracle-cov").sample(2048, "calib", np.float16)
    t = timed(lambda: orc.cov(X), seconds)
    out["cov"] = dict(gflops=round(2.0 * 2048 * 1024 * 1024 / t / 1e9, 2), cores=cores, sample="2048 tokens x 1024 channels (fp64)")
    R32 = np.eye(d, dtype=np.float32)
    cols = np.arange(16, dtype=np.int32)
    t = timed(lambda: orc.quantize(orc.rotate_weights_f32(R32, W, None, cols), bits, 128, K_SALIENT), seconds)
    out["rotate_quantize"] = dict(columns_per_s=round(16 / t, 1), cores=cores,
                                  sample="16 output columns of a 4096-row weight: fp32 chain of 4096 terms per element, then RTN")
    return out


def workload_string(bits):
    """Name of the timed workload, the same for both arms."""
    return ("LLaMA-7B decoder-layer linears (q,k,v,o,gate,up,down) + 3 online rotations (dense for q/k/v and gate/up "
            "inputs, head-wise 32 x 128 for o_proj input), M=64, INT%d g128, K=128 FP16 salient, seed 1" % bits)


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    vals, t_steps = [], []
    # a step is a bounded sample of the workload: the whole run takes about two minutes whatever K and W are
    for _ in range(args.warmup):
        oracle_sample(args.bits, seconds_hint=min(1.0, 20.0 / args.warmup))
    text, cores = "", 1
    for _ in range(args.steps):
        t0 = time.perf_counter()
        v, cores, text = oracle_sample(args.bits, seconds_hint=min(30.0, 120.0 / max(args.steps, 1)))
        t_steps.append(time.perf_counter() - t0)
        vals.append(v)
    v = float(np.mean(vals))
    print(json.dumps({
        "impl": "reference", "metric": METRIC.replace("w4", "w%d" % args.bits), "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(1e3 * float(np.mean(t_steps)), 3), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_string(args.bits), "bits": args.bits, "M": M_TOKENS,
                   "sample": "every step is a bounded sample of that workload on the host cores: " + text},
        "cpu_baseline": {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": text},
        "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))


# ----------------------------------------------------------------------------- main arm
def extras(line, args, ctx, rb, model, layers, runners, x, peaks, ms_per_step):
    """Everything next to the headline: the FP16 layer, the step as four launches, per-shape GEMM stages, and
    the other configurations (INT3 at several token counts, 13B shapes, the calibration stream)."""
    import torch
    from paper_2506_13472_b200 import synth
    full = [L for L in layers if L["fp16"] is not None]
    fms, _, _ = time_replays(fp16_layer_graph(full, x, model), len(full), min_seconds=0.3)
    line["fp16_layer"] = {"what": "the 7 GEMMs of the layer with fp16 weights through cuBLAS, same graph replay "
                                  "(2 layers of 415 MB in turn)",
                          "ms_per_step": round(fms, 5), "speedup_of_this_path": round(fms / ms_per_step, 3)}
    for r in runners:
        r.make_units()
    ums, _, _ = time_replays(layer_plans_graph(runners, units=True), len(runners), min_seconds=0.5)
    line["four_launches"] = {"what": "the same step as four rosaq_plan launches (rotation + q/k/v, rotation + o, "
                                     "rotation + gate/up, down): what a decoder layer with attention and an "
                                     "activation function between them could issue",
                             "ms_per_step": round(ums, 5), "gbs": round(line["config"]["bytes_per_step"] / ums / 1e6, 1)}
    for r in runners:
        for u in r.units:
            u.free()
        r.units = None
    line["gemm_stage"] = gemm_stage_table(ctx, model, args.bits, peaks)
    if args.quick:
        return
    configs = []
    other = 3 if args.bits == 4 else 4
    # the other code width: the layer step, and the GEMM stage over the token counts of the sweep
    gen = torch.Generator(device="cuda").manual_seed(2)
    for r in runners:
        r.plan.free()
    olayers = [build_layer_random(ctx, other, gen, model) for _ in range(len(layers))]
    orun = [LayerRunner(ctx, L, r.x, r.y, r.xr) for L, r in zip(olayers, runners)]
    oms, _, _ = time_replays(layer_plans_graph(orun), len(orun), min_seconds=0.5)
    ob = layer_bytes(model, other)
    configs.append({"config": "7B shapes, INT%d g128, K=128" % other,
                    "layer_step_m64": {"ms_per_step": round(oms, 5), "gbs": round(ob / oms / 1e6, 1), "bytes_per_step": ob,
                                       "frac_of_measured": round(ob / oms / 1e6 / peaks["hbm_gbs"], 4)},
                    "gemm_stage": gemm_stage_table(ctx, model, other, peaks, Ms=(1, 16, 64, 256), reps=8)})
    for r in orun:
        r.plan.free()
    del olayers, orun
    torch.cuda.empty_cache()
    m13 = synth.LLAMA_13B
    configs.append({"config": "13B shapes (5120 / 13824), K=128, M in {1, 64, 512}",
                    "gemm_stage_int4": gemm_stage_table(ctx, m13, 4, peaks, Ms=(1, 64, 512), reps=8),
                    "gemm_stage_int3": gemm_stage_table(ctx, m13, 3, peaks, Ms=(1, 64, 512), reps=8, with_cublas=False),
                    "calib_cov": calib_stream(ctx, peaks)})
    # prefill-sized batches: from a few hundred tokens on rosaq_linear runs 256 x 256 tiles on pairs of CTAs
    configs.append({"config": "prefill: 13B and 7B shapes, INT4, M in {1024, 2048}",
                    "gemm_stage_13b": gemm_stage_table(ctx, m13, 4, peaks, Ms=(1024, 2048), reps=5),
                    "gemm_stage_7b": gemm_stage_table(ctx, model, 4, peaks, Ms=(1024, 2048), reps=5)})
    line["configs"] = configs


def layer_plans_graph(runners, units=False):
    """One CUDA graph that runs every layer once, in turn."""
    if units:
        return capture(lambda: [r.run_units() for r in runners])
    return capture(lambda: [r.run() for r in runners])


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
    n_layers = args.layers
    layers, xs = build_workload(ctx, args.bits, seed=1 + rank, n_layers=n_layers, model=model)
    xin, x, yout, y, xr = step_buffers(model, xs)
    runners = [LayerRunner(ctx, L, x, y, xr) for L in layers]
    graph = layer_plans_graph(runners)
    step_bytes = layer_bytes(model, args.bits)
    gemm_only_bytes = sum(gemm_bytes(di, do, M_TOKENS, args.bits) for _, di, do, _ in synth.layer_shapes(model))

    # ---- device-resident timing.  The contract's K steps: K passes over a layer, taken round-robin over the
    # n_layers distinct layers (W warm-up steps first), barrier + synchronize on both sides ...
    def k_steps(k, start=0):
        full, rest = divmod(k, n_layers)
        for _ in range(full):
            graph.replay()
        for i in range(rest):
            runners[(start + i) % n_layers].run()

    k_steps(max(args.warmup, 3))
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(local) as clocks:
        e0.record()
        k_steps(args.steps)
        e1.record()
        torch.cuda.synchronize()
        ms_k = max_over_ranks(e0.elapsed_time(e1)) / args.steps
        # ... and, because K steps of 66 us are over before a clock sample is taken, the same replay for at
        # least a second in five segments: the median segment is the reported figure
        ms_per_step, steps_timed, ms_total = time_replays(graph, n_layers)
    ms_per_step = max_over_ranks(ms_per_step)
    value = world * step_bytes / (ms_per_step * 1e-3) / 1e9

    # ---- end to end: one pinned buffer each way, every step.  Steps are pipelined over three streams and two
    # sets of device buffers: while step i runs, the inputs of step i + 1 come in and the outputs of step
    # i - 1 go out (every step still copies all of its inputs in and all of its outputs out).
    hx = torch.empty(xin.shape, dtype=torch.float16).pin_memory()
    hx.copy_(xin.cpu())
    h2d, d2h = hx.numel() * 2, yout.numel() * 2
    sets = [(xin, yout, runners)]
    xin2, x2, yout2, y2, xr2 = step_buffers(model, xs)
    sets.append((xin2, yout2, [LayerRunner(ctx, L, x2, y2, xr2) for L in layers]))
    hys = [torch.empty(yout.shape, dtype=torch.float16).pin_memory() for _ in sets]
    s_c = torch.cuda.current_stream()
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    ev_in = [torch.cuda.Event() for _ in sets]
    ev_c = [torch.cuda.Event() for _ in sets]
    ev_out = [torch.cuda.Event() for _ in sets]

    def e2e_step(i):
        b = i % len(sets)
        xin_b, yout_b, runners_b = sets[b]
        with torch.cuda.stream(s_in):
            s_in.wait_event(ev_c[b])                      # the step that read this input buffer is done
            xin_b.copy_(hx, non_blocking=True)
            ev_in[b].record(s_in)
        s_c.wait_event(ev_in[b])
        s_c.wait_event(ev_out[b])                         # the previous outputs of this buffer have left
        runners_b[i % n_layers].run()
        ev_c[b].record(s_c)
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev_c[b])
            hys[b].copy_(yout_b, non_blocking=True)
            ev_out[b].record(s_out)

    def e2e_join():
        for b in range(len(sets)):
            s_c.wait_event(ev_out[b])

    for i in range(max(args.warmup, 3)):
        e2e_step(i)
    e2e_join()
    torch.cuda.synchronize()
    n_e2e = max(args.steps, 200)
    e0.record()
    for i in range(n_e2e):
        e2e_step(i)
    e2e_join()
    e1.record()
    torch.cuda.synchronize()
    e2e_ms = max_over_ranks(e0.elapsed_time(e1)) / n_e2e
    # the last step's outputs, read back on the host, are those of a plain run of the same layer
    last = (n_e2e - 1) % len(sets)
    ref_y = sets[last][1].clone()
    assert torch.equal(hys[last].cuda().view(torch.int16), ref_y.view(torch.int16))
    e2e_value = world * step_bytes / (e2e_ms * 1e-3) / 1e9
    assert ctx.last_status() == 0

    if rank != 0:
        return
    achieved = step_bytes / (ms_per_step * 1e-3) / 1e9
    gemm_formula = gemm_only_bytes / (ms_per_step * 1e-3) / 1e9
    line = {
        "metric": METRIC.replace("w4", "w%d" % args.bits), "value": round(value, 2), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(ms_per_step, 5), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f16", "data": "synthetic",
        "config": {"workload": workload_string(args.bits),
                   "bits": args.bits, "M": M_TOKENS, "bytes_per_step": step_bytes, "layers": n_layers,
                   "launch": "one persistent launch per step (rosaq_plan over the 10 operations of a layer)",
                   "cold_l2": "steps walk over %d layers of distinct weights (%d x %.0f MB, L2 is 126 MB)"
                              % (n_layers, n_layers, step_bytes / 1e6),
                   "timing": "median of 5 segments, %d steps in %.0f ms; the K=%d steps of the contract alone: %.5f ms per step"
                             % (steps_timed, ms_total, args.steps, ms_k),
                   "replicas": "independent replica per GPU, no collective" if world > 1 else "single GPU"},
        "clocks": clocks.summary(),
        "gpu_launches": LayerRunner.LAUNCHES * (args.steps + steps_timed),
        "e2e": {"value": round(e2e_value, 2), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": round(e2e_ms, 5), "steps": n_e2e,
                "how": "rosaq_plan_run per step with one pinned host->device copy of the step's inputs and one "
                       "device->host copy of its outputs; three streams and two sets of device buffers, so the "
                       "copies of neighbouring steps overlap the launch"},
        "roofline": {"bound": "hbm", "achieved": round(achieved, 1), "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": round(achieved / peaks["hbm_gbs"], 4), "traffic": recorded_traffic() if args.bits == 4 else None,
                     "peak_source": peaks["source"], "kernel": "linear_plan_kernel (the step's only launch)",
                     "frac_of_8tbs": round(achieved / NOMINAL_HBM_GBS, 4),
                     "without_rotation_bytes": {"what": "the same time against the bytes of the 7 GEMM stages only "
                                                        "(codes + scales + salient + activations; no R term)",
                                                "gbs": round(gemm_formula, 1),
                                                "frac_of_measured": round(gemm_formula / peaks["hbm_gbs"], 4),
                                                "frac_of_8tbs": round(gemm_formula / NOMINAL_HBM_GBS, 4)}},
    }
    if not args.no_table:
        extras(line, args, ctx, rb, model, layers, runners, x, peaks, ms_per_step)
    if not args.no_cpu_baseline and world == 1:
        v, cores, text = oracle_sample(args.bits)
        line["cpu_baseline"] = {"value": round(v, 4), "unit": UNIT, "cores": cores, "kind": "oracle", "sample": text,
                                "other_steps": oracle_extra_timings(args.bits)}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=640)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--bits", type=int, default=4, choices=[3, 4])
    ap.add_argument("--no-table", action="store_true", help="skip everything next to the headline")
    ap.add_argument("--quick", action="store_true", help="skip the other configurations (INT3 / 13B / calibration stream)")
    ap.add_argument("--layers", type=int, default=N_LAYERS, help="distinct layers the replay walks over")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--profile-shape", type=int, nargs=4, metavar=("D_IN", "D_OUT", "M", "BITS"),
                    help="time the GEMM stage alone on one shape (random weights) and exit")
    ap.add_argument("--profile-layer", type=int, nargs=2, metavar=("LAYERS", "BITS"),
                    help="run the 7B layer plan alone over LAYERS layers of random operands and exit")
    ap.add_argument("--profile-cov", type=int, nargs=2, metavar=("TOKENS", "D"),
                    help="time rosaq_calib_cov alone on TOKENS x D fp16 activations and exit")
    ap.add_argument("--copies", type=int, default=0, help="--profile-shape: distinct weight copies (default: 2 x L2)")
    ap.add_argument("--with-cublas", action="store_true", help="--profile-shape: also time a cuBLAS FP16 GEMM of the shape")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.profile_shape:
        args.steps = min(args.steps, 30)
        return profile_shape(args)
    if args.profile_layer:
        args.steps = min(args.steps, 30)
        return profile_layer(args)
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
