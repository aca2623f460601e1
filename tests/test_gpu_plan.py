"""GPU parity of rosaq_plan: several rotations and linears as one persistent launch.

Every output of a plan is compared with the CPU oracle's fp64 forward (2e-3 in Frobenius norm, and at the
full 7B layer size on every column, tile by tile and element by element), with the same operations issued
as separate calls (fp32 summation order: 2e-4), and with itself across runs and CUDA-graph replays (bit
for bit).
"""
import numpy as np
import pytest
import torch

from oracle import rosaq_oracle as orc
from paper_2506_13472_b200 import binding as rb
from paper_2506_13472_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = rb.Context(0)
    yield c
    c.close()


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def empty(M, n):
    return torch.full((M, n), float("nan"), dtype=torch.float16, device="cuda")


def householder_rotation(d, seed, key):
    vs = synth.householder_vectors(d, 6, synth.rng_for(seed, key, "R"))
    return synth.apply_householders(np.eye(d), vs)


@pytest.mark.parametrize("pairs", [True, False])
@pytest.mark.parametrize("bits,M", [(4, 4), (3, 64), (4, 33), (3, 1), (4, 128), (3, 90)])
def test_small_layer_plan_against_oracle_and_separate_calls(ctx, bits, M, pairs):
    """A decoder layer in miniature (d = 512, ffn = 1024, 4 heads): dense rotations for the attention and
    MLP inputs, a head-wise one with its permutation for the o_proj input, down_proj un-rotated."""
    d, f = 512, 1024
    ctx.set_plan_pairs(pairs)
    c, hw = H.config_tiny(), H.config_headwise()
    R2 = householder_rotation(d, 7, "plan-mlp")
    rots = {"attn": ctx.rotation_create(dev(c["R16"])),
            "mlp": ctx.rotation_create(dev(R2.astype(np.float16))),
            "o": ctx.rotation_create(dev(hw["Rb16"]), dev(hw["perm"]))}
    rot_np = {"attn": (c["R16"], None, c["R32"]), "mlp": (R2.astype(np.float16), None, R2.astype(np.float32)),
              "o": (hw["Rb16"], hw["perm"], hw["Rb32"])}
    shapes = [("q", d, d, "attn"), ("k", d, 200, "attn"), ("v", d, 136, "attn"), ("o", d, d, "o"), ("gate", d, f, "mlp"),
              ("up", d, f, "mlp"), ("down", f, d, None)]
    ws, qds = {}, {}
    for name, di, do, inp in shapes:
        W = synth.weights(di, do, 11, f"plan/{name}", outlier_frac=0.01)
        R16, perm, R32 = rot_np[inp] if inp else (None, None, None)
        ws[name] = ctx.quantize(dev(W), None if R32 is None else dev(R32), None if perm is None else dev(perm),
                                bits=bits, k_salient=128)
        qds[name] = H.oracle_quantized(W, R32, perm, bits, 128)
        H.assert_export_matches(H.export_to_numpy(ws[name].export()), qds[name])
    law = synth.ActivationLaw(d, 1.2, 0, "tiny", mix="qr")
    xs = {"attn": law.sample(M, "pa", np.float16), "mlp": law.sample(M, "pm", np.float16),
          "o": synth.HeadwiseActivationLaw(4, 128, 3, "hw").sample(M, "po", np.float16),
          "down": synth.rng_for(11, "down", M).standard_normal((M, f)).astype(np.float16)}
    xd = {k: dev(v) for k, v in xs.items()}
    xr = {k: empty(M, d) for k in ("attn", "mlp", "o")}
    ys = {name: empty(M, do) for name, _, do, _ in shapes}
    # rotations first, then the un-rotated down_proj, then the linears that read the rotated activations
    ops = [(xd["attn"], None, rots["attn"], xr["attn"]), (xd["mlp"], None, rots["mlp"], xr["mlp"]),
           (xd["o"], None, rots["o"], xr["o"]), (xd["down"], None, ws["down"], ys["down"]),
           (None, 0, ws["q"], ys["q"]), (None, 0, ws["k"], ys["k"]), (None, 0, ws["v"], ys["v"]),
           (None, 2, ws["o"], ys["o"]), (None, 1, ws["gate"], ys["gate"]), (None, 1, ws["up"], ys["up"])]
    plan = ctx.plan_create(M, ops)
    plan.run()
    assert ctx.last_status() == rb.ROSAQ_OK
    first = {k: v.clone() for k, v in ys.items()}
    for name, di, do, inp in shapes:
        got = ys[name].cpu().numpy()
        assert np.all(np.isfinite(got)), name
        R16, perm, _ = rot_np[inp] if inp else (None, None, None)
        y_ref = orc.forward(xs[inp or "down"], qds[name], R16, perm)
        assert H.rel_fro(got, y_ref) <= H.REL_TOL_Y, name
        sep = ctx.linear(xd[inp or "down"], ws[name], rots[inp] if inp else None).cpu().numpy()
        assert H.rel_fro(got, sep) <= 2e-4, name
    # the same bits on every run, also from a CUDA graph
    for t in ys.values():
        t.fill_(float("nan"))
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        plan.run()
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        plan.run()
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    assert ctx.last_status() == rb.ROSAQ_OK
    for k in ys:
        assert torch.equal(ys[k].view(torch.int16), first[k].view(torch.int16)), k
    plan.free()
    ctx.set_plan_pairs(False)


def test_plan_argument_errors(ctx):
    W = torch.zeros((256, 128), dtype=torch.float16, device="cuda")
    w4 = ctx.quantize(W, None, bits=4, k_salient=128)
    w3 = ctx.quantize(W, None, bits=3, k_salient=128)
    x, y, y2 = (torch.zeros((8, 256), dtype=torch.float16, device="cuda"), empty(8, 128), empty(8, 128))
    for ops, M, status in (
            ([(x, None, w4, y), (x, None, w3, y2)], 8, rb.ROSAQ_ERR_UNSUPPORTED_SHAPE),      # mixed code widths
            ([(None, 0, w4, y)], 8, rb.ROSAQ_ERR_INVALID_ARG),                              # reads from itself
            ([(x, None, w4, y), (None, 0, w4, y2)], 8, rb.ROSAQ_ERR_INVALID_ARG)):          # 128 columns feed d_in = 256
        with pytest.raises(rb.RosaqError) as e:
            ctx.plan_create(M, ops)
        assert e.value.status == status
    # races inside one launch: two operations writing one y, a y that is another operation's plain x,
    # an operation writing over its own input
    xs = torch.zeros((8, 256), dtype=torch.float16, device="cuda")
    wide = torch.zeros((8, 256), dtype=torch.float16, device="cuda")
    w_sq = ctx.quantize(torch.zeros((128, 128), dtype=torch.float16, device="cuda"), None, bits=4, k_salient=128)
    for ops in ([(x, None, w4, y), (xs, None, w4, y)],
                [(x, None, w4, wide[:, :128]), (wide[:, 64:192], None, w_sq, y2)],
                [(wide[:, :128], None, w_sq, wide[:, 64:192])]):
        with pytest.raises(rb.RosaqError) as e:
            ctx.plan_create(8, ops)
        assert e.value.status == rb.ROSAQ_ERR_INVALID_ARG
    # column ranges of one wider buffer are distinct outputs
    ctx.plan_create(8, [(x, None, w4, wide[:, :128]), (xs, None, w4, wide[:, 128:])]).free()
    x129 = torch.zeros((129, 256), dtype=torch.float16, device="cuda")
    with pytest.raises(rb.RosaqError) as e:
        ctx.plan_create(129, [(x129, None, w4, empty(129, 128))])
    assert e.value.status == rb.ROSAQ_ERR_UNSUPPORTED_SHAPE
    assert ctx.last_status() == rb.ROSAQ_OK


@pytest.mark.parametrize("pairs", [True, False])
@pytest.mark.parametrize("bits", [4, 3])
def test_7b_layer_plan_all_columns(ctx, bits, pairs):
    """The benchmark's step: the ten operations of a LLaMA-7B-shaped decoder layer at 64 tokens as one
    launch.  Weights are imported random codes (the quantizer is covered elsewhere); every output column
    is compared with the oracle's forward on the same arrays, fed the rotated activations the GPU
    produced, which are themselves compared with the oracle's x . R."""
    d, f, M = 4096, 11008, 64
    ctx.set_plan_pairs(pairs)
    g = torch.Generator(device="cuda").manual_seed(17 + bits)

    def packed(d_in, d_out):
        nq = d_in - 128
        nw = nq // 8 if bits == 4 else nq // 32 * 3
        qw = torch.randint(-2 ** 31, 2 ** 31 - 1, (nw, d_out), dtype=torch.int64, device="cuda", generator=g).to(torch.int32)
        sc = (torch.rand((nq // 128, d_out), device="cuda", generator=g) * 0.01 + 0.001).half()
        zr = torch.randint(0, 2 ** bits, (nq // 128, d_out), device="cuda", generator=g).half()
        sal = (torch.randn((128, d_out), device="cuda", generator=g) * 0.02).half()
        w = ctx.weight_import(d_in, d_out, bits, 128, 128, qw, sc, zr, sal)
        return w, H.qd_from_export(dict(qw=qw.cpu().numpy(), scales=sc.cpu().numpy(), zeros=zr.cpu().numpy(),
                                        salient=sal.cpu().numpy()), bits, 128)

    R = {k: householder_rotation(d, 5, f"layer/{k}").astype(np.float16) for k in ("attn", "mlp")}
    hw = synth.HeadwiseActivationLaw(32, 128, 3, "layer-o")
    Rb = np.stack([synth.orthogonal_qr(128, synth.rng_for(5, "layer/o", h)) for h in range(32)]).astype(np.float16)
    perm = synth.rng_for(5, "layer/o", "perm").permutation(d).astype(np.int32)
    rots = {"attn": ctx.rotation_create(dev(R["attn"])), "mlp": ctx.rotation_create(dev(R["mlp"])),
            "o": ctx.rotation_create(dev(Rb), dev(perm))}
    names = [("q", d, d, "attn"), ("k", d, d, "attn"), ("v", d, d, "attn"), ("o", d, d, "o"), ("gate", d, f, "mlp"),
             ("up", d, f, "mlp"), ("down", f, d, None)]
    ws, qds = {}, {}
    for name, di, do, _ in names:
        ws[name], qds[name] = packed(di, do)
    law = synth.ActivationLaw(d, 1.0, 5, "layer/x")
    xs = {"attn": law.sample(M, "a", np.float16), "mlp": law.sample(M, "m", np.float16), "o": hw.sample(M, "o", np.float16),
          "down": synth.ActivationLaw(f, 1.0, 5, "layer/xd").sample(M, "d", np.float16)}
    xd = {k: dev(v) for k, v in xs.items()}
    xr = {k: empty(M, d) for k in ("attn", "mlp", "o")}
    ys = {name: empty(M, do) for name, _, do, _ in names}
    ops = [(xd["attn"], None, rots["attn"], xr["attn"]), (xd["mlp"], None, rots["mlp"], xr["mlp"]),
           (xd["o"], None, rots["o"], xr["o"]), (xd["down"], None, ws["down"], ys["down"]),
           (None, 0, ws["q"], ys["q"]), (None, 0, ws["k"], ys["k"]), (None, 0, ws["v"], ys["v"]),
           (None, 2, ws["o"], ys["o"]), (None, 1, ws["gate"], ys["gate"]), (None, 1, ws["up"], ys["up"])]
    plan = ctx.plan_create(M, ops)
    plan.run()
    assert ctx.last_status() == rb.ROSAQ_OK
    first = {k: v.clone() for k, v in list(ys.items()) + [("xr_" + k, v) for k, v in xr.items()]}
    tiny = dict(qds["q"], salient=qds["q"]["salient"][:, :8], scales=qds["q"]["scales"][:, :8],
                zeros=qds["q"]["zeros"][:, :8], codes=qds["q"]["codes"][:, :8])
    for k, (Rk, pk) in {"attn": (R["attn"], None), "mlp": (R["mlp"], None), "o": (Rb, perm)}.items():
        _, xr_ref = orc.forward(xs[k], tiny, Rk, pk, return_xrot=True)
        assert H.rel_fro(xr[k].cpu().numpy(), xr_ref) <= 1e-3, k
    for name, _, _, inp in names:
        x_in = xr[inp].cpu().numpy() if inp else xs["down"]
        H.assert_y_all_columns(ys[name].cpu().numpy(), x_in, qds[name], where=f"layer plan {name}")
    for _ in range(3):
        plan.run()
    torch.cuda.synchronize()
    assert ctx.last_status() == rb.ROSAQ_OK
    for k, v in list(ys.items()) + [("xr_" + k, v) for k, v in xr.items()]:
        assert torch.equal(v.view(torch.int16), first[k].view(torch.int16)), k
    plan.free()
    ctx.set_plan_pairs(False)
