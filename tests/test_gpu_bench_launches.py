"""GPU parity of the launches the benchmark times, at their full sizes, against the CPU oracle.

The layer benchmark issues q + k + v and gate + up as one call each (rosaq_linear_multi on the rotated
activations).  Here those calls run at the LLaMA-7B / 13B sizes and every output column is compared with the
oracle's fp64 forward on the weights the GPU exported (tile by tile and element by element, see
helpers.assert_y_all_columns); the packed codes, scales, zeros and salient rows are compared bit for bit
on one column of every 128-column tile, which the oracle rotates and quantizes itself.

The Gram kernel that serves every dense calibration (two CTAs per 256 x 256 tile) is checked at the 13B
widths on a sample of channels that the oracle accumulates in fp64.
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


def householder_rotation(d, seed, key):
    vs = synth.householder_vectors(d, 6, synth.rng_for(seed, key, "R"))
    return synth.apply_householders(np.eye(d), vs)


def multi_case(ctx, d_in, widths, bits, Ms, seed, key, sigma=0.02, heavy_tail=False):
    """len(widths) linears on one rotated activation through rosaq_linear_multi, all columns checked."""
    R64 = householder_rotation(d_in, seed, key)
    R32, R16 = R64.astype(np.float32), R64.astype(np.float16)
    rot = ctx.rotation_create(dev(R16))
    ws, qds = [], []
    for i, n in enumerate(widths):
        W = synth.weights(d_in, n, seed, f"{key}/w{i}", sigma=sigma, outlier_frac=0.005 if heavy_tail else 0.01,
                          outlier_scale=10.0, heavy_tail=heavy_tail)
        w = ctx.quantize(dev(W), dev(R32), bits=bits, k_salient=128)
        e = H.export_to_numpy(w.export())
        cols = H.tile_columns(n, seed, f"{key}/w{i}")
        H.assert_export_matches(e, H.oracle_quantized(W, R32, None, bits, 128, cols=cols))   # bit-exact, every tile
        ws.append(w)
        qds.append(H.qd_from_export(e, bits, 128))
        del W, e
    law = synth.ActivationLaw(d_in, 1.0, seed, key + "/x")
    for M in Ms:
        x = law.sample(M, f"x{M}", np.float16)
        xr = ctx.rotate(dev(x), rot)
        outs = ctx.linear_multi(xr, ws, None)
        again = ctx.linear_multi(xr, ws, None)
        fused = ctx.linear_multi(dev(x), ws, rot)                # rotation inside the call
        ctx.set_linear_impl(4)                                   # ... and the whole call as one persistent launch
        try:
            one_launch = ctx.linear_multi(dev(x), ws, rot)
        finally:
            ctx.set_linear_impl(0)
        assert ctx.last_status() == rb.ROSAQ_OK
        xr_np = xr.cpu().numpy()
        _, xr_ref = orc.forward(x, dict(qds[0], salient=qds[0]["salient"][:, :8], scales=qds[0]["scales"][:, :8],
                                        zeros=qds[0]["zeros"][:, :8], codes=qds[0]["codes"][:, :8]), R16, None,
                                return_xrot=True)
        assert H.rel_fro(xr_np, xr_ref) <= 1e-3
        for i, (o, a, f) in enumerate(zip(outs, again, fused)):
            got = o.cpu().numpy()
            assert np.array_equal(got.view(np.uint16), a.cpu().numpy().view(np.uint16))     # reproducible
            H.assert_y_all_columns(got, xr_np, qds[i], where=f"{key} M={M} weight {i}")
            H.assert_y_all_columns(f.cpu().numpy(), xr_np, qds[i], where=f"{key} fused M={M} weight {i}")
            H.assert_y_all_columns(one_launch[i].cpu().numpy(), xr_np, qds[i], where=f"{key} one launch M={M} weight {i}")
    for w in ws:
        w.free()
    rot.free()


@pytest.mark.parametrize("bits", [4, 3])
def test_7b_gate_up_one_launch_all_columns(ctx, bits):
    multi_case(ctx, 4096, [11008, 11008], bits, [1, 16, 64], seed=1 if bits == 4 else 2, key=f"7b-gateup{bits}")


def test_7b_qkv_one_launch_all_columns(ctx):
    multi_case(ctx, 4096, [4096, 4096, 4096], 4, [64], seed=1, key="7b-qkv")


def test_13b_gate_up_one_launch_all_columns(ctx):
    multi_case(ctx, 5120, [13824, 13824], 4, [64], seed=4, key="13b-gateup", sigma=0.015, heavy_tail=True)


def test_7b_down_all_columns(ctx):
    """down_proj (11008 -> 4096, not rotated in the layer benchmark): single-weight call, all columns."""
    d_in, d_out, bits = 11008, 4096, 4
    W = synth.weights(d_in, d_out, 1, "7b-down-all", outlier_frac=0.01)
    w = ctx.quantize(dev(W), None, bits=bits, k_salient=128)
    e = H.export_to_numpy(w.export())
    cols = H.tile_columns(d_out, 1, "7b-down-all")
    H.assert_export_matches(e, H.oracle_quantized(W, None, None, bits, 128, cols=cols))
    qd = H.qd_from_export(e, bits, 128)
    x = synth.ActivationLaw(d_in, 1.0, 1, "7b-down-all/x").sample(64, "x", np.float16)
    y = ctx.linear(dev(x), w, None).cpu().numpy()
    assert ctx.last_status() == rb.ROSAQ_OK
    H.assert_y_all_columns(y, x, qd, where="7b down")
    w.free()


def test_7b_down_scaled_as_the_paper_runs_it(ctx):
    """down_proj the way the weight-splitting appendix runs it: not rotated, quantized as D W with an
    AWQ-style per-input-channel D, fed x D^-1.  Codes bit-exact on one column per tile, y on all columns."""
    from paper_2506_13472_b200 import pca
    d_in, d_out, bits = 11008, 4096, 4
    W = synth.weights(d_in, d_out, 1, "7b-down-scaled", outlier_frac=0.01)
    law = synth.ActivationLaw(d_in, 1.0, 1, "7b-down-scaled/x")
    dsc = pca.channel_scale(law.sample(512, "calib", np.float32))
    w = ctx.quantize(dev(W), None, bits=bits, k_salient=128, in_scale=dev(dsc))
    e = H.export_to_numpy(w.export())
    cols = H.tile_columns(d_out, 1, "7b-down-scaled")
    qd = orc.quantize(np.ascontiguousarray(orc.scale_rows_f32(W, dsc)[:, cols]), bits, 128, 128)
    qd["qw"], qd["cols"] = orc.pack(qd["codes"], bits), cols
    H.assert_export_matches(e, qd)
    x = law.sample(64, "x", np.float16)
    xs = (x.astype(np.float32) / dsc[None, :]).astype(np.float16)
    y = ctx.linear(dev(xs), w, None).cpu().numpy()
    assert ctx.last_status() == rb.ROSAQ_OK
    H.assert_y_all_columns(y, xs, H.qd_from_export(e, bits, 128), where="7b down, scaled")
    w.free()


# --------------------------------------------------------------------------- Gram kernel at the 13B widths
def sampled_channels(d, seed):
    """96 channels: 32 from the first 256-channel block, 32 from a middle one, 32 from the last."""
    rng = synth.rng_for(seed, "cov-sample", d)
    nb = (d + 255) // 256
    out = []
    for b in (0, nb // 2, nb - 1):
        lo, hi = b * 256, min((b + 1) * 256, d)
        out += sorted(rng.choice(np.arange(lo, hi), size=32, replace=False).tolist())
    return np.asarray(out, dtype=np.int64)


@pytest.mark.parametrize("d,chunks", [(5120, 1), (13824, 1), (5120, 16)])
def test_calib_cov_pair_kernel_13b_widths_on_sampled_channels(ctx, d, chunks):
    """16384-token chunks of the 13B-shaped calibration stream (one chunk, and the 16-chunk accumulation of
    the 262144-token stream) against the oracle's fp64 Gram matrix of the sampled channels."""
    n_tok = 16384
    law = synth.ActivationLaw(d, 1.0, 4, f"cov13b{d}")
    ch = sampled_channels(d, 4)
    Cg = torch.zeros((d, d), dtype=torch.float32, device="cuda")
    Cref = np.zeros((ch.size, ch.size))
    for c in range(chunks):
        X = law.sample(n_tok, f"chunk{c}", np.float16)
        ctx.calib_cov(dev(X), Cg)
        Cref += orc.cov(np.ascontiguousarray(X[:, ch]))
        del X
    assert ctx.last_status() == rb.ROSAQ_OK
    got = Cg[torch.from_numpy(ch).cuda()][:, torch.from_numpy(ch).cuda()].cpu().numpy().astype(np.float64)
    # per call the bound of helpers.cov_tolerance; the chunk results are added in fp32 round-to-nearest
    # (half an ulp of the running sum per chunk)
    dg = np.sqrt(np.diagonal(Cref))
    tol = chunks * H.cov_tolerance(Cref / chunks, n_tok) + chunks * 2.0 ** -24 * dg[:, None] * dg[None, :]
    ratio = float((np.abs(got - Cref) / tol).max())
    print(f"calib_cov d={d} chunks={chunks}: worst error = {ratio:.3f} of the bound")
    assert ratio <= 1.0
    sym = Cg[:512, :512]
    assert torch.equal(sym, sym.T)
