"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle.

Integer / byte results (packed codes, scales, zeros, salient fp16 bits) must be bit-exact.
y must satisfy ||y - y_ref||_F / ||y_ref||_F <= 2e-3 against the oracle's fp64 forward on the
same dequantised weights.
"""
import numpy as np
import pytest
import torch

from oracle import rosaq_oracle as orc
from paper_2506_13472_b200 import binding as rb
from paper_2506_13472_b200 import pca, synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = rb.Context(0)
    yield c
    c.close()


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def check_status(ctx):
    assert ctx.last_status() == rb.ROSAQ_OK


# --------------------------------------------------------------------------- quantize
@pytest.mark.parametrize("bits", [4, 3])
def test_quantize_tiny_config_bit_exact(ctx, bits):
    c = H.config_tiny()
    w = ctx.quantize(dev(c["W"]), dev(c["R32"]), bits=bits, k_salient=128)
    H.assert_export_matches(H.export_to_numpy(w.export()), H.oracle_quantized(c["W"], c["R32"], None, bits, 128))
    check_status(ctx)


@pytest.mark.parametrize("bits,k_salient,d_out", [(4, 0, 200), (3, 0, 129), (4, 256, 8), (3, 256, 128), (4, 128, 1)])
def test_quantize_no_rotation_ragged_and_degenerate(ctx, bits, k_salient, d_out):
    W = synth.weights(256, d_out, seed=21, key=f"nr{d_out}", outlier_rows=3, outlier_scale=20.0)
    W[130:140, 0] = 0.25          # constant stretch; column 0 of group 1 below gets fully constant
    W[128:256, d_out - 1] = 0.125 # a constant group: range floor, zero-point clamp
    w = ctx.quantize(dev(W), None, bits=bits, k_salient=k_salient)
    assert (w.d_in, w.d_out, w.bits, w.k_salient) == (256, d_out, bits, k_salient)
    H.assert_export_matches(H.export_to_numpy(w.export()), H.oracle_quantized(W, None, None, bits, k_salient))


@pytest.mark.parametrize("bits", [4, 3])
def test_quantize_headwise_blockdiag_with_permutation(ctx, bits):
    c = H.config_headwise()
    w = ctx.quantize(dev(c["W"]), dev(c["Rb32"]), dev(c["perm"]), bits=bits, k_salient=128)
    H.assert_export_matches(H.export_to_numpy(w.export()),
                            H.oracle_quantized(c["W"], c["Rb32"], c["perm"], bits, 128))
    # Eq. 6 == Eq. 7: the same weight through the dense path fed blockdiag . P
    Rd = orc.dense_from_blocks(c["Rb32"], c["perm"])
    w2 = ctx.quantize(dev(c["W"]), dev(Rd), bits=bits, k_salient=128)
    a, b = H.export_to_numpy(w.export()), H.export_to_numpy(w2.export())
    for k in a:
        assert np.array_equal(a[k], b[k]), k


@pytest.mark.parametrize("bits", [4, 3])
def test_import_export_round_trip(ctx, bits):
    rng = np.random.default_rng(5)
    d_in, d_out, K = 512, 300, 128
    nq = d_in - K
    codes = rng.integers(0, 2 ** bits, (nq, d_out)).astype(np.uint8)
    qw = orc.pack(codes, bits)
    sc = rng.uniform(1e-3, 1e-1, (nq // 128, d_out)).astype(np.float16)
    zr = rng.integers(0, 2 ** bits, (nq // 128, d_out)).astype(np.float16)
    sal = rng.standard_normal((K, d_out)).astype(np.float16)
    w = ctx.weight_import(d_in, d_out, bits, 128, K, dev(qw.view(np.int32)), dev(sc), dev(zr), dev(sal))
    e = H.export_to_numpy(w.export())
    assert np.array_equal(e["qw"].view(np.uint32), qw)
    assert np.array_equal(e["scales"], sc) and np.array_equal(e["zeros"], zr) and np.array_equal(e["salient"], sal)


@pytest.mark.parametrize("bits", [4, 3])
@pytest.mark.parametrize("rotated", [False, True])
def test_quantize_scaled_bit_exact_and_forward(ctx, bits, rotated):
    """rosaq_quantize_scaled: codes of D W (and of R^T D W) bit for bit against the oracle; the linear fed
    x D^-1 reproduces the oracle's forward on the same weights and stays close to the unscaled product x W."""
    c = H.config_tiny()
    d_in, d_out, M = 512, 200, 9
    W = synth.weights(d_in, d_out, seed=81, key="scaled", outlier_rows=4, outlier_scale=20.0)
    law = synth.ActivationLaw(d_in, 1.2, 0, "tiny", mix="qr")
    dsc = pca.channel_scale(law.sample(256, "scale-calib", np.float32))
    assert dsc.min() < 1.0 < dsc.max()
    R32, R16 = (c["R32"], c["R16"]) if rotated else (None, None)
    w = ctx.quantize(dev(W), None if R32 is None else dev(R32), bits=bits, k_salient=128, in_scale=dev(dsc))
    DW = orc.scale_rows_f32(W, dsc)
    Wp = orc.rotate_weights_f32(R32, DW) if rotated else DW
    qd = orc.quantize(Wp, bits, 128, 128)
    qd["qw"], qd["cols"] = orc.pack(qd["codes"], bits), np.arange(d_out, dtype=np.int32)
    H.assert_export_matches(H.export_to_numpy(w.export()), qd)
    x = law.sample(M, "scaled-x", np.float16)
    xs = (x.astype(np.float32) / dsc[None, :]).astype(np.float16)               # x D^-1, what the caller feeds
    rot = ctx.rotation_create(dev(R16)) if rotated else None
    y = ctx.linear(dev(xs), w, rot).cpu().numpy()
    check_status(ctx)
    assert H.rel_fro(y, orc.forward(xs, qd, R16)) <= H.REL_TOL_Y
    ref = x.astype(np.float64) @ W.astype(np.float64)
    assert H.rel_fro(y, ref) <= (0.2 if bits == 4 else 0.5)                      # the quantization error itself
    with pytest.raises(rb.RosaqError) as e:                                       # misaligned scale pointer: a code
        ctx.quantize(dev(W), None, bits=bits, k_salient=128, in_scale=dev(np.concatenate([dsc, dsc]))[1:d_in + 1])
    assert e.value.status == rb.ROSAQ_ERR_ALIGNMENT


# --------------------------------------------------------------------------- linear
def run_linear_case(ctx, x16, W16, Rb32, Rb16, perm, bits, k_salient, impl):
    """quantize on the GPU, check codes, then y against the oracle forward on the same inputs."""
    ctx.set_linear_impl(impl)
    try:
        w = ctx.quantize(dev(W16), None if Rb32 is None else dev(Rb32), None if perm is None else dev(perm),
                         bits=bits, k_salient=k_salient)
        qd = H.oracle_quantized(W16, Rb32, perm, bits, k_salient)
        H.assert_export_matches(H.export_to_numpy(w.export()), qd)
        rot = None if Rb16 is None else ctx.rotation_create(dev(Rb16), None if perm is None else dev(perm))
        y = ctx.linear(dev(x16), w, rot).cpu().numpy()
        y_ref, xr_ref = orc.forward(x16, qd, Rb16, perm, return_xrot=True)
        assert np.all(np.isfinite(y))
        assert H.rel_fro(y, y_ref) <= H.REL_TOL_Y
        if rot is not None:
            xr = ctx.rotate(dev(x16), rot).cpu().numpy()
            assert H.rel_fro(xr, xr_ref) <= 1e-3
            # pre-rotated input through the GEMM stage alone gives the same y bits
            y2 = ctx.linear(dev(xr), w, None).cpu().numpy()
            assert np.array_equal(y2.view(np.uint16), y.view(np.uint16))
            again = ctx.linear(dev(x16), w, rot).cpu().numpy()          # and so does a second run
            assert np.array_equal(again.view(np.uint16), y.view(np.uint16))
        check_status(ctx)
    finally:
        ctx.set_linear_impl(0)


@pytest.mark.parametrize("impl", [1, 0, 4, 5])
@pytest.mark.parametrize("bits", [4, 3])
def test_linear_tiny_config(ctx, bits, impl):
    c = H.config_tiny()
    run_linear_case(ctx, c["x"], c["W"], c["R32"], c["R16"], None, bits, 128, impl)


@pytest.mark.parametrize("impl", [1, 0, 4, 5])
@pytest.mark.parametrize("bits", [4, 3])
def test_linear_headwise(ctx, bits, impl):
    c = H.config_headwise()
    run_linear_case(ctx, c["x"], c["W"], c["Rb32"], c["Rb16"], c["perm"], bits, 128, impl)


@pytest.mark.parametrize("impl", [1, 0, 4, 5, 6])
@pytest.mark.parametrize("M,d_in,d_out,bits,k_salient", [
    (1, 256, 8, 4, 128), (3, 256, 136, 3, 0), (17, 384, 128, 4, 384), (64, 1024, 640, 4, 128),
    (130, 512, 256, 3, 128), (257, 256, 200, 4, 0)])
def test_linear_shapes_no_rotation(ctx, M, d_in, d_out, bits, k_salient, impl):
    W = synth.weights(d_in, d_out, seed=31, key=f"s{d_in}x{d_out}", outlier_frac=0.01)
    x = synth.rng_for(31, "x", M, d_in).standard_normal((M, d_in)).astype(np.float16)
    run_linear_case(ctx, x, W, None, None, None, bits, k_salient, impl)


@pytest.mark.parametrize("bits", [4, 3])
@pytest.mark.parametrize("M,d_in,d_out,k_salient", [(600, 1024, 1152, 128), (256, 2048, 256, 256), (129, 512, 384, 0)])
def test_linear_prefill_tiles(ctx, M, d_in, d_out, k_salient, bits):
    """256-column x 256-token tiles on pairs of CTAs (implementation 5 takes them at every size): several
    token blocks with a ragged last one, an odd number of 128-column tiles (the second CTA of the last pair
    has no tile of its own), two salient fp16 groups, none.  Every column against the oracle; the same bits on a
    second run; agreement with the per-call kernel to fp32 summation order."""
    W = synth.weights(d_in, d_out, seed=57, key=f"pf{d_in}x{d_out}", outlier_frac=0.01)
    x = synth.rng_for(57, "x", M, d_in).standard_normal((M, d_in)).astype(np.float16)
    w = ctx.quantize(dev(W), None, bits=bits, k_salient=k_salient)
    qd = H.oracle_quantized(W, None, None, bits, k_salient)
    y0 = ctx.linear(dev(x), w, None).cpu().numpy()
    ctx.set_linear_impl(5)
    try:
        out = torch.full((M + 1, d_out + 8), 7.0, dtype=torch.float16, device="cuda")     # a wider, longer buffer
        y = ctx.linear(dev(x), w, None, out=out[:M, :d_out]).cpu().numpy()
        check_status(ctx)
        again = ctx.linear(dev(x), w, None).cpu().numpy()
    finally:
        ctx.set_linear_impl(0)
    assert np.all(out[M:].cpu().numpy() == 7.0) and np.all(out[:, d_out:].cpu().numpy() == 7.0)   # nothing written outside
    assert H.rel_fro(y, orc.forward(x, qd, None)) <= H.REL_TOL_Y
    assert np.array_equal(again.view(np.uint16), y.view(np.uint16))
    assert H.rel_fro(y, y0.astype(np.float64)) <= 2e-4
    w.free()


@pytest.mark.parametrize("bits", [4, 3])
@pytest.mark.parametrize("M", [65, 128, 200, 600])
def test_linear_token_blocks_of_128(ctx, M, bits):
    """More than 64 tokens as blocks of 128 in one persistent launch (implementation 6): accumulators of 128
    tokens, a ragged last block, the dense rotation and the head-wise one with its column permutation (whose
    tiles are computed four times over, each copy writing a quarter of the token rows) -- all against the
    oracle, and the same bits on a second run."""
    c = H.config_headwise()
    d_in = c["W"].shape[0]
    x = synth.rng_for(61, "xb", M, d_in).standard_normal((M, d_in)).astype(np.float16)
    qd = H.oracle_quantized(c["W"], c["Rb32"], c["perm"], bits, 128)
    w = ctx.quantize(dev(c["W"]), dev(c["Rb32"]), dev(c["perm"]), bits=bits, k_salient=128)
    rot = ctx.rotation_create(dev(c["Rb16"]), dev(c["perm"]))
    y_ref, xr_ref = orc.forward(x, qd, c["Rb16"], c["perm"], return_xrot=True)
    ctx.set_linear_impl(6)
    try:
        xr = ctx.rotate(dev(x), rot)
        y = ctx.linear(dev(x), w, rot).cpu().numpy()
        again = ctx.linear(dev(x), w, rot).cpu().numpy()
        check_status(ctx)
    finally:
        ctx.set_linear_impl(0)
    assert H.rel_fro(xr.cpu().numpy(), xr_ref) <= 1e-3
    assert H.rel_fro(y, y_ref) <= H.REL_TOL_Y
    assert np.array_equal(again.view(np.uint16), y.view(np.uint16))
    t = H.config_tiny()                                                       # a dense rotation too
    xt = synth.rng_for(61, "xt", M, t["W"].shape[0]).standard_normal((M, t["W"].shape[0])).astype(np.float16)
    run_linear_case(ctx, xt, t["W"], t["R32"], t["R16"], None, bits, 128, 6)
    w.free()
    rot.free()


def test_linear_prefill_tiles_replayed_from_a_graph_follow_their_input(ctx):
    """A captured launch of the prefill tiles is replayed on other activations: the partial tiles that pairs of
    CTAs exchange, and the flags that announce them, must be those of the replay, not of an earlier one."""
    M, d_in, d_out = 520, 1024, 1152
    W = synth.weights(d_in, d_out, seed=58, key="pfg", outlier_frac=0.01)
    w = ctx.quantize(dev(W), None, bits=4, k_salient=128)
    rng = synth.rng_for(58, "xg", M, d_in)
    xa, xb = (rng.standard_normal((M, d_in)).astype(np.float16) for _ in range(2))
    x, y = dev(xa), torch.empty((M, d_out), dtype=torch.float16, device="cuda")
    ctx.set_linear_impl(5)
    try:
        want_a, want_b = (ctx.linear(dev(v), w, None).cpu().numpy() for v in (xa, xb))
        ctx.linear(x, w, None, out=y)                       # warm-up outside the capture
        torch.cuda.synchronize()
        s = torch.cuda.Stream()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(s):
            with torch.cuda.graph(g, stream=s):
                ctx.linear(x, w, None, out=y)
        for v, want in ((xa, want_a), (xb, want_b), (xa, want_a)):
            x.copy_(dev(v))
            torch.cuda.synchronize()
            g.replay()
            torch.cuda.synchronize()
            assert np.array_equal(y.cpu().numpy().view(np.uint16), want.view(np.uint16))
        check_status(ctx)
    finally:
        ctx.set_linear_impl(0)
    assert not np.array_equal(want_a, want_b)
    w.free()


def test_linear_strided_activations_and_output(ctx):
    c = H.config_tiny()
    w = ctx.quantize(dev(c["W"]), dev(c["R32"]), bits=4, k_salient=128)
    qd = H.oracle_quantized(c["W"], c["R32"], None, 4, 128)
    xbuf = torch.zeros((4, 512 + 64), dtype=torch.float16, device="cuda")
    xbuf[:, :512] = dev(c["x"])
    ybuf = torch.full((4, 512 + 8), 7.0, dtype=torch.float16, device="cuda")
    rot = ctx.rotation_create(dev(c["R16"]))
    ctx.linear(xbuf[:, :512], w, rot, out=ybuf[:, :512])
    assert H.rel_fro(ybuf[:, :512].cpu().numpy(), orc.forward(c["x"], qd, c["R16"])) <= H.REL_TOL_Y
    assert torch.all(ybuf[:, 512:] == 7.0)       # nothing written past d_out


@pytest.mark.parametrize("bits,M", [(4, 64), (3, 5), (4, 200)])
def test_linear_multi_gives_the_bits_of_separate_calls(ctx, bits, M):
    """q/k/v-style: three weights of different widths on one activation, one launch, with and without R."""
    c = H.config_tiny()
    widths = [512, 200, 136]
    Ws = [synth.weights(512, n, seed=51, key=f"multi{n}", outlier_frac=0.01) for n in widths]
    ws = [ctx.quantize(dev(W), dev(c["R32"]), bits=bits, k_salient=128) for W in Ws]
    rot = ctx.rotation_create(dev(c["R16"]))
    x = dev(synth.ActivationLaw(512, 1.2, 0, "tiny", mix="qr").sample(M, "xm", np.float16))
    want = [ctx.linear(x, w, rot).cpu().numpy() for w in ws]
    got = ctx.linear_multi(x, ws, rot)
    xr = ctx.rotate(x, rot)
    got2 = ctx.linear_multi(xr, ws, None)
    check_status(ctx)
    for a, b, b2 in zip(want, got, got2):
        assert np.array_equal(a.view(np.uint16), b.cpu().numpy().view(np.uint16))
        assert np.array_equal(a.view(np.uint16), b2.cpu().numpy().view(np.uint16))
    with pytest.raises(rb.RosaqError) as e:                  # mismatched geometry is an error code
        other = ctx.quantize(dev(Ws[0]), dev(c["R32"]), bits=bits, k_salient=256)
        ctx.linear_multi(x, [ws[0], other], rot)
    assert e.value.status == rb.ROSAQ_ERR_INVALID_ARG


@pytest.mark.parametrize("bits", [4, 3])
@pytest.mark.parametrize("M,d_in,d_out,k_salient", [(64, 1024, 512, 128), (128, 512, 256, 128), (32, 2048, 256, 0),
                                                      (200, 512, 512, 256)])
def test_linear_cta_pairs_give_the_bits_of_single_ctas(ctx, M, d_in, d_out, k_salient, bits):
    """Implementation 2 (two CTAs per MMA stream, cta_group::2) on shapes it accepts: within the oracle
    tolerance, and equal to the default implementation up to the fp32 summation order of the K splits."""
    W = synth.weights(d_in, d_out, seed=61, key=f"pair{d_in}x{d_out}", outlier_frac=0.01)
    x = synth.rng_for(61, "x", M, d_in).standard_normal((M, d_in)).astype(np.float16)
    R = H.config_tiny()["R16"] if d_in == 512 else None
    w = ctx.quantize(dev(W), None, bits=bits, k_salient=k_salient)
    rot = None if R is None else ctx.rotation_create(dev(R))
    qd = H.oracle_quantized(W, None, None, bits, k_salient)
    want = ctx.linear(dev(x), w, rot).cpu().numpy()
    ctx.set_linear_impl(2)
    try:
        got = ctx.linear(dev(x), w, rot).cpu().numpy()
        check_status(ctx)
    finally:
        ctx.set_linear_impl(0)
    assert np.all(np.isfinite(got))
    assert H.rel_fro(got, want) <= 2e-4
    assert H.rel_fro(got, orc.forward(x, qd, R)) <= H.REL_TOL_Y



# --------------------------------------------------------------------------- equal-share (stream-K) launches
@pytest.mark.parametrize("bits", [4, 3])
def test_linear_stream_k_path(ctx, bits):
    """At up to 64 tokens an operand with at least as many column tiles as SMs is cut into equal shares of
    the (tile, group) list, one per CTA, and tiles shared by several CTAs are finished through a workspace
    (implementation 0); implementation 3 always splits K across clusters.  Both must match the oracle on
    sampled columns; they agree up to the fp32 summation order; repeated launches give the same bits."""
    d_in, d_out = 1024, 150 * 128
    W = synth.weights(d_in, d_out, seed=71, key=f"sk{bits}", outlier_frac=0.01)
    cols = synth.sample_columns(d_out, 24, 71, f"sk{bits}")
    w = ctx.quantize(dev(W), None, bits=bits, k_salient=128)
    qd = H.oracle_quantized(W, None, None, bits, 128, cols=cols)
    H.assert_export_matches(H.export_to_numpy(w.export()), qd)
    for M in (1, 16, 64):
        x = synth.rng_for(71, "x", M, d_in).standard_normal((M, d_in)).astype(np.float16)
        got = ctx.linear(dev(x), w, None).cpu().numpy()
        again = ctx.linear(dev(x), w, None).cpu().numpy()
        ctx.set_linear_impl(3)
        try:
            want = ctx.linear(dev(x), w, None).cpu().numpy()
        finally:
            ctx.set_linear_impl(0)
        check_status(ctx)
        assert np.all(np.isfinite(got))
        assert np.array_equal(got.view(np.uint16), again.view(np.uint16))
        assert H.rel_fro(got, want) <= 2e-4
        assert H.rel_fro(got[:, cols], orc.forward(x, qd, None)) <= H.REL_TOL_Y
    w.free()


def test_linear_multi_stream_k_path(ctx):
    """Two weights whose column tiles together fill the equal-share launch (gate/up style), against the
    separate calls (which split K across clusters) and the oracle."""
    d_in, d_out, M = 1024, 75 * 128, 64
    Ws = [synth.weights(d_in, d_out, seed=72, key=f"skm{i}", outlier_frac=0.01) for i in range(2)]
    ws = [ctx.quantize(dev(W), None, bits=4, k_salient=128) for W in Ws]
    x = synth.rng_for(72, "x", M, d_in).standard_normal((M, d_in)).astype(np.float16)
    want = [ctx.linear(dev(x), w, None).cpu().numpy() for w in ws]
    got = [g.cpu().numpy() for g in ctx.linear_multi(dev(x), ws, None)]
    check_status(ctx)
    for i in range(2):
        cols = synth.sample_columns(d_out, 16, 72, f"skm{i}")
        qd = H.oracle_quantized(Ws[i], None, None, 4, 128, cols=cols)
        assert H.rel_fro(got[i], want[i]) <= 2e-4
        assert H.rel_fro(got[i][:, cols], orc.forward(x, qd, None)) <= H.REL_TOL_Y
    for w in ws:
        w.free()


def test_special_case_all_salient_is_plain_fp16_gemm(ctx):
    rng = np.random.default_rng(12)
    W = (rng.standard_normal((256, 128)) * 0.02).astype(np.float16)
    x = rng.standard_normal((9, 256)).astype(np.float16)
    w = ctx.quantize(dev(W), None, bits=4, k_salient=256)
    y = ctx.linear(dev(x), w).cpu().numpy()
    ref = x.astype(np.float64) @ W.astype(np.float64)
    assert H.rel_fro(y, ref) <= 1e-3


# --------------------------------------------------------------------------- calib_cov
cov_tolerance = H.cov_tolerance


@pytest.mark.parametrize("dtype,n_tokens,d,n_blocks", [
    (np.float32, 256, 512, 1), (np.float16, 300, 264, 1), (np.float16, 1000, 512, 4), (np.float16, 64, 8, 1),
    (np.float16, 2048, 640, 1), (np.float16, 777, 384, 3), (np.float16, 130, 72, 1)])
def test_calib_cov_matches_oracle_and_accumulates(ctx, dtype, n_tokens, d, n_blocks):
    law = synth.ActivationLaw(d, 1.0, seed=41, key=f"cov{d}", mix="householder")
    X = law.sample(n_tokens, "X", dtype)
    dh = d // n_blocks
    Cg = torch.zeros((n_blocks, dh, dh), dtype=torch.float32, device="cuda")
    half = n_tokens // 2 // 8 * 8
    Xd = dev(X)
    ctx.calib_cov(Xd[:half], Cg, n_blocks)        # two chunks: C accumulates
    ctx.calib_cov(Xd[half:], Cg, n_blocks)
    check_status(ctx)
    Cref = orc.cov(X, n_blocks).reshape(n_blocks, dh, dh)
    got = Cg.cpu().numpy().astype(np.float64)
    assert np.all(np.abs(got - Cref) <= cov_tolerance(Cref, n_tokens) + 1e-30)
    assert np.array_equal(got, np.swapaxes(got, -1, -2))          # both triangles written, symmetric


def test_pca_helper_gives_valid_eigenpairs_from_gpu_cov(ctx):
    c = H.config_tiny()
    Cg = torch.zeros((512, 512), dtype=torch.float32, device="cuda")
    ctx.calib_cov(dev(c["X"]), Cg)
    lam, R = pca.eigh_descending(Cg.cpu().numpy())
    C64 = orc.cov(c["X"])
    nC = np.linalg.norm(C64)
    assert np.all(np.diff(lam) <= 1e-9 * nC)
    assert np.abs(R.T @ R - np.eye(512)).max() <= 1e-10
    assert np.abs(C64 @ R - R * lam[None, :]).max() <= 1e-5 * nC
    assert np.allclose(lam[:64], c["lam"][:64], rtol=1e-4)


# --------------------------------------------------------------------------- argument errors
def test_argument_errors_are_codes_not_faults(ctx):
    W = torch.zeros((256, 128), dtype=torch.float16, device="cuda")
    with pytest.raises(rb.RosaqError) as e:
        ctx.quantize(W, None, bits=5)
    assert e.value.status == rb.ROSAQ_ERR_INVALID_ARG
    with pytest.raises(rb.RosaqError) as e:
        ctx.quantize(W, None, bits=4, k_salient=64)
    assert e.value.status == rb.ROSAQ_ERR_UNSUPPORTED_SHAPE
    with pytest.raises(rb.RosaqError) as e:
        ctx.quantize(torch.zeros((200, 128), dtype=torch.float16, device="cuda"), None)
    assert e.value.status == rb.ROSAQ_ERR_UNSUPPORTED_SHAPE
    w = ctx.quantize(W, None, bits=4, k_salient=128)
    x = torch.zeros((4, 264), dtype=torch.float16, device="cuda")
    with pytest.raises(rb.RosaqError) as e:
        ctx.linear(x[:, 1:257], w)                          # misaligned pointer
    assert e.value.status == rb.ROSAQ_ERR_ALIGNMENT
    with pytest.raises(rb.RosaqError) as e:
        ctx.linear(torch.zeros((4, 128), dtype=torch.float16, device="cuda"), w)   # ldx < d_in
    assert e.value.status == rb.ROSAQ_ERR_INVALID_ARG
    assert ctx.last_status() == rb.ROSAQ_OK


def test_a_perm_that_is_not_a_permutation_is_a_status_code(ctx):
    """A duplicated or out-of-range entry in rot->perm would make the kernels index and store through
    garbage: both calls that take a perm check it on the device first and return a code, launching nothing
    that uses it."""
    c = H.config_headwise()
    d = c["heads"] * c["head_dim"]
    for bad in (np.where(np.arange(d) == 5, c["perm"][6], c["perm"]).astype(np.int32),       # a value twice
                np.where(np.arange(d) == 9, d, c["perm"]).astype(np.int32),                  # out of range
                np.where(np.arange(d) == 0, -1, c["perm"]).astype(np.int32)):
        with pytest.raises(rb.RosaqError) as e:
            ctx.rotation_create(dev(c["Rb16"]), dev(bad))
        assert e.value.status == rb.ROSAQ_ERR_INVALID_ARG
        with pytest.raises(rb.RosaqError) as e:
            ctx.quantize(dev(c["W"]), dev(c["Rb32"]), dev(bad), bits=4, k_salient=128)
        assert e.value.status == rb.ROSAQ_ERR_INVALID_ARG
    assert ctx.last_status() == rb.ROSAQ_OK
    rot = ctx.rotation_create(dev(c["Rb16"]), dev(c["perm"]))                                  # the real one still works
    rot.free()


# --------------------------------------------------------------------------- bounded waits
@pytest.mark.parametrize("impl,d_in,d_out", [(3, 1024, 512), (0, 1024, 150 * 128), (4, 1024, 512), (4, 512, 512),
                                               (5, 1024, 512), (6, 1024, 512)])
def test_expired_waits_in_the_linear_kernels_leave_the_context_usable(ctx, impl, d_in, d_out):
    """With the wait limit cut to one poll the linear kernels (cluster split-K, equal shares with the
    workspace exchange, the persistent launch with and without a rotation) may give up anywhere: they must
    return ROSAQ_OK or ROSAQ_ERR_TIMEOUT, never hang or fault, and afterwards -- status read, limit
    restored -- the same call reproduces the earlier result bit for bit (no counter left behind)."""
    W = synth.weights(d_in, d_out, seed=91, key=f"tw{d_in}x{d_out}", outlier_frac=0.01)
    w = ctx.quantize(dev(W), None, bits=4, k_salient=128)
    rot = ctx.rotation_create(dev(H.config_tiny()["R16"])) if d_in == 512 else None
    M = 96 if impl == 6 else 64                                # (implementation 6 is about more than 64 tokens)
    x = dev(synth.rng_for(91, "x", d_in).standard_normal((M, d_in)).astype(np.float16))
    ctx.set_linear_impl(impl)
    try:
        want = ctx.linear(x, w, rot).cpu().numpy()
        assert ctx.last_status() == rb.ROSAQ_OK
        old = ctx.set_wait_limit(1)
        try:
            for _ in range(3):
                ctx.linear(x, w, rot)
                assert ctx.last_status() in (rb.ROSAQ_OK, rb.ROSAQ_ERR_TIMEOUT)
        finally:
            ctx.set_wait_limit(old)
        for _ in range(2):
            got = ctx.linear(x, w, rot).cpu().numpy()
            assert ctx.last_status() == rb.ROSAQ_OK
            assert np.array_equal(got.view(np.uint16), want.view(np.uint16))
    finally:
        ctx.set_linear_impl(0)
    w.free()



def test_expired_wait_is_reported_and_the_context_stays_usable(ctx):
    """Failure detection without a GPU fault: with the wait limit cut to one poll, a wait that cannot be
    satisfied in time (the Gram kernel's epilogue waiting for ~100 us of accumulation) gives up: the
    kernel lets its copies and MMAs in flight finish, frees its tensor memory and returns, the status
    word reports ROSAQ_ERR_TIMEOUT, and the same context then computes correct results again."""
    c = H.config_tiny()
    w = ctx.quantize(dev(c["W"]), dev(c["R32"]), bits=4, k_salient=128)
    rot = ctx.rotation_create(dev(c["R16"]))
    x = dev(c["x"])
    want = ctx.linear(x, w, rot).cpu().numpy()
    X = torch.randn((32768, 512), device="cuda").to(torch.float16)
    Cg = torch.zeros((512, 512), dtype=torch.float32, device="cuda")
    old = ctx.set_wait_limit(1)
    try:
        ctx.calib_cov(X, Cg)                                  # ~100 us of accumulation per tile
        assert ctx.last_status() == rb.ROSAQ_ERR_TIMEOUT
        assert ctx.last_status() == rb.ROSAQ_OK               # reading the status clears it
    finally:
        ctx.set_wait_limit(old)
    got = ctx.linear(x, w, rot).cpu().numpy()
    assert ctx.last_status() == rb.ROSAQ_OK
    assert np.array_equal(got.view(np.uint16), want.view(np.uint16))
    Cg.zero_()
    ctx.calib_cov(X[:1024], Cg)
    assert ctx.last_status() == rb.ROSAQ_OK
    Cref = X[:1024].double().T @ X[:1024].double()
    assert torch.allclose(Cg.double(), Cref, rtol=1e-3, atol=1e-2)
