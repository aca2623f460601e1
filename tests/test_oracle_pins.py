"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these needs a GPU.  Each test is chosen so that a plausible mistake in the
oracle (dropped term, wrong sign, wrong index, transposed operand, wrong sort
direction, wrong rounding) fails at least one of them.
"""
import itertools
from fractions import Fraction

import numpy as np
import pytest

from oracle import rosaq_oracle as orc
from paper_2506_13472_b200 import synth


# ----------------------------------------------------------------- binary16
def test_f16_to_f64_all_bit_patterns_match_numpy():
    bits = np.arange(65536, dtype=np.uint16)
    ours = orc.f16_to_f64(bits)
    ref = bits.view(np.float16).astype(np.float64)
    both_nan = np.isnan(ours) & np.isnan(ref)
    assert np.array_equal(ours[~both_nan], ref[~both_nan])
    assert np.array_equal(np.signbit(ours[~both_nan]), np.signbit(ref[~both_nan]))


def test_f32_to_f16_matches_numpy_rne_including_ties_and_edges():
    rng = np.random.default_rng(0)
    vals = [rng.standard_normal(200000).astype(np.float32) * s for s in (1e-8, 1e-6, 1e-4, 1.0, 300.0, 7e4)]
    # exact ties between neighbouring halves (normal and subnormal), and the overflow edge
    h = np.arange(0, 0x7bff, dtype=np.uint16).view(np.float16).astype(np.float64)
    ties = ((h[:-1] + h[1:]) / 2).astype(np.float32)
    edge = np.array([65504.0, 65519.996, 65520.0, 65536.0, 2.0 ** -24, 2.0 ** -25, 2.0 ** -25 * 1.0000001,
                     2.0 ** -14, 0.0, -0.0, np.inf, -np.inf], dtype=np.float32)
    f = np.concatenate(vals + [ties, -ties, edge])
    with np.errstate(over="ignore"):
        ref = f.astype(np.float16).view(np.uint16)
    assert np.array_equal(orc.f32_to_f16_bits(f), ref)


# ----------------------------------------------------------------- Eq. 4: covariance
def test_cov_brute_force_and_closed_forms():
    rng = np.random.default_rng(1)
    X = rng.standard_normal((7, 5))
    Cm = orc.cov(X)
    for i, j in itertools.product(range(5), range(5)):
        assert Cm[i, j] == pytest.approx(sum(X[t, i] * X[t, j] for t in range(7)), rel=1e-14, abs=1e-15)
    # a transposed operand (X X^T) would have the wrong shape; asymmetric closed form:
    X = np.zeros((3, 4))
    X[0, 1] = 2.0
    X[1, 1] = 3.0
    X[1, 2] = 5.0
    Cm = orc.cov(X)
    want = np.zeros((4, 4))
    want[1, 1], want[1, 2], want[2, 1], want[2, 2] = 13.0, 15.0, 15.0, 25.0
    assert np.array_equal(Cm, want)
    # no centring, no 1/N: a constant column c over N tokens gives N c^2
    assert orc.cov(np.full((10, 1), 3.0))[0, 0] == 90.0


def test_cov_matches_library_matmul_and_headwise_slices():
    rng = np.random.default_rng(2)
    X = rng.standard_normal((64, 24)).astype(np.float16)
    X64 = X.astype(np.float64)
    assert np.allclose(orc.cov(X), X64.T @ X64, rtol=1e-13, atol=1e-13)
    Cb = orc.cov(X, n_blocks=3)
    for h in range(3):
        s = X64[:, 8 * h:8 * h + 8]
        assert np.allclose(Cb[h], s.T @ s, rtol=1e-13, atol=1e-13)


# ----------------------------------------------------------------- Eq. 4: eigenpairs
def test_jacobi_closed_form_2x2_and_diagonal():
    lam, V = orc.eigh_jacobi(np.array([[2.0, 1.0], [1.0, 2.0]]))
    assert np.allclose(lam, [3.0, 1.0], atol=1e-14)
    r = np.sqrt(0.5)
    assert np.allclose(V[:, 0], [r, r], atol=1e-14)      # sign rule: largest entry (lowest index) positive
    assert np.allclose(V[:, 1], [r, -r], atol=1e-14)
    lam, V = orc.eigh_jacobi(np.diag([1.0, 5.0, 3.0]))     # sorted DESCENDING, vectors follow
    assert np.array_equal(lam, [5.0, 3.0, 1.0])
    assert np.array_equal(V, np.eye(3)[:, [1, 2, 0]])


def test_jacobi_eigenpairs_residual_orthogonality_trace_and_library_values():
    law = synth.ActivationLaw(96, 1.2, seed=5, key="pin", mix="qr")
    X = law.sample(64, "X", np.float32)      # N < d: a third of the spectrum is ~0, as in the configs
    Cm = orc.cov(X)
    lam, V = orc.eigh_jacobi(Cm)
    nC = np.linalg.norm(Cm)
    assert np.all(np.diff(lam) <= 1e-12 * nC)
    assert np.abs(Cm @ V - V * lam[None, :]).max() <= 1e-10 * nC
    assert np.abs(V.T @ V - np.eye(96)).max() <= 1e-12
    assert lam.sum() == pytest.approx(np.trace(Cm), rel=1e-12)
    X64 = X.astype(np.float64)
    assert np.allclose(np.sum((X64 @ V) ** 2, axis=0), lam, rtol=1e-9, atol=1e-10 * nC)
    ref = np.linalg.eigvalsh(Cm)[::-1]
    assert np.allclose(lam, ref, rtol=1e-10, atol=1e-12 * nC)


def test_pca_known_answer_recovers_planted_directions():
    d = 16
    law = synth.ActivationLaw(d, 1.5, seed=7, key="planted", mix="qr")
    X = law.sample(8 * 4096, "X", np.float64)
    lam, V = orc.eigh_jacobi(orc.cov(X))
    U = law.principal_directions()
    # top directions match the planted ones up to sign; eigenvalues ~ N * i^-1.5
    for j in range(4):
        assert abs(abs(V[:, j] @ U[:, j]) - 1.0) < 2e-2
    assert lam[0] / lam[1] == pytest.approx(2 ** 1.5, rel=0.1)


# ----------------------------------------------------------------- Eq. 1: rotational invariance
@pytest.mark.parametrize("headwise", [False, True])
def test_rotational_invariance_fp64(headwise):
    rng = np.random.default_rng(3)
    d, dout, M = 64, 24, 5
    W = rng.standard_normal((d, dout)) * 0.02
    x = rng.standard_normal((M, d))
    if headwise:
        H, dh = 4, 16
        Xc = rng.standard_normal((200, d)) * np.linspace(3, 0.1, d)[None, :]
        lams, Vs = zip(*[orc.eigh_jacobi(orc.cov(Xc[:, h * dh:(h + 1) * dh])) for h in range(H)])
        Rb, perm = orc.assemble_headwise_rotation(np.array(lams), np.array(Vs))
        flat = np.array(lams).reshape(-1)[perm]
        assert np.all(np.diff(flat) <= 0)                      # global descending order
    else:
        Xc = rng.standard_normal((200, d)) @ rng.standard_normal((d, d))
        _, V = orc.eigh_jacobi(orc.cov(Xc))
        Rb, perm = V, None
    Wp = orc.rotate_weights_f64(Rb, W, perm)
    # y through the oracle's own rotate (forward's first half) and an all-FP16-free product
    _, xr = orc.forward(x, dict(salient=np.zeros((0, dout), np.float16), scales=np.zeros((d // 16, dout), np.float16),
                                zeros=np.zeros((d // 16, dout), np.float16),
                                codes=np.zeros((d, dout), np.uint8), bits=4, group=16, k_salient=0),
                        Rb, perm, return_xrot=True)
    y = xr @ Wp
    ref = x @ W
    assert np.linalg.norm(y - ref) / np.linalg.norm(ref) <= 1e-10
    # and the rotate really is x.R with R = blockdiag . P (a transposed R would fail here)
    R = orc.dense_from_blocks(Rb, perm)
    assert np.allclose(xr, x @ R, rtol=1e-12, atol=1e-12)
    assert np.allclose(Wp, R.T @ W, rtol=1e-12, atol=1e-14)


def test_rotate_weights_asymmetric_known_answer():
    # R = a 90-degree plane rotation: R^T W swaps/negates rows; R W would give the other sign.
    R = np.array([[0.0, -1.0], [1.0, 0.0]])
    W = np.array([[1.0, 2.0], [3.0, 4.0]])
    assert np.array_equal(orc.rotate_weights_f64(R, W), np.array([[3.0, 4.0], [-1.0, -2.0]]))
    got32 = orc.rotate_weights_f32(R.astype(np.float32), W.astype(np.float16))
    assert np.array_equal(got32, np.array([[3.0, 4.0], [-1.0, -2.0]], np.float32))


def _round_f32(fr):
    """Exact round-to-nearest-even of a rational to fp32 (candidates: the fp32 nearest to the
    fp64 approximation and its two neighbours; the winner is chosen with exact arithmetic)."""
    c = np.float32(float(fr))
    cands = [np.nextafter(c, np.float32(-np.inf)), c, np.nextafter(c, np.float32(np.inf))]
    best = min(cands, key=lambda v: (abs(Fraction(float(v)) - fr), int(v.view(np.uint32)) & 1))
    return best


def test_rotate_weights_f32_chain_is_sequential_fma():
    rng = np.random.default_rng(4)
    d, dout = 40, 6
    R = rng.standard_normal((d, d)).astype(np.float32)
    W = (rng.standard_normal((d, dout)) * 0.02).astype(np.float16)
    got = orc.rotate_weights_f32(R, W)
    # brute force with exact rationals: each step is round_to_fp32(exact(a*b + acc))
    for i in range(d):
        for n in range(dout):
            acc = np.float32(0.0)
            for k in range(d):
                acc = _round_f32(Fraction(float(R[k, i])) * Fraction(float(W[k, n])) + Fraction(float(acc)))
            assert got[i, n] == acc
    # identity rotation leaves W untouched, exactly (one non-zero term per chain)
    assert np.array_equal(orc.rotate_weights_f32(np.eye(d, dtype=np.float32), W), W.astype(np.float32))
    # close to the fp64 result
    assert np.allclose(got, orc.rotate_weights_f64(R.astype(np.float64), W), rtol=0, atol=1e-5)


def test_headwise_equals_dense_blockdiag():
    """Eq. 6 (sum over heads) equals Eq. 7 fed the block-diagonal matrix."""
    rng = np.random.default_rng(5)
    H, dh, dout, M = 3, 16, 8, 4
    d = H * dh
    Vs = np.array([synth.orthogonal_qr(dh, rng) for _ in range(H)])
    lams = np.sort(rng.uniform(0.1, 10, (H, dh)), axis=1)[:, ::-1]
    Rb, perm = orc.assemble_headwise_rotation(lams, Vs)
    Rd = orc.dense_from_blocks(Rb, perm)
    W = (rng.standard_normal((d, dout)) * 0.02).astype(np.float16)
    x = rng.standard_normal((M, d)).astype(np.float16)
    a = orc.rotate_weights_f32(Rb.astype(np.float32), W, perm)
    b = orc.rotate_weights_f32(Rd.astype(np.float32), W)
    assert np.array_equal(a, b)          # extra exact-zero terms do not move an fma chain
    qd = orc.quantize(a, 4, group=16, k_salient=16)
    ya = orc.forward(x, qd, Rb.astype(np.float16), perm)
    yb = orc.forward(x, qd, Rd.astype(np.float16))
    assert np.allclose(ya, yb, rtol=1e-13, atol=1e-15)


# ----------------------------------------------------------------- quantizer (Eq. 3, Section 3.3)
@pytest.mark.parametrize("bits", [3, 4])
def test_quantizer_grid_round_trip(bits):
    rng = np.random.default_rng(6)
    qmax = 2 ** bits - 1
    g, ng, n = 128, 3, 9
    s = rng.uniform(1e-3, 5e-2, (ng, n)).astype(np.float16)
    z = rng.integers(0, qmax + 1, (ng, n))
    q = rng.integers(0, qmax + 1, (ng * g, n))
    for gi in range(ng):                      # both extremes present in every group and column
        q[gi * g + 3, :] = 0
        q[gi * g + 77, :] = qmax
    w = ((q - np.repeat(z, g, 0)) * np.repeat(s.astype(np.float64), g, 0)).astype(np.float32)
    qd = orc.quantize(w, bits, g, 0)
    assert np.array_equal(qd["codes"], q)
    assert np.array_equal(qd["scales"].view(np.uint16), s.view(np.uint16))
    assert np.array_equal(qd["zeros"].astype(np.int64), z)
    assert np.array_equal(orc.dequantize(qd).astype(np.float32), w)
    # without the top extreme the recomputed scale legitimately differs
    w2 = w.copy()
    top = q[:g, 0] == qmax
    w2[:g, 0][top] = w2[3, 0]
    assert orc.quantize(w2, bits, g, 0)["scales"][0, 0] < s[0, 0]


@pytest.mark.parametrize("bits", [3, 4])
def test_quantizer_error_bound_and_salient_cast(bits):
    W = synth.weights(512, 32, seed=11, key="eb", outlier_rows=4, outlier_scale=20.0).astype(np.float32)
    W *= np.float32(1.37)                               # off the fp16 grid
    qd = orc.quantize(W, bits, 128, 128)
    assert np.array_equal(qd["salient"], W[:128].astype(np.float16))
    qmax = 2 ** bits - 1
    assert qd["codes"].max() <= qmax
    what = orc.dequantize(qd)[128:]
    s = np.repeat(qd["scales"].astype(np.float64), 128, 0)
    z = np.repeat(qd["zeros"].astype(np.float64), 128, 0)
    inside = (W[128:] >= (0 - z) * s) & (W[128:] <= (qmax - z) * s)
    assert inside.mean() > 0.9
    assert np.all(np.abs(W[128:] - what)[inside] <= s[inside] / 2 * (1 + 2.0 ** -10))
    # the group minimum takes code 0 whenever the zero point is not clipped
    Wg = W[128:].reshape(3, 128, 32)
    amin = Wg.argmin(axis=1)
    cmin = np.take_along_axis(qd["codes"].reshape(3, 128, 32), amin[:, None, :], 1)[:, 0, :]
    zz = qd["zeros"].astype(np.float64)
    assert np.all(cmin[(zz > 0) & (zz < qmax)] == 0)


def test_quantizer_hand_computable_groups():
    g = 128
    # (a) two-level group {0, 1.5}: range 1.5, INT4 scale = fp16(0.1) = 0.0999755859375, zero 0, codes {0, 15}
    w = np.zeros((g, 1), np.float32)
    w[5:40] = 1.5
    qd = orc.quantize(w, 4, g, 0)
    assert float(qd["scales"][0, 0]) == float(np.float16(0.1)) == 0.0999755859375
    assert qd["zeros"].view(np.uint16)[0, 0] == 0        # +0, never -0
    assert set(np.unique(qd["codes"])) == {0, 15}
    # (b) ramp -1..+1 shifted: lo = -1, hi = 1, INT3: s = fp16(2/7), z = round(1/s) = round(3.5003..) = 4
    w = np.linspace(-1.0, 1.0, g, dtype=np.float32)[:, None]
    qd = orc.quantize(w, 3, g, 0)
    s = float(np.float16(np.float32(2.0) / np.float32(7.0)))
    assert float(qd["scales"][0, 0]) == s
    assert float(qd["zeros"][0, 0]) == 4.0
    assert qd["codes"][0, 0] == 0 and qd["codes"][-1, 0] == 7       # rint(-3.5003)+4 = 0; rint(3.5003)+4 = 8 -> clamp 7
    assert np.all(np.diff(qd["codes"][:, 0].astype(int)) >= 0)
    # (c) constant group: range floored at 1e-5, all-positive group => zero point clamps at 0 and codes clip at qmax
    w = np.full((g, 1), 0.25, np.float32)
    qd = orc.quantize(w, 4, g, 0)
    assert float(qd["scales"][0, 0]) == float(np.float16(np.float32(1e-5) / np.float32(15.0)))
    assert float(qd["zeros"][0, 0]) == 0.0 and np.all(qd["codes"] == 15)
    # (d) ties go to even: w/s = 0.5 -> 0, 1.5 -> 2, 2.5 -> 2  (s = 1/8 exactly, lo = 0 => z = 0)
    w = np.zeros((g, 1), np.float32)
    w[0], w[1], w[2], w[3] = 0.0625, 0.1875, 0.3125, 15 / 8
    qd = orc.quantize(w, 4, g, 0)
    assert float(qd["scales"][0, 0]) == 0.125
    assert qd["codes"][:4, 0].tolist() == [0, 2, 2, 15]
    # (e) all-negative group: z = qmax side; lo=-3, hi=-1 INT4: s=fp16(2/15), z=clamp(round(22.5..),0,15)=15
    w = np.linspace(-3.0, -1.0, g, dtype=np.float32)[:, None]
    qd = orc.quantize(w, 4, g, 0)
    assert float(qd["zeros"][0, 0]) == 15.0 and qd["codes"].min() == 0


# ----------------------------------------------------------------- packing
def _pack_reference_bigint(codes, bits):
    """Independent restatement with Python integers: little-endian bit string per block."""
    r, n = codes.shape
    per = 8 if bits == 4 else 32
    words = 1 if bits == 4 else 3
    out = np.zeros((r // per * words, n), np.uint32)
    for col in range(n):
        for b in range(r // per):
            big = 0
            for i in range(per):
                big |= int(codes[b * per + i, col]) << (bits * i)
            for w in range(words):
                out[b * words + w, col] = (big >> (32 * w)) & 0xFFFFFFFF
    return out


@pytest.mark.parametrize("bits", [3, 4])
def test_pack_unpack_bijection_and_known_words(bits):
    rng = np.random.default_rng(8)
    qmax = 2 ** bits - 1
    r, n = 256, 5
    cases = [np.zeros((r, n), np.uint8), np.full((r, n), qmax, np.uint8),
             (np.arange(r)[:, None] % (qmax + 1) * np.ones((1, n))).astype(np.uint8),
             rng.integers(0, qmax + 1, (r, n)).astype(np.uint8)]
    for c in cases:
        qw = orc.pack(c, bits)
        assert np.array_equal(qw, _pack_reference_bigint(c, bits))
        assert np.array_equal(orc.unpack(qw, r, bits), c)
    if bits == 4:
        c = np.arange(8, dtype=np.uint8)[:, None]
        assert orc.pack(c, 4)[0, 0] == 0x76543210
    else:
        # one code set at a time: rows 10 and 21 straddle words 0/1 and 1/2
        for row, want in [(0, (7, 0, 0)), (10, (0b11 << 30, 0b1, 0)), (21, (0, 0x80000000, 0b11)),
                          (31, (0, 0, 0b111 << 29))]:
            c = np.zeros((32, 1), np.uint8)
            c[row] = 7
            assert tuple(int(v) for v in orc.pack(c, 3)[:, 0]) == want


# ----------------------------------------------------------------- forward (Eq. 3)
def test_forward_brute_force_tiny():
    rng = np.random.default_rng(9)
    d, dout, M, g, K = 64, 6, 3, 16, 16
    Wp = (rng.standard_normal((d, dout)) * 0.05).astype(np.float32)
    x = rng.standard_normal((M, d)).astype(np.float16)
    for bits in (3, 4):
        qd = orc.quantize(Wp, bits, g, K)
        y = orc.forward(x, qd)
        for m in range(M):
            for n in range(dout):
                acc = 0.0
                for i in range(d):
                    if i < K:
                        w = float(qd["salient"][i, n])
                    else:
                        gi = (i - K) // g
                        w = (float(qd["codes"][i - K, n]) - float(qd["zeros"][gi, n])) * float(qd["scales"][gi, n])
                    acc += float(x[m, i]) * w
                assert y[m, n] == pytest.approx(acc, rel=1e-12, abs=1e-14)


def test_forward_special_cases_reduce_to_plain_products():
    rng = np.random.default_rng(10)
    d, dout, M = 256, 16, 4
    W = (rng.standard_normal((d, dout)) * 0.02).astype(np.float16)
    x = rng.standard_normal((M, d)).astype(np.float16)
    ref = x.astype(np.float64) @ W.astype(np.float64)
    # K = d_in: every channel salient => the plain fp16-weight product, exact in fp64
    qd = orc.quantize(W.astype(np.float32), 4, 128, d)
    assert qd["codes"].shape[0] == 0
    assert np.allclose(orc.forward(x, qd), ref, rtol=1e-13, atol=1e-16)
    # K = 0, no rotation: plain W4 g128 linear; error is the quantizer's, a few % at 4 bits
    qd = orc.quantize(W.astype(np.float32), 4, 128, 0)
    y = orc.forward(x, qd)
    assert np.allclose(y, x.astype(np.float64) @ orc.dequantize(qd), rtol=1e-13, atol=1e-16)
    assert np.linalg.norm(y - ref) / np.linalg.norm(ref) < 0.12


def test_mixed_precision_helps_in_rotated_space():
    """Sanity of the method itself on the tiny config: with the PCA rotation the salient FP16 group
    carries most of the activation energy, so the output error drops versus no rotation."""
    law = synth.ActivationLaw(256, 1.2, seed=0, key="mini", mix="qr")
    X = law.sample(128, "calib", np.float32)
    _, V = orc.eigh_jacobi(orc.cov(X))
    W = synth.weights(256, 64, seed=0, key="mini", outlier_rows=2, outlier_scale=20.0)
    x = law.sample(16, "x", np.float16)
    ref = x.astype(np.float64) @ W.astype(np.float64)
    q_rot = orc.quantize(orc.rotate_weights_f32(V.astype(np.float32), W), 3, 128, 128)
    y_rot = orc.forward(x, q_rot, V.astype(np.float16))
    q_id = orc.quantize(W.astype(np.float32), 3, 128, 128)
    y_id = orc.forward(x, q_id)
    e_rot = np.linalg.norm(y_rot - ref) / np.linalg.norm(ref)
    e_id = np.linalg.norm(y_id - ref) / np.linalg.norm(ref)
    assert e_rot < e_id


def test_frozen_quantizer_output_has_not_drifted():
    """The oracle's quantizer and bit layout are definitions of this repository (the paper gives none); a
    stored answer on a closed-form input makes any later change to them explicit."""
    import importlib.util
    import os
    here = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
    spec = importlib.util.spec_from_file_location("make_rtn_golden", os.path.join(here, "make_rtn_golden.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    W = mod.closed_form_weights()
    want = {}
    bits = None
    for line in open(os.path.join(here, "rtn_groups.txt")):
        if line.startswith("#"):
            continue
        key, *vals = line.split()
        if key == "bits":
            bits = int(vals[0])
            want[bits] = {}
        else:
            want[bits][key] = [int(v, 16) for v in vals]
    for b in (4, 3):
        qd = orc.quantize(W, b, 128, 128)
        qw = orc.pack(qd["codes"], b)
        assert list(qd["scales"].view(np.uint16).ravel()) == want[b]["scales"]
        assert list(qd["zeros"].view(np.uint16).ravel()) == want[b]["zeros"]
        assert list(qd["salient"].view(np.uint16)[0]) == want[b]["salient_row0"]
        for r in range(qw.shape[0]):
            assert list(qw[r]) == want[b][f"qw{r}"]


# --------------------------------------------------------------------------- scaling invariance (W_D variant)
def test_scaling_invariance_fp64_with_and_without_rotation():
    """X W = (X D^-1)(D W) for any invertible diagonal D (appendix on rotational and scaling invariance),
    alone and combined with an orthogonal R: (X D^-1 R)(R^T D W) = X W, <= 1e-10 in fp64."""
    rng = np.random.default_rng(31)
    d_in, d_out, M = 256, 24, 5
    W = rng.standard_normal((d_in, d_out))
    x = rng.standard_normal((M, d_in))
    d = rng.uniform(0.25, 4.0, d_in)
    ref = x @ W
    DW = orc.scale_rows_f64(W, d)
    assert np.array_equal(DW[7], d[7] * W[7])                              # row i scaled by d[i], nothing else
    assert np.linalg.norm((x / d) @ DW - ref) / np.linalg.norm(ref) <= 1e-10
    R = synth.orthogonal_qr(d_in, rng)
    Wp = orc.rotate_weights_f64(R, DW)
    assert np.linalg.norm(((x / d) @ R) @ Wp - ref) / np.linalg.norm(ref) <= 1e-10
    # a wrong side (D applied to the columns, or D^-1 forgotten) must not pass
    assert np.linalg.norm(x @ DW - ref) / np.linalg.norm(ref) > 1e-2


def test_scale_rows_f32_is_one_rounded_product_and_identity_for_ones():
    rng = np.random.default_rng(32)
    W = (rng.standard_normal((8, 6)) * 0.02).astype(np.float16)
    ones = np.ones(8, np.float32)
    assert np.array_equal(orc.scale_rows_f32(W, ones).view(np.uint32), W.astype(np.float32).view(np.uint32))
    d = np.array([0.5, 2.0, 3.0, 1.0 / 3.0, 0.1, 7.0, 1e-3, 1.5], np.float32)
    got = orc.scale_rows_f32(W, d)
    for i in range(8):
        for n in range(6):
            want = _round_f32(Fraction(float(d[i])) * Fraction(float(W[i, n])))
            assert got[i, n].view(np.uint32) == want.view(np.uint32)
    # exactly representable products: 0.75 * 3 = 2.25, 0.375 * 0.5 = 0.1875
    Wk = np.array([[0.75], [0.375]], np.float16)
    assert orc.scale_rows_f32(Wk, np.array([3.0, 0.5], np.float32)).tolist() == [[2.25], [0.1875]]


def test_scaled_quantization_hand_computed_group_and_unit_scale_is_todays_path():
    """A group whose rows are 0, 1, ..., 127 times 2^-10 scaled by D = 2 quantizes like the group 0 .. 127 times
    2^-9 (INT4: range 127 * 2^-9, fifteen steps); with D = 1 every output bit equals the unscaled path."""
    rows = (np.arange(128, dtype=np.float64) * 2.0 ** -10)
    W = np.concatenate([np.zeros((128, 1)), rows[:, None]], axis=0).astype(np.float16)      # salient group + one group
    two = np.full(256, 2.0, np.float32)
    a = orc.quantize(orc.scale_rows_f32(W, two), 4, 128, 128)
    b = orc.quantize((W.astype(np.float32) * np.float32(2.0)), 4, 128, 128)
    for k in ("salient", "scales", "zeros", "codes"):
        assert np.array_equal(a[k], b[k])
    s = np.float16(np.float32(127 * 2.0 ** -9) / np.float32(15))
    assert a["scales"][0, 0] == s and a["zeros"][0, 0] == 0
    assert a["codes"][0, 0] == 0 and a["codes"][127, 0] == 15
    assert a["codes"][64, 0] == int(np.rint(np.float32(64 * 2.0 ** -9) / np.float32(s)))
    one = np.ones(256, np.float32)
    c = orc.quantize(orc.scale_rows_f32(W, one), 4, 128, 128)
    e = orc.quantize(W.astype(np.float32), 4, 128, 128)
    for k in ("salient", "scales", "zeros", "codes"):
        assert np.array_equal(c[k], e[k])


def test_scaled_then_rotated_chain_takes_the_fp32_scaled_weight():
    rng = np.random.default_rng(33)
    d_in, d_out = 64, 5
    W = (rng.standard_normal((d_in, d_out)) * 0.02).astype(np.float16)
    R = synth.orthogonal_qr(d_in, rng).astype(np.float32)
    d = rng.uniform(0.5, 2.0, d_in).astype(np.float32)
    DW = orc.scale_rows_f32(W, d)
    got = orc.rotate_weights_f32(R, DW)
    for i in (0, 17, 63):
        for n in range(d_out):
            acc = np.float32(0.0)
            for k in range(d_in):
                acc = _round_f32(Fraction(float(R[k, i])) * Fraction(float(DW[k, n])) + Fraction(float(acc)))
            assert got[i, n].view(np.uint32) == acc.view(np.uint32)
    # and it is the same chain as the binary16 entry when the scaled weight happens to be the widened one
    assert np.array_equal(orc.rotate_weights_f32(R, W.astype(np.float32)).view(np.uint32),
                          orc.rotate_weights_f32(R, W).view(np.uint32))


# --------------------------------------------------------------------------- W_O layout and selection ablation
def test_per_head_salient_layout_is_a_permutation_and_keeps_eq1():
    """32 salient directions per head (weight-splitting appendix): the column order is a permutation, its
    first H * 32 entries are exactly each head's 32 largest-eigenvalue directions, and the rotated linear
    with this R still equals x W in fp64 (Eq. 1 / Eq. 6)."""
    rng = np.random.default_rng(41)
    H, dh, d_out, M = 4, 128, 12, 3
    lams = -np.sort(-rng.uniform(0.1, 5.0, (H, dh)), axis=1)
    Vs = np.array([synth.orthogonal_qr(dh, rng) for _ in range(H)])
    Rb, perm, K = orc.assemble_headwise_rotation_per_head(lams, Vs, 32)
    assert K == 128 and sorted(perm.tolist()) == list(range(H * dh))
    assert perm[:K].tolist() == [h * dh + i for h in range(H) for i in range(32)]
    for h in range(H):                                   # every salient column is among its head's 32 largest
        mine = [p % dh for p in perm[:K] if p // dh == h]
        assert sorted(mine) == list(range(32)) and lams[h, 31] >= lams[h, 32]
    W = rng.standard_normal((H * dh, d_out))
    x = rng.standard_normal((M, H * dh))
    R = orc.dense_from_blocks(Rb, perm)
    assert np.abs(R.T @ R - np.eye(H * dh)).max() <= 1e-12
    Wp = orc.rotate_weights_f64(Rb, W, perm)
    ref = x @ W
    assert np.linalg.norm((x @ R) @ Wp - ref) / np.linalg.norm(ref) <= 1e-10


@pytest.mark.parametrize("mode", ["top", "bottom", "random", "top_bottom"])
def test_selection_orders_are_permutations_with_the_named_salient_set(mode):
    rng = np.random.default_rng(42)
    d, K = 256, 128
    lam = -np.sort(-rng.uniform(0.0, 1.0, d))
    perm = orc.selection_order(lam, K, mode, rng)
    assert sorted(perm.tolist()) == list(range(d))
    sel = set(perm[:K].tolist())
    if mode == "top":
        assert perm.tolist() == list(range(d))
    elif mode == "bottom":
        assert sel == set(range(d - K, d))
    elif mode == "top_bottom":
        assert sel == set(range(K // 2)) | set(range(d - K // 2, d))
    assert np.all(np.diff(perm[K:]) > 0)                 # the others stay in descending-eigenvalue order
    V = synth.orthogonal_qr(d, rng)
    W = rng.standard_normal((d, 7))
    x = rng.standard_normal((2, d))
    Wp = orc.rotate_weights_f64(V, W, perm)
    ref = x @ W
    assert np.linalg.norm((x @ V[:, perm]) @ Wp - ref) / np.linalg.norm(ref) <= 1e-10
    # the product helper agrees with the oracle's index rule
    from paper_2506_13472_b200 import pca
    if mode != "random":
        assert np.array_equal(pca.selection_order(d, K, mode), perm)
