"""Shared builders for the parity tests: seeded configs, oracle-side expectations, comparisons."""
import functools

import numpy as np

from oracle import rosaq_oracle as orc
from paper_2506_13472_b200 import synth

REL_TOL_Y = 2e-3   # ||y - y_ref||_F / ||y_ref||_F, the bound the path is specified to


def rel_fro(a, b):
    a = np.asarray(a, np.float64)
    b = np.asarray(b, np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


@functools.lru_cache(maxsize=None)
def config_tiny(seed=0):
    """Config 1: d_in = d_out = 512, 256 calibration tokens (fp32), spectrum i^-1.2, QR mix,
    4 outlier input rows x20, M = 4.  R = oracle Jacobi eigenvectors of X^T X."""
    d = 512
    law = synth.ActivationLaw(d, 1.2, seed, "tiny", mix="qr")
    X = law.sample(256, "calib", np.float32)
    lam, V = orc.eigh_jacobi(orc.cov(X))
    W = synth.weights(d, d, seed, "tiny", sigma=0.02, outlier_rows=4, outlier_scale=20.0)
    x = law.sample(4, "x", np.float16)
    return dict(X=X, lam=lam, R64=V, R32=V.astype(np.float32), R16=V.astype(np.float16), W=W, x=x, d=d)


@functools.lru_cache(maxsize=None)
def config_headwise(seed=3, heads=4, head_dim=128, n_tokens=512, d_out=384, M=5):
    """Small head-wise case (Eq. 6): per-head PCA blocks + the global descending permutation."""
    law = synth.HeadwiseActivationLaw(heads, head_dim, seed, "hw")
    X = law.sample(n_tokens, "calib", np.float16)
    Cb = orc.cov(X, n_blocks=heads)
    lams, Vs = zip(*[orc.eigh_jacobi(Cb[h]) for h in range(heads)])
    Rb, perm = orc.assemble_headwise_rotation(np.array(lams), np.array(Vs))
    W = synth.weights(heads * head_dim, d_out, seed, "hw", outlier_frac=0.01)
    x = law.sample(M, "x", np.float16)
    return dict(X=X, Rb64=Rb, Rb32=Rb.astype(np.float32), Rb16=Rb.astype(np.float16), perm=perm, W=W, x=x,
                heads=heads, head_dim=head_dim)


def oracle_quantized(W16, R32_blocks, perm, bits, k_salient, cols=None, group=128):
    """Oracle expectation for rosaq_quantize on the listed columns: dict with packed qw too."""
    d_in, d_out = W16.shape
    cols = np.arange(d_out, dtype=np.int32) if cols is None else np.asarray(cols, np.int32)
    if R32_blocks is None:
        Wp = W16[:, cols].astype(np.float32)
    else:
        Wp = orc.rotate_weights_f32(R32_blocks, W16, perm, cols)
    qd = orc.quantize(Wp, bits, group, k_salient)
    qd["qw"] = orc.pack(qd["codes"], bits) if qd["codes"].shape[0] else np.zeros((0, cols.size), np.uint32)
    qd["cols"] = cols
    return qd


def assert_export_matches(exported, qd):
    """Bit-exact comparison of a GPU export (numpy arrays) with the oracle dict on qd['cols']."""
    cols = qd["cols"]
    got_qw = exported["qw"].view(np.uint32)[:, cols]
    assert np.array_equal(exported["salient"].view(np.uint16)[:, cols], qd["salient"].view(np.uint16)), "salient"
    assert np.array_equal(exported["scales"].view(np.uint16)[:, cols], qd["scales"].view(np.uint16)), "scales"
    assert np.array_equal(exported["zeros"].view(np.uint16)[:, cols], qd["zeros"].view(np.uint16)), "zeros"
    assert np.array_equal(got_qw, qd["qw"]), "packed codes"


def export_to_numpy(exported):
    return {k: v.cpu().numpy() for k, v in exported.items()}


def cov_tolerance(Cref, n_tokens):
    """Element-wise bound on |C_gpu - C_ref| for rosaq_calib_cov.  Products are exact in fp32
    (fp16 x fp16) or rounded once (fp32 inputs); what is left is the fp32 accumulation.  CUDA-core
    path: N sequential roundings, ~sqrt(N) u in practice.  Tensor-core path: one accumulator update per
    16 tokens, each within one unit in the last place (2^-23, the tensor core truncates) of the running
    sum, which Cauchy-Schwarz bounds by sqrt(C_ii C_jj).  The bound below covers both."""
    dg = np.sqrt(np.clip(np.diagonal(Cref, axis1=-2, axis2=-1), 0, None))
    steps = max(4.0 * np.sqrt(n_tokens) + 8.0, 2.0 * (n_tokens / 16.0 + 8.0))
    return 2.0 ** -24 * steps * dg[..., :, None] * dg[..., None, :]


def qd_from_export(exported, bits, k_salient, group=128):
    """The oracle's weight dict built from a GPU export (numpy arrays, all columns): what
    orc.forward needs to compute y_ref on exactly the weights the GPU holds."""
    d_q = exported["scales"].shape[0] * group
    codes = (orc.unpack(exported["qw"].view(np.uint32), d_q, bits) if d_q
             else np.zeros((0, exported["salient"].shape[1]), np.uint8))
    return dict(salient=exported["salient"], scales=exported["scales"], zeros=exported["zeros"], codes=codes,
                bits=bits, group=group, k_salient=k_salient)


def tile_columns(d_out, seed, key, tile=128):
    """One seeded column out of every `tile`-column tile, plus the first and last column of the matrix
    and both sides of the first tile edge."""
    rng = synth.rng_for(seed, key, "tilecols")
    cols = {0, d_out - 1, min(tile - 1, d_out - 1), min(tile, d_out - 1)}
    for t0 in range(0, d_out, tile):
        cols.add(int(t0 + rng.integers(0, min(tile, d_out - t0))))
    return np.asarray(sorted(cols), dtype=np.int32)


def assert_y_all_columns(y, x_in16, qd, tile=128, chunk=2048, where=""):
    """y (fp16, every column) against the oracle's fp64 forward on the same activations and the same
    dequantised weights:  the 2e-3 Frobenius bound on every `tile`-column tile (a bad tile cannot hide
    in the norm of the whole matrix), and element by element
        |y - y_ref| <= 2e-3 * (|x| . |W^|)_mn + ulp_fp16(y_ref)
    (the products carry at most one fp16 rounding of W^ each, the sum is fp32, y is rounded once).
    x_in16 is what the GEMM stage was fed (already rotated)."""
    y = np.asarray(y)
    M, d_out = y.shape
    assert np.all(np.isfinite(y)), where
    xa = np.abs(orc.f16_to_f64(np.ascontiguousarray(x_in16, np.float16)))
    worst_tile, worst_elem = 0.0, 0.0
    for c0 in range(0, d_out, chunk):
        c1 = min(c0 + chunk, d_out)
        sub = dict(qd, salient=qd["salient"][:, c0:c1], scales=qd["scales"][:, c0:c1], zeros=qd["zeros"][:, c0:c1],
                   codes=qd["codes"][:, c0:c1])
        y_ref = orc.forward(x_in16, sub)
        mag = xa @ np.abs(orc.dequantize(sub))
        got = y[:, c0:c1].astype(np.float64)
        bound = REL_TOL_Y * mag + np.spacing(np.abs(y_ref).astype(np.float16)).astype(np.float64)
        ratio = np.abs(got - y_ref) / np.maximum(bound, 1e-300)
        worst_elem = max(worst_elem, float(ratio.max()))
        bad = np.argwhere(ratio > 1.0)
        assert bad.size == 0, f"{where}: element (token {bad[0][0]}, column {c0 + bad[0][1]}) off by {ratio.max():.2f} bounds"
        for t0 in range(0, c1 - c0, tile):
            e = rel_fro(got[:, t0:t0 + tile], y_ref[:, t0:t0 + tile])
            worst_tile = max(worst_tile, e)
            assert e <= REL_TOL_Y, f"{where}: columns {c0 + t0}..{c0 + t0 + tile - 1}: {e:.2e}"
    return worst_tile, worst_elem
