"""ctypes front end of the ROSAQ oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.

Loads ``librosaq_oracle.so`` (built from ``rosaq_oracle.c`` by ``build_oracle``) and
exposes its functions on numpy arrays.  The arithmetic of the method lives in the C
file; this module only marshals arrays, except for the two pure index/assembly
steps that are clearer in numpy (``assemble_headwise_rotation``, ``dense_from_blocks``).
Nothing here imports or is imported by the CUDA package.

Notation follows the paper: X calibration activations, R rotation (eigenvectors of
X^T X, Eq. 4), W weight, W' = R^T W (Eq. 1), K salient channels (Eq. 3).
"""
import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "rosaq_oracle.c")
_LIB = os.path.join(_HERE, "librosaq_oracle.so")
_lib = None


def build_oracle(force=False):
    """Compile the C oracle in place.  Contraction is off so a*b+c is never fused."""
    if not force and os.path.exists(_LIB) and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC):
        return _LIB
    cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-mfma",
           "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    return _LIB


def _L():
    global _lib
    if _lib is None:
        build_oracle()
        _lib = C.CDLL(_LIB)
        _lib.oracle_eigh_jacobi.restype = C.c_int
        _lib.oracle_num_threads.restype = C.c_int
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _c(a, dt):
    return np.ascontiguousarray(a, dtype=dt)


def num_threads():
    return int(_L().oracle_num_threads())


# ---------------------------------------------------------------- conversions
def f16_to_f64(h):
    """binary16 array (np.float16 or uint16 bits) -> exact fp64 values."""
    hb = _c(np.asarray(h).view(np.uint16) if np.asarray(h).dtype == np.float16 else h, np.uint16)
    out = np.empty(hb.shape, np.float64)
    _L().oracle_f16_to_f64(_p(hb), C.c_int64(hb.size), _p(out))
    return out


def f32_to_f16_bits(f):
    fb = _c(f, np.float32)
    out = np.empty(fb.shape, np.uint16)
    _L().oracle_f32_to_f16(_p(fb), C.c_int64(fb.size), _p(out))
    return out


# ---------------------------------------------------------------- Eq. 4
def cov(X, n_blocks=1):
    """C = X^T X (uncentred, unnormalised); head-wise: [n_blocks][dh][dh]."""
    X64 = f16_to_f64(X) if np.asarray(X).dtype == np.float16 else _c(X, np.float64)
    n, d = X64.shape
    dh = d // n_blocks
    out = np.empty((n_blocks, dh, dh), np.float64)
    _L().oracle_cov(_p(X64), C.c_int64(n), C.c_int(d), C.c_int(n_blocks), _p(out))
    return out[0] if n_blocks == 1 else out


def eigh_jacobi(Cm):
    """(lambda descending, V with V[:, j] the eigenvector of lambda[j])."""
    Cm = _c(Cm, np.float64)
    d = Cm.shape[0]
    lam = np.empty(d, np.float64)
    V = np.empty((d, d), np.float64)
    sweeps = _L().oracle_eigh_jacobi(_p(Cm), C.c_int(d), _p(lam), _p(V))
    if sweeps < 0:
        raise RuntimeError("Jacobi did not converge")
    return lam, V


def assemble_headwise_rotation(lams, Vs):
    """Section 3.1.1 / Eq. 6 with one global salient group.

    lams [H][dh] descending per head, Vs [H][dh][dh].  The rotation is
    blockdiag(V_1..V_H) followed by the column permutation that orders all H*dh
    (eigenvalue, head, index) triples by descending eigenvalue (stable), so that
    the first K columns are the K most principal directions over all heads.
    Returns (Rb [H][dh][dh], perm [d] int32): column j of R is column perm[j] of
    the block-diagonal matrix.
    """
    lams = np.asarray(lams, np.float64)
    flat = lams.reshape(-1)
    perm = np.argsort(-flat, kind="stable").astype(np.int32)
    return np.ascontiguousarray(Vs, np.float64), perm


def assemble_headwise_rotation_per_head(lams, Vs, per_head=32):
    """The paper's own W_O layout (weight-splitting appendix): each head keeps its `per_head` largest-eigenvalue
    directions salient.  lams [H][dh] descending per head.  Column j of R is column perm[j] of
    blockdiag(V_1..V_H): the salient directions of head 0, 1, ... first, then every head's remaining ones.
    Returns (Rb, perm, K = H * per_head)."""
    lams = np.asarray(lams, np.float64)
    H, dh = lams.shape
    assert np.all(np.diff(lams, axis=1) <= 0)
    perm = [h * dh + i for h in range(H) for i in range(per_head)]
    perm += [h * dh + i for h in range(H) for i in range(per_head, dh)]
    return np.ascontiguousarray(Vs, np.float64), np.asarray(perm, np.int32), H * per_head


def selection_order(lam, k_salient, mode, rng=None):
    """Salient-selection ablation: the column order that puts the chosen k_salient directions first.  lam is
    the descending eigenvalue vector (only its length and order are used)."""
    d = len(lam)
    order = list(range(d))
    if mode == "top":
        sel = order[:k_salient]
    elif mode == "bottom":
        sel = order[d - k_salient:]
    elif mode == "random":
        sel = sorted(rng.choice(d, size=k_salient, replace=False).tolist())
    elif mode == "top_bottom":
        sel = order[:k_salient // 2] + order[d - (k_salient - k_salient // 2):]
    else:
        raise ValueError(mode)
    chosen = set(sel)
    return np.asarray(sel + [i for i in order if i not in chosen], np.int32)


def dense_from_blocks(Rb, perm=None):
    """The d x d matrix R that (Rb, perm) stands for."""
    Rb = np.asarray(Rb)
    if Rb.ndim == 2:
        Rb = Rb[None]
    H, dh, _ = Rb.shape
    R = np.zeros((H * dh, H * dh), Rb.dtype)
    for h in range(H):
        R[h * dh:(h + 1) * dh, h * dh:(h + 1) * dh] = Rb[h]
    return R if perm is None else R[:, np.asarray(perm)]


# ---------------------------------------------------------------- Eq. 1 / Eq. 3
def _blocks(Rb, dt):
    Rb = _c(Rb, dt)
    if Rb.ndim == 2:
        Rb = Rb[None]
    return Rb


def rotate_weights_f64(Rb, W, perm=None, cols=None):
    """W' = R^T W in fp64 on the listed output columns (default: all)."""
    Rb = _blocks(Rb, np.float64)
    W64 = f16_to_f64(W) if np.asarray(W).dtype == np.float16 else _c(W, np.float64)
    d_in, d_out = W64.shape
    cols = np.arange(d_out, dtype=np.int32) if cols is None else _c(cols, np.int32)
    perm = None if perm is None else _c(perm, np.int32)
    out = np.empty((d_in, cols.size), np.float64)
    _L().oracle_rotate_weights_f64(_p(Rb), C.c_int(d_in), C.c_int(Rb.shape[0]), _p(perm), _p(W64),
                                   C.c_int(d_out), _p(cols), C.c_int(cols.size), _p(out))
    return out


def rotate_weights_f32(Rb32, W, perm=None, cols=None):
    """The canonical fp32 fused-multiply-add chain (k ascending) that defines the codes.
    W is the binary16 weight, or an fp32 array (the scaled weight D W of scale_rows_f32)."""
    Rb = _blocks(Rb32, np.float32)
    w32 = np.asarray(W).dtype == np.float32
    W = _c(W, np.float32 if w32 else np.float16)
    d_in, d_out = W.shape
    cols = np.arange(d_out, dtype=np.int32) if cols is None else _c(cols, np.int32)
    perm = None if perm is None else _c(perm, np.int32)
    out = np.empty((d_in, cols.size), np.float32)
    fn = _L().oracle_rotate_weights_f32_w32 if w32 else _L().oracle_rotate_weights_f32
    fn(_p(Rb), C.c_int(d_in), C.c_int(Rb.shape[0]), _p(perm), _p(W if w32 else W.view(np.uint16)), C.c_int(d_out),
       _p(cols), C.c_int(cols.size), _p(out))
    return out


def scale_rows_f64(W, d):
    """D W in fp64 (scaling invariance: X W = (X D^-1)(D W))."""
    W64 = f16_to_f64(W) if np.asarray(W).dtype == np.float16 else _c(W, np.float64)
    d = _c(d, np.float64)
    out = np.empty(W64.shape, np.float64)
    _L().oracle_scale_rows_f64(_p(W64), C.c_int(W64.shape[0]), C.c_int(W64.shape[1]), _p(d), _p(out))
    return out


def scale_rows_f32(W16, d32):
    """D W in fp32, one rounding per product: the weight the scaled variant quantizes."""
    W16 = _c(W16, np.float16)
    d = _c(d32, np.float32)
    out = np.empty(W16.shape, np.float32)
    _L().oracle_scale_rows_f32(_p(W16.view(np.uint16)), C.c_int(W16.shape[0]), C.c_int(W16.shape[1]), _p(d), _p(out))
    return out


def quantize(Wp32, bits, group=128, k_salient=128):
    """Mixed-precision split of W' (fp32 [d_in][n]): dict of salient (f16), scales (f16),
    zeros (f16), codes (uint8 [d_in-K][n])."""
    Wp = _c(Wp32, np.float32)
    d_in, n = Wp.shape
    ng = (d_in - k_salient) // group
    sal = np.empty((k_salient, n), np.uint16)
    sc = np.empty((ng, n), np.uint16)
    zr = np.empty((ng, n), np.uint16)
    codes = np.empty((d_in - k_salient, n), np.uint8)
    _L().oracle_quantize(_p(Wp), C.c_int(d_in), C.c_int(n), C.c_int(bits), C.c_int(group),
                         C.c_int(k_salient), _p(sal), _p(sc), _p(zr), _p(codes))
    return dict(salient=sal.view(np.float16), scales=sc.view(np.float16), zeros=zr.view(np.float16),
                codes=codes, bits=bits, group=group, k_salient=k_salient)


def pack(codes, bits):
    codes = _c(codes, np.uint8)
    r, n = codes.shape
    nw = r // 8 if bits == 4 else r // 32 * 3
    qw = np.empty((nw, n), np.uint32)
    _L().oracle_pack(_p(codes), C.c_int(r), C.c_int(n), C.c_int(bits), _p(qw))
    return qw


def unpack(qw, n_rows, bits):
    qw = _c(qw, np.uint32)
    n = qw.shape[1]
    codes = np.empty((n_rows, n), np.uint8)
    _L().oracle_unpack(_p(qw), C.c_int(n_rows), C.c_int(n), C.c_int(bits), _p(codes))
    return codes


def forward(x16, qd, Rb16=None, perm=None, return_xrot=False):
    """y_ref (fp64) = (x . R) . W^ for the quantized dict `qd` (Eq. 3 / Eq. 6).

    x16 and Rb16 are binary16 arrays (what the GPU path is fed); they are widened
    exactly and nothing is rounded afterwards.  fp64 arrays are taken as they are
    (used by the identity checks)."""
    x = _c(x16, np.float64) if np.asarray(x16).dtype == np.float64 else f16_to_f64(_c(x16, np.float16))
    M, d_in = x.shape
    Rb = None
    nb = 1
    if Rb16 is not None:
        Rb = (_blocks(Rb16, np.float64) if np.asarray(Rb16).dtype == np.float64
              else f16_to_f64(_blocks(Rb16, np.float16)))
        nb = Rb.shape[0]
    perm = None if perm is None else _c(perm, np.int32)
    n = qd["codes"].shape[1] if qd["codes"].size else qd["salient"].shape[1]
    y = np.empty((M, n), np.float64)
    xr = np.empty((M, d_in), np.float64) if return_xrot else None
    sal = _c(qd["salient"], np.float16).view(np.uint16)
    sc = _c(qd["scales"], np.float16).view(np.uint16)
    zr = _c(qd["zeros"], np.float16).view(np.uint16)
    codes = _c(qd["codes"], np.uint8)
    _L().oracle_forward(_p(x), C.c_int(M), C.c_int(d_in), _p(Rb), C.c_int(nb), _p(perm), _p(sal),
                        _p(sc), _p(zr), _p(codes), C.c_int(qd["bits"]), C.c_int(qd["group"]),
                        C.c_int(qd["k_salient"]), C.c_int(n), _p(y), _p(xr))
    return (y, xr) if return_xrot else y


def dequantize(qd):
    """W^ in fp64: salient rows as stored, the rest (code - zero) * scale (exact)."""
    sal = f16_to_f64(qd["salient"])
    g = qd["group"]
    s = np.repeat(f16_to_f64(qd["scales"]), g, axis=0)
    z = np.repeat(f16_to_f64(qd["zeros"]), g, axis=0)
    return np.concatenate([sal, (qd["codes"].astype(np.float64) - z) * s], axis=0)
