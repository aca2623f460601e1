"""Host-side step between rosaq_calib_cov and rosaq_quantize: C = R Lambda R^T (Eq. 4).

The eigensolve is deliberately outside the C ABI (R is an input of the device calls);
this helper is what the benchmark and a user of the library call to get R from the
Gram matrix that rosaq_calib_cov produced.  LAPACK (through numpy) in fp64.
"""
import numpy as np


def eigh_descending(Cm):
    """(lambda, R): eigenvalues in descending order (Section 3.2: the largest are the salient
    ones), R[:, j] the unit eigenvector of lambda[j], sign chosen so that its largest-magnitude
    entry is positive (eigenvectors are only defined up to sign)."""
    Cm = np.asarray(Cm, dtype=np.float64)
    Cm = 0.5 * (Cm + Cm.T)
    lam, V = np.linalg.eigh(Cm)
    order = np.argsort(-lam, kind="stable")
    lam, V = lam[order], V[:, order]
    big = np.argmax(np.abs(V), axis=0)
    sgn = np.sign(V[big, np.arange(V.shape[1])])
    sgn[sgn == 0] = 1.0
    return lam, np.ascontiguousarray(V * sgn[None, :])


def headwise_rotation(C_blocks):
    """Head-wise PCA (Section 3.1.1, Eq. 6): one eigendecomposition per head block plus the
    global column order by descending eigenvalue, so that the first K columns of
    R = blockdiag(R_1..R_H)[:, perm] are the K most principal directions over all heads.
    Returns (Rb [H][dh][dh] fp64, perm [H*dh] int32, lambdas [H][dh])."""
    lams, Rs = zip(*[eigh_descending(Cb) for Cb in np.asarray(C_blocks)])
    lams = np.asarray(lams)
    perm = np.argsort(-lams.reshape(-1), kind="stable").astype(np.int32)
    return np.ascontiguousarray(Rs), perm, lams


def eigh_descending_device(C_dev):
    """Same contract as eigh_descending, computed in fp64 on the device the Gram matrix lives on
    (a library eigensolver; used when d is in the thousands).  Returns a torch fp64 tensor R."""
    import torch
    Cm = C_dev.to(torch.float64)
    Cm = 0.5 * (Cm + Cm.T)
    lam, V = torch.linalg.eigh(Cm)
    order = torch.argsort(lam, descending=True, stable=True)
    V = V[:, order]
    big = torch.argmax(V.abs(), dim=0)
    sgn = torch.sign(V[big, torch.arange(V.shape[1], device=V.device)])
    sgn[sgn == 0] = 1.0
    return (V * sgn[None, :]).contiguous()


def channel_scale(X, alpha=0.5):
    """Diagonal D for the scaled (AWQ-style) quantization of an un-rotated linear such as the down
    projection (weight-splitting appendix; scaling invariance X W = (X D^-1)(D W)).  The paper prints no rule
    for D; this is the fixed one used here: d_i = (mean_t |x_ti|)^alpha, divided by sqrt(max d * min d) so that
    the scales straddle 1.  Channels that are always zero get d_i = 1.  Returns fp32 [d]."""
    m = np.abs(np.asarray(X, dtype=np.float64)).mean(axis=0)
    d = np.where(m > 0, m, 1.0) ** float(alpha)
    d = d / np.sqrt(d.max() * d.min())
    d[m <= 0] = 1.0
    return d.astype(np.float32)


def headwise_rotation_per_head_salient(C_blocks, per_head=32):
    """Head-wise PCA with the paper's own W_O layout (weight-splitting appendix): every head keeps its
    `per_head` most principal directions in FP16, so K = H * per_head salient channels in all.  Column order
    of R = blockdiag(R_1..R_H)[:, perm]: first the top `per_head` directions of head 0, of head 1, ...,
    then the remaining directions head by head, each head's in descending eigenvalue order; the quantization
    groups (128 channels) run over that concatenation.  Returns (Rb [H][dh][dh] fp64, perm int32, K)."""
    lams, Rs = zip(*[eigh_descending(Cb) for Cb in np.asarray(C_blocks)])
    H, dh = len(Rs), Rs[0].shape[0]
    base = np.arange(H)[:, None] * dh
    top = (base + np.arange(per_head)[None, :]).reshape(-1)
    rest = (base + np.arange(per_head, dh)[None, :]).reshape(-1)
    return np.ascontiguousarray(Rs), np.concatenate([top, rest]).astype(np.int32), H * per_head


def selection_order(d, k_salient, mode, seed=0):
    """Column orders for the salient-selection ablation (appendix on selecting salient channels): given
    eigenvectors already in descending eigenvalue order, the permutation whose first k_salient columns are the
    chosen ones -- 'top' (the method), 'bottom', 'random', 'top_bottom' (half from each end) -- followed by
    the others in descending order.  Pass it as `perm` next to the dense R (n_blocks = 1)."""
    idx = np.arange(d)
    if mode == "top":
        sel = idx[:k_salient]
    elif mode == "bottom":
        sel = idx[d - k_salient:]
    elif mode == "random":
        sel = np.sort(np.random.Generator(np.random.PCG64(seed)).choice(d, size=k_salient, replace=False))
    elif mode == "top_bottom":
        sel = np.concatenate([idx[:k_salient // 2], idx[d - (k_salient - k_salient // 2):]])
    else:
        raise ValueError(mode)
    mask = np.ones(d, bool)
    mask[sel] = False
    return np.concatenate([sel, idx[mask]]).astype(np.int32)
