"""Seeded synthetic inputs shaped like the workloads of the ROSAQ paper.

Only random structure lives here -- no step of the method (no covariance, no
eigensolve, no rotation of weights, no quantizer).  Both the CPU oracle's tests
and the CUDA path's tests/benchmark draw their inputs from this module, so that the
two sides are always fed the same bits.

What stands in for what: the paper calibrates on text activations of LLaMA-family
models whose spectrum decays roughly like a power law with a few dominant
directions (its appendix table of activation magnitudes), and quantizes trained
weights that have a few large-magnitude input channels.  Here activations are
Gaussian with a power-law covariance spectrum mixed by a random orthogonal matrix,
and weights are Gaussian with a small fraction of amplified input rows.
Every tensor is rounded to its storage dtype when generated.
"""
import numpy as np

LLAMA_7B = dict(d=4096, ffn=11008, heads=32, head_dim=128)
LLAMA_13B = dict(d=5120, ffn=13824, heads=40, head_dim=128)


def layer_shapes(model):
    """(name, d_in, d_out, input-id) of the seven linears of one decoder layer; linears
    with the same input-id read the same activation and share one rotation."""
    d, f = model["d"], model["ffn"]
    return [("q", d, d, "attn_in"), ("k", d, d, "attn_in"), ("v", d, d, "attn_in"),
            ("o", d, d, "o_in"), ("gate", d, f, "mlp_in"), ("up", d, f, "mlp_in"),
            ("down", f, d, "down_in")]


def rng_for(seed, *key):
    """Independent stream per (seed, tensor key); keys are ints or short strings."""
    ints = [int.from_bytes(str(k).encode(), "little") % (2 ** 32) if not isinstance(k, int) else k
            for k in key]
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed] + ints)))


def orthogonal_qr(d, rng):
    """Haar-ish random orthogonal matrix: QR of a Gaussian matrix, R's diagonal made positive."""
    A = rng.standard_normal((d, d))
    Q, R = np.linalg.qr(A)
    return Q * np.sign(np.diag(R))[None, :]


def householder_vectors(d, count, rng):
    v = rng.standard_normal((count, d))
    return v / np.linalg.norm(v, axis=1, keepdims=True)


def apply_householders(Z, vs):
    """Z <- Z (I - 2 v v^T) for each v: an exactly orthogonal mix in O(d) per token."""
    for v in vs:
        Z = Z - 2.0 * np.outer(Z @ v, v)
    return Z


def power_law_spectrum(d, exponent):
    return np.arange(1, d + 1, dtype=np.float64) ** (-float(exponent))


class ActivationLaw:
    """x ~ N(0, U diag(lambda) U^T): lambda a power law, U a seeded orthogonal mix."""

    def __init__(self, d, exponent, seed, key, mix="householder", scale=1.0):
        rng = rng_for(seed, key, "law")
        self.d = d
        self.sqrt_lam = np.sqrt(power_law_spectrum(d, exponent)) * scale
        if mix == "qr":
            self.U = orthogonal_qr(d, rng)
            self.vs = None
        else:
            self.U = None
            self.vs = householder_vectors(d, 8, rng)
        self.seed, self.key = seed, key

    def sample(self, n_tokens, tag, dtype=np.float16):
        rng = rng_for(self.seed, self.key, tag)
        Z = rng.standard_normal((n_tokens, self.d)) * self.sqrt_lam[None, :]
        X = Z @ self.U.T if self.U is not None else apply_householders(Z, self.vs)
        return X.astype(dtype)

    def principal_directions(self):
        """Columns = the true covariance eigenvectors, in descending eigenvalue order."""
        if self.U is not None:
            return self.U
        return apply_householders(np.eye(self.d), self.vs).T


class HeadwiseActivationLaw:
    """Per-head independent laws (head_dim each) with per-head random exponents."""

    def __init__(self, heads, head_dim, seed, key, exp_lo=0.8, exp_hi=1.5):
        rng = rng_for(seed, key, "exponents")
        self.exponents = rng.uniform(exp_lo, exp_hi, size=heads)
        self.laws = [ActivationLaw(head_dim, self.exponents[h], seed, f"{key}/h{h}", mix="qr")
                     for h in range(heads)]
        self.heads, self.head_dim = heads, head_dim

    def sample(self, n_tokens, tag, dtype=np.float16):
        return np.concatenate([l.sample(n_tokens, tag, dtype) for l in self.laws], axis=1)


def weights(d_in, d_out, seed, key, sigma=0.02, outlier_rows=None, outlier_frac=0.0,
            outlier_scale=10.0, heavy_tail=False):
    """fp16 W [d_in][d_out] ~ N(0, sigma^2); a set of input rows is amplified by
    outlier_scale, or (heavy_tail) redrawn from Student-t(3) * sigma."""
    rng = rng_for(seed, key, "W")
    W = rng.standard_normal((d_in, d_out), dtype=np.float32) * np.float32(sigma)
    n_out = outlier_rows if outlier_rows is not None else int(round(outlier_frac * d_in))
    if n_out > 0:
        rows = rng.choice(d_in, size=n_out, replace=False)
        if heavy_tail:
            W[rows] = (rng.standard_t(3.0, size=(n_out, d_out)) * sigma).astype(np.float32)
        else:
            W[rows] *= np.float32(outlier_scale)
    return W.astype(np.float16)


def sample_columns(d_out, count, seed, key):
    """Sorted random output columns, always including the first, the last and a tile edge."""
    rng = rng_for(seed, key, "cols")
    must = {0, d_out - 1, min(127, d_out - 1), min(128, d_out - 1)}
    extra = rng.choice(d_out, size=min(count, d_out), replace=False).tolist()
    cols = sorted(must | set(extra))[: max(count, len(must))]
    return np.asarray(sorted(set(cols) | must), dtype=np.int32)
