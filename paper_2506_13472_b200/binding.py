"""Thin ctypes binding of librosaq.so: argument marshalling only.

Every function has the name of the C entry point it calls (see include/rosaq.h) and
takes torch CUDA tensors for the device pointers.  Nothing is computed here; if the
library is missing or a call fails, a RosaqError is raised -- there is no fallback.
"""
import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "librosaq.so")

ROSAQ_F16, ROSAQ_F32 = 0, 1
ROSAQ_OK = 0
ROSAQ_ERR_INVALID_ARG, ROSAQ_ERR_UNSUPPORTED_SHAPE, ROSAQ_ERR_ALIGNMENT = -1, -2, -3
ROSAQ_ERR_ALLOC, ROSAQ_ERR_CUDA, ROSAQ_ERR_TIMEOUT, ROSAQ_ERR_UNSUPPORTED_ARCH = -4, -5, -6, -7

EXPORTS = [
    "rosaq_create", "rosaq_destroy", "rosaq_strerror", "rosaq_last_status", "rosaq_set_wait_limit",
    "rosaq_set_linear_impl", "rosaq_calib_cov", "rosaq_quantize", "rosaq_quantize_scaled", "rosaq_weight_export",
    "rosaq_weight_import", "rosaq_weight_free", "rosaq_weight_info", "rosaq_rotation_create",
    "rosaq_rotation_free", "rosaq_rotate", "rosaq_linear", "rosaq_linear_multi", "rosaq_linear_static",
    "rosaq_plan_equal_shares", "rosaq_plan_create", "rosaq_plan_run", "rosaq_plan_free", "rosaq_plan_ctas",
    "rosaq_plan_schedule", "rosaq_set_plan_costs", "rosaq_set_plan_pairs",
]


class RosaqError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        super().__init__(f"{where}: {strerror(status)} ({status})")


class _Rot(C.Structure):
    _fields_ = [("d", C.c_int32), ("n_blocks", C.c_int32), ("q", C.c_void_p), ("q_dtype", C.c_int32),
                ("perm", C.c_void_p)]


class _Op(C.Structure):
    _fields_ = [("x", C.c_void_p), ("ldx", C.c_int64), ("x_from", C.c_int32), ("r", C.c_void_p), ("w", C.c_void_p),
                ("y", C.c_void_p), ("ldy", C.c_int64)]


_lib = None


def lib():
    """Loads librosaq.so (no build here: run paper_2506_13472_b200/build.py or __graft_entry__.build())."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} not built; run `python -m paper_2506_13472_b200.build`")
        L = C.CDLL(LIB_PATH)
        L.rosaq_strerror.restype = C.c_char_p
        L.rosaq_strerror.argtypes = [C.c_int]
        L.rosaq_set_wait_limit.restype = C.c_int64
        L.rosaq_set_wait_limit.argtypes = [C.c_void_p, C.c_int64]
        L.rosaq_set_linear_impl.argtypes = [C.c_void_p, C.c_int]
        L.rosaq_create.argtypes = [C.POINTER(C.c_void_p), C.c_int]
        L.rosaq_destroy.argtypes = [C.c_void_p]
        L.rosaq_last_status.argtypes = [C.c_void_p, C.c_void_p]
        L.rosaq_calib_cov.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int64, C.c_int, C.c_int64, C.c_int,
                                      C.c_void_p, C.c_void_p]
        L.rosaq_quantize.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.POINTER(_Rot), C.c_int, C.c_int,
                                     C.c_int, C.POINTER(C.c_void_p), C.c_void_p]
        L.rosaq_quantize_scaled.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.POINTER(_Rot), C.c_void_p, C.c_int,
                                            C.c_int, C.c_int, C.POINTER(C.c_void_p), C.c_void_p]
        L.rosaq_weight_export.argtypes = [C.c_void_p] * 7
        L.rosaq_weight_import.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_void_p,
                                          C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(C.c_void_p), C.c_void_p]
        L.rosaq_weight_free.argtypes = [C.c_void_p]
        L.rosaq_weight_info.argtypes = [C.c_void_p] + [C.POINTER(C.c_int)] * 5 + [C.POINTER(C.c_int64)]
        L.rosaq_rotation_create.argtypes = [C.c_void_p, C.POINTER(_Rot), C.POINTER(C.c_void_p), C.c_void_p]
        L.rosaq_rotation_free.argtypes = [C.c_void_p]
        L.rosaq_rotate.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int64, C.c_void_p, C.c_void_p, C.c_int64,
                                   C.c_void_p]
        L.rosaq_linear.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p,
                                   C.c_int64, C.c_void_p]
        L.rosaq_linear_static.argtypes = L.rosaq_linear.argtypes
        L.rosaq_linear_multi.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int64, C.c_void_p, C.c_int, C.c_void_p,
                                         C.c_void_p, C.c_void_p, C.c_void_p]
        L.rosaq_plan_equal_shares.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int, C.POINTER(C.c_int32)]
        L.rosaq_plan_create.argtypes = [C.c_void_p, C.c_int, C.c_int, C.POINTER(_Op), C.POINTER(C.c_void_p)]
        L.rosaq_plan_run.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
        L.rosaq_plan_free.argtypes = [C.c_void_p]
        L.rosaq_plan_ctas.argtypes = [C.c_void_p]
        L.rosaq_set_plan_costs.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int]
        L.rosaq_set_plan_pairs.argtypes = [C.c_void_p, C.c_int]
        L.rosaq_plan_schedule.argtypes = [C.c_int] + [C.POINTER(C.c_int32)] * 5 + [C.c_int, C.POINTER(C.c_int32),
                                                                                  C.POINTER(C.c_int32), C.c_int]
        _lib = L
    return _lib


def strerror(status):
    return lib().rosaq_strerror(int(status)).decode()


def _check(status, where):
    if status != ROSAQ_OK:
        raise RosaqError(status, where)


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _dt(t):
    if t.dtype == torch.float16:
        return ROSAQ_F16
    if t.dtype == torch.float32:
        return ROSAQ_F32
    raise TypeError(f"unsupported dtype {t.dtype}")


def _rot_struct(q, perm):
    """q: [d][d] or [n_blocks][dh][dh] CUDA tensor; perm: int32 [d] CUDA tensor or None."""
    assert q.is_cuda and q.is_contiguous()
    nb = 1 if q.dim() == 2 else q.shape[0]
    dh = q.shape[-1]
    assert q.shape[-2] == dh
    if perm is not None:
        assert perm.is_cuda and perm.dtype == torch.int32 and perm.is_contiguous() and perm.numel() == nb * dh
    return _Rot(nb * dh, nb, q.data_ptr(), _dt(q), None if perm is None else perm.data_ptr())


def plan_equal_shares(n_tiles, groups, g_fp16, n_ctas):
    """rosaq_plan_equal_shares: the n_ctas + 1 bounds of the equal-share cut (host only), or RosaqError."""
    out = (C.c_int32 * (max(n_ctas, 0) + 1))()
    _check(lib().rosaq_plan_equal_shares(n_tiles, groups, g_fp16, n_ctas, out), "rosaq_plan_equal_shares")
    return list(out)


PIECE_FIELDS = ("op", "tile", "g_begin", "g_end", "holders", "holder_idx", "slot0", "counter", "closer_idx", "closers",
                "tok_begin", "tok_end")


def plan_schedule(n_tiles, groups, g_fp16, x_from, n_ctas, copies=None):
    """rosaq_plan_schedule (host only): (piece_begin, pieces) with pieces a list of dicts keyed by PIECE_FIELDS."""
    n = len(n_tiles)
    arr = lambda v: (C.c_int32 * n)(*[int(a) for a in v])
    begin = (C.c_int32 * (n_ctas + 1))()
    args = (n, arr(n_tiles), arr(groups), arr(g_fp16), arr(x_from), None if copies is None else arr(copies), n_ctas, begin)
    total = lib().rosaq_plan_schedule(*args, None, 0)
    if total < 0:
        raise RosaqError(total, "rosaq_plan_schedule")
    raw = (C.c_int32 * (12 * max(total, 1)))()
    total2 = lib().rosaq_plan_schedule(*args, raw, total)
    assert total2 == total
    pieces = [dict(zip(PIECE_FIELDS, raw[12 * k:12 * k + 12])) for k in range(total)]
    return list(begin), pieces


class Context:
    """rosaq_ctx wrapper.  Methods carry the C names without the prefix."""

    def __init__(self, device=0):
        h = C.c_void_p()
        _check(lib().rosaq_create(C.byref(h), int(device)), "rosaq_create")
        self._h = h
        self.device = int(device)

    def close(self):
        if self._h:
            lib().rosaq_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def last_status(self, stream=None):
        return lib().rosaq_last_status(self._h, _stream(stream))

    def set_wait_limit(self, iterations):
        return lib().rosaq_set_wait_limit(self._h, int(iterations))

    def set_linear_impl(self, impl):
        return lib().rosaq_set_linear_impl(self._h, int(impl))

    # -- Eq. 4
    def calib_cov(self, X, C_out, n_blocks=1, stream=None):
        """C_out (fp32, zeroed by the caller before the first chunk) += X^T X."""
        assert X.is_cuda and C_out.is_cuda and C_out.dtype == torch.float32 and C_out.is_contiguous()
        assert X.dim() == 2 and X.stride(1) == 1
        _check(lib().rosaq_calib_cov(self._h, _ptr(X), _dt(X), X.shape[0], X.shape[1], X.stride(0), n_blocks,
                                     _ptr(C_out), _stream(stream)), "rosaq_calib_cov")
        return C_out

    # -- Eq. 3
    def quantize(self, W, q=None, perm=None, bits=4, group=128, k_salient=128, stream=None, in_scale=None):
        """rosaq_quantize, or rosaq_quantize_scaled when in_scale (fp32 CUDA tensor [d_in]) is given."""
        assert W.is_cuda and W.dtype == torch.float16 and W.is_contiguous() and W.dim() == 2
        rot = None if q is None else _rot_struct(q, perm)
        h = C.c_void_p()
        if in_scale is None:
            _check(lib().rosaq_quantize(self._h, _ptr(W), W.shape[0], W.shape[1],
                                        None if rot is None else C.byref(rot), bits, group, k_salient, C.byref(h),
                                        _stream(stream)), "rosaq_quantize")
        else:
            assert in_scale.is_cuda and in_scale.dtype == torch.float32 and in_scale.numel() == W.shape[0]
            _check(lib().rosaq_quantize_scaled(self._h, _ptr(W), W.shape[0], W.shape[1],
                                               None if rot is None else C.byref(rot), _ptr(in_scale.contiguous()), bits, group,
                                               k_salient, C.byref(h), _stream(stream)), "rosaq_quantize_scaled")
        return Weight(self, h)

    def weight_import(self, d_in, d_out, bits, group, k_salient, qw, scales, zeros, salient, stream=None):
        h = C.c_void_p()
        _check(lib().rosaq_weight_import(self._h, d_in, d_out, bits, group, k_salient, _ptr(qw), _ptr(scales),
                                         _ptr(zeros), _ptr(salient), C.byref(h), _stream(stream)),
               "rosaq_weight_import")
        return Weight(self, h)

    def rotation_create(self, q, perm=None, stream=None):
        rot = _rot_struct(q, perm)
        h = C.c_void_p()
        _check(lib().rosaq_rotation_create(self._h, C.byref(rot), C.byref(h), _stream(stream)),
               "rosaq_rotation_create")
        return Rotation(self, h, rot.d)

    def rotate(self, x, rotation, out=None, stream=None):
        assert x.is_cuda and x.dtype == torch.float16 and x.dim() == 2 and x.stride(1) == 1
        if out is None:
            out = torch.empty((x.shape[0], rotation.d), dtype=torch.float16, device=x.device)
        _check(lib().rosaq_rotate(self._h, _ptr(x), x.shape[0], x.stride(0), rotation._h, _ptr(out), out.stride(0),
                                  _stream(stream)), "rosaq_rotate")
        return out

    def linear(self, x, weight, rotation=None, out=None, stream=None):
        assert x.is_cuda and x.dtype == torch.float16 and x.dim() == 2 and x.stride(1) == 1
        if out is None:
            out = torch.empty((x.shape[0], weight.d_out), dtype=torch.float16, device=x.device)
        _check(lib().rosaq_linear(self._h, _ptr(x), x.shape[0], x.stride(0),
                                  None if rotation is None else rotation._h, weight._h, _ptr(out), out.stride(0),
                                  _stream(stream)), "rosaq_linear")
        return out

    def linear_multi(self, x, weights, rotation=None, outs=None, stream=None):
        """rosaq_linear_multi: the linears `weights` (same d_in / bits / k_salient) applied to one x in one launch."""
        assert x.is_cuda and x.dtype == torch.float16 and x.dim() == 2 and x.stride(1) == 1
        n = len(weights)
        if outs is None:
            outs = [torch.empty((x.shape[0], w.d_out), dtype=torch.float16, device=x.device) for w in weights]
        wa = (C.c_void_p * n)(*[w._h.value for w in weights])
        ya = (C.c_void_p * n)(*[o.data_ptr() for o in outs])
        la = (C.c_int64 * n)(*[o.stride(0) for o in outs])
        _check(lib().rosaq_linear_multi(self._h, _ptr(x), x.shape[0], x.stride(0),
                                        None if rotation is None else rotation._h, n, wa, ya, la, _stream(stream)),
               "rosaq_linear_multi")
        return outs

    def set_plan_costs(self, fp16_group, quant_group, tile):
        _check(lib().rosaq_set_plan_costs(self._h, fp16_group, quant_group, tile), "rosaq_set_plan_costs")

    def set_plan_pairs(self, enable):
        return lib().rosaq_set_plan_pairs(self._h, 1 if enable else 0)

    def plan_ctas(self):
        n = lib().rosaq_plan_ctas(self._h)
        if n < 0:
            raise RosaqError(n, "rosaq_plan_ctas")
        return n

    def plan_create(self, M, ops):
        """rosaq_plan_create.  ops: list of (x, x_from, handle, y) with x a CUDA fp16 tensor [M][.] or None when
        x_from >= 0, handle a Rotation or a Weight, y the CUDA fp16 output tensor [M][.]."""
        arr = (_Op * len(ops))()
        keep = []
        for o, (x, x_from, handle, y) in zip(arr, ops):
            assert y.is_cuda and y.dtype == torch.float16 and y.dim() == 2 and y.stride(1) == 1 and y.shape[0] == M
            if x is not None:
                assert x.is_cuda and x.dtype == torch.float16 and x.dim() == 2 and x.stride(1) == 1 and x.shape[0] == M
            o.x, o.ldx = (None if x is None else x.data_ptr()), (0 if x is None else x.stride(0))
            o.x_from = -1 if x_from is None else int(x_from)
            o.r = handle._h if isinstance(handle, Rotation) else None
            o.w = handle._h if isinstance(handle, Weight) else None
            o.y, o.ldy = y.data_ptr(), y.stride(0)
            keep += [x, handle, y]
        h = C.c_void_p()
        _check(lib().rosaq_plan_create(self._h, int(M), len(ops), arr, C.byref(h)), "rosaq_plan_create")
        return Plan(self, h, keep)

    def linear_static(self, x, weight, rotation=None, out=None, stream=None):
        """rosaq_linear_static: same result as `linear`, but the library allocates nothing (the rotated
        activations live in a fixed 4 MiB array inside the library).  Pass `out`: with out=None this
        wrapper itself asks torch for the output tensor, which a caller that cannot allocate would not do."""
        assert x.is_cuda and x.dtype == torch.float16 and x.dim() == 2 and x.stride(1) == 1
        if out is None:
            out = torch.empty((x.shape[0], weight.d_out), dtype=torch.float16, device=x.device)
        _check(lib().rosaq_linear_static(self._h, _ptr(x), x.shape[0], x.stride(0),
                                         None if rotation is None else rotation._h, weight._h, _ptr(out),
                                         out.stride(0), _stream(stream)), "rosaq_linear_static")
        return out


class Weight:
    """rosaq_weight wrapper."""

    def __init__(self, ctx, handle):
        self._ctx, self._h = ctx, handle
        vals = [C.c_int() for _ in range(5)]
        nbytes = C.c_int64()
        _check(lib().rosaq_weight_info(handle, *[C.byref(v) for v in vals], C.byref(nbytes)), "rosaq_weight_info")
        self.d_in, self.d_out, self.bits, self.group, self.k_salient = [v.value for v in vals]
        self.device_bytes = nbytes.value

    def export(self, stream=None):
        """dict of torch tensors in the interchange layout: qw (int32 view of uint32), scales, zeros, salient."""
        dev = torch.device("cuda", self._ctx.device)
        nq = self.d_in - self.k_salient
        nw = nq // 8 if self.bits == 4 else nq // 32 * 3
        qw = torch.empty((nw, self.d_out), dtype=torch.int32, device=dev)
        sc = torch.empty((nq // self.group, self.d_out), dtype=torch.float16, device=dev)
        zr = torch.empty_like(sc)
        sal = torch.empty((self.k_salient, self.d_out), dtype=torch.float16, device=dev)
        _check(lib().rosaq_weight_export(self._ctx._h, self._h, _ptr(qw), _ptr(sc), _ptr(zr), _ptr(sal),
                                         _stream(stream)), "rosaq_weight_export")
        return dict(qw=qw, scales=sc, zeros=zr, salient=sal)

    def free(self):
        if self._h:
            lib().rosaq_weight_free(self._h)
            self._h = None

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass


class Plan:
    """rosaq_plan wrapper; keeps the tensors and handles of its operations alive."""

    def __init__(self, ctx, handle, keep):
        self._ctx, self._h, self._keep = ctx, handle, keep

    def run(self, stream=None):
        _check(lib().rosaq_plan_run(self._ctx._h, self._h, _stream(stream)), "rosaq_plan_run")

    def free(self):
        if self._h:
            lib().rosaq_plan_free(self._h)
            self._h = None

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass


class Rotation:
    """rosaq_rotation wrapper."""

    def __init__(self, ctx, handle, d):
        self._ctx, self._h, self.d = ctx, handle, d

    def free(self):
        if self._h:
            lib().rosaq_rotation_free(self._h)
            self._h = None

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass
