"""rosaq_linear_static: the rotated linear for callers that cannot allocate device memory.

Some users of the library run where cudaMalloc is off limits -- a server whose memory pool owns the
whole device, a loop that cannot afford an allocation's device-wide synchronisation -- so the library
offers a variant of rosaq_linear that keeps the rotated activations in a fixed array of its own
instead of a workspace it would have to allocate.  This file checks, through the C ABI, that the
variant returns what rosaq_linear returns, twice in a row (the array is shared between calls and
keeps the previous call's contents), and that it refuses a call that does not fit the array.

Collected last on purpose (file name), so a run that stops at the first failure has already run
every other test.  It does not depend on anything the other tests leave behind.
"""
import numpy as np
import pytest
import torch

from oracle import rosaq_oracle as orc
from paper_2506_13472_b200 import binding as rb
from paper_2506_13472_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu

STATIC_SCRATCH_BYTES = 4 << 20


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def test_static_variant_matches_rosaq_linear_on_two_calls_in_a_row():
    ctx = rb.Context(0)
    try:
        c = H.config_headwise()                     # block-diagonal R with a permutation, d_in = 512
        w = ctx.quantize(dev(c["W"]), dev(c["Rb32"]), dev(c["perm"]), bits=4, k_salient=128)
        qd = H.oracle_quantized(c["W"], c["Rb32"], c["perm"], 4, 128)
        rot = ctx.rotation_create(dev(c["Rb16"]), dev(c["perm"]))
        law = synth.HeadwiseActivationLaw(c["heads"], c["head_dim"], 3, "hw")
        # first call: 37 tokens; second call: fewer tokens and other values, so stale rows of the
        # shared array from the first call would show up if they were read
        for M, tag in ((37, "static-a"), (5, "static-b")):
            x16 = law.sample(M, tag, np.float16)
            x = dev(x16)
            want = ctx.linear(x, w, rot)
            got = torch.full((M, w.d_out), float("nan"), dtype=torch.float16, device="cuda")
            ctx.linear_static(x, w, rot, out=got)
            assert ctx.last_status() == rb.ROSAQ_OK
            want, got = want.cpu().numpy(), got.cpu().numpy()
            assert np.all(np.isfinite(got))
            assert H.rel_fro(got, want) <= H.REL_TOL_Y
            assert H.rel_fro(got, want) <= 2e-4          # the same sums, up to the order the K splits are added in
            # and on its own feet: the CPU oracle's fp64 forward on the same inputs
            assert H.rel_fro(got, orc.forward(x16, qd, c["Rb16"], c["perm"])) <= H.REL_TOL_Y
        # r == NULL needs no scratch: plain GEMM stage on pre-rotated input
        xr = ctx.rotate(dev(law.sample(9, "static-c", np.float16)), rot)
        a = ctx.linear(xr, w, None).cpu().numpy()
        b = ctx.linear_static(xr, w, None, out=torch.empty((9, w.d_out), dtype=torch.float16, device="cuda"))
        assert H.rel_fro(b.cpu().numpy(), a) <= 2e-4
    finally:
        ctx.close()


def test_static_variant_rejects_what_does_not_fit_its_array():
    ctx = rb.Context(0)
    try:
        d = 256
        R = torch.eye(d, dtype=torch.float16, device="cuda")
        rot = ctx.rotation_create(R)
        w = ctx.quantize(torch.zeros((d, 128), dtype=torch.float16, device="cuda"), None, bits=4, k_salient=128)
        M_fit = STATIC_SCRATCH_BYTES // (2 * d)
        y = torch.empty((M_fit + 1, 128), dtype=torch.float16, device="cuda")
        x = torch.zeros((M_fit + 1, d), dtype=torch.float16, device="cuda")
        ctx.linear_static(x[:M_fit], w, rot, out=y[:M_fit])              # exactly at the limit: accepted
        with pytest.raises(rb.RosaqError) as e:
            ctx.linear_static(x, w, rot, out=y)                          # one row more: refused, nothing launched
        assert e.value.status == rb.ROSAQ_ERR_UNSUPPORTED_SHAPE
        assert ctx.last_status() == rb.ROSAQ_OK
    finally:
        ctx.close()
