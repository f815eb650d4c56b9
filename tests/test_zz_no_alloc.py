"""fasttps_mlp_decode_static: the fused MLP with its scratch in the library's fixed device array.

Collected last (file name), so that it also runs after every other GPU test has used the ordinary entry
points; it must pass alone as well.  Each case makes two calls in a row through the C ABI -- the second
with other inputs, so that anything left behind in the array by the first would show -- and compares
each with the existing entry point (same kernel, workspace scratch) and with the oracle.
"""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2607_11211_b200 import workload as wl
from tests.helpers import assert_close_bits, from_bf16_bits as F32, ulp_distance

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def fb():
    from paper_2607_11211_b200 import binding, build
    build.build()
    return binding


def inputs(dims, batch, seed):
    w = wl.layer_weights(dims, seed, device="cuda")
    x = wl.activations(dims, batch, seed=seed, device="cuda")["x"]
    wgu = (w["w_gu"].float() * 4).to(torch.bfloat16)
    wdn = (w["w_down"].float() * 4).to(torch.bfloat16)
    return x, wgu, wdn


@pytest.mark.parametrize("dims,batch", [(wl.TINY, 1), (wl.SMALL, 3), (wl.SMALL_GQA, 8), (wl.PHI3_MINI, 2)])
def test_static_scratch_matches_workspace_entry_point_twice_in_a_row(fb, dims, batch):
    ctx = fb.Context.from_dims(dims, batch, 64)
    for call, seed in enumerate((1, 2)):
        x, wgu, wdn = inputs(dims, batch, seed)
        pg, pd = ctx.pack_weight(fb.W_GATE_UP, wgu), ctx.pack_weight(fb.W_DOWN, wdn)
        got = torch.full((batch, dims.hidden), 3.0, dtype=torch.bfloat16, device="cuda")
        ref = torch.full((batch, dims.hidden), -3.0, dtype=torch.bfloat16, device="cuda")
        ctx.mlp_decode_static(x, pg, pd, got)
        ctx.mlp_decode(x, pg, pd, ref)
        assert ctx.get_status() == 0
        # same kernel, same data; only the order of the FP32 atomic additions may differ between two launches
        near = (ulp_distance(wl.bits(got), wl.bits(ref)) <= 1) | (np.abs(F32(wl.bits(got)) - F32(wl.bits(ref))) <= 1e-4)
        assert near.all(), f"call {call}"
        assert_close_bits(wl.bits(got), orc.mlp_decode(wl.bits(x), wl.bits(wgu), wl.bits(wdn)), what=f"static mlp, call {call}")
    ctx.close()


def test_static_scratch_rejects_what_does_not_fit(fb):
    dims = wl.SMALL
    ctx = fb.Context.from_dims(dims, 16, 64)
    x, wgu, wdn = inputs(dims, 9, 1)
    pg, pd = ctx.pack_weight(fb.W_GATE_UP, wgu), ctx.pack_weight(fb.W_DOWN, wdn)
    out = torch.zeros(9, dims.hidden, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(fb.FasttpsError, match="static scratch"):
        ctx.mlp_decode_static(x, pg, pd, out)
    assert (out == 0).all()
    ctx.mlp_decode(x, pg, pd, out)                      # the workspace entry point serves the same request
    assert ctx.get_status() == 0
    ctx.close()
