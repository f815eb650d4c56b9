"""The non-fused comparison arm (Algorithm 1 and Algorithm 2 as one kernel per operator, with a Concat of the whole
cache into a new buffer) computes the same attention and the same MLP as the fused path: checked against the same
oracle under the same output bar.  Its caches come out of the Concat: rows 0 .. L_b of every head, the last one
the rotated new key / the new value; the caller's caches are left untouched."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2607_11211_b200 import workload as wl
from tests.helpers import assert_close_bits, ulp_distance

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def fb():
    from paper_2607_11211_b200 import binding, build
    build.build()
    return binding


@pytest.mark.parametrize("dims,lens", [(wl.TINY, [0, 5, 63]), (wl.SMALL_GQA, [9, 200]), (wl.PHI3_MINI, [256]),
                                       (wl.PHI3_MINI, [1000, 17, 4095])])
def test_non_fused_attention_matches_the_oracle(fb, dims, lens):
    B, max_seq = len(lens), 4096
    lens = np.asarray(lens, np.int32)
    cat_seq = int(lens.max()) + 1
    act = wl.activations(dims, B, device="cuda")
    kc, vc = wl.kv_cache(dims, 0, B, max_seq, device="cuda")
    k0, v0 = wl.bits(kc), wl.bits(vc)
    out = torch.zeros(B, dims.n_q_heads, dims.head_dim, dtype=torch.bfloat16, device="cuda")
    L = torch.tensor(lens, device="cuda")
    k_cat, v_cat, us = fb.baseline_attn(act["q"], act["k_new"], act["v_new"], kc, vc, L, L, out, cat_seq, dims.rope_theta, timed=True)
    torch.cuda.synchronize()
    assert len(us) == 10 and all(u > 0 for u in us)
    assert (wl.bits(kc) == k0).all() and (wl.bits(vc) == v0).all()          # Concat writes NEW buffers
    ko, vo = k0.copy(), v0.copy()
    want = orc.attn_decode(wl.bits(act["q"]), wl.bits(act["k_new"]), wl.bits(act["v_new"]), ko, vo, lens, lens, dims.rope_theta)
    assert_close_bits(wl.bits(out), want, what="non-fused attention output")
    kg, vg = wl.bits(k_cat), wl.bits(v_cat)
    for b in range(B):
        n = int(lens[b]) + 1
        assert (kg[b, :, :n - 1] == k0[b, :, :n - 1]).all() and (vg[b, :, :n - 1] == v0[b, :, :n - 1]).all()
        assert ulp_distance(kg[b, :, n - 1], ko[b, :, n - 1]).max() <= 1
        assert (vg[b, :, n - 1] == vo[b, :, n - 1]).all()


@pytest.mark.parametrize("dims,batch", [(wl.TINY, 3), (wl.SMALL, 9), (wl.PHI3_MINI, 1), (wl.PHI3_MINI, 8)])
def test_non_fused_mlp_matches_the_oracle(fb, dims, batch):
    w = wl.layer_weights(dims, 0, device="cuda")
    x = wl.activations(dims, batch, device="cuda")["x"]
    K = dims.inter
    wt_gate = w["w_gu"][:, :K].t().contiguous()
    wt_up = w["w_gu"][:, K:].t().contiguous()
    wt_down = w["w_down"].t().contiguous()
    out = torch.zeros_like(x)
    us = fb.baseline_mlp(x, wt_gate, wt_up, wt_down, out, timed=True)
    torch.cuda.synchronize()
    assert len(us) == 5 and all(u > 0 for u in us)
    want = orc.mlp_decode(wl.bits(x), wl.bits(w["w_gu"]), wl.bits(w["w_down"]))
    assert_close_bits(wl.bits(out), want, what="non-fused MLP output")
