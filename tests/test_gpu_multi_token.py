"""Several new tokens per sequence in one step (Algorithm 3 and Algorithm 4 for general N): the CUDA path against the
oracle.  Token j of a sequence is rotated at position pos + j, goes into cache row len + j and attends the cached rows
and the new tokens up to itself; exactly B * N * H_kv runs of d cache elements change, the rest bit for bit not."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2607_11211_b200 import workload as wl
from tests.helpers import assert_close_bits, ulp_distance, layer_output_ok, from_bf16_bits as F32

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def fb():
    from paper_2607_11211_b200 import binding, build
    build.build()
    return binding


def i32(a):
    return torch.tensor(np.asarray(a, dtype=np.int32), device="cuda")


def dev(bits):
    return wl.from_bits(bits, "cuda")


# share 1: the tokens of a chunk (times the query heads of a K/V head) go through one pass over the cache on the tensor
# cores while there are at most 16 of them, one pass per token and query head otherwise; share 0: always the latter.
@pytest.mark.parametrize("dims,lens,n_new,share", [
    (wl.TINY, [0], 2, 1), (wl.TINY, [5, 64, 17], 3, 1), (wl.SMALL, [100, 3], 8, 1), (wl.SMALL_GQA, [9, 200, 31], 4, 1),
    (wl.SMALL_GQA, [9, 200, 31], 3, 1), (wl.SMALL_GQA, [50, 6], 8, 1), (wl.PHI3_MINI, [1000, 17], 4, 1),
    (wl.PHI3_MINI, [4088], 8, 1), (wl.SMALL, [40, 7, 100], 1, 1), (wl.TINY, [5, 64, 17], 3, 0),
    (wl.SMALL_GQA, [9, 200, 31], 5, 0), (wl.PHI3_MINI, [1000, 17], 4, 0), (wl.PHI3_MINI, [4088], 7, 2)])
def test_attn_decode_multi_matches_oracle(fb, dims, lens, n_new, share):
    B, max_seq = len(lens), 4096 if dims is wl.PHI3_MINI else 256
    lens = np.asarray(lens, np.int32)
    pos = lens + 3 if dims is not wl.PHI3_MINI else lens          # the rotary position need not be the cache row
    ctx = fb.Context.from_dims(dims, B * n_new, max_seq)
    ctx.set_option("gqa_share", share)
    d, Hq, Hkv = dims.head_dim, dims.n_q_heads, dims.n_kv_heads
    rng = np.random.default_rng(11)
    mk = lambda *s: orc.f32_to_bf16(rng.standard_normal(s).astype(np.float32))
    q, kn, vn = mk(B, n_new, Hq, d), mk(B, n_new, Hkv, d), mk(B, n_new, Hkv, d)
    kc, vc = wl.kv_cache(dims, 0, B, max_seq, device="cuda")
    k0, v0 = wl.bits(kc), wl.bits(vc)
    out = torch.zeros(B, n_new, Hq, d, dtype=torch.bfloat16, device="cuda")
    ctx.attn_decode_multi(dev(q), dev(kn), dev(vn), kc, vc, i32(pos), i32(lens), out)
    torch.cuda.synchronize()
    assert ctx.get_status() == 0
    ko, vo = k0.copy(), v0.copy()
    want = orc.attn_decode_multi(q, kn, vn, ko, vo, pos, lens, dims.rope_theta)
    assert_close_bits(wl.bits(out), want, what=f"multi-token attention, N = {n_new}")
    kg, vg = wl.bits(kc), wl.bits(vc)
    mask = np.ones(kg.shape, bool)
    for b in range(B):
        mask[b, :, lens[b]:lens[b] + n_new] = False
    assert (kg[mask] == k0[mask]).all() and (vg[mask] == v0[mask]).all()       # nothing but the N new rows changed
    for b in range(B):
        rows = slice(int(lens[b]), int(lens[b]) + n_new)
        assert ulp_distance(kg[b, :, rows], ko[b, :, rows]).max() <= 1
        assert (vg[b, :, rows] == vo[b, :, rows]).all()
    if n_new == 1:      # one new token per sequence is the decode step itself, bit for bit
        kc1, vc1 = dev(k0), dev(v0)
        o1 = torch.zeros(B, Hq, d, dtype=torch.bfloat16, device="cuda")
        ctx.set_option("gqa_share", 0)
        ctx.attn_decode(dev(q[:, 0]), dev(kn[:, 0]), dev(vn[:, 0]), kc1, vc1, i32(pos), i32(lens), o1)
        assert (wl.bits(o1) == wl.bits(out)[:, 0]).all() and (wl.bits(kc1) == kg).all()
    ctx.close()


def test_attn_decode_multi_reports_a_chunk_that_does_not_fit(fb):
    dims, n_new, max_seq = wl.SMALL, 4, 64
    lens = np.array([61, 10], np.int32)                  # sequence 0: rows 61..64, row 64 does not exist
    ctx = fb.Context.from_dims(dims, 2 * n_new, max_seq)
    act = lambda h: wl.normal_bf16(3, 50 + h, (2, n_new, h, dims.head_dim), device="cuda")
    q, kn, vn = act(dims.n_q_heads), act(dims.n_kv_heads), act(dims.n_kv_heads)
    kc, vc = wl.kv_cache(dims, 0, 2, max_seq, device="cuda")
    k0 = wl.bits(kc)
    out = torch.zeros(2, n_new, dims.n_q_heads, dims.head_dim, dtype=torch.bfloat16, device="cuda")
    ctx.attn_decode_multi(q, kn, vn, kc, vc, i32(lens), i32(lens), out)
    torch.cuda.synchronize()
    assert ctx.get_status() & fb.DEV_CACHE_FULL
    assert (wl.bits(kc)[0] == k0[0]).all() and (wl.bits(out)[0] == 0).all()     # skipped: nothing written
    want = orc.attn_decode_multi(wl.bits(q), wl.bits(kn), wl.bits(vn), k0.copy(), wl.bits(vc).copy(), lens, lens)
    assert_close_bits(wl.bits(out)[1], want[1], what="the sequence that fits")
    ctx.close()


@pytest.mark.parametrize("dims,lens,n_new", [(wl.TINY, [5, 30], 2), (wl.SMALL, [100, 3, 250], 4), (wl.PHI3_MINI, [256], 8),
                                             (wl.PHI3_MINI, [700, 64, 5], 4)])
def test_layer_decode_multi_matches_oracle(fb, dims, lens, n_new):
    B, max_seq = len(lens), 1024
    lens = np.asarray(lens, np.int32)
    rows = B * n_new
    ctx = fb.Context.from_dims(dims, rows, max_seq)
    w = wl.layer_weights(dims, 0, device="cuda")
    pw = ctx.pack_layer(w)
    wb = {k: wl.bits(v) for k, v in w.items()}
    x = wl.normal_bf16(5, 77, (rows, dims.hidden), device="cuda")
    kc, vc = wl.kv_cache(dims, 0, B, max_seq, device="cuda")
    k0, v0 = wl.bits(kc), wl.bits(vc)
    xo = torch.zeros_like(x)
    ctx.layer_decode_multi(pw["struct"], x, xo, n_new, kc, vc, i32(lens), i32(lens))
    torch.cuda.synchronize()
    assert ctx.get_status() == 0
    ko, vo = k0.copy(), v0.copy()
    want = orc.layer_decode_multi(wb, wl.bits(x), n_new, ko, vo, lens, lens, dims.rms_eps, dims.rope_theta)
    # the residual stream before its rounding, from the oracle's primitives (see tests/helpers.py: layer_output_ok)
    nq, nkv, d = dims.n_q_heads * dims.head_dim, dims.n_kv_heads * dims.head_dim, dims.head_dim
    qkv = orc.f64_to_bf16(orc.gemv(orc.rmsnorm(wl.bits(x), wb["g_attn"], dims.rms_eps), wb["w_qkv"]))
    sp = lambda t, h: t.reshape(B, n_new, h, d)
    a = orc.attn_decode_multi(sp(qkv[:, :nq], dims.n_q_heads), sp(qkv[:, nq:nq + nkv], dims.n_kv_heads),
                              sp(qkv[:, nq + nkv:], dims.n_kv_heads), k0.copy(), v0.copy(), lens, lens, dims.rope_theta)
    h_exact = F32(wl.bits(x)).astype(np.float64) + orc.gemv(a.reshape(rows, nq), wb["w_o"])
    ok = layer_output_ok(wl.bits(xo), want, h_exact)
    assert ok.all(), int((~ok).sum())
    kg, vg = wl.bits(kc), wl.bits(vc)
    mask = np.ones(kg.shape, bool)
    for b in range(B):
        mask[b, :, lens[b]:lens[b] + n_new] = False
    assert (kg[mask] == k0[mask]).all() and (vg[mask] == v0[mask]).all()
    for b in range(B):
        r = slice(int(lens[b]), int(lens[b]) + n_new)
        assert_close_bits(kg[b, :, r], ko[b, :, r], what="appended k rows")     # k, v are outputs of the QKV block here
        assert_close_bits(vg[b, :, r], vo[b, :, r], what="appended v rows")
    ctx.close()
