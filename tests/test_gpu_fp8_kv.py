"""Algorithm 3 over a KV cache of 8-bit E4M3 codes (the quantised cache of Section 6.2): the CUDA path against the
oracle.  The appended codes are an integer decision taken in FP32 on both sides (rotation, division by the scale,
nearest code): they are compared bit for bit, like every byte the step must not touch."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2607_11211_b200 import workload as wl
from tests.helpers import assert_close_bits, ulp_distance, from_bf16_bits as F32

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def fb():
    from paper_2607_11211_b200 import binding, build
    build.build()
    return binding


def i32(a):
    return torch.tensor(np.asarray(a, dtype=np.int32), device="cuda")


def run_case(fb, dims, lens, max_seq, k_scale, v_scale, pos=None, seed=5):
    B = len(lens)
    lens = np.asarray(lens, np.int32)
    pos = lens if pos is None else np.asarray(pos, np.int32)
    ctx = fb.Context.from_dims(dims, B, max_seq)
    act = wl.activations(dims, B, seed=seed, device="cuda")
    kc, vc = wl.kv_cache_e4m3(dims, 0, B, max_seq, k_scale, v_scale, seed=seed, device="cuda")
    k0, v0 = kc.cpu().numpy().copy(), vc.cpu().numpy().copy()
    out = torch.zeros(B, dims.n_q_heads, dims.head_dim, dtype=torch.bfloat16, device="cuda")
    ctx.attn_decode_fp8(act["q"], act["k_new"], act["v_new"], kc, vc, k_scale, v_scale, i32(pos), i32(lens), out)
    torch.cuda.synchronize()
    status = ctx.get_status()
    ko, vo = k0.copy(), v0.copy()
    want = orc.attn_decode_fp8(wl.bits(act["q"]), wl.bits(act["k_new"]), wl.bits(act["v_new"]), ko, vo, k_scale, v_scale,
                               pos, lens, dims.rope_theta)
    ctx.close()
    return wl.bits(out), want, kc.cpu().numpy(), vc.cpu().numpy(), ko, vo, k0, v0, status


@pytest.mark.parametrize("dims,lens,max_seq", [
    (wl.TINY, [0], 64), (wl.TINY, [5, 64, 17, 129], 256), (wl.SMALL, [100, 3, 255], 256), (wl.SMALL_GQA, [9, 200, 31], 256),
    (wl.PHI3_MINI, [1000, 17], 1024), (wl.PHI3_MINI, [4095], 4096), (wl.TABLE1["llama3-8b"], [777, 128, 2047], 2048),
    (wl.TABLE1["chatglm3-6b"], [300, 1500], 2048), (wl.TABLE1["llama3.2-1b"], [127, 128, 129, 1], 512)])
def test_attn_decode_fp8_matches_oracle(fb, dims, lens, max_seq):
    k_scale, v_scale = 0.0625 * 1.3, 0.05
    got, want, kg, vg, ko, vo, k0, v0, status = run_case(fb, dims, lens, max_seq, k_scale, v_scale)
    assert status == 0
    assert_close_bits(got, want, what="attention over an E4M3 cache")
    # the whole cache, byte for byte: the appended codes and every byte that must stay as it was
    assert (kg == ko).all() and (vg == vo).all()
    changed = (kg != k0) | (vg != v0)
    for b, L in enumerate(lens):
        changed[b, :, L] = False
    assert not changed.any()


def test_attn_decode_fp8_saturates_and_reports_a_full_cache(fb):
    dims, max_seq = wl.SMALL, 64
    lens = [64, 10]                                             # sequence 0 has no room
    got, want, kg, vg, ko, vo, k0, v0, status = run_case(fb, dims, lens, max_seq, 1e-4, 2e-4, pos=[3, 10])
    assert status & fb.DEV_CACHE_FULL
    assert (kg == ko).all() and (vg == vo).all() and (kg[0] == k0[0]).all()
    new = kg[1, :, 10] & 0x7f
    assert (new == 0x7e).mean() > 0.9                           # scales far too small: nearly every new code is +-448
    assert_close_bits(got[1:], want[1:], what="attention over a saturated E4M3 cache")


def test_attn_decode_fp8_keeps_subnormal_codes(fb):
    # a cache made of the SUBNORMAL codes of the format (magnitudes 2^-9 .. 7 * 2^-9) and of zeros only: widened to
    # fp16 they are normal numbers, and the products must see them (an implementation that flushed them would
    # return zeros)
    dims, max_seq, lens = wl.SMALL_GQA, 128, np.array([100, 37], np.int32)
    B, d, Hq, Hkv = 2, dims.head_dim, dims.n_q_heads, dims.n_kv_heads
    rng = np.random.default_rng(3)
    sub = lambda *s: (rng.integers(0, 8, size=s) | (rng.integers(0, 2, size=s) << 7)).astype(np.uint8)
    k0, v0 = sub(B, Hkv, max_seq, d), sub(B, Hkv, max_seq, d)
    q = orc.f32_to_bf16((rng.standard_normal((B, Hq, d)) * 8).astype(np.float32))
    tiny = orc.f32_to_bf16((rng.standard_normal((B, Hkv, d)) * 2.0 ** -8).astype(np.float32))
    ctx = fb.Context.from_dims(dims, B, max_seq)
    kc, vc = torch.from_numpy(k0.copy()).cuda(), torch.from_numpy(v0.copy()).cuda()
    out = torch.zeros(B, Hq, d, dtype=torch.bfloat16, device="cuda")
    k_scale, v_scale = 64.0, 2.0
    ctx.attn_decode_fp8(wl.from_bits(q, "cuda"), wl.from_bits(tiny, "cuda"), wl.from_bits(tiny, "cuda"), kc, vc, k_scale, v_scale,
                        i32(lens), i32(lens), out)
    torch.cuda.synchronize()
    assert ctx.get_status() == 0
    ko, vo = k0.copy(), v0.copy()
    want = orc.attn_decode_fp8(q, tiny, tiny, ko, vo, k_scale, v_scale, lens, lens, dims.rope_theta)
    got = wl.bits(out)
    assert (kc.cpu().numpy() == ko).all() and (vc.cpu().numpy() == vo).all()
    w = F32(want).astype(np.float64)
    assert np.abs(w).max() > 1e-3                                        # the expected outputs are far from zero
    assert ulp_distance(got, want).max() <= 2                            # outputs of about 0.01: two bf16 units are 2e-4
    ctx.close()


def test_attn_decode_fp8_rejects_bad_scales_and_groups(fb):
    dims = wl.SMALL
    ctx = fb.Context.from_dims(dims, 1, 64)
    act = wl.activations(dims, 1, device="cuda")
    kc, vc = wl.kv_cache_e4m3(dims, 0, 1, 64, 1.0, 1.0, device="cuda")
    out = torch.zeros(1, dims.n_q_heads, dims.head_dim, dtype=torch.bfloat16, device="cuda")
    for ks, vs in ((0.0, 1.0), (1.0, -2.0), (float("nan"), 1.0), (1.0, float("inf"))):
        with pytest.raises(fb.FasttpsError):
            ctx.attn_decode_fp8(act["q"], act["k_new"], act["v_new"], kc, vc, ks, vs, i32([0]), i32([0]), out)
    ctx.close()


def _e4m3_order(c):
    """Order-preserving integer image of E4M3 codes (+0 and -0 coincide)."""
    c = np.asarray(c, np.uint8).astype(np.int32)
    return np.where(c & 0x80, -(c & 0x7F), c)


@pytest.mark.parametrize("dims,lens", [(wl.TINY, [5, 30]), (wl.SMALL_GQA, [100, 3, 250]), (wl.PHI3_MINI, [700, 64, 5]),
                                       (wl.SMALL, [17] * 12)])
def test_layer_decode_fp8_matches_oracle(fb, dims, lens):
    from tests.helpers import layer_output_ok
    B, max_seq = len(lens), 1024
    lens = np.asarray(lens, np.int32)
    k_scale, v_scale = 0.0625 * 1.3, 0.05
    ctx = fb.Context.from_dims(dims, B, max_seq)
    w = wl.layer_weights(dims, 0, device="cuda")
    pw = ctx.pack_layer(w)
    wb = {k: wl.bits(v) for k, v in w.items()}
    x = wl.normal_bf16(5, 77, (B, dims.hidden), device="cuda")
    kc, vc = wl.kv_cache_e4m3(dims, 0, B, max_seq, k_scale, v_scale, device="cuda")
    k0, v0 = kc.cpu().numpy().copy(), vc.cpu().numpy().copy()
    xo = torch.zeros_like(x)
    ctx.layer_decode_fp8(pw["struct"], x, xo, kc, vc, k_scale, v_scale, i32(lens), i32(lens))
    torch.cuda.synchronize()
    assert ctx.get_status() == 0
    ko, vo = k0.copy(), v0.copy()
    want = orc.layer_decode_fp8(wb, wl.bits(x), ko, vo, k_scale, v_scale, lens, lens, dims.rms_eps, dims.rope_theta)
    # the residual stream before its rounding, from the oracle's primitives (see tests/helpers.py: layer_output_ok)
    nq, nkv, d = dims.n_q_heads * dims.head_dim, dims.n_kv_heads * dims.head_dim, dims.head_dim
    qkv = orc.f64_to_bf16(orc.gemv(orc.rmsnorm(wl.bits(x), wb["g_attn"], dims.rms_eps), wb["w_qkv"]))
    sp = lambda t, h: t.reshape(B, h, d)
    a = orc.attn_decode_fp8(sp(qkv[:, :nq], dims.n_q_heads), sp(qkv[:, nq:nq + nkv], dims.n_kv_heads),
                            sp(qkv[:, nq + nkv:], dims.n_kv_heads), k0.copy(), v0.copy(), k_scale, v_scale, lens, lens,
                            dims.rope_theta)
    h_exact = F32(wl.bits(x)).astype(np.float64) + orc.gemv(a.reshape(B, nq), wb["w_o"])
    ok = layer_output_ok(wl.bits(xo), want, h_exact)
    assert ok.all(), int((~ok).sum())
    kg, vg = kc.cpu().numpy(), vc.cpu().numpy()
    mask = np.ones(kg.shape, bool)
    for b in range(B):
        mask[b, :, lens[b]] = False
    assert (kg[mask] == k0[mask]).all() and (vg[mask] == v0[mask]).all()       # nothing but the new rows changed
    # k and v are outputs of the QKV block here: where the two sides round them to neighbouring bf16 values next to a
    # boundary between two codes, the stored codes are neighbours too; that must stay rare and never exceed one unit
    for got, ref in ((kg, ko), (vg, vo)):
        diff = np.abs(_e4m3_order(got[~mask]) - _e4m3_order(ref[~mask]))
        assert diff.max() <= 1 and (diff != 0).mean() < 0.01
    ctx.close()
