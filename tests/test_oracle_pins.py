"""Pins for the CPU oracle: closed forms, invariants, special cases and brute force.

Each test fixes the oracle to something other than itself, chosen so that a
dropped term, a wrong sign, index or transposed operand fails at least one.
Citations name the passage of the paper the pinned behaviour comes from.
"""
import math

import numpy as np
import pytest

from oracle import oracle as orc
from tests.helpers import to_bf16_bits as B16, from_bf16_bits as F32, ulp_distance, fig8_case, FIG8_BOUND, FIG8_LENGTHS

RNG = np.random.default_rng(7)


def rnd(*shape, scale=1.0):
    return B16(RNG.standard_normal(shape).astype(np.float32) * scale)


# ------------------------------------------------------------------- bf16

def test_bf16_roundtrip_exhaustive():
    allb = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    f = orc.bf16_to_f32(allb)
    back = orc.f32_to_bf16(f)
    nan = np.isnan(f)
    assert (back[~nan] == allb[~nan]).all()
    assert np.isnan(F32(back[nan])).all()
    # independent numpy implementation agrees on every bf16 value and on random floats
    assert (B16(f)[~nan] == allb[~nan]).all()
    x = (RNG.standard_normal(200000) * np.exp(RNG.uniform(-20, 20, 200000))).astype(np.float32)
    assert (orc.f32_to_bf16(x) == B16(x)).all()


def test_bf16_rne_halfway_cases():
    one = 0x3F80
    cases = {1.0 + 2 ** -8: one,             # tie -> even (1.0)
             1.0 + 3 * 2 ** -8: one + 2,     # tie -> even (1 + 2^-6)
             1.0 + 2 ** -8 + 2 ** -20: one + 1,
             1.0 + 2 ** -8 - 2 ** -20: one,
             -(1.0 + 3 * 2 ** -8): 0x8000 | (one + 2)}
    for x, want in cases.items():
        assert int(orc.f32_to_bf16([x])[0]) == want, x


def test_f64_to_bf16_rounds_once():
    # just above a tie: a float32 detour would land on the tie and round down to even
    x = 1.0 + 2 ** -8 + 2 ** -40
    assert np.float32(x) == np.float32(1.0 + 2 ** -8)
    assert int(orc.f64_to_bf16([x])[0]) == 0x3F81
    x = 1.0 + 3 * 2 ** -8 - 2 ** -40
    assert int(orc.f64_to_bf16([x])[0]) == 0x3F81
    v = RNG.standard_normal(10000)
    exact = B16(v.astype(np.float32))          # differs only when the float detour double-rounds
    got = orc.f64_to_bf16(v)
    assert ulp_distance(got, exact).max() <= 1
    assert (np.abs(F32(got).astype(np.float64) - v) <= np.abs(F32(exact).astype(np.float64) - v) + 1e-300).all()


# ---------------------------------------------------------------- RMSNorm

def test_rmsnorm_constant_vector_closed_form():
    # x = c*1  =>  y_i = g_i * c / sqrt(c^2 + eps)   (Algorithm 4 step 1)
    D, c, eps = 64, 0.5, 1e-5
    g = rnd(D)
    y = orc.rmsnorm(B16(np.full((1, D), c)), g, eps)
    want = F32(g).astype(np.float64) * c / math.sqrt(c * c + eps)
    assert (y[0] == orc.f64_to_bf16(want)).all()


def test_rmsnorm_zero_unit_rms_and_scale_invariance():
    D, eps = 96, 1e-5
    ones = B16(np.ones(D))
    assert (orc.rmsnorm(B16(np.zeros((1, D))), ones, eps) == 0).all()
    x = rnd(3, D)
    y = F32(orc.rmsnorm(x, ones, eps)).astype(np.float64)
    assert np.allclose(np.sqrt((y ** 2).mean(axis=1)), 1.0, atol=4e-3)
    x4 = B16(F32(x) * 4.0)                      # exact scaling by a power of two
    assert ulp_distance(orc.rmsnorm(x4, ones, eps), orc.rmsnorm(x, ones, eps)).max() <= 1


def test_rmsnorm_eps_is_inside_the_root():
    # tiny x: y = x / sqrt(x^2 + eps) ~ x / sqrt(eps); eps outside the root would give ~1
    D, eps = 8, 1e-2
    x = B16(np.full((1, D), 2.0 ** -10))
    y = F32(orc.rmsnorm(x, B16(np.ones(D)), eps))
    want = 2.0 ** -10 / math.sqrt(2.0 ** -20 + eps)
    assert np.allclose(y, want, rtol=4e-3)


# ------------------------------------------------------------------- GEMV

def test_gemv_integer_inputs_exact_and_orientation():
    # small integers: every partial sum is exact, so y must equal the integer product
    Bn, K, N = 3, 40, 24
    x = RNG.integers(-2, 3, (Bn, K))
    W = RNG.integers(-1, 2, (K, N))
    y = orc.gemv(B16(x), B16(W))
    assert (y == (x @ W)).all()
    # W[i, n] = n  =>  y_n = n * sum(x): catches a transposed read of W
    Wc = np.tile(np.arange(N), (K, 1))
    assert (orc.gemv(B16(x), B16(Wc)) == x.sum(1, keepdims=True) * np.arange(N)).all()
    # lm_head orientation [out, in]
    Wt = RNG.integers(-1, 2, (N, K))
    assert (orc.gemv_t(B16(x), B16(Wt)) == x @ Wt.T).all()


# ------------------------------------------------------------------- RoPE

def test_rope_position_zero_is_identity_bit_exact():
    v = F32(rnd(96))
    assert (orc.rope(v, 0).view(np.uint32) == v.view(np.uint32)).all()


def test_rope_d2_is_a_plane_rotation():
    # d = 2: one pair at frequency 1 => rotation by pos radians
    got = orc.rope(np.array([1.0, 0.0], np.float32), 1)
    assert got[0] == np.float32(math.cos(1.0)) and got[1] == np.float32(math.sin(1.0))
    assert abs(got[0] - 0.5403023) < 1e-6 and abs(got[1] - 0.8414710) < 1e-6
    got = orc.rope(np.array([0.0, 1.0], np.float32), 2)
    assert np.allclose(got, [-math.sin(2.0), math.cos(2.0)], atol=1e-7)   # sign of the sine terms


def test_rope_frequencies_half_split_pairing_theta_10000():
    # d = 96: pair i couples (i, i+48) with frequency 10000^(-2i/96); pair 24 -> 0.01
    d = 96
    for i, ang in ((0, 100.0), (24, 1.0), (47, 100.0 * 10000.0 ** (-94.0 / 96.0))):
        v = np.zeros(d, np.float32)
        v[i] = 1.0
        out = orc.rope(v, 100)
        want = np.zeros(d)
        want[i], want[i + 48] = math.cos(ang), math.sin(ang)
        assert np.allclose(out, want, atol=2e-6), i
    # theta actually used
    v = np.zeros(4, np.float32); v[1] = 1.0
    out = orc.rope(v, 10, theta=100.0)            # pair 1 of d=4: freq 100^(-1/2) = 0.1 -> 1 rad
    assert np.allclose(out, [0, math.cos(1.0), 0, math.sin(1.0)], atol=1e-6)


def test_rope_norms_group_law_and_relative_position():
    d = 64
    x, y = F32(rnd(d)), F32(rnd(d))
    r = orc.rope(x, 37)
    n0 = x[:32] ** 2 + x[32:] ** 2
    n1 = r[:32] ** 2 + r[32:] ** 2
    assert np.allclose(n0, n1, rtol=1e-5)
    assert np.allclose(orc.rope(orc.rope(x, 11), 26), r, atol=2e-5)
    lhs = float(orc.rope(x, 50).astype(np.float64) @ orc.rope(y, 20).astype(np.float64))
    rhs = float(orc.rope(x, 30).astype(np.float64) @ y.astype(np.float64))
    assert abs(lhs - rhs) < 1e-3


# -------------------------------------------------------------- KV append

def _caches(Bn, H, N, d, fill=None):
    if fill is None:
        return rnd(Bn, H, N, d), rnd(Bn, H, N, d)
    return (np.full((Bn, H, N, d), fill, np.uint16), np.full((Bn, H, N, d), fill, np.uint16))


def test_append_touches_exactly_the_rows_of_eq2():
    # Eq. 2: for h in [0, B*H): offset h*(Np+Nr)*d + Np*d, a run of d elements
    Bn, H, N, d = 2, 3, 9, 8
    kc, vc = _caches(Bn, H, N, d, fill=0x7FC1)           # NaN sentinel with a payload
    k0, v0 = kc.copy(), vc.copy()
    q, kn, vn = rnd(Bn, H, d), rnd(Bn, H, d), rnd(Bn, H, d)
    L = np.array([4, 0], np.int32)
    # rows below L must be finite for the attention part; fill them
    for b in range(Bn):
        kc[b, :, :L[b]] = rnd(H, L[b], d); vc[b, :, :L[b]] = rnd(H, L[b], d)
        k0[b, :, :L[b]] = kc[b, :, :L[b]]; v0[b, :, :L[b]] = vc[b, :, :L[b]]
    orc.attn_decode(q, kn, vn, kc, vc, L, L)
    changed_k = np.flatnonzero(kc.reshape(-1) != k0.reshape(-1))
    changed_v = np.flatnonzero(vc.reshape(-1) != v0.reshape(-1))
    want = []
    for b in range(Bn):
        for h in range(H):
            start = (b * H + h) * N * d + L[b] * d
            want.extend(range(start, start + d))
    assert changed_k.tolist() == want and changed_v.tolist() == want
    for b in range(Bn):
        assert (vc[b, :, L[b]] == vn[b]).all()                       # V row is a bit copy
        for h in range(H):
            kr = orc.f32_to_bf16(orc.rope(F32(kn[b, h]), L[b]))
            assert (kc[b, h, L[b]] == kr).all()                     # K row is bf16(rope(k))


def test_successive_steps_fill_successive_rows():
    Bn, H, N, d = 1, 2, 8, 4
    kc, vc = _caches(Bn, H, N, d, fill=0)
    for t in range(5):
        q, kn, vn = rnd(Bn, H, d), rnd(Bn, H, d), rnd(Bn, H, d)
        orc.attn_decode(q, kn, vn, kc, vc, [t], [t])
        assert (vc[0, :, t] == vn[0]).all()
        assert (vc[0, :, t + 1:] == 0).all() and (kc[0, :, t + 1:] == 0).all()


def test_full_cache_or_negative_position_skips_the_sequence():
    Bn, H, N, d = 2, 1, 4, 4
    kc, vc = _caches(Bn, H, N, d)
    k0, v0 = kc.copy(), vc.copy()
    out = orc.attn_decode(rnd(Bn, H, d), rnd(Bn, H, d), rnd(Bn, H, d), kc, vc, [4, -1], [4, 2])
    assert (kc == k0).all() and (vc == v0).all() and (out == 0).all()


# -------------------------------------------------------------- attention

def test_single_key_returns_the_value_row():
    # L = 0: the only key is the new token itself, softmax = 1  (Algorithm 3 steps 9-12)
    Bn, H, N, d = 2, 3, 4, 8
    kc, vc = _caches(Bn, H, N, d, fill=0x7FC1)
    q, kn, vn = rnd(Bn, H, d), rnd(Bn, H, d), rnd(Bn, H, d)
    out = orc.attn_decode(q, kn, vn, kc, vc, [5, 9], [0, 0])
    assert (out == vn).all()


def test_zero_query_gives_the_column_mean():
    Bn, H, N, d, L = 1, 2, 8, 4, 7                     # N_t = 8 rows, small integers: exact
    kc, vc = _caches(Bn, H, N, d)
    vc[:] = B16(RNG.integers(-8, 9, vc.shape))
    vn = B16(RNG.integers(-8, 9, (Bn, H, d)))
    out = orc.attn_decode(B16(np.zeros((Bn, H, d))), rnd(Bn, H, d), vn, kc, vc, [L], [L])
    assert (F32(out) == F32(vc).mean(axis=2)).all()


def test_two_keys_closed_form_weights_and_scale():
    # d = 4 (1/sqrt(d) = 1/2), pos 0 (no rotation): q = (2,0,0,0), keys (s1,..), (s2,..)
    # scores s1, s2  =>  p1 = 1 / (1 + exp(s2 - s1)); a missing 1/sqrt(d) would double the gap
    d = 4
    s1 = float(F32(B16([math.log(3.0)]))[0])
    kc, vc = _caches(1, 1, 2, d, fill=0)
    kc[0, 0, 0] = B16([s1, 5.0, -3.0, 1.0])
    vc[0, 0, 0] = B16([1.0, 0.0, 4.0, -2.0])
    kn = B16([[[0.0, 7.0, 1.0, 2.0]]])
    vn = B16([[[0.0, 1.0, -4.0, 2.0]]])
    q = B16([[[2.0, 0.0, 0.0, 0.0]]])
    out = orc.attn_decode(q, kn, vn, kc, vc, [0], [1])
    p1 = 1.0 / (1.0 + math.exp(-s1))
    want = p1 * F32(vc[0, 0, 0]).astype(np.float64) + (1 - p1) * F32(vn[0, 0]).astype(np.float64)
    assert abs(p1 - 0.75) < 1e-3
    assert (out[0, 0] == orc.f64_to_bf16(want)).all()


def test_shift_and_permutation_invariance():
    Bn, H, N, d, L = 1, 2, 16, 8, 11
    kc, vc = _caches(Bn, H, N, d)
    q, kn, vn = rnd(Bn, H, d), rnd(Bn, H, d), rnd(Bn, H, d)
    base = orc.attn_decode(q, kn, vn, kc.copy(), vc.copy(), [0], [L])
    perm = RNG.permutation(L)
    kp, vp = kc.copy(), vc.copy()
    kp[:, :, :L] = kc[:, :, perm]; vp[:, :, :L] = vc[:, :, perm]
    assert ulp_distance(orc.attn_decode(q, kn, vn, kp, vp, [0], [L]), base).max() <= 1
    # adding one vector to every key (cached and new) shifts all scores equally; use
    # integer-valued keys and shift so that the shifted keys stay exact in bf16
    ki = B16(RNG.integers(-4, 5, kc.shape)); kni = B16(RNG.integers(-4, 5, kn.shape))
    shift = RNG.integers(-3, 4, d).astype(np.float32)
    a = orc.attn_decode(q, kni, vn, ki.copy(), vc.copy(), [0], [L])
    b = orc.attn_decode(q, B16(F32(kni) + shift), vn, B16(F32(ki) + shift), vc.copy(), [0], [L])
    assert ulp_distance(a, b).max() <= 1


def test_huge_scores_do_not_overflow_and_select_the_top_row():
    d, L = 4, 3
    kc, vc = _caches(1, 1, 4, d)
    kc[0, 0, :L] = B16([[-1000.0, 0, 0, 0], [1000.0, 0, 0, 0], [996.0, 0, 0, 0]])
    kn = B16([[[-1000.0, 0, 0, 0]]])
    q = B16([[[2.0, 0, 0, 0]]])                         # scores -1000, 1000, 996, -1000
    out = orc.attn_decode(q, kn, rnd(1, 1, d), kc, vc, [0], [L])
    p = 1.0 / (1.0 + math.exp(-4.0))
    want = p * F32(vc[0, 0, 1]).astype(np.float64) + (1 - p) * F32(vc[0, 0, 2]).astype(np.float64)
    assert np.isfinite(F32(out)).all()
    assert (out[0, 0] == orc.f64_to_bf16(want)).all()


def test_softmax_rows_sum_to_one_and_rows_past_length_are_never_read():
    Bn, H, N, d, L = 2, 2, 32, 8, 20
    kc, vc = _caches(Bn, H, N, d)
    q, kn, vn = rnd(Bn, H, d), rnd(Bn, H, d), rnd(Bn, H, d)
    kc2, vc2 = kc.copy(), vc.copy()
    kc2[:, :, L + 1:] = 0x7FC0; vc2[:, :, L + 1:] = 0x7FC0      # NaN beyond the new row
    a = orc.attn_decode(q, kn, vn, kc, vc, [L, L], [L, L])
    b = orc.attn_decode(q, kn, vn, kc2, vc2, [L, L], [L, L])
    assert (a == b).all() and np.isfinite(F32(a)).all()
    for bb in range(Bn):
        for h in range(H):
            p = orc.attn_probs(q, kc, L, L, bb, h)
            assert abs(p.sum() - 1.0) < 1e-12 and (p >= 0).all()


def test_split_and_merge_equals_one_pass():
    # splitting [0, N_t) in two and merging (m, l, o) equals the one-pass result:
    # done here with the oracle's own probabilities of the two halves
    H, N, d, L = 1, 40, 8, 31
    kc, vc = _caches(1, H, N, d)
    q, kn, vn = rnd(1, H, d), rnd(1, H, d), rnd(1, H, d)
    out = orc.attn_decode(q, kn, vn, kc, vc, [L], [L])
    p = orc.attn_probs(q, kc, L, L, 0, 0)
    V = F32(vc[0, 0, :L + 1]).astype(np.float64)
    cut = 13
    l1, l2 = p[:cut].sum(), p[cut:].sum()
    o1, o2 = (p[:cut] / l1) @ V[:cut], (p[cut:] / l2) @ V[cut:]
    merged = (l1 * o1 + l2 * o2) / (l1 + l2)
    assert ulp_distance(orc.f64_to_bf16(merged), out[0, 0]).max() <= 1


def test_planted_key_selects_its_value_per_head_and_batch():
    # one cached key per (b, h) is a large multiple of rope(q): the output must be that
    # head's own value row; distinct rows per (b, h) catch head/batch index mix-ups
    Bn, H, N, d, L = 2, 3, 24, 8, 17
    kc, vc = _caches(Bn, H, N, d)
    q = rnd(Bn, H, d)
    pos = [L, L]
    planted = {}
    for b in range(Bn):
        for h in range(H):
            j = int(RNG.integers(0, L))
            qr = orc.rope(F32(q[b, h]), pos[b])
            kc[b, h, j] = B16(qr * (60.0 / float(qr @ qr)) * math.sqrt(d))     # score ~ 60
            vc[b, h, j] = B16(np.full(d, 100.0 * (b * H + h + 1)))
            planted[(b, h)] = 100.0 * (b * H + h + 1)
    out = F32(orc.attn_decode(q, rnd(Bn, H, d), rnd(Bn, H, d), kc, vc, pos, [L, L]))
    for (b, h), val in planted.items():
        assert np.allclose(out[b, h], val, rtol=1e-2), (b, h)


def test_gqa_query_heads_share_their_group():
    # Section 4.1: query head h reads kv head h // (Hq/Hkv)
    Hq, Hkv, N, d, L = 4, 2, 8, 4, 5
    kc, vc = rnd(1, Hkv, N, d), rnd(1, Hkv, N, d)
    q1 = rnd(1, 1, d)
    q = np.repeat(q1, Hq, axis=1)
    out = orc.attn_decode(q, rnd(1, Hkv, d), rnd(1, Hkv, d), kc, vc, [L], [L])
    assert (out[0, 0] == out[0, 1]).all() and (out[0, 2] == out[0, 3]).all()
    assert (out[0, 0] != out[0, 2]).any()



@pytest.mark.parametrize("n_t", FIG8_LENGTHS)
def test_bf16_attention_stays_within_the_papers_error_bound_of_a_float_baseline(n_t):
    # Section 5.4 "Accuracy Stability" / Fig. 8: maximum error of the bf16 path against a float baseline < 0.22 %,
    # dominated by the rounding of the output.  The baseline is written in numpy float64 from the definition and
    # shares nothing with the C oracle, so a wrong sign in RoPE, a missing scale, a dropped new row or a
    # transposed operand in either of them breaks the bound (outputs are ~0.5, the bound is 0.0022).
    q, kn, vn, kc, vc, pos, L = fig8_case(n_t)
    want = orc.attn_float_baseline(q, kn, vn, kc, vc, pos, L)
    got = F32(orc.attn_decode(q, kn, vn, kc.copy(), vc.copy(), pos, L)).astype(np.float64)
    err = np.abs(got - want)
    assert err.max() < FIG8_BOUND, (n_t, err.max())
    # output rounding alone: nearly every element is the correctly rounded baseline value
    assert (B16(want.astype(np.float32)) == B16(got.astype(np.float32))).mean() > 0.98
    # the outputs concentrate around 1/2 as the softmax flattens with length
    if n_t >= 1024:
        assert abs(want.mean() - 0.5) < 0.02 and want.std() < 0.05


# -------------------------------------------------------------------- MLP

def test_mlp_zero_weights_and_zero_gate_give_zero():
    Bn, D, K = 2, 16, 24
    x = rnd(Bn, D)
    z = np.zeros((D, 2 * K), np.uint16)
    assert (F32(orc.mlp_decode(x, z, rnd(K, D))) == 0).all()
    w = rnd(D, 2 * K)
    w[:, :K] = 0                                       # gate = 0 -> silu(0) = 0
    assert (F32(orc.mlp_decode(x, w, rnd(K, D))) == 0).all()
    assert (F32(orc.mlp_decode(x, rnd(D, 2 * K), np.zeros((K, D), np.uint16))) == 0).all()


def test_mlp_identity_construction_gives_silu_times_x():
    # D = K, W_gate = c I, W_up = W_down = I  =>  y_i = silu(c x_i) * x_i   (Eq. 1, Eq. 31:
    # SiLU acts on the FIRST half of the fused product, the second half multiplies)
    D = 8
    c = 2.0
    x = B16([[1.0, -1.0, 0.5, -100.0, 3.0, 0.0, -0.25, 2.0]])
    w = np.zeros((D, 2 * D), np.float32)
    w[:, :D] = c * np.eye(D); w[:, D:] = np.eye(D)
    y = orc.mlp_f64(x, B16(w), B16(np.eye(D)))
    xv = F32(x)[0].astype(np.float64)
    want = (c * xv) / (1.0 + np.exp(-c * xv)) * xv
    assert np.allclose(y[0], want, rtol=1e-12, atol=1e-300)
    assert not np.isnan(y).any() and abs(y[0, 3]) < 1e-80      # silu(-200) ~ -3e-85, not NaN
    # the textbook values of SiLU itself
    w1 = np.zeros((1, 2), np.float32); w1[0, 0] = 1.0; w1[0, 1] = 1.0
    for t, s in ((1.0, 0.7310586), (-1.0, -0.2689414)):
        y = orc.mlp_f64(B16([[t]]), B16(w1), B16([[1.0]]))
        assert abs(y[0, 0] - s * t) < 1e-6


def test_mlp_is_linear_in_w_down_and_maps_columns_to_rows():
    Bn, D, K = 1, 8, 12
    x, wgu = rnd(Bn, D), rnd(D, 2 * K)
    a = orc.gemv(x, wgu)
    act = a[0, :K] / (1 + np.exp(-a[0, :K])) * a[0, K:]
    for k in (0, 5, 11):                               # W_down = e_k e_n^T picks a_k into y_n
        wd = np.zeros((K, D), np.float32); wd[k, (k * 3) % D] = 2.0
        y = orc.mlp_f64(x, wgu, B16(wd))
        want = np.zeros(D); want[(k * 3) % D] = 2.0 * act[k]
        assert np.allclose(y[0], want, rtol=1e-12)


# ------------------------------------------------------------------ layer

def _tiny_layer(D=8, H=2, d=4, K=16, scale=0.3):
    return dict(g_attn=B16(1 + 0.1 * RNG.standard_normal(D)), w_qkv=rnd(D, 3 * H * d, scale=scale),
                w_o=rnd(H * d, D, scale=scale), g_mlp=B16(1 + 0.1 * RNG.standard_normal(D)),
                w_gu=rnd(D, 2 * K, scale=scale), w_down=rnd(K, D, scale=scale))


def test_layer_with_zero_output_weights_is_the_identity_but_still_appends():
    D, H, d, K, N, L = 8, 2, 4, 16, 6, 3
    w = _tiny_layer(D, H, d, K)
    w["w_o"] = np.zeros_like(w["w_o"]); w["w_down"] = np.zeros_like(w["w_down"])
    kc, vc = _caches(2, H, N, d)
    k0, v0 = kc.copy(), vc.copy()
    x = rnd(2, D)
    y = orc.layer_decode(w, x, kc, vc, [L, L - 1], [L, L - 1])
    assert (y == x).all()
    n1 = orc.rmsnorm(x, w["g_attn"], 1e-5)
    qkv = orc.gemv(n1, w["w_qkv"])
    for b, Lb in ((0, L), (1, L - 1)):
        kk = orc.f64_to_bf16(qkv[b, H * d:2 * H * d]).reshape(H, d)
        vv = orc.f64_to_bf16(qkv[b, 2 * H * d:]).reshape(H, d)
        for h in range(H):
            assert (kc[b, h, Lb] == orc.f32_to_bf16(orc.rope(F32(kk[h]), Lb))).all()
            assert (vc[b, h, Lb] == vv[h]).all()
        mask = np.ones(N, bool); mask[Lb] = False
        assert (kc[b][:, mask] == k0[b][:, mask]).all() and (vc[b][:, mask] == v0[b][:, mask]).all()


def _py_layer(w, x, kc, vc, L, pos, H, d, eps=1e-5, theta=10000.0):
    """Brute force of one tiny layer in Python floats with explicit loops (no numpy matmul),
    rounding to bf16 at the block boundaries through the test-side converter."""
    r = lambda v: float(F32(B16([v]))[0])
    f = lambda bits: [float(t) for t in F32(bits).reshape(-1)]
    D = len(x)
    def norm(v, g):
        ms = sum(t * t for t in v) / len(v)
        return [r(t / math.sqrt(ms + eps) * gi) for t, gi in zip(v, g)]
    def matvec(v, Wbits):
        W = F32(Wbits)
        return [sum(v[i] * float(W[i, n]) for i in range(W.shape[0])) for n in range(W.shape[1])]
    def rope(v):
        out = list(v)
        for i in range(d // 2):
            ang = pos * theta ** (-2.0 * i / d)
            c, s = float(np.float32(math.cos(ang))), float(np.float32(math.sin(ang)))
            out[i] = v[i] * c - v[i + d // 2] * s
            out[i + d // 2] = v[i + d // 2] * c + v[i] * s
        return out
    xv = f(x)
    n1 = norm(xv, f(w["g_attn"]))
    qkv = [r(t) for t in matvec(n1, w["w_qkv"])]
    attn = []
    for h in range(H):
        q = rope(qkv[h * d:(h + 1) * d])
        k = [r(t) for t in rope(qkv[(H + h) * d:(H + h + 1) * d])]
        v = qkv[(2 * H + h) * d:(2 * H + h + 1) * d]
        keys = [f(kc[h, j]) for j in range(L)] + [k]
        vals = [f(vc[h, j]) for j in range(L)] + [v]
        s = [sum(a * b for a, b in zip(q, kk)) / math.sqrt(d) for kk in keys]
        m = max(s)
        e = [math.exp(t - m) for t in s]
        z = sum(e)
        attn += [r(sum(e[j] / z * vals[j][c] for j in range(L + 1))) for c in range(d)]
    proj = matvec(attn, w["w_o"])
    hres = [r(a + b) for a, b in zip(xv, proj)]
    n2 = norm(hres, f(w["g_mlp"]))
    gu = matvec(n2, w["w_gu"])
    K = len(gu) // 2
    act = [gu[k] / (1 + math.exp(-gu[k])) * gu[K + k] for k in range(K)]
    y = matvec(act, w["w_down"])
    return [a + b for a, b in zip(hres, y)]


@pytest.mark.parametrize("L", [0, 1, 4])
def test_tiny_layer_brute_force(L):
    # hidden 8, 2 heads, d = 4, K = 16, N_t <= 5: explicit Python-float sums
    D, H, d, K, N = 8, 2, 4, 16, 6
    w = _tiny_layer(D, H, d, K)
    kc, vc = _caches(1, H, N, d)
    x = rnd(1, D)
    want = _py_layer(w, x[0], kc[0], vc[0], L, L + 2, H, d)
    got = orc.layer_decode(w, x, kc, vc, [L + 2], [L])
    # both sides are exact up to where intermediate bf16 roundings may flip: allow 1 ulp
    assert ulp_distance(got[0], B16(np.array(want, np.float32))).max() <= 1


# ------------------------------------------------------------------ model

def test_model_embedding_logits_and_argmax_tie():
    D, H, d, K, V, N = 8, 2, 4, 16, 12, 4
    w = _tiny_layer(D, H, d, K)
    w["w_o"] = np.zeros_like(w["w_o"]); w["w_down"] = np.zeros_like(w["w_down"])   # layer = identity
    embed = rnd(V, D)
    gf = B16(np.ones(D))
    wlm = rnd(V, D)
    wlm[7] = wlm[3]                                                 # rows 3 and 7 tie everywhere
    ids = np.array([5, 2], np.int32)
    kc, vc = _caches(2, H, N, d)
    logits, nxt, hid = orc.model_decode(embed, [w], gf, wlm, [kc], [vc], ids, [1, 1], [1, 1], want_hidden=True)
    assert (hid == embed[ids]).all()
    nf = orc.rmsnorm(embed[ids], gf, 1e-5)
    want = orc.gemv_t(nf, wlm).astype(np.float32)
    assert (logits == want).all()
    assert (logits[:, 3] == logits[:, 7]).all()
    # force the tie to be the maximum: lowest index must win
    wlm2 = np.zeros_like(wlm)
    wlm2[3] = B16(F32(nf[0])); wlm2[7] = wlm2[3]
    _, nxt = orc.model_decode(embed, [w], gf, wlm2, [kc], [vc], ids[:1], [1], [1])
    assert nxt[0] == 3


@pytest.mark.parametrize("n_layers", [2, 3, 4])
def test_model_layer_loop_equals_the_chain_of_single_layers(n_layers):
    # Figure 1 repeated over the stack: the model call must be exactly the chain embedding row -> layer 0 ->
    # layer 1 -> ... -> final norm -> logits, with layer l reading and appending to ITS weights and ITS caches.
    # Every layer has distinct weights and distinct caches, sequences have distinct lengths and positions, and an
    # odd and an even number of layers are run, so a wrong per-layer index or a wrong buffer after the ping-pong
    # of the activation buffers changes the hidden state or leaves the wrong cache row written.
    D, H, d, K, V, N = 8, 2, 4, 16, 12, 7
    layers = [_tiny_layer(D, H, d, K) for _ in range(n_layers)]
    embed, gf, wlm = rnd(V, D), B16(1 + 0.1 * RNG.standard_normal(D)), rnd(V, D)
    ids = np.array([5, 2, 9], np.int32)
    lens, pos = np.array([3, 0, 5], np.int32), np.array([4, 0, 6], np.int32)
    caches = [_caches(3, H, N, d) for _ in range(n_layers)]
    # the chain, one call per layer on private copies
    ck = [c[0].copy() for c in caches]
    cv = [c[1].copy() for c in caches]
    x = embed[ids].copy()
    for l in range(n_layers):
        x = orc.layer_decode(layers[l], x, ck[l], cv[l], pos, lens)
    want_logits = orc.gemv_t(orc.rmsnorm(x, gf, 1e-5), wlm).astype(np.float32)
    # the model call
    mk = [c[0].copy() for c in caches]
    mv = [c[1].copy() for c in caches]
    logits, nxt, hid = orc.model_decode(embed, layers, gf, wlm, mk, mv, ids, pos, lens, want_hidden=True)
    assert (hid == x).all()
    assert (logits == want_logits).all()
    assert (nxt == want_logits.argmax(axis=1)).all()
    for l in range(n_layers):
        assert (mk[l] == ck[l]).all() and (mv[l] == cv[l]).all(), l
        # and the appended rows of different layers really differ (the check above can tell the layers apart)
        for b in range(3):
            assert (mk[l][b, :, lens[b]] != caches[l][0][b, :, lens[b]]).any()
        if l:
            assert (mk[l][0, :, lens[0]] != mk[l - 1][0, :, lens[0]]).any()


# ------------------------------------------------- several new tokens per step (Algorithm 3 for general N)

def _multi_case(Bn=2, N=3, Hq=4, Hkv=2, d=8, max_seq=12):
    q, kn, vn = rnd(Bn, N, Hq, d), rnd(Bn, N, Hkv, d), rnd(Bn, N, Hkv, d)
    kc, vc = _caches(Bn, Hkv, max_seq, d)
    lens, pos = np.array([4, 0][:Bn], np.int32), np.array([6, 0][:Bn], np.int32)
    return q, kn, vn, kc, vc, pos, lens


def test_multi_token_step_equals_single_token_steps_in_sequence():
    # The chunk with its causal mask IS N decode steps taken one after the other: same rows written, same outputs,
    # bit for bit (the masked form appends all rows first and masks; the sequential form never has the later rows).
    q, kn, vn, kc, vc, pos, lens = _multi_case()
    k1, v1 = kc.copy(), vc.copy()
    want = np.zeros_like(q)
    for j in range(q.shape[1]):
        want[:, j] = orc.attn_decode(q[:, j].copy(), kn[:, j].copy(), vn[:, j].copy(), k1, v1, pos + j, lens + j)
    k2, v2 = kc.copy(), vc.copy()
    got = orc.attn_decode_multi(q, kn, vn, k2, v2, pos, lens)
    assert (got == want).all()
    assert (k2 == k1).all() and (v2 == v1).all()
    # one new token per sequence is the decode step itself
    g1 = orc.attn_decode_multi(q[:, :1].copy(), kn[:, :1].copy(), vn[:, :1].copy(), kc.copy(), vc.copy(), pos, lens)
    assert (g1[:, 0] == orc.attn_decode(q[:, 0].copy(), kn[:, 0].copy(), vn[:, 0].copy(), kc.copy(), vc.copy(), pos, lens)).all()


def test_multi_token_step_is_causal_inside_the_chunk_and_matches_the_masked_matrix_form():
    q, kn, vn, kc, vc, pos, lens = _multi_case(Bn=1, N=4)
    base = orc.attn_decode_multi(q, kn, vn, kc.copy(), vc.copy(), pos, lens)
    # changing token 2 (its q, k and v) leaves tokens 0 and 1 untouched and changes tokens 2 and 3
    q2, k2n, v2n = q.copy(), kn.copy(), vn.copy()
    q2[:, 2], k2n[:, 2], v2n[:, 2] = rnd(1, 4, 8), rnd(1, 2, 8), rnd(1, 2, 8)
    pert = orc.attn_decode_multi(q2, k2n, v2n, kc.copy(), vc.copy(), pos, lens)
    assert (pert[:, :2] == base[:, :2]).all()
    assert (pert[:, 2] != base[:, 2]).any() and (pert[:, 3] != base[:, 3]).any()
    # numpy float64, written as ONE masked score matrix per head: rows = new tokens, columns = cache rows
    Bn, N, Hq, d = q.shape
    Hkv, L, p0, G = kn.shape[2], int(lens[0]), int(pos[0]), q.shape[2] // kn.shape[2]
    K = F32(kc[0]).astype(np.float64)[:, :L + N].copy()
    V = F32(vc[0]).astype(np.float64)[:, :L + N].copy()
    for j in range(N):
        for h in range(Hkv):
            K[h, L + j] = F32(B16(orc.rope(F32(kn[0, j, h]), p0 + j)))
            V[h, L + j] = F32(vn[0, j, h])
    for h in range(Hq):
        Q = np.stack([orc.rope(F32(q[0, j, h]), p0 + j) for j in range(N)]).astype(np.float64)
        S = Q @ K[h // G].T / math.sqrt(d)
        mask = np.arange(L + N)[None, :] > (L + np.arange(N))[:, None]
        S[mask] = -np.inf
        P = np.exp(S - S.max(axis=1, keepdims=True))
        P /= P.sum(axis=1, keepdims=True)
        assert ulp_distance(base[0, :, h], B16((P @ V[h // G]).astype(np.float32))).max() <= 1, h


def test_multi_token_step_skips_a_sequence_whose_rows_do_not_all_fit():
    q, kn, vn, kc, vc, pos, lens = _multi_case(Bn=2, N=3, max_seq=6)      # sequence 0: rows 4, 5, 6 -> row 6 does not exist
    k2, v2 = kc.copy(), vc.copy()
    out = orc.attn_decode_multi(q, kn, vn, k2, v2, pos, lens)
    assert (k2[0] == kc[0]).all() and (v2[0] == vc[0]).all() and (out[0] == 0).all()
    assert (k2[1, :, :3] != kc[1, :, :3]).any() and (out[1] != 0).any()


def test_layer_with_several_new_tokens_equals_the_blocks_chained_by_hand():
    # every block but the attention treats the B*N token rows alike: the multi-token layer must be
    # norm -> QKV on all rows -> multi-token attention -> output projection + residual -> norm -> MLP + residual
    D, H, d, K, N, Bn, max_seq = 8, 2, 4, 16, 3, 2, 10
    w = _tiny_layer(D, H, d, K)
    x = rnd(Bn * N, D)
    kc, vc = _caches(Bn, H, max_seq, d)
    lens, pos = np.array([3, 0], np.int32), np.array([3, 1], np.int32)
    k1, v1 = kc.copy(), vc.copy()
    got = orc.layer_decode_multi(w, x, N, k1, v1, pos, lens)
    qkv = orc.f64_to_bf16(orc.gemv(orc.rmsnorm(x, w["g_attn"], 1e-5), w["w_qkv"]))
    nq = H * d
    sp = lambda t: t.reshape(Bn, N, H, d)
    k2, v2 = kc.copy(), vc.copy()
    a = orc.attn_decode_multi(sp(qkv[:, :nq]), sp(qkv[:, nq:2 * nq]), sp(qkv[:, 2 * nq:]), k2, v2, pos, lens)
    h = orc.f64_to_bf16(F32(x).astype(np.float64) + orc.gemv(a.reshape(Bn * N, nq), w["w_o"]))
    want = orc.f64_to_bf16(F32(h).astype(np.float64) + orc.mlp_f64(orc.rmsnorm(h, w["g_mlp"], 1e-5), w["w_gu"], w["w_down"]))
    assert (got == want).all() and (k1 == k2).all() and (v1 == v2).all()
    # and one new token per sequence is the decode layer itself
    x1 = x[::N].copy()
    assert (orc.layer_decode_multi(w, x1, 1, kc.copy(), vc.copy(), pos, lens) == orc.layer_decode(w, x1, kc.copy(), vc.copy(), pos, lens)).all()


# ------------------------------------------- attention over a cache of 8-bit (E4M3) codes (Section 6.2)

def _torch_e4m3_values():
    import torch
    return torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).float().numpy()


def test_e4m3_decode_is_the_format():
    allc = np.arange(256, dtype=np.uint8)
    f = orc.e4m3_to_f32(allc)
    # facts of the format: 1.0, the largest finite value 448, the smallest subnormal 2^-9 and normal 2^-6, two zeros,
    # NaN at 0x7f / 0xff and nowhere else, no infinities, 8 values per binade, magnitudes strictly increasing with the code
    assert f[0x38] == 1.0 and f[0x7e] == 448.0 and f[0x01] == 2.0 ** -9 and f[0x08] == 2.0 ** -6
    assert f[0] == 0 and f[0x80] == 0 and np.signbit(f[0x80]) and not np.signbit(f[0])
    assert np.isnan(f[[0x7f, 0xff]]).all() and np.isfinite(np.delete(f, [0x7f, 0xff])).all()
    assert (np.diff(f[:0x7f]) > 0).all() and (f[0x80:0xff] == -f[:0x7f]).all()
    assert (f[0x40:0x48] == 2.0 * f[0x38:0x40]).all()
    # and a library's table of the same format
    t = _torch_e4m3_values()
    assert ((f == t) | (np.isnan(f) & np.isnan(t))).all()


def test_e4m3_encode_rounds_to_nearest_even_and_saturates():
    import torch
    vals = orc.e4m3_to_f32(np.arange(0x7f, dtype=np.uint8)).astype(np.float64)
    allc = np.delete(np.arange(256, dtype=np.uint8), [0x7f, 0xff])
    assert (orc.f32_to_e4m3(orc.e4m3_to_f32(allc)) == allc).all()                     # every code is its own nearest
    mid = ((vals[:-1] + vals[1:]) / 2).astype(np.float32)                            # exact in FP32
    want_even = np.where(np.arange(0x7e) % 2 == 0, np.arange(0x7e), np.arange(0x7e) + 1)
    assert (orc.f32_to_e4m3(mid) == want_even).all() and (orc.f32_to_e4m3(-mid) == (want_even | 0x80)).all()
    assert (orc.f32_to_e4m3(np.nextafter(mid, np.float32(0))) == np.arange(0x7e)).all()      # just below a midpoint
    assert (orc.f32_to_e4m3(np.nextafter(mid, np.float32(1e9))) == np.arange(0x7e) + 1).all()
    assert (orc.f32_to_e4m3([449.0, 1e9, np.inf, -np.inf, -500.0]) == [0x7e, 0x7e, 0x7e, 0xfe, 0xfe]).all()
    assert orc.f32_to_e4m3([np.nan])[0] & 0x7f == 0x7f
    x = (RNG.standard_normal(4000) * np.exp(RNG.uniform(-8, 5, 4000))).astype(np.float32)
    x = x[np.abs(x) <= 448]
    lib_codes = torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert (orc.f32_to_e4m3(x) == lib_codes).all()


def _fp8_case(Bn=2, Hq=4, Hkv=2, d=8, max_seq=12, lens=(5, 0), on_grid=False):
    codes = lambda *s: RNG.choice(np.delete(np.arange(256), [0x7f, 0xff]), size=s).astype(np.uint8)
    kc, vc = codes(Bn, Hkv, max_seq, d), codes(Bn, Hkv, max_seq, d)
    # keep the codes moderate so that scores stay in a range where the softmax is not one-hot
    kc, vc = (kc & 0x80) | (0x20 + (kc & 0x1f)), (vc & 0x80) | (0x20 + (vc & 0x1f))
    q = rnd(Bn, Hq, d)
    if on_grid:       # new rows that ARE E4M3 values: quantising them changes nothing
        kn = B16(orc.e4m3_to_f32((codes(Bn, Hkv, d) & 0x9f) | 0x20))
        vn = B16(orc.e4m3_to_f32((codes(Bn, Hkv, d) & 0x9f) | 0x20))
    else:
        kn, vn = rnd(Bn, Hkv, d), rnd(Bn, Hkv, d)
    return q, kn, vn, kc.astype(np.uint8), vc.astype(np.uint8), np.asarray(lens, np.int32)


def test_fp8_attention_on_exactly_representable_data_is_the_bf16_attention():
    # power-of-two scales and position 0 (no rotation): every dequantised value is a bf16 number and the new rows
    # survive quantisation unchanged, so the step must equal the bf16 step on the dequantised cache, bit for bit
    q, kn, vn, kc, vc, lens = _fp8_case(on_grid=True)
    ks, vs = 0.25, 2.0
    pos = np.zeros_like(lens)
    kb = B16(orc.e4m3_to_f32(kc) * np.float32(ks))
    vb = B16(orc.e4m3_to_f32(vc) * np.float32(vs))
    knb, vnb = B16(F32(kn) * np.float32(ks)), B16(F32(vn) * np.float32(vs))
    out8 = orc.attn_decode_fp8(q, knb, vnb, kc, vc, ks, vs, pos, lens)
    out16 = orc.attn_decode(q, knb, vnb, kb, vb, pos, lens)
    assert (out8 == out16).all()
    assert (B16(orc.e4m3_to_f32(kc) * np.float32(ks)) == kb).all() and (B16(orc.e4m3_to_f32(vc) * np.float32(vs)) == vb).all()


def test_fp8_attention_against_the_definition_written_out():
    q, kn, vn, kc, vc, lens = _fp8_case()
    Bn, Hq, d = q.shape
    Hkv, max_seq = kn.shape[1], kc.shape[2]
    ks, vs = 0.37, 1.6                                     # scales that are not powers of two
    pos = lens + 2
    k0, v0 = kc.copy(), vc.copy()
    out = orc.attn_decode_fp8(q, kn, vn, kc, vc, ks, vs, pos, lens)
    for b in range(Bn):
        L = int(lens[b])
        for hk in range(Hkv):
            # the appended codes: FP32 rotation, FP32 division by the scale, nearest code; nothing else changes
            kr = orc.rope(F32(kn[b, hk]), pos[b]) / np.float32(ks)
            assert (kc[b, hk, L] == orc.f32_to_e4m3(kr)).all()
            assert (vc[b, hk, L] == orc.f32_to_e4m3(F32(vn[b, hk]) / np.float32(vs))).all()
            keep = np.arange(max_seq) != L
            assert (kc[b, hk, keep] == k0[b, hk, keep]).all() and (vc[b, hk, keep] == v0[b, hk, keep]).all()
        for h in range(Hq):
            hk = h // (Hq // Hkv)
            K = orc.e4m3_to_f32(kc[b, hk, :L + 1]).astype(np.float64) * np.float64(np.float32(ks))
            V = orc.e4m3_to_f32(vc[b, hk, :L + 1]).astype(np.float64) * np.float64(np.float32(vs))
            s = K @ orc.rope(F32(q[b, h]), pos[b]).astype(np.float64) / math.sqrt(d)
            p = np.exp(s - s.max())
            want = (p / p.sum()) @ V
            assert ulp_distance(out[b, h], orc.f64_to_bf16(want)).max() <= 1


def test_fp8_attention_skips_a_full_cache_and_saturates_large_rows():
    q, kn, vn, kc, vc, _ = _fp8_case(max_seq=6)
    lens = np.array([6, 2], np.int32)
    k0, v0 = kc.copy(), vc.copy()
    out = orc.attn_decode_fp8(q, kn, vn, kc, vc, 1.0, 1.0, lens, lens)
    assert (kc[0] == k0[0]).all() and (vc[0] == v0[0]).all() and (out[0] == 0).all() and (out[1] != 0).any()
    # a scale far too small: the stored magnitudes stop at 448
    vbig = B16(np.full(vn.shape, 3.0, np.float32))
    orc.attn_decode_fp8(q, kn, vbig, kc, vc, 1.0, 1e-3, lens, lens)
    assert (vc[1, :, 2] == 0x7e).all()


def test_fp8_layer_equals_the_blocks_chained_by_hand():
    # the layer over an E4M3 cache: norm -> QKV -> attention over the codes -> output projection + residual -> norm -> MLP
    D, H, d, K, Bn, max_seq = 8, 2, 4, 16, 2, 10
    w = _tiny_layer(D, H, d, K)
    x = rnd(Bn, D)
    _, _, _, kc, vc, _ = _fp8_case(Bn=Bn, Hq=H, Hkv=H, d=d, max_seq=max_seq)
    lens, pos = np.array([3, 0], np.int32), np.array([3, 1], np.int32)
    ks, vs = 0.3, 0.7
    k1, v1 = kc.copy(), vc.copy()
    got = orc.layer_decode_fp8(w, x, k1, v1, ks, vs, pos, lens)
    qkv = orc.f64_to_bf16(orc.gemv(orc.rmsnorm(x, w["g_attn"], 1e-5), w["w_qkv"]))
    nq = H * d
    sp = lambda t: t.reshape(Bn, H, d)
    k2, v2 = kc.copy(), vc.copy()
    a = orc.attn_decode_fp8(sp(qkv[:, :nq]), sp(qkv[:, nq:2 * nq]), sp(qkv[:, 2 * nq:]), k2, v2, ks, vs, pos, lens)
    h = orc.f64_to_bf16(F32(x).astype(np.float64) + orc.gemv(a.reshape(Bn, nq), w["w_o"]))
    want = orc.f64_to_bf16(F32(h).astype(np.float64) + orc.mlp_f64(orc.rmsnorm(h, w["g_mlp"], 1e-5), w["w_gu"], w["w_down"]))
    assert (got == want).all() and (k1 == k2).all() and (v1 == v2).all()
    # and the bf16 layer is untouched by the new path: same inputs, bf16 caches of the dequantised codes, position 0
    # rotation-free, is covered by test_fp8_attention_on_exactly_representable_data_is_the_bf16_attention
