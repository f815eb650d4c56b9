"""ctypes front end of the CPU oracle (``fasttps_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by the smoke check and by the
benchmark's CPU-baseline leg.  The product package never imports this module
and this module never imports the product package.

All bf16 tensors are numpy ``uint16`` arrays holding the raw bit patterns.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "fasttps_oracle.c"
_LIB = _HERE / "liboracle.so"

_u16p = C.POINTER(C.c_uint16)
_i32p = C.POINTER(C.c_int32)
_f32p = C.POINTER(C.c_float)
_f64p = C.POINTER(C.c_double)


def build(force: bool = False) -> Path:
    """Compile the oracle with gcc (no CUDA, no torch)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".tmp{os.getpid()}.so")
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-ffp-contract=off", "-shared", "-fPIC",
             "-o", str(tmp), str(_SRC), "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = C.CDLL(str(build()))
        _lib.orc_bf16_to_f32.restype = C.c_float
        _lib.orc_bf16_to_f32.argtypes = [C.c_uint16]
        _lib.orc_f32_to_bf16.restype = C.c_uint16
        _lib.orc_f32_to_bf16.argtypes = [C.c_float]
        _lib.orc_f64_to_bf16.restype = C.c_uint16
        _lib.orc_f64_to_bf16.argtypes = [C.c_double]
        _lib.orc_num_threads.restype = C.c_int
    return _lib


def num_threads() -> int:
    return int(lib().orc_num_threads())


def _u16(a) -> np.ndarray:
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, a.dtype
    return a


def _p(a, t):
    return a.ctypes.data_as(t)


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


# ----------------------------------------------------------------- helpers

def bf16_to_f32(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns (uint16) to float32."""
    return (np.asarray(bits, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def f32_to_bf16(x) -> np.ndarray:
    """Round-to-nearest-even float32 -> bf16 bits through the C routine."""
    x = np.ascontiguousarray(np.asarray(x, dtype=np.float32))
    out = np.empty(x.shape, dtype=np.uint16)
    lib().orc_f32_to_bf16_array(_p(x, _f32p), _p(out, _u16p), C.c_size_t(x.size))
    return out


def f64_to_bf16(x) -> np.ndarray:
    """Single-rounding float64 -> bf16 bits through the C routine."""
    x = np.ascontiguousarray(np.asarray(x, dtype=np.float64))
    out = np.empty(x.shape, dtype=np.uint16)
    lib().orc_f64_to_bf16_array(_p(x, _f64p), _p(out, _u16p), C.c_size_t(x.size))
    return out


# ------------------------------------------------------------------- calls

def rmsnorm(x, g, eps):
    x, g = _u16(x), _u16(g)
    B, D = x.shape
    y = np.empty_like(x)
    lib().orc_rmsnorm(_p(x, _u16p), _p(g, _u16p), _p(y, _u16p), C.c_int(B), C.c_int(D), C.c_double(eps))
    return y


def gemv(x, W):
    """x [B,in] bf16 bits, W [in,out] bf16 bits -> float64 [B,out]."""
    x, W = _u16(x), _u16(W)
    B, K = x.shape
    assert W.shape[0] == K
    N = W.shape[1]
    y = np.empty((B, N), dtype=np.float64)
    lib().orc_gemv(_p(x, _u16p), _p(W, _u16p), _p(y, _f64p), C.c_int(B), C.c_int(K), C.c_int(N))
    return y


def gemv_t(x, W):
    """x [B,in], W [out,in] -> float64 [B,out]."""
    x, W = _u16(x), _u16(W)
    B, K = x.shape
    assert W.shape[1] == K
    N = W.shape[0]
    y = np.empty((B, N), dtype=np.float64)
    lib().orc_gemv_t(_p(x, _u16p), _p(W, _u16p), _p(y, _f64p), C.c_int(B), C.c_int(K), C.c_int(N))
    return y


def rope(v, pos, theta=10000.0):
    """FP32 vector [d] -> rotated FP32 vector (copy)."""
    v = np.ascontiguousarray(np.asarray(v, dtype=np.float32)).copy()
    lib().orc_rope(_p(v, _f32p), C.c_int(v.size), C.c_int(int(pos)), C.c_double(theta))
    return v


def attn_decode(q, k_new, v_new, k_cache, v_cache, pos, seq_lens, theta=10000.0):
    """Appends in place to k_cache/v_cache ([B,Hkv,max_seq,d]); returns out [B,Hq,d]."""
    q, k_new, v_new = _u16(q), _u16(k_new), _u16(v_new)
    assert k_cache.dtype == np.uint16 and k_cache.flags.c_contiguous and k_cache.flags.writeable
    assert v_cache.dtype == np.uint16 and v_cache.flags.c_contiguous and v_cache.flags.writeable
    B, Hq, d = q.shape
    Hkv = k_new.shape[1]
    max_seq = k_cache.shape[2]
    assert k_cache.shape == (B, Hkv, max_seq, d) and v_cache.shape == k_cache.shape
    pos, seq_lens = _i32(pos), _i32(seq_lens)
    out = np.zeros((B, Hq, d), dtype=np.uint16)
    lib().orc_attn_decode(_p(q, _u16p), _p(k_new, _u16p), _p(v_new, _u16p),
                          _p(k_cache, _u16p), _p(v_cache, _u16p), _p(pos, _i32p), _p(seq_lens, _i32p),
                          _p(out, _u16p), C.c_int(B), C.c_int(Hq), C.c_int(Hkv), C.c_int(d),
                          C.c_int(max_seq), C.c_double(theta))
    return out


def attn_decode_multi(q, k_new, v_new, k_cache, v_cache, pos, seq_lens, theta=10000.0):
    """N new tokens per sequence: q [B,N,Hq,d], k_new / v_new [B,N,Hkv,d]; token j goes into row seq_lens[b] + j at
    rotary position pos[b] + j and attends rows 0 .. seq_lens[b] + j.  Appends in place; returns out [B,N,Hq,d]."""
    q, k_new, v_new = _u16(q), _u16(k_new), _u16(v_new)
    assert k_cache.dtype == np.uint16 and k_cache.flags.c_contiguous and k_cache.flags.writeable
    assert v_cache.dtype == np.uint16 and v_cache.flags.c_contiguous and v_cache.flags.writeable
    B, N, Hq, d = q.shape
    Hkv = k_new.shape[2]
    max_seq = k_cache.shape[2]
    assert k_new.shape == (B, N, Hkv, d) and k_cache.shape == (B, Hkv, max_seq, d) and v_cache.shape == k_cache.shape
    pos, seq_lens = _i32(pos), _i32(seq_lens)
    out = np.zeros((B, N, Hq, d), dtype=np.uint16)
    lib().orc_attn_decode_multi(_p(q, _u16p), _p(k_new, _u16p), _p(v_new, _u16p), _p(k_cache, _u16p), _p(v_cache, _u16p),
                                _p(pos, _i32p), _p(seq_lens, _i32p), _p(out, _u16p), C.c_int(B), C.c_int(N), C.c_int(Hq),
                                C.c_int(Hkv), C.c_int(d), C.c_int(max_seq), C.c_double(theta))
    return out


def e4m3_to_f32(codes) -> np.ndarray:
    """uint8 E4M3 codes -> float32 values (NaN for the two NaN codes)."""
    c = np.ascontiguousarray(np.asarray(codes, dtype=np.uint8))
    f = lib().orc_e4m3_to_f32
    f.restype, f.argtypes = C.c_float, [C.c_uint8]
    return np.array([f(int(v)) for v in c.ravel()], dtype=np.float32).reshape(c.shape)


def f32_to_e4m3(x) -> np.ndarray:
    """float32 values -> uint8 E4M3 codes: nearest, ties to even, saturating at 448."""
    v = np.ascontiguousarray(np.asarray(x, dtype=np.float32))
    f = lib().orc_f32_to_e4m3
    f.restype, f.argtypes = C.c_uint8, [C.c_float]
    return np.array([f(float(t)) for t in v.ravel()], dtype=np.uint8).reshape(v.shape)


def attn_decode_fp8(q, k_new, v_new, k_cache, v_cache, k_scale, v_scale, pos, seq_lens, theta=10000.0):
    """Algorithm 3 over a cache of E4M3 codes (uint8 [B,Hkv,max_seq,d], appended in place) with one scale per tensor;
    returns out [B,Hq,d] bf16 bits."""
    q, k_new, v_new = _u16(q), _u16(k_new), _u16(v_new)
    assert k_cache.dtype == np.uint8 and k_cache.flags.c_contiguous and k_cache.flags.writeable
    assert v_cache.dtype == np.uint8 and v_cache.flags.c_contiguous and v_cache.flags.writeable
    B, Hq, d = q.shape
    Hkv = k_new.shape[1]
    max_seq = k_cache.shape[2]
    assert k_cache.shape == (B, Hkv, max_seq, d) and v_cache.shape == k_cache.shape
    pos, seq_lens = _i32(pos), _i32(seq_lens)
    out = np.zeros((B, Hq, d), dtype=np.uint16)
    u8p = C.POINTER(C.c_uint8)
    lib().orc_attn_decode_fp8(_p(q, _u16p), _p(k_new, _u16p), _p(v_new, _u16p), _p(k_cache, u8p), _p(v_cache, u8p),
                              C.c_float(k_scale), C.c_float(v_scale), _p(pos, _i32p), _p(seq_lens, _i32p),
                              _p(out, _u16p), C.c_int(B), C.c_int(Hq), C.c_int(Hkv), C.c_int(d), C.c_int(max_seq),
                              C.c_double(theta))
    return out


def attn_probs(q, k_cache, pos, L, b, h, theta=10000.0):
    q = _u16(q)
    B, Hq, d = q.shape
    _, Hkv, max_seq, _ = k_cache.shape
    p = np.empty(L + 1, dtype=np.float64)
    lib().orc_attn_probs(_p(q, _u16p), _p(_u16(k_cache), _u16p), C.c_int(int(pos)), C.c_int(int(L)),
                         C.c_int(b), C.c_int(h), C.c_int(Hq), C.c_int(Hkv), C.c_int(d),
                         C.c_int(max_seq), C.c_double(theta), _p(p, _f64p))
    return p


def mlp_f64(x, w_gu, w_down):
    x, w_gu, w_down = _u16(x), _u16(w_gu), _u16(w_down)
    B, D = x.shape
    K = w_down.shape[0]
    assert w_gu.shape == (D, 2 * K) and w_down.shape == (K, D)
    y = np.empty((B, D), dtype=np.float64)
    lib().orc_mlp_f64(_p(x, _u16p), _p(w_gu, _u16p), _p(w_down, _u16p), _p(y, _f64p),
                      C.c_int(B), C.c_int(D), C.c_int(K))
    return y


def mlp_decode(x, w_gu, w_down):
    x, w_gu, w_down = _u16(x), _u16(w_gu), _u16(w_down)
    B, D = x.shape
    K = w_down.shape[0]
    assert w_gu.shape == (D, 2 * K) and w_down.shape == (K, D)
    out = np.empty((B, D), dtype=np.uint16)
    lib().orc_mlp_decode(_p(x, _u16p), _p(w_gu, _u16p), _p(w_down, _u16p), _p(out, _u16p),
                         C.c_int(B), C.c_int(D), C.c_int(K))
    return out


def layer_decode(w: dict, x_in, k_cache, v_cache, pos, seq_lens, eps=1e-5, theta=10000.0):
    """w: dict with g_attn [D], w_qkv [D,(Hq+2Hkv)d], w_o [Hq d,D], g_mlp [D],
    w_gu [D,2K], w_down [K,D] (bf16 bits).  Returns x_out [B,D]; caches appended in place."""
    x_in = _u16(x_in)
    B, D = x_in.shape
    _, Hkv, max_seq, d = k_cache.shape
    Hq = w["w_o"].shape[0] // d
    K = w["w_down"].shape[0]
    assert w["w_qkv"].shape == (D, (Hq + 2 * Hkv) * d)
    pos, seq_lens = _i32(pos), _i32(seq_lens)
    x_out = np.empty_like(x_in)
    lib().orc_layer_decode(_p(_u16(w["g_attn"]), _u16p), _p(_u16(w["w_qkv"]), _u16p), _p(_u16(w["w_o"]), _u16p),
                           _p(_u16(w["g_mlp"]), _u16p), _p(_u16(w["w_gu"]), _u16p), _p(_u16(w["w_down"]), _u16p),
                           _p(x_in, _u16p), _p(x_out, _u16p), _p(k_cache, _u16p), _p(v_cache, _u16p),
                           _p(pos, _i32p), _p(seq_lens, _i32p),
                           C.c_int(B), C.c_int(D), C.c_int(Hq), C.c_int(Hkv), C.c_int(d), C.c_int(K),
                           C.c_int(max_seq), C.c_double(eps), C.c_double(theta))
    return x_out


def layer_decode_multi(w: dict, x_in, n_new, k_cache, v_cache, pos, seq_lens, eps=1e-5, theta=10000.0):
    """layer_decode for n_new tokens per sequence: x_in [B*n_new, D] (token j of sequence b in row b*n_new + j),
    pos / seq_lens [B].  Returns x_out [B*n_new, D]; caches appended in place (n_new rows per head and sequence)."""
    x_in = _u16(x_in)
    rows, D = x_in.shape
    B = rows // n_new
    assert B * n_new == rows
    _, Hkv, max_seq, d = k_cache.shape
    Hq = w["w_o"].shape[0] // d
    K = w["w_down"].shape[0]
    pos, seq_lens = _i32(pos), _i32(seq_lens)
    assert pos.size == B and seq_lens.size == B
    x_out = np.empty_like(x_in)
    lib().orc_layer_decode_multi(_p(_u16(w["g_attn"]), _u16p), _p(_u16(w["w_qkv"]), _u16p), _p(_u16(w["w_o"]), _u16p),
                                 _p(_u16(w["g_mlp"]), _u16p), _p(_u16(w["w_gu"]), _u16p), _p(_u16(w["w_down"]), _u16p),
                                 _p(x_in, _u16p), _p(x_out, _u16p), _p(k_cache, _u16p), _p(v_cache, _u16p),
                                 _p(pos, _i32p), _p(seq_lens, _i32p), C.c_int(B), C.c_int(n_new), C.c_int(D), C.c_int(Hq),
                                 C.c_int(Hkv), C.c_int(d), C.c_int(K), C.c_int(max_seq), C.c_double(eps), C.c_double(theta))
    return x_out


def layer_decode_fp8(w: dict, x_in, k_cache, v_cache, k_scale, v_scale, pos, seq_lens, eps=1e-5, theta=10000.0):
    """layer_decode over caches of E4M3 codes (uint8 [B,Hkv,max_seq,d], appended in place); returns x_out [B, D]."""
    x_in = _u16(x_in)
    B, D = x_in.shape
    assert k_cache.dtype == np.uint8 and v_cache.dtype == np.uint8 and k_cache.flags.c_contiguous and v_cache.flags.c_contiguous
    _, Hkv, max_seq, d = k_cache.shape
    Hq = w["w_o"].shape[0] // d
    K = w["w_down"].shape[0]
    pos, seq_lens = _i32(pos), _i32(seq_lens)
    x_out = np.empty_like(x_in)
    u8p = C.POINTER(C.c_uint8)
    lib().orc_layer_decode_fp8(_p(_u16(w["g_attn"]), _u16p), _p(_u16(w["w_qkv"]), _u16p), _p(_u16(w["w_o"]), _u16p),
                               _p(_u16(w["g_mlp"]), _u16p), _p(_u16(w["w_gu"]), _u16p), _p(_u16(w["w_down"]), _u16p),
                               _p(x_in, _u16p), _p(x_out, _u16p), _p(k_cache, u8p), _p(v_cache, u8p),
                               C.c_float(k_scale), C.c_float(v_scale), _p(pos, _i32p), _p(seq_lens, _i32p), C.c_int(B),
                               C.c_int(D), C.c_int(Hq), C.c_int(Hkv), C.c_int(d), C.c_int(K), C.c_int(max_seq),
                               C.c_double(eps), C.c_double(theta))
    return x_out


def model_decode(embed, layers, g_final, w_lm, k_caches, v_caches, token_ids, pos, seq_lens,
                 eps=1e-5, theta=10000.0, want_hidden=False):
    """layers: list of dicts as in layer_decode.  Returns (logits f32 [B,V], next_ids i32 [B]
    [, hidden bf16 bits [B,D]]); caches appended in place."""
    embed, w_lm, g_final = _u16(embed), _u16(w_lm), _u16(g_final)
    V, D = embed.shape
    n = len(layers)
    _, Hkv, max_seq, d = k_caches[0].shape
    Hq = layers[0]["w_o"].shape[0] // d
    K = layers[0]["w_down"].shape[0]
    token_ids, pos, seq_lens = _i32(token_ids), _i32(pos), _i32(seq_lens)
    B = token_ids.size

    def arr(key):
        keep = [_u16(L[key]) for L in layers]
        return keep, (_u16p * n)(*[_p(a, _u16p) for a in keep])

    keep = []
    ptrs = []
    for key in ("g_attn", "w_qkv", "w_o", "g_mlp", "w_gu", "w_down"):
        k_, p_ = arr(key)
        keep.append(k_)
        ptrs.append(p_)
    kc = (_u16p * n)(*[_p(a, _u16p) for a in k_caches])
    vc = (_u16p * n)(*[_p(a, _u16p) for a in v_caches])
    logits = np.empty((B, V), dtype=np.float32)
    next_ids = np.empty(B, dtype=np.int32)
    hidden = np.empty((B, D), dtype=np.uint16)
    lib().orc_model_decode(_p(embed, _u16p), C.c_int(n), *ptrs, _p(g_final, _u16p), _p(w_lm, _u16p), kc, vc,
                           _p(token_ids, _i32p), _p(pos, _i32p), _p(seq_lens, _i32p),
                           _p(logits, _f32p), _p(next_ids, _i32p), _p(hidden, _u16p),
                           C.c_int(B), C.c_int(D), C.c_int(Hq), C.c_int(Hkv), C.c_int(d), C.c_int(K),
                           C.c_int(V), C.c_int(max_seq), C.c_double(eps), C.c_double(theta))
    if want_hidden:
        return logits, next_ids, hidden
    return logits, next_ids


def attn_float_baseline(q, k_new, v_new, k_cache, v_cache, pos, seq_lens, theta=10000.0):
    """Decode attention with no reduced-precision step after the inputs: the "float" baseline of the
    paper's accuracy experiment (Section 5.4, "Accuracy Stability"; Fig. 8), written out in numpy
    float64 from the definition (half-split RoPE, scores over the cached rows and the new row,
    softmax with the 1/sqrt(d) scale, PV).  Unlike ``attn_decode`` the rotated new K row is NOT
    rounded to bf16 before it is scored and the output is NOT rounded; the caches are not modified.
    Inputs are bf16 bit patterns; returns float64 [B, Hq, d].  Sequences the method would skip
    (full cache, negative position) are not handled here."""
    q, k_new, v_new = bf16_to_f32(_u16(q)).astype(np.float64), bf16_to_f32(_u16(k_new)).astype(np.float64), \
        bf16_to_f32(_u16(v_new)).astype(np.float64)
    B, Hq, d = q.shape
    Hkv = k_new.shape[1]
    G = Hq // Hkv
    half = d // 2
    freq = theta ** (-2.0 * np.arange(half) / d)
    out = np.zeros((B, Hq, d))

    def rot(v, p):
        c, s = np.cos(p * freq), np.sin(p * freq)
        return np.concatenate([v[:half] * c - v[half:] * s, v[half:] * c + v[:half] * s])

    for b in range(B):
        L, p = int(seq_lens[b]), int(pos[b])
        for h in range(Hq):
            hk = h // G
            K = np.vstack([bf16_to_f32(k_cache[b, hk, :L]).astype(np.float64), rot(k_new[b, hk], p)[None]])
            V = np.vstack([bf16_to_f32(v_cache[b, hk, :L]).astype(np.float64), v_new[b, hk][None]])
            s = K @ rot(q[b, h], p) / np.sqrt(d)
            e = np.exp(s - s.max())
            out[b, h] = (e / e.sum()) @ V
    return out
