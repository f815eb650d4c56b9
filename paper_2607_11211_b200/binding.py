"""Thin ctypes binding of ``libfasttps.so``: argument marshalling only.

Every step of the decode path runs in the library's CUDA kernels; torch is used
for device memory and streams.  The functions carry the names of the C entry
points.  There is no fallback: if the shared library is missing or a call
fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
from pathlib import Path

import torch

PKG = Path(__file__).resolve().parent
LIB_PATH = PKG / "libfasttps.so"

W_QKV, W_O, W_GATE_UP, W_DOWN, W_LM_HEAD = range(5)
DEV_CACHE_FULL, DEV_BAD_POSITION, DEV_WAIT_TIMEOUT, DEV_BAD_TOKEN = 1, 2, 4, 8


class FasttpsError(RuntimeError):
    pass


class Config(C.Structure):
    _fields_ = [("hidden", C.c_int), ("n_q_heads", C.c_int), ("n_kv_heads", C.c_int), ("head_dim", C.c_int),
                ("inter", C.c_int), ("vocab", C.c_int), ("n_layers", C.c_int), ("max_batch", C.c_int),
                ("max_seq", C.c_int), ("rms_eps", C.c_float), ("rope_theta", C.c_float), ("device", C.c_int)]


class LayerWeights(C.Structure):
    _fields_ = [("g_attn_norm", C.c_void_p), ("w_qkv", C.c_void_p), ("w_o", C.c_void_p),
                ("g_mlp_norm", C.c_void_p), ("w_gate_up", C.c_void_p), ("w_down", C.c_void_p)]


class BaselineAttnShape(C.Structure):
    _fields_ = [("batch", C.c_int), ("n_q_heads", C.c_int), ("n_kv_heads", C.c_int), ("head_dim", C.c_int),
                ("max_seq", C.c_int), ("cat_seq", C.c_int), ("rope_theta", C.c_float)]


class BaselineAttnBuffers(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("q_rope", "k_rope", "q_trans", "k_trans", "v_trans", "k_cat", "v_cat", "s", "p")]


class BaselineMlpBuffers(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("h_g", "h_s", "h_u", "h_m")]


_lib = None


def load_library() -> C.CDLL:
    """Loads the CUDA library; raises if it has not been built (no CPU fallback exists)."""
    global _lib
    if _lib is not None:
        return _lib
    if not LIB_PATH.exists():
        raise FasttpsError(f"{LIB_PATH} is missing: build it with `python -m paper_2607_11211_b200.build` "
                           "(the decode path has no CPU fallback)")
    lib = C.CDLL(str(LIB_PATH))
    vp, ip, i = C.c_void_p, C.c_void_p, C.c_int
    lib.fasttps_create.argtypes = [C.POINTER(vp), C.POINTER(Config)]
    lib.fasttps_destroy.argtypes = [vp]
    lib.fasttps_packed_bytes.argtypes = [vp, i]
    lib.fasttps_packed_bytes.restype = C.c_size_t
    lib.fasttps_pack_weight.argtypes = [vp, i, vp, vp, vp]
    lib.fasttps_unpack_weight.argtypes = [vp, i, vp, vp, vp]
    lib.fasttps_attn_decode.argtypes = [vp, vp, vp, vp, vp, vp, ip, ip, vp, i, vp]
    lib.fasttps_attn_decode_multi.argtypes = [vp, vp, vp, vp, vp, vp, ip, ip, vp, i, i, vp]
    lib.fasttps_attn_decode_fp8.argtypes = [vp, vp, vp, vp, vp, vp, C.c_float, C.c_float, ip, ip, vp, i, vp]
    lib.fasttps_layer_decode_fp8.argtypes = [vp, C.POINTER(LayerWeights), vp, vp, vp, vp, C.c_float, C.c_float, ip, ip, i, vp]
    lib.fasttps_layer_decode_multi.argtypes = [vp, C.POINTER(LayerWeights), vp, vp, vp, vp, ip, ip, i, i, vp]
    lib.fasttps_mlp_decode.argtypes = [vp, vp, vp, vp, vp, i, vp]
    lib.fasttps_mlp_decode_static.argtypes = [vp, vp, vp, vp, vp, i, vp]
    lib.fasttps_linear_decode.argtypes = [vp, i, vp, vp, vp, vp, vp, vp, i, vp]
    lib.fasttps_layer_decode.argtypes = [vp, C.POINTER(LayerWeights), vp, vp, vp, vp, ip, ip, i, vp]
    lib.fasttps_model_decode.argtypes = [vp, vp, C.POINTER(LayerWeights), vp, vp, C.POINTER(vp), C.POINTER(vp),
                                         ip, ip, ip, vp, ip, i, i, vp]
    lib.fasttps_model_decode_host.argtypes = [vp, vp, C.POINTER(LayerWeights), vp, vp, C.POINTER(vp), C.POINTER(vp),
                                              vp, ip, ip, vp, i, vp]
    lib.fasttps_model_generate.argtypes = [vp, vp, C.POINTER(LayerWeights), vp, vp, C.POINTER(vp), C.POINTER(vp),
                                           ip, ip, ip, ip, i, i, vp]
    lib.fasttps_get_status.argtypes = [vp, C.POINTER(C.c_uint32)]
    lib.fasttps_debug_leave_workspace_dirty.argtypes = [vp]
    lib.fasttps_profile.argtypes = [vp, i]
    lib.fasttps_profile_read.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(C.c_uint64)]
    lib.fasttps_launch_count.argtypes = [vp]
    lib.fasttps_launch_count.restype = C.c_uint64
    lib.fasttps_attn_splits.argtypes = [vp, i]
    lib.fasttps_attention_shares.argtypes = [vp, vp, i, i, i, i, vp, vp]
    lib.fasttps_attention_walk.argtypes = [vp, vp, i, i, i, i, vp, i]
    lib.fasttps_baseline_attn.argtypes = [C.POINTER(BaselineAttnShape), C.POINTER(BaselineAttnBuffers), vp, vp, vp, vp, vp,
                                          ip, ip, vp, vp, vp]
    lib.fasttps_baseline_mlp.argtypes = [i, i, i, C.POINTER(BaselineMlpBuffers), vp, vp, vp, vp, vp, vp, vp]
    lib.fasttps_strerror.argtypes = [i]
    lib.fasttps_strerror.restype = C.c_char_p
    lib.fasttps_last_error.restype = C.c_char_p
    _lib = lib
    return lib


def attention_shares(seq_lens, pos, max_seq: int, step: int, group_size: int):
    """How the step kernel cuts the rows of one query head (all sequences end to end, one new row each) into
    shares for the `group_size` CTAs of the head: (shares in use, per share a list of
    (sequence, first row, end row, first share of the sequence, number of shares of the sequence)).
    Host only: needs the library, not a GPU."""
    import numpy as np
    lib = load_library()
    sl = np.ascontiguousarray(seq_lens, dtype=np.int32)
    ps = np.ascontiguousarray(pos, dtype=np.int32)
    seg = np.zeros((group_size, 8, 5), dtype=np.int32)
    nseg = np.zeros(group_size, dtype=np.int32)
    rc = lib.fasttps_attention_shares(sl.ctypes.data, ps.ctypes.data, len(sl), int(max_seq), int(step), int(group_size),
                                      seg.ctypes.data, nseg.ctypes.data)
    if rc < 0:
        _check(rc, "fasttps_attention_shares")
    return rc, [[tuple(int(v) for v in seg[g, j]) for j in range(nseg[g])] for g in range(group_size)]


def attention_walk(seq_lens, pos, heads: int, max_seq: int, n_cta: int):
    """How the stand-alone attention kernel cuts the rows of all (sequence, head) pairs into shares for `n_cta` CTAs:
    a list of (CTA, sequence, head, first row, end row, first CTA of the head, number of CTAs of the head).
    Host only: needs the library, not a GPU."""
    import numpy as np
    lib = load_library()
    sl = np.ascontiguousarray(seq_lens, dtype=np.int32)
    ps = np.ascontiguousarray(pos, dtype=np.int32)
    cap = len(sl) * heads + n_cta + 8
    seg = np.zeros((cap, 7), dtype=np.int32)
    rc = lib.fasttps_attention_walk(sl.ctypes.data, ps.ctypes.data, len(sl), int(heads), int(max_seq), int(n_cta),
                                    seg.ctypes.data, cap)
    if rc < 0:
        _check(rc, "fasttps_attention_walk")
    assert rc <= cap
    return [tuple(int(v) for v in seg[i]) for i in range(rc)]


def _check(rc: int, what: str):
    if rc != 0:
        lib = load_library()
        raise FasttpsError(f"{what}: {lib.fasttps_strerror(rc).decode()} [{lib.fasttps_last_error().decode()}]")


def _ptr(t):
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "device tensors must be contiguous CUDA tensors"
    return t.data_ptr()


def _stream(stream=None):
    s = stream if stream is not None else torch.cuda.current_stream()
    return s.cuda_stream


class Context:
    """Owns a ``fasttps_ctx``.  Methods mirror the C entry points one to one."""

    def __init__(self, hidden, n_q_heads, n_kv_heads, head_dim, inter, vocab=0, n_layers=0, max_batch=1,
                 max_seq=4096, rms_eps=1e-5, rope_theta=10000.0, device=0):
        self.lib = load_library()
        self.cfg = Config(hidden, n_q_heads, n_kv_heads, head_dim, inter, vocab, n_layers, max_batch, max_seq,
                          rms_eps, rope_theta, device)
        self.handle = C.c_void_p()
        _check(self.lib.fasttps_create(C.byref(self.handle), C.byref(self.cfg)), "fasttps_create")
        self.device = torch.device("cuda", device)
        self._keep = []

    @classmethod
    def from_dims(cls, dims, max_batch, max_seq, device=0, n_layers=None):
        return cls(dims.hidden, dims.n_q_heads, dims.n_kv_heads, dims.head_dim, dims.inter, dims.vocab,
                   dims.n_layers if n_layers is None else n_layers, max_batch, max_seq, dims.rms_eps,
                   dims.rope_theta, device)

    def close(self):
        if self.handle:
            self.lib.fasttps_destroy(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- packing ---------------------------------------------------------
    def packed_bytes(self, kind: int) -> int:
        return int(self.lib.fasttps_packed_bytes(self.handle, kind))

    def pack_weight(self, kind: int, w: torch.Tensor, stream=None) -> torch.Tensor:
        dst = torch.empty(self.packed_bytes(kind) // 2, dtype=torch.bfloat16, device=self.device)
        # the packed form pads the output rows to a multiple of 16, so it can be a little larger
        assert w.dtype == torch.bfloat16 and w.numel() <= dst.numel() < w.numel() + 16 * max(w.shape)
        _check(self.lib.fasttps_pack_weight(self.handle, kind, _ptr(w), _ptr(dst), _stream(stream)), "fasttps_pack_weight")
        return dst

    def unpack_weight(self, kind: int, packed: torch.Tensor, shape, stream=None) -> torch.Tensor:
        dst = torch.empty(shape, dtype=torch.bfloat16, device=self.device)
        assert dst.numel() <= packed.numel()
        _check(self.lib.fasttps_unpack_weight(self.handle, kind, _ptr(packed), _ptr(dst), _stream(stream)),
               "fasttps_unpack_weight")
        return dst

    def pack_layer(self, w: dict) -> dict:
        """Logical layer weights (see workload.layer_weights) -> packed device tensors + LayerWeights struct."""
        p = dict(g_attn=w["g_attn"].to(self.device).contiguous(), g_mlp=w["g_mlp"].to(self.device).contiguous(),
                 w_qkv=self.pack_weight(W_QKV, w["w_qkv"].to(self.device).contiguous()),
                 w_o=self.pack_weight(W_O, w["w_o"].to(self.device).contiguous()),
                 w_gu=self.pack_weight(W_GATE_UP, w["w_gu"].to(self.device).contiguous()),
                 w_down=self.pack_weight(W_DOWN, w["w_down"].to(self.device).contiguous()))
        torch.cuda.synchronize(self.device)
        p["struct"] = LayerWeights(_ptr(p["g_attn"]), _ptr(p["w_qkv"]), _ptr(p["w_o"]), _ptr(p["g_mlp"]),
                                   _ptr(p["w_gu"]), _ptr(p["w_down"]))
        return p

    # -- decode calls ----------------------------------------------------
    def attn_decode(self, q, k_new, v_new, k_cache, v_cache, pos, seq_lens, out, stream=None):
        batch = q.shape[0]
        _check(self.lib.fasttps_attn_decode(self.handle, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(k_cache),
                                            _ptr(v_cache), _ptr(pos), _ptr(seq_lens), _ptr(out), batch,
                                            _stream(stream)), "fasttps_attn_decode")
        return out

    def debug_leave_workspace_dirty(self):
        """Test hook: the aftermath of an abandoned call, made with host-side memsets."""
        _check(self.lib.fasttps_debug_leave_workspace_dirty(self.handle), "fasttps_debug_leave_workspace_dirty")

    def attn_decode_fp8(self, q, k_new, v_new, k_cache, v_cache, k_scale, v_scale, pos, seq_lens, out, stream=None):
        """k_cache / v_cache: uint8 tensors of E4M3 codes [B,Hkv,max_seq,d]; a code c stands for c * scale."""
        batch = q.shape[0]
        _check(self.lib.fasttps_attn_decode_fp8(self.handle, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(k_cache),
                                                _ptr(v_cache), float(k_scale), float(v_scale), _ptr(pos), _ptr(seq_lens),
                                                _ptr(out), batch, _stream(stream)), "fasttps_attn_decode_fp8")
        return out

    def attn_decode_multi(self, q, k_new, v_new, k_cache, v_cache, pos, seq_lens, out, stream=None):
        """q [B,N,Hq,d]: N new tokens per sequence."""
        batch, n_new = q.shape[0], q.shape[1]
        _check(self.lib.fasttps_attn_decode_multi(self.handle, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(k_cache),
                                                  _ptr(v_cache), _ptr(pos), _ptr(seq_lens), _ptr(out), batch, n_new,
                                                  _stream(stream)), "fasttps_attn_decode_multi")
        return out

    def layer_decode_fp8(self, lw: LayerWeights, x_in, x_out, k_cache, v_cache, k_scale, v_scale, pos, seq_lens, stream=None):
        """The layer over uint8 caches of E4M3 codes."""
        _check(self.lib.fasttps_layer_decode_fp8(self.handle, C.byref(lw), _ptr(x_in), _ptr(x_out), _ptr(k_cache),
                                                 _ptr(v_cache), float(k_scale), float(v_scale), _ptr(pos), _ptr(seq_lens),
                                                 x_in.shape[0], _stream(stream)), "fasttps_layer_decode_fp8")
        return x_out

    def layer_decode_multi(self, lw: LayerWeights, x_in, x_out, n_new, k_cache, v_cache, pos, seq_lens, stream=None):
        """x_in [B * n_new, D]: token j of sequence b in row b * n_new + j."""
        _check(self.lib.fasttps_layer_decode_multi(self.handle, C.byref(lw), _ptr(x_in), _ptr(x_out), _ptr(k_cache),
                                                   _ptr(v_cache), _ptr(pos), _ptr(seq_lens), x_in.shape[0] // n_new, n_new,
                                                   _stream(stream)), "fasttps_layer_decode_multi")
        return x_out

    def mlp_decode(self, x, w_gate_up, w_down, out, stream=None):
        _check(self.lib.fasttps_mlp_decode(self.handle, _ptr(x), _ptr(w_gate_up), _ptr(w_down), _ptr(out),
                                           x.shape[0], _stream(stream)), "fasttps_mlp_decode")
        return out

    def mlp_decode_static(self, x, w_gate_up, w_down, out, stream=None):
        """fasttps_mlp_decode with the kernel's scratch in the library's fixed device array (no workspace)."""
        _check(self.lib.fasttps_mlp_decode_static(self.handle, _ptr(x), _ptr(w_gate_up), _ptr(w_down), _ptr(out),
                                                  x.shape[0], _stream(stream)), "fasttps_mlp_decode_static")
        return out

    def linear_decode(self, kind, x, g_norm, w, residual, out_bf16, out_f32, stream=None):
        _check(self.lib.fasttps_linear_decode(self.handle, kind, _ptr(x), _ptr(g_norm), _ptr(w), _ptr(residual),
                                              _ptr(out_bf16), _ptr(out_f32), x.shape[0], _stream(stream)),
               "fasttps_linear_decode")

    def layer_decode(self, lw: LayerWeights, x_in, x_out, k_cache, v_cache, pos, seq_lens, stream=None):
        _check(self.lib.fasttps_layer_decode(self.handle, C.byref(lw), _ptr(x_in), _ptr(x_out), _ptr(k_cache),
                                             _ptr(v_cache), _ptr(pos), _ptr(seq_lens), x_in.shape[0],
                                             _stream(stream)), "fasttps_layer_decode")
        return x_out

    def make_model(self, embed, layers_packed, g_final, w_lm_packed, k_caches, v_caches):
        """Bundles the host-side pointer arrays fasttps_model_decode takes."""
        n = len(layers_packed)
        arr = (LayerWeights * n)(*[p["struct"] for p in layers_packed])
        kc = (C.c_void_p * n)(*[_ptr(t) for t in k_caches])
        vc = (C.c_void_p * n)(*[_ptr(t) for t in v_caches])
        return dict(embed=embed, layers=arr, g_final=g_final, w_lm=w_lm_packed, kc=kc, vc=vc,
                    keep=(layers_packed, k_caches, v_caches))

    def model_decode(self, model, token_ids, pos, seq_lens, logits, next_ids, advance=True, stream=None):
        _check(self.lib.fasttps_model_decode(self.handle, _ptr(model["embed"]), model["layers"],
                                             _ptr(model["g_final"]), _ptr(model["w_lm"]), model["kc"], model["vc"],
                                             _ptr(token_ids), _ptr(pos), _ptr(seq_lens), _ptr(logits),
                                             _ptr(next_ids), token_ids.shape[0], 1 if advance else 0,
                                             _stream(stream)), "fasttps_model_decode")

    def model_generate(self, model, token_ids, pos, seq_lens, out_ids, stream=None):
        """out_ids: int32 device tensor [n_steps, B]; pos/seq_lens are advanced by n_steps."""
        n_steps, batch = out_ids.shape
        _check(self.lib.fasttps_model_generate(self.handle, _ptr(model["embed"]), model["layers"],
                                               _ptr(model["g_final"]), _ptr(model["w_lm"]), model["kc"], model["vc"],
                                               _ptr(token_ids), _ptr(pos), _ptr(seq_lens), _ptr(out_ids), n_steps,
                                               batch, _stream(stream)), "fasttps_model_generate")

    def model_decode_host(self, model, host_token_ids, pos, seq_lens, host_next_ids, stream=None):
        """host_token_ids / host_next_ids: numpy int32 arrays in host memory."""
        batch = int(host_token_ids.size)
        _check(self.lib.fasttps_model_decode_host(self.handle, _ptr(model["embed"]), model["layers"],
                                                  _ptr(model["g_final"]), _ptr(model["w_lm"]), model["kc"],
                                                  model["vc"], host_token_ids.ctypes.data, _ptr(pos), _ptr(seq_lens),
                                                  host_next_ids.ctypes.data, batch, _stream(stream)),
               "fasttps_model_decode_host")

    def get_status(self) -> int:
        st = C.c_uint32(0)
        _check(self.lib.fasttps_get_status(self.handle, C.byref(st)), "fasttps_get_status")
        return int(st.value)

    PROFILE_CLASSES = ("qkv", "attn", "o_proj", "mlp", "lm_head", "embed", "step")

    def profile(self, enable: bool):
        _check(self.lib.fasttps_profile(self.handle, 1 if enable else 0), "fasttps_profile")

    def profile_read(self) -> dict:
        """{class: (total_ms, launches)} of the launches recorded since profile(True)."""
        ms = (C.c_double * 7)()
        n = (C.c_uint64 * 7)()
        _check(self.lib.fasttps_profile_read(self.handle, ms, n), "fasttps_profile_read")
        return {k: (float(ms[i]), int(n[i])) for i, k in enumerate(self.PROFILE_CLASSES)}

    def set_option(self, name: str, value: int):
        self.lib.fasttps_set_option.argtypes = [C.c_void_p, C.c_char_p, C.c_int]
        _check(self.lib.fasttps_set_option(self.handle, name.encode(), int(value)), "fasttps_set_option")

    def launch_count(self) -> int:
        return int(self.lib.fasttps_launch_count(self.handle))

    def attn_splits(self, batch: int) -> int:
        return int(self.lib.fasttps_attn_splits(self.handle, batch))


# ---------------------------------------------------------------------------------------------------------
# The non-fused comparison arm (include/fasttps_baseline.h): argument marshalling only, as above.

def baseline_attn(q, k_new, v_new, k_cache, v_cache, pos, seq_lens, out, cat_seq, rope_theta=10000.0, timed=False, stream=None):
    """fasttps_baseline_attn: Algorithm 1 as ten separate launches.  Allocates the scratch tensors with torch and
    returns (k_cat, v_cat, launch_us or None); the caller's caches are not modified."""
    lib = load_library()
    B, Hq, d = q.shape
    Hkv, max_seq = k_cache.shape[1], k_cache.shape[2]
    dev = q.device
    e = lambda *shape, dt=torch.bfloat16: torch.empty(*shape, dtype=dt, device=dev)
    keep = dict(q_rope=e(B, Hq, d), k_rope=e(B, Hkv, d), q_trans=e(B, Hq, d), k_trans=e(B, Hkv, d), v_trans=e(B, Hkv, d),
                k_cat=e(B, Hkv, cat_seq, d), v_cat=e(B, Hkv, cat_seq, d), s=e(B, Hq, cat_seq, dt=torch.float32),
                p=e(B, Hq, cat_seq, dt=torch.float32))
    bufs = BaselineAttnBuffers(*[_ptr(keep[n]) for n, _ in BaselineAttnBuffers._fields_])
    shape = BaselineAttnShape(B, Hq, Hkv, d, max_seq, cat_seq, rope_theta)
    us = (C.c_float * 10)() if timed else None
    _check(lib.fasttps_baseline_attn(C.byref(shape), C.byref(bufs), _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(k_cache),
                                     _ptr(v_cache), _ptr(pos), _ptr(seq_lens), _ptr(out), us, _stream(stream)),
           "fasttps_baseline_attn")
    return keep["k_cat"], keep["v_cat"], (list(us) if timed else None)


def baseline_mlp(x, wt_gate, wt_up, wt_down, out, timed=False, stream=None):
    """fasttps_baseline_mlp: Algorithm 2 as five separate launches on the transposed row-major matrices."""
    lib = load_library()
    B, D = x.shape
    K = wt_gate.shape[0]
    keep = [torch.empty(B, K, dtype=torch.bfloat16, device=x.device) for _ in range(4)]
    bufs = BaselineMlpBuffers(*[_ptr(t) for t in keep])
    us = (C.c_float * 5)() if timed else None
    _check(lib.fasttps_baseline_mlp(B, D, K, C.byref(bufs), _ptr(x), _ptr(wt_gate), _ptr(wt_up), _ptr(wt_down), _ptr(out), us,
                                    _stream(stream)), "fasttps_baseline_mlp")
    return list(us) if timed else None
