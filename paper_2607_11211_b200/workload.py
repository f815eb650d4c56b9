"""Seeded synthetic inputs for the decode path.

This module holds none of the method's arithmetic: it only makes tensors.  It
serves both the CUDA library's tests/benchmark and the CPU oracle's tests, so
the two sides see bit-identical inputs without importing each other.

Generator.  ``normal_bf16(seed, tensor_id, n, scale)`` is counter based: element
``i`` depends only on ``(seed, tensor_id, i)``, so any slice of any tensor can
be re-derived anywhere (CPU or GPU) without holding the whole tensor.  Two
64-bit outputs of the SplitMix64 finaliser are cut into eight 16-bit uniforms;
their integer sum (Irwin-Hall, n = 8) is centred and scaled to unit variance
with one FP32 multiply, scaled by ``scale`` with a second FP32 multiply, and
rounded to bf16 (nearest even).  Only integer ops and single IEEE multiplies
are involved, so torch produces the same bits on the CPU and on a GPU.  The
distribution is a stand-in for N(0, scale^2): variance 1, tails cut at 4.9
sigma, excess kurtosis -0.15.

Recipes follow the five workload descriptions of the benchmark contract:
Phi-3-mini shapes, matrices ~ N(0, 0.02^2), norm gains 1 + 0.02 z, activations
and cache contents ~ N(0, 1).
"""
from __future__ import annotations

from dataclasses import dataclass, asdict

import numpy as np
import torch

MASTER_SEED = 20260711

_M1 = -4658895280553007687   # 0xBF58476D1CE4E5B9 as int64
_M2 = -7723592293110705685   # 0x94D049BB133111EB as int64
_GOLD = -7046029254386353131  # 0x9E3779B97F4A7C15 as int64

_IH_MEAN = 8 * 32767.5                       # 262140
_IH_INV_STD = float(np.float32(1.0 / (65536.0 * np.sqrt(8.0 / 12.0))))


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    return (x >> s) & ((1 << (64 - s)) - 1)


def _mix64(x: torch.Tensor) -> torch.Tensor:
    x = (x ^ _lsr(x, 30)) * _M1
    x = (x ^ _lsr(x, 27)) * _M2
    return x ^ _lsr(x, 31)


def _key(seed: int, tensor_id: int) -> int:
    k = (seed * 0x9E3779B97F4A7C15 + tensor_id * 0xD1B54A32D192ED03 + 0x2545F4914F6CDD1D) & (2 ** 64 - 1)
    return k - 2 ** 64 if k >= 2 ** 63 else k


def normal_f32(seed: int, tensor_id: int, start: int, n: int, device="cpu") -> torch.Tensor:
    """Unit-variance pseudo-normal FP32 values for elements [start, start+n)."""
    idx = torch.arange(start, start + n, dtype=torch.int64, device=device)
    key = _key(seed, tensor_id)
    total = torch.zeros(n, dtype=torch.int64, device=device)
    for j in range(2):
        h = _mix64((idx * 2 + j) * _GOLD + key)
        for sh in (0, 16, 32, 48):
            total += _lsr(h, sh) & 0xFFFF
    z = (total - int(_IH_MEAN)).to(torch.float32)
    return z * _IH_INV_STD


def normal_bf16(seed: int, tensor_id: int, shape, scale: float = 1.0, offset: float = 0.0,
                device="cpu", chunk: int = 1 << 24) -> torch.Tensor:
    """bf16 tensor of ``shape`` with value bf16(offset + scale * z), z ~ pseudo-N(0,1)."""
    n = int(np.prod(shape))
    out = torch.empty(n, dtype=torch.bfloat16, device=device)
    for s in range(0, n, chunk):
        m = min(chunk, n - s)
        v = normal_f32(seed, tensor_id, s, m, device) * float(np.float32(scale))
        if offset != 0.0:
            v = v + float(np.float32(offset))
        out[s:s + m] = v.to(torch.bfloat16)
    return out.view(*shape)


def bits(t: torch.Tensor) -> np.ndarray:
    """bf16 torch tensor -> numpy uint16 bit patterns (host copy)."""
    return t.detach().contiguous().cpu().view(torch.int16).numpy().view(np.uint16)


def from_bits(a: np.ndarray, device="cpu") -> torch.Tensor:
    """numpy uint16 bit patterns -> bf16 torch tensor."""
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16).to(device)


# ---------------------------------------------------------------------------
# shapes

@dataclass(frozen=True)
class Dims:
    hidden: int = 3072
    n_q_heads: int = 32
    n_kv_heads: int = 32
    head_dim: int = 96
    inter: int = 8192
    vocab: int = 32064
    n_layers: int = 32
    rms_eps: float = 1e-5
    rope_theta: float = 10000.0

    @property
    def qkv_out(self) -> int:
        return (self.n_q_heads + 2 * self.n_kv_heads) * self.head_dim

    @property
    def layer_weight_bytes(self) -> int:
        D, K = self.hidden, self.inter
        return 2 * (D * self.qkv_out + self.n_q_heads * self.head_dim * D + D * 2 * K + K * D + 2 * D)

    @property
    def kv_bytes_per_token_per_layer(self) -> int:
        return 2 * self.n_kv_heads * self.head_dim * 2

    def as_dict(self):
        return asdict(self)


PHI3_MINI = Dims()
TINY = Dims(hidden=128, n_q_heads=4, n_kv_heads=4, head_dim=32, inter=128, vocab=160, n_layers=2)
SMALL = Dims(hidden=256, n_q_heads=4, n_kv_heads=4, head_dim=64, inter=640, vocab=1000, n_layers=3)
SMALL_GQA = Dims(hidden=256, n_q_heads=8, n_kv_heads=2, head_dim=32, inter=384, vocab=520, n_layers=2)

# The other model shapes of the paper's Table 1 (query heads, K/V heads, head_dim and MLP width as printed there;
# hidden = query heads x head_dim; layer counts and vocabulary sizes of the public model cards, which only scale the
# work).  Synthetic weights of these shapes stand in for the checkpoints.
TABLE1 = {
    "llama3-8b": Dims(hidden=4096, n_q_heads=32, n_kv_heads=8, head_dim=128, inter=14336, vocab=128256, n_layers=32),
    "chatglm3-6b": Dims(hidden=4096, n_q_heads=32, n_kv_heads=2, head_dim=128, inter=13696, vocab=65024, n_layers=28),
    "llama2-7b": Dims(hidden=4096, n_q_heads=32, n_kv_heads=32, head_dim=128, inter=11008, vocab=32000, n_layers=32),
    "phi3-mini": PHI3_MINI,
    "llama3.2-1b": Dims(hidden=2048, n_q_heads=32, n_kv_heads=32, head_dim=64, inter=8192, vocab=128256, n_layers=16),
}

# tensor-id scheme: 1000*layer + kind; layer = 999 for model-level tensors
_KIND = dict(g_attn=1, w_qkv=2, w_o=3, g_mlp=4, w_gu=5, w_down=6, k_cache=7, v_cache=8,
             embed=11, g_final=12, w_lm=13, x=21, q=22, k_new=23, v_new=24)


def tid(kind: str, layer: int = 999) -> int:
    return 1000 * layer + _KIND[kind]


def layer_weights(dims: Dims, layer: int, seed: int = MASTER_SEED, device="cpu") -> dict:
    """Logical (unpacked) weights of one layer, bf16:
    g_attn [D], w_qkv [D,(Hq+2Hkv)d], w_o [Hq d,D], g_mlp [D], w_gu [D,2K] (gate|up), w_down [K,D]."""
    D, K, d = dims.hidden, dims.inter, dims.head_dim
    return dict(
        g_attn=normal_bf16(seed, tid("g_attn", layer), (D,), 0.02, 1.0, device),
        w_qkv=normal_bf16(seed, tid("w_qkv", layer), (D, dims.qkv_out), 0.02, 0.0, device),
        w_o=normal_bf16(seed, tid("w_o", layer), (dims.n_q_heads * d, D), 0.02, 0.0, device),
        g_mlp=normal_bf16(seed, tid("g_mlp", layer), (D,), 0.02, 1.0, device),
        w_gu=normal_bf16(seed, tid("w_gu", layer), (D, 2 * K), 0.02, 0.0, device),
        w_down=normal_bf16(seed, tid("w_down", layer), (K, D), 0.02, 0.0, device),
    )


def model_weights(dims: Dims, seed: int = MASTER_SEED, device="cpu") -> dict:
    return dict(
        embed=normal_bf16(seed, tid("embed"), (dims.vocab, dims.hidden), 0.02, 0.0, device),
        g_final=normal_bf16(seed, tid("g_final"), (dims.hidden,), 0.02, 1.0, device),
        w_lm=normal_bf16(seed, tid("w_lm"), (dims.vocab, dims.hidden), 0.02, 0.0, device),
        layers=[layer_weights(dims, l, seed, device) for l in range(dims.n_layers)],
    )


def kv_cache(dims: Dims, layer: int, batch: int, max_seq: int, seed: int = MASTER_SEED, device="cpu"):
    """Pre-filled caches [B,Hkv,max_seq,d] ~ N(0,1) (every row filled; rows past a
    sequence's length are simply never read)."""
    shp = (batch, dims.n_kv_heads, max_seq, dims.head_dim)
    return (normal_bf16(seed, tid("k_cache", layer), shp, 1.0, 0.0, device),
            normal_bf16(seed, tid("v_cache", layer), shp, 1.0, 0.0, device))


def kv_cache_e4m3(dims: Dims, layer: int, batch: int, max_seq: int, k_scale: float, v_scale: float,
                  seed: int = MASTER_SEED, device="cpu"):
    """The same N(0,1) caches stored as 8-bit E4M3 codes (uint8 tensors [B,Hkv,max_seq,d]) of value / scale; the
    conversion is the library's (round to nearest even; the values are clamped to the format's range first)."""
    out = []
    for t, s in zip(kv_cache(dims, layer, batch, max_seq, seed, device), (k_scale, v_scale)):
        out.append((t.float() / s).clamp_(-448.0, 448.0).to(torch.float8_e4m3fn).view(torch.uint8))
    return tuple(out)


def activations(dims: Dims, batch: int, seed: int = MASTER_SEED, device="cpu") -> dict:
    """Block-level inputs: x [B,D], q [B,Hq,d], k_new/v_new [B,Hkv,d] ~ N(0,1)."""
    d = dims.head_dim
    return dict(
        x=normal_bf16(seed, tid("x"), (batch, dims.hidden), 1.0, 0.0, device),
        q=normal_bf16(seed, tid("q"), (batch, dims.n_q_heads, d), 1.0, 0.0, device),
        k_new=normal_bf16(seed, tid("k_new"), (batch, dims.n_kv_heads, d), 1.0, 0.0, device),
        v_new=normal_bf16(seed, tid("v_new"), (batch, dims.n_kv_heads, d), 1.0, 0.0, device),
    )


def ragged_lengths(batch: int, lo: int, hi: int, seed: int = MASTER_SEED) -> np.ndarray:
    """Past lengths drawn uniformly from the integers lo..hi inclusive."""
    return np.random.default_rng(seed + 1).integers(lo, hi + 1, size=batch).astype(np.int32)


def token_ids(n: int, vocab: int, seed: int = MASTER_SEED) -> np.ndarray:
    return np.random.default_rng(seed + 2).integers(0, vocab, size=n).astype(np.int32)


# ---------------------------------------------------------------------------
# the five workload descriptions

@dataclass(frozen=True)
class Workload:
    name: str
    dims: Dims
    n_layers: int          # layers actually run (1 for the single-layer cases)
    full_stack: bool       # embedding + lm_head + argmax around the layers
    batch: int
    past_lens: tuple       # per-sequence tokens already cached
    max_seq: int
    n_steps: int           # consecutive decode steps of one "run"

    def algorithmic_bytes(self, step: int = 0) -> int:
        """Bytes one decode step must move: weights once + K/V rows read (past) and
        written (new) + block inputs/outputs (+ lm_head and logits for the full stack)."""
        dm = self.dims
        w = self.n_layers * dm.layer_weight_bytes
        kv = self.n_layers * dm.kv_bytes_per_token_per_layer * sum(int(l) + step + 1 for l in self.past_lens)
        act = self.batch * 2 * dm.hidden * 2
        if self.full_stack:
            w += 2 * dm.vocab * dm.hidden + 2 * dm.hidden          # lm_head + final gain
            act = self.batch * (2 * dm.hidden + 4 * dm.vocab)      # embedding row in, logits out
        return w + kv + act


def workload(name: str) -> Workload:
    P = PHI3_MINI
    if name == "cfg1":
        return Workload(name, P, 1, False, 1, (256,), 4096, 1)
    if name == "cfg2":
        return Workload(name, P, 1, False, 1, (4095,), 4096, 1)
    if name == "cfg3":
        return Workload(name, P, 32, True, 1, (1024,), 1280, 128)
    if name == "cfg4":
        return Workload(name, P, 32, True, 8, tuple(int(v) for v in ragged_lengths(8, 512, 4096)), 4224, 1)
    if name == "cfg5":
        return Workload(name, P, 32, True, 32, (4095,) * 32, 4096, 1)
    if name in TABLE1:          # a Table-1 shape as a full stack: batch 8, every sequence at 4095 cached tokens, one step
        dm = TABLE1[name]
        return Workload(name, dm, dm.n_layers, True, 8, (4095,) * 8, 4096, 1)
    raise KeyError(name)
