"""The seeded input generator: deterministic, sliceable, right shapes and moments."""
from pathlib import Path

import numpy as np
import torch

from paper_2607_11211_b200 import workload as wl


def test_generator_is_counter_based_and_deterministic():
    a = wl.normal_f32(wl.MASTER_SEED, 5, 0, 5000)
    b = wl.normal_f32(wl.MASTER_SEED, 5, 1234, 100)
    assert torch.equal(a[1234:1334], b)
    assert not torch.equal(a[:100], wl.normal_f32(wl.MASTER_SEED, 6, 0, 100))
    assert not torch.equal(a[:100], wl.normal_f32(wl.MASTER_SEED + 1, 5, 0, 100))
    t = wl.normal_bf16(1, 2, (7, 33), 0.02, chunk=50)
    assert torch.equal(t, wl.normal_bf16(1, 2, (7, 33), 0.02))


def test_generator_matches_a_scalar_python_evaluation():
    M = 2 ** 64 - 1

    def mix(x):
        x = ((x ^ (x >> 30)) * 0xBF58476D1CE4E5B9) & M
        x = ((x ^ (x >> 27)) * 0x94D049BB133111EB) & M
        return x ^ (x >> 31)

    seed, tid = 20260711, 1002
    key = (seed * 0x9E3779B97F4A7C15 + tid * 0xD1B54A32D192ED03 + 0x2545F4914F6CDD1D) & M
    got = wl.normal_f32(seed, tid, 0, 70000)
    for i in (0, 1, 77, 65535, 69999):
        tot = 0
        for j in range(2):
            h = mix(((i * 2 + j) * 0x9E3779B97F4A7C15 + key) & M)
            tot += sum((h >> s) & 0xFFFF for s in (0, 16, 32, 48))
        assert got[i].item() == float(np.float32(tot - 262140) * np.float32(wl._IH_INV_STD))


def test_moments_and_recipes():
    z = wl.normal_f32(3, 4, 0, 1 << 20).double()
    assert abs(z.mean()) < 5e-3 and abs(z.std() - 1) < 5e-3 and z.abs().max() < 4.9
    w = wl.layer_weights(wl.TINY, 0)
    assert w["w_qkv"].shape == (128, 384) and w["w_gu"].shape == (128, 256) and w["w_down"].shape == (128, 128)
    assert abs(w["w_gu"].float().std() - 0.02) < 2e-3
    assert abs(w["g_attn"].float().mean() - 1.0) < 2e-2
    L = wl.ragged_lengths(8, 512, 4096)
    assert L.min() >= 512 and L.max() <= 4096 and (L == wl.ragged_lengths(8, 512, 4096)).all()


def test_phi3_shape_matches_table1_and_byte_counts():
    rows = [l.split() for l in (Path(__file__).parent / "golden" / "table1_model_configs.txt").read_text().splitlines()
            if l and not l.startswith("#")]
    phi = next(r for r in rows if r[0].startswith("Phi3"))
    P = wl.PHI3_MINI
    assert [P.n_q_heads, P.n_kv_heads, P.head_dim, P.inter] == [int(v) for v in phi[1:]]
    assert P.hidden == P.n_q_heads * P.head_dim == 3072
    assert P.layer_weight_bytes == 226_492_416 + 12_288
    assert P.kv_bytes_per_token_per_layer == 12_288
    w1 = wl.workload("cfg1")
    assert w1.algorithmic_bytes() == 226_504_704 + 12_288 * 257 + 12_288
    assert wl.workload("cfg2").algorithmic_bytes() == 226_504_704 + 12_288 * 4096 + 12_288
