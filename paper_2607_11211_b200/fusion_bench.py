"""Fused against non-fused token phase on this GPU: the paper's Section 5.1-5.3 experiments (its Fig. 5, Fig. 6 and
Table 3) restated for one decoder layer of the Phi-3-mini shape.

    python -m paper_2607_11211_b200.fusion_bench [--batch 1] [--iters 50]

For N_t = 256 ... 4096 attended rows it times (CUDA events on the launch stream, rotating over enough cache sets that
nothing is still in the L2 when it is read again):
  * the fused attention, fasttps_attn_decode (Algorithm 3: joint RoPE, in-place append, QK^T, softmax, PV in one
    kernel), and the non-fused attention of include/fasttps_baseline.h (Algorithm 1: ten launches, with a Concat that
    copies the whole cache), as a whole and per operator -- the share of Concat is the paper's headline observation;
  * once, the fused MLP, fasttps_mlp_decode (Algorithm 4), and the non-fused MLP (Algorithm 2: five launches).
Prints one JSON line.
"""
import argparse
import json

import numpy as np
import torch

from . import binding as fb, build, workload as wl

OPS = ["rope_q", "rope_k", "transpose_q", "transpose_k", "transpose_v", "concat_k", "concat_v", "qk", "softmax", "pv"]


def timed(st, fn, iters):
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(st):
        fn(3)
        st.synchronize()
        e0.record(st)
        fn(iters)
        e1.record(st)
        st.synchronize()
    return e0.elapsed_time(e1) / iters * 1e3


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--batch", type=int, default=1)
    ap.add_argument("--iters", type=int, default=50)
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("needs a CUDA device: there is no CPU path")
    build.build()
    dims, B = wl.PHI3_MINI, args.batch
    st = torch.cuda.Stream()
    rows = []
    for n_t in (256, 512, 1024, 2048, 4096):
        L, max_seq = n_t - 1, n_t
        ctx = fb.Context.from_dims(dims, B, max_seq)
        cache_bytes = 2 * B * dims.n_kv_heads * max_seq * dims.head_dim * 2
        n_sets = max(2, -(-(400 << 20) // cache_bytes))
        sets = [wl.kv_cache(dims, i, B, max_seq, device="cuda") for i in range(n_sets)]
        act = wl.activations(dims, B, device="cuda")
        lens = torch.full((B,), L, dtype=torch.int32, device="cuda")
        out = torch.zeros(B, dims.n_q_heads, dims.head_dim, dtype=torch.bfloat16, device="cuda")
        torch.cuda.synchronize()            # the inputs were made on the default stream; the calls below use `st`

        def fused(n):
            for i in range(n):
                kc, vc = sets[i % n_sets]
                ctx.attn_decode(act["q"], act["k_new"], act["v_new"], kc, vc, lens, lens, out, stream=st)

        def non_fused(n):
            for i in range(n):
                kc, vc = sets[i % n_sets]
                fb.baseline_attn(act["q"], act["k_new"], act["v_new"], kc, vc, lens, lens, out, n_t, dims.rope_theta, stream=st)

        us_f = timed(st, fused, args.iters)
        us_b = timed(st, non_fused, args.iters)
        per_op = np.zeros(10)
        with torch.cuda.stream(st):
            for i in range(8):
                kc, vc = sets[i % n_sets]
                per_op += np.array(fb.baseline_attn(act["q"], act["k_new"], act["v_new"], kc, vc, lens, lens, out, n_t,
                                                    dims.rope_theta, timed=True, stream=st)[2])
        per_op /= 8
        rows.append({"n_t": n_t, "fused_us": us_f, "non_fused_us": us_b, "speedup": us_b / us_f,
                     "concat_share_of_non_fused": float((per_op[5] + per_op[6]) / per_op.sum()),
                     "per_operator_us": {k: float(v) for k, v in zip(OPS, per_op)}})
        status = ctx.get_status()
        assert status == 0, f"device status {status} at n_t = {n_t}"
        ctx.close()
        del sets
        torch.cuda.empty_cache()

    # ---- MLP ----
    ctx = fb.Context.from_dims(dims, B, 64)
    n_sets = 6                                                                  # 6 x 151 MB of weights
    ws = [wl.layer_weights(dims, i, device="cuda") for i in range(n_sets)]
    packed = [(ctx.pack_weight(fb.W_GATE_UP, w["w_gu"]), ctx.pack_weight(fb.W_DOWN, w["w_down"])) for w in ws]
    K = dims.inter
    plain = [(w["w_gu"][:, :K].t().contiguous(), w["w_gu"][:, K:].t().contiguous(), w["w_down"].t().contiguous()) for w in ws]
    del ws
    x = wl.activations(dims, B, device="cuda")["x"]
    y = torch.zeros_like(x)
    torch.cuda.synchronize()

    def mlp_fused(n):
        for i in range(n):
            ctx.mlp_decode(x, packed[i % n_sets][0], packed[i % n_sets][1], y, stream=st)

    def mlp_non_fused(n):
        for i in range(n):
            fb.baseline_mlp(x, *plain[i % n_sets], y, stream=st)

    mlp = {"fused_us": timed(st, mlp_fused, args.iters), "non_fused_us": timed(st, mlp_non_fused, args.iters)}
    mlp["speedup"] = mlp["non_fused_us"] / mlp["fused_us"]
    with torch.cuda.stream(st):
        mlp["per_operator_us"] = dict(zip(["gate", "silu", "up", "mul", "down"],
                                          [float(v) for v in fb.baseline_mlp(x, *plain[1], y, timed=True, stream=st)]))
    print(json.dumps({"shape": "phi3-mini layer", "batch": B, "attention": rows, "mlp": mlp}))
    ctx.close()


if __name__ == "__main__":
    main()
