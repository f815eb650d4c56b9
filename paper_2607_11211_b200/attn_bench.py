"""Times ``fasttps_attn_decode`` alone on one of the attention shapes the paper evaluates (its Table 1).

    python -m paper_2607_11211_b200.attn_bench --model llama3-8b --batch 8 --past 4095 [--gqa-share 0|1|2] [--n-new N] [--fp8]

The call is enqueued ``--iters`` times on one stream between two CUDA events, rotating over enough cache sets
that no K/V row is still in the L2 when it is read again.  Algorithmic bytes per call: every cached row of every
K/V head read once (K and V), the new rows written once, q and the output; with ``--gqa-share 0`` the kernel
reads a K/V head once per query head, and the same algorithmic bytes are charged.  ``--fp8``: the caches hold 8-bit
E4M3 codes (``fasttps_attn_decode_fp8``), one byte per cached element.  Prints one JSON line.
"""
import argparse
import json
from pathlib import Path

import numpy as np
import torch

from . import binding as fb, build, workload as wl

# (query heads, K/V heads, head_dim): the five rows of the paper's Table 1
SHAPES = {"llama3-8b": (32, 8, 128), "chatglm3-6b": (32, 2, 128), "llama2-7b": (32, 32, 128),
          "phi3-mini": (32, 32, 96), "llama3.2-1b": (32, 32, 64)}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--model", default="llama3-8b", choices=sorted(SHAPES))
    ap.add_argument("--batch", type=int, default=8)
    ap.add_argument("--past", type=int, default=4095, help="cached rows per sequence before the step")
    ap.add_argument("--iters", type=int, default=200)
    ap.add_argument("--gqa-share", type=int, default=1)
    ap.add_argument("--n-new", type=int, default=1,
                    help="new tokens per sequence and step (> 1: fasttps_attn_decode_multi, causal inside the chunk)")
    ap.add_argument("--fp8", action="store_true", help="KV cache of 8-bit E4M3 codes (fasttps_attn_decode_fp8)")
    args = ap.parse_args()
    if args.fp8 and args.n_new != 1:
        raise SystemExit("--fp8 times the one-token step")
    if not torch.cuda.is_available():
        raise SystemExit("needs a CUDA device: there is no CPU path")
    build.build()
    hq, hkv, d = SHAPES[args.model]
    dims = wl.Dims(hidden=hq * d, n_q_heads=hq, n_kv_heads=hkv, head_dim=d, inter=1024, vocab=1024, n_layers=1)
    B, L, N = args.batch, args.past, args.n_new
    max_seq = L + N
    ctx = fb.Context.from_dims(dims, B * N, max_seq)
    ctx.set_option("gqa_share", args.gqa_share)
    eb = 1 if args.fp8 else 2                                        # bytes per cached element
    k_scale, v_scale = 1.0 / 16, 1.0 / 16
    cache_bytes = 2 * B * hkv * max_seq * d * eb
    n_sets = max(2, -(-(400 << 20) // cache_bytes))                  # > 3 x the 126 MB L2 between two visits
    if args.fp8:
        sets = [wl.kv_cache_e4m3(dims, i, B, max_seq, k_scale, v_scale, wl.MASTER_SEED, device="cuda") for i in range(n_sets)]
    else:
        sets = [wl.kv_cache(dims, i, B, max_seq, wl.MASTER_SEED, device="cuda") for i in range(n_sets)]
    act = wl.activations(dims, B * N, wl.MASTER_SEED, device="cuda")
    if N > 1:
        act = {k: v.view(B, N, *v.shape[1:]) for k, v in act.items()}
    lens = torch.full((B,), L, dtype=torch.int32, device="cuda")
    out = torch.zeros(B * N, hq, d, dtype=torch.bfloat16, device="cuda").view(*act["q"].shape)
    torch.cuda.synchronize()
    st = torch.cuda.Stream()

    def run(n):
        for i in range(n):
            kc, vc = sets[i % n_sets]
            if args.fp8:
                ctx.attn_decode_fp8(act["q"], act["k_new"], act["v_new"], kc, vc, k_scale, v_scale, lens, lens, out, stream=st)
            elif N > 1:
                ctx.attn_decode_multi(act["q"], act["k_new"], act["v_new"], kc, vc, lens, lens, out, stream=st)
            else:
                ctx.attn_decode(act["q"], act["k_new"], act["v_new"], kc, vc, lens, lens, out, stream=st)

    with torch.cuda.stream(st):
        run(2 * n_sets)
        st.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(st)
        run(args.iters)
        e1.record(st)
        st.synchronize()
    us = e0.elapsed_time(e1) / args.iters * 1e3
    status = ctx.get_status()
    # every cached row once (whatever the number of new tokens), the new rows written, q in, the output out
    alg = 2 * B * hkv * (L + N) * d * eb + 2 * B * N * hq * d * 2
    peaks = Path(__file__).resolve().parent.parent / "MEASURED_PEAKS.json"
    peak = float(json.loads(peaks.read_text())["hbm_gbs"]) if peaks.exists() else 6650.0
    gbs = alg / (us * 1e-6) / 1e9
    print(json.dumps({"kernel": "attn_decode_kernel", "model": args.model, "q_heads": hq, "kv_heads": hkv, "head_dim": d,
                      "batch": B, "past": L, "n_new": N, "kv_dtype": "e4m3" if args.fp8 else "bf16", "gqa_share": args.gqa_share, "cache_sets": n_sets, "iters": args.iters,
                      "us_per_call": us, "algorithmic_bytes": alg, "achieved_gbs": gbs, "peak_gbs": peak,
                      "frac": gbs / peak, "peak_source": "of measured" if peaks.exists() else "of fallback",
                      "device_status": status}))
    ctx.close()


if __name__ == "__main__":
    main()
