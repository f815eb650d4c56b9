"""Phase timeline of the persistent decode-step kernel.

    python -m paper_2607_11211_b200.timeline [--batch 1] [--past 1024] [--layers 32] [--steps 4]

Runs a greedy multi-step decode of a Phi-3-mini-shaped stack (synthetic seeded weights and caches) in one
launch of the step kernel and prints, for the LAST step of the launch, how long the first and the last CTA
spent in each phase of a layer (QKV product, attention + output projection, fused MLP) and how long they then
waited at the grid-wide barrier that closes the phase.  The stamps come from fasttps_trace_read(): the two
CTAs read the GPU global timer immediately before and after every barrier.
"""
from __future__ import annotations

import argparse
import json

import numpy as np
import torch

from . import binding as fb, workload as wl


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--batch", type=int, default=1)
    ap.add_argument("--past", type=int, default=1024)
    ap.add_argument("--layers", type=int, default=32)
    ap.add_argument("--steps", type=int, default=4)
    args = ap.parse_args()
    dm, B, NL, NS = wl.PHI3_MINI, args.batch, args.layers, args.steps
    dev = torch.device("cuda", 0)
    max_seq = args.past + NS + 2
    ctx = fb.Context.from_dims(dm, B, max_seq, n_layers=NL)
    ctx.set_option("step_kernel", 1)
    names = ("qkv", "attn+o_proj", "mlp")                  # three phases per layer: attention and output projection are one
    P = len(names)
    seed = wl.MASTER_SEED
    layers = [ctx.pack_layer(wl.layer_weights(dm, i, seed, device=dev)) for i in range(NL)]
    caches = [wl.kv_cache(dm, i, B, max_seq, seed, device=dev) for i in range(NL)]
    embed = wl.normal_bf16(seed, wl.tid("embed"), (dm.vocab, dm.hidden), 0.02, device=dev)
    g_final = wl.normal_bf16(seed, wl.tid("g_final"), (dm.hidden,), 0.02, 1.0, device=dev)
    w_lm = ctx.pack_weight(fb.W_LM_HEAD, wl.normal_bf16(seed, wl.tid("w_lm"), (dm.vocab, dm.hidden), 0.02, device=dev))
    model = ctx.make_model(embed, layers, g_final, w_lm, [c[0] for c in caches], [c[1] for c in caches])
    tok = torch.tensor(wl.token_ids(B, dm.vocab, seed), device=dev)
    out = torch.zeros(NS, B, dtype=torch.int32, device=dev)
    ms = 0.0
    for _ in range(2):                                   # the second launch is the one reported
        pos = torch.full((B,), args.past, dtype=torch.int32, device=dev)
        sl = pos.clone()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        ctx.model_generate(model, tok, pos, sl, out)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1)
    status = ctx.get_status()
    first, last = ctx.trace_read()
    # stamps: 2 for the barrier after the embedding gather, then per step 2 per phase (P per layer + logits)
    # and 2 for the barrier that ends the step (absent after the last step)
    per_step = 2 * (P * NL + 2)
    report = {"batch": B, "past": args.past, "layers": NL, "steps": NS, "launch_ms": ms, "ms_per_step": ms / NS,
              "device_status": status}
    for name, stamps in (("first_cta", first), ("last_cta", last)):
        s = stamps.astype(np.int64)
        base = 2 + (NS - 1) * per_step
        st = s[base:base + per_step - 2]
        before, after = st[0::2], st[1::2]
        prev_after = np.concatenate([[s[base - 1]], after[:-1]])
        busy = (before - prev_after) / 1e3
        wait = (after - before) / 1e3
        b4, w4 = busy[:P * NL].reshape(NL, P), wait[:P * NL].reshape(NL, P)
        report[name] = {
            "step_us": float(st[-1] - s[base - 1]) / 1e3,
            "mean_busy_us": dict(zip(names, np.round(b4.mean(0), 2).tolist())),
            "mean_barrier_wait_us": dict(zip(names, np.round(w4.mean(0), 2).tolist())),
            "logits_busy_us": round(float(busy[P * NL]), 2), "logits_barrier_wait_us": round(float(wait[P * NL]), 2),
        }
    print(json.dumps(report, indent=1))
    ctx.close()


if __name__ == "__main__":
    main()
