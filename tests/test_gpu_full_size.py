"""Parity at the benchmark's full sizes, in the launch configuration `bench.py` times: the 32-layer
Phi-3-mini-shaped stack at batch 1 from a 1024-token cache (cfg3) and at batch 8 with ragged lengths (cfg4),
through the persistent step kernel (the library's default model path), and the batch-32 workload with every
cache filled to its last row (cfg5, cut to 1 and 2 layers) through the per-product kernels that serve batches above 8.

Checked against the oracle on the same seeded inputs: the logits of the step, the argmax wherever the
oracle's top-2 gap is beyond doubt, the appended K/V rows of every layer, and — on the device, over all 3.3 G
(cfg3) / 13 G (cfg4) cache elements — that nothing but the appended rows changed, bit for bit.  For cfg3 a
multi-token greedy launch is compared with the oracle's greedy loop as well.

Two depths.  With 1 layer (full width, full vocabulary, every CTA busy) the per-element output bar
|gpu - oracle| <= 2e-2 + 2e-2 |oracle| applies as it does to a single block (it is met with a margin of two
orders of magnitude in rms; already at 2 layers one logit in a million of the batch-32 case lands 4 % outside
it).  With more layers the two sides
run freely, and so would any two correct implementations: each rounds the residual stream and the branch
tensors to bf16 several times per layer; where an FP32 sum and a double sum differ they round to neighbouring
values, and these one-ulp differences are amplified by every layer that follows.  Measured on this workload the
relative rms difference of the logits grows smoothly with depth (1 layer 8e-5, 2: 1.5e-3, 4: 4e-3, 8: 8e-3,
16: 1.5e-2, 32: 2.4e-2), and the library's two model paths, which differ from each other only in summation
order, drift apart by as much (2.2e-2 at 32 layers) as either drifts from the oracle.  The bar for the
free-running full depth is therefore statistical: rms(gpu - oracle) <= 5e-2 rms(oracle), no element further off
than 0.25 + 5e-2 |oracle|, and the argmax equal wherever the oracle's top-2 gap is beyond that doubt.
"""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2607_11211_b200 import workload as wl
from tests.helpers import from_bf16_bits as F32

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def fb():
    from paper_2607_11211_b200 import binding, build
    build.build()
    return binding


def i32(a):
    return torch.tensor(np.asarray(a, dtype=np.int32), device="cuda")


def sure_rows(wlog, deep=False):
    top2 = np.sort(wlog, axis=1)[:, -2:]
    bar = (0.25 + 5e-2 * np.abs(top2[:, 1])) if deep else (2e-2 + 2e-2 * np.abs(top2[:, 1]))
    return (top2[:, 1] - top2[:, 0]) > 2 * bar


def check(got, want, deep, what):
    got, want = np.asarray(got, np.float64), np.asarray(want, np.float64)
    bar = 2e-2 + 2e-2 * np.abs(want)
    if not deep:
        assert (np.abs(got - want) <= bar).all(), what
        return
    assert np.sqrt(np.mean((got - want) ** 2)) <= 5e-2 * np.sqrt(np.mean(want ** 2)), what
    assert (np.abs(got - want) <= 0.25 + 5e-2 * np.abs(want)).all(), what


@pytest.mark.parametrize("name,n_layers,greedy_steps", [("cfg3", 1, 3), ("cfg3", 32, 3), ("cfg4", 1, 0), ("cfg4", 32, 0),
                                                        ("cfg5", 1, 0), ("cfg5", 2, 0)])
def test_full_stack_at_benchmark_size(fb, name, n_layers, greedy_steps):
    import dataclasses
    W = wl.workload(name)
    deep = n_layers > 1
    W = dataclasses.replace(W, n_layers=n_layers, dims=dataclasses.replace(W.dims, n_layers=n_layers))
    dims, batch, max_seq = W.dims, W.batch, W.max_seq
    lens = np.asarray(W.past_lens, np.int32)
    ctx = fb.Context.from_dims(dims, batch, max_seq, n_layers=W.n_layers)
    mw = wl.model_weights(dims, device="cuda")
    packed = [ctx.pack_layer(w) for w in mw["layers"]]
    caches = [wl.kv_cache(dims, l, batch, max_seq, device="cuda") for l in range(W.n_layers)]
    kcs, vcs = [c[0] for c in caches], [c[1] for c in caches]
    model = ctx.make_model(mw["embed"], packed, mw["g_final"], ctx.pack_weight(fb.W_LM_HEAD, mw["w_lm"]), kcs, vcs)
    k0 = [t.clone() for t in kcs]
    v0 = [t.clone() for t in vcs]
    ids = wl.token_ids(batch, dims.vocab)

    # ---- one decode step, logits out ----
    pos, sl = i32(lens), i32(lens)
    logits = torch.zeros(batch, dims.vocab, dtype=torch.float32, device="cuda")
    nxt = torch.zeros(batch, dtype=torch.int32, device="cuda")
    ctx.model_decode(model, i32(ids), pos, sl, logits, nxt, advance=False)
    torch.cuda.synchronize()
    assert ctx.get_status() == 0

    # nothing but row L_b of every head changed, bit for bit (compared on the device)
    for l in range(W.n_layers):
        for new, old in ((kcs[l], k0[l]), (vcs[l], v0[l])):
            diff = new.view(torch.int16) != old.view(torch.int16)
            for b in range(batch):
                diff[b, :, int(lens[b]), :] = False
            assert not bool(diff.any()), (name, l)
    del k0, v0

    # ---- the oracle on the same inputs ----
    ok = [wl.bits(t) for t in kcs]
    ov = [wl.bits(t) for t in vcs]
    for l in range(W.n_layers):                       # undo the device's append in the oracle's copy: it appends itself
        for b in range(batch):
            ok[l][b, :, lens[b]] = 0
            ov[l][b, :, lens[b]] = 0
    ow = [{k: wl.bits(v) for k, v in L.items()} for L in mw["layers"]]
    emb, gf, wlm = wl.bits(mw["embed"]), wl.bits(mw["g_final"]), wl.bits(mw["w_lm"])
    cur = lens.copy()
    wlog, wnext = orc.model_decode(emb, ow, gf, wlm, ok, ov, ids, cur, cur, dims.rms_eps, dims.rope_theta)
    check(logits.cpu().numpy(), wlog, deep, "logits")
    sure = sure_rows(wlog, deep)
    g = nxt.cpu().numpy()
    assert (g[sure] == wnext[sure]).all()
    for l in range(W.n_layers):
        for b in range(batch):
            r = int(lens[b])
            check(F32(wl.bits(kcs[l][b, :, r])), F32(ok[l][b, :, r]), deep, f"k row, layer {l}")
            check(F32(wl.bits(vcs[l][b, :, r])), F32(ov[l][b, :, r]), deep, f"v row, layer {l}")

    # ---- several greedy tokens in one launch against the oracle's greedy loop ----
    if greedy_steps:
        out = torch.zeros(greedy_steps, batch, dtype=torch.int32, device="cuda")
        pos, sl = i32(lens), i32(lens)
        ctx.model_generate(model, i32(ids), pos, sl, out)
        torch.cuda.synchronize()
        assert ctx.get_status() == 0
        gids = out.cpu().numpy()
        tok, alive, compared = ids.copy(), np.ones(batch, bool), 0
        for s in range(greedy_steps):
            if s > 0:
                wlog, wnext = orc.model_decode(emb, ow, gf, wlm, ok, ov, tok, cur, cur, dims.rms_eps, dims.rope_theta)
            chk = alive & sure_rows(wlog, deep)
            assert (gids[s][chk] == wnext[chk]).all(), s
            compared += int(chk.sum())
            alive &= gids[s] == wnext
            tok = wnext.astype(np.int32)
            cur = cur + 1
        assert compared >= 1 or deep
        assert (sl.cpu().numpy() == lens + greedy_steps).all()
    ctx.close()
