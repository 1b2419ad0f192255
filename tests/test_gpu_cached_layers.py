"""Config C2 (32 frames of 518x518, N = 43,968): the merge plan is computed at the first global
layer and reused by the next three (Sec. 3.4: indices are cached between recomputations), each
layer feeding the next through the residual.  Every layer's output is checked against the CPU
oracle applied to the GPU's own input of that layer with the cached plan, and the plan itself
against the oracle's plan on the first layer's features."""
import numpy as np
import pytest
import torch

import oracle as O
from synthdata import WORKLOADS, make_attention_weights, make_images, make_tokens
from helpers import bf16_bound, rel_err, to_f64

pytestmark = pytest.mark.gpu


def test_plan_cached_across_four_layers_c2():
    import paper_2512_04939_b200 as pkg

    wl = WORKLOADS["C2"]
    images = make_images(wl)
    tokens = make_tokens(wl, images)
    ctx = pkg.LiteVGGT(wl.frames, wl.grid_h, wl.grid_w, wl.merge_ratio, recompute_interval=wl.recompute_interval)
    x = tokens.cuda()
    grad = ctx.grad_map(images.cuda())
    plan = None
    rng = np.random.default_rng(11)
    m = ctx.n_merged
    rows = np.unique(np.concatenate([rng.choice(m, 40, replace=False), [0, m - 1]]))
    toks = np.unique(np.concatenate([rng.choice(ctx.n_tokens, 200, replace=False), [0, ctx.n_tokens - 1]]))
    builds = 0
    for layer in range(wl.global_layers):
        if ctx.should_refresh(plan, layer):
            plan = ctx.merge_plan(x, grad, plan)
            builds += 1
            ex = ctx.plan_export(plan)
            if layer == 0:
                # the plan against the oracle's on the same features
                ref = O.merge_plan(to_f64(tokens), O.grad_map(images.numpy()), wl.frames, wl.grid_h, wl.grid_w,
                                   merge_ratio=wl.merge_ratio)
                assert (ex["cls"] != ref["cls"]).mean() <= 1e-3
                if np.array_equal(ex["cls"], ref["cls"]):
                    margin = ref["best_sim"] - ref["second_sim"]
                    agree = ex["best_dst"] == ref["best_dst"]
                    assert np.all(agree[margin > 1e-3]) and agree.mean() >= 0.999
                    assert np.abs(ex["best_sim"] - ref["best_sim"]).max() <= 1e-5
                dst_of, size, kept = O.select_and_index(ex["cls"], ex["best_dst"], ex["best_sim"], ref["sizes"]["R"])
                assert np.array_equal(ex["dst_of"], dst_of) and np.array_equal(ex["size"], size)
        w = [t.cuda() for t in make_attention_weights(wl, layer)]
        xm = ctx.merge(plan, x)
        ym = ctx.global_attn(xm, *w)
        out = ctx.unmerge(plan, ym, x)
        ctx.poll()
        # oracle on this layer's GPU input with the cached indices (sampled outputs)
        x64 = to_f64(x)
        ref_m = O.merge(x64, ex["dst_of"], m)
        assert rel_err(to_f64(xm), ref_m) <= bf16_bound(ref_m), f"merge, layer {layer}"
        w64 = [to_f64(t) for t in w]
        ref_y = O.global_attention(to_f64(xm), *w64, heads=16, rows=rows)
        assert rel_err(to_f64(ym)[rows], ref_y) <= 2 * bf16_bound(ref_y), f"attention, layer {layer}"
        ref_out = O.unmerge(to_f64(ym), ex["dst_of"], x64)[toks]
        assert rel_err(to_f64(out)[toks], ref_out) <= bf16_bound(ref_out), f"unmerge, layer {layer}"
        # conservation of the size-weighted sum under the cached plan on drifting features
        lhs = (ex["size"][:, None] * ref_m).sum(0)
        np.testing.assert_allclose(lhs, x64.sum(0), rtol=0, atol=1e-6 * np.abs(x64).sum(0).max())
        x = out
    assert builds == 1  # four layers, interval 6: computed once, reused three times
    plan.destroy()
    ctx.close()
