"""Parity at the large configurations - C3 (200 frames), C4 (500 frames, every src token merged)
and C5 (1000 frames, N = 1,041,000 tokens, M = 520,500 merged rows, the configuration bench.py
times): one pass of the whole path on the GPU, then every step checked against the CPU oracle on
sampled outputs that the oracle can compute one by one (it is fed the GPU's own upstream result,
so each step is judged in isolation), plus the properties that hold at any size.  Tolerances are
those of the small-size parity tests."""
import numpy as np
import pytest
import torch

import oracle as O
from synthdata import WORKLOADS, make_attention_weights, make_block_weights, make_images, make_tokens
from helpers import bf16_bound, rel_err, to_f64

pytestmark = pytest.mark.gpu

@pytest.fixture(scope="module", params=["C3", "C4", "C5"])
def run(request):
    import paper_2512_04939_b200 as pkg

    wl = WORKLOADS[request.param]
    images = make_images(wl, "cuda")
    tokens = make_tokens(wl, images)
    ctx = pkg.LiteVGGT(wl.frames, wl.grid_h, wl.grid_w, wl.merge_ratio)
    weights = [t.cuda() for t in make_attention_weights(wl, 0)]
    grad = ctx.grad_map(images)
    plan = ctx.merge_plan(tokens, grad)
    xm = ctx.merge(plan, tokens)
    ym = ctx.global_attn(xm, *weights)
    out = ctx.unmerge(plan, ym, tokens)
    gathered = ctx.unmerge(plan, ym)
    ctx.poll()
    frames_sampled = (0, 1, (3 * wl.frames) // 8 + 2, wl.frames - 1)
    r = dict(frames_sampled=frames_sampled, wl=wl, ctx=ctx, images=images, tokens=tokens, weights=weights, grad=grad, plan=plan, xm=xm, ym=ym,
             out=out, gathered=gathered, ex=ctx.plan_export(plan), sizes=O.derived_sizes(
                 wl.frames, wl.grid_h, wl.grid_w, merge_ratio=wl.merge_ratio))
    yield r
    plan.destroy()
    ctx.close()
    del r
    torch.cuda.empty_cache()


def test_sizes_and_index_invariants(run):
    ex, sz, ctx = run["ex"], run["sizes"], run["ctx"]
    assert (ctx.n_tokens, ctx.n_merged, ctx.n_src, ctx.n_dst) == (sz["N"], sz["M"], sz["n_src"], sz["n_dst"])
    assert int(ex["size"].sum()) == sz["N"] and ex["size"].min() >= 1
    assert np.all(np.diff(ex["kept_idx"]) > 0)
    assert np.array_equal(ex["dst_of"][ex["kept_idx"]], np.arange(sz["M"]))
    assert ex["dst_of"].min() == 0 and ex["dst_of"].max() == sz["M"] - 1
    assert np.array_equal(np.bincount(ex["dst_of"], minlength=sz["M"]), ex["size"])
    # merged-away tokens are src tokens and point at rows owned by anchors
    kept = np.zeros(sz["N"], bool)
    kept[ex["kept_idx"]] = True
    assert np.all(ex["cls"][~kept] == O.CLS_SRC) and (~kept).sum() == sz["R"]
    owners = ex["kept_idx"][ex["dst_of"][~kept]]
    assert np.all(ex["cls"][owners] == O.CLS_DST)


def test_grad_var_ga_maps_on_sampled_frames(run):
    wl, ex = run["wl"], run["ex"]
    t = wl.tokens_per_frame
    grad_gpu = to_f64(run["grad"])
    for f in run["frames_sampled"]:
        ref_g = O.grad_map(run["images"][f:f + 1].cpu().numpy())[0]
        assert np.abs(grad_gpu[f] - ref_g).max() <= 1e-5 * max(ref_g.max(), 1e-3)
        ref_v = O.var_map(to_f64(run["tokens"][f * t:(f + 1) * t]), 1, wl.grid_h, wl.grid_w)[0]
        assert np.abs(ex["var"][f] - ref_v).max() <= 2e-5 * ref_v.max()
        ref_ga = O.ga_map(grad_gpu[f:f + 1], ex["var"][f:f + 1].astype(np.float64))[0]
        assert np.abs(ex["ga"][f] - ref_ga).max() <= 1e-5


def test_partition_counts_everywhere_and_classes_on_sampled_frames(run):
    wl, ex, sz = run["wl"], run["ex"], run["sizes"]
    per_frame = ex["cls"].reshape(wl.frames, wl.tokens_per_frame)
    assert np.all(per_frame[:, :5] == O.CLS_PROTECTED) and np.all(per_frame[0, 5:] == O.CLS_DST)
    rest = per_frame[1:, 5:]
    assert np.all((rest == O.CLS_DST).sum(1) == sz["n_dst_frame"])
    assert np.all((rest == O.CLS_GA).sum(1) == sz["n_ga_frame"])
    assert np.all((rest == O.CLS_SRC).sum(1) == sz["n_src_frame"])
    # exactly one anchor per (clipped) 2x2 cell in every frame but the first
    grid = (rest == O.CLS_DST).reshape(wl.frames - 1, wl.grid_h, wl.grid_w)
    pad = np.zeros((wl.frames - 1, wl.grid_h + wl.grid_h % 2, wl.grid_w + wl.grid_w % 2), bool)
    pad[:, :wl.grid_h, :wl.grid_w] = grid
    cells = pad.reshape(wl.frames - 1, pad.shape[1] // 2, 2, pad.shape[2] // 2, 2).sum(axis=(2, 4))
    assert np.all(cells == 1)
    for f in run["frames_sampled"][1:]:
        # the oracle's partition of the GPU's own GA map: classes may differ only at near-ties
        ga = ex["ga"][f:f + 1].astype(np.float64)
        # (the oracle treats the first frame of its input as the all-anchor frame: put a copy in front)
        ref = O.partition(np.concatenate([ga, ga]))[wl.tokens_per_frame:]
        diff = np.flatnonzero(per_frame[f] != ref)
        flat = ga.reshape(-1)
        for i in diff:
            others = np.delete(flat, i - 5)
            assert np.abs(others - flat[i - 5]).min() < 1e-5, "class differs without a near-tie"
        assert diff.size <= 4


def test_matches_on_sampled_src_rows(run):
    ex, tokens = run["ex"], run["tokens"]
    src_idx = np.flatnonzero(ex["cls"] == O.CLS_SRC)
    dst_idx = np.flatnonzero(ex["cls"] == O.CLS_DST)
    rng = np.random.default_rng(5)
    rows = np.sort(rng.choice(src_idx.size, 48, replace=False))
    # compact copy: anchors first, then the sampled src rows
    xd = to_f64(tokens[torch.from_numpy(dst_idx).cuda()])
    xs = to_f64(tokens[torch.from_numpy(src_idx[rows]).cuda()])
    x_small = np.concatenate([xd, xs])
    best, sim1, sim2 = O.match(x_small, dst_idx.size + np.arange(rows.size), np.arange(dst_idx.size))
    best_token = dst_idx[best]
    margin = sim1 - sim2
    agree = ex["best_dst"][rows] == best_token
    assert np.all(agree[margin > 1e-3]), "argmax differs although the oracle's margin exceeds 1e-3"
    assert np.abs(ex["best_sim"][rows] - sim1).max() <= 1e-5
    assert agree.mean() >= 0.9  # the full-population bound (99.9 %) is checked at the small sizes


def test_selection_and_index_arrays_bit_exact_given_the_matches(run):
    ex, sz = run["ex"], run["sizes"]
    dst_of, size, kept = O.select_and_index(ex["cls"], ex["best_dst"], ex["best_sim"], sz["R"])
    assert np.array_equal(ex["dst_of"], dst_of)
    assert np.array_equal(ex["size"], size)
    assert np.array_equal(ex["kept_idx"], kept)


def test_merge_and_unmerge_on_sampled_rows(run):
    ex, tokens, xm, sz = run["ex"], run["tokens"], run["xm"], run["sizes"]
    order = np.argsort(ex["dst_of"], kind="stable")
    starts = np.concatenate([[0], np.cumsum(ex["size"])])
    rng = np.random.default_rng(6)
    rows = np.unique(np.concatenate([rng.choice(sz["M"], 160, replace=False), np.argsort(ex["size"])[-16:],
                                     [0, sz["M"] - 1]]))
    ref = np.empty((rows.size, 1024))
    for k, j in enumerate(rows):
        members = order[starts[j]:starts[j + 1]]
        ref[k] = to_f64(tokens[torch.from_numpy(members).cuda()]).mean(axis=0)
    got = to_f64(xm[torch.from_numpy(rows).cuda()])
    assert rel_err(got, ref) <= bf16_bound(ref)
    single = ex["size"][rows] == 1
    assert np.array_equal(got[single], ref[single])  # untouched rows are bit-exact copies
    # unmerge: the gather is exact; with the residual one fp32 add and one rounding
    tok = np.unique(np.concatenate([rng.choice(sz["N"], 256, replace=False), [0, sz["N"] - 1]]))
    tok_t = torch.from_numpy(tok).cuda()
    ym_rows = to_f64(run["ym"][torch.from_numpy(ex["dst_of"][tok].astype(np.int64)).cuda()])
    assert np.array_equal(to_f64(run["gathered"][tok_t]), ym_rows)
    ref_out = ym_rows + to_f64(tokens[tok_t])
    assert rel_err(to_f64(run["out"][tok_t]), ref_out) <= bf16_bound(ref_out)


def test_attention_layer_on_sampled_rows(run):
    ctx, xm, sz = run["ctx"], run["xm"], run["sizes"]
    w_qkv, b_qkv, w_o, b_o = [to_f64(t) for t in run["weights"]]
    m = sz["M"]
    rng = np.random.default_rng(7)
    rows = np.unique(np.concatenate([rng.choice(m, 24, replace=False), [0, 127, 128, m - 1]]))
    rows_t = torch.from_numpy(rows).cuda()
    qkv_gpu = ctx.debug_buffer(0)
    o_gpu = ctx.debug_buffer(1)
    # projections on the sampled rows
    ref_qkv = O.linear(to_f64(xm[rows_t]), w_qkv, b_qkv)
    assert rel_err(to_f64(qkv_gpu[rows_t]), ref_qkv) <= bf16_bound(ref_qkv), "qkv projection"
    o_rows = to_f64(o_gpu[rows_t])
    ref_y = O.linear(o_rows, w_o, b_o)
    assert rel_err(to_f64(run["ym"][rows_t]), ref_y) <= bf16_bound(ref_y), "output projection"
    # attention core: the sampled queries against all M keys, three heads, one head at a time
    # (the oracle is called with heads=1 on that head's [Q | K | V] columns)
    for head in (0, 6, 15):
        cols = torch.arange(64, device="cuda") + 64 * head
        q = to_f64(qkv_gpu[:, cols])
        k = to_f64(qkv_gpu[:, 1024 + cols])
        v = to_f64(qkv_gpu[:, 2048 + cols])
        ref_o = O.attention_core(np.concatenate([q, k, v], axis=1), heads=1, rows=rows)
        weighted_abs = O.attention_core(np.concatenate([q, k, np.abs(v)], axis=1), heads=1, rows=rows)
        rms = float(np.sqrt(np.mean(ref_o * ref_o)))
        # Output rounding + bf16 probabilities (2^-8 * sum p|v| / sum p), as in the small-size test.
        # With so few sampled outputs the rounding term is the worst case for their magnitudes
        # (half a bf16 ulp) rather than the rounding error the reference values happen to have.
        half_ulp = float((2.0 ** (np.floor(np.log2(np.maximum(np.abs(ref_o), 1e-30))) - 8)).max()) / rms
        bound = max(1e-2, half_ulp + 2e-3) + 2.0 ** -8 * float(weighted_abs.max()) / rms
        assert rel_err(o_rows[:, 64 * head:64 * head + 64], ref_o) <= bound, f"attention core, head {head}"


def test_block_sublayers_on_sampled_rows_and_frames(run):
    """LayerNorm, frame-local attention and the MLP at N = 1,041,000 rows: sampled rows / whole sampled
    frames against the oracle, each fed the GPU's own upstream result."""
    ctx, wl, tokens = run["ctx"], run["wl"], run["tokens"]
    w = make_block_weights(wl, 0, "cuda")
    rng = np.random.default_rng(8)
    rows = np.unique(np.concatenate([rng.choice(wl.n_tokens, 96, replace=False), [0, wl.n_tokens - 1]]))
    rows_t = torch.from_numpy(rows).cuda()
    xn = ctx.layernorm(tokens, *w["ln1"], eps=1e-6)
    ref_n = O.layernorm(to_f64(tokens[rows_t]), to_f64(w["ln1"][0]), to_f64(w["ln1"][1]), 1e-6)
    assert rel_err(to_f64(xn[rows_t]), ref_n) <= bf16_bound(ref_n)
    y = ctx.frame_attn(xn, *w["attn"], residual=tokens)
    z = ctx.mlp(xn, *w["mlp"], residual=tokens)
    ctx.poll()
    t = wl.tokens_per_frame
    aw = [to_f64(u) for u in w["attn"]]
    for f in (0, wl.frames // 2 + 12, wl.frames - 1):
        sl = slice(f * t, (f + 1) * t)
        ref_y = O.frame_attention(to_f64(xn[sl]), 1, *aw, heads=16, residual=to_f64(tokens[sl]))
        assert rel_err(to_f64(y[sl]), ref_y) <= 2 * bf16_bound(ref_y), f"frame attention, frame {f}"
    ref_z = O.mlp(to_f64(xn[rows_t]), *[to_f64(u) for u in w["mlp"]], residual=to_f64(tokens[rows_t]))
    assert rel_err(to_f64(z[rows_t]), ref_z) <= 2 * bf16_bound(ref_z)


def test_qk_norm_and_rope_on_sampled_rows(run):
    """The optional Q/K normalisation and rotary embedding at full size: the transformed Q and K of
    sampled merged rows (first, last, tile edges, random) against the oracle on those rows, positions
    taken from the owner tokens.  Runs last in this module: it overwrites the layer's intermediates."""
    ctx, xm, sz, wl, ex = run["ctx"], run["xm"], run["sizes"], run["wl"], run["ex"]
    w_qkv, b_qkv, w_o, b_o = run["weights"]
    gen = torch.Generator().manual_seed(wl.seed + 77)
    affine = [(1.0 + 0.2 * torch.randn(64, generator=gen)).to(torch.bfloat16) if i % 2 == 0
              else (0.2 * torch.randn(64, generator=gen)).to(torch.bfloat16) for i in range(4)]
    dev = [t.cuda() for t in affine]
    y = ctx.global_attn_ext(run["plan"], xm, w_qkv, b_qkv, w_o, b_o, q_norm=(dev[0], dev[1]), k_norm=(dev[2], dev[3]),
                            rope=True)
    ctx.poll()
    m = sz["M"]
    rng = np.random.default_rng(13)
    rows = np.unique(np.concatenate([rng.choice(m, 200, replace=False), [0, 7, 8, 127, 128, m - 8, m - 1]]))
    rows_t = torch.from_numpy(rows).cuda()
    ref = O.linear(to_f64(xm[rows_t]), to_f64(w_qkv), to_f64(b_qkv))
    pos = O.token_positions(wl.frames, wl.grid_h, wl.grid_w)[ex["kept_idx"][rows]]
    got = to_f64(ctx.debug_buffer(0)[rows_t])
    for name, c0, g, b in (("Q", 0, affine[0], affine[1]), ("K", 1024, affine[2], affine[3])):
        part = ref[:, c0:c0 + 1024].reshape(len(rows), 16, 64)
        part = O.rope_2d(O.qk_norm(part, to_f64(g), to_f64(b), 1e-5), pos, 100.0).reshape(len(rows), 1024)
        assert rel_err(got[:, c0:c0 + 1024], part) <= 2 * bf16_bound(part), name
    assert rel_err(got[:, 2048:], ref[:, 2048:]) <= bf16_bound(ref[:, 2048:]), "V is only projected"
    ref_y = O.linear(to_f64(ctx.debug_buffer(1)[rows_t]), to_f64(w_o), to_f64(b_o))
    assert rel_err(to_f64(y[rows_t]), ref_y) <= bf16_bound(ref_y), "output projection"
