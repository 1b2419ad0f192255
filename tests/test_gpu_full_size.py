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
from synthdata import (WORKLOADS, make_attention_weights, make_block_weights, make_images,
                       make_peaked_attention_inputs, make_tokens)
from helpers import CORE_NOISE, K_FOLD, LAYER_NOISE, bf16_bound, check_bf16, fold_k, rel_err, report, to_f64

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
    check_invariants(run, run["ex"])


def check_invariants(run, ex):
    sz, ctx = run["sizes"], run["ctx"]
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


def check_maps_on_sampled_frames(run, ex, tokens):
    """Grad map, Var map of `tokens` and GA map of the plan export `ex` on the sampled frames."""
    wl = run["wl"]
    t = wl.tokens_per_frame
    grad_gpu = to_f64(run["grad"])
    for f in run["frames_sampled"]:
        ref_g = O.grad_map(run["images"][f:f + 1].cpu().numpy())[0]
        assert np.abs(grad_gpu[f] - ref_g).max() <= 1e-5 * max(ref_g.max(), 1e-3)
        ref_v = O.var_map(to_f64(tokens[f * t:(f + 1) * t]), 1, wl.grid_h, wl.grid_w)[0]
        assert np.abs(ex["var"][f] - ref_v).max() <= 2e-5 * ref_v.max()
        ref_ga = O.ga_map(grad_gpu[f:f + 1], ex["var"][f:f + 1].astype(np.float64))[0]
        assert np.abs(ex["ga"][f] - ref_ga).max() <= 1e-5


def test_grad_var_ga_maps_on_sampled_frames(run):
    check_maps_on_sampled_frames(run, run["ex"], run["tokens"])


def test_partition_counts_everywhere_and_classes_on_sampled_frames(run):
    check_partition(run, run["ex"])


def check_partition(run, ex):
    wl, sz = run["wl"], run["sizes"]
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


N_MATCH_ROWS = 4096


def test_matches_on_sampled_src_rows(run):
    check_matches_on_sampled_src_rows(run, run["ex"], run["tokens"], run["wl"].name)


def check_matches_on_sampled_src_rows(run, ex, tokens, tag):
    """4096 seeded src rows against every anchor of the sequence (the oracle's match on a compact
    copy: anchors first, then the sampled rows).  The stated tolerance in full: the argmax equals the
    oracle's wherever the oracle's top-1 / top-2 margin exceeds 1e-3, at least 99.9 % of the rows agree,
    and a row that differs is a near-tie (its similarity within 1e-5 of the oracle's best).  The margin
    histogram and the agreement are reported with the result."""
    src_idx = np.flatnonzero(ex["cls"] == O.CLS_SRC)
    dst_idx = np.flatnonzero(ex["cls"] == O.CLS_DST)
    rng = np.random.default_rng(5)
    rows = np.sort(rng.choice(src_idx.size, min(N_MATCH_ROWS, src_idx.size), replace=False))
    xd = to_f64(tokens[torch.from_numpy(dst_idx).cuda()])
    xs = to_f64(tokens[torch.from_numpy(src_idx[rows]).cuda()])
    x_small = np.concatenate([xd, xs])
    del xd, xs
    best, sim1, sim2 = O.match(x_small, dst_idx.size + np.arange(rows.size), np.arange(dst_idx.size), chunk=512)
    best_token = dst_idx[best]
    margin = sim1 - sim2
    agree = ex["best_dst"][rows] == best_token
    report(f"{tag}: matching on {rows.size} sampled src rows x {dst_idx.size} anchors",
           agreement=float(agree.mean()), near_ties_accepted=int((~agree).sum()),
           margin_below_1e_5=float((margin < 1e-5).mean()), margin_below_1e_4=float((margin < 1e-4).mean()),
           margin_below_1e_3=float((margin < 1e-3).mean()), margin_median=float(np.median(margin)),
           best_sim_max_abs_diff=float(np.abs(ex["best_sim"][rows] - sim1).max()))
    assert np.all(agree[margin > 1e-3]), "argmax differs although the oracle's margin exceeds 1e-3"
    assert np.abs(ex["best_sim"][rows] - sim1).max() <= 1e-5
    assert agree.mean() >= 0.999


def test_selection_and_index_arrays_bit_exact_given_the_matches(run):
    check_index_arrays(run, run["ex"])


def check_index_arrays(run, ex):
    sz = run["sizes"]
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
    ref_qkv = fold_k(O.linear(to_f64(xm[rows_t]), w_qkv, b_qkv))
    check_bf16(f"{run['wl'].name}: qkv projection", to_f64(qkv_gpu[rows_t]), ref_qkv, sampled=True)
    o_rows = to_f64(o_gpu[rows_t])
    ref_y = O.linear(o_rows, w_o, b_o)
    check_bf16(f"{run['wl'].name}: output projection", to_f64(run["ym"][rows_t]), ref_y, sampled=True)
    # attention core: the sampled queries against all M keys, three heads, one head at a time
    # (the oracle is called with heads=1 on that head's [Q | K | V] columns)
    for head in (0, 6, 15):
        cols = torch.arange(64, device="cuda") + 64 * head
        q = to_f64(qkv_gpu[:, cols])
        k = to_f64(qkv_gpu[:, 1024 + cols]) / K_FOLD  # the library's K carries the softmax scale
        v = to_f64(qkv_gpu[:, 2048 + cols])
        ref_o = O.attention_core(np.concatenate([q, k, v], axis=1), heads=1, rows=rows)
        check_bf16(f"{run['wl'].name}: attention core, stock weights, head {head}", o_rows[:, 64 * head:64 * head + 64],
                   ref_o, sampled=True, elem_noise=CORE_NOISE)


def key_chunk_edges(m):
    """First key row of every key chunk but the first, as the attention launcher splits a long
    sequence: tiles of 128 keys, balanced chunks of at most 512 tiles."""
    n_tiles = -(-m // 128)
    n_chunks = -(-n_tiles // 512)
    per_chunk = -(-n_tiles // n_chunks)
    return [c * per_chunk * 128 for c in range(1, n_chunks)], per_chunk * 128


@pytest.mark.parametrize("name,sharpness", [("C3", 4.0), ("C4", 4.0), ("C5", 4.0), ("C3", 16.0), ("C5", 16.0)])
def test_attention_core_with_peaked_softmax_across_key_chunks(name, sharpness):
    """The attention core at the merged lengths of C3, C4 and C5 on inputs whose softmax is far from
    uniform: every query's mass sits on itself and on the ~M/4099 rows of its group, which lie 4099
    rows apart through the whole sequence, so every key chunk (C3: 2, C4: 4, C5: 8) carries a share of every
    output.  Sampled queries sit on both sides of every chunk boundary, at tile edges and at random.
    A chunk left out on the oracle's side must move the result far beyond the tolerance.
    Sharpness 4 keeps every row's score bound under the limit of the fixed softmax reference;
    sharpness 16 puts them over it, so the running-maximum form and its combination of chunks with
    different references are the ones under test."""
    import paper_2512_04939_b200 as pkg

    wl = WORKLOADS[name]
    ctx = pkg.LiteVGGT(wl.frames, wl.grid_h, wl.grid_w, wl.merge_ratio)
    m = ctx.n_merged
    x, w_qkv, b_qkv, w_o, b_o = make_peaked_attention_inputs(m, wl.seed + 9, "cuda", sharpness=sharpness)
    ctx.global_attn(x, w_qkv, b_qkv, w_o, b_o)
    ctx.poll()
    name = f"{name}, sharpness {sharpness:g}"
    edges, chunk_rows = key_chunk_edges(m)
    rng = np.random.default_rng(17)
    rows = [0, 127, 128, 255, 256, m - 129, m - 128, m - 1] + list(rng.choice(m, 16, replace=False))
    for e in edges:
        rows += [e - 129, e - 128, e - 1, e, e + 127, e + 128]
    rows = np.unique(np.asarray(rows, dtype=np.int64))
    rows_t = torch.from_numpy(rows).cuda()
    qkv_gpu, o_gpu = ctx.debug_buffer(0), ctx.debug_buffer(1)
    o_rows = to_f64(o_gpu[rows_t])
    for head in (0, 9, 15):
        cols = torch.arange(64, device="cuda") + 64 * head
        qkv_h = np.concatenate([to_f64(qkv_gpu[:, cols]), to_f64(qkv_gpu[:, 1024 + cols]) / K_FOLD,
                                to_f64(qkv_gpu[:, 2048 + cols])], axis=1)
        ref_o = O.attention_core(qkv_h, heads=1, rows=rows)
        got = o_rows[:, 64 * head:64 * head + 64]
        check_bf16(f"{name}: attention core, peaked softmax, head {head}", got, ref_o, sampled=True, elem_noise=CORE_NOISE)
        bound = bf16_bound(ref_o)
        # planted on the oracle's side: without the keys of chunk c (queries taken outside it)
        for c in range(len(edges) + 1):
            lo, hi = c * chunk_rows, min(m, (c + 1) * chunk_rows)
            outside = (rows < lo) | (rows >= hi)
            kept = np.concatenate([qkv_h[:lo], qkv_h[hi:]])
            if kept.shape[0] == 0:
                continue
            moved = np.where(rows[outside] >= hi, rows[outside] - (hi - lo), rows[outside])
            ref_short = O.attention_core(kept, heads=1, rows=moved)
            lost = rel_err(got[outside], ref_short)
            report(f"{name}: head {head}, oracle without key chunk {c}", err_over_rms=lost, bound=bound)
            # a chunk holds 1/8 (C5) to 1/2 (C3) of every row's mass: several times the tolerance
            assert lost > 5 * bound, f"dropping key chunk {c} on the oracle's side goes unnoticed"
            del kept
        del qkv_h
    ctx.close()
    del x
    torch.cuda.empty_cache()


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
    taken from the owner tokens.  Runs after the checks of the plain layer: it overwrites the layer's
    intermediates."""
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
        if name == "K":
            part = part * K_FOLD
        assert rel_err(got[:, c0:c0 + 1024], part) <= 2 * bf16_bound(part), name
    assert rel_err(got[:, 2048:], ref[:, 2048:]) <= bf16_bound(ref[:, 2048:]), "V is only projected"
    ref_y = O.linear(to_f64(ctx.debug_buffer(1)[rows_t]), to_f64(w_o), to_f64(b_o))
    assert rel_err(to_f64(y[rows_t]), ref_y) <= bf16_bound(ref_y), "output projection"


def test_plan_refreshed_in_place_on_the_layer_output(run):
    """Sec. 3.4, cached token merging at full size: the plan of the fixture is rebuilt IN PLACE (same
    handle, its index arrays reused) on the features the layer has produced - the residual stream one
    layer on, which is what a refresh layer of the schedule sees - and judged like the first build:
    Var / GA maps and classes on sampled frames, matching on 4096 sampled src rows against all
    anchors, selection and index arrays bit-exact given the matches, and the merge under the new plan
    on sampled rows.  Last user of the fixture's plan."""
    ctx, plan, wl, sz = run["ctx"], run["plan"], run["wl"], run["sizes"]
    x2 = run["out"]
    handle = plan.handle.value
    assert ctx.merge_plan(x2, run["grad"], plan).handle.value == handle
    xm2 = ctx.merge(plan, x2)
    ctx.poll()
    ex2 = ctx.plan_export(plan)
    moved = float((ex2["dst_of"] != run["ex"]["dst_of"]).mean())
    report(f"{wl.name}: plan refreshed in place on the layer output", tokens_with_another_row=moved,
           classes_changed=float((ex2["cls"] != run["ex"]["cls"]).mean()))
    assert moved > 0.0, "the refresh changed nothing: the drifted features were not used"
    check_invariants(run, ex2)
    check_maps_on_sampled_frames(run, ex2, x2)
    check_partition(run, ex2)
    check_matches_on_sampled_src_rows(run, ex2, x2, f"{wl.name} refreshed")
    check_index_arrays(run, ex2)
    order = np.argsort(ex2["dst_of"], kind="stable")
    starts = np.concatenate([[0], np.cumsum(ex2["size"])])
    rng = np.random.default_rng(16)
    rows = np.unique(np.concatenate([rng.choice(sz["M"], 96, replace=False), np.argsort(ex2["size"])[-8:], [0, sz["M"] - 1]]))
    ref = np.empty((rows.size, 1024))
    for k, j in enumerate(rows):
        members = order[starts[j]:starts[j + 1]]
        ref[k] = to_f64(x2[torch.from_numpy(members).cuda()]).mean(axis=0)
    check_bf16(f"{wl.name} refreshed: merge", to_f64(xm2[torch.from_numpy(rows).cuda()]), ref, sampled=True)


@pytest.mark.parametrize("name", ["C3", "C5"])
def test_fp8_attention_variant_on_sampled_rows(name):
    """The E4M3 variant (qkv_dtype = 1) at the merged lengths of C3 and C5, on the near-duplicate
    groups so that every key chunk matters: per-head scales and the quantised codes of sampled rows
    bit for bit against the oracle's quantiser, and the attention core of sampled queries against
    the oracle on the GPU's own operands, dequantised (tolerances as in the small-size test)."""
    import paper_2512_04939_b200 as pkg
    from test_gpu_parity import FP8_PEAKED_NOISE

    wl = WORKLOADS[name]
    ctx = pkg.LiteVGGT(wl.frames, wl.grid_h, wl.grid_w, wl.merge_ratio, qkv_dtype=1)
    m = ctx.n_merged
    x, w_qkv, b_qkv, w_o, b_o = make_peaked_attention_inputs(m, wl.seed + 9, "cuda")
    ctx.global_attn(x, w_qkv, b_qkv, w_o, b_o)
    ctx.poll()
    qkv_gpu, o_gpu = ctx.debug_buffer(0), ctx.debug_buffer(1)
    f8 = ctx.debug_fp8_buffers()
    # scales: the largest magnitude of every (tensor, head) slice, exactly
    amax_ref = qkv_gpu.float().abs().reshape(m, 3, 16, 64).amax(dim=(0, 3))
    assert torch.equal(f8["amax"], amax_ref)
    scales = (f8["amax"].cpu().numpy() / np.float32(448.0)).astype(np.float32)
    edges, _ = key_chunk_edges(m)
    rng = np.random.default_rng(19)
    rows = [0, 127, 128, m - 1] + list(rng.choice(m, 12, replace=False))
    for e in edges:
        rows += [e - 1, e]
    rows = np.unique(np.asarray(rows, dtype=np.int64))
    rows_t = torch.from_numpy(rows).cuda()
    # codes of the sampled rows (Q, K row-major; V from the transposed copy)
    part = to_f64(qkv_gpu[rows_t])
    per_elem = np.repeat(scales.reshape(48), 64)[None, :]
    codes_ref, _ = O.quantize_e4m3(part, np.broadcast_to(per_elem, part.shape))
    got = np.concatenate([f8["q8"][rows_t].cpu().numpy(), f8["k8"][rows_t].cpu().numpy(),
                          f8["v8t"][:, rows_t].cpu().numpy().T], axis=1)
    nonzero = (codes_ref & 0x7f) != 0
    assert np.array_equal(got[nonzero], codes_ref[nonzero]) and np.all((got[~nonzero] & 0x7f) == 0)
    assert torch.all(f8["v8t"][:, m:] == 0)
    vals = np.concatenate([O.e4m3_values(), [np.nan]])
    decode = lambda c: np.where(c & 0x80, -1.0, 1.0) * vals[c & 0x7f]
    o_rows = to_f64(o_gpu[rows_t])
    for head in (0, 9, 15):
        sl = slice(64 * head, 64 * head + 64)
        q = decode(f8["q8"][:, sl].cpu().numpy()) * scales[0, head]
        k = decode(f8["k8"][:, sl].cpu().numpy()) * scales[1, head] / K_FOLD
        v = decode(f8["v8t"][sl, :m].cpu().numpy().T) * scales[2, head]
        ref_o = O.attention_core(np.concatenate([q, k, v], axis=1), heads=1, rows=rows)
        check_bf16(f"fp8 {name}: attention core, peaked softmax, head {head}", o_rows[:, sl], ref_o, noise=FP8_PEAKED_NOISE,
                   sampled=True)
    ctx.close()
    del x, f8
    torch.cuda.empty_cache()
