"""CPU oracle for geometry-aware cached token merging around VGGT's global attention.

TEST INFRASTRUCTURE ONLY.  This is a plain, slow float64 numpy restatement of what the
paper defines (Sec. 3.4 "Geometry-aware Cached Token Merging", Sec. 3.1 for the token
layout and the global attention layer).  It shares no code with the CUDA library and
must never be imported by it: only the test-suite, the smoke check and the benchmark's
CPU-baseline leg may call it.

Conventions
  * F frames; patch grid gh x gw; P = gh*gw patch tokens and S special tokens per
    frame (1 camera + 4 register, Sec. 3.1); T = P + S; N = F*T tokens; D channels.
  * token index i = f*T + t; t < S are the special tokens, t = S + py*gw + px patches.
  * inputs arrive as the same bf16 values the GPU sees, widened to float64; nothing in
    here rounds to a narrower type.
  * every tie is broken towards the lowest index.

Where the paper leaves a choice open (normalisation, window, padding, the merge-ratio
knob, odd grids ...) the reading taken is stated in the function's docstring.

Parity status: every function below is pinned by tests against closed forms,
invariants, library routines on special cases or brute force; the path as a whole is
"parity unpinned" against the authors' own implementation, which is not available.
"""
from __future__ import annotations

import numpy as np

CLS_PROTECTED = 0  # special tokens (never merged, never anchors)
CLS_GA = 1         # top geometric-importance tokens, excluded from merging
CLS_DST = 2        # anchors
CLS_SRC = 3        # merge candidates


# --------------------------------------------------------------------------------------
# sizes
# --------------------------------------------------------------------------------------
def derived_sizes(frames, grid_h, grid_w, n_special=5, merge_ratio=0.5, ga_keep_frac=0.10,
                  cell_h=2, cell_w=2):
    """Token counts that follow from the partition rules of Sec. 3.4 ("GA Token
    Partitioning").  Per non-first frame: one anchor per (clipped) cell, floor(frac*P)
    GA tokens, the rest are src.  First frame: all P patches are anchors.  The
    merge-ratio knob (not in the paper; the paper merges every src) removes
    R = min(|Src|, floor(r*N)) tokens."""
    p = grid_h * grid_w
    t = p + n_special
    n = frames * t
    n_dst_f = -(-grid_h // cell_h) * -(-grid_w // cell_w)
    n_ga_f = int(np.floor(ga_keep_frac * p + 1e-9))
    n_ga_f = min(n_ga_f, p - n_dst_f)
    n_src_f = p - n_dst_f - n_ga_f
    n_src = (frames - 1) * n_src_f
    n_dst = p + (frames - 1) * n_dst_f
    r = min(n_src, int(np.floor(merge_ratio * n + 1e-9)))
    return dict(P=p, T=t, N=n, n_dst_frame=n_dst_f, n_ga_frame=n_ga_f, n_src_frame=n_src_f,
                n_src=n_src, n_dst=n_dst, R=r, M=n - r)


# --------------------------------------------------------------------------------------
# step 1: geometry-aware map
# --------------------------------------------------------------------------------------
def grad_map(images, patch_px=14):
    """Grad map Psi_g (Sec. 3.4, "Pixel Gradient"): Sobel operator on image intensity,
    downsampled to token granularity.

    Reading: intensity = mean of R,G,B; 3x3 Sobel pair, replicate padding at the image
    border; magnitude sqrt(gx^2+gy^2); average over each patch_px x patch_px patch.
    images [F,3,H,W] -> [F, H/patch, W/patch]."""
    img = np.asarray(images, dtype=np.float64)
    f, c, h, w = img.shape
    assert c == 3 and h % patch_px == 0 and w % patch_px == 0
    grey = (img[:, 0] + img[:, 1] + img[:, 2]) / 3.0
    pad = np.pad(grey, ((0, 0), (1, 1), (1, 1)), mode="edge")
    # neighbours of pixel (y,x): pad[y+dy+1, x+dx+1]
    def nb(dy, dx):
        return pad[:, 1 + dy:1 + dy + h, 1 + dx:1 + dx + w]
    gx = (nb(-1, 1) - nb(-1, -1)) + 2.0 * (nb(0, 1) - nb(0, -1)) + (nb(1, 1) - nb(1, -1))
    gy = (nb(1, -1) - nb(-1, -1)) + 2.0 * (nb(1, 0) - nb(-1, 0)) + (nb(1, 1) - nb(-1, 1))
    mag = np.sqrt(gx * gx + gy * gy)
    gh, gw = h // patch_px, w // patch_px
    return mag.reshape(f, gh, patch_px, gw, patch_px).mean(axis=(2, 4))


def var_map(x, frames, grid_h, grid_w, n_special=5, window=3):
    """Var map Psi_v (Sec. 3.4, "Token Variance"): tokens rearranged to the 2-D patch
    grid, local average-pooled variance.

    Reading: for every grid position the window is the window x window neighbourhood
    clipped to the grid; per channel the population variance of the window's values;
    Psi_v is the mean of that variance over the D channels.  x [N,D] -> [F,gh,gw]."""
    x = np.asarray(x, dtype=np.float64)
    t = grid_h * grid_w + n_special
    d = x.shape[1]
    grid = x.reshape(frames, t, d)[:, n_special:, :].reshape(frames, grid_h, grid_w, d)
    half = window // 2
    out = np.zeros((frames, grid_h, grid_w))
    for py in range(grid_h):
        y0, y1 = max(0, py - half), min(grid_h, py + half + 1)
        for px in range(grid_w):
            x0, x1 = max(0, px - half), min(grid_w, px + half + 1)
            win = grid[:, y0:y1, x0:x1, :].reshape(frames, -1, d)
            mu = win.mean(axis=1, keepdims=True)
            out[:, py, px] = ((win - mu) ** 2).mean(axis=1).mean(axis=1)
    return out


def ga_map(grad, var, alpha=0.5, beta=0.5, eps=1e-6):
    """Psi_GA = alpha*norm(Psi_g) + beta*norm(Psi_v) (Sec. 3.4, unnumbered equation).
    Reading of norm(.): per-frame min-max, (v - min) / (max - min + eps)."""
    def norm(m):
        m = np.asarray(m, dtype=np.float64)
        lo = m.min(axis=(1, 2), keepdims=True)
        hi = m.max(axis=(1, 2), keepdims=True)
        return (m - lo) / (hi - lo + eps)
    return alpha * norm(grad) + beta * norm(var)


# --------------------------------------------------------------------------------------
# step 1 (cont.): partition into GA / dst / src
# --------------------------------------------------------------------------------------
def partition(ga, n_special=5, ga_keep_frac=0.10, cell_h=2, cell_w=2):
    """Token classes (Sec. 3.4, "GA Token Partitioning").

    Frame 0: every patch token is an anchor.  Other frames: cells of cell_h x cell_w
    anchored at the grid origin and clipped at the far edges; in each cell the patch
    with the lowest GA score becomes the anchor; among the patches that are not
    anchors, the floor(frac*P) highest GA scores become GA tokens; the rest are src.
    Special tokens of every frame are protected.  Returns cls [N] uint8."""
    ga = np.asarray(ga, dtype=np.float64)
    frames, gh, gw = ga.shape
    p = gh * gw
    t = p + n_special
    n_ga = int(np.floor(ga_keep_frac * p + 1e-9))
    cls = np.full(frames * t, CLS_PROTECTED, dtype=np.uint8)
    for f in range(frames):
        base = f * t + n_special
        if f == 0:
            cls[base:base + p] = CLS_DST
            continue
        score = ga[f].reshape(p)
        is_dst = np.zeros(p, dtype=bool)
        for cy in range(0, gh, cell_h):
            for cx in range(0, gw, cell_w):
                best, best_v = -1, np.inf
                for py in range(cy, min(gh, cy + cell_h)):
                    for px in range(cx, min(gw, cx + cell_w)):
                        if score[py * gw + px] < best_v:
                            best, best_v = py * gw + px, score[py * gw + px]
                is_dst[best] = True
        rest = np.flatnonzero(~is_dst)
        # highest score first, ties towards the lowest index
        order = rest[np.lexsort((rest, -score[rest]))]
        k = min(n_ga, rest.size)
        frame_cls = np.full(p, CLS_SRC, dtype=np.uint8)
        frame_cls[is_dst] = CLS_DST
        frame_cls[order[:k]] = CLS_GA
        cls[base:base + p] = frame_cls
    return cls


# --------------------------------------------------------------------------------------
# step 2: src -> dst matching
# --------------------------------------------------------------------------------------
def match(x, src_idx, dst_idx, rows=None, norm_eps=1e-12, chunk=2048):
    """Cosine matching (Sec. 3.4, "Cached Token Merging": src tokens are matched to
    dst tokens via cosine similarity, each to its most similar dst).

    Candidates are all anchors of all frames.  rows (optional) selects positions in
    src_idx to evaluate.  Returns (best_dst token index, best_sim, second_sim)."""
    x = np.asarray(x, dtype=np.float64)
    src_idx = np.asarray(src_idx, dtype=np.int64)
    dst_idx = np.asarray(dst_idx, dtype=np.int64)
    if rows is not None:
        src_idx = src_idx[np.asarray(rows, dtype=np.int64)]
    b = x[dst_idx]
    nb = np.maximum(np.sqrt((b * b).sum(axis=1)), norm_eps)
    best = np.empty(src_idx.size, dtype=np.int64)
    sim1 = np.empty(src_idx.size)
    sim2 = np.full(src_idx.size, -np.inf)
    for c0 in range(0, src_idx.size, chunk):
        a = x[src_idx[c0:c0 + chunk]]
        na = np.maximum(np.sqrt((a * a).sum(axis=1)), norm_eps)
        sim = (a @ b.T) / (na[:, None] * nb[None, :])
        j = sim.argmax(axis=1)  # first maximum = lowest anchor index
        rowsel = np.arange(a.shape[0])
        sim1[c0:c0 + chunk] = sim[rowsel, j]
        best[c0:c0 + chunk] = dst_idx[j]
        if dst_idx.size > 1:
            sim[rowsel, j] = -np.inf
            sim2[c0:c0 + chunk] = sim.max(axis=1)
    return best, sim1, sim2


# --------------------------------------------------------------------------------------
# step 2 (cont.): which src are merged, and the index arrays
# --------------------------------------------------------------------------------------
def select_and_index(cls, best_dst, best_sim, n_remove):
    """Merge indices.

    best_dst / best_sim are given per src token in ascending token order.  The
    n_remove src tokens with the highest best_sim (ties: lowest token index) are merged
    into their anchors; n_remove = |Src| is the paper's rule (every src is merged,
    Sec. 3.4 "Src Tokens").  Kept tokens keep their original order.  Returns
    dst_of [N] (row of the merged sequence each token maps to), size [M]
    (1 + number of src merged into the row), kept_idx [M] (token index of each row)."""
    cls = np.asarray(cls)
    n = cls.size
    src_idx = np.flatnonzero(cls == CLS_SRC)
    best_dst = np.asarray(best_dst, dtype=np.int64)
    best_sim = np.asarray(best_sim, dtype=np.float64)
    assert src_idx.size == best_dst.size == best_sim.size
    assert 0 <= n_remove <= src_idx.size
    order = np.lexsort((src_idx, -best_sim))  # primary: sim descending; then index
    merged_pos = np.sort(order[:n_remove])
    removed = np.zeros(n, dtype=bool)
    removed[src_idx[merged_pos]] = True
    kept_idx = np.flatnonzero(~removed)
    row_of = np.full(n, -1, dtype=np.int64)
    row_of[kept_idx] = np.arange(kept_idx.size)
    dst_of = row_of.copy()
    dst_of[src_idx[merged_pos]] = row_of[best_dst[merged_pos]]
    assert (dst_of >= 0).all()
    size = np.bincount(dst_of, minlength=kept_idx.size)
    return dst_of, size, kept_idx


# --------------------------------------------------------------------------------------
# step 3: merge, step 4 tail: unmerge
# --------------------------------------------------------------------------------------
def merge(x, dst_of, n_merged):
    """x'_d = (x_d + sum_{s in S_d} x_s) / (1 + |S_d|)  (Sec. 3.4, the merge equation).
    Rows that absorb nothing are returned unchanged."""
    x = np.asarray(x, dtype=np.float64)
    dst_of = np.asarray(dst_of, dtype=np.int64)
    acc = np.zeros((n_merged, x.shape[1]))
    np.add.at(acc, dst_of, x)
    size = np.bincount(dst_of, minlength=n_merged).astype(np.float64)
    return acc / size[:, None]


def unmerge(y_merged, dst_of, residual=None):
    """Token unmerging (Sec. 3.4): every member of {x_d} U S_d receives a copy of the
    merged row, restoring the original length; optional residual add."""
    out = np.asarray(y_merged, dtype=np.float64)[np.asarray(dst_of, dtype=np.int64)]
    if residual is not None:
        out = out + np.asarray(residual, dtype=np.float64)
    return out


# --------------------------------------------------------------------------------------
# step 4: global self-attention over the merged sequence
# --------------------------------------------------------------------------------------
def attention_core(qkv, heads=16, rows=None, chunk=1024):
    """Per head softmax(Q K^T / sqrt(dh)) V, non-causal, no mask, max-subtracted softmax.
    qkv [M, 3D] with columns [0,D) = Q, [D,2D) = K, [2D,3D) = V; head h owns channels
    [h*dh, (h+1)*dh) of each.  rows (optional) restricts the queries (all keys/values are
    still used).  Returns o [len(rows) or M, D]."""
    qkv = np.asarray(qkv, dtype=np.float64)
    d = qkv.shape[1] // 3
    dh = d // heads
    q, k, v = qkv[:, :d], qkv[:, d:2 * d], qkv[:, 2 * d:]
    if rows is not None:
        q = q[np.asarray(rows, dtype=np.int64)]
    o = np.empty((q.shape[0], d))
    scale = 1.0 / np.sqrt(dh)
    for h in range(heads):
        sl = slice(h * dh, (h + 1) * dh)
        kh, vh = k[:, sl], v[:, sl]
        for c0 in range(0, q.shape[0], chunk):
            s = (q[c0:c0 + chunk, sl] @ kh.T) * scale
            s -= s.max(axis=1, keepdims=True)
            p = np.exp(s)
            p /= p.sum(axis=1, keepdims=True)
            o[c0:c0 + chunk, sl] = p @ vh
    return o


def linear(a, w, b=None):
    """a @ w.T + b with output-feature-major weights w [n_out, n_in]."""
    y = np.asarray(a, dtype=np.float64) @ np.asarray(w, dtype=np.float64).T
    if b is not None:
        y = y + np.asarray(b, dtype=np.float64)
    return y


# --------------------------------------------------------------------------------------
# FP8 variant of the attention operands (Sec. 3.5 and supplementary "FP8 Quantization Details")
# --------------------------------------------------------------------------------------
E4M3_MAX = 448.0


def e4m3_values():
    """Every finite value of the E4M3 format the paper quantises to (supplementary "FP8 Quantization
    Details": 1 sign, 4 exponent, 3 mantissa bits, exponent bias 7; the variant without infinities,
    whose largest finite value is 448 and whose only NaN is the all-ones pattern).  Returns the 127
    non-negative values, ascending, index = bit pattern (0x00 .. 0x7e)."""
    vals = np.empty(127)
    for code in range(127):
        e, m = code >> 3, code & 7
        vals[code] = m * 2.0 ** -9 if e == 0 else (1.0 + m / 8.0) * 2.0 ** (e - 7)
    return vals


def quantize_e4m3(x, scale):
    """x / scale rounded to the nearest E4M3 value (ties to the even mantissa), saturating at +-448.
    Returns (codes uint8, dequantised values codes * scale as float64).

    The quotient is formed the way the kernel forms it - float32 value times the float32 reciprocal
    448 / amax - because this decision between two codes is taken in that precision; everything
    after it is exact."""
    x32 = np.asarray(x, dtype=np.float32)
    inv = np.float32(1.0) / np.asarray(scale, dtype=np.float32)
    y = (x32 * inv).astype(np.float64)
    vals = e4m3_values()
    a = np.minimum(np.abs(y), E4M3_MAX)
    hi = np.searchsorted(vals, a, side="left")          # first value >= a
    hi = np.minimum(hi, vals.size - 1)
    lo = np.maximum(hi - 1, 0)
    d_lo, d_hi = a - vals[lo], vals[hi] - a
    pick_hi = (d_hi < d_lo) | ((d_hi == d_lo) & (hi % 2 == 0))  # tie: the even code (even mantissa)
    code = np.where(pick_hi, hi, lo).astype(np.uint8)
    code = np.where(np.signbit(y), code | 0x80, code).astype(np.uint8)
    deq = np.where(code & 0x80, -1.0, 1.0) * vals[code & 0x7f] * np.asarray(scale, dtype=np.float32).astype(np.float64)
    return code, deq


def fp8_head_scales(t, heads=16):
    """Per-head scale of one of Q, K, V [M, D]: amax over the head's rows and channels divided by
    448, so that the largest entry of the head lands on the largest E4M3 value (current scaling:
    the statistics of the tensor being quantised; the paper's delayed scaling needs a history of
    earlier iterations, which a single forward pass does not have).  float32 [heads]; 1/448 where a
    head is all zero."""
    t = np.asarray(t, dtype=np.float32)
    m, d = t.shape
    amax = np.abs(t).reshape(m, heads, d // heads).max(axis=(0, 2))
    amax = np.where(amax > 0, amax, np.float32(1.0)).astype(np.float32)
    return (amax / np.float32(E4M3_MAX)).astype(np.float32)


def quantize_qkv_e4m3(qkv, heads=16):
    """Q, K and V of qkv [M, 3D] quantised head by head.  Returns (dequantised qkv float64, codes
    uint8 [M, 3D], scales float32 [3, heads])."""
    qkv = np.asarray(qkv, dtype=np.float64)
    m, d = qkv.shape[0], qkv.shape[1] // 3
    dh = d // heads
    deq = np.empty_like(qkv)
    codes = np.empty(qkv.shape, dtype=np.uint8)
    scales = np.empty((3, heads), dtype=np.float32)
    for i in range(3):
        part = qkv[:, i * d:(i + 1) * d]
        scales[i] = fp8_head_scales(part, heads)
        per_elem = np.repeat(scales[i], dh)[None, :]
        c, v = quantize_e4m3(part, np.broadcast_to(per_elem, part.shape))
        codes[:, i * d:(i + 1) * d] = c
        deq[:, i * d:(i + 1) * d] = v
    return deq, codes, scales


def token_positions(frames, grid_h, grid_w, n_special=5):
    """Integer (row, column) position of every token for the rotary embedding.  Reading (the paper
    prints none; VGGT's aggregator, which Sec. 3.1 keeps, works this way): the special tokens of
    a frame sit at (0, 0) and the patch at grid row py, column px at (py + 1, px + 1).  [N, 2]."""
    t = grid_h * grid_w + n_special
    pos = np.zeros((frames, t, 2), dtype=np.int64)
    py, px = np.divmod(np.arange(grid_h * grid_w), grid_w)
    pos[:, n_special:, 0] = py + 1
    pos[:, n_special:, 1] = px + 1
    return pos.reshape(frames * t, 2)


def qk_norm(v, gamma, beta, eps=1e-5):
    """LayerNorm over the channels of each head (population variance), the normalisation VGGT's
    attention applies to queries and keys before the scores.  v [M, heads, dh]; gamma, beta [dh]."""
    v = np.asarray(v, dtype=np.float64)
    mu = v.mean(axis=-1, keepdims=True)
    var = ((v - mu) ** 2).mean(axis=-1, keepdims=True)
    return (v - mu) / np.sqrt(var + eps) * np.asarray(gamma, dtype=np.float64) + np.asarray(beta, dtype=np.float64)


def rope_2d(v, pos, base=100.0):
    """Two-dimensional rotary position embedding of queries or keys.  v [M, heads, dh], pos [M, 2].

    The head's channels split into two halves of width h = dh/2: the first turns with the row
    position pos[:, 0], the second with the column position pos[:, 1].  Inside a half, channel i
    (i < h/2) and channel i + h/2 form a plane that is rotated by the angle position * base^(-2i/h).
    A rotation by an angle proportional to the position makes <rope(q, p), rope(k, p')> depend on
    p - p' only."""
    v = np.asarray(v, dtype=np.float64)
    pos = np.asarray(pos, dtype=np.float64)
    dh = v.shape[-1]
    h = dh // 2
    assert dh % 4 == 0
    theta = base ** (-2.0 * np.arange(h // 2) / h)  # [h/2]
    out = np.empty_like(v)
    for axis in range(2):
        ang = pos[:, axis, None] * theta[None, :]      # [M, h/2]
        c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
        a = v[..., axis * h: axis * h + h // 2]
        b = v[..., axis * h + h // 2: (axis + 1) * h]
        out[..., axis * h: axis * h + h // 2] = a * c - b * s
        out[..., axis * h + h // 2: (axis + 1) * h] = b * c + a * s
    return out


def global_attention(xm, w_qkv, b_qkv, w_o, b_o, heads=16, rows=None, chunk=1024,
                     return_parts=False, ext=None):
    """Standard multi-head self-attention over the whole (merged) sequence (Sec. 3.1:
    the frame-global attention concatenates all tokens for full-sequence attention).

    qkv = xm @ w_qkv.T + b_qkv (rows [0,D) of w_qkv produce Q, [D,2D) K, [2D,3D) V),
    o = attention_core(qkv), y = o @ w_o.T + b_o.  No positional terms, no mask.
    rows (optional) restricts the queries.

    ext (optional, a dict) switches on what VGGT's own attention has and the paper does not print:
    "q_gamma", "q_beta", "k_gamma", "k_beta" (+ "eps"): qk_norm of queries and keys;
    "pos" (+ "base"): rope_2d of queries and keys with one position per row of xm, applied after
    the normalisation."""
    qkv = linear(xm, w_qkv, b_qkv)
    if ext is not None:
        m, d = qkv.shape[0], qkv.shape[1] // 3
        q = qkv[:, :d].reshape(m, heads, d // heads)
        k = qkv[:, d:2 * d].reshape(m, heads, d // heads)
        if "q_gamma" in ext:
            q = qk_norm(q, ext["q_gamma"], ext["q_beta"], ext.get("eps", 1e-5))
            k = qk_norm(k, ext["k_gamma"], ext["k_beta"], ext.get("eps", 1e-5))
        if "pos" in ext:
            q = rope_2d(q, ext["pos"], ext.get("base", 100.0))
            k = rope_2d(k, ext["pos"], ext.get("base", 100.0))
        qkv = np.concatenate([q.reshape(m, d), k.reshape(m, d), qkv[:, 2 * d:]], axis=1)
    o = attention_core(qkv, heads, rows, chunk)
    y = linear(o, w_o, b_o)
    if return_parts:
        return y, qkv, o
    return y


# --------------------------------------------------------------------------------------
# the other sub-layers of an aggregator block (Sec. 3.1)
# --------------------------------------------------------------------------------------
def layernorm(x, gamma, beta, eps=1e-6):
    """LayerNorm over the channels of each row, population variance (the pre-norm of the
    transformer blocks the aggregator is built from, Sec. 3.1)."""
    x = np.asarray(x, dtype=np.float64)
    mu = x.mean(axis=1, keepdims=True)
    var = ((x - mu) ** 2).mean(axis=1, keepdims=True)
    return (x - mu) / np.sqrt(var + eps) * np.asarray(gamma, dtype=np.float64) + np.asarray(beta, dtype=np.float64)


def gelu(x):
    """Exact GELU: x * Phi(x), Phi the standard normal distribution function."""
    from math import erf, sqrt
    x = np.asarray(x, dtype=np.float64)
    return 0.5 * x * (1.0 + np.vectorize(erf)(x / sqrt(2.0)))


def mlp(x, w1, b1, w2, b2, residual=None):
    """Transformer MLP of ratio 4: gelu(x w1^T + b1) w2^T + b2 (+ residual)."""
    y = linear(gelu(linear(x, w1, b1)), w2, b2)
    if residual is not None:
        y = y + np.asarray(residual, dtype=np.float64)
    return y


def frame_attention(x, frames, w_qkv, b_qkv, w_o, b_o, heads=16, residual=None):
    """Frame-wise self-attention (Sec. 3.1): every frame's tokens attend only to the tokens of the
    same frame; the layer itself is the one of global_attention."""
    x = np.asarray(x, dtype=np.float64)
    t = x.shape[0] // frames
    y = np.concatenate([global_attention(x[f * t:(f + 1) * t], w_qkv, b_qkv, w_o, b_o, heads) for f in range(frames)])
    if residual is not None:
        y = y + np.asarray(residual, dtype=np.float64)
    return y


# --------------------------------------------------------------------------------------
# index cache
# --------------------------------------------------------------------------------------
def should_refresh(global_layer_idx, recompute_interval=6):
    """Merge indices are computed once every `recompute_interval` global layers and
    reused in between (Sec. 3.4: every 6 layers, 4 computations over 24 layers)."""
    return global_layer_idx % recompute_interval == 0


# --------------------------------------------------------------------------------------
# the whole plan, for convenience in tests and the CPU-baseline timing
# --------------------------------------------------------------------------------------
def merge_plan(x, grad, frames, grid_h, grid_w, n_special=5, merge_ratio=0.5,
               ga_keep_frac=0.10, alpha=0.5, beta=0.5, cell_h=2, cell_w=2, window=3):
    """Steps 1b-2 end to end.  Returns a dict with every intermediate."""
    sz = derived_sizes(frames, grid_h, grid_w, n_special, merge_ratio, ga_keep_frac, cell_h, cell_w)
    var = var_map(x, frames, grid_h, grid_w, n_special, window)
    ga = ga_map(grad, var, alpha, beta)
    cls = partition(ga, n_special, ga_keep_frac, cell_h, cell_w)
    src_idx = np.flatnonzero(cls == CLS_SRC)
    dst_idx = np.flatnonzero(cls == CLS_DST)
    assert src_idx.size == sz["n_src"] and dst_idx.size == sz["n_dst"]
    if src_idx.size:
        best_dst, sim1, sim2 = match(x, src_idx, dst_idx)
    else:
        best_dst = np.zeros(0, dtype=np.int64)
        sim1 = sim2 = np.zeros(0)
    dst_of, size, kept_idx = select_and_index(cls, best_dst, sim1, sz["R"])
    return dict(sizes=sz, var=var, ga=ga, cls=cls, src_idx=src_idx, dst_idx=dst_idx,
                best_dst=best_dst, best_sim=sim1, second_sim=sim2, dst_of=dst_of, size=size,
                kept_idx=kept_idx)
