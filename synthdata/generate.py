"""Seeded synthetic VGGT-shaped inputs (images, tokens, attention weights).

Stand-ins for the paper's evaluation sequences (ScanNet-50, 7Scenes, NRGBD, Tanks &
Temples, DTU, CO3Dv2 at 392x518 / 518x518), which are not available offline.  The
generator reproduces only what the method relies on: frame counts and resolutions,
5 special tokens per frame ahead of the patch tokens, flat (redundant) regions,
edge-rich regions, and overlapping content between neighbouring frames.

Everything is drawn with ``torch`` so the same recipe runs on the host (tests) and on
the device (benchmark at 1000 frames); a fixed ``(seed, device type)`` pair always
yields the same bytes.  No function here takes part in the method itself.
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import torch
import torch.nn.functional as F

PATCH_PX = 14
N_SPECIAL = 5
DIM = 1024
HEADS = 16
_FRAME_CHUNK = 25


@dataclass(frozen=True)
class Workload:
    """One of the five benchmark configurations."""

    name: str
    frames: int
    grid_h: int  # patch rows  (image height = 14 * grid_h)
    grid_w: int  # patch cols  (image width  = 14 * grid_w)
    merge_ratio: float
    scene: str  # "polygons": independent frames; "trajectory": crops of one scene
    global_layers: int
    recompute_interval: int
    seed: int

    @property
    def patches(self) -> int:
        return self.grid_h * self.grid_w

    @property
    def tokens_per_frame(self) -> int:
        return self.patches + N_SPECIAL

    @property
    def n_tokens(self) -> int:
        return self.frames * self.tokens_per_frame

    @property
    def img_h(self) -> int:
        return self.grid_h * PATCH_PX

    @property
    def img_w(self) -> int:
        return self.grid_w * PATCH_PX


WORKLOADS = {
    "C1": Workload("C1", 4, 16, 16, 0.5, "polygons", 1, 6, 1000),
    "C2": Workload("C2", 32, 37, 37, 0.5, "polygons", 4, 6, 2000),
    "C3": Workload("C3", 200, 28, 37, 0.6, "trajectory", 4, 6, 3000),
    "C4": Workload("C4", 500, 37, 37, 0.7, "polygons", 12, 6, 4000),
    "C5": Workload("C5", 1000, 28, 37, 0.5, "trajectory", 24, 6, 5000),
}


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _polygon_canvas(n_img: int, h: int, w: int, n_poly: int, g, device) -> torch.Tensor:
    """n_img images [n_img,3,h,w]: smooth background + flat-colour convex polygons
    with a linear shading term (piecewise smooth), painter's order."""
    ys = torch.linspace(0.0, 1.0, h, device=device).view(1, h, 1)
    xs = torch.linspace(0.0, 1.0, w, device=device).view(1, 1, w)
    base = torch.rand(n_img, 3, 1, 1, generator=g, device=device) * 0.5 + 0.25
    slope = (torch.rand(n_img, 3, 2, generator=g, device=device) - 0.5) * 0.3
    img = base + slope[..., 0].view(n_img, 3, 1, 1) * ys.unsqueeze(1) + slope[..., 1].view(n_img, 3, 1, 1) * xs.unsqueeze(1)
    img = img.contiguous()
    n_side = 5
    centre = torch.rand(n_img, n_poly, 2, generator=g, device=device)
    radius = torch.rand(n_img, n_poly, generator=g, device=device) * 0.22 + 0.06
    phase = torch.rand(n_img, n_poly, generator=g, device=device) * (2 * math.pi)
    colour = torch.rand(n_img, n_poly, 3, generator=g, device=device)
    shade = (torch.rand(n_img, n_poly, 3, 2, generator=g, device=device) - 0.5) * 0.4
    for p in range(n_poly):
        inside = torch.ones(n_img, h, w, dtype=torch.bool, device=device)
        cy = centre[:, p, 0].view(n_img, 1, 1)
        cx = centre[:, p, 1].view(n_img, 1, 1)
        for e in range(n_side):
            ang = phase[:, p] + (2 * math.pi * e) / n_side
            ny = torch.sin(ang).view(n_img, 1, 1)
            nx = torch.cos(ang).view(n_img, 1, 1)
            inside &= ((ys - cy) * ny + (xs - cx) * nx) <= radius[:, p].view(n_img, 1, 1)
        val = (
            colour[:, p].view(n_img, 3, 1, 1)
            + shade[:, p, :, 0].view(n_img, 3, 1, 1) * (ys - cy).unsqueeze(1)
            + shade[:, p, :, 1].view(n_img, 3, 1, 1) * (xs - cx).unsqueeze(1)
        )
        img = torch.where(inside.unsqueeze(1), val, img)
    return img


def make_images(wl: Workload, device="cpu") -> torch.Tensor:
    """Frames as fp32 [F,3,H,W] in [0,1] with N(0,0.02^2) pixel noise."""
    dev = torch.device(device)
    g = _gen(wl.seed + 1, dev)
    h, w, nf = wl.img_h, wl.img_w, wl.frames
    out = torch.empty(nf, 3, h, w, dtype=torch.float32, device=dev)
    if wl.scene == "polygons":
        for f0 in range(0, nf, _FRAME_CHUNK):
            f1 = min(nf, f0 + _FRAME_CHUNK)
            out[f0:f1] = _polygon_canvas(f1 - f0, h, w, 12, g, dev)
    else:
        side = 2048
        scene = _polygon_canvas(1, side, side, 96, g, dev)
        # smooth camera path: low-pass filtered random walk (x, y, zoom, roll)
        steps = torch.randn(4, nf + 64, generator=g, device=dev)
        kernel = torch.ones(1, 1, 65, device=dev) / 65.0
        path = F.conv1d(steps.cumsum(1).unsqueeze(1), kernel).squeeze(1)  # [4, nf]
        path = path - path.mean(1, keepdim=True)
        span = path.abs().amax(1, keepdim=True).clamp_min(1e-6)
        path = path / span
        half_w = 0.5 * w / side
        half_h = 0.5 * h / side
        reach_x = 1.0 - 1.2 * half_w * 2
        reach_y = 1.0 - 1.2 * half_h * 2
        cx = path[0] * reach_x * 0.9
        cy = path[1] * reach_y * 0.9
        zoom = 1.0 + 0.1 * path[2]
        roll = 0.08 * path[3]
        gy = torch.linspace(-1.0, 1.0, h, device=dev).view(h, 1).expand(h, w)
        gx = torch.linspace(-1.0, 1.0, w, device=dev).view(1, w).expand(h, w)
        for f0 in range(0, nf, _FRAME_CHUNK):
            f1 = min(nf, f0 + _FRAME_CHUNK)
            c, s = torch.cos(roll[f0:f1]).view(-1, 1, 1), torch.sin(roll[f0:f1]).view(-1, 1, 1)
            z = zoom[f0:f1].view(-1, 1, 1)
            ux = gx * (2 * half_w) * z
            uy = gy * (2 * half_h) * z
            sx = cx[f0:f1].view(-1, 1, 1) + c * ux - s * uy
            sy = cy[f0:f1].view(-1, 1, 1) + s * ux + c * uy
            grid = torch.stack([sx, sy], dim=-1)
            out[f0:f1] = F.grid_sample(
                scene.expand(f1 - f0, -1, -1, -1), grid, mode="bilinear", padding_mode="border", align_corners=True
            )
    for f0 in range(0, nf, _FRAME_CHUNK):
        f1 = min(nf, f0 + _FRAME_CHUNK)
        out[f0:f1] += 0.02 * torch.randn(f1 - f0, 3, h, w, generator=g, device=dev)
    return out.clamp_(0.0, 1.0)


def _patch_features(img: torch.Tensor) -> torch.Tensor:
    """[n,3,H,W] -> [n, gh*gw, 4]: per-patch mean R, G, B and mean edge strength."""
    grey = img.mean(1, keepdim=True)
    kx = torch.tensor([[-1.0, 0.0, 1.0], [-2.0, 0.0, 2.0], [-1.0, 0.0, 1.0]], device=img.device)
    k = torch.stack([kx, kx.t()]).unsqueeze(1)
    d = F.conv2d(F.pad(grey, (1, 1, 1, 1), mode="replicate"), k)
    edge = d.pow(2).sum(1, keepdim=True).sqrt()
    feat = torch.cat([img, edge], dim=1)
    feat = F.avg_pool2d(feat, PATCH_PX)  # [n,4,gh,gw]
    return feat.flatten(2).transpose(1, 2).contiguous()


def _binomial_blur(field: torch.Tensor) -> torch.Tensor:
    """[n,gh,gw,D]: two passes of the 3-tap binomial filter along both grid axes."""
    n, gh, gw, d = field.shape
    x = field.permute(0, 3, 1, 2).reshape(n * d, 1, gh, gw)
    k1 = torch.tensor([1.0, 2.0, 1.0], device=field.device) / 4.0
    for _ in range(2):
        x = F.conv2d(F.pad(x, (1, 1, 0, 0), mode="replicate"), k1.view(1, 1, 1, 3))
        x = F.conv2d(F.pad(x, (0, 0, 1, 1), mode="replicate"), k1.view(1, 1, 3, 1))
    return x.reshape(n, d, gh, gw).permute(0, 2, 3, 1)


def make_tokens(wl: Workload, images: torch.Tensor, dim: int = DIM) -> torch.Tensor:
    """Tokens as bf16 [N, dim]; per frame 5 special tokens then gh*gw patch tokens
    (row-major over the patch grid)."""
    dev = images.device
    g = _gen(wl.seed + 2, dev)
    nf, p, t = wl.frames, wl.patches, wl.tokens_per_frame
    w_map = torch.randn(4, dim, generator=g, device=dev)
    special = torch.randn(2, N_SPECIAL, dim, generator=g, device=dev)
    blur_gain = (70.0 / 256.0)  # std of unit white noise after the separable 5-tap blur
    out = torch.empty(nf, t, dim, dtype=torch.bfloat16, device=dev)
    for f0 in range(0, nf, _FRAME_CHUNK):
        f1 = min(nf, f0 + _FRAME_CHUNK)
        n = f1 - f0
        phi = _patch_features(images[f0:f1])  # [n,P,4]
        tok = phi @ w_map
        field = torch.randn(n, wl.grid_h, wl.grid_w, dim, generator=g, device=dev)
        tok = tok + (0.1 / blur_gain) * _binomial_blur(field).reshape(n, p, dim)
        tok = tok + 0.05 * torch.randn(n, p, dim, generator=g, device=dev)
        sp = special[1].unsqueeze(0).repeat(n, 1, 1)
        if f0 == 0:
            sp[0] = special[0]
        sp = sp + 0.05 * torch.randn(n, N_SPECIAL, dim, generator=g, device=dev)
        out[f0:f1, :N_SPECIAL] = sp.to(torch.bfloat16)
        out[f0:f1, N_SPECIAL:] = tok.to(torch.bfloat16)
    return out.view(nf * t, dim)


def make_attention_weights(wl: Workload, layer: int, device="cpu", dim: int = DIM):
    """(w_qkv [3*dim, dim], b_qkv [3*dim], w_o [dim, dim], b_o [dim]) in bf16.

    Weights are stored output-feature-major (row j holds the weights producing output
    feature j), entries ~ N(0, 0.02^2); biases are small but non-zero so that a
    dropped bias term is visible in parity tests."""
    dev = torch.device(device)
    g = _gen(wl.seed + 100 + layer, dev)
    w_qkv = (0.02 * torch.randn(3 * dim, dim, generator=g, device=dev)).to(torch.bfloat16)
    b_qkv = (0.02 * torch.randn(3 * dim, generator=g, device=dev)).to(torch.bfloat16)
    w_o = (0.02 * torch.randn(dim, dim, generator=g, device=dev)).to(torch.bfloat16)
    b_o = (0.02 * torch.randn(dim, generator=g, device=dev)).to(torch.bfloat16)
    return w_qkv, b_qkv, w_o, b_o


def make_peaked_attention_inputs(m: int, seed: int, device="cpu", groups: int = 4099, sharpness: float = 4.0,
                                 dim: int = DIM):
    """Rows and projection weights under which softmax attention is far from uniform.

    Row j = base[j % groups] + 0.5 * noise_j with unit-variance base and noise, and the query
    weights are ``sharpness`` times the key weights, so a query scores highest against itself and
    next against the other rows of its own group, which lie ``groups`` rows apart through the whole
    sequence (about m / groups of them, with different weights and different values).  Random-init
    0.02 weights on the token generator's rows give nearly uniform attention, under which a lost or
    repeated stretch of keys barely moves the output; these inputs make it move.
    Returns (x [m, dim] bf16, w_qkv, b_qkv, w_o, b_o) like make_attention_weights."""
    dev = torch.device(device)
    g = _gen(seed, dev)
    bf = torch.bfloat16
    base = torch.randn(groups, dim, generator=g, device=dev)
    x = torch.empty(m, dim, dtype=bf, device=dev)
    chunk = 1 << 16
    for r0 in range(0, m, chunk):
        r1 = min(m, r0 + chunk)
        idx = torch.arange(r0, r1, device=dev) % groups
        x[r0:r1] = (base[idx] + 0.5 * torch.randn(r1 - r0, dim, generator=g, device=dev)).to(bf)
    w_k = 0.02 * torch.randn(dim, dim, generator=g, device=dev)
    w_v = 0.02 * torch.randn(dim, dim, generator=g, device=dev)
    w_qkv = torch.cat([sharpness * w_k, w_k, w_v]).to(bf)
    b_qkv = (0.02 * torch.randn(3 * dim, generator=g, device=dev)).to(bf)
    w_o = (0.02 * torch.randn(dim, dim, generator=g, device=dev)).to(bf)
    b_o = (0.02 * torch.randn(dim, generator=g, device=dev)).to(bf)
    return x, w_qkv, b_qkv, w_o, b_o


def make_block_weights(wl: Workload, layer: int, device="cpu", dim: int = DIM):
    """Weights of the other sub-layers of one aggregator block, bf16: two LayerNorms (gamma near 1,
    beta near 0), the frame-attention layer (as make_attention_weights) and the MLP of ratio 4
    (w1 [4*dim, dim], b1, w2 [dim, 4*dim], b2 ~ N(0, 0.02^2))."""
    dev = torch.device(device)
    g = _gen(wl.seed + 500 + layer, dev)
    bf = torch.bfloat16
    ln = [((1.0 + 0.1 * torch.randn(dim, generator=g, device=dev)).to(bf), (0.1 * torch.randn(dim, generator=g, device=dev)).to(bf))
          for _ in range(2)]
    attn = [(0.02 * torch.randn(3 * dim, dim, generator=g, device=dev)).to(bf),
            (0.02 * torch.randn(3 * dim, generator=g, device=dev)).to(bf),
            (0.02 * torch.randn(dim, dim, generator=g, device=dev)).to(bf),
            (0.02 * torch.randn(dim, generator=g, device=dev)).to(bf)]
    mlp = [(0.02 * torch.randn(4 * dim, dim, generator=g, device=dev)).to(bf),
           (0.02 * torch.randn(4 * dim, generator=g, device=dev)).to(bf),
           (0.02 * torch.randn(dim, 4 * dim, generator=g, device=dev)).to(bf),
           (0.02 * torch.randn(dim, generator=g, device=dev)).to(bf)]
    return dict(ln1=ln[0], ln2=ln[1], attn=attn, mlp=mlp)


def make_workload_inputs(name: str, device="cpu"):
    """Convenience: (workload, images fp32 [F,3,H,W], tokens bf16 [N,D])."""
    wl = WORKLOADS[name]
    images = make_images(wl, device)
    tokens = make_tokens(wl, images)
    return wl, images, tokens
