"""Shared helpers for the parity tests (no method arithmetic lives here)."""
import json
import os

import numpy as np
import torch

_REPORT = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "gpurun_out", "parity_report.jsonl")


# What the bf16 intermediates that the GPU stores inside a layer (qkv and o of an attention layer, the
# hidden activations of an MLP) may add to the layer's output, in units of RMS(output), when the oracle
# rounds nothing.  The largest part is the rounding of the last intermediate passing through the next
# projection: 1024 (4096) independent errors of relative size up to 2^-8 / sqrt(12), about 1.0e-3 of
# RMS(y) at one sigma, 8.4e-3 at worst over the 556 K outputs of config C1.  The figure is reproduced
# on the CPU by test_oracle_pins.test_layer_noise_allowance_covers_stored_bf16_intermediates, which
# rounds the oracle's own intermediates.
LAYER_NOISE = 1e-2


# Entry-by-entry allowance of the attention core on top of the output's own rounding.  The
# probabilities enter the second tensor-core product as bf16, each off by up to 2^-9 relative and
# independently of the others; the row sum is formed from the same rounded values, so what is left is
# sum_i d_i p_i (v_i - o) / sum_i p_i with |d_i| <= 2^-9: at most 2^-9 times the spread of the values
# a row attends to, i.e. 2e-3 RMS per unit of spread.  Nearly uniform rows average it away (measured
# 3e-4); rows held by a handful of keys whose values lie two RMS apart reach 4e-3.
CORE_NOISE = 4e-3


# The library keeps K, wherever it is last rounded to bf16 (QKV projection, Q/K normalisation pass),
# multiplied by the softmax scale in base-2 units, 1/sqrt(64) * log2(e) in float32, so that its
# attention kernels can take 2^(q . k) directly.  The oracle knows nothing of this: a K taken from
# the library's buffers is divided by the constant before it is handed to the oracle, and a K
# computed by the oracle is multiplied by it before it is compared with the library's.
K_FOLD = float(np.float32(0.125) * np.float32(1.4426950408889634))


def unfold_k(qkv: np.ndarray) -> np.ndarray:
    """Copy of a [M, 3D] (or one head's [M, 3 dh]) qkv array with the K third divided by K_FOLD."""
    out = np.array(qkv, dtype=np.float64, copy=True)
    d = out.shape[1] // 3
    out[:, d:2 * d] /= K_FOLD
    return out


def fold_k(qkv: np.ndarray) -> np.ndarray:
    """The opposite direction: an oracle-made qkv with its K third multiplied by K_FOLD."""
    out = np.array(qkv, dtype=np.float64, copy=True)
    d = out.shape[1] // 3
    out[:, d:2 * d] *= K_FOLD
    return out


def to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


def bf16_round(a: np.ndarray) -> np.ndarray:
    return torch.from_numpy(np.asarray(a, dtype=np.float32)).to(torch.bfloat16).float().numpy().astype(np.float64)


def rel_err(got: np.ndarray, ref: np.ndarray) -> float:
    """max-abs-error / RMS(reference): the tolerance metric for bf16 outputs."""
    rms = float(np.sqrt(np.mean(ref * ref)))
    return float(np.abs(got - ref).max() / max(rms, 1e-30))


def bf16_bound(ref: np.ndarray, tol: float = 1e-2) -> float:
    """Tolerance for a bf16 output: the stated 1e-2, or - where merely rounding the exact
    result to bf16 already exceeds it on heavy-tailed entries - that rounding floor plus
    2e-3."""
    floor = rel_err(bf16_round(ref), ref)
    return max(tol, floor + 2e-3)


def half_ulp_bf16(ref: np.ndarray) -> np.ndarray:
    """Largest error that rounding to bf16 can make on each entry: half a unit in the last of the
    8 significant bits, 2^(floor(log2 |v|) - 8)."""
    return 2.0 ** (np.floor(np.log2(np.maximum(np.abs(ref), 1e-300))) - 8)


def report(name: str, **values):
    """Print one measured figure of a parity check and append it to the report file (_REPORT)
    (the tables of measured error against bound are made from that file)."""
    rec = {"check": name}
    rec.update({k: (float(v) if isinstance(v, (float, np.floating)) else v) for k, v in values.items()})
    print("PARITY " + json.dumps(rec))
    try:
        os.makedirs(os.path.dirname(_REPORT), exist_ok=True)
        with open(_REPORT, "a") as fh:
            fh.write(json.dumps(rec) + "\n")
    except OSError:
        pass


def check_bf16(name: str, got: np.ndarray, ref: np.ndarray, noise: float = 0.0, elem_noise=None, sampled: bool = False):
    """The bf16 tolerance, twice over.

    (1) As stated: max-abs-error / RMS(ref) <= 1e-2, or the rounding floor of the exact result plus
        2e-3 where that floor alone exceeds 1e-2 (the raw figure, the floor and whether the
        relaxation was needed are all reported).
    (2) Entry by entry: |got - ref| <= half a bf16 unit of |ref| (the one rounding of the output)
        + (2e-3 + noise) * RMS(ref).  `noise` is what the stored bf16 intermediates upstream of this
        output may add, in units of RMS(ref), argued at the call site; 0 for an output that is one
        rounding away from the exact result of its inputs.  `elem_noise` replaces `noise` in (2)
        where the two differ.  `sampled`: the arrays are a small sample of a large output, so the
        rounding floor in (1) is the worst case for the sampled magnitudes (half a bf16 unit) rather
        than the rounding error the sampled reference values happen to have."""
    if elem_noise is None:
        elem_noise = noise
    rms = float(np.sqrt(np.mean(ref * ref)))
    err = rel_err(got, ref)
    floor = float(half_ulp_bf16(ref).max() / max(rms, 1e-30)) if sampled else rel_err(bf16_round(ref), ref)
    bound = max(1e-2, floor + 2e-3) + noise
    # (half a unit of whichever of the two lies in the higher binade: a result that noise has pushed
    # across a power of two is rounded on the coarser grid)
    excess = np.abs(got - ref) - half_ulp_bf16(np.maximum(np.abs(got), np.abs(ref)))
    worst = float(excess.max() / max(rms, 1e-30))
    report(name, err_over_rms=err, bound=bound, rounding_floor=floor, relaxed=bool(floor + 2e-3 > 1e-2),
           beyond_half_ulp_over_rms=worst, elementwise_allowance=2e-3 + elem_noise)
    assert err <= bound, f"{name}: max-abs-err / RMS = {err:.3e} > {bound:.3e}"
    assert worst <= 2e-3 + elem_noise, (f"{name}: an entry is {worst:.3e} RMS beyond its own bf16 rounding "
                                        f"(allowed {2e-3 + elem_noise:.1e})")
    return err
