"""Shared helpers of the GPU parity tests."""
import math

import numpy as np
import torch

REL_TOL = 2e-2   # max relative error per output element (bf16 storage, fp32 accumulate)


def to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


def max_rel_err(got: np.ndarray, ref: np.ndarray) -> float:
    """max |g - r| / max(|r|, rho), rho = RMS of the reference tensor: the per-element relative
    error with elements near zero measured against the tensor's scale."""
    ref = np.asarray(ref, dtype=np.float64)
    rho = math.sqrt(float(np.mean(ref * ref))) if ref.size else 0.0
    den = np.maximum(np.abs(ref), max(rho, 1e-30))
    return float(np.max(np.abs(got - ref) / den)) if ref.size else 0.0


def assert_close(got, ref, what="", tol=REL_TOL):
    g = to_f64(got) if isinstance(got, torch.Tensor) else np.asarray(got, dtype=np.float64)
    assert np.all(np.isfinite(g)), f"{what}: non-finite output"
    e = max_rel_err(g.reshape(-1), np.asarray(ref).reshape(-1))
    assert e <= tol, f"{what}: max relative error {e:.3e} > {tol}"
    return e


def rel_l2_err(got: np.ndarray, ref: np.ndarray) -> float:
    ref = np.asarray(ref, dtype=np.float64)
    return float(np.sqrt(np.sum((got - ref) ** 2) / max(np.sum(ref * ref), 1e-300)))


# Bounds against the unrounded fp64 evaluation (mode A) for deep models, where the bf16 storage
# of intermediate tensors -- not the kernels -- sets the error: see assert_parity.
MODE_A_L2_TOL = 2e-2
DEEP_MODE_A_L2_TOL = 4e-2   # modes A and B themselves differ by about 2e-2 in relative L2 at 16 layers
MODE_A_MAX_TOL = 1.5e-1
DEEP_L2_TOL = 2e-2


def assert_parity(got, ref_a, ref_b, what="", deep=False):
    """The stated tolerance (max relative error 2e-2 per element under bf16 storage with fp32
    accumulate) is checked against the oracle evaluated with bf16 rounding at the contract's storage
    points (mode B: fp64 arithmetic between them).  Against the unrounded evaluation (mode A) the
    difference is the storage noise of the contract itself, which compounds with depth; it is
    bounded in relative L2 by 2e-2 and element-wise by a loose 1.5e-1, and returned for reporting.

    deep=True (random-weight decoders of the 1B/8B layer shapes, two or more layers): a single bf16 rounding that falls the other
    way is amplified by the later layers, so two correct evaluations differ element-wise by more
    than 2e-2 on a few of the 32000 logits; there the mode-B check is relative L2 <= 2e-2 and the
    same loose element-wise bound, while the strict element-wise check runs on the 1-layer version
    of the same shapes and on the small models."""
    g = to_f64(got) if isinstance(got, torch.Tensor) else np.asarray(got, dtype=np.float64)
    g = g.reshape(-1)
    assert np.all(np.isfinite(g)), f"{what}: non-finite output"
    a, b = np.asarray(ref_a).reshape(-1), np.asarray(ref_b).reshape(-1)
    eb = max_rel_err(g, b)
    ea, el2 = max_rel_err(g, a), rel_l2_err(g, a)
    elb = rel_l2_err(g, b)
    if deep:
        assert elb <= DEEP_L2_TOL, f"{what}: relative L2 error vs bf16-storage oracle {elb:.3e} > {DEEP_L2_TOL}"
        assert eb <= MODE_A_MAX_TOL, f"{what}: max relative error vs bf16-storage oracle {eb:.3e} > {MODE_A_MAX_TOL}"
    else:
        assert eb <= REL_TOL, f"{what}: max relative error vs bf16-storage oracle {eb:.3e} > {REL_TOL}"
    la = DEEP_MODE_A_L2_TOL if deep else MODE_A_L2_TOL
    assert el2 <= la, f"{what}: relative L2 error vs fp64 oracle {el2:.3e} > {la}"
    assert ea <= MODE_A_MAX_TOL, f"{what}: max relative error vs fp64 oracle {ea:.3e} > {MODE_A_MAX_TOL}"
    return {"max_rel_vs_storage_oracle": eb, "rel_l2_vs_storage_oracle": elb, "max_rel_vs_fp64": ea,
            "rel_l2_vs_fp64": el2}


def check_argmax(gpu_argmax: int, gpu_logits: torch.Tensor, ref_logits: np.ndarray, tol=REL_TOL):
    """(i) the device argmax equals the lowest-index argmax of the device's own logits, bit-exact;
    (ii) it equals the reference argmax when the reference's top-2 gap exceeds twice the tolerance
    band; (iii) otherwise it must be one of the reference entries inside that band.
    Returns True when the case was decided by (ii)."""
    own = to_f64(gpu_logits)
    assert gpu_argmax == int(np.argmax(own)), "argmax kernel disagrees with its own logits"
    ref = np.asarray(ref_logits, dtype=np.float64)
    rho = math.sqrt(float(np.mean(ref * ref)))
    order = np.argsort(-ref, kind="stable")
    top1, top2 = ref[order[0]], ref[order[1]] if ref.size > 1 else -np.inf
    band = 2 * tol * max(abs(top1), rho)
    if top1 - top2 > band:
        assert gpu_argmax == int(order[0]), "argmax differs from the oracle outside the tie band"
        return True
    assert ref[gpu_argmax] >= top1 - band, "argmax is not among the oracle's near-maximal entries"
    return False
