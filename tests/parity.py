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


# Bounds against the unrounded fp64 evaluation (mode A), where the bf16 storage of intermediate
# tensors -- not the kernels -- sets the error: see assert_parity.
MODE_A_L2_TOL = 2e-2
MODE_A_MAX_TOL = 1.5e-1
# Deep models, end to end: the device's distance from the bf16-storage evaluation (mode B) relative to the
# distance between the two correct evaluations (mode A and mode B) of the same request.  Once a single
# bf16 rounding falls the other way (fp32 against fp64 accumulation next to a rounding boundary), every
# element downstream moves by about 1e-4 relative and a few per cent of them round the other way in turn:
# within a few layers the device is one more "rounding realisation", as far from mode B as an independent
# set of roundings would be.  Measured on B200 (1B shapes, 16 layers; 8B shapes, 32 layers): 0.6 to 0.8 of
# the A-B gap in relative L2, 0.6 to 0.95 of it for the worst element.  So end to end the device must be
# closer to mode B than mode A is; the strict 2e-2 per element is checked layer by layer instead
# (tests/test_gpu_step.py::replay_layers), where nothing compounds.
DEEP_L2_FRACTION = 1.0
DEEP_MAX_FRACTION = 1.25
# Two correct evaluations of a deep random-weight decoder differ by this much at most (recorded by
# tests/test_oracle_pins.py::test_mode_a_vs_mode_b_gap_at_the_1b_layer_shapes: 1.8e-2 / 7.9e-2 at 16 layers).
DEEP_GAP_L2_CEIL = 4e-2
DEEP_GAP_MAX_CEIL = 1.5e-1


def assert_parity(got, ref_a, ref_b, what="", deep=False):
    """The stated tolerance (max relative error 2e-2 per element under bf16 storage with fp32
    accumulate) is checked against the oracle evaluated with bf16 rounding at the contract's storage
    points (mode B: fp64 arithmetic between them).  Against the unrounded evaluation (mode A) the
    difference is the storage noise of the contract itself, which compounds with depth; it is
    bounded in relative L2 by 2e-2 and element-wise by a loose 1.5e-1, and returned for reporting.

    deep=True (random-weight decoders of the 1B/8B layer shapes, two or more layers): a single bf16
    rounding that falls the other way is amplified by the later layers, so two correct evaluations
    (modes A and B) differ element-wise by more than 2e-2 on a few of the 32000 logits.  A fixed bound
    of that size would let a kernel error as large as the storage noise pass, so the bound is tied to
    the request's own gap between the two evaluations: the device must be closer to mode B (relative
    L2) than mode A is, and its worst element at most 1.25 x mode A's worst element away.  The gap
    itself must stay under the ceilings recorded on the CPU.  The strict element-wise check of such
    models is made layer by layer on the device's own layer inputs (replay_layers in
    tests/test_gpu_step.py), on the 1-layer version of the same shapes and on the small models."""
    g = to_f64(got) if isinstance(got, torch.Tensor) else np.asarray(got, dtype=np.float64)
    g = g.reshape(-1)
    assert np.all(np.isfinite(g)), f"{what}: non-finite output"
    a, b = np.asarray(ref_a).reshape(-1), np.asarray(ref_b).reshape(-1)
    eb = max_rel_err(g, b)
    ea, el2 = max_rel_err(g, a), rel_l2_err(g, a)
    elb = rel_l2_err(g, b)
    out = {"max_rel_vs_storage_oracle": eb, "rel_l2_vs_storage_oracle": elb, "max_rel_vs_fp64": ea, "rel_l2_vs_fp64": el2}
    if deep:
        gap_l2, gap_max = rel_l2_err(a, b), max_rel_err(a, b)
        out.update({"gap_rel_l2_a_vs_b": gap_l2, "gap_max_rel_a_vs_b": gap_max})
        print(f"{what}: rel L2 device-B {elb:.3e}, A-B {gap_l2:.3e}; max rel device-B {eb:.3e}, A-B {gap_max:.3e}; "
              f"device-A L2 {el2:.3e} max {ea:.3e}")
        assert gap_l2 <= DEEP_GAP_L2_CEIL and gap_max <= DEEP_GAP_MAX_CEIL, \
            f"{what}: the two oracle evaluations differ by {gap_l2:.3e} (L2) / {gap_max:.3e} (max): not a usable reference"
        assert elb <= DEEP_L2_FRACTION * gap_l2, \
            f"{what}: relative L2 vs bf16-storage oracle {elb:.3e} > {DEEP_L2_FRACTION} x the A-B gap {gap_l2:.3e}"
        assert eb <= DEEP_MAX_FRACTION * gap_max, \
            f"{what}: max relative error vs bf16-storage oracle {eb:.3e} > {DEEP_MAX_FRACTION} x the A-B gap {gap_max:.3e}"
        assert el2 <= 1.5 * gap_l2, f"{what}: relative L2 vs fp64 oracle {el2:.3e} > 1.5 x the A-B gap {gap_l2:.3e}"
        return out
    assert eb <= REL_TOL, f"{what}: max relative error vs bf16-storage oracle {eb:.3e} > {REL_TOL}"
    assert el2 <= MODE_A_L2_TOL, f"{what}: relative L2 error vs fp64 oracle {el2:.3e} > {MODE_A_L2_TOL}"
    assert ea <= MODE_A_MAX_TOL, f"{what}: max relative error vs fp64 oracle {ea:.3e} > {MODE_A_MAX_TOL}"
    return out


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
