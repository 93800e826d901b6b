"""Shared helpers of the GPU parity tests: tolerance rule, oracle <-> flat-layout conversion."""
import numpy as np

RTOL_F32 = 1e-5     # pooled embeddings, MLP outputs, updated parameters on the float path
RTOL_BF16 = 2e-2    # outputs of bf16 GEMMs
RTOL_SYNC = 1e-6    # outputs of the synchronisation kernels


def assert_close(got, want, rtol, what="", floor=0.0, outlier_frac=0.0):
    """|got - want| <= rtol * max(|want|, rms(want)) element-wise.

    A pure element-wise relative error is undefined at exact zeros (ReLU outputs, pads) and meaningless
    for elements far below the tensor's scale, so the tensor's RMS is the floor of the reference scale.
    `floor` raises that floor to the magnitude of the operands when a tensor is too short for its RMS to
    say anything (rounding error scales with the operands, not with a result that cancelled).
    `outlier_frac` > 0 is for gradients behind ReLU gates at large sizes: a hidden unit whose pre-activation
    lies within rounding of zero may be on for one side and off for the other, which moves the few gradient
    entries that unit feeds by its whole contribution.  Up to that fraction of the elements may then exceed
    rtol, but none by more than twice the reference scale (still a gradient of the right size, not garbage).
    """
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    assert got.shape == want.shape, (what, got.shape, want.shape)
    assert np.isfinite(got).all(), f"{what}: non-finite values"
    rms = float(np.sqrt(np.mean(want * want))) if want.size else 0.0
    scale = np.maximum(np.abs(want), max(rms, floor))
    err = np.abs(got - want)
    bad = err > rtol * scale + 1e-30
    if outlier_frac > 0.0 and bad.mean() <= outlier_frac and (err <= 2.0 * scale + 1e-30).all():
        return
    if bad.any():
        i = np.unravel_index(np.argmax(err / (scale + 1e-30)), err.shape)
        raise AssertionError(f"{what}: {int(bad.sum())}/{bad.size} beyond rtol={rtol}; worst at {i}: "
                             f"got {got[i]!r} want {want[i]!r} (scale {scale[i]:.3e})")
