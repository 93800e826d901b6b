"""Shared helpers of the GPU parity tests: tolerance rule, oracle <-> flat-layout conversion."""
import numpy as np

RTOL_F32 = 1e-5     # pooled embeddings, MLP outputs, updated parameters on the float path
RTOL_BF16 = 2e-2    # outputs of bf16 GEMMs
RTOL_SYNC = 1e-6    # outputs of the synchronisation kernels


def assert_close(got, want, rtol, what="", floor=0.0):
    """|got - want| <= rtol * max(|want|, rms(want)) element-wise.

    A pure element-wise relative error is undefined at exact zeros (ReLU outputs, pads) and meaningless
    for elements far below the tensor's scale, so the tensor's RMS is the floor of the reference scale.
    `floor` raises that floor to the magnitude of the operands when a tensor is too short for its RMS to
    say anything (rounding error scales with the operands, not with a result that cancelled).
    """
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    assert got.shape == want.shape, (what, got.shape, want.shape)
    assert np.isfinite(got).all(), f"{what}: non-finite values"
    rms = float(np.sqrt(np.mean(want * want))) if want.size else 0.0
    scale = np.maximum(np.abs(want), max(rms, floor))
    err = np.abs(got - want)
    bad = err > rtol * scale + 1e-30
    if bad.any():
        i = np.unravel_index(np.argmax(err / (scale + 1e-30)), err.shape)
        raise AssertionError(f"{what}: {int(bad.sum())}/{bad.size} beyond rtol={rtol}; worst at {i}: "
                             f"got {got[i]!r} want {want[i]!r} (scale {scale[i]:.3e})")


# How close to zero, relative to the RMS pre-activation of its layer, a hidden unit must be for its ReLU gate to
# count as "at the edge".  Both sides feed the unit the same bf16 weights, but an input activation whose float value
# lies within float rounding of a bf16 rounding boundary may come out one bf16 ulp apart (2^-8 of that input) on the
# two sides; one such input moves the pre-activation by |a_k w_k| 2^-8, about rms(z) 2^-8 / sqrt(K) for a layer of K
# inputs, and a unit has a handful of them at most.  Observed distances of switched units: up to 1.0e-3 rms (large
# model, 3456 inputs); the limit is twice that, half a bf16 ulp.
GATE_DELTA = 2.0 ** -9


def match_relu_gates(fwd, backward, got_grad_pooled, rtol, n_bottom, n_layers, delta=GATE_DELTA, max_flips=3):
    """Let the oracle's backward take the ReLU decisions the kernels took, for units at the edge only.

    A ReLU gate is an on/off decision read from a floating-point value.  For a hidden unit whose
    pre-activation is within rounding of zero the two sides may decide differently, and both are right;
    the gradient of that one sample then differs by the unit's whole contribution.  Per the rule that a
    discrete decision is compared in the kernel's precision, the oracle follows the kernel there: for each
    sample whose grad_pooled row misses the tolerance, units with |pre| < delta * rms(pre of the layer) are
    switched, greedily, while that brings the row closer; no other unit may change.  The sample must then
    match, which the caller checks with the strict tolerance on every output of the step.  Only gates of
    the top MLP are ever switched (grad_pooled, the evidence used here, sees no others): a bottom-MLP gate
    decided differently by the two sides is NOT explained away and fails the caller's strict comparison of
    that layer's weight and bias steps.

    fwd: the oracle's forward dict (not modified); backward(fwd) -> grad_pooled [B, C] float64.
    Returns (fwd with the switched pre-activations, list of (sample, layer, unit)).
    """
    got = np.asarray(got_grad_pooled, dtype=np.float64)
    want = backward(fwd)
    rms = float(np.sqrt(np.mean(want * want)))

    def row_err(w, b):
        return float(np.max(np.abs(got[b] - w[b]) / np.maximum(np.abs(w[b]), rms)))

    bad = [b for b in range(got.shape[0]) if row_err(want, b) > rtol]
    if not bad:
        return fwd, []
    hidden = range(n_bottom, n_layers - 1)             # top MLP; its last layer has no ReLU
    pre_rms = {l: float(np.sqrt(np.mean(fwd["pre"][l] ** 2))) for l in hidden}
    out = dict(fwd)
    out["pre"] = [p.copy() for p in fwd["pre"]]
    flips = []
    for b in bad:
        cands = [(l, int(j)) for l in hidden for j in np.flatnonzero(np.abs(fwd["pre"][l][b]) < delta * pre_rms[l])]
        err = row_err(want, b)
        for _ in range(max_flips):
            best = None
            for l, j in cands:
                if (b, l, j) in flips:
                    continue
                keep = out["pre"][l][b, j]
                out["pre"][l][b, j] = -keep if keep != 0.0 else 1.0
                e = row_err(backward(out), b)
                out["pre"][l][b, j] = keep
                if e < err and (best is None or e < best[0]):
                    best = (e, l, j)
            if best is None:
                break
            err, l, j = best
            keep = out["pre"][l][b, j]
            out["pre"][l][b, j] = -keep if keep != 0.0 else 1.0
            flips.append((b, l, j))
            if err <= rtol:
                break
    return out, flips


def oracle_step_following_gates(O, tables, row_state, layers, accs, n_bottom, batch, lr, eps, bf16,
                                got_grad_pooled, rtol):
    """The oracle's replica step (same calls, same order as O.replica_step), its ReLU gates at the edge
    following the kernels' (match_relu_gates).  Returns (forward dict as replica_step does, gate switches)."""
    B = batch.dense.shape[0]
    pooled = O.embbag_fwd(tables, batch.indices, batch.offsets, B)
    fwd = O.mlp_fwd(layers, n_bottom, batch.dense, pooled, batch.labels, bf16)
    fwd, flips = match_relu_gates(fwd, lambda f: O.mlp_bwd(layers, n_bottom, f, batch.labels, bf16)[1],
                                  got_grad_pooled, rtol, n_bottom, len(layers))
    grads, grad_pooled = O.mlp_bwd(layers, n_bottom, fwd, batch.labels, bf16)
    for (W, b), (aW, ab), (dW, db) in zip(layers, accs, grads):
        W[...], aW[...] = O.adagrad_dense(W, aW, dW, lr, eps)
        b[...], ab[...] = O.adagrad_dense(b, ab, db, lr, eps)
    gp32 = grad_pooled.astype(np.float32)
    uniq, seg, perm = O.embbag_bwd_adagrad(tables, row_state, batch.indices, batch.offsets, B, gp32, lr, eps)
    fwd.update(pooled=pooled, grad_pooled=gp32, grads=grads, uniq_keys=uniq, seg_off=seg, perm=perm)
    return fwd, flips
