"""Pins for the oracle's training step: embedding pooling, sort/unique, segment reduction with row-wise
Adagrad, MLP forward/backward, dense Adagrad.  CPU only; the pins are library routines (torch in
float64), finite differences, brute force and closed forms."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import shadowsync_oracle as O


def _bags(rng, T, N, B, max_len=5, min_len=0):
    lens = rng.integers(min_len, max_len + 1, T * B)
    offsets = np.zeros(T * B + 1, np.int32)
    offsets[1:] = np.cumsum(lens)
    indices = rng.integers(0, N, int(offsets[-1])).astype(np.int32)
    return indices, offsets


# ---------------------------------------------------------------- embedding forward
def test_embbag_fwd_all_ones_counts_bag_length():
    rng = np.random.default_rng(0)
    T, N, D, B = 3, 11, 4, 5
    idx, off = _bags(rng, T, N, B)
    pooled = O.embbag_fwd(np.ones((T, N, D), np.float32), idx, off, B)
    lens = np.diff(off).reshape(T, B).T
    assert np.array_equal(pooled, np.broadcast_to(lens[:, :, None], (B, T, D)).astype(np.float32))


def test_embbag_fwd_single_lookup_is_row_copy_and_duplicates_count_twice():
    tables = np.random.default_rng(1).normal(size=(2, 7, 3)).astype(np.float32)
    idx = np.array([4, 2, 6, 6], np.int32)          # table0: bag0=[4], bag1=[2]; table1: bag0=[6,6], bag1=[]
    off = np.array([0, 1, 2, 4, 4], np.int32)
    p = O.embbag_fwd(tables, idx, off, 2)
    assert np.array_equal(p[0, 0], tables[0, 4]) and np.array_equal(p[1, 0], tables[0, 2])
    assert np.array_equal(p[0, 1], 2 * tables[1, 6]) and not p[1, 1].any()


def test_embbag_fwd_matches_torch_embedding_bag():
    rng = np.random.default_rng(2)
    T, N, D, B = 4, 50, 8, 9
    tables = rng.normal(size=(T, N, D)).astype(np.float32)
    idx, off = _bags(rng, T, N, B, 6)
    p = O.embbag_fwd(tables, idx, off, B)
    for t in range(T):
        o = torch.from_numpy(off[t * B:(t + 1) * B + 1].astype(np.int64))
        i = torch.from_numpy(idx[int(o[0]):int(o[-1])].astype(np.int64))
        ref = torch.nn.functional.embedding_bag(i, torch.from_numpy(tables[t]).double(), o[:-1] - o[0], mode="sum")
        np.testing.assert_allclose(p[:, t], ref.numpy(), rtol=1e-6, atol=1e-7)


# ---------------------------------------------------------------- sort / unique
def test_sort_unique_against_python_sorted():
    rng = np.random.default_rng(3)
    T, N, B = 3, 6, 8
    idx, off = _bags(rng, T, N, B, 4)
    uniq, seg, perm = O.sort_unique(idx, off, T, N, B)
    L = int(off[-1])
    table_of = [next(bag for bag in range(T * B) if off[bag] <= p < off[bag + 1]) // B for p in range(L)]
    keys = [table_of[p] * N + int(idx[p]) for p in range(L)]
    want = sorted(range(L), key=lambda p: (keys[p], p))
    assert list(perm) == want
    assert list(uniq) == sorted(set(keys))
    for u, k in enumerate(uniq):
        assert [keys[p] for p in perm[seg[u]:seg[u + 1]]] == [k] * (seg[u + 1] - seg[u])
    assert seg[0] == 0 and seg[-1] == L


# ---------------------------------------------------------------- embedding backward + row-wise Adagrad
def test_embbag_bwd_segment_sums_match_torch_autograd_and_bruteforce():
    rng = np.random.default_rng(4)
    T, N, D, B = 3, 9, 4, 6
    tables0 = rng.normal(size=(T, N, D)).astype(np.float32)
    idx, off = _bags(rng, T, N, B, 5)
    gp = rng.normal(size=(B, T * D)).astype(np.float32)
    lr, eps = 0.1, 1e-8
    tables, state = tables0.copy(), np.zeros((T, N), np.float32)
    O.embbag_bwd_adagrad(tables, state, idx, off, B, gp, lr, eps)
    # dense table gradient from torch autograd (double) through embedding_bag
    for t in range(T):
        w = torch.from_numpy(tables0[t]).double().requires_grad_()
        o = torch.from_numpy(off[t * B:(t + 1) * B + 1].astype(np.int64))
        i = torch.from_numpy(idx[int(o[0]):int(o[-1])].astype(np.int64))
        out = torch.nn.functional.embedding_bag(i, w, o[:-1] - o[0], mode="sum")
        out.backward(torch.from_numpy(gp.reshape(B, T, D)[:, t]).double())
        G = w.grad.numpy()
        s = (G * G).mean(axis=1)
        touched = np.zeros(N, bool)
        touched[idx[int(o[0]):int(o[-1])]] = True
        want = tables0[t].astype(np.float64) - np.where(touched[:, None], lr * G / (np.sqrt(s)[:, None] + eps), 0.0)
        np.testing.assert_allclose(tables[t], want, rtol=2e-6, atol=1e-7)
        np.testing.assert_allclose(state[t], s, rtol=2e-6, atol=1e-12)
        assert np.array_equal(tables[t][~touched], tables0[t][~touched])


def test_rowwise_adagrad_d1_is_elementwise_adagrad_and_first_step_closed_form():
    # D = 1: mean over the row of g^2 is g^2 -> textbook Adagrad (torch.optim.Adagrad)
    N, B = 5, 4
    tables = np.linspace(-1, 1, N, dtype=np.float32).reshape(1, N, 1)
    state = np.zeros((1, N), np.float32)
    idx = np.array([0, 3, 3, 1], np.int32)
    off = np.arange(B + 1, dtype=np.int32)
    gp = np.array([[0.5], [-0.25], [1.0], [2.0]], np.float32)
    p = torch.nn.Parameter(torch.from_numpy(tables[0, :, 0].copy()).double())
    opt = torch.optim.Adagrad([p], lr=0.05, eps=1e-8)
    for step in range(3):
        O.embbag_bwd_adagrad(tables, state, idx, off, B, gp, 0.05, 1e-8)
        g = torch.zeros(N, dtype=torch.float64)
        g.index_add_(0, torch.from_numpy(idx.astype(np.int64)), torch.from_numpy(gp[:, 0]).double())
        p.grad = g
        opt.step()
        # torch also "updates" untouched rows with g = 0: no change there
        np.testing.assert_allclose(tables[0, :, 0], p.detach().numpy(), rtol=1e-6)
    # first touch of a row with D > 1 moves it by lr * g / (rms(g) + eps)
    D = 4
    tables = np.zeros((1, 2, D), np.float32)
    state = np.zeros((1, 2), np.float32)
    g = np.array([[1.0, -2.0, 3.0, 0.5]], np.float32)
    O.embbag_bwd_adagrad(tables, state, np.array([1], np.int32), np.array([0, 1], np.int32), 1, g, 0.1, 0.0)
    rms = math.sqrt(float((g.astype(np.float64) ** 2).mean()))
    np.testing.assert_allclose(tables[0, 1], -0.1 * g[0] / rms, rtol=1e-6)
    assert not tables[0, 0].any() and abs(state[0, 1] - rms * rms) < 1e-6


# ---------------------------------------------------------------- MLP
def _tiny_mlp(rng, bottom=(5, 7, 3), top=None, T=2, D=3):
    top = top or ((1 + T) * D, 6, 1)
    layers = []
    for dims in (bottom, top):
        for i in range(len(dims) - 1):
            a = math.sqrt(6.0 / (dims[i] + dims[i + 1]))
            layers.append((rng.uniform(-a, a, (dims[i + 1], dims[i])).astype(np.float32),
                           rng.uniform(-0.1, 0.1, dims[i + 1]).astype(np.float32)))
    return layers, len(bottom) - 1


def _torch_loss(layers, nb, dense, pooled, labels):
    ps = [(torch.from_numpy(W).double().requires_grad_(), torch.from_numpy(b).double().requires_grad_()) for W, b in layers]
    pooled_t = torch.from_numpy(pooled).double().requires_grad_()
    x = torch.from_numpy(dense).double()
    for l in range(nb):
        x = torch.relu(x @ ps[l][0].T + ps[l][1])
    x = torch.cat([x, pooled_t.reshape(x.shape[0], -1)], dim=1)
    for l in range(nb, len(ps)):
        x = x @ ps[l][0].T + ps[l][1]
        if l < len(ps) - 1:
            x = torch.relu(x)
    loss = torch.nn.functional.binary_cross_entropy_with_logits(x[:, 0], torch.from_numpy(labels).double())
    return loss, ps, pooled_t, x[:, 0]


def test_mlp_fwd_bwd_match_torch_autograd_double():
    rng = np.random.default_rng(5)
    layers, nb = _tiny_mlp(rng, bottom=(5, 7, 4, 3), top=(9, 6, 5, 1))
    B, T, D = 6, 2, 3
    dense = rng.normal(size=(B, 5)).astype(np.float32)
    pooled = rng.normal(size=(B, T, D)).astype(np.float32)
    labels = (rng.random(B) < 0.4).astype(np.float32)
    fwd = O.mlp_fwd(layers, nb, dense, pooled, labels)
    grads, gp = O.mlp_bwd(layers, nb, fwd, labels)
    loss, ps, pooled_t, z = _torch_loss(layers, nb, dense, pooled, labels)
    loss.backward()
    assert abs(fwd["loss"] - loss.item()) < 1e-12
    np.testing.assert_allclose(fwd["logit"], z.detach().numpy(), rtol=1e-12)
    np.testing.assert_allclose(fwd["prob"], torch.sigmoid(z).detach().numpy(), rtol=1e-12)
    for (dW, db), (W, b) in zip(grads, ps):
        np.testing.assert_allclose(dW, W.grad.numpy(), rtol=1e-9, atol=1e-14)
        np.testing.assert_allclose(db, b.grad.numpy(), rtol=1e-9, atol=1e-14)
    np.testing.assert_allclose(gp, pooled_t.grad.numpy().reshape(B, -1), rtol=1e-9, atol=1e-14)


def test_mlp_gradients_match_central_finite_differences():
    rng = np.random.default_rng(6)
    layers, nb = _tiny_mlp(rng)
    B, T, D = 4, 2, 3
    dense = rng.normal(size=(B, 5)).astype(np.float32)
    pooled = rng.normal(size=(B, T, D)).astype(np.float32)
    labels = np.array([1, 0, 0, 1], np.float32)
    fwd = O.mlp_fwd(layers, nb, dense, pooled, labels)
    grads, gp = O.mlp_bwd(layers, nb, fwd, labels)
    h = 1e-3  # float32 parameters: the step must survive the float32 store; the loss is smooth off the ReLU kinks

    def loss_with(l, which, ix, delta):
        lay = [(W.astype(np.float64).copy(), b.astype(np.float64).copy()) for W, b in layers]
        lay[l][which][ix] += delta
        # bypass float32 storage so the finite difference is exact in double
        return O.mlp_fwd([(W, b) for W, b in lay], nb, dense, pooled, labels)["loss"]

    for l in range(len(layers)):
        W, b = layers[l]
        for ix in [(0, 0), (W.shape[0] - 1, W.shape[1] - 1), (W.shape[0] // 2, W.shape[1] // 2)]:
            fd = (loss_with(l, 0, ix, h) - loss_with(l, 0, ix, -h)) / (2 * h)
            assert abs(fd - grads[l][0][ix]) < 2e-6 + 1e-3 * abs(fd), (l, ix, fd, grads[l][0][ix])
        fd = (loss_with(l, 1, (0,), h) - loss_with(l, 1, (0,), -h)) / (2 * h)
        assert abs(fd - grads[l][1][0]) < 2e-6 + 1e-3 * abs(fd)
    # gradient with respect to the pooled embeddings
    for (bi, ti, di) in [(0, 0, 0), (3, 1, 2), (2, 0, 1)]:
        pp, pm = pooled.astype(np.float64).copy(), pooled.astype(np.float64).copy()
        pp[bi, ti, di] += h
        pm[bi, ti, di] -= h
        fd = (O.mlp_fwd(layers, nb, dense, pp, labels)["loss"] - O.mlp_fwd(layers, nb, dense, pm, labels)["loss"]) / (2 * h)
        assert abs(fd - gp[bi, ti * D + di]) < 2e-6 + 1e-3 * abs(fd)


def test_mlp_zero_weights_give_ln2_and_half_minus_label():
    layers = [(np.zeros((4, 3), np.float32), np.zeros(4, np.float32)),
              (np.zeros((1, 4 + 2), np.float32), np.zeros(1, np.float32))]
    dense = np.ones((2, 3), np.float32)
    pooled = np.ones((2, 1, 2), np.float32)
    labels = np.array([1.0, 0.0], np.float32)
    fwd = O.mlp_fwd(layers, 1, dense, pooled, labels)
    assert abs(fwd["loss"] - math.log(2.0)) < 1e-15 and np.array_equal(fwd["prob"], [0.5, 0.5])
    grads, gp = O.mlp_bwd(layers, 1, fwd, labels)
    # d loss / d z = (p - y) / B = (-0.25, +0.25); concat = [relu(0)=0 | pooled=1]
    np.testing.assert_allclose(grads[1][1], [0.0])
    np.testing.assert_allclose(grads[1][0], [[0, 0, 0, 0, 0.0, 0.0]])


def test_single_linear_layer_hand_computation():
    # bottom: identity-like 1x1 layer; top: 2 -> 1.  z = w.[relu(a*x+c), e] + b
    layers = [(np.array([[2.0]], np.float32), np.array([1.0], np.float32)),
              (np.array([[0.5, -1.0]], np.float32), np.array([0.25], np.float32))]
    dense = np.array([[1.5]], np.float32)
    pooled = np.array([[[2.0]]], np.float32)
    y = np.array([1.0], np.float32)
    fwd = O.mlp_fwd(layers, 1, dense, pooled, y)
    z = 0.5 * (2 * 1.5 + 1) - 1.0 * 2.0 + 0.25            # = 0.25
    assert abs(fwd["logit"][0] - z) < 1e-15
    p = 1 / (1 + math.exp(-z))
    grads, gp = O.mlp_bwd(layers, 1, fwd, y)
    dz = p - 1.0
    np.testing.assert_allclose(grads[1][0], [[dz * 4.0, dz * 2.0]], rtol=1e-12)
    np.testing.assert_allclose(gp, [[dz * -1.0]], rtol=1e-12)
    np.testing.assert_allclose(grads[0][0], [[dz * 0.5 * 1.5]], rtol=1e-12)
    np.testing.assert_allclose(grads[0][1], [dz * 0.5], rtol=1e-12)


def test_bf16_mode_rounds_only_matrix_operands():
    rng = np.random.default_rng(7)
    layers, nb = _tiny_mlp(rng)
    B, T, D = 4, 2, 3
    dense = rng.normal(size=(B, 5)).astype(np.float32)
    pooled = rng.normal(size=(B, T, D)).astype(np.float32)
    labels = np.array([1, 0, 0, 1], np.float32)
    # inputs already representable in bf16 -> both modes agree on the first layer's pre-activation
    layers_r = [(O.round_bf16(W).astype(np.float32), b) for W, b in layers]
    dense_r = O.round_bf16(dense).astype(np.float32)
    a = O.mlp_fwd(layers_r, nb, dense_r, pooled, labels, bf16=False)
    b = O.mlp_fwd(layers_r, nb, dense_r, pooled, labels, bf16=True)
    np.testing.assert_allclose(a["pre"][0], b["pre"][0], rtol=1e-14)
    assert abs(a["loss"] - b["loss"]) < 2e-2 * abs(a["loss"])
    full = O.mlp_fwd(layers, nb, dense, pooled, labels, bf16=False)
    half = O.mlp_fwd(layers, nb, dense, pooled, labels, bf16=True)
    np.testing.assert_allclose(half["logit"], full["logit"], atol=3e-2)


# ---------------------------------------------------------------- dense Adagrad
def test_dense_adagrad_matches_torch_optim_and_first_step_is_lr_sign():
    rng = np.random.default_rng(8)
    th = rng.normal(size=20).astype(np.float32)
    acc = np.zeros(20, np.float32)
    p = torch.nn.Parameter(torch.from_numpy(th.copy()).double())
    opt = torch.optim.Adagrad([p], lr=0.01, eps=1e-8)
    th1, _ = O.adagrad_dense(th, acc, np.where(np.arange(20) % 2 == 0, 0.3, -7.0), 0.01, 1e-8)
    np.testing.assert_allclose(th1 - th, np.where(np.arange(20) % 2 == 0, -0.01, 0.01), rtol=1e-4)
    for _ in range(4):
        g = rng.normal(size=20)
        th, acc = O.adagrad_dense(th, acc, g, 0.01, 1e-8)
        p.grad = torch.from_numpy(g)
        opt.step()
        np.testing.assert_allclose(th, p.detach().numpy(), rtol=1e-5, atol=1e-7)


# ---------------------------------------------------------------- whole run
def test_train_run_tiny_shapes_loss_is_finite_and_sync_pulls_replicas_together():
    rng = np.random.default_rng(9)
    T, N, D, B, R, S = 2, 20, 3, 8, 2, 6
    layers, nb = _tiny_mlp(rng, bottom=(5, 7, 3), top=(9, 6, 1))

    class Bt:
        pass

    def batch():
        b = Bt()
        b.indices, b.offsets = _bags(rng, T, N, B, 4, 1)
        b.dense = rng.normal(size=(B, 5)).astype(np.float32)
        b.labels = (rng.random(B) < 0.3).astype(np.float32)
        return b

    batches = [[batch() for _ in range(S)] for _ in range(R)]

    def run(sync):
        tables = rng_tables.copy()
        reps = [[(W.copy(), b.copy()) for W, b in layers] for _ in range(R)]
        losses, _, centre = O.train_run(tables, reps, nb, batches, 0.05, 1e-8, sync, 2, 0.5)
        return losses, reps, centre

    rng_tables = rng.uniform(-0.05, 0.05, (T, N, D)).astype(np.float32)
    l0, reps0, _ = run(None)
    l1, reps1, c1 = run("easgd")
    assert np.isfinite(l0).all() and np.isfinite(l1).all()
    gap0 = np.abs(O.flatten(reps0[0]) - O.flatten(reps0[1])).max()
    gap1 = np.abs(O.flatten(reps1[0]) - O.flatten(reps1[1])).max()
    assert gap1 < gap0            # elastic averaging keeps the replicas closer than no sync
    assert np.array_equal(np.array(l0[:2]), np.array(l1[:2]))   # identical until the first sync


def test_gate_matching_recovers_planted_edge_gates_and_nothing_else():
    """The helper that lets the oracle follow the kernels' ReLU decisions switches only units whose
    pre-activation is within the stated distance of zero: planted switches at such units are found,
    a switch at an ordinary unit is left unexplained (the caller's strict comparison then fails)."""
    from parity import match_relu_gates
    from paper_2003_03477_b200 import synth
    cfg = synth.scaled(synth.CONFIGS["tiny"], B=24)
    layers = synth.initial_weights(cfg)
    nb = len(cfg.bottom) - 1
    batch = synth.make_batch(cfg, 0, 0)
    pooled = O.embbag_fwd(synth.tables_dense(cfg), batch.indices, batch.offsets, cfg.B)
    fwd = O.mlp_fwd(layers, nb, batch.dense, pooled, batch.labels, False)
    backward = lambda f: O.mlp_bwd(layers, nb, f, batch.labels, False)[1]
    # move two pre-activations to the edge, then produce the "other side's" gradient with their gates switched
    edge = dict(fwd); edge["pre"] = [p.copy() for p in fwd["pre"]]
    planted = [(3, nb, 1), (17, nb, 40), (17, nb, 7)]
    for b, l, j in planted:
        edge["pre"][l][b, j] = 1e-9
    other = dict(edge); other["pre"] = [p.copy() for p in edge["pre"]]
    for b, l, j in planted:
        other["pre"][l][b, j] = -1e-9
    got = backward(other)
    assert np.abs(got - backward(edge)).max() > 0
    matched, flips = match_relu_gates(edge, backward, got, 1e-9, nb, len(layers))
    assert sorted(flips) == sorted(planted)
    np.testing.assert_allclose(backward(matched), got, rtol=1e-12, atol=0)
    # a switched gate at a unit far from zero is a mistake, not a rounding decision
    far = dict(fwd); far["pre"] = [p.copy() for p in fwd["pre"]]
    b, l = 5, nb
    j = int(np.argmax(np.abs(fwd["pre"][l][b])))
    far["pre"][l][b, j] = -far["pre"][l][b, j]
    wrong = backward(far)
    assert np.abs(wrong - backward(fwd)).max() > 0
    matched, flips = match_relu_gates(fwd, backward, wrong, 1e-9, nb, len(layers))
    assert np.abs(backward(matched) - wrong)[b].max() > 0


# ---------------------------------------------------------------- bf16 backward: which tensors are rounded, and where
def _hand_bf16_case():
    """The hand-computed case of tests/golden/mlp_bwd_bf16_hand.txt (inputs typed in here, results read from the file)."""
    layers = [(np.array([[0.5]], np.float32), np.zeros(1, np.float32)),
              (np.array([[1.0078125, 1.005859375], [-1.0, 3.0]], np.float32), np.zeros(2, np.float32)),
              (np.array([[1.005859375, -0.75]], np.float32), np.zeros(1, np.float32))]
    fwd = dict(inputs=[np.array([[1.005859375], [5.0]]),
                       np.array([[0.75, 1.005859375], [0.0, -2.0078125]]),
                       np.array([[1.005859375, 0.0], [0.5, 2.0078125]])],
               pre=[np.array([[0.75], [-1.0]]), np.array([[1.005859375, -0.5], [0.5, 2.0078125]]), np.zeros((2, 1))],
               prob=np.array([0.25, 0.5029296875]), logit=np.zeros(2))
    want = {}
    with open(os.path.join(os.path.dirname(__file__), "golden", "mlp_bwd_bf16_hand.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                name, *vals = line.split()
                want[name] = np.array([float(v) for v in vals])
    return layers, fwd, np.array([1.0, 0.0]), want


def test_mlp_bwd_bf16_matches_the_hand_computed_case():
    """Pins the bf16 branch of the backward pass: gradients are rounded after the ReLU mask where they enter a
    product, weights and saved inputs are rounded as operands, bias gradients sum the rounded values, and the
    gradient of the pooled embeddings leaves unrounded.  All values are dyadic, so the comparison is exact."""
    layers, fwd, y, want = _hand_bf16_case()
    grads, gp = O.mlp_bwd(layers, 1, fwd, y, bf16=True)
    for l in range(3):
        assert np.array_equal(grads[l][0].ravel(), want[f"dW{l}"]), (l, grads[l][0])
        assert np.array_equal(grads[l][1].ravel(), want[f"db{l}"]), (l, grads[l][1])
    assert np.array_equal(gp.ravel(), want["grad_pooled"])
    # the case separates the readings: without any rounding every quantity but the masked zeros differs,
    # a rounded grad_pooled or bias gradients summed before rounding would differ too
    g64, gp64 = O.mlp_bwd(layers, 1, fwd, y, bf16=False)
    assert abs(g64[2][1][0] - want["db2"][0]) > 1e-4 and abs(g64[1][1][0] - want["db1"][0]) > 1e-4
    assert abs(g64[0][0][0, 0] - want["dW0"][0]) > 1e-3
    assert not np.array_equal(O.round_bf16(want["grad_pooled"]), want["grad_pooled"])
    d1 = np.array([[-0.3779296875, 0.0], [0.2539215087890625, -0.18896484375]])      # layer-1 gradient before rounding
    assert not np.array_equal(d1.sum(axis=0), want["db1"])


def test_mlp_fwd_bf16_rounds_operands_but_neither_bias_nor_pre_activation():
    """Forward, one unit by hand: r(1.005859375) * r(0.50390625) + 2^-12 with r(1.005859375) = 1.0078125 and
    0.50390625 = 0.5 * (1 + 2^-7) on the bf16 grid: 0.5078430175781250 + 0.000244140625, a value off the grid."""
    layers = [(np.array([[0.50390625]], np.float32), np.array([2.0 ** -12], np.float32)),
              (np.array([[1.0, 1.0]], np.float32), np.zeros(1, np.float32))]
    f = O.mlp_fwd(layers, 1, np.array([[1.005859375]], np.float32), np.zeros((1, 1, 1), np.float32),
                  np.array([1.0], np.float32), bf16=True)
    assert f["pre"][0][0, 0] == 1.0078125 * 0.50390625 + 2.0 ** -12
    # the next layer reads the activation rounded to bf16: r(0.508087158203125) = 0.5078125
    assert f["logit"][0] == 0.5078125
