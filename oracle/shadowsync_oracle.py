"""CPU oracle for the ShadowSync hot path.  TEST INFRASTRUCTURE, not the product.

A plain, slow numpy implementation of what the path computes: the DLRM-style
CTR training step of one trainer replica (paper Section 3.1 "Trainer", Fig. 1)
and the three background synchronisation rules (Algorithms 2, 3 and 4).  Only
the tests, the smoke check and the benchmark's CPU-baseline leg may import it;
it shares no code with the CUDA path and imports nothing from the package.

Precision.  Parameters, tables and optimizer state are stored in float32 (as
the GPU stores them); every function converts to float64, does all of its
arithmetic there and rounds the stored results to float32 once.  With
``bf16=True`` every operand of a matrix product is first rounded to bfloat16
(round to nearest even) — the products and sums stay in float64 — which is the
precision the tensor-core path computes in.

Pins (tests/test_oracle_*.py): finite differences and torch autograd in
float64 for the MLP, torch.optim.Adagrad for the dense update, torch
EmbeddingBag for pooling and its gradient, python sorted() for the sort,
brute-force loops for the segment reduction, closed forms and conservation
laws for Algorithms 2-4.  The row-wise Adagrad formula (one accumulator per
row, incremented by the mean of the squared gradient over the row) is not
given by the paper, which only names Adagrad (Section 3.2): parity unpinned by
the paper for that formula; it is pinned to its written definition, to the
D=1 case (= element-wise Adagrad) and to the first-step closed form.
"""
from __future__ import annotations

import numpy as np

F32 = np.float32
F64 = np.float64


# --------------------------------------------------------------------------------------
# helpers
# --------------------------------------------------------------------------------------
def round_bf16(x):
    """Round float values to the nearest bfloat16 (ties to even); returns float64 holding bf16 values."""
    f = np.ascontiguousarray(np.asarray(x, dtype=F32))
    u = f.view(np.uint32).astype(np.uint64)
    rounded = ((u + np.uint64(0x7FFF) + ((u >> np.uint64(16)) & np.uint64(1))) >> np.uint64(16)) << np.uint64(16)
    out = rounded.astype(np.uint32).view(F32)
    out = np.where(np.isnan(f), f, out)
    return out.astype(F64)


def _operand(x, bf16):
    return round_bf16(x) if bf16 else np.asarray(x, dtype=F64)


# --------------------------------------------------------------------------------------
# embedding lookup + pooling  (Section 3.1, "Embedding PS": pooling is done next to the table)
# --------------------------------------------------------------------------------------
def embbag_fwd(tables, indices, offsets, B):
    """pooled[b, t, :] = sum over the lookups j of bag (t, b) of tables[t, indices[j], :].

    tables float32 [T, N, D]; indices int [L]; offsets int [T*B+1] (CSR, bag id = t*B + b).
    Sum pooling, a row that occurs twice in a bag counts twice.  Returns float32 [B, T, D].
    """
    T, N, D = tables.shape
    pooled = np.zeros((B, T, D), dtype=F64)
    for t in range(T):
        for b in range(B):
            lo, hi = int(offsets[t * B + b]), int(offsets[t * B + b + 1])
            acc = np.zeros(D, dtype=F64)
            for j in range(lo, hi):
                acc += tables[t, int(indices[j])].astype(F64)
            pooled[b, t] = acc
    return pooled.astype(F32)


# --------------------------------------------------------------------------------------
# MLP forward: bottom MLP, concat interaction, top MLP, sigmoid + BCE  (Section 3.1, Fig. 1)
# --------------------------------------------------------------------------------------
def mlp_fwd(layers, n_bottom, dense, pooled, labels, bf16=False):
    """Forward pass of one replica on one batch.

    layers: list of (W [out,in], b [out]) float32, the n_bottom bottom layers first.
    dense [B, in0]; pooled [B, T, D]; labels [B] in {0,1}.
    Every bottom layer and every top layer but the last is Linear+ReLU; the last
    top layer is linear and gives the logit z.  The interaction is the
    concatenation [bottom_out | pooled_0 | ... | pooled_{T-1}].
    Returns a dict with the saved inputs of every layer (float64), concat,
    logit, prob, and the mean binary cross-entropy loss.
    """
    B = dense.shape[0]
    x = np.asarray(dense, dtype=F64)
    inputs, pre = [], []
    for l in range(n_bottom):
        W, b = layers[l]
        inputs.append(x)
        z = _operand(x, bf16) @ _operand(W, bf16).T + b.astype(F64)
        pre.append(z)
        x = np.maximum(z, 0.0)
    concat = np.concatenate([x, np.asarray(pooled, dtype=F64).reshape(B, -1)], axis=1)
    x = concat
    n_layers = len(layers)
    for l in range(n_bottom, n_layers):
        W, b = layers[l]
        inputs.append(x)
        z = _operand(x, bf16) @ _operand(W, bf16).T + b.astype(F64)
        pre.append(z)
        x = np.maximum(z, 0.0) if l < n_layers - 1 else z
    logit = x[:, 0]
    y = np.asarray(labels, dtype=F64)
    per_example = np.maximum(logit, 0.0) - logit * y + np.log1p(np.exp(-np.abs(logit)))
    prob = 1.0 / (1.0 + np.exp(-logit))
    return dict(inputs=inputs, pre=pre, concat=concat, logit=logit, prob=prob,
                loss=float(per_example.mean()))


# --------------------------------------------------------------------------------------
# MLP backward  (Section 3.1 "Trainer": gradients for all parameters; embedding grads go back to the tables)
# --------------------------------------------------------------------------------------
def mlp_bwd(layers, n_bottom, fwd, labels, bf16=False):
    """Gradients of the mean BCE loss.  Returns (grads, grad_pooled).

    grads: list of (dW, db) float64 per layer; grad_pooled [B, T*D] float64 is the
    gradient with respect to the pooled embeddings (columns D.. of the concat).
    In bf16 mode a gradient tensor is rounded to bfloat16 where it enters a matrix
    product (after the ReLU mask), and the bias gradient sums those rounded values.
    """
    n_layers = len(layers)
    B = fwd["logit"].shape[0]
    y = np.asarray(labels, dtype=F64)
    d_out = ((fwd["prob"] - y) / B)[:, None]          # d loss / d logit
    grads = [None] * n_layers
    grad_pooled = None
    D0 = layers[n_bottom - 1][0].shape[0]              # width of the bottom output
    for l in range(n_layers - 1, -1, -1):
        W, _ = layers[l]
        if l < n_layers - 1 and l != n_bottom - 1:
            d_out = d_out * (fwd["pre"][l] > 0.0)      # ReLU of a hidden layer
        if l == n_bottom - 1:
            # d_out currently holds d concat; split it, then apply the bottom output ReLU
            grad_pooled = d_out[:, D0:].copy()
            d_out = d_out[:, :D0] * (fwd["pre"][l] > 0.0)
        g = _operand(d_out, bf16)
        x = _operand(fwd["inputs"][l], bf16)
        dW = g.T @ x
        db = g.sum(axis=0)
        grads[l] = (dW, db)
        if l > 0:
            d_out = g @ _operand(W, bf16)
    return grads, grad_pooled


def adagrad_dense(theta, acc, g, lr, eps):
    """Element-wise Adagrad: acc += g^2; theta -= lr * g / (sqrt(acc) + eps).  Returns float32 (theta, acc)."""
    g = np.asarray(g, dtype=F64)
    a = acc.astype(F64) + g * g
    a32 = a.astype(F32)
    th = theta.astype(F64) - lr * g / (np.sqrt(a32.astype(F64)) + eps)
    return th.astype(F32), a32


# --------------------------------------------------------------------------------------
# embedding backward + row-wise Adagrad  (Section 3.2 "Embedding Tables": optimizer state lives with the rows)
# --------------------------------------------------------------------------------------
def sort_unique(indices, offsets, T, N, B):
    """Stable sort of all lookups by key = t*N + row.

    Returns (uniq_keys [U], seg_off [U+1], perm [L]): perm lists lookup positions in
    ascending key order, equal keys in ascending position; segment u is
    perm[seg_off[u]:seg_off[u+1]] and all its lookups hit row uniq_keys[u].
    """
    L = int(offsets[T * B])
    lens = np.diff(np.asarray(offsets, dtype=np.int64))
    table_of = np.repeat(np.arange(T * B, dtype=np.int64) // B, lens)
    keys = table_of * N + np.asarray(indices[:L], dtype=np.int64)
    perm = np.argsort(keys, kind="stable")
    sk = keys[perm]
    head = np.ones(L, dtype=bool)
    head[1:] = sk[1:] != sk[:-1]
    starts = np.flatnonzero(head)
    return sk[starts].astype(np.int64), np.append(starts, L).astype(np.int64), perm.astype(np.int64)


def embbag_bwd_adagrad(tables, row_state, indices, offsets, B, grad_pooled, lr, eps):
    """Gradient of the pooled outputs scattered back to the rows, then row-wise Adagrad, in place.

    For every distinct (table, row) u hit by the batch:
        g_u = sum over its lookups, in ascending position, of grad_pooled[b(lookup), t, :]
        s_u += mean_d(g_u[d]^2);   row_u -= lr * g_u / (sqrt(s_u) + eps)
    tables float32 [T,N,D] and row_state float32 [T,N] are updated in place.
    Returns (uniq_keys, seg_off, perm) of sort_unique().
    """
    T, N, D = tables.shape
    gp = np.asarray(grad_pooled, dtype=F64).reshape(B, T, D)
    uniq, seg, perm = sort_unique(indices, offsets, T, N, B)
    lens = np.diff(np.asarray(offsets, dtype=np.int64))
    bag_of = np.repeat(np.arange(T * B, dtype=np.int64), lens)
    for u in range(len(uniq)):
        t, row = divmod(int(uniq[u]), N)
        g = np.zeros(D, dtype=F64)
        for p in perm[seg[u]:seg[u + 1]]:
            g += gp[int(bag_of[p]) - t * B, t]
        s = F32(F64(row_state[t, row]) + np.mean(g * g))
        row_state[t, row] = s
        tables[t, row] = (tables[t, row].astype(F64) - lr * g / (np.sqrt(F64(s)) + eps)).astype(F32)
    return uniq, seg, perm


# --------------------------------------------------------------------------------------
# synchronisation rules  (Algorithms 2, 3, 4)
# --------------------------------------------------------------------------------------
def sync_easgd(ws, center, alpha, literal=False):
    """Shadow EASGD (Algorithm 2), the R trainers visiting the sync PS in turn, in place.

    For r = 0..R-1:  d = alpha * (w_r - c);  w_r -= d;  c += d      (both lines from the old values)
    literal=True takes Algorithm 2's two lines in sequence instead: the replica
    interpolates toward the already-updated centre.
    """
    c = center.astype(F64)
    for w in ws:
        w64 = w.astype(F64)
        c_new = (1.0 - alpha) * c + alpha * w64
        w_new = (1.0 - alpha) * w64 + alpha * (c_new if literal else c)
        w[...] = w_new.astype(F32)
        c = c_new.astype(F32).astype(F64)      # the centre is stored in float32 between visits
    center[...] = c.astype(F32)


def sync_ma(ws, alpha, global_out=None):
    """Shadow MA (Algorithm 3): m = mean_r w_r;  w_r <- (1-alpha) w_r + alpha m, in place."""
    m = np.mean(np.stack([w.astype(F64) for w in ws]), axis=0)
    if global_out is not None:
        global_out[...] = m.astype(F32)
    for w in ws:
        w[...] = ((1.0 - alpha) * w.astype(F64) + alpha * m).astype(F32)


def sync_bmuf(ws, g, delta, alpha, eta, mu=0.0, nesterov=False):
    """Shadow BMUF (Algorithm 4) with classical block momentum, in place.

    m = mean_r w_r;  desc = m - g;  delta <- mu*delta + eta*desc;  g <- g + delta;
    w_r <- (1-alpha) w_r + alpha g.   mu = 0 is Algorithm 4 as printed.
    nesterov=True (the acceleration Algorithm 4's comment mentions): the replicas interpolate toward
    the look-ahead point g + mu*delta instead of g.
    """
    m = np.mean(np.stack([w.astype(F64) for w in ws]), axis=0)
    d = mu * delta.astype(F64) + eta * (m - g.astype(F64))
    delta[...] = d.astype(F32)
    g_new = (g.astype(F64) + delta.astype(F64)).astype(F32)
    g[...] = g_new
    target = g_new.astype(F64) + (mu * delta.astype(F64) if nesterov else 0.0)
    for w in ws:
        w[...] = ((1.0 - alpha) * w.astype(F64) + alpha * target).astype(F32)


# --------------------------------------------------------------------------------------
# metrics  (Section 4, "Evaluation Metrics")
# --------------------------------------------------------------------------------------
def normalized_entropy(prob, labels):
    """NE = mean cross entropy of the predictions / entropy of the empirical CTR."""
    p_hat = np.asarray(prob, dtype=F64)
    y = np.asarray(labels, dtype=F64)
    ce = -np.mean(y * np.log(p_hat) + (1.0 - y) * np.log(1.0 - p_hat))
    p = y.mean()
    return float(ce / -(p * np.log(p) + (1.0 - p) * np.log(1.0 - p)))


def avg_sync_gap(iterations_per_sec, syncs_per_sec):
    """Average number of training iterations of a trainer between two of its syncs (Section 4.1.1)."""
    return iterations_per_sec / syncs_per_sec


# --------------------------------------------------------------------------------------
# one replica step and the deterministic schedule  (Algorithm 1)
# --------------------------------------------------------------------------------------
def replica_step(tables, row_state, layers, accs, n_bottom, batch, lr, eps, bf16=False):
    """One worker iteration of Algorithm 1: update h (tables) and the local w, in place.

    layers / accs: lists of (W, b) float32 parameters and their Adagrad accumulators.
    batch: object with indices, offsets, dense, labels.  Returns the forward dict
    (with 'pooled', 'grad_pooled', 'grads' and the sort outputs added).
    """
    B = batch.dense.shape[0]
    pooled = embbag_fwd(tables, batch.indices, batch.offsets, B)
    fwd = mlp_fwd(layers, n_bottom, batch.dense, pooled, batch.labels, bf16)
    grads, grad_pooled = mlp_bwd(layers, n_bottom, fwd, batch.labels, bf16)
    for l, ((W, b), (aW, ab), (dW, db)) in enumerate(zip(layers, accs, grads)):
        W[...], aW[...] = adagrad_dense(W, aW, dW, lr, eps)
        b[...], ab[...] = adagrad_dense(b, ab, db, lr, eps)
    gp32 = grad_pooled.astype(F32)
    uniq, seg, perm = embbag_bwd_adagrad(tables, row_state, batch.indices, batch.offsets, B, gp32, lr, eps)
    fwd.update(pooled=pooled, grad_pooled=gp32, grads=grads, uniq_keys=uniq, seg_off=seg, perm=perm)
    return fwd


def flatten(layers):
    return np.concatenate([np.concatenate([W.ravel(), b.ravel()]) for W, b in layers])


def unflatten_into(layers, flat):
    o = 0
    for W, b in layers:
        W[...] = flat[o:o + W.size].reshape(W.shape); o += W.size
        b[...] = flat[o:o + b.size]; o += b.size


def train_run(tables, replicas, n_bottom, batches, lr, eps, sync, sync_every, alpha,
              eta=1.0, mu=0.0, bf16=False):
    """Deterministic schedule of Algorithm 1 on one device.

    For step t = 1..S: replicas r = 0..R-1 in turn run replica_step on batches[r][t-1]
    against the current shared tables; after step t, if t % sync_every == 0, one
    synchronisation pass over all replicas (sync in {"easgd","ma","bmuf",None}).
    replicas: list of layer lists (each replica's own float32 copies of w0).
    The centre / global copy starts at w0 (replica 0's initial value), BMUF's delta at 0.
    Returns (losses [S][R], tables, replicas, centre).
    """
    T, N, D = tables.shape
    R = len(replicas)
    row_state = np.zeros((T, N), dtype=F32)
    accs = [[(np.zeros_like(W), np.zeros_like(b)) for W, b in rep] for rep in replicas]
    center = flatten(replicas[0]).copy()
    delta = np.zeros_like(center)
    losses = []
    S = len(batches[0])
    for t in range(1, S + 1):
        row = []
        for r in range(R):
            out = replica_step(tables, row_state, replicas[r], accs[r], n_bottom, batches[r][t - 1], lr, eps, bf16)
            row.append(out["loss"])
        losses.append(row)
        if sync and sync_every and t % sync_every == 0:
            flats = [flatten(rep) for rep in replicas]
            if sync == "easgd":
                sync_easgd(flats, center, alpha)
            elif sync == "ma":
                sync_ma(flats, alpha, center)
            elif sync == "bmuf":
                sync_bmuf(flats, center, delta, alpha, eta, mu)
            for rep, f in zip(replicas, flats):
                unflatten_into(rep, f)
    return losses, row_state, center
