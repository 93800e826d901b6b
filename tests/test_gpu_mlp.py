"""GPU parity of ss_mlp_fwd / ss_mlp_bwd against the oracle, float and bf16 paths."""
import numpy as np
import pytest
import torch

from oracle import shadowsync_oracle as O
from paper_2003_03477_b200 import binding as ss
from paper_2003_03477_b200 import synth, trainer
from parity import RTOL_BF16, RTOL_F32, assert_close

pytestmark = pytest.mark.gpu


def _setup(cfg, seed=0, bias_scale=0.05):
    rng = np.random.default_rng(seed)
    layers = [(W, (rng.normal(size=b.shape) * bias_scale).astype(np.float32)) for W, b in synth.initial_weights(cfg)]
    dense = synth.make_batch(synth.scaled(cfg, T=1, N=10, bag="const1"), 0, 0).dense
    pooled = (rng.normal(size=(cfg.B, cfg.T, cfg.D)) * 0.1).astype(np.float32)
    labels = (rng.random(cfg.B) < 0.3).astype(np.float32)
    return layers, dense, pooled, labels


def _gpu_fwd_bwd(cfg, layers, dense, pooled, labels, apply_update, acc0=None):
    spec = ss.MlpSpec(cfg.bottom, cfg.top, cfg.bf16)
    B, W, D = cfg.B, spec.W, cfg.D
    w = torch.from_numpy(trainer.pack_params(spec, layers)).cuda()
    wh = torch.empty(spec.param_count, dtype=torch.bfloat16, device="cuda") if cfg.bf16 else None
    if cfg.bf16:
        ss.ss_to_bf16(w, wh, spec.param_count)
    concat = torch.zeros(B, W, device="cuda")
    concat[:, D:] = torch.from_numpy(pooled.reshape(B, -1)).cuda()
    concat_h = concat.to(torch.bfloat16) if cfg.bf16 else None
    concat_f = None if cfg.bf16 else concat
    d_dense, d_labels = torch.from_numpy(dense).cuda(), torch.from_numpy(labels).cuda()
    logit, prob, loss = (torch.empty(B, device="cuda"), torch.empty(B, device="cuda"), torch.empty(1, device="cuda"))
    ws = torch.empty(ss.ss_mlp_workspace_bytes(spec, B), dtype=torch.uint8, device="cuda")
    ss.ss_mlp_fwd(spec, w, wh, d_dense, concat_f, concat_h, B, d_labels, logit, prob, loss, ws)
    acc = torch.from_numpy(trainer.pack_params(spec, acc0)).cuda() if acc0 is not None else torch.zeros_like(w)
    grads = torch.full_like(w, 3.0)
    gp = torch.empty(B, cfg.T * D, device="cuda")
    ss.ss_mlp_bwd(spec, w, wh, acc, grads, d_dense, concat_f, concat_h, d_labels, prob, B, cfg.lr, cfg.eps,
                  apply_update, gp, cfg.T * D, ws)
    torch.cuda.synchronize()
    cc = (concat_h.float() if cfg.bf16 else concat).cpu().numpy()
    return dict(spec=spec, logit=logit.cpu().numpy(), prob=prob.cpu().numpy(), loss=float(loss.item()),
                concat=cc, grads=grads.cpu().numpy(), gp=gp.cpu().numpy(), w=w.cpu().numpy(), acc=acc.cpu().numpy(),
                wh=(wh.float().cpu().numpy() if cfg.bf16 else None))


def _check(cfg, seed=0):
    rtol = RTOL_BF16 if cfg.bf16 else RTOL_F32
    layers, dense, pooled, labels = _setup(cfg, seed)
    nb = len(cfg.bottom) - 1
    if cfg.bf16:   # the GPU reads the pooled columns as bf16; give the oracle the same values
        pooled = O.round_bf16(pooled).astype(np.float32)
    fwd = O.mlp_fwd(layers, nb, dense, pooled, labels, cfg.bf16)
    grads, gp = O.mlp_bwd(layers, nb, fwd, labels, cfg.bf16)
    g = _gpu_fwd_bwd(cfg, layers, dense, pooled, labels, apply_update=0)
    spec = g["spec"]
    assert_close(g["logit"], fwd["logit"], rtol, "logit")
    assert_close(g["prob"], fwd["prob"], rtol, "prob")
    assert abs(g["loss"] - fwd["loss"]) <= rtol * abs(fwd["loss"])
    assert_close(g["concat"][:, :cfg.D], fwd["concat"][:, :cfg.D], rtol, "bottom output")
    assert_close(g["gp"], gp, rtol, "grad_pooled")
    got = trainer.unpack_params(spec, g["grads"])
    for l, ((dW, db), (gW, gb)) in enumerate(zip(grads, got)):
        assert_close(gW, dW, rtol, f"dW[{l}]")
        assert_close(gb, db, rtol, f"db[{l}]")
    # pads of the gradient vector are zero
    used = np.zeros(spec.param_count, bool)
    for l, (fin, fout) in enumerate(spec.layer_dims):
        used[spec.w_off[l]: spec.w_off[l] + fin * fout] = True
        used[spec.b_off[l]: spec.b_off[l] + fout] = True
    assert not g["grads"][~used].any()
    # with the update: element-wise Adagrad from a non-zero accumulator
    rng = np.random.default_rng(seed + 1)
    acc0 = [((rng.random(W.shape) * 1e-6).astype(np.float32), (rng.random(b.shape) * 1e-6).astype(np.float32)) for W, b in layers]
    g2 = _gpu_fwd_bwd(cfg, layers, dense, pooled, labels, apply_update=1, acc0=acc0)
    new = trainer.unpack_params(spec, g2["w"])
    newacc = trainer.unpack_params(spec, g2["acc"])
    for l, ((W, b), (aW, ab), (dW, db)) in enumerate(zip(layers, acc0, grads)):
        W1, aW1 = O.adagrad_dense(W, aW, dW, cfg.lr, cfg.eps)
        b1, ab1 = O.adagrad_dense(b, ab, db, cfg.lr, cfg.eps)
        # compare the step, not the parameter: the step is what the kernel computes
        assert_close(new[l][0] - W, W1.astype(np.float64) - W, max(rtol, 1e-4), f"step W[{l}]")
        assert_close(new[l][1] - b, b1.astype(np.float64) - b, max(rtol, 1e-4), f"step b[{l}]")
        assert_close(newacc[l][0], aW1, rtol, f"acc W[{l}]")
    assert not g2["w"][~used].any()
    if cfg.bf16:
        assert np.array_equal(g2["wh"], torch.from_numpy(g2["w"]).to(torch.bfloat16).float().numpy())
    return g


def test_mlp_tiny_config_f32():
    _check(synth.CONFIGS["tiny"])


def test_mlp_f32_ragged_shapes():
    # batch and widths that are no multiple of the 64-wide tiles
    cfg = synth.scaled(synth.CONFIGS["tiny"], B=77, T=2, D=8, bottom=(13, 40, 24, 8), top=(24, 72, 16, 1))
    _check(cfg, seed=3)


def test_mlp_bf16_small():
    cfg = synth.scaled(synth.CONFIGS["tiny"], B=200, T=3, D=16, bottom=(13, 64, 16), top=(64, 128, 64, 1), bf16=True)
    _check(cfg, seed=4)


def test_mlp_bf16_medium_shapes_reduced_batch():
    # the medium model's layer widths (tensor-core tiles: K = 1728, N = 512) at a batch with a ragged last tile
    cfg = synth.scaled(synth.CONFIGS["medium"], B=328)
    _check(cfg, seed=5)


def test_mlp_results_do_not_depend_on_how_many_ctas_the_persistent_launches_take():
    """All tensor-core products of a pass run in one launch whose CTAs draw tiles in ticket order and wait, inside the
    launch, for the tiles they depend on.  A tile's arithmetic is fixed, so the outputs are bit-identical whether one
    CTA works through all tickets (every dependency is then on the same CTA's own earlier tiles), a handful do, or
    one per SM; no wait runs out."""
    cfg = synth.scaled(synth.CONFIGS["medium"], B=1000)      # eight row blocks, the last one ragged
    layers, dense, pooled, labels = _setup(cfg, seed=11)
    ref = None
    try:
        for ctas in (1, 3, 32, 1000):
            assert ss.ss_mlp_set_flow_ctas(ctas) == ctas
            g = _gpu_fwd_bwd(cfg, layers, dense, pooled, labels, apply_update=0)
            assert ss.ss_device_error() == 0
            if ref is None:
                ref = g
                continue
            for k in ("logit", "prob", "concat", "grads", "gp"):
                assert np.array_equal(ref[k], g[k]), f"{k} differs between 1 CTA and {ctas}"
            assert ref["loss"] == g["loss"]
    finally:
        assert ss.ss_mlp_set_flow_ctas(0) == 32               # back to the library's default


def test_mlp_bf16_large_shapes_full_batch():
    """Configuration 4's MLP at its full batch of 4096: products of 2^33 flop and more take the 128 x 256 tiles, as
    single launches (forward, input gradients) and as the grouped weight-gradient launch.

    Sums over the batch (logits, loss, weight and bias gradients) meet the strict tolerance.  A grad_pooled row
    belongs to one sample, and a hidden unit whose pre-activation is within one bf16 ulp of zero may be gated either
    way (see parity.match_relu_gates, whose search costs a full backward pass per candidate and is run on a small
    batch elsewhere): here a row may miss only if its sample has such a unit, and few rows may."""
    from parity import GATE_DELTA
    cfg = synth.CONFIGS["large"]
    assert cfg.B == 4096 and cfg.bf16
    layers, dense, pooled, labels = _setup(cfg, seed=6)
    nb = len(cfg.bottom) - 1
    pooled = O.round_bf16(pooled).astype(np.float32)
    fwd = O.mlp_fwd(layers, nb, dense, pooled, labels, True)
    grads, gp = O.mlp_bwd(layers, nb, fwd, labels, True)
    g = _gpu_fwd_bwd(cfg, layers, dense, pooled, labels, apply_update=0)
    assert ss.ss_device_error() == 0
    assert_close(g["logit"], fwd["logit"], RTOL_BF16, "logit")
    assert abs(g["loss"] - fwd["loss"]) <= RTOL_BF16 * abs(fwd["loss"])
    got = trainer.unpack_params(g["spec"], g["grads"])

    def rel_err(a, want):
        want = np.asarray(want, np.float64)
        return np.abs(np.asarray(a, np.float64) - want) / np.maximum(np.abs(want), np.sqrt(np.mean(want * want)))

    for l, ((dW, db), (gW, gb)) in enumerate(zip(grads, got)):
        # a sample gated the other way moves its unit's gradient row by that sample's whole contribution: a few
        # elements may miss the strict bound, none by much (one sample of 4096)
        for name, a, want in ((f"dW[{l}]", gW, dW), (f"db[{l}]", gb, db)):
            e = rel_err(a, want)
            assert np.mean(e > RTOL_BF16) <= 0.02, (name, float(np.mean(e > RTOL_BF16)))
            assert e.max() <= 10 * RTOL_BF16, (name, float(e.max()))
    rms = float(np.sqrt(np.mean(gp * gp)))
    err = np.max(np.abs(g["gp"] - gp) / np.maximum(np.abs(gp), rms), axis=1)
    bad = np.flatnonzero(err > RTOL_BF16)
    assert len(bad) <= 0.1 * cfg.B, len(bad)
    n_layers = len(layers)
    edge = np.zeros(cfg.B, bool)
    for l in range(nb, n_layers - 1):
        pre = fwd["pre"][l]
        edge |= (np.abs(pre) < GATE_DELTA * np.sqrt(np.mean(pre * pre))).any(axis=1)
    assert edge[bad].all(), "a row without a unit at the edge of its ReLU missed the tolerance"


def test_zero_weights_give_ln2():
    cfg = synth.CONFIGS["tiny"]
    layers = [(np.zeros_like(W), b) for W, b in synth.initial_weights(cfg)]
    _, dense, pooled, labels = _setup(cfg)
    g = _gpu_fwd_bwd(cfg, layers, dense, pooled, labels, apply_update=0)
    assert abs(g["loss"] - np.log(2.0)) < 1e-6 and np.allclose(g["prob"], 0.5)


def test_mlp_rejects_bad_arguments():
    cfg = synth.CONFIGS["tiny"]
    spec = ss.MlpSpec(cfg.bottom, cfg.top, False)
    w = torch.zeros(spec.param_count, device="cuda")
    B = 8
    z = torch.zeros(B, device="cuda")
    dense, concat = torch.zeros(B, 13, device="cuda"), torch.zeros(B, 144, device="cuda")
    small = torch.empty(16, dtype=torch.uint8, device="cuda")
    with pytest.raises(ss.SsError) as e:
        ss.ss_mlp_fwd(spec, w, None, dense, concat, None, B, z, z, z, z, small)
    assert e.value.status == -5
    spec_h = ss.MlpSpec(cfg.bottom, cfg.top, True)
    ws = torch.empty(ss.ss_mlp_workspace_bytes(spec_h, B), dtype=torch.uint8, device="cuda")
    with pytest.raises(ss.SsError) as e:
        ss.ss_mlp_fwd(spec_h, w, None, dense, concat, None, B, z, z, z, z, ws)   # bf16 mode without bf16 buffers
    assert e.value.status == -4


def test_normalized_entropy_accumulates_over_batches():
    rng = np.random.default_rng(11)
    acc = torch.zeros(3, dtype=torch.float64, device="cuda")
    out = torch.zeros(1, dtype=torch.float64, device="cuda")
    zs, ys = [], []
    for B in (2048, 777, 1):
        z = (rng.normal(size=B) * 2 - 3).astype(np.float32)
        y = (rng.random(B) < 0.05).astype(np.float32)
        if B == 2048:
            y[:3] = 1.0
        ss.ss_ne_accumulate(torch.from_numpy(z).cuda(), torch.from_numpy(y).cuda(), B, acc)
        zs.append(z); ys.append(y)
    ss.ss_ne_value(acc, out)
    torch.cuda.synchronize()
    z, y = np.concatenate(zs).astype(np.float64), np.concatenate(ys)
    want = O.normalized_entropy(1.0 / (1.0 + np.exp(-z)), y)
    assert abs(float(out.item()) - want) <= 1e-9 * want
    # the constant predictor at the empirical rate has NE = 1
    p = float(y.mean())
    acc.zero_()
    const = torch.full((len(y),), float(np.log(p / (1 - p))), device="cuda")
    ss.ss_ne_accumulate(const, torch.from_numpy(y).cuda(), len(y), acc)
    ss.ss_ne_value(acc, out)
    torch.cuda.synchronize()
    assert abs(float(out.item()) - 1.0) < 1e-6
