"""End-to-end parity: whole replica steps and the deterministic schedule of Algorithm 1 against the oracle."""
import numpy as np
import pytest
import torch

from oracle import shadowsync_oracle as O
from paper_2003_03477_b200 import binding as ss
from paper_2003_03477_b200 import synth, trainer
from parity import RTOL_BF16, RTOL_F32, RTOL_SYNC, assert_close, oracle_step_following_gates

pytestmark = pytest.mark.gpu


def _model(cfg, tables, layers, max_L, keep=True):
    spec = ss.MlpSpec(cfg.bottom, cfg.top, cfg.bf16)
    w0 = torch.from_numpy(trainer.pack_params(spec, layers)).cuda()
    return trainer.Model(cfg.T, cfg.N, cfg.D, cfg.B, cfg.bottom, cfg.top, cfg.bf16, cfg.R, w0,
                         torch.from_numpy(tables.copy()).cuda(), cfg.lr, cfg.eps, max_L=max_L,
                         keep_sort_outputs=keep, keep_f32_concat=True)


def _dev_batch(b):
    return trainer.DeviceBatch(b.indices, b.offsets, b.dense, b.labels)


def _teacher_forced_steps(cfg, n_steps, rtol, acc0=0.0, step_rtol=None):
    """Every GPU step starts from the oracle's state, so per-step errors do not compound.

    acc0: initial value of the dense Adagrad accumulators.  From zero the first step is lr*g/(|g|+eps),
    a sign function of g: an entry whose gradient is within rounding of zero may step either way.  A
    positive start (both sides load the same state) keeps the step a smooth function of the gradient.
    step_rtol: tolerance of the parameter and table-row steps (default: the looser of rtol and 2e-4, which the
    zero start needs)."""
    step_rtol = max(rtol, 2e-4) if step_rtol is None else step_rtol
    tables = synth.tables_dense(cfg)
    layers = synth.initial_weights(cfg)
    nb = len(cfg.bottom) - 1
    batches = [synth.make_batch(cfg, 0, t) for t in range(n_steps)]
    m = _model(synth.scaled(cfg, R=1), tables, layers, max(b.L for b in batches))
    spec, rep = m.spec, m.replicas[0]
    row_state = np.zeros((cfg.T, cfg.N), np.float32)
    accs = [(np.full_like(W, acc0), np.full_like(b, acc0)) for W, b in layers]
    for t, b in enumerate(batches):
        # load the oracle's current state into the device buffers
        m.tables.copy_(torch.from_numpy(tables))
        m.row_state.copy_(torch.from_numpy(row_state.reshape(-1)))
        rep.w.copy_(torch.from_numpy(trainer.pack_params(spec, layers)))
        rep.acc.copy_(torch.from_numpy(trainer.pack_params(spec, accs)))
        if cfg.bf16:
            ss.ss_to_bf16(rep.w, rep.w_bf16, spec.param_count)
        t_before, w_before = tables.copy(), [(W.copy(), bb.copy()) for W, bb in layers]
        m.step(0, _dev_batch(b))
        torch.cuda.synchronize()
        assert m.status() == 0
        if cfg.bf16:
            # hidden units within rounding of zero: the oracle takes the gate the kernels took
            out, flips = oracle_step_following_gates(O, tables, row_state, layers, accs, nb, b, cfg.lr, cfg.eps, True,
                                                     rep.grad_pooled.cpu().numpy(), rtol)
            hidden_units = cfg.B * (sum(cfg.bottom[1:]) + sum(cfg.top[1:-1]))
            assert len(flips) <= max(2, 1e-4 * hidden_units), (len(flips), hidden_units)
            note = f" (step {t}: {len(flips)} top-MLP gates at the edge followed the kernel: {flips})"
        else:
            out = O.replica_step(tables, row_state, layers, accs, nb, b, cfg.lr, cfg.eps, False)
            note = ""
        U = int(rep.num_unique.item())
        assert U == len(out["uniq_keys"])
        assert np.array_equal(rep.uniq_keys.cpu().numpy()[:U], out["uniq_keys"])
        assert np.array_equal(rep.seg_off.cpu().numpy()[:U + 1], out["seg_off"])
        assert np.array_equal(rep.perm.cpu().numpy()[:b.L], out["perm"])
        assert_close(rep.concat_f32.cpu().numpy()[:, cfg.D:], out["pooled"].reshape(cfg.B, -1), RTOL_F32, "pooled")
        assert_close(rep.logit.cpu().numpy(), out["logit"], rtol, "logit")
        assert abs(float(rep.loss.item()) - out["loss"]) <= rtol * abs(out["loss"])
        assert_close(rep.grad_pooled.cpu().numpy(), out["grad_pooled"], rtol, "grad_pooled" + note)
        new = trainer.unpack_params(spec, rep.w.cpu().numpy())
        for l in range(len(layers)):
            # the updated parameters themselves, then the step they took (new - old, which is what the kernel computes).
            # A step is only known to one rounding of the float parameter it is read from: two float ulps of |w| are
            # allowed on top of the relative tolerance (for a weight of 0.3 that moved by 2e-3, one ulp is 1.3e-5 of the step)
            assert_close(new[l][0], layers[l][0], rtol, f"step {t} W[{l}]" + note)
            got_s = new[l][0].astype(np.float64) - w_before[l][0]
            want_s = layers[l][0].astype(np.float64) - w_before[l][0]
            ulps = 2.0 * 2.0 ** -24 * np.abs(layers[l][0].astype(np.float64))
            rms = float(np.sqrt(np.mean(want_s ** 2)))
            bad = np.abs(got_s - want_s) > step_rtol * np.maximum(np.abs(want_s), rms) + ulps
            assert not bad.any(), f"step {t} dW[{l}]: {int(bad.sum())}/{bad.size} beyond rtol={step_rtol}" + note
        # touched rows against the scale of the touched rows' steps; every other row bit-identical
        keys = out["uniq_keys"]
        got_t = m.tables.cpu().numpy().reshape(-1, cfg.D)
        before = t_before.reshape(-1, cfg.D)
        assert_close(got_t[keys] - before[keys], tables.reshape(-1, cfg.D)[keys].astype(np.float64) - before[keys],
                     max(step_rtol, 2e-5), f"step {t} table rows")
        untouched = np.ones(cfg.T * cfg.N, bool)
        untouched[keys] = False
        assert np.array_equal(got_t[untouched], before[untouched])
        assert_close(m.row_state.cpu().numpy().reshape(cfg.T, cfg.N), row_state, max(rtol, 2e-5), "row state")


def test_tiny_config_steps_teacher_forced():
    _teacher_forced_steps(synth.CONFIGS["tiny"], 4, RTOL_F32)


def test_tiny_config_steps_teacher_forced_at_the_float_tolerance():
    """The float path at the tolerance the float outputs are held to (1e-5; 2e-5 for table rows, whose gradient is a
    sum of up to hundreds of float terms): with accumulators that start positive the Adagrad step is a smooth
    function of the gradient, so no entry depends on the sign of a gradient that is zero up to rounding."""
    _teacher_forced_steps(synth.CONFIGS["tiny"], 4, RTOL_F32, acc0=1e-4, step_rtol=RTOL_F32)


def test_bf16_model_steps_teacher_forced():
    cfg = synth.scaled(synth.CONFIGS["medium"], T=4, N=5000, B=256, bottom=(13, 128, 64), top=(320, 128, 64, 1))
    _teacher_forced_steps(cfg, 2, RTOL_BF16)


def _run_tiny_schedule():
    cfg = synth.CONFIGS["tiny"]
    tables = synth.tables_dense(cfg)
    layers = synth.initial_weights(cfg)
    batches = [[synth.make_batch(cfg, r, t) for t in range(cfg.steps)] for r in range(cfg.R)]
    m = _model(cfg, tables, layers, max(b.L for bs in batches for b in bs), keep=False)
    dev = [[_dev_batch(b) for b in bs] for bs in batches]
    losses = []
    main = torch.cuda.current_stream()
    for t in range(1, cfg.steps + 1):
        for r in range(cfg.R):          # replicas in turn on one stream: the deterministic schedule
            m.step(r, dev[r][t - 1], stream=main)
            losses.append(m.replicas[r].loss.clone())
        if t % cfg.sync_every == 0:
            m.sync("easgd", cfg.alpha, stream=main)
    torch.cuda.synchronize()
    assert m.status() == 0
    return cfg, m, batches, tables, layers, torch.cat(losses).cpu().numpy().reshape(cfg.steps, cfg.R)


def test_tiny_config_full_schedule_against_oracle_and_bitwise_reproducible():
    cfg, m, batches, tables, layers, losses = _run_tiny_schedule()
    reps = [[(W.copy(), b.copy()) for W, b in layers] for _ in range(cfg.R)]
    t_o = tables.copy()
    l_o, row_state, centre = O.train_run(t_o, reps, len(cfg.bottom) - 1, batches, cfg.lr, cfg.eps, "easgd",
                                         cfg.sync_every, cfg.alpha)
    # the loss path is followed closely over all 20 steps x 2 replicas and 4 sync passes
    np.testing.assert_allclose(losses, np.array(l_o), rtol=2e-4)
    # early Adagrad steps are lr*g/(|g|+eps): a gradient within rounding of zero may take either sign, so a
    # handful of parameters can sit one step apart; everything else agrees closely
    spec = m.spec
    for r in range(cfg.R):
        got = np.concatenate([np.concatenate([W.ravel(), b]) for W, b in trainer.unpack_params(spec, m.replicas[r].w.cpu().numpy())])
        want = O.flatten(reps[r])
        far = np.abs(got - want) > 1e-3 * np.maximum(np.abs(want), np.sqrt(np.mean(want ** 2)))
        assert far.mean() < 2e-3, far.mean()
    tg = m.tables.cpu().numpy()
    far = np.abs(tg - t_o) > 1e-3 * 0.03
    assert far.mean() < 2e-3
    # first steps' losses are tight (no compounding yet)
    np.testing.assert_allclose(losses[0], np.array(l_o)[0], rtol=RTOL_F32)
    # deterministic mode is bitwise reproducible
    _, m2, *_rest, losses2 = _run_tiny_schedule()
    assert np.array_equal(losses, losses2)
    assert torch.equal(m.tables, m2.tables) and all(torch.equal(a.w, b.w) for a, b in zip(m.replicas, m2.replicas))
    assert torch.equal(m.center, m2.center)
    # loss heads toward the entropy of the label rate: H(0.03) = 0.1347 nats, from ln 2 at the start
    assert losses[0].mean() > 0.5 and losses[-1].mean() < 0.3


def test_shadow_loop_free_running_keeps_invariants():
    # background sync on the low-priority stream while the replicas train on their own streams: any
    # interleaving is legal (lock-free by design), so only invariants are checked
    cfg = synth.scaled(synth.CONFIGS["tiny"], steps=30)
    tables = synth.tables_dense(cfg)
    layers = synth.initial_weights(cfg)
    batches = [[_dev_batch(synth.make_batch(cfg, r, t)) for t in range(8)] for r in range(cfg.R)]
    m = _model(cfg, tables, layers, max(b.L for bs in batches for b in bs), keep=False)
    loop = trainer.ShadowLoop(m, "easgd", cfg.alpha, max_rounds=10_000).start()
    for t in range(cfg.steps):
        for r in range(cfg.R):
            m.step(r, batches[r][t % 8])
    for rep in m.replicas:
        rep.stream.synchronize()
    rounds = loop.stop()
    torch.cuda.synchronize()
    assert rounds >= 1 and m.status() == 0
    for rep in m.replicas:
        assert torch.isfinite(rep.w).all() and float(rep.loss.item()) < 0.7
    assert torch.isfinite(m.center).all() and torch.isfinite(m.tables).all()
    # elastic averaging keeps the replicas within a small distance of the centre
    assert float((m.replicas[0].w - m.center).abs().max()) < 0.5


def test_shadow_loop_pause_counts_completed_passes_and_resume_continues():
    """A paused shadow thread has no pass in flight: the vectors stay put until it is resumed, and the pass count
    read while paused equals the number of S-EASGD passes the vectors have actually been through."""
    n, R, alpha = 1 << 16, 2, 0.25
    ws = [torch.full((n,), float(r + 1), device="cuda") for r in range(R)]
    c = torch.zeros(n, device="cuda")
    s = torch.cuda.Stream()
    h = ss.ss_shadow_start("easgd", ws, c, None, n, alpha, stream=s, max_in_flight=2, max_rounds=1 << 40)
    import time
    time.sleep(0.02)
    ss.ss_shadow_pause(h, True)
    k = ss.ss_shadow_rounds(h)
    snap = [w.clone() for w in ws] + [c.clone()]
    time.sleep(0.02)
    assert ss.ss_shadow_rounds(h) == k and all(torch.equal(a, b) for a, b in zip(snap, ws + [c]))
    # k passes of Algorithm 2 on the scalars (1, 2 | 0), in the oracle
    w0 = [np.full(1, float(r + 1), np.float32) for r in range(R)]
    c0 = np.zeros(1, np.float32)
    for _ in range(k):
        O.sync_easgd(w0, c0, alpha)
    assert k >= 1
    for r in range(R):
        assert_close(ws[r][:1].cpu().numpy(), w0[r], 1e-5, "replica after k passes", floor=1.0)
    ss.ss_shadow_pause(h, False)
    time.sleep(0.02)
    assert ss.ss_shadow_stop(h) > k


def test_foreground_sync_variants_match_the_oracle_rules():
    # FR-EASGD: each replica interpolates with the centre on its own stream; FR-MA / FR-BMUF: one joint pass
    cfg = synth.scaled(synth.CONFIGS["tiny"], R=3)
    tables = synth.tables_dense(cfg)
    layers = synth.initial_weights(cfg)
    m = _model(cfg, tables, layers, 16, keep=False)
    rng = np.random.default_rng(2)
    n = m.spec.param_count
    for rep in m.replicas:
        rep.w.copy_(torch.from_numpy((rng.normal(size=n) * 0.02).astype(np.float32)))
    m.center.copy_(torch.from_numpy((rng.normal(size=n) * 0.02).astype(np.float32)))
    torch.cuda.synchronize()
    for rule in ("ma", "bmuf", "easgd"):
        ws = [rep.w.cpu().numpy().copy() for rep in m.replicas]
        c, d = m.center.cpu().numpy().copy(), m.delta.cpu().numpy().copy()
        m.foreground_sync(rule, 0.2, eta=0.8, mu=0.5)
        torch.cuda.synchronize()
        if rule == "ma":
            O.sync_ma(ws, 0.2, c)
        elif rule == "bmuf":
            O.sync_bmuf(ws, c, d, 0.2, 0.8, 0.5)
        else:
            # replicas' passes run on different streams: any visiting order is legal; each order is an oracle run
            import itertools
            got = [rep.w.cpu().numpy() for rep in m.replicas] + [m.center.cpu().numpy()]
            ok = False
            for order in itertools.permutations(range(cfg.R)):
                w2, c2 = [w.copy() for w in ws], c.copy()
                for r in order:
                    O.sync_easgd([w2[r]], c2, 0.2)
                if all(np.allclose(a, b, rtol=1e-6, atol=1e-9) for a, b in zip(got, w2 + [c2])):
                    ok = True
                    break
            assert ok, "FR-EASGD result matches no visiting order of the replicas"
            continue
        for rep, w in zip(m.replicas, ws):
            assert_close(rep.w.cpu().numpy(), w, RTOL_SYNC, f"FR-{rule} replica")
        assert_close(m.center.cpu().numpy(), c, RTOL_SYNC, f"FR-{rule} global")


def test_intra_replica_hogwild_workers_share_one_parameter_copy():
    # two workers per trainer, each on its own batches and streams, updating the trainer's single copy of the
    # parameters and optimizer state lock-free: any interleaving is legal, so invariants only
    cfg = synth.scaled(synth.CONFIGS["tiny"], steps=24)
    tables = synth.tables_dense(cfg)
    layers = synth.initial_weights(cfg)
    spec = ss.MlpSpec(cfg.bottom, cfg.top, cfg.bf16)
    w0 = torch.from_numpy(trainer.pack_params(spec, layers)).cuda()
    host = [[[synth.make_batch(cfg, 2 * r + k, t) for t in range(6)] for k in range(2)] for r in range(cfg.R)]
    m = trainer.Model(cfg.T, cfg.N, cfg.D, cfg.B, cfg.bottom, cfg.top, cfg.bf16, cfg.R, w0,
                      torch.from_numpy(tables.copy()).cuda(), cfg.lr, cfg.eps,
                      max_L=max(b.L for a in host for bs in a for b in bs), workers=2)
    dev = [[[_dev_batch(b) for b in bs] for bs in a] for a in host]
    assert m.workers[0][1].w.data_ptr() == m.replicas[0].w.data_ptr()          # shared parameters
    assert m.workers[0][1].logit.data_ptr() != m.replicas[0].logit.data_ptr()  # own activations
    first = None
    for t in range(cfg.steps):
        for r in range(cfg.R):
            for k in range(2):
                m.step(r, dev[r][k][t % 6], worker=k)
        if t == 0:
            torch.cuda.synchronize()
            first = float(m.replicas[0].loss.item())
    torch.cuda.synchronize()
    assert m.status() == 0
    for r in range(cfg.R):
        assert torch.isfinite(m.replicas[r].w).all() and torch.isfinite(m.replicas[r].acc).all()
        for k in range(2):
            assert float(m.workers[r][k].loss.item()) < first      # both workers' losses fell from ln 2
    assert first > 0.5 and torch.isfinite(m.tables).all()


def test_large_model_shapes_reduced_tables_one_step_and_model_averaging():
    # configuration 4's model (dim 128 rows, Poisson(8) bags clamped to 40, Zipf 1.2, 13-1024-512-128 bottom,
    # 3456-1024-1024-512-1 top, bf16 GEMMs) on shorter tables and a smaller batch, then one S-MA pass
    cfg = synth.scaled(synth.CONFIGS["large"], R=2, N=30_000, B=256)
    _teacher_forced_steps(cfg, 1, RTOL_BF16, acc0=1e-4)
    tables = synth.tables_dense(cfg)
    layers = synth.initial_weights(cfg)
    m = _model(cfg, tables, layers, 16, keep=False)
    rng = np.random.default_rng(4)
    n = m.spec.param_count
    for rep in m.replicas:
        rep.w.copy_(torch.from_numpy((rng.normal(size=n) * 0.02).astype(np.float32)))
    ws = [rep.w.cpu().numpy().copy() for rep in m.replicas]
    g = np.zeros(n, np.float32)
    m.sync("ma", cfg.alpha, stream=torch.cuda.current_stream())
    torch.cuda.synchronize()
    O.sync_ma(ws, cfg.alpha, g)
    for rep, w in zip(m.replicas, ws):
        assert_close(rep.w.cpu().numpy(), w, RTOL_SYNC, "S-MA replica")
        assert torch.equal(rep.w_bf16, rep.w.to(torch.bfloat16))      # mirror refreshed by the sync kernel
    assert_close(m.center.cpu().numpy(), g, RTOL_SYNC, "S-MA mean")


def test_bmuf_round_of_local_steps_then_one_pass():
    # configuration 3's schedule at reduced size: every replica takes 10 local steps, then one S-BMUF pass
    # (block momentum 0.9, block learning rate 1); the pass is checked on the state the GPU reached
    cfg = synth.scaled(synth.CONFIGS["medium_bmuf"], R=3, T=4, N=5000, B=128, bottom=(13, 128, 64), top=(320, 128, 64, 1))
    tables = synth.tables_dense(cfg)
    layers = synth.initial_weights(cfg)
    batches = [[synth.make_batch(cfg, r, t) for t in range(cfg.sync_every)] for r in range(cfg.R)]
    m = _model(cfg, tables, layers, max(b.L for bs in batches for b in bs), keep=False)
    main = torch.cuda.current_stream()
    for t in range(cfg.sync_every):
        for r in range(cfg.R):
            m.step(r, _dev_batch(batches[r][t]), stream=main)
    torch.cuda.synchronize()
    assert m.status() == 0
    losses = [float(rep.loss.item()) for rep in m.replicas]
    assert all(np.isfinite(l) and l < 0.69 for l in losses)              # below ln 2 after ten steps
    ws = [rep.w.cpu().numpy().copy() for rep in m.replicas]
    g, d = m.center.cpu().numpy().copy(), m.delta.cpu().numpy().copy()
    assert max(np.abs(ws[0] - ws[1]).max(), np.abs(ws[0] - ws[2]).max()) > 0   # replicas have drifted apart
    m.sync("bmuf", cfg.alpha, cfg.eta, cfg.mu, stream=main)
    torch.cuda.synchronize()
    O.sync_bmuf(ws, g, d, cfg.alpha, cfg.eta, cfg.mu)
    for rep, w in zip(m.replicas, ws):
        assert_close(rep.w.cpu().numpy(), w, RTOL_SYNC, "S-BMUF replica")
    assert_close(m.center.cpu().numpy(), g, RTOL_SYNC, "S-BMUF global")
    # the momentum is a difference of nearly equal weights: its rounding error scales with the weights
    assert_close(m.delta.cpu().numpy(), d, RTOL_SYNC, "S-BMUF momentum", floor=float(np.sqrt(np.mean(g * g))))
