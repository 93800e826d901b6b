"""Parity at the benchmark's full sizes, in the launch configuration the benchmark times (one captured CUDA
graph per replica step, sort forked onto the side stream): the medium workload's whole first step against the
oracle, and the sync kernels on HBM-sized vectors.

The oracle cannot hold 26 tables of a million rows, and does not need to: table rows are a pure function of
(table, row, column), so the batch is remapped onto a compact table of exactly the rows it touches (the remap is
monotone per table, so sort order, permutation and segment structure are unchanged) and the oracle runs the
complete step on that."""
import numpy as np
import pytest
import torch

from oracle import shadowsync_oracle as O
from paper_2003_03477_b200 import binding as ss
from paper_2003_03477_b200 import synth, trainer
from parity import RTOL_BF16, RTOL_F32, RTOL_SYNC, assert_close, oracle_step_following_gates

pytestmark = pytest.mark.gpu


def _compact(cfg, batch):
    lens = np.diff(batch.offsets.astype(np.int64))
    tbl = np.repeat(np.arange(cfg.T * cfg.B) // cfg.B, lens)
    keys = tbl * cfg.N + batch.indices
    uniq, inv = np.unique(keys, return_inverse=True)
    t_of = uniq // cfg.N
    counts = np.bincount(t_of, minlength=cfg.T)
    nmax = int(counts.max())
    starts = np.concatenate([[0], np.cumsum(counts)[:-1]])
    local = np.arange(len(uniq)) - starts[t_of]                  # rank of the row inside its table
    tables = np.zeros((cfg.T, nmax, cfg.D), np.float32)
    for t in range(cfg.T):
        rows = (uniq[t_of == t] % cfg.N)
        tables[t, :len(rows)] = synth.table_rows(cfg, t, rows)
    small = synth.Batch(local[inv].astype(np.int32), batch.offsets, batch.dense, batch.labels)
    return tables, small, uniq, t_of, local, nmax


def test_medium_workload_first_step_full_size_as_benchmarked():
    cfg = synth.scaled(synth.CONFIGS["medium"], R=1)
    batch = synth.make_batch(cfg, 0, 0)
    layers = synth.initial_weights(cfg)
    spec = ss.MlpSpec(cfg.bottom, cfg.top, cfg.bf16)
    w0 = torch.from_numpy(trainer.pack_params(spec, layers)).cuda()
    model = trainer.Model(cfg.T, cfg.N, cfg.D, cfg.B, cfg.bottom, cfg.top, cfg.bf16, 1, w0, trainer.device_tables(cfg),
                          cfg.lr, cfg.eps, max_L=batch.L, keep_sort_outputs=True, keep_f32_concat=True)
    dev = trainer.DeviceBatch(batch.indices, batch.offsets, batch.dense, batch.labels)
    rep = model.replicas[0]
    # first-use set-up happens outside capture, on a scratch copy of the state that is restored afterwards
    w_keep = rep.w.clone()
    model.step(0, dev)
    torch.cuda.synchronize()
    model.tables.copy_(trainer.device_tables(cfg))
    model.row_state.zero_()
    # dense accumulators start positive on both sides: from zero the first Adagrad step is lr*g/(|g|+eps), a
    # sign function of g, and an entry whose gradient is within rounding of zero may step either way
    acc0 = 1e-4
    rep.w.copy_(w_keep); rep.acc.fill_(acc0)
    ss.ss_to_bf16(rep.w, rep.w_bf16, spec.param_count)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=rep.stream):
        model.step(0, dev, stream=rep.stream)
    with torch.cuda.stream(rep.stream):
        g.replay()
    torch.cuda.synchronize()
    assert model.status() == 0 and ss.ss_device_error() == 0

    # ---- oracle on the compact problem
    tables_c, small, uniq, t_of, local, nmax = _compact(cfg, batch)
    t_before = tables_c.copy()
    state = np.zeros((cfg.T, nmax), np.float32)
    accs = [(np.full_like(W, acc0), np.full_like(b, acc0)) for W, b in layers]
    w_before = [(W.copy(), b.copy()) for W, b in layers]
    # hidden units within rounding of zero: the oracle takes the gate the kernels took (a few per batch)
    out, flips = oracle_step_following_gates(O, tables_c, state, layers, accs, len(cfg.bottom) - 1, small, cfg.lr,
                                             cfg.eps, cfg.bf16, rep.grad_pooled.cpu().numpy(), RTOL_BF16)
    assert len(flips) <= 1e-4 * cfg.B * (sum(cfg.bottom[1:]) + sum(cfg.top[1:-1])), flips
    note = f" ({len(flips)} top-MLP gates at the edge followed the kernel: {flips})"

    # integer outputs, bit-exact at full size (560k lookups: 26 per-table sorts in shared memory, 3 digit passes each)
    U = int(rep.num_unique.item())
    assert U == len(uniq) == len(out["uniq_keys"])
    assert np.array_equal(rep.uniq_keys.cpu().numpy()[:U], uniq)
    assert np.array_equal(rep.seg_off.cpu().numpy()[:U + 1], out["seg_off"])
    assert np.array_equal(rep.perm.cpu().numpy()[:batch.L], out["perm"])
    # pooled embeddings (float32 copy of the concat buffer), every bag
    assert_close(rep.concat_f32.cpu().numpy()[:, cfg.D:], out["pooled"].reshape(cfg.B, -1), RTOL_F32, "pooled")
    # MLP outputs through the tensor-core path
    assert_close(rep.logit.cpu().numpy(), out["logit"], RTOL_BF16, "logit")
    assert abs(float(rep.loss.item()) - out["loss"]) <= RTOL_BF16 * abs(out["loss"])
    assert_close(rep.grad_pooled.cpu().numpy(), out["grad_pooled"], RTOL_BF16, "grad_pooled" + note)
    new = trainer.unpack_params(spec, rep.w.cpu().numpy())
    for l in range(len(layers)):
        assert_close(new[l][0] - w_before[l][0], layers[l][0].astype(np.float64) - w_before[l][0], RTOL_BF16, f"dW[{l}]" + note)
        assert_close(new[l][1] - w_before[l][1], layers[l][1].astype(np.float64) - w_before[l][1], RTOL_BF16, f"db[{l}]" + note)
    # every touched row of the 6.7 GB tables, and its optimizer state
    rows_dev = model.tables.view(-1, cfg.D)[torch.from_numpy(uniq).cuda()].cpu().numpy()
    want = tables_c[t_of, local]
    assert_close(rows_dev - t_before[t_of, local], want.astype(np.float64) - t_before[t_of, local], RTOL_BF16, "row updates")
    assert_close(model.row_state[torch.from_numpy(uniq).cuda()].cpu().numpy(), state[t_of, local], RTOL_BF16, "row state")
    # rows the batch did not touch are unchanged (a sample)
    rng = np.random.default_rng(0)
    for t in (0, 13, 25):
        rows = np.setdiff1d(rng.integers(0, cfg.N, 400), uniq[t_of == t] % cfg.N)
        got = model.tables[t][torch.from_numpy(rows).cuda()].cpu().numpy()
        assert np.array_equal(got, synth.table_rows(cfg, t, rows))


def test_large_workload_embedding_path_full_size():
    """The embedding calls of the large workload at its full size (26 tables of 4 M rows x 128 floats = 53 GB filled
    on the device, batch 4096, about 852 k lookups with 27-bit keys): more lookups than the per-table shared-memory
    sort can hold, so the tiled radix passes run (three digits, about 208 tiles), the hottest row of a table has
    thousands of lookups (runs spanning hundreds of reduction windows) and rows are 128 floats wide.  Forward, sort
    (integers bit-exact) and reduction + row-wise Adagrad against the oracle on the compact table of touched rows;
    the gradient is a seeded synthetic matrix, so no MLP (and no ReLU gate) is involved."""
    cfg = synth.scaled(synth.CONFIGS["large"], R=1)
    T, N, D, B = cfg.T, cfg.N, cfg.D, cfg.B
    batch = synth.make_batch(cfg, 0, 0)
    L = batch.L
    assert L > T * ss.SS_TABLE_SORT_CAP                      # the tiled passes are certain
    tables_c, small, uniq, t_of, local, nmax = _compact(cfg, batch)
    tables = trainer.device_tables(cfg)
    state = torch.zeros(T * N, dtype=torch.float32, device="cuda")
    idx, off = torch.from_numpy(batch.indices).cuda(), torch.from_numpy(batch.offsets).cuda()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    W = (1 + T) * D
    concat = torch.zeros(B, W, device="cuda")
    ss.ss_embbag_fwd(tables, T, N, D, idx, off, B, concat, W, None, W, D, status)
    want_pooled = O.embbag_fwd(tables_c, small.indices, small.offsets, B)
    assert_close(concat.cpu().numpy()[:, D:], want_pooled.reshape(B, -1), RTOL_F32, "pooled")

    ws = torch.empty(ss.ss_embbag_bwd_workspace_bytes(T, N, D, B, L), dtype=torch.uint8, device="cuda")
    uk = torch.empty(L, dtype=torch.int32, device="cuda")
    so = torch.empty(L + 1, dtype=torch.int32, device="cuda")
    pm = torch.empty(L, dtype=torch.int32, device="cuda")
    nu = torch.zeros(1, dtype=torch.int32, device="cuda")
    ss.ss_embbag_bwd_sort(T, N, D, idx, off, B, L, ws, uk, so, pm, nu, status)
    torch.cuda.synchronize()
    want_uniq, want_seg, want_perm = O.sort_unique(batch.indices, batch.offsets, T, N, B)
    U = int(nu.item())
    assert U == len(want_uniq) == len(uniq)
    assert np.array_equal(uk.cpu().numpy()[:U], want_uniq)
    assert np.array_equal(so.cpu().numpy()[:U + 1], want_seg)
    assert np.array_equal(pm.cpu().numpy(), want_perm)
    assert int(np.diff(want_seg).max()) > 2000               # a run over hundreds of 16-position windows

    gp = (synth.normal_f32(synth.stream_key(cfg.seed, synth.stream_id(synth.KIND_VEC, 77)), B * T * D, 1e-3)
          .reshape(B, T * D))
    ss.ss_embbag_bwd_apply(tables, state, T, N, D, B, L, torch.from_numpy(gp).cuda(), T * D, 0, cfg.lr, cfg.eps, ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    t_before = tables_c.copy()
    state_c = np.zeros((T, nmax), np.float32)
    O.embbag_bwd_adagrad(tables_c, state_c, small.indices, small.offsets, B, gp, cfg.lr, cfg.eps)
    ukeys = torch.from_numpy(uniq).cuda()
    rows_dev = tables.view(-1, D)[ukeys].cpu().numpy()
    # the row step is lr * g / (sqrt(s) + eps): compared on the step, 2e-5 (a sum of up to thousands of float terms)
    assert_close(rows_dev - t_before[t_of, local], tables_c[t_of, local].astype(np.float64) - t_before[t_of, local],
                 2e-5, "row updates")
    assert_close(state[ukeys].cpu().numpy(), state_c[t_of, local], 2e-5, "row state")
    rng = np.random.default_rng(1)
    for t in (0, 12, 25):                                    # untouched rows keep their initial values
        rows = np.setdiff1d(rng.integers(0, N, 300), uniq[t_of == t] % N)
        assert np.array_equal(tables[t][torch.from_numpy(rows).cuda()].cpu().numpy(), synth.table_rows(cfg, t, rows))


def test_sort_with_one_table_beyond_the_shared_memory_sort_beside_tables_within_it():
    """Three tables in one call: the middle one has more lookups than one block of the per-table sort holds
    (its block raises the fallback word and the tiled passes redo the whole call), the outer two would fit."""
    T, N, B = 3, 1 << 20, 4096
    rng = np.random.default_rng(11)
    lens = np.concatenate([rng.integers(1, 4, B), rng.integers(6, 12, B), rng.integers(0, 3, B)])
    off = np.zeros(T * B + 1, np.int32)
    off[1:] = np.cumsum(lens)
    L = int(off[-1])
    assert int(off[2 * B] - off[B]) > ss.SS_TABLE_SORT_CAP and L <= T * ss.SS_TABLE_SORT_CAP
    idx = (rng.zipf(1.3, L) % N).astype(np.int32)
    ws = torch.empty(ss.ss_embbag_bwd_workspace_bytes(T, N, 64, B, L), dtype=torch.uint8, device="cuda")
    uk = torch.empty(L, dtype=torch.int32, device="cuda")
    so = torch.empty(L + 1, dtype=torch.int32, device="cuda")
    pm = torch.empty(L, dtype=torch.int32, device="cuda")
    nu = torch.zeros(1, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ss.ss_embbag_bwd_sort(T, N, 64, torch.from_numpy(idx).cuda(), torch.from_numpy(off).cuda(), B, L, ws, uk, so, pm, nu, status)
    torch.cuda.synchronize()
    want_uniq, want_seg, want_perm = O.sort_unique(idx, off, T, N, B)
    U = int(nu.item())
    assert int(status.item()) == 0 and U == len(want_uniq)
    assert np.array_equal(uk.cpu().numpy()[:U], want_uniq)
    assert np.array_equal(so.cpu().numpy()[:U + 1], want_seg)
    assert np.array_equal(pm.cpu().numpy(), want_perm)


@pytest.mark.parametrize("rule", ["easgd", "ma", "bmuf"])
def test_sync_rules_on_hbm_sized_vectors(rule):
    # 4 replicas of 64M floats (1.3 GB moved per pass); the rules are element-wise, so slices are checked exactly
    n, R = 1 << 26, 4
    g = torch.Generator(device="cuda").manual_seed(5)
    ws = [torch.randn(n, device="cuda", generator=g) * 0.02 for _ in range(R)]
    c = torch.randn(n, device="cuda", generator=g) * 0.02
    d = torch.randn(n, device="cuda", generator=g) * 0.002
    idx = [slice(0, 4096), slice(n // 2 - 1111, n // 2 + 3001), slice(n - 5000, n)]
    before = [([w[s].cpu().numpy().copy() for w in ws], c[s].cpu().numpy().copy(), d[s].cpu().numpy().copy()) for s in idx]
    if rule == "easgd":
        ss.ss_sync_easgd(ws, c, n, 0.1)
    elif rule == "ma":
        ss.ss_sync_ma(ws, c, n, 0.1)
    else:
        ss.ss_sync_bmuf(ws, c, d, n, 0.1, 1.0, 0.9)
    torch.cuda.synchronize()
    for s, (w0, c0, d0) in zip(idx, before):
        if rule == "easgd":
            O.sync_easgd(w0, c0, 0.1)
        elif rule == "ma":
            O.sync_ma(w0, 0.1, c0)
        else:
            O.sync_bmuf(w0, c0, d0, 0.1, 1.0, 0.9)
        for r in range(R):
            assert_close(ws[r][s].cpu().numpy(), w0[r], RTOL_SYNC, f"{rule} replica {r}")
        assert_close(c[s].cpu().numpy(), c0, RTOL_SYNC, f"{rule} centre")
        if rule == "bmuf":
            assert_close(d[s].cpu().numpy(), d0, RTOL_SYNC, "delta")
