"""GPU parity of ss_embbag_fwd and ss_embbag_bwd_adagrad against the oracle."""
import numpy as np
import pytest
import torch

from oracle import shadowsync_oracle as O
from paper_2003_03477_b200 import binding as ss
from paper_2003_03477_b200 import synth
from parity import RTOL_F32, assert_close

pytestmark = pytest.mark.gpu


def _cuda(a, dt=None):
    t = torch.from_numpy(np.ascontiguousarray(a)).cuda()
    return t if dt is None else t.to(dt)


def _fwd(tables, idx, off, B, col0=None, want_bf16=False):
    T, N, D = tables.shape
    col0 = D if col0 is None else col0
    W = col0 + T * D
    out = torch.full((B, W), -7.0, device="cuda")
    outh = torch.zeros(B, W, dtype=torch.bfloat16, device="cuda") if want_bf16 else None
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    ss.ss_embbag_fwd(_cuda(tables), T, N, D, _cuda(idx), _cuda(off), B, out, W, outh, W, col0, st)
    torch.cuda.synchronize()
    return out.cpu().numpy(), (outh.float().cpu().numpy() if want_bf16 else None), int(st.item())


@pytest.mark.parametrize("D", [4, 8, 16, 64, 128, 256])
def test_fwd_parity_small(D):
    cfg = synth.scaled(synth.CONFIGS["tiny"], T=3, N=500, D=D, B=37, bottom=(13, 64, D), top=(4 * D, 64, 1))
    b = synth.make_batch(cfg, 0, 0)
    tables = synth.tables_dense(cfg)
    want = O.embbag_fwd(tables, b.indices, b.offsets, cfg.B)
    got, goth, st = _fwd(tables, b.indices, b.offsets, cfg.B, want_bf16=True)
    assert st == 0
    assert_close(got[:, D:], want.reshape(cfg.B, -1), RTOL_F32, "pooled")
    assert (got[:, :D] == -7.0).all()                     # columns before col0 are not touched
    assert np.array_equal(goth[:, D:], torch.from_numpy(got[:, D:]).to(torch.bfloat16).float().numpy())


def test_fwd_tiny_config_full():
    cfg = synth.CONFIGS["tiny"]
    b = synth.make_batch(cfg, 1, 3)
    tables = synth.tables_dense(cfg)
    want = O.embbag_fwd(tables, b.indices, b.offsets, cfg.B)
    got, _, st = _fwd(tables, b.indices, b.offsets, cfg.B)
    assert st == 0
    assert_close(got[:, cfg.D:], want.reshape(cfg.B, -1), RTOL_F32, "pooled")


def test_fwd_edge_cases_empty_bags_single_row_duplicates_and_bad_index():
    tables = np.random.default_rng(0).normal(size=(2, 7, 8)).astype(np.float32)
    # table 0: bag0 = [], bag1 = [3], bag2 = [5, 5, 5]; table 1: bag0 = [6, 0], bag1 = [], bag2 = [9 (bad), 1]
    idx = np.array([3, 5, 5, 5, 6, 0, 9, 1], np.int32)
    off = np.array([0, 0, 1, 4, 6, 6, 8], np.int32)
    got, _, st = _fwd(tables, idx, off, 3, col0=0)
    assert st == ss.SS_DEV_BAD_INDEX
    assert not got[0, :8].any() and np.array_equal(got[1, :8], tables[0, 3])
    assert_close(got[2, :8], 3.0 * tables[0, 5].astype(np.float64), RTOL_F32)
    assert_close(got[0, 8:], tables[1, 6].astype(np.float64) + tables[1, 0], RTOL_F32)
    assert not got[1, 8:].any() and np.array_equal(got[2, 8:], tables[1, 1])   # the bad lookup is skipped
    # all-ones table: pooled = bag length exactly
    ones = np.ones((2, 7, 8), np.float32)
    idx[6] = 2
    got, _, st = _fwd(ones, idx, off, 3, col0=0)
    assert st == 0 and np.array_equal(got[:, 0], [0, 1, 3]) and np.array_equal(got[:, 8], [2, 0, 2])


def test_fwd_malformed_offsets_give_empty_bags_and_a_status_bit():
    """Offsets that decrease, are negative or point beyond the end of the index list (offsets[T*B]) must not
    become reads outside the list: such a bag pools to zero and SS_DEV_BAD_OFFSET is raised; the well-formed
    bags of the same call are unaffected."""
    tables = np.random.default_rng(1).normal(size=(1, 7, 8)).astype(np.float32)
    idx = np.array([3, 5, 6, 1], np.int32)
    for off, bad_bags in ((np.array([0, 1, 1 << 30, 3, 4], np.int32), (1, 2)),     # far beyond the list
                          (np.array([0, 2, 1, 3, 4], np.int32), (1,)),              # decreasing
                          (np.array([0, -5, 2, 3, 4], np.int32), (0, 1))):          # negative
        got, _, st = _fwd(tables, idx, off, 4, col0=0)
        assert st & ss.SS_DEV_BAD_OFFSET, off
        for b in range(4):
            if b in bad_bags:
                assert not got[b].any(), (off, b)
            else:
                want = tables[0, idx[off[b]:off[b + 1]]].astype(np.float64).sum(axis=0)
                assert_close(got[b], want, RTOL_F32, f"bag {b}", floor=1.0)


def _bwd(cfg, batch, tables, state, gp, keep=True):
    T, N, D, B, L = cfg.T, cfg.N, cfg.D, cfg.B, batch.L
    dt, ds = _cuda(tables), _cuda(state.reshape(-1))
    ws = torch.empty(ss.ss_embbag_bwd_workspace_bytes(T, N, D, B, L), dtype=torch.uint8, device="cuda")
    uniq = torch.full((max(L, 1),), -1, dtype=torch.int32, device="cuda")
    seg = torch.full((L + 1,), -1, dtype=torch.int32, device="cuda")
    perm = torch.full((max(L, 1),), -1, dtype=torch.int32, device="cuda")
    nu = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    ss.ss_embbag_bwd_adagrad(dt, ds, T, N, D, _cuda(batch.indices), _cuda(batch.offsets), B, L, _cuda(gp), T * D, 0,
                             cfg.lr, cfg.eps, ws, uniq, seg, perm, nu, st)
    torch.cuda.synchronize()
    U = int(nu.item())
    return (dt.cpu().numpy(), ds.cpu().numpy().reshape(T, N), uniq.cpu().numpy()[:U], seg.cpu().numpy()[:U + 1],
            perm.cpu().numpy()[:L], int(st.item()))


def _check_bwd(cfg, step=0, seed=0):
    b = synth.make_batch(cfg, 0, step)
    tables = synth.tables_dense(cfg)
    rng = np.random.default_rng(seed)
    state = (rng.random((cfg.T, cfg.N)) * 1e-4).astype(np.float32)
    gp = (rng.normal(size=(cfg.B, cfg.T * cfg.D)) * 1e-3).astype(np.float32)
    t_o, s_o = tables.copy(), state.copy()
    uniq, seg, perm = O.embbag_bwd_adagrad(t_o, s_o, b.indices, b.offsets, cfg.B, gp, cfg.lr, cfg.eps)
    t_g, s_g, uniq_g, seg_g, perm_g, st = _bwd(cfg, b, tables, state, gp)
    assert st == 0
    # integer outputs are bit-exact
    assert np.array_equal(uniq_g, uniq) and np.array_equal(seg_g, seg) and np.array_equal(perm_g, perm)
    # the update is compared on the *change* of the touched rows and on the state
    assert_close(t_g - tables, t_o.astype(np.float64) - tables, 2e-5, "table update")
    assert_close(s_g, s_o, RTOL_F32, "row state")
    untouched = np.ones((cfg.T, cfg.N), bool)
    untouched[uniq // cfg.N, uniq % cfg.N] = False
    assert np.array_equal(t_g[untouched], tables[untouched])
    return len(uniq), b.L


@pytest.mark.parametrize("D", [4, 16, 64, 128])
def test_bwd_parity_small_uniform(D):
    cfg = synth.scaled(synth.CONFIGS["tiny"], T=3, N=300, D=D, B=64, bottom=(13, 64, D), top=(4 * D, 64, 1))
    U, L = _check_bwd(cfg)
    assert U < L            # 300 rows per table: duplicates, segments longer than one


def test_bwd_parity_skewed_long_segments_cross_windows_and_sort_tiles():
    # Zipf rows: the hottest row of each table has hundreds of lookups -> runs spanning many 16-wide windows;
    # about 5k lookups per table: the per-table shared-memory sort takes them (the tiled passes are covered by the
    # malformed-input cases, the no-scratch entry point and the full-size test of the large workload)
    cfg = synth.scaled(synth.CONFIGS["medium"], T=4, N=20_000, D=64, B=512, bottom=(13, 64, 64), top=(320, 64, 1))
    U, L = _check_bwd(cfg)
    assert L > 4 * 4096 and U < L // 2


def test_bwd_tiny_config_full():
    _check_bwd(synth.CONFIGS["tiny"], step=2)


def test_bwd_edge_cases():
    # one row hit by every bag; bags of length 1; an empty table slice; a bad index
    T, N, D, B = 3, 50, 8, 40
    cfg = synth.scaled(synth.CONFIGS["tiny"], T=T, N=N, D=D, B=B)
    idx0 = np.full(B, 7, np.int32)                               # table 0: every bag hits row 7
    idx2 = (np.arange(B) % N).astype(np.int32)                   # table 2: bags of one lookup
    idx = np.concatenate([idx0, idx2])
    off = np.concatenate([np.arange(B + 1), np.full(B, B), B + 1 + np.arange(B)]).astype(np.int32)  # table 1 empty
    batch = synth.Batch(idx, off, np.zeros((B, 13), np.float32), np.zeros(B, np.float32))
    tables = synth.tables_dense(cfg)
    state = np.zeros((T, N), np.float32)
    gp = np.random.default_rng(1).normal(size=(B, T * D)).astype(np.float32)
    t_o, s_o = tables.copy(), state.copy()
    uniq, seg, perm = O.embbag_bwd_adagrad(t_o, s_o, idx, off, B, gp, cfg.lr, cfg.eps)
    t_g, s_g, uniq_g, seg_g, perm_g, st = _bwd(cfg, batch, tables, state, gp)
    assert st == 0 and np.array_equal(uniq_g, uniq) and np.array_equal(seg_g, seg) and np.array_equal(perm_g, perm)
    assert uniq[0] == 7 and seg[1] == B
    assert_close(t_g - tables, t_o.astype(np.float64) - tables, 2e-5, "table update")
    assert_close(s_g, s_o, RTOL_F32, "row state")
    # a bad index is flagged and skipped; the remaining lookups give the oracle's result on the cleaned input
    idx_bad = idx.copy()
    idx_bad[3] = N + 5
    batch_bad = synth.Batch(idx_bad, off, batch.dense, batch.labels)
    t_g, s_g, uniq_g, seg_g, perm_g, st = _bwd(cfg, batch_bad, tables, state, gp)
    assert st == ss.SS_DEV_BAD_INDEX
    assert seg_g[-1] == len(idx) - 1 and uniq_g[0] == 7 and seg_g[1] == B - 1
    assert 3 not in perm_g[: seg_g[-1]]


def test_bwd_empty_input():
    cfg = synth.scaled(synth.CONFIGS["tiny"], T=2, N=10, D=8, B=4)
    batch = synth.Batch(np.zeros(0, np.int32), np.zeros(9, np.int32), np.zeros((4, 13), np.float32), np.zeros(4, np.float32))
    tables = synth.tables_dense(cfg)
    t_g, s_g, uniq_g, seg_g, perm_g, st = _bwd(cfg, batch, tables, np.zeros((2, 10), np.float32),
                                                np.ones((4, 16), np.float32))
    assert st == 0 and len(uniq_g) == 0 and list(seg_g) == [0] and np.array_equal(t_g, tables)


def test_device_table_fill_matches_host_generator():
    from paper_2003_03477_b200 import trainer
    cfg = synth.scaled(synth.CONFIGS["tiny"], T=3, N=1000, D=16)
    dev = trainer.device_tables(cfg).cpu().numpy()
    assert np.array_equal(dev, synth.tables_dense(cfg))


def test_sort_once_apply_twice_matches_two_oracle_updates():
    # the two-call form: the sort half fills the workspace, the apply half may be repeated on it
    cfg = synth.scaled(synth.CONFIGS["medium"], T=3, N=4000, D=64, B=256, bottom=(13, 64, 64), top=(256, 64, 1))
    b = synth.make_batch(cfg, 0, 1)
    tables = synth.tables_dense(cfg)
    state = np.zeros((cfg.T, cfg.N), np.float32)
    rng = np.random.default_rng(3)
    gp = (rng.normal(size=(cfg.B, cfg.T * cfg.D)) * 1e-3).astype(np.float32)
    t_o, s_o = tables.copy(), state.copy()
    for _ in range(3):
        uniq, seg, perm = O.embbag_bwd_adagrad(t_o, s_o, b.indices, b.offsets, cfg.B, gp, cfg.lr, cfg.eps)
    T, N, D, B, L = cfg.T, cfg.N, cfg.D, cfg.B, b.L
    dt, ds = _cuda(tables), _cuda(state.reshape(-1))
    ws = torch.empty(ss.ss_embbag_bwd_workspace_bytes(T, N, D, B, L), dtype=torch.uint8, device="cuda")
    nu = torch.zeros(1, dtype=torch.int32, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    perm_d = torch.empty(L, dtype=torch.int32, device="cuda")
    ss.ss_embbag_bwd_sort(T, N, D, _cuda(b.indices), _cuda(b.offsets), B, L, ws, None, None, perm_d, nu, st)
    dg = _cuda(gp)
    for _ in range(3):
        ss.ss_embbag_bwd_apply(dt, ds, T, N, D, B, L, dg, T * D, 0, cfg.lr, cfg.eps, ws, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0 and int(nu.item()) == len(uniq) and np.array_equal(perm_d.cpu().numpy(), perm)
    assert_close(dt.cpu().numpy() - tables, t_o.astype(np.float64) - tables, 2e-5, "tables after three updates")
    assert_close(ds.cpu().numpy().reshape(T, N), s_o, RTOL_F32, "row state")


def test_apply_refuses_a_workspace_sorted_for_another_problem():
    # the apply half trusts the workspace only if the sort stamped it for the same T, N, L
    cfg = synth.scaled(synth.CONFIGS["medium"], T=3, N=4000, D=64, B=256, bottom=(13, 64, 64), top=(256, 64, 1))
    b1, b2 = synth.make_batch(cfg, 0, 1), synth.make_batch(cfg, 0, 2)
    assert b1.L != b2.L
    T, N, D, B = cfg.T, cfg.N, cfg.D, cfg.B
    Lmax = max(b1.L, b2.L)
    tables = synth.tables_dense(cfg)
    dt, ds = _cuda(tables), torch.zeros(T * N, device="cuda")
    ws = torch.zeros(ss.ss_embbag_bwd_workspace_bytes(T, N, D, B, Lmax), dtype=torch.uint8, device="cuda")
    nu = torch.zeros(1, dtype=torch.int32, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    dg = torch.ones(B, T * D, device="cuda")
    # never sorted: refused
    ss.ss_embbag_bwd_apply(dt, ds, T, N, D, B, b1.L, dg, T * D, 0, 0.1, 1e-8, ws, st)
    torch.cuda.synchronize()
    assert int(st.item()) == ss.SS_DEV_BAD_WORKSPACE and np.array_equal(dt.cpu().numpy(), tables)
    # sorted for batch 1, applied with batch 2's size: refused, tables untouched
    st.zero_()
    ss.ss_embbag_bwd_sort(T, N, D, _cuda(b1.indices), _cuda(b1.offsets), B, b1.L, ws, None, None, None, nu, st)
    ss.ss_embbag_bwd_apply(dt, ds, T, N, D, B, b2.L, dg, T * D, 0, 0.1, 1e-8, ws, st)
    torch.cuda.synchronize()
    assert int(st.item()) == ss.SS_DEV_BAD_WORKSPACE and np.array_equal(dt.cpu().numpy(), tables)
    # matching call goes through
    st.zero_()
    ss.ss_embbag_bwd_apply(dt, ds, T, N, D, B, b1.L, dg, T * D, 0, 0.1, 1e-8, ws, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0 and not np.array_equal(dt.cpu().numpy(), tables)
