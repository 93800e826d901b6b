"""GPU parity of ss_sync_easgd / ss_sync_ma / ss_sync_bmuf against the oracle (Algorithms 2-4)."""
import numpy as np
import pytest
import torch

from oracle import shadowsync_oracle as O
from paper_2003_03477_b200 import binding as ss
from paper_2003_03477_b200 import synth
from parity import RTOL_SYNC, assert_close

pytestmark = pytest.mark.gpu


def _dev(vs):
    return [torch.from_numpy(v.copy()).cuda() for v in vs]


def _run(rule, R, n, alpha, eta=1.0, mu=0.0, flags=0, mirror=False, seed=1, floor=0.0):
    ws = synth.sync_vectors(n, R, seed)
    c = synth.sync_vectors(n, 1, seed + 100)[0]
    d = synth.sync_vectors(n, 1, seed + 200)[0] if rule == "bmuf" else None
    dw, dc = _dev(ws), torch.from_numpy(c.copy()).cuda()
    dd = torch.from_numpy(d.copy()).cuda() if d is not None else None
    mir = [torch.zeros(n, dtype=torch.bfloat16, device="cuda") for _ in range(R)] if mirror else None
    if rule == "easgd":
        ss.ss_sync_easgd(dw, dc, n, alpha, flags, mir)
        O.sync_easgd(ws, c, alpha, literal=bool(flags & 1))
    elif rule == "ma":
        ss.ss_sync_ma(dw, dc, n, alpha, 0, mir)
        O.sync_ma(ws, alpha, c)
    else:
        ss.ss_sync_bmuf(dw, dc, dd, n, alpha, eta, mu, flags, mir)
        O.sync_bmuf(ws, c, d, alpha, eta, mu, nesterov=bool(flags & ss.SS_SYNC_BMUF_NESTEROV))
    torch.cuda.synchronize()
    for r in range(R):
        assert_close(dw[r].cpu().numpy(), ws[r], RTOL_SYNC, f"{rule} w[{r}]", floor)
        if mirror:
            assert torch.equal(mir[r], dw[r].to(torch.bfloat16)), "bf16 mirror must be the rounded new value"
    assert_close(dc.cpu().numpy(), c, RTOL_SYNC, f"{rule} centre", floor)
    if d is not None:
        assert_close(dd.cpu().numpy(), d, RTOL_SYNC, "bmuf delta", floor)
    return dw, dc


@pytest.mark.parametrize("rule", ["easgd", "ma", "bmuf"])
@pytest.mark.parametrize("R", [1, 2, 3, 4, 8, 16])
def test_sync_parity_ragged_sizes(rule, R):
    # several blocks of 1024 elements plus a tail that is not a multiple of 4
    _run(rule, R, 5 * 1024 + 3, 0.1, eta=1.0, mu=0.9)


@pytest.mark.parametrize("rule", ["easgd", "ma", "bmuf"])
def test_sync_parity_1m_with_mirror(rule):
    _run(rule, 4, 1 << 20, 0.05, eta=0.7, mu=0.5, mirror=True)


def test_sync_tiny_and_empty():
    for n in (0, 1, 3, 4, 5):
        if n == 0:
            w = [torch.zeros(4, device="cuda")]
            ss.ss_sync_easgd(w, torch.zeros(4, device="cuda"), 0, 0.1)
        else:
            # a handful of elements: the operands' scale (std 0.02) is the reference, not a cancelled result
            _run("easgd", 2, n, 0.3, floor=0.02)
            _run("bmuf", 2, n, 0.3, 0.5, 0.9, floor=0.02)


def test_bmuf_nesterov_flag():
    _run("bmuf", 4, 6 * 1024 + 1, 0.1, eta=1.0, mu=0.9, flags=ss.SS_SYNC_BMUF_NESTEROV, mirror=True)


def test_easgd_literal_flag():
    _run("easgd", 3, 4099, 0.2, flags=ss.SS_SYNC_EASGD_LITERAL)


def test_alpha_limits_and_invariants_on_device():
    n, R = 10007, 4
    ws = synth.sync_vectors(n, R, 3)
    c = synth.sync_vectors(n, 1, 4)[0]
    dw, dc = _dev(ws), torch.from_numpy(c.copy()).cuda()
    ss.ss_sync_easgd(dw, dc, n, 0.0)                      # alpha = 0: bitwise identity
    assert all(np.array_equal(a.cpu().numpy(), b) for a, b in zip(dw, ws)) and np.array_equal(dc.cpu().numpy(), c)
    before = c.astype(np.float64) + sum(w.astype(np.float64) for w in ws)
    ss.ss_sync_easgd(dw, dc, n, 0.1)                      # centre + replicas conserved
    after = dc.double().cpu().numpy() + sum(w.double().cpu().numpy() for w in dw)
    np.testing.assert_allclose(after, before, atol=(R + 1) * 1.5e-8)
    same = _dev([ws[0]] * 4)
    ss.ss_sync_ma(same, None, n, 0.37)                    # identical replicas: bitwise identity (R power of two)
    assert all(np.array_equal(a.cpu().numpy(), ws[0]) for a in same)
    dw = _dev(ws)
    g = torch.zeros(n, device="cuda")
    ss.ss_sync_ma(dw, g, n, 1.0)                          # alpha = 1: every replica becomes the mean
    for a in dw:                                          # (w + 1*(m - w) rounds once more than m itself)
        assert_close(a.cpu().numpy(), g.cpu().numpy(), RTOL_SYNC, "ma alpha=1")
    # BMUF with mu = 0, eta = 1 equals MA
    a, b = _dev(ws), _dev(ws)
    gg, dl = torch.from_numpy(c.copy()).cuda(), torch.zeros(n, device="cuda")
    ss.ss_sync_ma(a, None, n, 0.05)
    ss.ss_sync_bmuf(b, gg, dl, n, 0.05, 1.0, 0.0)
    for x, y in zip(a, b):
        assert_close(y.cpu().numpy(), x.cpu().numpy(), RTOL_SYNC, "bmuf(mu=0,eta=1) vs ma")


def test_sync_rejects_bad_arguments():
    w = [torch.zeros(8, device="cuda"), torch.zeros(8, device="cuda")]
    c = torch.zeros(8, device="cuda")
    with pytest.raises(ss.SsError) as e:
        ss.ss_sync_easgd(w, c, 8, 1.5)
    assert e.value.status == -8
    with pytest.raises(ss.SsError) as e:
        ss.ss_sync_easgd([w[0][1:5], w[1]], c, 4, 0.1)   # misaligned replica pointer
    assert e.value.status == -3
    with pytest.raises(ss.SsError) as e:
        ss.ss_sync_bmuf(w, c, torch.zeros(8, device="cuda"), 8, 0.1, 1.0, 1.0)   # mu must be < 1
    assert e.value.status == -8
