"""The allocation-free sort entry point against the workspace one.

ss_embbag_bwd_sort_noalloc is for callers that cannot obtain device memory when they need the sort (the
GPU's memory is already owned by someone else's pool, or an allocation's device-wide synchronisation is
not acceptable where they run): its scratch is a fixed array inside the library.  The test calls it
through the C boundary twice in a row on different batches -- the second call finds the array full of the
first call's data -- and requires integer outputs identical to ss_embbag_bwd_sort's, which is the
tolerance every sort test here uses.  This file sorts last on purpose, so that a run stopping at the
first failure has already been through every other test.
"""
import numpy as np
import pytest
import torch

from paper_2003_03477_b200 import binding as ss
from paper_2003_03477_b200 import synth

pytestmark = pytest.mark.gpu


def _sort_both(cfg, batch):
    T, N, D, B, L = cfg.T, cfg.N, cfg.D, cfg.B, batch.L
    idx = torch.from_numpy(batch.indices).cuda()
    off = torch.from_numpy(batch.offsets).cuda()

    def outputs():
        return (torch.full((L,), -1, dtype=torch.int32, device="cuda"),
                torch.full((L + 1,), -1, dtype=torch.int32, device="cuda"),
                torch.full((L,), -1, dtype=torch.int32, device="cuda"),
                torch.full((1,), -1, dtype=torch.int32, device="cuda"),
                torch.zeros(1, dtype=torch.int32, device="cuda"))

    ref = outputs()
    ws = torch.empty(ss.ss_embbag_bwd_workspace_bytes(T, N, D, B, L), dtype=torch.uint8, device="cuda")
    ss.ss_embbag_bwd_sort(T, N, D, idx, off, B, L, ws, ref[0], ref[1], ref[2], ref[3], ref[4])
    got = outputs()
    ss.ss_embbag_bwd_sort_noalloc(T, N, idx, off, B, L, got[0], got[1], got[2], got[3], got[4])
    torch.cuda.synchronize()
    U = int(ref[3].item())
    assert int(got[3].item()) == U and int(got[4].item()) == int(ref[4].item()) == 0
    assert torch.equal(got[0][:U], ref[0][:U]), "unique keys"
    assert torch.equal(got[1][:U + 1], ref[1][:U + 1]), "segment offsets"
    assert torch.equal(got[2], ref[2]), "permutation"
    # and both are a correct stable sort
    lens = np.diff(batch.offsets.astype(np.int64))
    keys = np.repeat(np.arange(T * B) // B, lens) * N + batch.indices
    assert np.array_equal(got[2].cpu().numpy(), np.argsort(keys, kind="stable"))
    return U


def test_noalloc_sort_matches_workspace_sort_on_two_calls_in_a_row():
    # Zipf-skewed rows, about 21k lookups: several sort tiles, a ragged last tile, long runs of equal keys
    cfg = synth.scaled(synth.CONFIGS["medium"], T=4, N=20_000, D=64, B=512, bottom=(13, 64, 64), top=(320, 64, 1))
    u1 = _sort_both(cfg, synth.make_batch(cfg, 0, 0))
    # second call, smaller and different: the built-in array still holds the first call's buffers
    small = synth.scaled(cfg, T=3, N=700, B=200)
    u2 = _sort_both(small, synth.make_batch(small, 1, 5))
    assert u1 > u2 > 0


def test_noalloc_sort_rejects_sizes_beyond_its_scratch():
    z = torch.zeros(8, dtype=torch.int32, device="cuda")
    with pytest.raises(ss.SsError) as e:
        ss.ss_embbag_bwd_sort_noalloc(2, 100, z, z, 2, 65537, z, z, z, z, z)
    assert e.value.status == -2
