"""The seeded input generators: determinism, shapes, and the distributions the workloads call for."""
import numpy as np

from paper_2003_03477_b200 import synth


def test_counter_based_values_are_pure_functions():
    cfg = synth.CONFIGS["tiny"]
    a = synth.table_rows(cfg, 3, [5, 9999])
    dense = synth.tables_dense(cfg)
    assert np.array_equal(a, dense[3, [5, 9999]])
    assert dense.dtype == np.float32 and dense.min() >= -0.05 and dense.max() < 0.05
    assert abs(float(dense.mean())) < 1e-3
    b1, b2 = synth.make_batch(cfg, 1, 7), synth.make_batch(cfg, 1, 7)
    assert np.array_equal(b1.indices, b2.indices) and np.array_equal(b1.dense, b2.dense)
    assert not np.array_equal(b1.indices, synth.make_batch(cfg, 0, 7).indices[:b1.L])


def test_tiny_batch_shape_and_bag_mix():
    cfg = synth.CONFIGS["tiny"]
    b = synth.make_batch(cfg, 0, 0)
    lens = np.diff(b.offsets)
    assert b.offsets.shape == (cfg.T * cfg.B + 1,) and b.offsets[0] == 0 and b.offsets[-1] == b.L
    assert lens.min() >= 1 and lens.max() <= 10 and abs(lens.mean() - 4.014) < 0.15
    assert b.indices.min() >= 0 and b.indices.max() < cfg.N
    assert b.dense.shape == (256, 13) and set(np.unique(b.labels)) <= {0.0, 1.0}


def test_zipf_rows_are_skewed_and_scattered():
    cfg = synth.scaled(synth.CONFIGS["medium"], B=512, T=2)
    b = synth.make_batch(cfg, 0, 0)
    lens = np.diff(b.offsets)
    assert lens.min() >= 1 and lens.max() <= 20 and abs(lens.mean() - 10.5) < 0.5
    t0 = b.indices[: b.offsets[cfg.B]]
    vals, counts = np.unique(t0, return_counts=True)
    share = counts.max() / t0.size
    assert 0.06 < share < 0.13                 # hottest row of Zipf(1.05) over 1e6 rows: about 9 %
    assert vals.size < 0.7 * t0.size           # many duplicates
    hot0 = vals[counts.argmax()]
    t1 = b.indices[b.offsets[cfg.B]: b.offsets[2 * cfg.B]]
    v1, c1 = np.unique(t1, return_counts=True)
    assert v1[c1.argmax()] != hot0             # hot rows differ between tables


def test_initial_weights_follow_the_uniform_rule():
    cfg = synth.CONFIGS["tiny"]
    ws = synth.initial_weights(cfg)
    assert [w.shape for w, _ in ws] == [(64, 13), (16, 64), (64, 144), (1, 64)]
    for (w, b), (fin, fout) in zip(ws, synth.layer_dims(cfg)):
        a = (6.0 / (fin + fout)) ** 0.5
        assert np.abs(w).max() <= a and not b.any()
    assert sum(w.size + b.size for w, b in ws) == 11281
