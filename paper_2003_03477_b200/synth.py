"""Seeded synthetic inputs for the ShadowSync hot path (click-log-shaped CTR data).

This module only *generates inputs*: host numpy arrays (indices, offsets, dense
features, labels, initial weights, initial tables).  It holds none of the
method's arithmetic and imports neither the CUDA binding nor the CPU oracle;
both consume the arrays produced here.

Random numbers come from one counter-based generator: the SplitMix64 output
function (Steele, Lea & Flood, "Fast splittable pseudorandom number
generators", OOPSLA 2014) applied to ``key + (counter + 1) * GAMMA`` where
``key = mix64(seed ^ mix64(stream + GAMMA))``.  A value is therefore a pure
function of (seed, stream, counter), which lets a 53 GB table be defined
without ever being materialised on the host: row ``r`` of table ``t`` is
``table_rows(cfg, t, [r])`` and the device fills the same function.

The paper trains on private production click logs (Section 4); the recipes
below stand in for them with the shapes, bag-length mixes and index skews of
the five benchmark configurations.
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Sequence, Tuple

import numpy as np

MASTER_SEED = 20030347
GAMMA = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)

# stream identifiers (kind of data); replica and step are folded in by stream_id()
KIND_TABLE, KIND_W0, KIND_BAGLEN, KIND_ROW, KIND_DENSE, KIND_LABEL, KIND_VEC = range(1, 8)


def mix64(x: np.ndarray) -> np.ndarray:
    """SplitMix64 output mixing function on uint64 arrays (wrapping arithmetic)."""
    x = np.asarray(x, dtype=np.uint64)
    with np.errstate(over="ignore"):
        x = (x ^ (x >> np.uint64(30))) * _M1
        x = (x ^ (x >> np.uint64(27))) * _M2
        return x ^ (x >> np.uint64(31))


def stream_key(seed: int, stream: int) -> np.uint64:
    with np.errstate(over="ignore"):
        s = mix64(np.uint64(stream & 0xFFFFFFFFFFFFFFFF) + GAMMA)
        return np.uint64(mix64(np.uint64(seed & 0xFFFFFFFFFFFFFFFF) ^ s))


def stream_id(kind: int, replica: int = 0, step: int = 0, sub: int = 0) -> int:
    """Pack (kind, replica, step, sub) into one stream number."""
    return (kind << 56) | ((replica & 0xFF) << 48) | ((sub & 0xFFFF) << 32) | (step & 0xFFFFFFFF)


def u32_at(key: np.uint64, counter: np.ndarray) -> np.ndarray:
    """32 random bits for each counter value under a stream key."""
    c = np.asarray(counter, dtype=np.uint64)
    with np.errstate(over="ignore"):
        return (mix64(np.uint64(key) + (c + np.uint64(1)) * GAMMA) >> np.uint64(32)).astype(np.uint32)


def unit_f32(u: np.ndarray) -> np.ndarray:
    """[0,1) on a 2^-24 grid, exact in float32: (u >> 8) * 2^-24."""
    return (u >> np.uint32(8)).astype(np.float32) * np.float32(2.0 ** -24)


def unit_f64(key: np.uint64, counter: np.ndarray) -> np.ndarray:
    """(0,1) in float64 from one 32-bit draw, never 0: (u + 0.5) * 2^-32."""
    return (u32_at(key, counter).astype(np.float64) + 0.5) * 2.0 ** -32


def uniform_hash_f32(key: np.uint64, counter: np.ndarray, lo: float, hi: float) -> np.ndarray:
    """U(lo,hi) in float32: ((u>>8)*2^-24 - 0.5) * (hi-lo) + mid, every step in float32.

    The device fill evaluates exactly these float32 operations, so host and
    device agree bit for bit.
    """
    x = unit_f32(u32_at(key, counter)) - np.float32(0.5)
    return x * np.float32(hi - lo) + np.float32(0.5 * (hi + lo))


def normal_f32(key: np.uint64, n: int, std: float = 1.0, counter0: int = 0) -> np.ndarray:
    """N(0, std^2) by Box-Muller in float64 on two draws per value, rounded to float32."""
    c = np.arange(n, dtype=np.uint64) * np.uint64(2) + np.uint64(2 * counter0)
    u1 = unit_f64(key, c)
    u2 = unit_f64(key, c + np.uint64(1))
    z = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * math.pi * u2)
    return (z * std).astype(np.float32)


# --------------------------------------------------------------------------------------
# workload configurations
# --------------------------------------------------------------------------------------
@dataclasses.dataclass(frozen=True)
class Config:
    name: str
    R: int                      # trainer replicas
    T: int                      # embedding tables
    N: int                      # rows per table
    D: int                      # embedding dim
    B: int                      # per-replica batch
    bottom: Tuple[int, ...]     # bottom MLP dims, e.g. (13, 64, 16)
    top: Tuple[int, ...]        # top MLP dims, e.g. (144, 64, 1)
    bag: str                    # "poisson4_1_10" | "uniform_1_20" | "poisson8_1_40"
    rows: str                   # "uniform" | "zipf1.05" | "zipf1.2"
    ctr: float                  # Bernoulli label rate
    bf16: bool                  # bf16 GEMM operands with fp32 master weights
    lr: float = 0.01
    eps: float = 1e-8
    sync: str = "easgd"
    alpha: float = 0.1
    eta: float = 1.0
    mu: float = 0.0
    sync_every: int = 0         # 0 = free-running background sync
    steps: int = 0
    seed: int = MASTER_SEED

    @property
    def W(self) -> int:
        return (1 + self.T) * self.D


CONFIGS = {
    # tiny fp32 model, S-EASGD alpha 0.1 every 5 steps, 20 steps per replica
    "tiny": Config("tiny", R=2, T=8, N=10_000, D=16, B=256, bottom=(13, 64, 16), top=(144, 64, 1),
                   bag="poisson4_1_10", rows="uniform", ctr=0.03, bf16=False,
                   sync="easgd", alpha=0.1, sync_every=5, steps=20),
    # medium model, bf16 GEMMs, S-EASGD alpha 0.05 continuously in the background
    "medium": Config("medium", R=4, T=26, N=1_000_000, D=64, B=2048, bottom=(13, 512, 256, 64),
                     top=(1728, 512, 256, 1), bag="uniform_1_20", rows="zipf1.05", ctr=0.03,
                     bf16=True, sync="easgd", alpha=0.05),
    # medium model, R=8, S-BMUF mu 0.9 eta 1.0, one sync pass per 10 local steps
    "medium_bmuf": Config("medium_bmuf", R=8, T=26, N=1_000_000, D=64, B=1024,
                          bottom=(13, 512, 256, 64), top=(1728, 512, 256, 1), bag="uniform_1_20",
                          rows="zipf1.05", ctr=0.05, bf16=True, sync="bmuf", alpha=0.05, eta=1.0,
                          mu=0.9, sync_every=10),
    # large model, R=16, S-MA continuously in the background
    "large": Config("large", R=16, T=26, N=4_000_000, D=128, B=4096, bottom=(13, 1024, 512, 128),
                    top=(3456, 1024, 1024, 512, 1), bag="poisson8_1_40", rows="zipf1.2", ctr=0.03,
                    bf16=True, sync="ma", alpha=0.05),
}


def scaled(cfg: Config, **kw) -> Config:
    """A copy of a configuration with some fields changed (smaller cases for parity tests)."""
    return dataclasses.replace(cfg, **kw)


# --------------------------------------------------------------------------------------
# tables and initial weights
# --------------------------------------------------------------------------------------
TABLE_LO, TABLE_HI = -0.05, 0.05


def table_key(cfg: Config) -> np.uint64:
    return stream_key(cfg.seed, stream_id(KIND_TABLE))


def table_rows(cfg: Config, t: int, rows: Sequence[int]) -> np.ndarray:
    """Initial values of some rows of table t: float32 [len(rows), D]; counter=(t*N+row)*D+d."""
    rows = np.asarray(rows, dtype=np.uint64)
    base = (np.uint64(t) * np.uint64(cfg.N) + rows) * np.uint64(cfg.D)
    c = base[:, None] + np.arange(cfg.D, dtype=np.uint64)[None, :]
    return uniform_hash_f32(table_key(cfg), c, TABLE_LO, TABLE_HI)


def tables_dense(cfg: Config) -> np.ndarray:
    """All tables as float32 [T, N, D] (only for configurations that fit on the host)."""
    n = cfg.T * cfg.N * cfg.D
    if n > (1 << 31):
        raise ValueError("tables too large to materialise on the host; use table_rows()")
    c = np.arange(n, dtype=np.uint64)
    return uniform_hash_f32(table_key(cfg), c, TABLE_LO, TABLE_HI).reshape(cfg.T, cfg.N, cfg.D)


def layer_dims(cfg: Config) -> List[Tuple[int, int]]:
    """(in, out) of every Linear layer, bottom layers first then top layers."""
    dims = []
    for d in (cfg.bottom, cfg.top):
        dims += [(d[i], d[i + 1]) for i in range(len(d) - 1)]
    return dims


def initial_weights(cfg: Config) -> List[Tuple[np.ndarray, np.ndarray]]:
    """w0: per layer (W [out,in] ~ U(-a,a) with a = sqrt(6/(in+out)), b = 0), float32."""
    out = []
    for li, (fin, fout) in enumerate(layer_dims(cfg)):
        key = stream_key(cfg.seed, stream_id(KIND_W0, sub=li))
        a = math.sqrt(6.0 / (fin + fout))
        w = uniform_hash_f32(key, np.arange(fin * fout, dtype=np.uint64), -a, a).reshape(fout, fin)
        out.append((w, np.zeros(fout, dtype=np.float32)))
    return out


# --------------------------------------------------------------------------------------
# batches
# --------------------------------------------------------------------------------------
def _poisson_clamped(u: np.ndarray, mean: float, lo: int, hi: int) -> np.ndarray:
    k = np.arange(0, 4 * hi + 64)
    logp = -mean + k * math.log(mean) - np.array([math.lgamma(x + 1.0) for x in k])
    cdf = np.cumsum(np.exp(logp))
    return np.clip(np.searchsorted(cdf, u, side="right"), lo, hi).astype(np.int64)


def bag_lengths(cfg: Config, key: np.uint64, n: int) -> np.ndarray:
    u = unit_f64(key, np.arange(n, dtype=np.uint64))
    if cfg.bag == "poisson4_1_10":
        return _poisson_clamped(u, 4.0, 1, 10)
    if cfg.bag == "poisson8_1_40":
        return _poisson_clamped(u, 8.0, 1, 40)
    if cfg.bag == "uniform_1_20":
        return 1 + np.minimum((u * 20.0).astype(np.int64), 19)
    if cfg.bag.startswith("const"):
        return np.full(n, int(cfg.bag[5:]), dtype=np.int64)
    raise ValueError(cfg.bag)


_ZIPF_CDF = {}


def _zipf_cdf(N: int, s: float) -> np.ndarray:
    if (N, s) not in _ZIPF_CDF:
        w = np.arange(1, N + 1, dtype=np.float64) ** (-s)
        c = np.cumsum(w)
        _ZIPF_CDF[(N, s)] = c / c[-1]
    return _ZIPF_CDF[(N, s)]


def scatter_multiplier(N: int) -> int:
    """An odd multiplier near 0.618*N that is coprime to N: rank -> row = (rank*A + C) mod N."""
    a = int(N * 0.6180339887) | 1
    while math.gcd(a, N) != 1:
        a += 2
    return a


def row_ids(cfg: Config, key: np.uint64, n: int, table: np.ndarray) -> np.ndarray:
    """n row indices; `table` (the table each lookup belongs to) shifts the hot rows per table."""
    u = unit_f64(key, np.arange(n, dtype=np.uint64))
    if cfg.rows == "uniform":
        return np.minimum((u * cfg.N).astype(np.int64), cfg.N - 1).astype(np.int32)
    s = float(cfg.rows[4:])
    rank = np.minimum(np.searchsorted(_zipf_cdf(cfg.N, s), u, side="left"), cfg.N - 1).astype(np.int64)
    a = scatter_multiplier(cfg.N)
    return ((rank * a + 7919 * (table.astype(np.int64) + 1)) % cfg.N).astype(np.int32)


@dataclasses.dataclass
class Batch:
    indices: np.ndarray   # int32 [L]   row ids, bags of table 0 first, then table 1, ...
    offsets: np.ndarray   # int32 [T*B+1] CSR; bag id = t*B + b
    dense: np.ndarray     # float32 [B, n_dense]
    labels: np.ndarray    # float32 [B] in {0,1}

    @property
    def L(self) -> int:
        return int(self.indices.shape[0])


def make_batch(cfg: Config, replica: int, step: int) -> Batch:
    nb = cfg.T * cfg.B
    lens = bag_lengths(cfg, stream_key(cfg.seed, stream_id(KIND_BAGLEN, replica, step)), nb)
    offsets = np.zeros(nb + 1, dtype=np.int64)
    np.cumsum(lens, out=offsets[1:])
    L = int(offsets[-1])
    tbl = np.repeat(np.arange(nb, dtype=np.int64) // cfg.B, lens)
    idx = row_ids(cfg, stream_key(cfg.seed, stream_id(KIND_ROW, replica, step)), L, tbl)
    nd = cfg.bottom[0]
    dense = normal_f32(stream_key(cfg.seed, stream_id(KIND_DENSE, replica, step)), cfg.B * nd).reshape(cfg.B, nd)
    ul = unit_f64(stream_key(cfg.seed, stream_id(KIND_LABEL, replica, step)), np.arange(cfg.B, dtype=np.uint64))
    labels = (ul < cfg.ctr).astype(np.float32)
    return Batch(idx, offsets.astype(np.int32), dense, labels)


def sync_vectors(n: int, R: int, seed: int = MASTER_SEED, std: float = 0.02) -> List[np.ndarray]:
    """R replica vectors of n float32 ~ N(0, std^2) for the isolated sync-kernel sweep."""
    return [normal_f32(stream_key(seed, stream_id(KIND_VEC, r)), n, std) for r in range(R)]
