"""Seeded synthetic ID streams shaped like the workloads of the Monolith paper.

This module only *draws inputs* (feature IDs, bag offsets, pooled gradients).
It holds none of the table's arithmetic: no hashing into buckets, no counting,
no pooling, no optimizer.  Both the CPU oracle's tests and the CUDA path's
tests read the arrays it returns, so the two sides see identical inputs.

Shape of the inputs (Section 2.1 of the paper, observations 1 and 2):
IDs are long-tail distributed (popular IDs occur orders of magnitude more often
than unpopular ones), come from a huge sparse space (2^48 in Section 3.1), and
new IDs keep arriving while old ones go stale.  The paper's own datasets
(MovieLens, Criteo, the internal one) are not reproduced; bounded Zipf ranks
mixed into random 64-bit patterns stand in for them.

A *bag* is one (example, feature slot) pair.  A step's IDs are laid out CSR
style: bag b owns ids[offsets[b]:offsets[b+1]].
"""
from __future__ import annotations

import dataclasses
from typing import Iterator, Optional

import numpy as np

_MASK64 = np.uint64(0xFFFFFFFFFFFFFFFF)
RESERVED_ID = 0xFFFFFFFFFFFFFFFF


def splitmix64(x: np.ndarray) -> np.ndarray:
    """SplitMix64 output function (Steele, Lea, Flood 2014) applied element-wise.

    Used only to turn Zipf ranks into well-spread 64-bit IDs; any bijection on
    64-bit words would do because both sides read the same arrays.
    """
    with np.errstate(over="ignore"):
        z = (np.asarray(x, dtype=np.uint64) + np.uint64(0x9E3779B97F4A7C15)) & _MASK64
        z = ((z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)) & _MASK64
        z = ((z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)) & _MASK64
        return z ^ (z >> np.uint64(31))


class BoundedZipf:
    """Exact sampler for P(r) proportional to r^-s on r in [1, V], any s > 0.

    Rejection-inversion (Hoermann and Derflinger, 1996): invert the integral of
    the hat x^-s over [0.5, V+0.5], round to the nearest integer and accept
    with the ratio of the true mass to the hat.  Acceptance is above 90 %, so
    the vectorised loop below finishes in two or three rounds.
    """

    def __init__(self, n_values: int, s: float):
        if n_values < 1 or s <= 0:
            raise ValueError("need n_values >= 1 and s > 0")
        self.n = int(n_values)
        self.s = float(s)
        self._h_x1 = self._H(1.5) - 1.0
        self._h_n = self._H(self.n + 0.5)
        self._cut = 2.0 - self._Hinv(self._H(2.5) - 2.0 ** (-self.s))

    def _H(self, x):
        x = np.asarray(x, dtype=np.float64)
        lx = np.log(x)
        t = (1.0 - self.s) * lx
        # (exp(t)-1)/t * log(x), stable near t = 0 (s = 1)
        small = np.abs(t) < 1e-8
        safe_t = np.where(small, 1.0, t)
        return np.where(small, 1.0 + t / 2.0, np.expm1(safe_t) / safe_t) * lx

    def _Hinv(self, y):
        y = np.asarray(y, dtype=np.float64)
        t = np.maximum(y * (1.0 - self.s), -1.0)
        small = np.abs(t) < 1e-8
        safe_t = np.where(small, 1.0, t)
        return np.exp(np.where(small, 1.0 - t / 2.0, np.log1p(safe_t) / safe_t) * y)

    def sample(self, rng: np.random.Generator, size: int) -> np.ndarray:
        out = np.empty(size, dtype=np.int64)
        todo = np.arange(size)
        while todo.size:
            u = self._h_n + rng.random(todo.size) * (self._h_x1 - self._h_n)
            x = self._Hinv(u)
            k = np.clip(np.floor(x + 0.5), 1, self.n)
            ok = (k - x <= self._cut) | (u >= self._H(k + 0.5) - np.exp(-self.s * np.log(k)))
            out[todo[ok]] = k[ok].astype(np.int64)
            todo = todo[~ok]
        return out


@dataclasses.dataclass(frozen=True)
class Config:
    """One workload configuration: the table's parameters and the stream's shape."""

    name: str
    capacity: int            # embedding rows
    dim: int                 # fp32 columns per row
    filter_threshold: int    # occurrences before an ID is admitted
    ttl: int                 # steps of inactivity after which an ID expires
    n_examples: int
    n_slots: int
    bag_len: tuple           # ("uniform", lo, hi) or ("geometric", mean, lo, hi)
    zipf_s: float
    n_distinct: int          # size of the ID universe (Zipf support)
    steps: int
    key_cells: int           # cells of the key store (tracked-ID capacity incl. slack)
    lr: float = 0.05
    eps: float = 1e-8
    init_acc: float = 0.0
    init_scale: float = 0.01
    grad_std: float = 0.01
    drift_period: int = 0    # steps between re-keyings of part of the universe; 0 = none
    drift_new_frac: float = 0.0
    seed: int = 20220923

    @property
    def n_bags(self) -> int:
        return self.n_examples * self.n_slots


CONFIGS = {
    "tiny": Config("tiny", capacity=1 << 17, dim=16, filter_threshold=2, ttl=10,
                   n_examples=1024, n_slots=8, bag_len=("uniform", 1, 4),
                   zipf_s=1.1, n_distinct=1 << 20, steps=20, key_cells=1 << 18),
    "medium": Config("medium", capacity=1 << 22, dim=32, filter_threshold=3, ttl=100,
                     n_examples=8192, n_slots=26, bag_len=("uniform", 1, 8),
                     zipf_s=1.05, n_distinct=1 << 24, steps=200, key_cells=1 << 24),
    "large": Config("large", capacity=1 << 26, dim=64, filter_threshold=5, ttl=1000,
                    n_examples=16384, n_slots=100, bag_len=("geometric", 5.0, 1, 20),
                    zipf_s=1.05, n_distinct=1 << 30, steps=100, key_cells=1 << 30),
    # the batch mix of `large` (half the examples) on a 3 GB table with the same row and key loads:
    # the case profiler captures that replay every kernel many times are taken on
    "large_profile": Config("large_profile", capacity=1 << 22, dim=64, filter_threshold=5, ttl=100,
                            n_examples=8192, n_slots=100, bag_len=("geometric", 5.0, 1, 20),
                            zipf_s=1.05, n_distinct=1 << 26, steps=100, key_cells=1 << 26),
    "drift": Config("drift", capacity=1 << 26, dim=32, filter_threshold=3, ttl=200,
                    n_examples=16384, n_slots=50, bag_len=("geometric", 5.0, 1, 20),
                    zipf_s=1.2, n_distinct=1 << 30, steps=400, key_cells=1 << 29,
                    drift_period=50, drift_new_frac=0.30),
    # the same stream on a table sized for it: the drift stream keeps about 5.4e6 rows and 2.9e7 tracked IDs
    # alive within its TTL, so this row store and key store run at load 0.85-0.9, where cuckoo
    # insertions displace other keys (on the 2^26-row table above they never have to)
    "drift_dense": Config("drift_dense", capacity=5_900_000, dim=32, filter_threshold=3, ttl=200,
                          n_examples=16384, n_slots=50, bag_len=("geometric", 5.0, 1, 20),
                          zipf_s=1.2, n_distinct=1 << 30, steps=400, key_cells=1 << 25,
                          drift_period=50, drift_new_frac=0.30),
}

# Mixed-dim multi-table configuration: 8 tables, 120 feature slots spread over them so that
# every table settles near (and below) 0.9 row load under its own Zipf exponent.
MULTI_TABLE_DIMS = (8, 16, 16, 32, 32, 64, 64, 128)
MULTI_TABLE_CAPACITY_LOG2 = (27, 26, 25, 24, 23, 22, 21, 20)
MULTI_TABLE_ZIPF_S = (0.9, 0.95, 1.0, 1.05, 1.1, 1.2, 1.25, 1.3)
MULTI_TABLE_SLOTS = (33, 22, 16, 12, 9, 12, 9, 7)
MULTI_TABLE_UNIVERSE_LOG2_EXTRA = (2, 2, 2, 2, 2, 2, 1, 1)


def multi_table_configs(n_examples: int = 32768, slots=MULTI_TABLE_SLOTS) -> list:
    """Eight Config objects, one per table of the mixed-dim configuration.
    `slots` is the number of feature slots per table (an int gives every table the same)."""
    if isinstance(slots, int):
        slots = (slots,) * 8
    out = []
    for t, (d, cl, s, sl, ex) in enumerate(zip(MULTI_TABLE_DIMS, MULTI_TABLE_CAPACITY_LOG2, MULTI_TABLE_ZIPF_S,
                                               slots, MULTI_TABLE_UNIVERSE_LOG2_EXTRA)):
        out.append(Config(f"multi{t}", capacity=1 << cl, dim=d, filter_threshold=3, ttl=500,
                          n_examples=n_examples, n_slots=sl,
                          bag_len=("uniform", 1, 8), zipf_s=s, n_distinct=1 << min(cl + ex, 30),
                          steps=50, key_cells=1 << min(cl + 2, 30), seed=20220923 + 101 * t))
    return out


def many_small_table_configs(n_tables: int = 64, n_examples: int = 4096) -> list:
    """The other end of Section 3.1's "many tables of very uneven size": `n_tables` small tables
    (2^17 rows, two feature slots each, dims cycling through 8, 16, 32, 64), each far too small to
    fill a GPU on its own -- the case grouped launches are for."""
    dims = (8, 16, 32, 64)
    return [Config(f"small{t}", capacity=1 << 17, dim=dims[t % 4], filter_threshold=2, ttl=50,
                   n_examples=n_examples, n_slots=2, bag_len=("uniform", 1, 4), zipf_s=1.0 + 0.05 * (t % 5),
                   n_distinct=1 << 18, steps=50, key_cells=1 << 19, seed=20220923 + 977 * t)
            for t in range(n_tables)]


def expected_steady_state(cfg: Config, window: Optional[int] = None):
    """Expected (tracked IDs, IDs with a row) after `window` steps of cfg's stream under the
    Poisson model of steady_state_population (ranks binned geometrically beyond the head)."""
    from math import lgamma
    window = cfg.ttl if window is None else window
    v = cfg.n_distinct
    head = np.arange(1, min(v, 2_000_000) + 1, dtype=np.float64)
    k, w = head, np.ones_like(head)
    if v > 2_000_000:
        e = np.unique(np.floor(np.geomspace(2_000_000, v, 200_000)).astype(np.int64))
        lo, hi = e[:-1] + 1, e[1:]
        k, w = np.concatenate([head, (lo + hi) / 2.0]), np.concatenate([w, (hi - lo + 1).astype(np.float64)])
    p = k ** (-cfg.zipf_s)
    p /= (p * w).sum()
    lam = cfg.n_bags * _mean_bag_len(cfg.bag_len) * window * p
    cdf = np.zeros_like(lam)
    for j in range(max(cfg.filter_threshold, 1)):
        cdf += np.exp(-lam + j * np.log(np.maximum(lam, 1e-300)) - lgamma(j + 1))
    return float((w * -np.expm1(-lam)).sum()), float((w * (1.0 - np.minimum(cdf, 1.0))).sum())


def scaled(cfg: Config, **kw) -> Config:
    """A copy of cfg with some fields replaced (shortened or shrunk test variants)."""
    return dataclasses.replace(cfg, **kw)


@dataclasses.dataclass
class Step:
    ids: np.ndarray          # uint64 [n_ids]
    offsets: np.ndarray      # int64 [n_bags + 1], offsets[0] = 0, offsets[-1] = n_ids
    grad_pooled: np.ndarray  # float32 [n_bags, dim]
    now: int


def _bag_lengths(rng: np.random.Generator, spec: tuple, n_bags: int) -> np.ndarray:
    kind = spec[0]
    if kind == "uniform":
        _, lo, hi = spec
        return rng.integers(lo, hi + 1, size=n_bags, dtype=np.int64)
    if kind == "geometric":
        _, mean, lo, hi = spec
        return np.clip(rng.geometric(1.0 / mean, size=n_bags), lo, hi).astype(np.int64)
    raise ValueError(f"unknown bag length spec {spec!r}")


class Stream:
    """Deterministic per-step generator for one Config.

    step(t) depends only on (cfg.seed, t), so any step can be regenerated on
    its own and both sides of a parity test can draw the same step twice.
    """

    def __init__(self, cfg: Config):
        self.cfg = cfg
        self._zipf = BoundedZipf(cfg.n_distinct, cfg.zipf_s)

    def _generation(self, ranks: np.ndarray, t: int) -> np.ndarray:
        """How many times each rank has been re-keyed up to step t (concept drift).

        At every drift_period boundary a rank draws a fresh identity with a
        probability that grows with its popularity so that about
        drift_new_frac of the next batch's occurrences are IDs never seen
        before; the draw is a pure function of (seed, rank, epoch).
        """
        cfg = self.cfg
        gen = np.zeros(ranks.shape, dtype=np.uint64)
        if cfg.drift_period <= 0:
            return gen
        n_epochs = t // cfg.drift_period
        thresh = np.uint64(int(cfg.drift_new_frac * float(1 << 53)))
        for e in range(1, n_epochs + 1):
            h = splitmix64(ranks.astype(np.uint64) * np.uint64(0x2545F4914F6CDD1D)
                           + np.uint64((cfg.seed * 1000003 + e) & 0xFFFFFFFFFFFFFFFF))
            gen += ((h >> np.uint64(11)) < thresh).astype(np.uint64)
        return gen

    def ids_from_ranks(self, ranks: np.ndarray, t: int) -> np.ndarray:
        cfg = self.cfg
        gen = self._generation(ranks, t)
        with np.errstate(over="ignore"):
            salt = splitmix64(np.uint64(cfg.seed & 0xFFFFFFFFFFFFFFFF) + gen * np.uint64(0x632BE59BD9B4E019))
            ids = splitmix64(ranks.astype(np.uint64) ^ salt)
        # the all-ones pattern is the table's reserved padding value
        ids[ids == np.uint64(RESERVED_ID)] = np.uint64(RESERVED_ID - 1)
        return ids

    def step(self, t: int, with_grad: bool = True) -> Step:
        cfg = self.cfg
        rng = np.random.default_rng([cfg.seed, t])
        lens = _bag_lengths(rng, cfg.bag_len, cfg.n_bags)
        offsets = np.zeros(cfg.n_bags + 1, dtype=np.int64)
        np.cumsum(lens, out=offsets[1:])
        ranks = self._zipf.sample(rng, int(offsets[-1]))
        ids = self.ids_from_ranks(ranks, t)
        if with_grad:
            grad = rng.standard_normal((cfg.n_bags, cfg.dim), dtype=np.float32) * np.float32(cfg.grad_std)
        else:
            grad = np.zeros((0, cfg.dim), dtype=np.float32)
        return Step(ids=ids, offsets=offsets, grad_pooled=grad, now=t)

    def __iter__(self) -> Iterator[Step]:
        for t in range(self.cfg.steps):
            yield self.step(t)


def steady_state_population(cfg: Config, now: int, window: Optional[int] = None,
                            seed_salt: int = 7, max_ranks: Optional[int] = None):
    """Draw a table population as it would stand after `window` steps of cfg's stream.

    Used to pre-fill a table before timing, so that timed steps run at a
    realistic load instead of on an empty table.  Under the Poisson model of
    the stream, rank k occurs Poisson(lambda_k) times per window with
    lambda_k = (IDs per step) * window * p_k.  For each rank that occurred at
    least once this returns its ID, its occurrence count (not yet saturated)
    and a last-seen step drawn so that hot ranks were seen at `now`.

    Returns (ids uint64, counts int64, last_seen int64).
    """
    window = int(window if window is not None else min(cfg.ttl, now + 1))
    rng = np.random.default_rng([cfg.seed, seed_salt, now])
    mean_len = _mean_bag_len(cfg.bag_len)
    n_per_step = cfg.n_bags * mean_len
    n_ranks = cfg.n_distinct if max_ranks is None else min(cfg.n_distinct, max_ranks)
    stream = Stream(cfg)
    norm = _zipf_norm(cfg.n_distinct, cfg.zipf_s)
    ids_l, cnt_l, seen_l = [], [], []
    chunk = 1 << 24
    for lo in range(1, n_ranks + 1, chunk):
        hi = min(lo + chunk, n_ranks + 1)
        ranks = np.arange(lo, hi, dtype=np.int64)
        p = ranks.astype(np.float64) ** (-cfg.zipf_s) / norm
        lam_step = n_per_step * p
        cnt = rng.poisson(lam_step * window)
        keep = cnt > 0
        ranks, cnt, lam_step = ranks[keep], cnt[keep], lam_step[keep]
        # steps since the most recent occurrence: geometric with the per-step hit
        # probability, conditioned on falling inside the window
        age = _truncated_geometric(rng.random(ranks.size), -np.expm1(-lam_step), window)
        ids_l.append(stream.ids_from_ranks(ranks, now))
        cnt_l.append(cnt.astype(np.int64))
        seen_l.append((now - age).astype(np.int64))
    return np.concatenate(ids_l), np.concatenate(cnt_l), np.concatenate(seen_l)


def _truncated_geometric(u, p_hit, window: int):
    """Inverse CDF of P(a) ~ (1-p)^a p on a in [0, window): uniform for tiny p."""
    p_hit = np.clip(p_hit, 1e-12, 1 - 1e-12)
    log_q = np.log1p(-p_hit)
    mass = -np.expm1(window * log_q)                  # 1 - q^window
    a = np.floor(np.log1p(-u * mass) / log_q)
    return np.clip(a, 0, window - 1).astype(np.int64)


def _mean_bag_len(spec: tuple) -> float:
    if spec[0] == "uniform":
        return (spec[1] + spec[2]) / 2.0
    _, mean, lo, hi = spec
    q = 1.0 - 1.0 / mean
    ks = np.arange(1, 2000)
    pk = (1 - q) * q ** (ks - 1)
    return float(np.sum(np.clip(ks, lo, hi) * pk))


def _zipf_norm(n: int, s: float) -> float:
    head = min(n, 1 << 20)
    k = np.arange(1, head + 1, dtype=np.float64)
    total = float(np.sum(k ** (-s)))
    if n > head:
        a, b = head + 0.5, n + 0.5
        total += (np.log(b / a) if abs(s - 1.0) < 1e-12 else (b ** (1 - s) - a ** (1 - s)) / (1 - s))
    return total


# ---------------------------------------------------------------------------
# Device-side twins of the generators above (torch), for benchmarks that need a
# table population of hundreds of millions of IDs without a slow host loop.
# They reproduce the numpy functions bit for bit (checked in the CPU tests).
# ---------------------------------------------------------------------------

def _signed64(c: int) -> int:
    c &= 0xFFFFFFFFFFFFFFFF
    return c - (1 << 64) if c >= (1 << 63) else c


def _lsr(x, k: int):
    """Logical shift right of an int64 tensor."""
    return (x >> k) & ((1 << (64 - k)) - 1)


def splitmix64_torch(x):
    """splitmix64() on an int64 torch tensor holding uint64 bit patterns."""
    z = x + _signed64(0x9E3779B97F4A7C15)
    z = (z ^ _lsr(z, 30)) * _signed64(0xBF58476D1CE4E5B9)
    z = (z ^ _lsr(z, 27)) * _signed64(0x94D049BB133111EB)
    return z ^ _lsr(z, 31)


def ids_from_ranks_torch(cfg: Config, ranks):
    """Stream.ids_from_ranks for a config without drift, on an int64 tensor of ranks."""
    import torch
    if cfg.drift_period > 0:
        raise ValueError("the device twin covers configs without drift")
    salt = int(splitmix64(np.array([cfg.seed & 0xFFFFFFFFFFFFFFFF], dtype=np.uint64))[0])
    ids = splitmix64_torch(ranks ^ _signed64(salt))
    return torch.where(ids == -1, torch.full_like(ids, -2), ids)


def steady_state_population_torch(cfg: Config, now: int, device, window: Optional[int] = None,
                                  chunk: int = 1 << 26, seed_salt: int = 7):
    """Device twin of steady_state_population: yields (ids int64, counts int32,
    last_seen int64) chunk by chunk, each a torch tensor on `device`.
    Same model (Poisson occurrences per rank over the window); its own random
    stream (torch's), so it is reproducible for a given seed but does not match
    the numpy draw element by element.
    """
    import torch
    window = int(window if window is not None else min(cfg.ttl, now + 1))
    gen = torch.Generator(device=device)
    gen.manual_seed((cfg.seed * 1000003 + seed_salt * 7919 + now) & 0x7FFFFFFFFFFFFFFF)
    n_per_step = cfg.n_bags * _mean_bag_len(cfg.bag_len)
    norm = _zipf_norm(cfg.n_distinct, cfg.zipf_s)
    for lo in range(1, cfg.n_distinct + 1, chunk):
        hi = min(lo + chunk, cfg.n_distinct + 1)
        ranks = torch.arange(lo, hi, dtype=torch.int64, device=device)
        lam_step = ranks.to(torch.float64).pow(-cfg.zipf_s).mul_(n_per_step / norm)
        cnt = torch.poisson((lam_step * window).to(torch.float32), generator=gen)
        keep = cnt > 0
        ranks, cnt, lam_step = ranks[keep], cnt[keep], lam_step[keep]
        # steps since the last occurrence: geometric, conditioned on lying inside the window
        p_hit = (-torch.expm1(-lam_step)).clamp_(1e-12, 1 - 1e-12)
        u = torch.rand(ranks.shape, dtype=torch.float64, device=device, generator=gen)
        log_q = torch.log1p(-p_hit)
        mass = -torch.expm1(window * log_q)
        age = torch.floor(torch.log1p(-u * mass) / log_q).clamp_(0, window - 1)
        yield ids_from_ranks_torch(cfg, ranks), cnt.to(torch.int32), (now - age).to(torch.int64)
