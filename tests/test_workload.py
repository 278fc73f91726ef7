"""The seeded input generator: distributions, shapes and reproducibility."""
import numpy as np
import pytest

from paper_2209_07663_b200 import workload as wl


@pytest.mark.parametrize("s", [0.9, 1.0, 1.05, 1.3])
def test_bounded_zipf_matches_exact_pmf(s):
    V = 200
    z = wl.BoundedZipf(V, s)
    x = z.sample(np.random.default_rng(1), 400_000)
    assert x.min() >= 1 and x.max() <= V
    emp = np.bincount(x, minlength=V + 1)[1:] / x.size
    p = np.arange(1, V + 1.0) ** -s
    p /= p.sum()
    assert np.abs(emp - p).max() < 4e-3
    assert abs(emp[:10].sum() - p[:10].sum()) < 4e-3


def test_zipf_huge_support_head_mass():
    z = wl.BoundedZipf(1 << 30, 1.05)
    x = z.sample(np.random.default_rng(2), 300_000)
    assert x.max() <= 1 << 30
    # rank 1 carries about 7.4 % of the mass at s = 1.05 over 2^30 values
    assert abs((x == 1).mean() - 1.0 / wl._zipf_norm(1 << 30, 1.05)) < 3e-3


def test_splitmix64_reference_values():
    # first outputs of SplitMix64 seeded with 0 (Steele, Lea, Flood 2014; the values
    # printed by the reference generator's test program): state advances by the golden gamma
    gamma = 0x9E3779B97F4A7C15
    states = np.array([(k * gamma) & 0xFFFFFFFFFFFFFFFF for k in range(3)], dtype=np.uint64)
    got = wl.splitmix64(states).tolist()
    assert got == [0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4, 0x06C45D188009454F]


@pytest.mark.parametrize("name", ["tiny", "medium"])
def test_step_shapes_and_determinism(name):
    cfg = wl.CONFIGS[name]
    st = wl.Stream(cfg)
    a, b = st.step(3), st.step(3)
    assert (a.ids == b.ids).all() and (a.offsets == b.offsets).all() and (a.grad_pooled == b.grad_pooled).all()
    assert a.offsets.shape == (cfg.n_bags + 1,) and a.offsets[0] == 0 and a.offsets[-1] == a.ids.size
    lens = np.diff(a.offsets)
    assert lens.min() >= cfg.bag_len[1] and lens.max() <= cfg.bag_len[2]
    assert a.grad_pooled.shape == (cfg.n_bags, cfg.dim) and a.grad_pooled.dtype == np.float32
    assert abs(a.grad_pooled.std() - cfg.grad_std) < 0.1 * cfg.grad_std
    assert (a.ids != wl.RESERVED_ID).all()
    c = st.step(4)
    assert not np.array_equal(a.ids[:100], c.ids[:100])
    # long tail: the most frequent ID owns several percent, most IDs occur once
    _, counts = np.unique(a.ids, return_counts=True)
    assert counts.max() / a.ids.size > 0.04 and (counts == 1).mean() > 0.5


def test_geometric_bag_lengths_of_the_large_shape():
    rng = np.random.default_rng(0)
    lens = wl._bag_lengths(rng, ("geometric", 5.0, 1, 20), 200_000)
    assert lens.min() == 1 and lens.max() == 20
    assert abs(lens.mean() - wl._mean_bag_len(("geometric", 5.0, 1, 20))) < 0.05
    assert 4.5 < lens.mean() < 5.0


def test_drift_rekeys_about_the_requested_share():
    cfg = wl.scaled(wl.CONFIGS["drift"], n_examples=2048, n_slots=10, n_distinct=1 << 20)
    st = wl.Stream(cfg)
    before = st.step(cfg.drift_period - 1)
    after = st.step(cfg.drift_period)
    seen = set(before.ids.tolist())
    new_frac_same_epoch = np.mean([i not in seen for i in st.step(cfg.drift_period - 2).ids.tolist()])
    new_frac_next_epoch = np.mean([i not in seen for i in after.ids.tolist()])
    # crossing the boundary adds about drift_new_frac of never-seen occurrences
    assert 0.15 < new_frac_next_epoch - new_frac_same_epoch < 0.45


def test_steady_state_population_is_consistent():
    cfg = wl.scaled(wl.CONFIGS["medium"], n_distinct=1 << 16)
    ids, cnt, seen = wl.steady_state_population(cfg, now=99)
    assert len(np.unique(ids)) == ids.size
    assert cnt.min() >= 1 and seen.max() <= 99 and seen.min() >= 0
    # hot ranks were seen in the very last step
    assert seen[0] == 99 and cnt[0] > cnt[-1]
    # cold IDs are spread over the whole window instead of piling up at its far end
    sparse = wl.scaled(cfg, n_examples=8, n_slots=4)
    _, cnt, seen = wl.steady_state_population(sparse, now=99)
    cold = seen[cnt == 1]
    assert cold.size > 1000
    assert (cold == 0).mean() < 0.05 and abs(cold.mean() - 49.5) < 5


def test_torch_twins_reproduce_the_numpy_generators():
    import torch
    x = np.array([0, 1, 2**63, 2**64 - 1, 0x9E3779B97F4A7C15, 123456789], dtype=np.uint64)
    got = wl.splitmix64_torch(torch.from_numpy(x.view(np.int64))).numpy().view(np.uint64)
    assert (got == wl.splitmix64(x)).all()
    cfg = wl.CONFIGS["medium"]
    ranks = np.array([1, 2, 3, 1000, 2**24], dtype=np.int64)
    want = wl.Stream(cfg).ids_from_ranks(ranks, 5)
    got = wl.ids_from_ranks_torch(cfg, torch.from_numpy(ranks)).numpy().view(np.uint64)
    assert (got == want).all()
    small = wl.scaled(cfg, n_distinct=1 << 14)
    chunks = list(wl.steady_state_population_torch(small, now=99, device="cpu", chunk=1 << 12))
    ids = torch.cat([c[0] for c in chunks]).numpy()
    cnt = torch.cat([c[1] for c in chunks]).numpy()
    seen = torch.cat([c[2] for c in chunks]).numpy()
    assert len(np.unique(ids)) == ids.size and cnt.min() >= 1
    assert seen.max() == 99 and seen.min() >= 0 and seen[0] == 99
    ref_ids, ref_cnt, _ = wl.steady_state_population(small, now=99)
    assert abs(ids.size - ref_ids.size) < 0.05 * ref_ids.size          # same model, different draws
    assert abs(int(cnt.sum()) - int(ref_cnt.sum())) < 0.05 * ref_cnt.sum()


def test_configured_streams_fit_their_tables():
    # steady state of every configured stream under the Poisson model: rows and keys fit
    for cfg in [wl.CONFIGS["tiny"], wl.CONFIGS["medium"], wl.CONFIGS["large"]] + wl.multi_table_configs():
        tracked, admitted = wl.expected_steady_state(cfg)
        assert admitted <= 0.93 * cfg.capacity, (cfg.name, admitted / cfg.capacity)
        assert tracked <= 0.80 * cfg.key_cells, (cfg.name, tracked / cfg.key_cells)
    assert sum(wl.MULTI_TABLE_SLOTS) == 120
    total = sum(c.capacity * c.dim * 8 + c.key_cells * 16 + c.capacity * 4 for c in wl.multi_table_configs())
    assert total < 120e9                                  # rows + accumulators + key stores + free lists
    t, a = wl.expected_steady_state(wl.CONFIGS["large"])
    assert 4.2e8 < t < 5.0e8 and 5.5e7 < a < 6.5e7        # the pre-fill the benchmark starts from
