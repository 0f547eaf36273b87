"""The seeded input generators: determinism, well-formed tables (oracle preconditions), mask
budgets, and the closed forms the synthetic masks are meant to reproduce (no GPU)."""
import numpy as np
import pytest

from oracle import vto
from harness import workloads as wl

SMALL = [
    lambda s: wl.tiny(seed=s),
    lambda s: wl.llama8b_h2o(seed=s, requests=6, lo=200, hi=800, layers=1, heads=1, head_dim=8),
    lambda s: wl.mistral7b_random(seed=s, requests=12, lo=100, hi=400, layers=1, heads=1, head_dim=8),
    lambda s: wl.longctx_scissor(seed=s, requests=3, lo=2000, hi=4000, layers=1, heads=1, head_dim=8),
    lambda s: wl.steady_state(seed=s, requests=16, lo=100, hi=1500, layers=1, heads=1, head_dim=8),
    lambda s: wl.streaming_window(seed=s, requests=6, lo=200, hi=900, window=64, layers=1, heads=1, head_dim=8),
]


@pytest.mark.parametrize("gen", SMALL, ids=[str(i) for i in range(len(SMALL))])
def test_generators_are_deterministic_and_well_formed(gen):
    a, b, c = gen(3), gen(3), gen(4)
    for f in ("bt_offsets", "bt_blocks", "tt_offsets", "tt_slots", "keep", "free_blocks"):
        assert np.array_equal(getattr(a, f), getattr(b, f))
    assert not np.array_equal(a.keep, c.keep) or a.name == "streaming_window"
    assert vto.validate(a.block_size, a.num_blocks, a.bt_offsets, a.bt_blocks, a.tt_offsets, a.tt_slots, a.keep,
                        a.free_blocks) == 0
    # the free list is large enough for every request the threshold lets through
    assert vto.plan_workload(a).num_deferred == 0
    assert sorted(a.free_blocks.tolist()) == a.free_blocks.tolist()


def test_h2o_mask_budget_sinks_and_recent_window():
    rng = np.random.default_rng(0)
    n = 1000
    score = rng.lognormal(0, 1.5, n)
    keep = wl.h2o_mask(np.arange(n), n, score, 200)
    assert keep.sum() == 200 and keep[:4].all() and keep[-64:].all()
    mid = np.arange(4, n - 64)
    kept_mid, dropped_mid = mid[keep[mid]], mid[~keep[mid]]
    assert score[kept_mid].min() >= score[dropped_mid].max()          # the heavy hitters
    # a budget below sinks + window keeps exactly those
    assert wl.h2o_mask(np.arange(n), n, score, 10).sum() == 68


def test_full_size_workloads_have_the_documented_sizes():
    for name, T, M in (("llama8b_h2o", 165772, 33180), ("mistral7b_random", 336030, 172149)):
        w = wl.CONFIGS[name](seed=0)
        s = wl.stats(w)
        assert s["logical_tokens"] == T and s["kept_tokens"] == M
        assert w.token_bytes == 131072 and w.row_bytes == 2048
    w = wl.CONFIGS["llama8b_h2o"](seed=0)
    assert abs(wl.stats(w)["keep_fraction_of_resident"] - 0.2) < 0.005


def test_random_mask_waste_ratio_tracks_one_minus_p():
    w = wl.mistral7b_random(seed=1, requests=64, lo=512, hi=2048, layers=1, heads=1, head_dim=8, rho_lo=0.5, rho_hi=0.5)
    F = wl.stats(w)["F_before"]
    assert abs(F - 0.5) < 0.02                                        # E[F] = 1 - p for i.i.d. keep probability p


def test_fill_is_roughly_standard_normal_bf16_and_slab_addressable():
    import torch
    x = wl.fill_slab(0, 0, 0, 2, 4096, 64)
    f = torch.from_numpy(x.view(np.int16)).view(torch.bfloat16).float()
    assert abs(float(f.mean())) < 0.01 and abs(float(f.std()) - 1.0) < 0.01
    # any row can be regenerated alone, and K, V and layers differ
    rows = wl.fill_rows(0, 0, 0, 2, 4096, 64, np.array([5, 4000]))
    assert np.array_equal(rows, x[[5, 4000]])
    assert not np.array_equal(wl.fill_slab(0, 1, 0, 2, 4096, 64), x)
    assert not np.array_equal(wl.fill_slab(0, 0, 1, 2, 4096, 64), x)
    assert not np.array_equal(wl.fill_slab(1, 0, 0, 2, 4096, 64), x)


def test_shared_prefix_layout():
    w, protect = wl.shared_prefix(seed=0, groups=2, degree=3, prefix_len=64, suffix_len=80, layers=1, heads=1,
                                  head_dim=8, block_size=16)
    assert w.num_requests == 6 and protect.sum() == 2 * 4
    first = [w.bt_blocks[w.bt_offsets[r]:w.bt_offsets[r] + 4].tolist() for r in range(6)]
    assert first[0] == first[1] == first[2] != first[3] == first[4] == first[5]
    own = [set(w.bt_blocks[w.bt_offsets[r] + 4:w.bt_offsets[r + 1]].tolist()) for r in range(6)]
    assert all(not (own[i] & own[j]) for i in range(6) for j in range(i))
