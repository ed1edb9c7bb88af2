"""Pins for the oracle's subnet generator (Algorithm 1, Sec. 3.1) against what the paper
and the mathematics fix: post-conditions, the feasibility bound, special cases, and the
uniformity of the random heuristic.  CPU only."""
import itertools
import os

import numpy as np
import pytest

from oracle import twist_oracle as o

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def test_mixer_matches_published_splitmix64_vectors():
    want = [int(l, 16) for l in open(os.path.join(GOLDEN, "splitmix64_vectors.txt")) if l.startswith("0x")]
    state, got = 0, []
    for _ in want:
        state = (state + 0x9E3779B97F4A7C15) % 2 ** 64
        got.append(int(o.mix64(np.uint64(state))))
    assert got == want


def test_keys_are_distinct_and_carry_the_block_index():
    k = o.block_keys(5, 3, 2, 1, o.STREAM_FILL, 4, 11008)
    assert len(np.unique(k)) == 11008
    assert np.array_equal(k & np.uint64(0xFFFF), np.arange(11008, dtype=np.uint64))
    # different counters give different streams
    k2 = o.block_keys(5, 3, 2, 1, o.STREAM_FILL, 5, 11008)
    assert np.mean((k >> np.uint64(16)) == (k2 >> np.uint64(16))) < 1e-3


def _check_postconditions(A, n_full, S, n_sub, common, cover_required):
    assert A.shape == (S, n_sub) and A.dtype == np.int32
    for s in range(S):
        row = A[s]
        assert np.all(np.diff(row) > 0), "rows sorted, entries unique"        # sorted + unique
        assert row.min() >= 0 and row.max() < n_full
        assert set(common) <= set(row.tolist()), "every subnet contains C"      # (i)
    if cover_required:
        assert set(A.reshape(-1).tolist()) == set(range(n_full)), "every block assigned"   # (ii)


@pytest.mark.parametrize("n_full,S,n_sub,common", [
    (12, 4, 4, []), (12, 4, 6, []), (12, 4, 12, []), (12, 3, 6, [0, 7]), (256, 2, 128, []),
    (3072, 4, 1536, []), (32, 4, 16, []), (32, 8, 8, []), (11008, 8, 2752, []), (100, 7, 16, [3]),
    (5632, 4, 2816, []), (12, 1, 12, []), (13, 5, 3, []),
])
def test_cover_mode_postconditions(n_full, S, n_sub, common):
    for rnd in range(3):
        A = o.sample_blueprint(n_full, S, n_sub, common, seed=11, rnd=rnd, layer=1, kind=0)
        _check_postconditions(A, n_full, S, n_sub, common, cover_required=True)


def test_feasibility_bound_is_the_papers_inequality():
    # (N_full + (S-1)|C|)/S <= N_sub <= N_full  <=>  feasible, for every small case
    for n_full, S, c in itertools.product(range(1, 10), range(1, 5), range(0, 4)):
        if c > n_full:
            continue
        for n_sub in range(0, n_full + 2):
            want = (n_full + (S - 1) * c) / S <= n_sub <= n_full
            assert o.feasible(n_full, S, n_sub, c) == want, (n_full, S, c, n_sub)


def test_infeasible_raises_and_iid_accepts():
    with pytest.raises(ValueError):
        o.sample_blueprint(11008, 2, 2752, [], 1, 0, 0, 0)           # 2*2752 < 11008
    A = o.sample_blueprint(11008, 2, 2752, [], 1, 0, 0, 0, mode=o.MODE_IID)
    _check_postconditions(A, 11008, 2, 2752, [], cover_required=False)
    with pytest.raises(ValueError):
        o.sample_blueprint(8, 2, 9, [], 1, 0, 0, 0, mode=o.MODE_IID)


def test_exact_partition_when_nfull_equals_s_times_nsub():
    # N_full = S * N_sub leaves no room for the fill step: rows partition the blocks.
    for seed in range(20):
        A = o.sample_blueprint(256, 2, 128, [], seed, 0, 0, 0)
        _, count, _ = o.cover_and_pos(A, 256)
        assert np.all(count == 1)
        assert sorted(A.reshape(-1).tolist()) == list(range(256))


def test_bruteforce_tiny_inputs_valid_and_uniform():
    # N_full <= 8, S <= 3: every output valid; over many seeds each block is kept by
    # subnet s with frequency N_sub / N_full (by symmetry of the random heuristic, C empty).
    n_seeds = 4000
    for n_full, S, n_sub in [(6, 2, 3), (6, 2, 4), (8, 3, 3), (8, 3, 5), (5, 3, 2), (7, 2, 6)]:
        freq = np.zeros((S, n_full))
        for seed in range(n_seeds):
            A = o.sample_blueprint(n_full, S, n_sub, [], seed, 0, 0, 0)
            _check_postconditions(A, n_full, S, n_sub, [], cover_required=True)
            for s in range(S):
                freq[s, A[s]] += 1
        p = n_sub / n_full
        sigma = np.sqrt(p * (1 - p) / n_seeds)
        assert np.all(np.abs(freq / n_seeds - p) < 4.5 * sigma), (n_full, S, n_sub, freq / n_seeds)


def test_fill_step_is_uniform_over_the_complement():
    # With C = {0,1} common and N_full=8, S=2, N_sub=6: after the cover step each subnet holds
    # 2 + 3 blocks and draws exactly 1 more from the 3 it lacks, uniformly.
    n_seeds, hits = 6000, []
    extra = np.zeros(8)
    for seed in range(n_seeds):
        A = o.sample_blueprint(8, 2, 6, [0, 1], seed, 0, 0, 0)
        both = set(A[0].tolist()) & set(A[1].tolist())
        assert {0, 1} <= both
        for b in both - {0, 1}:
            extra[b] += 1
    # non-common blocks are shared between both subnets equally often
    e = extra[2:] / n_seeds
    assert np.all(np.abs(e - e.mean()) < 0.03), e


def test_iid_rows_are_independent_uniform_subsets():
    n_full, n_sub, n_seeds = 10, 4, 6000
    inc = np.zeros(n_full)
    both = 0
    for seed in range(n_seeds):
        A = o.sample_blueprint(n_full, 2, n_sub, [], seed, 0, 0, 0, mode=o.MODE_IID)
        inc[A[0]] += 1
        both += len(set(A[0].tolist()) & set(A[1].tolist()))
    p = n_sub / n_full
    assert np.all(np.abs(inc / n_seeds - p) < 4.5 * np.sqrt(p * (1 - p) / n_seeds))
    # E|A0 & A1| = N_sub^2 / N_full for independent uniform subsets
    assert abs(both / n_seeds - n_sub * n_sub / n_full) < 0.06


def test_order_is_lexicographic_hash_then_index():
    # the composite key order equals sorting by (48-bit hash, block index)
    k = o.block_keys(9, 1, 0, 0, o.STREAM_PERM, 0, 500)
    by_tuple = sorted(range(500), key=lambda b: (int(k[b]) >> 16, b))
    assert by_tuple == np.argsort(k, kind="stable").tolist()


def test_round_layer_kind_change_the_blueprint():
    base = o.sample_blueprint(3072, 4, 1536, [], 3, 0, 0, 0)
    for kw in [dict(rnd=1, layer=0, kind=0), dict(rnd=0, layer=1, kind=0), dict(rnd=0, layer=0, kind=1)]:
        other = o.sample_blueprint(3072, 4, 1536, [], 3, **kw)
        assert not np.array_equal(base, other)
    assert np.array_equal(base, o.sample_blueprint(3072, 4, 1536, [], 3, 0, 0, 0))   # deterministic


def test_coverage_counts_match_masks():
    A = o.sample_blueprint(11008, 8, 2752, [], 3004, 2, 5, 0)
    cover, count, pos = o.cover_and_pos(A, 11008)
    naive = np.zeros(11008, dtype=np.int64)
    for s in range(8):
        for b in A[s]:
            naive[b] += 1
    assert np.array_equal(naive, count)
    assert count.min() >= 1 and count.sum() == 8 * 2752
    for s in range(8):
        held = np.flatnonzero(pos[s] >= 0)
        assert np.array_equal(held, A[s])
        assert np.array_equal(pos[s, A[s]], np.arange(2752))
        assert np.array_equal(((cover >> np.uint32(s)) & np.uint32(1)).astype(bool), pos[s] >= 0)


def test_kv_groups_follow_their_query_heads():
    head_idx = np.array([[0, 1, 9, 31], [8, 9, 10, 11]], dtype=np.int32)
    kv_idx, kv_count = o.kv_groups(head_idx, 32, 4)
    assert kv_count.tolist() == [3, 1]
    assert kv_idx[0].tolist() == [0, 1, 3, -1] and kv_idx[1].tolist() == [1, -1, -1, -1]
    # plain multi-head: groups are the heads themselves
    kv_idx, kv_count = o.kv_groups(head_idx, 32, 32)
    assert np.array_equal(kv_idx[:, :4], head_idx) and kv_count.tolist() == [4, 4]


def test_blueprint_regression_file():
    path = os.path.join(GOLDEN, "blueprint_regression.txt")
    for line in open(path):
        if line.startswith("#") or not line.strip():
            continue
        head, vals = line.split(":")
        n_full, S, n_sub, seed, rnd, layer, kind, mode = (int(v) for v in head.split())
        A = o.sample_blueprint(n_full, S, n_sub, [], seed, rnd, layer, kind, mode)
        assert A.reshape(-1).tolist() == [int(v) for v in vals.split()]
