"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the
header declares, and its pure-host helpers agree bit for bit with the oracle."""
import itertools
import os
import re

import numpy as np
import pytest

import oracle
from paper_2602_15318_b200 import binding as B
from paper_2602_15318_b200 import build, workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    build.build()


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "sparrow_attn.h")).read()
    declared = set(re.findall(r"\b(sparrow_[a-z_]+)\s*\(", header))
    assert declared == set(B.EXPORTS)
    L = B.lib()
    for name in declared:
        assert hasattr(L, name), name


def test_timeline_build_compiles_and_exports_its_calls():
    """The stamped variant of the library (-DSPARROW_TIMELINE) still builds and carries the three
    extra calls the timeline tool uses, beside everything the header declares."""
    import ctypes
    from paper_2602_15318_b200 import timeline
    L = ctypes.CDLL(timeline.build_timeline_library())
    for name in list(B.EXPORTS) + ["sparrow_timeline_read", "sparrow_timeline_clear", "sparrow_timeline_mark"]:
        assert hasattr(L, name), name
    assert not hasattr(B.lib(), "sparrow_timeline_read")         # the shipped library has no stamps


def test_ancestor_masks_match_oracle_all_small_trees():
    for T in range(1, 7):
        for par in itertools.product(*[range(-1, i) for i in range(T)]):
            assert B.sparrow_build_ancestor_masks(list(par)) == [int(x) for x in oracle.ancestor_masks(np.array(par, np.int32))]
    for seed in range(20):
        par = W.random_tree_parents(seed, 4, 64)
        assert B.sparrow_build_ancestor_masks(par) == [int(x) for x in oracle.ancestor_masks(np.array(par, np.int32))]


def test_ancestor_masks_reject_bad_trees():
    for bad in ([0], [-1, 1], [-1, 2, 0], [-2]):
        with pytest.raises(B.SparrowError) as e:
            B.sparrow_build_ancestor_masks(bad)
        assert e.value.status == 3


def test_anchor_idx_matches_oracle():
    rng = np.random.default_rng(3)
    for _ in range(50):
        L = int(rng.integers(0, 300))
        cuts = sorted(rng.integers(0, L + 1, size=4).tolist())
        spans = [[cuts[0], cuts[1]], [cuts[2], cuts[3]]]
        Wn = int(rng.integers(-1, 100)); T = int(rng.integers(0, 9))
        assert B.sparrow_build_anchor_idx(L, spans, Wn, T) == oracle.anchor_idx(L, spans, Wn, T).tolist()
    got = B.sparrow_build_anchor_idx(26112, [[64, 25664]], 1024, 8)
    assert got == oracle.anchor_idx(26112, [[64, 25664]], 1024, 8).tolist() and len(got) == 456


def test_split_plan_properties():
    cases = [([26128], 16), ([16448], 64), ([2056], 8), ([456], 8), ([1], 1),
             ([n + 32 for n in W.ragged_lengths(W.config_seed(4), 5, 8)], 32)]
    for n_keys, T in cases:
        for n_sm in (148, 132, 16):
            splits, n_items = B.sparrow_plan_splits(n_sm, 4, n_keys, T)
            M = 7 * T
            groups = -(-M // (128 if M <= 128 else 256))    # row groups of one or two 128-row blocks
            assert n_items == sum(4 * groups * s for s in splits)
            assert all(1 <= s <= n for s, n in zip(splits, n_keys))
            units = 4 * groups * len(n_keys)
            assert n_items <= max(n_sm, units)
            # pieces tile the key range exactly, in whole 128-key tiles, sizes within one tile of each other
            for s, n in zip(splits, n_keys):
                ranges = [B.sparrow_plan_piece_range(n, s, i) for i in range(s)]
                assert ranges[0][0] == 0 and ranges[-1][1] == n
                assert all(a[1] == b[0] for a, b in zip(ranges, ranges[1:]))
                assert all(b < e and b % 128 == 0 for b, e in ranges)
                assert all(e % 128 == 0 for _, e in ranges[:-1])
                tiles = [-(-(e - b) // 128) for b, e in ranges]
                assert max(tiles) - min(tiles) <= 1
    assert B.sparrow_plan_splits(148, 4, [26128], 16) == ([37], 148)


def test_piece_range_rejects_bad_arguments():
    for args in ((0, 1, 0), (100, 2, 0), (1000, 3, 3), (1000, 0, 0), (1000, 3, -1)):
        with pytest.raises(B.SparrowError):
            B.sparrow_plan_piece_range(*args)
    assert B.sparrow_plan_piece_range(1000, 3, 2) == (640, 1000)


def test_plan_rejects_bad_arguments():
    for args in ((148, 4, [0], 8), (148, 4, [100], 0), (148, 4, [100], 65), (0, 4, [100], 8)):
        with pytest.raises(B.SparrowError):
            B.sparrow_plan_splits(*args)


def test_create_without_gpu_fails_loudly():
    import torch
    if torch.cuda.is_available():
        pytest.skip("has a GPU")
    with pytest.raises(B.SparrowError):
        B.Context(1, 100, 4 * 100 * 128, 100 * 128, 0.1, allocate_workspace=False)


def test_status_strings():
    assert B.sparrow_status_string(0) == "ok"
    assert "anchor" in B.sparrow_status_string(4)


def test_window_first_visible_matches_the_oracles_visibility():
    """The first visible compact row per query, against the oracle's visibility matrix of the
    anchored tree mode (the visible text anchors of a query are a contiguous run)."""
    rng = np.random.default_rng(7)
    for _ in range(60):
        n_text = int(rng.integers(0, 120))
        T_tree = int(rng.integers(1, 20)); T_new = int(rng.integers(1, T_tree + 1))
        text = np.sort(rng.choice(2000, size=n_text, replace=False))
        tree_rows = 2000 + int(rng.integers(0, 50)) + np.arange(T_tree)
        idx = np.concatenate([text, tree_rows]).astype(np.int32)
        window = int(rng.integers(-1, 2500))
        par = W.random_tree_parents(int(rng.integers(1 << 30)), 8, T_tree)
        vis = oracle.anchor_tree_visibility(idx, window, np.array(par, np.int32), T_new)       # [T_new, n_anchor]
        first, lowest = B.sparrow_window_first_visible(idx.tolist(), window, T_tree, T_new)
        for t in range(T_new):
            row = vis[t, :n_text]
            want = int(np.argmax(row)) if row.any() else n_text
            assert first[t] == want
            assert row[first[t]:].all() and not row[:first[t]].any()        # a contiguous run up to the tree
        assert lowest == min(first)
    with pytest.raises(B.SparrowError) as e:
        B.sparrow_window_first_visible([1, 5, 5, 9], 3, 2, 2)
    assert e.value.status == 4
