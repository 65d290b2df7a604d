"""Host side of SDNN_FLAG_REORDER: the grouping of a layer's rows by the columns they share (no GPU needed).

The paper partitions the rows of W^k with a hypergraph whose nets are the columns, so that rows reading the same x
entries end up together (Section 5).  The library's stand-in is a greedy column-net clustering; these tests hold it to
what the structure of the input fixes: on a block pattern hidden behind a random renumbering of the neurons it must
find exactly the blocks, give every block one contiguous window of new column numbers, and renumber with a permutation;
on a uniformly random pattern it must report that there is nothing to find.
"""
import numpy as np
import pytest

import gen


@pytest.fixture(scope="module")
def pkg():
    import paper_2104_11805_b200 as p
    from paper_2104_11805_b200.build import build_library
    build_library()
    return p


def windows_of(col, k, group_of_row, col_label, n_groups):
    """Per group: the set of new column numbers its rows touch."""
    lab = col_label[col.reshape(-1, k)]
    return [np.unique(lab[group_of_row == g]) for g in range(n_groups)]


@pytest.mark.parametrize("n,window", [(4096, 1024), (2048, 256), (8192, 1024)])
def test_hidden_blocks_are_recovered_exactly(pkg, n, window):
    spec = gen.NetSpec("blocks", n, 3, pattern="windowed", window=window, config_id=4).shuffled()
    base = gen.NetSpec("blocks", n, 3, pattern="windowed", window=window, config_id=4)
    for layer in (0, 1, 2):
        col = gen.layer_pattern(spec, layer)
        grp, lab, ng, mw = pkg.cluster_layer(gen.row_ptr(spec), col)
        assert ng == n // window and mw == window
        assert np.array_equal(np.sort(lab), np.arange(n)), "the renumbering must be a permutation"
        # row r' of the shuffled layer is row q[r'] of the block pattern, whose block is q[r'] // window
        q = gen._renumbering(spec, layer)
        block = q // window
        for g in range(ng):
            assert len(np.unique(block[grp == g])) == 1, "a group mixes rows of different blocks"
        assert len(np.unique(grp)) == ng and len({int(block[grp == g][0]) for g in range(ng)}) == ng
        for w in windows_of(col, spec.k, grp, lab, ng):
            assert len(w) == window and w[-1] - w[0] + 1 == window, "a group's columns must be one contiguous range"
        # and on the pattern as generated (not shuffled) the same blocks come out
        grp0, lab0, ng0, mw0 = pkg.cluster_layer(gen.row_ptr(base), gen.layer_pattern(base, layer))
        assert ng0 == ng and mw0 == window and all(len(np.unique(grp0[b * window:(b + 1) * window])) == 1 for b in range(ng))


@pytest.mark.parametrize("n", [4096, 16384])
def test_uniformly_random_pattern_has_no_structure(pkg, n):
    spec = gen.NetSpec("uniform", n, 1, config_id=2)
    grp, lab, ng, mw = pkg.cluster_layer(gen.row_ptr(spec), gen.layer_pattern(spec, 0))
    assert ng == 0 and grp is None


def test_a_layer_that_fits_one_window_is_one_group(pkg):
    """1024 neurons: every column fits the window of 1536, whatever the pattern."""
    spec = gen.NetSpec("uniform", 1024, 1, config_id=2)
    grp, lab, ng, mw = pkg.cluster_layer(gen.row_ptr(spec), gen.layer_pattern(spec, 0))
    assert ng == 1 and mw <= 1024 and not grp.any() and np.array_equal(np.sort(lab), np.arange(1024))


def test_ragged_blocks_with_empty_rows(pkg):
    """Blocks of different sizes, rows of 0..9 entries, some rows empty: empty rows form a last group with no window."""
    rng = np.random.default_rng(3)
    sizes = [300, 50, 700, 129]
    n = sum(sizes)
    rows_of, cols_of, start = [], [], 0
    perm_r, perm_c = rng.permutation(n), rng.permutation(n)
    counts = np.zeros(n, dtype=np.int64)
    entries = {}
    for sz in sizes:
        for i in range(start, start + sz):
            m = int(rng.integers(0, 10))
            entries[perm_r[i]] = np.sort(perm_c[start + rng.choice(sz, size=min(m, sz), replace=False)])
            counts[perm_r[i]] = len(entries[perm_r[i]])
        start += sz
    rp = np.zeros(n + 1, dtype=np.int32); rp[1:] = np.cumsum(counts)
    col = np.concatenate([entries[i] for i in range(n)]).astype(np.int32)
    grp, lab, ng, mw = pkg.cluster_layer(rp, col, col_cap=1024, row_cap=4096)
    assert ng >= len(sizes) and mw <= 1024
    assert np.array_equal(np.sort(lab), np.arange(n))
    empty = counts == 0
    assert empty.any() and len(np.unique(grp[empty])) == 1 and grp[empty][0] == ng - 1
    inv_r = np.empty(n, dtype=np.int64); inv_r[perm_r] = np.arange(n)
    bounds = np.cumsum([0] + sizes)
    block_of_row = np.searchsorted(bounds, inv_r, side="right") - 1
    for g in range(ng - 1):
        members = np.flatnonzero((grp == g) & ~empty)
        assert len(np.unique(block_of_row[members])) == 1, "rows of different blocks share no column and must not be grouped"
        labs = np.unique(np.concatenate([lab[entries[i]] for i in members]))
        assert labs[-1] - labs[0] + 1 <= 1024


def test_caps_are_respected_and_bad_arguments_rejected(pkg):
    spec = gen.NetSpec("blocks", 2048, 1, pattern="windowed", window=512, config_id=4)
    rp, col = gen.row_ptr(spec), gen.layer_pattern(spec, 0)
    grp, lab, ng, mw = pkg.cluster_layer(rp, col, col_cap=512, row_cap=4096)
    assert ng == 4 and mw == 512
    grp, lab, ng, mw = pkg.cluster_layer(rp, col, col_cap=100, row_cap=4096)      # no window of 100 columns holds a block
    assert ng == 0
    with pytest.raises(pkg.SdnnError):
        pkg.cluster_layer(rp, col, col_cap=0)
