"""The allocation-free inference entry point (sdnn_infer_noalloc) against sdnn_infer_batch.

Some callers of this library cannot allocate device memory when they call it (their process has handed
the whole device to another allocator, they sit in a latency-critical loop, or their plug-in rules forbid
it), so this entry point keeps its activation scratch in a fixed array inside the library and takes the
network as the caller's own device arrays.  The test calls it through the C ABI twice in a row (the
second call with a smaller batch, so stale scratch contents from the first would show) and compares
with the handle-based entry point and with the float64 oracle; a second test runs nets whose rows have any
length (rows that do not start on a multiple of four entries take the kernel's one-entry-at-a-time path)
and batches of one to a few inputs.  This file is collected last on purpose.
"""
import numpy as np
import pytest

import gen
from oracle import OracleNet
from parity_util import check_close, ragged_net

pytestmark = pytest.mark.gpu


def test_noalloc_inference_matches_handle_inference_twice_in_a_row():
    torch = pytest.importorskip("torch")
    assert torch.cuda.is_available()
    import paper_2104_11805_b200 as pkg
    from paper_2104_11805_b200.build import build_library
    build_library()

    spec = gen.CFG2.scaled(4096, 10).live()
    rp, col, val, bias = gen.network(spec)
    L, n = spec.layers, spec.n
    h = pkg.Sdnn.create(rp, col, val, bias, max_batch=256)

    offsets = np.arange(L, dtype=np.int64) * spec.nnz_per_layer
    d_rp = torch.from_numpy(np.stack(rp)).cuda()
    d_col = torch.from_numpy(np.concatenate(col)).cuda()
    d_val = torch.from_numpy(np.concatenate(val)).cuda()
    d_bias = torch.from_numpy(np.stack(bias)).cuda()

    for cnt, start in ((200, 0), (37, 500)):
        x0 = torch.from_numpy(gen.inputs(spec, cnt, start=start)).cuda()
        want = torch.empty((cnt, n), device="cuda")
        got = torch.full((cnt, n), -1.0, device="cuda")
        h.infer_batch(x0, cnt, want, None, None, 0)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]          # the driver's count of free device bytes: sees any cudaMalloc
        pkg.infer_noalloc(L, n, d_rp, d_col, d_val, offsets, d_bias, x0, cnt, got)
        torch.cuda.synchronize()
        if start:       # the first call on a device may load the module; from the second on nothing may be taken
            assert torch.cuda.mem_get_info()[0] == free_before
        w, g = want.cpu().numpy(), got.cpu().numpy()
        assert np.abs(w).max() > 0
        assert np.abs(g - w).max() <= 1e-4 * np.abs(w).max()
        check_close(g, OracleNet(rp, col, val, bias).infer(gen.inputs(spec, cnt, start=start)), "x^L against the oracle")
    h.destroy()


@pytest.mark.parametrize("cnt", [1, 3, 5, 20, 150])
def test_noalloc_inference_on_ragged_rows_and_tiny_batches_matches_the_oracle(cnt):
    """Rows of 0..11 entries, so that most rows start off a multiple of four; each layer's entries start on one
    (the entry point's rule), which leaves up to three unused slots between layers."""
    torch = pytest.importorskip("torch")
    assert torch.cuda.is_available()
    import paper_2104_11805_b200 as pkg
    from paper_2104_11805_b200.build import build_library
    build_library()

    rng = np.random.default_rng(40 + cnt)
    n, L = 301, 4
    rp, col, val, bias = ragged_net(rng, n=n, layers=L, kmax=11, scale=0.5)
    offsets, run = [], 0
    for c in col:
        offsets.append(run)
        run += (len(c) + 3) // 4 * 4
    flat_col = np.zeros(run, dtype=np.int32); flat_val = np.zeros(run, dtype=np.float32)
    for o, c, v in zip(offsets, col, val):
        flat_col[o:o + len(c)] = c; flat_val[o:o + len(v)] = v
    assert all((np.asarray(r)[:-1] % 4 != 0).sum() > n // 2 for r in rp), "most rows should start off a multiple of four"
    d_rp, d_col, d_val = (torch.from_numpy(a).cuda() for a in (np.stack(rp), flat_col, flat_val))
    d_bias = torch.from_numpy(np.stack(bias)).cuda()
    x0 = rng.uniform(0, 1.0, size=(cnt, n)).astype(np.float32)
    want = OracleNet(rp, col, val, bias).infer(x0)
    assert np.abs(want).max() > 0
    for _ in range(2):
        got = torch.full((cnt, n), -1.0, device="cuda")
        pkg.infer_noalloc(L, n, d_rp, d_col, d_val, np.asarray(offsets, dtype=np.int64), d_bias, torch.from_numpy(x0).cuda(), cnt, got)
        torch.cuda.synchronize()
        check_close(got.cpu().numpy(), want, f"{cnt} inputs")


def test_noalloc_counts_and_skips_out_of_range_columns():
    """The entry point cannot validate device arrays on the host; its kernel does not follow a column index outside
    [0, n) and counts it.  Two corrupted entries (one negative, one too large), each seen by every input chunk once."""
    torch = pytest.importorskip("torch")
    assert torch.cuda.is_available()
    import paper_2104_11805_b200 as pkg
    from paper_2104_11805_b200.build import build_library
    build_library()
    spec = gen.CFG2.scaled(1024, 2).live()
    rp, col, val, bias = gen.network(spec)
    bad_col = [c.copy() for c in col]
    bad_col[0][5] = -3
    bad_col[1][77] = spec.n + 10
    good_val = [v.copy() for v in val]
    good_val[0][5] = 0.0; good_val[1][77] = 0.0                  # the net the kernel effectively evaluates
    offsets = np.arange(2, dtype=np.int64) * spec.nnz_per_layer
    d_rp, d_col, d_val = (torch.from_numpy(a).cuda() for a in (np.stack(rp), np.concatenate(bad_col), np.concatenate(val)))
    d_bias = torch.from_numpy(np.stack(bias)).cuda()
    x0 = gen.inputs(spec, 16)
    got = torch.empty((16, spec.n), device="cuda")
    before = pkg.infer_noalloc_bad_columns()
    pkg.infer_noalloc(2, spec.n, d_rp, d_col, d_val, offsets, d_bias, torch.from_numpy(x0).cuda(), 16, got)
    assert pkg.infer_noalloc_bad_columns() - before == 2
    check_close(got.cpu().numpy(), OracleNet(rp, col, good_val, bias).infer(x0), "bad entries skipped")


def test_noalloc_rejects_sizes_beyond_the_builtin_scratch():
    import paper_2104_11805_b200 as pkg
    from paper_2104_11805_b200.build import build_library
    build_library()
    n = 4096
    too_many = pkg.NOALLOC_MAX_TILE_FLOATS // n + 1
    with pytest.raises(pkg.SdnnError) as ei:
        pkg.infer_noalloc(1, n, 16, 16, 16, [0], 16, 16, too_many, 16)     # dummy non-NULL addresses: rejected before use
    assert ei.value.code == -1 and "scratch" in ei.value.message
