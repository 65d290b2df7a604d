"""The allocation-free inference entry point (sdnn_infer_noalloc) against sdnn_infer_batch.

Some callers of this library cannot allocate device memory when they call it (their process has handed
the whole device to another allocator, they sit in a latency-critical loop, or their plug-in rules forbid
it), so this entry point keeps its activation scratch in a fixed array inside the library and takes the
network as the caller's own device arrays.  The test calls it through the C ABI twice in a row (the
second call with a smaller batch, so stale scratch contents from the first would show) and compares
with the handle-based entry point.  This file is collected last on purpose.
"""
import numpy as np
import pytest

import gen

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
        reserved = torch.cuda.memory_reserved()
        pkg.infer_noalloc(L, n, d_rp, d_col, d_val, offsets, d_bias, x0, cnt, got)
        torch.cuda.synchronize()
        assert torch.cuda.memory_reserved() == reserved
        w, g = want.cpu().numpy(), got.cpu().numpy()
        assert np.abs(w).max() > 0
        assert np.abs(g - w).max() <= 1e-4 * np.abs(w).max()
    h.destroy()


def test_noalloc_rejects_sizes_beyond_the_builtin_scratch():
    import paper_2104_11805_b200 as pkg
    from paper_2104_11805_b200.build import build_library
    build_library()
    n = 4096
    too_many = pkg.NOALLOC_MAX_TILE_FLOATS // n + 1
    with pytest.raises(pkg.SdnnError) as ei:
        pkg.infer_noalloc(1, n, 16, 16, 16, [0], 16, 16, too_many, 16)     # dummy non-NULL addresses: rejected before use
    assert ei.value.code == -1 and "scratch" in ei.value.message
