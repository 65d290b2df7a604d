"""CPU-only checks of the C ABI: the library loads, exports what the header declares, and the host-side
validation rejects malformed networks before any device work (no compute call is made here)."""
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def pkg():
    import paper_2104_11805_b200 as p
    from paper_2104_11805_b200.build import build_library
    build_library()
    return p


def header_functions():
    text = open(os.path.join(ROOT, "include", "sdnn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sdnn_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(pkg):
    lib = pkg.load_library()
    names = header_functions()
    assert "sdnn_create" in names and "sdnn_infer_batch" in names and "sdnn_train_step" in names and "sdnn_get_weights" in names
    for name in names:
        assert hasattr(lib, name), f"{name} is declared in include/sdnn.h but not exported"
    assert set(names) == set(pkg.exported_symbols()), "binding prototypes and header disagree"
    assert b"sm_100a" in lib.sdnn_version()


def test_missing_library_fails_loudly(pkg, tmp_path):
    with pytest.raises(pkg.SdnnError):
        pkg.load_library(str(tmp_path / "nope.so"))


def good():
    rp = np.array([0, 2, 2, 3], dtype=np.int32)
    col = np.array([0, 2, 1], dtype=np.int32)
    val = np.array([0.5, -1.0, 0.0], dtype=np.float32)       # an explicit zero is a legal stored entry
    bias = np.zeros(3, dtype=np.float32)
    return rp, col, val, bias


def create(pkg, rp, col, val, bias, **kw):
    kw.setdefault("max_batch", 4)
    return pkg.Sdnn.create([rp], [col], [val], [bias], **kw)


@pytest.mark.parametrize("mutate,needle", [
    (lambda a: a[0].__setitem__(0, 1), "row_ptr[0]"),
    (lambda a: a[0].__setitem__(2, 1), "decreases"),
    (lambda a: a[1].__setitem__(1, 3), "out of range"),
    (lambda a: a[1].__setitem__(0, -1), "out of range"),
    (lambda a: a[1].__setitem__(1, 0), "duplicate"),
    (lambda a: (a[1].__setitem__(0, 2), a[1].__setitem__(1, 0)), "not ascending"),
    (lambda a: a[2].__setitem__(2, np.nan), "non-finite value"),
    (lambda a: a[3].__setitem__(1, np.inf), "non-finite bias"),
])
def test_bad_csr_is_rejected_on_the_host(pkg, mutate, needle):
    arrays = good()
    mutate(arrays)
    with pytest.raises(pkg.SdnnError) as ei:
        create(pkg, *arrays)
    assert ei.value.code == -2 and needle in ei.value.message


@pytest.mark.parametrize("kw,code", [
    (dict(max_batch=0), -1), (dict(clamp=0.0), -1), (dict(clamp=float("nan")), -1),
    (dict(activation=2), -6), (dict(max_batch=129, train=True), -1), (dict(flags=0x3), -1),
])
def test_bad_config_is_rejected(pkg, kw, code):
    with pytest.raises(pkg.SdnnError) as ei:
        create(pkg, *good(), **kw)
    assert ei.value.code == code


def test_valid_net_without_a_device_reports_cuda_error_not_a_fallback(pkg):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    with pytest.raises(pkg.SdnnError) as ei:
        create(pkg, *good())
    assert ei.value.code == -4          # there is no CPU path behind the ABI


def test_null_handle_calls_do_not_crash(pkg):
    lib = pkg.load_library()
    assert lib.sdnn_finalize(None) == -1
    assert lib.sdnn_train_step(None, None, None, 1, 0.1, None) == -1
    assert lib.sdnn_infer_batch(None, None, 0, None, None, None, 0, None) == -1
    assert lib.sdnn_get_weights(None, 0, None, None) == -1
    assert lib.sdnn_kernel_launches(None) == 0
    lib.sdnn_destroy(None)


def test_tile_beyond_4_gib_is_rejected_before_any_device_work(pkg):
    """One activation tile (n_neurons x padded max_batch floats) must stay below 4 GiB; checked on the host."""
    nnz = np.zeros(1, dtype=np.int64)
    with pytest.raises(pkg.SdnnError) as ei:
        pkg.Sdnn.create_deferred(1, 1 << 20, nnz, max_batch=1024)
    assert ei.value.code == -1 and "4 GiB" in ei.value.message


def test_batch_sizes_whose_padding_overflows_32_bits_are_rejected_on_the_host(pkg):
    """Rounding a batch of nearly 2^31 inputs up to the tile width must not wrap around: both the allocation-free entry
    point and handle creation refuse such sizes before touching a device (dummy non-NULL addresses: never used)."""
    for huge in (2**31 - 1, 2**31 - 100, 2**30 + 1):
        with pytest.raises(pkg.SdnnError) as ei:
            pkg.infer_noalloc(1, 1, 16, 16, 16, [0], 16, 16, huge, 16)
        assert ei.value.code == -1 and "scratch" in ei.value.message
        with pytest.raises(pkg.SdnnError) as ei:
            pkg.Sdnn.create_deferred(1, 1, np.zeros(1, dtype=np.int64), max_batch=huge)
        assert ei.value.code == -1 and "max_batch" in ei.value.message
