"""The C-ABI library loads and exports every symbol include/xsv.h declares (no GPU needed)."""
import ctypes
import os
import re

from paper_2602_21780_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    src = open(os.path.join(ROOT, "include", "xsv.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(xsv_[a-z_0-9]+)\s*\(", src)))


def test_library_exports_every_declared_symbol():
    import __graft_entry__ as ge
    ge.build()
    lib = ctypes.CDLL(binding.LIB_PATH)
    names = _declared()
    assert len(names) >= 15
    for n in names:
        assert hasattr(lib, n), f"{n} declared in xsv.h but not exported"
    assert set(names) == set(binding.SYMBOLS), "binding and header disagree on the entry points"


def test_host_side_argument_checks_need_no_gpu():
    lib = binding.load()
    h = ctypes.c_void_p()
    assert lib.xsv_cache_create(None, 1, 16, 64, 100, 4) == 1
    assert lib.xsv_cache_create(ctypes.byref(h), 0, 16, 64, 100, 4) == 1
    assert lib.xsv_cache_create(ctypes.byref(h), 1, 16, 128, 100, 4) == 1      # head_dim must be 64
    assert lib.xsv_cache_create(ctypes.byref(h), 1, 16, 64, 100, 3) == 1       # bits in {2,4,8,16}
    assert lib.xsv_cache_bytes(None) == 0
    assert lib.xsv_cache_len(None, 0) == -1
    assert lib.xsv_step(None, 0, None, None, None, 1, 0, None, None) == 1
    assert lib.xsv_strerror(6) == b"bounded device-side wait ran out"
    lib.xsv_cache_destroy(None)


def test_per_device_table_keeps_devices_apart():
    # kernel attributes are per CUDA device; the table that remembers them must not let one device's
    # entry stand for another's (host-only self-test inside the library)
    assert binding.load().xsv_selftest_device_table() == 0


def test_batched_streams_are_grouped_so_that_ctas_fit():
    # CTAs do not span streams: eight long streams on 148 multiprocessors go out as two launches of four (37 CTAs
    # each) rather than one of eight (18 or 19 each); four go out together; short streams stay in one launch, where
    # a second launch would cost more than the uneven split; other counts fall back to the best of n, 4, 2, 1
    F = 1374
    assert binding.plan_batch_groups([21984] * 8, [F] * 8, 16) == 4
    assert binding.plan_batch_groups([21984] * 4, [F] * 4, 16) == 4
    assert binding.plan_batch_groups([21984] * 2, [F] * 2, 16) == 2
    assert binding.plan_batch_groups([21984], [F], 16) == 1
    assert binding.plan_batch_groups([600] * 8, [200] * 8, 4) == 8
    assert binding.plan_batch_groups([21984] * 6, [F] * 6, 16) == 4                          # 37 x 4, then 74 x 2
    assert binding.plan_batch_groups([21984] * 7, [F] * 7, 16) == 7                          # 21 each: 147 of 148
    assert binding.plan_batch_groups([21984] * 8, [F] * 8, 16, multiprocessors=160) == 8      # 20 CTAs each: even
    assert binding.plan_batch_groups([], [], 16) == -1
    assert binding.plan_batch_groups([-1], [F], 16) == -1
