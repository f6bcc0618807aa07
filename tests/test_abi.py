"""The C-ABI library: it builds, loads without a GPU, exports every entry point
the header declares, and validates arguments on the host."""
import ctypes as C
import os
import re

import pytest

from paper_2506_15969_b200 import binding

HEADER = os.path.join(os.path.dirname(__file__), "..", "include", "lazyev.h")


def declared_symbols():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(lazyev_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = binding.lib()
    names = declared_symbols()
    assert len(names) >= 20 and "lazyev_decode_step" in names and "lazyev_evict" in names
    for name in names:
        assert hasattr(lib, name), f"{name} is declared in lazyev.h but not exported"
    for name in binding._PROTOS:
        assert name in names, f"binding wraps {name}, which the header does not declare"


def create(*args):
    h = C.c_void_p()
    return binding.lib().lazyev_create(C.byref(h), *args), h


def test_create_validates_arguments():
    ok, h = create(2, 8, 2, 128, 512, 128, 1e-3)
    assert ok == binding.OK and h.value
    assert binding.lib().lazyev_destroy(h) == binding.OK
    for bad in [(2, 8, 2, 64, 512, 128, 1e-3),       # head_dim other than 128
                (2, 8, 3, 128, 512, 128, 1e-3),      # q_heads not a multiple of kv_heads
                (2, 18, 2, 128, 512, 128, 1e-3),     # more than 8 query heads per KV head
                (0, 8, 2, 128, 512, 128, 1e-3),
                (2, 8, 2, 128, 128, 128, 1e-3),      # budget must exceed the window
                (2, 8, 2, 128, 512, 0, 1e-3),
                (2, 8, 2, 128, 512, 128, -1.0),
                (2, 8, 2, 128, 512, 128, float("nan"))]:
        rc, h = create(*bad)
        assert rc == binding.EINVAL and not h.value
    assert binding.lib().lazyev_create(None, 2, 8, 2, 128, 512, 128, 1e-3) == binding.EINVAL


def test_host_side_configuration_and_sizes():
    lib = binding.lib()
    rc, h = create(28, 28, 4, 128, 8192, 128, 1e-3)
    assert rc == binding.OK
    assert lib.lazyev_set_batch(h, 32) == binding.OK
    assert lib.lazyev_set_batch(h, 0) == binding.EINVAL
    assert b"batch" in lib.lazyev_last_error(h)
    assert lib.lazyev_set_protect(h, 128, 4) == binding.OK
    assert lib.lazyev_set_protect(h, 0, 0) == binding.EINVAL
    assert lib.lazyev_set_protect(h, 8000, 192) == binding.EINVAL
    assert lib.lazyev_set_budget(h, 4096) == binding.OK
    assert lib.lazyev_set_budget(h, 8193) == binding.EINVAL
    assert lib.lazyev_set_budget(h, 132) == binding.EINVAL
    assert lib.lazyev_set_score_mode(h, 3) == binding.OK
    assert lib.lazyev_set_score_mode(h, 4) == binding.EINVAL
    assert lib.lazyev_set_splits(h, 9) == binding.EINVAL and lib.lazyev_set_splits(h, 3) == binding.OK
    kv, st, sc = C.c_size_t(), C.c_size_t(), C.c_size_t()
    assert lib.lazyev_query_sizes(h, C.byref(kv), C.byref(st), C.byref(sc)) == binding.OK
    info = binding.Info()
    assert lib.lazyev_get_info(h, C.byref(info)) == binding.OK
    assert (info.units, info.capacity, info.pages_per_unit) == (3584, 8320, 130)
    assert kv.value == 3584 * 130 * 32768                       # 15.3 GB of pages
    assert st.value >= 3584 * 8320 * 16 and sc.value >= 3584 * 8192 * 4
    # calls that need a bound handle say so instead of touching the device
    assert lib.lazyev_prefill(h, 1, 1, 16) == binding.ESTATE
    assert lib.lazyev_decode_step(h, 1, 1, 1, 1) == binding.ESTATE
    assert lib.lazyev_evict(h, None) == binding.ESTATE
    assert lib.lazyev_decode_step(h, None, 1, 1, 1) == binding.EINVAL
    assert lib.lazyev_bind(h, None, None, None, None) == binding.EINVAL
    assert lib.lazyev_bind(h, 8, 256, 256, None) == binding.EINVAL  # misaligned
    assert lib.lazyev_destroy(h) == binding.OK
    assert lib.lazyev_strerror(binding.ECAPACITY) == b"cache capacity exceeded"
    assert lib.lazyev_set_max_prefill(None, 5) == binding.EINVAL


def test_capacity_grows_with_a_long_prompt():
    lib = binding.lib()
    rc, h = create(1, 8, 2, 128, 512, 128, 1e-3)
    info = binding.Info()
    lib.lazyev_get_info(h, C.byref(info))
    assert info.capacity == 640 and info.n_recent == 128 and info.n_initial == 0
    assert lib.lazyev_set_max_prefill(h, 1000) == binding.OK
    lib.lazyev_get_info(h, C.byref(info))
    assert info.capacity == 1152 and info.pages_per_unit == 18
    lib.lazyev_destroy(h)


def test_diagnostic_and_mode_setters_validate_arguments():
    """Host-side checks of the switches that need no device: wait limit, prompt mode, per-row dump range,
    page-ring starvation, in-launch append; and the calls that need a bound handle say so."""
    lib = binding.lib()
    rc, h = create(2, 8, 2, 128, 512, 128, 1e-3)
    assert rc == binding.OK
    assert lib.lazyev_set_wait_limit(h, 0.004) == binding.OK
    assert lib.lazyev_set_wait_limit(h, 0.0) == binding.EINVAL and lib.lazyev_set_wait_limit(h, 1e9) == binding.EINVAL
    assert lib.lazyev_set_wait_limit(h, float("nan")) == binding.EINVAL
    assert lib.lazyev_set_prompt_mode(h, binding.PROMPT_REPLAY) == binding.OK
    assert lib.lazyev_set_prompt_mode(h, 7) == binding.EINVAL
    assert lib.lazyev_debug_starve_page_ring(h, 3) == binding.OK and lib.lazyev_debug_starve_page_ring(h, -1) == binding.OK
    assert lib.lazyev_debug_starve_page_ring(h, -2) == binding.EINVAL
    assert lib.lazyev_set_fused_append(h, 0) == binding.OK and lib.lazyev_set_fused_append(h, 1) == binding.OK
    fake = C.c_void_p(256)                                     # never dereferenced: only the range is checked here
    assert lib.lazyev_set_prompt_dump(h, fake, 0, 4) == binding.OK           # units = 2 layers x 1 batch x 2 heads
    assert lib.lazyev_set_prompt_dump(h, fake, 3, 2) == binding.EINVAL
    assert lib.lazyev_set_prompt_dump(h, None, 0, 0) == binding.OK
    assert lib.lazyev_host_wait(h, 2) == binding.EINVAL and lib.lazyev_host_wait(h, 0) == binding.OK
    counters = binding.Counters()
    assert lib.lazyev_get_counters(h, C.byref(counters)) == binding.ESTATE   # before bind
    assert lib.lazyev_synchronize(h) == binding.ESTATE and lib.lazyev_reset(h) == binding.ESTATE
    assert lib.lazyev_copy_state(h, h) == binding.EINVAL
    rc2, h2 = create(2, 8, 2, 128, 512, 128, 1e-3)
    assert lib.lazyev_copy_state(h2, h) == binding.ESTATE      # neither handle is bound
    assert lib.lazyev_build_flags() in (0, 1)
    assert lib.lazyev_destroy(h) == binding.OK and lib.lazyev_destroy(h2) == binding.OK
