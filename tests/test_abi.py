"""The C-ABI library loads, exports every symbol include/treekv.h declares, and rejects bad arguments on the
host before touching a GPU.  No kernels run here."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    from paper_2501_04987_b200 import _build

    _build.build()
    from paper_2501_04987_b200 import binding as b

    return b


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "treekv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(treekv_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(binding):
    declared = _declared_symbols()
    assert len(declared) >= 16
    for name in declared:
        assert hasattr(binding.lib, name), name
    assert sorted(binding.EXPORTS) == declared


def test_version_and_status_strings(binding):
    assert re.match(r"^\d+\.\d+$", binding.treekv_version())
    assert binding.status_string(0) == "ok"
    assert len({binding.status_string(i) for i in range(7)}) == 7


def test_workspace_bytes_shapes(binding):
    wb = binding.treekv_workspace_bytes
    # decode-only Llama-2-7B-shaped layer: two slabs of 2c rows dominate
    n = wb(1024, 32, 32, 128, binding.TREEKV_BF16, 8, 0)
    slabs = 2 * 8 * 32 * 2048 * 128 * 2
    assert slabs <= n <= slabs * 1.05
    assert n % 256 == 0
    # unsupported shapes give 0
    assert wb(1, 32, 32, 128, 1, 8, 0) == 0          # budget < 2
    assert wb(1024, 32, 5, 128, 1, 8, 0) == 0        # heads not divisible
    assert wb(1024, 32, 32, 96, 1, 8, 0) == 0        # head_dim
    assert wb(1024, 32, 32, 128, 7, 8, 0) == 0       # dtype
    assert wb(1024, 32, 32, 128, 1, 0, 0) == 0       # batch
    assert wb(1024, 48, 4, 128, 1, 1, 0) == 0        # group size 12
    assert wb(1024, 32, 32, 128, 1, 8, 100000) == 0  # chunk too long
    # prefill scratch grows the workspace
    assert wb(2048, 32, 8, 128, 1, 4, 1024) > wb(2048, 32, 8, 128, 1, 4, 0)


def test_create_rejects_bad_arguments_on_the_host(binding):
    st, h = binding.treekv_create(1024, 32, 32, 96, 1, 8, 0, 0, 0)
    assert st == 4 and not h.value
    st, h = binding.treekv_create(64, 4, 4, 64, 0, 1, 0, 0, 0)           # null workspace
    assert st == 3 and not h.value
    n = binding.treekv_workspace_bytes(64, 4, 4, 64, 0, 1, 0)
    st, h = binding.treekv_create(64, 4, 4, 64, 0, 1, 0, 256 + 8, n)     # misaligned workspace
    assert st == 3 and not h.value
    st, h = binding.treekv_create(64, 4, 4, 64, 0, 1, 0, 4096, n - 1)    # too small
    assert st == 3 and not h.value


def test_null_context_is_an_error_not_a_crash(binding):
    assert binding.treekv_decode_step(None, 0, 0, 0, 0) == 1
    assert binding.treekv_prefill_chunk(None, 0, 0, 0, 0, None, 1) == 1
    assert binding.treekv_retained_positions(None, 0, 0) == 1
    assert binding.treekv_scores(None, 0) == 1
    assert binding.treekv_set_rule(None, 0) == 1
    assert binding.treekv_tokens_seen(None, 0) == -1
    binding.treekv_destroy(None)
