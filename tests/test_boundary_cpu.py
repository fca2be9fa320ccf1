"""Host-only checks of the C boundary: the library builds for sm_100a, loads without a GPU, exports every
symbol the header declares, and validates arguments before touching a device."""
import ctypes as C
import os
import re

import pytest

from paper_2402_08644_b200 import binding, build, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load_library()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "tandem.h")).read()
    return sorted(set(re.findall(r"TANDEM_API\s+[\w\s\*]+?\b(tandem_\w+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared_symbols()
    assert len(names) >= 13 and "tandem_block_step" in names and "tandem_speculative_generate" in names
    assert sorted(binding.EXPORTS) == [n for n in names if n in binding.EXPORTS]
    for n in names:
        assert hasattr(lib, n), n


def test_status_strings(lib):
    assert lib.tandem_status_string(0) == b"ok"
    assert lib.tandem_status_string(4) == b"capacity exceeded"
    assert len({lib.tandem_status_string(i) for i in range(9)}) == 9


def test_query_arena_validates_and_sizes(lib):
    shape = synth.named_config("small")
    cfg, keep = binding.make_config(shape, max_batch=1, max_seq=1024, gamma_max=3)
    n = binding.tandem_query_arena(cfg)
    kv = (12 * 2 * 1024 * 1024 + 4 * 2 * 1024 * 512) * 2          # both KV caches, bf16
    assert kv < n < kv + (1 << 30)
    bad, keep2 = binding.make_config(shape, max_batch=1, max_seq=1024, gamma_max=16)
    with pytest.raises(binding.TandemError) as e:
        binding.tandem_query_arena(bad)
    assert e.value.status == 1
    odd = synth.make_shape(synth.ModelDims(2, 96, 4, 128, 50, 32), synth.ModelDims(1, 64, 2, 64, 50, 32))
    cfg3, keep3 = binding.make_config(odd, 1, 32, 2)              # head size 24 is not supported
    with pytest.raises(binding.TandemError) as e:
        binding.tandem_query_arena(cfg3)
    assert e.value.status == 2
    out = C.c_size_t(0)
    assert lib.tandem_query_arena(None, C.byref(out)) == 1
    assert lib.tandem_query_arena(C.byref(cfg), None) == 1


def test_null_context_calls_fail_cleanly(lib):
    assert lib.tandem_destroy(None) == 1
    assert lib.tandem_block_step(None, 1, 0, 0, None) == 1
    assert lib.tandem_decode_attention_scratch_bytes(0, 1, 64, 1, 1) == 0
    assert lib.tandem_decode_attention_scratch_bytes(2, 16, 64, 1000, 4) >= 2 * 2 * 4
