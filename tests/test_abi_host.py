"""Host-only checks of the C ABI: the library loads, exports every symbol the header declares,
and rejects bad arguments before touching a device.  No compute calls, no GPU needed."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def D():
    from paper_2601_18383_b200 import build
    build.build()
    import paper_2601_18383_b200 as D
    return D


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "dynts.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dynts_[a-z_0-9]+)\s*\(", text)))


def test_header_symbols_are_exported(D):
    syms = declared_symbols()
    assert len(syms) >= 20
    lib = ctypes.CDLL(D.LIB_PATH)
    for s in syms:
        assert hasattr(lib, s), f"{s} declared in include/dynts.h but not exported"


def test_binding_covers_every_symbol(D):
    for s in declared_symbols():
        assert hasattr(D, s), f"binding lacks {s}"


def test_create_defaults_and_bad_arguments(D):
    h = D.dynts_cache_create(4, 2, 128, 256, 32)
    assert D.dynts_cache_capacity(h) == 256 + 64
    assert D.dynts_cache_len(h, 0) == 0
    assert D.dynts_cache_len(h, 5) == -1
    assert D.dynts_cache_scores(h) is None
    D.dynts_cache_set_shape(h, 3, 8, D.DYNTS_FP32, 16)
    assert D.dynts_cache_capacity(h) == 256 + 16
    with pytest.raises(D.DyntsError) as e:
        D.dynts_cache_set_shape(h, 3, 7, D.DYNTS_FP32, 16)          # q_heads not a multiple of kv_heads
    assert e.value.status == D.DYNTS_ERR_INVALID_ARG
    with pytest.raises(D.DyntsError):
        D.dynts_evict(h, 0)                                          # nothing stored yet
    D.dynts_cache_destroy(h)
    for bad in [(0, 2, 128, 256, 32), (4, 2, 100, 256, 32), (4, 2, 128, 0, 0), (4, 2, 128, 16, 32)]:
        with pytest.raises(D.DyntsError):
            D.dynts_cache_create(*bad)
    assert "invalid" in D.dynts_last_error()


def test_cache_bytes_accounts_for_slabs(D):
    cfg = D.make_config(32, 1, 32, 8, 128, 2048, 128, 64)
    nbytes = D.dynts_cache_bytes(cfg)
    kv = 32 * 8 * 2112 * 128 * 2 * 2
    assert kv < nbytes < kv * 1.12      # + positions, scores, compensation, gather list (16 B) and two halves of fp32 logits (32 B) per 512 B row
    assert D.dynts_cache_bytes(D.make_config(32, 1, 32, 8, 128, 2048, 4096, 64)) == 0   # window > budget
    assert D.dynts_cache_bytes(D.make_config(1, 1, 18, 2, 128, 64, 8, 8)) == 0          # G = 9 unsupported
    ragged = D.make_config(2, 3, 8, 2, 128, 1024, 128, 64, seq_budgets=[1024, 2048, 3072])
    assert D.dynts_cache_bytes(ragged) > D.dynts_cache_bytes(D.make_config(2, 3, 8, 2, 128, 1024, 128, 64))


def test_launch_knobs_validate(D):
    h = D.dynts_cache_create(1, 1, 64, 32, 4)
    D.dynts_cache_set_launch(h, 4, 1)
    with pytest.raises(D.DyntsError):
        D.dynts_cache_set_launch(h, 3, 0)
    with pytest.raises(D.DyntsError):
        D.dynts_cache_set_launch(h, 0, 9)
    assert D.dynts_cache_launch_count(h) == 0
    D.dynts_cache_destroy(h)


def test_product_does_not_import_oracle():
    """The product package must not reach the oracle (or any CPU fallback)."""
    pkg = os.path.join(ROOT, "paper_2601_18383_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower(), f"{f} mentions the oracle"
