"""Host-side checks that need no GPU: the library loads, exports every symbol
the headers declare, and argument validation that happens before any CUDA call."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2204_06514_b200 import build, binding
    build.build()
    return binding.load_library()


def declared_symbols():
    names = set()
    for h in ("fax.h", "fax_ops.h", "fax_dp.h"):
        text = open(os.path.join(ROOT, "include", h)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names |= set(re.findall(r"\b(fax_[a-z0-9_]+)\s*\(", text))
    return sorted(names)


def test_every_declared_symbol_is_exported(lib):
    syms = declared_symbols()
    assert len(syms) >= 20
    for s in syms:
        assert hasattr(lib, s), s


def test_binding_covers_every_declared_symbol(lib):
    from paper_2204_06514_b200 import binding, binding_ops, dp
    have = set(binding._SIGNATURES) | set(binding_ops._SIGNATURES) | set(dp._SIGNATURES)
    assert set(declared_symbols()) <= have


def test_status_strings(lib):
    from paper_2204_06514_b200 import binding as fx
    assert fx.status_string(0) == "FAX_OK"
    assert fx.status_string(fx.FAX_ERR_TIMEOUT) == "FAX_ERR_TIMEOUT"
    assert fx.status_string(-99) == "FAX_ERR_UNKNOWN"


def test_block_sizes_and_shape_validation(lib):
    from paper_2204_06514_b200 import binding as fx
    ok = fx.BlockCfg(2, 128, 256, 4, 64, 1024, 1e-5, fx.FAX_PREC_BF16)
    saved, scratch = fx.fax_block_sizes(ok)
    n, d, f = 256, 256, 1024
    assert saved >= 2 * n * (7 * d + 2 * f) and scratch >= 2 * n * (f + 5 * d)
    bad_heads = fx.BlockCfg(2, 128, 256, 4, 32, 1024, 1e-5, fx.FAX_PREC_BF16)
    with pytest.raises(fx.FaxError) as e:
        fx.fax_block_sizes(bad_heads)
    assert e.value.status == fx.FAX_ERR_INVALID_ARG
    bad_tile = fx.BlockCfg(2, 100, 256, 4, 64, 1024, 1e-5, fx.FAX_PREC_BF16)
    with pytest.raises(fx.FaxError) as e:
        fx.fax_block_sizes(bad_tile)
    assert e.value.status == fx.FAX_ERR_UNSUPPORTED_SHAPE
    # the float32 validation mode takes ragged sizes
    fx.fax_block_sizes(fx.BlockCfg(2, 5, 8, 2, 4, 16, 1e-5, fx.FAX_PREC_FP32_VALIDATE))


def test_lm_sizes(lib):
    from paper_2204_06514_b200 import binding as fx
    cfg = fx.LmCfg(12, 50304, 1024, fx.BlockCfg(16, 1024, 768, 12, 64, 3072, 1e-5, fx.FAX_PREC_BF16))
    saved, scratch = fx.fax_lm_sizes(cfg)
    assert saved > 12 * 16384 * 768 * 2 * 8
    with pytest.raises(fx.FaxError):
        fx.fax_lm_sizes(fx.LmCfg(12, 50304, 512, cfg.block))     # max_seq < seq


def test_null_context_is_rejected(lib):
    from paper_2204_06514_b200 import binding as fx
    hp = fx.AdamwHparams(1e-3, 0.9, 0.95, 1e-8, 1, 0)
    assert lib.fax_adamw_step(None, None, 0, C.byref(hp)) == fx.FAX_ERR_INVALID_ARG
    assert lib.fax_destroy(None) == fx.FAX_ERR_INVALID_ARG


def test_missing_library_fails_loudly(tmp_path):
    from paper_2204_06514_b200 import binding as fx
    with pytest.raises(RuntimeError):
        fx.load_library(str(tmp_path / "nope.so"))


def test_product_never_imports_oracle():
    pkg = os.path.join(ROOT, "paper_2204_06514_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.replace("test oracle", ""), f
