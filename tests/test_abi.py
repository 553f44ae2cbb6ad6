"""The C-ABI boundary without a GPU: librlkv.so loads, exports every function include/rlkv.h
declares, the Python binding has one function of the same name for each, and the host-side argument
checks that need no device answer with the documented codes."""
import ctypes
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "rlkv.h")


def declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"\b(rlkv_[a-z0-9_]+)\s*\(", text)
    return sorted(set(names))


@pytest.fixture(scope="module")
def binding():
    from paper_2510_08525_b200 import build
    build.build()
    import paper_2510_08525_b200.binding as b
    return b


def test_header_declares_the_three_calls_of_the_problem_statement():
    names = declared_functions()
    for must in ("rlkv_cache_create", "rlkv_append", "rlkv_decode_attention"):
        assert must in names
    assert len(names) >= 10


def test_library_exports_every_declared_symbol(binding):
    lib = ctypes.CDLL(binding.LIB_PATH)
    for name in declared_functions():
        assert hasattr(lib, name), f"librlkv.so does not export {name}"


def test_binding_has_the_same_names(binding):
    for name in declared_functions():
        assert callable(getattr(binding, name)), name
        assert name in binding.SIGNATURES
    assert sorted(binding.SIGNATURES) == declared_functions()


def test_error_codes_match_the_header(binding):
    text = open(HEADER).read()
    for name, value in re.findall(r"(RLKV_[A-Z]+)\s*=\s*(-?\d+)", text):
        assert getattr(binding, name) == int(value)
        assert binding.rlkv_strerror(int(value))
    assert binding.rlkv_strerror(-99) == "unknown error"


def test_host_side_argument_checks_need_no_device(binding):
    ok = dict(layers=2, kv_heads=2, q_heads=8, head_dim=128, batch=3, max_len=100,
              head_is_full=[1, 0, 0, 1], sink=4, window=12)
    size = binding.rlkv_cache_size(**ok)
    # two full heads of 128 rows (100 rounded up to the tile) and two compressed heads of 64 rows,
    # K and V, per batch row
    pool = 3 * (2 * 128 + 2 * 64) * 2 * 128 * 2
    assert size >= pool
    # compressed heads cost the same however long the sequence may grow
    longer = binding.rlkv_cache_size(**{**ok, "max_len": 100 + 64 * 10})
    assert longer - size == 3 * 2 * 640 * 2 * 128 * 2
    for bad in (dict(head_dim=96), dict(q_heads=7), dict(q_heads=18), dict(window=0), dict(sink=-1),
                dict(batch=0), dict(max_len=0)):
        with pytest.raises(binding.RlkvError) as e:
            binding.rlkv_cache_size(**{**ok, **bad})
        assert e.value.code == binding.RLKV_EINVAL
    with pytest.raises(ValueError):
        binding.rlkv_cache_size(**{**ok, "head_is_full": [1, 0, 0]})
    m = np.ones(4, np.uint8)
    out = ctypes.c_size_t(0)
    assert binding.lib.rlkv_cache_size(0, 2, 8, 128, 3, 100, m.ctypes.data, 4, 12, ctypes.byref(out)) == binding.RLKV_EINVAL
    assert binding.lib.rlkv_cache_size(2, 2, 8, 128, 3, 100, None, 4, 12, ctypes.byref(out)) == binding.RLKV_EINVAL
    assert binding.lib.rlkv_cache_size(2, 2, 8, 128, 3, 100, m.ctypes.data, 4, 12, None) == binding.RLKV_EINVAL
    # null handles are refused, not dereferenced
    for call in (lambda: binding.rlkv_length(0, 0), lambda: binding.rlkv_step_bytes(0, 0),
                 lambda: binding.rlkv_launch_count(0), lambda: binding.rlkv_cache_destroy(0)):
        with pytest.raises(binding.RlkvError) as e:
            call()
        assert e.value.code == binding.RLKV_EINVAL


def test_package_fails_loudly_without_the_library(tmp_path):
    """A copy of the package without librlkv.so must raise on first use: there is no fallback."""
    import shutil
    import subprocess
    import sys
    pkg = tmp_path / "paper_2510_08525_b200"
    shutil.copytree(os.path.join(ROOT, "paper_2510_08525_b200"), pkg,
                    ignore=shutil.ignore_patterns("*.so", "__pycache__"))
    code = ("import paper_2510_08525_b200 as p\n"
            "try:\n    p.rlkv_cache_size\nexcept ImportError as e:\n    print('IMPORTERROR', 'no fallback' in str(e))\n")
    res = subprocess.run([sys.executable, "-c", code], cwd=tmp_path, capture_output=True, text=True)
    assert "IMPORTERROR True" in res.stdout, res.stdout + res.stderr


def test_paged_size_and_argument_checks_need_no_device(binding):
    """rlkv_paged_size is host arithmetic: the page pool grows with n_pages and with the number of
    full heads only, the ring pool with max_seqs and the number of compressed heads only, and
    neither with max_seq_len (beyond the page table)."""
    ok = dict(layers=2, kv_heads=2, q_heads=8, head_dim=128, max_seqs=3, n_pages=10, max_seq_len=1000,
              head_is_full=[1, 0, 0, 1], sink=4, window=60)
    size = binding.rlkv_paged_size(**ok)
    page_bytes = 2 * 64 * 128 * 2                       # K and V rows of one page of one full head
    ring_bytes = 2 * 64 * 128 * 2                       # sink + window = 64 rows, K and V
    assert size >= 2 * (10 * page_bytes + 3 * ring_bytes)
    more_pages = binding.rlkv_paged_size(**{**ok, "n_pages": 10 + 1000})
    assert more_pages - size == 2 * 1000 * page_bytes   # one full head per layer
    # request slots beyond the 512 a launch can serve cost their rings and page-table rows, no scratch
    a, b = (binding.rlkv_paged_size(**{**ok, "max_seqs": m}) for m in (600, 600 + 256))
    assert b - a == 2 * 256 * ring_bytes + 256 * 16 * 4     # 1000 tokens = 16 page-table entries
    for bad in (dict(head_dim=96), dict(q_heads=7), dict(window=0), dict(sink=-1), dict(max_seqs=0), dict(n_pages=0),
                dict(max_seq_len=0), dict(max_seq_len=65537), dict(max_seqs=70000)):
        with pytest.raises(binding.RlkvError) as e:
            binding.rlkv_paged_size(**{**ok, **bad})
        assert e.value.code == binding.RLKV_EINVAL
    for call in (lambda: binding.rlkv_paged_seq_open(0), lambda: binding.rlkv_paged_seq_close(0, 0),
                 lambda: binding.rlkv_paged_pages(0), lambda: binding.rlkv_paged_length(0, 0, 0),
                 lambda: binding.rlkv_paged_destroy(0)):
        with pytest.raises(binding.RlkvError) as e:
            call()
        assert e.value.code == binding.RLKV_EINVAL


def test_paged_fp8_size_is_half_the_pool(binding):
    """8-bit storage: a page of a full head and a 64-row ring tile are 16 KB (K codes and transposed V
    codes) where the 16-bit cache needs 32 KB; the rest of the buffer is the same."""
    ok = dict(layers=2, kv_heads=2, q_heads=8, head_dim=128, max_seqs=600, n_pages=10, max_seq_len=1000,
              head_is_full=[1, 0, 0, 1], sink=4, window=60)
    page16, page8 = 2 * 64 * 128 * 2, 2 * 64 * 128
    for grow, unit in ((dict(n_pages=10 + 1000), 2 * 1000), (dict(max_seqs=600 + 256), 2 * 256)):
        d16 = binding.rlkv_paged_size(**{**ok, **grow}) - binding.rlkv_paged_size(**ok)
        d8 = binding.rlkv_paged_size_fp8(**{**ok, **grow}) - binding.rlkv_paged_size_fp8(**ok)
        assert d16 - d8 == unit * (page16 - page8)
    with pytest.raises(binding.RlkvError) as e:
        binding.rlkv_paged_size_fp8(**{**ok, "head_dim": 64})
    assert e.value.code == binding.RLKV_EINVAL


def test_fp8_cache_size_needs_no_device(binding):
    """rlkv_cache_size_fp8: host arithmetic only.  The cache is the paged 8-bit cache with one slot per
    batch row and batch * ceil(max_len / 64) pages plus a staging area for one step's k, v, q and
    results; a longer cache grows by 16 KB per full head, batch row and 64 tokens."""
    ok = dict(layers=2, kv_heads=2, q_heads=8, head_dim=128, batch=3, max_len=1000, head_is_full=[1, 0, 1, 1], sink=4, window=60)
    base = binding.rlkv_cache_size_fp8(**ok)
    pages = 3 * ((1000 + 63) // 64)
    paged = binding.rlkv_paged_size_fp8(2, 2, 8, 128, 3, pages, 1000, [1, 0, 1, 1], 4, 60)
    staging = 2 * 2 * 3 * 2 * 128 * 2 + 2 * 3 * 8 * 128 * 2 + 2 * 3 * 8 * 128 * 4    # k, v; q; results in fp32
    assert paged <= base - staging < paged + 1024 + 4 * 256                          # alignment only
    longer = binding.rlkv_cache_size_fp8(**{**ok, "max_len": 1000 + 64 * 10})
    grown = longer - base
    codes = 3 * 10 * 3 * 2 * 64 * 128                     # 3 full heads, 10 more pages per batch row, 16 KB a page
    assert codes <= grown < codes + (1 << 16)             # the rest: page tables and partial records
    for bad in (dict(head_dim=64), dict(batch=0), dict(max_len=0), dict(q_heads=7), dict(window=0)):
        with pytest.raises(binding.RlkvError) as e:
            binding.rlkv_cache_size_fp8(**{**ok, **bad})
        assert e.value.code == binding.RLKV_EINVAL
