"""The C ABI without a GPU: the library loads, exports what the header declares, and its
host-side size rules and argument checks agree with the oracle's."""
import ctypes
import os
import re

import pytest

from oracle import chunkkv_oracle as ora

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def ck():
    from paper_2502_00299_b200 import build
    build.build()
    import paper_2502_00299_b200 as ck
    return ck


def test_library_exports_every_declared_symbol(ck):
    text = open(os.path.join(ROOT, "include", "chunkkv.h")).read()
    names = re.findall(r"CHUNKKV_API\s+[\w\s\*]+?\b(chunkkv_\w+)\s*\(", text)
    assert len(names) >= 15 and "chunkkv_compress_layer" in names
    raw = ctypes.CDLL(ck.LIB_PATH)
    for n in names:
        assert hasattr(raw, n), f"{n} declared in chunkkv.h but not exported"


@pytest.mark.parametrize("L,w,c,budget", [
    (2048, 16, 10, 256), (32768, 32, 10, 3276), (131072, 64, 20, 4096), (103, 8, 10, 43),
    (26, 4, 5, 1000), (26, 4, 5, 4), (4, 4, 5, 4), (100, 1, 1, 50), (57, 7, 1000, 2000),
])
def test_size_rules_match_the_oracle(ck, L, w, c, budget):
    assert ck.num_chunks(L, w, c) == ora.num_chunks(L, w, c)
    assert ck.num_kept_chunks(L, w, c, budget) == ora.num_kept_chunks(L, w, c, budget)
    assert ck.out_len(L, w, c, budget) == ora.out_len(L, w, c, budget)


def test_invalid_sizes_are_rejected_on_the_host(ck):
    lib = ck.lib
    assert lib.chunkkv_out_len(10, 32, 10, 64) == -2          # L < w
    assert lib.chunkkv_out_len(100, 8, 10, 7) == -2           # budget < w
    assert lib.chunkkv_out_len(100, 0, 10, 7) == -2
    assert lib.chunkkv_num_chunks(100, 8, 0) == -2
    # shape errors are reported before any pointer is touched or anything is launched
    assert lib.chunkkv_score(None, None, 1024, 8, 3, 128, 16, 10, None, None, None) == -2   # Hq % Hkv
    assert lib.chunkkv_score(None, None, 1024, 8, 2, 96, 16, 10, None, None, None) == -2    # d
    assert lib.chunkkv_score(None, None, 1024, 64, 2, 128, 16, 10, None, None, None) == -2  # R = 512
    assert lib.chunkkv_score(None, None, 1024, 8, 2, 128, 16, 10, None, None, None) == -1   # NULL
    assert lib.chunkkv_score(16, 32, 1024, 8, 2, 128, 16, 10, None, 8, None) == -3          # alignment
    assert lib.chunkkv_select(None, 1024, 2, 16, 10, 8, None, None) == -2
    assert lib.chunkkv_select(None, 1024, 2, 16, 10, 256, None, None) == -1
    assert lib.chunkkv_gather(None, None, None, 1024, 2, 128, 100, None, None, None) == -1
    assert lib.chunkkv_gather(16, 16, 16, 1024, 2, 100, 100, 16, 16, None) == -2
    assert lib.chunkkv_compress_layer(None, None, None, 1024, 8, 2, 128, 16, 10, 4, None, None, None,
                                      None, None) == -2
    assert lib.chunkkv_compress_layer(None, None, None, 1024, 8, 2, 128, 16, 10, 256, None, None, None,
                                      None, None) == -1
    # the largest supported head set is Hkv * L < 2^23 keys; one key more is refused
    assert lib.chunkkv_compress_layer(None, None, None, (1 << 20) - 1, 8, 8, 128, 16, 10, 256, None, None, None,
                                      None, None) == -1        # sizes accepted, then the NULL pointers are seen
    assert lib.chunkkv_compress_layer(None, None, None, 1 << 20, 8, 8, 128, 16, 10, 256, None, None, None,
                                      None, None) == -2
    # the fixed-scratch scoring call applies the same limits (8 heads of 2^20 keys is one key too many)
    assert lib.chunkkv_score_noalloc(16, 16, 1 << 20, 8, 8, 128, 1, 64, 16, None) == -2
    assert lib.chunkkv_score_noalloc(16, 16, 1024, 8, 3, 128, 16, 10, 16, None) == -2
    assert lib.chunkkv_score_noalloc(None, None, 1024, 8, 2, 128, 16, 10, None, None) == -1
    # adapters: shapes, then pointers
    assert lib.chunkkv_window_queries(None, 100, 10, 8, 2, 64, 16, None, None, None, None) == -2      # T < w
    assert lib.chunkkv_window_queries(None, 100, 20, 8, 2, 64, 16, None, None, None, None) == -2      # row too short
    assert lib.chunkkv_window_queries(None, 768, 20, 8, 2, 64, 16, None, None, None, None) == -1
    assert lib.chunkkv_gather_paged(16, 16, 16, 100, 2, 64, 10, 16, 0, 4, 16, 16, None) == -2          # page_size
    assert lib.chunkkv_gather_paged(16, 16, 16, 100, 2, 64, 10, None, 4, 4, 16, 16, None) == -1
    assert lib.chunkkv_compress_model(0, None, None, None, 1024, 8, 2, 128, 16, 10, 256, 1, None, None, None, None) == -2
    assert lib.chunkkv_compress_model(2, None, None, None, 1024, 8, 2, 128, 16, 10, 256, 1, None, None, None, None) == -1
    # the new entry points check their arguments the same way
    assert lib.chunkkv_jaccard(None, None, 2, 10, 10, None, None, None) == -1
    assert lib.chunkkv_jaccard(None, None, 0, 10, 10, None, None, None) == -2
    assert lib.chunkkv_pipe_layer(None, None, None, None, 1024, 8, 2, 128, 16, 10, 256, None, None, None, None) == -1
    assert lib.chunkkv_pipe_join(None, None) == -1 and lib.chunkkv_pipe_close(None) == -1
    for code in range(-6, 1):
        assert ck.strerror(code) and ck.strerror(code) != "unknown status"
    assert ck.strerror(-99) == "unknown status"
