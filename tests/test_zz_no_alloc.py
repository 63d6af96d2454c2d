"""chunkkv_score_noalloc: the scoring entry point for callers that cannot allocate.

A serving process that gave every free byte of HBM to its own cache pool has no buffer left to
hand to chunkkv_set_workspace, and a plug-in that only sees raw pointers cannot reach an allocator
at all; they call this variant, whose scratch is a fixed 8 MiB array inside the library. It must
give the scores the method defines (checked against the CPU oracle and against chunkkv_score),
call after call (the array is shared and keeps old contents), leave the amount of free device
memory unchanged once warmed up, report an abandoned wait through its own status call, and refuse
shapes that do not fit. This file is collected last on purpose.
"""
import ctypes

import numpy as np
import pytest
import torch

from oracle import chunkkv_oracle as ora
from tests.helpers import Guarded, assert_scores_close, to_dev
from workloads import CONFIGS, make_layer, scaled

pytestmark = pytest.mark.gpu


def _lib():
    import paper_2502_00299_b200 as ck
    vp, i32 = ctypes.c_void_p, ctypes.c_int
    ck.lib.chunkkv_score_noalloc.restype = i32
    ck.lib.chunkkv_score_noalloc.argtypes = [vp, vp] + [i32] * 6 + [vp, vp]
    ck.lib.chunkkv_score_noalloc_status.restype = i32
    ck.lib.chunkkv_score_noalloc_status.argtypes = [vp]
    return ck


def _noalloc(ck, q, K, Hq, w, c, out):
    Hkv, L, d = K.shape
    return ck.lib.chunkkv_score_noalloc(q.data_ptr(), K.data_ptr(), L, Hq, Hkv, d, w, c, out.data_ptr(),
                                        torch.cuda.current_stream().cuda_stream or None)


def test_noalloc_scores_match_oracle_and_allocating_entry_point_twice_in_a_row():
    ck = _lib()
    # two different problems back to back: the second call sees the first call's leftovers
    cases = [(scaled(CONFIGS[2], L=4000), 0), (CONFIGS[1], 0), (scaled(CONFIGS[2], L=4000), 1)]
    warmed = False
    for wl, layer in cases:
        x = make_layer(wl, layer=layer)
        q, K = to_dev(x.q_obs), to_dev(x.K)
        assert ck.workspace_bytes(wl.L, wl.Hq, wl.Hkv, wl.d, wl.w, wl.c) <= 8 << 20
        ref, _ = ck.score(q, K, wl.w, wl.c)
        out = Guarded((wl.Hkv, ck.num_chunks(wl.L, wl.w, wl.c)), torch.float32)
        out.t.fill_(float("nan"))
        if not warmed:      # the warm-up call: the array's device address is looked up (and its memory taken) here
            assert _noalloc(ck, q, K, wl.Hq, wl.w, wl.c, out.t) == 0
            torch.cuda.synchronize()
            warmed = True
        free_before, _ = torch.cuda.mem_get_info()
        st = _noalloc(ck, q, K, wl.Hq, wl.w, wl.c, out.t)
        assert st == 0, ck.strerror(st)
        assert ck.lib.chunkkv_score_noalloc_status(torch.cuda.current_stream().cuda_stream or None) == 0
        free_after, _ = torch.cuda.mem_get_info()
        assert free_after == free_before, "a warm call changed the amount of free device memory"
        out.check("out_chunk_scores")
        R = wl.w * wl.Hq // wl.Hkv
        got = out.t.cpu().numpy()
        want = ora.chunk_scores(ora.token_scores(x.q_obs, x.K, wl.Hq, wl.Hkv, wl.w), wl.c)
        assert_scores_close(got, want, R, wl.L, f"{wl.name}: noalloc chunk scores vs oracle")
        assert_scores_close(got, ref.cpu().numpy().astype(np.float64), R, wl.L, f"{wl.name}: noalloc vs chunkkv_score")


def test_noalloc_refuses_what_does_not_fit_before_launching():
    ck = _lib()
    # a shape that needs more than the fixed scratch (real-size buffers, so that a regression shows
    # up as a wrong status code and not as a stray write)
    wl = CONFIGS[2]
    assert ck.workspace_bytes(wl.L, wl.Hq, wl.Hkv, wl.d, wl.w, wl.c) > 8 << 20
    q = torch.zeros((wl.Hq, wl.w, wl.d), dtype=torch.bfloat16, device="cuda")
    K = torch.zeros((wl.Hkv, wl.L, wl.d), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros((wl.Hkv, ck.num_chunks(wl.L, wl.w, wl.c)), dtype=torch.float32, device="cuda")
    st = _noalloc(ck, q, K, wl.Hq, wl.w, wl.c, out)
    assert st == -7 and "scratch" in ck.strerror(st)
    # a shape outside the library's limits (Hkv * L >= 2^23 keys) is a shape error here as everywhere
    assert ck.lib.chunkkv_score_noalloc(q.data_ptr(), K.data_ptr(), 1 << 20, 8, 8, 128, 1, 64, out.data_ptr(), None) == -2
    assert ck.lib.chunkkv_score_noalloc_status(None) == 0
