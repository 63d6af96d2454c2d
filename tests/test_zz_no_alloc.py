"""chunkkv_score_noalloc: the scoring entry point for callers that cannot allocate.

Servers that give all free HBM to their own cache pool, or loops that cannot afford the
device-wide synchronisation of cudaMalloc, call this variant; its scratch is a fixed 8 MiB array
inside the library instead of an allocated workspace. It must give the same chunk scores as
chunkkv_score, call after call (the array is shared and keeps old contents), and refuse shapes
that do not fit. This file is collected last on purpose.
"""
import numpy as np
import pytest
import torch

from tests.helpers import SCORE_RTOL, score_atol, to_dev
from workloads import CONFIGS, make_layer, scaled

pytestmark = pytest.mark.gpu


def _noalloc(ck, q, K, Hq, w, c):
    Hkv, L, d = K.shape
    out = torch.full((Hkv, ck.num_chunks(L, w, c)), float("nan"), dtype=torch.float32, device=K.device)
    st = ck.lib.chunkkv_score_noalloc(q.data_ptr(), K.data_ptr(), L, Hq, Hkv, d, w, c, out.data_ptr(),
                                      torch.cuda.current_stream().cuda_stream or None)
    return st, out


def test_noalloc_scores_match_the_allocating_entry_point_twice_in_a_row():
    import ctypes
    import paper_2502_00299_b200 as ck
    vp, i32 = ctypes.c_void_p, ctypes.c_int
    ck.lib.chunkkv_score_noalloc.restype = i32
    ck.lib.chunkkv_score_noalloc.argtypes = [vp, vp] + [i32] * 6 + [vp, vp]
    # two different problems back to back: the second call sees the first call's leftovers
    cases = [(scaled(CONFIGS[2], L=4000), 0), (CONFIGS[1], 0), (scaled(CONFIGS[2], L=4000), 1)]
    for wl, layer in cases:
        x = make_layer(wl, layer=layer)
        q, K = to_dev(x.q_obs), to_dev(x.K)
        assert ck.workspace_bytes(wl.L, wl.Hq, wl.Hkv, wl.d, wl.w, wl.c) <= 8 << 20
        ref, _ = ck.score(q, K, wl.w, wl.c)
        st, got = _noalloc(ck, q, K, wl.Hq, wl.w, wl.c)
        assert st == 0, ck.strerror(st)
        torch.cuda.synchronize()
        R = wl.w * wl.Hq // wl.Hkv
        err = (got - ref).abs().cpu().numpy()
        tol = SCORE_RTOL * ref.abs().cpu().numpy() + score_atol(R, wl.L)
        assert np.all(err <= tol), f"{wl.name}: worst abs error {err.max():.3e}"
    assert ck.device_status() == 0
    # a shape that needs more than the fixed scratch is refused before anything is launched
    wl = CONFIGS[2]
    assert ck.workspace_bytes(wl.L, wl.Hq, wl.Hkv, wl.d, wl.w, wl.c) > 8 << 20
    x = make_layer(scaled(wl, L=600))
    q, K = to_dev(x.q_obs), to_dev(x.K)
    out = torch.zeros(8, dtype=torch.float32, device="cuda")
    st = ck.lib.chunkkv_score_noalloc(q.data_ptr(), K.data_ptr(), wl.L, wl.Hq, wl.Hkv, wl.d, wl.w, wl.c,
                                      out.data_ptr(), None)
    assert st == -7 and "scratch" in ck.strerror(st)
