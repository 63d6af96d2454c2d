"""ctypes binding of the C ABI declared in include/chunkkv.h (argument marshalling only)."""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence, Tuple

import torch

LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libchunkkv.so")


class ChunkKVError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib.chunkkv_strerror(status).decode()
        extra = f" (cuda error {lib.chunkkv_last_cuda_error()})" if status == -5 else ""
        super().__init__(f"{where}: {msg}{extra} [status {status}]")


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2502_00299_b200.build` "
            "(needs nvcc). This package has no fallback path.")
    L = ctypes.CDLL(LIB_PATH)
    vp, i32, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
    L.chunkkv_strerror.restype = ctypes.c_char_p
    L.chunkkv_strerror.argtypes = [i32]
    L.chunkkv_last_cuda_error.restype = i32
    L.chunkkv_last_cuda_error.argtypes = []
    for name, n in (("chunkkv_num_chunks", 3), ("chunkkv_num_kept_chunks", 4), ("chunkkv_out_len", 4)):
        getattr(L, name).restype = i32
        getattr(L, name).argtypes = [i32] * n
    L.chunkkv_workspace_bytes.restype = sz
    L.chunkkv_workspace_bytes.argtypes = [i32] * 6
    L.chunkkv_set_workspace.restype = i32
    L.chunkkv_set_workspace.argtypes = [vp, sz]
    L.chunkkv_device_status.restype = i32
    L.chunkkv_device_status.argtypes = [vp]
    L.chunkkv_score.restype = i32
    L.chunkkv_score.argtypes = [vp, vp] + [i32] * 6 + [vp, vp, vp]
    L.chunkkv_select.restype = i32
    L.chunkkv_select.argtypes = [vp] + [i32] * 5 + [vp, vp]
    L.chunkkv_gather.restype = i32
    L.chunkkv_gather.argtypes = [vp, vp, vp] + [i32] * 4 + [vp, vp, vp]
    L.chunkkv_compress_layer.restype = i32
    L.chunkkv_compress_layer.argtypes = [vp, vp, vp] + [i32] * 7 + [vp, vp, vp, vp, vp]
    L.chunkkv_model_workspace_bytes.restype = sz
    L.chunkkv_model_workspace_bytes.argtypes = [i32] * 9
    L.chunkkv_compress_model_strided.restype = i32
    L.chunkkv_compress_model_strided.argtypes = [i32, vp, vp, vp] + [i32] * 8 + [ctypes.c_longlong] * 4 + [vp, vp, vp, vp]
    L.chunkkv_compress_model_paged.restype = i32
    L.chunkkv_compress_model_paged.argtypes = [i32, vp, vp, vp] + [i32] * 8 + [vp, i32, i32, vp, vp, vp, vp]
    L.chunkkv_compress_model.restype = i32
    L.chunkkv_compress_model.argtypes = [i32, vp, vp, vp] + [i32] * 8 + [vp, vp, vp, vp]
    L.chunkkv_window_queries.restype = i32
    L.chunkkv_window_queries.argtypes = [vp, ctypes.c_longlong] + [i32] * 5 + [vp, vp, vp, vp]
    L.chunkkv_gather_paged.restype = i32
    L.chunkkv_gather_paged.argtypes = [vp, vp, vp] + [i32] * 4 + [vp, i32, i32, vp, vp, vp]
    L.chunkkv_compress_layer_strided.restype = i32
    L.chunkkv_compress_layer_strided.argtypes = [vp, vp, vp] + [i32] * 7 + [ctypes.c_longlong] * 4 + [vp, vp, vp, vp, vp]
    L.chunkkv_compress_layer_paged.restype = i32
    L.chunkkv_compress_layer_paged.argtypes = [vp, vp, vp] + [i32] * 7 + [vp, vp, i32, i32, vp, vp, vp, vp]
    L.chunkkv_compress_layer_host.restype = i32
    L.chunkkv_compress_layer_host.argtypes = [vp, vp, vp] + [i32] * 7 + [vp] * 10
    L.chunkkv_lane_bytes.restype = sz
    L.chunkkv_lane_bytes.argtypes = [i32] * 7
    L.chunkkv_lane_init.restype = i32
    L.chunkkv_lane_init.argtypes = [vp, sz, vp]
    L.chunkkv_lane_status.restype = i32
    L.chunkkv_lane_status.argtypes = [vp, vp]
    L.chunkkv_compress_layer_lane.restype = i32
    L.chunkkv_compress_layer_lane.argtypes = [vp, vp, vp] + [i32] * 7 + [vp, vp, vp, vp, vp, sz, i32, vp]
    L.chunkkv_pipe_bytes.restype = sz
    L.chunkkv_pipe_bytes.argtypes = [i32] * 7
    L.chunkkv_pipe_open.restype = i32
    L.chunkkv_pipe_open.argtypes = [vp, sz, i32, ctypes.POINTER(vp)]
    L.chunkkv_pipe_layer.restype = i32
    L.chunkkv_pipe_layer.argtypes = [vp, vp, vp, vp] + [i32] * 7 + [vp, vp, vp, vp]
    L.chunkkv_pipe_join.restype = i32
    L.chunkkv_pipe_join.argtypes = [vp, vp]
    L.chunkkv_pipe_status.restype = i32
    L.chunkkv_pipe_status.argtypes = [vp, vp]
    L.chunkkv_pipe_close.restype = i32
    L.chunkkv_pipe_close.argtypes = [vp]
    L.chunkkv_jaccard.restype = i32
    L.chunkkv_jaccard.argtypes = [vp, vp, i32, i32, i32, vp, vp, vp]
    L.chunkkv_score_noalloc.restype = i32
    L.chunkkv_score_noalloc.argtypes = [vp, vp] + [i32] * 6 + [vp, vp]
    L.chunkkv_score_noalloc_status.restype = i32
    L.chunkkv_score_noalloc_status.argtypes = [vp]
    L.chunkkv_budget_from_ratio.restype = i32
    L.chunkkv_budget_from_ratio.argtypes = [i32, ctypes.c_double]
    L.chunkkv_num_kept_chunks_alg1.restype = i32
    L.chunkkv_num_kept_chunks_alg1.argtypes = [i32] * 4
    L.chunkkv_out_len_alg1.restype = i32
    L.chunkkv_out_len_alg1.argtypes = [i32] * 4
    L.chunkkv_select_alg1.restype = i32
    L.chunkkv_select_alg1.argtypes = [vp, i32, i32, i32, i32, i32, vp, vp]
    L.chunkkv_compress_layer_alg1.restype = i32
    L.chunkkv_compress_layer_alg1.argtypes = [vp, vp, vp] + [i32] * 7 + [vp, vp, vp, vp]
    L.chunkkv_profile_enable.restype = i32
    L.chunkkv_profile_enable.argtypes = [i32]
    L.chunkkv_profile_read.restype = i32
    L.chunkkv_profile_read.argtypes = [ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_int)]
    return L


lib = _load()


def _check(status: int, where: str) -> None:
    if status != 0:
        raise ChunkKVError(status, where)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream(stream: Optional[torch.cuda.Stream]) -> Optional[int]:
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream or None


def _dev(t: torch.Tensor, dtype: torch.dtype, name: str) -> torch.Tensor:
    if not t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise ValueError(f"{name} must be a contiguous CUDA tensor of dtype {dtype}")
    return t


def strerror(status: int) -> str:
    return lib.chunkkv_strerror(status).decode()


def num_chunks(L: int, w: int, c: int) -> int:
    v = lib.chunkkv_num_chunks(L, w, c)
    _check(min(v, 0), "chunkkv_num_chunks")
    return v


def num_kept_chunks(L: int, w: int, c: int, budget: int) -> int:
    v = lib.chunkkv_num_kept_chunks(L, w, c, budget)
    _check(min(v, 0), "chunkkv_num_kept_chunks")
    return v


def out_len(L: int, w: int, c: int, budget: int) -> int:
    v = lib.chunkkv_out_len(L, w, c, budget)
    _check(min(v, 0), "chunkkv_out_len")
    return v


def workspace_bytes(L: int, Hq: int, Hkv: int, d: int, w: int, c: int) -> int:
    return int(lib.chunkkv_workspace_bytes(L, Hq, Hkv, d, w, c))


_workspaces = {}      # device index -> uint8 tensor currently handed to the library


def set_workspace(buf: Optional[torch.Tensor]) -> None:
    """Hand the library a caller-owned scratch buffer (uint8 CUDA tensor on the current device), or
    None to detach it. The library itself never allocates; see ensure_workspace."""
    dev = torch.cuda.current_device()
    if buf is None:
        _check(lib.chunkkv_set_workspace(None, 0), "chunkkv_set_workspace")
        _workspaces.pop(dev, None)
    else:
        _check(lib.chunkkv_set_workspace(buf.data_ptr(), buf.numel() * buf.element_size()),
               "chunkkv_set_workspace")
        _workspaces[dev] = buf


def ensure_workspace(L: int, Hq: int, Hkv: int, d: int, w: int, c: int) -> None:
    """Make sure the current device's scratch covers this shape: the device memory is a torch
    tensor allocated here (grown when a larger shape arrives) and handed over with
    chunkkv_set_workspace. A buffer given through set_workspace is kept if it is large enough."""
    need = workspace_bytes(L, Hq, Hkv, d, w, c)
    if need == 0:
        raise ChunkKVError(-2, "chunkkv_workspace_bytes")
    dev = torch.cuda.current_device()
    cur = _workspaces.get(dev)
    if cur is not None and cur.numel() >= need:
        return
    set_workspace(torch.empty(need + (need >> 2), dtype=torch.uint8, device=torch.device("cuda", dev)))


def device_status(stream: Optional[torch.cuda.Stream] = None) -> int:
    """Synchronises the stream; returns 0 or CHUNKKV_EDEVICE (-6)."""
    return lib.chunkkv_device_status(_stream(stream))


def score(q_obs: torch.Tensor, K: torch.Tensor, w: int, c: int, want_token_scores: bool = False,
          stream: Optional[torch.cuda.Stream] = None) -> Tuple[torch.Tensor, Optional[torch.Tensor]]:
    """chunk scores [Hkv, C] f32 (and token scores [Hkv, P] f32 if asked)."""
    _dev(q_obs, torch.bfloat16, "q_obs"); _dev(K, torch.bfloat16, "K")
    Hq, d = q_obs.shape[0], q_obs.shape[2]
    Hkv, L = K.shape[0], K.shape[1]
    C = num_chunks(L, w, c)
    ensure_workspace(L, Hq, Hkv, d, w, c)
    if want_token_scores:
        ensure_workspace(L, Hq, Hkv, d, w, 1)
    cs = torch.empty((Hkv, C), dtype=torch.float32, device=K.device)
    ts = torch.empty((Hkv, L - w), dtype=torch.float32, device=K.device) if want_token_scores else None
    _check(lib.chunkkv_score(q_obs.data_ptr(), K.data_ptr(), L, Hq, Hkv, d, w, c, _ptr(ts),
                             cs.data_ptr(), _stream(stream)), "chunkkv_score")
    return cs, ts


def select(chunk_scores: torch.Tensor, L: int, w: int, c: int, budget: int,
           stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """idx [Hkv, n_max] int32 from chunk scores [Hkv, C] f32."""
    _dev(chunk_scores, torch.float32, "chunk_scores")
    Hkv = chunk_scores.shape[0]
    n_max = out_len(L, w, c, budget)
    idx = torch.empty((Hkv, n_max), dtype=torch.int32, device=chunk_scores.device)
    _check(lib.chunkkv_select(chunk_scores.data_ptr(), L, Hkv, w, c, budget, idx.data_ptr(),
                              _stream(stream)), "chunkkv_select")
    return idx


def budget_from_ratio(L: int, ratio: float) -> int:
    v = lib.chunkkv_budget_from_ratio(L, float(ratio))
    _check(min(v, 0), "chunkkv_budget_from_ratio")
    return v


def out_len_alg1(L: int, w: int, c: int, budget: int) -> int:
    v = lib.chunkkv_out_len_alg1(L, w, c, budget)
    _check(min(v, 0), "chunkkv_out_len_alg1")
    return v


def select_alg1(chunk_scores: torch.Tensor, L: int, w: int, c: int, budget: int,
                stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """idx [Hkv, n_max] int32 from chunk scores [Hkv, C] f32 under Algorithm 1's budget rule."""
    _dev(chunk_scores, torch.float32, "chunk_scores")
    Hkv = chunk_scores.shape[0]
    idx = torch.empty((Hkv, out_len_alg1(L, w, c, budget)), dtype=torch.int32, device=chunk_scores.device)
    _check(lib.chunkkv_select_alg1(chunk_scores.data_ptr(), L, Hkv, w, c, budget, idx.data_ptr(),
                                   _stream(stream)), "chunkkv_select_alg1")
    return idx


def compress_layer_alg1(q_obs: torch.Tensor, K: torch.Tensor, V: torch.Tensor, Hq: int, w: int, c: int, budget: int,
                        out_K: Optional[torch.Tensor] = None, out_V: Optional[torch.Tensor] = None,
                        out_idx: Optional[torch.Tensor] = None,
                        stream: Optional[torch.cuda.Stream] = None) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
    """out_K, out_V [Hkv, n_max, d], idx [Hkv, n_max] for one layer under Algorithm 1's budget rule."""
    _dev(q_obs, torch.bfloat16, "q_obs"); _dev(K, torch.bfloat16, "K"); _dev(V, torch.bfloat16, "V")
    Hkv, L, d = K.shape
    n_max = out_len_alg1(L, w, c, budget)
    ensure_workspace(L, Hq, Hkv, d, w, c)
    if out_K is None:
        out_K = torch.empty((Hkv, n_max, d), dtype=torch.bfloat16, device=K.device)
    if out_V is None:
        out_V = torch.empty((Hkv, n_max, d), dtype=torch.bfloat16, device=K.device)
    idx = out_idx if out_idx is not None else torch.empty((Hkv, n_max), dtype=torch.int32, device=K.device)
    _check(lib.chunkkv_compress_layer_alg1(q_obs.data_ptr(), K.data_ptr(), V.data_ptr(), L, Hq, Hkv, d, w, c, budget,
                                           out_K.data_ptr(), out_V.data_ptr(), idx.data_ptr(), _stream(stream)),
           "chunkkv_compress_layer_alg1")
    return out_K, out_V, idx


def gather(K: torch.Tensor, V: torch.Tensor, idx: torch.Tensor,
           out_K: Optional[torch.Tensor] = None, out_V: Optional[torch.Tensor] = None,
           stream: Optional[torch.cuda.Stream] = None) -> Tuple[torch.Tensor, torch.Tensor]:
    """out_K, out_V [Hkv, n_max, d] = K, V rows at idx [Hkv, n_max] (zero rows where idx < 0)."""
    _dev(K, torch.bfloat16, "K"); _dev(V, torch.bfloat16, "V"); _dev(idx, torch.int32, "idx")
    Hkv, L, d = K.shape
    n_max = idx.shape[1]
    if out_K is None:
        out_K = torch.empty((Hkv, n_max, d), dtype=torch.bfloat16, device=K.device)
    if out_V is None:
        out_V = torch.empty((Hkv, n_max, d), dtype=torch.bfloat16, device=K.device)
    _check(lib.chunkkv_gather(K.data_ptr(), V.data_ptr(), idx.data_ptr(), L, Hkv, d, n_max,
                              out_K.data_ptr(), out_V.data_ptr(), _stream(stream)), "chunkkv_gather")
    return out_K, out_V


def compress_layer(q_obs: Optional[torch.Tensor], K: torch.Tensor, V: torch.Tensor, Hq: int, w: int,
                   c: int, budget: int, reuse_idx: Optional[torch.Tensor] = None,
                   out_K: Optional[torch.Tensor] = None, out_V: Optional[torch.Tensor] = None,
                   out_idx: Optional[torch.Tensor] = None,
                   stream: Optional[torch.cuda.Stream] = None,
                   ) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
    """One layer: score -> chunk-sum -> top-k -> gather, or gather only with ``reuse_idx``."""
    _dev(K, torch.bfloat16, "K"); _dev(V, torch.bfloat16, "V")
    if q_obs is not None:
        _dev(q_obs, torch.bfloat16, "q_obs")
    if reuse_idx is not None:
        _dev(reuse_idx, torch.int32, "reuse_idx")
    Hkv, L, d = K.shape
    n_max = out_len(L, w, c, budget)
    dev = K.device
    if reuse_idx is None:
        ensure_workspace(L, Hq, Hkv, d, w, c)
    if out_K is None:
        out_K = torch.empty((Hkv, n_max, d), dtype=torch.bfloat16, device=dev)
    if out_V is None:
        out_V = torch.empty((Hkv, n_max, d), dtype=torch.bfloat16, device=dev)
    if out_idx is None:
        out_idx = torch.empty((Hkv, n_max), dtype=torch.int32, device=dev)
    _check(lib.chunkkv_compress_layer(_ptr(q_obs), K.data_ptr(), V.data_ptr(), L, Hq, Hkv, d, w, c,
                                      budget, _ptr(reuse_idx), out_K.data_ptr(), out_V.data_ptr(),
                                      out_idx.data_ptr(), _stream(stream)), "chunkkv_compress_layer")
    return out_K, out_V, out_idx


def window_queries(qkv: torch.Tensor, Hq: int, Hkv: int, d: int, w: int, cos_rows: torch.Tensor,
                   sin_rows: torch.Tensor, stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """q_obs [Hq, w, d] bf16 from the last w rows of a fused QKV activation [T, row_elems] bf16,
    with the rotary embedding of those rows applied (cos_rows, sin_rows [w, d / 2] f32)."""
    _dev(qkv, torch.bfloat16, "qkv"); _dev(cos_rows, torch.float32, "cos_rows"); _dev(sin_rows, torch.float32, "sin_rows")
    T, row_elems = qkv.shape
    out = torch.empty((Hq, w, d), dtype=torch.bfloat16, device=qkv.device)
    _check(lib.chunkkv_window_queries(qkv.data_ptr(), row_elems, T, Hq, Hkv, d, w, cos_rows.data_ptr(),
                                      sin_rows.data_ptr(), out.data_ptr(), _stream(stream)), "chunkkv_window_queries")
    return out


def gather_paged(K: torch.Tensor, V: torch.Tensor, idx: torch.Tensor, block_table: torch.Tensor, cache_K: torch.Tensor,
                 cache_V: torch.Tensor, stream: Optional[torch.cuda.Stream] = None) -> None:
    """Kept rows into a paged cache [num_pages, page_size, Hkv, d] through block_table (int32)."""
    _dev(K, torch.bfloat16, "K"); _dev(V, torch.bfloat16, "V"); _dev(idx, torch.int32, "idx")
    _dev(block_table, torch.int32, "block_table"); _dev(cache_K, torch.bfloat16, "cache_K"); _dev(cache_V, torch.bfloat16, "cache_V")
    Hkv, L, d = K.shape
    _check(lib.chunkkv_gather_paged(K.data_ptr(), V.data_ptr(), idx.data_ptr(), L, Hkv, d, idx.shape[1],
                                    block_table.data_ptr(), cache_K.shape[1], cache_K.shape[0], cache_K.data_ptr(),
                                    cache_V.data_ptr(), _stream(stream)), "chunkkv_gather_paged")


def compress_layer_strided(q_obs: Optional[torch.Tensor], K: torch.Tensor, V: torch.Tensor, Hq: int, w: int, c: int,
                           budget: int, reuse_idx: Optional[torch.Tensor] = None,
                           out_K: Optional[torch.Tensor] = None, out_V: Optional[torch.Tensor] = None,
                           out_idx: Optional[torch.Tensor] = None,
                           stream: Optional[torch.cuda.Stream] = None) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
    """One layer on K / V given as [Hkv, L, d] *views* with arbitrary token and head strides (the last
    dimension contiguous), e.g. ``cache.permute(1, 0, 2)`` of a token-major cache [L, Hkv, d]. Outputs
    are packed [Hkv, n_max, d]."""
    for t, name in ((K, "K"), (V, "V")):
        if not (t.is_cuda and t.dtype == torch.bfloat16 and t.dim() == 3 and t.stride(2) == 1):
            raise ValueError(f"{name}: a CUDA bf16 [Hkv, L, d] view with a contiguous last dimension is required")
    if q_obs is not None:
        _dev(q_obs, torch.bfloat16, "q_obs")
    if reuse_idx is not None:
        _dev(reuse_idx, torch.int32, "reuse_idx")
    Hkv, L, d = K.shape
    n_max = out_len(L, w, c, budget)
    dev = K.device
    if reuse_idx is None:
        ensure_workspace(L, Hq, Hkv, d, w, c)
    if out_K is None:
        out_K = torch.empty((Hkv, n_max, d), dtype=torch.bfloat16, device=dev)
    if out_V is None:
        out_V = torch.empty((Hkv, n_max, d), dtype=torch.bfloat16, device=dev)
    if out_idx is None:
        out_idx = torch.empty((Hkv, n_max), dtype=torch.int32, device=dev)
    _check(lib.chunkkv_compress_layer_strided(_ptr(q_obs), K.data_ptr(), V.data_ptr(), L, Hq, Hkv, d, w, c, budget,
                                              K.stride(1), K.stride(0), V.stride(1), V.stride(0), _ptr(reuse_idx),
                                              out_K.data_ptr(), out_V.data_ptr(), out_idx.data_ptr(), _stream(stream)),
           "chunkkv_compress_layer_strided")
    return out_K, out_V, out_idx


def compress_layer_paged(q_obs: Optional[torch.Tensor], K: torch.Tensor, V: torch.Tensor, Hq: int, w: int, c: int,
                         budget: int, block_table: torch.Tensor, cache_K: torch.Tensor, cache_V: torch.Tensor,
                         reuse_idx: Optional[torch.Tensor] = None, out_idx: Optional[torch.Tensor] = None,
                         stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """One layer into a paged cache; returns idx [Hkv, n_max]."""
    Hkv, L, d = K.shape
    n_max = out_len(L, w, c, budget)
    if reuse_idx is None:
        ensure_workspace(L, Hq, Hkv, d, w, c)
    if out_idx is None:
        out_idx = torch.empty((Hkv, n_max), dtype=torch.int32, device=K.device)
    _check(lib.chunkkv_compress_layer_paged(_ptr(q_obs), K.data_ptr(), V.data_ptr(), L, Hq, Hkv, d, w, c, budget,
                                            _ptr(reuse_idx), block_table.data_ptr(), cache_K.shape[1], cache_K.shape[0],
                                            cache_K.data_ptr(), cache_V.data_ptr(), out_idx.data_ptr(), _stream(stream)),
           "chunkkv_compress_layer_paged")
    return out_idx


def jaccard(idx_a: torch.Tensor, idx_b: torch.Tensor, stream: Optional[torch.cuda.Stream] = None,
            ) -> Tuple[torch.Tensor, torch.Tensor]:
    """chunkkv_jaccard: per-head similarity [Hkv] f32 and counts [Hkv, 3] int32 (|A n B|, |A|, |B|)."""
    idx_a = _dev(idx_a, torch.int32, "idx_a")
    idx_b = _dev(idx_b, torch.int32, "idx_b")
    Hkv = idx_a.shape[0]
    if idx_b.shape[0] != Hkv:
        raise ValueError("idx_a and idx_b must have the same number of heads")
    ratio = torch.empty(Hkv, dtype=torch.float32, device=idx_a.device)
    counts = torch.empty((Hkv, 3), dtype=torch.int32, device=idx_a.device)
    _check(lib.chunkkv_jaccard(idx_a.data_ptr(), idx_b.data_ptr(), Hkv, idx_a.shape[1], idx_b.shape[1],
                               ratio.data_ptr(), counts.data_ptr(), _stream(stream)), "chunkkv_jaccard")
    return ratio, counts


class Lane:
    """Caller-owned scratch plus a CTA budget: layers submitted to different lanes on different
    streams run concurrently (see chunkkv.h). The budgets of lanes used at the same time must add
    up to at most the number of SMs."""

    def __init__(self, L: int, Hq: int, Hkv: int, d: int, w: int, c: int, max_ctas: int = 0,
                 device: Optional[torch.device] = None, stream: Optional[torch.cuda.Stream] = None,
                 buf: Optional[torch.Tensor] = None):
        self.max_ctas = int(max_ctas)
        self.bytes = int(lib.chunkkv_lane_bytes(L, Hq, Hkv, d, w, c, self.max_ctas))
        if self.bytes == 0:
            raise ChunkKVError(-2, "chunkkv_lane_bytes")
        if buf is not None and buf.numel() * buf.element_size() < self.bytes:
            raise ValueError("the given scratch tensor is smaller than chunkkv_lane_bytes")
        self.buf = buf if buf is not None else torch.empty(self.bytes, dtype=torch.uint8, device=device or "cuda")
        self.stream = stream if stream is not None else torch.cuda.Stream(device=self.buf.device)
        _check(lib.chunkkv_lane_init(self.buf.data_ptr(), self.bytes, self.stream.cuda_stream or None),
               "chunkkv_lane_init")

    def status(self) -> int:
        return lib.chunkkv_lane_status(self.buf.data_ptr(), self.stream.cuda_stream or None)

    def compress_layer(self, q_obs: Optional[torch.Tensor], K: torch.Tensor, V: torch.Tensor, Hq: int, w: int,
                       c: int, budget: int, reuse_idx: Optional[torch.Tensor] = None,
                       out_K: Optional[torch.Tensor] = None, out_V: Optional[torch.Tensor] = None,
                       out_idx: Optional[torch.Tensor] = None,
                       ) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
        """chunkkv_compress_layer_lane on this lane's stream."""
        Hkv, L, d = K.shape
        n_max = out_len(L, w, c, budget)
        dev = K.device
        with torch.cuda.stream(self.stream):
            if out_K is None:
                out_K = torch.empty((Hkv, n_max, d), dtype=torch.bfloat16, device=dev)
            if out_V is None:
                out_V = torch.empty((Hkv, n_max, d), dtype=torch.bfloat16, device=dev)
            if out_idx is None:
                out_idx = torch.empty((Hkv, n_max), dtype=torch.int32, device=dev)
        _check(lib.chunkkv_compress_layer_lane(
            _ptr(q_obs), K.data_ptr(), V.data_ptr(), L, Hq, Hkv, d, w, c, budget, _ptr(reuse_idx),
            out_K.data_ptr(), out_V.data_ptr(), out_idx.data_ptr(), self.buf.data_ptr(), self.bytes,
            self.max_ctas, self.stream.cuda_stream or None), "chunkkv_compress_layer_lane")
        return out_K, out_V, out_idx


class Pipe:
    """A lane whose layers overlap each other (see chunkkv.h): scoring kernels back to back on
    `stream`, everything after scoring on the pipe's own stream. Call join() before using outputs."""

    def __init__(self, L: int, Hq: int, Hkv: int, d: int, w: int, c: int, max_ctas: int = 0,
                 device: Optional[torch.device] = None, stream: Optional[torch.cuda.Stream] = None,
                 buf: Optional[torch.Tensor] = None):
        self.max_ctas = int(max_ctas)
        self.bytes = int(lib.chunkkv_pipe_bytes(L, Hq, Hkv, d, w, c, self.max_ctas))
        if self.bytes == 0:
            raise ChunkKVError(-2, "chunkkv_pipe_bytes")
        if buf is not None and buf.numel() * buf.element_size() < self.bytes:
            raise ValueError("the given scratch tensor is smaller than chunkkv_pipe_bytes")
        self.buf = buf if buf is not None else torch.empty(self.bytes, dtype=torch.uint8, device=device or "cuda")
        self.stream = stream if stream is not None else torch.cuda.Stream(device=self.buf.device)
        handle = ctypes.c_void_p()
        _check(lib.chunkkv_pipe_open(self.buf.data_ptr(), self.bytes, self.max_ctas, ctypes.byref(handle)),
               "chunkkv_pipe_open")
        self.handle = handle

    def layer(self, q_obs: torch.Tensor, K: torch.Tensor, V: torch.Tensor, Hq: int, w: int, c: int, budget: int,
              out_K: Optional[torch.Tensor] = None, out_V: Optional[torch.Tensor] = None,
              out_idx: Optional[torch.Tensor] = None) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
        """chunkkv_pipe_layer; the outputs are complete after join()."""
        Hkv, L, d = K.shape
        n_max = out_len(L, w, c, budget)
        dev = K.device
        with torch.cuda.stream(self.stream):
            if out_K is None:
                out_K = torch.empty((Hkv, n_max, d), dtype=torch.bfloat16, device=dev)
            if out_V is None:
                out_V = torch.empty((Hkv, n_max, d), dtype=torch.bfloat16, device=dev)
            if out_idx is None:
                out_idx = torch.empty((Hkv, n_max), dtype=torch.int32, device=dev)
        _check(lib.chunkkv_pipe_layer(self.handle, q_obs.data_ptr(), K.data_ptr(), V.data_ptr(), L, Hq, Hkv, d, w, c,
                                      budget, out_K.data_ptr(), out_V.data_ptr(), out_idx.data_ptr(),
                                      self.stream.cuda_stream or None), "chunkkv_pipe_layer")
        return out_K, out_V, out_idx

    def join(self) -> None:
        _check(lib.chunkkv_pipe_join(self.handle, self.stream.cuda_stream or None), "chunkkv_pipe_join")

    def status(self) -> int:
        return lib.chunkkv_pipe_status(self.handle, self.stream.cuda_stream or None)

    def close(self) -> None:
        if self.handle is not None:
            _check(lib.chunkkv_pipe_close(self.handle), "chunkkv_pipe_close")
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def compress_layer_host(host_q: torch.Tensor, host_K: torch.Tensor, host_V: torch.Tensor, Hq: int,
                        w: int, c: int, budget: int, dev_bufs: Sequence[torch.Tensor],
                        host_outs: Sequence[torch.Tensor],
                        stream: Optional[torch.cuda.Stream] = None) -> None:
    """Host tensors in, host tensors out; ``dev_bufs`` = (q, K, V, out_K, out_V, out_idx) staging
    tensors on the GPU, ``host_outs`` = (out_K, out_V, out_idx) host tensors (pinned for speed)."""
    Hkv, L, d = host_K.shape
    dq, dK, dV, doK, doV, dI = dev_bufs
    hK, hV, hI = host_outs
    ensure_workspace(L, Hq, Hkv, d, w, c)
    _check(lib.chunkkv_compress_layer_host(
        host_q.data_ptr(), host_K.data_ptr(), host_V.data_ptr(), L, Hq, Hkv, d, w, c, budget,
        dq.data_ptr(), dK.data_ptr(), dV.data_ptr(), doK.data_ptr(), doV.data_ptr(), dI.data_ptr(),
        hK.data_ptr(), hV.data_ptr(), hI.data_ptr(), _stream(stream)), "chunkkv_compress_layer_host")


def _ensure_bytes(need: int) -> None:
    dev = torch.cuda.current_device()
    cur = _workspaces.get(dev)
    if cur is None or cur.numel() < need:
        set_workspace(torch.empty(need + (need >> 2), dtype=torch.uint8, device=torch.device("cuda", dev)))


def compress_model(layers: Sequence[Tuple[Optional[torch.Tensor], torch.Tensor, torch.Tensor]], Hq: int, w: int,
                   c, budget: int, n_reuse: int = 1,
                   stream: Optional[torch.cuda.Stream] = None,
                   outs: Optional[Sequence[Tuple[torch.Tensor, torch.Tensor, torch.Tensor]]] = None,
                   ) -> List[Tuple[torch.Tensor, torch.Tensor, torch.Tensor]]:
    """Layer-wise index reuse: layer l computes indices iff l % n_reuse == 0, otherwise it
    gathers with the indices of layer (l // n_reuse) * n_reuse. ``layers`` = (q_obs, K, V) per layer
    (q_obs may be None for layers that reuse). With one chunk size for all layers this is one
    chunkkv_compress_model call; with one chunk size per layer (chunk-level layers followed by
    token-level ones, c = 1) it is the same call sequence over chunkkv_compress_layer, a layer that
    reuses indices taking its source layer's chunk size. Only marshalling lives here."""
    n = len(layers)
    if not isinstance(c, int):
        cs = [int(v) for v in c]
        if len(cs) != n:
            raise ValueError("one chunk size per layer expected")
        res: List[Tuple[torch.Tensor, torch.Tensor, torch.Tensor]] = []
        for l, (q, K, V) in enumerate(layers):
            o = outs[l] if outs is not None else (None, None, None)
            if l % n_reuse == 0:
                res.append(compress_layer(q, K, V, Hq, w, cs[l], budget, out_K=o[0], out_V=o[1], out_idx=o[2], stream=stream))
            else:
                s_l = (l // n_reuse) * n_reuse
                res.append(compress_layer(None, K, V, Hq, w, cs[s_l], budget, reuse_idx=res[s_l][2], out_K=o[0],
                                          out_V=o[1], out_idx=o[2], stream=stream))
        return res
    Hkv, L, d = layers[0][1].shape
    for q, K, V in layers:
        _dev(K, torch.bfloat16, "K"); _dev(V, torch.bfloat16, "V")
        if q is not None:
            _dev(q, torch.bfloat16, "q_obs")
        if tuple(K.shape) != (Hkv, L, d) or tuple(V.shape) != (Hkv, L, d):
            raise ValueError("all layers must share one K/V shape")
    n_max = out_len(L, w, c, budget)
    dev = layers[0][1].device
    if outs is None:
        outs = [(torch.empty((Hkv, n_max, d), dtype=torch.bfloat16, device=dev),
                 torch.empty((Hkv, n_max, d), dtype=torch.bfloat16, device=dev),
                 torch.empty((Hkv, n_max), dtype=torch.int32, device=dev)) for _ in range(n)]
    _ensure_bytes(int(lib.chunkkv_model_workspace_bytes(n, L, Hq, Hkv, d, w, c, budget, n_reuse)))
    arr = ctypes.c_void_p * n
    qa = arr(*[None if t[0] is None else t[0].data_ptr() for t in layers])
    ka = arr(*[t[1].data_ptr() for t in layers])
    va = arr(*[t[2].data_ptr() for t in layers])
    oka = arr(*[o[0].data_ptr() for o in outs])
    ova = arr(*[o[1].data_ptr() for o in outs])
    oia = arr(*[o[2].data_ptr() for o in outs])
    _check(lib.chunkkv_compress_model(n, qa, ka, va, L, Hq, Hkv, d, w, c, budget, n_reuse, oka, ova, oia,
                                      _stream(stream)), "chunkkv_compress_model")
    return [tuple(o) for o in outs]


def compress_model_strided(layers: Sequence[Tuple[Optional[torch.Tensor], torch.Tensor, torch.Tensor]], Hq: int, w: int,
                           c: int, budget: int, n_reuse: int = 1,
                           stream: Optional[torch.cuda.Stream] = None,
                           outs: Optional[Sequence[Tuple[torch.Tensor, torch.Tensor, torch.Tensor]]] = None,
                           ) -> List[Tuple[torch.Tensor, torch.Tensor, torch.Tensor]]:
    """compress_model on K / V given as [Hkv, L, d] views that share one set of token and head strides
    (last dimension contiguous), e.g. ``cache.permute(1, 0, 2)`` of token-major caches [L, Hkv, d]."""
    n = len(layers)
    K0, V0 = layers[0][1], layers[0][2]
    Hkv, L, d = K0.shape
    ks, vs = (K0.stride(1), K0.stride(0)), (V0.stride(1), V0.stride(0))
    for q, K, V in layers:
        for t, name, st in ((K, "K", ks), (V, "V", vs)):
            if not (t.is_cuda and t.dtype == torch.bfloat16 and tuple(t.shape) == (Hkv, L, d) and t.stride(2) == 1
                    and (t.stride(1), t.stride(0)) == st):
                raise ValueError(f"{name}: CUDA bf16 [Hkv, L, d] views with the same strides in every layer are required")
        if q is not None:
            _dev(q, torch.bfloat16, "q_obs")
    n_max = out_len(L, w, c, budget)
    dev = K0.device
    if outs is None:
        outs = [(torch.empty((Hkv, n_max, d), dtype=torch.bfloat16, device=dev),
                 torch.empty((Hkv, n_max, d), dtype=torch.bfloat16, device=dev),
                 torch.empty((Hkv, n_max), dtype=torch.int32, device=dev)) for _ in range(n)]
    _ensure_bytes(max(int(lib.chunkkv_model_workspace_bytes(n, L, Hq, Hkv, d, w, c, budget, n_reuse)),
                      workspace_bytes(L, Hq, Hkv, d, w, c)))
    arr = ctypes.c_void_p * n
    qa = arr(*[None if t[0] is None else t[0].data_ptr() for t in layers])
    ka = arr(*[t[1].data_ptr() for t in layers])
    va = arr(*[t[2].data_ptr() for t in layers])
    oka = arr(*[o[0].data_ptr() for o in outs])
    ova = arr(*[o[1].data_ptr() for o in outs])
    oia = arr(*[o[2].data_ptr() for o in outs])
    _check(lib.chunkkv_compress_model_strided(n, qa, ka, va, L, Hq, Hkv, d, w, c, budget, n_reuse, ks[0], ks[1], vs[0], vs[1],
                                              oka, ova, oia, _stream(stream)), "chunkkv_compress_model_strided")
    return [tuple(o) for o in outs]


def compress_model_paged(layers: Sequence[Tuple[Optional[torch.Tensor], torch.Tensor, torch.Tensor]], Hq: int, w: int,
                         c: int, budget: int, block_tables: Sequence[torch.Tensor], caches: Sequence[Tuple[torch.Tensor, torch.Tensor]],
                         n_reuse: int = 1, stream: Optional[torch.cuda.Stream] = None,
                         out_idx: Optional[Sequence[torch.Tensor]] = None) -> List[torch.Tensor]:
    """compress_model with every layer's kept rows written to that layer's paged cache
    (caches[l] = (cache_K, cache_V) [num_pages, page_size, Hkv, d], block_tables[l] int32); returns the
    layers' idx [Hkv, n_max]."""
    n = len(layers)
    Hkv, L, d = layers[0][1].shape
    for q, K, V in layers:
        _dev(K, torch.bfloat16, "K"); _dev(V, torch.bfloat16, "V")
        if q is not None:
            _dev(q, torch.bfloat16, "q_obs")
    page_size, num_pages = caches[0][0].shape[1], caches[0][0].shape[0]
    for (cK, cV), bt in zip(caches, block_tables):
        _dev(cK, torch.bfloat16, "cache_K"); _dev(cV, torch.bfloat16, "cache_V"); _dev(bt, torch.int32, "block_table")
        if cK.shape[0] != num_pages or cK.shape[1] != page_size:
            raise ValueError("all layers' caches must share page_size and num_pages")
    n_max = out_len(L, w, c, budget)
    dev = layers[0][1].device
    if out_idx is None:
        out_idx = [torch.empty((Hkv, n_max), dtype=torch.int32, device=dev) for _ in range(n)]
    _ensure_bytes(max(int(lib.chunkkv_model_workspace_bytes(n, L, Hq, Hkv, d, w, c, budget, n_reuse)),
                      workspace_bytes(L, Hq, Hkv, d, w, c)))
    arr = ctypes.c_void_p * n
    qa = arr(*[None if t[0] is None else t[0].data_ptr() for t in layers])
    ka = arr(*[t[1].data_ptr() for t in layers])
    va = arr(*[t[2].data_ptr() for t in layers])
    bta = arr(*[t.data_ptr() for t in block_tables])
    cka = arr(*[t[0].data_ptr() for t in caches])
    cva = arr(*[t[1].data_ptr() for t in caches])
    oia = arr(*[t.data_ptr() for t in out_idx])
    _check(lib.chunkkv_compress_model_paged(n, qa, ka, va, L, Hq, Hkv, d, w, c, budget, n_reuse, bta, page_size, num_pages,
                                            cka, cva, oia, _stream(stream)), "chunkkv_compress_model_paged")
    return list(out_idx)


def profile_enable(on: bool) -> None:
    _check(lib.chunkkv_profile_enable(1 if on else 0), "chunkkv_profile_enable")


def profile_read() -> Tuple[List[float], List[int]]:
    ms = (ctypes.c_float * 4)()
    n = (ctypes.c_int * 4)()
    _check(lib.chunkkv_profile_read(ms, n), "chunkkv_profile_read")
    return list(ms), list(n)
