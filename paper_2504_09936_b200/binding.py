"""ctypes binding over libkeepkv.so: same names as the C ABI (``include/keepkv.h``), argument
marshalling only.  torch supplies device memory and streams; every step of the path runs in the
library's CUDA kernels.  There is no fallback: if the compiled library is missing, loading raises.
"""
from __future__ import annotations

import ctypes as C
import math
import os
from dataclasses import dataclass, field

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libkeepkv.so")

EXPORTS = ("keepkv_workspace_bytes", "keepkv_workspace_init", "keepkv_append", "keepkv_decode_attention",
           "keepkv_decode_step", "keepkv_compress", "keepkv_compress_scored", "keepkv_compress_merge_first", "keepkv_compress_inplace", "keepkv_complete_append_host", "keepkv_complete_load_host", "keepkv_prefill_scores", "keepkv_decode_step_host", "keepkv_decode_step_host_layers", "keepkv_decode_attention_static", "keepkv_debug_decode", "keepkv_status_string", "keepkv_last_cuda_error",
           "keepkv_last_launch_count")


class KeepKVError(RuntimeError):
    pass


class keepkv_params(C.Structure):
    _fields_ = [("B", C.c_int32), ("H_q", C.c_int32), ("H_kv", C.c_int32), ("d", C.c_int32), ("N_cap", C.c_int32),
                ("period", C.c_int32), ("n_sink", C.c_int32), ("n_recent", C.c_int32), ("sm_scale", C.c_float),
                ("ema_alpha", C.c_float), ("merge_threshold", C.c_float), ("gamma_min", C.c_float),
                ("gamma_max", C.c_float), ("flags", C.c_int32), ("reserved", C.c_int32 * 2)]


class keepkv_cache(C.Structure):
    _fields_ = [("K", C.c_void_p), ("V", C.c_void_p), ("votes", C.c_void_p), ("lscore", C.c_void_p),
                ("seq_len", C.c_void_p)]


FLAG_COMPRESS_STEADY = 1   # keepkv_params.flags: the caller promises steady-state units, one kernel compresses them
FLAG_CACHE_IDLE = 2        # decode calls: the preceding kernel of the stream does not write this cache
DEV_APPEND_FULL, DEV_TIMEOUT, DEV_NOT_STEADY, DEV_POSITIONS = 1, 2, 4, 8   # bits of *status_dev

STATS_FIELDS = ("n_retained", "n_evicted", "n_merged", "n_below_T", "n_guard_groups", "n_groups", "max_group",
                "reserved")

_lib = None


def lib() -> C.CDLL:
    """The loaded library.  Raises KeepKVError if it has not been built (no CPU path exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise KeepKVError(f"{LIB_PATH} not found: build it with `python -m paper_2504_09936_b200.build` "
                              "(there is no CPU fallback)")
        l = C.CDLL(LIB_PATH)
        for name in EXPORTS:
            getattr(l, name)  # AttributeError if a declared symbol is missing
        l.keepkv_status_string.restype = C.c_char_p
        l.keepkv_status_string.argtypes = [C.c_int]
        vp, i32, sz = C.c_void_p, C.c_int32, C.c_size_t
        pp, pc = C.POINTER(keepkv_params), C.POINTER(keepkv_cache)
        l.keepkv_workspace_bytes.argtypes = [pp, C.POINTER(sz)]
        l.keepkv_workspace_init.argtypes = [pp, vp, sz, vp]
        l.keepkv_append.argtypes = [pp, pc, vp, vp, vp, vp]
        l.keepkv_decode_attention.argtypes = [pp, pc, vp, vp, vp, C.c_int, vp, sz, vp, vp]
        l.keepkv_decode_step.argtypes = [pp, pc, vp, vp, vp, vp, vp, C.c_int, vp, sz, vp, vp]
        l.keepkv_decode_attention_static.argtypes = [pp, pc, vp, vp, vp, C.c_int, vp, vp]
        l.keepkv_debug_decode.argtypes = [C.c_int, C.c_int]
        l.keepkv_prefill_scores.argtypes = [pp, pc, vp, i32, vp, vp]
        l.keepkv_compress.argtypes = [pp, pc, pc, vp, i32, vp, vp, vp, vp, vp, sz, vp, vp]
        l.keepkv_compress_scored.argtypes = [pp, pc, pc, vp, vp, i32, vp, vp, vp, vp, vp, sz, vp, vp]
        l.keepkv_compress_merge_first.argtypes = [pp, pc, pc, vp, i32, vp, vp, vp, vp, sz, vp, vp]
        l.keepkv_complete_append_host.argtypes = [pp, vp, vp, vp, vp, vp]
        l.keepkv_complete_load_host.argtypes = [pp, vp, vp, vp, pc, vp]
        l.keepkv_compress_inplace.argtypes = [pp, pc, vp, vp, vp, vp, i32, vp, vp, vp, vp, vp, sz, vp, vp]
        l.keepkv_decode_step_host.argtypes = [pp, pc] + [vp] * 8 + [C.c_int, vp, sz, vp, vp]
        l.keepkv_decode_step_host_layers.argtypes = [pp, pc, i32] + [vp] * 8 + [C.c_int, vp, sz, vp, vp]
        _lib = l
    return _lib


def _check(rc: int, what: str):
    if rc != 0:
        name = lib().keepkv_status_string(rc).decode()
        extra = f" (cudaError {lib().keepkv_last_cuda_error()})" if rc == -5 else ""
        raise KeepKVError(f"{what}: {name}{extra}")


def make_params(B, H_q, H_kv, d, N_cap, period=0, n_sink=4, n_recent=0, sm_scale=None, ema_alpha=0.9,
                merge_threshold=0.8, gamma_min=0.0, gamma_max=4.0, flags=0) -> keepkv_params:
    return keepkv_params(B, H_q, H_kv, d, N_cap, period, n_sink, n_recent,
                         sm_scale if sm_scale is not None else 1.0 / math.sqrt(d), ema_alpha, merge_threshold,
                         gamma_min, gamma_max, flags, (C.c_int32 * 2)(0, 0))


@dataclass
class Cache:
    """One layer's cache as torch tensors on the GPU (see keepkv_cache in the header)."""
    K: torch.Tensor        # bf16 [B, H_kv, N_cap, d]
    V: torch.Tensor        # bf16 [B, H_kv, N_cap, d]
    votes: torch.Tensor    # f32  [B, H_kv, N_cap]
    lscore: torch.Tensor   # f32  [B, H_kv, N_cap]
    seq_len: torch.Tensor  # i32  [B]
    _c: keepkv_cache = field(default=None, repr=False)

    @staticmethod
    def empty(p: keepkv_params, device="cuda") -> "Cache":
        shp = (p.B, p.H_kv, p.N_cap)
        return Cache(torch.zeros(*shp, p.d, dtype=torch.bfloat16, device=device),
                     torch.zeros(*shp, p.d, dtype=torch.bfloat16, device=device),
                     torch.ones(*shp, dtype=torch.float32, device=device),
                     torch.full(shp, -math.inf, dtype=torch.float32, device=device),
                     torch.zeros(p.B, dtype=torch.int32, device=device))

    def c(self) -> keepkv_cache:
        if self._c is None:
            for t in (self.K, self.V, self.votes, self.lscore, self.seq_len):
                assert t.is_cuda and t.is_contiguous()
            self._c = keepkv_cache(self.K.data_ptr(), self.V.data_ptr(), self.votes.data_ptr(),
                                   self.lscore.data_ptr(), self.seq_len.data_ptr())
        return self._c


def _stream(stream=None) -> int:
    return (stream if stream is not None else torch.cuda.current_stream()).cuda_stream


def _ptr(t):
    return None if t is None else t.data_ptr()


def keepkv_workspace_bytes(p: keepkv_params) -> int:
    n = C.c_size_t()
    _check(lib().keepkv_workspace_bytes(C.byref(p), C.byref(n)), "keepkv_workspace_bytes")
    return n.value


def new_workspace(p: keepkv_params, device="cuda", stream=None) -> torch.Tensor:
    ws = torch.empty(keepkv_workspace_bytes(p), dtype=torch.uint8, device=device)
    _check(lib().keepkv_workspace_init(C.byref(p), ws.data_ptr(), ws.numel(), _stream(stream)),
           "keepkv_workspace_init")
    return ws


def new_status(device="cuda") -> torch.Tensor:
    return torch.zeros(1, dtype=torch.int32, device=device)


def keepkv_append(p, cache: Cache, k_new, v_new, status, stream=None):
    _check(lib().keepkv_append(C.byref(p), C.byref(cache.c()), k_new.data_ptr(), v_new.data_ptr(), status.data_ptr(),
                               _stream(stream)), "keepkv_append")


def keepkv_decode_attention(p, cache: Cache, q, out, lse, update_scores: bool, ws, status, stream=None):
    _check(lib().keepkv_decode_attention(C.byref(p), C.byref(cache.c()), q.data_ptr(), out.data_ptr(), _ptr(lse),
                                         int(update_scores), ws.data_ptr(), ws.numel(), status.data_ptr(),
                                         _stream(stream)), "keepkv_decode_attention")


def keepkv_decode_step(p, cache: Cache, q, k_new, v_new, out, lse, update_scores: bool, ws, status, stream=None):
    """keepkv_append followed by keepkv_decode_attention in one launch."""
    _check(lib().keepkv_decode_step(C.byref(p), C.byref(cache.c()), q.data_ptr(), k_new.data_ptr(), v_new.data_ptr(),
                                    out.data_ptr(), _ptr(lse), int(update_scores), ws.data_ptr(), ws.numel(),
                                    status.data_ptr(), _stream(stream)), "keepkv_decode_step")


def keepkv_decode_attention_static(p, cache: Cache, q, out, lse, update_scores: bool, status, stream=None):
    """keepkv_decode_attention without a caller workspace, for code that cannot allocate device memory:
    the scratch is a fixed array inside the library (shared by all calls on the GPU, so keep them
    on one stream; make the first call on a device outside stream capture)."""
    _check(lib().keepkv_decode_attention_static(C.byref(p), C.byref(cache.c()), q.data_ptr(), out.data_ptr(),
                                                _ptr(lse), int(update_scores), status.data_ptr(), _stream(stream)),
           "keepkv_decode_attention_static")


def keepkv_prefill_scores(p, cache: Cache, q_window, status, stream=None):
    """q_window: bf16 CUDA tensor [B, H_q, W, d], the last W prompt queries, oldest first (Eq. 8, first case)."""
    assert q_window.is_contiguous() and q_window.dim() == 4
    _check(lib().keepkv_prefill_scores(C.byref(p), C.byref(cache.c()), q_window.data_ptr(), int(q_window.shape[2]),
                                       status.data_ptr(), _stream(stream)), "keepkv_prefill_scores")


def keepkv_compress(p, src: Cache, dst: Cache, budget, ws, status, n_recent_dev=None, retained_idx=None,
                    target=None, stats=None, stream=None):
    """budget: int (same for every sequence) or an int32 CUDA tensor [B]."""
    bdev, bsc = (budget.data_ptr(), 0) if isinstance(budget, torch.Tensor) else (None, int(budget))
    _check(lib().keepkv_compress(C.byref(p), C.byref(src.c()), C.byref(dst.c()), bdev, bsc, _ptr(n_recent_dev),
                                 _ptr(retained_idx), _ptr(target), _ptr(stats), ws.data_ptr(), ws.numel(),
                                 status.data_ptr(), _stream(stream)), "keepkv_compress")


def keepkv_compress_scored(p, src: Cache, dst: Cache, select_score, budget, ws, status, n_recent_dev=None,
                           retained_idx=None, target=None, stats=None, stream=None):
    """keepkv_compress with the caller's importance scores (fp32 CUDA tensor [B, H_kv, N_cap]) driving the selection."""
    assert select_score.dtype == torch.float32 and select_score.is_contiguous()
    bdev, bsc = (budget.data_ptr(), 0) if isinstance(budget, torch.Tensor) else (None, int(budget))
    _check(lib().keepkv_compress_scored(C.byref(p), C.byref(src.c()), C.byref(dst.c()), select_score.data_ptr(), bdev,
                                        bsc, _ptr(n_recent_dev), _ptr(retained_idx), _ptr(target), _ptr(stats),
                                        ws.data_ptr(), ws.numel(), status.data_ptr(), _stream(stream)),
           "keepkv_compress_scored")


def keepkv_complete_append_host(p, K_host, V_host, seq_len_host, k_new_host, v_new_host):
    """Eq. 2 on a complete cache kept in host memory (CPU tensors; seq_len_host int32 [B] is advanced)."""
    for t in (K_host, V_host, seq_len_host, k_new_host, v_new_host):
        assert not t.is_cuda and t.is_contiguous()
    _check(lib().keepkv_complete_append_host(C.byref(p), K_host.data_ptr(), V_host.data_ptr(), seq_len_host.data_ptr(),
                                             k_new_host.data_ptr(), v_new_host.data_ptr()), "keepkv_complete_append_host")


def keepkv_complete_load_host(p, K_host, V_host, seq_len_host, dev: Cache, stream=None):
    """Loads the host-resident complete cache into a device cache (votes 1, no score history)."""
    for t in (K_host, V_host, seq_len_host):
        assert not t.is_cuda and t.is_contiguous()
    _check(lib().keepkv_complete_load_host(C.byref(p), K_host.data_ptr(), V_host.data_ptr(), seq_len_host.data_ptr(),
                                           C.byref(dev.c()), _stream(stream)), "keepkv_complete_load_host")


def keepkv_compress_inplace(p, cache: Cache, pos, pos_len, n_seen, budget, ws, status, n_recent_dev=None, moved_from=None,
                            target=None, stats=None, stream=None):
    """Algorithm 1 in place: pos int32 [B, H_kv, N_cap], pos_len and n_seen int32 [B] travel with the cache (see the header)."""
    for t in (pos, pos_len, n_seen):
        assert t.dtype == torch.int32 and t.is_cuda and t.is_contiguous()
    bdev, bsc = (budget.data_ptr(), 0) if isinstance(budget, torch.Tensor) else (None, int(budget))
    _check(lib().keepkv_compress_inplace(C.byref(p), C.byref(cache.c()), pos.data_ptr(), pos_len.data_ptr(), n_seen.data_ptr(),
                                         bdev, bsc, _ptr(n_recent_dev), _ptr(moved_from), _ptr(target), _ptr(stats),
                                         ws.data_ptr(), ws.numel(), status.data_ptr(), _stream(stream)),
           "keepkv_compress_inplace")


def keepkv_compress_merge_first(p, cache: Cache, scratch: Cache, budget, ws, status, n_recent_dev=None,
                                retained_idx=None, stats=None, stream=None):
    """Prefill compression, merge-first policy (Section 3.4): similar entries of the prompt are merged with each
    other, then the selection cuts the result to the budget.  In place on `cache`; `scratch` is destroyed."""
    bdev, bsc = (budget.data_ptr(), 0) if isinstance(budget, torch.Tensor) else (None, int(budget))
    _check(lib().keepkv_compress_merge_first(C.byref(p), C.byref(cache.c()), C.byref(scratch.c()), bdev, bsc,
                                             _ptr(n_recent_dev), _ptr(retained_idx), _ptr(stats), ws.data_ptr(),
                                             ws.numel(), status.data_ptr(), _stream(stream)),
           "keepkv_compress_merge_first")


def keepkv_decode_step_host(p, cache: Cache, q_host, k_new_host, v_new_host, out_host, q_dev, k_new_dev, v_new_dev,
                            out_dev, update_scores: bool, ws, status, stream=None):
    _check(lib().keepkv_decode_step_host(C.byref(p), C.byref(cache.c()), q_host.data_ptr(), k_new_host.data_ptr(),
                                         v_new_host.data_ptr(), out_host.data_ptr(), q_dev.data_ptr(),
                                         k_new_dev.data_ptr(), v_new_dev.data_ptr(), out_dev.data_ptr(),
                                         int(update_scores), ws.data_ptr(), ws.numel(), status.data_ptr(),
                                         _stream(stream)), "keepkv_decode_step_host")


def keepkv_decode_step_host_layers(p, caches, q_host, k_new_host, v_new_host, out_host, q_dev, k_new_dev, v_new_dev,
                                   out_dev, update_scores: bool, ws, status, stream=None):
    """caches: list of Cache, one per layer; host / staging tensors carry the layers as their first axis."""
    arr = (keepkv_cache * len(caches))(*[c.c() for c in caches])
    _check(lib().keepkv_decode_step_host_layers(C.byref(p), arr, len(caches), q_host.data_ptr(), k_new_host.data_ptr(),
                                                v_new_host.data_ptr(), out_host.data_ptr(), q_dev.data_ptr(),
                                                k_new_dev.data_ptr(), v_new_dev.data_ptr(), out_dev.data_ptr(),
                                                int(update_scores), ws.data_ptr(), ws.numel(), status.data_ptr(),
                                                _stream(stream)), "keepkv_decode_step_host_layers")


def keepkv_debug_decode(spin_limit: int = 0, withhold_tile: int = -1):
    """Test hook: bounded-wait poll count and a tile position whose copies are withheld (see the header)."""
    _check(lib().keepkv_debug_decode(int(spin_limit), int(withhold_tile)), "keepkv_debug_decode")


def last_launch_count() -> int:
    return int(lib().keepkv_last_launch_count())
