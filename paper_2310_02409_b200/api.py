"""Thin ctypes binding over the C ABI declared in ``include/dodo.h``.

Argument marshalling only: device tensors become raw pointers, host offset/length tables become
``int32`` arrays, and the current torch CUDA stream is passed along.  Every step of the path runs
in the library's kernels; there is no CPU or PyTorch fallback, and importing this module fails
loudly when ``libdodo.so`` has not been built (``python -m paper_2310_02409_b200.build``).
"""
from __future__ import annotations

import ctypes
from pathlib import Path

import numpy as np
import torch

LIB_PATH = Path(__file__).resolve().parent / "libdodo.so"

F32, BF16 = 0, 1
FORCE_LAST = 1
ACT_IDENTITY, ACT_RELU, ACT_GELU_TANH = 0, 1, 2
TUNE_ATTEND_TARGET_BLOCKS, TUNE_DENSE_MIN_QUERIES, TUNE_DENSE_BALANCE = 1, 3, 4
DEV_WAIT_TIMEOUT, DEV_BAD_INDEX = 1, 2
OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_CAPACITY, ERR_CUDA = 0, -1, -2, -3, -4

# every symbol include/dodo.h declares: name -> (restype, argtypes)
_vp, _i, _u, _f, _sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_uint32, ctypes.c_float, ctypes.c_size_t
SIGNATURES = {
    "dodo_create": (_i, [ctypes.POINTER(_vp), _i]),
    "dodo_destroy": (_i, [_vp]),
    "dodo_last_error": (ctypes.c_char_p, [_vp]),
    "dodo_reset": (_i, [_vp, _vp]),
    "dodo_device_status": (_i, [_vp, ctypes.POINTER(_i)]),
    "dodo_set_tuning": (_i, [_vp, _i, _i]),
    "dodo_cache_written": (_i, [_vp]),
    "dodo_num_nuggets": (_i, [_i, _i]),
    "dodo_score": (_i, [_vp, _vp, _i, _i, _vp, _f, _vp, _i, _vp, _vp]),
    "dodo_select": (_i, [_vp, _vp, _vp, _vp, _i, _u, _vp, _vp]),
    "dodo_score_mlp_workspace_bytes": (_sz, [_i, _i]),
    "dodo_score_mlp": (_i, [_vp, _vp, _i, _i, _vp, _vp, _vp, _f, _i, _i, _vp, _i, _vp, _vp, _sz, _vp]),
    "dodo_score_mlp_select": (_i, [_vp, _vp, _i, _i, _vp, _vp, _vp, _f, _i, _i, _vp, _vp, _i, _u, _vp, _vp, _vp, _sz, _vp]),
    "dodo_count_threshold": (_i, [_vp, _vp, _vp, _i, _f, _vp, _vp]),
    "dodo_select_threshold": (_i, [_vp, _vp, _vp, _vp, _i, _f, _vp, _vp]),
    "dodo_estimate_threshold": (_i, [_vp, _vp, _i, _i, _vp, _vp]),
    "dodo_score_select": (_i, [_vp, _vp, _i, _i, _vp, _f, _vp, _vp, _i, _u, _vp, _vp, _vp]),
    "dodo_gather_kv": (_i, [_vp, _vp, _vp, _i, _i, _i, _vp, _vp, _vp, _vp, _i, _vp, _vp, _vp, _vp, _vp, _vp]),
    "dodo_compress": (_i, [_vp, _vp, _i, _i, _vp, _f, _vp, _vp, _i, _i, _vp, _vp, _vp, _i, _u, _vp, _vp, _vp, _vp, _vp, _vp,
                           _vp, _vp]),
    "dodo_gather_kv_layers": (_i, [_vp, _i, _vp, _vp, _i, _i, _i, _vp, _vp, _vp, _vp, _i, _vp, _vp, _vp, _vp, _vp, _vp]),
    "dodo_pool_kv": (_i, [_vp, _vp, _vp, _i, _i, _i, _vp, _i, _vp, _i, _vp, _vp, _vp, _vp, _vp, _vp]),
    "dodo_attend_workspace_bytes": (_sz, [_vp, _i]),
    "dodo_attend": (_i, [_vp, _vp, _vp, _vp, _i, _i, _i, _f, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp,
                         _i, _i, _vp, _vp, _vp, _sz, _vp]),
    "dodo_attend_indexed": (_i, [_vp, _vp, _vp, _vp, _i, _i, _i, _f, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp,
                                 _i, _i, _vp, _vp, _vp, _sz, _vp]),
    "dodo_host_arena_bytes": (_sz, [_vp, _i, _i, _i, _i, _i, _i, _i, _i, _i]),
    "dodo_compress_decode_host": (_i, [_vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _vp, _vp, _i, _vp, _vp, _i, _vp, _i, _f,
                                       _vp, _vp, _sz, _vp]),
    "dodo_attend_noalloc": (_i, [_vp, _vp, _vp, _i, _i, _i, _f, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp,
                                 _i, _i, _vp, _vp, _vp, ctypes.c_char_p, _sz]),
}

_lib = None


def load() -> ctypes.CDLL:
    """Load ``libdodo.so`` and attach the signatures.  Raises if the library is missing."""
    global _lib
    if _lib is None:
        if not LIB_PATH.exists():
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2310_02409_b200.build` "
                              "(there is no fallback path)")
        lib = ctypes.CDLL(str(LIB_PATH))
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype, fn.argtypes = res, args
        _lib = lib
    return _lib


class DodoError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"dodo status {status}: {message}")
        self.status = status


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def _dev(t: torch.Tensor | None):
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("device arguments must be contiguous CUDA tensors")
    return t.data_ptr()


def _host_i32(a) -> np.ndarray | None:
    if a is None:
        return None
    return np.ascontiguousarray(a, dtype=np.int32)


def _hp(a: np.ndarray | None):
    return None if a is None else a.ctypes.data


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


class Dodo:
    """One library context on one CUDA device.  Methods mirror the C entry points one to one."""

    def __init__(self, device: int = 0):
        self._lib = load()
        self._ctx = _vp()
        rc = self._lib.dodo_create(ctypes.byref(self._ctx), int(device))
        if rc != OK:
            msg = self._lib.dodo_last_error(self._ctx).decode() if self._ctx else "no context"
            self._lib.dodo_destroy(self._ctx)
            self._ctx = None
            raise DodoError(rc, msg)
        self.device = torch.device("cuda", device)

    def close(self):
        if getattr(self, "_ctx", None):
            self._lib.dodo_destroy(self._ctx)
            self._ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc: int):
        if rc != OK:
            raise DodoError(rc, self._lib.dodo_last_error(self._ctx).decode())

    # -- helpers -------------------------------------------------------------------------------
    def num_nuggets(self, n: int, r: int) -> int:
        return int(self._lib.dodo_num_nuggets(int(n), int(r)))

    def device_status(self) -> int:
        out = _i(0)
        self._check(self._lib.dodo_device_status(self._ctx, ctypes.byref(out)))
        return int(out.value)

    def reset(self):
        self._check(self._lib.dodo_reset(self._ctx, _stream()))

    def cache_written(self):
        self._check(self._lib.dodo_cache_written(self._ctx))

    def set_tuning(self, knob: int, value: int):
        self._check(self._lib.dodo_set_tuning(self._ctx, int(knob), int(value)))

    def attend_workspace_bytes(self, dh: int) -> int:
        return int(self._lib.dodo_attend_workspace_bytes(self._ctx, int(dh)))

    def host_arena_bytes(self, dtype_code, d, H, dh, total_tokens, total_nuggets, B, local, steps) -> int:
        return int(self._lib.dodo_host_arena_bytes(self._ctx, dtype_code, d, H, dh, total_tokens, total_nuggets, B,
                                                   local, steps))

    def compress_decode_host(self, hX, hw, hK, hV, seq_off, nug_off, hLocK, hLocV, local, hQ, sm_scale, hO, arena):
        """``dodo_compress_decode_host``: the whole path of one layer on HOST tensors (pinned for
        asynchronous copies); ``arena`` is a device uint8 tensor of ``host_arena_bytes`` bytes."""
        so, no = _host_i32(seq_off), _host_i32(nug_off)
        for t in (hX, hw, hK, hV, hLocK, hLocV, hQ, hO):
            if t.is_cuda or not t.is_contiguous():
                raise ValueError("host arguments must be contiguous CPU tensors")
        steps, B, H, dh = hQ.shape
        self._check(self._lib.dodo_compress_decode_host(
            self._ctx, hX.data_ptr(), hw.data_ptr(), hK.data_ptr(), hV.data_ptr(), _dtype_code(hX), hX.shape[-1], H, dh,
            _hp(so), _hp(no), B, hLocK.data_ptr(), hLocV.data_ptr(), int(local), hQ.data_ptr(), steps, float(sm_scale),
            hO.data_ptr(), _dev(arena), arena.numel() * arena.element_size(), _stream()))

    # -- the path ------------------------------------------------------------------------------
    def score(self, X, w, bias, seq_off, scores):
        so = _host_i32(seq_off)
        self._check(self._lib.dodo_score(self._ctx, _dev(X), _dtype_code(X), X.shape[-1], _dev(w), float(bias),
                                         _hp(so), len(so) - 1, _dev(scores), _stream()))

    def select(self, scores, seq_off, nug_off, flags, idx):
        so, no = _host_i32(seq_off), _host_i32(nug_off)
        self._check(self._lib.dodo_select(self._ctx, _dev(scores), _hp(so), _hp(no), len(so) - 1, int(flags),
                                          _dev(idx), _stream()))

    def score_mlp_workspace_bytes(self, rows: int, dh: int) -> int:
        return int(self._lib.dodo_score_mlp_workspace_bytes(int(rows), int(dh)))

    def score_mlp(self, X, W1, b1, w2, b2, act, seq_off, scores, workspace):
        so = _host_i32(seq_off)
        ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
        self._check(self._lib.dodo_score_mlp(self._ctx, _dev(X), _dtype_code(X), int(X.shape[1]), _dev(W1), _dev(b1), _dev(w2),
                                             float(b2), int(W1.shape[0]), int(act), _hp(so), len(so) - 1, _dev(scores),
                                             _dev(workspace), ws_bytes, _stream()))

    def score_mlp_select(self, X, W1, b1, w2, b2, act, seq_off, nug_off, flags, scores, idx, workspace):
        so, no = _host_i32(seq_off), _host_i32(nug_off)
        ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
        self._check(self._lib.dodo_score_mlp_select(self._ctx, _dev(X), _dtype_code(X), int(X.shape[1]), _dev(W1), _dev(b1), _dev(w2),
                                                    float(b2), int(W1.shape[0]), int(act), _hp(so), _hp(no), len(so) - 1, int(flags),
                                                    _dev(scores), _dev(idx), _dev(workspace), ws_bytes, _stream()))

    def count_threshold(self, scores, seq_off, lam, counts):
        so = _host_i32(seq_off)
        self._check(self._lib.dodo_count_threshold(self._ctx, _dev(scores), _hp(so), len(so) - 1, float(lam),
                                                   _dev(counts), _stream()))

    def select_threshold(self, scores, seq_off, nug_off, lam, idx):
        so, no = _host_i32(seq_off), _host_i32(nug_off)
        self._check(self._lib.dodo_select_threshold(self._ctx, _dev(scores), _hp(so), _hp(no), len(so) - 1, float(lam),
                                                    _dev(idx), _stream()))

    def estimate_threshold(self, sample, r, lam_out):
        self._check(self._lib.dodo_estimate_threshold(self._ctx, _dev(sample), int(sample.numel()), int(r),
                                                      _dev(lam_out), _stream()))

    def score_select(self, X, w, bias, seq_off, nug_off, flags, scores, idx):
        so, no = _host_i32(seq_off), _host_i32(nug_off)
        self._check(self._lib.dodo_score_select(self._ctx, _dev(X), _dtype_code(X), X.shape[-1], _dev(w),
                                                float(bias), _hp(so), _hp(no), len(so) - 1, int(flags),
                                                _dev(scores), _dev(idx), _stream()))

    def gather_kv(self, K, V, seq_off, idx, nug_off, pos_base, cacheK, cacheV, cache_pos, cache_off, cache_len):
        """``cache_len`` must be an int32 numpy array; it is updated in place."""
        so, no, pb, co = _host_i32(seq_off), _host_i32(nug_off), _host_i32(pos_base), _host_i32(cache_off)
        if not (isinstance(cache_len, np.ndarray) and cache_len.dtype == np.int32 and cache_len.flags.c_contiguous):
            raise TypeError("cache_len must be a contiguous int32 numpy array (updated in place)")
        H, dh = K.shape[-2], K.shape[-1]
        self._check(self._lib.dodo_gather_kv(self._ctx, _dev(K), _dev(V), _dtype_code(K), H, dh, _hp(so), _dev(idx),
                                             _hp(no), _hp(pb), len(so) - 1, _dev(cacheK), _dev(cacheV),
                                             _dev(cache_pos), _hp(co), _hp(cache_len), _stream()))

    def compress(self, X, w, bias, K, V, seq_off, nug_off, pos_base, flags, scores, idx, cacheK, cacheV, cache_pos,
                 cache_off, cache_len):
        """``dodo_compress``: score, TopK and gather in one call; ``cache_len`` (int32 numpy array) is updated in place."""
        so, no, pb, co = _host_i32(seq_off), _host_i32(nug_off), _host_i32(pos_base), _host_i32(cache_off)
        if not (isinstance(cache_len, np.ndarray) and cache_len.dtype == np.int32 and cache_len.flags.c_contiguous):
            raise TypeError("cache_len must be a contiguous int32 numpy array (updated in place)")
        H, dh = K.shape[-2], K.shape[-1]
        self._check(self._lib.dodo_compress(self._ctx, _dev(X), _dtype_code(X), X.shape[-1], _dev(w), float(bias), _dev(K),
                                            _dev(V), H, dh, _hp(so), _hp(no), _hp(pb), len(so) - 1, int(flags), _dev(scores),
                                            _dev(idx), _dev(cacheK), _dev(cacheV), _dev(cache_pos), _hp(co), _hp(cache_len),
                                            _stream()))

    def pool_kv(self, K, V, seq_off, r, pos_base, cacheK, cacheV, cache_pos, cache_off, cache_len):
        """``dodo_pool_kv``: mean of every even chunk of r tokens appended to the caches; ``cache_len`` (int32 numpy
        array) is updated in place."""
        so, pb, co = _host_i32(seq_off), _host_i32(pos_base), _host_i32(cache_off)
        if not (isinstance(cache_len, np.ndarray) and cache_len.dtype == np.int32 and cache_len.flags.c_contiguous):
            raise TypeError("cache_len must be a contiguous int32 numpy array (updated in place)")
        H, dh = K.shape[-2], K.shape[-1]
        self._check(self._lib.dodo_pool_kv(self._ctx, _dev(K), _dev(V), _dtype_code(K), H, dh, _hp(so), int(r), _hp(pb),
                                           len(so) - 1, _dev(cacheK), _dev(cacheV), _dev(cache_pos), _hp(co), _hp(cache_len),
                                           _stream()))

    def gather_kv_layers(self, Ks, Vs, seq_off, idx, nug_off, pos_base, cacheKs, cacheVs, cache_pos, cache_off,
                         cache_len):
        """One shared selection, L layers: ``Ks``, ``Vs``, ``cacheKs``, ``cacheVs`` are sequences of L tensors of
        one shape and dtype each.  ``cache_len`` (int32 numpy array) is updated in place, once."""
        so, no, pb, co = _host_i32(seq_off), _host_i32(nug_off), _host_i32(pos_base), _host_i32(cache_off)
        if not (isinstance(cache_len, np.ndarray) and cache_len.dtype == np.int32 and cache_len.flags.c_contiguous):
            raise TypeError("cache_len must be a contiguous int32 numpy array (updated in place)")
        L = len(Ks)
        if not (len(Vs) == len(cacheKs) == len(cacheVs) == L):
            raise ValueError("Ks, Vs, cacheKs and cacheVs must name the same number of layers")
        if L == 0:
            return
        H, dh = Ks[0].shape[-2], Ks[0].shape[-1]
        for t in (*Ks, *Vs, *cacheKs, *cacheVs):
            if t.dtype != Ks[0].dtype or tuple(t.shape[-2:]) != (H, dh):
                raise ValueError("every layer's K, V and caches must share dtype, H and dh")
        ptrs = lambda ts: (ctypes.c_void_p * L)(*[_dev(t) for t in ts])
        self._check(self._lib.dodo_gather_kv_layers(self._ctx, L, ptrs(Ks), ptrs(Vs), _dtype_code(Ks[0]), H, dh, _hp(so),
                                                    _dev(idx), _hp(no), _hp(pb), len(so) - 1, ptrs(cacheKs),
                                                    ptrs(cacheVs), _dev(cache_pos), _hp(co), _hp(cache_len), _stream()))

    def attend(self, Q, q_off, q_pos0, sm_scale, cacheK, cacheV, cache_pos, cache_off, cache_len,
               locK, locV, loc_off, loc_len, loc_pos0, O, lse, workspace):
        qo, qp = _host_i32(q_off), _host_i32(q_pos0)
        co, cl = _host_i32(cache_off), _host_i32(cache_len)
        lo, ll, lp = _host_i32(loc_off), _host_i32(loc_len), _host_i32(loc_pos0)
        H, dh = Q.shape[-2], Q.shape[-1]
        loc_rows = 0 if locK is None else locK.shape[0]
        ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
        self._check(self._lib.dodo_attend(self._ctx, _dev(Q), _hp(qo), _hp(qp), _dtype_code(Q), H, dh, float(sm_scale),
                                          _dev(cacheK), _dev(cacheV), _dev(cache_pos), _hp(co), _hp(cl),
                                          _dev(locK), _dev(locV), _hp(lo), _hp(ll), _hp(lp), loc_rows,
                                          len(qo) - 1, _dev(O), _dev(lse), _dev(workspace), ws_bytes, _stream()))

    def attend_indexed(self, Q, q_off, q_pos0, sm_scale, K, V, seq_off, idx, nug_off, pos_base,
                       locK, locV, loc_off, loc_len, loc_pos0, O, lse, workspace):
        """``dodo_attend_indexed``: queries attend the rows ``idx`` names in the uncompressed K / V, then the local tokens."""
        qo, qp = _host_i32(q_off), _host_i32(q_pos0)
        so, no, pb = _host_i32(seq_off), _host_i32(nug_off), _host_i32(pos_base)
        lo, ll, lp = _host_i32(loc_off), _host_i32(loc_len), _host_i32(loc_pos0)
        H, dh = Q.shape[-2], Q.shape[-1]
        loc_rows = 0 if locK is None else locK.shape[0]
        ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
        self._check(self._lib.dodo_attend_indexed(self._ctx, _dev(Q), _hp(qo), _hp(qp), _dtype_code(Q), H, dh, float(sm_scale),
                                                  _dev(K), _dev(V), _hp(so), _dev(idx), _hp(no), _hp(pb), _dev(locK), _dev(locV),
                                                  _hp(lo), _hp(ll), _hp(lp), loc_rows, len(qo) - 1, _dev(O), _dev(lse),
                                                  _dev(workspace), ws_bytes, _stream()))


def attend_noalloc(Q, q_off, q_pos0, sm_scale, cacheK, cacheV, cache_pos, cache_off, cache_len,
                   locK, locV, loc_off, loc_len, loc_pos0, O, lse):
    """``dodo_attend_noalloc``: attention without a context or a workspace, for callers that are not
    allowed to allocate device memory (the scratch is a fixed array inside the library).  Runs on the
    current device and stream; at most 64 sequences per call; calls must not overlap on the GPU."""
    lib = load()
    qo, qp = _host_i32(q_off), _host_i32(q_pos0)
    co, cl = _host_i32(cache_off), _host_i32(cache_len)
    lo, ll, lp = _host_i32(loc_off), _host_i32(loc_len), _host_i32(loc_pos0)
    H, dh = Q.shape[-2], Q.shape[-1]
    loc_rows = 0 if locK is None else locK.shape[0]
    err = ctypes.create_string_buffer(512)
    rc = lib.dodo_attend_noalloc(_dev(Q), _hp(qo), _hp(qp), _dtype_code(Q), H, dh, float(sm_scale),
                                 _dev(cacheK), _dev(cacheV), _dev(cache_pos), _hp(co), _hp(cl),
                                 _dev(locK), _dev(locV), _hp(lo), _hp(ll), _hp(lp), loc_rows, len(qo) - 1,
                                 _dev(O), _dev(lse), _stream(), err, len(err))
    if rc != OK:
        raise DodoError(rc, err.value.decode())
