"""ctypes loader for the fp64 CPU oracle (``dodo_oracle.c``).

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the benchmark's CPU
baseline leg may import this package; the CUDA library and its Python binding
never do, and this package imports nothing from them.

Arrays are numpy.  Floating-point tensors are passed in their storage format:
``float32`` arrays as they are, bf16 tensors as ``uint16`` arrays holding the
bf16 bit patterns.  All results come back in fp64 (indices in int32).

The ragged-batch helpers at the bottom only loop the per-sequence C routines
over a batch described by offset arrays; they add no arithmetic of their own.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "dodo_oracle.c"
# DODO_ORACLE_SANITIZE=1 selects a second build of the same source with AddressSanitizer and
# UndefinedBehaviorSanitizer (the process must then run with libasan preloaded); the tests use it to
# run the oracle's pins over an instrumented oracle.
_SANITIZE = os.environ.get("DODO_ORACLE_SANITIZE", "") == "1"
_LIB = _HERE / ("libdodo_oracle_san.so" if _SANITIZE else "libdodo_oracle.so")

F32 = 0
BF16 = 1
FORCE_LAST = 1


def build(force: bool = False) -> Path:
    """Compile ``dodo_oracle.c`` with gcc (OpenMP on) unless it is up to date."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".so.tmp{os.getpid()}")
        opt = ["-O1", "-g", "-fsanitize=address,undefined", "-fno-sanitize-recover=undefined",
               "-fno-omit-frame-pointer"] if _SANITIZE else ["-O2"]
        cmd = ["gcc", *opt, "-std=c11", "-fopenmp", "-shared", "-fPIC", "-Wall",
               "-o", str(tmp), str(_SRC), "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        build()
        L = ctypes.CDLL(str(_LIB))
        vp, i32, dbl = ctypes.c_void_p, ctypes.c_int, ctypes.c_double
        L.oracle_num_nuggets.argtypes = [i32, i32]
        L.oracle_num_nuggets.restype = i32
        L.oracle_score.argtypes = [vp, i32, ctypes.c_long, i32, vp, dbl, vp]
        L.oracle_score.restype = None
        L.oracle_score_mlp.argtypes = [vp, i32, ctypes.c_long, i32, vp, vp, vp, dbl, i32, i32, vp]
        L.oracle_score_mlp.restype = None
        L.oracle_select.argtypes = [vp, i32, i32, ctypes.c_uint, vp]
        L.oracle_select.restype = i32
        L.oracle_select_threshold.argtypes = [vp, i32, dbl, vp]
        L.oracle_select_threshold.restype = i32
        L.oracle_estimate_threshold.argtypes = [vp, i32, i32]
        L.oracle_estimate_threshold.restype = dbl
        L.oracle_gather.argtypes = [vp, ctypes.c_size_t, vp, i32, i32, vp, vp, i32, i32]
        L.oracle_gather.restype = i32
        L.oracle_pool.argtypes = [vp, i32, i32, i32, i32, i32, vp, vp]
        L.oracle_pool.restype = i32
        L.oracle_attend.argtypes = [vp, i32, i32, i32, i32, i32, dbl,
                                    vp, vp, vp, i32, vp, vp, i32, i32, vp, vp]
        L.oracle_attend.restype = None
        L.oracle_threads.argtypes = []
        L.oracle_threads.restype = i32
        L.oracle_set_threads.argtypes = [i32]
        L.oracle_set_threads.restype = None
        _lib = L
    return _lib


def _dtype_code(a: np.ndarray) -> int:
    if a.dtype == np.float32:
        return F32
    if a.dtype == np.uint16:
        return BF16
    raise TypeError(f"oracle takes float32 or uint16 (bf16 bits) arrays, got {a.dtype}")


def _ptr(a: np.ndarray | None):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a: np.ndarray) -> np.ndarray:
    return np.ascontiguousarray(a)


def threads() -> int:
    return int(lib().oracle_threads())


def set_threads(t: int) -> None:
    lib().oracle_set_threads(int(t))


def num_nuggets(n: int, r: int) -> int:
    """k = ceil(n / r) (text before Eq. 14)."""
    return int(lib().oracle_num_nuggets(int(n), int(r)))


def score(X: np.ndarray, w: np.ndarray, bias: float = 0.0) -> np.ndarray:
    """s_i = w . x_i + bias in fp64 (Eq. 6 / Eq. 15, linear Scorer).  X: [rows, d]."""
    X, w = _c(X), _c(w)
    dt = _dtype_code(X)
    assert _dtype_code(w) == dt and X.ndim == 2 and w.shape == (X.shape[1],)
    out = np.empty(X.shape[0], dtype=np.float64)
    lib().oracle_score(_ptr(X), dt, X.shape[0], X.shape[1], _ptr(w), float(bias), _ptr(out))
    return out


ACT_IDENTITY, ACT_RELU, ACT_GELU_TANH = 0, 1, 2


def score_mlp(X: np.ndarray, W1: np.ndarray, b1: np.ndarray, w2: np.ndarray, b2: float = 0.0,
              act: int = ACT_RELU) -> np.ndarray:
    """Two-layer Scorer (Eq. 6, App. B.3): s = w2 . act(W1 x + b1) + b2 in fp64; W1 is [dh, d]."""
    X, W1, w2 = _c(X), _c(W1), _c(w2)
    b1 = np.ascontiguousarray(b1, dtype=np.float32)
    dt = _dtype_code(X)
    assert _dtype_code(W1) == dt and _dtype_code(w2) == dt
    assert X.ndim == 2 and W1.ndim == 2 and W1.shape[1] == X.shape[1] and b1.shape == (W1.shape[0],) and w2.shape == (W1.shape[0],)
    out = np.empty(X.shape[0], dtype=np.float64)
    lib().oracle_score_mlp(_ptr(X), dt, X.shape[0], X.shape[1], _ptr(W1), _ptr(b1), _ptr(w2), float(b2),
                           W1.shape[0], int(act), _ptr(out))
    return out


def select(scores: np.ndarray, k: int, flags: int = 0) -> np.ndarray:
    """TopK of one sequence (Eq. 14): ascending positions of the k best scores,
    ties to the lower position.  fp32 scores are widened exactly to fp64."""
    s = np.ascontiguousarray(scores, dtype=np.float64)
    idx = np.empty(int(k), dtype=np.int32)
    rc = lib().oracle_select(_ptr(s), s.shape[0], int(k), int(flags), _ptr(idx))
    if rc != 0:
        raise ValueError(f"oracle_select rejected n={s.shape[0]} k={k}")
    return idx


def select_threshold(scores: np.ndarray, lam: float) -> np.ndarray:
    """Threshold selection of one sequence (Eq. 8): ascending positions whose score is above Lambda."""
    s = np.ascontiguousarray(scores, dtype=np.float64)
    idx = np.empty(max(s.shape[0], 1), dtype=np.int32)
    n = lib().oracle_select_threshold(_ptr(s), s.shape[0], float(lam), _ptr(idx))
    return idx[:n].copy()


def estimate_threshold(sample: np.ndarray, r: int) -> float:
    """Lambda from sampled scores (text after Eq. 8): the (ceil(m/r)+1)-th largest, -inf if there is none."""
    s = np.ascontiguousarray(sample, dtype=np.float64)
    return float(lib().oracle_estimate_threshold(_ptr(s), s.shape[0], int(r)))


def gather(src: np.ndarray, idx: np.ndarray, pos_base: int, cache: np.ndarray,
           cache_pos: np.ndarray | None, length: int) -> int:
    """Append rows ``src[idx]`` to ``cache`` after ``length`` rows (Eq. 5), in place.

    ``src`` is [n, ...], ``cache`` is [capacity, ...] of the same dtype and row
    shape; returns the new length.
    """
    assert src.flags.c_contiguous and cache.flags.c_contiguous and src.dtype == cache.dtype
    row_bytes = src.strides[0]
    assert cache.strides[0] == row_bytes
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    new_len = lib().oracle_gather(_ptr(src), row_bytes, _ptr(idx), idx.shape[0], int(pos_base),
                                  _ptr(cache), _ptr(cache_pos), int(length), cache.shape[0])
    if new_len < 0:
        raise ValueError("oracle_gather: cache region overflow")
    return int(new_len)


def pool(src: np.ndarray, r: int, pos_base: int = 0):
    """Mean pooling of even chunks of r rows (Sec. 5.1, the Compressive baseline with mean pooling).

    ``src`` is [n, ...] in a storage dtype; returns (means [k, ...] fp64, positions int32[k]) with k = ceil(n / r),
    positions = pos_base + the last row of each chunk."""
    src = _c(src)
    n = src.shape[0]
    width = int(np.prod(src.shape[1:])) if src.ndim > 1 else 1
    k = num_nuggets(n, r)
    out = np.empty((k,) + src.shape[1:], dtype=np.float64)
    pos = np.empty(k, dtype=np.int32)
    got = lib().oracle_pool(_ptr(src), _dtype_code(src), n, width, int(r), int(pos_base), _ptr(out), _ptr(pos))
    assert got == k
    return out, pos


def attend(Q: np.ndarray, q_pos0: int, scale: float,
           cK: np.ndarray, cV: np.ndarray, cpos: np.ndarray, clen: int,
           lK: np.ndarray | None, lV: np.ndarray | None, llen: int, lpos0: int):
    """Attention of one sequence's queries over [nuggets ; local] (Eq. 4, 9, 13, 16).

    Q [Tq, H, dh]; cK/cV [>=clen, H, dh]; lK/lV [>=llen, H, dh] or None.
    Returns (O [Tq, H, dh] fp64, lse [Tq, H] fp64).
    """
    Q = _c(Q)
    dt = _dtype_code(Q)
    Tq, H, dh = Q.shape
    if clen > 0:
        cK, cV = _c(cK), _c(cV)
        cpos = np.ascontiguousarray(cpos, dtype=np.int32)
        assert _dtype_code(cK) == dt and cK.shape[1:] == (H, dh) and cK.shape[0] >= clen
    else:
        cK = cV = cpos = None
    if llen > 0:
        lK, lV = _c(lK), _c(lV)
        assert _dtype_code(lK) == dt and lK.shape[1:] == (H, dh) and lK.shape[0] >= llen
    else:
        lK = lV = None
    O = np.empty((Tq, H, dh), dtype=np.float64)
    lse = np.empty((Tq, H), dtype=np.float64)
    lib().oracle_attend(_ptr(Q), dt, Tq, int(q_pos0), H, dh, float(scale),
                        _ptr(cK), _ptr(cV), _ptr(cpos), int(clen),
                        _ptr(lK), _ptr(lV), int(llen), int(lpos0), _ptr(O), _ptr(lse))
    return O, lse


# ---------------------------------------------------------------------------
# Ragged-batch loops (sequence b owns rows [off[b], off[b+1]) of a packed array)
# ---------------------------------------------------------------------------

def select_ragged(scores: np.ndarray, seq_off, nug_off, flags: int = 0) -> np.ndarray:
    B = len(seq_off) - 1
    idx = np.empty(int(nug_off[B]), dtype=np.int32)
    for b in range(B):
        k = int(nug_off[b + 1] - nug_off[b])
        idx[nug_off[b]:nug_off[b + 1]] = select(scores[seq_off[b]:seq_off[b + 1]], k, flags)
    return idx


def gather_ragged(K: np.ndarray, V: np.ndarray, seq_off, idx: np.ndarray, nug_off, pos_base,
                  cacheK: np.ndarray, cacheV: np.ndarray, cache_pos: np.ndarray,
                  cache_off, cache_len) -> list[int]:
    """Per sequence: append its selected K and V rows to its cache region.  Returns new lengths."""
    B = len(seq_off) - 1
    out = []
    for b in range(B):
        ib = idx[nug_off[b]:nug_off[b + 1]]
        s0, s1 = int(seq_off[b]), int(seq_off[b + 1])
        c0, c1 = int(cache_off[b]), int(cache_off[b + 1])
        gather(K[s0:s1], ib, int(pos_base[b]), cacheK[c0:c1], cache_pos[c0:c1], int(cache_len[b]))
        out.append(gather(V[s0:s1], ib, int(pos_base[b]), cacheV[c0:c1], None, int(cache_len[b])))
    return out


def attend_ragged(Q: np.ndarray, q_off, q_pos0, scale: float,
                  cacheK, cacheV, cache_pos, cache_off, cache_len,
                  locK, locV, loc_off, loc_len, loc_pos0):
    """Loop ``attend`` over the sequences of a ragged batch.  Returns (O, lse) packed like Q."""
    B = len(q_off) - 1
    T, H, dh = Q.shape
    O = np.zeros((T, H, dh), dtype=np.float64)
    lse = np.full((T, H), -np.inf, dtype=np.float64)
    for b in range(B):
        t0, t1 = int(q_off[b]), int(q_off[b + 1])
        if t1 == t0:
            continue
        c0 = int(cache_off[b])
        clen = int(cache_len[b])
        llen = int(loc_len[b]) if loc_len is not None else 0
        l0 = int(loc_off[b]) if llen > 0 else 0
        o, l = attend(Q[t0:t1], int(q_pos0[b]), scale,
                      cacheK[c0:c0 + clen] if clen else None,
                      cacheV[c0:c0 + clen] if clen else None,
                      cache_pos[c0:c0 + clen] if clen else None, clen,
                      locK[l0:l0 + llen] if llen else None,
                      locV[l0:l0 + llen] if llen else None, llen,
                      int(loc_pos0[b]) if llen else 0)
        O[t0:t1] = o
        lse[t0:t1] = l
    return O, lse
