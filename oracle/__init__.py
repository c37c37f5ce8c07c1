"""fp64 CPU oracle for the first-layer cached attention path.

TEST INFRASTRUCTURE ONLY: only the tests, the smoke check and the CPU-baseline
leg of the benchmark may import this package.  It shares no code with the CUDA
path and imports nothing from it.  The arithmetic lives in
``lacache_oracle.c`` (plain C, double precision, OpenMP over rows); this module
only compiles it with gcc and marshals numpy arrays.

Functions mirror the paper's statements:
  * ``rope``            Eq. 1 (Sec. 3.3.2), half-split pairing.
  * ``attention``       the plain softmax-attention definition (Sec. 3.3.3,
                        App. B.2) on RoPE-rotated Q/K, with L = m + log l.
  * ``state_stream``    Eq. 2-6 recurrence over a subset of keys.
  * ``state_merge``     merge of two partial states implied by Eq. 2-6.
  * ``build_state``     Algorithm 1, GenStep=True, the cached triple.
  * ``reuse_step``      Algorithm 1, GenStep=False.
"""
import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lacache_oracle.c")
_LIB_PATH = os.path.join(_HERE, "liblacache_oracle.so")
_lib = None


def build(force=False):
    """Compile the C oracle with gcc (no CUDA involved)."""
    if (not force and os.path.exists(_LIB_PATH)
            and os.path.getmtime(_LIB_PATH) >= os.path.getmtime(_SRC)):
        return _LIB_PATH
    tmp = _LIB_PATH + ".tmp%d" % os.getpid()
    subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11",
                           "-o", tmp, _SRC, "-lm"])
    os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_num_threads.restype = ctypes.c_int
    return _lib


def num_threads():
    return int(_load().oracle_num_threads())


def _d(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def _p(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def _u8(a):
    return np.ascontiguousarray(a, dtype=np.uint8)


def rope(x, pos, theta):
    """y[t,h,:] = R(pos[t]) x[t,h,:]; x is [T,H,d]."""
    x = _d(x)
    T, H, d = x.shape
    pos = _i32(pos)
    y = np.empty_like(x)
    _load().oracle_rope(_p(x), _p(pos), T, H, d, ctypes.c_double(theta), _p(y))
    return y


def attention(q, k, v, cu_seqlens, theta, scale, rows=None):
    """Plain definition on pre-RoPE q [T,Hq,d], k,v [T,Hkv,d].

    Returns (out [n_rows,Hq,d], lse [n_rows,Hq]) for the listed packed rows
    (all rows when ``rows`` is None).
    """
    q, k, v = _d(q), _d(k), _d(v)
    cu = _i32(cu_seqlens)
    B = cu.shape[0] - 1
    T, Hq, d = q.shape
    Hkv = k.shape[1]
    assert cu[-1] == T and k.shape == v.shape == (T, Hkv, d) and Hq % Hkv == 0
    rows = _i32(np.arange(T) if rows is None else rows)
    out = np.empty((rows.shape[0], Hq, d), dtype=np.float64)
    lse = np.empty((rows.shape[0], Hq), dtype=np.float64)
    _load().oracle_attention(_p(q), _p(k), _p(v), _p(cu), B, Hq, Hkv, d,
                             ctypes.c_double(theta), ctypes.c_double(scale),
                             _p(rows), rows.shape[0], _p(out), _p(lse))
    return out, lse


def state_stream(qrot, krot, v, keep, scale, Bc, state=None):
    """Eq. 2-6 over the keys with keep[j] != 0; qrot [d], krot,v [n,d] (rotated).

    Returns (m, l, O).  ``state`` is the starting (m, l, O) or None for empty.
    """
    qrot, krot, v = _d(qrot), _d(krot), _d(v)
    n, d = krot.shape
    keep = _u8(keep)
    if state is None:
        m, l, O = -np.inf, 0.0, np.zeros(d)
    else:
        m, l, O = state
    mm = ctypes.c_double(m)
    ll = ctypes.c_double(l)
    O = _d(O).copy()
    _load().oracle_state_stream(_p(qrot), _p(krot), _p(v), _p(keep), n, d,
                                ctypes.c_double(scale), int(Bc),
                                ctypes.byref(mm), ctypes.byref(ll), _p(O))
    return mm.value, ll.value, O


def state_merge(s1, s2):
    """Merge two partial states (m, l, O) over disjoint key sets."""
    m1, l1, O1 = s1
    m2, l2, O2 = s2
    O1 = _d(O1).copy()
    O2 = _d(O2)
    mm = ctypes.c_double(m1)
    ll = ctypes.c_double(l1)
    _load().oracle_state_merge(ctypes.byref(mm), ctypes.byref(ll), _p(O1),
                               ctypes.c_double(m2), ctypes.c_double(l2), _p(O2),
                               O1.shape[0])
    return mm.value, ll.value, O1


def build_state(q, k, v, cu_seqlens, is_block, theta, scale, Bc=64):
    """Cached triple over the fixed keys for every (token, head)."""
    q, k, v = _d(q), _d(k), _d(v)
    cu = _i32(cu_seqlens)
    B = cu.shape[0] - 1
    T, Hq, d = q.shape
    Hkv = k.shape[1]
    isb = _u8(is_block)
    m = np.empty((T, Hq))
    l = np.empty((T, Hq))
    O = np.empty((T, Hq, d))
    _load().oracle_build_state(_p(q), _p(k), _p(v), _p(cu), B, _p(isb), Hq, Hkv, d,
                               ctypes.c_double(theta), ctypes.c_double(scale), int(Bc),
                               _p(m), _p(l), _p(O))
    return m, l, O


def reuse_step(q, k, v, cu_seqlens, is_block, theta, scale, state, Bc=64):
    """Algorithm 1 reuse pass; returns (out [T,Hq,d], lse [T,Hq])."""
    q, k, v = _d(q), _d(k), _d(v)
    cu = _i32(cu_seqlens)
    B = cu.shape[0] - 1
    T, Hq, d = q.shape
    Hkv = k.shape[1]
    isb = _u8(is_block)
    mc, lc, Oc = (_d(a) for a in state)
    out = np.empty((T, Hq, d))
    lse = np.empty((T, Hq))
    _load().oracle_reuse_step(_p(q), _p(k), _p(v), _p(cu), B, _p(isb), Hq, Hkv, d,
                              ctypes.c_double(theta), ctypes.c_double(scale), int(Bc),
                              _p(mc), _p(lc), _p(Oc), _p(out), _p(lse))
    return out, lse
