"""Thin ctypes binding over the C ABI of ``include/lacache.h``.

Argument marshalling only: every step of the path runs inside the CUDA
library.  Function names mirror the C entry points.  Tensors are torch tensors
(device memory for the plain calls, host memory for the ``*_host`` calls);
only their ``data_ptr()`` crosses the boundary.  There is no fallback: if
``liblacache.so`` is missing or cannot be loaded, ``load()`` raises.
"""
import ctypes
import os

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "liblacache.so")

OK, ERR_INVALID_ARG, ERR_SHAPE, ERR_STATE, ERR_UNSUPPORTED, ERR_OOM, ERR_CUDA, ERR_TIMEOUT = range(8)
DTYPE_BF16, DTYPE_FP32 = 0, 1
ENGINE_AUTO, ENGINE_SIMT, ENGINE_TCGEN05 = 0, 1, 2
OUT_BF16, OUT_FP32 = 0, 1
PRECISION_PLAIN, PRECISION_SPLIT, PRECISION_FP16 = 0, 1, 3
GRANULARITY_TOKEN, GRANULARITY_TILE = 0, 1

EXPORTS = [
    "lacache_version", "lacache_create", "lacache_destroy", "lacache_build", "lacache_step",
    "lacache_full_recompute", "lacache_build_host", "lacache_step_host", "lacache_export_state",
    "lacache_export_rope_cache", "lacache_export_index_meta", "lacache_total_tokens",
    "lacache_last_launch_count", "lacache_engine", "lacache_set_timing_events",
    "lacache_full_recompute_static", "lacache_poll_status", "lacache_last_error",
    "lacache_qkv_create", "lacache_qkv_destroy", "lacache_qkv_project", "lacache_build_tokens",
    "lacache_step_tokens", "lacache_qkv_set_timing_events", "lacache_qkv_last_launch_count",
    "lacache_qkv_poll_status", "lacache_qkv_last_error", "lacache_set_step_overlap",
    "lacache_build_tokens_update", "lacache_build_incremental", "lacache_build_advance",
    "lacache_build_tokens_incremental", "lacache_build_advance_tokens", "lacache_sample_block",
    "lacache_set_span_ring", "lacache_join_host", "lacache_qkv_set_wait_limit",
    "lacache_qkv_project_without_norm",
]


class LacacheConfig(ctypes.Structure):
    _fields_ = [
        ("dtype", ctypes.c_int), ("engine", ctypes.c_int),
        ("n_q_heads", ctypes.c_int), ("n_kv_heads", ctypes.c_int), ("head_dim", ctypes.c_int),
        ("rope_theta", ctypes.c_float), ("softmax_scale", ctypes.c_float),
        ("batch", ctypes.c_int), ("prompt_lens", ctypes.POINTER(ctypes.c_int32)),
        ("gen_len", ctypes.c_int), ("block_len", ctypes.c_int),
        ("sc_tiles_per_chunk", ctypes.c_int),
        ("out_dtype", ctypes.c_int), ("precision_mode", ctypes.c_int), ("cache_granularity", ctypes.c_int),
    ]


class LacacheQkvConfig(ctypes.Structure):
    _fields_ = [
        ("vocab", ctypes.c_int), ("d_model", ctypes.c_int), ("n_q_heads", ctypes.c_int),
        ("n_kv_heads", ctypes.c_int), ("head_dim", ctypes.c_int), ("rms_eps", ctypes.c_float),
        ("max_tokens", ctypes.c_int), ("embed", ctypes.c_void_p), ("norm_weight", ctypes.c_void_p),
        ("w_qkv", ctypes.c_void_p),
    ]


class LacacheError(RuntimeError):
    def __init__(self, status, message):
        super().__init__("lacache status %d: %s" % (status, message))
        self.status = status


_lib = None


def load():
    """Loads the CUDA library; raises if it is not built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError("%s not found: build it with `python -m paper_2607_16339_b200.build` "
                           "(there is no CPU fallback)" % LIB_PATH)
    lib = ctypes.CDLL(LIB_PATH)
    vp, ip = ctypes.c_void_p, ctypes.c_int
    lib.lacache_version.restype = ip
    lib.lacache_create.argtypes = [ctypes.POINTER(LacacheConfig), ctypes.POINTER(vp)]
    lib.lacache_destroy.argtypes = [vp]
    lib.lacache_build.argtypes = [vp, ip, vp, vp, vp, vp]
    lib.lacache_step.argtypes = [vp, vp, vp, vp, vp, vp, vp]
    lib.lacache_build_incremental.argtypes = [vp, ip, vp, vp, vp, vp]
    lib.lacache_build_advance.argtypes = [vp, vp, vp, vp, vp]
    lib.lacache_full_recompute.argtypes = [vp, vp, vp, vp, vp, vp, vp]
    lib.lacache_build_host.argtypes = [vp, ip, vp, vp, vp, vp]
    lib.lacache_step_host.argtypes = [vp, vp, vp, vp, vp, vp, vp]
    lib.lacache_export_state.argtypes = [vp, vp, vp, vp, vp]
    lib.lacache_export_rope_cache.argtypes = [vp, vp, vp, vp, vp]
    lib.lacache_export_index_meta.argtypes = [vp, vp, vp, vp, vp]
    lib.lacache_set_timing_events.argtypes = [vp, vp, vp]
    lib.lacache_set_step_overlap.argtypes = [vp, ip]
    lib.lacache_set_span_ring.argtypes = [vp, vp, ip]
    lib.lacache_join_host.argtypes = [vp, vp]
    lib.lacache_sample_block.argtypes = [vp, vp, ip, ip, vp, vp, vp, vp]
    lib.lacache_full_recompute_static.argtypes = [ip, ip, ip, ip, ip, ctypes.c_float, ctypes.c_float, vp, vp, vp, vp,
                                                  vp, vp]
    lib.lacache_total_tokens.argtypes = [vp]
    lib.lacache_last_launch_count.argtypes = [vp]
    lib.lacache_engine.argtypes = [vp]
    lib.lacache_poll_status.argtypes = [vp]
    lib.lacache_last_error.argtypes = [vp]
    lib.lacache_last_error.restype = ctypes.c_char_p
    lib.lacache_qkv_create.argtypes = [ctypes.POINTER(LacacheQkvConfig), ctypes.POINTER(vp)]
    lib.lacache_qkv_destroy.argtypes = [vp]
    lib.lacache_qkv_project.argtypes = [vp, vp, vp, ip, vp, vp, vp, vp, vp]
    lib.lacache_build_tokens.argtypes = [vp, vp, ip, vp, vp, vp]
    lib.lacache_build_tokens_incremental.argtypes = [vp, vp, ip, vp, vp, vp]
    lib.lacache_build_advance_tokens.argtypes = [vp, vp, vp, vp, vp]
    lib.lacache_step_tokens.argtypes = [vp, vp, vp, vp, vp, vp, vp]
    lib.lacache_build_tokens_update.argtypes = [vp, vp, ip, vp, vp, vp, ip, vp]
    lib.lacache_qkv_set_wait_limit.argtypes = [vp, ctypes.c_double]
    lib.lacache_qkv_project_without_norm.argtypes = [vp, vp, ip, vp, vp, vp, vp]
    lib.lacache_qkv_set_timing_events.argtypes = [vp, vp, vp]
    lib.lacache_qkv_last_launch_count.argtypes = [vp]
    lib.lacache_qkv_poll_status.argtypes = [vp]
    lib.lacache_qkv_last_error.argtypes = [vp]
    lib.lacache_qkv_last_error.restype = ctypes.c_char_p
    for name in EXPORTS:
        if name not in ("lacache_last_error", "lacache_qkv_last_error"):
            getattr(lib, name).restype = ip
    _lib = lib
    return lib


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        import torch
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def full_recompute_static(dtype, n_q_heads, n_kv_heads, head_dim, rope_theta, q_pre, k_pre, v_pre, out,
                          lse=None, softmax_scale=0.0, stream=None):
    """Plain attention for one sequence without any device allocation (the
    scratch is a fixed array inside the library).  Mirrors
    ``lacache_full_recompute_static``; raises LacacheError on a non-zero status."""
    lib = load()
    st = lib.lacache_full_recompute_static(int(dtype), int(q_pre.shape[0]), int(n_q_heads), int(n_kv_heads),
                                           int(head_dim), float(rope_theta), float(softmax_scale), _ptr(q_pre),
                                           _ptr(k_pre), _ptr(v_pre), _ptr(out), _ptr(lse), _stream(stream))
    if st != OK:
        raise LacacheError(st, (lib.lacache_last_error(None) or b"").decode())


class Context:
    """Owns one ``lacache_ctx``.  Methods mirror the C calls one to one."""

    def __init__(self, dtype, n_q_heads, n_kv_heads, head_dim, rope_theta, prompt_lens, gen_len,
                 block_len, softmax_scale=0.0, engine=ENGINE_AUTO, sc_tiles_per_chunk=0,
                 out_dtype=OUT_FP32, precision_mode=PRECISION_SPLIT, cache_granularity=GRANULARITY_TOKEN):
        self._lib = load()
        self._h = ctypes.c_void_p()
        pl = (ctypes.c_int32 * len(prompt_lens))(*[int(p) for p in prompt_lens])
        cfg = LacacheConfig(int(dtype), int(engine), int(n_q_heads), int(n_kv_heads), int(head_dim),
                            float(rope_theta), float(softmax_scale), len(prompt_lens), pl,
                            int(gen_len), int(block_len), int(sc_tiles_per_chunk), int(out_dtype),
                            int(precision_mode), int(cache_granularity))
        st = self._lib.lacache_create(ctypes.byref(cfg), ctypes.byref(self._h))
        if st != OK:
            self._h = ctypes.c_void_p()
            raise LacacheError(st, (self._lib.lacache_last_error(None) or b"").decode())
        self.n_q_heads, self.n_kv_heads, self.head_dim = n_q_heads, n_kv_heads, head_dim
        self.batch, self.block_len = len(prompt_lens), block_len
        self.out_dtype = out_dtype

    @classmethod
    def from_workload(cls, wl, **kw):
        return cls(DTYPE_BF16 if wl.dtype == "bf16" else DTYPE_FP32, wl.n_q_heads, wl.n_kv_heads,
                   wl.head_dim, wl.rope_theta, wl.prompt_lens, wl.gen_len, wl.block_len, **kw)

    def _check(self, st):
        if st != OK:
            raise LacacheError(st, (self._lib.lacache_last_error(self._h) or b"").decode())

    def destroy(self):
        if self._h:
            self._lib.lacache_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    @property
    def total_tokens(self):
        return self._lib.lacache_total_tokens(self._h)

    @property
    def engine(self):
        return self._lib.lacache_engine(self._h)

    @property
    def last_launch_count(self):
        return self._lib.lacache_last_launch_count(self._h)

    def build(self, block_idx, q_pre, k_pre, v_pre, stream=None):
        self._check(self._lib.lacache_build(self._h, int(block_idx), _ptr(q_pre), _ptr(k_pre),
                                            _ptr(v_pre), _stream(stream)))

    def build_incremental(self, block_idx, q_pre, k_pre, v_pre, stream=None):
        self._check(self._lib.lacache_build_incremental(self._h, int(block_idx), _ptr(q_pre), _ptr(k_pre),
                                                        _ptr(v_pre), _stream(stream)))

    def build_advance(self, q_fin, k_fin, v_fin, stream=None):
        self._check(self._lib.lacache_build_advance(self._h, _ptr(q_fin), _ptr(k_fin), _ptr(v_fin),
                                                    _stream(stream)))

    def step(self, q_blk, k_blk, v_blk, out, lse=None, stream=None):
        self._check(self._lib.lacache_step(self._h, _ptr(q_blk), _ptr(k_blk), _ptr(v_blk), _ptr(out),
                                           _ptr(lse), _stream(stream)))

    def full_recompute(self, q_pre, k_pre, v_pre, out, lse=None, stream=None):
        self._check(self._lib.lacache_full_recompute(self._h, _ptr(q_pre), _ptr(k_pre), _ptr(v_pre),
                                                     _ptr(out), _ptr(lse), _stream(stream)))

    def build_host(self, block_idx, q_pre, k_pre, v_pre, stream=None):
        self._check(self._lib.lacache_build_host(self._h, int(block_idx), _ptr(q_pre), _ptr(k_pre),
                                                 _ptr(v_pre), _stream(stream)))

    def step_host(self, q_blk, k_blk, v_blk, out, lse=None, stream=None):
        self._check(self._lib.lacache_step_host(self._h, _ptr(q_blk), _ptr(k_blk), _ptr(v_blk),
                                                _ptr(out), _ptr(lse), _stream(stream)))

    def join_host(self, stream=None):
        self._check(self._lib.lacache_join_host(self._h, _stream(stream)))

    def export_state(self, m, l, o_acc, stream=None):
        self._check(self._lib.lacache_export_state(self._h, _ptr(m), _ptr(l), _ptr(o_acc), _stream(stream)))

    def export_rope_cache(self, q_rot, k_rot, v, stream=None):
        self._check(self._lib.lacache_export_rope_cache(self._h, _ptr(q_rot), _ptr(k_rot), _ptr(v),
                                                        _stream(stream)))

    def export_index_meta(self):
        import numpy as np
        T = self.total_tokens
        seq = np.empty(T, np.int32); pos = np.empty(T, np.int32); isb = np.empty(T, np.int32)
        kvh = np.empty(self.n_q_heads, np.int32)
        p = lambda a: a.ctypes.data_as(ctypes.c_void_p)
        self._check(self._lib.lacache_export_index_meta(self._h, p(seq), p(pos), p(isb), p(kvh)))
        return seq, pos, isb, kvh

    def set_step_overlap(self, enable):
        self._check(self._lib.lacache_set_step_overlap(self._h, int(bool(enable))))

    def build_tokens(self, producer, block_idx, token_ids=None, hidden=None, stream=None):
        self._check(self._lib.lacache_build_tokens(self._h, producer._h, int(block_idx), _ptr(token_ids),
                                                   _ptr(hidden), _stream(stream)))

    def build_tokens_incremental(self, producer, block_idx, token_ids=None, hidden=None, stream=None):
        self._check(self._lib.lacache_build_tokens_incremental(self._h, producer._h, int(block_idx),
                                                               _ptr(token_ids), _ptr(hidden), _stream(stream)))

    def build_advance_tokens(self, producer, fin_token_ids=None, fin_hidden=None, stream=None):
        self._check(self._lib.lacache_build_advance_tokens(self._h, producer._h, _ptr(fin_token_ids),
                                                           _ptr(fin_hidden), _stream(stream)))

    def build_tokens_update(self, producer, block_idx, rows, token_ids=None, hidden=None, stream=None):
        self._check(self._lib.lacache_build_tokens_update(self._h, producer._h, int(block_idx), _ptr(rows),
                                                          _ptr(token_ids), _ptr(hidden), int(rows.shape[0]),
                                                          _stream(stream)))

    def step_tokens(self, producer, out, lse=None, blk_token_ids=None, blk_hidden=None, stream=None):
        self._check(self._lib.lacache_step_tokens(self._h, producer._h, _ptr(blk_token_ids), _ptr(blk_hidden),
                                                  _ptr(out), _ptr(lse), _stream(stream)))

    def sample_block(self, logits, conf, token, lse=None, stream=None):
        """logits [T, vocab] bf16 or fp32; conf fp32 / token int32 / lse fp32 [B * L_b]."""
        import torch
        dt = DTYPE_BF16 if logits.dtype == torch.bfloat16 else DTYPE_FP32
        self._check(self._lib.lacache_sample_block(self._h, _ptr(logits), dt, int(logits.shape[-1]), _ptr(conf),
                                                   _ptr(token), _ptr(lse), _stream(stream)))

    def set_span_ring(self, ring):
        """ring: int64 / uint64 device tensor [n_slots, 2] initialised to {UINT64_MAX, 0} by the caller, or
        None to switch the hook off."""
        if ring is None:
            self._check(self._lib.lacache_set_span_ring(self._h, None, 0))
        else:
            self._check(self._lib.lacache_set_span_ring(self._h, _ptr(ring), int(ring.shape[0])))

    def set_timing_events(self, ev_start, ev_stop):
        """torch.cuda.Event pair (already recorded once) or (None, None)."""
        h = lambda e: None if e is None else ctypes.c_void_p(e.cuda_event)
        self._check(self._lib.lacache_set_timing_events(self._h, h(ev_start), h(ev_stop)))

    def poll_status(self):
        st = self._lib.lacache_poll_status(self._h)
        return st, (self._lib.lacache_last_error(self._h) or b"").decode()


class QkvProducer:
    """Owns one ``lacache_qkv`` (the token-wise producer).  The weight tensors
    (bf16, on the device) are kept referenced here because the library does not
    copy them."""

    def __init__(self, embed, norm_weight, w_qkv, n_q_heads, n_kv_heads, head_dim, rms_eps, max_tokens):
        self._lib = load()
        self._h = ctypes.c_void_p()
        self._weights = (embed, norm_weight, w_qkv)
        vocab = 0 if embed is None else int(embed.shape[0])
        cfg = LacacheQkvConfig(vocab, int(w_qkv.shape[1]), int(n_q_heads), int(n_kv_heads), int(head_dim),
                               float(rms_eps), int(max_tokens),
                               None if embed is None else embed.data_ptr(), norm_weight.data_ptr(),
                               w_qkv.data_ptr())
        st = self._lib.lacache_qkv_create(ctypes.byref(cfg), ctypes.byref(self._h))
        if st != OK:
            self._h = ctypes.c_void_p()
            raise LacacheError(st, (self._lib.lacache_qkv_last_error(None) or b"").decode())

    def _check(self, st):
        if st != OK:
            raise LacacheError(st, (self._lib.lacache_qkv_last_error(self._h) or b"").decode())

    def destroy(self):
        if self._h:
            self._lib.lacache_qkv_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    def project(self, n_tokens, q, k, v, token_ids=None, hidden=None, h_out=None, stream=None):
        self._check(self._lib.lacache_qkv_project(self._h, _ptr(token_ids), _ptr(hidden), int(n_tokens),
                                                  _ptr(q), _ptr(k), _ptr(v), _ptr(h_out), _stream(stream)))

    def set_wait_limit(self, microseconds):
        self._check(self._lib.lacache_qkv_set_wait_limit(self._h, float(microseconds)))

    def project_without_norm(self, n_tokens, q, k, v, hidden, stream=None):
        """Test hook: the projection kernel alone, whose wait for its operand rows then runs out."""
        self._check(self._lib.lacache_qkv_project_without_norm(self._h, _ptr(hidden), int(n_tokens), _ptr(q),
                                                               _ptr(k), _ptr(v), _stream(stream)))

    def set_timing_events(self, ev_start, ev_stop):
        h = lambda e: None if e is None else ctypes.c_void_p(e.cuda_event)
        self._check(self._lib.lacache_qkv_set_timing_events(self._h, h(ev_start), h(ev_stop)))

    @property
    def last_launch_count(self):
        return self._lib.lacache_qkv_last_launch_count(self._h)

    def poll_status(self):
        st = self._lib.lacache_qkv_poll_status(self._h)
        return st, (self._lib.lacache_qkv_last_error(self._h) or b"").decode()
