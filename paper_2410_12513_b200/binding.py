"""ctypes binding of ``libfirst.so``: the same calls as ``include/first.h``, taking torch
CUDA tensors.  Argument marshalling only -- no arithmetic happens here."""
from __future__ import annotations

import ctypes as C
from pathlib import Path

import torch

_PKG = Path(__file__).resolve().parent
_LIBPATH = _PKG / "libfirst.so"
_lib = None

FIRST_DTYPE_F32, FIRST_DTYPE_BF16 = 0, 1
MEAN_OF_SIGMOID, SIGMOID_OF_MEAN = 0, 1
FLAG_KV_FULL, FLAG_BAD_TOKEN, FLAG_BAD_MASK, FLAG_WAIT_EXPIRED, FLAG_EMPTY_SEQ, FLAG_BAD_SEQ_TABLE = 1, 2, 4, 8, 16, 32


class FirstError(RuntimeError):
    def __init__(self, status, what):
        self.status = status
        msg = lib().first_status_string(status).decode()
        super().__init__(f"{what}: status {status} ({msg})")


class ModelDesc(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_q_heads", "n_kv_heads", "head_dim", "ffn_dim",
                                         "vocab")] + \
               [("rope_base", C.c_float), ("rms_eps", C.c_float), ("dtype", C.c_int32), ("max_batch", C.c_int32),
                ("max_tokens_per_seq", C.c_int32)]


class Weights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("lm_head", C.c_void_p), ("final_norm", C.c_void_p),
                ("attn_norm", C.POINTER(C.c_void_p)), ("wqkv", C.POINTER(C.c_void_p)),
                ("wo", C.POINTER(C.c_void_p)), ("ffn_norm", C.POINTER(C.c_void_p)),
                ("w_gate_up", C.POINTER(C.c_void_p)), ("w_down", C.POINTER(C.c_void_p))]


class KVCacheC(C.Structure):
    _fields_ = [("k", C.POINTER(C.c_void_p)), ("v", C.POINTER(C.c_void_p)), ("slab_off", C.c_void_p),
                ("slab_cap", C.c_void_p), ("len", C.c_void_p), ("pos", C.c_void_p), ("cap_total", C.c_int64),
                ("per_layer", C.c_int32), ("cap_total_l", C.POINTER(C.c_int64))]


def library_path() -> Path:
    return _LIBPATH


def lib():
    """Load the CUDA library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not _LIBPATH.exists():
            raise FileNotFoundError(f"{_LIBPATH} is missing: build it with `python -m paper_2410_12513_b200.build`")
        L = C.CDLL(str(_LIBPATH))
        L.first_status_string.restype = C.c_char_p
        L.first_status_string.argtypes = [C.c_int]
        L.first_create.argtypes = [C.POINTER(ModelDesc), C.POINTER(Weights), C.POINTER(C.c_void_p)]
        L.first_destroy.argtypes = [C.c_void_p]
        L.first_prefill_route.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_int32, C.c_void_p, C.c_int32,
                                          C.c_int64, C.c_void_p, C.c_void_p, C.c_float, C.c_int32, C.c_void_p,
                                          C.c_void_p, C.c_void_p]
        L.first_prefill_route_static.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_int32, C.c_void_p,
                                                 C.c_int32, C.c_int64, C.c_void_p, C.c_void_p, C.c_float, C.c_int32,
                                                 C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.first_prefill_route_static.restype = C.c_int
        L.first_prefill.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.POINTER(KVCacheC), C.c_void_p,
                                    C.c_void_p, C.c_float, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                    C.c_void_p]
        L.first_prefill.restype = C.c_int
        L.first_set_mask.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p]
        L.first_get_plan.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.first_decode_step.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(KVCacheC), C.c_void_p, C.c_void_p,
                                        C.c_void_p, C.c_void_p]
        L.first_last_device_flags.argtypes = [C.c_void_p, C.POINTER(C.c_uint32), C.c_void_p]
        L.first_launch_count.restype = C.c_int64
        L.first_launch_count.argtypes = [C.c_void_p]
        L.first_set_option.argtypes = [C.c_void_p, C.c_char_p, C.c_int64]
        L.first_set_sampling.argtypes = [C.c_void_p, C.c_int32, C.c_float, C.c_void_p]
        L.first_set_sampling.restype = C.c_int
        L.first_sample_topk.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_float, C.c_void_p, C.c_void_p,
                                        C.c_void_p]
        L.first_sample_topk.restype = C.c_int
        L.first_profile.argtypes = [C.c_void_p, C.c_int32]
        L.first_profile.restype = C.c_int
        L.first_profile_read.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]
        L.first_profile_read.restype = C.c_int
        L.first_set_mask_host.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p]
        L.first_set_mask_host.restype = C.c_int
        L.first_pool_create.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.POINTER(C.c_void_p), C.POINTER(C.c_void_p),
                                        C.POINTER(C.c_void_p)]
        L.first_pool_destroy.argtypes = [C.c_void_p]
        L.first_seq_join.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.POINTER(KVCacheC), C.c_int32, C.c_int32,
                                     C.POINTER(C.c_int32), C.c_void_p]
        L.first_seq_leave.argtypes = [C.c_void_p, C.c_int32, C.c_void_p]
        L.first_pool_commit.argtypes = [C.c_void_p, C.c_void_p]
        L.first_pool_kv.argtypes = [C.c_void_p, C.POINTER(KVCacheC)]
        L.first_pool_stats.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(C.c_int32)]
        for name in ("first_pool_create", "first_pool_destroy", "first_seq_join", "first_seq_leave", "first_pool_commit",
                     "first_pool_kv", "first_pool_stats"):
            getattr(L, name).restype = C.c_int
        L.first_graph_count.argtypes = [C.c_void_p]
        L.first_graph_count.restype = C.c_int64
        L.first_selftest_wait_expiry.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]
        L.first_selftest_wait_expiry.restype = C.c_int
        L.first_step_trace.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.first_step_trace.restype = C.c_int
        L.first_kernel_class_count.restype = C.c_int32
        L.first_kernel_class_name.restype = C.c_char_p
        L.first_kernel_class_name.argtypes = [C.c_int32]
        for name in ("first_create", "first_destroy", "first_prefill_route", "first_set_mask", "first_get_plan",
                     "first_decode_step", "first_last_device_flags", "first_set_option"):
            getattr(L, name).restype = C.c_int
        _lib = L
    return _lib


def _dev(t, dtype=None, what="tensor"):
    if t is None:
        return None
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise TypeError(f"{what} must be a CUDA tensor")
    if not t.is_contiguous():
        raise ValueError(f"{what} must be contiguous")
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"{what} must have dtype {dtype}, got {t.dtype}")
    return C.c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def _ptr_array(tensors, dtype, what):
    arr = (C.c_void_p * len(tensors))()
    for i, t in enumerate(tensors):
        arr[i] = None if t is None else _dev(t, dtype, f"{what}[{i}]").value
    return arr


class KVCache:
    """Marshals caller-owned cache tensors into ``first_kv_cache``.

    k, v: lists (one per layer) of CUDA tensors [Hkv][cap_total][hd] (None allowed for
    layers no sequence keeps); slab_off int64 [B]; slab_cap int32 [B]; len int32 [L][B];
    pos int32 [B].  With two-dimensional slab_off / slab_cap ([L][B]) the tables are per
    layer and every layer's tensors may have their own height (a layer then holds slabs
    only for the sequences that keep it)."""

    def __init__(self, k, v, slab_off, slab_cap, len_, pos):
        self.k, self.v, self.slab_off, self.slab_cap, self.len, self.pos = k, v, slab_off, slab_cap, len_, pos
        first = next(t for t in k if t is not None)
        self._ka = _ptr_array(k, first.dtype, "kv.k")
        self._va = _ptr_array(v, first.dtype, "kv.v")
        per_layer = slab_off.dim() == 2
        if per_layer != (slab_cap.dim() == 2):
            raise ValueError("slab_off and slab_cap must both be [B] or both be [L][B]")
        self._heights = (C.c_int64 * len(k))(*[0 if t is None else int(t.shape[1]) for t in k])
        self.c = KVCacheC(C.cast(self._ka, C.POINTER(C.c_void_p)), C.cast(self._va, C.POINTER(C.c_void_p)),
                          _dev(slab_off, torch.int64, "slab_off"), _dev(slab_cap, torch.int32, "slab_cap"),
                          _dev(len_, torch.int32, "len"), _dev(pos, torch.int32, "pos"),
                          0 if per_layer else int(first.shape[1]), int(per_layer),
                          C.cast(self._heights, C.POINTER(C.c_int64)))


def first_create(shape, dtype, max_batch, max_tokens_per_seq, weights):
    """weights: dict with embed, lm_head, final_norm and per-layer lists attn_norm, wqkv, wo,
    ffn_norm, w_gate_up, w_down (CUDA tensors).  Returns (handle, keepalive)."""
    wd = torch.float32 if dtype == FIRST_DTYPE_F32 else torch.bfloat16
    desc = ModelDesc(shape.n_layers, shape.d_model, shape.n_q_heads, shape.n_kv_heads, shape.head_dim,
                     shape.ffn_dim, shape.vocab, float(shape.rope_base), float(shape.rms_eps), dtype,
                     int(max_batch), int(max_tokens_per_seq))
    arrs = {k: _ptr_array(weights[k], torch.float32 if k.endswith("norm") else wd, k)
            for k in ("attn_norm", "wqkv", "wo", "ffn_norm", "w_gate_up", "w_down")}
    w = Weights(_dev(weights["embed"], wd, "embed"), _dev(weights["lm_head"], wd, "lm_head"),
                _dev(weights["final_norm"], torch.float32, "final_norm"),
                *[C.cast(arrs[k], C.POINTER(C.c_void_p)) for k in
                  ("attn_norm", "wqkv", "wo", "ffn_norm", "w_gate_up", "w_down")])
    h = C.c_void_p()
    rc = lib().first_create(C.byref(desc), C.byref(w), C.byref(h))
    if rc:
        raise FirstError(rc, "first_create")
    return h, (weights, arrs)


def first_destroy(h):
    lib().first_destroy(h)


def first_prefill_route(h, layer, hidden, cu_seqlens, router_w, router_b, tau, mode, mask, scores=None,
                        stream=None):
    if hidden.dtype not in (torch.float32, torch.bfloat16):
        raise TypeError("hidden must be float32 or bfloat16")
    hd = FIRST_DTYPE_F32 if hidden.dtype == torch.float32 else FIRST_DTYPE_BF16
    rc = lib().first_prefill_route(h, layer, _dev(hidden, None, "hidden"), hd,
                                   _dev(cu_seqlens, torch.int32, "cu_seqlens"), cu_seqlens.numel() - 1,
                                   hidden.shape[0], _dev(router_w, torch.float32, "router_w"),
                                   _dev(router_b, torch.float32, "router_b"), float(tau), int(mode),
                                   _dev(mask, torch.uint8, "mask"), _dev(scores, torch.float32, "scores"),
                                   _stream(stream))
    if rc:
        raise FirstError(rc, "first_prefill_route")


def first_prefill_route_static(layer, n_layers, hidden, cu_seqlens, router_w, router_b, tau, mode, mask,
                               scores=None, flags=None, stream=None):
    """Context-free router call that allocates nothing (built-in scratch of
    FIRST_STATIC_ROUTE_MAX_TOKENS token scores); see first.h for the limits."""
    if hidden.dtype not in (torch.float32, torch.bfloat16):
        raise TypeError("hidden must be float32 or bfloat16")
    hd = FIRST_DTYPE_F32 if hidden.dtype == torch.float32 else FIRST_DTYPE_BF16
    rc = lib().first_prefill_route_static(int(layer), int(n_layers), hidden.shape[1], _dev(hidden, None, "hidden"), hd,
                                          _dev(cu_seqlens, torch.int32, "cu_seqlens"), cu_seqlens.numel() - 1,
                                          hidden.shape[0], _dev(router_w, torch.float32, "router_w"),
                                          _dev(router_b, torch.float32, "router_b"), float(tau), int(mode),
                                          _dev(mask, torch.uint8, "mask"), _dev(scores, torch.float32, "scores"),
                                          _dev(flags, torch.int32, "flags"), _stream(stream))
    if rc:
        raise FirstError(rc, "first_prefill_route_static")


def first_prefill(h, tokens, cu_seqlens, kv: KVCache, router_w=None, router_b=None, tau=0.5, mode=0, mask=None,
                  scores=None, logits=None, next_tokens=None, stream=None):
    """Whole prompt phase of a ragged batch; cu_seqlens is a HOST int32 array (numpy or a CPU tensor)."""
    import numpy as np
    cu = np.ascontiguousarray(np.asarray(cu_seqlens), dtype=np.int32)
    rc = lib().first_prefill(h, _dev(tokens, torch.int32, "tokens"), cu.ctypes.data, cu.size - 1, C.byref(kv.c),
                             _dev(router_w, torch.float32, "router_w"), _dev(router_b, torch.float32, "router_b"),
                             float(tau), int(mode), _dev(mask, torch.uint8, "mask"),
                             _dev(scores, torch.float32, "scores"), _dev(logits, torch.float32, "logits"),
                             _dev(next_tokens, torch.int32, "next_tokens"), _stream(stream))
    if rc:
        raise FirstError(rc, "first_prefill")


def first_set_mask(h, mask, stream=None):
    rc = lib().first_set_mask(h, _dev(mask, torch.uint8, "mask"), mask.shape[0], _stream(stream))
    if rc:
        raise FirstError(rc, "first_set_mask")


def first_set_mask_host(h, mask, stream=None):
    """mask: HOST uint8 [B][L] (numpy or CPU tensor); no wait for the stream."""
    import numpy as np
    m = np.ascontiguousarray(np.asarray(mask), dtype=np.uint8)
    rc = lib().first_set_mask_host(h, m.ctypes.data, m.shape[0], _stream(stream))
    if rc:
        raise FirstError(rc, "first_set_mask_host")


class _PoolKV:
    """The pool's cache view (a first_kv_cache with per-layer tables that live in the pool)."""

    def __init__(self, c):
        self.c = c


class FirstPool:
    """Slab pool over caller-owned per-layer cache tensors for batches that change between steps
    (first_pool_* / first_seq_* in first.h).  k, v: lists of CUDA tensors [Hkv][rows_l][hd]."""

    def __init__(self, ctx, max_seqs, k, v):
        import numpy as np
        self._k, self._v, self._ctx = k, v, ctx
        self.L, self.B = len(k), int(max_seqs)
        rows = np.array([0 if t is None else int(t.shape[1]) for t in k], dtype=np.int64)
        first = next(t for t in k if t is not None)
        ka, va = _ptr_array(k, first.dtype, "pool.k"), _ptr_array(v, first.dtype, "pool.v")
        self.h = C.c_void_p()
        rc = lib().first_pool_create(ctx.h, self.B, rows.ctypes.data, C.cast(ka, C.POINTER(C.c_void_p)),
                                     C.cast(va, C.POINTER(C.c_void_p)), C.byref(self.h))
        if rc:
            raise FirstError(rc, "first_pool_create")
        c = KVCacheC()
        rc = lib().first_pool_kv(self.h, C.byref(c))
        if rc:
            raise FirstError(rc, "first_pool_kv")
        self.kv = _PoolKV(c)

    def close(self):
        if self.h:
            lib().first_pool_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def join(self, mask_row, capacity, src=None, src_seq=0, n_tokens=0, stream=None):
        import numpy as np
        m = np.ascontiguousarray(np.asarray(mask_row), dtype=np.uint8)
        slot = C.c_int32(-1)
        rc = lib().first_seq_join(self.h, m.ctypes.data, int(capacity), C.byref(src.c) if src is not None else None,
                                  int(src_seq), int(n_tokens), C.byref(slot), _stream(stream))
        if rc:
            raise FirstError(rc, "first_seq_join")
        return slot.value

    def leave(self, slot, stream=None):
        rc = lib().first_seq_leave(self.h, int(slot), _stream(stream))
        if rc:
            raise FirstError(rc, "first_seq_leave")

    def commit(self, stream=None):
        rc = lib().first_pool_commit(self.h, _stream(stream))
        if rc:
            raise FirstError(rc, "first_pool_commit")
        self._ctx.B = self.B

    def stats(self):
        import numpy as np
        held = np.zeros(self.L, dtype=np.int64)
        big = np.zeros(self.L, dtype=np.int64)
        live = C.c_int32(0)
        rc = lib().first_pool_stats(self.h, held.ctypes.data, big.ctypes.data, C.byref(live))
        if rc:
            raise FirstError(rc, "first_pool_stats")
        return held, big, live.value


def first_get_plan(h, B, L):
    import numpy as np
    idx = np.empty((L, B), dtype=np.int32)
    cnt = np.empty((L,), dtype=np.int32)
    slot = np.empty((L, B), dtype=np.int32)
    rc = lib().first_get_plan(h, idx.ctypes.data, cnt.ctypes.data, slot.ctypes.data)
    if rc:
        raise FirstError(rc, "first_get_plan")
    return idx, cnt, slot


def first_decode_step(h, tokens, kv: KVCache, logits=None, next_tokens=None, layer_inputs=None, stream=None):
    rc = lib().first_decode_step(h, _dev(tokens, torch.int32, "tokens"), C.byref(kv.c),
                                 _dev(logits, torch.float32, "logits"),
                                 _dev(next_tokens, torch.int32, "next_tokens"),
                                 _dev(layer_inputs, torch.float32, "layer_inputs"), _stream(stream))
    if rc:
        raise FirstError(rc, "first_decode_step")


def first_last_device_flags(h, stream=None):
    fl = C.c_uint32(0)
    rc = lib().first_last_device_flags(h, C.byref(fl), _stream(stream))
    if rc not in (0, -6):
        raise FirstError(rc, "first_last_device_flags")
    return fl.value


def first_set_option(h, name, value):
    rc = lib().first_set_option(h, name.encode(), int(value))
    if rc:
        raise FirstError(rc, "first_set_option")


def first_set_sampling(h, top_k, temperature, uniforms):
    """uniforms: CUDA float32 [B] (borrowed: refresh its contents before every step), or None with
    top_k <= 1 / temperature 0 to go back to argmax."""
    rc = lib().first_set_sampling(h, int(top_k), float(temperature), _dev(uniforms, torch.float32, "uniforms"))
    if rc:
        raise FirstError(rc, "first_set_sampling")


def first_sample_topk(logits, top_k, temperature, uniforms, tokens, stream=None):
    """logits CUDA float32 [B][vocab]; uniforms CUDA float32 [B]; tokens CUDA int32 [B] (output)."""
    B, V = logits.shape
    if uniforms.numel() != B or tokens.numel() != B:
        raise ValueError("uniforms and tokens must have one entry per row of logits")
    rc = lib().first_sample_topk(_dev(logits, torch.float32, "logits"), B, V, int(top_k), float(temperature),
                                 _dev(uniforms, torch.float32, "uniforms"), _dev(tokens, torch.int32, "tokens"),
                                 _stream(stream))
    if rc:
        raise FirstError(rc, "first_sample_topk")


def first_profile(h, enable):
    rc = lib().first_profile(h, int(bool(enable)))
    if rc:
        raise FirstError(rc, "first_profile")


def first_profile_read(h, stream=None):
    """-> {kernel class name: (total device ms, launches)}"""
    n = lib().first_kernel_class_count()
    ms = (C.c_double * n)()
    cnt = (C.c_int64 * n)()
    rc = lib().first_profile_read(h, n, ms, cnt, _stream(stream))
    if rc:
        raise FirstError(rc, "first_profile_read")
    return {lib().first_kernel_class_name(k).decode(): (ms[k], cnt[k]) for k in range(n)}


def first_step_trace(h, stream=None, max_n=2048):
    """Launches of the last step with option "stamp" on: [(class name, start_ns, end_ns)] in launch order."""
    import numpy as np
    cls = np.zeros(max_n, dtype=np.int32)
    t0 = np.zeros(max_n, dtype=np.uint64)
    t1 = np.zeros(max_n, dtype=np.uint64)
    n = C.c_int32(0)
    rc = lib().first_step_trace(h, max_n, cls.ctypes.data, t0.ctypes.data, t1.ctypes.data, C.byref(n), _stream(stream))
    if rc:
        raise FirstError(rc, "first_step_trace")
    names = [lib().first_kernel_class_name(int(k)).decode() for k in cls[:n.value]]
    return [(names[i], int(t0[i]), int(t1[i])) for i in range(n.value)]


class FirstContext:
    """Owns one library context; methods mirror the C calls."""

    def __init__(self, shape, dtype, max_batch, max_tokens_per_seq, weights):
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required; there is no CPU path")
        self.shape, self.dtype = shape, dtype
        self.h, self._keep = first_create(shape, dtype, max_batch, max_tokens_per_seq, weights)

    def close(self):
        if self.h is not None:
            first_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def prefill_route(self, layer, hidden, cu_seqlens, router_w, router_b, tau, mode, mask, scores=None, stream=None):
        first_prefill_route(self.h, layer, hidden, cu_seqlens, router_w, router_b, tau, mode, mask, scores, stream)

    def prefill(self, tokens, cu_seqlens, kv, router_w=None, router_b=None, tau=0.5, mode=0, mask=None, scores=None,
                logits=None, next_tokens=None, stream=None):
        first_prefill(self.h, tokens, cu_seqlens, kv, router_w, router_b, tau, mode, mask, scores, logits,
                      next_tokens, stream)

    def set_mask(self, mask, stream=None):
        first_set_mask(self.h, mask, stream)
        self.B = mask.shape[0]

    def set_mask_host(self, mask, stream=None):
        import numpy as np
        first_set_mask_host(self.h, mask, stream)
        self.B = np.asarray(mask).shape[0]

    def graph_count(self):
        return int(lib().first_graph_count(self.h))

    def get_plan(self):
        return first_get_plan(self.h, self.B, self.shape.n_layers)

    def decode_step(self, tokens, kv, logits=None, next_tokens=None, layer_inputs=None, stream=None):
        first_decode_step(self.h, tokens, kv, logits, next_tokens, layer_inputs, stream)

    def device_flags(self, stream=None):
        return first_last_device_flags(self.h, stream)

    def launch_count(self):
        return int(lib().first_launch_count(self.h))

    def set_option(self, name, value):
        first_set_option(self.h, name, value)

    def set_sampling(self, top_k, temperature, uniforms):
        self._uniforms = uniforms  # borrowed by the library until the next call
        first_set_sampling(self.h, top_k, temperature, uniforms)

    def selftest_wait_expiry(self, polls=1000, stream=None):
        """Runs a bounded wait that must give up; -> (what the wait returned, the abort word)."""
        r, a = C.c_int32(-1), C.c_int32(-1)
        rc = lib().first_selftest_wait_expiry(self.h, int(polls), C.byref(r), C.byref(a), _stream(stream))
        if rc:
            raise FirstError(rc, "first_selftest_wait_expiry")
        return r.value, a.value

    def step_trace(self, stream=None):
        return first_step_trace(self.h, stream)

    def profile(self, enable):
        first_profile(self.h, enable)

    def profile_read(self, stream=None):
        return first_profile_read(self.h, stream)
