"""ctypes binding of the host oracle (``first_oracle.c``).  TEST INFRASTRUCTURE.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this
package; the CUDA library and its Python binding never do.  Everything here is numpy
on host memory.  The C file is compiled on first use (gcc, OpenMP) into
``libfirst_oracle.so`` beside it and rebuilt whenever the source is newer.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "first_oracle.c"
_LIB = _HERE / "libfirst_oracle.so"
_lib = None


def _cpu_has(flag: str) -> bool:
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.startswith("flags"):
                    return flag in line.split()
    except OSError:
        pass
    return False


def build(force: bool = False) -> Path:
    """Compile the oracle with gcc; returns the shared library path."""
    stamp = _HERE / ".oracle_build_host"
    host = f"{os.uname().nodename}:{'avx2' if _cpu_has('avx2') else 'base'}"
    fresh = (_LIB.exists() and _LIB.stat().st_mtime >= _SRC.stat().st_mtime
             and stamp.exists() and stamp.read_text() == host)
    if fresh and not force:
        return _LIB
    flags = ["-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-fno-fast-math", "-ffp-contract=off"]
    if _cpu_has("avx2") and _cpu_has("fma"):
        flags += ["-mavx2"]
    tmp = _LIB.with_suffix(f".tmp{os.getpid()}.so")
    subprocess.run(["gcc", *flags, str(_SRC), "-o", str(tmp), "-lm"], check=True)
    os.replace(tmp, _LIB)
    stamp.write_text(host)
    return _LIB


class _Model(C.Structure):
    _fields_ = [(n, C.c_int32) for n in
                ("n_layers", "d_model", "n_q_heads", "n_kv_heads", "head_dim", "ffn_dim", "vocab",
                 "weight_dtype")] + [("rope_base", C.c_double), ("rms_eps", C.c_double), ("kv_dtype", C.c_int32)]


class _Weights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("lm_head", C.c_void_p), ("final_norm", C.c_void_p)] + \
               [(n, C.POINTER(C.c_void_p)) for n in
                ("attn_norm", "ffn_norm", "wq", "wk", "wv", "wo", "wg", "wu", "wd")]


class _KV(C.Structure):
    _fields_ = [("k", C.POINTER(C.c_void_p)), ("v", C.POINTER(C.c_void_p)),
                ("slab_off", C.c_void_p), ("slab_cap", C.c_void_p), ("len", C.c_void_p), ("pos", C.c_void_p)]


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(str(build()))
        _lib.fo_route.restype = C.c_int
        _lib.fo_decode_step.restype = C.c_int
        _lib.fo_forward_full.restype = C.c_int
        _lib.fo_plan.restype = C.c_int
        _lib.fo_argmax.restype = C.c_int32
        _lib.fo_sample_topk.restype = C.c_int32
    return _lib


def _ptr(a):
    return None if a is None else C.c_void_p(a.ctypes.data)


def _ptr_array(arrs):
    return (C.c_void_p * len(arrs))(*[a.ctypes.data for a in arrs])


@dataclass
class Shape:
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    ffn_dim: int
    vocab: int
    rope_base: float = 10000.0
    rms_eps: float = 1e-5


def _w_host(a):
    """Accept float32 arrays, or bfloat16 values as uint16 bit patterns."""
    a = np.ascontiguousarray(a)
    if a.dtype == np.float32:
        return a, 0
    if a.dtype == np.uint16:
        return a, 1
    raise TypeError(f"weights must be float32 or uint16 (bfloat16 bits), got {a.dtype}")


class OracleModel:
    """Holds host weights (kept alive) and the C descriptors.

    ``weights`` is a dict with keys embed, lm_head, final_norm and per-layer lists
    attn_norm, ffn_norm, wq, wk, wv, wo, wg, wu, wd (PyTorch Linear layout [out][in]).
    Matrices are float32 or uint16 (bfloat16 bits) -- all the same kind; norm gains
    are float32.
    """

    def __init__(self, shape: Shape, weights: dict, kv_bf16=None):
        """kv_bf16: cache storage format; default = bfloat16 iff the weights are bfloat16."""
        self.shape = shape
        L = shape.n_layers
        keep = {}
        dts = set()
        for k in ("embed", "lm_head"):
            keep[k], dt = _w_host(weights[k])
            dts.add(dt)
        for k in ("wq", "wk", "wv", "wo", "wg", "wu", "wd"):
            keep[k] = []
            for a in weights[k]:
                a, dt = _w_host(a)
                keep[k].append(a)
                dts.add(dt)
            assert len(keep[k]) == L
        assert len(dts) == 1, "all weight matrices must share one dtype"
        self.weight_dtype = dts.pop()
        keep["final_norm"] = np.ascontiguousarray(weights["final_norm"], dtype=np.float32)
        for k in ("attn_norm", "ffn_norm"):
            keep[k] = [np.ascontiguousarray(a, dtype=np.float32) for a in weights[k]]
        s = shape
        D, qd, kvd = s.d_model, s.n_q_heads * s.head_dim, s.n_kv_heads * s.head_dim
        assert keep["embed"].shape == (s.vocab, D) and keep["lm_head"].shape == (s.vocab, D)
        for l in range(L):
            assert keep["wq"][l].shape == (qd, D) and keep["wk"][l].shape == (kvd, D)
            assert keep["wv"][l].shape == (kvd, D) and keep["wo"][l].shape == (D, qd)
            assert keep["wg"][l].shape == (s.ffn_dim, D) and keep["wu"][l].shape == (s.ffn_dim, D)
            assert keep["wd"][l].shape == (D, s.ffn_dim)
        self._keep = keep
        self._arrs = {k: _ptr_array(keep[k]) for k in
                      ("attn_norm", "ffn_norm", "wq", "wk", "wv", "wo", "wg", "wu", "wd")}
        self.kv_dtype = self.weight_dtype if kv_bf16 is None else int(bool(kv_bf16))
        self.c_model = _Model(s.n_layers, s.d_model, s.n_q_heads, s.n_kv_heads, s.head_dim, s.ffn_dim,
                              s.vocab, self.weight_dtype, float(s.rope_base), float(s.rms_eps), self.kv_dtype)
        self.c_weights = _Weights(keep["embed"].ctypes.data, keep["lm_head"].ctypes.data,
                                  keep["final_norm"].ctypes.data,
                                  *[C.cast(self._arrs[k], C.POINTER(C.c_void_p)) for k in
                                    ("attn_norm", "ffn_norm", "wq", "wk", "wv", "wo", "wg", "wu", "wd")])


class OracleKV:
    """Float32 host cache: per layer ``[cap_total][Hkv*hd]``, sequence b at rows
    ``slab_off[b] .. slab_off[b]+slab_cap[b]``."""

    def __init__(self, shape: Shape, caps):
        caps = np.asarray(caps, dtype=np.int32)
        self.B = len(caps)
        self.L = shape.n_layers
        self.kvd = shape.n_kv_heads * shape.head_dim
        self.slab_cap = caps
        self.slab_off = np.concatenate([[0], np.cumsum(caps[:-1], dtype=np.int64)]).astype(np.int64)
        tot = int(caps.sum())
        self.k = [np.zeros((tot, self.kvd), dtype=np.float32) for _ in range(self.L)]
        self.v = [np.zeros((tot, self.kvd), dtype=np.float32) for _ in range(self.L)]
        self.len = np.zeros((self.L, self.B), dtype=np.int32)
        self.pos = np.zeros((self.B,), dtype=np.int32)
        self._ka, self._va = _ptr_array(self.k), _ptr_array(self.v)
        self.c = _KV(C.cast(self._ka, C.POINTER(C.c_void_p)), C.cast(self._va, C.POINTER(C.c_void_p)),
                     self.slab_off.ctypes.data, self.slab_cap.ctypes.data, self.len.ctypes.data,
                     self.pos.ctypes.data)

    def rows(self, l, b):
        o = int(self.slab_off[b])
        return self.k[l][o:o + int(self.slab_cap[b])], self.v[l][o:o + int(self.slab_cap[b])]


def _check(rc, what):
    if rc != 0:
        raise RuntimeError(f"oracle {what} failed with status {rc}")


def route(hidden, w, bias=None, tau=0.5, mode=0):
    """One sequence, one layer: returns (rho, keep)."""
    hidden = np.ascontiguousarray(hidden, dtype=np.float32)
    w = np.ascontiguousarray(w, dtype=np.float32)
    n, D = hidden.shape
    assert w.shape == (D,)
    b = None if bias is None else np.asarray([bias], dtype=np.float32)
    rho, keep = C.c_double(0), C.c_uint8(0)
    _check(lib().fo_route(_ptr(hidden), C.c_int32(n), C.c_int32(D), _ptr(w), _ptr(b), C.c_double(tau),
                          C.c_int32(mode), C.byref(rho), C.byref(keep)), "route")
    return rho.value, int(keep.value)


def route_batch(hidden, cu_seqlens, w, bias=None, tau=0.5, mode=0):
    """Ragged batch for one layer: hidden [sum_n][D], cu_seqlens [B+1] -> (rho[B], keep[B])."""
    B = len(cu_seqlens) - 1
    rho = np.zeros(B, dtype=np.float64)
    keep = np.zeros(B, dtype=np.uint8)
    for b in range(B):
        rho[b], keep[b] = route(hidden[cu_seqlens[b]:cu_seqlens[b + 1]], w, bias, tau, mode)
    return rho, keep


def decode_step(model: OracleModel, tokens, mask, kv: OracleKV, want_logits=True, want_layer_inputs=False):
    tokens = np.ascontiguousarray(tokens, dtype=np.int32)
    mask = np.ascontiguousarray(mask, dtype=np.uint8)
    B, s = len(tokens), model.shape
    assert mask.shape == (B, s.n_layers) and kv.B == B
    logits = np.empty((B, s.vocab), dtype=np.float32) if want_logits else None
    li = np.empty((s.n_layers, B, s.d_model), dtype=np.float32) if want_layer_inputs else None
    _check(lib().fo_decode_step(C.byref(model.c_model), C.byref(model.c_weights), C.c_int32(B), _ptr(tokens),
                                _ptr(mask), C.byref(kv.c), _ptr(logits), _ptr(li)), "decode_step")
    return (logits, li) if want_layer_inputs else logits


def forward_full(model: OracleModel, tokens, n_prompt=None, keep=None, want_kv=False, want_router_in=False,
                 logits_from=None):
    """Cache-free forward of one sequence; see ``fo_forward_full``.

    Returns dict(logits=[n-logits_from][V], k=[L][n][kvd], v=..., router_in=[L][n][D])."""
    tokens = np.ascontiguousarray(tokens, dtype=np.int32)
    n, s = len(tokens), model.shape
    n_prompt = n if n_prompt is None else int(n_prompt)
    logits_from = n - 1 if logits_from is None else int(logits_from)
    kvd = s.n_kv_heads * s.head_dim
    out = {}
    ka = va = None
    if want_kv:
        out["k"] = [np.zeros((n, kvd), dtype=np.float32) for _ in range(s.n_layers)]
        out["v"] = [np.zeros((n, kvd), dtype=np.float32) for _ in range(s.n_layers)]
        ka, va = _ptr_array(out["k"]), _ptr_array(out["v"])
    ri = np.empty((s.n_layers, n, s.d_model), dtype=np.float32) if want_router_in else None
    keep_a = None if keep is None else np.ascontiguousarray(keep, dtype=np.uint8)
    logits = np.empty((n - logits_from, s.vocab), dtype=np.float32)
    _check(lib().fo_forward_full(C.byref(model.c_model), C.byref(model.c_weights), C.c_int32(n), _ptr(tokens),
                                 C.c_int32(n_prompt), _ptr(keep_a), ka, va, _ptr(ri), C.c_int32(logits_from),
                                 _ptr(logits)), "forward_full")
    out["logits"] = logits
    if want_router_in:
        out["router_in"] = ri
    return out


def plan(mask):
    mask = np.ascontiguousarray(mask, dtype=np.uint8)
    B, L = mask.shape
    idx = np.empty((L, B), dtype=np.int32)
    cnt = np.empty((L,), dtype=np.int32)
    slot = np.empty((L, B), dtype=np.int32)
    _check(lib().fo_plan(_ptr(mask), C.c_int32(B), C.c_int32(L), _ptr(idx), _ptr(cnt), _ptr(slot)), "plan")
    return idx, cnt, slot


def argmax(logits):
    logits = np.ascontiguousarray(logits, dtype=np.float32)
    return np.array([lib().fo_argmax(_ptr(row), C.c_int32(row.shape[0])) for row in logits], dtype=np.int32)


def sample_topk(logits_row, k, temperature, u):
    """One row: -> (token, candidates[k] in order, probabilities[k])."""
    row = np.ascontiguousarray(logits_row, dtype=np.float32)
    cand = np.zeros(k, dtype=np.int32)
    prob = np.zeros(k, dtype=np.float64)
    t = lib().fo_sample_topk(_ptr(row), C.c_int32(row.shape[0]), C.c_int32(k), C.c_double(temperature),
                             C.c_double(u), _ptr(cand), _ptr(prob))
    _check(min(t, 0), "sample_topk")
    return int(t), cand, prob


def prefill(model: OracleModel, kv: OracleKV, b: int, tokens, want_router_in=True):
    """Prefill sequence b of the cache from its prompt (no skipping), returning the
    last position's logits and the per-layer router inputs."""
    r = forward_full(model, tokens, want_kv=True, want_router_in=want_router_in)
    n = len(tokens)
    for l in range(model.shape.n_layers):
        kr, vr = kv.rows(l, b)
        kr[:n] = r["k"][l]
        vr[:n] = r["v"][l]
        kv.len[l, b] = n
    kv.pos[b] = n
    return r
