"""Test-side glue: the same seeded inputs laid out for the host oracle (numpy) and for the
CUDA library (torch), router-weight calibration against the oracle, and comparisons."""
from __future__ import annotations

import numpy as np

import first_inputs as fi
import oracle


# ------------------------------------------------------------------ oracle side
from oracle.workload import oracle_model, stand_in_cache, widen  # noqa: E402,F401


# ------------------------------------------------------------------ CUDA side
def to_dev(a, bf16):
    import torch
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
    t = torch.from_numpy(np.ascontiguousarray(a)).cuda()
    return t


def gpu_weights(w, layers=None):
    """Generator dict -> the layout first_create takes (q,k,v rows concatenated; gate,up rows
    concatenated).  Layers not materialised stay None."""
    import torch
    L = len(w["wq"])
    bf16 = w["embed"].dtype == np.uint16
    out = {"embed": to_dev(w["embed"], bf16), "lm_head": to_dev(w["lm_head"], bf16),
           "final_norm": to_dev(w["final_norm"], False)}
    for k in ("attn_norm", "wqkv", "wo", "ffn_norm", "w_gate_up", "w_down"):
        out[k] = [None] * L
    for l in range(L):
        if w["wq"][l] is None:
            continue
        out["attn_norm"][l] = to_dev(w["attn_norm"][l], False)
        out["ffn_norm"][l] = to_dev(w["ffn_norm"][l], False)
        out["wqkv"][l] = torch.cat([to_dev(w[k][l], bf16) for k in ("wq", "wk", "wv")], 0).contiguous()
        out["wo"][l] = to_dev(w["wo"][l], bf16)
        out["w_gate_up"][l] = torch.cat([to_dev(w[k][l], bf16) for k in ("wg", "wu")], 0).contiguous()
        out["w_down"][l] = to_dev(w["wd"][l], bf16)
    return out


class GpuKV:
    """Caller-owned cache tensors in the library's layout, plus the binding struct."""

    def __init__(self, shape, caps, bf16, layers=None):
        import torch
        from paper_2410_12513_b200 import KVCache
        caps = np.asarray(caps, dtype=np.int32)
        self.shape, self.B, self.L = shape, len(caps), shape.n_layers
        self.caps = caps
        self.off = np.concatenate([[0], np.cumsum(caps[:-1], dtype=np.int64)]).astype(np.int64)
        tot = int(caps.sum())
        dt = torch.bfloat16 if bf16 else torch.float32
        layers = range(self.L) if layers is None else layers
        self.k = [None] * self.L
        self.v = [None] * self.L
        for l in layers:
            self.k[l] = torch.zeros((shape.n_kv_heads, tot, shape.head_dim), dtype=dt, device="cuda")
            self.v[l] = torch.zeros((shape.n_kv_heads, tot, shape.head_dim), dtype=dt, device="cuda")
        self.slab_off = torch.from_numpy(self.off).cuda()
        self.slab_cap = torch.from_numpy(caps).cuda()
        self.len = torch.zeros((self.L, self.B), dtype=torch.int32, device="cuda")
        self.pos = torch.zeros((self.B,), dtype=torch.int32, device="cuda")
        self.c = KVCache(self.k, self.v, self.slab_off, self.slab_cap, self.len, self.pos)

    def load_rows(self, l, b, k_rows, v_rows):
        """k_rows/v_rows: numpy [n][Hkv*hd] token-major (float32 or bf16 bits)."""
        import torch
        n = k_rows.shape[0]
        s = self.shape
        o = int(self.off[b])
        for dst, src in ((self.k[l], k_rows), (self.v[l], v_rows)):
            t = to_dev(src, src.dtype == np.uint16).to(dst.dtype)
            dst[:, o:o + n, :] = t.view(n, s.n_kv_heads, s.head_dim).permute(1, 0, 2)

    def set_len(self, lens, pos):
        import torch
        self.len.copy_(torch.from_numpy(np.ascontiguousarray(lens, dtype=np.int32)))
        self.pos.copy_(torch.from_numpy(np.ascontiguousarray(pos, dtype=np.int32)))

    def rows_host(self, l, b):
        """-> (k, v) numpy float32 [cap][Hkv*hd] token-major."""
        o, cp = int(self.off[b]), int(self.caps[b])
        f = lambda t: t[:, o:o + cp, :].permute(1, 0, 2).reshape(cp, -1).float().cpu().numpy()
        return f(self.k[l]), f(self.v[l])


def synthetic_caches(shape, lens, caps, seed, bf16, layers=None, with_gpu=True):
    """Stand-in prefilled caches N(0,1) for every (layer, sequence): identical values on both
    sides.  lens: [B] tokens present in every layer; pos = lens."""
    gkv = GpuKV(shape, caps, bf16, layers) if with_gpu else None
    okv = stand_in_cache(shape, lens, caps, seed, bf16, layers, sink=gkv.load_rows if gkv is not None else None)
    if gkv is not None:
        gkv.set_len(okv.len, okv.pos)
    return okv, gkv


# ------------------------------------------------------------------ router calibration
def calibrate_router(hiddens, target_keep, mode, seed, tau=0.5, margin=1e-3, tight=False, bias=None):
    """Router weights w[D] (no bias) that realise `target_keep` on the given per-sequence hidden
    states with every oracle score at least `margin` away from tau.  Least-norm solve on the
    pooled means (B <= D), scaled up until the oracle's own scores clear the margin.
    tight=True: scaled so that the score nearest to tau lies in [margin, 2*margin] -- the stated
    margin itself, not a comfortable multiple of it.  bias: a fixed router bias (for tau != 0.5 the
    bias logit(tau) centres the scores on tau, which a bias-free router cannot do near the margin)."""
    B = len(hiddens)
    pooled = np.stack([h.astype(np.float64).mean(0) for h in hiddens])  # [B][D]
    t = np.where(np.asarray(target_keep) > 0, 1.0, -1.0)
    pinv = np.linalg.pinv(pooled)

    # tight: the sequences' distances from tau are spread over [0.7, 1.3] x the middle one
    spread = np.random.default_rng(seed).permutation(np.linspace(0.7, 1.3, B)) if tight else np.ones(B)

    def scores(c):
        w = (pinv @ (c * t * spread)).astype(np.float32)
        rho = np.array([oracle.route(h, w, bias, tau, mode)[0] for h in hiddens])
        return w, rho

    if tight:
        c = 6.0 * margin  # sigmoid'(0) = 1/4: |rho - 1/2| ~ c/4 = 1.5 margin for the middle sequence
        for _ in range(40):
            w, rho = scores(c)
            gap = np.abs(rho - tau).min()
            if ((rho >= tau) == (t > 0)).all() and margin <= gap <= 2.0 * margin:
                return w, rho
            c *= (1.06 * margin / gap) if gap > 0 else 2.0  # aim the nearest score just outside the margin
        raise AssertionError("tight router calibration failed")
    c = 0.25
    for _ in range(12):
        w, rho = scores(c)
        keep = rho >= tau
        if (keep == (t > 0)).all() and np.abs(rho - tau).min() >= margin:
            return w, rho
        c *= 2.0
    raise AssertionError("router calibration failed")


# ------------------------------------------------------------------ comparisons
def logits_check(got, ref, rel=2e-2):
    """max-abs error relative to the row's logit range, and argmax agreement per row."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    rng = ref.max(-1) - ref.min(-1)
    err = np.abs(got - ref).max(-1) / rng
    agree = got.argmax(-1) == ref.argmax(-1)
    return err, agree
