"""Host-side glue between the seeded input generators and the oracle.  TEST INFRASTRUCTURE,
like the rest of this package: numpy only, used by the tests and by the benchmark's CPU-baseline
leg, never by the CUDA library or its binding."""
from __future__ import annotations

import numpy as np

import first_inputs as fi

from . import OracleKV, OracleModel, Shape


def oracle_model(shape, weights, kv_bf16=None):
    return OracleModel(Shape(**shape.asdict()), weights, kv_bf16)


def widen(a):
    """bfloat16 bit patterns (uint16) -> the float32 values they stand for; float32 passes through."""
    return fi.bf16_bits_to_f32(a) if a.dtype == np.uint16 else a


def stand_in_cache(shape, lens, caps, seed, bf16, layers=None, sink=None):
    """Oracle cache holding the generator's stand-in keys/values N(0,1) for every (layer, sequence):
    lens[b] tokens present in every layer, pos = lens.  sink(l, b, k_rows, v_rows), if given, receives
    the same rows (the tests load them into the device cache through it)."""
    B, L = len(lens), shape.n_layers
    okv = OracleKV(Shape(**shape.asdict()), caps)
    for l in (range(L) if layers is None else layers):
        for b in range(B):
            n = int(lens[b])
            kr = fi.synthetic_kv_rows(n, shape.kv_dim, seed, f"k{l}_{b}", bf16)
            vr = fi.synthetic_kv_rows(n, shape.kv_dim, seed, f"v{l}_{b}", bf16)
            ko, vo = okv.rows(l, b)
            ko[:n] = widen(kr)
            vo[:n] = widen(vr)
            if sink is not None:
                sink(l, b, kr, vr)
    okv.len[:] = np.asarray(lens, dtype=np.int32)[None, :]
    okv.pos[:] = np.asarray(lens, dtype=np.int32)
    return okv
