"""B200 (sm_100a) implementation of the router-selective decode step of FiRST
(arXiv 2410.12513): router scoring on prefill hidden states, per-layer active-row
compaction, and decode steps that run each layer only for the sequences that keep it.

All computation happens in the CUDA library ``libfirst.so`` (C ABI in ``include/first.h``);
this package only marshals torch tensors into that ABI.  There is no CPU fallback: without
the compiled library or without a CUDA device the calls raise.
"""
from .binding import (FirstContext, FirstError, FirstPool, KVCache, first_set_mask_host, first_create, first_decode_step, first_destroy,
                      first_get_plan, first_last_device_flags, first_prefill, first_prefill_route, first_prefill_route_static, first_profile, first_profile_read, first_sample_topk, first_set_mask,
                      first_set_option, first_set_sampling, first_step_trace, lib, library_path)

__all__ = ["FirstContext", "FirstError", "FirstPool", "KVCache", "first_set_mask_host", "first_create", "first_decode_step", "first_destroy",
           "first_get_plan", "first_last_device_flags", "first_prefill", "first_prefill_route", "first_prefill_route_static", "first_profile",
           "first_profile_read", "first_sample_topk", "first_set_mask",
           "first_set_option", "first_set_sampling", "first_step_trace", "lib", "library_path"]
