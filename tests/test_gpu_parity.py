"""CUDA library vs host oracle, element by element, through the C ABI (B200 only)."""
import numpy as np
import pytest

import first_inputs as fi
import oracle
from harness import (GpuKV, calibrate_router, gpu_weights, logits_check, oracle_model, synthetic_caches, to_dev,
                     widen)

pytestmark = pytest.mark.gpu

F32, BF16 = 0, 1


def _ctx(shape, bf16, max_batch, max_tokens, w):
    from paper_2410_12513_b200 import FirstContext
    return FirstContext(shape, BF16 if bf16 else F32, max_batch, max_tokens, gpu_weights(w))


# ------------------------------------------------------------------ router (a0)
@pytest.mark.parametrize("hidden_bf16", [False, True])
@pytest.mark.parametrize("mode", [0, 1])
def test_router_masks_bit_exact(hidden_bf16, mode):
    import torch
    shape = fi.TINY
    D, L = 512, 5
    shape = fi.ModelShape(L, D, 4, 4, 128, 1024, 64)
    w = fi.make_weights(shape, 1, False)
    ctx = _ctx(shape, False, 16, 1200, w)
    lens = [1, 7, 300, 33, 1111, 64, 2, 257]
    B = len(lens)
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    mask = torch.full((B, L), 9, dtype=torch.uint8, device="cuda")
    scores = torch.zeros((B, L), dtype=torch.float32, device="cuda")
    want_mask = np.zeros((B, L), np.uint8)
    want_rho = np.zeros((B, L))
    for l in range(L):
        hid = fi.normal((int(cu[-1]), D), 1.0, 7, f"hid{l}", hidden_bf16)
        hid_f = widen(hid)
        hs = [hid_f[cu[b]:cu[b + 1]] for b in range(B)]
        target = fi.mask_bernoulli(B, 3, 0.5, 100 + l)[:, 1]
        rw, _ = calibrate_router(hs, target, mode, l)
        bias = None if l % 2 == 0 else 0.0
        want_rho[:, l], want_mask[:, l] = oracle.route_batch(hid_f, cu, rw, bias, 0.5, mode)
        assert np.abs(want_rho[:, l] - 0.5).min() >= 1e-3
        ctx.prefill_route(l, to_dev(hid, hidden_bf16), torch.from_numpy(cu).cuda(), to_dev(rw, False),
                          None if bias is None else torch.zeros(1, device="cuda"), 0.5, mode, mask, scores)
    assert ctx.device_flags() == 0
    assert np.array_equal(mask.cpu().numpy(), want_mask)
    assert np.abs(scores.cpu().numpy() - want_rho).max() < 1e-5


@pytest.mark.parametrize("hidden_bf16", [False, True])
@pytest.mark.parametrize("mode", [0, 1])
def test_router_masks_bit_exact_at_the_stated_margin(hidden_bf16, mode):
    """Scores as close to tau as the stated margin allows: the router weights are scaled so that the
    nearest oracle score sits between 1e-3 and 2e-3 from tau (the others up to 2.2e-3).  Identical
    hidden states on both sides; both router entry points; sequence lengths 1 .. 1111."""
    import torch
    from paper_2410_12513_b200 import first_prefill_route_static
    D, L = 512, 4
    shape = fi.ModelShape(L, D, 4, 4, 128, 1024, 64)
    ctx = _ctx(shape, False, 16, 1200, fi.make_weights(shape, 1, False))
    lens = [1, 7, 300, 33, 1111, 64, 2, 257, 1024, 5]
    B = len(lens)
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    mask = torch.full((B, L), 9, dtype=torch.uint8, device="cuda")
    mask_s = mask.clone()
    scores = torch.zeros((B, L), dtype=torch.float32, device="cuda")
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    want_mask = np.zeros((B, L), np.uint8)
    want_rho = np.zeros((B, L))
    for l in range(L):
        hid = fi.normal((int(cu[-1]), D), 1.0, 17, f"hid{l}", hidden_bf16)
        hid_f = widen(hid)
        hs = [hid_f[cu[b]:cu[b + 1]] for b in range(B)]
        target = fi.mask_bernoulli(B, 3, 0.5, 200 + l)[:, 1]
        tau = 0.5 if l < 3 else 0.4
        bias = None if l < 3 else float(np.log(tau / (1.0 - tau)))  # centres the scores on tau
        rw, _ = calibrate_router(hs, target, mode, l, tau=tau, tight=True, bias=bias)
        want_rho[:, l], want_mask[:, l] = oracle.route_batch(hid_f, cu, rw, bias, tau, mode)
        gap = np.abs(want_rho[:, l] - tau)
        assert 1e-3 <= gap.min() <= 2e-3 and gap.max() <= 2.5e-3, gap
        assert np.array_equal(want_mask[:, l], target)
        b_t = None if bias is None else torch.tensor([bias], dtype=torch.float32, device="cuda")
        args = (to_dev(hid, hidden_bf16), torch.from_numpy(cu).cuda(), to_dev(rw, False), b_t, tau, mode)
        ctx.prefill_route(l, *args, mask, scores)
        first_prefill_route_static(l, L, *args, mask_s, None, flags)
    assert ctx.device_flags() == 0 and int(flags.item()) == 0
    assert np.array_equal(mask.cpu().numpy(), want_mask)
    assert np.array_equal(mask_s.cpu().numpy(), want_mask)
    # the device scores are a float32 rounding of the float64 mean: far inside the margin
    assert np.abs(scores.cpu().numpy() - want_rho).max() < 2e-6


def test_router_sequence_table_is_checked_against_total_tokens():
    """A cu_seqlens whose entries leave [0, total_tokens] or run backwards is never followed: the
    sequence is flagged, nothing of it is read, its mask byte and score stay as they were."""
    import torch
    from paper_2410_12513_b200 import first_prefill_route_static
    shape = fi.ModelShape(2, 64, 2, 2, 32, 64, 32)
    ctx = _ctx(shape, False, 4, 64, fi.make_weights(shape, 1, False))
    hid_h = fi.normal((10, 64), 1.0, 1, "h")
    hid = to_dev(hid_h, False)
    rw_h = fi.normal((64,), 0.1, 1, "rw")
    rw = to_dev(rw_h, False)
    _, want = oracle.route_batch(hid_h, np.array([0, 4, 10]), rw_h, None, 0.5, 0)
    for bad in ([0, 4, 11], [0, 12, 10], [-1, 4, 10], [0, 4, 2**31 - 1]):
        cu = torch.tensor(bad, dtype=torch.int32, device="cuda")
        for static in (False, True):
            mask = torch.full((2, 2), 7, dtype=torch.uint8, device="cuda")
            sc = torch.full((2, 2), -3.0, dtype=torch.float32, device="cuda")
            if static:
                fl = torch.zeros(1, dtype=torch.int32, device="cuda")
                first_prefill_route_static(1, 2, hid, cu, rw, None, 0.5, 0, mask, sc, fl)
                torch.cuda.synchronize()
                got_flags = int(fl.item())
            else:
                ctx.prefill_route(1, hid, cu, rw, None, 0.5, 0, mask, sc)
                got_flags = ctx.device_flags()
            assert got_flags == 32, (bad, static, got_flags)
            m, s_ = mask.cpu().numpy(), sc.cpu().numpy()
            good = [b for b in range(2) if 0 <= bad[b] <= bad[b + 1] <= 10]
            for b in range(2):
                if b in good:
                    assert m[b, 1] in (0, 1) and s_[b, 1] != -3.0
                    if bad[b:b + 2] == [0, 4]:
                        assert m[b, 1] == want[0]
                else:
                    assert m[b, 1] == 7 and s_[b, 1] == -3.0
            assert (m[:, 0] == 7).all()


def test_router_tie_keeps_and_empty_sequence_flag():
    import torch
    shape = fi.ModelShape(2, 64, 2, 2, 32, 64, 32)
    ctx = _ctx(shape, False, 4, 64, fi.make_weights(shape, 1, False))
    hid = to_dev(fi.normal((10, 64), 1.0, 1, "h"), False)
    mask = torch.full((2, 2), 7, dtype=torch.uint8, device="cuda")
    cu = torch.tensor([0, 4, 10], dtype=torch.int32, device="cuda")
    ctx.prefill_route(1, hid, cu, torch.zeros(64, device="cuda"), None, 0.5, 0, mask)
    assert ctx.device_flags() == 0
    assert mask.cpu().numpy().tolist() == [[7, 1], [7, 1]]  # rho == 0.5 exactly: kept; column 0 untouched
    cu = torch.tensor([0, 0, 10], dtype=torch.int32, device="cuda")
    ctx.prefill_route(0, hid, cu, torch.zeros(64, device="cuda"), None, 0.5, 0, mask)
    assert ctx.device_flags() == 16


# ------------------------------------------------------------------ plan (a1)
@pytest.mark.parametrize("B", [1, 2, 3, 31, 32, 33, 255, 256])
def test_plan_bit_exact(B):
    import torch
    shape = fi.ModelShape(6, 64, 2, 2, 32, 64, 32)
    ctx = _ctx(shape, False, 256, 8, fi.make_weights(shape, 1, False))
    mask = fi.mask_bernoulli(B, 6, 0.6, B)
    mask[:, 2] = 0
    mask[:, 3] = 1
    ctx.set_mask(torch.from_numpy(mask).cuda())
    idx, cnt, slot = ctx.get_plan()
    oi, oc, os_ = oracle.plan(mask)
    assert np.array_equal(idx, oi) and np.array_equal(cnt, oc) and np.array_equal(slot, os_)


def test_bad_mask_byte_is_rejected():
    import torch
    from paper_2410_12513_b200 import FirstError
    shape = fi.ModelShape(2, 64, 2, 2, 32, 64, 32)
    ctx = _ctx(shape, False, 4, 8, fi.make_weights(shape, 1, False))
    mask = torch.ones((3, 2), dtype=torch.uint8, device="cuda")
    mask[1, 1] = 2
    with pytest.raises(FirstError) as e:
        ctx.set_mask(mask)
    assert e.value.status == -6
    ctx.device_flags()


# ------------------------------------------------------------------ decode on stand-in caches
def _run_decode_case(shape, bf16, lens, mask, steps, seed, rel_tol, options=None, check_rows=None):
    """Both sides start from identical stand-in caches and run `steps` teacher-forced steps."""
    import torch
    B, L = len(lens), shape.n_layers
    w = fi.make_weights(shape, seed, bf16)
    om = oracle_model(shape, w)
    caps = [int(n) + steps for n in lens]
    caps[0] += 3  # capacities need not be tight
    okv, gkv = synthetic_caches(shape, lens, caps, seed, bf16)
    ctx = _ctx(shape, bf16, B, max(caps), w)
    for k, v in (options or {}).items():
        ctx.set_option(k, v)
    before = {(l, b): gkv.rows_host(l, b) for l in range(L) for b in range(B) if not mask[b, l]}
    ctx.set_mask(torch.from_numpy(mask).cuda())
    toks = fi.tokens(shape, B, seed, "first")
    logits = torch.empty((B, shape.vocab), dtype=torch.float32, device="cuda")
    nxt = torch.empty((B,), dtype=torch.int32, device="cuda")
    errs, agrees = [], []
    for t in range(steps):
        ref = oracle.decode_step(om, toks, mask, okv)
        ctx.decode_step(torch.from_numpy(toks).cuda(), gkv.c, logits, nxt)
        got = logits.cpu().numpy()
        assert ctx.device_flags() == 0
        err, agree = logits_check(got, ref)
        errs.append(err)
        agrees.append(agree)
        assert np.array_equal(nxt.cpu().numpy(), oracle.argmax(got))  # the oracle's greedy rule on the same logits
        assert np.array_equal(nxt.cpu().numpy(), got.argmax(-1).astype(np.int32))
        toks = oracle.argmax(ref)  # teacher forcing with the oracle's tokens
    errs, agrees = np.stack(errs), np.stack(agrees)
    assert errs.max() <= rel_tol, errs.max()
    # bookkeeping: len advanced only where kept, pos for everyone; skipped slabs untouched
    assert np.array_equal(gkv.len.cpu().numpy(), okv.len)
    assert np.array_equal(gkv.pos.cpu().numpy(), okv.pos)
    for (l, b), (k0, v0) in before.items():
        k1, v1 = gkv.rows_host(l, b)
        assert np.array_equal(k0, k1) and np.array_equal(v0, v1)
    # appended keys/values agree with the oracle's (bf16 cache: to rounding)
    tol = 2e-2 if bf16 else 1e-4
    for l in range(L):
        for b in range(B):
            if mask[b, l]:
                k1, v1 = gkv.rows_host(l, b)
                ko, vo = okv.rows(l, b)
                n = int(lens[b])
                assert np.abs(k1[n:n + steps] - ko[n:n + steps]).max() <= tol * max(1.0, np.abs(ko[n:n + steps]).max())
                assert np.abs(v1[n:n + steps] - vo[n:n + steps]).max() <= tol * max(1.0, np.abs(vo[n:n + steps]).max())
    return errs, agrees


@pytest.mark.parametrize("B", [1, 2, 3, 9, 33])
def test_decode_f32_tiny_ragged(B):
    shape = fi.TINY
    lens = fi.prompt_lengths(B, 1, 70, B)
    mask = fi.mask_bernoulli(B, shape.n_layers, 0.6, B + 50)
    if B >= 3:
        mask[:, 1] = 0   # a layer nobody keeps: no launch
        mask[2, :] = 0   # a sequence that skips everything
    errs, agrees = _run_decode_case(shape, False, lens, mask, 3, 5, 1e-4)
    assert agrees.all()


@pytest.mark.parametrize("shape", [fi.TINY_GQA, fi.ModelShape(2, 256, 8, 2, 128, 512, 1000, 500000.0),
                                   fi.ModelShape(2, 384, 6, 2, 64, 512, 1000, 500000.0),    # 3 query heads per KV head
                                   fi.ModelShape(2, 384, 3, 1, 128, 512, 1000, 500000.0)])  # (the Llama-3.2-3B grouping)
def test_decode_bf16_gqa_ragged(shape):
    B = 7
    lens = fi.prompt_lengths(B, 1, 300, 3)
    mask = fi.mask_bernoulli(B, shape.n_layers, 0.7, 4)
    errs, agrees = _run_decode_case(shape, True, lens, mask, 3, 6, 2e-2)
    assert agrees.mean() >= 0.9  # tiny vocab-independent sanity; the aggregate bar is checked at scale


@pytest.mark.parametrize("B", [70, 200, 300])
def test_decode_bf16_many_rows(B):
    """Many active rows: wide activation tiles (one projection CTA per SM), and with 300 rows more than one
    256-row projection launch per matrix.  Once with the default kernels (CTA pairs from 96 rows on), once with
    the single-CTA kernel at every size."""
    shape = fi.ModelShape(2, 256, 8, 2, 128, 512, 1000, 500000.0)
    lens = fi.prompt_lengths(B, 1, 90, 13)
    mask = fi.mask_bernoulli(B, shape.n_layers, 0.85, 14)
    errs, agrees = _run_decode_case(shape, True, lens, mask, 2, 16, 2e-2)
    assert agrees.mean() >= 0.98
    errs, agrees = _run_decode_case(shape, True, lens, mask, 2, 16, 2e-2, options={"tc2_min_rows": 0})
    assert agrees.mean() >= 0.98


@pytest.mark.parametrize("B", [100, 40, 130, 200, 256, 300])
def test_decode_bf16_cta_pair_projections(B):
    """The CTA-pair projection kernel (two CTAs per tile pair, activation rows split between them), forced from 33
    rows on: 33..64 rows (one 16-row group per CTA and a ragged second), 100, 130, 200, 256 rows, and 300 rows
    (a 256-row launch plus a 44-row launch per matrix)."""
    shape = fi.ModelShape(2, 512, 8, 2, 128, 1024, 1000, 500000.0)
    lens = fi.prompt_lengths(B, 1, 90, 13)
    mask = fi.mask_bernoulli(B, shape.n_layers, 0.85, 14)
    errs, agrees = _run_decode_case(shape, True, lens, mask, 2, 16, 2e-2, options={"tc2_min_rows": 33})
    assert agrees.mean() >= 0.98


@pytest.mark.parametrize("hq,hkv,hd", [(8, 2, 128), (8, 2, 64), (6, 2, 128), (8, 1, 64), (4, 4, 128)])
def test_decode_bf16_split_rows_merged_through_a_cluster(hq, hkv, hd):
    """Rows long enough to be split into several attention chunks, with the chunks of a (row, kv head) merged through
    the shared memory of a thread-block cluster (option attn_cluster) and, for comparison, through global memory:
    1 to 5 chunks per row (chunks of 64 tokens), rows of one token, a full slab among them."""
    shape = fi.ModelShape(2, hq * hd // 2 if hq * hd // 2 >= 256 else 256, hq, hkv, hd, 512, 1000, 500000.0)
    lens = np.array([300, 1, 64, 65, 129, 200, 17, 256], np.int32)
    mask = fi.mask_bernoulli(len(lens), shape.n_layers, 0.8, 4)
    for opts in ({"attn_chunk": 64, "attn_cluster": 1}, {"attn_chunk": 64, "attn_cluster": 0},
                 {"attn_chunk": 128, "attn_cluster": 1}):
        errs, agrees = _run_decode_case(shape, True, lens, mask, 3, 6, 2e-2, options=opts)
        assert agrees.mean() >= 0.9


@pytest.mark.parametrize("ffn", [320, 352, 448])
def test_decode_bf16_many_rows_with_ragged_feature_counts(ffn):
    """120-150 active rows (CTA-pair projections) on widths that do not fill the last weight tile: FFN widths that
    are a multiple of 64 but not of 256 (fused SwiGLU falls back to the single-CTA kernel), or not even of 64 (gate/up
    as a plain reducing projection through the CTA pairs + the separate activation kernel), vocabulary 1000."""
    shape = fi.ModelShape(2, 320, 5, 5, 64, ffn, 1000, 500000.0)
    B = 150
    lens = fi.prompt_lengths(B, 1, 70, 17)
    mask = fi.mask_bernoulli(B, shape.n_layers, 0.85, 18)
    errs, agrees = _run_decode_case(shape, True, lens, mask, 2, 19, 2e-2)
    assert agrees.mean() >= 0.98


def test_decode_bf16_gemv_path_and_general_attention_by_option():
    """The CUDA-core GEMV projections and the general attention kernel, forced by option, on a bf16 model."""
    shape = fi.ModelShape(2, 256, 8, 2, 128, 512, 1000, 500000.0)
    lens = fi.prompt_lengths(5, 1, 200, 23)
    mask = fi.mask_bernoulli(5, shape.n_layers, 0.7, 24)
    _run_decode_case(shape, True, lens, mask, 2, 26, 2e-2, options={"max_gemv_rows": 8, "attn_simple": 1})
    _run_decode_case(shape, True, lens, mask, 2, 26, 2e-2, options={"fuse_swiglu": 0, "use_pdl": 0, "use_graph": 0})
    _run_decode_case(shape, True, lens, mask, 2, 26, 2e-2, options={"fuse_rope": 0})


@pytest.mark.parametrize("bf16", [False, True])
def test_greedy_token_on_exact_ties_is_the_lowest_index(bf16):
    """lm_head rows v and v + V/2 are the same vector, so every logit occurs (at least) twice, exactly:
    the greedy token must be the lower index, on the device as in the oracle."""
    import torch
    shape = fi.ModelShape(2, 256, 4, 2, 64, 512, 1000, 10000.0)
    B, V = 6, shape.vocab
    w = fi.make_weights(shape, 31, bf16)
    w["lm_head"][V // 2:] = w["lm_head"][:V // 2]
    om = oracle_model(shape, w)
    lens = fi.prompt_lengths(B, 1, 40, 31)
    okv, gkv = synthetic_caches(shape, lens, [int(n) + 2 for n in lens], 31, bf16)
    ctx = _ctx(shape, bf16, B, int(max(lens)) + 2, w)
    mask = fi.mask_bernoulli(B, shape.n_layers, 0.7, 32)
    ctx.set_mask(torch.from_numpy(mask).cuda())
    toks = fi.tokens(shape, B, 31, "first")
    logits = torch.empty((B, V), dtype=torch.float32, device="cuda")
    nxt = torch.empty((B,), dtype=torch.int32, device="cuda")
    nxt_only = torch.empty((B,), dtype=torch.int32, device="cuda")
    ref = oracle.decode_step(om, toks, mask, okv)
    ctx.decode_step(torch.from_numpy(toks).cuda(), gkv.c, logits, nxt)
    got = logits.cpu().numpy()
    assert np.array_equal(ref[:, :V // 2], ref[:, V // 2:]) and np.array_equal(got[:, :V // 2], got[:, V // 2:])
    want = oracle.argmax(ref)
    assert (want < V // 2).all()
    assert np.array_equal(nxt.cpu().numpy(), oracle.argmax(got)) and (nxt.cpu().numpy() < V // 2).all()
    if not bf16:
        assert np.array_equal(nxt.cpu().numpy(), want)
    assert ctx.device_flags() == 0


def test_all_skip_and_all_keep_masks():
    shape = fi.TINY
    lens = [5, 9]
    _run_decode_case(shape, False, lens, np.zeros((2, shape.n_layers), np.uint8), 2, 8, 1e-4)
    _run_decode_case(shape, False, lens, np.ones((2, shape.n_layers), np.uint8), 2, 8, 1e-4)


def test_batch_rows_are_independent_on_gpu():
    """A row's logits do not depend on who else is in the batch (f32 path: bit-identical)."""
    import torch
    shape = fi.TINY
    w = fi.make_weights(shape, 2, False)
    lens = [12, 30, 7, 19]
    mask = fi.mask_bernoulli(4, shape.n_layers, 0.6, 77)
    toks = fi.tokens(shape, 4, 2, "t")

    def run(rows):
        _, gkv = synthetic_caches(shape, [lens[r] for r in rows], [lens[r] + 2 for r in rows], 0, False)
        # caches must hold the same values for the same sequence whatever its batch slot
        for l in range(shape.n_layers):
            for i, r in enumerate(rows):
                n = lens[r]
                gkv.load_rows(l, i, fi.synthetic_kv_rows(n, shape.kv_dim, 9, f"k{l}_{r}", False),
                              fi.synthetic_kv_rows(n, shape.kv_dim, 9, f"v{l}_{r}", False))
        ctx = _ctx(shape, False, len(rows), 64, w)
        ctx.set_mask(torch.from_numpy(mask[rows]).cuda())
        lg = torch.empty((len(rows), shape.vocab), dtype=torch.float32, device="cuda")
        ctx.decode_step(torch.from_numpy(toks[rows]).cuda(), gkv.c, lg)
        return lg.cpu().numpy()

    base = run([0, 1, 2, 3])
    perm = [2, 0, 3, 1]
    assert np.array_equal(run(perm), base[perm])
    assert np.array_equal(run([1])[0], base[1])


def test_new_mask_with_the_same_buffers_takes_effect():
    """A second first_set_mask on the same context, with the same token / cache / logits buffers,
    must change what the next step computes (cached launch sequences belong to the old plan)."""
    import torch
    shape = fi.TINY
    w = fi.make_weights(shape, 2, False)
    om = oracle_model(shape, w)
    lens = [6, 11, 3]
    ctx = _ctx(shape, False, 3, 32, w)
    toks = np.array([3, 4, 5], np.int32)
    t_dev = torch.from_numpy(toks).cuda()
    logits = torch.empty((3, shape.vocab), dtype=torch.float32, device="cuda")
    masks = [np.ones((3, shape.n_layers), np.uint8), np.array([[1, 0, 0, 1], [0, 0, 1, 1], [1, 1, 0, 0]], np.uint8),
             np.zeros((3, shape.n_layers), np.uint8)]
    okv, gkv = synthetic_caches(shape, lens, [n + 8 for n in lens], 3, False)
    for mk in masks:
        ctx.set_mask(torch.from_numpy(mk).cuda())
        for _ in range(2):  # twice: the second call replays what the first recorded
            ref = oracle.decode_step(om, toks, mk, okv)
            ctx.decode_step(t_dev, gkv.c, logits)
            err, agree = logits_check(logits.cpu().numpy(), ref)
            assert err.max() <= 1e-4 and agree.all()
    assert np.array_equal(gkv.len.cpu().numpy(), okv.len)


def test_full_slab_sets_flag_and_leaves_cache():
    import torch
    shape = fi.TINY
    w = fi.make_weights(shape, 2, False)
    okv, gkv = synthetic_caches(shape, [4, 4], [4, 6], 1, False)
    ctx = _ctx(shape, False, 2, 8, w)
    ctx.set_mask(torch.ones((2, shape.n_layers), dtype=torch.uint8, device="cuda"))
    k0 = gkv.rows_host(0, 0)[0].copy()
    ctx.decode_step(torch.tensor([1, 2], dtype=torch.int32, device="cuda"), gkv.c)
    assert ctx.device_flags() == 1
    assert np.array_equal(gkv.rows_host(0, 0)[0], k0)
    assert gkv.len.cpu().numpy()[:, 0].tolist() == [4] * shape.n_layers
    assert gkv.len.cpu().numpy()[:, 1].tolist() == [5] * shape.n_layers


def test_full_slab_on_the_tuned_attention_path():
    """bfloat16 cache, head_dim 128: the attention kernel itself appends the new key/value; a full slab must be
    left alone (flag raised, length kept) while the other sequence appends as usual."""
    import torch
    shape = fi.ModelShape(2, 256, 8, 2, 128, 512, 1000, 500000.0)
    w = fi.make_weights(shape, 2, True)
    okv, gkv = synthetic_caches(shape, [70, 70], [70, 72], 1, True)
    ctx = _ctx(shape, True, 2, 80, w)
    ctx.set_mask(torch.ones((2, shape.n_layers), dtype=torch.uint8, device="cuda"))
    full_before = [gkv.rows_host(l, 0) for l in range(shape.n_layers)]
    logits = torch.empty((2, shape.vocab), dtype=torch.float32, device="cuda")
    toks = fi.tokens(shape, 2, 5, "t")
    ctx.decode_step(torch.from_numpy(toks).cuda(), gkv.c, logits)
    assert ctx.device_flags() == 1  # FIRST_FLAG_KV_FULL
    for l in range(shape.n_layers):
        k1, v1 = gkv.rows_host(l, 0)
        assert np.array_equal(k1, full_before[l][0]) and np.array_equal(v1, full_before[l][1])
    assert gkv.len.cpu().numpy()[:, 0].tolist() == [70] * shape.n_layers
    assert gkv.len.cpu().numpy()[:, 1].tolist() == [71] * shape.n_layers
    # the sequence with room is unaffected by its neighbour: same logits as when it runs alone
    om = oracle_model(shape, w)
    okv1, _ = synthetic_caches(shape, [70, 70], [70, 72], 1, True, with_gpu=False)
    solo = oracle.OracleKV(oracle.Shape(**shape.asdict()), [72])
    for l in range(shape.n_layers):
        ks, vs = okv1.rows(l, 1)
        kd, vd = solo.rows(l, 0)
        kd[:], vd[:] = ks, vs
    solo.len[:] = 70
    solo.pos[:] = 70
    ref = oracle.decode_step(om, toks[1:2], np.ones((1, shape.n_layers), np.uint8), solo)
    err, _ = logits_check(logits[1:2].cpu().numpy(), ref)
    assert err.max() <= 2e-2


@pytest.mark.parametrize("options", [None, {"fuse_rope": 0}, {"attn_simple": 1}])
def test_slab_longer_than_the_context_was_sized_for_is_full_at_that_size(options):
    """slab_cap may exceed max_tokens_per_seq (the caller's table, never checked on the host): such a slab is used
    up to max_tokens_per_seq and then counts as full -- flag raised, cache and length untouched -- instead of
    outrunning the attention launch, which is sized by max_tokens_per_seq."""
    import torch
    shape = fi.ModelShape(2, 256, 8, 2, 128, 512, 1000, 500000.0)
    w = fi.make_weights(shape, 2, True)
    MAXT = 70
    okv, gkv = synthetic_caches(shape, [70, 40], [70 + 64, 60], 1, True)   # slab 0: 134 rows, 70 present
    ctx = _ctx(shape, True, 2, MAXT, w)
    for k, v in (options or {}).items():
        ctx.set_option(k, v)
    ctx.set_mask(torch.ones((2, shape.n_layers), dtype=torch.uint8, device="cuda"))
    before = [gkv.rows_host(l, 0) for l in range(shape.n_layers)]
    logits = torch.empty((2, shape.vocab), dtype=torch.float32, device="cuda")
    toks = fi.tokens(shape, 2, 5, "t")
    for step in range(2):
        ctx.decode_step(torch.from_numpy(toks).cuda(), gkv.c, logits)
        assert ctx.device_flags() == 1  # FIRST_FLAG_KV_FULL, every step
    for l in range(shape.n_layers):
        k1, v1 = gkv.rows_host(l, 0)
        assert np.array_equal(k1, before[l][0]) and np.array_equal(v1, before[l][1])
    assert gkv.len.cpu().numpy()[:, 0].tolist() == [70] * shape.n_layers
    assert gkv.len.cpu().numpy()[:, 1].tolist() == [42] * shape.n_layers
    assert np.isfinite(logits.cpu().numpy()).all()


def test_a_wait_that_runs_out_raises_the_flag_and_the_context_stays_usable():
    """The give-up path of the kernels' bounded waits, made to run out on purpose (a barrier nothing completes,
    no copy in flight): the kernel returns, the abort word and FIRST_FLAG_WAIT_EXPIRED are set, and the same
    context then decodes correctly."""
    import torch
    shape = fi.TINY
    errs, _ = _run_decode_case(shape, False, [5, 9], np.ones((2, shape.n_layers), np.uint8), 1, 8, 1e-4)
    from paper_2410_12513_b200 import FirstContext
    w = fi.make_weights(shape, 8, False)
    ctx = _ctx(shape, False, 2, 16, w)
    assert ctx.selftest_wait_expiry(1000) == (0, 1)
    assert ctx.device_flags() == 8
    assert ctx.device_flags() == 0
    # still good for a step
    om = oracle_model(shape, w)
    okv, gkv = synthetic_caches(shape, [5, 9], [8, 12], 8, False)
    mask = np.ones((2, shape.n_layers), np.uint8)
    ctx.set_mask(torch.from_numpy(mask).cuda())
    toks = fi.tokens(shape, 2, 8, "first")
    logits = torch.empty((2, shape.vocab), dtype=torch.float32, device="cuda")
    ctx.decode_step(torch.from_numpy(toks).cuda(), gkv.c, logits)
    err, _ = logits_check(logits.cpu().numpy(), oracle.decode_step(om, toks, mask, okv))
    assert err.max() <= 1e-4 and ctx.device_flags() == 0


def test_bad_token_sets_flag():
    import torch
    shape = fi.TINY
    _, gkv = synthetic_caches(shape, [4], [6], 1, False)
    ctx = _ctx(shape, False, 1, 8, fi.make_weights(shape, 2, False))
    ctx.set_mask(torch.ones((1, shape.n_layers), dtype=torch.uint8, device="cuda"))
    ctx.decode_step(torch.tensor([shape.vocab], dtype=torch.int32, device="cuda"), gkv.c)
    assert ctx.device_flags() == 2


# ------------------------------------------------------------------ config 0 end to end
def test_config0_prefill_route_decode_end_to_end():
    """Tiny fp32 decoder, batch 2, prompts of 32 tokens, 16 greedy steps: prompts are prefilled
    token by token with an all-keep mask, routers run on the captured layer inputs, the mask
    they give is fixed, and 16 routed steps follow.  Masks bit-exact, logits to fp32 rounding."""
    import torch
    shape, B, n, S = fi.TINY, 2, 32, 16
    L, D = shape.n_layers, shape.d_model
    w = fi.make_weights(shape, 0, False)
    om = oracle_model(shape, w)
    prompts = [fi.tokens(shape, n, 0, f"prompt{b}") for b in range(B)]
    okv = oracle.OracleKV(om.shape, [n + S] * B)
    pre = [oracle.prefill(om, okv, b, prompts[b]) for b in range(B)]
    target = np.array([[1, 0, 1, 1], [1, 1, 0, 1]], np.uint8)  # masks differ across the two sequences
    routers = [calibrate_router([pre[b]["router_in"][l] for b in range(B)], target[:, l], 1, l)[0] for l in range(L)]

    gkv = GpuKV(shape, [n + S] * B, False)
    ctx = _ctx(shape, False, B, n + S, w)
    ctx.set_mask(torch.ones((B, L), dtype=torch.uint8, device="cuda"))
    li = torch.empty((n, L, B, D), dtype=torch.float32, device="cuda")
    logits = torch.empty((B, shape.vocab), dtype=torch.float32, device="cuda")
    ptoks = torch.from_numpy(np.stack(prompts)).cuda()
    for j in range(n):
        ctx.decode_step(ptoks[:, j].contiguous(), gkv.c, logits, None, li[j])
    assert ctx.device_flags() == 0
    first_ref = np.stack([pre[b]["logits"][0] for b in range(B)])
    err, agree = logits_check(logits.cpu().numpy(), first_ref)
    assert err.max() <= 1e-4 and agree.all()
    # routers on the GPU's own prefill hidden states
    mask = torch.zeros((B, L), dtype=torch.uint8, device="cuda")
    scores = torch.zeros((B, L), dtype=torch.float32, device="cuda")
    cu = torch.tensor([0, n, 2 * n], dtype=torch.int32, device="cuda")
    for l in range(L):
        hid = li[:, l].permute(1, 0, 2).reshape(B * n, D).contiguous()  # [b][j] order
        ref_h = np.concatenate([pre[b]["router_in"][l] for b in range(B)])
        assert np.abs(hid.cpu().numpy() - ref_h).max() <= 1e-4
        ctx.prefill_route(l, hid, cu, to_dev(routers[l], False), None, 0.5, 1, mask, scores)
    assert np.array_equal(mask.cpu().numpy(), target)
    ctx.set_mask(mask)
    toks = oracle.argmax(first_ref)
    for t in range(S):
        ref = oracle.decode_step(om, toks, target, okv)
        ctx.decode_step(torch.from_numpy(toks).cuda(), gkv.c, logits)
        err, agree = logits_check(logits.cpu().numpy(), ref)
        assert err.max() <= 1e-4 and agree.all(), (t, err.max())
        toks = oracle.argmax(ref)
    assert ctx.device_flags() == 0
    assert np.array_equal(gkv.len.cpu().numpy(), okv.len)


def test_batch_changes_between_steps():
    """Continuous batching at the step boundary: with one context, a finished sequence's slot is
    handed to a new sequence with its own mask row, then the batch shrinks by one. Each phase is a
    new first_set_mask over caller-owned slabs; every sequence's logits follow the oracle run on
    that sequence's own history (decisions stay fixed per sequence for its whole decode)."""
    import torch
    from paper_2410_12513_b200 import KVCache
    shape, seed = fi.TINY, 31
    L = shape.n_layers
    w = fi.make_weights(shape, seed, False)
    om = oracle_model(shape, w)
    lens = [9, 14, 6, 11]
    caps = [40, 40, 40, 40]
    okv, gkv = synthetic_caches(shape, lens, caps, seed, False)
    mask = fi.mask_bernoulli(4, L, 0.6, seed)
    ctx = _ctx(shape, False, 4, 40, w)
    logits = torch.empty((4, shape.vocab), dtype=torch.float32, device="cuda")

    def steps(n, B, m, kvc, okv_, toks):
        for _ in range(n):
            ref = oracle.decode_step(om, toks, m, okv_)
            ctx.decode_step(torch.from_numpy(toks).cuda(), kvc, logits[:B])
            assert ctx.device_flags() == 0
            err, agree = logits_check(logits[:B].cpu().numpy(), ref)
            assert err.max() <= 1e-4 and agree.all()
            toks = oracle.argmax(ref)
        return toks

    ctx.set_mask(torch.from_numpy(mask).cuda())
    toks = steps(2, 4, mask, gkv.c, okv, fi.tokens(shape, 4, seed, "first"))

    # slot 1 finishes; a new sequence (prompt of 5 tokens, its own decisions) takes the slot
    n_new = 5
    new_row = fi.mask_bernoulli(1, L, 0.5, seed + 1)[0]
    new_row[1] = 0
    mask2 = mask.copy()
    mask2[1] = new_row
    for l in range(L):
        kr = fi.synthetic_kv_rows(n_new, shape.kv_dim, seed + 2, f"k{l}", False)
        vr = fi.synthetic_kv_rows(n_new, shape.kv_dim, seed + 2, f"v{l}", False)
        ko, vo = okv.rows(l, 1)
        ko[:], vo[:] = 0, 0
        ko[:n_new], vo[:n_new] = kr, vr
        gkv.load_rows(l, 1, kr, vr)
    okv.len[:, 1] = n_new
    okv.pos[1] = n_new
    gkv.set_len(okv.len, okv.pos)
    ctx.set_mask(torch.from_numpy(mask2).cuda())
    toks = toks.copy()
    toks[1] = fi.tokens(shape, 1, seed + 3, "new")[0]
    toks = steps(2, 4, mask2, gkv.c, okv, toks)

    # slot 3 finishes and is not refilled: the same slabs described as a batch of three
    o3 = oracle.OracleKV(oracle.Shape(**shape.asdict()), caps[:3])
    for l in range(L):
        for b in range(3):
            ks, vs = okv.rows(l, b)
            kd, vd = o3.rows(l, b)
            kd[:], vd[:] = ks, vs
    o3.len[:] = okv.len[:, :3]
    o3.pos[:] = okv.pos[:3]
    len3 = gkv.len[:, :3].contiguous()
    pos3 = gkv.pos[:3].contiguous()
    kv3 = KVCache(gkv.k, gkv.v, gkv.slab_off[:3].contiguous(), gkv.slab_cap[:3].contiguous(), len3, pos3)
    ctx.set_mask(torch.from_numpy(mask2[:3].copy()).cuda())
    steps(2, 3, mask2[:3].copy(), kv3, o3, toks[:3].copy())
    assert np.array_equal(len3.cpu().numpy(), o3.len) and np.array_equal(pos3.cpu().numpy(), o3.pos)


# ------------------------------------------------------------------ sampling (temperature + top-k)
def _sample_agrees(row, k, T, u, got):
    """The oracle's token; where the draw sits within 1e-5 of a boundary of the oracle's cumulative
    distribution (float32 on the device, float64 in the oracle) either neighbour is right."""
    tok, cand, prob = oracle.sample_topk(row, k, T, u)
    if got == tok:
        return True
    cdf = np.cumsum(prob)
    j = list(cand).index(tok)
    near = [cand[i] for i in (j - 1, j + 1) if 0 <= i < k and min(abs(cdf[min(i, j)] - u), 1) < 1e-5]
    return got in near


@pytest.mark.parametrize("V", [1000, 1003, 128256])
def test_sample_topk_matches_oracle(V):
    import torch
    from paper_2410_12513_b200 import first_sample_topk
    B = 6
    g = np.random.default_rng(V)
    logits = g.normal(0, 3, (B, V)).astype(np.float32)
    logits[1] = np.round(logits[1] * 2) / 2          # many equal values: candidates enter in index order
    logits[2, ::3] = -np.inf
    logits[3] = 0.0                                    # all equal: the first k indices, equal shares
    logits[4, V - 1] = 50.0                            # the last (tail) element wins
    dl = torch.from_numpy(logits).cuda()
    out = torch.empty(B, dtype=torch.int32, device="cuda")
    for k, T in ((1, 0.8), (2, 0.8), (10, 0.8), (16, 1.7), (10, 0.0), (10, 0.05)):
        for rep in range(6):
            u = g.random(B).astype(np.float32)
            if rep == 0:
                u[:] = 0.0
            first_sample_topk(dl, k, T, torch.from_numpy(u).cuda(), out)
            got = out.cpu().numpy()
            for b in range(B):
                assert _sample_agrees(logits[b], k, T, float(u[b]), int(got[b])), (V, k, T, b, u[b], got[b])
    # an even grid of draws visits every candidate of a row in proportion (coarse check of the whole table)
    n = 512
    rows = torch.from_numpy(np.repeat(logits[:1], n, 0)).cuda()
    u = ((np.arange(n) + 0.5) / n).astype(np.float32)
    outn = torch.empty(n, dtype=torch.int32, device="cuda")
    first_sample_topk(rows, 10, 0.8, torch.from_numpy(u).cuda(), outn)
    _, cand, prob = oracle.sample_topk(logits[0], 10, 0.8, 0.0)
    counts = np.array([(outn.cpu().numpy() == c).sum() for c in cand])
    assert counts.sum() == n and np.abs(counts / n - prob).max() <= 2.0 / n


def test_sample_topk_rejects_bad_arguments():
    import torch
    from paper_2410_12513_b200 import FirstError, first_sample_topk
    lg = torch.zeros((2, 64), device="cuda")
    u = torch.zeros(2, device="cuda")
    out = torch.empty(2, dtype=torch.int32, device="cuda")
    for k, T in ((0, 1.0), (17, 1.0), (65, 1.0), (4, -1.0)):
        with pytest.raises(FirstError):
            first_sample_topk(lg, k, T, u, out)


def test_decode_step_samples_when_asked():
    """first_set_sampling switches the step's next-token kernel: the sampled tokens are the
    oracle's sampling rule applied to the step's own logits (which are checked against the
    oracle's as in every other case); switching back restores argmax."""
    import torch
    shape, seed, B = fi.TINY, 41, 5
    w = fi.make_weights(shape, seed, False)
    om = oracle_model(shape, w)
    lens = fi.prompt_lengths(B, 1, 40, seed)
    okv, gkv = synthetic_caches(shape, lens, [int(n) + 4 for n in lens], seed, False)
    mask = fi.mask_bernoulli(B, shape.n_layers, 0.6, seed)
    ctx = _ctx(shape, False, B, int(max(lens)) + 4, w)
    ctx.set_mask(torch.from_numpy(mask).cuda())
    u_dev = torch.zeros(B, dtype=torch.float32, device="cuda")
    ctx.set_sampling(10, 0.8, u_dev)
    logits = torch.empty((B, shape.vocab), dtype=torch.float32, device="cuda")
    nxt = torch.empty(B, dtype=torch.int32, device="cuda")
    toks = fi.tokens(shape, B, seed, "first")
    g = np.random.default_rng(seed)
    for step in range(3):
        if step == 2:
            ctx.set_sampling(0, 0.0, None)
        u = g.random(B).astype(np.float32)
        u_dev.copy_(torch.from_numpy(u))
        ref = oracle.decode_step(om, toks, mask, okv)
        ctx.decode_step(torch.from_numpy(toks).cuda(), gkv.c, logits, nxt)
        got, tok = logits.cpu().numpy(), nxt.cpu().numpy()
        err, _ = logits_check(got, ref)
        assert err.max() <= 1e-4
        for b in range(B):
            if step < 2:
                assert _sample_agrees(got[b], 10, 0.8, float(u[b]), int(tok[b]))
            else:
                assert tok[b] == got[b].argmax()
        toks = oracle.argmax(ref)
    assert ctx.device_flags() == 0


@pytest.mark.parametrize("bf16", [False, True])
def test_per_layer_slab_tables(bf16):
    """Once the masks are fixed a layer only needs slabs for the sequences that keep it ("Inference for
    FiRST", item 2).  The same decode, run from caches that hold exactly those slabs (per-layer tables,
    per-layer tensor heights), gives the same logits as from full caches (bit for bit on the float32 path),
    and the oracle's."""
    import torch
    from paper_2410_12513_b200 import KVCache
    shape = fi.ModelShape(3, 256, 8, 2, 128, 512, 1000, 500000.0) if bf16 else fi.TINY
    seed, B, steps = 51, 6, 3
    L = shape.n_layers
    w = fi.make_weights(shape, seed, bf16)
    om = oracle_model(shape, w)
    lens = fi.prompt_lengths(B, 1, 150, seed)
    caps = [int(n) + steps + (b % 2) for b, n in enumerate(lens)]
    mask = fi.mask_bernoulli(B, L, 0.6, seed)
    mask[:, 1] = 0  # a layer nobody keeps: no tensors at all for it
    okv, gkv = synthetic_caches(shape, lens, caps, seed, bf16)
    # per-layer caches: only the kept sequences' slabs, packed
    k2, v2 = [None] * L, [None] * L
    off2 = np.zeros((L, B), np.int64)
    cap2 = np.zeros((L, B), np.int32)
    for l in range(L):
        kept = [b for b in range(B) if mask[b, l]]
        if not kept:
            continue
        cap2[l, kept] = [caps[b] for b in kept]
        off2[l, kept] = np.concatenate([[0], np.cumsum([caps[b] for b in kept])[:-1]])
        height = int(cap2[l].sum())
        k2[l] = torch.zeros((shape.n_kv_heads, height, shape.head_dim), dtype=gkv.k[l].dtype, device="cuda")
        v2[l] = torch.zeros_like(k2[l])
        for b in kept:
            o, o2, cp = int(gkv.off[b]), int(off2[l, b]), caps[b]
            k2[l][:, o2:o2 + cp] = gkv.k[l][:, o:o + cp]
            v2[l][:, o2:o2 + cp] = gkv.v[l][:, o:o + cp]
    full_rows = L * sum(caps)
    kept_rows = int(cap2.sum())
    assert kept_rows == sum(caps[b] for b in range(B) for l in range(L) if mask[b, l]) and kept_rows < 0.75 * full_rows
    kv2 = KVCache(k2, v2, torch.from_numpy(off2).cuda(), torch.from_numpy(cap2).cuda(), gkv.len.clone(), gkv.pos.clone())
    ctx = _ctx(shape, bf16, B, max(caps), w)
    ctx.set_mask(torch.from_numpy(mask).cuda())
    la = torch.empty((B, shape.vocab), dtype=torch.float32, device="cuda")
    lb = torch.empty_like(la)
    toks = fi.tokens(shape, B, seed, "first")
    for _ in range(steps):
        ref = oracle.decode_step(om, toks, mask, okv)
        td = torch.from_numpy(toks).cuda()
        ctx.decode_step(td, gkv.c, la)
        ctx.decode_step(td, kv2, lb)
        assert ctx.device_flags() == 0
        if bf16:  # the tensor-core projections reduce K ranges with float atomics: run-to-run order differs
            assert logits_check(lb.cpu().numpy(), la.cpu().numpy())[0].max() <= 1e-4
        else:
            assert torch.equal(la, lb)
        err, _ = logits_check(lb.cpu().numpy(), ref)
        assert err.max() <= (2e-2 if bf16 else 1e-4)
        toks = oracle.argmax(ref)
    assert torch.equal(kv2.len, gkv.len) and torch.equal(kv2.pos, gkv.pos)


def test_in_step_trace_lists_every_launch_in_order():
    """Option "stamp": every launch of a step records first-CTA start and last-warp end; the trace has one entry
    per launch, in launch order, with start <= end, ends non-decreasing along the dependency chain, and the logits
    are the same as without it."""
    import torch
    shape = fi.ModelShape(3, 256, 8, 2, 64, 512, 1000, 500000.0)
    B = 6
    w = fi.make_weights(shape, 3, True)
    lens = fi.prompt_lengths(B, 1, 100, 3)
    mask = fi.mask_bernoulli(B, shape.n_layers, 0.7, 4)
    mask[:, 1] = 0                                   # a layer nobody keeps: no launches for it
    okv, gkv = synthetic_caches(shape, lens, [int(n) + 4 for n in lens], 3, True)
    ctx = _ctx(shape, True, B, int(max(lens)) + 4, w)
    ctx.set_mask(torch.from_numpy(mask).cuda())
    toks = torch.from_numpy(fi.tokens(shape, B, 3, "first")).cuda()
    logits = torch.empty((B, shape.vocab), dtype=torch.float32, device="cuda")
    l0 = ctx.launch_count()
    ctx.decode_step(toks, gkv.c, logits)
    per_step = ctx.launch_count() - l0
    plain = logits.cpu().numpy().copy()
    gkv.set_len(okv.len, okv.pos)
    ctx.set_option("stamp", 1)
    ctx.decode_step(toks, gkv.c, logits)
    tr = ctx.step_trace()
    assert len(tr) == per_step == 1 + 7 * 2 + 3      # begin, 7 per kept layer, final norm + lm_head + end
    names = [t[0] for t in tr]
    assert names[0] == "step_begin" and names[-1] == "step_end" and names.count("attn_split") == 2
    assert names.count("rmsnorm_rows") == 5 and names.count("gemm_tc") == 9
    assert all(0 < t0 <= t1 for _, t0, t1 in tr)
    ends = [t1 for _, _, t1 in tr]
    assert all(b >= a for a, b in zip(ends, ends[1:]))   # each kernel ends after the one it depends on
    assert (ends[-1] - tr[0][1]) < 50_000_000            # one clock, nanoseconds: the step took well under 50 ms
    err, _ = logits_check(logits.cpu().numpy(), plain)
    assert err.max() <= 1e-3                               # same step (float32 reduction order may differ)
    ctx.set_option("stamp", 0)
    with pytest.raises(Exception):
        ctx.step_trace()
    assert ctx.device_flags() == 0


def test_documented_error_statuses():
    """The statuses the header promises: unsupported shapes at create, call order, capacity, sampling limits."""
    import dataclasses
    import torch
    from paper_2410_12513_b200 import FirstError
    w = fi.make_weights(fi.TINY, 3, False)
    gw = gpu_weights(w)
    from paper_2410_12513_b200 import FirstContext

    def create_status(shape):
        try:
            FirstContext(shape, F32, 2, 16, gw)
        except FirstError as e:
            return e.status
        return 0

    assert create_status(dataclasses.replace(fi.TINY, n_q_heads=5, n_kv_heads=1, head_dim=64)) == -3   # 5 query heads per KV head
    assert create_status(dataclasses.replace(fi.TINY, head_dim=48)) in (-2, -3)                        # head_dim not 32/64/128
    assert create_status(dataclasses.replace(fi.TINY, n_q_heads=4, n_kv_heads=3)) == -2                # heads do not divide
    ctx = _ctx(fi.TINY, False, 2, 16, w)
    _, gkv = synthetic_caches(fi.TINY, [3, 3], [8, 8], 1, False)
    toks = torch.zeros(2, dtype=torch.int32, device="cuda")
    with pytest.raises(FirstError) as e:   # decode before any mask
        ctx.decode_step(toks, gkv.c)
    assert e.value.status == -7
    with pytest.raises(FirstError) as e:   # batch beyond max_batch
        ctx.set_mask(torch.ones((3, fi.TINY.n_layers), dtype=torch.uint8, device="cuda"))
    assert e.value.status == -4
    with pytest.raises(FirstError) as e:   # top_k beyond the device limit
        ctx.set_sampling(17, 0.8, torch.zeros(2, device="cuda"))
    assert e.value.status == -3
    with pytest.raises(FirstError) as e:   # sampling without draws
        ctx.set_sampling(10, 0.8, None)
    assert e.value.status == -1
    ctx.set_mask(torch.ones((2, fi.TINY.n_layers), dtype=torch.uint8, device="cuda"))
    ctx.decode_step(toks, gkv.c)           # and the context still works afterwards
    assert ctx.device_flags() == 0


def test_next_tokens_without_a_logits_buffer():
    """next_tokens alone (the library keeps the logits to itself) gives the same tokens as asking for both,
    greedy and sampled."""
    import torch
    shape, seed, B = fi.TINY, 61, 4
    w = fi.make_weights(shape, seed, False)
    lens = [5, 9, 3, 12]
    ctx = _ctx(shape, False, B, 24, w)
    mask = fi.mask_bernoulli(B, shape.n_layers, 0.7, seed)
    ctx.set_mask(torch.from_numpy(mask).cuda())
    toks = torch.from_numpy(fi.tokens(shape, B, seed, "t")).cuda()
    u = torch.tensor([0.1, 0.5, 0.7, 0.95], dtype=torch.float32, device="cuda")
    for sampled in (False, True):
        ctx.set_sampling(10 if sampled else 0, 0.8 if sampled else 0.0, u if sampled else None)
        out = []
        for with_logits in (True, False):
            _, gkv = synthetic_caches(shape, lens, [16] * B, seed, False)
            nxt = torch.full((B,), -1, dtype=torch.int32, device="cuda")
            logits = torch.empty((B, shape.vocab), dtype=torch.float32, device="cuda") if with_logits else None
            ctx.decode_step(toks, gkv.c, logits, nxt)
            assert ctx.device_flags() == 0
            out.append(nxt.cpu().numpy())
        assert (out[0] >= 0).all() and np.array_equal(out[0], out[1])
