"""Batches that change between decode steps: the slab pool (first_pool_*, first_seq_join / first_seq_leave),
the plan update without a stream wait (first_set_mask_host) and the reuse of recorded step graphs, against
per-sequence runs of the host oracle.  "Inference for FiRST", item 2: a sequence's layer decisions are fixed for
its whole decode and a skipped layer needs no cache, so sequences join and leave independently and a sequence
holds cache rows only in the layers it keeps."""
import numpy as np
import pytest

import first_inputs as fi
import oracle
from harness import GpuKV, calibrate_router, gpu_weights, logits_check, oracle_model, to_dev

pytestmark = pytest.mark.gpu


class _Seq:
    """One sequence on the oracle side: its own cache (batch of one), mask, next token."""

    def __init__(self, om, shape, prompt, mask_row, cap):
        self.om, self.mask = om, np.asarray(mask_row, np.uint8)[None, :]
        self.kv = oracle.OracleKV(om.shape, [cap])
        pre = oracle.prefill(om, self.kv, 0, prompt, want_router_in=False)
        self.tok = oracle.argmax(np.asarray(pre["logits"]).reshape(-1, shape.vocab)[:1])
        self.slot = None
        self.steps = 0

    def step(self):
        ref = oracle.decode_step(self.om, self.tok, self.mask, self.kv)
        fed = int(self.tok[0])
        self.tok = oracle.argmax(ref)
        self.steps += 1
        return fed, ref[0]


@pytest.mark.parametrize("bf16", [False, True])
def test_join_leave_schedule_against_per_sequence_oracle_runs(bf16):
    import torch
    from paper_2410_12513_b200 import FirstContext, FirstPool
    shape = fi.ModelShape(4, 256, 8, 2, 64, 512, 1000, 500000.0) if bf16 else fi.TINY
    L, MAXS, NEW = shape.n_layers, 5, 12
    w = fi.make_weights(shape, 77, bf16)
    om = oracle_model(shape, w)
    gw = gpu_weights(w)
    ctx = FirstContext(shape, 1 if bf16 else 0, 64, 96, gw)
    # 14 sequences, prompts 1..60 tokens, masks with 0..L-1 skipped layers (first layer always kept)
    rng = np.random.default_rng(5)
    n_seq = 14
    lens = [int(x) for x in rng.integers(1, 61, n_seq)]
    lens[3] = 1
    prompts = [fi.tokens(shape, n, 77, f"p{i}") for i, n in enumerate(lens)]
    masks = fi.mask_bernoulli(n_seq, L, 0.6, 78)
    masks[:, 0] = 1
    masks[5, :] = 1
    masks[6, 1:] = 0
    rows = [600] * L
    dt = torch.bfloat16 if bf16 else torch.float32
    pk = [torch.zeros((shape.n_kv_heads, r, shape.head_dim), dtype=dt, device="cuda") for r in rows]
    pv = [torch.zeros((shape.n_kv_heads, r, shape.head_dim), dtype=dt, device="cuda") for r in rows]
    pool = FirstPool(ctx, MAXS, pk, pv)
    # staging cache for one prompt at a time (every layer, as the prompt phase fills it)
    stage = GpuKV(shape, [64], bf16)
    live, events, checked = {}, 0, 0
    tokens = torch.zeros((MAXS,), dtype=torch.int32, device="cuda")
    logits = torch.empty((MAXS, shape.vocab), dtype=torch.float32, device="cuda")
    tol = 2e-2 if bf16 else 1e-4

    def join(i):
        nonlocal events
        cap = lens[i] + NEW
        sq = _Seq(om, shape, prompts[i], masks[i], cap)
        ctx.prefill(torch.from_numpy(prompts[i].astype(np.int32)).cuda(), np.array([0, lens[i]], np.int32), stage.c)
        sq.slot = pool.join(masks[i], cap, src=stage.c, src_seq=0, n_tokens=lens[i])
        assert sq.slot not in [s.slot for s in live.values()]
        live[i] = sq
        events += 1

    def leave(i):
        nonlocal events
        pool.leave(live.pop(i).slot)
        events += 1

    def held_expected():
        return [sum((lens[i] + NEW) for i in live if masks[i, l]) for l in range(L)]

    def steps(n):
        nonlocal checked
        for _ in range(n):
            refs = {}
            tk = np.zeros(MAXS, np.int32)
            for i, sq in live.items():
                tk[sq.slot], refs[i] = sq.step()
            tokens.copy_(torch.from_numpy(tk))
            ctx.decode_step(tokens, pool.kv, logits)
            got = logits.cpu().numpy()
            for i, sq in live.items():
                err, _ = logits_check(got[sq.slot][None], refs[i][None])
                assert err.max() <= tol, (i, sq.slot, sq.steps, err.max())
                checked += 1
        assert ctx.device_flags() == 0

    schedule = [("join", 0), ("join", 1), ("join", 2), ("commit", 2), ("leave", 1), ("join", 3), ("join", 4), ("commit", 2),
                ("leave", 0), ("leave", 3), ("join", 5), ("commit", 3), ("join", 6), ("join", 7), ("commit", 2), ("leave", 2),
                ("leave", 5), ("join", 8), ("join", 9), ("commit", 2), ("leave", 4), ("leave", 6), ("leave", 7), ("join", 10),
                ("commit", 2), ("join", 11), ("join", 12), ("commit", 1), ("leave", 8), ("leave", 9), ("leave", 10), ("join", 13),
                ("commit", 3), ("leave", 11), ("leave", 12), ("leave", 13), ("commit", 1)]
    for what, arg in schedule:
        if what == "join":
            join(arg)
        elif what == "leave":
            leave(arg)
        else:
            pool.commit()
            held, _, n_live = pool.stats()
            assert n_live == len(live) and held.tolist() == held_expected()  # rows held = sum over kept (sequence, layer)
            steps(arg)
    assert events >= 28 and checked >= 40
    held, big, n_live = pool.stats()
    assert n_live == 0 and not held.any() and big.tolist() == rows  # everything came back, ranges merged again
    # the batch rows are a resource too: a sixth sequence is refused
    for i in range(MAXS):
        pool.join(np.ones(L, np.uint8), 8)
    with pytest.raises(Exception) as e:
        pool.join(np.ones(L, np.uint8), 8)
    assert e.value.status == -4
    pool.close()


def test_refused_join_takes_nothing():
    import torch
    from paper_2410_12513_b200 import FirstContext, FirstError, FirstPool
    shape = fi.TINY
    ctx = FirstContext(shape, 0, 8, 64, gpu_weights(fi.make_weights(shape, 1, False)))
    L = shape.n_layers
    rows = [100, 100, 40, 100]
    pk = [torch.zeros((shape.n_kv_heads, r, shape.head_dim), device="cuda") for r in rows]
    pv = [torch.zeros((shape.n_kv_heads, r, shape.head_dim), device="cuda") for r in rows]
    pool = FirstPool(ctx, 4, pk, pv)
    a = pool.join(np.ones(L, np.uint8), 30)
    with pytest.raises(FirstError) as e:
        pool.join(np.ones(L, np.uint8), 30)          # layer 2 has 10 rows left
    assert e.value.status == -4
    assert pool.stats()[0].tolist() == [30, 30, 30, 30] and pool.stats()[2] == 1
    b = pool.join(np.array([1, 1, 0, 1], np.uint8), 30)  # the same sequence fits if it skips layer 2
    assert pool.stats()[0].tolist() == [60, 60, 30, 60] and {a, b} == {0, 1}
    with pytest.raises(FirstError) as e:
        pool.leave(3)
    assert e.value.status == -7
    with pytest.raises(FirstError):
        pool.join(np.array([1, 2, 0, 1], np.uint8), 4)
    pool.leave(a)
    assert pool.stats()[0].tolist() == [30, 30, 0, 30] and pool.stats()[1].tolist() == [40, 40, 40, 40]
    pool.leave(b)
    assert pool.stats()[1].tolist() == rows
    pool.close()


def test_host_mask_plan_matches_device_plan_and_step_graphs_survive_batch_changes():
    """first_set_mask_host gives the plan first_set_mask gives, without reading anything back; the launches are sized
    from counts rounded up to 16 while the kernels read the exact counts, so logits agree with the exact-count path
    and a mask change that keeps the buckets replays the recorded graph."""
    import torch
    from paper_2410_12513_b200 import FirstContext
    from harness import synthetic_caches
    shape = fi.ModelShape(3, 256, 8, 2, 64, 512, 1000, 500000.0)
    B, L = 40, shape.n_layers
    w = fi.make_weights(shape, 9, True)
    om = oracle_model(shape, w)
    lens = fi.prompt_lengths(B, 1, 50, 9)
    ctx = FirstContext(shape, 1, B, 64, gpu_weights(w))
    toks = fi.tokens(shape, B, 9, "first")
    logits = torch.empty((B, shape.vocab), dtype=torch.float32, device="cuda")
    masks = [fi.mask_bernoulli(B, L, 0.7, 10 + i) for i in range(4)]
    masks[2][:, 1] = 0                        # a layer nobody keeps
    masks[3] = masks[0].copy()                # same counts as mask 0 per layer, other rows: swap two rows' masks
    masks[3][[0, 1]] = masks[3][[1, 0]]
    graphs = []
    toks_d = torch.from_numpy(toks).cuda()
    okv, gkv = synthetic_caches(shape, lens, [int(n) + 8 for n in lens], 9, True)
    len0, pos0 = okv.len.copy(), okv.pos.copy()
    for i, mask in enumerate(masks):
        okv.len[:], okv.pos[:] = len0, pos0   # every mask starts from the same caches (same buffers: same graph key)
        gkv.set_len(len0, pos0)
        ctx.set_mask_host(mask)
        idx, cnt, slot = ctx.get_plan()
        oi, oc, os_ = oracle.plan(mask)
        assert np.array_equal(idx, oi) and np.array_equal(cnt, oc) and np.array_equal(slot, os_)
        ref = oracle.decode_step(om, toks, mask, okv)
        ctx.decode_step(toks_d, gkv.c, logits)
        err, _ = logits_check(logits.cpu().numpy(), ref)
        assert err.max() <= 2e-2, (i, err.max())
        assert np.array_equal(gkv.len.cpu().numpy(), okv.len)
        assert ctx.device_flags() == 0
        graphs.append(ctx.graph_count())
    assert graphs[3] == graphs[2]             # mask 3 has mask 0's per-layer counts: its recorded graph is replayed
    assert graphs[0] >= 1
    with pytest.raises(Exception):
        bad = masks[0].copy()
        bad[3, 1] = 2
        ctx.set_mask_host(bad)
