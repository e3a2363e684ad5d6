"""first_prefill (whole prompt phase in one call) vs the host oracle's prefill, through the C ABI (B200 only).

"Inference for FiRST": (1) the prompt runs through every layer, (2) the routers' decisions on the
prompt are then fixed for the decode steps.  Checked here: keys/values of every layer, len/pos,
first-token logits, router scores and masks (bit-exact), and routed decode steps that continue
from the prefilled caches.
"""
import numpy as np
import pytest

import first_inputs as fi
import oracle
from harness import GpuKV, calibrate_router, gpu_weights, logits_check, oracle_model, to_dev

pytestmark = pytest.mark.gpu

F32, BF16 = 0, 1
SMALL_GQA = fi.ModelShape(3, 256, 8, 2, 64, 512, 2048, 500000.0)


def _ctx(shape, bf16, max_batch, max_tokens, w):
    from paper_2410_12513_b200 import FirstContext
    return FirstContext(shape, BF16 if bf16 else F32, max_batch, max_tokens, gpu_weights(w))


def _prefill_case(shape, bf16, lens, max_batch, steps, seed, mode, keep_p, rel_tol, options=None, tight=False,
                  sharpen=(0, 0)):
    """Oracle prefill per sequence -> routers calibrated on its layer inputs -> one first_prefill
    call on the GPU -> everything it leaves behind compared -> `steps` routed decode steps."""
    import torch
    B, L = len(lens), shape.n_layers
    w = fi.make_weights(shape, seed, bf16)
    if sharpen != (0, 0):  # query / key projections times 2^a / 2^b (exact in bfloat16): attention scores of several units
        assert bf16
        for l in range(L):
            w["wq"][l] = (w["wq"][l] + np.uint16(sharpen[0] << 7)).astype(np.uint16)
            w["wk"][l] = (w["wk"][l] + np.uint16(sharpen[1] << 7)).astype(np.uint16)
    om = oracle_model(shape, w)
    prompts = [fi.tokens(shape, int(n), seed, f"prompt{b}") for b, n in enumerate(lens)]
    caps = [int(n) + steps + (3 if b == 0 else 0) for b, n in enumerate(lens)]
    okv = oracle.OracleKV(om.shape, caps)
    pre = [oracle.prefill(om, okv, b, prompts[b]) for b in range(B)]
    target = fi.mask_bernoulli(B, L, keep_p, seed + 7)
    routers, rho = [], []
    for l in range(L):
        rw, r = calibrate_router([pre[b]["router_in"][l] for b in range(B)], target[:, l], mode, l, tight=tight)
        routers.append(rw)
        rho.append(r)
    rho = np.stack(rho, 1)  # [B][L]
    if tight:
        assert 1e-3 <= np.abs(rho - 0.5).min() <= 2e-3

    gkv = GpuKV(shape, caps, bf16)
    ctx = _ctx(shape, bf16, max_batch, max(caps), w)
    for k, v in (options or {}).items():
        ctx.set_option(k, v)
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    toks = torch.from_numpy(np.concatenate(prompts).astype(np.int32)).cuda()
    mask = torch.full((B, L), 7, dtype=torch.uint8, device="cuda")
    scores = torch.zeros((B, L), dtype=torch.float32, device="cuda")
    logits = torch.empty((B, shape.vocab), dtype=torch.float32, device="cuda")
    nxt = torch.empty((B,), dtype=torch.int32, device="cuda")
    ctx.prefill(toks, cu, gkv.c, to_dev(np.stack(routers), False), None, 0.5, mode, mask, scores, logits, nxt)
    assert ctx.device_flags() == 0

    # bookkeeping and caches: every layer holds the whole prompt
    assert np.array_equal(gkv.len.cpu().numpy(), okv.len)
    assert np.array_equal(gkv.pos.cpu().numpy(), okv.pos)
    tol = 2e-2 if bf16 else 1e-4
    for l in range(L):
        for b in range(B):
            n = int(lens[b])
            k1, v1 = gkv.rows_host(l, b)
            ko, vo = okv.rows(l, b)
            assert np.abs(k1[:n] - ko[:n]).max() <= tol * max(1.0, np.abs(ko[:n]).max()), (l, b)
            assert np.abs(v1[:n] - vo[:n]).max() <= tol * max(1.0, np.abs(vo[:n]).max()), (l, b)
            assert not k1[n:].any() and not v1[n:].any()  # nothing written past the prompt
    # first-token logits and greedy token
    ref0 = np.stack([pre[b]["logits"][0] if pre[b]["logits"].ndim > 1 else pre[b]["logits"] for b in range(B)])
    got0 = logits.cpu().numpy()
    err, agree = logits_check(got0, ref0)
    assert err.max() <= rel_tol, err.max()
    assert np.array_equal(nxt.cpu().numpy(), got0.argmax(-1).astype(np.int32))
    # routers: masks bit-exact, scores close
    assert np.array_equal(mask.cpu().numpy(), target)
    assert np.abs(scores.cpu().numpy() - rho).max() <= (5e-3 if bf16 else 1e-5)

    # the decode steps that follow obey the masks and continue from these caches
    with pytest.raises(Exception):
        ctx.decode_step(nxt, gkv.c, logits)  # the prefill dropped the plan: a mask must be set first
    ctx.set_mask(mask)
    toks_t = oracle.argmax(ref0)
    for t in range(steps):
        ref = oracle.decode_step(om, toks_t, target, okv)
        ctx.decode_step(torch.from_numpy(toks_t).cuda(), gkv.c, logits)
        err, agree = logits_check(logits.cpu().numpy(), ref)
        assert err.max() <= rel_tol, (t, err.max())
        toks_t = oracle.argmax(ref)
    assert ctx.device_flags() == 0
    assert np.array_equal(gkv.len.cpu().numpy(), okv.len)
    assert np.array_equal(gkv.pos.cpu().numpy(), okv.pos)
    return err


def test_prefill_config0_chunks_cross_sequence_boundaries():
    """Tiny fp32 decoder, batch 2, prompts of 32 tokens (config 0), pooled-sigmoid routers; chunks of
    24 rows: 24 + 24 + 16, the second one holding the end of sequence 0 and the start of sequence 1."""
    _prefill_case(fi.TINY, False, [32, 32], 24, 4, 0, 1, 0.6, 1e-4)


@pytest.mark.parametrize("mode", [0, 1])
def test_prefill_f32_router_masks_at_the_stated_margin(mode):
    """float32 model, routers scaled so that the nearest oracle score is 1e-3 .. 2e-3 from tau: the hidden
    states are the device's own float32 prefill here (not shared bytes), and the masks are still bit-exact."""
    _prefill_case(fi.TINY, False, [32, 32, 7, 1, 50], 24, 2, 40 + mode, mode, 0.6, 1e-4, tight=True)


@pytest.mark.parametrize("max_batch", [5, 64, 300])
def test_prefill_f32_ragged(max_batch):
    """Ragged prompts (one of a single token), the paper's router order, three chunk sizes: a chunk per
    few tokens, chunks of 64, and one chunk shorter than the 256-row limit for the whole batch."""
    _prefill_case(fi.TINY, False, [1, 17, 64, 9, 40], max_batch, 3, 3, 0, 0.5, 1e-4)


@pytest.mark.parametrize("max_batch", [48, 256])
def test_prefill_bf16_gqa_ragged(max_batch):
    """bfloat16 weights and caches, 4 query heads per KV head, head_dim 64: tensor-core projections and
    the tuned attention kernel on chunk rows."""
    _prefill_case(SMALL_GQA, True, [8, 200, 77, 130, 1], max_batch, 3, 5, 0, 0.6, 2e-2)


@pytest.mark.parametrize("hq,hkv,hd", [(4, 4, 64), (4, 2, 128), (6, 2, 64), (8, 1, 64)])
def test_prefill_bf16_query_head_groupings(hq, hkv, hd):
    """1, 2, 3 and 8 query heads per KV head: the first three let two consecutive prompt tokens share an
    attention work item (their query heads fit the spare fragment rows), the last does not."""
    shape = fi.ModelShape(2, hq * hd, hq, hkv, hd, 512, 1024, 500000.0)
    _prefill_case(shape, True, [70, 3, 131], 64, 2, 8, 0, 0.6, 2e-2)


def test_prefill_bf16_pairing_off_by_option():
    """Every prompt token with attention work items of its own (neither groups of eight nor pairs)."""
    _prefill_case(SMALL_GQA, True, [33, 90, 5], 32, 2, 6, 1, 0.6, 2e-2,
                  {"prefill_tc": 0, "prefill_group": 0, "prefill_pair": 0, "prefill_rows": 20})


def test_prefill_bf16_pairs_by_option():
    """The pair form (two consecutive tokens per work item), which groups of eight replaced (option `prefill_tc` 0, `prefill_group` 0)."""
    _prefill_case(SMALL_GQA, True, [33, 90, 5], 32, 2, 6, 1, 0.6, 2e-2, {"prefill_tc": 0, "prefill_group": 0, "prefill_rows": 20})
    _prefill_case(SMALL_GQA, True, [33, 90, 5, 1, 2, 200], 256, 2, 7, 0, 0.6, 2e-2, {"prefill_tc": 0, "prefill_group": 0})


@pytest.mark.parametrize("rows,chunk_tokens", [(20, 64), (256, 64), (37, 128), (256, 1024)])
def test_prefill_bf16_groups_of_eight(rows, chunk_tokens):
    """Groups of up to eight consecutive tokens per attention work item (`prefill_tc` 0: the mma.sync form), at chunk heights that cut
    groups at odd places (20, 37 rows), with prompts of 1, 2, 7, 8, 9 tokens (groups of every size, sequences that
    start in the middle of a chunk) and prompts long enough for several token chunks per group (merged by ticket)."""
    _prefill_case(SMALL_GQA, True, [33, 90, 5, 1, 2, 7, 8, 9, 300, 16], rows, 2, 8, 1, 0.6, 2e-2,
                  {"prefill_tc": 0, "prefill_rows": rows, "attn_chunk": chunk_tokens})


@pytest.mark.parametrize("hd", [64, 128])
def test_prefill_bf16_many_tiny_prompts(hd):
    """Dozens of prompts of one to five tokens side by side: almost every window of eight rows holds several group
    leaders, which one attention CTA serves one after the other while its producer already fetches the next group's
    tiles; a few longer prompts in between (several tiles, several token chunks)."""
    shape = fi.ModelShape(2, 256, 8, 2, hd, 512, 2048, 500000.0)
    lens = [1, 2, 3, 1, 1, 2, 5, 1, 4, 1, 150, 2, 1, 3, 1, 1, 70, 2, 2, 1, 5, 1, 1, 3, 9, 1, 2, 1, 1, 4] * 2
    _prefill_case(shape, True, lens, 256, 1, 9, 1, 0.6, 2e-2, {"prefill_tc": 0, "attn_chunk": 64})
    _prefill_case(shape, True, lens, 64, 1, 9, 0, 0.6, 2e-2, {"prefill_tc": 0})


@pytest.mark.parametrize("rows,chunk_tokens", [(20, 64), (256, 64), (37, 128), (256, 1024)])
def test_prefill_bf16_tensor_core_blocks(rows, chunk_tokens):
    """Attention of prompt chunks on the tcgen05 tensor cores (option `prefill_tc`, the default): blocks of 128/G consecutive
    tokens per work item, at chunk heights that cut blocks at odd places, with prompts of 1 .. 300 tokens (blocks of
    every size, sequences that start in the middle of a chunk, several tiles and several token chunks per block)."""
    _prefill_case(SMALL_GQA, True, [33, 90, 5, 1, 2, 7, 8, 9, 300, 16], rows, 2, 8, 1, 0.6, 2e-2,
                  {"prefill_rows": rows, "attn_chunk": chunk_tokens, "prefill_tc": 1})


@pytest.mark.parametrize("hq,hkv,hd", [(4, 4, 64), (4, 2, 128), (6, 2, 64), (8, 1, 64), (8, 2, 128), (6, 2, 128)])
def test_prefill_bf16_tensor_core_blocks_head_groupings(hq, hkv, hd):
    """1, 2, 3, 4 and 8 query heads per KV head at both head sizes: blocks of 128, 64, 42, 32 and 16 tokens."""
    shape = fi.ModelShape(2, hq * hd, hq, hkv, hd, 512, 1024, 500000.0)
    _prefill_case(shape, True, [70, 3, 131, 260], 256, 2, 8, 0, 0.6, 2e-2, {"prefill_tc": 1})


@pytest.mark.parametrize("hd", [64, 128])
def test_prefill_bf16_tensor_core_blocks_many_tiny_prompts(hd):
    """Dozens of prompts of one to five tokens side by side: a window of 32 rows holds many block starts, which one
    CTA serves one after the other (ring stages, buffer parities and barrier phases run on from block to block)."""
    shape = fi.ModelShape(2, 256, 8, 2, hd, 512, 2048, 500000.0)
    lens = [1, 2, 3, 1, 1, 2, 5, 1, 4, 1, 150, 2, 1, 3, 1, 1, 70, 2, 2, 1, 5, 1, 1, 3, 9, 1, 2, 1, 1, 4] * 2
    _prefill_case(shape, True, lens, 256, 1, 9, 1, 0.6, 2e-2, {"attn_chunk": 64, "prefill_tc": 1})
    _prefill_case(shape, True, lens, 64, 1, 9, 0, 0.6, 2e-2, {"prefill_tc": 1})


@pytest.mark.parametrize("hd,slack", [(64, 0), (128, 0), (64, 8), (64, 2)])
def test_prefill_bf16_tensor_core_blocks_moving_maximum(hd, slack):
    """Attention scores with a spread of several units (query projection x 8, key projection x 4), prompts of
    several tiles and token chunks: the softmax's reference maximum has to move while outputs are already
    accumulated.  `prefill_slack` 0 makes it follow the running maximum exactly, so the accumulated output is
    rescaled on most tiles; 8 is the production setting, 2 in between: all must give the oracle's result."""
    shape = fi.ModelShape(2, 4 * hd, 4, 2, hd, 512, 1024, 500000.0)
    _prefill_case(shape, True, [420, 37, 300, 150], 256, 2, 12, 0, 0.6, 2e-2,
                  {"prefill_slack": slack, "attn_chunk": 256}, sharpen=(3, 2))


def test_prefill_bf16_plain_activations_by_option():
    """Option `prefill_lo` 0: the prompt chunks' projections use the bfloat16 hi half of the activations alone.  At
    three layers this stays inside the bars of the default path (at 32 layers of the 8B shape it does not, which is
    why it is an option); the decode steps that follow use both halves again."""
    _prefill_case(SMALL_GQA, True, [8, 200, 77, 130, 1], 256, 3, 5, 0, 0.6, 2e-2, {"prefill_lo": 0})


def test_prefill_bf16_general_kernels_by_option():
    _prefill_case(SMALL_GQA, True, [33, 90, 5], 32, 2, 6, 1, 0.6, 2e-2, {"attn_simple": 1, "max_gemv_rows": 1024})


def test_prefill_without_routers_and_outputs():
    """router_w = NULL leaves mask and scores alone; logits/next_tokens may be omitted."""
    import torch
    shape, lens = fi.TINY, [12, 5]
    w = fi.make_weights(shape, 1, False)
    om = oracle_model(shape, w)
    prompts = [fi.tokens(shape, n, 1, f"p{b}") for b, n in enumerate(lens)]
    okv = oracle.OracleKV(om.shape, [20, 20])
    for b in range(2):
        oracle.prefill(om, okv, b, prompts[b], want_router_in=False)
    gkv = GpuKV(shape, [20, 20], False)
    ctx = _ctx(shape, False, 8, 20, w)
    cu = np.array([0, 12, 17], np.int32)
    ctx.prefill(torch.from_numpy(np.concatenate(prompts).astype(np.int32)).cuda(), cu, gkv.c)
    assert ctx.device_flags() == 0
    assert np.array_equal(gkv.len.cpu().numpy(), okv.len) and np.array_equal(gkv.pos.cpu().numpy(), okv.pos)
    for l in range(shape.n_layers):
        for b in range(2):
            k1, v1 = gkv.rows_host(l, b)
            ko, vo = okv.rows(l, b)
            assert np.abs(k1 - ko).max() <= 1e-4 and np.abs(v1 - vo).max() <= 1e-4


def test_prefill_argument_errors_and_short_slab():
    import torch
    from paper_2410_12513_b200 import FirstError
    shape = fi.TINY
    w = fi.make_weights(shape, 2, False)
    ctx = _ctx(shape, False, 4, 16, w)
    gkv = GpuKV(shape, [16, 6], False)
    toks = torch.zeros((64,), dtype=torch.int32, device="cuda")

    def status(cu, kv=gkv.c):
        with pytest.raises(FirstError) as e:
            ctx.prefill(toks, np.asarray(cu, np.int32), kv)
        return e.value.status

    assert status([0, 4, 4]) == -1            # empty prompt
    assert status([1, 4, 6]) == -1            # cu_seqlens[0] != 0
    assert status([0, 17, 20]) == -4          # prompt longer than max_tokens_per_seq
    assert status([0, 1, 2, 3, 4, 5]) == -4   # batch larger than max_batch
    # a slab shorter than its prompt: flagged, the tokens that fit are kept, the neighbouring slab is not touched
    guard = GpuKV(shape, [6, 16], False)
    ctx.prefill(toks, np.array([0, 8, 11], np.int32), guard.c)
    assert ctx.device_flags() == 1
    assert guard.len.cpu().numpy().tolist() == [[6, 3]] * shape.n_layers
    assert guard.pos.cpu().numpy().tolist() == [8, 3]
    for l in range(shape.n_layers):
        k1, v1 = guard.rows_host(l, 1)
        assert k1[:3].any() and not k1[3:].any() and not v1[3:].any()


def test_prefill_joins_a_running_batch():
    """Continuous batching with the one-call prompt phase: two sequences are prefilled together and decode;
    a third then joins (prefilled alone into its own slab of the same cache tensors, routed by its own prompt)
    and the three decode together.  The join must leave the running sequences' slabs bit-identical, and every
    sequence must follow the oracle run on that sequence alone."""
    import torch
    from paper_2410_12513_b200 import KVCache
    shape, seed, bf16 = SMALL_GQA, 41, True
    L = shape.n_layers
    w = fi.make_weights(shape, seed, bf16)
    om = oracle_model(shape, w)
    lens, caps = [37, 52, 20], [48, 64, 32]
    prompts = [fi.tokens(shape, n, seed, f"prompt{b}") for b, n in enumerate(lens)]
    okvs = [oracle.OracleKV(om.shape, [caps[b]]) for b in range(3)]
    pre = [oracle.prefill(om, okvs[b], 0, prompts[b]) for b in range(3)]
    target = np.array([[1, 0, 1], [1, 1, 0], [0, 1, 1]], np.uint8)
    # one router set serves all three prompts (as it would in a deployment)
    routers = np.stack([calibrate_router([pre[b]["router_in"][l] for b in range(3)], target[:, l], 0, l)[0]
                        for l in range(L)])
    gkv = GpuKV(shape, caps, bf16)
    ctx = _ctx(shape, bf16, 16, max(caps), w)
    rw = to_dev(routers, False)
    mask = torch.zeros((3, L), dtype=torch.uint8, device="cuda")
    logits = torch.empty((3, shape.vocab), dtype=torch.float32, device="cuda")

    def sub_kv(rows):
        r = torch.tensor(rows, device="cuda")
        return (KVCache(gkv.k, gkv.v, gkv.slab_off[r].contiguous(), gkv.slab_cap[r].contiguous(),
                        gkv.len[:, r].contiguous(), gkv.pos[r].contiguous()), r)

    def write_back(kvc, r):
        gkv.len[:, r] = kvc.len
        gkv.pos[r] = kvc.pos

    def first_logits(b):
        return np.asarray(pre[b]["logits"]).reshape(-1, shape.vocab)[0]

    def decode(rows, kvc, toks, n):
        for _ in range(n):
            ref = np.stack([oracle.decode_step(om, toks[i:i + 1], target[b:b + 1], okvs[b])[0] for i, b in enumerate(rows)])
            ctx.decode_step(torch.from_numpy(toks).cuda(), kvc, logits[:len(rows)])
            err, agree = logits_check(logits[:len(rows)].cpu().numpy(), ref)
            assert err.max() <= 2e-2, err.max()
            toks = oracle.argmax(ref)
        assert ctx.device_flags() == 0
        return toks

    # sequences 0 and 2 arrive first
    kv02, r02 = sub_kv([0, 2])
    m02 = torch.zeros((2, L), dtype=torch.uint8, device="cuda")
    cu = np.array([0, lens[0], lens[0] + lens[2]], np.int32)
    ctx.prefill(torch.from_numpy(np.concatenate([prompts[0], prompts[2]]).astype(np.int32)).cuda(), cu, kv02, rw,
                None, 0.5, 0, m02, None, logits[:2])
    assert np.array_equal(m02.cpu().numpy(), target[[0, 2]])
    err, _ = logits_check(logits[:2].cpu().numpy(), np.stack([first_logits(0), first_logits(2)]))
    assert err.max() <= 2e-2
    ctx.set_mask(m02)
    toks = decode([0, 2], kv02, oracle.argmax(np.stack([first_logits(0), first_logits(2)])), 2)
    write_back(kv02, r02)

    # sequence 1 joins: its prompt phase must not touch the other slabs
    before = {(l, b): gkv.rows_host(l, b) for l in range(L) for b in (0, 2)}
    kv1, r1 = sub_kv([1])
    m1 = torch.zeros((1, L), dtype=torch.uint8, device="cuda")
    ctx.prefill(torch.from_numpy(prompts[1].astype(np.int32)).cuda(), np.array([0, lens[1]], np.int32), kv1, rw, None,
                0.5, 0, m1, None, logits[:1])
    write_back(kv1, r1)
    assert np.array_equal(m1.cpu().numpy(), target[1:2])
    for (l, b), (k0, v0) in before.items():
        k1, v1 = gkv.rows_host(l, b)
        assert np.array_equal(k0, k1) and np.array_equal(v0, v1)
    tok1 = oracle.argmax(first_logits(1)[None])
    mask.copy_(torch.from_numpy(target))
    ctx.set_mask(mask)
    toks3 = np.array([toks[0], tok1[0], toks[1]], np.int32)
    decode([0, 1, 2], gkv.c, toks3, 3)
    want_len = np.stack([okvs[b].len[:, 0] for b in range(3)], 1)
    assert np.array_equal(gkv.len.cpu().numpy(), want_len)
    assert gkv.pos.cpu().numpy().tolist() == [int(okvs[b].pos[0]) for b in range(3)]
