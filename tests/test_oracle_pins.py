"""Pins of the host oracle against things other than itself: a library model, closed
forms, hand-worked values, invariants of the paper's recursions, brute force."""
import math
from pathlib import Path

import numpy as np
import pytest

import first_inputs as fi
import oracle

GOLDEN = Path(__file__).parent / "golden"


def make(shape, seed=0, bf16=False):
    w = fi.make_weights(shape, seed, bf16)
    return oracle.OracleModel(oracle.Shape(**shape.asdict()), w), w


@pytest.fixture(scope="module")
def tiny():
    return make(fi.TINY)


@pytest.fixture(scope="module")
def tiny_gqa():
    return make(fi.TINY_GQA, seed=3)


# ---------------------------------------------------------------- P1: library special case
def _hf_model(shape, w):
    torch = pytest.importorskip("torch")
    tr = pytest.importorskip("transformers")
    cfg = tr.LlamaConfig(vocab_size=shape.vocab, hidden_size=shape.d_model, intermediate_size=shape.ffn_dim,
                         num_hidden_layers=shape.n_layers, num_attention_heads=shape.n_q_heads,
                         num_key_value_heads=shape.n_kv_heads, head_dim=shape.head_dim,
                         rms_norm_eps=shape.rms_eps, rope_theta=shape.rope_base, attention_bias=False,
                         mlp_bias=False, tie_word_embeddings=False, max_position_embeddings=512)
    cfg._attn_implementation = "eager"
    hf = tr.LlamaForCausalLM(cfg).to(torch.float32).eval()
    sd = {"model.embed_tokens.weight": w["embed"], "lm_head.weight": w["lm_head"], "model.norm.weight": w["final_norm"]}
    names = {"attn_norm": "input_layernorm", "ffn_norm": "post_attention_layernorm", "wq": "self_attn.q_proj",
             "wk": "self_attn.k_proj", "wv": "self_attn.v_proj", "wo": "self_attn.o_proj", "wg": "mlp.gate_proj",
             "wu": "mlp.up_proj", "wd": "mlp.down_proj"}
    for l in range(shape.n_layers):
        for k, n in names.items():
            sd[f"model.layers.{l}.{n}.weight"] = w[k][l]
    missing, unexpected = hf.load_state_dict({k: torch.from_numpy(np.array(v)) for k, v in sd.items()}, strict=False)
    assert not unexpected and all("rotary" in m or "inv_freq" in m for m in missing), (missing, unexpected)
    return hf


@pytest.mark.parametrize("which", ["tiny", "tiny_gqa"])
def test_all_keep_equals_huggingface_llama(which, request):
    """All-keep mask = plain decoder (Eq. 1); the plain decoder = the public LLaMA block.
    Pins RoPE pairing, GQA head mapping, RMSNorm placement, SwiGLU, causal softmax."""
    import torch
    model, w = request.getfixturevalue(which)
    shape = fi.TINY if which == "tiny" else fi.TINY_GQA
    hf = _hf_model(shape, w)
    toks = fi.tokens(shape, 24, 11)
    with torch.no_grad():
        ref = hf(torch.from_numpy(toks.astype(np.int64))[None]).logits[0].numpy()
    got = oracle.forward_full(model, toks, logits_from=0)["logits"]
    assert np.abs(got - ref).max() <= 1e-4 * max(1.0, np.abs(ref).max())
    # KV-cached decode with an all-keep mask continues the same sequence
    n = 16
    kv = oracle.OracleKV(model.shape, [24])
    oracle.prefill(model, kv, 0, toks[:n])
    keep = np.ones((1, shape.n_layers), dtype=np.uint8)
    for j in range(n, 24):
        lg = oracle.decode_step(model, toks[j:j + 1], keep, kv)
        assert np.abs(lg[0] - ref[j]).max() <= 1e-4 * max(1.0, np.abs(ref).max())


# ---------------------------------------------------------------- P6: router closed forms
def _golden_router_rows():
    rows = []
    for line in (GOLDEN / "router_hand_examples.txt").read_text().splitlines():
        if not line.strip() or line.startswith("#"):
            continue
        name, z, r0, r1 = [c.strip() for c in line.split("|")]
        rows.append((name, [float(t) for t in z.split()], float(r0), float(r1)))
    return rows


@pytest.mark.parametrize("name,zs,rho0,rho1", _golden_router_rows())
def test_router_hand_examples(name, zs, rho0, rho1):
    """Tokens are built so that w.h_j equals the tabulated score: h_j = z_j * e_0, w = ln3 * e_0."""
    D = 8
    hidden = np.zeros((len(zs), D), dtype=np.float32)
    hidden[:, 0] = np.array(zs, dtype=np.float32)
    hidden[:, 1:] = fi.normal((len(zs), D - 1), 1.0, 5, name)  # ignored: w is zero there
    w = np.zeros(D, dtype=np.float32)
    w[0] = math.log(3.0)
    for mode, want in ((0, rho0), (1, rho1)):
        rho, keep = oracle.route(hidden, w, None, 0.5, mode)
        assert abs(rho - want) < 2e-7, (mode, rho, want)
        assert keep == (1 if want >= 0.5 else 0)


def test_router_tie_keeps_and_modes_agree_on_one_token():
    D = 64
    h = fi.normal((7, D), 1.0, 1, "h")
    rho, keep = oracle.route(h, np.zeros(D, np.float32), None, 0.5, 0)
    assert rho == 0.5 and keep == 1  # equality passes the layer
    rho, keep = oracle.route(h, np.zeros(D, np.float32), None, 0.5, 1)
    assert rho == 0.5 and keep == 1
    w = fi.normal((D,), 0.3, 1, "w")
    a = oracle.route(h[:1], w, None, 0.5, 0)
    b = oracle.route(h[:1], w, None, 0.5, 1)
    assert a == b


def test_router_matches_numpy_and_is_permutation_invariant():
    D, n = 96, 37
    h = fi.normal((n, D), 1.0, 2, "h")
    w = fi.normal((D,), 0.2, 2, "w")
    z = h.astype(np.float64) @ w.astype(np.float64)
    sig = lambda t: 1.0 / (1.0 + np.exp(-t))
    rho0, _ = oracle.route(h, w, None, 0.5, 0)
    rho1, _ = oracle.route(h, w, None, 0.5, 1)
    assert abs(rho0 - sig(z).mean()) < 1e-12
    assert abs(rho1 - sig(w.astype(np.float64) @ h.astype(np.float64).mean(0))) < 1e-12  # pooled the other way round
    perm = np.random.default_rng(0).permutation(n)
    assert abs(oracle.route(h[perm], w, None, 0.5, 0)[0] - rho0) < 1e-12
    # bias shifts every token score
    rho0b, _ = oracle.route(h, w, 0.25, 0.5, 0)
    assert abs(rho0b - sig(z + 0.25).mean()) < 1e-12
    # other thresholds compare in probability space
    assert oracle.route(h, w, None, rho0 + 1e-9, 0)[1] == 0 and oracle.route(h, w, None, rho0 - 1e-9, 0)[1] == 1


def test_router_parameter_fraction_printed_in_paper():
    """Sec. "Computational overhead of Routers" prints 0.0027 % and 0.0016 % for the two
    models; one bias-free D-vector per layer gives L*D / params = 0.0016 % for the 8B
    shape and 0.0027 % for the 3B shape (the text attaches the figures the other way round)."""
    s8, s3 = fi.LLAMA_8B, fi.LLAMA_3B
    p8 = s8.n_layers * (s8.layer_params() + 2 * s8.d_model) + 2 * s8.vocab * s8.d_model + s8.d_model
    p3 = s3.n_layers * (s3.layer_params() + 2 * s3.d_model) + s3.vocab * s3.d_model + s3.d_model  # tied embeddings
    assert round(p8 / 1e9, 2) == 8.03 and round(p3 / 1e9, 2) == 3.21
    router8 = s8.n_layers * s8.d_model  # the shape the oracle's router takes: w[D], no bias
    router3 = s3.n_layers * s3.d_model
    assert f"{100 * router8 / p8:.4f}" == "0.0016"
    assert f"{100 * router3 / p3:.4f}" == "0.0027"


# ---------------------------------------------------------------- P3: all-skip closed form
def test_all_skip_is_lm_head_of_normed_embedding(tiny):
    model, w = tiny
    s = fi.TINY
    toks = fi.tokens(s, 3, 4)
    kv = oracle.OracleKV(model.shape, [4, 4, 4])
    logits = oracle.decode_step(model, toks, np.zeros((3, s.n_layers), np.uint8), kv)
    e = w["embed"][toks].astype(np.float64)
    xn = e / np.sqrt((e * e).mean(-1, keepdims=True) + s.rms_eps) * w["final_norm"].astype(np.float64)
    ref = xn @ w["lm_head"].astype(np.float64).T
    assert np.abs(logits - ref).max() < 1e-5
    assert (kv.len == 0).all() and all((k == 0).all() for k in kv.k)


# ---------------------------------------------------------------- P2 / P4: skip = identity, cache untouched
def test_skipped_layer_is_identity_and_leaves_cache_untouched(tiny):
    model, _ = tiny
    s = fi.TINY
    B, n = 3, 9
    prompts = [fi.tokens(s, n, 20 + b) for b in range(B)]

    def run(mask):
        kv = oracle.OracleKV(model.shape, [n + 4] * B)
        for b in range(B):
            oracle.prefill(model, kv, b, prompts[b])
        for l in range(s.n_layers):  # a recognisable non-zero fill beyond each prompt, so a stray write shows
            for b in range(B):
                kr, vr = kv.rows(l, b)
                kr[n:] = 777.0 + l
                vr[n:] = -777.0 - l
        before = [(k.copy(), v.copy()) for k, v in zip(kv.k, kv.v)]
        tok = np.array([5, 6, 7], np.int32)
        out = []
        for t in range(3):
            lg, li = oracle.decode_step(model, tok, mask, kv, want_layer_inputs=True)
            out.append((lg, li))
            tok = oracle.argmax(lg)
        return kv, before, out

    keep_all = np.ones((B, s.n_layers), np.uint8)
    mask = keep_all.copy()
    mask[1, 2] = 0
    mask[1, 1] = 0
    kv_a, _, out_a = run(keep_all)
    kv_m, before, out_m = run(mask)
    for t in range(3):
        lg_a, li_a = out_a[t]
        lg_m, li_m = out_m[t]
        # rows 0 and 2 do not know that row 1 skipped anything: bit-identical
        assert np.array_equal(lg_a[[0, 2]], lg_m[[0, 2]])
        # row 1: residual entering layer 2 equals the one entering layer 1, and layer 3's input too
        assert np.array_equal(li_m[1, 1], li_m[2, 1]) and np.array_equal(li_m[2, 1], li_m[3, 1])
        assert not np.array_equal(li_m[0, 1], li_m[1, 1])
        assert not np.array_equal(lg_a[1], lg_m[1])
    for l in (1, 2):
        kb, vb = before[l]
        o = int(kv_m.slab_off[1])
        assert np.array_equal(kv_m.k[l][o:o + n + 4], kb[o:o + n + 4])
        assert np.array_equal(kv_m.v[l][o:o + n + 4], vb[o:o + n + 4])
        assert kv_m.len[l, 1] == n and kv_m.len[l, 0] == n + 3
    assert (kv_m.pos == n + 3).all()


# ---------------------------------------------------------------- P5: cached decode = recompute
@pytest.mark.parametrize("which,mask_row", [("tiny", [1, 0, 1, 1]), ("tiny", [1, 0, 0, 1]), ("tiny", [0, 0, 0, 0]),
                                            ("tiny_gqa", [1, 0, 1]), ("tiny_gqa", [1, 1, 1])])
def test_cached_decode_matches_full_recompute(which, mask_row, request):
    model, _ = request.getfixturevalue(which)
    s = model.shape
    n, S = 10, 5
    toks = fi.tokens(s.vocab, n + S, 31)
    kv = oracle.OracleKV(s, [n + S])
    oracle.prefill(model, kv, 0, toks[:n])
    mask = np.array([mask_row], np.uint8)
    cached = [oracle.decode_step(model, toks[n + t:n + t + 1], mask, kv)[0] for t in range(S)]
    full = oracle.forward_full(model, toks, n_prompt=n, keep=mask[0], logits_from=n)["logits"]
    assert np.abs(np.stack(cached) - full).max() <= 1e-5
    # prompt positions ran every layer even where decode skips: the prefill logits do not depend on the mask
    a = oracle.forward_full(model, toks, n_prompt=n, keep=mask[0], logits_from=0)["logits"][:n]
    b = oracle.forward_full(model, toks[:n], logits_from=0)["logits"]
    assert np.array_equal(a, b)


# ---------------------------------------------------------------- P8: batch independence
def test_batch_permutation_and_single_row_equivalence(tiny):
    model, _ = tiny
    s = fi.TINY
    B = 4
    lens = [5, 9, 7, 12]
    prompts = [fi.tokens(s, lens[b], 40 + b) for b in range(B)]
    mask = fi.mask_bernoulli(B, s.n_layers, 0.6, 9)
    mask[2] = 0

    def run(order):
        kv = oracle.OracleKV(model.shape, [lens[b] + 2 for b in order])
        for i, b in enumerate(order):
            oracle.prefill(model, kv, i, prompts[b])
        tok = np.array([100 + b for b in order], np.int32)
        return oracle.decode_step(model, tok, mask[order], kv)

    base = run([0, 1, 2, 3])
    perm = [2, 0, 3, 1]
    assert np.array_equal(run(perm), base[perm])
    for b in range(B):
        assert np.array_equal(run([b])[0], base[b])


# ---------------------------------------------------------------- greedy rule (lowest index among equal maxima)
def test_argmax_takes_the_lowest_index_among_equal_maxima():
    # hand cases: the expected index is written out, not computed
    cases = [
        ([1.0, 3.0, 3.0, 2.0], 1),                       # tie between 1 and 2 -> 1
        ([5.0, 5.0, 5.0], 0),                            # all equal -> 0
        ([0.0, -1.0, 2.5], 2),                           # maximum at the last index
        ([-np.inf, -np.inf, -3.0, -np.inf], 2),          # -inf entries never win over a finite value
        ([-np.inf, -np.inf], 0),                         # all -inf: still the lowest index
        ([-0.0, 0.0], 0),                                # signed zeros compare equal
        ([7.0], 0),
        ([-2.0, -1.0, -1.0, -3.0, -1.0], 1),
    ]
    for row, want in cases:
        assert oracle.argmax(np.array([row], np.float32)).tolist() == [want], row
    # a tie planted far apart in a long row, and at the two ends
    v = np.full(128256, -1.0, np.float32)
    v[[100000, 17, 128255]] = 4.0
    assert oracle.argmax(v[None])[0] == 17
    v[:] = 0.0
    v[128255] = 1e-30
    assert oracle.argmax(v[None])[0] == 128255
    # random rows without and with many ties: numpy's argmax has the same first-occurrence rule
    rng = np.random.default_rng(5)
    a = rng.standard_normal((64, 1003)).astype(np.float32)
    assert np.array_equal(oracle.argmax(a), a.argmax(-1))
    q = rng.integers(0, 4, (64, 1003)).astype(np.float32)
    assert np.array_equal(oracle.argmax(q), q.argmax(-1))
    # a mistake of the ">=" kind would return the LAST maximum: make sure that is told apart
    assert oracle.argmax(q)[0] != len(q[0]) - 1 - q[0][::-1].argmax()


def test_plan_lists_active_rows_in_order():
    mask = np.array([[1, 0, 1], [0, 0, 1], [1, 0, 0], [1, 0, 1]], np.uint8)
    idx, cnt, slot = oracle.plan(mask)
    assert cnt.tolist() == [3, 0, 3]
    assert idx[0].tolist() == [0, 2, 3, -1] and idx[1].tolist() == [-1] * 4 and idx[2].tolist() == [0, 1, 3, -1]
    assert slot[0].tolist() == [0, -1, 1, 2] and slot[2].tolist() == [0, 1, -1, 2]


def test_capacity_and_argument_errors(tiny):
    model, _ = tiny
    s = fi.TINY
    kv = oracle.OracleKV(model.shape, [1])
    keep = np.ones((1, s.n_layers), np.uint8)
    oracle.decode_step(model, np.array([1], np.int32), keep, kv)
    with pytest.raises(RuntimeError):
        oracle.decode_step(model, np.array([1], np.int32), keep, kv)  # slab full
    with pytest.raises(RuntimeError):
        oracle.decode_step(model, np.array([s.vocab], np.int32), keep, oracle.OracleKV(model.shape, [2]))
    bad = keep.copy()
    bad[0, 0] = 2
    with pytest.raises(RuntimeError):
        oracle.decode_step(model, np.array([1], np.int32), bad, oracle.OracleKV(model.shape, [2]))


def test_bf16_weights_are_widened_exactly():
    """The same bfloat16-rounded values, given once as bit patterns and once widened to
    float32, give identical results."""
    s = fi.TINY_GQA
    wb = fi.make_weights(s, 8, True)
    wf = {k: ([fi.bf16_bits_to_f32(a) if a.dtype == np.uint16 else a for a in v] if isinstance(v, list)
              else (fi.bf16_bits_to_f32(v) if v.dtype == np.uint16 else v)) for k, v in wb.items()}
    mb = oracle.OracleModel(oracle.Shape(**s.asdict()), wb, kv_bf16=False)
    mf = oracle.OracleModel(oracle.Shape(**s.asdict()), wf, kv_bf16=False)
    assert mb.weight_dtype == 1 and mf.weight_dtype == 0
    toks = fi.tokens(s, 6, 2)
    assert np.array_equal(oracle.forward_full(mb, toks)["logits"], oracle.forward_full(mf, toks)["logits"])


def test_bf16_cache_storage_rounds_once_like_torch():
    """kv_dtype = bfloat16: keys/values are rounded to bfloat16 when they enter the cache (nearest,
    ties to even -- checked against torch's conversion) and attention reads the rounded values;
    nothing else changes.  Layer 0 sees identical inputs in both modes, so its stored keys are the
    rounded float32-mode keys exactly."""
    torch = pytest.importorskip("torch")
    s = fi.TINY_GQA
    wb = fi.make_weights(s, 8, True)
    m32 = oracle.OracleModel(oracle.Shape(**s.asdict()), wb, kv_bf16=False)
    m16 = oracle.OracleModel(oracle.Shape(**s.asdict()), wb)  # default: cache format follows the weights
    assert m32.kv_dtype == 0 and m16.kv_dtype == 1
    toks = fi.tokens(s, 12, 3)
    a = oracle.forward_full(m32, toks, want_kv=True, logits_from=0)
    b = oracle.forward_full(m16, toks, want_kv=True, logits_from=0)
    rnd = lambda x: torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(b["k"][0], rnd(a["k"][0])) and np.array_equal(b["v"][0], rnd(a["v"][0]))
    for l in range(s.n_layers):
        assert np.array_equal(b["k"][l], rnd(b["k"][l])) and np.array_equal(b["v"][l], rnd(b["v"][l]))
    d = np.abs(a["logits"] - b["logits"]).max() / (a["logits"].max() - a["logits"].min())
    assert 0 < d < 2e-2
    # cached decode in bf16-cache mode still equals the cache-free recompute in the same mode
    kv = oracle.OracleKV(m16.shape, [12])
    oracle.prefill(m16, kv, 0, toks[:8])
    keep = np.array([[1, 0, 1]], np.uint8)
    cached = np.stack([oracle.decode_step(m16, toks[8 + t:9 + t], keep, kv)[0] for t in range(4)])
    full = oracle.forward_full(m16, toks, n_prompt=8, keep=keep[0], logits_from=8)["logits"]
    assert np.abs(cached - full).max() <= 1e-5
    # ties round to even: 1 + 2^-8 is exactly between two bfloat16 values
    tie = np.array([[1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8]], np.float32)
    assert rnd(tie).tolist() == [[1.0, 1.015625]]


# ------------------------------------------------------------------ sampling (temperature + top-k)
def test_sampling_hand_worked_two_candidates():
    """logits (1,3,2,0), k=2: candidates are tokens 1 then 2; at T=1 the first has probability
    1/(1+e^-1) = 0.731059, at T=0.5 it has 1/(1+e^-2) = 0.880797 (worked by hand)."""
    z = np.array([1.0, 3.0, 2.0, 0.0], np.float32)
    t, cand, prob = oracle.sample_topk(z, 2, 1.0, 0.70)
    assert list(cand) == [1, 2] and t == 1
    assert abs(prob[0] - 0.7310585786) < 1e-9 and abs(prob.sum() - 1) < 1e-12
    assert oracle.sample_topk(z, 2, 1.0, 0.74)[0] == 2
    _, _, p = oracle.sample_topk(z, 2, 0.5, 0.0)
    assert abs(p[0] - 0.8807970780) < 1e-9          # a lower temperature sharpens, not flattens
    assert oracle.sample_topk(z, 2, 0.5, 0.87)[0] == 1 and oracle.sample_topk(z, 2, 0.5, 0.89)[0] == 2


def test_sampling_reduces_to_greedy_and_to_plain_softmax_sampling():
    g = np.random.default_rng(5)
    z = g.normal(0, 2, 500).astype(np.float32)
    for u in (0.0, 0.3, 0.999):
        assert oracle.sample_topk(z, 1, 0.8, u)[0] == int(z.argmax())
        assert oracle.sample_topk(z, 10, 0.0, u)[0] == int(z.argmax())
    # k = n: inverse-CDF sampling from softmax(z/T) in descending order, by library routines
    from scipy.special import softmax
    order = np.argsort(-z.astype(np.float64), kind="stable")
    cdf = np.cumsum(softmax(z.astype(np.float64)[order] / 0.8))
    for u in g.random(200):
        j = int(np.searchsorted(cdf, u, side="right"))
        if abs(cdf[min(j, 499)] - u) < 1e-9 or (j and abs(cdf[j - 1] - u) < 1e-9):
            continue
        assert oracle.sample_topk(z, 500, 0.8, float(u))[0] == int(order[min(j, 499)])
    _, cand, prob = oracle.sample_topk(z, 10, 0.8, 0.5)
    assert list(cand) == list(order[:10])
    assert np.allclose(prob, softmax(z.astype(np.float64)[order[:10]] / 0.8), atol=1e-12)


def test_sampling_frequencies_and_ties():
    """Over an even grid of draws each candidate is chosen in proportion to its probability;
    equal logits enter in index order and share the mass equally; the rest is never chosen."""
    z = np.array([0.5, 2.0, 2.0, -1.0, 2.0, 1.5], np.float32)
    _, cand, prob = oracle.sample_topk(z, 4, 0.8, 0.0)
    assert list(cand) == [1, 2, 4, 5]
    assert prob[0] == prob[1] == prob[2] and abs(prob[3] / prob[0] - np.exp(-0.5 / 0.8)) < 1e-12
    n = 4000
    counts = np.zeros(6)
    for i in range(n):
        counts[oracle.sample_topk(z, 4, 0.8, (i + 0.5) / n)[0]] += 1
    assert counts[0] == 0 and counts[3] == 0
    assert np.abs(counts[cand] / n - prob).max() <= 1.0 / n + 1e-12


def test_sampling_rejects_bad_arguments():
    z = np.zeros(4, np.float32)
    for k, T, u in ((0, 1.0, 0.5), (5, 1.0, 0.5), (2, -1.0, 0.5), (2, 1.0, 1.0), (2, 1.0, -0.1)):
        with pytest.raises(RuntimeError):
            oracle.sample_topk(z, k, T, u)


def _sampling_rows():
    rows = []
    for line in (GOLDEN / "sampling_hand_examples.txt").read_text().splitlines():
        if not line.strip() or line.startswith("#"):
            continue
        name, logits, k, T, cands, p0 = [c.strip() for c in line.split("|")]
        rows.append((name, [float(x) for x in logits.split()], int(k), float(T), [int(x) for x in cands.split()], float(p0)))
    return rows


@pytest.mark.parametrize("name,logits,k,T,cands,p0", _sampling_rows())
def test_sampling_hand_examples(name, logits, k, T, cands, p0):
    _, cand, prob = oracle.sample_topk(np.array(logits, np.float32), k, T, 0.0)
    assert list(cand) == cands
    assert abs(prob[0] - p0) < 1e-6 and abs(prob.sum() - 1.0) < 1e-12
