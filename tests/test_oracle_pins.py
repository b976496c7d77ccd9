"""Pins of the CPU oracle against things other than itself: library decoders of the same
architectures, torch's elementary routines, closed forms, invariants and brute force.

All CPU.  A plausible slip in the oracle (a dropped term, a wrong sign, index or pairing
convention, a transposed operand) fails at least one test here.
"""
import math
import os

import numpy as np
import pytest
import torch

import synth

torch.set_num_threads(max(1, min(8, os.cpu_count() or 1)))


# --------------------------------------------------------------------------------------------
# helpers
# --------------------------------------------------------------------------------------------

def _small_desc(**kw):
    d = dict(n_layers=2, d_model=64, n_q_heads=4, n_kv_heads=2, head_dim=16, d_ff=96, vocab=128,
             rope_theta=1e6, rms_eps=1e-6, qk_norm=0, qkv_bias=0, tied_embed=1)
    d.update(kw)
    return d


def _weights(desc, seed=7, std=0.3, gains=True):
    w = synth.make_weights(desc, seed=seed, std=std)
    if gains:
        synth.perturb_gains(w, seed=seed)
    return w


def _load_into_hf(hf, desc, w):
    sd = {}
    f = lambda t: t.to(torch.float64)
    sd["model.embed_tokens.weight"] = f(w["embed"])
    sd["model.norm.weight"] = f(w["final_norm"])
    sd["lm_head.weight"] = f(w["embed"] if desc["tied_embed"] else w["lm_head"])
    for l in range(desc["n_layers"]):
        p = f"model.layers.{l}."
        sd[p + "input_layernorm.weight"] = f(w["ln1"][l])
        sd[p + "post_attention_layernorm.weight"] = f(w["ln2"][l])
        for hn, on in (("q_proj", "wq"), ("k_proj", "wk"), ("v_proj", "wv"), ("o_proj", "wo")):
            sd[p + f"self_attn.{hn}.weight"] = f(w[on][l])
        if desc["qkv_bias"]:
            for hn, on in (("q_proj", "bq"), ("k_proj", "bk"), ("v_proj", "bv")):
                sd[p + f"self_attn.{hn}.bias"] = f(w[on][l])
        if desc["qk_norm"]:
            sd[p + "self_attn.q_norm.weight"] = f(w["q_norm"][l])
            sd[p + "self_attn.k_norm.weight"] = f(w["k_norm"][l])
        for hn, on in (("gate_proj", "w_gate"), ("up_proj", "w_up"), ("down_proj", "w_down")):
            sd[p + f"mlp.{hn}.weight"] = f(w[on][l])
    missing, unexpected = hf.load_state_dict(sd, strict=False)
    assert not unexpected, unexpected
    assert all("rotary" in m or "inv_freq" in m for m in missing), missing


def _hf_model(kind, desc):
    common = dict(vocab_size=desc["vocab"], hidden_size=desc["d_model"],
                  intermediate_size=desc["d_ff"], num_hidden_layers=desc["n_layers"],
                  num_attention_heads=desc["n_q_heads"], num_key_value_heads=desc["n_kv_heads"],
                  head_dim=desc["head_dim"], rms_norm_eps=desc["rms_eps"],
                  tie_word_embeddings=bool(desc["tied_embed"]), max_position_embeddings=512,
                  hidden_act="silu", attn_implementation="eager")
    rope = dict(rope_theta=desc["rope_theta"])
    if kind == "qwen3":
        from transformers import Qwen3Config, Qwen3ForCausalLM
        cfg = Qwen3Config(attention_bias=False, **common, **rope)
        m = Qwen3ForCausalLM(cfg)
    elif kind == "llama":
        from transformers import LlamaConfig, LlamaForCausalLM
        cfg = LlamaConfig(attention_bias=False, mlp_bias=False, **common, **rope)
        m = LlamaForCausalLM(cfg)
    else:
        from transformers import Qwen2Config, Qwen2ForCausalLM
        cfg = Qwen2Config(**common, **rope)
        m = Qwen2ForCausalLM(cfg)
    # the rope base must really be the one asked for, whatever the config class calls it
    inv = m.model.rotary_emb.inv_freq
    want = desc["rope_theta"] ** (-torch.arange(0, desc["head_dim"], 2, dtype=torch.float64)
                                   / desc["head_dim"])
    assert torch.allclose(inv.double(), want, rtol=1e-5), "library rope base differs from desc"
    return m.double().eval()


# --------------------------------------------------------------------------------------------
# whole decoder against library decoders of the same architecture
# --------------------------------------------------------------------------------------------

@pytest.mark.parametrize("kind,over", [
    ("qwen3", dict(qk_norm=1, tied_embed=1, rope_theta=1e6, rms_eps=1e-6)),
    ("llama", dict(qk_norm=0, tied_embed=0, rope_theta=5e5, rms_eps=1e-5)),
    ("qwen2", dict(qk_norm=0, qkv_bias=1, tied_embed=0, rope_theta=1e4, n_kv_heads=1)),
])
def test_decoder_matches_library_decoder(oracle, kind, over):
    desc = _small_desc(**over)
    w = _weights(desc)
    hf = _hf_model(kind, desc)
    _load_into_hf(hf, desc, w)
    toks = synth.token_ids(11, 0, 37, desc["vocab"]).tolist()
    with torch.no_grad():
        ref = hf(torch.tensor([toks])).logits[0].numpy()          # [T, V], row t = after token t
    m = oracle.Model(desc, w)
    cache = m.new_cache(64)
    for t, tok in enumerate(toks):
        got = m.decode_step(cache, tok)
        # library rope angles are fp32, hence 1e-5 rather than 1e-12
        np.testing.assert_allclose(got, ref[t], rtol=0, atol=2e-5 * max(1.0, np.abs(ref[t]).max()))
    assert len(cache) == len(toks)
    # a deliberate slip must be visible at this tolerance: compare against the wrong row
    assert np.abs(got - ref[-2]).max() > 1e-2


def test_prefill_equals_stepwise_decode_and_last_row(oracle):
    desc = _small_desc(qk_norm=1)
    w = _weights(desc)
    m = oracle.Model(desc, w)
    toks = synth.token_ids(3, 1, 21, desc["vocab"]).tolist()
    c1 = m.new_cache(32)
    last = m.prefill(c1, toks)
    c2 = m.new_cache(32)
    for tok in toks:
        step = m.decode_step(c2, tok)
    np.testing.assert_array_equal(last, step)
    hf = _hf_model("qwen3", desc)
    _load_into_hf(hf, desc, w)
    with torch.no_grad():
        ref = hf(torch.tensor([toks])).logits[0, -1].numpy()
    np.testing.assert_allclose(last, ref, atol=2e-5 * np.abs(ref).max())


def test_zero_block_weights_reduce_to_embedding_readout(oracle):
    """With W_o = W_down = 0 every layer is the identity on x, so
    logits = E . (g_f * E[t] / rms(E[t])) -- a closed form with no attention in it."""
    desc = _small_desc()
    w = _weights(desc)
    for l in range(desc["n_layers"]):
        w["wo"][l] = torch.zeros_like(w["wo"][l])
        w["w_down"][l] = torch.zeros_like(w["w_down"][l])
    m = oracle.Model(desc, w)
    cache = m.new_cache(8)
    E = w["embed"].double().numpy()
    g = w["final_norm"].double().numpy()
    for tok in (5, 77, 0):
        got, trace = m.decode_step(cache, tok, want_trace=True)
        x = E[tok]
        want = E @ (x / math.sqrt((x * x).mean() + desc["rms_eps"]) * g)
        np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-12)
        for l in range(desc["n_layers"] + 1):
            np.testing.assert_array_equal(trace[l], x)


# --------------------------------------------------------------------------------------------
# elementary pieces against library routines and closed forms
# --------------------------------------------------------------------------------------------

def test_softmax(oracle):
    rng = np.random.default_rng(0)
    s = rng.normal(size=257) * 5
    p = oracle.softmax(s)
    np.testing.assert_allclose(p, torch.softmax(torch.from_numpy(s), 0).numpy(), rtol=1e-13)
    assert abs(p.sum() - 1) < 1e-12
    np.testing.assert_allclose(oracle.softmax(s + 123.0), p, rtol=1e-10)
    np.testing.assert_allclose(oracle.softmax(np.full(9, -3.0)), np.full(9, 1 / 9), rtol=1e-15)
    big = np.array([1000.0, 1000.0, -1000.0])
    np.testing.assert_allclose(oracle.softmax(big), [0.5, 0.5, 0.0], atol=1e-300)


def test_rmsnorm(oracle):
    rng = np.random.default_rng(1)
    x = rng.normal(size=96) * 3
    g = (1 + 0.2 * torch.randn(96, generator=torch.Generator().manual_seed(2))).to(torch.bfloat16)
    got = oracle.rmsnorm(x, g, 1e-6)
    want = torch.nn.functional.rms_norm(torch.from_numpy(x), (96,), g.double(), 1e-6).numpy()
    np.testing.assert_allclose(got, want, rtol=1e-13)
    ones = torch.ones(96, dtype=torch.bfloat16)
    y = oracle.rmsnorm(x, ones, 0.0)
    assert abs(math.sqrt((y * y).mean()) - 1) < 1e-13
    np.testing.assert_allclose(oracle.rmsnorm(7.5 * x, ones, 0.0), y, rtol=1e-13)
    # eps sits inside the square root: x = 0 gives 0, tiny x is damped by eps
    tiny = np.full(4, 1e-4)
    np.testing.assert_allclose(oracle.rmsnorm(tiny, torch.ones(4, dtype=torch.bfloat16), 1e-6),
                               tiny / math.sqrt(1e-8 + 1e-6), rtol=1e-13)


def test_silu_and_matvec(oracle):
    for u in (-20.0, -1.0, 0.0, 0.5, 3.0, 30.0):
        want = torch.nn.functional.silu(torch.tensor(u, dtype=torch.float64)).item()
        assert abs(oracle.silu(u) - want) <= 1e-15 * max(1, abs(want))
    assert oracle.silu(0.0) == 0.0
    assert abs(oracle.silu(40.0) - 40.0) < 1e-12
    g = torch.Generator().manual_seed(3)
    W = torch.randn(13, 29, generator=g).to(torch.bfloat16)
    b = torch.randn(13, generator=g).to(torch.bfloat16)
    x = np.random.default_rng(4).normal(size=29)
    np.testing.assert_allclose(oracle.matvec(W, x, b), W.double().numpy() @ x + b.double().numpy(),
                               rtol=1e-13)
    eye = torch.eye(8, dtype=torch.bfloat16)
    np.testing.assert_array_equal(oracle.matvec(eye, x[:8]), x[:8])
    # a transposed operand would break a non-square matrix with one hot entry
    W1 = torch.zeros(3, 5, dtype=torch.bfloat16); W1[2, 4] = 1
    np.testing.assert_array_equal(oracle.matvec(W1, np.arange(5.0)), [0, 0, 4.0])


def test_rope_closed_forms_and_invariants(oracle):
    # head_dim 2: one pair, frequency theta^0 = 1 -> plain rotation by `pos` radians
    v = oracle.rope(np.array([1.0, 0.0]), 3, 10000.0)
    np.testing.assert_allclose(v, [math.cos(3), math.sin(3)], rtol=1e-15)
    # head_dim 4, theta 1e4: pairs (0,2) at frequency 1 and (1,3) at frequency 1e4^(-1/2) = 0.01
    v = oracle.rope(np.array([1.0, 2.0, 0.0, 0.0]), 50, 10000.0)
    np.testing.assert_allclose(v, [math.cos(50), 2 * math.cos(0.5), math.sin(50), 2 * math.sin(0.5)],
                               rtol=1e-13)
    rng = np.random.default_rng(5)
    q, k = rng.normal(size=64), rng.normal(size=64)
    np.testing.assert_array_equal(oracle.rope(q, 0, 1e6), q)
    for pos in (1, 17, 4097, 16383):
        assert abs(np.linalg.norm(oracle.rope(q, pos, 1e6)) - np.linalg.norm(q)) < 1e-12
    # scores depend on the distance between positions only
    base = oracle.rope(q, 40, 1e6) @ oracle.rope(k, 33, 1e6)
    for shift in (1, 100, 5000):
        other = oracle.rope(q, 40 + shift, 1e6) @ oracle.rope(k, 33 + shift, 1e6)
        assert abs(base - other) < 1e-9
    assert abs(base - oracle.rope(q, 41, 1e6) @ oracle.rope(k, 33, 1e6)) > 1e-4
    # direction of rotation: library convention x*cos + rotate_half(x)*sin, rotate_half = (-x2, x1)
    pos, theta, hd = 9, 1e4, 8
    inv = theta ** (-np.arange(0, hd, 2) / hd)
    ang = np.concatenate([pos * inv, pos * inv])
    x = rng.normal(size=hd)
    rot_half = np.concatenate([-x[hd // 2:], x[:hd // 2]])
    np.testing.assert_allclose(oracle.rope(x, pos, theta), x * np.cos(ang) + rot_half * np.sin(ang),
                               rtol=1e-13, atol=1e-15)


def _filled_cache(oracle, desc, n_ctx, seed=9, page_size=0, n_pool_pages=0, block_table=None):
    w = synth.make_weights(desc, seed=1)
    m = oracle.Model(desc, w)
    cache = m.new_cache(max(n_ctx, 1), page_size, n_pool_pages, block_table)
    ks, vs = [], []
    for l in range(desc["n_layers"]):
        k, v = synth.synthetic_kv(seed, 0, l, n_ctx, desc["n_kv_heads"], desc["head_dim"])
        cache.load_bf16(l, k, v)
        ks.append(k.double()); vs.append(v.double())
    cache.set_len(n_ctx)
    return m, cache, ks, vs


@pytest.mark.parametrize("hq,hkv", [(4, 4), (4, 2), (8, 1), (6, 2)])
def test_attention_matches_library_attention(oracle, hq, hkv):
    desc = _small_desc(n_q_heads=hq, n_kv_heads=hkv, head_dim=16)
    n_ctx = 45
    m, cache, ks, vs = _filled_cache(oracle, desc, n_ctx)
    q = np.random.default_rng(6).normal(size=(hq, 16))
    for layer in (0, 1):
        got = oracle.attention(q, cache, layer, n_ctx)
        K = ks[layer].permute(1, 0, 2)   # [Hkv, T, hd]
        V = vs[layer].permute(1, 0, 2)
        rep = hq // hkv
        want = torch.nn.functional.scaled_dot_product_attention(
            torch.from_numpy(q)[:, None, :], K.repeat_interleave(rep, 0), V.repeat_interleave(rep, 0))
        np.testing.assert_allclose(got, want[:, 0, :].numpy(), rtol=1e-12, atol=1e-14)
        # attending to a shorter prefix is a different, also checkable, result
        got_s = oracle.attention(q, cache, layer, 7)
        want_s = torch.nn.functional.scaled_dot_product_attention(
            torch.from_numpy(q)[:, None, :], K.repeat_interleave(rep, 0)[:, :7],
            V.repeat_interleave(rep, 0)[:, :7])
        np.testing.assert_allclose(got_s, want_s[:, 0, :].numpy(), rtol=1e-12, atol=1e-14)


@pytest.mark.parametrize("hq,hkv,paged", [(4, 2, False), (8, 1, True)])
def test_cache_loaded_from_fp16_values(oracle, hq, hkv, paged):
    """Cache.load with a non-bf16 tensor (the loader the fp16-page parity tests feed the oracle through):
    what is read back equals the source exactly, row by row, and attention over the loaded cache equals
    library attention over the same fp16 values -- with values that bf16 cannot hold, a distinct key at
    every position and head, so that a shifted row, a swapped k / v or a lost mantissa bit shows."""
    hd, n_ctx = 16, 37
    desc = _small_desc(n_q_heads=hq, n_kv_heads=hkv, head_dim=hd)
    w = synth.make_weights(desc, seed=1)
    m = oracle.Model(desc, w)
    perm = [5, 0, 3, 1, 4, 2]
    cache = m.new_cache(n_ctx, 8, 6, perm) if paged else m.new_cache(n_ctx)
    g = torch.Generator().manual_seed(17)
    ks, vs = [], []
    for l in range(desc["n_layers"]):
        k = (torch.randn(n_ctx, hkv, hd, generator=g) * 1.7).to(torch.float16)
        v = (torch.randn(n_ctx, hkv, hd, generator=g) * 0.9).to(torch.float16)
        assert not torch.equal(k.to(torch.bfloat16).to(torch.float16), k)      # needs the 11-bit mantissa
        cache.load(l, k, v)
        ks.append(k.double()); vs.append(v.double())
    cache.set_len(n_ctx)
    for l in range(desc["n_layers"]):
        for pos in (0, 1, 7, 8, 20, n_ctx - 1):
            k_got, v_got = cache.read(l, pos)
            np.testing.assert_array_equal(k_got, ks[l][pos].numpy())
            np.testing.assert_array_equal(v_got, vs[l][pos].numpy())
        q = np.random.default_rng(60 + l).normal(size=(hq, hd))
        rep = hq // hkv
        K = ks[l].permute(1, 0, 2).repeat_interleave(rep, 0)
        V = vs[l].permute(1, 0, 2).repeat_interleave(rep, 0)
        for n in (n_ctx, 9):
            want = torch.nn.functional.scaled_dot_product_attention(torch.from_numpy(q)[:, None, :], K[:, :n], V[:, :n])
            np.testing.assert_allclose(oracle.attention(q, cache, l, n), want[:, 0, :].numpy(), rtol=1e-12, atol=1e-14)


def test_attention_degenerate_cases(oracle):
    desc = _small_desc(n_q_heads=4, n_kv_heads=2, head_dim=16)
    m, cache, ks, vs = _filled_cache(oracle, desc, 12)
    q = np.random.default_rng(7).normal(size=(4, 16))
    one = oracle.attention(q, cache, 0, 1)                       # a single key: o = v exactly
    for a in range(4):
        np.testing.assert_array_equal(one[a], vs[0][0, a // 2].numpy())
    # identical keys -> uniform weights -> o = mean(v)
    k = ks[0].clone(); k[:] = k[0]
    cache.load_bf16(0, k.to(torch.bfloat16), vs[0].to(torch.bfloat16))
    out = oracle.attention(q, cache, 0, 12)
    for a in range(4):
        np.testing.assert_allclose(out[a], vs[0][:, a // 2].mean(0).numpy(), rtol=1e-12)


def test_split_context_merge_equals_unsplit(oracle):
    desc = _small_desc(n_q_heads=4, n_kv_heads=2, head_dim=16)
    n_ctx = 53
    m, cache, _, _ = _filled_cache(oracle, desc, n_ctx)
    q = 3 * np.random.default_rng(8).normal(size=(4, 16))
    whole = oracle.attention(q, cache, 1, n_ctx)
    for cuts in ([0, 53], [0, 16, 32, 48, 53], [0, 1, 52, 53], [0, 20, 53]):
        for a in range(4):
            ms, ls, os_ = [], [], []
            for t0, t1 in zip(cuts[:-1], cuts[1:]):
                mm, ll, oo = oracle.attention_piece(q[a], cache, 1, t0, t1, a // 2)
                ms.append(mm); ls.append(ll); os_.append(oo)
            got = oracle.attention_merge(ms, ls, np.stack(os_))
            np.testing.assert_allclose(got, whole[a], rtol=1e-12, atol=1e-14)


def test_paged_cache_equals_contiguous_bit_for_bit(oracle):
    desc = _small_desc(qk_norm=1)
    w = _weights(desc)
    m = oracle.Model(desc, w)
    toks = synth.token_ids(5, 2, 41, desc["vocab"]).tolist()   # 41 tokens: 2 full pages + a tail
    P, pool = 16, 11
    table = [7, 2, 9, 0]                                       # shuffled, non-adjacent pages
    flat = m.new_cache(64)
    paged = m.new_cache(64, P, pool, table)
    for tok in toks:
        a = m.decode_step(flat, tok)
        b = m.decode_step(paged, tok)
        np.testing.assert_array_equal(a, b)
    for pos in (0, 15, 16, 40):
        for l in range(desc["n_layers"]):
            ka, va = flat.read(l, pos); kb, vb = paged.read(l, pos)
            np.testing.assert_array_equal(ka, kb); np.testing.assert_array_equal(va, vb)


def test_kv_bf16_switch_only_rounds_the_cache(oracle):
    desc = _small_desc()
    w = _weights(desc)
    m = oracle.Model(desc, w)
    c1, c2 = m.new_cache(8), m.new_cache(8)
    a = m.decode_step(c1, 3); b = m.decode_step(c2, 3, kv_as_bf16=True)
    k1, v1 = c1.read(0, 0); k2, v2 = c2.read(0, 0)
    np.testing.assert_array_equal(k2, torch.from_numpy(k1).to(torch.bfloat16).double().numpy())
    np.testing.assert_array_equal(v2, torch.from_numpy(v1).to(torch.bfloat16).double().numpy())
    assert 0 < np.abs(a - b).max() < 0.05


# --------------------------------------------------------------------------------------------
# sampler
# --------------------------------------------------------------------------------------------

def test_sampler_special_cases(oracle):
    lg = np.array([0.1, 2.0, -1.0, 2.0, 1.5])
    zero = np.zeros(5, np.float32)
    tok, z, gap = oracle.sample(lg, zero, 1.0)
    assert tok == 1 and z == np.float32(2.0) and gap == 0.0      # tie -> lowest index
    noise = np.array([0, 0, 0, 0, 1.0], np.float32)
    assert oracle.sample(lg, noise, 1.0)[0] == 4                 # 1.5 + 1 beats 2.0
    assert oracle.sample(lg, noise, 0.25)[0] == 1                # logits / T: 8.0 beats 6 + 1
    tok, z, gap = oracle.sample(np.array([1.0, 3.0]), np.zeros(2, np.float32), 2.0)
    assert tok == 1 and z == np.float32(1.5) and gap == np.float32(1.0)


def test_sampler_is_a_draw_from_softmax(oracle):
    """Gumbel-max theorem by brute force on a tiny vocabulary, at two temperatures."""
    V, N = 6, 60000
    lg = np.array([0.3, -1.2, 1.1, 0.0, 2.0, -0.4])
    for T in (1.0, 0.6):
        p = torch.softmax(torch.from_numpy(lg) / T, 0).numpy()
        noise = synth.gumbel_noise(99, 0, N, V).numpy()
        counts = np.zeros(V)
        for i in range(N):
            counts[oracle.sample(lg, noise[i], T)[0]] += 1
        sigma = np.sqrt(N * p * (1 - p))
        assert np.all(np.abs(counts - N * p) < 4 * sigma), (counts, N * p)


def test_golden_actor_settings_are_what_the_workloads_use():
    here = os.path.dirname(os.path.abspath(__file__))
    vals = {}
    for line in open(os.path.join(here, "golden", "actor_sampling.txt")):
        if line.strip() and not line.startswith("#"):
            k, v = line.split()
            vals[k] = float(v)
    assert vals == {"max_response_tokens": 8192, "temperature": 1.0, "top_p": 1.0, "top_k": -1}


def test_log_prob_matches_library_log_softmax_and_sampler(oracle):
    """log_prob is log softmax(logits / T)[token]: against torch.log_softmax, against the closed form
    on uniform logits (-log V), and exp of it summed over the vocabulary is 1."""
    rng = np.random.default_rng(3)
    for T in (0.6, 1.0, 2.5):
        lg = rng.normal(size=257) * 3
        ref = torch.log_softmax(torch.tensor(lg, dtype=torch.float64) / T, dim=0).numpy()
        for tok in (0, 100, 256):
            assert abs(oracle.log_prob(lg, tok, T) - ref[tok]) < 1e-12
        assert abs(sum(np.exp(oracle.log_prob(lg, t, T)) for t in range(257)) - 1.0) < 1e-12
    assert abs(oracle.log_prob(np.full(64, 7.5), 13, 1.3) + np.log(64)) < 1e-12


# ---- nucleus (top-p) sampling: the paper's evaluation setting --------------------------------------

def _logits_of(probs):
    return np.log(np.asarray(probs, dtype=np.float64))


def test_nucleus_hand_example_and_limits(oracle):
    """Probabilities 0.5 / 0.3 / 0.15 / 0.05 (temperature 1): the shortest most-probable-first prefix
    reaching top_p.  Mass 0.4 -> {0}; 0.79 -> {0, 1}; 0.81 -> {0, 1, 2}; 0.96 -> all.  The decision
    exactly at a prefix sum (0.5, 0.8) is decided by rounding, so the pins stay off those points."""
    lg = _logits_of([0.5, 0.3, 0.15, 0.05])[[2, 0, 3, 1]]         # shuffled: tokens 1, 3, 0, 2 by probability
    want = {0.4: {1}, 0.79: {1, 3}, 0.81: {1, 3, 0}, 0.96: {0, 1, 2, 3}, 1e-9: {1}}
    for top_p, kept_want in want.items():
        kept, _, margin = oracle.nucleus_kept(lg, 1.0, top_p)
        assert set(np.flatnonzero(kept)) == kept_want, (top_p, kept)
        assert margin > 5e-3 or top_p < 1e-6
    # the temperature sharpens before the truncation: at T = 0.5 the probabilities are proportional to p^2
    # = 0.25, 0.09, 0.0225, 0.0025 -> 0.685, 0.247, 0.062, 0.007: top_p 0.9 keeps two tokens, 0.95 three
    assert set(np.flatnonzero(oracle.nucleus_kept(lg, 0.5, 0.9)[0])) == {1, 3}
    assert set(np.flatnonzero(oracle.nucleus_kept(lg, 0.5, 0.95)[0])) == {1, 3, 0}


def test_nucleus_against_sorted_prefix_search(oracle):
    """Against the textbook formulation on random logits (no ties): sort by probability, cumulative sum,
    keep up to and including the first position where the sum reaches top_p."""
    rng = np.random.default_rng(11)
    for trial in range(40):
        V = int(rng.integers(2, 400))
        lg = rng.normal(size=V) * rng.uniform(0.5, 4.0)
        T = float(rng.choice([0.6, 1.0, 1.7]))
        top_p = float(rng.uniform(0.05, 0.999))
        kept, z, margin = oracle.nucleus_kept(lg, T, top_p)
        pr = torch.softmax(torch.tensor(z.astype(np.float64)), dim=0).numpy()
        order = np.argsort(-pr, kind="stable")
        cs = np.cumsum(pr[order])
        n_keep = int(np.searchsorted(cs, top_p, side="left")) + 1
        if margin > 1e-9:                     # otherwise rounding of the cumulative sum decides
            assert set(np.flatnonzero(kept)) == set(order[:min(n_keep, V)].tolist()), (trial, V, top_p)


def test_nucleus_ties_and_sampler_reductions(oracle):
    """Equally probable tokens at the cut are all kept; top_p = 1 is the untruncated Gumbel-argmax of
    the rollout sampler; a vanishing top_p is greedy decoding whatever the noise."""
    lg = _logits_of([0.4, 0.2, 0.2, 0.1, 0.1])
    assert set(np.flatnonzero(oracle.nucleus_kept(lg, 1.0, 0.5)[0])) == {0, 1, 2}      # 0.4 < 0.5: the tied pair enters
    assert set(np.flatnonzero(oracle.nucleus_kept(lg, 1.0, 0.85)[0])) == {0, 1, 2, 3, 4}
    rng = np.random.default_rng(5)
    for trial in range(20):
        V = 300
        lg = rng.normal(size=V) * 2
        g = synth.gumbel_noise(77, trial, 1, V)[0].numpy()
        T = 0.6 + 0.1 * trial
        assert oracle.nucleus_sample(lg, g, T, 1.0)[0] == oracle.sample(lg, g, T)[0]
        assert oracle.nucleus_sample(lg, g, T, 1e-12)[0] == int(np.argmax(lg))


def test_nucleus_draws_follow_the_renormalised_distribution(oracle):
    """Gumbel-argmax over the kept set samples the kept tokens in proportion to their probabilities and
    never leaves the set: 20 000 draws with seeded noise on six tokens."""
    probs = np.array([0.35, 0.25, 0.2, 0.1, 0.06, 0.04])
    lg = _logits_of(probs)
    kept = oracle.nucleus_kept(lg, 1.0, 0.85)[0]
    assert set(np.flatnonzero(kept)) == {0, 1, 2, 3}                                   # 0.8 < 0.85 <= 0.9
    n = 20000
    noise = synth.gumbel_noise(123, 0, n, 6).numpy()
    counts = np.zeros(6)
    for i in range(n):
        counts[oracle.nucleus_sample(lg, noise[i], 1.0, 0.85)[0]] += 1
    assert counts[4] == 0 and counts[5] == 0
    want = probs[:4] / probs[:4].sum()
    sigma = np.sqrt(want * (1 - want) / n)
    assert np.all(np.abs(counts[:4] / n - want) < 4.5 * sigma), (counts / n, want)


# ---- role-conditioned advantage estimation (Algorithm 1, Eq. 2) ---------------------------------------

def test_rae_closed_forms(oracle):
    """Constant return R from b = 0: after k updates b = R (1 - alpha^k), advantage R alpha^k.  alpha = 0
    tracks the last return (advantage 0); alpha = 1 never moves the baseline."""
    alpha, R = 0.95, 0.8
    b = [[0.0, 0.0]]
    adv = oracle.rae_update(b, alpha, [0] * 30, [[R, -R]] * 30)
    for k in range(1, 31):
        assert abs(adv[k - 1][0] - R * alpha ** k) < 1e-13
        assert abs(adv[k - 1][1] + R * alpha ** k) < 1e-13          # zero-sum: the roles mirror each other
    assert abs(b[0][0] - R * (1 - alpha ** 30)) < 1e-13 and abs(b[0][0] + b[0][1]) < 1e-15
    b = [[0.3, -0.1]]
    assert oracle.rae_update(b, 0.0, [0], [[1.0, -1.0]]) == [[0.0, 0.0]] and b == [[1.0, -1.0]]
    b = [[0.3, -0.1]]
    adv = oracle.rae_update(b, 1.0, [0], [[1.0, -1.0]])
    assert b == [[0.3, -0.1]] and abs(adv[0][0] - 0.7) < 1e-15 and abs(adv[0][1] + 0.9) < 1e-15


def test_rae_is_an_exponential_average_per_game_and_role(oracle):
    """Against the unrolled sum b_k = (1 - alpha) sum_j alpha^(k-j) R_j, games kept apart, the advantage
    using the baseline after its own update, and the order of the batch mattering."""
    rng = np.random.default_rng(2)
    alpha = 0.9
    game_of = rng.integers(0, 3, size=40).tolist()
    ret = [[float(r), float(-r)] for r in rng.choice([-1.0, 0.0, 1.0], size=40)]
    b = [[0.0, 0.0] for _ in range(3)]
    adv = oracle.rae_update(b, alpha, game_of, ret)
    for g in range(3):
        mine = [t for t in range(40) if game_of[t] == g]
        for p in (0, 1):
            run = 0.0
            for k, t in enumerate(mine):
                run = (1 - alpha) * sum(alpha ** (k - j) * ret[mine[j]][p] for j in range(k + 1))
                assert abs(adv[t][p] - (ret[t][p] - run)) < 1e-12
            assert abs(b[g][p] - run) < 1e-12
    b1, b2 = [[0.0, 0.0]], [[0.0, 0.0]]
    oracle.rae_update(b1, alpha, [0, 0], [[1.0, -1.0], [-1.0, 1.0]])
    oracle.rae_update(b2, alpha, [0, 0], [[-1.0, 1.0], [1.0, -1.0]])
    assert abs(b1[0][0] + b2[0][0]) < 1e-15 and abs(b1[0][0] - (-0.1 + 0.09)) < 1e-15


def test_rae_host_routine_of_the_library_matches(oracle):
    """spiral_rae_update is host arithmetic (no device work): same numbers as the oracle's loop."""
    sp = pytest.importorskip("paper_2506_24119_b200")
    rng = np.random.default_rng(4)
    game_of = rng.integers(0, 5, size=200).tolist()
    ret = [[float(r), float(-r)] for r in rng.normal(size=200)]
    b_ref = [[0.0, 0.0] for _ in range(5)]
    adv_ref = np.array(oracle.rae_update(b_ref, 0.95, game_of, ret))
    b = np.zeros((5, 2))
    adv = sp.spiral_rae_update(b, 0.95, game_of, ret)
    assert np.abs(adv - adv_ref).max() < 1e-15 and np.abs(b - np.array(b_ref)).max() < 1e-15
    with pytest.raises(sp.SpiralError):
        sp.spiral_rae_update(b, 1.5, game_of, ret)
    before = b.copy()
    with pytest.raises(sp.SpiralError):
        sp.spiral_rae_update(b, 0.95, [0, 7], [[1, -1], [1, -1]])
    assert np.array_equal(b, before)


def test_golden_evaluation_and_learner_settings():
    """The evaluation sampler's setting and the RAE decay as the paper prints them ("Evaluation Settings";
    hyperparameter table): the values the nucleus-decoding and RAE pins above are run at."""
    here = os.path.dirname(os.path.abspath(__file__))
    vals = {}
    for line in open(os.path.join(here, "golden", "evaluation_and_learner_settings.txt")):
        if line.strip() and not line.startswith("#"):
            k, v = line.split()
            vals[k] = float(v)
    assert vals == {"eval_temperature": 0.6, "eval_top_p": 0.95, "rae_ema_decay": 0.95}
