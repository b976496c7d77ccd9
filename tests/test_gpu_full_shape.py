"""Full-depth, full-width shapes of the paper's model families at a small batch: the oracle can
afford a few tokens per game, which is enough to see how rounding accumulates over all layers."""
import time

import numpy as np
import pytest
import torch

import synth
from harness import TOL_MAX_ABS, TOL_REL_RMS, Pair, compare_logits
from test_gpu_parity import _check, _run_teacher_forced

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("shape_name,n_games,prompt,steps", [
    ("qwen3_4b", 3, 20, 6),
    ("llama31_8b", 2, 12, 4),
    ("qwen25_7b", 2, 12, 4),
])
def test_full_shape_short_context(shape_name, n_games, prompt, steps):
    desc = synth.shape(shape_name)
    t0 = time.time()
    pair = Pair(desc, max_batch=4, max_ctx=64, n_games=4, gains=False, generate_on_gpu=True)
    try:
        games = list(range(n_games))
        prompts = [synth.token_ids(synth.MASTER_SEED, 40 + i, prompt - i, desc["vocab"]).tolist()
                   for i in range(n_games)]
        res = _run_teacher_forced(pair, games, prompts, steps, synth.MASTER_SEED + 1)
        print(shape_name, "max|d| %.2e rel-rms %.2e agree %.4f" % res[:3], res[3], "%.0fs" % (time.time() - t0))
        _check(*res)
    finally:
        pair.close()


def _sampled_games_at_full_depth(shape_name, n_games, lens, sampled, steps, seed=7):
    """A configured workload at its own sizes: every sequence's cache holds seeded random keys/values (loaded
    identically on both sides for the sampled sequences), decode steps run on a side stream so that the second
    one is the recorded CUDA graph, and the sampled sequences' logits and tokens are checked against the oracle."""
    desc = synth.shape(shape_name)
    max_len = max(lens)
    t0 = time.time()
    pair = Pair(desc, max_batch=n_games, max_ctx=max_len + 16, n_games=n_games, gains=False, generate_on_gpu=True,
                pool_pages=sum((l + steps + 15) // 16 for l in lens) + 8)
    try:
        sp, V = pair.sp, desc["vocab"]
        Hkv, hd = desc["n_kv_heads"], desc["head_dim"]
        games = list(range(n_games))
        for layer in range(desc["n_layers"]):
            n = n_games * max_len * Hkv * hd
            k = synth.uniform_bf16(seed, 2 * layer, n, 2.0, "cuda").to(torch.float16).view(n_games, max_len, Hkv, hd)
            v = synth.uniform_bf16(seed, 2 * layer + 1, n, 1.0, "cuda").to(torch.float16).view(n_games, max_len, Hkv, hd)
            for g in games:
                sp.spiral_kv_load(pair.ctx, pair.kv, g, layer, k[g, :lens[g]], v[g, :lens[g]])
            for g in sampled:
                pair.oracle_cache(g).load(layer, k[g, :lens[g]].cpu(), v[g, :lens[g]].cpu())
        for g in sampled:
            pair.oracle_cache(g).set_len(lens[g])
        del k, v
        stream = torch.cuda.Stream()
        torch.cuda.synchronize()
        worst_abs, worst_rms, mism, total = 0.0, 0.0, [], 0
        with torch.cuda.stream(stream):
            tok_out = torch.empty(n_games, dtype=torch.int32, device="cuda")
            logits = torch.empty(n_games, V, dtype=torch.float32, device="cuda")
            for s in range(steps):
                tok_in = synth.token_ids(seed, 1000 + s, n_games, V, stream=synth.STREAM_TEACHER)
                noise = synth.gumbel_noise(seed, s, n_games, V, "cuda")
                sp.spiral_decode_step(pair.ctx, pair.kv, games, tok_in.cuda(), noise, 1.0, tok_out, logits, stream)
                stream.synchronize()
                got_tok = tok_out.cpu().numpy()
                for g in sampled:
                    ref = pair.oracle.decode_step(pair.oracle_cache(g), int(tok_in[g]))
                    a, r = compare_logits(logits[g].cpu().numpy(), ref)
                    worst_abs, worst_rms = max(worst_abs, a), max(worst_rms, r)
                    tok, _, gap = pair.oracle_mod.sample(ref, noise[g].cpu().numpy(), 1.0)
                    total += 1
                    if tok != got_tok[g]:
                        mism.append((s, g, tok, int(got_tok[g]), gap))
        rc, detail = sp.spiral_last_status(pair.ctx)
        assert rc == 0, (rc, detail)
        print("%s x %d: max|d| %.2e rel-rms %.2e mismatches %s  %.0fs" % (shape_name, n_games, worst_abs, worst_rms, mism, time.time() - t0))
        _check(worst_abs, worst_rms, 1.0 - len(mism) / total, mism, total)
    finally:
        pair.close()


def test_benchmark_workload_sampled_games():
    """The benchmark's own configuration: Qwen3-4B shape, 128 concurrent games with 512 cached tokens each."""
    _sampled_games_at_full_depth("qwen3_4b", 128, [512] * 128, [0, 77, 127], 2)


def test_llama31_8b_workload_sampled_sequences():
    """The Llama-3.1-8B-shaped configuration at its own sizes (Section 4 trains this family): 64 sequences with
    1 024 to 4 096 cached tokens, untied LM head, eps 1e-5, theta 5e5; the shortest, a middling and the longest
    sequence are checked over all 32 layers."""
    lens = synth.lengths(11, 3, 64, 1024, 4096)
    order = sorted(range(64), key=lambda g: lens[g])
    _sampled_games_at_full_depth("llama31_8b", 64, lens, [order[0], order[31], order[63]], 2, seed=11)


def test_qwen25_7b_long_context_sampled_sequence():
    """The Qwen2.5-7B-shaped long-reasoning configuration at its own sizes (the R1-Distill-Qwen-7B row of
    Table 1): 64 sequences with 16 368 cached tokens -- the step takes them to the configuration's 16 384 --
    seven query heads per KV head, QKV bias; one sequence is checked over all 28 layers."""
    _sampled_games_at_full_depth("qwen25_7b", 64, [16368] * 64, [41], 2, seed=13)


def test_benchmark_append_sampled_game():
    """The benchmark's context-append configuration -- Qwen3-4B shape at full depth, 128 games with 512
    cached tokens each, 300 new tokens per game in one spiral_prefill call (dense passes of 9 472 token
    rows that cut games in the middle) -- checked on one sampled game the oracle can afford: the logits
    after its last appended token and after one decode step behind it."""
    desc = synth.shape("qwen3_4b")
    n_games, ctx_len, n_new = 128, 512, 300
    sampled = 77
    t0 = time.time()
    pair = Pair(desc, max_batch=n_games, max_ctx=ctx_len + n_new + 16, n_games=n_games, gains=False, generate_on_gpu=True)
    try:
        sp, V = pair.sp, desc["vocab"]
        Hkv, hd = desc["n_kv_heads"], desc["head_dim"]
        games = list(range(n_games))
        for layer in range(desc["n_layers"]):
            n = n_games * ctx_len * Hkv * hd
            k = synth.uniform_bf16(7, 2 * layer, n, 2.0, "cuda").to(torch.float16).view(n_games, ctx_len, Hkv, hd)
            v = synth.uniform_bf16(7, 2 * layer + 1, n, 1.0, "cuda").to(torch.float16).view(n_games, ctx_len, Hkv, hd)
            for g in games:
                sp.spiral_kv_load(pair.ctx, pair.kv, g, layer, k[g], v[g])
            pair.oracle_cache(sampled).load(layer, k[sampled].cpu(), v[sampled].cpu())
        pair.oracle_cache(sampled).set_len(ctx_len)
        del k, v
        new_tok = synth.token_ids(9, 1, n_games * n_new, V, "cuda")
        offs = [i * n_new for i in range(n_games + 1)]
        last = torch.empty(n_games, V, dtype=torch.float32, device="cuda")
        launches0 = sp.spiral_launch_count(pair.ctx)
        sp.spiral_prefill(pair.ctx, pair.kv, games, new_tok, offs, last)
        torch.cuda.synchronize()
        # five passes (38 400 rows in passes of 9 472), eight kernels per layer each: the dense path ran
        assert sp.spiral_launch_count(pair.ctx) - launches0 <= 5 * (8 * desc["n_layers"] + 3) + 4
        mine = new_tok[sampled * n_new:(sampled + 1) * n_new].cpu().tolist()
        ref = pair.oracle.prefill(pair.oracle_cache(sampled), mine)
        a0, r0 = compare_logits(last[sampled].cpu().numpy(), ref)
        tok_in = synth.token_ids(9, 2, n_games, V, stream=synth.STREAM_TEACHER)
        noise = synth.gumbel_noise(9, 3, n_games, V, "cuda")
        tok_out = torch.empty(n_games, dtype=torch.int32, device="cuda")
        logits = torch.empty(n_games, V, dtype=torch.float32, device="cuda")
        sp.spiral_decode_step(pair.ctx, pair.kv, games, tok_in.cuda(), noise, 1.0, tok_out, logits)
        ref = pair.oracle.decode_step(pair.oracle_cache(sampled), int(tok_in[sampled]))
        a1, r1 = compare_logits(logits[sampled].cpu().numpy(), ref)
        rc, detail = sp.spiral_last_status(pair.ctx)
        assert rc == 0, (rc, detail)
        print("bench append: after append max|d| %.2e rel-rms %.2e; after a step %.2e %.2e  %.0fs" % (a0, r0, a1, r1, time.time() - t0))
        assert max(a0, a1) <= TOL_MAX_ABS and max(r0, r1) <= TOL_REL_RMS
    finally:
        pair.close()
