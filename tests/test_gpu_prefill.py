"""Dense context append (the tensor-core prefill path) against the oracle.

Between two turns the environment appends an observation of tens to hundreds of tokens to every
game's context.  When a call carries more new tokens than one decode-shaped step holds, the
library runs them as dense passes (256-token GEMM tiles, causal block attention).  The checks go
through what the path leaves behind: the logits after the last appended token and the logits of
the decode steps that follow, which read every key and value the append wrote.
"""
import time

import numpy as np
import pytest
import torch

import synth
from harness import TOL_MAX_ABS, TOL_REL_RMS, Pair, compare_logits
from test_gpu_parity import _check, _run_teacher_forced

pytestmark = pytest.mark.gpu


def _append(pair, games, new_tokens):
    """One spiral_prefill call on both sides; returns (worst max|delta|, worst rel rms) of the last-token logits."""
    sp, V = pair.sp, pair.desc["vocab"]
    flat = torch.tensor(sum(new_tokens, []), dtype=torch.int32).cuda()
    offs = np.concatenate([[0], np.cumsum([len(t) for t in new_tokens])]).tolist()
    last = torch.empty(len(games), V, dtype=torch.float32, device="cuda")
    sp.spiral_prefill(pair.ctx, pair.kv, games, flat, offs, last)
    last = last.cpu().numpy()
    worst_abs, worst_rms = 0.0, 0.0
    for i, g in enumerate(games):
        ref = pair.oracle.prefill(pair.oracle_cache(g), new_tokens[i])
        a, r = compare_logits(last[i], ref)
        worst_abs, worst_rms = max(worst_abs, a), max(worst_rms, r)
    return worst_abs, worst_rms


def _decode(pair, games, steps, seed):
    sp, V = pair.sp, pair.desc["vocab"]
    n = len(games)
    tok_out = torch.empty(n, dtype=torch.int32, device="cuda")
    logits = torch.empty(n, V, dtype=torch.float32, device="cuda")
    worst_abs, worst_rms = 0.0, 0.0
    for s in range(steps):
        tok_in = synth.token_ids(seed, 1000 + s, n, V, stream=synth.STREAM_TEACHER)
        noise = synth.gumbel_noise(seed, s, n, V)
        sp.spiral_decode_step(pair.ctx, pair.kv, games, tok_in.cuda(), noise.cuda(), 1.0, tok_out, logits)
        lg = logits.cpu().numpy()
        for i, g in enumerate(games):
            ref = pair.oracle.decode_step(pair.oracle_cache(g), int(tok_in[i]))
            a, r = compare_logits(lg[i], ref)
            worst_abs, worst_rms = max(worst_abs, a), max(worst_rms, r)
    return worst_abs, worst_rms


@pytest.mark.parametrize("shape_name,overrides,chunk", [
    ("tiny_qknorm", {}, 256),                                        # 2 query heads per KV head, head_dim 64
    ("tiny_bias", {}, 512),                                          # 4 per KV head, QKV bias
    ("tiny", dict(n_q_heads=8, n_kv_heads=1, head_dim=128), 256),    # 8 per KV head, head_dim 128
    ("tiny", dict(n_q_heads=2, n_kv_heads=2, head_dim=128), 0),      # no grouping; one pass
    ("tiny", dict(n_q_heads=7, n_kv_heads=1, head_dim=64, d_model=448), 256),   # a group that does not divide 128 rows
])
def test_dense_append_in_several_passes(monkeypatch, shape_name, overrides, chunk):
    """Five games, ragged lengths (one token, below a page, page-aligned, several tiles), a pass size
    that cuts games in the middle: the later pass must find the earlier pass's keys in the pages."""
    if chunk:
        monkeypatch.setenv("SPIRAL_PREFILL_CHUNK", str(chunk))
    desc = synth.shape(shape_name, **overrides)
    lens = [300, 1, 129, 256, 40, 13]
    pair = Pair(desc, max_batch=16, max_ctx=320, n_games=8)
    try:
        games = [5, 0, 3, 7, 1, 2]
        prompts = [synth.token_ids(synth.MASTER_SEED, 900 + i, lens[i], desc["vocab"]).tolist() for i in range(len(games))]
        res = _run_teacher_forced(pair, games, prompts, 4, synth.MASTER_SEED + 21)
        print(shape_name, overrides, "max|d| %.2e rel-rms %.2e agree %.4f" % res[:3], res[3])
        _check(*res)
    finally:
        pair.close()


def test_dense_append_onto_existing_context():
    """Turn structure: append, decode a few tokens, append again at positions that are not page
    aligned, decode again; some games sit out the second append."""
    desc = synth.shape("tiny_qknorm")
    n_games = 6
    pair = Pair(desc, max_batch=16, max_ctx=256, n_games=n_games)
    try:
        V = desc["vocab"]
        games = list(range(n_games))
        obs = [synth.token_ids(11, g, 21 + 7 * g, V).tolist() for g in games]
        launches0 = pair.sp.spiral_launch_count(pair.ctx)
        worst = [_append(pair, games, obs)]
        # one pass = eight kernels per layer plus embedding, row gather, final norm and head -- not one
        # decode-shaped step per 16 tokens
        assert pair.sp.spiral_launch_count(pair.ctx) - launches0 <= 8 * desc["n_layers"] + 6
        worst.append(_decode(pair, games, 3, 31))
        later = [4, 1, 2]
        obs2 = [synth.token_ids(12, g, 50 + 30 * i, V).tolist() for i, g in enumerate(later)]
        worst.append(_append(pair, later, obs2))
        worst.append(_decode(pair, games, 3, 32))
        rc, detail = pair.sp.spiral_last_status(pair.ctx)
        assert rc == 0, detail
        print("append/decode/append/decode:", worst)
        assert max(w[0] for w in worst) <= TOL_MAX_ABS
        assert max(w[1] for w in worst) <= TOL_REL_RMS
    finally:
        pair.close()


@pytest.mark.parametrize("attn", ["mma", "tc1"])
def test_other_attention_kernels_of_the_append_still_available(monkeypatch, attn):
    """SPIRAL_APPEND_ATTN=mma runs the append's attention on mma.sync instead of tcgen05, =tc1 on tcgen05
    with one query tile per CTA and two CTAs per SM: same bars."""
    monkeypatch.setenv("SPIRAL_APPEND_ATTN", attn)
    monkeypatch.setenv("SPIRAL_PREFILL_CHUNK", "256")
    for name, over in [("tiny_bias", {}), ("tiny", dict(n_q_heads=7, n_kv_heads=1, head_dim=128, d_model=448))]:
        desc = synth.shape(name, **over)
        pair = Pair(desc, max_batch=16, max_ctx=320, n_games=4)
        try:
            lens = [300, 17, 130]
            prompts = [synth.token_ids(synth.MASTER_SEED, 950 + i, lens[i], desc["vocab"]).tolist() for i in range(3)]
            res = _run_teacher_forced(pair, [3, 0, 1], prompts, 3, synth.MASTER_SEED + 23)
            _check(*res)
        finally:
            pair.close()


def test_step_shaped_append_still_available(monkeypatch):
    """SPIRAL_PREFILL_DENSE=0 keeps the append on decode-shaped steps (the path of small batches
    and bf16 caches): same result within the tolerances."""
    monkeypatch.setenv("SPIRAL_PREFILL_DENSE", "0")
    desc = synth.shape("tiny_qknorm")
    pair = Pair(desc, max_batch=24, max_ctx=160, n_games=3)
    try:
        games = [2, 0]
        prompts = [synth.token_ids(synth.MASTER_SEED, 300 + i, 97 - 40 * i, desc["vocab"]).tolist() for i in range(2)]
        res = _run_teacher_forced(pair, games, prompts, 4, synth.MASTER_SEED + 9)
        _check(*res)
    finally:
        pair.close()


def test_dense_append_full_width():
    """Qwen3-4B width (d_model 2560, 32/8 heads of 128, d_ff 9728, 151 936-row head) at three layers,
    so that the oracle can afford observations of the paper's size (hundreds of tokens): two rounds
    of append + decode on three games."""
    desc = synth.shape("qwen3_4b", n_layers=3)
    t0 = time.time()
    pair = Pair(desc, max_batch=16, max_ctx=704, n_games=3, gains=False, generate_on_gpu=True)
    try:
        V = desc["vocab"]
        games = [0, 1, 2]
        obs = [synth.token_ids(13, g, [300, 170, 45][g], V).tolist() for g in games]
        worst = [_append(pair, games, obs)]
        worst.append(_decode(pair, games, 2, 41))
        obs2 = [synth.token_ids(14, g, [40, 300, 10][g], V).tolist() for g in games]
        worst.append(_append(pair, games, obs2))
        worst.append(_decode(pair, games, 2, 42))
        rc, detail = pair.sp.spiral_last_status(pair.ctx)
        assert rc == 0, detail
        print("full width:", worst, "%.0fs" % (time.time() - t0))
        assert max(w[0] for w in worst) <= TOL_MAX_ABS
        assert max(w[1] for w in worst) <= TOL_REL_RMS
    finally:
        pair.close()


@pytest.mark.parametrize("attn", ["tc", "mma"])
def test_dense_append_long_contexts(monkeypatch, attn):
    """Contexts of a few thousand tokens (hundreds of pages per game: the attention kernels' page-id
    windows and ring phases wrap many times), appended in two rounds with decode steps between."""
    monkeypatch.setenv("SPIRAL_APPEND_ATTN", attn)
    desc = synth.shape("tiny_bias")
    pair = Pair(desc, max_batch=16, max_ctx=2500, n_games=2)
    try:
        V = desc["vocab"]
        games = [1, 0]
        obs = [synth.token_ids(19, g, [2049, 700][i], V).tolist() for i, g in enumerate(games)]
        worst = [_append(pair, games, obs)]
        worst.append(_decode(pair, games, 2, 51))
        obs2 = [synth.token_ids(20, g, [40, 301][i], V).tolist() for i, g in enumerate(games)]
        worst.append(_append(pair, games, obs2))
        worst.append(_decode(pair, games, 2, 52))
        rc, detail = pair.sp.spiral_last_status(pair.ctx)
        assert rc == 0, detail
        print("long contexts (%s):" % attn, worst)
        assert max(w[0] for w in worst) <= TOL_MAX_ABS
        assert max(w[1] for w in worst) <= TOL_REL_RMS
    finally:
        pair.close()
