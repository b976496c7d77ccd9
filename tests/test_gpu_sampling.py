"""Nucleus (top-p) sampling on the GPU against the oracle: the sampler alone on logits of the real
vocabulary size, and the decode step that ends in it (the paper's evaluation setting: temperature
0.6, top-p 0.95).  Keep/drop decisions compare a sum of probabilities with top_p; where the oracle
reports that a decision was within rounding of flipping (margin), the GPU's token only has to come
from the kept set widened by that band."""
import numpy as np
import pytest
import torch

import synth
from harness import TOL_TOKEN_AGREE, Pair, compare_logits
from test_gpu_parity import allowed_flips

pytestmark = pytest.mark.gpu

MARGIN = 2e-5          # fp32 sums of up to 151 936 probabilities against fp64: decisions closer than this may differ


def _token_ok(oracle_mod, logits, noise, T, top_p, got):
    """(matches the oracle's token, acceptable) for one row."""
    tok, kept, margin = oracle_mod.nucleus_sample(logits, noise, T, top_p)
    if tok == got:
        return True, True
    if margin > MARGIN:
        return False, False
    # a decision near top_p: the token must be the draw of a set kept at top_p - MARGIN or top_p + MARGIN
    alt = {oracle_mod.nucleus_sample(logits, noise, T, top_p + s * 2 * MARGIN)[0] for s in (-1, 1)}
    return False, got in alt


@pytest.mark.parametrize("vocab,scale", [(4096, 2.0), (151936, 1.0), (151936, 4.0)])
def test_nucleus_sampler_alone(vocab, scale):
    desc = synth.shape("tiny", vocab=vocab)
    n = 12
    pair = Pair(desc, max_batch=16, max_ctx=32, n_games=2)
    try:
        sp = pair.sp
        # Gumbel-distributed values as logits: a long right tail, so the nucleus holds from a handful of
        # tokens (scale 4) to most of the vocabulary (scale 1)
        logits = (synth.gumbel_noise(31, 0, n, vocab) * scale).contiguous()
        logits[3, 100:108] = logits[3].max() + 1.0             # eight exactly tied leaders
        logits[5] = 0.25                                       # a uniform row
        noise = synth.gumbel_noise(31, 1, n, vocab)
        tok = torch.empty(n, dtype=torch.int32, device="cuda")
        lg_np, nz_np = logits.numpy().astype(np.float64), noise.numpy()
        for T, top_p in [(0.6, 0.95), (1.0, 0.5), (0.6, 0.05), (1.3, 1.0), (0.6, 1e-6)]:
            sp.spiral_sample_nucleus(pair.ctx, logits.cuda(), noise.cuda(), T, top_p, tok)
            got = tok.cpu().numpy()
            for i in range(n if vocab < 100000 else 7):         # the oracle's sort is a Python loop
                same, ok = _token_ok(pair.oracle_mod, lg_np[i], nz_np[i], T, top_p, int(got[i]))
                assert ok, (vocab, scale, T, top_p, i, int(got[i]))
        # without noise the draw is the most probable token (lowest index among the tied leaders)
        sp.spiral_sample_nucleus(pair.ctx, logits.cuda(), None, 0.6, 0.95, tok)
        assert tok.cpu().tolist() == [int(np.argmax(lg_np[i])) for i in range(n)]
        rc, detail = sp.spiral_last_status(pair.ctx)
        assert rc == 0, detail
    finally:
        pair.close()


@pytest.mark.parametrize("shape_name,n_games", [("tiny_qknorm", 5), ("tiny", 24)])
def test_decode_step_with_nucleus_sampling(shape_name, n_games):
    """Decode steps at temperature 0.6 / top-p 0.95 (and a tight nucleus), CUDA-core head at 5 games and
    tensor-core head at 24, on the default stream and on a side stream (second use of a size replays the
    recorded graph): tokens against the oracle's draw from the GPU's own logits (the sampler) and from
    the oracle's logits (the whole step)."""
    desc = synth.shape(shape_name)
    pair = Pair(desc, max_batch=n_games, max_ctx=64, n_games=n_games, std=0.08)
    try:
        sp, V = pair.sp, desc["vocab"]
        games = list(range(n_games))
        lens = synth.lengths(synth.MASTER_SEED, 8, n_games, 2, 12)
        prompts = [synth.token_ids(synth.MASTER_SEED, 700 + i, lens[i], V).tolist() for i in range(n_games)]
        flat = torch.tensor(sum(prompts, []), dtype=torch.int32).cuda()
        offs = np.concatenate([[0], np.cumsum(lens)]).tolist()
        sp.spiral_prefill(pair.ctx, pair.kv, games, flat, offs)
        for g, pr in zip(games, prompts):
            pair.oracle.prefill(pair.oracle_cache(g), pr)
        side = torch.cuda.Stream()
        tok_out = torch.empty(n_games, dtype=torch.int32, device="cuda")
        logits = torch.empty(n_games, V, dtype=torch.float32, device="cuda")
        agree, total = 0, 0
        for s, (T, top_p, stream) in enumerate([(0.6, 0.95, None), (0.6, 0.95, side), (0.6, 0.95, side), (0.6, 0.3, side),
                                                (1.0, 1.0, side)]):
            tok_in = synth.token_ids(23, s, n_games, V, stream=synth.STREAM_TEACHER)
            noise = synth.gumbel_noise(23, s, n_games, V)
            torch.cuda.synchronize()
            if stream is None:
                sp.spiral_decode_step_nucleus(pair.ctx, pair.kv, games, tok_in.cuda(), noise.cuda(), T, top_p, tok_out, logits)
            else:
                with torch.cuda.stream(stream):
                    sp.spiral_decode_step_nucleus(pair.ctx, pair.kv, games, tok_in.cuda(), noise.cuda(), T, top_p, tok_out,
                                                  logits, stream)
                stream.synchronize()
            torch.cuda.synchronize()
            got, lg = tok_out.cpu().numpy(), logits.cpu().numpy().astype(np.float64)
            for i, g in enumerate(games):
                ref = pair.oracle.decode_step(pair.oracle_cache(g), int(tok_in[i]))
                assert compare_logits(lg[i], ref)[0] <= 0.05
                _, ok = _token_ok(pair.oracle_mod, lg[i], noise[i].numpy(), T, top_p, int(got[i]))
                assert ok, (s, i, int(got[i]))
                total += 1
                agree += int(pair.oracle_mod.nucleus_sample(ref, noise[i].numpy(), T, top_p)[0] == int(got[i]))
                n_kept = int(pair.oracle_mod.nucleus_kept(ref, T, top_p)[0].sum())
                assert top_p == 1.0 or n_kept < V         # the truncation really removes tokens
        assert total - agree <= allowed_flips(total), (agree, total)
        rc, detail = sp.spiral_last_status(pair.ctx)
        assert rc == 0, detail
    finally:
        pair.close()
