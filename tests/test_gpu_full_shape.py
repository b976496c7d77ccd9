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
