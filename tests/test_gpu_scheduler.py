"""Episode scheduler (continuous batching of multi-turn games) against the oracle.

More games than batch slots, a pool too small to hold every game's worst case at once, ragged
observations and budgets, several turns per game, greedy decoding (zero noise) so that a game's
tokens do not depend on which batch row it was given.  The oracle replays every game's full history
(observation, response, observation, ...) and must pick the same next token at every generated
position; since it reads the whole context, a key or value cached twice, dropped or misplaced at a
turn boundary shows up as a stream of disagreements."""
import numpy as np
import pytest
import torch

import synth
from harness import TOL_MAX_ABS, Pair
from test_gpu_parity import allowed_flips

pytestmark = pytest.mark.gpu


def _play(pair, n_games, n_turns, eos, max_batch, seed, eager=False, noise_seed=None):
    """Runs all games to completion; returns per game the list of (observation, response, reason) per turn."""
    sp, V = pair.sp, pair.desc["vocab"]
    sched = sp.spiral_sched_create(pair.ctx, pair.kv, eos)
    if eager:
        sp.spiral_sched_policy(sched, 1, max_batch)          # admit as soon as a row and the pages are there
    zeros = torch.zeros(max_batch, V, dtype=torch.float32, device="cuda")
    obs_len = [synth.lengths(seed, 10 + t, n_games, 1, 40) for t in range(n_turns)]
    budget = [synth.lengths(seed, 20 + t, n_games, 1, 12) for t in range(n_turns)]
    games = [sp.spiral_sched_open(sched) for _ in range(n_games)]
    assert sorted(games) == list(range(n_games))
    with pytest.raises(sp.SpiralError):
        sp.spiral_sched_open(sched)                       # every cache row is taken
    history = {g: [] for g in games}
    turn_of = {g: 0 for g in games}

    def queue_turn(g):
        t = turn_of[g]
        obs = synth.token_ids(seed, 1000 * t + g, obs_len[t][g], V).tolist()
        sp.spiral_sched_turn(sched, g, obs, budget[t][g])
        history[g].append([obs, None, None])
    for g in games:
        queue_turn(g)
    stream = torch.cuda.Stream()
    open_turns, ticks, max_running = n_games, 0, 0
    with torch.cuda.stream(stream):
        while open_turns:
            noise = zeros if noise_seed is None else synth.gumbel_noise(noise_seed, ticks, max_batch, V, "cuda")
            n = sp.spiral_sched_tick(sched, noise, 1.0 if noise_seed is None else 0.8, stream)
            ticks += 1
            assert ticks < 5000
            st = sp.spiral_sched_stats(sched)
            max_running = max(max_running, st["running"])
            assert st["running"] <= max_batch and st["reserved_pages"] <= st["free_pages"]
            while True:
                done = sp.spiral_sched_poll(sched)
                if done is None:
                    break
                g, resp, why = done
                t = turn_of[g]
                assert 1 <= len(resp) <= budget[t][g]
                assert (why == 1 and resp[-1] == eos and eos not in resp[:-1]) or \
                       (why == 2 and len(resp) == budget[t][g] and eos not in resp)
                history[g][-1][1:] = [resp, why]
                turn_of[g] += 1
                open_turns -= 1
                if turn_of[g] < n_turns:
                    queue_turn(g)
                    open_turns += 1
    stream.synchronize()
    stats = sp.spiral_sched_stats(sched)
    rc, detail = sp.spiral_last_status(pair.ctx)
    assert rc == 0, detail
    assert stats["waiting"] == 0 and stats["running"] == 0 and stats["reserved_pages"] == 0
    # every game's cached length: its observations and responses, minus a final token not cached yet
    for g in games:
        toks = sum(len(o) + len(r) for o, r, _ in history[g])
        assert sp.spiral_kv_seq_len(pair.kv, g) in (toks, toks - 1)
    for g in games:
        sp.spiral_sched_close(sched, g)
    sp.spiral_sched_free(sched)
    return history, stats, max_running


def test_scheduler_plays_ragged_multi_turn_games():
    desc = synth.shape("tiny_qknorm")
    n_games, n_turns, max_batch = 24, 3, 16
    # worst case per game: 3 x (40 + 12) tokens = 10 pages; 24 games would need 240, the pool has 150
    pair = Pair(desc, max_batch=max_batch, max_ctx=176, n_games=n_games, pool_pages=150)
    try:
        sp = pair.sp
        free0 = sp.spiral_kv_free_pages(pair.kv)
        hist, stats, max_running = _play(pair, n_games, n_turns, -1, max_batch, 5, eager=True)
        assert max_running == max_batch                        # the batch was filled
        assert sp.spiral_kv_free_pages(pair.kv) == free0       # every page came back
        assert stats["dropped"] == 0                           # no end-of-sequence token: no late step
        # an end-of-sequence token that some responses contain: the same games again
        counts = {}
        for g in hist:
            for _, resp, _ in hist[g]:
                for tok in resp[:-1]:
                    counts[tok] = counts.get(tok, 0) + 1
        eos = max(counts, key=lambda t: (counts[t], -t))
        hist2, stats2, _ = _play(pair, n_games, n_turns, eos, max_batch, 5)
        assert sp.spiral_kv_free_pages(pair.kv) == free0
        n_eos = sum(1 for g in hist2 for _, _, why in hist2[g] if why == 1)
        assert n_eos >= 1
        # first turns see the same context in both runs: the response is the earlier one cut at the token
        for g in hist:
            first, again = hist[g][0][1], hist2[g][0][1]
            cut = first[:first.index(eos) + 1] if eos in first else first
            assert again == cut, (g, first, again)
        # the oracle replays each game of the second run and must choose the same tokens
        flips, total, worst_gap = 0, 0, 0.0
        for g in sorted(hist2):
            cache = pair.oracle.new_cache(176)
            logits = None
            for obs, resp, _ in hist2[g]:
                logits = pair.oracle.prefill(cache, obs)
                for tok in resp:
                    order = np.argsort(-logits, kind="stable")
                    total += 1
                    if int(order[0]) != tok:
                        flips += 1
                        gap = float(logits[order[0]] - logits[tok])
                        worst_gap = max(worst_gap, gap)
                        assert gap <= 4 * TOL_MAX_ABS, (g, tok, int(order[0]), gap)
                    logits = pair.oracle.decode_step(cache, tok)
        print("scheduler: %d generated tokens, %d flips (worst gap %.3g), %d end-of-sequence turns, dropped %d" %
              (total, flips, worst_gap, n_eos, stats2["dropped"]))
        assert flips <= allowed_flips(total), (flips, total)
        assert stats2["decoded"] == total + stats2["dropped"]
    finally:
        pair.close()


def test_scheduler_with_sampling_noise_keeps_its_books():
    """The same games with real Gumbel noise at temperature 0.8 (tokens then depend on the batch row a game
    happens to get, so there is no token-by-token reference): every response respects its budget and the
    end-of-sequence rule, the batch fills up, reservations never exceed the free pages, every page comes back."""
    desc = synth.shape("tiny")
    n_games, n_turns, max_batch = 24, 3, 16
    pair = Pair(desc, max_batch=max_batch, max_ctx=176, n_games=n_games, pool_pages=150)
    try:
        free0 = pair.sp.spiral_kv_free_pages(pair.kv)
        eos = 1234
        hist, stats, max_running = _play(pair, n_games, n_turns, eos, max_batch, 6, noise_seed=77)
        assert max_running == max_batch
        assert pair.sp.spiral_kv_free_pages(pair.kv) == free0
        total = sum(len(r) for g in hist for _, r, _ in hist[g])
        assert stats["decoded"] == total + stats["dropped"]
        assert all(0 <= tok < desc["vocab"] for g in hist for _, r, _ in hist[g] for tok in r)
    finally:
        pair.close()


def test_scheduler_refuses_what_cannot_fit():
    desc = synth.shape("tiny")
    pair = Pair(desc, max_batch=16, max_ctx=64, n_games=4, pool_pages=6)
    try:
        sp = pair.sp
        sched = sp.spiral_sched_create(pair.ctx, pair.kv, -1)
        g = sp.spiral_sched_open(sched)
        with pytest.raises(sp.SpiralError):                    # beyond max_ctx
            sp.spiral_sched_turn(sched, g, [1] * 60, 10)
        with pytest.raises(sp.SpiralError):                    # empty observation
            sp.spiral_sched_turn(sched, g, [], 4)
        sp.spiral_sched_turn(sched, g, [1, 2, 3], 4)
        with pytest.raises(sp.SpiralError):                    # a turn is already waiting
            sp.spiral_sched_turn(sched, g, [1], 1)
        with pytest.raises(sp.SpiralError):                    # cannot close a game with a waiting turn
            sp.spiral_sched_close(sched, g)
        zeros = torch.zeros(16, desc["vocab"], dtype=torch.float32, device="cuda")
        done = None
        for _ in range(12):
            sp.spiral_sched_tick(sched, zeros, 1.0)
            done = done or sp.spiral_sched_poll(sched)
        assert done is not None and done[0] == g and len(done[1]) == 4 and done[2] == 2
        assert sp.spiral_sched_tick(sched, zeros, 1.0) == 0    # nothing left to do
        sp.spiral_sched_close(sched, g)
        sp.spiral_sched_free(sched)
    finally:
        pair.close()


def test_games_forked_from_a_shared_prompt():
    """A system prompt is appended once to a template game; games forked from it share its full pages
    (no copy, no new pages) and get a private copy of its partly filled last page.  Each fork then plays a
    turn of its own through the scheduler; the oracle, which appends prompt + observation per game from
    scratch, must choose the same tokens.  Pages are counted once while shared and all come back."""
    desc = synth.shape("tiny_bias")
    n_forks, max_batch = 6, 16
    pair = Pair(desc, max_batch=max_batch, max_ctx=160, n_games=8, pool_pages=40)
    try:
        sp, V = pair.sp, desc["vocab"]
        free0 = sp.spiral_kv_free_pages(pair.kv)
        sched = sp.spiral_sched_create(pair.ctx, pair.kv, -1)
        zeros = torch.zeros(max_batch, V, dtype=torch.float32, device="cuda")
        prompt = synth.token_ids(17, 0, 53, V).tolist()              # 3 full pages + 5 tokens
        template = sp.spiral_sched_open(sched)
        # the template's context: the prompt (all of it cached: a one-token budget, whose sample the next
        # turn of a fork would append first -- so the template is filled with spiral_prefill instead)
        sp.spiral_prefill(pair.ctx, pair.kv, [template], torch.tensor(prompt, dtype=torch.int32).cuda(), [0, len(prompt)])
        used_by_template = free0 - sp.spiral_kv_free_pages(pair.kv)
        assert used_by_template == 4
        forks = [sp.spiral_sched_fork(sched, template) for _ in range(n_forks)]
        assert len(set(forks + [template])) == n_forks + 1
        # three shared pages cost nothing; every fork copied the partly filled fourth page
        assert free0 - sp.spiral_kv_free_pages(pair.kv) == used_by_template + n_forks
        for g in forks:
            assert sp.spiral_kv_seq_len(pair.kv, g) == len(prompt)
        with pytest.raises(sp.SpiralError) as e:                     # cutting a game inside a shared page
            sp.spiral_kv_truncate(pair.kv, [forks[0]], [20])
        assert e.value.code == sp.SPIRAL_ERR_UNSUPPORTED
        obs = {g: synth.token_ids(17, 10 + i, 7 + 9 * i, V).tolist() for i, g in enumerate(forks)}
        for g in forks:
            sp.spiral_sched_turn(sched, g, obs[g], 6)
        sp.spiral_sched_turn(sched, template, [5, 6, 7], 3)          # the template itself keeps playing too
        responses = {}
        for _ in range(40):
            sp.spiral_sched_tick(sched, zeros, 1.0)
            while True:
                done = sp.spiral_sched_poll(sched)
                if done is None:
                    break
                responses[done[0]] = done[1]
            if len(responses) == n_forks + 1:
                break
        assert len(responses) == n_forks + 1
        flips = 0
        for g in forks + [template]:
            cache = pair.oracle.new_cache(160)
            logits = pair.oracle.prefill(cache, prompt + (obs[g] if g in obs else [5, 6, 7]))
            for tok in responses[g]:
                best = int(np.argmax(logits))
                if best != tok:
                    flips += 1
                    assert float(logits[best] - logits[tok]) <= 4 * TOL_MAX_ABS, (g, tok, best)
                logits = pair.oracle.decode_step(cache, tok)
        assert flips <= 1
        # releasing the template first leaves the shared pages with the forks
        sp.spiral_sched_close(sched, template)
        assert free0 - sp.spiral_kv_free_pages(pair.kv) >= 3 + n_forks
        for g in forks:
            sp.spiral_sched_close(sched, g)
        assert sp.spiral_kv_free_pages(pair.kv) == free0
        rc, detail = sp.spiral_last_status(pair.ctx)
        assert rc == 0, detail
        sp.spiral_sched_free(sched)
    finally:
        pair.close()


def test_multi_turn_episode_configuration_sampled_games():
    """The multi-turn self-play configuration at its own sizes on the tiny decoder: 256 concurrent games
    of 8 turns, each turn a 150-token observation and a move of length uniform in [64, 512] (contexts grow
    to about 5 K tokens, ragged; finished games leave), page size 16, a pool that cannot hold every game's
    worst case, so later turns queue for pages.  Greedy decoding; the oracle replays a sample of games
    in full and must choose the same token at every generated position."""
    desc = synth.shape("tiny")
    n_games, n_turns, obs_len, max_batch = 256, 8, 150, 256
    max_ctx = n_turns * (obs_len + 512) + 16
    worst_pages = n_games * ((max_ctx + 15) // 16)
    pair = Pair(desc, max_batch=max_batch, max_ctx=max_ctx, n_games=n_games, pool_pages=int(0.45 * worst_pages))
    try:
        sp, V = pair.sp, desc["vocab"]
        free0 = sp.spiral_kv_free_pages(pair.kv)
        sched = sp.spiral_sched_create(pair.ctx, pair.kv, -1)
        zeros = torch.zeros(max_batch, V, dtype=torch.float32, device="cuda")
        budget = [synth.lengths(8, 30 + t, n_games, 64, 512) for t in range(n_turns)]
        games = [sp.spiral_sched_open(sched) for _ in range(n_games)]
        sampled = [0, 41, 128, 200, 255]
        history = {g: [] for g in games}
        turn_of = {g: 0 for g in games}

        def queue_turn(g):
            t = turn_of[g]
            obs = synth.token_ids(8, 1000 * t + g, obs_len, V).tolist()
            sp.spiral_sched_turn(sched, g, obs, budget[t][g])
            history[g].append([obs, None])
        for g in games:
            queue_turn(g)
        stream = torch.cuda.Stream()
        left, ticks, waited, max_running = n_games, 0, 0, 0
        with torch.cuda.stream(stream):
            while left:
                sp.spiral_sched_tick(sched, zeros, 1.0, stream)
                ticks += 1
                assert ticks < 20000
                if ticks % 64 == 0:
                    st = sp.spiral_sched_stats(sched)
                    waited = max(waited, st["waiting"])
                    max_running = max(max_running, st["running"])
                    assert st["reserved_pages"] <= st["free_pages"]
                while True:
                    done = sp.spiral_sched_poll(sched)
                    if done is None:
                        break
                    g, resp, why = done
                    assert why == 2 and len(resp) == budget[turn_of[g]][g]
                    history[g][-1][1] = resp
                    turn_of[g] += 1
                    if turn_of[g] < n_turns:
                        queue_turn(g)
                    else:
                        sp.spiral_sched_close(sched, g)           # a finished game leaves and frees its pages
                        left -= 1
        stream.synchronize()
        rc, detail = sp.spiral_last_status(pair.ctx)
        assert rc == 0, detail
        stats = sp.spiral_sched_stats(sched)
        assert sp.spiral_kv_free_pages(pair.kv) == free0
        assert stats["decoded"] == sum(sum(b[g] for b in budget) for g in range(n_games))
        assert waited > 0 and max_running > n_games // 2        # the pool made turns wait; the batch still ran wide
        flips, total = 0, 0
        for g in sampled:
            cache = pair.oracle.new_cache(max_ctx)
            for obs, resp in history[g]:
                logits = pair.oracle.prefill(cache, obs)
                for tok in resp:
                    best = int(np.argmax(logits))
                    total += 1
                    if best != tok:
                        flips += 1
                        assert float(logits[best] - logits[tok]) <= 4 * TOL_MAX_ABS, (g, tok, best)
                    logits = pair.oracle.decode_step(cache, tok)
        print("episode configuration: %d ticks, %d tokens decoded, %d checked on %d games, %d flips, most waiting %d" %
              (ticks, stats["decoded"], total, len(sampled), flips, waited))
        assert flips <= allowed_flips(total)
        sp.spiral_sched_free(sched)
    finally:
        pair.close()


def test_scheduler_returns_log_probabilities_of_its_samples():
    """With log-probability collection on, every response comes back with log pi(token) under the sampling
    policy (temperature 0.8, real Gumbel noise).  The oracle replays each game along the tokens the GPU
    drew and computes log softmax(logits / T)[token] itself.  Batches shrink from 20 games (tensor-core
    LM head) to a few (CUDA-core head) as games finish, so both producers of the value are covered."""
    desc = synth.shape("tiny_qknorm")
    n_games, max_batch, T = 20, 24, 0.8
    pair = Pair(desc, max_batch=max_batch, max_ctx=128, n_games=n_games)
    try:
        sp, V = pair.sp, desc["vocab"]
        sched = sp.spiral_sched_create(pair.ctx, pair.kv, -1)
        sp.spiral_sched_collect_logprob(sched, True)
        budget = synth.lengths(9, 1, n_games, 2, 30)
        games = [sp.spiral_sched_open(sched) for _ in range(n_games)]
        obs = {g: synth.token_ids(9, 10 + g, 5 + 3 * (g % 7), V).tolist() for g in games}
        for g in games:
            sp.spiral_sched_turn(sched, g, obs[g], budget[g])
        out = {}
        for tick in range(200):
            sp.spiral_sched_tick(sched, synth.gumbel_noise(9, tick, max_batch, V, "cuda"), T)
            while True:
                done = sp.spiral_sched_poll_logprob(sched)
                if done is None:
                    break
                out[done[0]] = (done[1], done[2])
            if len(out) == n_games:
                break
        assert len(out) == n_games
        worst = 0.0
        for g in games:
            toks, lps = out[g]
            assert len(toks) == len(lps) == budget[g]
            cache = pair.oracle.new_cache(128)
            logits = pair.oracle.prefill(cache, obs[g])
            for tok, lp in zip(toks, lps):
                worst = max(worst, abs(lp - pair.oracle_mod.log_prob(logits, tok, T)))
                logits = pair.oracle.decode_step(cache, tok)
        print("scheduler log-probabilities: worst |delta| %.2e" % worst)
        assert worst <= 2 * TOL_MAX_ABS
        rc, detail = sp.spiral_last_status(pair.ctx)
        assert rc == 0, detail
        for g in games:
            sp.spiral_sched_close(sched, g)
        sp.spiral_sched_free(sched)
    finally:
        pair.close()


def test_turn_waiting_behind_a_shut_gate_is_not_starved():
    """Every running turn reaches its budget on the same step while another turn waits in the queue behind a
    shut admission gate (the batch has not drained, too few tokens are waiting).  Nothing can be launched for the
    running turns, nothing is admitted: the scheduler has to read the last step's tokens and retire the turns --
    which is what opens the gate -- instead of waiting for a launch that never comes."""
    desc = synth.shape("tiny_qknorm")
    n_games = 8
    pair = Pair(desc, max_batch=n_games, max_ctx=128, n_games=n_games)
    try:
        sp, V = pair.sp, desc["vocab"]
        sched = sp.spiral_sched_create(pair.ctx, pair.kv, -1)
        sp.spiral_sched_policy(sched, 100000, 0)         # gate: open only when nothing is running
        zeros = torch.zeros(n_games, V, dtype=torch.float32, device="cuda")
        games = [sp.spiral_sched_open(sched) for _ in range(n_games)]
        for g in games:
            sp.spiral_sched_turn(sched, g, synth.token_ids(2, g, 5, V).tolist(), 2 if g == 0 else 6)
        stream = torch.cuda.Stream()
        polled, requeued, ticks = {}, False, 0
        with torch.cuda.stream(stream):
            while len(polled) < n_games + 1:
                sp.spiral_sched_tick(sched, zeros, 1.0, stream)
                ticks += 1
                assert ticks < 60, (ticks, polled, sp.spiral_sched_stats(sched))
                while True:
                    done = sp.spiral_sched_poll(sched)
                    if done is None:
                        break
                    g, resp, why = done
                    polled[(g, len(polled))] = len(resp)
                    if g == 0 and not requeued:          # the short turn comes back with a new observation
                        sp.spiral_sched_turn(sched, 0, synth.token_ids(2, 99, 30, V).tolist(), 3)
                        requeued = True
        stream.synchronize()
        assert sorted(polled.values()) == [2, 3] + [6] * 7
        assert sp.spiral_last_status(pair.ctx) == (0, 0)
        for g in games:
            sp.spiral_sched_close(sched, g)
        sp.spiral_sched_free(sched)
    finally:
        pair.close()
