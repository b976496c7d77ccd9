"""Parity of the CUDA path (through the C ABI) with the CPU oracle on identical seeded inputs."""
import numpy as np
import pytest
import torch

import synth
from harness import TOL_MAX_ABS, TOL_REL_RMS, TOL_TOKEN_AGREE, Pair, compare_logits

pytestmark = pytest.mark.gpu


def _run_teacher_forced(pair: Pair, games, prompts, n_steps, seed, temperature=1.0, use_prefill=True, stream=None):
    """Prefill the prompts, then n_steps decode steps feeding seeded random tokens (teacher forcing).
    Returns (worst max|delta|, worst rel rms, token agreement, mismatch records).
    With a side stream the library may replay its recorded CUDA graph of the step (it cannot on
    the default stream); the torch copies are put on the same stream."""
    if stream is not None:
        torch.cuda.synchronize()
        with torch.cuda.stream(stream):
            out = _run_teacher_forced_on(pair, games, prompts, n_steps, seed, temperature, stream)
        stream.synchronize()
        return out
    return _run_teacher_forced_on(pair, games, prompts, n_steps, seed, temperature, None)


def _run_teacher_forced_on(pair: Pair, games, prompts, n_steps, seed, temperature, stream):
    sp, desc = pair.sp, pair.desc
    V = desc["vocab"]
    n = len(games)
    flat = torch.cat([torch.tensor(p, dtype=torch.int32) for p in prompts]).cuda()
    offsets = np.concatenate([[0], np.cumsum([len(p) for p in prompts])]).tolist()
    last = torch.empty(n, V, dtype=torch.float32, device="cuda")
    sp.spiral_prefill(pair.ctx, pair.kv, games, flat, offsets, last, stream)
    worst_abs, worst_rms = 0.0, 0.0
    last = last.cpu().numpy()
    for i, g in enumerate(games):
        ref = pair.oracle.prefill(pair.oracle_cache(g), prompts[i])
        a, r = compare_logits(last[i], ref)
        worst_abs, worst_rms = max(worst_abs, a), max(worst_rms, r)
        assert sp.spiral_kv_seq_len(pair.kv, g) == len(prompts[i])
    agree, total, mism = 0, 0, []
    tok_out = torch.empty(n, dtype=torch.int32, device="cuda")
    logits = torch.empty(n, V, dtype=torch.float32, device="cuda")
    for s in range(n_steps):
        tok_in = synth.token_ids(seed, 1000 + s, n, V, stream=synth.STREAM_TEACHER)
        noise = synth.gumbel_noise(seed, s, n, V)
        sp.spiral_decode_step(pair.ctx, pair.kv, games, tok_in.cuda(), noise.cuda(), temperature, tok_out, logits, stream)
        got_tok = tok_out.cpu().numpy()
        got_logits = logits.cpu().numpy()
        for i, g in enumerate(games):
            ref = pair.oracle.decode_step(pair.oracle_cache(g), int(tok_in[i]))
            a, r = compare_logits(got_logits[i], ref)
            worst_abs, worst_rms = max(worst_abs, a), max(worst_rms, r)
            tok, _, gap = pair.oracle_mod.sample(ref, noise[i].numpy(), temperature)
            total += 1
            if tok == got_tok[i]:
                agree += 1
            else:
                mism.append((s, i, tok, int(got_tok[i]), gap))
    rc, detail = sp.spiral_last_status(pair.ctx)
    assert rc == 0, (rc, detail)
    return worst_abs, worst_rms, agree / total, mism, total


def allowed_flips(total: int) -> int:
    """Token disagreements tolerated among `total` sampled steps: the 0.5 % bar itself for large
    samples; for small samples the same rate plus three Poisson standard deviations, since a
    single legitimate near-tie would otherwise exceed 0.5 % of a few dozen steps."""
    lam = (1.0 - TOL_TOKEN_AGREE) * total
    return int(lam) if total >= 4000 else int(lam + 3.0 * lam ** 0.5 + 1.0)


def _check(worst_abs, worst_rms, agree, mism, total=None):
    assert worst_abs <= TOL_MAX_ABS, worst_abs
    assert worst_rms <= TOL_REL_RMS, worst_rms
    if total is None:
        assert agree >= TOL_TOKEN_AGREE, (agree, mism)
    else:
        assert len(mism) <= allowed_flips(total), (len(mism), total, mism)
    # a flipped token is only acceptable when the oracle's top-2 gap is within the logit error
    for (_, _, _, _, gap) in mism:
        assert gap <= 4 * worst_abs, mism


@pytest.mark.parametrize("shape_name,kv_bf16", [("tiny", False), ("tiny_qknorm", False), ("tiny_bias", False),
                                                ("tiny", True), ("tiny_qknorm", True)])
def test_tiny_config_end_to_end(shape_name, kv_bf16):
    """Tiny decoder, batch 4, prompts of 64..128 random ids, 32 teacher-forced decode steps."""
    desc = synth.shape(shape_name)
    pair = Pair(desc, max_batch=4, max_ctx=192, n_games=6, kv_bf16=kv_bf16)
    try:
        games = [4, 1, 5, 2]                      # not 0..3 and not sorted: exercises the indirection
        lens = synth.lengths(synth.MASTER_SEED, 1, 4, 64, 128)
        prompts = [synth.token_ids(synth.MASTER_SEED, 10 + i, lens[i], desc["vocab"]).tolist() for i in range(4)]
        res = _run_teacher_forced(pair, games, prompts, 32, synth.MASTER_SEED)
        print(shape_name, "max|d| %.2e rel-rms %.2e agree %.4f" % res[:3], res[3])
        _check(*res[:4])
        for g, p in zip(games, prompts):
            assert pair.sp.spiral_kv_seq_len(pair.kv, g) == len(p) + 32
    finally:
        pair.close()


def test_sampling_temperature_and_ties():
    """Temperature divides the logits before the noise is added; ties go to the lowest index."""
    desc = synth.shape("tiny")
    pair = Pair(desc, max_batch=4, max_ctx=64, n_games=4)
    try:
        sp, V = pair.sp, desc["vocab"]
        games = [0, 1, 2]
        tok_in = torch.tensor([5, 6, 7], dtype=torch.int32)
        tok_out = torch.empty(3, dtype=torch.int32, device="cuda")
        logits = torch.empty(3, V, dtype=torch.float32, device="cuda")
        for step, T in enumerate((0.6, 1.0, 2.5)):
            noise = synth.gumbel_noise(7, step, 3, V)
            sp.spiral_decode_step(pair.ctx, pair.kv, games, tok_in.cuda(), noise.cuda(), T, tok_out, logits)
            lg = logits.cpu().numpy().astype(np.float64)
            for i in range(3):
                # the sampler must agree with the oracle's sampler applied to the GPU's own logits exactly
                tok, _, _ = pair.oracle_mod.sample(lg[i], noise[i].numpy(), T)
                assert tok == int(tok_out[i])
        # huge constant noise on two entries -> exact tie in fp32 -> lowest index wins
        noise = torch.zeros(3, V)
        noise[:, 100] = 1e9
        noise[:, 37] = 1e9
        sp.spiral_decode_step(pair.ctx, pair.kv, games, tok_in.cuda(), noise.cuda(), 1.0, tok_out, None)
        assert tok_out.cpu().tolist() == [37, 37, 37]
    finally:
        pair.close()


@pytest.mark.parametrize("hq,hkv,hd,kv_bf16", [(4, 2, 64, False), (8, 2, 128, False), (7, 1, 128, False),
                                                (8, 8, 64, True), (8, 1, 128, False), (8, 2, 128, True)])
def test_attention_component_against_oracle(hq, hkv, hd, kv_bf16):
    """Paged split-context attention kernel on synthetic bf16 caches at lengths around page and
    chunk boundaries, several games of different length in one launch."""
    desc = synth.shape("tiny", n_q_heads=hq, n_kv_heads=hkv, head_dim=hd, n_layers=2)
    lens = [1, 15, 16, 17, 255, 1000, 4097, 64]
    pair = Pair(desc, max_batch=8, max_ctx=4112, n_games=8, pool_pages=sum((l + 15) // 16 for l in lens) + 4,
                kv_bf16=kv_bf16)
    try:
        sp = pair.sp
        for g, n_tok in enumerate(lens):
            cache = pair.oracle_cache(g)
            for layer in range(2):
                k, v = synth.synthetic_kv(5, g, layer, n_tok, hkv, hd)
                if not kv_bf16:
                    # fp16 pages hold 11-bit mantissas: perturb the bf16 values so the low bits are used
                    k = (k.float() * (1 + 2.0 ** -10)).to(torch.float16)
                    v = (v.float() * (1 - 2.0 ** -10)).to(torch.float16)
                cache.load(layer, k, v)
                sp.spiral_kv_load(pair.ctx, pair.kv, g, layer, k.cuda(), v.cuda())
            cache.set_len(n_tok)
        q = (synth.uniform_bf16(9, 1, 8 * hq * hd, 3.0).float().view(8, hq, hd)
             + 1e-3 * synth.uniform_bf16(9, 2, 8 * hq * hd, 1.0).float().view(8, hq, hd))
        for layer in (1, 0):
            for ctx_len in (lens, [max(1, l // 2) for l in lens]):
                out = sp.spiral_attention(pair.ctx, pair.kv, layer, list(range(8)), ctx_len, q.cuda()).cpu().numpy()
                for g in range(8):
                    ref = pair.oracle_mod.attention(q[g].double().numpy(), pair.oracle_cache(g), layer, ctx_len[g])
                    np.testing.assert_allclose(out[g], ref, rtol=0, atol=3e-4)
        rc, detail = sp.spiral_last_status(pair.ctx)
        assert rc == 0, detail
    finally:
        pair.close()


@pytest.mark.parametrize("rows,k,n", [(256, 256, 4), (1376, 256, 3), (37, 688, 1), (4096, 256, 8), (300, 1024, 17)])
def test_linear_cuda_core_path_against_oracle(rows, k, n):
    desc = synth.shape("tiny")
    pair = Pair(desc, max_batch=32, max_ctx=32, n_games=1)
    try:
        w = synth.normal_bf16(3, 1, rows * k, 0.05).view(rows, k)
        x = synth.normal_bf16(3, 2, n * k, 1.0).view(n, k).to(torch.float16)   # exact: 8-bit mantissas
        y = pair.sp.spiral_linear(pair.ctx, w.cuda(), x.cuda(), path=1).cpu().numpy()
        for b in range(n):
            ref = pair.oracle_mod.matvec(w, x[b].double().numpy())
            np.testing.assert_allclose(y[b], ref, rtol=0, atol=2e-5 * np.abs(ref).max() + 1e-6)
    finally:
        pair.close()


def test_error_codes_and_page_accounting():
    desc = synth.shape("tiny")
    pair = Pair(desc, max_batch=4, max_ctx=64, n_games=4, pool_pages=5)
    try:
        sp, V = pair.sp, desc["vocab"]
        tok = torch.zeros(4, dtype=torch.int32, device="cuda")
        out = torch.zeros(4, dtype=torch.int32, device="cuda")
        noise = torch.zeros(4, V, device="cuda")
        assert sp.spiral_kv_free_pages(pair.kv) == 5
        with pytest.raises(sp.SpiralError) as e:
            sp.spiral_decode_step(pair.ctx, pair.kv, [0, 0], tok, noise, 1.0, out)     # duplicate id
        assert e.value.code == sp.SPIRAL_ERR_INVALID
        with pytest.raises(sp.SpiralError) as e:
            sp.spiral_decode_step(pair.ctx, pair.kv, [0, 9], tok, noise, 1.0, out)     # id out of range
        assert e.value.code == sp.SPIRAL_ERR_INVALID
        with pytest.raises(sp.SpiralError) as e:
            sp.spiral_decode_step(pair.ctx, pair.kv, [0, 1], tok, noise, 0.0, out)     # T <= 0
        assert e.value.code == sp.SPIRAL_ERR_INVALID
        assert sp.spiral_kv_free_pages(pair.kv) == 5
        # 40 tokens for game 0 -> 3 pages; 33 for game 1 would need 3 more -> pool exhausted, nothing changes
        toks = synth.token_ids(1, 1, 80, V).cuda()
        sp.spiral_prefill(pair.ctx, pair.kv, [0], toks, [0, 40])
        assert sp.spiral_kv_free_pages(pair.kv) == 2 and sp.spiral_kv_seq_len(pair.kv, 0) == 40
        with pytest.raises(sp.SpiralError) as e:
            sp.spiral_prefill(pair.ctx, pair.kv, [1], toks, [0, 33])
        assert e.value.code == sp.SPIRAL_ERR_OOM
        assert sp.spiral_kv_free_pages(pair.kv) == 2 and sp.spiral_kv_seq_len(pair.kv, 1) == 0
        sp.spiral_prefill(pair.ctx, pair.kv, [1, 2], toks, [0, 16, 32])
        assert sp.spiral_kv_free_pages(pair.kv) == 0
        with pytest.raises(sp.SpiralError) as e:                                      # both need a new page
            sp.spiral_decode_step(pair.ctx, pair.kv, [1, 2], tok, noise, 1.0, out)
        assert e.value.code == sp.SPIRAL_ERR_OOM
        assert sp.spiral_kv_seq_len(pair.kv, 1) == 16
        sp.spiral_kv_release(pair.kv, [0])
        assert sp.spiral_kv_free_pages(pair.kv) == 3 and sp.spiral_kv_seq_len(pair.kv, 0) == 0
        sp.spiral_decode_step(pair.ctx, pair.kv, [1, 2], tok, noise, 1.0, out)
        assert sp.spiral_kv_free_pages(pair.kv) == 1
        sp.spiral_kv_release(pair.kv, [1, 2])
        assert sp.spiral_kv_free_pages(pair.kv) == 5
        rc, detail = sp.spiral_last_status(pair.ctx)
        assert rc == 0, detail
    finally:
        pair.close()


def _two_good_steps(pair, games, first_seed):
    """Prefill + decode steps against the oracle on a context that has just reported a device-side finding."""
    desc = pair.desc
    prompts = [synth.token_ids(first_seed, 70 + i, 5 + 2 * i, desc["vocab"]).tolist() for i in range(len(games))]
    res = _run_teacher_forced(pair, games, prompts, 2, first_seed + 1)
    _check(*res)


def test_bad_token_id_is_reported_and_the_context_stays_usable():
    """A token id outside the vocabulary is a caller error the host cannot see (the ids live on the device): the
    embedding kernel reads token 0 instead, nothing faults, spiral_last_status reports the device-side check once,
    and after rolling the games back the same context decodes correctly."""
    desc = synth.shape("tiny_qknorm")
    pair = Pair(desc, max_batch=24, max_ctx=64, n_games=24)
    try:
        sp, V = pair.sp, desc["vocab"]
        games = list(range(20))
        tok = synth.token_ids(3, 1, 20, V).cuda()
        tok[7] = V + 5
        tok[11] = -2
        out = torch.empty(20, dtype=torch.int32, device="cuda")
        sp.spiral_decode_step(pair.ctx, pair.kv, games, tok, torch.zeros(20, V, device="cuda"), 1.0, out)
        rc, detail = sp.spiral_last_status(pair.ctx)
        assert rc == sp.SPIRAL_ERR_DEVICE_CHECK and detail == 1, (rc, detail)
        assert sp.spiral_last_status(pair.ctx) == (0, 0)                     # reported once, then cleared
        assert ((out.cpu() >= 0) & (out.cpu() < V)).all()
        sp.spiral_kv_truncate(pair.kv, games, [0] * 20)
        _two_good_steps(pair, games, 31)
    finally:
        pair.close()


@pytest.mark.parametrize("which", [0, 1])
def test_a_wait_that_runs_out_is_reported_and_the_context_stays_usable(which):
    """Every device-side wait is bounded.  spiral_selftest_wait_timeout lowers the bound to a millisecond and runs
    the GEMM kernel (0) or the attention kernel (1) with one load deliberately left out, so that a wait must run
    out: the kernel has to raise its abort flag, let every role leave its loop, wait for the copies in flight,
    free its tensor memory and return.  The status word then says timeout, and the same context goes on to decode
    correctly (batch of 20: tensor-core GEMMs, split attention)."""
    desc = synth.shape("tiny_qknorm")
    pair = Pair(desc, max_batch=24, max_ctx=64, n_games=24)
    try:
        sp, V = pair.sp, desc["vocab"]
        games = list(range(20))
        # some context for game 0 (the attention self-test reads it)
        toks = synth.token_ids(5, 1, 40, V).cuda()
        sp.spiral_prefill(pair.ctx, pair.kv, [0], toks, [0, 40])
        assert sp.spiral_last_status(pair.ctx) == (0, 0)
        sp.spiral_selftest_wait_timeout(pair.ctx, pair.kv, which)
        rc, detail = sp.spiral_last_status(pair.ctx)
        assert rc == sp.SPIRAL_ERR_TIMEOUT and detail in (16, 17, 18), (rc, detail)
        assert sp.spiral_last_status(pair.ctx) == (0, 0)
        sp.spiral_kv_truncate(pair.kv, [0], [0])
        _two_good_steps(pair, games, 41 + which)
    finally:
        pair.close()


def test_plain_launches_and_graph_replay_agree(monkeypatch):
    """SPIRAL_NO_GRAPH=1 (what the profiling commands use to see every kernel) launches each step kernel by kernel;
    by default the step is replayed from a recorded CUDA graph from its second use on.  Same tokens, same logits."""
    desc = synth.shape("tiny_qknorm")
    outs = []
    for no_graph in ("1", "0"):
        monkeypatch.setenv("SPIRAL_NO_GRAPH", no_graph)
        pair = Pair(desc, max_batch=20, max_ctx=64, n_games=20)
        try:
            sp, V = pair.sp, desc["vocab"]
            games = list(range(20))
            stream = torch.cuda.Stream()
            torch.cuda.synchronize()
            with torch.cuda.stream(stream):
                toks = synth.token_ids(6, 1, 20 * 11, V).cuda()
                sp.spiral_prefill(pair.ctx, pair.kv, games, toks, [11 * i for i in range(21)], None, stream)
                tok = synth.token_ids(6, 2, 20, V).cuda()
                out = torch.empty(20, dtype=torch.int32, device="cuda")
                logits = torch.empty(20, V, dtype=torch.float32, device="cuda")
                l0 = sp.spiral_launch_count(pair.ctx)
                rec = []
                for s_ in range(4):
                    sp.spiral_decode_step(pair.ctx, pair.kv, games, tok, synth.gumbel_noise(6, s_, 20, V, "cuda"), 1.0, out, logits, stream)
                    stream.synchronize()
                    rec.append((out.cpu().clone(), logits.cpu().clone()))
                    tok = out.clone()
            outs.append(rec)
            assert sp.spiral_launch_count(pair.ctx) > l0
            assert sp.spiral_last_status(pair.ctx) == (0, 0)
        finally:
            pair.close()
    for (t0, l0_), (t1, l1_) in zip(*outs):
        assert torch.equal(t0, t1) and torch.equal(l0_, l1_)


def test_read_only_bandwidth_probe():
    """spiral_read_ceiling streams a caller-owned buffer and reports a rate: linear copies and tiled boxes, the three
    chunk orders; sizes the SM cannot hold and misaligned buffers are refused before anything is launched."""
    import paper_2506_24119_b200 as sp
    buf = torch.zeros(512 << 20, dtype=torch.uint8, device="cuda")
    rates = []
    for tiled in (False, True):
        for order in (0, 1, 2):
            rates.append(sp.spiral_read_ceiling(0, buf, 16384, 6, 1, order, tiled, 2))
    assert all(1000.0 < r < 20000.0 for r in rates), rates           # GB/s: an HBM device, and not a no-op
    with pytest.raises(sp.SpiralError) as e:
        sp.spiral_read_ceiling(0, buf, 32768, 8, 1, 0, False, 1)      # 8 x 32 KB does not fit an SM's shared memory
    assert e.value.code == sp.SPIRAL_ERR_UNSUPPORTED
    with pytest.raises(sp.SpiralError) as e:
        sp.spiral_read_ceiling(0, buf[64:], 16384, 4, 1, 0, False, 1)  # not 128-byte aligned
    assert e.value.code == sp.SPIRAL_ERR_INVALID
    with pytest.raises(sp.SpiralError) as e:
        sp.spiral_read_ceiling(0, buf, 1000, 4, 1, 0, False, 1)       # stage size not a multiple of 1024
    assert e.value.code == sp.SPIRAL_ERR_INVALID


def test_multi_turn_cache_survives_and_matches_oracle():
    """Turns: append an observation (prefill), decode a move, repeat; games leave when done."""
    desc = synth.shape("tiny_qknorm")
    n_games, turns = 6, 3
    pair = Pair(desc, max_batch=8, max_ctx=256, n_games=n_games)
    try:
        sp, V = pair.sp, desc["vocab"]
        free0 = sp.spiral_kv_free_pages(pair.kv)
        move_len = [synth.lengths(5, 20 + t, n_games, 3, 12) for t in range(turns)]
        n_turns = synth.lengths(5, 19, n_games, 1, turns)       # game g plays n_turns[g] turns
        worst_abs, agree, total = 0.0, 0, 0
        for t in range(turns):
            games = [g for g in range(n_games) if n_turns[g] > t]
            obs = [synth.token_ids(5, 100 * t + g, 21, V).tolist() for g in games]
            flat = torch.tensor(sum(obs, []), dtype=torch.int32).cuda()
            offs = np.concatenate([[0], np.cumsum([len(o) for o in obs])]).tolist()
            sp.spiral_prefill(pair.ctx, pair.kv, games, flat, offs)
            for g, o in zip(games, obs):
                pair.oracle.prefill(pair.oracle_cache(g), o)
            step = 0
            while True:
                active = [g for g in games if move_len[t][g] > step]
                if not active:
                    break
                n = len(active)
                tok_in = synth.token_ids(5, 5000 + 100 * t + step, n, V, stream=synth.STREAM_TEACHER)
                noise = synth.gumbel_noise(5, 100 * t + step, n, V)
                tok_out = torch.empty(n, dtype=torch.int32, device="cuda")
                logits = torch.empty(n, V, dtype=torch.float32, device="cuda")
                sp.spiral_decode_step(pair.ctx, pair.kv, active, tok_in.cuda(), noise.cuda(), 1.0, tok_out, logits)
                lg = logits.cpu().numpy()
                for i, g in enumerate(active):
                    ref = pair.oracle.decode_step(pair.oracle_cache(g), int(tok_in[i]))
                    a, _ = compare_logits(lg[i], ref)
                    worst_abs = max(worst_abs, a)
                    total += 1
                    agree += int(pair.oracle_mod.sample(ref, noise[i].numpy(), 1.0)[0] == int(tok_out[i]))
                step += 1
            done = [g for g in games if n_turns[g] == t + 1]
            sp.spiral_kv_release(pair.kv, done)
        assert worst_abs <= TOL_MAX_ABS and agree / total >= TOL_TOKEN_AGREE, (worst_abs, agree, total)
        assert sp.spiral_kv_free_pages(pair.kv) == free0          # no page leaked
    finally:
        pair.close()


@pytest.mark.parametrize("rows,k,n", [(128, 64, 16), (256, 256, 16), (1376, 256, 24), (512, 688, 17), (4096, 256, 128),
                                      (640, 1024, 100), (384, 2560, 128), (2560, 512, 256), (300, 320, 3), (130, 128, 20),
                                      (259, 192, 140)])
def test_linear_tensor_core_path_against_oracle(rows, k, n):
    """tcgen05 skinny GEMM (stream-K pieces reduced by the entry point): ragged row tiles, ragged
    last k block, batch sizes that are not multiples of 16, the largest batch, and row counts that are no
    multiple of 4 (their pieces cannot leave through TMA stores: the kernel's plain-store epilogue)."""
    desc = synth.shape("tiny")
    pair = Pair(desc, max_batch=256, max_ctx=32, n_games=1)
    try:
        w = synth.normal_bf16(3, 1, rows * k, 0.05).view(rows, k)
        x = (synth.normal_bf16(3, 2, n * k, 1.0).float() * (1 + 2.0 ** -9)).view(n, k).to(torch.float16)
        y = pair.sp.spiral_linear(pair.ctx, w.cuda(), x.cuda(), path=2).cpu().numpy()
        rc, detail = pair.sp.spiral_last_status(pair.ctx)
        assert rc == 0, detail
        for b in range(n):              # every batch column: every TMEM column group of the epilogue
            ref = pair.oracle_mod.matvec(w, x[b].double().numpy())
            np.testing.assert_allclose(y[b], ref, rtol=0, atol=2e-5 * np.abs(ref).max() + 1e-6)
        # a second call on the same matrix with new contents must not reuse the old fp16 copy
        w2 = synth.normal_bf16(4, 1, rows * k, 0.05).view(rows, k).cuda()
        wd = w.cuda()
        wd.copy_(w2)
        y2 = pair.sp.spiral_linear(pair.ctx, wd, x.cuda(), path=2).cpu().numpy()
        ref = pair.oracle_mod.matvec(w2.cpu(), x[n - 1].double().numpy())
        np.testing.assert_allclose(y2[n - 1], ref, rtol=0, atol=2e-5 * np.abs(ref).max() + 1e-6)
    finally:
        pair.close()


@pytest.mark.parametrize("shape_name,n_games", [("tiny", 20), ("tiny_qknorm", 33), ("tiny_bias", 16)])
def test_batched_step_on_tensor_cores(shape_name, n_games):
    """Enough games for the tensor-core GEMMs and the fused LM head + Gumbel-argmax to carry the
    step: teacher-forced parity of logits and sampled tokens, then a run without the logits
    pointer must sample the same tokens."""
    desc = synth.shape(shape_name)
    pair = Pair(desc, max_batch=n_games, max_ctx=64, n_games=n_games)
    try:
        games = list(range(n_games))[::-1]
        lens = synth.lengths(synth.MASTER_SEED, 3, n_games, 5, 20)
        prompts = [synth.token_ids(synth.MASTER_SEED, 70 + i, lens[i], desc["vocab"]).tolist() for i in range(n_games)]
        res = _run_teacher_forced(pair, games, prompts, 8, synth.MASTER_SEED + 3)
        print(shape_name, "max|d| %.2e rel-rms %.2e agree %.4f" % res[:3], res[3])
        _check(*res)
        # same state twice: with and without the debug logits
        sp, V = pair.sp, desc["vocab"]
        tok_in = synth.token_ids(9, 1, n_games, V).cuda()
        noise = synth.gumbel_noise(9, 1, n_games, V).cuda()
        a = torch.empty(n_games, dtype=torch.int32, device="cuda")
        b = torch.empty_like(a)
        logits = torch.empty(n_games, V, dtype=torch.float32, device="cuda")
        before = [sp.spiral_kv_seq_len(pair.kv, g) for g in games]
        sp.spiral_decode_step(pair.ctx, pair.kv, games, tok_in, noise, 0.8, a, logits)
        sp.spiral_kv_truncate(pair.kv, games, before)
        sp.spiral_decode_step(pair.ctx, pair.kv, games, tok_in, noise, 0.8, b, None)
        assert torch.equal(a, b)
        lg = logits.cpu().numpy().astype(np.float64)
        nz = noise.cpu().numpy()
        for i in range(n_games):
            assert pair.oracle_mod.sample(lg[i], nz[i], 0.8)[0] == int(a[i])
    finally:
        pair.close()


@pytest.mark.parametrize("shape_name,n_games", [("tiny_qknorm", 5), ("tiny", 24), ("tiny_bias", 40)])
def test_recorded_step_graph_on_a_side_stream(shape_name, n_games):
    """On a non-default stream the second and later steps of a batch size are replayed from a CUDA
    graph of the launch sequence: parity with the oracle must hold exactly as for plain launches,
    for the CUDA-core path (few games) and for the tensor-core path."""
    desc = synth.shape(shape_name)
    pair = Pair(desc, max_batch=n_games, max_ctx=64, n_games=n_games)
    try:
        games = list(range(n_games))
        lens = synth.lengths(synth.MASTER_SEED, 4, n_games, 3, 18)
        prompts = [synth.token_ids(synth.MASTER_SEED, 90 + i, lens[i], desc["vocab"]).tolist() for i in range(n_games)]
        stream = torch.cuda.Stream()
        launches0 = pair.sp.spiral_launch_count(pair.ctx)
        res = _run_teacher_forced(pair, games, prompts, 10, synth.MASTER_SEED + 5, stream=stream)
        print(shape_name, "max|d| %.2e rel-rms %.2e agree %.4f" % res[:3], res[3])
        _check(*res)
        assert pair.sp.spiral_launch_count(pair.ctx) > launches0
        for g, p in zip(games, prompts):
            assert pair.sp.spiral_kv_seq_len(pair.kv, g) == len(p) + 10
    finally:
        pair.close()


@pytest.mark.parametrize("shape_name,max_batch", [("tiny_qknorm", 24), ("tiny_bias", 7)])
def test_chunked_prefill_of_few_long_prompts(shape_name, max_batch):
    """Two games with long prompts and a batch capacity above the number of games: a prefill chunk
    then carries many positions of the same game (tensor-core path at 24 slots, CUDA-core path at
    7), which must give the causal result -- checked through the logits after the prompt and the
    decode steps that follow."""
    desc = synth.shape(shape_name)
    pair = Pair(desc, max_batch=max_batch, max_ctx=160, n_games=3)
    try:
        games = [2, 0]
        prompts = [synth.token_ids(synth.MASTER_SEED, 300 + i, 97 - 40 * i, desc["vocab"]).tolist() for i in range(2)]
        res = _run_teacher_forced(pair, games, prompts, 6, synth.MASTER_SEED + 9)
        print(shape_name, "max|d| %.2e rel-rms %.2e agree %.4f" % res[:3], res[3])
        _check(*res)
    finally:
        pair.close()


@pytest.mark.parametrize("shape_name,n_games,temperature", [("tiny_qknorm", 5, 0.7), ("tiny", 24, 1.0),
                                                            ("tiny_bias", 40, 1.6)])
def test_log_prob_of_the_sampled_token(shape_name, n_games, temperature):
    """spiral_decode_step_logprob: the log-probability the sampling policy gave to each drawn token,
    accumulated in the LM-head epilogue (tensor-core path) or by the small-batch sampler.  Checked
    against the oracle's log_prob of the oracle's own logits (loose: logits differ within tolerance)
    and of the GPU's logits (tight: the reduction itself)."""
    desc = synth.shape(shape_name)
    pair = Pair(desc, max_batch=n_games, max_ctx=64, n_games=n_games)
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
        tok_out = torch.empty(n_games, dtype=torch.int32, device="cuda")
        lp = torch.full((n_games,), float("nan"), dtype=torch.float32, device="cuda")
        logits = torch.empty(n_games, V, dtype=torch.float32, device="cuda")
        for s in range(3):
            tok_in = synth.token_ids(21, s, n_games, V, stream=synth.STREAM_TEACHER)
            noise = synth.gumbel_noise(21, s, n_games, V)
            want_logits = logits if s != 1 else None          # also without the debug logits
            sp.spiral_decode_step_logprob(pair.ctx, pair.kv, games, tok_in.cuda(), noise.cuda(), temperature, tok_out,
                                          lp, want_logits)
            got_tok, got_lp = tok_out.cpu().numpy(), lp.cpu().numpy()
            lg = logits.cpu().numpy().astype(np.float64)
            for i, g in enumerate(games):
                ref = pair.oracle.decode_step(pair.oracle_cache(g), int(tok_in[i]))
                assert np.isfinite(got_lp[i]) and got_lp[i] < 0
                assert abs(got_lp[i] - pair.oracle_mod.log_prob(ref, int(got_tok[i]), temperature)) <= 2 * TOL_MAX_ABS
                if want_logits is not None:
                    assert abs(got_lp[i] - pair.oracle_mod.log_prob(lg[i], int(got_tok[i]), temperature)) <= 2e-4
        rc, detail = sp.spiral_last_status(pair.ctx)
        assert rc == 0, detail
    finally:
        pair.close()


@pytest.mark.parametrize("shape_name,n_games", [("tiny_qknorm", 5), ("tiny", 24)])
def test_host_buffer_entry_point(shape_name, n_games):
    """spiral_decode_step_host takes tokens and noise from host memory and returns host tokens (the
    noise is uploaded on a stream of its own while the layers run; the LM head waits for it).  Several
    steps on a side stream (so that the recorded graph of the layers is replayed), with pinned and with
    pageable buffers: tokens against the oracle's."""
    desc = synth.shape(shape_name)
    pair = Pair(desc, max_batch=n_games, max_ctx=64, n_games=n_games)
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
        stream = torch.cuda.Stream()
        torch.cuda.synchronize()
        mism, total = [], 0
        for s in range(5):
            tok_in = synth.token_ids(29, s, n_games, V, stream=synth.STREAM_TEACHER)
            noise = synth.gumbel_noise(29, s, n_games, V)
            tok_out = torch.full((n_games,), -1, dtype=torch.int32)
            if s % 2 == 0:
                tok_in, noise, tok_out = tok_in.pin_memory(), noise.pin_memory(), tok_out.pin_memory()
            sp.spiral_decode_step_host(pair.ctx, pair.kv, games, tok_in, noise, 1.0, tok_out, stream if s else None)
            for i, g in enumerate(games):          # the call has synchronised: the tokens are there
                ref = pair.oracle.decode_step(pair.oracle_cache(g), int(tok_in[i]))
                tok, _, gap = pair.oracle_mod.sample(ref, noise[i].numpy(), 1.0)
                total += 1
                if tok != int(tok_out[i]):
                    mism.append((s, i, tok, int(tok_out[i]), gap))
        assert len(mism) <= allowed_flips(total), mism
        for m in mism:
            assert m[4] <= 4 * TOL_MAX_ABS, mism
        rc, detail = sp.spiral_last_status(pair.ctx)
        assert rc == 0, detail
    finally:
        pair.close()


def test_attention_component_at_the_longest_configured_context():
    """The long-reasoning configuration's attention: 28 query / 4 KV heads of 128 (seven query heads per KV
    head), contexts up to 16 384 tokens (1 024 pages per game), several games of different length in one
    launch -- every work range of the split-context schedule then holds many pages of one game."""
    hq, hkv, hd = 28, 4, 128
    desc = synth.shape("tiny", n_q_heads=hq, n_kv_heads=hkv, head_dim=hd, n_layers=1, d_model=448)
    lens = [16384, 16369, 9000, 33]
    pair = Pair(desc, max_batch=4, max_ctx=16384, n_games=4, pool_pages=sum((l + 15) // 16 for l in lens) + 2)
    try:
        sp = pair.sp
        for g, n_tok in enumerate(lens):
            k, v = synth.synthetic_kv(6, g, 0, n_tok, hkv, hd)
            k = (k.float() * (1 + 2.0 ** -10)).to(torch.float16)
            v = (v.float() * (1 - 2.0 ** -10)).to(torch.float16)
            pair.oracle_cache(g).load(0, k, v)
            pair.oracle_cache(g).set_len(n_tok)
            sp.spiral_kv_load(pair.ctx, pair.kv, g, 0, k.cuda(), v.cuda())
        q = synth.uniform_bf16(9, 5, 4 * hq * hd, 3.0).float().view(4, hq, hd)
        out = sp.spiral_attention(pair.ctx, pair.kv, 0, list(range(4)), lens, q.cuda()).cpu().numpy()
        for g in range(4):
            ref = pair.oracle_mod.attention(q[g].double().numpy(), pair.oracle_cache(g), 0, lens[g])
            np.testing.assert_allclose(out[g], ref, rtol=0, atol=3e-4)
        rc, detail = sp.spiral_last_status(pair.ctx)
        assert rc == 0, detail
    finally:
        pair.close()
