"""spiral_attention_static: the attention entry point for callers that may not allocate.

Some users of the library run where cudaMalloc is not an option (a plugin whose host application
owns all device memory, a latency-critical loop that must stay clear of the allocator's locks and
implicit synchronisation, a process that has handed every free byte to one pool).  For them the
library keeps the attention scratch in a fixed array inside its own image.  This test drives that
entry point through the C ABI on a pool and block table the caller owns and checks it against the
CPU oracle's attention and against the regular entry point (spiral_attention, which works out of
the workspace spiral_init allocated), twice in a row with different queries and lengths, because
the second call finds the scratch as the first one left it; it then plants a page id outside the
pool in the caller's block table and reads the finding back with spiral_attention_static_status.
The file sorts last on purpose: a run that stops at the first failure has then already been
through every other test.
"""
import numpy as np
import pytest
import torch

import synth
from harness import Pair

pytestmark = pytest.mark.gpu

ATOL = 3e-4          # the tolerance of the attention component test


@pytest.mark.parametrize("hq,hkv,hd,kv_bf16", [(8, 2, 128, False), (4, 2, 64, True), (7, 1, 128, False)])
def test_static_attention_matches_the_oracle_and_the_workspace_entry_point(hq, hkv, hd, kv_bf16):
    desc = synth.shape("tiny", n_q_heads=hq, n_kv_heads=hkv, head_dim=hd, n_layers=2)
    lens = [1, 15, 16, 17, 255, 1000, 2049, 64]
    n = len(lens)
    max_ctx = 2064
    n_pages = sum((l + 15) // 16 for l in lens) + 4
    pair = Pair(desc, max_batch=n, max_ctx=max_ctx, n_games=n, pool_pages=n_pages, kv_bf16=kv_bf16)
    try:
        sp = pair.sp
        for g, n_tok in enumerate(lens):
            cache = pair.oracle_cache(g)
            for layer in range(2):
                k, v = synth.synthetic_kv(5, g, layer, n_tok, hkv, hd)
                if not kv_bf16:
                    k = (k.float() * (1 + 2.0 ** -10)).to(torch.float16)
                    v = (v.float() * (1 - 2.0 ** -10)).to(torch.float16)
                cache.load(layer, k, v)
                sp.spiral_kv_load(pair.ctx, pair.kv, g, layer, k.cuda(), v.cuda())
            cache.set_len(n_tok)
        # the caller's own block table, from the library's host-side bookkeeping
        max_pages = (max_ctx + 15) // 16
        table = torch.full((n, max_pages), -1, dtype=torch.int32)
        for g in range(n):
            pages = sp.spiral_kv_block_table(pair.kv, g)
            assert len(pages) == (lens[g] + 15) // 16
            table[g, :len(pages)] = torch.tensor(pages, dtype=torch.int32)
        table = table.cuda()
        kv_dtype = sp.SPIRAL_KV_BF16 if kv_bf16 else sp.SPIRAL_KV_F16
        out = torch.empty(n, hq, hd, dtype=torch.float32, device="cuda")          # caller-owned output
        for call, (layer, ctx_len) in enumerate([(1, lens), (0, [max(1, l // 2) for l in lens])]):
            q_cpu = synth.uniform_bf16(9, 10 + call, n * hq * hd, 3.0).float().view(n, hq, hd)
            q = q_cpu.cuda()
            want = sp.spiral_attention(pair.ctx, pair.kv, layer, list(range(n)), ctx_len, q)
            out.fill_(float("nan"))
            sp.spiral_attention_static(pair.pool, n_pages, 2, layer, kv_dtype, hq, hkv, hd, table, ctx_len, q, out)
            torch.cuda.synchronize()
            got, ref = out.cpu().numpy(), want.cpu().numpy()
            assert np.isfinite(got).all()
            for g in range(n):
                exact = pair.oracle_mod.attention(q_cpu[g].double().numpy(), pair.oracle_cache(g), layer, ctx_len[g])
                np.testing.assert_allclose(got[g], exact, rtol=0, atol=ATOL)
            np.testing.assert_allclose(got, ref, rtol=0, atol=ATOL)
            assert sp.spiral_attention_static_status(0) == (0, 0)
        rc, detail = sp.spiral_last_status(pair.ctx)
        assert rc == 0, detail
        # a page id outside the pool in the caller's block table: the kernel reads page 0 instead (nothing
        # faults), the finding stays in the static status word until it is read, and reading clears it
        bad = table.clone()
        bad[5, 3] = n_pages + 7
        sp.spiral_attention_static(pair.pool, n_pages, 2, 0, kv_dtype, hq, hkv, hd, bad, lens, q, out)
        rc, detail = sp.spiral_attention_static_status(0)
        assert rc == sp.SPIRAL_ERR_DEVICE_CHECK and detail == 2, (rc, detail)
        assert sp.spiral_attention_static_status(0) == (0, 0)
        sp.spiral_attention_static(pair.pool, n_pages, 2, 1, kv_dtype, hq, hkv, hd, table, lens, q, out)
        assert sp.spiral_attention_static_status(0) == (0, 0)
        g = 5
        exact = pair.oracle_mod.attention(q_cpu[g].double().numpy(), pair.oracle_cache(g), 1, lens[g])
        np.testing.assert_allclose(out[g].cpu().numpy(), exact, rtol=0, atol=ATOL)
    finally:
        pair.close()


def test_static_attention_refuses_more_than_its_fixed_capacity():
    import paper_2506_24119_b200 as sp
    pool = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
    table = torch.zeros(300, 1, dtype=torch.int32, device="cuda")
    q = torch.zeros(300, 4, 64, dtype=torch.float32, device="cuda")
    out = torch.empty_like(q)
    with pytest.raises(sp.SpiralError) as e:       # 300 sequences > SPIRAL_STATIC_ATTN_MAX_SEQS
        sp.spiral_attention_static(pool, 8, 1, 0, sp.SPIRAL_KV_F16, 4, 2, 64, table, [1] * 300, q, out)
    assert e.value.code == sp.SPIRAL_ERR_TOO_LARGE
    with pytest.raises(sp.SpiralError) as e:       # 100 sequences x 8 KV heads > SPIRAL_STATIC_ATTN_MAX_ITEMS
        sp.spiral_attention_static(pool, 8, 1, 0, sp.SPIRAL_KV_F16, 8, 8, 64, table[:100], [1] * 100,
                                   q[:100, :, :].new_zeros(100, 8, 64), out.new_zeros(100, 8, 64))
    assert e.value.code == sp.SPIRAL_ERR_TOO_LARGE
