"""Glue used by the GPU parity tests: builds the same model on both sides, drives the C ABI
and the oracle on identical seeded inputs, and measures the differences."""
from __future__ import annotations

import numpy as np
import torch

import synth

TOL_MAX_ABS = 0.05        # per-logit max |delta|
TOL_REL_RMS = 1e-2        # rms(delta) / rms(oracle logits)
TOL_TOKEN_AGREE = 0.995   # fraction of steps with identical sampled token


def to_device(w: dict, device) -> dict:
    out = {}
    for k, v in w.items():
        if isinstance(v, list):
            out[k] = [t.to(device) if t is not None else None for t in v]
        else:
            out[k] = v.to(device) if v is not None else None
    return out


def to_cuda(w: dict) -> dict:
    return to_device(w, "cuda")


class Pair:
    """One decoder living on both sides: the CUDA library (through the binding) and the oracle."""

    def __init__(self, desc: dict, seed: int = synth.MASTER_SEED, max_batch: int = 8, max_ctx: int = 512,
                 n_games: int = 8, pool_pages: int | None = None, gains: bool = True, std: float = 0.02,
                 weights_cpu: dict | None = None, generate_on_gpu: bool = False, kv_bf16: bool = False):
        import paper_2506_24119_b200 as sp
        from oracle import oracle
        self.sp, self.oracle_mod = sp, oracle
        self.desc = desc
        w_gpu = None
        if weights_cpu is None:
            # the generators are integer hashes, bit-identical on either device; big models are
            # generated on the GPU (seconds) and copied to the host for the oracle
            w_gpu = synth.make_weights(desc, seed=seed, std=std, device="cuda" if generate_on_gpu else "cpu")
            if gains:
                synth.perturb_gains(w_gpu, seed=seed)
            weights_cpu = to_device(w_gpu, "cpu") if generate_on_gpu else w_gpu
            w_gpu = w_gpu if generate_on_gpu else None
        self.w_cpu = weights_cpu
        self.oracle = oracle.Model(desc, weights_cpu)
        self.packed = sp.pack_weights(w_gpu if w_gpu is not None else to_cuda(weights_cpu))
        del w_gpu
        self.ctx = sp.spiral_init(desc, self.packed, 0, max_batch, max_ctx)
        page_bytes = sp.spiral_kv_page_bytes(desc, 16)
        if pool_pages is None:
            pool_pages = n_games * ((max_ctx + 15) // 16)
        self.pool = torch.empty(pool_pages * page_bytes, dtype=torch.uint8, device="cuda")
        # poison the pool so that any read of an unwritten slot shows up as NaN
        self.pool.view(torch.int16).fill_(0x7FC0 if kv_bf16 else 0x7E00)
        self.kv_dtype = torch.bfloat16 if kv_bf16 else torch.float16
        self.kv = sp.spiral_kv_alloc(self.ctx, self.pool, 16, n_games, max_ctx,
                                     sp.SPIRAL_KV_BF16 if kv_bf16 else sp.SPIRAL_KV_F16)
        self.max_ctx = max_ctx
        self.caches = {}

    def oracle_cache(self, game: int):
        if game not in self.caches:
            self.caches[game] = self.oracle.new_cache(self.max_ctx)
        return self.caches[game]

    def close(self):
        self.sp.spiral_free(self.ctx, self.kv)


def compare_logits(gpu: np.ndarray, ref: np.ndarray) -> tuple[float, float]:
    delta = gpu.astype(np.float64) - ref
    return float(np.abs(delta).max()), float(np.sqrt((delta ** 2).mean()) / np.sqrt((ref ** 2).mean()))
