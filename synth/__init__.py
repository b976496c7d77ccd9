"""Seeded synthetic inputs for the rollout-decoding path (weights, token ids, lengths, noise).

This module is the only code shared by the CPU oracle's tests and the CUDA path's tests and
benchmark.  It holds none of the decoder's arithmetic: it only turns (seed, stream, index)
into numbers.  Every generator is a counter-based hash evaluated with integer tensor ops, so
the same (seed, stream, index) gives the same bits on the CPU and on a GPU, in any chunking.

The workloads it stands in for are the self-play rollouts of Algorithm 1 (one shared policy
generates a multi-token response per game per turn, sampled at temperature 1.0 with no
truncation, Table "Hyperparameter configurations", Actor block).  Game text, tokenizers and
trained weights are not available, so shapes, lengths and value distributions are kept and
the values themselves are random.
"""
from __future__ import annotations

import math

import torch

MASTER_SEED = 250624119

# stream ids (sub-seeds): one per kind of data so that no two tensors share a counter range
STREAM_WEIGHT = 1
STREAM_TOKEN = 2
STREAM_LENGTH = 3
STREAM_NOISE = 4
STREAM_KV = 5
STREAM_BIAS = 6
STREAM_TEACHER = 7

_M32 = 0xFFFFFFFF


def _fmix32(x: torch.Tensor) -> torch.Tensor:
    """32-bit avalanche mixer on int64 tensors holding values in [0, 2^32)."""
    x = x ^ (x >> 16)
    x = (x * 0x85EBCA6B) & _M32
    x = x ^ (x >> 13)
    x = (x * 0xC2B2AE35) & _M32
    x = x ^ (x >> 16)
    return x


def _key(seed: int, stream: int, tensor_id: int) -> int:
    """Scalar key for one tensor, computed with Python ints (exact)."""
    def fm(v: int) -> int:
        v &= _M32
        v ^= v >> 16
        v = (v * 0x85EBCA6B) & _M32
        v ^= v >> 13
        v = (v * 0xC2B2AE35) & _M32
        v ^= v >> 16
        return v
    k = fm(seed & _M32)
    k = fm(k ^ ((seed >> 32) & _M32) ^ 0x9E3779B9)
    k = fm(k ^ (stream * 0x7F4A7C15 & _M32))
    k = fm(k ^ (tensor_id & _M32) ^ 0x51ED270B)
    k = fm(k ^ ((tensor_id >> 32) & _M32))
    return k


def hash_u32(seed: int, stream: int, tensor_id: int, start: int, count: int,
             device="cpu", lane: int = 0) -> torch.Tensor:
    """count hashed 32-bit values for counters start..start+count-1, as an int64 tensor."""
    key = _key(seed, stream, tensor_id) ^ ((lane * 0x632BE5AB) & _M32)
    idx = torch.arange(start, start + count, dtype=torch.int64, device=device)
    lo = idx & _M32
    hi = (idx >> 32) & _M32
    h = _fmix32(hi ^ key)
    h = _fmix32(lo ^ h ^ 0x2545F491)
    h = _fmix32(((h + lo * 0x9E3779B1) & _M32) ^ key)
    return h


_CHUNK = 1 << 24


def normal_bf16(seed: int, tensor_id: int, numel: int, std: float, device="cpu",
                stream: int = STREAM_WEIGHT) -> torch.Tensor:
    """numel values ~ N(0, std) (12-term Irwin-Hall, |z| <= 6), rounded to bf16 once (RNE).

    Integer arithmetic up to the final scale, so bits do not depend on the device."""
    out = torch.empty(numel, dtype=torch.bfloat16, device=device)
    scale = float(std) / 256.0           # sum of 12 bytes has standard deviation 256 (to 4 digits)
    for s in range(0, numel, _CHUNK):
        n = min(_CHUNK, numel - s)
        acc = torch.zeros(n, dtype=torch.int64, device=device)
        for lane in range(3):
            h = hash_u32(seed, stream, tensor_id, s, n, device, lane)
            acc += (h & 0xFF) + ((h >> 8) & 0xFF) + ((h >> 16) & 0xFF) + ((h >> 24) & 0xFF)
        z = (acc - 1530).to(torch.float32)          # exact: |acc-1530| <= 1530
        out[s:s + n] = (z * scale).to(torch.bfloat16)
    return out


def uniform_bf16(seed: int, tensor_id: int, numel: int, half_width: float, device="cpu",
                 stream: int = STREAM_KV) -> torch.Tensor:
    """numel values uniform in (-half_width, half_width), rounded to bf16 (for synthetic K/V)."""
    out = torch.empty(numel, dtype=torch.bfloat16, device=device)
    for s in range(0, numel, _CHUNK):
        n = min(_CHUNK, numel - s)
        h = hash_u32(seed, stream, tensor_id, s, n, device)
        z = ((h >> 8).to(torch.float32) + 0.5) * (2.0 ** -23) - 1.0   # exact in fp32
        out[s:s + n] = (z * float(half_width)).to(torch.bfloat16)
    return out


def token_ids(seed: int, tensor_id: int, count: int, vocab: int, device="cpu",
              stream: int = STREAM_TOKEN) -> torch.Tensor:
    """count token ids uniform in [0, vocab) as int32."""
    h = hash_u32(seed, stream, tensor_id, 0, count, device)
    return (h % vocab).to(torch.int32)


def lengths(seed: int, tensor_id: int, count: int, lo: int, hi: int) -> list[int]:
    """count integers uniform in [lo, hi] inclusive (host list)."""
    h = hash_u32(seed, STREAM_LENGTH, tensor_id, 0, count, "cpu")
    return (lo + h % (hi - lo + 1)).tolist()


def gumbel_noise(seed: int, step: int, n_games: int, vocab: int, device="cpu") -> torch.Tensor:
    """Standard Gumbel noise [n_games, vocab] fp32 for one decode step.

    u = (k + 0.5) / 2^24 with k the top 24 bits of the hash, so u is never 0 or 1 and the
    noise is finite; gamma = -log(-log u) in fp64, stored as fp32.  The same array must be
    handed to every implementation being compared (the logs are not bit-portable)."""
    numel = n_games * vocab
    out = torch.empty(numel, dtype=torch.float32, device=device)
    for s in range(0, numel, _CHUNK):
        n = min(_CHUNK, numel - s)
        h = hash_u32(seed, STREAM_NOISE, step, s, n, device)
        u = ((h >> 8).to(torch.float64) + 0.5) * (2.0 ** -24)
        out[s:s + n] = (-torch.log(-torch.log(u))).to(torch.float32)
    return out.view(n_games, vocab)


# ---------------------------------------------------------------------------------------------
# Model shapes of the workloads (architectures only; weights are random)
# ---------------------------------------------------------------------------------------------

SHAPES = {
    # tiny decoder for end-to-end checks on the CPU in seconds
    "tiny": dict(n_layers=2, d_model=256, n_q_heads=4, n_kv_heads=2, head_dim=64, d_ff=688,
                 vocab=4096, rope_theta=1e6, rms_eps=1e-6, qk_norm=0, qkv_bias=0, tied_embed=1),
    # tiny variants that switch the optional features on, for coverage
    "tiny_qknorm": dict(n_layers=2, d_model=256, n_q_heads=4, n_kv_heads=2, head_dim=64, d_ff=688,
                        vocab=4096, rope_theta=1e6, rms_eps=1e-6, qk_norm=1, qkv_bias=0, tied_embed=1),
    "tiny_bias": dict(n_layers=2, d_model=256, n_q_heads=4, n_kv_heads=1, head_dim=64, d_ff=688,
                      vocab=4096, rope_theta=1e4, rms_eps=1e-6, qk_norm=0, qkv_bias=1, tied_embed=0),
    "qwen3_4b": dict(n_layers=36, d_model=2560, n_q_heads=32, n_kv_heads=8, head_dim=128,
                     d_ff=9728, vocab=151936, rope_theta=1e6, rms_eps=1e-6, qk_norm=1, qkv_bias=0,
                     tied_embed=1),
    "llama31_8b": dict(n_layers=32, d_model=4096, n_q_heads=32, n_kv_heads=8, head_dim=128,
                       d_ff=14336, vocab=128256, rope_theta=5e5, rms_eps=1e-5, qk_norm=0,
                       qkv_bias=0, tied_embed=0),
    "qwen25_7b": dict(n_layers=28, d_model=3584, n_q_heads=28, n_kv_heads=4, head_dim=128,
                      d_ff=18944, vocab=152064, rope_theta=1e4, rms_eps=1e-6, qk_norm=0,
                      qkv_bias=1, tied_embed=0),
}


def shape(name: str, **overrides) -> dict:
    d = dict(SHAPES[name])
    d.update(overrides)
    return d


_TENSOR_IDS = {"embed": 1, "lm_head": 2, "final_norm": 3}
_LAYER_TENSORS = ["ln1", "wq", "wk", "wv", "bq", "bk", "bv", "q_norm", "k_norm", "wo", "ln2",
                  "w_gate", "w_up", "w_down"]


def make_weights(desc: dict, seed: int = MASTER_SEED, device="cpu", std: float = 0.02) -> dict:
    """Random-init weights of one decoder, all bf16, in the plain per-matrix layout.

    Matrices are [out_features, in_features] row-major.  Norm gains are 1.0; projection
    matrices and the embedding are ~N(0, std); QKV biases (when present) are ~N(0, std).
    Returns {"embed", "lm_head" (None if tied), "final_norm", and per-layer lists}."""
    L, d = desc["n_layers"], desc["d_model"]
    Hq, Hkv, hd, F, V = (desc["n_q_heads"], desc["n_kv_heads"], desc["head_dim"], desc["d_ff"],
                         desc["vocab"])
    ones = lambda n: torch.ones(n, dtype=torch.bfloat16, device=device)

    def mat(tid, rows, cols, stream=STREAM_WEIGHT):
        return normal_bf16(seed, tid, rows * cols, std, device, stream).view(rows, cols)

    w = {"embed": mat(_TENSOR_IDS["embed"], V, d),
         "lm_head": None if desc["tied_embed"] else mat(_TENSOR_IDS["lm_head"], V, d),
         "final_norm": ones(d)}
    for name in _LAYER_TENSORS:
        w[name] = []
    for l in range(L):
        base = 1000 + 100 * l
        w["ln1"].append(ones(d))
        w["ln2"].append(ones(d))
        w["wq"].append(mat(base + 1, Hq * hd, d))
        w["wk"].append(mat(base + 2, Hkv * hd, d))
        w["wv"].append(mat(base + 3, Hkv * hd, d))
        w["wo"].append(mat(base + 4, d, Hq * hd))
        w["w_gate"].append(mat(base + 5, F, d))
        w["w_up"].append(mat(base + 6, F, d))
        w["w_down"].append(mat(base + 7, d, F))
        if desc["qkv_bias"]:
            w["bq"].append(normal_bf16(seed, base + 8, Hq * hd, std, device, STREAM_BIAS))
            w["bk"].append(normal_bf16(seed, base + 9, Hkv * hd, std, device, STREAM_BIAS))
            w["bv"].append(normal_bf16(seed, base + 10, Hkv * hd, std, device, STREAM_BIAS))
        else:
            w["bq"].append(None); w["bk"].append(None); w["bv"].append(None)
        if desc["qk_norm"]:
            w["q_norm"].append(ones(hd)); w["k_norm"].append(ones(hd))
        else:
            w["q_norm"].append(None); w["k_norm"].append(None)
    return w


def perturb_gains(w: dict, seed: int = MASTER_SEED, amount: float = 0.25) -> dict:
    """Replace the all-ones norm gains by 1 + U(-amount, amount) (bf16) so that tests exercise
    the gain multiplications; the workloads themselves keep gains at 1.0."""
    def g(t, tid):
        if t is None:
            return None
        u = uniform_bf16(seed, tid, t.numel(), amount, t.device, STREAM_BIAS).float()
        return (1.0 + u).to(torch.bfloat16)
    w["final_norm"] = g(w["final_norm"], 77)
    for l in range(len(w["ln1"])):
        w["ln1"][l] = g(w["ln1"][l], 2000 + 10 * l)
        w["ln2"][l] = g(w["ln2"][l], 2001 + 10 * l)
        w["q_norm"][l] = g(w["q_norm"][l], 2002 + 10 * l)
        w["k_norm"][l] = g(w["k_norm"][l], 2003 + 10 * l)
    return w


def synthetic_kv(seed: int, game: int, layer: int, n_tokens: int, n_kv_heads: int, head_dim: int,
                 device="cpu") -> tuple[torch.Tensor, torch.Tensor]:
    """Random bf16 K and V of one game and layer, each [n_tokens, n_kv_heads, head_dim].

    Used to start decode parity checks at long contexts without running a prefill on the
    CPU.  K is uniform in (-2, 2) (comparable to normalised, rotated keys), V in (-1, 1)."""
    n = n_tokens * n_kv_heads * head_dim
    tid = (game << 20) | (layer << 1)
    k = uniform_bf16(seed, tid, n, 2.0, device).view(n_tokens, n_kv_heads, head_dim)
    v = uniform_bf16(seed, tid | 1, n, 1.0, device).view(n_tokens, n_kv_heads, head_dim)
    return k, v


def weight_bytes_per_step(desc: dict) -> int:
    """Bytes of bf16 weight matrices one decode step has to read (embedding rows excluded
    unless the LM head is tied to them, in which case they are the LM head)."""
    L, d = desc["n_layers"], desc["d_model"]
    Hq, Hkv, hd, F, V = (desc["n_q_heads"], desc["n_kv_heads"], desc["head_dim"], desc["d_ff"],
                         desc["vocab"])
    per_layer = d * (Hq + 2 * Hkv) * hd + Hq * hd * d + 3 * d * F
    return 2 * (L * per_layer + V * d)


def kv_bytes_per_token(desc: dict) -> int:
    """Bytes of bf16 K and V one cached token occupies over all layers."""
    return desc["n_layers"] * 2 * desc["n_kv_heads"] * desc["head_dim"] * 2


def expected_gumbel_moments() -> tuple[float, float]:
    """Mean (Euler-Mascheroni) and variance (pi^2/6) of the standard Gumbel law."""
    return 0.5772156649015329, math.pi ** 2 / 6.0
