"""ctypes front end of the CPU oracle (spiral_oracle.c).  TEST INFRASTRUCTURE, not product code.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this.  It shares
nothing with the CUDA path; inputs arrive as numpy arrays / torch CPU tensors.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "spiral_oracle.c")
_LIB = os.path.join(_HERE, "libspiral_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math, no contraction) if it is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-fPIC",
                               "-shared", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _Desc(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_q_heads", "n_kv_heads",
                                          "head_dim", "d_ff", "vocab")] + \
               [("rope_theta", C.c_double), ("rms_eps", C.c_double)] + \
               [(n, C.c_int32) for n in ("qk_norm", "qkv_bias", "tied_embed")]


_PP = C.POINTER(C.c_void_p)


class _Weights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("lm_head", C.c_void_p), ("final_norm", C.c_void_p)] + \
               [(n, _PP) for n in ("ln1", "wq", "wk", "wv", "bq", "bk", "bv", "q_norm", "k_norm",
                                   "wo", "ln2", "w_gate", "w_up", "w_down")]


_DP = C.POINTER(C.c_double)


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = C.CDLL(build())
            lib.oracle_cache_new.restype = C.c_void_p
            lib.oracle_cache_new.argtypes = [C.POINTER(_Desc), C.c_int32, C.c_int32, C.c_int32,
                                             C.POINTER(C.c_int32)]
            lib.oracle_cache_free.argtypes = [C.c_void_p]
            lib.oracle_cache_len.restype = C.c_int32
            lib.oracle_cache_len.argtypes = [C.c_void_p]
            lib.oracle_cache_set_len.argtypes = [C.c_void_p, C.c_int32]
            lib.oracle_cache_load_bf16.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p,
                                                   C.c_void_p]
            lib.oracle_cache_load_f64.argtypes = [C.c_void_p, C.c_int32, C.c_int32, _DP, _DP]
            lib.oracle_cache_read.argtypes = [C.c_void_p, C.c_int32, C.c_int32, _DP, _DP]
            lib.oracle_decode_step.restype = C.c_int32
            lib.oracle_decode_step.argtypes = [C.POINTER(_Desc), C.POINTER(_Weights), C.c_void_p,
                                               C.c_int32, C.c_int32, _DP, _DP, _DP]
            lib.oracle_prefill.restype = C.c_int32
            lib.oracle_prefill.argtypes = [C.POINTER(_Desc), C.POINTER(_Weights), C.c_void_p,
                                           C.POINTER(C.c_int32), C.c_int32, C.c_int32, _DP]
            lib.oracle_sample.restype = C.c_int32
            lib.oracle_sample.argtypes = [_DP, C.POINTER(C.c_float), C.c_float, C.c_int32,
                                          C.POINTER(C.c_float), C.POINTER(C.c_float)]
            lib.oracle_rmsnorm.argtypes = [_DP, C.c_void_p, C.c_double, C.c_int32, _DP]
            lib.oracle_rope.argtypes = [_DP, C.c_int32, C.c_int32, C.c_double]
            lib.oracle_softmax.argtypes = [_DP, C.c_int32]
            lib.oracle_silu.restype = C.c_double
            lib.oracle_silu.argtypes = [C.c_double]
            lib.oracle_matvec.argtypes = [C.c_void_p, C.c_void_p, _DP, C.c_int32, C.c_int32, _DP]
            lib.oracle_attention.argtypes = [_DP, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, _DP]
            lib.oracle_attention_piece.argtypes = [_DP, C.c_void_p, C.c_int32, C.c_int32, C.c_int32,
                                                   C.c_int32, _DP, _DP, _DP]
            lib.oracle_attention_merge.argtypes = [C.c_int32, _DP, _DP, _DP, C.c_int32, _DP]
            _lib = lib
    return _lib


def _dp(a: np.ndarray):
    assert a.dtype == np.float64 and a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(_DP)


def _bf16_bits(t) -> np.ndarray:
    """torch bf16 CPU tensor -> contiguous uint16 numpy array of its bit patterns."""
    if isinstance(t, np.ndarray):
        assert t.dtype == np.uint16
        return np.ascontiguousarray(t)
    assert t.dtype == torch.bfloat16 and t.device.type == "cpu"
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def num_threads() -> int:
    """Threads the OpenMP loops of the oracle will use."""
    n = os.environ.get("OMP_NUM_THREADS")
    return int(n) if n else (os.cpu_count() or 1)


class Model:
    """Holds a decoder description and its bf16 weights for the oracle."""

    def __init__(self, desc: dict, weights: dict):
        self.lib = _load()
        self.desc_dict = dict(desc)
        self.desc = _Desc(**{k: desc[k] for k, _ in _Desc._fields_})
        self._keep = []
        L = desc["n_layers"]

        def one(t):
            if t is None:
                return None
            a = _bf16_bits(t)
            self._keep.append(a)
            return a.ctypes.data

        def per_layer(name):
            arr = (C.c_void_p * L)(*[one(t) for t in weights[name]])
            self._keep.append(arr)
            return C.cast(arr, _PP)

        self.w = _Weights(embed=one(weights["embed"]), lm_head=one(weights.get("lm_head")),
                          final_norm=one(weights["final_norm"]),
                          **{n: per_layer(n) for n in ("ln1", "wq", "wk", "wv", "bq", "bk", "bv",
                                                       "q_norm", "k_norm", "wo", "ln2", "w_gate",
                                                       "w_up", "w_down")})

    def new_cache(self, max_ctx: int, page_size: int = 0, n_pool_pages: int = 0,
                  block_table=None) -> "Cache":
        return Cache(self, max_ctx, page_size, n_pool_pages, block_table)

    def decode_step(self, cache: "Cache", token: int, kv_as_bf16: bool = False,
                    want_trace: bool = False, want_hidden: bool = False, want_logits: bool = True):
        d = self.desc_dict
        logits = np.empty(d["vocab"], np.float64) if want_logits else None
        trace = np.empty((d["n_layers"] + 1, d["d_model"]), np.float64) if want_trace else None
        hidden = np.empty(d["d_model"], np.float64) if want_hidden else None
        rc = self.lib.oracle_decode_step(C.byref(self.desc), C.byref(self.w), cache.ptr,
                                         int(token), int(kv_as_bf16),
                                         _dp(logits) if want_logits else None,
                                         _dp(trace) if want_trace else None,
                                         _dp(hidden) if want_hidden else None)
        if rc != 0:
            raise RuntimeError("oracle_decode_step failed (bad token, full cache or no memory)")
        out = [logits]
        if want_trace:
            out.append(trace)
        if want_hidden:
            out.append(hidden)
        return out[0] if len(out) == 1 else tuple(out)

    def prefill(self, cache: "Cache", tokens, kv_as_bf16: bool = False) -> np.ndarray:
        toks = np.ascontiguousarray(np.asarray(tokens, dtype=np.int32))
        logits = np.empty(self.desc_dict["vocab"], np.float64)
        rc = self.lib.oracle_prefill(C.byref(self.desc), C.byref(self.w), cache.ptr,
                                     toks.ctypes.data_as(C.POINTER(C.c_int32)), len(toks),
                                     int(kv_as_bf16), _dp(logits))
        if rc != 0:
            raise RuntimeError("oracle_prefill failed")
        return logits


class Cache:
    def __init__(self, model: Model, max_ctx: int, page_size: int, n_pool_pages: int, block_table):
        self.model = model
        bt = None
        if page_size > 0:
            bt = np.ascontiguousarray(np.asarray(block_table, dtype=np.int32))
            assert len(bt) >= (max_ctx + page_size - 1) // page_size
        self.ptr = model.lib.oracle_cache_new(
            C.byref(model.desc), max_ctx, page_size, n_pool_pages,
            bt.ctypes.data_as(C.POINTER(C.c_int32)) if bt is not None else None)
        if not self.ptr:
            raise MemoryError("oracle_cache_new")

    def __del__(self):
        if getattr(self, "ptr", None):
            self.model.lib.oracle_cache_free(self.ptr)
            self.ptr = None

    def __len__(self):
        return self.model.lib.oracle_cache_len(self.ptr)

    def set_len(self, n: int):
        self.model.lib.oracle_cache_set_len(self.ptr, n)

    def load_bf16(self, layer: int, k, v):
        """k, v: bf16 [n_tokens, n_kv_heads, head_dim]; fills positions 0..n_tokens-1."""
        kb, vb = _bf16_bits(k), _bf16_bits(v)
        self.model.lib.oracle_cache_load_bf16(self.ptr, layer, k.shape[0], kb.ctypes.data,
                                              vb.ctypes.data)

    def load(self, layer: int, k, v):
        """k, v: torch tensors [n_tokens, n_kv_heads, head_dim] of any float type (widened exactly)."""
        if k.dtype == torch.bfloat16:
            return self.load_bf16(layer, k, v)
        kd = np.ascontiguousarray(k.double().numpy())
        vd = np.ascontiguousarray(v.double().numpy())
        self.model.lib.oracle_cache_load_f64(self.ptr, layer, k.shape[0], _dp(kd), _dp(vd))

    def read(self, layer: int, pos: int):
        d = self.model.desc_dict
        k = np.empty((d["n_kv_heads"], d["head_dim"]), np.float64)
        v = np.empty_like(k)
        self.model.lib.oracle_cache_read(self.ptr, layer, pos, _dp(k), _dp(v))
        return k, v


# ------------------------------------------------------------------------------------------------
# elementary functions (numpy in / numpy out)
# ------------------------------------------------------------------------------------------------

def sample(logits: np.ndarray, gumbel: np.ndarray, temperature: float = 1.0):
    """Returns (token, best score, gap to the runner-up)."""
    lib = _load()
    lg = np.ascontiguousarray(logits, dtype=np.float64)
    g = np.ascontiguousarray(gumbel, dtype=np.float32)
    bz, gap = C.c_float(), C.c_float()
    tok = lib.oracle_sample(_dp(lg), g.ctypes.data_as(C.POINTER(C.c_float)), float(temperature),
                            len(lg), C.byref(bz), C.byref(gap))
    return tok, bz.value, gap.value


def log_prob(logits: np.ndarray, token: int, temperature: float = 1.0) -> float:
    """log softmax(logits / T)[token] in fp64: the probability the sampling policy of the Actor
    block (temperature T, no truncation) gave to `token`, as the learner's importance ratio needs it."""
    z = np.asarray(logits, dtype=np.float64) / float(temperature)
    m = z.max()
    return float(z[token] - (m + np.log(np.exp(z - m).sum())))


def nucleus_kept(logits: np.ndarray, temperature: float, top_p: float):
    """Nucleus (top-p) truncation, the paper's evaluation sampling ("Evaluation Settings": temperature 0.6,
    top-p 0.95).  With z = logits / T (the division in fp32, the precision the sampler takes its decisions
    in) and p = softmax(z) in fp64: walk the tokens from the most probable down and keep them until the kept
    mass reaches top_p; tokens exactly as probable as the last one kept are kept too (so the result does not
    depend on how ties are ordered), and the most probable token is always kept.  Equivalently: token v is
    kept iff the mass of the tokens strictly more probable than v is below top_p.
    Returns (kept mask, z as fp32, margin) where margin is the smallest |mass above v - top_p| over all v:
    how far the closest keep/drop decision was from flipping."""
    z = (np.asarray(logits, dtype=np.float64).astype(np.float32) / np.float32(temperature)).astype(np.float32)
    z64 = z.astype(np.float64)
    p = np.exp(z64 - z64.max())
    p /= p.sum()
    kept = np.zeros(len(z), dtype=bool)
    order = sorted(range(len(z)), key=lambda v: -z64[v])
    mass_above, margin = 0.0, np.inf          # mass of the tokens strictly more probable than the current group
    i = 0
    while i < len(order):
        j = i
        while j < len(order) and z64[order[j]] == z64[order[i]]:
            j += 1                            # order[i:j]: tokens of equal probability
        margin = min(margin, abs(mass_above - top_p))
        if mass_above < top_p or i == 0:
            for v in order[i:j]:
                kept[v] = True
        mass_above += float(sum(p[v] for v in order[i:j]))
        i = j
    return kept, z, margin


def nucleus_sample(logits: np.ndarray, gumbel: np.ndarray, temperature: float, top_p: float):
    """Gumbel-argmax over the nucleus: argmax over the kept tokens of fp32(z_v + gumbel_v), lowest index on
    ties -- a draw from the kept tokens' renormalised distribution.  Returns (token, kept mask, margin)."""
    kept, z, margin = nucleus_kept(logits, temperature, top_p)
    score = (z + np.asarray(gumbel, dtype=np.float32)).astype(np.float32)
    score = np.where(kept, score, -np.inf)
    return int(np.argmax(score)), kept, margin


def rae_update(baselines, alpha: float, game_of, returns):
    """Role-conditioned advantage estimation (Algorithm 1, policy-optimisation loop; Eq. 2), in fp64: for
    every trajectory of the batch in order and both roles p, b[G][p] <- alpha b[G][p] + (1 - alpha) R_p and
    A_p = R_p - b[G][p] with the baseline just updated.  `baselines` (list of [b0, b1] per game, zero at the
    start of training) is updated in place; returns the advantages, one [A0, A1] per trajectory."""
    adv = []
    for t, g in enumerate(game_of):
        row = []
        for p in (0, 1):
            r = float(returns[t][p])
            baselines[g][p] = alpha * baselines[g][p] + (1.0 - alpha) * r
            row.append(r - baselines[g][p])
        adv.append(row)
    return adv


def rmsnorm(x: np.ndarray, gain_bf16, eps: float) -> np.ndarray:
    lib = _load()
    x = np.ascontiguousarray(x, dtype=np.float64)
    g = _bf16_bits(gain_bf16)
    out = np.empty_like(x)
    lib.oracle_rmsnorm(_dp(x), g.ctypes.data, eps, len(x), _dp(out))
    return out


def rope(vec: np.ndarray, pos: int, theta: float) -> np.ndarray:
    lib = _load()
    v = np.array(vec, dtype=np.float64, copy=True)
    lib.oracle_rope(_dp(v), len(v), pos, theta)
    return v


def softmax(s: np.ndarray) -> np.ndarray:
    lib = _load()
    v = np.array(s, dtype=np.float64, copy=True)
    lib.oracle_softmax(_dp(v), len(v))
    return v


def silu(u: float) -> float:
    return _load().oracle_silu(float(u))


def matvec(w_bf16, x: np.ndarray, bias_bf16=None) -> np.ndarray:
    lib = _load()
    wb = _bf16_bits(w_bf16)
    rows, cols = w_bf16.shape
    x = np.ascontiguousarray(x, dtype=np.float64)
    y = np.empty(rows, np.float64)
    bb = _bf16_bits(bias_bf16) if bias_bf16 is not None else None
    lib.oracle_matvec(wb.ctypes.data, bb.ctypes.data if bb is not None else None, _dp(x), rows,
                      cols, _dp(y))
    return y


def attention(q: np.ndarray, cache: Cache, layer: int, n_ctx: int) -> np.ndarray:
    """q [n_q_heads, head_dim] -> out [n_q_heads, head_dim] over cache positions 0..n_ctx-1."""
    lib = _load()
    q = np.ascontiguousarray(q, dtype=np.float64)
    out = np.empty_like(q)
    lib.oracle_attention(_dp(q), cache.ptr, layer, n_ctx, q.shape[0], _dp(out))
    return out


def attention_piece(q_head: np.ndarray, cache: Cache, layer: int, t0: int, t1: int, kv_head: int):
    lib = _load()
    q = np.ascontiguousarray(q_head, dtype=np.float64)
    m, l = C.c_double(), C.c_double()
    o = np.empty_like(q)
    lib.oracle_attention_piece(_dp(q), cache.ptr, layer, t0, t1, kv_head, C.byref(m), C.byref(l),
                               _dp(o))
    return m.value, l.value, o


def attention_merge(m, l, o: np.ndarray) -> np.ndarray:
    lib = _load()
    m = np.ascontiguousarray(m, dtype=np.float64)
    l = np.ascontiguousarray(l, dtype=np.float64)
    o = np.ascontiguousarray(o, dtype=np.float64)
    out = np.empty(o.shape[1], np.float64)
    lib.oracle_attention_merge(len(m), _dp(m), _dp(l), _dp(o), o.shape[1], _dp(out))
    return out
