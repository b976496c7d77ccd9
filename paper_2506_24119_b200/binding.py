"""ctypes binding of libspiral.so: same names as the C ABI, argument marshalling only.

torch is used for device memory and streams; every step of the decode path runs inside the
library's CUDA kernels.  If the shared library is missing the import fails loudly."""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# SPIRAL_LIB_PATH selects a differently built copy of the library (e.g. an instrumented build)
LIB_PATH = os.environ.get("SPIRAL_LIB_PATH") or os.path.join(_HERE, "libspiral.so")

SPIRAL_OK = 0
SPIRAL_ERR_INVALID = -1
SPIRAL_ERR_OOM = -2
SPIRAL_ERR_CUDA = -3
SPIRAL_ERR_TIMEOUT = -4
SPIRAL_ERR_DEVICE_CHECK = -5
SPIRAL_ERR_UNSUPPORTED = -6
SPIRAL_ERR_TOO_LARGE = -7
SPIRAL_KV_F16 = 0
SPIRAL_KV_BF16 = 1

EXPORTS = ["spiral_init", "spiral_kv_page_bytes", "spiral_kv_alloc", "spiral_kv_release",
           "spiral_kv_truncate", "spiral_profile", "spiral_profile_read", "spiral_kv_seq_len",
           "spiral_kv_block_table", "spiral_attention_static", "spiral_attention_static_status", "spiral_kv_free_pages", "spiral_kv_load", "spiral_prefill",
           "spiral_decode_step", "spiral_decode_step_logprob", "spiral_decode_step_nucleus", "spiral_sample_nucleus",
           "spiral_rae_update", "spiral_kv_fork", "spiral_sched_fork", "spiral_sched_create", "spiral_sched_free", "spiral_sched_open", "spiral_sched_close",
           "spiral_sched_turn", "spiral_sched_collect_logprob", "spiral_sched_poll_logprob", "spiral_sched_policy", "spiral_sched_tick", "spiral_sched_poll", "spiral_sched_stats", "spiral_decode_step_host", "spiral_linear", "spiral_attention",
           "spiral_read_ceiling", "spiral_selftest_wait_timeout", "spiral_launch_count", "spiral_last_status", "spiral_free", "spiral_strerror",
           "spiral_last_cuda_error"]

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2506_24119_b200.build` "
        "(nvcc, sm_100a). There is no CPU or PyTorch fallback for the decode path.")

_lib = C.CDLL(LIB_PATH)


class ModelDesc(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_q_heads", "n_kv_heads", "head_dim",
                                          "d_ff", "vocab")] + \
               [("rope_theta", C.c_double), ("rms_eps", C.c_double)] + \
               [(n, C.c_int32) for n in ("qk_norm", "qkv_bias", "tied_embed")]


_PP = C.POINTER(C.c_void_p)


class Weights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("lm_head", C.c_void_p), ("final_norm", C.c_void_p)] + \
               [(n, _PP) for n in ("ln1", "wqkv", "bqkv", "q_norm", "k_norm", "wo", "ln2", "w_gate_up",
                                   "w_down")]


_I32P = C.POINTER(C.c_int32)
_lib.spiral_init.restype = C.c_int
_lib.spiral_init.argtypes = [C.POINTER(C.c_void_p), C.POINTER(ModelDesc), C.POINTER(Weights), C.c_int,
                             C.c_int, C.c_int]
_lib.spiral_kv_page_bytes.restype = C.c_size_t
_lib.spiral_kv_page_bytes.argtypes = [C.POINTER(ModelDesc), C.c_int]
_lib.spiral_kv_alloc.restype = C.c_int
_lib.spiral_kv_alloc.argtypes = [C.c_void_p, C.c_void_p, C.c_size_t, C.c_int, C.c_int, C.c_int, C.c_int,
                                 C.POINTER(C.c_void_p)]
_lib.spiral_kv_release.restype = C.c_int
_lib.spiral_kv_release.argtypes = [C.c_void_p, C.c_int, _I32P]
_lib.spiral_kv_truncate.restype = C.c_int
_lib.spiral_kv_truncate.argtypes = [C.c_void_p, C.c_int, _I32P, _I32P]
_lib.spiral_profile.restype = C.c_int
_lib.spiral_profile.argtypes = [C.c_void_p, C.c_uint32]
_lib.spiral_profile_read.restype = C.c_int
_lib.spiral_profile_read.argtypes = [C.c_void_p, C.c_int, C.POINTER(C.c_double), C.POINTER(C.c_int64)]
_lib.spiral_kv_seq_len.restype = C.c_int
_lib.spiral_kv_seq_len.argtypes = [C.c_void_p, C.c_int, _I32P]
_lib.spiral_kv_free_pages.restype = C.c_int
_lib.spiral_kv_free_pages.argtypes = [C.c_void_p, _I32P]
_lib.spiral_kv_load.restype = C.c_int
_lib.spiral_kv_load.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p,
                                C.c_void_p]
_lib.spiral_prefill.restype = C.c_int
_lib.spiral_prefill.argtypes = [C.c_void_p, C.c_void_p, C.c_int, _I32P, C.c_void_p, _I32P, C.c_void_p,
                                C.c_void_p]
_lib.spiral_decode_step.restype = C.c_int
_lib.spiral_decode_step.argtypes = [C.c_void_p, C.c_void_p, C.c_int, _I32P, C.c_void_p, C.c_void_p,
                                    C.c_float, C.c_void_p, C.c_void_p, C.c_void_p]
_lib.spiral_decode_step_logprob.restype = C.c_int
_lib.spiral_decode_step_logprob.argtypes = [C.c_void_p, C.c_void_p, C.c_int, _I32P, C.c_void_p, C.c_void_p,
                                            C.c_float, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
_lib.spiral_decode_step_nucleus.restype = C.c_int
_lib.spiral_decode_step_nucleus.argtypes = [C.c_void_p, C.c_void_p, C.c_int, _I32P, C.c_void_p, C.c_void_p,
                                            C.c_float, C.c_float, C.c_void_p, C.c_void_p, C.c_void_p]
_lib.spiral_sample_nucleus.restype = C.c_int
_lib.spiral_sample_nucleus.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_float, C.c_float, C.c_void_p,
                                       C.c_void_p]
_lib.spiral_rae_update.restype = C.c_int
_lib.spiral_rae_update.argtypes = [C.POINTER(C.c_double), C.c_int, C.c_double, C.c_int, _I32P, C.POINTER(C.c_double),
                                   C.POINTER(C.c_double)]
_lib.spiral_kv_fork.restype = C.c_int
_lib.spiral_kv_fork.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p]
_lib.spiral_sched_fork.restype = C.c_int
_lib.spiral_sched_fork.argtypes = [C.c_void_p, C.c_int, _I32P, C.c_void_p]
_lib.spiral_sched_create.restype = C.c_int
_lib.spiral_sched_create.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.POINTER(C.c_void_p)]
_lib.spiral_sched_free.restype = None
_lib.spiral_sched_free.argtypes = [C.c_void_p]
_lib.spiral_sched_open.restype = C.c_int
_lib.spiral_sched_open.argtypes = [C.c_void_p, _I32P]
_lib.spiral_sched_close.restype = C.c_int
_lib.spiral_sched_close.argtypes = [C.c_void_p, C.c_int]
_lib.spiral_sched_turn.restype = C.c_int
_lib.spiral_sched_turn.argtypes = [C.c_void_p, C.c_int, C.c_int, _I32P, C.c_int]
_lib.spiral_sched_collect_logprob.restype = C.c_int
_lib.spiral_sched_collect_logprob.argtypes = [C.c_void_p, C.c_int]
_lib.spiral_sched_poll_logprob.restype = C.c_int
_lib.spiral_sched_poll_logprob.argtypes = [C.c_void_p, _I32P, _I32P, C.POINTER(C.c_float), C.c_int, _I32P, _I32P]
_lib.spiral_sched_policy.restype = C.c_int
_lib.spiral_sched_policy.argtypes = [C.c_void_p, C.c_int, C.c_int]
_lib.spiral_sched_tick.restype = C.c_int
_lib.spiral_sched_tick.argtypes = [C.c_void_p, C.c_void_p, C.c_float, C.c_void_p]
_lib.spiral_sched_poll.restype = C.c_int
_lib.spiral_sched_poll.argtypes = [C.c_void_p, _I32P, _I32P, C.c_int, _I32P, _I32P]
_lib.spiral_sched_stats.restype = C.c_int
_lib.spiral_sched_stats.argtypes = [C.c_void_p, C.POINTER(C.c_int64), C.c_int]
_lib.spiral_decode_step_host.restype = C.c_int
_lib.spiral_decode_step_host.argtypes = [C.c_void_p, C.c_void_p, C.c_int, _I32P, C.c_void_p, C.c_void_p,
                                         C.c_float, C.c_void_p, C.c_void_p]
_lib.spiral_linear.restype = C.c_int
_lib.spiral_linear.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_int, C.c_void_p,
                               C.c_int, C.c_void_p]
_lib.spiral_attention.restype = C.c_int
_lib.spiral_attention.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, _I32P, _I32P, C.c_void_p,
                                  C.c_void_p, C.c_void_p]
_lib.spiral_kv_block_table.restype = C.c_int
_lib.spiral_kv_block_table.argtypes = [C.c_void_p, C.c_int, _I32P, C.c_int]
_lib.spiral_attention_static.restype = C.c_int
_lib.spiral_attention_static.argtypes = [C.c_int, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int,
                                         C.c_int, C.c_void_p, C.c_int, C.c_int, _I32P, C.c_void_p, C.c_void_p,
                                         C.c_void_p]
_lib.spiral_launch_count.restype = C.c_int64
_lib.spiral_launch_count.argtypes = [C.c_void_p]
_lib.spiral_last_status.restype = C.c_int
_lib.spiral_last_status.argtypes = [C.c_void_p, _I32P]
_lib.spiral_free.restype = None
_lib.spiral_free.argtypes = [C.c_void_p, C.c_void_p]
_lib.spiral_strerror.restype = C.c_char_p
_lib.spiral_strerror.argtypes = [C.c_int]
_lib.spiral_last_cuda_error.restype = C.c_char_p
_lib.spiral_last_cuda_error.argtypes = []


class SpiralError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = f"{where}: {spiral_strerror(code)} ({code})"
        if code == SPIRAL_ERR_CUDA:
            msg += f" [{spiral_last_cuda_error()}]"
        super().__init__(msg)


def _check(code: int, where: str):
    if code != SPIRAL_OK:
        raise SpiralError(code, where)


def spiral_strerror(code: int) -> str:
    return _lib.spiral_strerror(code).decode()


def spiral_last_cuda_error() -> str:
    return _lib.spiral_last_cuda_error().decode()


def _ids(ids):
    arr = (C.c_int32 * len(ids))(*[int(i) for i in ids])
    return arr


def _stream_ptr(stream=None):
    s = stream if stream is not None else torch.cuda.current_stream()
    return C.c_void_p(s.cuda_stream)


def _ptr(t):
    return C.c_void_p(t.data_ptr()) if t is not None else None


def pack_weights(w: dict) -> dict:
    """Plain per-matrix weights (wq, wk, wv, w_gate, w_up, ...) -> the layout the library reads:
    wqkv = rows of q, k, v stacked; w_gate_up = gate and up rows interleaved (2i gate, 2i+1 up)."""
    L = len(w["wq"])
    out = {"embed": w["embed"].contiguous(), "lm_head": w.get("lm_head"), "final_norm": w["final_norm"],
           "ln1": w["ln1"], "ln2": w["ln2"], "wo": [t.contiguous() for t in w["wo"]],
           "w_down": [t.contiguous() for t in w["w_down"]], "q_norm": w["q_norm"], "k_norm": w["k_norm"],
           "wqkv": [], "bqkv": [], "w_gate_up": []}
    for l in range(L):
        out["wqkv"].append(torch.cat([w["wq"][l], w["wk"][l], w["wv"][l]], 0).contiguous())
        if w["bq"][l] is not None:
            out["bqkv"].append(torch.cat([w["bq"][l], w["bk"][l], w["bv"][l]], 0).contiguous())
        else:
            out["bqkv"].append(None)
        g, u = w["w_gate"][l], w["w_up"][l]
        out["w_gate_up"].append(torch.stack([g, u], 1).reshape(2 * g.shape[0], g.shape[1]).contiguous())
    return out


class Ctx:
    """Owner of a spiral_ctx handle; keeps the weight tensors alive."""

    def __init__(self, handle, desc, packed, keep):
        self.handle, self.desc, self.packed, self._keep = handle, desc, packed, keep


class Kv:
    def __init__(self, handle, ctx, pool):
        self.handle, self.ctx, self.pool = handle, ctx, pool


def spiral_init(desc: dict, packed: dict, device: int = 0, max_batch: int = 128, max_ctx: int = 4096) -> Ctx:
    """desc: architecture dict (see ModelDesc); packed: output of pack_weights on CUDA tensors."""
    md = ModelDesc(**{k: desc[k] for k, _ in ModelDesc._fields_})
    L = desc["n_layers"]
    keep = []

    def arr(name, present=True):
        if not present:
            return None
        a = (C.c_void_p * L)(*[t.data_ptr() if t is not None else None for t in packed[name]])
        keep.append(a)
        return C.cast(a, _PP)

    for name in ("embed", "final_norm"):
        assert packed[name].is_cuda and packed[name].dtype == torch.bfloat16
    w = Weights(embed=packed["embed"].data_ptr(),
                lm_head=packed["lm_head"].data_ptr() if packed.get("lm_head") is not None else None,
                final_norm=packed["final_norm"].data_ptr(),
                ln1=arr("ln1"), wqkv=arr("wqkv"), bqkv=arr("bqkv", bool(desc["qkv_bias"])),
                q_norm=arr("q_norm", bool(desc["qk_norm"])), k_norm=arr("k_norm", bool(desc["qk_norm"])),
                wo=arr("wo"), ln2=arr("ln2"), w_gate_up=arr("w_gate_up"), w_down=arr("w_down"))
    h = C.c_void_p()
    _check(_lib.spiral_init(C.byref(h), C.byref(md), C.byref(w), device, max_batch, max_ctx), "spiral_init")
    return Ctx(h, dict(desc), packed, keep)


def spiral_kv_page_bytes(desc: dict, page_size: int = 16) -> int:
    md = ModelDesc(**{k: desc[k] for k, _ in ModelDesc._fields_})
    return _lib.spiral_kv_page_bytes(C.byref(md), page_size)


def spiral_kv_alloc(ctx: Ctx, pool: torch.Tensor, page_size: int, max_games: int, max_ctx: int,
                    kv_dtype: int = SPIRAL_KV_F16) -> Kv:
    """pool: a CUDA tensor the caller keeps alive; its bytes become the page pool."""
    h = C.c_void_p()
    nbytes = pool.numel() * pool.element_size()
    _check(_lib.spiral_kv_alloc(ctx.handle, _ptr(pool), nbytes, page_size, kv_dtype, max_games, max_ctx,
                                C.byref(h)), "spiral_kv_alloc")
    kv = Kv(h, ctx, pool)
    kv.dtype = torch.float16 if kv_dtype == SPIRAL_KV_F16 else torch.bfloat16
    return kv


def spiral_kv_release(kv: Kv, game_ids) -> None:
    _check(_lib.spiral_kv_release(kv.handle, len(game_ids), _ids(game_ids)), "spiral_kv_release")


def spiral_kv_truncate(kv: Kv, game_ids, new_len) -> None:
    _check(_lib.spiral_kv_truncate(kv.handle, len(game_ids), _ids(game_ids), _ids(new_len)), "spiral_kv_truncate")


KERNEL_CLASSES = ["attn", "attn_merge", "qkv", "o", "gate_up", "down", "lm_head", "other"]


def spiral_profile(ctx: Ctx, class_mask: int) -> None:
    _check(_lib.spiral_profile(ctx.handle, class_mask), "spiral_profile")


def spiral_profile_read(ctx: Ctx, kernel_class: int) -> tuple[float, int]:
    """(summed device milliseconds, launches) of one kernel class since the last spiral_profile."""
    ms, n = C.c_double(), C.c_int64()
    _check(_lib.spiral_profile_read(ctx.handle, kernel_class, C.byref(ms), C.byref(n)), "spiral_profile_read")
    return ms.value, n.value


def spiral_kv_seq_len(kv: Kv, game_id: int) -> int:
    out = C.c_int32()
    _check(_lib.spiral_kv_seq_len(kv.handle, game_id, C.byref(out)), "spiral_kv_seq_len")
    return out.value


def spiral_kv_free_pages(kv: Kv) -> int:
    out = C.c_int32()
    _check(_lib.spiral_kv_free_pages(kv.handle, C.byref(out)), "spiral_kv_free_pages")
    return out.value


def spiral_kv_load(ctx: Ctx, kv: Kv, game_id: int, layer: int, k: torch.Tensor, v: torch.Tensor, stream=None):
    assert k.is_cuda and k.dtype == kv.dtype and v.dtype == kv.dtype and k.is_contiguous() and v.is_contiguous()
    _check(_lib.spiral_kv_load(ctx.handle, kv.handle, game_id, layer, k.shape[0], _ptr(k), _ptr(v),
                               _stream_ptr(stream)), "spiral_kv_load")


def spiral_prefill(ctx: Ctx, kv: Kv, game_ids, tokens: torch.Tensor, offsets, last_logits=None, stream=None):
    assert tokens.is_cuda and tokens.dtype == torch.int32
    _check(_lib.spiral_prefill(ctx.handle, kv.handle, len(game_ids), _ids(game_ids), _ptr(tokens),
                               _ids(offsets), _ptr(last_logits), _stream_ptr(stream)), "spiral_prefill")


def spiral_decode_step(ctx: Ctx, kv: Kv, game_ids, tok_in: torch.Tensor, gumbel: torch.Tensor,
                       temperature: float, tok_out: torch.Tensor, logits_dbg=None, stream=None):
    assert tok_in.is_cuda and tok_in.dtype == torch.int32 and tok_out.dtype == torch.int32
    assert gumbel.is_cuda and gumbel.dtype == torch.float32 and gumbel.is_contiguous()
    ids = game_ids if isinstance(game_ids, C.Array) else _ids(game_ids)
    _check(_lib.spiral_decode_step(ctx.handle, kv.handle, len(ids), ids, _ptr(tok_in), _ptr(gumbel),
                                   float(temperature), _ptr(tok_out), _ptr(logits_dbg), _stream_ptr(stream)),
           "spiral_decode_step")


def spiral_decode_step_logprob(ctx: Ctx, kv: Kv, game_ids, tok_in: torch.Tensor, gumbel: torch.Tensor,
                               temperature: float, tok_out: torch.Tensor, logprob: torch.Tensor, logits_dbg=None,
                               stream=None):
    """spiral_decode_step that also writes log softmax(logits / T)[sampled token] into `logprob` (fp32 [n])."""
    assert tok_in.is_cuda and tok_in.dtype == torch.int32 and tok_out.dtype == torch.int32
    assert gumbel.is_cuda and gumbel.dtype == torch.float32 and gumbel.is_contiguous()
    assert logprob.is_cuda and logprob.dtype == torch.float32 and logprob.numel() >= len(game_ids)
    ids = game_ids if isinstance(game_ids, C.Array) else _ids(game_ids)
    _check(_lib.spiral_decode_step_logprob(ctx.handle, kv.handle, len(ids), ids, _ptr(tok_in), _ptr(gumbel),
                                           float(temperature), _ptr(tok_out), _ptr(logprob), _ptr(logits_dbg),
                                           _stream_ptr(stream)), "spiral_decode_step_logprob")


def spiral_decode_step_nucleus(ctx: Ctx, kv: Kv, game_ids, tok_in: torch.Tensor, gumbel: torch.Tensor,
                               temperature: float, top_p: float, tok_out: torch.Tensor, logits_dbg=None, stream=None):
    """spiral_decode_step with nucleus (top-p) sampling."""
    assert tok_in.is_cuda and tok_in.dtype == torch.int32 and tok_out.dtype == torch.int32
    assert gumbel.is_cuda and gumbel.dtype == torch.float32 and gumbel.is_contiguous()
    ids = game_ids if isinstance(game_ids, C.Array) else _ids(game_ids)
    _check(_lib.spiral_decode_step_nucleus(ctx.handle, kv.handle, len(ids), ids, _ptr(tok_in), _ptr(gumbel),
                                           float(temperature), float(top_p), _ptr(tok_out), _ptr(logits_dbg),
                                           _stream_ptr(stream)), "spiral_decode_step_nucleus")


def spiral_sample_nucleus(ctx: Ctx, logits: torch.Tensor, gumbel, temperature: float, top_p: float,
                          tok_out: torch.Tensor, stream=None):
    """Nucleus sampler alone on fp32 logits [n][vocab] held by the caller."""
    assert logits.is_cuda and logits.dtype == torch.float32 and logits.is_contiguous() and logits.dim() == 2
    assert gumbel is None or (gumbel.is_cuda and gumbel.dtype == torch.float32 and gumbel.is_contiguous())
    assert tok_out.is_cuda and tok_out.dtype == torch.int32
    _check(_lib.spiral_sample_nucleus(ctx.handle, logits.shape[0], _ptr(logits), _ptr(gumbel), float(temperature),
                                      float(top_p), _ptr(tok_out), _stream_ptr(stream)), "spiral_sample_nucleus")


def spiral_rae_update(baselines, alpha: float, game_of, returns):
    """Role-conditioned advantage estimation on the host.  baselines: float64 numpy [n_games][2], updated
    in place; game_of: ints [n_traj]; returns: [n_traj][2].  Gives the advantages, float64 [n_traj][2]."""
    import numpy as np
    assert isinstance(baselines, np.ndarray) and baselines.dtype == np.float64 and baselines.flags.c_contiguous
    assert baselines.ndim == 2 and baselines.shape[1] == 2
    ret = np.ascontiguousarray(np.asarray(returns, dtype=np.float64)).reshape(-1, 2)
    adv = np.empty_like(ret)
    dp = C.POINTER(C.c_double)
    _check(_lib.spiral_rae_update(baselines.ctypes.data_as(dp), baselines.shape[0], float(alpha), ret.shape[0],
                                  _ids(list(game_of)), ret.ctypes.data_as(dp), adv.ctypes.data_as(dp)),
           "spiral_rae_update")
    return adv


class Sched:
    """Handle of an episode scheduler (spiral_sched_*)."""

    def __init__(self, handle, ctx, kv):
        self.handle, self.ctx, self.kv = handle, ctx, kv
        self.poll_buf = None            # reused by spiral_sched_poll


SCHED_STATS = ["waiting", "running", "finished_unread", "free_pages", "reserved_pages", "decoded", "dropped", "appended"]


def spiral_sched_create(ctx: Ctx, kv: Kv, eos_token: int = -1) -> Sched:
    h = C.c_void_p()
    _check(_lib.spiral_sched_create(ctx.handle, kv.handle, int(eos_token), C.byref(h)), "spiral_sched_create")
    return Sched(h, ctx, kv)


def spiral_sched_free(sched: Sched) -> None:
    if sched.handle:
        _lib.spiral_sched_free(sched.handle)
        sched.handle = None


def spiral_sched_open(sched: Sched) -> int:
    g = (C.c_int32 * 1)()
    _check(_lib.spiral_sched_open(sched.handle, g), "spiral_sched_open")
    return int(g[0])


def spiral_kv_fork(ctx: Ctx, kv: Kv, src_game: int, dst_game: int, n_tokens: int, stream=None) -> None:
    _check(_lib.spiral_kv_fork(ctx.handle, kv.handle, int(src_game), int(dst_game), int(n_tokens), _stream_ptr(stream)),
           "spiral_kv_fork")


def spiral_sched_fork(sched: Sched, src_game: int, stream=None) -> int:
    g = (C.c_int32 * 1)()
    _check(_lib.spiral_sched_fork(sched.handle, int(src_game), g, _stream_ptr(stream)), "spiral_sched_fork")
    return int(g[0])


def spiral_sched_close(sched: Sched, game: int) -> None:
    _check(_lib.spiral_sched_close(sched.handle, int(game)), "spiral_sched_close")


def spiral_sched_turn(sched: Sched, game: int, obs_tokens, max_new_tokens: int) -> None:
    obs = list(obs_tokens)
    _check(_lib.spiral_sched_turn(sched.handle, int(game), len(obs), _ids(obs), int(max_new_tokens)), "spiral_sched_turn")


def spiral_sched_policy(sched: Sched, admit_tokens: int, low_water: int) -> None:
    _check(_lib.spiral_sched_policy(sched.handle, int(admit_tokens), int(low_water)), "spiral_sched_policy")


def spiral_sched_tick(sched: Sched, gumbel: torch.Tensor, temperature: float = 1.0, stream=None) -> int:
    assert gumbel.is_cuda and gumbel.dtype == torch.float32 and gumbel.is_contiguous()
    rc = _lib.spiral_sched_tick(sched.handle, _ptr(gumbel), float(temperature), _stream_ptr(stream))
    if rc < 0:
        _check(rc, "spiral_sched_tick")
    return rc


def spiral_sched_poll(sched: Sched, max_tokens: int = 1 << 16):
    """None, or (game, response tokens, reason) of one finished turn; reason 1 = end-of-sequence, 2 = budget."""
    g, n, why = (C.c_int32 * 1)(), (C.c_int32 * 1)(), (C.c_int32 * 1)()
    if sched.poll_buf is None or len(sched.poll_buf) < max_tokens:
        sched.poll_buf = (C.c_int32 * max_tokens)()
    buf = sched.poll_buf
    rc = _lib.spiral_sched_poll(sched.handle, g, buf, max_tokens, n, why)
    if rc < 0:
        _check(rc, "spiral_sched_poll")
    if rc == 0:
        return None
    return int(g[0]), [int(buf[i]) for i in range(n[0])], int(why[0])


def spiral_sched_collect_logprob(sched: Sched, on: bool = True) -> None:
    _check(_lib.spiral_sched_collect_logprob(sched.handle, int(bool(on))), "spiral_sched_collect_logprob")


def spiral_sched_poll_logprob(sched: Sched, max_tokens: int = 1 << 16):
    """None, or (game, response tokens, their log-probabilities, reason) of one finished turn."""
    g, n, why = (C.c_int32 * 1)(), (C.c_int32 * 1)(), (C.c_int32 * 1)()
    if sched.poll_buf is None or len(sched.poll_buf) < max_tokens:
        sched.poll_buf = (C.c_int32 * max_tokens)()
    lp = (C.c_float * max_tokens)()
    rc = _lib.spiral_sched_poll_logprob(sched.handle, g, sched.poll_buf, lp, max_tokens, n, why)
    if rc < 0:
        _check(rc, "spiral_sched_poll_logprob")
    if rc == 0:
        return None
    return int(g[0]), [int(sched.poll_buf[i]) for i in range(n[0])], [float(lp[i]) for i in range(n[0])], int(why[0])


def spiral_sched_stats(sched: Sched) -> dict:
    out = (C.c_int64 * 8)()
    _check(_lib.spiral_sched_stats(sched.handle, out, 8), "spiral_sched_stats")
    return {k: int(out[i]) for i, k in enumerate(SCHED_STATS)}


def spiral_decode_step_host(ctx: Ctx, kv: Kv, game_ids, tok_in: torch.Tensor, gumbel: torch.Tensor,
                            temperature: float, tok_out: torch.Tensor, stream=None):
    """tok_in / gumbel / tok_out are HOST tensors (pinned recommended)."""
    assert not tok_in.is_cuda and not gumbel.is_cuda and not tok_out.is_cuda
    ids = game_ids if isinstance(game_ids, C.Array) else _ids(game_ids)
    _check(_lib.spiral_decode_step_host(ctx.handle, kv.handle, len(ids), ids, _ptr(tok_in), _ptr(gumbel),
                                        float(temperature), _ptr(tok_out), _stream_ptr(stream)),
           "spiral_decode_step_host")


def spiral_linear(ctx: Ctx, w: torch.Tensor, x: torch.Tensor, path: int = 0, stream=None) -> torch.Tensor:
    assert w.dtype == torch.bfloat16 and x.dtype == torch.float16 and w.is_contiguous() and x.is_contiguous()
    y = torch.empty(x.shape[0], w.shape[0], dtype=torch.float32, device=x.device)
    _check(_lib.spiral_linear(ctx.handle, _ptr(w), w.shape[0], w.shape[1], _ptr(x), x.shape[0], _ptr(y), path,
                              _stream_ptr(stream)), "spiral_linear")
    return y


def spiral_attention(ctx: Ctx, kv: Kv, layer: int, game_ids, ctx_len, q: torch.Tensor, stream=None):
    assert q.dtype == torch.float32 and q.is_contiguous()
    out = torch.empty_like(q)
    _check(_lib.spiral_attention(ctx.handle, kv.handle, layer, len(game_ids), _ids(game_ids), _ids(ctx_len),
                                 _ptr(q), _ptr(out), _stream_ptr(stream)), "spiral_attention")
    return out


def spiral_kv_block_table(kv: Kv, game_id: int, max_entries: int = 4096) -> list[int]:
    """Page ids the game owns, in position order (host bookkeeping, no device work)."""
    out = (C.c_int32 * max_entries)()
    n = _lib.spiral_kv_block_table(kv.handle, game_id, out, max_entries)
    if n < 0:
        raise SpiralError(n, "spiral_kv_block_table")
    return list(out[:n])


def spiral_attention_static(pool: torch.Tensor, n_pages: int, n_layers: int, layer: int, kv_dtype: int,
                            n_q_heads: int, n_kv_heads: int, head_dim: int, block_table: torch.Tensor, ctx_len,
                            q: torch.Tensor, out: torch.Tensor, stream=None) -> None:
    """Attention over a caller-owned paged pool without any allocation inside the library: every
    buffer, `out` included, comes from the caller (see include/spiral.h for who needs that)."""
    assert block_table.is_cuda and block_table.dtype == torch.int32 and block_table.is_contiguous()
    assert q.dtype == torch.float32 and q.is_contiguous() and out.dtype == torch.float32 and out.is_contiguous()
    _check(_lib.spiral_attention_static(pool.device.index or 0, _ptr(pool), n_pages, n_layers, layer, kv_dtype,
                                        n_q_heads, n_kv_heads, head_dim, _ptr(block_table), block_table.shape[1],
                                        block_table.shape[0], _ids(ctx_len), _ptr(q), _ptr(out),
                                        _stream_ptr(stream)), "spiral_attention_static")


_lib.spiral_attention_static_status.restype = C.c_int
_lib.spiral_attention_static_status.argtypes = [C.c_int, _I32P]


def spiral_attention_static_status(device: int = 0) -> tuple[int, int]:
    """(return code, raw status word) of the static attention entry point's device-side checks."""
    d = C.c_int32()
    rc = _lib.spiral_attention_static_status(device, C.byref(d))
    return rc, d.value


_lib.spiral_selftest_wait_timeout.restype = C.c_int
_lib.spiral_selftest_wait_timeout.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p]


def spiral_selftest_wait_timeout(ctx: Ctx, kv, which: int, stream=None) -> None:
    """Runs one kernel whose bounded wait must run out (see include/spiral.h); the finding is read with
    spiral_last_status."""
    _check(_lib.spiral_selftest_wait_timeout(ctx.handle, kv.handle if kv is not None else None, which,
                                             _stream_ptr(stream)), "spiral_selftest_wait_timeout")


_lib.spiral_read_ceiling.restype = C.c_int
_lib.spiral_read_ceiling.argtypes = [C.c_int, C.c_void_p, C.c_size_t, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int,
                                     C.c_int, C.c_void_p, C.POINTER(C.c_double)]


def spiral_read_ceiling(device: int, buf, stage_bytes: int = 16384, stages: int = 6, ctas_per_sm: int = 1,
                        blocked: int = 0, tiled: int = 0, passes: int = 1, stream=None) -> float:
    """GB/s of a pure read stream over `buf` (a device tensor several times the L2 size)."""
    out = C.c_double()
    nbytes = buf.numel() * buf.element_size()
    _check(_lib.spiral_read_ceiling(device, _ptr(buf), nbytes, stage_bytes, stages, ctas_per_sm, int(blocked), int(tiled), passes,
                                    _stream_ptr(stream), C.byref(out)), "spiral_read_ceiling")
    return out.value


def spiral_launch_count(ctx: Ctx) -> int:
    return _lib.spiral_launch_count(ctx.handle)


def spiral_last_status(ctx: Ctx) -> tuple[int, int]:
    d = C.c_int32()
    rc = _lib.spiral_last_status(ctx.handle, C.byref(d))
    return rc, d.value


def spiral_free(ctx: Ctx | None, kv: Kv | None) -> None:
    _lib.spiral_free(ctx.handle if ctx else None, kv.handle if kv else None)
    if ctx:
        ctx.handle = None
    if kv:
        kv.handle = None


__all__ = [n for n in dir() if n.startswith("spiral_") or n.startswith("SPIRAL_")] + \
          ["pack_weights", "SpiralError", "Ctx", "Kv", "ModelDesc", "Weights", "EXPORTS", "LIB_PATH", "KERNEL_CLASSES", "Sched", "SCHED_STATS"]
