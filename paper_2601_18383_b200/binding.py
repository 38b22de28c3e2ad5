"""ctypes binding of libdynts.so: argument marshalling only.

Every function has the name and the argument order of its C counterpart in include/dynts.h.
Tensor arguments may be torch tensors (their data_ptr() is passed), integers (raw addresses) or
None.  Nothing here computes: every step of the path runs in the library's CUDA kernels.  If
the library has not been built, importing this module raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdynts.so")

DYNTS_OK = 0
DYNTS_ERR_INVALID_ARG = 1
DYNTS_ERR_OOM = 2
DYNTS_ERR_CAPACITY = 3
DYNTS_ERR_BUDGET = 4
DYNTS_ERR_STATE = 5
DYNTS_ERR_CUDA = 6
DYNTS_ERR_DEVICE = 7
DYNTS_BF16 = 0
DYNTS_FP32 = 1
DYNTS_BF16_KV8 = 2
DYNTS_SCORE_ATTENTION = 0
DYNTS_SCORE_EXTERNAL = 1

_STATUS_NAMES = {
    0: "DYNTS_OK", 1: "DYNTS_ERR_INVALID_ARG", 2: "DYNTS_ERR_OOM", 3: "DYNTS_ERR_CAPACITY",
    4: "DYNTS_ERR_BUDGET", 5: "DYNTS_ERR_STATE", 6: "DYNTS_ERR_CUDA", 7: "DYNTS_ERR_DEVICE",
}


class DyntsError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{_STATUS_NAMES.get(status, status)}: {message}")
        self.status = status


class dynts_config_t(C.Structure):
    _fields_ = [
        ("layers", C.c_int), ("batch", C.c_int), ("q_heads", C.c_int), ("kv_heads", C.c_int),
        ("head_dim", C.c_int), ("budget", C.c_int), ("window", C.c_int), ("evict_interval", C.c_int),
        ("capacity", C.c_int), ("dtype", C.c_int),
        ("seq_budgets", C.POINTER(C.c_int)),
        ("storage", C.c_void_p), ("storage_bytes", C.c_size_t), ("stream", C.c_void_p),
    ]


if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python paper_2601_18383_b200/build.py` "
        "(there is no CPU fallback)")

lib = C.CDLL(LIB_PATH)

_P = C.c_void_p
_sigs = {
    "dynts_cache_create": (_P, [C.c_int] * 5),
    "dynts_cache_set_shape": (C.c_int, [_P, C.c_int, C.c_int, C.c_int, C.c_int]),
    "dynts_cache_bytes": (C.c_size_t, [C.POINTER(dynts_config_t)]),
    "dynts_cache_create_ex": (C.c_int, [C.POINTER(dynts_config_t), C.POINTER(_P)]),
    "dynts_cache_destroy": (None, [_P]),
    "dynts_cache_set_stream": (C.c_int, [_P, _P]),
    "dynts_prefill": (C.c_int, [_P, _P, _P, C.c_int, C.c_int]),
    "dynts_prefill_attn": (C.c_int, [_P, _P, _P, _P, _P, C.c_int, C.c_int]),
    "dynts_prompt_attn": (C.c_int, [_P, _P, _P, _P, _P, C.c_int]),
    "dynts_prefill_attn_layer": (C.c_int, [_P, C.c_int, _P, _P, _P, _P, C.c_int, C.c_int]),
    "dynts_cache_refresh_lengths": (C.c_int, [_P]),
    "dynts_prefill_seq": (C.c_int, [_P, C.c_int, _P, _P, C.c_int, C.c_int]),
    "dynts_decode_attn": (C.c_int, [_P, _P, _P, _P, _P, _P]),
    "dynts_decode_attn_layer": (C.c_int, [_P, C.c_int, _P, _P, _P, _P, _P]),
    "dynts_decode_attn_host": (C.c_int, [_P, _P, _P, _P, _P]),
    "dynts_evict": (C.c_int, [_P, C.c_int]),
    "dynts_evict_global": (C.c_int, [_P, C.c_int]),
    "dynts_aggregate_scores": (C.c_int, [_P, _P]),
    "dynts_evict_ex": (C.c_int, [_P, C.POINTER(C.c_int)]),
    "dynts_evict_noalloc": (C.c_int, [_P, _P, _P, _P] + [C.c_int] * 8 + [_P]),
    "dynts_evict_noalloc_status": (C.c_int, [_P]),
    "dynts_seq_reset": (C.c_int, [_P, C.c_int]),
    "dynts_cache_len": (C.c_int, [_P, C.c_int]),
    "dynts_cache_capacity": (C.c_int, [_P]),
    "dynts_cache_scores": (_P, [_P]),
    "dynts_cache_export": (C.c_int, [_P, C.c_int, C.c_int, C.c_int, _P, _P, _P, _P, C.POINTER(C.c_int)]),
    "dynts_cache_import": (C.c_int, [_P, C.c_int, C.c_int, C.c_int, _P, _P, _P, _P, C.c_int, C.c_int]),
    "dynts_poll_error": (C.c_int, [_P]),
    "dynts_synchronize": (C.c_int, [_P]),
    "dynts_cache_set_launch": (C.c_int, [_P, C.c_int, C.c_int]),
    "dynts_cache_set_evict_launch": (C.c_int, [_P, C.c_int]),
    "dynts_cache_set_wait_limit": (C.c_int, [_P, C.c_uint]),
    "dynts_debug_drop_tile_load": (C.c_int, [_P, C.c_int]),
    "dynts_cache_launch_count": (C.c_longlong, [_P]),
    "dynts_cache_set_score_source": (C.c_int, [_P, C.c_int]),
    "dynts_cache_set_kv_scale": (C.c_int, [_P, C.c_float, C.c_float]),
    "dynts_append_scores": (C.c_int, [_P, _P]),
    "dynts_evict_at_budget": (C.c_int, [_P, C.c_int, C.c_double]),
    "dynts_predictor_mlp_scratch_bytes": (C.c_size_t, [C.c_int, C.c_int]),
    "dynts_predictor_mlp": (C.c_int, [_P] * 7 + [C.c_int, C.c_int, C.c_int, _P, C.c_size_t, _P, _P]),
    "dynts_evict_stats": (C.c_int, [_P, C.POINTER(C.c_longlong), C.POINTER(C.c_longlong)]),
    "dynts_last_error": (C.c_char_p, []),
    "dynts_version": (C.c_char_p, []),
}
for _name, (_res, _args) in _sigs.items():
    _fn = getattr(lib, _name)
    _fn.restype = _res
    _fn.argtypes = _args


def _ptr(x):
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if hasattr(x, "data_ptr"):
        return x.data_ptr()
    if hasattr(x, "ctypes"):          # numpy array (host buffers)
        return x.ctypes.data
    raise TypeError(f"cannot take the address of {type(x)}")


def dynts_last_error() -> str:
    return lib.dynts_last_error().decode()


def dynts_version() -> str:
    return lib.dynts_version().decode()


def _check(status: int) -> int:
    if status != DYNTS_OK:
        raise DyntsError(status, dynts_last_error())
    return status


def dynts_cache_create(layers, kv_heads, head_dim, budget, window):
    h = lib.dynts_cache_create(layers, kv_heads, head_dim, budget, window)
    if not h:
        raise DyntsError(DYNTS_ERR_INVALID_ARG, dynts_last_error())
    return h


def dynts_cache_set_shape(c, batch, q_heads, dtype, evict_interval):
    return _check(lib.dynts_cache_set_shape(c, batch, q_heads, dtype, evict_interval))


def make_config(layers, batch, q_heads, kv_heads, head_dim, budget, window, evict_interval, dtype=DYNTS_BF16,
                capacity=0, seq_budgets: Optional[Sequence[int]] = None, storage=None, storage_bytes=0, stream=None):
    cfg = dynts_config_t()
    cfg.layers, cfg.batch, cfg.q_heads, cfg.kv_heads, cfg.head_dim = layers, batch, q_heads, kv_heads, head_dim
    cfg.budget, cfg.window, cfg.evict_interval, cfg.capacity, cfg.dtype = budget, window, evict_interval, capacity, dtype
    if seq_budgets is not None:
        arr = (C.c_int * len(seq_budgets))(*[int(x) for x in seq_budgets])
        cfg._keep = arr
        cfg.seq_budgets = C.cast(arr, C.POINTER(C.c_int))
    cfg.storage = _ptr(storage)
    cfg.storage_bytes = storage_bytes
    cfg.stream = stream
    return cfg


def dynts_cache_bytes(cfg: dynts_config_t) -> int:
    return lib.dynts_cache_bytes(C.byref(cfg))


def dynts_cache_create_ex(cfg: dynts_config_t):
    out = _P()
    _check(lib.dynts_cache_create_ex(C.byref(cfg), C.byref(out)))
    return out.value


def dynts_cache_destroy(c):
    lib.dynts_cache_destroy(c)


def dynts_cache_set_stream(c, stream):
    return _check(lib.dynts_cache_set_stream(c, stream))


def dynts_prefill(c, k, v, n_tokens, n_pinned):
    return _check(lib.dynts_prefill(c, _ptr(k), _ptr(v), n_tokens, n_pinned))


def dynts_prefill_attn(c, q, k, v, out, n_tokens, n_pinned):
    return _check(lib.dynts_prefill_attn(c, _ptr(q), _ptr(k), _ptr(v), _ptr(out), n_tokens, n_pinned))


def dynts_prefill_attn_layer(c, layer, q, k, v, out, n_tokens, n_pinned):
    return _check(lib.dynts_prefill_attn_layer(c, layer, _ptr(q), _ptr(k), _ptr(v), _ptr(out), n_tokens, n_pinned))


def dynts_cache_refresh_lengths(c):
    return _check(lib.dynts_cache_refresh_lengths(c))


def dynts_prompt_attn(c, q, k, v, out, n_tokens):
    return _check(lib.dynts_prompt_attn(c, _ptr(q), _ptr(k), _ptr(v), _ptr(out), n_tokens))


def dynts_prefill_seq(c, seq, k, v, n_tokens, n_pinned):
    return _check(lib.dynts_prefill_seq(c, seq, _ptr(k), _ptr(v), n_tokens, n_pinned))


def dynts_decode_attn(c, q, k_new, v_new, out, scores=None):
    return _check(lib.dynts_decode_attn(c, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(out), _ptr(scores)))


def dynts_decode_attn_layer(c, layer, q, k_new, v_new, out, scores=None):
    return _check(lib.dynts_decode_attn_layer(c, layer, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(out), _ptr(scores)))


def dynts_decode_attn_host(c, q, k_new, v_new, out):
    return _check(lib.dynts_decode_attn_host(c, _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(out)))


def dynts_evict(c, budget=0):
    return _check(lib.dynts_evict(c, budget))


def dynts_evict_global(c, budget=0):
    return _check(lib.dynts_evict_global(c, budget))


def dynts_aggregate_scores(c, agg):
    return _check(lib.dynts_aggregate_scores(c, _ptr(agg)))


def dynts_evict_ex(c, seq_targets: Sequence[int]):
    arr = (C.c_int * len(seq_targets))(*[int(x) for x in seq_targets])
    return _check(lib.dynts_evict_ex(c, arr))


def dynts_evict_noalloc(K, V, pos, score, n_slabs, head_dim, dtype, capacity, n_rows, n_pinned, window, target,
                        stream=None):
    """In-place eviction of caller-owned slabs without any allocation (see include/dynts.h)."""
    return _check(lib.dynts_evict_noalloc(_ptr(K), _ptr(V), _ptr(pos), _ptr(score), n_slabs, head_dim, dtype,
                                          capacity, n_rows, n_pinned, window, target, stream))


def dynts_evict_noalloc_status(stream=None):
    """Waits for the stream; raises if the last allocation-free eviction recorded a device-side check."""
    return _check(lib.dynts_evict_noalloc_status(stream))


def dynts_seq_reset(c, seq):
    return _check(lib.dynts_seq_reset(c, seq))


def dynts_cache_len(c, seq=0) -> int:
    return lib.dynts_cache_len(c, seq)


def dynts_cache_capacity(c) -> int:
    return lib.dynts_cache_capacity(c)


def dynts_cache_scores(c) -> Optional[int]:
    return lib.dynts_cache_scores(c)


def dynts_cache_export(c, layer, seq, head, K, V, pos, score) -> int:
    n = C.c_int(0)
    _check(lib.dynts_cache_export(c, layer, seq, head, _ptr(K), _ptr(V), _ptr(pos), _ptr(score), C.byref(n)))
    return n.value


def dynts_cache_import(c, layer, seq, head, K, V, pos, score, n, n_pinned):
    return _check(lib.dynts_cache_import(c, layer, seq, head, _ptr(K), _ptr(V), _ptr(pos), _ptr(score), n, n_pinned))


def dynts_poll_error(c):
    return _check(lib.dynts_poll_error(c))


def dynts_synchronize(c):
    return _check(lib.dynts_synchronize(c))


def dynts_cache_set_launch(c, cluster=0, variant=0):
    return _check(lib.dynts_cache_set_launch(c, cluster, variant))


def dynts_cache_set_wait_limit(c, polls):
    return _check(lib.dynts_cache_set_wait_limit(c, polls))


def dynts_debug_drop_tile_load(c, item):
    return _check(lib.dynts_debug_drop_tile_load(c, item))


def dynts_cache_set_evict_launch(c, split=0):
    return _check(lib.dynts_cache_set_evict_launch(c, split))


def dynts_cache_set_score_source(c, source):
    return _check(lib.dynts_cache_set_score_source(c, source))


def dynts_cache_set_kv_scale(c, k_scale, v_scale):
    return _check(lib.dynts_cache_set_kv_scale(c, float(k_scale), float(v_scale)))


def dynts_append_scores(c, s_new):
    return _check(lib.dynts_append_scores(c, _ptr(s_new)))


def dynts_evict_at_budget(c, budget_B, ratio):
    return _check(lib.dynts_evict_at_budget(c, budget_B, ratio))


def dynts_predictor_mlp_scratch_bytes(d, batch) -> int:
    return lib.dynts_predictor_mlp_scratch_bytes(d, batch)


def dynts_predictor_mlp(h, W1, b1, W2, b2, W3, b3, d, batch, activation, scratch, scratch_bytes, scores, stream=None):
    return _check(lib.dynts_predictor_mlp(_ptr(h), _ptr(W1), _ptr(b1), _ptr(W2), _ptr(b2), _ptr(W3), _ptr(b3), d, batch,
                                          activation, _ptr(scratch), scratch_bytes, _ptr(scores), stream))


def dynts_evict_stats(c):
    """(rows scanned, rows moved) of the most recent eviction."""
    a, b = C.c_longlong(0), C.c_longlong(0)
    _check(lib.dynts_evict_stats(c, C.byref(a), C.byref(b)))
    return a.value, b.value


def dynts_cache_launch_count(c) -> int:
    return lib.dynts_cache_launch_count(c)


class Cache:
    """Convenience holder: takes the cache's device storage from PyTorch and keeps it alive.

    It only forwards to the functions above."""

    def __init__(self, layers, batch, q_heads, kv_heads, head_dim, budget, window, evict_interval,
                 dtype="bf16", seq_budgets=None, capacity=0, device="cuda:0"):
        import torch
        self.torch = torch
        self.device = torch.device(device)
        self.dtype_name = dtype
        self.torch_dtype = {"bf16": torch.bfloat16, "fp32": torch.float32, "bf16_kv8": torch.bfloat16}[dtype]   # q, k, v, out
        self.slab_dtype = torch.uint8 if dtype == "bf16_kv8" else self.torch_dtype   # rows as exported (E4M3 codes)
        self.layers, self.batch, self.q_heads, self.kv_heads, self.head_dim = layers, batch, q_heads, kv_heads, head_dim
        cfg = make_config(layers, batch, q_heads, kv_heads, head_dim, budget, window, evict_interval,
                          {"bf16": DYNTS_BF16, "fp32": DYNTS_FP32, "bf16_kv8": DYNTS_BF16_KV8}[dtype], capacity, seq_budgets)
        nbytes = dynts_cache_bytes(cfg)
        if nbytes == 0:
            raise DyntsError(DYNTS_ERR_INVALID_ARG, "invalid cache configuration")
        with torch.cuda.device(self.device):
            self.storage = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
            base = self.storage.data_ptr()
            cfg.storage = (base + 255) // 256 * 256
            cfg.storage_bytes = nbytes
            cfg.stream = torch.cuda.current_stream(self.device).cuda_stream
            self.handle = dynts_cache_create_ex(cfg)
        self.nbytes = nbytes
        self.capacity = dynts_cache_capacity(self.handle)

    def close(self):
        if getattr(self, "handle", None):
            dynts_cache_destroy(self.handle)
            self.handle = None
            self.storage = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def prefill(self, k, v, n_pinned=None):
        T = k.shape[-2]
        return dynts_prefill(self.handle, k, v, T, T if n_pinned is None else n_pinned)

    def prefill_attn(self, q, k, v, out, n_pinned=None):
        T = k.shape[-2]
        return dynts_prefill_attn(self.handle, q, k, v, out, T, T if n_pinned is None else n_pinned)

    def prefill_attn_layer(self, layer, q, k, v, out, n_pinned=None):
        T = k.shape[-2]
        return dynts_prefill_attn_layer(self.handle, layer, q, k, v, out, T, T if n_pinned is None else n_pinned)

    def refresh_lengths(self):
        return dynts_cache_refresh_lengths(self.handle)

    def prompt_attn(self, q, k, v, out):
        return dynts_prompt_attn(self.handle, q, k, v, out, k.shape[-2])

    def prefill_seq(self, seq, k, v, n_pinned=None):
        T = k.shape[-2]
        return dynts_prefill_seq(self.handle, seq, k, v, T, T if n_pinned is None else n_pinned)

    def decode_attn(self, q, k_new, v_new, out, scores=None):
        return dynts_decode_attn(self.handle, q, k_new, v_new, out, scores)

    def decode_attn_layer(self, layer, q, k_new, v_new, out, scores=None):
        return dynts_decode_attn_layer(self.handle, layer, q, k_new, v_new, out, scores)

    def decode_attn_host(self, q, k_new, v_new, out):
        return dynts_decode_attn_host(self.handle, q, k_new, v_new, out)

    def evict(self, budget=0):
        return dynts_evict(self.handle, budget)

    def evict_global(self, budget=0):
        return dynts_evict_global(self.handle, budget)

    def aggregate_scores(self, agg):
        return dynts_aggregate_scores(self.handle, agg)

    def evict_ex(self, targets):
        return dynts_evict_ex(self.handle, targets)

    def seq_reset(self, seq):
        return dynts_seq_reset(self.handle, seq)

    def len(self, seq=0):
        return dynts_cache_len(self.handle, seq)

    def set_launch(self, cluster=0, variant=0):
        return dynts_cache_set_launch(self.handle, cluster, variant)

    def set_wait_limit(self, polls):
        return dynts_cache_set_wait_limit(self.handle, polls)

    def debug_drop_tile_load(self, item):
        return dynts_debug_drop_tile_load(self.handle, item)

    def set_evict_launch(self, split=0):
        return dynts_cache_set_evict_launch(self.handle, split)

    def set_stream(self, stream):
        return dynts_cache_set_stream(self.handle, stream.cuda_stream if hasattr(stream, "cuda_stream") else stream)

    def synchronize(self):
        return dynts_synchronize(self.handle)

    def poll_error(self):
        return dynts_poll_error(self.handle)

    def set_score_source(self, source):
        return dynts_cache_set_score_source(self.handle, source)

    def set_kv_scale(self, k_scale, v_scale):
        return dynts_cache_set_kv_scale(self.handle, k_scale, v_scale)

    def append_scores(self, s_new):
        return dynts_append_scores(self.handle, s_new)

    def evict_at_budget(self, budget_B, ratio):
        r = dynts_evict_at_budget(self.handle, budget_B, ratio)
        return r

    def evict_stats(self):
        return dynts_evict_stats(self.handle)

    def launch_count(self):
        return dynts_cache_launch_count(self.handle)

    def scores_tensor(self):
        """A torch view (no copy) of the device score accumulator [L, Nb, Hkv, cap]."""
        torch = self.torch
        ptr = dynts_cache_scores(self.handle)
        off = ptr - self.storage.data_ptr()
        n = self.layers * self.batch * self.kv_heads * self.capacity
        return self.storage[off:off + 4 * n].view(torch.float32).view(self.layers, self.batch, self.kv_heads, self.capacity)

    def export_slab(self, layer, seq, head):
        """Host copies (K, V, pos, score) of one slab's n rows."""
        torch = self.torch
        n = self.len(seq)
        K = torch.empty((n, self.head_dim), dtype=self.slab_dtype)
        V = torch.empty((n, self.head_dim), dtype=self.slab_dtype)
        pos = torch.empty((n,), dtype=torch.int32)
        score = torch.empty((n,), dtype=torch.float32)
        m = dynts_cache_export(self.handle, layer, seq, head, K, V, pos, score)
        assert m == n
        return K, V, pos, score

    def import_slab(self, layer, seq, head, K, V, pos, score, n_pinned):
        n = K.shape[0]
        return dynts_cache_import(self.handle, layer, seq, head, K.contiguous(), V.contiguous(),
                                  pos.contiguous(), score.contiguous(), n, n_pinned)
