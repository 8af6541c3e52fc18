"""Thin ctypes binding of ``libkvq.so`` (see ``include/kvq.h``).

Argument marshalling only: every step of the path runs in the CUDA kernels of
the library.  Functions carry the C names; tensors are passed as
``tensor.data_ptr()`` of contiguous CUDA tensors and the stream as
``torch.cuda.current_stream().cuda_stream``.  If the library has not been
built the import of this module's ``lib()`` raises -- there is no fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libkvq.so")

KVQ_OK = 0
KVQ_ERR_ARG = -1
KVQ_ERR_CAPACITY = -2
KVQ_ERR_NO_CONTROLLER = -3
KVQ_ERR_CUDA = -4
KVQ_ERR_EMPTY = -5
KVQ_ERR_DEVICE_FLAG = -6
KVQ_ERR_NOMEM = -7
KVQ_ERR_TOO_LARGE = -8
KVQ_STATIC_MAX_PARTIALS = 8192
KVQ_EXPORT_ROW_BYTES = 128

_vp, _i, _u64p = C.c_void_p, C.c_int, C.POINTER(C.c_uint64)

# name -> (restype, argtypes); mirrors include/kvq.h one to one
SIGNATURES = {
    "kvq_create": (_i, [C.POINTER(_vp), _i, _i, _i, _i, _i, _i]),
    "kvq_create_arena": (_i, [C.POINTER(_vp), _i, _i, _i, _i, _i, _i, C.c_uint64]),
    "kvq_create_grouped": (_i, [C.POINTER(_vp), _i, _i, _i, _i, _i, _i, C.c_uint64, _i]),
    "kvq_create_perchannel": (_i, [C.POINTER(_vp), _i, _i, _i, _i, _i, _i, C.c_uint64]),
    "kvq_export_k_channels": (_i, [_vp, _i, _i, _i, _i, _i, _vp]),
    "kvq_workspace_bytes": (_i, [_i, _i, _i, _i, _i, _i, C.c_uint64, _i, C.POINTER(C.c_uint64)]),
    "kvq_create_in": (_i, [C.POINTER(_vp), _i, _i, _i, _i, _i, _i, C.c_uint64, _i, _vp, C.c_uint64]),
    "kvq_arena_usage": (_i, [_vp, _u64p, _u64p, _u64p]),
    "kvq_destroy": (_i, [_vp]),
    "kvq_set_controller": (_i, [_vp, _i, _vp, _vp, _vp, _vp, _vp, _vp]),
    "kvq_select_bits": (_i, [_vp, _vp, _i, _vp, _vp, _vp]),
    "kvq_append": (_i, [_vp, _i, _vp, _vp, _vp, _i, _vp]),
    "kvq_append_fused": (_i, [_vp, _i, _vp, _vp, _vp, _i, _vp, _vp]),
    "kvq_append_ragged": (_i, [_vp, _i, _vp, _vp, _vp, _vp, _i, _vp, _vp, _vp]),
    "kvq_seq_lens": (_i, [_vp, _i, _vp]),
    "kvq_decode_attn": (_i, [_vp, _i, _vp, _vp, _vp]),
    "kvq_decode_attn_var": (_i, [_vp, _i, _vp, _vp, _vp, _vp]),
    "kvq_token_features": (_i, [_vp, _i, _i, _i, _vp, _vp, C.c_uint64, C.c_uint32, _vp, _vp, _vp]),
    "kvq_attend_last": (_i, [_vp, _i, _vp, _vp, _i, _vp]),
    "kvq_decode_attn_static": (_i, [_vp, _i, _vp, _vp, _vp]),
    "kvq_decode_step": (_i, [_vp, _i, _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "kvq_decode_step_host": (_i, [_vp, _i, _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "kvq_reset": (_i, [_vp, _vp]),
    "kvq_seq_len": (_i, [_vp, _i, C.POINTER(_i)]),
    "kvq_set_splits": (_i, [_vp, _i]),
    "kvq_state_bytes": (_i, [_vp, C.POINTER(C.c_uint64)]),
    "kvq_save_state": (_i, [_vp, _vp, C.c_uint64]),
    "kvq_load_state": (_i, [_vp, _vp, C.c_uint64]),
    "kvq_set_append_chunk": (_i, [_vp, _i]),
    "kvq_export_range": (_i, [_vp, _i, _i, _i, _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "kvq_export_token": (_i, [_vp, _i, _i, _i, _vp, _vp, _vp, _vp, _vp, _vp]),
    "kvq_stats": (_i, [_vp, _i, _vp, _u64p, C.POINTER(C.c_double)]),
    "kvq_set_profiling": (_i, [_vp, _i]),
    "kvq_profile_read": (_i, [_vp, C.POINTER(C.c_double), C.POINTER(_i)]),
    "kvq_device_status": (_i, [_vp, C.POINTER(C.c_uint32)]),
    "kvq_recover": (_i, [_vp]),
    "kvq_device_bytes": (_i, [_vp, _u64p]),
    "kvq_launch_count": (_i, [_vp, _u64p]),
    "kvq_last_cuda_error": (_i, [_vp]),
    "kvq_strerror": (C.c_char_p, [_i]),
}

_lib: Optional[C.CDLL] = None


def lib() -> C.CDLL:
    """Load the CUDA library; raises if it is missing (build it with ``python -m paper_2604_04722_b200.build``)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                "libkvq.so is not built (%s); run `python -m paper_2604_04722_b200.build` -- "
                "there is no CPU fallback" % LIB_PATH)
        handle = C.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(handle, name)
            fn.restype = res
            fn.argtypes = args
        _lib = handle
    return _lib


class KvqError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__("%s: %s (%d)" % (where, lib().kvq_strerror(code).decode(), code))


def check(code: int, where: str) -> None:
    if code != KVQ_OK:
        raise KvqError(code, where)


def _ptr(t) -> Optional[int]:
    """Device or host address of a tensor / numpy array / int, or None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if hasattr(t, "data_ptr"):
        assert t.is_contiguous(), "tensors must be contiguous"
        return t.data_ptr()
    return t.ctypes.data          # numpy


def _stream(stream=None) -> int:
    if stream is not None:
        return int(stream)
    import torch
    return int(torch.cuda.current_stream().cuda_stream)


# ---- the C calls, same names, raising on error ---------------------------------------

def kvq_create(layers: int, q_heads: int, kv_heads: int, head_dim: int, max_ctx: int, batch: int) -> int:
    h = _vp()
    check(lib().kvq_create(C.byref(h), layers, q_heads, kv_heads, head_dim, max_ctx, batch), "kvq_create")
    return h.value


def kvq_create_arena(layers: int, q_heads: int, kv_heads: int, head_dim: int, max_ctx: int, batch: int,
                     arena_bytes: int) -> int:
    h = _vp()
    check(lib().kvq_create_arena(C.byref(h), layers, q_heads, kv_heads, head_dim, max_ctx, batch, arena_bytes),
          "kvq_create_arena")
    return h.value


def kvq_create_grouped(layers: int, q_heads: int, kv_heads: int, head_dim: int, max_ctx: int, batch: int,
                       arena_bytes: int, scale_groups: int) -> int:
    h = _vp()
    check(lib().kvq_create_grouped(C.byref(h), layers, q_heads, kv_heads, head_dim, max_ctx, batch, arena_bytes,
                                   scale_groups), "kvq_create_grouped")
    return h.value


def kvq_create_perchannel(layers: int, q_heads: int, kv_heads: int, head_dim: int, max_ctx: int, batch: int,
                          arena_bytes: int = 0) -> int:
    h = _vp()
    check(lib().kvq_create_perchannel(C.byref(h), layers, q_heads, kv_heads, head_dim, max_ctx, batch, arena_bytes),
          "kvq_create_perchannel")
    return h.value


def kvq_export_k_channels(ctx: int, layer: int, b: int, kv_head: int, bits: int, window: int):
    """Returns the window's {scale, zero-point} pairs as numpy u16 [64][2]."""
    import numpy as np
    out = np.zeros((64, 2), np.uint16)
    check(lib().kvq_export_k_channels(ctx, layer, b, kv_head, bits, window, out.ctypes.data), "kvq_export_k_channels")
    return out


def kvq_workspace_bytes(layers: int, q_heads: int, kv_heads: int, head_dim: int, max_ctx: int, batch: int,
                        arena_bytes: int = 0, scale_groups: int = 1) -> int:
    n = C.c_uint64()
    check(lib().kvq_workspace_bytes(layers, q_heads, kv_heads, head_dim, max_ctx, batch, arena_bytes, scale_groups,
                                    C.byref(n)), "kvq_workspace_bytes")
    return n.value


def kvq_create_in(layers: int, q_heads: int, kv_heads: int, head_dim: int, max_ctx: int, batch: int, arena_bytes: int,
                  scale_groups: int, workspace, workspace_bytes: int) -> int:
    h = _vp()
    check(lib().kvq_create_in(C.byref(h), layers, q_heads, kv_heads, head_dim, max_ctx, batch, arena_bytes, scale_groups,
                              _ptr(workspace), workspace_bytes), "kvq_create_in")
    return h.value


def kvq_arena_usage(ctx: int):
    """Returns (blocks_in_use, blocks_total, block_bytes)."""
    a, b, c = C.c_uint64(), C.c_uint64(), C.c_uint64()
    check(lib().kvq_arena_usage(ctx, C.byref(a), C.byref(b), C.byref(c)), "kvq_arena_usage")
    return a.value, b.value, c.value


def kvq_destroy(ctx: int) -> None:
    check(lib().kvq_destroy(ctx), "kvq_destroy")


def kvq_set_controller(ctx: int, hidden: int, W1, b1, W2, b2, W3, b3) -> None:
    import numpy as np
    arrs = [np.ascontiguousarray(a, dtype=np.float32) for a in (W1, b1, W2, b2, W3, b3)]
    assert arrs[0].shape == (hidden, 4) and arrs[2].shape == (hidden, hidden) and arrs[4].shape == (4, hidden)
    check(lib().kvq_set_controller(ctx, hidden, *[a.ctypes.data for a in arrs]), "kvq_set_controller")


def kvq_select_bits(ctx: int, feats, n: int, bits, logits=None, stream=None) -> None:
    check(lib().kvq_select_bits(ctx, _ptr(feats), n, _ptr(bits), _ptr(logits), _stream(stream)), "kvq_select_bits")


def kvq_append(ctx: int, layer: int, K, V, bits, n_new: int, stream=None) -> None:
    check(lib().kvq_append(ctx, layer, _ptr(K), _ptr(V), _ptr(bits), n_new, _stream(stream)), "kvq_append")


def kvq_append_fused(ctx: int, layer: int, K, V, feats, n_new: int, bits_out=None, stream=None) -> None:
    check(lib().kvq_append_fused(ctx, layer, _ptr(K), _ptr(V), _ptr(feats), n_new, _ptr(bits_out), _stream(stream)),
          "kvq_append_fused")


def kvq_append_ragged(ctx: int, layer: int, K, V, bits, feats, n_max: int, lens, bits_out=None, stream=None) -> None:
    import numpy as np
    lens = np.ascontiguousarray(lens, dtype=np.int32)
    check(lib().kvq_append_ragged(ctx, layer, _ptr(K), _ptr(V), _ptr(bits), _ptr(feats), n_max, lens.ctypes.data,
                                  _ptr(bits_out), _stream(stream)), "kvq_append_ragged")


def kvq_seq_lens(ctx: int, layer: int, batch: int):
    import numpy as np
    out = np.zeros(batch, np.int32)
    check(lib().kvq_seq_lens(ctx, layer, out.ctypes.data), "kvq_seq_lens")
    return out


def kvq_decode_attn(ctx: int, layer: int, Q, O, stream=None) -> None:
    check(lib().kvq_decode_attn(ctx, layer, _ptr(Q), _ptr(O), _stream(stream)), "kvq_decode_attn")


def kvq_decode_attn_var(ctx: int, layer: int, Q, O, var_out, stream=None) -> None:
    check(lib().kvq_decode_attn_var(ctx, layer, _ptr(Q), _ptr(O), _ptr(var_out), _stream(stream)), "kvq_decode_attn_var")


def kvq_token_features(logits, logits_are_fp32: bool, n: int, vocab: int, token_ids, counts, total_count: int,
                       observed_tokens: int, attn_var, feats, stream=None) -> None:
    check(lib().kvq_token_features(_ptr(logits), int(bool(logits_are_fp32)), n, vocab, _ptr(token_ids), _ptr(counts),
                                   total_count, observed_tokens, _ptr(attn_var), _ptr(feats), _stream(stream)),
          "kvq_token_features")


def kvq_attend_last(ctx: int, layer: int, Q, O, n_queries: int, stream=None) -> None:
    check(lib().kvq_attend_last(ctx, layer, _ptr(Q), _ptr(O), n_queries, _stream(stream)), "kvq_attend_last")


def kvq_decode_attn_static(ctx: int, layer: int, Q, O, stream=None) -> None:
    """kvq_decode_attn with the split partials in the library's fixed device array: allocates nothing."""
    check(lib().kvq_decode_attn_static(ctx, layer, _ptr(Q), _ptr(O), _stream(stream)), "kvq_decode_attn_static")


def kvq_decode_step(ctx: int, layer: int, feats, K, V, Q, O, bits_out=None, stream=None) -> None:
    """One decode step on device buffers: kvq_append_fused of one token per sequence, then kvq_decode_attn."""
    check(lib().kvq_decode_step(ctx, layer, _ptr(feats), _ptr(K), _ptr(V), _ptr(Q), _ptr(O), _ptr(bits_out),
                                _stream(stream)), "kvq_decode_step")


def kvq_decode_step_host(ctx: int, layer: int, feats, K, V, Q, O, bits_out=None, stream=None) -> None:
    check(lib().kvq_decode_step_host(ctx, layer, _ptr(feats), _ptr(K), _ptr(V), _ptr(Q), _ptr(O), _ptr(bits_out),
                                     _stream(stream)), "kvq_decode_step_host")


def kvq_reset(ctx: int, stream=None) -> None:
    check(lib().kvq_reset(ctx, _stream(stream)), "kvq_reset")


def kvq_seq_len(ctx: int, layer: int) -> int:
    n = _i()
    check(lib().kvq_seq_len(ctx, layer, C.byref(n)), "kvq_seq_len")
    return n.value


def kvq_state_bytes(ctx: int) -> int:
    n = C.c_uint64()
    check(lib().kvq_state_bytes(ctx, C.byref(n)), "kvq_state_bytes")
    return n.value


def kvq_save_state(ctx: int):
    """Returns the snapshot as a numpy uint8 array."""
    import numpy as np
    blob = np.empty(kvq_state_bytes(ctx), np.uint8)
    check(lib().kvq_save_state(ctx, blob.ctypes.data, blob.size), "kvq_save_state")
    return blob


def kvq_load_state(ctx: int, blob) -> None:
    check(lib().kvq_load_state(ctx, blob.ctypes.data, blob.size), "kvq_load_state")


def kvq_set_append_chunk(ctx: int, chunk_tokens: int) -> None:
    check(lib().kvq_set_append_chunk(ctx, chunk_tokens), "kvq_set_append_chunk")


def kvq_set_splits(ctx: int, splits: int) -> None:
    check(lib().kvq_set_splits(ctx, splits), "kvq_set_splits")


def kvq_export_range(ctx: int, layer: int, pos0: int, n: int, bits=None, pool_slot=None, k_codes=None,
                     v_codes=None, k_meta=None, v_meta=None, stream=None) -> None:
    check(lib().kvq_export_range(ctx, layer, pos0, n, _ptr(bits), _ptr(pool_slot), _ptr(k_codes), _ptr(v_codes),
                                 _ptr(k_meta), _ptr(v_meta), _stream(stream)), "kvq_export_range")


def kvq_export_token(ctx: int, layer: int, b: int, pos: int, kv_heads: int, scale_groups: int = 1):
    """Returns (bits, pool_slot, k_codes [H][128] u8, v_codes, k_meta [H][2 * scale_groups] u16, v_meta) as numpy."""
    import numpy as np
    bits = np.zeros(1, np.uint8)
    ps = np.zeros(1, np.uint32)
    kc = np.zeros((kv_heads, KVQ_EXPORT_ROW_BYTES), np.uint8)
    vc = np.zeros_like(kc)
    km = np.zeros((kv_heads, 2 * scale_groups), np.uint16)
    vm = np.zeros_like(km)
    check(lib().kvq_export_token(ctx, layer, b, pos, _ptr(bits), _ptr(ps), _ptr(kc), _ptr(vc), _ptr(km), _ptr(vm)),
          "kvq_export_token")
    return int(bits[0]), int(ps[0]), kc, vc, km, vm


def kvq_stats(ctx: int, layer: int, batch: int):
    """Returns (counts [batch][4] numpy u32, resident_bytes, expected_bits)."""
    import numpy as np
    counts = np.zeros((batch, 4), np.uint32)
    rb = C.c_uint64()
    eb = C.c_double()
    check(lib().kvq_stats(ctx, layer, _ptr(counts), C.byref(rb), C.byref(eb)), "kvq_stats")
    return counts, rb.value, eb.value


def kvq_set_profiling(ctx: int, on: bool) -> None:
    check(lib().kvq_set_profiling(ctx, int(bool(on))), "kvq_set_profiling")


def kvq_profile_read(ctx: int):
    """Returns (attn_ms_total, calls) of the decode calls recorded since the last read."""
    a, n = C.c_double(), _i()
    check(lib().kvq_profile_read(ctx, C.byref(a), C.byref(n)), "kvq_profile_read")
    return a.value, n.value


def kvq_device_status(ctx: int) -> int:
    """Device flag word (cleared on read); does not raise on a set flag."""
    f = C.c_uint32()
    rc = lib().kvq_device_status(ctx, C.byref(f))
    if rc not in (KVQ_OK, KVQ_ERR_DEVICE_FLAG):
        raise KvqError(rc, "kvq_device_status")
    return f.value


def kvq_recover(ctx: int) -> None:
    check(lib().kvq_recover(ctx), "kvq_recover")


def kvq_device_bytes(ctx: int) -> int:
    v = C.c_uint64()
    check(lib().kvq_device_bytes(ctx, C.byref(v)), "kvq_device_bytes")
    return v.value


def kvq_launch_count(ctx: int) -> int:
    v = C.c_uint64()
    check(lib().kvq_launch_count(ctx, C.byref(v)), "kvq_launch_count")
    return v.value


def kvq_last_cuda_error(ctx: int) -> int:
    return lib().kvq_last_cuda_error(ctx)


def kvq_strerror(code: int) -> str:
    return lib().kvq_strerror(code).decode()
