"""Thin ctypes binding of the C ABI in include/gva.h: argument marshalling only.

Every function mirrors the C entry point of the same name.  Device buffers are torch CUDA
tensors (torch is used for device memory and streams, nothing else); each call enqueues on the
current torch stream.  There is no CPU fallback: if libgva.so is missing or fails to load, the
first call raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("GVA_LIBRARY", os.path.join(_HERE, "libgva.so"))   # override: load another build of the library

GVA_OK = 0
GVA_ERR_INVALID_ARG, GVA_ERR_UNSUPPORTED, GVA_ERR_WORKSPACE, GVA_ERR_CUDA = 1, 2, 3, 4
GVA_ERR_BAD_PAGE, GVA_ERR_SEQ_LEN, GVA_ERR_TIMEOUT, GVA_ERR_STATIC_LIMIT = 5, 6, 7, 8
GVA_STATIC_SCRATCH_BYTES = 16 << 20
GVA_F32, GVA_BF16, GVA_E4M3 = 0, 1, 2
GVA_KERNEL_AUTO, GVA_KERNEL_FMA, GVA_KERNEL_MMA = 0, 1, 2

EXPORTS = ["gva_create", "gva_destroy", "gva_decode_workspace_bytes", "gva_absorb_query", "gva_append_cache",
           "gva_decode", "gva_decode_static", "gqa_decode", "gva_decode_step", "gva_step_scratch_bytes", "gva_decode_step_host", "gva_input_width", "gva_pack_input_weights", "gva_pack_bf16",
           "gva_project_in", "gva_project_out", "gva_layer_step", "gva_last_num_splits", "gva_last_kernel", "gva_last_tile_tokens",
           "gva_status_string", "gva_append_chunk", "gva_prefill", "gva_decode_multi_workspace_bytes", "gva_decode_multi", "gva_decode_tokens_workspace_bytes", "gva_decode_tokens", "gva_decode_tokens_ragged"]


class GvaConfig(ctypes.Structure):
    _fields_ = [("H", ctypes.c_int32), ("G", ctypes.c_int32), ("d_v", ctypes.c_int32), ("d_c", ctypes.c_int32),
                ("d_r", ctypes.c_int32), ("page_size", ctypes.c_int32), ("cache_dtype", ctypes.c_int32),
                ("kernel", ctypes.c_int32), ("rope_base", ctypes.c_double), ("softmax_scale", ctypes.c_float),
                ("reserved", ctypes.c_int32)]


class GvaCache(ctypes.Structure):
    _fields_ = [("v_pool", ctypes.c_void_p), ("kr_pool", ctypes.c_void_p), ("block_table", ctypes.c_void_p),
                ("num_pages", ctypes.c_int32), ("max_pages_per_seq", ctypes.c_int32)]


class GqaCache(ctypes.Structure):
    _fields_ = [("k_pool", ctypes.c_void_p), ("v_pool", ctypes.c_void_p), ("block_table", ctypes.c_void_p),
                ("num_pages", ctypes.c_int32), ("max_pages_per_seq", ctypes.c_int32)]


class GvaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (gva_status {status})")


_lib: Optional[ctypes.CDLL] = None


def load() -> ctypes.CDLL:
    """dlopen libgva.so and declare the prototypes.  Raises if the library has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} not found: build it with `python -m paper_2609_13285_b200.build` "
                           "(there is no CPU fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, ip, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
    lib.gva_create.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(GvaConfig), ip]
    lib.gva_destroy.argtypes = [vp]
    lib.gva_decode_workspace_bytes.argtypes = [vp, ip, ip, ip]
    lib.gva_decode_workspace_bytes.restype = sz
    lib.gva_decode_step.argtypes = [vp, ctypes.POINTER(GvaCache)] + [vp] * 11 + [sz, ip, ip, ip, vp, vp]
    lib.gva_step_scratch_bytes.argtypes = [vp, ip, ip, ip]
    lib.gva_step_scratch_bytes.restype = sz
    lib.gva_decode_step_host.argtypes = [vp, ctypes.POINTER(GvaCache), vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, ip, ip,
                                         ip, vp, vp]
    lib.gva_absorb_query.argtypes = [vp, vp, vp, vp, vp, vp, ip, vp]
    lib.gva_append_cache.argtypes = [vp, ctypes.POINTER(GvaCache), vp, vp, vp, ip, vp, vp]
    lib.gva_decode.argtypes = [vp, ctypes.POINTER(GvaCache), vp, vp, vp, vp, vp, sz, ip, ip, ip, vp, vp]
    lib.gva_append_chunk.argtypes = [vp, ctypes.POINTER(GvaCache), vp, vp, vp, vp, ip, ip, vp, vp]
    lib.gva_prefill.argtypes = [vp, ctypes.POINTER(GvaCache), vp, vp, vp, vp, vp, ip, ip, vp, vp]
    lib.gva_decode_multi_workspace_bytes.argtypes = [vp, ip, ip, ip, ip, ip]
    lib.gva_decode_tokens_workspace_bytes.argtypes = [vp, ip, ip, ip, ip]
    lib.gva_decode_tokens_workspace_bytes.restype = sz
    lib.gva_decode_tokens.argtypes = [vp, ctypes.POINTER(GvaCache), vp, vp, vp, vp, vp, sz, ip, ip, ip, ip, vp, vp]
    lib.gva_decode_tokens_ragged.argtypes = [vp, ctypes.POINTER(GvaCache), vp, vp, vp, vp, vp, vp, sz, ip, ip, ip, ip, vp, vp]
    lib.gva_decode_multi_workspace_bytes.restype = sz
    lib.gva_decode_multi.argtypes = [vp, ctypes.POINTER(GvaCache), vp, vp, vp, vp, vp, vp, sz, ip, ip, ip, ip, ip, vp, vp]
    lib.gva_decode_static.argtypes = [vp, ctypes.POINTER(GvaCache), vp, vp, vp, vp, ip, ip, ip, vp, vp]
    lib.gqa_decode.argtypes = [vp, ctypes.POINTER(GqaCache), vp, vp, vp, vp, vp, sz, ip, ip, ip, vp, vp]
    lib.gva_input_width.argtypes = [vp]
    lib.gva_pack_input_weights.argtypes = [vp, vp, vp, vp, vp, vp, ip, vp]
    lib.gva_pack_bf16.argtypes = [vp, vp, sz]
    lib.gva_project_in.argtypes = [vp, ctypes.POINTER(GvaCache), vp, vp, ip, vp, vp, ip, vp, vp]
    lib.gva_project_out.argtypes = [vp, vp, vp, ip, vp, ip, vp]
    lib.gva_layer_step.argtypes = [vp, ctypes.POINTER(GvaCache), vp, vp, vp, ip, vp, vp, vp, vp, vp, vp, sz, ip, ip, ip,
                                   vp, vp]
    for name in ("gva_last_num_splits", "gva_last_kernel", "gva_last_tile_tokens"):
        getattr(lib, name).argtypes = [vp]
    lib.gva_status_string.argtypes = [ip]
    lib.gva_status_string.restype = ctypes.c_char_p
    for name in EXPORTS:
        if name not in ("gva_decode_workspace_bytes", "gva_step_scratch_bytes", "gva_status_string", "gva_pack_bf16"):
            getattr(lib, name).restype = ip
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load().gva_status_string(int(status)).decode()


def _ptr(t) -> Optional[int]:
    return None if t is None else int(t.data_ptr())


def _stream() -> int:
    import torch
    return int(torch.cuda.current_stream().cuda_stream)


def _check(rc: int, where: str) -> None:
    if rc != GVA_OK:
        raise GvaError(rc, where)


def gva_create(*, H: int, G: int, d_v: int, d_c: int, d_r: int, page_size: int, cache_dtype: int = GVA_BF16,
               kernel: int = GVA_KERNEL_AUTO, rope_base: float = 10000.0, softmax_scale: float = 0.0,
               device: int = 0) -> int:
    cfg = GvaConfig(H, G, d_v, d_c, d_r, page_size, cache_dtype, kernel, rope_base, softmax_scale, 0)
    h = ctypes.c_void_p()
    _check(load().gva_create(ctypes.byref(h), ctypes.byref(cfg), int(device)), "gva_create")
    return h.value


def gva_destroy(handle: int) -> None:
    _check(load().gva_destroy(handle), "gva_destroy")


def gva_decode_workspace_bytes(handle: int, B: int, max_seq_len: int, num_splits: int = 0) -> int:
    return int(load().gva_decode_workspace_bytes(handle, int(B), int(max_seq_len), int(num_splits)))


def gva_absorb_query(handle: int, q_c, q_r, M, q_pos, q_abs, B: int, check: bool = True) -> int:
    rc = load().gva_absorb_query(handle, _ptr(q_c), _ptr(q_r), _ptr(M), _ptr(q_pos), _ptr(q_abs), int(B), _stream())
    if check:
        _check(rc, "gva_absorb_query")
    return rc


def make_cache(v_pool, kr_pool, block_table, num_pages: int, max_pages_per_seq: int) -> GvaCache:
    return GvaCache(_ptr(v_pool), _ptr(kr_pool), _ptr(block_table), int(num_pages), int(max_pages_per_seq))


def make_gqa_cache(k_pool, v_pool, block_table, num_pages: int, max_pages_per_seq: int) -> GqaCache:
    return GqaCache(_ptr(k_pool), _ptr(v_pool), _ptr(block_table), int(num_pages), int(max_pages_per_seq))


def gva_append_cache(handle: int, cache: GvaCache, v_new, kr_new, pos, B: int, dev_status=None,
                     check: bool = True) -> int:
    rc = load().gva_append_cache(handle, ctypes.byref(cache), _ptr(v_new), _ptr(kr_new), _ptr(pos), int(B),
                                 _ptr(dev_status), _stream())
    if check:
        _check(rc, "gva_append_cache")
    return rc


def gva_append_chunk(handle: int, cache: GvaCache, v_new, kr_new, cu_q, ctx_lens, B: int, n_q: int, dev_status=None,
                     check: bool = True) -> int:
    rc = load().gva_append_chunk(handle, ctypes.byref(cache), _ptr(v_new), _ptr(kr_new), _ptr(cu_q), _ptr(ctx_lens), int(B),
                                 int(n_q), _ptr(dev_status), _stream())
    if check:
        _check(rc, "gva_append_chunk")
    return rc


def gva_prefill(handle: int, cache: GvaCache, q_abs, cu_q, ctx_lens, out, lse, B: int, max_q_len: int, dev_status=None,
                check: bool = True) -> int:
    rc = load().gva_prefill(handle, ctypes.byref(cache), _ptr(q_abs), _ptr(cu_q), _ptr(ctx_lens), _ptr(out), _ptr(lse), int(B),
                            int(max_q_len), _ptr(dev_status), _stream())
    if check:
        _check(rc, "gva_prefill")
    return rc


def gva_decode_multi_workspace_bytes(handle: int, B: int, n_q: int, max_q_len: int, max_seq_len: int, num_splits: int = 0) -> int:
    return int(load().gva_decode_multi_workspace_bytes(handle, int(B), int(n_q), int(max_q_len), int(max_seq_len), int(num_splits)))


def gva_decode_multi(handle: int, cache: GvaCache, q_abs, cu_q, ctx_lens, out, lse, workspace, B: int, n_q: int, max_q_len: int,
                     max_seq_len: int, num_splits: int = 0, dev_status=None, check: bool = True) -> int:
    rc = load().gva_decode_multi(handle, ctypes.byref(cache), _ptr(q_abs), _ptr(cu_q), _ptr(ctx_lens), _ptr(out), _ptr(lse),
                                 _ptr(workspace), 0 if workspace is None else int(workspace.numel() * workspace.element_size()),
                                 int(B), int(n_q), int(max_q_len), int(max_seq_len), int(num_splits), _ptr(dev_status), _stream())
    if check:
        _check(rc, "gva_decode_multi")
    return rc


def gva_decode_tokens_workspace_bytes(handle: int, B: int, q_len: int, max_seq_len: int, num_splits: int = 0) -> int:
    return int(load().gva_decode_tokens_workspace_bytes(handle, int(B), int(q_len), int(max_seq_len), int(num_splits)))


def gva_decode_tokens(handle: int, cache: GvaCache, q_abs, seq_lens, out, lse, workspace, B: int, q_len: int, max_seq_len: int,
                      num_splits: int = 0, dev_status=None, check: bool = True) -> int:
    rc = load().gva_decode_tokens(handle, ctypes.byref(cache), _ptr(q_abs), _ptr(seq_lens), _ptr(out), _ptr(lse), _ptr(workspace),
                                  0 if workspace is None else int(workspace.numel() * workspace.element_size()), int(B),
                                  int(q_len), int(max_seq_len), int(num_splits), _ptr(dev_status), _stream())
    if check:
        _check(rc, "gva_decode_tokens")
    return rc


def gva_decode_tokens_ragged(handle: int, cache: GvaCache, q_abs, cu_q, seq_lens, out, lse, workspace, B: int, max_q_len: int,
                             max_seq_len: int, num_splits: int = 0, dev_status=None, check: bool = True) -> int:
    rc = load().gva_decode_tokens_ragged(handle, ctypes.byref(cache), _ptr(q_abs), _ptr(cu_q), _ptr(seq_lens), _ptr(out), _ptr(lse),
                                         _ptr(workspace),
                                         0 if workspace is None else int(workspace.numel() * workspace.element_size()), int(B),
                                         int(max_q_len), int(max_seq_len), int(num_splits), _ptr(dev_status), _stream())
    if check:
        _check(rc, "gva_decode_tokens_ragged")
    return rc


def gva_decode(handle: int, cache: GvaCache, q_abs, seq_lens, out, lse, workspace, B: int, max_seq_len: int,
               num_splits: int = 0, dev_status=None, workspace_bytes: Optional[int] = None, check: bool = True) -> int:
    wb = (workspace.numel() * workspace.element_size() if workspace is not None else 0) \
        if workspace_bytes is None else int(workspace_bytes)
    rc = load().gva_decode(handle, ctypes.byref(cache), _ptr(q_abs), _ptr(seq_lens), _ptr(out), _ptr(lse),
                           _ptr(workspace), wb, int(B), int(max_seq_len), int(num_splits), _ptr(dev_status), _stream())
    if check:
        _check(rc, "gva_decode")
    return rc


def gva_decode_static(handle: int, cache: GvaCache, q_abs, seq_lens, out, lse, B: int, max_seq_len: int,
                      num_splits: int = 0, dev_status=None, check: bool = True) -> int:
    """gva_decode without a caller workspace: the partial results use the library's built-in scratch
    (GVA_STATIC_SCRATCH_BYTES per GPU).  For callers that must not allocate device memory; calls on
    one GPU must be stream-ordered, and the first call on a device should come before any stream capture."""
    rc = load().gva_decode_static(handle, ctypes.byref(cache), _ptr(q_abs), _ptr(seq_lens), _ptr(out), _ptr(lse),
                                  int(B), int(max_seq_len), int(num_splits), _ptr(dev_status), _stream())
    if check:
        _check(rc, "gva_decode_static")
    return rc


def gqa_decode(handle: int, cache: GqaCache, q, seq_lens, out, lse, workspace, B: int, max_seq_len: int,
               num_splits: int = 0, dev_status=None, workspace_bytes: Optional[int] = None, check: bool = True) -> int:
    wb = (workspace.numel() * workspace.element_size() if workspace is not None else 0) \
        if workspace_bytes is None else int(workspace_bytes)
    rc = load().gqa_decode(handle, ctypes.byref(cache), _ptr(q), _ptr(seq_lens), _ptr(out), _ptr(lse),
                           _ptr(workspace), wb, int(B), int(max_seq_len), int(num_splits), _ptr(dev_status), _stream())
    if check:
        _check(rc, "gqa_decode")
    return rc


def gva_decode_step(handle: int, cache: GvaCache, M, q_c, q_r, v_new, kr_new, pos, seq_lens, q_abs, out, lse, workspace,
                    B: int, max_seq_len: int, num_splits: int = 0, dev_status=None, check: bool = True) -> int:
    rc = load().gva_decode_step(handle, ctypes.byref(cache), _ptr(M), _ptr(q_c), _ptr(q_r), _ptr(v_new), _ptr(kr_new),
                                _ptr(pos), _ptr(seq_lens), _ptr(q_abs), _ptr(out), _ptr(lse), _ptr(workspace),
                                workspace.numel() * workspace.element_size(), int(B), int(max_seq_len), int(num_splits),
                                _ptr(dev_status), _stream())
    if check:
        _check(rc, "gva_decode_step")
    return rc


def gva_step_scratch_bytes(handle: int, B: int, max_seq_len: int, num_splits: int = 0) -> int:
    return int(load().gva_step_scratch_bytes(handle, int(B), int(max_seq_len), int(num_splits)))


def gva_decode_step_host(handle: int, cache: GvaCache, M, q_c_host, q_r_host, v_new_host, kr_new_host, pos_host,
                         seq_lens_host, out_host, scratch, B: int, max_seq_len: int, num_splits: int = 0,
                         dev_status=None, check: bool = True) -> int:
    """Host tensors are CPU torch tensors (pinned for asynchronous copies); M, scratch, dev_status are CUDA tensors."""
    rc = load().gva_decode_step_host(handle, ctypes.byref(cache), _ptr(M), _ptr(q_c_host), _ptr(q_r_host),
                                     _ptr(v_new_host), _ptr(kr_new_host), _ptr(pos_host), _ptr(seq_lens_host),
                                     _ptr(out_host), _ptr(scratch), scratch.numel() * scratch.element_size(), int(B),
                                     int(max_seq_len), int(num_splits), _ptr(dev_status), _stream())
    if check:
        _check(rc, "gva_decode_step_host")
    return rc


def prepare_call(name: str, *args):
    """Any entry point with its arguments marshalled once: `args` as the C signature lists them after the handle's
    position included (tensors, None, a GvaCache / GqaCache, integers), the trailing stream taken from torch's current
    stream when left out.  Returns a callable that enqueues the call and returns its status (GvaError on a non-zero one).
    The arguments are kept alive by the callable; it is for loops that reuse their buffers."""
    fn = getattr(load(), name)
    types = fn.argtypes
    args = list(args)
    if len(args) == len(types) - 1:
        args.append(_stream())
    if len(args) != len(types):
        raise TypeError(f"{name} takes {len(types)} arguments, {len(args)} given")
    conv = []
    for a, t in zip(args, types):
        if isinstance(a, ctypes.Structure):
            conv.append(ctypes.byref(a))
        elif t is ctypes.c_void_p:
            conv.append(ctypes.c_void_p(a if isinstance(a, int) else _ptr(a)))
        else:
            conv.append(t(int(a)))
    conv = tuple(conv)

    def call(_keep=tuple(args)) -> int:
        rc = fn(*conv)
        if rc != GVA_OK:
            raise GvaError(rc, name)
        return rc

    return call


def prepare_decode_step_host(handle: int, cache: GvaCache, M, q_c_host, q_r_host, v_new_host, kr_new_host, pos_host,
                             seq_lens_host, out_host, scratch, B: int, max_seq_len: int, num_splits: int = 0,
                             dev_status=None):
    """gva_decode_step_host with its arguments marshalled once: returns a callable that enqueues one step on the stream
    that was current here and returns the status.  For a serving loop that reuses its buffers: per call the interpreter
    then makes one foreign call instead of a dozen pointer look-ups.  The tensors are kept alive by the callable."""
    fn = load().gva_decode_step_host
    keep = (cache, M, q_c_host, q_r_host, v_new_host, kr_new_host, pos_host, seq_lens_host, out_host, scratch, dev_status)
    args = (ctypes.c_void_p(handle), ctypes.byref(cache), ctypes.c_void_p(_ptr(M)), ctypes.c_void_p(_ptr(q_c_host)),
            ctypes.c_void_p(_ptr(q_r_host)), ctypes.c_void_p(_ptr(v_new_host)), ctypes.c_void_p(_ptr(kr_new_host)),
            ctypes.c_void_p(_ptr(pos_host)), ctypes.c_void_p(_ptr(seq_lens_host)), ctypes.c_void_p(_ptr(out_host)),
            ctypes.c_void_p(_ptr(scratch)), ctypes.c_size_t(scratch.numel() * scratch.element_size()), ctypes.c_int(int(B)),
            ctypes.c_int(int(max_seq_len)), ctypes.c_int(int(num_splits)), ctypes.c_void_p(_ptr(dev_status)),
            ctypes.c_void_p(_stream()))

    def call(_keep=keep) -> int:
        rc = fn(*args)
        if rc != GVA_OK:
            raise GvaError(rc, "gva_decode_step_host")
        return rc

    return call


def gva_input_width(handle: int) -> int:
    return int(load().gva_input_width(handle))


def _np_ptr(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def gva_pack_input_weights(handle: int, W_q_nope, W_q_rope, W_v, W_r, M, d_model: int):
    """Host-side offline packing (numpy float32 in, numpy uint16 bf16 bit patterns [d_model, N_in] out)."""
    import numpy as np
    arrs = [np.ascontiguousarray(a, dtype=np.float32) for a in (W_q_nope, W_q_rope, W_v, W_r, M)]
    out = np.empty((d_model, gva_input_width(handle)), dtype=np.uint16)
    _check(load().gva_pack_input_weights(handle, *[_np_ptr(a) for a in arrs], int(d_model), _np_ptr(out)),
           "gva_pack_input_weights")
    return out


def gva_pack_bf16(src):
    import numpy as np
    src = np.ascontiguousarray(src, dtype=np.float32)
    out = np.empty(src.shape, dtype=np.uint16)
    _check(load().gva_pack_bf16(_np_ptr(src), _np_ptr(out), src.size), "gva_pack_bf16")
    return out


def gva_project_in(handle: int, cache: GvaCache, x, W_in, d_model: int, pos, q_abs, B: int, dev_status=None,
                   check: bool = True) -> int:
    rc = load().gva_project_in(handle, ctypes.byref(cache), _ptr(x), _ptr(W_in), int(d_model), _ptr(pos), _ptr(q_abs),
                               int(B), _ptr(dev_status), _stream())
    if check:
        _check(rc, "gva_project_in")
    return rc


def gva_project_out(handle: int, attn, W_o, d_model: int, y, B: int, check: bool = True) -> int:
    rc = load().gva_project_out(handle, _ptr(attn), _ptr(W_o), int(d_model), _ptr(y), int(B), _stream())
    if check:
        _check(rc, "gva_project_out")
    return rc


def gva_layer_step(handle: int, cache: GvaCache, x, W_in, W_o, d_model: int, pos, seq_lens, q_abs, attn, y, workspace,
                   B: int, max_seq_len: int, num_splits: int = 0, dev_status=None, check: bool = True) -> int:
    rc = load().gva_layer_step(handle, ctypes.byref(cache), _ptr(x), _ptr(W_in), _ptr(W_o), int(d_model), _ptr(pos),
                               _ptr(seq_lens), _ptr(q_abs), _ptr(attn), _ptr(y), _ptr(workspace),
                               workspace.numel() * workspace.element_size(), int(B), int(max_seq_len), int(num_splits),
                               _ptr(dev_status), _stream())
    if check:
        _check(rc, "gva_layer_step")
    return rc


def gva_last_num_splits(handle: int) -> int:
    return int(load().gva_last_num_splits(handle))


def gva_last_kernel(handle: int) -> int:
    return int(load().gva_last_kernel(handle))


def gva_last_tile_tokens(handle: int) -> int:
    return int(load().gva_last_tile_tokens(handle))
