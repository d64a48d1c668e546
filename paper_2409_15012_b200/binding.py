"""ctypes binding of libmixattn.so: the same calls as include/mixattn.h.

Argument marshalling only.  Device tensors are torch tensors (torch supplies
device memory and streams); host arrays are numpy int32 arrays or sequences.
There is no fallback: if the library is missing the import fails, and a call
on a host-only context that needs the GPU returns MIXATTN_ERR_CUDA.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np

FULL, SLIDING = 0, 1
F32, BF16 = 0, 1
KV_NATIVE, KV_FP8_E4M3 = 0, 1

OK = 0
ERR_INVALID_ARG = -1
ERR_INVALID_LAYOUT = -2
ERR_NOT_OWNER = -3
ERR_OUT_OF_PAGES = -4
ERR_EMPTY_CONTEXT = -5
ERR_BAD_SEQ = -6
ERR_UNSUPPORTED = -7
ERR_CUDA = -8
ERR_TOO_LARGE = -9

K_APPEND, K_DECODE_FULL, K_DECODE_SLIDING, K_COMBINE, K_PREFILL_FULL, K_PREFILL_SLIDING, K_GATHER = range(7)

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libmixattn.so")


class LayerDesc(C.Structure):
    _fields_ = [("kind", C.c_int32), ("window", C.c_int32), ("kv_owner_layer", C.c_int32)]


class Config(C.Structure):
    _fields_ = [
        ("n_layers", C.c_int32),
        ("layers", C.POINTER(LayerDesc)),
        ("n_q_heads", C.c_int32),
        ("n_kv_heads", C.c_int32),
        ("head_dim", C.c_int32),
        ("dtype", C.c_int32),
        ("max_seqs", C.c_int32),
        ("page_size", C.c_int32),
        ("n_pages", C.c_int32),
        ("max_seq_len", C.c_int32),
        ("free_order", C.POINTER(C.c_int32)),
        ("softmax_scale", C.c_float),
        ("device", C.c_int32),
        ("arena", C.c_void_p),
        ("arena_bytes", C.c_size_t),
        ("chunk_scratch_tokens", C.c_int32),
        ("kv_format", C.c_int32),
    ]


def _load() -> C.CDLL:
    if not os.path.exists(_LIB_PATH):
        raise ImportError(
            f"{_LIB_PATH} is missing: build it with `python -m paper_2409_15012_b200.build` "
            "(there is no fallback implementation)")
    lib = C.CDLL(_LIB_PATH)
    i32, p32, vp = C.c_int32, C.POINTER(C.c_int32), C.c_void_p
    cfgp = C.POINTER(Config)
    sig = {
        "mixattn_arena_bytes": [cfgp, C.POINTER(C.c_size_t)],
        "mixattn_cache_bytes": [cfgp, C.POINTER(C.c_size_t)],
        "mixattn_create": [cfgp, C.POINTER(vp)],
        "mixattn_destroy": [vp],
        "mixattn_seq_reset": [vp, i32],
        "mixattn_append_kv": [vp, i32, i32, p32, p32, vp, vp, vp],
        "mixattn_append_kv_rope": [vp, i32, i32, p32, p32, vp, vp, C.c_float, vp],
        "mixattn_decode": [vp, i32, i32, p32, vp, vp, vp],
        "mixattn_decode_static_scratch": [vp, i32, i32, p32, vp, vp, vp],
        "mixattn_decode_layers": [vp, i32, i32, i32, p32, C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), vp, p32],
        "mixattn_attend_chunk": [vp, i32, i32, p32, p32, vp, vp, vp, vp, vp],
        "mixattn_prefill": [vp, i32, i32, p32, p32, vp, vp, vp, vp, vp],
        "mixattn_get_len": [vp, i32, i32, p32],
        "mixattn_get_block_table": [vp, i32, p32, i32, p32],
        "mixattn_get_n_free_pages": [vp, p32],
        "mixattn_get_ring_state": [vp, i32, i32, p32, p32],
        "mixattn_locate": [vp, i32, i32, i32, p32, p32],
        "mixattn_debug_read_kv": [vp, i32, i32, i32, vp, vp],
        "mixattn_debug_read_kv_fp8": [vp, i32, i32, i32, vp, vp, vp, vp],
        "mixattn_get_device_status": [vp, p32],
        "mixattn_set_split_tokens": [vp, i32],
        "mixattn_set_chunk_gather_reuse": [vp, i32],
        "mixattn_set_chunk_ring_direct": [vp, i32],
        "mixattn_profile_enable": [vp, i32],
        "mixattn_profile_read": [vp, i32, p32, C.POINTER(C.c_float)],
        "mixattn_get_launch_count": [vp, C.POINTER(C.c_int64)],
    }
    for name, args in sig.items():
        fn = getattr(lib, name)
        fn.argtypes = args
        fn.restype = C.c_int
    lib.mixattn_strerror.argtypes = [C.c_int]
    lib.mixattn_strerror.restype = C.c_char_p
    return lib


lib = _load()
EXPORTS = [
    "mixattn_arena_bytes", "mixattn_cache_bytes", "mixattn_create", "mixattn_destroy",
    "mixattn_seq_reset", "mixattn_append_kv", "mixattn_append_kv_rope", "mixattn_decode", "mixattn_decode_static_scratch", "mixattn_decode_layers", "mixattn_prefill",
    "mixattn_attend_chunk",
    "mixattn_get_len", "mixattn_get_block_table", "mixattn_get_n_free_pages",
    "mixattn_get_ring_state", "mixattn_locate", "mixattn_debug_read_kv", "mixattn_debug_read_kv_fp8",
    "mixattn_get_device_status", "mixattn_set_split_tokens", "mixattn_set_chunk_gather_reuse",
    "mixattn_set_chunk_ring_direct",
    "mixattn_profile_enable",
    "mixattn_profile_read", "mixattn_get_launch_count", "mixattn_strerror",
]


class MixAttnError(RuntimeError):
    def __init__(self, code: int, where: str):
        super().__init__(f"{where}: {lib.mixattn_strerror(code).decode()} ({code})")
        self.code = code


def strerror(code: int) -> str:
    return lib.mixattn_strerror(code).decode()


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int32)


def _p32(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.POINTER(C.c_int32))


def _dev(t) -> Optional[int]:
    return None if t is None else int(t.data_ptr())


def _stream(stream) -> Optional[int]:
    if stream is None:
        return None
    return int(getattr(stream, "cuda_stream", stream))


def make_config(layout: Sequence, n_q_heads: int, n_kv_heads: int, head_dim: int, dtype: int,
                max_seqs: int, n_pages: int, max_seq_len: int = 0, free_order=None,
                softmax_scale: float = 0.0, device: int = -1, page_size: int = 16,
                chunk_scratch_tokens: int = 0, kv_format: int = KV_NATIVE):
    """Returns (Config, keepalive): keepalive owns the arrays the struct points to."""
    layers = (LayerDesc * max(1, len(layout)))()
    for i, (kind, window, owner) in enumerate(layout):
        layers[i] = LayerDesc(int(kind), int(window), int(owner))
    fo = None if free_order is None else _i32(free_order)
    cfg = Config(len(layout), layers, n_q_heads, n_kv_heads, head_dim, dtype, max_seqs, page_size,
                 n_pages, max_seq_len, _p32(fo), float(softmax_scale), device, None, 0,
                 int(chunk_scratch_tokens), int(kv_format))
    return cfg, (layers, fo)


def arena_bytes(cfg: Config) -> int:
    out = C.c_size_t(0)
    rc = lib.mixattn_arena_bytes(C.byref(cfg), C.byref(out))
    if rc:
        raise MixAttnError(rc, "mixattn_arena_bytes")
    return out.value


def cache_bytes(cfg: Config) -> int:
    out = C.c_size_t(0)
    rc = lib.mixattn_cache_bytes(C.byref(cfg), C.byref(out))
    if rc:
        raise MixAttnError(rc, "mixattn_cache_bytes")
    return out.value


class Context:
    """Owns a mixattn_ctx and (on a GPU) the torch tensor that backs its arena.

    Methods have the names of the C calls without the prefix and raise
    MixAttnError on a non-zero status (`rc_*` variants return the status).
    """

    def __init__(self, layout, n_q_heads, n_kv_heads, head_dim, dtype, max_seqs, n_pages,
                 max_seq_len=0, free_order=None, softmax_scale=0.0, device=-1, chunk_scratch_tokens=0,
                 kv_format=KV_NATIVE):
        self.cfg, self._keep = make_config(layout, n_q_heads, n_kv_heads, head_dim, dtype, max_seqs,
                                           n_pages, max_seq_len, free_order, softmax_scale, device,
                                           chunk_scratch_tokens=chunk_scratch_tokens, kv_format=kv_format)
        self.arena = None
        if device >= 0:
            import torch
            nbytes = arena_bytes(self.cfg)
            self.arena = torch.empty(nbytes, dtype=torch.uint8, device=f"cuda:{device}")
            self.cfg.arena = self.arena.data_ptr()
            self.cfg.arena_bytes = nbytes
        h = C.c_void_p()
        rc = lib.mixattn_create(C.byref(self.cfg), C.byref(h))
        if rc:
            raise MixAttnError(rc, "mixattn_create")
        self.h = h
        self.n_q_heads, self.n_kv_heads, self.head_dim, self.dtype = n_q_heads, n_kv_heads, head_dim, dtype

    def close(self):
        if getattr(self, "h", None):
            lib.mixattn_destroy(self.h)
            self.h = None
        self.arena = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- calls -------------------------------------------------------------
    def rc_append_kv(self, layer, seq_ids, n_new=None, k=None, v=None, stream=None) -> int:
        s = _i32(seq_ids)
        n = None if n_new is None else _i32(n_new)
        return lib.mixattn_append_kv(self.h, layer, len(s), _p32(s), _p32(n), _dev(k), _dev(v), _stream(stream))

    def append_kv(self, layer, seq_ids, n_new=None, k=None, v=None, stream=None):
        rc = self.rc_append_kv(layer, seq_ids, n_new, k, v, stream)
        if rc:
            raise MixAttnError(rc, "mixattn_append_kv")

    def rc_append_kv_rope(self, layer, seq_ids, n_new, k, v, rope_theta, stream=None) -> int:
        s = _i32(seq_ids)
        n = None if n_new is None else _i32(n_new)
        return lib.mixattn_append_kv_rope(self.h, layer, len(s), _p32(s), _p32(n), _dev(k), _dev(v),
                                          float(rope_theta), _stream(stream))

    def append_kv_rope(self, layer, seq_ids, n_new, k, v, rope_theta, stream=None):
        rc = self.rc_append_kv_rope(layer, seq_ids, n_new, k, v, rope_theta, stream)
        if rc:
            raise MixAttnError(rc, "mixattn_append_kv_rope")

    def rc_decode(self, layer, seq_ids, q, out, stream=None) -> int:
        s = _i32(seq_ids)
        return lib.mixattn_decode(self.h, layer, len(s), _p32(s), _dev(q), _dev(out), _stream(stream))

    def decode(self, layer, seq_ids, q, out, stream=None):
        rc = self.rc_decode(layer, seq_ids, q, out, stream)
        if rc:
            raise MixAttnError(rc, "mixattn_decode")

    def rc_decode_static_scratch(self, layer, seq_ids, q, out, stream=None) -> int:
        """mixattn_decode_static_scratch: decode whose split partials live in the
        library's static device array instead of the arena workspace."""
        s = _i32(seq_ids)
        return lib.mixattn_decode_static_scratch(self.h, layer, len(s), _p32(s), _dev(q), _dev(out),
                                                 _stream(stream))

    def pointer_table(self, tensors):
        """Host array of device pointers, one per layer (None -> NULL), for mixattn_decode_layers.
        `tensors` maps a layer index to a tensor, or is a sequence indexed by layer."""
        n = self.cfg.n_layers
        arr = (C.c_void_p * n)()
        for l in range(n):
            t = tensors.get(l) if isinstance(tensors, dict) else tensors[l]
            arr[l] = None if t is None else int(t.data_ptr())
        return arr

    def rc_decode_layers(self, layer_begin, layer_end, seq_ids, q_tab, k_tab, v_tab, out_tab, stream=None):
        """mixattn_decode_layers with pointer tables from pointer_table(); returns (status, layers_done)."""
        s = _i32(seq_ids)
        done = C.c_int32(0)
        rc = lib.mixattn_decode_layers(self.h, layer_begin, layer_end, len(s), _p32(s), q_tab, k_tab, v_tab, out_tab,
                                       _stream(stream), C.byref(done))
        return rc, done.value

    def decode_layers(self, layer_begin, layer_end, seq_ids, q_tab, k_tab, v_tab, out_tab, stream=None):
        rc, _ = self.rc_decode_layers(layer_begin, layer_end, seq_ids, q_tab, k_tab, v_tab, out_tab, stream)
        if rc:
            raise MixAttnError(rc, "mixattn_decode_layers")

    def rc_prefill(self, layer, seq_ids, seq_lens, q, k, v, out, stream=None) -> int:
        s, n = _i32(seq_ids), _i32(seq_lens)
        return lib.mixattn_prefill(self.h, layer, len(s), _p32(s), _p32(n), _dev(q), _dev(k), _dev(v),
                                   _dev(out), _stream(stream))

    def prefill(self, layer, seq_ids, seq_lens, q, k, v, out, stream=None):
        rc = self.rc_prefill(layer, seq_ids, seq_lens, q, k, v, out, stream)
        if rc:
            raise MixAttnError(rc, "mixattn_prefill")

    def rc_attend_chunk(self, layer, seq_ids, seq_lens, q, k, v, out, stream=None) -> int:
        s, n = _i32(seq_ids), _i32(seq_lens)
        return lib.mixattn_attend_chunk(self.h, layer, len(s), _p32(s), _p32(n), _dev(q), _dev(k), _dev(v),
                                        _dev(out), _stream(stream))

    def attend_chunk(self, layer, seq_ids, seq_lens, q, k, v, out, stream=None):
        rc = self.rc_attend_chunk(layer, seq_ids, seq_lens, q, k, v, out, stream)
        if rc:
            raise MixAttnError(rc, "mixattn_attend_chunk")

    def seq_reset(self, seq):
        rc = lib.mixattn_seq_reset(self.h, seq)
        if rc:
            raise MixAttnError(rc, "mixattn_seq_reset")

    def get_len(self, layer, seq) -> int:
        out = C.c_int32()
        rc = lib.mixattn_get_len(self.h, layer, seq, C.byref(out))
        if rc:
            raise MixAttnError(rc, "mixattn_get_len")
        return out.value

    def get_block_table(self, seq):
        n = C.c_int32()
        rc = lib.mixattn_get_block_table(self.h, seq, None, 0, C.byref(n))
        if rc:
            raise MixAttnError(rc, "mixattn_get_block_table")
        buf = np.zeros(max(1, n.value), dtype=np.int32)
        rc = lib.mixattn_get_block_table(self.h, seq, _p32(buf), n.value, C.byref(n))
        if rc:
            raise MixAttnError(rc, "mixattn_get_block_table")
        return buf[:n.value].tolist()

    def get_n_free_pages(self) -> int:
        out = C.c_int32()
        rc = lib.mixattn_get_n_free_pages(self.h, C.byref(out))
        if rc:
            raise MixAttnError(rc, "mixattn_get_n_free_pages")
        return out.value

    def get_ring_state(self, layer, seq):
        a, b = C.c_int32(), C.c_int32()
        rc = lib.mixattn_get_ring_state(self.h, layer, seq, C.byref(a), C.byref(b))
        if rc:
            raise MixAttnError(rc, "mixattn_get_ring_state")
        return a.value, b.value

    def locate(self, layer, seq, pos):
        a, b = C.c_int32(), C.c_int32()
        rc = lib.mixattn_locate(self.h, layer, seq, pos, C.byref(a), C.byref(b))
        if rc:
            raise MixAttnError(rc, "mixattn_locate")
        return a.value, b.value

    def debug_read_kv(self, layer, seq, pos):
        """Returns (K, V) as torch CPU tensors [Hkv, D] in the context dtype."""
        import torch
        dt = torch.bfloat16 if self.dtype == BF16 else torch.float32
        k = torch.empty(self.n_kv_heads, self.head_dim, dtype=dt)
        v = torch.empty_like(k)
        rc = lib.mixattn_debug_read_kv(self.h, layer, seq, pos, k.data_ptr(), v.data_ptr())
        if rc:
            raise MixAttnError(rc, "mixattn_debug_read_kv")
        return k, v

    def debug_read_kv_fp8(self, layer, seq, pos):
        """Quantised storage: (k_codes, k_exp, v_codes, v_exp) as numpy arrays: uint8 [Hkv, D]
        codes and int32 [Hkv] shared exponents."""
        kc = np.zeros((self.n_kv_heads, self.head_dim), dtype=np.uint8)
        vc = np.zeros_like(kc)
        kx = np.zeros(self.n_kv_heads, dtype=np.int32)
        vx = np.zeros_like(kx)
        rc = lib.mixattn_debug_read_kv_fp8(self.h, layer, seq, pos, kc.ctypes.data, kx.ctypes.data,
                                           vc.ctypes.data, vx.ctypes.data)
        if rc:
            raise MixAttnError(rc, "mixattn_debug_read_kv_fp8")
        return kc, kx, vc, vx

    def get_device_status(self) -> int:
        out = C.c_int32()
        rc = lib.mixattn_get_device_status(self.h, C.byref(out))
        if rc:
            raise MixAttnError(rc, "mixattn_get_device_status")
        return out.value

    def set_split_tokens(self, tokens: int):
        rc = lib.mixattn_set_split_tokens(self.h, tokens)
        if rc:
            raise MixAttnError(rc, "mixattn_set_split_tokens")

    def set_chunk_gather_reuse(self, enable: bool):
        """Layers that share a cache gather the same rows for a chunk: copy them once per run of
        such calls (the caller keeps k / v unchanged between them)."""
        rc = lib.mixattn_set_chunk_gather_reuse(self.h, 1 if enable else 0)
        if rc:
            raise MixAttnError(rc, "mixattn_set_chunk_gather_reuse")

    def set_chunk_ring_direct(self, enable: bool):
        """Sliding-window chunk calls read the ring in place where its window is a whole number of
        128-key tiles (on by default); off = they copy the cached keys like every other chunk call."""
        rc = lib.mixattn_set_chunk_ring_direct(self.h, 1 if enable else 0)
        if rc:
            raise MixAttnError(rc, "mixattn_set_chunk_ring_direct")

    def profile_enable(self, enable: bool):
        rc = lib.mixattn_profile_enable(self.h, 1 if enable else 0)
        if rc:
            raise MixAttnError(rc, "mixattn_profile_enable")

    def profile_read(self, kernel_class: int):
        n, ms = C.c_int32(), C.c_float()
        rc = lib.mixattn_profile_read(self.h, kernel_class, C.byref(n), C.byref(ms))
        if rc:
            raise MixAttnError(rc, "mixattn_profile_read")
        return n.value, ms.value

    def get_launch_count(self) -> int:
        out = C.c_int64()
        rc = lib.mixattn_get_launch_count(self.h, C.byref(out))
        if rc:
            raise MixAttnError(rc, "mixattn_get_launch_count")
        return out.value
