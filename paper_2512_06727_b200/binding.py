"""ctypes binding of libkvcar.so: argument marshalling only.

Every function below maps one-to-one onto the C entry point of the same name in
include/kvcar.h; all arithmetic of the decode path runs in the CUDA library.
There is no fallback: if the library cannot be loaded the import fails.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence, Tuple

import numpy as np

from . import build as _build

F32, BF16 = 0, 1
K, V = 0, 1
KERNEL_AUTO, KERNEL_GENERIC, KERNEL_TENSOR, KERNEL_RAW = 0, 1, 2, 3
INCLUDE_CURRENT_EXACT = 1
ABSORBED = 2
ABSORBED_V = 4
MAX_BATCH = 512

STATUS_NAMES = {0: "OK", 1: "INVALID_ARG", 2: "STATE", 3: "OOM_PAGES", 4: "WORKSPACE", 5: "UNSUPPORTED",
                6: "CUDA", 7: "DEVICE_TIMEOUT", 8: "GUARD"}

EXPORTS = [
    "kvcar_create", "kvcar_destroy", "kvcar_set_reuse_map", "kvcar_set_autoencoder", "kvcar_required_bytes",
    "kvcar_bind_memory", "kvcar_set_kernel", "kvcar_seq_open", "kvcar_seq_close", "kvcar_reserve",
    "kvcar_encode_append", "kvcar_encode_append_tensor", "kvcar_advance", "kvcar_decode_attention", "kvcar_decode_attention_static",
    "kvcar_step_layer", "kvcar_step_layer_host",
    "kvcar_debug_resolve", "kvcar_debug_locate", "kvcar_seq_len", "kvcar_pool_layout", "kvcar_pool_quant_layout",
    "kvcar_cache_bytes_per_token", "kvcar_layer_work_per_token", "kvcar_layer_work_absorbed", "kvcar_launch_count", "kvcar_layer_kernel", "kvcar_sync_status",
    "kvcar_last_error", "kvcar_debug_expire_wait", "kvcar_debug_check",
    "kvcar_head_l1_scratch_bytes", "kvcar_head_l1_distance", "kvcar_reuse_map_from_l1",
]


class KvcarError(RuntimeError):
    def __init__(self, status: int, msg: str):
        super().__init__(f"kvcar: {STATUS_NAMES.get(status, status)}: {msg}")
        self.status = status


class Config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "n_q_heads", "n_kv_heads", "head_dim", "page_tokens",
                                          "max_seqs", "max_pages", "max_pages_per_seq", "storage",
                                          "latent_quant")]


_FP = C.POINTER(C.c_float)


class AE(C.Structure):
    _fields_ = [("in_dim", C.c_int32), ("hidden", C.c_int32), ("latent", C.c_int32),
                ("leaky_slope", C.c_float), ("bn_eps", C.c_float)] + \
               [(n, _FP) for n in ("enc_w1", "enc_b1", "enc_bn", "enc_w2", "enc_b2",
                                   "dec_w1", "dec_b1", "dec_bn", "dec_w2", "dec_b2")]


def lib_path() -> str:
    return _build.LIB


_LIB: Optional[C.CDLL] = None


def load(trace: bool = False) -> C.CDLL:
    """The library, built if its sources are newer, loaded once per process.  trace: the time-stamping build of
    the same sources (must be the first load of the process)."""
    global _LIB
    if _LIB is None:
        _LIB = _load(trace)
    return _LIB


def _load(trace: bool = False) -> C.CDLL:
    path = _build.TRACE_LIB if trace else lib_path()
    if _build.needs_build(path):
        _build.build(trace=trace)
    if not os.path.exists(path):
        raise ImportError(f"{path} is missing and could not be built; the CUDA library is required")
    lib = C.CDLL(path)
    vp, i32, u32, sz = C.c_void_p, C.c_int32, C.c_uint32, C.c_size_t
    ip = C.POINTER(C.c_int32)
    sig = {
        "kvcar_create": [C.POINTER(Config), C.POINTER(vp)],
        "kvcar_destroy": [vp],
        "kvcar_set_reuse_map": [vp, ip, ip],
        "kvcar_set_autoencoder": [vp, i32, i32, C.POINTER(AE)],
        "kvcar_required_bytes": [vp, C.POINTER(sz), C.POINTER(sz), C.POINTER(sz)],
        "kvcar_bind_memory": [vp, vp, sz, vp, sz, vp, sz, vp],
        "kvcar_set_kernel": [vp, i32],
        "kvcar_seq_open": [vp, i32],
        "kvcar_seq_close": [vp, i32],
        "kvcar_reserve": [vp, ip, i32, i32],
        "kvcar_encode_append": [vp, i32, ip, i32, i32, vp, vp, vp],
        "kvcar_encode_append_tensor": [vp, i32, ip, i32, i32, vp, vp, vp],
        "kvcar_advance": [vp, ip, i32, i32, vp],
        "kvcar_decode_attention": [vp, i32, ip, i32, vp, vp, u32, vp],
        "kvcar_decode_attention_static": [vp, i32, ip, i32, vp, vp, u32, vp],
        "kvcar_step_layer": [vp, i32, ip, i32, vp, vp, vp, vp, u32, vp],
        "kvcar_step_layer_host": [vp, i32, ip, i32, vp, vp, vp, vp, u32, vp],
        "kvcar_debug_resolve": [vp, i32, i32, i32, ip, ip, ip],
        "kvcar_debug_locate": [vp, i32, i32, ip, C.POINTER(C.c_int64)],
        "kvcar_seq_len": [vp, i32, ip],
        "kvcar_pool_layout": [vp, i32, i32, C.POINTER(sz), C.POINTER(sz), ip],
        "kvcar_pool_quant_layout": [vp, i32, i32, C.POINTER(sz)],
        "kvcar_cache_bytes_per_token": [vp, C.POINTER(C.c_double), C.POINTER(C.c_double)],
        "kvcar_layer_work_per_token": [vp, i32, C.POINTER(C.c_double), C.POINTER(C.c_double)],
        "kvcar_layer_work_absorbed": [vp, i32, i32, C.POINTER(C.c_double)],
        "kvcar_launch_count": [vp, C.POINTER(C.c_int64)],
        "kvcar_layer_kernel": [vp, i32, ip],
        "kvcar_sync_status": [vp, vp],
        "kvcar_debug_expire_wait": [vp, C.c_uint64, vp],
        "kvcar_debug_check": [vp, vp, C.POINTER(C.c_int32), C.POINTER(C.c_int64)],
        "kvcar_head_l1_scratch_bytes": [i32, i32, C.c_int64, C.POINTER(sz)],
        "kvcar_head_l1_distance": [i32, i32, i32, i32, vp, C.c_int64, vp, sz, vp, vp],
        "kvcar_reuse_map_from_l1": [C.POINTER(C.c_float), i32, i32, i32, ip],
    }
    for name, args in sig.items():
        fn = getattr(lib, name)
        fn.argtypes = args
        fn.restype = C.c_int
    lib.kvcar_last_error.argtypes = [vp]
    lib.kvcar_last_error.restype = C.c_char_p
    return lib


# -- the context-free calls: choosing the reuse map (argument marshalling only) -------------------
def head_l1_scratch_bytes(n_layers: int, n_kv_heads: int, n_rows: int) -> int:
    out = C.c_size_t()
    st = load().kvcar_head_l1_scratch_bytes(n_layers, n_kv_heads, n_rows, C.byref(out))
    if st != 0:
        raise KvcarError(st, "kvcar_head_l1_scratch_bytes")
    return out.value


def head_l1_distance(n_layers: int, n_kv_heads: int, head_dim: int, storage: int, x: int, n_rows: int, scratch: int,
                     scratch_bytes: int, dist: int, stream: int = 0) -> None:
    """x, scratch, dist: device addresses (see kvcar_head_l1_distance in kvcar.h)."""
    st = load().kvcar_head_l1_distance(n_layers, n_kv_heads, head_dim, storage, x, n_rows, scratch, scratch_bytes, dist,
                                       stream)
    if st != 0:
        raise KvcarError(st, "kvcar_head_l1_distance")


def reuse_map_from_l1(dist: Sequence[float], n_layers: int, n_kv_heads: int, n_reuse: int) -> List[int]:
    arr = (C.c_float * len(dist))(*dist)
    src = (C.c_int32 * (n_layers * n_kv_heads))()
    st = load().kvcar_reuse_map_from_l1(arr, n_layers, n_kv_heads, n_reuse, src)
    if st != 0:
        raise KvcarError(st, "kvcar_reuse_map_from_l1")
    return list(src)


def _ints(seq: Sequence[int]):
    arr = (C.c_int32 * len(seq))(*seq)
    return arr


class Context:
    """One kvcar_ctx.  Methods carry the C names without the prefix and take raw
    device addresses (ints, e.g. tensor.data_ptr()) for device buffers."""

    def __init__(self, n_layers: int, n_q_heads: int, n_kv_heads: int, head_dim: int, page_tokens: int,
                 max_seqs: int, max_pages: int, max_pages_per_seq: int, storage: int, latent_quant: int = 0):
        self.lib = load()
        self.cfg = Config(n_layers, n_q_heads, n_kv_heads, head_dim, page_tokens, max_seqs, max_pages,
                          max_pages_per_seq, storage, latent_quant)
        self._h = C.c_void_p()
        st = self.lib.kvcar_create(C.byref(self.cfg), C.byref(self._h))
        if st != 0:
            raise KvcarError(st, "kvcar_create rejected the configuration")
        self._keep = []
        self._seq_cache = {}

    # -- plumbing --------------------------------------------------------
    def _check(self, st: int):
        if st != 0:
            raise KvcarError(st, self.lib.kvcar_last_error(self._h).decode())

    def _seqs(self, seqs: Sequence[int]):
        key = tuple(seqs)
        arr = self._seq_cache.get(key)
        if arr is None:
            arr = _ints(seqs)
            if len(self._seq_cache) < 64:
                self._seq_cache[key] = arr
        return arr

    def destroy(self):
        if self._h:
            self.lib.kvcar_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    # -- set-up ------------------------------------------------------------
    def set_reuse_map(self, src_k, src_v):
        a = np.ascontiguousarray(src_k, dtype=np.int32)
        b = np.ascontiguousarray(src_v, dtype=np.int32)
        n = self.cfg.n_layers * self.cfg.n_kv_heads
        if a.size != n or b.size != n:
            raise ValueError("reuse map must have n_layers*n_kv_heads entries")
        ip = C.POINTER(C.c_int32)
        self._check(self.lib.kvcar_set_reuse_map(self._h, a.ctypes.data_as(ip), b.ctypes.data_as(ip)))

    def set_autoencoder(self, layer: int, which: int, ae: dict):
        s = AE()
        s.in_dim, s.hidden, s.latent = ae["in_dim"], ae["hidden"], ae["latent"]
        s.leaky_slope, s.bn_eps = ae["leaky_slope"], ae["bn_eps"]
        hold = []
        shapes = {"enc_w1": s.hidden * s.in_dim, "enc_b1": s.hidden, "enc_bn": 4 * s.hidden,
                  "enc_w2": s.latent * s.hidden, "enc_b2": s.latent, "dec_w1": s.hidden * s.latent,
                  "dec_b1": s.hidden, "dec_bn": 4 * s.hidden, "dec_w2": s.in_dim * s.hidden, "dec_b2": s.in_dim}
        for name, n in shapes.items():
            arr = np.ascontiguousarray(ae[name], dtype=np.float32)
            if arr.size != n:
                raise ValueError(f"{name}: expected {n} elements, got {arr.size}")
            hold.append(arr)
            setattr(s, name, arr.ctypes.data_as(_FP))
        self._check(self.lib.kvcar_set_autoencoder(self._h, layer, which, C.byref(s)))

    def required_bytes(self) -> Tuple[int, int, int]:
        a, b, c = C.c_size_t(), C.c_size_t(), C.c_size_t()
        self._check(self.lib.kvcar_required_bytes(self._h, C.byref(a), C.byref(b), C.byref(c)))
        return a.value, b.value, c.value

    def bind_memory(self, pool: int, pool_bytes: int, weights: int, weights_bytes: int, workspace: int,
                    workspace_bytes: int, stream: int = 0):
        self._check(self.lib.kvcar_bind_memory(self._h, pool, pool_bytes, weights, weights_bytes, workspace,
                                               workspace_bytes, stream))

    def set_kernel(self, kernel: int):
        self._check(self.lib.kvcar_set_kernel(self._h, kernel))

    # -- sequences ---------------------------------------------------------
    def seq_open(self, seq: int):
        self._check(self.lib.kvcar_seq_open(self._h, seq))

    def seq_close(self, seq: int):
        self._check(self.lib.kvcar_seq_close(self._h, seq))

    def reserve(self, seqs: Sequence[int], n_tokens: int):
        self._check(self.lib.kvcar_reserve(self._h, self._seqs(seqs), len(seqs), n_tokens))

    # -- hot path ----------------------------------------------------------
    def encode_append(self, layer: int, seqs: Sequence[int], n_tokens: int, k: int, v: int, stream: int = 0):
        self._check(self.lib.kvcar_encode_append(self._h, layer, self._seqs(seqs), len(seqs), n_tokens, k, v, stream))

    def encode_append_tensor(self, layer: int, seqs: Sequence[int], n_tokens: int, k: int, v: int, stream: int = 0):
        self._check(self.lib.kvcar_encode_append_tensor(self._h, layer, self._seqs(seqs), len(seqs), n_tokens, k, v,
                                                        stream))

    def advance(self, seqs: Sequence[int], n_tokens: int, stream: int = 0):
        self._check(self.lib.kvcar_advance(self._h, self._seqs(seqs), len(seqs), n_tokens, stream))

    def decode_attention(self, layer: int, seqs: Sequence[int], q: int, out: int,
                         flags: int = INCLUDE_CURRENT_EXACT, stream: int = 0):
        self._check(self.lib.kvcar_decode_attention(self._h, layer, self._seqs(seqs), len(seqs), q, out, flags, stream))

    def decode_attention_static(self, layer: int, seqs: Sequence[int], q: int, out: int,
                                flags: int = INCLUDE_CURRENT_EXACT, stream: int = 0):
        """Decode attention whose split-KV scratch is the library's built-in array
        (allocates nothing; see kvcar_decode_attention_static in kvcar.h)."""
        self._check(self.lib.kvcar_decode_attention_static(self._h, layer, self._seqs(seqs), len(seqs), q, out,
                                                           flags, stream))

    def step_layer(self, layer: int, seqs: Sequence[int], k: int, v: int, q: int, out: int,
                   flags: int = INCLUDE_CURRENT_EXACT, stream: int = 0):
        """encode_append (one token) + decode_attention of one layer in one call, device buffers."""
        self._check(self.lib.kvcar_step_layer(self._h, layer, self._seqs(seqs), len(seqs), k, v, q, out, flags, stream))

    def step_layer_host(self, layer: int, seqs: Sequence[int], k_host: int, v_host: int, q_host: int,
                        out_host: int, flags: int = INCLUDE_CURRENT_EXACT, stream: int = 0):
        self._check(self.lib.kvcar_step_layer_host(self._h, layer, self._seqs(seqs), len(seqs), k_host, v_host,
                                                   q_host, out_host, flags, stream))

    # -- observability -------------------------------------------------------
    def debug_resolve(self, layer: int, kv_head: int, which: int) -> Tuple[int, int, int]:
        a, b, c = C.c_int32(), C.c_int32(), C.c_int32()
        self._check(self.lib.kvcar_debug_resolve(self._h, layer, kv_head, which, C.byref(a), C.byref(b), C.byref(c)))
        return a.value, b.value, c.value

    def debug_locate(self, seq: int, token: int) -> Tuple[int, int]:
        p, r = C.c_int32(), C.c_int64()
        self._check(self.lib.kvcar_debug_locate(self._h, seq, token, C.byref(p), C.byref(r)))
        return p.value, r.value

    def seq_len(self, seq: int) -> int:
        n = C.c_int32()
        self._check(self.lib.kvcar_seq_len(self._h, seq, C.byref(n)))
        return n.value

    def pool_layout(self, layer: int, which: int) -> Tuple[int, int, int]:
        off, pitch, width = C.c_size_t(), C.c_size_t(), C.c_int32()
        self._check(self.lib.kvcar_pool_layout(self._h, layer, which, C.byref(off), C.byref(pitch), C.byref(width)))
        return off.value, pitch.value, width.value

    def pool_quant_layout(self, layer: int, which: int) -> int:
        off = C.c_size_t()
        self._check(self.lib.kvcar_pool_quant_layout(self._h, layer, which, C.byref(off)))
        return off.value

    def cache_bytes_per_token(self) -> Tuple[float, float]:
        a, b = C.c_double(), C.c_double()
        self._check(self.lib.kvcar_cache_bytes_per_token(self._h, C.byref(a), C.byref(b)))
        return a.value, b.value

    def layer_work_per_token(self, layer: int) -> Tuple[float, float]:
        a, b = C.c_double(), C.c_double()
        self._check(self.lib.kvcar_layer_work_per_token(self._h, layer, C.byref(a), C.byref(b)))
        return a.value, b.value

    def layer_work_absorbed(self, layer: int, both_sides: bool = False) -> float:
        a = C.c_double()
        self._check(self.lib.kvcar_layer_work_absorbed(self._h, layer, int(both_sides), C.byref(a)))
        return a.value

    def launch_count(self) -> int:
        n = C.c_int64()
        self._check(self.lib.kvcar_launch_count(self._h, C.byref(n)))
        return n.value

    def layer_kernel(self, layer: int) -> int:
        k = C.c_int32()
        self._check(self.lib.kvcar_layer_kernel(self._h, layer, C.byref(k)))
        return k.value

    def sync_status(self, stream: int = 0):
        self._check(self.lib.kvcar_sync_status(self._h, stream))

    def debug_expire_wait(self, limit_ns: int, stream: int = 0):
        self._check(self.lib.kvcar_debug_expire_wait(self._h, limit_ns, stream))

    def debug_check(self, stream: int = 0):
        """(status, what, where) of kvcar_debug_check; status 0 = guards and device tables intact."""
        what, where = C.c_int32(), C.c_int64()
        st = self.lib.kvcar_debug_check(self._h, stream, C.byref(what), C.byref(where))
        return st, what.value, where.value
