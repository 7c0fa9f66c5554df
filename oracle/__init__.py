"""Float64 CPU oracle for Cartridge decode attention.  TEST INFRASTRUCTURE ONLY.

Nothing in the product package imports this.  Allowed users: the test-suite, the smoke check and
the benchmark's CPU-baseline / reference legs.  The arithmetic lives in ``cart_oracle.c`` (plain C,
OpenMP over (request, KV head)); this module only builds it with gcc, marshals numpy arrays into it
and keeps the bookkeeping of which KV tokens a request attends to (Cartridges first, in composition
order, then the request's own suffix -- the cache layout of the paper's Sec. 3.2 / Sec. 3.3).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "cart_oracle.c")
_LIB = os.path.join(_HERE, "libcart_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP) if the shared object is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.cart_oracle_num_threads.restype = ctypes.c_int
        lib.cart_oracle_decode_layer.restype = ctypes.c_int
        lib.cart_oracle_decode_layer.argtypes = [
            ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_double,
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        _lib = lib
    return _lib


def num_threads() -> int:
    """Threads the C oracle will use (OpenMP's maximum)."""
    return int(_load().cart_oracle_num_threads())


Segment = Tuple[np.ndarray, np.ndarray]  # (K bits, V bits), each uint16 [Hkv][n][D]


def decode_layer(q_bits: np.ndarray, segments: Sequence[Sequence[Segment]], scale: float
                 ) -> Tuple[np.ndarray, np.ndarray]:
    """Eq. 1 at the last position for every request of a batch, one layer.

    q_bits    uint16 [B][Hq][D], bf16 bit patterns.
    segments  per request, the ordered list of (K, V) blocks the request attends to; each block is
              uint16 [Hkv][n][D].
    Returns (out float64 [B][Hq][D], lse float64 [B][Hq]).
    """
    lib = _load()
    q_bits = np.ascontiguousarray(q_bits, dtype=np.uint16)
    B, Hq, D = q_bits.shape
    assert len(segments) == B
    keep = []  # keeps the arrays alive while C reads them
    seg_begin = np.zeros(B + 1, dtype=np.int32)
    k_ptrs: List[int] = []
    v_ptrs: List[int] = []
    ns: List[int] = []
    strides: List[int] = []
    Hkv: Optional[int] = None
    for b, segs in enumerate(segments):
        for (k, v) in segs:
            assert k.dtype == np.uint16 and v.dtype == np.uint16 and k.shape == v.shape
            assert k.ndim == 3 and k.shape[2] == D
            if Hkv is None:
                Hkv = k.shape[0]
            assert k.shape[0] == Hkv
            n = k.shape[1]
            k = np.ascontiguousarray(k)
            v = np.ascontiguousarray(v)
            keep.append((k, v))
            k_ptrs.append(k.ctypes.data)
            v_ptrs.append(v.ctypes.data)
            ns.append(n)
            strides.append(n * D)
        seg_begin[b + 1] = len(ns)
    if Hkv is None:
        raise ValueError("no KV segment given")
    k_arr = np.asarray(k_ptrs, dtype=np.uint64)
    v_arr = np.asarray(v_ptrs, dtype=np.uint64)
    n_arr = np.asarray(ns, dtype=np.int64)
    s_arr = np.asarray(strides, dtype=np.int64)
    out = np.empty((B, Hq, D), dtype=np.float64)
    lse = np.empty((B, Hq), dtype=np.float64)
    rc = lib.cart_oracle_decode_layer(
        B, Hq, Hkv, D, float(scale), q_bits.ctypes.data, seg_begin.ctypes.data,
        k_arr.ctypes.data, v_arr.ctypes.data, n_arr.ctypes.data, s_arr.ctypes.data,
        out.ctypes.data, lse.ctypes.data)
    if rc == 2:
        raise ValueError("a request has an empty KV cache")
    if rc != 0:
        raise RuntimeError("cart_oracle_decode_layer failed with code %d" % rc)
    return out, lse


class OracleCache:
    """Bookkeeping twin of the serving state: Cartridges, compositions, requests with suffixes.

    A Cartridge is a pair of uint16 arrays [L][Hkv][p][D] (the trained key and value vectors of
    Sec. 3.2, here synthetic).  ``compose`` returns a handle that stands for the concatenation of
    its parts along the token axis, in list order (Sec. 3.1 "capable of composition", Sec. 5.4).  A
    request attends to its Cartridge handle's tokens followed by its own suffix, which grows by one
    token per ``append`` (decode phase of Sec. 2.3).
    """

    def __init__(self, n_layers: int, n_q_heads: int, n_kv_heads: int, head_dim: int, scale: float):
        self.L, self.Hq, self.Hkv, self.D = n_layers, n_q_heads, n_kv_heads, head_dim
        self.scale = float(scale)
        self._carts: Dict[int, List[Tuple[np.ndarray, np.ndarray]]] = {}
        self._reqs: Dict[int, dict] = {}
        self._next_cart = 0
        self._next_req = 0

    def register(self, k_bits: np.ndarray, v_bits: np.ndarray) -> int:
        assert k_bits.shape == v_bits.shape and k_bits.shape[0] == self.L
        assert k_bits.shape[1] == self.Hkv and k_bits.shape[3] == self.D
        cid = self._next_cart
        self._next_cart += 1
        self._carts[cid] = [(np.asarray(k_bits, dtype=np.uint16), np.asarray(v_bits, dtype=np.uint16))]
        return cid

    def compose(self, parts: Sequence[int]) -> int:
        blocks: List[Tuple[np.ndarray, np.ndarray]] = []
        for p in parts:
            blocks.extend(self._carts[p])
        cid = self._next_cart
        self._next_cart += 1
        self._carts[cid] = blocks
        return cid

    def open(self, cart: Optional[int]) -> int:
        rid = self._next_req
        self._next_req += 1
        empty = np.zeros((self.Hkv, 0, self.D), dtype=np.uint16)
        self._reqs[rid] = {"cart": cart, "k": [empty.copy() for _ in range(self.L)],
                           "v": [empty.copy() for _ in range(self.L)]}
        return rid

    def append(self, layer: int, reqs: Sequence[int], k_new: np.ndarray, v_new: np.ndarray) -> None:
        """k_new, v_new: uint16 [len(reqs)][Hkv][D]; token i goes to the end of reqs[i]'s suffix."""
        for i, r in enumerate(reqs):
            st = self._reqs[r]
            st["k"][layer] = np.concatenate([st["k"][layer], k_new[i][:, None, :]], axis=1)
            st["v"][layer] = np.concatenate([st["v"][layer], v_new[i][:, None, :]], axis=1)

    def extend(self, layer: int, req: int, k_new: np.ndarray, v_new: np.ndarray) -> None:
        """k_new, v_new: uint16 [T][Hkv][D]; the T tokens go, in order, to the end of req's suffix
        (what prefill of the user's message leaves in the cache, Sec. 2.3)."""
        st = self._reqs[req]
        st["k"][layer] = np.concatenate([st["k"][layer], np.transpose(k_new, (1, 0, 2))], axis=1)
        st["v"][layer] = np.concatenate([st["v"][layer], np.transpose(v_new, (1, 0, 2))], axis=1)

    def suffix_len(self, req: int, layer: int) -> int:
        return int(self._reqs[req]["k"][layer].shape[1])

    def segments(self, layer: int, req: int) -> List[Segment]:
        st = self._reqs[req]
        segs: List[Segment] = []
        if st["cart"] is not None:
            for (k, v) in self._carts[st["cart"]]:
                segs.append((k[layer], v[layer]))
        if st["k"][layer].shape[1] > 0:
            segs.append((st["k"][layer], st["v"][layer]))
        return segs

    def kv_tokens(self, layer: int, req: int) -> int:
        return sum(k.shape[1] for (k, _) in self.segments(layer, req))

    def decode(self, layer: int, reqs: Sequence[int], q_bits: np.ndarray
               ) -> Tuple[np.ndarray, np.ndarray]:
        return decode_layer(q_bits, [self.segments(layer, r) for r in reqs], self.scale)
