"""ctypes wrapper around the fp64 CPU oracle (``moe_vqlr_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the benchmark's
CPU-baseline leg.  Nothing here is shared with, or imported by, the CUDA library or its
Python binding.  Inputs are plain numpy arrays (bf16 as ``uint16`` bit patterns).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "moe_vqlr_oracle.c")
_LIB = os.path.join(_HERE, "libmoe_vqlr_oracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP) if the shared object is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.run(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-std=c11", "-Wall",
                        "-o", _LIB, _SRC, "-lm"], check=True)
    return _LIB


class _Proj(C.Structure):
    _fields_ = [("kind", C.c_int32), ("idx_bytes", C.c_int32), ("codebook", C.c_void_p),
                ("idx", C.c_void_p), ("basis", C.c_void_p), ("factor", C.c_void_p),
                ("dense", C.c_void_p)]


class _Layer(C.Structure):
    _fields_ = [("H", C.c_int32), ("I", C.c_int32), ("E", C.c_int32), ("k", C.c_int32),
                ("S", C.c_int32), ("d", C.c_int32), ("K", C.c_int32), ("r", C.c_int32),
                ("renorm_topk", C.c_int32), ("act", C.c_int32), ("router_w", C.c_void_p),
                ("router_bias", C.c_void_p), ("gate", _Proj), ("up", _Proj), ("down", _Proj)]


ACTIVATIONS = {"silu": 0, "gelu_tanh": 1, "relu2": 2}     # ORACLE_ACT_* of the C file ("relu2": up-only experts)

_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.oracle_threads.restype = C.c_int
        _lib.oracle_decode_layer.restype = C.c_int
        _lib.oracle_activation.restype = C.c_double
        _lib.oracle_activation.argtypes = [C.c_double, C.c_int]
        _lib.oracle_reconstruct.restype = C.c_int
        _lib.oracle_storage_bits_per_weight.restype = C.c_double
        _lib.oracle_storage_bits_per_weight.argtypes = [C.c_int] * 10
    return _lib


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _c(a, dtype):
    return None if a is None else np.ascontiguousarray(a, dtype=dtype)


@dataclass
class LayerResult:
    out: np.ndarray            # [T][n_out] f64
    logits: np.ndarray         # [T][E] f64
    topk_id: np.ndarray        # [T][k] i32
    topk_w: np.ndarray         # [T][k] f64
    counts: np.ndarray         # [E] i32
    offsets: np.ndarray        # [E+1] i32
    pair_token: np.ndarray     # [T*k] i32
    pair_slot: np.ndarray      # [T*k] i32
    y_pair: np.ndarray         # [T][k+S][n_out] f64
    bad_index: bool


class OracleLayer:
    """Holds the arrays of one layer alive and exposes the oracle's steps."""

    def __init__(self, *, H, I, E, k, S, d, K, r, router_w, router_bias, gate, up, down,
                 renorm_topk=True, act="silu"):
        self.H, self.I, self.E, self.k, self.S, self.d, self.K, self.r = H, I, E, k, S, d, K, r
        self._keep = []
        L = _Layer()
        L.H, L.I, L.E, L.k, L.S, L.d, L.K, L.r = H, I, E, k, S, d, K, r
        L.renorm_topk = 1 if renorm_topk else 0
        L.act = ACTIVATIONS[act]
        rw = _c(router_w, np.uint16)
        rb = _c(router_bias, np.float32)
        self._keep += [rw, rb]
        L.router_w = _ptr(rw)
        L.router_bias = _ptr(rb)
        for name, p in (("gate", gate), ("up", up), ("down", down)):
            setattr(L, name, self._proj(p))
        self._L = L

    def _proj(self, p) -> _Proj:
        P = _Proj()
        if p is None:              # up-only experts have no gate projection
            return P
        P.kind = int(p.kind)
        idx = None
        if p.idx is not None:
            idx = np.ascontiguousarray(p.idx)
            assert idx.dtype in (np.uint8, np.uint16)
            P.idx_bytes = 12 if getattr(p, "idx_bits", 0) == 12 else idx.dtype.itemsize
        else:
            P.idx_bytes = 1
        arrs = dict(codebook=_c(p.codebook, np.uint16), idx=idx, basis=_c(p.basis, np.uint16),
                    factor=_c(p.factor, np.uint16), dense=_c(p.dense, np.uint16))
        for key, a in arrs.items():
            self._keep.append(a)
            setattr(P, key, _ptr(a))
        return P

    @classmethod
    def from_synth(cls, layer, renorm_topk=True, act=None) -> "OracleLayer":
        s = layer.shape
        return cls(H=s.H, I=s.I, E=s.E, k=s.k, S=s.S, d=s.d, K=s.K, r=s.r,
                   router_w=layer.router_w, router_bias=layer.router_bias, gate=layer.gate,
                   up=layer.up, down=layer.down, renorm_topk=renorm_topk,
                   act=act or getattr(s, "act", "silu"))

    # ---- steps -------------------------------------------------------------------------
    def router_logits(self, x_bits: np.ndarray) -> np.ndarray:
        x = _c(x_bits, np.uint16)
        T = x.shape[0]
        out = np.empty((T, self.E), np.float64)
        lib().oracle_router_logits(C.byref(self._L), _ptr(x), C.c_int(T), _ptr(out))
        return out

    def reconstruct(self, proj: str, e: int) -> np.ndarray:
        out_dim, in_dim = (self.H, self.I) if proj == "down" else (self.I, self.H)
        W = np.empty((out_dim, in_dim), np.float64)
        P = getattr(self._L, proj)
        rc = lib().oracle_reconstruct(C.byref(P), C.c_int(e), C.c_int(out_dim), C.c_int(in_dim),
                                      C.c_int(self.d), C.c_int(self.K), C.c_int(self.r), _ptr(W))
        if rc:
            raise ValueError("index >= K")
        return W

    def project_shared(self, proj: str, e: int, x: np.ndarray) -> np.ndarray:
        """Projection output via the projection code book and z (the paper's evaluation order)."""
        out_dim, in_dim = (self.H, self.I) if proj == "down" else (self.I, self.H)
        xv = _c(x, np.float64)
        o = np.empty(out_dim, np.float64)
        P = getattr(self._L, proj)
        lib().oracle_project_shared(C.byref(P), C.c_int(e), C.c_int(out_dim), C.c_int(in_dim),
                                    C.c_int(self.d), C.c_int(self.K), C.c_int(self.r), _ptr(xv),
                                    _ptr(o))
        return o

    def decode_layer(self, x_bits: np.ndarray,
                     down_rows: Optional[Sequence[int]] = None) -> LayerResult:
        x = _c(x_bits, np.uint16)
        T = x.shape[0]
        E, k, S = self.E, self.k, self.S
        rows = None if down_rows is None else np.ascontiguousarray(down_rows, dtype=np.int32)
        n_out = self.H if rows is None else len(rows)
        out = np.empty((T, n_out), np.float64)
        logits = np.empty((T, E), np.float64)
        ids = np.empty((T, k), np.int32)
        w = np.empty((T, k), np.float64)
        counts = np.empty(E, np.int32)
        offsets = np.empty(E + 1, np.int32)
        ptok = np.empty(T * k, np.int32)
        pslot = np.empty(T * k, np.int32)
        ypair = np.empty((T, k + S, n_out), np.float64)
        rc = lib().oracle_decode_layer(C.byref(self._L), _ptr(x), C.c_int(T), _ptr(out),
                                       _ptr(logits), _ptr(ids), _ptr(w), _ptr(counts),
                                       _ptr(offsets), _ptr(ptok), _ptr(pslot), _ptr(ypair),
                                       _ptr(rows), C.c_int(0 if rows is None else len(rows)))
        if rc == 2:
            raise MemoryError("oracle allocation failed")
        return LayerResult(out, logits, ids, w, counts, offsets, ptok, pslot, ypair, rc == 1)


def activation(v, act: str = "silu") -> np.ndarray:
    """The expert activation phi (Section 2.1) applied elementwise."""
    a = np.atleast_1d(np.asarray(v, dtype=np.float64))
    f = lib().oracle_activation
    return np.array([f(float(t), ACTIVATIONS[act]) for t in a.ravel()]).reshape(a.shape)


def read_index(idx: np.ndarray, idx_bytes: int, pos: int) -> int:
    """Index number ``pos`` of a flat index map stored with 1 or 2 bytes per index, or (12) as
    twelve-bit indices packed two to three bytes."""
    a = np.ascontiguousarray(idx)
    f = lib().oracle_read_index
    f.restype = C.c_uint32
    f.argtypes = [C.c_void_p, C.c_int, C.c_size_t]
    return int(f(a.ctypes.data_as(C.c_void_p), idx_bytes, pos))


def topk_affinity(logits: np.ndarray, k: int, renorm: bool = True):
    l = _c(logits, np.float64)
    T, E = l.shape
    ids = np.empty((T, k), np.int32)
    w = np.empty((T, k), np.float64)
    lib().oracle_topk_affinity(_ptr(l), C.c_int(T), C.c_int(E), C.c_int(k),
                               C.c_int(1 if renorm else 0), _ptr(ids), _ptr(w))
    return ids, w


def group_by_expert(ids: np.ndarray, E: int):
    ids = _c(ids, np.int32)
    T, k = ids.shape
    counts = np.empty(E, np.int32)
    offsets = np.empty(E + 1, np.int32)
    ptok = np.empty(T * k, np.int32)
    pslot = np.empty(T * k, np.int32)
    lib().oracle_group_by_expert(_ptr(ids), C.c_int(T), C.c_int(k), C.c_int(E), _ptr(counts),
                                 _ptr(offsets), _ptr(ptok), _ptr(pslot))
    return counts, offsets, ptok, pslot


def storage_bits_per_weight(d, K, r, H, I, E, b_J=8, b_C=16, b_B=16, b_D=16) -> float:
    return float(lib().oracle_storage_bits_per_weight(d, K, r, H, I, E, b_J, b_C, b_B, b_D))


def work_counts(H, I, d, K, r, b_J=8) -> dict:
    out = np.empty(9, np.float64)
    lib().oracle_work_counts(C.c_int(H), C.c_int(I), C.c_int(d), C.c_int(K), C.c_int(r),
                             C.c_int(b_J), _ptr(out))
    names = ["shared_codebook_macs", "shared_basis_macs", "shared_codebook_bits",
             "shared_basis_bits", "private_index_bits", "private_coeff_bits",
             "private_selections", "private_vq_adds", "private_lowrank_macs"]
    return dict(zip(names, out.tolist()))


def threads() -> int:
    return int(lib().oracle_threads())


def set_threads(n: int) -> None:
    lib().oracle_set_threads(C.c_int(n))
