"""Thin ctypes binding of the C ABI in ``include/moe_vqlr.h`` and ``include/moe_vqlr_bench.h``: argument marshalling only.

Every step of the layer runs in the CUDA library; there is no Python or CPU fallback.  Importing
this module loads ``csrc/libmoe_vqlr.so`` and raises if it is missing (build it with
``python -m paper_2609_21137_b200.build``).  PyTorch is used for device memory and streams.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import numpy as np
import torch

from . import build as _build

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_CUDA, ERR_OOM, ERR_TIMEOUT, ERR_BAD_INDEX = range(7)
PROJ_VQLR, PROJ_DENSE_BF16 = 0, 1
FLAG_VALIDATE_INDICES = 1
FLAG_PERSISTENT = 2
FLAG_ACT_GELU_TANH = 4
FLAG_ABLATE_Z_PER_EXPERT = 8
FLAG_ABLATE_PER_EXPERT_LAUNCH = 16
FLAG_TEST_BARRIER_TIMEOUT = 32
FLAG_NO_FUSED = 64
FLAG_FORCE_FUSED = 128
FLAG_GENERIC_KERNELS = 256
FLAG_PROJECTION_CODE_BOOK = 512
FLAG_PHASE_CLOCKS = 1024
FLAG_ACT_RELU2_UP_ONLY = 4096
FLAG_IDX12 = 8192
FLAG_NO_SPECIALIZE = 16384

EXPORTS = ["moe_vqlr_create", "moe_vqlr_decode_layer", "moe_vqlr_decode_layer_host",
           "moe_vqlr_destroy", "moe_vqlr_last_error", "moe_vqlr_last_status", "moe_vqlr_specialized",
           "moe_vqlr_specialization_note", "moe_vqlr_set_jit_toolkit", "moe_vqlr_launch_count",
           "moe_vqlr_workspace_bytes", "moe_vqlr_set_profiling", "moe_vqlr_last_stage_times",
           "moe_vqlr_stage_count", "moe_vqlr_stage_name", "moe_vqlr_route_noalloc",
           "moe_vqlr_run_stage", "moe_vqlr_phase_clocks", "moe_vqlr_probe_lookup_rate"]


class MoeVqlrError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"moe_vqlr status {status}: {message}")
        self.status = status


class _Proj(C.Structure):
    _fields_ = [("kind", C.c_int32), ("reserved", C.c_int32), ("codebook", C.c_void_p),
                ("idx", C.c_void_p), ("basis", C.c_void_p), ("factor", C.c_void_p),
                ("dense", C.c_void_p)]


class _Config(C.Structure):
    _fields_ = [("hidden", C.c_int32), ("inter", C.c_int32), ("n_experts", C.c_int32),
                ("top_k", C.c_int32), ("n_shared", C.c_int32), ("vq_dim", C.c_int32),
                ("codebook_size", C.c_int32), ("rank", C.c_int32), ("max_tokens", C.c_int32),
                ("renorm_topk", C.c_int32), ("flags", C.c_uint32), ("reserved", C.c_int32),
                ("router_w", C.c_void_p), ("router_bias", C.c_void_p),
                ("gate", _Proj), ("up", _Proj), ("down", _Proj)]


class _Debug(C.Structure):
    _fields_ = [("logits", C.c_void_p), ("topk_id", C.c_void_p), ("topk_w", C.c_void_p),
                ("counts", C.c_void_p), ("offsets", C.c_void_p), ("pair_token", C.c_void_p),
                ("pair_slot", C.c_void_p)]


def _load():
    path = _build.LIB_PATH
    if not os.path.exists(path):
        raise ImportError(f"{path} is missing: the CUDA library is not built "
                          "(run `python -m paper_2609_21137_b200.build`); there is no fallback")
    lib = C.CDLL(path)
    lib.moe_vqlr_create.restype = C.c_int
    lib.moe_vqlr_create.argtypes = [C.POINTER(_Config), C.POINTER(C.c_void_p)]
    lib.moe_vqlr_decode_layer.restype = C.c_int
    lib.moe_vqlr_decode_layer.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p,
                                          C.POINTER(_Debug), C.c_void_p]
    lib.moe_vqlr_decode_layer_host.restype = C.c_int
    lib.moe_vqlr_decode_layer_host.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p,
                                               C.c_void_p]
    lib.moe_vqlr_destroy.restype = C.c_int
    lib.moe_vqlr_destroy.argtypes = [C.c_void_p]
    lib.moe_vqlr_last_error.restype = C.c_char_p
    lib.moe_vqlr_last_error.argtypes = [C.c_void_p]
    lib.moe_vqlr_last_status.restype = C.c_int
    lib.moe_vqlr_last_status.argtypes = [C.c_void_p]
    lib.moe_vqlr_specialized.restype = C.c_int
    lib.moe_vqlr_specialized.argtypes = [C.c_void_p]
    lib.moe_vqlr_specialization_note.restype = C.c_char_p
    lib.moe_vqlr_specialization_note.argtypes = [C.c_void_p]
    lib.moe_vqlr_set_jit_toolkit.restype = C.c_int
    lib.moe_vqlr_set_jit_toolkit.argtypes = [C.c_char_p, C.c_char_p]
    lib.moe_vqlr_launch_count.restype = C.c_int64
    lib.moe_vqlr_launch_count.argtypes = [C.c_void_p]
    lib.moe_vqlr_workspace_bytes.restype = C.c_int64
    lib.moe_vqlr_workspace_bytes.argtypes = [C.c_void_p]
    lib.moe_vqlr_set_profiling.restype = C.c_int
    lib.moe_vqlr_set_profiling.argtypes = [C.c_void_p, C.c_int32]
    lib.moe_vqlr_last_stage_times.restype = C.c_int
    lib.moe_vqlr_last_stage_times.argtypes = [C.c_void_p, C.POINTER(C.c_float), C.c_int32]
    lib.moe_vqlr_stage_count.restype = C.c_int
    lib.moe_vqlr_stage_count.argtypes = []
    lib.moe_vqlr_stage_name.restype = C.c_char_p
    lib.moe_vqlr_stage_name.argtypes = [C.c_int32]
    lib.moe_vqlr_run_stage.restype = C.c_int
    lib.moe_vqlr_run_stage.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]
    lib.moe_vqlr_phase_clocks.restype = C.c_int64
    lib.moe_vqlr_phase_clocks.argtypes = [C.c_void_p, C.c_void_p, C.c_int64]
    lib.moe_vqlr_probe_lookup_rate.restype = C.c_int
    lib.moe_vqlr_probe_lookup_rate.argtypes = [C.c_int32, C.c_int32, C.POINTER(C.c_double)]
    lib.moe_vqlr_route_noalloc.restype = C.c_int
    lib.moe_vqlr_route_noalloc.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p] + [C.c_int32] * 5 + \
                                          [C.c_void_p, C.c_void_p, C.c_void_p]
    return lib


_lib = _load()


def pip_toolkit():
    """(libnvrtc path, CUDA include dir) of the nvidia-cuda-nvrtc / nvidia-cuda-runtime packages of this
    Python environment, or (None, None)."""
    try:
        import nvidia
    except ImportError:
        return None, None
    import glob
    for base in list(getattr(nvidia, "__path__", [])):
        libs = sorted(glob.glob(os.path.join(base, "cuda_nvrtc", "lib", "libnvrtc.so.12*")))
        inc = os.path.join(base, "cuda_runtime", "include")
        if libs and os.path.exists(os.path.join(inc, "cuda_bf16.h")):
            return libs[0], inc
    return None, None


def set_jit_toolkit(nvrtc_library: Optional[str], cuda_include_dir: Optional[str]) -> None:
    """Where create() finds NVRTC and the CUDA headers for the per-shape compilation (None: default)."""
    _lib.moe_vqlr_set_jit_toolkit(None if nvrtc_library is None else nvrtc_library.encode(),
                                  None if cuda_include_dir is None else cuda_include_dir.encode())


# No CUDA toolkit in the usual place: point the library at the toolkit pieces of the Python environment.
if not os.path.exists("/usr/local/cuda/include/cuda_bf16.h"):
    _nvrtc, _inc = pip_toolkit()
    if _nvrtc:
        set_jit_toolkit(_nvrtc, _inc)


def library():
    return _lib


def bits_to_device(a: Optional[np.ndarray], device) -> Optional[torch.Tensor]:
    """numpy array (bf16 bit patterns as uint16, uint8/uint16 indices, float32) -> device tensor
    holding the same bytes."""
    if a is None:
        return None
    a = np.ascontiguousarray(a)
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).to(device)
    return torch.from_numpy(a).to(device)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def probe_lookup_rate(codebook_size: int, replicated: bool = False) -> float:
    """Random 16-byte shared-memory lookups per clock per SM on the current device (measured)."""
    out = C.c_double()
    rc = _lib.moe_vqlr_probe_lookup_rate(codebook_size, 1 if replicated else 0, C.byref(out))
    if rc != OK:
        raise MoeVqlrError(rc, "lookup-rate probe failed")
    return float(out.value)


def route_noalloc(x: torch.Tensor, router_w: torch.Tensor, router_bias: Optional[torch.Tensor],
                  k: int, topk_id: torch.Tensor, topk_w: torch.Tensor, renorm_topk: bool = True,
                  stream: Optional[torch.cuda.Stream] = None) -> int:
    """Routing only, for callers that must not allocate on the device: the library keeps the
    logits in a fixed array of its own and makes no allocation.  The caller supplies the output
    tensors (topk_id [T][k] int32, topk_w [T][k] float32).  Limits: T <= 16, E <= 1024, k <= 32;
    calls on one device must not overlap.  Returns the status code (no exception), so that the
    caller can test the limits."""
    T, H = x.shape
    E = router_w.shape[0]
    st = stream or torch.cuda.current_stream(x.device)
    with torch.cuda.device(x.device):
        return int(_lib.moe_vqlr_route_noalloc(_ptr(x), _ptr(router_w), _ptr(router_bias), T, E, H, k,
                                               1 if renorm_topk else 0, _ptr(topk_id), _ptr(topk_w),
                                               C.c_void_p(st.cuda_stream)))


class MoeVqlrLayer:
    """One layer handle.  Weights are torch tensors on the GPU (any 2-byte dtype for bf16 data,
    uint8 / 2-byte for indices); the handle borrows their storage, this object keeps them alive.

    ``gate``/``up``/``down`` are dicts with keys among codebook, idx, basis, factor, dense.
    """

    def __init__(self, *, H, I, E, k, S=0, d=8, K=0, r=0, max_tokens=16, router_w, router_bias=None,
                 gate=None, up, down, renorm_topk=True, flags=0, act="silu", idx12=False):
        self.H, self.I, self.E, self.k, self.S, self.K, self.r = H, I, E, k, S, K, r
        self.max_tokens = max_tokens
        self._keep = [router_w, router_bias, gate, up, down]
        self.device = router_w.device
        cfg = _Config()
        cfg.hidden, cfg.inter, cfg.n_experts, cfg.top_k, cfg.n_shared = H, I, E, k, S
        cfg.vq_dim, cfg.codebook_size, cfg.rank, cfg.max_tokens = d, K, r, max_tokens
        cfg.renorm_topk = 1 if renorm_topk else 0
        if act not in ("silu", "gelu_tanh", "relu2"):
            raise ValueError(f"unknown expert activation {act!r}")
        cfg.flags = flags | {"silu": 0, "gelu_tanh": FLAG_ACT_GELU_TANH, "relu2": FLAG_ACT_RELU2_UP_ONLY}[act] \
            | (FLAG_IDX12 if idx12 else 0)
        cfg.router_w = router_w.data_ptr()
        cfg.router_bias = None if router_bias is None else router_bias.data_ptr()
        for name, p in (("gate", gate), ("up", up), ("down", down)):
            if p is None:              # up-only experts ("relu2") have no gate projection
                continue
            P = getattr(cfg, name)
            dense = p.get("dense")
            P.kind = PROJ_DENSE_BF16 if dense is not None else PROJ_VQLR
            for key in ("codebook", "idx", "basis", "factor", "dense"):
                t = p.get(key)
                setattr(P, key, None if t is None else t.data_ptr())
        self._cfg = cfg
        handle = C.c_void_p()
        with torch.cuda.device(self.device):
            rc = _lib.moe_vqlr_create(C.byref(cfg), C.byref(handle))
        if rc != OK:
            raise MoeVqlrError(rc, _lib.moe_vqlr_last_error(None).decode())
        self._h = handle

    @classmethod
    def from_synth(cls, layer, device="cuda", max_tokens=None, flags=0, renorm_topk=True):
        """Upload a ``synth.Layer`` (numpy bit patterns) and create a handle on it."""
        s = layer.shape
        cache = {}

        def up(a):
            if a is None:
                return None
            if id(a) not in cache:          # aliased arrays stay aliased on the device
                cache[id(a)] = bits_to_device(a, device)
            return cache[id(a)]

        def proj(p):
            if p is None:
                return None
            return dict(codebook=up(p.codebook), idx=up(p.idx), basis=up(p.basis),
                        factor=up(p.factor), dense=up(p.dense))

        return cls(H=s.H, I=s.I, E=s.E, k=s.k, S=s.S, d=s.d, K=s.K, r=s.r,
                   max_tokens=max_tokens or max(s.T, 1), router_w=up(layer.router_w),
                   router_bias=up(layer.router_bias), gate=proj(layer.gate), up=proj(layer.up),
                   down=proj(layer.down), renorm_topk=renorm_topk,
                   flags=flags | (FLAG_IDX12 if getattr(s, "idx12", False) else 0), act=s.act)

    # -----------------------------------------------------------------------------------
    def _check(self, rc):
        if rc != OK:
            raise MoeVqlrError(rc, _lib.moe_vqlr_last_error(self._h).decode())

    def decode(self, x: torch.Tensor, out: Optional[torch.Tensor] = None, debug: bool = False,
               stream: Optional[torch.cuda.Stream] = None):
        """x: [T][H] 2-byte tensor holding bf16 on the GPU.  Returns out ([T][H] bf16), or
        (out, dict of routing tensors) with ``debug=True``."""
        T = x.shape[0]
        if out is None:
            out = torch.empty((T, self.H), dtype=torch.bfloat16, device=x.device)
        st = stream or torch.cuda.current_stream(x.device)
        dbg = None
        tensors = None
        if debug:
            i32 = dict(dtype=torch.int32, device=x.device)
            tensors = dict(logits=torch.empty((T, self.E), dtype=torch.float32, device=x.device),
                           topk_id=torch.empty((T, self.k), **i32),
                           topk_w=torch.empty((T, self.k), dtype=torch.float32, device=x.device),
                           counts=torch.empty(self.E, **i32), offsets=torch.empty(self.E + 1, **i32),
                           pair_token=torch.empty(T * self.k, **i32),
                           pair_slot=torch.empty(T * self.k, **i32))
            dbg = _Debug(**{k: v.data_ptr() for k, v in tensors.items()})
        self._check(_lib.moe_vqlr_decode_layer(self._h, _ptr(x), T, _ptr(out),
                                               None if dbg is None else C.byref(dbg),
                                               C.c_void_p(st.cuda_stream)))
        return (out, tensors) if debug else out

    def decode_host(self, x_host: torch.Tensor, out_host: torch.Tensor,
                    stream: Optional[torch.cuda.Stream] = None):
        """Host buffers in and out (pinned recommended); returns when the result is in out_host."""
        T = x_host.shape[0]
        st = stream or torch.cuda.current_stream(self.device)
        self._check(_lib.moe_vqlr_decode_layer_host(self._h, _ptr(x_host), T, _ptr(out_host),
                                                    C.c_void_p(st.cuda_stream)))
        return out_host

    def run_stage(self, stage: str, x: torch.Tensor, out: torch.Tensor,
                  stream: Optional[torch.cuda.Stream] = None) -> None:
        """Enqueue one stage's kernel only (measurement aid; needs an earlier full call)."""
        names = [_lib.moe_vqlr_stage_name(i).decode() for i in range(_lib.moe_vqlr_stage_count())]
        st = stream or torch.cuda.current_stream(x.device)
        self._check(_lib.moe_vqlr_run_stage(self._h, names.index(stage), _ptr(x), x.shape[0], _ptr(out),
                                            C.c_void_p(st.cuda_stream)))

    def phase_clocks(self):
        """Phase stamps of the last call as an int64 array [4][blocks][16][16], or None when the
        handle was not created with FLAG_PHASE_CLOCKS (or the library was built without tracing)."""
        n = int(_lib.moe_vqlr_phase_clocks(self._h, None, 0))
        if n <= 0:
            return None
        buf = np.zeros(n, np.int64)
        got = int(_lib.moe_vqlr_phase_clocks(self._h, buf.ctypes.data_as(C.c_void_p), n))
        return buf.reshape(4, -1, 16, 16) if got == n else None

    def last_status(self) -> int:
        """Status word of the handle (0, or the code a kernel recorded); reading clears it.
        Synchronize the stream of the calls in question first."""
        return int(_lib.moe_vqlr_last_status(self._h))

    def specialized(self) -> int:
        """Number of kernels of the single-token path that create() compiled for this layer's shape."""
        return int(_lib.moe_vqlr_specialized(self._h))

    def specialization_note(self) -> str:
        """Why there are none (empty string if there are)."""
        return _lib.moe_vqlr_specialization_note(self._h).decode()

    def set_profiling(self, on: bool) -> None:
        self._check(_lib.moe_vqlr_set_profiling(self._h, 1 if on else 0))

    def last_stage_times_ms(self) -> dict:
        n = _lib.moe_vqlr_stage_count()
        buf = (C.c_float * n)()
        self._check(_lib.moe_vqlr_last_stage_times(self._h, buf, n))
        return {_lib.moe_vqlr_stage_name(i).decode(): float(buf[i]) for i in range(n)}

    @property
    def launch_count(self) -> int:
        return int(_lib.moe_vqlr_launch_count(self._h))

    @property
    def workspace_bytes(self) -> int:
        return int(_lib.moe_vqlr_workspace_bytes(self._h))

    def close(self):
        if getattr(self, "_h", None):
            _lib.moe_vqlr_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
