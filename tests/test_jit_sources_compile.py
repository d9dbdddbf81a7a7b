"""The translation units that moe_vqlr_create() hands to NVRTC (the kernels compiled for one layer
shape) must compile for sm_100a.  NVRTC needs no GPU, so this runs with the CPU tests: it takes the
two source strings out of csrc/jit_host.cuh and compiles them with the constants of the Qwen3-shaped
layer, which catches a broken MOE_VQLR_JIT section before any GPU run does."""
import ctypes as C
import glob
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CSRC = os.path.join(ROOT, "paper_2609_21137_b200", "csrc")
CUDA_ROOTS = ["/usr/local/cuda", "/usr/local/cuda-12.9", "/usr/local/cuda-12", "/opt/cuda"]


def _nvrtc():
    for r in CUDA_ROOTS:
        for p in sorted(glob.glob(r + "/lib64/libnvrtc.so.12*")):
            try:
                return C.CDLL(p), r + "/include"
            except OSError:
                pass
    return None, None


def _c_string(name: str) -> str:
    """The value of `const char <name>[] = "..." "..." ;` in jit_host.cuh."""
    text = open(os.path.join(CSRC, "jit_host.cuh")).read()
    body = text[text.index(f"const char {name}[] ="):]
    body = body[:body.index(";\n\n")]
    parts = re.findall(r'"((?:[^"\\]|\\.)*)"', body)
    return "".join(parts).encode().decode("unicode_escape")


# the Qwen3-30B-A3B-shaped layer (H 2048, I 768, E 128, k 8, K 4096, r 64), single token / chain plans
BASE = dict(J_H=2048, J_I=768, J_E=128, J_TOPK=8, J_S=0, J_K=4096, J_R=64, J_RENORM=1, J_ACT=0, J_D=8, J_IDX12=0,
            J_ZREPEAT=1, J_NZROWS=128, J_ZSLOT_G=0, J_ZSLOT_U=1, J_NBOOKS=1, J_LR=1, J_SP="false",
            J_SZ_PARAMS="sizeof(Params)", J_SZ_PLAN="sizeof(StagePlan)", J_SZ_FPLAN="sizeof(FusedPlan)")
SINGLE = dict(J_NB=256, J_NSLICES=8, J_NLR=2, J_NPARTS=10, J_REPL=0, J_XSMEM=1, J_TPS=6, J_NSL=16, J_TLAST=6, J_JD=2,
              J_RP_LOG2=6, J_DEPTH_G=3, J_DEPTH_D=16, J_WARPS=16, J_IDXT="uint16_t", J_DENSE="false", J_D4="false")


def _plan(prefix, **kw):
    return {f"J_{prefix}_{k}": v for k, v in kw.items()}


CHAIN = {**_plan("GU", NB=256, NSLICES=8, NLR=2, NPARTS=8, TILES=96, DEPTH=3, CHUNK=16, XSMEM=1, REPL=0, W=2368, TPU=1, TAIL=0),
         **_plan("DN", NB=96, NSLICES=3, NLR=2, NPARTS=3, TILES=64, DEPTH=3, CHUNK=64, XSMEM=0, REPL=0, W=1776, TPU=4, TAIL=0),
         "J_GU_IDXT": "uint16_t", "J_DN_IDXT": "uint16_t", "J_GU_DENSE": "false", "J_DN_DENSE": "false",
         "J_GU_D4": "false", "J_DN_D4": "false", "J_LRF": 1, "J_DN_TPUT": 4}

STDINT = (b"typedef signed char int8_t; typedef short int16_t; typedef int int32_t; typedef long long int64_t;\n"
          b"typedef unsigned char uint8_t; typedef unsigned short uint16_t; typedef unsigned int uint32_t;\n"
          b"typedef unsigned long long uint64_t;\n")


@pytest.mark.parametrize("name,defs,kernels", [
    ("kJitSource", {**BASE, **SINGLE}, ["k_router_z_jit", "k_expert_fused_jit", "k_combine_fused_jit"]),
    ("kJitChainSource", {**BASE, **CHAIN}, ["k_gateup_mma_jit", "k_down_mma_jit", "k_combine_jit"]),
])
def test_run_time_translation_units_compile_for_sm100a(name, defs, kernels):
    lib, cuda_inc = _nvrtc()
    if lib is None or not os.path.exists(os.path.join(cuda_inc, "cuda_bf16.h")):
        pytest.skip("no NVRTC / CUDA headers on this machine")
    src = _c_string(name).encode()
    for k in kernels:
        assert k.encode() in src
    prog = C.c_void_p()
    hdr_src = (C.c_char_p * 1)(STDINT)
    hdr_name = (C.c_char_p * 1)(b"stdint.h")
    lib.nvrtcCreateProgram.argtypes = [C.POINTER(C.c_void_p), C.c_char_p, C.c_char_p, C.c_int,
                                       C.POINTER(C.c_char_p), C.POINTER(C.c_char_p)]
    assert lib.nvrtcCreateProgram(C.byref(prog), src, b"moe_vqlr_jit.cu", 1, hdr_src, hdr_name) == 0
    opts = [b"--gpu-architecture=sm_100a", b"-std=c++17", f"-I{CSRC}".encode(),
            f"-I{os.path.join(ROOT, 'include')}".encode(), f"-I{cuda_inc}".encode()]
    opts += [f"-D{k}={v}".encode() for k, v in defs.items()]
    arr = (C.c_char_p * len(opts))(*opts)
    lib.nvrtcCompileProgram.argtypes = [C.c_void_p, C.c_int, C.POINTER(C.c_char_p)]
    rc = lib.nvrtcCompileProgram(prog, len(opts), arr)
    n = C.c_size_t()
    lib.nvrtcGetProgramLogSize.argtypes = [C.c_void_p, C.POINTER(C.c_size_t)]
    lib.nvrtcGetProgramLogSize(prog, C.byref(n))
    log = C.create_string_buffer(n.value or 1)
    lib.nvrtcGetProgramLog.argtypes = [C.c_void_p, C.c_char_p]
    lib.nvrtcGetProgramLog(prog, log)
    assert rc == 0, log.value.decode(errors="replace")[:2000]
    size = C.c_size_t()
    lib.nvrtcGetCUBINSize.argtypes = [C.c_void_p, C.POINTER(C.c_size_t)]
    assert lib.nvrtcGetCUBINSize(prog, C.byref(size)) == 0 and size.value > 10000
    lib.nvrtcDestroyProgram.argtypes = [C.POINTER(C.c_void_p)]
    lib.nvrtcDestroyProgram(C.byref(prog))
