// Run-time compilation of the hot kernels for ONE layer shape: the three kernels of a single-token
// call, and the gate/up, down and weighted-sum kernels of the chain that serves several tokens.
//
// At batch 1 every block of the router -> expert -> weighted-sum path runs most of its code once,
// so the path costs what its instruction stream costs: the generic kernels carry every shape,
// index width, code-book layout and token count behind run-time branches, and a copy compiled
// with this layer's integers as constants (hidden and intermediate size, expert count, top-k,
// rank, code-book size, slice plan, ring depths) is about half the size and measurably faster.
// The paper's system also compiles one mapping per model (Section 4); this is that step on a GPU.
//
// The copy is the SAME source (fused_kernel.cuh and what it includes, read from the directory this
// library was loaded from; a static_assert on the sizes of the argument structures refuses files
// that no longer match the library) given to NVRTC with -DMOE_VQLR_JIT and one -DJ_* per constant, the
// result loaded through the runtime's library API and launched like any other kernel.  NVRTC is
// opened with dlopen at the first create() that wants it (from the place moe_vqlr_set_jit_toolkit
// names, else from the CUDA toolkit under /usr/local/cuda); without it, or when anything on the way
// fails, the handle keeps the precompiled kernels (moe_vqlr_specialized() tells how many were compiled,
// moe_vqlr_specialization_note() why not).  Compiled kernels are cached per process, device and option
// string: the layers of a model share one compilation.
#pragma once
#include <dlfcn.h>
#include <nvrtc.h>      // types only: the library itself is opened at run time

#include <cstdio>
#include <cstdlib>
#include <map>
#include <mutex>
#include <string>
#include <vector>

namespace {

struct NvrtcApi {
  bool tried = false, ok = false;
  std::string why;
  decltype(&nvrtcCreateProgram) create_program = nullptr;
  decltype(&nvrtcCompileProgram) compile_program = nullptr;
  decltype(&nvrtcDestroyProgram) destroy_program = nullptr;
  decltype(&nvrtcGetCUBINSize) get_cubin_size = nullptr;
  decltype(&nvrtcGetCUBIN) get_cubin = nullptr;
  decltype(&nvrtcGetProgramLogSize) get_log_size = nullptr;
  decltype(&nvrtcGetProgramLog) get_log = nullptr;
  decltype(&nvrtcGetErrorString) error_string = nullptr;
  std::string cuda_include;      // directory that holds cuda_bf16.h
  std::string src_dir, api_include;
};

std::mutex g_jit_mu;
NvrtcApi g_nvrtc;
std::string g_jit_nvrtc_path, g_jit_include_dir;      // moe_vqlr_set_jit_toolkit: tried before the standard places
std::map<std::string, cudaLibrary_t> g_jit_cache;     // "<device>|<options>" -> loaded library (never unloaded)

bool file_exists(const std::string& p) {
  FILE* f = fopen(p.c_str(), "rb");
  if (!f) return false;
  fclose(f);
  return true;
}

// Called with g_jit_mu held.
void nvrtc_open() {
  NvrtcApi& a = g_nvrtc;
  if (a.tried) return;
  a.tried = true;
  // the kernel sources sit beside this library, the public header two directories up
  Dl_info info;
  if (!dladdr(reinterpret_cast<const void*>(&nvrtc_open), &info) || !info.dli_fname) { a.why = "cannot locate the library file"; return; }
  std::string self = info.dli_fname;
  const size_t slash = self.find_last_of('/');
  a.src_dir = slash == std::string::npos ? std::string(".") : self.substr(0, slash);
  a.api_include = a.src_dir + "/../../include";
  if (!file_exists(a.src_dir + "/fused_kernel.cuh") || !file_exists(a.api_include + "/moe_vqlr.h")) {
    a.why = "kernel sources not found beside the library (" + a.src_dir + ")";
    return;
  }
  const char* roots[] = {"/usr/local/cuda", "/usr/local/cuda-12.9", "/usr/local/cuda-12", "/opt/cuda"};
  void* so = nullptr;
  if (!g_jit_include_dir.empty() && file_exists(g_jit_include_dir + "/cuda_bf16.h")) a.cuda_include = g_jit_include_dir;
  if (!g_jit_nvrtc_path.empty()) so = dlopen(g_jit_nvrtc_path.c_str(), RTLD_NOW | RTLD_LOCAL);
  for (const char* r : roots) {
    if (a.cuda_include.empty() && file_exists(std::string(r) + "/include/cuda_bf16.h")) a.cuda_include = std::string(r) + "/include";
    if (!so) so = dlopen((std::string(r) + "/lib64/libnvrtc.so.12").c_str(), RTLD_NOW | RTLD_LOCAL);
  }
  if (!so) so = dlopen("libnvrtc.so.12", RTLD_NOW | RTLD_LOCAL);
  if (!so) so = dlopen("libnvrtc.so", RTLD_NOW | RTLD_LOCAL);
  if (!so) { a.why = "libnvrtc not found"; return; }
  if (a.cuda_include.empty()) { a.why = "CUDA headers (cuda_bf16.h) not found"; return; }
#define MOE_VQLR_NVRTC_SYM(field, name) \
  a.field = reinterpret_cast<decltype(a.field)>(dlsym(so, name)); \
  if (!a.field) { a.why = std::string("libnvrtc lacks ") + name; return; }
  MOE_VQLR_NVRTC_SYM(create_program, "nvrtcCreateProgram")
  MOE_VQLR_NVRTC_SYM(compile_program, "nvrtcCompileProgram")
  MOE_VQLR_NVRTC_SYM(destroy_program, "nvrtcDestroyProgram")
  MOE_VQLR_NVRTC_SYM(get_cubin_size, "nvrtcGetCUBINSize")
  MOE_VQLR_NVRTC_SYM(get_cubin, "nvrtcGetCUBIN")
  MOE_VQLR_NVRTC_SYM(get_log_size, "nvrtcGetProgramLogSize")
  MOE_VQLR_NVRTC_SYM(get_log, "nvrtcGetProgramLog")
  MOE_VQLR_NVRTC_SYM(error_string, "nvrtcGetErrorString")
#undef MOE_VQLR_NVRTC_SYM
  a.ok = true;
}

// The translation unit NVRTC sees: the library's own kernel source plus one extern "C" entry per
// specialised kernel (J_* come from the option list).
const char kJitSource[] =
    "#define MOE_VQLR_JIT 1\n"
    "#include \"fused_kernel.cuh\"\n"
    "static_assert(sizeof(Params) == J_SZ_PARAMS && sizeof(StagePlan) == J_SZ_PLAN && sizeof(FusedPlan) == J_SZ_FPLAN,\n"
    "              \"the kernel sources beside the library are not the ones it was built from\");\n"
    "extern \"C\" __global__ void __launch_bounds__(32 * kRouterWarps)\n"
    "k_router_z_jit(const Params P, const bf16* __restrict__ x, int T) { router_z_pdl_body<true>(P, x, T); }\n"
    "extern \"C\" __global__ void __launch_bounds__(32 * J_WARPS, 1)\n"
    "k_expert_fused_jit(const Params P, const bf16* __restrict__ x, int T, const StagePlan pg, const FusedPlan fp,\n"
    "                   int n_books, int want_dbg, const J_IDXT* __restrict__ idx_dp) {\n"
    "  expert_fused_body<J_IDXT, J_DENSE, J_JD, J_D4, J_SP, true>(P, x, T, pg, fp, n_books, want_dbg, idx_dp);\n"
    "}\n"
    "extern \"C\" __global__ void __launch_bounds__(kCfThreads)\n"
    "k_combine_fused_jit(const Params P, bf16* __restrict__ out, int T, int n_sl, int lr) {\n"
    "  combine_fused_body<true>(P, out, T, n_sl, lr);\n"
    "}\n";

// The chain of kernels for calls of several tokens, compiled for one layer shape: the same constants
// (the token count stays an argument), plus the two work plans of the gate/up and down kernels.
// Only the three kernels that gain from it: the router and the activation kernel measured SLOWER as
// per-shape copies at 4-16 tokens (router 4.4 -> 5.6 us, activation + z_d 5.6 -> 7.2 us on the Qwen3
// shape at batch 16: with constant trip counts the compiler unrolls their loops into long straight-line
// code, which is exactly what a kernel that runs once per call should not be).
const char kJitChainSource[] =
    "#define MOE_VQLR_JIT 1\n"
    "#define MOE_VQLR_JIT_CHAIN 1\n"
    "#include \"fast_kernels.cuh\"\n"
    "static_assert(sizeof(Params) == J_SZ_PARAMS && sizeof(StagePlan) == J_SZ_PLAN,\n"
    "              \"the kernel sources beside the library are not the ones it was built from\");\n"
    "extern \"C\" __global__ void __launch_bounds__(J_GU_DENSE ? kDenseThreads : kFastThreads, 1)\n"
    "k_gateup_mma_jit(const Params P, const bf16* __restrict__ x, int T, const StagePlan pl, int n_books, int want_dbg) {\n"
    "  gateup_mma_body<J_GU_IDXT, J_GU_DENSE, J_GU_D4, J_LRF, J_SP>(P, x, T, pl, n_books, want_dbg);\n"
    "}\n"
    "extern \"C\" __global__ void __launch_bounds__(kDownThreads, 1)\n"
    "k_down_mma_jit(const Params P, int T, const StagePlan pl) {\n"
    "  down_mma_body<J_DN_IDXT, J_DN_DENSE, J_DN_D4, J_DN_TPUT, J_SP>(P, T, pl);\n"
    "}\n"
    "extern \"C\" __global__ void __launch_bounds__(kCombineCols * kCombineSlots)\n"
    "k_combine_jit(const Params P, bf16* __restrict__ out, int T, int n_parts) { combine_body(P, out, T, n_parts); }\n";

// NVRTC has no host headers; the public header asks for <stdint.h>.
const char kJitStdint[] =
    "typedef signed char int8_t; typedef short int16_t; typedef int int32_t; typedef long long int64_t;\n"
    "typedef unsigned char uint8_t; typedef unsigned short uint16_t; typedef unsigned int uint32_t;\n"
    "typedef unsigned long long uint64_t;\n";

// Compiles (or finds) the specialised kernels of `source` (kJitSource or kJitChainSource) for `defs`
// on the current device.  Returns the loaded library, or nullptr with *why set.
cudaLibrary_t jit_library(const char* source, const std::vector<std::string>& defs, std::string* why) {
  std::lock_guard<std::mutex> lock(g_jit_mu);
  nvrtc_open();
  NvrtcApi& a = g_nvrtc;
  if (!a.ok) { *why = a.why; return nullptr; }
  int dev = 0;
  cudaDeviceProp prop;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaGetDeviceProperties(&prop, dev) != cudaSuccess) { *why = "no current device"; cudaGetLastError(); return nullptr; }
  char arch[64];
  snprintf(arch, sizeof arch, "--gpu-architecture=sm_%d%d%s", prop.major, prop.minor, prop.major >= 9 ? "a" : "");
  std::vector<std::string> opts = {arch, "-std=c++17", "-I" + a.src_dir, "-I" + a.api_include, "-I" + a.cuda_include};
  opts.insert(opts.end(), defs.begin(), defs.end());
#ifdef MOE_VQLR_JIT_EXTRA_ENV      // development builds only: extra options for A/B runs of kernel variants
  if (const char* extra = getenv("MOE_VQLR_JIT_EXTRA")) {
    std::string e(extra);
    size_t at = 0;
    while (at < e.size()) {
      size_t sp = e.find(' ', at);
      if (sp == std::string::npos) sp = e.size();
      if (sp > at) opts.push_back(e.substr(at, sp - at));
      at = sp + 1;
    }
  }
#endif
#ifdef MOE_VQLR_TRACE
  opts.push_back("-DMOE_VQLR_TRACE");
#ifdef MOE_VQLR_TRACE_GLOBAL
  opts.push_back("-DMOE_VQLR_TRACE_GLOBAL");
#endif
#endif
  std::string key = std::to_string(dev) + (source == kJitChainSource ? "|chain" : "|single");
  for (const std::string& o : opts) { key += '|'; key += o; }
  auto hit = g_jit_cache.find(key);
  if (hit != g_jit_cache.end()) {
    if (!hit->second) *why = "an earlier compilation of this shape failed";
    return hit->second;
  }
  cudaLibrary_t& slot = g_jit_cache[key];
  slot = nullptr;
  nvrtcProgram prog = nullptr;
  const char* hdr_names[] = {"stdint.h"};
  const char* hdr_src[] = {kJitStdint};
  nvrtcResult r = a.create_program(&prog, source, "moe_vqlr_jit.cu", 1, hdr_src, hdr_names);
  if (r != NVRTC_SUCCESS) { *why = std::string("nvrtcCreateProgram: ") + a.error_string(r); return nullptr; }
  std::vector<const char*> argv;
  for (const std::string& o : opts) argv.push_back(o.c_str());
  r = a.compile_program(prog, (int)argv.size(), argv.data());
  if (r != NVRTC_SUCCESS) {
    size_t n = 0;
    a.get_log_size(prog, &n);
    std::string log(n, '\0');
    if (n) a.get_log(prog, &log[0]);
    *why = std::string("nvrtcCompileProgram: ") + a.error_string(r) + ": " + log.substr(0, 300);
    a.destroy_program(&prog);
    return nullptr;
  }
  size_t n = 0;
  std::vector<char> cubin;
  if (a.get_cubin_size(prog, &n) == NVRTC_SUCCESS && n > 0) { cubin.resize(n); r = a.get_cubin(prog, cubin.data()); }
  a.destroy_program(&prog);
  if (cubin.empty() || r != NVRTC_SUCCESS) { *why = "NVRTC returned no device code"; return nullptr; }
  cudaLibrary_t lib = nullptr;
  const cudaError_t ce = cudaLibraryLoadData(&lib, cubin.data(), nullptr, nullptr, 0, nullptr, nullptr, 0);
  if (ce != cudaSuccess) { *why = std::string("cudaLibraryLoadData: ") + cudaGetErrorString(ce); cudaGetLastError(); return nullptr; }
  slot = lib;
  return lib;
}

}  // namespace
