// moe_vqlr_probe_lookup_rate: measures how many random 16-byte shared-memory reads per clock one
// SM sustains from a K-entry code book (the unit of work the compressed projections are made
// of).  Used by the benchmark to state the lookup-rate bound next to the HBM roofline.
#include "moe_vqlr_bench.h"

#include <cuda_runtime.h>

namespace {

__global__ void k_probe_lookups(int K, int repl, int iters, unsigned long long* clocks, unsigned int* sink) {
  extern __shared__ uint4 tab[];
  const int n = repl ? K * 8 : K;
  for (int i = threadIdx.x; i < n; i += blockDim.x) tab[i] = make_uint4(i, i * 3, i * 5, i * 7);
  __syncthreads();
  unsigned int s = 12345u ^ (threadIdx.x * 2654435761u) ^ (blockIdx.x * 40503u);
  unsigned int acc = 0;
  const unsigned long long t0 = clock64();
  for (int it = 0; it < iters; ++it) {
    unsigned int idx[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      s = s * 1664525u + 1013904223u;
      idx[j] = (s >> 8) % (unsigned int)K;
      if (repl) idx[j] = (idx[j] << 3) | (threadIdx.x & 7);
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const uint4 v = tab[idx[j]];
      acc ^= v.x + v.y + v.z + v.w;
    }
  }
  const unsigned long long t1 = clock64();
  if (threadIdx.x == 0) clocks[blockIdx.x] = t1 - t0;
  sink[blockIdx.x * blockDim.x + threadIdx.x] = acc;
}

}  // namespace

extern "C" int moe_vqlr_probe_lookup_rate(int32_t codebook_size, int32_t replicated, double* lookups_per_clk_per_sm) {
  if (!lookups_per_clk_per_sm || codebook_size < 1) return MOE_VQLR_ERR_INVALID_ARG;
  const size_t smem = (size_t)codebook_size * 16 * (replicated ? 8 : 1);
  int dev = 0, sms = 0, max_smem = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return MOE_VQLR_ERR_CUDA;
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  if (smem > (size_t)max_smem) return MOE_VQLR_ERR_UNSUPPORTED;
  const int threads = 512, iters = 2000;
  unsigned long long* d_clk = nullptr;
  unsigned int* d_sink = nullptr;
  if (cudaMalloc(&d_clk, sizeof(unsigned long long) * sms) != cudaSuccess) return MOE_VQLR_ERR_OOM;
  if (cudaMalloc(&d_sink, sizeof(unsigned int) * sms * threads) != cudaSuccess) { cudaFree(d_clk); return MOE_VQLR_ERR_OOM; }
  cudaFuncSetAttribute(k_probe_lookups, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  int rc = MOE_VQLR_OK;
  unsigned long long* h = new unsigned long long[sms];
  for (int rep = 0; rep < 2; ++rep) k_probe_lookups<<<sms, threads, smem>>>(codebook_size, replicated ? 1 : 0, iters, d_clk, d_sink);
  if (cudaMemcpy(h, d_clk, sizeof(unsigned long long) * sms, cudaMemcpyDeviceToHost) != cudaSuccess) rc = MOE_VQLR_ERR_CUDA;
  if (rc == MOE_VQLR_OK) {
    double avg = 0;
    for (int i = 0; i < sms; ++i) avg += (double)h[i];
    avg /= sms;
    *lookups_per_clk_per_sm = (double)threads * iters * 8 / avg;
  }
  delete[] h;
  cudaFree(d_clk);
  cudaFree(d_sink);
  return rc;
}
