// Register-only micro-benchmarks of the two issue pipes that bound the fused passes: the fp32 FMA pipe and the
// special-function pipe (ex2 / rsqrt / sqrt / rcp).  They give the measured denominators for the rooflines of the
// arithmetic-bound kernels; nothing on the IDKM path calls them.
#include <cuda_runtime.h>
#include <stdint.h>
#include "../../include/idkm.h"

namespace {

constexpr int PIPE_CHAINS = 8;        // independent dependency chains per thread: no chain ever waits on itself
constexpr int PIPE_THREADS = 256;
constexpr int PIPE_BLOCKS_PER_SM = 8; // 64 warps per SM: every scheduler always has an eligible warp
constexpr int PIPE_ITERS = 8192;

__device__ float g_pipe_sink;

__global__ void __launch_bounds__(PIPE_THREADS) pipe_fma(int iters, float a, float b) {
  float x[PIPE_CHAINS];
#pragma unroll
  for (int i = 0; i < PIPE_CHAINS; ++i) x[i] = threadIdx.x * 1e-3f + i;
  for (int it = 0; it < iters; ++it) {
#pragma unroll
    for (int i = 0; i < PIPE_CHAINS; ++i) x[i] = fmaf(x[i], a, b);
  }
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < PIPE_CHAINS; ++i) s += x[i];
  if (s == 123.456f) g_pipe_sink = s;   // never true in practice; keeps the chains alive
}

__global__ void __launch_bounds__(PIPE_THREADS) pipe_ex2(int iters) {
  float x[PIPE_CHAINS];
#pragma unroll
  for (int i = 0; i < PIPE_CHAINS; ++i) x[i] = -(threadIdx.x * 1e-3f + i);
  for (int it = 0; it < iters; ++it) {
#pragma unroll
    for (int i = 0; i < PIPE_CHAINS; ++i) asm volatile("ex2.approx.ftz.f32 %0, %0;" : "+f"(x[i]));
  }
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < PIPE_CHAINS; ++i) s += x[i];
  if (s == 123.456f) g_pipe_sink = s;
}

template <typename L>
int best_of(L launch, cudaStream_t st, float* best_ms) {
  cudaEvent_t e0, e1;
  if (cudaEventCreate(&e0) != cudaSuccess) return IDKM_ERR_CUDA;
  if (cudaEventCreate(&e1) != cudaSuccess) { cudaEventDestroy(e0); return IDKM_ERR_CUDA; }
  int rc = IDKM_OK;
  float best = 3.0e38f;
  for (int r = 0; r < 7 && rc == IDKM_OK; ++r) {   // the first two repetitions warm up and are not scored
    if (cudaEventRecord(e0, st) != cudaSuccess) rc = IDKM_ERR_CUDA;
    launch();
    if (cudaGetLastError() != cudaSuccess) rc = IDKM_ERR_CUDA;
    if (cudaEventRecord(e1, st) != cudaSuccess) rc = IDKM_ERR_CUDA;
    if (rc == IDKM_OK && cudaEventSynchronize(e1) != cudaSuccess) rc = IDKM_ERR_CUDA;
    float ms = 0.f;
    if (rc == IDKM_OK && cudaEventElapsedTime(&ms, e0, e1) != cudaSuccess) rc = IDKM_ERR_CUDA;
    if (rc == IDKM_OK && r >= 2 && ms < best) best = ms;
  }
  cudaEventDestroy(e0);
  cudaEventDestroy(e1);
  *best_ms = best;
  return rc;
}

}  // namespace

extern "C" int idkm_measure_pipe_rates(double* fp32_lane_ops_per_s, double* sfu_lane_ops_per_s, void* cuda_stream) {
  if (fp32_lane_ops_per_s == nullptr || sfu_lane_ops_per_s == nullptr) return IDKM_ERR_NULL;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return IDKM_ERR_CUDA;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) return IDKM_ERR_CUDA;
  const int blocks = sms * PIPE_BLOCKS_PER_SM;
  const double lane_ops = (double)blocks * PIPE_THREADS * (double)PIPE_ITERS * PIPE_CHAINS;
  float ms = 0.f;
  int rc = best_of([&] { pipe_fma<<<blocks, PIPE_THREADS, 0, st>>>(PIPE_ITERS, 0.999f, 0.001f); }, st, &ms);
  if (rc != IDKM_OK) return rc;
  *fp32_lane_ops_per_s = lane_ops / (ms * 1e-3);
  // the special-function pipe is eight times narrower: an eighth of the iterations keeps the launch as short
  rc = best_of([&] { pipe_ex2<<<blocks, PIPE_THREADS, 0, st>>>(PIPE_ITERS / 8); }, st, &ms);
  if (rc != IDKM_OK) return rc;
  *sfu_lane_ops_per_s = lane_ops / 8.0 / (ms * 1e-3);
  return IDKM_OK;
}
