// Hard assignment q(w) = argmin_c ||w - c|| (Section 3.1: what the soft quantiser r_tau tends to as tau -> 0): the
// codes and the dequantised weights one ships after training.  One pass over W; the codebook sits in shared memory.
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include "../../include/idkm.h"

namespace {

constexpr int ASSIGN_BLOCK = 256;
constexpr int ASSIGN_MAX_K = 256;

// A thread takes the 8 / BITS consecutive weights whose codes share one byte (one weight for 8-bit codes), so every
// byte of the output is written by exactly one thread, whole.
template <int D, int BITS>
__global__ void __launch_bounds__(ASSIGN_BLOCK) idkm_assign_kernel(const float* __restrict__ W, long long m,
                                                                   const float* __restrict__ C, int k,
                                                                   unsigned char* __restrict__ codes,
                                                                   float* __restrict__ Wq) {
  constexpr int NW = 8 / BITS;
  __shared__ __align__(16) float cs[ASSIGN_MAX_K * D];
  for (int o = threadIdx.x; o < k * D; o += ASSIGN_BLOCK) cs[o] = C[o];
  __syncthreads();
  const long long n_bytes = (m * BITS + 7) / 8;
  for (long long byte = (long long)blockIdx.x * ASSIGN_BLOCK + threadIdx.x; byte < n_bytes;
       byte += (long long)gridDim.x * ASSIGN_BLOCK) {
    const long long i0 = byte * NW;
    float w[NW][D];
#pragma unroll
    for (int q = 0; q < NW; ++q)
#pragma unroll
      for (int a = 0; a < D; ++a) w[q][a] = (i0 + q < m) ? __ldg(W + (i0 + q) * D + a) : 0.f;
    float bd[NW];
    int bj[NW];
#pragma unroll
    for (int q = 0; q < NW; ++q) {
      bd[q] = 3.0e38f;
      bj[q] = 0;
    }
    for (int j = 0; j < k; ++j) {
      float c[D];
#pragma unroll
      for (int a = 0; a < D; ++a) c[a] = cs[j * D + a];
#pragma unroll
      for (int q = 0; q < NW; ++q) {
        float sq = 0.f;
#pragma unroll
        for (int a = 0; a < D; ++a) {
          const float df = w[q][a] - c[a];
          sq = fmaf(df, df, sq);
        }
        if (sq < bd[q]) {   // strict: ties keep the lower index
          bd[q] = sq;
          bj[q] = j;
        }
      }
    }
    if (codes != nullptr) {
      unsigned int v = 0u;
#pragma unroll
      for (int q = 0; q < NW; ++q)
        if (i0 + q < m) v |= (unsigned int)bj[q] << (q * BITS);
      codes[byte] = (unsigned char)v;
    }
    if (Wq != nullptr) {
#pragma unroll
      for (int q = 0; q < NW; ++q)
        if (i0 + q < m)
#pragma unroll
          for (int a = 0; a < D; ++a) Wq[(i0 + q) * D + a] = cs[bj[q] * D + a];
    }
  }
}

int code_bits(int k) { return k <= 2 ? 1 : (k <= 4 ? 2 : (k <= 16 ? 4 : 8)); }

template <int D>
cudaError_t launch_assign(int bits, int grid, cudaStream_t st, const float* W, long long m, const float* C, int k,
                          unsigned char* codes, float* Wq) {
  switch (bits) {
    case 1: idkm_assign_kernel<D, 1><<<grid, ASSIGN_BLOCK, 0, st>>>(W, m, C, k, codes, Wq); break;
    case 2: idkm_assign_kernel<D, 2><<<grid, ASSIGN_BLOCK, 0, st>>>(W, m, C, k, codes, Wq); break;
    case 4: idkm_assign_kernel<D, 4><<<grid, ASSIGN_BLOCK, 0, st>>>(W, m, C, k, codes, Wq); break;
    default: idkm_assign_kernel<D, 8><<<grid, ASSIGN_BLOCK, 0, st>>>(W, m, C, k, codes, Wq); break;
  }
  return cudaGetLastError();
}

}  // namespace

extern "C" int idkm_code_bits(int k) { return (k >= 1 && k <= ASSIGN_MAX_K) ? code_bits(k) : 0; }

extern "C" size_t idkm_codes_bytes(int64_t m, int k) {
  if (m < 1 || k < 1 || k > ASSIGN_MAX_K) return 0;
  return (size_t)((m * code_bits(k) + 7) / 8);
}

extern "C" int idkm_assign(const float* W, int64_t m, int d, const float* C, int k, unsigned char* codes_out,
                           float* Wq_out, void* cuda_stream) {
  if (!W || !C || (!codes_out && !Wq_out)) return IDKM_ERR_NULL;
  if (!(d == 1 || d == 2 || d == 4) || k < 1 || k > ASSIGN_MAX_K) return IDKM_ERR_UNSUPPORTED;
  if (m < 1) return IDKM_ERR_SHAPE;
  if (Wq_out == W) return IDKM_ERR_PARAM;
  const int bits = code_bits(k);
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
    return IDKM_ERR_CUDA;
  const long long n_bytes = ((long long)m * bits + 7) / 8;
  long long grid = (n_bytes + ASSIGN_BLOCK - 1) / ASSIGN_BLOCK;
  if (grid > (long long)sms * 8) grid = (long long)sms * 8;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  cudaError_t rc;
  if (d == 1) rc = launch_assign<1>(bits, (int)grid, st, W, m, C, k, codes_out, Wq_out);
  else if (d == 2) rc = launch_assign<2>(bits, (int)grid, st, W, m, C, k, codes_out, Wq_out);
  else rc = launch_assign<4>(bits, (int)grid, st, W, m, C, k, codes_out, Wq_out);
  return rc == cudaSuccess ? IDKM_OK : IDKM_ERR_CUDA;
}
