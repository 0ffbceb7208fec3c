// Hard assignment q(w) = argmin_c ||w - c|| (Section 3.1: what the soft quantiser r_tau tends to as tau -> 0): the
// codes and the dequantised weights one ships after training.  One pass over W; the codebook sits in shared memory.
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include "../../include/idkm.h"

namespace {

constexpr int ASSIGN_BLOCK = 256;
constexpr int ASSIGN_MAX_K = 256;

// A lane takes 4 / d consecutive weights per trip -- one 128-bit load, consecutive lanes on consecutive rows -- and
// packs their codes; where that is less than a byte the lanes that share the byte combine by shuffles and the first of
// them writes it, otherwise the lane writes its own bytes.  Every byte is written once, whole.
template <int D, int BITS>
__global__ void __launch_bounds__(ASSIGN_BLOCK) idkm_assign_kernel(const float* __restrict__ W, long long m,
                                                                   const float* __restrict__ C, int k,
                                                                   unsigned char* __restrict__ codes,
                                                                   float* __restrict__ Wq) {
  constexpr int VEC = 4 / D;                        // weights per lane per trip
  constexpr int LBITS = VEC * BITS;                 // code bits a lane produces per trip
  constexpr int NL = LBITS < 8 ? 8 / LBITS : 1;     // lanes that share one byte
  constexpr int NB = LBITS < 8 ? 1 : LBITS / 8;     // bytes a lane (or lane group) writes per trip
  __shared__ __align__(16) float cs[ASSIGN_MAX_K * D];
  for (int o = threadIdx.x; o < k * D; o += ASSIGN_BLOCK) cs[o] = C[o];
  __syncthreads();
  const int lane = threadIdx.x & 31;
  const long long groups = (m + VEC - 1) / VEC;             // 128-bit groups of rows
  const long long groups_up = (groups + 31) / 32 * 32;      // whole warps stay in the loop together (shuffles)
  for (long long g = (long long)blockIdx.x * ASSIGN_BLOCK + threadIdx.x; g < groups_up;
       g += (long long)gridDim.x * ASSIGN_BLOCK) {
    const long long i0 = g * VEC;
    float w[VEC][D];
    if (i0 + VEC <= m) {
      const float4 x = __ldg(reinterpret_cast<const float4*>(W) + g);
      const float xs[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
      for (int v = 0; v < VEC; ++v)
#pragma unroll
        for (int a = 0; a < D; ++a) w[v][a] = xs[v * D + a];
    } else {
#pragma unroll
      for (int v = 0; v < VEC; ++v)
#pragma unroll
        for (int a = 0; a < D; ++a) w[v][a] = (i0 + v < m) ? __ldg(W + (i0 + v) * D + a) : 0.f;
    }
    float bd[VEC];
    int bj[VEC];
#pragma unroll
    for (int v = 0; v < VEC; ++v) {
      bd[v] = 3.0e38f;
      bj[v] = 0;
    }
    for (int j = 0; j < k; ++j) {
      float c[D];
#pragma unroll
      for (int a = 0; a < D; ++a) c[a] = cs[j * D + a];
#pragma unroll
      for (int v = 0; v < VEC; ++v) {
        float sq = 0.f;
#pragma unroll
        for (int a = 0; a < D; ++a) {
          const float df = w[v][a] - c[a];
          sq = fmaf(df, df, sq);
        }
        if (sq < bd[v]) {   // strict: ties keep the lower index
          bd[v] = sq;
          bj[v] = j;
        }
      }
    }
    if (codes != nullptr) {
      unsigned int v32 = 0u;
#pragma unroll
      for (int v = 0; v < VEC; ++v)
        if (i0 + v < m) v32 |= (unsigned int)bj[v] << (v * BITS);
      if constexpr (NL > 1) {
        v32 <<= (lane % NL) * LBITS;
#pragma unroll
        for (int o = 1; o < NL; o <<= 1) v32 |= __shfl_xor_sync(0xffffffffu, v32, o);
        if ((lane % NL) == 0 && i0 < m) codes[g / NL] = (unsigned char)v32;
      } else {
        const long long n_bytes = (m * BITS + 7) / 8;
#pragma unroll
        for (int q = 0; q < NB; ++q)
          if (g * NB + q < n_bytes) codes[g * NB + q] = (unsigned char)(v32 >> (8 * q));
      }
    }
    if (Wq != nullptr) {
      if (i0 + VEC <= m) {
        float os[4];
#pragma unroll
        for (int v = 0; v < VEC; ++v)
#pragma unroll
          for (int a = 0; a < D; ++a) os[v * D + a] = cs[bj[v] * D + a];
        reinterpret_cast<float4*>(Wq)[g] = make_float4(os[0], os[1], os[2], os[3]);
      } else {
#pragma unroll
        for (int v = 0; v < VEC; ++v)
          if (i0 + v < m)
#pragma unroll
            for (int a = 0; a < D; ++a) Wq[(i0 + v) * D + a] = cs[bj[v] * D + a];
      }
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
  if (((uintptr_t)W | (uintptr_t)(Wq_out ? Wq_out : W)) & 15u) return IDKM_ERR_ALIGN;   // vector loads and stores
  const int bits = code_bits(k);
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
    return IDKM_ERR_CUDA;
  const long long groups = ((long long)m * d + 3) / 4;   // one 128-bit group of rows per thread and trip
  long long grid = (groups + ASSIGN_BLOCK - 1) / ASSIGN_BLOCK;
  if (grid > (long long)sms * 8) grid = (long long)sms * 8;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  cudaError_t rc;
  if (d == 1) rc = launch_assign<1>(bits, (int)grid, st, W, m, C, k, codes_out, Wq_out);
  else if (d == 2) rc = launch_assign<2>(bits, (int)grid, st, W, m, C, k, codes_out, Wq_out);
  else rc = launch_assign<4>(bits, (int)grid, st, W, m, C, k, codes_out, Wq_out);
  return rc == cudaSuccess ? IDKM_OK : IDKM_ERR_CUDA;
}
