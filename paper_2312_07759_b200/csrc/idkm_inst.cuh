// Instantiates every (d, codebook layout) variant of one pass and exports its dispatch table.
// Included by one translation unit per pass so that the units compile in parallel.
#pragma once
#include "idkm_kernels.cuh"

#include <stdlib.h>
#include <string.h>

namespace idkm {

// Launch with programmatic dependent launch: the next kernel of the stream may be scheduled while this one drains
// (it waits in griddepcontrol.wait until this grid has completed and its writes are visible), which hides the launch
// latency between the short dependent kernels of a loop.
template <typename Kernel>
static cudaError_t launch_pdl(Kernel kernel, const PassParams& p, int grid, int dyn_smem, cudaStream_t stream) {
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3((unsigned)grid, 1, 1);
  cfg.blockDim = dim3(BLOCK, 1, 1);
  cfg.dynamicSmemBytes = (size_t)dyn_smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  static const bool pdl_off = (getenv("IDKM_NO_PDL") != nullptr);   // tuning knob: plain stream order
  cfg.attrs = attr;
  cfg.numAttrs = pdl_off ? 0 : 1;
  return cudaLaunchKernelEx(&cfg, kernel, p);
}

template <int MODE, int D, int KPL, int LPW, bool SQ>
static cudaError_t launch_one(const PassParams& p, int grid, cudaStream_t stream) {
  constexpr int DYN = PassCfg<MODE, D, KPL, LPW>::DYN_SMEM;
  static bool configured = false;   // static + dynamic shared memory may exceed the 48 KB default
  if (!configured) {
    const cudaError_t rc = cudaFuncSetAttribute(idkm_pass<MODE, D, KPL, LPW, SQ>,
                                                cudaFuncAttributeMaxDynamicSharedMemorySize, DYN > 0 ? DYN : 1);
    if (rc != cudaSuccess) return rc;
    configured = true;
  }
  return launch_pdl(idkm_pass<MODE, D, KPL, LPW, SQ>, p, grid, DYN, stream);
}

// IDKM_SQ selects which variant a translation unit instantiates: the Euclidean distance of Algorithm 1 (default) or
// the squared distance (the *_sq.cu units define it as true before including this header).
#ifndef IDKM_SQ
#define IDKM_SQ false
#endif
#define IDKM_ENTRY(MODE, D, KPL, LPW)                                                                       \
  {                                                                                                         \
    &launch_one<MODE, D, KPL, LPW, IDKM_SQ>, (const void*)&idkm_pass<MODE, D, KPL, LPW, IDKM_SQ>, KPL, LPW, \
        PassCfg<MODE, D, KPL, LPW>::TILE, PassCfg<MODE, D, KPL, LPW>::PLEN,                                 \
        PassCfg<MODE, D, KPL, LPW>::DYN_SMEM                                                                \
  }

template <int D, int KPL, int LPW>
static cudaError_t launch_precise(const PassParams& p, int grid, cudaStream_t stream) {
  return launch_pdl(idkm_step_precise<D, KPL, LPW>, p, grid, 0, stream);
}
#define IDKM_PRECISE_ENTRY(D, KPL, LPW)                                                           \
  {                                                                                               \
    &launch_precise<D, KPL, LPW>, (const void*)&idkm_step_precise<D, KPL, LPW>, KPL, LPW,         \
        PreciseCfg<D, KPL, LPW>::TILE, PreciseCfg<D, KPL, LPW>::PLEN, 0                           \
  }
// Bulk-copy variant of the forward step (thread-per-weight layouts only; see BULK in idkm_kernels.cuh): the stages
// of the copy pipeline follow the second-level sums in dynamic shared memory.
template <int D, int KPL>
static cudaError_t launch_step_bulk(const PassParams& p, int grid, cudaStream_t stream) {
  using Cfg = PassCfg<STEP, D, KPL, 1>;
  constexpr int DYN = Cfg::DYN_SMEM + BULK_STAGES * Cfg::UNROLL * BLOCK * 16;
  static bool configured = false;
  if (!configured) {
    const cudaError_t rc = cudaFuncSetAttribute(idkm_pass<STEP, D, KPL, 1, false, true>,
                                                cudaFuncAttributeMaxDynamicSharedMemorySize, DYN);
    if (rc != cudaSuccess) return rc;
    configured = true;
  }
  return launch_pdl(idkm_pass<STEP, D, KPL, 1, false, true>, p, grid, DYN, stream);
}
#define IDKM_BULK_ENTRY(D, KPL)                                                                              \
  {                                                                                                          \
    &launch_step_bulk<D, KPL>, (const void*)&idkm_pass<STEP, D, KPL, 1, false, true>, KPL, 1,                \
        PassCfg<STEP, D, KPL, 1>::TILE, PassCfg<STEP, D, KPL, 1>::PLEN,                                      \
        PassCfg<STEP, D, KPL, 1>::DYN_SMEM + BULK_STAGES * PassCfg<STEP, D, KPL, 1>::UNROLL * BLOCK * 16     \
  }
#define IDKM_BULK_ROW(D)                                                                                     \
  {                                                                                                          \
    IDKM_BULK_ENTRY(D, 2), IDKM_BULK_ENTRY(D, 4), IDKM_BULK_ENTRY(D, 8), IDKM_BULK_ENTRY(D, 16),             \
        IDKM_NO_ENTRY, IDKM_NO_ENTRY, IDKM_NO_ENTRY, IDKM_NO_ENTRY, IDKM_NO_ENTRY, IDKM_NO_ENTRY,            \
        IDKM_NO_ENTRY                                                                                        \
  }

#define IDKM_PRECISE_ROW(D)                                                                       \
  {                                                                                               \
    IDKM_PRECISE_ENTRY(D, 2, 1), IDKM_PRECISE_ENTRY(D, 4, 1), IDKM_PRECISE_ENTRY(D, 8, 1),        \
        IDKM_PRECISE_ENTRY(D, 8, 2), IDKM_PRECISE_ENTRY(D, 8, 4), IDKM_PRECISE_ENTRY(D, 8, 8),    \
        IDKM_PRECISE_ENTRY(D, 8, 16), IDKM_PRECISE_ENTRY(D, 8, 32), IDKM_PRECISE_ENTRY(D, 8, 32), \
        IDKM_NO_ENTRY, IDKM_NO_ENTRY                                                              \
  }

template <int D, int KPL>
static cudaError_t launch_jacobian(const PassParams& p, int grid, cudaStream_t stream) {
  return launch_pdl(idkm_jacobian<D, KPL>, p, grid, 0, stream);
}
#define IDKM_JAC_ENTRY(D, KPL)                                                                    \
  {                                                                                               \
    &launch_jacobian<D, KPL>, (const void*)&idkm_jacobian<D, KPL>, KPL, 1, JacCfg<D, KPL>::TILE,  \
        JacCfg<D, KPL>::PLEN, 0                                                                   \
  }
#define IDKM_NO_ENTRY {nullptr, nullptr, 0, 0, 1, 1, 0}

// forward passes keep 16 centroids per lane, backward passes 8 (they also hold F_j and u_j/S_j)
#define IDKM_FWD_ROW(MODE, D)                                                                     \
  {                                                                                               \
    IDKM_ENTRY(MODE, D, 2, 1), IDKM_ENTRY(MODE, D, 4, 1), IDKM_ENTRY(MODE, D, 8, 1),              \
        IDKM_ENTRY(MODE, D, 16, 1), IDKM_ENTRY(MODE, D, 16, 2), IDKM_ENTRY(MODE, D, 16, 4),       \
        IDKM_ENTRY(MODE, D, 16, 8), IDKM_ENTRY(MODE, D, 16, 16), IDKM_ENTRY(MODE, D, 8, 32),      \
        IDKM_ENTRY(MODE, D, 4, 4), IDKM_ENTRY(MODE, D, 8, 2)                                      \
  }
#define IDKM_BWD_ROW(MODE, D)                                                                     \
  {                                                                                               \
    IDKM_ENTRY(MODE, D, 2, 1), IDKM_ENTRY(MODE, D, 4, 1), IDKM_ENTRY(MODE, D, 8, 1),              \
        IDKM_ENTRY(MODE, D, 8, 2), IDKM_ENTRY(MODE, D, 8, 4), IDKM_ENTRY(MODE, D, 8, 8),          \
        IDKM_ENTRY(MODE, D, 8, 16), IDKM_ENTRY(MODE, D, 8, 32), IDKM_ENTRY(MODE, D, 8, 32),       \
        IDKM_ENTRY(MODE, D, 4, 4), IDKM_ENTRY(MODE, D, 8, 2)                                      \
  }
// The adjoint step's last entry is the half-warp layout with 16 centroids per lane (one block of 8 warps per SM,
// 254 registers): half the per-row overhead and one shuffle stage fewer per pair than 8 centroids on a full warp, and
// the registers keep w - c_j from the distance to the accumulation.
#define IDKM_ADJ_ROW(D)                                                                           \
  {                                                                                               \
    IDKM_ENTRY(ADJ, D, 2, 1), IDKM_ENTRY(ADJ, D, 4, 1), IDKM_ENTRY(ADJ, D, 8, 1),                 \
        IDKM_ENTRY(ADJ, D, 8, 2), IDKM_ENTRY(ADJ, D, 8, 4), IDKM_ENTRY(ADJ, D, 8, 8),             \
        IDKM_ENTRY(ADJ, D, 8, 16), IDKM_ENTRY(ADJ, D, 8, 32), IDKM_ENTRY(ADJ, D, 16, 16),         \
        IDKM_ENTRY(ADJ, D, 4, 4), IDKM_ENTRY(ADJ, D, 8, 2)                                        \
  }

}  // namespace idkm
