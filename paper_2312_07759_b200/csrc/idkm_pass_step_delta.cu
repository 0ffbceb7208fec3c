// fp32 increment-form forward step for collapsing layers (delta_body): one instantiation per codebook layout.
#include "idkm_inst.cuh"
namespace idkm {

template <int D, int KPL, int LPW>
static cudaError_t launch_delta(const PassParams& p, int grid, cudaStream_t stream) {
  constexpr int DYN = DeltaCfg<D, KPL, LPW>::DYN_SMEM;
  static bool configured = false;   // static + dynamic shared memory may exceed the 48 KB default
  if (!configured) {
    const cudaError_t rc = cudaFuncSetAttribute(idkm_step_delta<D, KPL, LPW>, cudaFuncAttributeMaxDynamicSharedMemorySize, DYN);
    if (rc != cudaSuccess) return rc;
    configured = true;
  }
  return launch_pdl(idkm_step_delta<D, KPL, LPW>, p, grid, DYN, stream);
}
#define IDKM_DELTA_ENTRY(D, KPL, LPW)                                                             \
  {                                                                                               \
    &launch_delta<D, KPL, LPW>, (const void*)&idkm_step_delta<D, KPL, LPW>, KPL, LPW,             \
        DeltaCfg<D, KPL, LPW>::TILE, DeltaCfg<D, KPL, LPW>::PLEN, DeltaCfg<D, KPL, LPW>::DYN_SMEM \
  }
#define IDKM_DELTA_ROW(D)                                                                         \
  {                                                                                               \
    IDKM_DELTA_ENTRY(D, 2, 1), IDKM_DELTA_ENTRY(D, 4, 1), IDKM_DELTA_ENTRY(D, 8, 1),              \
        IDKM_DELTA_ENTRY(D, 8, 2), IDKM_DELTA_ENTRY(D, 8, 4), IDKM_DELTA_ENTRY(D, 8, 8),          \
        IDKM_DELTA_ENTRY(D, 8, 16), IDKM_DELTA_ENTRY(D, 8, 32), IDKM_DELTA_ENTRY(D, 8, 32),       \
        IDKM_NO_ENTRY, IDKM_NO_ENTRY                                                              \
  }
extern const KernelEntry k_table_step_delta[3][N_FAMILY] = {IDKM_DELTA_ROW(1), IDKM_DELTA_ROW(2), IDKM_DELTA_ROW(4)};
}
