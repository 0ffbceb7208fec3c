// Instantiations of the single-launch forward loop for batched or large small-codebook layers (idkm_step_loop).
#include "idkm_inst.cuh"

namespace idkm {

template <int D, int KPL, int LPW, int KPLQ, int LPWQ>
static cudaError_t launch_loop(const LoopParams& lp, int grid, cudaStream_t stream) {
  constexpr int DYN = LoopCfg<D, KPL, LPW, KPLQ, LPWQ>::DYN_SMEM;
  static bool configured = false;
  if (!configured) {
    const cudaError_t rc = cudaFuncSetAttribute(idkm_step_loop<D, KPL, LPW, KPLQ, LPWQ>,
                                                cudaFuncAttributeMaxDynamicSharedMemorySize, DYN > 0 ? DYN : 1);
    if (rc != cudaSuccess) return rc;
    configured = true;
  }
  void* args[1] = {const_cast<LoopParams*>(&lp)};
  // cooperative launch: refused (instead of hanging at the first barrier) if the grid cannot be co-resident
  return cudaLaunchCooperativeKernel((const void*)&idkm_step_loop<D, KPL, LPW, KPLQ, LPWQ>, dim3((unsigned)grid, 1, 1),
                                     dim3(BLOCK, 1, 1), args, (size_t)DYN, stream);
}
#define IDKM_LOOP_ENTRY(D, KPL, LPW, KPLQ, LPWQ)                                                              \
  {                                                                                                          \
    &launch_loop<D, KPL, LPW, KPLQ, LPWQ>, (const void*)&idkm_step_loop<D, KPL, LPW, KPLQ, LPWQ>,            \
        LoopCfg<D, KPL, LPW, KPLQ, LPWQ>::DYN_SMEM                                                           \
  }
// [d index][codebook class: k <= 2, 4, 8, 16]: the layouts the fp32 step and the increment-form step pick for that k
// (16 centroids: one thread at d = 1, lane pairs with 8 each at d >= 2; the increment form always uses lane pairs)
extern const LoopEntry k_table_step_loop[3][4] = {
    {IDKM_LOOP_ENTRY(1, 2, 1, 2, 1), IDKM_LOOP_ENTRY(1, 4, 1, 4, 1), IDKM_LOOP_ENTRY(1, 8, 1, 8, 1), IDKM_LOOP_ENTRY(1, 16, 1, 8, 2)},
    {IDKM_LOOP_ENTRY(2, 2, 1, 2, 1), IDKM_LOOP_ENTRY(2, 4, 1, 4, 1), IDKM_LOOP_ENTRY(2, 8, 1, 8, 1), IDKM_LOOP_ENTRY(2, 8, 2, 8, 2)},
    {IDKM_LOOP_ENTRY(4, 2, 1, 2, 1), IDKM_LOOP_ENTRY(4, 4, 1, 4, 1), IDKM_LOOP_ENTRY(4, 8, 1, 8, 1), IDKM_LOOP_ENTRY(4, 8, 2, 8, 2)}};

}  // namespace idkm
