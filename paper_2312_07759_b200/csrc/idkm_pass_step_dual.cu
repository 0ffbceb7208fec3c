// Instantiations of the dual (fp32 + fp64 in one launch) forward step.
#include "idkm_inst.cuh"

namespace idkm {

template <int D, int KPL, bool DELTA>
static cudaError_t launch_dual(const DualParams& dp, int grid, cudaStream_t stream) {
  constexpr int DYN_A = PassCfg<STEP, D, KPL, 1>::DYN_SMEM, DYN_B = DELTA ? DeltaCfg<D, KPL, 1>::DYN_SMEM : 0;
  constexpr int DYN = DYN_A > DYN_B ? DYN_A : DYN_B;   // the two halves use the dynamic region one after the other
  static bool configured = false;
  if (!configured) {
    const cudaError_t rc = cudaFuncSetAttribute(idkm_step_dual<D, KPL, DELTA>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                DYN > 0 ? DYN : 1);
    if (rc != cudaSuccess) return rc;
    configured = true;
  }
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3((unsigned)grid, 1, 1);
  cfg.blockDim = dim3(BLOCK, 1, 1);
  cfg.dynamicSmemBytes = (size_t)DYN;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  static const bool pdl_off = (getenv("IDKM_NO_PDL") != nullptr);
  cfg.attrs = attr;
  cfg.numAttrs = pdl_off ? 0 : 1;
  return cudaLaunchKernelEx(&cfg, idkm_step_dual<D, KPL, DELTA>, dp);
}

#define IDKM_DUAL_ENTRY(D, KPL) { &launch_dual<D, KPL, false>, (const void*)&idkm_step_dual<D, KPL, false>, PassCfg<STEP, D, KPL, 1>::DYN_SMEM }
#define IDKM_DUAL_DELTA_ENTRY(D, KPL)                                                                \
  {                                                                                                  \
    &launch_dual<D, KPL, true>, (const void*)&idkm_step_dual<D, KPL, true>,                          \
        (PassCfg<STEP, D, KPL, 1>::DYN_SMEM > DeltaCfg<D, KPL, 1>::DYN_SMEM ? PassCfg<STEP, D, KPL, 1>::DYN_SMEM \
                                                                             : DeltaCfg<D, KPL, 1>::DYN_SMEM)   \
  }
#define IDKM_DUAL_NONE { nullptr, nullptr, 0 }
// [d index][family 0..1]: (2,1) for d = 1, 2; (4,1) for d = 1
extern const DualEntry k_table_dual[3][2] = {{IDKM_DUAL_ENTRY(1, 2), IDKM_DUAL_ENTRY(1, 4)},
                                             {IDKM_DUAL_ENTRY(2, 2), IDKM_DUAL_NONE},
                                             {IDKM_DUAL_NONE, IDKM_DUAL_NONE}};
// the same with the collapsing layers in the fp32 increment form
extern const DualEntry k_table_dual_delta[3][2] = {{IDKM_DUAL_DELTA_ENTRY(1, 2), IDKM_DUAL_DELTA_ENTRY(1, 4)},
                                                   {IDKM_DUAL_DELTA_ENTRY(2, 2), IDKM_DUAL_NONE},
                                                   {IDKM_DUAL_NONE, IDKM_DUAL_NONE}};

}  // namespace idkm
