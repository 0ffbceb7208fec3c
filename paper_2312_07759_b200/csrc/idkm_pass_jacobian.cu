#include "idkm_inst.cuh"
#include "idkm_jacobian_tile.cuh"
namespace idkm {

template <int D, int KP>
static cudaError_t launch_jacobian_tile(const PassParams& p, int grid, cudaStream_t stream) {
  return launch_pdl(idkm_jacobian_tile<D, KP>, p, grid, JacTileCfg<D, KP>::DYN_SMEM, stream);
}
#define IDKM_JACT_ENTRY(D, KP)                                                                          \
  {                                                                                                     \
    &launch_jacobian_tile<D, KP>, (const void*)&idkm_jacobian_tile<D, KP>, KP, 1, JacTileCfg<D, KP>::TILE, \
        JacTileCfg<D, KP>::PLEN, JacTileCfg<D, KP>::DYN_SMEM                                            \
  }

// explicit-Jacobian adjoint: k d <= 8 in a thread's registers (families 0-2), 8 < k d <= 64 spread over a block
// (families 3-5: 16, 32, 64 centroids)
extern const KernelEntry k_table_jacobian[3][N_FAMILY] = {
    {IDKM_JAC_ENTRY(1, 2), IDKM_JAC_ENTRY(1, 4), IDKM_JAC_ENTRY(1, 8), IDKM_JACT_ENTRY(1, 16), IDKM_JACT_ENTRY(1, 32),
     IDKM_JACT_ENTRY(1, 64), IDKM_NO_ENTRY, IDKM_NO_ENTRY, IDKM_NO_ENTRY, IDKM_NO_ENTRY, IDKM_NO_ENTRY},
    {IDKM_JAC_ENTRY(2, 2), IDKM_JAC_ENTRY(2, 4), IDKM_JACT_ENTRY(2, 8), IDKM_JACT_ENTRY(2, 16), IDKM_JACT_ENTRY(2, 32),
     IDKM_NO_ENTRY, IDKM_NO_ENTRY, IDKM_NO_ENTRY, IDKM_NO_ENTRY, IDKM_NO_ENTRY, IDKM_NO_ENTRY},
    {IDKM_JAC_ENTRY(4, 2), IDKM_JACT_ENTRY(4, 4), IDKM_JACT_ENTRY(4, 8), IDKM_JACT_ENTRY(4, 16), IDKM_NO_ENTRY,
     IDKM_NO_ENTRY, IDKM_NO_ENTRY, IDKM_NO_ENTRY, IDKM_NO_ENTRY, IDKM_NO_ENTRY, IDKM_NO_ENTRY}};
}
