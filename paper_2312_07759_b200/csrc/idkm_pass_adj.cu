#include "idkm_inst.cuh"
namespace idkm {
// The last entry is the half-warp layout with 16 centroids per lane (one block of 8 warps per SM, 254 registers):
// half the per-row overhead and one shuffle stage fewer per pair than 8 centroids on a full warp, and the registers
// keep w - c_j from the distance to the accumulation.
#define IDKM_ADJ_ROW(D)                                                                        \
  {                                                                                            \
    IDKM_ENTRY(ADJ, D, 2, 1), IDKM_ENTRY(ADJ, D, 4, 1), IDKM_ENTRY(ADJ, D, 8, 1),              \
        IDKM_ENTRY(ADJ, D, 8, 2), IDKM_ENTRY(ADJ, D, 8, 4), IDKM_ENTRY(ADJ, D, 8, 8),          \
        IDKM_ENTRY(ADJ, D, 8, 16), IDKM_ENTRY(ADJ, D, 8, 32), IDKM_ENTRY(ADJ, D, 16, 16)       \
  }
extern const KernelEntry k_table_adj[3][N_FAMILY] = {IDKM_ADJ_ROW(1), IDKM_ADJ_ROW(2), IDKM_ADJ_ROW(4)};
}
