#include "idkm_inst.cuh"
namespace idkm {
// explicit-Jacobian adjoint: only the thread-per-weight layouts with k d <= 8
extern const KernelEntry k_table_jacobian[3][N_FAMILY] = {
    {IDKM_JAC_ENTRY(1, 2), IDKM_JAC_ENTRY(1, 4), IDKM_JAC_ENTRY(1, 8), IDKM_NO_ENTRY, IDKM_NO_ENTRY, IDKM_NO_ENTRY,
     IDKM_NO_ENTRY, IDKM_NO_ENTRY, IDKM_NO_ENTRY},
    {IDKM_JAC_ENTRY(2, 2), IDKM_JAC_ENTRY(2, 4), IDKM_NO_ENTRY, IDKM_NO_ENTRY, IDKM_NO_ENTRY, IDKM_NO_ENTRY, IDKM_NO_ENTRY,
     IDKM_NO_ENTRY, IDKM_NO_ENTRY},
    {IDKM_JAC_ENTRY(4, 2), IDKM_NO_ENTRY, IDKM_NO_ENTRY, IDKM_NO_ENTRY, IDKM_NO_ENTRY, IDKM_NO_ENTRY, IDKM_NO_ENTRY,
     IDKM_NO_ENTRY, IDKM_NO_ENTRY}};
}
