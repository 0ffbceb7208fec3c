// squared-distance variant of this pass (see idkm_inst.cuh)
#define IDKM_SQ true
#include "idkm_inst.cuh"
namespace idkm {
extern const KernelEntry k_table_scatter_sq[3][N_FAMILY] = {IDKM_BWD_ROW(SCATTER, 1), IDKM_BWD_ROW(SCATTER, 2), IDKM_BWD_ROW(SCATTER, 4)};
}
