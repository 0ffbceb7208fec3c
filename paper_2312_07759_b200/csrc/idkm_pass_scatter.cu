#include "idkm_inst.cuh"
namespace idkm {
extern const KernelEntry k_table_scatter[3][N_FAMILY] = {IDKM_BWD_ROW(SCATTER, 1), IDKM_BWD_ROW(SCATTER, 2), IDKM_BWD_ROW(SCATTER, 4)};
}
