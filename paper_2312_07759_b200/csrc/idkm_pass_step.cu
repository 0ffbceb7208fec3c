#include "idkm_inst.cuh"
namespace idkm {
extern const KernelEntry k_table_step[3][N_FAMILY] = {IDKM_FWD_ROW(STEP, 1), IDKM_FWD_ROW(STEP, 2), IDKM_FWD_ROW(STEP, 4)};
}
