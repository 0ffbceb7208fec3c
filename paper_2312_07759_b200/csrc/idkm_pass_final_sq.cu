// squared-distance variant of this pass (see idkm_inst.cuh)
#define IDKM_SQ true
#include "idkm_inst.cuh"
namespace idkm {
extern const KernelEntry k_table_final_sq[3][N_FAMILY] = {IDKM_FWD_ROW(FINAL, 1), IDKM_FWD_ROW(FINAL, 2), IDKM_FWD_ROW(FINAL, 4)};
}
