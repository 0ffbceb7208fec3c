#include "idkm_inst.cuh"
namespace idkm {
extern const KernelEntry k_table_step_precise[3][N_FAMILY] = {IDKM_PRECISE_ROW(1), IDKM_PRECISE_ROW(2), IDKM_PRECISE_ROW(4)};
}
