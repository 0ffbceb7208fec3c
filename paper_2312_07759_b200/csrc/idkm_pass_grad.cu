#include "idkm_inst.cuh"
namespace idkm {
extern const KernelEntry k_table_grad[3][N_FAMILY] = {IDKM_BWD_ROW(GRAD, 1), IDKM_BWD_ROW(GRAD, 2), IDKM_BWD_ROW(GRAD, 4)};
}
