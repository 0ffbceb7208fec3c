// squared-distance variant of this pass (see idkm_inst.cuh)
#define IDKM_SQ true
#include "idkm_inst.cuh"
namespace idkm {
extern const KernelEntry k_table_adj_sq[3][N_FAMILY] = {IDKM_ADJ_ROW(1), IDKM_ADJ_ROW(2), IDKM_ADJ_ROW(4)};
}
