#include "idkm_inst.cuh"
namespace idkm {
extern const KernelEntry k_table_adj[3][N_FAMILY] = {IDKM_ADJ_ROW(1), IDKM_ADJ_ROW(2), IDKM_ADJ_ROW(4)};
}
