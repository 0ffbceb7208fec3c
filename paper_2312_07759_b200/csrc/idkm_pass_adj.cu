#include "idkm_inst.cuh"
namespace idkm {
extern const KernelEntry k_table_adj[3][N_FAMILY] = {IDKM_BWD_ROW(ADJ, 1), IDKM_BWD_ROW(ADJ, 2), IDKM_BWD_ROW(ADJ, 4)};
}
