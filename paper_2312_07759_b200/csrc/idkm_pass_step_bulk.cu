// forward step with the rows streamed by bulk asynchronous copies (thread-per-weight layouts)
#include "idkm_inst.cuh"
namespace idkm {
extern const KernelEntry k_table_step_bulk[3][N_FAMILY] = {IDKM_BULK_ROW(1), IDKM_BULK_ROW(2), IDKM_BULK_ROW(4)};
}
