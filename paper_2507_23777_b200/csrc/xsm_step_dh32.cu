// Step kernel instances for heads of 32 elements.
#include "xsm_device.cuh"

namespace xsm {

cudaError_t launch_step_dh32(const Dev &D, int dtype, int st_lo, int st_hi, int n_steps, uint32_t serial0, int grid,
                              int smem_bytes, cudaStream_t st, int *max_grid) {
    return launch_step_dh<32>(D, dtype, st_lo, st_hi, n_steps, serial0, grid, smem_bytes, st, max_grid);
}

}  // namespace xsm
