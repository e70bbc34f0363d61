// The lookup-table kernel's instantiations for q = 1 bit-planes (a translation unit per q keeps the build parallel).
#include "bcq_lut_kernel.cuh"

namespace bcq {

cudaError_t launch_lut_q1(int sub, int cols, bool test, const LutOne *one, const LutMany *many, cudaStream_t st)
{
    return launch_lut_for_q<1>(sub, cols, test, one, many, st);
}
cudaError_t lut_status_take_q1(int *status) { return lut_status_take_here(status); }

}  // namespace bcq
