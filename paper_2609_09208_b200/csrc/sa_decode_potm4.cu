// Instantiations of the decode kernel for one key code (see sa_decode_kernel.cuh).
#include "sa_decode_kernel.cuh"

namespace sa {
void launch_decode_potm4(int d, int mode, const DecodeArgs& a, int GT, dim3 grid, cudaStream_t s) {
    launch_code<4, false>(d, mode, a, GT, grid, s);
}
void launch_decode_potm4_lost_copy(const DecodeArgs& a, dim3 grid, cudaStream_t s) {
    launch_one<64, 4, false, 8, 4>(a, grid, s);
}
}  // namespace sa
