// Instantiations of the decode kernel for one key code (see sa_decode_kernel.cuh).
#include "sa_decode_kernel.cuh"

namespace sa {
void launch_decode_int8(int d, const DecodeArgs& a, int GT, dim3 grid, cudaStream_t s) {
    launch_code<8, false>(d, 0, a, GT, grid, s);
}
}  // namespace sa
