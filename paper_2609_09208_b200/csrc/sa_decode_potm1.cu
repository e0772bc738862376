// Instantiations of the decode kernel for one key code (see sa_decode_kernel.cuh).
#include "sa_decode_kernel.cuh"

namespace sa {
void launch_decode_potm1(bool nib, int d, int mode, const DecodeArgs& a, int GT, dim3 grid, cudaStream_t s) {
    if (nib) launch_code<1, true>(d, mode, a, GT, grid, s);        // dense planar container
    else launch_code<1, false>(d, mode, a, GT, grid, s);
}
}  // namespace sa
