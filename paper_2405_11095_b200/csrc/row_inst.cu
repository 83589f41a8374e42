// One instantiation unit of the contiguous-tile pass per tile size (compile with
// -DFOSGD_ROW_T=<10..15>), so that the tile sizes build in parallel.
#include "common.cuh"

#ifndef FOSGD_ROW_T
#error "define FOSGD_ROW_T"
#endif
#define FOSGD_CAT2(a, b) a##b
#define FOSGD_CAT(a, b) FOSGD_CAT2(a, b)

#include "row_kernels.cuh"

namespace fosgd {
cudaError_t FOSGD_CAT(launch_row_, FOSGD_ROW_T)(int src, int sink, const PassParams& p, cudaStream_t s)
{
    return launch_row_T<FOSGD_ROW_T>(src, sink, p, s);
}

// synchronising read of this unit's counter
cudaError_t FOSGD_CAT(row_timeouts_, FOSGD_ROW_T)(int* out)
{
    return cudaMemcpyFromSymbol(out, g_async_wait_timeouts, sizeof(int));
}
}  // namespace fosgd
