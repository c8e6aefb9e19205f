// Host-side pieces shared by the source files of the library.
#pragma once

namespace qadam {

// Remembers the cudaError_t of a failed CUDA call for qadam_last_cuda_error (per thread).
void record_cuda_error(int cuda_error);

}  // namespace qadam
