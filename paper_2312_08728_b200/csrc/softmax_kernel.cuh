// Softmax (multinomial logistic) BMGD step kernels: bf16 rows, fp32 parameters W [p][C].
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace bmgdk {

struct SoftmaxLaunchInfo {
    int launches, grid_ctas, cluster_size, threads, depth, smem, cuda_error;
};

inline int64_t softmax_scratch_bytes(int /*p*/, int /*C*/) { return 256; }

inline int softmax_run(const void*, const void*, int64_t, int, int, void*, void*, int*, int, int, double,
                       unsigned long long, int, unsigned long long, int, int, int, int, int, cudaStream_t,
                       SoftmaxLaunchInfo* info) {
    if (info) *info = SoftmaxLaunchInfo{};
    return -8;  // BMGD_ERR_UNIMPLEMENTED
}

}  // namespace bmgdk
