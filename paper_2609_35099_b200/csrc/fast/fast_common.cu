// Kernels shared by all signature-specialised entries.
#include "fast_common.cuh"

namespace e3j {
namespace fast {

__global__ void fwd_fixup_kernel(int n_cta, int row_f4, const float4* __restrict__ partial,
                                 const int32_t* __restrict__ part_recv, float4* __restrict__ out) {
    const int c = blockIdx.x;
    const int b = part_recv[2 * c + 1];  // a row whose first piece is this CTA's tail
    if (b < 0) return;
    int last = c;
    while (last + 1 < n_cta && part_recv[2 * (last + 1)] == b) ++last;
    for (int i = threadIdx.x; i < row_f4; i += blockDim.x) {
        float4 sum = partial[(size_t)(2 * c + 1) * row_f4 + i];
        for (int c2 = c + 1; c2 <= last; ++c2) {
            const float4 v = partial[(size_t)(2 * c2) * row_f4 + i];
            sum.x += v.x; sum.y += v.y; sum.z += v.z; sum.w += v.w;
        }
        out[(size_t)b * row_f4 + i] = sum;
    }
}

}  // namespace fast
}  // namespace e3j

