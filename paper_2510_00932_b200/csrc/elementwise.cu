// Dispatch from (op, dtype) to the explicitly instantiated kernel families.
#include "elementwise.cuh"
namespace streamops {
cudaError_t launch_elementwise(int op, int dtype, const VecLaunch &c, const void *x, const void *y,
                               void *out, double scalar, size_t n, cudaStream_t st) {
    using u64 = unsigned long long;
    using u32 = unsigned int;
    const bool d = dtype == DT_F64;
    switch (op) {
        case OP_COPY:
            return d ? launch_op<u64, OP_COPY>(c, (const u64 *)x, nullptr, (u64 *)out, 0.0, n, st)
                     : launch_op<u32, OP_COPY>(c, (const u32 *)x, nullptr, (u32 *)out, 0.0, n, st);
        case OP_SCALE:
            return d ? launch_op<double, OP_SCALE>(c, (const double *)x, nullptr, (double *)out, scalar, n, st)
                     : launch_op<float, OP_SCALE>(c, (const float *)x, nullptr, (float *)out, scalar, n, st);
        case OP_ADD:
            return d ? launch_op<double, OP_ADD>(c, (const double *)x, (const double *)y, (double *)out, scalar, n, st)
                     : launch_op<float, OP_ADD>(c, (const float *)x, (const float *)y, (float *)out, scalar, n, st);
        case OP_TRIAD:
            return d ? launch_op<double, OP_TRIAD>(c, (const double *)x, (const double *)y, (double *)out, scalar, n, st)
                     : launch_op<float, OP_TRIAD>(c, (const float *)x, (const float *)y, (float *)out, scalar, n, st);
        default: return cudaErrorInvalidValue;
    }
}
}  // namespace streamops
