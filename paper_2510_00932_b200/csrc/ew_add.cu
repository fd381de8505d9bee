// ADD kernels (Table 1 of the paper), fp64 and fp32.
#include "elementwise.cuh"
namespace streamops {
template cudaError_t launch_op<double, OP_ADD>(const VecLaunch &, const double *, const double *, double *, double, size_t, cudaStream_t);
template cudaError_t launch_op<float, OP_ADD>(const VecLaunch &, const float *, const float *, float *, double, size_t, cudaStream_t);
}
