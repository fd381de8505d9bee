// Copy kernels (Table 1, "Copy"): raw-word moves, shared by both element types.
#include "elementwise.cuh"
namespace streamops {
// for the word types the scalar is unused; (T)scalar must still compile
template cudaError_t launch_op<unsigned long long, OP_COPY>(const VecLaunch &, const unsigned long long *, const unsigned long long *, unsigned long long *, double, size_t, cudaStream_t);
template cudaError_t launch_op<unsigned int, OP_COPY>(const VecLaunch &, const unsigned int *, const unsigned int *, unsigned int *, double, size_t, cudaStream_t);
}
