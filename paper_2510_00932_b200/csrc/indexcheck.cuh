// Index checking for debugging builds (compiled in with -DSTREAMOPS_CHECK_INDICES, otherwise every
// check below is the constant `true` and disappears).
//
// A tool that watches every memory access of a kernel from outside is not always available; this is
// the in-kernel substitute. In a checking build every global access of the register-vector kernels
// (elementwise and Dot: the default path) first asks index_ok(offset, width, limit): an access that
// would pass the end of its array is NOT made; the first such access per translation unit is
// recorded (which access, its byte offset, the array's byte length) and the host reads the record
// with streamops_index_violation(). Nothing faults and nothing is written out of bounds: a wrong
// index shows up as a record and as missing output, not as a corrupted neighbour.
//
// Each translation unit has its own record (a file-scope __device__ variable, so no relocatable
// device code is needed) and registers a reader for it with the C-ABI layer.
#pragma once
#include <cuda_runtime.h>

namespace streamops {

struct IndexViolation {
    int flag;                      // 0 = none recorded
    int where;                     // which access: see the W_* constants
    unsigned long long offset;     // byte offset of the access within its array
    unsigned long long limit;      // byte length of the array
};

enum : int { W_EW_LOAD_X = 1, W_EW_LOAD_Y = 2, W_EW_STORE = 3, W_EW_TAIL = 4, W_DOT_LOAD_X = 5, W_DOT_LOAD_Y = 6,
             W_DOT_TAIL = 7, W_SELFTEST = 99 };

// api.cu: registry of the per-translation-unit readers
typedef cudaError_t (*violation_reader_t)(IndexViolation *out, bool clear);
void register_violation_reader(violation_reader_t reader);

#ifdef STREAMOPS_CHECK_INDICES
namespace {
__device__ IndexViolation tu_index_violation;

cudaError_t read_tu_violation(IndexViolation *out, bool clear) {
    cudaError_t e = cudaMemcpyFromSymbol(out, tu_index_violation, sizeof(IndexViolation));
    if (e == cudaSuccess && clear && out->flag) {
        const IndexViolation zero{0, 0, 0, 0};
        e = cudaMemcpyToSymbol(tu_index_violation, &zero, sizeof(IndexViolation));
    }
    return e;
}
struct ViolationReaderRegistration {
    ViolationReaderRegistration() { register_violation_reader(read_tu_violation); }
};
ViolationReaderRegistration tu_violation_registration;
}  // namespace

__device__ __forceinline__ bool index_ok(size_t offset, size_t width, size_t limit, int where) {
    if (offset + width <= limit) return true;
    if (atomicCAS(&tu_index_violation.flag, 0, 1) == 0) {
        tu_index_violation.where = where;
        tu_index_violation.offset = offset;
        tu_index_violation.limit = limit;
    }
    return false;
}
#else
__device__ __forceinline__ constexpr bool index_ok(size_t, size_t, size_t, int) { return true; }
#endif

}  // namespace streamops
