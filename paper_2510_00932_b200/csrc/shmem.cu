// Shared-memory exchange microkernel: the library's stand-in for the shared-memory benchmark the
// paper lists in Table 1 (a kernel bound by shared-memory loads and stores, with a repetition
// count as its one parameter). The paper does not define that benchmark; the operation below is
// this library's own.
//
//   The n 32-bit words are cut into tiles of 8 rows x 1024 columns (row-major, 32 KiB). One round
//   replaces row k by row k + row (k + 1) mod 8 + row (k + 2) mod 8, all rows taken from before
//   the round, modulo 2^32. A word past the last whole tile is a one-row tile of its own (its
//   neighbours are itself): a round triples it. out = the array after `rounds` rounds.
//   The round is a bijection (1 + x + x^2 is a unit modulo x^8 - 1 and 2^32; 3 is odd), so the
//   result depends on every input word and on every round at any repetition count.
//
// A block stages a tile in shared memory; thread t owns VW adjacent columns, i.e. one 4*VW-byte
// piece of every row, eight pieces in all. A round is eight shared-memory loads, one three-input
// add per word, and eight shared-memory stores per thread (the store of row k is issued as soon as
// row k + 2 has been loaded, so loads and stores alternate); every value travels through shared memory every round
// (the accesses are inline PTX, so the compiler cannot keep them in registers across rounds).
// Pieces of one row are contiguous across the threads of a warp: no bank conflicts at any width.
// No thread ever reads a column another thread writes, so there is no barrier in the loop --
// the time is shared-memory bandwidth: 2 * rounds * 4 bytes per word, against 128 bytes per
// clock per SM.
#include <atomic>

#include "../../include/streamops.h"
#include "internal.cuh"

namespace streamops {

namespace {

constexpr int kRows = 8, kCols = 1024, kTileWords = kRows * kCols;
constexpr int kRowBytes = kCols * 4;

template <int VW> struct Piece { uint32_t w[VW]; };

template <int VW> __device__ __forceinline__ void lds(Piece<VW> &p, uint32_t addr);
template <> __device__ __forceinline__ void lds<1>(Piece<1> &p, uint32_t addr) {
    asm volatile("ld.shared.b32 %0, [%1];" : "=r"(p.w[0]) : "r"(addr) : "memory");
}
template <> __device__ __forceinline__ void lds<2>(Piece<2> &p, uint32_t addr) {
    asm volatile("ld.shared.v2.b32 {%0,%1}, [%2];" : "=r"(p.w[0]), "=r"(p.w[1]) : "r"(addr) : "memory");
}
template <> __device__ __forceinline__ void lds<4>(Piece<4> &p, uint32_t addr) {
    asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(p.w[0]), "=r"(p.w[1]), "=r"(p.w[2]), "=r"(p.w[3]) : "r"(addr) : "memory");
}
template <int VW> __device__ __forceinline__ void sts(uint32_t addr, const Piece<VW> &p);
template <> __device__ __forceinline__ void sts<1>(uint32_t addr, const Piece<1> &p) {
    asm volatile("st.shared.b32 [%0], %1;" :: "r"(addr), "r"(p.w[0]) : "memory");
}
template <> __device__ __forceinline__ void sts<2>(uint32_t addr, const Piece<2> &p) {
    asm volatile("st.shared.v2.b32 [%0], {%1,%2};" :: "r"(addr), "r"(p.w[0]), "r"(p.w[1]) : "memory");
}
template <> __device__ __forceinline__ void sts<4>(uint32_t addr, const Piece<4> &p) {
    asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};"
                 :: "r"(addr), "r"(p.w[0]), "r"(p.w[1]), "r"(p.w[2]), "r"(p.w[3]) : "memory");
}

// global <-> registers, 4*VW bytes at a time (the pointers are aligned to that width)
template <int VW> __device__ __forceinline__ void ldg_piece(Piece<VW> &p, const uint32_t *src) {
    if constexpr (VW == 1) p.w[0] = *src;
    else if constexpr (VW == 2) { const uint2 v = *reinterpret_cast<const uint2 *>(src); p.w[0] = v.x; p.w[1] = v.y; }
    else { const uint4 v = *reinterpret_cast<const uint4 *>(src); p.w[0] = v.x; p.w[1] = v.y; p.w[2] = v.z; p.w[3] = v.w; }
}
template <int VW> __device__ __forceinline__ void stg_piece(uint32_t *dst, const Piece<VW> &p) {
    if constexpr (VW == 1) *dst = p.w[0];
    else if constexpr (VW == 2) *reinterpret_cast<uint2 *>(dst) = make_uint2(p.w[0], p.w[1]);
    else *reinterpret_cast<uint4 *>(dst) = make_uint4(p.w[0], p.w[1], p.w[2], p.w[3]);
}

template <int VW>
__global__ void __launch_bounds__(kCols / VW)
shmem_mix_kernel(const uint32_t *x, uint32_t *out, unsigned rounds, size_t n) {
    extern __shared__ __align__(16) uint32_t tile[];                 // kTileWords words
    constexpr int TH = kCols / VW;
    const size_t tiles = n / kTileWords;
    const uint32_t mine = (uint32_t)__cvta_generic_to_shared(tile) + threadIdx.x * (VW * 4);

    for (size_t t = blockIdx.x; t < tiles; t += gridDim.x) {
        const uint32_t *src = x + t * kTileWords + threadIdx.x * VW;
        uint32_t *dst = out + t * kTileWords + threadIdx.x * VW;
        Piece<VW> row[kRows];
#pragma unroll
        for (int k = 0; k < kRows; ++k) ldg_piece<VW>(row[k], src + k * kCols);
#pragma unroll
        for (int k = 0; k < kRows; ++k) sts<VW>(mine + k * kRowBytes, row[k]);
        for (unsigned r = 0; r < rounds; ++r) {
            // Row k's new value needs the old rows k, k + 1 and k + 2 only, so its store is issued as soon as
            // row k + 2 has been loaded: loads and stores alternate instead of eight of one kind following
            // eight of the other, and a warp's round is not one long load-then-store dependence.
            lds<VW>(row[0], mine);
            lds<VW>(row[1], mine + kRowBytes);
            const Piece<VW> first = row[0], second = row[1];
#pragma unroll
            for (int k = 0; k < kRows; ++k) {
                if (k + 2 < kRows) lds<VW>(row[k + 2], mine + (k + 2) * kRowBytes);
                Piece<VW> nv;
#pragma unroll
                for (int e = 0; e < VW; ++e)
                    nv.w[e] = row[k].w[e] + (k + 1 < kRows ? row[k + 1].w[e] : first.w[e]) +
                              (k + 2 < kRows ? row[k + 2].w[e] : (k + 2 == kRows ? first.w[e] : second.w[e]));
                sts<VW>(mine + k * kRowBytes, nv);
            }
        }
#pragma unroll
        for (int k = 0; k < kRows; ++k) lds<VW>(row[k], mine + k * kRowBytes);
#pragma unroll
        for (int k = 0; k < kRows; ++k) stg_piece<VW>(dst + k * kCols, row[k]);
    }
    // ragged tail: every word is a one-row tile of its own, tripled once per round, through shared memory too.
    // The staging word is the first word of the thread's OWN piece of row 0: other warps of this
    // block may still be working on their pieces of the last tile, and there is no barrier.
    if (blockIdx.x == (unsigned)(tiles % gridDim.x)) {
        const uint32_t slot = mine;
        for (size_t i = tiles * kTileWords + threadIdx.x; i < n; i += TH) {
            Piece<1> w;
            w.w[0] = x[i];
            sts<1>(slot, w);
            for (unsigned r = 0; r < rounds; ++r) {
                lds<1>(w, slot);
                w.w[0] += w.w[0] + w.w[0];
                sts<1>(slot, w);
            }
            lds<1>(w, slot);
            out[i] = w.w[0];
        }
    }
}

std::atomic<int> g_width_bytes{16};

template <int VW>
cudaError_t launch_width(const uint32_t *x, uint32_t *out, unsigned rounds, size_t n, int sm_count, cudaStream_t st) {
    constexpr int TH = kCols / VW;
    const size_t smem = (size_t)kTileWords * 4;
    int per_sm = 0;
    cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, shmem_mix_kernel<VW>, TH, smem);
    if (e != cudaSuccess) return e;
    if (per_sm < 1) per_sm = 1;
    size_t tiles = n / kTileWords, grid = (size_t)per_sm * (size_t)sm_count;
    if (grid > tiles) grid = tiles;
    if (grid < 1) grid = 1;
    shmem_mix_kernel<VW><<<(unsigned)grid, TH, smem, st>>>(x, out, rounds, n);
    return cudaGetLastError();
}

}  // namespace
}  // namespace streamops

using namespace streamops;

extern "C" int shmem_mix_u32(const unsigned *x, unsigned *out, unsigned rounds, size_t n, streamops_stream_t stream_) {
    cudaStream_t stream = (cudaStream_t)stream_;
    if (n == 0) return STREAMOPS_OK;
    if (!x || !out) return STREAMOPS_ERR_NULL;
    if (((uintptr_t)x % 4) || ((uintptr_t)out % 4)) return STREAMOPS_ERR_ALIGN;
    if (n > ((size_t)1 << 48)) return STREAMOPS_ERR_ARG;
    const uintptr_t x0 = (uintptr_t)x, o0 = (uintptr_t)out;
    if (x0 != o0 && x0 < o0 + n * 4 && o0 < x0 + n * 4) return STREAMOPS_ERR_OVERLAP;
    int device = 0, sm_count = 0;
    cudaError_t e = cudaGetDevice(&device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, device);
    if (e != cudaSuccess) return note_cuda_error(e);
    int width = g_width_bytes.load();
    const uintptr_t bits = x0 | o0;
    while (width > 4 && (bits % (uintptr_t)width)) width >>= 1;          // narrower pieces for less aligned arrays
    if (width == 16) e = launch_width<4>(x, out, rounds, n, sm_count, stream);
    else if (width == 8) e = launch_width<2>(x, out, rounds, n, sm_count, stream);
    else e = launch_width<1>(x, out, rounds, n, sm_count, stream);
    if (e != cudaSuccess) return note_cuda_error(e);
    note_launches(1);
    return STREAMOPS_OK;
}

extern "C" int streamops_set_shmem_width(int bytes) {
    if (bytes != 4 && bytes != 8 && bytes != 16) return STREAMOPS_ERR_ARG;
    g_width_bytes.store(bytes);
    return STREAMOPS_OK;
}

extern "C" int streamops_get_shmem_width(void) { return g_width_bytes.load(); }
