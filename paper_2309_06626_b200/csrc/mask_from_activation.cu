// Data-dependent masks: mask[r] = 1 iff some channel of row r of a bf16 activation tensor is
// strictly positive.  The paper's masks are fixed per layer; Section 2 contrasts them with sparsity
// that comes from the activations themselves (ReLU zeros).  This kernel produces such a mask on the
// device, one entry per lowered row, ready for asx_set_mask with a device pointer.
//
// HBM-bound streaming: rows * C * 2 bytes read, rows bytes written.  Fast path (C a multiple of 8,
// at most 256, 16-byte aligned input): C / 8 lanes own one row, each loads 16 bytes; the lanes of
// a row combine with a ballot.  A value is positive iff its sign bit is clear and its magnitude
// bits are in (0, 0x7f80]: zero of either sign and NaN are not positive, denormals and +inf are.
#include <cuda_bf16.h>
#include "asx_internal.h"
#include "ptx_sm100.cuh"

namespace asx {

namespace {

__device__ __forceinline__ bool positive_bf16(uint32_t bits16)
{
    return bits16 != 0u && bits16 <= 0x7f80u;          // sign clear (< 0x8000), non-zero, not NaN
}
__device__ __forceinline__ bool any_positive8(const uint4& v)
{
    const uint32_t w4[4] = {v.x, v.y, v.z, v.w};
    bool p = false;
#pragma unroll
    for (int i = 0; i < 4; ++i) p = p || positive_bf16(w4[i] & 0xffffu) || positive_bf16(w4[i] >> 16);
    return p;
}

// lanes_per_row = C / 8 is a power of two <= 32
__global__ void __launch_bounds__(256) mask_from_activation_vec_kernel(const uint4* __restrict__ x, long long rows,
                                                                       int lanes_per_row, uint8_t* __restrict__ mask)
{
    ptx::grid_launch_dependents();
    ptx::grid_dependency_wait();
    const int lane = threadIdx.x & 31;
    const int rows_per_warp = 32 / lanes_per_row;
    const int sub = lane / lanes_per_row;                       // which of the warp's rows this lane works on
    const unsigned group = (lanes_per_row == 32 ? 0xffffffffu : ((1u << lanes_per_row) - 1u)) << (sub * lanes_per_row);
    const long long warp = (blockIdx.x * (long long)blockDim.x + threadIdx.x) >> 5;
    const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
    for (long long r0 = warp * rows_per_warp; r0 < rows; r0 += nwarps * rows_per_warp) {
        const long long r = r0 + sub;
        bool p = false;
        if (r < rows) p = any_positive8(__ldcg(x + r0 * lanes_per_row + lane));     // read once, and past L1: the
                                                                                          // kernel before may have written it
        const unsigned b = __ballot_sync(0xffffffffu, p);
        if (r < rows && (lane % lanes_per_row) == 0) mask[r] = (b & group) ? 1 : 0;
    }
}

// any C, 2-byte alignment: one warp per row, lanes stride over the channels
__global__ void __launch_bounds__(256) mask_from_activation_gen_kernel(const unsigned short* __restrict__ x, long long rows,
                                                                       int C, uint8_t* __restrict__ mask)
{
    ptx::grid_launch_dependents();
    ptx::grid_dependency_wait();
    const int lane = threadIdx.x & 31;
    const long long warp = (blockIdx.x * (long long)blockDim.x + threadIdx.x) >> 5;
    const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
    for (long long r = warp; r < rows; r += nwarps) {
        bool p = false;
        for (int c = lane; c < C; c += 32) p = p || positive_bf16(__ldcg(x + r * C + c));
        const unsigned b = __ballot_sync(0xffffffffu, p);
        if (lane == 0) mask[r] = b ? 1 : 0;
    }
}

}  // namespace

cudaError_t launch_mask_from_activation(const void* x, long long rows, int C, uint8_t* mask, int num_sms, cudaStream_t st)
{
    if (rows == 0) return cudaSuccess;
    const int lpr = C / 8;
    const bool vec = (C % 8 == 0) && lpr >= 1 && lpr <= 32 && (lpr & (lpr - 1)) == 0 &&
                     (reinterpret_cast<uintptr_t>(x) & 15) == 0;
    const long long warps_needed = vec ? (rows + (32 / lpr) - 1) / (32 / lpr) : rows;
    long long blocks = (warps_needed + 7) / 8;                   // 8 warps per block
    const long long cap = (long long)num_sms * 8;                // resident blocks: a multiple of the SM count
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    if (vec)
        return launch_pdl(mask_from_activation_vec_kernel, dim3((unsigned)blocks), dim3(256), 0, st,
                          static_cast<const uint4*>(x), rows, lpr, mask);
    return launch_pdl(mask_from_activation_gen_kernel, dim3((unsigned)blocks), dim3(256), 0, st,
                      static_cast<const unsigned short*>(x), rows, C, mask);
}

}  // namespace asx
