// Internal declarations shared by the library's translation units (not installed).
#pragma once
#include <cuda_runtime.h>
#include <cuda.h>
#include <stdint.h>
#include "asx.h"

namespace asx {

// Geometry of one call, passed by value to the kernels.
struct ConvGeom {
    int Nb, H, W, C_in, C_out, kh, kw, stride, pad, Ho, Wo;
    int stride_w, pad_w;   // horizontal stride and left padding (equal to stride, pad unless the host
                           // re-expressed the input as pixel pairs)
    int K;            // kh*kw*C_in
    int P;            // Ho*Wo
    int M;            // Nb*P
    int rows;         // mask length: P (shared by the batch) or M (one entry per lowered row)
};

// Device status word values (bit flags), reported as ASX_ERR_TIMEOUT.
enum : int { DEV_OK = 0, DEV_TIMEOUT_PIPE = 2, DEV_BAD_INDEX = 4 };

// Launch with the programmatic-stream-serialization attribute: the kernel may begin while its
// predecessor in the stream is still running and must execute griddepcontrol.wait before it
// touches anything an earlier kernel produced (and before it writes anything one may still read).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                              Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// ---- S1: mask compaction (compact.cu)
constexpr int COMPACT_SMALL_MAX_ROWS = 1024 * 16;   // one block handles masks up to this size
constexpr int FUSED_COMPACT_MAX_ROWS = 1024 * 32;   // the fused kernels rebuild lists of up to this many rows themselves (positions fit 16 bits)
constexpr int COMPACT_THREADS = 256;
constexpr int COMPACT_PER_THREAD = 16;
constexpr int COMPACT_TILE = COMPACT_THREADS * COMPACT_PER_THREAD;
int64_t compact_scratch_bytes(int64_t rows);
// mask_written_by_copies_only: the mask buffer is never written by a kernel (a layer's own copy), so
// the write pass may read it before its dependency wait; false for a caller's buffer.
cudaError_t launch_compact(const uint8_t* mask, int64_t rows, int32_t* kept, int32_t* count,
                           void* scratch, cudaStream_t st, bool mask_written_by_copies_only);

// ---- debug reference kernels (naive.cu)
cudaError_t launch_naive(const ConvGeom& g, const void* x, const void* w, const float* bias, void* y,
                         const uint8_t* mask, const int32_t* kept, const int32_t* count, int relu, int f32,
                         cudaStream_t st);

// ---- the tensor-core path (masked_conv_sm100.cu)
struct FastPlan {
    int BN;           // UMMA N per tile (multiple of 16, <= 256)
    int n_tiles;      // ceil(C_out / BN)
    int stages;
    int smem_bytes;
    int vec;          // gather mode: 1 cp.async 16 B (a pixel's channels are whole 16-byte chunks), 2 TMA row
                      // gather (they are whole 128-byte runs)
    int ksplit;       // work items per output tile (shares of the k-blocks); > 1 needs the workspace
    long long ws_items;   // m_tiles * n_tiles * ksplit for the estimated kept rows
    double est_cost_us;   // the planner's estimate of the launch's duration
};
// elem_bytes: 2 (bf16 storage) or 4 (fp32 storage, TF32 contraction)
bool plan_fast(const ConvGeom& g, int num_sms, long long est_kept_rows, int fused_list_rows, bool allow_split, int elem_bytes,
               FastPlan* plan);
cudaError_t launch_fast(const ConvGeom& g, const FastPlan& plan, const CUtensorMap& tmap_w,
                        const CUtensorMap& tmap_x, const void* x, const float* bias, void* y, const uint8_t* mask,
                        const int32_t* kept, const int32_t* count, int relu, int* dev_status,
                        int num_sms, int fuse_compact, long long host_kept, float* ws_partial, int* ws_counters,
                        int out_compact, const int32_t* in_rank, int in_kept, const void* residual, int f32, int wait_limit_kcycles,
                        cudaStream_t st);
// ---- the window-patch form of the tensor-core path (masked_conv_patch_sm100.cu): stride-1 layers with
// several filter taps and C_in % 64 == 0, bf16, dense input, dense or compact output
struct PatchPlan {
    int BN, n_tiles;
    int a_stages, b_stages;
    int G;                 // filter taps per pipeline stage
    int cap_rows;          // padded input rows one patch buffer holds: every tile's windows must span at most this many
    int Hp, Wp, Wp8;       // padded input height and width, Wp rounded up to a multiple of 8
    int p_bufs_log2;       // 1 or 2: two or four patch buffers of cap_rows rows
    int epi8;              // eight epilogue warps and twelve fill warps instead of four and sixteen
    int px32;              // pixels are overlapping runs of four 32-byte blocks (the 2x2-block form of a first layer)
    int smem_bytes;
    double est_cost_us;    // the planner's estimate of the launch's duration
};
// false: this geometry does not take the window-patch form
// px32: g describes the 2x2-block form (64 channels = four 32-byte blocks, kw = 1, no padding, pixels 32 bytes apart)
bool plan_patch(const ConvGeom& g, int fused_list_rows, int px32, PatchPlan* plan);
// fills plan->est_cost_us for a mask that the host cut into n_mtiles row tiles
void plan_patch_cost(const ConvGeom& g, int num_sms, long long n_mtiles, PatchPlan* plan);
// tmap_x4: x as a 4-D tensor (C_in, W, H, Nb) with box (64, Wp, 1, 1), 128-byte swizzle, zero fill; for a px32 plan
// W counts units of four blocks (64 values)
cudaError_t launch_patch(const ConvGeom& g, const PatchPlan& plan, const CUtensorMap& tmap_w, const CUtensorMap& tmap_x4,
                         const float* bias, void* y, const uint8_t* mask, const int32_t* kept, const int32_t* count,
                         int relu, int* dev_status, int num_sms, int fuse_compact, long long host_kept,
                         const void* residual, const void* tiles, int n_mtiles, long long kept_rows, int out_compact,
                         int wait_limit_kcycles, cudaStream_t st);
// src[rows][C] -> dst[rows][Cp] with zero channels added (Cp = 4 or a multiple of 8; rows*Cp % 8 == 0)
cudaError_t launch_pad_channels(const void* src, void* dst, long long rows, int C, int Cp, cudaStream_t st);
// filters for the pixel-pair form: w[C_out][kh][kw][C] -> w2[C_out][kh][kw2][2][4], where pair kxx,
// half j holds the original tap kx = 2*kxx + j - shift (zero when outside 0..kw-1 or c >= C)
cudaError_t launch_mask_from_activation(const void* x, long long rows, int C, uint8_t* mask, int num_sms, cudaStream_t st);
// 2x2-block form of a first layer: the staged input (xs) and the packed filters (w2), one launch
cudaError_t launch_stage_blocks2x2(const void* x, void* xs, int Nb, int H, int W, int C, int Hs, int Ws, int h0,
                                   const void* w, void* w2, int C_out, int kh, int kw, int kh2, int shift, cudaStream_t st);
cudaError_t launch_pack_pair_filters(const void* w, void* w2, int C_out, int kh, int kw, int C, int kw2, int shift,
                                     cudaStream_t st);

}  // namespace asx
