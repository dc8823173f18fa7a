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
    int K;            // kh*kw*C_in
    int P;            // Ho*Wo
    int M;            // Nb*P
    int rows;         // mask length: P (shared by the batch) or M (one entry per lowered row)
};

// Device status word values (bit flags), reported as ASX_ERR_TIMEOUT.
enum : int { DEV_OK = 0, DEV_TIMEOUT_SCAN = 1, DEV_TIMEOUT_PIPE = 2, DEV_BAD_INDEX = 4 };

// ---- S1: mask compaction (compact.cu)
constexpr int COMPACT_THREADS = 256;
constexpr int COMPACT_PER_THREAD = 16;
constexpr int COMPACT_TILE = COMPACT_THREADS * COMPACT_PER_THREAD;
int64_t compact_scratch_bytes(int64_t rows);
cudaError_t launch_compact(const uint8_t* mask, int64_t rows, int32_t* kept, int32_t* count,
                           void* scratch, cudaStream_t st);

// ---- debug reference kernels (naive.cu)
cudaError_t launch_naive(const ConvGeom& g, const void* x, const void* w, const float* bias, void* y,
                         const uint8_t* mask, const int32_t* kept, const int32_t* count, int relu,
                         cudaStream_t st);

// ---- the tensor-core path (masked_conv_sm100.cu)
struct FastPlan {
    int BN;           // UMMA N per tile (multiple of 16, <= 256)
    int n_tiles;      // ceil(C_out / BN)
    int stages;
    int smem_bytes;
    int vec;          // gather mode: 0 element loads (any C_in), 1 cp.async 16 B (C_in % 8 == 0),
                      // 2 TMA row gather (C_in % 64 == 0)
    int Kpad;         // K rounded up to 64
};
bool plan_fast(const ConvGeom& g, int num_sms, long long est_kept_rows, FastPlan* plan);
cudaError_t launch_fast(const ConvGeom& g, const FastPlan& plan, const CUtensorMap& tmap_w,
                        const CUtensorMap& tmap_x, const void* x, const float* bias, void* y, const uint8_t* mask,
                        const int32_t* kept, const int32_t* count, int relu, int* dev_status,
                        int num_sms, cudaStream_t st);
// repack w[C_out][K] into wp[C_out][Kw] (zero padded), for K not a multiple of 8
cudaError_t launch_repack_w(const void* w, void* wp, int C_out, int K, int Kw, cudaStream_t st);

}  // namespace asx
