// Host side of the C ABI (include/asx.h): argument checks, the layer handle and its device
// buffers, mask generation, tensor-map encoding and the launches.  No arithmetic of the
// method runs on the host.
#include <algorithm>
#include <cstdlib>
#include <cstring>
#include <new>
#include <cmath>
#include <vector>

#include "asx_internal.h"

using namespace asx;

struct asx_layer {
    int C_in, C_out, kh, kw, stride, pad;
    int device = -1;
    int num_sms = 0;
    // mask state (device)
    int64_t rows = 0, cap_rows = 0;
    uint8_t* d_mask = nullptr;
    int32_t* d_kept = nullptr;
    void* d_scratch = nullptr;
    int32_t* d_small = nullptr;        // [0] kept count, [1] status word
    bool has_mask = false;
    int64_t host_kept = -1;            // kept entries of the mask when it came from the host, else -1
    const void* residual = nullptr;    // caller-owned shortcut tensor added in the epilogue, or null
    int32_t* d_in_rank = nullptr;      // compact input: row of each input position within its image, -1 = dropped
    int64_t in_rows = 0, in_rank_cap = 0;
    int64_t in_kept = 0;
    // staging copies with zero-padded channels, for C_in not a multiple of 8
    void* d_wpack = nullptr;
    size_t wpack_bytes = 0;
    void* d_ws = nullptr;              // split-K workspace: fp32 partial tiles, then the tile counters
    size_t ws_bytes = 0;
    int* d_wscnt = nullptr;
    size_t wscnt_ints = 0;
    void* d_xpad = nullptr;
    size_t xpad_bytes = 0;
    // tensor map cache
    CUtensorMap tmap;
    const void* tmap_ptr = nullptr;
    int tmap_BN = 0, tmap_Kw = 0;
    int tmap_es = 0, tmapx_es = 0;     // element size the cached tensor maps were encoded for
    CUtensorMap tmap_x;                // x as a [pixels][C_in] matrix, for the TMA row gather
    const void* tmapx_ptr = nullptr;
    int64_t tmapx_pixels = 0;
    int tmapx_stride = 0;              // bytes between rows of the input view
    cudaStream_t last_stream = nullptr;
    // what the host knows about the current mask (masks that came from host memory, up to 2^24 rows)
    std::vector<uint8_t> host_mask;
    uint64_t mask_epoch = 0;           // bumped by every asx_set_mask*
    // window-patch form: rows of padded input the windows of one 128-row tile span at most, cached per geometry
    // window-patch form: the row tiles cut from the host's mask, cached per geometry and buffer size
    uint64_t tiles_epoch = ~0ull;
    int tiles_Nb = 0, tiles_H = 0, tiles_W = 0, tiles_cap = 0;
    std::vector<int32_t> host_tiles;   // per tile: first kept lowered row, rows, first padded input row of its patch, patch rows
    int64_t tiles_rows = 0;            // kept lowered rows they cover
    void* d_tiles = nullptr;
    size_t d_tiles_bytes = 0;
    CUtensorMap tmap_x4;               // x as a 4-D tensor (C_in, W, H, Nb) with one padded row of 64 channels per box
    const void* tmapx4_ptr = nullptr;
    int tmapx4_Nb = 0, tmapx4_H = 0, tmapx4_W = 0, tmapx4_Wp = 0;
    int tmapx4_px32 = 0;
    int wait_limit_kcycles = 0;
    int last_form = ASX_FORM_NONE;     // producer form of the last asx_run        // bound of the in-kernel waits in units of 1024 cycles (0: the default, about 2 s)
};

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (fn == nullptr) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

asx_status from_cuda(cudaError_t e)
{
    if (e == cudaSuccess) return ASX_OK;
    if (e == cudaErrorMemoryAllocation) return ASX_ERR_OOM;
    return ASX_ERR_CUDA;
}

asx_status bind_device(asx_layer* L)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return ASX_ERR_CUDA;
    if (L->device < 0) {
        cudaDeviceProp prop;
        if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return ASX_ERR_CUDA;
        if (prop.major != 10) return ASX_ERR_UNSUPPORTED;     // built for sm_100a only
        L->device = dev;
        L->num_sms = prop.multiProcessorCount;
    } else if (L->device != dev) {
        return ASX_ERR_INVALID_ARG;                          // a layer stays on its first device
    }
    return ASX_OK;
}

asx_status ensure_mask_buffers(asx_layer* L, int64_t rows)
{
    if (L->d_small == nullptr) {
        if (cudaMalloc(&L->d_small, 2 * sizeof(int32_t)) != cudaSuccess) return ASX_ERR_OOM;
        if (cudaMemset(L->d_small, 0, 2 * sizeof(int32_t)) != cudaSuccess) return ASX_ERR_CUDA;
    }
    if (rows <= L->cap_rows) return ASX_OK;
    if (L->cap_rows > 0) cudaStreamSynchronize(L->last_stream);
    cudaFree(L->d_mask); cudaFree(L->d_kept); cudaFree(L->d_scratch);
    L->d_mask = nullptr; L->d_kept = nullptr; L->d_scratch = nullptr; L->cap_rows = 0;
    const size_t mask_bytes = ((size_t)rows + 15) / 16 * 16;
    if (cudaMalloc(&L->d_mask, mask_bytes) != cudaSuccess) return ASX_ERR_OOM;
    if (cudaMalloc(&L->d_kept, sizeof(int32_t) * (size_t)rows) != cudaSuccess) return ASX_ERR_OOM;
    if (cudaMalloc(&L->d_scratch, (size_t)compact_scratch_bytes(rows)) != cudaSuccess) return ASX_ERR_OOM;
    L->cap_rows = rows;
    return ASX_OK;
}

asx_status run_compaction(asx_layer* L, cudaStream_t st)
{
    return from_cuda(launch_compact(L->d_mask, L->rows, L->d_kept, L->d_small, L->d_scratch, st, true));
}

// Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3", 2011).
void philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int r = 0; r < 10; ++r) {
        const uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        const uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        const uint32_t n1 = (uint32_t)p1;
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        const uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// Window-patch form: cut the kept lowered rows (ascending in image and output row) into tiles of at
// most `max_rows` (<= 128) consecutive rows whose windows span at most `cap` zero-padded input rows.  Pure index
// bookkeeping on the mask the host holds; four ints per tile (first kept lowered row, rows, first
// padded input row of the patch, patch rows); returns the kept lowered rows, or -1 without memory.
int64_t cut_row_tiles(const std::vector<uint8_t>& mask, int Nb, int P, int Wo, int Hp, int kh, int cap, int max_rows,
                      std::vector<int32_t>* tiles)
{
    std::vector<int32_t> kept;
    tiles->clear();
    try {
        kept.reserve(mask.size());
        for (size_t i = 0; i < mask.size(); ++i)
            if (mask[i] != 0) kept.push_back((int32_t)i);
        const bool shared = (int64_t)mask.size() == (int64_t)P;
        const int64_t Pk = (int64_t)kept.size(), Mk = shared ? Pk * Nb : Pk;
        auto padded_row = [&](int64_t rk) -> int64_t {
            const int64_t row = shared ? (rk / Pk) * P + kept[(size_t)(rk % Pk)] : kept[(size_t)rk];
            return (row / P) * Hp + (row % P) / Wo;
        };
        tiles->reserve((size_t)(Mk / 64 + 2));
        for (int64_t r0 = 0; r0 < Mk;) {
            const int64_t first = padded_row(r0);
            int64_t n = 1;
            while (n < max_rows && r0 + n < Mk && padded_row(r0 + n) - first + kh <= cap) ++n;
            tiles->push_back((int32_t)r0);
            tiles->push_back((int32_t)n);
            tiles->push_back((int32_t)first);                                     // first padded input row of the patch
            tiles->push_back((int32_t)(padded_row(r0 + n - 1) - first + kh));     // its rows
            r0 += n;
        }
        return Mk;
    } catch (const std::bad_alloc&) {
        tiles->clear();
        return -1;
    }
}

}  // namespace

extern "C" {

const char* asx_status_string(asx_status s)
{
    switch (s) {
        case ASX_OK: return "ok";
        case ASX_ERR_INVALID_ARG: return "invalid argument";
        case ASX_ERR_UNSUPPORTED: return "unsupported configuration";
        case ASX_ERR_NO_MASK: return "no mask set";
        case ASX_ERR_SHAPE: return "mask length does not match the output geometry";
        case ASX_ERR_ALIGN: return "pointer alignment";
        case ASX_ERR_OOM: return "out of memory";
        case ASX_ERR_CUDA: return "CUDA error";
        case ASX_ERR_TIMEOUT: return "bounded wait in a kernel ran out";
    }
    return "unknown status";
}

asx_status asx_create_layer(int C_in, int C_out, int kh, int kw, int stride, int pad, asx_layer** out)
{
    if (out == nullptr) return ASX_ERR_INVALID_ARG;
    *out = nullptr;
    if (C_in < 1 || C_out < 1 || kh < 1 || kw < 1 || stride < 1 || pad < 0) return ASX_ERR_INVALID_ARG;
    if ((int64_t)kh * kw * C_in >= (1ll << 24) || C_out >= (1 << 20) || kh > 255 || kw > 255 || pad > 255)
        return ASX_ERR_UNSUPPORTED;
    asx_layer* L = new (std::nothrow) asx_layer();
    if (L == nullptr) return ASX_ERR_OOM;
    L->C_in = C_in; L->C_out = C_out; L->kh = kh; L->kw = kw; L->stride = stride; L->pad = pad;
    *out = L;
    return ASX_OK;
}

asx_status asx_set_mask(asx_layer* L, const uint8_t* mask, int64_t rows, void* cuda_stream)
{
    if (L == nullptr || mask == nullptr) return ASX_ERR_INVALID_ARG;
    if (rows < 1 || rows >= (1ll << 31)) return ASX_ERR_INVALID_ARG;
    asx_status s = bind_device(L);
    if (s != ASX_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    s = ensure_mask_buffers(L, rows);
    if (s != ASX_OK) return s;
    cudaPointerAttributes attr;
    bool on_device = false;
    if (cudaPointerGetAttributes(&attr, mask) == cudaSuccess)
        on_device = (attr.type == cudaMemoryTypeDevice || attr.type == cudaMemoryTypeManaged);
    else
        cudaGetLastError();
    cudaError_t e;
    if (on_device) {
        e = cudaMemcpyAsync(L->d_mask, mask, (size_t)rows, cudaMemcpyDeviceToDevice, st);
        L->host_kept = -1;
        L->host_mask.clear();
    } else {
        int64_t kept = 0;                                         // only sizes the tiles (a launch heuristic)
        for (int64_t i = 0; i < rows; ++i) kept += mask[i] != 0;
        L->host_kept = kept;
        L->host_mask.clear();
        if (rows <= (1ll << 24)) {
            try {
                L->host_mask.assign(mask, mask + rows);
            } catch (const std::bad_alloc&) {
                L->host_mask.clear();                              // only costs the choice of kernel form
            }
        }
        e = cudaMemcpyAsync(L->d_mask, mask, (size_t)rows, cudaMemcpyHostToDevice, st);
        if (e == cudaSuccess) e = cudaStreamSynchronize(st);      // the caller may free a host mask on return
    }
    if (e != cudaSuccess) return from_cuda(e);
    L->rows = rows;
    L->last_stream = st;
    ++L->mask_epoch;
    s = run_compaction(L, st);
    L->has_mask = (s == ASX_OK);
    return s;
}

asx_status asx_set_mask_random(asx_layer* L, int64_t rows, double sparsity, int block, uint64_t seed,
                               void* cuda_stream)
{
    if (L == nullptr) return ASX_ERR_INVALID_ARG;
    if (rows < 1 || rows >= (1ll << 31) || block < 1 || !(sparsity >= 0.0 && sparsity <= 1.0))
        return ASX_ERR_INVALID_ARG;
    const int64_t nblocks = (rows + block - 1) / block;
    int64_t n_drop = (int64_t)(sparsity * (double)nblocks + 0.5);
    if (n_drop > nblocks) n_drop = nblocks;
    std::vector<uint8_t> mask;
    std::vector<std::pair<uint64_t, int64_t>> score;
    try {
        mask.assign((size_t)rows, 1);
        score.resize((size_t)nblocks);
    } catch (const std::bad_alloc&) {
        return ASX_ERR_OOM;
    }
    const uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
    for (int64_t b = 0; b < nblocks; ++b) {
        const uint32_t ctr[4] = {(uint32_t)b, (uint32_t)((uint64_t)b >> 32), 0u, 0u};
        uint32_t o[4];
        philox4x32_10(ctr, key, o);
        score[(size_t)b] = {((uint64_t)o[1] << 32) | o[0], b};
    }
    if (n_drop > 0 && n_drop < nblocks)
        std::nth_element(score.begin(), score.begin() + (n_drop - 1), score.end());
    for (int64_t i = 0; i < n_drop; ++i) {
        const int64_t b = score[(size_t)i].second;
        const int64_t lo = b * block, hi = std::min<int64_t>(rows, lo + block);
        std::memset(mask.data() + lo, 0, (size_t)(hi - lo));
    }
    return asx_set_mask(L, mask.data(), rows, cuda_stream);
}

asx_status asx_mask_from_scores(const float* score, int H0, int W0, int Ho, int Wo, double sparsity,
                                uint8_t* mask_out)
{
    if (score == nullptr || mask_out == nullptr || H0 < 1 || W0 < 1 || Ho < 1 || Wo < 1 || Ho > H0 || Wo > W0 ||
        !(sparsity >= 0.0 && sparsity <= 1.0) || (int64_t)Ho * Wo >= (1ll << 31))
        return ASX_ERR_INVALID_ARG;
    const int rh = H0 / Ho, rw = W0 / Wo;                 // ratio = input_res // layer.res
    const int64_t P = (int64_t)Ho * Wo;
    std::vector<std::pair<double, int64_t>> ranked;       // (pooled score, position): ordered by score, then position
    try {
        ranked.resize((size_t)P);
    } catch (const std::bad_alloc&) {
        return ASX_ERR_OOM;
    }
    for (int i = 0; i < Ho; ++i)
        for (int j = 0; j < Wo; ++j) {
            double acc = 0.0;                              // window sum in fp64, raster order of the window
            const float* win = score + (size_t)i * rh * W0 + (size_t)j * rw;
            for (int a2 = 0; a2 < rh; ++a2)
                for (int b2 = 0; b2 < rw; ++b2) acc += (double)win[(size_t)a2 * W0 + b2];
            const int64_t p = (int64_t)i * Wo + j;
            ranked[(size_t)p] = {acc / (double)(rh * rw), p};
        }
    int64_t n_drop = (int64_t)std::floor(sparsity * (double)P + 0.5);
    if (n_drop > P) n_drop = P;
    if (n_drop > 0 && n_drop < P) std::nth_element(ranked.begin(), ranked.begin() + (n_drop - 1), ranked.end());
    std::memset(mask_out, 1, (size_t)P);
    for (int64_t k = 0; k < n_drop; ++k) mask_out[(size_t)ranked[(size_t)k].second] = 0;
    return ASX_OK;
}

asx_status asx_set_mask_from_scores(asx_layer* L, const float* score, int H0, int W0, int Ho, int Wo,
                                    double sparsity, void* cuda_stream)
{
    if (L == nullptr) return ASX_ERR_INVALID_ARG;
    if (Ho < 1 || Wo < 1) return ASX_ERR_INVALID_ARG;
    std::vector<uint8_t> mask;
    try {
        mask.resize((size_t)Ho * (size_t)Wo);
    } catch (const std::bad_alloc&) {
        return ASX_ERR_OOM;
    }
    const asx_status s = asx_mask_from_scores(score, H0, W0, Ho, Wo, sparsity, mask.data());
    if (s != ASX_OK) return s;
    return asx_set_mask(L, mask.data(), (int64_t)Ho * Wo, cuda_stream);
}

asx_status asx_set_residual(asx_layer* L, const void* residual_dev)
{
    if (L == nullptr) return ASX_ERR_INVALID_ARG;
    L->residual = residual_dev;
    return ASX_OK;
}

asx_status asx_set_input_mask(asx_layer* L, const uint8_t* mask, int64_t rows, void* cuda_stream)
{
    if (L == nullptr || mask == nullptr || rows < 1 || rows >= (1ll << 31)) return ASX_ERR_INVALID_ARG;
    const asx_status s = bind_device(L);
    if (s != ASX_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    std::vector<uint8_t> host;
    std::vector<int32_t> rank;
    try {
        host.resize((size_t)rows);
        rank.resize((size_t)rows);
    } catch (const std::bad_alloc&) {
        return ASX_ERR_OOM;
    }
    cudaPointerAttributes attr;
    const bool on_device = cudaPointerGetAttributes(&attr, mask) == cudaSuccess &&
                           (attr.type == cudaMemoryTypeDevice || attr.type == cudaMemoryTypeManaged);
    if (on_device) {
        if (cudaStreamSynchronize(st) != cudaSuccess) return ASX_ERR_CUDA;        // whatever writes the mask is on this stream
        if (cudaMemcpy(host.data(), mask, (size_t)rows, cudaMemcpyDeviceToHost) != cudaSuccess) return ASX_ERR_CUDA;
    } else {
        cudaGetLastError();
        std::memcpy(host.data(), mask, (size_t)rows);
    }
    int32_t kept = 0;
    for (int64_t p = 0; p < rows; ++p) rank[(size_t)p] = host[(size_t)p] != 0 ? kept++ : -1;
    if (rows > L->in_rank_cap) {
        if (cudaStreamSynchronize(L->last_stream) != cudaSuccess) return ASX_ERR_CUDA;
        cudaFree(L->d_in_rank);
        L->d_in_rank = nullptr; L->in_rank_cap = 0;
        if (cudaMalloc(&L->d_in_rank, (size_t)rows * sizeof(int32_t)) != cudaSuccess) return ASX_ERR_OOM;
        L->in_rank_cap = rows;
    }
    // a launch that still reads the old table is ordered before this copy when it used the same stream
    if (cudaMemcpyAsync(L->d_in_rank, rank.data(), (size_t)rows * sizeof(int32_t), cudaMemcpyHostToDevice, st) != cudaSuccess)
        return ASX_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return ASX_ERR_CUDA;            // `rank` goes out of scope
    L->in_rows = rows;
    L->in_kept = kept;
    L->last_stream = st;
    return ASX_OK;
}

asx_status asx_recompact(asx_layer* L, void* cuda_stream)
{
    if (L == nullptr) return ASX_ERR_INVALID_ARG;
    if (!L->has_mask) return ASX_ERR_NO_MASK;
    const asx_status s = bind_device(L);
    if (s != ASX_OK) return s;
    L->last_stream = static_cast<cudaStream_t>(cuda_stream);
    return run_compaction(L, L->last_stream);
}

asx_status asx_run(asx_layer* L, const void* x, int Nb, int H, int W, const void* w, const float* bias,
                   void* y, int flags, void* cuda_stream)
{
    if (L == nullptr || x == nullptr || w == nullptr || y == nullptr) return ASX_ERR_INVALID_ARG;
    if (Nb < 1 || H < 1 || W < 1) return ASX_ERR_INVALID_ARG;
    if (flags & ~(ASX_ACT_RELU | ASX_RECOMPACT | ASX_IMPL_NAIVE | ASX_OUT_COMPACT | ASX_IN_COMPACT | ASX_ACT_SILU | ASX_F32 | ASX_IMPL_ROW_GATHER | ASX_IMPL_WINDOW_PATCH)) return ASX_ERR_INVALID_ARG;
    if ((flags & ASX_IMPL_ROW_GATHER) && (flags & ASX_IMPL_WINDOW_PATCH)) return ASX_ERR_INVALID_ARG;
    const bool f32 = (flags & ASX_F32) != 0;
    const int ES = f32 ? 4 : 2;                 // bytes per element of x, w and y
    const int EPC = 16 / ES;                    // elements per 16-byte chunk
    // fp32 storage runs on dense tensors without a fused shortcut
    if (f32 && ((flags & (ASX_OUT_COMPACT | ASX_IN_COMPACT)) || L->residual != nullptr)) return ASX_ERR_UNSUPPORTED;
    if ((flags & ASX_ACT_RELU) && (flags & ASX_ACT_SILU)) return ASX_ERR_INVALID_ARG;      // one activation at most
    if ((flags & ASX_IMPL_NAIVE) && ((flags & (ASX_OUT_COMPACT | ASX_IN_COMPACT)) || L->residual != nullptr)) return ASX_ERR_INVALID_ARG;
    if (L->residual != nullptr && (reinterpret_cast<uintptr_t>(L->residual) & ((L->C_out % 8 == 0) ? 15 : 1))) return ASX_ERR_ALIGN;
    if (H + 2 * L->pad < L->kh || W + 2 * L->pad < L->kw) return ASX_ERR_INVALID_ARG;
    if (!L->has_mask) return ASX_ERR_NO_MASK;
    asx_status s = bind_device(L);
    if (s != ASX_OK) return s;

    ConvGeom g;
    g.Nb = Nb; g.H = H; g.W = W; g.C_in = L->C_in; g.C_out = L->C_out;
    g.kh = L->kh; g.kw = L->kw; g.stride = L->stride; g.pad = L->pad;
    g.stride_w = L->stride; g.pad_w = L->pad;
    g.Ho = (H + 2 * L->pad - L->kh) / L->stride + 1;
    g.Wo = (W + 2 * L->pad - L->kw) / L->stride + 1;
    g.K = L->kh * L->kw * L->C_in;
    const int64_t P = (int64_t)g.Ho * g.Wo, M = P * Nb;
    const int64_t lim = (1ll << 31) - 1;
    if (H > 32767 || W > 32767) return ASX_ERR_UNSUPPORTED;
    if (M > lim || (int64_t)Nb * H * W * L->C_in > lim || M * L->C_out > lim) return ASX_ERR_UNSUPPORTED;
    if (L->rows != P && L->rows != M) return ASX_ERR_SHAPE;
    g.P = (int)P; g.M = (int)M; g.rows = (int)L->rows;
    const bool in_compact = (flags & ASX_IN_COMPACT) != 0, out_compact = (flags & ASX_OUT_COMPACT) != 0;
    if (out_compact && L->rows != P) return ASX_ERR_SHAPE;            // kept order n*P' + j needs one mask for the batch
    if (in_compact) {
        if (L->d_in_rank == nullptr) return ASX_ERR_NO_MASK;
        if (L->in_rows != (int64_t)H * W) return ASX_ERR_SHAPE;
        if (L->C_in % 8 != 0 || L->in_kept < 1) return ASX_ERR_UNSUPPORTED;
    }
    const int64_t x_rows = in_compact ? (int64_t)Nb * L->in_kept : (int64_t)Nb * H * W;     // rows of x in memory

    const bool vec_in = (L->C_in % EPC == 0);
    const uintptr_t in_align = vec_in ? 15 : (uintptr_t)(ES - 1);
    if ((reinterpret_cast<uintptr_t>(x) & in_align) || (reinterpret_cast<uintptr_t>(w) & in_align))
        return ASX_ERR_ALIGN;
    if (reinterpret_cast<uintptr_t>(y) & ((L->C_out % EPC == 0) ? 15 : (uintptr_t)(ES - 1))) return ASX_ERR_ALIGN;
    if (bias != nullptr && (reinterpret_cast<uintptr_t>(bias) & 3)) return ASX_ERR_ALIGN;
    {
        const uintptr_t xb = reinterpret_cast<uintptr_t>(x), xe = xb + (uintptr_t)x_rows * L->C_in * ES;
        // a compact output holds Nb * P' rows (P' is known on the host for a mask that came from the host)
        const int64_t y_rows = (out_compact && L->host_kept >= 0) ? (int64_t)Nb * L->host_kept : M;
        const uintptr_t yb = reinterpret_cast<uintptr_t>(y), ye = yb + (uintptr_t)y_rows * L->C_out * ES;
        if (xb < ye && yb < xe) return ASX_ERR_INVALID_ARG;
    }

    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    L->last_stream = st;
    // Small masks are compacted inside the fused kernel itself (no launches of its own, and the list stays in
    // shared memory as 16-bit positions); the reference kernel and large masks take the stand-alone compaction
    // kernels.  Up to 16384 rows always; up to FUSED_COMPACT_MAX_ROWS when the list (2 bytes per row) still
    // leaves the plan its pipeline stages (decided below, once the geometry the kernel sees is known).
    bool fuse_compact = (flags & ASX_RECOMPACT) && !(flags & ASX_IMPL_NAIVE) && L->rows <= FUSED_COMPACT_MAX_ROWS;
    if ((flags & ASX_RECOMPACT) && !fuse_compact) {
        s = run_compaction(L, st);
        if (s != ASX_OK) return s;
    }
    const int relu = (flags & ASX_ACT_SILU) ? 2 : (flags & ASX_ACT_RELU) ? 1 : 0;      // activation code: 0 identity, 1 ReLU, 2 SiLU
    int32_t* d_count = L->d_small;
    int* d_status = reinterpret_cast<int*>(L->d_small + 1);

    if (flags & ASX_IMPL_NAIVE) L->last_form = ASX_FORM_NAIVE;
    if (flags & ASX_IMPL_NAIVE)
        return from_cuda(launch_naive(g, x, w, bias, y, L->d_mask, L->d_kept, d_count, relu, f32 ? 1 : 0, st));

    // Channel counts that are not a multiple of 8 are padded with zero channels in staging
    // copies of x and w (a filter tap of a pixel is then a whole number of 16-byte chunks); the
    // kernel runs on the padded geometry, the zero channels contribute nothing.
    const void* xsrc = x;
    const void* wsrc = w;
    int x_row_stride = 0;              // bytes between rows of the TMA view of the input (0: C_in * 2)
    // 2x2-block form for the classic network stem (tiny channel count, stride 2, a 7- or 8-wide
    // filter): pad the channels to 4 and store every aligned 2x2 pixel block as 16 contiguous
    // values (32 bytes), in a copy with zero borders.  Four horizontally adjacent blocks are then one
    // contiguous 128-byte run holding two filter rows of a window (8 columns x 2 rows x 4 channels),
    // i.e. exactly one row of a 64-wide k-block, and consecutive output pixels are consecutive
    // blocks.  The kernel sees 64 channels per "pixel", ceil((kh + shift) / 2) vertical taps, one
    // horizontal tap, stride 1 and no padding, and gathers the runs with the TMA row gather through
    // a view whose rows are 32 bytes apart (rows overlap; the borders make every tap in bounds).
    // shift = pad & 1 aligns the window to the blocks; the filter gets zero rows / columns there.
    const int bshift = L->pad & 1;
    const bool blocks2x2 = !f32 && !in_compact && L->C_in <= 4 && L->stride == 2 && (W % 2) == 0 && (H % 2) == 0 &&
                           (L->kw + bshift + 1) / 2 == 4 && L->kh + bshift <= 32;
    if (blocks2x2) {
        const int kh2 = (L->kh + bshift + 1) / 2;
        const int h0 = (L->pad + bshift) / 2;                              // border on the top and left, in blocks
        const int Hs = (h0 + H / 2 > g.Ho + kh2 - 1) ? h0 + H / 2 : g.Ho + kh2 - 1;
        const int Ws = (((h0 + W / 2 > g.Wo + 3) ? h0 + W / 2 : g.Wo + 3) + 3) / 4 * 4;     // whole 128-byte units of four blocks
        const int64_t nblocks = (int64_t)Nb * Hs * Ws;
        if (nblocks * 16 > lim) return ASX_ERR_UNSUPPORTED;
        const size_t need_x = (size_t)nblocks * 32 + 128, need_w = (size_t)L->C_out * kh2 * 64 * 2;
        if (need_x > L->xpad_bytes || need_w > L->wpack_bytes) {
            cudaStreamSynchronize(st);
            if (need_x > L->xpad_bytes) {
                cudaFree(L->d_xpad);
                L->d_xpad = nullptr; L->xpad_bytes = 0;
                if (cudaMalloc(&L->d_xpad, need_x) != cudaSuccess) return ASX_ERR_OOM;
                L->xpad_bytes = need_x;
            }
            if (need_w > L->wpack_bytes) {
                cudaFree(L->d_wpack);
                L->d_wpack = nullptr; L->wpack_bytes = 0;
                if (cudaMalloc(&L->d_wpack, need_w) != cudaSuccess) return ASX_ERR_OOM;
                L->wpack_bytes = need_w;
            }
            L->tmap_ptr = nullptr;
            L->tmapx_ptr = nullptr;
        }
        cudaError_t e = launch_stage_blocks2x2(x, L->d_xpad, Nb, H, W, L->C_in, Hs, Ws, h0, w, L->d_wpack, L->C_out, L->kh, L->kw, kh2, bshift, st);
        if (e != cudaSuccess) return from_cuda(e);
        xsrc = L->d_xpad;
        wsrc = L->d_wpack;
        g.C_in = 64;
        g.kh = kh2;
        g.kw = 1;
        g.K = kh2 * 64;
        g.H = Hs;
        g.W = Ws;
        g.stride = 1; g.stride_w = 1;
        g.pad = 0; g.pad_w = 0;
        x_row_stride = 32;
    } else if (f32 && L->C_in % 4 != 0) {
        // fp32 storage: zero channels up to a multiple of 4 (one 16-byte chunk); the padding kernel
        // moves 2-byte units, so an fp32 tensor goes through it as twice as many of those.
        const int Cp = (L->C_in + 3) / 4 * 4;
        const int64_t pixels = (int64_t)Nb * H * W, taps = (int64_t)L->C_out * L->kh * L->kw;
        if (pixels * Cp > lim) return ASX_ERR_UNSUPPORTED;
        const size_t need_x = (size_t)pixels * Cp * 4, need_w = (size_t)taps * Cp * 4;
        if (need_x > L->xpad_bytes || need_w > L->wpack_bytes) {
            cudaStreamSynchronize(st);
            if (need_x > L->xpad_bytes) {
                cudaFree(L->d_xpad);
                L->d_xpad = nullptr; L->xpad_bytes = 0;
                if (cudaMalloc(&L->d_xpad, need_x) != cudaSuccess) return ASX_ERR_OOM;
                L->xpad_bytes = need_x;
            }
            if (need_w > L->wpack_bytes) {
                cudaFree(L->d_wpack);
                L->d_wpack = nullptr; L->wpack_bytes = 0;
                if (cudaMalloc(&L->d_wpack, need_w) != cudaSuccess) return ASX_ERR_OOM;
                L->wpack_bytes = need_w;
            }
            L->tmap_ptr = nullptr;
            L->tmapx_ptr = nullptr;
        }
        cudaError_t e = launch_pad_channels(x, L->d_xpad, pixels, 2 * L->C_in, 2 * Cp, st);
        if (e == cudaSuccess) e = launch_pad_channels(w, L->d_wpack, taps, 2 * L->C_in, 2 * Cp, st);
        if (e != cudaSuccess) return from_cuda(e);
        xsrc = L->d_xpad;
        wsrc = L->d_wpack;
        g.C_in = Cp;
        g.K = L->kh * L->kw * Cp;
    } else if (!f32 && L->C_in % 8 != 0) {
        // Pixel-pair form for tiny channel counts under stride 2 (a network's first layer): pad the
        // channels to 4 and read two horizontally adjacent pixels as one 8-channel pixel.  The
        // convolution then has ceil((kw + shift) / 2) horizontal taps, horizontal stride 1 and left
        // padding (pad + shift) / 2 with shift = pad & 1, each filter row of a window is one
        // contiguous run of memory, and K shrinks (7x7x3: 224 instead of 392 with 8-channel padding).
        const bool pairs = (L->C_in <= 4 && L->stride == 2 && (W % 2) == 0);
        const int Cp = pairs ? 4 : (L->C_in + 7) / 8 * 8;
        const int shift = pairs ? (L->pad & 1) : 0;
        const int kw2 = pairs ? (L->kw + shift + 1) / 2 : L->kw;
        const int Ck = pairs ? 8 : Cp;                                     // channels the kernel sees
        const int64_t pixels = (int64_t)Nb * H * W, taps = (int64_t)L->C_out * L->kh * kw2;
        if (pixels * Cp > lim) return ASX_ERR_UNSUPPORTED;
        const size_t need_x = (size_t)pixels * Cp * 2, need_w = (size_t)taps * Ck * 2;
        if (need_x > L->xpad_bytes || need_w > L->wpack_bytes) {
            cudaStreamSynchronize(st);
            if (need_x > L->xpad_bytes) {
                cudaFree(L->d_xpad);
                L->d_xpad = nullptr; L->xpad_bytes = 0;
                if (cudaMalloc(&L->d_xpad, need_x) != cudaSuccess) return ASX_ERR_OOM;
                L->xpad_bytes = need_x;
            }
            if (need_w > L->wpack_bytes) {
                cudaFree(L->d_wpack);
                L->d_wpack = nullptr; L->wpack_bytes = 0;
                if (cudaMalloc(&L->d_wpack, need_w) != cudaSuccess) return ASX_ERR_OOM;
                L->wpack_bytes = need_w;
            }
            L->tmap_ptr = nullptr;
        }
        cudaError_t e = launch_pad_channels(x, L->d_xpad, pixels, L->C_in, Cp, st);
        if (e == cudaSuccess)
            e = pairs ? launch_pack_pair_filters(w, L->d_wpack, L->C_out, L->kh, L->kw, L->C_in, kw2, shift, st)
                      : launch_pad_channels(w, L->d_wpack, (int64_t)L->C_out * L->kh * L->kw, L->C_in, Cp, st);
        if (e != cudaSuccess) return from_cuda(e);
        xsrc = L->d_xpad;
        wsrc = L->d_wpack;
        g.C_in = Ck;
        g.kw = kw2;
        g.K = L->kh * kw2 * Ck;
        if (pairs) {
            g.W = W / 2;
            g.stride_w = 1;
            g.pad_w = (L->pad + shift) / 2;
        }
    }
    FastPlan plan;
    long long est_rows = M;                                       // unknown on the host: assume every row kept
    if (L->host_kept >= 0) est_rows = (L->rows == P) ? L->host_kept * Nb : L->host_kept;
    // Sharing a tile's k-blocks between blocks needs the exact tile count (to size the workspace)
    // and 16-byte output stores.
    const bool allow_split = !f32 && L->host_kept >= 0 && L->C_out % 8 == 0 && (reinterpret_cast<uintptr_t>(y) & 15) == 0;
    if (!plan_fast(g, L->num_sms, est_rows, fuse_compact ? (int)L->rows : 0, allow_split, ES, &plan)) {
        if (!(fuse_compact && L->rows > COMPACT_SMALL_MAX_ROWS)) return ASX_ERR_UNSUPPORTED;
        // no room for the list beside the pipeline stages: the stand-alone compaction, and the list in global memory
        fuse_compact = false;
        s = run_compaction(L, st);
        if (s != ASX_OK) return s;
        if (!plan_fast(g, L->num_sms, est_rows, 0, allow_split, ES, &plan)) return ASX_ERR_UNSUPPORTED;
    }
    // Stride-1 layers with several filter taps and whole 64-channel slices take the window-patch form
    // when the host knows the mask, every tile's windows fit the patch buffers and the planner's
    // estimate favours it; compact inputs and fp32 storage stay with the row gather.
    PatchPlan pplan;
    bool use_patch = false;
    // The window-patch kernel sees the input as [Nb][H][W] pixels of C_in channels.  In the 2x2-block form a
    // "pixel" is the 128-byte run of four blocks that starts at a block, pixels are 32 bytes apart (they
    // overlap); the patch holds every block once, Wo + 3 per row, and only the first Ho + kh - 1 block rows
    // are ever read.
    ConvGeom gp = g;
    if (blocks2x2) gp.H = g.Ho + g.kh - 1;
    if (!f32 && !in_compact && !(flags & ASX_IMPL_ROW_GATHER) && !L->host_mask.empty() &&
        (reinterpret_cast<uintptr_t>(y) & 15) == 0 && plan_patch(gp, fuse_compact ? (int)L->rows : 0, blocks2x2 ? 1 : 0, &pplan)) {
        if (L->tiles_epoch != L->mask_epoch || L->tiles_Nb != Nb || L->tiles_H != H || L->tiles_W != W || L->tiles_cap != pplan.cap_rows) {
            L->tiles_rows = cut_row_tiles(L->host_mask, Nb, gp.P, gp.Wo, pplan.Hp, gp.kh, pplan.cap_rows, 128, &L->host_tiles);
            // Level the waves: with T tiles of 128 rows on S blocks the last of ceil(T / S) waves is partly
            // empty; tiles of fewer rows that fill every wave cost less (a tile's patch reads and epilogue
            // shrink with its rows, only the filter slabs do not), as long as the wave count stays.
            if (L->tiles_rows > 0) {
                const long long t128 = (long long)(L->host_tiles.size() / 4);
                const long long per_wave = std::max<long long>(1, L->num_sms / pplan.n_tiles);      // row tiles one wave takes
                const long long waves = (t128 + per_wave - 1) / per_wave;
                const long long target = waves * per_wave;
                if (target > t128) {
                    int rows_per_tile = (int)((L->tiles_rows + target - 1) / target);
                    rows_per_tile = std::min(128, (rows_per_tile + 7) / 8 * 8);
                    std::vector<int32_t> level;
                    if (rows_per_tile >= 32 && rows_per_tile < 128 &&
                        cut_row_tiles(L->host_mask, Nb, gp.P, gp.Wo, pplan.Hp, gp.kh, pplan.cap_rows, rows_per_tile, &level) == L->tiles_rows &&
                        (long long)(level.size() / 4) <= target)
                        L->host_tiles.swap(level);
                }
            }
            L->tiles_epoch = L->mask_epoch; L->tiles_Nb = Nb; L->tiles_H = H; L->tiles_W = W; L->tiles_cap = pplan.cap_rows;
            const size_t need = L->host_tiles.size() * sizeof(int32_t);
            if (L->tiles_rows > 0 && need > 0) {
                if (need > L->d_tiles_bytes) {
                    cudaStreamSynchronize(st);
                    cudaFree(L->d_tiles);
                    L->d_tiles = nullptr; L->d_tiles_bytes = 0;
                    if (cudaMalloc(&L->d_tiles, need) != cudaSuccess) return ASX_ERR_OOM;
                    L->d_tiles_bytes = need;
                }
                // ordered on the stream behind any launch that still reads the old table; host_tiles lives on in the layer
                if (cudaMemcpyAsync(L->d_tiles, L->host_tiles.data(), need, cudaMemcpyHostToDevice, st) != cudaSuccess) return ASX_ERR_CUDA;
                if (cudaStreamSynchronize(st) != cudaSuccess) return ASX_ERR_CUDA;
            }
        }
        if (L->tiles_rows > 0 && L->tiles_rows == est_rows) {
            plan_patch_cost(gp, L->num_sms, (long long)(L->host_tiles.size() / 4), &pplan);
            use_patch = pplan.est_cost_us <= plan.est_cost_us || (flags & ASX_IMPL_WINDOW_PATCH);
        }
    }
    if (plan.ksplit > 1 && !use_patch) {
        const size_t need = (size_t)plan.ws_items * 128 * (size_t)plan.BN * sizeof(float);
        if (need > L->ws_bytes) {
            cudaFree(L->d_ws);
            L->d_ws = nullptr; L->ws_bytes = 0;
            if (cudaMalloc(&L->d_ws, need) != cudaSuccess) return ASX_ERR_OOM;
            L->ws_bytes = need;
        }
        const size_t ints = 2 * (size_t)(plan.ws_items / plan.ksplit);
        if (ints > L->wscnt_ints) {
            cudaFree(L->d_wscnt);
            L->d_wscnt = nullptr; L->wscnt_ints = 0;
            if (cudaMalloc(&L->d_wscnt, ints * sizeof(int)) != cudaSuccess) return ASX_ERR_OOM;
            L->wscnt_ints = ints;
            if (cudaMemsetAsync(L->d_wscnt, 0, ints * sizeof(int), st) != cudaSuccess) return ASX_ERR_CUDA;
        }
    }
    const int BNsel = use_patch ? pplan.BN : plan.BN;
    const int Kw = g.K;
    const CUtensorMapDataType tm_type = f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
    const cuuint32_t box_k = (cuuint32_t)(128 / ES);           // one 128-byte swizzled row of K elements
    if (L->tmap_ptr != wsrc || L->tmap_BN != BNsel || L->tmap_Kw != Kw || L->tmap_es != ES) {
        EncodeTiledFn enc = encode_tiled_fn();
        if (enc == nullptr) return ASX_ERR_CUDA;
        const cuuint64_t dims[2] = {(cuuint64_t)Kw, (cuuint64_t)L->C_out};
        const cuuint64_t strides[1] = {(cuuint64_t)Kw * ES};
        const cuuint32_t box[2] = {box_k, (cuuint32_t)BNsel};
        const cuuint32_t estr[2] = {1u, 1u};
        const CUresult r = enc(&L->tmap, tm_type, 2, const_cast<void*>(wsrc), dims,
                               strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                               CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return ASX_ERR_CUDA;
        L->tmap_ptr = wsrc; L->tmap_BN = BNsel; L->tmap_Kw = Kw; L->tmap_es = ES;
    }
    if (use_patch) {
        if (L->tmapx4_ptr != xsrc || L->tmapx4_Nb != Nb || L->tmapx4_H != g.H || L->tmapx4_W != g.W || L->tmapx4_Wp != pplan.Wp ||
            L->tmapx4_px32 != pplan.px32) {
            EncodeTiledFn enc = encode_tiled_fn();
            if (enc == nullptr) return ASX_ERR_CUDA;
            // g.H x g.W pixels of g.C_in channels; in the 2x2-block form block rows of g.W / 4 units of four blocks
            // (64 values), which the box takes whole
            const cuuint64_t wu = pplan.px32 ? (cuuint64_t)g.W / 4 : (cuuint64_t)g.W;
            const cuuint64_t dims[4] = {(cuuint64_t)g.C_in, wu, (cuuint64_t)g.H, (cuuint64_t)Nb};
            const cuuint64_t strides[3] = {(cuuint64_t)g.C_in * 2, wu * g.C_in * 2, (cuuint64_t)g.H * wu * g.C_in * 2};
            const cuuint32_t box[4] = {64u, (cuuint32_t)pplan.Wp, 1u, 1u};
            const cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
            const CUresult r = enc(&L->tmap_x4, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(xsrc), dims, strides, box, estr,
                                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            if (r != CUDA_SUCCESS) return ASX_ERR_CUDA;
            L->tmapx4_ptr = xsrc; L->tmapx4_Nb = Nb; L->tmapx4_H = g.H; L->tmapx4_W = g.W; L->tmapx4_Wp = pplan.Wp;
            L->tmapx4_px32 = pplan.px32;
        }
        L->last_form = ASX_FORM_WINDOW_PATCH;
        return from_cuda(launch_patch(gp, pplan, L->tmap, L->tmap_x4, bias, y, L->d_mask, L->d_kept, d_count, relu, d_status, L->num_sms,
                                      fuse_compact ? 1 : 0, L->host_kept, L->residual, L->d_tiles, (int)(L->host_tiles.size() / 4), L->tiles_rows,
                                      out_compact ? 1 : 0, L->wait_limit_kcycles, st));
    }
    if (plan.vec == 2) {
        const int64_t pixels = in_compact ? x_rows : (int64_t)Nb * g.H * g.W;
        const int row_stride = x_row_stride ? x_row_stride : g.C_in * ES;
        if (L->tmapx_ptr != xsrc || L->tmapx_pixels != pixels || L->tmapx_stride != row_stride || L->tmapx_es != ES) {
            EncodeTiledFn enc = encode_tiled_fn();
            if (enc == nullptr) return ASX_ERR_CUDA;
            const cuuint64_t dims[2] = {(cuuint64_t)g.C_in, (cuuint64_t)pixels};
            const cuuint64_t strides[1] = {(cuuint64_t)row_stride};
            const cuuint32_t box[2] = {box_k, 1u};
            const cuuint32_t estr[2] = {1u, 1u};
            const CUresult r = enc(&L->tmap_x, tm_type, 2, const_cast<void*>(xsrc), dims,
                                   strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                   CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
            if (r != CUDA_SUCCESS) return ASX_ERR_CUDA;
            L->tmapx_ptr = xsrc; L->tmapx_pixels = pixels; L->tmapx_stride = row_stride; L->tmapx_es = ES;
        }
    }
    L->last_form = plan.vec == 2 ? ASX_FORM_ROW_GATHER_TMA : ASX_FORM_ROW_GATHER_COPY;
    return from_cuda(launch_fast(g, plan, L->tmap, plan.vec == 2 ? L->tmap_x : L->tmap, xsrc, bias, y, L->d_mask, L->d_kept, d_count, relu, d_status,
                                 L->num_sms, fuse_compact ? 1 : 0, L->host_kept, static_cast<float*>(L->d_ws), L->d_wscnt,
                                 out_compact ? 1 : 0, in_compact ? L->d_in_rank : nullptr, (int)L->in_kept, L->residual, f32 ? 1 : 0, L->wait_limit_kcycles, st));
}

asx_status asx_get_kept(asx_layer* L, int64_t* count, const int32_t** dev_kept)
{
    if (L == nullptr) return ASX_ERR_INVALID_ARG;
    if (!L->has_mask) return ASX_ERR_NO_MASK;
    if (cudaStreamSynchronize(L->last_stream) != cudaSuccess) return ASX_ERR_CUDA;
    int32_t c = 0;
    if (cudaMemcpy(&c, L->d_small, sizeof(c), cudaMemcpyDeviceToHost) != cudaSuccess) return ASX_ERR_CUDA;
    if (count) *count = c;
    if (dev_kept) *dev_kept = L->d_kept;
    return ASX_OK;
}

asx_status asx_get_kept_host(asx_layer* L, int32_t* host_out, int64_t capacity, int64_t* count)
{
    if (L == nullptr || count == nullptr || capacity < 0 || (capacity > 0 && host_out == nullptr))
        return ASX_ERR_INVALID_ARG;
    int64_t c = 0;
    const asx_status s = asx_get_kept(L, &c, nullptr);
    if (s != ASX_OK) return s;
    *count = c;
    const int64_t n = c < capacity ? c : capacity;
    if (n > 0 && cudaMemcpy(host_out, L->d_kept, sizeof(int32_t) * (size_t)n, cudaMemcpyDeviceToHost) != cudaSuccess)
        return ASX_ERR_CUDA;
    return ASX_OK;
}

asx_status asx_get_mask(asx_layer* L, uint8_t* host_mask_out, int64_t rows)
{
    if (L == nullptr || host_mask_out == nullptr) return ASX_ERR_INVALID_ARG;
    if (!L->has_mask) return ASX_ERR_NO_MASK;
    if (rows != L->rows) return ASX_ERR_SHAPE;
    if (cudaStreamSynchronize(L->last_stream) != cudaSuccess) return ASX_ERR_CUDA;
    return from_cuda(cudaMemcpy(host_mask_out, L->d_mask, (size_t)rows, cudaMemcpyDeviceToHost));
}

asx_status asx_last_device_status(asx_layer* L)
{
    if (L == nullptr) return ASX_ERR_INVALID_ARG;
    if (L->d_small == nullptr) return ASX_OK;
    if (cudaStreamSynchronize(L->last_stream) != cudaSuccess) return ASX_ERR_CUDA;
    int32_t word = 0;
    if (cudaMemcpy(&word, L->d_small + 1, sizeof(word), cudaMemcpyDeviceToHost) != cudaSuccess) return ASX_ERR_CUDA;
    int32_t scan_err = 0;
    if (L->d_scratch != nullptr &&
        cudaMemcpy(&scan_err, static_cast<int32_t*>(L->d_scratch) + 1, sizeof(scan_err), cudaMemcpyDeviceToHost) != cudaSuccess)
        return ASX_ERR_CUDA;
    if (word != 0 && cudaMemset(L->d_small + 1, 0, sizeof(word)) != cudaSuccess) return ASX_ERR_CUDA;
    // a launch that gave up may have left tile counters of the split-K exchange half way
    if (word != 0 && L->d_wscnt != nullptr && cudaMemset(L->d_wscnt, 0, L->wscnt_ints * sizeof(int)) != cudaSuccess) return ASX_ERR_CUDA;
    return (word != 0 || scan_err != 0) ? ASX_ERR_TIMEOUT : ASX_OK;
}

asx_status asx_last_run_form(const asx_layer* L, int* form)
{
    if (L == nullptr || form == nullptr) return ASX_ERR_INVALID_ARG;
    *form = L->last_form;
    return ASX_OK;
}

asx_status asx_set_wait_limit(asx_layer* L, int64_t cycles)
{
    if (L == nullptr) return ASX_ERR_INVALID_ARG;
    if (cycles <= 0) {
        L->wait_limit_kcycles = 0;
    } else {
        const int64_t k = (cycles + 1023) / 1024;
        L->wait_limit_kcycles = (int)std::min<int64_t>(k, 1 << 30);
    }
    return ASX_OK;
}

asx_status asx_debug_set_split_counter(asx_layer* L, int64_t tile, int32_t value, void* cuda_stream)
{
    if (L == nullptr) return ASX_ERR_INVALID_ARG;
    if (L->d_wscnt == nullptr || L->wscnt_ints == 0) return ASX_ERR_UNSUPPORTED;
    if (tile < 0 || (size_t)(2 * tile) >= L->wscnt_ints) return ASX_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    // the value is copied out of this frame before the call returns (pageable source)
    if (cudaMemcpyAsync(L->d_wscnt + 2 * tile, &value, sizeof(value), cudaMemcpyHostToDevice, st) != cudaSuccess) return ASX_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return ASX_ERR_CUDA;
    return ASX_OK;
}

asx_status asx_destroy(asx_layer* L)
{
    if (L == nullptr) return ASX_OK;
    if (L->device >= 0) {
        cudaStreamSynchronize(L->last_stream);
        cudaFree(L->d_mask); cudaFree(L->d_kept); cudaFree(L->d_scratch);
        cudaFree(L->d_small); cudaFree(L->d_wpack); cudaFree(L->d_xpad); cudaFree(L->d_ws); cudaFree(L->d_wscnt); cudaFree(L->d_in_rank); cudaFree(L->d_tiles);
    }
    delete L;
    return ASX_OK;
}

int64_t asx_compact_scratch_bytes(int64_t rows)
{
    if (rows < 0) return 0;
    return compact_scratch_bytes(rows);
}

asx_status asx_compact(const uint8_t* mask_dev, int64_t rows, int32_t* kept_dev, int32_t* count_dev,
                       void* scratch_dev, int64_t scratch_bytes, void* cuda_stream)
{
    if (rows < 0 || rows >= (1ll << 31) || count_dev == nullptr || scratch_dev == nullptr) return ASX_ERR_INVALID_ARG;
    if (rows > 0 && (mask_dev == nullptr || kept_dev == nullptr)) return ASX_ERR_INVALID_ARG;
    if (scratch_bytes < compact_scratch_bytes(rows)) return ASX_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(scratch_dev) & 7) return ASX_ERR_ALIGN;
    if ((reinterpret_cast<uintptr_t>(kept_dev) & 3) || (reinterpret_cast<uintptr_t>(count_dev) & 3)) return ASX_ERR_ALIGN;
    return from_cuda(launch_compact(mask_dev, rows, kept_dev, count_dev, scratch_dev,
                                    static_cast<cudaStream_t>(cuda_stream), false));
}

asx_status asx_mask_from_activation(const void* x_dev, int64_t rows, int C, uint8_t* mask_dev, void* cuda_stream)
{
    if (rows < 0 || rows >= (1ll << 31) || C < 1 || C > (1 << 20)) return ASX_ERR_INVALID_ARG;
    if (rows > 0 && (x_dev == nullptr || mask_dev == nullptr)) return ASX_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(x_dev) & 1) return ASX_ERR_ALIGN;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
        return ASX_ERR_CUDA;
    return from_cuda(launch_mask_from_activation(x_dev, rows, C, mask_dev, sms, static_cast<cudaStream_t>(cuda_stream)));
}

asx_status asx_compact_status(const void* scratch_dev, void* cuda_stream)
{
    if (scratch_dev == nullptr) return ASX_ERR_INVALID_ARG;
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) return ASX_ERR_CUDA;
    int32_t err = 0;
    if (cudaMemcpy(&err, static_cast<const int32_t*>(scratch_dev) + 1, sizeof(err), cudaMemcpyDeviceToHost) != cudaSuccess)
        return ASX_ERR_CUDA;
    return err != 0 ? ASX_ERR_TIMEOUT : ASX_OK;
}

}  // extern "C"
