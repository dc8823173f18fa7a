// S1 — mask compaction: kept[j] = position of the j-th non-zero mask byte, ascending.
//
// Appendix A, Algorithm 2 (first function) walks the output positions in raster order and
// appends an entry for every position whose mask is 1; the running index of that loop is an
// exclusive prefix sum of the mask.  Here the prefix sum has two levels: inside a 16384-row
// tile (4 x 16 mask bytes per thread, popcount, a shuffle scan inside each warp and across the
// warp totals) and across runs of tiles (one run per resident block: a counting pass, then a
// writing pass in which every block sums the counts in front of its run).  Masks of at most
// 16384 rows take one block and one pass.
#include "asx_internal.h"
#include "ptx_sm100.cuh"

namespace asx {

namespace {

struct ScratchHeader {       // first 8 bytes of the scratch; the tile counts follow
    unsigned int reserved;   // kept zero
    int error;               // device status word of the compaction (kept zero: nothing here can time out)
};

__device__ __forceinline__ unsigned nonzero_bytes4(unsigned w)
{
    unsigned t = ((w & 0x7f7f7f7fu) + 0x7f7f7f7fu) | w;     // bit 7 of each byte: byte != 0
    return ((t >> 7) & 1u) | ((t >> 14) & 2u) | ((t >> 21) & 4u) | ((t >> 28) & 8u);
}

// The sixteen flags of one 16-byte load, one bit per mask byte, in the order the arithmetic gives them
// cheapest: byte b of word k (row 4 k + b of the sixteen) lands on bit 8 b + k.
__device__ __forceinline__ constexpr int flag_bit(int j) { return 8 * (j & 3) + (j >> 2); }

__device__ __forceinline__ unsigned nonzero_flags16(const uint4& v)
{
    const unsigned w[4] = {v.x, v.y, v.z, v.w};
    unsigned u = 0;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const unsigned t = ((w[k] & 0x7f7f7f7fu) + 0x7f7f7f7fu) | w[k];     // bit 7 of each byte: byte != 0
        u |= (t >> (7 - k)) & (0x01010101u << k);
    }
    return u;
}

// A block takes COMPACT_SUB consecutive 4096-row sub-tiles and loads all their mask bytes before
// anything else: four 16-byte loads in flight per thread instead of one.
constexpr int COMPACT_SUB = 4;
constexpr int COMPACT_BIG_TILE = COMPACT_SUB * COMPACT_TILE;
constexpr int COMPACT_RESIDENT = 8;      // blocks per SM of the two passes over a large mask

// ---- Large masks: two passes over a grid of resident blocks, no block ever waits for another.  Block g
// owns a run of consecutive 16384-row tiles.  Pass 1 counts the kept rows of every run; in pass 2 a block
// adds up the counts of the runs in front of its own (a few loads per thread, all L2 hits), then writes
// its tiles' indices one tile after another, carrying the offset along.  The mask is read twice, i.e.
// `rows` more bytes than a single-pass chained scan (tiles that publish their totals and look back over
// their predecessors' status words) would move; that form was built first and measured slower (0.150-0.152
// ms on 2^27 rows), and it needs a ticket, cleared status words and bounded spin-waits, which this one
// does not.
__device__ __forceinline__ void load_tile_flags(const uint8_t* __restrict__ mask, long long rows, long long tile_first,
                                                int tid, unsigned (&flags)[COMPACT_SUB])
{
    const bool aligned = (reinterpret_cast<uintptr_t>(mask) & 15) == 0;
    uint4 raw[COMPACT_SUB];
    bool fast[COMPACT_SUB];
#pragma unroll
    for (int sub = 0; sub < COMPACT_SUB; ++sub) {
        const long long first = tile_first + (long long)sub * COMPACT_TILE + (long long)tid * COMPACT_PER_THREAD;
        fast[sub] = aligned && first + COMPACT_PER_THREAD <= rows;
        raw[sub] = make_uint4(0, 0, 0, 0);
        if (fast[sub]) raw[sub] = __ldcg(reinterpret_cast<const uint4*>(mask + first));     // past L1: a kernel may have written the mask
    }
#pragma unroll
    for (int sub = 0; sub < COMPACT_SUB; ++sub) {
        const long long first = tile_first + (long long)sub * COMPACT_TILE + (long long)tid * COMPACT_PER_THREAD;
        unsigned f = 0;
        if (fast[sub]) {
            f = nonzero_flags16(raw[sub]);
        } else {
            for (int j = 0; j < COMPACT_PER_THREAD; ++j)
                if (first + j < rows && __ldcg(mask + first + j) != 0) f |= 1u << flag_bit(j);
        }
        flags[sub] = f;
    }
}

__device__ __forceinline__ void run_of_block(int tiles, int& t0, int& t1)
{
    t0 = (int)((long long)tiles * blockIdx.x / gridDim.x);
    t1 = (int)((long long)tiles * (blockIdx.x + 1) / gridDim.x);
}

// Sum of v over the block, returned to every thread (two barriers).
__device__ __forceinline__ int block_sum(int v, int* s_warp, int* s_total)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
    if (lane == 0) s_warp[warp] = v;
    __syncthreads();
    if (tid == 0) {
        int t = 0;
#pragma unroll
        for (int i = 0; i < COMPACT_THREADS / 32; ++i) t += s_warp[i];
        *s_total = t;
    }
    __syncthreads();
    return *s_total;
}

__global__ void __launch_bounds__(COMPACT_THREADS, COMPACT_RESIDENT)
compact_count_kernel(const uint8_t* __restrict__ mask, long long rows, int tiles, unsigned* __restrict__ run_count)
{
    __shared__ int s_warp[COMPACT_THREADS / 32];
    __shared__ int s_total;
    const int tid = threadIdx.x;
    ptx::grid_launch_dependents();
    ptx::grid_dependency_wait();          // the scratch may still be read by an earlier call's kernels
    int t0, t1;
    run_of_block(tiles, t0, t1);
    int v = 0;
    for (int t = t0; t < t1; ++t) {
        unsigned flags[COMPACT_SUB];
        load_tile_flags(mask, rows, (long long)t * COMPACT_BIG_TILE, tid, flags);
#pragma unroll
        for (int sub = 0; sub < COMPACT_SUB; ++sub) v += __popc(flags[sub]);
    }
    const int total = block_sum(v, s_warp, &s_total);
    if (tid == 0) run_count[blockIdx.x] = (unsigned)total;
}

// Pass 2: the indices of a 4096-row sub-tile are put in order in shared memory and copied to the list
// with full-width stores (direct stores of each 32-row ballot word's indices, without the staging,
// write half-filled lines and were 12 % slower; 16-byte stores from the unaligned staging buffer 3 %; a
// staging index swizzled against bank conflicts 18 %: the pass is bound by the instructions it issues).
// EARLY_MASK: the mask is only ever written by stream-ordered copies (a layer's own copy of its mask), so
// the first tile's mask bytes may be loaded and scanned before the dependency wait, while the pass before
// still runs.  A caller's mask buffer may have been written by the kernel just before this call (a
// data-dependent mask), which, launched as a programmatic predecessor, can still be storing it: then the
// load waits like everything else.
template <bool EARLY_MASK>
__global__ void __launch_bounds__(COMPACT_THREADS, COMPACT_RESIDENT)
compact_write_kernel(const uint8_t* __restrict__ mask, long long rows, int tiles, int32_t* __restrict__ kept,
                     const unsigned* __restrict__ run_count, int32_t* __restrict__ count, ScratchHeader* hdr)
{
    __shared__ int32_t s_idx[COMPACT_TILE];
    __shared__ int s_warp_total[COMPACT_SUB][COMPACT_THREADS / 32];
    __shared__ int s_total;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    ptx::grid_launch_dependents();
    int t0, t1;
    run_of_block(tiles, t0, t1);
    unsigned flags[COMPACT_SUB];
    if (!EARLY_MASK) ptx::grid_dependency_wait();
    if (t0 < t1) load_tile_flags(mask, rows, (long long)t0 * COMPACT_BIG_TILE, tid, flags);
    if (EARLY_MASK) ptx::grid_dependency_wait();          // the counts come from the pass before; the list may still be read
    // Offset of this block's run: the counts of all runs in front of it.  Read past L1: this block was
    // launched while the pass before was running, L1 is not invalidated in between, and the SM may hold
    // a stale line of the scratch.
    int before = 0;
    for (int i = tid; i < (int)blockIdx.x; i += COMPACT_THREADS) before += (int)__ldcg(run_count + i);
    int exclusive = block_sum(before, s_warp_total[0], &s_total);
    for (int t = t0; t < t1; ++t) {
        const long long tile_first = (long long)t * COMPACT_BIG_TILE;
        if (t != t0) load_tile_flags(mask, rows, tile_first, tid, flags);
        int mine[COMPACT_SUB], incl[COMPACT_SUB];
#pragma unroll
        for (int sub = 0; sub < COMPACT_SUB; ++sub) {
            mine[sub] = __popc(flags[sub]);
            int v = mine[sub];
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const int u = __shfl_up_sync(0xffffffffu, v, d);
                if (lane >= d) v += u;
            }
            incl[sub] = v;
            if (lane == 31) s_warp_total[sub][warp] = v;
        }
        __syncthreads();
#pragma unroll
        for (int sub = 0; sub < COMPACT_SUB; ++sub) {
            // lanes 0..7 hold the eight warp totals; a three-step scan gives every warp its prefix and the tile total
            const int wt = lane < COMPACT_THREADS / 32 ? s_warp_total[sub][lane] : 0;
            int winc = wt;
#pragma unroll
            for (int d = 1; d < COMPACT_THREADS / 32; d <<= 1) {
                const int u = __shfl_up_sync(0xffffffffu, winc, d);
                if (lane >= d) winc += u;
            }
            const int wp = __shfl_sync(0xffffffffu, winc - wt, warp);
            const int tot = __shfl_sync(0xffffffffu, winc, COMPACT_THREADS / 32 - 1);
            const long long first = tile_first + (long long)sub * COMPACT_TILE + (long long)tid * COMPACT_PER_THREAD;
            const int at = wp + incl[sub] - mine[sub];
            const unsigned f = flags[sub];
            if (f) {                                               // sixteen predicated stores, no loop over set bits
                int pos = at;
                const int32_t v0 = (int32_t)first;
#pragma unroll
                for (int j = 0; j < COMPACT_PER_THREAD; ++j)
                    if ((f >> flag_bit(j)) & 1u) { s_idx[pos] = v0 + j; ++pos; }
            }
            __syncthreads();
            {
                int32_t* dst = kept + exclusive;
                int i = tid;
                for (; i + 3 * COMPACT_THREADS < tot; i += 4 * COMPACT_THREADS) {      // four loads ahead of four stores
                    const int32_t a0 = s_idx[i], a1 = s_idx[i + COMPACT_THREADS], a2 = s_idx[i + 2 * COMPACT_THREADS],
                                  a3 = s_idx[i + 3 * COMPACT_THREADS];
                    dst[i] = a0;
                    dst[i + COMPACT_THREADS] = a1;
                    dst[i + 2 * COMPACT_THREADS] = a2;
                    dst[i + 3 * COMPACT_THREADS] = a3;
                }
                for (; i < tot; i += COMPACT_THREADS) dst[i] = s_idx[i];
            }
            exclusive += tot;
            __syncthreads();                                       // s_idx and, after the last sub-tile, the warp totals are reused
        }
    }
    if (blockIdx.x == gridDim.x - 1 && tid == 0) {
        *count = (int32_t)exclusive;
        hdr->reserved = 0;                   // a status query must find a clean word
        hdr->error = 0;
    }
}

// Masks of up to 16 384 rows (every per-layer mask of a classification network) need no second
// scan: one block of 1024 threads, 16 mask bytes per thread, a shuffle scan within and across
// the warps, and each thread writes its own indices.
__global__ void __launch_bounds__(1024)
compact_small_kernel(const uint8_t* __restrict__ mask, int rows, int32_t* __restrict__ kept,
                     int32_t* __restrict__ count, ScratchHeader* hdr)
{
    __shared__ int s_warp_total[32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    ptx::grid_launch_dependents();
    ptx::grid_dependency_wait();
    const int first = tid * COMPACT_PER_THREAD;
    unsigned flags = 0;
    const bool aligned = (reinterpret_cast<uintptr_t>(mask) & 15) == 0;
    if (aligned && first + COMPACT_PER_THREAD <= rows) {
        const uint4 v = __ldcg(reinterpret_cast<const uint4*>(mask + first));      // past L1: a kernel may have written the mask
        flags = nonzero_bytes4(v.x) | (nonzero_bytes4(v.y) << 4) | (nonzero_bytes4(v.z) << 8) |
                (nonzero_bytes4(v.w) << 12);
    } else {
        for (int j = 0; j < COMPACT_PER_THREAD; ++j)
            if (first + j < rows && __ldcg(mask + first + j) != 0) flags |= 1u << j;
    }
    const int mine = __popc(flags);
    int incl = mine;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += t;
    }
    if (lane == 31) s_warp_total[warp] = incl;
    __syncthreads();
    // every warp scans the 32 warp totals itself: lane i holds the total of warp i
    int wt = s_warp_total[lane], winc = wt;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, winc, d);
        if (lane >= d) winc += t;
    }
    const int warp_prefix = __shfl_sync(0xffffffffu, winc - wt, warp);
    const int total = __shfl_sync(0xffffffffu, winc, 31);
    int at = warp_prefix + incl - mine;
    unsigned f = flags;
    while (f) {
        const int j = __ffs(f) - 1;
        f &= f - 1;
        kept[at++] = first + j;
    }
    if (tid == 0) {
        *count = total;
        if (hdr != nullptr) { hdr->reserved = 0; hdr->error = 0; }     // a status query must find a clean word
    }
}

}  // namespace

static int resident_sms()               // SM count of the current device (looked up once per device)
{
    static int sms[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (sms[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) n = 148;
        sms[dev] = n;
    }
    return sms[dev];
}

static int tiles_for(int64_t rows)      // 4096-row units: sizes the scratch (8 bytes each; the passes use 4 bytes per resident block, at most one block per 16384 rows)
{
    int64_t t = (rows + COMPACT_TILE - 1) / COMPACT_TILE;
    return (int)(t < 1 ? 1 : t);
}

int64_t compact_scratch_bytes(int64_t rows)
{
    return (int64_t)sizeof(ScratchHeader) + 8 * (int64_t)tiles_for(rows);
}

cudaError_t launch_compact(const uint8_t* mask, int64_t rows, int32_t* kept, int32_t* count,
                           void* scratch, cudaStream_t st, bool mask_written_by_copies_only)
{
    auto* hdr = static_cast<ScratchHeader*>(scratch);
    if (rows <= COMPACT_SMALL_MAX_ROWS)
        return launch_pdl(compact_small_kernel, dim3(1), dim3(1024), 0, st, mask, (int)rows, kept, count, hdr);
    const int tiles = (int)((rows + COMPACT_BIG_TILE - 1) / COMPACT_BIG_TILE);
    // one resident block per run of tiles: eight blocks per SM, never more blocks than tiles (the scratch has
    // 8 bytes per 4096 rows, i.e. room for eight 32-bit counts per tile)
    const int grid = tiles < COMPACT_RESIDENT * resident_sms() ? tiles : COMPACT_RESIDENT * resident_sms();
    unsigned* run_count = reinterpret_cast<unsigned*>(hdr + 1);
    cudaError_t e = launch_pdl(compact_count_kernel, dim3(grid), dim3(COMPACT_THREADS), 0, st, mask, (long long)rows, tiles, run_count);
    if (e == cudaSuccess)
        e = mask_written_by_copies_only
                ? launch_pdl(compact_write_kernel<true>, dim3(grid), dim3(COMPACT_THREADS), 0, st, mask, (long long)rows, tiles, kept,
                             static_cast<const unsigned*>(run_count), count, hdr)
                : launch_pdl(compact_write_kernel<false>, dim3(grid), dim3(COMPACT_THREADS), 0, st, mask, (long long)rows, tiles, kept,
                             static_cast<const unsigned*>(run_count), count, hdr);
    return e;
}

}  // namespace asx

// ---------------------------------------------------------------------------------------------
// asx_compact_static: the same compaction for callers that must not allocate.
//
// The compaction of a large mask needs a little global scratch (a header and the per-tile counts,
// sized at 8 bytes per 4096 rows).  Every other entry point takes that scratch from the caller or from
// memory the layer allocated.  Some callers can do neither at the moment they need a kept-row
// list: a serving loop that must not call cudaMalloc because it synchronises the whole device and
// stalls every other stream; code running after a framework has claimed all device memory for
// its own pool; a plug-in that only holds the raw buffers its host handed in.  For them the
// scratch lives in the library image itself, in the array below: no allocation call of any
// kind is made, at the price of a fixed upper size and of one array shared between all calls.
namespace {

constexpr long long STATIC_MAX_ROWS = ASX_COMPACT_STATIC_MAX_ROWS;
constexpr size_t STATIC_SCRATCH_BYTES = 8 + 8 * (size_t)(STATIC_MAX_ROWS / asx::COMPACT_TILE);

// Held by every GPU that loads the library until the process exits (about 32 KB).
static __device__ __align__(256) unsigned char g_static_scratch[STATIC_SCRATCH_BYTES];

// In host code `g_static_scratch` is only a handle for the runtime, not an address the GPU
// understands, so the device address is looked up once per device and remembered here.
constexpr int MAX_DEVICES = 64;
void* g_static_scratch_addr[MAX_DEVICES] = {nullptr};

}  // namespace

extern "C" asx_status asx_compact_static(const uint8_t* mask_dev, int64_t rows, int32_t* kept_dev,
                                         int32_t* count_dev, void* cuda_stream)
{
    if (rows < 0 || count_dev == nullptr) return ASX_ERR_INVALID_ARG;
    if (rows > 0 && (mask_dev == nullptr || kept_dev == nullptr)) return ASX_ERR_INVALID_ARG;
    if (rows > STATIC_MAX_ROWS) return ASX_ERR_UNSUPPORTED;          // the built-in scratch is too small
    if ((reinterpret_cast<uintptr_t>(kept_dev) & 3) || (reinterpret_cast<uintptr_t>(count_dev) & 3)) return ASX_ERR_ALIGN;
    if ((size_t)asx::compact_scratch_bytes(rows) > STATIC_SCRATCH_BYTES) return ASX_ERR_UNSUPPORTED;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return ASX_ERR_CUDA;
    if (dev < 0 || dev >= MAX_DEVICES) return ASX_ERR_UNSUPPORTED;
    if (g_static_scratch_addr[dev] == nullptr) {
        // first call on this device: resolve the array's device address (not a stream operation)
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) {
            cudaGetLastError();
            return ASX_ERR_CUDA;
        }
        g_static_scratch_addr[dev] = p;
    }
    // launch_compact overwrites every word of the array it later reads (tile counts, header), in
    // stream order, so whatever the previous call left in the array does not matter.
    return asx::launch_compact(mask_dev, rows, kept_dev, count_dev, g_static_scratch_addr[dev],
                               static_cast<cudaStream_t>(cuda_stream), false) == cudaSuccess
               ? ASX_OK
               : ASX_ERR_CUDA;
}
