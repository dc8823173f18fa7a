// S1 — mask compaction: kept[j] = position of the j-th non-zero mask byte, ascending.
//
// Appendix A, Algorithm 2 (first function) walks the output positions in raster order and
// appends an entry for every position whose mask is 1; the running index of that loop is an
// exclusive prefix sum of the mask.  Here the prefix sum is a single-pass chained scan:
// each 16384-row tile counts its kept rows (4 x 16 mask bytes per thread, popcount, a shuffle
// scan inside each warp and across the warp totals), publishes its total, and finds the
// number of kept rows before it by looking back over its predecessors' published values,
// 32 predecessors at a time with a warp ballot.  Tiles take their numbers from an atomic
// ticket so that every predecessor of a running tile has already started; the look-back
// wait is bounded and reports through the error word instead of spinning for ever.
#include "asx_internal.h"
#include "ptx_sm100.cuh"

namespace asx {

namespace {

constexpr unsigned long long FLAG_AGGREGATE = 1ull << 32;   // value = this tile's own count
constexpr unsigned long long FLAG_INCLUSIVE = 2ull << 32;   // value = count up to and including this tile
constexpr long long LOOKBACK_CYCLE_LIMIT = 2000000000ll;    // about one second

struct ScratchHeader {
    unsigned int ticket;
    int error;
};

__device__ __forceinline__ unsigned nonzero_bytes4(unsigned w)
{
    unsigned t = ((w & 0x7f7f7f7fu) + 0x7f7f7f7fu) | w;     // bit 7 of each byte: byte != 0
    return ((t >> 7) & 1u) | ((t >> 14) & 2u) | ((t >> 21) & 4u) | ((t >> 28) & 8u);
}

// A block takes COMPACT_SUB consecutive 4096-row sub-tiles: all their mask bytes are loaded before
// anything else (four 16-byte loads in flight per thread instead of one: with one, the kernel was
// bound by the latency of a tile's load -> scan -> look-back -> store chain at 1.5 TB/s), one
// look-back serves all of them, and the index staging buffer is reused sub-tile by sub-tile.
constexpr int COMPACT_SUB = 4;
constexpr int COMPACT_BIG_TILE = COMPACT_SUB * COMPACT_TILE;

__global__ void __launch_bounds__(COMPACT_THREADS, 8)
compact_kernel(const uint8_t* __restrict__ mask, long long rows, int32_t* __restrict__ kept,
               int32_t* __restrict__ count, ScratchHeader* hdr,
               volatile unsigned long long* status, int num_tiles)
{
    __shared__ int32_t s_idx[COMPACT_TILE];
    __shared__ int s_warp_total[COMPACT_SUB][COMPACT_THREADS / 32];
    __shared__ int s_tile;
    __shared__ int s_exclusive;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    ptx::grid_launch_dependents();
    ptx::grid_dependency_wait();          // the list being rebuilt may still be read by an earlier kernel
    if (tid == 0) s_tile = (int)atomicAdd(&hdr->ticket, 1u);
    __syncthreads();
    const int tile = s_tile;
    if (tile >= num_tiles) return;

    // 16 mask bytes per thread and sub-tile -> 16 flag bits each
    const long long tile_first = (long long)tile * COMPACT_BIG_TILE;
    const bool aligned = (reinterpret_cast<uintptr_t>(mask) & 15) == 0;
    unsigned flags[COMPACT_SUB];
    uint4 raw[COMPACT_SUB];
    bool fast[COMPACT_SUB];
#pragma unroll
    for (int sub = 0; sub < COMPACT_SUB; ++sub) {
        const long long first = tile_first + (long long)sub * COMPACT_TILE + (long long)tid * COMPACT_PER_THREAD;
        fast[sub] = aligned && first + COMPACT_PER_THREAD <= rows;
        raw[sub] = make_uint4(0, 0, 0, 0);
        if (fast[sub]) raw[sub] = *reinterpret_cast<const uint4*>(mask + first);
    }
    int mine[COMPACT_SUB], incl[COMPACT_SUB];
#pragma unroll
    for (int sub = 0; sub < COMPACT_SUB; ++sub) {
        const long long first = tile_first + (long long)sub * COMPACT_TILE + (long long)tid * COMPACT_PER_THREAD;
        unsigned f = 0;
        if (fast[sub]) {
            f = nonzero_bytes4(raw[sub].x) | (nonzero_bytes4(raw[sub].y) << 4) | (nonzero_bytes4(raw[sub].z) << 8) |
                (nonzero_bytes4(raw[sub].w) << 12);
        } else {
            for (int j = 0; j < COMPACT_PER_THREAD; ++j)
                if (first + j < rows && mask[first + j] != 0) f |= 1u << j;
        }
        flags[sub] = f;
        mine[sub] = __popc(f);
        // inclusive shuffle scan inside the warp
        int v = mine[sub];
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, v, d);
            if (lane >= d) v += t;
        }
        incl[sub] = v;
        if (lane == 31) s_warp_total[sub][warp] = v;
    }
    __syncthreads();
    int warp_prefix[COMPACT_SUB], sub_total[COMPACT_SUB], tile_total = 0;
#pragma unroll
    for (int sub = 0; sub < COMPACT_SUB; ++sub) {
        int wp = 0, tot = 0;
#pragma unroll
        for (int i = 0; i < COMPACT_THREADS / 32; ++i) {
            const int t = s_warp_total[sub][i];
            if (i < warp) wp += t;
            tot += t;
        }
        warp_prefix[sub] = wp;
        sub_total[sub] = tot;
        tile_total += tot;
    }

    // chained scan across tiles
    if (warp == 0) {
        if (tile == 0) {
            if (lane == 0) {
                status[0] = FLAG_INCLUSIVE | (unsigned)tile_total;
                s_exclusive = 0;
            }
        } else {
            if (lane == 0) status[tile] = FLAG_AGGREGATE | (unsigned)tile_total;
            int exclusive = 0;
            int idx = tile - 1 - lane;
            bool failed = false;
            while (true) {
                unsigned long long st = FLAG_INCLUSIVE;       // before tile 0: nothing kept
                if (idx >= 0) {
                    st = status[idx];
                    if ((st >> 32) == 0) {
                        const long long t0 = clock64();
                        while (((st = status[idx]) >> 32) == 0) {
                            if (clock64() - t0 > LOOKBACK_CYCLE_LIMIT) { failed = true; break; }
                            __nanosleep(40);
                        }
                    }
                }
                if (__any_sync(0xffffffffu, failed)) { failed = true; break; }
                const unsigned has_inclusive = __ballot_sync(0xffffffffu, (st >> 32) == 2);
                const int stop = __ffs(has_inclusive) - 1;    // nearest predecessor with a full prefix
                int v = (stop < 0 || lane <= stop) ? (int)(unsigned)(st & 0xffffffffu) : 0;
#pragma unroll
                for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
                exclusive += v;
                if (stop >= 0) break;
                idx -= 32;
            }
            if (lane == 0) {
                if (failed) {
                    atomicOr(&hdr->error, DEV_TIMEOUT_SCAN);
                    exclusive = 0;
                }
                status[tile] = FLAG_INCLUSIVE | (unsigned)(exclusive + tile_total);
                s_exclusive = exclusive;
            }
        }
    }

    // ordered write, sub-tile by sub-tile: into shared memory first, then coalesced to the list
    int base = 0;                                              // kept rows of this tile before the sub-tile
#pragma unroll
    for (int sub = 0; sub < COMPACT_SUB; ++sub) {
        const long long first = tile_first + (long long)sub * COMPACT_TILE + (long long)tid * COMPACT_PER_THREAD;
        const int at = warp_prefix[sub] + incl[sub] - mine[sub];
        const unsigned f = flags[sub];
        if (f) {                                               // sixteen independent predicated stores, no loop over set bits
#pragma unroll
            for (int j = 0; j < COMPACT_PER_THREAD; ++j)
                if ((f >> j) & 1u) s_idx[at + __popc(f & ((1u << j) - 1u))] = (int32_t)(first + j);
        }
        __syncthreads();                                       // also publishes s_exclusive on the first pass
        const int exclusive = s_exclusive + base;
        for (int i = tid; i < sub_total[sub]; i += COMPACT_THREADS) kept[exclusive + i] = s_idx[i];
        base += sub_total[sub];
        __syncthreads();                                       // s_idx is reused
    }
    if (tile == num_tiles - 1 && tid == 0) *count = s_exclusive + tile_total;
}

// Masks of up to 16 384 rows (every per-layer mask of a classification network) need no chained
// scan: one block of 1024 threads, 16 mask bytes per thread, a shuffle scan within and across
// the warps, and each thread writes its own indices.  No ticket, no status words, no clearing.
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
        const uint4 v = *reinterpret_cast<const uint4*>(mask + first);
        flags = nonzero_bytes4(v.x) | (nonzero_bytes4(v.y) << 4) | (nonzero_bytes4(v.z) << 8) |
                (nonzero_bytes4(v.w) << 12);
    } else {
        for (int j = 0; j < COMPACT_PER_THREAD; ++j)
            if (first + j < rows && mask[first + j] != 0) flags |= 1u << j;
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
        if (hdr != nullptr) { hdr->ticket = 0; hdr->error = 0; }     // a status query must find a clean word
    }
}

}  // namespace

static int tiles_for(int64_t rows)      // 4096-row units: sizes the scratch (one status word each; the kernel uses every fourth)
{
    int64_t t = (rows + COMPACT_TILE - 1) / COMPACT_TILE;
    return (int)(t < 1 ? 1 : t);
}

int64_t compact_scratch_bytes(int64_t rows)
{
    return (int64_t)sizeof(ScratchHeader) + 8 * (int64_t)tiles_for(rows);
}

cudaError_t launch_compact(const uint8_t* mask, int64_t rows, int32_t* kept, int32_t* count,
                           void* scratch, cudaStream_t st)
{
    auto* hdr = static_cast<ScratchHeader*>(scratch);
    if (rows <= COMPACT_SMALL_MAX_ROWS)
        return launch_pdl(compact_small_kernel, dim3(1), dim3(1024), 0, st, mask, (int)rows, kept, count, hdr);
    const int tiles = (int)((rows + COMPACT_BIG_TILE - 1) / COMPACT_BIG_TILE);
    cudaError_t e = cudaMemsetAsync(scratch, 0, (size_t)compact_scratch_bytes(rows), st);
    if (e != cudaSuccess) return e;
    auto* status = reinterpret_cast<volatile unsigned long long*>(hdr + 1);
    return launch_pdl(compact_kernel, dim3(tiles), dim3(COMPACT_THREADS), 0, st, mask, (long long)rows, kept, count,
                      hdr, status, tiles);
}

}  // namespace asx

// ---------------------------------------------------------------------------------------------
// asx_compact_static: the same compaction for callers that must not allocate.
//
// The chained scan needs a little global scratch (a ticket, an error word and one 64-bit status
// word per 4096-row tile).  Every other entry point takes that scratch from the caller or from
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
    // launch_compact clears (or, for small masks, never uses) the ticket, the error word and the
    // status words on the stream, so whatever the previous call left in the array does not matter.
    return asx::launch_compact(mask_dev, rows, kept_dev, count_dev, g_static_scratch_addr[dev],
                               static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess
               ? ASX_OK
               : ASX_ERR_CUDA;
}
