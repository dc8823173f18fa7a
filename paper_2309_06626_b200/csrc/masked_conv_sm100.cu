// S2 + S3 + S4 — the masked convolution as one persistent, warp-specialised sm_100a kernel.
//
// Section 3.2 / Appendix A describe three stages: an indirection-based lowering that skips
// masked positions, an unmodified dense GEMM over the reduced range, and a post-processing
// pass that re-inserts zeros.  Here the three are one kernel over tiles of 128 kept rows:
//
//   producer warps  gather the kept windows of x straight into the shared-memory operand
//                   layout the tensor core reads (K-major rows of 64 bf16 with the 128-byte
//                   swizzle); nothing is lowered to global memory.  Padding taps and rows
//                   past the end of the kept list are filled with zeros.
//   TMA thread      streams the matching 64-wide K slab of the filter matrix w[C_out][K].
//   MMA thread      issues tcgen05.mma (128 x BN x 16, bf16 -> fp32) into one of two
//                   accumulators in tensor memory, so the epilogue of tile i overlaps the
//                   main loop of tile i+1.
//   epilogue warps  read the accumulator, add the bias, apply ReLU, round to bf16 and store
//                   each kept row at its NHWC position.
//   zero warps      write zeros to the dropped rows of this block's share of the output,
//                   straight from the mask.  Every output element is written exactly once.
//
// The kept-row list comes from device memory or, for masks of at most 16384 rows, is built by
// every block in its own shared memory at the start of this kernel (stage i of Section 3.2 fused
// in); either way the host never has to know the count.  Layers with few kept rows and a long
// reduction may share a tile's k-blocks between blocks (split K with a fixed-order exchange).
// All waits are bounded: a wait that runs out sets the status word and every role leaves.
#include <cuda_bf16.h>
#include "asx_internal.h"
#include "ptx_sm100.cuh"
#include "conv_common.cuh"

namespace asx {

namespace {

constexpr int BM = 128;                 // kept rows per tile (UMMA M)
constexpr int BK = 64;                  // K elements per pipeline stage (one 128-byte swizzled row)
constexpr int A_STAGE_BYTES = BM * BK * 2;
static_assert(BK == 64, "the MMA loop issues four K=16 instructions per stage");
constexpr int MAX_STAGES = 8;
constexpr int MIN_STAGES = 4;
constexpr int WARP_TMA = 0, WARP_MMA = 1, WARP_EPI0 = 2, WARP_PROD0 = 6;
constexpr int NUM_PROD_WARPS = 16, NUM_EPI_WARPS = 4;
constexpr int GROUP_WARPS = 8;          // gather warps per group: 8 warps x 16 rows = one 128-row stage
constexpr int INFO_RING = 8;            // tiles whose row coordinates are kept in shared memory (power of two)
constexpr int WARP_ZERO0 = WARP_PROD0 + NUM_PROD_WARPS, NUM_ZERO_WARPS = 4;
constexpr int WARP_INFO = WARP_ZERO0 + NUM_ZERO_WARPS;
constexpr int NUM_THREADS = 32 * (WARP_INFO + 1);
static_assert(NUM_EPI_WARPS * 32 == BM, "one epilogue thread per tile row");
static_assert(NUM_THREADS / 32 < 32, "the fused compaction keeps its running count in slot 31 of the warp totals");
struct FastArgs {
    FastDiv fdP, fdWo;           // divisions by P and Wo
    FastDiv fdNt;                // division by n_tiles
    FastDiv fdKs;                // division by ksplit
    FastDiv fdCin, fdkw, fdS;    // divisions by C_in, kw and the number of stages (cp.async gather)
    FastDiv fdcnt_host;          // division by the kept count when the host knows it (d = 0: it does not)
    const __nv_bfloat16* x;
    const float* bias;
    __nv_bfloat16* y;
    const uint8_t* mask;
    const int32_t* kept;
    const int32_t* count;
    int* dev_status;
    int relu;
    int BN, n_tiles, stages, tmem_cols;
    int vec_out;        // C_out % 8 == 0 and y 16-byte aligned: 16-byte stores
    int st32;           // bf16, C_out % 16 == 0, y 32-byte aligned and the layer is paced by its stores: 32-byte epilogue stores
    int fuse_compact;   // rebuild the kept-row list from the mask inside this kernel (small masks)
    int32_t* kept_out;  // where the fused compaction writes the list and its count
    int32_t* count_out;
    const __nv_bfloat16* residual;   // non-null: added to acc + bias before the activation, same layout as y
    int out_compact;    // y holds the kept rows only, in kept order (row rk at y[rk][*]); nothing is zero-filled
    const int32_t* in_rank;   // non-null: x holds only the rows its own mask kept; in_rank[pos] = row of input position
                              // pos within its image's in_kept rows, or -1 for a dropped position (read as zeros)
    int in_kept;        // kept input positions per image
    int ksplit;         // work items per output tile: each takes a contiguous share of the k-blocks
    float* ws_partial;  // ksplit > 1: [item][128][BN] fp32 partial tiles
    int* ws_counters;   // ksplit > 1: per output tile {partials written, slices reduced}, zero between launches
    int ws_items;       // capacity of ws_partial in items
    int wait_limit_kcycles;   // bound of every wait in the kernel, in units of 1024 clock cycles
};

struct alignas(16) Shared {           // lives after the operand stages
    int2 rowinfo[INFO_RING][BM];   // per tile row: first input pixel index, (iy0 << 16) | (ix0 & 0xffff)
    float bias[2][256];   // bias of the tile's columns, double buffered
    unsigned long long info_full[INFO_RING];
    unsigned long long info_empty[INFO_RING];
    unsigned long long full[MAX_STAGES];
    unsigned long long empty[MAX_STAGES];
    unsigned long long acc_full[2];
    unsigned long long acc_empty[2];
    unsigned int tmem_base;
    WaitCtl ctl;          // abort flag and the wait limit of this launch
    int scan_total[32];   // fused compaction: kept rows per warp
};

enum : int { GATHER_CPASYNC = 1, GATHER_TMA = 2 };

// Work item t = (output tile, k share): tile = t / ksplit, share ks = t % ksplit covers k-blocks
// [ks KB / ksplit, (ks + 1) KB / ksplit).  The shares of a tile are consecutive items, so they run
// on different blocks at the same time.
struct Item {
    int tile, ks, m_tile, n_tile, kb_lo, kb_hi;
};
__device__ __forceinline__ Item item_of(int t, int KB, const FastArgs& a)
{
    Item it;
    if (a.ksplit == 1) {
        it.tile = t;
        it.ks = 0;
        it.kb_lo = 0;
        it.kb_hi = KB;
    } else {
        it.tile = (int)fd_div((uint32_t)t, a.fdKs);
        it.ks = t - it.tile * a.ksplit;
        it.kb_lo = (int)fd_div((uint32_t)(it.ks * KB), a.fdKs);
        it.kb_hi = (int)fd_div((uint32_t)((it.ks + 1) * KB), a.fdKs);
    }
    it.m_tile = (int)fd_div((uint32_t)it.tile, a.fdNt);
    it.n_tile = it.tile - it.m_tile * a.n_tiles;
    return it;
}

// What the gather warps need to know about the rk-th kept lowered row: the pixel index of its
// window's corner, (n H + iy0) W + ix0 (with a compact input: the first input row of its image,
// n * in_kept), and the corner's coordinates packed as iy0 << 16 | ix0.
// Rows past the end get iy0 = -32768, for which no filter tap is inside the image.
// (row: the output row of the kept row, as out_row_of gives it, or -1 past the end)
__device__ __forceinline__ int2 row_info_from_row(int row, const ConvGeom& g, const FastArgs& a)
{
    int2 info = make_int2(0, (int)0x80000000u);
    if (row >= 0) {
        if (row < g.M) {
            const int n = (int)fd_div((uint32_t)row, a.fdP), p = row - n * g.P;
            const int oy = (int)fd_div((uint32_t)p, a.fdWo), ox = p - oy * g.Wo;
            const int iy0 = oy * g.stride - g.pad, ix0 = ox * g.stride_w - g.pad_w;
            info.x = a.in_rank != nullptr ? n * a.in_kept : (n * g.H + iy0) * g.W + ix0;
            info.y = (iy0 << 16) | (ix0 & 0xffff);
        } else {
            atomicOr(a.dev_status, DEV_BAD_INDEX);
        }
    }
    return info;
}
__device__ __forceinline__ int2 row_info_of(int rk, int Mk, const FastDiv& fdcnt, const ConvGeom& g, const FastArgs& a,
                                            const KeptList& kept)
{
    return row_info_from_row(rk < Mk ? out_row_of(rk, fdcnt, g, kept) : -1, g, a);
}

// SILU: the activation is z / (1 + exp(-z)) instead of the run-time choice between ReLU and identity
// (an instance of its own, like RESIDUAL: the plain path pays for every extra branch in the epilogue).
// F32: x, w and y are fp32 (the storage type of Appendix A); a pipeline stage is still 128 rows of
// 128 bytes, i.e. 32 K-elements, and the tensor core reads the operands as TF32.
template <int MODE, bool IN_COMPACT, bool RESIDUAL, bool SILU, bool F32>
__global__ void __launch_bounds__(NUM_THREADS, 1)
masked_conv_sm100_kernel(const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ CUtensorMap tmap_x,
                         const ConvGeom g, const FastArgs a)
{
    extern __shared__ uint8_t smem_raw[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    // Let the next kernel of the stream start its own prologue; everything up to the dependency
    // wait below touches only this block's shared and tensor memory.
    ptx::grid_launch_dependents();
    const int N = g.C_out;

    const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    const int BN = a.BN, S = a.stages;
    const int stage_bytes = A_STAGE_BYTES + BN * (BK * 2);
    Shared* sh = reinterpret_cast<Shared*>(smem_raw + (smem_base - ptx::smem_u32(smem_raw)) + S * stage_bytes);
    volatile WaitCtl* abort_flag = &sh->ctl;

    constexpr int BKE = F32 ? 32 : BK;      // K elements per stage
    constexpr int ES = F32 ? 4 : 2;         // bytes per element of x, w and y
    constexpr int EPC = 16 / ES;            // elements per 16-byte chunk
    const int KB = (g.K + BKE - 1) / BKE;

    // The layer's mask is only ever written by stream-ordered copies, never by a kernel, so the
    // fused compaction may read it while the preceding kernel is still running; the read is
    // issued first so that its latency overlaps the set-up below.
    uint4 early_mask = make_uint4(0, 0, 0, 0);
    const bool early_ok = a.fuse_compact && tid * 16 + 16 <= g.rows && (reinterpret_cast<uintptr_t>(a.mask) & 15) == 0;
    if (early_ok) early_mask = ptx::ld_global_v4_keep_in_l2(a.mask + tid * 16);

    // barrier initialisation, one barrier per thread (a single thread took about 1300 clocks over them); the
    // threads are those of the last warps, so that the tensor-memory allocation of warp 1 runs beside it
    {
        constexpr int NB = 2 * MAX_STAGES + 2 * INFO_RING + 4;
        int i = tid - (NUM_THREADS - NB);
        if (i >= 0) {
            unsigned long long* bar;
            uint32_t count;
            // full: the filter thread's expect_tx arrival (which in TMA mode also announces the gathered
            // bytes) + in the copy modes every gather lane's arrival
            if (i < MAX_STAGES) { bar = &sh->full[i]; count = 1 + (MODE == GATHER_TMA ? 0 : GROUP_WARPS * 32); }
            else if ((i -= MAX_STAGES) < MAX_STAGES) { bar = &sh->empty[i]; count = 1; }
            else if ((i -= MAX_STAGES) < INFO_RING) { bar = &sh->info_full[i]; count = 1; }
            else if ((i -= INFO_RING) < INFO_RING) { bar = &sh->info_empty[i]; count = NUM_PROD_WARPS; }    // one arrival per gather warp
            else if ((i -= INFO_RING) < 2) { bar = &sh->acc_full[i]; count = 1; }
            else { i -= 2; bar = &sh->acc_empty[i]; count = NUM_EPI_WARPS; }
            ptx::mbar_init(ptx::smem_u32(bar), count);
            ptx::fence_mbar_init();
        }
        if (tid == 0) {
            sh->ctl.abort = 0;
            sh->ctl.limit_kcycles = a.wait_limit_kcycles;
        }
    }
    if (warp == WARP_MMA) {
        ptx::tmem_alloc(ptx::smem_u32(&sh->tmem_base), (uint32_t)a.tmem_cols);
        ptx::tmem_relinquish();
    }
    if (warp == WARP_TMA && lane == 0) {
        ptx::prefetch_tensormap(&tmap_w);
        if (MODE == GATHER_TMA) ptx::prefetch_tensormap(&tmap_x);
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = sh->tmem_base;

    int cnt = 0;
    KeptList kept_list{a.kept, nullptr};
    unsigned short* kept_s = reinterpret_cast<unsigned short*>(sh + 1);     // after the barriers
    if (a.fuse_compact) {
        cnt = block_compact(a.mask, g.rows, early_mask, early_ok, kept_s, sh->scan_total, NUM_THREADS);
        kept_list.s = kept_s;
    }
    // Without the fused compaction the list and its count were written by an earlier kernel: wait
    // for it here.  With it, the wait comes after the row decoding below, which needs only the list.
    if (!a.fuse_compact) {
        ptx::grid_dependency_wait();
        cnt = __ldcg(a.count);
    }
    const int Mk = (g.rows == g.P) ? g.Nb * cnt : cnt;
    // With every position dropped there are no tiles; the zero warps then write the whole output
    // (Algorithm 2, mask == 0 branch).
    const int m_tiles = (Mk + BM - 1) / BM;
    int total_tiles = m_tiles * a.n_tiles * a.ksplit;     // work items
    if (a.ksplit > 1 && total_tiles > a.ws_items) {       // cannot happen when the host sized the workspace from this mask
        if (tid == 0) atomicOr(a.dev_status, DEV_BAD_INDEX);
        total_tiles = 0;
    }
    FastDiv fdcnt = a.fdcnt_host;
    if (cnt <= 0 || fdcnt.d != (uint32_t)cnt) fdcnt = make_fastdiv((uint32_t)(cnt > 0 ? cnt : 1));   // the host did not know the count

    // Row coordinates of this block's first INFO_RING tiles, one row per thread: a single warp
    // working through them is 1.5 us of dependent arithmetic in front of the first gather.
    {
        for (int idx = tid; idx < INFO_RING * BM; idx += NUM_THREADS) {
            const int jj = idx / BM, rr = idx - jj * BM;
            const long long t = blockIdx.x + (long long)jj * gridDim.x;
            if (t < total_tiles)
                sh->rowinfo[jj][rr] = row_info_of(item_of((int)t, KB, a).m_tile * BM + rr, Mk, fdcnt, g, a, kept_list);
        }
        __syncthreads();
        if (tid < INFO_RING && blockIdx.x + (long long)tid * gridDim.x < total_tiles) ptx::mbar_arrive(ptx::smem_u32(&sh->info_full[tid]));
    }
    // From here on the kernel reads what earlier kernels wrote (the input, the filters) and writes
    // the output and the list, so it waits for them to have finished.
    if (a.fuse_compact) {
        ptx::grid_dependency_wait();
        if (blockIdx.x == 0) {      // the list in global memory, for asx_get_kept and later runs
            for (int i = tid; i < cnt; i += NUM_THREADS) a.kept_out[i] = (int32_t)kept_s[i];
            if (tid == 0) *a.count_out = cnt;
        }
    }

    if (warp == WARP_TMA) {
        // ------------------------------------------------------------------ filter slabs by TMA
        if (lane == 0) {
            int s = 0;
            uint32_t ph = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
                const Item item = item_of(t, KB, a);
                const int n_tile = item.n_tile;
                for (int kb = item.kb_lo; kb < item.kb_hi; ++kb) {
                    if (!wait_bar<40>(ptx::smem_u32(&sh->empty[s]), ph ^ 1u, abort_flag, a.dev_status)) { ok = false; break; }
                    const uint32_t full = ptx::smem_u32(&sh->full[s]);
                    ptx::mbar_arrive_expect_tx(full, (uint32_t)(BN * BK * 2 + (MODE == GATHER_TMA ? A_STAGE_BYTES : 0)));
                    ptx::tma_load_2d(smem_base + s * stage_bytes + A_STAGE_BYTES, &tmap_w, full, kb * BKE, n_tile * BN);
                    if (++s == S) { s = 0; ph ^= 1u; }
                }
            }
            if (!ok) {   // let loads already issued land before the block's shared memory goes away
                for (int i = 0; i < 64; ++i) __nanosleep(1000);
            }
        }
    } else if (warp == WARP_INFO) {
        // ------------------------------------------------------------------ row coordinates
        // Decodes the kept rows of upcoming tiles into the shared-memory ring, four rows per lane,
        // running ahead of the gather warps by up to INFO_RING tiles.
        int j = INFO_RING;                        // the first INFO_RING tiles were decoded by the whole block
        for (long long t = blockIdx.x + (long long)INFO_RING * gridDim.x; t < total_tiles; t += gridDim.x, ++j) {
            const int r = j % INFO_RING;
            int good = 1;
            if (lane == 0)
                good = wait_bar<200>(ptx::smem_u32(&sh->info_empty[r]), ((uint32_t)(j / INFO_RING) & 1u) ^ 1u, abort_flag, a.dev_status) ? 1 : 0;
            good = __shfl_sync(0xffffffffu, good, 0);
            if (!good) break;
            const int m_tile = item_of((int)t, KB, a).m_tile;
            // the four list entries first (with the list in global memory each is a trip to L2: one after the other
            // they were 2.7 us per tile, which paced every layer with one k-block per tile and a mask too large for
            // the fused compaction), then the arithmetic
            int rows4[4];
#pragma unroll
            for (int q2 = 0; q2 < 4; ++q2) {
                const int rk = m_tile * BM + lane * 4 + q2;
                rows4[q2] = rk < Mk ? out_row_of(rk, fdcnt, g, kept_list) : -1;
            }
#pragma unroll
            for (int q2 = 0; q2 < 4; ++q2) sh->rowinfo[r][lane * 4 + q2] = row_info_from_row(rows4[q2], g, a);
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&sh->info_full[r]));
        }
    } else if (warp == WARP_MMA) {
        // ------------------------------------------------------------------ MMA issue
        // The whole warp runs the loop so that descriptors and counters stay in uniform registers;
        // one elected lane issues the tcgen05 instructions (issuing from inside a divergent
        // single-lane branch costs about 100 cycles per instruction).
        const uint32_t idesc = F32 ? ptx::umma_idesc_tf32(BM, BN) : ptx::umma_idesc_bf16(BM, BN);
        const uint64_t adesc0 = ptx::umma_desc_k_major_sw128(smem_base);
        int s = 0, ti = 0;
        uint32_t ph = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, ++ti) {
            const int buf = ti & 1;
            const uint32_t use = (uint32_t)(ti >> 1) & 1u;
            ok = warp_wait_bar<0>(ptx::smem_u32(&sh->acc_empty[buf]), use ^ 1u, abort_flag, a.dev_status);
            if (!ok) break;
            ptx::tc_fence_after_sync();
            const uint32_t d = tmem_base + (uint32_t)(buf * BN);
            const Item item = item_of(t, KB, a);
            for (int kb = item.kb_lo; kb < item.kb_hi; ++kb) {
                ok = warp_wait_bar<0>(ptx::smem_u32(&sh->full[s]), ph, abort_flag, a.dev_status);
                if (!ok) break;
                // Only the cp.async gather writes the stage through the generic proxy without a fence
                // of its own (TMA writes through the async proxy, the element gather fences after
                // its stores).
                if (MODE == GATHER_CPASYNC) ptx::fence_proxy_async_smem();
                ptx::tc_fence_after_sync();
                const uint64_t adesc = adesc0 + (uint64_t)(s * (stage_bytes >> 4));   // start-address field
                const uint64_t bdesc = adesc + (A_STAGE_BYTES >> 4);
                if (ptx::elect_one()) {
                    if (F32) {                                                          // 8 K-elements = 32 bytes
                        ptx::umma_tf32(d, adesc, bdesc, idesc, kb != item.kb_lo ? 1u : 0u);
                        ptx::umma_tf32(d, adesc + 2, bdesc + 2, idesc, 1u);
                        ptx::umma_tf32(d, adesc + 4, bdesc + 4, idesc, 1u);
                        ptx::umma_tf32(d, adesc + 6, bdesc + 6, idesc, 1u);
                    } else {
                        ptx::umma_bf16(d, adesc, bdesc, idesc, kb != item.kb_lo ? 1u : 0u);       // 16 K-elements = 32 bytes
                        ptx::umma_bf16(d, adesc + 2, bdesc + 2, idesc, 1u);             //   = 2 descriptor units
                        ptx::umma_bf16(d, adesc + 4, bdesc + 4, idesc, 1u);
                        ptx::umma_bf16(d, adesc + 6, bdesc + 6, idesc, 1u);
                    }
                    ptx::umma_commit(ptx::smem_u32(&sh->empty[s]));
                }
                __syncwarp();
                if (++s == S) { s = 0; ph ^= 1u; }
            }
            if (ok && ptx::elect_one()) ptx::umma_commit(ptx::smem_u32(&sh->acc_full[buf]));
            __syncwarp();
        }
    } else if (warp < WARP_PROD0) {
        // ------------------------------------------------------------------ epilogue
        const int q = warp & 3;                       // TMEM lanes 32q .. 32q+31 belong to this warp
        unsigned short* y2 = reinterpret_cast<unsigned short*>(a.y);
        int ti = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, ++ti) {
            const Item item = item_of(t, KB, a);
            const int m_tile = item.m_tile, n_tile = item.n_tile;
            const int n0 = n_tile * BN;
            // kept rows from the accumulator
            const int buf = ti & 1;
            const uint32_t use = (uint32_t)(ti >> 1) & 1u;
            const int rk = m_tile * BM + q * 32 + lane;
            const bool valid = rk < Mk;
            const long long yoff = valid ? (long long)(a.out_compact ? rk : out_row_of(rk, fdcnt, g, kept_list)) * N : 0;
            {
                float* sb = sh->bias[buf];
                const int et = (warp - WARP_EPI0) * 32 + lane;
                for (int c1 = et; c1 < BN; c1 += NUM_EPI_WARPS * 32)
                    sb[c1] = (a.bias != nullptr && n0 + c1 < N) ? __ldg(a.bias + n0 + c1) : 0.f;
                asm volatile("bar.sync 1, %0;" ::"n"(NUM_EPI_WARPS * 32) : "memory");
            }
            const float* sbias = sh->bias[buf];
            if (!warp_wait_bar<100>(ptx::smem_u32(&sh->acc_full[buf]), use, abort_flag, a.dev_status)) { ok = false; break; }
            ptx::tc_fence_after_sync();
            const uint32_t tacc = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * BN);
            if (!F32 && a.ksplit > 1) {
                // ---- split K: this item holds a partial sum.  Every share writes its partial tile
                // to the workspace; when all shares of the tile are there, each share adds up the
                // partials of its slice of the tile's rows, always in share order (so the result
                // does not depend on which block finished first), and writes that slice of y.
                const int et = (warp - WARP_EPI0) * 32 + lane;
                // A partial tile is stored as [BN / 4 column groups][128 rows] float4, so that the
                // warps (one row per lane) write and read whole consecutive lines.
                float4* mine = reinterpret_cast<float4*>(a.ws_partial) + (size_t)t * (BN >> 2) * BM + (q * 32 + lane);
                for (int c0 = 0; c0 < BN; c0 += 32) {
                    uint32_t r[32];
                    if (c0 + 32 <= BN) {
                        ptx::tmem_ld_32(tacc + (uint32_t)c0, r);
                    } else {
                        uint32_t r16[16];
                        ptx::tmem_ld_16(tacc + (uint32_t)c0, r16);
#pragma unroll
                        for (int j = 0; j < 16; ++j) { r[j] = r16[j]; r[16 + j] = 0; }
                    }
                    ptx::tmem_ld_wait();
#pragma unroll
                    for (int h = 0; h < 8; ++h)
                        if (c0 + 4 * h < BN)
                            __stcg(mine + (size_t)((c0 >> 2) + h) * BM,
                                   make_float4(__uint_as_float(r[4 * h]), __uint_as_float(r[4 * h + 1]),
                                               __uint_as_float(r[4 * h + 2]), __uint_as_float(r[4 * h + 3])));
                }
                ptx::tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&sh->acc_empty[buf]));     // the accumulator is free again
                int* counters = a.ws_counters + 2 * item.tile;
                __threadfence();
                asm volatile("bar.sync 1, %0;" ::"n"(NUM_EPI_WARPS * 32) : "memory");
                if (et == 0) {
                    atomicAdd(counters, 1);
                    const long long t0 = clock64();
                    while (*reinterpret_cast<volatile int*>(counters) < a.ksplit) {
                        if (abort_flag->abort) break;
                        if (clock64() - t0 > ((long long)abort_flag->limit_kcycles << 10)) {
                            abort_flag->abort = 1;
                            atomicOr(a.dev_status, DEV_TIMEOUT_PIPE);
                            break;
                        }
                        __nanosleep(64);
                    }
                    __threadfence();
                }
                asm volatile("bar.sync 1, %0;" ::"n"(NUM_EPI_WARPS * 32) : "memory");
                if (abort_flag->abort) { ok = false; break; }
                // this share's slice: 8-column groups [g_lo, g_hi) of all 128 rows, one row per lane
                const int G = BN >> 3;
                const int g_lo = item.ks * G / a.ksplit, g_hi = (item.ks + 1) * G / a.ksplit;
                const float4* __restrict__ tile_ws = reinterpret_cast<const float4*>(a.ws_partial) + (size_t)item.tile * a.ksplit * (BN >> 2) * BM;
                uint4* __restrict__ yv = reinterpret_cast<uint4*>(a.y);
                const int rk2 = m_tile * BM + et;              // NUM_EPI_WARPS * 32 == BM: thread et owns row et
                const long long yrow = rk2 < Mk ? (long long)(a.out_compact ? rk2 : out_row_of(rk2, fdcnt, g, kept_list)) * N : -1;
#pragma unroll 2
                for (int gq = g_lo; gq < g_hi; ++gq) {
                    if (yrow < 0 || n0 + gq * 8 >= N) continue;
                    float4 lo4 = make_float4(0.f, 0.f, 0.f, 0.f), hi4 = lo4;
                    for (int sp0 = 0; sp0 < a.ksplit; sp0 += 4) {
                        float4 pl[4], phh[4];
#pragma unroll
                        for (int d2 = 0; d2 < 4; ++d2) {
                            const int sp = sp0 + d2;
                            if (sp < a.ksplit) {
                                const float4* src = tile_ws + ((size_t)sp * (BN >> 2) + 2 * gq) * BM + et;
                                pl[d2] = __ldcg(src);
                                phh[d2] = __ldcg(src + BM);
                            } else {
                                pl[d2] = make_float4(0.f, 0.f, 0.f, 0.f);
                                phh[d2] = pl[d2];
                            }
                        }
#pragma unroll
                        for (int d2 = 0; d2 < 4; ++d2) {          // always in share order
                            lo4.x += pl[d2].x; lo4.y += pl[d2].y; lo4.z += pl[d2].z; lo4.w += pl[d2].w;
                            hi4.x += phh[d2].x; hi4.y += phh[d2].y; hi4.z += phh[d2].z; hi4.w += phh[d2].w;
                        }
                    }
                    float v[8] = {lo4.x, lo4.y, lo4.z, lo4.w, hi4.x, hi4.y, hi4.z, hi4.w};
                    if (RESIDUAL) {
                        float res[8];
                        load_residual8(a.residual, yrow + n0 + gq * 8, 8, 1, res);
#pragma unroll
                        for (int j = 0; j < 8; ++j) v[j] += res[j];
                    }
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const float f = v[j] + sbias[gq * 8 + j];
                        v[j] = SILU ? silu(f) : a.relu ? fmaxf(f, 0.f) : f;
                    }
                    uint4 o;
                    o.x = pack_bf16(v[0], v[1]);
                    o.y = pack_bf16(v[2], v[3]);
                    o.z = pack_bf16(v[4], v[5]);
                    o.w = pack_bf16(v[6], v[7]);
                    yv[(yrow + n0 + gq * 8) >> 3] = o;
                }
                asm volatile("bar.sync 1, %0;" ::"n"(NUM_EPI_WARPS * 32) : "memory");
                if (et == 0) {
                    // the last share to finish its slice puts the tile's counters back to zero
                    if (atomicAdd(counters + 1, 1) == a.ksplit - 1) {
                        atomicExch(counters, 0);
                        atomicExch(counters + 1, 0);
                    }
                }
                continue;
            }
            for (int c0 = 0; c0 < BN; c0 += 32) {
                const int col0 = n0 + c0;
                if (col0 >= N) break;
                uint32_t r[32];
                const bool wide = (c0 + 32 <= BN);
                if (wide) {
                    ptx::tmem_ld_32(tacc + (uint32_t)c0, r);
                } else {
                    uint32_t r16[16];
                    ptx::tmem_ld_16(tacc + (uint32_t)c0, r16);
#pragma unroll
                    for (int j = 0; j < 16; ++j) { r[j] = r16[j]; r[16 + j] = 0; }
                }
                ptx::tmem_ld_wait();
                if (valid) {
                    uint4 hold = make_uint4(0, 0, 0, 0);
#pragma unroll
                    for (int h = 0; h < 4; ++h) {
                        const int colh = col0 + 8 * h;
                        if (colh >= N || c0 + 8 * h >= BN) break;      // the tile's last chunk may be 16 columns wide
                        float v[8];
#pragma unroll
                        for (int j = 0; j < 8; ++j) v[j] = __uint_as_float(r[8 * h + j]) + sbias[c0 + 8 * h + j];
                        if (RESIDUAL) {                        // a separate instance: even an untaken branch here costs the plain path 3 %
                            float res[8];
                            load_residual8(a.residual, yoff + colh, N - colh, a.vec_out, res);
#pragma unroll
                            for (int j = 0; j < 8; ++j) v[j] += res[j];
                        }
                        if (SILU) {
#pragma unroll
                            for (int j = 0; j < 8; ++j) v[j] = silu(v[j]);
                        } else if (a.relu) {
#pragma unroll
                            for (int j = 0; j < 8; ++j) v[j] = fmaxf(v[j], 0.f);
                        }
                        if (F32) {
                            float* yf = reinterpret_cast<float*>(a.y) + yoff + colh;
                            if (a.vec_out) {                   // C_out % 4 == 0: the row ends on a 16-byte boundary
                                *reinterpret_cast<float4*>(yf) = make_float4(v[0], v[1], v[2], v[3]);
                                if (colh + 4 < N) *reinterpret_cast<float4*>(yf + 4) = make_float4(v[4], v[5], v[6], v[7]);
                            } else {
#pragma unroll
                                for (int j = 0; j < 8; ++j)
                                    if (colh + j < N) yf[j] = v[j];
                            }
                        } else if (a.vec_out) {
                            uint4 o;
                            o.x = pack_bf16(v[0], v[1]);
                            o.y = pack_bf16(v[2], v[3]);
                            o.z = pack_bf16(v[4], v[5]);
                            o.w = pack_bf16(v[6], v[7]);
                            if (a.st32) {              // C_out % 16 == 0: chunks come in pairs, one whole sector per store
                                if (h & 1) ptx::st_global_v8(y2 + yoff + colh - 8, hold, o);
                                else hold = o;
                            } else {
                                *reinterpret_cast<uint4*>(y2 + yoff + colh) = o;
                            }
                        } else {
#pragma unroll
                            for (int j = 0; j < 8; ++j)
                                if (colh + j < N) y2[yoff + colh + j] = __bfloat16_as_ushort(__float2bfloat16_rn(v[j]));
                        }
                    }
                }
            }
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&sh->acc_empty[buf]));
        }
    } else if (warp >= WARP_ZERO0 && a.out_compact) {
        // a compact output has no dropped rows
    } else if (warp >= WARP_ZERO0) {   // (the row-coordinate warp was handled above)
        // ------------------------------------------------------------------ zeros for dropped rows
        zero_fill_dropped_rows<F32, NUM_ZERO_WARPS * 32>(a.y, a.mask, g, a.vec_out, (warp - WARP_ZERO0) * 32 + lane);
    } else {
        // ------------------------------------------------------------------ gather producers
        // Two groups of eight warps take the pipeline stages in turn (stage it belongs to group
        // it % 2); within a group each warp owns 16 of the tile's 128 rows.  The rows' coordinates
        // are read from the shared-memory ring once per tile; the k loop then only forms addresses
        // and issues copies whose completion is reported to the stage's mbarrier asynchronously, so
        // the warps run ahead of the tensor core by up to S stages.  With narrow tiles the loop is
        // bound by how fast one warp gets through an iteration, hence the two groups.
        const int pw = warp - WARP_PROD0;
        const int grp = pw / GROUP_WARPS, pwg = pw - grp * GROUP_WARPS;
        const uint8_t* xb = reinterpret_cast<const uint8_t*>(a.x);
        if (MODE == GATHER_TMA) {
            // Lanes 0..3 of each warp run the loop on their own: each fetches four rows per stage
            // with one TMA row gather (one 64-channel slice of one filter tap per stage; padding
            // taps point past the end of the tensor and read zeros).  The bytes are announced to
            // the stage's barrier by the filter thread.  A row gather costs its warp about 100
            // cycles plus 56 per further lane, hence few issuing lanes in many warps.
            if (lane < 4) {
                const int oob = IN_COMPACT ? g.Nb * a.in_kept : g.Nb * g.H * g.W;
                int s = 0, j = 0, it = 0;
                uint32_t ph = 0;
                bool ok = true;
                for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, ++j) {
                    const int r = j & (INFO_RING - 1);
                    if (!wait_bar<100>(ptx::smem_u32(&sh->info_full[r]), (uint32_t)(j / INFO_RING) & 1u, abort_flag, a.dev_status)) break;
                    const int2* info = sh->rowinfo[r] + 16 * pwg + 4 * lane;
                    const int4 ra = *reinterpret_cast<const int4*>(info);
                    const int4 rb = *reinterpret_cast<const int4*>(info + 2);
                    const int pix[4] = {ra.x, ra.z, rb.x, rb.z}, yx[4] = {ra.y, ra.w, rb.y, rb.w};
                    __syncwarp(0xfu);
                    if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&sh->info_empty[r]));    // the ring slot is in registers now
                    const Item item = item_of(t, KB, a);
                    int ky = 0, kx = 0, ci = 0;
                    if (item.kb_lo != 0) {                 // a later k share starts inside the window
                        const int tap = item.kb_lo * BKE / g.C_in;
                        ci = item.kb_lo * BKE - tap * g.C_in;
                        ky = tap / g.kw;
                        kx = tap - ky * g.kw;
                    }
                    // Compact input: the rank of every tap's input position comes from a table in global
                    // memory.  Looked up right in front of the row gather that needs it, the load's latency
                    // (the table competes with everything else for the little L1 the stages leave) sat in the
                    // issuing lane's serial loop; so the ranks of this lane's NEXT k-block are requested right
                    // after a gather is issued and arrive while the lane waits for the stage after that.
                    int rn[4] = {-1, -1, -1, -1};
                    auto request_ranks = [&](int kbn) {
                        const int tapn = (int)fd_div((uint32_t)(kbn * BKE), a.fdCin);
                        const int kyn = (int)fd_div((uint32_t)tapn, a.fdkw), kxn = tapn - kyn * g.kw;
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const int iy = (yx[i] >> 16) + kyn, ix = (int)(short)(yx[i] & 0xffff) + kxn;
                            const bool in = (unsigned)iy < (unsigned)g.H && (unsigned)ix < (unsigned)g.W;
                            rn[i] = in ? __ldg(a.in_rank + iy * g.W + ix) : -1;
                        }
                    };
                    if (IN_COMPACT) {
                        const int kb0 = item.kb_lo + (((it & 1) == grp) ? 0 : 1);       // this lane's first k-block of the tile
                        if (kb0 < item.kb_hi) request_ranks(kb0);
                    }
                    for (int kb = item.kb_lo; kb < item.kb_hi; ++kb, ++it) {
                        if ((it & 1) == grp) {
                            const int koff = ky * g.W + kx;
                            int idx[4];
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                if (!IN_COMPACT) {
                                    const int iy = (yx[i] >> 16) + ky, ix = (int)(short)(yx[i] & 0xffff) + kx;
                                    const bool in = (unsigned)iy < (unsigned)g.H && (unsigned)ix < (unsigned)g.W;
                                    idx[i] = in ? pix[i] + koff : oob;
                                } else {               // compact input: a dropped position reads zeros like padding
                                    idx[i] = rn[i] >= 0 ? pix[i] + rn[i] : oob;
                                }
                            }
                            if (!wait_bar<20>(ptx::smem_u32(&sh->empty[s]), ph ^ 1u, abort_flag, a.dev_status)) { ok = false; break; }
                            ptx::tma_gather4_2d(smem_base + s * stage_bytes + (uint32_t)(16 * pwg + 4 * lane) * 128u, &tmap_x,
                                                ptx::smem_u32(&sh->full[s]), ci, idx[0], idx[1], idx[2], idx[3]);
                            if (IN_COMPACT && kb + 2 < item.kb_hi) request_ranks(kb + 2);
                        }
                        ci += BKE;                         // next 128 bytes of channels, or the next tap
                        if (ci >= g.C_in) {
                            ci = 0;
                            if (++kx == g.kw) { kx = 0; ++ky; }
                        }
                        if (++s == S) { s = 0; ph ^= 1u; }
                    }
                }
            }
            __syncwarp();
        } else {
            const int c = lane & 7;                        // 16-byte chunk of the 128-byte row
            const int rq = lane >> 3;                      // rows 16pwg + rq + {0,4,8,12}
            // A group owns every second k-block of the whole launch, so its loop steps by two
            // k-blocks: 128 K elements = adv_tap filter taps and adv_ci channels.
            const int adv_tap = (2 * BKE) / g.C_in, adv_ci = (2 * BKE) - adv_tap * g.C_in;
            // destination of this lane's chunk inside a stage: rows rq, rq + 8 share a swizzle
            // phase, rows rq + 4, rq + 12 the other
            const uint32_t dst_a = (uint32_t)((16 * pwg + rq) * 128 + ((c ^ rq) << 4));
            const uint32_t dst_b = (uint32_t)((16 * pwg + rq + 4) * 128 + ((c ^ (rq + 4)) << 4));
            int j = 0;
            uint32_t it0 = 0;                              // k-blocks of the launch before this tile
            bool ok = true;
            for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, ++j) {
                const int r = j & (INFO_RING - 1);
                if (!warp_wait_bar<100>(ptx::smem_u32(&sh->info_full[r]), (uint32_t)(j / INFO_RING) & 1u, abort_flag, a.dev_status)) break;
                const int2* info = sh->rowinfo[r] + 16 * pwg;
                int base[4], yx[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int2 ri = info[rq + 4 * i];
                    base[i] = ri.x * g.C_in;               // element offset of the window's corner
                    yx[i] = ri.y;
                }
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&sh->info_empty[r]));    // the ring slot is in registers now

                const Item item = item_of(t, KB, a);
                const int kb0 = item.kb_lo + (int)((it0 ^ (uint32_t)grp) & 1u);          // this group's first k-block of the tile
                // window position (filter tap, channel) of this lane's chunk in k-block kb0
                int tap, ci;
                {
                    const int k_first = kb0 * BKE + c * EPC;
                    tap = (int)fd_div((uint32_t)k_first, a.fdCin);
                    ci = k_first - tap * g.C_in;
                }
                uint32_t itk = it0 + (uint32_t)(kb0 - item.kb_lo);
                for (int kb = kb0; kb < item.kb_hi; kb += 2, itk += 2) {
                    const int ky = (int)fd_div((uint32_t)tap, a.fdkw), kx = tap - ky * g.kw;
                    const bool kvalid = ky < g.kh;         // past K: the window is exhausted
                    const int tapoff = (ky * g.W + kx) * g.C_in + ci;
                    const uint32_t lap = fd_div(itk, a.fdS);
                    const int s = (int)(itk - lap * (uint32_t)S);
                    if (!warp_wait_bar<40>(ptx::smem_u32(&sh->empty[s]), (lap & 1u) ^ 1u, abort_flag, a.dev_status)) { ok = false; break; }
                    const uint32_t stage = smem_base + s * stage_bytes;
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int iy = (yx[i] >> 16) + ky, ix = (int)(short)(yx[i] & 0xffff) + kx;
                        bool in = kvalid && (unsigned)iy < (unsigned)g.H && (unsigned)ix < (unsigned)g.W;
                        int off = base[i] + tapoff;
                        if (IN_COMPACT) {                      // compact input: base is the image's first row
                            const int rnk = in ? __ldg(a.in_rank + iy * g.W + ix) : -1;
                            in = rnk >= 0;
                            off = base[i] + rnk * g.C_in + ci;
                        }
                        ptx::cp_async_16(stage + ((i & 1) ? dst_b : dst_a) + (uint32_t)((i >> 1) * 1024),
                                         xb + (in ? (long long)off * ES : 0), in ? 16u : 0u);
                    }
                    ptx::cp_async_mbar_arrive_noinc(ptx::smem_u32(&sh->full[s]));
                    tap += adv_tap;
                    ci += adv_ci;
                    if (ci >= g.C_in) { ci -= g.C_in; ++tap; }
                }
                it0 += (uint32_t)(item.kb_hi - item.kb_lo);
            }
            ptx::cp_async_wait<0>();              // nothing of this thread is in flight at exit
        }
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == WARP_MMA) {
        __syncwarp();
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, (uint32_t)a.tmem_cols);
    }
}

// Channel padding: src[rows][C] -> dst[rows][Cp] with zeros in the added channels, Cp = 4 or a
// multiple of 8.  Used for inputs and filters whose channel count is not a multiple of 8, so that
// the gather can work in 16-byte chunks.  One thread per 16-byte chunk (8 elements) of dst.
__global__ void pad_channels_kernel(const unsigned short* __restrict__ src, uint4* __restrict__ dst,
                                    long long rows, int C, int Cp)
{
    ptx::grid_launch_dependents();
    ptx::grid_dependency_wait();
    const long long total = rows * Cp / 8;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        long long row = (i * 8) / Cp;
        int c = (int)((i * 8) - row * Cp);
        unsigned short e[8];
#pragma unroll
        for (int q2 = 0; q2 < 8; ++q2) {
            e[q2] = (c < C) ? __ldcg(src + row * C + c) : (unsigned short)0;     // past L1, like everything an earlier kernel may have written
            if (++c == Cp) { c = 0; ++row; }
        }
        uint4 v;
        v.x = e[0] | ((uint32_t)e[1] << 16);
        v.y = e[2] | ((uint32_t)e[3] << 16);
        v.z = e[4] | ((uint32_t)e[5] << 16);
        v.w = e[6] | ((uint32_t)e[7] << 16);
        dst[i] = v;
    }
}

// Filters of the pixel-pair form (see asx_run): one thread per output element.
__global__ void pack_pair_filters_kernel(const unsigned short* __restrict__ w, unsigned short* __restrict__ w2,
                                         int C_out, int kh, int kw, int C, int kw2, int shift)
{
    ptx::grid_launch_dependents();
    ptx::grid_dependency_wait();
    const long long total = (long long)C_out * kh * kw2 * 8;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        const int c = (int)(i & 3), j = (int)((i >> 2) & 1);
        long long rest = i >> 3;
        const int kxx = (int)(rest % kw2); rest /= kw2;
        const int ky = (int)(rest % kh);
        const int co = (int)(rest / kh);
        const int kx = 2 * kxx + j - shift;
        w2[i] = (kx >= 0 && kx < kw && c < C) ? w[(((long long)co * kh + ky) * kw + kx) * C + c] : (unsigned short)0;
    }
}

// Filters of the 2x2-block form: w2[co][ky2][kx2][r][px][4] = w[co][2 ky2 + r - shift][2 kx2 + px - shift][c],
// zero outside the filter and for c >= C.  kx2 runs over 4 blocks (one 128-byte run of the input per
// filter block row).  One thread per output element, `nthreads` threads of which this is number `t`.
__device__ __forceinline__ void pack_block_filters(const unsigned short* __restrict__ w, unsigned short* __restrict__ w2,
                                                   int C_out, int kh, int kw, int C, int kh2, int shift, int t, int nthreads)
{
    const int total = C_out * kh2 * 64;
    for (int i = t; i < total; i += nthreads) {
        const int c = i & 3, px = (i >> 2) & 1, r = (i >> 3) & 1, kx2 = (i >> 4) & 3;
        const int rest = i >> 6;
        const int ky2 = rest % kh2, co = rest / kh2;
        const int ky = 2 * ky2 + r - shift, kx = 2 * kx2 + px - shift;
        w2[i] = (ky >= 0 && ky < kh && kx >= 0 && kx < kw && c < C) ? w[(((long long)co * kh + ky) * kw + kx) * C + c]
                                                                     : (unsigned short)0;
    }
}

// Input of the 2x2-block form (see asx_run): xs[n][ys][xs][r][px][4] holds the 2x2 pixel block
// whose top-left pixel is (2 (ys - h0), 2 (xs - h0)), channels padded to 4, zeros outside the image.
// Block (ys, n) of the grid writes one staged row, one thread per 2x2 block (32 bytes), so that nothing
// divides; the blocks with n = Nb pack the filters instead (the same launch does both).
__global__ void __launch_bounds__(128) stage_blocks2x2_kernel(const unsigned short* __restrict__ x, uint4* __restrict__ xs, int Nb, int H, int W,
                                                              int C, int Hs, int Ws, int h0, const unsigned short* __restrict__ w,
                                                              unsigned short* __restrict__ w2, int C_out, int kh, int kw, int kh2, int shift)
{
    ptx::grid_launch_dependents();
    ptx::grid_dependency_wait();
    const int by = blockIdx.x, n = blockIdx.y;
    if (n == Nb) {
        pack_block_filters(w, w2, C_out, kh, kw, C, kh2, shift, by * blockDim.x + threadIdx.x, gridDim.x * blockDim.x);
        return;
    }
    const long long row0 = ((long long)n * Hs + by) * Ws;
    const bool words = (C == 3 && (reinterpret_cast<uintptr_t>(x) & 3) == 0);
    if (words && (reinterpret_cast<uintptr_t>(x) & 7) == 0 && (h0 & 1) == 0 && (W & 3) == 0 && (Ws & 1) == 0) {
        // three channels, two blocks per thread: the four pixels of a block-row pair are 24 contiguous bytes at an
        // 8-byte aligned offset (first column a multiple of 4, W a multiple of 4), i.e. three 64-bit loads per image row
        for (int bp = threadIdx.x; 2 * bp < Ws; bp += blockDim.x) {
            const int bx = 2 * bp;
            uint4 o[2][2];                      // [block][image row]
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                const int iy = 2 * (by - h0) + r, ix = 2 * (bx - h0);
                const bool in = iy >= 0 && iy < H && ix >= 0 && ix < W;       // ix and W are multiples of 4: all four pixels or none
                uint2 q0 = make_uint2(0, 0), q1 = q0, q2 = q0;
                if (in) {
                    const uint2* src = reinterpret_cast<const uint2*>(x + (((long long)n * H + iy) * W + ix) * 3);
                    q0 = __ldcg(src); q1 = __ldcg(src + 1); q2 = __ldcg(src + 2);
                }
                // 12 values p0c0 p0c1 p0c2 p1c0 | p1c1 p1c2 p2c0 p2c1 | p2c2 p3c0 p3c1 p3c2 -> two blocks of (px0 c0..2 0, px1 c0..2 0)
                o[0][r] = make_uint4(q0.x, q0.y & 0xffffu, (q0.y >> 16) | (q1.x << 16), q1.x >> 16);
                o[1][r] = make_uint4(q1.y, q2.x & 0xffffu, (q2.x >> 16) | (q2.y << 16), q2.y >> 16);
            }
            uint4* dst = xs + 2 * (row0 + bx);
            dst[0] = o[0][0]; dst[1] = o[0][1]; dst[2] = o[1][0]; dst[3] = o[1][1];
        }
        return;
    }
    for (int bx = threadIdx.x; bx < Ws; bx += blockDim.x) {
        unsigned short v[16];
        if (words) {
            // three channels: the two pixels of a block row are 12 contiguous bytes at a 4-byte
            // aligned offset (the block's first column is even), i.e. three 32-bit loads
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                const int iy = 2 * (by - h0) + r, ix = 2 * (bx - h0);
                const bool in = iy >= 0 && iy < H && ix >= 0 && ix < W;       // W is even: both pixels or none
                uint32_t q0 = 0, q1 = 0, q2 = 0;
                if (in) {
                    const uint32_t* src = reinterpret_cast<const uint32_t*>(x + (((long long)n * H + iy) * W + ix) * 3);
                    q0 = __ldcg(src); q1 = __ldcg(src + 1); q2 = __ldcg(src + 2);
                }
                v[r * 8 + 0] = (unsigned short)(q0 & 0xffffu); v[r * 8 + 1] = (unsigned short)(q0 >> 16);
                v[r * 8 + 2] = (unsigned short)(q1 & 0xffffu); v[r * 8 + 3] = 0;
                v[r * 8 + 4] = (unsigned short)(q1 >> 16);     v[r * 8 + 5] = (unsigned short)(q2 & 0xffffu);
                v[r * 8 + 6] = (unsigned short)(q2 >> 16);     v[r * 8 + 7] = 0;
            }
        } else {
#pragma unroll
            for (int r = 0; r < 2; ++r)
#pragma unroll
                for (int px = 0; px < 2; ++px) {
                    const int iy = 2 * (by - h0) + r, ix = 2 * (bx - h0) + px;
                    const bool in = iy >= 0 && iy < H && ix >= 0 && ix < W;
                    const unsigned short* src = x + (((long long)n * H + (in ? iy : 0)) * W + (in ? ix : 0)) * C;
#pragma unroll
                    for (int c = 0; c < 4; ++c) v[(r * 2 + px) * 4 + c] = (in && c < C) ? __ldcg(src + c) : (unsigned short)0;
                }
        }
        uint4 lo, hi;
        lo.x = v[0] | ((uint32_t)v[1] << 16); lo.y = v[2] | ((uint32_t)v[3] << 16);
        lo.z = v[4] | ((uint32_t)v[5] << 16); lo.w = v[6] | ((uint32_t)v[7] << 16);
        hi.x = v[8] | ((uint32_t)v[9] << 16); hi.y = v[10] | ((uint32_t)v[11] << 16);
        hi.z = v[12] | ((uint32_t)v[13] << 16); hi.w = v[14] | ((uint32_t)v[15] << 16);
        xs[2 * (row0 + bx)] = lo;
        xs[2 * (row0 + bx) + 1] = hi;
    }
}

}  // namespace

bool plan_fast(const ConvGeom& g, int num_sms, long long est_kept_rows, int fused_list_rows, bool allow_split, int elem_bytes,
               FastPlan* plan)
{
    const int N = g.C_out;
    const int bke = 128 / elem_bytes;             // K elements per stage: 64 bf16 or 32 fp32
    const int KB = (g.K + bke - 1) / bke;
    const long long m_tiles = (est_kept_rows + BM - 1) / BM > 0 ? (est_kept_rows + BM - 1) / BM : 1;
    // Tile width and k shares.  A wider tile does more work per gathered byte, a narrower one
    // gives more tiles when a layer has few kept rows, and sharing a tile's k-blocks between
    // blocks gives more work items still, at the price of exchanging fp32 partial tiles.  Pick
    // the pair with the lowest estimated time, from figures measured on B200: a 64-wide k-block
    // of a 128 x BN tile takes about 0.30 + 0.001 BN microseconds (the loop is bound by the TMA
    // requests and bytes one SM can pull from L2: 16 KB of gathered rows in 32 requests of about
    // 13 clocks, plus the BN x 128-byte filter slab), the last tile's epilogue about 0.012 BN,
    // and the exchange of partial tiles about 7 + 0.025 BN (a chain of write, fence, counter and
    // read latencies).  Sharing pays where there are far fewer tiles than SMs and K is long.
    int best_BN = 0, best_KS = 1;
    double best_cost = 0.0;
    for (int n_tiles = (N + 255) / 256; ; n_tiles *= 2) {
        const int per = (N + n_tiles - 1) / n_tiles;
        const int BN = ((per + 15) / 16) * 16;
        const int nt = (N + BN - 1) / BN;
        const double t_kb = 0.30 + 0.001 * BN;                                // microseconds
        for (int KS = 1; KS <= (allow_split ? 8 : 1); ++KS) {
            if (KS > 1 && KB / KS < 4) break;
            const long long items = m_tiles * nt * KS;
            const long long waves = (items + num_sms - 1) / num_sms;
            const int kbi = (KB + KS - 1) / KS;
            const double cost = (double)waves * (kbi * t_kb + 0.3) + 0.012 * BN + (KS > 1 ? 7.0 + 0.025 * BN : 0.0);
            if (best_BN == 0 || cost < best_cost * 0.97) { best_BN = BN; best_KS = KS; best_cost = cost; }
        }
        if (BN <= 64) break;
    }
    const int BN = best_BN;
    const int n_tiles = (N + BN - 1) / BN;
    const int stage_bytes = A_STAGE_BYTES + BN * BK * 2;
    const int list_bytes = (fused_list_rows * 2 + 15) / 16 * 16;     // 16-bit kept list of the fused compaction
    const int budget = 227 * 1024 - 1024 - (int)sizeof(Shared) - list_bytes;
    int S = budget / stage_bytes;
    if (S > MAX_STAGES) S = MAX_STAGES;
    if (S < MIN_STAGES) return false;
    plan->BN = BN;
    plan->n_tiles = n_tiles;
    plan->ksplit = best_KS;
    plan->est_cost_us = best_cost;
    plan->ws_items = (long long)m_tiles * n_tiles * best_KS;
    plan->stages = S;
    int smem = 1024 + S * stage_bytes + (int)sizeof(Shared) + list_bytes;
    if (smem < 120 * 1024) smem = 120 * 1024;      // one block per SM: tensor memory is not shared out
    plan->smem_bytes = smem;
    if (g.C_in % (16 / elem_bytes) != 0) return false;      // the caller pads the channels first
    plan->vec = (g.C_in % bke == 0) ? GATHER_TMA : GATHER_CPASYNC;
    return true;
}

cudaError_t launch_fast(const ConvGeom& g, const FastPlan& plan, const CUtensorMap& tmap_w,
                        const CUtensorMap& tmap_x, const void* x, const float* bias, void* y, const uint8_t* mask,
                        const int32_t* kept, const int32_t* count, int relu, int* dev_status,
                        int num_sms, int fuse_compact, long long host_kept, float* ws_partial, int* ws_counters,
                        int out_compact, const int32_t* in_rank, int in_kept, const void* residual, int f32, int wait_limit_kcycles,
                        cudaStream_t st)
{
    if (f32 && (in_rank != nullptr || residual != nullptr || plan.ksplit != 1)) return cudaErrorInvalidValue;
    FastArgs a;
    a.fdcnt_host = make_fastdiv((uint32_t)(host_kept > 0 && host_kept < (1ll << 31) ? host_kept : 1));
    if (!(host_kept > 0 && host_kept < (1ll << 31))) a.fdcnt_host.d = 0;
    a.fuse_compact = fuse_compact;
    a.kept_out = const_cast<int32_t*>(kept);
    a.count_out = const_cast<int32_t*>(count);
    a.x = static_cast<const __nv_bfloat16*>(x);
    a.bias = bias;
    a.y = static_cast<__nv_bfloat16*>(y);
    a.mask = mask;
    a.kept = kept;
    a.count = count;
    a.dev_status = dev_status;
    a.relu = relu == 1 ? 1 : 0;
    a.out_compact = out_compact;
    a.residual = static_cast<const __nv_bfloat16*>(residual);
    a.in_rank = in_rank;
    a.in_kept = in_kept;
    a.BN = plan.BN;
    a.fdP = make_fastdiv((uint32_t)g.P);
    a.fdWo = make_fastdiv((uint32_t)g.Wo);
    a.n_tiles = plan.n_tiles;
    a.fdNt = make_fastdiv((uint32_t)plan.n_tiles);
    a.ksplit = plan.ksplit;
    a.fdCin = make_fastdiv((uint32_t)g.C_in);
    a.fdkw = make_fastdiv((uint32_t)g.kw);
    a.fdS = make_fastdiv((uint32_t)plan.stages);
    a.fdKs = make_fastdiv((uint32_t)plan.ksplit);
    a.ws_partial = ws_partial;
    a.ws_counters = ws_counters;
    a.ws_items = (int)plan.ws_items;
    a.wait_limit_kcycles = wait_limit_kcycles > 0 ? wait_limit_kcycles : WAIT_LIMIT_KCYCLES_DEFAULT;
    a.stages = plan.stages;
    int cols = 32;
    while (cols < 2 * plan.BN) cols <<= 1;
    a.tmem_cols = cols;
    a.vec_out = (g.C_out % (f32 ? 4 : 8) == 0 && (reinterpret_cast<uintptr_t>(y) & 15) == 0) ? 1 : 0;
    // Whole-sector stores pay where the epilogue's stores pace the kernel: few k-blocks per tile (the network's
    // first layers, 1x1 convolutions) and rows that are written without a residual read in between.
    a.st32 = (!f32 && a.vec_out && g.C_out % 16 == 0 && plan.BN % 16 == 0 && (reinterpret_cast<uintptr_t>(y) & 31) == 0 &&
              plan.ksplit == 1 && out_compact == 0) ? 1 : 0;

    long long tiles = ((long long)g.M + BM - 1) / BM * plan.n_tiles * plan.ksplit;
    int grid = (int)(tiles < num_sms ? tiles : num_sms);
    if (grid < 1) grid = 1;
    const int variant = plan.vec + (in_rank != nullptr ? 2 : 0);      // 1, 2: dense input; 3, 4: compact input
    const bool has_res = residual != nullptr, is_silu = relu == 2;
    using Kern = void (*)(const CUtensorMap, const CUtensorMap, const ConvGeom, const FastArgs);
    Kern kern = nullptr;
#define ASX_PICK(MODE, IC)                                                                                          \
    kern = has_res ? (is_silu ? masked_conv_sm100_kernel<MODE, IC, true, true, false> : masked_conv_sm100_kernel<MODE, IC, true, false, false>) \
                   : (is_silu ? masked_conv_sm100_kernel<MODE, IC, false, true, false> : masked_conv_sm100_kernel<MODE, IC, false, false, false>)
    if (f32) {      // fp32 storage: dense input, no residual
        if (variant == 2) kern = is_silu ? masked_conv_sm100_kernel<GATHER_TMA, false, false, true, true> : masked_conv_sm100_kernel<GATHER_TMA, false, false, false, true>;
        else kern = is_silu ? masked_conv_sm100_kernel<GATHER_CPASYNC, false, false, true, true> : masked_conv_sm100_kernel<GATHER_CPASYNC, false, false, false, true>;
    }
    else if (variant == 2) { ASX_PICK(GATHER_TMA, false); }
    else if (variant == 1) { ASX_PICK(GATHER_CPASYNC, false); }
    else if (variant == 4) { ASX_PICK(GATHER_TMA, true); }
    else { ASX_PICK(GATHER_CPASYNC, true); }
#undef ASX_PICK
    static int smem_set_all[40] = {0};          // largest dynamic shared memory size enabled so far, per instance
    int* smem_set = smem_set_all + (has_res ? 5 : 0) + (is_silu ? 10 : 0) + (f32 ? 20 : 0);
    if (plan.smem_bytes > smem_set[variant]) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, plan.smem_bytes);
        if (e != cudaSuccess) return e;
        smem_set[variant] = plan.smem_bytes;
    }
    return launch_pdl(kern, dim3(grid), dim3(NUM_THREADS), (size_t)plan.smem_bytes, st, tmap_w, tmap_x, g, a);
}

cudaError_t launch_pad_channels(const void* src, void* dst, long long rows, int C, int Cp, cudaStream_t st)
{
    const long long total = rows * Cp / 8;
    int blocks = (int)((total + 255) / 256 < 148 * 16 ? (total + 255) / 256 : 148 * 16);
    if (blocks < 1) blocks = 1;
    return launch_pdl(pad_channels_kernel, dim3(blocks), dim3(256), 0, st, static_cast<const unsigned short*>(src),
                      static_cast<uint4*>(dst), rows, C, Cp);
}

cudaError_t launch_pack_pair_filters(const void* w, void* w2, int C_out, int kh, int kw, int C, int kw2, int shift,
                                     cudaStream_t st)
{
    const long long total = (long long)C_out * kh * kw2 * 8;
    int blocks = (int)((total + 255) / 256 < 1024 ? (total + 255) / 256 : 1024);
    if (blocks < 1) blocks = 1;
    return launch_pdl(pack_pair_filters_kernel, dim3(blocks), dim3(256), 0, st, static_cast<const unsigned short*>(w),
                      static_cast<unsigned short*>(w2), C_out, kh, kw, C, kw2, shift);
}

cudaError_t launch_stage_blocks2x2(const void* x, void* xs, int Nb, int H, int W, int C, int Hs, int Ws, int h0,
                                   const void* w, void* w2, int C_out, int kh, int kw, int kh2, int shift, cudaStream_t st)
{
    if (Hs < 1 || Nb < 1 || Nb >= 65535 || (long long)C_out * kh2 * 64 >= (1ll << 31)) return cudaErrorInvalidValue;
    return launch_pdl(stage_blocks2x2_kernel, dim3(Hs, Nb + 1), dim3(128), 0, st, static_cast<const unsigned short*>(x),
                      static_cast<uint4*>(xs), Nb, H, W, C, Hs, Ws, h0, static_cast<const unsigned short*>(w),
                      static_cast<unsigned short*>(w2), C_out, kh, kw, kh2, shift);
}

}  // namespace asx
