// S2 + S3 + S4 for multi-tap stride-1 layers — the window-patch form of the fused kernel.
//
// Section 3 lowers a convolution to a matrix with one row of k*k*c values per sliding window, and
// Section 3.2 / Appendix A skip the masked windows while building it.  Neighbouring windows overlap
// (Section 3.1, Fig. 2: a pixel masked in one window is still live in the next), so gathering every
// filter tap of every kept row separately moves each input pixel up to kh*kw times from L2 into the
// SM.  Here the kept rows of a tile are consecutive entries of an ascending list, so all their
// windows lie in one contiguous range of zero-padded input rows.  That range (the tile's "patch")
// is loaded ONCE per 64-channel slice into shared memory with large TMA boxes, and the A operand of
// the tensor core is built from it in TENSOR MEMORY: for every filter tap, thread r of a fill warp
// reads the 128 bytes of row r's tap pixel from the patch and writes them to lane r of an A stage
// with tcgen05.st; tcgen05.mma then takes A from tensor memory and only the filter slab from shared
// memory.  Shared memory carries the patch once and the filter slab, not a repacked A tile.
//
//   patch thread    TMA: one box of (64 channels x padded row width) per input row of the patch;
//                   rows above/below the image and the left/right border are out-of-range
//                   coordinates and arrive as zeros (the convolution's zero padding).
//   filter thread   TMA: the BN x 64 slab of w[C_out][K] of each k-block (a tap of a slice).
//   fill warps      16 warps = 4 groups; group (stage mod 4) fills the A stage.
//   MMA thread      tcgen05.mma 128 x BN x 16, A from tensor memory, accumulators double buffered.
//
// A pipeline stage is a CHUNK of up to G filter taps of one slice (a filter row for 3x3), i.e. G
// k-blocks of 64: one thread issues every tcgen05.mma, and its per-stage cost (two barrier waits, two
// commits, each a shared-memory round trip of 150-250 clocks) is as long as the four instructions of a
// k-block take on the tensor core at BN = 64; with three k-blocks per stage it is paid once per twelve.
//   epilogue warps  bias, activation, bf16, 16-byte stores at the kept rows' NHWC positions.
//   zero warps      zeros for the dropped rows.  Every output element is written exactly once.
//
// Tiles are cut on the host, which knows the mask: consecutive kept rows, at most 128, as long as
// their windows span no more input rows than a patch buffer holds (a tile with fewer rows leaves
// lanes of the tensor core idle; the host weighs that against the row-gather form).  The kernel
// checks each tile again and reports a status word instead of running past a buffer.  All waits are
// bounded.
#include <cuda_bf16.h>
#include "asx_internal.h"
#include "ptx_sm100.cuh"
#include "conv_common.cuh"

namespace asx {

namespace {

constexpr int BM = 128;                 // kept rows per tile (UMMA M)
constexpr int INFO_RING = 8;            // tiles whose row coordinates are kept in shared memory (power of two)
constexpr int MAX_B_STAGES = 8;
constexpr int MAX_A_STAGES = 12;
constexpr int TAP_COLS = 32;            // 64 bf16 per row = 32 columns of tensor memory per filter tap
constexpr int MAX_P_BUFS = 4;           // patch buffers: two, or four where four still hold a tile's rows each
constexpr int FULL_RING = 24;           // 'stage full' barriers: a multiple of every A and filter ring depth in use (2, 3, 4)
// Warp roles.  The two loader warps come last: they take no part in the mask compaction and the row
// decoding (threads 0 .. WORK_THREADS-1 do, meeting on hardware barrier 2) but start fetching filter
// slabs and input patches as soon as the barriers exist, from the tile table the host cut.
constexpr int W_MMA = 0, W_INFO = 1, W_EPI0 = 2, NUM_EPI_WARPS = 4, W_ZERO_A = 6, W_FILL0 = 8, NUM_FILL_WARPS = 16,
              W_ZERO_B = 24, NUM_ZERO_WARPS = 4, W_FILTER = 26, W_PATCH = 27;
constexpr int WORK_THREADS = 32 * W_FILTER;
constexpr int NUM_THREADS = 32 * (W_PATCH + 1);
static_assert(NUM_THREADS / 32 < 32, "the fused compaction keeps its running count in slot 31 of the warp totals");
static_assert((W_FILL0 & 3) == 0 && (NUM_FILL_WARPS & 3) == 0, "fill warps come in groups of four lane quarters");

struct PatchArgs {
    FastDiv fdP, fdWo;           // divisions by P and Wo
    FastDiv fdNt;                // division by n_tiles
    FastDiv fdHp;                // division by the padded input height
    FastDiv fdcnt_host;          // division by the kept count when the host knows it (d = 0: it does not)
    const float* bias;
    __nv_bfloat16* y;
    const uint8_t* mask;
    const int32_t* kept;
    const int32_t* count;
    int* dev_status;
    int relu;
    int out_compact;    // y holds the kept rows only, in kept order (row rk at y[rk][*]); nothing is zero-filled
    int st32;           // 32-byte epilogue stores: C_out % 16 == 0, BN % 16 == 0 and y 32-byte aligned
    int BN, n_tiles, b_stages, a_stages;
    int cap_rows;       // padded input rows one patch buffer holds
    int p_bufs_log2;    // 1 or 2: two or four patch buffers
    int epi8;           // few k-blocks per tile: the last four fill warps are epilogue warps too (each warp of a lane
                        // quarter's pair takes every other 32-column chunk), three fill groups remain
    int Hp, Wp, Wp8;    // padded input height and width; Wp rounded up to a multiple of 8 (row pitch in pixels)
    int px32;           // 2x2-block form of a network's first layer: a "pixel" is a 32-byte block, a window row is the
                        // 128 bytes of four consecutive blocks (kw = 1), so neighbouring pixels overlap; the patch holds
                        // each block once instead of 128 bytes per pixel: Wp counts the 128-byte units (four blocks) a
                        // row's box has, Wp8 the row pitch in blocks (a multiple of 32: rows start 1024-byte aligned)
    int slices;         // C_in / 64
    int G;              // filter taps per pipeline stage (a chunk); chunks = ceil(kh*kw / G) per slice
    int fuse_compact;   // rebuild the kept-row list from the mask inside this kernel (small masks)
    int32_t* kept_out;
    int32_t* count_out;
    const __nv_bfloat16* residual;
    const int4* tiles;  // per row tile: first kept lowered row, number of rows (1..128), first padded input row of
                        // its patch, patch rows; cut by the host from the mask
    int n_mtiles;       // row tiles
    int Mk_host;        // kept lowered rows the tiles cover; must equal what the device counts
    int wait_limit_kcycles;
};

struct alignas(16) PShared {          // lives after the patch buffers and the filter stages
    int rowpix[INFO_RING][BM];        // per tile row: pixel index of the window's corner within the tile's patch, or -1
    float bias[2][128];
    unsigned long long info_full[INFO_RING];
    unsigned long long info_empty[INFO_RING];
    // One 'full' barrier per pipeline stage, indexed by the stage's number in the launch modulo
    // FULL_RING: the filter slab's bytes and the four fill warps' arrivals complete the same phase, so
    // the issuing thread waits once per stage although the two rings differ in depth.
    unsigned long long full[FULL_RING];
    unsigned long long b_empty[MAX_B_STAGES];
    unsigned long long a_empty[MAX_A_STAGES];
    unsigned long long p_full[MAX_P_BUFS];
    unsigned long long p_empty[MAX_P_BUFS];
    unsigned long long acc_full[2];
    unsigned long long acc_empty[2];
    unsigned int tmem_base;
    WaitCtl ctl;
    int scan_total[32];
};

// Padded input row and column of the window of the rk-th kept lowered row, as one pixel index
// (n Hp + oy) Wp8 + ox: tap (ky, kx) of that row is pixel index + ky Wp8 + kx.  -1 past the end.
__device__ __forceinline__ int row_pixel_of(int rk, int Mk, const FastDiv& fdcnt, const ConvGeom& g, const PatchArgs& a,
                                            const KeptList& kept, int* padded_row)
{
    *padded_row = -1;
    if (rk >= Mk) return -1;
    const int row = out_row_of(rk, fdcnt, g, kept);
    if (row >= g.M) {
        atomicOr(a.dev_status, DEV_BAD_INDEX);
        return -1;
    }
    const int n = (int)fd_div((uint32_t)row, a.fdP), p = row - n * g.P;
    const int oy = (int)fd_div((uint32_t)p, a.fdWo), ox = p - oy * g.Wo;
    *padded_row = n * a.Hp + oy;
    return (n * a.Hp + oy) * a.Wp8 + ox;
}

struct PItem {
    int m_tile, n_tile;
};
__device__ __forceinline__ PItem pitem_of(int t, const PatchArgs& a)
{
    PItem it;
    it.m_tile = (int)fd_div((uint32_t)t, a.fdNt);
    it.n_tile = t - it.m_tile * a.n_tiles;
    return it;
}

// Row coordinates of one tile row into ring slot jj, relative to the tile's patch.
__device__ __forceinline__ void decode_row(PShared* sh, int jj, int rr, int m_tile, int Mk, const FastDiv& fdcnt,
                                           const ConvGeom& g, const PatchArgs& a, const KeptList& kept)
{
    const int4 tl = __ldg(a.tiles + m_tile);            // written by a stream-ordered copy, never by a kernel
    int prow;
    const int px = row_pixel_of(rr < tl.y ? tl.x + rr : Mk, Mk, fdcnt, g, a, kept, &prow);
    // relative to the patch's first pixel; a row whose window the host's patch range does not cover
    // (the table was cut for another mask) is flagged and reads pixel 0
    int rel = -1;
    if (px >= 0) {
        rel = px - tl.z * a.Wp8;
        if (prow < tl.z || prow + g.kh > tl.z + tl.w || tl.w > a.cap_rows) {
            atomicOr(a.dev_status, DEV_BAD_INDEX);
            rel = -1;
        }
    }
    sh->rowpix[jj][rr] = rel;
}

template <bool RESIDUAL, bool SILU>
__global__ void __launch_bounds__(NUM_THREADS, 1)
masked_conv_patch_sm100_kernel(const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ CUtensorMap tmap_x,
                               const ConvGeom g, const PatchArgs a)
{
    extern __shared__ uint8_t smem_raw[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    // Let the next kernel of the stream start its own prologue; everything up to the dependency
    // wait below touches only this block's shared and tensor memory (and the layer's mask, which
    // is only ever written by stream-ordered copies).
    ptx::grid_launch_dependents();
    const int N = g.C_out, BN = a.BN, BS = a.b_stages, AS = a.a_stages;
    const int taps = g.kh * g.kw, G = a.G;
    const int chunks = (taps + G - 1) / G;                            // pipeline stages per slice
    const int NST = chunks * a.slices;                                // pipeline stages per work item
    const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t px_bytes = a.px32 ? 32u : 128u;
    const uint32_t row_bytes = (uint32_t)a.Wp8 * px_bytes;            // one padded input row of one slice
    const uint32_t patch_bytes = ((uint32_t)a.cap_rows * row_bytes + 1023u) & ~1023u;
    const uint32_t PB = 1u << a.p_bufs_log2;                         // patch buffers (2 or 4)
    const uint32_t b_base = smem_base + PB * patch_bytes;
    const uint32_t b_tap_bytes = (uint32_t)BN * 128u;                 // the filter slab of one tap of one slice
    const uint32_t b_stage_bytes = (uint32_t)G * b_tap_bytes;
    const uint32_t a_stage_cols = (uint32_t)(G * TAP_COLS);
    PShared* sh = reinterpret_cast<PShared*>(smem_raw + (smem_base - ptx::smem_u32(smem_raw)) + PB * patch_bytes + (uint32_t)BS * b_stage_bytes);
    volatile WaitCtl* ctl = &sh->ctl;

    uint4 early_mask = make_uint4(0, 0, 0, 0);
    const bool early_ok = a.fuse_compact && tid < WORK_THREADS && tid * 16 + 16 <= g.rows && (reinterpret_cast<uintptr_t>(a.mask) & 15) == 0;
    if (early_ok) early_mask = ptx::ld_global_v4_keep_in_l2(a.mask + tid * 16);

    // barrier initialisation, one barrier per thread (a single thread took about 1500 clocks over them), by the
    // block's last threads, so that warp 0's tensor-memory allocation runs beside it
    {
        constexpr int NB = FULL_RING + MAX_B_STAGES + MAX_A_STAGES + 2 * INFO_RING + 2 * MAX_P_BUFS + 4;
        if (tid >= NUM_THREADS - NB) {
            int i = tid - (NUM_THREADS - NB);
            unsigned long long* bar;
            uint32_t count;
            if (i < FULL_RING) { bar = &sh->full[i]; count = 5; }                        // the filter thread's expect_tx + one arrival per lane quarter
            else if ((i -= FULL_RING) < MAX_B_STAGES) { bar = &sh->b_empty[i]; count = 1; }
            else if ((i -= MAX_B_STAGES) < MAX_A_STAGES) { bar = &sh->a_empty[i]; count = 1; }
            else if ((i -= MAX_A_STAGES) < INFO_RING) { bar = &sh->info_full[i]; count = 1; }
            else if ((i -= INFO_RING) < INFO_RING) { bar = &sh->info_empty[i]; count = a.epi8 ? NUM_FILL_WARPS - 4 : NUM_FILL_WARPS; }
            else if ((i -= INFO_RING) < MAX_P_BUFS) { bar = &sh->p_full[i]; count = 1; }
            else if ((i -= MAX_P_BUFS) < MAX_P_BUFS) { bar = &sh->p_empty[i]; count = a.epi8 ? NUM_FILL_WARPS - 4 : NUM_FILL_WARPS; }
            else if ((i -= MAX_P_BUFS) < 2) { bar = &sh->acc_full[i]; count = 1; }
            else { i -= 2; bar = &sh->acc_empty[i]; count = a.epi8 ? 2 * NUM_EPI_WARPS : NUM_EPI_WARPS; }
            ptx::mbar_init(ptx::smem_u32(bar), count);
            ptx::fence_mbar_init();
        }
        if (tid == 0) {
            sh->ctl.abort = 0;
            sh->ctl.limit_kcycles = a.wait_limit_kcycles;
        }
    }
    if (warp == W_MMA) {
        ptx::tmem_alloc(ptx::smem_u32(&sh->tmem_base), 512u);       // two accumulators and the A stages
        ptx::tmem_relinquish();
    }
    if (warp == W_FILTER && lane == 0) ptx::prefetch_tensormap(&tmap_w);
    if (warp == W_PATCH && lane == 0) ptx::prefetch_tensormap(&tmap_x);
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = sh->tmem_base;
    const uint32_t a_col0 = (uint32_t)(2 * BN);                      // the A stages follow the two accumulators

    const int host_tiles = a.n_mtiles * a.n_tiles;      // what the host's tile table says; the workers check it against the mask
    if (warp >= W_FILTER) {
        // ================================================================== loader warps
        // They need neither the kept-row list nor the row coordinates: the tile table gives each tile's
        // patch range, so the first filter slabs and the first patches are on their way while the other
        // warps still compact the mask and decode rows.  Each loader thread waits for the preceding
        // kernel by itself before its first load.
        if (lane == 0) {
            ptx::grid_dependency_wait();
            bool ok = true;
            if (warp == W_FILTER) {
                // ---------------------------------------------------------- filter slabs by TMA
                // Stages run slice by slice (all taps of channels 64 s .. 64 s + 63, then the next slice),
                // so that one slice of the patch is in use at a time; in w[C_out][kh][kw][C_in] the slab
                // of (tap, slice) starts at K index tap * C_in + 64 * slice.
                // When the ring holds a whole work item's stages and there is one column tile, stage s always
                // gets the same slab: it is loaded for the block's first tile only and stays (the stage's
                // barrier still gets this thread's arrival, in step with the MMA warp's releases).
                const bool resident = (NST == BS && a.n_tiles == 1);
                int s = 0, fi = 0;
                uint32_t ph = 0;
                for (int t = blockIdx.x; t < host_tiles && ok; t += gridDim.x) {
                    const int n_tile = pitem_of(t, a).n_tile;
                    for (int sl = 0; sl < a.slices && ok; ++sl)
                        for (int tap0 = 0; tap0 < taps; tap0 += G) {
                            const int gc = taps - tap0 < G ? taps - tap0 : G;
                            if (!wait_bar<40>(ptx::smem_u32(&sh->b_empty[s]), ph ^ 1u, ctl, a.dev_status)) { ok = false; break; }
                            const uint32_t full = ptx::smem_u32(&sh->full[fi]);
                            if (resident && t != (int)blockIdx.x) {
                                ptx::mbar_arrive(full);
                            } else {
                                ptx::mbar_arrive_expect_tx(full, (uint32_t)gc * b_tap_bytes);
                                for (int i = 0; i < gc; ++i)
                                    ptx::tma_load_2d(b_base + (uint32_t)s * b_stage_bytes + (uint32_t)i * b_tap_bytes, &tmap_w, full,
                                                     (tap0 + i) * g.C_in + sl * 64, n_tile * BN);
                            }
                            if (++s == BS) { s = 0; ph ^= 1u; }
                            if (++fi == FULL_RING) fi = 0;
                        }
                }
            } else {
                // ---------------------------------------------------------- input patches by TMA
                // Per tile and slice: the padded input rows of the tile's patch, one box of Wp pixels x 64
                // channels each, starting Wp8 pixels apart in the buffer (every box 1024-byte aligned, so
                // the 128-byte swizzle phase of a pixel is its index within the buffer modulo 8).
                uint32_t use = 0;
                for (int t = blockIdx.x; t < host_tiles && ok; t += gridDim.x) {
                    const int4 tl = __ldg(a.tiles + pitem_of(t, a).m_tile);
                    int nrows = tl.w;
                    if (nrows > a.cap_rows || nrows < 1) {                 // cannot happen when the host planned from this mask
                        atomicOr(a.dev_status, DEV_BAD_INDEX);
                        nrows = nrows < 1 ? 1 : a.cap_rows;
                    }
                    const int n_lo = (int)fd_div((uint32_t)tl.z, a.fdHp);
                    for (int sl = 0; sl < a.slices; ++sl, ++use) {
                        const uint32_t b = use & (PB - 1u);
                        if (!wait_bar<40>(ptx::smem_u32(&sh->p_empty[b]), ((use >> a.p_bufs_log2) & 1u) ^ 1u, ctl, a.dev_status)) { ok = false; break; }
                        const uint32_t full = ptx::smem_u32(&sh->p_full[b]);
                        ptx::mbar_arrive_expect_tx(full, (uint32_t)nrows * (uint32_t)a.Wp * 128u);
                        int n = n_lo, yy = tl.z - n_lo * a.Hp;             // padded row yy of image n
                        uint32_t dst = smem_base + b * patch_bytes;
                        for (int i = 0; i < nrows; ++i) {
                            ptx::tma_load_4d(dst, &tmap_x, full, sl * 64, -g.pad_w, yy - g.pad, n);
                            dst += row_bytes;
                            if (++yy == a.Hp) { yy = 0; ++n; }
                        }
                    }
                }
            }
            if (!ok) {   // let loads already issued land before the block's shared memory goes away
                for (int i = 0; i < 64; ++i) __nanosleep(1000);
            }
        }
    } else {
    // ====================================================================== worker warps
    int cnt = 0;
    KeptList kept_list{a.kept, nullptr};
    unsigned short* kept_s = reinterpret_cast<unsigned short*>(sh + 1);
    if (a.fuse_compact) {
        cnt = block_compact(a.mask, g.rows, early_mask, early_ok, kept_s, sh->scan_total, WORK_THREADS, 2);
        kept_list.s = kept_s;
    } else {
        ptx::grid_dependency_wait();
        cnt = __ldcg(a.count);
    }
    const int Mk = (g.rows == g.P) ? g.Nb * cnt : cnt;
    int total_tiles = host_tiles;
    if (Mk != a.Mk_host) {                     // the tiles were cut for another mask: nothing can be computed
        if (tid == 0) {
            atomicOr(a.dev_status, DEV_BAD_INDEX);
            sh->ctl.abort = 1;                 // the loader warps leave their waits
        }
        total_tiles = 0;
    }
    FastDiv fdcnt = a.fdcnt_host;
    if (cnt <= 0 || fdcnt.d != (uint32_t)cnt) fdcnt = make_fastdiv((uint32_t)(cnt > 0 ? cnt : 1));

    // Row coordinates of this block's first INFO_RING tiles, one row per thread.
    {
        for (int idx = tid; idx < INFO_RING * BM; idx += WORK_THREADS) {
            const int jj = idx / BM, rr = idx - jj * BM;
            const long long t = blockIdx.x + (long long)jj * gridDim.x;
            if (t < total_tiles) decode_row(sh, jj, rr, pitem_of((int)t, a).m_tile, Mk, fdcnt, g, a, kept_list);
        }
        asm volatile("bar.sync 2, %0;" ::"n"(WORK_THREADS) : "memory");
        if (tid < INFO_RING && blockIdx.x + (long long)tid * gridDim.x < total_tiles) ptx::mbar_arrive(ptx::smem_u32(&sh->info_full[tid]));
    }
    if (a.fuse_compact) {
        ptx::grid_dependency_wait();
        if (blockIdx.x == 0) {      // the list in global memory, for asx_get_kept and later runs
            for (int i = tid; i < cnt; i += WORK_THREADS) a.kept_out[i] = (int32_t)kept_s[i];
            if (tid == 0) *a.count_out = cnt;
        }
    }

    if (warp == W_INFO) {
        // ------------------------------------------------------------------ row coordinates
        int j = INFO_RING;                        // the first INFO_RING tiles were decoded by the whole block
        for (long long t = blockIdx.x + (long long)INFO_RING * gridDim.x; t < total_tiles; t += gridDim.x, ++j) {
            const int r = j % INFO_RING;
            if (!warp_wait_bar<200>(ptx::smem_u32(&sh->info_empty[r]), ((uint32_t)(j / INFO_RING) & 1u) ^ 1u, ctl, a.dev_status)) break;
            const int m_tile = pitem_of((int)t, a).m_tile;
#pragma unroll
            for (int q2 = 0; q2 < 4; ++q2) decode_row(sh, r, lane * 4 + q2, m_tile, Mk, fdcnt, g, a, kept_list);
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&sh->info_full[r]));
        }
    } else if (warp == W_MMA) {
        // ------------------------------------------------------------------ MMA issue
        // Warp-uniform loop; one elected lane issues.  A comes from tensor memory (lane = tile row,
        // 8 columns per K = 16 step), B from the shared-memory slab.
        const uint32_t idesc = ptx::umma_idesc_bf16(BM, BN);
        const uint64_t bdesc0 = ptx::umma_desc_k_major_sw128(b_base);
        int s = 0, as = 0, fi = 0, ti = 0;
        uint32_t fph = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, ++ti) {
            const int buf = ti & 1;
            const uint32_t use = (uint32_t)(ti >> 1) & 1u;
            ok = warp_wait_bar<0>(ptx::smem_u32(&sh->acc_empty[buf]), use ^ 1u, ctl, a.dev_status);
            if (!ok) break;
            ptx::tc_fence_after_sync();
            const uint32_t d = tmem_base + (uint32_t)(buf * BN);
            int tap0 = 0;
            for (int stg = 0; stg < NST; ++stg) {
                const int gc = taps - tap0 < G ? taps - tap0 : G;
                ok = warp_wait_bar<0>(ptx::smem_u32(&sh->full[fi]), fph, ctl, a.dev_status);
                if (!ok) break;
                ptx::tc_fence_after_sync();
                const uint64_t bdesc = bdesc0 + (uint64_t)((uint32_t)s * (b_stage_bytes >> 4));
                const uint32_t at = tmem_base + a_col0 + (uint32_t)as * a_stage_cols;
                if (ptx::elect_one()) {
                    for (int i = 0; i < gc; ++i) {
                        const uint64_t bd = bdesc + (uint64_t)((uint32_t)i * (b_tap_bytes >> 4));
                        const uint32_t ai = at + (uint32_t)(i * TAP_COLS);
                        ptx::umma_bf16_a_tmem(d, ai, bd, idesc, (stg | i) != 0 ? 1u : 0u);
                        ptx::umma_bf16_a_tmem(d, ai + 8, bd + 2, idesc, 1u);
                        ptx::umma_bf16_a_tmem(d, ai + 16, bd + 4, idesc, 1u);
                        ptx::umma_bf16_a_tmem(d, ai + 24, bd + 6, idesc, 1u);
                    }
                    ptx::umma_commit(ptx::smem_u32(&sh->b_empty[s]));
                    ptx::umma_commit(ptx::smem_u32(&sh->a_empty[as]));
                }
                __syncwarp();
                if (++s == BS) s = 0;
                if (++as == AS) as = 0;
                if (++fi == FULL_RING) { fi = 0; fph ^= 1u; }
                tap0 += G;
                if (tap0 >= taps) tap0 = 0;
            }
            if (ok && ptx::elect_one()) ptx::umma_commit(ptx::smem_u32(&sh->acc_full[buf]));
            __syncwarp();
        }
    } else if ((warp >= W_EPI0 && warp < W_EPI0 + NUM_EPI_WARPS) || (a.epi8 && warp >= W_FILL0 + NUM_FILL_WARPS - 4 && warp < W_FILL0 + NUM_FILL_WARPS)) {
        // ------------------------------------------------------------------ epilogue
        const int q = warp & 3;                       // TMEM lanes 32q .. 32q+31 belong to this warp
        const int half = warp >= W_FILL0 ? 1 : 0;     // with eight epilogue warps: which of the pair this one is
        const int epi_threads = a.epi8 ? 2 * NUM_EPI_WARPS * 32 : NUM_EPI_WARPS * 32;
        const int c_step = a.epi8 ? 64 : 32;
        unsigned short* y2 = reinterpret_cast<unsigned short*>(a.y);
        int ti = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, ++ti) {
            const PItem item = pitem_of(t, a);
            const int n0 = item.n_tile * BN;
            const int buf = ti & 1;
            const uint32_t use = (uint32_t)(ti >> 1) & 1u;
            const int4 tl = __ldg(a.tiles + item.m_tile);
            const int rk = tl.x + q * 32 + lane;
            const bool valid = q * 32 + lane < tl.y;
            const long long yoff = valid ? (long long)(a.out_compact ? rk : out_row_of(rk, fdcnt, g, kept_list)) * N : 0;
            {
                float* sb = sh->bias[buf];
                const int et = half * (NUM_EPI_WARPS * 32) + q * 32 + lane;
                if (et < BN) sb[et] = (a.bias != nullptr && n0 + et < N) ? __ldg(a.bias + n0 + et) : 0.f;
                asm volatile("bar.sync 1, %0;" ::"r"(epi_threads) : "memory");
            }
            const float* sbias = sh->bias[buf];
            if (!warp_wait_bar<100>(ptx::smem_u32(&sh->acc_full[buf]), use, ctl, a.dev_status)) { ok = false; break; }
            ptx::tc_fence_after_sync();
            const uint32_t tacc = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * BN);
            for (int c0 = half * 32; c0 < BN; c0 += c_step) {
                const int col0 = n0 + c0;
                if (col0 >= N) break;
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
                if (valid) {
                    uint4 ov[4];
                    int nh = 0;
#pragma unroll
                    for (int h = 0; h < 4; ++h) {
                        const int colh = col0 + 8 * h;
                        if (colh >= N || c0 + 8 * h >= BN) break;      // the tile's last chunk may be 16 columns wide
                        float v[8];
#pragma unroll
                        for (int j = 0; j < 8; ++j) v[j] = __uint_as_float(r[8 * h + j]) + sbias[c0 + 8 * h + j];
                        if (RESIDUAL) {
                            float res[8];
                            load_residual8(a.residual, yoff + colh, N - colh, 1, res);
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
                        ov[h].x = pack_bf16(v[0], v[1]);
                        ov[h].y = pack_bf16(v[2], v[3]);
                        ov[h].z = pack_bf16(v[4], v[5]);
                        ov[h].w = pack_bf16(v[6], v[7]);
                        nh = h + 1;
                    }
                    // a kept row's neighbours in memory are mostly dropped rows, so this thread's stores share
                    // their sectors with no other thread: whole 32-byte sectors where the layout allows
                    unsigned short* dst = y2 + yoff + col0;
                    if (a.st32) {
#pragma unroll
                        for (int h = 0; h < 4; h += 2) {
                            if (h + 1 < nh) ptx::st_global_v8(dst + 8 * h, ov[h], ov[h + 1]);
                            else if (h < nh) *reinterpret_cast<uint4*>(dst + 8 * h) = ov[h];
                        }
                    } else {
#pragma unroll
                        for (int h = 0; h < 4; ++h)
                            if (h < nh) *reinterpret_cast<uint4*>(dst + 8 * h) = ov[h];
                    }
                }
            }
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&sh->acc_empty[buf]));
        }
    } else if (warp == W_ZERO_A || warp == W_ZERO_A + 1 || warp == W_ZERO_B || warp == W_ZERO_B + 1) {
        // ------------------------------------------------------------------ zeros for dropped rows (a compact output has none)
        // Each block zeroes a fixed share of the output rows, independent of the tile loop.  (Zeroing tile by
        // tile - the dropped rows between a tile's first kept row and the next tile's, so that a stretch of the
        // output leaves one SM at one time - was measured: the short ranges are all latency, 87 us against 71
        // on the first layer.)
        if (!a.out_compact) zero_fill_dropped_rows<false, NUM_ZERO_WARPS * 32>(a.y, a.mask, g, 1, ((warp >= W_ZERO_B ? warp - W_ZERO_B + 2 : warp - W_ZERO_A) * 32 + lane));
    } else {
        // ------------------------------------------------------------------ A operand: patch -> tensor memory
        // Warp (quarter q, group grp) owns tile rows 32 q .. 32 q + 31 (tensor-memory lanes a warp can
        // reach are fixed by its index modulo 4) and the pipeline stages with index % NG == grp, counted
        // over the whole launch.  NG = min(4, a_stages) divides a_stages, so an A stage is always filled by
        // the same group: its waits on that stage's 'empty' barrier follow each other phase by phase (a
        // group that skipped a use could run two phases ahead, which a parity wait cannot tell from none).
        const int q = warp & 3, grp = (warp - W_FILL0) >> 2;
        const uint32_t trow = tmem_base + ((uint32_t)(q * 32) << 16) + a_col0;
        // every tap of a row must stay inside the buffer even if the plan were wrong
        const int max_base = a.cap_rows * a.Wp8 - ((g.kh - 1) * a.Wp8 + (a.px32 ? 4 : g.kw));
        uint32_t it = 0, use = 0, aph = 0;          // stage counter of the launch, its A stage and phase
        int as = 0, fi = 0, j = 0, gsel = 0;
        const int NG = a.epi8 ? 3 : (AS < 4 ? AS : 4);
        bool ok = true;
        for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, ++j) {
            const int r = j & (INFO_RING - 1);
            if (!warp_wait_bar<100>(ptx::smem_u32(&sh->info_full[r]), (uint32_t)(j / INFO_RING) & 1u, ctl, a.dev_status)) break;
            const int px = sh->rowpix[r][q * 32 + lane];
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&sh->info_empty[r]));        // the ring slot is in registers now
            int base = px >= 0 ? px : 0;                                           // rows past the end read pixel 0; their results are never stored
            base = base < 0 ? 0 : (base > max_base ? max_base : base);
            for (int sl = 0; sl < a.slices && ok; ++sl, ++use) {
                const uint32_t b = use & (PB - 1u);
                if (!warp_wait_bar<20>(ptx::smem_u32(&sh->p_full[b]), (use >> a.p_bufs_log2) & 1u, ctl, a.dev_status)) { ok = false; break; }
                const uint32_t pb = smem_base + b * patch_bytes;
                int ky = 0, kx = 0;
                for (int tap0 = 0; tap0 < taps; tap0 += G, ++it) {
                    const int gc = taps - tap0 < G ? taps - tap0 : G;
                    if (gsel == grp) {
                        if (!warp_wait_bar<20>(ptx::smem_u32(&sh->a_empty[as]), aph ^ 1u, ctl, a.dev_status)) { ok = false; break; }
                        ptx::tc_fence_after_sync();
                        const uint32_t tdst = trow + (uint32_t)as * a_stage_cols;
                        int kyi = ky, kxi = kx;
#pragma unroll 1
                        for (int i = 0; i < gc; ++i) {
                            const int pix = base + kyi * a.Wp8 + kxi;
                            uint32_t v[32];
                            if (a.px32) {
                                // blocks pix .. pix + 3, 16 bytes at a time, through the 128-byte swizzle of the rows
                                // (1024-byte aligned): it is also what keeps eight neighbouring rows' reads, 32 bytes
                                // apart, on different banks
                                const uint32_t off = (uint32_t)pix * 32u;
#pragma unroll
                                for (int c = 0; c < 8; ++c) {
                                    const uint32_t o = off + (uint32_t)c * 16u;
                                    ptx::ld_shared_v4(pb + (o ^ ((o >> 3) & 0x70u)), v[4 * c], v[4 * c + 1], v[4 * c + 2], v[4 * c + 3]);
                                }
                            } else {
                                const uint32_t src = pb + (uint32_t)pix * 128u;
                                const uint32_t sw = (uint32_t)(pix & 7);
#pragma unroll
                                for (int c = 0; c < 8; ++c)
                                    ptx::ld_shared_v4(src + (((uint32_t)c ^ sw) << 4), v[4 * c], v[4 * c + 1], v[4 * c + 2], v[4 * c + 3]);
                            }
                            ptx::tmem_st_32(tdst + (uint32_t)(i * TAP_COLS), v);
                            if (++kxi == g.kw) { kxi = 0; ++kyi; }
                        }
                        ptx::tmem_st_wait();
                        ptx::tc_fence_before_sync();
                        __syncwarp();
                        if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&sh->full[fi]));
                    }
                    if (++as == AS) { as = 0; aph ^= 1u; }
                    if (++fi == FULL_RING) fi = 0;
                    if (++gsel == NG) gsel = 0;
                    kx += gc;                                   // advance the window position by the chunk's taps
                    while (kx >= g.kw) { kx -= g.kw; ++ky; }
                }
                __syncwarp();
                if (ok && lane == 0) ptx::mbar_arrive(ptx::smem_u32(&sh->p_empty[b]));   // this warp has read all it needs of the slice
            }
        }
    }

    }   // worker warps

    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == W_MMA) {
        __syncwarp();
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, 512u);
    }
}

int round_up(int v, int m) { return (v + m - 1) / m * m; }

}  // namespace

bool plan_patch(const ConvGeom& g, int fused_list_rows, int px32, PatchPlan* plan)
{
    if (g.stride != 1 || g.stride_w != 1 || g.C_in % 64 != 0 || g.kh * g.kw < 2 || g.C_out % 8 != 0) return false;
    if (px32 && (g.C_in != 64 || g.kw != 1 || g.pad != 0 || g.pad_w != 0)) return false;
    // px32: a patch row holds the Wo + 3 blocks that the row's windows touch, loaded as whole 128-byte units of
    // four blocks (the staged rows are a multiple of four blocks long)
    const int Wp = px32 ? (g.Wo + 3 + 3) / 4 : g.W + 2 * g.pad_w, Hp = g.H + 2 * g.pad;
    if (px32 && (g.W % 4 != 0 || Wp * 4 > g.W)) return false;
    if (Wp > 256 || g.kh > Hp || g.kw > Wp) return false;
    // Hp and Wp as the kernel uses them need the output to be the full stride-1 range
    if (g.Ho != Hp - g.kh + 1 || (!px32 && g.Wo != Wp - g.kw + 1)) return false;
    const int N = g.C_out;
    const int n_tiles = (N + 127) / 128;
    const int BN = round_up((N + n_tiles - 1) / n_tiles, 16);
    // Taps per stage: enough tensor-core work per stage to cover the issuing thread's fixed cost (a
    // tap of a 128 x BN tile is 4 instructions of BN/2 clocks), little enough that three filter stages
    // leave room for the patches and two A stages fit beside the accumulators in tensor memory.
    int G = BN <= 32 ? 4 : BN <= 64 ? 3 : 2;
    if (g.kh * g.kw < G) G = g.kh * g.kw;
    while (G > 1 && (512 - 2 * BN) / (G * TAP_COLS) < 2) --G;
    // 2x2-block form: a tile has only kh taps (four for a 7- or 8-wide filter), so the per-stage and per-tile
    // bookkeeping of the issuing thread and the fill warps weighs as much as the work; all taps in one stage
    // when three A stages of that size fit beside the accumulators.
    if (px32 && g.kh * g.kw <= 4 && (512 - 2 * BN) / (g.kh * g.kw * TAP_COLS) >= 3) G = g.kh * g.kw;
    else if (px32 && G > 2 && (g.kh * g.kw) % G != 0 && (g.kh * g.kw) % (G - 1) == 0) --G;
    const int Wp8 = px32 ? round_up(Wp * 4, 32) : round_up(Wp, 8);      // row pitch in pixels: rows start 1024-byte aligned
    const int px_bytes = px32 ? 32 : 128;
    const int list_bytes = (fused_list_rows * 2 + 15) / 16 * 16;
    // Wide rows (the 112-pixel rows of a network's first layer are 14 KB each) leave few patch rows beside
    // three filter stages; a tile should span at least three output rows, or most of its 128 rows stay
    // empty.  Then the filter ring shrinks first to stages of two taps, then to two stages.
    int b_stages = 3, cap_rows = 0, half = 0;
    for (int attempt = 0; attempt < 3; ++attempt) {
        if (attempt == 1) { if (G <= 2) continue; G = 2; }
        if (attempt == 2) b_stages = 2;
        if (px32 && (g.kh * g.kw) % G == 0 && (g.kh * g.kw) / G <= 3) b_stages = (g.kh * g.kw) / G;     // the whole filter stays in the ring
        const int budget = 227 * 1024 - 1024 - (int)sizeof(PShared) - list_bytes - b_stages * G * BN * 128;
        half = budget < 0 ? 0 : budget / 2 / 1024 * 1024;                // a buffer is a multiple of 1024 bytes
        cap_rows = half / (Wp8 * px_bytes);
        if (cap_rows >= g.kh + 2) break;
    }
    // The rows of the 2x2-block form are short (a quarter of a 128-byte-per-pixel row), a tile's patch is a
    // few KB and arrives after one memory latency: four buffers keep three loads in flight instead of one.
    int p_bufs_log2 = 1;
    if (px32 && (half / 2 / 1024 * 1024) / (Wp8 * px_bytes) >= g.kh + 4) { p_bufs_log2 = 2; cap_rows = (half / 2 / 1024 * 1024) / (Wp8 * px_bytes); }
    if (cap_rows > 64) cap_rows = 64;
    int a_stages = (512 - 2 * BN) / (G * TAP_COLS);
    if (a_stages > 4) a_stages = 4;             // ring depths divide FULL_RING
    // Up to four k-blocks per tile: the epilogue, not the main loop, sets the pace, so four of the sixteen fill
    // warps join it; the twelve that remain are three groups, which take three A stages.
    const int epi8 = (g.kh * g.kw * (g.C_in / 64) <= 4 && BN % 64 == 0 && a_stages >= 3) ? 1 : 0;
    if (epi8) a_stages = 3;
    if (a_stages < 2) return false;
    if (cap_rows < g.kh) return false;
    plan->BN = BN;
    plan->n_tiles = (N + BN - 1) / BN;
    plan->a_stages = a_stages;
    plan->G = G;
    plan->b_stages = b_stages;
    plan->cap_rows = cap_rows;
    plan->Hp = Hp;
    plan->Wp = Wp;
    plan->Wp8 = Wp8;
    plan->px32 = px32;
    plan->p_bufs_log2 = p_bufs_log2;
    plan->epi8 = epi8;
    plan->smem_bytes = 1024 + (1 << p_bufs_log2) * round_up(cap_rows * Wp8 * px_bytes, 1024) + b_stages * G * BN * 128 + (int)sizeof(PShared) + list_bytes;
    plan->est_cost_us = 0.0;          // set by plan_patch_cost once the tiles are cut
    return true;
}

void plan_patch_cost(const ConvGeom& g, int num_sms, long long n_mtiles, PatchPlan* plan)
{
    // Estimated duration, in the terms of the row-gather planner and from the same kind of measurement:
    // a 64-wide k-block of a 128 x BN tile takes about 0.21 + 0.001 BN microseconds here (against
    // 0.30 + 0.001 BN for the row gather).  Both forms are bound by shared-memory bandwidth: per k-block
    // this one moves 16 KB of patch reads, the filter slab in and out (BN x 256 bytes) and its share of
    // the patch, the row gather 32 KB of A rows in and out plus the same slab.
    const long long items = n_mtiles * plan->n_tiles;
    const long long waves = (items + num_sms - 1) / num_sms;
    const int KB = g.kh * g.kw * (g.C_in / 64);
    const double t_tile = KB * (0.21 + 0.001 * plan->BN);
    plan->est_cost_us = (double)waves * (t_tile + 0.3) + 0.012 * plan->BN;
}

cudaError_t launch_patch(const ConvGeom& g, const PatchPlan& plan, const CUtensorMap& tmap_w, const CUtensorMap& tmap_x4,
                         const float* bias, void* y, const uint8_t* mask, const int32_t* kept, const int32_t* count,
                         int relu, int* dev_status, int num_sms, int fuse_compact, long long host_kept,
                         const void* residual, const void* tiles, int n_mtiles, long long kept_rows, int out_compact,
                         int wait_limit_kcycles, cudaStream_t st)
{
    PatchArgs a;
    a.fdcnt_host = make_fastdiv((uint32_t)(host_kept > 0 && host_kept < (1ll << 31) ? host_kept : 1));
    if (!(host_kept > 0 && host_kept < (1ll << 31))) a.fdcnt_host.d = 0;
    a.fdP = make_fastdiv((uint32_t)g.P);
    a.fdWo = make_fastdiv((uint32_t)g.Wo);
    a.fdNt = make_fastdiv((uint32_t)plan.n_tiles);
    a.fdHp = make_fastdiv((uint32_t)plan.Hp);
    a.bias = bias;
    a.y = static_cast<__nv_bfloat16*>(y);
    a.mask = mask;
    a.kept = kept;
    a.count = count;
    a.dev_status = dev_status;
    a.relu = relu == 1 ? 1 : 0;
    a.out_compact = out_compact;
    a.st32 = (g.C_out % 16 == 0 && (reinterpret_cast<uintptr_t>(y) & 31) == 0) ? 1 : 0;
    a.BN = plan.BN;
    a.n_tiles = plan.n_tiles;
    a.b_stages = plan.b_stages;
    a.a_stages = plan.a_stages;
    a.G = plan.G;
    a.cap_rows = plan.cap_rows;
    a.Hp = plan.Hp;
    a.Wp = plan.Wp;
    a.Wp8 = plan.Wp8;
    a.px32 = plan.px32;
    a.p_bufs_log2 = plan.p_bufs_log2;
    a.epi8 = plan.epi8;
    a.slices = g.C_in / 64;
    a.fuse_compact = fuse_compact;
    a.kept_out = const_cast<int32_t*>(kept);
    a.count_out = const_cast<int32_t*>(count);
    a.residual = static_cast<const __nv_bfloat16*>(residual);
    a.wait_limit_kcycles = wait_limit_kcycles > 0 ? wait_limit_kcycles : WAIT_LIMIT_KCYCLES_DEFAULT;
    a.tiles = static_cast<const int4*>(tiles);
    a.n_mtiles = n_mtiles;
    a.Mk_host = (int)kept_rows;

    long long items = (long long)n_mtiles * plan.n_tiles;
    int grid = (int)(items < num_sms ? items : num_sms);
    if (grid < 1) grid = 1;
    const bool has_res = residual != nullptr, is_silu = relu == 2;
    using Kern = void (*)(const CUtensorMap, const CUtensorMap, const ConvGeom, const PatchArgs);
    Kern kern = has_res ? (is_silu ? masked_conv_patch_sm100_kernel<true, true> : masked_conv_patch_sm100_kernel<true, false>)
                        : (is_silu ? masked_conv_patch_sm100_kernel<false, true> : masked_conv_patch_sm100_kernel<false, false>);
    static int smem_set[4] = {0, 0, 0, 0};      // largest dynamic shared memory size enabled so far, per instance
    const int vi = (has_res ? 1 : 0) + (is_silu ? 2 : 0);
    if (plan.smem_bytes > smem_set[vi]) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, plan.smem_bytes);
        if (e != cudaSuccess) return e;
        smem_set[vi] = plan.smem_bytes;
    }
    return launch_pdl(kern, dim3(grid), dim3(NUM_THREADS), (size_t)plan.smem_bytes, st, tmap_w, tmap_x4, g, a);
}

}  // namespace asx
