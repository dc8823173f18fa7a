// Device helpers shared by the two fused convolution kernels (the row-gather form and the
// window-patch form): divisions by launch constants, bounded mbarrier waits, the in-kernel mask
// compaction (S1), the kept-row list, the zero fill of dropped rows and small epilogue helpers.
#pragma once
#include <cuda_bf16.h>
#include "asx_internal.h"
#include "ptx_sm100.cuh"

namespace asx {

// Division of a 32-bit unsigned number by a divisor fixed for the whole launch, as a multiply-high
// and two shifts (Granlund and Montgomery's round-up method: l = ceil(log2 d),
// m = floor(2^32 (2^l - d) / d) + 1, q = (t + ((n - t) >> min(l,1))) >> max(l-1,0) with
// t = mulhi(m, n); exact for every n < 2^32 and 1 <= d < 2^31).  A hardware-less 32-bit division
// is about 35 dependent instructions, and the row-coordinate warp did twelve per tile.
struct FastDiv {
    uint32_t d, m, s1, s2;
};
__host__ __device__ inline FastDiv make_fastdiv(uint32_t d)
{
    uint32_t l = 0;
    while ((1ull << l) < d) ++l;
    const unsigned long long m = ((((1ull << l) - d) << 32) / d) + 1ull;
    FastDiv f;
    f.d = d;
    f.m = (uint32_t)m;
    f.s1 = l ? 1u : 0u;
    f.s2 = l ? l - 1u : 0u;
    return f;
}
__device__ __forceinline__ uint32_t fd_div(uint32_t n, const FastDiv& f)
{
    const uint32_t t = __umulhi(f.m, n);
    return (t + ((n - t) >> f.s1)) >> f.s2;
}

// Every wait in the kernels is bounded.  The limit is a launch parameter (in units of 1024 clock
// cycles; the default is about two seconds) kept beside the block's abort flag in shared memory.
constexpr int WAIT_LIMIT_KCYCLES_DEFAULT = 4000000;
struct WaitCtl {
    int abort;            // set by the first waiter that gives up; every role then leaves
    int limit_kcycles;
};

// Bounded wait on an mbarrier phase.  The waiter is suspended by the hardware between polls
// (and woken when the phase completes), so waiting warps do not take issue slots from the warps
// that share their scheduler.  SLEEP_NS is kept as a per-call-site label of how relaxed the
// waiter may be; it scales the suspend-time hint.
template <int SLEEP_NS>
__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, volatile WaitCtl* ctl, int* dev_status)
{
    if (ptx::mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!ptx::mbar_try_wait_suspend(bar, parity, 2000u + 10u * SLEEP_NS)) {
        if (ctl->abort) return false;
        if (clock64() - t0 > ((long long)ctl->limit_kcycles << 10)) {
            ctl->abort = 1;
            atomicOr(dev_status, DEV_TIMEOUT_PIPE);
            return false;
        }
    }
    return true;
}

// The same wait for a whole converged warp: lane 0 polls, the result is broadcast.  Polling from
// every lane multiplies the barrier traffic in shared memory by 32 and slows every waiter down.
template <int SLEEP_NS>
__device__ __forceinline__ bool warp_wait_bar(uint32_t bar, uint32_t parity, volatile WaitCtl* ctl, int* dev_status)
{
    int ok = 1;
    if ((threadIdx.x & 31) == 0) ok = wait_bar<SLEEP_NS>(bar, parity, ctl, dev_status) ? 1 : 0;
    return __shfl_sync(0xffffffffu, ok, 0) != 0;
}

// S1 inside the fused kernel, for masks of at most 16384 rows: the whole block scans the mask
// (16 bytes per thread, popcount, shuffle scan within the warps, warp totals through shared
// memory) and writes the ascending kept positions as 16-bit values into its own shared memory
// (every block writing the list to the same global addresses serialises in L2 and cost 10-20 us;
// block 0 alone copies it out).  Returns the count.  The first `nthreads` threads of the block take part
// (a multiple of 32; they meet on hardware barrier `barrier_id`), the others may do something else.
// Bit q of the result: byte q of the 16 mask bytes in v is non-zero.
__device__ __forceinline__ unsigned nonzero_bytes16(const uint4& v)
{
    const unsigned w4[4] = {v.x, v.y, v.z, v.w};
    unsigned flags = 0;
#pragma unroll
    for (int q2 = 0; q2 < 4; ++q2) {
        const unsigned t = ((w4[q2] & 0x7f7f7f7fu) + 0x7f7f7f7fu) | w4[q2];      // bit 7 of each byte: byte != 0
        flags |= (((t >> 7) & 1u) | ((t >> 14) & 2u) | ((t >> 21) & 4u) | ((t >> 28) & 8u)) << (4 * q2);
    }
    return flags;
}
// Bit q of the result: mask[first + q] != 0, for the 16 mask bytes starting at `first`.
__device__ __forceinline__ unsigned mask_flags16(const uint8_t* __restrict__ mask, int rows, int first)
{
    if (first + 16 <= rows && (reinterpret_cast<uintptr_t>(mask) & 15) == 0)
        return nonzero_bytes16(*reinterpret_cast<const uint4*>(mask + first));
    unsigned flags = 0;
    for (int q2 = 0; q2 < 16; ++q2)
        if (first + q2 < rows && mask[first + q2] != 0) flags |= 1u << q2;
    return flags;
}

// `early` holds mask bytes 16 tid .. 16 tid + 15 when `early_ok` (the caller read them before the
// kernel's set-up so that the latency of the read is hidden behind it).
__device__ __forceinline__ int block_compact(const uint8_t* __restrict__ mask, int rows, const uint4& early, bool early_ok,
                                             unsigned short* kept_s, int* scan_total, int nthreads, int barrier_id = 0)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = nthreads >> 5;
    int running = 0;
    for (int base = 0; base < rows; base += nthreads * 16) {
        const int first = base + tid * 16;
        const bool wactive = base + warp * 512 < rows;      // warps past the end of the mask only keep the barriers
        unsigned flags = 0;
        int mine = 0, incl = 0;
        if (wactive) {
            flags = (base == 0 && early_ok) ? nonzero_bytes16(early) : mask_flags16(mask, rows, first);
            mine = __popc(flags);
            incl = mine;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const int t = __shfl_up_sync(0xffffffffu, incl, d);
                if (lane >= d) incl += t;
            }
        }
        if (lane == 31) scan_total[warp] = incl;
        asm volatile("bar.sync %0, %1;" ::"r"(barrier_id), "r"(nthreads) : "memory");
        if (wactive) {
            // scan of the (at most 27) warp totals with shuffles
            const int wt = lane < nwarps ? scan_total[lane] : 0;
            int winc = wt;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const int t = __shfl_up_sync(0xffffffffu, winc, d);
                if (lane >= d) winc += t;
            }
            const int prefix = __shfl_sync(0xffffffffu, winc - wt, warp);
            const int total = __shfl_sync(0xffffffffu, winc, 31);
            const int at = running + prefix + incl - mine;
            if (flags) {
                // sixteen independent predicated stores instead of a loop over the set bits
#pragma unroll
                for (int q2 = 0; q2 < 16; ++q2)
                    if ((flags >> q2) & 1u) kept_s[at + __popc(flags & ((1u << q2) - 1u))] = (unsigned short)(first + q2);
            }
            if (tid == 0) scan_total[31] = running + total;     // slot 31 is no warp's total (27 warps)
        }
        asm volatile("bar.sync %0, %1;" ::"r"(barrier_id), "r"(nthreads) : "memory");
        running = scan_total[31];
    }
    return running;
}

// Output row (n*P + p) of the rk-th kept lowered row.
// What the kernel before this one in the stream wrote (the list, its count, a residual tensor) is read
// past L1 (ld.global.cg): a kernel launched as a programmatic dependent starts while its predecessor
// runs, L1 is not invalidated between the two, and an SM can still hold a line with the older
// contents of an address (seen with the compaction passes: blocks read the count they had written
// in the pass before instead of the scanned offset).
struct KeptList {
    const int32_t* g;            // in global memory, or
    const unsigned short* s;     // this block's 16-bit copy in shared memory (fused compaction)
    __device__ __forceinline__ int at(int i) const { return s != nullptr ? (int)s[i] : __ldcg(g + i); }
};
__device__ __forceinline__ int out_row_of(int rk, const FastDiv& fdcnt, const ConvGeom& g, const KeptList& kept)
{
    if (g.rows == g.P) {
        const int n = (int)fd_div((uint32_t)rk, fdcnt);
        return n * g.P + kept.at(rk - n * (int)fdcnt.d);
    }
    return kept.at(rk);
}

// Eight values of the residual tensor (the shortcut branch of a residual block, laid out like the
// output) starting at element `off`, as fp32; zeros when there is no residual.  `left` = columns left
// in the row (only the first min(left, 8) are read on the element-wise path).
__device__ __forceinline__ void load_residual8(const __nv_bfloat16* residual, long long off, int left, int vec, float* res)
{
#pragma unroll
    for (int j = 0; j < 8; ++j) res[j] = 0.f;
    if (residual == nullptr) return;
    if (vec) {
        const uint4 q = __ldcg(reinterpret_cast<const uint4*>(residual + off));
        const uint32_t w4[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            res[2 * j] = __uint_as_float(w4[j] << 16);
            res[2 * j + 1] = __uint_as_float(w4[j] & 0xffff0000u);
        }
    } else {
#pragma unroll
        for (int j = 0; j < 8; ++j)
            if (j < left) res[j] = __uint_as_float((uint32_t)__ldcg(reinterpret_cast<const unsigned short*>(residual) + off + j) << 16);
    }
}

// z * sigmoid(z) with the fast exponential and division (relative error about 1e-6, far below the
// bf16 rounding of the result); exp(-z) = inf for very negative z gives -0.
__device__ __forceinline__ float silu(float z)
{
    return __fdividef(z, 1.f + __expf(-z));
}

__device__ __forceinline__ uint32_t pack_bf16(float a, float b)
{
    const __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<const uint32_t*>(&v);
}


// Zeros for dropped rows.  Algorithm 2's post-processing writes zeros wherever the mask is 0.  The
// calling warps (ZT threads, this one is number zt) stream over this block's share of the output rows,
// independent of the tile loop.  Kept rows are written by the epilogue, so each element is written
// exactly once.
// Fast path (16-byte stores, chunks per row dividing the thread count): every thread keeps one
// 16-byte column of the row and walks down the rows with a constant stride, so a warp writes whole
// consecutive rows; four mask bytes are fetched before the four stores they guard, and nothing in
// the loop divides.
template <bool F32, int ZT>
__device__ __forceinline__ void zero_fill_dropped_rows(void* y, const uint8_t* __restrict__ mask, const ConvGeom& g, int vec_out, int zt)
{
    constexpr int ES = F32 ? 4 : 2, EPC = 16 / ES;
    const int N = g.C_out, lane = zt & 31;
    uint8_t* yb = reinterpret_cast<uint8_t*>(y);
    const long long lo = (long long)g.M * blockIdx.x / gridDim.x;
    const long long hi = (long long)g.M * (blockIdx.x + 1) / gridDim.x;
    const int cpr = N / EPC;                                  // 16-byte chunks per row
    const bool shared_mask = (g.rows == g.P);
    if (vec_out && cpr <= ZT && ZT % cpr == 0) {
        const int rpp = ZT / cpr;                             // rows covered by one pass of all threads
        const int sub = zt / cpr, cc = zt - sub * cpr;
        long long row = lo + sub;
        int p = shared_mask ? (int)(row % g.P) : 0;           // mask index of `row`, kept incrementally
        const int pstep = rpp % g.P;
        uint4* dst = reinterpret_cast<uint4*>(yb + (row * N + cc * EPC) * ES);
        const long long dstep = (long long)rpp * cpr;         // in 16-byte units
        while (row < hi) {
            bool drop[4];
            int pk = p;
#pragma unroll
            for (int k2 = 0; k2 < 4; ++k2) {
                const long long rk = row + (long long)k2 * rpp;
                drop[k2] = (rk < hi) && __ldg(mask + (shared_mask ? (long long)pk : rk)) == 0;
                pk += pstep;
                if (pk >= g.P) pk -= g.P;
            }
#pragma unroll
            for (int k2 = 0; k2 < 4; ++k2)
                if (drop[k2]) dst[k2 * dstep] = make_uint4(0, 0, 0, 0);
            p = pk;
            row += 4LL * rpp;
            dst += 4 * dstep;
        }
    } else {
        // general path: one warp per dropped row
        const int zw = zt >> 5;
        for (long long row = lo + zw; row < hi; row += ZT / 32) {
            const long long pm = shared_mask ? row % g.P : row;
            if (__ldg(mask + pm) != 0) continue;
            if (vec_out) {
                for (int c1 = lane; c1 < cpr; c1 += 32)
                    *reinterpret_cast<uint4*>(yb + (row * N + c1 * EPC) * ES) = make_uint4(0, 0, 0, 0);
            } else if (F32) {
                for (int c1 = lane; c1 < N; c1 += 32) reinterpret_cast<float*>(yb)[row * N + c1] = 0.f;
            } else {
                for (int c1 = lane; c1 < N; c1 += 32) reinterpret_cast<unsigned short*>(yb)[row * N + c1] = 0;
            }
        }
    }
}

}  // namespace asx
