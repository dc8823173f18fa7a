/*
 * asx — masked convolution as a compacted GEMM on NVIDIA B200 (sm_100a).
 *
 * The library computes the inference path of "Accelerating Deep Neural Networks via
 * Semi-Structured Activation Sparsity" (arXiv 2309.06626), Section 3.2 and Appendix A
 * (Algorithm 2): a convolution lowered to a matrix product in which a per-layer binary mask
 * with one entry per output spatial position removes whole rows of the lowered activation
 * matrix.  The product runs on the kept rows only; dropped positions are zero in every
 * channel.  With x[Nb][H][W][C_in] (NHWC), w[C_out][kh][kw][C_in], bias[C_out]:
 *
 *     y[n][oy][ox][co] = mask(n,oy,ox) ? act(bias[co] + sum_{ky,kx,ci} x[n][oy*s-p+ky][ox*s-p+kx][ci]
 *                                                                    * w[co][ky][kx][ci])
 *                                      : 0
 *
 * (cross-correlation, zero padding p on all sides, dilation 1, groups 1).  x, w and y are
 * bfloat16, the bias is fp32, products are accumulated in fp32 on the tensor cores, and y is
 * rounded to bfloat16 (nearest even).  A dropped position is the bit pattern 0x0000 in all
 * channels: neither bias nor activation is applied there.
 *
 * Conventions for every function:
 *  - returns an asx_status; nothing throws or aborts; arguments are checked on the host
 *    before any launch and a failed check launches nothing;
 *  - "device pointer" means memory of the current CUDA device, owned by the caller;
 *  - `cuda_stream` is a cudaStream_t passed as void* (NULL = the legacy default stream);
 *    work is enqueued on it and the call returns without waiting unless stated;
 *  - a layer handle may be used by one host thread at a time;
 *  - there is no CPU fallback: without a usable CUDA device the calls return ASX_ERR_CUDA.
 */
#ifndef ASX_H_
#define ASX_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct asx_layer asx_layer;   /* opaque, owned by the library */

typedef enum {
    ASX_OK = 0,
    ASX_ERR_INVALID_ARG = 1,   /* null pointer, non-positive size, unknown flag */
    ASX_ERR_UNSUPPORTED = 2,   /* a legal convolution this library cannot run */
    ASX_ERR_NO_MASK = 3,       /* asx_run before any asx_set_mask* */
    ASX_ERR_SHAPE = 4,         /* mask length does not match the output geometry */
    ASX_ERR_ALIGN = 5,         /* a pointer is not aligned as documented */
    ASX_ERR_OOM = 6,           /* device or host allocation failed */
    ASX_ERR_CUDA = 7,          /* a CUDA runtime or driver call failed */
    ASX_ERR_TIMEOUT = 8        /* a bounded wait inside a kernel gave up */
} asx_status;

/* flags of asx_run */
enum {
    ASX_ACT_RELU = 1,      /* y = max(acc + bias, 0) on kept rows (default: acc + bias) */
    ASX_RECOMPACT = 2,     /* rebuild the kept-row list from the stored mask inside this call */
    ASX_IMPL_NAIVE = 4,    /* run the slow one-thread-per-output CUDA kernel (debug reference) */
    ASX_OUT_COMPACT = 8,   /* y holds the kept rows only: [Nb*P'][C_out] in kept order, nothing zero-filled */
    ASX_IN_COMPACT = 16,   /* x holds only the positions kept by the mask given to asx_set_input_mask */
    ASX_ACT_SILU = 32,     /* y = z / (1 + exp(-z)), z = acc + bias, on kept rows (the activation of the YOLOv5
                              network of Section 4); not together with ASX_ACT_RELU (ASX_ERR_INVALID_ARG) */
    ASX_F32 = 64,          /* x, w and y are fp32, the storage type of Appendix A, Algorithm 2 (its sizeof(float));
                              the products run on the tensor cores in TF32, see asx_run */
    ASX_IMPL_ROW_GATHER = 128, /* always build the lowered rows by gathering every filter tap of every kept row
                              separately (the general form of the producer), also where the library would load a
                              tile's window range once and cut the taps out of it (stride-1 layers with several
                              taps and C_in % 64 == 0 whose mask came from host memory).  Same results up to
                              summation order; a tuning and test switch */
    ASX_IMPL_WINDOW_PATCH = 256  /* the opposite switch: take the window-range form wherever it can run, also where
                              the library's cost estimate prefers the row gather.  Layers it cannot run
                              (see ASX_IMPL_ROW_GATHER) are not affected.  Not together with ASX_IMPL_ROW_GATHER
                              (ASX_ERR_INVALID_ARG) */
};

/* Human-readable name of a status code; never NULL; static storage. */
const char* asx_status_string(asx_status s);

/*
 * Create a layer: the convolution geometry of Section 3 (filter size, stride, padding).
 * C_in, C_out, kh, kw, stride >= 1, pad >= 0.  On success *out receives a handle to be
 * released with asx_destroy.  No device memory is allocated here.
 */
asx_status asx_create_layer(int C_in, int C_out, int kh, int kw, int stride, int pad,
                            asx_layer** out);

/*
 * Set the layer's binary mask (Appendix A, Algorithm 2: mask == 1 keeps an output position,
 * mask == 0 drops it) and build the kept-row list (stage i of Section 3.2, the running index
 * of the indirection initialisation): kept[j] = position of the j-th non-zero mask entry in
 * ascending order, index p = oy*Wo + ox.
 *   mask : `rows` bytes, each 0 or non-zero, host or device pointer (the library finds out
 *          which); it is copied, the caller may free it after the call returns.
 *   rows : Ho*Wo (one mask shared by every image of a batch, the paper's constant per-layer
 *          mask) or Nb*Ho*Wo (one entry per lowered row); checked against the geometry at
 *          asx_run.  0 < rows < 2^31.
 * The copy and the compaction kernel are enqueued on `cuda_stream`; a host mask is copied
 * synchronously.  Device buffers owned by the layer are (re)allocated when `rows` grows.
 */
asx_status asx_set_mask(asx_layer* layer, const uint8_t* mask, int64_t rows, void* cuda_stream);

/*
 * Generate and set a mask with `rows` entries in which blocks of `block` consecutive rows
 * (raster order, last block possibly short) are kept or dropped together.  The number of
 * dropped blocks is floor(sparsity * nblocks + 1/2), nblocks = ceil(rows / block).  Block b
 * gets the 64-bit score (out[1] << 32 | out[0]) of Philox4x32-10 with counter (b_lo, b_hi, 0, 0)
 * and key (seed_lo, seed_hi); the blocks with the smallest (score, b) are dropped (a random
 * ranking, as in Algorithm 1's getMask).  0 <= sparsity <= 1, block >= 1.
 */
asx_status asx_set_mask_random(asx_layer* layer, int64_t rows, double sparsity, int block,
                               uint64_t seed, void* cuda_stream);

/*
 * The mask generator of the paper's training pipeline (Algorithm 1, function getMask) for one layer:
 * a 2-D score at the input image's resolution is brought to the layer's resolution by an average
 * pooling with window = stride = ratio, ratio = input_res // layer_res per axis, the layer's
 * positions are ranked by their pooled score, and the mask is 0 at the ranked fraction `sparsity`.
 * Using one score for all layers of a network gives masks that agree across resolutions
 * (Section 3.1).  Where the paper is silent this library takes: the floor(sparsity*P + 1/2)
 * positions with the SMALLEST pooled score are dropped (P = Ho*Wo); equal scores are ordered by
 * position (raster order); output cell (i, j) pools score rows i*rh .. i*rh+rh-1 and columns
 * j*rw .. j*rw+rw-1 with rh = H0 / Ho, rw = W0 / Wo (integer division; what lies beyond is unused);
 * window sums are accumulated in fp64 in raster order and divided by rh*rw in fp64.
 *   score    : HOST pointer, H0*W0 floats, row-major.  1 <= Ho <= H0, 1 <= Wo <= W0, 0 <= sparsity <= 1.
 *   mask_out : HOST pointer, receives Ho*Wo bytes (1 keep / 0 drop).
 * asx_mask_from_scores runs on the host only (no CUDA call); asx_set_mask_from_scores generates the
 * mask and sets it like asx_set_mask (mask shared by the batch).
 */
asx_status asx_mask_from_scores(const float* score, int H0, int W0, int Ho, int Wo, double sparsity,
                                uint8_t* mask_out);
asx_status asx_set_mask_from_scores(asx_layer* layer, const float* score, int H0, int W0, int Ho, int Wo,
                                    double sparsity, void* cuda_stream);

/*
 * Layer chaining without re-densifying.  The paper expands every masked layer's output back to the
 * dense shape only because the layer that follows expects an ordinary dense tensor (Section 3.2, stage
 * iii) and names that post-processing as one of its two overheads (Section 4.3).  Here a layer run
 * with ASX_OUT_COMPACT writes row j of the kept list of image n at y[n*P' + j][0..C_out) and writes
 * nothing else, and the layer that consumes it is run with ASX_IN_COMPACT after being told the
 * producer's mask with asx_set_input_mask: its gather then reads input position p of image n at
 * x[n*P'_in + rank(p)] when p was kept and zeros when it was dropped, which is what the dense
 * tensor would have held.
 *   mask : `rows` bytes (0 / non-zero), host or device pointer (a device mask is copied to the host,
 *          which waits for it); rows must equal H*W of the tensors this layer is run on (one mask
 *          per image, shared by the batch).  0 < rows < 2^31.
 * ASX_IN_COMPACT needs C_in % 8 == 0 and at least one kept input position (else ASX_ERR_UNSUPPORTED),
 * and is not available with ASX_IMPL_NAIVE.
 */
asx_status asx_set_input_mask(asx_layer* layer, const uint8_t* mask, int64_t rows, void* cuda_stream);

/*
 * Residual add in the epilogue (the shortcut of a residual block; part of chaining layers without
 * extra passes over the activations): with a residual tensor set, asx_run computes
 *     y = mask ? act(acc + bias + residual) : 0
 * where `residual` is a bfloat16 tensor laid out exactly like y in that call (dense
 * [Nb][Ho][Wo][C_out], or [Nb*P'][C_out] with ASX_OUT_COMPACT).  Only kept rows of it are read.
 *   residual_dev : device pointer owned by the caller, aligned like y, valid during every following
 *                  asx_run of this layer; NULL (the default) switches the add off.
 * Not available with ASX_IMPL_NAIVE (asx_run returns ASX_ERR_INVALID_ARG).
 */
asx_status asx_set_residual(asx_layer* layer, const void* residual_dev);

/*
 * Rebuild the kept-row list from the stored mask (stage i alone; the same work the
 * ASX_RECOMPACT flag does inside asx_run).  Asynchronous on `cuda_stream`; allocates nothing.
 * ASX_ERR_NO_MASK before any asx_set_mask*.
 */
asx_status asx_recompact(asx_layer* layer, void* cuda_stream);

/*
 * Run the layer (Section 3.2 stages i-iii fused): gather the kept windows of x, multiply by
 * the filters on the tensor cores, add the bias, apply the activation, write kept rows to
 * their NHWC positions and zeros to the dropped ones.  Every element of y is written once.
 *   x    : device, bf16 [Nb][H][W][C_in], 16-byte aligned when C_in % 8 == 0, else 2-byte.
 *   w    : device, bf16 [C_out][kh][kw][C_in], same alignment rule.
 *   bias : device, fp32 [C_out], 4-byte aligned, or NULL for zero bias.
 *   y    : device, bf16 [Nb][Ho][Wo][C_out], Ho = (H + 2*pad - kh)/stride + 1 (Wo alike);
 *          16-byte aligned when C_out % 8 == 0, else 2-byte; must not overlap x.
 *   flags: OR of ASX_ACT_RELU or ASX_ACT_SILU, ASX_RECOMPACT, ASX_IMPL_NAIVE, ASX_OUT_COMPACT, ASX_IN_COMPACT, ASX_F32,
 *          ASX_IMPL_ROW_GATHER or ASX_IMPL_WINDOW_PATCH.
 *          Dropped positions are 0 under every activation (each maps 0 to 0; no bias is added there).  With
 *          ASX_OUT_COMPACT y is bf16 [Nb*P'][C_out] (P' = kept entries of the mask, which must then be
 *          shared by the batch); with ASX_IN_COMPACT x is bf16 [Nb*P'_in][C_in] (see asx_set_input_mask).
 *          With ASX_F32 x, w and y are fp32 with the same shapes (16-byte aligned when the channel
 *          count is a multiple of 4, else 4-byte; channel counts that are not are zero-padded to one
 *          in layer-owned copies).  The tensor cores then read each operand as TF32: sign, exponent
 *          and the upper 10 mantissa bits, the lower 13 bits are ignored (so inputs whose lower 13
 *          mantissa bits are zero are multiplied exactly); sums, bias and activation are fp32 and y is
 *          written unrounded.  ASX_IMPL_NAIVE with ASX_F32 multiplies the full fp32 values.  Not
 *          together with ASX_OUT_COMPACT, ASX_IN_COMPACT or a residual (ASX_ERR_UNSUPPORTED).
 * Asynchronous on `cuda_stream`.  Allocates in two cases only, on first use and when the buffers
 * must grow: when C_in % 8 != 0 the layer keeps copies of x and w with the channels zero-padded to
 * a multiple of 8 (refreshed by a small kernel on every call); and when a layer has far fewer
 * 128-row tiles than the GPU has SMs and a long reduction (K of a few thousand), the k range of a
 * tile is shared between thread blocks that exchange fp32 partial tiles through a layer-owned
 * workspace (tiles x shares x 128 x tile width floats).  Partial sums are added in a fixed order,
 * so results do not depend on scheduling.  Errors: ASX_ERR_NO_MASK, ASX_ERR_SHAPE when
 * the mask length is neither Ho*Wo nor Nb*Ho*Wo, ASX_ERR_INVALID_ARG, ASX_ERR_ALIGN,
 * ASX_ERR_UNSUPPORTED when Nb*Ho*Wo or a tensor's element count reaches 2^31.
 */
asx_status asx_run(asx_layer* layer, const void* x, int Nb, int H, int W,
                   const void* w, const float* bias, void* y, int flags, void* cuda_stream);

/*
 * Kept-row list of the current mask.  Waits for the stream last used with this layer.
 * *count receives the number of kept mask entries; *dev_kept a device pointer to `count`
 * ascending int32 positions, owned by the layer and valid until the next asx_set_mask*,
 * ASX_RECOMPACT run or asx_destroy.  Either output pointer may be NULL.
 */
asx_status asx_get_kept(asx_layer* layer, int64_t* count, const int32_t** dev_kept);

/*
 * Copy the kept-row list to host memory.  Waits for the stream last used with this layer.
 * *count receives the number of kept entries; at most `capacity` of them are written to
 * host_out (which may be NULL when capacity is 0).
 */
asx_status asx_get_kept_host(asx_layer* layer, int32_t* host_out, int64_t capacity, int64_t* count);

/* Copy the stored mask (0/1 bytes) to host memory; `rows` must equal the stored length. */
asx_status asx_get_mask(asx_layer* layer, uint8_t* host_mask_out, int64_t rows);

/*
 * Waits for the stream last used with this layer and reports the kernels' status word:
 * ASX_OK, or ASX_ERR_TIMEOUT if a bounded wait inside a kernel ran out (the output of that
 * call is then undefined; the CUDA context stays usable).  The word is cleared by the call.
 */
asx_status asx_last_device_status(asx_layer* layer);

/*
 * Which form of the lowering (Section 3.2, stage i) the last asx_run on this layer used:
 *   ASX_FORM_NONE (no run yet), ASX_FORM_NAIVE (ASX_IMPL_NAIVE), ASX_FORM_ROW_GATHER_COPY (16-byte copies per
 *   filter tap and kept row), ASX_FORM_ROW_GATHER_TMA (TMA row gather per filter tap and kept row),
 *   ASX_FORM_WINDOW_PATCH (a tile's window range loaded once, filter taps cut out of it into tensor memory).
 * All forms compute the same result up to summation order; this only reports the choice (tests, tuning).
 */
enum { ASX_FORM_NONE = 0, ASX_FORM_NAIVE = 1, ASX_FORM_ROW_GATHER_COPY = 2, ASX_FORM_ROW_GATHER_TMA = 3, ASX_FORM_WINDOW_PATCH = 4 };
asx_status asx_last_run_form(const asx_layer* layer, int* form);

/*
 * Bound of every wait inside the fused kernels of this layer (on a pipeline barrier or on another
 * block's partial sums), in GPU clock cycles; cycles <= 0 restores the default of about two seconds.
 * A wait that runs out makes every role of the kernel leave, the call's output is undefined and
 * asx_last_device_status reports ASX_ERR_TIMEOUT; the next asx_run starts clean.  The method itself has
 * no such notion (the paper runs on one CPU thread pool); this is a property of the GPU pipeline.
 */
asx_status asx_set_wait_limit(asx_layer* layer, int64_t cycles);

/*
 * Test hook for the bounded waits (no counterpart in the paper).  Layers with few kept rows and a long
 * reduction share a tile's k-blocks between thread blocks, which meet at a per-tile arrival counter in
 * the layer's workspace.  This call overwrites the arrival counter of output tile `tile` with `value`
 * (in stream order); a value the arrivals can never lift to the number of shares makes the waiting
 * blocks run into their wait limit, which is how the time-out path is exercised from the host without
 * faulting or hanging the GPU.  ASX_ERR_UNSUPPORTED if the layer's last plan did not share k-blocks (no
 * counters exist), ASX_ERR_INVALID_ARG for a tile outside the workspace.  asx_last_device_status puts
 * the counters back to zero after a reported time-out.
 */
asx_status asx_debug_set_split_counter(asx_layer* layer, int64_t tile, int32_t value, void* cuda_stream);

/* Free the layer and the device memory it owns.  NULL is allowed. */
asx_status asx_destroy(asx_layer* layer);

/*
 * Stand-alone mask compaction (the kept-row enumeration of Algorithm 2's first function).
 *   mask_dev  : device, `rows` bytes (0 / non-zero), any alignment.
 *   kept_dev  : device, room for `rows` int32; receives the ascending kept positions.
 *   count_dev : device, one int32; receives the number of kept positions.
 *   scratch_dev, scratch_bytes : device scratch of at least asx_compact_scratch_bytes(rows)
 *               bytes, 8-byte aligned; contents on entry are irrelevant (every word that is
 *               read is written first, in stream order).  Calls sharing one scratch buffer
 *               must not overlap.
 * Masks of more than 16384 rows take two launches (kept rows counted per run of tiles, then the
 * ordered write, in which every block sums the counts in front of its run; the mask is read
 * twice), smaller ones a single block; no block waits for another.
 * 0 <= rows < 2^31.  Asynchronous on `cuda_stream`; allocates nothing.
 */
int64_t asx_compact_scratch_bytes(int64_t rows);
asx_status asx_compact(const uint8_t* mask_dev, int64_t rows, int32_t* kept_dev,
                       int32_t* count_dev, void* scratch_dev, int64_t scratch_bytes,
                       void* cuda_stream);
/* Waits for `cuda_stream`, then reports the status word the last asx_compact left in this scratch
 * buffer: ASX_OK, or ASX_ERR_TIMEOUT if a kernel gave up in a bounded wait.  The compaction kernels
 * no longer contain any wait on another block, so after a completed call this always reports
 * ASX_OK; the entry point is kept so that callers built against it keep linking. */
asx_status asx_compact_status(const void* scratch_dev, void* cuda_stream);

/*
 * Data-dependent mask (the family the paper contrasts its fixed masks with in Section 2: sparsity
 * that comes from the activations themselves, such as the zeros a ReLU leaves): mask_dev[r] = 1 iff
 * at least one of the C channels of row r of a bfloat16 tensor [rows][C] is strictly positive
 * (zeros of either sign and NaN are not positive; denormals and +inf are).  The result has one
 * entry per lowered row and can be given to asx_set_mask as a device pointer (rows = Nb*Ho*Wo),
 * followed by asx_run with ASX_RECOMPACT or not.
 *   x_dev    : device, bf16 [rows][C], 2-byte aligned (16-byte aligned input with C in
 *              {8, 16, 32, 64, 128, 256} takes the vectorised kernel).
 *   mask_dev : device, `rows` bytes, written 0 / 1.   0 <= rows < 2^31, 1 <= C <= 2^20.
 * Asynchronous on `cuda_stream`; allocates nothing.
 */
asx_status asx_mask_from_activation(const void* x_dev, int64_t rows, int C, uint8_t* mask_dev, void* cuda_stream);

/*
 * Mask compaction without any allocation (the paper has no counterpart: this is a convenience
 * of this library).  Same inputs, outputs and result as asx_compact, but the scan's scratch is
 * a fixed array inside the library, so neither the caller nor the library allocates anything:
 * no cudaMalloc, no cudaFree, no pooled allocator.  Meant for callers that cannot allocate where
 * they stand: a latency-critical serving loop (cudaMalloc synchronises the device), code that
 * runs after another framework took all device memory, a plug-in that only receives raw buffers.
 *   rows : 0 <= rows <= ASX_COMPACT_STATIC_MAX_ROWS; more returns ASX_ERR_UNSUPPORTED and
 *          launches nothing (use asx_compact with your own scratch instead).
 *   mask_dev, kept_dev (room for `rows` int32), count_dev (one int32): device pointers as for
 *          asx_compact.
 * The array (about 32 KB) is part of the library image on every GPU that loads it.  The first
 * call on each device looks up the array's device address; make that first call outside any
 * stream capture, and do not let two host threads make a device's first call at the same moment
 * (both would look the address up; they store the same value).  All calls on a device share the
 * one array and it keeps the last call's contents: every call overwrites, in stream order, each
 * word it later reads, so nothing needs clearing, but two calls that may overlap on the GPU
 * (different streams without an ordering between them) race on it and give undefined lists.
 * The mask may have been written by the kernel launched just before on the same stream (for
 * instance asx_mask_from_activation): the kernels read it only after that kernel has finished.
 */
#define ASX_COMPACT_STATIC_MAX_ROWS (1 << 24)
asx_status asx_compact_static(const uint8_t* mask_dev, int64_t rows, int32_t* kept_dev,
                              int32_t* count_dev, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* ASX_H_ */
