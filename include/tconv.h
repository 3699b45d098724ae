/*
 * tconv.h -- C ABI of the temporal convolution of the Mix-FFN and of its block-causal form with a
 * one-frame cache (sm_100a).
 *
 * The operation (Sec. 3.1 "Mix-FFN with Spatial-Temporal Mixture"; Sec. 3.2 "Block Causal Mix-FFN"; the
 * conv cache f of Algorithm 1): a 1D convolution with kernel size 3 over the frame axis, added to its
 * input through a shortcut, at the end of the Mix-FFN.  For frames x_t of HW positions and D channels
 *
 *     y_t = x_t + w0 * x_{t-1} + w1 * x_t + w2 * x_{t+1}        (per position and channel)
 *
 *   bidirectional (tconv_forward): x_{-1} = x_T = 0.
 *   block-causal (tconv_block_step, tconv_prefill): frames come in blocks; the frame after a block's last
 *   one is an all-zero frame (a block never sees a later block), the frame before a block's first one is
 *   the last frame of the previous block, which is all the layer keeps of the past: a cache of ONE frame,
 *   B*HW*D elements whatever the number of blocks seen.  Before the first block the cache is all zero.
 *
 * Readings where the paper is silent: the taps are per channel (w[tau][c], tau = 0: previous frame,
 * 1: the frame itself, 2: next frame; a cross-correlation), there is no bias.
 *
 * Conventions
 *  - x, y, cache and w are DEVICE pointers owned by the caller; nothing is allocated, freed or kept.
 *  - x and y are [B][T][HW][D] with D contiguous, positions and frames dense; element (b, t, p, c) of x is at
 *    b*stride_b + (t*HW + p)*D + c (of y: stride_b_y), a stride of 0 selecting the dense T*HW*D.  (A block of
 *    a longer tensor is the sub-view at its first frame with the long tensor's batch stride.)
 *  - dtype LINATTN_BF16: x, y, cache bfloat16, arithmetic fp32 (y = round_to_nearest_even of
 *    fma(w2, x_next, fma(w1, x, fma(w0, x_prev, x)))); LINATTN_F32: fp32 throughout.
 *  - w is fp32 [3][D].  cache is [B][HW][D] of the tensors' dtype, dense.
 *  - D must be a multiple of 8 (bf16) or 4 (fp32); pointers 16-byte aligned; batch strides multiples
 *    of 8 / 4 elements.  y must not overlap x; the cache must overlap neither.
 *  - `stream` is a cudaStream_t passed as void*.  Calls enqueue one kernel and return.
 *  - Returns LINATTN_OK or a negative linattn_status (linattn.h); arguments are checked before the
 *    launch; T = 0 is a successful no-op.  No device-side waits exist in these kernels.
 */
#ifndef TCONV_H_
#define TCONV_H_

#include "linattn.h"

#ifdef __cplusplus
extern "C" {
#endif

typedef struct tconv_desc {
  int32_t B;           /* batch entries */
  int32_t HW;          /* positions of one frame */
  int32_t D;           /* channels */
  int32_t dtype;       /* linattn_dtype */
  int64_t stride_b;    /* elements between batch entries of x; 0 = dense */
  int64_t stride_b_y;  /* the same for y; 0 = dense */
} tconv_desc;

/* Bytes of the conv cache: one frame, B*HW*D elements. */
LINATTN_API int tconv_cache_bytes(const tconv_desc* desc, size_t* cache_bytes);

/* Zero the cache (the state before the first block). */
LINATTN_API int tconv_cache_reset(const tconv_desc* desc, void* cache, void* stream);

/* Bidirectional layer over T frames (Sec. 3.1). */
LINATTN_API int tconv_forward(const tconv_desc* desc, int64_t T, const void* x, const float* w, void* y, void* stream);

/* One block of T_b frames with the cached frame in front and the zero frame behind (Sec. 3.2).
 * commit != 0: afterwards the cache holds this block's last frame (the clean block of Algorithm 1);
 * commit == 0: the cache is only read (a denoising step of Algorithm 1).  y may be NULL with commit != 0:
 * the block is only absorbed into the cache. */
LINATTN_API int tconv_block_step(const tconv_desc* desc, int64_t T_b, const void* x_blk, const float* w, void* cache,
                                 void* y_blk, int commit, void* stream);

/* n_blocks consecutive blocks of T_b frames in one launch over [B][n_blocks*T_b][HW][D] tensors, starting
 * from the cache and leaving the last block's last frame in it: the result of n_blocks calls of
 * tconv_block_step with commit, bit for bit. */
LINATTN_API int tconv_prefill(const tconv_desc* desc, int64_t n_blocks, int64_t T_b, const void* x, const float* w,
                              void* cache, void* y, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* TCONV_H_ */
