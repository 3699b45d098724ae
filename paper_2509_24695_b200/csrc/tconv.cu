// Temporal convolution of the Mix-FFN (kernel size 3 over frames, per channel, with a shortcut) and its
// block-causal form with a one-frame cache (Sec. 3.1, Sec. 3.2 "Block Causal Mix-FFN", Algorithm 1's conv cache).
//
// The work is a pure stream: every element of x is needed by three output frames, every element of y is
// written once; 2 * sizeof(element) bytes per element is all that has to cross HBM.  One thread owns
// 16 bytes of a frame (8 bf16 / 4 fp32 channels of one position) and walks the frame axis with the previous,
// current and next frame's values in registers, so x is read from memory exactly once and no shared memory or
// cache reuse is involved; the loads of the frame after next are issued before the current frame's arithmetic,
// which keeps three 16-byte loads per thread in flight.  Consecutive threads take consecutive 16-byte pieces
// (fully coalesced 512-byte warp accesses).  The cached frame is read by, and the new cache written by, the same
// thread that owns that piece, so updating the cache in place needs no ordering between threads.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "common.cuh"
#include "tconv.h"

namespace linattn {
namespace {

// 16 bytes of T: kept packed in registers, widened to floats only where the arithmetic happens
template <typename T>
struct Vec;

template <>
struct Vec<__nv_bfloat16> {
  static constexpr int N = 8;
  uint4 r;
  __device__ __forceinline__ void load(const __nv_bfloat16* p) { r = __ldcs(reinterpret_cast<const uint4*>(p)); }
  __device__ __forceinline__ void zero() { r = make_uint4(0, 0, 0, 0); }
  __device__ __forceinline__ void unpack(float (&f)[8]) const {
    const unsigned u[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      f[2 * i] = __uint_as_float(u[i] << 16);
      f[2 * i + 1] = __uint_as_float(u[i] & 0xffff0000u);
    }
  }
  __device__ __forceinline__ void pack(const float (&f)[8]) {
    unsigned u[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const __nv_bfloat162 h = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
      u[i] = *reinterpret_cast<const unsigned*>(&h);
    }
    r = make_uint4(u[0], u[1], u[2], u[3]);
  }
  __device__ __forceinline__ void store(__nv_bfloat16* p, bool streaming) const {
    if (streaming) __stcs(reinterpret_cast<uint4*>(p), r);
    else *reinterpret_cast<uint4*>(p) = r;
  }
};

template <>
struct Vec<float> {
  static constexpr int N = 4;
  float4 r;
  __device__ __forceinline__ void load(const float* p) { r = __ldcs(reinterpret_cast<const float4*>(p)); }
  __device__ __forceinline__ void zero() { r = make_float4(0.f, 0.f, 0.f, 0.f); }
  __device__ __forceinline__ void unpack(float (&f)[4]) const { f[0] = r.x; f[1] = r.y; f[2] = r.z; f[3] = r.w; }
  __device__ __forceinline__ void pack(const float (&f)[4]) { r = make_float4(f[0], f[1], f[2], f[3]); }
  __device__ __forceinline__ void store(float* p, bool streaming) const {
    if (streaming) __stcs(reinterpret_cast<float4*>(p), r);
    else *reinterpret_cast<float4*>(p) = r;
  }
};

struct TconvParams {
  const void* x;
  void* y;                // null: only the cache is updated
  const float* w;         // [3][D]
  const void* cache_in;   // null: zeros in front of the first frame
  void* cache_out;        // null: the cache is not written
  long long T, T_b;       // frames, frames per block (the frame after a block's last one counts as zero)
  long long frame;        // elements of one frame: HW * D
  long long sb, sby;      // elements between batch entries of x, of y
  int D;
};

template <typename T>
__global__ void __launch_bounds__(256, 4) tconv_kernel(const TconvParams p) {
  using V = Vec<T>;
  const long long col = ((long long)blockIdx.x * blockDim.x + threadIdx.x) * V::N;   // element within a frame
  if (col >= p.frame) return;
  const int b = blockIdx.y;
  const T* x = static_cast<const T*>(p.x) + b * p.sb + col;
  T* cache_out = p.cache_out ? static_cast<T*>(p.cache_out) + b * p.frame + col : nullptr;
  if (!p.y) {  // absorb only: the cache becomes the last frame
    V last;
    last.load(x + (p.T - 1) * p.frame);
    if (cache_out) last.store(cache_out, false);
    return;
  }
  T* y = static_cast<T*>(p.y) + b * p.sby + col;

  const int c0 = (int)(col % p.D);
  float w0[V::N], w1[V::N], w2[V::N];
#pragma unroll
  for (int i = 0; i < V::N; i += 4) {
    const float4 a = __ldg(reinterpret_cast<const float4*>(p.w + c0 + i));
    const float4 c = __ldg(reinterpret_cast<const float4*>(p.w + p.D + c0 + i));
    const float4 d = __ldg(reinterpret_cast<const float4*>(p.w + 2 * p.D + c0 + i));
    w0[i] = a.x; w0[i + 1] = a.y; w0[i + 2] = a.z; w0[i + 3] = a.w;
    w1[i] = c.x; w1[i + 1] = c.y; w1[i + 2] = c.z; w1[i + 3] = c.w;
    w2[i] = d.x; w2[i + 1] = d.y; w2[i + 2] = d.z; w2[i + 3] = d.w;
  }

  V prev, cur, nxt, ahead;
  if (p.cache_in) prev.load(static_cast<const T*>(p.cache_in) + b * p.frame + col);
  else prev.zero();
  cur.load(x);
  if (p.T > 1) nxt.load(x + p.frame); else nxt.zero();
  long long in_block = 0;   // index of frame t within its block
  for (long long t = 0; t < p.T; ++t) {
    if (t + 2 < p.T) ahead.load(x + (t + 2) * p.frame); else ahead.zero();
    const bool block_end = ++in_block == p.T_b || t + 1 == p.T;
    if (block_end) in_block = 0;
    float fp[V::N], fc[V::N], fn[V::N], fo[V::N];
    prev.unpack(fp); cur.unpack(fc); nxt.unpack(fn);
#pragma unroll
    for (int i = 0; i < V::N; ++i) {
      const float n = block_end ? 0.f : fn[i];
      fo[i] = fmaf(w2[i], n, fmaf(w1[i], fc[i], fmaf(w0[i], fp[i], fc[i])));
    }
    V out;
    out.pack(fo);
    out.store(y + t * p.frame, true);
    prev = cur; cur = nxt; nxt = ahead;
  }
  if (cache_out) prev.store(cache_out, false);   // prev is now the last frame
}

int check(const tconv_desc* d, long long T, long long* frame, long long* sb, long long* sby, size_t* esz) {
  if (!d || T < 0) return LINATTN_ERR_INVALID_ARG;
  if (d->B < 1 || d->HW < 1 || d->D < 1 || d->stride_b < 0 || d->stride_b_y < 0) return LINATTN_ERR_INVALID_ARG;
  if (d->dtype != LINATTN_BF16 && d->dtype != LINATTN_F32) return LINATTN_ERR_INVALID_ARG;
  if (d->B > 65535) return LINATTN_ERR_UNSUPPORTED;
  const int vec = d->dtype == LINATTN_BF16 ? 8 : 4;
  if (d->D % vec) return LINATTN_ERR_UNSUPPORTED;
  *esz = d->dtype == LINATTN_BF16 ? 2 : 4;
  *frame = (long long)d->HW * d->D;
  *sb = d->stride_b ? d->stride_b : T * *frame;
  *sby = d->stride_b_y ? d->stride_b_y : T * *frame;
  if (*sb % vec || *sby % vec) return LINATTN_ERR_BAD_ALIGNMENT;
  if (*sb < T * *frame || *sby < T * *frame) return LINATTN_ERR_INVALID_ARG;
  return LINATTN_OK;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

bool overlap(const void* a, size_t na, const void* b, size_t nb) {
  const char* pa = static_cast<const char*>(a);
  const char* pb = static_cast<const char*>(b);
  return a && b && pa < pb + nb && pb < pa + na;
}

int run(const tconv_desc* d, long long T, long long T_b, const void* x, const float* w, const void* cache_in,
        void* cache_out, void* y, void* stream) {
  long long frame, sb, sby;
  size_t esz;
  int st = check(d, T, &frame, &sb, &sby, &esz);
  if (st != LINATTN_OK) return st;
  if (T == 0) return LINATTN_OK;
  if (!x || (!w && y) || T_b < 1) return LINATTN_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(y) || !aligned16(w) || !aligned16(cache_in) || !aligned16(cache_out))
    return LINATTN_ERR_BAD_ALIGNMENT;
  const size_t span = (size_t)((d->B - 1) * sb + T * frame) * esz, span_y = (size_t)((d->B - 1) * sby + T * frame) * esz;
  const size_t cbytes = (size_t)d->B * frame * esz;
  if (overlap(x, span, y, span_y) || overlap(x, span, cache_in, cbytes) || overlap(x, span, cache_out, cbytes) ||
      overlap(y, span_y, cache_in, cbytes) || overlap(y, span_y, cache_out, cbytes))
    return LINATTN_ERR_INVALID_ARG;
  TconvParams p{x, y, w, cache_in, cache_out, T, T_b, frame, sb, sby, d->D};
  const int vec = d->dtype == LINATTN_BF16 ? 8 : 4;
  const long long cols = frame / vec;
  dim3 grid((unsigned)((cols + 255) / 256), (unsigned)d->B);
  if (d->dtype == LINATTN_BF16) tconv_kernel<__nv_bfloat16><<<grid, 256, 0, (cudaStream_t)stream>>>(p);
  else tconv_kernel<float><<<grid, 256, 0, (cudaStream_t)stream>>>(p);
  count_launches(1);
  return cudaGetLastError() == cudaSuccess ? LINATTN_OK : LINATTN_ERR_CUDA;
}

}  // namespace
}  // namespace linattn

using namespace linattn;

extern "C" {

int tconv_cache_bytes(const tconv_desc* desc, size_t* cache_bytes) {
  long long frame, sb, sby;
  size_t esz;
  if (!cache_bytes) return LINATTN_ERR_INVALID_ARG;
  int st = check(desc, 0, &frame, &sb, &sby, &esz);
  if (st != LINATTN_OK) return st;
  *cache_bytes = (size_t)desc->B * frame * esz;
  return LINATTN_OK;
}

int tconv_cache_reset(const tconv_desc* desc, void* cache, void* stream) {
  size_t bytes;
  int st = tconv_cache_bytes(desc, &bytes);
  if (st != LINATTN_OK) return st;
  if (!cache) return LINATTN_ERR_INVALID_ARG;
  return cudaMemsetAsync(cache, 0, bytes, (cudaStream_t)stream) == cudaSuccess ? LINATTN_OK : LINATTN_ERR_CUDA;
}

int tconv_forward(const tconv_desc* desc, int64_t T, const void* x, const float* w, void* y, void* stream) {
  if (T > 0 && !y) return LINATTN_ERR_INVALID_ARG;
  return run(desc, T, T > 0 ? T : 1, x, w, nullptr, nullptr, y, stream);
}

int tconv_block_step(const tconv_desc* desc, int64_t T_b, const void* x_blk, const float* w, void* cache, void* y_blk,
                     int commit, void* stream) {
  if (!cache || (!y_blk && !commit && T_b > 0)) return LINATTN_ERR_INVALID_ARG;
  return run(desc, T_b, T_b > 0 ? T_b : 1, x_blk, w, cache, commit ? cache : nullptr, y_blk, stream);
}

int tconv_prefill(const tconv_desc* desc, int64_t n_blocks, int64_t T_b, const void* x, const float* w, void* cache,
                  void* y, void* stream) {
  if (!cache || n_blocks < 0 || T_b < 0) return LINATTN_ERR_INVALID_ARG;
  if (n_blocks > 0 && T_b > 0 && !y) return LINATTN_ERR_INVALID_ARG;
  return run(desc, n_blocks * T_b, T_b > 0 ? T_b : 1, x, w, cache, cache, y, stream);
}

}  // extern "C"
