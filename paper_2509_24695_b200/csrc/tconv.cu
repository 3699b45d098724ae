// Temporal convolution of the Mix-FFN (kernel size 3 over frames, per channel, with a shortcut) and its
// block-causal form with a one-frame cache (Sec. 3.1, Sec. 3.2 "Block Causal Mix-FFN", Algorithm 1's conv cache).
//
// The work is a pure stream: every element of x is needed by three output frames, every element of y is
// written once; 2 * sizeof(element) bytes per element is all that has to cross HBM.  One thread owns
// 16 bytes of a frame (8 bf16 / 4 fp32 channels of one position) and walks the frame axis with the previous,
// current and next frame's values in registers, so x is read from memory exactly once and no shared memory or
// cache reuse is involved; the loads of three further frames are in flight while a frame is computed.  Consecutive threads take consecutive 16-byte pieces
// (fully coalesced 512-byte warp accesses).  The cached frame is read by, and the new cache written by, the same
// thread that owns that piece, so updating the cache in place needs no ordering between threads.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "common.cuh"
#include "tconv.h"

namespace linattn {
namespace {

// 16 bytes of a frame as they sit in memory, and as pairs of floats for the arithmetic
template <typename T>
struct Piece;

template <>
struct Piece<__nv_bfloat16> {
  static constexpr int PAIRS = 4;
  using Raw = uint4;
  static __device__ __forceinline__ Raw zero() { return make_uint4(0, 0, 0, 0); }
  static __device__ __forceinline__ void unpack(const Raw& r, float2 (&f)[4]) {
    const unsigned u[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) f[i] = make_float2(__uint_as_float(u[i] << 16), __uint_as_float(u[i] & 0xffff0000u));
  }
  static __device__ __forceinline__ Raw pack(const float2 (&f)[4]) {   // round to nearest even
    unsigned u[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const __nv_bfloat162 h = __floats2bfloat162_rn(f[i].x, f[i].y);
      u[i] = *reinterpret_cast<const unsigned*>(&h);
    }
    return make_uint4(u[0], u[1], u[2], u[3]);
  }
};

template <>
struct Piece<float> {
  static constexpr int PAIRS = 2;
  using Raw = float4;
  static __device__ __forceinline__ Raw zero() { return make_float4(0.f, 0.f, 0.f, 0.f); }
  static __device__ __forceinline__ void unpack(const Raw& r, float2 (&f)[2]) {
    f[0] = make_float2(r.x, r.y);
    f[1] = make_float2(r.z, r.w);
  }
  static __device__ __forceinline__ Raw pack(const float2 (&f)[2]) { return make_float4(f[0].x, f[0].y, f[1].x, f[1].y); }
};

// Two fp32 fused multiply-adds in one instruction (sm_100 has a packed f32x2 FMA pipe): the kernel issues an
// instruction on every other cycle per scheduler as it is, so halving the FMA count shows in the run time.
__device__ __forceinline__ float2 fma2(float2 a, float2 b, float2 c) {
  unsigned long long ra, rb, rc, rd;
  asm("mov.b64 %0, {%1, %2};" : "=l"(ra) : "f"(a.x), "f"(a.y));
  asm("mov.b64 %0, {%1, %2};" : "=l"(rb) : "f"(b.x), "f"(b.y));
  asm("mov.b64 %0, {%1, %2};" : "=l"(rc) : "f"(c.x), "f"(c.y));
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(rd) : "l"(ra), "l"(rb), "l"(rc));
  float2 d;
  asm("mov.b64 {%0, %1}, %2;" : "=f"(d.x), "=f"(d.y) : "l"(rd));
  return d;
}

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

// kAhead: frames in flight beyond the next one.  Long clips run with 3 (79 registers, 3 blocks per SM); a block
// step of up to three frames has all its frames in flight with 1 and fits 4 blocks per SM.
template <typename T, int kAhead>
__global__ void __launch_bounds__(256, kAhead > 1 ? 3 : 4) tconv_kernel(const TconvParams p) {
  using Pc = Piece<T>;
  using Raw = typename Pc::Raw;
  constexpr int PAIRS = Pc::PAIRS;
  const unsigned col = (blockIdx.x * blockDim.x + threadIdx.x) * (2 * PAIRS);   // element within a frame (< 2^31)
  if (col >= p.frame) return;
  const int b = blockIdx.y;
  const T* x = static_cast<const T*>(p.x) + b * p.sb + col;
  Raw* cache_out = p.cache_out ? reinterpret_cast<Raw*>(static_cast<T*>(p.cache_out) + b * p.frame + col) : nullptr;
  auto frame_of = [&](long long t) { return __ldcs(reinterpret_cast<const Raw*>(x + t * p.frame)); };
  if (!p.y) {  // absorb only: the cache becomes the last frame
    if (cache_out) *cache_out = frame_of(p.T - 1);
    return;
  }
  T* y = static_cast<T*>(p.y) + b * p.sby + col;

  const int c0 = (int)(col % (unsigned)p.D);
  float2 w[3][PAIRS];
#pragma unroll
  for (int tau = 0; tau < 3; ++tau)
#pragma unroll
    for (int i = 0; i < PAIRS; i += 2) {
      const float4 a = __ldg(reinterpret_cast<const float4*>(p.w + tau * p.D + c0 + 2 * i));
      w[tau][i] = make_float2(a.x, a.y);
      w[tau][i + 1] = make_float2(a.z, a.w);
    }

  // frames t-1, t, t+1 as floats (each frame is widened once), frames t+2 .. t+1+kAhead as loaded
  Raw r_prev = Pc::zero(), r_cur, r_nxt = Pc::zero(), raw[kAhead];
  if (p.cache_in) r_prev = __ldcs(reinterpret_cast<const Raw*>(static_cast<const T*>(p.cache_in) + b * p.frame + col));
  r_cur = frame_of(0);
  if (p.T > 1) r_nxt = frame_of(1);
#pragma unroll
  for (int i = 0; i < kAhead; ++i) raw[i] = 2 + i < p.T ? frame_of(2 + i) : Pc::zero();
  float2 fp[PAIRS], fc[PAIRS], fn[PAIRS];
  Pc::unpack(r_prev, fp); Pc::unpack(r_cur, fc); Pc::unpack(r_nxt, fn);
  long long in_block = 0;   // index of frame t within its block
  for (long long t = 0; t < p.T; ++t) {
    Raw fresh = Pc::zero();
    if (t + 2 + kAhead < p.T) fresh = frame_of(t + 2 + kAhead);
    const bool block_end = ++in_block == p.T_b || t + 1 == p.T;   // the same for every thread: no divergence
    if (block_end) in_block = 0;
    float2 fo[PAIRS];
#pragma unroll
    for (int i = 0; i < PAIRS; ++i) fo[i] = fma2(w[1][i], fc[i], fma2(w[0][i], fp[i], fc[i]));
    if (!block_end) {   // behind a block's last frame stands the all-zero frame: nothing to add
#pragma unroll
      for (int i = 0; i < PAIRS; ++i) fo[i] = fma2(w[2][i], fn[i], fo[i]);
    }
    __stcs(reinterpret_cast<Raw*>(y + t * p.frame), Pc::pack(fo));
#pragma unroll
    for (int i = 0; i < PAIRS; ++i) { fp[i] = fc[i]; fc[i] = fn[i]; }
    Pc::unpack(raw[0], fn);
#pragma unroll
    for (int i = 0; i + 1 < kAhead; ++i) raw[i] = raw[i + 1];
    raw[kAhead - 1] = fresh;
  }
  if (cache_out) *cache_out = Pc::pack(fp);   // fp is now the last frame; packing widened elements is exact
}

// Block steps of up to three frames (the paper's blocks are three latent frames).  Here a thread's share is only
// four 16-byte loads (the cached frame and the block's frames), so what bounds the kernel is how many bytes an
// SM keeps in flight, and registers are the wrong place to hold them: each thread streams its pieces into a
// private ring in shared memory with cp.async (no registers held, nothing to poll: cp.async.wait_group is a
// hardware wait), three tiles deep, and a persistent grid of four CTAs per SM walks the tiles (measured: threads
// matter more than depth; 3 x 4 beat 6 x 2 by 12 % and 12 x 1 by 35 %; five CTAs per SM spill).  A tile is 256
// consecutive 16-byte pieces of one batch entry's frame; no data is shared between threads, so no CTA-wide
// synchronisation is needed.  Same arithmetic, in the same order, as tconv_kernel: the results are the same bits.
constexpr int kStepStages = 3;
constexpr int kStepSegs = 4;   // cached frame + up to three frames
constexpr int kStepCtasPerSm = 4;

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((unsigned)__cvta_generic_to_shared(smem_dst)), "l"(gmem_src)
               : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

template <typename T>
__global__ void __launch_bounds__(256, kStepCtasPerSm) tconv_step_kernel(const TconvParams p, int tiles_per_batch, int total_tiles) {
  using Pc = Piece<T>;
  using Raw = typename Pc::Raw;
  constexpr int PAIRS = Pc::PAIRS;
  extern __shared__ uint4 ring_raw[];
  Raw* ring = reinterpret_cast<Raw*>(ring_raw);   // [stage][segment][thread]
  const int tid = (int)threadIdx.x;
  const int nf = (int)p.T;                        // 1..3 frames
  auto locate = [&](int tile, int& b, unsigned& col) {
    b = tile / tiles_per_batch;
    col = (unsigned)((tile - b * tiles_per_batch) * 256 + tid) * (2 * PAIRS);
  };
  auto issue = [&](int tile, int stage) {
    if (tile < total_tiles) {
      int b;
      unsigned col;
      locate(tile, b, col);
      if (col < p.frame) {
        Raw* dst = ring + (stage * kStepSegs) * 256 + tid;
        cp_async16(dst, static_cast<const T*>(p.cache_in) + (long long)b * p.frame + col);
        const T* x = static_cast<const T*>(p.x) + b * p.sb + col;
        for (int t = 0; t < nf; ++t) cp_async16(dst + (1 + t) * 256, x + t * p.frame);
      }
    }
    cp_async_commit();   // one group per tile, empty or not, so that the count below stays uniform
  };
  const int first = (int)blockIdx.x, step = (int)gridDim.x;
#pragma unroll
  for (int s = 0; s < kStepStages - 1; ++s) issue(first + s * step, s);
  int k = 0;
  for (int tile = first; tile < total_tiles; tile += step, ++k) {
    issue(tile + (kStepStages - 1) * step, (k + kStepStages - 1) % kStepStages);
    cp_async_wait<kStepStages - 1>();   // this thread's copies of `tile` have landed
    int b;
    unsigned col;
    locate(tile, b, col);
    if (col >= p.frame) continue;
    const int c0 = (int)(col % (unsigned)p.D);
    float2 w[3][PAIRS];
#pragma unroll
    for (int tau = 0; tau < 3; ++tau)
#pragma unroll
      for (int i = 0; i < PAIRS; i += 2) {
        const float4 a = __ldg(reinterpret_cast<const float4*>(p.w + tau * p.D + c0 + 2 * i));
        w[tau][i] = make_float2(a.x, a.y);
        w[tau][i + 1] = make_float2(a.z, a.w);
      }
    const Raw* src = ring + ((k % kStepStages) * kStepSegs) * 256 + tid;
    float2 fp[PAIRS], fc[PAIRS], fn[PAIRS];
    Pc::unpack(src[0], fp);
    Pc::unpack(src[256], fc);
    T* y = static_cast<T*>(p.y) + b * p.sby + col;
    for (int t = 0; t < nf; ++t) {
      const bool last = t + 1 == nf;
      if (!last) Pc::unpack(src[(2 + t) * 256], fn);
      float2 fo[PAIRS];
#pragma unroll
      for (int i = 0; i < PAIRS; ++i) fo[i] = fma2(w[1][i], fc[i], fma2(w[0][i], fp[i], fc[i]));
      if (!last) {
#pragma unroll
        for (int i = 0; i < PAIRS; ++i) fo[i] = fma2(w[2][i], fn[i], fo[i]);
      }
      __stcs(reinterpret_cast<Raw*>(y + t * p.frame), Pc::pack(fo));
#pragma unroll
      for (int i = 0; i < PAIRS; ++i) { fp[i] = fc[i]; fc[i] = fn[i]; }
    }
    if (p.cache_out)   // fp is now the block's last frame
      *reinterpret_cast<Raw*>(static_cast<T*>(p.cache_out) + (long long)b * p.frame + col) = Pc::pack(fp);
  }
  cp_async_wait<0>();
}

int sm_count_of_device() {
  int dev = 0, n = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return 0;
  return n;
}

template <typename T>
cudaError_t launch_step(const TconvParams& p, int B, cudaStream_t stream) {
  constexpr int vec = 2 * Piece<T>::PAIRS;
  const long long cols = p.frame / vec;
  const long long tpb = (cols + 255) / 256, total = tpb * B;
  if (total >= (1ll << 31)) return cudaErrorInvalidValue;
  constexpr size_t smem = (size_t)kStepStages * kStepSegs * 256 * 16;
  // the opt-in to more than 48 KB of dynamic shared memory is a per-device setting of the kernel
  static bool attr_set[64] = {false};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  if (!attr_set[dev]) {
    const cudaError_t e = cudaFuncSetAttribute(tconv_step_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    attr_set[dev] = true;
  }
  const int sms = sm_count_of_device();
  if (!sms) return cudaErrorUnknown;
  const int grid = (int)(total < kStepCtasPerSm * sms ? total : kStepCtasPerSm * sms);
  tconv_step_kernel<T><<<grid, 256, smem, stream>>>(p, (int)tpb, (int)total);
  return cudaGetLastError();
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
  if (*frame >= (1ll << 31)) return LINATTN_ERR_UNSUPPORTED;
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
  const bool few = T <= 3;
  cudaError_t e;
  // The staged kernel treats all T frames as ONE block (only the last frame gets the zero frame behind it), so it
  // takes single blocks only; a prefill of several short blocks goes to the kernel that honours T_b.
  if (few && T_b >= T && cache_in && y) {   // a block step of the paper's size: the staged kernel
    e = d->dtype == LINATTN_BF16 ? launch_step<__nv_bfloat16>(p, d->B, (cudaStream_t)stream)
                                 : launch_step<float>(p, d->B, (cudaStream_t)stream);
  } else {
    if (d->dtype == LINATTN_BF16) {
      if (few) tconv_kernel<__nv_bfloat16, 1><<<grid, 256, 0, (cudaStream_t)stream>>>(p);
      else tconv_kernel<__nv_bfloat16, 3><<<grid, 256, 0, (cudaStream_t)stream>>>(p);
    } else {
      if (few) tconv_kernel<float, 1><<<grid, 256, 0, (cudaStream_t)stream>>>(p);
      else tconv_kernel<float, 3><<<grid, 256, 0, (cudaStream_t)stream>>>(p);
    }
    e = cudaGetLastError();
  }
  count_launches(1);
  return e == cudaSuccess ? LINATTN_OK : LINATTN_ERR_CUDA;
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
