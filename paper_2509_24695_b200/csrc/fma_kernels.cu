// Plain fp32-FMA kernels for ReLU linear attention (Eq. 2 / Eq. 3 of the paper).
//
// They serve the fp32 I/O path (fp32 in, fp32 arithmetic, fp32 out) and the bf16
// shapes the tensor-core kernels do not take (head dims other than 32/64/112/128).
// Any head dim 1..128 and any element strides are accepted.
//
//   fma_state_partial : one CTA per (split-N chunk, unit) accumulates phi(K)^T V and sum phi(K)
//                       over its token range into registers and writes one partial state.
//   fma_state_reduce  : sums the chunks of a unit in a fixed order (fp64 running sum), optionally
//                       on top of an existing state (the cache update of Eq. 3).
//   fma_apply         : S and z of a unit in shared memory; 64 tokens per CTA.
#include "common.cuh"

namespace linattn {
namespace {

constexpr int kThreads = 256;
constexpr int kPitch = 132;      // shared-memory row pitch in floats (128 + 4: breaks bank alignment of rows)
constexpr int kApplyTile = 64;   // tokens per CTA in the apply kernel

template <typename T>
__device__ __forceinline__ float load_f32(const T* p);
template <>
__device__ __forceinline__ float load_f32<float>(const float* p) { return *p; }
template <>
__device__ __forceinline__ float load_f32<__nv_bfloat16>(const __nv_bfloat16* p) { return __bfloat162float(*p); }

template <typename T>
__device__ __forceinline__ void store_out(T* p, float x);
template <>
__device__ __forceinline__ void store_out<float>(float* p, float x) { *p = x; }
template <>
__device__ __forceinline__ void store_out<__nv_bfloat16>(__nv_bfloat16* p, float x) { *p = __float2bfloat16_rn(x); }

// grid (P, units).  R = ceil(d/16): each thread owns an R x R register tile of S:
// rows i = ti + 16*r (key feature), columns j = tj + 16*c (value feature).
// ROPE (Eq. 2 with its rotary factors): S is built from the rotated phi(k) (pair (2p, 2p+1) of token n turned
// by the angle whose (cosine, sine) is tab[n][p]), z from the plain phi(k).
template <typename T, int R, bool ROPE>
__global__ void __launch_bounds__(kThreads)
fma_state_partial(const T* __restrict__ k, const T* __restrict__ v, Problem p, int P, float* __restrict__ partials,
                  const __half2* __restrict__ tab) {
  constexpr int kStateTile = ROPE ? 16 : 32;  // tokens staged per iteration (three staging arrays with ROPE)
  __shared__ float Ks[kStateTile * kPitch];
  __shared__ float Vs[kStateTile * kPitch];
  __shared__ float Zs[ROPE ? kStateTile * kPitch : 1];  // plain phi(k), for z
  const int d = p.d;
  const int u = blockIdx.y, c = blockIdx.x;
  const int b = u / p.H, h = u % p.H;
  const long long chunk = (p.N + P - 1) / P;
  const long long n_begin = (long long)c * chunk;
  const long long n_end = min(p.N, n_begin + chunk);
  const int tid = threadIdx.x, ti = tid >> 4, tj = tid & 15;
  const long long base = (long long)b * p.sb + (long long)h * p.sh;

  float acc[R][R];
  float zacc[R];
#pragma unroll
  for (int r = 0; r < R; ++r) {
    zacc[r] = 0.f;
#pragma unroll
    for (int s = 0; s < R; ++s) acc[r][s] = 0.f;
  }

  for (long long n0 = n_begin; n0 < n_end; n0 += kStateTile) {
    __syncthreads();
    for (int idx = tid; idx < kStateTile * 16 * R; idx += kThreads) {
      const int n = idx / (16 * R), e = idx % (16 * R);
      float kv = 0.f, vv = 0.f, kplain = 0.f;
      if (n0 + n < n_end && e < d) {
        const long long off = base + (n0 + n) * p.sn + e;
        kv = kplain = fmaxf(load_f32<T>(k + off), 0.f);  // phi = ReLU on the keys
        vv = load_f32<T>(v + off);
        if (ROPE && (e ^ 1) < d) {  // rotate after the ReLU; an unpaired last feature stays
          const float other = fmaxf(load_f32<T>(k + off + ((e ^ 1) - e)), 0.f);
          const float2 cssn = __half22float2(tab[(n0 + n) * (long long)(d / 2) + e / 2]);
          const float c = cssn.x, sgn = cssn.y;
          kv = (e & 1) ? other * sgn + kplain * c : kplain * c - other * sgn;
        }
      }
      Ks[n * kPitch + e] = kv;
      Vs[n * kPitch + e] = vv;
      if (ROPE) Zs[n * kPitch + e] = kplain;
    }
    __syncthreads();
#pragma unroll 4
    for (int n = 0; n < kStateTile; ++n) {
      float a[R], bb[R];
#pragma unroll
      for (int r = 0; r < R; ++r) {
        a[r] = Ks[n * kPitch + ti + 16 * r];
        bb[r] = Vs[n * kPitch + tj + 16 * r];
      }
#pragma unroll
      for (int r = 0; r < R; ++r) {
        zacc[r] += ROPE ? Zs[n * kPitch + ti + 16 * r] : a[r];
#pragma unroll
        for (int s = 0; s < R; ++s) acc[r][s] = fmaf(a[r], bb[s], acc[r][s]);
      }
    }
  }

  // partial state in the library's layout: W[j][i] = S[i][j], W[d][i] = z[i]
  float* out = partials + ((long long)u * P + c) * p.state_elems();
#pragma unroll
  for (int r = 0; r < R; ++r) {
    const int i = ti + 16 * r;
    if (i >= d) continue;
#pragma unroll
    for (int s = 0; s < R; ++s) {
      const int j = tj + 16 * s;
      if (j < d) out[(long long)j * d + i] = acc[r][s];
    }
    if (tj == 0) out[(long long)d * d + i] = zacc[r];
  }
}

// grid (ceil(E/256), units): state[u][e] = (accumulate ? state[u][e] : 0) + sum_c partial[u][c][e], c ascending.
__global__ void __launch_bounds__(kThreads)
fma_state_reduce(const float* __restrict__ partials, int P, long long E, float* __restrict__ state, int accumulate) {
  const long long e = (long long)blockIdx.x * kThreads + threadIdx.x;
  const int u = blockIdx.y;
  if (e >= E) return;
  double sum = accumulate ? (double)state[(long long)u * E + e] : 0.0;
  for (int c = 0; c < P; ++c) sum += (double)partials[((long long)u * P + c) * E + e];
  state[(long long)u * E + e] = (float)sum;
}

// grid (ceil(N/64), units).  Thread (tn, tj) owns tokens tn + 16*r (r < 4) and outputs j = tj + 16*c.
// ROPE: the numerator uses the rotated phi(q), the denominator the plain phi(q).
template <typename T, int R, bool ROPE>
__global__ void __launch_bounds__(kThreads)
fma_apply_kernel(const T* __restrict__ q, const float* __restrict__ state, T* __restrict__ o, Problem p, float eps,
                 const __half2* __restrict__ tab) {
  extern __shared__ float smem[];
  const int d = p.d;
  float* Ss = smem;                     // [d][kPitch]  Ss[i][j] = S[i][j]
  float* zs = Ss + d * kPitch;          // [d]
  float* Qs = zs + 128;                 // [kApplyTile][kPitch], phi(q) (rotated with ROPE)
  float* Qp = Qs + kApplyTile * kPitch; // [kApplyTile][kPitch], plain phi(q) (ROPE only)
  const int u = blockIdx.y;
  const int b = u / p.H, h = u % p.H;
  const long long n0 = (long long)blockIdx.x * kApplyTile;
  const int tid = threadIdx.x, tn = tid >> 4, tj = tid & 15;
  const float* W = state + (long long)u * p.state_elems();

  for (int idx = tid; idx < d * d; idx += kThreads) {
    const int j = idx / d, i = idx % d;
    Ss[i * kPitch + j] = W[idx];
  }
  for (int i = tid; i < d; i += kThreads) zs[i] = W[(long long)d * d + i];
  for (int idx = tid; idx < d * (16 * R - d); idx += kThreads) {  // zero the padded columns
    const int i = idx / (16 * R - d), j = d + idx % (16 * R - d);
    Ss[i * kPitch + j] = 0.f;
  }
  const long long base = (long long)b * p.sb + (long long)h * p.sh;
  for (int idx = tid; idx < kApplyTile * d; idx += kThreads) {
    const int n = idx / d, e = idx % d;
    float x = 0.f, plain = 0.f;
    if (n0 + n < p.N) {
      const long long off = base + (n0 + n) * p.sn + e;
      x = plain = fmaxf(load_f32<T>(q + off), 0.f);  // phi = ReLU on the queries
      if (ROPE && (e ^ 1) < d) {
        const float other = fmaxf(load_f32<T>(q + off + ((e ^ 1) - e)), 0.f);
        const float2 cssn = __half22float2(tab[(n0 + n) * (long long)(d / 2) + e / 2]);
        const float c = cssn.x, sgn = cssn.y;
        x = (e & 1) ? other * sgn + plain * c : plain * c - other * sgn;
      }
    }
    Qs[n * kPitch + e] = x;
    if (ROPE) Qp[n * kPitch + e] = plain;
  }
  __syncthreads();

  float acc[4][R];
  float den[4];
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    den[r] = 0.f;
#pragma unroll
    for (int s = 0; s < R; ++s) acc[r][s] = 0.f;
  }
  for (int i = 0; i < d; ++i) {
    float a[4], bb[R];
    const float zz = zs[i];
#pragma unroll
    for (int r = 0; r < 4; ++r) a[r] = Qs[(tn + 16 * r) * kPitch + i];
#pragma unroll
    for (int s = 0; s < R; ++s) bb[s] = Ss[i * kPitch + tj + 16 * s];
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      den[r] = fmaf(ROPE ? Qp[(tn + 16 * r) * kPitch + i] : a[r], zz, den[r]);
#pragma unroll
      for (int s = 0; s < R; ++s) acc[r][s] = fmaf(a[r], bb[s], acc[r][s]);
    }
  }
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const long long n = n0 + tn + 16 * r;
    if (n >= p.N) continue;
    const float dn = den[r] + eps;  // eps added once, after the dot product
#pragma unroll
    for (int s = 0; s < R; ++s) {
      const int j = tj + 16 * s;
      if (j < d) store_out<T>(o + base + n * p.sn + j, acc[r][s] / dn);
    }
  }
}

template <typename T, int R>
cudaError_t launch_state_partial(const Problem& p, const void* k, const void* v, int P, float* partials,
                                 const __half2* tab, cudaStream_t stream) {
  dim3 grid(P, p.units());
  if (tab)
    fma_state_partial<T, R, true><<<grid, kThreads, 0, stream>>>((const T*)k, (const T*)v, p, P, partials, tab);
  else
    fma_state_partial<T, R, false><<<grid, kThreads, 0, stream>>>((const T*)k, (const T*)v, p, P, partials, tab);
  count_launches(1);
  return cudaGetLastError();
}

template <typename T, int R>
cudaError_t launch_apply(const Problem& p, const void* q, const float* state, void* o, float eps, const __half2* tab,
                         cudaStream_t stream) {
  const size_t smem = sizeof(float) * ((size_t)p.d * kPitch + 128 + (size_t)(tab ? 2 : 1) * kApplyTile * kPitch);
  cudaError_t e = tab ? cudaFuncSetAttribute(fma_apply_kernel<T, R, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)
                     : cudaFuncSetAttribute(fma_apply_kernel<T, R, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  dim3 grid((unsigned)((p.N + kApplyTile - 1) / kApplyTile), p.units());
  if (tab)
    fma_apply_kernel<T, R, true><<<grid, kThreads, smem, stream>>>((const T*)q, state, (T*)o, p, eps, tab);
  else
    fma_apply_kernel<T, R, false><<<grid, kThreads, smem, stream>>>((const T*)q, state, (T*)o, p, eps, tab);
  count_launches(1);
  return cudaGetLastError();
}

#define LINATTN_DISPATCH_R(FN, T, ...)                                   \
  switch ((p.d + 15) / 16) {                                             \
    case 1: return FN<T, 1>(__VA_ARGS__);                                \
    case 2: return FN<T, 2>(__VA_ARGS__);                                \
    case 3: return FN<T, 3>(__VA_ARGS__);                                \
    case 4: return FN<T, 4>(__VA_ARGS__);                                \
    case 5: return FN<T, 5>(__VA_ARGS__);                                \
    case 6: return FN<T, 6>(__VA_ARGS__);                                \
    case 7: return FN<T, 7>(__VA_ARGS__);                                \
    default: return FN<T, 8>(__VA_ARGS__);                               \
  }

cudaError_t state_partial_any(const Problem& p, const void* k, const void* v, int P, float* partials,
                              const __half2* tab, cudaStream_t stream) {
  if (p.dtype == LINATTN_F32) {
    LINATTN_DISPATCH_R(launch_state_partial, float, p, k, v, P, partials, tab, stream)
  } else {
    LINATTN_DISPATCH_R(launch_state_partial, __nv_bfloat16, p, k, v, P, partials, tab, stream)
  }
}

cudaError_t apply_any(const Problem& p, const void* q, const float* state, void* o, float eps, const __half2* tab,
                      cudaStream_t stream) {
  if (p.dtype == LINATTN_F32) {
    LINATTN_DISPATCH_R(launch_apply, float, p, q, state, o, eps, tab, stream)
  } else {
    LINATTN_DISPATCH_R(launch_apply, __nv_bfloat16, p, q, state, o, eps, tab, stream)
  }
}

// (cos, sin) of every pair rotation as one fp16 pair, round to nearest.
__global__ void rope_pack_kernel(const float* __restrict__ cs, const float* __restrict__ sn, long long count,
                                 __half2* __restrict__ out) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < count) out[i] = __floats2half2_rn(cs[i], sn[i]);
}

// Inclusive prefix over the blocks of a prefill: blk[b][m] := cache[b] + blk[b][0] + ... + blk[b][m] (added in
// that order), cache[b] := blk[b][M-1].  One thread per float4 of a (batch, head) state.
__global__ void prefix_states_kernel(float4* __restrict__ blk, float4* __restrict__ cache, int M, long long per_batch4) {
  const long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= per_batch4) return;
  const int b = blockIdx.y;
  float4 run = cache[b * per_batch4 + e];
  for (int m = 0; m < M; ++m) {
    float4* x = blk + ((long long)b * M + m) * per_batch4 + e;
    const float4 a = *x;
    run.x += a.x; run.y += a.y; run.z += a.z; run.w += a.w;
    *x = run;
  }
  cache[b * per_batch4 + e] = run;
}

}  // namespace

cudaError_t prefix_states(float* blk, float* cache, int B, int M, long long floats_per_batch, cudaStream_t stream) {
  const long long n4 = floats_per_batch / 4;
  dim3 grid((unsigned)((n4 + 255) / 256), (unsigned)B);
  prefix_states_kernel<<<grid, 256, 0, stream>>>(reinterpret_cast<float4*>(blk), reinterpret_cast<float4*>(cache), M, n4);
  count_launches(1);
  return cudaGetLastError();
}

cudaError_t rope_pack(const float* cs, const float* sn, long long count, __half2* out, cudaStream_t stream) {
  if (count == 0) return cudaSuccess;
  rope_pack_kernel<<<(unsigned)((count + 255) / 256), 256, 0, stream>>>(cs, sn, count, out);
  count_launches(1);
  return cudaGetLastError();
}

cudaError_t fma_state(const Problem& p, const void* k, const void* v, float* state_out, bool accumulate,
                      float* partials, cudaStream_t stream, const __half2* rope) {
  const long long E = p.state_elems();
  if (p.N == 0) {
    if (accumulate) return cudaSuccess;
    return cudaMemsetAsync(state_out, 0, sizeof(float) * E * p.units(), stream);
  }
  const int P = fma_chunks(p.N);
  cudaError_t e = state_partial_any(p, k, v, P, partials, rope, stream);
  if (e != cudaSuccess) return e;
  dim3 grid((unsigned)((E + kThreads - 1) / kThreads), p.units());
  fma_state_reduce<<<grid, kThreads, 0, stream>>>(partials, P, E, state_out, accumulate ? 1 : 0);
  count_launches(1);
  return cudaGetLastError();
}

cudaError_t fma_apply(const Problem& p, const void* q, const float* state, void* o, float eps, cudaStream_t stream,
                      const __half2* rope) {
  if (p.N == 0) return cudaSuccess;
  return apply_any(p, q, state, o, eps, rope, stream);
}

}  // namespace linattn
