// Tensor-core kernels for bf16 ReLU linear attention on sm_100a: TMA tiles into shared memory,
// a ReLU pass in place, tcgen05.mma with fp32 accumulators in tensor memory, results streamed out.
//
// Both contractions of the method are dense and run on the tensor cores, but the kernels are
// HBM-bound (about d/2 FLOP per byte); everything here is organised around keeping TMA loads in
// flight on every SM.
//
//   umma_state_kernel   S = sum_n phi(k_n)^T v_n and z = sum_n phi(k_n)   (Eq. 2 / Eq. 3 state).
//                       A = phi(K)^T and B = [V | 1] are both token-major in memory, i.e. MN-major
//                       UMMA operands; the contraction index is the token.  The extra "ones" column
//                       makes z fall out of the same MMA as column 128 of the accumulator.
//                       Work is split over tokens across the grid (split-N); every CTA writes one
//                       fp32 partial per (head group) segment it covered.
//   umma_reduce_kernel  sums the partials of each head in a fixed order (deterministic), optionally
//                       on top of the existing state: the cache update of Eq. 3.
//   umma_apply_kernel   o_n = phi(q_n) S / (phi(q_n).z + eps).  A = phi(Q) tile (K-major), B = S
//                       split into bf16 hi + lo parts (two MMAs per K step, so S keeps ~16 mantissa
//                       bits), with z as an extra row of B so the denominator is one more
//                       accumulator column.  The epilogue divides, rounds to bf16 and TMA-stores.
//
// Head dims 32 and 64 pack 4 / 2 heads into one 128-feature operand (the cross-head blocks of the
// product are ignored / zero); 112 pads to 128 through TMA out-of-bounds zero fill.
//
// Warp roles (320 threads): warp 0 TMA producer, warp 1 MMA issuer and TMEM owner, warps 2-5 ReLU
// pass, warps 6-9 epilogue.  All cross-role synchronisation is by mbarriers with bounded waits; a
// wait that runs out raises a CTA-wide abort flag, records LINATTN_ERR_TIMEOUT in the workspace
// status word, and every role falls through to the common teardown (TMEM is freed, loads in flight
// are waited for with a bound).
#include <cuda.h>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace linattn {
namespace {

using namespace ptx;

constexpr int kThreads = 320;
constexpr int kReluThread0 = 64;    // warps 2-5
constexpr int kEpiThread0 = 192;    // warps 6-9
constexpr int kTileApply = 128;     // tokens per apply tile (= UMMA M)
constexpr int kTileState = 64;      // tokens per state stage (4 UMMA K steps of 16 tokens)
constexpr int kRowBytes = 128;      // one swizzle row: 64 bf16
constexpr int kTmemCols = 512;
constexpr int kAccStride = 256;     // TMEM columns between the two accumulator buffers

template <int D>
struct Cfg {
  static constexpr int G = D == 32 ? 4 : D == 64 ? 2 : 1;   // heads packed into one 128-feature operand
  static constexpr int FEAT = G * D;                         // 112 or 128 live features per group
  static constexpr int KSTEPS = FEAT / 16;                   // apply: K steps over features
  static constexpr int ZROW = D == 112 ? 112 : 128;          // apply: accumulator column of the first denominator
  static constexpr int NAPPLY = D == 112 ? 128 : 144;        // apply MMA N
  static constexpr int NSTATE = 144;                         // state MMA N: 128 value columns + the ones chunk
  static constexpr int BOX_D = D < 64 ? D : 64;              // TMA box: features ...
  static constexpr int BOX_H = 64 / BOX_D;                   // ... x heads = 64 elements = one 128-byte row
  static constexpr int SBOX_BYTES = NAPPLY * kRowBytes;      // one 64-feature K box of the S operand
  static constexpr int S_BYTES = 4 * SBOX_BYTES;             // (hi, lo) x 2 K boxes
  static constexpr int APPLY_SLOTS = D == 112 ? 5 : 4;
  static constexpr int APPLY_SLOT_BYTES = 2 * kTileApply * kRowBytes;  // 32 KB: two 64-feature boxes
  static constexpr int STATE_STAGES = 5;
  static constexpr int BOX_BYTES_STATE = kTileState * kRowBytes;       // 8 KB
  static constexpr int STATE_STAGE_BYTES = 5 * BOX_BYTES_STATE;        // V0 V1 ONES K0 K1
  static constexpr size_t APPLY_SMEM = 1024 + S_BYTES + APPLY_SLOTS * APPLY_SLOT_BYTES + 512;
  static constexpr size_t STATE_SMEM = 1024 + STATE_STAGES * STATE_STAGE_BYTES + 512;
};

struct UmmaParams {
  int B, H, HG;            // HG: head groups per batch entry = ceil(H / G)
  long long N;
  int tiles_per_unit;      // token tiles per (batch, head group) unit
  long long total_tiles;   // units * tiles_per_unit
  const float* state_in;   // apply: [B][H][(d+1)][d]
  float* partials;         // state: one record of G head-states per (CTA, unit) segment
  float eps;
  int* status;             // workspace status word
};

// TMA coordinates (feature, head) of 64-element box `box` (0/1) of head group hg
template <int D>
__device__ __forceinline__ void box_coords(int box, int hg, int& c0, int& c1) {
  using C = Cfg<D>;
  if (C::G == 1) { c0 = 64 * box; c1 = hg; }
  else if (C::G == 2) { c0 = 0; c1 = 2 * hg + box; }
  else { c0 = 0; c1 = 4 * hg + 2 * box; }
}

__device__ __forceinline__ uint8_t* align1024(uint8_t* p) {
  return reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(p) + 1023) & ~(uintptr_t)1023);
}

// In-place ReLU over `nchunks` 16-byte chunks starting at `base`, 128 threads, thread `t`.
// With FEAT = 112 the chunks that hold only the zero padding (features 112..127) are skipped.
template <int FEAT>
__device__ __forceinline__ void relu_pass(uint8_t* base, int nchunks, int chunks_per_box, int t) {
  for (int idx = t; idx < nchunks; idx += 128) {
    if (FEAT < 128) {
      const int in_box = idx % chunks_per_box;
      const int box = (idx / chunks_per_box) & 1;
      const int row = in_box >> 3, phys = in_box & 7;
      if (box == 1 && (((phys ^ (row & 7)) << 3) + 64) >= FEAT) continue;
    }
    uint4* p = reinterpret_cast<uint4*>(base + (size_t)idx * 16);
    uint4 x = *p;
    x.x = relu_bf16x2(x.x); x.y = relu_bf16x2(x.y); x.z = relu_bf16x2(x.z); x.w = relu_bf16x2(x.w);
    *p = x;
  }
}

// ============================================================================ state kernel
// grid: persistent, CTA j covers flat stage indices [j*W/G, (j+1)*W/G) over (unit, 64-token stage).
template <int D>
__global__ void __launch_bounds__(kThreads, 1)
umma_state_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v, UmmaParams p) {
  using C = Cfg<D>;
  constexpr int NS = C::STATE_STAGES;
  constexpr int BOX = C::BOX_BYTES_STATE;
  constexpr int STAGE = C::STATE_STAGE_BYTES;
  constexpr uint32_t IDESC = make_idesc_bf16(128, C::NSTATE, true, true);
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = align1024(smem_raw);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + NS * STAGE);
  uint64_t* full = bars;             // TMA landed
  uint64_t* ready = bars + NS;       // ReLU pass done
  uint64_t* empty = bars + 2 * NS;   // MMAs that read the stage are complete
  uint64_t* tfull = bars + 3 * NS;   // [2] accumulator complete
  uint64_t* tempty = tfull + 2;      // [2] accumulator drained by the epilogue
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(tempty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long t_begin = (long long)blockIdx.x * p.total_tiles / gridDim.x;
  const long long t_end = (long long)(blockIdx.x + 1) * p.total_tiles / gridDim.x;
  const int tpu = p.tiles_per_unit;

  if (threadIdx.x == 0) {
    for (int s = 0; s < NS; ++s) { mbar_init(&full[s], 1); mbar_init(&ready[s], 128); mbar_init(&empty[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&tfull[b], 1); mbar_init(&tempty[b], 128); }
    *abort_flag = 0;
    fence_mbar_init();
    prefetch_tensormap(&map_k);
    prefetch_tensormap(&map_v);
  }
  // the constant "ones" chunk of every stage: value columns 128..191 of B, of which column 128 is 1
  for (int idx = threadIdx.x; idx < NS * (BOX / 16); idx += kThreads) {
    const int s = idx / (BOX / 16), c = idx % (BOX / 16);
    const int row = c >> 3, phys = c & 7;
    uint4 val = make_uint4(0, 0, 0, 0);
    if ((phys ^ (row & 7)) == 0) val.x = 0x3F80u;  // bf16 1.0 in element 0 of logical chunk 0
    *reinterpret_cast<uint4*>(smem + s * STAGE + 2 * BOX + c * 16) = val;
  }
  fence_proxy_async_smem();
  if (warp == 1) { tmem_alloc(tmem_holder, kTmemCols); tmem_relinquish(); }
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  const uint32_t tmem_base = *tmem_holder;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t it = 0;
      for (long long t = t_begin; t < t_end; ++t, ++it) {
        const int s = it % NS;
        if (!mbar_wait(&empty[s], ((it / NS) & 1) ^ 1, abort_flag)) break;
        const int u = (int)(t / tpu), tt = (int)(t % tpu);
        const int b = u / p.HG, hg = u % p.HG;
        uint8_t* st = smem + s * STAGE;
        mbar_arrive_expect_tx(&full[s], 4 * BOX);
        int c0, c1;
        box_coords<D>(0, hg, c0, c1);
        tma_load_4d(st + 3 * BOX, &map_k, &full[s], c0, c1, tt * kTileState, b);
        tma_load_4d(st + 0 * BOX, &map_v, &full[s], c0, c1, tt * kTileState, b);
        box_coords<D>(1, hg, c0, c1);
        tma_load_4d(st + 4 * BOX, &map_k, &full[s], c0, c1, tt * kTileState, b);
        tma_load_4d(st + 1 * BOX, &map_v, &full[s], c0, c1, tt * kTileState, b);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      uint32_t it = 0, seg = 0;
      bool ok = true;
      for (long long t = t_begin; t < t_end && ok; ++t, ++it) {
        const int s = it % NS;
        const int tt = (int)(t % tpu);
        const bool seg_first = (t == t_begin) || tt == 0;
        const bool seg_last = (t + 1 == t_end) || tt == tpu - 1;
        const uint32_t acc = seg & 1;
        if (seg_first) ok = mbar_wait(&tempty[acc], ((seg >> 1) & 1) ^ 1, abort_flag);
        if (ok) ok = mbar_wait(&ready[s], (it / NS) & 1, abort_flag);
        if (!ok) break;
        tcgen05_fence_after();
        const uint32_t d_tmem = tmem_base + acc * kAccStride;
        const uint32_t st = smem_u32(smem + s * STAGE);
#pragma unroll
        for (int kk = 0; kk < kTileState / 16; ++kk) {
          const uint64_t a = make_smem_desc_sw128(st + 3 * BOX + kk * 2048, BOX, 1024);  // phi(K)^T, MN-major
          const uint64_t bq = make_smem_desc_sw128(st + kk * 2048, BOX, 1024);           // [V | 1], MN-major
          umma_bf16(d_tmem, a, bq, IDESC, (seg_first && kk == 0) ? 0u : 1u);
        }
        umma_commit(&empty[s]);
        if (seg_last) { umma_commit(&tfull[acc]); ++seg; }
      }
    }
  } else if (warp < 6) {
    // ------------------------------------------------------------ ReLU pass over the K boxes
    const int tr = threadIdx.x - kReluThread0;
    uint32_t it = 0;
    for (long long t = t_begin; t < t_end; ++t, ++it) {
      const int s = it % NS;
      if (!mbar_wait(&full[s], (it / NS) & 1, abort_flag)) break;
      relu_pass<C::FEAT>(smem + s * STAGE + 3 * BOX, 2 * BOX / 16, BOX / 16, tr);
      fence_proxy_async_smem();
      mbar_arrive(&ready[s]);
    }
  } else {
    // ------------------------------------------------------------ epilogue: accumulator -> partial record
    const int wq = warp & 3;
    const int i = wq * 32 + lane;           // accumulator lane = key feature within the group
    const int g = i / D, il = i % D;        // head within the group, feature within the head
    uint32_t seg = 0;
    for (long long t = t_begin; t < t_end; ++t) {
      const int tt = (int)(t % tpu);
      const bool seg_last = (t + 1 == t_end) || tt == tpu - 1;
      if (!seg_last) continue;
      const uint32_t acc = seg & 1;
      bool ok = mbar_wait(&tfull[acc], (seg >> 1) & 1, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tcgen05_fence_after();
      const int u = (int)(t / tpu);
      const int b = u / p.HG, hg = u % p.HG;
      const int h = hg * C::G + g;
      const bool live = i < C::FEAT && h < p.H;
      (void)b;
      // record of this (CTA, unit) segment: G consecutive head-states in the library's layout
      float* out = p.partials + ((size_t)(blockIdx.x + u) * C::G + g) * ((size_t)(D + 1) * D);
      const uint32_t trow = tmem_base + acc * kAccStride + ((uint32_t)(wq * 32) << 16);
#pragma unroll 1
      for (int cc = 0; cc < 4; ++cc) {
        uint32_t r[32];
        tmem_ld_x32(trow + cc * 32, r);
        tmem_ld_wait();
        if (live) {
#pragma unroll
          for (int x = 0; x < 32; ++x) {
            const int j = cc * 32 + x;             // value feature within the group
            const int jl = j - g * D;
            if (jl >= 0 && jl < D) out[(size_t)jl * D + il] = __uint_as_float(r[x]);
          }
        }
      }
      uint32_t zr[4];
      tmem_ld_x4(trow + 128, zr);
      tmem_ld_wait();
      if (live) out[(size_t)D * D + il] = __uint_as_float(zr[0]);
      tcgen05_fence_before();
      mbar_arrive(&tempty[acc]);
      ++seg;
    }
  }

  // ------------------------------------------------------------ teardown
  tcgen05_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (threadIdx.x == 0) {
      *p.status = LINATTN_ERR_TIMEOUT;
      // loads still in flight target this CTA's shared memory: give each stage a bounded wait
      for (int s = 0; s < NS; ++s)
        for (int par = 0; par < 2; ++par)
          for (int spin = 0; spin < 4096 && !mbar_try_wait(&full[s], par); ++spin) __nanosleep(64);
    }
    __syncthreads();
  }
  if (warp == 1) {
    __syncwarp();
    tcgen05_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ============================================================================ reduce kernel
// grid (ceil(E/256), B*H).  state[b][h][e] = (accumulate ? state : 0) + sum over the CTAs that
// covered this head's group, in ascending CTA order.
__device__ __forceinline__ long long cta_start(long long j, long long total, int grid) { return j * total / grid; }
__device__ __forceinline__ int cta_of_tile(long long t, long long total, int grid) {
  long long j = t * grid / total;
  while (j + 1 < grid && cta_start(j + 1, total, grid) <= t) ++j;
  while (j > 0 && cta_start(j, total, grid) > t) --j;
  return (int)j;
}

__global__ void __launch_bounds__(256)
umma_reduce_kernel(const float* __restrict__ partials, float* __restrict__ state, int H, int HG, int G, int d,
                   int tiles_per_unit, long long total_tiles, int grid_state, int accumulate) {
  const long long E = (long long)(d + 1) * d;
  const long long e = (long long)blockIdx.x * 256 + threadIdx.x;
  if (e >= E) return;
  const int bh = blockIdx.y;
  const int b = bh / H, h = bh % H;
  const int u = b * HG + h / G, g = h % G;
  const int j_lo = cta_of_tile((long long)u * tiles_per_unit, total_tiles, grid_state);
  const int j_hi = cta_of_tile((long long)(u + 1) * tiles_per_unit - 1, total_tiles, grid_state);
  float sum = accumulate ? state[(long long)bh * E + e] : 0.f;
  for (int j = j_lo; j <= j_hi; ++j) sum += partials[((size_t)(j + u) * G + g) * E + e];
  state[(long long)bh * E + e] = sum;
}

// ============================================================================ apply kernel
// Builds the B operand of the apply MMA for head group (b, hg) from the fp32 state: for every head
// of the group, rows = value features (plus one row for z), K = key features, split into bf16 hi + lo.
template <int D>
__device__ __forceinline__ void build_s_operand(uint8_t* s_op, const float* __restrict__ state, int b, int hg, int H,
                                                int part, int nparts) {
  using C = Cfg<D>;
  constexpr int CPR = D / 8;       // 16-byte chunks per state row
  constexpr int ROWS = D + 1;
  for (int idx = part; idx < C::G * ROWS * CPR; idx += nparts) {
    const int g = idx / (ROWS * CPR);
    const int rem = idx - g * ROWS * CPR;
    const int j = rem / CPR, c = rem % CPR;
    const int h = hg * C::G + g;
    float x[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    if (h < H) {
      const float4* src = reinterpret_cast<const float4*>(state + ((size_t)(b * H + h) * ROWS + j) * D + c * 8);
      const float4 a = __ldcg(src), bq = __ldcg(src + 1);
      x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = bq.x; x[5] = bq.y; x[6] = bq.z; x[7] = bq.w;
    }
    uint32_t hi[4], lo[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const __nv_bfloat16 h0 = __float2bfloat16_rn(x[2 * e]), h1 = __float2bfloat16_rn(x[2 * e + 1]);
      hi[e] = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
      lo[e] = pack_bf16x2(x[2 * e] - __bfloat162float(h0), x[2 * e + 1] - __bfloat162float(h1));
    }
    const int jrow = j < D ? g * D + j : C::ZROW + g;  // operand row: value feature, or the head's z row
    const int i0 = g * D + c * 8;                      // first key feature of this chunk
    const int off = (i0 >> 6) * C::SBOX_BYTES + jrow * kRowBytes + ((((i0 & 63) >> 3) ^ (jrow & 7)) << 4);
    *reinterpret_cast<uint4*>(s_op + off) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
    *reinterpret_cast<uint4*>(s_op + 2 * C::SBOX_BYTES + off) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
  }
}

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
umma_apply_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_o, UmmaParams p) {
  using C = Cfg<D>;
  constexpr int NS = C::APPLY_SLOTS;
  constexpr int SLOT = C::APPLY_SLOT_BYTES;
  constexpr int HALF = SLOT / 2;  // one 64-feature box of 128 tokens
  constexpr uint32_t IDESC = make_idesc_bf16(128, C::NAPPLY, false, false);
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = align1024(smem_raw);
  uint8_t* s_op = smem;
  uint8_t* slots = smem + C::S_BYTES;
  uint64_t* bars = reinterpret_cast<uint64_t*>(slots + NS * SLOT);
  uint64_t* full = bars;             // Q tile landed
  uint64_t* ready = bars + NS;       // ReLU pass done
  uint64_t* empty = bars + 2 * NS;   // O tile stored: slot reusable
  uint64_t* tfull = bars + 3 * NS;   // [2] accumulator complete
  uint64_t* tempty = tfull + 2;      // [2] accumulator drained
  uint64_t* s_ready = tempty + 2;    // S operand of the current segment is in shared memory
  uint64_t* seg_done = s_ready + 1;  // every MMA of the finished segment is complete
  uint64_t* o_staged = seg_done + 1; // the 128 epilogue threads have written their O rows
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(o_staged + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long t_begin = (long long)blockIdx.x * p.total_tiles / gridDim.x;
  const long long t_end = (long long)(blockIdx.x + 1) * p.total_tiles / gridDim.x;
  const int tpu = p.tiles_per_unit;

  if (threadIdx.x == 0) {
    for (int s = 0; s < NS; ++s) { mbar_init(&full[s], 1); mbar_init(&ready[s], 128); mbar_init(&empty[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&tfull[b], 1); mbar_init(&tempty[b], 128); }
    mbar_init(s_ready, 256);
    mbar_init(seg_done, 128);
    mbar_init(o_staged, 128);
    *abort_flag = 0;
    fence_mbar_init();
    prefetch_tensormap(&map_q);
    prefetch_tensormap(&map_o);
  }
  // rows of the S operand that no head ever writes (padding rows, cross-head blocks) stay zero
  for (int idx = threadIdx.x; idx < C::S_BYTES / 16; idx += kThreads)
    *reinterpret_cast<uint4*>(s_op + idx * 16) = make_uint4(0, 0, 0, 0);
  fence_proxy_async_smem();
  if (warp == 1) { tmem_alloc(tmem_holder, kTmemCols); tmem_relinquish(); }
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  const uint32_t tmem_base = *tmem_holder;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer: Q tiles
    if (lane == 0) {
      uint32_t it = 0;
      for (long long t = t_begin; t < t_end; ++t, ++it) {
        const int s = it % NS;
        if (!mbar_wait(&empty[s], ((it / NS) & 1) ^ 1, abort_flag)) break;
        const int u = (int)(t / tpu), tt = (int)(t % tpu);
        const int b = u / p.HG, hg = u % p.HG;
        uint8_t* sl = slots + s * SLOT;
        mbar_arrive_expect_tx(&full[s], SLOT);
        int c0, c1;
        box_coords<D>(0, hg, c0, c1);
        tma_load_4d(sl, &map_q, &full[s], c0, c1, tt * kTileApply, b);
        box_coords<D>(1, hg, c0, c1);
        tma_load_4d(sl + HALF, &map_q, &full[s], c0, c1, tt * kTileApply, b);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      uint32_t it = 0, seg = 0;
      bool ok = true;
      for (long long t = t_begin; t < t_end && ok; ++t, ++it) {
        const int s = it % NS;
        const int tt = (int)(t % tpu);
        if (t == t_begin || tt == 0) { ok = mbar_wait(s_ready, seg & 1, abort_flag); ++seg; }
        const uint32_t acc = it & 1;
        if (ok) ok = mbar_wait(&tempty[acc], ((it >> 1) & 1) ^ 1, abort_flag);
        if (ok) ok = mbar_wait(&ready[s], (it / NS) & 1, abort_flag);
        if (!ok) break;
        tcgen05_fence_after();
        const uint32_t d_tmem = tmem_base + acc * kAccStride;
        const uint32_t a0 = smem_u32(slots + s * SLOT);
        const uint32_t b0 = smem_u32(s_op);
#pragma unroll
        for (int k = 0; k < C::KSTEPS; ++k) {
          const uint32_t koff = (k >> 2) * HALF + (k & 3) * 32;
          const uint32_t boff = (k >> 2) * C::SBOX_BYTES + (k & 3) * 32;
          const uint64_t a = make_smem_desc_sw128(a0 + koff, 16, 1024);                           // phi(Q), K-major
          const uint64_t bh = make_smem_desc_sw128(b0 + boff, 16, 1024);                          // S hi
          const uint64_t bl = make_smem_desc_sw128(b0 + 2 * C::SBOX_BYTES + boff, 16, 1024);      // S lo
          umma_bf16(d_tmem, a, bh, IDESC, k == 0 ? 0u : 1u);
          umma_bf16(d_tmem, a, bl, IDESC, 1u);
        }
        umma_commit(&tfull[acc]);
      }
    }
  } else if (warp < 6) {
    // ------------------------------------------------------------ ReLU pass over Q tiles (+ half of the S build)
    const int tr = threadIdx.x - kReluThread0;
    uint32_t it = 0, seg = 0;
    bool ok = true;
    for (long long t = t_begin; t < t_end && ok; ++t, ++it) {
      const int s = it % NS;
      const int tt = (int)(t % tpu);
      if (t == t_begin || tt == 0) {
        // the previous segment's MMAs must be done before its S operand is overwritten
        if (seg > 0) ok = mbar_wait(seg_done, (seg - 1) & 1, abort_flag);
        if (!ok) break;
        const int u = (int)(t / tpu);
        build_s_operand<D>(s_op, p.state_in, u / p.HG, u % p.HG, p.H, tr, 256);
        fence_proxy_async_smem();
        mbar_arrive(s_ready);
        ++seg;
      }
      if (!mbar_wait(&full[s], (it / NS) & 1, abort_flag)) break;
      relu_pass<C::FEAT>(slots + s * SLOT, SLOT / 16, HALF / 16, tr);
      fence_proxy_async_smem();
      mbar_arrive(&ready[s]);
    }
  } else {
    // ------------------------------------------------------------ epilogue: divide, round, store
    const int te = threadIdx.x - kEpiThread0;
    const int wq = warp & 3;
    const int r = wq * 32 + lane;  // accumulator lane = token row of the tile
    uint32_t it = 0;
    for (long long t = t_begin; t < t_end; ++t, ++it) {
      const int s = it % NS;
      const int u = (int)(t / tpu), tt = (int)(t % tpu);
      const int b = u / p.HG, hg = u % p.HG;
      if (t == t_begin || tt == 0) {
        // this thread has seen the last accumulator of the previous segment complete: S may be rebuilt
        build_s_operand<D>(s_op, p.state_in, b, hg, p.H, 128 + te, 256);
        fence_proxy_async_smem();
        mbar_arrive(s_ready);
      }
      const uint32_t acc = it & 1;
      bool ok = mbar_wait(&tfull[acc], (it >> 1) & 1, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tcgen05_fence_after();
      if ((t + 1 == t_end) || tt == tpu - 1) mbar_arrive(seg_done);
      const uint32_t trow = tmem_base + acc * kAccStride + ((uint32_t)(wq * 32) << 16);
      uint32_t dn[4];
      tmem_ld_x4(trow + C::ZROW, dn);
      tmem_ld_wait();
      float rinv[C::G];
#pragma unroll
      for (int g = 0; g < C::G; ++g) rinv[g] = 1.0f / (__uint_as_float(dn[g]) + p.eps);  // eps added once, after the dot product
      uint8_t* sl = slots + s * SLOT;
#pragma unroll
      for (int cc = 0; cc < 4; ++cc) {
        if (cc * 32 >= C::FEAT) break;
        uint32_t v[32];
        tmem_ld_x32(trow + cc * 32, v);
        tmem_ld_wait();
        if (cc == 3 || (cc + 1) * 32 >= C::FEAT) {  // last read of this accumulator: hand it back to the MMA warp
          tcgen05_fence_before();
          mbar_arrive(&tempty[acc]);
        }
        const float ri = rinv[(cc * 32) / D < C::G ? (cc * 32) / D : 0];
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) {
          const int lc = cc * 4 + q4;  // logical 16-byte chunk of the 256-byte padded row
          if (lc * 8 >= C::FEAT) break;
          uint4 pk;
          pk.x = pack_bf16x2(__uint_as_float(v[q4 * 8 + 0]) * ri, __uint_as_float(v[q4 * 8 + 1]) * ri);
          pk.y = pack_bf16x2(__uint_as_float(v[q4 * 8 + 2]) * ri, __uint_as_float(v[q4 * 8 + 3]) * ri);
          pk.z = pack_bf16x2(__uint_as_float(v[q4 * 8 + 4]) * ri, __uint_as_float(v[q4 * 8 + 5]) * ri);
          pk.w = pack_bf16x2(__uint_as_float(v[q4 * 8 + 6]) * ri, __uint_as_float(v[q4 * 8 + 7]) * ri);
          *reinterpret_cast<uint4*>(sl + (lc >> 3) * HALF + r * kRowBytes + (((lc & 7) ^ (r & 7)) << 4)) = pk;
        }
      }
      fence_proxy_async_smem();
      mbar_arrive(o_staged);
      bool stored = true;
      if (te == 0) {
        stored = mbar_wait(o_staged, it & 1, abort_flag);
        if (stored) {
          int c0, c1;
          box_coords<D>(0, hg, c0, c1);
          tma_store_4d(&map_o, sl, c0, c1, tt * kTileApply, b);
          box_coords<D>(1, hg, c0, c1);
          tma_store_4d(&map_o, sl + HALF, c0, c1, tt * kTileApply, b);
          tma_store_commit();
          tma_store_wait_read();
          mbar_arrive(&empty[s]);
        }
      }
      if (!__all_sync(0xffffffffu, stored)) break;  // leave the loop as a whole warp
    }
    if (te == 0) tma_store_wait_all();
  }

  // ------------------------------------------------------------ teardown
  tcgen05_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (threadIdx.x == 0) {
      *p.status = LINATTN_ERR_TIMEOUT;
      for (int s = 0; s < NS; ++s)
        for (int par = 0; par < 2; ++par)
          for (int spin = 0; spin < 4096 && !mbar_try_wait(&full[s], par); ++spin) __nanosleep(64);
    }
    __syncthreads();
  }
  if (warp == 1) {
    __syncwarp();
    tcgen05_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ============================================================================ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = [] {
    void* f = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      return (EncodeTiledFn) nullptr;
    return (EncodeTiledFn)f;
  }();
  return fn;
}

// 4-D bf16 map over (feature, head, token, batch) with a (box_d, box_h, tokens, 1) box, 128-byte swizzle,
// zero fill outside the tensor.
bool make_map(CUtensorMap* map, const Problem& p, const void* base, int box_d, int box_h, int box_tokens) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[4] = {(cuuint64_t)p.d, (cuuint64_t)p.H, (cuuint64_t)p.N, (cuuint64_t)p.B};
  cuuint64_t strides[3] = {(cuuint64_t)p.sh * 2, (cuuint64_t)p.sn * 2, (cuuint64_t)p.sb * 2};
  cuuint32_t box[4] = {(cuuint32_t)box_d, (cuuint32_t)box_h, (cuuint32_t)box_tokens, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int sm_count() {
  static int cached[64] = {0};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
  if (!cached[dev]) {
    int n = 0, major = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess || major != 10) return 0;
    cached[dev] = n > kMaxCtas ? kMaxCtas : n;
  }
  return cached[dev];
}

inline int groups_of(int d) { return d == 32 ? 4 : d == 64 ? 2 : 1; }

template <int D>
int launch_state(const Problem& p, const void* k, const void* v, float* state, bool accumulate, float* partials,
                 int* status, cudaStream_t stream) {
  using C = Cfg<D>;
  const int sms = sm_count();
  if (!sms) return LINATTN_ERR_CUDA;
  UmmaParams up{};
  up.B = p.B; up.H = p.H; up.HG = (p.H + C::G - 1) / C::G; up.N = p.N;
  up.tiles_per_unit = (int)((p.N + kTileState - 1) / kTileState);
  up.total_tiles = (long long)p.B * up.HG * up.tiles_per_unit;
  up.partials = partials; up.status = status;
  const int grid = (int)(up.total_tiles < sms ? up.total_tiles : sms);
  CUtensorMap mk, mv;
  if (!make_map(&mk, p, k, C::BOX_D, C::BOX_H, kTileState) || !make_map(&mv, p, v, C::BOX_D, C::BOX_H, kTileState))
    return LINATTN_ERR_CUDA;
  static bool attr_set = false;
  if (!attr_set) {
    if (cudaFuncSetAttribute(umma_state_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)C::STATE_SMEM) !=
        cudaSuccess)
      return LINATTN_ERR_CUDA;
    attr_set = true;
  }
  umma_state_kernel<D><<<grid, kThreads, C::STATE_SMEM, stream>>>(mk, mv, up);
  if (cudaGetLastError() != cudaSuccess) return LINATTN_ERR_CUDA;
  const long long E = p.state_elems();
  dim3 rgrid((unsigned)((E + 255) / 256), (unsigned)(p.B * p.H));
  umma_reduce_kernel<<<rgrid, 256, 0, stream>>>(partials, state, p.H, up.HG, C::G, D, up.tiles_per_unit, up.total_tiles,
                                                grid, accumulate ? 1 : 0);
  count_launches(2);
  return cudaGetLastError() == cudaSuccess ? LINATTN_OK : LINATTN_ERR_CUDA;
}

template <int D>
int launch_apply(const Problem& p, const void* q, const float* state, void* o, float eps, int* status,
                 cudaStream_t stream) {
  using C = Cfg<D>;
  const int sms = sm_count();
  if (!sms) return LINATTN_ERR_CUDA;
  UmmaParams up{};
  up.B = p.B; up.H = p.H; up.HG = (p.H + C::G - 1) / C::G; up.N = p.N;
  up.tiles_per_unit = (int)((p.N + kTileApply - 1) / kTileApply);
  up.total_tiles = (long long)p.B * up.HG * up.tiles_per_unit;
  up.state_in = state; up.eps = eps; up.status = status;
  const int grid = (int)(up.total_tiles < sms ? up.total_tiles : sms);
  CUtensorMap mq, mo;
  if (!make_map(&mq, p, q, C::BOX_D, C::BOX_H, kTileApply) || !make_map(&mo, p, o, C::BOX_D, C::BOX_H, kTileApply))
    return LINATTN_ERR_CUDA;
  static bool attr_set = false;
  if (!attr_set) {
    if (cudaFuncSetAttribute(umma_apply_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)C::APPLY_SMEM) !=
        cudaSuccess)
      return LINATTN_ERR_CUDA;
    attr_set = true;
  }
  umma_apply_kernel<D><<<grid, kThreads, C::APPLY_SMEM, stream>>>(mq, mo, up);
  count_launches(1);
  return cudaGetLastError() == cudaSuccess ? LINATTN_OK : LINATTN_ERR_CUDA;
}

}  // namespace

bool umma_supported(const Problem& p) {
  // d = 32 is not taken yet: a 64-byte inner TMA box is padded to the 128-byte swizzle pitch in shared
  // memory, so four heads cannot be packed into one operand row with this layout.
  return p.dtype == LINATTN_BF16 && (p.d == 64 || p.d == 112 || p.d == 128) &&
         p.N < (1ll << 31) && p.sh * 2 < (1ll << 40) && p.sn * 2 < (1ll << 40) && p.sb * 2 < (1ll << 40);
}

// One partial record (G head-states) per (CTA, unit) segment: at most kMaxCtas + units records.
size_t umma_partial_bytes(const Problem& p) {
  const int G = groups_of(p.d);
  const size_t units = (size_t)p.B * ((p.H + G - 1) / G);
  return ((size_t)kMaxCtas + units) * G * (size_t)p.state_elems() * sizeof(float);
}

int umma_state(const Problem& p, const void* k, const void* v, float* state_out, bool accumulate, void* workspace,
               cudaStream_t stream) {
  if (p.N == 0) {
    if (accumulate) return LINATTN_OK;
    return cudaMemsetAsync(state_out, 0, sizeof(float) * p.state_elems() * p.units(), stream) == cudaSuccess
               ? LINATTN_OK : LINATTN_ERR_CUDA;
  }
  float* partials = reinterpret_cast<float*>(static_cast<char*>(workspace) + LINATTN_WORKSPACE_CTRL_BYTES);
  int* status = &static_cast<WorkspaceCtrl*>(workspace)->status;
  switch (p.d) {
    case 64: return launch_state<64>(p, k, v, state_out, accumulate, partials, status, stream);
    case 112: return launch_state<112>(p, k, v, state_out, accumulate, partials, status, stream);
    case 128: return launch_state<128>(p, k, v, state_out, accumulate, partials, status, stream);
  }
  return LINATTN_ERR_UNSUPPORTED;
}

int umma_apply(const Problem& p, const void* q, const float* state, void* o, float eps, int* status,
               cudaStream_t stream) {
  if (p.N == 0) return LINATTN_OK;
  switch (p.d) {
    case 64: return launch_apply<64>(p, q, state, o, eps, status, stream);
    case 112: return launch_apply<112>(p, q, state, o, eps, status, stream);
    case 128: return launch_apply<128>(p, q, state, o, eps, status, stream);
  }
  return LINATTN_ERR_UNSUPPORTED;
}

}  // namespace linattn
