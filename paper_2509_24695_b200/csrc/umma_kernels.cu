// Tensor-core kernel for bf16 ReLU linear attention on sm_100a: TMA tiles into shared memory, a ReLU
// pass in place, tcgen05.mma with fp32 accumulators in tensor memory, results streamed out.
//
// Both contractions of the method are dense and run on the tensor cores, but the work is HBM-bound
// (about d/2 FLOP per byte); everything here is organised around keeping TMA loads in flight on every SM.
//
// ONE persistent, cooperatively launched kernel runs up to three passes back to back:
//
//   state pass   S = sum_n phi(k_n)^T v_n and z = sum_n phi(k_n)   (Eq. 2 / Eq. 3 state).
//                A = phi(K)^T and B = [V | 1] are both token-major in memory, i.e. MN-major UMMA
//                operands; the contraction index is the token.  The "ones" column makes z fall out of
//                the same MMA as one more accumulator column.  Work is split over tokens across the
//                grid (split-N); every CTA writes one fp32 partial record per unit segment it covered.
//   reduce       after a grid barrier the state is summed over the partial records in a fixed order
//                (deterministic), optionally on top of the existing state: the cache update of Eq. 3.
//                Either every CTA sums a slice of the whole state, or (one-head units, fused launch) the
//                CTAs of a unit share its reduce and also leave the unit's apply operand (S as bf16
//                hi + lo, z as one more row, in the shared-memory layout) in a per-unit image.  A second
//                grid barrier publishes state and images.
//   apply pass   o_n = phi(q_n) S / (phi(q_n).z + eps).  A = phi(Q) tile (K-major), B = S split into
//                bf16 hi + lo parts (two MMAs per K step, so S keeps ~16 mantissa bits), with z as an
//                extra row of B so the denominator is one more accumulator column.  B comes into shared
//                memory once per unit segment: one bulk copy of the unit's image, or built from the fp32
//                state.  The epilogue divides, rounds to bf16 and a dedicated warp TMA-stores the tile.
//
// The first Q tiles of the apply pass are fetched before the grid barriers (Q does not depend on the
// state), so HBM stays busy while the partials are reduced.
//
// Head dims 32 and 64 pack four / two heads into one 128-feature operand (the cross-head blocks of the
// product are ignored / zero); 112 pads to 128 through TMA out-of-bounds zero fill.
//
// Warp roles (352 threads): warp 0 TMA producer, warp 1 MMA issuer and TMEM owner, warps 2-5 ReLU
// pass, warps 6-9 epilogue, warp 10 output stores.  All cross-role synchronisation is by mbarriers
// with bounded waits, and the grid barrier is bounded too; a wait that runs out raises a CTA-wide
// abort flag, records LINATTN_ERR_TIMEOUT in the workspace status word, and every role falls through
// to the common teardown (TMEM is freed, loads in flight are waited for with a bound).
#include <cuda.h>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace linattn {
namespace {

using namespace ptx;

// Warp roles: warp 0 TMA producer, warp 1 MMA issuer, then the ReLU warps, four epilogue warps, one store
// warp.  The rotary variant does several times the arithmetic per element in the ReLU role (rotation,
// sums for z, denominators), so it runs that role on eight warps instead of four.
template <bool ROPE>
struct Roles {
  static constexpr int RELU_WARPS = ROPE ? 8 : 4;
  static constexpr int RELU_THREADS = RELU_WARPS * 32;
  static constexpr int EPI_WARP0 = 2 + RELU_WARPS;
  static constexpr int EPI_THREAD0 = EPI_WARP0 * 32;
  static constexpr int STORE_WARP = EPI_WARP0 + 4;
  static constexpr int THREADS = (STORE_WARP + 1) * 32;
};
constexpr int kReluThread0 = 64;
constexpr int kTileApply = 128;     // tokens per apply tile (= UMMA M)
constexpr int kTileState = 64;      // tokens per state stage (4 UMMA K steps of 16 tokens)
constexpr int kRowBytes = 128;      // one swizzle row: 64 bf16
constexpr int kBox = kTileState * kRowBytes;  // 8 KB: one 64-feature box of a state stage
constexpr int kTmemCols = 512;
constexpr int kAccStride = 256;     // TMEM columns between the two accumulator buffers

template <int D>
struct Cfg {
  static constexpr int G = D == 32 ? 4 : D == 64 ? 2 : 1;   // heads packed into one 128-feature operand
  static constexpr int FEAT = G * D;                         // 112 or 128 live features per group
  static constexpr int KSTEPS = FEAT / 16;                   // apply: K steps over features
  static constexpr int ZROW = D == 112 ? 112 : 128;          // apply: accumulator column of the first denominator
  static constexpr int NAPPLY = D == 112 ? 128 : 144;        // apply MMA N
  // state: with D = 112 the 1 sits in value column 112 (zero padding the TMA wrote), else in a
  // constant extra chunk of the stage
  static constexpr bool ONES_BOX = D != 112;
  static constexpr int NSTATE = ONES_BOX ? 144 : 128;        // state MMA N
  static constexpr int ZCOL = ONES_BOX ? 128 : 112;          // state accumulator column that holds z
  // The tensor core truncates when it adds into the fp32 accumulator, so a long chain of updates drifts
  // (about 2^-24 relative per update).  The state pass therefore deals its MMAs round-robin to several
  // accumulators, which the epilogue adds up (round to nearest) once per segment: shorter chains.
  static constexpr int STATE_ACCS = ONES_BOX ? 3 : 4;
  static constexpr int STATE_ACC_STRIDE = ONES_BOX ? 160 : 128;   // TMEM columns between them
  static constexpr int BOX_D = 64;                           // TMA box: features ...
  static constexpr int BOX_H = 1;                            // ... x heads
  static constexpr int SBOX_BYTES = NAPPLY * kRowBytes;      // one 64-feature K box of the S operand
  static constexpr int S_BYTES = 4 * SBOX_BYTES;             // (hi, lo) x 2 K boxes
  static constexpr int APPLY_SLOTS = D == 112 ? 5 : 4;
  static constexpr int SLOT_BYTES = 2 * kTileApply * kRowBytes;        // 32 KB: two 64-feature boxes
  static constexpr int STAGE_BYTES = (ONES_BOX ? 5 : 4) * kBox;        // V0 V1 [ONES] K0 K1
  static constexpr int KOFF = (ONES_BOX ? 3 : 2) * kBox;               // K boxes within a stage
  static constexpr int DATA_BYTES = S_BYTES + APPLY_SLOTS * SLOT_BYTES;
  // The data area would hold up to seven stages, but four measured fastest: with more bytes in flight
  // per SM the memory system's queues grow and the SMs' shares of the bandwidth drift apart.
  static constexpr int STATE_STAGES = DATA_BYTES / STAGE_BYTES < 4 ? DATA_BYTES / STAGE_BYTES : 4;
  static constexpr int BAR_BYTES = 1024;
  // rotary variant without row padding (every head dim but 112): the denominators of a tile's rows travel in a small
  // array per slot and head of the group
  static constexpr int DEN_BYTES = D == 112 ? 0 : G * APPLY_SLOTS * kTileApply * 4;
  static constexpr size_t SMEM = 1024 + DATA_BYTES + BAR_BYTES;
  static constexpr size_t SMEM_ROPE = SMEM + DEN_BYTES;
  // rotary variant: 16-byte chunk of a token's table row (d/2 fp16 pairs) that goes with logical chunk lc of box 0 / 1.
  // With packed heads (d = 32, 64) box 1 starts a new head, so both boxes use the same chunk.
  static constexpr bool SAME_TAB = 64 % D == 0;
  __host__ __device__ static constexpr int tab_chunk(int box, int lc) { return ((64 * box + 8 * lc) % D) / 8; }
};

// How the (unit, token tile) work of one pass is dealt to the persistent grid.
//
// A unit is one (batch, head group); its tiles are consecutive token ranges.  With U units and `grid`
// CTAs, the first P*U CTAs ("column" CTAs, P = grid / U) take tiles [c*Lc, (c+1)*Lc) of unit j % U with
// c = j / U and Lc = ceil(U*tpu / grid); the remaining R CTAs split the tiles [P*Lc, tpu) of all units
// evenly, unit after unit.  Column CTAs of neighbouring heads therefore walk the same token range at
// the same time.  That matters for head dims whose rows are not whole 128-byte lines (112 features =
// 224 bytes): a line shared by two heads comes from DRAM once if both heads ask for it while it is
// still in L2, and twice if their CTAs reach it tens of microseconds apart.
struct Sched {
  int U, tpu, grid;
  int P, Lc, R;
  int m;  // tiles per unit left to the R trailing CTAs: tpu - min(P*Lc, tpu)
};

// One CTA's share: flat positions [f0, f1); position f is tile tile_base + f % mm of unit
// unit_base + f / mm, and the partial record of that unit's segment is rec_base + f / mm.
struct Work {
  long long f0, f1;
  int mm, tile_base, unit_base, rec_base;
};

__host__ __device__ inline Work work_of(const Sched& s, int j) {
  Work w;
  w.f0 = w.f1 = 0; w.mm = 1; w.tile_base = 0; w.unit_base = 0; w.rec_base = 0;
  if (j >= s.grid) return w;
  if (j < s.P * s.U) {
    const int t0 = (j / s.U) * s.Lc;
    const int t1 = t0 + s.Lc < s.tpu ? t0 + s.Lc : s.tpu;
    w.f1 = t1 > t0 ? t1 - t0 : 0;
    w.mm = 0x7fffffff; w.tile_base = t0; w.unit_base = j % s.U; w.rec_base = j;
  } else {
    const int r = j - s.P * s.U;
    const long long tot = (long long)s.U * s.m;
    w.f0 = r * tot / s.R; w.f1 = (r + 1) * tot / s.R;
    w.mm = s.m > 0 ? s.m : 1; w.tile_base = s.P * s.Lc; w.rec_base = s.P * s.U + r;
  }
  return w;
}

// `seg_cost`: what starting one more unit segment costs a CTA, in tiles (drain of the accumulators /
// rebuild of the S operand).  Trailing CTAs cross several units, so the columns are made a little longer
// until the trailing CTAs' tiles plus their segment starts fit into a column's time.
inline Sched make_sched(int U, long long tpu, int max_ctas, int seg_cost) {
  Sched s;
  const long long total = (long long)U * tpu;
  s.U = U; s.tpu = (int)tpu;
  s.grid = (int)(total < max_ctas ? total : max_ctas);
  if (s.grid < 1) s.grid = 1;
  s.P = s.grid / U;
  s.R = s.grid - s.P * U;
  const int lc0 = (int)((total + s.grid - 1) / s.grid);
  s.Lc = lc0;
  if (s.P > 0 && s.R > 0) {
    for (int lc = lc0; lc < lc0 + 8; ++lc) {
      const long long m = (long long)s.P * lc >= tpu ? 0 : tpu - (long long)s.P * lc;
      const long long tiles = (U * m + s.R - 1) / s.R;
      const long long segs = m > 0 ? (tiles + m - 1) / m + 1 : 0;
      if (tiles + segs * seg_cost <= lc) { s.Lc = lc; break; }
    }
  }
  const long long covered = (long long)s.P * s.Lc;
  s.m = covered >= tpu ? 0 : (int)(tpu - covered);
  return s;
}

// Walks a Work range tile by tile.
struct TileWalk {
  const Work w;
  long long f;
  int uo, tp;
  __device__ explicit TileWalk(const Work& w_) : w(w_), f(w_.f0), uo((int)(w_.f0 / w_.mm)), tp((int)(w_.f0 % w_.mm)) {}
  __device__ bool done() const { return f >= w.f1; }
  __device__ int unit() const { return w.unit_base + uo; }
  __device__ int tile() const { return w.tile_base + tp; }
  __device__ int record() const { return w.rec_base + uo; }
  __device__ bool seg_first() const { return f == w.f0 || tp == 0; }
  __device__ bool seg_last() const { return f + 1 == w.f1 || tp == w.mm - 1; }
  __device__ void next() { ++f; if (++tp == w.mm) { tp = 0; ++uo; } }
};

struct FusedParams {
  int B, H, HG;            // HG: head groups per batch entry = ceil(H / G)
  Sched sa, sc;            // state pass (64-token stages) and apply pass (128-token tiles)
  int do_state, do_apply;
  int accumulate;          // reduce on top of state_base
  float* state;            // [B][H][(d+1)][d]: written by the reduce, read by the apply pass
  const float* state_base; // the state the new one is added to (the cache; may be `state` itself)
  float* partials;         // one record of G head-states per (CTA, unit) segment of the state pass
  float eps;
  WorkspaceCtrl* ctrl;
  uint8_t* s_image;        // non-null: the reduce also leaves every unit's S operand (bf16 hi + lo, in the shared-memory
                           // layout) here, S_BYTES per unit, and the apply pass fetches it with one bulk copy
  const uint4* rope;       // rotary variant: [N][d/8] chunks of four (cos, sin) fp16 pairs; null otherwise
  long long N;             // tokens (bound of the rotary table)
};

// rotary variant: floats a partial record carries for z: per warp that sums plain phi(k) (the eight ReLU warps, and
// the four epilogue warps, which take a share of the second K box in the state pass), per feature
constexpr int kZSlots = 12;
constexpr int kZParts = kZSlots * 128;

// TMA coordinates (feature, head) of 64-element box `box` (0/1) of head group hg
template <int D>
__device__ __forceinline__ void box_coords(int box, int hg, int& c0, int& c1) {
  if (Cfg<D>::G == 1) { c0 = 64 * box; c1 = hg; }
  else if (Cfg<D>::G == 2) { c0 = 0; c1 = 2 * hg + box; }
  else { c0 = 128 * hg + 64 * box; c1 = 0; }  // d = 32: the map sees a token's heads as one row of H*32 features
}

__device__ __forceinline__ uint8_t* align1024(uint8_t* p) {
  return reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(p) + 1023) & ~(uintptr_t)1023);
}

// In-place ReLU over the two 64-feature boxes (ROWS token rows of 128 bytes each, 128-byte swizzle) of a
// tile, 128 threads, thread `t`.  A thread owns one 16-byte column position of rows t/8 + 16*i; with the
// 128-byte swizzle the logical chunk at that position is the same for all of its rows, so with FEAT = 112
// a thread whose chunk of the second box holds only zero padding (features 112..127) skips that box.
// All loads of a box are issued before the first store.
template <int FEAT, int ROWS>
__device__ __forceinline__ void relu_pass(uint8_t* box0, uint8_t* box1, int t) {
  const int row0 = t >> 3, pc = t & 7;
  const int lc = pc ^ (row0 & 7);
  uint8_t* p0 = box0 + row0 * kRowBytes + pc * 16;
  uint8_t* p1 = box1 + row0 * kRowBytes + pc * 16;
  uint4 x[ROWS / 16];
#pragma unroll
  for (int i = 0; i < ROWS / 16; ++i) x[i] = *reinterpret_cast<uint4*>(p0 + i * 16 * kRowBytes);
#pragma unroll
  for (int i = 0; i < ROWS / 16; ++i) {
    x[i].x = relu_bf16x2(x[i].x); x[i].y = relu_bf16x2(x[i].y); x[i].z = relu_bf16x2(x[i].z); x[i].w = relu_bf16x2(x[i].w);
    *reinterpret_cast<uint4*>(p0 + i * 16 * kRowBytes) = x[i];
  }
  if (FEAT >= 128 || 64 + lc * 8 < FEAT) {
#pragma unroll
    for (int i = 0; i < ROWS / 16; ++i) x[i] = *reinterpret_cast<uint4*>(p1 + i * 16 * kRowBytes);
#pragma unroll
    for (int i = 0; i < ROWS / 16; ++i) {
      x[i].x = relu_bf16x2(x[i].x); x[i].y = relu_bf16x2(x[i].y); x[i].z = relu_bf16x2(x[i].z); x[i].w = relu_bf16x2(x[i].w);
      *reinterpret_cast<uint4*>(p1 + i * 16 * kRowBytes) = x[i];
    }
  }
}

// Rotary variant: a 16-byte chunk holds four feature pairs; `tab` holds their (cos, sin) as fp16 pairs.
// (a, b) -> (a c - b s, a s + b c), rounded to bf16.
// The ReLU role of the rotary variant is bound by instruction issue, so the clamp is done on the packed bf16
// pairs and the sums, the rotation and the denominators use the packed f32x2 instructions.
__device__ __forceinline__ void unpack_relu8(const uint4& x, float2 (&f)[4]) {
  const uint32_t w[4] = {relu_bf16x2(x.x), relu_bf16x2(x.y), relu_bf16x2(x.z), relu_bf16x2(x.w)};
#pragma unroll
  for (int e = 0; e < 4; ++e) f[e] = make_float2(__uint_as_float(w[e] << 16), __uint_as_float(w[e] & 0xFFFF0000u));
}
__device__ __forceinline__ uint4 rotate_pack8(const float2 (&f)[4], const uint4& tab) {
  const uint32_t t[4] = {tab.x, tab.y, tab.z, tab.w};
  uint32_t o[4];
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const float2 cs = __half22float2(*reinterpret_cast<const __half2*>(&t[e]));
    // (a, b) -> (a c - b s, b c + a s) = (-b, a) * (s, s) + (a, b) * (c, c)
    const float2 r = fma2(make_float2(-f[e].y, f[e].x), make_float2(cs.y, cs.y), mul2(f[e], make_float2(cs.x, cs.x)));
    o[e] = pack_bf16x2(r.x, r.y);
  }
  return make_uint4(o[0], o[1], o[2], o[3]);
}
constexpr uint32_t kRopeIdentity = 0x00003C00u;  // (cos, sin) = (1, 0) as an fp16 pair

// ---------------------------------------------------------------- grid barrier
__device__ __forceinline__ unsigned ld_acquire_gpu(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// All CTAs of the (cooperatively launched, hence co-resident) grid meet here.  One word holds an arrival count
// (low 16 bits) and a generation (high 16 bits).  Before a barrier the count is pre-set to 2^16 - grid (CTA 0 adds
// that: at kernel start for the first barrier, on leaving a barrier for the next one), so the last arrival's own
// atomic add carries into the generation: the CTAs polling the word see the barrier open one L2 round trip after
// the last arrival, with no second, dependent atomic in between (that cost 0.6 us per barrier).  All updates are
// atomic adds, which commute, so the carry happens at the (grid + 1)-th add whatever their order, and the count is
// back at zero after the launch's last barrier.  Every CTA has read the generation at kernel start (it cannot
// change before the CTA's own arrival), so it knows which value to wait for and starts polling without waiting for
// the answer to its own add (0.3-0.5 us per launch); the answer is only used afterwards, as a check.  The poll is
// bounded (about a second); on expiry the CTA raises its abort flag and goes on to the teardown.
__device__ __forceinline__ void grid_barrier_preset(WorkspaceCtrl* ctrl) {
  atomicAdd(&ctrl->barrier[0], 0x10000u - gridDim.x);
}

__device__ __forceinline__ void grid_barrier(WorkspaceCtrl* ctrl, volatile int* abort_flag, bool another_follows, unsigned gen_before) {
  tcgen05_fence_before();
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned* word = &ctrl->barrier[0];
    // release: the CTA's writes (seen by this thread through the bar.sync) are visible before the arrival is.
    // The value the add returns is looked at only after the poll, so the poll does not wait for it.
    unsigned old;
    asm volatile("atom.add.release.gpu.global.u32 %0, [%1], 1;" : "=r"(old) : "l"(word) : "memory");
    const unsigned long long t0 = global_timer_ns();
    while (((ld_acquire_gpu(word) >> 16) & 0xFFFFu) == (gen_before & 0xFFFFu)) {
      if (global_timer_ns() - t0 > kWaitLimitNs) { *abort_flag = 1; break; }
    }
    // a word that was not in the state a finished launch leaves it in (count zero) can carry early: the generation
    // this CTA met at its arrival then differs from the one it read at kernel start, and the launch is given up
    if (((old >> 16) & 0xFFFFu) != (gen_before & 0xFFFFu)) *abort_flag = 1;
    if (another_follows && blockIdx.x == 0 && !*abort_flag) grid_barrier_preset(ctrl);
  }
  __syncthreads();
  tcgen05_fence_after();
}

// ---------------------------------------------------------------- reduce
// This CTA's slice of the state: state[b][h][e] = (accumulate ? state : 0) + the partial records of
// the head's unit, column CTAs first (ascending), then the trailing CTAs (ascending).
//
// The reduce sits between two grid barriers with HBM idle, so it is written for latency: a thread takes
// up to NE elements (float4) of the slice, works out where all their records are, issues every load
// (NE x NR independent 16-byte loads, plus the old state when accumulating) and only then adds, in the
// fixed order.  Index arithmetic is 32-bit wherever the sizes allow: 64-bit division is a long
// subroutine, and a handful of them per element used to cost more time than the loads.

// Trailing CTA r covers the flat positions [r*tot/R, (r+1)*tot/R) (work_of); the one that holds position f is
// the largest r with r*tot/R <= f, i.e. floor(((f+1)*R - 1) / tot): one division.
__device__ __forceinline__ int trailing_cta_of(long long f, long long tot, int R) {
  if ((tot + 1) * R < 0xffffffffLL) return (int)((((unsigned)f + 1u) * (unsigned)R - 1u) / (unsigned)tot);
  return (int)(((f + 1) * R - 1) / tot);
}

__device__ __forceinline__ void add4(float4& a, const float4& b) { a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w; }

template <int D, bool ROPE, int NE, int NR>
__device__ __forceinline__ void reduce_elements(const FusedParams& p, int first, int i1, int ncol) {
  using C = Cfg<D>;
  constexpr int E4 = (D + 1) * D / 4;  // float4 per head state
  constexpr int REC4 = C::G * E4 + (ROPE ? kZParts / 4 : 0);  // float4 per partial record
  const Sched& s = p.sa;
  const long long ttot = (long long)s.U * s.m;
  float4* state4 = reinterpret_cast<float4*>(p.state);
  const float4* src[NE];
  int u_of[NE], r_lo[NE], nrec[NE];
  bool live[NE], zpart[NE];
  float4 sum[NE], v[NE][NR];
#pragma unroll
  for (int k = 0; k < NE; ++k) {
    const int idx = first + k * (int)blockDim.x;
    live[k] = idx < i1;
    zpart[k] = false;
    if (!live[k]) continue;
    sum[k] = p.accumulate ? __ldcg(reinterpret_cast<const float4*>(p.state_base) + idx) : make_float4(0.f, 0.f, 0.f, 0.f);
    const int bh = idx / E4, e = idx - bh * E4;
    const int b = bh / p.H, h = bh - b * p.H;
    const int u = b * p.HG + h / C::G, g = h % C::G;
    u_of[k] = u;
    src[k] = reinterpret_cast<const float4*>(p.partials) + (size_t)g * E4 + e;
    int ntrail = 0;
    r_lo[k] = 0;
    if (s.m > 0) {
      r_lo[k] = trailing_cta_of((long long)u * s.m, ttot, s.R);
      ntrail = trailing_cta_of((long long)(u + 1) * s.m - 1, ttot, s.R) - r_lo[k] + 1;
    }
    nrec[k] = ncol + ntrail;
    zpart[k] = ROPE && e >= D * D / 4;
  }
  auto record_of = [&](int k, int kk) { return kk < ncol ? kk * s.U + u_of[k] : s.P * s.U + r_lo[k] + (kk - ncol) + u_of[k]; };
  int nmax = 0;
#pragma unroll
  for (int k = 0; k < NE; ++k)
    if (live[k] && !zpart[k] && nrec[k] > nmax) nmax = nrec[k];
  for (int k0 = 0; k0 < nmax; k0 += NR) {
#pragma unroll
    for (int k = 0; k < NE; ++k)
#pragma unroll
      for (int r = 0; r < NR; ++r)
        if (live[k] && !zpart[k] && k0 + r < nrec[k]) v[k][r] = __ldcg(src[k] + (size_t)record_of(k, k0 + r) * REC4);
#pragma unroll
    for (int k = 0; k < NE; ++k)
#pragma unroll
      for (int r = 0; r < NR; ++r)
        if (live[k] && !zpart[k] && k0 + r < nrec[k]) add4(sum[k], v[k][r]);
  }
#pragma unroll
  for (int k = 0; k < NE; ++k) {
    if (!live[k]) continue;
    const int idx = first + k * (int)blockDim.x;
    if (ROPE && zpart[k]) {
      // rotary variant: z comes from the plain phi(k) sums that the ReLU warps of every segment left
      // behind the record (per warp, per feature): per warp slot the records in their fixed order, then the
      // slots as a balanced tree over sixteen, the missing ones zero (the association reduce_image's shuffles give)
      const int e = idx % E4;
      const int ft4 = (((idx / E4) % p.H) % C::G) * (D / 4) + (e - D * D / 4);   // float4 of the operand's 128 features
      const float4* zp = reinterpret_cast<const float4*>(p.partials) + C::G * E4 + ft4;
      // (one slot after the other: this form only runs when the operand images are not in use, and the
      // rotary kernel has no registers to spare)
      const bool upper = ft4 >= 16;   // features 64..: the epilogue warps' slots hold a share too
      // (computed depth first, a few registers at a time: this form only runs when the operand images are not in
      // use, and the rotary kernel has no registers to spare)
      auto slot = [&](int w) {
        float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
        if (w < 8 || (w < kZSlots && upper)) {
#pragma unroll 2
          for (int kk = 0; kk < nrec[k]; ++kk) add4(a, __ldcg(zp + (size_t)record_of(k, kk) * REC4 + w * 32));
        }
        return a;
      };
      auto pair = [&](int w) { float4 a = slot(w); add4(a, slot(w + 1)); return a; };
      auto quad = [&](int w) { float4 a = pair(w); add4(a, pair(w + 2)); return a; };
      float4 tree = quad(0);
      add4(tree, quad(4));
      float4 high = quad(8);
      add4(high, quad(12));
      add4(tree, high);
      add4(sum[k], tree);
    }
    state4[idx] = sum[k];
  }
}

template <int D, bool ROPE>
__device__ void reduce_slice(const FusedParams& p) {
  constexpr int E4 = (D + 1) * D / 4;
  const Sched& s = p.sa;
  const int tot = p.B * p.H * E4;   // < 2^31: at most 65535 units of at most 4128 float4
  const int per = tot / (int)gridDim.x, rem = tot - per * (int)gridDim.x, me = (int)blockIdx.x;
  const int i0 = me * per + (me < rem ? me : rem);
  const int i1 = i0 + per + (me < rem ? 1 : 0);
  const int ncol = s.P == 0 ? 0 : (s.P < (s.tpu + s.Lc - 1) / s.Lc ? s.P : (s.tpu + s.Lc - 1) / s.Lc);
  // few elements per thread: more records per batch; more elements: fewer records each (about 20 loads either way;
  // half as many in the rotary variant, whose 480 threads have 128 registers each)
  if (i1 - i0 <= 2 * (int)blockDim.x) {
    for (int first = i0 + (int)threadIdx.x; first < i1; first += 2 * (int)blockDim.x)
      reduce_elements<D, ROPE, 2, ROPE ? 5 : 10>(p, first, i1, ncol);
  } else {
    for (int first = i0 + (int)threadIdx.x; first < i1; first += 3 * (int)blockDim.x)
      reduce_elements<D, ROPE, 3, ROPE ? 3 : 6>(p, first, i1, ncol);
  }
}

// ---------------------------------------------------------------- reduce, with the S operand as a by-product
// Fused launches of one-head units (d = 112, 128) with at least one column CTA per unit: the column CTAs of a
// unit share its reduce (part c of P), in 32-byte chunks of a state row, and besides the fp32 state each chunk's
// sum is split into bf16 hi + lo and stored where the apply MMA wants it (the layout build_s_operand writes to
// shared memory), in a per-unit image in the workspace.  After the second barrier a CTA gets its unit's operand
// with one bulk copy instead of re-reading and converting the whole state: the conversion is done once per
// unit, not once per CTA, and the serial section between the passes is about 2 us shorter.  Same records in the
// same order as reduce_slice, so the state comes out bit for bit the same.
template <int D, bool ROPE, int NE, int NR>
__device__ __forceinline__ void reduce_image_chunks(const FusedParams& p, int u, int first, int hi_end, int ncol, int r_lo,
                                                    int nrec) {
  using C = Cfg<D>;
  constexpr int CPR = D / 8;                 // 32-byte chunks per state row
  constexpr int E4 = (D + 1) * D / 4;        // float4 per head state
  constexpr int REC4 = E4 + (ROPE ? kZParts / 4 : 0);
  const Sched& s = p.sa;
  auto record_of = [&](int kk) { return kk < ncol ? kk * s.U + u : s.P * s.U + r_lo + (kk - ncol) + u; };
  const float4* part4 = reinterpret_cast<const float4*>(p.partials);
  float4 sum[NE][2], v[NE][NR][2];
  int j_of[NE], c_of[NE];
  bool live[NE], zrow[NE];
#pragma unroll
  for (int k = 0; k < NE; ++k) {
    const int idx = first + k * (int)blockDim.x;
    live[k] = idx < hi_end;
    zrow[k] = false;
    if (!live[k]) continue;
    j_of[k] = idx / CPR;
    c_of[k] = idx - j_of[k] * CPR;
    zrow[k] = false;   // (rotary variant: the z row is not among the chunks, see reduce_image_zrow)
    const size_t e4 = (size_t)u * E4 + (size_t)j_of[k] * (D / 4) + 2 * c_of[k];
    if (p.accumulate) {
      sum[k][0] = __ldcg(reinterpret_cast<const float4*>(p.state_base) + e4);
      sum[k][1] = __ldcg(reinterpret_cast<const float4*>(p.state_base) + e4 + 1);
    } else {
      sum[k][0] = sum[k][1] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
  }
  for (int k0 = 0; k0 < nrec; k0 += NR) {
#pragma unroll
    for (int k = 0; k < NE; ++k)
#pragma unroll
      for (int r = 0; r < NR; ++r)
        if (live[k] && !zrow[k] && k0 + r < nrec) {
          const float4* src = part4 + (size_t)record_of(k0 + r) * REC4 + j_of[k] * (D / 4) + 2 * c_of[k];
          v[k][r][0] = __ldcg(src);
          v[k][r][1] = __ldcg(src + 1);
        }
#pragma unroll
    for (int k = 0; k < NE; ++k)
#pragma unroll
      for (int r = 0; r < NR; ++r)
        if (live[k] && !zrow[k] && k0 + r < nrec) { add4(sum[k][0], v[k][r][0]); add4(sum[k][1], v[k][r][1]); }
  }
#pragma unroll
  for (int k = 0; k < NE; ++k) {
    if (!live[k]) continue;
    const int j = j_of[k], c = c_of[k];
    float4* dst = reinterpret_cast<float4*>(p.state) + (size_t)u * E4 + (size_t)j * (D / 4) + 2 * c;
    dst[0] = sum[k][0];
    dst[1] = sum[k][1];
    const float x[8] = {sum[k][0].x, sum[k][0].y, sum[k][0].z, sum[k][0].w, sum[k][1].x, sum[k][1].y, sum[k][1].z, sum[k][1].w};
    uint32_t hi[4], lo[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const __nv_bfloat16 h0 = __float2bfloat16_rn(x[2 * e]), h1 = __float2bfloat16_rn(x[2 * e + 1]);
      hi[e] = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
      lo[e] = pack_bf16x2(x[2 * e] - __bfloat162float(h0), x[2 * e + 1] - __bfloat162float(h1));
    }
    const int jrow = j < D ? j : C::ZROW;   // operand row: value feature, or the z row
    const int i0 = c * 8;                   // first key feature of this chunk
    const int off = (i0 >> 6) * C::SBOX_BYTES + jrow * kRowBytes + ((((i0 & 63) >> 3) ^ (jrow & 7)) << 4);
    uint8_t* img = p.s_image + (size_t)u * C::S_BYTES;
    *reinterpret_cast<uint4*>(img + off) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
    *reinterpret_cast<uint4*>(img + 2 * C::SBOX_BYTES + off) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
  }
}

// Rotary variant: z of unit u from the plain phi(k) sums that the warps of every segment left behind the record,
// [12 warp slots][128 features] (the epilogue warps' slots 8..11 only for features 64..).  Thread (float4 hc of z,
// slot w of 16) adds its slot over the records in their fixed order (all loads in flight together; slots that
// do not exist count as zero), shuffles add the sixteen as a balanced tree, lane w = 0 adds the old z when
// accumulating; two neighbouring float4 make the 32-byte chunk of the operand image.
template <int D>
__device__ __forceinline__ void reduce_image_zrow(const FusedParams& p, int u, int ncol, int r_lo, int nrec) {
  using C = Cfg<D>;
  constexpr int E4 = (D + 1) * D / 4, REC4 = E4 + kZParts / 4, Z4 = D / 4, NR = 6;
  static_assert((16 * Z4) % 32 == 0 && Z4 % 2 == 0, "whole warps take part in the shuffles");
  // sixteen threads per float4 of z; with fewer than 16 * Z4 threads (d = 128: 512 wanted, 480 there) the first warps
  // take a second turn (whole warps: the shuffles below stay inside a warp)
  for (int t = (int)threadIdx.x; t < 16 * Z4; t += ((int)blockDim.x / 32) * 32) {
  const int hc = t >> 4, w = t & 15;
  const Sched& s = p.sa;
  auto record_of = [&](int kk) { return kk < ncol ? kk * s.U + u : s.P * s.U + r_lo + (kk - ncol) + u; };
  const float4* zp = reinterpret_cast<const float4*>(p.partials) + E4 + w * 32 + hc;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  if (w < 8 || (w < kZSlots && hc >= 16)) {
    for (int k0 = 0; k0 < nrec; k0 += NR) {
      float4 v[NR];
#pragma unroll
      for (int r = 0; r < NR; ++r)
        if (k0 + r < nrec) v[r] = __ldcg(zp + (size_t)record_of(k0 + r) * REC4);
#pragma unroll
      for (int r = 0; r < NR; ++r)
        if (k0 + r < nrec) add4(acc, v[r]);
    }
  }
#pragma unroll
  for (int st = 1; st < 16; st *= 2) {
    float4 o;
    o.x = __shfl_xor_sync(0xffffffffu, acc.x, st); o.y = __shfl_xor_sync(0xffffffffu, acc.y, st);
    o.z = __shfl_xor_sync(0xffffffffu, acc.z, st); o.w = __shfl_xor_sync(0xffffffffu, acc.w, st);
    add4(acc, o);
  }
  const size_t e4 = (size_t)u * E4 + (size_t)D * (D / 4) + hc;
  float4 sum = p.accumulate ? __ldcg(reinterpret_cast<const float4*>(p.state_base) + e4) : make_float4(0.f, 0.f, 0.f, 0.f);
  add4(sum, acc);
  float4 up;   // the upper half of this chunk, from the lane that holds float4 hc + 1
  up.x = __shfl_xor_sync(0xffffffffu, sum.x, 16); up.y = __shfl_xor_sync(0xffffffffu, sum.y, 16);
  up.z = __shfl_xor_sync(0xffffffffu, sum.z, 16); up.w = __shfl_xor_sync(0xffffffffu, sum.w, 16);
  if (w != 0) continue;
  reinterpret_cast<float4*>(p.state)[e4] = sum;
  if (hc & 1) continue;
  const float x[8] = {sum.x, sum.y, sum.z, sum.w, up.x, up.y, up.z, up.w};
  uint32_t hi[4], lo[4];
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const __nv_bfloat16 h0 = __float2bfloat16_rn(x[2 * e]), h1 = __float2bfloat16_rn(x[2 * e + 1]);
    hi[e] = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
    lo[e] = pack_bf16x2(x[2 * e] - __bfloat162float(h0), x[2 * e + 1] - __bfloat162float(h1));
  }
  const int jrow = C::ZROW, i0 = (hc >> 1) * 8;
  const int off = (i0 >> 6) * C::SBOX_BYTES + jrow * kRowBytes + ((((i0 & 63) >> 3) ^ (jrow & 7)) << 4);
  uint8_t* img = p.s_image + (size_t)u * C::S_BYTES;
  *reinterpret_cast<uint4*>(img + off) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
  *reinterpret_cast<uint4*>(img + 2 * C::SBOX_BYTES + off) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
  }
}

template <int D, bool ROPE>
__device__ void reduce_image(const FusedParams& p) {
  constexpr int TOTAL = (D + (ROPE ? 0 : 1)) * (D / 8);   // chunks of a unit (rotary: the z row goes separately)
  const Sched& s = p.sa;
  const int me = (int)blockIdx.x;
  if (me < s.P * s.U) {
    const int u = me % s.U, c = me / s.U;
    const int lo_i = c * TOTAL / s.P, hi_i = (c + 1) * TOTAL / s.P;
    const int ncol = s.P < (s.tpu + s.Lc - 1) / s.Lc ? s.P : (s.tpu + s.Lc - 1) / s.Lc;
    int r_lo = 0, ntrail = 0;
    if (s.m > 0) {
      const long long ttot = (long long)s.U * s.m;
      r_lo = trailing_cta_of((long long)u * s.m, ttot, s.R);
      ntrail = trailing_cta_of((long long)(u + 1) * s.m - 1, ttot, s.R) - r_lo + 1;
    }
    const int nrec = ncol + ntrail;
    if (hi_i - lo_i <= (int)blockDim.x) {
      reduce_image_chunks<D, ROPE, 1, ROPE ? 6 : 10>(p, u, lo_i + (int)threadIdx.x, hi_i, ncol, r_lo, nrec);
    } else {
      for (int first = lo_i + (int)threadIdx.x; first < hi_i; first += 2 * (int)blockDim.x)
        reduce_image_chunks<D, ROPE, 2, ROPE ? 3 : 6>(p, u, first, hi_i, ncol, r_lo, nrec);
    }
    if (ROPE && D % 8 == 0 && c == 0) reduce_image_zrow<D>(p, u, ncol, r_lo, nrec);
  }
  fence_proxy_async_all();   // the images are read through the async proxy (bulk copy) after the barrier
}

// ---------------------------------------------------------------- S operand of the apply pass
// Builds the B operand of the apply MMA for head group (b, hg) from the fp32 state: for every head
// of the group, rows = value features (plus one row for z), K = key features, split into bf16 hi + lo.
template <int D>
__device__ __forceinline__ void build_s_operand(uint8_t* s_op, const float* __restrict__ state, int b, int hg, int H,
                                                int part, int nparts) {
  using C = Cfg<D>;
  constexpr int CPR = D / 8;       // 16-byte chunks per state row
  constexpr int ROWS = D + 1;
  constexpr int TOTAL = C::G * ROWS * CPR;
  constexpr int BATCH = 7;         // chunks whose loads are in flight together (all of a thread's share at d = 112)
  for (int base = part; base < TOTAL; base += BATCH * nparts) {
    float4 lo4[BATCH], hi4[BATCH];
#pragma unroll
    for (int k = 0; k < BATCH; ++k) {
      const int idx = base + k * nparts;
      lo4[k] = hi4[k] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (idx < TOTAL) {
        const int g = idx / (ROWS * CPR);
        const int rem = idx - g * ROWS * CPR;
        const int j = rem / CPR, c = rem % CPR;
        const int h = hg * C::G + g;
        if (h < H) {
          const float4* src = reinterpret_cast<const float4*>(state + ((size_t)(b * H + h) * ROWS + j) * D + c * 8);
          lo4[k] = __ldcg(src);
          hi4[k] = __ldcg(src + 1);
        }
      }
    }
#pragma unroll
    for (int k = 0; k < BATCH; ++k) {
      const int idx = base + k * nparts;
      if (idx >= TOTAL) break;
      const int g = idx / (ROWS * CPR);
      const int rem = idx - g * ROWS * CPR;
      const int j = rem / CPR, c = rem % CPR;
      const float x[8] = {lo4[k].x, lo4[k].y, lo4[k].z, lo4[k].w, hi4[k].x, hi4[k].y, hi4[k].z, hi4[k].w};
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
}

// ============================================================================ the kernel
template <int D, bool ROPE>
__global__ void __launch_bounds__(Roles<ROPE>::THREADS, 1)
umma_fused_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                  const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_o, FusedParams p) {
  using C = Cfg<D>;
  using R = Roles<ROPE>;
  constexpr int NSA = C::STATE_STAGES;
  constexpr int STAGE = C::STAGE_BYTES;
  constexpr int NSC = C::APPLY_SLOTS;
  constexpr int SLOT = C::SLOT_BYTES;
  constexpr int HALF = SLOT / 2;  // one 64-feature box of 128 tokens
  constexpr uint32_t IDESC_A = make_idesc_bf16(128, C::NSTATE, true, true);
  constexpr uint32_t IDESC_C = make_idesc_bf16(128, C::NAPPLY, false, false);
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = align1024(smem_raw);
  uint8_t* s_op = smem;                    // apply pass: S operand ...
  uint8_t* slots = smem + C::S_BYTES;      // ... and the Q/O slots; the state pass stages cover both
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::DATA_BYTES);
  // state pass
  uint64_t* a_full = bars;                 // TMA landed
  uint64_t* a_ready = a_full + NSA;        // ReLU pass done
  uint64_t* a_empty = a_ready + NSA;       // MMAs that read the stage are complete
  uint64_t* a_tfull = a_empty + NSA;       // the segment's accumulators are complete
  uint64_t* a_tempty = a_tfull + 2;        // ... and drained by the epilogue
  uint64_t* a_done = a_tempty + 2;         // every MMA of the state pass is complete: stages are free
  // apply pass
  uint64_t* c_full = a_done + 1;           // Q tile landed
  uint64_t* c_ready = c_full + NSC;        // ReLU pass done
  uint64_t* c_empty = c_ready + NSC;       // O tile read out by its TMA store: slot reusable
  uint64_t* c_staged = c_empty + NSC;      // the 128 epilogue threads have written their O rows
  uint64_t* c_tfull = c_staged + NSC;      // [2] accumulator complete
  uint64_t* c_tempty = c_tfull + 2;        // [2] accumulator drained
  uint64_t* s_ready = c_tempty + 2;        // S operand of the current segment is in shared memory
  uint64_t* seg_done = s_ready + 1;        // every MMA of the finished segment is complete
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(seg_done + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);
  float* den_rows = reinterpret_cast<float*>(smem + C::DATA_BYTES + C::BAR_BYTES);   // [NSC][G][128]: rotary variant, every head dim but 112
  static_assert((3 * NSA + 5 + 4 * NSC + 6) * 8 + 8 <= C::BAR_BYTES, "barrier block too small");

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const Work wa = p.do_state ? work_of(p.sa, blockIdx.x) : work_of(p.sa, 0x7fffffff);
  const Work wc = p.do_apply ? work_of(p.sc, blockIdx.x) : work_of(p.sc, 0x7fffffff);

  // generation of the grid-barrier word before this launch's first barrier (it cannot move until every CTA, this
  // one included, has arrived): read once, early, so that an arrival needs no answer from memory
  unsigned gen0 = 0;
  if (threadIdx.x == 0 && p.do_state) gen0 = ld_acquire_gpu(&p.ctrl->barrier[0]) >> 16;
  if (threadIdx.x == 0) {
    if (blockIdx.x == 0 && p.do_state) grid_barrier_preset(p.ctrl);   // for the first grid barrier
    for (int s = 0; s < NSA; ++s) { mbar_init(&a_full[s], 1); mbar_init(&a_ready[s], R::RELU_THREADS + (ROPE ? 128 : 0)); mbar_init(&a_empty[s], 1); }
    mbar_init(a_tfull, 1);
    mbar_init(a_tempty, 128);
    mbar_init(a_done, 1);
    for (int s = 0; s < NSC; ++s) {
      mbar_init(&c_full[s], 1); mbar_init(&c_ready[s], R::RELU_THREADS); mbar_init(&c_empty[s], 1); mbar_init(&c_staged[s], 128);
    }
    for (int b = 0; b < 2; ++b) { mbar_init(&c_tfull[b], 1); mbar_init(&c_tempty[b], 128); }
    mbar_init(s_ready, R::RELU_THREADS + 128);
    mbar_init(seg_done, 128);
    *abort_flag = 0;
    fence_mbar_init();
    prefetch_tensormap(&map_k);
    prefetch_tensormap(&map_v);
    prefetch_tensormap(&map_q);
    prefetch_tensormap(&map_o);
  }
  if (C::ONES_BOX && wa.f1 > wa.f0) {
    // the constant "ones" chunk of every stage: value columns 128..191 of B, of which column 128 is 1
    for (int idx = threadIdx.x; idx < NSA * (kBox / 16); idx += R::THREADS) {
      const int s = idx / (kBox / 16), c = idx % (kBox / 16);
      const int row = c >> 3, phys = c & 7;
      uint4 val = make_uint4(0, 0, 0, 0);
      if ((phys ^ (row & 7)) == 0) val.x = 0x3F80u;  // bf16 1.0 in element 0 of logical chunk 0
      *reinterpret_cast<uint4*>(smem + s * STAGE + 2 * kBox + c * 16) = val;
    }
    fence_proxy_async_smem();
  }
  if (warp == 1) { tmem_alloc(tmem_holder, kTmemCols); tmem_relinquish(); }
  tcgen05_fence_before();
  __syncthreads();
  tcgen05_fence_after();
  const uint32_t tmem_base = *tmem_holder;

  // apply-pass producer state lives across the grid barriers (the first tiles are fetched before them)
  TileWalk cw(wc);
  uint32_t c_it = 0;
  auto load_q_tile = [&]() -> bool {
    const int s = c_it % NSC;
    if (!mbar_wait(&c_empty[s], ((c_it / NSC) & 1) ^ 1, abort_flag)) return false;
    const int u = cw.unit(), b = u / p.HG, hg = u % p.HG;
    uint8_t* sl = slots + s * SLOT;
    mbar_arrive_expect_tx(&c_full[s], SLOT);
    int c0, c1;
    box_coords<D>(0, hg, c0, c1);
    tma_load_4d(sl, &map_q, &c_full[s], c0, c1, cw.tile() * kTileApply, b);
    box_coords<D>(1, hg, c0, c1);
    tma_load_4d(sl + HALF, &map_q, &c_full[s], c0, c1, cw.tile() * kTileApply, b);
    cw.next();
    ++c_it;
    return true;
  };

  // ==================================================================== state pass
  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t it = 0;
      for (TileWalk t(wa); !t.done(); t.next(), ++it) {
        const int s = it % NSA;
        if (!mbar_wait(&a_empty[s], ((it / NSA) & 1) ^ 1, abort_flag)) break;
        const int u = t.unit(), b = u / p.HG, hg = u % p.HG;
        uint8_t* st = smem + s * STAGE;
        mbar_arrive_expect_tx(&a_full[s], 4 * kBox);
        int c0, c1;
        box_coords<D>(0, hg, c0, c1);
        tma_load_4d(st + C::KOFF, &map_k, &a_full[s], c0, c1, t.tile() * kTileState, b);
        tma_load_4d(st, &map_v, &a_full[s], c0, c1, t.tile() * kTileState, b);
        box_coords<D>(1, hg, c0, c1);
        tma_load_4d(st + C::KOFF + kBox, &map_k, &a_full[s], c0, c1, t.tile() * kTileState, b);
        tma_load_4d(st + kBox, &map_v, &a_full[s], c0, c1, t.tile() * kTileState, b);
      }
      // Q does not depend on the state: fill the slots as soon as every MMA of this pass is complete (the
      // stages are free then).  Asking for tiles earlier or further ahead with TMA prefetches into L2
      // measured slower at every distance tried (0-24 tiles).
      if (wc.f1 > wc.f0 && mbar_wait(a_done, 0, abort_flag)) {
        while (!cw.done() && c_it < (uint32_t)NSC)
          if (!load_q_tile()) break;
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      uint32_t it = 0, seg = 0, n_mma = 0;
      bool ok = true;
      for (TileWalk t(wa); !t.done() && ok; t.next(), ++it) {
        const int s = it % NSA;
        const bool seg_first = t.seg_first();
        if (seg_first) { ok = mbar_wait(a_tempty, (seg & 1) ^ 1, abort_flag); n_mma = 0; }
        if (ok) ok = mbar_wait(&a_ready[s], (it / NSA) & 1, abort_flag);
        if (!ok) break;
        tcgen05_fence_after();
        const uint32_t st = smem_u32(smem + s * STAGE);
#pragma unroll
        for (int kk = 0; kk < kTileState / 16; ++kk, ++n_mma) {
          const uint64_t a = make_smem_desc_sw128(st + C::KOFF + kk * 2048, kBox, 1024);  // phi(K)^T, MN-major
          const uint64_t bq = make_smem_desc_sw128(st + kk * 2048, kBox, 1024);           // [V | 1], MN-major
          const uint32_t d_tmem = tmem_base + (n_mma % C::STATE_ACCS) * C::STATE_ACC_STRIDE;
          umma_bf16(d_tmem, a, bq, IDESC_A, n_mma < (uint32_t)C::STATE_ACCS ? 0u : 1u);  // first use of each: overwrite
        }
        umma_commit(&a_empty[s]);
        if (t.seg_last()) { umma_commit(a_tfull); ++seg; }
      }
      if (it > 0) umma_commit(a_done); else mbar_arrive(a_done);
    }
  } else if (warp < R::EPI_WARP0) {
    // ------------------------------------------------------------ ReLU pass over the K boxes
    const int tr = threadIdx.x - kReluThread0;
    uint32_t it = 0;
    // rotary variant: this thread's 16-byte column holds logical chunk lc of every row it touches
    const int row0 = tr >> 3, pc = tr & 7, lc = pc ^ (row0 & 7);
    const bool box1_live = 64 + lc * 8 < C::FEAT;
    float2 zacc[8];  // sums of the plain phi(k) over the segment: features 8*lc.. of box 0, 64 + 8*lc.. of box 1
#pragma unroll
    for (int e = 0; e < 8; ++e) zacc[e] = make_float2(0.f, 0.f);
    // The rotations of a row do not depend on K: they are fetched one stage ahead, each register reloaded
    // for the next stage right after its use, so that their latency is off the stage's critical path.
    // Of the second K box these warps take the first 32 token rows of a stage; the epilogue warps, idle until the
    // segment's accumulators are complete, take the other 32 (this role is what the pass waits for).
    uint4 tab0[kTileState / 32], tab1[1];
    auto fetch_rot = [&](int tile, int i) {
      const long long n = (long long)tile * kTileState + row0 + 32 * i;
      tab0[i] = make_uint4(kRopeIdentity, kRopeIdentity, kRopeIdentity, kRopeIdentity);
      if (i == 0) tab1[0] = tab0[i];
      if (n < p.N) {
        tab0[i] = __ldg(p.rope + n * (D / 8) + C::tab_chunk(0, lc));
        if (i == 0) {
          if (C::SAME_TAB) tab1[0] = tab0[0];
          else if (box1_live) tab1[0] = __ldg(p.rope + n * (D / 8) + C::tab_chunk(1, lc));
        }
      }
    };
    if (ROPE) {
      TileWalk t0(wa);
      if (!t0.done()) {
#pragma unroll
        for (int i = 0; i < kTileState / 32; ++i) fetch_rot(t0.tile(), i);
      }
    }
    for (TileWalk t(wa); !t.done(); t.next(), ++it) {
      const int s = it % NSA;
      uint8_t* st = smem + s * STAGE;
      if (ROPE) {
        TileWalk tn = t;
        tn.next();
        if (!__all_sync(0xffffffffu, mbar_wait(&a_full[s], (it / NSA) & 1, abort_flag))) break;  // leave as a whole warp
        uint8_t* p0 = st + C::KOFF + row0 * kRowBytes + pc * 16;
#pragma unroll
        for (int i = 0; i < kTileState / 32; ++i) {
          float2 f[4];
          uint4* c0 = reinterpret_cast<uint4*>(p0 + i * 32 * kRowBytes);
          unpack_relu8(*c0, f);
#pragma unroll
          for (int e = 0; e < 4; ++e) zacc[e] = add2(zacc[e], f[e]);
          *c0 = rotate_pack8(f, tab0[i]);
          if (i == 0 && box1_live) {
            uint4* c1 = reinterpret_cast<uint4*>(p0 + kBox);
            unpack_relu8(*c1, f);
#pragma unroll
            for (int e = 0; e < 4; ++e) zacc[4 + e] = add2(zacc[4 + e], f[e]);
            *c1 = rotate_pack8(f, tab1[0]);
          }
          if (!tn.done()) fetch_rot(tn.tile(), i);
        }
        fence_proxy_async_smem();
        mbar_arrive(&a_ready[s]);
        if (t.seg_last()) {
          // leave the segment's sums behind the record: the four lanes of this warp that share a chunk add
          // up in a fixed order, then one of them stores
          const int w = tr >> 5, r = (tr >> 3) & 3;
          float tot[16];
#pragma unroll
          for (int e = 0; e < 16; ++e) tot[e] = 0.f;
#pragma unroll
          for (int rr = 0; rr < 4; ++rr) {
            const int src = (rr << 3) | (lc ^ ((4 * (w & 1) + rr) & 7));
#pragma unroll
            for (int e = 0; e < 16; ++e) tot[e] += __shfl_sync(0xffffffffu, (e & 1) ? zacc[e >> 1].y : zacc[e >> 1].x, src);
          }
          if (r == 0) {
            float* zp = p.partials + (size_t)t.record() * (C::G * (D + 1) * D + kZParts) + C::G * (D + 1) * D + w * 128;
            *reinterpret_cast<float4*>(zp + 8 * lc) = make_float4(tot[0], tot[1], tot[2], tot[3]);
            *reinterpret_cast<float4*>(zp + 8 * lc + 4) = make_float4(tot[4], tot[5], tot[6], tot[7]);
            if (box1_live) {
              *reinterpret_cast<float4*>(zp + 64 + 8 * lc) = make_float4(tot[8], tot[9], tot[10], tot[11]);
              *reinterpret_cast<float4*>(zp + 64 + 8 * lc + 4) = make_float4(tot[12], tot[13], tot[14], tot[15]);
            }
          }
#pragma unroll
          for (int e = 0; e < 8; ++e) zacc[e] = make_float2(0.f, 0.f);
        }
        continue;
      }
      if (!mbar_wait(&a_full[s], (it / NSA) & 1, abort_flag)) break;
      relu_pass<C::FEAT, kTileState>(st + C::KOFF, st + C::KOFF + kBox, tr);
      if (!C::ONES_BOX && tr < kTileState) {
        // value column 112 := 1 (logical chunk 6 of the second V box, element 0), so z is accumulator column 112
        *reinterpret_cast<uint16_t*>(st + kBox + tr * kRowBytes + ((6 ^ (tr & 7)) << 4)) = 0x3F80u;
      }
      fence_proxy_async_smem();
      mbar_arrive(&a_ready[s]);
    }
  } else if (warp < R::STORE_WARP) {
    // ------------------------------------------------------------ epilogue: accumulator -> partial record
    const int wq = warp & 3;
    const int i = wq * 32 + lane;           // accumulator lane = key feature within the group
    const int g = i / D, il = i % D;        // head within the group, feature within the head
    uint32_t seg = 0;
    // rotary variant: token rows 32..63 of the second K box of every stage (see the ReLU role); thread te owns
    // the 16-byte column position pch of rows 32 + row0h + 16 j, which holds logical chunk lch in all of them
    const int te = threadIdx.x - R::EPI_THREAD0;
    const int row0h = te >> 3, pch = te & 7, lch = pch ^ (row0h & 7);
    const bool h_live = 64 + lch * 8 < C::FEAT;
    float2 zh[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) zh[e] = make_float2(0.f, 0.f);
    uint4 tabh[2];
    auto fetch_roth = [&](int tile, int j) {
      const long long n = (long long)tile * kTileState + 32 + row0h + 16 * j;
      tabh[j] = make_uint4(kRopeIdentity, kRopeIdentity, kRopeIdentity, kRopeIdentity);
      if (h_live && n < p.N) tabh[j] = __ldg(p.rope + n * (D / 8) + C::tab_chunk(1, lch));
    };
    if (ROPE) {
      TileWalk t0(wa);
      if (!t0.done()) { fetch_roth(t0.tile(), 0); fetch_roth(t0.tile(), 1); }
    }
    uint32_t it = 0;
    for (TileWalk t(wa); !t.done(); t.next(), ++it) {
      if (ROPE) {
        const int s = it % NSA;
        TileWalk tn = t;
        tn.next();
        if (!__all_sync(0xffffffffu, mbar_wait(&a_full[s], (it / NSA) & 1, abort_flag))) break;  // leave as a whole warp
        uint8_t* p1 = smem + s * STAGE + C::KOFF + kBox + (32 + row0h) * kRowBytes + pch * 16;
#pragma unroll
        for (int j = 0; j < 2; ++j) {
          if (h_live) {
            float2 f[4];
            uint4* c1 = reinterpret_cast<uint4*>(p1 + j * 16 * kRowBytes);
            unpack_relu8(*c1, f);
#pragma unroll
            for (int e = 0; e < 4; ++e) zh[e] = add2(zh[e], f[e]);
            *c1 = rotate_pack8(f, tabh[j]);
          }
          if (!tn.done()) fetch_roth(tn.tile(), j);
        }
        fence_proxy_async_smem();
        mbar_arrive(&a_ready[s]);
        if (t.seg_last()) {
          // this warp's share of the segment's z: the four lanes that share a chunk add up in a fixed order
          const int rq = (te >> 3) & 3;
          float tot[8];
#pragma unroll
          for (int e = 0; e < 8; ++e) tot[e] = 0.f;
#pragma unroll
          for (int rr = 0; rr < 4; ++rr) {
            const int src = (rr << 3) | (lch ^ ((4 * ((te >> 5) & 1) + rr) & 7));
#pragma unroll
            for (int e = 0; e < 8; ++e) tot[e] += __shfl_sync(0xffffffffu, (e & 1) ? zh[e >> 1].y : zh[e >> 1].x, src);
          }
          if (rq == 0 && h_live) {
            float* zp = p.partials + (size_t)t.record() * (C::G * (D + 1) * D + kZParts) + C::G * (D + 1) * D + (8 + (te >> 5)) * 128;
            *reinterpret_cast<float4*>(zp + 64 + 8 * lch) = make_float4(tot[0], tot[1], tot[2], tot[3]);
            *reinterpret_cast<float4*>(zp + 64 + 8 * lch + 4) = make_float4(tot[4], tot[5], tot[6], tot[7]);
          }
#pragma unroll
          for (int e = 0; e < 4; ++e) zh[e] = make_float2(0.f, 0.f);
        }
      }
      if (!t.seg_last()) continue;
      bool ok = mbar_wait(a_tfull, seg & 1, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tcgen05_fence_after();
      const int u = t.unit(), hg = u % p.HG;
      const int h = hg * C::G + g;
      const bool live = i < C::FEAT && h < p.H;
      // record of this (CTA, unit) segment: G consecutive head-states in the library's layout
      float* out = p.partials + (size_t)t.record() * (C::G * (D + 1) * D + (ROPE ? kZParts : 0)) + (size_t)g * ((D + 1) * D);
      const uint32_t trow = tmem_base + ((uint32_t)(wq * 32) << 16);
#pragma unroll 1
      for (int cc = 0; cc < 4; ++cc) {
        // the accumulators are added in a fixed order (round to nearest)
        float sum[32];
        {
          uint32_t r[32];
          tmem_ld_x32(trow + cc * 32, r);
          tmem_ld_wait();
#pragma unroll
          for (int x = 0; x < 32; ++x) sum[x] = __uint_as_float(r[x]);
        }
#pragma unroll 1
        for (int a = 1; a < C::STATE_ACCS; ++a) {
          uint32_t r[32];
          tmem_ld_x32(trow + a * C::STATE_ACC_STRIDE + cc * 32, r);
          tmem_ld_wait();
#pragma unroll
          for (int x = 0; x < 32; ++x) sum[x] += __uint_as_float(r[x]);
        }
        if (live) {
#pragma unroll
          for (int x = 0; x < 32; ++x) {
            const int j = cc * 32 + x;             // value feature within the group
            const int jl = j - g * D;
            if (jl >= 0 && jl < D) out[(size_t)jl * D + il] = sum[x];
            if (!C::ONES_BOX && !ROPE && j == C::ZCOL) out[(size_t)D * D + il] = sum[x];  // (rotary: z comes from the ReLU warps)
          }
        }
      }
      if (C::ONES_BOX && !ROPE) {   // (rotary: z comes from the ReLU warps)
        float zsum = 0.f;
#pragma unroll 1
        for (int a = 0; a < C::STATE_ACCS; ++a) {
          uint32_t zr[4];
          tmem_ld_x4(trow + a * C::STATE_ACC_STRIDE + C::ZCOL, zr);
          tmem_ld_wait();
          zsum = a == 0 ? __uint_as_float(zr[0]) : zsum + __uint_as_float(zr[0]);
        }
        if (live) out[(size_t)D * D + il] = zsum;
      }
      tcgen05_fence_before();
      mbar_arrive(a_tempty);
      ++seg;
    }
  } else if (C::G == 1 && p.s_image && p.accumulate && p.do_state && (int)blockIdx.x < p.sa.P * p.sa.U) {
    // ------------------------------------------------------------ store warp (idle in this pass)
    // A cached step adds to the old state, which the K, V stream has pushed out of L2 since the last step:
    // once this CTA's loads are all issued, ask for its share of it (reduce_image's split), so that the
    // reduce finds it in L2 instead of waiting for DRAM between the two grid barriers.
    if (__all_sync(0xffffffffu, mbar_wait(a_done, 0, abort_flag))) {
      constexpr int TOTAL = (D + (ROPE ? 0 : 1)) * (D / 8);
      const int u = (int)blockIdx.x % p.sa.U, c = (int)blockIdx.x / p.sa.U;
      const int lo_i = c * TOTAL / p.sa.P, hi_i = (c + 1) * TOTAL / p.sa.P;
      const char* base = reinterpret_cast<const char*>(p.state_base + (size_t)u * ((D + 1) * D)) + (size_t)lo_i * 32;
      for (int off = lane * 128; off < (hi_i - lo_i) * 32; off += 32 * 128)
        asm volatile("prefetch.global.L2 [%0];" ::"l"(base + off) : "memory");
    }
  }

  // ==================================================================== reduce
  if (p.do_state) {
    grid_barrier(p.ctrl, abort_flag, p.do_apply != 0, gen0);
    if (!*abort_flag) {
      if (C::G == 1 && p.s_image) reduce_image<D, ROPE>(p);
      else reduce_slice<D, ROPE>(p);
    }
    if (p.do_apply) grid_barrier(p.ctrl, abort_flag, false, gen0 + 1);
  }
  if (C::G > 1 && wc.f1 > wc.f0) {
    // cross-head blocks of the packed S operand are never written by a head: they must read as zero
    for (int idx = threadIdx.x; idx < C::S_BYTES / 16; idx += R::THREADS)
      *reinterpret_cast<uint4*>(s_op + idx * 16) = make_uint4(0, 0, 0, 0);
    __syncthreads();
  }

  // ==================================================================== apply pass
  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer: the remaining Q tiles
    if (lane == 0) {
      while (!cw.done())
        if (!load_q_tile()) break;
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      uint32_t it = 0, seg = 0;
      bool ok = true;
      for (TileWalk t(wc); !t.done() && ok; t.next(), ++it) {
        const int s = it % NSC;
        if (t.seg_first()) { ok = mbar_wait(s_ready, seg & 1, abort_flag); ++seg; }
        const uint32_t acc = it & 1;
        if (ok) ok = mbar_wait(&c_tempty[acc], ((it >> 1) & 1) ^ 1, abort_flag);
        if (ok) ok = mbar_wait(&c_ready[s], (it / NSC) & 1, abort_flag);
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
          umma_bf16(d_tmem, a, bh, IDESC_C, k == 0 ? 0u : 1u);
          umma_bf16(d_tmem, a, bl, IDESC_C, 1u);
        }
        umma_commit(&c_tfull[acc]);
      }
    }
  } else if (warp < R::EPI_WARP0) {
    // ------------------------------------------------------------ ReLU pass over Q tiles (+ half of the S build)
    const int tr = threadIdx.x - kReluThread0;
    uint32_t it = 0, seg = 0;
    bool ok = true;
    // rotary variant: this thread's 16-byte column holds logical chunk lc of every row it touches
    const int row0 = tr >> 3, pc = tr & 7, lc = pc ^ (row0 & 7);
    const bool box1_live = 64 + lc * 8 < C::FEAT;
    float2 zc[8];  // the segment's z at this thread's features (8*lc.. of box 0, 64 + 8*lc.. of box 1)
#pragma unroll
    for (int e = 0; e < 8; ++e) zc[e] = make_float2(0.f, 0.f);
    // rotations one tile ahead, as in the state pass
    uint4 tab0[kTileApply / 32], tab1[kTileApply / 32];
    auto fetch_rot = [&](int tile, int i) {
      const long long n = (long long)tile * kTileApply + row0 + 32 * i;
      tab0[i] = tab1[i] = make_uint4(kRopeIdentity, kRopeIdentity, kRopeIdentity, kRopeIdentity);
      if (n < p.N) {
        tab0[i] = __ldg(p.rope + n * (D / 8) + C::tab_chunk(0, lc));
        if (C::SAME_TAB) tab1[i] = tab0[i];
        else if (box1_live) tab1[i] = __ldg(p.rope + n * (D / 8) + C::tab_chunk(1, lc));
      }
    };
    if (ROPE) {
      TileWalk t0(wc);
      if (!t0.done()) {
#pragma unroll
        for (int i = 0; i < kTileApply / 32; ++i) fetch_rot(t0.tile(), i);
      }
    }
    for (TileWalk t(wc); !t.done() && ok; t.next(), ++it) {
      const int s = it % NSC;
      if (t.seg_first()) {
        // the previous segment's MMAs must be done before its S operand is overwritten
        if (seg > 0) ok = mbar_wait(seg_done, (seg - 1) & 1, abort_flag);
        if (!ok) break;
        const int u = t.unit();
        if (C::G == 1 && p.s_image) {
          if (tr == 0) {   // the unit's operand image, made by the reduce: one bulk copy
            fence_proxy_async_all();
            mbar_arrive_expect_tx(s_ready, C::S_BYTES);
            bulk_load(s_op, p.s_image + (size_t)u * C::S_BYTES, C::S_BYTES, s_ready);
          } else {
            mbar_arrive(s_ready);
          }
        } else {
          build_s_operand<D>(s_op, p.state, u / p.HG, u % p.HG, p.H, tr, R::RELU_THREADS + 128);
        }
        if (ROPE) {
          // feature 64 * box + 8 * lc of the operand is feature fl of head g of the group
#pragma unroll
          for (int box = 0; box < 2; ++box) {
            const int f0 = 64 * box + 8 * lc, g = f0 / D, fl = f0 - g * D;
            const int h = (u % p.HG) * C::G + g;
            float4 a0 = make_float4(0.f, 0.f, 0.f, 0.f), a1 = a0;
            if ((box == 0 || box1_live) && h < p.H) {
              const float4* zrow = reinterpret_cast<const float4*>(p.state + ((size_t)((u / p.HG) * p.H + h) * (D + 1) + D) * D);
              a0 = __ldcg(zrow + fl / 4);
              a1 = __ldcg(zrow + fl / 4 + 1);
            }
            zc[4 * box + 0] = make_float2(a0.x, a0.y); zc[4 * box + 1] = make_float2(a0.z, a0.w);
            zc[4 * box + 2] = make_float2(a1.x, a1.y); zc[4 * box + 3] = make_float2(a1.z, a1.w);
          }
        }
        if (!(C::G == 1 && p.s_image)) {
          fence_proxy_async_smem();
          mbar_arrive(s_ready);
        }
        ++seg;
      }
      if (ROPE) {
        // numerator operand: rotated phi(q); denominator: plain phi(q) . z, added up over the eight lanes that
        // share a row and left in the row's zero padding (features 112..) for the epilogue
        uint8_t* sl = slots + s * SLOT;
        TileWalk tn = t;
        tn.next();
        if (!__all_sync(0xffffffffu, mbar_wait(&c_full[s], (it / NSC) & 1, abort_flag))) break;  // leave as a whole warp
        uint8_t* p0 = sl + row0 * kRowBytes + pc * 16;
#pragma unroll
        for (int i = 0; i < kTileApply / 32; ++i) {
          float2 f[4];
          uint4* c0 = reinterpret_cast<uint4*>(p0 + i * 32 * kRowBytes);
          unpack_relu8(*c0, f);
          float2 den2 = make_float2(0.f, 0.f);
#pragma unroll
          for (int e = 0; e < 4; ++e) den2 = fma2(f[e], zc[e], den2);
          *c0 = rotate_pack8(f, tab0[i]);
          uint4* c1 = reinterpret_cast<uint4*>(p0 + HALF + i * 32 * kRowBytes);
          float2 den2b = make_float2(0.f, 0.f);   // packed heads: box 1 belongs to other heads than box 0
          if (box1_live) {
            unpack_relu8(*c1, f);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              if (C::G == 1) den2 = fma2(f[e], zc[4 + e], den2);
              else den2b = fma2(f[e], zc[4 + e], den2b);
            }
            *c1 = rotate_pack8(f, tab1[i]);
          }
          float den = den2.x + den2.y;
          if (!tn.done()) fetch_rot(tn.tile(), i);  // this row's rotations for the next tile
          // The eight lanes of a row hold one chunk of each box.  One head per operand: add all of it over the eight.
          // Packed heads: box 1 belongs to other heads, and with d = 32 a head is four lanes wide; the first exchange
          // hands one box's sum to the partner lane, so that each half of the lanes reduces one box.
          const int row = row0 + 32 * i;
          if (C::G == 1) {
            den += __shfl_xor_sync(0xffffffffu, den, 1);
            den += __shfl_xor_sync(0xffffffffu, den, 2);
            den += __shfl_xor_sync(0xffffffffu, den, 4);
            if (D == 112) {
              if (lc == 6) *reinterpret_cast<float*>(c1) = den;  // chunk 6 of the second box: features 112..119
            } else {
              if (pc == 0) den_rows[s * kTileApply + row] = den;   // no padding to carry it
            }
          } else {
            const float denb = den2b.x + den2b.y;
            constexpr int XB = C::G == 2 ? 4 : 2;             // lane bit that picks the box after the exchange
            const bool second = (pc & XB) != 0;
            float x = second ? denb : den;
            x += __shfl_xor_sync(0xffffffffu, second ? den : denb, XB);
            x += __shfl_xor_sync(0xffffffffu, x, 1);
            if (C::G == 2) x += __shfl_xor_sync(0xffffffffu, x, 2);
            // d = 64: lane 0 of the row has head 0 (box 0), lane 4 head 1.  d = 32: lanes with the same pc / 4 share
            // a head, whose place in its box is lc / 4; lanes 0 and 4 have box 0, lanes 2 and 6 box 1
            if (C::G == 2) {
              if ((pc & 3) == 0) den_rows[(s * 2 + (second ? 1 : 0)) * kTileApply + row] = x;
            } else {
              if ((pc & 1) == 0) den_rows[(s * 4 + (second ? 2 : 0) + (lc >> 2)) * kTileApply + row] = x;
            }
          }
        }
        fence_proxy_async_smem();
        mbar_arrive(&c_ready[s]);
        continue;
      }
      if (!mbar_wait(&c_full[s], (it / NSC) & 1, abort_flag)) break;
      relu_pass<C::FEAT, kTileApply>(slots + s * SLOT, slots + s * SLOT + HALF, tr);
      fence_proxy_async_smem();
      mbar_arrive(&c_ready[s]);
    }
  } else if (warp < R::STORE_WARP) {
    // ------------------------------------------------------------ epilogue: divide, round, stage the O tile
    const int wq = warp & 3;
    const int te = threadIdx.x - R::EPI_THREAD0;
    const int r = wq * 32 + lane;  // accumulator lane = token row of the tile
    uint32_t it = 0;
    for (TileWalk t(wc); !t.done(); t.next(), ++it) {
      const int s = it % NSC;
      if (t.seg_first()) {
        // this thread has seen the last accumulator of the previous segment complete: S may be rebuilt
        const int u = t.unit();
        if (!(C::G == 1 && p.s_image)) {
          build_s_operand<D>(s_op, p.state, u / p.HG, u % p.HG, p.H, R::RELU_THREADS + te, R::RELU_THREADS + 128);
          fence_proxy_async_smem();
        }
        mbar_arrive(s_ready);
      }
      const uint32_t acc = it & 1;
      bool ok = mbar_wait(&c_tfull[acc], (it >> 1) & 1, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tcgen05_fence_after();
      if (t.seg_last()) mbar_arrive(seg_done);
      const uint32_t trow = tmem_base + acc * kAccStride + ((uint32_t)(wq * 32) << 16);
      uint8_t* sl = slots + s * SLOT;
      float rinv[C::G];
      if (ROPE) {
        // the ReLU warps left phi(q) . z of this row in the row's padding
        if (D == 112) {
          rinv[0] = 1.0f / (*reinterpret_cast<const float*>(sl + HALF + r * kRowBytes + ((6 ^ (r & 7)) << 4)) + p.eps);
        } else {
#pragma unroll
          for (int g = 0; g < C::G; ++g) rinv[g] = 1.0f / (den_rows[(s * C::G + g) * kTileApply + r] + p.eps);
        }
      } else {
        uint32_t dn[4];
        tmem_ld_x4(trow + C::ZROW, dn);
        tmem_ld_wait();
#pragma unroll
        for (int g = 0; g < C::G; ++g) rinv[g] = 1.0f / (__uint_as_float(dn[g]) + p.eps);  // eps added once, after the dot product
      }
#pragma unroll
      for (int cc = 0; cc < 4; ++cc) {
        if (cc * 32 >= C::FEAT) break;
        uint32_t v[32];
        tmem_ld_x32(trow + cc * 32, v);
        tmem_ld_wait();
        if (cc == 3 || (cc + 1) * 32 >= C::FEAT) {  // last read of this accumulator: hand it back to the MMA warp
          tcgen05_fence_before();
          mbar_arrive(&c_tempty[acc]);
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
      mbar_arrive(&c_staged[s]);
    }
  } else {
    // ------------------------------------------------------------ store warp: O tiles out, slots back to the producer
    if (lane == 0) {
      uint32_t it = 0;
      // A head row that is not a whole number of 128-byte lines (d = 112) shares lines with its neighbours,
      // and each head's part of such a line arrives from another SM: the O tiles are stored with the L2
      // evict-last policy so that a line is still there when its other part comes, and goes to DRAM once,
      // whole (measured: 5 % on the forward; evict-first on the K, V loads helped the state pass alone but
      // not the forward, on the Q loads it brought the over-fetch of shared lines back).
      constexpr bool kKeepStores = (C::FEAT * 2) % 128 != 0;
      const uint64_t store_policy = kKeepStores ? make_l2_policy_evict_last() : 0;
      for (TileWalk t(wc); !t.done(); t.next(), ++it) {
        const int s = it % NSC;
        if (!mbar_wait(&c_staged[s], (it / NSC) & 1, abort_flag)) break;
        const int u = t.unit(), b = u / p.HG, hg = u % p.HG;
        uint8_t* sl = slots + s * SLOT;
        int c0, c1;
        box_coords<D>(0, hg, c0, c1);
        if (kKeepStores) {
          tma_store_4d_hint(&map_o, sl, c0, c1, t.tile() * kTileApply, b, store_policy);
          box_coords<D>(1, hg, c0, c1);
          tma_store_4d_hint(&map_o, sl + HALF, c0, c1, t.tile() * kTileApply, b, store_policy);
        } else {
          tma_store_4d(&map_o, sl, c0, c1, t.tile() * kTileApply, b);
          box_coords<D>(1, hg, c0, c1);
          tma_store_4d(&map_o, sl + HALF, c0, c1, t.tile() * kTileApply, b);
        }
        tma_store_commit();
        tma_store_wait_read();
        mbar_arrive(&c_empty[s]);
      }
      tma_store_wait_all();
    }
  }

  // ------------------------------------------------------------ teardown
  tcgen05_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (threadIdx.x == 0) {
      p.ctrl->status = LINATTN_ERR_TIMEOUT;
      // loads still in flight target this CTA's shared memory: give each stage a bounded wait
      for (int s = 0; s < NSA + NSC; ++s)
        for (int par = 0; par < 2; ++par)
          for (int spin = 0; spin < 4096 && !mbar_try_wait(s < NSA ? &a_full[s] : &c_full[s - NSA], par); ++spin)
            __nanosleep(64);
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
  if (p.d == 32) {
    // A 64-byte box row would be padded to the 128-byte swizzle pitch, so with d = 32 (heads contiguous:
    // stride_h = 32) the heads of a token are one row of H*32 features and a box takes 64 of them (two heads).
    dims[0] = (cuuint64_t)p.H * 32; dims[1] = 1;
    strides[0] = (cuuint64_t)p.sn * 2;
  }
  cuuint32_t box[4] = {(cuuint32_t)box_d, (cuuint32_t)box_h, (cuuint32_t)box_tokens, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// SM count of the current device (0: not an sm_100 device, or no cooperative launch).
int sm_count() {
  static int cached[64] = {0};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
  if (!cached[dev]) {
    int n = 0, major = 0, coop = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess || major != 10) return 0;
    if (cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess || !coop) return 0;
    cached[dev] = n > kMaxCtas ? kMaxCtas : n;
  }
  return cached[dev];
}

inline int groups_of(int d) { return d == 32 ? 4 : d == 64 ? 2 : 1; }

template <int D, bool ROPE>
int launch_fused(const Problem& p, const UmmaCall& c, void* workspace, cudaStream_t stream) {
  using C = Cfg<D>;
  const int sms = sm_count();
  if (!sms) return LINATTN_ERR_CUDA;
  const bool do_state = c.k != nullptr, do_apply = c.q != nullptr;
  FusedParams fp{};
  fp.B = p.B; fp.H = p.H; fp.HG = (p.H + C::G - 1) / C::G;
  const int U = p.B * fp.HG;
  fp.sa = make_sched(U, (p.N + kTileState - 1) / kTileState, sms, 2);
  fp.do_state = do_state; fp.do_apply = do_apply; fp.accumulate = c.accumulate ? 1 : 0;
  fp.state = c.state;
  fp.state_base = c.state_base ? c.state_base : c.state;
  fp.partials = reinterpret_cast<float*>(static_cast<char*>(workspace) + LINATTN_WORKSPACE_CTRL_BYTES);
  fp.eps = c.eps;
  fp.ctrl = static_cast<WorkspaceCtrl*>(workspace);
  fp.rope = static_cast<const uint4*>(c.rope);
  fp.N = p.N;
  fp.s_image = nullptr;
  if (do_state && do_apply && C::G == 1 && fp.sa.P >= 1) {
    // The operand images live at the end of the partials area, which is sized for kMaxCtas + U records while a
    // launch writes at most P*U + R + U of them: used when they fit behind the records in use.
    const size_t rec_bytes = ((size_t)p.state_elems() + (ROPE ? kZParts : 0)) * sizeof(float);
    const size_t used = ((size_t)fp.sa.P * U + fp.sa.R + U) * rec_bytes;
    const size_t total = umma_partial_bytes(p, ROPE), img = (size_t)U * C::S_BYTES;
    if (total >= img + 1024) {
      const size_t off = (total - img) & ~(size_t)1023;
      if (off >= used) fp.s_image = reinterpret_cast<uint8_t*>(fp.partials) + off;
    }
  }
  // a unit switch costs the apply pass about one tile when the S operand comes as an image, two when the CTA
  // builds it from the fp32 state
  fp.sc = make_sched(U, (p.N + kTileApply - 1) / kTileApply, sms, fp.s_image ? 1 : 2);
  int grid = 0;
  if (do_state) grid = fp.sa.grid;
  if (do_apply && fp.sc.grid > grid) grid = fp.sc.grid;
  CUtensorMap mk, mv, mq, mo;
  if (do_state) {
    if (!make_map(&mk, p, c.k, C::BOX_D, C::BOX_H, kTileState) || !make_map(&mv, p, c.v, C::BOX_D, C::BOX_H, kTileState))
      return LINATTN_ERR_CUDA;
  }
  if (do_apply) {
    if (!make_map(&mq, p, c.q, C::BOX_D, C::BOX_H, kTileApply) || !make_map(&mo, p, c.o, C::BOX_D, C::BOX_H, kTileApply))
      return LINATTN_ERR_CUDA;
  } else {
    mq = mk; mo = mk;  // never dereferenced
  }
  if (!do_state) { mk = mq; mv = mq; }
  // the opt-in to more than 48 KB of dynamic shared memory is a per-device setting of the kernel
  static bool attr_set[64] = {false};
  constexpr size_t kSmem = ROPE ? C::SMEM_ROPE : C::SMEM;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return LINATTN_ERR_CUDA;
  if (!attr_set[dev]) {
    if (cudaFuncSetAttribute(umma_fused_kernel<D, ROPE>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmem) !=
        cudaSuccess)
      return LINATTN_ERR_CUDA;
    attr_set[dev] = true;
  }
  void* args[] = {&mk, &mv, &mq, &mo, &fp};
  const cudaError_t e = cudaLaunchCooperativeKernel((const void*)umma_fused_kernel<D, ROPE>, dim3(grid), dim3(Roles<ROPE>::THREADS), args,
                                                    kSmem, stream);
  if (e != cudaSuccess) { cudaGetLastError(); return LINATTN_ERR_CUDA; }
  count_launches(1);
  return LINATTN_OK;
}

}  // namespace

bool umma_supported(const Problem& p) {
  // d = 32 packs four heads into one operand row, which needs the heads of a token to be contiguous
  return p.dtype == LINATTN_BF16 && (p.d == 64 || p.d == 112 || p.d == 128 || (p.d == 32 && p.sh == 32)) &&
         p.N < (1ll << 31) && p.sh * 2 < (1ll << 40) && p.sn * 2 < (1ll << 40) && p.sb * 2 < (1ll << 40);
}

// One partial record (G head-states) per (CTA, unit) segment of the state pass: at most kMaxCtas + units.
size_t umma_partial_bytes(const Problem& p, bool rope) {
  const int G = groups_of(p.d);
  const size_t units = (size_t)p.B * ((p.H + G - 1) / G);
  return ((size_t)kMaxCtas + units) * (G * (size_t)p.state_elems() + (rope ? kZParts : 0)) * sizeof(float);
}

// The rotary variant runs on the tensor cores wherever the plain kernel does.  d = 112, the paper's: the denominators
// travel in the zero padding of the 112-feature rows; every other head dim: in a small shared-memory array per slot
// and head of the group.  With packed heads (d = 32, 64) both boxes of a row use the same 16-byte chunk of the
// rotation table, since box 1 starts a new head.  Everything else takes the FMA kernels.
bool umma_rope_supported(const Problem& p) { return umma_supported(p); }

int umma_run(const Problem& p, const UmmaCall& c, void* workspace, cudaStream_t stream) {
  if (p.N == 0 || (!c.k && !c.q)) return LINATTN_OK;
  switch (p.d) {
    case 32: return c.rope ? launch_fused<32, true>(p, c, workspace, stream) : launch_fused<32, false>(p, c, workspace, stream);
    case 64: return c.rope ? launch_fused<64, true>(p, c, workspace, stream) : launch_fused<64, false>(p, c, workspace, stream);
    case 112: return c.rope ? launch_fused<112, true>(p, c, workspace, stream) : launch_fused<112, false>(p, c, workspace, stream);
    case 128: return c.rope ? launch_fused<128, true>(p, c, workspace, stream) : launch_fused<128, false>(p, c, workspace, stream);
  }
  return LINATTN_ERR_UNSUPPORTED;
}

}  // namespace linattn
