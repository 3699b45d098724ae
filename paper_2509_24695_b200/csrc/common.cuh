// Internal declarations shared by the library's translation units (not part of the C ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "linattn.h"

namespace linattn {

// A descriptor with its strides resolved for one call.
struct Problem {
  int B, H, d;
  int dtype;
  long long sb, sn, sh;  // element strides of (batch, token, head); the feature axis is contiguous
  long long N;           // tokens in this call
  __host__ __device__ int units() const { return B * H; }
  __host__ __device__ long long state_elems() const { return (long long)(d + 1) * d; }  // floats per (b,h) state
};

// Control block at the start of every workspace.
struct WorkspaceCtrl {
  int status;            // LINATTN_OK or LINATTN_ERR_TIMEOUT, written by kernels
  int pad0[15];
  unsigned barrier[16];  // grid-barrier counters of the fused kernels
  unsigned unit_arrivals[960];
};
static_assert(sizeof(WorkspaceCtrl) <= LINATTN_WORKSPACE_CTRL_BYTES, "control block too large");

struct Rope3dLayout;   // defined below, with the rotary declarations

// Kernel-launch counter behind linattn_kernel_launches().
void count_launches(int n);

constexpr int kMaxCtas = 256;        // upper bound on the persistent grid (B200 has 148 SMs)
constexpr int kFmaMaxChunks = 64;    // split-N partials per unit on the FMA path
constexpr int kFmaMinChunkTokens = 512;

inline int fma_chunks(long long N) {
  long long p = (N + kFmaMinChunkTokens - 1) / kFmaMinChunkTokens;
  if (p < 1) p = 1;
  return p > kFmaMaxChunks ? kFmaMaxChunks : (int)p;
}

// ---- FMA kernels (fp32 I/O path, and bf16 shapes the tensor-core kernels do not take) ----
// state_out = (accumulate ? state_out : 0) + state of tokens [0, N); partials is scratch.
// rope: Eq. 2 with its rotary factors, table [N][d/2] of (cos, sin) fp16 pairs, one per pair rotation.
cudaError_t fma_state(const Problem& p, const void* k, const void* v, float* state_out, bool accumulate,
                      float* partials, cudaStream_t stream, const __half2* rope = nullptr);
cudaError_t fma_apply(const Problem& p, const void* q, const float* state, void* o, float eps, cudaStream_t stream,
                      const __half2* rope = nullptr);
// blk: [B][M][H][(d+1)*d] per-block states -> running states after each block (on top of cache [B][H][..]), cache := last.
cudaError_t prefix_states(float* blk, float* cache, int B, int M, long long floats_per_batch, cudaStream_t stream);
cudaError_t rope_pack(const float* cs, const float* sn, long long count, __half2* out, cudaStream_t stream);
// per-axis tables: cs[a], sn[a] are [positions][pairs of axis a] fp32 device arrays
cudaError_t rope3d_pack(const Rope3dLayout& lay, const float* const cs[3], const float* const sn[3], void* table,
                        cudaStream_t stream);

// ---- tensor-core (tcgen05 + TMA) kernel, bf16, d in {32 (heads contiguous), 64, 112, 128} ----
// One launch runs the state pass (k, v non-null), the apply pass (q, o non-null), or both back to back.
struct UmmaCall {
  const void* k;
  const void* v;
  const void* q;
  void* o;
  float* state;     // written by the state pass, read by the apply pass
  const float* state_base;  // `accumulate`: the reduce adds the new state to this one (may be `state` itself)
  bool accumulate;
  float eps;
  const void* rope;  // rotary variant (Eq. 2 with its rotary factors): packed (cos, sin) fp16 table [N][d/2]; else null
  const struct Rope3dHost* rope3d = nullptr;  // rotary variant with per-axis tables (3D RoPE); else null
};

// Rotary factors given per axis of the latent grid (see linattn_rope3d in linattn.h).
struct Rope3dHost {
  int T, Hh, Ww, pt, ph, pw;
  const void* table;        // packed by linattn_rope3d_pack
  long long token_offset;   // grid index of the call's first token
};

// Layout of the packed per-axis table: axis a (0 frame, 1 row, 2 column) owns the feature pairs [start, start + pairs);
// its sub-table holds, per position, the 16-byte chunks (four pairs each) clo .. clo + nch - 1 that touch that range.
struct Rope3dLayout {
  unsigned base[3], nch[3], clo[3], start[3], count[3], positions[3];
  size_t bytes;
};
inline bool rope3d_layout(int T, int Hh, int Ww, int pt, int ph, int pw, int d, Rope3dLayout* out) {
  if (T < 1 || Hh < 1 || Ww < 1 || pt < 0 || ph < 0 || pw < 0 || (d & 1) || pt + ph + pw != d / 2) return false;
  if ((long long)T * Hh * Ww >= (1ll << 31)) return false;
  const int pairs[3] = {pt, ph, pw}, pos[3] = {T, Hh, Ww};
  int start = 0;
  size_t off = 0;
  for (int a = 0; a < 3; ++a) {
    out->start[a] = (unsigned)start; out->count[a] = (unsigned)pairs[a]; out->positions[a] = (unsigned)pos[a];
    out->clo[a] = (unsigned)(start / 4);
    out->nch[a] = pairs[a] > 0 ? (unsigned)((start + pairs[a] - 1) / 4 - start / 4 + 1) : 0u;
    out->base[a] = (unsigned)off;
    off += (size_t)pos[a] * out->nch[a] * 16;
    start += pairs[a];
  }
  // at most two axes may meet in one chunk of four pairs (the kernel reads at most two sub-tables per chunk)
  for (int c = 0; c * 4 < d / 2; ++c) {
    bool seen[3] = {false, false, false};
    for (int pair = c * 4; pair < c * 4 + 4 && pair < d / 2; ++pair) seen[pair < pt ? 0 : pair < pt + ph ? 1 : 2] = true;
    if (seen[0] && seen[1] && seen[2]) return false;
  }
  if (off >= (1ull << 31)) return false;
  out->bytes = off > 0 ? off : 16;
  return true;
}
bool umma_supported(const Problem& p);
size_t umma_partial_bytes(const Problem& p, bool rope = false);
bool umma_rope_supported(const Problem& p);
// Returns LINATTN_OK or an error status.
int umma_run(const Problem& p, const UmmaCall& call, void* workspace, cudaStream_t stream);

}  // namespace linattn
