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
};
bool umma_supported(const Problem& p);
size_t umma_partial_bytes(const Problem& p, bool rope = false);
bool umma_rope_supported(const Problem& p);
// Returns LINATTN_OK or an error status.
int umma_run(const Problem& p, const UmmaCall& call, void* workspace, cudaStream_t stream);

}  // namespace linattn
