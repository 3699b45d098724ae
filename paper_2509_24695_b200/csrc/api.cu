// C ABI of the linear-attention library: argument validation, workspace layout, kernel selection
// and the host-side cache handle.  See include/linattn.h for the contract of each entry point.
#include <atomic>
#include <new>

#include "common.cuh"

using namespace linattn;

namespace linattn {
static std::atomic<uint64_t> g_kernel_launches{0};
void count_launches(int n) { g_kernel_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }
}  // namespace linattn

namespace {

constexpr uint32_t kCacheMagic = 0x4C41434Bu;  // "LACK"

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Validates a descriptor and resolves its strides for N tokens.
int resolve(const linattn_desc* desc, long long N, Problem* out) {
  if (!desc || N < 0) return LINATTN_ERR_INVALID_ARG;
  if (desc->B < 1 || desc->H < 1 || desc->d < 1) return LINATTN_ERR_INVALID_ARG;
  if (desc->dtype != LINATTN_BF16 && desc->dtype != LINATTN_F32) return LINATTN_ERR_INVALID_ARG;
  if (desc->stride_b < 0 || desc->stride_n < 0 || desc->stride_h < 0) return LINATTN_ERR_INVALID_ARG;
  if (desc->d > 128) return LINATTN_ERR_UNSUPPORTED;
  if ((long long)desc->B * desc->H > 65535) return LINATTN_ERR_UNSUPPORTED;
  Problem p;
  p.B = desc->B; p.H = desc->H; p.d = desc->d; p.dtype = desc->dtype; p.N = N;
  p.sh = desc->stride_h ? desc->stride_h : desc->d;
  p.sn = desc->stride_n ? desc->stride_n : (long long)desc->H * desc->d;
  p.sb = desc->stride_b ? desc->stride_b : (long long)N * desc->H * desc->d;
  if (p.sh < p.d) return LINATTN_ERR_INVALID_ARG;
  *out = p;
  return LINATTN_OK;
}

// Alignment rule of the header: 16-byte pointers, strides multiples of 16 bytes.  Enforced for the
// shapes the tensor-core kernels take (their TMA descriptors need it); the FMA kernels use scalar
// accesses and only need natural alignment.
int check_alignment(const Problem& p, const void* a, const void* b, const void* c, const void* d) {
  if (!umma_supported(p)) return LINATTN_OK;
  const void* ptrs[4] = {a, b, c, d};
  for (const void* x : ptrs)
    if (x && !aligned16(x)) return LINATTN_ERR_BAD_ALIGNMENT;
  if ((p.sb % 8) || (p.sn % 8) || (p.sh % 8)) return LINATTN_ERR_BAD_ALIGNMENT;
  return LINATTN_OK;
}

size_t partial_bytes(const Problem& p) {
  if (umma_supported(p)) return umma_partial_bytes(p);
  return sizeof(float) * (size_t)p.state_elems() * p.units() * fma_chunks(p.N);
}

inline size_t round256(size_t b) { return (b + 255) & ~(size_t)255; }

inline size_t state_bytes_of(const Problem& p) { return sizeof(float) * (size_t)p.state_elems() * p.units(); }

// Workspace layout: [control block][split-N partials][one state, used by linattn_forward].
size_t state_slot_offset(const Problem& p) { return round256(LINATTN_WORKSPACE_CTRL_BYTES + partial_bytes(p)); }

size_t workspace_need(const Problem& p) { return round256(state_slot_offset(p) + state_bytes_of(p)); }

inline float* partials_of(void* workspace) {
  return reinterpret_cast<float*>(static_cast<char*>(workspace) + LINATTN_WORKSPACE_CTRL_BYTES);
}

int cuda_status(cudaError_t e) { return e == cudaSuccess ? LINATTN_OK : LINATTN_ERR_CUDA; }

// state = (accumulate ? base : 0) + state(k, v), then (q non-null) o = apply(q, state).  `base` is the
// state that is added to; null means `state` itself (in place).  On the tensor-core path everything
// runs in one launch.
int run_passes(const Problem& p, const void* k, const void* v, const void* q, void* o, float* state, bool accumulate,
               float eps, void* workspace, cudaStream_t stream, const float* base = nullptr) {
  if (umma_supported(p)) {
    UmmaCall c{k, v, q, o, state, base, accumulate, eps, nullptr};
    return umma_run(p, c, workspace, stream);
  }
  if (k && accumulate && base && base != state) {
    if (cudaMemcpyAsync(state, base, state_bytes_of(p), cudaMemcpyDeviceToDevice, stream) != cudaSuccess)
      return LINATTN_ERR_CUDA;
  }
  if (k) {
    int st = cuda_status(fma_state(p, k, v, state, accumulate, partials_of(workspace), stream));
    if (st != LINATTN_OK) return st;
  }
  if (q) return cuda_status(fma_apply(p, q, state, o, eps, stream));
  return LINATTN_OK;
}

// Workspace of the rotary entry point: [control block][split-N partials][one state].
size_t rope_partial_bytes(const Problem& p) {
  if (umma_rope_supported(p)) return umma_partial_bytes(p, true);
  return sizeof(float) * (size_t)p.state_elems() * p.units() * fma_chunks(p.N);
}
size_t rope_state_offset(const Problem& p) { return round256(LINATTN_WORKSPACE_CTRL_BYTES + rope_partial_bytes(p)); }
size_t rope_workspace_need(const Problem& p) { return round256(rope_state_offset(p) + state_bytes_of(p)); }

// Eq. 2 with its rotary factors: state from the rotated keys (z from the plain ones), apply with the rotated
// queries (denominator from the plain ones).
// `base` as in run_passes: the state that is added to (null: `state` itself); q may be null (state only).
int run_rope(const Problem& p, const void* q, const void* k, const void* v, void* o, float* state, bool accumulate,
             float eps, const __half2* rope, void* workspace, cudaStream_t stream, const float* base = nullptr) {
  if (umma_rope_supported(p)) {  // one launch on the tensor cores
    UmmaCall c{k, v, q, o, state, base, accumulate, eps, rope};
    return umma_run(p, c, workspace, stream);
  }
  if (accumulate && base && base != state) {
    if (cudaMemcpyAsync(state, base, state_bytes_of(p), cudaMemcpyDeviceToDevice, stream) != cudaSuccess)
      return LINATTN_ERR_CUDA;
  }
  int st = cuda_status(fma_state(p, k, v, state, accumulate, partials_of(workspace), stream, rope));
  if (st != LINATTN_OK || !q) return st;
  return cuda_status(fma_apply(p, q, state, o, eps, stream, rope));
}

}  // namespace

// Scratch of linattn_state_static_scratch: part of the library image, so no call has to allocate it.
// In host code this name is only a handle for the runtime; the device address comes from
// cudaGetSymbolAddress, once per device.
static __device__ __align__(256) unsigned char g_static_scratch[LINATTN_STATIC_SCRATCH_BYTES];

static void* static_scratch_address() {
  static void* cached[64] = {nullptr};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  if (!cached[dev]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess) {
      cudaGetLastError();
      return nullptr;
    }
    cached[dev] = ptr;
  }
  return cached[dev];
}

// Host-side plumbing of linattn_forward_host: a second stream for the downloads and the events that
// order it against the caller's stream (no device memory), created once per device.
constexpr int kHostChunks = 8;
struct HostPipe {
  cudaStream_t down;
  cudaEvent_t chunk_done[kHostChunks + 1];
  cudaEvent_t all_down;
};
static HostPipe* host_pipe() {
  static HostPipe pipes[64];
  static bool ready[64] = {false};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  if (!ready[dev]) {
    HostPipe& hp = pipes[dev];
    if (cudaStreamCreateWithFlags(&hp.down, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
    for (cudaEvent_t& ev : hp.chunk_done)
      if (cudaEventCreateWithFlags(&ev, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    if (cudaEventCreateWithFlags(&hp.all_down, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    ready[dev] = true;
  }
  return &pipes[dev];
}

struct blocklin_cache {
  uint32_t magic;
  linattn_desc desc;
  float eps;
  float* state;
  size_t state_bytes;
  void* workspace;
  size_t workspace_bytes;
  long long blocks_seen;
  long long tokens_seen;
  int joint_prefill;   // blocklin_prefill may take all blocks together (asked for: it changes the low bits)
};

// One block: commit (cache += (S_blk, z_blk)), then read (the block's queries see the updated cache).
static int step_impl(blocklin_cache* cache, const Problem& p, const void* q_blk, const void* k_blk,
                     const void* v_blk, void* o_blk, cudaStream_t stream) {
  if ((q_blk == nullptr) != (o_blk == nullptr)) return LINATTN_ERR_INVALID_ARG;
  if (p.N > 0 && (!k_blk || !v_blk)) return LINATTN_ERR_INVALID_ARG;
  if (o_blk && (o_blk == q_blk || o_blk == k_blk || o_blk == v_blk)) return LINATTN_ERR_INVALID_ARG;
  int st = check_alignment(p, q_blk, k_blk, v_blk, o_blk);
  if (st != LINATTN_OK) return st;
  if (cache->workspace_bytes < workspace_need(p)) return LINATTN_ERR_WORKSPACE_TOO_SMALL;
  if (p.N == 0) return LINATTN_OK;
  st = run_passes(p, k_blk, v_blk, q_blk, o_blk, cache->state, true, cache->eps, cache->workspace, stream);
  if (st != LINATTN_OK) return st;
  cache->blocks_seen += 1;
  cache->tokens_seen += p.N;
  return LINATTN_OK;
}

// One block with the rotary factors of Eq. 2.  commit: the cache takes the block (blocklin_step_rope); otherwise the
// sum of cache and block goes to the state slot of the workspace and the cache is only read (blocklin_peek_rope).
static int step_rope_impl(blocklin_cache* cache, const Problem& p, const void* q_blk, const void* k_blk,
                          const void* v_blk, void* o_blk, const void* rope_table_blk, bool commit, cudaStream_t stream) {
  if (p.d & 1) return LINATTN_ERR_UNSUPPORTED;
  if ((q_blk == nullptr) != (o_blk == nullptr)) return LINATTN_ERR_INVALID_ARG;
  if (p.N > 0 && (!k_blk || !v_blk || !rope_table_blk)) return LINATTN_ERR_INVALID_ARG;
  if (o_blk && (o_blk == q_blk || o_blk == k_blk || o_blk == v_blk)) return LINATTN_ERR_INVALID_ARG;
  int st = check_alignment(p, q_blk, k_blk, v_blk, o_blk);
  if (st != LINATTN_OK) return st;
  // the tensor-core kernel fetches the rotations in 16-byte chunks; the FMA kernels pair by pair
  if (reinterpret_cast<uintptr_t>(rope_table_blk) & (umma_rope_supported(p) ? 15u : 3u)) return LINATTN_ERR_BAD_ALIGNMENT;
  if (cache->workspace_bytes < rope_workspace_need(p)) return LINATTN_ERR_WORKSPACE_TOO_SMALL;
  if (p.N == 0) return LINATTN_OK;
  const __half2* rope = static_cast<const __half2*>(rope_table_blk);
  if (!commit) {
    float* tmp = reinterpret_cast<float*>(static_cast<char*>(cache->workspace) + rope_state_offset(p));
    return run_rope(p, q_blk, k_blk, v_blk, o_blk, tmp, true, cache->eps, rope, cache->workspace, stream, cache->state);
  }
  st = run_rope(p, q_blk, k_blk, v_blk, o_blk, cache->state, true, cache->eps, rope, cache->workspace, stream);
  if (st != LINATTN_OK) return st;
  cache->blocks_seen += 1;
  cache->tokens_seen += p.N;
  return LINATTN_OK;
}

extern "C" {

const char* linattn_status_string(int status) {
  switch (status) {
    case LINATTN_OK: return "ok";
    case LINATTN_ERR_INVALID_ARG: return "invalid argument";
    case LINATTN_ERR_UNSUPPORTED: return "unsupported shape or layout";
    case LINATTN_ERR_BAD_ALIGNMENT: return "pointer or stride not 16-byte aligned";
    case LINATTN_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case LINATTN_ERR_CUDA: return "CUDA call failed";
    case LINATTN_ERR_TIMEOUT: return "bounded device-side wait expired";
    case LINATTN_ERR_BAD_HANDLE: return "bad cache handle";
    case LINATTN_ERR_SCRATCH_LIMIT: return "problem exceeds the built-in scratch of linattn_state_static_scratch";
    default: return "unknown status";
  }
}

int linattn_state_bytes(const linattn_desc* desc, size_t* bytes) {
  Problem p;
  if (!bytes) return LINATTN_ERR_INVALID_ARG;
  int st = resolve(desc, 0, &p);
  if (st != LINATTN_OK) return st;
  *bytes = sizeof(float) * (size_t)p.state_elems() * p.units();
  return LINATTN_OK;
}

int linattn_workspace_bytes(const linattn_desc* desc, int64_t N, size_t* bytes) {
  Problem p;
  if (!bytes) return LINATTN_ERR_INVALID_ARG;
  int st = resolve(desc, N, &p);
  if (st != LINATTN_OK) return st;
  *bytes = workspace_need(p);
  return LINATTN_OK;
}

int linattn_workspace_init(void* workspace, size_t workspace_bytes, void* stream) {
  if (!workspace || workspace_bytes < LINATTN_WORKSPACE_CTRL_BYTES) return LINATTN_ERR_INVALID_ARG;
  return cuda_status(cudaMemsetAsync(workspace, 0, LINATTN_WORKSPACE_CTRL_BYTES, (cudaStream_t)stream));
}

int linattn_workspace_status(const void* workspace, void* stream, int* status) {
  if (!workspace || !status) return LINATTN_ERR_INVALID_ARG;
  int word = 0;
  cudaError_t e = cudaMemcpyAsync(&word, workspace, sizeof(int), cudaMemcpyDeviceToHost, (cudaStream_t)stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize((cudaStream_t)stream);
  if (e != cudaSuccess) return LINATTN_ERR_CUDA;
  *status = word;
  return LINATTN_OK;
}

int linattn_state(const linattn_desc* desc, int64_t N, const void* k, const void* v, float* state, void* workspace,
                  size_t workspace_bytes, void* stream) {
  Problem p;
  int st = resolve(desc, N, &p);
  if (st != LINATTN_OK) return st;
  if (!state || !workspace) return LINATTN_ERR_INVALID_ARG;
  if (N > 0 && (!k || !v)) return LINATTN_ERR_INVALID_ARG;
  if ((st = check_alignment(p, k, v, state, workspace)) != LINATTN_OK) return st;
  if (workspace_bytes < workspace_need(p)) return LINATTN_ERR_WORKSPACE_TOO_SMALL;
  if (N == 0) return cuda_status(cudaMemsetAsync(state, 0, state_bytes_of(p), (cudaStream_t)stream));  // empty sum
  return run_passes(p, k, v, nullptr, nullptr, state, false, 0.f, workspace, (cudaStream_t)stream);
}

int linattn_state_static_scratch(const linattn_desc* desc, int64_t N, const void* k, const void* v, float* state,
                                 void* stream) {
  Problem p;
  int st = resolve(desc, N, &p);
  if (st != LINATTN_OK) return st;
  if (!state) return LINATTN_ERR_INVALID_ARG;
  if (N > 0 && (!k || !v)) return LINATTN_ERR_INVALID_ARG;
  if ((st = check_alignment(p, k, v, state, nullptr)) != LINATTN_OK) return st;
  // control block + split-N partials; the state slot that linattn_forward keeps behind them is not needed
  if (state_slot_offset(p) > sizeof(g_static_scratch)) return LINATTN_ERR_SCRATCH_LIMIT;
  void* scratch = static_scratch_address();
  if (!scratch) return LINATTN_ERR_CUDA;
  if (N == 0) return cuda_status(cudaMemsetAsync(state, 0, state_bytes_of(p), (cudaStream_t)stream));  // empty sum
  // the array keeps the last call's contents: the barrier word and the status word must start at zero
  if (cudaMemsetAsync(scratch, 0, LINATTN_WORKSPACE_CTRL_BYTES, (cudaStream_t)stream) != cudaSuccess)
    return LINATTN_ERR_CUDA;
  return run_passes(p, k, v, nullptr, nullptr, state, false, 0.f, scratch, (cudaStream_t)stream);
}

int linattn_static_scratch_status(void* stream, int* status) {
  if (!status) return LINATTN_ERR_INVALID_ARG;
  void* scratch = static_scratch_address();
  if (!scratch) return LINATTN_ERR_CUDA;
  return linattn_workspace_status(scratch, stream, status);
}

int linattn_apply(const linattn_desc* desc, int64_t N, const void* q, const float* state, void* o, float eps,
                  void* workspace, size_t workspace_bytes, void* stream) {
  Problem p;
  int st = resolve(desc, N, &p);
  if (st != LINATTN_OK) return st;
  if (!state || !workspace) return LINATTN_ERR_INVALID_ARG;
  if (N > 0 && (!q || !o || q == o)) return LINATTN_ERR_INVALID_ARG;
  if ((st = check_alignment(p, q, o, state, workspace)) != LINATTN_OK) return st;
  if (workspace_bytes < LINATTN_WORKSPACE_CTRL_BYTES) return LINATTN_ERR_WORKSPACE_TOO_SMALL;
  if (N == 0) return LINATTN_OK;
  return run_passes(p, nullptr, nullptr, q, o, const_cast<float*>(state), false, eps, workspace, (cudaStream_t)stream);
}

int linattn_forward(const linattn_desc* desc, int64_t N, const void* q, const void* k, const void* v, void* o,
                    float eps, void* workspace, size_t workspace_bytes, void* stream) {
  Problem p;
  int st = resolve(desc, N, &p);
  if (st != LINATTN_OK) return st;
  if (!workspace) return LINATTN_ERR_INVALID_ARG;
  if (N > 0 && (!q || !k || !v || !o || o == q || o == k || o == v)) return LINATTN_ERR_INVALID_ARG;
  if ((st = check_alignment(p, q, k, v, o)) != LINATTN_OK) return st;
  if (!aligned16(workspace)) return LINATTN_ERR_BAD_ALIGNMENT;
  if (workspace_bytes < workspace_need(p)) return LINATTN_ERR_WORKSPACE_TOO_SMALL;
  if (N == 0) return LINATTN_OK;
  // the forward keeps its reduced state in the workspace, after the partials
  float* state = reinterpret_cast<float*>(static_cast<char*>(workspace) + state_slot_offset(p));
  return run_passes(p, k, v, q, o, state, false, eps, workspace, (cudaStream_t)stream);
}

int linattn_rope_workspace_bytes(const linattn_desc* desc, int64_t N, size_t* bytes) {
  Problem p;
  if (!bytes) return LINATTN_ERR_INVALID_ARG;
  int st = resolve(desc, N, &p);
  if (st != LINATTN_OK) return st;
  *bytes = rope_workspace_need(p);
  return LINATTN_OK;
}

int linattn_rope_table_bytes(int64_t N, int32_t d, size_t* bytes) {
  if (!bytes || N < 0 || d < 2) return LINATTN_ERR_INVALID_ARG;
  if (d & 1) return LINATTN_ERR_UNSUPPORTED;
  *bytes = (size_t)N * (size_t)(d / 2) * sizeof(__half2);
  return LINATTN_OK;
}

int linattn_rope_pack(int64_t N, int32_t d, const float* rope_cos, const float* rope_sin, void* table, void* stream) {
  if (N < 0 || d < 2) return LINATTN_ERR_INVALID_ARG;
  if (d & 1) return LINATTN_ERR_UNSUPPORTED;
  if (N > 0 && (!rope_cos || !rope_sin || !table)) return LINATTN_ERR_INVALID_ARG;
  if (!aligned16(table)) return LINATTN_ERR_BAD_ALIGNMENT;
  return cuda_status(rope_pack(rope_cos, rope_sin, (long long)N * (d / 2), static_cast<__half2*>(table), (cudaStream_t)stream));
}

int linattn_forward_rope(const linattn_desc* desc, int64_t N, const void* q, const void* k, const void* v, void* o,
                         float eps, const void* rope_table, void* workspace, size_t workspace_bytes, void* stream) {
  Problem p;
  int st = resolve(desc, N, &p);
  if (st != LINATTN_OK) return st;
  if (!workspace) return LINATTN_ERR_INVALID_ARG;
  if (p.d & 1) return LINATTN_ERR_UNSUPPORTED;  // the rotation pairs features (2p, 2p+1)
  if (N > 0 && (!q || !k || !v || !o || !rope_table || o == q || o == k || o == v))
    return LINATTN_ERR_INVALID_ARG;
  if ((st = check_alignment(p, q, k, v, o)) != LINATTN_OK) return st;
  if (!aligned16(workspace) || !aligned16(rope_table)) return LINATTN_ERR_BAD_ALIGNMENT;
  if (workspace_bytes < rope_workspace_need(p)) return LINATTN_ERR_WORKSPACE_TOO_SMALL;
  if (N == 0) return LINATTN_OK;
  float* state = reinterpret_cast<float*>(static_cast<char*>(workspace) + rope_state_offset(p));
  return run_rope(p, q, k, v, o, state, false, eps, static_cast<const __half2*>(rope_table), workspace, (cudaStream_t)stream);
}

uint64_t linattn_kernel_launches(void) { return g_kernel_launches.load(std::memory_order_relaxed); }

int linattn_forward_host_bytes(const linattn_desc* desc, int64_t N, size_t* bytes) {
  Problem p;
  if (!bytes) return LINATTN_ERR_INVALID_ARG;
  int st = resolve(desc, N, &p);
  if (st != LINATTN_OK) return st;
  if (desc->stride_b || desc->stride_n || desc->stride_h) return LINATTN_ERR_UNSUPPORTED;
  const size_t esz = p.dtype == LINATTN_BF16 ? 2 : 4;
  const size_t tensor = round256((size_t)p.B * (size_t)N * p.H * p.d * esz);
  *bytes = workspace_need(p) + 4 * tensor;
  return LINATTN_OK;
}

int linattn_forward_host(const linattn_desc* desc, int64_t N, const void* q_host, const void* k_host,
                         const void* v_host, void* o_host, float eps, void* dev_staging, size_t dev_staging_bytes,
                         void* stream) {
  size_t need = 0;
  int st = linattn_forward_host_bytes(desc, N, &need);
  if (st != LINATTN_OK) return st;
  if (!dev_staging || (reinterpret_cast<uintptr_t>(dev_staging) & 255u)) return LINATTN_ERR_BAD_ALIGNMENT;
  if (dev_staging_bytes < need) return LINATTN_ERR_WORKSPACE_TOO_SMALL;
  if (N == 0) return LINATTN_OK;
  if (!q_host || !k_host || !v_host || !o_host) return LINATTN_ERR_INVALID_ARG;
  Problem p;
  resolve(desc, N, &p);
  const size_t esz = p.dtype == LINATTN_BF16 ? 2 : 4;
  const size_t bytes = (size_t)p.B * (size_t)N * p.H * p.d * esz;
  const size_t tensor = round256(bytes);
  const size_t ws = workspace_need(p);
  char* base = static_cast<char*>(dev_staging);
  void* dq = base + ws;
  void* dk = base + ws + tensor;
  void* dv = base + ws + 2 * tensor;
  void* dout = base + ws + 3 * tensor;
  cudaStream_t s = (cudaStream_t)stream;
  // K and V first: the state pass needs them.  Then Q goes up and O comes down in token chunks, the
  // download of chunk c (on a second stream) running under the upload and the apply pass of chunk c+1:
  // the two copy directions do not share an engine.
  HostPipe* pipe = host_pipe();
  if (!pipe) return LINATTN_ERR_CUDA;
  cudaError_t e = cudaMemcpyAsync(dk, k_host, bytes, cudaMemcpyHostToDevice, s);
  if (e == cudaSuccess) e = cudaMemcpyAsync(dv, v_host, bytes, cudaMemcpyHostToDevice, s);
  if (e != cudaSuccess) return LINATTN_ERR_CUDA;
  float* state = reinterpret_cast<float*>(base + state_slot_offset(p));
  st = run_passes(p, dk, dv, nullptr, nullptr, state, false, 0.f, dev_staging, s);
  if (st != LINATTN_OK) return st;
  const long long chunk_tokens = N >= 8 * 1024 ? (((N + kHostChunks - 1) / kHostChunks + 127) / 128) * 128 : N;
  const size_t row = (size_t)p.H * p.d * esz;  // bytes of one token
  int c = 0;
  for (long long n0 = 0; n0 < N; n0 += chunk_tokens, ++c) {
    const long long nc = N - n0 < chunk_tokens ? N - n0 : chunk_tokens;
    const size_t off = (size_t)n0 * row;
    // dense [B, N, H, d]: the chunk is B pieces of nc*row bytes, N*row bytes apart
    e = cudaMemcpy2DAsync(static_cast<char*>(dq) + off, (size_t)N * row, static_cast<const char*>(q_host) + off,
                          (size_t)N * row, (size_t)nc * row, p.B, cudaMemcpyHostToDevice, s);
    if (e != cudaSuccess) return LINATTN_ERR_CUDA;
    Problem pc = p;
    pc.N = nc;  // strides stay those of the whole tensor
    st = run_passes(pc, nullptr, nullptr, static_cast<char*>(dq) + off, static_cast<char*>(dout) + off, state, false, eps,
                    dev_staging, s);
    if (st != LINATTN_OK) return st;
    if (cudaEventRecord(pipe->chunk_done[c], s) != cudaSuccess ||
        cudaStreamWaitEvent(pipe->down, pipe->chunk_done[c], 0) != cudaSuccess)
      return LINATTN_ERR_CUDA;
    e = cudaMemcpy2DAsync(static_cast<char*>(o_host) + off, (size_t)N * row, static_cast<char*>(dout) + off,
                          (size_t)N * row, (size_t)nc * row, p.B, cudaMemcpyDeviceToHost, pipe->down);
    if (e != cudaSuccess) return LINATTN_ERR_CUDA;
  }
  // the caller's stream is complete only when the last download is
  if (cudaEventRecord(pipe->all_down, pipe->down) != cudaSuccess || cudaStreamWaitEvent(s, pipe->all_down, 0) != cudaSuccess)
    return LINATTN_ERR_CUDA;
  return LINATTN_OK;
}

int blocklin_cache_bytes(const linattn_desc* desc, int64_t max_T_b, size_t* state_bytes, size_t* workspace_bytes) {
  Problem p;
  int st = resolve(desc, max_T_b, &p);
  if (st != LINATTN_OK) return st;
  if (!state_bytes || !workspace_bytes) return LINATTN_ERR_INVALID_ARG;
  *state_bytes = sizeof(float) * (size_t)p.state_elems() * p.units();
  *workspace_bytes = workspace_need(p);
  if ((p.d & 1) == 0 && rope_workspace_need(p) > *workspace_bytes) *workspace_bytes = rope_workspace_need(p);  // blocklin_step_rope
  return LINATTN_OK;
}

int blocklin_cache_init(blocklin_cache** out, const linattn_desc* desc, float eps, void* dev_state,
                        size_t state_bytes, void* dev_workspace, size_t workspace_bytes, void* stream) {
  if (!out) return LINATTN_ERR_INVALID_ARG;
  *out = nullptr;
  Problem p;
  int st = resolve(desc, 0, &p);
  if (st != LINATTN_OK) return st;
  if (!dev_state || !dev_workspace) return LINATTN_ERR_INVALID_ARG;
  if (!aligned16(dev_state) || !aligned16(dev_workspace)) return LINATTN_ERR_BAD_ALIGNMENT;
  const size_t need_state = state_bytes_of(p);
  if (state_bytes < need_state) return LINATTN_ERR_INVALID_ARG;
  if (workspace_bytes < workspace_need(p)) return LINATTN_ERR_WORKSPACE_TOO_SMALL;
  blocklin_cache* c = new (std::nothrow) blocklin_cache;
  if (!c) return LINATTN_ERR_INVALID_ARG;
  c->magic = kCacheMagic;
  c->desc = *desc;
  c->eps = eps;
  c->state = static_cast<float*>(dev_state);
  c->state_bytes = need_state;
  c->workspace = dev_workspace;
  c->workspace_bytes = workspace_bytes;
  c->blocks_seen = 0;
  c->tokens_seen = 0;
  c->joint_prefill = 0;
  cudaError_t e = cudaMemsetAsync(dev_state, 0, need_state, (cudaStream_t)stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(dev_workspace, 0, LINATTN_WORKSPACE_CTRL_BYTES, (cudaStream_t)stream);
  if (e != cudaSuccess) {
    c->magic = 0;
    delete c;
    return LINATTN_ERR_CUDA;
  }
  *out = c;
  return LINATTN_OK;
}

int blocklin_cache_reset(blocklin_cache* cache, void* stream) {
  if (!cache || cache->magic != kCacheMagic) return LINATTN_ERR_BAD_HANDLE;
  cache->blocks_seen = 0;
  cache->tokens_seen = 0;
  // the control block too: a recorded timeout and the barrier word it left half-counted go away with the past
  cudaError_t e = cudaMemsetAsync(cache->state, 0, cache->state_bytes, (cudaStream_t)stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(cache->workspace, 0, LINATTN_WORKSPACE_CTRL_BYTES, (cudaStream_t)stream);
  return cuda_status(e);
}

int blocklin_cache_status(const blocklin_cache* cache, void* stream, int* status) {
  if (!cache || cache->magic != kCacheMagic) return LINATTN_ERR_BAD_HANDLE;
  return linattn_workspace_status(cache->workspace, stream, status);
}

int blocklin_step(blocklin_cache* cache, int64_t T_b, const void* q_blk, const void* k_blk, const void* v_blk,
                  void* o_blk, void* stream) {
  if (!cache || cache->magic != kCacheMagic) return LINATTN_ERR_BAD_HANDLE;
  Problem p;
  int st = resolve(&cache->desc, T_b, &p);
  if (st != LINATTN_OK) return st;
  return step_impl(cache, p, q_blk, k_blk, v_blk, o_blk, (cudaStream_t)stream);
}

int blocklin_step_rope(blocklin_cache* cache, int64_t T_b, const void* q_blk, const void* k_blk, const void* v_blk,
                       void* o_blk, const void* rope_table_blk, void* stream) {
  if (!cache || cache->magic != kCacheMagic) return LINATTN_ERR_BAD_HANDLE;
  Problem p;
  int st = resolve(&cache->desc, T_b, &p);
  if (st != LINATTN_OK) return st;
  return step_rope_impl(cache, p, q_blk, k_blk, v_blk, o_blk, rope_table_blk, true, (cudaStream_t)stream);
}

int blocklin_peek_rope(blocklin_cache* cache, int64_t T_b, const void* q_blk, const void* k_blk, const void* v_blk,
                       void* o_blk, const void* rope_table_blk, void* stream) {
  if (!cache || cache->magic != kCacheMagic) return LINATTN_ERR_BAD_HANDLE;
  Problem p;
  int st = resolve(&cache->desc, T_b, &p);
  if (st != LINATTN_OK) return st;
  if (p.N > 0 && (!q_blk || !o_blk)) return LINATTN_ERR_INVALID_ARG;
  return step_rope_impl(cache, p, q_blk, k_blk, v_blk, o_blk, rope_table_blk, false, (cudaStream_t)stream);
}

int blocklin_prefill_rope(blocklin_cache* cache, int64_t n_blocks, int64_t T_b, const void* q, const void* k,
                          const void* v, void* o, const void* rope_table, void* stream) {
  if (!cache || cache->magic != kCacheMagic) return LINATTN_ERR_BAD_HANDLE;
  if (n_blocks < 0 || T_b < 0) return LINATTN_ERR_INVALID_ARG;
  if ((q == nullptr) != (o == nullptr)) return LINATTN_ERR_INVALID_ARG;
  if (n_blocks == 0 || T_b == 0) return LINATTN_OK;
  if (!k || !v || !rope_table) return LINATTN_ERR_INVALID_ARG;
  Problem p;
  int st = resolve(&cache->desc, n_blocks * T_b, &p);   // every block keeps the whole sequence's strides
  if (st != LINATTN_OK) return st;
  if ((st = check_alignment(p, q, k, v, o)) != LINATTN_OK) return st;
  p.N = T_b;
  const size_t esz = cache->desc.dtype == LINATTN_BF16 ? 2 : 4;
  const size_t row = (size_t)(p.d / 2) * sizeof(__half2);   // one token's rotations
  for (int64_t i = 0; i < n_blocks && st == LINATTN_OK; ++i) {
    const size_t off = (size_t)(i * T_b) * (size_t)p.sn * esz;
    st = step_rope_impl(cache, p, q ? static_cast<const char*>(q) + off : nullptr, static_cast<const char*>(k) + off,
                        static_cast<const char*>(v) + off, o ? static_cast<char*>(o) + off : nullptr,
                        static_cast<const char*>(rope_table) + (size_t)(i * T_b) * row, true, (cudaStream_t)stream);
  }
  return st;
}

int blocklin_peek(blocklin_cache* cache, int64_t T_b, const void* q_blk, const void* k_blk, const void* v_blk,
                  void* o_blk, void* stream) {
  if (!cache || cache->magic != kCacheMagic) return LINATTN_ERR_BAD_HANDLE;
  Problem p;
  int st = resolve(&cache->desc, T_b, &p);
  if (st != LINATTN_OK) return st;
  if (p.N > 0 && (!q_blk || !k_blk || !v_blk || !o_blk)) return LINATTN_ERR_INVALID_ARG;
  if (o_blk && (o_blk == q_blk || o_blk == k_blk || o_blk == v_blk)) return LINATTN_ERR_INVALID_ARG;
  if ((st = check_alignment(p, q_blk, k_blk, v_blk, o_blk)) != LINATTN_OK) return st;
  if (cache->workspace_bytes < workspace_need(p)) return LINATTN_ERR_WORKSPACE_TOO_SMALL;
  if (p.N == 0) return LINATTN_OK;
  // cache + state(block) goes to the state slot of the workspace; the cache itself is only read
  float* tmp = reinterpret_cast<float*>(static_cast<char*>(cache->workspace) + state_slot_offset(p));
  return run_passes(p, k_blk, v_blk, q_blk, o_blk, tmp, true, cache->eps, cache->workspace, (cudaStream_t)stream,
                    cache->state);
}

int blocklin_shard_state(blocklin_cache* cache, int64_t T_shard, const void* k_shard, const void* v_shard,
                         float* state_out, int include_cache, void* stream) {
  if (!cache || cache->magic != kCacheMagic) return LINATTN_ERR_BAD_HANDLE;
  Problem p;
  int st = resolve(&cache->desc, T_shard, &p);
  if (st != LINATTN_OK) return st;
  if (!state_out || state_out == cache->state) return LINATTN_ERR_INVALID_ARG;
  if (p.N > 0 && (!k_shard || !v_shard)) return LINATTN_ERR_INVALID_ARG;
  if ((st = check_alignment(p, k_shard, v_shard, state_out, nullptr)) != LINATTN_OK) return st;
  if (cache->workspace_bytes < workspace_need(p)) return LINATTN_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t s = (cudaStream_t)stream;
  if (p.N == 0)   // a rank without tokens of this block contributes the cache (or nothing) alone
    return cuda_status(include_cache ? cudaMemcpyAsync(state_out, cache->state, cache->state_bytes, cudaMemcpyDeviceToDevice, s)
                                     : cudaMemsetAsync(state_out, 0, cache->state_bytes, s));
  return run_passes(p, k_shard, v_shard, nullptr, nullptr, state_out, include_cache != 0, 0.f, cache->workspace, s,
                    include_cache ? cache->state : nullptr);
}

int blocklin_shard_commit(blocklin_cache* cache, const float* state_in, int64_t block_tokens, void* stream) {
  if (!cache || cache->magic != kCacheMagic) return LINATTN_ERR_BAD_HANDLE;
  if (!state_in || block_tokens < 0) return LINATTN_ERR_INVALID_ARG;
  if (state_in != cache->state &&
      cudaMemcpyAsync(cache->state, state_in, cache->state_bytes, cudaMemcpyDeviceToDevice, (cudaStream_t)stream) != cudaSuccess)
    return LINATTN_ERR_CUDA;
  cache->blocks_seen += 1;
  cache->tokens_seen += block_tokens;
  return LINATTN_OK;
}

int blocklin_prefill(blocklin_cache* cache, int64_t n_blocks, int64_t T_b, const void* q, const void* k,
                     const void* v, void* o, void* stream) {
  if (!cache || cache->magic != kCacheMagic) return LINATTN_ERR_BAD_HANDLE;
  if (n_blocks < 0 || T_b < 0) return LINATTN_ERR_INVALID_ARG;
  if ((q == nullptr) != (o == nullptr)) return LINATTN_ERR_INVALID_ARG;
  if (n_blocks == 0 || T_b == 0) return LINATTN_OK;
  if (!k || !v) return LINATTN_ERR_INVALID_ARG;
  // The tensors are [B, n_blocks*T_b, H, d]; block i is the token range [i*T_b, (i+1)*T_b) of each batch
  // entry, so every block keeps the whole sequence's strides.
  Problem p;
  int st = resolve(&cache->desc, n_blocks * T_b, &p);
  if (st != LINATTN_OK) return st;
  if ((st = check_alignment(p, q, k, v, o)) != LINATTN_OK) return st;
  if (o && (o == q || o == k || o == v)) return LINATTN_ERR_INVALID_ARG;
  // All blocks at once: with the blocks of every batch entry viewed as batch entries of their own (possible when
  // the batch stride is that of a dense [B, n_blocks*T_b, ...] tensor), ONE state pass gives every block's own
  // state, a prefix sum over the blocks turns them into the cache after each block (Eq. 3), and ONE apply pass
  // reads block m's queries against prefix m.  Taken when the cache's workspace is large enough for it
  // (blocklin_prefill_workspace_bytes); otherwise the blocks are stepped one by one.
  Problem pv = p;
  pv.B = p.B * (int)n_blocks;
  pv.N = T_b;
  pv.sb = T_b * p.sn;
  const bool batch_dense = p.B == 1 || p.sb == n_blocks * T_b * p.sn;
  if (cache->joint_prefill && n_blocks > 1 && batch_dense && (long long)pv.B * pv.H <= 65535 &&
      (p.state_elems() * p.H) % 4 == 0 &&
      cache->workspace_bytes >= workspace_need(pv)) {
    cudaStream_t s = (cudaStream_t)stream;
    float* blk = reinterpret_cast<float*>(static_cast<char*>(cache->workspace) + state_slot_offset(pv));
    st = run_passes(pv, k, v, nullptr, nullptr, blk, false, 0.f, cache->workspace, s);
    if (st != LINATTN_OK) return st;
    if (prefix_states(blk, cache->state, p.B, (int)n_blocks, (long long)p.H * p.state_elems(), s) != cudaSuccess)
      return LINATTN_ERR_CUDA;
    if (q) {
      st = run_passes(pv, nullptr, nullptr, q, o, blk, false, cache->eps, cache->workspace, s);
      if (st != LINATTN_OK) return st;
    }
    cache->blocks_seen += n_blocks;
    cache->tokens_seen += n_blocks * T_b;
    return LINATTN_OK;
  }
  p.N = T_b;
  const size_t esz = cache->desc.dtype == LINATTN_BF16 ? 2 : 4;
  for (int64_t i = 0; i < n_blocks && st == LINATTN_OK; ++i) {
    const size_t off = (size_t)(i * T_b) * (size_t)p.sn * esz;
    st = step_impl(cache, p, q ? static_cast<const char*>(q) + off : nullptr, static_cast<const char*>(k) + off,
                   static_cast<const char*>(v) + off, o ? static_cast<char*>(o) + off : nullptr,
                   (cudaStream_t)stream);
  }
  return st;
}

int blocklin_prefill_workspace_bytes(const linattn_desc* desc, int64_t n_blocks, int64_t T_b, size_t* workspace_bytes) {
  Problem p;
  if (!workspace_bytes || n_blocks < 1) return LINATTN_ERR_INVALID_ARG;
  int st = resolve(desc, T_b, &p);
  if (st != LINATTN_OK) return st;
  Problem pv = p;
  if ((long long)p.B * n_blocks * p.H > 65535) return LINATTN_ERR_UNSUPPORTED;
  pv.B = p.B * (int)n_blocks;
  const size_t steps = workspace_need(p), all = workspace_need(pv);
  *workspace_bytes = all > steps ? all : steps;
  return LINATTN_OK;
}

int blocklin_cache_joint_prefill(blocklin_cache* cache, int enable) {
  if (!cache || cache->magic != kCacheMagic) return LINATTN_ERR_BAD_HANDLE;
  cache->joint_prefill = enable ? 1 : 0;
  return LINATTN_OK;
}

int blocklin_cache_info(const blocklin_cache* cache, int64_t* blocks_seen, int64_t* tokens_seen,
                        size_t* state_bytes) {
  if (!cache || cache->magic != kCacheMagic) return LINATTN_ERR_BAD_HANDLE;
  if (blocks_seen) *blocks_seen = cache->blocks_seen;
  if (tokens_seen) *tokens_seen = cache->tokens_seen;
  if (state_bytes) *state_bytes = cache->state_bytes;
  return LINATTN_OK;
}

int blocklin_cache_destroy(blocklin_cache* cache) {
  if (!cache || cache->magic != kCacheMagic) return LINATTN_ERR_BAD_HANDLE;
  cache->magic = 0;
  delete cache;
  return LINATTN_OK;
}

}  // extern "C"
