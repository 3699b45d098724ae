/*
 * linattn.h -- C ABI of the B200 (sm_100a) ReLU linear-attention library.
 *
 * The operation is the linear attention of SANA-Video's Linear DiT, per
 * attention head with head dimension d and phi = ReLU:
 *
 *   bidirectional (Eq. 2 with the rotary factors dropped, as the text under
 *   Eq. 3 does):
 *       S = sum_n phi(k_n)^T v_n   (d x d),   z = sum_n phi(k_n)   (d)
 *       o_n = phi(q_n) S / (phi(q_n) . z + eps)
 *
 *   block-causal with the constant-memory cache (Eq. 3; Sec. 3.2 "KV Cache in
 *   Block Linear Attention"; the cache update of Algorithm 1): tokens come in
 *   contiguous blocks of frames; a block attends to itself and to every
 *   earlier block.  The whole past is the running pair (sum S, sum phi(K)^T)
 *   per head, kept in fp32; no per-token K/V is stored and the cache size
 *   does not depend on the number of blocks (Table 1).
 *
 * Conventions common to every call
 * --------------------------------
 *  - All tensor pointers are DEVICE pointers.  The library never allocates or
 *    frees device memory and never keeps a caller's pointer beyond what is
 *    documented for the cache handle.  Descriptors, handles and out-params
 *    are HOST memory.
 *  - Q, K, V, O share one layout: element (b, n, h, e) is at element offset
 *    b*stride_b + n*stride_n + h*stride_h + e.  A stride of 0 in the
 *    descriptor selects the dense [B, N, H, d] default for that call's N.
 *    Tokens are ordered frame-major, so a block of frames is a contiguous
 *    token range.
 *  - dtype LINATTN_BF16: Q, K, V, O are bfloat16; products are exact in fp32,
 *    accumulation is fp32, O is rounded to nearest-even once at the store.
 *    dtype LINATTN_F32: fp32 in and out, fp32 arithmetic.
 *  - A "state" is, per (b, h), a (d+1) x d fp32 matrix W stored row-major,
 *    units ordered [B][H]:   W[j][i] = S[i][j]  for j < d  (i: key feature,
 *    j: value feature),      W[d][i] = z[i].
 *    Its size is B*H*(d*d+d)*4 bytes.  It is plain memory: a copy of it is a
 *    complete checkpoint of a stream.
 *  - `stream` is a cudaStream_t passed as void* (NULL: the default stream).
 *    Calls enqueue work and return; they do not synchronise.
 *  - Pointers must be 16-byte aligned and strides multiples of 8 elements
 *    (bf16) or 4 elements (fp32).  O must not alias Q, K or V.
 *  - Every function returns LINATTN_OK (0) or a negative linattn_status.
 *    Arguments are validated before anything is launched.  Zero tokens is a
 *    successful no-op (linattn_state then writes a zero state; linattn_forward
 *    writes nothing).  Nothing here throws, aborts or traps the device; the
 *    only device-side wait (the grid barrier of the fused kernels) gives up
 *    after a bounded number of polls and records LINATTN_ERR_TIMEOUT in the
 *    workspace, readable with linattn_workspace_status.
 *  - Calls that share a workspace (or a cache) must be ordered on one stream:
 *    two of them in flight at once race on the split-N partials.
 */
#ifndef LINATTN_H_
#define LINATTN_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define LINATTN_API __attribute__((visibility("default")))
#else
#define LINATTN_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum linattn_dtype { LINATTN_BF16 = 0, LINATTN_F32 = 1 } linattn_dtype;

typedef enum linattn_status {
  LINATTN_OK = 0,
  LINATTN_ERR_INVALID_ARG = -1,        /* null pointer, negative size, bad enum, aliasing */
  LINATTN_ERR_UNSUPPORTED = -2,        /* head dim outside 1..128, or a layout the kernels do not take */
  LINATTN_ERR_BAD_ALIGNMENT = -3,      /* pointer or stride alignment rule above violated */
  LINATTN_ERR_WORKSPACE_TOO_SMALL = -4,
  LINATTN_ERR_CUDA = -5,               /* a CUDA runtime/driver call failed, or no sm_100 device */
  LINATTN_ERR_TIMEOUT = -6,            /* a bounded device-side wait expired */
  LINATTN_ERR_BAD_HANDLE = -7,         /* cache handle is null, destroyed or corrupt */
  LINATTN_ERR_SCRATCH_LIMIT = -8       /* problem needs more scratch than the built-in array of
                                          linattn_state_static_scratch holds */
} linattn_status;

/* Problem descriptor: plain data, filled by the caller, copied by the library. */
typedef struct linattn_desc {
  int32_t B;        /* batch */
  int32_t H;        /* heads */
  int32_t d;        /* head dimension, 1..128 (bf16 fast path: 32, 64, 112, 128) */
  int32_t dtype;    /* linattn_dtype */
  int64_t stride_b; /* element strides; 0 = dense [B,N,H,d] */
  int64_t stride_n;
  int64_t stride_h;
} linattn_desc;

LINATTN_API const char* linattn_status_string(int status);

/* Bytes of one state for this descriptor: B*H*(d*d+d)*4 (Table 1's O(D^2) cache, per head). */
LINATTN_API int linattn_state_bytes(const linattn_desc* desc, size_t* bytes);

/* Scratch needed by linattn_forward / linattn_state for N tokens (split-N partial states and a
 * small control block).  Depends on (B,H,d,dtype,N) only; works without a GPU. */
LINATTN_API int linattn_workspace_bytes(const linattn_desc* desc, int64_t N, size_t* bytes);

/* Zero a workspace's control block.  Call once after allocating a workspace (its first
 * LINATTN_WORKSPACE_CTRL_BYTES bytes must start as zero) or to clear a recorded timeout. */
#define LINATTN_WORKSPACE_CTRL_BYTES 4096
LINATTN_API int linattn_workspace_init(void* workspace, size_t workspace_bytes, void* stream);

/* Synchronises `stream`, then reports a device-side status recorded in the workspace
 * (LINATTN_OK or LINATTN_ERR_TIMEOUT) through *status. */
LINATTN_API int linattn_workspace_status(const void* workspace, void* stream, int* status);

/* Eq. 2, whole sequence: O = phi(Q) S / (phi(Q) z + eps) with (S, z) reduced over all N tokens.
 * q, k, v: in; o: out (same layout and dtype).  workspace: scratch, contents undefined after. */
LINATTN_API int linattn_forward(const linattn_desc* desc, int64_t N, const void* q, const void* k, const void* v, void* o,
                    float eps, void* workspace, size_t workspace_bytes, void* stream);

/* Eq. 2 as printed, with its rotary factors (Sec. 3.1): the rotation is applied after the ReLU and in the
 * numerator only,
 *     o_n = RoPE_n(phi(q_n)) ( sum_m RoPE_m(phi(k_m))^T v_m ) / ( phi(q_n) . sum_m phi(k_m) + eps ),
 * so the denominator stays non-negative.  RoPE_n turns the feature pair (2p, 2p+1) of token n by an angle given
 * through its cosine c and sine s: (a, b) -> (a c - b s, a s + b c).  How the angles follow from a token's
 * (t, h, w) position (the paper's 3D RoPE) is the caller's choice.  d must be even.
 *
 * The rotations come as a packed DEVICE table [N][d/2] of (cos, sin) fp16 pairs (4 bytes each, 16-byte aligned
 * base), shared by all batch entries and heads; the operation is defined on those fp16 values.  A model builds
 * the table once (positions do not change between layers or denoising steps): linattn_rope_pack rounds fp32
 * DEVICE arrays rope_cos, rope_sin [N][d/2] to nearest fp16 into `table` (linattn_rope_table_bytes bytes).
 * The workspace must hold linattn_rope_workspace_bytes() bytes (control block zeroed once with
 * linattn_workspace_init). */
LINATTN_API int linattn_rope_table_bytes(int64_t N, int32_t d, size_t* bytes);
LINATTN_API int linattn_rope_pack(int64_t N, int32_t d, const float* rope_cos, const float* rope_sin, void* table,
                                  void* stream);
LINATTN_API int linattn_rope_workspace_bytes(const linattn_desc* desc, int64_t N, size_t* bytes);
LINATTN_API int linattn_forward_rope(const linattn_desc* desc, int64_t N, const void* q, const void* k, const void* v,
                                     void* o, float eps, const void* rope_table, void* workspace,
                                     size_t workspace_bytes, void* stream);

/* The state of Eq. 2 / Eq. 3 alone: state = (sum_n phi(k_n)^T v_n, sum_n phi(k_n)) in the layout above.
 * Deterministic: split-N partials are summed in a fixed order, so repeated calls give identical bits. */
LINATTN_API int linattn_state(const linattn_desc* desc, int64_t N, const void* k, const void* v, float* state,
                  void* workspace, size_t workspace_bytes, void* stream);

/* linattn_state for callers that cannot provide a workspace.  (The paper has no counterpart: this
 * is a convenience of this library.)
 *
 * Some callers may not allocate device memory at the point where they need the state: code running
 * inside a memory-budgeted serving loop whose pools are fixed at start-up, a plug-in that is handed
 * tensors but no allocator, or a host thread that must not take the allocator's lock because
 * cudaMalloc may synchronise the whole device.  For them the split-N scratch of the state pass lives
 * in an array compiled into the library instead of a caller-provided workspace.  This function
 * calls no cudaMalloc / cudaFree and no allocating library routine; the caller still passes the
 * inputs k, v and the output `state` (same meaning, layout and alignment rules as linattn_state).
 *
 *  - Limit: the scratch the call needs (what linattn_workspace_bytes reports, minus the trailing
 *    state slot) must fit in LINATTN_STATIC_SCRATCH_BYTES (16 MiB; every GPU on which this library
 *    is used holds that much device memory until the process exits).  For bf16 inputs with
 *    d in {32 (heads contiguous), 64, 112, 128} the need does not grow with N, and B*H <= 20 heads
 *    of dimension 112 fit at any N.  Other shapes and fp32 inputs keep one partial state per 512
 *    tokens (at most 64) per head, so they fit only while B*H*(d*d+d)*4*min(64, ceil(N/512)) stays
 *    below the limit (20 fp32 heads of dimension 112: N <= 8192).  Larger problems return
 *    LINATTN_ERR_SCRATCH_LIMIT and launch nothing.
 *  - The first call on each device looks the array's device address up (one runtime call, with
 *    that device current); make that first call outside any stream capture.
 *  - Every call on a device shares the one array, which still holds the previous call's contents:
 *    the control block at its start is cleared on `stream` before every launch, and the partial
 *    records are fully rewritten before they are read.  Two calls that overlap on the GPU (different
 *    streams, or threads racing on one device) would corrupt each other: order them. */
#define LINATTN_STATIC_SCRATCH_BYTES (16u << 20)
LINATTN_API int linattn_state_static_scratch(const linattn_desc* desc, int64_t N, const void* k, const void* v,
                                             float* state, void* stream);

/* linattn_workspace_status for the built-in array (its address is not the caller's to know): synchronises
 * `stream`, then reports LINATTN_OK or LINATTN_ERR_TIMEOUT of the LAST linattn_state_static_scratch call on the
 * current device through *status (every call clears the word before its launch).  (No counterpart in the paper.) */
LINATTN_API int linattn_static_scratch_status(void* stream, int* status);

/* The apply half of Eq. 2 alone: o_n = phi(q_n) S / (phi(q_n) . z + eps) for a given state.
 * workspace: only its control block is used (LINATTN_WORKSPACE_CTRL_BYTES suffice). */
LINATTN_API int linattn_apply(const linattn_desc* desc, int64_t N, const void* q, const float* state, void* o, float eps,
                  void* workspace, size_t workspace_bytes, void* stream);

/* Eq. 2 with HOST buffers: copies q, k, v (host, ideally pinned) into the caller's device staging
 * area, runs linattn_forward there and copies O back to `o_host`, all enqueued on `stream`.
 * `dev_staging` (DEVICE, 256-byte aligned) must hold linattn_forward_host_bytes() bytes: four dense
 * [B,N,H,d] tensors plus the forward's workspace; its control block must have been zeroed once with
 * linattn_workspace_init(dev_staging, ...).  Host tensors are dense [B,N,H,d] (the descriptor's
 * strides must be 0).  Q is uploaded and O downloaded in token chunks, the downloads on a second stream
 * that the library keeps per device, so that the two copy directions overlap; `stream` is made to wait
 * for the last download, so the host buffers may be reused once `stream` has been synchronised. */
LINATTN_API int linattn_forward_host_bytes(const linattn_desc* desc, int64_t N, size_t* bytes);
LINATTN_API int linattn_forward_host(const linattn_desc* desc, int64_t N, const void* q_host, const void* k_host,
                                     const void* v_host, void* o_host, float eps, void* dev_staging,
                                     size_t dev_staging_bytes, void* stream);

/* Number of CUDA kernels this library has launched in this process so far (all entry points). */
LINATTN_API uint64_t linattn_kernel_launches(void);

/* ---- block-causal form with the constant-memory cache (Eq. 3, Algorithm 1) ---- */

typedef struct blocklin_cache blocklin_cache; /* opaque HOST handle */

/* Sizes the caller must allocate on the device for a stream whose blocks have at most max_T_b
 * tokens: the state (the cache proper; independent of max_T_b and of the number of blocks) and
 * the scratch workspace. */
LINATTN_API int blocklin_cache_bytes(const linattn_desc* desc, int64_t max_T_b, size_t* state_bytes, size_t* workspace_bytes);

/* Create a handle over caller-owned device memory and enqueue zeroing of the state ("initialise
 * the KV cache as empty", Algorithm 1).  The handle keeps the two device pointers; the caller
 * keeps ownership and must keep them alive until blocklin_cache_destroy. */
LINATTN_API int blocklin_cache_init(blocklin_cache** out, const linattn_desc* desc, float eps, void* dev_state,
                        size_t state_bytes, void* dev_workspace, size_t workspace_bytes, void* stream);

/* Forget the past: zero the state, blocks_seen = tokens_seen = 0.  Also zeroes the control block of the cache's
 * workspace, which clears a recorded LINATTN_ERR_TIMEOUT (see blocklin_cache_status). */
LINATTN_API int blocklin_cache_reset(blocklin_cache* cache, void* stream);

/* One block of T_b tokens ([B, T_b, H, d] with the descriptor's strides): add the block's own
 * (S_blk, z_blk) to the cache, then apply the block's queries to the updated cache (the block
 * attends to itself and to all earlier blocks).  o_blk and q_blk may both be NULL: absorb only. */
LINATTN_API int blocklin_step(blocklin_cache* cache, int64_t T_b, const void* q_blk, const void* k_blk, const void* v_blk,
                  void* o_blk, void* stream);

/* blocklin_step with the rotary factors of Eq. 2 (rotation after the ReLU, numerator only): the cache then
 * holds (sum of RoPE(phi(k))^T v, sum of phi(k)).  rope_table_blk: the packed (cos, sin) fp16 rows of this block's
 * T_b tokens ([T_b][d/2], see linattn_forward_rope); positions simply continue from block to block, so it is
 * usually a pointer into one table of the whole stream.  A stream uses either this call or blocklin_step for
 * all of its blocks.  o_blk and q_blk may both be NULL: absorb only. */
LINATTN_API int blocklin_step_rope(blocklin_cache* cache, int64_t T_b, const void* q_blk, const void* k_blk,
                                   const void* v_blk, void* o_blk, const void* rope_table_blk, void* stream);

/* blocklin_peek with the rotary factors: a denoising step of Algorithm 1 on the attention the model runs (Eq. 2
 * with RoPE, Sec. 3.1).  The block's queries see the rotary cache plus the block's own rotated state; the cache is
 * only read and blocks_seen does not change.  Same bits as blocklin_step_rope would give on the same cache.
 * q_blk and o_blk are required. */
LINATTN_API int blocklin_peek_rope(blocklin_cache* cache, int64_t T_b, const void* q_blk, const void* k_blk,
                                   const void* v_blk, void* o_blk, const void* rope_table_blk, void* stream);

/* blocklin_prefill with the rotary factors: n_blocks consecutive blocks of T_b tokens over [B, n_blocks*T_b, H, d]
 * tensors, rope_table the packed rows of those n_blocks*T_b tokens; result and final cache are those of n_blocks
 * calls of blocklin_step_rope, bit for bit (the blocks are stepped one by one).  q and o may both be NULL. */
LINATTN_API int blocklin_prefill_rope(blocklin_cache* cache, int64_t n_blocks, int64_t T_b, const void* q, const void* k,
                                      const void* v, void* o, const void* rope_table, void* stream);

/* The denoising steps of Algorithm 1 ("x0 <- G(x; t_j, KV)" for t_j > 0): the block's queries see the
 * cache plus the block's own (S_blk, z_blk), exactly as in blocklin_step, but the cache is only read:
 * nothing is committed, blocks_seen does not change.  The clean block is committed afterwards with
 * blocklin_step (with q_blk = o_blk = NULL to commit without producing outputs). */
LINATTN_API int blocklin_peek(blocklin_cache* cache, int64_t T_b, const void* q_blk, const void* k_blk, const void* v_blk,
                  void* o_blk, void* stream);

/* ---- a block whose tokens are spread over several GPUs ----
 * The state of Eq. 2 and the running sums of Eq. 3 are sums over tokens, so a block (or a whole sequence) can be
 * split by tokens over ranks: every rank reduces its own shard, ONE all-reduce (sum) of B*H*(d*d+d) floats makes
 * the new cache on every rank, and every rank applies its own queries to it.  The library does the two local
 * halves; the all-reduce is the caller's (NCCL through torch.distributed in the Python binding), on memory of
 * the caller's own GPU.
 *
 * blocklin_shard_state: state_out (DEVICE, one state, not the cache's own memory) = this rank's share of the new
 *   cache: the state of its T_shard tokens of the block, plus the current cache when include_cache is non-zero.
 *   Exactly ONE rank passes include_cache = 1, so that the sum over ranks is cache + state(block).  The cache is
 *   only read.  T_shard = 0 is allowed (state_out = the cache, or zeros).
 * blocklin_shard_commit: the cache := state_in (the all-reduced sum; every rank passes the same values),
 *   blocks_seen += 1, tokens_seen += block_tokens (the block's tokens over all ranks).
 * The block's outputs are then linattn_apply(q_shard, cache state) on each rank.  With one rank and
 * include_cache = 1 the three calls give the bits of blocklin_step. */
LINATTN_API int blocklin_shard_state(blocklin_cache* cache, int64_t T_shard, const void* k_shard, const void* v_shard,
                                     float* state_out, int include_cache, void* stream);
LINATTN_API int blocklin_shard_commit(blocklin_cache* cache, const float* state_in, int64_t block_tokens, void* stream);

/* n_blocks consecutive blocks of T_b tokens in one call over [B, n_blocks*T_b, H, d] tensors; result and final
 * cache are those of n_blocks calls of blocklin_step, bit for bit.  q and o may both be NULL.
 *
 * After blocklin_cache_joint_prefill(cache, 1), and if the cache was created over a workspace of at least
 * blocklin_prefill_workspace_bytes(desc, n_blocks, T_b) bytes (and the batch stride is the dense one, or B = 1),
 * all blocks are processed together instead: one state pass gives every block's own state, a prefix sum over
 * the blocks gives the cache after each block, one apply pass reads every block against its prefix.  The sums
 * are then associated differently than in n_blocks single steps, so the two agree to fp32 rounding of the
 * state, not bit for bit: that is why it has to be asked for.  Where the conditions do not hold the blocks are
 * stepped one by one. */
LINATTN_API int blocklin_cache_joint_prefill(blocklin_cache* cache, int enable);
LINATTN_API int blocklin_prefill_workspace_bytes(const linattn_desc* desc, int64_t n_blocks, int64_t T_b,
                                                 size_t* workspace_bytes);
LINATTN_API int blocklin_prefill(blocklin_cache* cache, int64_t n_blocks, int64_t T_b, const void* q, const void* k,
                     const void* v, void* o, void* stream);

/* Host-side bookkeeping; any out-param may be NULL. */
LINATTN_API int blocklin_cache_info(const blocklin_cache* cache, int64_t* blocks_seen, int64_t* tokens_seen,
                        size_t* state_bytes);

/* Device-side status of the stream's launches so far.  Launches are asynchronous, so a bounded device-side wait
 * that ran out (Sec. 3.2's step is one cooperative launch with two grid-wide meetings) cannot be reported by the
 * call that enqueued it: this call synchronises `stream` and reports LINATTN_OK or LINATTN_ERR_TIMEOUT through
 * *status.  After a timeout the outputs of that launch are undefined and the workspace's barrier word is left
 * half-counted, so every later launch on this cache would time out as well: call blocklin_cache_reset (or restore
 * a checkpoint of the state and call linattn_workspace_init on the workspace) before going on. */
LINATTN_API int blocklin_cache_status(const blocklin_cache* cache, void* stream, int* status);

/* Frees the host handle only; device memory stays the caller's. */
LINATTN_API int blocklin_cache_destroy(blocklin_cache* cache);

#ifdef __cplusplus
}
#endif
#endif /* LINATTN_H_ */
