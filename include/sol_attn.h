/*
 * sol_attn.h -- C ABI of the B200 (sm_100a) Sol-Attn forward path.
 *
 * Sol-Attn ("on-the-fly attention sparsification") computes, for every query block i of a
 * head, softmax attention in which key/value blocks whose pooled proxy score exceeds a
 * query-dependent threshold are processed exactly and all other blocks are folded in through
 * their pooled key and summed value, all inside one online-softmax pass.
 *
 * Conventions shared by every entry point
 *   - q, k, v, out: DEVICE pointers to contiguous row-major [B, H, N, d] bf16 tensors,
 *     16-byte aligned.  N is the number of tokens per (batch, head) (the paper's L).
 *   - Every logit is multiplied by scale = 1/sqrt(d) unless the _ex call overrides it.
 *   - `threshold` is the standardized cutoff beta of Eq. (4): tau_i = mu_i + beta*sigma_i.
 *     +INFINITY routes nothing to the exact branch, -INFINITY routes everything.
 *   - The library owns no device memory, creates no stream and never synchronises unless
 *     stated.  All work is enqueued on `stream` (a cudaStream_t passed as void*; NULL is the
 *     legacy default stream) and the call returns after the last launch.  Errors that the
 *     host can see (bad pointers, unsupported shapes, too-small workspace, wrong GPU
 *     architecture) are returned before anything is launched.  Errors found on the device
 *     (a bounded wait that expired) are recorded in a status word inside the workspace and
 *     read back with sol_attn_read_device_status().
 *   - Scratch memory is a caller-allocated device workspace of sol_attn_workspace_bytes()
 *     bytes, 1024-byte aligned, attached with sol_attn_bind_workspace() (process-wide, one at
 *     a time; not thread-safe) or passed per call through sol_attn_args.  Its contents are
 *     overwritten by every call.  Calls that share a workspace and overlap on the GPU race.
 *   - Supported shapes: d in {64, 128}; block_q == block_k in {64, 128} for the fused
 *     kernels (the pooling pre-pass accepts any block size in [1, 1024]); B, H, N >= 1;
 *     ceil(N / block_k) <= 65535; B * H <= 65535.  Anything else returns SOL_ERR_UNSUPPORTED_SHAPE.
 */
#ifndef SOL_ATTN_H_
#define SOL_ATTN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t sol_status_t;
typedef void*   sol_stream_t;   /* a cudaStream_t */

enum {
  SOL_OK                    =  0,
  SOL_ERR_INVALID_ARG       = -1,  /* NULL / misaligned pointer, non-positive size, NaN threshold */
  SOL_ERR_UNSUPPORTED_SHAPE = -2,  /* d, block sizes or N outside the supported set            */
  SOL_ERR_UNSUPPORTED_ARCH  = -3,  /* current device is not compute capability 10.x            */
  SOL_ERR_WORKSPACE         = -4,  /* no workspace bound / workspace too small or misaligned   */
  SOL_ERR_CUDA              = -5,  /* a CUDA runtime or driver call failed (launch, tensor map)*/
  SOL_ERR_DEVICE_TIMEOUT    = -6,  /* a bounded device-side wait expired; output is invalid    */
  SOL_ERR_SCRATCH_LIMIT     = -7,  /* problem larger than the library's built-in scratch array */
  SOL_ERR_STATIC_SCRATCH    = -8   /* the built-in scratch array could not be set up on this device */
};

/* what the fused kernel computes */
enum {
  SOL_MODE_SOL        = 0,  /* Algorithm 1: exact branch + proxy-score-reuse approximation     */
  SOL_MODE_DENSE      = 1,  /* Eq. (1): every block exact, no routing                          */
  SOL_MODE_EXACT_ONLY = 2   /* Eq. (2): routed blocks exact, unselected blocks dropped         */
};

/* how sigma_i of Eq. (4) is estimated in the pre-attention pass */
enum {
  SOL_EST_MOMENTS  = 0,   /* exact: full second moment of the pooled keys, Eq. (5)                */
  SOL_EST_DIAGONAL = 1    /* diagonal of the pooled-key covariance only (appendix, diagonal
                             threshold estimator): O(d) per query block                         */
};

/* which implementation of the fused kernel runs */
enum {
  SOL_IMPL_AUTO     = 0,  /* the tcgen05 kernel                                                */
  SOL_IMPL_TCGEN05  = 1,  /* TMA + tcgen05.mma + TMEM kernel (all supported shapes)            */
  SOL_IMPL_MMA_SYNC = 2   /* portable warp-level mma.sync kernel (all supported shapes)        */
};

/* memory layout of q, k, v and out (all four the same); d channels of a token are contiguous */
enum {
  SOL_LAYOUT_BHND = 0,    /* [B, H, N, d] row-major: the paper's per-head view (default)         */
  SOL_LAYOUT_BNHD = 1     /* [B, N, H, d] row-major: what a fused QKV projection of a DiT block
                             leaves behind; the heads of a token are interleaved, no transpose
                             is needed before or after the operator                              */
};

/* where the comparison of Eq. (4), s_ij > tau_i, is evaluated */
enum {
  SOL_ROUTING_FUSED   = 0,  /* inside the fused kernel, as Algorithm 1 has it: no routing decision ever
                               reaches memory (the default)                                          */
  SOL_ROUTING_PREPASS = 1   /* by a small kernel before the fused one, kept as ONE BIT per (query block,
                               key block) pair in `mask_out` (which must then be given; 1.7 MB at
                               75 600 tokens x 40 heads) and read back by the fused kernel.  The proxy
                               scores themselves are still never stored.  Same decisions up to fp32
                               summation order, i.e. identical outside the rounding band of the
                               threshold.  Pays off at low routing densities, where the in-kernel
                               router paces the work item; tcgen05 implementation only (with
                               SOL_IMPL_MMA_SYNC the call returns SOL_ERR_INVALID_ARG); ignored in
                               SOL_MODE_DENSE                                                         */
};

/* Human-readable name of a status code; never NULL, static storage. */
const char* sol_attn_status_string(sol_status_t status);

/* Bytes of device workspace needed for the given problem (0 if the shape is unsupported).
 * The workspace holds the pre-attention results of Sec. 3.1-3.2 -- pooled queries Qbar, pooled
 * keys KC (token mean, Eq. 3), summed values VC (defined before Eq. 9), bf16 operand copies,
 * pooled-key moments (Eq. 5), mu/sigma/tau per query block (Eq. 4) -- plus a status word. */
size_t sol_attn_workspace_bytes(int B, int H, int N, int d, int block_q, int block_k);

/* Byte offsets of the parity-relevant arrays inside a workspace laid out for the given problem.
 * All arrays are fp32.  qbar: [B,H,Nq,d] mean of each query block;
 * kc: [B,H,Nk,d] mean of each key block; vc: [B,H,Nk,d] SUM of each value block;
 * mu, sigma, tau: [B,H,Nq]; status: int32[16] (word 0 = device status, see below). */
typedef struct {
  size_t status, qbar, kc, vc, mu, sigma, tau, total_bytes;
  int32_t n_q_blocks, n_k_blocks;
} sol_attn_ws_view;
sol_status_t sol_attn_workspace_view(int B, int H, int N, int d, int block_q, int block_k,
                                     sol_attn_ws_view* view /* host, out */);

/* Attach a device workspace and (optionally) a device int32 [B, H, ceil(N/block_q)] array that
 * receives, per query block, the number of key blocks routed to the exact branch (|S_i| of
 * Eq. 4; overwritten, not accumulated, by every forward).  dev_counts may be NULL.  The size is
 * checked against each later call's shape.  Passing dev_ws == NULL detaches. */
sol_status_t sol_attn_bind_workspace(void* dev_ws, size_t bytes, int32_t* dev_counts);

/* Pre-attention pass (Eq. 3 pooling; Eq. 5 moments; Eq. 4 thresholds): one bandwidth-bound
 * read of q, k, v that fills the bound workspace.  `threshold` is beta.  q may be NULL when
 * only K/V pooling is wanted (thresholds are then not produced). */
sol_status_t sol_attn_pool(const void* q, const void* k, const void* v,
                           int B, int H, int N, int d, int block_q, int block_k,
                           float threshold, sol_stream_t stream);

/* Threshold step alone (Eq. 5 pooled-key moments, Eq. 4 mu, sigma, tau) on the pooled tensors a
 * previous sol_attn_pool / forward left in the bound workspace: re-thresholds the same q, k, v
 * with another beta (density calibration, a per-step schedule) without reading them again.
 * `scale` <= 0 selects 1/sqrt(d); `estimator` is SOL_EST_*.  Overwrites mu, sigma, tau in the
 * workspace; a following sol_attn_forward_ex with skip_pool = 1 uses them. */
sol_status_t sol_attn_thresholds(int B, int H, int N, int d, int block_q, int block_k, float threshold,
                                 float scale, int estimator, sol_stream_t stream);

/* Algorithm 1 end to end: the pooling pre-pass followed by the fused single-pass kernel
 * (on-the-fly thresholding, exact branch on routed blocks, approximate branch on the rest,
 * Eqs. 9-10), using the bound workspace.  Rows >= N of `out` do not exist and are never
 * written. */
sol_status_t sol_attn_forward(const void* q, const void* k, const void* v, void* out,
                              int B, int H, int N, int d, int block_q, int block_k,
                              float threshold, sol_stream_t stream);

/* Dense softmax attention, Eq. (1), through the same fused kernel with routing off
 * (block size 128 for d = 128, 64 for d = 64).  counts, when bound, receive ceil(N/block). */
sol_status_t sol_attn_dense(const void* q, const void* k, const void* v, void* out,
                            int B, int H, int N, int d, sol_stream_t stream);

/* Routing decisions alone (the pre-pass of SOL_ROUTING_PREPASS): evaluates Eq. (4), s_ij > tau_i, for every
 * (query block, key block) pair on the pooled tensors and thresholds a previous sol_attn_pool /
 * sol_attn_thresholds / forward left in the bound workspace, and writes one bit per pair to `mask`
 * (device, uint32 [B, H, Nq, ceil(Nk / 32)], bit j % 32 of word j / 32; caller-owned).  `tau_override`
 * (device fp32 [B, H, Nq]) replaces the workspace's thresholds when not NULL; `forced_blocks` as in
 * sol_attn_args.  `scale` <= 0 selects 1/sqrt(d).  One kernel on `stream`; does not synchronise. */
sol_status_t sol_attn_route_mask(int B, int H, int N, int d, int block_q, int block_k, float scale,
                                 const float* tau_override, const uint8_t* forced_blocks, uint32_t* mask,
                                 sol_stream_t stream);

/* Fully explicit variant: nothing is taken from the bound state. */
typedef struct {
  const void* q; const void* k; const void* v;  /* device, bf16 [B,H,N,d]                       */
  void*       out;                              /* device, bf16 [B,H,N,d]                       */
  int32_t B, H, N, d, block_q, block_k;
  float   threshold;                            /* beta (ignored in SOL_MODE_DENSE)             */
  float   scale;                                /* logit scale; <= 0 selects 1/sqrt(d)          */
  int32_t mode;                                 /* SOL_MODE_*                                   */
  int32_t impl;                                 /* SOL_IMPL_*                                   */
  int32_t skip_pool;                            /* 1: reuse the workspace filled by a previous
                                                   sol_attn_pool / forward of the same q, k, v  */
  const float* tau_override;                    /* device fp32 [B,H,Nq] raw thresholds replacing
                                                   mu + beta*sigma (Algorithm 1's own `tau`
                                                   argument), or NULL                           */
  void*   workspace; size_t workspace_bytes;    /* device scratch, 1024-byte aligned            */
  int32_t* counts;                              /* device int32 [B,H,Nq] or NULL                */
  uint32_t* mask_out;                           /* debug: device bitmask [B,H,Nq,ceil(Nk/32)],
                                                   bit j%32 of word j/32 set when block j is in
                                                   S_i; NULL in production (the proxy map is
                                                   never written to memory otherwise); with
                                                   SOL_ROUTING_PREPASS: required, written by the
                                                   pre-pass and read by the fused kernel        */
  sol_stream_t stream;
  int32_t estimator;                            /* SOL_EST_* (0 = Eq. 5 moments)                */
  const uint8_t* forced_blocks;                 /* device uint8 [ceil(N/block_k)] or NULL: key
                                                   blocks with a nonzero entry are always routed
                                                   to the exact branch, whatever their proxy score
                                                   (text / sink key-value tokens kept exact, as in
                                                   the paper's MMDiT integrations); shared by all
                                                   batches and heads; counts include them         */
  int32_t layout;                               /* SOL_LAYOUT_* of q, k, v and out (0 = [B,H,N,d]) */
  int32_t routing;                              /* SOL_ROUTING_* (0 = inside the fused kernel)   */
} sol_attn_args;
/* Everything sol_attn_forward_ex enqueues is ordinary work on `stream` (a memset of the status words
 * and kernels), so the call may be captured into a CUDA graph and replayed; sol_attn_forward_host may
 * not (it creates events and uses streams of its own). */
sol_status_t sol_attn_forward_ex(const sol_attn_args* args /* host */);

/* End-to-end convenience for callers whose tensors live in HOST memory ([B,H,N,d] layout;
 * pinned memory makes the copies asynchronous).  Heads are independent, so the call is cut into
 * groups of heads (about 64 MB per tensor) and pipelined: the kernels of one group run on
 * `stream` while the next group's q, k, v are copied into the caller's device staging buffers
 * dq, dk, dv and the previous group's part of dout is copied to hout.  The copies use two streams
 * that the library creates on first use (per device, kept until the process ends); `stream` is
 * made to wait for the last copy back, so work queued on it afterwards sees hout complete.
 * Uses the bound workspace and counts.  Does not synchronise the host.  The environment variable
 * SOL_ATTN_HOST_GROUP_BYTES, when set to a positive number, replaces the 64 MB group size. */
sol_status_t sol_attn_forward_host(const void* hq, const void* hk, const void* hv, void* hout,
                                   void* dq, void* dk, void* dv, void* dout,
                                   int B, int H, int N, int d, int block_q, int block_k,
                                   float threshold, sol_stream_t stream);

/* Synchronises `stream`, then returns the device status word of the bound workspace
 * (SOL_OK, or SOL_ERR_DEVICE_TIMEOUT when a kernel gave up on a bounded wait) and clears it. */
sol_status_t sol_attn_read_device_status(sol_stream_t stream);

/* Threshold step for callers that cannot allocate device memory.  (The paper has no counterpart:
 * this is an interface variant, it computes the same mu, sigma, tau of Eq. 4 / Eq. 5.)
 *
 * Who needs it: code that is handed only its inputs and outputs -- an operator running inside
 * another framework's memory pool, a process whose device memory was reserved up front, a
 * serving loop in which an allocation would synchronise the device.  Such callers cannot provide
 * the workspace the other entry points keep the pooled-key moments in, so here the moments live
 * in a fixed array inside the library image: 4 MiB of device memory on every GPU that has made its
 * first call (see below), held until the process exits.
 *
 *   qbar   device fp32 [B,H,Nq,d]  mean of each query block (as produced by sol_attn_pool)
 *   kc     device fp32 [B,H,Nk,d]  mean of each key block
 *   mu, sigma, tau   device fp32 [B,H,Nq] outputs, owned by the caller
 *   scale  logit scale, <= 0 selects 1/sqrt(d);  threshold = beta
 *
 * Limit: B*H*d*(d+1) <= sol_attn_thresholds_static_max_floats() (2^20), i.e. B*H <= 63 for d = 128
 * and B*H <= 252 for d = 64; larger problems return SOL_ERR_SCRATCH_LIMIT and launch nothing.  A NaN
 * threshold or a NaN or infinite scale is SOL_ERR_INVALID_ARG, a device that is not compute capability
 * 10.x SOL_ERR_UNSUPPORTED_ARCH, both before anything is launched.
 * The FIRST call on each device is a set-up call: it makes the CUDA runtime load the part of the library
 * that holds the array -- which is when the 4 MiB are reserved on that device and can, like any module
 * load, fail (SOL_ERR_STATIC_SCRATCH) or synchronise -- and looks up the array's device address.  Make
 * that first call at start-up, before the process reserves its memory and outside any stream capture.
 * Every later call allocates and frees nothing, enqueues three kernels on `stream` and returns.  The
 * address is kept for the life of the process; after a cudaDeviceReset() the library has to be reloaded.
 * All calls on a device share the one array and every call overwrites the part it uses before
 * reading it, so nothing needs clearing between calls -- but two calls that overlap on the GPU
 * (different streams, no ordering) race on it and must be serialised by the caller. */
sol_status_t sol_attn_thresholds_static(const float* qbar, const float* kc, int B, int H, int Nq, int Nk,
                                        int d, float scale, float threshold,
                                        float* mu, float* sigma, float* tau, sol_stream_t stream);
size_t sol_attn_thresholds_static_max_floats(void);

/* Materialised routing baselines: the two policies the paper compares its on-the-fly thresholding
 * with (introduction, limitation L1; routing-latency figure).  The block proxy map of Eq. (3),
 * s_ij = scale * Qbar_i . KC_j, is written to `proxy_map`, every row is read back and sorted, and
 *   SOL_ROUTE_TOPK: the `param` (a block count, truncated to an integer, clamped to [0, Nk])
 *                   highest-scoring key blocks of every query block are kept;
 *   SOL_ROUTE_TOPP: blocks are kept in order of descending score until their share of the row's
 *                   softmax mass, softmax_j(s_ij), reaches `param` = p in [0, 1].
 * Equal scores are ordered by block index.
 *
 *   qbar, kc    device fp32 [B,H,Nq,d], [B,H,Nk,d]: pooled queries / keys (sol_attn_pool)
 *   proxy_map   device fp32 [B,H,Nq,Nk], out: the materialised map (caller-owned, required)
 *   order       device int32 [B,H,Nq,Nk] or NULL, out: block indices of each row by descending
 *               score (the routing indices; the first counts[i] of them are the kept blocks)
 *   tau         device fp32 [B,H,Nq], out: a cutoff equivalent to the selection -- the midpoint
 *               between the last kept and the first dropped score (+inf: none kept, -inf: all) --
 *               which sol_attn_forward_ex accepts as `tau_override`, so either policy can drive
 *               the fused kernel
 *   counts      device int32 [B,H,Nq] or NULL, out: kept blocks per query block
 *
 * Limits: Nk <= 8192 (a row is sorted in shared memory), d a multiple of 32; beyond them
 * SOL_ERR_UNSUPPORTED_SHAPE and nothing is launched.  Allocates nothing; two kernels on `stream`. */
enum { SOL_ROUTE_TOPK = 0, SOL_ROUTE_TOPP = 1 };
sol_status_t sol_attn_route_materialized(const float* qbar, const float* kc, int B, int H, int Nq, int Nk,
                                         int d, float scale, int policy, float param, float* proxy_map,
                                         int32_t* order, float* tau, int32_t* counts, sol_stream_t stream);

/* Number of kernels the library has launched since it was loaded (for launch accounting). */
int64_t sol_attn_launch_count(void);

/* Testing hook for the device-side failure path (the paper has no counterpart).  Every wait inside the
 * tcgen05 kernel is bounded; this call sets, for all later launches of the process, the bound in SM
 * clocks (wait_cycles <= 0 restores the default of about two seconds) and the index of one tile per CTA
 * whose "value GEMM finished" signal is left out (withhold_tile < 0: none).  With a tile withheld the
 * waits on that signal run out, every warp role drains, TMEM is released, the kernel returns and
 * sol_attn_read_device_status() reports SOL_ERR_DEVICE_TIMEOUT; the outputs of that launch are invalid.
 * Nothing faults, traps or spins without a bound.  Not for production use; not thread-safe. */
void sol_attn_debug_set_wait(int64_t wait_cycles, int32_t withhold_tile);

#ifdef __cplusplus
}
#endif
#endif  /* SOL_ATTN_H_ */
